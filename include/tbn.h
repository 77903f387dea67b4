/*
 * libtbn -- inference forward of Tiled Bit Network layers on NVIDIA B200 (sm_100a).
 *
 * A tiled layer (Tiled Bit Networks, Sec. 3) stores ONE binary tile t of q = N/k
 * bits plus one scaling factor alpha per layer (Eq. 6) or per tile (Eq. 7-8).  The
 * layer's N-element weight tensor is the tile repeated k times, reshaped in
 * row-major order (Eq. 4-5), each repetition scaled by its alpha:
 *
 *     B_hat[f] = alpha[f / q] * (bit(t, f % q) ? +1 : -1),   f = row-major flat index
 *
 * (k here is the paper's compression factor p.)  The library never materialises
 * B_hat in device memory except in tbn_expand_tile, which exists for testing.
 *
 * General conventions
 *   - Every pointer is a DEVICE pointer unless its name ends in _host or the
 *     comment says "host".  The caller owns every buffer; the library allocates
 *     no device memory, keeps no reference after the call returns and frees nothing.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *     All work is enqueued on it and the call returns without synchronising,
 *     except the *_host entry points, which synchronise the stream before returning.
 *   - Base pointers must be 16-byte aligned.  Matrices are dense row-major with no
 *     row padding.
 *   - Return value: a tbn_status.  Argument errors are detected on the host before
 *     anything is launched.  No entry point throws, aborts or exits.
 *   - Same inputs give the same bits out on every call (no order-dependent atomics).
 *   - Packed tile format: bit i of the tile is bit (i % 32) of 32-bit word (i / 32),
 *     least-significant bit first; 1 encodes +1, 0 encodes -1.  A packed tile
 *     occupies tbn_tile_words(q) words (a multiple of 4, i.e. of 128 bits); the
 *     padding bits are zero.
 */
#ifndef TBN_H_
#define TBN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    TBN_OK = 0,
    TBN_ERR_INVALID_ARG = -1, /* null pointer, negative size, unknown enum value, misaligned pointer */
    TBN_ERR_SHAPE = -2,       /* k does not divide N (Sec. 3 requires k*q = N), or sizes inconsistent */
    TBN_ERR_UNSUPPORTED = -3, /* a combination the library does not implement */
    TBN_ERR_WORKSPACE = -4,   /* workspace missing or smaller than the matching *_workspace_bytes() */
    TBN_ERR_CUDA = -5,        /* a CUDA runtime / driver call failed */
    TBN_ERR_TIMEOUT = -6      /* a device-side bounded wait gave up (see tbn_last_device_status) */
} tbn_status;

typedef enum { TBN_F32 = 0, TBN_BF16 = 1, TBN_I32 = 2 /* only as y_dtype of tbn_linear_bin_fwd */ } tbn_dtype;
typedef enum { TBN_ALPHA_PER_LAYER = 0, TBN_ALPHA_PER_TILE = 1 } tbn_alpha_mode; /* 1 or k floats */
/* GELU is the erf form v * Phi(v): evaluated to 4e-7 for fp32 outputs; bf16 outputs of the tensor-core kernels use a
 * tanh form fitted to it whose difference (<= 2.5e-5 + 2.5e-4 |v|) stays below the bf16 rounding of the result. */
typedef enum { TBN_ACT_NONE = 0, TBN_ACT_RELU = 1, TBN_ACT_GELU = 2 } tbn_act;

/* Which kernel family executes a forward call.  AUTO picks by shape. */
typedef enum {
    TBN_PATH_AUTO = 0,
    TBN_PATH_GENERIC = 1, /* CUDA-core kernel; any shape and any alignment of q against the row length */
    TBN_PATH_SMALL = 2,   /* small-batch kernel; needs q % in_features == 0 */
    TBN_PATH_TENSOR = 3   /* tcgen05 / TMEM kernel; needs q % in_features == 0 and in_features % 8 == 0 */
} tbn_path;

/* ceil(q/32) rounded up to a multiple of 4: the number of uint32 words of a packed tile. */
int64_t tbn_tile_words(int64_t q);

const char *tbn_status_string(int status);

/* ------------------------------------------------------------------------------------------------
 * Tile construction (Sec. 3, Eq. 1-3 and Eq. 6-8).
 *
 *   s_i     = sum_{j<k} W[j*q + i]      fp32, added sequentially in increasing j     (Eq. 1-2)
 *   bit_i   = (s_i > 0)                 zero, negative zero and NaN give 0 (= -1)    (Eq. 3)
 *   alpha   = ||S||_1 / N               per layer                                    (Eq. 6)
 *   alpha_j = ||S[j*q, (j+1)*q)||_1 / q per tile, j < k                              (Eq. 7-8)
 * where S = A when A is not NULL (the paper's separate tensor for alpha), else W.
 *
 * W, A      : N fp32 values, the layer's weight tensor in row-major order.
 * tile_bits : out, tbn_tile_words(N/k) words.
 * alpha     : out, 1 float (per layer) or k floats (per tile).
 * workspace : scratch of at least tbn_aggregate_workspace_bytes(N, k) bytes; contents undefined after.
 * Errors    : N % k != 0 -> TBN_ERR_SHAPE; N == 0 is TBN_ERR_INVALID_ARG.
 * The bits equal the CPU definition exactly.  For alpha a thread adds the |.| of at most 16 values of one
 * tile repetition in fp32, everything above that (per thread, per block, across blocks) is added in fp64
 * in a fixed order, so alpha is reproducible from run to run and within 1e-6 of an fp64 sum.
 */
size_t tbn_aggregate_workspace_bytes(int64_t N, int32_t k);
int tbn_aggregate_tile(const float *W, const float *A, int64_t N, int32_t k, int alpha_mode,
                       uint32_t *tile_bits, float *alpha, void *workspace, size_t workspace_bytes,
                       void *stream);

/* Variant of tbn_aggregate_tile for callers that cannot provide scratch memory.  (The paper has no
 * counterpart: this is a convenience of this library.)  Some callers run where device allocation is not
 * an option -- inside a latency-critical serving loop that must never hit the allocator, in a plug-in that
 * is handed its input and output buffers and nothing else, or under a memory manager that forbids
 * cudaMalloc after start-up.  For them the scratch lives in an array built into the library: 1 MiB per GPU
 * that loads the library, held until the process exits.  The call allocates nothing and calls no
 * allocating routine.
 *   Limit : tbn_aggregate_workspace_bytes(N, k) must not exceed 1 MiB (N up to about 500 million weights);
 *           larger layers are refused with TBN_ERR_WORKSPACE before anything is launched.
 *   Set-up: the first call on a device looks up the array's device address.  Make that first call with
 *           the device current and before any stream capture begins.  The look-up is not synchronised:
 *           threads that might make the first call on a device at the same time must take turns.
 *   Sharing: every call on a device uses the same array.  The call clears the part that must start at
 *           zero, so calls that follow one another on a stream are fine; calls that may overlap on the GPU
 *           (different streams, no ordering between them) race on the array and must be serialised by the
 *           caller.
 * Arguments, results and the remaining errors are those of tbn_aggregate_tile without the workspace pair. */
int tbn_aggregate_tile_static(const float *W, const float *A, int64_t N, int32_t k, int alpha_mode,
                              uint32_t *tile_bits, float *alpha, void *stream);

/* ------------------------------------------------------------------------------------------------
 * Training-side tiling module (Sec. 3).  The paper trains full-precision W (and optionally A), builds the tiled
 * weight in the forward pass of a custom differentiation module (Eq. 1-5), and passes the gradient straight
 * through the non-differentiable steps on the way back (the paragraph after Eq. 5: dL/dW := dL/dB).
 *
 * tbn_tile_fwd: one read of W (and A) -> tile_bits and alpha exactly as tbn_aggregate_tile, and
 *     B_hat[j*q + i] = alpha_j * (bit_i ? +1 : -1)        N values, fp32 or bf16 (b_dtype), row-major like W:
 *   the weight the training forward then contracts with the inputs.  B_hat is written from the bits; W is not
 *   read a second time.  workspace: tbn_aggregate_workspace_bytes(N, k).
 * tbn_tile_bwd: G = dL/dB_hat (N fp32 values) ->
 *     dalpha_j = sum_i G[j*q + i] * t_i                   (per layer: one sum over all N; fp64, fixed order)
 *     dW[f]    = alpha_j * G[f]                           the straight-through part, one fp32 multiply
 *     dS[f]    = dalpha_j * sign(S[f]) / q                the scaling factors are differentiated as ordinary
 *                                                         functions of S (Eq. 6-8; sign(0) = 0; / N per layer)
 *   With a separate tensor (A != NULL) dS is written to dA; without one (A == NULL, dA == NULL) S = W and dS is
 *   added to dW.  dalpha (1 or k floats) may be NULL.  The paper states the straight-through rule only; taking the
 *   gradient of the scaling factors as well is this library's reading (it is what automatic differentiation of
 *   Eq. 6-8 gives).  workspace: tbn_tile_bwd_workspace_bytes(N, k).  Errors as tbn_aggregate_tile.
 */
int tbn_tile_fwd(const float *W, const float *A, int64_t N, int32_t k, int alpha_mode, void *B_hat, int b_dtype,
                 uint32_t *tile_bits, float *alpha, void *workspace, size_t workspace_bytes, void *stream);
size_t tbn_tile_bwd_workspace_bytes(int64_t N, int32_t k);
int tbn_tile_bwd(const float *G, const uint32_t *tile_bits, const float *alpha, const float *W, const float *A,
                 int64_t N, int32_t k, int alpha_mode, float *dW, float *dA, float *dalpha,
                 void *workspace, size_t workspace_bytes, void *stream);

/* Pack an existing real-valued tile (Sec. 5.1: tiles are stored one bit per element):
 * src[i] > 0 -> bit 1, else 0.  src: q fp32 values.  tile_bits: tbn_tile_words(q) words. */
int tbn_pack_tile(const float *src, int64_t q, uint32_t *tile_bits, void *stream);

/* Testing aid, not on the hot path: write B_hat (Eq. 4-5 plus the alpha scaling) as N fp32 values. */
int tbn_expand_tile(const uint32_t *tile_bits, int64_t N, int32_t k, const float *alpha, int alpha_mode,
                    float *B_hat, void *stream);

/* ------------------------------------------------------------------------------------------------
 * Fully-connected forward (Sec. 3, the paragraph after Eq. 8: the scaled tensor B_hat is what meets the
 * inputs; Algorithm 1):
 *
 *     y[t][o] = act( sum_j B_hat[o][j] * x[t][j] + bias[o] ),   B_hat is out_f x in_f (row-major)
 *
 * x    : T x in_f, fp32 or bf16 (x_dtype).      y : T x out_f, fp32 or bf16 (y_dtype).
 * tile_bits, k, alpha, alpha_mode: as produced by tbn_aggregate_tile with N = out_f*in_f.
 * alpha values must be non-negative, as the means of absolute values of Eq. 6-8 always are: the tensor-core
 * kernels and the compact MLP chain use relu(alpha * z) = alpha * relu(z).  (The same holds for
 * tbn_conv2d_fwd and tbn_mlp_fwd.)
 * bias : out_f fp32 values or NULL (the paper uses none).
 * Products are accumulated in fp32.  On the TENSOR path fp32 activations are rounded to bf16 first
 * (into the workspace); the other paths use them as given.
 * Where the tile spans whole rows (q % in_f == 0) only the q/in_f distinct rows are contracted and the
 * result is written k times, each copy scaled by its alpha (Sec. 4.1, replicated channels).
 * workspace: at least tbn_linear_workspace_bytes(...) bytes (may be NULL when that is 0).
 * T == 0 is a successful no-op.
 */
size_t tbn_linear_workspace_bytes(int64_t T, int32_t in_f, int32_t out_f, int32_t k, int x_dtype);
int tbn_linear_fwd(const void *x, int x_dtype, int64_t T, int32_t in_f, int32_t out_f,
                   const uint32_t *tile_bits, int32_t k, const float *alpha, int alpha_mode,
                   const float *bias, int act, void *y, int y_dtype,
                   void *workspace, size_t workspace_bytes, void *stream);
/* Same, with the kernel family forced (TBN_ERR_UNSUPPORTED if the shape does not qualify). */
int tbn_linear_fwd_path(const void *x, int x_dtype, int64_t T, int32_t in_f, int32_t out_f,
                        const uint32_t *tile_bits, int32_t k, const float *alpha, int alpha_mode,
                        const float *bias, int act, void *y, int y_dtype,
                        void *workspace, size_t workspace_bytes, void *stream, int path);
/* The family TBN_PATH_AUTO resolves to for this shape (a tbn_path), or a negative tbn_status. */
int tbn_linear_select_path(int64_t T, int32_t in_f, int32_t out_f, int32_t k, int x_dtype);

/* Same layer with a residual input: y = act(...) + residual, where residual is a tensor shaped and typed like y (NULL:
 * exactly tbn_linear_fwd_path).  The residual connections of a Transformer block around the tiled projection and
 * feed-forward layers (Sec. 4.3) are the use; the paper itself writes no formula for it.  residual must not be y.
 * The CUDA-core kernels add it in their epilogue; after the tensor-core kernel it is added by a pass of its own. */
int tbn_linear_res_fwd(const void *x, int x_dtype, int64_t T, int32_t in_f, int32_t out_f,
                       const uint32_t *tile_bits, int32_t k, const float *alpha, int alpha_mode,
                       const float *bias, int act, const void *residual, void *y, int y_dtype,
                       void *workspace, size_t workspace_bytes, void *stream, int path);

/* Compact chaining of two tiled layers through any activation (Sec. 4.1: with a tile that spans whole rows the k
 * repetitions of an output channel are the same pre-activation z scaled by different alphas).  The first layer writes
 * only its r_z distinct pre-activations -- call tbn_linear_fwd with out_f = r_z, k = 1 and an alpha of 1.0 on the same
 * tile (a tile of r_z rows IS a k = 1 layer of r_z outputs) -- and this call consumes them:
 *
 *     x[t][j*r_z + c] = act_z(alpha_z[j] * z[t][c])        j < k_z, c < r_z     (never written to memory)
 *     y[t][o]         = act( sum_i B_hat[o][i] * x[t][i] + bias[o] )             B_hat: out_f x (r_z * k_z), tiled
 *
 * The activation of the first layer is evaluated while the activation operand is staged on chip, so the k_z-fold
 * larger tensor x is neither written by the first layer nor read by the second.  (With ReLU or no activation
 * tbn_mlp_fwd gets the same saving by folding alpha_z into the weights; this call is what covers GELU.)
 * z: T x r_z bf16.  alpha_z: 1 or k_z floats (alpha_mode_z), k_z <= 64.  Needs r_z % 64 == 0 and a tile that spans
 * whole rows (q % (r_z*k_z) == 0); TBN_ERR_UNSUPPORTED otherwise.  Tensor-core kernel; no workspace.  Other arguments as
 * tbn_linear_fwd. */
int tbn_linear_compact_fwd(const void *z, int64_t T, int32_t rz, int32_t kz, const float *alpha_z, int alpha_mode_z, int act_z,
                           int32_t out_f, const uint32_t *tile_bits, int32_t k, const float *alpha, int alpha_mode,
                           const float *bias, int act, void *y, int y_dtype, void *stream);

/*
 * Full-precision tiled weights (Sec. 5.2: the "FP, Tiled" kernel measured in Table 7 and Fig. 6; named as future
 * work for large models in Sec. 7).  The layer stores a tile of q = in_f*out_f/k REAL values; the weight matrix is
 * the tile repeated k times and reshaped row-major exactly as in Eq. 4-5, with no threshold and no scaling factor:
 *     y[t][i] = act( sum_j tile[(i*in_f + j) mod q] * x[t][j] + bias[i] ).
 * tile_values: device, q elements of tile_dtype (TBN_F32 or TBN_BF16), 16-byte aligned, never written.
 * When the tile spans whole rows (q % in_f == 0, in_f % 8 == 0) its q/in_f rows feed the tensor-core kernel
 * directly as the weight operand (an fp32 tile is first rounded to bf16 into the workspace; a bf16 tile is read in
 * place) and every row is written k times; other shapes run on the index-walk kernel with the tile's own precision.
 * Rounding an fp32 tile to bf16 costs a relative weight error of 2^-9, i.e. about 1e-3 of the output's scale;
 * TBN_PATH_GENERIC keeps fp32 weights exactly.
 * path: TBN_PATH_AUTO, TBN_PATH_GENERIC or TBN_PATH_TENSOR (TBN_PATH_SMALL decodes bits: TBN_ERR_UNSUPPORTED).
 * workspace: tbn_linear_fp_tile_workspace_bytes(...) bytes.  Other arguments, ownership and errors as tbn_linear_fwd.
 */
size_t tbn_linear_fp_tile_workspace_bytes(int64_t T, int32_t in_f, int32_t out_f, int32_t k, int x_dtype,
                                          int tile_dtype);
int tbn_linear_fp_tile_fwd(const void *x, int x_dtype, int64_t T, int32_t in_f, int32_t out_f,
                           const void *tile_values, int tile_dtype, int32_t k,
                           const float *bias, int act, void *y, int y_dtype,
                           void *workspace, size_t workspace_bytes, void *stream, int path);

/* Same layer with HOST activations: x_host and y_host are host buffers (pinned memory recommended; with
 * pageable memory the copies do not overlap anything).
 * The call copies x to the device, runs tbn_linear_fwd, copies y back and synchronises `stream`; it returns
 * when y_host is complete.  Token rows are independent (Algorithm 1 treats one input vector at a time), so a
 * batch whose transfers exceed about 32 MiB goes through in up to 32 chunks of whole token rows: while one
 * chunk is computed on `stream`, the next is copied in and the previous one copied out on two copy streams
 * that the library creates once per device at the first such call (no device memory is allocated; calls on
 * one device take turns on these streams).  Work queued on `stream` before the call is waited for first.
 * workspace (device) must hold tbn_linear_host_workspace_bytes(...) bytes: staging for x and y plus
 * the forward's own scratch.  tile_bits, alpha and bias stay device pointers (model state). */
size_t tbn_linear_host_workspace_bytes(int64_t T, int32_t in_f, int32_t out_f, int32_t k,
                                       int x_dtype, int y_dtype);
int tbn_linear_fwd_host(const void *x_host, int x_dtype, int64_t T, int32_t in_f, int32_t out_f,
                        const uint32_t *tile_bits, int32_t k, const float *alpha, int alpha_mode,
                        const float *bias, int act, void *y_host, int y_dtype,
                        void *workspace, size_t workspace_bytes, void *stream);

/* ------------------------------------------------------------------------------------------------
 * Binary activations (Sec. 7 names tiled networks with binary weights AND binary activations as the next step;
 * Sec. 2 describes such networks: sign activations with a real scaling factor, contracted by XNOR and
 * popcount).  The paper gives no formula for this case; this library takes the smallest extension of Sec. 3:
 *
 *     a[t][j] = x[t][j] > 0 ? +1 : -1             the threshold rule of Eq. 3 (zero, -0 and NaN give -1)
 *     beta[t] = ||x[t][:]||_1 / in_f              the scale of Eq. 6 applied to one input row
 *     D[t][o] = sum_j b[o][j] * a[t][j]           b = the unscaled +-1 tiled weight of Eq. 4-5; an integer
 *     y[t][o] = act( beta[t] * sum_j B_hat[o][j] * a[t][j] + bias[o] )
 *
 * (where the tile spans whole rows: y[t][j*r + c] = act(beta[t] * alpha_j * D[t][c] + bias), D contracted once per
 * distinct row and written k times, Sec. 4.1).  D is computed exactly: D = cnt - 2 popcount(w xor x) on the
 * CUDA-core path, 4 popcount(w and x) - 2 popcount(w) - 2 popcount(x) + in_f with the and-popcount as an 8-bit
 * integer tensor-core product on the tensor path.
 *
 * tbn_binarize_fwd: x (T x in_f, fp32 or bf16) -> x_bits: T rows of tbn_row_words(in_f) words each (row pitch a
 *   multiple of 128 bits; bit j of a row at word j/32, position j%32; padding bits zero), and beta (T floats; may be
 *   NULL when the caller wants no scale).  beta is accumulated in fp64 in a fixed order.
 * tbn_linear_bin_fwd: x_bits as written by tbn_binarize_fwd; beta: T floats or NULL (= 1; must be >= 0, like alpha);
 *   tile_bits, k, alpha, alpha_mode, bias, act as for tbn_linear_fwd.  y: T x out_f; y_dtype TBN_F32 or TBN_BF16,
 *   or TBN_I32 for the raw integers D (alpha, beta, bias and act are then not applied).
 *   path: TBN_PATH_AUTO; TBN_PATH_GENERIC = the popcount kernel (any shape, any alignment of the tile against the rows;
 *   one packed activation row must fit 48 KB); TBN_PATH_TENSOR = the integer tensor-core kernel (needs
 *   q % in_f == 0 and in_f % 32 == 0; TBN_ERR_UNSUPPORTED otherwise).  No workspace.  T == 0 is a no-op.
 * tbn_bin_expand_fwd / tbn_linear_bin_bytes_fwd: the tensor path with the activation signs held as bytes, which a
 *   layer's activations are expanded to ONCE (instead of on chip by every row block of the layer): x_bytes is T rows of
 *   in_f bytes, 0x00 for -1 and 0xFF for +1, and byte 4 s + j (s < 8, j < 4) of every group of 32 elements holds element
 *   8 j + 7 - s of the group (the order in which the kernel expands the weight bits; any order works as long as both
 *   operands share it); x_pop is T int32 values, the number of +1 elements of each row.  Both are written by
 *   tbn_bin_expand_fwd from x_bits.  in_f % 32 == 0 (TBN_ERR_UNSUPPORTED otherwise); x_bytes 16-byte aligned.
 *   tbn_linear_bin_bytes_fwd has otherwise the arguments and results of tbn_linear_bin_fwd on TBN_PATH_TENSOR: the
 *   integers D are identical.
 * tbn_binarize_bytes_fwd: tbn_binarize_fwd and tbn_bin_expand_fwd in one pass over x (x_bits, beta, x_bytes and x_pop as
 *   above, bit for bit the same; in_f % 32 == 0).
 */
int64_t tbn_row_words(int32_t in_f);
int tbn_binarize_fwd(const void *x, int x_dtype, int64_t T, int32_t in_f, uint32_t *x_bits, float *beta, void *stream);
int tbn_linear_bin_fwd(const uint32_t *x_bits, int64_t T, int32_t in_f, int32_t out_f,
                       const uint32_t *tile_bits, int32_t k, const float *alpha, int alpha_mode,
                       const float *beta, const float *bias, int act, void *y, int y_dtype, void *stream, int path);
int tbn_bin_expand_fwd(const uint32_t *x_bits, int64_t T, int32_t in_f, void *x_bytes, int32_t *x_pop, void *stream);
int tbn_binarize_bytes_fwd(const void *x, int x_dtype, int64_t T, int32_t in_f, uint32_t *x_bits, float *beta, void *x_bytes,
                           int32_t *x_pop, void *stream);
int tbn_linear_bin_bytes_fwd(const void *x_bytes, const int32_t *x_pop, int64_t T, int32_t in_f, int32_t out_f,
                             const uint32_t *tile_bits, int32_t k, const float *alpha, int alpha_mode,
                             const float *beta, const float *bias, int act, void *y, int y_dtype, void *stream);

/* ------------------------------------------------------------------------------------------------
 * 2-D convolution forward.  The paper defines tiling for convolutional layers (Sec. 3: the tile
 * fills the whole weight tensor) but ships no convolution kernel (Sec. 6 lists it as future work).
 * The weight tensor is (Cout, Cin, kh, kw) in row-major order, N = Cout*Cin*kh*kw:
 *
 *   y[b][co][oh][ow] = act( sum_{ci,u,v} B_hat[co][ci][u][v] * x[b][ci][oh*stride+u-pad][ow*stride+v-pad]
 *                           + bias[co] )
 *
 * Cross-correlation (no kernel flip), zero padding, same stride and padding in both directions,
 * dilation 1, one group.  x: NCHW (Nb, Cin, H, Wd).  y: NCHW (Nb, Cout, Ho, Wo) with
 * Ho = (H + 2*pad - kh)/stride + 1, Wo likewise.  Where the tile spans whole filters
 * (q % (Cin*kh*kw) == 0) each distinct filter is applied once and its output channel is written k
 * times with the k alphas (Sec. 4.1).
 */
size_t tbn_conv2d_workspace_bytes(int32_t Nb, int32_t Cin, int32_t H, int32_t Wd, int32_t Cout,
                                  int32_t kh, int32_t kw, int32_t stride, int32_t pad, int32_t k,
                                  int x_dtype);
int tbn_conv2d_fwd(const void *x, int x_dtype, int32_t Nb, int32_t Cin, int32_t H, int32_t Wd,
                   int32_t Cout, int32_t kh, int32_t kw, int32_t stride, int32_t pad,
                   const uint32_t *tile_bits, int32_t k, const float *alpha, int alpha_mode,
                   const float *bias, int act, void *y, int y_dtype,
                   void *workspace, size_t workspace_bytes, void *stream);
int tbn_conv2d_fwd_path(const void *x, int x_dtype, int32_t Nb, int32_t Cin, int32_t H, int32_t Wd,
                        int32_t Cout, int32_t kh, int32_t kw, int32_t stride, int32_t pad,
                        const uint32_t *tile_bits, int32_t k, const float *alpha, int alpha_mode,
                        const float *bias, int act, void *y, int y_dtype,
                        void *workspace, size_t workspace_bytes, void *stream, int path);

/* The full-precision ends of a convolution stack.  Layers below the size threshold of Sec. 3 (hyperparameter lambda)
 * are not tiled: in a ResNet-style stack the first convolution and the classifier stay full precision.
 * tbn_conv2d_dense_fwd: the convolution above with an explicit fp32 weight (Cout, Cin, kh, kw) instead of a tile, for
 *   short contractions (Cin*kh*kw <= 512; TBN_ERR_UNSUPPORTED beyond); x, y NCHW, fp32 or bf16; bias Cout floats or NULL.
 * tbn_global_avgpool_fwd: y[b][c] = mean over the H*Wd positions of x[b][c]; x NCHW, y (Nb, C); fp32 accumulation.
 * tbn_avgpool_linear_fwd: the pooling above followed by a full-precision classifier in one launch:
 *   y[b][o] = sum_c weight[o][c] * mean(x[b][c]) + bias[o]; weight (out_f, C) fp32 row-major, bias out_f floats or NULL,
 *   y (Nb, out_f) fp32; C <= 4096 (TBN_ERR_UNSUPPORTED beyond).
 * (A full-precision classifier on its own is tbn_linear_fp_tile_fwd with k = 1.)  None of these is defined by the paper;
 * they are ordinary layers that the stack needs to run end to end. */
int tbn_conv2d_dense_fwd(const void *x, int x_dtype, int32_t Nb, int32_t Cin, int32_t H, int32_t Wd, int32_t Cout, int32_t kh,
                         int32_t kw, int32_t stride, int32_t pad, const float *weight, const float *bias, int act, void *y,
                         int y_dtype, void *stream);
int tbn_global_avgpool_fwd(const void *x, int x_dtype, int32_t Nb, int32_t C, int32_t H, int32_t Wd, void *y, int y_dtype,
                           void *stream);
int tbn_avgpool_linear_fwd(const void *x, int x_dtype, int32_t Nb, int32_t C, int32_t H, int32_t Wd, const float *weight,
                           const float *bias, int32_t out_f, float *y, void *stream);

/* ------------------------------------------------------------------------------------------------
 * Chain of L fully-connected tiled layers (Sec. 5.1: an MLP with a fused ReLU):
 *     h_0 = x;  h_{l+1} = hidden_act(layer_l(h_l)) for l < L-1;  y = layer_{L-1}(h_{L-1}).
 * dims (host, L+1 ints): dims[l] -> dims[l+1] is layer l.  ks, alpha_modes: host arrays of L values.
 * tiles, alphas: HOST arrays of L DEVICE pointers.  No biases.  x: T x dims[0];  y: T x dims[L].
 * Compact chain: when the hidden activation is ReLU or none, every layer's tile spans whole rows and the
 * numbers of distinct rows of the hidden layers are multiples of 8, a hidden layer writes only its distinct
 * columns g = act(Z) (bf16, T x r) to the workspace -- its k repetitions are alpha_j * g (Sec. 4.1; alpha >= 0
 * so relu(alpha z) = alpha relu(z)) -- and the next layer contracts g with its distinct rows folded with
 * those alphas, computed on the device at every call from the tiles and alphas: the k-fold broadcast never
 * goes to HBM and the next contraction is k times shorter.  Otherwise layers run one by one with full bf16
 * hidden tensors in the workspace.  Both give the layer-by-layer result up to bf16 rounding of the hidden
 * tensors / folded rows.
 * The folding kernels of the compact chain run on a side stream that the library creates once per device (at the
 * first call whose `stream` is not being captured into a graph; no device memory is allocated): they start after
 * the work already queued on `stream` and `stream` waits for them before the second layer, so the call keeps
 * stream semantics.  When the last layer has at most 16 distinct rows and the one before it at most 256 (a
 * multiple of 32, like its input width), the two run as one kernel.
 */
size_t tbn_mlp_workspace_bytes(int64_t T, int32_t L, const int32_t *dims, const int32_t *ks, int x_dtype);
int tbn_mlp_fwd(const void *x, int x_dtype, int64_t T, int32_t L, const int32_t *dims,
                const uint32_t *const *tiles, const int32_t *ks, const float *const *alphas,
                const int *alpha_modes, int hidden_act, void *y, int y_dtype,
                void *workspace, size_t workspace_bytes, void *stream);

/* ------------------------------------------------------------------------------------------------
 * Transformer encoder block with tiled linears (Sec. 4.3 trains Vision Transformers whose Q, K, V, projection and
 * feed-forward layers are tiled; Sec. 5.2 measures the kernel inside one).  The block is the standard pre-norm one:
 *
 *     x1 = x  + proj( attention( qkv( LN(x) ) ) )
 *     y  = x1 + fc2( gelu( fc1( LN(x1) ) ) )
 *
 * with the four linears tiled (no biases, as in the paper), LayerNorm without affine parameters (eps 1e-5), the erf
 * form of GELU and softmax(q k^T / sqrt(d_head)) v attention.  Everything but the four linears is ordinary glue that
 * the paper does not define; it is here so that the block runs end to end on the device.
 *
 * tbn_layernorm_fwd: y[t][:] = (x[t][:] - mean) / sqrt(var + eps) * gamma + beta over the d values of a row (biased
 *   variance, statistics in fp32); gamma, beta: d floats each or NULL.  x, y: T x d, fp32 or bf16.
 * tbn_attention_fwd: qkv: (Nb*S) x (3*heads*d_head) bf16, columns (q | k | v), head h at h*d_head inside each third;
 *   out: (Nb*S) x (heads*d_head) bf16.  bf16 operands, fp32 accumulation and softmax.  d_head must be 64 and
 *   S <= 208 (TBN_ERR_UNSUPPORTED otherwise).  Both pointers 16-byte aligned.
 * tbn_vit_block_fwd: x, y: (Nb*S) x d bf16.  tiles / ks / alphas / alpha_modes: HOST arrays of 4 entries in the order
 *   qkv (d -> 3d), proj (d -> d), fc1 (d -> mlp_dim), fc2 (mlp_dim -> d); tiles and alphas hold DEVICE pointers.
 *   workspace: tbn_vit_block_workspace_bytes(...) bytes (the block's intermediate tensors in bf16 plus the linears'
 *   scratch).  Seven launches on `stream`; intermediate tensors are stored as bf16.
 */
int tbn_layernorm_fwd(const void *x, int x_dtype, int64_t T, int32_t d, const float *gamma, const float *beta, float eps,
                      void *y, int y_dtype, void *stream);
int tbn_attention_fwd(const void *qkv, int32_t Nb, int32_t S, int32_t heads, int32_t d_head, void *out, void *stream);
size_t tbn_vit_block_workspace_bytes(int32_t Nb, int32_t S, int32_t d, int32_t mlp_dim, const int32_t *ks);
int tbn_vit_block_fwd(const void *x, int32_t Nb, int32_t S, int32_t d, int32_t heads, int32_t mlp_dim,
                      const uint32_t *const *tiles, const int32_t *ks, const float *const *alphas, const int *alpha_modes,
                      void *y, void *workspace, size_t workspace_bytes, void *stream);

/* ------------------------------------------------------------------------------------------------
 * Device-side status.  Kernels that wait on hardware barriers bound every wait; when a wait gives
 * up the kernel records TBN_ERR_TIMEOUT and a detail word (which barrier, which block), abandons
 * its remaining work and returns normally.  This call synchronises `stream`, reads the record of
 * the current device into *code / *detail (TBN_OK when nothing was recorded) and clears it.
 * Returns TBN_OK, or TBN_ERR_CUDA if the synchronisation or the copy failed.
 */
int tbn_last_device_status(void *stream, int *code, int *detail);
/* Testing aid: enqueue a kernel that records (code, detail) exactly as a kernel whose wait gave up would --
 * it waits on nothing, so it cannot hang -- to exercise the status plumbing without starving a real pipeline. */
int tbn_debug_record_status(int code, int detail, void *stream);
/* Testing aids for the bounded waits themselves.  tbn_debug_set_wait_limit_us sets the limit of every device-side
 * wait on the current device (microseconds; 0 restores the default of 2 s; the call synchronises the device first).
 * tbn_debug_wait_timeout_probe enqueues a one-block kernel whose threads wait, through the same bounded-wait routines
 * the tensor-core kernels use, on a barrier that nothing arrives at: the waits run out after the limit, the kernel
 * records TBN_ERR_TIMEOUT with `detail`, takes the abort path (one warp times out, another leaves through the block's
 * abort flag, then the quiet drain wait) and returns normally, so the context stays usable.  Set a short limit first:
 * with the default the probe takes 2 s. */
int tbn_debug_set_wait_limit_us(int limit_us);
int tbn_debug_wait_timeout_probe(int detail, void *stream);
/* Testing / tuning aids, process-wide, to be set while no forward call is in progress.  They replace nothing on
 * the normal path: without them the library chooses by shape.
 *   tbn_debug_force_linear_config: the tensor-core linear kernel runs tile shape `candidate` (an index into its
 *     table of shapes) with the contraction split over `splits` CTAs per output tile (1, 2, 4, 8 or 16; lowered
 *     at launch until every split has at least two stages; without enough workspace the call runs unsplit).
 *     candidate < 0 restores the automatic choice.  TBN_ERR_INVALID_ARG for anything else.
 *   tbn_debug_force_mlp_layerwise: non-zero makes tbn_mlp_fwd run layer by layer with full hidden tensors even
 *     where the compact chain applies (the two must agree; tests compare them). */
int tbn_debug_force_linear_config(int candidate, int splits);
int tbn_debug_force_mlp_layerwise(int on);
/* Same for the tile shape of the binary-activation tensor-core kernel (candidate < 0: automatic). */
int tbn_debug_force_bin_config(int candidate);
int tbn_debug_force_attention_path(int path); /* 0 automatic, 1 the warp-level MMA kernel, 2 the tcgen05 kernel; tests */

#ifdef __cplusplus
}
#endif
#endif /* TBN_H_ */
