// Shared declarations of the libtbn translation units (internal; the public surface is include/tbn.h).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "tbn.h"

namespace tbn {

// ---- scalar helpers ---------------------------------------------------------------------------
__device__ __forceinline__ float load_as_float(const float *p, int64_t i) { return p[i]; }
__device__ __forceinline__ float load_as_float(const __nv_bfloat16 *p, int64_t i) {
    return __bfloat162float(p[i]);
}
__device__ __forceinline__ void store_from_float(float *p, int64_t i, float v) { p[i] = v; }
__device__ __forceinline__ void store_from_float(__nv_bfloat16 *p, int64_t i, float v) {
    p[i] = __float2bfloat16_rn(v);
}

// GELU in its erf form, v * Phi(v) with Phi(v) = (1 + erf(v / sqrt 2)) / 2.  erfc(u), u >= 0, is evaluated branch-free
// with the rational approximation 7.1.26 of Abramowitz & Stegun (absolute error below 1.5e-7, i.e. fp32 round-off):
// erfc(u) = (a1 t + ... + a5 t^5) exp(-u^2), t = 1 / (1 + p u); Phi(v) = erfc(u)/2 for v < 0 and 1 - erfc(u)/2
// otherwise, so the negative tail keeps its relative accuracy.  About a dozen instructions, two of them on the
// special-function unit, against a divergent library erff: the activation runs in the epilogue warps of the
// tensor-core kernels, where it would otherwise cost several times the contraction itself.
__device__ __forceinline__ float gelu_erf(float v) {
    const float u = fabsf(v) * 0.70710678118654752440f;
    const float t = __fdividef(1.0f, fmaf(0.3275911f, u, 1.0f));
    float poly = fmaf(1.061405429f, t, -1.453152027f);
    poly = fmaf(poly, t, 1.421413741f);
    poly = fmaf(poly, t, -0.284496736f);
    poly = fmaf(poly, t, 0.254829592f);
    const float half_erfc = 0.5f * poly * t * __expf(-u * u);
    return v * (v < 0.0f ? half_erfc : 1.0f - half_erfc);
}

// GELU for outputs that are rounded to bf16 anyway: v * Phi(v) with Phi(v) = (1 + tanh(v (c0 + c1 v^2 + c2 v^4))) / 2,
// the constants fitted to the erf form above (largest difference 2.5e-5 over the reals; v^2 is capped at 50, beyond
// which tanh is 1 in fp32).  tanh comes from the special-function unit (tanh.approx.f32, relative error about
// 2^-11), so the result is within 2.5e-5 + 2.5e-4 |v| of the erf form -- an eighth of a bf16 ulp for v > 0, and an
// absolute 7e-4 at worst in the negative tail, where the erf form above keeps relative accuracy and this one does
// not.  Seven FMA-pipe instructions and one special-function instruction, against sixteen and two: the epilogue
// warps of a layer with k-fold replicated outputs evaluate the activation k times per accumulator element.
__device__ __forceinline__ float gelu_tanh_bf16(float v) {
    const float s = fminf(v * v, 50.0f);
    const float inner = fmaf(fmaf(-3.51516788e-4f, s, 3.70056460e-2f), s, 7.97507884e-1f);
    float th;
    asm("tanh.approx.f32 %0, %1;" : "=f"(th) : "f"(v * inner));
    const float hv = 0.5f * v;
    return fmaf(hv, th, hv);
}

// Two values at once with the packed fp32 instructions of sm_100 (fma/mul .f32x2: one FMA-pipe slot for two lanes'
// worth of arithmetic): the same formula and constants as gelu_tanh_bf16, applied to v = al * z + b.  Only the cap
// on v^2 and the tanh itself stay scalar.
__device__ __forceinline__ uint64_t f32x2_pack(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void f32x2_unpack(uint64_t r, float &lo, float &hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(r));
}
__device__ __forceinline__ uint64_t f32x2_fma(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ uint64_t f32x2_mul(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ void gelu_tanh_bf16_pair(float al, float z0, float z1, float b0, float b1, float &o0, float &o1) {
    const uint64_t v = f32x2_fma(f32x2_pack(al, al), f32x2_pack(z0, z1), f32x2_pack(b0, b1));
    float s0, s1;
    f32x2_unpack(f32x2_mul(v, v), s0, s1);
    const uint64_t s = f32x2_pack(fminf(s0, 50.0f), fminf(s1, 50.0f));
    const uint64_t inner = f32x2_fma(f32x2_fma(f32x2_pack(-3.51516788e-4f, -3.51516788e-4f), s,
                                               f32x2_pack(3.70056460e-2f, 3.70056460e-2f)),
                                     s, f32x2_pack(7.97507884e-1f, 7.97507884e-1f));
    float a0, a1, t0, t1;
    f32x2_unpack(f32x2_mul(v, inner), a0, a1);
    asm("tanh.approx.f32 %0, %1;" : "=f"(t0) : "f"(a0));
    asm("tanh.approx.f32 %0, %1;" : "=f"(t1) : "f"(a1));
    const uint64_t hv = f32x2_mul(v, f32x2_pack(0.5f, 0.5f));
    f32x2_unpack(f32x2_fma(hv, f32x2_pack(t0, t1), hv), o0, o1);
}

__device__ __forceinline__ float apply_act(float v, int act) {
    if (act == TBN_ACT_RELU) return fmaxf(v, 0.0f);
    if (act == TBN_ACT_GELU) return gelu_erf(v);
    return v;
}

// One bit of a packed tile (LSB-first 32-bit words).
__device__ __forceinline__ uint32_t tile_bit(const uint32_t *__restrict__ words, int64_t i) {
    return (__ldg(words + (i >> 5)) >> (uint32_t)(i & 31)) & 1u;
}

// ---- programmatic dependent launch ----------------------------------------------------------------
// A kernel launched with launch_pdl() may be scheduled while the previous kernel of the stream is still draining:
// it calls pdl_launch_dependents() first thing (so that ITS successor may be scheduled early too) and pdl_wait()
// before it reads or writes any global memory another kernel may touch; pdl_wait() returns once every earlier
// kernel of the stream has completed and its writes are visible.  In a kernel launched the ordinary way both are
// no-ops.  Only the launch latency is hidden; nothing runs out of order.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// ---- description of one layer call, filled by the C entry points --------------------------------
struct LayerArgs {
    const void *x;
    void *y;
    const uint32_t *tile;
    const void *dense_a;   // tensor-core linear only: bf16 weight rows [q/n][n] used instead of the tile (MLP chain)
    const void *fp_tile;   // full-precision tile (Sec. 5.2): q values used as they are instead of bits and alphas
    int fp_tile_dtype;     // TBN_F32 or TBN_BF16
    const float *alpha;
    const float *bias;
    const void *residual;  // fully-connected only: a tensor shaped and typed like y, added after the activation (or null);
                           // the CUDA-core kernels add it in their epilogue, the tensor-core path in a pass of its own
    int64_t T;       // rows of the contraction: tokens, or Nb*Ho*Wo output pixels
    int32_t n;       // contraction length: in_features or Cin*kh*kw
    int32_t m;       // output features / channels
    int32_t k;       // number of tile repetitions
    int64_t q;       // tile length in bits
    int x_dtype, y_dtype, alpha_mode, act;
    // convolution geometry (is_conv == 0 for fully-connected)
    int is_conv;
    int32_t Nb, Cin, H, Wd, kh, kw, stride, pad, Ho, Wo;
};

// ---- binary-activation layer (bit-packed activations; see bin_act.cu) ---------------------------------
struct BinArgs {
    const uint32_t *x_bits;   // [T][x_row_words] packed activation signs, padding bits zero
    const void *x_bytes;      // optional: the same signs as bytes 0x00 / 0xFF, [T][n] (tensor path only), or null
    const int32_t *x_pop;     // with x_bytes: popcount of every row
    const uint32_t *tile;
    const float *alpha;
    const float *beta;        // per-token scale, or null (= 1)
    const float *bias;
    void *y;
    int64_t T;
    int64_t q;
    int32_t x_row_words;
    int32_t n, m, k;
    int alpha_mode, act, y_dtype;   // y_dtype TBN_I32: the raw integer accumulators
};
cudaError_t launch_binarize(const void *x, int x_dtype, int64_t T, int32_t n, uint32_t *bits, float *beta, void *bytes_out,
                            int32_t *row_pop, cudaStream_t s);
cudaError_t launch_bin_expand(const uint32_t *bits, int64_t T, int32_t n, int32_t row_words, void *bytes, int32_t *row_pop,
                              cudaStream_t s);
bool bin_popc_supported(const BinArgs &a);
cudaError_t launch_bin_popc(const BinArgs &a, cudaStream_t s);
bool bin_tensor_supported(const BinArgs &a);
int launch_bin_tensor(const BinArgs &a, int *device_status, cudaStream_t s);
int force_bin_config(int candidate);                           // testing / tuning aid: candidate < 0 clears

// ---- training-side tiling module (train.cu) ---------------------------------------------------------
cudaError_t launch_tile_expand(const uint32_t *tile, int64_t N, int32_t k, const float *alpha, int per_tile, void *B_hat,
                               int b_dtype, cudaStream_t s);
size_t tile_bwd_workspace_bytes(int64_t N, int32_t k);
cudaError_t launch_tile_bwd(const float *G, const uint32_t *tile, const float *alpha, const float *W, const float *A,
                            int64_t N, int32_t k, int per_tile, float *dW, float *dA, float *dalpha_out, void *workspace,
                            cudaStream_t s);

// ---- encoder-block glue (block.cu) ----------------------------------------------------------------------
bool add_layernorm_supported(int32_t d);
// y = LayerNorm(bf16(a + b)) with the rounded sum also written to sum_out (b = nullptr: plain LayerNorm of a); bf16, 16-byte
// aligned rows
cudaError_t launch_add_layernorm(const void *a, const void *b, void *sum_out, int64_t T, int32_t d, const float *gamma,
                                 const float *beta, float eps, void *y, cudaStream_t s);
cudaError_t launch_layernorm(const void *x, int x_dtype, int64_t T, int32_t d, const float *gamma, const float *beta, float eps,
                             void *y, int y_dtype, cudaStream_t s);
bool attention_supported(int32_t S, int32_t heads, int32_t d_head);
// returns a tbn_status; the tcgen05 kernel (tc_attention.cu) unless forced otherwise, the warp-level MMA kernel as the other path
int launch_attention(const void *qkv, int32_t Nb, int32_t S, int32_t heads, int32_t d_head, void *out, int *device_status,
                     cudaStream_t s);
int force_attention_path(int path);                            // testing aid: 0 automatic, 1 warp-level MMA, 2 tcgen05
bool tc_attention_supported(int32_t Nb, int32_t S, int32_t heads, int32_t d_head);
int launch_tc_attention(const void *qkv, int32_t Nb, int32_t S, int32_t heads, int32_t d_head, void *out, int *device_status,
                        cudaStream_t s);

// ---- full-precision ends of a convolution stack (dense_ends.cu) ---------------------------------------------
bool dense_conv_supported(int32_t Cin, int32_t kh, int32_t kw);
cudaError_t launch_dense_conv(const void *x, int x_dtype, const float *w, const float *bias, void *y, int y_dtype, int32_t Nb,
                              int32_t Cin, int32_t H, int32_t Wd, int32_t Cout, int32_t kh, int32_t kw, int32_t stride, int32_t pad,
                              int act, cudaStream_t s);
bool avgpool_linear_supported(int32_t C);
cudaError_t launch_avgpool_linear(const void *x, int x_dtype, int32_t Nb, int32_t C, int32_t hw, const float *w, const float *bias,
                                  int32_t out_f, float *y, cudaStream_t s);
cudaError_t launch_global_avgpool(const void *x, int x_dtype, int64_t planes, int32_t hw, void *y, int y_dtype, cudaStream_t s);

// ---- layer fed with the compact form of the previous tiled layer's output (tc_linear_compact.cu) ---------
struct CompactArgs {
    const void *z;            // [T][rz] bf16: distinct pre-activations of the previous layer
    const float *alpha_z;     // its alphas (1 or kz)
    const uint32_t *tile;
    const float *alpha;
    const float *bias;
    void *y;
    int64_t T;
    int64_t q;                // this layer's tile length in bits
    int32_t rz, kz;           // this layer's input width is rz * kz
    int32_t m, k;
    int alpha_mode_z, act_z, alpha_mode, act, y_dtype;
};
bool compact_linear_supported(const CompactArgs &a);
int launch_compact_linear(const CompactArgs &a, int *device_status, cudaStream_t s);

// ---- launchers implemented in the other translation units ---------------------------------------
cudaError_t launch_aggregate(const float *W, const float *A, int64_t N, int32_t k, int per_tile,
                             uint32_t *tile_bits, float *alpha, void *workspace, cudaStream_t s);
size_t aggregate_workspace_bytes(int64_t N, int32_t k);
size_t aggregate_static_scratch_capacity();
cudaError_t launch_aggregate_static(const float *W, const float *A, int64_t N, int32_t k, int per_tile,
                                    uint32_t *tile_bits, float *alpha, cudaStream_t s);
cudaError_t launch_pack(const float *src, int64_t q, uint32_t *tile_bits, cudaStream_t s);
cudaError_t launch_expand(const uint32_t *tile_bits, int64_t N, int32_t k, const float *alpha,
                          int per_tile, float *B_hat, cudaStream_t s);
// Folding jobs of an MLP chain (one per layer after the first), executed by one launch.
constexpr int kMaxFoldJobs = 8;
struct FoldJob {
    const uint32_t *tile_next;   // tile of the layer whose rows are folded
    const float *alpha_prev;     // alphas of the layer before it
    __nv_bfloat16 *w_eff;        // out: rows x r_prev
    int32_t rows, n_next, per_tile_prev, k_prev, r_prev;
};
struct FoldJobs {
    FoldJob job[kMaxFoldJobs];
    int32_t count;
};
cudaError_t launch_fold(const FoldJobs &jobs, cudaStream_t s);
cudaError_t launch_f32_to_bf16(const float *src, __nv_bfloat16 *dst, int64_t count, cudaStream_t s);
cudaError_t launch_add_inplace(void *y, const void *res, int64_t count, int dtype, cudaStream_t s);   // y += res

cudaError_t launch_generic(const LayerArgs &a, cudaStream_t s);

bool small_batch_supported(const LayerArgs &a);
cudaError_t launch_small_batch(const LayerArgs &a, cudaStream_t s);
double small_batch_estimate_us(const LayerArgs &a);
// Thin layer (at most 16 distinct rows) with full-precision rows in dense_a: the head of a compact MLP chain.
bool thin_dense_supported(const LayerArgs &a);
cudaError_t launch_thin_dense(const LayerArgs &a, cudaStream_t s);
// The last two layers of a compact MLP chain (folded rows; the last one thin) in one launch.
bool mlp_tail_supported(const LayerArgs &hidden, const LayerArgs &last);
cudaError_t launch_mlp_tail(const LayerArgs &hidden, const LayerArgs &last, cudaStream_t s);

// The tensor-core path reports through a tbn_status because it also uses the driver API.
bool tensor_path_supported(const LayerArgs &a);
size_t tensor_linear_scratch_bytes(const LayerArgs &a);   // split-K partial tiles + arrival counters
int launch_tensor_linear(const LayerArgs &a, int *device_status, void *scratch, size_t scratch_bytes, cudaStream_t s);
int force_linear_config(int candidate, int splits);          // testing / tuning aid: candidate < 0 clears
cudaError_t launch_wait_probe(int *status, int detail, cudaStream_t s);   // testing aid: a bounded wait that runs out
bool tensor_conv_supported(const LayerArgs &a);
int launch_tensor_conv(const LayerArgs &a, int *device_status, cudaStream_t s);

}  // namespace tbn
