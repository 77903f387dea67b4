// C entry points of libtbn: argument validation, path selection, workspace carving.
// Every step of the computation runs in the kernels of the other translation units; nothing here
// touches the data on the host, and there is no CPU fallback.
#include <atomic>
#include <cstring>
#include <mutex>

#include "common.cuh"

namespace tbn {

// Device-side status record: {code, detail, wait limit in microseconds (0 = default), reserved}.  Kernels receive its address.
__device__ int g_device_status[4];

__global__ void record_status_kernel(int *status, int code, int detail)
{
    if (atomicCAS(status, 0, code) == 0) status[1] = detail;
}

namespace {

int *device_status_ptr()
{
    // one address per device, looked up lazily (the symbol has a distinct instance on each device)
    static int *cache[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    if (!cache[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_device_status) != cudaSuccess) return nullptr;
        cache[dev] = static_cast<int *>(p);
    }
    return cache[dev];
}

inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool valid_dtype(int d) { return d == TBN_F32 || d == TBN_BF16; }
inline bool valid_alpha_mode(int a) { return a == TBN_ALPHA_PER_LAYER || a == TBN_ALPHA_PER_TILE; }
inline bool valid_act(int a) { return a == TBN_ACT_NONE || a == TBN_ACT_RELU || a == TBN_ACT_GELU; }
inline size_t dtype_bytes(int d) { return d == TBN_BF16 ? 2 : 4; }
inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// ---- host-buffer forward: chunking and the per-device copy streams ------------------------------------------
constexpr int kHostMaxChunks = 32;
constexpr size_t kHostChunkBytes = 16u << 20;          // per direction and chunk: long enough for full link rate

// Tokens per chunk of the host-buffer forward (a multiple of 256), or T when the batch goes through in one piece.
int64_t host_chunk_tokens(int64_t T, int32_t in_f, int32_t out_f, int x_dtype, int y_dtype)
{
    const size_t x_row = (size_t)in_f * dtype_bytes(x_dtype), y_row = (size_t)out_f * dtype_bytes(y_dtype);
    const size_t row = x_row > y_row ? x_row : y_row;
    int64_t chunk = (int64_t)((kHostChunkBytes + row - 1) / row);
    const int64_t at_most = (T + kHostMaxChunks - 1) / kHostMaxChunks;
    if (chunk < at_most) chunk = at_most;
    chunk = (chunk + 255) / 256 * 256;
    return chunk * 2 > T ? T : chunk;                   // fewer than two full chunks: not worth the pipeline
}

// Scratch of the forward calls behind the host-buffer entry point: the largest need among the chunk sizes it runs.
size_t host_inner_bytes(int64_t T, int32_t in_f, int32_t out_f, int32_t k, int x_dtype, int64_t chunk)
{
    if (chunk >= T) return tbn_linear_workspace_bytes(T, in_f, out_f, k, x_dtype);
    size_t need = tbn_linear_workspace_bytes(chunk, in_f, out_f, k, x_dtype);
    if (T % chunk != 0) {
        const size_t tail = tbn_linear_workspace_bytes(T % chunk, in_f, out_f, k, x_dtype);
        need = tail > need ? tail : need;
    }
    return need;
}

struct HostPipe {
    std::mutex mu;
    bool ready = false;
    cudaStream_t in = nullptr, out = nullptr;
    cudaEvent_t ev_in[kHostMaxChunks] = {}, ev_comp[kHostMaxChunks] = {}, ev_start = nullptr, ev_done = nullptr;
};

// The copy streams and events of the current device, created on first use (no device memory is allocated).
HostPipe *host_pipe()
{
    static HostPipe pipes[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    HostPipe &hp = pipes[dev];
    std::lock_guard<std::mutex> guard(hp.mu);
    if (!hp.ready) {
        bool ok = cudaStreamCreateWithFlags(&hp.in, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaStreamCreateWithFlags(&hp.out, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaEventCreateWithFlags(&hp.ev_start, cudaEventDisableTiming) == cudaSuccess &&
                  cudaEventCreateWithFlags(&hp.ev_done, cudaEventDisableTiming) == cudaSuccess;
        for (int i = 0; i < kHostMaxChunks && ok; ++i)
            ok = cudaEventCreateWithFlags(&hp.ev_in[i], cudaEventDisableTiming) == cudaSuccess &&
                 cudaEventCreateWithFlags(&hp.ev_comp[i], cudaEventDisableTiming) == cudaSuccess;
        if (!ok) return nullptr;
        hp.ready = true;
    }
    return &hp;
}

// ---- MLP chain: a side stream for the folds ---------------------------------------------------------------------
// The folds depend on the parameters only, so they can run beside the first layer.  One side stream and two events per
// device, created at the first call that is not being captured into a graph (creating them would break the capture;
// such a call, and any call after a failed creation, simply keeps the folds on the caller's stream).
struct MlpFork {
    std::mutex mu;
    int state = 0;                                     // 0 = not created yet, 1 = ready, -1 = creation failed
    cudaStream_t side = nullptr;
    cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
};

MlpFork *mlp_fork(cudaStream_t s)
{
    static MlpFork forks[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    MlpFork &f = forks[dev];
    std::lock_guard<std::mutex> guard(f.mu);
    if (f.state == 0) {
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(s, &cap) != cudaSuccess || cap != cudaStreamCaptureStatusNone) return nullptr;
        const bool ok = cudaStreamCreateWithFlags(&f.side, cudaStreamNonBlocking) == cudaSuccess &&
                        cudaEventCreateWithFlags(&f.ev_fork, cudaEventDisableTiming) == cudaSuccess &&
                        cudaEventCreateWithFlags(&f.ev_join, cudaEventDisableTiming) == cudaSuccess;
        f.state = ok ? 1 : -1;
    }
    return f.state == 1 ? &f : nullptr;
}

// Validation shared by the fully-connected and convolution entry points.
int check_layer_common(const void *x, int x_dtype, const uint32_t *tile, int32_t k, const float *alpha,
                       int alpha_mode, const float *bias, int act, const void *y, int y_dtype, int path,
                       bool empty)
{
    if (!tile || !alpha) return TBN_ERR_INVALID_ARG;
    if (!empty && (!x || !y)) return TBN_ERR_INVALID_ARG;   // an empty batch may come with null data pointers
    if (!valid_dtype(x_dtype) || !valid_dtype(y_dtype) || !valid_alpha_mode(alpha_mode) || !valid_act(act))
        return TBN_ERR_INVALID_ARG;
    if (path < TBN_PATH_AUTO || path > TBN_PATH_TENSOR) return TBN_ERR_INVALID_ARG;
    if (k <= 0) return TBN_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(y) || !aligned16(tile)) return TBN_ERR_INVALID_ARG;
    if (bias && (reinterpret_cast<uintptr_t>(bias) & 3u)) return TBN_ERR_INVALID_ARG;
    return TBN_OK;
}

int select_linear_path(const LayerArgs &a)
{
    const bool tensor = tensor_path_supported(a), small = small_batch_supported(a);
    if (tensor && small) {
        // Both estimates are fits to launch-to-launch times measured on B200.  With few tokens the tensor-core
        // kernel is bound by decoding the tile (about 2 ns per input feature and CTA, split-K included) until
        // the output tiles outnumber the SMs.
        const double r = (double)(a.q / a.n);
        const double small_us = small_batch_estimate_us(a);
        const double fill = (double)a.T * r / (64.0 * 4096.0) * 0.75;
        const double tensor_us = 6.0 + 0.002 * (double)a.n * (fill > 1.0 ? fill : 1.0);
        return small_us < tensor_us ? TBN_PATH_SMALL : TBN_PATH_TENSOR;
    }
    if (tensor) return TBN_PATH_TENSOR;
    if (small) return TBN_PATH_SMALL;
    return TBN_PATH_GENERIC;
}

size_t tensor_scratch_bytes(int64_t T, int32_t in_f, int x_dtype)
{
    // fp32 activations are rounded to bf16 before the tensor-core kernel stages them with TMA
    return x_dtype == TBN_F32 ? round_up((size_t)T * (size_t)in_f * 2, 256) : 0;
}

// Runs one layer on the chosen path.  `a` is fully validated.
int run_layer(LayerArgs a, int path, void *workspace, size_t workspace_bytes, cudaStream_t s)
{
    if (a.T == 0) return TBN_OK;
    if (path == TBN_PATH_AUTO)
        path = a.is_conv ? (tensor_conv_supported(a) ? TBN_PATH_TENSOR : TBN_PATH_GENERIC) : select_linear_path(a);
    cudaError_t e = cudaSuccess;
    switch (path) {
    case TBN_PATH_GENERIC:
        e = launch_generic(a, s);
        break;
    case TBN_PATH_SMALL:
        if (a.is_conv || !small_batch_supported(a)) return TBN_ERR_UNSUPPORTED;
        e = launch_small_batch(a, s);
        break;
    case TBN_PATH_TENSOR: {
        if (a.is_conv ? !tensor_conv_supported(a) : !tensor_path_supported(a)) return TBN_ERR_UNSUPPORTED;
        const int64_t x_count = a.is_conv ? (int64_t)a.Nb * a.Cin * a.H * a.Wd : a.T * (int64_t)a.n;
        // workspace layout: [bf16 copy of fp32 activations][split-K scratch of the linear kernel]
        char *rest = static_cast<char *>(workspace);
        size_t rest_bytes = workspace ? workspace_bytes : 0;
        if (a.x_dtype == TBN_F32) {
            const size_t need = round_up((size_t)x_count * 2, 256);
            if (!workspace || workspace_bytes < need || !aligned16(workspace)) return TBN_ERR_WORKSPACE;
            rest += need;
            rest_bytes -= need;
            e = launch_f32_to_bf16(static_cast<const float *>(a.x), static_cast<__nv_bfloat16 *>(workspace),
                                   x_count, s);
            if (e != cudaSuccess) return TBN_ERR_CUDA;
            a.x = workspace;
            a.x_dtype = TBN_BF16;
        }
        int *st = device_status_ptr();
        if (!st) return TBN_ERR_CUDA;
        if (rest_bytes == 0 || !aligned16(rest)) { rest = nullptr; rest_bytes = 0; }
        if (a.is_conv) return launch_tensor_conv(a, st, s);
        const int rc = launch_tensor_linear(a, st, rest, rest_bytes, s);
        if (rc != TBN_OK || a.residual == nullptr) return rc;
        return launch_add_inplace(a.y, a.residual, a.T * (int64_t)a.m, a.y_dtype, s) == cudaSuccess ? TBN_OK : TBN_ERR_CUDA;
    }
    default:
        return TBN_ERR_INVALID_ARG;
    }
    return e == cudaSuccess ? TBN_OK : TBN_ERR_CUDA;
}

int fill_linear(LayerArgs &a, const void *x, int x_dtype, int64_t T, int32_t in_f, int32_t out_f,
                const uint32_t *tile_bits, int32_t k, const float *alpha, int alpha_mode,
                const float *bias, int act, void *y, int y_dtype, int path)
{
    if (T < 0 || in_f <= 0 || out_f <= 0) return TBN_ERR_INVALID_ARG;
    int rc = check_layer_common(x, x_dtype, tile_bits, k, alpha, alpha_mode, bias, act, y, y_dtype, path, T == 0);
    if (rc != TBN_OK) return rc;
    const int64_t N = (int64_t)in_f * out_f;
    if (N % k != 0) return TBN_ERR_SHAPE;
    std::memset(&a, 0, sizeof(a));
    a.x = x; a.y = y; a.tile = tile_bits; a.alpha = alpha; a.bias = bias;
    a.T = T; a.n = in_f; a.m = out_f; a.k = k; a.q = N / k;
    a.x_dtype = x_dtype; a.y_dtype = y_dtype; a.alpha_mode = alpha_mode; a.act = act;
    a.is_conv = 0;
    return TBN_OK;
}

std::atomic<int> g_mlp_layerwise{0};        // testing aid: 1 = tbn_mlp_fwd runs layer by layer even where the compact chain applies

__device__ float g_device_one = 1.0f;       // alpha of the compact (unscaled) hidden tensors of the MLP chain

const float *device_one_ptr()
{
    static float *cache[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    if (!cache[dev]) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_device_one) != cudaSuccess) return nullptr;
        cache[dev] = static_cast<float *>(p);
    }
    return cache[dev];
}

// Workspace layout of the compact MLP chain; false when the shapes do not allow it (every layer's tile must span
// whole rows and the compact widths must keep 16-byte row pitches).
constexpr int kMaxChainLayers = 64;
struct MlpChainPlan {
    size_t g_off[2], weff_off[kMaxChainLayers], xconv_off, scratch_off, scratch_bytes, total_bytes;
};

bool plan_mlp_chain(int64_t T, int32_t L, const int32_t *dims, const int32_t *ks, int x_dtype, MlpChainPlan &plan);

int check_mlp(int64_t T, int32_t L, const int32_t *dims, const int32_t *ks)
{
    if (T < 0 || L <= 0 || !dims || !ks) return TBN_ERR_INVALID_ARG;
    for (int32_t l = 0; l <= L; ++l)
        if (dims[l] <= 0) return TBN_ERR_INVALID_ARG;
    for (int32_t l = 0; l < L; ++l) {
        if (ks[l] <= 0) return TBN_ERR_INVALID_ARG;
        if (((int64_t)dims[l] * dims[l + 1]) % ks[l] != 0) return TBN_ERR_SHAPE;
    }
    return TBN_OK;
}

bool plan_mlp_chain(int64_t T, int32_t L, const int32_t *dims, const int32_t *ks, int x_dtype, MlpChainPlan &plan)
{
    if (L < 2 || L > kMaxChainLayers || dims[0] % 8 != 0) return false;
    int32_t r_max = 0;
    for (int32_t l = 0; l < L; ++l) {
        const int64_t N = (int64_t)dims[l] * dims[l + 1];
        if (N % ks[l] != 0 || (N / ks[l]) % dims[l] != 0) return false;          // tile spans whole rows
        const int32_t r = dims[l + 1] / ks[l];
        if (l < L - 1) {
            if (r % 8 != 0) return false;                                        // TMA row pitch of the compact tensor
            r_max = r > r_max ? r : r_max;
        }
    }
    size_t off = 0;
    const size_t g = round_up((size_t)T * r_max * 2, 256);
    plan.g_off[0] = off; off += g;
    plan.g_off[1] = off; off += g;
    size_t scratch = 0;
    int32_t n_cur = dims[0];
    for (int32_t l = 0; l < L; ++l) {
        const int32_t r = dims[l + 1] / ks[l];
        plan.weff_off[l] = off;
        if (l > 0) off += round_up((size_t)r * n_cur * 2, 256);
        LayerArgs a;
        std::memset(&a, 0, sizeof(a));
        a.T = T; a.n = n_cur; a.q = (int64_t)r * n_cur; a.x_dtype = TBN_BF16; a.y_dtype = TBN_BF16;
        a.m = l == L - 1 ? dims[l + 1] : r; a.k = l == L - 1 ? ks[l] : 1;
        const size_t b = round_up(tensor_linear_scratch_bytes(a), 256);
        scratch = b > scratch ? b : scratch;
        n_cur = r;
    }
    plan.xconv_off = off;
    if (x_dtype == TBN_F32) off += round_up((size_t)T * dims[0] * 2, 256);
    plan.scratch_off = off;
    plan.scratch_bytes = scratch;
    plan.total_bytes = off + scratch;
    return true;
}

}  // namespace
}  // namespace tbn

using namespace tbn;

extern "C" {

int64_t tbn_tile_words(int64_t q)
{
    if (q <= 0) return 0;
    return ((q + 31) / 32 + 3) / 4 * 4;
}

const char *tbn_status_string(int status)
{
    switch (status) {
    case TBN_OK: return "ok";
    case TBN_ERR_INVALID_ARG: return "invalid argument";
    case TBN_ERR_SHAPE: return "shape error: k must divide the number of weights";
    case TBN_ERR_UNSUPPORTED: return "unsupported combination";
    case TBN_ERR_WORKSPACE: return "workspace missing or too small";
    case TBN_ERR_CUDA: return "CUDA call failed";
    case TBN_ERR_TIMEOUT: return "device-side wait timed out";
    default: return "unknown status";
    }
}

size_t tbn_aggregate_workspace_bytes(int64_t N, int32_t k)
{
    if (N <= 0 || k <= 0 || N % k != 0) return 0;
    return round_up(aggregate_workspace_bytes(N, k), 256);
}

int tbn_aggregate_tile(const float *W, const float *A, int64_t N, int32_t k, int alpha_mode,
                       uint32_t *tile_bits, float *alpha, void *workspace, size_t workspace_bytes,
                       void *stream)
{
    if (!W || !tile_bits || !alpha || N <= 0 || k <= 0 || !valid_alpha_mode(alpha_mode))
        return TBN_ERR_INVALID_ARG;
    if (N % k != 0) return TBN_ERR_SHAPE;
    if (!aligned16(W) || (A && !aligned16(A)) || !aligned16(tile_bits)) return TBN_ERR_INVALID_ARG;
    if (!workspace || !aligned16(workspace) || workspace_bytes < aggregate_workspace_bytes(N, k))
        return TBN_ERR_WORKSPACE;
    cudaError_t e = launch_aggregate(W, A, N, k, alpha_mode == TBN_ALPHA_PER_TILE, tile_bits, alpha,
                                     workspace, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? TBN_OK : TBN_ERR_CUDA;
}

int tbn_aggregate_tile_static(const float *W, const float *A, int64_t N, int32_t k, int alpha_mode,
                              uint32_t *tile_bits, float *alpha, void *stream)
{
    if (!W || !tile_bits || !alpha || N <= 0 || k <= 0 || !valid_alpha_mode(alpha_mode))
        return TBN_ERR_INVALID_ARG;
    if (N % k != 0) return TBN_ERR_SHAPE;
    if (!aligned16(W) || (A && !aligned16(A)) || !aligned16(tile_bits)) return TBN_ERR_INVALID_ARG;
    if (aggregate_workspace_bytes(N, k) > aggregate_static_scratch_capacity())
        return TBN_ERR_WORKSPACE;           // the layer needs more scratch than the built-in array holds
    cudaError_t e = launch_aggregate_static(W, A, N, k, alpha_mode == TBN_ALPHA_PER_TILE, tile_bits, alpha,
                                            static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? TBN_OK : TBN_ERR_CUDA;
}

int tbn_pack_tile(const float *src, int64_t q, uint32_t *tile_bits, void *stream)
{
    if (!src || !tile_bits || q <= 0) return TBN_ERR_INVALID_ARG;
    if (!aligned16(tile_bits)) return TBN_ERR_INVALID_ARG;
    cudaError_t e = launch_pack(src, q, tile_bits, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? TBN_OK : TBN_ERR_CUDA;
}

int tbn_expand_tile(const uint32_t *tile_bits, int64_t N, int32_t k, const float *alpha, int alpha_mode,
                    float *B_hat, void *stream)
{
    if (!tile_bits || !alpha || !B_hat || N <= 0 || k <= 0 || !valid_alpha_mode(alpha_mode))
        return TBN_ERR_INVALID_ARG;
    if (N % k != 0) return TBN_ERR_SHAPE;
    cudaError_t e = launch_expand(tile_bits, N, k, alpha, alpha_mode == TBN_ALPHA_PER_TILE, B_hat,
                                  static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? TBN_OK : TBN_ERR_CUDA;
}

size_t tbn_linear_workspace_bytes(int64_t T, int32_t in_f, int32_t out_f, int32_t k, int x_dtype)
{
    if (T <= 0 || in_f <= 0 || out_f <= 0 || k <= 0 || ((int64_t)in_f * out_f) % k != 0) return 0;
    LayerArgs a;
    std::memset(&a, 0, sizeof(a));
    a.T = T; a.n = in_f; a.m = out_f; a.k = k; a.q = (int64_t)in_f * out_f / k;
    a.x_dtype = TBN_BF16; a.y_dtype = TBN_BF16;
    // bf16 copy of fp32 activations + the tensor-core kernel's split-K scratch (partial tiles and counters)
    return tensor_scratch_bytes(T, in_f, x_dtype) + round_up(tensor_linear_scratch_bytes(a), 256);
}

int tbn_linear_select_path(int64_t T, int32_t in_f, int32_t out_f, int32_t k, int x_dtype)
{
    if (T < 0 || in_f <= 0 || out_f <= 0 || k <= 0 || !valid_dtype(x_dtype)) return TBN_ERR_INVALID_ARG;
    if (((int64_t)in_f * out_f) % k != 0) return TBN_ERR_SHAPE;
    LayerArgs a;
    std::memset(&a, 0, sizeof(a));
    a.T = T; a.n = in_f; a.m = out_f; a.k = k; a.q = (int64_t)in_f * out_f / k;
    a.x_dtype = x_dtype; a.y_dtype = TBN_BF16;
    return select_linear_path(a);
}

size_t tbn_linear_fp_tile_workspace_bytes(int64_t T, int32_t in_f, int32_t out_f, int32_t k, int x_dtype,
                                          int tile_dtype)
{
    if (T <= 0 || in_f <= 0 || out_f <= 0 || k <= 0 || ((int64_t)in_f * out_f) % k != 0) return 0;
    const int64_t q = (int64_t)in_f * out_f / k;
    // bf16 copy of an fp32 tile for the tensor-core kernel, then what the binary layer of this shape needs
    const size_t rows = tile_dtype == TBN_F32 ? round_up((size_t)q * 2, 256) : 0;
    return rows + tbn_linear_workspace_bytes(T, in_f, out_f, k, x_dtype);
}

int tbn_linear_fp_tile_fwd(const void *x, int x_dtype, int64_t T, int32_t in_f, int32_t out_f,
                           const void *tile_values, int tile_dtype, int32_t k,
                           const float *bias, int act, void *y, int y_dtype,
                           void *workspace, size_t workspace_bytes, void *stream, int path)
{
    if (T < 0 || in_f <= 0 || out_f <= 0 || k <= 0 || !tile_values) return TBN_ERR_INVALID_ARG;
    if (!valid_dtype(x_dtype) || !valid_dtype(y_dtype) || !valid_dtype(tile_dtype)) return TBN_ERR_INVALID_ARG;
    if (act != TBN_ACT_NONE && act != TBN_ACT_RELU && act != TBN_ACT_GELU) return TBN_ERR_INVALID_ARG;
    if (T > 0 && (!x || !y)) return TBN_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(y) || !aligned16(tile_values)) return TBN_ERR_INVALID_ARG;
    if (bias && (reinterpret_cast<uintptr_t>(bias) & 3u)) return TBN_ERR_INVALID_ARG;
    const int64_t N = (int64_t)in_f * out_f;
    if (N % k != 0) return TBN_ERR_SHAPE;
    if (T == 0) return TBN_OK;
    cudaStream_t s = static_cast<cudaStream_t>(stream);

    LayerArgs a;
    std::memset(&a, 0, sizeof(a));
    a.x = x; a.y = y; a.bias = bias;
    a.T = T; a.n = in_f; a.m = out_f; a.k = k; a.q = N / k;
    a.x_dtype = x_dtype; a.y_dtype = y_dtype; a.alpha_mode = TBN_ALPHA_PER_LAYER; a.act = act;
    a.alpha = device_one_ptr();                      // no scaling factors: every repetition is scaled by 1
    if (!a.alpha) return TBN_ERR_CUDA;

    if (path == TBN_PATH_AUTO) path = tensor_path_supported(a) ? TBN_PATH_TENSOR : TBN_PATH_GENERIC;
    if (path == TBN_PATH_GENERIC) {
        a.fp_tile = tile_values; a.fp_tile_dtype = tile_dtype;
        return launch_generic(a, s) == cudaSuccess ? TBN_OK : TBN_ERR_CUDA;
    }
    if (path != TBN_PATH_TENSOR) return TBN_ERR_UNSUPPORTED;   // the bit-decoding small-batch kernels do not apply
    if (!tensor_path_supported(a)) return TBN_ERR_UNSUPPORTED;

    // the tile's r = q / in_f rows are the A operand of the tensor-core kernel as they are (rounded to bf16)
    char *rest = static_cast<char *>(workspace);
    size_t rest_bytes = workspace ? workspace_bytes : 0;
    if (tile_dtype == TBN_F32) {
        const size_t need = round_up((size_t)a.q * 2, 256);
        if (!workspace || !aligned16(workspace) || workspace_bytes < need) return TBN_ERR_WORKSPACE;
        if (launch_f32_to_bf16(static_cast<const float *>(tile_values), reinterpret_cast<__nv_bfloat16 *>(rest), a.q, s) !=
            cudaSuccess)
            return TBN_ERR_CUDA;
        a.dense_a = rest;
        rest += need;
        rest_bytes -= need;
    } else {
        a.dense_a = tile_values;
    }
    return run_layer(a, TBN_PATH_TENSOR, rest_bytes ? rest : nullptr, rest_bytes, s);
}

int tbn_linear_fwd_path(const void *x, int x_dtype, int64_t T, int32_t in_f, int32_t out_f,
                        const uint32_t *tile_bits, int32_t k, const float *alpha, int alpha_mode,
                        const float *bias, int act, void *y, int y_dtype,
                        void *workspace, size_t workspace_bytes, void *stream, int path)
{
    LayerArgs a;
    int rc = fill_linear(a, x, x_dtype, T, in_f, out_f, tile_bits, k, alpha, alpha_mode, bias, act, y,
                         y_dtype, path);
    if (rc != TBN_OK) return rc;
    return run_layer(a, path, workspace, workspace_bytes, static_cast<cudaStream_t>(stream));
}

int tbn_linear_res_fwd(const void *x, int x_dtype, int64_t T, int32_t in_f, int32_t out_f,
                       const uint32_t *tile_bits, int32_t k, const float *alpha, int alpha_mode,
                       const float *bias, int act, const void *residual, void *y, int y_dtype,
                       void *workspace, size_t workspace_bytes, void *stream, int path)
{
    LayerArgs a;
    int rc = fill_linear(a, x, x_dtype, T, in_f, out_f, tile_bits, k, alpha, alpha_mode, bias, act, y,
                         y_dtype, path);
    if (rc != TBN_OK) return rc;
    if (residual && (!aligned16(residual) || residual == y)) return TBN_ERR_INVALID_ARG;   // the output may not alias it
    a.residual = residual;
    return run_layer(a, path, workspace, workspace_bytes, static_cast<cudaStream_t>(stream));
}

int tbn_linear_fwd(const void *x, int x_dtype, int64_t T, int32_t in_f, int32_t out_f,
                   const uint32_t *tile_bits, int32_t k, const float *alpha, int alpha_mode,
                   const float *bias, int act, void *y, int y_dtype,
                   void *workspace, size_t workspace_bytes, void *stream)
{
    return tbn_linear_fwd_path(x, x_dtype, T, in_f, out_f, tile_bits, k, alpha, alpha_mode, bias, act, y,
                               y_dtype, workspace, workspace_bytes, stream, TBN_PATH_AUTO);
}

size_t tbn_linear_host_workspace_bytes(int64_t T, int32_t in_f, int32_t out_f, int32_t k,
                                       int x_dtype, int y_dtype)
{
    if (T <= 0 || in_f <= 0 || out_f <= 0 || !valid_dtype(x_dtype) || !valid_dtype(y_dtype)) return 0;
    return round_up((size_t)T * in_f * dtype_bytes(x_dtype), 256) +
           round_up((size_t)T * out_f * dtype_bytes(y_dtype), 256) +
           host_inner_bytes(T, in_f, out_f, k, x_dtype, host_chunk_tokens(T, in_f, out_f, x_dtype, y_dtype));
}

int tbn_linear_fwd_host(const void *x_host, int x_dtype, int64_t T, int32_t in_f, int32_t out_f,
                        const uint32_t *tile_bits, int32_t k, const float *alpha, int alpha_mode,
                        const float *bias, int act, void *y_host, int y_dtype,
                        void *workspace, size_t workspace_bytes, void *stream)
{
    if (!x_host || !y_host || !valid_dtype(x_dtype) || !valid_dtype(y_dtype) || T < 0 || in_f <= 0 ||
        out_f <= 0)
        return TBN_ERR_INVALID_ARG;
    if (T == 0) return TBN_OK;
    const size_t x_row = (size_t)in_f * dtype_bytes(x_dtype), y_row = (size_t)out_f * dtype_bytes(y_dtype);
    const size_t xb = round_up((size_t)T * x_row, 256);
    const size_t yb = round_up((size_t)T * y_row, 256);
    const int64_t chunk = host_chunk_tokens(T, in_f, out_f, x_dtype, y_dtype);
    const size_t inner = host_inner_bytes(T, in_f, out_f, k, x_dtype, chunk);
    if (!workspace || !aligned16(workspace) || workspace_bytes < xb + yb + inner) return TBN_ERR_WORKSPACE;
    char *ws = static_cast<char *>(workspace);
    char *x_dev = ws, *y_dev = ws + xb;
    void *inner_ws = ws + xb + yb;
    cudaStream_t s = static_cast<cudaStream_t>(stream);

    if (chunk >= T) {                     // small transfers: copy in, run, copy out on the caller's stream
        if (cudaMemcpyAsync(x_dev, x_host, (size_t)T * x_row, cudaMemcpyHostToDevice, s) != cudaSuccess)
            return TBN_ERR_CUDA;
        int rc = tbn_linear_fwd(x_dev, x_dtype, T, in_f, out_f, tile_bits, k, alpha, alpha_mode, bias, act, y_dev,
                                y_dtype, inner_ws, inner, stream);
        if (rc != TBN_OK) return rc;
        if (cudaMemcpyAsync(y_host, y_dev, (size_t)T * y_row, cudaMemcpyDeviceToHost, s) != cudaSuccess)
            return TBN_ERR_CUDA;
        return cudaStreamSynchronize(s) == cudaSuccess ? TBN_OK : TBN_ERR_CUDA;
    }

    // Token rows are independent, so the batch goes through in chunks: chunk c+1 is copied in and chunk c-1 copied
    // out (two copy streams, both directions of the host link busy) while chunk c is computed on the caller's stream.
    HostPipe *hp = host_pipe();
    if (!hp) return TBN_ERR_CUDA;
    std::lock_guard<std::mutex> guard(hp->mu);        // the copy streams and events are shared by the calls on a device
    bool cuda_ok = cudaEventRecord(hp->ev_start, s) == cudaSuccess &&
                   cudaStreamWaitEvent(hp->in, hp->ev_start, 0) == cudaSuccess &&
                   cudaStreamWaitEvent(hp->out, hp->ev_start, 0) == cudaSuccess;
    int rc = TBN_OK;
    int c = 0;
    for (int64_t t0 = 0; t0 < T && cuda_ok && rc == TBN_OK; t0 += chunk, ++c) {
        const int64_t tc = T - t0 < chunk ? T - t0 : chunk;
        cuda_ok = cudaMemcpyAsync(x_dev + t0 * x_row, static_cast<const char *>(x_host) + t0 * x_row, tc * x_row,
                                  cudaMemcpyHostToDevice, hp->in) == cudaSuccess &&
                  cudaEventRecord(hp->ev_in[c], hp->in) == cudaSuccess &&
                  cudaStreamWaitEvent(s, hp->ev_in[c], 0) == cudaSuccess;
        if (!cuda_ok) break;
        rc = tbn_linear_fwd(x_dev + t0 * x_row, x_dtype, tc, in_f, out_f, tile_bits, k, alpha, alpha_mode, bias, act,
                            y_dev + t0 * y_row, y_dtype, inner_ws, inner, stream);
        if (rc != TBN_OK) break;
        cuda_ok = cudaEventRecord(hp->ev_comp[c], s) == cudaSuccess &&
                  cudaStreamWaitEvent(hp->out, hp->ev_comp[c], 0) == cudaSuccess &&
                  cudaMemcpyAsync(static_cast<char *>(y_host) + t0 * y_row, y_dev + t0 * y_row, tc * y_row,
                                  cudaMemcpyDeviceToHost, hp->out) == cudaSuccess;
    }
    // join: the caller's stream continues after the last copy out, then the call waits for it.  The copy streams are
    // drained even after an error, so nothing of this call is still in flight when it returns.
    const bool joined = cudaEventRecord(hp->ev_done, hp->out) == cudaSuccess &&
                        cudaStreamWaitEvent(s, hp->ev_done, 0) == cudaSuccess;
    const bool drained = cudaStreamSynchronize(hp->in) == cudaSuccess && cudaStreamSynchronize(hp->out) == cudaSuccess &&
                         cudaStreamSynchronize(s) == cudaSuccess;
    if (rc != TBN_OK) return rc;
    return cuda_ok && joined && drained ? TBN_OK : TBN_ERR_CUDA;
}

size_t tbn_conv2d_workspace_bytes(int32_t Nb, int32_t Cin, int32_t H, int32_t Wd, int32_t, int32_t, int32_t,
                                  int32_t, int32_t, int32_t, int x_dtype)
{
    // the tensor-core path rounds fp32 activations to bf16 first
    if (x_dtype != TBN_F32 || Nb <= 0 || Cin <= 0 || H <= 0 || Wd <= 0) return 0;
    return round_up((size_t)Nb * Cin * H * Wd * 2, 256);
}

int tbn_conv2d_fwd_path(const void *x, int x_dtype, int32_t Nb, int32_t Cin, int32_t H, int32_t Wd,
                        int32_t Cout, int32_t kh, int32_t kw, int32_t stride, int32_t pad,
                        const uint32_t *tile_bits, int32_t k, const float *alpha, int alpha_mode,
                        const float *bias, int act, void *y, int y_dtype,
                        void *workspace, size_t workspace_bytes, void *stream, int path)
{
    if (Nb < 0 || Cin <= 0 || H <= 0 || Wd <= 0 || Cout <= 0 || kh <= 0 || kw <= 0 || stride <= 0 || pad < 0)
        return TBN_ERR_INVALID_ARG;
    int rc = check_layer_common(x, x_dtype, tile_bits, k, alpha, alpha_mode, bias, act, y, y_dtype, path, Nb == 0);
    if (rc != TBN_OK) return rc;
    if (H + 2 * pad < kh || Wd + 2 * pad < kw) return TBN_ERR_SHAPE;
    const int64_t n = (int64_t)Cin * kh * kw;
    if (n > 0x7fffffffLL) return TBN_ERR_UNSUPPORTED;
    const int64_t N = n * Cout;
    if (N % k != 0) return TBN_ERR_SHAPE;
    LayerArgs a;
    std::memset(&a, 0, sizeof(a));
    a.x = x; a.y = y; a.tile = tile_bits; a.alpha = alpha; a.bias = bias;
    a.n = (int32_t)n; a.m = Cout; a.k = k; a.q = N / k;
    a.x_dtype = x_dtype; a.y_dtype = y_dtype; a.alpha_mode = alpha_mode; a.act = act;
    a.is_conv = 1;
    a.Nb = Nb; a.Cin = Cin; a.H = H; a.Wd = Wd; a.kh = kh; a.kw = kw; a.stride = stride; a.pad = pad;
    a.Ho = (H + 2 * pad - kh) / stride + 1;
    a.Wo = (Wd + 2 * pad - kw) / stride + 1;
    a.T = (int64_t)Nb * a.Ho * a.Wo;
    return run_layer(a, path, workspace, workspace_bytes, static_cast<cudaStream_t>(stream));
}

int tbn_conv2d_fwd(const void *x, int x_dtype, int32_t Nb, int32_t Cin, int32_t H, int32_t Wd,
                   int32_t Cout, int32_t kh, int32_t kw, int32_t stride, int32_t pad,
                   const uint32_t *tile_bits, int32_t k, const float *alpha, int alpha_mode,
                   const float *bias, int act, void *y, int y_dtype,
                   void *workspace, size_t workspace_bytes, void *stream)
{
    return tbn_conv2d_fwd_path(x, x_dtype, Nb, Cin, H, Wd, Cout, kh, kw, stride, pad, tile_bits, k, alpha,
                               alpha_mode, bias, act, y, y_dtype, workspace, workspace_bytes, stream,
                               TBN_PATH_AUTO);
}

size_t tbn_mlp_workspace_bytes(int64_t T, int32_t L, const int32_t *dims, const int32_t *ks, int x_dtype)
{
    if (check_mlp(T, L, dims, ks) != TBN_OK || T == 0) return 0;
    // (a) layer-by-layer chain: two ping-pong bf16 hidden buffers sized for the widest hidden layer + the
    //     largest per-layer scratch
    int32_t widest = 0;
    for (int32_t l = 1; l < L; ++l) widest = dims[l] > widest ? dims[l] : widest;
    const size_t hidden = round_up((size_t)T * widest * 2, 256);
    size_t scratch = 0;
    for (int32_t l = 0; l < L; ++l) {
        const size_t b = tbn_linear_workspace_bytes(T, dims[l], dims[l + 1], ks[l], l == 0 ? x_dtype : TBN_BF16);
        scratch = b > scratch ? b : scratch;
    }
    const size_t unfused = 2 * hidden + scratch;
    // (b) compact chain (see tbn_mlp_fwd): sized whenever the shapes allow it
    MlpChainPlan plan;
    const size_t chained = plan_mlp_chain(T, L, dims, ks, x_dtype, plan) ? plan.total_bytes : 0;
    return unfused > chained ? unfused : chained;
}

int tbn_mlp_fwd(const void *x, int x_dtype, int64_t T, int32_t L, const int32_t *dims,
                const uint32_t *const *tiles, const int32_t *ks, const float *const *alphas,
                const int *alpha_modes, int hidden_act, void *y, int y_dtype,
                void *workspace, size_t workspace_bytes, void *stream)
{
    int rc = check_mlp(T, L, dims, ks);
    if (rc != TBN_OK) return rc;
    if (!x || !y || !tiles || !alphas || !alpha_modes || !valid_act(hidden_act)) return TBN_ERR_INVALID_ARG;
    if (!valid_dtype(x_dtype) || !valid_dtype(y_dtype)) return TBN_ERR_INVALID_ARG;
    for (int32_t l = 0; l < L; ++l)
        if (!tiles[l] || !alphas[l] || !valid_alpha_mode(alpha_modes[l])) return TBN_ERR_INVALID_ARG;
    if (T == 0) return TBN_OK;
    const size_t need = tbn_mlp_workspace_bytes(T, L, dims, ks, x_dtype);
    if (need > 0 && (!workspace || !aligned16(workspace) || workspace_bytes < need)) return TBN_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    char *ws = static_cast<char *>(workspace);

    // Compact chain.  With a ReLU (or no) hidden activation, layer l's output is alpha_j * g[:, c] for its k
    // repetitions j (Sec. 4.1), so only the r distinct columns g = act(Z) are written (bf16, [T, r]) and the
    // next layer contracts g with its distinct rows folded with layer l's alphas (launch_fold): the k-fold
    // broadcast of a hidden layer never goes to HBM and the next contraction is k times shorter.
    MlpChainPlan plan;
    if (L >= 2 && (hidden_act == TBN_ACT_RELU || hidden_act == TBN_ACT_NONE) && g_mlp_layerwise.load() == 0 &&
        plan_mlp_chain(T, L, dims, ks, x_dtype, plan) && aligned16(x) && aligned16(y)) {
        int *st = device_status_ptr();
        const float *one = device_one_ptr();
        if (!st || !one) return TBN_ERR_CUDA;
        const void *cur = x;
        if (x_dtype == TBN_F32) {
            if (launch_f32_to_bf16(static_cast<const float *>(x), reinterpret_cast<__nv_bfloat16 *>(ws + plan.xconv_off),
                                   T * (int64_t)dims[0], s) != cudaSuccess)
                return TBN_ERR_CUDA;
            cur = ws + plan.xconv_off;
        }
        // all folds, kMaxFoldJobs layers per launch.  They depend on the parameters only and are first needed by
        // layer 1, so they go to the side stream (ordered after everything already queued on the caller's stream,
        // which may still be reading this workspace) and the caller's stream joins them after launching layer 0.
        MlpFork *fork = mlp_fork(s);
        cudaStream_t fold_stream = s;
        {
            std::unique_lock<std::mutex> fork_guard;
            if (fork) {
                fork_guard = std::unique_lock<std::mutex>(fork->mu);   // record + wait pairs of one call stay together
                if (cudaEventRecord(fork->ev_fork, s) != cudaSuccess ||
                    cudaStreamWaitEvent(fork->side, fork->ev_fork, 0) != cudaSuccess)
                    return TBN_ERR_CUDA;
                fold_stream = fork->side;
            }
            FoldJobs jobs;
            jobs.count = 0;
            int32_t r_prev = dims[1] / ks[0];
            for (int32_t l = 1; l < L; ++l) {
                FoldJob &J = jobs.job[jobs.count++];
                J.tile_next = tiles[l]; J.alpha_prev = alphas[l - 1];
                J.w_eff = reinterpret_cast<__nv_bfloat16 *>(ws + plan.weff_off[l]);
                J.rows = dims[l + 1] / ks[l]; J.n_next = dims[l];
                J.per_tile_prev = alpha_modes[l - 1] == TBN_ALPHA_PER_TILE; J.k_prev = ks[l - 1]; J.r_prev = r_prev;
                r_prev = J.rows;
                if (jobs.count == kMaxFoldJobs || l == L - 1) {
                    if (launch_fold(jobs, fold_stream) != cudaSuccess) return TBN_ERR_CUDA;
                    jobs.count = 0;
                }
            }
            if (fork && cudaEventRecord(fork->ev_join, fork->side) != cudaSuccess) return TBN_ERR_CUDA;
        }
        // layer l of the chain as the kernels see it: input `in` of compact width n_in
        auto layer_args = [&](int32_t l, const void *in, int32_t n_in) {
            const int32_t r = dims[l + 1] / ks[l];
            LayerArgs a;
            std::memset(&a, 0, sizeof(a));
            a.x = in; a.x_dtype = TBN_BF16; a.T = T; a.n = n_in; a.tile = tiles[l];
            if (l > 0) a.dense_a = ws + plan.weff_off[l];
            a.q = (int64_t)r * n_in;
            if (l == L - 1) {
                a.m = dims[l + 1]; a.k = ks[l]; a.alpha = alphas[l]; a.alpha_mode = alpha_modes[l];
                a.act = TBN_ACT_NONE; a.y = y; a.y_dtype = y_dtype;
            } else {
                a.m = r; a.k = 1; a.alpha = one; a.alpha_mode = TBN_ALPHA_PER_LAYER;
                a.act = hidden_act; a.y = ws + plan.g_off[l & 1]; a.y_dtype = TBN_BF16;
            }
            return a;
        };
        int32_t n_cur = dims[0];
        for (int32_t l = 0; l < L; ++l) {
            const int32_t r = dims[l + 1] / ks[l];
            const LayerArgs a = layer_args(l, cur, n_cur);
            if (l == 1 && fork && cudaStreamWaitEvent(s, fork->ev_join, 0) != cudaSuccess) return TBN_ERR_CUDA;
            if (l >= 1 && l == L - 2) {                 // a narrow hidden layer and a thin last layer: one launch for both
                const LayerArgs b = layer_args(l + 1, a.y, r);
                if (mlp_tail_supported(a, b)) {
                    if (launch_mlp_tail(a, b, s) != cudaSuccess) return TBN_ERR_CUDA;
                    break;
                }
            }
            if (thin_dense_supported(a)) {              // a few output rows: not worth a tensor-core launch
                if (launch_thin_dense(a, s) != cudaSuccess) return TBN_ERR_CUDA;
            } else {
                if (!tensor_path_supported(a)) return TBN_ERR_UNSUPPORTED;
                rc = launch_tensor_linear(a, st, ws + plan.scratch_off, plan.scratch_bytes, s);
                if (rc != TBN_OK) return rc;
            }
            cur = a.y;
            n_cur = r;
        }
        return TBN_OK;
    }

    // Layer-by-layer chain: hidden tensors are written in full (bf16) and read back.
    int32_t widest = 0;
    for (int32_t l = 1; l < L; ++l) widest = dims[l] > widest ? dims[l] : widest;
    const size_t hidden = round_up((size_t)T * widest * 2, 256);
    void *buf[2] = {ws, ws + hidden};
    void *scratch = ws + 2 * hidden;
    const size_t scratch_bytes = workspace_bytes - 2 * hidden;

    const void *cur = x;
    int cur_dtype = x_dtype;
    for (int32_t l = 0; l < L; ++l) {
        const bool last = l == L - 1;
        void *out = last ? y : buf[l & 1];
        rc = tbn_linear_fwd(cur, cur_dtype, T, dims[l], dims[l + 1], tiles[l], ks[l], alphas[l],
                            alpha_modes[l], nullptr, last ? TBN_ACT_NONE : hidden_act, out,
                            last ? y_dtype : TBN_BF16, scratch, scratch_bytes, stream);
        if (rc != TBN_OK) return rc;
        cur = out;
        cur_dtype = TBN_BF16;
    }
    return TBN_OK;
}

size_t tbn_tile_bwd_workspace_bytes(int64_t N, int32_t k)
{
    if (N <= 0 || k <= 0 || N % k != 0) return 0;
    return round_up(tile_bwd_workspace_bytes(N, k), 256);
}

int tbn_tile_fwd(const float *W, const float *A, int64_t N, int32_t k, int alpha_mode, void *B_hat, int b_dtype,
                 uint32_t *tile_bits, float *alpha, void *workspace, size_t workspace_bytes, void *stream)
{
    if (!B_hat || !valid_dtype(b_dtype) || !aligned16(B_hat)) return TBN_ERR_INVALID_ARG;
    int rc = tbn_aggregate_tile(W, A, N, k, alpha_mode, tile_bits, alpha, workspace, workspace_bytes, stream);
    if (rc != TBN_OK) return rc;
    return launch_tile_expand(tile_bits, N, k, alpha, alpha_mode == TBN_ALPHA_PER_TILE, B_hat, b_dtype,
                              static_cast<cudaStream_t>(stream)) == cudaSuccess ? TBN_OK : TBN_ERR_CUDA;
}

int tbn_tile_bwd(const float *G, const uint32_t *tile_bits, const float *alpha, const float *W, const float *A,
                 int64_t N, int32_t k, int alpha_mode, float *dW, float *dA, float *dalpha,
                 void *workspace, size_t workspace_bytes, void *stream)
{
    if (!G || !tile_bits || !alpha || !W || !dW || N <= 0 || k <= 0 || !valid_alpha_mode(alpha_mode)) return TBN_ERR_INVALID_ARG;
    if ((A == nullptr) != (dA == nullptr)) return TBN_ERR_INVALID_ARG;       // dA goes with a separate A
    if (N % k != 0) return TBN_ERR_SHAPE;
    if (!aligned16(G) || !aligned16(W) || !aligned16(dW) || (A && (!aligned16(A) || !aligned16(dA))) || !aligned16(tile_bits))
        return TBN_ERR_INVALID_ARG;
    if (!workspace || !aligned16(workspace) || workspace_bytes < tile_bwd_workspace_bytes(N, k)) return TBN_ERR_WORKSPACE;
    return launch_tile_bwd(G, tile_bits, alpha, W, A, N, k, alpha_mode == TBN_ALPHA_PER_TILE, dW, dA, dalpha, workspace,
                           static_cast<cudaStream_t>(stream)) == cudaSuccess ? TBN_OK : TBN_ERR_CUDA;
}

int tbn_linear_compact_fwd(const void *z, int64_t T, int32_t rz, int32_t kz, const float *alpha_z, int alpha_mode_z, int act_z,
                           int32_t out_f, const uint32_t *tile_bits, int32_t k, const float *alpha, int alpha_mode,
                           const float *bias, int act, void *y, int y_dtype, void *stream)
{
    if (T < 0 || rz <= 0 || kz <= 0 || out_f <= 0 || k <= 0) return TBN_ERR_INVALID_ARG;
    if (!alpha_z || !tile_bits || !alpha || !valid_alpha_mode(alpha_mode_z) || !valid_alpha_mode(alpha_mode) || !valid_act(act_z) ||
        !valid_act(act) || !valid_dtype(y_dtype))
        return TBN_ERR_INVALID_ARG;
    if (T > 0 && (!z || !y)) return TBN_ERR_INVALID_ARG;
    if (!aligned16(z) || !aligned16(y) || !aligned16(tile_bits)) return TBN_ERR_INVALID_ARG;
    if (bias && (reinterpret_cast<uintptr_t>(bias) & 3u)) return TBN_ERR_INVALID_ARG;
    const int64_t n = (int64_t)rz * kz;
    const int64_t N = n * out_f;
    if (N % k != 0) return TBN_ERR_SHAPE;
    if (T == 0) return TBN_OK;
    CompactArgs a;
    std::memset(&a, 0, sizeof(a));
    a.z = z; a.alpha_z = alpha_z; a.tile = tile_bits; a.alpha = alpha; a.bias = bias; a.y = y;
    a.T = T; a.q = N / k; a.rz = rz; a.kz = kz; a.m = out_f; a.k = k;
    a.alpha_mode_z = alpha_mode_z; a.act_z = act_z; a.alpha_mode = alpha_mode; a.act = act; a.y_dtype = y_dtype;
    if (!compact_linear_supported(a)) return TBN_ERR_UNSUPPORTED;
    int *st = device_status_ptr();
    if (!st) return TBN_ERR_CUDA;
    return launch_compact_linear(a, st, static_cast<cudaStream_t>(stream));
}

int tbn_layernorm_fwd(const void *x, int x_dtype, int64_t T, int32_t d, const float *gamma, const float *beta, float eps,
                      void *y, int y_dtype, void *stream)
{
    if (T < 0 || d <= 0 || !valid_dtype(x_dtype) || !valid_dtype(y_dtype) || !(eps >= 0.0f)) return TBN_ERR_INVALID_ARG;
    if (T == 0) return TBN_OK;
    if (!x || !y) return TBN_ERR_INVALID_ARG;
    return launch_layernorm(x, x_dtype, T, d, gamma, beta, eps, y, y_dtype, static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? TBN_OK : TBN_ERR_CUDA;
}

int tbn_attention_fwd(const void *qkv, int32_t Nb, int32_t S, int32_t heads, int32_t d_head, void *out, void *stream)
{
    if (Nb < 0 || S <= 0 || heads <= 0 || d_head <= 0) return TBN_ERR_INVALID_ARG;
    if (Nb == 0) return TBN_OK;
    if (!qkv || !out || !aligned16(qkv) || !aligned16(out)) return TBN_ERR_INVALID_ARG;
    if (!attention_supported(S, heads, d_head) || (int64_t)Nb * heads > 0x7fffffffLL) return TBN_ERR_UNSUPPORTED;
    return launch_attention(qkv, Nb, S, heads, d_head, out, device_status_ptr(), static_cast<cudaStream_t>(stream));
}

// workspace layout of the encoder block: [h: T x d][qkv: T x 3d][att: T x d][x1: T x d][f: T x mlp] bf16, then the
// largest scratch of its four linears
static size_t block_offsets(int64_t T, int32_t d, int32_t mlp, const int32_t *ks, size_t off[6])
{
    size_t o = 0;
    const size_t sizes[5] = {(size_t)T * d * 2, (size_t)T * 3 * d * 2, (size_t)T * d * 2, (size_t)T * d * 2, (size_t)T * mlp * 2};
    for (int i = 0; i < 5; ++i) { off[i] = o; o += round_up(sizes[i], 256); }
    off[5] = o;
    size_t scratch = 0;
    const int32_t shapes[4][2] = {{d, 3 * d}, {d, d}, {d, mlp}, {mlp, d}};
    for (int l = 0; l < 4; ++l) {
        const size_t b = tbn_linear_workspace_bytes(T, shapes[l][0], shapes[l][1], ks[l], TBN_BF16);
        scratch = b > scratch ? b : scratch;
    }
    return o + scratch;
}

size_t tbn_vit_block_workspace_bytes(int32_t Nb, int32_t S, int32_t d, int32_t mlp_dim, const int32_t *ks)
{
    if (Nb <= 0 || S <= 0 || d <= 0 || mlp_dim <= 0 || !ks) return 0;
    size_t off[6];
    return block_offsets((int64_t)Nb * S, d, mlp_dim, ks, off);
}

int tbn_vit_block_fwd(const void *x, int32_t Nb, int32_t S, int32_t d, int32_t heads, int32_t mlp_dim,
                      const uint32_t *const *tiles, const int32_t *ks, const float *const *alphas, const int *alpha_modes,
                      void *y, void *workspace, size_t workspace_bytes, void *stream)
{
    if (Nb < 0 || S <= 0 || d <= 0 || heads <= 0 || mlp_dim <= 0 || !tiles || !ks || !alphas || !alpha_modes)
        return TBN_ERR_INVALID_ARG;
    if (d % heads != 0) return TBN_ERR_SHAPE;
    for (int l = 0; l < 4; ++l)
        if (!tiles[l] || !alphas[l] || ks[l] <= 0 || !valid_alpha_mode(alpha_modes[l])) return TBN_ERR_INVALID_ARG;
    if (Nb == 0) return TBN_OK;
    if (!x || !y || !aligned16(x) || !aligned16(y)) return TBN_ERR_INVALID_ARG;
    if (!attention_supported(S, heads, d / heads)) return TBN_ERR_UNSUPPORTED;
    const int64_t T = (int64_t)Nb * S;
    size_t off[6];
    const size_t need = block_offsets(T, d, mlp_dim, ks, off);
    if (!workspace || !aligned16(workspace) || workspace_bytes < need) return TBN_ERR_WORKSPACE;
    char *ws = static_cast<char *>(workspace);
    void *h = ws + off[0], *qkv = ws + off[1], *att = ws + off[2], *x1 = ws + off[3], *f = ws + off[4], *scratch = ws + off[5];
    const size_t scratch_bytes = workspace_bytes - off[5];
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int B16 = TBN_BF16, AUTO = TBN_PATH_AUTO;
    int rc;
    if (launch_layernorm(x, B16, T, d, nullptr, nullptr, 1e-5f, h, B16, s) != cudaSuccess) return TBN_ERR_CUDA;
    rc = tbn_linear_fwd_path(h, B16, T, d, 3 * d, tiles[0], ks[0], alphas[0], alpha_modes[0], nullptr, TBN_ACT_NONE, qkv, B16,
                             scratch, scratch_bytes, stream, AUTO);
    if (rc != TBN_OK) return rc;
    rc = launch_attention(qkv, Nb, S, heads, d / heads, att, device_status_ptr(), s);
    if (rc != TBN_OK) return rc;
    if (add_layernorm_supported(d)) {
        // the projection writes into x1; one pass then forms x1 = x + projection and h = LayerNorm(x1)
        rc = tbn_linear_fwd_path(att, B16, T, d, d, tiles[1], ks[1], alphas[1], alpha_modes[1], nullptr, TBN_ACT_NONE, x1, B16,
                                 scratch, scratch_bytes, stream, AUTO);
        if (rc != TBN_OK) return rc;
        if (launch_add_layernorm(x, x1, x1, T, d, nullptr, nullptr, 1e-5f, h, s) != cudaSuccess) return TBN_ERR_CUDA;
    } else {
        rc = tbn_linear_res_fwd(att, B16, T, d, d, tiles[1], ks[1], alphas[1], alpha_modes[1], nullptr, TBN_ACT_NONE, x, x1, B16,
                                scratch, scratch_bytes, stream, AUTO);
        if (rc != TBN_OK) return rc;
        if (launch_layernorm(x1, B16, T, d, nullptr, nullptr, 1e-5f, h, B16, s) != cudaSuccess) return TBN_ERR_CUDA;
    }
    rc = tbn_linear_fwd_path(h, B16, T, d, mlp_dim, tiles[2], ks[2], alphas[2], alpha_modes[2], nullptr, TBN_ACT_GELU, f, B16,
                             scratch, scratch_bytes, stream, AUTO);
    if (rc != TBN_OK) return rc;
    return tbn_linear_res_fwd(f, B16, T, mlp_dim, d, tiles[3], ks[3], alphas[3], alpha_modes[3], nullptr, TBN_ACT_NONE, x1, y, B16,
                              scratch, scratch_bytes, stream, AUTO);
}

int tbn_conv2d_dense_fwd(const void *x, int x_dtype, int32_t Nb, int32_t Cin, int32_t H, int32_t Wd, int32_t Cout, int32_t kh,
                         int32_t kw, int32_t stride, int32_t pad, const float *weight, const float *bias, int act, void *y,
                         int y_dtype, void *stream)
{
    if (Nb < 0 || Cin <= 0 || H <= 0 || Wd <= 0 || Cout <= 0 || kh <= 0 || kw <= 0 || stride <= 0 || pad < 0) return TBN_ERR_INVALID_ARG;
    if (!weight || !valid_dtype(x_dtype) || !valid_dtype(y_dtype) || !valid_act(act)) return TBN_ERR_INVALID_ARG;
    if (H + 2 * pad < kh || Wd + 2 * pad < kw) return TBN_ERR_SHAPE;
    if (Nb == 0) return TBN_OK;
    if (!x || !y) return TBN_ERR_INVALID_ARG;
    if (!dense_conv_supported(Cin, kh, kw) || Cout > 65535 * 8) return TBN_ERR_UNSUPPORTED;
    return launch_dense_conv(x, x_dtype, weight, bias, y, y_dtype, Nb, Cin, H, Wd, Cout, kh, kw, stride, pad, act,
                             static_cast<cudaStream_t>(stream)) == cudaSuccess ? TBN_OK : TBN_ERR_CUDA;
}

int tbn_global_avgpool_fwd(const void *x, int x_dtype, int32_t Nb, int32_t C, int32_t H, int32_t Wd, void *y, int y_dtype, void *stream)
{
    if (Nb < 0 || C <= 0 || H <= 0 || Wd <= 0 || !valid_dtype(x_dtype) || !valid_dtype(y_dtype)) return TBN_ERR_INVALID_ARG;
    if (Nb == 0) return TBN_OK;
    if (!x || !y) return TBN_ERR_INVALID_ARG;
    if ((int64_t)H * Wd > 0x7fffffffLL) return TBN_ERR_UNSUPPORTED;
    return launch_global_avgpool(x, x_dtype, (int64_t)Nb * C, H * Wd, y, y_dtype, static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? TBN_OK : TBN_ERR_CUDA;
}

int tbn_avgpool_linear_fwd(const void *x, int x_dtype, int32_t Nb, int32_t C, int32_t H, int32_t Wd, const float *weight,
                           const float *bias, int32_t out_f, float *y, void *stream)
{
    if (Nb < 0 || C <= 0 || H <= 0 || Wd <= 0 || out_f <= 0 || !valid_dtype(x_dtype) || !weight) return TBN_ERR_INVALID_ARG;
    if (Nb == 0) return TBN_OK;
    if (!x || !y) return TBN_ERR_INVALID_ARG;
    if ((int64_t)H * Wd > 0x7fffffffLL || !avgpool_linear_supported(C)) return TBN_ERR_UNSUPPORTED;
    return launch_avgpool_linear(x, x_dtype, Nb, C, H * Wd, weight, bias, out_f, y, static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? TBN_OK : TBN_ERR_CUDA;
}

int64_t tbn_row_words(int32_t n) { return tbn_tile_words(n); }

int tbn_binarize_fwd(const void *x, int x_dtype, int64_t T, int32_t in_f, uint32_t *x_bits, float *beta, void *stream)
{
    if (T < 0 || in_f <= 0 || !valid_dtype(x_dtype)) return TBN_ERR_INVALID_ARG;
    if (T == 0) return TBN_OK;
    if (!x || !x_bits || !aligned16(x) || !aligned16(x_bits)) return TBN_ERR_INVALID_ARG;
    if (beta && (reinterpret_cast<uintptr_t>(beta) & 3u)) return TBN_ERR_INVALID_ARG;
    return launch_binarize(x, x_dtype, T, in_f, x_bits, beta, nullptr, nullptr, static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? TBN_OK : TBN_ERR_CUDA;
}

int tbn_binarize_bytes_fwd(const void *x, int x_dtype, int64_t T, int32_t in_f, uint32_t *x_bits, float *beta, void *x_bytes,
                           int32_t *x_pop, void *stream)
{
    if (T < 0 || in_f <= 0 || !valid_dtype(x_dtype)) return TBN_ERR_INVALID_ARG;
    if (in_f % 32 != 0) return TBN_ERR_UNSUPPORTED;
    if (T == 0) return TBN_OK;
    if (!x || !x_bits || !x_bytes || !x_pop || !aligned16(x) || !aligned16(x_bits) || !aligned16(x_bytes)) return TBN_ERR_INVALID_ARG;
    if ((beta && (reinterpret_cast<uintptr_t>(beta) & 3u)) || (reinterpret_cast<uintptr_t>(x_pop) & 3u)) return TBN_ERR_INVALID_ARG;
    return launch_binarize(x, x_dtype, T, in_f, x_bits, beta, x_bytes, x_pop, static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? TBN_OK : TBN_ERR_CUDA;
}

int tbn_linear_bin_fwd(const uint32_t *x_bits, int64_t T, int32_t in_f, int32_t out_f,
                       const uint32_t *tile_bits, int32_t k, const float *alpha, int alpha_mode,
                       const float *beta, const float *bias, int act, void *y, int y_dtype, void *stream, int path)
{
    if (T < 0 || in_f <= 0 || out_f <= 0 || k <= 0) return TBN_ERR_INVALID_ARG;
    if (!tile_bits || !alpha || !valid_alpha_mode(alpha_mode) || !valid_act(act)) return TBN_ERR_INVALID_ARG;
    if (!(valid_dtype(y_dtype) || y_dtype == TBN_I32)) return TBN_ERR_INVALID_ARG;
    if (path < TBN_PATH_AUTO || path > TBN_PATH_TENSOR) return TBN_ERR_INVALID_ARG;
    if (T > 0 && (!x_bits || !y)) return TBN_ERR_INVALID_ARG;
    if (!aligned16(x_bits) || !aligned16(y) || !aligned16(tile_bits)) return TBN_ERR_INVALID_ARG;
    if ((bias && (reinterpret_cast<uintptr_t>(bias) & 3u)) || (beta && (reinterpret_cast<uintptr_t>(beta) & 3u)))
        return TBN_ERR_INVALID_ARG;
    const int64_t N = (int64_t)in_f * out_f;
    if (N % k != 0) return TBN_ERR_SHAPE;
    if (T == 0) return TBN_OK;
    BinArgs a;
    std::memset(&a, 0, sizeof(a));
    a.x_bits = x_bits; a.tile = tile_bits; a.alpha = alpha; a.beta = beta; a.bias = bias; a.y = y;
    a.T = T; a.q = N / k; a.x_row_words = (int32_t)tbn_row_words(in_f); a.n = in_f; a.m = out_f; a.k = k;
    a.alpha_mode = alpha_mode; a.act = act; a.y_dtype = y_dtype;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (path == TBN_PATH_AUTO) {
        // A handful of tokens is bound by reading the tile once and by launch latency: the popcount kernel.  From a
        // few dozen tokens on the 8-bit tensor-core contraction is an order of magnitude faster than popcounts.
        path = (bin_tensor_supported(a) && T >= 32) ? TBN_PATH_TENSOR : TBN_PATH_GENERIC;
    }
    if (path == TBN_PATH_TENSOR) {
        if (!bin_tensor_supported(a)) return TBN_ERR_UNSUPPORTED;
        int *st = device_status_ptr();
        if (!st) return TBN_ERR_CUDA;
        return launch_bin_tensor(a, st, s);
    }
    if (path != TBN_PATH_GENERIC || !bin_popc_supported(a)) return TBN_ERR_UNSUPPORTED;
    return launch_bin_popc(a, s) == cudaSuccess ? TBN_OK : TBN_ERR_CUDA;
}

int tbn_bin_expand_fwd(const uint32_t *x_bits, int64_t T, int32_t in_f, void *x_bytes, int32_t *x_pop, void *stream)
{
    if (T < 0 || in_f <= 0) return TBN_ERR_INVALID_ARG;
    if (in_f % 32 != 0) return TBN_ERR_UNSUPPORTED;
    if (T == 0) return TBN_OK;
    if (!x_bits || !x_bytes || !x_pop || !aligned16(x_bits) || !aligned16(x_bytes) || (reinterpret_cast<uintptr_t>(x_pop) & 3u))
        return TBN_ERR_INVALID_ARG;
    return launch_bin_expand(x_bits, T, in_f, (int32_t)tbn_row_words(in_f), x_bytes, x_pop, static_cast<cudaStream_t>(stream)) ==
                   cudaSuccess ? TBN_OK : TBN_ERR_CUDA;
}

int tbn_linear_bin_bytes_fwd(const void *x_bytes, const int32_t *x_pop, int64_t T, int32_t in_f, int32_t out_f,
                             const uint32_t *tile_bits, int32_t k, const float *alpha, int alpha_mode,
                             const float *beta, const float *bias, int act, void *y, int y_dtype, void *stream)
{
    if (T < 0 || in_f <= 0 || out_f <= 0 || k <= 0) return TBN_ERR_INVALID_ARG;
    if (!tile_bits || !alpha || !valid_alpha_mode(alpha_mode) || !valid_act(act)) return TBN_ERR_INVALID_ARG;
    if (!(valid_dtype(y_dtype) || y_dtype == TBN_I32)) return TBN_ERR_INVALID_ARG;
    if (T > 0 && (!x_bytes || !x_pop || !y)) return TBN_ERR_INVALID_ARG;
    if (!aligned16(x_bytes) || !aligned16(y) || !aligned16(tile_bits) || (reinterpret_cast<uintptr_t>(x_pop) & 3u))
        return TBN_ERR_INVALID_ARG;
    if ((bias && (reinterpret_cast<uintptr_t>(bias) & 3u)) || (beta && (reinterpret_cast<uintptr_t>(beta) & 3u)))
        return TBN_ERR_INVALID_ARG;
    const int64_t N = (int64_t)in_f * out_f;
    if (N % k != 0) return TBN_ERR_SHAPE;
    if (T == 0) return TBN_OK;
    BinArgs a;
    std::memset(&a, 0, sizeof(a));
    a.x_bytes = x_bytes; a.x_pop = x_pop; a.tile = tile_bits; a.alpha = alpha; a.beta = beta; a.bias = bias; a.y = y;
    a.T = T; a.q = N / k; a.x_row_words = (int32_t)tbn_row_words(in_f); a.n = in_f; a.m = out_f; a.k = k;
    a.alpha_mode = alpha_mode; a.act = act; a.y_dtype = y_dtype;
    if (!bin_tensor_supported(a)) return TBN_ERR_UNSUPPORTED;
    int *st = device_status_ptr();
    if (!st) return TBN_ERR_CUDA;
    return launch_bin_tensor(a, st, static_cast<cudaStream_t>(stream));
}

int tbn_debug_force_bin_config(int candidate) { return force_bin_config(candidate); }

int tbn_debug_force_attention_path(int path) { return force_attention_path(path); }

int tbn_last_device_status(void *stream, int *code, int *detail)
{
    if (!code || !detail) return TBN_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int *st = device_status_ptr();
    if (!st) return TBN_ERR_CUDA;
    int host[4] = {0, 0, 0, 0};
    if (cudaStreamSynchronize(s) != cudaSuccess) return TBN_ERR_CUDA;
    if (cudaMemcpy(host, st, sizeof(host), cudaMemcpyDeviceToHost) != cudaSuccess) return TBN_ERR_CUDA;
    *code = host[0];
    *detail = host[1];
    if (host[0] != 0 && cudaMemset(st, 0, 2 * sizeof(int)) != cudaSuccess) return TBN_ERR_CUDA;   // code and detail only
    return TBN_OK;
}

int tbn_debug_set_wait_limit_us(int limit_us)
{
    if (limit_us < 0) return TBN_ERR_INVALID_ARG;
    int *st = device_status_ptr();
    if (!st) return TBN_ERR_CUDA;
    if (cudaDeviceSynchronize() != cudaSuccess) return TBN_ERR_CUDA;      // no kernel may be reading the word meanwhile
    return cudaMemcpy(st + 2, &limit_us, sizeof(int), cudaMemcpyHostToDevice) == cudaSuccess ? TBN_OK : TBN_ERR_CUDA;
}

int tbn_debug_wait_timeout_probe(int detail, void *stream)
{
    int *st = device_status_ptr();
    if (!st) return TBN_ERR_CUDA;
    return launch_wait_probe(st, detail, static_cast<cudaStream_t>(stream)) == cudaSuccess ? TBN_OK : TBN_ERR_CUDA;
}

int tbn_debug_force_linear_config(int candidate, int splits) { return force_linear_config(candidate, splits); }

int tbn_debug_force_mlp_layerwise(int on)
{
    g_mlp_layerwise.store(on ? 1 : 0);
    return TBN_OK;
}

int tbn_debug_record_status(int code, int detail, void *stream)
{
    int *st = device_status_ptr();
    if (!st) return TBN_ERR_CUDA;
    record_status_kernel<<<1, 1, 0, static_cast<cudaStream_t>(stream)>>>(st, code, detail);
    return cudaGetLastError() == cudaSuccess ? TBN_OK : TBN_ERR_CUDA;
}

}  // extern "C"
