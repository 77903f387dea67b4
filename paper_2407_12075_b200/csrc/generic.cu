// Generic CUDA-core forward for a tiled layer: any shape, any alignment of the tile length q
// against the row length n, fully-connected or convolution.  It is the correctness backstop of the
// library (it never uses the replicated-row shortcut, so it also cross-checks the kernels that do).
//
// The kernel walks the flat weight index f = o*n + j exactly as Algorithm 1 does: a tile index that
// wraps at q and an alpha index that advances at every wrap.  Because alpha may change in the middle
// of a row, each thread keeps a running segment sum that is scaled by the current alpha and folded
// into the row total whenever the tile index wraps (and once at the end of the row).
//
// Block = 128 threads = 128 output rows x 16 tokens.  The activation chunk (32 x 16 values) is staged
// in shared memory as fp32 and read with broadcast 128-bit loads; the tile word is fetched through the
// read-only path once per 32 weights.
#include "common.cuh"

namespace tbn {

namespace {

constexpr int kRows = 128;   // output rows per block (one per thread)
constexpr int kTok = 16;     // tokens per block
constexpr int kKC = 32;      // contraction elements per shared-memory chunk

__device__ __forceinline__ float fetch_x(const LayerArgs &a, int64_t tok, int32_t j)
{
    if (tok >= a.T || j >= a.n) return 0.0f;
    int64_t idx;
    if (!a.is_conv) {
        idx = tok * a.n + j;
    } else {
        // token -> (image, out row, out col); j -> (in channel, filter row, filter col)
        const int32_t ow = (int32_t)(tok % a.Wo);
        const int64_t r = tok / a.Wo;
        const int32_t oh = (int32_t)(r % a.Ho);
        const int64_t b = r / a.Ho;
        const int32_t v = j % a.kw;
        const int32_t u = (j / a.kw) % a.kh;
        const int32_t ci = j / (a.kw * a.kh);
        const int32_t ih = oh * a.stride + u - a.pad;
        const int32_t iw = ow * a.stride + v - a.pad;
        if (ih < 0 || ih >= a.H || iw < 0 || iw >= a.Wd) return 0.0f;   // zero padding
        idx = ((b * a.Cin + ci) * a.H + ih) * (int64_t)a.Wd + iw;
    }
    return a.x_dtype == TBN_BF16 ? load_as_float(static_cast<const __nv_bfloat16 *>(a.x), idx)
                                 : load_as_float(static_cast<const float *>(a.x), idx);
}

__global__ void __launch_bounds__(kRows)
generic_kernel(const LayerArgs a)
{
    // xs[kk][4 groups of 4 tokens]; the group index is XOR-swizzled with kk to spread the banks on store
    __shared__ __align__(16) float xs[kKC][kTok];

    const int tid = threadIdx.x;
    const int32_t o = blockIdx.y * kRows + tid;
    const int64_t t0 = (int64_t)blockIdx.x * kTok;
    const bool active = o < a.m;

    // position of this row's first weight inside the tile, and its alpha index
    const int64_t f0 = (int64_t)(active ? o : 0) * a.n;
    int64_t idx = f0 % a.q;
    int64_t aidx = f0 / a.q;
    const bool per_tile = a.alpha_mode == TBN_ALPHA_PER_TILE;
    // a full-precision tile is used as it is: the weight is t[idx] and every scaling factor is 1
    const bool fp = a.fp_tile != nullptr;
    const float *fp32_tile = static_cast<const float *>(a.fp_tile);
    const __nv_bfloat16 *bf16_tile = static_cast<const __nv_bfloat16 *>(a.fp_tile);
    float alpha_cur = fp ? 1.0f : per_tile ? __ldg(a.alpha + aidx) : __ldg(a.alpha);
    uint32_t word = fp ? 0u : __ldg(a.tile + (idx >> 5));

    float seg[kTok], tot[kTok];
#pragma unroll
    for (int t = 0; t < kTok; ++t) { seg[t] = 0.0f; tot[t] = 0.0f; }

    for (int32_t k0 = 0; k0 < a.n; k0 += kKC) {
        __syncthreads();
#pragma unroll
        for (int i = 0; i < kKC * kTok / kRows; ++i) {
            const int e = tid + i * kRows;
            const int kk = e % kKC, t = e / kKC;
            const int g = (t >> 2) ^ (kk & 3);
            xs[kk][g * 4 + (t & 3)] = fetch_x(a, t0 + t, k0 + kk);
        }
        __syncthreads();
        if (!active) continue;
        const int kc = min(kKC, a.n - k0);
        for (int kk = 0; kk < kc; ++kk) {
            const float sgn = fp ? (a.fp_tile_dtype == TBN_BF16 ? load_as_float(bf16_tile, idx) : __ldg(fp32_tile + idx))
                                 : ((word >> (uint32_t)(idx & 31)) & 1u) ? 1.0f : -1.0f;
#pragma unroll
            for (int g = 0; g < 4; ++g) {
                const float4 xv = *reinterpret_cast<const float4 *>(&xs[kk][(g ^ (kk & 3)) * 4]);
                seg[g * 4 + 0] = fmaf(sgn, xv.x, seg[g * 4 + 0]);   // binary tile: +-1 * x is exact
                seg[g * 4 + 1] = fmaf(sgn, xv.y, seg[g * 4 + 1]);
                seg[g * 4 + 2] = fmaf(sgn, xv.z, seg[g * 4 + 2]);
                seg[g * 4 + 3] = fmaf(sgn, xv.w, seg[g * 4 + 3]);
            }
            ++idx;
            if (idx == a.q) {                    // end of the tile: next repetition, next alpha
#pragma unroll
                for (int t = 0; t < kTok; ++t) { tot[t] = fmaf(alpha_cur, seg[t], tot[t]); seg[t] = 0.0f; }
                idx = 0;
                ++aidx;
                if (!fp && per_tile && aidx < a.k) alpha_cur = __ldg(a.alpha + aidx);
                if (!fp) word = __ldg(a.tile);
            } else if (!fp && (idx & 31) == 0) {
                word = __ldg(a.tile + (idx >> 5));
            }
        }
    }
    if (!active) return;

    const float b = a.bias ? __ldg(a.bias + o) : 0.0f;
#pragma unroll
    for (int t = 0; t < kTok; ++t) {
        const int64_t tok = t0 + t;
        if (tok >= a.T) break;
        float v = apply_act(fmaf(alpha_cur, seg[t], tot[t]) + b, a.act);
        int64_t yi;
        if (!a.is_conv) {
            yi = tok * a.m + o;
        } else {
            const int64_t hw = (int64_t)a.Ho * a.Wo;
            yi = ((tok / hw) * a.m + o) * hw + tok % hw;
        }
        if (a.residual != nullptr)
            v += a.y_dtype == TBN_BF16 ? load_as_float(static_cast<const __nv_bfloat16 *>(a.residual), yi)
                                       : load_as_float(static_cast<const float *>(a.residual), yi);
        if (a.y_dtype == TBN_BF16) store_from_float(static_cast<__nv_bfloat16 *>(a.y), yi, v);
        else store_from_float(static_cast<float *>(a.y), yi, v);
    }
}

}  // namespace

cudaError_t launch_generic(const LayerArgs &a, cudaStream_t s)
{
    const int64_t gx = (a.T + kTok - 1) / kTok;                  // tokens on x (up to 2^31 - 1 blocks)
    const int64_t gy = ((int64_t)a.m + kRows - 1) / kRows;       // output rows on y
    if (gx > 0x7fffffffLL || gy > 65535) return cudaErrorInvalidConfiguration;
    generic_kernel<<<dim3((unsigned)gx, (unsigned)gy), kRows, 0, s>>>(a);
    return cudaGetLastError();
}

}  // namespace tbn
