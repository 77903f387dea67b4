// Training-side tiling module (Sec. 3): the forward builds the scaled tiled weight B_hat from the full-precision
// parameters in one read of W (Eq. 1-5, then Eq. 6 / Eq. 7-8), the backward passes the gradient straight through
// the non-differentiable steps and differentiates the scaling factors as ordinary functions.
//
//   forward : tile, alpha = aggregate(W, A)        (prepare.cu: W and A are read once)
//             B_hat[j*q + i] = alpha_j * t_i       (this file: written from the bits, W is not read again)
//   backward: G = dL/dB_hat
//             dalpha_j = sum_i G[j*q + i] * t_i
//             dW[f]    = alpha_j * G[f]                              straight-through: dL/dW := dL/dB
//             dS[f]    = dalpha_j * sign(S[f]) / q                    S = A, or W without a separate tensor (then added to dW)
//
// All kernels are streaming and HBM-bound; reductions add block partial sums in a fixed order (fp64), so results
// are reproducible from run to run.
#include "common.cuh"

namespace tbn {

namespace {

constexpr int kTrThreads = 256;
constexpr int kTrIter = 4;
constexpr int kTrChunk = kTrThreads * 4 * kTrIter;     // 4096 tile positions per block and repetition

__device__ __forceinline__ void store4(float *p, float a, float b, float c, float d) {
    *reinterpret_cast<float4 *>(p) = make_float4(a, b, c, d);
}
__device__ __forceinline__ void store4(__nv_bfloat16 *p, float a, float b, float c, float d) {
    const __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
    *reinterpret_cast<uint2 *>(p) = make_uint2(*reinterpret_cast<const uint32_t *>(&lo), *reinterpret_cast<const uint32_t *>(&hi));
}

// grid (chunks of the tile, repetitions): no division or modulo per element, 16-byte stores when q % 4 == 0
template <typename OT>
__global__ void __launch_bounds__(kTrThreads)
tile_expand_kernel(const uint32_t *__restrict__ tile, int64_t q, int32_t k, const float *__restrict__ alpha, int per_tile,
                   OT *__restrict__ B_hat)
{
    const bool vec = (q & 3) == 0;
    for (int32_t j = blockIdx.y; j < k; j += gridDim.y) {
        const float a = per_tile ? __ldg(alpha + j) : __ldg(alpha);
        OT *dst = B_hat + (int64_t)j * q;
#pragma unroll
        for (int it = 0; it < kTrIter; ++it) {
            const int64_t i0 = (int64_t)blockIdx.x * kTrChunk + ((int64_t)it * kTrThreads + threadIdx.x) * 4;
            if (i0 >= q) break;
            const uint32_t nib = __ldg(tile + (i0 >> 5)) >> (uint32_t)(i0 & 31);     // 4 positions never straddle a word
            const float v0 = (nib & 1u) ? a : -a, v1 = (nib & 2u) ? a : -a, v2 = (nib & 4u) ? a : -a, v3 = (nib & 8u) ? a : -a;
            if (vec) {
                store4(dst + i0, v0, v1, v2, v3);
            } else {
                const float v[4] = {v0, v1, v2, v3};
                for (int e = 0; e < 4 && i0 + e < q; ++e) store_from_float(dst, i0 + e, v[e]);
            }
        }
    }
}

// dalpha partial sums: partial[j * chunks + chunk] = sum over the chunk of G[j*q + i] * t_i
__global__ void __launch_bounds__(kTrThreads)
tile_bwd_partial_kernel(const float *__restrict__ G, const uint32_t *__restrict__ tile, int64_t q, int32_t k,
                        double *__restrict__ partial)
{
    __shared__ double warp_sum[kTrThreads / 32];
    const bool vec = (q & 3) == 0;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int32_t j = blockIdx.y; j < k; j += gridDim.y) {
        const float *g = G + (int64_t)j * q;
        float acc = 0.0f;
#pragma unroll
        for (int it = 0; it < kTrIter; ++it) {
            const int64_t i0 = (int64_t)blockIdx.x * kTrChunk + ((int64_t)it * kTrThreads + threadIdx.x) * 4;
            if (i0 >= q) break;
            const uint32_t nib = __ldg(tile + (i0 >> 5)) >> (uint32_t)(i0 & 31);
            float v[4] = {0.f, 0.f, 0.f, 0.f};
            if (vec) {
                const float4 t = __ldg(reinterpret_cast<const float4 *>(g + i0));
                v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
            } else {
                for (int e = 0; e < 4 && i0 + e < q; ++e) v[e] = __ldg(g + i0 + e);
            }
#pragma unroll
            for (int e = 0; e < 4; ++e) acc += ((nib >> e) & 1u) ? v[e] : -v[e];
        }
        double d = (double)acc;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) d += __shfl_xor_sync(0xffffffffu, d, off);
        if (lane == 0) warp_sum[warp] = d;
        __syncthreads();
        if (threadIdx.x == 0) {
            double t = 0.0;
#pragma unroll
            for (int w = 0; w < kTrThreads / 32; ++w) t += warp_sum[w];
            partial[(int64_t)j * gridDim.x + blockIdx.x] = t;
        }
        __syncthreads();
    }
}

// one block per scaling factor: adds its partial sums in a fixed order
__global__ void __launch_bounds__(kTrThreads)
tile_bwd_final_kernel(const double *__restrict__ partial, int64_t count_per_group, int32_t groups, double *__restrict__ dalpha,
                      float *__restrict__ dalpha_out)
{
    __shared__ double red[kTrThreads];
    for (int32_t j = blockIdx.x; j < groups; j += gridDim.x) {
        double t = 0.0;
        for (int64_t b = threadIdx.x; b < count_per_group; b += kTrThreads) t += partial[(int64_t)j * count_per_group + b];
        red[threadIdx.x] = t;
        __syncthreads();
        for (int off = kTrThreads / 2; off > 0; off >>= 1) {
            if ((int)threadIdx.x < off) red[threadIdx.x] += red[threadIdx.x + off];
            __syncthreads();
        }
        if (threadIdx.x == 0) {
            dalpha[j] = red[0];
            if (dalpha_out) dalpha_out[j] = (float)red[0];
        }
        __syncthreads();
    }
}

__device__ __forceinline__ float sign_of(float v) { return v > 0.0f ? 1.0f : (v < 0.0f ? -1.0f : 0.0f); }

// dW = alpha_j * G (+ dalpha_j * sign(W) / count without a separate A);  dA = dalpha_j * sign(A) / count
template <bool HAS_A>
__global__ void __launch_bounds__(kTrThreads)
tile_bwd_apply_kernel(const float *__restrict__ G, const float *__restrict__ W, const float *__restrict__ A, int64_t q, int32_t k,
                      const float *__restrict__ alpha, const double *__restrict__ dalpha, int per_tile, double inv_count,
                      float *__restrict__ dW, float *__restrict__ dA)
{
    const bool vec = (q & 3) == 0;
    for (int32_t j = blockIdx.y; j < k; j += gridDim.y) {
        const float a = per_tile ? __ldg(alpha + j) : __ldg(alpha);
        const float ds = (float)(dalpha[per_tile ? j : 0] * inv_count);
        const int64_t base = (int64_t)j * q;
#pragma unroll
        for (int it = 0; it < kTrIter; ++it) {
            const int64_t i0 = (int64_t)blockIdx.x * kTrChunk + ((int64_t)it * kTrThreads + threadIdx.x) * 4;
            if (i0 >= q) break;
            const int64_t f = base + i0;
            if (vec) {
                const float4 g = __ldg(reinterpret_cast<const float4 *>(G + f));
                const float4 s = __ldg(reinterpret_cast<const float4 *>((HAS_A ? A : W) + f));
                if (HAS_A) {
                    store4(dW + f, __fmul_rn(a, g.x), __fmul_rn(a, g.y), __fmul_rn(a, g.z), __fmul_rn(a, g.w));
                    store4(dA + f, ds * sign_of(s.x), ds * sign_of(s.y), ds * sign_of(s.z), ds * sign_of(s.w));
                } else {
                    store4(dW + f, fmaf(a, g.x, ds * sign_of(s.x)), fmaf(a, g.y, ds * sign_of(s.y)),
                           fmaf(a, g.z, ds * sign_of(s.z)), fmaf(a, g.w, ds * sign_of(s.w)));
                }
            } else {
                for (int e = 0; e < 4 && i0 + e < q; ++e) {
                    const float g = __ldg(G + f + e), s = __ldg((HAS_A ? A : W) + f + e);
                    if (HAS_A) { dW[f + e] = __fmul_rn(a, g); dA[f + e] = ds * sign_of(s); }
                    else dW[f + e] = fmaf(a, g, ds * sign_of(s));
                }
            }
        }
    }
}

inline dim3 train_grid(int64_t q, int32_t k)
{
    const int64_t chunks = (q + kTrChunk - 1) / kTrChunk;
    return dim3((unsigned)chunks, (unsigned)(k < 65535 ? k : 65535));
}

}  // namespace

cudaError_t launch_tile_expand(const uint32_t *tile, int64_t N, int32_t k, const float *alpha, int per_tile, void *B_hat,
                               int b_dtype, cudaStream_t s)
{
    const int64_t q = N / k;
    if ((q + kTrChunk - 1) / kTrChunk > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    if (b_dtype == TBN_BF16)
        tile_expand_kernel<__nv_bfloat16><<<train_grid(q, k), kTrThreads, 0, s>>>(tile, q, k, alpha, per_tile,
                                                                                 static_cast<__nv_bfloat16 *>(B_hat));
    else
        tile_expand_kernel<float><<<train_grid(q, k), kTrThreads, 0, s>>>(tile, q, k, alpha, per_tile, static_cast<float *>(B_hat));
    return cudaGetLastError();
}

size_t tile_bwd_workspace_bytes(int64_t N, int32_t k)
{
    const int64_t q = N / k;
    const int64_t chunks = (q + kTrChunk - 1) / kTrChunk;
    return (size_t)k * (size_t)chunks * sizeof(double) + (size_t)k * sizeof(double);     // partial sums, then dalpha
}

cudaError_t launch_tile_bwd(const float *G, const uint32_t *tile, const float *alpha, const float *W, const float *A,
                            int64_t N, int32_t k, int per_tile, float *dW, float *dA, float *dalpha_out, void *workspace,
                            cudaStream_t s)
{
    const int64_t q = N / k;
    const int64_t chunks = (q + kTrChunk - 1) / kTrChunk;
    if (chunks > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    double *partial = static_cast<double *>(workspace);
    double *dalpha = partial + (size_t)k * chunks;
    // with more than 65535 repetitions grid.y wraps; the partial array is indexed by (j, chunk) all the same
    tile_bwd_partial_kernel<<<train_grid(q, k), kTrThreads, 0, s>>>(G, tile, q, k, partial);
    const int32_t groups = per_tile ? k : 1;
    const int64_t per_group = per_tile ? chunks : (int64_t)k * chunks;
    tile_bwd_final_kernel<<<(unsigned)(groups < 148 * 8 ? groups : 148 * 8), kTrThreads, 0, s>>>(partial, per_group, groups, dalpha,
                                                                                              dalpha_out);
    const double inv_count = 1.0 / (per_tile ? (double)q : (double)N);
    if (A)
        tile_bwd_apply_kernel<true><<<train_grid(q, k), kTrThreads, 0, s>>>(G, W, A, q, k, alpha, dalpha, per_tile, inv_count, dW, dA);
    else
        tile_bwd_apply_kernel<false><<<train_grid(q, k), kTrThreads, 0, s>>>(G, W, nullptr, q, k, alpha, dalpha, per_tile, inv_count, dW,
                                                                            nullptr);
    return cudaGetLastError();
}

}  // namespace tbn
