// Tile construction kernels: chunk-sum + threshold + bit packing (Eq. 1-3), scaling factors
// (Eq. 6-8), packing of an existing tile, and the test-only expansion (Eq. 4-5).
//
// All of them are streaming, HBM-bound kernels: W (and A) are read exactly once with coalesced
// 128-byte warp accesses, the packed tile is written once.
#include "common.cuh"

namespace tbn {

namespace {

constexpr int kAggThreads = 256;
constexpr int kAggVec = 4;                                // columns per 16-byte load
constexpr int kAggIter = 4;                               // 16-byte loads per thread and tile repetition
constexpr int kAggCols = kAggThreads * kAggVec * kAggIter;   // columns per block (4096)
constexpr int kAggJB = 8;                                 // repetitions whose |.| sums are reduced together

struct AggScratch {          // layout of the caller's workspace
    unsigned int ticket;     // blocks that have published their partial sums
    unsigned int pad[3];
    // followed by k * gridDim.x doubles: partial[j * blocks + b]
};

// Block b owns columns [b*kAggCols, (b+1)*kAggCols) of the k x q view of W; a thread owns kAggIter groups
// of 4 consecutive columns.  For every column it forms s = ((0 + W[0][c]) + W[1][c]) + ... in fp32, one
// rounding per add, exactly the sequential sum the CPU definition uses, so the sign -- and therefore the
// bit -- is identical.  Alongside, the block accumulates |S| per tile in fp64 and publishes it (one
// block-level reduction per kAggJB repetitions, so up to 32 independent 16-byte loads per thread are in
// flight between synchronisations); the last block to finish adds the partials of all blocks in a fixed
// order, which makes alpha reproducible from run to run.  VEC selects 16-byte loads (q % 4 == 0).
template <bool VEC>
__global__ void __launch_bounds__(kAggThreads)
aggregate_kernel(const float *__restrict__ W, const float *__restrict__ A, int64_t q, int32_t k,
                 int per_tile, uint32_t *__restrict__ tile_bits, int64_t n_words,
                 float *__restrict__ alpha, AggScratch *scratch)
{
    __shared__ double warp_part[kAggJB][kAggThreads / 32];
    __shared__ double red[kAggThreads];
    __shared__ unsigned int s_ticket;

    const int tid = threadIdx.x;
    const int lane = tid & 31, warp = tid >> 5;
    const int64_t base = (int64_t)blockIdx.x * kAggCols;
    double *partial = reinterpret_cast<double *>(scratch + 1);
    const unsigned int blocks = gridDim.x;

    float s[kAggIter][kAggVec];
#pragma unroll
    for (int it = 0; it < kAggIter; ++it)
#pragma unroll
        for (int e = 0; e < kAggVec; ++e) s[it][e] = 0.0f;

    for (int32_t j0 = 0; j0 < k; j0 += kAggJB) {
        float a_abs[kAggJB];
#pragma unroll
        for (int jj = 0; jj < kAggJB; ++jj) {
            a_abs[jj] = 0.0f;
            const int32_t j = j0 + jj;
            if (j >= k) continue;
            const int64_t row = (int64_t)j * q;
#pragma unroll
            for (int it = 0; it < kAggIter; ++it) {
                const int64_t c = base + ((int64_t)it * kAggThreads + tid) * kAggVec;
                float w[kAggVec], av[kAggVec];
                if (VEC) {
                    if (c < q) {                       // q % 4 == 0: the whole group is in range
                        const float4 t = __ldg(reinterpret_cast<const float4 *>(W + row + c));
                        w[0] = t.x; w[1] = t.y; w[2] = t.z; w[3] = t.w;
                        if (A) {
                            const float4 u = __ldg(reinterpret_cast<const float4 *>(A + row + c));
                            av[0] = u.x; av[1] = u.y; av[2] = u.z; av[3] = u.w;
                        }
                    } else {
#pragma unroll
                        for (int e = 0; e < kAggVec; ++e) { w[e] = 0.0f; av[e] = 0.0f; }
                    }
                } else {
#pragma unroll
                    for (int e = 0; e < kAggVec; ++e) {
                        const bool in = c + e < q;
                        w[e] = in ? __ldg(W + row + c + e) : 0.0f;
                        av[e] = (in && A) ? __ldg(A + row + c + e) : 0.0f;
                    }
                }
#pragma unroll
                for (int e = 0; e < kAggVec; ++e) {
                    s[it][e] = __fadd_rn(s[it][e], w[e]);          // never fused, never reassociated
                    a_abs[jj] += fabsf(A ? av[e] : w[e]);
                }
            }
        }
        // block-level reduction of the group's |.| sums
#pragma unroll
        for (int jj = 0; jj < kAggJB; ++jj) {
            double d = (double)a_abs[jj];
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) d += __shfl_xor_sync(0xffffffffu, d, off);
            if (lane == 0) warp_part[jj][warp] = d;
        }
        __syncthreads();
        if (tid < kAggJB && j0 + tid < k) {
            double t = 0.0;
#pragma unroll
            for (int w = 0; w < kAggThreads / 32; ++w) t += warp_part[tid][w];
            partial[(int64_t)(j0 + tid) * blocks + blockIdx.x] = t;
        }
        __syncthreads();
    }

    // Eq. 3 + packing: a thread holds 4 consecutive columns (a nibble), 8 lanes make one 32-bit word.
#pragma unroll
    for (int it = 0; it < kAggIter; ++it) {
        uint32_t nib = 0;
#pragma unroll
        for (int e = 0; e < kAggVec; ++e) nib |= (s[it][e] > 0.0f ? 1u : 0u) << e;   // NaN and +-0 give 0
        uint32_t word = nib << (4 * (lane & 7));
        word |= __shfl_xor_sync(0xffffffffu, word, 1);
        word |= __shfl_xor_sync(0xffffffffu, word, 2);
        word |= __shfl_xor_sync(0xffffffffu, word, 4);
        const int64_t c0 = base + ((int64_t)it * kAggThreads + (tid & ~7)) * kAggVec;   // first column of the word
        const int64_t widx = c0 >> 5;
        if ((lane & 7) == 0 && widx < n_words) tile_bits[widx] = word;
    }

    // Publish, then let the last block reduce.
    __threadfence();
    __syncthreads();
    if (tid == 0) s_ticket = atomicAdd(&scratch->ticket, 1u);
    __syncthreads();
    if (s_ticket != blocks - 1) return;
    __threadfence();

    const volatile double *vp = partial;
    if (per_tile) {
        for (int32_t j = 0; j < k; ++j) {
            double t = 0.0;
            for (unsigned int b = tid; b < blocks; b += kAggThreads) t += vp[(int64_t)j * blocks + b];
            red[tid] = t;
            __syncthreads();
            for (int off = kAggThreads / 2; off > 0; off >>= 1) {
                if (tid < off) red[tid] += red[tid + off];
                __syncthreads();
            }
            if (tid == 0) alpha[j] = (float)(red[0] / (double)q);
            __syncthreads();
        }
    } else {
        double t = 0.0;
        const int64_t total = (int64_t)k * blocks;
        for (int64_t b = tid; b < total; b += kAggThreads) t += vp[b];
        red[tid] = t;
        __syncthreads();
        for (int off = kAggThreads / 2; off > 0; off >>= 1) {
            if (tid < off) red[tid] += red[tid + off];
            __syncthreads();
        }
        if (tid == 0) alpha[0] = (float)(red[0] / ((double)q * (double)k));
    }
}

// Streaming form for k <= kAggStreamK: a fixed grid of blocks walks the column chunks (chunk = block, block + grid,
// ...), so the per-block cost of publishing partial sums, the fence and the ticket is paid once per block instead of
// once per 4096 columns, and a thread keeps its |.| sums per tile in fp64 registers across chunks.  Loads are
// issued kAggRows rows x kAggIter groups at a time (8 independent 16-byte loads per thread and source) before the
// sequential fp32 adds that the bit rule requires.
constexpr int kAggStreamK = 16;
constexpr int kAggRows = 2;

template <bool VEC, bool HAS_A>
__global__ void __launch_bounds__(kAggThreads, 2)
aggregate_stream_kernel(const float *__restrict__ W, const float *__restrict__ A, int64_t q, int32_t k,
                        int per_tile, uint32_t *__restrict__ tile_bits, int64_t n_words,
                        float *__restrict__ alpha, AggScratch *scratch, int64_t n_chunks)
{
    __shared__ double warp_part[kAggStreamK][kAggThreads / 32];
    __shared__ double red[kAggThreads];
    __shared__ unsigned int s_ticket;

    const int tid = threadIdx.x;
    const int lane = tid & 31, warp = tid >> 5;
    double *partial = reinterpret_cast<double *>(scratch + 1);
    const unsigned int blocks = gridDim.x;

    double acc[kAggStreamK];
#pragma unroll
    for (int j = 0; j < kAggStreamK; ++j) acc[j] = 0.0;

    for (int64_t chunk = blockIdx.x; chunk < n_chunks; chunk += blocks) {
        const int64_t base = chunk * kAggCols;
        float s[kAggIter][kAggVec];
#pragma unroll
        for (int it = 0; it < kAggIter; ++it)
#pragma unroll
            for (int e = 0; e < kAggVec; ++e) s[it][e] = 0.0f;

#pragma unroll
        for (int j0 = 0; j0 < kAggStreamK; j0 += kAggRows) {
            if (j0 >= k) break;                           // uniform
            float w[kAggRows][kAggIter][kAggVec];
            float av[HAS_A ? kAggRows : 1][kAggIter][kAggVec];
#pragma unroll
            for (int jj = 0; jj < kAggRows; ++jj) {
                const bool row_ok = j0 + jj < k;
                const int64_t row = (int64_t)(row_ok ? j0 + jj : 0) * q;
#pragma unroll
                for (int it = 0; it < kAggIter; ++it) {
                    const int64_t c = base + ((int64_t)it * kAggThreads + tid) * kAggVec;
                    if (VEC) {
                        float4 t = make_float4(0.f, 0.f, 0.f, 0.f), u = t;
                        if (row_ok && c < q) {            // q % 4 == 0: the whole group is in range
                            t = __ldg(reinterpret_cast<const float4 *>(W + row + c));
                            if (HAS_A) u = __ldg(reinterpret_cast<const float4 *>(A + row + c));
                        }
                        w[jj][it][0] = t.x; w[jj][it][1] = t.y; w[jj][it][2] = t.z; w[jj][it][3] = t.w;
                        if (HAS_A) { av[jj][it][0] = u.x; av[jj][it][1] = u.y; av[jj][it][2] = u.z; av[jj][it][3] = u.w; }
                    } else {
#pragma unroll
                        for (int e = 0; e < kAggVec; ++e) {
                            const bool in = row_ok && c + e < q;
                            w[jj][it][e] = in ? __ldg(W + row + c + e) : 0.0f;
                            if (HAS_A) av[jj][it][e] = in ? __ldg(A + row + c + e) : 0.0f;
                        }
                    }
                }
            }
#pragma unroll
            for (int jj = 0; jj < kAggRows; ++jj) {
                if (j0 + jj >= k) break;                  // uniform; a skipped row must not enter the fp32 sum
                float ab = 0.0f;
#pragma unroll
                for (int it = 0; it < kAggIter; ++it)
#pragma unroll
                    for (int e = 0; e < kAggVec; ++e) {
                        s[it][e] = __fadd_rn(s[it][e], w[jj][it][e]);      // never fused, never reassociated
                        ab += fabsf(HAS_A ? av[HAS_A ? jj : 0][it][e] : w[jj][it][e]);
                    }
                acc[j0 + jj] += (double)ab;
            }
        }

        // Eq. 3 + packing: a thread holds 4 consecutive columns (a nibble), 8 lanes make one 32-bit word.
#pragma unroll
        for (int it = 0; it < kAggIter; ++it) {
            uint32_t nib = 0;
#pragma unroll
            for (int e = 0; e < kAggVec; ++e) nib |= (s[it][e] > 0.0f ? 1u : 0u) << e;   // NaN and +-0 give 0
            uint32_t word = nib << (4 * (lane & 7));
            word |= __shfl_xor_sync(0xffffffffu, word, 1);
            word |= __shfl_xor_sync(0xffffffffu, word, 2);
            word |= __shfl_xor_sync(0xffffffffu, word, 4);
            const int64_t c0 = base + ((int64_t)it * kAggThreads + (tid & ~7)) * kAggVec;
            const int64_t widx = c0 >> 5;
            if ((lane & 7) == 0 && widx < n_words) tile_bits[widx] = word;
        }
    }

    // one block-level reduction per tile, then publish
#pragma unroll
    for (int j = 0; j < kAggStreamK; ++j) {
        if (j >= k) break;
        double d = acc[j];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) d += __shfl_xor_sync(0xffffffffu, d, off);
        if (lane == 0) warp_part[j][warp] = d;
    }
    __syncthreads();
    if (tid < k) {
        double t = 0.0;
#pragma unroll
        for (int w = 0; w < kAggThreads / 32; ++w) t += warp_part[tid][w];
        partial[(int64_t)tid * blocks + blockIdx.x] = t;
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) s_ticket = atomicAdd(&scratch->ticket, 1u);
    __syncthreads();
    if (s_ticket != blocks - 1) return;
    __threadfence();

    // last block: add the blocks' partial sums in a fixed order
    const volatile double *vp = partial;
    const int32_t groups = per_tile ? k : 1;
    for (int32_t j = 0; j < groups; ++j) {
        double t = 0.0;
        const int64_t lo = per_tile ? (int64_t)j * blocks : 0;
        const int64_t cnt = per_tile ? (int64_t)blocks : (int64_t)k * blocks;
        for (int64_t b = tid; b < cnt; b += kAggThreads) t += vp[lo + b];
        red[tid] = t;
        __syncthreads();
        for (int off = kAggThreads / 2; off > 0; off >>= 1) {
            if (tid < off) red[tid] += red[tid + off];
            __syncthreads();
        }
        if (tid == 0) alpha[j] = (float)(red[0] / ((double)q * (per_tile ? 1.0 : (double)k)));
        __syncthreads();
    }
}

__global__ void __launch_bounds__(256)
pack_kernel(const float *__restrict__ src, int64_t q, uint32_t *__restrict__ tile_bits, int64_t n_words)
{
    const int lane = threadIdx.x & 31;
    const int64_t warp_global = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t warps_total = ((int64_t)gridDim.x * blockDim.x) >> 5;
    for (int64_t w = warp_global; w < n_words; w += warps_total) {
        const int64_t i = w * 32 + lane;
        const bool pos = (i < q) && (__ldg(src + i) > 0.0f);
        const uint32_t word = __ballot_sync(0xffffffffu, pos);
        if (lane == 0) tile_bits[w] = word;
    }
}

__global__ void __launch_bounds__(256)
expand_kernel(const uint32_t *__restrict__ tile_bits, int64_t N, int64_t q, const float *__restrict__ alpha,
              int per_tile, float *__restrict__ B_hat)
{
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t f = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; f < N; f += stride) {
        const int64_t i = f % q;
        const float a = per_tile ? __ldg(alpha + f / q) : __ldg(alpha);
        B_hat[f] = tile_bit(tile_bits, i) ? a : -a;
    }
}

__global__ void __launch_bounds__(256)
f32_to_bf16_kernel(const float *__restrict__ src, __nv_bfloat16 *__restrict__ dst, int64_t count)
{
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    const int64_t pairs = count >> 1;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < pairs; i += stride) {
        const float2 v = __ldg(reinterpret_cast<const float2 *>(src) + i);
        reinterpret_cast<__nv_bfloat162 *>(dst)[i] = __floats2bfloat162_rn(v.x, v.y);
    }
    if ((count & 1) && blockIdx.x == 0 && threadIdx.x == 0)
        dst[count - 1] = __float2bfloat16_rn(src[count - 1]);
}

// Folding the previous layer's alphas into the next layer's distinct rows (MLP chain with ReLU or no hidden
// activation).  The previous layer's output is h[t][j*r1 + c] = alpha1_j * g[t][c] with g = act(z) (alpha >= 0, so
// relu(alpha z) = alpha relu(z)), hence  sum_j sum_c B2[o][j*r1 + c] h[t][j*r1 + c] = sum_c g[t][c] * W[o][c]  with
//     W[o][c] = sum_j alpha1_j * (bit2(o*n2 + j*r1 + c) ? +1 : -1),   n2 = k1 * r1.
// One thread per (o, c); fp32 sum in increasing j, one rounding to bf16.  The jobs of a launch run side by side
// (blockIdx.y = job); the previous layer's alphas sit in shared memory and the k bit loads of an element are
// independent of one another, so they are in flight together.
constexpr int kFoldAlphas = 256;

__global__ void __launch_bounds__(256)
fold_kernel(const FoldJobs jobs)
{
    // the block's job, selected with compile-time indices so the parameter block is read in place
    FoldJob J = jobs.job[0];
#pragma unroll
    for (int jb = 1; jb < kMaxFoldJobs; ++jb)
        if ((int)blockIdx.y == jb) J = jobs.job[jb];
    __shared__ float al_s[kFoldAlphas];
    for (int j = threadIdx.x; j < J.k_prev && j < kFoldAlphas; j += blockDim.x)
        al_s[j] = __ldg(J.alpha_prev + (J.per_tile_prev ? j : 0));
    __syncthreads();

    const int64_t total = (int64_t)J.rows * J.r_prev;
    const bool narrow = total <= 0x7fffffff;                      // 32-bit division then
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += stride) {
        int64_t o, c;
        if (narrow) {
            const uint32_t oo = (uint32_t)e / (uint32_t)J.r_prev;
            o = oo; c = (uint32_t)e - oo * (uint32_t)J.r_prev;
        } else {
            o = e / J.r_prev; c = e % J.r_prev;
        }
        const int64_t first = o * J.n_next + c;                   // bit of repetition 0; repetition j is j * r_prev on
        float acc = 0.0f;
#pragma unroll 8
        for (int32_t j = 0; j < J.k_prev; ++j) {
            const float al = j < kFoldAlphas ? al_s[j] : __ldg(J.alpha_prev + (J.per_tile_prev ? j : 0));
            acc += tile_bit(J.tile_next, first + (int64_t)j * J.r_prev) ? al : -al;
        }
        J.w_eff[e] = __float2bfloat16_rn(acc);
    }
}

// y += res element by element (same shape and type): the residual connection after a tensor-core layer.  Fusing the
// residual loads into that kernel's epilogue measured slower than this pass: its four epilogue warps cannot keep
// enough loads in flight next to the k-fold replicated stores.
template <typename YT>
__global__ void __launch_bounds__(256)
add_inplace_kernel(YT *__restrict__ y, const YT *__restrict__ res, int64_t count)
{
    constexpr int V = 16 / sizeof(YT);
    const int64_t vecs = count / V;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < vecs; i += stride) {
        uint4 a = reinterpret_cast<const uint4 *>(y)[i];
        const uint4 b = __ldg(reinterpret_cast<const uint4 *>(res) + i);
        YT *pa = reinterpret_cast<YT *>(&a);
        const YT *pb = reinterpret_cast<const YT *>(&b);
#pragma unroll
        for (int e = 0; e < V; ++e) store_from_float(pa, e, load_as_float(pa, e) + load_as_float(pb, e));
        reinterpret_cast<uint4 *>(y)[i] = a;
    }
    if (blockIdx.x == 0)
        for (int64_t i = vecs * V + threadIdx.x; i < count; i += blockDim.x)
            store_from_float(y, i, load_as_float(y, i) + load_as_float(res, i));
}

int grid_for(int64_t work_items, int threads, int cap_blocks)
{
    int64_t b = (work_items + threads - 1) / threads;
    if (b < 1) b = 1;
    if (b > cap_blocks) b = cap_blocks;
    return (int)b;
}

}  // namespace

size_t aggregate_workspace_bytes(int64_t N, int32_t k)
{
    const int64_t q = N / k;
    const int64_t blocks = (q + kAggCols - 1) / kAggCols;
    return sizeof(AggScratch) + (size_t)k * (size_t)blocks * sizeof(double);
}

cudaError_t launch_aggregate(const float *W, const float *A, int64_t N, int32_t k, int per_tile,
                             uint32_t *tile_bits, float *alpha, void *workspace, cudaStream_t s)
{
    const int64_t q = N / k;
    const int64_t blocks = (q + kAggCols - 1) / kAggCols;
    cudaError_t e = cudaMemsetAsync(workspace, 0, sizeof(AggScratch), s);
    if (e != cudaSuccess) return e;
    if (k <= kAggStreamK) {
        // fixed grid: two blocks per SM, never more blocks than chunks (the scratch is sized for one block per chunk)
        int dev = 0, sms = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
            return cudaErrorUnknown;
        const int64_t grid = blocks < 2 * (int64_t)sms ? blocks : 2 * (int64_t)sms;
        auto kern = q % kAggVec == 0 ? (A ? aggregate_stream_kernel<true, true> : aggregate_stream_kernel<true, false>)
                                     : (A ? aggregate_stream_kernel<false, true> : aggregate_stream_kernel<false, false>);
        kern<<<(unsigned)grid, kAggThreads, 0, s>>>(W, A, q, k, per_tile, tile_bits, tbn_tile_words(q), alpha,
                                                   static_cast<AggScratch *>(workspace), blocks);
        return cudaGetLastError();
    }
    if (q % kAggVec == 0)      // every repetition then starts on a 16-byte boundary (W and A are 16-byte aligned)
        aggregate_kernel<true><<<(unsigned)blocks, kAggThreads, 0, s>>>(
            W, A, q, k, per_tile, tile_bits, tbn_tile_words(q), alpha, static_cast<AggScratch *>(workspace));
    else
        aggregate_kernel<false><<<(unsigned)blocks, kAggThreads, 0, s>>>(
            W, A, q, k, per_tile, tile_bits, tbn_tile_words(q), alpha, static_cast<AggScratch *>(workspace));
    return cudaGetLastError();
}

// ---- built-in scratch for callers that cannot allocate ---------------------------------------------
// One array per device that loads the library, held until the process exits.  Host code must not hand
// the symbol itself to a kernel (on the host it is only a stand-in); the device address is looked up
// once per device with cudaGetSymbolAddress and cached.
constexpr size_t kStaticScratchBytes = 1u << 20;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

size_t aggregate_static_scratch_capacity() { return kStaticScratchBytes; }

cudaError_t launch_aggregate_static(const float *W, const float *A, int64_t N, int32_t k, int per_tile,
                                    uint32_t *tile_bits, float *alpha, cudaStream_t s)
{
    static void *cache[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!cache[dev]) {                       // set-up: first call on this device, with the device current
        void *ptr = nullptr;
        e = cudaGetSymbolAddress((void **)&ptr, g_static_scratch);
        if (e != cudaSuccess) return e;
        cache[dev] = ptr;
    }
    // launch_aggregate clears the ticket word that must start at zero; the partial sums are written
    // before they are read, so the previous call's contents do not matter.
    return launch_aggregate(W, A, N, k, per_tile, tile_bits, alpha, cache[dev], s);
}

cudaError_t launch_pack(const float *src, int64_t q, uint32_t *tile_bits, cudaStream_t s)
{
    const int64_t n_words = tbn_tile_words(q);
    pack_kernel<<<grid_for(n_words * 32, 256, 148 * 8), 256, 0, s>>>(src, q, tile_bits, n_words);
    return cudaGetLastError();
}

cudaError_t launch_expand(const uint32_t *tile_bits, int64_t N, int32_t k, const float *alpha,
                          int per_tile, float *B_hat, cudaStream_t s)
{
    expand_kernel<<<grid_for(N, 256, 148 * 8), 256, 0, s>>>(tile_bits, N, N / k, alpha, per_tile, B_hat);
    return cudaGetLastError();
}

cudaError_t launch_fold(const FoldJobs &jobs, cudaStream_t s)
{
    int64_t most = 1;
    for (int32_t j = 0; j < jobs.count; ++j) {
        const int64_t t = (int64_t)jobs.job[j].rows * jobs.job[j].r_prev;
        most = t > most ? t : most;
    }
    fold_kernel<<<dim3((unsigned)grid_for(most, 256, 148 * 8), (unsigned)jobs.count), 256, 0, s>>>(jobs);
    return cudaGetLastError();
}

cudaError_t launch_add_inplace(void *y, const void *res, int64_t count, int dtype, cudaStream_t s)
{
    const int v = dtype == TBN_BF16 ? 8 : 4;
    const int grid = grid_for(count / v + 1, 256, 148 * 16);
    if (dtype == TBN_BF16)
        add_inplace_kernel<<<grid, 256, 0, s>>>(static_cast<__nv_bfloat16 *>(y), static_cast<const __nv_bfloat16 *>(res), count);
    else
        add_inplace_kernel<<<grid, 256, 0, s>>>(static_cast<float *>(y), static_cast<const float *>(res), count);
    return cudaGetLastError();
}

cudaError_t launch_f32_to_bf16(const float *src, __nv_bfloat16 *dst, int64_t count, cudaStream_t s)
{
    f32_to_bf16_kernel<<<grid_for(count / 2 + 1, 256, 148 * 8), 256, 0, s>>>(src, dst, count);
    return cudaGetLastError();
}

}  // namespace tbn
