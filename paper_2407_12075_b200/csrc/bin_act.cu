// Binary activations (Sec. 7 of the paper names tiled networks with binary weights AND binary activations as the
// next step): the activation threshold / packing kernel and the CUDA-core XNOR-popcount forward.
//
//   a[t][j] = x[t][j] > 0 ? +1 : -1          (the rule of Eq. 3 applied to the activations)
//   beta[t] = ||x[t][:]||_1 / n              (the scale of Eq. 6 applied to one input row)
//   D[t][i] = sum_j b[i][j] a[t][j] = cnt - 2 popcount(x_bits xor w_bits)     (exact in integers)
//   y[t][i] = act(beta[t] * sum over tile segments of alpha_seg * D_seg + bias[i])
//
// The popcount kernel takes every shape (any alignment of the tile length against the row length, like the
// index walk of Algorithm 1) and is the path for small batches, where the layer is bound by reading the tile once
// and by launch latency; large batches of row-aligned shapes go to the tensor-core kernel (tc_linear_bin.cu).
#include "common.cuh"

namespace tbn {

namespace {

// ---- threshold + packing + row scale ---------------------------------------------------------------------------
// One warp per token row.  A lane takes 8 consecutive values per step (one 16-byte load for bf16, two for fp32),
// turns them into a byte of bits; 4 neighbouring lanes make a 32-bit word.  |x| is added 8 values at a time in
// fp32 and across steps in fp64; the lanes are added in a fixed order (shuffle tree), so beta is reproducible.
template <typename XT>
__device__ __forceinline__ void load8f(const XT *p, float (&v)[8]);
template <>
__device__ __forceinline__ void load8f<__nv_bfloat16>(const __nv_bfloat16 *p, float (&v)[8]) {
    const uint4 u = __ldg(reinterpret_cast<const uint4 *>(p));
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        v[2 * i] = __uint_as_float(w[i] << 16);
        v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}
template <>
__device__ __forceinline__ void load8f<float>(const float *p, float (&v)[8]) {
    const float4 a = __ldg(reinterpret_cast<const float4 *>(p));
    const float4 b = __ldg(reinterpret_cast<const float4 *>(p) + 1);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
    v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}

template <typename XT, bool VEC>
__global__ void __launch_bounds__(256)
binarize_kernel(const XT *__restrict__ x, int64_t T, int32_t n, int32_t row_words, uint32_t *__restrict__ bits,
                float *__restrict__ beta, uint8_t *__restrict__ bytes, int32_t *__restrict__ row_pop)
{
    // bytes / row_pop (both or neither; n a multiple of 32): the byte form of the signs for the tensor-core kernel, in
    // its element order (see bin_expand_kernel), and the number of +1 elements of each row, written in the same pass
    const int lane = threadIdx.x & 31;
    const int64_t warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    for (int64_t t = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5; t < T; t += warps) {
        const XT *row = x + t * n;
        uint32_t *out = bits + t * row_words;
        double acc = 0.0;
        int32_t pop = 0;
        // whole groups of 256 values (8 words) per step; row_words * 32 >= n, words past n are written as zero
        for (int32_t j0 = 0; j0 < row_words * 32; j0 += 256) {
            const int32_t j = j0 + lane * 8;
            float v[8];
            if (VEC && j + 8 <= n) {
                load8f<XT>(row + j, v);
            } else {
#pragma unroll
                for (int e = 0; e < 8; ++e) v[e] = (j + e < n) ? load_as_float(row, j + e) : 0.0f;
            }
            uint32_t byte = 0;
            float ab = 0.0f;
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                byte |= (v[e] > 0.0f ? 1u : 0u) << e;            // zero, negative zero and NaN give 0 (= -1)
                ab += fabsf(v[e]);
            }
            acc += (double)ab;
            uint32_t word = byte << (8 * (lane & 3));
            word |= __shfl_xor_sync(0xffffffffu, word, 1);
            word |= __shfl_xor_sync(0xffffffffu, word, 2);
            const int32_t w = (j0 >> 5) + (lane >> 2);
            if ((lane & 3) == 0 && w < row_words) out[w] = word;
            if (bytes != nullptr && w * 32 < n) {
                // the quad shares the word: lane j of it writes registers s = 2 j and 2 j + 1 of the word's 32 bytes
                if ((lane & 3) == 0) pop += __popc(word);
                const uint32_t s0 = 2u * (uint32_t)(lane & 3);
                uint32_t e0, e1;
                asm("prmt.b32 %0, %1, %1, 0xBA98;" : "=r"(e0) : "r"(word << s0));
                asm("prmt.b32 %0, %1, %1, 0xBA98;" : "=r"(e1) : "r"(word << (s0 + 1u)));
                *reinterpret_cast<uint2 *>(bytes + t * n + (int64_t)w * 32 + 4 * s0) = make_uint2(e0, e1);
            }
        }
        if (row_pop != nullptr) {
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) pop += __shfl_xor_sync(0xffffffffu, pop, off);
            if (lane == 0) row_pop[t] = pop;
        }
        if (beta != nullptr) {
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
            if (lane == 0) beta[t] = (float)(acc / (double)n);
        }
    }
}

// ---- XNOR-popcount forward on CUDA cores -------------------------------------------------------------------------
// 32 tile bits starting at bit `pos` (pos + 32 may run past the last word: the extra bits are masked by the caller).
__device__ __forceinline__ uint32_t tile_bits32(const uint32_t *__restrict__ tile, int64_t pos, int64_t last_word) {
    const int64_t w = pos >> 5;
    const uint32_t lo = __ldg(tile + w);
    const uint32_t hi = __ldg(tile + (w < last_word ? w + 1 : last_word));
    return __funnelshift_r(lo, hi, (uint32_t)pos & 31u);
}

constexpr int kPopcWarps = 8;

// A block stages TT token rows of activation bits in shared memory; a warp owns one weight row at a time (a distinct
// row when the tile spans whole rows, an output row otherwise), its lanes split the row's 32-bit words, and the
// per-token sums are combined with warp shuffles.  When a word crosses the end of the tile the walk wraps to bit 0
// and moves to the next alpha, as Algorithm 1 does.
template <int TT>
__global__ void __launch_bounds__(kPopcWarps * 32)
bin_popc_kernel(const BinArgs a)
{
    extern __shared__ uint32_t xs[];                       // [TT][xw]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t t0 = (int64_t)blockIdx.y * TT;
    const int32_t xw = a.x_row_words;
    for (int32_t i = threadIdx.x; i < TT * xw; i += blockDim.x) {
        const int32_t tt = i / xw, w = i - tt * xw;
        xs[i] = (t0 + tt < a.T) ? __ldg(a.x_bits + (t0 + tt) * xw + w) : 0u;
    }
    __syncthreads();

    const bool aligned = a.q % a.n == 0;
    const int32_t r = aligned ? (int32_t)(a.q / a.n) : a.m;
    const int32_t n_words = (a.n + 31) >> 5;
    const int64_t last_word = ((a.q + 31) >> 5) - 1;      // last word that holds tile bits
    const bool raw = a.y_dtype == TBN_I32;
    const bool per_tile = a.alpha_mode == TBN_ALPHA_PER_TILE;

    for (int32_t row = blockIdx.x * kPopcWarps + warp; row < r; row += gridDim.x * kPopcWarps) {
        const int64_t f0 = (int64_t)row * a.n;             // flat index of the row's first weight
        int32_t di[TT];
        float df[TT];
#pragma unroll
        for (int t = 0; t < TT; ++t) { di[t] = 0; df[t] = 0.0f; }
        for (int32_t w = lane; w < n_words; w += 32) {
            int32_t cnt = min(32, a.n - 32 * w);           // bits of this word that belong to the row
            int64_t f = f0 + 32 * (int64_t)w;
            int32_t off = 0;                               // bits of the word already consumed
            while (cnt > 0) {
                const int64_t pos = aligned ? f : f % a.q;
                const int32_t take = (int32_t)min((int64_t)cnt, a.q - pos);
                const uint32_t mask = take == 32 ? 0xffffffffu : ((1u << take) - 1u);
                const uint32_t wb = tile_bits32(a.tile, pos, last_word) & mask;
                const float al = (aligned || raw) ? 1.0f : __ldg(a.alpha + (per_tile ? f / a.q : 0));
#pragma unroll
                for (int t = 0; t < TT; ++t) {
                    const uint32_t xb = (xs[t * xw + w] >> off) & mask;
                    const int32_t d = take - 2 * __popc(xb ^ wb);
                    di[t] += d;
                    df[t] = fmaf(al, (float)d, df[t]);
                }
                cnt -= take; off += take; f += take;
            }
        }
#pragma unroll
        for (int t = 0; t < TT; ++t) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                di[t] += __shfl_xor_sync(0xffffffffu, di[t], o);
                df[t] += __shfl_xor_sync(0xffffffffu, df[t], o);
            }
        }
        // every lane holds all sums: spread the (repetition, token) stores over the lanes
        const int32_t reps = aligned ? a.k : 1;
        for (int32_t e = lane; e < reps * TT; e += 32) {
            const int32_t j = e / TT, t = e - j * TT;
            if (t0 + t >= a.T) continue;
            int32_t dsel = 0;
            float fsel = 0.0f;
#pragma unroll
            for (int t2 = 0; t2 < TT; ++t2)
                if (t2 == t) { dsel = di[t2]; fsel = df[t2]; }
            const int32_t o = j * r + row;
            const int64_t yi = (t0 + t) * a.m + o;
            if (raw) {
                static_cast<int32_t *>(a.y)[yi] = dsel;
                continue;
            }
            const float bt = a.beta ? __ldg(a.beta + t0 + t) : 1.0f;
            const float z = aligned ? (per_tile ? __ldg(a.alpha + j) : __ldg(a.alpha)) * (float)dsel : fsel;
            const float v = apply_act(fmaf(bt, z, a.bias ? __ldg(a.bias + o) : 0.0f), a.act);
            if (a.y_dtype == TBN_BF16) store_from_float(static_cast<__nv_bfloat16 *>(a.y), yi, v);
            else store_from_float(static_cast<float *>(a.y), yi, v);
        }
    }
}

// Packed activation signs -> one byte per element, 0x00 (bit 0) or 0xFF (bit 1), in the element order of the 8-bit
// tensor-core kernel: byte 4 s + j of every group of 32 elements holds bit 8 j + 7 - s of the group's word (one byte
// permute in sign mode per four elements); and the popcount of every row.  One warp per row, one word per lane and
// step, two 16-byte stores per word.
__global__ void __launch_bounds__(256)
bin_expand_kernel(const uint32_t *__restrict__ bits, int64_t T, int32_t nw, int32_t row_words, uint8_t *__restrict__ bytes,
                  int32_t *__restrict__ row_pop)
{
    const int lane = threadIdx.x & 31;
    const int64_t warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    for (int64_t t = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5; t < T; t += warps) {
        int32_t cnt = 0;
        for (int32_t w = lane; w < nw; w += 32) {
            const uint32_t v = __ldg(bits + t * row_words + w);
            cnt += __popc(v);
            uint32_t e[8];
#pragma unroll
            for (int sft = 0; sft < 8; ++sft) asm("prmt.b32 %0, %1, %1, 0xBA98;" : "=r"(e[sft]) : "r"(v << sft));
            uint4 *dst = reinterpret_cast<uint4 *>(bytes + (t * nw + w) * 32);
            dst[0] = make_uint4(e[0], e[1], e[2], e[3]);
            dst[1] = make_uint4(e[4], e[5], e[6], e[7]);
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, off);
        if (lane == 0) row_pop[t] = cnt;
    }
}

}  // namespace

cudaError_t launch_bin_expand(const uint32_t *bits, int64_t T, int32_t n, int32_t row_words, void *bytes, int32_t *row_pop,
                              cudaStream_t s)
{
    if (n % 32 != 0) return cudaErrorInvalidValue;
    const int64_t blocks_needed = (T + 7) / 8;
    const unsigned grid = (unsigned)(blocks_needed < 148 * 32 ? (blocks_needed > 0 ? blocks_needed : 1) : 148 * 32);
    bin_expand_kernel<<<grid, 256, 0, s>>>(bits, T, n / 32, row_words, static_cast<uint8_t *>(bytes), row_pop);
    return cudaGetLastError();
}

cudaError_t launch_binarize(const void *x, int x_dtype, int64_t T, int32_t n, uint32_t *bits, float *beta, void *bytes_out,
                            int32_t *row_pop, cudaStream_t s)
{
    uint8_t *bytes = static_cast<uint8_t *>(bytes_out);
    const int32_t rw = (int32_t)tbn_row_words(n);
    const int64_t blocks_needed = (T + 7) / 8;
    const unsigned grid = (unsigned)(blocks_needed < 148 * 16 ? (blocks_needed > 0 ? blocks_needed : 1) : 148 * 16);
    const bool vec = (n % 8 == 0) && (reinterpret_cast<uintptr_t>(x) & 15) == 0;
    if (x_dtype == TBN_BF16) {
        const __nv_bfloat16 *xp = static_cast<const __nv_bfloat16 *>(x);
        if (vec) binarize_kernel<__nv_bfloat16, true><<<grid, 256, 0, s>>>(xp, T, n, rw, bits, beta, bytes, row_pop);
        else binarize_kernel<__nv_bfloat16, false><<<grid, 256, 0, s>>>(xp, T, n, rw, bits, beta, bytes, row_pop);
    } else {
        const float *xp = static_cast<const float *>(x);
        if (vec) binarize_kernel<float, true><<<grid, 256, 0, s>>>(xp, T, n, rw, bits, beta, bytes, row_pop);
        else binarize_kernel<float, false><<<grid, 256, 0, s>>>(xp, T, n, rw, bits, beta, bytes, row_pop);
    }
    return cudaGetLastError();
}

bool bin_popc_supported(const BinArgs &a)
{
    return (size_t)a.x_row_words * 4 <= 48 * 1024;          // one token row of bits must fit the static shared-memory window
}

cudaError_t launch_bin_popc(const BinArgs &a, cudaStream_t s)
{
    const bool aligned = a.q % a.n == 0;
    const int64_t rows = aligned ? a.q / a.n : a.m;
    const size_t row_bytes = (size_t)a.x_row_words * 4;
    int tt = a.T >= 8 ? 8 : a.T >= 4 ? 4 : a.T >= 2 ? 2 : 1;
    while (tt > 1 && tt * row_bytes > 48 * 1024) tt >>= 1;
    const int64_t tok_blocks = (a.T + tt - 1) / tt;
    if (tok_blocks > 65535) return cudaErrorInvalidConfiguration;
    int64_t row_blocks = (rows + kPopcWarps - 1) / kPopcWarps;
    const int64_t cap = (148 * 8 + tok_blocks - 1) / tok_blocks;     // about eight blocks per SM in all
    if (row_blocks > cap) row_blocks = cap > 0 ? cap : 1;
    const dim3 grid((unsigned)row_blocks, (unsigned)tok_blocks);
    const size_t smem = tt * row_bytes;
    switch (tt) {
    case 8: bin_popc_kernel<8><<<grid, kPopcWarps * 32, smem, s>>>(a); break;
    case 4: bin_popc_kernel<4><<<grid, kPopcWarps * 32, smem, s>>>(a); break;
    case 2: bin_popc_kernel<2><<<grid, kPopcWarps * 32, smem, s>>>(a); break;
    default: bin_popc_kernel<1><<<grid, kPopcWarps * 32, smem, s>>>(a); break;
    }
    return cudaGetLastError();
}

}  // namespace tbn
