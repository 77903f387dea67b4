// Small-batch forward (a handful of tokens): the matrix-vector regime of Algorithm 1.
//
// Needs the tile to span whole rows (q % n == 0), so only r = q/n distinct rows exist; each is
// contracted once and written k times with the k alphas (Sec. 4.1, replicated channels).
//
// One warp owns RW distinct rows.  Lane l walks the row in groups of 256 weights and takes the 8
// weights [256*i + 8*l, +8): one 16-byte (bf16) or two 16-byte (fp32) coalesced activation loads per
// token, shared by the warp's RW rows, and one byte of tile bits per row (32 consecutive bytes per
// warp).  A weight bit becomes the float +-1 by OR-ing its inverted value into the sign position of
// 1.0f, so the inner operation is a single FMA per token.  Lanes are combined with warp shuffles.
#include "common.cuh"

namespace tbn {

namespace {

constexpr int kWarps = 4;

template <typename XT> struct XVec;
template <> struct XVec<__nv_bfloat16> {
    static __device__ __forceinline__ void load8(const __nv_bfloat16 *p, float (&v)[8]) {
        const uint4 u = __ldg(reinterpret_cast<const uint4 *>(p));
        const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            v[2 * i] = __uint_as_float(w[i] << 16);
            v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
};
template <> struct XVec<float> {
    static __device__ __forceinline__ void load8(const float *p, float (&v)[8]) {
        const float4 a = __ldg(reinterpret_cast<const float4 *>(p));
        const float4 b = __ldg(reinterpret_cast<const float4 *>(p) + 1);
        v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
        v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
    }
};

template <typename XT, int RW, int TT>
__global__ void __launch_bounds__(kWarps * 32)
small_batch_kernel(const LayerArgs a, int32_t r)
{
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int32_t row0 = (blockIdx.x * kWarps + warp) * RW;      // first distinct row of this warp
    const int64_t t0 = (int64_t)blockIdx.y * TT;
    if (row0 >= r) return;

    const XT *x = static_cast<const XT *>(a.x);
    const uint8_t *bits = reinterpret_cast<const uint8_t *>(a.tile);
    const int32_t n = a.n;
    const int32_t row_bytes = n >> 3;

    float acc[RW][TT];
#pragma unroll
    for (int rr = 0; rr < RW; ++rr)
#pragma unroll
        for (int t = 0; t < TT; ++t) acc[rr][t] = 0.0f;

    for (int32_t e0 = lane * 8; e0 < n; e0 += 256) {
        float xv[TT][8];
#pragma unroll
        for (int t = 0; t < TT; ++t) {
            if (t0 + t < a.T) {
                XVec<XT>::load8(x + (t0 + t) * n + e0, xv[t]);
            } else {
#pragma unroll
                for (int b = 0; b < 8; ++b) xv[t][b] = 0.0f;
            }
        }
#pragma unroll
        for (int rr = 0; rr < RW; ++rr) {
            const int32_t row = min(row0 + rr, r - 1);            // clamp: extra rows are not stored
            const uint32_t nb = ~(uint32_t)__ldg(bits + (int64_t)row * row_bytes + (e0 >> 3));
#pragma unroll
            for (int b = 0; b < 8; ++b) {
                const float sgn = __uint_as_float(0x3f800000u | ((nb << (31 - b)) & 0x80000000u));
#pragma unroll
                for (int t = 0; t < TT; ++t) acc[rr][t] = fmaf(sgn, xv[t][b], acc[rr][t]);
            }
        }
    }

#pragma unroll
    for (int rr = 0; rr < RW; ++rr)
#pragma unroll
        for (int t = 0; t < TT; ++t) {
            float v = acc[rr][t];
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
            acc[rr][t] = v;
        }

    // every lane now holds all sums; spread the k x RW x TT stores over the lanes
    const bool per_tile = a.alpha_mode == TBN_ALPHA_PER_TILE;
    const int total = a.k * RW * TT;
    for (int e = lane; e < total; e += 32) {
        const int t = e % TT;
        const int rr = (e / TT) % RW;
        const int j = e / (TT * RW);
        const int32_t row = row0 + rr;
        if (row >= r || t0 + t >= a.T) continue;
        float z = 0.0f;
#pragma unroll
        for (int r2 = 0; r2 < RW; ++r2)
#pragma unroll
            for (int t2 = 0; t2 < TT; ++t2)
                if (r2 == rr && t2 == t) z = acc[r2][t2];
        const int32_t o = j * r + row;
        const float al = per_tile ? __ldg(a.alpha + j) : __ldg(a.alpha);
        float v = apply_act(fmaf(al, z, a.bias ? __ldg(a.bias + o) : 0.0f), a.act);
        const int64_t yi = (t0 + t) * a.m + o;
        if (a.residual != nullptr)
            v += a.y_dtype == TBN_BF16 ? load_as_float(static_cast<const __nv_bfloat16 *>(a.residual), yi)
                                       : load_as_float(static_cast<const float *>(a.residual), yi);
        if (a.y_dtype == TBN_BF16) store_from_float(static_cast<__nv_bfloat16 *>(a.y), yi, v);
        else store_from_float(static_cast<float *>(a.y), yi, v);
    }
}

// ---- bf16 activations, word-aligned rows: warp-level tensor-core form --------------------------------------
//
// A block owns 16 distinct rows and 8*NT tokens; its warps split the contraction dimension and are summed in
// warp order through shared memory, so the result does not depend on scheduling.  Each warp issues
// m16n8k16 MMAs whose A fragment is decoded from tile bits in registers and whose B fragment is the
// activations as loaded.  The contraction index may be permuted freely as long as A and B agree, which
// removes every shuffle: within a span of 128 weights lane (g, c) (g = lane / 4, c = lane % 4) takes the
// 32-weight chunk c, i.e. ONE 32-bit word of bits for row g and one for row g + 8, and 64 bytes of
// activations of token g; MMA u of the span contracts weights 4u..4u+3 of all four chunks.
__device__ __forceinline__ void mma_bf16_16x8x16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                                 uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Bits 2p and 2p+1 of a 16-bit field, spread by spread16(), become the bf16 pair (+-1, +-1): bit set -> +1.
__device__ __forceinline__ uint32_t spread16(uint32_t h)       // h < 65536: even bits stay, odd bits move up 15
{
    return (h | (h << 15)) & 0x55555555u;
}
__device__ __forceinline__ uint32_t sign_pair(uint32_t v, int p)
{
    return ((v << (15 - 2 * p)) & 0x80008000u) ^ 0xBF80BF80u;
}

constexpr int kMmaMaxWarps = 32;

// What lane (g, c) holds of one span: a word of bits for rows g and g + 8, and 32 activations per token tile.
template <int NT> struct SpanRegs {
    uint32_t w_lo, w_hi;
    uint4 xb[NT][4];
};

// Loads of one span.  xrow[nt] points at this lane's token row (null when the lane has no token in that tile: its
// registers were zeroed once and stay zero); `live` is false only for chunks past the end of a ragged last span.
template <int NT>
__device__ __forceinline__ void load_span(SpanRegs<NT> &sr, const uint32_t *bits_lo, const uint32_t *bits_hi,
                                          const __nv_bfloat16 *const (&xrow)[NT], int32_t chunk, bool live)
{
    const int32_t ch = live ? chunk : 0;
    sr.w_lo = __ldg(bits_lo + ch);
    sr.w_hi = __ldg(bits_hi + ch);
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        if (xrow[nt] != nullptr) {
            if (live) {
                const uint4 *px = reinterpret_cast<const uint4 *>(xrow[nt] + ch * 32);
#pragma unroll
                for (int i = 0; i < 4; ++i) sr.xb[nt][i] = __ldg(px + i);
            } else {
#pragma unroll
                for (int i = 0; i < 4; ++i) sr.xb[nt][i] = make_uint4(0u, 0u, 0u, 0u);
            }
        }
    }
}

template <int NT>
__device__ __forceinline__ void contract_span(const SpanRegs<NT> &sr, float (&acc)[NT == 1 ? 2 : NT][4])
{
#pragma unroll
    for (int half = 0; half < 2; ++half) {                       // 16 bits of each row word at a time
        const uint32_t v_lo = spread16(half ? sr.w_lo >> 16 : sr.w_lo & 0xffffu);
        const uint32_t v_hi = spread16(half ? sr.w_hi >> 16 : sr.w_hi & 0xffffu);
#pragma unroll
        for (int uu = 0; uu < 4; ++uu) {                         // MMA u = 4 * half + uu: weights 4u..4u+3 of the chunk
            const uint32_t a0 = sign_pair(v_lo, 2 * uu), a2 = sign_pair(v_lo, 2 * uu + 1);
            const uint32_t a1 = sign_pair(v_hi, 2 * uu), a3 = sign_pair(v_hi, 2 * uu + 1);
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                const uint4 q = sr.xb[nt][half * 2 + (uu >> 1)];
                const uint32_t b0 = (uu & 1) ? q.z : q.x, b1 = (uu & 1) ? q.w : q.y;
                // a single token tile alternates between two accumulators: two independent MMA chains
                mma_bf16_16x8x16(acc[NT == 1 ? (uu & 1) : nt], a0, a1, a2, a3, b0, b1);
            }
        }
    }
}

template <int NT>
__global__ void __launch_bounds__(kMmaMaxWarps / NT * 32, NT == 4 ? 2 : NT)
small_mma_kernel(const LayerArgs a, int32_t r)
{
    __shared__ float red[kMmaMaxWarps / NT][NT][16][8];          // [warp][token tile][row][token]: 16 KB
    __shared__ float alpha_s[64];
    pdl_launch_dependents();
    pdl_wait();                                                  // the activations may come from the previous kernel

    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int nw = blockDim.x >> 5;
    const int g = lane >> 2, c = lane & 3;
    const int32_t row0 = blockIdx.x * 16;
    const int64_t t0 = (int64_t)blockIdx.y * (8 * NT);
    const int32_t n = a.n;
    const int32_t n_chunks = n >> 5;                             // n % 32 == 0
    const int32_t n_spans = (n_chunks + 3) >> 2;
    const bool per_tile = a.alpha_mode == TBN_ALPHA_PER_TILE;

    // the scales are needed only at the very end: fetch them now, off the critical path
    if ((int)threadIdx.x < min(a.k, 64)) alpha_s[threadIdx.x] = __ldg(a.alpha + (per_tile ? threadIdx.x : 0));

    const int32_t row_words = n >> 5;
    const uint32_t *bits_lo = a.tile + (int64_t)min(row0 + g, r - 1) * row_words;     // clamped rows are not stored
    const uint32_t *bits_hi = a.tile + (int64_t)min(row0 + g + 8, r - 1) * row_words;
    const __nv_bfloat16 *x = static_cast<const __nv_bfloat16 *>(a.x);

    float acc[NT == 1 ? 2 : NT][4];
#pragma unroll
    for (int nt = 0; nt < (NT == 1 ? 2 : NT); ++nt)
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[nt][i] = 0.0f;

    const __nv_bfloat16 *xrow[NT];                               // this lane's token row per tile, or null
    SpanRegs<NT> sr;
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        const int64_t t = t0 + nt * 8 + g;
        xrow[nt] = t < a.T ? x + t * n : nullptr;
#pragma unroll
        for (int i = 0; i < 4; ++i) sr.xb[nt][i] = make_uint4(0u, 0u, 0u, 0u);
    }
    const int32_t full_spans = n_chunks >> 2;                    // spans whose four chunks all exist
    int32_t span = warp;
    for (; span < full_spans; span += nw) {
        load_span<NT>(sr, bits_lo, bits_hi, xrow, span * 4 + c, true);
        contract_span<NT>(sr, acc);
    }
    if (span < n_spans) {                                        // the ragged last span, if this warp owns it
        load_span<NT>(sr, bits_lo, bits_hi, xrow, span * 4 + c, span * 4 + c < n_chunks);
        contract_span<NT>(sr, acc);
    }

    if (NT == 1) {
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[0][i] += acc[1][i];
    }
    // accumulator fragment: [0],[1] = row g, tokens 2c, 2c+1; [2],[3] = row g + 8
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        *reinterpret_cast<float2 *>(&red[warp][nt][g][2 * c]) = make_float2(acc[nt][0], acc[nt][1]);
        *reinterpret_cast<float2 *>(&red[warp][nt][g + 8][2 * c]) = make_float2(acc[nt][2], acc[nt][3]);
    }
    __syncthreads();

    for (int e = threadIdx.x; e < NT * 8 * 16; e += blockDim.x) {
        const int row = e & 15, tok = e >> 4;                    // rows fastest: 16 neighbouring outputs per token
        const int32_t grow = row0 + row;
        const int64_t t = t0 + tok;
        if (grow >= r || t >= a.T) continue;
        float z = 0.0f;                                          // warps are summed in warp order: deterministic
#pragma unroll 8
        for (int w = 0; w < nw; ++w) z += red[w][tok >> 3][row][tok & 7];
        for (int32_t j = 0; j < a.k; ++j) {
            const int32_t o = j * r + grow;
            const float al = j < 64 ? alpha_s[j] : __ldg(a.alpha + (per_tile ? j : 0));
            float v = apply_act(fmaf(al, z, a.bias ? __ldg(a.bias + o) : 0.0f), a.act);
            const int64_t yi = t * a.m + o;
            if (a.residual != nullptr)
                v += a.y_dtype == TBN_BF16 ? load_as_float(static_cast<const __nv_bfloat16 *>(a.residual), yi)
                                           : load_as_float(static_cast<const float *>(a.residual), yi);
            if (a.y_dtype == TBN_BF16) store_from_float(static_cast<__nv_bfloat16 *>(a.y), yi, v);
            else store_from_float(static_cast<float *>(a.y), yi, v);
        }
    }
}

bool small_mma_supported(const LayerArgs &a)
{
    return a.x_dtype == TBN_BF16 && (a.n & 31) == 0 && (reinterpret_cast<uintptr_t>(a.x) & 15) == 0;
}

cudaError_t launch_small_mma(const LayerArgs &a, int32_t r, cudaStream_t s)
{
    const int nt = a.T <= 8 ? 1 : a.T <= 16 ? 2 : 4;
    const int64_t row_blocks = (r + 15) / 16;
    const int64_t tok_blocks = (a.T + 8 * nt - 1) / (8 * nt);
    const int32_t n_spans = (a.n / 32 + 3) / 4;
    // about 16 warps per SM in total, at least one span per warp, and the reduction buffer bounds warps x NT
    int nw = 1;
    while (nw < kMmaMaxWarps / nt && nw < n_spans && row_blocks * tok_blocks * nw < 148 * 16) nw *= 2;
    const dim3 grid((unsigned)row_blocks, (unsigned)tok_blocks);
    if (nt == 1) return launch_pdl(small_mma_kernel<1>, grid, dim3(nw * 32), 0, s, a, r);
    if (nt == 2) return launch_pdl(small_mma_kernel<2>, grid, dim3(nw * 32), 0, s, a, r);
    return launch_pdl(small_mma_kernel<4>, grid, dim3(nw * 32), 0, s, a, r);
}

template <typename XT, int RW>
cudaError_t launch_tt(const LayerArgs &a, int32_t r, cudaStream_t s)
{
    const int rows_per_block = kWarps * RW;
    const unsigned gx = (unsigned)((r + rows_per_block - 1) / rows_per_block);
    if (a.T <= 1) {
        small_batch_kernel<XT, RW, 1><<<dim3(gx, 1), kWarps * 32, 0, s>>>(a, r);
    } else if (a.T <= 2) {
        small_batch_kernel<XT, RW, 2><<<dim3(gx, 1), kWarps * 32, 0, s>>>(a, r);
    } else {
        small_batch_kernel<XT, RW, 4><<<dim3(gx, (unsigned)((a.T + 3) / 4)), kWarps * 32, 0, s>>>(a, r);
    }
    return cudaGetLastError();
}

template <typename XT>
cudaError_t launch_rw(const LayerArgs &a, int32_t r, cudaStream_t s)
{
    // more rows per warp reuse each activation load more often, but small layers need the blocks
    if (r >= 148 * 4 * kWarps * 4) return launch_tt<XT, 4>(a, r, s);
    if (r >= 148 * 2 * kWarps * 2) return launch_tt<XT, 2>(a, r, s);
    return launch_tt<XT, 1>(a, r, s);
}

// ---- thin layer with full-precision rows (the last layer of a compact MLP chain) -------------------------------
//
// y[t][j*r + c] = act(alpha_j * sum_i x[t][i] * W[c][i] + bias) for r <= 16 bf16 rows W (a classifier head).  The
// whole weight block sits in shared memory as fp32; a warp owns a token, lane l takes inputs [256 g + 8 l, +8) of
// every 256-input group, and the r sums are combined with warp shuffles.  A launch of the tensor-core kernel costs
// several microseconds of fixed set-up, far more than this layer's arithmetic.
constexpr int kThinRows = 16;
constexpr int kThinMaxWeights = 8192;      // r * n fp32 values in shared memory (32 KB)

__global__ void __launch_bounds__(256)
thin_dense_kernel(const LayerArgs a, int32_t r)
{
    __shared__ __align__(16) float w_s[kThinMaxWeights];
    const int32_t n = a.n;
    const __nv_bfloat16 *W = static_cast<const __nv_bfloat16 *>(a.dense_a);
    // 16-byte loads (n % 8 == 0, the rows are 16-byte aligned), all of a thread's loads in flight together
    const int32_t groups = (r * n) >> 3;
#pragma unroll 4
    for (int32_t gidx = threadIdx.x; gidx < groups; gidx += blockDim.x) {
        float v[8];
        XVec<__nv_bfloat16>::load8(W + 8 * gidx, v);
        *reinterpret_cast<float4 *>(w_s + 8 * gidx) = make_float4(v[0], v[1], v[2], v[3]);
        *reinterpret_cast<float4 *>(w_s + 8 * gidx + 4) = make_float4(v[4], v[5], v[6], v[7]);
    }
    __syncthreads();

    const int lane = threadIdx.x & 31;
    const int warps = (gridDim.x * blockDim.x) >> 5;
    const __nv_bfloat16 *x = static_cast<const __nv_bfloat16 *>(a.x);
    const bool per_tile = a.alpha_mode == TBN_ALPHA_PER_TILE;
    for (int64_t t = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; t < a.T; t += warps) {
        float acc[kThinRows];
#pragma unroll
        for (int c = 0; c < kThinRows; ++c) acc[c] = 0.0f;
        for (int32_t i0 = lane * 8; i0 < n; i0 += 256) {             // n % 8 == 0
            float xv[8];
            XVec<__nv_bfloat16>::load8(x + t * n + i0, xv);
#pragma unroll
            for (int c = 0; c < kThinRows; ++c) {
                if (c >= r) break;
                const float4 w0 = *reinterpret_cast<const float4 *>(w_s + c * n + i0);
                const float4 w1 = *reinterpret_cast<const float4 *>(w_s + c * n + i0 + 4);
                acc[c] = fmaf(xv[0], w0.x, acc[c]); acc[c] = fmaf(xv[1], w0.y, acc[c]);
                acc[c] = fmaf(xv[2], w0.z, acc[c]); acc[c] = fmaf(xv[3], w0.w, acc[c]);
                acc[c] = fmaf(xv[4], w1.x, acc[c]); acc[c] = fmaf(xv[5], w1.y, acc[c]);
                acc[c] = fmaf(xv[6], w1.z, acc[c]); acc[c] = fmaf(xv[7], w1.w, acc[c]);
            }
        }
        float mine = 0.0f;                                          // lane c ends up with the sum of row c
#pragma unroll
        for (int c = 0; c < kThinRows; ++c) {
            if (c >= r) break;
            float v = acc[c];
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
            if (lane == c) mine = v;
        }
        if (lane < r) {
            for (int32_t j = 0; j < a.k; ++j) {
                const int32_t o = j * r + lane;
                const float al = per_tile ? __ldg(a.alpha + j) : __ldg(a.alpha);
                const float v = apply_act(fmaf(al, mine, a.bias ? __ldg(a.bias + o) : 0.0f), a.act);
                const int64_t yi = t * a.m + o;
                if (a.y_dtype == TBN_BF16) store_from_float(static_cast<__nv_bfloat16 *>(a.y), yi, v);
                else store_from_float(static_cast<float *>(a.y), yi, v);
            }
        }
    }
}


// ---- the last two layers of a compact MLP chain in one launch ----------------------------------------------------
//
// Layer A: g2[t][o] = act(sum_i Wa[o][i] * g1[t][i]) with full-precision (folded) rows Wa [ra][na], ra <= 256;
// layer B: y[t][j*rb + c] = alpha_j * sum_o Wb[c][o] * g2[t][o] with rb <= 16 folded rows Wb [rb][ra] (a classifier
// head).  Both contractions are a few hundred kiloflops per token, so two launches of the 128-row tensor-memory
// pipeline cost several times their arithmetic in fixed set-up; here a block of 8 warps owns 8*NT tokens, warp w
// takes rows [32 w, 32 w + 32) of layer A with warp-level MMAs, the block's g2 (rounded to bf16, as the chain's
// hidden tensors are) stays in shared memory and warps 0..NT-1 contract it with Wb.  Operand fragments are 16-byte
// loads: within a span of 32 inputs lane (g, c) holds inputs [8c, 8c + 8) of row g / token g, and MMA u of the span
// contracts inputs 8c + 4u .. 8c + 4u + 3 of all four c (A and B agree on the permutation, so no shuffles).
constexpr int kTailRows = 256;          // rows of layer A at most (8 warps x 2 MMA row tiles)
constexpr int kTailPad = 32;            // g2 row padding in shared memory: rows 16 banks apart

struct TailArgs {
    const __nv_bfloat16 *g1;            // [T][na]
    const __nv_bfloat16 *Wa;            // [ra][na]
    const __nv_bfloat16 *Wb;            // [rb][ra]
    const float *alpha;                 // last layer's alphas
    void *y;
    int64_t T;
    int32_t na, ra, rb, kb, mb;         // mb = kb * rb outputs
    int per_tile, act_a, y_dtype;
};

template <int NT>
__global__ void __launch_bounds__(256)
mlp_tail_kernel(const TailArgs a)
{
    extern __shared__ __align__(16) uint8_t tail_smem[];
    __nv_bfloat16 *g2 = reinterpret_cast<__nv_bfloat16 *>(tail_smem);          // [8 NT tokens][ra + kTailPad]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, c = lane & 3;
    const int64_t t0 = (int64_t)blockIdx.x * (8 * NT);
    const int32_t na = a.na, ra = a.ra;
    const int32_t pitch = ra + kTailPad;

    // ---- layer A ----
    const int32_t m0 = warp * 32;
    if (m0 < ra) {
        const __nv_bfloat16 *arow[2][2];                                       // [row tile][g / g + 8], clamped
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
            for (int h = 0; h < 2; ++h) arow[mt][h] = a.Wa + (int64_t)min(m0 + 16 * mt + 8 * h + g, ra - 1) * na + 8 * c;
        const __nv_bfloat16 *brow[NT];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            const int64_t t = t0 + 8 * nt + g;
            brow[nt] = t < a.T ? a.g1 + t * na + 8 * c : nullptr;
        }
        float acc[2][NT][4];
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int i = 0; i < 4; ++i) acc[mt][nt][i] = 0.0f;

        const int32_t spans = na >> 5;                                         // na % 32 == 0
        uint4 wa[2][2][2], xb[2][NT];                                          // two register sets: [set][...]
        auto load = [&](int set, int32_t sp) {
#pragma unroll
            for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                for (int h = 0; h < 2; ++h) wa[set][mt][h] = __ldg(reinterpret_cast<const uint4 *>(arow[mt][h] + 32 * sp));
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
                xb[set][nt] = brow[nt] ? __ldg(reinterpret_cast<const uint4 *>(brow[nt] + 32 * sp)) : make_uint4(0u, 0u, 0u, 0u);
        };
        auto contract = [&](int set) {
#pragma unroll
            for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    mma_bf16_16x8x16(acc[mt][nt], wa[set][mt][0].x, wa[set][mt][1].x, wa[set][mt][0].y, wa[set][mt][1].y,
                                     xb[set][nt].x, xb[set][nt].y);
                    mma_bf16_16x8x16(acc[mt][nt], wa[set][mt][0].z, wa[set][mt][1].z, wa[set][mt][0].w, wa[set][mt][1].w,
                                     xb[set][nt].z, xb[set][nt].w);
                }
        };
        load(0, 0);
        for (int32_t sp = 0; sp < spans; sp += 2) {                            // next span's loads before this span's MMAs
            if (sp + 1 < spans) load(1, sp + 1);
            contract(0);
            if (sp + 1 >= spans) break;
            if (sp + 2 < spans) load(0, sp + 2);
            contract(1);
        }
        // accumulator fragment: [0],[1] = row g, tokens 2c, 2c+1; [2],[3] = row g + 8
#pragma unroll
        for (int mt = 0; mt < 2; ++mt)
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int32_t row = m0 + 16 * mt + 8 * (i >> 1) + g;
                    const int tok = 8 * nt + 2 * c + (i & 1);
                    float v = acc[mt][nt][i];
                    if (a.act_a == TBN_ACT_RELU) v = fmaxf(v, 0.0f);
                    if (row < ra) g2[tok * pitch + row] = __float2bfloat16_rn(v);
                }
    }
    __syncthreads();

    // ---- layer B: one 16-row MMA tile (rows >= rb are zero), warp nt takes tokens [8 nt, 8 nt + 8) ----
    if (warp < NT) {
        const int nt = warp;
        float acc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
        const bool lo_ok = g < a.rb, hi_ok = g + 8 < a.rb;
        const __nv_bfloat16 *wlo = a.Wb + (int64_t)(lo_ok ? g : 0) * ra + 8 * c;
        const __nv_bfloat16 *whi = a.Wb + (int64_t)(hi_ok ? g + 8 : 0) * ra + 8 * c;
        const __nv_bfloat16 *brow = g2 + (8 * nt + g) * pitch + 8 * c;
        const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
        const int32_t spans = ra >> 5;                                         // ra % 32 == 0
#pragma unroll 4
        for (int32_t sp = 0; sp < spans; ++sp) {
            const uint4 lo = lo_ok ? __ldg(reinterpret_cast<const uint4 *>(wlo + 32 * sp)) : zero;
            const uint4 hi = hi_ok ? __ldg(reinterpret_cast<const uint4 *>(whi + 32 * sp)) : zero;
            const uint4 b = *reinterpret_cast<const uint4 *>(brow + 32 * sp);
            mma_bf16_16x8x16(acc, lo.x, hi.x, lo.y, hi.y, b.x, b.y);
            mma_bf16_16x8x16(acc, lo.z, hi.z, lo.w, hi.w, b.z, b.w);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int32_t row = 8 * (i >> 1) + g;
            const int64_t t = t0 + 8 * nt + 2 * c + (i & 1);
            if (row >= a.rb || t >= a.T) continue;
            for (int32_t j = 0; j < a.kb; ++j) {
                const float al = __ldg(a.alpha + (a.per_tile ? j : 0));
                const int64_t yi = t * a.mb + (int64_t)j * a.rb + row;
                if (a.y_dtype == TBN_BF16) store_from_float(static_cast<__nv_bfloat16 *>(a.y), yi, al * acc[i]);
                else store_from_float(static_cast<float *>(a.y), yi, al * acc[i]);
            }
        }
    }
}

}  // namespace

bool small_batch_supported(const LayerArgs &a)
{
    if (a.is_conv) return false;
    if (a.q % a.n != 0) return false;          // tile must span whole rows
    if (a.n % 8 != 0) return false;            // 16-byte activation vectors, byte-aligned bit rows
    if (a.T > 65535 * 4) return false;
    return true;
}

// Launch-to-launch time in microseconds, fitted to measurements on B200 (in = 768 .. 8192, k = 2 .. 16).
double small_batch_estimate_us(const LayerArgs &a)
{
    const double r = (double)(a.q / a.n);
    if (!small_mma_supported(a))                                 // FMA kernel: ~8.5e6 multiply-adds per microsecond
        return 5.0 + (double)a.T * r * (double)a.n / 8.5e6;
    // MMA kernel: a block (16 rows x 8*NT tokens) costs c(NT) us per 1e6 weights of a full 148-SM wave; the
    // legacy warp-level MMA rate, not memory, sets c for NT = 4
    const int nt = a.T <= 8 ? 1 : a.T <= 16 ? 2 : 4;
    const double c = nt == 1 ? 0.19 : nt == 2 ? 0.33 : 0.64;
    const double blocks = (double)((int64_t)((r + 15) / 16) * ((a.T + 8 * nt - 1) / (8 * nt)));
    const double per_block = c * 16.0 * (double)a.n * 148.0 / 1e6;
    return 2.5 + per_block * (blocks > 148.0 ? blocks / 148.0 : 1.0) + 0.06 * a.k;
}

bool thin_dense_supported(const LayerArgs &a)
{
    if (a.is_conv || a.dense_a == nullptr || a.x_dtype != TBN_BF16 || a.q % a.n != 0 || a.n % 8 != 0) return false;
    const int64_t r = a.q / a.n;
    return r <= kThinRows && r * a.n <= kThinMaxWeights && (reinterpret_cast<uintptr_t>(a.x) & 15) == 0 &&
           (reinterpret_cast<uintptr_t>(a.dense_a) & 15) == 0;
}

cudaError_t launch_thin_dense(const LayerArgs &a, cudaStream_t s)
{
    const int32_t r = (int32_t)(a.q / a.n);
    const int64_t blocks_needed = (a.T + 7) / 8;                    // 8 warps (tokens) per block
    // every block fills its own copy of the weight block: one token per warp while that fill is small (the layer is
    // latency-bound: one pass of loads, sums and stores), two blocks per SM otherwise
    const int64_t cap = (int64_t)r * a.n <= kThinMaxWeights / 2 ? 6 * 148 : 2 * 148;
    const unsigned grid = (unsigned)(blocks_needed < cap ? (blocks_needed > 0 ? blocks_needed : 1) : cap);
    thin_dense_kernel<<<grid, 256, 0, s>>>(a, r);
    return cudaGetLastError();
}

// The fused tail takes: a hidden layer `A` with folded rows (dense_a, k = 1, scale one, ReLU or no activation, bf16
// compact output) followed by a last layer `B` with at most 16 folded rows, no bias and no activation.
bool mlp_tail_supported(const LayerArgs &A, const LayerArgs &B)
{
    if (A.is_conv || B.is_conv || !A.dense_a || !B.dense_a || A.bias || B.bias) return false;
    if (A.x_dtype != TBN_BF16 || A.k != 1 || (A.act != TBN_ACT_RELU && A.act != TBN_ACT_NONE) || B.act != TBN_ACT_NONE)
        return false;
    if (A.q % A.n != 0 || B.q % B.n != 0) return false;
    const int64_t ra = A.q / A.n, rb = B.q / B.n;
    if (ra != A.m || ra != B.n || ra > kTailRows || ra % 32 != 0 || A.n % 32 != 0 || rb > 16 || rb < 1) return false;
    if ((int64_t)B.k * rb != B.m) return false;
    return (reinterpret_cast<uintptr_t>(A.x) & 15) == 0 && (reinterpret_cast<uintptr_t>(A.dense_a) & 15) == 0 &&
           (reinterpret_cast<uintptr_t>(B.dense_a) & 15) == 0;
}

cudaError_t launch_mlp_tail(const LayerArgs &A, const LayerArgs &B, cudaStream_t s)
{
    TailArgs t;
    t.g1 = static_cast<const __nv_bfloat16 *>(A.x);
    t.Wa = static_cast<const __nv_bfloat16 *>(A.dense_a);
    t.Wb = static_cast<const __nv_bfloat16 *>(B.dense_a);
    t.alpha = B.alpha; t.y = B.y; t.T = A.T;
    t.na = A.n; t.ra = A.m; t.rb = (int32_t)(B.q / B.n); t.kb = B.k; t.mb = B.m;
    t.per_tile = B.alpha_mode == TBN_ALPHA_PER_TILE; t.act_a = A.act; t.y_dtype = B.y_dtype;
    // 32 tokens per block while that still gives every SM a block, 16 below
    const bool wide = A.T >= 32 * 148;
    const int tokens = wide ? 32 : 16;
    const size_t smem = (size_t)tokens * (t.ra + kTailPad) * sizeof(__nv_bfloat16);
    const unsigned grid = (unsigned)((A.T + tokens - 1) / tokens);
    if (wide) mlp_tail_kernel<4><<<grid, 256, smem, s>>>(t);
    else mlp_tail_kernel<2><<<grid, 256, smem, s>>>(t);
    return cudaGetLastError();
}

cudaError_t launch_small_batch(const LayerArgs &a, cudaStream_t s)
{
    const int32_t r = (int32_t)(a.q / a.n);
    if (small_mma_supported(a)) return launch_small_mma(a, r, s);
    return a.x_dtype == TBN_BF16 ? launch_rw<__nv_bfloat16>(a, r, s) : launch_rw<float>(a, r, s);
}

}  // namespace tbn
