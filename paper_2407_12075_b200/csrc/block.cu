// Glue of a Transformer encoder block around the tiled linears (Sec. 4.3 tiles the Q, K, V, projection and
// feed-forward layers of Vision Transformers; Sec. 5.2 profiles the kernel inside one): LayerNorm and multi-head
// softmax attention.  Neither is a tiled layer and neither is specific to the paper; they exist so that the block
// runs end to end on the device with activations produced by the previous kernel.
#include "common.cuh"

namespace tbn {

namespace {

// ---- LayerNorm: one warp per row, statistics in fp32 (mean first, then the centred second moment) -------------
template <typename XT, typename YT>
__global__ void __launch_bounds__(256)
layernorm_kernel(const XT *__restrict__ x, int64_t T, int32_t d, const float *__restrict__ gamma, const float *__restrict__ beta,
                 float eps, YT *__restrict__ y)
{
    const int lane = threadIdx.x & 31;
    const int64_t warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    for (int64_t t = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5; t < T; t += warps) {
        const XT *row = x + t * d;
        float s = 0.0f;
        for (int32_t j = lane; j < d; j += 32) s += load_as_float(row, j);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
        const float mu = s / (float)d;
        float v = 0.0f;
        for (int32_t j = lane; j < d; j += 32) { const float c = load_as_float(row, j) - mu; v = fmaf(c, c, v); }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
        const float rstd = rsqrtf(v / (float)d + eps);
        YT *out = y + t * d;
        for (int32_t j = lane; j < d; j += 32) {
            float o = (load_as_float(row, j) - mu) * rstd;
            if (gamma) o *= __ldg(gamma + j);
            if (beta) o += __ldg(beta + j);
            store_from_float(out, j, o);
        }
    }
}

// ---- multi-head softmax attention, bf16 operands, fp32 accumulation and softmax ---------------------------------
// One block per (image, head): Q, K (row pitch 72 elements) and V transposed (key index contiguous) sit in shared
// memory; a warp owns 16 query rows at a time and keeps the whole score row block in registers (S <= 16 * NT16
// keys), so the softmax is exact (no running rescale).  Both contractions are warp-level m16n8k16 MMAs; the
// probabilities are rounded to bf16 for the second one.
constexpr int kAttD = 64;
constexpr int kAttPitch = 72;           // 36 words: the 8 rows a fragment load touches fall on different banks
constexpr int kAttWarps = 7;

__device__ __forceinline__ void att_mma(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t *>(&h);
}

template <int NT16>
__global__ void __launch_bounds__(kAttWarps * 32)
attention_kernel(const __nv_bfloat16 *__restrict__ qkv, int32_t S, int32_t heads, __nv_bfloat16 *__restrict__ out)
{
    constexpr int SP = NT16 * 16;                       // padded sequence length
    constexpr int kVtPitch = SP + 8;                    // (SP + 8) / 2 words = 12 mod 32 for SP = 208, 4 mod 32 for 64 / 128
    extern __shared__ __align__(16) uint8_t att_smem[];
    __nv_bfloat16 *Qs = reinterpret_cast<__nv_bfloat16 *>(att_smem);
    __nv_bfloat16 *Ks = Qs + SP * kAttPitch;
    __nv_bfloat16 *Vt = Ks + SP * kAttPitch;            // [64][kVtPitch]
    const int b = blockIdx.x / heads, h = blockIdx.x % heads;
    const int64_t row_pitch = (int64_t)3 * heads * kAttD;
    const __nv_bfloat16 *base = qkv + (int64_t)b * S * row_pitch + h * kAttD;

    // stage Q, K (16-byte pieces) and V transposed; rows past the sequence are zero
    for (int idx = threadIdx.x; idx < SP * 8; idx += blockDim.x) {
        const int s = idx >> 3, c = idx & 7;
        uint4 q = make_uint4(0u, 0u, 0u, 0u), k = q, v = q;
        if (s < S) {
            const __nv_bfloat16 *src = base + (int64_t)s * row_pitch + c * 8;
            q = __ldg(reinterpret_cast<const uint4 *>(src));
            k = __ldg(reinterpret_cast<const uint4 *>(src + heads * kAttD));
            v = __ldg(reinterpret_cast<const uint4 *>(src + 2 * heads * kAttD));
        }
        *reinterpret_cast<uint4 *>(Qs + s * kAttPitch + c * 8) = q;
        *reinterpret_cast<uint4 *>(Ks + s * kAttPitch + c * 8) = k;
        const uint32_t vw[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            reinterpret_cast<unsigned short *>(Vt)[(c * 8 + 2 * e) * kVtPitch + s] = (unsigned short)(vw[e] & 0xffffu);
            reinterpret_cast<unsigned short *>(Vt)[(c * 8 + 2 * e + 1) * kVtPitch + s] = (unsigned short)(vw[e] >> 16);
        }
    }
    __syncthreads();

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, c = lane & 3;
    const float scale = 0.125f * 1.4426950408889634f;   // 1/sqrt(64) * log2(e): the softmax runs on exp2
    for (int qt = warp; qt < NT16; qt += kAttWarps) {
        if (qt * 16 >= S) break;
        // scores of 16 query rows against all keys
        uint32_t aq[4][4];
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
            const __nv_bfloat16 *q0 = Qs + (qt * 16 + g) * kAttPitch + kk * 16 + 2 * c;
            aq[kk][0] = *reinterpret_cast<const uint32_t *>(q0);
            aq[kk][1] = *reinterpret_cast<const uint32_t *>(q0 + 8 * kAttPitch);
            aq[kk][2] = *reinterpret_cast<const uint32_t *>(q0 + 8);
            aq[kk][3] = *reinterpret_cast<const uint32_t *>(q0 + 8 * kAttPitch + 8);
        }
        float sc[2 * NT16][4];
#pragma unroll
        for (int nt = 0; nt < 2 * NT16; ++nt) {
            sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.0f;
            const __nv_bfloat16 *k0 = Ks + (nt * 8 + g) * kAttPitch + 2 * c;
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
                att_mma(sc[nt], aq[kk][0], aq[kk][1], aq[kk][2], aq[kk][3], *reinterpret_cast<const uint32_t *>(k0 + kk * 16),
                        *reinterpret_cast<const uint32_t *>(k0 + kk * 16 + 8));
        }
        // mask the padded keys, row maxima (rows g and g + 8), exponentials, row sums
        float m0 = -INFINITY, m1 = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < 2 * NT16; ++nt) {
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                if (nt * 8 + 2 * c + e >= S) { sc[nt][e] = -INFINITY; sc[nt][2 + e] = -INFINITY; }
                m0 = fmaxf(m0, sc[nt][e]);
                m1 = fmaxf(m1, sc[nt][2 + e]);
            }
        }
        m0 = fmaxf(m0, __shfl_xor_sync(0xffffffffu, m0, 1)); m0 = fmaxf(m0, __shfl_xor_sync(0xffffffffu, m0, 2));
        m1 = fmaxf(m1, __shfl_xor_sync(0xffffffffu, m1, 1)); m1 = fmaxf(m1, __shfl_xor_sync(0xffffffffu, m1, 2));
        float l0 = 0.0f, l1 = 0.0f;
#pragma unroll
        for (int nt = 0; nt < 2 * NT16; ++nt) {
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                sc[nt][e] = exp2f((sc[nt][e] - m0) * scale);
                sc[nt][2 + e] = exp2f((sc[nt][2 + e] - m1) * scale);
                l0 += sc[nt][e];
                l1 += sc[nt][2 + e];
            }
        }
        l0 += __shfl_xor_sync(0xffffffffu, l0, 1); l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
        l1 += __shfl_xor_sync(0xffffffffu, l1, 1); l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
        // weighted sum of the values: the score fragments are the A operand of the second contraction as they are
        float o[8][4];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.0f;
#pragma unroll
        for (int kk = 0; kk < NT16; ++kk) {
            const uint32_t a0 = pack_bf16(sc[2 * kk][0], sc[2 * kk][1]), a1 = pack_bf16(sc[2 * kk][2], sc[2 * kk][3]);
            const uint32_t a2 = pack_bf16(sc[2 * kk + 1][0], sc[2 * kk + 1][1]), a3 = pack_bf16(sc[2 * kk + 1][2], sc[2 * kk + 1][3]);
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) {
                const __nv_bfloat16 *v0 = Vt + (nt * 8 + g) * kVtPitch + kk * 16 + 2 * c;
                att_mma(o[nt], a0, a1, a2, a3, *reinterpret_cast<const uint32_t *>(v0), *reinterpret_cast<const uint32_t *>(v0 + 8));
            }
        }
        const float r0 = 1.0f / l0, r1 = 1.0f / l1;
        const int row0 = qt * 16 + g, row1 = row0 + 8;
        __nv_bfloat16 *out0 = out + ((int64_t)b * S + row0) * (heads * kAttD) + h * kAttD + 2 * c;
        __nv_bfloat16 *out1 = out + ((int64_t)b * S + row1) * (heads * kAttD) + h * kAttD + 2 * c;
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            if (row0 < S) *reinterpret_cast<uint32_t *>(out0 + nt * 8) = pack_bf16(o[nt][0] * r0, o[nt][1] * r0);
            if (row1 < S) *reinterpret_cast<uint32_t *>(out1 + nt * 8) = pack_bf16(o[nt][2] * r1, o[nt][3] * r1);
        }
    }
}

template <int NT16>
cudaError_t launch_attention_nt(const __nv_bfloat16 *qkv, int32_t Nb, int32_t S, int32_t heads, __nv_bfloat16 *out, cudaStream_t s)
{
    constexpr int SP = NT16 * 16;
    const size_t smem = (size_t)(2 * SP * kAttPitch + kAttD * (SP + 8)) * sizeof(__nv_bfloat16);
    auto kern = attention_kernel<NT16>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    kern<<<(unsigned)(Nb * heads), kAttWarps * 32, smem, s>>>(qkv, S, heads, out);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_layernorm(const void *x, int x_dtype, int64_t T, int32_t d, const float *gamma, const float *beta, float eps,
                             void *y, int y_dtype, cudaStream_t s)
{
    const int64_t blocks_needed = (T + 7) / 8;
    const unsigned grid = (unsigned)(blocks_needed < 148 * 16 ? (blocks_needed > 0 ? blocks_needed : 1) : 148 * 16);
    if (x_dtype == TBN_BF16 && y_dtype == TBN_BF16)
        layernorm_kernel<<<grid, 256, 0, s>>>(static_cast<const __nv_bfloat16 *>(x), T, d, gamma, beta, eps, static_cast<__nv_bfloat16 *>(y));
    else if (x_dtype == TBN_BF16)
        layernorm_kernel<<<grid, 256, 0, s>>>(static_cast<const __nv_bfloat16 *>(x), T, d, gamma, beta, eps, static_cast<float *>(y));
    else if (y_dtype == TBN_BF16)
        layernorm_kernel<<<grid, 256, 0, s>>>(static_cast<const float *>(x), T, d, gamma, beta, eps, static_cast<__nv_bfloat16 *>(y));
    else
        layernorm_kernel<<<grid, 256, 0, s>>>(static_cast<const float *>(x), T, d, gamma, beta, eps, static_cast<float *>(y));
    return cudaGetLastError();
}

bool attention_supported(int32_t S, int32_t heads, int32_t d_head)
{
    return d_head == kAttD && S >= 1 && S <= 208 && heads >= 1;
}

cudaError_t launch_attention(const void *qkv, int32_t Nb, int32_t S, int32_t heads, int32_t d_head, void *out, cudaStream_t s)
{
    (void)d_head;
    const __nv_bfloat16 *q = static_cast<const __nv_bfloat16 *>(qkv);
    __nv_bfloat16 *o = static_cast<__nv_bfloat16 *>(out);
    if (S <= 64) return launch_attention_nt<4>(q, Nb, S, heads, o, s);
    if (S <= 128) return launch_attention_nt<8>(q, Nb, S, heads, o, s);
    return launch_attention_nt<13>(q, Nb, S, heads, o, s);
}

}  // namespace tbn
