// Glue of a Transformer encoder block around the tiled linears (Sec. 4.3 tiles the Q, K, V, projection and
// feed-forward layers of Vision Transformers; Sec. 5.2 profiles the kernel inside one): LayerNorm and multi-head
// softmax attention.  Neither is a tiled layer and neither is specific to the paper; they exist so that the block
// runs end to end on the device with activations produced by the previous kernel.
#include <atomic>

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

// bf16 rows of up to 256 * NP elements (a multiple of 8), one warp per row, the row held in registers: each lane takes
// 16-byte pieces lane, lane + 32, ...  With a second operand b the row normalised is the bf16-rounded sum a + b,
// which is also written out (the residual stream of an encoder block: one pass instead of an addition pass followed
// by a normalisation pass; sum_out may be b itself, every piece is read before it is written by the same thread).
template <int NP>
__global__ void __launch_bounds__(256)
add_layernorm_bf16_kernel(const __nv_bfloat16 *__restrict__ a, const __nv_bfloat16 *b, __nv_bfloat16 *sum_out, int64_t T, int32_t d,
                          const float *__restrict__ gamma, const float *__restrict__ beta, float eps, __nv_bfloat16 *__restrict__ y)
{
    const int lane = threadIdx.x & 31;
    const int32_t pieces = d >> 3;
    const int64_t warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    for (int64_t t = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5; t < T; t += warps) {
        const int64_t row = t * d;
        float v[NP][8];
        float s = 0.0f;
#pragma unroll
        for (int i = 0; i < NP; ++i) {
            const int32_t pc = lane + 32 * i;
#pragma unroll
            for (int e = 0; e < 8; ++e) v[i][e] = 0.0f;
            if (pc < pieces) {
                const uint4 ua = *reinterpret_cast<const uint4 *>(a + row + pc * 8);
                const uint32_t wa[4] = {ua.x, ua.y, ua.z, ua.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    v[i][2 * e] = __uint_as_float(wa[e] << 16);
                    v[i][2 * e + 1] = __uint_as_float(wa[e] & 0xffff0000u);
                }
                if (b != nullptr) {
                    const uint4 ub = *reinterpret_cast<const uint4 *>(b + row + pc * 8);
                    const uint32_t wb[4] = {ub.x, ub.y, ub.z, ub.w};
                    uint32_t ws[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const __nv_bfloat162 h2 = __floats2bfloat162_rn(v[i][2 * e] + __uint_as_float(wb[e] << 16),
                                                                        v[i][2 * e + 1] + __uint_as_float(wb[e] & 0xffff0000u));
                        ws[e] = *reinterpret_cast<const uint32_t *>(&h2);
                        v[i][2 * e] = __uint_as_float(ws[e] << 16);
                        v[i][2 * e + 1] = __uint_as_float(ws[e] & 0xffff0000u);
                    }
                    *reinterpret_cast<uint4 *>(sum_out + row + pc * 8) = make_uint4(ws[0], ws[1], ws[2], ws[3]);
                }
#pragma unroll
                for (int e = 0; e < 8; ++e) s += v[i][e];
            }
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
        const float mu = s / (float)d;
        float q = 0.0f;
#pragma unroll
        for (int i = 0; i < NP; ++i)
            if (lane + 32 * i < pieces) {
#pragma unroll
                for (int e = 0; e < 8; ++e) { const float c = v[i][e] - mu; q = fmaf(c, c, q); }
            }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) q += __shfl_xor_sync(0xffffffffu, q, off);
        const float rstd = rsqrtf(q / (float)d + eps);
#pragma unroll
        for (int i = 0; i < NP; ++i) {
            const int32_t pc = lane + 32 * i;
            if (pc >= pieces) continue;
            uint32_t wo[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                float o0 = (v[i][2 * e] - mu) * rstd, o1 = (v[i][2 * e + 1] - mu) * rstd;
                if (gamma) { o0 *= __ldg(gamma + pc * 8 + 2 * e); o1 *= __ldg(gamma + pc * 8 + 2 * e + 1); }
                if (beta) { o0 += __ldg(beta + pc * 8 + 2 * e); o1 += __ldg(beta + pc * 8 + 2 * e + 1); }
                const __nv_bfloat162 h2 = __floats2bfloat162_rn(o0, o1);
                wo[e] = *reinterpret_cast<const uint32_t *>(&h2);
            }
            *reinterpret_cast<uint4 *>(y + row + pc * 8) = make_uint4(wo[0], wo[1], wo[2], wo[3]);
        }
    }
}

// ---- multi-head softmax attention, bf16 operands, fp32 accumulation and softmax ---------------------------------
// One block per (image, head): Q, K and V sit in shared memory as they are in the input (row = token, 64 elements,
// row pitch 72); a warp owns 16 query rows at a time and keeps the whole score row block in registers (S <= 16 * NT16
// keys), so the softmax is exact (no running rescale).  Both contractions are warp-level m16n8k16 MMAs whose operand
// fragments come from ldmatrix: four 8 x 8 blocks per instruction, K as stored (key-major = the "col" operand of
// Q K^T), V through the transposing form (the contraction index of P V is the key, which is V's row).  The
// probabilities are rounded to bf16 for the second contraction.  The score MMAs run with the contraction step
// outermost so that consecutive MMAs write different accumulators (no dependent chains).
constexpr int kAttD = 64;
constexpr int kAttPitch = 72;           // 36 words: the 8 rows of an 8 x 8 block fall on different banks
constexpr int kAttWarps = 7;

__device__ __forceinline__ void att_mma(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void att_ldsm4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void att_ldsm4_t(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t *>(&h);
}

template <int NT16>
__global__ void __launch_bounds__(kAttWarps * 32, 2)
attention_kernel(const __nv_bfloat16 *__restrict__ qkv, int32_t S, int32_t heads, __nv_bfloat16 *__restrict__ out)
{
    constexpr int SP = NT16 * 16;                       // padded sequence length
    constexpr int NT8 = 2 * NT16;                       // 8-key score blocks
    extern __shared__ __align__(16) uint8_t att_smem[];
    __nv_bfloat16 *Qs = reinterpret_cast<__nv_bfloat16 *>(att_smem);
    __nv_bfloat16 *Ks = Qs + SP * kAttPitch;
    __nv_bfloat16 *Vs = Ks + SP * kAttPitch;
    const int b = blockIdx.x / heads, h = blockIdx.x % heads;
    const int64_t row_pitch = (int64_t)3 * heads * kAttD;
    const __nv_bfloat16 *base = qkv + (int64_t)b * S * row_pitch + h * kAttD;

    // stage Q, K, V in 16-byte pieces; rows past the sequence are zero (a zero V row keeps 0 * V finite)
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
        *reinterpret_cast<uint4 *>(Vs + s * kAttPitch + c * 8) = v;
    }
    __syncthreads();

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, c = lane & 3;
    const int mat = lane >> 3, l8 = lane & 7;           // ldmatrix: lanes 8 i .. 8 i + 7 give the row addresses of block i
    const uint32_t q_s = (uint32_t)__cvta_generic_to_shared(Qs), k_s = (uint32_t)__cvta_generic_to_shared(Ks),
                   v_s = (uint32_t)__cvta_generic_to_shared(Vs);
    // K blocks of one instruction: keys nt * 8 + l8, columns (32 kp) + 8 mat -> b0, b1 of steps 2 kp and 2 kp + 1
    const uint32_t k_lane = k_s + (uint32_t)(l8 * kAttPitch + mat * 8) * 2u;
    // V blocks (transposed on load): keys 16 kk + 8 (mat & 1) + l8, columns 16 np + 8 (mat >> 1) -> b0, b1 of column
    // blocks 2 np and 2 np + 1
    const uint32_t v_lane = v_s + (uint32_t)(((mat & 1) * 8 + l8) * kAttPitch + (mat >> 1) * 8) * 2u;
    const float scale = 0.125f * 1.4426950408889634f;   // 1/sqrt(64) * log2(e): the softmax runs on exp2
    for (int qt = warp; qt < NT16; qt += kAttWarps) {
        if (qt * 16 >= S) break;
        // Q blocks: rows 16 qt + 8 (mat & 1) + l8, columns 16 kk + 8 (mat >> 1) -> a0 .. a3 of step kk
        uint32_t aq[4][4];
        const uint32_t q_lane = q_s + (uint32_t)((qt * 16 + (mat & 1) * 8 + l8) * kAttPitch + (mat >> 1) * 8) * 2u;
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) att_ldsm4(q_lane + kk * 32, aq[kk][0], aq[kk][1], aq[kk][2], aq[kk][3]);
        // scores of 16 query rows against all keys
        float sc[NT8][4];
#pragma unroll
        for (int nt = 0; nt < NT8; ++nt) sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.0f;
#pragma unroll
        for (int kp = 0; kp < 2; ++kp) {
#pragma unroll
            for (int nt = 0; nt < NT8; nt += 2) {
                uint32_t b[2][4];
                att_ldsm4(k_lane + (uint32_t)(nt * 8 * kAttPitch * 2 + kp * 64), b[0][0], b[0][1], b[0][2], b[0][3]);
                att_ldsm4(k_lane + (uint32_t)((nt + 1) * 8 * kAttPitch * 2 + kp * 64), b[1][0], b[1][1], b[1][2], b[1][3]);
                att_mma(sc[nt], aq[2 * kp][0], aq[2 * kp][1], aq[2 * kp][2], aq[2 * kp][3], b[0][0], b[0][1]);
                att_mma(sc[nt + 1], aq[2 * kp][0], aq[2 * kp][1], aq[2 * kp][2], aq[2 * kp][3], b[1][0], b[1][1]);
                att_mma(sc[nt], aq[2 * kp + 1][0], aq[2 * kp + 1][1], aq[2 * kp + 1][2], aq[2 * kp + 1][3], b[0][2], b[0][3]);
                att_mma(sc[nt + 1], aq[2 * kp + 1][0], aq[2 * kp + 1][1], aq[2 * kp + 1][2], aq[2 * kp + 1][3], b[1][2], b[1][3]);
            }
        }
        // mask the padded keys, row maxima (rows g and g + 8), exponentials, row sums
        float m0 = -INFINITY, m1 = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < NT8; ++nt) {
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                if (nt * 8 + 2 * c + e >= S) { sc[nt][e] = -INFINITY; sc[nt][2 + e] = -INFINITY; }
                m0 = fmaxf(m0, sc[nt][e]);
                m1 = fmaxf(m1, sc[nt][2 + e]);
            }
        }
        m0 = fmaxf(m0, __shfl_xor_sync(0xffffffffu, m0, 1)); m0 = fmaxf(m0, __shfl_xor_sync(0xffffffffu, m0, 2));
        m1 = fmaxf(m1, __shfl_xor_sync(0xffffffffu, m1, 1)); m1 = fmaxf(m1, __shfl_xor_sync(0xffffffffu, m1, 2));
        // exponentials, row sums (of the unrounded values), and the bf16 pairs that are the A fragments of the second
        // contraction: block pair (2 kk, 2 kk + 1) of the scores is exactly the a0 .. a3 layout of step kk
        float l0 = 0.0f, l1 = 0.0f;
        uint32_t pa[NT16][4];
        const float ms0 = m0 * scale, ms1 = m1 * scale;
#pragma unroll
        for (int nt = 0; nt < NT8; ++nt) {
            const float e0 = exp2f(fmaf(sc[nt][0], scale, -ms0)), e1 = exp2f(fmaf(sc[nt][1], scale, -ms0));
            const float e2 = exp2f(fmaf(sc[nt][2], scale, -ms1)), e3 = exp2f(fmaf(sc[nt][3], scale, -ms1));
            l0 += e0 + e1;
            l1 += e2 + e3;
            pa[nt >> 1][(nt & 1) * 2] = pack_bf16(e0, e1);
            pa[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16(e2, e3);
        }
        l0 += __shfl_xor_sync(0xffffffffu, l0, 1); l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
        l1 += __shfl_xor_sync(0xffffffffu, l1, 1); l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
        float o[8][4];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.0f;
#pragma unroll
        for (int kk = 0; kk < NT16; ++kk) {
#pragma unroll
            for (int np = 0; np < 4; ++np) {
                uint32_t v0, v1, v2, v3;
                att_ldsm4_t(v_lane + (uint32_t)(kk * 16 * kAttPitch * 2 + np * 32), v0, v1, v2, v3);
                att_mma(o[2 * np], pa[kk][0], pa[kk][1], pa[kk][2], pa[kk][3], v0, v1);
                att_mma(o[2 * np + 1], pa[kk][0], pa[kk][1], pa[kk][2], pa[kk][3], v2, v3);
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
    const size_t smem = (size_t)(3 * SP * kAttPitch) * sizeof(__nv_bfloat16);
    auto kern = attention_kernel<NT16>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    kern<<<(unsigned)(Nb * heads), kAttWarps * 32, smem, s>>>(qkv, S, heads, out);
    return cudaGetLastError();
}

}  // namespace

bool add_layernorm_supported(int32_t d) { return d > 0 && d % 8 == 0 && d <= 1024; }

cudaError_t launch_add_layernorm(const void *a, const void *b, void *sum_out, int64_t T, int32_t d, const float *gamma,
                                 const float *beta, float eps, void *y, cudaStream_t s)
{
    if (!add_layernorm_supported(d)) return cudaErrorInvalidValue;
    const int64_t blocks_needed = (T + 7) / 8;
    const unsigned grid = (unsigned)(blocks_needed < 148 * 16 ? (blocks_needed > 0 ? blocks_needed : 1) : 148 * 16);
    const __nv_bfloat16 *pa = static_cast<const __nv_bfloat16 *>(a), *pb = static_cast<const __nv_bfloat16 *>(b);
    __nv_bfloat16 *ps = static_cast<__nv_bfloat16 *>(sum_out), *py = static_cast<__nv_bfloat16 *>(y);
    if (d <= 256) add_layernorm_bf16_kernel<1><<<grid, 256, 0, s>>>(pa, pb, ps, T, d, gamma, beta, eps, py);
    else if (d <= 512) add_layernorm_bf16_kernel<2><<<grid, 256, 0, s>>>(pa, pb, ps, T, d, gamma, beta, eps, py);
    else if (d <= 768) add_layernorm_bf16_kernel<3><<<grid, 256, 0, s>>>(pa, pb, ps, T, d, gamma, beta, eps, py);
    else add_layernorm_bf16_kernel<4><<<grid, 256, 0, s>>>(pa, pb, ps, T, d, gamma, beta, eps, py);
    return cudaGetLastError();
}

cudaError_t launch_layernorm(const void *x, int x_dtype, int64_t T, int32_t d, const float *gamma, const float *beta, float eps,
                             void *y, int y_dtype, cudaStream_t s)
{
    const int64_t blocks_needed = (T + 7) / 8;
    const unsigned grid = (unsigned)(blocks_needed < 148 * 16 ? (blocks_needed > 0 ? blocks_needed : 1) : 148 * 16);
    if (add_layernorm_supported(d) && x_dtype == TBN_BF16 && y_dtype == TBN_BF16 && !(reinterpret_cast<uintptr_t>(x) & 15u) &&
        !(reinterpret_cast<uintptr_t>(y) & 15u))
        return launch_add_layernorm(x, nullptr, nullptr, T, d, gamma, beta, eps, y, s);
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

namespace {
std::atomic<int> g_attention_path{0};
}

int force_attention_path(int path)
{
    if (path < 0 || path > 2) return TBN_ERR_INVALID_ARG;
    g_attention_path.store(path);
    return TBN_OK;
}

int launch_attention(const void *qkv, int32_t Nb, int32_t S, int32_t heads, int32_t d_head, void *out, int *device_status,
                     cudaStream_t s)
{
    const int forced = g_attention_path.load(std::memory_order_relaxed);
    if (forced != 1 && device_status && tc_attention_supported(Nb, S, heads, d_head))
        return launch_tc_attention(qkv, Nb, S, heads, d_head, out, device_status, s);
    if (forced == 2) return TBN_ERR_UNSUPPORTED;
    const __nv_bfloat16 *q = static_cast<const __nv_bfloat16 *>(qkv);
    __nv_bfloat16 *o = static_cast<__nv_bfloat16 *>(out);
    cudaError_t e;
    if (S <= 64) e = launch_attention_nt<4>(q, Nb, S, heads, o, s);
    else if (S <= 128) e = launch_attention_nt<8>(q, Nb, S, heads, o, s);
    else e = launch_attention_nt<13>(q, Nb, S, heads, o, s);
    return e == cudaSuccess ? TBN_OK : TBN_ERR_CUDA;
}

}  // namespace tbn
