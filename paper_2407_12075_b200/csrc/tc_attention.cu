// Multi-head softmax attention on the tcgen05 tensor cores (head dimension 64, up to 208 keys): glue of the encoder
// block, not a tiled layer.  Same arithmetic as the warp-level kernel in block.cu (bf16 operands, fp32 accumulation,
// exact softmax over the whole score row, probabilities rounded to bf16 for the second contraction).
//
// One block per (image, head, block of 128 query rows).  TMA brings Q (128 x 64), K and V (SP x 64 each, SP = the key
// count rounded up to 16) into shared memory as they are stored, 128-byte swizzled (a row of 64 bf16 is exactly one
// swizzle row).
//   scores  S = Q K^T : both operands from shared memory, K-major (the contraction index, the head dimension, is
//                       contiguous in both); M = 128 query rows, N = SP keys, four MMAs of K = 16; fp32 in tensor memory.
//   softmax           : tensor-memory lane = query row, so a thread owns a whole score row: one pass for the maximum,
//                       one for exp2 / row sum / rounding to bf16; the probabilities go back into tensor memory as
//                       the A operand of the second contraction, over the scores they came from (a 32-score chunk is
//                       in registers before its first half is overwritten).
//   output  O = P V   : A = P from tensor memory, B = V from shared memory in its stored form, i.e. with the output
//                       index (head dimension) contiguous: the "MN-major" operand form (instruction descriptor bit 16),
//                       whose 128-byte-swizzled canonical layout is eight contraction rows of 128 bytes per 1024-byte
//                       group -- exactly the TMA tile.  SP / 16 MMAs of N = 64; O sits in tensor-memory columns
//                       128..191, which the scores no longer need.
// Tensor memory: 256 columns per block, so two blocks share an SM and one's softmax runs beside the other's MMAs.
// Keys past S (rows of the next image or TMA zero fill) are masked in the softmax; V rows past S are zeroed in shared
// memory so that 0 * V stays finite; query rows past S are computed and not stored.
// Warp roles (6 warps): 0 TMA loader, 1 MMA issuer / TMEM owner, 2-5 softmax and output (one lane quadrant each).
// Every wait is bounded (tc_common.cuh); a block that gives up frees its tensor memory and records the status.
#include <cstring>

#include "tc_common.cuh"

namespace tbn {

namespace {

using namespace tc;

constexpr int kTaThreads = 6 * 32;
constexpr int kTaD = 64;
constexpr uint32_t kTaTmemCols = 256;
constexpr uint32_t kTaOBase = 128;                 // O accumulator columns 128..191
constexpr uint64_t kTaDescHi = (64ull << 32) | (1ull << 46) | (2ull << 61);   // stride 1024 bytes between 8-row groups, SW128

struct TaControl {
    uint64_t bar_qk, bar_v, bar_s, bar_p, bar_o, bar_drain;
    uint32_t tmem_base;
    int abort_flag;
};

struct TaParams {
    __nv_bfloat16 *out;
    int *status;
    int32_t Nb, S, SP, heads, nqb;
};

// D[tmem] (+)= A[smem] * B[smem]^T, bf16 -> fp32, M = 128 (whole converged warp executes, the elected lane performs)
__device__ __forceinline__ void ta_mma_ss(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo, uint32_t b_hi, uint32_t idesc,
                                          uint32_t accumulate, uint32_t leader) {
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t.reg .b64 ad, bd;\n\t"
        "setp.ne.b32 q, %7, 0;\n\t"
        "setp.ne.b32 p, %6, 0;\n\t"
        "mov.b64 ad, {%1, %2};\n\t"
        "mov.b64 bd, {%3, %4};\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%0], ad, bd, %5, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate), "r"(leader) : "memory");
}

__device__ __forceinline__ float ta_exp2(float v) {
    float r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(v));
    return r;
}
__device__ __forceinline__ uint32_t ta_pack(float lo, float hi) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t *>(&h);
}

__global__ void __launch_bounds__(kTaThreads)
tc_attention_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap kv_map, const TaParams p)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    uint8_t *smem = smem_raw + ((1024u - (raw & 1023u)) & 1023u);
    const uint32_t kv_bytes = (uint32_t)p.SP * 128u;                       // a multiple of 2048
    const uint32_t q_s = smem_u32(smem), k_s = q_s + 16384u, v_s = k_s + kv_bytes;
    TaControl *ctl = reinterpret_cast<TaControl *>(smem + 16384u + 2u * kv_bytes);
    volatile int *abort_flag = &ctl->abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int32_t qb = blockIdx.x % p.nqb;
    const int32_t bh = blockIdx.x / p.nqb;
    const int32_t b = bh / p.heads, h = bh % p.heads;
    const int detail = (int)(blockIdx.x & 0xffff);

    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&ctl->bar_qk), 1);
        mbar_init(smem_u32(&ctl->bar_v), 1);
        mbar_init(smem_u32(&ctl->bar_s), 1);
        mbar_init(smem_u32(&ctl->bar_p), 128);
        mbar_init(smem_u32(&ctl->bar_o), 1);
        mbar_init(smem_u32(&ctl->bar_drain), 1);
        ctl->abort_flag = 0;
        fence_barrier_init();
        fence_proxy_async();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&ctl->tmem_base), kTaTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;
    bool ok = true;

    if (warp == 0) {
        // ---------------- loader ----------------
        if (lane == 0) {
            const int32_t row0 = b * p.S;
            mbar_arrive_expect_tx(smem_u32(&ctl->bar_qk), 16384u + kv_bytes);
            tma_load_2d(q_s, &q_map, h * kTaD, row0 + qb * 128, smem_u32(&ctl->bar_qk));
            tma_load_2d(k_s, &kv_map, (p.heads + h) * kTaD, row0, smem_u32(&ctl->bar_qk));
            mbar_arrive_expect_tx(smem_u32(&ctl->bar_v), kv_bytes);
            tma_load_2d(v_s, &kv_map, (2 * p.heads + h) * kTaD, row0, smem_u32(&ctl->bar_v));
        }
        __syncwarp();
        // the copies have landed before this block's shared memory goes away, whatever the other warps do
        drain_wait(smem_u32(&ctl->bar_qk), 0);
        drain_wait(smem_u32(&ctl->bar_v), 0);
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        const uint32_t tmem_u = __shfl_sync(0xffffffffu, tmem_base, 0);
        const uint32_t leader = elect_one();
        constexpr uint32_t kHi = (uint32_t)(kTaDescHi >> 32);
        const uint32_t n1 = (uint32_t)p.SP;
        // instruction descriptors: D fp32, A and B bf16, M = 128; scores: both K-major, N = SP; output: B MN-major, N = 64
        const uint32_t idesc_s = (1u << 4) | (1u << 7) | (1u << 10) | ((n1 >> 3) << 17) | (8u << 24);
        const uint32_t idesc_o = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((64u >> 3) << 17) | (8u << 24);
        ok = wait_bar(smem_u32(&ctl->bar_qk), 0, abort_flag, p.status, (20 << 24) | detail);
        if (ok) {
            tc_fence_after();
            const uint32_t a_lo = ((q_s & 0x3FFFFu) >> 4) | (1u << 16), b_lo = ((k_s & 0x3FFFFu) >> 4) | (1u << 16);
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)                       // 16 head-dimension elements = 32 bytes per step
                ta_mma_ss(tmem_u, a_lo + kk * 2, kHi, b_lo + kk * 2, kHi, idesc_s, kk > 0 ? 1u : 0u, leader);
            tc_commit_elect(smem_u32(&ctl->bar_s), leader);
            ok = wait_bar(smem_u32(&ctl->bar_v), 0, abort_flag, p.status, (21 << 24) | detail) &&
                 wait_bar(smem_u32(&ctl->bar_p), 0, abort_flag, p.status, (22 << 24) | detail);
        }
        if (ok) {
            tc_fence_after();
            // 16 keys per step: two 8-row groups of V (2048 bytes), eight tensor-memory columns of P
            const uint32_t v_lo = ((v_s & 0x3FFFFu) >> 4) | (64u << 16);
            const int steps = p.SP >> 4;
            for (int kk = 0; kk < steps; ++kk)
                tc_mma_ts_elect(tmem_u + kTaOBase, tmem_u + (uint32_t)kk * 8u, v_lo + (uint32_t)kk * 128u, kHi, idesc_o,
                                kk > 0 ? 1u : 0u, leader);
            tc_commit_elect(smem_u32(&ctl->bar_o), leader);
        }
        __syncwarp();
    } else {
        // ---------------- softmax and output: thread = query row ----------------
        const int qd = warp & 3;
        const uint32_t t_row = tmem_base + ((uint32_t)(qd * 32) << 16);
        const int32_t qrow = qb * 128 + qd * 32 + lane;
        const bool warp_live = qb * 128 + qd * 32 < p.S;                  // some row of this warp is a query of the image
        const int32_t S = p.S;
        const int nfull = p.SP >> 5;
        const bool tail = (p.SP & 31) != 0;                               // 16 more score columns
        const float scale = 0.125f * 1.4426950408889634f;                 // 1/sqrt(64) * log2(e): softmax on exp2
        float l = 0.0f;
        ok = wait_bar(smem_u32(&ctl->bar_s), 0, abort_flag, p.status, (23 << 24) | detail);
        if (ok && warp_live) {
            tc_fence_after();
            float m = -INFINITY;
#pragma unroll 1
            for (int c = 0; c < nfull; ++c) {
                uint32_t v[32];
                tmem_ld_32x32(t_row + (uint32_t)c * 32u, v);
                tc_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; ++i) m = (c * 32 + i < S) ? fmaxf(m, __uint_as_float(v[i])) : m;
            }
            if (tail) {
                uint32_t v[16];
                tmem_ld_32x16(t_row + (uint32_t)nfull * 32u, v);
                tc_wait_ld();
#pragma unroll
                for (int i = 0; i < 16; ++i) m = (nfull * 32 + i < S) ? fmaxf(m, __uint_as_float(v[i])) : m;
            }
            const float ms = m * scale;
#pragma unroll 1
            for (int c = 0; c < nfull; ++c) {
                uint32_t v[32], pk[16];
                tmem_ld_32x32(t_row + (uint32_t)c * 32u, v);
                tc_wait_ld();
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const int col = c * 32 + 2 * i;
                    const float e0 = col < S ? ta_exp2(fmaf(__uint_as_float(v[2 * i]), scale, -ms)) : 0.0f;
                    const float e1 = col + 1 < S ? ta_exp2(fmaf(__uint_as_float(v[2 * i + 1]), scale, -ms)) : 0.0f;
                    l += e0 + e1;
                    pk[i] = ta_pack(e0, e1);
                }
                tmem_st_32x8(t_row + (uint32_t)c * 16u, pk);
                tmem_st_32x8(t_row + (uint32_t)c * 16u + 8u, pk + 8);
            }
            if (tail) {
                uint32_t v[16], pk[8];
                tmem_ld_32x16(t_row + (uint32_t)nfull * 32u, v);
                tc_wait_ld();
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int col = nfull * 32 + 2 * i;
                    const float e0 = col < S ? ta_exp2(fmaf(__uint_as_float(v[2 * i]), scale, -ms)) : 0.0f;
                    const float e1 = col + 1 < S ? ta_exp2(fmaf(__uint_as_float(v[2 * i + 1]), scale, -ms)) : 0.0f;
                    l += e0 + e1;
                    pk[i] = ta_pack(e0, e1);
                }
                tmem_st_32x8(t_row + (uint32_t)nfull * 16u, pk);
            }
            tc_wait_st();
        }
        if (ok) {
            // V rows past the last key hold the next image's rows (or zero fill): zero them, 16 bytes per thread
            bool v_ok = true;
            if (p.SP > S) {
                v_ok = wait_bar(smem_u32(&ctl->bar_v), 0, abort_flag, p.status, (24 << 24) | detail);
                const int idx = (warp - 2) * 32 + lane;
                if (v_ok && idx < (p.SP - S) * 8) sts_v4(v_s + (uint32_t)(S + (idx >> 3)) * 128u + (uint32_t)(idx & 7) * 16u, 0u, 0u, 0u, 0u);
                fence_proxy_async();
            }
            ok = v_ok;
        }
        if (ok) {
            tc_fence_before();
            mbar_arrive(smem_u32(&ctl->bar_p));
            ok = wait_bar(smem_u32(&ctl->bar_o), 0, abort_flag, p.status, (25 << 24) | detail);
        }
        if (ok && warp_live) {
            tc_fence_after();
            uint32_t o0[32], o1[32];
            tmem_ld_32x32(t_row + kTaOBase, o0);
            tmem_ld_32x32(t_row + kTaOBase + 32u, o1);
            tc_wait_ld();
            if (qrow < S) {
                const float r = 1.0f / l;
                uint4 *dst = reinterpret_cast<uint4 *>(p.out + ((int64_t)b * S + qrow) * ((int64_t)p.heads * kTaD) + h * kTaD);
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    dst[i] = make_uint4(ta_pack(__uint_as_float(o0[8 * i]) * r, __uint_as_float(o0[8 * i + 1]) * r),
                                        ta_pack(__uint_as_float(o0[8 * i + 2]) * r, __uint_as_float(o0[8 * i + 3]) * r),
                                        ta_pack(__uint_as_float(o0[8 * i + 4]) * r, __uint_as_float(o0[8 * i + 5]) * r),
                                        ta_pack(__uint_as_float(o0[8 * i + 6]) * r, __uint_as_float(o0[8 * i + 7]) * r));
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    dst[4 + i] = make_uint4(ta_pack(__uint_as_float(o1[8 * i]) * r, __uint_as_float(o1[8 * i + 1]) * r),
                                            ta_pack(__uint_as_float(o1[8 * i + 2]) * r, __uint_as_float(o1[8 * i + 3]) * r),
                                            ta_pack(__uint_as_float(o1[8 * i + 4]) * r, __uint_as_float(o1[8 * i + 5]) * r),
                                            ta_pack(__uint_as_float(o1[8 * i + 6]) * r, __uint_as_float(o1[8 * i + 7]) * r));
            }
        }
    }

    // ---------------- teardown ----------------
    if (warp == 1 && *abort_flag) {
        // no MMA may still be reading shared or tensor memory when they are released
        tc_commit_elect(smem_u32(&ctl->bar_drain), elect_one());
        __syncwarp();
        drain_wait(smem_u32(&ctl->bar_drain), 0);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTaTmemCols);
    }
}

}  // namespace

bool tc_attention_supported(int32_t Nb, int32_t S, int32_t heads, int32_t d_head)
{
    if (d_head != kTaD || S < 1 || S > 208 || heads < 1 || Nb < 1) return false;
    const int64_t blocks = (int64_t)Nb * heads * ((S + 127) / 128);
    return blocks <= 0x7fffffffLL && (int64_t)Nb * S < ((int64_t)1 << 31) - 256 && (int64_t)3 * heads * kTaD < ((int64_t)1 << 31);
}

int launch_tc_attention(const void *qkv, int32_t Nb, int32_t S, int32_t heads, int32_t d_head, void *out, int *device_status,
                        cudaStream_t s)
{
    if (!tc_attention_supported(Nb, S, heads, d_head)) return TBN_ERR_UNSUPPORTED;
    EncodeTiledFn encode = encode_tiled_fn();
    if (!encode) return TBN_ERR_CUDA;
    TaParams p;
    p.out = static_cast<__nv_bfloat16 *>(out); p.status = device_status;
    p.Nb = Nb; p.S = S; p.SP = (S + 15) / 16 * 16; p.heads = heads; p.nqb = (S + 127) / 128;
    // qkv as (3 * heads * 64 columns, Nb * S rows); a box is 64 columns (one head of q, k or v) by 128 or SP rows
    CUtensorMap q_map, kv_map;
    const cuuint64_t dims[2] = {(cuuint64_t)3 * heads * kTaD, (cuuint64_t)Nb * S};
    const cuuint64_t strides[1] = {(cuuint64_t)3 * heads * kTaD * 2};
    const cuuint32_t estr[2] = {1, 1};
    const cuuint32_t box_q[2] = {(cuuint32_t)kTaD, 128}, box_kv[2] = {(cuuint32_t)kTaD, (cuuint32_t)p.SP};
    if (encode(&q_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(qkv), dims, strides, box_q, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS ||
        encode(&kv_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(qkv), dims, strides, box_kv, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return TBN_ERR_CUDA;
    const size_t smem = 16384 + 2 * (size_t)p.SP * 128 + sizeof(TaControl) + 1024;
    if (cudaFuncSetAttribute(tc_attention_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return TBN_ERR_CUDA;
    const unsigned grid = (unsigned)((int64_t)Nb * heads * p.nqb);
    tc_attention_kernel<<<grid, kTaThreads, smem, s>>>(q_map, kv_map, p);
    return cudaGetLastError() == cudaSuccess ? TBN_OK : TBN_ERR_CUDA;
}

}  // namespace tbn
