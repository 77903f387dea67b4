// Multi-head softmax attention on the tcgen05 tensor cores (head dimension 64, up to 208 keys): glue of the encoder
// block, not a tiled layer.  Same arithmetic as the warp-level kernel in block.cu (bf16 operands, fp32 accumulation,
// exact softmax over the whole score row, probabilities rounded to bf16 for the second contraction).
//
// A work item is (image, head, block of 128 query rows); a block (one per SM) takes items block, block + grid, ... and
// keeps two in flight (three shared-memory stages filled ahead, two 256-column tensor-memory buffers, two groups of softmax warps).  TMA brings Q (128 x 64), K and V (SP x 64 each, SP = the key
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
// Tensor memory: 256 columns per item in flight, so one item's softmax runs beside the other's MMAs and copies.
// Keys past S (rows of the next image or TMA zero fill) are masked in the softmax; V rows past S are zeroed in shared
// memory so that 0 * V stays finite; query rows past S are computed and not stored.
// Warp roles (10 warps): 0 TMA loader, 1 MMA issuer / TMEM owner, 2-5 and 6-9 softmax and output of the even and the odd
// items (one lane quadrant per warp).
// Every wait is bounded (tc_common.cuh); a block that gives up frees its tensor memory and records the status.
#include <cstring>

#include "tc_common.cuh"

namespace tbn {

namespace {

using namespace tc;

constexpr int kTaThreads = 10 * 32;
constexpr int kTaD = 64;
constexpr int kTaStages = 3;                       // Q/K/V stages in shared memory (copies run ahead of the two buffers)
constexpr uint32_t kTaTmemCols = 512;              // two buffers of 256 columns
constexpr uint32_t kTaBufCols = 256;
constexpr uint32_t kTaOBase = 128;                 // O accumulator: columns 128..191 of a buffer
constexpr uint64_t kTaDescHi = (64ull << 32) | (1ull << 46) | (2ull << 61);   // stride 1024 bytes between 8-row groups, SW128

struct TaControl {
    uint64_t full_qk[kTaStages], full_v[kTaStages], stage_free[kTaStages];
    uint64_t s_full[2], p_full[2], o_full[2], t_empty[2], bar_drain;
    uint32_t tmem_base;
    int abort_flag;
};

struct TaParams {
    __nv_bfloat16 *out;
    int *status;
    int32_t Nb, S, SP, heads, nqb, items;
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

// maxima of N score columns starting at col0 into four partial maxima; MASK: columns >= S do not count
template <int N, bool MASK>
__device__ __forceinline__ void ta_max(const uint32_t (&v)[32], int col0, int S, float (&mx)[4]) {
#pragma unroll
    for (int i = 0; i < N; ++i) {
        float x = __uint_as_float(v[i]);
        if (MASK) x = col0 + i < S ? x : -INFINITY;
        mx[i & 3] = fmaxf(mx[i & 3], x);
    }
}
// exp2(score * scale - ms) of N columns: bf16 pairs into pk, four partial sums of the unrounded values
template <int N, bool MASK>
__device__ __forceinline__ void ta_exp(const uint32_t (&v)[32], int col0, int S, float scale, float ms, float (&ls)[4], uint32_t (&pk)[16]) {
#pragma unroll
    for (int i = 0; i < N / 2; ++i) {
        float e0 = ta_exp2(fmaf(__uint_as_float(v[2 * i]), scale, -ms)), e1 = ta_exp2(fmaf(__uint_as_float(v[2 * i + 1]), scale, -ms));
        if (MASK) {
            e0 = col0 + 2 * i < S ? e0 : 0.0f;
            e1 = col0 + 2 * i + 1 < S ? e1 : 0.0f;
        }
        ls[i & 3] += e0 + e1;
        pk[i] = ta_pack(e0, e1);
    }
}

// Item j of a block (its items are block, block + grid, ...) uses shared-memory stage j mod 3 and buffer j mod 2 -- 256
// tensor-memory columns and one group of four softmax warps -- and completes phase (j div 3) mod 2 of the stage's and
// (j div 2) mod 2 of the buffer's barriers.  The MMA warp interleaves: scores of item j, then output of item j - 1, so each group's softmax runs beside
// the other item's MMAs and the loader's copies.
__global__ void __launch_bounds__(kTaThreads, 1)
tc_attention_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap kv_map, const TaParams p)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    uint8_t *smem = smem_raw + ((1024u - (raw & 1023u)) & 1023u);
    const uint32_t kv_bytes = (uint32_t)p.SP * 128u;                       // a multiple of 2048
    const uint32_t buf_bytes = 16384u + 2u * kv_bytes;
    const uint32_t smem0 = smem_u32(smem);
    TaControl *ctl = reinterpret_cast<TaControl *>(smem + (uint32_t)kTaStages * buf_bytes);
    volatile int *abort_flag = &ctl->abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int detail = (int)(blockIdx.x & 0xffff);
    const int32_t n_local = (p.items - (int32_t)blockIdx.x + (int32_t)gridDim.x - 1) / (int32_t)gridDim.x;

    if (threadIdx.x == 0) {
        for (int st = 0; st < kTaStages; ++st) {
            mbar_init(smem_u32(&ctl->full_qk[st]), 1);
            mbar_init(smem_u32(&ctl->full_v[st]), 1);
            mbar_init(smem_u32(&ctl->stage_free[st]), 1);
        }
        for (int u = 0; u < 2; ++u) {
            mbar_init(smem_u32(&ctl->s_full[u]), 1);
            mbar_init(smem_u32(&ctl->p_full[u]), 128);
            mbar_init(smem_u32(&ctl->o_full[u]), 1);
            mbar_init(smem_u32(&ctl->t_empty[u]), 128);
        }
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
        int issued = 0;
        for (int32_t j = 0; j < n_local && ok; ++j) {
            const int st = j % kTaStages;
            if (j >= kTaStages) {   // the stage is free once the output MMAs of its previous item have completed
                ok = wait_bar(smem_u32(&ctl->stage_free[st]), (uint32_t)(j / kTaStages - 1) & 1u, abort_flag, p.status,
                              (26 << 24) | detail);
                if (!ok) break;
            }
            if (lane == 0) {
                const int32_t item = (int32_t)blockIdx.x + j * (int32_t)gridDim.x;
                const int32_t qb = item % p.nqb, bh = item / p.nqb;
                const int32_t b = bh / p.heads, h = bh % p.heads;
                const int32_t row0 = b * p.S;
                const uint32_t q_s = smem0 + (uint32_t)st * buf_bytes, k_s = q_s + 16384u, v_s = k_s + kv_bytes;
                mbar_arrive_expect_tx(smem_u32(&ctl->full_qk[st]), 16384u + kv_bytes);
                tma_load_2d(q_s, &q_map, h * kTaD, row0 + qb * 128, smem_u32(&ctl->full_qk[st]));
                tma_load_2d(k_s, &kv_map, (p.heads + h) * kTaD, row0, smem_u32(&ctl->full_qk[st]));
                mbar_arrive_expect_tx(smem_u32(&ctl->full_v[st]), kv_bytes);
                tma_load_2d(v_s, &kv_map, (2 * p.heads + h) * kTaD, row0, smem_u32(&ctl->full_v[st]));
            }
            issued = j + 1;
            __syncwarp();
        }
        if (!ok) {   // let copies in flight land before the block's shared memory goes away
            for (int32_t j = issued > kTaStages ? issued - kTaStages : 0; j < issued; ++j) {
                drain_wait(smem_u32(&ctl->full_qk[j % kTaStages]), (uint32_t)(j / kTaStages) & 1u);
                drain_wait(smem_u32(&ctl->full_v[j % kTaStages]), (uint32_t)(j / kTaStages) & 1u);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        const uint32_t tmem_u = __shfl_sync(0xffffffffu, tmem_base, 0);
        const uint32_t leader = elect_one();
        constexpr uint32_t kHi = (uint32_t)(kTaDescHi >> 32);
        // instruction descriptors: D fp32, A and B bf16, M = 128; scores: both K-major, N = SP; output: B MN-major, N = 64
        const uint32_t idesc_s = (1u << 4) | (1u << 7) | (1u << 10) | (((uint32_t)p.SP >> 3) << 17) | (8u << 24);
        const uint32_t idesc_o = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((64u >> 3) << 17) | (8u << 24);
        const int steps = p.SP >> 4;
        for (int32_t j = 0; j <= n_local && ok; ++j) {
            if (j < n_local) {                                   // scores of item j
                const int u = j & 1, st = j % kTaStages;
                ok = wait_bar(smem_u32(&ctl->full_qk[st]), (uint32_t)(j / kTaStages) & 1u, abort_flag, p.status, (20 << 24) | detail);
                if (ok && j >= 2)                                // the buffer's previous output has been read
                    ok = wait_bar(smem_u32(&ctl->t_empty[u]), (uint32_t)((j - 2) >> 1) & 1u, abort_flag, p.status, (27 << 24) | detail);
                if (!ok) break;
                tc_fence_after();
                const uint32_t q_s = smem0 + (uint32_t)st * buf_bytes, k_s = q_s + 16384u;
                const uint32_t a_lo = ((q_s & 0x3FFFFu) >> 4) | (1u << 16), b_lo = ((k_s & 0x3FFFFu) >> 4) | (1u << 16);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)                   // 16 head-dimension elements = 32 bytes per step
                    ta_mma_ss(tmem_u + (uint32_t)u * kTaBufCols, a_lo + kk * 2, kHi, b_lo + kk * 2, kHi, idesc_s, kk > 0 ? 1u : 0u,
                              leader);
                tc_commit_elect(smem_u32(&ctl->s_full[u]), leader);
            }
            if (j >= 1) {                                        // output of item j - 1
                const int u = (j - 1) & 1, st = (j - 1) % kTaStages;
                const uint32_t ph = (uint32_t)((j - 1) >> 1) & 1u;
                ok = wait_bar(smem_u32(&ctl->full_v[st]), (uint32_t)((j - 1) / kTaStages) & 1u, abort_flag, p.status, (21 << 24) | detail) &&
                     wait_bar(smem_u32(&ctl->p_full[u]), ph, abort_flag, p.status, (22 << 24) | detail);
                if (!ok) break;
                tc_fence_after();
                // 16 keys per step: two 8-row groups of V (2048 bytes), eight tensor-memory columns of P
                const uint32_t v_s = smem0 + (uint32_t)st * buf_bytes + 16384u + kv_bytes;
                const uint32_t v_lo = ((v_s & 0x3FFFFu) >> 4) | (64u << 16);
                const uint32_t t_buf = tmem_u + (uint32_t)u * kTaBufCols;
                for (int kk = 0; kk < steps; ++kk)
                    tc_mma_ts_elect(t_buf + kTaOBase, t_buf + (uint32_t)kk * 8u, v_lo + (uint32_t)kk * 128u, kHi, idesc_o,
                                    kk > 0 ? 1u : 0u, leader);
                tc_commit_elect(smem_u32(&ctl->o_full[u]), leader);
                tc_commit_elect(smem_u32(&ctl->stage_free[st]), leader);
            }
        }
        __syncwarp();
    } else {
        // ---------------- softmax and output: group g = buffer g, thread = query row ----------------
        const int g = (warp - 2) >> 2;
        const int qd = warp & 3;
        const uint32_t t_row = tmem_base + ((uint32_t)(qd * 32) << 16) + (uint32_t)g * kTaBufCols;
        const int32_t S = p.S;
        const int nfull = p.SP >> 5;
        const int nch = nfull + ((p.SP & 31) != 0 ? 1 : 0);               // SP % 32 == 16: a last chunk of 16 columns
        const float scale = 0.125f * 1.4426950408889634f;                 // 1/sqrt(64) * log2(e): softmax on exp2
        for (int32_t j = g; j < n_local && ok; j += 2) {
            const uint32_t ph = (uint32_t)(j >> 1) & 1u;
            const int32_t item = (int32_t)blockIdx.x + j * (int32_t)gridDim.x;
            const int32_t qb = item % p.nqb, bh = item / p.nqb;
            const int32_t b = bh / p.heads, h = bh % p.heads;
            const int32_t qrow = qb * 128 + qd * 32 + lane;
            const bool warp_live = qb * 128 + qd * 32 < S;                // some row of this warp is a query of the image
            float l = 0.0f;
            ok = wait_bar(smem_u32(&ctl->s_full[g]), ph, abort_flag, p.status, (23 << 24) | detail);
            if (!ok) break;
            if (warp_live) {
                tc_fence_after();
                // Two passes over the row in chunks of 32 columns (a last one of 16), the load of chunk c + 1 in flight
                // while chunk c is processed; four partial maxima / sums keep the arithmetic chains short; only chunks
                // that reach past the last key pay for the mask.
                uint32_t va[32], vb[32];
                auto ld = [&](uint32_t (&v)[32], int c) {
                    if (c < nfull) tmem_ld_32x32(t_row + (uint32_t)c * 32u, v);
                    else tmem_ld_32x16(t_row + (uint32_t)c * 32u, *reinterpret_cast<uint32_t (*)[16]>(v));
                };
                float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
                auto max_chunk = [&](const uint32_t (&v)[32], int c) {
                    const int col0 = c * 32;
                    if (c < nfull) {
                        if (col0 + 32 <= S) ta_max<32, false>(v, col0, S, mx); else ta_max<32, true>(v, col0, S, mx);
                    } else {
                        if (col0 + 16 <= S) ta_max<16, false>(v, col0, S, mx); else ta_max<16, true>(v, col0, S, mx);
                    }
                };
                ld(va, 0);
#pragma unroll 1
                for (int c = 0; c < nch; c += 2) {
                    tc_wait_ld();
                    if (c + 1 < nch) ld(vb, c + 1);
                    max_chunk(va, c);
                    if (c + 1 >= nch) break;
                    tc_wait_ld();
                    if (c + 2 < nch) ld(va, c + 2);
                    max_chunk(vb, c + 1);
                }
                const float ms = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * scale;
                float ls[4] = {0.0f, 0.0f, 0.0f, 0.0f};
                auto exp_chunk = [&](const uint32_t (&v)[32], int c) {
                    const int col0 = c * 32;
                    uint32_t pk[16];
                    if (c < nfull) {
                        if (col0 + 32 <= S) ta_exp<32, false>(v, col0, S, scale, ms, ls, pk); else ta_exp<32, true>(v, col0, S, scale, ms, ls, pk);
                        tmem_st_32x8(t_row + (uint32_t)c * 16u, pk);
                        tmem_st_32x8(t_row + (uint32_t)c * 16u + 8u, pk + 8);
                    } else {
                        if (col0 + 16 <= S) ta_exp<16, false>(v, col0, S, scale, ms, ls, pk); else ta_exp<16, true>(v, col0, S, scale, ms, ls, pk);
                        tmem_st_32x8(t_row + (uint32_t)c * 16u, pk);
                    }
                };
                ld(va, 0);
#pragma unroll 1
                for (int c = 0; c < nch; c += 2) {
                    tc_wait_ld();
                    if (c + 1 < nch) ld(vb, c + 1);
                    exp_chunk(va, c);
                    if (c + 1 >= nch) break;
                    tc_wait_ld();
                    if (c + 2 < nch) ld(va, c + 2);
                    exp_chunk(vb, c + 1);
                }
                l = (ls[0] + ls[1]) + (ls[2] + ls[3]);
                tc_wait_st();
            }
            // V rows past the last key hold the next image's rows (or zero fill): zero them, 16 bytes per thread
            if (p.SP > S) {
                const int st = j % kTaStages;
                const uint32_t v_s = smem0 + (uint32_t)st * buf_bytes + 16384u + kv_bytes;
                ok = wait_bar(smem_u32(&ctl->full_v[st]), (uint32_t)(j / kTaStages) & 1u, abort_flag, p.status, (24 << 24) | detail);
                if (!ok) break;
                const int idx = ((warp - 2) & 3) * 32 + lane;
                if (idx < (p.SP - S) * 8) sts_v4(v_s + (uint32_t)(S + (idx >> 3)) * 128u + (uint32_t)(idx & 7) * 16u, 0u, 0u, 0u, 0u);
                fence_proxy_async();
            }
            tc_fence_before();
            mbar_arrive(smem_u32(&ctl->p_full[g]));
            ok = wait_bar(smem_u32(&ctl->o_full[g]), ph, abort_flag, p.status, (25 << 24) | detail);
            if (!ok) break;
            if (warp_live) {
                tc_fence_after();
                uint32_t o0[32], o1[32];
                tmem_ld_32x32(t_row + kTaOBase, o0);
                tmem_ld_32x32(t_row + kTaOBase + 32u, o1);
                tc_wait_ld();
                tc_fence_before();
                mbar_arrive(smem_u32(&ctl->t_empty[g]));               // the buffer's tensor memory may be overwritten
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
            } else {
                mbar_arrive(smem_u32(&ctl->t_empty[g]));
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
    p.items = (int32_t)((int64_t)Nb * heads * p.nqb);
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
    const size_t smem = kTaStages * (16384 + 2 * (size_t)p.SP * 128) + sizeof(TaControl) + 1024;
    if (cudaFuncSetAttribute(tc_attention_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return TBN_ERR_CUDA;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
        return TBN_ERR_CUDA;
    const unsigned grid = (unsigned)(p.items < sms ? p.items : sms);
    tc_attention_kernel<<<grid, kTaThreads, smem, s>>>(q_map, kv_map, p);
    return cudaGetLastError() == cudaSuccess ? TBN_OK : TBN_ERR_CUDA;
}

}  // namespace tbn
