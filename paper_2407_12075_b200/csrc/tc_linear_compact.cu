// Tensor-core forward of a tiled layer whose INPUT is the compact form of the previous tiled layer's output
// (Sec. 4.1: with a tile that spans whole rows, the k repetitions of an output channel differ only by their alpha).
//
// The previous layer (tile of r_z distinct rows, k_z repetitions, alphas a_j) would write
//     h[t][j * r_z + c] = act_z(a_j * z[t][c]),      j < k_z, c < r_z,
// a tensor k_z times larger than the r_z distinct pre-activations z it is made of.  Here the previous layer writes
// only z (bf16, T x r_z) and this kernel rebuilds the activation operand while it stages it: TMA brings the raw z
// of a stage into the swizzled K-major shared-memory stage that tcgen05.mma reads, and producer warps apply
// act_z(a_j * .) to it in place for the repetition j the stage belongs to.  The k_z-fold broadcast never exists in HBM: the
// previous layer writes k_z times fewer bytes and this one reads k_z times fewer.  With a ReLU (or no) activation the
// same saving is had by folding the alphas into the weights (the MLP chain does that); with GELU there is nothing to
// fold, and the activation is evaluated here instead of in the previous layer's epilogue (the same number of
// evaluations, T * k_z * r_z, but spread over this kernel's main loop).
//
// Everything else is the bf16 kernel's design: decoded +-1 weights are the A operand in tensor memory, fp32
// accumulators in tensor memory (two buffers), k-fold replicated epilogue.  Warp roles (18 warps): 0-7 activation
// producers, 8 MMA issuer / TMEM owner, 9-12 weight decode, 13-16 epilogue, 17 TMA loader.  Every wait is bounded (tc_common.cuh).
#include <cstddef>

#include "tc_common.cuh"

namespace tbn {

namespace {

using namespace tc;

constexpr int kCpProdWarps = 8;
constexpr int kCpProd = kCpProdWarps * 32;       // producer threads
constexpr int kCpMmaWarp = kCpProdWarps;
constexpr int kCpLoadWarp = kCpProdWarps + 9;
constexpr int kCpThreads = (kCpProdWarps + 10) * 32;
constexpr int kCpAtomK = 64;                     // bf16 elements per 128-byte swizzle row
constexpr int kCpKA = 2;                         // swizzle rows per stage: 128 contraction elements
constexpr int kCpStageK = kCpKA * kCpAtomK;
constexpr int kCpAStages = 4;                    // decoded-weight stages in tensor memory, 64 columns each
constexpr int kCpACols = kCpKA * 32;
constexpr int kCpXPitch = 132;

template <int SX>
struct CpControl {
    uint64_t raw_full[SX], x_full[SX], x_empty[SX];
    uint64_t a_full[kCpAStages], a_empty[kCpAStages];
    uint64_t d_full[2], d_empty[2];
    uint32_t tmem_base;
    int abort_flag;
    float alpha[64];                             // this layer's alphas
    float alpha_z[64];                           // the previous layer's alphas
    alignas(16) float exchange[32 * kCpXPitch];
};

struct CpParams {
    const __nv_bfloat16 *z;      // [T][rz]
    const float *alpha_z;
    const uint32_t *tile;
    const float *alpha;
    const float *bias;
    void *y;
    int *status;
    int64_t T;
    int64_t n_words;
    int32_t rz, kz;              // distinct columns and repetitions of the previous layer; n = rz * kz
    int32_t n, m, r, k;
    int32_t k_stages, w_tiles, t_tiles;
    int per_tile_z, act_z, per_tile, act, y_bf16;
};

// 16 tile bits -> 8 registers of two bf16 each (+1.0 = 0x3F80, -1.0 = 0xBF80): even bits in the low halves
__device__ __forceinline__ void cp_decode16(uint32_t h, uint32_t *out) {
    const uint32_t v = (h | (h << 15)) & 0x55555555u;
#pragma unroll
    for (int j = 0; j < 8; ++j) out[j] = ((v << (15 - 2 * j)) & 0x80008000u) ^ 0xBF80BF80u;
}

__device__ __forceinline__ void cp_epi_bar() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
__device__ __forceinline__ int cp_epi_bar_count(bool pred) {
    int n;
    asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %1, 0;\nbar.red.popc.u32 %0, 1, 128, p;\n}"
                 : "=r"(n) : "r"((int)pred) : "memory");
    return n;
}

// act_z(a * v) for two packed bf16 values -> two packed bf16 values
__device__ __forceinline__ uint32_t cp_act_pair(uint32_t packed, float a, int act_z) {
    const float v0 = a * __uint_as_float(packed << 16), v1 = a * __uint_as_float(packed & 0xffff0000u);
    float o0, o1;
    if (act_z == TBN_ACT_GELU) {
        gelu_tanh_bf16_pair(1.0f, v0, v1, 0.0f, 0.0f, o0, o1);
    } else if (act_z == TBN_ACT_RELU) {
        o0 = fmaxf(v0, 0.0f); o1 = fmaxf(v1, 0.0f);
    } else {
        o0 = v0; o1 = v1;
    }
    const __nv_bfloat162 h = __floats2bfloat162_rn(o0, o1);
    return *reinterpret_cast<const uint32_t *>(&h);
}

constexpr uint64_t kCpBDescHi = (64ull << 32) | (1ull << 46) | (2ull << 61);   // SW128, K-major (as the bf16 kernel)

template <int NTOK, int SX>
__global__ void __launch_bounds__(kCpThreads, 1)
tc_linear_compact_kernel(const __grid_constant__ CUtensorMap z_map, const CpParams p)
{
    static_assert(NTOK == 128 && kCpProd == 256, "a producer thread owns one 16-byte piece of four token rows per swizzle row");
    constexpr int DB = 2;
    constexpr uint32_t kAtomBytes = NTOK * 128;
    constexpr uint32_t kStageBytes = kCpKA * kAtomBytes;
    constexpr uint32_t kDCols = NTOK;
    constexpr uint32_t kABase = DB * kDCols;
    constexpr uint32_t kTmemCols = 512;
    static_assert(kABase + kCpAStages * kCpACols <= kTmemCols, "tensor memory budget");
    // instruction descriptor: D fp32, A and B bf16, both K-major, N = NTOK, M = 128
    constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(NTOK >> 3) << 17) | (8u << 24);

    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    uint8_t *smem = smem_raw + ((1024u - (raw & 1023u)) & 1023u);
    CpControl<SX> *ctl = reinterpret_cast<CpControl<SX> *>(smem + SX * kStageBytes);
    const uint32_t stage0 = smem_u32(smem);
    volatile int *abort_flag = &ctl->abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int bid = blockIdx.x;

    if (threadIdx.x == 0) {
        for (int s = 0; s < SX; ++s) { mbar_init(smem_u32(&ctl->raw_full[s]), 1); mbar_init(smem_u32(&ctl->x_full[s]), kCpProdWarps); mbar_init(smem_u32(&ctl->x_empty[s]), 1); }
        for (int s = 0; s < kCpAStages; ++s) { mbar_init(smem_u32(&ctl->a_full[s]), 128); mbar_init(smem_u32(&ctl->a_empty[s]), 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(smem_u32(&ctl->d_full[s]), 1); mbar_init(smem_u32(&ctl->d_empty[s]), 128); }
        ctl->abort_flag = 0;
        fence_barrier_init();
        fence_proxy_async();
    }
    if (threadIdx.x < 64) {
        if ((int)threadIdx.x < p.k) ctl->alpha[threadIdx.x] = p.per_tile ? __ldg(p.alpha + threadIdx.x) : __ldg(p.alpha);
        if ((int)threadIdx.x < p.kz) ctl->alpha_z[threadIdx.x] = p.per_tile_z ? __ldg(p.alpha_z + threadIdx.x) : __ldg(p.alpha_z);
    }
    if (warp == kCpMmaWarp) {
        tmem_alloc(smem_u32(&ctl->tmem_base), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;

    // a tile index enumerates (token tile, row block) with the row block fastest
    const int32_t n_tiles = p.w_tiles * p.t_tiles;
    bool ok = true;

    if (warp < kCpMmaWarp) {
        // ---------------- activation producers: z -> act_z(a_j z) -> swizzled shared-memory stage ----------------
        // The loader warp brings raw z into the stage by TMA (below); here thread tid owns the 16-byte piece c = tid mod 8
        // of token rows (tid div 8) + 32 i, i < 4, in both swizzle rows of every stage, reads it back, applies
        // act_z(a_j .) and stores it in place.  Piece c of row R sits at position c xor (R mod 8); R mod 8 is the same for
        // a thread's four rows, and a warp's access covers four whole 128-byte rows (no bank conflicts).  A swizzle row
        // that lies past the last input column is not loaded: it is written as zeros here.
        const int tid = threadIdx.x;
        const int c = tid & 7, rg = tid >> 3;
        const uint32_t own = (uint32_t)rg * 128u + ((uint32_t)(c ^ (rg & 7)) << 4);
        Pipe px;
        for (int32_t tile = bid; tile < n_tiles && ok; tile += gridDim.x) {
            for (int32_t ks = 0; ks < p.k_stages; ++ks) {
                // one lane per warp polls; then every lane observes the completed phase itself (one probe, no spinning)
                const uint32_t raw_bar = smem_u32(&ctl->raw_full[px.stage]);
                int landed = 1;
                if (lane == 0) landed = wait_one(raw_bar, px.phase, abort_flag, p.status, (7 << 24) | (px.stage << 16) | (bid & 0xffff));
                ok = __shfl_sync(0xffffffffu, landed, 0) != 0;
                if (!ok) break;
                (void)mbar_try_wait(raw_bar, px.phase);
                const uint32_t base = stage0 + px.stage * kStageBytes + own;
                // all reads first, then all arithmetic, then all writes: eight independent chains per thread
                uint4 v[kCpKA * 4];
                float al[kCpKA];
#pragma unroll
                for (int at = 0; at < kCpKA; ++at) {
                    const int32_t K0 = ks * kCpStageK + at * kCpAtomK;
                    const bool live = K0 < p.n;
                    al[at] = live ? ctl->alpha_z[min(K0 / p.rz, 63)] : 0.0f;
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        v[at * 4 + i] = live ? lds_v4(base + (uint32_t)at * kAtomBytes + (uint32_t)i * 32u * 128u)
                                             : make_uint4(0u, 0u, 0u, 0u);
                }
#pragma unroll
                for (int u = 0; u < kCpKA * 4; ++u) {
                    const float a = al[u >> 2];
                    v[u].x = cp_act_pair(v[u].x, a, p.act_z);
                    v[u].y = cp_act_pair(v[u].y, a, p.act_z);
                    v[u].z = cp_act_pair(v[u].z, a, p.act_z);
                    v[u].w = cp_act_pair(v[u].w, a, p.act_z);
                }
#pragma unroll
                for (int at = 0; at < kCpKA; ++at)
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        sts_v4(base + (uint32_t)at * kAtomBytes + (uint32_t)i * 32u * 128u, v[at * 4 + i].x, v[at * 4 + i].y,
                               v[at * 4 + i].z, v[at * 4 + i].w);
                fence_proxy_async();                           // generic-proxy writes -> visible to the tensor core
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctl->x_full[px.stage]));      // one arrival per warp
                px.advance(SX);
            }
        }
    } else if (warp == kCpLoadWarp) {
        // ---------------- loader: raw z -> shared-memory stage by TMA (rows past T arrive as zeros) ----------------
        Pipe px;
        uint32_t issued_mask = 0, issued_phase = 0;
        for (int32_t tile = bid; tile < n_tiles && ok; tile += gridDim.x) {
            const int32_t tok0 = (tile / p.w_tiles) * NTOK;
            for (int32_t ks = 0; ks < p.k_stages; ++ks) {
                ok = wait_bar(smem_u32(&ctl->x_empty[px.stage]), px.phase ^ 1u, abort_flag, p.status,
                              (1 << 24) | (px.stage << 16) | (bid & 0xffff));
                if (!ok) break;
                if (lane == 0) {
                    const uint32_t bar = smem_u32(&ctl->raw_full[px.stage]);
                    const int32_t K0 = ks * kCpStageK;
                    const int live = K0 + kCpAtomK < p.n ? 2 : 1;          // K0 < n always
                    mbar_arrive_expect_tx(bar, live * kAtomBytes);
                    for (int at = 0; at < live; ++at)
                        tma_load_2d(stage0 + px.stage * kStageBytes + at * kAtomBytes, &z_map,
                                    (K0 + at * kCpAtomK) % p.rz, tok0, bar);
                }
                issued_mask |= 1u << px.stage;
                issued_phase = (issued_phase & ~(1u << px.stage)) | (px.phase << px.stage);
                __syncwarp();
                px.advance(SX);
            }
        }
        if (!ok) {   // let copies in flight land before the block's shared memory goes away
            for (int s = 0; s < SX; ++s)
                if (issued_mask & (1u << s)) drain_wait(smem_u32(&ctl->raw_full[s]), (issued_phase >> s) & 1u);
        }
    } else if (warp == kCpMmaWarp) {
        // ---------------- MMA issuer: the whole warp runs the loop, one elected lane performs each MMA ----------------
        const uint32_t tmem_u = __shfl_sync(0xffffffffu, tmem_base, 0);
        const uint32_t leader = elect_one();
        Pipe px, pa, pd;
        bool ready = false;
        constexpr uint32_t kDescHi = (uint32_t)(kCpBDescHi >> 32);
        constexpr int kSteps = kCpKA * 4;
        for (int32_t tile = bid; tile < n_tiles && ok; tile += gridDim.x) {
            ok = wait_bar(smem_u32(&ctl->d_empty[pd.stage]), pd.phase ^ 1u, abort_flag, p.status, (2 << 24) | (bid & 0xffff));
            if (!ok) break;
            tc_fence_after();
            const uint32_t d_addr = tmem_u + pd.stage * kDCols;
            for (int32_t ks = 0; ks < p.k_stages; ++ks) {
                if (!ready) {
                    ok = wait_bar(smem_u32(&ctl->x_full[px.stage]), px.phase, abort_flag, p.status,
                                  (3 << 24) | (px.stage << 16) | (bid & 0xffff)) &&
                         wait_bar(smem_u32(&ctl->a_full[pa.stage]), pa.phase, abort_flag, p.status,
                                  (4 << 24) | (pa.stage << 16) | (bid & 0xffff));
                    if (!ok) break;
                }
                tc_fence_after();
                const uint32_t b_lo = (((stage0 + px.stage * kStageBytes) & 0x3FFFFu) >> 4) | (1u << 16);
                const uint32_t a_addr = tmem_u + kABase + pa.stage * kCpACols;
                Pipe nx = px, na = pa;
                nx.advance(SX);
                na.advance(kCpAStages);
                // a ragged last stage holds zeros past the row's end on the activation side: all K steps run
#pragma unroll
                for (int st = 0; st < kSteps; ++st) {
                    const int a2 = st >> 2, kk = st & 3;
                    tc_mma_ts_elect(d_addr, a_addr + a2 * 32 + kk * 8, b_lo + a2 * (kAtomBytes >> 4) + kk * 2, kDescHi, kIdesc,
                                    st > 0 ? 1u : (uint32_t)(ks > 0), leader);
                    if (st == kSteps / 2 - 1)
                        ready = __all_sync(0xffffffffu, mbar_test_wait(smem_u32(&ctl->x_full[nx.stage]), nx.phase) &&
                                                            mbar_test_wait(smem_u32(&ctl->a_full[na.stage]), na.phase)) != 0;
                }
                tc_commit_elect(smem_u32(&ctl->x_empty[px.stage]), leader);
                tc_commit_elect(smem_u32(&ctl->a_empty[pa.stage]), leader);
                if (ks == p.k_stages - 1) tc_commit_elect(smem_u32(&ctl->d_full[pd.stage]), leader);
                px = nx;
                pa = na;
            }
            pd.advance(DB);
        }
        __syncwarp();
    } else if (warp < kCpMmaWarp + 5) {
        // ---------------- weight decode: tile bits -> +-1 bf16 pairs -> tensor memory ----------------
        // Thread (quadrant qd, lane) owns TMEM lane L = weight row L of the block: 128 bits per stage.  Bits past the
        // row's end (ragged last stage) meet zero activations, so they need no masking.
        const int qd = warp & 3;
        const int L = qd * 32 + lane;
        const uint32_t lane_base = (uint32_t)(qd * 32) << 16;
        const int64_t last_word = p.n_words - 1;
        Pipe pa;
        for (int32_t tile = bid; tile < n_tiles && ok; tile += gridDim.x) {
            const int32_t wrow = min((tile % p.w_tiles) * 128 + L, p.r - 1);     // rows past the end are never stored
            const int64_t bitoff = (int64_t)wrow * p.n;
            const uint32_t sh = (uint32_t)bitoff & 31u;
            uint32_t w[5];
            {
                const int64_t wi = bitoff >> 5;
#pragma unroll
                for (int i = 0; i < 5; ++i) w[i] = __ldg(p.tile + min(wi + i, last_word));
            }
            for (int32_t ks = 0; ks < p.k_stages && ok; ++ks) {
                uint32_t b[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) b[i] = __funnelshift_r(w[i], w[i + 1], sh);
                w[0] = w[4];
                if (ks + 1 < p.k_stages) {
                    const int64_t wi = (bitoff + (int64_t)(ks + 1) * kCpStageK) >> 5;
#pragma unroll
                    for (int i = 1; i < 5; ++i) w[i] = __ldg(p.tile + min(wi + i, last_word));
                }
                uint32_t v[kCpKA][32];
#pragma unroll
                for (int a2 = 0; a2 < kCpKA; ++a2) {
                    cp_decode16(b[2 * a2] & 0xffffu, v[a2]);
                    cp_decode16(b[2 * a2] >> 16, v[a2] + 8);
                    cp_decode16(b[2 * a2 + 1] & 0xffffu, v[a2] + 16);
                    cp_decode16(b[2 * a2 + 1] >> 16, v[a2] + 24);
                }
                ok = wait_bar(smem_u32(&ctl->a_empty[pa.stage]), pa.phase ^ 1u, abort_flag, p.status,
                              (5 << 24) | (pa.stage << 16) | (bid & 0xffff));
                if (!ok) break;
                tc_fence_after();
#pragma unroll
                for (int a2 = 0; a2 < kCpKA; ++a2)
                    tmem_st_32x32(tmem_base + lane_base + kABase + pa.stage * kCpACols + a2 * 32, v[a2]);
                tc_wait_st();
                tc_fence_before();
                mbar_arrive(smem_u32(&ctl->a_full[pa.stage]));
                pa.advance(kCpAStages);
            }
        }
    } else if (warp < kCpLoadWarp) {
        // ---------------- epilogue: TMEM -> exchange -> alpha / bias / activation -> k replicated stores ----------------
        // As in the bf16 kernel: the four warps exchange each 128-row x 32-token block through shared memory [token][row]
        // so that a lane holds 8 consecutive features of a token and a warp store covers 2 tokens x 256 contiguous bytes.
        const int qd = warp & 3;
        const int ew = warp - (kCpMmaWarp + 5);
        const uint32_t lane_base = (uint32_t)(qd * 32) << 16;
        float (*xbuf)[kCpXPitch] = reinterpret_cast<float (*)[kCpXPitch]>(ctl->exchange);
        Pipe pd;
        const bool vec_ok = (p.m % 8 == 0) && (p.r % 8 == 0);
        const int f0 = 8 * (lane & 15);
        const int tsub = lane >> 4;
        const bool plain = p.bias == nullptr && (p.act == TBN_ACT_NONE || p.act == TBN_ACT_RELU);
        for (int32_t tile = bid; tile < n_tiles; tile += gridDim.x) {
            const int64_t tok0 = (int64_t)(tile / p.w_tiles) * NTOK;
            ok = wait_bar(smem_u32(&ctl->d_full[pd.stage]), pd.phase, abort_flag, p.status, (6 << 24) | (bid & 0xffff));
            if (cp_epi_bar_count(ok) != 128) { ok = false; break; }        // the four warps go on together or not at all
            tc_fence_after();
            const int n_chunks = (int)min((int64_t)(NTOK / 32), (p.T - tok0 + 31) / 32);
            const int32_t blk0 = (tile % p.w_tiles) * 128;
            const int rows_valid = max(0, min(128, p.r - blk0));
#pragma unroll 1
            for (int ch = 0; ch < n_chunks; ++ch) {
                __syncwarp();
                uint32_t v[32];
                tmem_ld_32x32(tmem_base + lane_base + pd.stage * kDCols + ch * 32, v);
                tc_wait_ld();
                if (ch == n_chunks - 1) {                   // accumulator fully read: hand it back early
                    tc_fence_before();
                    mbar_arrive(smem_u32(&ctl->d_empty[pd.stage]));
                }
                cp_epi_bar();                               // the previous block has been read by everyone
#pragma unroll
                for (int i = 0; i < 32; ++i) xbuf[i][qd * 32 + lane] = __uint_as_float(v[i]);
                cp_epi_bar();
                const int nvalid = rows_valid - f0;
                if (nvalid <= 0) continue;
                float z[4][8];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float4 lo = *reinterpret_cast<const float4 *>(&xbuf[8 * ew + tsub + 2 * i][f0]);
                    const float4 hi = *reinterpret_cast<const float4 *>(&xbuf[8 * ew + tsub + 2 * i][f0 + 4]);
                    z[i][0] = lo.x; z[i][1] = lo.y; z[i][2] = lo.z; z[i][3] = lo.w;
                    z[i][4] = hi.x; z[i][5] = hi.y; z[i][6] = hi.z; z[i][7] = hi.w;
                }
                if (p.act == TBN_ACT_RELU && p.bias == nullptr) {
                    // alpha >= 0, so relu(alpha * z) = alpha * relu(z): clamp once, outside the k loop
#pragma unroll
                    for (int i = 0; i < 4; ++i)
#pragma unroll
                        for (int e = 0; e < 8; ++e) z[i][e] = fmaxf(z[i][e], 0.0f);
                }
                const int64_t tok_first = tok0 + ch * 32 + 8 * ew + tsub;
                if (plain && p.y_bf16 && vec_ok && nvalid >= 8) {
                    __nv_bfloat16 *yb[4];
                    bool tv[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int64_t tok = tok_first + 2 * i;
                        tv[i] = tok < p.T;
                        yb[i] = static_cast<__nv_bfloat16 *>(p.y) + tok * p.m + blk0 + f0;
                    }
                    const int32_t kk = p.k, rr = p.r;
                    for (int32_t j = 0; j < kk; ++j) {
                        const float al = j < 64 ? ctl->alpha[j] : (p.per_tile ? __ldg(p.alpha + j) : __ldg(p.alpha));
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            uint32_t pk[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const __nv_bfloat162 h2 = __floats2bfloat162_rn(al * z[i][2 * e], al * z[i][2 * e + 1]);
                                pk[e] = *reinterpret_cast<const uint32_t *>(&h2);
                            }
                            if (tv[i]) *reinterpret_cast<uint4 *>(yb[i]) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                            yb[i] += rr;
                        }
                    }
                    continue;
                }
                for (int32_t j = 0; j < p.k; ++j) {
                    const float al = j < 64 ? ctl->alpha[j] : (p.per_tile ? __ldg(p.alpha + j) : __ldg(p.alpha));
                    const int64_t o0 = (int64_t)j * p.r + blk0 + f0;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int64_t tok = tok_first + 2 * i;
                        if (tok >= p.T) continue;
                        float o[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            const float bb = (p.bias != nullptr && e < nvalid) ? __ldg(p.bias + o0 + e) : 0.0f;
                            const float val = fmaf(al, z[i][e], bb);
                            o[e] = plain ? val : (p.act == TBN_ACT_GELU && p.y_bf16) ? gelu_tanh_bf16(val) : apply_act(val, p.act);
                        }
                        const int64_t yi = tok * p.m + o0;
                        if (vec_ok && nvalid >= 8) {
                            if (p.y_bf16) {
                                uint32_t pk[4];
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    const __nv_bfloat162 h2 = __floats2bfloat162_rn(o[2 * e], o[2 * e + 1]);
                                    pk[e] = *reinterpret_cast<const uint32_t *>(&h2);
                                }
                                *reinterpret_cast<uint4 *>(static_cast<__nv_bfloat16 *>(p.y) + yi) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                            } else {
                                float4 *dst = reinterpret_cast<float4 *>(static_cast<float *>(p.y) + yi);
                                dst[0] = make_float4(o[0], o[1], o[2], o[3]);
                                dst[1] = make_float4(o[4], o[5], o[6], o[7]);
                            }
                        } else {
                            for (int e = 0; e < 8 && e < nvalid; ++e) {
                                if (p.y_bf16) static_cast<__nv_bfloat16 *>(p.y)[yi + e] = __float2bfloat16_rn(o[e]);
                                else static_cast<float *>(p.y)[yi + e] = o[e];
                            }
                        }
                    }
                }
            }
            pd.advance(DB);
        }
    }

    // ---------------- teardown ----------------
    if (warp == kCpMmaWarp && *abort_flag) {
        // make sure no MMA is still reading shared or tensor memory before they are released
        tc_commit_elect(smem_u32(&ctl->x_empty[0]), elect_one());
        __syncwarp();
        drain_wait(smem_u32(&ctl->x_empty[0]), 0);
        drain_wait(smem_u32(&ctl->x_empty[0]), 1);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == kCpMmaWarp) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

int cp_sm_count()
{
    static int cache[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    if (!cache[dev]) cudaDeviceGetAttribute(&cache[dev], cudaDevAttrMultiProcessorCount, dev);
    return cache[dev];
}

}  // namespace

bool compact_linear_supported(const CompactArgs &a)
{
    if (a.rz <= 0 || a.kz <= 0 || a.kz > 64 || a.rz % 64 != 0) return false;     // a swizzle row lies inside one repetition
    const int64_t n = (int64_t)a.rz * a.kz;
    if (n > 0x7fffffffLL || a.q % n != 0) return false;                        // the tile must span whole rows
    if (a.T >= ((int64_t)1 << 31) - 256) return false;
    return true;
}

int launch_compact_linear(const CompactArgs &a, int *device_status, cudaStream_t s)
{
    if (!compact_linear_supported(a)) return TBN_ERR_UNSUPPORTED;
    constexpr int NTOK = 128, SX = 6;
    CpParams p;
    p.z = static_cast<const __nv_bfloat16 *>(a.z); p.alpha_z = a.alpha_z; p.tile = a.tile; p.alpha = a.alpha; p.bias = a.bias;
    p.y = a.y; p.status = device_status;
    p.T = a.T; p.n_words = tbn_tile_words(a.q);
    p.rz = a.rz; p.kz = a.kz; p.n = a.rz * a.kz; p.m = a.m; p.r = (int32_t)(a.q / p.n); p.k = a.k;
    p.k_stages = (p.n + kCpStageK - 1) / kCpStageK;
    p.w_tiles = (p.r + 127) / 128;
    p.t_tiles = (int32_t)((a.T + NTOK - 1) / NTOK);
    p.per_tile_z = a.alpha_mode_z == TBN_ALPHA_PER_TILE; p.act_z = a.act_z;
    p.per_tile = a.alpha_mode == TBN_ALPHA_PER_TILE; p.act = a.act; p.y_bf16 = a.y_dtype == TBN_BF16;
    EncodeTiledFn encode = encode_tiled_fn();
    if (!encode) return TBN_ERR_CUDA;
    CUtensorMap map;                                       // z: T rows of r_z bf16; a box is one swizzle row of a stage
    const cuuint64_t dims[2] = {(cuuint64_t)a.rz, (cuuint64_t)a.T};
    const cuuint64_t strides[1] = {(cuuint64_t)a.rz * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kCpAtomK, (cuuint32_t)NTOK};
    const cuuint32_t estr[2] = {1, 1};
    if (encode(&map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(a.z), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return TBN_ERR_CUDA;
    const size_t smem = (size_t)SX * kCpKA * NTOK * 128 + sizeof(CpControl<SX>) + 1024;
    auto kern = tc_linear_compact_kernel<NTOK, SX>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return TBN_ERR_CUDA;
    const int sms = cp_sm_count();
    if (sms <= 0) return TBN_ERR_CUDA;
    const int64_t tiles = (int64_t)p.w_tiles * p.t_tiles;
    const unsigned grid = (unsigned)(tiles < sms ? tiles : sms);
    kern<<<grid, kCpThreads, smem, s>>>(map, p);
    return cudaGetLastError() == cudaSuccess ? TBN_OK : TBN_ERR_CUDA;
}

}  // namespace tbn
