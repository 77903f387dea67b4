// Tensor-core forward of a tiled fully-connected layer on sm_100a: tcgen05.mma with the decoded
// weights as the A operand in tensor memory and the activations as the B operand in shared memory.
//
// Problem.  The tile spans r = q/n whole rows, so only Z[T, r] = X[T, n] * Wd[r, n]^T has to be
// contracted (Wd = the r distinct +-1 rows, Sec. 4.1); the output is Y[:, j*r + c] = act(alpha_j *
// Z[:, c] + bias) for the k repetitions j.  The kernel computes Z^T tiles: the UMMA M dimension (the
// 128 TMEM lanes) runs over weight rows, the N dimension over tokens.
//
// Why the weights go to tensor memory.  The packed tile is 1/16 of the bf16 weight bytes and is
// expanded in registers; writing the expansion with tcgen05.st into TMEM costs no shared-memory
// bandwidth, and tcgen05.mma then reads A from TMEM and only the activation operand from shared
// memory.  Each decoded 128 x 64 block is reused for all NTOK tokens of the CTA tile, and each
// activation stage is reused by NA blocks of 128 weight rows.
//
// Warp roles (10 warps, 14 with EPI == 8): 0 = TMA producer (activation stages, 128-byte swizzle), 1 = MMA issuer and
// TMEM owner, 2-5 = tile decode (bits -> +-1 bf16 pairs -> tcgen05.st), 6-9 = epilogue (tcgen05.ld ->
// alpha/bias/activation -> k-fold replicated stores), 10-13 = optional epilogue helpers (half of the
// arithmetic and stores when the activation is expensive; they never touch tensor memory).  All hand-offs are mbarriers; every wait is
// bounded by a wall-clock limit, after which the CTA records TBN_ERR_TIMEOUT, drains and returns.
#include <atomic>
#include <cstddef>

#include "tc_common.cuh"

namespace tbn {

namespace {

using namespace tc;

constexpr int kBaseThreads = 192;      // TMA, MMA and the four decode warps; the epilogue warps follow
constexpr int kAtomK = 64;             // contraction elements per 128-byte swizzle row (one TMA box, 4 MMA K steps)
constexpr int kMaxAStages = 4;         // decoded-weight stages in tensor memory: 2, or 4 where the columns allow
constexpr int kMaxAlpha = 64;          // alphas cached in shared memory

// 16 tile bits (low half of h, upper half zero) -> 8 registers of two bf16 each: bit 2j in the low half,
// bit 2j+1 in the high half; bit 1 -> +1.0 (0x3F80), bit 0 -> -1.0 (0xBF80).  v keeps the even bits at
// positions 2j and moves the odd bits to 2j+16, so one shift lines both up with the two sign positions.
__device__ __forceinline__ void decode16(uint32_t h, uint32_t *out) {
    const uint32_t v = (h | (h << 15)) & 0x55555555u;
#pragma unroll
    for (int j = 0; j < 8; ++j) out[j] = ((v << (15 - 2 * j)) & 0x80008000u) ^ 0xBF80BF80u;
}
// 64 consecutive tile bits (b0 = first 32) -> one 128-lane x 32-column row of the A operand
__device__ __forceinline__ void decode64(uint32_t b0, uint32_t b1, uint32_t (&v)[32]) {
    decode16(b0 & 0xffffu, v);
    decode16(b0 >> 16, v + 8);
    decode16(b1 & 0xffffu, v + 16);
    decode16(b1 >> 16, v + 24);
}

constexpr int kXPitch = 132;             // floats per token row of the epilogue exchange buffer (128 + 4: 16-byte rows)

// Named barrier 1 belongs to the epilogue warps (THREADS of them in all).
template <int THREADS>
__device__ __forceinline__ void epi_bar() { asm volatile("bar.sync 1, %0;" ::"n"(THREADS) : "memory"); }
// Same barrier, returning how many of its threads passed `pred`.
template <int THREADS>
__device__ __forceinline__ int epi_bar_count(bool pred) {
    int n;
    asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %1, 0;\nbar.red.popc.u32 %0, 1, %2, p;\n}"
                 : "=r"(n) : "r"((int)pred), "n"(THREADS) : "memory");
    return n;
}

// ---- shared-memory control block -----------------------------------------------------------------
template <int SX>
struct Control {
    uint64_t x_full[SX], x_empty[SX];
    uint64_t a_full[kMaxAStages], a_empty[kMaxAStages];
    uint64_t d_full[2], d_empty[2];
    uint32_t tmem_base;
    int abort_flag;
    float alpha[kMaxAlpha];
    unsigned int ticket;                 // split-K: this CTA's arrival number, broadcast to the epilogue warps
    alignas(16) float exchange[32 * kXPitch];   // epilogue (read with 16-byte loads): one 32-token x 128-row block, [token][row], padded rows
};

static_assert(offsetof(Control<3>, exchange) % 16 == 0 && offsetof(Control<8>, exchange) % 16 == 0, "16-byte loads");

struct TcParams {
    const uint32_t *tile;
    const __nv_bfloat16 *dense_a;   // non-null: full-precision weight rows [r][n] instead of tile bits
    const float *alpha;
    const float *bias;
    void *y;
    int *status;
    int64_t T;
    int64_t n_words;     // words of the packed tile
    int32_t n, m, r, k;
    int32_t k_stages;    // ceil(n / 64)
    int32_t w_tiles, t_tiles;
    int32_t splits;      // split-K factor: CTAs that share one output tile, each walking 1/splits of the contraction
    float *partial;      // splits > 1: fp32 partial tiles [out tile][split][NA][128 rows][NTOK tokens]
    unsigned int *tickets;   // splits > 1: arrival counters [out tile][4 lane quadrants], zeroed before the launch
    int per_tile, act, y_bf16;
};

// Shared-memory matrix descriptor of the activation operand: K-major, 128-byte swizzle, rows of 128 bytes,
// 8-row groups 1024 bytes apart (stride offset 64 x 16 bytes), descriptor version 1, leading offset 1.
// The low word carries the start address in 16-byte units; advancing it by 2 selects the next 16-element
// K slice inside the swizzled row.
constexpr uint64_t kBDescHi = (64ull << 32) | (1ull << 46) | (2ull << 61);

// NTOK tokens x (NA x 128) weight rows per CTA tile; KA 64-element K atoms per pipeline stage; SX activation
// stages in shared memory; DB accumulator buffers (2 = the epilogue of one tile overlaps the main loop of the
// next).  Tensor memory: DB x NA accumulators of NTOK columns, then 2 or 4 decoded-weight stages of
// NA x KA x 32 columns.
template <int NTOK, int NA, int KA, int SX, int DB, int EPI>
__global__ void __launch_bounds__(kBaseThreads + 32 * EPI, 1)
tc_linear_kernel(const __grid_constant__ CUtensorMap x_map, const TcParams p)
{
    static_assert(NTOK % 32 == 0 && NTOK >= 32 && NTOK <= 256, "token tile");
    static_assert(EPI == 4 || EPI == 8, "epilogue warps: the four tensor-memory readers, optionally four helpers");
    constexpr int kEpiThreads = 32 * EPI;
    constexpr int kSlots = EPI == 8 ? 2 : 4;             // token slots (of a lane's four per block) handled by one warp set
    constexpr uint32_t kAtomBytes = NTOK * 128;
    constexpr uint32_t kStageBytes = KA * kAtomBytes;
    constexpr int kStageK = KA * kAtomK;
    constexpr uint32_t kDCols = NA * NTOK;
    constexpr uint32_t kACols = NA * KA * 32;
    constexpr uint32_t kABase = DB * kDCols;             // first column of the decoded-weight stages
    // four decoded-weight stages when they fit the 512 columns next to the accumulators (the decode warps then run
    // two stages further ahead of the MMAs and their hand-off latency no longer shows), else two
    constexpr int kAStages = (kABase + 4 * kACols <= 512) ? 4 : 2;
    constexpr uint32_t kTmemCols = next_pow2_cols(kABase + kAStages * kACols);
    static_assert(kTmemCols <= 512, "tensor memory budget");
    // instruction descriptor: D fp32, A and B bf16, both K-major, N = NTOK, M = 128
    constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(NTOK >> 3) << 17) | (8u << 24);

    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    uint8_t *smem = smem_raw + ((1024u - (raw & 1023u)) & 1023u);
    Control<SX> *ctl = reinterpret_cast<Control<SX> *>(smem + SX * kStageBytes);
    const uint32_t stage0 = smem_u32(smem);
    volatile int *abort_flag = &ctl->abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int bid = blockIdx.x;

    if (threadIdx.x == 0) {
        for (int s = 0; s < SX; ++s) { mbar_init(smem_u32(&ctl->x_full[s]), 1); mbar_init(smem_u32(&ctl->x_empty[s]), 1); }
        for (int s = 0; s < kAStages; ++s) { mbar_init(smem_u32(&ctl->a_full[s]), 128); mbar_init(smem_u32(&ctl->a_empty[s]), 1); }
        for (int s = 0; s < 2; ++s) { mbar_init(smem_u32(&ctl->d_full[s]), 1); mbar_init(smem_u32(&ctl->d_empty[s]), 128); }
        ctl->abort_flag = 0;
        fence_barrier_init();
        fence_proxy_async();
    }
    if (threadIdx.x < kMaxAlpha && (int)threadIdx.x < p.k)
        ctl->alpha[threadIdx.x] = p.per_tile ? __ldg(p.alpha + threadIdx.x) : __ldg(p.alpha);
    if (warp == 1) {
        tmem_alloc(smem_u32(&ctl->tmem_base), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;

    // A tile index enumerates (token tile, row block, K split) with the split fastest, so the CTAs that share an
    // output tile run at the same time.  Split s walks stages [s*k_stages/S, (s+1)*k_stages/S).
    const int32_t n_tiles = p.w_tiles * p.t_tiles * p.splits;
    bool ok = true;

    if (warp == 0) {
        // ---------------- TMA producer: activation stages ----------------
        Pipe px;
        uint32_t issued_mask = 0, issued_phase = 0;
        for (int32_t tile = bid; tile < n_tiles && ok; tile += gridDim.x) {
            const int32_t split = tile % p.splits, out_tile = tile / p.splits;
            const int32_t tok0 = (out_tile / p.w_tiles) * NTOK;
            const int32_t ks0 = (int32_t)((int64_t)split * p.k_stages / p.splits);
            const int32_t ks1 = (int32_t)((int64_t)(split + 1) * p.k_stages / p.splits);
            for (int32_t ks = ks0; ks < ks1 && ok; ++ks) {
                ok = wait_bar(smem_u32(&ctl->x_empty[px.stage]), px.phase ^ 1u, abort_flag, p.status,
                              (1 << 24) | (px.stage << 16) | (bid & 0xffff));
                if (!ok) break;
                if (lane == 0) {
                    const uint32_t bar = smem_u32(&ctl->x_full[px.stage]);
                    mbar_arrive_expect_tx(bar, kStageBytes);
#pragma unroll
                    for (int at = 0; at < KA; ++at)   // a box that lies past the last column is zero-filled
                        tma_load_2d(stage0 + px.stage * kStageBytes + at * kAtomBytes, &x_map,
                                    ks * kStageK + at * kAtomK, tok0, bar);
                }
                issued_mask |= 1u << px.stage;
                issued_phase = (issued_phase & ~(1u << px.stage)) | (px.phase << px.stage);
                __syncwarp();
                px.advance(SX);
            }
        }
        if (!ok) {   // let copies in flight land before the CTA's shared memory goes away
            for (int s = 0; s < SX; ++s)
                if (issued_mask & (1u << s)) drain_wait(smem_u32(&ctl->x_full[s]), (issued_phase >> s) & 1u);
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        // tcgen05.mma is issued by one thread, and that thread's instructions execute back to back with no
        // other warp to hide their latency: every instruction between two MMAs is dead time for the tensor
        // cores once their small queue has drained.  So the K steps of a full stage are unrolled with all
        // offsets immediate (two adds per MMA) and the NEXT stage's barriers are polled in the middle of the
        // current stage (if they are already complete, the common case, the next stage starts at once).
        {
            // all 32 lanes run the loop in lockstep; one elected lane performs each MMA and commit (see tc_mma_ts_elect)
            const uint32_t tmem_u = __shfl_sync(0xffffffffu, tmem_base, 0);
            const uint32_t leader = elect_one();
            Pipe px, pa, pd;
            bool ready = false;
            constexpr uint32_t kDescHi = (uint32_t)(kBDescHi >> 32);
            constexpr int kSteps = KA * 4;             // 16-element K steps per full stage
            for (int32_t tile = bid; tile < n_tiles && ok; tile += gridDim.x) {
                ok = wait_bar(smem_u32(&ctl->d_empty[pd.stage]), pd.phase ^ 1u, abort_flag, p.status,
                              (2 << 24) | (bid & 0xffff));
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_addr = tmem_u + pd.stage * kDCols;
                const int32_t split = tile % p.splits;
                const int32_t ks0 = (int32_t)((int64_t)split * p.k_stages / p.splits);
                const int32_t ks1 = (int32_t)((int64_t)(split + 1) * p.k_stages / p.splits);
                for (int32_t ks = ks0; ks < ks1; ++ks) {
                    if (!ready) {
                        ok = wait_bar(smem_u32(&ctl->x_full[px.stage]), px.phase, abort_flag, p.status,
                                      (3 << 24) | (px.stage << 16) | (bid & 0xffff)) &&
                             wait_bar(smem_u32(&ctl->a_full[pa.stage]), pa.phase, abort_flag, p.status,
                                      (4 << 24) | (pa.stage << 16) | (bid & 0xffff));
                        if (!ok) break;
                    }
                    tc_fence_after();
                    // descriptor low word: start address in 16-byte units | leading offset 1 << 16
                    const uint32_t b_lo = (((stage0 + px.stage * kStageBytes) & 0x3FFFFu) >> 4) | (1u << 16);
                    const uint32_t a_addr = tmem_u + kABase + pa.stage * kACols;
                    Pipe nx = px, na = pa;
                    nx.advance(SX);
                    na.advance(kAStages);
                    const int32_t rem = p.n - ks * kStageK;
                    if (rem >= kStageK) {
#pragma unroll
                        for (int st = 0; st < kSteps; ++st) {
                            const int at = st >> 2, kk = st & 3;
#pragma unroll
                            for (int a = 0; a < NA; ++a)
                                tc_mma_ts_elect(d_addr + a * NTOK, a_addr + (a * KA + at) * 32 + kk * 8,
                                          b_lo + at * (kAtomBytes >> 4) + kk * 2, kDescHi, kIdesc,
                                          st > 0 ? 1u : (uint32_t)(ks > ks0), leader);
                            if (st == kSteps / 2 - 1)
                                ready = __all_sync(0xffffffffu, mbar_test_wait(smem_u32(&ctl->x_full[nx.stage]), nx.phase) &&
                                                                    mbar_test_wait(smem_u32(&ctl->a_full[na.stage]), na.phase)) != 0;
                        }
                    } else {                              // ragged last stage: only the K steps that hold data
                        const int steps = (rem + 15) >> 4;
                        for (int st = 0; st < steps; ++st) {
                            const int at = st >> 2, kk = st & 3;
#pragma unroll
                            for (int a = 0; a < NA; ++a)
                                tc_mma_ts_elect(d_addr + a * NTOK, a_addr + (a * KA + at) * 32 + kk * 8,
                                          b_lo + at * (kAtomBytes >> 4) + kk * 2, kDescHi, kIdesc,
                                          (ks > ks0 || st > 0) ? 1u : 0u, leader);
                        }
                        ready = false;
                    }
                    tc_commit_elect(smem_u32(&ctl->x_empty[px.stage]), leader);
                    tc_commit_elect(smem_u32(&ctl->a_empty[pa.stage]), leader);
                    if (ks == ks1 - 1) tc_commit_elect(smem_u32(&ctl->d_full[pd.stage]), leader);
                    px = nx;
                    pa = na;
                }
                pd.advance(DB);
            }
        }
        __syncwarp();
    } else if (warp < 6) {
        // ---------------- tile decode: bits -> +-1 bf16 pairs -> tensor memory ----------------
        // Thread (quadrant qd, lane) owns TMEM lane L = 32*qd + lane, i.e. weight row L of each of the NA
        // blocks.  Per stage it needs 64*KA consecutive bits of each row; the words for the next stage are
        // requested before this stage is decoded, so their latency overlaps the ALU work.
        constexpr int kW = 2 * KA;                 // 32-bit words of tile bits per row and stage
        const int qd = warp & 3;
        const int L = qd * 32 + lane;
        const uint32_t lane_base = (uint32_t)(qd * 32) << 16;
        const int64_t last_word = p.n_words - 1;
        Pipe pa;
        if (p.dense_a != nullptr) {
            // Full-precision rows instead of tile bits (weights folded with the previous layer's alphas, see
            // the MLP chain): row L of each block is n bf16 values, 64*KA of them per stage, copied as they are.
            const uint4 *rows = reinterpret_cast<const uint4 *>(p.dense_a);
            const int32_t row_vecs = p.n >> 3;                       // 16-byte vectors per row (n % 8 == 0)
            for (int32_t tile = bid; tile < n_tiles && ok; tile += gridDim.x) {
                const int32_t split = tile % p.splits, out_tile = tile / p.splits;
                const int32_t ks0 = (int32_t)((int64_t)split * p.k_stages / p.splits);
                const int32_t ks1 = (int32_t)((int64_t)(split + 1) * p.k_stages / p.splits);
                const int32_t row_base = (out_tile % p.w_tiles) * (NA * 128) + L;
                for (int32_t ks = ks0; ks < ks1 && ok; ++ks) {
                    uint32_t v[NA][KA][32];
#pragma unroll
                    for (int a = 0; a < NA; ++a) {
                        const int32_t row = min(row_base + a * 128, p.r - 1);
                        const uint4 *src = rows + (int64_t)row * row_vecs;
                        const int32_t v0 = ks * (kStageK >> 3);
#pragma unroll
                        for (int at = 0; at < KA; ++at)
#pragma unroll
                            for (int i = 0; i < 8; ++i) {
                                const int32_t vi = v0 + at * 8 + i;
                                const uint4 q4 = vi < row_vecs ? __ldg(src + vi) : make_uint4(0u, 0u, 0u, 0u);
                                v[a][at][4 * i] = q4.x; v[a][at][4 * i + 1] = q4.y; v[a][at][4 * i + 2] = q4.z; v[a][at][4 * i + 3] = q4.w;
                            }
                    }
                    ok = wait_bar(smem_u32(&ctl->a_empty[pa.stage]), pa.phase ^ 1u, abort_flag, p.status,
                                  (5 << 24) | (pa.stage << 16) | (bid & 0xffff));
                    if (!ok) break;
                    tc_fence_after();
#pragma unroll
                    for (int a = 0; a < NA; ++a)
#pragma unroll
                        for (int at = 0; at < KA; ++at)
                            tmem_st_32x32(tmem_base + lane_base + kABase + pa.stage * kACols + (a * KA + at) * 32, v[a][at]);
                    tc_wait_st();
                    tc_fence_before();
                    mbar_arrive(smem_u32(&ctl->a_full[pa.stage]));
                    pa.advance(kAStages);
                }
            }
        } else
        for (int32_t tile = bid; tile < n_tiles && ok; tile += gridDim.x) {
            const int32_t split = tile % p.splits, out_tile = tile / p.splits;
            const int32_t ks0 = (int32_t)((int64_t)split * p.k_stages / p.splits);
            const int32_t ks1 = (int32_t)((int64_t)(split + 1) * p.k_stages / p.splits);
            const int32_t row_base = (out_tile % p.w_tiles) * (NA * 128) + L;
            int64_t bitoff[NA];
            uint32_t w[NA][kW + 1];
#pragma unroll
            for (int a = 0; a < NA; ++a) {
                const int32_t row = min(row_base + a * 128, p.r - 1);   // rows past the end are never stored
                bitoff[a] = (int64_t)row * p.n;
                const int64_t wi = (bitoff[a] + (int64_t)ks0 * kStageK) >> 5;
#pragma unroll
                for (int i = 0; i <= kW; ++i) w[a][i] = __ldg(p.tile + min(wi + i, last_word));
            }
            for (int32_t ks = ks0; ks < ks1 && ok; ++ks) {
                uint32_t b[NA][kW];
#pragma unroll
                for (int a = 0; a < NA; ++a) {
                    const uint32_t sh = (uint32_t)bitoff[a] & 31u;      // constant along the row: stages are 64*KA bits
#pragma unroll
                    for (int i = 0; i < kW; ++i) b[a][i] = __funnelshift_r(w[a][i], w[a][i + 1], sh);
                    w[a][0] = w[a][kW];
                    if (ks + 1 < ks1) {
                        const int64_t wi = (bitoff[a] + (int64_t)(ks + 1) * kStageK) >> 5;
#pragma unroll
                        for (int i = 1; i <= kW; ++i) w[a][i] = __ldg(p.tile + min(wi + i, last_word));
                    }
                }
                // decode into registers BEFORE waiting for the tensor-memory stage: the ALU work then overlaps the
                // MMAs that still read that stage, and only the stores sit between "stage free" and "stage full"
                uint32_t v[NA][KA][32];
#pragma unroll
                for (int a = 0; a < NA; ++a)
#pragma unroll
                    for (int at = 0; at < KA; ++at) decode64(b[a][2 * at], b[a][2 * at + 1], v[a][at]);
                ok = wait_bar(smem_u32(&ctl->a_empty[pa.stage]), pa.phase ^ 1u, abort_flag, p.status,
                              (5 << 24) | (pa.stage << 16) | (bid & 0xffff));
                if (!ok) break;
                tc_fence_after();
#pragma unroll
                for (int a = 0; a < NA; ++a)
#pragma unroll
                    for (int at = 0; at < KA; ++at)
                        tmem_st_32x32(tmem_base + lane_base + kABase + pa.stage * kACols + (a * KA + at) * 32, v[a][at]);
                tc_wait_st();
                tc_fence_before();
                mbar_arrive(smem_u32(&ctl->a_full[pa.stage]));
                pa.advance(kAStages);
            }
        }
    } else {
        // ---------------- epilogue: TMEM -> exchange -> alpha / bias / activation -> k replicated stores ------
        // tcgen05.ld hands thread (quadrant qd, lane) one weight row and 32 consecutive tokens, but the output is
        // row-major [token][feature]: a store instruction whose lanes are 32 different tokens touches 32 separate
        // lines and the load/store unit, not HBM, then bounds the epilogue.  So the four warps exchange each
        // 128-row x 32-token block through one shared buffer [token][row] and come back with lane = 8 consecutive
        // features of a token: a warp store covers 2 tokens x 256 contiguous bytes (bf16).  Every repetition j is
        // then one multiply per element (fp32), a pack to bf16 and one 16-byte store per token.
        // Warps 6-9 read tensor memory (and do the split-K traffic).  With EPI == 8, warps 10-13 help with the
        // arithmetic and the stores: of a lane's four tokens per block, the readers take the first two and the
        // helpers the last two (worth it when the activation is expensive; a plain epilogue is bound by the stores).
        const bool reader = warp < 10;
        const int qd = warp & 3;                          // tensor-memory lane quadrant a reader warp may read
        const int ew = (warp - 6) & 3;                    // this warp stores tokens 8*ew .. 8*ew+7 of each 32-token block
        const int iset = (warp - 6) >> 2;                 // token slots kSlots*iset .. of the lane's four
        const uint32_t lane_base = (uint32_t)(qd * 32) << 16;
        float (*xbuf)[kXPitch] = reinterpret_cast<float (*)[kXPitch]>(ctl->exchange);
        Pipe pd;                                          // accumulator buffer (stage) and its phase
        const bool vec_ok = (p.m % 8 == 0) && (p.r % 8 == 0);       // 16-byte aligned groups of 8 features
        const bool bias_vec = (reinterpret_cast<uintptr_t>(p.bias) & 15) == 0;
        const int f0 = 8 * (lane & 15);                   // first of this lane's 8 rows inside the 128-row block
        const int tsub = lane >> 4;                       // this lane's tokens: 8*ew + tsub + 2*i, i = 2*iset, 2*iset+1
        const bool plain = p.bias == nullptr && (p.act == TBN_ACT_NONE || p.act == TBN_ACT_RELU);
        for (int32_t tile = bid; tile < n_tiles; tile += gridDim.x) {
            const int32_t split = tile % p.splits, out_tile = tile / p.splits;
            const int64_t tok0 = (int64_t)(out_tile / p.w_tiles) * NTOK;
            ok = reader ? wait_bar(smem_u32(&ctl->d_full[pd.stage]), pd.phase, abort_flag, p.status, (6 << 24) | (bid & 0xffff))
                        : (*abort_flag == 0);
            // the eight warps go on together or not at all (they share named barrier 1 below)
            if (epi_bar_count<kEpiThreads>(ok) != kEpiThreads) { ok = false; break; }
            tc_fence_after();
            const int n_chunks = (int)min((int64_t)(NTOK / 32), (p.T - tok0 + 31) / 32);
            // fp32 partial tile of (out_tile, split): [NA][128 rows][NTOK tokens]; this thread owns one row per block
            float *part_row = nullptr;
            if (p.splits > 1) {
                constexpr int64_t kTileFloats = (int64_t)NA * 128 * NTOK;
                part_row = p.partial + ((int64_t)out_tile * p.splits + split) * kTileFloats + (int64_t)(qd * 32 + lane) * NTOK;
                // pass 1: dump this CTA's partial sums (128 contiguous bytes per thread and chunk)
#pragma unroll 1
                for (int a = 0; a < (reader ? NA : 0); ++a) {
#pragma unroll 1
                    for (int ch = 0; ch < n_chunks; ++ch) {
                        __syncwarp();
                        uint32_t v[32];
                        tmem_ld_32x32(tmem_base + lane_base + pd.stage * kDCols + a * NTOK + ch * 32, v);
                        tc_wait_ld();
                        uint4 *dst = reinterpret_cast<uint4 *>(part_row + (int64_t)a * 128 * NTOK + ch * 32);
#pragma unroll
                        for (int i = 0; i < 8; ++i) __stcg(dst + i, make_uint4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]));
                    }
                }
                if (reader) {
                    tc_fence_before();
                    mbar_arrive(smem_u32(&ctl->d_empty[pd.stage]));       // accumulator fully read
                }
                // the CTA that arrives last for this output tile adds the partials and stores
                __threadfence();
                epi_bar<kEpiThreads>();
                if (warp == 6 && lane == 0) ctl->ticket = atomicAdd(p.tickets + (int64_t)out_tile * 4, 1u);
                epi_bar<kEpiThreads>();
                const unsigned int old = ctl->ticket;
                if (old != (unsigned int)(p.splits - 1)) { pd.advance(DB); continue; }
                __threadfence();
                part_row -= (int64_t)split * kTileFloats;                  // row of split 0
            }
#pragma unroll 1
            for (int a = 0; a < NA; ++a) {
                const int32_t blk0 = (out_tile % p.w_tiles) * (NA * 128) + a * 128;   // first distinct row of the block
                const int rows_valid = max(0, min(128, p.r - blk0));
#pragma unroll 1
                for (int ch = 0; ch < n_chunks; ++ch) {
                    __syncwarp();                                 // reconverge before the warp-wide TMEM load
                    uint32_t v[32];
                    if (!reader) {
                        // helpers wait at the barriers below for the readers' block
                    } else if (p.splits > 1) {
                        // sum of the splits in a fixed order (split 0, 1, ...): the result does not depend on
                        // which CTA arrived last
                        constexpr int64_t kTileFloats = (int64_t)NA * 128 * NTOK;
                        float acc[32];
#pragma unroll
                        for (int i = 0; i < 32; ++i) acc[i] = 0.0f;
                        // two splits per round (splits is a power of two): 16 independent 16-byte loads in flight
                        for (int32_t sp = 0; sp < p.splits; sp += 2) {
                            const float4 *src0 = reinterpret_cast<const float4 *>(part_row + (int64_t)sp * kTileFloats +
                                                                                  (int64_t)a * 128 * NTOK + ch * 32);
                            const float4 *src1 = src0 + kTileFloats / 4;
                            float4 q0[8], q1[8];
#pragma unroll
                            for (int i = 0; i < 8; ++i) { q0[i] = __ldcg(src0 + i); q1[i] = __ldcg(src1 + i); }
#pragma unroll
                            for (int i = 0; i < 8; ++i) {
                                acc[4 * i] += q0[i].x; acc[4 * i + 1] += q0[i].y; acc[4 * i + 2] += q0[i].z; acc[4 * i + 3] += q0[i].w;
                            }
#pragma unroll
                            for (int i = 0; i < 8; ++i) {
                                acc[4 * i] += q1[i].x; acc[4 * i + 1] += q1[i].y; acc[4 * i + 2] += q1[i].z; acc[4 * i + 3] += q1[i].w;
                            }
                        }
#pragma unroll
                        for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(acc[i]);
                    } else {
                        tmem_ld_32x32(tmem_base + lane_base + pd.stage * kDCols + a * NTOK + ch * 32, v);
                        tc_wait_ld();
                        if (a == NA - 1 && ch == n_chunks - 1) {  // accumulator fully read: hand it back early
                            tc_fence_before();
                            mbar_arrive(smem_u32(&ctl->d_empty[pd.stage]));
                        }
                    }
                    epi_bar<kEpiThreads>();                                    // the previous block has been read by everyone
                    if (reader) {
#pragma unroll
                        for (int i = 0; i < 32; ++i) xbuf[i][qd * 32 + lane] = __uint_as_float(v[i]);
                    }
                    epi_bar<kEpiThreads>();
                    float z[kSlots][8];
#pragma unroll
                    for (int i = 0; i < kSlots; ++i) {
                        const float4 lo = *reinterpret_cast<const float4 *>(&xbuf[8 * ew + tsub + 2 * (kSlots * iset + i)][f0]);
                        const float4 hi = *reinterpret_cast<const float4 *>(&xbuf[8 * ew + tsub + 2 * (kSlots * iset + i)][f0 + 4]);
                        z[i][0] = lo.x; z[i][1] = lo.y; z[i][2] = lo.z; z[i][3] = lo.w;
                        z[i][4] = hi.x; z[i][5] = hi.y; z[i][6] = hi.z; z[i][7] = hi.w;
                    }
                    const int nvalid = rows_valid - f0;           // this lane's rows that exist
                    if (nvalid <= 0) continue;
                    if (p.act == TBN_ACT_RELU && p.bias == nullptr) {
                        // alpha >= 0, so relu(alpha * z) = alpha * relu(z): clamp once, outside the k loop
#pragma unroll
                        for (int i = 0; i < kSlots; ++i)
#pragma unroll
                            for (int e = 0; e < 8; ++e) z[i][e] = fmaxf(z[i][e], 0.0f);
                    }
                    const int64_t tok_first = tok0 + ch * 32 + 8 * ew + tsub + 2 * kSlots * iset;
                    if (plain && p.y_bf16 && vec_ok && nvalid >= 8) {
                        // The common case, with everything that does not depend on j hoisted out of the k loop: per
                        // repetition 8 multiplies, 4 packs and one 16-byte store per token, nothing else.
                        __nv_bfloat16 *yb[kSlots];
                        bool tv[kSlots];
#pragma unroll
                        for (int i = 0; i < kSlots; ++i) {
                            const int64_t tok = tok_first + 2 * i;
                            tv[i] = tok < p.T;
                            yb[i] = static_cast<__nv_bfloat16 *>(p.y) + tok * p.m + blk0 + f0;
                        }
                        const int32_t kk = p.k, rr = p.r;
                        for (int32_t j = 0; j < kk; ++j) {
                            const float al = j < kMaxAlpha ? ctl->alpha[j]
                                                           : (p.per_tile ? __ldg(p.alpha + j) : __ldg(p.alpha));
#pragma unroll
                            for (int i = 0; i < kSlots; ++i) {
                                uint32_t pk[4];
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    const __nv_bfloat162 h = __floats2bfloat162_rn(al * z[i][2 * e], al * z[i][2 * e + 1]);
                                    pk[e] = *reinterpret_cast<const uint32_t *>(&h);
                                }
                                if (tv[i]) *reinterpret_cast<uint4 *>(yb[i]) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                                yb[i] += rr;
                            }
                        }
                        continue;
                    }
                    for (int32_t j = 0; j < p.k; ++j) {
                        const float al = j < kMaxAlpha ? ctl->alpha[j]
                                                       : (p.per_tile ? __ldg(p.alpha + j) : __ldg(p.alpha));
                        const int64_t o0 = (int64_t)j * p.r + blk0 + f0;
                        if (vec_ok && nvalid >= 8) {
                            float b[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
                            if (!plain) {
                                if (p.bias != nullptr && bias_vec) {          // o0 is a multiple of 8 here
                                    const float4 t0 = __ldg(reinterpret_cast<const float4 *>(p.bias + o0));
                                    const float4 t1 = __ldg(reinterpret_cast<const float4 *>(p.bias + o0) + 1);
                                    b[0] = t0.x; b[1] = t0.y; b[2] = t0.z; b[3] = t0.w;
                                    b[4] = t1.x; b[5] = t1.y; b[6] = t1.z; b[7] = t1.w;
                                } else {
#pragma unroll
                                    for (int e = 0; e < 8; ++e) b[e] = p.bias ? __ldg(p.bias + o0 + e) : 0.0f;
                                }
                            }
                            // all outputs first (the activation's instruction streams interleave), then the stores
                            float o[kSlots][8];
                            if (plain) {
#pragma unroll
                                for (int i = 0; i < kSlots; ++i)
#pragma unroll
                                    for (int e = 0; e < 8; ++e) o[i][e] = al * z[i][e];
                            } else if (p.act == TBN_ACT_GELU && p.y_bf16) {
#pragma unroll
                                for (int i = 0; i < kSlots; ++i)
#pragma unroll
                                    for (int e = 0; e < 8; e += 2)
                                        gelu_tanh_bf16_pair(al, z[i][e], z[i][e + 1], b[e], b[e + 1], o[i][e], o[i][e + 1]);
                            } else if (p.act == TBN_ACT_GELU) {
#pragma unroll
                                for (int i = 0; i < kSlots; ++i)
#pragma unroll
                                    for (int e = 0; e < 8; ++e) o[i][e] = gelu_erf(fmaf(al, z[i][e], b[e]));
                            } else if (p.act == TBN_ACT_RELU) {
#pragma unroll
                                for (int i = 0; i < kSlots; ++i)
#pragma unroll
                                    for (int e = 0; e < 8; ++e) o[i][e] = fmaxf(fmaf(al, z[i][e], b[e]), 0.0f);
                            } else {
#pragma unroll
                                for (int i = 0; i < kSlots; ++i)
#pragma unroll
                                    for (int e = 0; e < 8; ++e) o[i][e] = fmaf(al, z[i][e], b[e]);
                            }
#pragma unroll
                            for (int i = 0; i < kSlots; ++i) {
                                const int64_t tok = tok_first + 2 * i;
                                if (tok >= p.T) continue;
                                const int64_t yi = tok * p.m + o0;
                                if (p.y_bf16) {
                                    uint32_t pk[4];
#pragma unroll
                                    for (int e = 0; e < 4; ++e) {
                                        const __nv_bfloat162 h = __floats2bfloat162_rn(o[i][2 * e], o[i][2 * e + 1]);
                                        pk[e] = *reinterpret_cast<const uint32_t *>(&h);
                                    }
                                    *reinterpret_cast<uint4 *>(static_cast<__nv_bfloat16 *>(p.y) + yi) =
                                        make_uint4(pk[0], pk[1], pk[2], pk[3]);
                                } else {
                                    float4 *dst = reinterpret_cast<float4 *>(static_cast<float *>(p.y) + yi);
                                    dst[0] = make_float4(o[i][0], o[i][1], o[i][2], o[i][3]);
                                    dst[1] = make_float4(o[i][4], o[i][5], o[i][6], o[i][7]);
                                }
                            }
                        } else {
                            // ragged or unaligned rows: element by element
#pragma unroll
                            for (int i = 0; i < kSlots; ++i) {
                                const int64_t tok = tok_first + 2 * i;
                                if (tok >= p.T) continue;
#pragma unroll
                                for (int e = 0; e < 8; ++e) {
                                    if (e >= nvalid) break;
                                    const float bb = p.bias ? __ldg(p.bias + o0 + e) : 0.0f;
                                    const float val = apply_act(fmaf(al, z[i][e], bb), p.act);
                                    const int64_t yi = tok * p.m + o0 + e;
                                    if (p.y_bf16) static_cast<__nv_bfloat16 *>(p.y)[yi] = __float2bfloat16_rn(val);
                                    else static_cast<float *>(p.y)[yi] = val;
                                }
                            }
                        }
                    }
                }
            }
            pd.advance(DB);
        }
    }

    // ---------------- teardown ----------------
    if (warp == 1 && *abort_flag) {
        // make sure no MMA is still reading shared or tensor memory before they are released
        tc_commit_elect(smem_u32(&ctl->x_empty[0]), elect_one());     // by the lane that issued the MMAs
        __syncwarp();
        drain_wait(smem_u32(&ctl->x_empty[0]), 0);
        drain_wait(smem_u32(&ctl->x_empty[0]), 1);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// ---- host side -----------------------------------------------------------------------------------
int sm_count()
{
    static int cache[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    if (!cache[dev]) cudaDeviceGetAttribute(&cache[dev], cudaDevAttrMultiProcessorCount, dev);
    return cache[dev];
}

template <int NTOK, int NA, int KA, int SX, int DB>
int launch_config(const LayerArgs &a, TcParams p, int splits, void *scratch, cudaStream_t s)
{
    EncodeTiledFn encode = encode_tiled_fn();
    if (!encode) return TBN_ERR_CUDA;
    CUtensorMap map;
    const cuuint64_t dims[2] = {(cuuint64_t)a.n, (cuuint64_t)a.T};
    const cuuint64_t strides[1] = {(cuuint64_t)a.n * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kAtomK, (cuuint32_t)NTOK};
    const cuuint32_t estr[2] = {1, 1};
    if (encode(&map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(a.x), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return TBN_ERR_CUDA;

    p.w_tiles = (p.r + NA * 128 - 1) / (NA * 128);
    p.t_tiles = (int32_t)((a.T + NTOK - 1) / NTOK);
    p.k_stages = (a.n + KA * kAtomK - 1) / (KA * kAtomK);
    p.splits = splits;
    const int64_t out_tiles = (int64_t)p.w_tiles * p.t_tiles;
    if (splits > 1) {
        // scratch: [tickets: out_tiles x 4 counters, padded to 256 bytes][partials]
        const size_t ticket_bytes = ((size_t)out_tiles * 4 * sizeof(unsigned int) + 255) / 256 * 256;
        p.tickets = static_cast<unsigned int *>(scratch);
        p.partial = reinterpret_cast<float *>(static_cast<char *>(scratch) + ticket_bytes);
        if (cudaMemsetAsync(scratch, 0, ticket_bytes, s) != cudaSuccess) return TBN_ERR_CUDA;
    } else {
        p.tickets = nullptr;
        p.partial = nullptr;
    }
    const size_t smem = (size_t)SX * KA * NTOK * 128 + sizeof(Control<SX>) + 1024;
    // four helper warps for the epilogue when its arithmetic is heavy (GELU); a plain epilogue is bound by its stores
    const bool helpers = a.act == TBN_ACT_GELU;
    auto kern = helpers ? tc_linear_kernel<NTOK, NA, KA, SX, DB, 8> : tc_linear_kernel<NTOK, NA, KA, SX, DB, 4>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return TBN_ERR_CUDA;
    const int sms = sm_count();
    if (sms <= 0) return TBN_ERR_CUDA;
    const int64_t tiles = out_tiles * splits;
    const unsigned grid = (unsigned)(tiles < sms ? tiles : sms);
    kern<<<grid, kBaseThreads + (helpers ? 256 : 128), smem, s>>>(map, p);
    return cudaGetLastError() == cudaSuccess ? TBN_OK : TBN_ERR_CUDA;
}

// Tile shape and split-K factor for one call.  Cost model in nanoseconds per CTA, fitted to timelines and sweeps on
// B200 (n = 8192; T = 64 .. 16384): the issuing thread needs about 77 ns per MMA whatever the token tile, plus 0.09 ns
// per token; a configuration with only two decoded-weight slots pays about 100 ns of hand-off per stage; the epilogue
// is bound by its stores (about 38 bytes per ns and SM, i.e. 6.7 ns per token and repetition for 128 rows) plus 250 ns
// per 32-token block; every tile costs about 1.5 us of hand-over.  With two accumulator buffers the epilogue hides
// behind the next tile's main loop except for the last tile.
// When the output has fewer tiles than the GPU has SMs, the contraction is split over several CTAs per tile
// (each dumps an fp32 partial tile; the last to arrive adds them in a fixed order and stores).
struct Cand { int ntok, na, ka, db; };
// 224 tokens: 74 token tiles at T = 16384, so 4 or 8 row blocks give an exact multiple of 148 CTAs
constexpr Cand kCands[] = {{256, 1, 2, 1}, {192, 1, 2, 2}, {128, 2, 2, 1}, {128, 1, 2, 2}, {64, 1, 2, 2}, {32, 1, 2, 2},
                           {224, 1, 2, 1}};
constexpr int kNumCands = 7;

struct Plan { int cand, splits; size_t scratch_bytes; };

// Forced tile shape / split factor (testing and tuning aid; -1 = the cost model decides).
std::atomic<int> g_forced_cand{-1}, g_forced_splits{1};

Plan plan_linear(const LayerArgs &a)
{
    const int sms = sm_count() > 0 ? sm_count() : 148;
    const int32_t r = (int32_t)(a.q / a.n);
    const double atoms = (double)((a.n + kAtomK - 1) / kAtomK);
    Plan best = {0, 1, 0};
    double best_cost = 1e300;
    for (int i = 0; i < kNumCands; ++i) {
        const Cand &c = kCands[i];
        const int64_t wt = (r + c.na * 128 - 1) / (c.na * 128);
        const int64_t tt = (a.T + c.ntok - 1) / c.ntok;
        const int64_t out_tiles = wt * tt;
        const int k_stages = (a.n + c.ka * kAtomK - 1) / (c.ka * kAtomK);
        const bool four_slots = c.db * c.na * c.ntok + 4 * c.na * c.ka * 32 <= 512;    // decoded-weight slots in tensor memory
        const double stage = c.na * c.ka * 4 * (0.09 * c.ntok + 77.0) + (four_slots ? 0.0 : 100.0);
        const double epi = c.na * (double)c.ntok * a.k * 6.7 + c.na * (c.ntok / 32.0) * 250.0;
        const double per_tile = 1500.0;                 // tile hand-over: first bit words, barrier round trips
        const double dump = c.na * (c.ntok / 32.0) * 60.0 * 2.0;
        for (int sp = 1; sp <= 16; sp *= 2) {
            if (sp > 1 && (k_stages < 2 * sp || out_tiles * sp > sms)) break;   // >= 2 stages per split, one wave
            const int64_t waves = (out_tiles * sp + sms - 1) / sms;
            const double mainloop = atoms / c.ka / sp * stage;
            double cost;
            if (sp == 1) cost = c.db == 2 ? mainloop + (waves - 1) * ((mainloop > epi ? mainloop : epi) + per_tile) + epi + per_tile
                                          : waves * (mainloop + epi + per_tile);
            else cost = mainloop + dump + epi + 1500.0 +                        // ticket / partial round trip
                        c.na * (c.ntok < a.T ? c.ntok : (double)a.T) / 32.0 * (sp / 2) * 1000.0;   // reduction: one L2 round per two splits and 32 tokens
            if (cost < best_cost) {
                best_cost = cost;
                best.cand = i;
                best.splits = sp;
                best.scratch_bytes = sp == 1 ? 0
                    : ((size_t)out_tiles * 4 * sizeof(unsigned int) + 255) / 256 * 256 +
                      (size_t)out_tiles * sp * c.na * 128 * c.ntok * sizeof(float);
            }
        }
    }
    return best;
}

}  // namespace

// Exercises the bounded waits themselves: a block waits on an mbarrier that nothing ever arrives at.  Warp 0 (all
// lanes) runs out of time, records the status and raises the block's abort flag; warp 1's single waiting lane leaves
// through the abort flag; one thread then runs the quiet drain wait.  The kernel returns normally.
__global__ void __launch_bounds__(64, 1)
wait_probe_kernel(int *status, int detail)
{
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        abort_flag = 0;
        fence_barrier_init();
    }
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    bool ok = true;
    if (warp == 0) ok = wait_bar(smem_u32(&bar), 0u, &abort_flag, status, detail);
    else if (lane == 0) ok = wait_one(smem_u32(&bar), 0u, &abort_flag, status, detail + 1);
    __syncthreads();
    if (threadIdx.x == 0) {
        drain_wait(smem_u32(&bar), 0u);
        if (ok) status[1] = -1;          // the wait must not have succeeded: nothing arrives at this barrier
    }
}

cudaError_t launch_wait_probe(int *status, int detail, cudaStream_t s)
{
    wait_probe_kernel<<<1, 64, 0, s>>>(status, detail);
    return cudaGetLastError();
}

int force_linear_config(int candidate, int splits)
{
    if (candidate < 0) { g_forced_cand.store(-1); g_forced_splits.store(1); return TBN_OK; }
    // the epilogue adds the partial tiles in pairs: only powers of two up to 16 are valid split factors
    if (candidate >= kNumCands || (splits != 1 && splits != 2 && splits != 4 && splits != 8 && splits != 16))
        return TBN_ERR_INVALID_ARG;
    g_forced_splits.store(splits);
    g_forced_cand.store(candidate);
    return TBN_OK;
}

bool tensor_path_supported(const LayerArgs &a)
{
    if (a.is_conv) return false;
    if (a.q % a.n != 0) return false;            // the tile must span whole rows
    if (a.n % 8 != 0) return false;              // TMA: row pitch a multiple of 16 bytes
    if (a.T >= (int64_t)1 << 31) return false;   // TMA coordinates are 32-bit
    return true;
}

size_t tensor_linear_scratch_bytes(const LayerArgs &a)
{
    return tensor_path_supported(a) ? plan_linear(a).scratch_bytes : 0;
}

int launch_tensor_linear(const LayerArgs &a, int *device_status, void *scratch, size_t scratch_bytes, cudaStream_t s)
{
    if (a.x_dtype != TBN_BF16) return TBN_ERR_UNSUPPORTED;
    TcParams p;
    p.tile = a.tile; p.dense_a = static_cast<const __nv_bfloat16 *>(a.dense_a); p.alpha = a.alpha; p.bias = a.bias; p.y = a.y; p.status = device_status;
    p.T = a.T; p.n_words = a.dense_a ? 1 : tbn_tile_words(a.q);
    p.n = a.n; p.m = a.m; p.r = (int32_t)(a.q / a.n); p.k = a.k;
    p.k_stages = 0;
    p.w_tiles = 0; p.t_tiles = 0; p.splits = 1; p.partial = nullptr; p.tickets = nullptr;
    p.per_tile = a.alpha_mode == TBN_ALPHA_PER_TILE; p.act = a.act; p.y_bf16 = a.y_dtype == TBN_BF16;

    Plan plan = plan_linear(a);
    const int forced = g_forced_cand.load(std::memory_order_relaxed);
    if (forced >= 0 && forced < kNumCands) {            // testing / tuning aid, see force_linear_config()
        plan.cand = forced;
        plan.splits = g_forced_splits.load(std::memory_order_relaxed);
        const Cand &c = kCands[plan.cand];
        const int64_t out_tiles = (int64_t)((p.r + c.na * 128 - 1) / (c.na * 128)) * ((a.T + c.ntok - 1) / c.ntok);
        const int k_stages = (a.n + c.ka * kAtomK - 1) / (c.ka * kAtomK);
        while (plan.splits > 1 && k_stages < 2 * plan.splits) plan.splits >>= 1;   // at least two stages per split
        plan.scratch_bytes = plan.splits == 1 ? 0
            : ((size_t)out_tiles * 4 * sizeof(unsigned int) + 255) / 256 * 256 +
              (size_t)out_tiles * plan.splits * c.na * 128 * c.ntok * sizeof(float);
    }
    if (plan.splits > 1 && (!scratch || scratch_bytes < plan.scratch_bytes)) {
        plan.splits = 1;                              // not enough scratch: run unsplit (same result, slower)
    }
    switch (plan.cand) {
    case 0: return launch_config<256, 1, 2, 3, 1>(a, p, plan.splits, scratch, s);
    case 1: return launch_config<192, 1, 2, 4, 2>(a, p, plan.splits, scratch, s);
    case 2: return launch_config<128, 2, 2, 5, 1>(a, p, plan.splits, scratch, s);
    case 3: return launch_config<128, 1, 2, 6, 2>(a, p, plan.splits, scratch, s);
    case 4: return launch_config<64, 1, 2, 8, 2>(a, p, plan.splits, scratch, s);
    case 6: return launch_config<224, 1, 2, 3, 1>(a, p, plan.splits, scratch, s);
    default: return launch_config<32, 1, 2, 8, 2>(a, p, plan.splits, scratch, s);
    }
}

}  // namespace tbn
