// Tensor-core forward of a tiled layer with BINARY activations on sm_100a (Sec. 7 of the paper: binary weights and
// binary activations): the XNOR / popcount contraction mapped onto the 8-bit integer tcgen05.mma.
//
// Problem.  The tile spans r = q/n whole rows; the activations arrive as one sign bit per value (bit 1 = +1).  For
// distinct row c and token t the layer needs D[t][c] = sum_j b[c][j] a[t][j] over +-1 values.  With the bits
// w, x in {0,1}:   D = n - 2 popcount(w xor x) = 4 P - 2 popcount(w) - 2 popcount(x) + n,   P = popcount(w and x).
// P is an ordinary matrix product of 0/1 matrices, so it runs on the tensor cores: both bit rows are expanded on chip
// into bytes 0x00 / 0xFF (0 and -1 as signed 8-bit values; (-1)(-1) = +1, so the int32 accumulator is exactly P),
// and popcount(w), popcount(x) are counted by the warps that expand them.  Everything is exact in integers.
//
// Why bytes of 0 / -1 rather than +-1: the expansion is the kernel's ALU cost, and "byte = its top bit replicated"
// is ONE byte-permute per four elements (prmt in sign mode on the word shifted left by s gives bits 7-s, 15-s, 23-s,
// 31-s); +-1 would need another operation per four elements on both operands.  The contraction index inside a
// 32-bit word is permuted by this (element 4s + j of the word's group holds bit 8j + 7 - s) -- identically for the
// weights and for the activations, so the product is unchanged.
//
// Operand roles as in the bf16 kernel: decoded weights are the A operand in tensor memory (UMMA M = 128 rows, written
// with tcgen05.st), activations are the B operand in shared memory (K-major, 128-byte swizzle; written by producer
// warps with ordinary stores in the swizzled layout, since no copy engine expands bits), accumulators in tensor memory.
// A stage is 256 contraction elements: 8 words of bits per row, 8 MMAs of K = 32.
//
// Byte form of the activations (template flag BYTES): when the caller has expanded the activation bits to the same
// 0x00 / 0xFF bytes in global memory once (tbn_bin_expand_fwd, same element order), the stage is filled by TMA like the
// bf16 kernel's and the producer warps only fetch the row popcounts (counted once, with the bytes): the shared-memory stores of the expansion, which
// bind the bit form, disappear, at the price of an 8 times larger activation tensor in HBM.
//
// Warp roles (13 warps): 0-3 activation producers, 4 MMA issuer / TMEM owner, 5-8 weight decode, 9-12 epilogue
// (tcgen05.ld -> integer combine -> exchange through shared memory -> beta_t alpha_j scaling, bias, activation ->
// k-fold replicated stores).  All hand-offs are mbarriers; every wait is bounded (see tc_common.cuh).
#include <atomic>
#include <cstddef>
#include <cstring>

#include "tc_common.cuh"

namespace tbn {

namespace {

using namespace tc;

constexpr int kBinThreads = 13 * 32;
constexpr int kBinProd = 128;            // producer threads (warps 0-3)
constexpr int kBinMmaWarp = 4;
constexpr int kBinAtomK = 128;           // contraction elements (bytes) per 128-byte swizzle row
constexpr int kBinKA = 2;                // swizzle rows per stage
constexpr int kBinStageK = kBinKA * kBinAtomK;      // 256 elements = 8 words of bits per row and stage
constexpr int kBinAStages = 4;           // decoded-weight stages in tensor memory, 64 columns each
constexpr int kBinACols = kBinStageK / 4;
constexpr int kBinXPitch = 132;          // words per token row of the epilogue exchange buffer

template <int SX>
struct BinControl {
    uint64_t x_full[SX], x_empty[SX];
    uint64_t a_full[kBinAStages], a_empty[kBinAStages];
    uint64_t d_full[2], d_empty[2];
    uint64_t side_full[2], side_empty[2];          // popcounts of the tile's token rows and weight rows
    uint32_t tmem_base;
    int abort_flag;
    float alpha[64];
    int32_t px[2][256];
    int32_t pw[2][128];
    alignas(16) uint32_t exchange[32 * kBinXPitch];
};

struct BinParams {
    const uint32_t *x_bits;
    const int32_t *x_pop;    // byte form: popcount of every activation row
    const uint32_t *tile;
    const float *alpha;
    const float *beta;
    const float *bias;
    void *y;
    int *status;
    int64_t T;
    int32_t xw;          // words per activation row (a multiple of 4)
    int32_t n, m, r, k;
    int32_t nw;          // n / 32
    int32_t k_stages;    // ceil(n / 256)
    int32_t w_tiles, t_tiles;
    int per_tile, act, y_mode;   // y_mode: 0 fp32, 1 bf16, 2 raw int32
};

// byte j of the result = bit 7 of byte j of v, replicated (0x00 or 0xFF)
__device__ __forceinline__ uint32_t top_bits_to_bytes(uint32_t v) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %1, 0xBA98;" : "=r"(d) : "r"(v));
    return d;
}
// 32 bits -> 32 bytes (8 registers): register s, byte j <- bit 8j + 7 - s
__device__ __forceinline__ void expand_word(uint32_t w, uint32_t *out) {
#pragma unroll
    for (int s = 0; s < 8; ++s) out[s] = top_bits_to_bytes(w << s);
}

__device__ __forceinline__ void epi_bar128() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
__device__ __forceinline__ int epi_bar128_count(bool pred) {
    int n;
    asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %1, 0;\nbar.red.popc.u32 %0, 1, 128, p;\n}"
                 : "=r"(n) : "r"((int)pred) : "memory");
    return n;
}

// D[tmem] (+)= A[tmem] * B[smem]^T, signed 8-bit x signed 8-bit -> int32, M = 128, K = 32
// (executed by the whole converged warp, performed by the elected lane: see tc_mma_ts_elect)
__device__ __forceinline__ void tc_mma_ts_i8(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_desc_lo, uint32_t b_desc_hi,
                                             uint32_t idesc, uint32_t accumulate, uint32_t leader) {
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t.reg .b64 bd;\n\t"
        "setp.ne.b32 q, %6, 0;\n\t"
        "setp.ne.b32 p, %5, 0;\n\t"
        "mov.b64 bd, {%2, %3};\n\t"
        "@q tcgen05.mma.cta_group::1.kind::i8 [%0], [%1], bd, %4, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "r"(b_desc_lo), "r"(b_desc_hi), "r"(idesc), "r"(accumulate), "r"(leader) : "memory");
}

constexpr uint64_t kBinBDescHi = (64ull << 32) | (1ull << 46) | (2ull << 61);   // as the bf16 kernel: SW128, K-major

template <int NTOK, int SX, int DB, bool BYTES>
__global__ void __launch_bounds__(kBinThreads, 1)
tc_linear_bin_kernel(const __grid_constant__ CUtensorMap xb_map, const BinParams p)
{
    // BYTES: the activation bytes exist in global memory (tbn_bin_expand_fwd) and TMA stages them; warp 0 issues the
    // copies, warps 1-3 fetch the tile's row popcounts
    constexpr uint32_t kXFullCount = BYTES ? 1u : (uint32_t)kBinProd;
    constexpr uint32_t kSideProd = BYTES ? 96u : (uint32_t)kBinProd;
    static_assert(NTOK == 128 || NTOK == 256, "token tile");
    constexpr uint32_t kAtomBytes = NTOK * 128;
    constexpr uint32_t kStageBytes = kBinKA * kAtomBytes;
    constexpr uint32_t kDCols = NTOK;
    constexpr uint32_t kABase = DB * kDCols;
    constexpr uint32_t kTmemCols = 512;
    static_assert(kABase + kBinAStages * kBinACols <= kTmemCols, "tensor memory budget");
    // instruction descriptor: D int32, A and B signed 8-bit, both K-major, N = NTOK, M = 128
    constexpr uint32_t kIdesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(NTOK >> 3) << 17) | (8u << 24);

    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    uint8_t *smem = smem_raw + ((1024u - (raw & 1023u)) & 1023u);
    BinControl<SX> *ctl = reinterpret_cast<BinControl<SX> *>(smem + SX * kStageBytes);
    const uint32_t stage0 = smem_u32(smem);
    volatile int *abort_flag = &ctl->abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int bid = blockIdx.x;

    if (threadIdx.x == 0) {
        for (int s = 0; s < SX; ++s) { mbar_init(smem_u32(&ctl->x_full[s]), kXFullCount); mbar_init(smem_u32(&ctl->x_empty[s]), 1); }
        for (int s = 0; s < kBinAStages; ++s) { mbar_init(smem_u32(&ctl->a_full[s]), 128); mbar_init(smem_u32(&ctl->a_empty[s]), 1); }
        for (int s = 0; s < 2; ++s) {
            mbar_init(smem_u32(&ctl->d_full[s]), 1); mbar_init(smem_u32(&ctl->d_empty[s]), 128);
            mbar_init(smem_u32(&ctl->side_full[s]), kSideProd + 128); mbar_init(smem_u32(&ctl->side_empty[s]), 128);
        }
        ctl->abort_flag = 0;
        fence_barrier_init();
        fence_proxy_async();
    }
    if (threadIdx.x < 64 && (int)threadIdx.x < p.k)
        ctl->alpha[threadIdx.x] = p.per_tile ? __ldg(p.alpha + threadIdx.x) : __ldg(p.alpha);
    if (warp == kBinMmaWarp) {
        tmem_alloc(smem_u32(&ctl->tmem_base), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;

    // A tile index enumerates (token tile, row block) with the row block fastest: CTAs running at one time share a
    // few token panels.
    const int32_t n_tiles = p.w_tiles * p.t_tiles;
    bool ok = true;

    if (BYTES && warp == 0) {
        // ---------------- loader: activation bytes -> swizzled shared-memory stage by TMA ----------------
        // Rows past T and columns past n arrive as zeros (and still count their bytes on the barrier).
        Pipe px;
        uint32_t issued_mask = 0, issued_phase = 0;
        for (int32_t tile = bid; tile < n_tiles && ok; tile += gridDim.x) {
            const int32_t tok0 = (tile / p.w_tiles) * NTOK;
            for (int32_t ks = 0; ks < p.k_stages; ++ks) {
                ok = wait_bar(smem_u32(&ctl->x_empty[px.stage]), px.phase ^ 1u, abort_flag, p.status,
                              (1 << 24) | (px.stage << 16) | (bid & 0xffff));
                if (!ok) break;
                if (lane == 0) {
                    const uint32_t bar = smem_u32(&ctl->x_full[px.stage]);
                    mbar_arrive_expect_tx(bar, kStageBytes);
#pragma unroll
                    for (int at = 0; at < kBinKA; ++at)
                        tma_load_2d(stage0 + px.stage * kStageBytes + at * kAtomBytes, &xb_map, ks * kBinStageK + at * kBinAtomK,
                                    tok0, bar);
                }
                issued_mask |= 1u << px.stage;
                issued_phase = (issued_phase & ~(1u << px.stage)) | (px.phase << px.stage);
                __syncwarp();
                px.advance(SX);
            }
        }
        if (!ok) {   // let copies in flight land before the block's shared memory goes away
            for (int s = 0; s < SX; ++s)
                if (issued_mask & (1u << s)) drain_wait(smem_u32(&ctl->x_full[s]), (issued_phase >> s) & 1u);
        }
    } else if (BYTES && warp < kBinMmaWarp) {
        // ---------------- row popcounts of the tile's tokens, counted once when the bytes were written (warps 1-3) ----------------
        uint32_t sd = 0, sd_phase = 0;
        for (int32_t tile = bid; tile < n_tiles; tile += gridDim.x) {
            ok = wait_bar(smem_u32(&ctl->side_empty[sd]), sd_phase ^ 1u, abort_flag, p.status, (9 << 24) | (bid & 0xffff));
            if (!ok) break;
            const int64_t tok0 = (int64_t)(tile / p.w_tiles) * NTOK;
            for (int row = (warp - 1) * 32 + lane; row < NTOK; row += 96) {
                const int64_t tok = tok0 + row;
                ctl->px[sd][row] = tok < p.T ? __ldg(p.x_pop + tok) : 0;
            }
            __syncwarp();
            mbar_arrive(smem_u32(&ctl->side_full[sd]));
            sd ^= 1u;
            if (sd == 0) sd_phase ^= 1u;
        }
    } else if (warp < kBinMmaWarp) {
        // ---------------- activation producers: bits -> bytes -> swizzled shared-memory stage ----------------
        // Thread tid owns token rows tid, tid + 128 (, ...) of the tile: per stage it reads the row's 8 words (one
        // 32-byte sector), expands them and writes the row's 128-byte line of each of the two swizzle rows: the
        // 16-byte piece c of row R goes to position c xor (R mod 8), so the 8 lanes of a quarter warp hit 8
        // different bank groups.
        // The bits of a stage are requested two stages ahead (across tile boundaries too): a stage's loads are a
        // round trip to L2, longer than the expansion of a stage, and nothing else would hide it.
        const int tid = threadIdx.x;
        constexpr int H = NTOK / 128;
        Pipe px;
        uint32_t sd = 0, sd_phase = 0;
        auto load_bits = [&](uint4 (&v)[H][2], int32_t tl, int32_t ks) {
            const int64_t tok0 = (int64_t)(tl / p.w_tiles) * NTOK;
#pragma unroll
            for (int h = 0; h < H; ++h) {
                const int64_t tok = tok0 + tid + 128 * h;
                v[h][0] = v[h][1] = make_uint4(0u, 0u, 0u, 0u);
                if (tl < n_tiles && tok < p.T) {
                    const uint4 *src = reinterpret_cast<const uint4 *>(p.x_bits + tok * p.xw + ks * 8);
                    if (ks * 8 < p.xw) v[h][0] = __ldg(src);
                    if (ks * 8 + 4 < p.xw) v[h][1] = __ldg(src + 1);
                }
            }
        };
        auto next_item = [&](int32_t &tl, int32_t &ks) {
            if (++ks == p.k_stages) { ks = 0; tl += gridDim.x; }
        };
        int32_t tile = bid, ks = 0;                         // the stage being expanded
        int32_t ltile = bid, lks = 0;                       // the stage being requested
        uint4 cur[H][2], nx1[H][2], nx2[H][2];
        load_bits(cur, ltile, lks); next_item(ltile, lks);
        load_bits(nx1, ltile, lks); next_item(ltile, lks);
        int32_t pc[H];
#pragma unroll
        for (int h = 0; h < H; ++h) pc[h] = 0;
        while (tile < n_tiles) {
            load_bits(nx2, ltile, lks); next_item(ltile, lks);
            ok = wait_bar(smem_u32(&ctl->x_empty[px.stage]), px.phase ^ 1u, abort_flag, p.status,
                          (1 << 24) | (px.stage << 16) | (bid & 0xffff));
            if (!ok) break;
#pragma unroll
            for (int h = 0; h < H; ++h) {
                const int row = tid + 128 * h;
                const uint32_t sw = (uint32_t)row & 7u;
#pragma unroll
                for (int at = 0; at < kBinKA; ++at) {
                    const uint32_t w4[4] = {cur[h][at].x, cur[h][at].y, cur[h][at].z, cur[h][at].w};
                    const uint32_t line = stage0 + px.stage * kStageBytes + at * kAtomBytes + (uint32_t)row * 128u;
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        pc[h] += __popc(w4[i]);
                        uint32_t e[8];
                        expand_word(w4[i], e);
                        sts_v4(line + (((uint32_t)(2 * i) ^ sw) << 4), e[0], e[1], e[2], e[3]);
                        sts_v4(line + (((uint32_t)(2 * i + 1) ^ sw) << 4), e[4], e[5], e[6], e[7]);
                    }
                }
            }
            fence_proxy_async();                           // generic-proxy stores -> visible to the tensor core
            mbar_arrive(smem_u32(&ctl->x_full[px.stage]));
            px.advance(SX);
            if (ks == p.k_stages - 1) {
                // the tile's row popcounts for the epilogue
                ok = wait_bar(smem_u32(&ctl->side_empty[sd]), sd_phase ^ 1u, abort_flag, p.status, (9 << 24) | (bid & 0xffff));
                if (!ok) break;
#pragma unroll
                for (int h = 0; h < H; ++h) { ctl->px[sd][tid + 128 * h] = pc[h]; pc[h] = 0; }
                mbar_arrive(smem_u32(&ctl->side_full[sd]));
                sd ^= 1u;
                if (sd == 0) sd_phase ^= 1u;
            }
            next_item(tile, ks);
#pragma unroll
            for (int h = 0; h < H; ++h) {
                cur[h][0] = nx1[h][0]; cur[h][1] = nx1[h][1];
                nx1[h][0] = nx2[h][0]; nx1[h][1] = nx2[h][1];
            }
        }
    } else if (warp == kBinMmaWarp) {
        // ---------------- MMA issuer: 8 MMAs of K = 32 per stage ----------------
        {
            const uint32_t tmem_u = __shfl_sync(0xffffffffu, tmem_base, 0);
            const uint32_t leader = elect_one();
            Pipe px, pa, pd;
            bool ready = false;
            constexpr uint32_t kDescHi = (uint32_t)(kBinBDescHi >> 32);
            constexpr int kSteps = kBinKA * 4;
            for (int32_t tile = bid; tile < n_tiles && ok; tile += gridDim.x) {
                ok = wait_bar(smem_u32(&ctl->d_empty[pd.stage]), pd.phase ^ 1u, abort_flag, p.status,
                              (2 << 24) | (bid & 0xffff));
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
                    const uint32_t a_addr = tmem_u + kABase + pa.stage * kBinACols;
                    Pipe nx = px, na = pa;
                    nx.advance(SX);
                    na.advance(kBinAStages);
                    // a ragged last stage holds zeros past the row's end on both sides: all K steps run
#pragma unroll
                    for (int st = 0; st < kSteps; ++st) {
                        const int at = st >> 2, kk = st & 3;
                        tc_mma_ts_i8(d_addr, a_addr + at * 32 + kk * 8, b_lo + at * (kAtomBytes >> 4) + kk * 2, kDescHi,
                                     kIdesc, st > 0 ? 1u : (uint32_t)(ks > 0), leader);
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
        }
        __syncwarp();
    } else if (warp < kBinMmaWarp + 5) {
        // ---------------- weight decode: row bits -> bytes -> tensor memory ----------------
        // Thread (quadrant qd, lane) owns TMEM lane L = 32 qd + lane = weight row L of the block; rows start on word
        // boundaries (n is a multiple of 32).  Words past the row's end are taken as zero.
        const int qd = warp & 3;
        const int L = qd * 32 + lane;
        const uint32_t lane_base = (uint32_t)(qd * 32) << 16;
        Pipe pa;
        uint32_t sd = 0, sd_phase = 0;
        for (int32_t tile = bid; tile < n_tiles && ok; tile += gridDim.x) {
            const int32_t row = min((tile % p.w_tiles) * 128 + L, p.r - 1);      // rows past the end are never stored
            const uint32_t *wrow = p.tile + (int64_t)row * p.nw;
            int32_t pcw = 0;
            uint32_t w[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) w[i] = i < p.nw ? __ldg(wrow + i) : 0u;
            for (int32_t ks = 0; ks < p.k_stages && ok; ++ks) {
                uint32_t v[kBinKA][32];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    pcw += __popc(w[i]);
                    expand_word(w[i], &v[i >> 2][8 * (i & 3)]);
                }
                if (ks + 1 < p.k_stages) {
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const int32_t wi = (ks + 1) * 8 + i;
                        w[i] = wi < p.nw ? __ldg(wrow + wi) : 0u;
                    }
                }
                ok = wait_bar(smem_u32(&ctl->a_empty[pa.stage]), pa.phase ^ 1u, abort_flag, p.status,
                              (5 << 24) | (pa.stage << 16) | (bid & 0xffff));
                if (!ok) break;
                tc_fence_after();
#pragma unroll
                for (int at = 0; at < kBinKA; ++at)
                    tmem_st_32x32(tmem_base + lane_base + kABase + pa.stage * kBinACols + at * 32, v[at]);
                tc_wait_st();
                tc_fence_before();
                mbar_arrive(smem_u32(&ctl->a_full[pa.stage]));
                pa.advance(kBinAStages);
            }
            if (!ok) break;
            ok = wait_bar(smem_u32(&ctl->side_empty[sd]), sd_phase ^ 1u, abort_flag, p.status, (10 << 24) | (bid & 0xffff));
            if (!ok) break;
            ctl->pw[sd][L] = pcw;
            mbar_arrive(smem_u32(&ctl->side_full[sd]));
            sd ^= 1u;
            if (sd == 0) sd_phase ^= 1u;
        }
    } else {
        // ---------------- epilogue ----------------
        // tcgen05.ld gives thread (qd, lane) weight row L and 32 consecutive tokens of P; the thread turns them into
        // D = 4 P - 2 popcount(w_L) - 2 popcount(x_t) + n, and the four warps exchange each 128-row x 32-token block
        // through shared memory [token][row] so that a lane comes back with 8 consecutive features of a token: a warp
        // store covers 2 tokens x 256 contiguous bytes (bf16).  Each repetition j is then a multiply by alpha_j on the
        // value already scaled by the token's beta.
        const int qd = warp & 3;
        const int ew = warp - (kBinMmaWarp + 5);          // stores tokens 8 ew .. 8 ew + 7 of each 32-token block
        const uint32_t lane_base = (uint32_t)(qd * 32) << 16;
        uint32_t (*xbuf)[kBinXPitch] = reinterpret_cast<uint32_t (*)[kBinXPitch]>(ctl->exchange);
        Pipe pd;
        uint32_t sd = 0, sd_phase = 0;
        const bool vec_ok = (p.m % 8 == 0) && (p.r % 8 == 0);
        const int f0 = 8 * (lane & 15);
        const int tsub = lane >> 4;
        const bool plain = p.bias == nullptr && (p.act == TBN_ACT_NONE || p.act == TBN_ACT_RELU);
        for (int32_t tile = bid; tile < n_tiles; tile += gridDim.x) {
            const int64_t tok0 = (int64_t)(tile / p.w_tiles) * NTOK;
            ok = wait_bar(smem_u32(&ctl->d_full[pd.stage]), pd.phase, abort_flag, p.status, (6 << 24) | (bid & 0xffff)) &&
                 wait_bar(smem_u32(&ctl->side_full[sd]), sd_phase, abort_flag, p.status, (11 << 24) | (bid & 0xffff));
            if (epi_bar128_count(ok) != 128) { ok = false; break; }       // the four warps go on together or not at all
            tc_fence_after();
            const int n_chunks = (int)min((int64_t)(NTOK / 32), (p.T - tok0 + 31) / 32);
            const int32_t base_term = p.n - 2 * ctl->pw[sd][qd * 32 + lane];
            const int32_t blk0 = (tile % p.w_tiles) * 128;
            const int rows_valid = max(0, min(128, p.r - blk0));
#pragma unroll 1
            for (int ch = 0; ch < n_chunks; ++ch) {
                __syncwarp();
                uint32_t v[32];
                tmem_ld_32x32(tmem_base + lane_base + pd.stage * kDCols + ch * 32, v);
                tc_wait_ld();
                int32_t d[32];
#pragma unroll
                for (int i = 0; i < 32; ++i) d[i] = 4 * (int32_t)v[i] + base_term - 2 * ctl->px[sd][ch * 32 + i];
                if (ch == n_chunks - 1) {                   // accumulator and popcounts fully read: hand both back
                    tc_fence_before();
                    mbar_arrive(smem_u32(&ctl->d_empty[pd.stage]));
                    mbar_arrive(smem_u32(&ctl->side_empty[sd]));
                }
                epi_bar128();                               // the previous block has been read by everyone
                if (p.y_mode == 2) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) xbuf[i][qd * 32 + lane] = (uint32_t)d[i];
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) xbuf[i][qd * 32 + lane] = __float_as_uint((float)d[i]);
                }
                epi_bar128();
                const int nvalid = rows_valid - f0;
                if (nvalid <= 0) continue;
                const int64_t tok_first = tok0 + ch * 32 + 8 * ew + tsub;
                if (p.y_mode == 2) {
                    // raw accumulators: every repetition of a distinct row has the same integer
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int64_t tok = tok_first + 2 * i;
                        if (tok >= p.T) continue;
                        const uint32_t *src = &xbuf[8 * ew + tsub + 2 * i][f0];
                        for (int32_t j = 0; j < p.k; ++j)
                            for (int e = 0; e < 8 && e < nvalid; ++e)
                                static_cast<int32_t *>(p.y)[tok * p.m + (int64_t)j * p.r + blk0 + f0 + e] = (int32_t)src[e];
                    }
                    continue;
                }
                float z[4][8];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int64_t tok = tok_first + 2 * i;
                    const float bt = (p.beta != nullptr && tok < p.T) ? __ldg(p.beta + tok) : 1.0f;
                    const float4 lo = *reinterpret_cast<const float4 *>(&xbuf[8 * ew + tsub + 2 * i][f0]);
                    const float4 hi = *reinterpret_cast<const float4 *>(&xbuf[8 * ew + tsub + 2 * i][f0 + 4]);
                    z[i][0] = bt * lo.x; z[i][1] = bt * lo.y; z[i][2] = bt * lo.z; z[i][3] = bt * lo.w;
                    z[i][4] = bt * hi.x; z[i][5] = bt * hi.y; z[i][6] = bt * hi.z; z[i][7] = bt * hi.w;
                }
                if (p.act == TBN_ACT_RELU && p.bias == nullptr) {
                    // alpha >= 0 and beta >= 0: relu(alpha beta d) = alpha relu(beta d), clamped once outside the k loop
#pragma unroll
                    for (int i = 0; i < 4; ++i)
#pragma unroll
                        for (int e = 0; e < 8; ++e) z[i][e] = fmaxf(z[i][e], 0.0f);
                }
                if (plain && p.y_mode == 1 && vec_ok && nvalid >= 8) {
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
                            o[e] = plain ? val : (p.act == TBN_ACT_GELU && p.y_mode == 1) ? gelu_tanh_bf16(val) : apply_act(val, p.act);
                        }
                        const int64_t yi = tok * p.m + o0;
                        if (vec_ok && nvalid >= 8) {
                            if (p.y_mode == 1) {
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
                                if (p.y_mode == 1) static_cast<__nv_bfloat16 *>(p.y)[yi + e] = __float2bfloat16_rn(o[e]);
                                else static_cast<float *>(p.y)[yi + e] = o[e];
                            }
                        }
                    }
                }
            }
            pd.advance(DB);
            sd ^= 1u;
            if (sd == 0) sd_phase ^= 1u;
        }
    }

    // ---------------- teardown ----------------
    if (warp == kBinMmaWarp && *abort_flag) {
        // make sure no MMA is still reading shared or tensor memory before they are released
        tc_commit_elect(smem_u32(&ctl->x_empty[0]), elect_one());     // by the lane that issued the MMAs
        __syncwarp();
        drain_wait(smem_u32(&ctl->x_empty[0]), 0);
        drain_wait(smem_u32(&ctl->x_empty[0]), 1);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == kBinMmaWarp) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

int bin_sm_count()
{
    static int cache[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    if (!cache[dev]) cudaDeviceGetAttribute(&cache[dev], cudaDevAttrMultiProcessorCount, dev);
    return cache[dev];
}

template <int NTOK, int SX, int DB>
int launch_bin_config(BinParams p, const void *x_bytes, cudaStream_t s)
{
    p.w_tiles = (p.r + 127) / 128;
    p.t_tiles = (int32_t)((p.T + NTOK - 1) / NTOK);
    const size_t smem = (size_t)SX * kBinKA * NTOK * 128 + sizeof(BinControl<SX>) + 1024;
    CUtensorMap map;
    std::memset(&map, 0, sizeof(map));
    if (x_bytes) {                                         // T rows of n bytes; a box is one swizzle row of a stage
        EncodeTiledFn encode = encode_tiled_fn();
        if (!encode) return TBN_ERR_CUDA;
        const cuuint64_t dims[2] = {(cuuint64_t)p.n, (cuuint64_t)p.T};
        const cuuint64_t strides[1] = {(cuuint64_t)p.n};
        const cuuint32_t box[2] = {(cuuint32_t)kBinAtomK, (cuuint32_t)NTOK};
        const cuuint32_t estr[2] = {1, 1};
        if (encode(&map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void *>(x_bytes), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return TBN_ERR_CUDA;
    }
    auto kern = x_bytes ? tc_linear_bin_kernel<NTOK, SX, DB, true> : tc_linear_bin_kernel<NTOK, SX, DB, false>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return TBN_ERR_CUDA;
    const int sms = bin_sm_count();
    if (sms <= 0) return TBN_ERR_CUDA;
    const int64_t tiles = (int64_t)p.w_tiles * p.t_tiles;
    const unsigned grid = (unsigned)(tiles < sms ? tiles : sms);
    kern<<<grid, kBinThreads, smem, s>>>(map, p);
    return cudaGetLastError() == cudaSuccess ? TBN_OK : TBN_ERR_CUDA;
}

constexpr int kBinCands = 3;
std::atomic<int> g_forced_bin{-1};

}  // namespace

int force_bin_config(int candidate)
{
    if (candidate >= kBinCands) return TBN_ERR_INVALID_ARG;
    g_forced_bin.store(candidate < 0 ? -1 : candidate);
    return TBN_OK;
}

bool bin_tensor_supported(const BinArgs &a)
{
    if (a.q % a.n != 0) return false;                 // the tile must span whole rows
    if (a.n % 32 != 0) return false;                  // rows of weight bits start on word boundaries
    if (a.T >= ((int64_t)1 << 31) - 256) return false;
    if (a.x_bytes && (a.n % 16 != 0 || !a.x_pop)) return false;       // row pitch of the byte form (implied by n % 32 == 0)
    return true;
}

int launch_bin_tensor(const BinArgs &a, int *device_status, cudaStream_t s)
{
    if (!bin_tensor_supported(a)) return TBN_ERR_UNSUPPORTED;
    BinParams p;
    p.x_bits = a.x_bits; p.x_pop = a.x_pop; p.tile = a.tile; p.alpha = a.alpha; p.beta = a.beta; p.bias = a.bias; p.y = a.y;
    p.status = device_status;
    p.T = a.T; p.xw = a.x_row_words; p.n = a.n; p.m = a.m; p.r = (int32_t)(a.q / a.n); p.k = a.k;
    p.nw = a.n / 32; p.k_stages = (a.n + kBinStageK - 1) / kBinStageK;
    p.w_tiles = 0; p.t_tiles = 0;
    p.per_tile = a.alpha_mode == TBN_ALPHA_PER_TILE; p.act = a.act;
    p.y_mode = a.y_dtype == TBN_I32 ? 2 : a.y_dtype == TBN_BF16 ? 1 : 0;
    // 256-token tiles (one accumulator buffer) halve the shared-memory traffic per tile and measured faster wherever
    // they fill the GPU; when they would leave SMs idle, 128-token tiles with two accumulator buffers (the k-fold
    // store loop of one tile runs under the main loop of the next) give twice as many tiles.
    const int sms = bin_sm_count() > 0 ? bin_sm_count() : 148;
    const int64_t tiles256 = (int64_t)((p.r + 127) / 128) * ((a.T + 255) / 256);
    int cand = tiles256 >= sms ? 0 : 1;
    const int forced = g_forced_bin.load(std::memory_order_relaxed);
    if (forced >= 0) cand = forced;
    switch (cand) {
    case 0: return launch_bin_config<256, 3, 1>(p, a.x_bytes, s);
    case 1: return launch_bin_config<128, 5, 2>(p, a.x_bytes, s);
    default: return launch_bin_config<128, 5, 1>(p, a.x_bytes, s);
    }
}

}  // namespace tbn
