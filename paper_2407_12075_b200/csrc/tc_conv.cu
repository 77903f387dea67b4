// Tensor-core forward of a tiled 3x3 convolution on sm_100a (implicit GEMM without im2col duplication).
//
// GEMM view: D[channel][position] = sum over (ci, u, v) of W[channel][(ci,u,v)] * X[ci][position shifted by (u,v)].
// As in the fully-connected kernel the decoded +-1 weights are the tcgen05.mma A operand in tensor memory
// (UMMA M = 128 output channels) and the activations are the B operand in shared memory (UMMA N = output
// positions).  What is new is how the B operand is staged.
//
// Shifted windows instead of im2col.  For each 16-channel K step the producers copy the input patch of the
// CTA tile ONCE into shared memory as [8-channel chunk][patch position][8 channels] (16 bytes per position;
// the un-swizzled K-major UMMA layout with consecutive positions 16 bytes apart).  Because positions are
// linear with the patch row pitch PW, the operand of filter tap (u,v) is the same buffer read from a start
// address advanced by (du*PW + dv) positions: nine MMAs per K step read nine shifted views of one staged
// patch, so shared memory holds each input element once and HBM/L2 traffic is not multiplied by 9.  The MMA
// N index runs over patch positions, halo columns included; outputs at halo positions are discarded by
// the epilogue.  For stride 2 the patch is split into its 4 parity planes (row parity, column parity): all
// inputs of one tap lie in one plane with unit pitch.
//
// The weight bits of 16 consecutive input channels and all 9 taps are 144 consecutive tile bits (row-major
// (Cout, Cin, kh, kw)); the decode warps gather bit ci*9 + tap for each tap into that tap's A block.  The
// K order inside the kernel is therefore (channel group, tap, channel), which the MMA does not care about.
//
// Lanes are output channels (not distinct filters): channel o uses tile row o mod r and alpha[o div r], so
// the k-fold replication of Sec. 4.1 costs no epilogue work here.  (With r < 128, as in the benchmark's
// conv layers, the tensor core would idle on the missing lanes anyway.)
//
// Warp roles (16 warps): 0-5 patch producers, 6 MMA issuer / TMEM owner, 7-10 tile decode, 11-14 epilogue,
// 15 TMA loader of raw patches.
// Two accumulator buffers: the epilogue of one tile overlaps the main loop of the next.  Every wait is
// bounded (see tc_common.cuh).
#include <cstring>

#include "tc_common.cuh"

namespace tbn {

namespace {

// (lo, hi) -> bf16x2 with round-to-nearest-even and negative values replaced by +0: ReLU for free.
__device__ __forceinline__ uint32_t pack_bf16x2_relu(float lo, float hi) {
    uint32_t d;
    asm("cvt.rn.relu.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}

using namespace tc;

constexpr int kProdWarps = 6;           // patch producers
constexpr int kProdThreads = kProdWarps * 32;
constexpr int kMmaWarp = kProdWarps;    // then 4 decode warps, 4 epilogue warps, 1 TMA warp
constexpr int kConvThreads = (kProdWarps + 10) * 32;
constexpr int kTaps = 9;               // 3 x 3
constexpr int kChanPerStage = 16;      // one UMMA K step per tap and stage
constexpr int kNMax = 176;             // max positions per tile: 2 x 176 accumulator columns + 2 x 72 weight columns <= 512
constexpr int kSX = 4;                 // patch stages in shared memory
constexpr int kRS = 3;                 // raw (untransposed) patch stages in shared memory
constexpr int kACols = kTaps * 8;      // 72 columns per decoded-weight stage
constexpr int kABase = 2 * kNMax;      // first weight column
constexpr uint32_t kConvTmemCols = 512;

struct ConvParams {
    const __nv_bfloat16 *x;
    void *y;
    const uint32_t *tile;
    const float *alpha;
    const float *bias;
    int *status;
    int64_t n_words;
    int32_t Nb, Cin, H, W, Ho, Wo, m, r, k, n;   // n = Cin * 9
    int32_t stride, pad;
    int32_t planes;            // stride * stride
    int32_t du_min, dv_min;    // smallest plane-row / plane-column offset over the taps
    int32_t PW;                // patch pitch (positions per patch row) = Wo + column offset range
    int32_t PHt;               // patch rows per image slot = R + row offset range
    int32_t R;                 // output rows per image slot
    int32_t G;                 // image slots per tile (G > 1 only when R == Ho)
    int32_t bands;             // row bands per image = ceil(Ho / R)
    int32_t n_pos;             // UMMA N: positions per tile, a multiple of 16, <= kNMax
    int32_t slot_pos;          // PHt * PW
    int32_t buf_pos;           // positions held per (plane, chunk) buffer >= n_pos + largest tap offset
    int32_t wide;              // 1: W % 8 == 0, raw patches arrive by TMA
    int32_t raw_rows;          // input rows per image slot and stage = stride * PHt
    uint32_t raw_slot_bytes, raw_stage_bytes;   // 16 channels x raw_rows x W bf16 (per slot / per stage)
    uint32_t magic_rows, magic_gw;   // floor(2^32 / d) + 1 for d = raw_rows, W / 8: x / d == umulhi(x, magic) for small x
    int32_t tap_plane[kTaps];  // parity plane read by tap t
    int32_t tap_off[kTaps];    // start offset (positions) of tap t inside its plane
    int32_t m_blocks, s_tiles; // 128-lane accumulator blocks, spatial tiles
    int32_t rep;               // 128-channel output blocks written from one accumulator block (see plan_conv)
    int32_t k_stages;          // Cin / 16
    int per_tile, act, y_bf16;
};

struct ConvControl {
    uint64_t x_full[kSX], x_empty[kSX];
    uint64_t a_full[2], a_empty[2];
    uint64_t d_full[2], d_empty[2];
    uint64_t raw_full[kRS], raw_empty[kRS];
    uint32_t tmem_base;
    int abort_flag;
};
constexpr int kCtlBytes = (sizeof(ConvControl) + 15) / 16 * 16;

__global__ void __launch_bounds__(kConvThreads, 1)
tc_conv3x3_kernel(const __grid_constant__ CUtensorMap x_map, const ConvParams p)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    uint8_t *smem = smem_raw + ((1024u - (raw & 1023u)) & 1023u);
    const uint32_t stage_bytes = (uint32_t)p.planes * 2u * (uint32_t)p.buf_pos * 16u;
    ConvControl *ctl = reinterpret_cast<ConvControl *>(smem + kSX * stage_bytes);
    const uint32_t stage0 = smem_u32(smem);
    const uint32_t raw_off = (kSX * stage_bytes + kCtlBytes + 127u) & ~127u;   // raw ring, 128-byte aligned
    volatile int *abort_flag = &ctl->abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int bid = blockIdx.x;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kSX; ++s) { mbar_init(smem_u32(&ctl->x_full[s]), kProdThreads); mbar_init(smem_u32(&ctl->x_empty[s]), 1); }
        for (int s = 0; s < 2; ++s) {
            mbar_init(smem_u32(&ctl->a_full[s]), 128); mbar_init(smem_u32(&ctl->a_empty[s]), 1);
            mbar_init(smem_u32(&ctl->d_full[s]), 1);   mbar_init(smem_u32(&ctl->d_empty[s]), 128);
        }
        for (int s = 0; s < kRS; ++s) { mbar_init(smem_u32(&ctl->raw_full[s]), 1); mbar_init(smem_u32(&ctl->raw_empty[s]), kProdThreads); }
        ctl->abort_flag = 0;
        fence_barrier_init();
        fence_proxy_async();
    }
    if (warp == kMmaWarp) {
        tmem_alloc(smem_u32(&ctl->tmem_base), kConvTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;

    const int32_t n_tiles = p.m_blocks * p.s_tiles;
    bool ok = true;

    if (warp < kProdWarps) {
        // ---------------- patch producers: -> [plane][chunk][position][8 channels] ----------------
        // Wide rows (W % 8 == 0): a TMA warp brings the raw NCHW patch of the stage ([16 channels][rows][W],
        // rows outside the image and images outside the batch zero-filled) into a shared-memory ring, so HBM
        // latency is hidden by the ring depth.  These four warps transpose shared memory -> shared memory: a
        // unit is 8 consecutive pixels of one raw row for 8 channels -- eight 16-byte loads, an 8 x 8
        // transpose of 16-bit values in registers (byte permutes), eight 16-byte stores.  Patch positions that
        // no pixel maps to (the zero padding left and right) are zeroed once, before the first stage.
        // Other widths: gather straight from global memory with 2-byte loads.
        const int tid = threadIdx.x;                       // 0..kProdThreads-1
        const int32_t fill_pos = p.G * p.slot_pos;
        const int32_t items = p.planes * 2 * fill_pos;
        const int64_t plane_elems = (int64_t)p.H * p.W;
        const unsigned short *xs = reinterpret_cast<const unsigned short *>(p.x);
        if (p.wide) {
            for (uint32_t off = tid * 16u; off < kSX * stage_bytes; off += kProdThreads * 16u) sts_v4(stage0 + off, 0u, 0u, 0u, 0u);
        }
        Pipe px, pr;
        for (int32_t tile = bid; tile < n_tiles && ok; tile += gridDim.x) {
            const int32_t st = tile / p.m_blocks;
            const int32_t img0 = p.G > 1 ? st * p.G : st / p.bands;
            const int32_t oh0 = p.G > 1 ? 0 : (st % p.bands) * p.R;
            for (int32_t ks = 0; ks < p.k_stages && ok; ++ks) {
                ok = wait_bar(smem_u32(&ctl->x_empty[px.stage]), px.phase ^ 1u, abort_flag, p.status,
                              (1 << 24) | (px.stage << 16) | (bid & 0xffff));
                if (!ok) break;
                uint8_t *stage = smem + px.stage * stage_bytes;
                if (p.wide) {
                    ok = wait_bar(smem_u32(&ctl->raw_full[pr.stage]), pr.phase, abort_flag, p.status,
                                  (7 << 24) | (pr.stage << 16) | (bid & 0xffff));
                    if (!ok) break;
                    const uint32_t raw_addr = stage0 + raw_off + pr.stage * p.raw_stage_bytes;   // shared addresses
                    const uint32_t stage_addr = stage0 + px.stage * stage_bytes;
                    const uint32_t ch_bytes = (uint32_t)(p.raw_rows * p.W) * 2u;                 // between channels
                    const uint32_t chunk_bytes = (uint32_t)p.buf_pos * 16u;                      // between (plane, chunk) buffers
                    const int32_t gw = p.W >> 3;
                    const int32_t units = 2 * p.G * gw * p.raw_rows;
                    const int32_t ssh = p.stride - 1;          // stride is 1 or 2: x / stride == x >> ssh, x % stride == x & ssh
                    for (int32_t u = tid; u < units; u += kProdThreads) {
                        // unit -> (chunk, image slot, raw row, pixel group); the pixel group varies fastest across
                        // lanes, so a warp reads 512 contiguous bytes of the raw patch per load (no bank conflicts)
                        int32_t t = gw == 1 ? u : (int32_t)__umulhi((uint32_t)u, p.magic_gw);
                        const int32_t gx = u - t * gw;
                        const int32_t t2 = (int32_t)__umulhi((uint32_t)t, p.magic_rows);
                        const int32_t rr = t - t2 * p.raw_rows;
                        const int32_t chunk = t2 >= p.G ? 1 : 0;
                        const int32_t g = t2 - chunk * p.G;
                        const uint32_t src = raw_addr + (uint32_t)(((g * 16 + chunk * 8) * p.raw_rows + rr) * p.W + gx * 8) * 2u;
                        uint32_t rg[8][4];
#pragma unroll
                        for (int c = 0; c < 8; ++c) {
                            const uint4 q4 = lds_v4(src + c * ch_bytes);
                            rg[c][0] = q4.x; rg[c][1] = q4.y; rg[c][2] = q4.z; rg[c][3] = q4.w;
                        }
                        const int32_t py = rr & ssh, a_l = rr >> ssh;
                        // destination of pixel e: plane (py, iw & ssh), column ((iw >> ssh) - dv_min)
                        const uint32_t row_dst = stage_addr + (uint32_t)chunk * chunk_bytes +
                                                 (uint32_t)(g * p.slot_pos + a_l * p.PW) * 16u +
                                                 (uint32_t)(py * p.stride * 2) * chunk_bytes;
                        const int32_t b0 = ((gx * 8) >> ssh) - p.dv_min;     // column of pixel 0 (gx*8 is even)
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            const int32_t pxx = e & ssh;
                            const int32_t b_l = b0 + (e >> ssh);
                            if (b_l < 0 || b_l >= p.PW) continue;
                            const uint32_t sel = (e & 1) ? 0x7632u : 0x5410u;      // high or low halves of the pixel pair
                            sts_v4(row_dst + (uint32_t)(pxx * 2) * chunk_bytes + (uint32_t)b_l * 16u,
                                   __byte_perm(rg[0][e >> 1], rg[1][e >> 1], sel), __byte_perm(rg[2][e >> 1], rg[3][e >> 1], sel),
                                   __byte_perm(rg[4][e >> 1], rg[5][e >> 1], sel), __byte_perm(rg[6][e >> 1], rg[7][e >> 1], sel));
                        }
                    }
                    mbar_arrive(smem_u32(&ctl->raw_empty[pr.stage]));   // raw stage consumed by this thread
                    pr.advance(kRS);
                } else {
                    for (int32_t id = tid; id < items; id += kProdThreads) {
                        const int32_t pos = id % fill_pos;
                        const int32_t pc = id / fill_pos;
                        const int32_t chunk = pc & 1, plane = pc >> 1;
                        const int32_t g = pos / p.slot_pos;
                        const int32_t rem = pos - g * p.slot_pos;
                        const int32_t a_l = rem / p.PW, b_l = rem - a_l * p.PW;
                        const int32_t py = plane / p.stride, pxx = plane - py * p.stride;
                        const int32_t ih = p.stride * (oh0 + a_l + p.du_min) + py;
                        const int32_t iw = p.stride * (b_l + p.dv_min) + pxx;
                        const int32_t img = img0 + g;
                        uint32_t v[4] = {0u, 0u, 0u, 0u};
                        if (img < p.Nb && ih >= 0 && ih < p.H && iw >= 0 && iw < p.W) {
                            const unsigned short *src =
                                xs + ((int64_t)img * p.Cin + ks * kChanPerStage + chunk * 8) * plane_elems + (int64_t)ih * p.W + iw;
    #pragma unroll
                            for (int c = 0; c < 4; ++c) {
                                const uint32_t lo = __ldg(src + (2 * c) * plane_elems);
                                const uint32_t hi = __ldg(src + (2 * c + 1) * plane_elems);
                                v[c] = lo | (hi << 16);
                            }
                        }
                        *reinterpret_cast<uint4 *>(stage + ((size_t)(plane * 2 + chunk) * p.buf_pos + pos) * 16) =
                            make_uint4(v[0], v[1], v[2], v[3]);
                    }
                }
                fence_proxy_async();                       // generic-proxy stores -> visible to the tensor core
                mbar_arrive(smem_u32(&ctl->x_full[px.stage]));
                px.advance(kSX);
            }
        }
    } else if (warp == kMmaWarp) {
        // ---------------- MMA issuer: 9 shifted-window MMAs per 16-channel stage ----------------
        {
            // all 32 lanes run the loop in lockstep, one elected lane performs each MMA and commit (see tc_mma_ts_elect)
            const uint32_t tmem_u = __shfl_sync(0xffffffffu, tmem_base, 0);
            const uint32_t leader = elect_one();
            Pipe px, pa, pd;
            bool ready = false;
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.n_pos >> 3) << 17) | (8u << 24);
            // un-swizzled K-major descriptor: stride offset 128 bytes (next 8 positions), leading offset =
            // distance between the two 8-channel chunks, version 1
            const uint32_t desc_hi = 8u | (1u << 14);
            const uint32_t lbo = (uint32_t)p.buf_pos << 16;
            uint32_t tap_disp[kTaps];                   // start of tap t's window inside a stage, in 16-byte units
#pragma unroll
            for (int t = 0; t < kTaps; ++t) tap_disp[t] = (uint32_t)(p.tap_plane[t] * 2 * p.buf_pos + p.tap_off[t]);
            for (int32_t tile = bid; tile < n_tiles && ok; tile += gridDim.x) {
                ok = wait_bar(smem_u32(&ctl->d_empty[pd.stage]), pd.phase ^ 1u, abort_flag, p.status,
                              (2 << 24) | (bid & 0xffff));
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_addr = tmem_u + pd.stage * kNMax;
                for (int32_t ks = 0; ks < p.k_stages; ++ks) {
                    if (!ready) {
                        ok = wait_bar(smem_u32(&ctl->x_full[px.stage]), px.phase, abort_flag, p.status,
                                      (3 << 24) | (px.stage << 16) | (bid & 0xffff)) &&
                             wait_bar(smem_u32(&ctl->a_full[pa.stage]), pa.phase, abort_flag, p.status,
                                      (4 << 24) | (pa.stage << 16) | (bid & 0xffff));
                        if (!ok) break;
                    }
                    tc_fence_after();
                    const uint32_t b_base = ((stage0 + px.stage * stage_bytes) & 0x3FFFFu) >> 4;   // 16-byte units
                    const uint32_t a_addr = tmem_u + kABase + pa.stage * kACols;
                    Pipe nx = px, na = pa;
                    nx.advance(kSX);
                    na.advance(2);
#pragma unroll
                    for (int t = 0; t < kTaps; ++t) {
                        const uint32_t b_lo = (b_base + tap_disp[t]) | lbo;
                        tc_mma_ts_elect(d_addr, a_addr + t * 8, b_lo, desc_hi, idesc, t > 0 ? 1u : (uint32_t)(ks > 0), leader);
                        if (t == 4)
                            ready = __all_sync(0xffffffffu, mbar_test_wait(smem_u32(&ctl->x_full[nx.stage]), nx.phase) &&
                                                                mbar_test_wait(smem_u32(&ctl->a_full[na.stage]), na.phase)) != 0;
                    }
                    tc_commit_elect(smem_u32(&ctl->x_empty[px.stage]), leader);
                    tc_commit_elect(smem_u32(&ctl->a_empty[pa.stage]), leader);
                    if (ks == p.k_stages - 1) tc_commit_elect(smem_u32(&ctl->d_full[pd.stage]), leader);
                    px = nx;
                    pa = na;
                }
                pd.advance(2);
            }
        }
        __syncwarp();
    } else if (warp < kMmaWarp + 5) {
        // ---------------- tile decode: 144 bits (16 channels x 9 taps) -> nine 128 x 16 A blocks ----------------
        const int qd = warp & 3;
        const int L = qd * 32 + lane;
        const uint32_t lane_base = (uint32_t)(qd * 32) << 16;
        const int64_t last_word = p.n_words - 1;
        Pipe pa;
        for (int32_t tile = bid; tile < n_tiles && ok; tile += gridDim.x) {
            const int32_t o = min((tile % p.m_blocks) * p.rep * 128 + L, p.m - 1);   // channels past the end are never stored
            const int64_t row_bit = (int64_t)(o % p.r) * p.n;                  // tile row of this channel
            uint32_t w[6];
            {
                const int64_t wi = row_bit >> 5;
#pragma unroll
                for (int i = 0; i < 6; ++i) w[i] = __ldg(p.tile + min(wi + i, last_word));
            }
            for (int32_t ks = 0; ks < p.k_stages && ok; ++ks) {
                const int64_t off = row_bit + (int64_t)ks * (kChanPerStage * kTaps);
                const uint32_t sh = (uint32_t)off & 31u;
                uint32_t b[5];
#pragma unroll
                for (int i = 0; i < 5; ++i) b[i] = __funnelshift_r(w[i], w[i + 1], sh);
                if (ks + 1 < p.k_stages) {                       // next stage's words, in flight during the decode
                    const int64_t wi = (off + kChanPerStage * kTaps) >> 5;
#pragma unroll
                    for (int i = 0; i < 6; ++i) w[i] = __ldg(p.tile + min(wi + i, last_word));
                }
                // decode into registers first: the ALU work overlaps the MMAs that still read the stage's slot, and only
                // the nine stores sit between "slot free" and "slot full"
                uint32_t v[kTaps][8];
#pragma unroll
                for (int t = 0; t < kTaps; ++t) {
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        // channels 2i and 2i+1 of the stage at tap t: bits (2i)*9 + t and (2i+1)*9 + t
                        const int pe = (2 * i) * kTaps + t, po = pe + kTaps;
                        const uint32_t be = (b[pe >> 5] >> (pe & 31)) & 1u;
                        const uint32_t bo = (b[po >> 5] >> (po & 31)) & 1u;
                        v[t][i] = ((be << 15) | (bo << 31)) ^ 0xBF80BF80u;    // bit 1 -> +1.0, bit 0 -> -1.0
                    }
                }
                ok = wait_bar(smem_u32(&ctl->a_empty[pa.stage]), pa.phase ^ 1u, abort_flag, p.status,
                              (5 << 24) | (pa.stage << 16) | (bid & 0xffff));
                if (!ok) break;
                tc_fence_after();
                const uint32_t a_addr = tmem_base + lane_base + kABase + pa.stage * kACols;
#pragma unroll
                for (int t = 0; t < kTaps; ++t) tmem_st_32x8(a_addr + t * 8, v[t]);
                tc_wait_st();
                tc_fence_before();
                mbar_arrive(smem_u32(&ctl->a_full[pa.stage]));
                pa.advance(2);
            }
        }
    } else if (warp < kMmaWarp + 9) {
        // ---------------- epilogue: thread = output channel, 32 patch positions per TMEM load ----------------
        const int qd = warp & 3;
        const int L = qd * 32 + lane;
        const uint32_t lane_base = (uint32_t)(qd * 32) << 16;
        Pipe pd;
        const int n_chunks = (p.n_pos + 31) / 32;
        const int64_t out_plane = (int64_t)p.Ho * p.Wo;
        // bf16 outputs whose rows are whole 16-byte pieces are stored straight from the accumulator rows
        const bool rows_direct = p.y_bf16 && (p.Wo % 8 == 0);
        for (int32_t tile = bid; tile < n_tiles && ok; tile += gridDim.x) {
            const int32_t st = tile / p.m_blocks;
            const int32_t img0 = p.G > 1 ? st * p.G : st / p.bands;
            const int32_t oh0 = p.G > 1 ? 0 : (st % p.bands) * p.R;
            // this thread's channel, scale and bias of the first pass are fetched before the wait for the accumulator,
            // those of the next pass at the start of each pass: the loads stay off the critical path
            int32_t o_nx = (tile % p.m_blocks) * p.rep * 128 + L;
            bool valid_nx = o_nx < p.m;
            float al_nx = valid_nx ? (p.per_tile ? __ldg(p.alpha + o_nx / p.r) : __ldg(p.alpha)) : 0.0f;
            float bs_nx = (valid_nx && p.bias) ? __ldg(p.bias + o_nx) : 0.0f;
            ok = wait_bar(smem_u32(&ctl->d_full[pd.stage]), pd.phase, abort_flag, p.status, (6 << 24) | (bid & 0xffff));
            if (!ok) break;
            tc_fence_after();
            // one pass per channel block that shares this accumulator; the last pass hands the accumulator back
#pragma unroll 1
            for (int32_t rb = 0; rb < p.rep; ++rb) {
            const bool last_pass = rb == p.rep - 1;
            const int32_t o = o_nx;
            const bool ch_valid = valid_nx;
            const float al = al_nx, bs = bs_nx;
            if (!last_pass) {
                o_nx = o + 128;
                valid_nx = o_nx < p.m;
                al_nx = valid_nx ? (p.per_tile ? __ldg(p.alpha + o_nx / p.r) : __ldg(p.alpha)) : 0.0f;
                bs_nx = (valid_nx && p.bias) ? __ldg(p.bias + o_nx) : 0.0f;
            }
            if (rows_direct && ((p.Wo & 15) == 0 || p.Wo == 8)) {
                // Rows made of whole 16-pixel items (32 bytes of bf16): software-pipelined.  The tensor-memory load of
                // item i+1 is issued before item i is scaled, converted and stored, so its latency is off the path;
                // the accumulator goes back to the MMA warp right after the last load.  Items are walked with
                // counters (image, row, item in row): no divisions in this single-warp instruction stream.
                // With 8-pixel rows an item is two consecutive rows (contiguous in NCHW); the unit "row" below is then
                // a row pair and a pair without a second row is stored as 16 bytes.
                const bool pair_rows = p.Wo == 8;
                const int32_t real_rows = min(p.R, p.Ho - oh0);
                const int32_t rows_here = pair_rows ? (real_rows + 1) >> 1 : real_rows;
                const int32_t per_row = pair_rows ? 1 : p.Wo >> 4;
                const int32_t row_cols = pair_rows ? 2 * p.PW : p.PW;       // accumulator columns per unit row
                const int32_t row_elems = pair_rows ? 16 : p.Wo;            // output elements per unit row
                const int32_t imgs = min(p.G, p.Nb - img0);
                const int32_t n_items = imgs * rows_here * per_row;
                const int64_t img_pitch = (int64_t)p.m * out_plane;
                __nv_bfloat16 *dst = static_cast<__nv_bfloat16 *>(p.y) +
                                     ((int64_t)img0 * p.m + (ch_valid ? o : 0)) * out_plane + (int64_t)oh0 * p.Wo;
                uint32_t col = tmem_base + lane_base + pd.stage * kNMax;     // column of the item being loaded
                int32_t ld_pc = 0, ld_oh = 0, ld_g = 0;                      // its coordinates
                int32_t st_pc = 0, st_oh = 0;                                // coordinates of the item being stored
                uint32_t cur[16], nxt[16];
                auto load_item = [&](uint32_t c, int32_t unit_row, uint32_t (&dstv)[16]) {
                    if (!pair_rows) {
                        tmem_ld_32x16(c, dstv);
                    } else {
                        uint32_t lo[8], hi[8];
                        tmem_ld_32x8(c, lo);
                        // a missing second row re-reads the first (in range); it is not stored
                        tmem_ld_32x8(c + (2 * unit_row + 1 < real_rows ? (uint32_t)p.PW : 0u), hi);
#pragma unroll
                        for (int i = 0; i < 8; ++i) { dstv[i] = lo[i]; dstv[i + 8] = hi[i]; }
                    }
                };
                __syncwarp();
                if (n_items > 0) load_item(col, 0, cur);
                tc_wait_ld();
                for (int32_t it = 0; it < n_items; ++it) {
                    const bool more = it + 1 < n_items;
                    if (more) {                                            // advance the load cursor and issue the next load
                        if (++ld_pc == per_row) {
                            ld_pc = 0;
                            if (++ld_oh == rows_here) { ld_oh = 0; ++ld_g; }
                        }
                        col = tmem_base + lane_base + pd.stage * kNMax + ld_g * p.slot_pos + ld_oh * row_cols + ld_pc * 16;
                        __syncwarp();
                        load_item(col, ld_oh, nxt);
                    } else if (last_pass) {                                // everything is in registers: hand the accumulator back
                        tc_fence_before();
                        mbar_arrive(smem_u32(&ctl->d_empty[pd.stage]));
                    }
                    uint32_t pk[8];
                    if (p.act == TBN_ACT_RELU) {
#pragma unroll
                        for (int i = 0; i < 8; ++i)     // the conversion clamps negative values to zero: no separate max
                            pk[i] = pack_bf16x2_relu(fmaf(al, __uint_as_float(cur[2 * i]), bs),
                                                     fmaf(al, __uint_as_float(cur[2 * i + 1]), bs));
                    } else if (p.act == TBN_ACT_GELU) {
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            const float v0 = gelu_tanh_bf16(fmaf(al, __uint_as_float(cur[2 * i]), bs));
                            const float v1 = gelu_tanh_bf16(fmaf(al, __uint_as_float(cur[2 * i + 1]), bs));
                            const __nv_bfloat162 h = __floats2bfloat162_rn(v0, v1);
                            pk[i] = *reinterpret_cast<const uint32_t *>(&h);
                        }
                    } else {
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            const __nv_bfloat162 h = __floats2bfloat162_rn(fmaf(al, __uint_as_float(cur[2 * i]), bs),
                                                                           fmaf(al, __uint_as_float(cur[2 * i + 1]), bs));
                            pk[i] = *reinterpret_cast<const uint32_t *>(&h);
                        }
                    }
                    if (ch_valid) {
                        __nv_bfloat16 *q = dst + st_oh * row_elems + st_pc * 16;
                        const bool both = !pair_rows || 2 * st_oh + 1 < real_rows;
                        if (both && (reinterpret_cast<uintptr_t>(q) & 31u) == 0) {
                            st_global_v8(q, pk);
                        } else {                                           // odd image height: 16-byte aligned only
                            *reinterpret_cast<uint4 *>(q) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                            if (both) *reinterpret_cast<uint4 *>(q + 8) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
                        }
                    }
                    if (++st_pc == per_row) {
                        st_pc = 0;
                        if (++st_oh == rows_here) { st_oh = 0; dst += img_pitch; }
                    }
                    if (more) {
                        tc_wait_ld();
#pragma unroll
                        for (int i = 0; i < 16; ++i) cur[i] = nxt[i];
                    }
                }
                if (n_items <= 0 && last_pass) {
                    tc_fence_before();
                    mbar_arrive(smem_u32(&ctl->d_empty[pd.stage]));
                }
                continue;
            }
            if (rows_direct) {
                // One TMEM load per output row piece: 8 consecutive accumulator columns starting at the row's first
                // position are 8 consecutive output pixels of this thread's channel -> one 16-byte store (two
                // pieces that share a 32-byte sector go out as one 32-byte store).  All loops are warp-uniform.
                const int32_t rows_here = min(p.R, p.Ho - oh0);
                const int32_t pieces = p.Wo >> 3;
                for (int32_t g = 0; g < p.G && img0 + g < p.Nb; ++g) {
                    __nv_bfloat16 *img_dst = static_cast<__nv_bfloat16 *>(p.y) +
                                             ((int64_t)(img0 + g) * p.m + (ch_valid ? o : 0)) * out_plane + (int64_t)oh0 * p.Wo;
                    for (int32_t oh = 0; oh < rows_here; ++oh) {
                        const uint32_t col0 = tmem_base + lane_base + pd.stage * kNMax + g * p.slot_pos + oh * p.PW;
                        __nv_bfloat16 *row_dst = img_dst + oh * p.Wo;
                        for (int32_t pc = 0; pc < pieces; pc += 2) {
                            uint32_t v[16];
                            const bool two = pc + 1 < pieces;
                            __syncwarp();
                            if (two) {
                                tmem_ld_32x16(col0 + pc * 8, v);
                            } else {
                                uint32_t v8[8];
                                tmem_ld_32x8(col0 + pc * 8, v8);
#pragma unroll
                                for (int i = 0; i < 8; ++i) { v[i] = v8[i]; v[i + 8] = 0u; }
                            }
                            tc_wait_ld();
                            uint32_t pk[8];
#pragma unroll
                            for (int i = 0; i < 8; ++i) {
                                float v0 = fmaf(al, __uint_as_float(v[2 * i]), bs), v1 = fmaf(al, __uint_as_float(v[2 * i + 1]), bs);
                                if (p.act == TBN_ACT_RELU) { v0 = fmaxf(v0, 0.0f); v1 = fmaxf(v1, 0.0f); }
                                else if (p.act == TBN_ACT_GELU) { v0 = gelu_tanh_bf16(v0); v1 = gelu_tanh_bf16(v1); }
                                const __nv_bfloat162 h = __floats2bfloat162_rn(v0, v1);
                                pk[i] = *reinterpret_cast<const uint32_t *>(&h);
                            }
                            if (ch_valid) {
                                __nv_bfloat16 *dst = row_dst + pc * 8;
                                if (two && (((uintptr_t)dst) & 31u) == 0) {
                                    st_global_v8(dst, pk);
                                } else {
                                    *reinterpret_cast<uint4 *>(dst) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                                    if (two) *reinterpret_cast<uint4 *>(dst + 8) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
                                }
                            }
                        }
                    }
                }
                if (last_pass) {
                    tc_fence_before();
                    mbar_arrive(smem_u32(&ctl->d_empty[pd.stage]));  // accumulator fully read
                }
                continue;
            }
            int32_t g = 0, oh = 0, ow = 0;                     // patch coordinates of the next position
#pragma unroll 1
            for (int ch = 0; ch < n_chunks; ++ch) {
                __syncwarp();
                uint32_t v[32];
                tmem_ld_32x32(tmem_base + lane_base + pd.stage * kNMax + ch * 32, v);
                tc_wait_ld();
                if (ch == n_chunks - 1 && last_pass) {           // accumulator fully read: hand it back early
                    tc_fence_before();
                    mbar_arrive(smem_u32(&ctl->d_empty[pd.stage]));
                }
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    const int32_t img = img0 + g, row = oh0 + oh;
                    if (ch_valid && g < p.G && img < p.Nb && oh < p.R && row < p.Ho && ow < p.Wo) {
                        const float val = apply_act(fmaf(al, __uint_as_float(v[i]), bs), p.act);
                        const int64_t yi = ((int64_t)img * p.m + o) * out_plane + (int64_t)row * p.Wo + ow;
                        if (p.y_bf16) static_cast<__nv_bfloat16 *>(p.y)[yi] = __float2bfloat16_rn(val);
                        else static_cast<float *>(p.y)[yi] = val;
                    }
                    if (++ow == p.PW) { ow = 0; if (++oh == p.PHt) { oh = 0; ++g; } }
                }
            }
            }   // channel blocks of this accumulator
            pd.advance(2);
        }
    } else {
        // ---------------- TMA loader (last warp): raw input patches into the shared-memory ring ----------------
        if (p.wide) {
            Pipe pr;
            uint32_t issued_mask = 0, issued_phase = 0;
            for (int32_t tile = bid; tile < n_tiles && ok; tile += gridDim.x) {
                const int32_t st = tile / p.m_blocks;
                const int32_t img0 = p.G > 1 ? st * p.G : st / p.bands;
                const int32_t oh0 = p.G > 1 ? 0 : (st % p.bands) * p.R;
                const int32_t ih_lo = p.stride * (oh0 + p.du_min);     // may be negative: those rows are zero-filled
                for (int32_t ks = 0; ks < p.k_stages && ok; ++ks) {
                    ok = wait_bar(smem_u32(&ctl->raw_empty[pr.stage]), pr.phase ^ 1u, abort_flag, p.status,
                                  (8 << 24) | (pr.stage << 16) | (bid & 0xffff));
                    if (!ok) break;
                    if (lane == 0) {
                        const uint32_t bar = smem_u32(&ctl->raw_full[pr.stage]);
                        mbar_arrive_expect_tx(bar, p.raw_stage_bytes);
                        for (int32_t g = 0; g < p.G; ++g)                // images past the batch are zero-filled
                            tma_load_4d(stage0 + raw_off + pr.stage * p.raw_stage_bytes + g * p.raw_slot_bytes, &x_map, 0,
                                        ih_lo, ks * kChanPerStage, img0 + g, bar);
                    }
                    issued_mask |= 1u << pr.stage;
                    issued_phase = (issued_phase & ~(1u << pr.stage)) | (pr.phase << pr.stage);
                    __syncwarp();
                    pr.advance(kRS);
                }
            }
            if (!ok) {   // let copies in flight land before the CTA's shared memory goes away
                for (int s = 0; s < kRS; ++s)
                    if (issued_mask & (1u << s)) drain_wait(smem_u32(&ctl->raw_full[s]), (issued_phase >> s) & 1u);
            }
        }
    }

    // ---------------- teardown ----------------
    if (warp == kMmaWarp && *abort_flag) {
        tc_commit_elect(smem_u32(&ctl->x_empty[0]), elect_one());     // by the lane that issued the MMAs
        __syncwarp();
        drain_wait(smem_u32(&ctl->x_empty[0]), 0);
        drain_wait(smem_u32(&ctl->x_empty[0]), 1);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kConvTmemCols);
    }
}

size_t conv_smem_bytes(const ConvParams &p)
{
    size_t b = (size_t)kSX * p.planes * 2 * p.buf_pos * 16 + kCtlBytes + 128;
    if (p.wide) b += (size_t)kRS * p.raw_stage_bytes;
    return b + 1024;
}

inline int floor_div(int a, int b) { return (a >= 0) ? a / b : -((-a + b - 1) / b); }

int conv_sm_count()
{
    static int cache[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    if (!cache[dev]) cudaDeviceGetAttribute(&cache[dev], cudaDevAttrMultiProcessorCount, dev);
    return cache[dev];
}

// Geometry of the shifted-window staging for one call; false when the shape does not fit this kernel.
bool plan_conv(const LayerArgs &a, ConvParams &p)
{
    if (!a.is_conv || a.kh != 3 || a.kw != 3) return false;
    if (a.stride != 1 && a.stride != 2) return false;
    if (a.pad < 0 || a.pad > 2) return false;
    if (a.q % a.n != 0) return false;                 // the tile must span whole filters
    if (a.Cin % kChanPerStage != 0) return false;
    if (a.Nb <= 0 || a.Ho <= 0 || a.Wo <= 0) return false;
    const int s = a.stride;
    int du[3], py[3];
    int dmin = 1 << 30, dmax = -(1 << 30);
    for (int u = 0; u < 3; ++u) {
        du[u] = floor_div(u - a.pad, s);
        py[u] = (u - a.pad) - s * du[u];
        dmin = du[u] < dmin ? du[u] : dmin;
        dmax = du[u] > dmax ? du[u] : dmax;
    }
    const int range = dmax - dmin;                    // same for rows and columns (square filter, same padding)
    p.stride = s; p.pad = a.pad; p.planes = s * s;
    p.du_min = dmin; p.dv_min = dmin;
    p.PW = a.Wo + range;
    if (p.PW > kNMax) return false;
    const int slot_full = (a.Ho + range) * p.PW;
    // Lane L of channel block b holds filter (128 b + L) mod r.  When r divides 128 and the channel count is a whole
    // number of blocks, every block has the same filters on the same lanes, hence the same accumulator: it is
    // computed once and the epilogue writes it to all the blocks with their own alphas and biases (Sec. 4.1's
    // replicated channels; with fewer than 128 distinct filters the tensor core has no smaller shape to offer,
    // but it need not repeat whole blocks).
    {
        const int64_t r = a.q / a.n;
        p.rep = (a.m > 128 && a.m % 128 == 0 && r <= 128 && 128 % r == 0) ? a.m / 128 : 1;
    }
    p.m_blocks = (a.m + 127) / 128 / p.rep;
    if ((a.Ho * p.PW) <= kNMax) {                     // whole images: possibly several per tile
        p.R = a.Ho;
        p.PHt = a.Ho + range;
        int g_max = (kNMax - p.R * p.PW) / slot_full + 1;
        if (g_max > a.Nb) g_max = a.Nb;
        // Images per tile.  The main loop of a tile costs the same whatever its width (the MMA count is fixed by the
        // input channels and an MMA takes ~112 cycles for any N <= 256) while its epilogue grows with the images it
        // holds, so more images per tile pay only while they save a whole round of tiles over the SMs.
        const int sms = conv_sm_count() > 0 ? conv_sm_count() : 148;
        const double main_cycles = (double)(a.Cin / kChanPerStage) * 9.0 * 112.0 + 1500.0;
        const double image_cycles = 350.0 * ((a.Ho * a.Wo + 15) / 16) * p.rep;
        double best = 0.0;
        p.G = 1;
        for (int g = 1; g <= g_max; ++g) {
            const int64_t tiles = (int64_t)((a.Nb + g - 1) / g) * p.m_blocks;
            const double cost = (double)((tiles + sms - 1) / sms) * (main_cycles + g * image_cycles);
            if (g == 1 || cost <= best) { best = cost; p.G = g; }
        }
        p.bands = 1;
    } else {                                          // row bands of one image
        p.G = 1;
        int R = kNMax / p.PW;
        p.bands = (a.Ho + R - 1) / R;
        p.R = (a.Ho + p.bands - 1) / p.bands;
        p.PHt = p.R + range;
    }
    p.slot_pos = p.PHt * p.PW;
    const int used = (p.G - 1) * p.slot_pos + p.R * p.PW;
    p.n_pos = (used + 15) / 16 * 16;
    if (p.n_pos > kNMax || p.n_pos < 16) return false;
    const int max_off = range * p.PW + range;
    int need = p.n_pos + max_off;
    if (need < p.G * p.slot_pos) need = p.G * p.slot_pos;
    p.buf_pos = (need + 7) / 8 * 8 + 2;     // = 2 mod 8: the (plane, chunk) buffers start 32 bytes apart modulo 128,
                                            // which spreads the producers' 16-byte stores over the banks
    for (int u = 0; u < 3; ++u)
        for (int v = 0; v < 3; ++v) {
            p.tap_plane[u * 3 + v] = py[u] * s + py[v];
            p.tap_off[u * 3 + v] = (du[u] - dmin) * p.PW + (du[v] - dmin);
        }
    p.s_tiles = p.G > 1 ? (a.Nb + p.G - 1) / p.G : a.Nb * p.bands;
    p.k_stages = a.Cin / kChanPerStage;
    p.raw_rows = s * p.PHt;
    p.raw_slot_bytes = (uint32_t)(kChanPerStage * p.raw_rows * a.Wd * 2);
    p.raw_stage_bytes = p.raw_slot_bytes * (uint32_t)p.G;           // a multiple of 256 when W % 8 == 0
    p.wide = (a.Wd % 8 == 0 && a.Wd <= 256 && p.raw_rows <= 256) ? 1 : 0;
    p.magic_rows = (uint32_t)(0x100000000ull / (uint32_t)p.raw_rows) + 1u;
    p.magic_gw = (a.Wd >= 16) ? (uint32_t)(0x100000000ull / (uint32_t)(a.Wd / 8)) + 1u : 0u;   // W / 8 == 1 needs no division
    if (p.wide && conv_smem_bytes(p) > 227 * 1024) p.wide = 0;      // no room for the raw ring: gather from global
    if (conv_smem_bytes(p) > 227 * 1024) return false;
    return true;
}

}  // namespace

bool tensor_conv_supported(const LayerArgs &a)
{
    ConvParams p;
    return plan_conv(a, p);
}

int launch_tensor_conv(const LayerArgs &a, int *device_status, cudaStream_t s)
{
    if (a.x_dtype != TBN_BF16) return TBN_ERR_UNSUPPORTED;
    ConvParams p;
    if (!plan_conv(a, p)) return TBN_ERR_UNSUPPORTED;
    p.x = static_cast<const __nv_bfloat16 *>(a.x); p.y = a.y; p.tile = a.tile; p.alpha = a.alpha; p.bias = a.bias;
    p.status = device_status;
    p.n_words = tbn_tile_words(a.q);
    p.Nb = a.Nb; p.Cin = a.Cin; p.H = a.H; p.W = a.Wd; p.Ho = a.Ho; p.Wo = a.Wo;
    p.m = a.m; p.r = (int32_t)(a.q / a.n); p.k = a.k; p.n = a.n;
    p.per_tile = a.alpha_mode == TBN_ALPHA_PER_TILE; p.act = a.act; p.y_bf16 = a.y_dtype == TBN_BF16;
    const size_t smem = conv_smem_bytes(p);
    if (cudaFuncSetAttribute(tc_conv3x3_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return TBN_ERR_CUDA;
    // tensor map of x as (W, H, Cin, Nb); one box = all columns x raw_rows rows x 16 channels of one image
    CUtensorMap map;
    std::memset(&map, 0, sizeof(map));
    if (p.wide) {
        EncodeTiledFn encode = encode_tiled_fn();
        if (!encode) return TBN_ERR_CUDA;
        const cuuint64_t dims[4] = {(cuuint64_t)a.Wd, (cuuint64_t)a.H, (cuuint64_t)a.Cin, (cuuint64_t)a.Nb};
        const cuuint64_t strides[3] = {(cuuint64_t)a.Wd * 2, (cuuint64_t)a.H * a.Wd * 2,
                                       (cuuint64_t)a.Cin * a.H * a.Wd * 2};
        const cuuint32_t box[4] = {(cuuint32_t)a.Wd, (cuuint32_t)p.raw_rows, (cuuint32_t)kChanPerStage, 1};
        const cuuint32_t estr[4] = {1, 1, 1, 1};
        if (encode(&map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(a.x), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return TBN_ERR_CUDA;
    }
    const int sms = conv_sm_count();
    if (sms <= 0) return TBN_ERR_CUDA;
    const int64_t tiles = (int64_t)p.m_blocks * p.s_tiles;
    const unsigned grid = (unsigned)(tiles < sms ? tiles : sms);
    tc_conv3x3_kernel<<<grid, kConvThreads, smem, s>>>(map, p);
    return cudaGetLastError() == cudaSuccess ? TBN_OK : TBN_ERR_CUDA;
}

}  // namespace tbn
