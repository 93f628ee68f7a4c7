// Router of slices of 96 to 256 elements (Section 3.1: relu(X Wr1^T + br1) Wr2^T + br2 -> softmax -> top-k), bf16
// storage, router hidden width 256, up to 64 experts, k <= 8 (sm_100a: tcgen05 + TMEM + TMA).
//
// The whole of Wr1 (up to 128 KB) and Wr2 stay in shared memory for the life of the CTA, so a tile's GEMM-1 runs as
// wide MMAs against operands that are written to shared memory once per launch, not once per tile: what a tile
// moves through shared memory is its own rows and the operand reads of its MMAs.  Rows come as 64-column panels
// with a full / empty barrier pair each: rows of 192 / 256 (four panels, Wr1 = 128 KB) leave room for exactly ONE
// row tile, rows of 96 / 128 (two panels, Wr1 = 64 KB) for three.  GEMM-1 is issued panel by panel, all of a tile's
// MMAs on a panel before the next panel: the tile is done with a panel, and the next copy into its slot is
// requested, eight MMAs after the panel has landed, while the tile's other panels are still on their way -- with one
// row tile of shared memory the row loads still run a whole tile ahead.
//
// One CTA of 768 threads per SM walks a contiguous range of 128-row tiles.  A tile's hidden layer is two units, a
// narrow one (hidden 0 .. 63) and a wide one (64 .. 255): the wide unit has two buffers of tensor memory (the tile's
// parity picks one), the narrow unit one -- it is the first through the activation and through GEMM-2, so its
// buffer is free again by the time the next tile's first panel lands, and no tile waits for a buffer.  (Two units of
// 128 columns on three buffers: the second unit of every tile waited ~1.2 k cycles for the previous tile's first.)
// The activation warps turn a buffer's fp32 values in place into a truncated bf16 and the rounded remainder (GEMM-2
// runs over both, so the logits keep fp32-level accuracy and the top-k decision does not hang on a bf16 rounding of
// the hidden layer), GEMM-2 reads them from tensor memory into ONE logit accumulator, which the output warps have
// long loaded when the next tile's GEMM-2 starts.  Warp roles:
//   warp 0       row panels by TMA          warp 3  GEMM-1 issue        warp 1  GEMM-2 issue
//   warp 2       zeroes this CTA's rows of h' (forward: the experts add into it)
//   warps 4-19   activation (four warpgroups, 16 of the narrow and 48 of the wide unit's columns each; a thread
//                owns one tile row)
//   warps 20-23  softmax, top-k (ties to the lower id), this CTA's per-expert counts
// All hand-offs are mbarriers with bounded waits; a run-out sets the status word and every role leaves.
#include <mutex>

#include "pp_body.cuh"

namespace slicemoe {
namespace {

constexpr int kWrHr = 256;                    // router hidden width
constexpr int kWrPanelA = kTileM * 128;       // bytes: 128 rows x 64 bf16
constexpr int kWrPanelW1 = kWrHr * 128;       // bytes: 256 hidden units x 64 bf16
constexpr int kWrMaxE = 64;
constexpr int kWrMaxSlots = 6;                // row-panel slots: 1 tile x 4 panels or 3 tiles x 2 panels
constexpr int kWrMaxKP = 4;

struct WrShared {
    __align__(8) uint64_t bars[32];
    int hist[kWrMaxE];
    uint32_t tmem_base;
    int abort_flag;
    int tiles_out;               // tiles whose top-k has been written (paces the zeroing of h')
    __align__(16) float bias1_f32[kWrHr];
    __align__(16) float bias2_f32[kWrMaxE];
};

struct WrBars {
    static constexpr int A_FULL = 0;                        // [slots]
    static constexpr int A_EMPTY = A_FULL + kWrMaxSlots;    // [slots]
    static constexpr int W1_FULL = A_EMPTY + kWrMaxSlots;   // [KP] one per K panel of Wr1
    static constexpr int W2_FULL = W1_FULL + kWrMaxKP;
    static constexpr int ACC1_FULL = W2_FULL + 1;           // [3]
    static constexpr int ACC1_EMPTY = ACC1_FULL + 3;        // [3]
    static constexpr int HID_FULL = ACC1_EMPTY + 3;         // [3]
    static constexpr int ACC2_FULL = HID_FULL + 3;          // [2]
    static constexpr int ACC2_EMPTY = ACC2_FULL + 2;        // [2]
    static constexpr int DRAIN = ACC2_EMPTY + 2;            // [2]
    static constexpr int COUNT = DRAIN + 2;
};
static_assert(WrBars::COUNT <= 32, "barrier slots");

// EP: experts (padded), KP: 64-column panels of a row tile
template <int EP, int KP>
struct WrCfg {
    static constexpr int NT = KP == 4 ? 1 : 3;              // row tiles in shared memory
    static constexpr int SLOTS = NT * KP;
    static constexpr int W2_CHUNK = EP * 128;               // bytes: EP experts x 64 hidden units
    static constexpr int OFF_A = 0;
    static constexpr int OFF_W1 = OFF_A + SLOTS * kWrPanelA;
    static constexpr int OFF_W2 = OFF_W1 + KP * kWrPanelW1;
    static constexpr int SMEM_BYTES = OFF_W2 + (kWrHr / 64) * W2_CHUNK;
    // (at least 120 KB so that two CTAs never share an SM: each allocates all of tensor memory)
    static constexpr int SMEM_ALLOC = SMEM_BYTES + 1024 > 120 * 1024 ? SMEM_BYTES + 1024 : 120 * 1024;
    // The hidden layer of a tile as two units: a narrow one (hidden 0 .. 63) and a wide one (64 .. 255).  Tensor
    // memory: two wide buffers (the tile's parity picks one), one narrow buffer, one logit accumulator.
    static constexpr int NARROW = 64, WIDE = kWrHr - NARROW;
    static constexpr int WIDE_COL0 = 0, NARROW_COL = 2 * WIDE, LOGIT_COL = NARROW_COL + NARROW;
    static_assert(LOGIT_COL + kWrMaxE <= 512, "tensor memory");
    static_assert(KP == 2 || KP == 4, "row width");
    static_assert(SLOTS <= kWrMaxSlots && KP <= kWrMaxKP, "barrier slots");
    static_assert(SMEM_ALLOC + sizeof(WrShared) + 64 <= 232448, "shared memory budget");
    static_assert(EP % 16 == 0 && EP <= kWrMaxE, "expert count");
};

__device__ __forceinline__ uint32_t wr_bar(WrShared& sh, int i) { return smem_u32(&sh.bars[i]); }

// KBIG: k may exceed 2 (a kernel of its own: the extra picks' code and registers cost the k <= 2 kernel 4 % of its
// time on 64 experts when they share one)
template <int EP, int KP, bool KBIG>
__global__ void __launch_bounds__(kPpThreads, 1)
route_wide_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW1,
                  const __grid_constant__ CUtensorMap tmW2, const PpParams p) {
    using C = WrCfg<EP, KP>;
    using B = WrBars;
    constexpr int NT = C::NT;
    extern __shared__ uint8_t smem_raw[];
    __shared__ WrShared sh;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    volatile int* abort = &sh.abort_flag;

    const int total_tiles = (p.n_rows + kTileM - 1) / kTileM;
    const int per_cta = (total_tiles + gridDim.x - 1) / gridDim.x;
    const int t_begin = min(total_tiles, (int)blockIdx.x * per_cta);
    const int ntiles = min(total_tiles, t_begin + per_cta) - t_begin;
    const uint32_t sA = smem_base + C::OFF_A, sW1 = smem_base + C::OFF_W1, sW2 = smem_base + C::OFF_W2;

    if (warp == 1) {
        tmem_alloc(smem_u32(&sh.tmem_base), 512);
        tmem_relinquish();
    }
    if (threadIdx.x == 0) {
        prefetch_tensormap(&tmX);
        sh.abort_flag = 0;
        sh.tiles_out = 0;
        for (int i = 0; i < C::SLOTS; ++i) { mbar_init(wr_bar(sh, B::A_FULL + i), 1); mbar_init(wr_bar(sh, B::A_EMPTY + i), 1); }
        for (int i = 0; i < 3; ++i) {
            mbar_init(wr_bar(sh, B::ACC1_FULL + i), 1);
            mbar_init(wr_bar(sh, B::ACC1_EMPTY + i), 1);
            mbar_init(wr_bar(sh, B::HID_FULL + i), 16);
        }
        for (int r = 0; r < 2; ++r) {
            mbar_init(wr_bar(sh, B::ACC2_FULL + r), 1);
            mbar_init(wr_bar(sh, B::ACC2_EMPTY + r), 4);
            mbar_init(wr_bar(sh, B::DRAIN + r), 1);
        }
        fence_mbar_init();
        // the first tiles' panels come from DRAM and are what the pass waits for: requested right here
        for (int ta = 0; ta < min(ntiles, NT); ++ta)
            for (int kp = 0; kp < KP; ++kp) {
                mbar_arrive_expect_tx(wr_bar(sh, B::A_FULL + ta * KP + kp), kWrPanelA);
                tma_load_2d(sA + (ta * KP + kp) * kWrPanelA, &tmX, kp * 64, (t_begin + ta) * kTileM, wr_bar(sh, B::A_FULL + ta * KP + kp));
            }
    } else if (threadIdx.x == 64) {
        prefetch_tensormap(&tmW1);
        prefetch_tensormap(&tmW2);
        for (int i = 0; i < KP; ++i) mbar_init(wr_bar(sh, B::W1_FULL + i), 1);
        mbar_init(wr_bar(sh, B::W2_FULL), 1);
        fence_mbar_init();
        if (ntiles > 0) {
            for (int kp = 0; kp < KP; ++kp) {
                mbar_arrive_expect_tx(wr_bar(sh, B::W1_FULL + kp), kWrPanelW1);
                tma_load_2d(sW1 + kp * kWrPanelW1, &tmW1, kp * 64, 0, wr_bar(sh, B::W1_FULL + kp));
            }
            mbar_arrive_expect_tx(wr_bar(sh, B::W2_FULL), (uint32_t)((kWrHr / 64) * C::W2_CHUNK));
            for (int c = 0; c < kWrHr / 64; ++c) tma_load_2d(sW2 + c * C::W2_CHUNK, &tmW2, c * 64, 0, wr_bar(sh, B::W2_FULL));
        }
    }
    for (int e = threadIdx.x; e < kWrMaxE; e += kPpThreads) sh.hist[e] = 0;
    for (int i = threadIdx.x; i < kWrHr; i += kPpThreads) sh.bias1_f32[i] = p.br1 ? __bfloat162float(p.br1[i]) : 0.0f;
    for (int i = threadIdx.x; i < EP; i += kPpThreads)
        sh.bias2_f32[i] = i >= p.experts_real ? -INFINITY : (p.br2 ? __bfloat162float(p.br2[i]) : 0.0f);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = sh.tmem_base;

    if (warp == 0) {
        // ================= row panels: a tile's panel as soon as the tile NT back has let go of its slot =====
        if (lane == 0 && ntiles > 0) {
            bool ok = true;
            int requested = min(ntiles, NT) * KP;             // panels requested so far (the first tiles': above)
            for (int ta = NT; ta < ntiles && ok; ++ta) {
                const int sb = (ta % NT) * KP;
                for (int kp = 0; kp < KP; ++kp) {
                    if (!mbar_wait(wr_bar(sh, B::A_EMPTY + sb + kp), ((uint32_t)(ta / NT) & 1u) ^ 1u, abort, kWaitLimitNs)) { ok = false; break; }
                    mbar_arrive_expect_tx(wr_bar(sh, B::A_FULL + sb + kp), kWrPanelA);
                    tma_load_2d(sA + (sb + kp) * kWrPanelA, &tmX, kp * 64, (t_begin + ta) * kTileM, wr_bar(sh, B::A_FULL + sb + kp));
                    ++requested;
                }
            }
            if (!ok || *abort) {
                // giving up: the copies in flight still have to land before the CTA may leave (the last SLOTS
                // requests cover every slot once)
                volatile int never = 0;
                for (int kp = 0; kp < KP; ++kp) mbar_wait(wr_bar(sh, B::W1_FULL + kp), 0u, &never, 10000000ull);
                mbar_wait(wr_bar(sh, B::W2_FULL), 0u, &never, 10000000ull);
                for (int q = requested - 1; q >= 0 && q >= requested - C::SLOTS; --q) {
                    const int ta = q / KP;
                    mbar_wait(wr_bar(sh, B::A_FULL + (ta % NT) * KP + q % KP), (uint32_t)(ta / NT) & 1u, &never, 10000000ull);
                }
            }
        }
    } else if (warp == 3) {
        // ================= GEMM-1 issue ======================================================================
        // Panel by panel, both units on a panel before the next panel, so that a panel is released (and the next
        // tile's copy of it requested) eight MMAs after it has landed.  The wide unit's buffer alternates with the
        // tile and is long free; the narrow unit's single buffer is free once the previous tile's narrow unit
        // -- first through the activation, 8 MMAs of GEMM-2 -- has been consumed, which is about when this tile's
        // first panel lands.  From the second panel on the narrow unit goes first, so that it completes four
        // MMAs before the tile does and its activation starts under them.
        if (ntiles > 0) {
            constexpr uint32_t idescW = make_idesc(128, C::WIDE, kFmtBF16, kFmtBF16);
            constexpr uint32_t idescN = make_idesc(128, C::NARROW, kFmtBF16, kFmtBF16);
            const uint32_t dA = desc_lo_sw128(sA), dW1 = desc_lo_sw128(sW1);
            bool ok = true;
#pragma unroll 1
            for (int ta = 0; ta < ntiles && ok; ++ta) {
                const int wb = ta & 1;                  // wide buffer of this tile
                const int sb = (ta % NT) * KP;
                // (the buffer also held the hidden values of the tile two back: GEMM-2 must have read them)
                if (!pp_wait(wr_bar(sh, B::ACC1_EMPTY + wb), ((uint32_t)(ta >> 1) & 1u) ^ 1u, abort)) { ok = false; break; }
                const uint32_t dW = tmem_base + C::WIDE_COL0 + wb * C::WIDE, dN = tmem_base + C::NARROW_COL;
#pragma unroll
                for (int kp = 0; kp < KP; ++kp) {
                    if (ta == 0 && !pp_wait(wr_bar(sh, B::W1_FULL + kp), 0u, abort)) { ok = false; break; }
                    if (!pp_wait(wr_bar(sh, B::A_FULL + sb + kp), (uint32_t)(ta / NT) & 1u, abort)) { ok = false; break; }
                    tc_fence_after_sync();
                    const uint32_t a0 = dA + (((sb + kp) * kWrPanelA) >> 4);
                    const uint32_t wN = dW1 + ((kp * kWrPanelW1) >> 4), wW = wN + ((C::NARROW * 128) >> 4);
                    if (kp == 0) {
                        if (elect_one_sync()) {
#pragma unroll
                            for (int kk = 0; kk < 4; ++kk) {
                                if (kk == 0) mma_ss<0>(dW, a0, wW, idescW);
                                else mma_ss<1>(dW, a0 + ((kk * 32) >> 4), wW + ((kk * 32) >> 4), idescW);
                            }
                        }
                        __syncwarp();
                        if (!pp_wait(wr_bar(sh, B::ACC1_EMPTY + 2), ((uint32_t)ta & 1u) ^ 1u, abort)) { ok = false; break; }
                        tc_fence_after_sync();
                        if (elect_one_sync()) {
#pragma unroll
                            for (int kk = 0; kk < 4; ++kk) {
                                if (kk == 0) mma_ss<0>(dN, a0, wN, idescN);
                                else mma_ss<1>(dN, a0 + ((kk * 32) >> 4), wN + ((kk * 32) >> 4), idescN);
                            }
                            mma_commit(wr_bar(sh, B::A_EMPTY + sb + kp));       // the tile is done with the panel
                        }
                        __syncwarp();
                    } else {
                        if (elect_one_sync()) {
#pragma unroll
                            for (int kk = 0; kk < 4; ++kk) mma_ss<1>(dN, a0 + ((kk * 32) >> 4), wN + ((kk * 32) >> 4), idescN);
                            if (kp == KP - 1) mma_commit(wr_bar(sh, B::ACC1_FULL + 2));
#pragma unroll
                            for (int kk = 0; kk < 4; ++kk) mma_ss<1>(dW, a0 + ((kk * 32) >> 4), wW + ((kk * 32) >> 4), idescW);
                            mma_commit(wr_bar(sh, B::A_EMPTY + sb + kp));
                            if (kp == KP - 1) mma_commit(wr_bar(sh, B::ACC1_FULL + wb));
                        }
                        __syncwarp();
                    }
                }
            }
            if (!ok || *abort) {
                volatile int never = 0;
                if (lane == 0) {
                    mma_commit(wr_bar(sh, B::DRAIN));
                    mbar_wait(wr_bar(sh, B::DRAIN), 0u, &never, 10000000ull);
                }
                __syncwarp();
            }
        }
    } else if (warp == 1) {
        // ================= GEMM-2 issue: logits = hidden(hi) Wr2^T + hidden(lo) Wr2^T ==========================
        // K step kk of a unit: hi halves in the unit's columns 16 kk .. 16 kk + 7, lo halves in the next eight.
        // The narrow unit (hidden 0 .. 63, Wr2's first panel) first: its buffer is the one the next tile waits for.
        if (ntiles > 0) {
            constexpr uint32_t idesc2 = make_idesc(128, EP, kFmtBF16, kFmtBF16);
            const uint32_t dW2 = desc_lo_sw128(sW2);
            bool ok = pp_wait(wr_bar(sh, B::W2_FULL), 0u, abort);
#pragma unroll 1
            for (int ta = 0; ta < ntiles && ok; ++ta) {
                const int wb = ta & 1;
                const uint32_t d = tmem_base + C::LOGIT_COL;
                // (one logit accumulator: the output warps must have loaded the previous tile's)
                if (!pp_wait(wr_bar(sh, B::ACC2_EMPTY), ((uint32_t)ta & 1u) ^ 1u, abort)) { ok = false; break; }
                if (!pp_wait(wr_bar(sh, B::HID_FULL + 2), (uint32_t)ta & 1u, abort)) { ok = false; break; }
                tc_fence_after_sync();
                if (elect_one_sync()) {
                    const uint32_t a = tmem_base + C::NARROW_COL;
#pragma unroll
                    for (int part = 0; part < 2; ++part) {
#pragma unroll
                        for (int kk = 0; kk < C::NARROW / 16; ++kk) {
                            const uint32_t bd = dW2 + ((kk * 32) >> 4);
                            if (part == 0 && kk == 0) mma_ts<0>(d, a, bd, idesc2);
                            else mma_ts<1>(d, a + kk * 16 + part * 8, bd, idesc2);
                        }
                    }
                    mma_commit(wr_bar(sh, B::ACC1_EMPTY + 2));
                }
                __syncwarp();
                if (!pp_wait(wr_bar(sh, B::HID_FULL + wb), (uint32_t)(ta >> 1) & 1u, abort)) { ok = false; break; }
                tc_fence_after_sync();
                if (elect_one_sync()) {
                    const uint32_t a = tmem_base + C::WIDE_COL0 + wb * C::WIDE;
#pragma unroll
                    for (int part = 0; part < 2; ++part) {
#pragma unroll
                        for (int kk = 0; kk < C::WIDE / 16; ++kk) {
                            // hidden units NARROW + 16 kk ..: panel (NARROW + 16 kk) / 64 of Wr2
                            constexpr int kk0 = C::NARROW / 16;
                            const uint32_t bd = dW2 + (((((kk + kk0) >> 2) * C::W2_CHUNK) + ((kk + kk0) & 3) * 32) >> 4);
                            mma_ts<1>(d, a + kk * 16 + part * 8, bd, idesc2);
                        }
                    }
                    mma_commit(wr_bar(sh, B::ACC1_EMPTY + wb));
                    mma_commit(wr_bar(sh, B::ACC2_FULL));
                }
                __syncwarp();
            }
            if (!ok || *abort) {
                volatile int never = 0;
                if (lane == 0) {
                    mma_commit(wr_bar(sh, B::DRAIN + 1));
                    mbar_wait(wr_bar(sh, B::DRAIN + 1), 0u, &never, 10000000ull);
                }
                __syncwarp();
            }
        }
    } else if (warp == 2) {
        // ================= zero this CTA's rows of h' ========================================================
        // Tile by tile, at the pace of the tiles' results (two tiles ahead of the output warps): written in one
        // burst at the start, the 2 x 64 KB per tile that this pass writes crowd out the row loads of the first
        // tiles, whose latency is on the critical path of a pipeline with a single row-tile buffer.
        if (p.zero_out != nullptr) {
            const uint4 z = make_uint4(0u, 0u, 0u, 0u);
            volatile int* done = &sh.tiles_out;
            bool ok = true;
#pragma unroll 1
            for (int ta = 0; ta < ntiles && ok; ++ta) {
                if (ta >= 2 && *done < ta - 1) {
                    const uint64_t t0 = globaltimer_ns();
                    while (*done < ta - 1) {
                        __nanosleep(256);
                        if (*abort || globaltimer_ns() - t0 > kWaitLimitNs) { ok = false; break; }
                    }
                    if (!ok) break;
                }
                const long long row_lo = (long long)(t_begin + ta) * kTileM;
                long long row_hi = row_lo + kTileM;
                if (row_hi > p.n_rows) row_hi = p.n_rows;
                uint4* dst = reinterpret_cast<uint4*>(p.zero_out + row_lo * p.row_elems);
                const int nvec = (int)(row_hi - row_lo) * p.row_elems / 8;
#pragma unroll 4
                for (int i = lane; i < nvec; i += 32) dst[i] = z;
            }
            // (a pass that gave up leaves its status word set; the rows not zeroed are then not results)
        }
    } else if (warp < 20) {
        // ================= activation warps: warpgroup g, lane group lg ======================================
        // relu(acc + bias) as hi + lo, in place: hi = the value truncated to bf16 (negative -> 0 by .relu), lo = the
        // rounded remainder (for a negative value the remainder is the value itself and its .relu is 0 too).  A
        // 16-column piece becomes 8 columns of hi pairs and 8 of lo pairs = one K step of GEMM-2.
        const int g = (warp - 4) >> 2;
        const int lg = warp & 3;
        const uint32_t tlane = tmem_base + ((uint32_t)(lg * 32) << 16);
        const bool has_br1 = p.br1 != nullptr;
        auto split_piece = [&](const uint32_t* acc, const float* bias, uint32_t col) {
            float a[16];
            if (has_br1) {
#pragma unroll
                for (int i = 0; i < 16; i += 4) {
                    const float4 bb = *reinterpret_cast<const float4*>(bias + i);
                    add2(a[i], a[i + 1], __uint_as_float(acc[i]), __uint_as_float(acc[i + 1]), bb.x, bb.y);
                    add2(a[i + 2], a[i + 3], __uint_as_float(acc[i + 2]), __uint_as_float(acc[i + 3]), bb.z, bb.w);
                }
            } else {
#pragma unroll
                for (int i = 0; i < 16; ++i) a[i] = __uint_as_float(acc[i]);
            }
            uint32_t hl[16];
#pragma unroll
            for (int i = 0; i < 8; ++i) hl[i] = cvt_rz_relu_bf16x2(a[2 * i], a[2 * i + 1]);
#pragma unroll
            for (int i = 0; i < 8; ++i)
                hl[8 + i] = cvt_rn_relu_bf16x2(a[2 * i] - __uint_as_float(hl[i] << 16), a[2 * i + 1] - __uint_as_float(hl[i] & 0xFFFF0000u));
            tmem_st_x16(col, hl);
        };
        bool ok = true;
#pragma unroll 1
        for (int ta = 0; ta < ntiles && ok; ++ta) {
            const int wb = ta & 1;
            // ---- the narrow unit (hidden 0 .. 63): 16 columns per warpgroup
            ok = pp_wait(wr_bar(sh, B::ACC1_FULL + 2), (uint32_t)ta & 1u, abort);
            if (!ok) break;
            tc_fence_after_sync();
            {
                const uint32_t col = tlane + C::NARROW_COL + 16 * g;
                uint32_t acc[16];
                tmem_ld_x16(col, acc);
                tmem_ld_wait();
                split_piece(acc, sh.bias1_f32 + 16 * g, col);
                tmem_st_wait();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(wr_bar(sh, B::HID_FULL + 2));
            }
            // ---- the wide unit (hidden 64 .. 255): 48 columns per warpgroup
            ok = pp_wait(wr_bar(sh, B::ACC1_FULL + wb), (uint32_t)(ta >> 1) & 1u, abort);
            if (!ok) break;
            tc_fence_after_sync();
            {
                const uint32_t col = tlane + C::WIDE_COL0 + wb * C::WIDE + 48 * g;
                const float* bias = sh.bias1_f32 + C::NARROW + 48 * g;
                // three pieces, each loaded under the arithmetic of the one before (16-column loads: the
                // warpgroups' column offsets are multiples of 16 only)
                uint32_t acc0[16], acc1[16];
                tmem_ld_x16(col, acc0);
                tmem_ld_wait();
                tmem_ld_x16(col + 16, acc1);
                split_piece(acc0, bias, col);
                tmem_ld_wait();
                tmem_ld_x16(col + 32, acc0);
                split_piece(acc1, bias + 16, col + 16);
                tmem_ld_wait();
                split_piece(acc0, bias + 32, col + 32);
                tmem_st_wait();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(wr_bar(sh, B::HID_FULL + wb));
            }
        }
    } else {
        // ================= output warpgroup: softmax + top-k of a tile's logits ==============================
        const int lg = warp & 3;
        const int row = lg * 32 + lane;
        const uint32_t tlane = tmem_base + ((uint32_t)(lg * 32) << 16) + C::LOGIT_COL;
        bool ok = true;
#pragma unroll 1
        for (int ta = 0; ta < ntiles && ok; ++ta) {
            ok = pp_wait(wr_bar(sh, B::ACC2_FULL), (uint32_t)ta & 1u, abort);
            if (!ok) break;
            tc_fence_after_sync();
            uint32_t v[EP];
#pragma unroll
            for (int c = 0; c < EP; c += 16) tmem_ld_x16(tlane + c, v + c);
            tmem_ld_wait();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(wr_bar(sh, B::ACC2_EMPTY));
            const int n = (t_begin + ta) * kTileM + row;
            const bool valid = n < p.n_rows;
            // one pass keeping the best two (strict comparisons in ascending id order: the picks of repeated
            // arg-max with ties to the lower id); the logits stay in v as raw bits + bias
            float b1 = -INFINITY, b2 = -INFINITY;
            int i1 = 0, i2 = 0;
#pragma unroll
            for (int i = 0; i < EP; ++i) {
                const float gl = __uint_as_float(v[i]) + sh.bias2_f32[i];
                v[i] = __float_as_uint(gl);
                const bool gt1 = gl > b1, gt2 = gl > b2;
                b2 = gt1 ? b1 : (gt2 ? gl : b2);
                i2 = gt1 ? i1 : (gt2 ? i : i2);
                b1 = gt1 ? gl : b1;
                i1 = gt1 ? i : i1;
            }
            const float sc = p.softmax_scale;
            const float msc = b1 * sc;
            float sum = 0.0f;
#pragma unroll
            for (int i = 0; i < EP; ++i) sum += ex2_approx(fmaf(__uint_as_float(v[i]), sc, -msc));
            const float inv = 1.0f / sum;
            const float p2 = ex2_approx(fmaf(b2, sc, -msc)) * inv;
            if (lane == 0 && lg == 0) sh.tiles_out = ta + 1;
            if (valid) {
                const size_t at = (size_t)n * p.k;
                atomicAdd(&sh.hist[i1], 1);
                if (p.k == 1) {
                    p.topk_idx[at] = i1;
                    p.topk_p[at] = inv;
                } else {
                    if (!KBIG || p.k == 2) {
                        *reinterpret_cast<int2*>(p.topk_idx + at) = make_int2(i1, i2);
                        *reinterpret_cast<float2*>(p.topk_p + at) = make_float2(inv, p2);
                    } else {
                        p.topk_idx[at] = i1;     p.topk_p[at] = inv;
                        p.topk_idx[at + 1] = i2; p.topk_p[at + 1] = p2;
                    }
                    atomicAdd(&sh.hist[i2], 1);
                    // k > 2: the rest by repeated arg-max over what is left (ties to the lower id)
                    unsigned long long taken = (1ull << i1) | (1ull << i2);
                    for (int j = 2; KBIG && j < p.k; ++j) {
                        int best = -1;
                        float bv = 0.0f;
#pragma unroll
                        for (int i = 0; i < EP; ++i) {
                            const float gl = __uint_as_float(v[i]);
                            const bool free_i = !((taken >> i) & 1ull);
                            if (free_i && (best < 0 || gl > bv)) { best = i; bv = gl; }
                        }
                        taken |= 1ull << best;
                        p.topk_idx[at + j] = best;
                        p.topk_p[at + j] = ex2_approx(fmaf(bv, sc, -msc)) * inv;
                        atomicAdd(&sh.hist[best], 1);
                    }
                }
            }
        }
    }

    // ---- teardown ---------------------------------------------------------------------------------------
    tc_fence_before_sync();
    __syncthreads();
    if (threadIdx.x == 0 && sh.abort_flag) atomicExch(p.status, (int)SLICEMOE_ERR_DEVICE_TIMEOUT);
    if (p.cta_hist)
        for (int i = threadIdx.x; i < p.experts_real; i += kPpThreads) p.cta_hist[(size_t)blockIdx.x * p.experts_real + i] = sh.hist[i];
    if (p.assigned_out && ntiles > 0)
        for (int i = threadIdx.x; i < p.experts_real; i += kPpThreads)
            if (sh.hist[i] > 0) atomicAdd(p.assigned_out + i, sh.hist[i]);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (warp == 1) {
        __syncwarp();
        tmem_dealloc(sh.tmem_base, 512);
    }
}

template <int EP, int KP, bool KBIG>
int launch_wide(const Dims& D, const slicemoe_weights& w, const void* h, const PpParams& rp, int grid, cudaStream_t st) {
    CUtensorMap mX, mW1, mW2;
    int rc;
    // (rows of 96 / 192 elements: the boxes reach past the tensors' edge and are zero-filled there)
    if ((rc = make_tmap(&mX, h, (uint64_t)D.N, (uint64_t)D.ds, kTileM))) return rc;
    if ((rc = make_tmap(&mW1, w.Wr1, (uint64_t)D.Hr, (uint64_t)D.ds, kWrHr))) return rc;
    if ((rc = make_tmap(&mW2, w.Wr2, (uint64_t)D.E, (uint64_t)D.Hr, EP))) return rc;      // (E = 8: zero-filled up to 16)
    auto kern = route_wide_kernel<EP, KP, KBIG>;
    static bool attr_set[kAttrMaxDevices] = {};
    static std::mutex attr_mutex;
    {
        std::lock_guard<std::mutex> lock(attr_mutex);
        if ((rc = set_smem_limit_once(kern, WrCfg<EP, KP>::SMEM_ALLOC, attr_set))) return rc;
    }
    kern<<<grid, kPpThreads, WrCfg<EP, KP>::SMEM_ALLOC, st>>>(mX, mW1, mW2, rp);
    SLICEMOE_LAUNCH_CHECK(1);
    return SLICEMOE_OK;
}

template <int EP>
int launch_wide_e(const Dims& D, const slicemoe_weights& w, const void* h, const PpParams& rp, int grid, cudaStream_t st) {
    if (D.k > 2) return D.ds <= 128 ? launch_wide<EP, 2, true>(D, w, h, rp, grid, st) : launch_wide<EP, 4, true>(D, w, h, rp, grid, st);
    return D.ds <= 128 ? launch_wide<EP, 2, false>(D, w, h, rp, grid, st) : launch_wide<EP, 4, false>(D, w, h, rp, grid, st);
}

}  // namespace

bool wide_route_supported(const Dims& D) {
    if (D.dtype != SLICEMOE_BF16 || (D.ds != 256 && D.ds != 192 && D.ds != 128 && D.ds != 96) || D.N <= 0) return false;
    if (D.E != 8 && D.E != 16 && D.E != 32 && D.E != 64) return false;
    if (D.k > 8 || D.k > D.E || D.noise_sigma > 0.0f) return false;
    return D.Hr == kWrHr;
}

int launch_route_wide(const Dims& D, const slicemoe_weights& w, const void* h, int32_t* topk_idx, float* topk_p,
                      int32_t* assigned, int32_t* status, cudaStream_t st, int32_t* cta_hist, void* zero_out,
                      int grid_rows) {
    if (assigned) SLICEMOE_CUDA_TRY(cudaMemsetAsync(assigned, 0, sizeof(int32_t) * D.E, st));
    PpParams r{};
    r.status = status; r.n_rows = D.N; r.HID = D.Hr; r.experts_real = D.E; r.k = D.k;
    r.softmax_scale = 1.4426950408889634f * D.inv_tau;
    r.br1 = (const bf16*)w.br1; r.br2 = (const bf16*)w.br2;
    r.topk_idx = topk_idx; r.topk_p = topk_p;
    r.assigned_out = assigned; r.cta_hist = cta_hist;
    r.zero_out = (bf16*)zero_out; r.row_elems = D.ds;
    // The rows are split over the CTAs as tc_route_grid says (CTAs past the last tile have none); with grid_rows the
    // launch has that many CTAs, each of which writes its row of cta_hist (zeros where it has no tile).
    int grid = 0, rows_per_cta = 0;
    tc_route_grid(D, &grid, &rows_per_cta);
    if (grid_rows > grid) grid = grid_rows;
    switch (D.E) {
        case 8:
        case 16: return launch_wide_e<16>(D, w, h, r, grid, st);
        case 32: return launch_wide_e<32>(D, w, h, r, grid, st);
        case 64: return launch_wide_e<64>(D, w, h, r, grid, st);
        default: return SLICEMOE_ERR_UNSUPPORTED;
    }
}

}  // namespace slicemoe
