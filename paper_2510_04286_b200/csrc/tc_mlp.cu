// Tensor-core path (sm_100a: tcgen05 + TMEM + TMA) for the two MLPs of the layer, bf16 storage:
//
//   router  (Section 3.1): relu(X Wr1^T + br1) Wr2^T + br2 -> softmax -> top-k   (per 128-row tile)
//   experts (Section 3.1 / 3.4): act(X~_e W1_e^T + b1_e) W2_e^T + b2_e           (per 128-row tile of
//                                                                                 one expert's rows)
//
// Both are the same kernel: GEMM-1 into a TMEM accumulator, an epilogue that applies bias +
// activation and writes the hidden chunk as bf16 into shared memory in the K-major 128-byte
// swizzled layout, GEMM-2 from that chunk into a second TMEM accumulator, and a final epilogue
// (softmax + top-k + histogram for the router; bias + store for the experts).  The hidden layer is
// processed in chunks of HC units and never leaves the SM.
//
// One persistent CTA per SM walks a contiguous range of tiles (expert-major, so expert weights
// stay in shared memory while the expert does not change).  Warp roles:
//   warp 0        TMA producer (one lane): row tiles and weight chunks
//   warp 1        TMEM allocation + MMA issue (one lane)
//   warps 2..     epilogue warps (two warpgroups; a warp owns TMEM lanes 32*(warp_id % 4)..+31,
//                 one row per thread; the warpgroups split the columns)
// All hand-offs are mbarriers; every wait is bounded and a run-out sets the status word and makes
// all roles leave.
#include <cuda.h>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace slicemoe {
namespace {

using namespace ptx;

constexpr uint64_t kWaitLimitNs = 2000000000ull;   // a wait that takes 2 s is a bug, not load
constexpr int kMaxHid = 1024;
constexpr int kMaxE = 256;

struct TcParams {
    const int32_t* offsets;   // experts: [E+1] device row ranges; router: nullptr
    int n_rows;               // router: N
    int E;                    // experts: E; router: 1
    int HID;                  // Hr or F
    const bf16* bias1;        // [E, HID] or nullptr
    const bf16* bias2;        // [E, N2]  or nullptr
    bf16* yperm;              // experts: output rows [R, N2]
    int32_t* topk_idx;        // router outputs
    float* topk_p;
    int32_t* assigned;
    float* probs;             // or nullptr
    int k;
    int32_t* status;
};

constexpr int pow2_at_least(int x) {
    int p = 32;
    while (p < x) p <<= 1;
    return p;
}

template <int K1_, int N2_, bool ROUTER_, int ACT_>
struct TcCfg {
    static constexpr int K1 = K1_, N2 = N2_, ACT = ACT_;
    static constexpr bool ROUTER = ROUTER_;
    static constexpr int HC = (K1 == 64) ? 128 : 64;           // hidden units per chunk
    static constexpr int A_BUFS = (K1 <= 128) ? 2 : 1;
    static constexpr int W_STAGES = (K1 == 128) ? 3 : 2;
    static constexpr int EPI_WG = 2;
    static constexpr int EPI_WARPS = EPI_WG * 4;
    static constexpr int EPI_THREADS = EPI_WG * 128;
    static constexpr int THREADS = 64 + EPI_THREADS;
    static constexpr int ACC2_BUFS = (N2 <= 128) ? 2 : 1;
    static constexpr int TMEM_COLS = pow2_at_least(2 * HC + ACC2_BUFS * N2);
    static constexpr int KP1 = K1 / 64;                         // 64-wide K panels of GEMM-1
    static constexpr int KP2 = HC / 64;                         // K panels of GEMM-2 per chunk
    static constexpr int A_PANEL = 128 * 128;                   // bytes: 128 rows x 128 B
    static constexpr int A_BYTES = KP1 * A_PANEL;
    static constexpr int W1_PANEL = HC * 128;
    static constexpr int W1C_BYTES = KP1 * W1_PANEL;
    static constexpr int W2_PANEL = N2 * 128;
    static constexpr int W2C_BYTES = KP2 * W2_PANEL;
    static constexpr int W_STAGE_BYTES = W1C_BYTES + W2C_BYTES;
    static constexpr int H_PANEL = 128 * 128;
    // The router keeps the hidden layer as a bf16 pair (hi + lo = 16 mantissa bits): GEMM-2 runs
    // over both halves against the same weights, so that the logits carry fp32-level accuracy and
    // the top-k decision does not depend on bf16 rounding of the hidden layer.
    static constexpr int H_PARTS = ROUTER_ ? 2 : 1;
    static constexpr int H_BYTES = H_PARTS * KP2 * H_PANEL;
    static constexpr int OFF_A = 0;
    static constexpr int OFF_W = OFF_A + A_BUFS * A_BYTES;
    static constexpr int OFF_H = OFF_W + W_STAGES * W_STAGE_BYTES;
    static constexpr int SMEM_BYTES = OFF_H + 2 * H_BYTES;
    static constexpr int SMEM_ALLOC = SMEM_BYTES + 1024;        // slack for the 1024-byte alignment
    static constexpr int COLS1 = HC / EPI_WG;                   // hidden columns per epilogue thread
    static_assert(W_STAGE_BYTES % 1024 == 0 && W1C_BYTES % 1024 == 0, "operand tiles must stay 1024-byte aligned");
    static_assert(N2 % 16 == 0 && N2 >= 16 && N2 <= 256, "MMA N");
    static_assert(COLS1 % 32 == 0, "epilogue loads are 32 columns wide");
    static_assert(SMEM_ALLOC <= 232448, "shared memory budget");
    static_assert(2 * HC + ACC2_BUFS * N2 <= 512, "TMEM budget");
};

// Barrier slots in shared memory.
template <class C>
struct Bars {
    static constexpr int A_FULL = 0;
    static constexpr int A_EMPTY = A_FULL + C::A_BUFS;
    static constexpr int W_FULL = A_EMPTY + C::A_BUFS;
    static constexpr int W_EMPTY = W_FULL + C::W_STAGES;
    static constexpr int ACC1_FULL = W_EMPTY + C::W_STAGES;
    static constexpr int ACC1_EMPTY = ACC1_FULL + 2;
    static constexpr int H_FULL = ACC1_EMPTY + 2;
    static constexpr int H_EMPTY = H_FULL + 2;
    static constexpr int ACC2_FULL = H_EMPTY + 2;
    static constexpr int ACC2_EMPTY = ACC2_FULL + C::ACC2_BUFS;
    static constexpr int DRAIN = ACC2_EMPTY + C::ACC2_BUFS;
    static constexpr int COUNT = DRAIN + 1;
};

__device__ __forceinline__ void locate_tile(const int* tile_start, const int* offs, int t, int& e,
                                            int& row0, int& rows) {
    while (t >= tile_start[e + 1]) ++e;
    row0 = offs[e] + (t - tile_start[e]) * kTileM;
    rows = min(kTileM, offs[e + 1] - row0);
}

__device__ __forceinline__ float tanh_approx(float x) {
    float y;
    asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <int ACT>
__device__ __forceinline__ float activate(float z) {
    if (ACT == SLICEMOE_ACT_RELU) return fmaxf(z, 0.0f);
    // GELU, tanh form: 0.5 z (1 + tanh(sqrt(2/pi) (z + 0.044715 z^3)))
    const float u = z * fmaf(0.0356774081f, z * z, 0.7978845608f);
    const float hz = 0.5f * z;
    return fmaf(hz, tanh_approx(u), hz);
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

template <class C>
__global__ void __launch_bounds__(C::THREADS, 1)
tc_mlp_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmW1,
              const __grid_constant__ CUtensorMap tmW2, const TcParams p) {
    using B = Bars<C>;
    extern __shared__ uint8_t smem_raw[];
    __shared__ __align__(8) uint64_t bars[B::COUNT];
    __shared__ int tile_start[kMaxE + 1];
    __shared__ int offs[kMaxE + 1];
    __shared__ int hist[kMaxE];
    __shared__ uint32_t tmem_base_smem;
    __shared__ int abort_flag;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    volatile int* abort = &abort_flag;
    const int nchunks = p.HID / C::HC;
    const bool resident = nchunks <= C::W_STAGES;
    auto bar = [&](int i) { return smem_u32(&bars[i]); };

    // ---- set-up ---------------------------------------------------------------------------
    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int i = 0; i < C::A_BUFS; ++i) { mbar_init(bar(B::A_FULL + i), 1); mbar_init(bar(B::A_EMPTY + i), 1); }
        for (int i = 0; i < C::W_STAGES; ++i) { mbar_init(bar(B::W_FULL + i), 1); mbar_init(bar(B::W_EMPTY + i), 1); }
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar(B::ACC1_FULL + i), 1);
            mbar_init(bar(B::ACC1_EMPTY + i), C::EPI_WARPS);
            mbar_init(bar(B::H_FULL + i), C::EPI_WARPS);
            mbar_init(bar(B::H_EMPTY + i), 1);
        }
        for (int i = 0; i < C::ACC2_BUFS; ++i) {
            mbar_init(bar(B::ACC2_FULL + i), 1);
            mbar_init(bar(B::ACC2_EMPTY + i), C::EPI_WARPS);
        }
        mbar_init(bar(B::DRAIN), 1);
        fence_mbar_init();
        prefetch_tensormap(&tmA);
        prefetch_tensormap(&tmW1);
        prefetch_tensormap(&tmW2);
    }
    for (int e = threadIdx.x; e <= p.E; e += C::THREADS) offs[e] = p.offsets ? p.offsets[e] : (e == 0 ? 0 : p.n_rows);
    for (int e = threadIdx.x; e < kMaxE; e += C::THREADS) hist[e] = 0;
    if (warp == 1) {
        tmem_alloc(smem_u32(&tmem_base_smem), C::TMEM_COLS);
        tmem_relinquish();
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int run = 0;
        for (int e = 0; e < p.E; ++e) {
            tile_start[e] = run;
            run += (offs[e + 1] - offs[e] + kTileM - 1) / kTileM;
        }
        tile_start[p.E] = run;
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = tmem_base_smem;
    const int total_tiles = tile_start[p.E];
    const int per_cta = (total_tiles + gridDim.x - 1) / gridDim.x;
    const int t_begin = min(total_tiles, (int)blockIdx.x * per_cta);
    const int t_end = min(total_tiles, t_begin + per_cta);

    const uint32_t sA = smem_base + C::OFF_A, sW = smem_base + C::OFF_W, sH = smem_base + C::OFF_H;

    if (warp == 0) {
        // ================= TMA producer =====================================================
        if (lane == 0 && t_begin < t_end) {
            int e = 0, prev_e = -1;
            uint32_t g = 0;
            uint32_t w_loads[C::W_STAGES];
            uint32_t last_w_bar[C::W_STAGES], last_w_par[C::W_STAGES];
            uint32_t last_a_bar[C::A_BUFS], last_a_par[C::A_BUFS];
            for (int i = 0; i < C::W_STAGES; ++i) { w_loads[i] = 0; last_w_bar[i] = 0; last_w_par[i] = 0; }
            for (int i = 0; i < C::A_BUFS; ++i) { last_a_bar[i] = 0; last_a_par[i] = 0; }
            bool ok = true;
            for (int t = t_begin, ta = 0; t < t_end && ok; ++t, ++ta) {
                int row0, rows;
                locate_tile(tile_start, offs, t, e, row0, rows);
                const int ab = ta % C::A_BUFS;
                const uint32_t an = ta / C::A_BUFS;
                if (!mbar_wait(bar(B::A_EMPTY + ab), (an & 1u) ^ 1u, abort, kWaitLimitNs)) { ok = false; break; }
                mbar_arrive_expect_tx(bar(B::A_FULL + ab), C::A_BYTES);
#pragma unroll
                for (int kp = 0; kp < C::KP1; ++kp)
                    tma_load_2d(sA + ab * C::A_BYTES + kp * C::A_PANEL, &tmA, kp * 64, row0, bar(B::A_FULL + ab));
                last_a_bar[ab] = bar(B::A_FULL + ab);
                last_a_par[ab] = an & 1u;
                const bool reload = !resident || (e != prev_e);
                prev_e = e;
                for (int c = 0; c < nchunks && ok; ++c, ++g) {
                    if (!reload) continue;
                    const int slot = resident ? c : (int)(g % C::W_STAGES);
                    const uint32_t n = w_loads[slot]++;
                    if (!mbar_wait(bar(B::W_EMPTY + slot), (n & 1u) ^ 1u, abort, kWaitLimitNs)) { ok = false; break; }
                    mbar_arrive_expect_tx(bar(B::W_FULL + slot), C::W_STAGE_BYTES);
                    const uint32_t dst = sW + slot * C::W_STAGE_BYTES;
#pragma unroll
                    for (int kp = 0; kp < C::KP1; ++kp)
                        tma_load_2d(dst + kp * C::W1_PANEL, &tmW1, kp * 64, e * p.HID + c * C::HC, bar(B::W_FULL + slot));
#pragma unroll
                    for (int kp = 0; kp < C::KP2; ++kp)
                        tma_load_2d(dst + C::W1C_BYTES + kp * C::W2_PANEL, &tmW2, c * C::HC + kp * 64, e * C::N2,
                                    bar(B::W_FULL + slot));
                    last_w_bar[slot] = bar(B::W_FULL + slot);
                    last_w_par[slot] = n & 1u;
                }
            }
            if (!ok || *abort) {
                // leaving early: let this thread's copies in flight land first (bounded)
                volatile int never = 0;
                for (int i = 0; i < C::A_BUFS; ++i)
                    if (last_a_bar[i]) mbar_wait(last_a_bar[i], last_a_par[i], &never, 10000000ull);
                for (int i = 0; i < C::W_STAGES; ++i)
                    if (last_w_bar[i]) mbar_wait(last_w_bar[i], last_w_par[i], &never, 10000000ull);
            }
        }
    } else if (warp == 1) {
        // ================= MMA issue =========================================================
        if (lane == 0 && t_begin < t_end) {
            constexpr uint32_t idesc1 = make_idesc_bf16(128, C::HC);
            constexpr uint32_t idesc2 = make_idesc_bf16(128, C::N2);
            uint32_t w_uses[C::W_STAGES];
            for (int i = 0; i < C::W_STAGES; ++i) w_uses[i] = 0;
            bool ok = true;

            struct Item { int t, ta, c, e; uint32_t g; bool valid, reload, release; };
            auto enter_tile = [&](Item& it, int prev_e) {
                int row0, rows;
                locate_tile(tile_start, offs, it.t, it.e, row0, rows);
                it.reload = !resident || (it.e != prev_e);
                bool rel = !resident;
                if (resident && it.t + 1 < t_end) {
                    int e2 = it.e, r0, rr;
                    locate_tile(tile_start, offs, it.t + 1, e2, r0, rr);
                    rel = (e2 != it.e);
                }
                it.release = rel;
            };
            auto advance = [&](Item& it) {
                ++it.c; ++it.g;
                if (it.c == nchunks) {
                    it.c = 0; ++it.t; ++it.ta;
                    if (it.t < t_end) { const int pe = it.e; enter_tile(it, pe); } else it.valid = false;
                }
            };
            auto issue_g1 = [&](const Item& it) -> bool {
                const int ab = it.ta % C::A_BUFS;
                if (it.c == 0 &&
                    !mbar_wait(bar(B::A_FULL + ab), (uint32_t)(it.ta / C::A_BUFS) & 1u, abort, kWaitLimitNs)) return false;
                const int slot = resident ? it.c : (int)(it.g % C::W_STAGES);
                if (it.reload) {
                    const uint32_t n = w_uses[slot]++;
                    if (!mbar_wait(bar(B::W_FULL + slot), n & 1u, abort, kWaitLimitNs)) return false;
                }
                const uint32_t b = it.g & 1u, n1 = it.g >> 1;
                if (!mbar_wait(bar(B::ACC1_EMPTY + b), (n1 & 1u) ^ 1u, abort, kWaitLimitNs)) return false;
                tc_fence_after_sync();
                const uint32_t a0 = sA + ab * C::A_BYTES, w0 = sW + slot * C::W_STAGE_BYTES;
#pragma unroll
                for (int kk = 0; kk < C::K1 / 16; ++kk) {
                    const uint64_t ad = make_desc_sw128(a0 + (kk >> 2) * C::A_PANEL + (kk & 3) * 32);
                    const uint64_t bd = make_desc_sw128(w0 + (kk >> 2) * C::W1_PANEL + (kk & 3) * 32);
                    mma_bf16_ss(tmem_base + b * C::HC, ad, bd, idesc1, kk > 0 ? 1u : 0u);
                }
                mma_commit(bar(B::ACC1_FULL + b));
                if (it.c == nchunks - 1) mma_commit(bar(B::A_EMPTY + ab));
                return true;
            };
            auto issue_g2 = [&](const Item& it) -> bool {
                const uint32_t b = it.g & 1u, n1 = it.g >> 1;
                if (!mbar_wait(bar(B::H_FULL + b), n1 & 1u, abort, kWaitLimitNs)) return false;
                const int buf = it.ta % C::ACC2_BUFS;
                if (it.c == 0 && !mbar_wait(bar(B::ACC2_EMPTY + buf), ((uint32_t)(it.ta / C::ACC2_BUFS) & 1u) ^ 1u,
                                            abort, kWaitLimitNs)) return false;
                tc_fence_after_sync();
                const int slot = resident ? it.c : (int)(it.g % C::W_STAGES);
                const uint32_t h0 = sH + b * C::H_BYTES, w0 = sW + slot * C::W_STAGE_BYTES + C::W1C_BYTES;
#pragma unroll
                for (int part = 0; part < C::H_PARTS; ++part) {
#pragma unroll
                    for (int kk = 0; kk < C::HC / 16; ++kk) {
                        const uint64_t ad = make_desc_sw128(h0 + (part * C::KP2 + (kk >> 2)) * C::H_PANEL + (kk & 3) * 32);
                        const uint64_t bd = make_desc_sw128(w0 + (kk >> 2) * C::W2_PANEL + (kk & 3) * 32);
                        mma_bf16_ss(tmem_base + 2 * C::HC + buf * C::N2, ad, bd, idesc2,
                                    (it.c > 0 || kk > 0 || part > 0) ? 1u : 0u);
                    }
                }
                mma_commit(bar(B::H_EMPTY + b));
                if (it.release) mma_commit(bar(B::W_EMPTY + slot));
                if (it.c == nchunks - 1) mma_commit(bar(B::ACC2_FULL + buf));
                return true;
            };

            Item nxt;
            nxt.t = t_begin; nxt.ta = 0; nxt.c = 0; nxt.e = 0; nxt.g = 0; nxt.valid = true;
            enter_tile(nxt, -1);
            ok = issue_g1(nxt);
            while (ok && nxt.valid) {
                const Item cur = nxt;
                advance(nxt);
                if (nxt.valid) ok = issue_g1(nxt);
                if (ok) ok = issue_g2(cur);
            }
            if (!ok || *abort) {
                // make sure no MMA is still running before TMEM is released
                volatile int never = 0;
                mma_commit(bar(B::DRAIN));
                mbar_wait(bar(B::DRAIN), 0u, &never, 10000000ull);
            }
        }
    } else {
        // ================= epilogue warps ====================================================
        const int ew = warp - 2;
        const int wg = ew >> 2;                       // column split
        const int lg = warp & 3;                      // TMEM lane group this warp may read
        const int row = lg * 32 + lane;               // row of the tile owned by this thread
        const uint32_t tmem_lane = tmem_base + ((uint32_t)(lg * 32) << 16);
        bool ok = true;
        int e = 0;
        uint32_t g = 0;
        for (int t = t_begin, ta = 0; t < t_end && ok; ++t, ++ta) {
            int row0, rows;
            locate_tile(tile_start, offs, t, e, row0, rows);
            for (int c = 0; c < nchunks && ok; ++c, ++g) {
                const uint32_t b = g & 1u, n1 = g >> 1;
                ok = mbar_wait(bar(B::ACC1_FULL + b), n1 & 1u, abort, kWaitLimitNs);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after_sync();
                uint32_t v[C::COLS1];
#pragma unroll
                for (int q = 0; q < C::COLS1 / 32; ++q)
                    tmem_ld_x32(tmem_lane + b * C::HC + wg * C::COLS1 + q * 32, v + q * 32);
                tmem_ld_wait();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(B::ACC1_EMPTY + b));
                // bias (same address for the whole warp: one broadcast load per 8 columns) +
                // activation, packed to bf16 pairs
                if (p.bias1) {
                    const bf16* gb = p.bias1 + (size_t)e * p.HID + c * C::HC + wg * C::COLS1;
#pragma unroll
                    for (int j = 0; j < C::COLS1; j += 8) {
                        float bb[8];
                        unpack16<bf16>(__ldg(reinterpret_cast<const uint4*>(gb + j)), bb);
#pragma unroll
                        for (int i = 0; i < 8; ++i) v[j + i] = __float_as_uint(__uint_as_float(v[j + i]) + bb[i]);
                    }
                }
                uint32_t packed[C::COLS1 / 2];
#pragma unroll
                for (int j = 0; j < C::COLS1; j += 2) {
                    const float a0 = activate<C::ACT>(__uint_as_float(v[j]));
                    const float a1 = activate<C::ACT>(__uint_as_float(v[j + 1]));
                    packed[j / 2] = pack_bf16x2(a0, a1);
                    if constexpr (C::H_PARTS == 2) {
                        // remainder after the bf16 rounding, itself rounded to bf16 (reuses v)
                        const float r0 = a0 - __uint_as_float(packed[j / 2] << 16);
                        const float r1 = a1 - __uint_as_float(packed[j / 2] & 0xFFFF0000u);
                        v[j / 2] = pack_bf16x2(r0, r1);
                    }
                }
                ok = mbar_wait(bar(B::H_EMPTY + b), (n1 & 1u) ^ 1u, abort, kWaitLimitNs);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                // hidden chunk -> shared memory, K-major rows of 64 bf16 with the 128-byte swizzle
                uint8_t* hrow = smem_gen + C::OFF_H + b * C::H_BYTES + (row >> 3) * 1024 + (row & 7) * 128;
#pragma unroll
                for (int q = 0; q < C::COLS1 / 8; ++q) {
                    const int col = wg * C::COLS1 + q * 8;
                    const int panel = col >> 6, j16 = (col & 63) >> 3;
                    uint4 val = make_uint4(packed[q * 4], packed[q * 4 + 1], packed[q * 4 + 2], packed[q * 4 + 3]);
                    *reinterpret_cast<uint4*>(hrow + panel * C::H_PANEL + ((j16 ^ (row & 7)) << 4)) = val;
                    if constexpr (C::H_PARTS == 2) {
                        uint4 lo = make_uint4(v[q * 4], v[q * 4 + 1], v[q * 4 + 2], v[q * 4 + 3]);
                        *reinterpret_cast<uint4*>(hrow + (C::KP2 + panel) * C::H_PANEL + ((j16 ^ (row & 7)) << 4)) = lo;
                    }
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(B::H_FULL + b));
            }
            if (!ok) break;
            // ---- final epilogue of the tile -----------------------------------------------
            const int buf = ta % C::ACC2_BUFS;
            ok = mbar_wait(bar(B::ACC2_FULL + buf), (uint32_t)(ta / C::ACC2_BUFS) & 1u, abort, kWaitLimitNs);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after_sync();
            const uint32_t acc2 = tmem_lane + 2 * C::HC + buf * C::N2;
            if constexpr (C::ROUTER) {
                constexpr int E = C::N2;
                uint32_t v[E];
                if (wg == 0) {
#pragma unroll
                    for (int q = 0; q < E / 16; ++q) tmem_ld_x16(acc2 + q * 16, v + q * 16);
                    tmem_ld_wait();
                }
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(B::ACC2_EMPTY + buf));
                if (wg == 0 && row < rows) {
                    float gl[E];
#pragma unroll
                    for (int i = 0; i < E; ++i)
                        gl[i] = __uint_as_float(v[i]) + (p.bias2 ? __bfloat162float(__ldg(p.bias2 + i)) : 0.0f);
                    const int n = row0 + row;
                    // top-k by repeated arg-max over the logits; ties go to the lower id
                    unsigned long long taken = 0ull;
                    float m = 0.0f;
                    int sel[8];
                    float gsel[8];
                    for (int j = 0; j < p.k; ++j) {
                        int best = -1;
                        float bv = 0.0f;
#pragma unroll
                        for (int i = 0; i < E; ++i) {
                            const bool free_i = !((taken >> i) & 1ull);
                            if (free_i && (best < 0 || gl[i] > bv)) { best = i; bv = gl[i]; }
                        }
                        taken |= 1ull << best;
                        sel[j] = best;
                        gsel[j] = bv;
                        if (j == 0) m = bv;
                    }
                    float sum = 0.0f;
#pragma unroll
                    for (int i = 0; i < E; ++i) sum += __expf(gl[i] - m);
                    const float inv = 1.0f / sum;
                    for (int j = 0; j < p.k; ++j) {
                        p.topk_idx[(size_t)n * p.k + j] = sel[j];
                        p.topk_p[(size_t)n * p.k + j] = __expf(gsel[j] - m) * inv;
                        atomicAdd(&hist[sel[j]], 1);
                    }
                    if (p.probs) {
                        float4* dst = reinterpret_cast<float4*>(p.probs + (size_t)n * E);
#pragma unroll
                        for (int i = 0; i < E; i += 4)
                            dst[i / 4] = make_float4(__expf(gl[i] - m) * inv, __expf(gl[i + 1] - m) * inv,
                                                     __expf(gl[i + 2] - m) * inv, __expf(gl[i + 3] - m) * inv);
                    }
                }
            } else {
                constexpr int COLS2 = C::N2 / C::EPI_WG;
                uint32_t v[COLS2];
#pragma unroll
                for (int q = 0; q < COLS2 / 16; ++q) tmem_ld_x16(acc2 + wg * COLS2 + q * 16, v + q * 16);
                tmem_ld_wait();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(B::ACC2_EMPTY + buf));
                if (row < rows) {
                    bf16* dst = p.yperm + (size_t)(row0 + row) * C::N2 + wg * COLS2;
#pragma unroll
                    for (int q = 0; q < COLS2 / 8; ++q) {
                        float bb[8];
                        if (p.bias2) {
                            unpack16<bf16>(__ldg(reinterpret_cast<const uint4*>(p.bias2 + (size_t)e * C::N2 + wg * COLS2 + q * 8)), bb);
                        } else {
#pragma unroll
                            for (int i = 0; i < 8; ++i) bb[i] = 0.0f;
                        }
                        uint32_t o[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i)
                            o[i] = pack_bf16x2(__uint_as_float(v[q * 8 + 2 * i]) + bb[2 * i],
                                               __uint_as_float(v[q * 8 + 2 * i + 1]) + bb[2 * i + 1]);
                        *reinterpret_cast<uint4*>(dst + q * 8) = make_uint4(o[0], o[1], o[2], o[3]);
                    }
                }
            }
        }
    }

    // ---- teardown -------------------------------------------------------------------------
    tc_fence_before_sync();
    __syncthreads();
    if (threadIdx.x == 0 && abort_flag) atomicExch(p.status, (int)SLICEMOE_ERR_DEVICE_TIMEOUT);
    if constexpr (C::ROUTER) {
        // per-CTA histogram -> global counts (Section 3.2's per-expert counts)
        for (int i = threadIdx.x; i < C::N2; i += C::THREADS)
            if (hist[i]) atomicAdd(&p.assigned[i], hist[i]);
    }
    if (warp == 1) {
        __syncwarp();
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, C::TMEM_COLS);
    }
}

// ---- host side --------------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = [] {
        void* f = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            f = nullptr;
        return reinterpret_cast<EncodeTiledFn>(f);
    }();
    return fn;
}

// bf16 matrix [rows, cols] row-major; box = 64 columns (128 bytes) x box_rows, 128-byte swizzle.
int make_tmap(CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return SLICEMOE_ERR_CUDA;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 2};
    const cuuint32_t box[2] = {64, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? SLICEMOE_OK : SLICEMOE_ERR_CUDA;
}

int sm_count() {
    static int n = [] {
        int dev = 0, v = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
            v = 148;
        return v;
    }();
    return n;
}

template <class C>
int launch_tc(const void* A, uint64_t a_rows, const void* W1, const void* W2, int n_experts, const TcParams& p,
              int max_tiles, cudaStream_t st) {
    CUtensorMap tmA, tmW1, tmW2;
    int rc;
    if ((rc = make_tmap(&tmA, A, a_rows, C::K1, 128))) return rc;
    if ((rc = make_tmap(&tmW1, W1, (uint64_t)n_experts * p.HID, C::K1, C::HC))) return rc;
    if ((rc = make_tmap(&tmW2, W2, (uint64_t)n_experts * C::N2, p.HID, C::N2))) return rc;
    auto kern = tc_mlp_kernel<C>;
    static bool attr_set = false;
    if (!attr_set) {
        SLICEMOE_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::SMEM_ALLOC));
        attr_set = true;
    }
    const int grid = max_tiles < sm_count() ? max_tiles : sm_count();
    kern<<<grid, C::THREADS, C::SMEM_ALLOC, st>>>(tmA, tmW1, tmW2, p);
    SLICEMOE_LAUNCH_CHECK(1);
    return SLICEMOE_OK;
}

template <int K1, int ACT>
int launch_ffn_k1(const Dims& D, const slicemoe_weights& w, const void* xperm, const TcParams& p, cudaStream_t st) {
    using C = TcCfg<K1, K1, false, ACT>;
    return launch_tc<C>(xperm, (uint64_t)D.R, w.W1, w.W2, D.E, p, max_tiles(D), st);
}

template <int K1, int E>
int launch_route_k1e(const Dims& D, const slicemoe_weights& w, const void* h, const TcParams& p, cudaStream_t st) {
    using C = TcCfg<K1, E, true, SLICEMOE_ACT_RELU>;
    return launch_tc<C>(h, (uint64_t)D.N, w.Wr1, w.Wr2, 1, p, (D.N + kTileM - 1) / kTileM, st);
}

template <int K1>
int launch_route_k1(const Dims& D, const slicemoe_weights& w, const void* h, const TcParams& p, cudaStream_t st) {
    switch (D.E) {
        case 16: return launch_route_k1e<K1, 16>(D, w, h, p, st);
        case 32: return launch_route_k1e<K1, 32>(D, w, h, p, st);
        case 64: return launch_route_k1e<K1, 64>(D, w, h, p, st);
        default: return SLICEMOE_ERR_UNSUPPORTED;
    }
}

}  // namespace

bool tc_route_supported(const Dims& D) {
    if (D.dtype != SLICEMOE_BF16) return false;
    if (D.ds != 64 && D.ds != 128 && D.ds != 256) return false;
    if (D.E != 16 && D.E != 32 && D.E != 64) return false;
    const int hc = D.ds == 64 ? 128 : 64;
    // at least two hidden chunks: the MMA warp issues GEMM-1 of the next chunk before GEMM-2 of the
    // current one, and with resident weights that look-ahead must not need the slot it is still using
    return D.Hr % hc == 0 && D.Hr >= 2 * hc && D.Hr <= kMaxHid && D.k <= 8;
}

bool tc_ffn_supported(const Dims& D) {
    if (D.dtype != SLICEMOE_BF16) return false;
    if (D.ds != 64 && D.ds != 128) return false;
    const int hc = D.ds == 64 ? 128 : 64;
    return D.F % hc == 0 && D.F >= 2 * hc && D.F <= kMaxHid;
}

int launch_route_tc(const Dims& D, const slicemoe_weights& w, const void* h, int32_t* topk_idx, float* topk_p,
                    int32_t* assigned, float* probs_opt, int32_t* status, cudaStream_t st) {
    SLICEMOE_CUDA_TRY(cudaMemsetAsync(assigned, 0, sizeof(int32_t) * D.E, st));
    if (D.N == 0) return SLICEMOE_OK;
    TcParams p{};
    p.offsets = nullptr; p.n_rows = D.N; p.E = 1; p.HID = D.Hr;
    p.bias1 = (const bf16*)w.br1; p.bias2 = (const bf16*)w.br2;
    p.topk_idx = topk_idx; p.topk_p = topk_p; p.assigned = assigned; p.probs = probs_opt; p.k = D.k;
    p.status = status;
    switch (D.ds) {
        case 64: return launch_route_k1<64>(D, w, h, p, st);
        case 128: return launch_route_k1<128>(D, w, h, p, st);
        case 256: return launch_route_k1<256>(D, w, h, p, st);
        default: return SLICEMOE_ERR_UNSUPPORTED;
    }
}

int launch_ffn_tc(const Dims& D, const slicemoe_weights& w, const void* xperm, const int32_t* offsets, void* yperm,
                  int32_t* status, cudaStream_t st) {
    if (D.R == 0) return SLICEMOE_OK;
    TcParams p{};
    p.offsets = offsets; p.n_rows = 0; p.E = D.E; p.HID = D.F;
    p.bias1 = (const bf16*)w.b1; p.bias2 = (const bf16*)w.b2;
    p.yperm = (bf16*)yperm; p.status = status;
    const bool gelu = D.act == SLICEMOE_ACT_GELU_TANH;
    if (D.ds == 64)
        return gelu ? launch_ffn_k1<64, SLICEMOE_ACT_GELU_TANH>(D, w, xperm, p, st)
                    : launch_ffn_k1<64, SLICEMOE_ACT_RELU>(D, w, xperm, p, st);
    if (D.ds == 128)
        return gelu ? launch_ffn_k1<128, SLICEMOE_ACT_GELU_TANH>(D, w, xperm, p, st)
                    : launch_ffn_k1<128, SLICEMOE_ACT_RELU>(D, w, xperm, p, st);
    return SLICEMOE_ERR_UNSUPPORTED;
}

}  // namespace slicemoe
