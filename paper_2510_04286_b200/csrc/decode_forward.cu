// Decode-shaped forward of the layer (Section 3.1, Eq. 1; Section 3.4): a few thousand 128-wide slices, so few
// that the step is bound by reading the expert weights once (E experts of 128 -> 512 -> 128, 256 KB each) and by
// latency rather than by arithmetic.  One cooperative launch, one CTA per SM:
//
//   router    the last ceil(N / 128) CTAs route one 128-row tile each on the tensor pipe: relu(X Wr1^T + br1)
//             Wr2^T + br2 -> softmax -> top-k, the hidden layer split into a bf16 pair per value so that the
//             logits keep fp32 accuracy.  Each pair (n, j) is appended with its gate to its expert's list with
//             one atomic per expert and warp.  A router CTA zeroes its rows of h'.
//   prefetch  CTA c < 2 E is the home of expert c % E: unless it routes, it streams the first half of that
//             expert's weights (128 KB) into shared memory while the router CTAs work
//   barrier   ONE grid barrier (bounded)
//   schedule  work items are 128-row tiles of one expert's list.  Every CTA derives the same assignment from
//             the E counts: tile 0 of expert e goes to CTA e, tile 1 to CTA E + e (their prefetched weights
//             fit), further tiles to CTAs without one, then round-robin.  A skewed router therefore costs
//             tiles on otherwise idle SMs, not a long tail on one.
//   experts   per item: the tile's rows of h copied into a swizzled A tile; the hidden layer in four chunks of 128
//             units through a two-slot weight ring: GEMM-1 (tcgen05, N = 128) into tensor memory, gate * acc +
//             b1 -> GELU/ReLU in fp32 -> bf16 hidden in place, GEMM-2 with the hidden chunk as its tensor-
//             memory operand accumulating over the chunks; 0.5 acc + b2 is added into row n of h' (two bf16
//             terms per row of h': the sum commutes, so the result does not depend on arrival order)
//
// Every wait is bounded; a run-out sets the status word and all roles leave.
#include <mutex>

#include "pp_body.cuh"

namespace slicemoe {
namespace {

constexpr int kDecThreads = 320;          // warps 0-7 workers, warp 8 weight loads, warp 9 MMA issue
constexpr int kDecWorkers = 256;
constexpr int kDecDs = 128, kDecF = 512, kDecHC = 128, kDecNC = kDecF / kDecHC, kDecHr = 256;
constexpr int kDecMaxE = 64;
// The per-expert list counters sit one per 128-byte line: the router CTAs' warps append at about the same time
// (thousands of atomics within a microsecond or two), and atomics on one line are served one after the other.
constexpr int kDecCountStride = 32;       // ints between two experts' counters
constexpr int kDecMaxItems = 16;          // items one CTA can take in one launch (N <= 4096: at most 96 tiles in all)

// shared memory (from a 1024-byte aligned base)
constexpr int kDecW1 = 0;                          // 2 slots x 2 K-panels of [128 rows x 128 B]; router: Wr1, 2 panels of [256 x 128 B]
constexpr int kDecW2 = 65536;                      // 2 slots x 2 K-panels of [128 rows x 128 B]; router: Wr2, 4 panels of [E x 128 B]
constexpr int kDecA = 131072;                      // 2 K-panels of [128 rows x 128 B]: the rows of a tile
constexpr int kDecSmem = 1024 + kDecA + 32768;

struct DecParams {
    const bf16* X;            // h as [N, 128]
    bf16* Y;                  // h' as [N, 128]
    const bf16 *Wr1, *br1, *Wr2, *br2, *b1, *b2;
    int32_t* topk_idx;
    float* topk_p;
    int32_t *assigned, *kept;
    int2* lists;              // [E][N] (pair index, gate bits), in arrival order
    int32_t* counts;          // [2][kDecMaxE] device words (kDecCountStride ints apart), used alternately by successive launches
    int32_t* status;
    unsigned long long* sync_word;
    int N, k, E, n_router;     // n_router: the last ceil(N / 128) CTAs route
    float softmax_scale;
    int clear_status;
};

struct DecShared {
    __align__(8) uint64_t bars[24];
    uint32_t tmem_base;
    int abort_flag;
    int n_items;
    int bias_e;               // the expert whose biases sit in bias1 / bias2 (-1: none)
    unsigned long long base;
    int item_e[kDecMaxItems], item_t[kDecMaxItems];
    int cnt[kDecMaxE];
    float br2[kDecMaxE];
    float xb1[kTileM], xb2[kTileM], xsum[kTileM];      // router: the upper column half's top two and sum, per row
    int xi1[kTileM], xi2[kTileM];
    uint16_t pair[kTileM];
    float gate[kTileM];
    __align__(16) float bias1[kDecF];
    __align__(16) float bias2[kDecDs];
};
namespace DB {
enum { W1_FULL = 0, W2_FULL = 2, W1_EMPTY = 4, W2_EMPTY = 6, A_FULL = 8, A_EMPTY = 9, ACC1_FULL = 10, HID_FULL = 12,
       ACC2_FULL = 14, ACC2_FREE = 15, R_FULL = 16, R_ACC1 = 17, R_HID = 18, R_ACC2 = 19, DRAIN = 20 };
}

__device__ unsigned long long g_dec_sync;
__device__ int32_t g_dec_counts[2 * kDecMaxE * kDecCountStride];

// Grid barrier on ONE monotonic 64-bit arrival counter: every launch adds gridDim.x to it, so the count a CTA
// finds at entry, rounded down to a multiple of gridDim.x, is this launch's base whichever CTAs have already
// arrived, and base + gridDim.x is the value to wait for.  One release-add and acquire polls: no last-arriver step.
__device__ __forceinline__ unsigned long long dec_barrier_base(unsigned long long* word) {
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(word) : "memory");
    return v - v % gridDim.x;
}
__device__ __forceinline__ bool dec_grid_barrier(unsigned long long* word, unsigned long long base, DecShared& sh) {
    fence_proxy_async_smem();
    __syncthreads();
    if (threadIdx.x == 0) {
        asm volatile("red.release.gpu.global.add.u64 [%0], 1;" ::"l"(word) : "memory");
        const unsigned long long target = base + gridDim.x;
        const uint64_t t0 = globaltimer_ns();
        for (;;) {
            unsigned long long v;
            asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(word) : "memory");
            if (v >= target) break;
            if (globaltimer_ns() - t0 > kWaitLimitNs) {
                sh.abort_flag = 1;
                break;
            }
        }
    }
    __syncthreads();
    return sh.abort_flag == 0;
}

// ---- router: 128 rows per router CTA on the tensor pipe ------------------------------------------------------
// The last ceil(N / 128) CTAs of the grid route one 128-row tile each (every CTA routing a few rows would have
// every SM read the router's 96 KB of weights: 15 MB through L2 for 0.4 GFLOP).  relu(X Wr1^T + br1) Wr2^T + br2
// -> softmax -> top-k: GEMM-1 (N = 256) into tensor memory; the fp32 hidden values are split in place into a
// truncated bf16 and the rounded remainder (ReLU rides on the conversions), so that the logits keep fp32
// accuracy; GEMM-2 takes both as tensor-memory operands.  Each pair (n, j) is appended with its gate to its
// expert's list: one atomic per expert and warp, both choices' atomics in flight together.
// Shared memory: Wr1 in the W1 ring's place, Wr2 in the W2 ring's, the rows in the A tile.
template <int E>
__device__ __forceinline__ void dec_route(const CUtensorMap* tmX, const CUtensorMap* tmWr1, const CUtensorMap* tmWr2,
                                          const DecParams& p, DecShared& sh, uint32_t smem_base, uint32_t tmem_base, int rt,
                                          int32_t* counts) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int* abort = &sh.abort_flag;
    auto bar = [&](int i) { return smem_u32(&sh.bars[i]); };
    const int row0 = rt * kTileM;
    const int rows = min(kTileM, p.N - row0);
    constexpr uint32_t kWr2Panel = E * 128;            // bytes of one 64-column panel of Wr2
    if (warp == 8) {
        if (lane == 0) {
            mbar_arrive_expect_tx(bar(DB::R_FULL), 65536u + 4u * kWr2Panel + 32768u);
            for (int j = 0; j < 2; ++j) tma_load_2d(smem_base + kDecA + j * 16384, tmX, 64 * j, row0, bar(DB::R_FULL));
            for (int j = 0; j < 2; ++j) tma_load_2d(smem_base + kDecW1 + j * 32768, tmWr1, 64 * j, 0, bar(DB::R_FULL));
            for (int j = 0; j < 4; ++j) tma_load_2d(smem_base + kDecW2 + j * kWr2Panel, tmWr2, 64 * j, 0, bar(DB::R_FULL));
        }
        __syncwarp();
    } else if (warp == 9) {
        constexpr uint32_t idesc1 = make_idesc(128, kDecHr, kFmtBF16, kFmtBF16);
        constexpr uint32_t idesc2 = make_idesc(128, E, kFmtBF16, kFmtBF16);
        const uint32_t dA = desc_lo_sw128(smem_base + kDecA), dW1 = desc_lo_sw128(smem_base + kDecW1),
                       dW2 = desc_lo_sw128(smem_base + kDecW2);
        bool ok = pp_wait(bar(DB::R_FULL), 0u, abort);
        if (ok) {
            tc_fence_after_sync();
            if (elect_one_sync()) {
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)
                    mma_ss_dyn(tmem_base, dA + (((kk >> 2) * 16384 + (kk & 3) * 32) >> 4),
                               dW1 + (((kk >> 2) * 32768 + (kk & 3) * 32) >> 4), idesc1, kk > 0 ? 1u : 0u);
                mma_commit(bar(DB::R_ACC1));
            }
            __syncwarp();
            ok = pp_wait(bar(DB::R_HID), 0u, abort);
        }
        if (ok) {
            tc_fence_after_sync();
            if (elect_one_sync()) {
                // piece pc = hidden units [16 pc, +16): truncated halves in columns 16 pc .. +7, remainders in +8 .. +15
#pragma unroll
                for (int pc = 0; pc < kDecHr / 16; ++pc) {
                    const uint32_t b = dW2 + (((pc >> 2) * kWr2Panel + (pc & 3) * 32) >> 4);
                    mma_ts_dyn(tmem_base + 256, tmem_base + 16 * pc, b, idesc2, pc > 0 ? 1u : 0u);
                    mma_ts_dyn(tmem_base + 256, tmem_base + 16 * pc + 8, b, idesc2, 1u);
                }
                mma_commit(bar(DB::R_ACC2));
            }
            __syncwarp();
            // (the workers wait for R_ACC2: the ring's regions are free again when they leave)
        }
    } else {
        const int lg = warp & 3, g = warp >> 2;
        const int row = lg * 32 + lane;
        const uint32_t tlane = tmem_base + ((uint32_t)(lg * 32) << 16);
        // biases as fp32; zeros into my rows of h'
        sh.bias1[threadIdx.x] = p.br1 ? __bfloat162float(p.br1[threadIdx.x]) : 0.0f;
        if (threadIdx.x < E) sh.br2[threadIdx.x] = p.br2 ? __bfloat162float(p.br2[threadIdx.x]) : 0.0f;
        for (int c = threadIdx.x; c < rows * 16; c += kDecWorkers)
            *reinterpret_cast<uint4*>(p.Y + (size_t)row0 * kDecDs + (size_t)c * 8) = make_uint4(0u, 0u, 0u, 0u);
        named_barrier_sync(1, kDecWorkers);
        bool ok = pp_wait(bar(DB::R_ACC1), 0u, abort);
        if (ok) {
            tc_fence_after_sync();
            const uint32_t base = tlane + 128 * g;
            uint32_t v[2][16];
            tmem_ld_x16(base, v[0]);
#pragma unroll
            for (int pc = 0; pc < 8; ++pc) {
                uint32_t* cur = v[pc & 1];
                tmem_ld_wait();
                if (pc + 1 < 8) tmem_ld_x16(base + (pc + 1) * 16, v[(pc + 1) & 1]);
                uint32_t hi[8], lo[8];
                bias_relu_split_piece(cur, sh.bias1 + 128 * g + pc * 16, hi, lo);
                tmem_st_x8(base + pc * 16, hi);
                tmem_st_x8(base + pc * 16 + 8, lo);
            }
            tmem_st_wait();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(DB::R_HID));
            ok = pp_wait(bar(DB::R_ACC2), 0u, abort);
        }
        // softmax + top-k of a row (ties go to the lower id): the two threads of a row (one per column half) each
        // keep the best two of E / 2 logits and the sum of exponentials about their own maximum; the thread of
        // the upper half hands its result over through shared memory
        float b1 = -INFINITY, b2 = -INFINITY, sum = 0.0f;
        int i1 = 0, i2 = 0;
        const float sc = p.softmax_scale;
        if (ok) {
            tc_fence_after_sync();
            constexpr int HE = E / 2;
            uint32_t v[HE];
#pragma unroll
            for (int c = 0; c < HE; c += 8) tmem_ld_x8(tlane + 256 + g * HE + c, v + c);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < HE; ++i) {
                const float gl = __uint_as_float(v[i]) + sh.br2[g * HE + i];
                v[i] = __float_as_uint(gl);
                const bool gt1 = gl > b1, gt2 = gl > b2;
                b2 = gt1 ? b1 : (gt2 ? gl : b2);
                i2 = gt1 ? i1 : (gt2 ? g * HE + i : i2);
                b1 = gt1 ? gl : b1;
                i1 = gt1 ? g * HE + i : i1;
            }
            const float msc = b1 * sc;
#pragma unroll
            for (int i = 0; i < HE; ++i) sum += ex2_approx(fmaf(__uint_as_float(v[i]), sc, -msc));
            if (g == 1) {
                sh.xb1[row] = b1; sh.xb2[row] = b2; sh.xi1[row] = i1; sh.xi2[row] = i2; sh.xsum[row] = sum;
            }
        }
        named_barrier_sync(1, kDecWorkers);
        if (ok && g == 0) {
            const float o1 = sh.xb1[row], o2 = sh.xb2[row], osum = sh.xsum[row];
            const int oi1 = sh.xi1[row], oi2 = sh.xi2[row];
            // (every id of the upper half is larger than every id of the lower half: the upper half wins only if strictly greater)
            const bool up = o1 > b1;
            const float w1 = up ? o1 : b1, l1 = up ? b1 : o1, w2 = up ? o2 : b2;
            const int wi1 = up ? oi1 : i1, li1 = up ? i1 : oi1, wi2 = up ? oi2 : i2;
            const bool sec = l1 > w2 || (l1 == w2 && li1 < wi2);
            sum = up ? fmaf(sum, ex2_approx((b1 - o1) * sc), osum) : fmaf(osum, ex2_approx((o1 - b1) * sc), sum);
            b1 = w1; i1 = wi1;
            b2 = sec ? l1 : w2; i2 = sec ? li1 : wi2;
            const float msc = b1 * sc;
            const float inv = 1.0f / sum;
            const float p2 = ex2_approx(fmaf(b2, sc, -msc)) * inv;
            const bool on = row < rows;
            if (on) {
                const size_t at = (size_t)(row0 + row) * p.k;
                p.topk_idx[at] = i1;
                p.topk_p[at] = inv;
                if (p.k > 1) {
                    p.topk_idx[at + 1] = i2;
                    p.topk_p[at + 1] = p2;
                }
            }
            int e[2], base[2], leader[2];
            uint32_t m[2];
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                e[j] = (on && j < p.k) ? (j ? i2 : i1) : -1 - lane;
                m[j] = __match_any_sync(0xffffffffu, e[j]);
                leader[j] = __ffs(m[j]) - 1;
                base[j] = 0;
                if (e[j] >= 0 && lane == leader[j]) base[j] = atomicAdd(counts + e[j] * kDecCountStride, __popc(m[j]));
            }
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                base[j] = __shfl_sync(0xffffffffu, base[j], leader[j]);
                if (e[j] >= 0)
                    p.lists[(size_t)e[j] * p.N + base[j] + __popc(m[j] & ((1u << lane) - 1u))] =
                        make_int2((row0 + row) * p.k + j, __float_as_int(j ? p2 : inv));
            }
        }
        tc_fence_before_sync();
    }
}

// ---- schedule: this CTA's items from the E counts (the same function of the counts in every CTA) -------------
// lane l of warp 0 holds experts l and l + 32
template <int E>
__device__ __forceinline__ void dec_schedule(DecShared& sh, int lane) {
    const int G = (int)gridDim.x, c = (int)blockIdx.x;
    const int e0 = lane, e1 = lane + 32;
    const int nt0 = e0 < E ? (sh.cnt[e0] + kTileM - 1) / kTileM : 0, nt1 = e1 < E ? (sh.cnt[e1] + kTileM - 1) / kTileM : 0;
    // exclusive prefix over the experts (lanes' first experts, then their second ones) and the total
    auto scan2 = [&](int a, int b, int& ea, int& eb, int& total) {
        int s = a;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int o = __shfl_up_sync(0xffffffffu, s, d);
            if (lane >= d) s += o;
        }
        const int tot_a = __shfl_sync(0xffffffffu, s, 31);
        int s2 = b;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int o = __shfl_up_sync(0xffffffffu, s2, d);
            if (lane >= d) s2 += o;
        }
        ea = s - a;
        eb = tot_a + s2 - b;
        total = tot_a + __shfl_sync(0xffffffffu, s2, 31);
    };
    int ov_pre0, ov_pre1, O;            // tiles past the first two, in (e, t) order
    scan2(nt0 > 2 ? nt0 - 2 : 0, nt1 > 2 ? nt1 - 2 : 0, ov_pre0, ov_pre1, O);
    int lt2_pre0, lt2_pre1, n_lt2;      // experts whose second home CTA has no tile
    scan2((e0 < E && nt0 < 2) ? 1 : 0, (e1 < E && nt1 < 2) ? 1 : 0, lt2_pre0, lt2_pre1, n_lt2);
    int lt1_pre0, lt1_pre1, n_lt1;      // experts whose first home CTA has no tile
    scan2((e0 < E && nt0 < 1) ? 1 : 0, (e1 < E && nt1 < 1) ? 1 : 0, lt1_pre0, lt1_pre1, n_lt1);
    // this CTA: its own tile, or its rank among the CTAs without one (spare CTAs first, then second homes, then first homes)
    int own_e = -1, own_t = 0, free_rank = -1;
    const int spare = G > 2 * E ? G - 2 * E : 0;
    if (c >= 2 * E) {
        free_rank = c - 2 * E;
    } else {
        const int he = c % E, second = c >= E ? 1 : 0;
        const int src = he & 31;
        const int nt_h = __shfl_sync(0xffffffffu, he < 32 ? nt0 : nt1, src);
        const int p2 = __shfl_sync(0xffffffffu, he < 32 ? lt2_pre0 : lt2_pre1, src);
        const int p1 = __shfl_sync(0xffffffffu, he < 32 ? lt1_pre0 : lt1_pre1, src);
        if (nt_h > second) { own_e = he; own_t = second; }
        else free_rank = second ? spare + p2 : spare + n_lt2 + p1;
    }
    const int NF = spare + n_lt2 + n_lt1;
    // overflow tile x -> (e, t): the lane whose expert's range holds x answers
    auto locate = [&](int x, int& e, int& t) {
        const bool in0 = x >= ov_pre0 && x < ov_pre0 + (nt0 > 2 ? nt0 - 2 : 0);
        const bool in1 = x >= ov_pre1 && x < ov_pre1 + (nt1 > 2 ? nt1 - 2 : 0);
        const uint32_t m = __ballot_sync(0xffffffffu, in0 || in1);
        const int src = __ffs(m) - 1;
        const int ee = in0 ? e0 : e1, tt = 2 + x - (in0 ? ov_pre0 : ov_pre1);
        e = __shfl_sync(0xffffffffu, ee, src);
        t = __shfl_sync(0xffffffffu, tt, src);
    };
    int n = 0;
    if (own_e >= 0) {
        if (lane == 0) { sh.item_e[n] = own_e; sh.item_t[n] = own_t; }
        ++n;
    }
    if (free_rank >= 0 && free_rank < O) {
        int e, t;
        locate(free_rank, e, t);
        if (lane == 0) { sh.item_e[n] = e; sh.item_t[n] = t; }
        ++n;
    }
    for (int x = NF + c; x < O && n < kDecMaxItems; x += G) {
        int e, t;
        locate(x, e, t);
        if (lane == 0) { sh.item_e[n] = e; sh.item_t[n] = t; }
        ++n;
    }
    if (lane == 0) sh.n_items = n;
}

template <int E, int ACT>
__global__ void __launch_bounds__(kDecThreads, 1)
decode_forward_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmWr1,
                      const __grid_constant__ CUtensorMap tmWr2, const __grid_constant__ CUtensorMap tmW1,
                      const __grid_constant__ CUtensorMap tmW2, const DecParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ DecShared sh;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));
    const int home = (int)blockIdx.x < 2 * E ? (int)blockIdx.x % E : -1;
    const int rt = (int)blockIdx.x - ((int)gridDim.x - p.n_router);      // >= 0: this CTA routes rows [128 rt, +128)
    volatile int* abort = &sh.abort_flag;
    auto bar = [&](int i) { return smem_u32(&sh.bars[i]); };

    if (threadIdx.x == 0) {
        sh.base = dec_barrier_base(p.sync_word);
        if (blockIdx.x == 0 && p.clear_status) *p.status = SLICEMOE_OK;
        sh.abort_flag = 0;
        sh.n_items = 0;
        sh.bias_e = -1;
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar(DB::W1_FULL + b), 1);
            mbar_init(bar(DB::W2_FULL + b), 1);
            mbar_init(bar(DB::W1_EMPTY + b), 1);
            mbar_init(bar(DB::W2_EMPTY + b), 1);
            mbar_init(bar(DB::ACC1_FULL + b), 1);
            mbar_init(bar(DB::HID_FULL + b), 8);
        }
        mbar_init(bar(DB::A_FULL), 1);
        mbar_init(bar(DB::A_EMPTY), 1);
        mbar_init(bar(DB::ACC2_FULL), 1);
        mbar_init(bar(DB::ACC2_FREE), 8);
        mbar_init(bar(DB::R_FULL), 1);
        mbar_init(bar(DB::R_ACC1), 1);
        mbar_init(bar(DB::R_HID), 8);
        mbar_init(bar(DB::R_ACC2), 1);
        mbar_init(bar(DB::DRAIN), 1);
        fence_mbar_init();
    }
    if (warp == 9) {
        tmem_alloc(smem_u32(&sh.tmem_base), 512);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = sh.tmem_base;
    const unsigned long long base = sh.base;
    // successive launches alternate between two sets of counters: this one's were zeroed by the previous launch
    const int parity = (int)((base / gridDim.x) & 1ull);
    int32_t* counts = p.counts + parity * (kDecMaxE * kDecCountStride);

    // weights of chunk c of expert e into ring slot s (W1: rows [128 c, +128) of W1_e; W2: columns [128 c, +128) of W2_e)
    auto load_w1 = [&](int e, int c, int s) {
        mbar_arrive_expect_tx(bar(DB::W1_FULL + s), 32768u);
        for (int j = 0; j < 2; ++j)
            tma_load_2d(smem_base + kDecW1 + s * 32768 + j * 16384, &tmW1, 64 * j, e * kDecF + c * kDecHC, bar(DB::W1_FULL + s));
    };
    auto load_w2 = [&](int e, int c, int s) {
        mbar_arrive_expect_tx(bar(DB::W2_FULL + s), 32768u);
        for (int j = 0; j < 2; ++j)
            tma_load_2d(smem_base + kDecW2 + s * 32768 + j * 16384, &tmW2, c * kDecHC + 64 * j, e * kDecDs, bar(DB::W2_FULL + s));
    };

    if (warp == 8 && blockIdx.x == 0) {
        // (nobody uses the other counter set during this launch)
        int32_t* other = p.counts + (parity ^ 1) * (kDecMaxE * kDecCountStride);
        for (int i = lane; i < kDecMaxE; i += 32) other[i * kDecCountStride] = 0;
    }
    if (warp == 8 && lane == 0) {
        prefetch_tensormap(&tmW1);
        prefetch_tensormap(&tmW2);
    }
    const bool prefetched = home >= 0 && rt < 0;
    if (rt >= 0) {
        dec_route<E>(&tmX, &tmWr1, &tmWr2, p, sh, smem_base, tmem_base, rt, counts);
    } else if (warp == 8) {
        if (prefetched && lane == 0) {
            // the home expert's first two chunks
            load_w1(home, 0, 0);
            load_w2(home, 0, 0);
            load_w1(home, 1, 1);
            load_w2(home, 1, 1);
        }
        __syncwarp();
    } else if (warp == 9 && prefetched) {
        // and its biases, as fp32
        for (int i = lane; i < kDecF; i += 32) sh.bias1[i] = p.b1 ? __bfloat162float(p.b1[(size_t)home * kDecF + i]) : 0.0f;
        for (int i = lane; i < kDecDs; i += 32) sh.bias2[i] = p.b2 ? __bfloat162float(p.b2[(size_t)home * kDecDs + i]) : 0.0f;
        if (lane == 0) sh.bias_e = home;
    }

    bool ok = dec_grid_barrier(p.sync_word, base, sh);

    // ---- schedule ----------------------------------------------------------------------------------------
    if (ok && threadIdx.x < E) sh.cnt[threadIdx.x] = __ldcg(counts + threadIdx.x * kDecCountStride);
    __syncthreads();
    if (ok && warp == 0) dec_schedule<E>(sh, lane);
    if (ok && blockIdx.x == 0 && threadIdx.x >= 64 && threadIdx.x < 64 + E) {
        const int e = threadIdx.x - 64;
        if (p.assigned) p.assigned[e] = sh.cnt[e];
        if (p.kept) p.kept[e] = sh.cnt[e];
    }
    __syncthreads();
    const int n_items = ok ? sh.n_items : 0;
    const int kshift = p.k - 1;          // k is 1 or 2
    // the prefetched chunks serve the first item if it belongs to the home expert; otherwise those two fills of
    // the ring are discarded (the ring's "full" barriers then run one phase ahead)
    const bool wasted = prefetched && !(n_items > 0 && sh.item_e[0] == home);
    const int fill_shift = wasted ? 1 : 0;

    if (warp < 8) {
        // ================= workers: tile list, gathers, activation, output ==================================
        const int lg = warp & 3, g = warp >> 2;
        const int row = lg * 32 + lane;
        const uint32_t tlane = tmem_base + ((uint32_t)(lg * 32) << 16);
        bool wok = true;
        int bias_e = sh.bias_e;               // (written before the grid barrier; every worker keeps its own copy from here on)
        for (int it = 0; it < n_items && wok; ++it) {
            const int e = sh.item_e[it], t = sh.item_t[it];
            const int rows = min(kTileM, sh.cnt[e] - t * kTileM);
            // The tile's rows of h: two threads per row, each copies one 64-column panel (eight 16-byte pieces)
            // into the 128-byte-swizzled A tile.  (Four-row TMA gathers take the copy engine ~60 cycles each:
            // 64 of them were 2-3 us here; plain loads from L2 are all in flight at once.)
            if (it > 0 && !pp_wait(bar(DB::A_EMPTY), (uint32_t)(it - 1) & 1u, abort)) { wok = false; break; }
            {
                // this expert's biases as fp32, unless they are there already (requested first: their latency
                // runs under the two dependent round trips below)
                const bool need_bias = bias_e != e;
                bias_e = e;
                float bv[3] = {0.0f, 0.0f, 0.0f};
                if (need_bias) {
                    if (p.b1) {
                        bv[0] = __bfloat162float(p.b1[(size_t)e * kDecF + threadIdx.x]);
                        bv[1] = __bfloat162float(p.b1[(size_t)e * kDecF + kDecWorkers + threadIdx.x]);
                    }
                    if (p.b2 && threadIdx.x < kDecDs) bv[2] = __bfloat162float(p.b2[(size_t)e * kDecDs + threadIdx.x]);
                }
                const int r = threadIdx.x >> 1, half = threadIdx.x & 1;
                if (r < rows) {
                    const int2 ent = __ldcg(p.lists + (size_t)e * p.N + t * kTileM + r);
                    const uint4* src = reinterpret_cast<const uint4*>(p.X + (size_t)(ent.x >> kshift) * kDecDs + half * 64);
                    uint4 v[8];
#pragma unroll
                    for (int c = 0; c < 8; ++c) v[c] = __ldg(src + c);
                    uint8_t* dst = smem + kDecA + half * 16384 + r * 128;
#pragma unroll
                    for (int c = 0; c < 8; ++c) *reinterpret_cast<uint4*>(dst + ((c ^ (r & 7)) << 4)) = v[c];
                    if (half == 0) {
                        sh.pair[r] = (uint16_t)ent.x;
                        sh.gate[r] = __int_as_float(ent.y);
                    }
                } else if (half == 0) {
                    sh.pair[r] = 0;
                    sh.gate[r] = 0.0f;
                }
                if (need_bias) {
                    sh.bias1[threadIdx.x] = bv[0];
                    sh.bias1[kDecWorkers + threadIdx.x] = bv[1];
                    if (threadIdx.x < kDecDs) sh.bias2[threadIdx.x] = bv[2];
                }
            }
            fence_proxy_async_smem();          // the tensor pipe reads the tile through the async proxy
            named_barrier_sync(1, kDecWorkers);
            if (threadIdx.x == 0) mbar_arrive(bar(DB::A_FULL));
            const float gs = sh.gate[row];
            const bool has_b1 = p.b1 != nullptr;
            const bool live = lg * 32 < rows;        // a warp whose 32 rows are all padding only passes the hand-offs on
            for (int c = 0; c < kDecNC && wok; ++c) {
                const int cc = it * kDecNC + c, r = cc & 1;
                if (!pp_wait(bar(DB::ACC1_FULL + r), (uint32_t)(cc >> 1) & 1u, abort)) { wok = false; break; }
                tc_fence_after_sync();
                if (live) {
                    // the thread's 64 hidden units of the chunk, eight at a time as a software pipeline around the tanh
                    // unit (pre of piece j + 1 and post of piece j - 1 under the tanh of piece j); two pieces per
                    // tensor-memory load and store; no shared-memory bias reads without a first-layer bias
                    const uint32_t region = tlane + r * kDecHC + 64 * g;
                    const float* bias = sh.bias1 + c * kDecHC + 64 * g;
                    uint32_t acc[16], hid[8];
                    float z[2][8], u[2][8];
                    tmem_ld_x16(region, acc);
                    tmem_ld_wait();
                    pp_pre8<ACT>(acc, gs, bias, has_b1, z[0], u[0]);
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        pp_tanh8<ACT>(u[j & 1]);
                        if (j + 1 < 8) {
                            if (((j + 1) & 1) == 0) tmem_ld_wait();
                            pp_pre8<ACT>(acc + 8 * ((j + 1) & 1), gs, bias + 8 * (j + 1), has_b1, z[(j + 1) & 1], u[(j + 1) & 1]);
                            if (((j + 1) & 1) == 1 && j + 2 < 8) tmem_ld_x16(region + 8 * (j + 2), acc);
                        }
                        pp_post8<ACT>(z[j & 1], u[j & 1], hid + 4 * (j & 1));
                        if (j & 1) tmem_st_x8(region + 4 * (j - 1), hid);
                    }
                    tmem_st_wait();
                }
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(DB::HID_FULL + r));
            }
            if (!wok) break;
            if (!pp_wait(bar(DB::ACC2_FULL), (uint32_t)it & 1u, abort)) { wok = false; break; }
            tc_fence_after_sync();
            uint32_t v[64];
            if (live) {
                const uint32_t acc2 = tlane + 2 * kDecHC + 64 * g;
#pragma unroll
                for (int q = 0; q < 4; ++q) tmem_ld_x16(acc2 + 16 * q, v + 16 * q);
                tmem_ld_wait();
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(DB::ACC2_FREE));
            if (row < rows) {
                bf16* dst = p.Y + (size_t)((int)sh.pair[row] >> kshift) * kDecDs + 64 * g;
                const float* b2 = sh.bias2 + 64 * g;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    uint32_t o[4];
                    if (p.b2) {
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            o[j] = pack_bf16x2(fmaf(__uint_as_float(v[8 * i + 2 * j]), kOutScale<ACT>, b2[8 * i + 2 * j]),
                                               fmaf(__uint_as_float(v[8 * i + 2 * j + 1]), kOutScale<ACT>, b2[8 * i + 2 * j + 1]));
                    } else {
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            o[j] = pack_bf16x2(__uint_as_float(v[8 * i + 2 * j]) * kOutScale<ACT>, __uint_as_float(v[8 * i + 2 * j + 1]) * kOutScale<ACT>);
                    }
                    red_add_bf16x8(dst + 8 * i, o[0], o[1], o[2], o[3]);
                }
            }
            // (the next item rewrites the pair / gate / bias arrays: all workers are past them after this)
            named_barrier_sync(1, kDecWorkers);
        }
    } else if (warp == 8) {
        // ================= weight ring producer =============================================================
        // chunk n = 4 it + c goes to slot n & 1; it may be loaded once the chunk two before it has been consumed
        bool pok = true;
        if (wasted) {
            // let the discarded fills land before their slots are refilled
            pok = pp_wait(bar(DB::W1_FULL + 0), 0u, abort) && pp_wait(bar(DB::W2_FULL + 0), 0u, abort) &&
                  pp_wait(bar(DB::W1_FULL + 1), 0u, abort) && pp_wait(bar(DB::W2_FULL + 1), 0u, abort);
        }
        for (int it = 0; it < n_items && pok; ++it) {
            const int e = sh.item_e[it];
            for (int c = 0; c < kDecNC && pok; ++c) {
                const int n = it * kDecNC + c, s = n & 1;
                if (n < 2 && prefetched && !wasted) continue;          // already in the ring
                if (n >= 2) pok = pp_wait(bar(DB::W1_EMPTY + s), (uint32_t)((n >> 1) - 1) & 1u, abort);
                if (pok && lane == 0) load_w1(e, c, s);
                __syncwarp();
                if (n >= 2 && pok) pok = pp_wait(bar(DB::W2_EMPTY + s), (uint32_t)((n >> 1) - 1) & 1u, abort);
                if (pok && lane == 0) load_w2(e, c, s);
                __syncwarp();
            }
        }
        if ((n_items == 0 || !pok || *abort) && prefetched) {
            // a CTA that leaves early still lets its prefetch land first
            volatile int never = 0;
            for (int s = 0; s < 2; ++s) {
                mbar_wait(bar(DB::W1_FULL + s), 0u, &never, 100000000ull);
                mbar_wait(bar(DB::W2_FULL + s), 0u, &never, 100000000ull);
            }
        }
    } else {
        // ================= MMA issue ========================================================================
        constexpr uint32_t idesc = make_idesc(128, 128, kFmtBF16, kFmtBF16);
        const uint32_t dA = desc_lo_sw128(smem_base + kDecA), dW1 = desc_lo_sw128(smem_base + kDecW1),
                       dW2 = desc_lo_sw128(smem_base + kDecW2);
        bool mok = true;
        auto full_parity = [&](int n) { return (uint32_t)((n >> 1) + fill_shift) & 1u; };
        auto gemm1 = [&](int it, int c) -> bool {
            const int n = it * kDecNC + c, s = n & 1;
            if (c == 0 && !pp_wait(bar(DB::A_FULL), (uint32_t)it & 1u, abort)) return false;
            if (!pp_wait(bar(DB::W1_FULL + s), full_parity(n), abort)) return false;
            tc_fence_after_sync();
            const uint32_t d = tmem_base + s * kDecHC;
            if (elect_one_sync()) {
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {
                    const uint32_t off = ((kk >> 2) * 16384 + (kk & 3) * 32) >> 4;
                    mma_ss_dyn(d, dA + off, dW1 + ((s * 32768) >> 4) + off, idesc, kk > 0 ? 1u : 0u);
                }
                mma_commit(bar(DB::ACC1_FULL + s));
                mma_commit(bar(DB::W1_EMPTY + s));
                if (c == kDecNC - 1) mma_commit(bar(DB::A_EMPTY));
            }
            __syncwarp();
            return true;
        };
        auto gemm2 = [&](int it, int c) -> bool {
            const int n = it * kDecNC + c, s = n & 1;
            if (c == 0 && it > 0 && !pp_wait(bar(DB::ACC2_FREE), (uint32_t)(it - 1) & 1u, abort)) return false;
            if (!pp_wait(bar(DB::W2_FULL + s), full_parity(n), abort)) return false;
            if (!pp_wait(bar(DB::HID_FULL + s), (uint32_t)(n >> 1) & 1u, abort)) return false;
            tc_fence_after_sync();
            const uint32_t hid = tmem_base + s * kDecHC, d2 = tmem_base + 2 * kDecHC;
            if (elect_one_sync()) {
                // K step u = hidden units [16 u, +16) of the chunk = packed columns 64 (u / 4) + 8 (u % 4)
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const uint32_t off = ((u >> 2) * 16384 + (u & 3) * 32) >> 4;
                    mma_ts_dyn(d2, hid + 64 * (u >> 2) + 8 * (u & 3), dW2 + ((s * 32768) >> 4) + off, idesc, (c > 0 || u > 0) ? 1u : 0u);
                }
                mma_commit(bar(DB::W2_EMPTY + s));
                if (c == kDecNC - 1) mma_commit(bar(DB::ACC2_FULL));
            }
            __syncwarp();
            return true;
        };
        for (int it = 0; it < n_items && mok; ++it) {
            // GEMM-1 runs one chunk ahead of GEMM-2; the tensor pipe executes them in issue order, so a GEMM-1 never
            // overwrites a hidden chunk that an earlier GEMM-2 still reads
            mok = gemm1(it, 0);
            for (int c = 0; c < kDecNC && mok; ++c) {
                if (c + 1 < kDecNC) mok = gemm1(it, c + 1);
                if (mok) mok = gemm2(it, c);
            }
        }
        if (!mok || *abort) {
            volatile int never = 0;
            if (lane == 0) {
                mma_commit(bar(DB::DRAIN));
                mbar_wait(bar(DB::DRAIN), 0u, &never, 10000000ull);
            }
            __syncwarp();
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (threadIdx.x == 0 && (sh.abort_flag || !ok)) atomicExch(p.status, (int)SLICEMOE_ERR_DEVICE_TIMEOUT);
    if (warp == 9) {
        __syncwarp();
        tmem_dealloc(tmem_base, 512);
    }
}

std::mutex g_dec_mutex;
unsigned long long* g_dec_sync_addr[kAttrMaxDevices] = {};
int32_t* g_dec_counts_addr[kAttrMaxDevices] = {};
bool g_dec_attr[8][kAttrMaxDevices] = {};

int dec_device_words(unsigned long long** sync, int32_t** counts) {
    int dev = -1;
    SLICEMOE_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kAttrMaxDevices) return SLICEMOE_ERR_NO_DEVICE;
    std::lock_guard<std::mutex> lock(g_dec_mutex);
    if (!g_dec_sync_addr[dev]) {
        void *q = nullptr, *c = nullptr;
        SLICEMOE_CUDA_TRY(cudaGetSymbolAddress(&q, g_dec_sync));
        SLICEMOE_CUDA_TRY(cudaGetSymbolAddress(&c, g_dec_counts));
        if (!q || !c) return SLICEMOE_ERR_CUDA;
        g_dec_sync_addr[dev] = static_cast<unsigned long long*>(q);
        g_dec_counts_addr[dev] = static_cast<int32_t*>(c);
    }
    *sync = g_dec_sync_addr[dev];
    *counts = g_dec_counts_addr[dev];
    return SLICEMOE_OK;
}

template <int E, int ACT>
int dec_launch(const Dims& D, const slicemoe_weights& w, const void* h, const DecParams& p, int grid, cudaStream_t st) {
    CUtensorMap mX, mWr1, mWr2, mW1, mW2;
    int rc;
    if ((rc = make_tmap(&mX, h, (uint64_t)D.N, (uint64_t)kDecDs, kTileM))) return rc;
    if ((rc = make_tmap(&mWr1, w.Wr1, (uint64_t)kDecHr, (uint64_t)kDecDs, kDecHr))) return rc;
    if ((rc = make_tmap(&mWr2, w.Wr2, (uint64_t)D.E, (uint64_t)kDecHr, E))) return rc;
    if ((rc = make_tmap(&mW1, w.W1, (uint64_t)D.E * kDecF, (uint64_t)kDecDs, kDecHC))) return rc;
    if ((rc = make_tmap(&mW2, w.W2, (uint64_t)D.E * kDecDs, (uint64_t)kDecF, kDecDs))) return rc;
    auto kern = decode_forward_kernel<E, ACT>;
    constexpr int slot = (E == 16 ? 0 : E == 32 ? 1 : 2) * 2 + (ACT == SLICEMOE_ACT_RELU ? 0 : 1);
    {
        std::lock_guard<std::mutex> lock(g_dec_mutex);
        if ((rc = set_smem_limit_once(kern, kDecSmem, g_dec_attr[slot]))) return rc;
    }
    cudaLaunchConfig_t lc{};
    lc.gridDim = dim3(grid);
    lc.blockDim = dim3(kDecThreads);
    lc.dynamicSmemBytes = kDecSmem;
    lc.stream = st;
    cudaLaunchAttribute attrs[1];
    attrs[0].id = cudaLaunchAttributeCooperative;   // all CTAs resident at once (they meet at a grid barrier)
    attrs[0].val.cooperative = 1;
    lc.attrs = attrs;
    lc.numAttrs = 1;
    SLICEMOE_CUDA_TRY(cudaLaunchKernelEx(&lc, kern, mX, mWr1, mWr2, mW1, mW2, p));
    SLICEMOE_LAUNCH_CHECK(1);
    return SLICEMOE_OK;
}

template <int E>
int dec_launch_act(const Dims& D, const slicemoe_weights& w, const void* h, const DecParams& p, int grid, cudaStream_t st) {
    return D.act == SLICEMOE_ACT_GELU_TANH ? dec_launch<E, SLICEMOE_ACT_GELU_TANH>(D, w, h, p, grid, st)
                                           : dec_launch<E, SLICEMOE_ACT_RELU>(D, w, h, p, grid, st);
}

// one CTA per SM
int dec_grid() { return sm_count(); }

}  // namespace

bool decode_forward_supported(const Dims& D) {
    if (D.dtype != SLICEMOE_BF16 || D.ds != kDecDs || D.F != kDecF || D.Hr != kDecHr || D.N <= 0) return false;
    if (D.E != 16 && D.E != 32 && D.E != 64) return false;
    if (D.k > 2 || D.capacity != 0 || D.noise_sigma > 0.0f) return false;
    const int grid = dec_grid();
    if (grid < 2 * D.E) return false;
    if (D.N > 4096 || (D.N + kTileM - 1) / kTileM > grid) return false;
    if (4 * D.E > D.k * kDecDs) return false;          // the lists (E * N * 8 bytes) live in the stacked-row scratch (N * k * 256 bytes)
    int dev = 0, coop = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess)
        return false;
    return coop != 0;
}

int launch_forward_decode(const Dims& D, const slicemoe_weights& w, const void* h, void* h_out, int32_t* topk_idx,
                          float* topk_p, int32_t* assigned, int32_t* kept, void* lists, int32_t* status,
                          bool clear_status, cudaStream_t st) {
    DecParams p{};
    int rc = dec_device_words(&p.sync_word, &p.counts);
    if (rc) return rc;
    const int grid = dec_grid();
    p.X = (const bf16*)h; p.Y = (bf16*)h_out;
    p.Wr1 = (const bf16*)w.Wr1; p.br1 = (const bf16*)w.br1; p.Wr2 = (const bf16*)w.Wr2; p.br2 = (const bf16*)w.br2;
    p.b1 = (const bf16*)w.b1; p.b2 = (const bf16*)w.b2;
    p.topk_idx = topk_idx; p.topk_p = topk_p; p.assigned = assigned; p.kept = kept; p.status = status;
    p.lists = static_cast<int2*>(lists);
    p.N = D.N; p.k = D.k; p.E = D.E;
    p.n_router = (D.N + kTileM - 1) / kTileM;
    p.softmax_scale = 1.4426950408889634f * D.inv_tau;
    p.clear_status = clear_status ? 1 : 0;
    switch (D.E) {
        case 16: return dec_launch_act<16>(D, w, h, p, grid, st);
        case 32: return dec_launch_act<32>(D, w, h, p, grid, st);
        default: return dec_launch_act<64>(D, w, h, p, grid, st);
    }
}

int decode_forward_reset_sync(cudaStream_t st) {
    unsigned long long* words = nullptr;
    int32_t* counts = nullptr;
    int rc = dec_device_words(&words, &counts);
    if (rc) return rc;
    SLICEMOE_CUDA_TRY(cudaMemsetAsync(words, 0, sizeof(unsigned long long), st));
    SLICEMOE_CUDA_TRY(cudaMemsetAsync(counts, 0, 2 * kDecMaxE * kDecCountStride * sizeof(int32_t), st));
    SLICEMOE_CUDA_TRY(cudaStreamSynchronize(st));
    return SLICEMOE_OK;
}

}  // namespace slicemoe
