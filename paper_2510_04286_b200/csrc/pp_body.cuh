// Tensor-core pipeline for 64-wide slices, bf16 storage (sm_100a: tcgen05 + TMEM + TMA), used by the forward of
// the layer (Section 3.1, Eq. 1; Section 3.4):
//
//   router  : relu(X Wr1^T + br1) Wr2^T + br2 -> softmax -> top-k, per 128-row tile
//   experts : act(p (x W1_e^T) + b1_e) W2_e^T + b2_e, per 128-row tile of one expert's rows, rows gathered
//             from h and results added into h'
//
// One CTA of 768 threads per SM walks a contiguous range of tiles.  Hand-offs are per whole tile, never per
// chunk: a tile's GEMM-1 writes the whole hidden layer (fp32) into one of two 256-column regions of tensor
// memory, the activation warps turn it IN PLACE into packed bf16 (the A operand of GEMM-2, which therefore never
// leaves tensor memory), GEMM-2 writes the tile's output accumulator into the same region's upper half.  While
// one region is in the activation, the other is in its GEMMs or its output.  Expert pass, warp roles:
//
//   warp 0       weight sets by TMA (W1 and W2 of an expert stay in shared memory for a run of tiles of that
//                expert; two sets; the first run's set is requested by the GEMM-1 warp, which waits for it) and
//                four-row TMA gathers of tile rows 64-127
//   warp 2       four-row TMA gathers of tile rows 0-63; both gather warps also copy the rows' (pair, gate)
//                into a ring in shared memory
//   warp 3       GEMM-1 issue (one elected lane), warp 1  GEMM-2 issue: two issuing warps, because the small
//                MMAs of this layer are bound by issue, not by the tensor pipe
//   warps 4-19   activation: four warpgroups that split a tile's hidden columns; a thread owns one tile row:
//                gate * acc + b1 and GELU in fp32 (packed two-wide multiply-adds, tanh.approx.f32), 8 columns
//                at a time as a software pipeline around the tanh unit
//   warps 20-23  output: 0.5 acc + b2 -> bf16, staged in shared memory by row and added into row n of h' with
//                16-byte reductions that cover four whole rows per warp instruction
//
// The router pass has the same shape with its hidden layer in units of 128 (three buffers), the fp32 hidden
// values split in place into a truncated bf16 and the rounded remainder (so that the logits keep fp32
// accuracy), and an output warpgroup that does softmax, top-k, the train-mode gates of Section 3.3 where asked
// for, and the dispatch: either each pair's rank among its CTA's pairs of the same expert, or (up to 32 experts)
// the pairs' entries appended to per-expert lists.  All hand-offs are mbarriers with bounded waits (status word
// on run-out); the two 128- / 512-thread rendezvous inside the output and activation warpgroups are plain named
// barriers, reached by all their warps after the same bounded wait.
//
// With ~200 KB of shared memory per CTA there is next to no L1 left for local memory: everything the role
// loops call is inlined and sized to compile without a stack frame or a spill.
#pragma once
#include "philox.cuh"
#include "tc_mlp_body.cuh"

namespace slicemoe {
namespace {

constexpr int kPpThreads = 768;
constexpr int kPpABufs = 4;              // row-tile buffers
// Depth of the per-tile metadata ring: an entry is written up to kPpABufs tiles ahead of GEMM-1 and read by
// the output warps, which run at most three tiles behind GEMM-1 (two regions and the tile being written).
constexpr int kPpMetaRing = 8;
constexpr int kPpABytes = 128 * 128;     // 128 rows x 64 bf16
constexpr int kPpHC = 64;                // hidden units per chunk
constexpr int kPpMaxF = 256;             // expert hidden width (both weight sets stay in shared memory)
constexpr int kPpMaxHr = 512;            // router hidden width
constexpr int kPpStreamCols = 256;       // TMEM columns per stream
// The per-expert list counters sit one per 128-byte line: all CTAs reserve at about the same times, and
// atomics on one line are served one after the other by one L2 slice (16 counters in one line cost every flush
// of the router's lists about 2 k cycles).
constexpr int kPpCountStride = 32;       // ints between two experts' counters

// ---- tanh unit ------------------------------------------------------------------------------------
__device__ __forceinline__ float tanh_approx(float x) {
    float t;
    asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(x));
    return t;
}
// Bounded wait of a whole (converged) warp.  (Inline, like everything the role loops call: an out-of-line
// call costs a stack frame, and with ~200 KB of shared memory per CTA there is next to no L1 left for
// local memory -- a kernel that spills runs every piece of scalar book-keeping at L2 latency.)
__device__ __forceinline__ bool pp_wait(uint32_t bar, uint32_t parity, volatile int* abort) {
    // most waits of this pipeline find their phase complete: a plain test is several times cheaper than a try
    if (__all_sync(0xffffffffu, mbar_test_wait(bar, parity))) return true;
    return (bool)__all_sync(0xffffffffu, mbar_wait(bar, parity, abort, kWaitLimitNs));
}

// Four rows of a 2-D tensor (row indices y0..y3, columns from x on, one box of the map wide; the map's box is
// one row high) into four consecutive 128-byte rows of shared memory, swizzled like a tiled load.
__device__ __forceinline__ void tma_gather4(uint32_t smem_dst, const CUtensorMap* m, int x, int y0, int y1, int y2, int y3,
                                            uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile::gather4.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
        ::"r"(smem_dst), "l"(reinterpret_cast<uint64_t>(m)), "r"(x), "r"(y0), "r"(y1), "r"(y2), "r"(y3), "r"(bar)
        : "memory");
}

__device__ __forceinline__ void named_barrier_sync(int id, int nthreads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}


// Shared-memory state of one CTA besides the operand tiles.
struct PpShared {
    __align__(8) uint64_t bars[48];
    int tile_start[kMaxE + 1];
    int offs[kMaxE + 1];
    int hist[kMaxE];
    uint32_t tmem_base;
    int abort_flag;
    int counts_set;             // which of the two sets of list counters this launch uses (written at kernel entry)
    // experts: first-layer bias of the run each stream is in, as fp32; router: br1 / br2 as fp32
    // (experts: two halves of kPpMaxF, by run parity; router: one array of up to kPpMaxHr)
    __align__(16) float bias1_f32[kPpMaxHr];
    __align__(16) float bias2_f32[kMaxE];
    // experts: per tile in flight (ring over the CTA's tile counter), written by the gather warps with the
    // tile's rows: each row's (pair index, gate), and the tile's expert, run and row count
    __align__(16) int2 pair_gate_s[kPpMetaRing][kTileM];
    int4 tile_s[kPpMetaRing];
};

// Barrier slots.
struct PpBars {
    static constexpr int A_FULL = 0;                      // [kPpABufs]
    static constexpr int A_EMPTY = A_FULL + kPpABufs;     // [kPpABufs]
    static constexpr int W_FULL = A_EMPTY + kPpABufs;     // [2] weight sets (router: [0] only)
    static constexpr int W_EMPTY = W_FULL + 2;            // [2] one arrival per stream
    static constexpr int STREAM0 = W_EMPTY + 2;
    // per stream (3 accumulator slots; the experts use two of them):
    static constexpr int ACC1_FULL = 0, ACC1_EMPTY = 3, HID_FULL = 6, HID_EMPTY = 9, ACC2_FULL = 12, ACC2_EMPTY = 13;
    static constexpr int PER_STREAM = 14;
    static constexpr int DRAIN = STREAM0 + 2 * PER_STREAM;   // [2]
    static constexpr int COUNT = DRAIN + 2;
};
static_assert(PpBars::COUNT <= 48, "barrier slots");
static_assert(2 * kPpMaxF <= kPpMaxHr, "the experts' two bias halves share the router's array");

// Walks the CTA's tile list in order; `run` counts the expert changes seen so far (a run = consecutive
// tiles of one expert = one weight set).
struct PpWalk {
    int ta, e, run, row0, rows;
    __device__ __forceinline__ void init() { ta = -1; e = 0; run = 0; row0 = 0; rows = 0; }
    // advances to local tile `to` (> ta); returns through `crossed` how many run boundaries were passed
    __device__ __forceinline__ int advance(const PpShared& sh, int t_begin, int to) {
        int crossed = 0;
        while (ta < to) {
            ++ta;
            const int e_prev = e;
            locate_tile(sh.tile_start, sh.offs, t_begin + ta, e, row0, rows);
            if (ta > 0 && e != e_prev) { ++run; ++crossed; }
        }
        return crossed;
    }
};

struct PpParams {
    // ---- both passes
    int32_t* status;
    int n_rows;                 // router: N; experts: R
    int HID;                    // Hr or F (multiple of 64)
    // ---- router
    int experts_real;           // E (<= the padded width the kernel is built for)
    int k;
    float softmax_scale;        // log2(e) / tau
    const bf16* br1;            // [Hr] or nullptr
    const bf16* br2;            // [E] or nullptr
    int32_t* topk_idx;          // [N, k]
    float* topk_p;              // [N, k]
    int32_t* local_rank;        // [N, k] rank of the pair among this CTA's pairs of the same expert (or nullptr)
    int32_t* assigned_out;      // [E] pairs per expert, added to with one atomic per expert and CTA (or nullptr; the
                                // caller zeroes it)
    int32_t* cta_hist;          // [grid, E]
    bf16* zero_out;             // h' as [N, 64]: this CTA zeroes the rows it routes (or nullptr)
    int train_gates;            // 1: the gates are Section 3.3's (cross-slice dropout) instead of the probabilities
    uint32_t drop_key0, drop_key1;          // generator key (low, high word of the seed)
    unsigned long long drop_threshold;      // an assignment is dropped iff its 32-bit draw < this
    int2* lists_out;            // per-expert lists of (pair index, gate) filled by the router itself (or nullptr): expert e's
    int32_t* list_counts;       // list starts at lists_out + e * list_stride; its length is counter e (one per kPpCountStride
                                // ints) of set sh.counts_set (sets are kMaxE * kPpCountStride ints apart)
    // ---- experts
    int E;
    const int32_t* offsets;     // [E + 1] (read when the offsets are not already in shared memory)
    const bf16* b1;             // [E, F] or nullptr
    const bf16* b2;             // [E, 64] or nullptr
    const bf16* gather_src;     // h as X[N, 64]
    const int2* pair_gate;      // [R] stacked row -> (pair index n k + j, gate as float bits); or per-expert lists
    int list_stride;            // 0: pair_gate is indexed by stacked row; else expert e's rows start at e * list_stride
    uint32_t gather_magic, gather_shift;
    bf16* scatter_out;          // h' as Y[N, 64]
    int row_elems;              // real slice width (<= 64)
};

__device__ __forceinline__ uint32_t pp_bar(PpShared& sh, int i) { return smem_u32(&sh.bars[i]); }
__device__ __forceinline__ uint32_t pp_sbar(PpShared& sh, int s, int i) {
    return smem_u32(&sh.bars[PpBars::STREAM0 + s * PpBars::PER_STREAM + i]);
}

// First tile of every expert (exclusive scan of the tile counts), by warp 0.
__device__ __forceinline__ void pp_tile_starts(PpShared& sh, int E, int lane) {
    int run = 0;
    for (int e0 = 0; e0 < E; e0 += 32) {
        const int e = e0 + lane;
        const int nt = e < E ? (sh.offs[e + 1] - sh.offs[e] + kTileM - 1) / kTileM : 0;
        int incl = nt;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int up = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += up;
        }
        if (e < E) sh.tile_start[e] = run + incl - nt;
        run += __shfl_sync(0xffffffffu, incl, 31);
    }
    if (lane == 0) sh.tile_start[E] = run;
}

// =====================================================================================================
// Expert pass.  N2: real slice width (48 or 64) = N of the second GEMM; F in {128, 256}.
// Shared memory (1024-aligned): A buffers 4 x 16 KB | weight set 0 | weight set 1, a set = W1 [F, 64]
// (F/64 panels of 8 KB) then W2 as F/64 panels [N2, 64] of N2 x 128 B each.
//
// One stream of tiles; tile t works in tensor-memory region t mod 2 (256 columns each):
//   GEMM-1 of the whole hidden width (N = F) into columns [0, F) of the region;
//   the 16 row-thread warps (4 warpgroups x 4 lane groups) turn it into the hidden layer: warpgroup g
//   owns hidden units [32 g, 32 g + 32) and (F = 256) [128 + 32 g, 128 + 32 g + 32); a thread reads 32
//   fp32 columns of its row, applies gate, bias and activation in fp32 and writes 16 packed bf16
//   columns over accumulator columns it has already read: [32 g, 32 g + 16) and [32 g + 16, 32 g + 32),
//   so the hidden layer ends up in columns [0, 128) and columns [128, 192) are free for
//   GEMM-2's accumulator by the time all hidden values are written;
//   GEMM-2 reads the hidden layer from tensor memory (K step by K step) into [128, 128 + N2);
//   the output step (0.5 acc + b2 -> bf16 -> add into h') of tile t runs in the middle of tile t + 1's
//   activation, each warpgroup on 16 of the 64 output columns.
// A row thread waits on two barriers per tile, both usually long complete: GEMM-1 of tile t + 1 is issued
// while tile t is being activated, GEMM-2 of tile t runs under the first half of tile t + 1's activation.
// The tanh unit (16 results per clock per SM) is what bounds the pass; 16 warps that interleave
// activation and output keep it busy.
// =====================================================================================================
template <int N2>
struct PpFfnCfg {
    static constexpr int W1_SET = kPpMaxF * 128;                 // bytes
    static constexpr int W2_CHUNK = N2 * 128;
    static constexpr int W2_SET = (kPpMaxF / kPpHC) * W2_CHUNK;
    static constexpr int SET_BYTES = W1_SET + ((W2_SET + 1023) / 1024) * 1024;
    static constexpr int OFF_A = 0;
    static constexpr int OFF_W = kPpABufs * kPpABytes;
    // output staging: one row of N2 bf16 per tile row, at a pitch of 16 bytes more than a 128-byte row so that
    // the 16-byte stores of eight neighbouring row threads fall on different banks
    static constexpr int OFF_OUT = OFF_W + 2 * SET_BYTES;
    static constexpr int OUT_PITCH = 144;
    static constexpr int SMEM_BYTES = OFF_OUT + kTileM * OUT_PITCH;
    static constexpr int SMEM_ALLOC = SMEM_BYTES + 1024;
    static constexpr int ACC2_COL = 128;
    static_assert(N2 % 16 == 0 && N2 <= 64, "output width");
    static_assert(SMEM_ALLOC <= 218 * 1024, "shared memory budget");
};

// The activation of one row, eight hidden units (a "piece") at a time, in three steps that the row threads run
// as a software pipeline (the tanh of piece j is in flight while piece j + 1 is prepared and piece j - 1 is
// finished, so that the tanh unit, 16 results per clock per SM, never waits for the other pipes):
//   pre   z = acc * gate + bias; u = sqrt(2/pi) (z + 0.044715 z^3)        (packed two-wide multiply-adds)
//   tanh  t = tanh(u)
//   post  hidden = z t + z = 2 gelu(z), packed bf16 (the factor 0.5 is applied to the second GEMM's accumulator
//         in the output step: exact, a power of two)
// ReLU needs no tanh: post packs relu(z).
template <int ACT>
__device__ __forceinline__ void pp_pre8(const uint32_t* acc, float gs, const float* bias /* shared, 8 floats */, bool has_bias,
                                        float* z, float* u) {
    if (has_bias) {
#pragma unroll
        for (int i = 0; i < 8; i += 4) {
            const float4 b = *reinterpret_cast<const float4*>(bias + i);   // same address for the whole warp
            fma2(z[i], z[i + 1], __uint_as_float(acc[i]), __uint_as_float(acc[i + 1]), gs, gs, b.x, b.y);
            fma2(z[i + 2], z[i + 3], __uint_as_float(acc[i + 2]), __uint_as_float(acc[i + 3]), gs, gs, b.z, b.w);
        }
    } else {
#pragma unroll
        for (int i = 0; i < 8; i += 2) mul2(z[i], z[i + 1], __uint_as_float(acc[i]), __uint_as_float(acc[i + 1]), gs, gs);
    }
    if constexpr (ACT != SLICEMOE_ACT_RELU) {
        constexpr float c0 = 0.7978845608028654f, c1 = 0.7978845608028654f * 0.044715f;
#pragma unroll
        for (int i = 0; i < 8; i += 2) {
            float s0, s1, n0, n1;
            mul2(s0, s1, z[i], z[i + 1], z[i], z[i + 1]);
            fma2(n0, n1, s0, s1, c1, c1, c0, c0);
            mul2(u[i], u[i + 1], z[i], z[i + 1], n0, n1);
        }
    }
}
template <int ACT>
__device__ __forceinline__ void pp_tanh8(float* u) {
    if constexpr (ACT != SLICEMOE_ACT_RELU) {
#pragma unroll
        for (int i = 0; i < 8; ++i) u[i] = tanh_approx(u[i]);
    }
}
template <int ACT>
__device__ __forceinline__ void pp_post8(const float* z, const float* t, uint32_t* out) {
    if constexpr (ACT == SLICEMOE_ACT_RELU) {
#pragma unroll
        for (int i = 0; i < 4; ++i) out[i] = cvt_rn_relu_bf16x2(z[2 * i], z[2 * i + 1]);
    } else {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float r0, r1;
            fma2(r0, r1, z[2 * i], z[2 * i + 1], t[2 * i], t[2 * i + 1], z[2 * i], z[2 * i + 1]);
            out[i] = pack_bf16x2(r0, r1);
        }
    }
}

// The same activation in turns of 16 units without the pipeline (decode-shaped forward).
// 16 column pairs of one row: z = acc * gate (+ bias), hidden = 2 gelu(z) or relu(z), packed bf16.
// GELU, tanh form: 0.5 z (1 + tanh(sqrt(2/pi) (z + 0.044715 z^3))); the factor 0.5 is applied to the
// second GEMM's accumulator in the output step (exact, a power of two).
// z = acc * gate (+ bias) for 16 columns of one row
__device__ __forceinline__ void pp_scale16(const uint32_t* acc, float gs, const float* bias /* shared, 16 floats */,
                                           bool has_bias, float* z) {
    if (has_bias) {
#pragma unroll
        for (int i = 0; i < 16; i += 4) {
            const float4 b = *reinterpret_cast<const float4*>(bias + i);   // same address for the whole warp
            fma2(z[i], z[i + 1], __uint_as_float(acc[i]), __uint_as_float(acc[i + 1]), gs, gs, b.x, b.y);
            fma2(z[i + 2], z[i + 3], __uint_as_float(acc[i + 2]), __uint_as_float(acc[i + 3]), gs, gs, b.z, b.w);
        }
    } else {
#pragma unroll
        for (int i = 0; i < 16; i += 2) mul2(z[i], z[i + 1], __uint_as_float(acc[i]), __uint_as_float(acc[i + 1]), gs, gs);
    }
}
// eight column pairs: hidden = 2 gelu(z) or relu(z), packed bf16 (enough independent work for the tanh
// unit's latency, few live registers)
template <int ACT>
__device__ __forceinline__ void pp_act8(const float* z, uint32_t* out) {
    if constexpr (ACT == SLICEMOE_ACT_RELU) {
#pragma unroll
        for (int i = 0; i < 8; ++i) out[i] = cvt_rn_relu_bf16x2(z[2 * i], z[2 * i + 1]);
    } else {
        constexpr float c0 = 0.7978845608028654f, c1 = 0.7978845608028654f * 0.044715f;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            float s0, s1, n0, n1, u0, u1, r0, r1;
            mul2(s0, s1, z[2 * i], z[2 * i + 1], z[2 * i], z[2 * i + 1]);
            fma2(n0, n1, s0, s1, c1, c1, c0, c0);
            mul2(u0, u1, z[2 * i], z[2 * i + 1], n0, n1);
            const float t0 = tanh_approx(u0), t1 = tanh_approx(u1);
            fma2(r0, r1, z[2 * i], z[2 * i + 1], t0, t1, z[2 * i], z[2 * i + 1]);
            out[i] = pack_bf16x2(r0, r1);
        }
    }
}

// Barriers of the expert pass (one thread; the CTA synchronises before anybody waits on them).
__device__ __forceinline__ void pp_ffn_init_bars(PpShared& sh, const CUtensorMap* tmXg_p, const CUtensorMap* tmW1_p,
                                                 const CUtensorMap* tmW2_p) {
    using B = PpBars;
    sh.abort_flag = 0;
    for (int i = 0; i < kPpABufs; ++i) { mbar_init(pp_bar(sh, B::A_FULL + i), 2); mbar_init(pp_bar(sh, B::A_EMPTY + i), 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(pp_bar(sh, B::W_FULL + i), 1); mbar_init(pp_bar(sh, B::W_EMPTY + i), 1); }
    mbar_init(pp_bar(sh, B::DRAIN + 1), 1);
    for (int r = 0; r < 2; ++r) {                                  // per tensor-memory region
        mbar_init(pp_sbar(sh, r, B::ACC1_FULL), 1);
        mbar_init(pp_sbar(sh, r, B::HID_FULL), 16);
        mbar_init(pp_sbar(sh, r, B::ACC2_FULL), 1);
        mbar_init(pp_sbar(sh, r, B::ACC2_EMPTY), 4);
    }
    mbar_init(pp_bar(sh, B::DRAIN), 1);
    fence_mbar_init();
    prefetch_tensormap(tmXg_p);
    prefetch_tensormap(tmW1_p);
    prefetch_tensormap(tmW2_p);
}

// Called by all kPpThreads threads; TMEM (512 columns at sh.tmem_base) is allocated and freed by the
// caller.  SAME_LAUNCH: pair_gate (and the offsets) were written earlier in this launch.
// READY: the caller has initialised the barriers (pp_ffn_init_bars), filled sh.offs and sh.tile_start and
// synchronised the CTA.  Rows come from gather_src through pair_gate and results are added into scatter_out.
// STAGED (the staged call, slicemoe_expert_ffn): the rows are already stacked and weighted (Eq. 1): a tile's rows
// are one tiled load through tmXg_p (then a map of the stacked rows with a 128-row box), every gate is 1 and a
// row's result is stored to the same row of scatter_out (the stacked outputs) instead of added.
template <int N2, int ACT, bool SAME_LAUNCH, bool READY, bool STAGED = false>
__device__ __forceinline__ void pp_ffn_body(const CUtensorMap* tmXg_p, const CUtensorMap* tmW1_p, const CUtensorMap* tmW2_p,
                                            const PpParams& p, PpShared& sh, uint8_t* smem_raw) {
    using C = PpFfnCfg<N2>;
    using B = PpBars;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    volatile int* abort = &sh.abort_flag;
    const int npanels = p.HID / kPpHC;
    const bool has_b1 = p.b1 != nullptr;
    const bool wide = p.HID == 256;          // two 32-unit sub-chunks per row thread and tile, else one

    // ---- set-up -----------------------------------------------------------------------------------
    if (!READY) {
        if (threadIdx.x == 0) pp_ffn_init_bars(sh, tmXg_p, tmW1_p, tmW2_p);
        for (int e = threadIdx.x; e <= p.E; e += kPpThreads) sh.offs[e] = SAME_LAUNCH ? __ldcg(p.offsets + e) : p.offsets[e];
        __syncthreads();
        if (warp == 0) pp_tile_starts(sh, p.E, lane);
        tc_fence_before_sync();
        __syncthreads();
        tc_fence_after_sync();
    }
    const uint32_t tmem_base = sh.tmem_base;
    const int total_tiles = sh.tile_start[p.E];
    const int per_cta = (total_tiles + gridDim.x - 1) / gridDim.x;
    const int t_begin = min(total_tiles, (int)blockIdx.x * per_cta);
    const int ntiles = min(total_tiles, t_begin + per_cta) - t_begin;
    const uint32_t sA = smem_base + C::OFF_A, sW = smem_base + C::OFF_W;

    if (false) {
    } else if (warp == 3) {
        // ================= GEMM-1 issue ===============================================================
        // GEMM-1 of tile t goes into region t mod 2 once the output accumulator of tile t - 2 has been
        // read: it runs up to two tiles ahead of the activation.  Two issuing warps (this one and the
        // GEMM-2 warp): an issuing warp's waits and book-keeping are serial work on the tile's critical path.
        // All lanes run the loop (descriptors stay in uniform registers); one elected lane issues.
        if (ntiles > 0) {
            const uint32_t idesc1 = make_idesc(128, p.HID, kFmtBF16, kFmtBF16);
            const uint32_t dA = desc_lo_sw128(sA), dW = desc_lo_sw128(sW);
            bool ok = true;
            PpWalk w1;
            w1.init();
            int run1 = -1;
            // The first run's weights are requested here, by the warp that waits for them: the gather warps
            // are busy with the first tiles' lists and rows, and issuing a set's eight copies takes a thread
            // about a thousand cycles.
            w1.advance(sh, t_begin, 0);
            if (lane == 0) {
                mbar_arrive_expect_tx(pp_bar(sh, B::W_FULL), (uint32_t)(p.HID * 128 + npanels * C::W2_CHUNK));
                for (int c = 0; c < npanels; ++c) {
                    tma_load_2d(sW + c * (kPpHC * 128), tmW1_p, 0, w1.e * p.HID + c * kPpHC, pp_bar(sh, B::W_FULL));
                    tma_load_2d(sW + C::W1_SET + c * C::W2_CHUNK, tmW2_p, c * kPpHC, w1.e * N2, pp_bar(sh, B::W_FULL));
                }
            }
            __syncwarp();
#pragma unroll 1
            for (int ta = 0; ta < ntiles && ok; ++ta) {
                const int ab = ta % kPpABufs, r = ta & 1;
                w1.advance(sh, t_begin, ta);
                if (w1.run != run1) {
                    if (!pp_wait(pp_bar(sh, B::W_FULL + (w1.run & 1)), ((uint32_t)w1.run >> 1) & 1u, abort)) { ok = false; break; }
                    run1 = w1.run;
                }
                if (!pp_wait(pp_bar(sh, B::A_FULL + ab), (uint32_t)(ta / kPpABufs) & 1u, abort)) { ok = false; break; }
                if (!pp_wait(pp_sbar(sh, r, B::ACC2_EMPTY), ((uint32_t)(ta >> 1) & 1u) ^ 1u, abort)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t wset = dW + (((w1.run & 1) * C::SET_BYTES) >> 4);
                const uint32_t a0 = dA + ((ab * kPpABytes) >> 4);
                const uint32_t d = tmem_base + r * kPpStreamCols;
                if (elect_one_sync()) {
                    mma_ss<0>(d, a0, wset, idesc1);
#pragma unroll
                    for (int kk = 1; kk < 4; ++kk) mma_ss<1>(d, a0 + ((kk * 32) >> 4), wset + ((kk * 32) >> 4), idesc1);
                    mma_commit(pp_sbar(sh, r, B::ACC1_FULL));
                    mma_commit(pp_bar(sh, B::A_EMPTY + ab));
                }
                __syncwarp();
            }
            if (!ok || *abort) {
                volatile int never = 0;
                if (lane == 0) {
                    mma_commit(pp_bar(sh, B::DRAIN));
                    mbar_wait(pp_bar(sh, B::DRAIN), 0u, &never, 10000000ull);
                    mbar_wait(pp_bar(sh, B::W_FULL), 0u, &never, 10000000ull);     // (the copies this warp requested)
                }
                __syncwarp();
            }
        }
    } else if (warp == 1) {
        // ================= GEMM-2 issue ===============================================================
        if (ntiles > 0) {
            constexpr uint32_t idesc2 = make_idesc(128, N2, kFmtBF16, kFmtBF16);
            const uint32_t dW = desc_lo_sw128(sW);
            bool ok = true;
            PpWalk w2;
            w2.init();
            w2.advance(sh, t_begin, 0);
#pragma unroll 1
            for (int ta = 0; ta < ntiles && ok; ++ta) {
                const int r = ta & 1;
                const uint32_t w2d = dW + (((w2.run & 1) * C::SET_BYTES + C::W1_SET) >> 4);
                const int run_before = w2.run;
                const int crossed = ta + 1 < ntiles ? w2.advance(sh, t_begin, ta + 1) : 0;   // (before the wait: off the critical path)
                if (!pp_wait(pp_sbar(sh, r, B::HID_FULL), (uint32_t)(ta >> 1) & 1u, abort)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t d = tmem_base + r * kPpStreamCols;
                if (elect_one_sync()) {
                    // K step kk = hidden units [16 kk, 16 kk + 16): units below 128 sit at packed column
                    // 32 (u / 32) + 8 ((u / 16) & 1), units from 128 on 16 columns further
#pragma unroll 8
                    for (int kk = 0; kk < p.HID / 16; ++kk) {
                        const int u = (kk & 7) * 16;
                        const uint32_t a = d + 32 * (u >> 5) + 8 * ((u >> 4) & 1) + (kk >= 8 ? 16 : 0);
                        const uint32_t bd = w2d + (((kk >> 2) * C::W2_CHUNK + (kk & 3) * 32) >> 4);
                        mma_ts_dyn(d + C::ACC2_COL, a, bd, idesc2, kk > 0 ? 1u : 0u);
                    }
                    mma_commit(pp_sbar(sh, r, B::ACC2_FULL));
                    // a run that ends here hands its weight set back (GEMM-1 of these tiles finished before
                    // their GEMM-2 began, so this commit covers the other issuing warp's reads as well)
                    if (crossed) mma_commit(pp_bar(sh, B::W_EMPTY + (run_before & 1)));
                }
                __syncwarp();
            }
            if (!ok || *abort) {
                volatile int never = 0;
                if (lane == 0) {
                    mma_commit(pp_bar(sh, B::DRAIN + 1));
                    mbar_wait(pp_bar(sh, B::DRAIN + 1), 0u, &never, 10000000ull);
                }
                __syncwarp();
            }
        }
    } else if (warp == 0 || warp == 2) {
        // ================= gather warps (tile rows 0..63: warp 2; 64..127: warp 0, which also loads the weights)
        // Row r of tile ta is stacked row row0 + r = pair (n, j); its A row is X[n, :].  A lane fetches four
        // tile rows with one four-row gather of the copy engine (no per-lane address arithmetic, nothing
        // through the load/store pipe that the activation warps' tanh instructions share), up to four tiles
        // ahead; a warp's gathers are issued one after the other, hence two warps of 16 lanes.  Rows past the
        // tile's end fetch row 0: they are computed and never stored.
        // Weights: one set (W1 and W2 of an expert) per run of tiles of the same expert, two sets in shared
        // memory; a set is loaded as soon as the run before the previous one has been computed.
        if (ntiles > 0) {
            const int rbase = warp == 2 ? 0 : 64;
            PpWalk wn;
            wn.init();
            int2 nnext[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) nnext[q] = make_int2(-1, 0);
            int loaded_run = 0, cur_e = 0, cur_run = 0, cur_rows = 0, next_row0 = 0;      // (run 0's weights: the GEMM-1 warp)
            uint32_t last_bar = 0, last_par = 0;
            bool ok = true;
            const uint32_t set_tx = (uint32_t)(p.HID * 128 + npanels * C::W2_CHUNK);
#pragma unroll 1
            for (int ta = -1; ta < ntiles && ok; ++ta) {
                int nrow[4];
                int2 cur_pg[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    cur_pg[q] = nnext[q];
                    nrow[q] = nnext[q].x < 0 ? 0 : pair_to_row(nnext[q].x, p.gather_magic, p.gather_shift);
                }
                if (ta >= 0) { cur_e = wn.e; cur_run = wn.run; cur_rows = wn.rows; }
                if (ta + 1 < ntiles) {
                    wn.advance(sh, t_begin, ta + 1);
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const int r = rbase + 4 * (lane & 15) + q;
                        nnext[q] = make_int2(-1, 0);
                        if (STAGED) {
                            if (r < wn.rows) nnext[q] = make_int2(wn.row0 + r, __float_as_int(1.0f));
                        } else {
                            const size_t at = p.list_stride ? (size_t)wn.e * p.list_stride + (wn.row0 - sh.offs[wn.e]) + r : (size_t)wn.row0 + r;
                            if (r < wn.rows) nnext[q] = SAME_LAUNCH ? __ldcg(p.pair_gate + at) : __ldg(p.pair_gate + at);
                        }
                    }
                }
                const int cur_row0 = next_row0;
                next_row0 = wn.row0;
                if (ta < 0) continue;
                // weights of a new run
                const int want_run = cur_run, want_e = cur_e;
                if (warp == 0 && want_run != loaded_run) {
                    loaded_run = want_run;
                    const int set = want_run & 1;
                    const uint32_t n = (uint32_t)want_run >> 1;
                    ok = pp_wait(pp_bar(sh, B::W_EMPTY + set), (n & 1u) ^ 1u, abort);
                    if (!ok) break;
                    if (lane == 0) {
                        mbar_arrive_expect_tx(pp_bar(sh, B::W_FULL + set), set_tx);
                        const uint32_t w1 = sW + set * C::SET_BYTES, w2 = w1 + C::W1_SET;
                        for (int c = 0; c < npanels; ++c) {
                            tma_load_2d(w1 + c * (kPpHC * 128), tmW1_p, 0, want_e * p.HID + c * kPpHC, pp_bar(sh, B::W_FULL + set));
                            tma_load_2d(w2 + c * C::W2_CHUNK, tmW2_p, c * kPpHC, want_e * N2, pp_bar(sh, B::W_FULL + set));
                        }
                    }
                    __syncwarp();
                    last_bar = pp_bar(sh, B::W_FULL + set);
                    last_par = n & 1u;
                }
                const int ab = ta % kPpABufs;
                ok = pp_wait(pp_bar(sh, B::A_EMPTY + ab), ((uint32_t)(ta / kPpABufs) & 1u) ^ 1u, abort);
                if (!ok) break;
                // the tile's metadata (its ring entry was last read by the output warps of tile ta - kPpMetaRing,
                // long before GEMM-1 of tile ta - kPpABufs, whose completion this warp has just waited for)
                if (lane < 16) {
                    int2* dst = &sh.pair_gate_s[ta % kPpMetaRing][rbase + 4 * lane];
                    reinterpret_cast<int4*>(dst)[0] = make_int4(cur_pg[0].x, cur_pg[0].y, cur_pg[1].x, cur_pg[1].y);
                    reinterpret_cast<int4*>(dst)[1] = make_int4(cur_pg[2].x, cur_pg[2].y, cur_pg[3].x, cur_pg[3].y);
                }
                if (lane == 0 && warp == 2) sh.tile_s[ta % kPpMetaRing] = make_int4(cur_e, cur_run, cur_rows, 0);
                __syncwarp();
                if (lane == 0) {
                    if (warp == 2) mbar_arrive_expect_tx(pp_bar(sh, B::A_FULL + ab), kPpABytes);
                    else mbar_arrive(pp_bar(sh, B::A_FULL + ab));
                }
                if (STAGED) {
                    // (rows past the expert's last one belong to the next expert or lie past the matrix, where the
                    // copy engine fills zeros: computed and never stored)
                    if (lane == 0 && warp == 2) tma_load_2d(sA + ab * kPpABytes, tmXg_p, 0, cur_row0, pp_bar(sh, B::A_FULL + ab));
                } else if (lane < 16) {
                    tma_gather4(sA + ab * kPpABytes + (rbase / 4 + lane) * 512, tmXg_p, 0, nrow[0], nrow[1], nrow[2], nrow[3], pp_bar(sh, B::A_FULL + ab));
                }
            }
            if (!ok || *abort) {
                // (bounded) let the copies in flight land before shared memory is reused
                volatile int never = 0;
                const int last = ntiles - 1;
                if (last >= 0) mbar_wait(pp_bar(sh, B::A_FULL + last % kPpABufs), (uint32_t)(last / kPpABufs) & 1u, &never, 10000000ull);
                if (last_bar) mbar_wait(last_bar, last_par, &never, 10000000ull);
            }
        }
    } else if (warp < 20) {
        // ================= activation warps: warpgroup g, lane group lg ================================
        // Piece j = eight hidden units of the thread's row: [32 g + 8 j, +8) for j < 4 and [128 + 32 g + 8 (j - 4),
        // +8) for j >= 4 (F = 256 only); its four packed columns go to [32 g + 4 j, +4), which this thread has read
        // before.  The pieces of a tile run as a software pipeline (pre of piece j + 1 and post of piece j - 1 under
        // the tanh of piece j); the accumulator columns of piece j + 2 are requested as soon as piece j + 1 has
        // been taken from its registers, so the load's latency runs under the tanh work as well.
        // (Measured and left out: the same pipeline carried across tile boundaries, with GEMM-1 in two halves so
        // that a region's lower half need not wait for the read-out of its previous tile: no faster, the row
        // threads are bound by their own instruction stream next to the MMAs and the output warps, not by the
        // bubbles at tile boundaries.)
        const int g = (warp - 4) >> 2;
        const int lg = warp & 3;
        const int row = lg * 32 + lane;
        const uint32_t tlane = tmem_base + ((uint32_t)(lg * 32) << 16);
        const int np = wide ? 8 : 4;
        bool ok = true;
        int run_bias = -1;
#pragma unroll 1
        for (int ta = 0; ta < ntiles && ok; ++ta) {
            const int r = ta & 1;
            ok = pp_wait(pp_sbar(sh, r, B::ACC1_FULL), (uint32_t)(ta >> 1) & 1u, abort);
            if (!ok) break;
            tc_fence_after_sync();
            // (the tile's rows, and with them its ring entry, landed before GEMM-1 could run)
            const float gs = __int_as_float(sh.pair_gate_s[ta % kPpMetaRing][row].y);
            if (has_b1) {
                const int4 ti = sh.tile_s[ta % kPpMetaRing];
                if (ti.y != run_bias) {
                    // a new run: its expert's first-layer bias as fp32 (two buffers by run parity: the other
                    // one may still be in use by warps that are behind)
                    for (int f = g * 128 + row; f < p.HID; f += 512) sh.bias1_f32[(ti.y & 1) * kPpMaxF + f] = __bfloat162float(p.b1[(size_t)ti.x * p.HID + f]);
                    named_barrier_sync(1, 512);
                    run_bias = ti.y;
                }
            }
            const float* bias = sh.bias1_f32 + (run_bias & 1) * kPpMaxF + 32 * g;
            const uint32_t region = tlane + r * kPpStreamCols + 32 * g;
            auto piece_col = [&](int j) -> uint32_t { return region + (j < 4 ? 8 * j : 128 + 8 * (j - 4)); };
            auto piece_bias = [&](int j) -> const float* { return bias + (j < 4 ? 8 * j : 128 + 8 * (j - 4)); };
            // (two pieces per tensor-memory load and per store: every such instruction passes through the same
            // queue as the other warps' loads and stores)
            uint32_t acc[16], hid[8];
            float z[2][8], u[2][8];
            tmem_ld_x16(piece_col(0), acc);
            tmem_ld_wait();
            pp_pre8<ACT>(acc, gs, piece_bias(0), has_b1, z[0], u[0]);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                if (j >= np) break;
                pp_tanh8<ACT>(u[j & 1]);
                if (j + 1 < np) {
                    if (((j + 1) & 1) == 0) tmem_ld_wait();
                    pp_pre8<ACT>(acc + 8 * ((j + 1) & 1), gs, piece_bias(j + 1), has_b1, z[(j + 1) & 1], u[(j + 1) & 1]);
                    if (((j + 1) & 1) == 1 && j + 2 < np) tmem_ld_x16(piece_col(j + 2), acc);
                }
                pp_post8<ACT>(z[j & 1], u[j & 1], hid + 4 * (j & 1));
                if (j & 1) tmem_st_x8(region + 4 * (j - 1), hid);
            }
            tmem_st_wait();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(pp_sbar(sh, r, B::HID_FULL));
        }
    } else {
        // ================= output warpgroup ===========================================================
        // 0.5 acc + b2 -> bf16 -> add into row n of h' (the sum over the row's k experts), 16 columns at a time
        const int lg = warp & 3;
        const int row = lg * 32 + lane;
        const uint32_t tlane = tmem_base + ((uint32_t)(lg * 32) << 16);
        const uint32_t swarp = smem_base + C::OFF_OUT + lg * 32 * C::OUT_PITCH;       // this warp's 32 staging rows
        const uint32_t srow = swarp + lane * C::OUT_PITCH;
        bool ok = true;
#pragma unroll 1
        for (int ta = 0; ta < ntiles && ok; ++ta) {
            const int r = ta & 1;
            ok = pp_wait(pp_sbar(sh, r, B::ACC2_FULL), (uint32_t)(ta >> 1) & 1u, abort);
            if (!ok) break;
            tc_fence_after_sync();
            const int4 ti = sh.tile_s[ta % kPpMetaRing];       // (expert, run, rows) of the tile
            const bool live = row < ti.z;
            const int e_cur = ti.x;
            const uint32_t acc2 = tlane + r * kPpStreamCols + C::ACC2_COL;
            constexpr float sc = kOutScale<ACT>;
            // the whole accumulator row goes into registers as packed bf16 (32 columns' loads in flight at a time),
            // so that the region is handed back early: its next GEMM-1 waits for this
            uint32_t o[N2 / 2];
#pragma unroll
            for (int cb = 0; cb < N2; cb += 32) {
                uint32_t v[32];
                if (cb + 16 < N2) tmem_ld_x32(acc2 + cb, v);
                else tmem_ld_x16(acc2 + cb, v);
                tmem_ld_wait();
#pragma unroll
                for (int c = 0; c < 32 && cb + c < N2; c += 8) {
                    if (p.b2) {
                        float bb[8];
                        unpack16<bf16>(__ldg(reinterpret_cast<const uint4*>(p.b2 + (size_t)e_cur * N2 + cb + c)), bb);
#pragma unroll
                        for (int q = 0; q < 4; ++q)
                            o[(cb + c) / 2 + q] = pack_bf16x2(fmaf(__uint_as_float(v[c + 2 * q]), sc, bb[2 * q]),
                                                              fmaf(__uint_as_float(v[c + 2 * q + 1]), sc, bb[2 * q + 1]));
                    } else {
#pragma unroll
                        for (int q = 0; q < 4; ++q)
                            o[(cb + c) / 2 + q] = pack_bf16x2(__uint_as_float(v[c + 2 * q]) * sc, __uint_as_float(v[c + 2 * q + 1]) * sc);
                    }
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(pp_sbar(sh, r, B::ACC2_EMPTY));
            // The row goes into this thread's staging row; the warp then reads its 32 rows back with eight
            // neighbouring lanes on one row, so that a warp-wide 16-byte reduction covers four whole rows of h'
            // (4 contiguous 128-byte requests instead of 32 scattered 16-byte ones: the row-per-thread form is
            // bound by the number of requests an SM can send, not by their bytes).
            __syncwarp();                 // (the warp has read the previous tile's rows)
#pragma unroll
            for (int c = 0; c < N2; c += 8) st_shared_v4(srow + c * 2, o[c / 2], o[c / 2 + 1], o[c / 2 + 2], o[c / 2 + 3]);
            __syncwarp();
            const int n_own = !live ? -1 : STAGED ? sh.pair_gate_s[ta % kPpMetaRing][row].x
                                                  : pair_to_row(sh.pair_gate_s[ta % kPpMetaRing][row].x, p.gather_magic, p.gather_shift);
            const int sub = lane >> 3, chunk = lane & 7;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int rl = 4 * i + sub;                                   // row of this warp's 32
                const int n_i = __shfl_sync(0xffffffffu, n_own, rl);
                const uint4 t = ld_shared_v4(swarp + rl * C::OUT_PITCH + chunk * 16);
                if (n_i >= 0 && chunk < N2 / 8) {
                    if (STAGED) *reinterpret_cast<uint4*>(p.scatter_out + (size_t)n_i * N2 + chunk * 8) = t;
                    else red_add_bf16x8(p.scatter_out + (size_t)n_i * N2 + chunk * 8, t.x, t.y, t.z, t.w);
                }
            }
        }
    }

    // ---- teardown ---------------------------------------------------------------------------------
    tc_fence_before_sync();
    __syncthreads();
    if (threadIdx.x == 0 && sh.abort_flag) atomicExch(p.status, (int)SLICEMOE_ERR_DEVICE_TIMEOUT);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
}

// =====================================================================================================
// Router pass.  EP: expert count the kernel is built for (16 / 32 / 64; fewer real experts are padded,
// their logits set to -inf).  Shared memory: X buffers 4 x 16 KB | Wr1 [Hr, 64] | Wr2 as Hr/64 panels
// of [EP, 64].
// The hidden layer of a tile is taken in halves of 128 units ("units of work"): GEMM-1 (N = 128) into one
// of three 128-column buffers of tensor memory; the 16 activation warps (warpgroup g: columns [32 g, 32 g +
// 32), 16 at a time) add the bias and write relu(.) back over the accumulator as a bf16 pair hi + lo (16
// mantissa bits: K step kk of a half is at columns 16 kk (hi) and 16 kk + 8 (lo)), so that the logits do
// not depend on 16-bit rounding of the hidden layer; GEMM-2 runs over hi and lo from tensor memory into
// one of two logit accumulators (columns [384, 448) and [448, 512)), accumulating over the halves; the
// output warpgroup turns a tile's logits into softmax probabilities, the top-k and each pair's rank among
// this CTA's pairs of its expert.  GEMM-1 runs two units ahead of GEMM-2.
// =====================================================================================================
template <int EP>
struct PpRouteCfg {
    static constexpr int W2_CHUNK = EP * 128;
    static constexpr int OFF_A = 0;
    static constexpr int OFF_W1 = kPpABufs * kPpABytes;
    static constexpr int OFF_W2 = OFF_W1 + kPpMaxHr * 128;
    // list dispatch by the output warps (EP <= 32): the (pair, gate, expert, rank) entries of up to LIST_GROUP tiles
    // wait here until the group's list ranges have been reserved
    static constexpr int LIST_GROUP = 4;
    static constexpr int OFF_STAGE = OFF_W2 + (kPpMaxHr / kPpHC) * W2_CHUNK;
    static constexpr int STAGE_BYTES = EP <= 32 ? LIST_GROUP * 2 * kTileM * 16 : 0;
    static constexpr int SMEM_BYTES = OFF_STAGE + STAGE_BYTES;
    static constexpr int SMEM_ALLOC = SMEM_BYTES + 1024;
    static constexpr int HB_COLS = 128, LOGIT_COL = 384;
    static_assert(SMEM_ALLOC <= 212 * 1024, "shared memory budget");
    static_assert(EP % 16 == 0 && EP <= 64, "expert count");
};

template <int EP>
__device__ __forceinline__ void pp_route_body(const CUtensorMap* tmX_p, const CUtensorMap* tmW1_p, const CUtensorMap* tmW2_p,
                                              const PpParams& p, PpShared& sh, uint8_t* smem_raw) {
    using C = PpRouteCfg<EP>;
    using B = PpBars;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    volatile int* abort = &sh.abort_flag;
    const int npanels = p.HID / kPpHC;
    const int nhalf = p.HID / 128;            // units of work per tile

    const int total_tiles = (p.n_rows + kTileM - 1) / kTileM;
    const int per_cta = (total_tiles + gridDim.x - 1) / gridDim.x;
    const int t_begin = min(total_tiles, (int)blockIdx.x * per_cta);
    const int ntiles = min(total_tiles, t_begin + per_cta) - t_begin;
    const int nunits = ntiles * nhalf;
    const uint32_t sA = smem_base + C::OFF_A, sW1 = smem_base + C::OFF_W1, sW2 = smem_base + C::OFF_W2;
    const int npre = min(ntiles, kPpABufs);       // row tiles requested during set-up

    // Barrier use in this pass (slots of "stream" 0): ACC1_FULL[3] / ACC1_EMPTY[3] / HID_FULL[3] per hidden
    // buffer; the logit accumulators use ACC2_FULL / ACC2_EMPTY of "streams" 0 and 1.
    if (threadIdx.x == 0) {
        prefetch_tensormap(tmX_p);
        sh.abort_flag = 0;
        for (int i = 0; i < kPpABufs; ++i) { mbar_init(pp_bar(sh, B::A_FULL + i), 1); mbar_init(pp_bar(sh, B::A_EMPTY + i), 1); }
        for (int i = 0; i < 3; ++i) {
            mbar_init(pp_sbar(sh, 0, B::ACC1_FULL + i), 1);
            mbar_init(pp_sbar(sh, 0, B::ACC1_EMPTY + i), 1);
            mbar_init(pp_sbar(sh, 0, B::HID_FULL + i), 16);
        }
        for (int r = 0; r < 2; ++r) {
            mbar_init(pp_sbar(sh, r, B::ACC2_FULL), 1);
            mbar_init(pp_sbar(sh, r, B::ACC2_EMPTY), 4);
        }
        mbar_init(pp_bar(sh, B::DRAIN), 1);
        mbar_init(pp_bar(sh, B::DRAIN + 1), 1);
        fence_mbar_init();
        // The first row tiles (all buffers are free) are requested right here, by the thread that has just
        // initialised their barriers: the first tile comes from DRAM and is what the pass waits for.  (The
        // weights are requested by another warp at the same time: issuing a dozen copies takes one thread
        // more than a thousand cycles.)
        for (int ta = 0; ta < npre; ++ta) {
            mbar_arrive_expect_tx(pp_bar(sh, B::A_FULL + ta), kPpABytes);
            tma_load_2d(sA + ta * kPpABytes, tmX_p, 0, (t_begin + ta) * kTileM, pp_bar(sh, B::A_FULL + ta));
        }
    } else if (threadIdx.x == 64) {
        prefetch_tensormap(tmW1_p);
        prefetch_tensormap(tmW2_p);
        mbar_init(pp_bar(sh, B::W_FULL), 1);
        fence_mbar_init();
        if (ntiles > 0) {
            mbar_arrive_expect_tx(pp_bar(sh, B::W_FULL), (uint32_t)(p.HID * 128 + npanels * C::W2_CHUNK));
            for (int c = 0; c < npanels; ++c) {
                tma_load_2d(sW1 + c * (kPpHC * 128), tmW1_p, 0, c * kPpHC, pp_bar(sh, B::W_FULL));
                tma_load_2d(sW2 + c * C::W2_CHUNK, tmW2_p, c * kPpHC, 0, pp_bar(sh, B::W_FULL));
            }
        }
    }
    for (int e = threadIdx.x; e < kMaxE; e += kPpThreads) sh.hist[e] = 0;
    for (int i = threadIdx.x; i < p.HID; i += kPpThreads) sh.bias1_f32[i] = p.br1 ? __bfloat162float(p.br1[i]) : 0.0f;
    for (int i = threadIdx.x; i < EP; i += kPpThreads)
        sh.bias2_f32[i] = i >= p.experts_real ? -INFINITY : (p.br2 ? __bfloat162float(p.br2[i]) : 0.0f);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = sh.tmem_base;

    if (warp == 0) {
        // ================= TMA producer ===============================================================
        if (lane == 0 && ntiles > 0) {
            bool ok = true;
            uint32_t last_bar = pp_bar(sh, B::A_FULL + npre - 1), last_par = 0;
            for (int ta = npre; ta < ntiles; ++ta) {
                const int ab = ta % kPpABufs;
                if (!mbar_wait(pp_bar(sh, B::A_EMPTY + ab), ((uint32_t)(ta / kPpABufs) & 1u) ^ 1u, abort, kWaitLimitNs)) { ok = false; break; }
                mbar_arrive_expect_tx(pp_bar(sh, B::A_FULL + ab), kPpABytes);
                tma_load_2d(sA + ab * kPpABytes, tmX_p, 0, (t_begin + ta) * kTileM, pp_bar(sh, B::A_FULL + ab));
                last_bar = pp_bar(sh, B::A_FULL + ab);
                last_par = (uint32_t)(ta / kPpABufs) & 1u;
            }
            if (!ok || *abort) {
                volatile int never = 0;
                mbar_wait(pp_bar(sh, B::W_FULL), 0u, &never, 10000000ull);
                mbar_wait(last_bar, last_par, &never, 10000000ull);
            }
        }
    } else if (warp == 3) {
        // ================= GEMM-1 issue (two units ahead of GEMM-2: three hidden buffers) =============
        if (nunits > 0) {
            constexpr uint32_t idesc1 = make_idesc(128, 128, kFmtBF16, kFmtBF16);
            const uint32_t dA = desc_lo_sw128(sA), dW1 = desc_lo_sw128(sW1);
            bool ok = true;
            ok = pp_wait(pp_bar(sh, B::W_FULL), 0u, abort);
#pragma unroll 1
            for (int u = 0; u < nunits && ok; ++u) {
                const int ta = u / nhalf, hf = u - ta * nhalf;
                const int ab = ta % kPpABufs;
                if (hf == 0 && !pp_wait(pp_bar(sh, B::A_FULL + ab), (uint32_t)(ta / kPpABufs) & 1u, abort)) { ok = false; break; }
                const uint32_t b = (uint32_t)u % 3u, n = (uint32_t)u / 3u;
                // (the buffer also held the hidden values of the unit three back: GEMM-2 must have read them)
                if (!pp_wait(pp_sbar(sh, 0, B::ACC1_EMPTY + b), (n & 1u) ^ 1u, abort)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t a0 = dA + ((ab * kPpABytes) >> 4), w0 = dW1 + ((hf * (128 * 128)) >> 4);
                const uint32_t d = tmem_base + b * C::HB_COLS;
                if (elect_one_sync()) {
                    mma_ss<0>(d, a0, w0, idesc1);
#pragma unroll
                    for (int kk = 1; kk < 4; ++kk) mma_ss<1>(d, a0 + ((kk * 32) >> 4), w0 + ((kk * 32) >> 4), idesc1);
                    mma_commit(pp_sbar(sh, 0, B::ACC1_FULL + b));
                    if (hf == nhalf - 1) mma_commit(pp_bar(sh, B::A_EMPTY + ab));
                }
                __syncwarp();
            }
            if (!ok || *abort) {
                volatile int never = 0;
                if (lane == 0) {
                    mma_commit(pp_bar(sh, B::DRAIN));
                    mbar_wait(pp_bar(sh, B::DRAIN), 0u, &never, 10000000ull);
                }
                __syncwarp();
            }
        }
    } else if (warp == 1) {
        // ================= GEMM-2 issue ===============================================================
        if (nunits > 0) {
            constexpr uint32_t idesc2 = make_idesc(128, EP, kFmtBF16, kFmtBF16);
            const uint32_t dW2 = desc_lo_sw128(sW2);
            bool ok = true;
            ok = pp_wait(pp_bar(sh, B::W_FULL), 0u, abort);
#pragma unroll 1
            for (int u = 0; u < nunits && ok; ++u) {
                const int ta = u / nhalf, hf = u - ta * nhalf;
                const int r = ta & 1;
                if (hf == 0 && !pp_wait(pp_sbar(sh, r, B::ACC2_EMPTY), ((uint32_t)(ta >> 1) & 1u) ^ 1u, abort)) { ok = false; break; }
                const uint32_t b = (uint32_t)u % 3u, n = (uint32_t)u / 3u;
                if (!pp_wait(pp_sbar(sh, 0, B::HID_FULL + b), n & 1u, abort)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t w0 = dW2 + ((hf * 2 * C::W2_CHUNK) >> 4);
                const uint32_t d = tmem_base + C::LOGIT_COL + r * 64, a = tmem_base + b * C::HB_COLS;
                if (elect_one_sync()) {
#pragma unroll
                    for (int part = 0; part < 2; ++part) {
#pragma unroll
                        for (int kk = 0; kk < 8; ++kk) {
                            const uint32_t bd = w0 + (((kk >> 2) * C::W2_CHUNK + (kk & 3) * 32) >> 4);
                            if (part == 0 && kk == 0) mma_ts_dyn(d, a, bd, idesc2, hf > 0 ? 1u : 0u);
                            else mma_ts<1>(d, a + kk * 16 + part * 8, bd, idesc2);
                        }
                    }
                    mma_commit(pp_sbar(sh, 0, B::ACC1_EMPTY + b));
                    if (hf == nhalf - 1) mma_commit(pp_sbar(sh, r, B::ACC2_FULL));
                }
                __syncwarp();
            }
            if (!ok || *abort) {
                volatile int never = 0;
                if (lane == 0) {
                    mma_commit(pp_bar(sh, B::DRAIN + 1));
                    mbar_wait(pp_bar(sh, B::DRAIN + 1), 0u, &never, 10000000ull);
                }
                __syncwarp();
            }
        }
    } else if (warp == 2) {
        // ================= zero this CTA's rows of h' =================================================
        if (p.zero_out != nullptr && ntiles > 0) {
            const long long row_lo = (long long)t_begin * kTileM;
            long long row_hi = (long long)(t_begin + ntiles) * kTileM;
            if (row_hi > p.n_rows) row_hi = p.n_rows;
            uint4* dst = reinterpret_cast<uint4*>(p.zero_out + row_lo * p.row_elems);
            const long long nvec = (row_hi - row_lo) * p.row_elems / 8;
            const uint4 z = make_uint4(0u, 0u, 0u, 0u);
            for (long long i = lane; i < nvec; i += 32) dst[i] = z;
        }
    } else if (warp < 20) {
        // ================= activation warps: warpgroup g, lane group lg ================================
        const int g = (warp - 4) >> 2;
        const int lg = warp & 3;
        const uint32_t tlane = tmem_base + ((uint32_t)(lg * 32) << 16) + 32 * g;
        const bool has_br1 = p.br1 != nullptr;
        bool ok = true;
#pragma unroll 1
        for (int u = 0; u < nunits && ok; ++u) {
            const int ta = u / nhalf, hf = u - ta * nhalf;
            const uint32_t b = (uint32_t)u % 3u, par = ((uint32_t)u / 3u) & 1u;
            ok = pp_wait(pp_sbar(sh, 0, B::ACC1_FULL + b), par, abort);
            if (!ok) break;
            tc_fence_after_sync();
            const uint32_t acol = tlane + b * C::HB_COLS;
            const float* bias = sh.bias1_f32 + hf * 128 + 32 * g;
            // relu(acc + bias) as hi + lo: hi = the value truncated to bf16 (negative -> 0 by .relu), lo = the
            // rounded remainder (for a negative value the remainder is the value itself and its .relu is 0 as
            // well).  The thread's 32 columns come with one tensor-memory load.
            uint32_t acc32[32];
            tmem_ld_x32(acol, acc32);
            tmem_ld_wait();
#pragma unroll
            for (int pc = 0; pc < 2; ++pc) {
                const uint32_t* acc = acc32 + 16 * pc;
                float a[16];
                if (has_br1) {
#pragma unroll
                    for (int i = 0; i < 16; i += 4) {
                        const float4 bb = *reinterpret_cast<const float4*>(bias + pc * 16 + i);
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
                tmem_st_x16(acol + 16 * pc, hl);
            }
            tmem_st_wait();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(pp_sbar(sh, 0, B::HID_FULL + b));
        }
    } else {
        // ================= output warpgroup ===========================================================
        // softmax + top-k of a tile's logits (ties go to the lower id), then either each pair's rank among this
        // CTA's pairs of its expert (for a ranked dispatch later) or, with lists_out, the dispatch itself: over a
        // group of up to LIST_GROUP tiles the pairs are counted per expert in shared memory and their entries
        // staged there; at the group's end ONE atomic per expert reserves a range of that expert's list and every
        // row thread appends its entries (few atomics per address however large the batch is).
        const int lg = warp & 3;
        const int row = lg * 32 + lane;
        const uint32_t tlane = tmem_base + ((uint32_t)(lg * 32) << 16) + C::LOGIT_COL;
        const bool lists = EP <= 32 && p.lists_out != nullptr;      // (more experts than 32 never take the list form)
        int* group_base = sh.tile_start;            // (unused by this pass otherwise)
        int32_t* counts = lists ? p.list_counts + sh.counts_set * (kMaxE * kPpCountStride) : nullptr;
        int4* stage = reinterpret_cast<int4*>(smem_raw + (smem_base - smem_u32(smem_raw)) + C::OFF_STAGE);
        bool ok = true;
#pragma unroll 1
        for (int ta = 0; ta < ntiles && ok; ++ta) {
            const int r = ta & 1;
            ok = pp_wait(pp_sbar(sh, r, B::ACC2_FULL), (uint32_t)(ta >> 1) & 1u, abort);
            if (!ok) break;
            tc_fence_after_sync();
            uint32_t v[EP];
#pragma unroll
            for (int c = 0; c < EP; c += 16) tmem_ld_x16(tlane + r * 64 + c, v + c);
            tmem_ld_wait();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(pp_sbar(sh, r, B::ACC2_EMPTY));
            const int n = (t_begin + ta) * kTileM + row;
            const bool valid = n < p.n_rows;
            // one pass keeping the best two (strict comparisons in ascending id order: same picks as
            // repeated arg-max with ties to the lower id); the logits stay in v as raw bits + bias
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
            float inv = 1.0f / sum;
            float p2 = ex2_approx(fmaf(b2, sc, -msc)) * inv;
            if (p.train_gates) {
                // Section 3.3: each assignment dropped iff the first word of Philox4x32-10(key = seed, counter =
                // (n, j, 0, 0)) is below the threshold; survivors divided by their sum; none left: top-1 gets 1
                uint32_t x[4];
                philox4x32_10((uint32_t)n, 0u, 0u, 0u, p.drop_key0, p.drop_key1, x);
                const bool d1 = (unsigned long long)x[0] < p.drop_threshold;
                bool d2 = true;
                if (p.k > 1) {
                    philox4x32_10((uint32_t)n, 1u, 0u, 0u, p.drop_key0, p.drop_key1, x);
                    d2 = (unsigned long long)x[0] < p.drop_threshold;
                }
                float kept_sum = 0.0f;
                if (!d1) kept_sum += inv;
                if (!d2) kept_sum += p2;
                const bool none = (d1 && d2) || !(kept_sum > 0.0f);
                inv = none ? 1.0f : (d1 ? 0.0f : inv / kept_sum);
                p2 = none ? 0.0f : (d2 ? 0.0f : p2 / kept_sum);
            }
            const size_t at = (size_t)n * p.k;
            int r1 = 0, r2 = 0;
            if (valid) {
                r1 = atomicAdd(&sh.hist[i1], 1);
                if (p.k > 1) {
                    // (k = 2: a row's two ids and its two probabilities as one 8-byte store each)
                    *reinterpret_cast<int2*>(p.topk_idx + at) = make_int2(i1, i2);
                    *reinterpret_cast<float2*>(p.topk_p + at) = make_float2(inv, p2);
                    r2 = atomicAdd(&sh.hist[i2], 1);
                } else {
                    p.topk_idx[at] = i1;
                    p.topk_p[at] = inv;
                }
                if (!lists && p.local_rank) {
                    p.local_rank[at] = r1;
                    if (p.k > 1) p.local_rank[at + 1] = r2;
                }
            }
            if (lists) {
                const int gt = ta % C::LIST_GROUP;           // tile of the group
                stage[(gt * 2 + 0) * kTileM + row] = make_int4(valid ? (int)at : -1, __float_as_int(inv), i1, r1);
                if (p.k > 1) stage[(gt * 2 + 1) * kTileM + row] = make_int4(valid ? (int)at + 1 : -1, __float_as_int(p2), i2, r2);
                if (gt == C::LIST_GROUP - 1 || ta == ntiles - 1) {
                    named_barrier_sync(2, 128);              // all of the group's pairs are counted
                    if (row < p.experts_real) {
                        const int cnt = sh.hist[row];
                        sh.hist[row] = 0;
                        group_base[row] = cnt > 0 ? atomicAdd(counts + row * kPpCountStride, cnt) : 0;
                    }
                    named_barrier_sync(2, 128);
                    for (int g = 0; g <= gt; ++g)
                        for (int j = 0; j < p.k; ++j) {
                            const int4 en = stage[(g * 2 + j) * kTileM + row];     // (this thread's own entry)
                            if (en.x >= 0) p.lists_out[(size_t)en.z * p.list_stride + group_base[en.z] + en.w] = make_int2(en.x, en.y);
                        }
                }
            }
        }
    }

    // ---- teardown ---------------------------------------------------------------------------------
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
}

// =====================================================================================================
// Dispatch without a capacity limit: the router left every pair's rank among its CTA's pairs of the same
// expert (local_rank) and each CTA's per-expert counts (table[c][e]).  A pair's stacked row is
// offsets[e] + (pairs of expert e in earlier CTAs) + local rank.  The order inside an expert is then the
// order in which the router's row threads drew their ranks, which varies from run to run; the layer's
// output does not depend on it (each stacked row is computed on its own, and the sum of at most two bf16
// values commutes), but `perm` / `dest` do, so this form is used only where they are not outputs and
// nothing is dropped (capacity limits need the stable order of the other dispatch).
// offs_out: shared memory, E + 1 ints.  `sm`: at least (2 E + 1 + G E) ints of shared memory.
// =====================================================================================================
template <int NT, bool SAME_LAUNCH>
__device__ __forceinline__ void pp_dispatch_body(const int32_t* topk_idx, const float* topk_p, const int32_t* local_rank,
                                                 const int32_t* table, int G, int chunk, int R, int E, int pairs_per_chunk,
                                                 int32_t* assigned, int32_t* kept, int32_t* offsets, int32_t* dest,
                                                 int2* pair_gate, int* sm, int* offs_out) {
    int* base = sm;            // [E] pairs of expert e in earlier CTAs, then + offsets
    int* total = sm + E;       // [E]
    int* tab = sm + 2 * E + 1; // [G * E] copy of the table
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long begin = (long long)chunk * pairs_per_chunk;
    long long end = begin + pairs_per_chunk;
    if (end > R) end = R;
    // Everything this CTA needs from global memory is requested up front, so that it pays the latency once:
    // the table (coalesced) and the first kPre of its own pairs per thread.
    constexpr int kPre = 4;
    int pe[kPre], pr[kPre];
    float pp[kPre];
#pragma unroll
    for (int q = 0; q < kPre; ++q) {
        const long long i = begin + threadIdx.x + (long long)q * NT;
        pe[q] = -1;
        if (i < end) {
            pe[q] = SAME_LAUNCH ? __ldcg(topk_idx + i) : topk_idx[i];
            pr[q] = SAME_LAUNCH ? __ldcg(local_rank + i) : local_rank[i];
            pp[q] = SAME_LAUNCH ? __ldcg(topk_p + i) : topk_p[i];
        }
    }
    for (int i = threadIdx.x; i < G * E; i += NT) tab[i] = SAME_LAUNCH ? __ldcg(table + i) : table[i];
    __syncthreads();
    // warp w sums experts w, w + NT/32, ...: lanes stride over the CTAs of the table
    for (int e = warp; e < E; e += NT / 32) {
        int before = 0, tot = 0;
        for (int c = lane; c < G; c += 32) {
            const int v = tab[c * E + e];
            tot += v;
            if (c < chunk) before += v;
        }
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) {
            before += __shfl_xor_sync(0xffffffffu, before, d);
            tot += __shfl_xor_sync(0xffffffffu, tot, d);
        }
        if (lane == 0) { base[e] = before; total[e] = tot; }
    }
    __syncthreads();
    if (warp == 0) {
        int run = 0;
        for (int e0 = 0; e0 < E; e0 += 32) {
            const int e = e0 + lane;
            const int tot = e < E ? total[e] : 0;
            int incl = tot;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const int up = __shfl_up_sync(0xffffffffu, incl, d);
                if (lane >= d) incl += up;
            }
            if (e < E) {
                const int o = run + incl - tot;
                offs_out[e] = o;
                base[e] += o;
                if (chunk == 0) {
                    if (assigned) assigned[e] = tot;
                    if (kept) kept[e] = tot;
                    offsets[e] = o;
                }
            }
            run += __shfl_sync(0xffffffffu, incl, 31);
        }
        if (lane == 0) {
            offs_out[E] = run;
            if (chunk == 0) offsets[E] = run;
        }
    }
    __syncthreads();
#pragma unroll
    for (int q = 0; q < kPre; ++q) {
        if (pe[q] >= 0) {
            const long long i = begin + threadIdx.x + (long long)q * NT;
            const int d = base[pe[q]] + pr[q];
            dest[i] = d;
            pair_gate[d] = make_int2((int)i, __float_as_int(pp[q]));
        }
    }
    for (long long i = begin + threadIdx.x + (long long)kPre * NT; i < end; i += NT) {
        const int e = SAME_LAUNCH ? __ldcg(topk_idx + i) : topk_idx[i];
        const int r = SAME_LAUNCH ? __ldcg(local_rank + i) : local_rank[i];
        const float pr2 = SAME_LAUNCH ? __ldcg(topk_p + i) : topk_p[i];
        const int d = base[e] + r;
        dest[i] = d;
        pair_gate[d] = make_int2((int)i, __float_as_int(pr2));
    }
}

// =====================================================================================================
// One-barrier form of the dispatch (one launch, E * 8 <= k * 128 so that the lists fit in the stacked-row
// scratch): the router's output warps fill per-expert lists themselves (pp_route_body with lists_out); after
// the grid barrier the counters are the experts' totals.  Expert e's list starts at lists + e * list_stride.
// =====================================================================================================
// After the barrier: the experts' row ranges from the counters (E <= 32: one warp).
__device__ __forceinline__ void pp_offsets_from_counts(const int32_t* counts, int E, int lane, bool write_out, int32_t* assigned,
                                                       int32_t* kept, int32_t* offsets, int* offs_out) {
    const int cnt = lane < E ? __ldcg(counts + lane * kPpCountStride) : 0;
    int incl = cnt;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const int up = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += up;
    }
    if (lane < E) {
        offs_out[lane] = incl - cnt;
        if (write_out) {
            if (assigned) assigned[lane] = cnt;
            if (kept) kept[lane] = cnt;
            offsets[lane] = incl - cnt;
        }
    }
    const int total = __shfl_sync(0xffffffffu, incl, 31);
    if (lane == 0) {
        offs_out[E] = total;
        if (write_out) offsets[E] = total;
    }
}

}  // namespace
}  // namespace slicemoe
