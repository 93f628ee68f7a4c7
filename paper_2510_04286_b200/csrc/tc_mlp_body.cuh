// Tensor-core path (sm_100a: tcgen05 + TMEM + TMA) for the two MLPs of the layer, bf16 storage:
//
//   router  (Section 3.1): relu(X Wr1^T + br1) Wr2^T + br2 -> softmax -> top-k   (per 128-row tile)
//   experts (Section 3.1 / 3.4): act(X~_e W1_e^T + b1_e) W2_e^T + b2_e           (per 128-row tile of
//                                                                                 one expert's rows)
//
// Both are the same pipeline (tc_body): GEMM-1 into a TMEM accumulator, an epilogue that applies
// gate, bias and activation and writes the hidden chunk as bf16 pairs back into TMEM, GEMM-2 with
// that chunk as its TMEM-resident A operand into a second TMEM accumulator, and a final epilogue
// (softmax + top-k + histogram for the router; bias + store or add for the experts).  The hidden
// layer is processed in chunks of HC units and never leaves tensor memory.
//
// One persistent CTA per SM walks a contiguous range of tiles (expert-major, so expert weights
// stay in shared memory while the expert does not change).  Warp roles:
//   warp 0            TMA producer (one lane): weight chunks with their bias, and the row tiles
//                     unless they are gathered
//   warp 1            GEMM-1 issue (one lane)
//   warp 2            GEMM-2 issue (one lane); two issuing threads because the small MMAs of this
//                     layer (N <= 128) are issue-bound, not tensor-bound
//   warp 3            fused forward only.  Router: zeroes this CTA's rows of h' (the experts add
//                     into it).  Experts: gathers the next tiles' rows of h through perm with
//                     asynchronous 16-byte copies into the swizzled A buffers, together with the
//                     rows' gates and pair indices
//   activation warps  two groups that take the hidden chunks in turn, each two warpgroups that
//                     split a chunk's columns; GEMM-1 accumulators are double-buffered
//   last warpgroup    output: final accumulator -> softmax/top-k, or bias + store / add into h'
// A warp reads TMEM lanes 32*(warp_id % 4)..+31: one tile row per thread.
// All hand-offs are mbarriers; every wait is bounded and a run-out sets the status word and makes
// all roles leave.
//
// This header holds the device code and the launch helpers; tc_mlp.cu wraps tc_body in the router
// and expert kernels, fused_forward.cu in the single-kernel forward.
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace slicemoe {
namespace {

using namespace ptx;

constexpr uint64_t kWaitLimitNs = 2000000000ull;   // a wait that takes 2 s is a bug, not load
constexpr int kMaxHid = 1024;
constexpr int kMaxE = 256;
// Depth of the per-tile metadata ring.  An entry is rewritten once GEMM-1 of the tile kMetaRing - 3
// tiles later has finished (three A buffers), by which time the activation warps have read their
// accumulators for the old tile and the output warps, at most two accumulators and one tile of
// GEMM-1 run-ahead behind, have stored it.
constexpr int kMetaRing = 8;
constexpr int kMaxBars = 48;
// Slots of the first-layer bias ring, indexed by the running count of W1 chunk loads.  Slot q is
// rewritten by load q + kBiasRing, which needs a free W1 slot, i.e. GEMM-1 of load q + kBiasRing -
// W_STAGES done, i.e. (accumulator hand-back) the activation of the chunks before it, load q's among
// them, finished; with resident weights a new expert's loads must not touch the previous expert's
// slots, hence at least two full sets.
constexpr int kBiasRing = 8;

struct TcParams {
    int experts_real;         // router: the real number of experts (<= the N2 the kernel is built for: E = 8 runs
                              // on the 16-wide instantiation, the padded experts' logits set to -inf)
    int row_elems;            // elements per row of X (= ds); at most the K1 the kernel is built for: a narrower
                              // row (the paper's own ds = 96 under K1 = 128) is zero-filled up to K1
    float softmax_scale;      // router: log2(e) / tau (Figure 7's temperature; top-k does not depend on it)
    const int32_t* offsets;   // experts: [E+1] device row ranges; router: nullptr
    int n_rows;               // router: N; experts: R (length of the stacked-row arrays)
    int E;                    // experts: E; router: 1
    int HID;                  // Hr or F
    const bf16* bias1;        // [E, HID] or nullptr
    const bf16* bias2;        // [E, N2]  or nullptr
    bf16* yperm;              // experts: output rows [R, N2]
    // experts, fused forward: A rows are gathered instead of read from stacked rows
    const bf16* gather_src;   // h viewed as X[N, K1], or nullptr (A = stacked rows via TMA)
    const int32_t* perm;      // [R] pair index n*k + j of each stacked row
    const float* gate;        // [R] gate value of each stacked row
    uint32_t gather_magic, gather_shift;   // row of pair i = (i * magic) >> shift = i / k (see pair_to_row)
    bf16* scatter_out;        // fused forward, k <= 2: h' viewed as Y[N, N2]; the row of pair (n, j) is added to
                              // Y[n, :] (h' zeroed beforehand) instead of being stored to yperm; or nullptr
    // experts, scatter_out with k = 1: a batch that leaves more than half of the CTAs without a tile is run as two
    // tiles per tile, each over one half of the hidden layer (two "virtual experts" per expert that share the
    // expert's rows: W1 / b1 rows [half HID/2, ...), W2 columns likewise, b2 with the first half only); both add
    // into the row of h', and a sum of two bf16 terms does not depend on their order
    int split_hidden;
    // router, fused forward: this CTA also zeroes the rows of zero_out that it routes
    bf16* zero_out;           // h' viewed as Y[N, zero_cols], or nullptr
    int zero_cols;
    int32_t* topk_idx;        // router outputs
    float* topk_p;
    int32_t* assigned;        // global counts, added atomically (or nullptr)
    int32_t* cta_hist;        // [gridDim.x, N2] this CTA's counts (or nullptr): input of the fused dispatch
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
    // 64-wide expert rows: four narrow chunks in flight, one warpgroup each (see NGRP below)
    static constexpr bool FOUR_GROUPS = (K1 == 64) && !ROUTER_;
    static constexpr int HC = (K1 == 64 && ROUTER_) ? 128 : 64;   // hidden units per chunk
    // row-tile buffers: three where they fit (the fused forward gathers two tiles ahead); with
    // 256-wide rows (64 KB per tile) the router gets two and the experts, whose weight stages are
    // larger, one
    static constexpr int A_BUFS = (K1 <= 128) ? 3 : (ROUTER_ ? 2 : 1);
    static constexpr int W_STAGES = (K1 == 128) ? 3 : (FOUR_GROUPS ? 4 : 2);
    // Activation warps: NGRP groups that take the hidden chunks in turn (chunk g goes to group
    // g mod NGRP), each group GWG warpgroups that split the chunk's columns.  With two groups one
    // group's accumulator loads, tails and stores run while the other group's tanh work occupies
    // the tanh unit.  256-wide rows get one group: their wide output epilogue needs the larger
    // register budget of a 512-thread CTA.
    // 64-wide expert rows run four groups of one warpgroup on four 64-column chunks instead: the
    // warps of a sub-partition are then in four different phases, and a warp in its tanh phase is
    // more often there to use the unit while the others load, convert and store.
    // Gather warps of the expert pass (forward): four, one per block of 32 rows of a tile (warp 3 and
    // three warps of an extra warpgroup behind the output warpgroup), because a single warp's copies and
    // address arithmetic were a bottleneck of the pass.  Where the warps come from:
    //   64-wide rows   three activation groups do as well as four (measured): the fourth's warpgroup
    //   128-wide rows  two groups of one warpgroup instead of two groups of two (a third group would
    //                  need a third accumulator, see NBUF >= NGRP below)
    //   256-wide rows  their CTA has room for another warpgroup (32 copies per block of rows here, four
    //                  times the 64-wide case)
    static constexpr bool ONE_WG_128 = !ROUTER_ && K1 == 128;
    static constexpr bool GATHER4 = !ROUTER_ && (FOUR_GROUPS || K1 == 256 || ONE_WG_128);
    // the router of the single-kernel forward runs in the same CTA: same number of threads
    static constexpr bool PAD_WARPGROUP = ROUTER_ && K1 == 256;
    static constexpr int GATHER_WARPS = GATHER4 ? 4 : 1;
    static constexpr int NGRP = (K1 == 256) ? 1 : (FOUR_GROUPS ? (GATHER4 ? 3 : 4) : 2);
    static constexpr int GWG = (FOUR_GROUPS || ONE_WG_128) ? 1 : 2;
    static constexpr int NWG = NGRP * GWG;
    // GEMM-1 accumulator / hidden buffers.  The router's hidden pair lives inside the accumulator it
    // came from (see the TMEM map), which leaves room for a third accumulator: GEMM-1 of the next two
    // chunks can then be issued while GEMM-2 still reads this one.
    static constexpr int NBUF = ROUTER_ ? 3 : (FOUR_GROUPS ? 4 : 2);
    static constexpr int GRP_WARPS = GWG * 4;                   // warps that work on one chunk
    // (ONE_WG_128: one more, idle, warpgroup so that the pass has the 768 threads of its router)
    static constexpr int THREADS = 128 + NWG * 128 + 128 + ((GATHER4 || PAD_WARPGROUP) ? 128 : 0) + (ONE_WG_128 ? 128 : 0);
    static constexpr int OUT_WARP0 = 4 + NWG * 4;               // first warp of the output warpgroup
    static constexpr int ACC2_BUFS = (N2 <= 128) ? 2 : 1;
    // The router keeps the hidden layer as a bf16 pair (hi + lo = 16 mantissa bits): GEMM-2 runs
    // over both halves against the same weights, so that the logits carry fp32-level accuracy and
    // the top-k decision does not depend on bf16 rounding of the hidden layer.
    // The experts keep it as plain bf16; their activation math is packed 2-wide bf16.
    // (A and B of one MMA must have the same 16-bit format: fp16 hidden x bf16 weights is an
    // illegal instruction on sm_100a.)
    static constexpr int H_PARTS = ROUTER_ ? 2 : 1;
    // How the two MMA-issuing warps run.  Router: all 32 lanes run the issue loop and one elected
    // lane issues, so that descriptors and addresses stay in uniform registers (its 40 small MMAs per
    // tile make it issue-bound: 153 -> 118 us on the largest workload), and so do the experts of
    // 256-wide rows (16 MMAs per chunk: 180 -> 176 us).  The other experts: one lane runs the loop;
    // their tile waits for the activation warps, and the wider issue warps only take issue slots from
    // those (64-wide rows: 260 -> 272 us with the router's scheme; 128-wide: no difference).
    static constexpr bool UNIFORM_ISSUE = ROUTER_ || K1 == 256;
    static constexpr bool PACKED_ACT = !ROUTER_;
    // TMEM columns:
    //   [0, NBUF HC)         GEMM-1 accumulators.  Warpgroup w of the group that has the chunk owns
    //                        columns [w HC/GWG, (w+1) HC/GWG).  Router: once a thread has read a
    //                        16-column piece (= one K step of GEMM-2) it writes the piece's hi half
    //                        into the piece's first 8 columns and the lo half into its last 8, so
    //                        K step kk of the hidden chunk is at columns 16 kk (hi) and 16 kk + 8 (lo).
    //   then (experts only)  NBUF hidden buffers of HC/2 packed columns (so GEMM-1 of a later chunk
    //                        need not wait for GEMM-2).
    //   then                 ACC2_BUFS final accumulators of N2 columns.
    static constexpr int H_COL0 = NBUF * HC;
    static constexpr int ACC2_COL0 = H_COL0 + (ROUTER_ ? 0 : NBUF * (HC / 2));
    static constexpr int TMEM_COLS = pow2_at_least(ACC2_COL0 + ACC2_BUFS * N2);
    static constexpr int KSTEPS_PER_WG = HC / (16 * GWG);       // 16-element K steps in one warpgroup's columns
    static constexpr int KP1 = K1 / 64;                         // 64-wide K panels of GEMM-1
    static constexpr int KP2 = HC / 64;                         // K panels of GEMM-2 per chunk
    static constexpr int A_PANEL = 128 * 128;                   // bytes: 128 rows x 128 B
    static constexpr int A_BYTES = KP1 * A_PANEL;
    static constexpr int W1_PANEL = HC * 128;
    static constexpr int W1C_BYTES = KP1 * W1_PANEL;
    static constexpr int W2_PANEL = N2 * 128;
    static constexpr int W2C_BYTES = KP2 * W2_PANEL;
    // W1 and W2 chunks live in two rings of W_STAGES slots each with their own barriers: a W1 slot
    // is handed back as soon as GEMM-1 has read it, so the next chunk's W1 streams in under this
    // chunk's activation and GEMM-2 instead of after them.
    static constexpr int OFF_A = 0;
    static constexpr int OFF_W = OFF_A + A_BUFS * A_BYTES;
    static constexpr int OFF_W2 = OFF_W + W_STAGES * W1C_BYTES;
    // The first layer's bias chunk arrives with W1 but is read after GEMM-1, by the activation
    // warps, so it has a ring of its own, deep enough that a slot is rewritten only by a W1 load
    // that cannot be issued before the old chunk's activation has finished (see kBiasRing).
    static constexpr int B1_BYTES = HC * 2;
    static constexpr int OFF_B1 = OFF_W2 + W_STAGES * W2C_BYTES;
    static constexpr int SMEM_BYTES = OFF_B1 + kBiasRing * B1_BYTES;
    // at least 120 KiB is requested so that two CTAs never share an SM (each allocates most of TMEM)
    static constexpr int SMEM_ALLOC = (SMEM_BYTES + 1024 > 120 * 1024) ? SMEM_BYTES + 1024 : 120 * 1024;
    static constexpr int PIECE = 16;                            // accumulator columns per piece
    static constexpr int NPIECE = HC / (PIECE * GWG);           // pieces per thread and chunk
    static constexpr int SUB = (NPIECE > 2) ? 2 : NPIECE;       // pieces held in registers at once (experts)
    static_assert(NPIECE % SUB == 0, "piece-to-batch map");
    static_assert(NPIECE >= 1, "hidden chunk too narrow for the activation warpgroups");
    static_assert(W2C_BYTES % 1024 == 0 && W1C_BYTES % 1024 == 0, "operand tiles must stay 1024-byte aligned");
    static_assert(kBiasRing >= 2 * W_STAGES, "bias ring");
    static_assert(N2 % 16 == 0 && N2 >= 16 && N2 <= 256, "MMA N");
    static_assert(SMEM_ALLOC <= 232448, "shared memory budget");
    static_assert(ACC2_COL0 + ACC2_BUFS * N2 <= 512, "TMEM budget");
    // A group waits on an accumulator's "full" barrier, and on a hidden buffer's "consumed" barrier, only
    // for its own chunks and so skips phases; the parity test of its next wait is only right if the phase
    // before the awaited one is over by then.  Both GEMMs finish in chunk order; the group's previous
    // chunk is NGRP chunks back (its accumulator was complete, and the GEMM-2 that freed its hidden
    // buffer was NGRP + NBUF chunks back), the barrier's previous phase NBUF (2 NBUF) chunks back: fine
    // as long as NBUF >= NGRP.
    static_assert(NBUF >= NGRP, "accumulator barriers: a group must not run a whole phase ahead");
};

// Barrier slots in shared memory.
template <class C>
struct Bars {
    static constexpr int A_FULL = 0;
    static constexpr int A_EMPTY = A_FULL + C::A_BUFS;
    static constexpr int W1_FULL = A_EMPTY + C::A_BUFS;
    static constexpr int W1_EMPTY = W1_FULL + C::W_STAGES;    // GEMM-1 has read the W1 slot
    static constexpr int W2_FULL = W1_EMPTY + C::W_STAGES;
    static constexpr int W2_EMPTY = W2_FULL + C::W_STAGES;    // GEMM-2 has read the W2 slot
    static constexpr int ACC1_FULL = W2_EMPTY + C::W_STAGES;  // GEMM-1 done (MMA -> activation)
    // accumulator may be overwritten: experts, all activation warps have read it;
    // router (hidden chunk lives in it), GEMM-2 has consumed it
    static constexpr int ACC1_EMPTY = ACC1_FULL + C::NBUF;
    static constexpr int H_FULL = ACC1_EMPTY + C::NBUF;       // hidden chunk written (activation -> MMA)
    static constexpr int H_EMPTY = H_FULL + C::NBUF;          // experts: GEMM-2 has consumed the hidden buffer
    static constexpr int ACC2_FULL = H_EMPTY + C::NBUF;
    static constexpr int ACC2_EMPTY = ACC2_FULL + C::ACC2_BUFS;
    static constexpr int DRAIN = ACC2_EMPTY + C::ACC2_BUFS;
    static constexpr int COUNT = DRAIN + 2;
};

// (s: 0, or 1 when every expert is two virtual experts over the same rows; e counts virtual experts)
__device__ __forceinline__ void locate_tile(const int* tile_start, const int* offs, int t, int& e,
                                            int& row0, int& rows, int s = 0) {
    while (t >= tile_start[e + 1]) ++e;
    row0 = offs[e >> s] + (t - tile_start[e]) * kTileM;
    rows = min(kTileM, offs[(e >> s) + 1] - row0);
}

// Row n = pair / k of a pair index, k = 1..8, without a division: (pair * magic) >> shift with
// magic = ceil(2^shift / k) (1 and log2 k for a power of two); the reciprocal's error stays below 1/k
// over 31-bit pair indices (checked exhaustively at the edges and on random indices for every k).
__device__ __forceinline__ int pair_to_row(int pair, uint32_t magic, uint32_t shift) {
    return (int)(((unsigned long long)(uint32_t)pair * magic) >> shift);
}
inline void pair_to_row_magic(int k, uint32_t* magic, uint32_t* shift) {
    if ((k & (k - 1)) == 0) {
        *magic = 1u;
        *shift = 0u;
        while ((1 << *shift) < k) ++*shift;
    } else {
        *shift = k == 3 ? 33u : 34u;
        *magic = (uint32_t)(((1ull << *shift) + (unsigned)k - 1) / (unsigned)k);
    }
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// packed fp32 arithmetic (two lanes per instruction)
__device__ __forceinline__ void fma2(float& d0, float& d1, float a0, float a1, float b0, float b1, float c0, float c1) {
    asm("{\n\t.reg .b64 ra, rb, rc, rd;\n\t"
        "mov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\tmov.b64 rc, {%6, %7};\n\t"
        "fma.rn.f32x2 rd, ra, rb, rc;\n\t"
        "mov.b64 {%0, %1}, rd;\n\t}"
        : "=f"(d0), "=f"(d1) : "f"(a0), "f"(a1), "f"(b0), "f"(b1), "f"(c0), "f"(c1));
}
__device__ __forceinline__ void mul2(float& d0, float& d1, float a0, float a1, float b0, float b1) {
    asm("{\n\t.reg .b64 ra, rb, rd;\n\t"
        "mov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\t"
        "mul.rn.f32x2 rd, ra, rb;\n\t"
        "mov.b64 {%0, %1}, rd;\n\t}"
        : "=f"(d0), "=f"(d1) : "f"(a0), "f"(a1), "f"(b0), "f"(b1));
}
__device__ __forceinline__ void add2(float& d0, float& d1, float a0, float a1, float b0, float b1) {
    asm("{\n\t.reg .b64 ra, rb, rd;\n\t"
        "mov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\t"
        "add.rn.f32x2 rd, ra, rb;\n\t"
        "mov.b64 {%0, %1}, rd;\n\t}"
        : "=f"(d0), "=f"(d1) : "f"(a0), "f"(a1), "f"(b0), "f"(b1));
}
// Expert activation, all arithmetic 2-wide in bf16 on one thread's 16-column piece of a row:
//   convert   z = bf16(acc * gate + bias)             Eq. 1's gate and the bias meet the fp32 accumulator before the
//                                                     first rounding: one packed fp32 multiply-add, one conversion
//   pre       t = tanh(z (c0 + c1 z^2))               three multiply-adds and one packed tanh per pair
//   post      2 gelu(z) = z t + z                     one multiply-add per pair
// GELU, tanh form: 0.5 z (1 + tanh(sqrt(2/pi) (z + 0.044715 z^3))); the factor 0.5 is applied to
// the GEMM-2 accumulator in the output epilogue (exact: a power of two).  Where z^2 overflows, tanh
// saturates to +-1 and the formula still returns 2z (z > 0) or 0 (z < 0).
// The tanh unit (16 results per clock per SM) is the scarce resource; the instruction count around
// it is kept low enough that the issue slots are not the next one.
__device__ __forceinline__ void convert_piece_bf16x2(const uint32_t* cur, float gate, const uint4* bias8, bool has_bias,
                                                     __nv_bfloat162* z) {
    uint4 braw[2];
    if (has_bias) { braw[0] = bias8[0]; braw[1] = bias8[1]; }      // 16 packed bf16, warp-wide broadcast
    else braw[0] = braw[1] = make_uint4(0u, 0u, 0u, 0u);
    const uint32_t* b2 = reinterpret_cast<const uint32_t*>(braw);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        float z0, z1;                                               // (a bf16 is the upper half of its fp32)
        fma2(z0, z1, __uint_as_float(cur[2 * i]), __uint_as_float(cur[2 * i + 1]), gate, gate,
             __uint_as_float(b2[i] << 16), __uint_as_float(b2[i] & 0xffff0000u));
        z[i] = __floats2bfloat162_rn(z0, z1);
    }
}
template <int ACT>
__device__ __forceinline__ void activate_pre_bf16x2(const __nv_bfloat162* z, __nv_bfloat162* t) {
    constexpr int P = 8;   // column pairs per piece
    if (ACT == SLICEMOE_ACT_RELU) return;
    const __nv_bfloat162 c0 = __float2bfloat162_rn(0.7978845608f), c1 = __float2bfloat162_rn(0.0356774081f);
#pragma unroll
    for (int i = 0; i < P; ++i) {
        const __nv_bfloat162 inner = __hfma2(__hmul2(z[i], z[i]), c1, c0);
        const __nv_bfloat162 u = __hmul2(z[i], inner);
        uint32_t ur = *reinterpret_cast<const uint32_t*>(&u), tr;
        asm volatile("tanh.approx.bf16x2 %0, %1;" : "=r"(tr) : "r"(ur));
        t[i] = *reinterpret_cast<__nv_bfloat162*>(&tr);
    }
}
template <int ACT>
__device__ __forceinline__ void activate_post_bf16x2(const __nv_bfloat162* z, const __nv_bfloat162* t, uint32_t* out) {
    constexpr int P = 8;
    constexpr bool relu = ACT == SLICEMOE_ACT_RELU;
    if constexpr (relu) {
        const __nv_bfloat162 zero = __float2bfloat162_rn(0.0f);
#pragma unroll
        for (int i = 0; i < P; ++i) {
            const __nv_bfloat162 r = __hmax2(z[i], zero);
            out[i] = *reinterpret_cast<const uint32_t*>(&r);
        }
    } else {
#pragma unroll
        for (int i = 0; i < P; ++i) {
            const __nv_bfloat162 r = __hfma2(z[i], t[i], z[i]);
            out[i] = *reinterpret_cast<const uint32_t*>(&r);
        }
    }
}
// factor the output epilogue applies to the GEMM-2 accumulator (see above)
template <int ACT>
constexpr float kOutScale =
    (ACT == SLICEMOE_ACT_RELU) ? 1.0f : 0.5f;

// Router: relu(acc + bias) as a bf16 pair per value: hi = the value truncated to bf16, lo = the
// rounded remainder; hi + lo carries 16 mantissa bits of the fp32 value.  The ReLU rides on the two
// conversions: hi is converted round-toward-zero with .relu (a negative value gives hi = 0), so the
// remainder a - hi is a itself for a < 0 and non-negative otherwise, and the .relu of the second
// conversion zeroes exactly the negative inputs.  Per column pair: 2 adds, 1 conversion, 2 unpacks,
// 2 subtractions, 1 conversion.
__device__ __forceinline__ uint32_t cvt_rz_relu_bf16x2(float lo, float hi) {
    uint32_t d;
    asm("cvt.rz.relu.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}
__device__ __forceinline__ uint32_t cvt_rn_relu_bf16x2(float lo, float hi) {
    uint32_t d;
    asm("cvt.rn.relu.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}
// (has_bias = false: no shared-memory reads and no adds; every load the row threads issue passes through the same
// queue as their tensor-memory loads and stores)
__device__ __forceinline__ void bias_relu_split_piece(const uint32_t* cur, const float* bias /* 16 fp32, shared */,
                                                      uint32_t* hi, uint32_t* lo, bool has_bias = true) {
    constexpr int P = 8;
    float a[2 * P];
    if (has_bias) {
#pragma unroll
        for (int i = 0; i < 2 * P; i += 4) {
            const float4 b = *reinterpret_cast<const float4*>(bias + i);      // same address for the whole warp
            a[i] = __uint_as_float(cur[i]) + b.x;
            a[i + 1] = __uint_as_float(cur[i + 1]) + b.y;
            a[i + 2] = __uint_as_float(cur[i + 2]) + b.z;
            a[i + 3] = __uint_as_float(cur[i + 3]) + b.w;
        }
    } else {
#pragma unroll
        for (int i = 0; i < 2 * P; ++i) a[i] = __uint_as_float(cur[i]);
    }
#pragma unroll
    for (int i = 0; i < P; ++i) hi[i] = cvt_rz_relu_bf16x2(a[2 * i], a[2 * i + 1]);
#pragma unroll
    for (int i = 0; i < P; ++i)
        lo[i] = cvt_rn_relu_bf16x2(a[2 * i] - __uint_as_float(hi[i] << 16), a[2 * i + 1] - __uint_as_float(hi[i] & 0xFFFF0000u));
}

// Shared-memory state of one CTA besides the operand tiles.
struct TcShared {
    __align__(8) uint64_t bars[kMaxBars];
    int tile_start[kMaxE + 1];
    int offs[kMaxE + 1];
    int hist[kMaxE];
    uint32_t tmem_base;
    int abort_flag;
    int split_shift;          // 1: two virtual experts per expert (TcParams::split_hidden), else 0
    // fused forward: per-row gate (Eq. 1) and pair index of the tiles in flight, copied in by the
    // gather warp with the rows themselves (ring over the CTA's tile counter)
    float gate_s[kMetaRing][kTileM];
    int pair_s[kMetaRing][kTileM];
    // router: the first layer's bias as fp32 (the router's weights never change inside a pass)
    __align__(16) float bias1_f32[kMaxHid];
    __align__(16) float bias2_f32[kMaxE];
};

// Loads of data that an earlier phase of the same launch may have written (single-kernel forward)
// must not take the non-coherent path.
template <bool SAME_LAUNCH>
__device__ __forceinline__ int ld_index(const int32_t* ptr) {
    if (SAME_LAUNCH) return __ldcg(ptr);
    return __ldg(ptr);
}

// One pass of the two-layer MLP pipeline over this CTA's share of the row tiles: the body of the
// router and expert kernels, and of the router and expert phases of the single-kernel forward.
// Called by all threads of the CTA; TMEM (sh.tmem_base, at least C::TMEM_COLS columns) is allocated
// and freed by the caller.  SAME_LAUNCH: offsets / perm / gate were written earlier in this launch;
// OFFS_IN_SMEM: sh.offs already holds the row ranges.
template <class C, bool SAME_LAUNCH, bool OFFS_IN_SMEM = false, bool FUSED = false>
__device__ __forceinline__ void tc_body(const CUtensorMap* tmA_p, const CUtensorMap* tmW1_p, const CUtensorMap* tmW2_p,
                                        const TcParams& p, TcShared& sh, uint8_t* smem_raw) {
    using B = Bars<C>;
    static_assert(B::COUNT <= kMaxBars, "barrier slots");
    const CUtensorMap& tmA = *tmA_p;
    const CUtensorMap& tmW1 = *tmW1_p;
    const CUtensorMap& tmW2 = *tmW2_p;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    volatile int* abort = &sh.abort_flag;
    // FUSED (the single-kernel forward): what that caller always asks for is fixed at compile time --
    // rows gathered and results added into h' (experts); no probability matrix, no global counts, k <= 2,
    // h' zeroed (router) -- so that the other variants' code is not part of its hot loops
    const bool gather = !C::ROUTER && (FUSED || p.gather_src != nullptr);
    auto bar = [&](int i) { return smem_u32(&sh.bars[i]); };

    // ---- set-up ---------------------------------------------------------------------------
    if (threadIdx.x == 0) {
        sh.abort_flag = 0;
        for (int i = 0; i < C::A_BUFS; ++i) { mbar_init(bar(B::A_FULL + i), gather ? 32 * C::GATHER_WARPS : 1); mbar_init(bar(B::A_EMPTY + i), 1); }
        for (int i = 0; i < C::W_STAGES; ++i) {
            mbar_init(bar(B::W1_FULL + i), 1); mbar_init(bar(B::W1_EMPTY + i), 1);
            mbar_init(bar(B::W2_FULL + i), 1); mbar_init(bar(B::W2_EMPTY + i), 1);
        }
        for (int i = 0; i < C::NBUF; ++i) {
            mbar_init(bar(B::ACC1_FULL + i), 1);
            mbar_init(bar(B::ACC1_EMPTY + i), C::ROUTER ? 1 : C::GRP_WARPS);
            mbar_init(bar(B::H_FULL + i), C::GRP_WARPS);
            mbar_init(bar(B::H_EMPTY + i), 1);
        }
        for (int i = 0; i < C::ACC2_BUFS; ++i) {
            mbar_init(bar(B::ACC2_FULL + i), 1);
            mbar_init(bar(B::ACC2_EMPTY + i), 4);
        }
        mbar_init(bar(B::DRAIN), 1);
        mbar_init(bar(B::DRAIN + 1), 1);
        fence_mbar_init();
        prefetch_tensormap(&tmA);
        prefetch_tensormap(&tmW1);
        prefetch_tensormap(&tmW2);
    }
    // row ranges: the router's single range, the experts' offsets from global memory, or (single-kernel
    // forward) already in sh.offs, left there by the dispatch phase of this CTA
    if (!OFFS_IN_SMEM)
        for (int e = threadIdx.x; e <= p.E; e += C::THREADS) sh.offs[e] = p.offsets ? p.offsets[e] : (e == 0 ? 0 : p.n_rows);
    for (int e = threadIdx.x; e < kMaxE; e += C::THREADS) sh.hist[e] = 0;
    if constexpr (C::ROUTER)
        for (int i = threadIdx.x; i < p.HID; i += C::THREADS)
            sh.bias1_f32[i] = p.bias1 ? __bfloat162float(p.bias1[i]) : 0.0f;
    // experts without a first-layer bias: the ring the activation warps read their bias chunks from
    // stays all zero (no loads into it), so that their loop has no second, bias-free copy
    if constexpr (!C::ROUTER)
        if (p.bias1 == nullptr)
            for (int i = threadIdx.x; i < kBiasRing * C::B1_BYTES / 4; i += C::THREADS)
                reinterpret_cast<uint32_t*>(smem_raw + (smem_base - smem_u32(smem_raw)) + C::OFF_B1)[i] = 0u;
    if constexpr (C::ROUTER)
        for (int i = threadIdx.x; i < C::N2; i += C::THREADS)
            sh.bias2_f32[i] = i >= p.experts_real ? -INFINITY : (p.bias2 ? __bfloat162float(p.bias2[i]) : 0.0f);
    __syncthreads();
    if (warp == 0) {
        // first tile of every (virtual) expert: exclusive scan of the tile counts, 32 experts at a time; a second
        // time over two virtual experts per expert when that still leaves every CTA at most one tile
        // (256-wide rows only: that is where a tile is long enough for the split to pay -- 29.7 -> 22.6 us for the 40
        // tiles of the skewed benchmark batch -- and the narrower instantiations keep their register budget)
        const bool may_split = !C::ROUTER && C::K1 == 256 && p.split_hidden && p.HID % (2 * C::HC) == 0 &&
                               p.HID >= 4 * C::HC && 2 * p.E <= kMaxE;
        int s = 0;
        for (;;) {
            const int EV = p.E << s;
            int run = 0;
            for (int e0 = 0; e0 < EV; e0 += 32) {
                const int e = e0 + lane;
                const int nt = e < EV ? (sh.offs[(e >> s) + 1] - sh.offs[e >> s] + kTileM - 1) / kTileM : 0;
                int incl = nt;
#pragma unroll
                for (int d = 1; d < 32; d <<= 1) {
                    const int up = __shfl_up_sync(0xffffffffu, incl, d);
                    if (lane >= d) incl += up;
                }
                if (e < EV) sh.tile_start[e] = run + incl - nt;
                run += __shfl_sync(0xffffffffu, incl, 31);
            }
            if (lane == 0) sh.tile_start[EV] = run;
            __syncwarp();
            if (s == 0 && may_split && run > 0 && 2 * run <= (int)gridDim.x) s = 1;
            else break;
        }
        if (lane == 0) sh.split_shift = s;
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = sh.tmem_base;
    const int vs = (C::ROUTER || C::K1 != 256) ? 0 : sh.split_shift;          // virtual-expert shift
    const int hid = p.HID >> vs;                             // hidden units per (virtual) expert
    const int nchunks = hid / C::HC;
    const bool resident = nchunks <= C::W_STAGES;
    const int total_tiles = sh.tile_start[p.E << vs];
    const int per_cta = (total_tiles + gridDim.x - 1) / gridDim.x;
    const int t_begin = min(total_tiles, (int)blockIdx.x * per_cta);
    const int t_end = min(total_tiles, t_begin + per_cta);

    const uint32_t sA = smem_base + C::OFF_A, sW = smem_base + C::OFF_W;

    // result of a wait in an MMA-issuing warp: with all lanes in the loop they must leave it together
    auto all_lanes_agree = [](bool r) { return C::UNIFORM_ISSUE ? (bool)__all_sync(0xffffffffu, r) : r; };
    if (warp == 0) {
        // ================= TMA producer =====================================================
        // One thread, per tile: the row tile (unless rows are gathered), then per chunk W1 (with its
        // bias) and W2, each into its own ring behind its own "slot free" barrier.  All waits park
        // the thread (no polling).  W1 of chunk g waits for GEMM-1 of the chunk that had the slot;
        // W2 of chunk g for GEMM-2 of the chunk that had its slot, which may come a little later
        // than the next W1 slot frees up -- a short delay, against a full weight round trip on the
        // critical path when both halves shared one slot.
        if (lane == 0 && t_begin < t_end) {
            int e = 0, prev_e = -1;
            uint32_t g = 0, reloads = 0;             // chunks seen; tiles that (re)loaded weights
            uint32_t wq = 0;                         // W1 chunk loads issued (bias ring position)
            uint32_t last_bar[3] = {0, 0, 0}, last_par[3] = {0, 0, 0};
            bool ok = true;
            for (int t = t_begin, ta = 0; t < t_end && ok; ++t, ++ta) {
                int row0, rows;
                locate_tile(sh.tile_start, sh.offs, t, e, row0, rows, vs);
                const int ab = ta % C::A_BUFS;
                const uint32_t an = ta / C::A_BUFS;
                if (!gather) {
                    if (!mbar_wait(bar(B::A_EMPTY + ab), (an & 1u) ^ 1u, abort, kWaitLimitNs)) { ok = false; break; }
                    mbar_arrive_expect_tx(bar(B::A_FULL + ab), C::A_BYTES);
#pragma unroll
                    for (int kp = 0; kp < C::KP1; ++kp)
                        tma_load_2d(sA + ab * C::A_BYTES + kp * C::A_PANEL, &tmA, kp * 64, row0, bar(B::A_FULL + ab));
                    last_bar[0] = bar(B::A_FULL + ab);
                    last_par[0] = an & 1u;
                }
                const bool reload = !resident || (e != prev_e);
                prev_e = e;
                if (!reload) { g += nchunks; continue; }
                for (int c = 0; c < nchunks && ok; ++c, ++g) {
                    // resident weights: slot = chunk, n-th load of the slot = n-th reloading tile;
                    // streamed weights: slots in ring order
                    const int slot = resident ? c : (int)(g % C::W_STAGES);
                    const uint32_t n = resident ? reloads : g / C::W_STAGES;
                    if (!mbar_wait(bar(B::W1_EMPTY + slot), (n & 1u) ^ 1u, abort, kWaitLimitNs)) { ok = false; break; }
                    mbar_arrive_expect_tx(bar(B::W1_FULL + slot), C::W1C_BYTES + (p.bias1 ? C::B1_BYTES : 0));
                    if (p.bias1)
                        bulk_load(smem_base + C::OFF_B1 + (wq % kBiasRing) * C::B1_BYTES,
                                  p.bias1 + (size_t)e * hid + c * C::HC, C::B1_BYTES, bar(B::W1_FULL + slot));
#pragma unroll
                    for (int kp = 0; kp < C::KP1; ++kp)
                        tma_load_2d(sW + slot * C::W1C_BYTES + kp * C::W1_PANEL, &tmW1, kp * 64, e * hid + c * C::HC,
                                    bar(B::W1_FULL + slot));
                    last_bar[1] = bar(B::W1_FULL + slot);
                    last_par[1] = n & 1u;
                    ++wq;
                    if (!mbar_wait(bar(B::W2_EMPTY + slot), (n & 1u) ^ 1u, abort, kWaitLimitNs)) { ok = false; break; }
                    mbar_arrive_expect_tx(bar(B::W2_FULL + slot), C::W2C_BYTES);
#pragma unroll
                    for (int kp = 0; kp < C::KP2; ++kp)
                        tma_load_2d(smem_base + C::OFF_W2 + slot * C::W2C_BYTES + kp * C::W2_PANEL, &tmW2,
                                    (e & vs) * hid + c * C::HC + kp * 64, (e >> vs) * C::N2, bar(B::W2_FULL + slot));
                    last_bar[2] = bar(B::W2_FULL + slot);
                    last_par[2] = n & 1u;
                }
                ++reloads;
            }
            if (!ok || *abort) {
                // leaving early: let this thread's last copies land first (bounded; the copies
                // complete on their own, earlier ones of a stream were issued before its last)
                volatile int never = 0;
                for (int i = 0; i < 3; ++i)
                    if (last_bar[i]) mbar_wait(last_bar[i], last_par[i], &never, 10000000ull);
            }
        }
    } else if (warp == 1) {
        // ================= GEMM-1 issue ======================================================
        // (UNIFORM_ISSUE: all lanes run the loop and one elected lane issues, see elect_one_sync;
        // otherwise lane 0 alone)
        if (t_begin < t_end && (C::UNIFORM_ISSUE || lane == 0)) {
            constexpr uint32_t idesc1 = make_idesc(128, C::HC, kFmtBF16, kFmtBF16);
            const uint32_t dA = desc_lo_sw128(sA), dW = desc_lo_sw128(sW);
            bool ok = true;
            int e = 0, prev_e = -1;
            uint32_t g = 0, reloads = 0;
            for (int t = t_begin, ta = 0; t < t_end && ok; ++t, ++ta) {
                int r0, rr;
                locate_tile(sh.tile_start, sh.offs, t, e, r0, rr, vs);
                const bool reload = !resident || (e != prev_e);
                prev_e = e;
                const int ab = ta % C::A_BUFS;
                ok = all_lanes_agree(mbar_wait(bar(B::A_FULL + ab), (uint32_t)(ta / C::A_BUFS) & 1u, abort, kWaitLimitNs));
                if (!ok) break;
                if (gather) fence_proxy_async_smem();   // rows written by cp.async -> visible to the MMA's reads
                for (int c = 0; c < nchunks; ++c, ++g) {
                    const int slot = resident ? c : (int)(g % C::W_STAGES);
                    if (reload) {
                        const uint32_t n = resident ? reloads : g / C::W_STAGES;
                        ok = all_lanes_agree(mbar_wait(bar(B::W1_FULL + slot), n & 1u, abort, kWaitLimitNs));
                        if (!ok) break;
                    }
                    const uint32_t b = g % C::NBUF, n1 = g / C::NBUF;
                    ok = all_lanes_agree(mbar_wait(bar(B::ACC1_EMPTY + b), (n1 & 1u) ^ 1u, abort, kWaitLimitNs));
                    if (!ok) break;
                    tc_fence_after_sync();
                    const uint32_t a0 = dA + ((ab * C::A_BYTES) >> 4), w0 = dW + ((slot * C::W1C_BYTES) >> 4);
                    const uint32_t d = tmem_base + b * C::HC;
                    if (!C::UNIFORM_ISSUE || elect_one_sync()) {
                        mma_ss<0>(d, a0, w0, idesc1);
#pragma unroll
                        for (int kk = 1; kk < C::K1 / 16; ++kk)
                            mma_ss<1>(d, a0 + (((kk >> 2) * C::A_PANEL + (kk & 3) * 32) >> 4),
                                      w0 + (((kk >> 2) * C::W1_PANEL + (kk & 3) * 32) >> 4), idesc1);
                        mma_commit(bar(B::ACC1_FULL + b));
                        // streamed weights: the W1 slot is free as soon as these MMAs have read it
                        // (resident weights are handed back by the GEMM-2 warp at an expert change)
                        if (!resident) mma_commit(bar(B::W1_EMPTY + slot));
                        if (c == nchunks - 1) mma_commit(bar(B::A_EMPTY + ab));
                    }
                    if (C::UNIFORM_ISSUE) __syncwarp();
                }
                if (reload) ++reloads;
            }
            if (!ok || *abort) {
                // make sure no MMA of this warp is still running before TMEM is released
                volatile int never = 0;
                if (lane == 0) {
                    mma_commit(bar(B::DRAIN));
                    mbar_wait(bar(B::DRAIN), 0u, &never, 10000000ull);
                }
                if (C::UNIFORM_ISSUE) __syncwarp();
            }
        }
    } else if (warp == 2) {
        // ================= GEMM-2 issue ======================================================
        if (t_begin < t_end && (C::UNIFORM_ISSUE || lane == 0)) {
            constexpr uint32_t idesc2 = make_idesc(128, C::N2, kFmtBF16, kFmtBF16);
            const uint32_t dW = desc_lo_sw128(smem_base + C::OFF_W2);
            bool ok = true;
            int e = 0, prev_e = -1;
            uint32_t g = 0, reloads = 0;
            for (int t = t_begin, ta = 0; t < t_end && ok; ++t, ++ta) {
                int r0, rr;
                locate_tile(sh.tile_start, sh.offs, t, e, r0, rr, vs);
                const bool reload = !resident || (e != prev_e);
                prev_e = e;
                // resident weights are handed back only when the next tile brings another expert
                bool release = !resident;
                if (resident && t + 1 < t_end) {
                    int e2 = e;
                    locate_tile(sh.tile_start, sh.offs, t + 1, e2, r0, rr, vs);
                    release = (e2 != e);
                }
                const int buf = ta % C::ACC2_BUFS;
                for (int c = 0; c < nchunks; ++c, ++g) {
                    const int slot = resident ? c : (int)(g % C::W_STAGES);
                    if (reload) {
                        const uint32_t n = resident ? reloads : g / C::W_STAGES;
                        ok = all_lanes_agree(mbar_wait(bar(B::W2_FULL + slot), n & 1u, abort, kWaitLimitNs));
                        if (!ok) break;
                    }
                    const uint32_t b = g % C::NBUF, n1 = g / C::NBUF;
                    ok = all_lanes_agree(mbar_wait(bar(B::H_FULL + b), n1 & 1u, abort, kWaitLimitNs));
                    if (!ok) break;
                    if (c == 0) {
                        ok = all_lanes_agree(mbar_wait(bar(B::ACC2_EMPTY + buf), ((uint32_t)(ta / C::ACC2_BUFS) & 1u) ^ 1u,
                                                               abort, kWaitLimitNs));
                        if (!ok) break;
                    }
                    tc_fence_after_sync();
                    const uint32_t w0 = dW + ((slot * C::W2C_BYTES) >> 4);
                    const uint32_t d = tmem_base + C::ACC2_COL0 + buf * C::N2;
                    const uint32_t hbuf = tmem_base + C::H_COL0 + b * (C::HC / 2);   // experts: the hidden chunk
                    const uint32_t hacc = tmem_base + b * C::HC;                     // router: hi / lo inside the accumulator
                    if (!C::UNIFORM_ISSUE || elect_one_sync()) {
#pragma unroll
                        for (int part = 0; part < C::H_PARTS; ++part) {
#pragma unroll
                            for (int kk = 0; kk < C::HC / 16; ++kk) {
                                uint32_t a;
                                if (C::ROUTER)
                                    a = hacc + kk * 16 + part * 8;
                                else
                                    a = hbuf + kk * 8;
                                const uint32_t bd = w0 + (((kk >> 2) * C::W2_PANEL + (kk & 3) * 32) >> 4);
                                if (part == 0 && kk == 0) mma_ts_dyn(d, a, bd, idesc2, c > 0 ? 1u : 0u);
                                else mma_ts<1>(d, a, bd, idesc2);
                            }
                        }
                        mma_commit(bar((C::ROUTER ? B::ACC1_EMPTY : B::H_EMPTY) + b));
                        if (release) {
                            mma_commit(bar(B::W2_EMPTY + slot));
                            if (resident) mma_commit(bar(B::W1_EMPTY + slot));   // GEMM-1 of this chunk finished before its GEMM-2 began
                        }
                        if (c == nchunks - 1) mma_commit(bar(B::ACC2_FULL + buf));
                    }
                    if (C::UNIFORM_ISSUE) __syncwarp();
                }
                if (reload) ++reloads;
            }
            if (!ok || *abort) {
                volatile int never = 0;
                if (lane == 0) {
                    mma_commit(bar(B::DRAIN + 1));
                    mbar_wait(bar(B::DRAIN + 1), 0u, &never, 10000000ull);
                }
                if (C::UNIFORM_ISSUE) __syncwarp();
            }
        }
    } else if (warp == 3 || (C::GATHER4 && warp >= C::OUT_WARP0 + 4 && warp < C::OUT_WARP0 + 7)) {
        if constexpr (C::ROUTER) {
            // ============= zero this CTA's rows of h' (router, fused forward) ================
            if ((FUSED || p.zero_out != nullptr) && t_begin < t_end) {
                const long long row_lo = (long long)t_begin * kTileM;
                long long row_hi = (long long)t_end * kTileM;
                if (row_hi > p.n_rows) row_hi = p.n_rows;
                uint4* dst = reinterpret_cast<uint4*>(p.zero_out + row_lo * p.zero_cols);
                const long long nvec = (row_hi - row_lo) * p.zero_cols / 8;
                const uint4 z = make_uint4(0u, 0u, 0u, 0u);
                for (long long i = lane; i < nvec; i += 32) dst[i] = z;
            }
        } else if (gather && t_begin < t_end) {
            // ============= gather warp (experts, fused forward) ===============================
            // Row r of a tile is stacked row row0 + r = pair perm[row0 + r] = (n, j); its A row is
            // X[n, :], copied asynchronously (no registers) into the K-major 128-byte-swizzled
            // layout.  The gate of Eq. 1 multiplies the GEMM-1 accumulator instead of the row.
            // The warp runs ahead of the MMAs by as many tiles as there are A buffers.
            constexpr int CPR = C::K1 / 8;            // 16-byte chunks per row
            constexpr int RPI = 32 / CPR;             // rows covered by one warp-wide copy
            const int ch = lane % CPR, rsub = lane / CPR;
            int ge = 0, gm = 0;
            bool ok = true;
            // Blocks of 32 rows per gather warp: all four, or one each with four gather warps (warp 3 and
            // the three after the output warpgroup: one per sub-partition).
            constexpr int QPW = 4 / C::GATHER_WARPS;
            const int q0 = C::GATHER4 ? (warp == 3 ? 0 : warp - (C::OUT_WARP0 + 4) + 1) : 0;
            int nrow[QPW], nnext[QPW];                   // source rows of tile rows lane + 32 (q0 + q); pairs of the next tile
#pragma unroll
            for (int q = 0; q < QPW; ++q) nnext[q] = -1;
            // The first turn (t = t_begin - 1) only fetches the first tile's pair indices; a tile's indices
            // are fetched one tile ahead and left untouched until then, so that the load's latency is not
            // waited for.
#pragma unroll 1
            for (int t = t_begin - 1, ta = -1; t < t_end && ok; ++t, ++ta) {
#pragma unroll
                for (int q = 0; q < QPW; ++q) nrow[q] = nnext[q] < 0 ? -1 : pair_to_row(nnext[q], p.gather_magic, p.gather_shift);
                if (t + 1 < t_end) {
                    int row0, rows;
                    locate_tile(sh.tile_start, sh.offs, t + 1, ge, row0, rows, vs);
#pragma unroll
                    for (int q = 0; q < QPW; ++q) {
                        const int r = lane + 32 * (q0 + q);
                        nnext[q] = (r < rows) ? ld_index<SAME_LAUNCH>(p.perm + row0 + r) : -1;
                    }
                }
                if (ta < 0) continue;
                const int ab = ta % C::A_BUFS;
                ok = mbar_wait(bar(B::A_EMPTY + ab), ((uint32_t)(ta / C::A_BUFS) & 1u) ^ 1u, abort, kWaitLimitNs);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                const uint32_t dst0 = sA + ab * C::A_BYTES + (ch >> 3) * C::A_PANEL;
                const bool in_row = ch * 8 < p.row_elems;       // chunks past the row's real width are zero-filled
                auto copy_block = [&](int q, int nrow_q) {       // 32 rows of the tile
#pragma unroll 8
                    for (int i = 0; i < 32 / RPI; ++i) {
                        const int r32 = i * RPI + rsub;             // row within this block of 32
                        const int r = q * 32 + r32;
                        const int n = __shfl_sync(0xffffffffu, nrow_q, r32);
                        const bool real = n >= 0 && in_row;          // (rows past the tile's end are zero-filled too)
                        const bf16* src = p.gather_src + (real ? (size_t)n * p.row_elems + ch * 8 : 0);
                        cp_async_16(dst0 + (r >> 3) * 1024 + (r & 7) * 128 + (((ch & 7) ^ (r & 7)) << 4), src,
                                    real ? 16u : 0u);
                    }
                };
                // The four blocks: a rolled loop in the single-kernel forward, unrolled in the stand-alone
                // kernel (measured both ways in both: 472 -> 465 us there, 298 -> 327 us here on cfg2).  How
                // far to unroll is a trade: this warp shares its sub-partition with five busier ones and gets
                // an instruction in every ~8 cycles, so it needs independent work in flight (fully rolled, 32
                // dependent turns per tile made it the slowest stage: 465 -> 562 us), while fully unrolled its
                // ~2000 instructions per tile sweep the other warps' loops out of the instruction cache.
                if constexpr (QPW == 1) {
                    copy_block(q0, nrow[0]);
                } else if constexpr (FUSED) {
#pragma unroll 1
                    for (int q = 0; q < 4; ++q) copy_block(q, q == 0 ? nrow[0] : q == 1 ? nrow[1] : q == 2 ? nrow[2] : nrow[3]);
                } else {
#pragma unroll
                    for (int q = 0; q < 4; ++q) copy_block(q, nrow[q]);
                }
                {
                    int row0, rows;
                    locate_tile(sh.tile_start, sh.offs, t, gm, row0, rows, vs);
#pragma unroll
                    for (int q = 0; q < QPW; ++q) {
                        // rows past the tile's end take a neighbour's values: their A rows are zero and
                        // they are never stored
                        const int r = lane + 32 * (q0 + q), src = min(row0 + r, p.n_rows - 1);
                        cp_async_4(smem_u32(&sh.gate_s[ta % kMetaRing][r]), p.gate + src);
                        cp_async_4(smem_u32(&sh.pair_s[ta % kMetaRing][r]), p.perm + src);
                    }
                }
                cp_async_mbar_arrive_noinc(bar(B::A_FULL + ab));
            }
            cp_async_wait_all();
        }
    } else if (warp >= 4 && warp < C::OUT_WARP0) {
        // ================= activation warpgroups =============================================
        const int grp = (warp - 4) / C::GRP_WARPS;    // which chunks: g mod NGRP == grp
        const int w = ((warp - 4) >> 2) % C::GWG;     // warpgroup within the group = which part of the chunk's columns
        const int lg = warp & 3;                      // TMEM lane group this warp may access
        const uint32_t lane_base = tmem_base + ((uint32_t)(lg * 32) << 16);
        constexpr int WCOLS = C::HC / C::GWG;         // accumulator columns per thread and chunk
        bool ok = true;
        int e = 0;
        uint32_t g = 0;
        int prev_e = -1;
        uint32_t q_tile = 0, q_next = 0;              // bias ring: W1 load count of this tile's chunk 0 / after it
        for (int t = t_begin; t < t_end && ok; ++t) {
            int row0, rows;
            locate_tile(sh.tile_start, sh.offs, t, e, row0, rows, vs);
            if (!resident || e != prev_e) {           // this tile's weights (and biases) were loaded for it
                q_tile = q_next;
                q_next += nchunks;
            }
            prev_e = e;
            float gs = 1.0f;                          // Eq. 1's gate of this thread's row (fused forward; the
                                                      // staged call's rows arrive weighted), read per chunk
            for (int c = 0; c < nchunks && ok; ++c, ++g) {
                if (C::NGRP > 1 && (int)(g % C::NGRP) != grp) continue;               // the other group's chunk
                const uint32_t b = g % C::NBUF, n1 = g / C::NBUF;
                const uint32_t acc1 = lane_base + b * C::HC + w * WCOLS;               // my accumulator columns
                const uint32_t hdst = lane_base + C::H_COL0 + b * (C::HC / 2) + w * (WCOLS / 2);
                ok = mbar_wait(bar(B::ACC1_FULL + b), n1 & 1u, abort, kWaitLimitNs);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                // (the tile's A rows, and with them its ring entry, landed before GEMM-1 could run)
                if (gather) gs = sh.gate_s[(t - t_begin) % kMetaRing][lg * 32 + lane];
                tc_fence_after_sync();
                // this chunk's bias came into shared memory with its W1 (same barrier, own ring)
                const int bslot = (int)((q_tile + c) % kBiasRing);
                const uint8_t* sb1 = smem_raw + (smem_base - smem_u32(smem_raw)) + C::OFF_B1 + bslot * C::B1_BYTES + w * WCOLS * 2;
                if constexpr (C::PACKED_ACT) {
                    // Experts.  The whole accumulator chunk is brought into registers as packed bf16
                    // (SUB pieces at a time) and handed back at once, so that GEMM-1 of this group's
                    // next chunk runs under this chunk's activation.  Then piece by piece: the argument
                    // and tanh of piece pc, and behind them the tail and the store of piece pc - 1,
                    // whose tanh results have arrived by then.
                    __nv_bfloat162 z[C::NPIECE][C::PIECE / 2];
#pragma unroll
                    for (int s0 = 0; s0 < C::NPIECE; s0 += C::SUB) {
                        uint32_t v[C::SUB][C::PIECE];
#pragma unroll
                        for (int i = 0; i < C::SUB; ++i) tmem_ld_x16(acc1 + (s0 + i) * C::PIECE, v[i]);
                        tmem_ld_wait();
#pragma unroll
                        for (int i = 0; i < C::SUB; ++i)
                            convert_piece_bf16x2(v[i], gs, reinterpret_cast<const uint4*>(sb1 + (s0 + i) * C::PIECE * 2),
                                                 p.bias1 != nullptr, z[s0 + i]);      // (no shared-memory reads without a bias)
                    }
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar(B::ACC1_EMPTY + b));
                    __nv_bfloat162 th[2][C::PIECE / 2];
#pragma unroll
                    for (int pc = 0; pc <= C::NPIECE; ++pc) {
                        if (pc < C::NPIECE) activate_pre_bf16x2<C::ACT>(z[pc], th[pc & 1]);
                        if (pc == 0) {
                            // GEMM-2 of two chunks ago must be done with this hidden buffer
                            ok = mbar_wait(bar(B::H_EMPTY + b), (n1 & 1u) ^ 1u, abort, kWaitLimitNs);
                            ok = __all_sync(0xffffffffu, ok);
                            if (!ok) break;
                        } else {
                            uint32_t hi[C::PIECE / 2];
                            activate_post_bf16x2<C::ACT>(z[pc - 1], th[(pc - 1) & 1], hi);
                            tmem_st_x8(hdst + (pc - 1) * (C::PIECE / 2), hi);
                        }
                    }
                } else {
                    uint32_t v[2][C::PIECE];
                    tmem_ld_x16(acc1, v[0]);
#pragma unroll
                    for (int pc = 0; pc < C::NPIECE; ++pc) {
                        uint32_t* cur = v[pc & 1];
                        tmem_ld_wait();
                        if (pc + 1 < C::NPIECE) tmem_ld_x16(acc1 + (pc + 1) * C::PIECE, v[(pc + 1) & 1]);   // overlaps the math below
                        uint32_t hi[C::PIECE / 2], lo[C::PIECE / 2];
                        bias_relu_split_piece(cur, sh.bias1_f32 + c * C::HC + w * WCOLS + pc * C::PIECE, hi, lo, p.bias1 != nullptr);
                        tmem_st_x8(acc1 + pc * C::PIECE, hi);                    // over the piece just read
                        tmem_st_x8(acc1 + pc * C::PIECE + C::PIECE / 2, lo);
                    }
                }
                if (!ok) break;
                tmem_st_wait();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(B::H_FULL + b));
            }
        }
    } else if (warp >= C::OUT_WARP0 && warp < C::OUT_WARP0 + 4) {
        // ================= output warpgroup ==================================================
        const int lg = warp & 3;
        const int row = lg * 32 + lane;
        const uint32_t tmem_lane = tmem_base + ((uint32_t)(lg * 32) << 16);
        bool ok = true;
        int e = 0;
        // Fused forward: this thread's row of a tile is pair perm[row0 + row] = (n, j); its output is
        // added into row n of Y.
        for (int t = t_begin, ta = 0; t < t_end && ok; ++t, ++ta) {
            int row0, rows;
            locate_tile(sh.tile_start, sh.offs, t, e, row0, rows, vs);
            const int buf = ta % C::ACC2_BUFS;
            ok = mbar_wait(bar(B::ACC2_FULL + buf), (uint32_t)(ta / C::ACC2_BUFS) & 1u, abort, kWaitLimitNs);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after_sync();
            const int pair_cur = gather ? sh.pair_s[ta % kMetaRing][row] : 0;
            const uint32_t acc2 = tmem_lane + C::ACC2_COL0 + buf * C::N2;
            if constexpr (C::ROUTER) {
                constexpr int E = C::N2;
                uint32_t v[E];
#pragma unroll
                for (int q = 0; q < E / 16; ++q) tmem_ld_x16(acc2 + q * 16, v + q * 16);
                tmem_ld_wait();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(B::ACC2_EMPTY + buf));
                if (row >= rows) continue;
                float gl[E];
#pragma unroll
                for (int i = 0; i < E; i += 4) {
                    const float4 b = *reinterpret_cast<const float4*>(sh.bias2_f32 + i);   // same address for the whole warp
                    gl[i] = __uint_as_float(v[i]) + b.x;
                    gl[i + 1] = __uint_as_float(v[i + 1]) + b.y;
                    gl[i + 2] = __uint_as_float(v[i + 2]) + b.z;
                    gl[i + 3] = __uint_as_float(v[i + 3]) + b.w;
                }
                const int n = row0 + row;
                // top-k over the logits; ties go to the lower id
                float m;
                int sel[8];
                float gsel[8];
                if (FUSED || p.k <= 2) {
                    // one pass keeping the best two (strict comparisons in ascending id order give the
                    // same picks as repeated arg-max)
                    float b1 = gl[0], b2 = -INFINITY;
                    int i1 = 0, i2 = 0;
#pragma unroll
                    for (int i = 1; i < E; ++i) {
                        const float g = gl[i];
                        const bool gt1 = g > b1, gt2 = g > b2;
                        b2 = gt1 ? b1 : (gt2 ? g : b2);
                        i2 = gt1 ? i1 : (gt2 ? i : i2);
                        b1 = gt1 ? g : b1;
                        i1 = gt1 ? i : i1;
                    }
                    sel[0] = i1; gsel[0] = b1; sel[1] = i2; gsel[1] = b2;
                    m = b1;
                } else {
                    // repeated arg-max
                    unsigned long long taken = 0ull;
                    m = 0.0f;
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
                }
                const float sc = p.softmax_scale;
                float sum = 0.0f;
#pragma unroll
                for (int i = 0; i < E; ++i) sum += ex2_approx((gl[i] - m) * sc);
                const float inv = 1.0f / sum;
                for (int j = 0; j < p.k; ++j) {
                    p.topk_idx[(size_t)n * p.k + j] = sel[j];
                    p.topk_p[(size_t)n * p.k + j] = ex2_approx((gsel[j] - m) * sc) * inv;
                    atomicAdd(&sh.hist[sel[j]], 1);
                }
                if (!FUSED && p.probs) {
                    float4* dst = reinterpret_cast<float4*>(p.probs + (size_t)n * p.experts_real);
#pragma unroll
                    for (int i = 0; i < E; i += 4)
                        if (i < p.experts_real)                      // (the real count is a multiple of 8)
                            dst[i / 4] = make_float4(ex2_approx((gl[i] - m) * sc) * inv, ex2_approx((gl[i + 1] - m) * sc) * inv,
                                                     ex2_approx((gl[i + 2] - m) * sc) * inv, ex2_approx((gl[i + 3] - m) * sc) * inv);
                }
            } else {
                // OB output columns at a time: accumulator -> registers -> bias -> bf16 -> global
                // (16 columns per turn of a rolled loop, not 64 unrolled: the shorter body is worth more
                // than the saved accumulator-load waits -- the pass is sensitive to the size of its hot code,
                // see mbar_wait_poll: cfg2 forward 506 -> 472 us)
                constexpr int OB = 16;
                static_assert(C::N2 % OB == 0, "output width");
                const bool scatter = gather && (FUSED || p.scatter_out != nullptr);
                const bool live = row < rows;
                bf16* dst = nullptr;
                if (live) dst = scatter ? p.scatter_out + (size_t)pair_to_row(pair_cur, p.gather_magic, p.gather_shift) * C::N2
                                        : p.yperm + (size_t)(row0 + row) * C::N2;
#pragma unroll 1
                for (int cb = 0; cb < C::N2; cb += OB) {
                    uint32_t v[OB];
#pragma unroll
                    for (int q = 0; q < OB / 16; ++q) tmem_ld_x16(acc2 + cb + q * 16, v + q * 16);
                    tmem_ld_wait();
                    if (cb + OB >= C::N2) {
                        // the accumulator is in registers: GEMM-2 of a later tile may overwrite it
                        tc_fence_before_sync();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar(B::ACC2_EMPTY + buf));
                    }
                    if (!live) continue;
#pragma unroll
                    for (int q = 0; q < OB / 8; ++q) {
                        float bb[8];
                        if (p.bias2 && (e & vs) == 0) {
                            unpack16<bf16>(__ldg(reinterpret_cast<const uint4*>(p.bias2 + (size_t)(e >> vs) * C::N2 + cb + q * 8)), bb);
                        } else {
#pragma unroll
                            for (int i = 0; i < 8; ++i) bb[i] = 0.0f;
                        }
                        uint32_t o[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i)
                            o[i] = pack_bf16x2(fmaf(__uint_as_float(v[q * 8 + 2 * i]), kOutScale<C::ACT>, bb[2 * i]),
                                               fmaf(__uint_as_float(v[q * 8 + 2 * i + 1]), kOutScale<C::ACT>, bb[2 * i + 1]));
                        if (scatter) red_add_bf16x8(dst + cb + q * 8, o[0], o[1], o[2], o[3]);   // sum over the row's k experts
                        else *reinterpret_cast<uint4*>(dst + cb + q * 8) = make_uint4(o[0], o[1], o[2], o[3]);
                    }
                }
            }
        }
    }

    // ---- teardown -------------------------------------------------------------------------
    tc_fence_before_sync();
    __syncthreads();
    if (threadIdx.x == 0 && sh.abort_flag) atomicExch(p.status, (int)SLICEMOE_ERR_DEVICE_TIMEOUT);
    if constexpr (C::ROUTER) {
        // per-CTA histogram -> global counts (Section 3.2's per-expert counts)
        for (int i = threadIdx.x; i < p.experts_real; i += C::THREADS) {
            if (!FUSED && p.assigned && sh.hist[i]) atomicAdd(&p.assigned[i], sh.hist[i]);
            if (p.cta_hist) p.cta_hist[(size_t)blockIdx.x * p.experts_real + i] = sh.hist[i];
        }
    }
    tc_fence_before_sync();
    __syncthreads();          // nothing of this pass is in flight any more: barriers and TMEM may be reused
    tc_fence_after_sync();
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

// cudaFuncSetAttribute applies to the current device only: raise a kernel's dynamic shared-memory limit once
// per (kernel, device).  `done` is the kernel instantiation's own table (one bool per device).
constexpr int kAttrMaxDevices = 64;
template <class K>
int set_smem_limit_once(K kern, int bytes, bool (&done)[kAttrMaxDevices]) {
    int dev = -1;
    SLICEMOE_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kAttrMaxDevices) return SLICEMOE_ERR_NO_DEVICE;
    if (!done[dev]) {
        SLICEMOE_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
        done[dev] = true;
    }
    return SLICEMOE_OK;
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

template <class C> constexpr int kSmemLaunch = C::SMEM_ALLOC;

}  // namespace
}  // namespace slicemoe
