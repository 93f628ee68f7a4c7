// Shared declarations of the SliceMoE CUDA library (internal; the public ABI is include/slicemoe.h).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "slicemoe.h"

namespace slicemoe {

typedef __nv_bfloat16 bf16;

// Derived sizes of one layer call (paper notation; rows are slices, pairs are (row, j)).
struct Dims {
    int T, d, S, E, k, Hr, F;
    int ds;   // slice width d/S
    int N;    // rows  = T*S
    int R;    // pairs = N*k
    int dtype, act;
    int capacity;  // 0 = unlimited; clamped to R
    float inv_tau;        // 1 / softmax temperature
    float noise_sigma;    // 0 = no logit noise
    uint64_t noise_seed;
    int train_gates;                     // forward calls: Section 3.3's gates instead of the probabilities
    unsigned long long drop_threshold;   // an assignment is dropped iff its 32-bit draw < this (floor(rate 2^32))
    uint64_t drop_seed;
};

// Pairs handled by one dispatch chunk (one CTA of the histogram / scatter kernels).
constexpr int kDispatchChunk = 2048;
// Rows per CTA tile of the tensor-core kernels.
constexpr int kTileM = 128;

// Sub-buffers of the caller's workspace (byte offsets, each 256-byte aligned).
struct Workspace {
    size_t status;      // int32[256]: [0] device status word (the rest is spare, used by development builds)
    size_t topk_idx;    // int32[R]
    size_t topk_p;      // float[R]
    size_t assigned;    // int32[E]
    size_t kept;        // int32[E]
    size_t offsets;     // int32[E+1]
    size_t dest;        // int32[R]
    size_t perm;        // int32[R]
    size_t gate;        // float[R]   gate value of each stacked row (fused forward)
    size_t chunk_hist;  // int32[nchunks*E]
    size_t cta_hist;    // int32[256*E]  per-CTA expert counts of the tensor-core router (fused forward)
    size_t tiles;       // int32[4 + 2*max_tiles]  tile list of the grouped expert kernel
    size_t xperm;       // dtype[R*ds]
    size_t yperm;       // dtype[R*ds]
    size_t h_dev;       // dtype[T*d]  staging of slicemoe_forward_host
    size_t hout_dev;    // dtype[T*d]
    size_t total;
};

Workspace workspace_layout(const Dims& D);
inline int num_chunks(const Dims& D) { return (D.R + kDispatchChunk - 1) / kDispatchChunk; }
inline int max_tiles(const Dims& D) { return (D.R + kTileM - 1) / kTileM + D.E; }
inline size_t elem_bytes(const Dims& D) { return D.dtype == SLICEMOE_BF16 ? 2 : 4; }

// Checks a config and derives the sizes (SLICEMOE_OK or an error status).
int make_dims(const slicemoe_config* c, Dims& D);
// SLICEMOE_OK if the current device is an sm_100 part.
int check_device();
void count_launches(int n);
void note_cuda_error(cudaError_t e);

#define SLICEMOE_CUDA_TRY(expr)                          \
    do {                                                 \
        cudaError_t _e = (expr);                         \
        if (_e != cudaSuccess) {                         \
            ::slicemoe::note_cuda_error(_e);             \
            return SLICEMOE_ERR_CUDA;                    \
        }                                                \
    } while (0)

// Checks the launch that was just enqueued.
#define SLICEMOE_LAUNCH_CHECK(nlaunches)                 \
    do {                                                 \
        ::slicemoe::count_launches(nlaunches);           \
        SLICEMOE_CUDA_TRY(cudaGetLastError());           \
    } while (0)

// ---- per-stage launchers (each returns a slicemoe_status) ---------------------------------

// Router on CUDA cores, fp32 arithmetic in both storage types.
int launch_route_simt(const Dims& D, const slicemoe_weights& w, const void* h, int32_t* topk_idx,
                      float* topk_p, int32_t* assigned, float* probs_opt, cudaStream_t st);

// Stable counting sort of the pairs by expert + optional row gather.
// xperm may be NULL (no gather); gate_opt (float[R], gate of each stacked row) may be NULL.
int launch_dispatch(const Dims& D, const void* h, const int32_t* topk_idx, const float* topk_p,
                    int32_t* kept, int32_t* offsets, int32_t* dest, int32_t* perm, void* xperm,
                    float* gate_opt, int32_t* chunk_hist, cudaStream_t st);

// Grouped expert FFN on CUDA cores.
int launch_ffn_simt(const Dims& D, const slicemoe_weights& w, const void* xperm,
                    const int32_t* offsets, void* yperm, cudaStream_t st);

// Tensor-core (tcgen05 / TMEM / TMA) router and grouped expert FFN, bf16 storage only.
bool tc_route_supported(const Dims& D);
bool tc_ffn_supported(const Dims& D);
// assigned may be NULL (no global counts); cta_hist (int32[grid, E], see tc_route_grid) receives each
// CTA's own counts for the fused dispatch.
int launch_route_tc(const Dims& D, const slicemoe_weights& w, const void* h, int32_t* topk_idx,
                    float* topk_p, int32_t* assigned, float* probs_opt, int32_t* status, cudaStream_t st,
                    int32_t* cta_hist = nullptr, void* zero_out = nullptr);
// The router of slices of 96 / 128 / 192 / 256 elements (router hidden width 256, k <= 8) with Wr1 and Wr2 resident
// in shared memory; same outputs, grid and row partition as launch_route_tc without the probability matrix.
// grid_rows: launch at least that many CTAs, so that cta_hist has that many rows (the single-kernel forward's
// dispatch reads one row per CTA of ITS grid, the number of SMs).
bool wide_route_supported(const Dims& D);
int launch_route_wide(const Dims& D, const slicemoe_weights& w, const void* h, int32_t* topk_idx, float* topk_p,
                      int32_t* assigned, int32_t* status, cudaStream_t st, int32_t* cta_hist = nullptr,
                      void* zero_out = nullptr, int grid_rows = 0);
// Grid of the tensor-core router and the rows each of its CTAs routes (CTA c: rows [c*rows_per_cta, ...)).
void tc_route_grid(const Dims& D, int* grid, int* rows_per_cta);
// Fused dispatch after the tensor-core router: one kernel that turns the router's per-CTA counts into
// assigned / kept / offsets and ranks every pair (dest, perm, gate); no stacked-row copy.
int launch_dispatch_fused(const Dims& D, const int32_t* topk_idx, const float* topk_p, const int32_t* cta_hist,
                          int grid, int rows_per_cta, int32_t* assigned, int32_t* kept, int32_t* offsets,
                          int32_t* dest, int32_t* perm, float* gate, cudaStream_t st);
// zero_out (router): each CTA also zeroes its rows of that [N, ds] matrix.
// scatter_out (experts, with gather_h, k <= 2): expert outputs are added to row perm[r] / k of that
// [N, ds] matrix (zeroed before) instead of being stored to yperm, which makes the combine step part
// of the kernel; the sum of at most two bf16 values does not depend on the order of the additions.
// With gather_h != nullptr the rows are not read from xperm: row r of the stacked order is
// bf16(gate[r] * X[perm[r] / k, :]) gathered from h inside the kernel (fused forward).
int launch_ffn_tc(const Dims& D, const slicemoe_weights& w, const void* xperm, const int32_t* offsets,
                  void* yperm, int32_t* status, cudaStream_t st, const void* gather_h = nullptr,
                  const int32_t* perm = nullptr, const float* gate = nullptr, void* scatter_out = nullptr);

// The whole forward as one cooperative launch (router phase, dispatch phase, expert phase with grid
// barriers between them): bf16 shapes that both tensor-core kernels take, k <= 2.  The kernel clears
// the status word itself (no memset before it).  topk_idx/topk_p/dest/perm/gate/cta_hist as in the
// three-launch path; assigned/kept/offsets are written by CTA 0.
// router_done: an earlier launch on the stream (launch_route_wide with cta_hist and zero_out) has routed the batch
// over the same grid and row partition; the kernel starts at its dispatch phase.
// fused_forward_reset_sync: puts the device's grid-barrier words back to zero (after a launch whose
// bounded waits ran out).
bool fused_forward_supported(const Dims& D);
int launch_forward_fused(const Dims& D, const slicemoe_weights& w, const void* h, void* h_out, int32_t* topk_idx,
                         float* topk_p, int32_t* assigned, int32_t* kept, int32_t* offsets, int32_t* dest,
                         int32_t* perm, float* gate, int32_t* cta_hist, int32_t* status, bool clear_status,
                         cudaStream_t st, bool router_done = false);
int fused_forward_reset_sync(cudaStream_t st);
int fused_forward_grid();      // CTAs of the single kernel (one per SM)

// The same forward on the two-stream pipeline (pp_body.cuh): 64-wide slices, k <= 2, no capacity limit.
// one_launch: a single cooperative launch; otherwise one launch per phase with the stage events recorded.
// dest doubles as the router's scratch for the pairs' ranks inside their CTA; pair_gate is int2[R]
// (stacked row -> pair index and gate); the order of the stacked rows inside an expert is not the stable
// (n, j) order of slicemoe_dispatch.
bool pp_forward_supported(const Dims& D);
bool pp_route_supported(const Dims& D);
bool pp_ffn_supported(const Dims& D);
int launch_ffn_pp(const Dims& D, const slicemoe_weights& w, const void* xperm, const int32_t* offsets, void* yperm,
                  int32_t* status, cudaStream_t st);
int launch_route_pp(const Dims& D, const slicemoe_weights& w, const void* h, int32_t* topk_idx, float* topk_p,
                    int32_t* assigned, int32_t* status, cudaStream_t st);
int launch_forward_pp(const Dims& D, const slicemoe_weights& w, const void* h, void* h_out, int32_t* topk_idx,
                      float* topk_p, int32_t* assigned, int32_t* kept, int32_t* offsets, int32_t* dest, void* pair_gate,
                      int32_t* cta_hist, int32_t* status, bool clear_status, bool one_launch, void* const* events,
                      cudaStream_t st);
int pp_forward_reset_sync(cudaStream_t st);

// Decode-shaped forward (decode_forward.cu): 128-wide slices, F = 512, Hr = 256, at most 32 rows per SM, k <= 2, no
// capacity limit; one cooperative launch.  `lists` is scratch of at least E * N * 2 bytes.
bool decode_forward_supported(const Dims& D);
int launch_forward_decode(const Dims& D, const slicemoe_weights& w, const void* h, void* h_out, int32_t* topk_idx,
                          float* topk_p, int32_t* assigned, int32_t* kept, void* lists, int32_t* status,
                          bool clear_status, cudaStream_t st);
int decode_forward_reset_sync(cudaStream_t st);

// Section 3.3's gates in place of the top-k probabilities (gate_dropout.cu).
int launch_gate_dropout(const Dims& D, float* topk_p, uint64_t seed, unsigned long long threshold, cudaStream_t st);
int launch_combine(const Dims& D, const void* yperm, const int32_t* dest, void* h_out,
                   cudaStream_t st);

// out[t, c] = in[t, perm[c]] (inverse = false) or out[t, perm[c]] = in[t, c] (inverse = true).
int launch_permute_columns(const Dims& D, const void* in, void* out, const int32_t* perm, bool inverse,
                           cudaStream_t st);

// ---- storage-type helpers ---------------------------------------------------------------------

template <typename T> struct Vec;  // 16-byte vector of T
template <> struct Vec<float> { static constexpr int n = 4; };
template <> struct Vec<bf16> { static constexpr int n = 8; };

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(bf16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f32<bf16>(float v) { return __float2bfloat16_rn(v); }

// Unpacks one 16-byte vector into Vec<T>::n floats.
template <typename T> __device__ __forceinline__ void unpack16(const uint4& raw, float* out);
template <> __device__ __forceinline__ void unpack16<float>(const uint4& raw, float* out) {
    out[0] = __uint_as_float(raw.x); out[1] = __uint_as_float(raw.y);
    out[2] = __uint_as_float(raw.z); out[3] = __uint_as_float(raw.w);
}
template <> __device__ __forceinline__ void unpack16<bf16>(const uint4& raw, float* out) {
    const uint32_t u[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        out[2 * i] = __uint_as_float(u[i] << 16);
        out[2 * i + 1] = __uint_as_float(u[i] & 0xFFFF0000u);
    }
}
template <typename T> __device__ __forceinline__ uint4 pack16(const float* in);
template <> __device__ __forceinline__ uint4 pack16<float>(const float* in) {
    return make_uint4(__float_as_uint(in[0]), __float_as_uint(in[1]), __float_as_uint(in[2]),
                      __float_as_uint(in[3]));
}
template <> __device__ __forceinline__ uint4 pack16<bf16>(const float* in) {
    uint32_t u[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        __nv_bfloat162 v = __floats2bfloat162_rn(in[2 * i], in[2 * i + 1]);
        u[i] = *reinterpret_cast<uint32_t*>(&v);
    }
    return make_uint4(u[0], u[1], u[2], u[3]);
}

// GELU in its tanh form, fp32.
__device__ __forceinline__ float gelu_tanh_f32(float z) {
    const float c = 0.7978845608028654f;
    return 0.5f * z * (1.0f + tanhf(c * (z + 0.044715f * z * z * z)));
}
__device__ __forceinline__ float apply_act(float z, int act) {
    return act == SLICEMOE_ACT_RELU ? fmaxf(z, 0.0f) : gelu_tanh_f32(z);
}

}  // namespace slicemoe
