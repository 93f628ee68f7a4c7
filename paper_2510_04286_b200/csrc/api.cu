// C ABI of the SliceMoE layer forward: argument checking, workspace layout and the sequencing of
// the stage kernels on the caller's stream.  No step of the layer is computed here.
#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstring>

#include <cstdlib>
#include <mutex>

#include "common.cuh"

namespace slicemoe {

static std::atomic<long long> g_launches{0};
static thread_local char g_cuda_error[256] = "";

void count_launches(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }
void note_cuda_error(cudaError_t e) {
    std::snprintf(g_cuda_error, sizeof(g_cuda_error), "%s: %s", cudaGetErrorName(e), cudaGetErrorString(e));
    (void)cudaGetLastError();  // clear the sticky-less error state
}

static size_t align_up(size_t x, size_t a = 256) { return (x + a - 1) / a * a; }

Workspace workspace_layout(const Dims& D) {
    Workspace W;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t at = off; off = align_up(off + (bytes ? bytes : 1)); return at; };
    const size_t R = (size_t)D.R, E = (size_t)D.E, b = elem_bytes(D);
    W.status = take(sizeof(int32_t) * 256);
    W.topk_idx = take(sizeof(int32_t) * R);
    W.topk_p = take(sizeof(float) * R);
    W.assigned = take(sizeof(int32_t) * E);
    W.kept = take(sizeof(int32_t) * E);
    W.offsets = take(sizeof(int32_t) * (E + 1));
    W.dest = take(sizeof(int32_t) * R);
    W.perm = take(sizeof(int32_t) * R);
    W.gate = take(sizeof(float) * R);
    W.chunk_hist = take(sizeof(int32_t) * (size_t)num_chunks(D) * E);
    W.cta_hist = take(sizeof(int32_t) * 256 * E);
    W.tiles = take(sizeof(int32_t) * (4 + 2 * (size_t)max_tiles(D)));
    W.xperm = take(b * R * D.ds);
    W.yperm = take(b * R * D.ds);
    W.h_dev = take(b * (size_t)D.T * D.d);
    W.hout_dev = take(b * (size_t)D.T * D.d);
    W.total = off;
    return W;
}

int make_dims(const slicemoe_config* c, Dims& D) {
    if (!c) return SLICEMOE_ERR_NULL;
    if (c->T < 0 || c->d < 1 || c->S < 1 || c->E < 1 || c->k < 1 || c->Hr < 1 || c->F < 1 || c->capacity < 0)
        return SLICEMOE_ERR_SHAPE;
    if (c->d % c->S != 0 || c->k > c->E) return SLICEMOE_ERR_SHAPE;
    if (c->dtype != SLICEMOE_BF16 && c->dtype != SLICEMOE_F32) return SLICEMOE_ERR_UNSUPPORTED;
    if (c->act != SLICEMOE_ACT_RELU && c->act != SLICEMOE_ACT_GELU_TANH) return SLICEMOE_ERR_UNSUPPORTED;
    const long long N = (long long)c->T * c->S, R = N * c->k;
    const long long lim = 0x7fffffffLL;
    if (R >= lim || (long long)c->T * c->d >= lim) return SLICEMOE_ERR_SHAPE;
    // (row and pair counts are 32-bit; the weight tensors are indexed with 64-bit element offsets, so a
    // token-level layer with E F d past 2^31 elements per tensor is fine; a tensor map's row count E F is not)
    if ((long long)c->E * c->F >= lim) return SLICEMOE_ERR_SHAPE;
    const int V = c->dtype == SLICEMOE_BF16 ? 8 : 4;
    const int ds = c->d / c->S;
    if (ds % V || c->Hr % V || c->F % V) return SLICEMOE_ERR_UNSUPPORTED;
    if (c->k > 8 || c->E > 256) return SLICEMOE_ERR_UNSUPPORTED;
    if (!(c->temperature >= 0.0f) || !(c->noise_sigma >= 0.0f) || std::isinf(c->temperature) ||
        std::isinf(c->noise_sigma))
        return SLICEMOE_ERR_SHAPE;
    if (c->train_gates != 0 && c->train_gates != 1) return SLICEMOE_ERR_SHAPE;
    if (c->train_gates && (!(c->dropout_rate >= 0.0f) || c->dropout_rate > 1.0f)) return SLICEMOE_ERR_SHAPE;
    D.train_gates = c->train_gates;
    D.drop_threshold = c->train_gates ? (unsigned long long)((double)c->dropout_rate * 4294967296.0) : 0ull;   // 2^32 when rate = 1
    D.drop_seed = c->dropout_seed;
    D.inv_tau = c->temperature > 0.0f ? 1.0f / c->temperature : 1.0f;
    D.noise_sigma = c->noise_sigma;
    D.noise_seed = c->noise_seed;
    D.T = c->T; D.d = c->d; D.S = c->S; D.E = c->E; D.k = c->k; D.Hr = c->Hr; D.F = c->F;
    D.ds = ds; D.N = (int)N; D.R = (int)R; D.dtype = c->dtype; D.act = c->act;
    D.capacity = (int)(c->capacity > R ? R : c->capacity);
    if (c->capacity > 0 && D.capacity == 0) D.capacity = 1;  // R == 0: keep "limited" semantics harmless
    return SLICEMOE_OK;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static int check_weights(const slicemoe_weights* w, bool router, bool experts) {
    if (!w) return SLICEMOE_ERR_NULL;
    if (router) {
        if (!w->Wr1 || !w->Wr2) return SLICEMOE_ERR_NULL;
        if (!aligned16(w->Wr1) || !aligned16(w->Wr2) || !aligned16(w->br1) || !aligned16(w->br2))
            return SLICEMOE_ERR_ALIGN;
    }
    if (experts) {
        if (!w->W1 || !w->W2) return SLICEMOE_ERR_NULL;
        if (!aligned16(w->W1) || !aligned16(w->W2) || !aligned16(w->b1) || !aligned16(w->b2))
            return SLICEMOE_ERR_ALIGN;
    }
    return SLICEMOE_OK;
}

int check_device() {
    static std::atomic<int> state{0};  // 0 unknown, 1 ok, 2 bad
    int s = state.load();
    if (s == 0) {
        int dev = 0, major = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
            (void)cudaGetLastError();
            s = 2;
        } else {
            s = (major == 10) ? 1 : 2;
        }
        state.store(s);
    }
    return s == 1 ? SLICEMOE_OK : SLICEMOE_ERR_NO_DEVICE;
}

static int check_ws(const Dims& D, const void* ws, size_t ws_bytes, Workspace& W) {
    W = workspace_layout(D);
    if (!ws || ws_bytes < W.total) return SLICEMOE_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(ws) & 255u) return SLICEMOE_ERR_ALIGN;
    return SLICEMOE_OK;
}

template <typename U> static U* at(void* ws, size_t off) {
    return reinterpret_cast<U*>(static_cast<char*>(ws) + off);
}

// Clears the device status word that kernels with bounded waits report into.
static int reset_status(void* ws, const Workspace& W, cudaStream_t st) {
    SLICEMOE_CUDA_TRY(cudaMemsetAsync(at<char>(ws, W.status), 0, sizeof(int32_t) * 64, st));
    return SLICEMOE_OK;
}

// The tensor-core kernels take bf16 shapes inside their tile set; everything else (fp32 storage,
// other widths) runs on the CUDA-core kernels.  Both are this library's own kernels.
static int route_any(const Dims& D, const slicemoe_weights& w, const void* h, int32_t* idx, float* p,
                     int32_t* assigned, float* probs, int32_t* status, cudaStream_t st) {
    // (64-wide slices without the full probability matrix: the whole-tile pipeline's router)
    if (!probs && pp_route_supported(D)) return launch_route_pp(D, w, h, idx, p, assigned, status, st);
    // (wide slices, likewise: the router that keeps both weight matrices in shared memory)
    if (!probs && wide_route_supported(D)) return launch_route_wide(D, w, h, idx, p, assigned, status, st);
    if (tc_route_supported(D)) return launch_route_tc(D, w, h, idx, p, assigned, probs, status, st);
    return launch_route_simt(D, w, h, idx, p, assigned, probs, st);
}

static int ffn_any(const Dims& D, const slicemoe_weights& w, const void* xperm, const int32_t* offsets,
                   void* yperm, int32_t* status, cudaStream_t st) {
    // (64-wide slices: the whole-tile pipeline's expert pass on the stacked rows)
    if (pp_ffn_supported(D)) return launch_ffn_pp(D, w, xperm, offsets, yperm, status, st);
    if (tc_ffn_supported(D)) return launch_ffn_tc(D, w, xperm, offsets, yperm, status, st);
    return launch_ffn_simt(D, w, xperm, offsets, yperm, st);
}

static int forward_impl(const Dims& D, const slicemoe_weights& w, const void* h, void* h_out,
                        int32_t* assigned_opt, int32_t* kept_opt, int32_t* idx_opt, float* p_opt,
                        void* ws, const Workspace& W, cudaStream_t st, void* const* events,
                        bool clear_status = true) {
    int32_t* idx = idx_opt ? idx_opt : at<int32_t>(ws, W.topk_idx);
    float* p = p_opt ? p_opt : at<float>(ws, W.topk_p);
    int32_t* assigned = assigned_opt ? assigned_opt : at<int32_t>(ws, W.assigned);
    int32_t* kept = kept_opt ? kept_opt : at<int32_t>(ws, W.kept);
    int32_t* offsets = at<int32_t>(ws, W.offsets);
    int32_t* dest = at<int32_t>(ws, W.dest);
    int32_t* perm = at<int32_t>(ws, W.perm);
    void* xperm = at<char>(ws, W.xperm);
    void* yperm = at<char>(ws, W.yperm);
    auto mark = [&](int i) -> int {
        if (events) SLICEMOE_CUDA_TRY(cudaEventRecord(static_cast<cudaEvent_t>(events[i]), st));
        return SLICEMOE_OK;
    };
    int rc;
    // 64-wide slices without a capacity limit: the two-stream pipeline, as one launch or one per phase
    if (pp_forward_supported(D)) {
        if (events && clear_status && (rc = reset_status(ws, W, st))) return rc;
        return launch_forward_pp(D, w, h, h_out, idx, p, assigned, kept, offsets, dest, xperm, at<int32_t>(ws, W.cta_hist),
                                 at<int32_t>(ws, W.status), clear_status, /*one_launch=*/!events, events, st);
    }
    // decode-shaped batches: one launch that streams each expert's weights once
    // (train mode: the other one-launch kernels have no gate step; the stage-by-stage forms below do)
    if (!events && !D.train_gates && decode_forward_supported(D))
        return launch_forward_decode(D, w, h, h_out, idx, p, assigned, kept, xperm, at<int32_t>(ws, W.status), clear_status, st);
    const bool one_launch = !events && !D.train_gates && fused_forward_supported(D);
    // The router with resident weights is a launch of its own (its weights leave no shared memory for the other
    // phases' state) and the single kernel then takes over at the dispatch.  Rows of 192 / 256: 15 % faster than
    // the single kernel alone.  Rows of 96 / 128: the shorter router (31 -> 23 us on 131 072 rows of 96) and the
    // second launch cancel, so the forward stays one launch there and only the stage-by-stage forms use it.
    const bool wide = wide_route_supported(D) && (D.ds > 128 || !one_launch);
    // (the single kernel clears the status word itself; a later chunk of one host-buffer call keeps
    // what an earlier chunk reported)
    if ((!one_launch || wide) && clear_status && (rc = reset_status(ws, W, st))) return rc;
    if ((rc = mark(0))) return rc;
    // With both tensor-core kernels available the stacked rows are never materialised: the router
    // leaves its per-CTA expert counts, one dispatch kernel ranks the pairs (dest, perm, gate) and
    // the expert kernel gathers its rows from h.
    const bool fused = tc_route_supported(D) && tc_ffn_supported(D) && D.N > 0;
    float* gate = at<float>(ws, W.gate);
    // One cooperative launch does all of it; the stage-timed call keeps the three launches so that
    // the stages stay separable.
    if (one_launch) {
        if (wide && (rc = launch_route_wide(D, w, h, idx, p, nullptr, at<int32_t>(ws, W.status), st,
                                            at<int32_t>(ws, W.cta_hist), h_out, fused_forward_grid()))) return rc;
        return launch_forward_fused(D, w, h, h_out, idx, p, assigned, kept, offsets, dest, perm, gate,
                                    at<int32_t>(ws, W.cta_hist), at<int32_t>(ws, W.status), clear_status && !wide, st,
                                    /*router_done=*/wide);
    }
    if (fused) {
        int grid = 0, rows_per_cta = 0;
        tc_route_grid(D, &grid, &rows_per_cta);
        int32_t* cta_hist = at<int32_t>(ws, W.cta_hist);
        // k <= 2: the experts add their rows straight into h' (zeroed by the router), so there is no
        // stacked output and no combine kernel; the two-term bf16 sum is order-independent.
        const bool scatter = D.k <= 2;
        if (wide) {
            if ((rc = launch_route_wide(D, w, h, idx, p, nullptr, at<int32_t>(ws, W.status), st, cta_hist,
                                        scatter ? h_out : nullptr))) return rc;
        } else if ((rc = launch_route_tc(D, w, h, idx, p, nullptr, nullptr, at<int32_t>(ws, W.status), st, cta_hist,
                                         scatter ? h_out : nullptr))) return rc;
        if ((rc = mark(1))) return rc;
        if (D.train_gates && (rc = launch_gate_dropout(D, p, D.drop_seed, D.drop_threshold, st))) return rc;
        if ((rc = launch_dispatch_fused(D, idx, p, cta_hist, grid, rows_per_cta, assigned, kept, offsets, dest, perm,
                                        gate, st))) return rc;
        if ((rc = mark(2))) return rc;
        if ((rc = launch_ffn_tc(D, w, nullptr, offsets, yperm, at<int32_t>(ws, W.status), st, h, perm, gate,
                                scatter ? h_out : nullptr))) return rc;
        if (scatter) {
            if ((rc = mark(3))) return rc;
            return mark(4);
        }
    } else {
        if ((rc = route_any(D, w, h, idx, p, assigned, nullptr, at<int32_t>(ws, W.status), st))) return rc;
        if ((rc = mark(1))) return rc;
        if (D.train_gates && (rc = launch_gate_dropout(D, p, D.drop_seed, D.drop_threshold, st))) return rc;
        const bool gather = tc_ffn_supported(D);
        if ((rc = launch_dispatch(D, h, idx, p, kept, offsets, dest, perm, gather ? nullptr : xperm,
                                  gather ? gate : nullptr, at<int32_t>(ws, W.chunk_hist), st))) return rc;
        if ((rc = mark(2))) return rc;
        if (gather) {
            if ((rc = launch_ffn_tc(D, w, nullptr, offsets, yperm, at<int32_t>(ws, W.status), st, h, perm, gate))) return rc;
        } else {
            if ((rc = ffn_any(D, w, xperm, offsets, yperm, at<int32_t>(ws, W.status), st))) return rc;
        }
    }
    if ((rc = mark(3))) return rc;
    if ((rc = launch_combine(D, yperm, dest, h_out, st))) return rc;
    return mark(4);
}

static bool overlaps(const void* a, const void* b, size_t bytes) {
    const uintptr_t x = reinterpret_cast<uintptr_t>(a), y = reinterpret_cast<uintptr_t>(b);
    return x < y + bytes && y < x + bytes;
}

}  // namespace slicemoe

using namespace slicemoe;

extern "C" {

int slicemoe_workspace_bytes(const slicemoe_config* cfg, size_t* bytes) {
    if (!bytes) return SLICEMOE_ERR_NULL;
    Dims D;
    int rc = make_dims(cfg, D);
    if (rc) return rc;
    *bytes = workspace_layout(D).total;
    return SLICEMOE_OK;
}

int slicemoe_route(const slicemoe_config* cfg, const slicemoe_weights* w, const void* h,
                   int32_t* topk_idx, float* topk_p, int32_t* assigned, float* probs_opt, void* ws,
                   size_t ws_bytes, void* stream) {
    Dims D;
    int rc = make_dims(cfg, D);
    if (rc) return rc;
    if ((rc = check_weights(w, true, false))) return rc;
    if (!h || !topk_idx || !topk_p || !assigned) return SLICEMOE_ERR_NULL;
    if (!aligned16(h) || !aligned16(topk_idx) || !aligned16(topk_p) || !aligned16(probs_opt))
        return SLICEMOE_ERR_ALIGN;
    Workspace W;
    if ((rc = check_ws(D, ws, ws_bytes, W))) return rc;
    if ((rc = check_device())) return rc;
    if ((rc = reset_status(ws, W, static_cast<cudaStream_t>(stream)))) return rc;
    return route_any(D, *w, h, topk_idx, topk_p, assigned, probs_opt, at<int32_t>(ws, W.status),
                     static_cast<cudaStream_t>(stream));
}

int slicemoe_dispatch(const slicemoe_config* cfg, const void* h, const int32_t* topk_idx,
                      const float* topk_p, int32_t* kept, int32_t* offsets, int32_t* dest,
                      int32_t* perm, void* xperm, void* ws, size_t ws_bytes, void* stream) {
    Dims D;
    int rc = make_dims(cfg, D);
    if (rc) return rc;
    if (!topk_idx || !topk_p || !kept || !offsets || !dest || !perm) return SLICEMOE_ERR_NULL;
    if (xperm && !h) return SLICEMOE_ERR_NULL;
    if (!aligned16(h) || !aligned16(xperm)) return SLICEMOE_ERR_ALIGN;
    Workspace W;
    if ((rc = check_ws(D, ws, ws_bytes, W))) return rc;
    if ((rc = check_device())) return rc;
    if ((rc = reset_status(ws, W, static_cast<cudaStream_t>(stream)))) return rc;
    return launch_dispatch(D, h, topk_idx, topk_p, kept, offsets, dest, perm, xperm, nullptr,
                           at<int32_t>(ws, W.chunk_hist), static_cast<cudaStream_t>(stream));
}

int slicemoe_expert_ffn(const slicemoe_config* cfg, const slicemoe_weights* w, const void* xperm,
                        const int32_t* offsets, void* yperm, void* ws, size_t ws_bytes, void* stream) {
    Dims D;
    int rc = make_dims(cfg, D);
    if (rc) return rc;
    if ((rc = check_weights(w, false, true))) return rc;
    if (!xperm || !offsets || !yperm) return SLICEMOE_ERR_NULL;
    if (!aligned16(xperm) || !aligned16(yperm)) return SLICEMOE_ERR_ALIGN;
    Workspace W;
    if ((rc = check_ws(D, ws, ws_bytes, W))) return rc;
    if ((rc = check_device())) return rc;
    if ((rc = reset_status(ws, W, static_cast<cudaStream_t>(stream)))) return rc;
    return ffn_any(D, *w, xperm, offsets, yperm, at<int32_t>(ws, W.status), static_cast<cudaStream_t>(stream));
}

int slicemoe_combine(const slicemoe_config* cfg, const void* yperm, const int32_t* dest, void* h_out,
                     void* stream) {
    Dims D;
    int rc = make_dims(cfg, D);
    if (rc) return rc;
    if (!yperm || !dest || !h_out) return SLICEMOE_ERR_NULL;
    if (!aligned16(yperm) || !aligned16(h_out)) return SLICEMOE_ERR_ALIGN;
    if ((rc = check_device())) return rc;
    return launch_combine(D, yperm, dest, h_out, static_cast<cudaStream_t>(stream));
}

static int forward_checked(const slicemoe_config* cfg, const slicemoe_weights* w, const void* h,
                           void* h_out, int32_t* assigned_opt, int32_t* kept_opt, int32_t* topk_idx_opt,
                           float* topk_p_opt, void* ws, size_t ws_bytes, void* stream,
                           void* const* events) {
    Dims D;
    int rc = make_dims(cfg, D);
    if (rc) return rc;
    if ((rc = check_weights(w, true, true))) return rc;
    if (D.T > 0 && (!h || !h_out)) return SLICEMOE_ERR_NULL;
    if (!aligned16(h) || !aligned16(h_out) || !aligned16(topk_idx_opt) || !aligned16(topk_p_opt))
        return SLICEMOE_ERR_ALIGN;
    if (D.T > 0 && overlaps(h, h_out, elem_bytes(D) * (size_t)D.T * D.d)) return SLICEMOE_ERR_ALIAS;
    Workspace W;
    if ((rc = check_ws(D, ws, ws_bytes, W))) return rc;
    if ((rc = check_device())) return rc;
    return forward_impl(D, *w, h, h_out, assigned_opt, kept_opt, topk_idx_opt, topk_p_opt, ws, W,
                        static_cast<cudaStream_t>(stream), events);
}

int slicemoe_forward(const slicemoe_config* cfg, const slicemoe_weights* w, const void* h, void* h_out,
                     int32_t* assigned_opt, int32_t* kept_opt, int32_t* topk_idx_opt, float* topk_p_opt,
                     void* ws, size_t ws_bytes, void* stream) {
    return forward_checked(cfg, w, h, h_out, assigned_opt, kept_opt, topk_idx_opt, topk_p_opt, ws,
                           ws_bytes, stream, nullptr);
}

int slicemoe_forward_profiled(const slicemoe_config* cfg, const slicemoe_weights* w, const void* h,
                              void* h_out, int32_t* assigned_opt, int32_t* kept_opt,
                              int32_t* topk_idx_opt, float* topk_p_opt, void* ws, size_t ws_bytes,
                              void* stream, void* const* events) {
    if (!events) return SLICEMOE_ERR_NULL;
    for (int i = 0; i < SLICEMOE_N_STAGE_EVENTS; ++i)
        if (!events[i]) return SLICEMOE_ERR_NULL;
    return forward_checked(cfg, w, h, h_out, assigned_opt, kept_opt, topk_idx_opt, topk_p_opt, ws,
                           ws_bytes, stream, events);
}

// ---- host-buffer forward ------------------------------------------------------------------------
// The copies dominate this call (PCIe), and the link carries both directions at once: the batch is
// cut into chunks of tokens and chunk j's copy in, forward and copy out run on three streams (the
// caller's for the kernels, two of the library's for the copies), so that the copy out of chunk j
// overlaps the copy in of chunk j + 1.  Only without a capacity limit (with one, which pair is
// dropped depends on the whole batch's order).
namespace slicemoe {
namespace {

constexpr int kPipeChunks = 4;
constexpr int kPipeMinTokensPerChunk = 512;
constexpr double kPipeEdgeShare = 0.5;        // first / last chunk relative to an inner chunk
constexpr int kPipeMaxDevices = 64;

struct HostPipe {
    bool ready = false;
    cudaStream_t s_in = nullptr, s_out = nullptr;
    cudaEvent_t begin = nullptr, done = nullptr, in[kPipeChunks] = {}, fwd[kPipeChunks] = {};
};
HostPipe g_pipe[kPipeMaxDevices];
std::mutex g_pipe_mutex;     // held while a call enqueues: calls share the two copy streams and the events

int host_pipe(HostPipe** out) {
    int dev = -1;
    SLICEMOE_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kPipeMaxDevices) return SLICEMOE_ERR_NO_DEVICE;
    HostPipe& p = g_pipe[dev];
    if (!p.ready) {
        SLICEMOE_CUDA_TRY(cudaStreamCreateWithFlags(&p.s_in, cudaStreamNonBlocking));
        SLICEMOE_CUDA_TRY(cudaStreamCreateWithFlags(&p.s_out, cudaStreamNonBlocking));
        SLICEMOE_CUDA_TRY(cudaEventCreateWithFlags(&p.begin, cudaEventDisableTiming));
        SLICEMOE_CUDA_TRY(cudaEventCreateWithFlags(&p.done, cudaEventDisableTiming));
        for (int i = 0; i < kPipeChunks; ++i) {
            SLICEMOE_CUDA_TRY(cudaEventCreateWithFlags(&p.in[i], cudaEventDisableTiming));
            SLICEMOE_CUDA_TRY(cudaEventCreateWithFlags(&p.fwd[i], cudaEventDisableTiming));
        }
        p.ready = true;
    }
    *out = &p;
    return SLICEMOE_OK;
}

__global__ void add_counts_kernel(const int32_t* __restrict__ a, const int32_t* __restrict__ k, int32_t* A, int32_t* K,
                                  int E) {
    const int e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e < E) {
        if (A) A[e] += a[e];
        if (K) K[e] += k[e];
    }
}

}  // namespace
}  // namespace slicemoe

int slicemoe_forward_host(const slicemoe_config* cfg, const slicemoe_weights* w, const void* h_host,
                          void* h_out_host, int32_t* assigned_opt, int32_t* kept_opt, void* ws,
                          size_t ws_bytes, void* stream) {
    Dims D;
    int rc = make_dims(cfg, D);
    if (rc) return rc;
    if ((rc = check_weights(w, true, true))) return rc;
    if (!h_host || !h_out_host) return SLICEMOE_ERR_NULL;
    Workspace W;
    if ((rc = check_ws(D, ws, ws_bytes, W))) return rc;
    if ((rc = check_device())) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t row_bytes = elem_bytes(D) * (size_t)D.d;
    const size_t bytes = row_bytes * (size_t)D.T;
    char* h_dev = at<char>(ws, W.h_dev);
    char* hout_dev = at<char>(ws, W.hout_dev);

    // (not with logit noise either: its draws are keyed by the row's index in the whole batch, and a chunk's
    // router counts rows from the chunk's start)
    // (logit noise and dropout draws are counted by global row numbers: such batches are not cut)
    const bool pipelined = D.capacity == 0 && D.noise_sigma == 0.0f && !D.train_gates && D.T >= kPipeChunks * kPipeMinTokensPerChunk;
    if (!pipelined) {
        if (bytes) SLICEMOE_CUDA_TRY(cudaMemcpyAsync(h_dev, h_host, bytes, cudaMemcpyHostToDevice, st));
        if ((rc = forward_impl(D, *w, h_dev, hout_dev, assigned_opt, kept_opt, nullptr, nullptr, ws, W, st,
                               nullptr)))
            return rc;
        if (bytes) SLICEMOE_CUDA_TRY(cudaMemcpyAsync(h_out_host, hout_dev, bytes, cudaMemcpyDeviceToHost, st));
        return SLICEMOE_OK;
    }

    std::lock_guard<std::mutex> lock(g_pipe_mutex);
    HostPipe* pipe = nullptr;
    if ((rc = host_pipe(&pipe))) return rc;
    // everything already queued on the caller's stream (an earlier call's use of the staging
    // buffers among it) comes first
    SLICEMOE_CUDA_TRY(cudaEventRecord(pipe->begin, st));
    SLICEMOE_CUDA_TRY(cudaStreamWaitEvent(pipe->s_in, pipe->begin, 0));
    SLICEMOE_CUDA_TRY(cudaStreamWaitEvent(pipe->s_out, pipe->begin, 0));
    if (assigned_opt) SLICEMOE_CUDA_TRY(cudaMemsetAsync(assigned_opt, 0, sizeof(int32_t) * D.E, st));
    if (kept_opt) SLICEMOE_CUDA_TRY(cudaMemsetAsync(kept_opt, 0, sizeof(int32_t) * D.E, st));
    const bool counts = assigned_opt || kept_opt;
    // Chunk boundaries in tokens.  The first and the last chunk are short: nothing overlaps the first
    // copy in or the last copy out.
    int bounds[kPipeChunks + 1];
    int nchunks_host = kPipeChunks;
    const double edge = kPipeEdgeShare;
    {
        // edge chunks get `edge` times the share of an inner chunk
        const double inner = 1.0 / (nchunks_host - 2 + 2 * edge);
        double acc = 0.0;
        bounds[0] = 0;
        for (int i = 0; i < nchunks_host; ++i) {
            acc += (nchunks_host < 3 || (i > 0 && i < nchunks_host - 1)) ? (nchunks_host < 3 ? 1.0 / nchunks_host : inner) : edge * inner;
            int b = (int)(acc * D.T + 0.5);
            if (b < bounds[i]) b = bounds[i];
            if (b > D.T) b = D.T;
            bounds[i + 1] = b;
        }
        bounds[nchunks_host] = D.T;
    }
    for (int j = 0; j < nchunks_host; ++j) {
        const int t0 = bounds[j], tc = bounds[j + 1] - bounds[j];
        if (tc <= 0) continue;
        const size_t off = row_bytes * (size_t)t0, cb = row_bytes * (size_t)tc;
        SLICEMOE_CUDA_TRY(cudaMemcpyAsync(h_dev + off, static_cast<const char*>(h_host) + off, cb,
                                          cudaMemcpyHostToDevice, pipe->s_in));
        SLICEMOE_CUDA_TRY(cudaEventRecord(pipe->in[j], pipe->s_in));
        SLICEMOE_CUDA_TRY(cudaStreamWaitEvent(st, pipe->in[j], 0));
        slicemoe_config cc = *cfg;
        cc.T = tc;
        Dims Dc;
        if ((rc = make_dims(&cc, Dc))) return rc;
        // the chunk's counts go to the workspace's own arrays and are added up below
        if ((rc = forward_impl(Dc, *w, h_dev + off, hout_dev + off, nullptr, nullptr, nullptr, nullptr, ws, W, st,
                               nullptr, /*clear_status=*/j == 0)))
            return rc;
        if (counts) {
            add_counts_kernel<<<(D.E + 127) / 128, 128, 0, st>>>(at<int32_t>(ws, W.assigned), at<int32_t>(ws, W.kept),
                                                                assigned_opt, kept_opt, D.E);
            SLICEMOE_LAUNCH_CHECK(1);
        }
        SLICEMOE_CUDA_TRY(cudaEventRecord(pipe->fwd[j], st));
        SLICEMOE_CUDA_TRY(cudaStreamWaitEvent(pipe->s_out, pipe->fwd[j], 0));
        SLICEMOE_CUDA_TRY(cudaMemcpyAsync(static_cast<char*>(h_out_host) + off, hout_dev + off, cb,
                                          cudaMemcpyDeviceToHost, pipe->s_out));
    }
    // the caller's stream is done when the last copy out is
    SLICEMOE_CUDA_TRY(cudaEventRecord(pipe->done, pipe->s_out));
    SLICEMOE_CUDA_TRY(cudaStreamWaitEvent(st, pipe->done, 0));
    return SLICEMOE_OK;
}

int slicemoe_event_create(void** event) {
    if (!event) return SLICEMOE_ERR_NULL;
    cudaEvent_t ev;
    SLICEMOE_CUDA_TRY(cudaEventCreate(&ev));
    *event = ev;
    return SLICEMOE_OK;
}

int slicemoe_event_destroy(void* event) {
    if (!event) return SLICEMOE_ERR_NULL;
    SLICEMOE_CUDA_TRY(cudaEventDestroy(static_cast<cudaEvent_t>(event)));
    return SLICEMOE_OK;
}

int slicemoe_event_elapsed_ms(void* start, void* stop, float* ms) {
    if (!start || !stop || !ms) return SLICEMOE_ERR_NULL;
    SLICEMOE_CUDA_TRY(cudaEventSynchronize(static_cast<cudaEvent_t>(stop)));
    SLICEMOE_CUDA_TRY(cudaEventElapsedTime(ms, static_cast<cudaEvent_t>(start), static_cast<cudaEvent_t>(stop)));
    return SLICEMOE_OK;
}

int slicemoe_last_status(const void* ws, void* stream) {
    if (!ws) return SLICEMOE_ERR_NULL;
    int32_t word = 0;
    SLICEMOE_CUDA_TRY(cudaMemcpyAsync(&word, ws, sizeof(word), cudaMemcpyDeviceToHost,
                                      static_cast<cudaStream_t>(stream)));
    SLICEMOE_CUDA_TRY(cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
    if (word == SLICEMOE_ERR_DEVICE_TIMEOUT) {
        // a launch gave up inside a grid barrier: put the barrier words back in order
        int rc = slicemoe::fused_forward_reset_sync(static_cast<cudaStream_t>(stream));
        if (rc) return rc;
        if ((rc = slicemoe::pp_forward_reset_sync(static_cast<cudaStream_t>(stream)))) return rc;
        if ((rc = slicemoe::decode_forward_reset_sync(static_cast<cudaStream_t>(stream)))) return rc;
    }
    return word;
}

int64_t slicemoe_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char* slicemoe_last_cuda_error(void) { return g_cuda_error; }

const char* slicemoe_status_string(int status) {
    switch (status) {
        case SLICEMOE_OK: return "ok";
        case SLICEMOE_ERR_NULL: return "a required pointer is NULL";
        case SLICEMOE_ERR_SHAPE: return "inconsistent shape";
        case SLICEMOE_ERR_UNSUPPORTED: return "shape, dtype or activation outside the built set";
        case SLICEMOE_ERR_ALIGN: return "a pointer is not aligned as required";
        case SLICEMOE_ERR_WORKSPACE: return "workspace missing or too small";
        case SLICEMOE_ERR_ALIAS: return "h_out overlaps h";
        case SLICEMOE_ERR_CUDA: return "a CUDA runtime call failed";
        case SLICEMOE_ERR_DEVICE_TIMEOUT: return "a bounded wait inside a kernel ran out";
        case SLICEMOE_ERR_NO_DEVICE: return "no usable sm_100 device";
        case SLICEMOE_ERR_STATIC_SCRATCH: return "problem too large for the fixed scratch of the allocation-free call";
        default: return "unknown status";
    }
}

}  // extern "C"
