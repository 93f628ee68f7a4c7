// The whole forward of the layer (Section 3.1, Eq. 1; Section 3.4) as ONE cooperative launch:
//
//   phase 1  router       tc_body over this CTA's share of the row tiles: top-k ids and probabilities,
//                         this CTA's per-expert counts (one row of the table), its rows of h' zeroed
//                         (wide slices: a launch of its own before this one, route_wide.cu, and the kernel
//                         starts at phase 2)
//   -- grid barrier --    (the table is complete)
//   phase 2  dispatch     this CTA ranks the pairs its own router phase produced: dest, perm, gate;
//                         CTA 0 also writes assigned / kept / offsets
//   -- grid barrier --    (perm, gate and offsets are complete)
//   phase 3  experts      tc_body over this CTA's share of the expert tiles, rows gathered from h
//                         through perm, outputs added into h'
//
// One CTA per SM, all resident (cooperative launch), so the two grid barriers cannot deadlock; they
// are bounded anyway and a run-out sets the status word.  Against three launches this saves two
// kernel launches, two set-ups (barriers, TMEM allocation, tensor-map fetch) and the drain of the
// machine between them; TMEM is allocated once for both MLPs.
#include <cstdlib>
#include <mutex>

#include "dispatch_body.cuh"
#include "tc_mlp_body.cuh"

namespace slicemoe {
namespace {

struct FusedParams {
    TcParams route, ffn;
    int R, E, pairs_per_chunk, capacity;
    int32_t *assigned, *kept, *offsets, *dest, *perm;
    float* gate;
    int32_t* sync_words;      // g_grid_sync of this device
    int clear_status;         // set the status word to OK at entry
    int router_done;          // phase 1 ran as a launch of its own before this one (same grid, same row partition)
};

// Grid barrier words (arrival count, generation), one pair per device, owned by the library: zero
// when the module is loaded, and left ready for the next barrier by every barrier that completes
// (the last CTA to arrive sets the count back to zero and advances the generation the others poll),
// so that no launch has to clear them.  Two forwards cannot be inside their barrier phases at the
// same time on one device: a CTA of the later launch only becomes resident on an SM whose CTA of the
// earlier launch has exited, which is after its last barrier.
__device__ int32_t g_grid_sync[2];

// All CTAs of the grid arrive; returns false when the wait ran out (or this CTA had given up
// before).  Called by every thread of the CTA.  gen_before: the generation before this barrier
// (read once at kernel entry, plus the number of barriers passed since).
__device__ __forceinline__ bool grid_barrier(int32_t* words, int32_t gen_before, TcShared& sh) {
    // the phases reuse the same shared memory through different proxies (TMA / plain stores)
    fence_proxy_async_smem();
    __syncthreads();
    if (threadIdx.x == 0) {
        volatile int32_t* count = words;
        volatile int32_t* gen = words + 1;
        __threadfence();                                  // this CTA's writes before its arrival
        if (atomicAdd(words, 1) == (int)gridDim.x - 1) {
            *count = 0;
            __threadfence();
            atomicAdd(words + 1, 1);
        } else {
            const uint64_t t0 = globaltimer_ns();
            while (*gen == gen_before) {
                if (globaltimer_ns() - t0 > kWaitLimitNs) {
                    sh.abort_flag = 1;
                    break;
                }
                __nanosleep(64);
            }
        }
        __threadfence();
    }
    __syncthreads();
    return sh.abort_flag == 0;
}

template <class RC, class EC>
__global__ void __launch_bounds__(RC::THREADS, 1)
fused_forward_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmWr1,
                     const __grid_constant__ CUtensorMap tmWr2, const __grid_constant__ CUtensorMap tmW1,
                     const __grid_constant__ CUtensorMap tmW2, const FusedParams fp) {
    static_assert(RC::THREADS == EC::THREADS, "router and expert phases share the CTA");
    constexpr int TMEM_COLS = RC::TMEM_COLS > EC::TMEM_COLS ? RC::TMEM_COLS : EC::TMEM_COLS;
    extern __shared__ uint8_t smem_raw[];
    __shared__ TcShared sh;
    const int warp = threadIdx.x >> 5;
    int32_t gen0 = 0;
    if (threadIdx.x == 0) {
        gen0 = *reinterpret_cast<volatile int32_t*>(fp.sync_words + 1);   // no barrier can complete without this CTA
        if (blockIdx.x == 0 && fp.clear_status) *fp.ffn.status = SLICEMOE_OK;              // run-outs (>= seconds later) overwrite it
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&sh.tmem_base), TMEM_COLS);
        tmem_relinquish();
    }

    // ---- phase 1: router -----------------------------------------------------------------------
    bool ok = true;
    if (!fp.router_done) {
        tc_body<RC, false, false, true>(&tmX, &tmWr1, &tmWr2, fp.route, sh, smem_raw);
        ok = sh.abort_flag == 0;
        ok = grid_barrier(fp.sync_words, gen0, sh) && ok;
        ++gen0;
    } else {
        if (threadIdx.x == 0) sh.abort_flag = 0;
        __syncthreads();
    }

    // ---- phase 2: dispatch of this CTA's own pairs -----------------------------------------------
    if (ok) {
        int* dsm = reinterpret_cast<int*>((reinterpret_cast<uintptr_t>(smem_raw) + 15) & ~uintptr_t(15));
        dispatch_fused_body<RC::THREADS, true>(fp.route.topk_idx, fp.route.topk_p, fp.route.cta_hist, (int)gridDim.x,
                                               (int)blockIdx.x, fp.R, fp.E, fp.pairs_per_chunk, fp.capacity,
                                               fp.assigned, fp.kept, fp.offsets, fp.dest, fp.perm, fp.gate, dsm, sh.offs);
    }
    ok = grid_barrier(fp.sync_words, gen0, sh) && ok;

    // ---- phase 3: experts ------------------------------------------------------------------------
    if (ok) tc_body<EC, true, true, true>(&tmX, &tmW1, &tmW2, fp.ffn, sh, smem_raw);
    if (threadIdx.x == 0 && !ok) atomicExch(fp.ffn.status, (int)SLICEMOE_ERR_DEVICE_TIMEOUT);

    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tmem_dealloc(sh.tmem_base, TMEM_COLS);
    }
}

template <class RC, class EC>
int launch_fused(const Dims& D, const slicemoe_weights& w, const void* h, const FusedParams& fp, cudaStream_t st) {
    CUtensorMap tmX, tmWr1, tmWr2, tmW1, tmW2;
    int rc;
    // (rows narrower than K1 are zero-filled by the copies: the box reaches past the tensor's edge)
    if ((rc = make_tmap(&tmX, h, (uint64_t)D.N, (uint64_t)D.ds, 128))) return rc;
    if ((rc = make_tmap(&tmWr1, w.Wr1, (uint64_t)D.Hr, (uint64_t)D.ds, RC::HC))) return rc;
    if ((rc = make_tmap(&tmWr2, w.Wr2, (uint64_t)D.E, D.Hr, RC::N2))) return rc;   // (E = 8: zero-filled up to 16)
    if ((rc = make_tmap(&tmW1, w.W1, (uint64_t)D.E * D.F, (uint64_t)D.ds, EC::HC))) return rc;
    if ((rc = make_tmap(&tmW2, w.W2, (uint64_t)D.E * EC::N2, D.F, EC::N2))) return rc;
    const int grid = sm_count();
    size_t smem = RC::SMEM_ALLOC > EC::SMEM_ALLOC ? RC::SMEM_ALLOC : EC::SMEM_ALLOC;
    const size_t dsm = dispatch_fused_smem_bytes(D.E, grid, RC::THREADS) + 16;
    if (dsm > smem) smem = dsm;
    if (smem + sizeof(TcShared) + 64 > 227 * 1024) return SLICEMOE_ERR_UNSUPPORTED;
    auto kern = fused_forward_kernel<RC, EC>;
    static bool attr_set[kAttrMaxDevices] = {};
    if ((rc = set_smem_limit_once(kern, (int)(227 * 1024 - sizeof(TcShared) - 64), attr_set))) return rc;
    // One CTA per SM, all resident at once: a cooperative launch states that requirement.
    // (Programmatic dependent launch on top of it was measured and bought nothing: the next grid's
    // CTAs cannot become resident before this grid's CTAs leave their SMs.)
    cudaLaunchConfig_t lc{};
    lc.gridDim = dim3(grid);
    lc.blockDim = dim3(RC::THREADS);
    lc.dynamicSmemBytes = smem;
    lc.stream = st;
    cudaLaunchAttribute attrs[1];
    attrs[0].id = cudaLaunchAttributeCooperative;
    attrs[0].val.cooperative = 1;
    lc.attrs = attrs;
    lc.numAttrs = 1;
    SLICEMOE_CUDA_TRY(cudaLaunchKernelEx(&lc, kern, tmX, tmWr1, tmWr2, tmW1, tmW2, fp));
    SLICEMOE_LAUNCH_CHECK(1);
    return SLICEMOE_OK;
}

template <int K1, int E, int N2>
int launch_fused_k1e(const Dims& D, const slicemoe_weights& w, const void* h, const FusedParams& fp, cudaStream_t st) {
    using RC = TcCfg<K1, E, true, SLICEMOE_ACT_RELU>;
    if (D.act == SLICEMOE_ACT_GELU_TANH)
        return launch_fused<RC, TcCfg<K1, N2, false, SLICEMOE_ACT_GELU_TANH>>(D, w, h, fp, st);
    return launch_fused<RC, TcCfg<K1, N2, false, SLICEMOE_ACT_RELU>>(D, w, h, fp, st);
}

// K1: the width the kernels are built for; N2: the real slice width (= the second expert GEMM's N)
template <int K1, int N2 = K1>
int launch_fused_k1(const Dims& D, const slicemoe_weights& w, const void* h, const FusedParams& fp, cudaStream_t st) {
    switch (D.E) {
        case 8:
        case 16: return launch_fused_k1e<K1, 16, N2>(D, w, h, fp, st);
        case 32: return launch_fused_k1e<K1, 32, N2>(D, w, h, fp, st);
        case 64: return launch_fused_k1e<K1, 64, N2>(D, w, h, fp, st);
        default: return SLICEMOE_ERR_UNSUPPORTED;
    }
}

constexpr int kMaxDevices = 64;
std::mutex g_sync_mutex;
int32_t* g_sync_addr[kMaxDevices] = {};

// Device address of g_grid_sync on the current device, looked up once per device.
int grid_sync_address(int32_t** out) {
    int dev = -1;
    SLICEMOE_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return SLICEMOE_ERR_NO_DEVICE;
    std::lock_guard<std::mutex> lock(g_sync_mutex);
    if (!g_sync_addr[dev]) {
        void* p = nullptr;
        SLICEMOE_CUDA_TRY(cudaGetSymbolAddress(&p, g_grid_sync));
        if (!p) return SLICEMOE_ERR_CUDA;
        g_sync_addr[dev] = static_cast<int32_t*>(p);
    }
    *out = g_sync_addr[dev];
    return SLICEMOE_OK;
}

bool cooperative_launch_available() {
    static int ok = [] {
        int dev = 0, v = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&v, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess)
            v = 0;
        return v;
    }();
    return ok != 0;
}

}  // namespace

int fused_forward_reset_sync(cudaStream_t st) {
    int32_t* words = nullptr;
    int rc = grid_sync_address(&words);
    if (rc) return rc;
    SLICEMOE_CUDA_TRY(cudaMemsetAsync(words, 0, 2 * sizeof(int32_t), st));
    SLICEMOE_CUDA_TRY(cudaStreamSynchronize(st));
    return SLICEMOE_OK;
}

int fused_forward_grid() { return sm_count(); }

bool fused_forward_supported(const Dims& D) {
    return tc_route_supported(D) && tc_ffn_supported(D) && D.N > 0 && D.k <= 2 && cooperative_launch_available();
}

int launch_forward_fused(const Dims& D, const slicemoe_weights& w, const void* h, void* h_out, int32_t* topk_idx,
                         float* topk_p, int32_t* assigned, int32_t* kept, int32_t* offsets, int32_t* dest,
                         int32_t* perm, float* gate, int32_t* cta_hist, int32_t* status, bool clear_status,
                         cudaStream_t st, bool router_done) {
    FusedParams fp{};
    fp.clear_status = clear_status ? 1 : 0;
    fp.router_done = router_done ? 1 : 0;
    int rc = grid_sync_address(&fp.sync_words);
    if (rc) return rc;
    const int grid = sm_count();
    const int tiles = (D.N + kTileM - 1) / kTileM;
    const int rows_per_cta = ((tiles + grid - 1) / grid) * kTileM;

    TcParams& r = fp.route;
    r.offsets = nullptr; r.n_rows = D.N; r.E = 1; r.HID = D.Hr;
    r.bias1 = (const bf16*)w.br1; r.bias2 = (const bf16*)w.br2;
    r.topk_idx = topk_idx; r.topk_p = topk_p; r.assigned = nullptr; r.cta_hist = cta_hist; r.probs = nullptr; r.k = D.k;
    r.status = status;
    r.zero_out = (bf16*)h_out; r.zero_cols = D.ds;

    TcParams& f = fp.ffn;
    f.offsets = offsets; f.n_rows = (int)D.R; f.E = D.E; f.HID = D.F;
    f.bias1 = (const bf16*)w.b1; f.bias2 = (const bf16*)w.b2;
    f.yperm = nullptr; f.status = status;
    f.gather_src = (const bf16*)h; f.perm = perm; f.gate = gate; pair_to_row_magic(D.k, &f.gather_magic, &f.gather_shift);
    f.scatter_out = (bf16*)h_out;
    f.split_hidden = D.k == 1 ? 1 : 0;     // (k = 1: a row of h' has one writer, two with the hidden layer in halves)

    fp.R = (int)D.R; fp.E = D.E; fp.pairs_per_chunk = rows_per_cta * D.k; fp.capacity = (int)D.capacity;
    fp.assigned = assigned; fp.kept = kept; fp.offsets = offsets; fp.dest = dest; fp.perm = perm; fp.gate = gate;
    r.row_elems = D.ds;
    f.row_elems = D.ds;
    r.experts_real = D.E;
    r.softmax_scale = 1.4426950408889634f * D.inv_tau;
    switch (D.ds) {
        case 48: return launch_fused_k1<64, 48>(D, w, h, fp, st);
        case 64: return launch_fused_k1<64>(D, w, h, fp, st);
        case 96: return launch_fused_k1<128, 96>(D, w, h, fp, st);
        case 128: return launch_fused_k1<128>(D, w, h, fp, st);
        case 192: return launch_fused_k1<256, 192>(D, w, h, fp, st);
        case 256: return launch_fused_k1<256>(D, w, h, fp, st);
        default: return SLICEMOE_ERR_UNSUPPORTED;
    }
}

}  // namespace slicemoe
