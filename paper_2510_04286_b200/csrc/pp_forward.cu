// The forward of the layer (Section 3.1, Eq. 1; Section 3.4) on the pipeline of pp_body.cuh, for 64-wide slices
// without a capacity limit: as ONE cooperative launch
//
//   phase 1  router     top-k ids and probabilities, this CTA's rows of h' zeroed, and the dispatch: where the
//                       per-expert lists fit the scratch (E * 8 <= k * 128) the router's output warps append each
//                       pair's (pair, gate) entry to its expert's list, reserving list ranges with one atomic per
//                       expert and group of four tiles; otherwise they leave each pair's rank among the CTA's pairs
//                       of its expert and the CTA's per-expert counts
//   -- grid barrier --
//   phase 2  experts    row ranges from the experts' totals; rows gathered from h, outputs added into h'
//
// (for larger E a ranked dispatch phase between two grid barriers takes the place of the lists), and as one
// launch per phase (the stage-timed call).
#include <mutex>

#include "pp_body.cuh"

namespace slicemoe {
namespace {

struct PpFusedParams {
    PpParams route, ffn;
    int R, E, pairs_per_chunk;
    int32_t *assigned, *kept, *offsets, *dest;
    int2* pair_gate;
    unsigned long long* sync_word;
    int32_t* counts;          // [2][kMaxE] per-expert counters (kPpCountStride ints apart) of the one-barrier dispatch, used alternately by successive launches
    int lists;                // 1: one-barrier dispatch (per-expert lists), 0: ranked dispatch between two barriers
    int clear_status;
};

// Grid barriers of this file's cooperative kernel on ONE monotonic 64-bit arrival counter per device (zero at
// module load): a launch passes two barriers, i.e. adds 2 * gridDim.x.  The count a CTA finds at entry, rounded
// down to a multiple of that, is the launch's base whichever CTAs have already arrived; the barriers wait for
// base + gridDim.x and base + 2 * gridDim.x.  One release-add and acquire polls each: no last-arriver step.
__device__ unsigned long long g_pp_sync;
__device__ int32_t g_pp_counts[2 * kMaxE * kPpCountStride];

__device__ __forceinline__ bool pp_grid_barrier(unsigned long long* word, unsigned long long inc, unsigned long long target, PpShared& sh) {
    fence_proxy_async_smem();     // the phases reuse shared memory through different proxies
    __syncthreads();
    if (threadIdx.x == 0) {
        asm volatile("red.release.gpu.global.add.u64 [%0], %1;" ::"l"(word), "l"(inc) : "memory");
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

template <int EP, int N2, int ACT>
__global__ void __launch_bounds__(kPpThreads, 1)
pp_forward_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmXg,
                  const __grid_constant__ CUtensorMap tmWr1, const __grid_constant__ CUtensorMap tmWr2,
                  const __grid_constant__ CUtensorMap tmW1, const __grid_constant__ CUtensorMap tmW2,
                  const PpFusedParams fp) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ PpShared sh;
    const int warp = threadIdx.x >> 5;
    __shared__ unsigned long long base_s;
    // (not thread 0: that one requests the first row tiles at once and must not wait for this load)
    if (threadIdx.x == 96) {
        unsigned long long v;
        asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(fp.sync_word) : "memory");
        base_s = v - v % (2ull * gridDim.x);
        // successive launches alternate between two sets of list counters: each launch zeroes the set of the
        // next one (nobody touches that set during this launch)
        sh.counts_set = (int)((base_s / (2ull * gridDim.x)) & 1ull);
        if (blockIdx.x == 0 && fp.clear_status) *fp.ffn.status = SLICEMOE_OK;
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&sh.tmem_base), 512);
        tmem_relinquish();
    }
    pp_route_body<EP>(&tmX, &tmWr1, &tmWr2, fp.route, sh, smem_raw);       // (syncs the CTA: base_s and counts_set are visible in and after it)
    const unsigned long long base = base_s;
    const int parity = sh.counts_set;
    int32_t* counts = fp.counts + parity * (kMaxE * kPpCountStride);
    bool ok = sh.abort_flag == 0;
    int* dsm = reinterpret_cast<int*>((reinterpret_cast<uintptr_t>(smem_raw) + 15) & ~uintptr_t(15));
    if (blockIdx.x == 0 && (int)threadIdx.x < kMaxE) fp.counts[((parity ^ 1) * kMaxE + threadIdx.x) * kPpCountStride] = 0;
    if (fp.lists) {
        // (the router pass is over: the expert pass's barriers are set up while the CTA would wait anyway)
        if (threadIdx.x == 0) pp_ffn_init_bars(sh, &tmXg, &tmW1, &tmW2);
        ok = pp_grid_barrier(fp.sync_word, 2ull, base + 2ull * gridDim.x, sh) && ok;
        if (ok && warp == 0) {
            pp_offsets_from_counts(counts, fp.E, (int)(threadIdx.x & 31), blockIdx.x == 0, fp.assigned, fp.kept, fp.offsets, sh.offs);
            __syncwarp();
            pp_tile_starts(sh, fp.E, (int)(threadIdx.x & 31));
        }
    } else {
        ok = pp_grid_barrier(fp.sync_word, 1ull, base + gridDim.x, sh) && ok;
        if (ok)
            pp_dispatch_body<kPpThreads, true>(fp.route.topk_idx, fp.route.topk_p, fp.route.local_rank, fp.route.cta_hist,
                                               (int)gridDim.x, (int)blockIdx.x, fp.R, fp.E, fp.pairs_per_chunk, fp.assigned,
                                               fp.kept, fp.offsets, fp.dest, fp.pair_gate, dsm, sh.offs);
        if (threadIdx.x == 0) pp_ffn_init_bars(sh, &tmXg, &tmW1, &tmW2);
        ok = pp_grid_barrier(fp.sync_word, 1ull, base + 2ull * gridDim.x, sh) && ok;
        if (ok && warp == 0) pp_tile_starts(sh, fp.E, (int)(threadIdx.x & 31));
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (ok) pp_ffn_body<N2, ACT, true, true>(&tmXg, &tmW1, &tmW2, fp.ffn, sh, smem_raw);
    if (threadIdx.x == 0 && !ok) atomicExch(fp.ffn.status, (int)SLICEMOE_ERR_DEVICE_TIMEOUT);
    __syncthreads();
    if (warp == 1) {
        __syncwarp();
        tmem_dealloc(sh.tmem_base, 512);
    }
}

// ---- one launch per phase -------------------------------------------------------------------------
template <int EP>
__global__ void __launch_bounds__(kPpThreads, 1)
pp_route_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmWr1,
                const __grid_constant__ CUtensorMap tmWr2, const PpParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ PpShared sh;
    const int warp = threadIdx.x >> 5;
    if (warp == 1) {
        tmem_alloc(smem_u32(&sh.tmem_base), 512);
        tmem_relinquish();
    }
    pp_route_body<EP>(&tmX, &tmWr1, &tmWr2, p, sh, smem_raw);
    if (warp == 1) {
        __syncwarp();
        tmem_dealloc(sh.tmem_base, 512);
    }
}

__global__ void __launch_bounds__(kPpThreads, 1)
pp_dispatch_kernel(const int32_t* topk_idx, const float* topk_p, const int32_t* local_rank, const int32_t* table, int R,
                   int E, int pairs_per_chunk, int32_t* assigned, int32_t* kept, int32_t* offsets, int32_t* dest,
                   int2* pair_gate) {
    extern __shared__ int sm[];          // (2 E + 1 + G E) ints
    __shared__ int offs[kMaxE + 1];
    pp_dispatch_body<kPpThreads, false>(topk_idx, topk_p, local_rank, table, (int)gridDim.x, (int)blockIdx.x, R, E,
                                        pairs_per_chunk, assigned, kept, offsets, dest, pair_gate, sm, offs);
}

template <int N2, int ACT, bool STAGED = false>
__global__ void __launch_bounds__(kPpThreads, 1)
pp_ffn_kernel(const __grid_constant__ CUtensorMap tmXg, const __grid_constant__ CUtensorMap tmW1,
              const __grid_constant__ CUtensorMap tmW2, const PpParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ PpShared sh;
    const int warp = threadIdx.x >> 5;
    if (warp == 1) {
        tmem_alloc(smem_u32(&sh.tmem_base), 512);
        tmem_relinquish();
    }
    pp_ffn_body<N2, ACT, false, false, STAGED>(&tmXg, &tmW1, &tmW2, p, sh, smem_raw);
    if (warp == 1) {
        __syncwarp();
        tmem_dealloc(sh.tmem_base, 512);
    }
}

constexpr int kMaxDevices = 64;
std::mutex g_pp_mutex;
unsigned long long* g_pp_sync_addr[kMaxDevices] = {};
int32_t* g_pp_counts_addr[kMaxDevices] = {};
bool g_pp_attr[kMaxDevices][16] = {};      // per device and kernel instantiation: shared-memory limit raised

int pp_sync_address(unsigned long long** out, int32_t** counts_out) {
    int dev = -1;
    SLICEMOE_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return SLICEMOE_ERR_NO_DEVICE;
    std::lock_guard<std::mutex> lock(g_pp_mutex);
    if (!g_pp_sync_addr[dev]) {
        void* p = nullptr;
        SLICEMOE_CUDA_TRY(cudaGetSymbolAddress(&p, g_pp_sync));
        if (!p) return SLICEMOE_ERR_CUDA;
        g_pp_sync_addr[dev] = static_cast<unsigned long long*>(p);
        void* c = nullptr;
        SLICEMOE_CUDA_TRY(cudaGetSymbolAddress(&c, g_pp_counts));
        if (!c) return SLICEMOE_ERR_CUDA;
        g_pp_counts_addr[dev] = static_cast<int32_t*>(c);
    }
    *out = g_pp_sync_addr[dev];
    if (counts_out) *counts_out = g_pp_counts_addr[dev];
    return SLICEMOE_OK;
}

// cudaFuncSetAttribute is per device: once per (device, kernel).
template <class K>
int pp_set_smem(K kern, int slot, int bytes) {
    int dev = -1;
    SLICEMOE_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return SLICEMOE_ERR_NO_DEVICE;
    std::lock_guard<std::mutex> lock(g_pp_mutex);
    if (!g_pp_attr[dev][slot]) {
        SLICEMOE_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
        g_pp_attr[dev][slot] = true;
    }
    return SLICEMOE_OK;
}

struct PpMaps {
    CUtensorMap X, Xg, Wr1, Wr2, W1, W2;     // Xg: the rows of h with a one-row box (four-row gathers)
};

template <int EP, int N2>
int pp_make_maps(const Dims& D, const slicemoe_weights& w, const void* h, PpMaps& m) {
    int rc;
    if ((rc = make_tmap(&m.X, h, (uint64_t)D.N, (uint64_t)D.ds, 128))) return rc;
    if ((rc = make_tmap(&m.Xg, h, (uint64_t)D.N, (uint64_t)D.ds, 1))) return rc;
    if ((rc = make_tmap(&m.Wr1, w.Wr1, (uint64_t)D.Hr, (uint64_t)D.ds, kPpHC))) return rc;
    if ((rc = make_tmap(&m.Wr2, w.Wr2, (uint64_t)D.E, (uint64_t)D.Hr, EP))) return rc;       // (E = 8: zero-filled up to 16)
    if ((rc = make_tmap(&m.W1, w.W1, (uint64_t)D.E * D.F, (uint64_t)D.ds, kPpHC))) return rc;
    if ((rc = make_tmap(&m.W2, w.W2, (uint64_t)D.E * N2, (uint64_t)D.F, N2))) return rc;
    return SLICEMOE_OK;
}

void pp_fill_params(const Dims& D, const slicemoe_weights& w, const void* h, void* h_out, int32_t* topk_idx, float* topk_p,
                    int32_t* dest, int32_t* offsets, int2* pair_gate, int32_t* cta_hist, int32_t* status, PpParams& r,
                    PpParams& f) {
    r = PpParams{};
    r.status = status; r.n_rows = D.N; r.HID = D.Hr; r.experts_real = D.E; r.k = D.k;
    r.softmax_scale = 1.4426950408889634f * D.inv_tau;
    r.br1 = (const bf16*)w.br1; r.br2 = (const bf16*)w.br2;
    r.topk_idx = topk_idx; r.topk_p = topk_p; r.local_rank = dest; r.cta_hist = cta_hist;
    r.zero_out = (bf16*)h_out; r.row_elems = D.ds;
    r.train_gates = D.train_gates; r.drop_key0 = (uint32_t)D.drop_seed; r.drop_key1 = (uint32_t)(D.drop_seed >> 32);
    r.drop_threshold = D.drop_threshold;
    f = PpParams{};
    f.status = status; f.n_rows = D.R; f.HID = D.F; f.E = D.E; f.offsets = offsets;
    f.b1 = (const bf16*)w.b1; f.b2 = (const bf16*)w.b2;
    f.gather_src = (const bf16*)h; f.pair_gate = pair_gate;
    pair_to_row_magic(D.k, &f.gather_magic, &f.gather_shift);
    f.scatter_out = (bf16*)h_out; f.row_elems = D.ds; f.k = D.k;
}

template <int EP, int N2, int ACT>
int pp_launch_fused(const Dims& D, const slicemoe_weights& w, const void* h, const PpFusedParams& fp, cudaStream_t st) {
    PpMaps m;
    int rc = pp_make_maps<EP, N2>(D, w, h, m);
    if (rc) return rc;
    constexpr int smem = PpFfnCfg<N2>::SMEM_ALLOC > PpRouteCfg<EP>::SMEM_ALLOC ? PpFfnCfg<N2>::SMEM_ALLOC : PpRouteCfg<EP>::SMEM_ALLOC;
    static_assert(smem >= 120 * 1024, "one CTA per SM (each allocates all of tensor memory)");
    auto kern = pp_forward_kernel<EP, N2, ACT>;
    constexpr int slot = (EP == 16 ? 0 : EP == 32 ? 1 : 2) * 2 + (ACT == SLICEMOE_ACT_RELU ? 0 : 1);
    if ((rc = pp_set_smem(kern, slot, smem))) return rc;
    cudaLaunchConfig_t lc{};
    lc.gridDim = dim3(sm_count());
    lc.blockDim = dim3(kPpThreads);
    lc.dynamicSmemBytes = smem;
    lc.stream = st;
    cudaLaunchAttribute attrs[1];
    attrs[0].id = cudaLaunchAttributeCooperative;   // one CTA per SM, all resident at once
    attrs[0].val.cooperative = 1;
    lc.attrs = attrs;
    lc.numAttrs = 1;
    SLICEMOE_CUDA_TRY(cudaLaunchKernelEx(&lc, kern, m.X, m.Xg, m.Wr1, m.Wr2, m.W1, m.W2, fp));
    SLICEMOE_LAUNCH_CHECK(1);
    return SLICEMOE_OK;
}

template <int EP, int N2, int ACT>
int pp_launch_staged(const Dims& D, const slicemoe_weights& w, const void* h, const PpFusedParams& fp, cudaStream_t st,
                     void* const* events) {
    PpMaps m;
    int rc = pp_make_maps<EP, N2>(D, w, h, m);
    if (rc) return rc;
    const int tiles = (D.N + kTileM - 1) / kTileM;
    const int grid = tiles < sm_count() ? tiles : sm_count();
    const int rows_per_cta = ((tiles + grid - 1) / grid) * kTileM;
    auto mark = [&](int i) -> int {
        if (events) SLICEMOE_CUDA_TRY(cudaEventRecord(static_cast<cudaEvent_t>(events[i]), st));
        return SLICEMOE_OK;
    };
    constexpr int slot_r = 6 + (EP == 16 ? 0 : EP == 32 ? 1 : 2);
    constexpr int slot_f = 9 + (ACT == SLICEMOE_ACT_RELU ? 0 : 1);
    auto kr = pp_route_kernel<EP>;
    auto kf = pp_ffn_kernel<N2, ACT>;
    constexpr int smem_r = PpRouteCfg<EP>::SMEM_ALLOC > 120 * 1024 ? PpRouteCfg<EP>::SMEM_ALLOC : 120 * 1024;
    if ((rc = pp_set_smem(kr, slot_r, smem_r))) return rc;
    if ((rc = pp_set_smem(kf, slot_f, PpFfnCfg<N2>::SMEM_ALLOC))) return rc;
    if ((rc = mark(0))) return rc;
    kr<<<grid, kPpThreads, smem_r, st>>>(m.X, m.Wr1, m.Wr2, fp.route);
    SLICEMOE_LAUNCH_CHECK(1);
    if ((rc = mark(1))) return rc;
    pp_dispatch_kernel<<<grid, kPpThreads, sizeof(int) * (2 * D.E + 1 + (size_t)grid * D.E), st>>>(fp.route.topk_idx, fp.route.topk_p, fp.route.local_rank,
                                                    fp.route.cta_hist, fp.R, fp.E, rows_per_cta * D.k, fp.assigned, fp.kept,
                                                    fp.offsets, fp.dest, fp.pair_gate);
    SLICEMOE_LAUNCH_CHECK(1);
    if ((rc = mark(2))) return rc;
    const int ffn_grid = max_tiles(D) < sm_count() ? max_tiles(D) : sm_count();
    kf<<<ffn_grid, kPpThreads, PpFfnCfg<N2>::SMEM_ALLOC, st>>>(m.Xg, m.W1, m.W2, fp.ffn);
    SLICEMOE_LAUNCH_CHECK(1);
    if ((rc = mark(3))) return rc;
    return mark(4);
}

template <int EP, int N2>
int pp_launch_act(const Dims& D, const slicemoe_weights& w, const void* h, const PpFusedParams& fp, cudaStream_t st,
                  bool one_launch, void* const* events) {
    if (D.act == SLICEMOE_ACT_GELU_TANH)
        return one_launch ? pp_launch_fused<EP, N2, SLICEMOE_ACT_GELU_TANH>(D, w, h, fp, st)
                          : pp_launch_staged<EP, N2, SLICEMOE_ACT_GELU_TANH>(D, w, h, fp, st, events);
    return one_launch ? pp_launch_fused<EP, N2, SLICEMOE_ACT_RELU>(D, w, h, fp, st)
                      : pp_launch_staged<EP, N2, SLICEMOE_ACT_RELU>(D, w, h, fp, st, events);
}

bool pp_cooperative_launch_available() {
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

int pp_forward_reset_sync(cudaStream_t st) {
    unsigned long long* words = nullptr;
    int32_t* counts = nullptr;
    int rc = pp_sync_address(&words, &counts);
    if (rc) return rc;
    SLICEMOE_CUDA_TRY(cudaMemsetAsync(words, 0, sizeof(unsigned long long), st));
    SLICEMOE_CUDA_TRY(cudaMemsetAsync(counts, 0, 2 * kMaxE * kPpCountStride * sizeof(int32_t), st));
    SLICEMOE_CUDA_TRY(cudaStreamSynchronize(st));
    return SLICEMOE_OK;
}

bool pp_forward_supported(const Dims& D) {
    if (D.dtype != SLICEMOE_BF16 || D.ds != 64 || D.N <= 0) return false;
    if (D.E != 8 && D.E != 16 && D.E != 32 && D.E != 64) return false;
    if (D.k > 2 || D.capacity != 0 || D.noise_sigma > 0.0f) return false;
    if (D.Hr % 128 || D.Hr < 128 || D.Hr > kPpMaxHr) return false;      // (the router takes its hidden layer in halves of 128)
    if (D.F != 128 && D.F != kPpMaxF) return false;                    // (the activation takes the hidden layer in turns of 64 or 128 columns per warpgroup)
    return pp_cooperative_launch_available();
}

// The router pass as the staged call's kernel (slicemoe_route without the full probability matrix): top-k ids
// and probabilities, `assigned` by one atomic per expert and CTA.
bool pp_route_supported(const Dims& D) {
    if (D.dtype != SLICEMOE_BF16 || D.ds != 64 || D.N <= 0) return false;
    if (D.E != 8 && D.E != 16 && D.E != 32 && D.E != 64) return false;
    if (D.k > 2 || D.noise_sigma > 0.0f) return false;
    return D.Hr % 128 == 0 && D.Hr >= 128 && D.Hr <= kPpMaxHr;
}

template <int EP>
static int pp_launch_route_only(const Dims& D, const slicemoe_weights& w, const void* h, const PpParams& rp, cudaStream_t st) {
    PpMaps m;      // (only the router's three maps: the expert weights may be absent in this call)
    int rc;
    if ((rc = make_tmap(&m.X, h, (uint64_t)D.N, (uint64_t)D.ds, 128))) return rc;
    if ((rc = make_tmap(&m.Wr1, w.Wr1, (uint64_t)D.Hr, (uint64_t)D.ds, kPpHC))) return rc;
    if ((rc = make_tmap(&m.Wr2, w.Wr2, (uint64_t)D.E, (uint64_t)D.Hr, EP))) return rc;
    const int tiles = (D.N + kTileM - 1) / kTileM;
    const int grid = tiles < sm_count() ? tiles : sm_count();
    constexpr int slot_r = 6 + (EP == 16 ? 0 : EP == 32 ? 1 : 2);
    auto kr = pp_route_kernel<EP>;
    constexpr int smem_r = PpRouteCfg<EP>::SMEM_ALLOC > 120 * 1024 ? PpRouteCfg<EP>::SMEM_ALLOC : 120 * 1024;
    if ((rc = pp_set_smem(kr, slot_r, smem_r))) return rc;
    kr<<<grid, kPpThreads, smem_r, st>>>(m.X, m.Wr1, m.Wr2, rp);
    SLICEMOE_LAUNCH_CHECK(1);
    return SLICEMOE_OK;
}

int launch_route_pp(const Dims& D, const slicemoe_weights& w, const void* h, int32_t* topk_idx, float* topk_p,
                    int32_t* assigned, int32_t* status, cudaStream_t st) {
    if (assigned) SLICEMOE_CUDA_TRY(cudaMemsetAsync(assigned, 0, sizeof(int32_t) * D.E, st));
    PpParams r{}, f{};
    pp_fill_params(D, w, h, nullptr, topk_idx, topk_p, nullptr, nullptr, nullptr, nullptr, status, r, f);
    r.zero_out = nullptr;
    r.local_rank = nullptr;
    r.assigned_out = assigned;
    r.train_gates = 0;            // (the staged router returns the probabilities; slicemoe_gate_dropout is a call of its own)
    switch (D.E) {
        case 8:
        case 16: return pp_launch_route_only<16>(D, w, h, r, st);
        case 32: return pp_launch_route_only<32>(D, w, h, r, st);
        case 64: return pp_launch_route_only<64>(D, w, h, r, st);
        default: return SLICEMOE_ERR_UNSUPPORTED;
    }
}

// The expert pass as the staged call's kernel (slicemoe_expert_ffn on stacked, already weighted rows).
bool pp_ffn_supported(const Dims& D) {
    if (D.dtype != SLICEMOE_BF16 || D.ds != 64 || D.R <= 0 || D.E > kMaxE) return false;
    return D.F == 128 || D.F == kPpMaxF;
}

template <int ACT>
static int pp_launch_ffn_only(const Dims& D, const slicemoe_weights& w, const void* xperm, const PpParams& fpar, cudaStream_t st) {
    CUtensorMap mX, mW1, mW2;
    int rc;
    if ((rc = make_tmap(&mX, xperm, (uint64_t)D.R, (uint64_t)D.ds, 128))) return rc;
    if ((rc = make_tmap(&mW1, w.W1, (uint64_t)D.E * D.F, (uint64_t)D.ds, kPpHC))) return rc;
    if ((rc = make_tmap(&mW2, w.W2, (uint64_t)D.E * 64, (uint64_t)D.F, 64))) return rc;
    auto kf = pp_ffn_kernel<64, ACT, true>;
    constexpr int slot_f = 11 + (ACT == SLICEMOE_ACT_RELU ? 0 : 1);
    if ((rc = pp_set_smem(kf, slot_f, PpFfnCfg<64>::SMEM_ALLOC))) return rc;
    const int grid = max_tiles(D) < sm_count() ? max_tiles(D) : sm_count();
    kf<<<grid, kPpThreads, PpFfnCfg<64>::SMEM_ALLOC, st>>>(mX, mW1, mW2, fpar);
    SLICEMOE_LAUNCH_CHECK(1);
    return SLICEMOE_OK;
}

int launch_ffn_pp(const Dims& D, const slicemoe_weights& w, const void* xperm, const int32_t* offsets, void* yperm,
                  int32_t* status, cudaStream_t st) {
    PpParams r{}, f{};
    pp_fill_params(D, w, xperm, yperm, nullptr, nullptr, nullptr, const_cast<int32_t*>(offsets), nullptr, nullptr, status, r, f);
    f.gather_src = nullptr;
    f.pair_gate = nullptr;
    f.list_stride = 0;
    return D.act == SLICEMOE_ACT_GELU_TANH ? pp_launch_ffn_only<SLICEMOE_ACT_GELU_TANH>(D, w, xperm, f, st)
                                           : pp_launch_ffn_only<SLICEMOE_ACT_RELU>(D, w, xperm, f, st);
}

int launch_forward_pp(const Dims& D, const slicemoe_weights& w, const void* h, void* h_out, int32_t* topk_idx,
                      float* topk_p, int32_t* assigned, int32_t* kept, int32_t* offsets, int32_t* dest, void* pair_gate,
                      int32_t* cta_hist, int32_t* status, bool clear_status, bool one_launch, void* const* events,
                      cudaStream_t st) {
    PpFusedParams fp{};
    fp.clear_status = clear_status ? 1 : 0;
    int rc = pp_sync_address(&fp.sync_word, &fp.counts);
    if (rc) return rc;
    const int grid = sm_count();
    const int tiles = (D.N + kTileM - 1) / kTileM;
    const int rows_per_cta = ((tiles + grid - 1) / grid) * kTileM;
    pp_fill_params(D, w, h, h_out, topk_idx, topk_p, dest, offsets, static_cast<int2*>(pair_gate), cta_hist, status,
                   fp.route, fp.ffn);
    fp.R = D.R; fp.E = D.E; fp.pairs_per_chunk = rows_per_cta * D.k;
    fp.assigned = assigned; fp.kept = kept; fp.offsets = offsets; fp.dest = dest;
    fp.pair_gate = static_cast<int2*>(pair_gate);
    // the per-expert lists (E * N entries of 8 bytes) must fit in the stacked-row scratch (N * k rows of 128 bytes)
    fp.lists = (one_launch && D.E * 8 <= D.k * 128) ? 1 : 0;
    fp.ffn.list_stride = fp.lists ? D.N : 0;
    if (fp.lists) {          // the router's output warps fill the lists themselves (the counter set is chosen in the kernel)
        fp.route.lists_out = fp.pair_gate;
        fp.route.list_counts = fp.counts;
        fp.route.list_stride = D.N;
        fp.route.cta_hist = nullptr;
    }
    switch (D.E) {
        case 8:
        case 16: return pp_launch_act<16, 64>(D, w, h, fp, st, one_launch, events);
        case 32: return pp_launch_act<32, 64>(D, w, h, fp, st, one_launch, events);
        case 64: return pp_launch_act<64, 64>(D, w, h, fp, st, one_launch, events);
        default: return SLICEMOE_ERR_UNSUPPORTED;
    }
}

}  // namespace slicemoe
