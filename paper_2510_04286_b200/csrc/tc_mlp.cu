// Router and expert kernels of the tensor-core path: tc_body (tc_mlp_body.cuh) with its own TMEM
// allocation, one launch per MLP.
#include "tc_mlp_body.cuh"

namespace slicemoe {
namespace {

template <class C>
__global__ void __launch_bounds__(C::THREADS, 1)
tc_mlp_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmW1,
              const __grid_constant__ CUtensorMap tmW2, const TcParams p) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ TcShared sh;
    const int warp = threadIdx.x >> 5;
    if (warp == 1) {
        tmem_alloc(smem_u32(&sh.tmem_base), C::TMEM_COLS);
        tmem_relinquish();
    }
    tc_body<C, false>(&tmA, &tmW1, &tmW2, p, sh, smem_raw);
    if (warp == 1) {
        __syncwarp();
        tmem_dealloc(sh.tmem_base, C::TMEM_COLS);
    }
}

template <class C>
int launch_tc(const void* A, uint64_t a_rows, const void* W1, const void* W2, int n_experts, const TcParams& p,
              int max_tiles, cudaStream_t st) {
    CUtensorMap tmA, tmW1, tmW2;
    int rc;
    // (a row narrower than K1 is zero-filled by the copies: the box reaches past the tensor's edge)
    if ((rc = make_tmap(&tmA, A, a_rows, (uint64_t)p.row_elems, 128))) return rc;
    if ((rc = make_tmap(&tmW1, W1, (uint64_t)n_experts * p.HID, (uint64_t)p.row_elems, C::HC))) return rc;
    // (router: the real expert count; a box taller than the tensor is zero-filled below its edge)
    if ((rc = make_tmap(&tmW2, W2, C::ROUTER ? (uint64_t)p.experts_real : (uint64_t)n_experts * C::N2, p.HID, C::N2))) return rc;
    auto kern = tc_mlp_kernel<C>;
    static bool attr_set[kAttrMaxDevices] = {};
    if ((rc = set_smem_limit_once(kern, kSmemLaunch<C>, attr_set))) return rc;
    const int grid = max_tiles < sm_count() ? max_tiles : sm_count();
    kern<<<grid, C::THREADS, kSmemLaunch<C>, st>>>(tmA, tmW1, tmW2, p);
    SLICEMOE_LAUNCH_CHECK(1);
    return SLICEMOE_OK;
}

template <int K1, int ACT, int N2 = K1>
int launch_ffn_k1(const Dims& D, const slicemoe_weights& w, const void* xperm, const TcParams& p, cudaStream_t st) {
    using C = TcCfg<K1, N2, false, ACT>;
    return launch_tc<C>(xperm, (uint64_t)(p.gather_src ? D.N : D.R), w.W1, w.W2, D.E, p, max_tiles(D), st);
}

template <int K1, int E>
int launch_route_k1e(const Dims& D, const slicemoe_weights& w, const void* h, const TcParams& p, cudaStream_t st) {
    using C = TcCfg<K1, E, true, SLICEMOE_ACT_RELU>;
    return launch_tc<C>(h, (uint64_t)D.N, w.Wr1, w.Wr2, 1, p, (D.N + kTileM - 1) / kTileM, st);
}

template <int K1>
int launch_route_k1(const Dims& D, const slicemoe_weights& w, const void* h, const TcParams& p, cudaStream_t st) {
    switch (D.E) {
        case 8:                                                     // padded to 16, see TcParams::experts_real
        case 16: return launch_route_k1e<K1, 16>(D, w, h, p, st);
        case 32: return launch_route_k1e<K1, 32>(D, w, h, p, st);
        case 64: return launch_route_k1e<K1, 64>(D, w, h, p, st);
        default: return SLICEMOE_ERR_UNSUPPORTED;
    }
}

}  // namespace


// Slice widths the tensor-core pipeline is built for.  The paper's own model (d = 768, S = 8) has
// ds = 96: it runs on the 128-wide instantiation, the copies zero-filling columns 96..127 of the row
// and weight tiles (a quarter of GEMM-1's MMA work multiplies zeros), with a 96-wide second GEMM.
// Likewise its S = 16 and S = 4 variants: ds = 48 under 64, ds = 192 under 256.
static bool tc_width_supported(int ds) {
    return ds == 48 || ds == 64 || ds == 96 || ds == 128 || ds == 192 || ds == 256;
}

bool tc_route_supported(const Dims& D) {
    if (D.dtype != SLICEMOE_BF16) return false;
    if (!tc_width_supported(D.ds)) return false;
    if (D.E != 8 && D.E != 16 && D.E != 32 && D.E != 64) return false;
    if (D.noise_sigma > 0.0f) return false;   // noisy logits (an ablation) stay on the CUDA-core router
    const int hc = D.ds <= 64 ? 128 : 64;
    // at least two hidden chunks: GEMM-1 is issued ahead of GEMM-2, and with resident weights that
    // look-ahead must not need the weight slot that the chunk in flight is still using
    return D.Hr % hc == 0 && D.Hr >= 2 * hc && D.Hr <= kMaxHid && D.k <= 8;
}

bool tc_ffn_supported(const Dims& D) {
    if (D.dtype != SLICEMOE_BF16) return false;
    if (!tc_width_supported(D.ds)) return false;
    const int hc = 64;
    return D.F % hc == 0 && D.F >= 2 * hc && D.F <= kMaxHid;
}

void tc_route_grid(const Dims& D, int* grid, int* rows_per_cta) {
    const int tiles = (D.N + kTileM - 1) / kTileM;
    const int g = tiles < sm_count() ? tiles : sm_count();
    *grid = g;
    *rows_per_cta = g > 0 ? ((tiles + g - 1) / g) * kTileM : 0;
}

int launch_route_tc(const Dims& D, const slicemoe_weights& w, const void* h, int32_t* topk_idx, float* topk_p,
                    int32_t* assigned, float* probs_opt, int32_t* status, cudaStream_t st, int32_t* cta_hist,
                    void* zero_out) {
    if (assigned) SLICEMOE_CUDA_TRY(cudaMemsetAsync(assigned, 0, sizeof(int32_t) * D.E, st));
    if (D.N == 0) return SLICEMOE_OK;
    TcParams p{};
    p.offsets = nullptr; p.n_rows = D.N; p.E = 1; p.HID = D.Hr;
    p.bias1 = (const bf16*)w.br1; p.bias2 = (const bf16*)w.br2;
    p.topk_idx = topk_idx; p.topk_p = topk_p; p.assigned = assigned; p.cta_hist = cta_hist; p.probs = probs_opt; p.k = D.k;
    p.status = status;
    p.zero_out = (bf16*)zero_out; p.zero_cols = D.ds;
    p.row_elems = D.ds;
    p.experts_real = D.E;
    p.softmax_scale = 1.4426950408889634f * D.inv_tau;
    switch (D.ds) {
        case 48:
        case 64: return launch_route_k1<64>(D, w, h, p, st);
        case 96:
        case 128: return launch_route_k1<128>(D, w, h, p, st);
        case 192:
        case 256: return launch_route_k1<256>(D, w, h, p, st);
        default: return SLICEMOE_ERR_UNSUPPORTED;
    }
}

int launch_ffn_tc(const Dims& D, const slicemoe_weights& w, const void* xperm, const int32_t* offsets, void* yperm,
                  int32_t* status, cudaStream_t st, const void* gather_h, const int32_t* perm, const float* gate,
                  void* scatter_out) {
    if (D.R == 0) return SLICEMOE_OK;
    TcParams p{};
    p.offsets = offsets; p.n_rows = (int)D.R; p.E = D.E; p.HID = D.F;
    p.bias1 = (const bf16*)w.b1; p.bias2 = (const bf16*)w.b2;
    p.yperm = (bf16*)yperm; p.status = status;
    p.gather_src = (const bf16*)gather_h; p.perm = perm; p.gate = gate; pair_to_row_magic(D.k, &p.gather_magic, &p.gather_shift);
    p.scatter_out = gather_h ? (bf16*)scatter_out : nullptr;
    p.split_hidden = p.scatter_out && D.k == 1 ? 1 : 0;
    if (gather_h) xperm = gather_h;   // the A tensor map is not used in gather mode; any valid matrix will do
    p.row_elems = D.ds;
    const bool gelu = D.act == SLICEMOE_ACT_GELU_TANH;
    if (D.ds == 48)
        return gelu ? launch_ffn_k1<64, SLICEMOE_ACT_GELU_TANH, 48>(D, w, xperm, p, st)
                    : launch_ffn_k1<64, SLICEMOE_ACT_RELU, 48>(D, w, xperm, p, st);
    if (D.ds == 96)
        return gelu ? launch_ffn_k1<128, SLICEMOE_ACT_GELU_TANH, 96>(D, w, xperm, p, st)
                    : launch_ffn_k1<128, SLICEMOE_ACT_RELU, 96>(D, w, xperm, p, st);
    if (D.ds == 192)
        return gelu ? launch_ffn_k1<256, SLICEMOE_ACT_GELU_TANH, 192>(D, w, xperm, p, st)
                    : launch_ffn_k1<256, SLICEMOE_ACT_RELU, 192>(D, w, xperm, p, st);
    if (D.ds == 64)
        return gelu ? launch_ffn_k1<64, SLICEMOE_ACT_GELU_TANH>(D, w, xperm, p, st)
                    : launch_ffn_k1<64, SLICEMOE_ACT_RELU>(D, w, xperm, p, st);
    if (D.ds == 128)
        return gelu ? launch_ffn_k1<128, SLICEMOE_ACT_GELU_TANH>(D, w, xperm, p, st)
                    : launch_ffn_k1<128, SLICEMOE_ACT_RELU>(D, w, xperm, p, st);
    if (D.ds == 256)
        return gelu ? launch_ffn_k1<256, SLICEMOE_ACT_GELU_TANH>(D, w, xperm, p, st)
                    : launch_ffn_k1<256, SLICEMOE_ACT_RELU>(D, w, xperm, p, st);
    return SLICEMOE_ERR_UNSUPPORTED;
}

}  // namespace slicemoe
