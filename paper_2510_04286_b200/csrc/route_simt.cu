// Router of Section 3.1 on CUDA cores: Linear(ds->Hr) + ReLU, Linear(Hr->E), softmax, top-k.
// All arithmetic is fp32 with a fixed summation order, whatever the storage type.  This is the
// fp32 path of the library and the path for shapes the tensor-core router does not take.
// Ablation knobs (Figures 6 and 7): the softmax and the top-k see (g + sigma * eps) / tau, eps a
// standard normal per (row, expert) from Philox4x32-10, key = seed, counter (n, e, 1, 0), through
// Box-Muller on 24-bit uniforms.
#include "common.cuh"
#include "philox.cuh"

namespace slicemoe {
namespace {

constexpr int kThreads = 256;
constexpr int kMaxK = 8;

// One CTA routes ROWS consecutive rows.
template <typename T, int ROWS>
__global__ void __launch_bounds__(kThreads)
route_simt_kernel(const T* __restrict__ X, const T* __restrict__ Wr1, const T* __restrict__ br1,
                  const T* __restrict__ Wr2, const T* __restrict__ br2, int N, int ds, int Hr, int E,
                  int k, int32_t* __restrict__ topk_idx, float* __restrict__ topk_p,
                  int32_t* __restrict__ assigned, float* __restrict__ probs, float inv_tau, float sigma,
                  uint32_t key0, uint32_t key1) {
    extern __shared__ __align__(16) float smem[];
    float* xs = smem;                 // [ROWS][ds]
    float* hs = xs + ROWS * ds;       // [ROWS][Hr]
    float* gs = hs + ROWS * Hr;       // [ROWS][E]   logits, then probabilities
    int* cnt = reinterpret_cast<int*>(gs + ROWS * E);  // [E]
    constexpr int V = Vec<T>::n;
    const int tid = threadIdx.x;
    const int row0 = blockIdx.x * ROWS;
    const int rows = min(ROWS, N - row0);

    for (int e = tid; e < E; e += kThreads) cnt[e] = 0;
    // stage the rows (zero padding past N)
    for (int v = tid; v < ROWS * ds / V; v += kThreads) {
        const int r = (v * V) / ds;
        float f[V];
        if (r < rows) {
            const uint4 raw = *reinterpret_cast<const uint4*>(X + (size_t)row0 * ds + (size_t)v * V);
            unpack16<T>(raw, f);
        } else {
#pragma unroll
            for (int i = 0; i < V; ++i) f[i] = 0.0f;
        }
#pragma unroll
        for (int i = 0; i < V; ++i) xs[v * V + i] = f[i];
    }
    __syncthreads();

    // layer 1: hidden unit i for all staged rows
    for (int i = tid; i < Hr; i += kThreads) {
        float acc[ROWS];
        const float b = br1 ? to_f32(br1[i]) : 0.0f;
#pragma unroll
        for (int r = 0; r < ROWS; ++r) acc[r] = b;
        const T* wrow = Wr1 + (size_t)i * ds;
        for (int q = 0; q < ds; q += V) {
            float wv[V];
            unpack16<T>(*reinterpret_cast<const uint4*>(wrow + q), wv);
#pragma unroll
            for (int u = 0; u < V; ++u) {
#pragma unroll
                for (int r = 0; r < ROWS; ++r) acc[r] = fmaf(wv[u], xs[r * ds + q + u], acc[r]);
            }
        }
#pragma unroll
        for (int r = 0; r < ROWS; ++r) hs[r * Hr + i] = fmaxf(acc[r], 0.0f);
    }
    __syncthreads();

    // layer 2: one (row, expert) logit per work item
    for (int item = tid; item < ROWS * E; item += kThreads) {
        const int r = item / E, e = item - r * E;
        float acc = br2 ? to_f32(br2[e]) : 0.0f;
        const T* wrow = Wr2 + (size_t)e * Hr;
        const float* hrow = hs + r * Hr;
        int i = 0;
        for (; i + V <= Hr; i += V) {
            float wv[V];
            unpack16<T>(*reinterpret_cast<const uint4*>(wrow + i), wv);
#pragma unroll
            for (int u = 0; u < V; ++u) acc = fmaf(wv[u], hrow[i + u], acc);
        }
        for (; i < Hr; ++i) acc = fmaf(to_f32(wrow[i]), hrow[i], acc);
        if (sigma > 0.0f && r < rows) acc = fmaf(sigma, logit_noise(row0 + r, e, key0, key1), acc);
        gs[r * E + e] = acc * inv_tau;
    }
    __syncthreads();

    // softmax and top-k, one thread per row, fp32
    if (tid < rows) {
        float* g = gs + tid * E;
        const int n = row0 + tid;
        int chosen[kMaxK];
        float gsel[kMaxK];
        for (int j = 0; j < k; ++j) {
            int best = -1;
            float bv = 0.0f;
            for (int e = 0; e < E; ++e) {
                bool taken = false;
                for (int i = 0; i < j; ++i) taken |= (chosen[i] == e);
                if (taken) continue;
                const float v = g[e];
                if (best < 0 || v > bv) { best = e; bv = v; }
            }
            chosen[j] = best;
            gsel[j] = bv;
        }
        const float m = gsel[0];
        float sum = 0.0f;
        for (int e = 0; e < E; ++e) sum += expf(g[e] - m);
        const float inv = 1.0f / sum;
        for (int j = 0; j < k; ++j) {
            topk_idx[(size_t)n * k + j] = chosen[j];
            topk_p[(size_t)n * k + j] = expf(gsel[j] - m) * inv;
            atomicAdd(&cnt[chosen[j]], 1);
        }
        if (probs) {
            for (int e = 0; e < E; ++e) probs[(size_t)n * E + e] = expf(g[e] - m) * inv;
        }
    }
    __syncthreads();
    for (int e = tid; e < E; e += kThreads)
        if (cnt[e]) atomicAdd(&assigned[e], cnt[e]);
}

template <typename T, int ROWS>
int launch_rows(const Dims& D, const slicemoe_weights& w, const void* h, int32_t* topk_idx,
                float* topk_p, int32_t* assigned, float* probs, cudaStream_t st) {
    const size_t smem = sizeof(float) * (size_t)ROWS * (D.ds + D.Hr + D.E) + sizeof(int) * D.E;
    auto kern = route_simt_kernel<T, ROWS>;
    SLICEMOE_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    const int grid = (D.N + ROWS - 1) / ROWS;
    kern<<<grid, kThreads, smem, st>>>((const T*)h, (const T*)w.Wr1, (const T*)w.br1, (const T*)w.Wr2,
                                      (const T*)w.br2, D.N, D.ds, D.Hr, D.E, D.k, topk_idx, topk_p,
                                      assigned, probs, D.inv_tau, D.noise_sigma, (uint32_t)D.noise_seed,
                                      (uint32_t)(D.noise_seed >> 32));
    SLICEMOE_LAUNCH_CHECK(1);
    return SLICEMOE_OK;
}

template <typename T>
int launch_typed(const Dims& D, const slicemoe_weights& w, const void* h, int32_t* topk_idx,
                 float* topk_p, int32_t* assigned, float* probs, cudaStream_t st) {
    const size_t per_row = sizeof(float) * (size_t)(D.ds + D.Hr + D.E);
    const size_t budget = 200 * 1024 - sizeof(int) * D.E;
    if (16 * per_row <= budget) return launch_rows<T, 16>(D, w, h, topk_idx, topk_p, assigned, probs, st);
    if (4 * per_row <= budget) return launch_rows<T, 4>(D, w, h, topk_idx, topk_p, assigned, probs, st);
    if (per_row <= budget) return launch_rows<T, 1>(D, w, h, topk_idx, topk_p, assigned, probs, st);
    return SLICEMOE_ERR_UNSUPPORTED;
}

}  // namespace

int launch_route_simt(const Dims& D, const slicemoe_weights& w, const void* h, int32_t* topk_idx,
                      float* topk_p, int32_t* assigned, float* probs_opt, cudaStream_t st) {
    if (D.k > kMaxK) return SLICEMOE_ERR_UNSUPPORTED;
    SLICEMOE_CUDA_TRY(cudaMemsetAsync(assigned, 0, sizeof(int32_t) * D.E, st));
    if (D.N == 0) return SLICEMOE_OK;
    if (D.dtype == SLICEMOE_BF16)
        return launch_typed<bf16>(D, w, h, topk_idx, topk_p, assigned, probs_opt, st);
    return launch_typed<float>(D, w, h, topk_idx, topk_p, assigned, probs_opt, st);
}

}  // namespace slicemoe
