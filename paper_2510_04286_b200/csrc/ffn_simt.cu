// Grouped expert FFN of Section 3.1 / 3.4 on CUDA cores: for each expert e and each stacked row r
// of its range, y = W2_e act(W1_e x + b1_e) + b2_e.  fp32 arithmetic with a fixed summation order
// in both storage types.  This is the fp32 path of the library and the path for shapes the
// tensor-core kernel does not take.
//
// One CTA owns one tile of TM rows of one expert.  The tile is found on the device from
// `offsets` (no host synchronisation): the grid is the upper bound ceil(R/TM) + E and surplus
// CTAs leave at once.  The hidden layer is processed in chunks of kFC units that never leave
// shared memory.
#include "common.cuh"

namespace slicemoe {
namespace {

constexpr int kThreads = 256;
constexpr int kFC = 256;  // hidden units per chunk (one per thread)

template <typename T, int TM>
__global__ void __launch_bounds__(kThreads)
ffn_simt_kernel(const T* __restrict__ xperm, const int32_t* __restrict__ offsets,
                const T* __restrict__ W1, const T* __restrict__ b1, const T* __restrict__ W2,
                const T* __restrict__ b2, T* __restrict__ yperm, int E, int ds, int F, int act) {
    extern __shared__ __align__(16) float smem[];
    float* xs = smem;              // [TM][ds]
    float* ys = xs + TM * ds;      // [TM][ds]
    float* us = ys + TM * ds;      // [TM][kFC]
    __shared__ int tile_info[3];   // expert, first row, rows
    constexpr int V = Vec<T>::n;
    const int tid = threadIdx.x;

    if (tid == 0) {
        int t = blockIdx.x, found = -1, row0 = 0, rows = 0;
        for (int e = 0; e < E; ++e) {
            const int lo = offsets[e], n_e = offsets[e + 1] - lo;
            const int nt = (n_e + TM - 1) / TM;
            if (t < nt) { found = e; row0 = lo + t * TM; rows = min(TM, n_e - t * TM); break; }
            t -= nt;
        }
        tile_info[0] = found; tile_info[1] = row0; tile_info[2] = rows;
    }
    __syncthreads();
    const int e = tile_info[0], row0 = tile_info[1], rows = tile_info[2];
    if (e < 0) return;

    const T* W1e = W1 + (size_t)e * F * ds;
    const T* W2e = W2 + (size_t)e * ds * F;

    for (int v = tid; v < TM * ds / V; v += kThreads) {
        const int r = (v * V) / ds;
        float f[V];
        if (r < rows) {
            unpack16<T>(*reinterpret_cast<const uint4*>(xperm + (size_t)row0 * ds + (size_t)v * V), f);
        } else {
#pragma unroll
            for (int i = 0; i < V; ++i) f[i] = 0.0f;
        }
#pragma unroll
        for (int i = 0; i < V; ++i) xs[v * V + i] = f[i];
    }
    for (int i = tid; i < TM * ds; i += kThreads) {
        const int c = i % ds;
        ys[i] = b2 ? to_f32(b2[(size_t)e * ds + c]) : 0.0f;
    }
    __syncthreads();

    // layer 2 work split: (group g, column c) items; each item owns rows [g*rpg, (g+1)*rpg)
    const int groups = ds >= kThreads ? 1 : min(TM, kThreads / ds);
    const int rpg = (TM + groups - 1) / groups;

    for (int f0 = 0; f0 < F; f0 += kFC) {
        const int fc = min(kFC, F - f0);
        // layer 1: hidden unit f0 + tid for all rows
        if (tid < fc) {
            const int f = f0 + tid;
            float acc[TM];
            const float b = b1 ? to_f32(b1[(size_t)e * F + f]) : 0.0f;
#pragma unroll
            for (int r = 0; r < TM; ++r) acc[r] = b;
            const T* wrow = W1e + (size_t)f * ds;
            for (int q = 0; q < ds; q += V) {
                float wv[V];
                unpack16<T>(*reinterpret_cast<const uint4*>(wrow + q), wv);
#pragma unroll
                for (int u = 0; u < V; ++u) {
#pragma unroll
                    for (int r = 0; r < TM; ++r) acc[r] = fmaf(wv[u], xs[r * ds + q + u], acc[r]);
                }
            }
#pragma unroll
            for (int r = 0; r < TM; ++r) us[r * kFC + tid] = apply_act(acc[r], act);
        }
        __syncthreads();
        // layer 2: add this chunk's contribution to the outputs
        for (int item = tid; item < groups * ds; item += kThreads) {
            const int g = item / ds, c = item - g * ds;
            const T* wrow = W2e + (size_t)c * F + f0;
            float acc[TM];
#pragma unroll
            for (int r = 0; r < TM; ++r) acc[r] = 0.0f;
            for (int f = 0; f < fc; f += V) {
                float wv[V];
                unpack16<T>(*reinterpret_cast<const uint4*>(wrow + f), wv);
#pragma unroll
                for (int u = 0; u < V; ++u) {
#pragma unroll
                    for (int r = 0; r < TM; ++r) {
                        const int row = g * rpg + r;
                        if (r < rpg && row < TM) acc[r] = fmaf(wv[u], us[row * kFC + f + u], acc[r]);
                    }
                }
            }
#pragma unroll
            for (int r = 0; r < TM; ++r) {
                const int row = g * rpg + r;
                if (r < rpg && row < TM) ys[row * ds + c] += acc[r];
            }
        }
        __syncthreads();
    }

    for (int v = tid; v < rows * ds / V; v += kThreads) {
        float f[V];
#pragma unroll
        for (int i = 0; i < V; ++i) f[i] = ys[v * V + i];
        *reinterpret_cast<uint4*>(yperm + (size_t)row0 * ds + (size_t)v * V) = pack16<T>(f);
    }
}

template <typename T, int TM>
int launch_tm(const Dims& D, const slicemoe_weights& w, const void* xperm, const int32_t* offsets,
              void* yperm, cudaStream_t st) {
    const size_t smem = sizeof(float) * (size_t)TM * (2 * D.ds + kFC);
    auto kern = ffn_simt_kernel<T, TM>;
    SLICEMOE_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    const int grid = (D.R + TM - 1) / TM + D.E;
    kern<<<grid, kThreads, smem, st>>>((const T*)xperm, offsets, (const T*)w.W1, (const T*)w.b1,
                                      (const T*)w.W2, (const T*)w.b2, (T*)yperm, D.E, D.ds, D.F, D.act);
    SLICEMOE_LAUNCH_CHECK(1);
    return SLICEMOE_OK;
}

template <typename T>
int launch_typed(const Dims& D, const slicemoe_weights& w, const void* xperm, const int32_t* offsets,
                 void* yperm, cudaStream_t st) {
    const size_t budget = 200 * 1024;
    if (sizeof(float) * 32 * (size_t)(2 * D.ds + kFC) <= budget)
        return launch_tm<T, 32>(D, w, xperm, offsets, yperm, st);
    if (sizeof(float) * 4 * (size_t)(2 * D.ds + kFC) <= budget)
        return launch_tm<T, 4>(D, w, xperm, offsets, yperm, st);
    return SLICEMOE_ERR_UNSUPPORTED;
}

}  // namespace

int launch_ffn_simt(const Dims& D, const slicemoe_weights& w, const void* xperm,
                    const int32_t* offsets, void* yperm, cudaStream_t st) {
    if (D.R == 0) return SLICEMOE_OK;
    if (D.dtype == SLICEMOE_BF16) return launch_typed<bf16>(D, w, xperm, offsets, yperm, st);
    return launch_typed<float>(D, w, xperm, offsets, yperm, st);
}

}  // namespace slicemoe
