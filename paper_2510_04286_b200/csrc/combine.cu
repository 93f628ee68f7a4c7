// Combine of Section 3.1: the k expert outputs of a row are summed (in j order, fp32, rounded
// once) and written at the row's own place in h'.  Dropped pairs add nothing; a row with no kept
// pair becomes zero.  One thread per 16-byte vector of h'; reads and writes are coalesced per row.
#include "common.cuh"

namespace slicemoe {
namespace {

constexpr int kThreads = 256;

template <typename T>
__global__ void __launch_bounds__(kThreads)
combine_kernel(const T* __restrict__ yperm, const int32_t* __restrict__ dest, T* __restrict__ h_out,
               long long nvec, int vec_per_row, int k, int ds) {
    constexpr int V = Vec<T>::n;
    for (long long v = (long long)blockIdx.x * kThreads + threadIdx.x; v < nvec;
         v += (long long)gridDim.x * kThreads) {
        const long long n = v / vec_per_row;
        const int col = (int)(v - n * vec_per_row);
        float acc[V];
#pragma unroll
        for (int i = 0; i < V; ++i) acc[i] = 0.0f;
        for (int j = 0; j < k; ++j) {
            const int r = dest[n * k + j];
            if (r >= 0) {
                float f[V];
                unpack16<T>(*reinterpret_cast<const uint4*>(yperm + (size_t)r * ds + (size_t)col * V), f);
#pragma unroll
                for (int i = 0; i < V; ++i) acc[i] += f[i];
            }
        }
        *reinterpret_cast<uint4*>(h_out + (size_t)v * V) = pack16<T>(acc);
    }
}

}  // namespace

int launch_combine(const Dims& D, const void* yperm, const int32_t* dest, void* h_out,
                   cudaStream_t st) {
    if (D.N == 0) return SLICEMOE_OK;
    const int V = D.dtype == SLICEMOE_BF16 ? 8 : 4;
    const int vec_per_row = D.ds / V;
    const long long nvec = (long long)D.N * vec_per_row;
    long long blocks = (nvec + kThreads - 1) / kThreads;
    const long long cap = 148LL * 32;
    const int grid = (int)(blocks < cap ? blocks : cap);
    if (D.dtype == SLICEMOE_BF16)
        combine_kernel<bf16><<<grid, kThreads, 0, st>>>((const bf16*)yperm, dest, (bf16*)h_out, nvec,
                                                      vec_per_row, D.k, D.ds);
    else
        combine_kernel<float><<<grid, kThreads, 0, st>>>((const float*)yperm, dest, (float*)h_out, nvec,
                                                       vec_per_row, D.k, D.ds);
    SLICEMOE_LAUNCH_CHECK(1);
    return SLICEMOE_OK;
}

}  // namespace slicemoe
