// Routing statistics from the per-expert counts the forward already produces:
//   Eq. 2            L_cap = alpha * (std(counts) / mean(counts))^2, population standard deviation
//   Section 4        ELE = -sum_e load_e log load_e / log E, load_e = counts_e / sum(counts)
// E numbers in, two doubles out: one warp, fp64, fixed summation order (lane-strided partial sums,
// then a shuffle tree), so the result is deterministic.
#include <cmath>

#include "common.cuh"

namespace slicemoe {
namespace {

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
    return v;
}

__global__ void __launch_bounds__(32) load_stats_kernel(const int32_t* __restrict__ counts, int E, double alpha,
                                                        double* __restrict__ out) {
    const int lane = threadIdx.x;
    double total = 0.0;
    for (int e = lane; e < E; e += 32) total += (double)counts[e];
    total = warp_sum(total);
    if (total <= 0.0) {                      // nothing routed: both are defined as 0
        if (lane == 0) { out[0] = 0.0; out[1] = 0.0; }
        return;
    }
    const double mean = total / E;
    double var = 0.0, ent = 0.0;
    for (int e = lane; e < E; e += 32) {
        const double c = (double)counts[e];
        var += (c - mean) * (c - mean);
        const double load = c / total;
        if (load > 0.0) ent -= load * log(load);          // 0 log 0 = 0
    }
    var = warp_sum(var) / E;
    ent = warp_sum(ent);
    if (lane == 0) {
        out[0] = alpha * var / (mean * mean);
        out[1] = (E == 1) ? 1.0 : ent / log((double)E);
    }
}

}  // namespace
}  // namespace slicemoe

extern "C" int slicemoe_load_stats(const int32_t* counts, int32_t E, double alpha, double* out, void* stream) {
    using namespace slicemoe;
    if (!counts || !out) return SLICEMOE_ERR_NULL;
    if (E < 1) return SLICEMOE_ERR_SHAPE;
    if (reinterpret_cast<uintptr_t>(out) & 7u) return SLICEMOE_ERR_ALIGN;
    int rc = check_device();
    if (rc) return rc;
    load_stats_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(counts, E, alpha, out);
    SLICEMOE_LAUNCH_CHECK(1);
    return SLICEMOE_OK;
}
