// Section 3.3, cross-slice dropout: train-mode gates from the top-k probabilities.
//
// Each of a row's k assignment probabilities is zeroed independently with probability `rate`; the
// survivors are divided by their sum; if none survives, the top-1 assignment (j = 0, the router
// writes its picks in descending order) gets weight 1.  The draw for assignment j of row n is the
// first word of Philox4x32-10 (Salmon et al., SC'11) with key = seed and counter = (n, j, 0, 0);
// dropped iff word < floor(rate * 2^32).  One thread per row, in place; k <= 8.
#include "common.cuh"
#include "philox.cuh"

namespace slicemoe {
namespace {

__device__ __forceinline__ uint32_t philox_first_word(uint32_t c0, uint32_t c1, uint32_t k0, uint32_t k1) {
    uint32_t x[4];
    philox4x32_10(c0, c1, 0u, 0u, k0, k1, x);
    return x[0];
}

__global__ void __launch_bounds__(256) gate_dropout_kernel(float* __restrict__ topk_p, int N, int k, uint32_t key0,
                                                           uint32_t key1, unsigned long long threshold) {
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    if (n >= N) return;
    float p[8];
    unsigned dropped = 0u;
    float kept_sum = 0.0f;
    for (int j = 0; j < k; ++j) {
        p[j] = topk_p[(size_t)n * k + j];
        const bool drop = (unsigned long long)philox_first_word((uint32_t)n, (uint32_t)j, key0, key1) < threshold;
        if (drop) dropped |= 1u << j;
        else kept_sum += p[j];
    }
    const bool none = dropped == (1u << k) - 1u || !(kept_sum > 0.0f);
    for (int j = 0; j < k; ++j) {
        float g;
        if (none) g = (j == 0) ? 1.0f : 0.0f;
        else g = ((dropped >> j) & 1u) ? 0.0f : p[j] / kept_sum;
        topk_p[(size_t)n * k + j] = g;
    }
}

}  // namespace

int launch_gate_dropout(const Dims& D, float* topk_p, uint64_t seed, unsigned long long threshold, cudaStream_t st) {
    if (D.N == 0) return SLICEMOE_OK;
    if (D.k > 8) return SLICEMOE_ERR_SHAPE;
    gate_dropout_kernel<<<(D.N + 255) / 256, 256, 0, st>>>(topk_p, D.N, D.k, (uint32_t)seed, (uint32_t)(seed >> 32), threshold);
    SLICEMOE_LAUNCH_CHECK(1);
    return SLICEMOE_OK;
}
}  // namespace slicemoe

extern "C" int slicemoe_gate_dropout(const slicemoe_config* cfg, float* topk_p, uint64_t seed, double rate,
                                     void* stream) {
    using namespace slicemoe;
    Dims D;
    int rc = make_dims(cfg, D);
    if (rc) return rc;
    if (!topk_p) return SLICEMOE_ERR_NULL;
    if (!(rate >= 0.0) || rate > 1.0 || D.k > 8) return SLICEMOE_ERR_SHAPE;
    if ((rc = check_device())) return rc;
    const unsigned long long threshold = (unsigned long long)(rate * 4294967296.0);   // 2^32 when rate = 1
    return launch_gate_dropout(D, topk_p, seed, threshold, static_cast<cudaStream_t>(stream));
}
