// Shuffled slices (Section 5.2, Figure 5): a fixed permutation of the d columns applied before the
// layer and undone on its output.  HBM-bound copy: a CTA stages whole rows in shared memory, so
// that both the global reads and the global writes are 16-byte vectors in row order and the
// permutation itself happens on shared-memory addresses.
//   forward: out[t, c] = in[t, perm[c]]        inverse: out[t, perm[c]] = in[t, c]
#include "common.cuh"

namespace slicemoe {
namespace {

constexpr int kThreads = 256;
constexpr int kStageBytes = 16 * 1024;   // rows staged per step: as many as fit here (at least one)

// V consecutive entries of the permutation (16-byte aligned: V is 4 or 8 and the start a multiple of V).
template <int V>
__device__ __forceinline__ void load_perm(const int32_t* __restrict__ p, int* out) {
#pragma unroll
    for (int i = 0; i < V; i += 4) {
        const int4 q = __ldg(reinterpret_cast<const int4*>(p + i));
        out[i] = q.x; out[i + 1] = q.y; out[i + 2] = q.z; out[i + 3] = q.w;
    }
}

template <typename T, bool INVERSE>
__global__ void __launch_bounds__(kThreads)
permute_columns_kernel(const T* __restrict__ in, T* __restrict__ out, const int32_t* __restrict__ perm,
                       int n_rows, int d, int rows_per_step) {
    extern __shared__ __align__(16) unsigned char stage_raw[];
    T* stage = reinterpret_cast<T*>(stage_raw);          // [rows_per_step][d]
    constexpr int V = Vec<T>::n;
    const int vec_per_row = d / V;
    for (long long r0 = (long long)blockIdx.x * rows_per_step; r0 < n_rows;
         r0 += (long long)gridDim.x * rows_per_step) {
        const int rows = (int)min((long long)rows_per_step, n_rows - r0);
        const int nvec = rows * vec_per_row;
        const uint4* src = reinterpret_cast<const uint4*>(in + (size_t)r0 * d);
        uint4* dst = reinterpret_cast<uint4*>(out + (size_t)r0 * d);
        if (!INVERSE) {
            for (int v = threadIdx.x; v < nvec; v += kThreads) reinterpret_cast<uint4*>(stage)[v] = __ldg(src + v);
            __syncthreads();
            for (int v = threadIdx.x; v < nvec; v += kThreads) {
                const int r = v / vec_per_row, c0 = (v - r * vec_per_row) * V;
                __align__(16) T tmp[V];
                int src_col[V];
                load_perm<V>(perm + c0, src_col);
#pragma unroll
                for (int i = 0; i < V; ++i) tmp[i] = stage[r * d + src_col[i]];
                dst[v] = *reinterpret_cast<const uint4*>(tmp);
            }
        } else {
            for (int v = threadIdx.x; v < nvec; v += kThreads) {
                const int r = v / vec_per_row, c0 = (v - r * vec_per_row) * V;
                __align__(16) T tmp[V];
                *reinterpret_cast<uint4*>(tmp) = __ldg(src + v);
                int dst_col[V];
                load_perm<V>(perm + c0, dst_col);
#pragma unroll
                for (int i = 0; i < V; ++i) stage[r * d + dst_col[i]] = tmp[i];
            }
            __syncthreads();
            for (int v = threadIdx.x; v < nvec; v += kThreads) dst[v] = reinterpret_cast<const uint4*>(stage)[v];
        }
        __syncthreads();
    }
}

template <typename T>
int launch_typed(const Dims& D, const void* in, void* out, const int32_t* perm, bool inverse, cudaStream_t st) {
    const size_t row_bytes = sizeof(T) * (size_t)D.d;
    if (row_bytes > 200 * 1024) return SLICEMOE_ERR_UNSUPPORTED;
    const int rows_per_step = row_bytes >= (size_t)kStageBytes ? 1 : (int)(kStageBytes / row_bytes);
    const size_t smem = row_bytes * rows_per_step;
    const long long steps = ((long long)D.T + rows_per_step - 1) / rows_per_step;
    const long long cap = 148LL * 8;
    const int grid = (int)(steps < cap ? steps : cap);
    auto launch = [&](auto kern) -> int {
        SLICEMOE_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        kern<<<grid, kThreads, smem, st>>>((const T*)in, (T*)out, perm, D.T, D.d, rows_per_step);
        SLICEMOE_LAUNCH_CHECK(1);
        return SLICEMOE_OK;
    };
    return inverse ? launch(permute_columns_kernel<T, true>) : launch(permute_columns_kernel<T, false>);
}

}  // namespace

int launch_permute_columns(const Dims& D, const void* in, void* out, const int32_t* perm, bool inverse,
                           cudaStream_t st) {
    if (D.T == 0) return SLICEMOE_OK;
    if (D.dtype == SLICEMOE_BF16) return launch_typed<bf16>(D, in, out, perm, inverse, st);
    return launch_typed<float>(D, in, out, perm, inverse, st);
}

}  // namespace slicemoe

extern "C" int slicemoe_permute_columns(const slicemoe_config* cfg, const void* in, void* out,
                                        const int32_t* perm, int inverse, void* stream) {
    using namespace slicemoe;
    Dims D;
    int rc = make_dims(cfg, D);
    if (rc) return rc;
    if (D.T > 0 && (!in || !out)) return SLICEMOE_ERR_NULL;
    if (!perm) return SLICEMOE_ERR_NULL;
    auto misaligned = [](const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; };
    if (misaligned(in) || misaligned(out) || misaligned(perm)) return SLICEMOE_ERR_ALIGN;
    if (D.T > 0) {
        const size_t bytes = elem_bytes(D) * (size_t)D.T * D.d;
        const char* a = static_cast<const char*>(in);
        const char* b = static_cast<const char*>(out);
        if (a < b + bytes && b < a + bytes) return SLICEMOE_ERR_ALIAS;
    }
    if ((rc = check_device())) return rc;
    return launch_permute_columns(D, in, out, perm, inverse != 0, static_cast<cudaStream_t>(stream));
}
