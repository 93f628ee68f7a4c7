// Dispatch of Section 3.4 / Eq. 1: a stable counting sort of the (row, j) pairs by expert, with
// the optional hard capacity, followed by the gather of the probability-weighted rows into
// contiguous per-expert tiles.  Three kernels, no host synchronisation, no atomics on the
// positions (ranks come from prefix sums, so the order inside an expert is ascending (n, j) and
// the result is the same on every run).
//
//   1. histogram : per chunk of kDispatchChunk pairs, how many go to each expert
//   2. scan      : per expert, exclusive prefix over chunks; kept = min(total, C); offsets
//   3. scatter   : per chunk, the stable rank of each pair -> dest / perm, then a coalesced
//                  16-byte-vector copy of p * X[n, :] to its destination row
#include <mutex>

#include "common.cuh"
#include "dispatch_body.cuh"

namespace slicemoe {
namespace {

// Histogram table of slicemoe_dispatch_static: lives in the library's device image, so that the
// call needs no workspace.  Host code must not use this name as a pointer; it asks the runtime
// for the device address once per device (static_scratch_address below).
static __device__ __align__(256) int32_t g_static_chunk_hist[SLICEMOE_STATIC_SCRATCH_INTS];

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kPairsPerWarp = kDispatchChunk / kWarps;  // 256
constexpr int kIters = kPairsPerWarp / 32;              // 8

__global__ void __launch_bounds__(kThreads)
dispatch_hist_kernel(const int32_t* __restrict__ topk_idx, int R, int E,
                     int32_t* __restrict__ chunk_hist) {
    extern __shared__ int cnt[];  // [E]
    for (int e = threadIdx.x; e < E; e += kThreads) cnt[e] = 0;
    __syncthreads();
    const int base = blockIdx.x * kDispatchChunk;
    for (int i = threadIdx.x; i < kDispatchChunk; i += kThreads) {
        const int pair = base + i;
        if (pair < R) {
            const int e = topk_idx[pair];
            if (e >= 0 && e < E) atomicAdd(&cnt[e], 1);
        }
    }
    __syncthreads();
    for (int e = threadIdx.x; e < E; e += kThreads) chunk_hist[(size_t)blockIdx.x * E + e] = cnt[e];
}

// One CTA.  Warp w scans experts w, w+32, ... over the chunks; chunk_hist becomes the exclusive
// prefix (the rank of the chunk's first pair inside its expert).
__global__ void __launch_bounds__(1024)
dispatch_scan_kernel(int32_t* __restrict__ chunk_hist, int nchunks, int E, int capacity,
                     int32_t* __restrict__ kept, int32_t* __restrict__ offsets) {
    extern __shared__ int total[];  // [E]
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int e = warp; e < E; e += 32) {
        int carry = 0;
        for (int c0 = 0; c0 < nchunks; c0 += 32) {
            const int c = c0 + lane;
            const int v = c < nchunks ? chunk_hist[(size_t)c * E + e] : 0;
            int incl = v;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int t = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += t;
            }
            if (c < nchunks) chunk_hist[(size_t)c * E + e] = carry + incl - v;
            carry += __shfl_sync(0xffffffffu, incl, 31);
        }
        if (lane == 0) total[e] = carry;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int run = 0;
        for (int e = 0; e < E; ++e) {
            const int kp = (capacity > 0 && total[e] > capacity) ? capacity : total[e];
            kept[e] = kp;
            offsets[e] = run;
            run += kp;
        }
        offsets[E] = run;
    }
}

constexpr int kScatterThreads = 1024;   // 8 ranking warps; 32 warps of independent 16-byte copies keep enough bytes in flight
template <typename T>
__global__ void __launch_bounds__(kScatterThreads)
dispatch_scatter_kernel(const T* __restrict__ X, const int32_t* __restrict__ topk_idx,
                        const float* __restrict__ topk_p, const int32_t* __restrict__ chunk_base,
                        const int32_t* __restrict__ offsets, int R, int E, int k, int ds, int capacity,
                        int32_t* __restrict__ dest, int32_t* __restrict__ perm, T* __restrict__ xperm,
                        float* __restrict__ gate) {
    extern __shared__ int wcnt[];  // [kWarps][E]
    constexpr int V = Vec<T>::n;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int chunk = blockIdx.x;
    const int warp_base = chunk * kDispatchChunk + warp * kPairsPerWarp;
    // (the first kWarps warps rank the chunk's pairs; all warps of the CTA copy the rows)
    const bool ranker = warp < kWarps;
    int* mine = wcnt + (ranker ? warp : 0) * E;

    if (ranker) {
        for (int e = lane; e < E; e += 32) mine[e] = 0;
        __syncwarp();
        // pass A: this warp's count per expert
        for (int it = 0; it < kIters; ++it) {
            const int pair = warp_base + it * 32 + lane;
            if (pair < R) {
                const int e = topk_idx[pair];
                if (e >= 0 && e < E) atomicAdd(&mine[e], 1);
            }
        }
    }
    __syncthreads();
    // exclusive prefix over the warps, seeded with the chunk's base rank
    for (int e = threadIdx.x; e < E; e += kScatterThreads) {
        int run = chunk_base[(size_t)chunk * E + e];
        for (int w = 0; w < kWarps; ++w) {
            const int t = wcnt[w * E + e];
            wcnt[w * E + e] = run;
            run += t;
        }
    }
    __syncthreads();
    // pass B: stable rank of each pair; its destination and gate also go to shared memory for the copy
    int* sd = wcnt + kWarps * E;                                      // [kDispatchChunk] destination row or -1
    float* sp = reinterpret_cast<float*>(sd + kDispatchChunk);        // [kDispatchChunk] gate
    for (int it = 0; ranker && it < kIters; ++it) {
        const int pair = warp_base + it * 32 + lane;
        int e = -1;
        float p = 0.0f;
        if (pair < R) {
            e = topk_idx[pair];
            p = topk_p[pair];
            if (e < 0 || e >= E) e = -1;
        }
        // lanes with the same expert form a group; invalid lanes get private keys
        const int key = e >= 0 ? e : -1 - lane;
        const unsigned grp = __match_any_sync(0xffffffffu, key);
        const int before = __popc(grp & ((1u << lane) - 1u));
        int d = -1;
        if (e >= 0) {
            const int rank = mine[e] + before;
            if (capacity == 0 || rank < capacity) d = offsets[e] + rank;
        }
        __syncwarp();
        if (e >= 0 && before == 0) mine[e] += __popc(grp);
        __syncwarp();
        if (pair < R) {
            dest[pair] = d;
            if (d >= 0) {
                perm[d] = pair;
                if (gate) gate[d] = p;
            }
        }
        sd[warp * kPairsPerWarp + it * 32 + lane] = d;
        sp[warp * kPairsPerWarp + it * 32 + lane] = p;
    }
    if (xperm == nullptr) return;
    __syncthreads();
    // the row copies of the whole chunk as one flat loop over 16-byte pieces: consecutive threads take
    // consecutive pieces of a row, and several independent loads per thread are in flight
    const int vec_per_row = ds / V;
    const int total = kDispatchChunk * vec_per_row;
    const int chunk_pair0 = chunk * kDispatchChunk;
#pragma unroll 4
    for (int v = threadIdx.x; v < total; v += kScatterThreads) {
        const int item = v / vec_per_row, col = v - item * vec_per_row;
        const int d_i = sd[item];
        if (d_i >= 0) {
            const float p_i = sp[item];
            const int n = (chunk_pair0 + item) / k;
            float f[V];
            unpack16<T>(*reinterpret_cast<const uint4*>(X + (size_t)n * ds + (size_t)col * V), f);
#pragma unroll
            for (int i = 0; i < V; ++i) f[i] *= p_i;
            *reinterpret_cast<uint4*>(xperm + (size_t)d_i * ds + (size_t)col * V) = pack16<T>(f);
        }
    }
}


constexpr int kFusedThreads = 512;

__global__ void __launch_bounds__(kFusedThreads)
dispatch_fused_kernel(const int32_t* __restrict__ topk_idx, const float* __restrict__ topk_p,
                      const int32_t* __restrict__ table, int G, int R, int E, int pairs_per_chunk,
                      int capacity, int32_t* __restrict__ assigned, int32_t* __restrict__ kept,
                      int32_t* __restrict__ offsets, int32_t* __restrict__ dest, int32_t* __restrict__ perm,
                      float* __restrict__ gate) {
    extern __shared__ __align__(16) int sm[];
    dispatch_fused_body<kFusedThreads, false>(topk_idx, topk_p, table, G, (int)blockIdx.x, R, E, pairs_per_chunk,
                                              capacity, assigned, kept, offsets, dest, perm, gate, sm);
}

}  // namespace

int launch_dispatch(const Dims& D, const void* h, const int32_t* topk_idx, const float* topk_p,
                    int32_t* kept, int32_t* offsets, int32_t* dest, int32_t* perm, void* xperm,
                    float* gate_opt, int32_t* chunk_hist, cudaStream_t st) {
    const int nchunks = num_chunks(D);
    if (nchunks > 0) {
        dispatch_hist_kernel<<<nchunks, kThreads, sizeof(int) * D.E, st>>>(topk_idx, D.R, D.E, chunk_hist);
        SLICEMOE_LAUNCH_CHECK(1);
    }
    dispatch_scan_kernel<<<1, 1024, sizeof(int) * D.E, st>>>(chunk_hist, nchunks, D.E, D.capacity, kept,
                                                            offsets);
    SLICEMOE_LAUNCH_CHECK(1);
    if (nchunks > 0) {
        const size_t smem = sizeof(int) * kWarps * D.E + (sizeof(int) + sizeof(float)) * kDispatchChunk;
        if (D.dtype == SLICEMOE_BF16)
            dispatch_scatter_kernel<bf16><<<nchunks, kScatterThreads, smem, st>>>(
                (const bf16*)h, topk_idx, topk_p, chunk_hist, offsets, D.R, D.E, D.k, D.ds, D.capacity,
                dest, perm, (bf16*)xperm, gate_opt);
        else
            dispatch_scatter_kernel<float><<<nchunks, kScatterThreads, smem, st>>>(
                (const float*)h, topk_idx, topk_p, chunk_hist, offsets, D.R, D.E, D.k, D.ds, D.capacity,
                dest, perm, (float*)xperm, gate_opt);
        SLICEMOE_LAUNCH_CHECK(1);
    }
    return SLICEMOE_OK;
}

int launch_dispatch_fused(const Dims& D, const int32_t* topk_idx, const float* topk_p, const int32_t* cta_hist,
                          int grid, int rows_per_cta, int32_t* assigned, int32_t* kept, int32_t* offsets,
                          int32_t* dest, int32_t* perm, float* gate, cudaStream_t st) {
    if (grid <= 0) return SLICEMOE_ERR_SHAPE;
    const size_t smem = dispatch_fused_smem_bytes(D.E, grid, kFusedThreads);
    if (smem > 227 * 1024) return SLICEMOE_ERR_UNSUPPORTED;
    if (smem > 48 * 1024)
        SLICEMOE_CUDA_TRY(cudaFuncSetAttribute(dispatch_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    dispatch_fused_kernel<<<grid, kFusedThreads, smem, st>>>(topk_idx, topk_p, cta_hist, grid, D.R, D.E,
                                                            rows_per_cta * D.k, D.capacity, assigned, kept, offsets,
                                                            dest, perm, gate);
    SLICEMOE_LAUNCH_CHECK(1);
    return SLICEMOE_OK;
}

}  // namespace slicemoe

// ---- allocation-free dispatch ------------------------------------------------------------------

namespace slicemoe {
namespace {

constexpr int kMaxDevices = 64;
std::mutex g_scratch_mutex;
int32_t* g_scratch_addr[kMaxDevices] = {};

// Device address of g_static_chunk_hist on the current device, looked up once per device.
int static_scratch_address(int32_t** out) {
    int dev = -1;
    SLICEMOE_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return SLICEMOE_ERR_NO_DEVICE;
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_addr[dev]) {
        void* p = nullptr;
        SLICEMOE_CUDA_TRY(cudaGetSymbolAddress(&p, g_static_chunk_hist));
        if (!p) return SLICEMOE_ERR_CUDA;
        g_scratch_addr[dev] = static_cast<int32_t*>(p);
    }
    *out = g_scratch_addr[dev];
    return SLICEMOE_OK;
}

}  // namespace
}  // namespace slicemoe

extern "C" int slicemoe_dispatch_static(const slicemoe_config* cfg, const void* h,
                                        const int32_t* topk_idx, const float* topk_p, int32_t* kept,
                                        int32_t* offsets, int32_t* dest, int32_t* perm, void* xperm,
                                        void* stream) {
    using namespace slicemoe;
    Dims D;
    int rc = make_dims(cfg, D);
    if (rc) return rc;
    if (!topk_idx || !topk_p || !kept || !offsets || !dest || !perm) return SLICEMOE_ERR_NULL;
    if (xperm && !h) return SLICEMOE_ERR_NULL;
    if ((reinterpret_cast<uintptr_t>(h) & 15u) || (reinterpret_cast<uintptr_t>(xperm) & 15u))
        return SLICEMOE_ERR_ALIGN;
    if ((long long)num_chunks(D) * D.E > SLICEMOE_STATIC_SCRATCH_INTS) return SLICEMOE_ERR_STATIC_SCRATCH;
    if ((rc = check_device())) return rc;
    int32_t* scratch = nullptr;
    if ((rc = static_scratch_address(&scratch))) return rc;
    // The histogram kernel writes every entry of the table that the later kernels read, so the
    // previous call's contents need no clearing.
    return launch_dispatch(D, h, topk_idx, topk_p, kept, offsets, dest, perm, xperm, nullptr, scratch,
                           static_cast<cudaStream_t>(stream));
}
