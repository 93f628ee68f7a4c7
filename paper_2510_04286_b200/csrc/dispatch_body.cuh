// Fused dispatch (ranking of the routed pairs), as a device function shared by the stand-alone
// kernel and by the dispatch phase of the single-kernel forward.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace slicemoe {

// Fused dispatch for the forward call.  Chunk c is the row range that CTA c of the tensor-core
// router handled; `table[c][e]` is how many pairs of that chunk chose expert e (written by the
// router).  Every CTA derives from the table (G x E, a few KB) the rank of its chunk's first pair
// inside each expert, the totals, kept = min(total, C) and the offsets -- redundantly, which is
// cheaper than a separate scan launch -- and then ranks its own pairs in stable (n, j) order.
// The chunk is taken in segments of kSegPairs pairs: a segment's expert ids and probabilities are
// brought into shared memory with all loads in flight at once (the ranking loop itself is a chain
// of dependent warp votes and would otherwise pay the memory latency once per 32 pairs), then
// counted per warp, prefixed over warps, and ranked with match-any inside the warp.
// offs_out (shared memory, E + 1 ints, or NULL) receives a copy of the offsets.
// NT threads take part (the whole CTA: the body synchronises with __syncthreads); `sm` is 16-byte
// aligned shared memory of dispatch_fused_smem_bytes(E, G, NT) bytes.  SAME_LAUNCH: the router phase
// of the same launch wrote topk_idx / topk_p / table, so they are not read through the
// non-coherent path.
constexpr int kSegPairs = 8192;

__host__ __device__ inline size_t dispatch_fused_smem_bytes(int E, int G, int nthreads) {
    return sizeof(int) * (2 * (size_t)kSegPairs + (size_t)E * (nthreads / 32 + 3 + G) + 1);
}

template <int NT, bool SAME_LAUNCH>
__device__ __forceinline__ void dispatch_fused_body(
    const int32_t* __restrict__ topk_idx, const float* __restrict__ topk_p, const int32_t* __restrict__ table,
    int G, int chunk, int R, int E, int pairs_per_chunk, int capacity, int32_t* __restrict__ assigned,
    int32_t* __restrict__ kept, int32_t* __restrict__ offsets, int32_t* __restrict__ dest,
    int32_t* __restrict__ perm, float* __restrict__ gate, int* sm, int* offs_out = nullptr) {
    constexpr int kFusedThreads = NT, kFusedWarps = NT / 32;
    int* seg_e = sm;                               // [kSegPairs]  (16-byte aligned: first)
    float* seg_p = reinterpret_cast<float*>(seg_e + kSegPairs);   // [kSegPairs]
    int* base = seg_e + 2 * kSegPairs;             // [E]   rank of the next segment's first pair inside each expert
    int* total = base + E;                         // [E]
    int* offs = total + E;                         // [E+1]
    int* wcnt = offs + E + 1;                      // [kFusedWarps][E]
    int* tab = wcnt + kFusedWarps * E;             // [G][E] copy of the table
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long chunk_begin = (long long)chunk * pairs_per_chunk;
    long long chunk_end = chunk_begin + pairs_per_chunk;
    if (chunk_end > R) chunk_end = R;

    // Segment loader.  chunk_begin and kSegPairs are multiples of 4, both arrays 16-byte aligned.
    auto load_segment = [&](long long seg_begin, int n) {
        const int nvec = n >> 2;
        const int4* gi = reinterpret_cast<const int4*>(topk_idx + seg_begin);
        const float4* gp = reinterpret_cast<const float4*>(topk_p + seg_begin);
#pragma unroll 4
        for (int v = threadIdx.x; v < nvec; v += kFusedThreads) {
            reinterpret_cast<int4*>(seg_e)[v] = SAME_LAUNCH ? __ldcg(gi + v) : __ldg(gi + v);
            reinterpret_cast<float4*>(seg_p)[v] = SAME_LAUNCH ? __ldcg(gp + v) : __ldg(gp + v);
        }
        for (int i = (nvec << 2) + threadIdx.x; i < n; i += kFusedThreads) {
            seg_e[i] = SAME_LAUNCH ? __ldcg(topk_idx + seg_begin + i) : topk_idx[seg_begin + i];
            seg_p[i] = SAME_LAUNCH ? __ldcg(topk_p + seg_begin + i) : topk_p[seg_begin + i];
        }
    };
    // the first segment's loads go out before the table work
    const bool has_pairs = chunk_begin < chunk_end;
    if (has_pairs) load_segment(chunk_begin, (int)min((long long)kSegPairs, chunk_end - chunk_begin));

    for (int i = threadIdx.x; i < G * E; i += kFusedThreads) tab[i] = SAME_LAUNCH ? __ldcg(table + i) : table[i];   // coalesced
    for (int e = threadIdx.x; e < 2 * E; e += kFusedThreads) base[e] = 0;        // base and total
    __syncthreads();
    {
        // thread (part, e) sums the table rows c = part, part + parts, ... of expert e
        const int parts = kFusedThreads / E > 0 ? kFusedThreads / E : 1;
        for (int idx = threadIdx.x; idx < parts * E; idx += kFusedThreads) {
            const int e = idx % E, part = idx / E;
            int before = 0, tot = 0;
            for (int c = part; c < G; c += parts) {
                const int v = tab[c * E + e];
                if (c < chunk) before += v;
                tot += v;
            }
            if (before) atomicAdd(&base[e], before);
            if (tot) atomicAdd(&total[e], tot);
        }
    }
    __syncthreads();
    if (warp == 0) {
        // kept = min(total, C) and its exclusive scan over the experts
        int run = 0;
        for (int e0 = 0; e0 < E; e0 += 32) {
            const int e = e0 + lane;
            const int tot = e < E ? total[e] : 0;
            const int kp = (capacity > 0 && tot > capacity) ? capacity : tot;
            int incl = kp;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const int up = __shfl_up_sync(0xffffffffu, incl, d);
                if (lane >= d) incl += up;
            }
            if (e < E) {
                offs[e] = run + incl - kp;
                if (chunk == 0) {
                    if (assigned) assigned[e] = tot;
                    kept[e] = kp;
                    offsets[e] = run + incl - kp;
                }
            }
            run += __shfl_sync(0xffffffffu, incl, 31);
        }
        if (lane == 0) {
            offs[E] = run;
            if (chunk == 0) offsets[E] = run;
        }
    }
    __syncthreads();
    // (single-kernel forward: every CTA keeps the offsets it has just derived for its expert pass)
    if (offs_out)
        for (int e = threadIdx.x; e <= E; e += kFusedThreads) offs_out[e] = offs[e];
    if (!has_pairs) return;

    int* mine = wcnt + warp * E;
    for (long long seg_begin = chunk_begin; seg_begin < chunk_end; seg_begin += kSegPairs) {
        const int n = (int)min((long long)kSegPairs, chunk_end - seg_begin);
        if (seg_begin != chunk_begin) {
            __syncthreads();             // everyone is done with the previous segment's staging
            load_segment(seg_begin, n);
        }
        for (int e = lane; e < E; e += 32) mine[e] = 0;
        __syncthreads();
        const int per_warp = ((n + kFusedWarps - 1) / kFusedWarps + 31) / 32 * 32;   // multiple of 32
        const int w_begin = warp * per_warp;
        const int w_end = min(n, w_begin + per_warp);
        for (int i = w_begin + lane; i < w_end; i += 32) {
            const int e = seg_e[i];
            if (e >= 0 && e < E) atomicAdd(&mine[e], 1);
        }
        __syncthreads();
        for (int e = threadIdx.x; e < E; e += kFusedThreads) {
            int run = base[e];
            for (int w = 0; w < kFusedWarps; ++w) {
                const int t = wcnt[w * E + e];
                wcnt[w * E + e] = run;
                run += t;
            }
            base[e] = run;               // rank of the next segment's first pair
        }
        __syncthreads();
        for (int i0 = w_begin; i0 < w_end; i0 += 32) {
            const int i = i0 + lane;
            int e = -1;
            float p = 0.0f;
            if (i < w_end) {
                e = seg_e[i];
                p = seg_p[i];
                if (e < 0 || e >= E) e = -1;
            }
            const int key = e >= 0 ? e : -1 - lane;
            const unsigned grp = __match_any_sync(0xffffffffu, key);
            const int before = __popc(grp & ((1u << lane) - 1u));
            int d = -1;
            if (e >= 0) {
                const int rank = mine[e] + before;
                if (capacity == 0 || rank < capacity) d = offs[e] + rank;
            }
            __syncwarp();
            if (e >= 0 && before == 0) mine[e] += __popc(grp);
            __syncwarp();
            if (i < w_end) {
                const long long pair = seg_begin + i;
                dest[pair] = d;
                if (d >= 0) {
                    perm[d] = (int)pair;
                    gate[d] = p;
                }
            }
        }
    }
}


}  // namespace slicemoe
