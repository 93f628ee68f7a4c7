// Backward of the SliceMoE layer (Section 3.1: router and experts are trained end to end with the
// task loss).  Given gout = dL/dh', computes dL/dh and the gradients of all eight weight tensors by
// the chain rule on the forward of Section 3.1 / Eq. 1.  The chosen expert ids are constants of the
// backward; the router learns through Eq. 1's gate x~ = p_e x, p being the softmax over all E
// experts; a pair dropped by the capacity receives nothing.  With dropout_gates the gates are Section 3.3's
// re-normalised survivors and that re-normalisation is differentiated as well; logit noise is redrawn.
//
// CUDA-core kernels, fp32 arithmetic in both storage types, weight gradients always fp32:
//   1. the dispatch of the forward is redone from topk_idx (deterministic: same dest / perm / offsets)
//   2. expert kernel : one CTA per (expert, tile of TM stacked rows); recomputes z and u, then
//        dz = (W2^T dy) * act'(z), dW2 += dy u^T, dW1 += dz (p x)^T, db1, db2, and per pair
//        dxp = p * W1^T dz (its share of dL/dx) and dp = <W1^T dz, x> (gradient of its gate)
//   3. router kernel : one CTA per tile of TR rows; recomputes a and p, turns the dp of the row's kept
//        pairs into logit gradients dg = p (dp - sum p dp) / tau, then dWr2, dbr2, dWr1, dbr1 and
//        dL/dx = Wr1^T dpre + sum_j dxp
// Weight gradients are reduced over the tile in shared memory / registers and added to global memory
// with one fp32 atomic per element and tile, so their summation order (not their value beyond fp32
// rounding) varies from run to run; dL/dh is deterministic.
#include "common.cuh"
#include "philox.cuh"

namespace slicemoe {
namespace {

constexpr int kThreads = 256;
constexpr int kFC = 256;  // hidden units per chunk of the expert kernel

// u = act(z) and du/dz with one tanh between them.
__device__ __forceinline__ void act_and_grad(float z, int act, float& u, float& g) {
    if (act == SLICEMOE_ACT_RELU) { u = fmaxf(z, 0.0f); g = z > 0.0f ? 1.0f : 0.0f; return; }
    const float c = 0.7978845608028654f, b = 0.044715f;
    const float t = tanhf(c * (z + b * z * z * z));
    u = 0.5f * z * (1.0f + t);
    g = 0.5f * (1.0f + t) + 0.5f * z * (1.0f - t * t) * c * (1.0f + 3.0f * b * z * z);
}

// Loads `rows` rows of width ds (row r from src + index[r]*ds) into dst as fp32, optionally scaled per
// row; rows beyond `rows` become zero.
template <typename T, int TM>
__device__ __forceinline__ void load_rows(float* dst, const T* __restrict__ src, const int* row_of,
                                          const float* scale, int rows, int ds) {
    constexpr int V = Vec<T>::n;
    for (int v = threadIdx.x; v < TM * ds / V; v += kThreads) {
        const int r = (v * V) / ds, c = v * V - r * ds;
        float f[V];
        if (r < rows) {
            unpack16<T>(*reinterpret_cast<const uint4*>(src + (size_t)row_of[r] * ds + c), f);
            if (scale) {
                const float s = scale[r];
#pragma unroll
                for (int i = 0; i < V; ++i) f[i] *= s;
            }
        } else {
#pragma unroll
            for (int i = 0; i < V; ++i) f[i] = 0.0f;
        }
#pragma unroll
        for (int i = 0; i < V; ++i) dst[v * V + i] = f[i];
    }
}

// out[f, q] += sum_r A[r, f] * B[r, q] for f < nf, q < nq (A: [TM, lda], B: [TM, ldb] in shared memory,
// fp32; nq and ldb multiples of 4); out is global with row stride ldo.  One atomic per element.  A thread
// owns a 4 x 4 block of `out` when nf and lda are multiples of 4 (two 16-byte shared-memory loads per 16
// multiply-adds; with one row of four the loop is bound by shared-memory bandwidth), else a 1 x 4 block.
template <int TM>
__device__ __forceinline__ void outer_accumulate(float* __restrict__ out, int ldo, const float* A, int lda,
                                                 int nf, const float* B, int ldb, int nq) {
    const int q4n = nq >> 2;
    if (((nf | lda) & 3) == 0) {
        for (int it = threadIdx.x; it < (nf >> 2) * q4n; it += kThreads) {
            const int f = (it / q4n) << 2, q = (it % q4n) << 2;
            float s[4][4];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) s[i][j] = 0.0f;
#pragma unroll 4
            for (int r = 0; r < TM; ++r) {
                const float4 a = *reinterpret_cast<const float4*>(A + r * lda + f);
                const float4 b = *reinterpret_cast<const float4*>(B + r * ldb + q);
                const float av[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    s[i][0] = fmaf(av[i], b.x, s[i][0]); s[i][1] = fmaf(av[i], b.y, s[i][1]);
                    s[i][2] = fmaf(av[i], b.z, s[i][2]); s[i][3] = fmaf(av[i], b.w, s[i][3]);
                }
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                float* o = out + (size_t)(f + i) * ldo + q;
#pragma unroll
                for (int j = 0; j < 4; ++j) atomicAdd(o + j, s[i][j]);
            }
        }
        return;
    }
    for (int it = threadIdx.x; it < nf * q4n; it += kThreads) {
        const int f = it / q4n, q = (it - f * q4n) << 2;
        float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll 8
        for (int r = 0; r < TM; ++r) {
            const float a = A[r * lda + f];
            const float4 b = *reinterpret_cast<const float4*>(B + r * ldb + q);
            s0 = fmaf(a, b.x, s0); s1 = fmaf(a, b.y, s1); s2 = fmaf(a, b.z, s2); s3 = fmaf(a, b.w, s3);
        }
        float* o = out + (size_t)f * ldo + q;
        atomicAdd(o, s0); atomicAdd(o + 1, s1); atomicAdd(o + 2, s2); atomicAdd(o + 3, s3);
    }
}

// value(row, q) = sum_{f < nf} Wt[f*ldw + q] * D[row, f]: the product with the transposed weight, W read
// from global memory (coalesced over q), D [TM, ldd] from shared memory, handed to `sink(row, q, value)`.
// Work items are (group of RPG rows, q); RPG is a compile-time constant so that the row loop carries no
// predicated-off iterations.
template <typename T, int TM, int RPG, typename Sink>
__device__ __forceinline__ void times_w_transposed_rpg(const T* __restrict__ Wt, int ldw, int nf, const float* D,
                                                       int ldd, int nq, Sink sink) {
    constexpr int groups = TM / RPG;
    for (int item = threadIdx.x; item < groups * nq; item += kThreads) {
        const int g = item / nq, q = item - g * nq;
        const float* Dg = D + g * RPG * ldd;
        float acc[RPG];
#pragma unroll
        for (int r = 0; r < RPG; ++r) acc[r] = 0.0f;
        for (int f = 0; f < nf; f += 4) {
            const float w0 = to_f32(Wt[(size_t)f * ldw + q]), w1 = to_f32(Wt[(size_t)(f + 1) * ldw + q]);
            const float w2 = to_f32(Wt[(size_t)(f + 2) * ldw + q]), w3 = to_f32(Wt[(size_t)(f + 3) * ldw + q]);
#pragma unroll
            for (int r = 0; r < RPG; ++r) {
                const float4 dv = *reinterpret_cast<const float4*>(Dg + r * ldd + f);
                acc[r] = fmaf(w0, dv.x, fmaf(w1, dv.y, fmaf(w2, dv.z, fmaf(w3, dv.w, acc[r]))));
            }
        }
#pragma unroll
        for (int r = 0; r < RPG; ++r) sink(g * RPG + r, q, acc[r]);
    }
}

// Picks the rows per group so that groups * nq covers the CTA's threads where it can.
template <typename T, int TM, typename Sink>
__device__ __forceinline__ void times_w_transposed(const T* __restrict__ Wt, int ldw, int nf, const float* D,
                                                   int ldd, int nq, Sink sink) {
    if (nq * 8 <= kThreads && TM >= 8) times_w_transposed_rpg<T, TM, (TM >= 8 ? TM / 8 : 1)>(Wt, ldw, nf, D, ldd, nq, sink);
    else if (nq * 4 <= kThreads && TM >= 4) times_w_transposed_rpg<T, TM, (TM >= 4 ? TM / 4 : 1)>(Wt, ldw, nf, D, ldd, nq, sink);
    else if (nq * 2 <= kThreads) times_w_transposed_rpg<T, TM, TM / 2>(Wt, ldw, nf, D, ldd, nq, sink);
    else times_w_transposed_rpg<T, TM, TM>(Wt, ldw, nf, D, ldd, nq, sink);
}

// ---- expert kernel ------------------------------------------------------------------------------
// Tile = TM stacked rows of one expert (found from `offsets` like the forward's CUDA-core kernel).
// Shared memory: xps = p * x, dys = dy, dxs = accumulated W1^T dz, zs = dz, us = u, per chunk of kFC
// hidden units.  Rows beyond the tile's end are zero and add nothing.
template <typename T, int TM>
__global__ void __launch_bounds__(kThreads)
bwd_expert_kernel(const T* __restrict__ h, const T* __restrict__ gout, const int32_t* __restrict__ offsets,
                  const int32_t* __restrict__ perm, const float* __restrict__ topk_p,
                  const T* __restrict__ W1, const T* __restrict__ b1, const T* __restrict__ W2,
                  float* __restrict__ dW1, float* __restrict__ db1, float* __restrict__ dW2,
                  float* __restrict__ db2, float* __restrict__ dxp, float* __restrict__ dp,
                  int E, int ds, int F, int k, int act) {
    extern __shared__ __align__(16) float smem[];
    float* xps = smem;             // [TM][ds]
    float* dys = xps + TM * ds;    // [TM][ds]
    float* dxs = dys + TM * ds;    // [TM][ds]
    float* zs = dxs + TM * ds;     // [TM][kFC]
    float* us = zs + TM * kFC;     // [TM][kFC]
    __shared__ int tile_info[3];
    __shared__ int row_of[TM];     // row n of X for each tile row
    __shared__ int pair_of[TM];
    __shared__ float ps[TM];
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
    if (tid < TM) {
        const int pair = tid < rows ? perm[row0 + tid] : 0;
        pair_of[tid] = pair;
        row_of[tid] = pair / k;
        ps[tid] = tid < rows ? topk_p[pair] : 0.0f;
    }
    __syncthreads();
    load_rows<T, TM>(xps, h, row_of, ps, rows, ds);
    load_rows<T, TM>(dys, gout, row_of, nullptr, rows, ds);
    for (int i = tid; i < TM * ds; i += kThreads) dxs[i] = 0.0f;
    __syncthreads();

    const T* W1e = W1 + (size_t)e * F * ds;
    const T* W2e = W2 + (size_t)e * ds * F;
    float* dW1e = dW1 + (size_t)e * F * ds;
    float* dW2e = dW2 + (size_t)e * ds * F;
    constexpr int V = Vec<T>::n;

    for (int f0 = 0; f0 < F; f0 += kFC) {
        const int fc = min(kFC, F - f0);
        if (tid < fc) {
            const int f = f0 + tid;
            float acc[TM], du[TM];
#pragma unroll
            for (int r = 0; r < TM; ++r) { acc[r] = 0.0f; du[r] = 0.0f; }
            const T* wrow = W1e + (size_t)f * ds;
            for (int q = 0; q < ds; q += V) {
                float wv[V];
                unpack16<T>(*reinterpret_cast<const uint4*>(wrow + q), wv);
#pragma unroll
                for (int u4 = 0; u4 < V; u4 += 4) {
#pragma unroll
                    for (int r = 0; r < TM; ++r) {
                        const float4 xv = *reinterpret_cast<const float4*>(xps + r * ds + q + u4);
                        acc[r] = fmaf(wv[u4], xv.x, fmaf(wv[u4 + 1], xv.y,
                                 fmaf(wv[u4 + 2], xv.z, fmaf(wv[u4 + 3], xv.w, acc[r]))));
                    }
                }
            }
            for (int q = 0; q < ds; q += 4) {
                const float w0 = to_f32(W2e[(size_t)q * F + f]), w1 = to_f32(W2e[(size_t)(q + 1) * F + f]);
                const float w2 = to_f32(W2e[(size_t)(q + 2) * F + f]), w3 = to_f32(W2e[(size_t)(q + 3) * F + f]);
#pragma unroll
                for (int r = 0; r < TM; ++r) {
                    const float4 gv = *reinterpret_cast<const float4*>(dys + r * ds + q);
                    du[r] = fmaf(w0, gv.x, fmaf(w1, gv.y, fmaf(w2, gv.z, fmaf(w3, gv.w, du[r]))));
                }
            }
            const float b = b1 ? to_f32(b1[(size_t)e * F + f]) : 0.0f;
            float bsum = 0.0f;
#pragma unroll
            for (int r = 0; r < TM; ++r) {
                const float z = acc[r] + b;
                float u, g;
                act_and_grad(z, act, u, g);
                const float dz = du[r] * g;
                us[r * kFC + tid] = u;
                zs[r * kFC + tid] = dz;
                bsum += dz;
            }
            if (db1) atomicAdd(db1 + (size_t)e * F + f, bsum);
        }
        __syncthreads();
        // dx~ += W1^T dz ; dW1 += dz (p x)^T ; dW2 += dy u^T
        times_w_transposed<T, TM>(W1e + (size_t)f0 * ds, ds, fc, zs, kFC, ds,
                                  [&](int row, int q, float v) { dxs[row * ds + q] += v; });
        outer_accumulate<TM>(dW1e + (size_t)f0 * ds, ds, zs, kFC, fc, xps, ds, ds);
        outer_accumulate<TM>(dW2e + f0, F, dys, ds, ds, us, kFC, fc);
        __syncthreads();
    }

    if (db2) {
        for (int q = tid; q < ds; q += kThreads) {
            float s = 0.0f;
            for (int r = 0; r < TM; ++r) s += dys[r * ds + q];
            atomicAdd(db2 + (size_t)e * ds + q, s);
        }
    }
    // per pair: gradient of the gate, <W1^T dz, x>, and the pair's share of dL/dx, p * W1^T dz
    const int warp = tid >> 5, lane = tid & 31;
    for (int r = warp; r < rows; r += kThreads / 32) {
        const T* xrow = h + (size_t)row_of[r] * ds;
        float* out = dxp + (size_t)pair_of[r] * ds;
        const float p = ps[r];
        float s = 0.0f;
        for (int q = lane; q < ds; q += 32) {
            const float v = dxs[r * ds + q];
            s = fmaf(v, to_f32(xrow[q]), s);
            out[q] = p * v;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if (lane == 0) dp[pair_of[r]] = s;
    }
}

// ---- router kernel ------------------------------------------------------------------------------
// Tile = TR consecutive rows.  Shared memory: xs = x [TR][ds], dxs [TR][ds], as = a, later dpre
// [TR][Hr], gs = logits / tau, then p, then dg [TR][Eld], Eld = E | 1:
// the odd row stride keeps the one-thread-per-row softmax off a single shared-memory bank.
template <typename T, int TR>
__global__ void __launch_bounds__(kThreads)
bwd_router_kernel(const T* __restrict__ h, const int32_t* __restrict__ topk_idx, const int32_t* __restrict__ dest,
                  const float* __restrict__ dp, const float* __restrict__ dxp, const float* __restrict__ gates,
                  const T* __restrict__ Wr1, const T* __restrict__ br1, const T* __restrict__ Wr2,
                  const T* __restrict__ br2, float* __restrict__ dWr1, float* __restrict__ dbr1,
                  float* __restrict__ dWr2, float* __restrict__ dbr2, T* __restrict__ dh,
                  int N, int ds, int Hr, int E, int k, float inv_tau, float sigma, uint32_t key0, uint32_t key1) {
    extern __shared__ __align__(16) float smem[];
    float* xs = smem;              // [TR][ds]
    float* dxs = xs + TR * ds;     // [TR][ds]
    const int Hld = Hr + 4;        // row stride of as: rows land on different banks, 16-byte loads stay aligned
    float* as = dxs + TR * ds;     // [TR][Hld]
    float* gs = as + TR * Hld;     // [TR][Eld]
    const int Eld = E | 1;
    __shared__ int row_of[TR];
    const int tid = threadIdx.x;
    const int n0 = blockIdx.x * TR, rows = min(TR, N - n0);
    constexpr int V = Vec<T>::n;
    if (tid < TR) row_of[tid] = n0 + tid;
    __syncthreads();
    load_rows<T, TR>(xs, h, row_of, nullptr, rows, ds);
    __syncthreads();

    // a = relu(Wr1 x + br1)
    for (int i = tid; i < Hr; i += kThreads) {
        float acc[TR];
        const float b = br1 ? to_f32(br1[i]) : 0.0f;
#pragma unroll
        for (int r = 0; r < TR; ++r) acc[r] = b;
        const T* wrow = Wr1 + (size_t)i * ds;
        for (int q = 0; q < ds; q += V) {
            float wv[V];
            unpack16<T>(*reinterpret_cast<const uint4*>(wrow + q), wv);
#pragma unroll
            for (int u4 = 0; u4 < V; u4 += 4) {
#pragma unroll
                for (int r = 0; r < TR; ++r) {
                    const float4 xv = *reinterpret_cast<const float4*>(xs + r * ds + q + u4);
                    acc[r] = fmaf(wv[u4], xv.x, fmaf(wv[u4 + 1], xv.y,
                             fmaf(wv[u4 + 2], xv.z, fmaf(wv[u4 + 3], xv.w, acc[r]))));
                }
            }
        }
#pragma unroll
        for (int r = 0; r < TR; ++r) as[r * Hld + i] = fmaxf(acc[r], 0.0f);
    }
    __syncthreads();
    // logits / tau.  The lanes of a warp take 32 rows of one expert: the weight row is one broadcast
    // load for the warp (with the expert varying over the lanes it was 32 cache lines per load).
    for (int it = tid; it < TR * E; it += kThreads) {
        const int e = it / TR, r = it - e * TR;
        float g = br2 ? to_f32(br2[e]) : 0.0f;
        const T* wrow = Wr2 + (size_t)e * Hr;
        for (int i = 0; i < Hr; i += 4) {
            const float4 av = *reinterpret_cast<const float4*>(as + r * Hld + i);
            g = fmaf(to_f32(wrow[i]), av.x, fmaf(to_f32(wrow[i + 1]), av.y,
                fmaf(to_f32(wrow[i + 2]), av.z, fmaf(to_f32(wrow[i + 3]), av.w, g))));
        }
        // the forward's logit noise (Figure 6) is a constant of the backward, but the probabilities need it
        if (sigma > 0.0f && r < rows) g = fmaf(sigma, logit_noise(n0 + r, e, key0, key1), g);
        gs[r * Eld + e] = g * inv_tau;
    }
    __syncthreads();
    // softmax, then dg_e = p_e (dp_e - sum_m p_m dp_m) / tau with dp nonzero on the kept pairs only
    if (tid < TR) {
        float* g = gs + tid * Eld;
        if (tid < rows) {
            float m = -INFINITY, sum = 0.0f;
            for (int e = 0; e < E; ++e) m = fmaxf(m, g[e]);
            for (int e = 0; e < E; ++e) { g[e] = __expf(g[e] - m); sum += g[e]; }
            const float inv = 1.0f / sum;
            const int n = n0 + tid;
            for (int e = 0; e < E; ++e) g[e] *= inv;   // p
            float s = 0.0f, pd[8];                      // k <= 8; pd[j] = p_j * dL/dp_j
            if (!gates) {                               // Eq. 1: the gate is the probability itself
                for (int j = 0; j < k; ++j) {
                    const bool kept = dest[(size_t)n * k + j] >= 0;
                    pd[j] = kept ? g[topk_idx[(size_t)n * k + j]] * dp[(size_t)n * k + j] : 0.0f;
                    s += pd[j];
                }
            } else {
                // Section 3.3: gate w_j = m_j p_j / Z over the row's chosen experts, m_j = [w_j != 0];
                // dL/dp_j = m_j (dw_j - sum_i w_i dw_i) / Z.  A lone survivor, and the all-dropped rule's
                // constant gate 1, come out as exactly zero.
                float Z = 0.0f, sw = 0.0f, dw[8], gt[8];
                for (int j = 0; j < k; ++j) {
                    gt[j] = gates[(size_t)n * k + j];
                    dw[j] = dest[(size_t)n * k + j] >= 0 ? dp[(size_t)n * k + j] : 0.0f;
                    const int e = topk_idx[(size_t)n * k + j];
                    if (e < 0 || e >= E) gt[j] = 0.0f;              // an id outside [0, E) was never routed
                    if (gt[j] != 0.0f) Z += g[e];
                    sw = fmaf(gt[j], dw[j], sw);
                }
                for (int j = 0; j < k; ++j) {
                    pd[j] = (gt[j] != 0.0f && Z > 0.0f) ? g[topk_idx[(size_t)n * k + j]] * (dw[j] - sw) / Z : 0.0f;
                    s += pd[j];
                }
            }
            for (int e = 0; e < E; ++e) g[e] = -g[e] * s * inv_tau;
            for (int j = 0; j < k; ++j) {
                const int e = topk_idx[(size_t)n * k + j];
                if (e >= 0 && e < E) g[e] += pd[j] * inv_tau;   // ids outside [0, E) were never routed
            }
        } else {
            for (int e = 0; e < E; ++e) g[e] = 0.0f;
        }
    }
    __syncthreads();
    // dbr2 += sum_r dg ; dWr2 += dg a^T
    if (dbr2) {
        for (int e = tid; e < E; e += kThreads) {
            float s = 0.0f;
            for (int r = 0; r < TR; ++r) s += gs[r * Eld + e];
            atomicAdd(dbr2 + e, s);
        }
    }
    outer_accumulate<TR>(dWr2, Hr, gs, Eld, E, as, Hld, Hr);
    __syncthreads();
    // dpre = (Wr2^T dg) * [a > 0], written over a by the thread that owns hidden unit i
    for (int i = tid; i < Hr; i += kThreads) {
        float da[TR];
#pragma unroll
        for (int r = 0; r < TR; ++r) da[r] = 0.0f;
        for (int e = 0; e < E; ++e) {
            const float w = to_f32(Wr2[(size_t)e * Hr + i]);
#pragma unroll
            for (int r = 0; r < TR; ++r) da[r] = fmaf(w, gs[r * Eld + e], da[r]);
        }
        float bsum = 0.0f;
#pragma unroll
        for (int r = 0; r < TR; ++r) {
            const float v = as[r * Hld + i] > 0.0f ? da[r] : 0.0f;
            as[r * Hld + i] = v;
            bsum += v;
        }
        if (dbr1) atomicAdd(dbr1 + i, bsum);
    }
    __syncthreads();
    // dWr1 += dpre x^T ; dL/dx = Wr1^T dpre + the kept pairs' shares from the expert kernel
    outer_accumulate<TR>(dWr1, ds, as, Hld, Hr, xs, ds, ds);
    times_w_transposed<T, TR>(Wr1, ds, Hr, as, Hld, ds, [&](int row, int q, float v) { dxs[row * ds + q] = v; });
    __syncthreads();
    for (int v = tid; v < rows * ds / V; v += kThreads) {
        const int r = (v * V) / ds, c = v * V - r * ds;
        const int n = n0 + r;
        float f[V];
#pragma unroll
        for (int i = 0; i < V; ++i) f[i] = dxs[v * V + i];
        for (int j = 0; j < k; ++j) {
            if (dest[(size_t)n * k + j] < 0) continue;
            const float* src = dxp + ((size_t)n * k + j) * ds + c;
#pragma unroll
            for (int i = 0; i < V; i += 4) {
                const float4 t = *reinterpret_cast<const float4*>(src + i);
                f[i] += t.x; f[i + 1] += t.y; f[i + 2] += t.z; f[i + 3] += t.w;
            }
        }
        *reinterpret_cast<uint4*>(dh + (size_t)n * ds + c) = pack16<T>(f);
    }
}

// ---- host side ----------------------------------------------------------------------------------

constexpr size_t kSmemBudget = 200 * 1024;

size_t expert_smem(int TM, const Dims& D) { return sizeof(float) * (size_t)TM * (3 * (size_t)D.ds + 2 * kFC); }
size_t router_smem(int TR, const Dims& D) { return sizeof(float) * (size_t)TR * (2 * (size_t)D.ds + D.Hr + 4 + (D.E | 1)); }

struct BwdWorkspace {
    size_t kept, offsets, dest, perm, chunk_hist, dp, dxp, total;
};

BwdWorkspace bwd_layout(const Dims& D) {
    BwdWorkspace W;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t at = off; off = (off + (bytes ? bytes : 1) + 255) & ~(size_t)255; return at; };
    const size_t R = (size_t)D.R, E = (size_t)D.E;
    W.kept = take(sizeof(int32_t) * E);
    W.offsets = take(sizeof(int32_t) * (E + 1));
    W.dest = take(sizeof(int32_t) * R);
    W.perm = take(sizeof(int32_t) * R);
    W.chunk_hist = take(sizeof(int32_t) * (size_t)num_chunks(D) * E);
    W.dp = take(sizeof(float) * R);
    W.dxp = take(sizeof(float) * R * D.ds);
    W.total = off;
    return W;
}

int bwd_supported(const Dims& D) {
    if (expert_smem(8, D) > kSmemBudget || router_smem(8, D) > kSmemBudget) return SLICEMOE_ERR_UNSUPPORTED;
    return SLICEMOE_OK;
}

template <typename T, int TM>
int launch_expert(const Dims& D, const slicemoe_weights& w, const slicemoe_grads& g, const void* h, const void* gout,
                  const int32_t* offsets, const int32_t* perm, const float* topk_p, float* dxp, float* dp,
                  cudaStream_t st) {
    const size_t smem = expert_smem(TM, D);
    auto kern = bwd_expert_kernel<T, TM>;
    SLICEMOE_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    const int grid = (D.R + TM - 1) / TM + D.E;
    kern<<<grid, kThreads, smem, st>>>((const T*)h, (const T*)gout, offsets, perm, topk_p, (const T*)w.W1,
                                      (const T*)w.b1, (const T*)w.W2, g.dW1, g.db1, g.dW2, g.db2, dxp, dp, D.E,
                                      D.ds, D.F, D.k, D.act);
    SLICEMOE_LAUNCH_CHECK(1);
    return SLICEMOE_OK;
}

template <typename T, int TR>
int launch_router(const Dims& D, const slicemoe_weights& w, const slicemoe_grads& g, const void* h,
                  const int32_t* topk_idx, const int32_t* dest, const float* dp, const float* dxp,
                  const float* gates, void* dh, cudaStream_t st) {
    const size_t smem = router_smem(TR, D);
    auto kern = bwd_router_kernel<T, TR>;
    SLICEMOE_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    const int grid = (D.N + TR - 1) / TR;
    kern<<<grid, kThreads, smem, st>>>((const T*)h, topk_idx, dest, dp, dxp, gates, (const T*)w.Wr1, (const T*)w.br1,
                                      (const T*)w.Wr2, (const T*)w.br2, g.dWr1, g.dbr1, g.dWr2, g.dbr2, (T*)dh,
                                      D.N, D.ds, D.Hr, D.E, D.k, D.inv_tau, D.noise_sigma, (uint32_t)D.noise_seed,
                                      (uint32_t)(D.noise_seed >> 32));
    SLICEMOE_LAUNCH_CHECK(1);
    return SLICEMOE_OK;
}

template <typename T>
int launch_typed(const Dims& D, const slicemoe_weights& w, const slicemoe_grads& g, const void* h, const void* gout,
                 const int32_t* topk_idx, const float* topk_p, const int32_t* offsets, const int32_t* dest,
                 const int32_t* perm, float* dxp, float* dp, const float* gates, void* dh, cudaStream_t st) {
    int rc;
    if (expert_smem(32, D) <= kSmemBudget)
        rc = launch_expert<T, 32>(D, w, g, h, gout, offsets, perm, topk_p, dxp, dp, st);
    else
        rc = launch_expert<T, 8>(D, w, g, h, gout, offsets, perm, topk_p, dxp, dp, st);
    if (rc) return rc;
    if (router_smem(32, D) <= kSmemBudget) return launch_router<T, 32>(D, w, g, h, topk_idx, dest, dp, dxp, gates, dh, st);
    return launch_router<T, 8>(D, w, g, h, topk_idx, dest, dp, dxp, gates, dh, st);
}

}  // namespace
}  // namespace slicemoe

extern "C" int slicemoe_backward_workspace_bytes(const slicemoe_config* cfg, size_t* bytes) {
    using namespace slicemoe;
    if (!bytes) return SLICEMOE_ERR_NULL;
    Dims D;
    int rc = make_dims(cfg, D);
    if (rc) return rc;
    if ((rc = bwd_supported(D))) return rc;
    *bytes = bwd_layout(D).total;
    return SLICEMOE_OK;
}

extern "C" int slicemoe_backward(const slicemoe_config* cfg, const slicemoe_weights* w, const void* h,
                                 const void* grad_out, const int32_t* topk_idx, const float* topk_p, void* grad_h,
                                 const slicemoe_grads* grads, int accumulate, int dropout_gates, void* ws,
                                 size_t ws_bytes, void* stream) {
    using namespace slicemoe;
    Dims D;
    int rc = make_dims(cfg, D);
    if (rc) return rc;
    if ((rc = bwd_supported(D))) return rc;
    if (!w || !grads) return SLICEMOE_ERR_NULL;
    // an empty batch has no rows to point at
    if (D.N > 0 && (!h || !grad_out || !topk_idx || !topk_p || !grad_h)) return SLICEMOE_ERR_NULL;
    if (!w->Wr1 || !w->Wr2 || !w->W1 || !w->W2) return SLICEMOE_ERR_NULL;
    if (!grads->dWr1 || !grads->dWr2 || !grads->dW1 || !grads->dW2) return SLICEMOE_ERR_NULL;
    const void* aligned[] = {h, grad_out, grad_h, w->Wr1, w->Wr2, w->W1, w->W2, w->br1, w->br2, w->b1,
                             grads->dWr1, grads->dWr2, grads->dW1, grads->dW2};
    for (const void* p : aligned)
        if (reinterpret_cast<uintptr_t>(p) & 15u) return SLICEMOE_ERR_ALIGN;
    const size_t io_bytes = elem_bytes(D) * (size_t)D.T * D.d;
    auto overlaps = [&](const void* a, const void* b) {
        const char *x = static_cast<const char*>(a), *y = static_cast<const char*>(b);
        return x < y + io_bytes && y < x + io_bytes;
    };
    if (overlaps(grad_h, h) || overlaps(grad_h, grad_out)) return SLICEMOE_ERR_ALIAS;
    const BwdWorkspace W = bwd_layout(D);
    if (D.N > 0 && (!ws || ws_bytes < W.total)) return SLICEMOE_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(ws) & 255u) return SLICEMOE_ERR_ALIGN;
    if ((rc = check_device())) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t ds = D.ds, E = D.E, F = D.F, Hr = D.Hr;
    if (!accumulate) {
        SLICEMOE_CUDA_TRY(cudaMemsetAsync(grads->dWr1, 0, sizeof(float) * Hr * ds, st));
        SLICEMOE_CUDA_TRY(cudaMemsetAsync(grads->dWr2, 0, sizeof(float) * E * Hr, st));
        SLICEMOE_CUDA_TRY(cudaMemsetAsync(grads->dW1, 0, sizeof(float) * E * F * ds, st));
        SLICEMOE_CUDA_TRY(cudaMemsetAsync(grads->dW2, 0, sizeof(float) * E * ds * F, st));
        if (grads->dbr1) SLICEMOE_CUDA_TRY(cudaMemsetAsync(grads->dbr1, 0, sizeof(float) * Hr, st));
        if (grads->dbr2) SLICEMOE_CUDA_TRY(cudaMemsetAsync(grads->dbr2, 0, sizeof(float) * E, st));
        if (grads->db1) SLICEMOE_CUDA_TRY(cudaMemsetAsync(grads->db1, 0, sizeof(float) * E * F, st));
        if (grads->db2) SLICEMOE_CUDA_TRY(cudaMemsetAsync(grads->db2, 0, sizeof(float) * E * ds, st));
    }
    if (D.N == 0) return SLICEMOE_OK;
    char* base = static_cast<char*>(ws);
    int32_t* kept = reinterpret_cast<int32_t*>(base + W.kept);
    int32_t* offsets = reinterpret_cast<int32_t*>(base + W.offsets);
    int32_t* dest = reinterpret_cast<int32_t*>(base + W.dest);
    int32_t* perm = reinterpret_cast<int32_t*>(base + W.perm);
    int32_t* chunk_hist = reinterpret_cast<int32_t*>(base + W.chunk_hist);
    float* dp = reinterpret_cast<float*>(base + W.dp);
    float* dxp = reinterpret_cast<float*>(base + W.dxp);
    const float* gates = dropout_gates ? topk_p : nullptr;
    // the forward's grouping, redone from its expert ids (same stable order, same capacity drops)
    if ((rc = launch_dispatch(D, nullptr, topk_idx, topk_p, kept, offsets, dest, perm, nullptr, nullptr, chunk_hist, st)))
        return rc;
    if (D.dtype == SLICEMOE_BF16)
        return launch_typed<bf16>(D, *w, *grads, h, grad_out, topk_idx, topk_p, offsets, dest, perm, dxp, dp, gates, grad_h, st);
    return launch_typed<float>(D, *w, *grads, h, grad_out, topk_idx, topk_p, offsets, dest, perm, dxp, dp, gates, grad_h, st);
}
