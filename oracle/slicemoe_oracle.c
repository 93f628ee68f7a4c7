/*
 * fp64 CPU oracle of the SliceMoE layer forward (and its backward).  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the slow, plain statement of what the layer computes, written
 * from the paper's Section 3 / 3.1 / 3.4 and Eq. 1.  It shares no code with
 * the CUDA library and must never be called from the product path: only the
 * tests, the smoke check and the bench's CPU-baseline leg may use it.
 *
 * Everything is row by row, in double precision, in the paper's order:
 *   slice (Section 3)  ->  router MLP + softmax + top-k (Section 3.1)
 *   -> weight the slice by its routing probability (Eq. 1)
 *   -> group by expert (Section 3.4), with an optional hard capacity
 *   -> two-layer expert FFN (Section 3.1)  -> sum the k outputs of a slice
 *   and write it back at the slice's position in h' (Section 3.1).
 *
 * A row is one slice: row n = t*S + s is columns [s*ds, (s+1)*ds) of token t,
 * which in a row-major h[T, d] is simply elements [n*ds, (n+1)*ds).
 *
 * Parallelism: an OpenMP `for` over independent rows only; the capacity walk
 * is serial, so results do not depend on the thread count.
 *
 * Pins (tests/test_oracle_pins.py): brute-force per-slice loop on tiny
 * inputs, a hand-worked example, identity experts, E = 1, zero router,
 * Zipf-bias capacity closed form, reshape (S = 1) equivalence, permutation
 * equivariance, an affine special case and a dense-MLP special case checked
 * against numpy matmul; load statistics against their closed forms; cross-slice
 * dropout (tests/test_dropout.py) against the generator's published known-answer
 * vectors, a pure-Python restatement, and its invariants; router temperature and
 * logit noise (tests/test_router_knobs.py) against the log-odds identities of a
 * softmax, the limits tau -> 0 and infinity, and normality tests of the noise; the backward
 * (tests/test_oracle_backward.py) against finite differences of the forward, reverse-mode
 * differentiation by torch of a separately written forward, and closed forms.
 * No function here is unpinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int32_t T, d, S, E, k, Hr, F;
    int32_t act;       /* 0 = ReLU, 1 = GELU (tanh form) */
    int64_t capacity;  /* 0 = unlimited */
    /* router ablation knobs (Section 5.2, Figure 6; Appendix B, Figure 7); zeros = plain layer */
    double temperature;   /* softmax temperature tau; 0 stands for 1 */
    double noise_sigma;   /* std of the Gaussian noise on the logits; 0 = none */
    uint64_t noise_seed;
} oracle_cfg;

enum { ORACLE_OK = 0, ORACLE_BAD_SHAPE = 1, ORACLE_NO_MEMORY = 2 };

int slicemoe_oracle_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

static int check_cfg(const oracle_cfg *c) {
    if (c->T < 0 || c->d < 1 || c->S < 1 || c->E < 1 || c->k < 1 || c->Hr < 1 || c->F < 1) return ORACLE_BAD_SHAPE;
    if (c->d % c->S != 0) return ORACLE_BAD_SHAPE;
    if (c->k > c->E) return ORACLE_BAD_SHAPE;
    if (c->capacity < 0) return ORACLE_BAD_SHAPE;
    if (!(c->temperature >= 0.0) || !(c->noise_sigma >= 0.0)) return ORACLE_BAD_SHAPE;
    return ORACLE_OK;
}

/* Section 3.1: expert activation.  ReLU, or GELU in its tanh form. */
static double activation(double z, int act) {
    if (act == 0) return z > 0.0 ? z : 0.0;
    const double c = 0.7978845608028654; /* sqrt(2/pi) */
    return 0.5 * z * (1.0 + tanh(c * (z + 0.044715 * z * z * z)));
}

static void philox4x32_10(const uint32_t ctr_in[4], const uint32_t key_in[2], uint32_t out[4]);

/* Figure 6: the standard normal added (times sigma) to logit e of row n.  Readings: one draw per
 * (row, expert); Philox4x32-10 with key = seed and counter (n, e, 1, 0) gives words x0, x1,
 * u_i = ((x_i >> 8) + 0.5) / 2^24 lies strictly inside (0, 1), and Box-Muller turns the pair into
 * eps = sqrt(-2 ln u0) cos(2 pi u1). */
static double logit_noise(uint64_t seed, int64_t n, int e) {
    const uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
    const uint32_t ctr[4] = {(uint32_t)n, (uint32_t)e, 1u, 0u};
    uint32_t x[4];
    philox4x32_10(ctr, key, x);
    const double u0 = ((double)(x[0] >> 8) + 0.5) / 16777216.0;
    const double u1 = ((double)(x[1] >> 8) + 0.5) / 16777216.0;
    return sqrt(-2.0 * log(u0)) * cos(2.0 * 3.14159265358979323846 * u1);
}

/* Section 3.1: router MLP Linear(ds->Hr), ReLU, Linear(Hr->E), then softmax.
 * x[ds] (row n) -> p[E].  a[Hr] is scratch.  With the ablation knobs the softmax sees
 * (g + sigma * eps(n, e)) / tau: noise on the logits before the softmax (Figure 6), softmax
 * temperature tau (Figure 7). */
static void router_probs_row(const oracle_cfg *c, int64_t n, const double *x,
                             const double *Wr1, const double *br1,
                             const double *Wr2, const double *br2,
                             double *a, double *p) {
    const int ds = c->d / c->S;
    const double tau = c->temperature > 0.0 ? c->temperature : 1.0;
    for (int i = 0; i < c->Hr; ++i) {
        double z = br1 ? br1[i] : 0.0;
        for (int q = 0; q < ds; ++q) z += Wr1[(size_t)i * ds + q] * x[q];
        a[i] = z > 0.0 ? z : 0.0;
    }
    double m = -INFINITY;
    for (int e = 0; e < c->E; ++e) {
        double g = br2 ? br2[e] : 0.0;
        for (int i = 0; i < c->Hr; ++i) g += Wr2[(size_t)e * c->Hr + i] * a[i];
        if (c->noise_sigma > 0.0) g += c->noise_sigma * logit_noise(c->noise_seed, n, e);
        g /= tau;
        p[e] = g;
        if (g > m) m = g;
    }
    double sum = 0.0;
    for (int e = 0; e < c->E; ++e) { p[e] = exp(p[e] - m); sum += p[e]; }
    for (int e = 0; e < c->E; ++e) p[e] /= sum;
}

/* Section 3.1: the k most probable experts of one slice, most probable first;
 * equal probabilities go to the lower expert id.  gap = p_(k) - p_(k+1). */
static void topk_row(const oracle_cfg *c, const double *p, int32_t *idx, double *pk, double *gap) {
    for (int j = 0; j < c->k; ++j) {
        int best = -1;
        for (int e = 0; e < c->E; ++e) {
            int taken = 0;
            for (int i = 0; i < j; ++i) taken |= (idx[i] == e);
            if (taken) continue;
            if (best < 0 || p[e] > p[best]) best = e;
        }
        idx[j] = best;
        pk[j] = p[best];
    }
    if (gap) {
        if (c->k == c->E) { *gap = INFINITY; return; }
        double next = -INFINITY;
        for (int e = 0; e < c->E; ++e) {
            int taken = 0;
            for (int i = 0; i < c->k; ++i) taken |= (idx[i] == e);
            if (!taken && p[e] > next) next = p[e];
        }
        *gap = pk[c->k - 1] - next;
    }
}

/* Section 3.1: one expert's two-layer FFN on one (already weighted) slice.
 * xt[ds] -> y[ds]; u[F] is scratch.  W1[E,F,ds], b1[E,F], W2[E,ds,F], b2[E,ds]. */
static void expert_ffn_row(const oracle_cfg *c, int e, const double *xt,
                           const double *W1, const double *b1,
                           const double *W2, const double *b2,
                           double *u, double *y) {
    const int ds = c->d / c->S, F = c->F;
    const double *W1e = W1 + (size_t)e * F * ds;
    const double *W2e = W2 + (size_t)e * ds * F;
    for (int f = 0; f < F; ++f) {
        double z = b1 ? b1[(size_t)e * F + f] : 0.0;
        for (int q = 0; q < ds; ++q) z += W1e[(size_t)f * ds + q] * xt[q];
        u[f] = activation(z, c->act);
    }
    for (int q = 0; q < ds; ++q) {
        double z = b2 ? b2[(size_t)e * ds + q] : 0.0;
        for (int f = 0; f < F; ++f) z += W2e[(size_t)q * F + f] * u[f];
        y[q] = z;
    }
}

/*
 * Route every slice (Section 3.1).
 * in : h[T*d]; Wr1[Hr*ds], br1[Hr] or NULL, Wr2[E*Hr], br2[E] or NULL
 * out: probs[N*E] (or NULL), topk_idx[N*k], topk_p[N*k], gap[N] (or NULL),
 *      assigned[E] = how many (slice, j) pairs chose each expert (Section 3.2's counts).
 */
int slicemoe_oracle_route(const oracle_cfg *c, const double *h,
                          const double *Wr1, const double *br1,
                          const double *Wr2, const double *br2,
                          double *probs, int32_t *topk_idx, double *topk_p,
                          double *gap, int64_t *assigned) {
    int rc = check_cfg(c);
    if (rc) return rc;
    const int ds = c->d / c->S;
    const int64_t N = (int64_t)c->T * c->S;
    int failed = 0;
#pragma omp parallel
    {
        double *a = (double *)malloc(sizeof(double) * (size_t)c->Hr);
        double *p = (double *)malloc(sizeof(double) * (size_t)c->E);
        if (!a || !p) {
#pragma omp atomic write
            failed = 1;
        }
#pragma omp barrier
        if (!failed) {
#pragma omp for schedule(static)
            for (int64_t n = 0; n < N; ++n) {
                router_probs_row(c, n, h + n * ds, Wr1, br1, Wr2, br2, a, p);
                if (probs) memcpy(probs + n * c->E, p, sizeof(double) * (size_t)c->E);
                topk_row(c, p, topk_idx + n * c->k, topk_p + n * c->k, gap ? gap + n : NULL);
            }
        }
        free(a);
        free(p);
    }
    if (failed) return ORACLE_NO_MEMORY;
    if (assigned) {
        for (int e = 0; e < c->E; ++e) assigned[e] = 0;
        for (int64_t i = 0; i < N * c->k; ++i) assigned[topk_idx[i]] += 1;
    }
    return ORACLE_OK;
}

/*
 * Group the routed (slice, j) pairs by expert (Section 3.4), with the hard
 * per-expert capacity of the skewed-routing workload: pairs are ranked inside
 * their expert in ascending (n, j) order; a pair whose rank reaches the
 * capacity is dropped (dest = -1).
 * in : topk_idx[N*k]
 * out: assigned[E], kept[E] = min(assigned, capacity), offsets[E+1] = exclusive
 *      scan of kept, dest[N*k] = offsets[e] + rank or -1, perm[sum kept] =
 *      the flat pair index n*k + j stored at each destination row.
 */
int slicemoe_oracle_dispatch(const oracle_cfg *c, const int32_t *topk_idx,
                             int64_t *assigned, int64_t *kept, int64_t *offsets,
                             int64_t *dest, int64_t *perm) {
    int rc = check_cfg(c);
    if (rc) return rc;
    const int64_t R = (int64_t)c->T * c->S * c->k;
    for (int e = 0; e < c->E; ++e) assigned[e] = 0;
    for (int64_t i = 0; i < R; ++i) {
        if (topk_idx[i] < 0 || topk_idx[i] >= c->E) return ORACLE_BAD_SHAPE;
        assigned[topk_idx[i]] += 1;
    }
    offsets[0] = 0;
    for (int e = 0; e < c->E; ++e) {
        kept[e] = (c->capacity > 0 && assigned[e] > c->capacity) ? c->capacity : assigned[e];
        offsets[e + 1] = offsets[e] + kept[e];
    }
    int64_t *running = (int64_t *)calloc((size_t)c->E, sizeof(int64_t));
    if (!running) return ORACLE_NO_MEMORY;
    for (int64_t i = 0; i < R; ++i) {
        const int e = topk_idx[i];
        const int64_t rank = running[e]++;
        if (c->capacity == 0 || rank < c->capacity) {
            dest[i] = offsets[e] + rank;
            if (perm) perm[dest[i]] = i;
        } else {
            dest[i] = -1;
        }
    }
    free(running);
    return ORACLE_OK;
}

/* Eq. 1: every kept (slice, j) pair contributes the row p_j * x at its
 * destination.  xperm[sum kept, ds]. */
int slicemoe_oracle_weight_slices(const oracle_cfg *c, const double *h,
                                  const double *topk_p, const int64_t *dest,
                                  double *xperm) {
    int rc = check_cfg(c);
    if (rc) return rc;
    const int ds = c->d / c->S;
    const int64_t N = (int64_t)c->T * c->S;
    for (int64_t n = 0; n < N; ++n)
        for (int j = 0; j < c->k; ++j) {
            const int64_t r = dest[n * c->k + j];
            if (r < 0) continue;
            for (int q = 0; q < ds; ++q) xperm[r * ds + q] = topk_p[n * c->k + j] * h[n * ds + q];
        }
    return ORACLE_OK;
}

/* Section 3.1 / 3.4: each expert's FFN over its stacked rows.
 * xperm[Rk, ds], offsets[E+1] -> yperm[Rk, ds]. */
int slicemoe_oracle_expert_ffn(const oracle_cfg *c, const double *xperm, const int64_t *offsets,
                               const double *W1, const double *b1,
                               const double *W2, const double *b2, double *yperm) {
    int rc = check_cfg(c);
    if (rc) return rc;
    const int ds = c->d / c->S;
    int failed = 0;
#pragma omp parallel
    {
        double *u = (double *)malloc(sizeof(double) * (size_t)c->F);
        if (!u) {
#pragma omp atomic write
            failed = 1;
        }
#pragma omp barrier
        if (!failed) {
            for (int e = 0; e < c->E; ++e) {
#pragma omp for schedule(static) nowait
                for (int64_t r = offsets[e]; r < offsets[e + 1]; ++r)
                    expert_ffn_row(c, e, xperm + r * ds, W1, b1, W2, b2, u, yperm + r * ds);
            }
        }
        free(u);
    }
    return failed ? ORACLE_NO_MEMORY : ORACLE_OK;
}

/* Section 3.1: the k expert outputs of a slice are summed (dropped pairs add
 * nothing; a slice with no kept pair becomes zero) and the sum is written at
 * the slice's own columns of h'. */
int slicemoe_oracle_combine(const oracle_cfg *c, const double *yperm, const int64_t *dest,
                            double *h_out) {
    int rc = check_cfg(c);
    if (rc) return rc;
    const int ds = c->d / c->S;
    const int64_t N = (int64_t)c->T * c->S;
    for (int64_t n = 0; n < N; ++n)
        for (int q = 0; q < ds; ++q) {
            double acc = 0.0;
            for (int j = 0; j < c->k; ++j) {
                const int64_t r = dest[n * c->k + j];
                if (r >= 0) acc += yperm[r * ds + q];
            }
            h_out[n * ds + q] = acc;
        }
    return ORACLE_OK;
}

/*
 * The whole layer: the five steps above in order.
 * forced_idx == NULL : experts are the router's own top-k.
 * forced_idx != NULL : the expert ids [N*k] are taken from the caller while the
 *   gate values are still the router's probabilities of those ids; used to
 *   grade outputs where another implementation legitimately resolved a
 *   near-tie differently.
 * Optional outputs may be NULL: probs[N*E], topk_idx[N*k], topk_p[N*k],
 * gap[N], assigned[E], kept[E], offsets[E+1], dest[N*k].
 */
int slicemoe_oracle_forward(const oracle_cfg *c, const double *h,
                            const double *Wr1, const double *br1,
                            const double *Wr2, const double *br2,
                            const double *W1, const double *b1,
                            const double *W2, const double *b2,
                            const int32_t *forced_idx,
                            double *h_out, double *probs_out,
                            int32_t *topk_idx_out, double *topk_p_out, double *gap_out,
                            int64_t *assigned_out, int64_t *kept_out,
                            int64_t *offsets_out, int64_t *dest_out) {
    int rc = check_cfg(c);
    if (rc) return rc;
    const int ds = c->d / c->S;
    const int64_t N = (int64_t)c->T * c->S, R = N * c->k;
    const size_t E = (size_t)c->E;
    double *probs = (double *)malloc(sizeof(double) * (size_t)(N > 0 ? N : 1) * E);
    int32_t *idx = (int32_t *)malloc(sizeof(int32_t) * (size_t)(R > 0 ? R : 1));
    double *pk = (double *)malloc(sizeof(double) * (size_t)(R > 0 ? R : 1));
    int64_t *assigned = (int64_t *)malloc(sizeof(int64_t) * E);
    int64_t *kept = (int64_t *)malloc(sizeof(int64_t) * E);
    int64_t *offsets = (int64_t *)malloc(sizeof(int64_t) * (E + 1));
    int64_t *dest = (int64_t *)malloc(sizeof(int64_t) * (size_t)(R > 0 ? R : 1));
    double *xperm = NULL, *yperm = NULL;
    rc = ORACLE_NO_MEMORY;
    if (!probs || !idx || !pk || !assigned || !kept || !offsets || !dest) goto done;

    rc = slicemoe_oracle_route(c, h, Wr1, br1, Wr2, br2, probs, idx, pk, gap_out, assigned);
    if (rc) goto done;
    if (forced_idx) {
        for (int64_t i = 0; i < R; ++i) {
            if (forced_idx[i] < 0 || forced_idx[i] >= c->E) { rc = ORACLE_BAD_SHAPE; goto done; }
            idx[i] = forced_idx[i];
            pk[i] = probs[(i / c->k) * c->E + forced_idx[i]];
        }
    }
    rc = slicemoe_oracle_dispatch(c, idx, assigned, kept, offsets, dest, NULL);
    if (rc) goto done;
    {
        const size_t rows = (size_t)(offsets[c->E] > 0 ? offsets[c->E] : 1);
        xperm = (double *)malloc(sizeof(double) * rows * (size_t)ds);
        yperm = (double *)malloc(sizeof(double) * rows * (size_t)ds);
        if (!xperm || !yperm) { rc = ORACLE_NO_MEMORY; goto done; }
    }
    rc = slicemoe_oracle_weight_slices(c, h, pk, dest, xperm);
    if (rc) goto done;
    rc = slicemoe_oracle_expert_ffn(c, xperm, offsets, W1, b1, W2, b2, yperm);
    if (rc) goto done;
    rc = slicemoe_oracle_combine(c, yperm, dest, h_out);
    if (rc) goto done;

    if (probs_out) memcpy(probs_out, probs, sizeof(double) * (size_t)N * E);
    if (topk_idx_out) memcpy(topk_idx_out, idx, sizeof(int32_t) * (size_t)R);
    if (topk_p_out) memcpy(topk_p_out, pk, sizeof(double) * (size_t)R);
    if (assigned_out) memcpy(assigned_out, assigned, sizeof(int64_t) * E);
    if (kept_out) memcpy(kept_out, kept, sizeof(int64_t) * E);
    if (offsets_out) memcpy(offsets_out, offsets, sizeof(int64_t) * (E + 1));
    if (dest_out) memcpy(dest_out, dest, sizeof(int64_t) * (size_t)R);
done:
    free(probs); free(idx); free(pk); free(assigned); free(kept); free(offsets); free(dest);
    free(xperm); free(yperm);
    return rc;
}

/*
 * Outputs of a chosen subset of slices, one by one (for full-size workloads
 * where only sampled rows are graded).  For sampled row i: n = rows[i]; its
 * experts are idx[i*k + j]; pair j contributes only if keep[i*k + j] != 0
 * (the caller gets keep from slicemoe_oracle_dispatch on the full routing).
 * Gate values are this oracle's router probabilities of those experts (Eq. 1).
 * out: y[nrows*ds]; p_out[nrows*k] (or NULL).
 */
int slicemoe_oracle_rows(const oracle_cfg *c, const double *h,
                         const double *Wr1, const double *br1,
                         const double *Wr2, const double *br2,
                         const double *W1, const double *b1,
                         const double *W2, const double *b2,
                         int64_t nrows, const int64_t *rows, const int32_t *idx,
                         const int32_t *keep, double *y, double *p_out) {
    int rc = check_cfg(c);
    if (rc) return rc;
    const int ds = c->d / c->S;
    const int64_t N = (int64_t)c->T * c->S;
    for (int64_t i = 0; i < nrows; ++i)
        if (rows[i] < 0 || rows[i] >= N) return ORACLE_BAD_SHAPE;
    for (int64_t i = 0; i < nrows * c->k; ++i)
        if (idx[i] < 0 || idx[i] >= c->E) return ORACLE_BAD_SHAPE;
    int failed = 0;
#pragma omp parallel
    {
        double *a = (double *)malloc(sizeof(double) * (size_t)c->Hr);
        double *p = (double *)malloc(sizeof(double) * (size_t)c->E);
        double *u = (double *)malloc(sizeof(double) * (size_t)c->F);
        double *xt = (double *)malloc(sizeof(double) * (size_t)ds);
        double *yj = (double *)malloc(sizeof(double) * (size_t)ds);
        if (!a || !p || !u || !xt || !yj) {
#pragma omp atomic write
            failed = 1;
        }
#pragma omp barrier
        if (!failed) {
#pragma omp for schedule(dynamic, 16)
            for (int64_t i = 0; i < nrows; ++i) {
                const double *x = h + rows[i] * ds;
                router_probs_row(c, rows[i], x, Wr1, br1, Wr2, br2, a, p);
                for (int q = 0; q < ds; ++q) y[i * ds + q] = 0.0;
                for (int j = 0; j < c->k; ++j) {
                    const int e = idx[i * c->k + j];
                    if (p_out) p_out[i * c->k + j] = p[e];
                    if (!keep[i * c->k + j]) continue;
                    for (int q = 0; q < ds; ++q) xt[q] = p[e] * x[q];
                    expert_ffn_row(c, e, xt, W1, b1, W2, b2, u, yj);
                    for (int q = 0; q < ds; ++q) y[i * ds + q] += yj[q];
                }
            }
        }
        free(a); free(p); free(u); free(xt); free(yj);
    }
    return failed ? ORACLE_NO_MEMORY : ORACLE_OK;
}

/*
 * Balance statistics of the per-expert counts.
 * Eq. 2: L_cap = alpha * (std(counts) / mean(counts))^2 with the population
 * standard deviation.  Section 4 (Metrics): ELE = -sum_e load_e log load_e / log E
 * with load_e the fraction of routed slices on expert e (0 log 0 = 0; E = 1 gives 1).
 */
int slicemoe_oracle_load_stats(const int64_t *counts, int32_t E, double alpha,
                               double *l_cap, double *ele) {
    if (E < 1) return ORACLE_BAD_SHAPE;
    double total = 0.0;
    for (int e = 0; e < E; ++e) total += (double)counts[e];
    if (total <= 0.0) { *l_cap = 0.0; *ele = 0.0; return ORACLE_OK; }
    const double mean = total / E;
    double var = 0.0;
    for (int e = 0; e < E; ++e) var += ((double)counts[e] - mean) * ((double)counts[e] - mean);
    var /= E;
    *l_cap = alpha * var / (mean * mean);
    double ent = 0.0;
    for (int e = 0; e < E; ++e) {
        const double load = (double)counts[e] / total;
        if (load > 0.0) ent -= load * log(load);
    }
    *ele = (E == 1) ? 1.0 : ent / log((double)E);
    return ORACLE_OK;
}

/* ---- Section 3.3, cross-slice dropout (train-mode gates) ------------------------------
 *
 * After top-k, each of a slice's k assignment probabilities is set to zero independently
 * with probability `rate` (Appendix A: rate 0.2, "20% of selected expert assignments per
 * slice dropped"); the survivors are re-normalised to sum to 1.  Readings: the paper's
 * "a fraction of these k probabilities" is taken as one Bernoulli draw per assignment (k is
 * 1..3, so a fixed fraction of k is not an integer); when all k are dropped the top-1
 * assignment keeps weight 1 ("ensuring information flow is maintained"); a dropped
 * assignment stays routed with gate 0 (Eq. 1 with p = 0).
 *
 * The draws come from the counter-based generator Philox4x32-10 (Salmon et al., SC'11):
 * key = the 64-bit seed, counter = (n, j, 0, 0) for assignment j of row n, the first output
 * word u decides: dropped iff u < floor(rate * 2^32).  The CUDA path implements the same
 * generator on its own; the decision is an integer compare, so both sides agree bit for bit.
 */
static void philox4x32_10(const uint32_t ctr_in[4], const uint32_t key_in[2], uint32_t out[4]) {
    uint32_t c0 = ctr_in[0], c1 = ctr_in[1], c2 = ctr_in[2], c3 = ctr_in[3];
    uint32_t k0 = key_in[0], k1 = key_in[1];
    for (int round = 0; round < 10; ++round) {
        const uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        const uint32_t n1 = (uint32_t)p1;
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        const uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

double slicemoe_oracle_logit_noise(uint64_t seed, int64_t n, int32_t e) { return logit_noise(seed, n, e); }

void slicemoe_oracle_philox4x32(const uint32_t *ctr, const uint32_t *key, uint32_t *out) {
    philox4x32_10(ctr, key, out);
}

int slicemoe_oracle_gate_dropout(const double *topk_p /* [N, k] */, int64_t N, int32_t k,
                                 uint64_t seed, double rate, double *p_out /* [N, k] */,
                                 uint8_t *dropped /* [N, k] */) {
    if (N < 0 || k < 1 || !(rate >= 0.0) || rate > 1.0) return ORACLE_BAD_SHAPE;
    const uint64_t threshold = (uint64_t)(rate * 4294967296.0);       /* 2^32 when rate = 1 */
    const uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
    for (int64_t n = 0; n < N; ++n) {
        double kept_sum = 0.0;
        int kept = 0;
        for (int j = 0; j < k; ++j) {
            const uint32_t ctr[4] = {(uint32_t)n, (uint32_t)j, 0u, 0u};
            uint32_t r[4];
            philox4x32_10(ctr, key, r);
            const int drop = (uint64_t)r[0] < threshold;
            dropped[n * k + j] = (uint8_t)drop;
            if (!drop) { kept_sum += topk_p[n * k + j]; ++kept; }
        }
        for (int j = 0; j < k; ++j) {
            if (kept == 0 || !(kept_sum > 0.0)) p_out[n * k + j] = (j == 0) ? 1.0 : 0.0;
            else p_out[n * k + j] = dropped[n * k + j] ? 0.0 : topk_p[n * k + j] / kept_sum;
        }
    }
    return ORACLE_OK;
}

/* ---- Backward of the layer -------------------------------------------------------------
 *
 * Section 3.1 trains router and experts end to end with the task loss, so the layer needs
 * the gradient of a scalar loss L with respect to its input and all its weights, given
 * gout = dL/dh'.  The paper prints no formulas for it; what follows is the chain rule on the
 * forward exactly as stated above.  Readings: the top-k choice is piecewise constant, so it
 * carries no gradient (the chosen ids are constants of the backward); the router learns
 * through Eq. 1's gate, x~ = p_e x, where p is the softmax over ALL E experts (its Jacobian
 * therefore reaches the logits of unchosen experts too); a pair dropped by the capacity
 * contributed nothing forward and receives nothing backward; logit noise is an additive
 * constant.  Without a dropout mask the gates are the plain probabilities; with one, see "Train
 * mode" below.
 *
 * Per row n (x = its slice, a = relu(Wr1 x + br1), p = softmax((Wr2 a + br2) / tau)) and kept
 * pair j with expert e, gate p_e, z = W1_e (p_e x) + b1_e, u = act(z), y = W2_e u + b2_e:
 *   dy = gout[n];  db2_e += dy;  dW2_e += dy u^T;  du = W2_e^T dy;  dz = du * act'(z);
 *   db1_e += dz;  dW1_e += dz (p_e x)^T;  dx~ = W1_e^T dz;  dx += p_e dx~;  dp_e += <dx~, x>.
 * Softmax: s = sum_e p_e dp_e;  dg_e = p_e (dp_e - s) / tau.
 * Router:  dbr2 += dg;  dWr2 += dg a^T;  da = Wr2^T dg;  dpre = da * [a > 0];
 *          dbr1 += dpre;  dWr1 += dpre x^T;  dx += Wr1^T dpre.
 *
 * Train mode (Section 3.3): with `dropped` != NULL ([N*k], 1 = this assignment was dropped by
 * cross-slice dropout) the gates are w_j = m_j p_j / Z, Z = sum_i m_i p_i over the row's k chosen
 * experts (m = 1 - dropped), and the expert input is w_j x.  Then with dw_j = <dx~_j, x>:
 *   dp_j = m_j (dw_j - sum_i w_i dw_i) / Z.
 * A row whose k assignments were all dropped gives its first-listed expert the constant gate 1,
 * which carries no gradient to the router.  A capacity-dropped pair has dw = 0 but its
 * probability still sits in Z.
 *
 * Serial over rows, fp64; every gradient array is overwritten.  Bias gradients may be NULL.
 * forced_idx as in slicemoe_oracle_forward.
 * Pins (tests/test_oracle_backward.py): central finite differences of the (separately pinned)
 * forward, reverse-mode differentiation by torch of an independently written fp64 forward,
 * and closed forms (E = 1, identity experts, softmax-Jacobian invariants, dropped pairs).
 */
static double activation_grad(double z, int act) {
    if (act == 0) return z > 0.0 ? 1.0 : 0.0;
    const double c = 0.7978845608028654, b = 0.044715;
    const double t = tanh(c * (z + b * z * z * z));
    return 0.5 * (1.0 + t) + 0.5 * z * (1.0 - t * t) * c * (1.0 + 3.0 * b * z * z);
}

int slicemoe_oracle_backward(const oracle_cfg *c, const double *h,
                             const double *Wr1, const double *br1,
                             const double *Wr2, const double *br2,
                             const double *W1, const double *b1,
                             const double *W2, const double *b2,
                             const int32_t *forced_idx, const uint8_t *dropped, const double *gout,
                             double *dh, double *dWr1, double *dbr1, double *dWr2, double *dbr2,
                             double *dW1, double *db1, double *dW2, double *db2) {
    int rc = check_cfg(c);
    if (rc) return rc;
    const int ds = c->d / c->S, E = c->E, Hr = c->Hr, F = c->F, k = c->k;
    const int64_t N = (int64_t)c->T * c->S, R = N * k;
    const double tau = c->temperature > 0.0 ? c->temperature : 1.0;
    if (k > 64) return ORACLE_BAD_SHAPE;
    (void)b2; /* the output bias does not enter any gradient */
    int32_t *idx = (int32_t *)malloc(sizeof(int32_t) * (size_t)(R > 0 ? R : 1));
    double *pk = (double *)malloc(sizeof(double) * (size_t)(R > 0 ? R : 1));
    int64_t *dest = (int64_t *)malloc(sizeof(int64_t) * (size_t)(R > 0 ? R : 1));
    int64_t *cnt = (int64_t *)malloc(sizeof(int64_t) * (size_t)(3 * E + 1));
    double *a = (double *)malloc(sizeof(double) * (size_t)Hr);
    double *p = (double *)malloc(sizeof(double) * (size_t)E);
    double *dp = (double *)malloc(sizeof(double) * (size_t)E);
    double *z = (double *)malloc(sizeof(double) * (size_t)F);
    double *dz = (double *)malloc(sizeof(double) * (size_t)F);
    double *dx = (double *)malloc(sizeof(double) * (size_t)ds);
    rc = ORACLE_NO_MEMORY;
    if (!idx || !pk || !dest || !cnt || !a || !p || !dp || !z || !dz || !dx) goto done;

    /* the forward's routing and capacity decisions */
    if (forced_idx) {
        for (int64_t i = 0; i < R; ++i) {
            if (forced_idx[i] < 0 || forced_idx[i] >= E) { rc = ORACLE_BAD_SHAPE; goto done; }
            idx[i] = forced_idx[i];
        }
    } else {
        rc = slicemoe_oracle_route(c, h, Wr1, br1, Wr2, br2, NULL, idx, pk, NULL, NULL);
        if (rc) goto done;
    }
    rc = slicemoe_oracle_dispatch(c, idx, cnt, cnt + E, cnt + 2 * E, dest, NULL);
    if (rc) goto done;

    memset(dWr1, 0, sizeof(double) * (size_t)Hr * ds);
    memset(dWr2, 0, sizeof(double) * (size_t)E * Hr);
    memset(dW1, 0, sizeof(double) * (size_t)E * F * ds);
    memset(dW2, 0, sizeof(double) * (size_t)E * ds * F);
    if (dbr1) memset(dbr1, 0, sizeof(double) * (size_t)Hr);
    if (dbr2) memset(dbr2, 0, sizeof(double) * (size_t)E);
    if (db1) memset(db1, 0, sizeof(double) * (size_t)E * F);
    if (db2) memset(db2, 0, sizeof(double) * (size_t)E * ds);

    for (int64_t n = 0; n < N; ++n) {
        const double *x = h + n * ds, *dy = gout + n * ds;
        router_probs_row(c, n, x, Wr1, br1, Wr2, br2, a, p);
        for (int q = 0; q < ds; ++q) dx[q] = 0.0;
        for (int e = 0; e < E; ++e) dp[e] = 0.0;
        /* gates: the plain probabilities (Eq. 1) or the re-normalised survivors (Section 3.3) */
        double gate[64], dgate[64], Z = 0.0;
        int survivors = 0;
        for (int j = 0; j < k; ++j) {
            dgate[j] = 0.0;
            gate[j] = p[idx[n * k + j]];
            if (dropped && !dropped[n * k + j]) { Z += gate[j]; ++survivors; }
        }
        if (dropped)
            for (int j = 0; j < k; ++j)
                gate[j] = survivors ? (dropped[n * k + j] ? 0.0 : gate[j] / Z) : (j == 0 ? 1.0 : 0.0);
        for (int j = 0; j < k; ++j) {
            if (dest[n * k + j] < 0) continue;
            const int e = idx[n * k + j];
            const double pe = gate[j];
            const double *W1e = W1 + (size_t)e * F * ds, *W2e = W2 + (size_t)e * ds * F;
            double *dW1e = dW1 + (size_t)e * F * ds, *dW2e = dW2 + (size_t)e * ds * F;
            for (int f = 0; f < F; ++f) {
                double v = b1 ? b1[(size_t)e * F + f] : 0.0;
                for (int q = 0; q < ds; ++q) v += W1e[(size_t)f * ds + q] * (pe * x[q]);
                z[f] = v;
            }
            for (int f = 0; f < F; ++f) {
                const double u = activation(z[f], c->act);
                double du = 0.0;
                for (int q = 0; q < ds; ++q) {
                    du += W2e[(size_t)q * F + f] * dy[q];
                    dW2e[(size_t)q * F + f] += dy[q] * u;
                }
                dz[f] = du * activation_grad(z[f], c->act);
                if (db1) db1[(size_t)e * F + f] += dz[f];
            }
            if (db2) for (int q = 0; q < ds; ++q) db2[(size_t)e * ds + q] += dy[q];
            for (int q = 0; q < ds; ++q) {
                double dxt = 0.0;
                for (int f = 0; f < F; ++f) {
                    dxt += W1e[(size_t)f * ds + q] * dz[f];
                    dW1e[(size_t)f * ds + q] += dz[f] * (pe * x[q]);
                }
                dx[q] += pe * dxt;
                dgate[j] += dxt * x[q];
            }
        }
        if (!dropped) {
            for (int j = 0; j < k; ++j) dp[idx[n * k + j]] += dgate[j];
        } else if (survivors) {
            double sw = 0.0;
            for (int j = 0; j < k; ++j) sw += gate[j] * dgate[j];
            for (int j = 0; j < k; ++j)
                if (!dropped[n * k + j]) dp[idx[n * k + j]] += (dgate[j] - sw) / Z;
        }
        double s = 0.0;
        for (int e = 0; e < E; ++e) s += p[e] * dp[e];
        for (int e = 0; e < E; ++e) dp[e] = p[e] * (dp[e] - s) / tau; /* dp now holds dg */
        for (int e = 0; e < E; ++e) {
            if (dbr2) dbr2[e] += dp[e];
            for (int i = 0; i < Hr; ++i) dWr2[(size_t)e * Hr + i] += dp[e] * a[i];
        }
        for (int i = 0; i < Hr; ++i) {
            double da = 0.0;
            for (int e = 0; e < E; ++e) da += Wr2[(size_t)e * Hr + i] * dp[e];
            const double dpre = a[i] > 0.0 ? da : 0.0;
            if (dbr1) dbr1[i] += dpre;
            for (int q = 0; q < ds; ++q) {
                dWr1[(size_t)i * ds + q] += dpre * x[q];
                dx[q] += Wr1[(size_t)i * ds + q] * dpre;
            }
        }
        for (int q = 0; q < ds; ++q) dh[n * ds + q] = dx[q];
    }
    rc = ORACLE_OK;
done:
    free(idx); free(pk); free(dest); free(cnt); free(a); free(p); free(dp); free(z); free(dz); free(dx);
    return rc;
}
