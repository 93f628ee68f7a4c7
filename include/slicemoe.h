/*
 * slicemoe.h -- C ABI of the B200 (sm_100a) SliceMoE layer: the forward and its backward.
 *
 * The layer (paper Section 3): a token vector h in R^d is cut into S contiguous
 * slices of ds = d/S elements.  A router MLP shared by all slices
 * (Linear ds->H_r, ReLU, Linear H_r->E) scores each slice, a softmax turns the
 * scores into probabilities and the k most probable experts are chosen per
 * slice (Section 3.1).  Each chosen expert e_j runs its two-layer FFN on the
 * slice scaled by its probability (Eq. 1); slices bound for the same expert
 * are stacked so that an expert works on one contiguous batch (Section 3.4);
 * the k outputs of a slice are summed and written at the slice's own columns
 * of h' (Section 3.1).
 *
 * Rows.  With h row-major [T, d], slice s of token t is the contiguous run of
 * ds elements starting at (t*S + s)*ds.  The library therefore works on the
 * matrix X[N, ds], N = T*S, which is the same memory as h; row n = t*S + s.
 * "Pair" (n, j) is the j-th chosen expert of row n, flat index n*k + j;
 * R = N*k pairs.
 *
 * Conventions for every call below
 *   - All pointers are CUDA DEVICE pointers unless the comment says HOST.
 *     `cfg` and `w` themselves are HOST structs (read during the call).
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default
 *     stream).  Calls only enqueue work on it: no allocation, no host
 *     synchronisation, unless stated.
 *   - The caller owns every buffer, including the workspace `ws`
 *     (slicemoe_workspace_bytes(), 256-byte aligned).  The library allocates no
 *     device memory.  Its device image holds a few KB of words of its own per
 *     GPU, shared by every caller on that GPU: the arrival counters of the
 *     one-launch forwards' grid barriers, two sets of per-expert list counters
 *     that successive launches use alternately, and the table of
 *     slicemoe_dispatch_static.  One-launch forwards are cooperative launches
 *     (every SM holds one CTA), so two of them never run on a GPU at once.
 *     slicemoe_forward_host additionally creates, once per device, two streams
 *     and ten events of its own and serialises callers on a process-wide lock
 *     while they enqueue.
 *   - Tensors are dense row-major, 16-byte aligned, of cfg->dtype
 *     (bf16 or fp32) unless a type is written.  Weights use the nn.Linear
 *     layout [out, in] with `in` contiguous.  Bias pointers may be NULL (= 0).
 *   - With T = 0 the token-sized buffers may be NULL; the per-expert outputs are still written.
 *   - Return value: 0 (SLICEMOE_OK) or a slicemoe_status error; on an error
 *     found by argument checking nothing has been launched.  Nothing throws.
 *   - Routing arithmetic (logits, softmax, top-k) is fp32 in both dtypes; with
 *     bf16 storage the GEMMs take bf16 operands and accumulate in fp32.
 *   - Ties between equal router scores go to the lower expert id; the k
 *     experts of a row are listed most probable first.
 */
#ifndef SLICEMOE_H_
#define SLICEMOE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SLICEMOE_OK = 0,
    SLICEMOE_ERR_NULL = 1,           /* a required pointer is NULL */
    SLICEMOE_ERR_SHAPE = 2,          /* d % S != 0, k > E, k < 1, E < 1, T < 0, sizes overflow int32 ... */
    SLICEMOE_ERR_UNSUPPORTED = 3,    /* shape, dtype or activation outside the built set */
    SLICEMOE_ERR_ALIGN = 4,          /* a tensor pointer is not 16-byte aligned */
    SLICEMOE_ERR_WORKSPACE = 5,      /* ws is NULL or smaller than slicemoe_workspace_bytes() */
    SLICEMOE_ERR_ALIAS = 6,          /* h_out overlaps h */
    SLICEMOE_ERR_CUDA = 7,           /* a CUDA runtime call failed (see slicemoe_last_cuda_error) */
    SLICEMOE_ERR_DEVICE_TIMEOUT = 8, /* a bounded wait inside a kernel ran out (slicemoe_last_status) */
    SLICEMOE_ERR_NO_DEVICE = 9,      /* no usable sm_100 device */
    SLICEMOE_ERR_STATIC_SCRATCH = 10 /* too large for slicemoe_dispatch_static's fixed scratch */
} slicemoe_status;

typedef enum { SLICEMOE_BF16 = 0, SLICEMOE_F32 = 1 } slicemoe_dtype;
typedef enum { SLICEMOE_ACT_RELU = 0, SLICEMOE_ACT_GELU_TANH = 1 } slicemoe_act;

/* Shape of one layer (paper notation).  Limits of the built set:
 * ds = d/S a multiple of 8 (bf16) or 4 (fp32); 1 <= k <= 8; E <= 256;
 * T*S*k < 2^31. */
typedef struct {
    int32_t T;        /* tokens in the batch */
    int32_t d;        /* hidden size */
    int32_t S;        /* slices per token (Section 3) */
    int32_t E;        /* experts */
    int32_t k;        /* experts per slice (Section 3.1) */
    int32_t Hr;       /* router hidden width (256 in the paper, Appendix A) */
    int32_t F;        /* expert FFN hidden width */
    int32_t dtype;    /* slicemoe_dtype: storage type of h, h', weights and stacked rows */
    int32_t act;      /* slicemoe_act: activation between the two expert layers */
    int64_t capacity; /* hard per-expert limit on kept pairs; 0 = unlimited */
    /* Router ablation knobs (Section 5.2 and Appendix B); all-zero = the plain layer. */
    float temperature;   /* softmax temperature tau > 0 (Figure 7); 0 stands for 1 */
    float noise_sigma;   /* std of the Gaussian noise added to the logits before the
                          * softmax (Figure 6); 0 = none */
    uint64_t noise_seed; /* key of the counter-based noise generator (slicemoe_route) */
    /* Train mode of the slicemoe_forward* calls (Section 3.3, cross-slice dropout; Appendix A uses
     * rate 0.2).  train_gates = 0: Eq. 1's gates are the router's probabilities.  train_gates = 1:
     * each of a row's k assignments is dropped with probability dropout_rate, the survivors'
     * probabilities are divided by their sum, and if none survives the top-1 assignment gets weight 1
     * (slicemoe_gate_dropout's rule and generator with seed = dropout_seed, applied between the
     * router and the dispatch); topk_p_opt then returns those gates.  dropout_rate outside [0, 1]:
     * SLICEMOE_ERR_SHAPE.  The staged calls ignore these fields. */
    int32_t train_gates;
    float dropout_rate;
    uint64_t dropout_seed;
} slicemoe_config;

/* Caller-owned weights, dtype = cfg->dtype. */
typedef struct {
    const void *Wr1; /* [Hr, ds]   router layer 1 (Section 3.1) */
    const void *br1; /* [Hr]       or NULL */
    const void *Wr2; /* [E, Hr]    router layer 2 */
    const void *br2; /* [E]        or NULL */
    const void *W1;  /* [E, F, ds] expert layer 1 */
    const void *b1;  /* [E, F]     or NULL */
    const void *W2;  /* [E, ds, F] expert layer 2 */
    const void *b2;  /* [E, ds]    or NULL */
} slicemoe_weights;

/* Bytes of workspace that any call below needs for `cfg` (the maximum over the
 * calls, slicemoe_forward_host's device staging included).  `bytes` is a HOST
 * out-pointer. */
int slicemoe_workspace_bytes(const slicemoe_config *cfg, size_t *bytes);

/*
 * Section 3.1, router: for every row n of X[N, ds]
 *   a = relu(Wr1 x + br1),  g = Wr2 a + br2,  p = softmax(g),
 *   topk_idx[n, :] = the k experts with the largest p (ties: lower id first),
 *   topk_p[n, :]   = their probabilities, descending.
 * out: topk_idx int32 [N, k]; topk_p float [N, k]; assigned int32 [E] =
 *      number of pairs that chose each expert (the counts of Section 3.2);
 *      probs_opt float [N, E] (NULL to skip).
 * With the ablation knobs of cfg (Figures 6 and 7) the softmax and the top-k see
 *   g'[n, e] = (g[n, e] + noise_sigma * eps(n, e)) / tau
 * instead of g.  eps(n, e) is a standard normal drawn per (row, expert) from a
 * counter-based generator, so a call is reproducible and independent of the
 * launch shape: Philox4x32-10 with key = (low, high word of noise_seed) and
 * counter (n, e, 1, 0) gives words x0, x1; u_i = ((x_i >> 8) + 0.5) / 2^24;
 * eps = sqrt(-2 ln u_0) * cos(2 pi u_1) (Box-Muller), evaluated in fp32.
 * temperature < 0, noise_sigma < 0 or a non-finite value: SLICEMOE_ERR_SHAPE.
 * Noisy routing runs on the CUDA-core router whatever the shape.
 */
int slicemoe_route(const slicemoe_config *cfg, const slicemoe_weights *w, const void *h,
                   int32_t *topk_idx, float *topk_p, int32_t *assigned, float *probs_opt,
                   void *ws, size_t ws_bytes, void *stream);

/*
 * Eq. 1 and Section 3.4, dispatch: group the pairs by expert and stack their
 * probability-weighted rows.  Inside an expert, pairs keep ascending (n, j)
 * order (a stable counting sort, so the result is unique and deterministic).
 * With cfg->capacity = C > 0 a pair whose rank inside its expert is >= C is
 * dropped.
 * in : h [T, d]; topk_idx int32 [N, k]; topk_p float [N, k]
 * out: kept int32 [E]      = min(assigned, C) (= assigned when C = 0);
 *      offsets int32 [E+1] = exclusive scan of kept;
 *      dest int32 [N, k]   = offsets[e] + rank, or -1 if dropped;
 *      perm int32 [R]      = perm[dest(n, j)] = n*k + j (first offsets[E] entries are written);
 *      xperm [R, ds]       = xperm[dest(n, j), :] = dtype(topk_p[n, j] * X[n, :])
 *                            (first offsets[E] rows are written; NULL to skip).
 * An expert id outside [0, E) in topk_idx is treated as a dropped pair.
 */
int slicemoe_dispatch(const slicemoe_config *cfg, const void *h, const int32_t *topk_idx,
                      const float *topk_p, int32_t *kept, int32_t *offsets, int32_t *dest,
                      int32_t *perm, void *xperm, void *ws, size_t ws_bytes, void *stream);

/*
 * slicemoe_dispatch for callers that cannot allocate device memory.  (The paper
 * has no counterpart; this is a deployment variant of the call above.)
 *
 * Some hosts of this library may not call cudaMalloc at the point where they
 * need a dispatch: a plugin running inside another runtime's memory arena, a
 * real-time serving loop whose memory was pinned down at start-up, code that
 * runs after the process has handed all free HBM to a caching allocator.  The
 * ordinary call needs a workspace for its per-chunk histogram table; this one
 * keeps that table in a fixed array inside the library's own device image, so
 * the caller passes only inputs and outputs and nothing is allocated or freed,
 * by this call or by anything it calls.
 *
 * Limit: ceil(T*S*k / 2048) * E <= SLICEMOE_STATIC_SCRATCH_INTS (65536 int32 =
 * 256 KiB, held by every GPU that loads the library until the process exits).
 * Larger problems return SLICEMOE_ERR_STATIC_SCRATCH and launch nothing.
 *
 * The first call on each device looks up the array's device address (with that
 * device current); make that first call outside any stream capture.  All calls
 * share the one array, which keeps whatever the last call left in it: every
 * entry a call reads is first written by that same call, so nothing needs
 * clearing, but two calls that overlap on the GPU (different streams, or
 * different threads) race on it -- serialise them.
 *
 * Arguments and results are exactly those of slicemoe_dispatch.
 */
#define SLICEMOE_STATIC_SCRATCH_INTS 65536
int slicemoe_dispatch_static(const slicemoe_config *cfg, const void *h, const int32_t *topk_idx,
                             const float *topk_p, int32_t *kept, int32_t *offsets, int32_t *dest,
                             int32_t *perm, void *xperm, void *stream);

/*
 * Section 3.1 / 3.4, experts: for every expert e and every stacked row r in
 * [offsets[e], offsets[e+1])
 *   yperm[r, :] = W2_e act(W1_e xperm[r, :] + b1_e) + b2_e
 * The row ranges are read from `offsets` on the device (no host sync); rows at
 * or beyond offsets[E] are not touched.
 */
int slicemoe_expert_ffn(const slicemoe_config *cfg, const slicemoe_weights *w, const void *xperm,
                        const int32_t *offsets, void *yperm, void *ws, size_t ws_bytes,
                        void *stream);

/*
 * Section 3.1, combine: Y[n, :] = sum over j with dest[n, j] >= 0 of
 * yperm[dest[n, j], :], added in j order in fp32 and rounded once; a row whose
 * pairs were all dropped becomes zero.  h_out [T, d] is the same memory as
 * Y[N, ds], so every slice lands at its own columns of its token.
 */
int slicemoe_combine(const slicemoe_config *cfg, const void *yperm, const int32_t *dest,
                     void *h_out, void *stream);

/*
 * Section 3.3, cross-slice dropout: turns the router's top-k probabilities into
 * train-mode gates, in place, between slicemoe_route and slicemoe_dispatch.
 * Each of a row's k probabilities is set to zero independently with probability
 * `rate` (Appendix A: 0.2) and the survivors are divided by their sum; if none
 * survives, the top-1 assignment (j = 0) gets weight 1.  Readings of the paper:
 * one Bernoulli draw per assignment; a dropped assignment stays routed, with
 * gate 0 (Eq. 1 with p = 0); rate = 0 still re-normalises.  The draw for
 * assignment j of row n is the first word of Philox4x32-10 with key = seed and
 * counter (n, j, 0, 0); dropped iff word < floor(rate * 2^32) -- reproducible
 * from (seed, n, j) alone.  topk_p: DEVICE float [N, k], k <= 8; 0 <= rate <= 1.
 * The one-launch slicemoe_forward has no train mode; compose the staged calls.
 */
int slicemoe_gate_dropout(const slicemoe_config *cfg, float *topk_p, uint64_t seed, double rate,
                          void *stream);

/*
 * Shuffled slices (Section 5.2, Figure 5): slices are cut from a fixed
 * permutation of the d columns instead of from contiguous runs.
 *   inverse = 0:  out[t, c] = in[t, perm[c]]      (shuffle before the layer)
 *   inverse = 1:  out[t, perm[c]] = in[t, c]      (undo it on the layer's output)
 * so that  permute(0) -> any of the calls above -> permute(1)  is the layer
 * whose slice s of token t holds columns perm[s*ds .. (s+1)*ds - 1] of h and
 * writes its result back to those columns.  in, out: [T, d] of cfg->dtype, not
 * overlapping; perm: DEVICE int32 [d], a permutation of 0..d-1 (not checked:
 * with a repeated entry, inverse = 1 leaves columns of `out` unwritten).
 */
int slicemoe_permute_columns(const slicemoe_config *cfg, const void *in, void *out,
                             const int32_t *perm, int inverse, void *stream);

/*
 * Routing statistics from per-expert counts (such as `assigned` of the forward):
 *   out[0] = L_cap of Eq. 2 = alpha * (std(counts) / mean(counts))^2, with the
 *            population standard deviation (divide by E) -- the paper does not
 *            say which; alpha is the paper's coefficient (0.01 ... 0.2)
 *   out[1] = ELE of Section 4 (Metrics) = -sum_e load_e log load_e / log E,
 *            load_e = counts_e / sum(counts), 0 log 0 = 0; E = 1 gives 1
 * Both are 0 when nothing was routed.  counts: DEVICE int32 [E]; out: DEVICE
 * double [2], 8-byte aligned.  fp64, deterministic; asynchronous on `stream`.
 */
int slicemoe_load_stats(const int32_t *counts, int32_t E, double alpha, double *out, void *stream);

/*
 * The whole layer forward, h [T, d] -> h_out [T, d], equal to
 * route -> dispatch -> expert_ffn -> combine up to rounding, and bit-equal on
 * topk_idx / assigned / kept.  h_out must not overlap h.
 * Optional outputs (NULL to skip): assigned_opt int32 [E], kept_opt int32 [E],
 * topk_idx_opt int32 [N, k], topk_p_opt float [N, k].
 * For bf16 layers with ds in {48, 64, 96, 128, 192, 256}, E in {8, 16, 32, 64}, k <= 2 and
 * hidden widths that are multiples of the chunk width, the whole forward is ONE
 * kernel launch (router, dispatch and expert phases separated by grid-wide
 * barriers, one CTA per SM); other shapes run one kernel per step.  Every wait
 * inside is bounded: a run-out leaves SLICEMOE_ERR_DEVICE_TIMEOUT in the status
 * word (slicemoe_last_status) and the call's outputs undefined.
 * With cfg->train_gates the gates of Eq. 1 are Section 3.3's (see slicemoe_config)
 * and topk_p_opt returns them; the result equals route -> slicemoe_gate_dropout
 * (dropout_seed, dropout_rate) -> dispatch -> expert_ffn -> combine.  64-wide
 * slices keep their single launch in train mode; the other one-launch shapes
 * then run one kernel per step.
 */
int slicemoe_forward(const slicemoe_config *cfg, const slicemoe_weights *w, const void *h,
                     void *h_out, int32_t *assigned_opt, int32_t *kept_opt,
                     int32_t *topk_idx_opt, float *topk_p_opt, void *ws, size_t ws_bytes,
                     void *stream);

/*
 * slicemoe_forward with HOST tokens: h_host and h_out_host are HOST buffers
 * (pinned memory makes the copies asynchronous).  Enqueues the host->device
 * copy of h into the workspace, the forward, and the device->host copy of h'.
 * Weights and the optional outputs stay DEVICE pointers.  The caller
 * synchronises the stream before reading h_out_host.
 * Without a capacity limit, logit noise or train-mode gates, and from 2048 tokens on, the batch is processed in
 * four chunks of tokens whose copies in and out run on two streams that the
 * library creates once per device, so that the two directions of the link are
 * busy at the same time; in stream order the call still behaves as one
 * operation on `stream` (later work on `stream` sees h_out_host complete).
 * Concurrent calls from several host threads are serialised while they enqueue.
 */
int slicemoe_forward_host(const slicemoe_config *cfg, const slicemoe_weights *w,
                          const void *h_host, void *h_out_host, int32_t *assigned_opt,
                          int32_t *kept_opt, void *ws, size_t ws_bytes, void *stream);

/*
 * slicemoe_forward that also records CUDA events at its stage boundaries, for
 * measurement.  `events` is a HOST array of SLICEMOE_N_STAGE_EVENTS
 * cudaEvent_t handles (as void*) created by slicemoe_event_create(): event i is
 * recorded before stage i and event i+1 after it, stages being
 * 0 route, 1 dispatch, 2 expert FFN, 3 combine.  Where the library folds a
 * stage into its neighbour (bf16 with k <= 2: the experts add their outputs
 * straight into h', so stage 3 is empty) the two events are recorded back to
 * back.
 */
#define SLICEMOE_N_STAGE_EVENTS 5
int slicemoe_forward_profiled(const slicemoe_config *cfg, const slicemoe_weights *w, const void *h,
                              void *h_out, int32_t *assigned_opt, int32_t *kept_opt,
                              int32_t *topk_idx_opt, float *topk_p_opt, void *ws, size_t ws_bytes,
                              void *stream, void *const *events);
int slicemoe_event_create(void **event /* HOST out */);
int slicemoe_event_destroy(void *event);
/* Milliseconds between two recorded events; synchronises on `stop`.  `ms` is a HOST out-pointer. */
int slicemoe_event_elapsed_ms(void *start, void *stop, float *ms);

/*
 * Backward of the layer.  Section 3.1 trains router and experts end to end with
 * the task loss; the paper prints no gradient formulas, so this is the chain
 * rule on the forward as declared above: given grad_out = dL/dh' it returns
 * dL/dh and the gradients of all weights.  Readings: the chosen expert ids
 * (topk_idx, as returned by the forward) are constants; the router receives
 * its gradient through Eq. 1's gate p_e x, p being the softmax over all E
 * experts at temperature cfg->temperature; pairs dropped by cfg->capacity
 * receive nothing (the forward's grouping is redone from topk_idx, same
 * order, same drops); the logit noise of cfg->noise_sigma is a constant of the
 * backward and is redrawn identically when the probabilities are recomputed.
 * dropout_gates == 0: topk_p holds the router's own probabilities (Eq. 1).
 * dropout_gates != 0: topk_p holds the train-mode gates that
 * slicemoe_gate_dropout made of them (Section 3.3), w_j = m_j p_j / Z with
 * m_j = [w_j != 0] and Z the surviving probabilities' sum, and that
 * re-normalisation is differentiated too: dL/dp_j = m_j (dL/dw_j -
 * sum_i w_i dL/dw_i) / Z (zero for a lone survivor and for the constant gate
 * 1 of the all-dropped rule).
 *
 * h, grad_out, grad_h: DEVICE [T, d] of cfg->dtype, 16-byte aligned; grad_h
 * overlaps neither of the other two (with T == 0 the data pointers may be NULL).  topk_idx int32 [N, k], topk_p float
 * [N, k]: DEVICE, outputs of the forward on the same h and weights (an id
 * outside [0, E) counts as not routed).
 * Gradients of the weights: DEVICE fp32 whatever cfg->dtype, shaped like the
 * weights, caller-owned; the four bias gradients may be NULL (skipped).  With
 * accumulate == 0 the call first clears them, otherwise it adds to what they
 * hold.  They are summed with fp32 atomics: values agree from run to run to
 * fp32 rounding, not bit for bit; grad_h is deterministic.
 * ws: DEVICE, 256-byte aligned, slicemoe_backward_workspace_bytes(cfg) bytes.
 * fp32 arithmetic on CUDA cores; asynchronous on `stream`; no allocation, no
 * host synchronisation.  Slices too wide for the kernels' shared-memory tiles
 * (about ds > 2000): SLICEMOE_ERR_UNSUPPORTED.
 */
typedef struct {
    float *dWr1; /* [Hr, ds]   */
    float *dbr1; /* [Hr]       or NULL */
    float *dWr2; /* [E, Hr]    */
    float *dbr2; /* [E]        or NULL */
    float *dW1;  /* [E, F, ds] */
    float *db1;  /* [E, F]     or NULL */
    float *dW2;  /* [E, ds, F] */
    float *db2;  /* [E, ds]    or NULL */
} slicemoe_grads;
int slicemoe_backward_workspace_bytes(const slicemoe_config *cfg, size_t *bytes /* HOST out */);
int slicemoe_backward(const slicemoe_config *cfg, const slicemoe_weights *w, const void *h,
                      const void *grad_out, const int32_t *topk_idx, const float *topk_p,
                      void *grad_h, const slicemoe_grads *grads, int accumulate, int dropout_gates,
                      void *ws, size_t ws_bytes, void *stream);

/* Device status word of the last kernels that used `ws` (0 = fine, else a
 * slicemoe_status such as SLICEMOE_ERR_DEVICE_TIMEOUT).  Synchronises `stream`.
 * After a time-out it also puts the device's grid-barrier words, which the
 * aborted launch may have left half-counted, back to zero. */
int slicemoe_last_status(const void *ws, void *stream);

/* Number of kernels this library has launched in this process so far (HOST counter). */
int64_t slicemoe_launch_count(void);

/* Text of the last CUDA runtime error seen by this library on this thread (HOST string). */
const char *slicemoe_last_cuda_error(void);
const char *slicemoe_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* SLICEMOE_H_ */
