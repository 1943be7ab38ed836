/*
 * ada.h -- C ABI of the B200 (sm_100a) Gram-threshold representative-token
 * selection library (the selection hot path of Cascade ADA).
 *
 * Notation follows the paper: X in R^{T x d} is one layer's activation matrix
 * (row t = token t), Xhat = D^-1 X its row-normalised form (Section 2.1),
 * G = Xhat Xhat^T the cosine Gram, tau in (0,1) the Gram threshold,
 * thr = 1 - tau^2, R^(l) the representative index set of layer l.
 *
 * Conventions shared by every call
 *   - All data pointers are DEVICE pointers unless the function name ends in
 *     `_host`.  `stream` is a cudaStream_t passed as void* (NULL = default
 *     stream).  Device-pointer calls only enqueue work: they never synchronise
 *     and never read a count back to the host, so the outputs of one layer can
 *     feed the next call directly.
 *   - X is row-major, B independent sequences stacked: element (b,t,k) lives at
 *     X[(b*T + t)*ldx + k].  ldx >= d, and X, ldx*es and d*es must be multiples
 *     of 16 bytes (es = 4 for ADA_F32, 2 for ADA_BF16); otherwise
 *     ADA_ERR_UNSUPPORTED.  X is never written.
 *   - Index lists are int32, strictly ascending token indices in [0,T), with a
 *     capacity of T entries per sequence: sequence b uses list + b*T and
 *     count[b].  Counts are int32 on the device.
 *   - The caller owns every buffer it passes.  The library owns only the
 *     context (workspace: inverse norms, gathered representative rows, gamma
 *     scratch, role map, status word).  One context serves one stream at a
 *     time: calls on the same context that overlap on the GPU race on the
 *     workspace.
 *   - Host-checkable faults (bad sizes, NULL required pointers, tau outside
 *     (0,1), misalignment, sizes above the context's maxima) return an error
 *     at once and enqueue nothing.  Device-detected faults (an inherited list
 *     that is not strictly ascending or leaves [0,T), a count outside [0,T],
 *     NaN/Inf in X, an expired bounded wait) set bits in the context's device
 *     status word, leave the call's outputs in bounds but meaningless, and are
 *     reported by ada_device_status.
 *   - The first call that reaches a given kernel on a context performs one-time host-side
 *     set-up (function attributes, an occupancy query); make one call of each kind before
 *     capturing calls into a CUDA graph.  After that the device-pointer calls are plain
 *     stream-ordered launches with no host synchronisation.
 *   - Arithmetic: squared norms and Gram accumulation in fp32.  ADA_BF16
 *     multiplies the stored bf16 values on the tensor cores (products exact in
 *     fp32) and applies 1/(|x_s| |x_t|) in the epilogue; a normalised bf16 copy
 *     of X is never fed to the Gram.  gamma is compared in fp32 with
 *     (float)(1 - tau*tau), strict "<".
 */
#ifndef ADA_H_
#define ADA_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    ADA_OK = 0,
    ADA_ERR_INVALID_ARG = 1,   /* NULL pointer, size < 1, tau outside (0,1), ldx < d        */
    ADA_ERR_UNSUPPORTED = 2,   /* alignment rule broken, dtype differs from the context's   */
    ADA_ERR_WORKSPACE = 3,     /* B, T or d above the maxima given to ada_create            */
    ADA_ERR_CUDA = 4,          /* a CUDA runtime / driver call failed                       */
    ADA_ERR_BAD_INDEX_SET = 5, /* device: inherited list not ascending / out of range       */
    ADA_ERR_NONFINITE = 6,     /* device: NaN or Inf in X                                   */
    ADA_ERR_TIMEOUT = 7,       /* device: a bounded wait inside a kernel expired            */
    ADA_ERR_BAD_TAU = 8        /* device: a threshold state outside (0,1) (adaptive step)   */
} ada_status;

typedef enum { ADA_F32 = 0, ADA_BF16 = 1 } ada_dtype;

/* flags of ada_cascade_step */
#define ADA_CROSS_CAUSAL 1u /* restrict Algorithm 1 line 8 to valid representatives s < t */

/* Which Gram kernel family a context uses.  AUTO: tensor cores (tcgen05), one- or two-CTA
 * form by problem size.  ADA_BF16 feeds the stored values to the MMA; ADA_F32 is split into
 * three bf16 terms per value and contracted as the six leading cross terms (error at fp32
 * rounding level, fp32 accumulation), at the price of a 6x longer contraction and a
 * workspace of 48 bytes per element.  FFMA is the plain fp32 ALU kernel (any storage type;
 * for ADA_BF16 a slow cross-check of the tensor-core path).  TCGEN05 forces the one-CTA
 * kernel (128-row tiles), TCGEN05_PAIR the two-CTA kernel (cta_group::2, 256-row tiles
 * shared by the two SMs of a TPC). */
typedef enum {
    ADA_ENGINE_AUTO = 0,
    ADA_ENGINE_FFMA = 1,
    ADA_ENGINE_TCGEN05 = 2,
    ADA_ENGINE_TCGEN05_PAIR = 3
} ada_engine;

typedef struct ada_ctx ada_ctx; /* opaque */

/* Create a context on `device` able to serve up to maxB sequences of maxT
 * tokens of width maxd in storage type dt.  Allocates the workspace
 * (cudaMalloc; about maxB*maxT*(maxd*es + 32) bytes, plus 48*maxB*maxT*maxd for ADA_F32).
 * maxT may not exceed ADA_MAX_T (the list counts of one sequence are kept in 21-bit fields),
 * nor maxB*maxT 2^30: ADA_ERR_INVALID_ARG.  *out is NULL on error. */
#define ADA_MAX_T ((int64_t)2097151)
ada_status ada_create(ada_ctx** out, int device, int64_t maxB, int64_t maxT, int64_t maxd,
                      ada_dtype dt);
ada_status ada_destroy(ada_ctx* ctx);
ada_status ada_set_engine(ada_ctx* ctx, ada_engine e);
/* The fused cascade launch has CTAs that wait on results of other CTAs of the same grid, so
 * it is launched cooperatively (the driver guarantees that all CTAs are resident, or refuses
 * the launch).  on = 0 launches it as an ordinary grid of one CTA per SM instead: same
 * kernel and results, but if other work keeps some SMs busy for long the in-kernel waits
 * can expire (ADA_ERR_TIMEOUT).  Meant for profilers that cannot replay cooperative
 * launches.  Default: on. */
ada_status ada_set_cooperative(ada_ctx* ctx, int on);

/* Algorithm 1 line 6 forms the cross-Gram from the tokens OUTSIDE the inherited set.  On the
 * pair-CTA kernel, when the inherited set holds two fifths of a sequence's tokens or more, the
 * rows outside it are copied out in token order inside the launch and the cross tiles run over
 * those rows only, instead of streaming all T rows and discarding the inherited ones -- for
 * sequences of at least `min_rows` tokens (default 8192: below that the copy was measured to
 * cost more than the tiles it saves).  Results do not depend on it.  min_rows >= 1;
 * a huge value turns it off. */
ada_status ada_set_row_compaction(ada_ctx* ctx, int64_t min_rows);

/* Programmatic dependent launch of the library's kernels (on by default).  When on, every
 * kernel is launched with the stream-serialization attribute and begins with a grid-dependency
 * wait, so that its blocks can be placed, and its set-up that reads nothing (barriers, TMEM
 * allocation) can run, while the previous kernel of the stream drains; results do not change.
 * It concerns only the order between consecutive kernels of one stream; work from other
 * sources enqueued between two calls is ordered as usual.  Turn it off for tools that cannot
 * follow such launches.  Host-only: ADA_ERR_INVALID_ARG for a NULL context. */
ada_status ada_set_dependent_launch(ada_ctx* ctx, int on);

/*
 * Row normalisation and representative gather (Section 2.1; Algorithm 1
 * lines 1-2).  Each output may be NULL:
 *   inv_norm[B*T]  fp32, 1/||x_t||_2 (0 for a zero row; such rows are counted)
 *   Xhat           same type/shape as X with row stride d: Xhat = D^-1 X
 *   Xrep           if rep_idx/rep_cnt are given: Xrep[(b*T+i)*d + k] =
 *                  X[b, rep_idx[b*T+i], k] for i < rep_cnt[b] (raw rows,
 *                  same type as X, row stride d)
 * One pass over X; rows are read once with 128-bit loads.
 */
ada_status ada_normalize(ada_ctx* ctx, const void* X, int64_t B, int64_t T, int64_t d,
                         int64_t ldx, ada_dtype dt, void* Xhat, float* inv_norm,
                         const int32_t* rep_idx, const int32_t* rep_cnt, void* Xrep,
                         void* stream);

/*
 * Full selection (Definition 1; used at layer 0, Section 4.1):
 *   gamma_t = max_{s<t} |G_st|  (gamma_0 = 0),   R = { t : gamma_t < 1 - tau^2 }.
 * The maximum runs over ALL earlier tokens.  The T x T Gram is never stored:
 * mask, |.|, row maximum and compare are fused into the Gram kernel's epilogue.
 * Outputs: rep_idx (B*T capacity) ascending, rep_cnt[B]; gamma[B*T] optional.
 */
ada_status ada_select_full(ada_ctx* ctx, const void* X, int64_t B, int64_t T, int64_t d,
                           int64_t ldx, ada_dtype dt, double tau, int32_t* rep_idx,
                           int32_t* rep_cnt, float* gamma, void* stream);

/*
 * One cascade step (Algorithm 1, lines 1-11) on X = X^(l+1):
 *   lines 3-5  gamma_rep_i = max_{j<i} |G(rho_i, rho_j)| over ALL inherited
 *              representatives earlier in token order; valid iff < thr
 *   lines 6-9  for every t outside the inherited set,
 *              gamma_cross_t = max_{s in R_valid} |G_ts|; new iff < thr
 *              (ADA_CROSS_CAUSAL: only s < t)
 *   lines 10-11 rep_out = R_valid u R_new (ascending)
 * plus the lists of Eq. (6): add = R_new, rem = R^(l) \ R_valid.
 * rep_in_cnt[b] = 0 is legal (every token is added).  rep_out may not alias
 * rep_in.  Optional outputs, both indexed by token and of size B*T:
 * gamma_rep (0 for tokens outside the inherited set) and gamma_cross (0 for
 * inherited representatives).
 */
ada_status ada_cascade_step(ada_ctx* ctx, const void* X, int64_t B, int64_t T, int64_t d,
                            int64_t ldx, ada_dtype dt, double tau, const int32_t* rep_in,
                            const int32_t* rep_in_cnt, int32_t* rep_out, int32_t* rep_out_cnt,
                            int32_t* add_idx, int32_t* add_cnt, int32_t* rem_idx,
                            int32_t* rem_cnt, float* gamma_rep, float* gamma_cross,
                            uint32_t flags, void* stream);

/*
 * Cascade step with a device-resident, per-sequence threshold that follows the turnover
 * (Section 8.1: tau^(l) set from the turnover rate of Eq. (6), which the cascade step yields as
 * a by-product; a stable set tolerates a tighter threshold, an evolving one needs a looser one).
 * The paper proposes this and gives no formula; the rule built here is a clipped proportional
 * step toward a target turnover, each operation rounded once in fp64, in this order:
 *     rho  = (|add| + |rem|) / |R_in|                        (Eq. 6; undefined for |R_in| = 0)
 *     tau' = min(tau_max, max(tau_min, tau + gain * (target_turnover - rho)))
 * and tau' = clip(tau) when rho is undefined.
 *   tau_state  DEVICE double[B], in/out: sequence b's step uses tau = tau_state[b] (threshold
 *              (float)(1 - tau^2), as for a host-side tau) and, if policy != NULL, leaves tau'
 *              there for the next layer.  Nothing returns to the host between layers.  A value
 *              outside (0,1) or NaN is reported by ada_device_status as ADA_ERR_BAD_TAU.
 *   policy     HOST struct, read during the call; NULL = leave tau_state unchanged (a fixed
 *              per-sequence threshold read from device memory).  ADA_ERR_INVALID_ARG unless
 *              gain >= 0, target_turnover >= 0, 0 < tau_min <= tau_max < 1.
 *   turnover   DEVICE float[B], optional: rho of this step (NaN where undefined).
 * Every other argument, the lists and the error behaviour are those of ada_cascade_step.
 */
typedef struct {
    double target_turnover;
    double gain;
    double tau_min, tau_max;
} ada_tau_policy;

ada_status ada_cascade_step_adaptive(ada_ctx* ctx, const void* X, int64_t B, int64_t T, int64_t d,
                                     int64_t ldx, ada_dtype dt, double* tau_state,
                                     const ada_tau_policy* policy, const int32_t* rep_in,
                                     const int32_t* rep_in_cnt, int32_t* rep_out,
                                     int32_t* rep_out_cnt, int32_t* add_idx, int32_t* add_cnt,
                                     int32_t* rem_idx, int32_t* rem_cnt, float* gamma_rep,
                                     float* gamma_cross, float* turnover, uint32_t flags,
                                     void* stream);

/*
 * Per-head selection (Section 8.5: one representative set per attention head, h separate
 * validations per layer at h * T * r_h * d_h operations).  X is ONE sequence of T tokens whose
 * row holds the h heads side by side: head j of token t is the d_h elements starting at
 * X[t * ldx + j * d_h] (ldx >= h * d_h; d_h * element size a multiple of 16 bytes), the layout
 * a projection writes.  The h heads are h independent problems of width d_h, each computed
 * exactly as ada_select_full / ada_cascade_step compute a sequence, in one launch sequence and
 * without a transposed copy of X.  Every per-sequence array of those calls is per head here:
 * lists and gamma arrays have h * T entries (head j at offset j * T), counts have h.  The
 * context must have been created with maxB >= h, maxT >= T, maxd >= d_h.  Errors, ownership
 * and stream semantics are those of the calls they mirror.
 */
ada_status ada_select_full_heads(ada_ctx* ctx, const void* X, int64_t T, int64_t h, int64_t d_h,
                                 int64_t ldx, ada_dtype dt, double tau, int32_t* rep_idx,
                                 int32_t* rep_cnt, float* gamma, void* stream);
ada_status ada_cascade_step_heads(ada_ctx* ctx, const void* X, int64_t T, int64_t h, int64_t d_h,
                                  int64_t ldx, ada_dtype dt, double tau, const int32_t* rep_in,
                                  const int32_t* rep_in_cnt, int32_t* rep_out,
                                  int32_t* rep_out_cnt, int32_t* add_idx, int32_t* add_cnt,
                                  int32_t* rem_idx, int32_t* rem_cnt, float* gamma_rep,
                                  float* gamma_cross, uint32_t flags, void* stream);

/*
 * Nearest-representative map (Section 2.3: the attention output of a redundant token is
 * taken from the representative s* in R maximising |G_ts*|).  For every token t of X and a
 * representative set R given as an ascending list (e.g. the output of ada_select_full or
 * ada_cascade_step on the same X):
 *   nearest_idx[t] = argmax_{s in R} |G_ts|, the lowest index on ties; a representative maps
 *                    to itself; -1 when R is empty
 *   nearest_gamma[t] (optional) = that maximum |G_ts*| (1 for a representative, 0 for zero rows)
 * One T x r cross-Gram on the tensor cores with an argmax epilogue (both storage types;
 * fp32 through the three-term split), whatever engine the context is set to; the Gram is
 * not stored.  Sizes B*T for both outputs.
 */
ada_status ada_nearest_rep(ada_ctx* ctx, const void* X, int64_t B, int64_t T, int64_t d,
                           int64_t ldx, ada_dtype dt, const int32_t* rep_idx,
                           const int32_t* rep_cnt, int32_t* nearest_idx, float* nearest_gamma,
                           void* stream);

/*
 * Attention on the representative set (Section 2.3, Eq. 2):
 *     Attn_R = softmax(Q_R K_R^T / sqrt(d_h)) V_R        (an r x r problem per head)
 * with Q_R, K_R, V_R the rows of Q, K, V at the representatives, and the expansion stated with
 * it: a token outside R takes the attention output of its nearest representative.
 *   Q, K, V      bf16, ONE sequence of T tokens, h heads side by side in a token's row: head j
 *                of token t starts at X[t * ld + j * d_h] (ld >= h * d_h); d_h a multiple of 16,
 *                at most 128; otherwise ADA_ERR_UNSUPPORTED (also for ADA_F32 contexts/inputs)
 *   rep_idx/cnt  R as an ascending list (device), e.g. the output of a selection call
 *   nearest_idx  optional, T entries (device), e.g. from ada_nearest_rep on the same R: token t
 *                receives out[nearest_idx[t]] (a representative maps to itself; -1 gives zeros).
 *                NULL: only the representatives' rows of `out` are written
 *   out          fp32, T rows of h * d_h with row stride ldo: out[rho_i] = Attn_R row i
 *   flags        0: Eq. 2 as printed, every representative attends to every representative;
 *                ADA_ATTN_CAUSAL: row i only to the representatives at or before it in token
 *                order (the mask a causal language model applies; the paper's equation has none)
 * Both contractions run on the tensor cores (tcgen05, accumulators in TMEM), the probabilities
 * are rounded to bf16 between them, the softmax statistics are fp32.  The gathered copies of
 * Q_R, K_R and V_R^T live in a buffer of the context allocated on the first call (3 x T x h x
 * d_h bf16): make that call before capturing into a CUDA graph.  The context must have been
 * created with maxT >= T and maxd >= h * d_h.  Enqueues on `stream`, never synchronises.
 */
#define ADA_ATTN_CAUSAL 1u
ada_status ada_attention_reps(ada_ctx* ctx, const void* Q, const void* K, const void* V, int64_t T,
                              int64_t h, int64_t d_h, int64_t ld, ada_dtype dt, const int32_t* rep_idx,
                              const int32_t* rep_cnt, const int32_t* nearest_idx, float* out,
                              int64_t ldo, uint32_t flags, void* stream);

/* Same operations with HOST buffers: inputs are copied to the device (staging
 * buffers owned by the context, allocated on first use), the device-pointer
 * call above runs, results are copied back, all on `stream`, and the call
 * returns after synchronising that stream.  Counts are int32[B] on the host.
 * Pinned host memory makes the copies asynchronous DMA transfers.  The context
 * must have been created with maxima covering the sizes. */
ada_status ada_select_full_host(ada_ctx* ctx, const void* X, int64_t B, int64_t T, int64_t d,
                                ada_dtype dt, double tau, int32_t* rep_idx, int32_t* rep_cnt,
                                float* gamma, void* stream);
ada_status ada_cascade_step_host(ada_ctx* ctx, const void* X, int64_t B, int64_t T, int64_t d,
                                 ada_dtype dt, double tau, const int32_t* rep_in,
                                 const int32_t* rep_in_cnt, int32_t* rep_out,
                                 int32_t* rep_out_cnt, int32_t* add_idx, int32_t* add_cnt,
                                 int32_t* rem_idx, int32_t* rem_cnt, float* gamma_rep,
                                 float* gamma_cross, uint32_t flags, void* stream);

/*
 * Full selection for callers that cannot allocate device memory (the paper has no
 * counterpart; this is a deployment variant of ada_select_full for ONE sequence).
 *
 * Who needs it: a process whose device memory was handed in full to its own pool at
 * start-up, a latency-critical loop that cannot take the device-wide synchronisation an
 * allocation implies, a plug-in whose host forbids allocator calls.  None of them can
 * create an ada_ctx, because its workspace is one cudaMalloc.  This call takes no context
 * and performs no cudaMalloc / cudaFree and calls no allocating library routine: its
 * scratch (gamma bit patterns, inverse norms, a few status words; about 128 KiB) is a fixed
 * array inside the library image, present on every GPU that loads the library until the
 * process exits.
 *
 * Arguments as ada_select_full with B = 1: device pointers, X row-major T x d with row
 * stride ldx, rep_idx capacity T, rep_cnt one int32, gamma optional (T floats); the work
 * is enqueued on `stream` for the CURRENT device and the call does not synchronise.
 *   - T above ADA_NOALLOC_MAX_T returns ADA_ERR_WORKSPACE and enqueues nothing.
 *   - The first call on each device also performs a one-time set-up (it looks up the
 *     scratch array's device address and the SM count); make that first call before any
 *     stream capture begins.
 *   - All calls on a device share the one scratch array, and it keeps the previous call's
 *     contents; the call itself clears what must start at zero.  Two calls whose kernels
 *     overlap on the GPU (different streams) race on it: keep them stream-ordered.
 *   - Device-detected faults (NaN/Inf in X, an expired bounded wait) cannot be read back
 *     through a context here; check the inputs upstream if that matters.
 *   - ADA_F32 input runs on the plain fp32 (FFMA) Gram kernel here, ADA_BF16 on the
 *     one-CTA tensor-core kernel.
 *   - The host side is safe to call from several threads (the per-device set-up runs once,
 *     under a guard); the GPU work of concurrent callers must still be stream-ordered.
 */
#define ADA_NOALLOC_MAX_T 16384
ada_status ada_select_full_noalloc(const void* X, int64_t T, int64_t d, int64_t ldx,
                                   ada_dtype dt, double tau, int32_t* rep_idx, int32_t* rep_cnt,
                                   float* gamma, void* stream);

/* Gram operation counts of Eq. (4)/(5), d included: cascade == 0 -> T^2 d;
 * cascade != 0 -> r^2 d + (T - r) r d with r the INHERITED count.  Pure host
 * arithmetic; returns 0 for negative arguments or r > T. */
uint64_t ada_gram_op_count(int cascade, int64_t T, int64_t d, int64_t r);

/* Synchronise `stream`, then report and clear the device status word: returns
 * ADA_OK or the most severe device-detected error since the last call.
 * n_zero_norm_rows (optional, host) receives the number of zero rows seen. */
ada_status ada_device_status(ada_ctx* ctx, void* stream, int64_t* n_zero_norm_rows);

/* Self-test of the bounded-wait machinery: runs a one-warp kernel that waits, with a limit
 * of `limit_ms` milliseconds, on a counter that nothing ever sets -- the same wait the Gram
 * kernels use between CTAs.  The wait runs out, the kernel raises the TIMEOUT bit and returns
 * normally; ada_device_status then reports ADA_ERR_TIMEOUT and the context stays usable.
 * Nothing faults, traps or hangs. */
ada_status ada_selftest_wait_timeout(ada_ctx* ctx, int limit_ms, void* stream);

/* Per-kernel timing (for benchmarks): when enabled, every kernel launch of
 * this context is bracketed by CUDA events on the launching stream.
 * ada_profile_read synchronises those events, fills up to `cap` entries
 * (kernel name, launches, total milliseconds), resets the counters and
 * returns the number of kernels known. */
ada_status ada_profile_enable(ada_ctx* ctx, int on);
int ada_profile_read(ada_ctx* ctx, const char** names, int64_t* launches, double* total_ms,
                     int cap);

const char* ada_status_string(ada_status s);

#ifdef __cplusplus
}
#endif
#endif /* ADA_H_ */
