/*
 * cs.h -- C boundary of the compressed-sensing-guided sparse FFN step for NVIDIA B200 (sm_100a).
 *
 * One transformer SwiGLU FFN layer is executed as the paper's control loop (Sec. 5):
 *   sensor    y = S n                 a random sketch of the layer's input          (cs_sketch)
 *   estimator z <- H_k(z + mu Phi^T (y - Phi z)), T times; support = supp(z)         (cs_recover)
 *   actuator  out = sum over the k recovered channel groups of the SwiGLU FFN        (cs_ffn_exec)
 * cs_layer_step runs the three for a batch of decode tokens with independent supports;
 * cs_prompt_support / cs_ffn_exec_shared are the prompt-level variant (Sec. 4) in which one
 * support is recovered from the mean prompt sketch and shared by every token of the prompt.
 *
 * Conventions that hold for every call unless a comment says otherwise
 *   - Every data pointer is a DEVICE pointer owned by the caller; the library neither frees nor
 *     keeps it after the call's work has run.  cs_config / cs_layer structs are HOST memory and
 *     are read before the call returns.
 *   - Calls only enqueue work on `stream` (a cudaStream_t passed as void*, NULL = default
 *     stream) and return without synchronising.  A plan must not be used from two streams at
 *     once: its scratch is shared by all calls.
 *   - Matrices are dense row-major.  "f32" is IEEE binary32; "bf16" is bfloat16.
 *   - Errors are return codes.  Arguments are validated on the host before anything is
 *     launched; on any code other than CS_OK nothing was enqueued.  There is no CPU fallback:
 *     a shape outside the supported set returns CS_ERR_UNSUPPORTED.
 *   - Supported shapes: group in {64, 128}; d_ff = G * group with G <= 128; m <= 64;
 *     1 <= k <= G; d a multiple of 64 and d <= 8192; 1 <= B <= max_tokens.
 */
#ifndef CS_H_
#define CS_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    CS_OK = 0,
    CS_ERR_NULL = 1,        /* a required pointer is NULL */
    CS_ERR_SHAPE = 2,       /* sizes inconsistent with the plan (B > max_tokens, n <= 0, ...) */
    CS_ERR_UNSUPPORTED = 3, /* valid request outside the supported shapes / dtypes */
    CS_ERR_SUPPORT = 4,     /* device check: a support row is not ascending, distinct and in [0,G) */
    CS_ERR_NONFINITE = 5,   /* host check: mu or rms_eps is not finite / not positive; device check: a
                               recovery met a NaN or infinite iterate (its outputs are valid indices, NaN values) */
    CS_ERR_CUDA = 6,        /* a CUDA runtime call failed; see cs_last_cuda_error */
    CS_ERR_TIMEOUT = 7      /* device check: a bounded wait inside a kernel gave up */
} cs_status;

typedef enum { CS_F32 = 0, CS_BF16 = 1 } cs_dtype;

/* Shape of one FFN layer and of the recovery problem; fixed for the life of a plan. */
typedef struct {
    int32_t d;          /* hidden size */
    int32_t d_ff;       /* SwiGLU intermediate size = G * group */
    int32_t group;      /* channels per structured unit ("feed-forward subblock", Sec. 3) */
    int32_t m;          /* sketch rows (measurement budget m_t, Sec. 3) */
    int32_t k;          /* active groups per token (sparsity level k_t, Sec. 9) */
    int32_t T;          /* iterations of the projected iteration (Sec. 8); T = 0 is allowed */
    int32_t w_dtype;    /* cs_dtype of W_gate / W_up / Wd_t */
    int32_t max_tokens; /* largest B (and largest prompt length n) any call will pass */
    float rms_eps;      /* epsilon of the optional RMSNorm */
} cs_config;

/* Parameters of one layer (device pointers, caller-owned). */
typedef struct {
    const float *S;         /* [m, d]    f32  sketch matrix S = Phi * A, precomputed by the caller */
    const float *Phi;       /* [m, G]    f32  measurement matrix of the recovery problem */
    const void *W_gate;     /* [d_ff, d] w_dtype */
    const void *W_up;       /* [d_ff, d] w_dtype */
    const void *Wd_t;       /* [d_ff, d] w_dtype, W_down TRANSPOSED: row c is column c of W_down */
    const float *rms_gamma; /* [d] f32 RMSNorm gain, or NULL for no normalisation */
    float mu;               /* step size of the iteration; 1/||Phi||_2^2 keeps the residual monotone */
    int32_t add_residual;   /* cs_layer_step: x_out = x + FFN(n) when non-zero, else FFN(n) */
} cs_layer;

typedef struct cs_plan cs_plan; /* opaque; owns only device scratch sized from cs_config */

/* Validates the configuration and allocates the plan's device scratch on the current device
 * (the only allocation the library ever makes).  *plan is written only on CS_OK. */
cs_status cs_plan_create(const cs_config *cfg, cs_plan **plan);
/* Frees the scratch.  The caller must have synchronised every stream that used the plan. */
cs_status cs_plan_destroy(cs_plan *plan);

/*
 * Sensor (Sec. 8, z_t = A_t u_t):  y[t, r] = sum_i S[r, i] * h[t, i].
 *   S [m,d] f32, h [B,d] f32  ->  y [B,m] f32.  h and y must not overlap.
 */
cs_status cs_sketch(cs_plan *plan, const float *S, const float *h, int32_t B, float *y, void *stream);

/*
 * Estimator (Sec. 7 projection onto the feasible supports, run as the fixed-iteration projected
 * method of Sec. 8).  For each token independently, from z = 0, T times:
 *     v = z + mu * Phi^T (y - Phi z);   z = H_k(v)
 * where H_k keeps the k entries first in the order (|v| descending, group index ascending) and
 * zeroes the rest.  Always returns exactly k indices (T = 0 gives 0..k-1 and z = 0).
 *   Phi [m,G] f32, y [B,m] f32  ->  support [B,k] int32 ascending, z [B,k] f32 (z at those
 *   indices), resid [B] f32 = ||y - Phi z_T||_2 (resid may be NULL; z may be NULL).
 */
cs_status cs_recover(cs_plan *plan, const float *Phi, float mu, const float *y, int32_t B,
                     int32_t *support, float *z, float *resid, void *stream);

/*
 * Warm-started estimator (Sec. 5: the support may be updated incrementally from the previous
 * decoding step; Sec. 8 lists a warm start from the previous token among the cheap solvers; Sec. 11,
 * incremental recovery under slow support drift).  The same iteration as cs_recover, T times, but
 * from the k-sparse iterate z_0 with z_0[support0[t, j]] = z0[t, j] and zero elsewhere, e.g. the
 * previous token's result, so that fewer iterations than the plan's T are needed when the support
 * drifts slowly.  T >= 1 is this call's iteration count (the plan's is not used).
 *   support0 [B,k] int32 ascending, distinct, in [0,G) (checked on the device, CS_ERR_SUPPORT through
 *   cs_last_device_status), z0 [B,k] f32; other arguments and outputs as cs_recover.  The outputs may
 *   alias the warm-start inputs.
 */
cs_status cs_recover_warm(cs_plan *plan, const float *Phi, float mu, const float *y, int32_t B, int32_t T,
                          const int32_t *support0, const float *z0, int32_t *support, float *z, float *resid,
                          void *stream);

/*
 * Support drift between consecutive decoding steps (Sec. 11, incremental recovery):
 *     drift[t] = |S_t symmetric-difference S_{t-1}|
 * for the supports of the previous and the current step, the quantity a caller watches to decide
 * how many iterations (cs_recover_warm) or measurements the next step gets.
 *   support_prev, support_cur [B,k] int32, ascending and distinct as cs_recover returns them
 *   (checked on the device, CS_ERR_SUPPORT through cs_last_device_status)  ->  drift [B] int32,
 *   even, between 0 and 2k.
 */
cs_status cs_support_drift(cs_plan *plan, const int32_t *support_prev, const int32_t *support_cur, int32_t B,
                           int32_t *drift, void *stream);

/*
 * Normalised support drift between consecutive decoding steps (Sec. 15 metric suite):
 *     D[t] = |S_t symmetric-difference S_{t-1}| / |S_t union S_{t-1}|,
 * 0 for identical supports, 1 for disjoint ones.  Arguments as cs_support_drift; `delta` (the count of
 * cs_support_drift) and `D` may each be NULL.
 */
cs_status cs_support_drift_ratio(cs_plan *plan, const int32_t *support_prev, const int32_t *support_cur, int32_t B,
                                 int32_t *delta, float *D, void *stream);

/*
 * Options of one estimation / one step (cs_recover_ex, cs_layer_step_ex).  A zero-filled struct with
 * T = -1 asks for exactly what cs_recover / cs_layer_step do.  HOST memory, read before the call returns;
 * the pointers inside are DEVICE pointers.
 */
typedef enum {
    CS_SOLVER_IHT = 0,   /* fixed step mu (cs_recover) */
    CS_SOLVER_NIHT = 1,  /* the step of every iteration chosen from the current support S:
                            mu_t = ||g_S||^2 / ||Phi g_S||^2, g = Phi^T (y - Phi z)  (Sec. 8: a projected method with
                            a small fixed number of iterations; no line search follows the step).  `mu` is only
                            the fallback when the denominator vanishes. */
    CS_SOLVER_OMP = 2    /* orthogonal matching pursuit over the feasible supports, any k of the G groups (Sec. 8;
                            Sec. 9 incoherence proposition): k picks by normalised correlation with the residual
                            (ties: lowest index), each followed by the least-squares refit.  Needs k <= 64. */
} cs_solver;

typedef struct {
    int32_t solver;              /* cs_solver */
    int32_t T;                   /* iterations of CS_SOLVER_IHT / NIHT for this call; < 0: the plan's */
    const int32_t *support_prev; /* [B,k] supports of the previous decoding step (ascending, distinct), or NULL */
    const float *z_prev;         /* [B,k] its coefficients (needed with support_prev unless only drift is asked) */
    int32_t warm_start;          /* CS_SOLVER_IHT: start from (support_prev, z_prev) instead of 0 (Sec. 8 warm start) */
    float gamma;                 /* CS_SOLVER_IHT: weight of the temporal regulariser gamma ||z - z_prev||^2 (Sec. 5);
                                    the step becomes  v = z + mu (Phi^T (y - Phi z) - 2 gamma (z - z_prev)).  0: none */
    int32_t reuse_support;       /* cs_layer_step_ex: skip sensing and recovery and execute on support_prev
                                    (Sec. 5: "updated every step, every few steps, or event-triggered") */
    const uint32_t *srht_sign;   /* cs_layer_step_ex: sense with the subsampled randomized Hadamard operator */
    const int32_t *srht_rows;    /*   (cs_sketch_srht) instead of layer->S; both NULL: the dense sketch */
    int32_t *delta_out;          /* [B] |S_t symmetric-difference S_{t-1}| against support_prev, or NULL */
    float *drift_out;            /* [B] the normalised drift D_t, or NULL */
} cs_step_options;

/* The estimator with options: solver, iteration count, warm start, temporal term.  Outputs as cs_recover. */
cs_status cs_recover_ex(cs_plan *plan, const float *Phi, float mu, const float *y, int32_t B,
                        const cs_step_options *opt, int32_t *support, float *z, float *resid, void *stream);

/*
 * Structured sensor (Sec. 8: "subsampled randomized Hadamard operators when implementation efficiency is
 * important"):  y[t, r] = (1/sqrt(m)) sum_i H[rows[r], i] s_i h[t, i],  H[a, i] = (-1)^popcount(a & i), s_i = -1
 * where bit i of sign_bits is set (bit i of word i / 32), else +1.  The fast transform costs d log2 d additions
 * and reads d / 8 + 4 m bytes of operator instead of the 4 m d bytes of a dense S.
 *   sign_bits [d/32] uint32, rows [m] int32 distinct in [0, d), h [B,d] f32 -> y [B,m] f32.
 * d must be a power of two between 256 and 8192 (CS_ERR_UNSUPPORTED otherwise).  The recovery that follows
 * uses Phi = (this operator) * Psi, which the caller precomputes as it precomputes S = Phi * A for the dense one.
 */
cs_status cs_sketch_srht(cs_plan *plan, const uint32_t *sign_bits, const int32_t *rows, const float *h, int32_t B,
                         float *y, void *stream);

/*
 * Uncertainty-driven sensing controller (Sec. 8.1): per token, the predictive entropy of the
 * previous decoding step's distribution over the vocabulary and the measurement budget for the
 * current step,
 *     p = softmax(logits[t, :]),  H = -sum_v p_v log p_v  (natural logarithm, 0 log 0 = 0),
 *     m_t = clip(floor(m_base * (1 + gamma * H)), m_min, m_max).
 *   logits [B,V] f32 (entries of -inf count as p = 0)  ->  m_t [B] int32, H [B] f32 (H may be NULL).
 * The entropy is accumulated in f32 and the floor taken in double precision from it; a row whose
 * entropy is NaN (a NaN or +inf logit) gets m_max.  The budget selects how many rows of the
 * measurement bank the next cs_sketch / cs_recover use: S [m_max,d] and Phi [m_max,G] are row-major,
 * so their first m_t rows are the operands of a plan created with m = m_t (with the step mu of that
 * row prefix); the caller reads m_t back with the sampled token and picks the plan.
 * Uses the plan's scratch: order it on the stream of the plan's other calls.  1 <= m_min <= m_max,
 * m_base > 0, gamma >= 0, B <= max_tokens (else CS_ERR_SHAPE / CS_ERR_NONFINITE).
 */
cs_status cs_uds_budget(cs_plan *plan, const float *logits, int32_t B, int32_t V, float m_base, float gamma,
                        int32_t m_min, int32_t m_max, float *H, int32_t *m_t, void *stream);

/*
 * Actuator (Sec. 3, execution only on the support), per token t with support s_t:
 *   a[c]   = silu(W_gate[c,:] . h_t) * (W_up[c,:] . h_t)     for every channel c of a group in s_t
 *   out[t] = (residual ? residual[t] : 0) + sum_c a[c] * Wd_t[c, :]
 * silu(x) = x / (1 + exp(-x)).  Products accumulate in f32.
 *   h [B,d] f32 (the FFN input, already normalised), support [B,k] int32 ascending, distinct,
 *   in [0,G); residual [B,d] f32 or NULL; out [B,d] f32.  out may alias residual, not h.
 * layer->S, Phi, rms_gamma, mu and add_residual are ignored.  Small batches run as a gather GEMV
 * that streams each token's active rows once; large batches bucket tokens by group and run the
 * active blocks on the tensor cores; f32 activations enter those GEMMs as two bf16 parts (value and
 * remainder), which keeps the result at f32-level accuracy.
 */
cs_status cs_ffn_exec(cs_plan *plan, const cs_layer *layer, const float *h, const int32_t *support,
                      int32_t B, const float *residual, float *out, void *stream);

/*
 * Dispatch step between estimator and actuator (Sec. 7: the estimator's output selects which
 * precompiled execution path runs, here which tokens each group's weight block serves): inverts
 * token -> groups into group -> tokens.
 *   support [B,k] int32 ascending  ->  counts [G] (tokens per group), offsets [G+1] (exclusive
 *   prefix sums), token_ids [B*k] (the tokens of group g, ascending, at offsets[g] .. offsets[g+1]).
 * cs_ffn_exec runs this itself for large batches; the call exists for callers that want the
 * buckets (support diversity statistics, their own scheduling).
 */
cs_status cs_bucket(cs_plan *plan, const int32_t *support, int32_t B, int32_t *counts, int32_t *offsets,
                    int32_t *token_ids, void *stream);

/*
 * cs_ffn_exec for callers that cannot allocate device memory.  (No counterpart in the paper: this
 * is a deployment convenience of the library.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a host framework that owns
 * the whole device heap and forbids side allocations, in a process whose memory budget was fixed
 * at start-up, or at a point where an allocation's implicit device synchronisation is not
 * acceptable.  Such callers cannot create a cs_plan, because a plan's scratch comes from
 * cudaMalloc.  This call needs no plan: the partial sums of the down projection are kept in an
 * 8 MiB array that is compiled into the library (so every GPU that loads the library holds those
 * 8 MiB until the process exits), and the call performs no cudaMalloc, cudaFree or any other
 * allocating routine.
 *
 * Same mathematics, arguments and layouts as cs_ffn_exec (gather path), with the shape taken from
 * `cfg` (d, d_ff, group, k, w_dtype are read; m, T, max_tokens, rms_eps are ignored).  Pointers must
 * be 16-byte aligned (CS_ERR_UNSUPPORTED otherwise, before anything is launched).  There is no
 * status word without a plan, so supports are not reported on: pass supports that are ascending,
 * distinct and in [0, G), such as cs_recover writes.  A group index outside [0, G) is never turned
 * into an address; the channels of such an entry contribute zero.
 *
 * Limit: B * nx * d * 4 bytes must fit in the 8 MiB array, where nx >= ceil(k * group / 32) is the
 * number of CTAs a token's rows are split over; e.g. d = 4096, k * group = 2816 allows B <= 5.
 * Larger requests return CS_ERR_SHAPE and launch nothing.
 *
 * The first call on each device looks up the array's device address and raises the kernels'
 * shared-memory limit; make that first call with the device current and before any stream
 * capture begins.  If it is also the process's first use of the library on that device, the CUDA
 * runtime loads the library's device code at that point, which places the 8 MiB array and may
 * synchronise the device: make that call during start-up, not inside a latency-critical section.
 * A failed launch is reported as CS_ERR_CUDA; if the second of the call's two kernels fails to
 * launch, the first is already enqueued and `out` is left unwritten.  All calls share the one array, which simply keeps whatever the last call
 * left there (every call overwrites all it later reads, so nothing has to be cleared).  Two calls
 * whose kernels can overlap on the GPU -- different streams, or different host threads on the
 * same device -- would race on it: keep calls to this entry point ordered on one stream per device.
 */
cs_status cs_ffn_exec_static(const cs_config *cfg, const cs_layer *layer, const float *h,
                             const int32_t *support, int32_t B, const float *residual, float *out,
                             void *stream);

/*
 * One decode step of one layer for B tokens with independent supports (Sec. 5; Sec. 12 online
 * phase):  n = rms_gamma ? RMSNorm(x) * rms_gamma : x;  y = S n;  (support, z) = recover(y);
 * x_out = (add_residual ? x : 0) + FFN(n, support).
 *   x [B,d] f32 -> x_out [B,d] f32 (x_out may alias x).  support_out [B,k], z_out [B,k],
 *   resid_out [B] may each be NULL.
 */
cs_status cs_layer_step(cs_plan *plan, const cs_layer *layer, const float *x, int32_t B, float *x_out,
                        int32_t *support_out, float *z_out, float *resid_out, void *stream);

/*
 * cs_layer_step with options (opt == NULL: cs_layer_step itself): another estimator, a warm start and
 * the temporal term from the previous step's result, the structured sensor, the drift against the
 * previous supports, or no estimation at all (reuse_support).  The stages run one after the other on
 * `stream` (the overlap of cs_layer_step's default path is not used).  With srht_sign / srht_rows the
 * layer must have no RMSNorm (rms_gamma == NULL) and layer->S is not read.
 */
cs_status cs_layer_step_ex(cs_plan *plan, const cs_layer *layer, const float *x, int32_t B,
                           const cs_step_options *opt, float *x_out, int32_t *support_out, float *z_out,
                           float *resid_out, void *stream);

/*
 * Confidence fallback (Sec. 12, online phase: when "the recovery confidence falls below a threshold, the
 * system may revert temporarily to a denser support").  Runs cs_layer_step_ex on `plan`; a token whose
 * relative residual ||y - Phi z_T|| / ||y|| exceeds `tau` is not trusted, and the step is run again for
 * those tokens alone on `dense`, a plan of the same layer shape with a larger k (k = G: the dense FFN),
 * whose outputs replace theirs in x_out.
 *   flags_out [B] int32 (device; 1 = fell back) may be NULL; *n_fallback (HOST) receives their number.
 *   support_out / z_out / resid_out describe the FIRST recovery of every token (a token that fell back
 *   executed on the k_dense groups its second recovery kept, which are not returned).
 * THIS CALL SYNCHRONISES `stream` once (the number of low-confidence tokens decides what is launched
 * next), so it cannot be captured in a graph; opt->reuse_support must be 0.
 */
cs_status cs_layer_step_fallback(cs_plan *plan, cs_plan *dense, const cs_layer *layer, const float *x, int32_t B,
                                 const cs_step_options *opt, float tau, float *x_out, int32_t *support_out,
                                 float *z_out, float *resid_out, int32_t *flags_out, int32_t *n_fallback,
                                 void *stream);

/*
 * Prompt-level support (Sec. 4): one support for the whole prompt from the mean prompt sketch,
 *   ybar = (1/n) sum_i S h_i  (computed as S applied to the mean hidden state, equal by linearity),
 * followed by the recovery of cs_recover on ybar.
 *   H [n,d] bf16  ->  support [k] int32 ascending, z [k] f32 (may be NULL), resid [1] (may be NULL).
 */
cs_status cs_prompt_support(cs_plan *plan, const float *S, const float *Phi, float mu, const void *H,
                            int32_t n, int32_t *support, float *z, float *resid, void *stream);

/*
 * FFN of every prompt token over ONE shared support (Sec. 4), as grouped dense GEMMs over the k
 * active row blocks on the tensor cores: bf16 operands, f32 accumulation, the intermediate
 * activation rounded to bf16 between the two GEMMs.
 *   H [n,d] bf16, support [k] int32 (device) -> out [n,d] bf16.  Requires w_dtype = CS_BF16,
 *   group = 128.  out must not overlap H.
 */
cs_status cs_ffn_exec_shared(cs_plan *plan, const cs_layer *layer, const void *H, int32_t n,
                             const int32_t *support, void *out, void *stream);

/*
 * cs_layer_step for callers whose activations live in HOST memory (ideally pinned): copies
 * x_host [B,d] f32 to plan scratch, runs the step, copies x_out [B,d] f32 (and, if not NULL,
 * the supports [B,k] int32) back, all enqueued on `stream`.  The host buffers must stay valid
 * until the stream has been synchronised.  Per step it moves 4*B*d bytes each way.  When both
 * buffers are page-locked, 16-byte aligned and small (at most 64 KB in the small-batch regime,
 * 4 MB on the tensor-core path), the bytes cross the bus inside the step's own kernels (a staging
 * kernel loads x, the last kernel stores x_out into the caller's buffer) instead of through the
 * copy engine; otherwise by cudaMemcpyAsync.
 */
cs_status cs_layer_step_host(cs_plan *plan, const cs_layer *layer, const float *x_host, int32_t B,
                             float *x_out_host, int32_t *support_host, void *stream);

/*
 * Regime crossover (Sec. 7: which precompiled execution path a batch takes).  Decode batches of at
 * least `tokens` tokens (and at most 128) run on the tensor cores, smaller ones as the gather GEMV.
 * A plan starts at max(2, min(16, ceil(1.15 * G / k))), the point where streaming every group once
 * moves fewer bytes than streaming k groups per token; 1 <= tokens <= 129 (129: never below 129
 * tokens).  Only shapes the tensor-core path supports (bf16 weights, 128-channel groups, d a
 * multiple of 256) are affected.  cs_plan_crossover returns the current value.
 */
cs_status cs_plan_set_crossover(cs_plan *plan, int32_t tokens);
int32_t cs_plan_crossover(const cs_plan *plan);

/*
 * Speculative start of the actuator at small batches (Sec. 5: the support is estimated while the
 * model runs; Sec. 15 asks that the sensing stage be accounted for, not hidden).  Off by default.  When
 * on, cs_layer_step below the regime crossover runs sketch and recovery in ONE launch and starts the
 * gather FFN's weight stream on the support of the FIRST iterate while the remaining iterations
 * run; rows requested for a group that later leaves the support are fetched again, so the supports
 * are those of the plain path and the outputs agree with it to rounding (the rows of a token are
 * dealt to one CTA fewer, which changes the order of the partial sums).  It needs k <= 32, G <= 128 and m <= 32
 * (CS_ERR_UNSUPPORTED otherwise).  On the shapes measured so far it is not faster than the plain chain
 * of launches (the recovery it overlaps costs less than the bookkeeping it adds), which is why it
 * is opt-in.
 * on = 2 is the lighter form: the same single sketch-and-recovery launch, but the plain gather kernel
 * behind it, which before it waits for the final supports only asks L2 (bulk prefetch) for the weight
 * blocks of the first iterate's groups.  A hint and nothing else: supports and outputs are those of the
 * plain path bit for bit.  Measured at the 7B shape it is not faster either (the gather kernel already
 * streams at the HBM rate between its first request and its last row, and gains 2.5 us from weights that
 * are all in L2, which the embedded recovery's exposed prologue costs again).
 * on outside {0, 1, 2}: CS_ERR_SHAPE.
 */
cs_status cs_plan_set_speculative(cs_plan *plan, int32_t on);

/*
 * Stage timing (the paper asks for sensing / recovery overhead to be reported apart from the
 * sparse kernel itself, Sec. 15 metric suite).  While enabled, every launch of a stage is bracketed
 * by CUDA events on the call's stream.  cs_plan_stage_times synchronises `stream` and returns the
 * device time in milliseconds of each stage's kernels in the most recent call that ran it.
 */
enum { CS_STAGE_SKETCH = 0, CS_STAGE_RECOVER = 1, CS_STAGE_EXEC = 2, CS_STAGE_REDUCE = 3,
       CS_STAGE_EXEC2 = 4 /* down GEMM of the tensor-core decode path */, CS_STAGE_COUNT = 5 };
cs_status cs_plan_enable_timing(cs_plan *plan, int32_t on);
cs_status cs_plan_stage_times(cs_plan *plan, void *stream, float ms[CS_STAGE_COUNT]);

/* Reads (and clears) the plan's device status word, synchronising `stream` first: CS_OK, or the
 * first CS_ERR_SUPPORT / CS_ERR_TIMEOUT a kernel recorded since the last read. */
cs_status cs_last_device_status(cs_plan *plan, void *stream, int32_t *code);

/* Number of kernels the library has launched through this plan since it was created. */
int64_t cs_launch_count(const cs_plan *plan);

/* Text of the last CUDA runtime error seen by this plan ("" if none); valid until the next call. */
const char *cs_last_cuda_error(const cs_plan *plan);

const char *cs_status_string(cs_status s);

#ifdef __cplusplus
}
#endif
#endif /* CS_H_ */
