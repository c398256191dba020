/* sgc.h -- C ABI of the B200 (sm_100a) implementation of one Sparse Gradient Compression step.
 *
 * One SGC step for one flat parameter vector W in R^d with gradient G in R^d (the paper treats every
 * weight matrix as a vector, Section 3 footnote; the flat row-major element index is the column
 * index of the measurement matrix A in R^{k x d}):
 *
 *   a1  G~ = Sparsify_s(G)                      keep the s largest |g_i|                (Section 3.2)
 *   a2  p = A G~ ,  q = A G~^2                  Eq. (4) and the equation after it; Algorithm 2
 *   a3  M <- b1 M + (1-b1) p ; V <- b2 V + (1-b2) q ; M^ = M/(1-b1^t) ; V^ = V/(1-b2^t)
 *                                                Algorithm 2
 *   a4  x^M = OMP_A(M^) , x^V = OMP_A(V^)       Eq. (7); Appendix B Algorithm 3
 *   a5  N = alpha x^M / (sqrt(x^V) + eps) ; W <- W - lr N          Eq. (8), Eq. (3); Algorithm 2
 *
 * A is never stored.  A[j][i] = sigma_k * Z(seed, j, i), sigma_k = fl32(1/sqrt(k)), where Z is a
 * counter-based, approximately standard-normal function of (seed, row, column) evaluated on the fly
 * (i.i.d. zero-mean entries of standard deviation 1/sqrt(k), Section 3.3).  Two states created with
 * the same (seed, k) therefore see the same A on their common columns.
 *
 * Conventions
 *   - Every function returns 0 on success, a negative SGC_ERR_* code for a rejected argument and a
 *     positive value (a cudaError_t) when a CUDA call failed.  Nothing aborts, traps or asserts.
 *   - "device pointer" = memory of the current CUDA device, "host pointer" = ordinary host memory.
 *   - All work of sgc_step is enqueued on the caller's stream; the call does not synchronise.
 *   - A state belongs to the device that was current in sgc_create; calls on one state must not overlap.
 *   - Data-dependent conditions (non-finite gradient, dependent OMP column, support mismatch) are
 *     recorded in a device status word that sgc_get(SGC_GET_STATUS) returns; see SGC_STATUS_*.
 */
#ifndef SGC_H_
#define SGC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define SGC_API __attribute__((visibility("default")))
#else
#define SGC_API
#endif

typedef struct sgc_state sgc_state;

enum {
    SGC_OK = 0,
    SGC_ERR_NULL = -1,        /* a required pointer is NULL                                   */
    SGC_ERR_DIM = -2,         /* d < 1, k < 1, s < 1, s > k, s > d, d >= 2^32, k or s too large */
    SGC_ERR_HYPER = -3,       /* beta outside [0,1), eps <= 0, lr or alpha not finite          */
    SGC_ERR_ALIGN = -4,       /* grad or weight not 16-byte aligned                            */
    SGC_ERR_WHAT = -5,        /* unknown selector for sgc_get                                  */
    SGC_ERR_SIZE = -6,        /* destination buffer too small                                  */
    SGC_ERR_GROUP = -7,       /* states of a group do not share (d, k, s, seed)                */
    SGC_ERR_NOSTEP = -8,      /* a record was requested before the first step                  */
    SGC_ERR_DEVICE = -9       /* the current device is not the one the state was created on    */
};

/* bits of the status word (sticky until sgc_clear_status) */
enum {
    SGC_STATUS_NONFINITE_INPUT = 1u << 0,  /* the gradient held a NaN or an infinity              */
    SGC_STATUS_DEPENDENT_COLUMN = 1u << 1, /* OMP stopped early: new column dependent on support  */
    SGC_STATUS_SUPPORT_MISMATCH = 1u << 2, /* supports of OMP(M^) and OMP(V^) differ (Section 3.3 expects equal) */
    SGC_STATUS_NEGATIVE_V = 1u << 3,       /* a recovered second-moment entry was <= 0; skipped   */
    SGC_STATUS_CANDIDATE_OVERFLOW = 1u << 4, /* a bounded candidate buffer overflowed.  In the speculative recovery the
                                                step then fell back to its slower exact path (result unaffected).  In the
                                                lock-step recovery more than 16 columns came within 2e-3 of the best fp32
                                                score of one pick (a block that keeps such a column beyond the two it
                                                forwards has its range screened again, so up to 16 always reach the fp64
                                                decision): the pick may then differ from the exact argmax by a near-tie */
    SGC_STATUS_SELECT_FALLBACK = 1u << 5,  /* the sampled top-s threshold missed; exact fallback ran */
    SGC_STATUS_TIMEOUT = 1u << 6           /* a bounded wait inside a tensor-core screening pass ran out; the pass's
                                              reports were discarded and the step finished on its slower exact path */
};

/* selectors for sgc_get: records of the LAST step, copied to a host buffer */
enum {
    SGC_GET_T = 0,          /* int64      step counter t                                        */
    SGC_GET_M = 1,          /* float[k]   first-moment state (not bias corrected)               */
    SGC_GET_V = 2,          /* float[k]   second-moment state                                   */
    SGC_GET_SEL_IDX = 3,    /* uint32[s]  support of Sparsify_s(G), ascending                   */
    SGC_GET_SEL_VAL = 4,    /* float[s]   the kept gradient entries                             */
    SGC_GET_P = 5,          /* double[k]  p = A G~                                              */
    SGC_GET_Q = 6,          /* double[k]  q = A G~^2                                            */
    SGC_GET_LAM_M = 7,      /* uint32[s]  columns picked by OMP(M^), in selection order; 0xFFFFFFFF = not picked */
    SGC_GET_LAM_V = 8,      /* uint32[s]  same for OMP(V^)                                      */
    SGC_GET_X_M = 9,        /* double[s]  least-squares coefficients aligned with LAM_M         */
    SGC_GET_X_V = 10,       /* double[s]  aligned with LAM_V                                    */
    SGC_GET_UPD_IDX = 11,   /* uint32[s]  positions of W that were updated, ascending; first N_UPD valid */
    SGC_GET_UPD_VAL = 12,   /* double[s]  lr * N at those positions                             */
    SGC_GET_N_UPD = 13,     /* int32      number of updated positions                           */
    SGC_GET_STATUS = 14,    /* uint32     status word                                           */
    SGC_GET_MISMATCH = 15,  /* int32      entries of LAM_M absent from LAM_V in the last step   */
    SGC_GET_NEGV = 16,      /* int32      common entries skipped because x^V <= 0               */
    SGC_GET_DONE_M = 17,    /* int32      completed OMP iterations for M^                       */
    SGC_GET_DONE_V = 18,    /* int32      completed OMP iterations for V^                       */
    SGC_GET_RNORM_M = 19,   /* double[s]  residual norm after each OMP(M^) iteration            */
    SGC_GET_RNORM_V = 20,   /* double[s]  same for OMP(V^)                                      */
    SGC_GET_ROUNDS = 21,    /* int32      screening passes over all d columns that the last step needed (speculative recovery) */
    SGC_GET_FALLBACK = 22,  /* int32      1 when the last step finished (or ran entirely) in lock-step  */
    SGC_GET_N_CAND = 23,    /* int32      length of the candidate list kept for the next step           */
    SGC_GET_LIST_ROUNDS = 25, /* int32     list passes (screening passes over the wide lists only) that the last step resolved */
    SGC_GET_PASS_ROWS = 26, /* int32       residual rows screened by the passes over all d columns of the last step, summed over
                               those passes (a state stepped alone; 2 k d flops of contraction per row)       */
    SGC_GET_ROUND_TRACE = 24 /* int32[24][3] per screening pass of the last step: picks of M^ confirmed so far, picks of V^ confirmed so
                                far, length of the candidate list after it (rows past SGC_GET_ROUNDS are zero)               */
};

/* How the recovery (a4) finds the picks of Algorithm 3; the picks themselves do not depend on it. */
enum {
    SGC_MODE_AUTO = 0,        /* speculative when k is a multiple of 64 and d >= 65536, lock-step otherwise */
    SGC_MODE_LOCKSTEP = 1,    /* one pass over all d columns per OMP iteration                             */
    SGC_MODE_SPECULATIVE = 2  /* OMP on a candidate list, confirmed by batched tensor-core screening passes */
};

/* Problem statement of Section 3 (Eq. 3) with the method of Algorithm 2.
 * Allocates the optimizer state M, V in R^k (zero, Section 3.3: M_0 = V_0 = 0), t = 0 and all
 * workspace on the current device; the library owns them until sgc_destroy.
 *   out    host pointer receiving the handle (set to NULL on failure)
 *   d      length of the flat weight / gradient vector, 1 <= d < 2^32
 *   k      rows of A (dimension of the compressed space), 1 <= k <= 16384
 *   s      sparsity, 1 <= s <= min(k, d), s <= 1024
 *   seed   names the matrix A
 *   lr     learning rate eta of Eq. (3); beta1, beta2, eps: Algorithm 2 "Require"
 * The scale alpha of Eq. (8) defaults to 1 (sgc_set_alpha). */
SGC_API int sgc_create(sgc_state** out, int64_t d, int32_t k, int32_t s, uint64_t seed, float lr, float beta1,
               float beta2, float eps);

/* One step of Algorithm 2 followed by Eq. (3): W <- W - lr * SGC(G).
 *   grad    device pointer, d floats, 16-byte aligned, read only
 *   weight  device pointer, d floats, 16-byte aligned, modified in place at no more than s positions
 *   stream  a cudaStream_t (NULL = the default stream)
 * Returns after enqueueing; the caller keeps grad and weight alive until the stream has drained. */
SGC_API int sgc_step(sgc_state* st, const float* grad, float* weight, void* stream);

/* Same result as n independent sgc_step calls, for states that share (d, k, s, seed) and hence the
 * same A (Section 4.4 lets equal-sized vectors share one A): their 2n residuals are correlated
 * against each generated tile of A together.
 *   states, grads, weights   host arrays of n handles / device pointers */
SGC_API int sgc_step_group(sgc_state* const* states, const float* const* grads, float* const* weights, int32_t n,
                   void* stream);

/* Memory-efficient SGC (MESGC, Section 4.4 "Efficient SGC"): the gradient is split into c equal chunks, SGC with
 * s_c = s / c entries runs on every chunk, and all chunks share one small matrix A (k x d/c).  The caller creates c
 * states with sgc_create(d / c, k, s_c, seed, ...) -- the same seed, hence the same A -- and passes the whole vectors:
 *   grad, weight   device pointers, c * (d / c) floats; chunk i occupies [i * d/c, (i + 1) * d/c)
 * d / c must be a multiple of 4 (16-byte aligned chunks).  The result is that of sgc_step_group on the c chunk
 * pointers.  Chunk lists with small problems (s_c <= 32, k <= 256, all chunks at the same step with the same
 * hyper-parameters, no sgc_set_recovery variant, no forced speculative mode, profiling off) are served by batched
 * kernels, 2 + 2 s_c launches for all chunks together; the first such call for a given list of states allocates a
 * table of their buffers (one cudaMalloc and one synchronous copy; freed by sgc_destroy of states[0]), so it should
 * not happen inside a stream capture.  SGC_ERR_GROUP when the states differ in (d, k, s, seed) or one appears twice. */
SGC_API int sgc_step_chunked(sgc_state* const* states, int32_t c, const float* grad, float* weight, void* stream);

/* Compute-efficient SGC (CESGC, Section 4.4 "Efficient SGC"): the gradient of an m x n weight matrix is first
 * compressed with a projection B (r x m, rows orthonormal; the paper takes the first r left-singular vectors of a
 * gradient and renews them every fixed number of iterations -- computing B is the caller's business), SGC runs on the
 * r x n matrix B G, chunked as in sgc_step_chunked, and the update returns through B^T:
 *     W <- W - eta B^T SGC(B G).
 *   states       c states created with sgc_create(r * n / c, k, s_c, seed, ...); chunk i covers the flat range
 *                [i * r n / c, (i + 1) * r n / c) of the row-major r x n matrix (r * n / c a multiple of 4)
 *   B            device, r x m row-major floats, read-only; r <= 64
 *   grad         device, m x n row-major floats, read-only
 *   weight       device, m x n row-major floats; column j changes where SGC's update has a non-zero in column j
 *   scratch      device, 2 * r * n floats, 16-byte aligned, owned by the caller, overwritten: B G, then -eta N
 * B G is accumulated to about 44 bits and rounded to fp32 once, so the kept entries are those of the exactly projected
 * gradient (a product formed in fp64 differs by one ulp in a few elements per ten thousand).
 * Enqueued on stream.  Errors: as sgc_step_chunked; SGC_ERR_DIM for r < 1, r > 64, m < 1, n < 1 or c not dividing r * n. */
SGC_API int sgc_cesgc_step(sgc_state* const* states, int32_t c, const float* B, int32_t r, int32_t m, int32_t n,
                           const float* grad, float* weight, float* scratch, void* stream);

/* Waits for the state's last enqueued work, then frees everything.  NULL is accepted. */
SGC_API int sgc_destroy(sgc_state* st);

/* alpha of Eq. (8) ("a scaling factor"); must be finite. */
SGC_API int sgc_set_alpha(sgc_state* st, float alpha);

/* SGCA re-projection (Appendix C, Algorithm 4): replaces the measurement matrix by the one that new_seed
 * names and re-aligns the optimizer state with it, M <- A' OMP_A(M), V <- A' OMP_A(V).  Call it after the sgc_step of
 * an iteration t with t mod T = 0: the recoveries of that step are reused, since OMP_A(M) = (1 - beta1^t) OMP_A(M^)
 * (OMP is scale-equivariant; the paper itself notes that the results of the first call can be kept).  From the next
 * step on, p, q and both recoveries use A'.  Enqueued on stream; SGC_ERR_NOSTEP before the first step. */
SGC_API int sgc_reproject(sgc_state* st, uint64_t new_seed, void* stream);

/* Chooses the recovery strategy (SGC_MODE_*).  Both strategies return the picks of Algorithm 3 (Appendix B):
 * the speculative one runs OMP on a short candidate list and then proves, with one tensor-core pass over all
 * d columns against the residuals of all iterations at once, that no other column would have been picked; a
 * refuted pick is replaced by the true argmax and the round repeats from there.
 * SGC_ERR_DIM when SGC_MODE_SPECULATIVE is requested and k is not a multiple of 64.  States with d < 65536 never
 * speculate on their own accord and are created without the buffers of that strategy (some 50 MB plus 6.5 bytes per
 * column); asking for SGC_MODE_SPECULATIVE allocates them here (one cudaMalloc, synchronises; a CUDA error code if it fails). */
SGC_API int sgc_set_mode(sgc_state* st, int32_t mode);

/* Opt-in variant of the recovery, built on the remark after Eq. (8) that OMP_A(M_t) and OMP_A(V_t) have their
 * non-zeros at the same positions.  The default (0, 0.0) is Algorithm 2 as printed: two independent recoveries of s
 * iterations each.
 *   shared_support  1: only OMP_A(M^) selects columns; x^V is the least-squares fit of V^ on those columns (same
 *                   order), so both supports are equal by construction and Eq. (8) applies on all of it where
 *                   x^V > 0.  The per-iteration residual norms of V^ (SGC_GET_RNORM_V) are not recorded (zeros).
 *   residual_tol    > 0: a recovery ends after the first iteration that leaves ||r|| <= residual_tol * ||y||
 *                   (fewer than s picks; SGC_GET_DONE_* tell how many).  The picks made before the stop are those of
 *                   Algorithm 3; the coefficients are the least-squares fit on them.  Must be finite and >= 0.
 * Takes effect from the next step; sgc_reproject reuses whatever the last step recovered. */
SGC_API int sgc_set_recovery(sgc_state* st, int32_t shared_support, double residual_tol);

/* Synchronises with the state's last step and copies one record to host memory (selectors above).
 *   dst    host pointer; bytes = its capacity, must cover the record */
SGC_API int sgc_get(sgc_state* st, int32_t what, void* dst, size_t bytes);

/* Overwrites the optimizer state: M, V host pointers to k floats each, t >= 0 (checkpoint resume). */
SGC_API int sgc_set_state(sgc_state* st, const float* M, const float* V, int64_t t);

/* Clears the sticky status word. */
SGC_API int sgc_clear_status(sgc_state* st);

/* The status word (SGC_STATUS_* bits, sticky until sgc_clear_status): synchronises with the state's last step and
 * stores the word in *out (host pointer).  Same value as sgc_get(st, SGC_GET_STATUS, ...). */
SGC_API int sgc_status(sgc_state* st, uint32_t* out);

/* Bound, in nanoseconds, of every wait on a hardware barrier inside the tensor-core screening pass (the only kernel of
 * this library whose warps wait for one another through memory).  When a wait runs out, the pass records the fact,
 * lets the copies and matrix operations in flight finish, releases its tensor memory and returns; the step then
 * discards the pass's reports, finishes on the exact lock-step path and sets SGC_STATUS_TIMEOUT.  The paper has no
 * counterpart: this is failure handling, and the setter exists so that the path can be exercised (a bound of a few
 * nanoseconds makes ordinary waits run out without anything being broken).
 *   st   the state whose passes are meant; NULL sets the bound used by sgc_screen (process-wide)
 *   ns   0 restores the default of two seconds */
SGC_API int sgc_set_wait_limit(sgc_state* st, uint64_t ns);

/* Upper bound on the speculation rounds (candidate-list OMP + screening pass + resolve) that one step of this state
 * enqueues; the picks that the rounds leave open are made on the exact lock-step path, so the result is Algorithm 3's
 * (Appendix B) for every bound.  The paper has no counterpart: the bound caps the work a step enqueues ahead of time.
 *   rounds   0 (the default) lets the library choose from the number of rounds the last finished step needed (twice that
 *            plus three, at most 24); negative: SGC_ERR_DIM.  In a group (sgc_step_group) the largest bound of a batch holds. */
SGC_API int sgc_set_max_rounds(sgc_state* st, int32_t rounds);

/* Number of kernel launches the last sgc_step / sgc_step_group enqueued for this state. */
SGC_API int sgc_last_launches(sgc_state* st, int32_t* out);

/* Top-s selection (step a1 alone) for callers that cannot allocate device memory.  The paper has no
 * counterpart: this is the same selection that sgc_step performs first, offered on its own with its
 * scratch (278 784 bytes: threshold histogram, candidate list, counters) held in a static device array
 * inside the library instead of in a state object.  Meant for hosts where a cudaMalloc is off the table at
 * call time, e.g. a framework that has already claimed all device memory for its own pool, or a thread
 * that cannot afford cudaMalloc's device-wide synchronisation.  The call makes no cudaMalloc/cudaFree and
 * uses no allocating routine.
 *   grad        device pointer, d floats, 16-byte aligned, read only
 *   d, s        1 <= s <= min(d, 1024), d < 2^32; anything larger is rejected with SGC_ERR_DIM
 *   out_idx     device pointer, s uint32: positions of the s largest |g| (ties -> lower index), ascending
 *   out_val     device pointer, s floats: the gradient values at those positions
 *   out_status  device pointer to one uint32 receiving SGC_STATUS_* bits of this call, or NULL
 *   stream      a cudaStream_t; all work is enqueued there, the call does not synchronise
 * The first call on each device looks up the device address of the static array (cudaGetSymbolAddress)
 * and should therefore come before any stream capture; devices with an index of 64 or more are not served
 * (SGC_ERR_DIM).  Every call on a device shares that array and
 * finds the previous call's contents in it: what must start at zero is cleared on `stream` first.  Calls
 * that overlap on the GPU race on the array; serialise them (one stream, or events between streams). */
SGC_API int sgc_sparsify_static(const float* grad, int64_t d, int32_t s, uint32_t* out_idx, float* out_val,
                                uint32_t* out_status, void* stream);

/* Per-kernel timing of the steps that follow (no counterpart in the paper: measurement support).
 * While enabled, sgc_step brackets every kernel launch with CUDA events on the caller's stream;
 * sgc_get_profile synchronises and returns the totals accumulated since sgc_set_profile(st, 1):
 *   ms[0] top-s sample    ms[1] top-s filter (the pass over the gradient)   ms[2] top-s pick
 *   ms[3] projection+Adam ms[4] OMP kernels (candidate-list and lock-step)   ms[5] resolve + bookkeeping
 *   ms[6] combine+scatter ms[7] tensor-core screening passes
 *   launches[i] = number of kernel launches behind ms[i].   Both are host arrays of 8 entries. */
SGC_API int sgc_set_profile(sgc_state* st, int enable);
SGC_API int sgc_get_profile(sgc_state* st, float* ms, int32_t* launches);

/* Fills a device buffer with Z(seed, row0 + r, col0 + c), r < nrows, c < ncols, row-major
 * (the A definition above without the scale); for checking the generator.
 *   out   device pointer, nrows*ncols floats */
SGC_API int sgc_z_block(uint64_t seed, int64_t row0, int64_t nrows, int64_t col0, int64_t ncols, float* out, void* stream);

/* The screening pass of the recovery on its own ("Projection" of Algorithm 3 for n residuals at once):
 * reports every pair (column i, residual j) with |<Z_i, R_j>| / ||Z_i|| >= tau[j], where Z_i is column i of
 * the unscaled measurement matrix of (seed, k) and R_j row j of rt.  Runs on the tensor cores.
 *   d, k        1 <= d < 2^32; k a multiple of 64, 64 <= k <= 65536
 *   n           number of residuals, a multiple of 32, 32 <= n <= 256
 *   rt          device pointer, n x k binary16 (IEEE half) bit patterns, row-major, 16-byte aligned, read only
 *   tau         device pointer, n floats (+infinity disables a residual)
 *   rep_count   device pointer, n uint32: number of reports per residual (may exceed rep_cap)
 *   rep         device pointer, n x rep_cap pairs (uint32 column, float score bits); the first
 *               min(rep_count[j], rep_cap) pairs of row j are valid, in no particular order
 *   error_flag  device pointer to one int32, set to 1 if the kernel gave up on an internal wait (results invalid)
 * Scores carry a relative error of up to 1e-3 (the norm ||Z_i|| is accumulated in short binary16 partial sums), so a
 * pair whose exact score lies within that distance of its threshold may or may not be reported.
 * Everything is enqueued on stream; the call does not synchronise. */
SGC_API int sgc_screen(uint64_t seed, int64_t d, int32_t k, int32_t n, const uint16_t* rt, const float* tau, uint32_t* rep_count,
                       uint32_t* rep, int32_t rep_cap, int32_t* error_flag, void* stream);

/* Human-readable text for a return code of this library (static storage). */
SGC_API const char* sgc_strerror(int code);

/* Library version, major*10000 + minor*100 + patch. */
SGC_API int sgc_version(void);

#ifdef __cplusplus
}
#endif
#endif /* SGC_H_ */
