/*
 * csd.h -- C ABI of the verification-and-rescue step of Calibrated Speculative
 * Decoding (CSD) for NVIDIA B200 (sm_100a).
 *
 * One step takes the target model's logits for the gamma drafted positions plus
 * the bonus position, the gamma draft tokens, the Online Correction Memory (OCM)
 * and the gate threshold tau, and returns the number of accepted draft tokens,
 * the token to emit after them, and the rejections to feed back to the memory:
 * the verification loop of Algorithm 1 in its greedy (T = 0) form, the mode of
 * the paper's evaluation (Sec. 5.1).
 *
 * Notation: B batch rows, K = gamma draft tokens per row, V vocabulary size,
 * z[b,i,v] target logits, d[b,i] draft token, t[b,i] = argmax_v z[b,i,v]
 * (lowest index on ties), m[b,i] = z[b,i,t].
 *
 * Conventions
 *   - Every tensor pointer is a DEVICE pointer owned by the caller unless the
 *     argument is documented as a host pointer.  The library owns only the
 *     memory behind a csd_ocm_t.
 *   - All work is enqueued on the CUDA stream passed as `stream` (a cudaStream_t
 *     cast to void*; NULL is the legacy default stream).  Nothing synchronises
 *     unless documented.  Calls on one csd_ocm_t must be stream-ordered (but see
 *     csd_ocm_set_shared).
 *   - Every function returns a csd_status_t and never throws or aborts.  Misuse
 *     that the host can see is refused before anything is launched.  Conditions
 *     only the device can see (a NaN logit, a draft id outside [0,V), a full
 *     table) set sticky flags / counters readable with csd_ocm_stats; the device
 *     never traps.  Within a launch no block waits for another (arrival counters
 *     only); the one exception are the two blocks of a thread-block cluster in the
 *     LM-head pair kernel, which the hardware schedules together: their barrier
 *     waits on each other are bounded in time, and every path of both blocks reaches
 *     the two cluster barriers they meet at.  With csd_set_overlap on, the warps that finalise a batch row wait for
 *     the PREVIOUS launch on the stream: a bounded poll (2^14 loads) of a completion
 *     word, then the hardware's wait for that grid to retire, which always ends.
 *   - Determinism: for fixed (B,K,V,dtype) every output, including the sums s,
 *     is bit-reproducible from run to run.
 */
#ifndef CSD_H_
#define CSD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct csd_ocm csd_ocm_t;

typedef enum {
    CSD_OK = 0,
    CSD_ERR_INVALID_ARG = 1,
    CSD_ERR_CUDA = 2,
    CSD_ERR_OOM = 3,
    CSD_ERR_UNSUPPORTED = 4,
    CSD_ERR_WORKSPACE = 5,
    CSD_ERR_IO = 6
} csd_status_t;

typedef enum { CSD_F32 = 0, CSD_BF16 = 1 } csd_dtype_t;

/* Largest K (draft tokens per row) a step accepts: one warp lane per position. */
#define CSD_MAX_K 32

/* sticky device flags reported in csd_stats_t.flags */
#define CSD_FLAG_NAN_LOGIT      0x1u  /* a row's sum came out NaN (NaN / +inf logit, or a row of -inf) */
#define CSD_FLAG_BAD_DRAFT      0x2u  /* a draft id outside [0, V) was seen                            */
#define CSD_FLAG_PROBE_EXHAUSTED 0x4u /* a hash probe visited every slot (cannot happen below capacity) */
#define CSD_FLAG_COUNT_SATURATED 0x8u /* a count reached 2^32 - 1                                      */
#define CSD_FLAG_INTERNAL       0x10u /* an index check inside the library failed: a bug of the library,
                                         the step's results are unreliable (csd_stats_t.debug_site says
                                         which check).  The access was skipped; nothing trapped.  One
                                         check (a partial-result slot) is always compiled in; a library
                                         built with -DCSD_DEBUG checks every index it computes.        */

/* Optional per-position diagnostics.  Any member may be NULL.  Row arrays have
 * B*(K+1) entries, position arrays B*K, both row-major.  Values are defined for
 * every position, also past a row's first un-rescued rejection. */
typedef struct {
    float   *m;      /* [B,K+1] max logit                                                  */
    float   *s;      /* [B,K+1] sum_v exp(z_v - m): the soft-max normaliser of Eq. 3      */
    float   *lse;    /* [B,K+1] m + ln s                                                   */
    int32_t *t;      /* [B,K+1] argmax, lowest index on ties (t* of Algorithm 1 at T = 0) */
    float   *zd;     /* [B,K]   z[b,i,d[b,i]]   (NaN if d is outside [0,V))                */
    float   *score;  /* [B,K]   exp(zd - m) = p(d)/p(t*), the Score of Fig. 1 / Eq. 3      */
    float   *p_d;    /* [B,K]   soft-max probability of the draft token                    */
    float   *p_t;    /* [B,K]   soft-max probability of t*                                 */
    uint32_t *cnt;   /* [B,K]   OCM count of (d, t*) at the start of the step (0 = absent) */
} csd_diag_t;

typedef struct {
    uint64_t n_slots;       /* capacity in slots (power of two)                      */
    uint64_t key_limit;     /* most distinct pairs the table admits (= n_slots / 2)  */
    uint64_t n_keys;        /* distinct pairs stored                                 */
    uint64_t n_dropped;     /* update occurrences dropped because the table was full */
    uint64_t steps;         /* csd_verify / csd_step calls                           */
    uint64_t positions;     /* draft positions verified (B*K per step)               */
    uint64_t matches;       /* reached positions with d == t*                        */
    uint64_t rescues;       /* reached mismatches accepted through OCM + SCG         */
    uint64_t rejections;    /* pairs handed to the memory update                     */
    uint32_t lambda;        /* frequency threshold in force                          */
    uint32_t flags;         /* CSD_FLAG_* (sticky until csd_ocm_reset)               */
    uint32_t debug_site;    /* first failed index check (0 = none), see CSD_FLAG_INTERNAL */
    uint32_t reserved;
} csd_stats_t;

/* ---- Online Correction Memory (Sec. 4.2): frequency table of ordered pairs ----
 *
 * The table T of Algorithm 1: (draft token, target token) -> count, an
 * open-addressed hash table in device memory (16-byte slots, linear probing).
 * The paper fixes no capacity rule; this library's rule is: at most n_slots/2
 * distinct pairs; a pair already present always counts; a new pair is admitted,
 * in the canonical order of the update (index order), only while fewer than
 * n_slots/2 pairs are stored, else that occurrence is dropped and counted in
 * n_dropped; nothing is evicted.  Counts are 32-bit and saturate.
 */

/* Allocate an empty table on `device` (cudaSetDevice is called and left set).
 * n_slots: power of two, 64 .. 2^30.  lambda: frequency threshold of the candidate
 * proposal test T[(d,t*)] >= lambda (the paper's main protocol uses 6; 0 makes
 * every divergence a candidate).  Synchronises the device once.
 * Errors: INVALID_ARG (null out, bad n_slots), OOM, CUDA. */
csd_status_t csd_ocm_create(csd_ocm_t **out, uint64_t n_slots, uint32_t lambda, int device);

/* Empty the table and zero its statistics and flags (asynchronous on `stream`). */
csd_status_t csd_ocm_reset(csd_ocm_t *ocm, void *stream);

/* Free the table.  The caller makes sure no work using it is still running. */
csd_status_t csd_ocm_destroy(csd_ocm_t *ocm);

/* Change lambda for subsequent calls (host side; stream-ordered like any call). */
csd_status_t csd_ocm_set_lambda(csd_ocm_t *ocm, uint32_t lambda);

/* Several streams on one memory (the paper's Limitations leave concurrent updates of T open; this is
 * the library's reading).  By default all calls on one csd_ocm_t are stream-ordered, which is what makes
 * every look-up of a step see exactly the step-start counts and admission near the key limit follow the
 * canonical order.  With sharing switched on, csd_step / csd_step_sampled / csd_ocm_update /
 * csd_ocm_import calls on DIFFERENT streams (each with its own workspace and output buffers) may run at
 * the same time on one memory:
 *   - every recorded pair is counted exactly once whatever the interleaving (counts are the multiset
 *     union of all streams' recorded pairs, as long as no pair is dropped for lack of room);
 *   - a look-up sees the count of its pair at some moment between the start and the end of its own
 *     step: pairs recorded by the SAME step are never seen (they are added after its last look-up),
 *     pairs that other streams record meanwhile may or may not be;
 *   - the table never holds more than n_slots/2 pairs; which new pairs are admitted when it is nearly
 *     full depends on arrival order (each new pair takes one unit of the remaining room atomically, and
 *     claims in flight -- at most B*K per step, 1024 per bulk update -- count against the room, so within
 *     that margin of the limit a new pair may be dropped, and counted in n_dropped, although room remains).
 * Calls that rebuild or read the whole table (csd_ocm_reset / age / merge / export / save) must still
 * not run beside anything else.  Host function; set it while no work on the memory is in flight
 * (switching it off synchronises the device). */
csd_status_t csd_ocm_set_shared(csd_ocm_t *ocm, int enable);

/* ---- one verification step ---------------------------------------------------- */

/* Bytes of scratch csd_verify / csd_step need for this shape (0 on invalid shape).
 * The scratch holds, four times over (consecutive launches take the copies in turn),
 * per-block partial reductions, slot hints and arrival counters. */
size_t csd_workspace_bytes(int B, int K, int V, csd_dtype_t dtype);

/* Zero a workspace.  Do it once before its first use (and after any aborted
 * launch); the kernels leave the counters zeroed again on completion, so the
 * same workspace can be reused step after step without further clearing.  (The
 * library also clears a workspace by itself the first time it sees its address,
 * and whenever the launch shape it was last used with differs from the current
 * one; memory that is freed and handed out again at the same address with stale
 * contents is the case only this call covers.)  One workspace serves one step at
 * a time, and all steps that use it are issued on one stream. */
csd_status_t csd_workspace_init(void *workspace, size_t workspace_bytes, void *stream);

/* The verification loop of Algorithm 1 (greedy) for all B rows, read-only on the
 * memory.  For each row b and position i < K:
 *     t* = argmax z[b,i,:]                     (residual resample at T = 0)
 *     match   = (d[b,i] == t*)                 (acceptance test at T = 0)
 *     is_freq = T[(d[b,i], t*)] >= lambda      (candidate proposal, Sec. 4.2)
 *     is_safe = z[b,i,d] - z[b,i,t*] >= ln tau (Eq. 3; decided in double on the
 *               exact inputs against (float) log((double) tau); equality passes)
 *     position accepted iff  match or (is_freq and is_safe)
 * accept_len[b] = number of leading accepted positions (n of Algorithm 1);
 * next_token[b] = t* of the first non-accepted position, or argmax z[b,K,:] (the
 * bonus token) when all K are accepted; rescued_mask[b,i] = 1 for non-matching
 * positions inside the accepted prefix.  rej_draft/rej_target[b,i] hold the pair
 * (d, t*) for every divergence the loop reaches (rescued ones and the one that
 * ends the row), -1 elsewhere: exactly the UpdateMemory calls of Algorithm 1.
 * All look-ups see the table as it is when the call starts.
 *
 * logits : [B, K+1, V], element (b,i,v) at  b*stride_b + i*stride_k + v  (strides
 *          in elements, V contiguous); CSD_F32 or CSD_BF16.  128-bit loads are
 *          used when the base and both strides are 16-byte multiples, a slower
 *          element-wise path otherwise.
 * draft  : [B, K] int32.  An id outside [0,V) is a mismatch that cannot be
 *          rescued and is not recorded (flag CSD_FLAG_BAD_DRAFT).
 * tau    : gate threshold, >= 0 and not NaN.  0 disables the gate (memory only);
 *          tau > 1 can never pass.
 * accept_len, next_token : [B] int32.   rescued_mask : [B,K] uint8.
 * rej_draft, rej_target  : [B,K] int32.
 * diag   : NULL, or a HOST pointer to a struct of optional device arrays.
 * workspace : >= csd_workspace_bytes(B,K,V,dtype) bytes, 16-byte aligned,
 *          initialised with csd_workspace_init.
 * Errors: INVALID_ARG (null pointer, B,K,V <= 0, bad tau or strides),
 *         UNSUPPORTED (K > CSD_MAX_K), WORKSPACE (too small / misaligned), CUDA.
 * One kernel launch; asynchronous. */
csd_status_t csd_verify(const void *logits, csd_dtype_t dtype, int B, int K, int V,
                        int64_t stride_b, int64_t stride_k,
                        const int32_t *draft, const csd_ocm_t *ocm, float tau,
                        int32_t *accept_len, int32_t *next_token, uint8_t *rescued_mask,
                        int32_t *rej_draft, int32_t *rej_target,
                        const csd_diag_t *diag,
                        void *workspace, size_t workspace_bytes, void *stream);

/* UpdateMemory of Algorithm 1 for a batch of n pairs: count[(rej_draft[j],
 * rej_target[j])] += 1 for j = 0..n-1 in index order (the order only matters for
 * admission when the table is nearly full).  Entries with a negative member are
 * skipped.  Duplicates each count.  n may be any size >= 0.  Asynchronous. */
csd_status_t csd_ocm_update(csd_ocm_t *ocm, const int32_t *rej_draft, const int32_t *rej_target,
                            int64_t n, void *stream);

/* csd_verify followed by csd_ocm_update of the step's rejections in (b,i) order,
 * fused into the same single launch: the online adaptation of Sec. 4.2 (look-up
 * before update: a pair recorded in this step can reach lambda only for later
 * steps).  Arguments as csd_verify. */
csd_status_t csd_step(const void *logits, csd_dtype_t dtype, int B, int K, int V,
                      int64_t stride_b, int64_t stride_k,
                      const int32_t *draft, csd_ocm_t *ocm, float tau,
                      int32_t *accept_len, int32_t *next_token, uint8_t *rescued_mask,
                      int32_t *rej_draft, int32_t *rej_target,
                      const csd_diag_t *diag,
                      void *workspace, size_t workspace_bytes, void *stream);

/* csd_step in two phases, for steps in which many rows stop early.  Algorithm 1 returns at a row's first
 * un-rescued rejection and never looks at the positions after it; csd_step nevertheless streams all K+1 logit
 * rows of every batch row, because it decides everything in one pass.  This variant first verifies positions
 * 0 .. f-1 of every batch row (reading logit rows 0 .. f), then positions f .. K-1 and the bonus row only of the
 * batch rows that accepted all of the first f (reading their logit rows f .. K), and finally updates the memory
 * with all recorded pairs in (b, i) order -- after the last look-up, as csd_step does.  Results are those of
 * csd_step; the optional diagnostics are written only for the logit rows that were read.  Bytes read:
 * B (f+1) V + (rows still alive) (K+1-f) V elements instead of B (K+1) V.
 * first_phase_positions: f, 1 .. K-1 (0 = automatic, about K/3).  K >= 2.  The launches of this call are
 * plain stream-ordered launches whatever csd_set_overlap says.
 * workspace: csd_early_exit_workspace_bytes bytes for the same first_phase_positions, 16-byte aligned.
 * Three launches; asynchronous.  Errors as csd_step; UNSUPPORTED for K < 2. */
size_t csd_early_exit_workspace_bytes(int B, int K, int V, csd_dtype_t dtype, int first_phase_positions);
csd_status_t csd_step_early_exit(const void *logits, csd_dtype_t dtype, int B, int K, int V,
                                 int64_t stride_b, int64_t stride_k,
                                 const int32_t *draft, csd_ocm_t *ocm, float tau, int first_phase_positions,
                                 int32_t *accept_len, int32_t *next_token, uint8_t *rescued_mask,
                                 int32_t *rej_draft, int32_t *rej_target, const csd_diag_t *diag,
                                 void *workspace, size_t workspace_bytes, void *stream);

/* csd_verify without a workspace argument and without any allocation.  (The paper has
 * no counterpart: this is a deployment convenience of the library.)
 *
 * Who needs it: code that runs the verification from a place where device memory can
 * no longer be obtained -- an inference server whose framework reserved the whole GPU
 * for its own pool at start-up, a plug-in that is handed tensors but no allocator, a
 * latency-critical loop where an allocation (which may synchronise the device or
 * fail) is not acceptable.  Such a caller cannot provide the workspace csd_verify
 * asks for.  Here the kernel's scratch is a fixed array of CSD_STATIC_SCRATCH_BYTES
 * that is part of the library image: every GPU that loads the library holds it until
 * the process exits.  The call performs no cudaMalloc / cudaFree and calls no
 * allocating routine.  (The csd_ocm_t it reads was allocated earlier by
 * csd_ocm_create, which such a caller runs during its set-up phase.)
 *
 * Arguments and results are those of csd_verify (inputs and outputs remain the
 * caller's device buffers); the current device must be the memory's device.
 * Shapes whose csd_workspace_bytes exceeds CSD_STATIC_SCRATCH_BYTES are refused with
 * CSD_ERR_WORKSPACE before anything is launched (all five reference workloads need
 * less than 200 KiB).  The first call on each device looks up the array's device
 * address; make that first call outside any stream capture.  All calls share the one
 * array, which keeps the previous call's contents, so every call first clears the
 * part it uses (asynchronously, on `stream`); two calls that overlap on the GPU (two
 * streams, or this call next to a csd_step launched with csd_set_overlap) would race
 * on it: issue them on one stream, one after the other. */
#define CSD_STATIC_SCRATCH_BYTES (1u << 20)
csd_status_t csd_verify_static(const void *logits, csd_dtype_t dtype, int B, int K, int V,
                               int64_t stride_b, int64_t stride_k,
                               const int32_t *draft, const csd_ocm_t *ocm, float tau,
                               int32_t *accept_len, int32_t *next_token, uint8_t *rescued_mask,
                               int32_t *rej_draft, int32_t *rej_target,
                               const csd_diag_t *diag, void *stream);

/* ---- stochastic verification: Algorithm 1 as printed, temperature T > 0 ----------
 *
 * With p_i = softmax(z_i / T) (target) and q_i = softmax(y_i / T) (draft), for each row
 * b and position i < K, in order:
 *     alpha = min(1, p_i(d) / q_i(d));  the position passes iff r[b,i] <= alpha   (Eq. 2)
 *     otherwise  t* ~ norm(max(0, p_i - q_i))        (the residual distribution, Sec. 3.1)
 *                is_freq = T[(d, t*)] >= lambda      (candidate proposal, Sec. 4.2)
 *                is_safe = z_i(d) - z_i(t*) >= ln tau  (Eq. 3: raw logits, whatever T is;
 *                          against a drawn t* the ratio may exceed 1)
 *                the pair (d, t*) is recorded for UpdateMemory; rescued iff is_freq and
 *                is_safe, else the row stops here and emits t*
 * accept_len[b] = positions passed or rescued before the stop; next_token[b] = t* of the
 * stopping position, or a draw from p_K (the bonus token) when all K went through.
 *
 * The paper does not say how the draws are made; this library's reading:
 *   - the uniforms r of the acceptance test are an INPUT ([B,K] float, in [0,1));
 *   - a draw from weights w(v) is an exponential race, argmax w / E (lowest index on ties),
 *     run in TWO levels: first among the groups of 8 consecutive tokens (group g = tokens
 *     8g .. 8g+7, tokens at or beyond V weigh 0, group weight W_g = the sum of its tokens'
 *     weights), then among the 8 tokens of the winning group.  P(v) = W_g / sum W * w(v) / W_g
 *     = w(v) / sum w.  Clocks: E = -ln(1 - u), u = (j + 1/2) / 2^23, j = the top 23 bits of a
 *     32-bit word of Philox4x32-10 (Salmon et al., SC'11) under key (seed low, seed high);
 *     clock number n of stream s of the draw of row = b*(K+1)+i (i = K: the bonus draw) is word
 *     (n & 3) of counter (n >> 2, row, s, 0).  Group g uses clock g of stream 0; token v of the
 *     winning group uses clock v of stream 1.  The group size and the clock grid are part of
 *     this contract: a caller can reproduce every drawn token from (seed, b, i) and the logits.
 * Draws are made only where a row can need them.  A large step makes them in two rounds: first for every
 * row's first failed position (or its bonus draw if every position went through), then the later failed
 * positions and the bonus draw of the rows whose first failure was rescued.  A small step (the two logit
 * tensors under 32 MB; see csd_sampled_set_rounds) makes every failed position's draw and every bonus draw
 * in one round, because two more launches cost more there than the draws saved.  diag.t_star and diag.bonus
 * are -1 where no draw was made (never at a position the row reaches); which draws are made beyond those a row
 * reaches is not part of the contract, their values are.
 * Look-ups see the memory as it is when the call starts; a draft id outside [0,V) fails
 * the test, cannot be rescued and is not recorded.
 *
 * draft_logits: y[B, K, V], same dtype as logits, strides in elements, V contiguous.
 * temperature > 0; tau as for csd_verify.  workspace: csd_sampled_workspace_bytes bytes,
 * 16-byte aligned, no initialisation needed.  diag: NULL or a HOST struct of optional
 * device arrays.  Six kernel launches (statistics, decision, two rounds of races and
 * finalisation) or four (one round); csd_step_sampled appends the memory update of the recorded
 * pairs in (b,i) order.
 * Errors as csd_verify; also INVALID_ARG for temperature <= 0 or NaN.  Asynchronous. */
typedef struct {
    float    *alpha;     /* [B,K]   min(1, p(d)/q(d))                                        */
    uint8_t  *accepted;  /* [B,K]   1 where r <= alpha                                       */
    int32_t  *t_star;    /* [B,K]   residual draw where one was made (see above), else -1     */
    float    *lse_p;     /* [B,K+1] ln sum_v exp(z_v / T)                                    */
    float    *lse_q;     /* [B,K]   ln sum_v exp(y_v / T)                                    */
    float    *score;     /* [B,K]   exp(z_d - z_t*) where the test failed (NaN elsewhere)    */
    uint32_t *cnt;       /* [B,K]   memory count of (d, t*) at the start of the step         */
    int32_t  *bonus;     /* [B]     the draw from p_K where one was made, else -1            */
} csd_sampled_diag_t;

size_t csd_sampled_workspace_bytes(int B, int K, int V, csd_dtype_t dtype);
/* Expert knob, process-wide: 0 = automatic (above), 1 = always one round of draws, 2 = always two.  Outputs do
 * not depend on it.  Host function; INVALID_ARG outside 0..2. */
csd_status_t csd_sampled_set_rounds(int mode);
/* Kernel launches of one csd_step_sampled call of this shape under the current setting (7 or 5; csd_verify_sampled
 * makes one fewer); 0 for an unsupported shape.  Host function. */
int csd_sampled_launches(int B, int K, int V, csd_dtype_t dtype);

csd_status_t csd_verify_sampled(const void *logits, const void *draft_logits, csd_dtype_t dtype,
                                int B, int K, int V,
                                int64_t stride_b, int64_t stride_k, int64_t draft_stride_b, int64_t draft_stride_k,
                                const int32_t *draft, const float *r_accept, uint64_t seed, float temperature,
                                const csd_ocm_t *ocm, float tau,
                                int32_t *accept_len, int32_t *next_token, uint8_t *rescued_mask,
                                int32_t *rej_draft, int32_t *rej_target,
                                const csd_sampled_diag_t *diag,
                                void *workspace, size_t workspace_bytes, void *stream);

csd_status_t csd_step_sampled(const void *logits, const void *draft_logits, csd_dtype_t dtype,
                              int B, int K, int V,
                              int64_t stride_b, int64_t stride_k, int64_t draft_stride_b, int64_t draft_stride_k,
                              const int32_t *draft, const float *r_accept, uint64_t seed, float temperature,
                              csd_ocm_t *ocm, float tau,
                              int32_t *accept_len, int32_t *next_token, uint8_t *rescued_mask,
                              int32_t *rej_draft, int32_t *rej_target,
                              const csd_sampled_diag_t *diag,
                              void *workspace, size_t workspace_bytes, void *stream);

/* ---- the step taken straight from the LM head: logits never stored -------------------------------
 *
 * Algorithm 1 gets the distributions of all gamma + 1 positions from ONE parallel target pass, and the paper's
 * starting point is that this pass is bound by memory traffic (Introduction).  Its last operation is the LM
 * head, z[b, i, v] = sum_h hidden[b, i, h] * weight[v, h]; these entry points take the inputs of that operation
 * instead of its result.  A tensor-core GEMM produces the logits tile by tile and reduces each tile at once to
 * the row statistics of csd_verify (max, lowest arg-max, sum of exponentials) and the draft tokens' logits, so
 * the [B, K+1, V] logit tensor is neither written nor read; everything after that is csd_verify / csd_step.
 *
 * hidden : [B, K+1, H] bf16, dense, 16-byte aligned.   weight : [V, H] bf16, dense, 16-byte aligned.
 * Shapes: H a multiple of 64; any B, K <= 32, V.  Logit rows are processed in groups of 256, and the weight
 * matrix is streamed once per group: up to 256 rows the step is bound by that stream, beyond by the contraction.
 * The logits are the fp32 tensor-core accumulations of the exact bf16 products, NOT rounded to bf16: they
 * differ from an exactly summed product by at most about 2^-16 * ||hidden row|| * max ||weight row|| (see
 * the tests), so an arg-max or a gate decision that hangs on a smaller difference may come out either way;
 * everything else is the result csd_verify would give on the exact logits.  diag as for csd_verify.
 * workspace: csd_lmhead_workspace_bytes bytes, 16-byte aligned, no initialisation needed.
 * Three launches (GEMM + statistics, decisions, memory update); asynchronous.  With csd_set_overlap on, the
 * GEMM of up to 128 logit rows (one block per SM) is launched programmatically: behind this library's own kernels on the same stream it starts, and streams
 * the weight matrix, while the decisions and the update of the step before finish; it reads only this step's
 * inputs until its first store into the workspace and waits for everything before it on the stream ahead of that,
 * so back-to-back steps may share one workspace.  csd_set_overlap's condition applies to hidden, weight and
 * draft: complete before the step before was enqueued.  A wait inside the GEMM kernel that does not end within
 * about two seconds raises CSD_FLAG_INTERNAL (debug_site 30 or 31).
 * Errors as csd_verify; UNSUPPORTED for H not a multiple of 64; CUDA if the driver offers no
 * tensor-map encoder. */
size_t csd_lmhead_workspace_bytes(int B, int K, int H, int V);
csd_status_t csd_verify_lmhead(const void *hidden, const void *weight, int B, int K, int H, int V,
                               const int32_t *draft, const csd_ocm_t *ocm, float tau,
                               int32_t *accept_len, int32_t *next_token, uint8_t *rescued_mask,
                               int32_t *rej_draft, int32_t *rej_target, const csd_diag_t *diag,
                               void *workspace, size_t workspace_bytes, void *stream);
csd_status_t csd_step_lmhead(const void *hidden, const void *weight, int B, int K, int H, int V,
                             const int32_t *draft, csd_ocm_t *ocm, float tau,
                             int32_t *accept_len, int32_t *next_token, uint8_t *rescued_mask,
                             int32_t *rej_draft, int32_t *rej_target, const csd_diag_t *diag,
                             void *workspace, size_t workspace_bytes, void *stream);
/* How the vocabulary is cut for this shape: blocks of the GEMM grid, columns per tile, number of tiles and
 * tiles per block.  Host function; for reports and tests. */
csd_status_t csd_lmhead_shape(int B, int K, int H, int V, int *grid, int *tile_cols, int *tiles, int *tiles_per_block);
/* 1 if the GEMM of this shape would run as pairs of blocks (see csd_lmhead_set_pairing), else 0.  Host function. */
int csd_lmhead_uses_pairs(int B, int K);
/* Expert knobs, process-wide.  kblocks_per_stage: how many 64-column k-blocks travel through the shared-memory
 * ring together (1 to 4; 0 = automatic; the pair kernel always takes 1).  More per stage means longer contiguous
 * reads of each weight row and fewer, larger stages.  mma_cols: the N of one tensor-core instruction, a multiple
 * of 16 from 16 to 256 (0 = automatic: the widest that gives every block the same number of tiles); a tile has
 * mma_cols columns with one block per SM and 2 mma_cols with pairs.  Results do not depend on either beyond the
 * rounding order of the sums.  Host function; INVALID_ARG outside these ranges. */
csd_status_t csd_lmhead_set_tuning(int kblocks_per_stage, int mma_cols);
/* Expert knob, process-wide: which GEMM kernel runs.  0 = automatic (the default), 1 = one block per SM, each on
 * its own vocabulary tiles with up to 256 logit rows; 2 = pairs of blocks on neighbouring SMs (thread-block clusters
 * of two), each block holding half of the logit rows against a tile twice as wide, which halves the share of the
 * hidden states in an SM's shared-memory traffic.  Automatic takes pairs for more than 128 logit rows.  Results
 * are the same up to which vocabulary ranges the per-block partial sums cover (the last bits of s, lse and the
 * probabilities).  csd_lmhead_shape reports the cut of the kernel that would run; for pairs, tile_cols is the
 * width of a pair's tile and tiles_per_block the tiles per pair.  A wait that runs out in the pair kernel reports
 * debug_site 31.  Host function; INVALID_ARG outside 0..2. */
csd_status_t csd_lmhead_set_pairing(int mode);

/* csd_step for callers whose tensors live in HOST memory (pinned memory gives
 * the full copy rate).  Copies logits and draft to `staging`, runs the step, and
 * copies accept_len, next_token and rescued_mask back; returns after the stream
 * has been synchronised, so the host outputs are valid on return.
 * logits_host is dense [B,K+1,V].  staging: DEVICE scratch of at least
 * csd_host_staging_bytes(B,K,V,dtype) bytes, 256-byte aligned; it needs no
 * initialisation and may be reused. */
size_t csd_host_staging_bytes(int B, int K, int V, csd_dtype_t dtype);
csd_status_t csd_step_host(const void *logits_host, csd_dtype_t dtype, int B, int K, int V,
                           const int32_t *draft_host, csd_ocm_t *ocm, float tau,
                           int32_t *accept_len_host, int32_t *next_token_host,
                           uint8_t *rescued_mask_host,
                           void *staging, size_t staging_bytes, void *stream);

/* ---- memory life cycle: checkpoint / restore (prior calibration, Sec. 4.2 Phase 1) ---- */

/* Write every stored pair to the DEVICE arrays d, t, cnt (capacity `cap` triples,
 * order unspecified) and the number of stored pairs to the HOST word *n_out.
 * Synchronises `stream`.  If more than `cap` pairs are stored only `cap` are
 * written and *n_out still reports the total. */
csd_status_t csd_ocm_export(const csd_ocm_t *ocm, int32_t *d, int32_t *t, uint32_t *cnt,
                            uint64_t cap, uint64_t *n_out, void *stream);

/* Add n weighted pairs: count[(d[j], t[j])] += cnt[j] (saturating), admission as
 * in csd_ocm_update.  Loading a table built offline (Phase 1) or restoring an
 * export is csd_ocm_reset followed by csd_ocm_import.  Device arrays; asynchronous. */
csd_status_t csd_ocm_import(csd_ocm_t *ocm, const int32_t *d, const int32_t *t, const uint32_t *cnt,
                            uint64_t n, void *stream);

/* Ageing, an opt-in alternative to "frozen once full" (the paper's Sec. 4.2 lets the memory
 * evolve online and names no forgetting rule; this one is the library's): every count is
 * halved, rounding down, and the pairs that reach zero are forgotten, which frees their room
 * for new pairs.  The result depends only on the stored set.  The serving loop calls it at
 * the cadence it wants (say every N steps), stream-ordered like any call; n_dropped and the
 * step statistics are untouched.  Two launches; asynchronous; nothing is allocated. */
csd_status_t csd_ocm_age(csd_ocm_t *ocm, void *stream);

/* dst += src: every pair of src, in ascending (draft, target) order, is added to dst with its
 * count as the weight, under the admission rule of csd_ocm_update (common pairs add, saturating;
 * new pairs enter while dst has room, else that entry is dropped and counted once).  Combining
 * the tables of several calibration runs (Sec. 4.2, Phase 1) is a sequence of merges.  Both
 * memories live on the same device; src is unchanged.  Allocates temporaries; synchronises. */
csd_status_t csd_ocm_merge(csd_ocm_t *dst, const csd_ocm_t *src, void *stream);

/* The memory as a file: what calibration hands to deployment (Sec. 4.2: the table is built
 * offline, then loaded and kept evolving online).  Little-endian layout:
 *     offset  0  char     magic[8]   "CSDOCM\0\0"
 *             8  uint32   version    1
 *            12  uint32   lambda
 *            16  uint64   n_slots    capacity of the table that was saved
 *            24  uint64   n          number of stored pairs
 *            32  uint64   n_dropped  occurrences dropped so far (informational)
 *            40  uint8    reserved[24]  zero
 *            64  n records { int32 draft; int32 target; uint32 count; }, strictly ascending
 *                in (draft, target)
 * csd_ocm_save writes it (synchronises `stream`; host path).  csd_ocm_load creates a new
 * memory on `device` with the file's lambda and n_slots slots (0 = as saved) and adds the
 * records in file order, so a smaller table keeps the first n_slots/2 pairs in (draft, target)
 * order and counts the rest as dropped.  Errors: IO (cannot open / short / bad magic, version
 * or order), plus those of csd_ocm_create. */
csd_status_t csd_ocm_save(const csd_ocm_t *ocm, const char *path, void *stream);
csd_status_t csd_ocm_load(csd_ocm_t **out, const char *path, uint64_t n_slots, int device);

/* Copy the statistics block to the HOST struct.  Synchronises `stream`. */
csd_status_t csd_ocm_stats(const csd_ocm_t *ocm, csd_stats_t *host_out, void *stream);

/* ---- helpers ---- */

/* (float) log((double) tau): the threshold the gate of Eq. 3 compares against.
 * -inf for tau == 0.  Host function. */
float csd_scg_threshold(float tau);

/* Launch shape a step of this size uses under the current csd_set_overlap setting: grid blocks (each owns an equal contiguous
 * share of the logits), threads per block, elements per chunk (the run of one logit row
 * that a warp reduces at a time) and partial results kept per logit row.  Host function;
 * for reports and tests. */
csd_status_t csd_launch_shape(int B, int K, int V, csd_dtype_t dtype,
                              int *grid, int *block, int *chunk_elems, int *parts_per_row);

/* Expert knob, process-wide: override the automatic work split.  chunk_bytes: bytes of
 * one logit row reduced by a warp at a time (multiple of 512; 0 = automatic, 4 to 32 KiB);
 * ctas_per_sm: blocks of the persistent grid per SM (0 = automatic: 4, or 1 with
 * csd_set_overlap); block_threads:
 * threads per block (multiple of 32, at most 1024; 0 = automatic, 256).  Changes
 * csd_workspace_bytes: size workspaces after calling it.  Results stay
 * bit-reproducible for a fixed setting; the low-order bits of the sums s may differ
 * between settings (different summation trees).  Host function. */
csd_status_t csd_set_tuning(int chunk_bytes, int ctas_per_sm, int block_threads);

/* Process-wide, off by default: for callers that issue steps back to back.  When on,
 * csd_verify / csd_step launch with programmatic stream serialization: the kernel may
 * start, and stream logits, while earlier kernels on the stream are still running; it
 * waits for the previous step before it first touches the memory or any output.  If
 * that previous step was launched on the same stream with the same workspace, memory,
 * output buffers and shape (and no other call of this library came between), the wait
 * is on a completion count that the previous step leaves in the workspace; in every
 * other case it is the hardware's wait for the previous kernel on the stream to
 * retire.  The automatic launch shape also changes: one block per SM and launch
 * instead of four, so that several steps are resident at a time (the low-order bits of
 * the diagnostic sums s may therefore differ from those with overlap off; all decisions
 * are identical).  Turn it on only if the logits and draft tokens of every step were
 * complete (their producer finished, and a normal stream dependency, event or host
 * synchronisation passed) BEFORE the step before it was enqueued: a step reads its inputs
 * before it waits for its predecessor on the stream, and CUDA makes a predecessor's writes
 * visible only after that wait.  Back-to-back steps over inputs that are already resident
 * qualify; a kernel that writes a step's inputs between two steps does not -- a decode loop
 * with the model's forward pass between steps keeps the default.  Steps that share a memory
 * or output buffers are issued on one stream (but see csd_ocm_set_shared).  Changing the
 * setting, or csd_set_tuning, changes the layout of the scratch inside a workspace; the
 * library notices a workspace that last held another layout and clears it before use, so
 * no re-initialisation is needed.  Host function. */
csd_status_t csd_set_overlap(int enable);

const char *csd_status_string(csd_status_t status);

#ifdef __cplusplus
}
#endif
#endif /* CSD_H_ */
