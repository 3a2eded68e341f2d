/*
 * libfopd -- fused loss path of freshness-aware on-policy distillation (f-OPD)
 * for NVIDIA B200 (sm_100a).  C ABI: plain pointers and sizes, no C++ or
 * framework types.
 *
 * What the path computes (citations are to the f-OPD paper):
 *
 *   per token row n (student logits S[n,:], teacher logits T[n,:], stored token
 *   y_n, behaviour log-prob b_n = log pi^{r(i)}(y_n), loss mask):
 *     lse_s, lse_t   log-normalisers of the softmax policies          (Sec. 3.1)
 *     lp_s, lp_t     log-probabilities of y_n under student / teacher  (Sec. 4.1)
 *     kl_n           token loss of Eq. 12, read as the full-vocabulary reverse
 *                    KL  sum_v p_s(v) (log p_s(v) - log p_t(v))
 *     rho_n, k3_n    policy ratio exp(lp_s - b_n) and the per-token integrand
 *                    rho log rho - rho + 1 of the rollout drift D_roll (Eq. 10)
 *   per sample i (rows with mask = 1 are its aligned positions U_i):
 *     D_roll_i, l_i  means of k3_n and kl_n over U_i                (Eq. 10, 12)
 *     f_i            exp(-alpha sqrt(D_roll_i) - beta sqrt(D_sup_i)) / (tau_i+1)
 *                                                                      (Eq. 11)
 *     w_i            max(f_i - xi, 0), the ReLU gate                   (Eq. 13)
 *     m_i            |U_i| / H_i, the alignment ratio             (Algorithm 1)
 *   per batch:
 *     L = (1/B) sum_i w_i (l_i + lambda D_roll_i)          (Eq. 16, Algorithm 1)
 *     dL/dS[n,v] with w_i held constant.
 *
 * Calling sequence for one batch of B samples supplied in one or more chunks of
 * token rows (rows of a sample are contiguous, in order, within and across
 * chunks):
 *
 *     zero acc[B,4], loss_acc[B,2], status[1]
 *     for each chunk:  fopd_token_stats(...)      measurement phase of Algorithm 1
 *     fopd_sample_freshness(...)                  Eq. 11, Eq. 13
 *     for each chunk:  fopd_loss_fwd_bwd(...)     Eq. 16 and its gradient
 *     fopd_loss_finalize(...)
 *     fopd_check_status(...)
 *
 * (fopd_token_stats_student may take the place of fopd_token_stats: the
 * measurement phase needs the student rows only; the loss calls then get no
 * row_ws.)
 *
 * Memory and ownership.  Unless a parameter says HOST, every pointer is a DEVICE
 * pointer to memory the caller owns; the library keeps no pointer after a call
 * returns.  Where a call needs temporary device memory
 * that the caller did not supply (see row_ws) it takes it from a stream-ordered
 * memory pool of its own on the caller's stream and returns it there.  All
 * work is enqueued on `stream` (a cudaStream_t passed as void*, NULL = default
 * stream) and the call returns without synchronising, except
 * fopd_check_status and fopd_step_host.
 *
 * Process-wide state (all of it; none is read from the environment):
 *   - one memory pool per device for those temporaries.  It keeps what it has
 *     grown to (a few bytes per token row of the largest chunk seen) until
 *     fopd_release_device_memory;
 *   - the launch shape chosen for fopd_loss_fwd_bwd(row_ws = NULL) per (device,
 *     dtype, vocabulary), made on first use and cached: fopd_loss_fwd_bwd_plan
 *     reads it, fopd_loss_fwd_bwd_set_plan sets it;
 *   - two streams and a few events per device used by fopd_step_host, made on
 *     its first call, with a lock that lets one host-buffer step run at a time
 *     per device; fopd_release_device_memory destroys them;
 *   - the fixed scratch array of fopd_token_stats_static and its cached device
 *     address per device.
 * Calls with disjoint buffers may run concurrently from several host threads
 * and on several streams.
 *
 * Errors.  Every function returns FOPD_OK or a negative fopd_status found on
 * the host before anything is enqueued.  Conditions only visible on the device
 * (a token or sample id out of range, tau < 0, H <= 0) never trap: the kernel
 * ORs a bit into *status (if status is not NULL), treats the row as masked or
 * the sample as invalid, and carries on.
 */
#ifndef FOPD_H_
#define FOPD_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define FOPD_VERSION 201

typedef enum { FOPD_BF16 = 0, FOPD_F32 = 1 } fopd_dtype;

/*
 * Form of the token loss l(pi_theta, pi_teacher) of Eq. 12, which the paper leaves generic.
 *
 *   FOPD_LOSS_FULL_KL     kl_n = sum_v p_s(v) (log p_s(v) - log p_t(v)), the reverse KL over the
 *                         whole vocabulary (the default everywhere in this header).
 *   FOPD_LOSS_SAMPLED_KL  l_n = rho_n (log p_s(y_n) - log p_t(y_n)) on the stored token y_n,
 *                         rho_n = pi^t(y_n) / pi^r(y_n): the sampled-token reverse KL with an
 *                         importance ratio of the setup Sec. 5 says the experiments follow
 *                         (Appendix B's sampled-token objectives).  Its expectation over y_n
 *                         drawn from the behaviour policy is kl_n.  In the gradient the ratio
 *                         carries the derivative and the log-ratio is a constant (the reward of
 *                         a policy-gradient step):
 *                           dlogits[n,v] = coef_i rho_n ( (log p_s(y_n) - log p_t(y_n))
 *                                          + lambda d_n ) ( 1[v = y_n] - p_s(v) ),
 *                         which needs the student row only.
 */
typedef enum { FOPD_LOSS_FULL_KL = 0, FOPD_LOSS_SAMPLED_KL = 1 } fopd_loss_kind;

typedef enum {
  FOPD_OK = 0,
  FOPD_ERR_NULL = -1,   /* a required pointer is NULL                          */
  FOPD_ERR_ALIGN = -2,  /* logits base or row pitch not 16-byte aligned         */
  FOPD_ERR_SIZE = -3,   /* negative size, row_stride < vocab, vocab too large   */
  FOPD_ERR_DTYPE = -4,  /* dtype is neither FOPD_BF16 nor FOPD_F32              */
  FOPD_ERR_PARAM = -5,  /* alpha/beta negative or a parameter not finite        */
  FOPD_ERR_CUDA = -6,   /* a CUDA runtime call failed (launch, allocation)      */
  FOPD_ERR_ALIAS = -7,  /* dlogits overlaps student or teacher                  */
  FOPD_ERR_DEVICE = -8, /* fopd_check_status: the device status word is non-zero */
  FOPD_ERR_KIND = -9    /* loss_kind unknown, or not supported by this entry point */
} fopd_status;

/* Bits ORed into the device status word. */
#define FOPD_DEV_BAD_TOKEN 1    /* mask = 1 row with token outside [0, vocab)   */
#define FOPD_DEV_BAD_SAMPLE 2   /* row with sample id outside [0, B)            */
#define FOPD_DEV_BAD_TAU 4      /* staleness < 0                                */
#define FOPD_DEV_BAD_LENGTH 8   /* seq_len <= 0 or aligned count > seq_len      */
#define FOPD_DEV_TIMEOUT 16     /* a bounded in-kernel wait ran out; results of
                                   that call are not to be trusted               */

/* alpha, beta >= 0 scale the two drift diagnostics (Eq. 11); xi is the gate
 * threshold (Eq. 13); lambda weights the rollout anchor (Eq. 16).  The paper
 * gives no values; they are run-time parameters. */
typedef struct {
  float alpha, beta, xi, lambda;
} fopd_params;

/* One chunk of token rows.  student/teacher: [n_rows, vocab] row-major with a
 * pitch of row_stride elements (row_stride >= vocab), same dtype; base address
 * and pitch in bytes must be multiples of 16.  Rows with mask = 0 (padding,
 * tool output) are never read.  Logits must be finite.  The sweeps subtract the
 * row maximum before scaling and form log-probabilities and the KL from the
 * maxima and the logs of the sums separately, so their accuracy (~1e-6) does
 * not depend on how far the logits are from zero; only the stored
 * log-normalisers themselves carry their fp32 rounding (6e-8 * |lse|). */
typedef struct {
  const void *student;
  const void *teacher;
  const float *behav_logprob; /* [n_rows] log pi_behaviour(y_n)                 */
  const int32_t *tokens;      /* [n_rows] 0 <= y_n < vocab                      */
  const uint8_t *mask;        /* [n_rows] 1 = aligned response token            */
  const int32_t *sample_id;   /* [n_rows] 0 <= id < B, non-decreasing           */
  int64_t n_rows;
  int64_t vocab;
  int64_t row_stride;
  int32_t dtype;              /* fopd_dtype                                     */
  int32_t loss_kind;          /* fopd_loss_kind; the same for every chunk and call of a batch */
} fopd_chunk;

/* Columns of the per-row workspace row_ws[n_rows, 4] (fp32). */
#define FOPD_WS_LSE_S 0
#define FOPD_WS_LSE_T 1
#define FOPD_WS_KL 2 /* FOPD_LOSS_SAMPLED_KL: log p_s(y_n) - log p_t(y_n) instead */
#define FOPD_WS_D 3 /* d_n = lp_s - b_n = log rho_n */

/* Columns of acc[B, 4] (fp64): aligned-row count, sum of k3, sum of kl, rows seen. */
#define FOPD_ACC_CNT 0
#define FOPD_ACC_K3 1
#define FOPD_ACC_KL 2
#define FOPD_ACC_ROWS 3

/*
 * Per-token statistics of one chunk and their per-sample sums: one streaming
 * pass over the student and teacher rows (online max / sum-exp), the gather of
 * the stored token, the Eq. 12 token loss and the Eq. 10 drift integrand.
 *
 *   lp_s, lp_t, kl, ratio  [n_rows] fp32 outputs, any may be NULL.  Rows with
 *                          mask = 0 or a bad id get exactly 0.  kl is the token loss
 *                          in the chunk's loss_kind (and so is the sum in acc).
 *   row_ws                 optional [n_rows, 4] fp32 output (columns above),
 *                          16-byte aligned; pass it to fopd_loss_fwd_bwd for
 *                          the same chunk to let that call skip its own
 *                          reduction sweep.  NULL: a temporary of the same size
 *                          is taken from the stream-ordered allocator.
 *   acc                    [B, 4] fp64, ADDED to (the caller zeroes it before
 *                          the first chunk of a batch).  The sums are formed in
 *                          a fixed order, so results are reproducible bit for bit.
 *   status                 device int32 status word, or NULL.
 */
int fopd_token_stats(const fopd_chunk *chunk /* HOST */, int32_t B, float *lp_s,
                     float *lp_t, float *kl, float *ratio, float *row_ws,
                     double *acc, int32_t *status, void *stream);

/*
 * The student's half of fopd_token_stats: what the measurement loop of Algorithm 1
 * needs and no more.  The rollout drift (Eq. 10), the freshness score (Eq. 11) and
 * the gate (Eq. 13) depend on the student's and the behaviour policy's
 * log-probabilities of the stored tokens only, so this call reads the student rows
 * alone (V * e bytes per aligned row instead of 2 * V * e) and never touches
 * chunk->teacher, which may be NULL.  acc gets the count, the k3 sum and the row
 * count; its FOPD_ACC_KL column is left as it is, so fopd_sample_freshness reports
 * l_distill = 0 for such a batch.  The loss phase then runs fopd_loss_fwd_bwd with
 * row_ws = NULL (this call leaves no row statistics behind): 4 * V * e bytes per
 * differentiated token for the whole step instead of 5 * V * e.
 *
 *   lp_s, ratio   [n_rows] fp32 outputs, either may be NULL; exactly 0 for rows
 *                 with mask = 0 or a bad id.
 *   acc, status, stream, errors, the temporary: as for fopd_token_stats.
 */
int fopd_token_stats_student(const fopd_chunk *chunk /* HOST */, int32_t B, float *lp_s,
                             float *ratio, double *acc, int32_t *status, void *stream);

/*
 * fopd_token_stats for callers that must not allocate device memory.  (The
 * paper has no counterpart; this is an interface convenience.)
 *
 * Who needs it: a trainer that has handed all of the GPU's memory to its own
 * allocator, so that the CUDA memory pool fopd_token_stats(row_ws = NULL) draws
 * from may have nothing left; and code with a strict no-allocation rule inside
 * its steady-state loop, where an allocation could stall on the device or fail
 * in the middle of a step.  Such callers would otherwise have to carve a
 * row_ws buffer out of their own memory.
 *
 * Same arguments, outputs and results as fopd_token_stats without the row_ws
 * parameter: the per-row scratch lives in a fixed array compiled into the
 * library, FOPD_STATIC_MAX_ROWS * 16 bytes = 1 MiB for the rows plus
 * FOPD_STATIC_MAX_SAMPLES * 16 bytes = 256 KiB for the samples' row ranges, on
 * every GPU that loads the library, held until the process exits.  The call makes no cudaMalloc,
 * cudaFree or other allocating call.
 *
 *   - chunk->n_rows > FOPD_STATIC_MAX_ROWS or B > FOPD_STATIC_MAX_SAMPLES returns
 *     FOPD_ERR_SIZE and enqueues nothing; split the chunk (or the batch).
 *   - The first call on each device looks the array's device address up
 *     (cudaGetSymbolAddress, with that device current) and caches it.  With
 *     CUDA's lazy module loading that first call is also what loads the part of
 *     the library that holds the array and these kernels onto the device, which
 *     does reserve device memory once: make the first call on each device
 *     outside any stream capture and before the rest of the device's memory is
 *     handed to another allocator.  If it fails it returns FOPD_ERR_CUDA and
 *     can be repeated.
 *   - All calls on a device share the two arrays, which still hold the previous
 *     call's values.  The caller has nothing to clear: each call overwrites the
 *     entries of all its rows and samples before it reads them.  Two calls whose kernels can
 *     overlap on the GPU (different streams, or the same entry point from two
 *     threads) race on the array; order them on one stream.
 */
#define FOPD_STATIC_MAX_ROWS 65536
#define FOPD_STATIC_MAX_SAMPLES 16384
int fopd_token_stats_static(const fopd_chunk *chunk /* HOST */, int32_t B, float *lp_s,
                            float *lp_t, float *kl, float *ratio, double *acc,
                            int32_t *status, void *stream);

/*
 * Per-sample freshness (Eq. 11), ReLU gate (Eq. 13), alignment ratio and the
 * per-token weight coef_i = w_i / (B |U_i|) that fopd_loss_fwd_bwd applies.
 * A sample with no aligned row, seq_len <= 0 or staleness < 0 is invalid:
 * f = w = m = coef = 0 (Algorithm 1, the |U| = 0 branch).
 *
 *   acc        [B, 4] fp64 from fopd_token_stats (all chunks done)
 *   staleness  [B] int32 tau_i = t - r(i);  seq_len [B] int32 H_i
 *   d_sup      [B] fp32 supervision drift D_sup_i, or NULL for 0 (teacher and
 *              context unchanged since grading); +infinity marks a sample
 *              without aligned supervision positions: invalid
 *   f, w, d_roll, l_distill, m_align, coef   [B] fp32 outputs; coef is
 *              required, the others may be NULL
 *   buffer_means  optional [2] fp32: mean f_i and mean m_i over the B samples
 *              (the buffer statistics of Eq. 14)
 */
int fopd_sample_freshness(const double *acc, const int32_t *staleness,
                          const int32_t *seq_len, const float *d_sup, int32_t B,
                          fopd_params p, float *f, float *w, float *d_roll,
                          float *l_distill, float *m_align, float *coef,
                          float *buffer_means, int32_t *status, void *stream);

/*
 * Fused loss forward + backward for one chunk (Eq. 16 with w_i constant).  For
 * an aligned row n of a sample with coef_i != 0:
 *
 *   dlogits[n,v] = coef_i { p_s(v) [ (log p_s(v) - log p_t(v)) - kl_n ]
 *                           + lambda rho_n d_n ( 1[v = y_n] - p_s(v) ) }
 *
 * (chunk->loss_kind = FOPD_LOSS_SAMPLED_KL: the formula given with fopd_loss_kind; with
 * row_ws that call is one pass that reads S and writes dlogits, without it the statistics
 * sweep runs first.)  Every other row of dlogits (masked, padded, bad id, gated or invalid sample)
 * is written as +0 and its logits are not read.  The per-sample sums of kl and
 * k3 over the rows this call differentiated are ADDED to loss_acc.
 *
 *   coef      [B] fp32 from fopd_sample_freshness
 *   row_ws    the workspace fopd_token_stats wrote for THIS chunk, or NULL.
 *             With it the call is one streaming pass (read S, read T, write
 *             dlogits).  Without it the kernel stages each row on chip, does
 *             the reduction sweep and the gradient sweep from there, and still
 *             reads S and T from memory once.
 *   dlogits   [n_rows, vocab] with the same dtype and pitch as student; must
 *             not overlap student or teacher
 *   loss_acc  [B, 2] fp64 {sum kl, sum k3}, ADDED to; caller zeroes per batch
 */
int fopd_loss_fwd_bwd(const fopd_chunk *chunk /* HOST */, int32_t B,
                      const float *coef, const float *row_ws, fopd_params p,
                      void *dlogits, double *loss_acc, int32_t *status,
                      void *stream);

/*
 * Launch shape fopd_loss_fwd_bwd(row_ws = NULL) uses on the current device for
 * a vocabulary and dtype: CTAs per thread-block cluster (one cluster per row),
 * threads per CTA, clusters resident at once and dynamic shared memory per CTA
 * (three slice buffers that rows' copies land in; the rows being worked on are
 * held in registers).  All outputs are HOST pointers and may be NULL.
 * *cluster_size = 0 means that the call runs the statistics sweep and the
 * streaming gradient sweep instead: no on-chip shape fits (a CTA's slice of a row
 * must fit its threads' registers: bf16 rows of up to about 295,000 logits in
 * sixteen CTAs), or the row is so long that fewer than two thirds of the SMs
 * would hold a resident CTA.  The shape is chosen once per (device, dtype,
 * vocabulary) from cudaOccupancyMaxActiveClusters -- the cluster size that keeps
 * the most CTAs resident -- and cached.
 */
int fopd_loss_fwd_bwd_plan(int32_t dtype, int64_t vocab, int32_t *cluster_size,
                           int32_t *block_threads, int32_t *resident_clusters,
                           int32_t *smem_bytes);

/*
 * Sets that launch shape for (current device, dtype, vocab) instead of letting
 * the library choose: cluster_size > 0 pins the CTAs per cluster (FOPD_ERR_SIZE if
 * a cluster of that size cannot hold a row of this vocabulary on this device,
 * in which case the plan is left as it was), cluster_size < 0 makes the call
 * always run the two streaming sweeps, cluster_size = 0 goes back to the
 * library's own choice.  Takes effect for calls made after it returns.
 */
int fopd_loss_fwd_bwd_set_plan(int32_t dtype, int64_t vocab, int32_t cluster_size);

/*
 * After the last chunk: per_sample_loss[i] = w_i (l_i + lambda D_roll_i) with
 * l_i, D_roll_i = loss_acc[i] / acc[i].cnt, and loss_out[0] = (1/B) sum_i of
 * it (Eq. 16; Algorithm 1 divides by the minibatch size, gated samples
 * included).  per_sample_loss may be NULL.
 */
int fopd_loss_finalize(const double *loss_acc, const double *acc, const float *w,
                       int32_t B, fopd_params p, float *per_sample_loss,
                       float *loss_out, void *stream);

/*
 * Row-wise divergence diagnostics of one chunk: for every row with mask = 1 the
 * full-vocabulary KL(p || q), p = softmax(first[n,:]), q = softmax(second[n,:]),
 * and the entropy of p.  With first = teacher logits under the current context
 * and second = teacher logits under the context stored at grading time, and
 * mask = the supervision-aligned positions U^sup, the per-sample mean of the KL
 * is the supervision drift D_sup of Eq. 10 (second row).  With first = student
 * and second = teacher it is the token loss of Eq. 12 again, and the entropy is
 * the response entropy the paper logs as a monitoring signal (Appendix B).
 *
 *   first, second   [n_rows, vocab] at a pitch of row_stride elements, same
 *                   layout rules as fopd_chunk
 *   mask, sample_id [n_rows]; rows with mask = 0 are not read and get 0
 *   kl, entropy     [n_rows] fp32 outputs, either may be NULL
 *   acc             [B, 3] fp64 {rows with mask = 1, sum kl, sum entropy} per
 *                   sample, ADDED to in a fixed order (caller zeroes per batch)
 */
int fopd_row_divergence(const void *first, const void *second, const uint8_t *mask,
                        const int32_t *sample_id, int64_t n_rows, int64_t vocab,
                        int64_t row_stride, int32_t dtype, int32_t B, float *kl,
                        float *entropy, double *acc, int32_t *status, void *stream);

/*
 * Per-sample supervision drift and alignment ratio from the sums of
 * fopd_row_divergence: d_sup[i] = sum kl / |U_i^sup| (Eq. 10), m_sup[i] =
 * |U_i^sup| / H_i (Algorithm 1), mean_entropy[i].  A sample with no aligned
 * supervision position gets d_sup = +infinity and m_sup = 0; passed to
 * fopd_sample_freshness that makes the sample invalid (f = w = m = coef = 0),
 * which is Algorithm 1's |U^sup| = 0 branch.  Outputs [B] fp32, any may be NULL.
 */
int fopd_supervision_drift(const double *acc, const int32_t *seq_len, int32_t B,
                           float *d_sup, float *m_sup, float *mean_entropy, void *stream);

/*
 * Buffer statistics (Eq. 14) and the adaptive-refresh rule (Eq. 15):
 * means[0..2] = mean f_i, mean m_i^roll, mean m_i^sup over the B samples;
 * refresh when  mean f <= kappa_f  or  mean m^roll < kappa_roll  or
 * mean m^sup < kappa_sup  (operators as the paper prints them), but at most
 * once every min_interval steps (Appendix B uses 200): steps_since_refresh is
 * the number of optimizer steps since the last refresh.
 *
 *   f, m_roll   [B] fp32 from fopd_sample_freshness (f, m_align)
 *   m_sup       [B] fp32 from fopd_supervision_drift, or NULL for m_roll (one
 *               aligned set for both diagnostics)
 *   means       [3] fp32 output or NULL
 *   decision    [2] int32 output: decision[0] = bit 0 freshness condition, bit 1
 *               rollout alignment, bit 2 supervision alignment, bit 3 a
 *               condition holds but the interval has not passed;
 *               decision[1] = 1 if the buffer is to be refreshed now
 */
int fopd_refresh_decision(const float *f, const float *m_roll, const float *m_sup,
                          int32_t B, float kappa_f, float kappa_roll, float kappa_sup,
                          int64_t steps_since_refresh, int64_t min_interval,
                          float *means, int32_t *decision, void *stream);

/*
 * Vocabulary-sharded rows (a tensor-parallel LM head): each holder has the columns
 * [vocab_offset, vocab_offset + shard->vocab) of every row, of a vocabulary of
 * vocab_total columns.  The softmax normalisers of Sec. 4.1 and the sum of Eq. 12
 * split over a partition of the vocabulary: with m_k = max, Z_k = sum e^{x - m_k}
 * and A_k = sum e^{s - m_k}(s - t) over part k,
 *   lse = log sum_k Z_k e^{m_k},   sum_v p_s(v)(s_v - t_v) = sum_k A_k e^{m_k} / sum_k Z_k e^{m_k}.
 * These entry points take FOPD_LOSS_FULL_KL only (FOPD_ERR_KIND otherwise).
 * Calling sequence on every holder, per chunk: fopd_shard_stats -> exchange the
 * partial sums so that every holder has all parts (the caller's job: an all-gather
 * of [n_rows, 8] floats per holder; the library makes no collective call) ->
 * fopd_shard_merge -> (all chunks) fopd_sample_freshness -> per chunk
 * fopd_shard_loss_fwd_bwd -> fopd_loss_finalize.  Every holder computes the same
 * row statistics, sums, freshness and loss (the merge runs in a fixed order, part 0
 * first) and the gradient of its own columns.
 *
 *   shard       DEVICE chunk whose student/teacher point at the shard's first
 *               column of row 0 (row pitch = row_stride elements, base and pitch
 *               16-byte aligned), vocab = columns in this shard; tokens are ids in
 *               the FULL vocabulary; the other arrays as in fopd_chunk
 *   partial     DEVICE [n_rows, 8] fp32 output (16-byte aligned), columns
 *               FOPD_PART_*; rows with mask = 0 are not read and give zeros
 */
#define FOPD_PART_MAX_S 0
#define FOPD_PART_Z_S 1
#define FOPD_PART_A_S 2
#define FOPD_PART_MAX_T 3
#define FOPD_PART_Z_T 4
#define FOPD_PART_TOKEN_S 5 /* student logit of the stored token, if it lies in this shard */
#define FOPD_PART_TOKEN_T 6
#define FOPD_PART_HAS_TOKEN 7 /* 1.0 if it does, else 0.0 */
int fopd_shard_stats(const fopd_chunk *shard, int64_t vocab_offset, int64_t vocab_total,
                     float *partial, void *stream);

/*
 * Merges the parts of every row into the outputs fopd_token_stats gives for
 * unsharded rows, and adds the rows to the per-sample sums.
 *
 *   partials    DEVICE [n_parts, n_rows, 8] fp32, part k from the holder of the
 *               k-th column range (any order of ranges; every column in exactly
 *               one part)
 *   rows        the chunk's per-row arrays (DEVICE) with vocab = vocab_total;
 *               student, teacher and row_stride are ignored
 *   lp_s .. ratio   optional [n_rows] outputs;  row_ws [n_rows, 4] REQUIRED
 *   acc, status as for fopd_token_stats.  A row whose token is found in no part
 *               or in several sets FOPD_DEV_BAD_TOKEN and is treated as masked.
 */
int fopd_shard_merge(const float *partials, int32_t n_parts, const fopd_chunk *rows, int32_t B,
                     float *lp_s, float *lp_t, float *kl, float *ratio, float *row_ws,
                     double *acc, int32_t *status, void *stream);

/*
 * Gradient of the shard's columns (same formula as fopd_loss_fwd_bwd, from the
 * merged row statistics; one streaming pass).  dlogits has the shard's layout
 * (DEVICE, 16-byte aligned, pitch row_stride) and must not overlap the logits.
 * loss_acc may be NULL (the sums do not depend on the shard: every holder that
 * passes it gets the same numbers).
 */
int fopd_shard_loss_fwd_bwd(const fopd_chunk *shard, int64_t vocab_offset, int64_t vocab_total,
                            int32_t B, const float *coef, const float *row_ws, fopd_params p,
                            void *dlogits, double *loss_acc, void *stream);

/*
 * Gives back what the library holds on the current device between calls: trims
 * its memory pool to what pending work still uses and destroys the streams and
 * events of fopd_step_host (both come back on the next call that needs them).
 * Waits for a host-buffer step in progress on that device; synchronise the
 * streams other calls were enqueued on first if all of the pool is to be freed.
 */
int fopd_release_device_memory(void);

/*
 * Self-test of the bounded in-kernel wait.  Every wait on a barrier inside the
 * library's kernels gives up after a fixed number of SM cycles, records
 * FOPD_DEV_TIMEOUT in the status word and lets the kernel end.  This call runs
 * that wait on one CTA against a barrier that is one arrival short, with a
 * limit of limit_cycles SM cycles (0 <= limit_cycles <= 200,000,000): the wait
 * must run out, *status gets FOPD_DEV_TIMEOUT and *waited_cycles (DEVICE int64,
 * may be NULL) the cycles the wait took.  The context stays usable.
 */
int fopd_selftest_bounded_wait(int64_t limit_cycles, int32_t *status, int64_t *waited_cycles,
                               void *stream);

/* Synchronises `stream`, reads the device status word and returns FOPD_OK,
 * FOPD_ERR_DEVICE (word non-zero; *bits_out receives it if not NULL, HOST) or
 * FOPD_ERR_CUDA. */
int fopd_check_status(const int32_t *status, int32_t *bits_out /* HOST */, void *stream);

/*
 * Whole batch from HOST memory: the calling sequence above (statistics for every
 * chunk, freshness, fused loss forward + backward for every chunk, finalize;
 * Algorithm 1's measurement and optimisation phases) with the host<->device
 * copies done by the library.  For callers whose logits live in host memory
 * (pinned memory copies fastest).
 *
 *   chunks      HOST array of n_chunks descriptors whose pointers are HOST
 *               pointers (same layout rules as for device chunks).  The logits
 *               of rows with mask = 0 are not uploaded (they are never read).
 *   staleness, seq_len, d_sup   HOST [B] (d_sup may be NULL)
 *   dlogits     HOST array of n_chunks HOST pointers; dlogits[j] receives
 *               chunk j's gradient, [n_rows_j, vocab] at the chunk's pitch
 *   out         HOST outputs, [B] each (any may be NULL) and loss[1] (required);
 *               status_bits[1] receives the device status word
 *   workspace   DEVICE scratch owned by the caller, 256-byte aligned, at least
 *               fopd_step_host_workspace_bytes(.., resident = 0) bytes.  If it
 *               is at least the resident = 1 size, all logits stay on the device
 *               and are uploaded once, in pieces of up to 256 MiB, on `stream`;
 *               two library-owned streams take each piece's statistics as it
 *               lands, differentiate a sample's rows as soon as its last row
 *               has been measured (coef_i depends on sample i alone, Eq. 11)
 *               and return finished gradient pieces while later rows are still
 *               going up, so both directions of the host link are busy at once.
 *               Otherwise every chunk is uploaded twice (once per phase) and
 *               everything runs on `stream` in order.
 *
 * Host-buffer steps on one device run one at a time (a lock around that device's
 * shared streams); work queued on `stream` before the call is waited for first.
 * Synchronises `stream` before returning.  Returns FOPD_ERR_SIZE if the
 * workspace is too small, FOPD_ERR_DEVICE if the status word is non-zero (the
 * outputs are still written).
 */
typedef struct {
  float *f, *w, *d_roll, *l_distill, *m_align, *per_sample_loss; /* [B] or NULL */
  float *buffer_means;                                            /* [2] or NULL */
  float *loss;                                                    /* [1]         */
  int32_t *status_bits;                                           /* [1] or NULL */
  int64_t *copied_bytes; /* [2] or NULL: bytes this call copied host->device, device->host */
} fopd_host_outputs;

uint64_t fopd_step_host_workspace_bytes(const fopd_chunk *chunks /* HOST */, int32_t n_chunks,
                                        int32_t B, int32_t resident);

int fopd_step_host(const fopd_chunk *chunks /* HOST */, int32_t n_chunks, int32_t B,
                   const int32_t *staleness, const int32_t *seq_len, const float *d_sup,
                   fopd_params p, void *const *dlogits, const fopd_host_outputs *out,
                   void *workspace, uint64_t workspace_bytes, void *stream);

const char *fopd_strerror(int code);
int fopd_version(void);

#ifdef __cplusplus
}
#endif
#endif /* FOPD_H_ */
