/* espo.h -- C ABI of the ESPO early-stopping hot path for NVIDIA B200 (sm_100a).
 *
 * ESPO (Early-Stopping Proximal Policy Optimization) ends a rollout during decoding
 * once a smoothed, normalised regret signal computed from the policy's own logits
 * exceeds a threshold gated by the critic's value estimate, and trains on the
 * truncated prefix as an absorbing failure transition.  This library implements the
 * two data-parallel pieces of that method:
 *
 *   espo_step        one pass of the rollout loop body (Algorithm 1) over a batch of
 *                    logit rows: log-softmax statistics, Philox Gumbel-max sampling,
 *                    surrogate regret (Eq. 6), normalisation (Eq. 9), smoothing (Eq. 10),
 *                    value-gated stop test (Eq. 11), per-trajectory bookkeeping;
 *   espo_advantages  TD errors and GAE (Eq. 4-5) over ragged truncated trajectories with
 *                    the failure transition of Eq. 13.
 *
 * Conventions for every entry point
 *   - "device" pointers are CUDA device memory owned by the caller, on the device that
 *     was current when the state was created; "host" pointers are ordinary memory.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Work is
 *     only enqueued; no entry point synchronises the host unless it says so.
 *   - Every function returns an int: ESPO_OK (0) or a negative ESPO_ERR_* code.
 *     Argument errors are found on the host before anything is launched.  Conditions
 *     found on the device (unusable logit rows, bad slot ids, a wait that ran out) are
 *     recorded in a sticky device status word, never trapped.
 *   - There is no CPU fallback: without a CUDA device the calls return ESPO_ERR_CUDA.
 */
#ifndef ESPO_H_
#define ESPO_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* ---- return codes ------------------------------------------------------------------ */
#define ESPO_OK              0
#define ESPO_ERR_NULL       -1   /* a required pointer was NULL                          */
#define ESPO_ERR_BAD_DTYPE  -2   /* dtype code is not ESPO_F32 / ESPO_BF16                */
#define ESPO_ERR_BAD_SHAPE  -3   /* a size is non-positive, or a stride is shorter than V */
#define ESPO_ERR_ALIGN      -4   /* a pointer is not aligned to its element type          */
#define ESPO_ERR_CAPACITY   -5   /* more rows / tokens than the state or workspace holds  */
#define ESPO_ERR_CUDA       -6   /* a CUDA runtime call failed (see espo_last_cuda_error) */
#define ESPO_ERR_BAD_PARAM  -7   /* a parameter is outside its documented range           */

/* ---- element types of caller buffers ----------------------------------------------- */
#define ESPO_F32   0
#define ESPO_BF16  1

/* ---- sampler ------------------------------------------------------------------------ */
/* Both draw a_t ~ softmax(logits / temperature) exactly, by Gumbel-max with Philox4x32-10
 * noise keyed by (seed; batch_id, trajectory slot, step, index).  They differ in how many
 * draws they need and therefore return different (equally valid) tokens.
 *   FLAT  one draw per vocabulary id: a_t = argmax_a (x_a + G_a).
 *   HIER  the same argmax taken level by level -- first over blocks of 1024 ids scored by
 *         their log-sum-exp, then over sub-blocks of 32 ids inside the winner, then over
 *         the 32 ids -- which needs ~V/1024 + 64 draws per row instead of V.            */
#define ESPO_SAMPLER_FLAT  0
#define ESPO_SAMPLER_HIER  1

/* ---- stop rule (espo_params.stop_mode): the method's own rule and the ablation's replacements (Sec. 6) ---- */
#define ESPO_STOP_ESPO         0   /* z_t > beta * max(V_phi(s_t), eps)            (Eq. 11)          */
#define ESPO_STOP_VALUE_ONLY   1   /* V_phi(s_t) < tau                             (variant D)       */
#define ESPO_STOP_REGRET_ONLY  2   /* z_t > tau                                    (variant E)       */
#define ESPO_STOP_RANDOM       3   /* with probability p_random on every step      (variant F)       */

/* ---- per-trajectory status (espo_state_view: status[]) ------------------------------ */
#define ESPO_ROW_ACTIVE   0
#define ESPO_ROW_STOPPED  1   /* ESPO's rule fired (Eq. 11): failure transition            */
#define ESPO_ROW_EOS      2   /* sampled the end-of-sequence token                          */
#define ESPO_ROW_TMAX     3   /* reached the horizon t_max                                  */
#define ESPO_ROW_BAD      4   /* the logit row held NaN / +inf, or no finite entry          */

/* ---- bits of the sticky device status word (espo_state_status) ---------------------- */
#define ESPO_DEV_BAD_ROW     1u   /* some row was marked ESPO_ROW_BAD                       */
#define ESPO_DEV_BAD_SLOT    2u   /* a row_ids entry was outside [0, capacity)              */
#define ESPO_DEV_TIMEOUT     4u   /* a bounded in-kernel wait ran out; results incomplete   */
                                  /* (the launch's row tickets are left stale: call        */
                                  /* espo_reset_state before the state is used again)      */
#define ESPO_DEV_NAN_VALUE   8u   /* a value estimate was NaN (that row did not stop)       */
#define ESPO_DEV_BAD_LENGTHS 16u  /* espo_advantages: sum(lengths) != total_tokens or L < 0 */

/* Parameters that stay frozen for a whole rollout batch (Sec. 4.2: the statistics are
 * only updated at batch boundaries).  Plain data, passed by host pointer, copied at call. */
typedef struct espo_params {
  float   temperature;      /* > 0 samples from softmax(logits/temperature); 0 = greedy    */
  float   mu_g;             /* running mean of the regret, Eq. 7                            */
  float   sigma2_g;         /* running variance of the regret, Eq. 8 (>= 0)                 */
  float   delta;            /* stabiliser under the square root in Eq. 9 (sigma2_g+delta>0) */
  float   clip_c;           /* clipping bound c of Eq. 9 (> 0)                              */
  float   alpha_s;          /* smoothing factor of Eq. 10, in [0, 1)                         */
  float   beta;             /* threshold multiplier of Eq. 11                               */
  float   eps;              /* value floor epsilon of Eq. 11                                */
  int32_t warmup_complete;  /* 0: the stop test is disabled (critic warm-up); z still runs  */
  int32_t t_max;            /* horizon T_max (> 0)                                          */
  int32_t eos_token;        /* end-of-sequence id, or -1 for none                           */
  int32_t sampler;          /* ESPO_SAMPLER_FLAT or ESPO_SAMPLER_HIER                       */
  int32_t stop_mode;        /* ESPO_STOP_*; every rule is gated by warmup_complete          */
  int32_t shadow;           /* != 0: the first step at which the rule holds is recorded in   */
                            /* t_stop, but the trajectory is not ended and stop_out stays 0  */
                            /* (the "Original" curves of the analysis section)               */
  float   tau;              /* threshold of ESPO_STOP_VALUE_ONLY / ESPO_STOP_REGRET_ONLY     */
  float   p_random;         /* per-step stop probability of ESPO_STOP_RANDOM, in [0, 1]; the */
                            /* draw is Philox level 3, index 0 of the step's stream          */
  int32_t want_entropy;     /* != 0: also compute the policy entropy H(pi(.|s_t)) in the same */
                            /* pass (the quantity tracked in the analysis section); needs    */
                            /* ESPO_SAMPLER_HIER                                              */
  /* Filtered sampling (the paper's evaluation decodes with top-p 0.7, Sec. 5; it gives no rule for ties): a token
   * stays in the support iff the tokens strictly more probable than it weigh less than top_p and number fewer than
   * top_k, so equally probable tokens stay or go together; the token is drawn from the renormalised support and
   * log pi(a_t) refers to it, the regret of Eq. 6 is unchanged.  Needs ESPO_SAMPLER_FLAT; ignored when greedy.
   * A filtered step runs its own kernel (one CTA per row, the row re-read from L2 once per 8 bits of the logit
   * type), not the single-sweep one. */
  float   top_p;            /* in (0, 1): nucleus mass; <= 0 or >= 1: no filter                */
  int32_t top_k;            /* > 0: at most the k most probable (more if tied); 0: no filter  */
} espo_params;

/* Opaque per-rollout-batch state: for each of `capacity` trajectory slots the smoothed
 * regret z, the step counter t, the status, and running sums of g; plus the library's
 * scratch.  Created and destroyed by the library; lives on the device current at creation. */
typedef struct espo_state espo_state;

/* Create the state for up to `capacity` trajectories over a vocabulary of V ids
 * (the initialisation of Algorithm 1: z = 0, t = 0, not done -- for every slot).
 *   out       host pointer that receives the handle
 *   seed      64-bit Philox key;  batch_id  rollout-batch number (< 2^30), part of the counter
 * Allocates device memory (this call and espo_free_state are the only ones that do for the
 * step path) and enqueues the initialisation on `stream`.
 * Errors: NULL, BAD_SHAPE (capacity or V < 1), BAD_PARAM (batch_id >= 2^30), CAPACITY, CUDA. */
int espo_init_state(espo_state** out, int32_t capacity, int32_t V, uint64_t seed, uint64_t batch_id,
                    void* stream);

/* Start a new rollout batch in an existing state: every slot back to z = 0, t = 0, active,
 * sums cleared, sticky status cleared; new batch_id.  Enqueued on `stream`. */
int espo_reset_state(espo_state* st, uint64_t batch_id, void* stream);

/* Release the state and its device memory (synchronises the device). NULL is ignored. */
void espo_free_state(espo_state* st);

/* One decode step for n_rows trajectories (Algorithm 1, loop body; Eq. 6, 9, 10, 11).
 *   logits      device, [n_rows, V] row-major, element type logits_dtype, rows row_stride
 *               ELEMENTS apart (row_stride >= V).  Read exactly once from DRAM.  Entries may
 *               be -inf (masked ids).  The fast path needs a 16-byte aligned base and
 *               row_stride*sizeof(elem) and V*sizeof(elem) multiples of 16; anything else
 *               takes a slower element-wise loader with identical results.
 *   values      device, [n_rows] critic estimates V_phi(s_t) for the same positions, values_dtype
 *   row_ids     device, [n_rows] trajectory slot of each row, or NULL for row i = slot i.
 *               Slots must be distinct within a call.
 *   n_rows      0 <= n_rows <= capacity (0 is a no-op)
 *   params      host pointer; copied before the call returns
 *   tokens_out  device int32 [n_rows]: the sampled token a_t; -1 for a row whose slot is not
 *               active (such rows are otherwise left untouched); 0 for an unusable row
 *   stop_out    device uint8 [n_rows]: 1 iff ESPO's rule fired for the row on this step.
 *               EOS and T_max endings are reported through status[], not here; a sampled
 *               EOS takes precedence over a stop on the same step.
 * For an active row with step counter t the call draws a_t (Philox counter uses t), forms
 * g_t = (max logit - logit[a_t]) / temperature, g~_t, z <- alpha_s z + (1-alpha_s) g~_t,
 * adds g_t and g_t^2 to the slot's running sums, sets t <- t+1, and updates status/t_stop.
 * mu_g, sigma2_g and beta are never modified.  Enqueued on `stream`; calls on the same
 * state must not overlap on the device.
 * Errors: NULL, BAD_DTYPE, BAD_SHAPE, ALIGN, CAPACITY, BAD_PARAM, CUDA. */
int espo_step(const void* logits, int32_t logits_dtype, int64_t row_stride,
              const void* values, int32_t values_dtype,
              const int32_t* row_ids, int32_t n_rows,
              espo_state* st, const espo_params* params,
              int32_t* tokens_out, uint8_t* stop_out, void* stream);

/* Read-only device pointers to the per-slot arrays (each of length capacity); any output
 * pointer may be NULL.  g, g_tilde and logp hold the values of each slot's latest step
 * (logp = log pi(a_t | s_t) under the temperature-scaled distribution).  t is the number
 * of tokens generated; t_stop is the index of the stop step or -1; sum_g, sum_g2 are the
 * double-precision sums over the slot's tokens that the batch statistics of Eq. 7-8 need;
 * entropy is the policy entropy of the slot's latest step and sum_h its running sum (both only
 * maintained by steps with want_entropy set). */
int espo_state_view(espo_state* st, const float** z, const float** g, const float** g_tilde,
                    const float** logp, const int32_t** t, const uint8_t** status,
                    const int32_t** t_stop, const double** sum_g, const double** sum_g2,
                    const float** entropy, const double** sum_h);

/* Expert knob: override the step kernel's launch shape for this state.  consumer_warps =
 * streaming warps per CTA (1..31), stages = blocks of 1024 ids each warp keeps in flight,
 * ctas_per_sm = resident CTAs per SM; 0 keeps the library default for any of them, and the
 * library shrinks what does not fit in shared memory.  Results never depend on it.
 * Errors: NULL, BAD_PARAM. */
int espo_set_launch_config(espo_state* st, int32_t consumer_warps, int32_t stages, int32_t ctas_per_sm);

/* Programmatic dependent launch for the step kernel of ESPO_SAMPLER_HIER (the paper has no counterpart; it is how a
 * decode loop hides launch latency on this hardware).  With enable != 0, espo_step launches its kernel so that the
 * GPU may set it up -- place its thread blocks, run the part that touches no global memory -- while the kernel
 * that precedes it in the stream is still finishing; the step kernel waits for that kernel's completion before it
 * reads or writes any global memory, so what it computes does not change.  The step kernel in turn lets a
 * kernel launched after it in the same way start early; espo_compact_active is launched the same way.  Off by
 * default.  Errors: NULL. */
int espo_set_dependent_launch(espo_state* st, int32_t enable);

/* Stable compaction of the active set: writes the slots whose status is ESPO_ROW_ACTIVE, in
 * increasing order, to row_ids_out (device int32 [capacity]) and their number to
 * n_active_out (device int32 [1]).  Enqueued on `stream`. */
int espo_compact_active(espo_state* st, int32_t* row_ids_out, int32_t* n_active_out, void* stream);

/* Batch boundary (Sec. 4.2, Eq. 7-8 and Sec. 4.3, Eq. 12), to be called after the last step of a
 * rollout batch and before espo_reset_state.  Over the slots that took part (t > 0) it forms, on
 * the device, the mean and the population variance of every regret value g generated in the
 * batch (stop-step tokens included) and the empirical stop rate rho = stopped / took part, then
 *   mu_g     <- alpha_ema mu_g     + (1 - alpha_ema) mean      (set to mean if first_update)
 *   sigma2_g <- alpha_ema sigma2_g + (1 - alpha_ema) variance  (set to variance if first_update)
 *   beta     <- clip(beta + eta_beta (rho - tau), beta_min, beta_max)
 * reading the old values from *params_inout (host) and writing the new ones back to it; the
 * other fields are left alone.  The paper's values: alpha_ema 0.99, eta_beta 0.1, tau 0.25,
 * beta_min 0; it names beta_max without a value.  A batch without tokens changes nothing.
 *   stats_out  host double [6] or NULL: mean, variance, rho, tokens, trajectories, stopped
 * Synchronises `stream`.  Errors: NULL, BAD_PARAM (alpha_ema outside [0,1], NaN, beta_min >
 * beta_max), CUDA. */
int espo_end_batch(espo_state* st, float alpha_ema, float eta_beta, float tau, float beta_min,
                   float beta_max, int32_t first_update, espo_params* params_inout,
                   double* stats_out, void* stream);

/* The batch boundary when the rollout batch's trajectories are spread over several states (one per GPU): every
 * part calls espo_end_batch on a scratch copy of the parameters to obtain its stats_out, the parts exchange those six
 * numbers (one all-gather), and every part calls this with all of them and with the real parameters.  The pooled mean,
 * population variance and stop rate are what espo_end_batch would have found over all trajectories at once, and the
 * same updates (Eq. 7, 8, 12) are applied to *params_inout, so all parts end with identical parameters.  Host only.
 *   stats      host double [n_parts][6], each row as written by espo_end_batch
 *   stats_out  host double [6] or NULL: the pooled mean, variance, rho, tokens, trajectories, stopped
 * Errors: NULL, BAD_SHAPE, BAD_PARAM (as espo_end_batch; also negative counts or NaN in stats). */
int espo_end_batch_merge(const double* stats, int32_t n_parts, float alpha_ema, float eta_beta, float tau,
                         float beta_min, float beta_max, int32_t first_update, espo_params* params_inout,
                         double* stats_out);

/* ---- vocabulary shards (a tensor-parallel LM head leaves every GPU with V/N of each logit row) ----
 * The paper samples from whole rows (Algorithm 1); this pair of calls computes the same step when a row's logits
 * are spread over several buffers.  Every shard reduces its part of the rows to one espo_partial per row
 * (espo_step_partial), the partials of all shards are brought together (one all-gather of 32 bytes per row and
 * shard when the shards live on different GPUs; the library does not communicate) and espo_step_merge finishes the
 * step on the trajectory state: regret, normalisation, smoothing, stop rule, bookkeeping (Eq. 6, 9-11), exactly as
 * espo_step does.  With the flat sampler the Gumbel draws belong to token ids, so the perturbed maximum over the
 * shards is the perturbed maximum over the row and the token does not depend on how the row is cut.  With the
 * hierarchical sampler the block-level draws belong to blocks of 1024 ids of the whole vocabulary: shards that start
 * on such a block give exactly the token of espo_step (each shard resolves the token inside its own best block and
 * reports that block's perturbed score; the merge takes the best of them).  Greedy decoding (temperature 0) and the
 * entropy are offered with the flat sampler only. */
typedef struct espo_partial {
  float m;             /* largest logit of the shard's part of the row (-inf if it has no finite entry)           */
  float s;             /* sum over the part of exp((x - m) / temperature)                                          */
  float best;          /* largest perturbed score x/T + G of the part (greedy: the largest logit; hierarchical       */
                       /* sampler: the best block's score m_b/T + ln s_b + G_b)                                     */
  int32_t best_id;     /* global token id that attains it, lowest id on ties (hierarchical: the token drawn inside  */
                       /* that block); -1: none                                                                     */
  float x_best;        /* that token's logit                                                                        */
  uint32_t flags;      /* bit 0: the part held NaN or +inf; bit 1: nothing computed (bad slot or ended trajectory) */
  uint32_t reserved[2];
} espo_partial;        /* 32 bytes */

/* One shard's share of a decode step.  Reads the state (step counter and slot choose the random stream) and writes
 * partial_out; changes nothing else, so the shards of a step may run in any order or on different GPUs with
 * replicas of the state.
 *   logits_shard   device [n_rows, v_shard] with row_stride elements between rows, dtype as for espo_step
 *   vocab_offset   global id of the shard's first logit; a multiple of 4 (ESPO_SAMPLER_HIER: of 1024);
 *                  vocab_offset + v_shard <= V
 *   partial_out    device espo_partial [n_rows], 16-byte aligned
 *   params         either sampler; ESPO_SAMPLER_HIER needs temperature > 0 and want_entropy = 0 (else
 *                  ESPO_ERR_BAD_PARAM); with ESPO_SAMPLER_FLAT temperature 0 = greedy
 * Calls that use the same state must not overlap on the device (they share its scratch).
 * Errors: NULL, BAD_SHAPE, BAD_DTYPE, BAD_PARAM, ALIGN, CAPACITY, CUDA. */
int espo_step_partial(const void* logits_shard, int32_t logits_dtype, int64_t row_stride, int32_t v_shard,
                      int32_t vocab_offset, const int32_t* row_ids, int32_t n_rows, espo_state* st,
                      const espo_params* params, espo_partial* partial_out, void* stream);

/* Merges the shards' partials and commits the step, with the outputs and state changes of espo_step.
 *   partials      device espo_partial: shard k's result for row r at partials[k * shard_stride + r]
 *   n_shards >= 1, shard_stride >= n_rows (elements)
 *   values, row_ids, tokens_out, stop_out, params: as for espo_step, with the same params as the partial calls
 * A row is marked ESPO_ROW_BAD if any shard flagged NaN / +inf or no shard held a finite logit.
 * Errors: NULL, BAD_SHAPE, BAD_DTYPE, BAD_PARAM, ALIGN, CAPACITY, CUDA. */
int espo_step_merge(const espo_partial* partials, int32_t n_shards, int64_t shard_stride, const void* values,
                    int32_t values_dtype, const int32_t* row_ids, int32_t n_rows, espo_state* st,
                    const espo_params* params, int32_t* tokens_out, uint8_t* stop_out, void* stream);

/* Copy the sticky device status word (ESPO_DEV_* bits) to *host_out.  Synchronises `stream`. */
int espo_state_status(espo_state* st, uint32_t* host_out, void* stream);

/* TD errors and GAE over B ragged trajectories (Eq. 4-5) with ESPO's failure transition
 * (Eq. 13).  Trajectory i owns tokens [off_i, off_i + lengths[i]) of the packed arrays,
 * off = exclusive prefix sum of lengths.
 *   rewards, values  device float32 [total_tokens]
 *   lengths          device int32 [B] (>= 0; the stop-step token of a stopped trajectory is
 *                    its last token)
 *   stopped          device uint8 [B]: 1 = ended by ESPO's rule; its last reward is REPLACED
 *                    by r_fail
 *   total_tokens     host value of sum(lengths); a mismatch sets ESPO_DEV_BAD_LENGTHS
 *   adv_out          device float32 [total_tokens]
 * With r'_t the (possibly replaced) rewards and V_L := 0 for every trajectory (nothing is
 * bootstrapped past the last token): delta_t = r'_t + gamma V_{t+1} - V_t and
 * A_t = delta_t + gamma*lambda*A_{t+1}, A_L := 0.
 * Trajectories do not interact: a NaN or infinity among one trajectory's rewards or values
 * spoils that trajectory's advantages only.
 * Uses a per-device workspace that grows on demand: a call that needs more than any
 * earlier call (or espo_advantages_reserve) allocates device memory after synchronising
 * the device; otherwise nothing is allocated.  Calls on one device must not overlap.
 * Errors: NULL, BAD_SHAPE, ALIGN (arrays must be 16-byte aligned), CUDA. */
int espo_advantages(const float* rewards, const float* values, const int32_t* lengths,
                    const uint8_t* stopped, int32_t B, int64_t total_tokens,
                    float gamma, float lambda, float r_fail, float* adv_out, void* stream);

/* espo_advantages that also writes the value targets of the critic, returns_t = A_t + V(s_t) (the
 * lambda-return that goes with the GAE of Eq. 5), in the same pass.
 *   returns_out  device float32 [total_tokens], 16-byte aligned, or NULL (then exactly espo_advantages)
 * Everything else as for espo_advantages. */
int espo_advantages_returns(const float* rewards, const float* values, const int32_t* lengths,
                            const uint8_t* stopped, int32_t B, int64_t total_tokens,
                            float gamma, float lambda, float r_fail, float* adv_out,
                            float* returns_out, void* stream);

/* espo_advantages_returns that also leaves the two sums a trainer normalises ("whitens") a batch of advantages
 * with.  The paper does not normalise advantages (Sec. 3 uses the GAE of Eq. 5 as it is); this is the usual
 * PPO companion step, offered because the sums fall out of the same pass.
 *   stats_out    device float64 [2], 8-byte aligned, or NULL (then exactly espo_advantages_returns):
 *                stats_out[0] = sum_t A_t, stats_out[1] = sum_t A_t^2 over all total_tokens tokens, taken in
 *                double precision before the advantages are rounded to float32; mean = stats_out[0] / total_tokens,
 *                variance = stats_out[1] / total_tokens - mean^2.  With B == 0 or total_tokens == 0 both are set to 0.
 * Every CTA adds up its own tokens and the CTA that finishes last adds up the CTAs' sums in a fixed order, so
 * repeated calls on the same input give bit-identical sums.  Everything else as for espo_advantages. */
int espo_advantages_stats(const float* rewards, const float* values, const int32_t* lengths,
                          const uint8_t* stopped, int32_t B, int64_t total_tokens,
                          float gamma, float lambda, float r_fail, float* adv_out,
                          float* returns_out, double* stats_out, void* stream);

/* Pre-size the advantage workspace of the current device so that later calls with
 * B <= max_B and total_tokens <= max_tokens allocate nothing. */
int espo_advantages_reserve(int32_t max_B, int64_t max_tokens);

/* Copy the advantage workspace's sticky status word (ESPO_DEV_TIMEOUT, ESPO_DEV_BAD_LENGTHS)
 * of the current device to *host_out and clear it.  Synchronises `stream`. */
int espo_advantages_status(uint32_t* host_out, void* stream);

/* espo_advantages_returns for the padded layout: rewards, values and the outputs are [B, t_max] row-major and
 * trajectory i owns the first lengths[i] entries of row i (Eq. 4-5 and 13 as for espo_advantages; the layout is this
 * library's, the paper does not fix one).
 *   rewards, values  device float32 [B * t_max], 16-byte aligned; what the padding holds is never used (it may be
 *                    NaN)
 *   lengths          device int32 [B], 0 <= lengths[i] <= t_max; a value outside sets ESPO_DEV_BAD_LENGTHS and is
 *                    clamped
 *   adv_out          device float32 [B * t_max]; padding entries are written as 0
 *   returns_out      device float32 [B * t_max] or NULL; padding entries are written as 0
 * The pass writes all B * t_max entries and reads all but the 3072-entry chunks that lie wholly inside one row's
 * padding; a batch that is mostly padding is cheaper packed.  Workspace and errors as for espo_advantages. */
int espo_advantages_padded(const float* rewards, const float* values, const int32_t* lengths,
                           const uint8_t* stopped, int32_t B, int32_t t_max,
                           float gamma, float lambda, float r_fail, float* adv_out,
                           float* returns_out, void* stream);

/* Limits of espo_advantages_noalloc. */
#define ESPO_NOALLOC_MAX_B       4096          /* trajectories per call                          */
#define ESPO_NOALLOC_MAX_TOKENS  16777216      /* sum(lengths) per call (2^24)                   */

/* espo_advantages for callers that must not allocate device memory.  (The paper has no
 * counterpart of this entry point; it computes exactly what espo_advantages computes.)
 *
 * Who needs it: a rollout worker whose serving engine claimed all free device memory for its
 * own pools at start-up, so that a cudaMalloc issued by a library fails; and a training loop
 * that cannot afford the device-wide synchronisation that cudaMalloc/cudaFree imply.  This call
 * never calls cudaMalloc, cudaFree or any other allocating routine: its scratch is a fixed
 * array of about 55 KB that is part of the library image, so every device that loads the
 * library holds that array until the process exits.
 *
 * Arguments are those of espo_advantages, plus
 *   status_out   device uint32 [1] or NULL: ESPO_DEV_TIMEOUT / ESPO_DEV_BAD_LENGTHS bits are
 *                OR-ed into it (the caller clears it); with NULL they go to a word inside the
 *                scratch that cannot be read back.
 * Limits: B <= ESPO_NOALLOC_MAX_B and total_tokens <= ESPO_NOALLOC_MAX_TOKENS, otherwise
 * ESPO_ERR_CAPACITY and nothing is launched.
 * The first call on each device looks up the scratch array's device address (with that device
 * current) and remembers it; make that first call outside any stream capture.
 * All calls on a device share the one array and it keeps the previous call's contents; no
 * part of it has to start at zero, because each call rewrites every entry it later reads.
 * Two calls that overlap on the device (different streams, no dependency) race on it:
 * serialise them.
 * Errors: BAD_SHAPE, CAPACITY, NULL, ALIGN (16-byte arrays), BAD_PARAM, CUDA. */
int espo_advantages_noalloc(const float* rewards, const float* values, const int32_t* lengths,
                            const uint8_t* stopped, int32_t B, int64_t total_tokens,
                            float gamma, float lambda, float r_fail, float* adv_out,
                            uint32_t* status_out, void* stream);

/* Text for a return code; never NULL. */
const char* espo_strerror(int code);

/* The last cudaError_t (as int) seen by this library on the calling thread, 0 if none. */
int espo_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* ESPO_H_ */
