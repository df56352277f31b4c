/*
 * impact.h -- C ABI of the IMPACT learner hot path for NVIDIA B200 (sm_100a).
 *
 * The library computes, per train batch of B trajectories x T steps, the loss and the
 * gradients that IMPACT's learner needs (Luo et al., "IMPACT: Importance Weighted
 * Asynchronous Architectures with Clipped Target Networks", arXiv 1912.00167), and keeps
 * the paper's circular buffer C(N, K) as a ring of device-resident batches.
 *
 * Conventions for every call
 *  - Return value: int32 status, IMPACT_OK (0) or a negative IMPACT_ERR_* code.
 *    Arguments are validated on the host before anything is enqueued; a call that
 *    returns an error has enqueued nothing and changed no state.
 *  - Unless a parameter says "host", tensor pointers are caller-owned DEVICE memory,
 *    dense, row-major, trajectory-major: [B, T] or [B, T, A].  Base pointers must be
 *    16-byte aligned.  The library never frees or keeps them beyond the call.
 *  - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls only
 *    enqueue work on it and return; no call synchronises the device unless it says so.
 *  - Same inputs give bit-identical outputs from run to run (no floating-point atomics).
 *  - There is no CPU fallback: without a CUDA device the compute calls return
 *    IMPACT_ERR_CUDA.
 */
#ifndef IMPACT_H_
#define IMPACT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define IMPACT_VERSION 300 /* major*10000 + minor*100 + patch */

/* ---- status codes -------------------------------------------------------------------- */
#define IMPACT_OK 0
#define IMPACT_ERR_INVALID_ARG (-1)        /* null / misaligned pointer, non-positive size, bad enum or scalar */
#define IMPACT_ERR_UNSUPPORTED (-2)        /* shape or dtype outside what the kernels were built for */
#define IMPACT_ERR_WORKSPACE_TOO_SMALL (-3)
#define IMPACT_ERR_EMPTY (-4)              /* circular buffer holds no live batch */
#define IMPACT_ERR_FULL (-5)               /* every slot of the circular buffer is still live */
#define IMPACT_ERR_CUDA (-6)               /* a CUDA runtime call failed; see impact_last_cuda_error() */

/* ---- enums ---------------------------------------------------------------------------- */
#define IMPACT_DTYPE_F32 0
#define IMPACT_DTYPE_BF16 1

/* Which two policies form the truncated importance weights rho_t, c_t of the value
 * recursion: Section 3.1 uses pi_target / pi_worker; Section 2.2 (V-trace as in IMPALA)
 * uses pi_theta / pi_worker.  Either way the weights are constants for the gradient. */
#define IMPACT_IS_TARGET_OVER_WORKER 0
#define IMPACT_IS_LEARNER_OVER_WORKER 1
#define IMPACT_IS_NONE 2 /* rho_t = c_t = 1 before truncation: plain GAE-lambda, as PPO uses it (Section 2.1) */

/* What the policy is trained on:
 *   CLIPPED_SURROGATE  min(R A, clip(R, 1-eps, 1+eps) A) with the ratio of `ratio_mode` (IMPACT, Section 3.1 and
 *                      Appendix E; PPO is R2 with IMPACT_IS_NONE, Section 2.1);
 *   VTRACE_PG          IMPALA's importance-weighted policy gradient (Section 2.2, Appendix D): the weight
 *                      rho_t (r_t + gamma_t v_{t+1} - V_t), v the V-trace target, multiplies grad log pi_theta;
 *                      the policy term reported is -mean(weight * log pi_theta), nothing is clipped
 *                      (clip_eps, rho_tw and ratio_mode are ignored; IMPACT_TERM_MEAN_RATIO is mean rho_t). */
#define IMPACT_OBJECTIVE_CLIPPED_SURROGATE 0
#define IMPACT_OBJECTIVE_VTRACE_PG 1

/* Likelihood ratio of the surrogate (Section 4.1):
 *   R3 = pi_theta / max(pi_target, pi_worker / rho_tw)   (the IMPACT objective, Section 3.1)
 *   R1 = pi_theta / pi_target,  R2 = pi_theta / pi_worker (the ablations). */
#define IMPACT_RATIO_R3 0
#define IMPACT_RATIO_R1 1
#define IMPACT_RATIO_R2 2

/* Circular-buffer draw: uniform over the live slots from a seeded counter-based draw, or
 * the next live slot in ring order. */
#define IMPACT_SAMPLE_UNIFORM 0
#define IMPACT_SAMPLE_ROUND_ROBIN 1

/* Where the source of a buffer push lives. */
#define IMPACT_SRC_DEVICE 0
#define IMPACT_SRC_HOST 1

/* Index of each entry of `loss_terms` (8 floats, device memory). */
#define IMPACT_TERM_TOTAL 0      /* policy + vf_coef*value - ent_coef*entropy + kl_coef*kl */
#define IMPACT_TERM_POLICY 1     /* -(1/M) sum_t surrogate_t */
#define IMPACT_TERM_VALUE 2      /* (1/M) sum_t 1/2 (V_t - Vhat_t)^2 */
#define IMPACT_TERM_ENTROPY 3    /* (1/M) sum_t H(pi_theta(.|s_t)) */
#define IMPACT_TERM_KL 4         /* (1/M) sum_t KL(pi_target(.|s_t) || pi_theta(.|s_t)); evaluated only
                                    when kl_coef != 0, reported as 0 otherwise */
#define IMPACT_TERM_CLIP_FRAC 5  /* share of steps whose policy gradient the eps-clip removed */
#define IMPACT_TERM_RHO_FRAC 6   /* share of steps whose importance weight exceeded rho_bar */
#define IMPACT_TERM_MEAN_RATIO 7 /* (1/M) sum_t R_t */
#define IMPACT_NUM_TERMS 8

/* Coefficients of the loss (Algorithm 1; hyper-parameter tables of Appendix B).
 * Plain data, passed by HOST pointer, read during the call only. */
typedef struct impact_coefficients {
    float vf_coef;         /* weight of the value loss */
    float ent_coef;        /* weight of the entropy bonus (subtracted from the loss) */
    float kl_coef;         /* eta of Algorithm 1: weight of KL(pi_target || pi_theta) */
    float lambda_;         /* lambda of V-trace GAE-lambda (Section 3.1); 1 gives V-trace targets */
    float rho_tw;          /* rho > 0 of the target-worker clipping (Section 3.1); beta = 1/rho */
    int32_t is_source;     /* IMPACT_IS_* */
    int32_t ratio_mode;    /* IMPACT_RATIO_* */
    int32_t dlogits_dtype; /* IMPACT_DTYPE_*: storage type of the policy-gradient outputs */
    int32_t objective;     /* IMPACT_OBJECTIVE_* */
    int64_t global_steps;  /* the M of the 1/M normaliser (Algorithm 1); 0 = B*T, this call's own steps.  A caller
                              that splits one train batch over several calls or GPUs (trajectories are
                              independent) passes the steps of the WHOLE batch here in every call: gradients then
                              carry the whole batch's 1/M, and the calls' loss_terms ADD UP to the whole batch's
                              (they are sums over this call's steps divided by M).  Must be 0 or >= B*T. */
} impact_coefficients;

/* ---- housekeeping --------------------------------------------------------------------- */
int32_t impact_version(void);
/* Static, NUL-terminated description of a status code. */
const char* impact_status_string(int32_t status);
/* cudaError_t value of the most recent CUDA failure seen by this thread's calls (0 if none). */
int32_t impact_last_cuda_error(void);

/*
 * Launch options of the loss calls: process-wide performance knobs with working defaults; none changes a
 * result.  (The paper prescribes no kernel design, so these have no counterpart there.)  A value set here is
 * used by every later loss call of the process; setting one while another thread is inside a loss call is safe
 * (that call uses the old or the new value).
 *   IMPACT_OPT_EARLY_PREFETCH  1 (default): a loss call whose thread blocks have four to eight tiles each (of at
 *       least 10 KB, rows of at most 32 actions: batches of roughly 75 000 to 150 000 steps of 18 actions) enqueues
 *       a one-warp-per-block companion kernel right before its loss kernel.  The companion runs beside whatever
 *       kernel is still busy on the stream, asks L2 for the batch's first tiles, and then waits for the stream's
 *       previous kernel, so stream order is kept exactly; the loss kernel finds its first tiles in L2 instead of
 *       waiting for HBM.  0: no companion; the loss kernel asks for its first tiles itself when it starts.
 *   IMPACT_OPT_PREFETCH_BYTES  upper bound on the bytes one call asks L2 for ahead of time (default 48 MiB).
 *   IMPACT_OPT_WINDOW_BYTES    bytes of tiles a block keeps in flight from global to shared memory: 0 (default)
 *       lets each launch choose (48 KiB where a block has eight tiles or fewer, 72 KiB beyond), else
 *       16 KiB .. 160 KiB.
 * impact_set_option returns IMPACT_ERR_INVALID_ARG for an unknown option or a value out of range;
 * impact_get_option returns -1 for an unknown option.
 */
#define IMPACT_OPT_EARLY_PREFETCH 0
#define IMPACT_OPT_PREFETCH_BYTES 1
#define IMPACT_OPT_WINDOW_BYTES 2
#define IMPACT_NUM_OPTIONS 3
int32_t impact_set_option(int32_t option, int64_t value);
int64_t impact_get_option(int32_t option);

/* ---- loss and gradients --------------------------------------------------------------- */

/*
 * Bytes of scratch that impact_loss_fwd_bwd / impact_loss_fwd_bwd_gaussian need for a batch
 * of B x T steps: partial sums and counter words (a fixed 193 KB), plus, for trajectories
 * longer than 64 steps, 16 bytes per 64 steps of every trajectory (the aggregates that link
 * the tiles of a trajectory that is worked on by several thread blocks at once).  A workspace
 * with the fixed part only -- impact_loss_workspace_bytes(1, 1) -- serves every batch too: long
 * trajectories are then swept by one thread block each, which is slower when there are few of
 * them.  Returns 0 for non-positive sizes.
 */
size_t impact_loss_workspace_bytes(int64_t B, int64_t T);

/*
 * Clears a workspace (enqueues a memset on `stream`).  A workspace must be cleared once
 * before its first use; every loss call leaves it ready for the next (it also keeps a count
 * of the launches that used it, which tells one launch's partial sums from the previous
 * one's), so one buffer serves any number of calls on ONE stream.  Calls that may overlap on the GPU need a workspace each.
 */
int32_t impact_loss_workspace_init(void* workspace, size_t workspace_bytes, void* stream);

/*
 * Reads a workspace's error word into *flag_out (HOST): 0 = no loss call that used this
 * workspace ever gave up waiting for one of its own asynchronous copies; non-zero = at least
 * one did (the wait inside the kernels is bounded, so a copy that never lands becomes this
 * flag instead of a hang, and that call's outputs are not to be trusted).  The word is
 * cleared by impact_loss_workspace_init only.  Synchronises `stream` before reading.
 */
int32_t impact_loss_workspace_status(const void* workspace, size_t workspace_bytes, int32_t* flag_out,
                                     void* stream);

/*
 * IMPACT loss and gradients for a discrete-action policy (Algorithm 1, "Compute policy
 * and value network gradients"), in one fused pass.  With M = B*T, per step t of a
 * trajectory (a = actions[b,t], gamma_t = discounts[b,t]):
 *
 *   l_theta, l_target   log-softmax of the learner / target logits at a
 *   x_t   = l_target - worker_logp      (or l_theta - worker_logp, see is_source)
 *   rho_t = min(rho_bar, exp x_t),  c_t = min(c_bar, exp x_t)           (Section 2.2, 3.1)
 *   delta_t = rho_t (r_t + gamma_t V_{t+1} - V_t),  V_T = bootstrap_values[b]
 *   A_t   = delta_t + lambda gamma_t c_t A_{t+1},  A_T = 0   (V-trace GAE-lambda, Section 3.1)
 *   Vhat_t = V_t + A_t                      (the V-trace target of Section 2.2 at lambda = 1)
 *   R_t   = exp(l_theta - max(l_target, worker_logp - ln rho_tw))       (Section 3.1)
 *   s_t   = min(R_t A_t, clip(R_t, 1-eps, 1+eps) A_t)                   (Appendix E)
 *   total = -mean s + vf_coef mean 1/2 (V - Vhat)^2 - ent_coef mean H(pi_theta)
 *           + kl_coef mean KL(pi_target || pi_theta)
 *
 * and the gradient of `total` with respect to the learner logits and the values, with A_t
 * and Vhat_t treated as constants (Algorithm 1 differentiates neither).  The policy term of
 * a step is dropped exactly when the clipped branch is the strictly smaller one
 * (A_t > 0 and R_t > 1+eps, or A_t < 0 and R_t < 1-eps).
 *
 * Inputs (device):
 *   learner_logits, target_logits [B,T,A]  f32 or bf16 according to `logits_dtype`
 *   worker_logp [B,T] f32   log-probability the worker's policy gave the action it took
 *   actions [B,T] i32       must lie in [0, A); out-of-range actions are clamped into range
 *   rewards, discounts, values [B,T] f32;  bootstrap_values [B] f32
 *   discounts[b,t] = gamma * (1 - done_t): a zero cuts both the bootstrap and the trace.
 * Scalars: rho_bar, c_bar >= 0 (+inf allowed), clip_eps >= 0; `coef` is a HOST pointer.
 * Outputs (device):
 *   loss_terms [8] f32 (see IMPACT_TERM_*)
 *   dlogits [B,T,A] f32 or bf16 per coef->dlogits_dtype;  dvalues [B,T] f32
 *   vtarget, advantage [B,T] f32: optional, NULL to skip.
 * Outputs must not alias inputs.
 * workspace: device scratch of at least impact_loss_workspace_bytes(B,T) bytes, cleared
 *   once with impact_loss_workspace_init.
 * Limits: 1 <= A <= 512; B*T*A < 2^40.  No input is clamped or sanitised: NaN/Inf inputs
 * give NaN/Inf outputs wherever the arithmetic above carries them -- and, because trajectories
 * shorter than 128 steps are worked on several to a tile with the recursion cut between them by
 * a factor of zero, possibly also in the trajectories that precede the affected one within its
 * tile (floor(128 / T) consecutive trajectories).  No wait depends on a value: nothing hangs.
 * Errors: INVALID_ARG, UNSUPPORTED, WORKSPACE_TOO_SMALL, CUDA (launch failure).
 */
int32_t impact_loss_fwd_bwd(
    const void* learner_logits, const void* target_logits, const float* worker_logp,
    const int32_t* actions, const float* rewards, const float* discounts, const float* values,
    const float* bootstrap_values, float rho_bar, float c_bar, float clip_eps,
    const impact_coefficients* coef, int64_t B, int64_t T, int32_t A, int32_t logits_dtype,
    float* loss_terms, void* dlogits, float* dvalues, float* vtarget, float* advantage,
    void* workspace, size_t workspace_bytes, void* stream);

/*
 * The arguments of impact_loss_fwd_bwd as one plain struct, for callers that issue the same
 * call many times (a learner loop over fixed buffers): fill it once, then pass its HOST
 * address to impact_loss_fwd_bwd_call.  Field meanings, layouts, limits and errors are those
 * of impact_loss_fwd_bwd; `coef` is embedded by value.
 */
struct impact_loss_inputs;
typedef struct impact_loss_call {
    const void* learner_logits;
    const void* target_logits;
    const float* worker_logp;
    const int32_t* actions;
    const float* rewards;
    const float* discounts;
    const float* values;
    const float* bootstrap_values;
    float rho_bar, c_bar, clip_eps;
    int32_t logits_dtype;
    impact_coefficients coef;
    int32_t A;
    int64_t B, T;
    float* loss_terms;
    void* dlogits;
    float* dvalues;
    float* vtarget;
    float* advantage;
    void* workspace;
    size_t workspace_bytes;
    void* target_logits_copy; /* optional (NULL = none): [B,T,A], same type as the logits.  The call also writes
                                 target_logits there, byte for byte -- the "store the target network's output with
                                 the batch" of a batch's first traversal (Algorithm 1; impact_buffer_append) done by
                                 the loss kernel itself, which has the rows in shared memory anyway, instead of by a
                                 copy of its own.  Typically a slot of the circular buffer
                                 (impact_buffer_slot_ptr).  Must not overlap any other argument. */
    const struct impact_loss_inputs* inputs_on_device; /* optional (NULL = none): DEVICE pointer to a record written by
                                 impact_buffer_device_step earlier on the same stream.  The kernel then takes its
                                 eight input pointers and target_logits_copy from that record (read once the stream's
                                 previous work is complete) instead of from the fields above, which are ignored and
                                 may be NULL.  Shapes, types and outputs come from this struct as usual.  Served by
                                 the persistent kernel only: A in {4, 6, 9, 18, 64} and T <= 128 (64 for A = 64);
                                 else IMPACT_ERR_UNSUPPORTED. */
} impact_loss_call;

/* impact_loss_fwd_bwd with its arguments taken from `call` (Algorithm 1, gradient step). */
int32_t impact_loss_fwd_bwd_call(const impact_loss_call* call, void* stream);

/*
 * The same loss for a diagonal-Gaussian policy with D action dimensions (continuous
 * control, Section 4.3; Appendix E).  sigma = exp(logstd), per step:
 *   log pi(a|s)  = sum_d [ -1/2 ((a_d - mu_d)/sigma_d)^2 - logstd_d - 1/2 ln 2pi ]
 *   H            = sum_d [ logstd_d + 1/2 ln(2 pi e) ]
 *   KL(tgt||th)  = sum_d [ logstd_th - logstd_tg + (sigma_tg^2 + (mu_tg - mu_th)^2)/(2 sigma_th^2) - 1/2 ]
 * Inputs: learner_mean, learner_logstd, target_mean, target_logstd, actions [B,T,D] f32;
 * the [B,T] inputs as in impact_loss_fwd_bwd.  Outputs: dmean, dlogstd [B,T,D] f32,
 * dvalues [B,T] f32, loss_terms [8]; vtarget/advantage optional.  coef->dlogits_dtype must
 * be IMPACT_DTYPE_F32.  Limits: 1 <= D <= 256.
 */
int32_t impact_loss_fwd_bwd_gaussian(
    const float* learner_mean, const float* learner_logstd, const float* target_mean,
    const float* target_logstd, const float* worker_logp, const float* actions,
    const float* rewards, const float* discounts, const float* values,
    const float* bootstrap_values, float rho_bar, float c_bar, float clip_eps,
    const impact_coefficients* coef, int64_t B, int64_t T, int32_t D,
    float* loss_terms, float* dmean, float* dlogstd, float* dvalues, float* vtarget,
    float* advantage, void* workspace, size_t workspace_bytes, void* stream);

/*
 * impact_loss_fwd_bwd for callers that cannot allocate device memory.  (The paper has no
 * counterpart of this call; it exists for the way the library gets embedded.)
 *
 * Some hosts of this library run where cudaMalloc is off limits: a plugin called from
 * inside another framework's step, whose memory pool owns the whole device; a real-time
 * control loop that may not block on the driver's allocator; a process that was handed
 * fixed buffers by its parent and nothing else.  Such a caller has no workspace to pass.
 * This entry point therefore takes none: the per-block sums and the completion counter
 * live in a 98,560-byte array that is part of the library image (one copy on every GPU that
 * loads the library, held until the process exits).  Inputs, outputs, arithmetic and
 * results are those of impact_loss_fwd_bwd; nothing is allocated or freed, here or in
 * anything this call uses.
 *
 * Limits: A <= 64, and the batch must split into at most 1024 tiles of 128 steps:
 * ceil(B / floor(128 / T)) <= 1024 when T <= 128, else B <= 1024.  (B=1024, T=128 is the
 * largest batch of full-length trajectories.  Rows wider than 32 actions may be worked on in
 * tiles of 64 steps and then fit half as much: count 64 for 128 above.)  Larger batches return
 * IMPACT_ERR_WORKSPACE_TOO_SMALL, A > 64 returns IMPACT_ERR_UNSUPPORTED; use
 * impact_loss_fwd_bwd with a workspace for those.
 *
 * The first call on a device looks up the array's device address (a driver query, with that
 * device current); make that first call outside any stream capture.  Every call enqueues a
 * small clear of the counter before its kernel, since the array still holds what the
 * previous call left.  All calls on a device share the one array: two calls whose kernels
 * may run at the same time (different streams, or different host threads without ordering)
 * corrupt each other's sums.  Keep them on one stream or order them with events.
 * The array's error word (see impact_loss_workspace_status) is sticky across calls: read it,
 * and clear it, with impact_loss_static_scratch_status.
 */
int32_t impact_loss_fwd_bwd_static_scratch(
    const void* learner_logits, const void* target_logits, const float* worker_logp,
    const int32_t* actions, const float* rewards, const float* discounts, const float* values,
    const float* bootstrap_values, float rho_bar, float c_bar, float clip_eps,
    const impact_coefficients* coef, int64_t B, int64_t T, int32_t A, int32_t logits_dtype,
    float* loss_terms, void* dlogits, float* dvalues, float* vtarget, float* advantage,
    void* stream);

/*
 * The error word of the built-in scratch of impact_loss_fwd_bwd_static_scratch on the current device, into
 * *flag_out (HOST): 0 = no call through that entry point has given up a bounded wait since the word was last
 * cleared; non-zero = at least one did, and the outputs of such a call are not to be trusted.  clear != 0 also
 * resets the word.  Synchronises `stream`; allocates nothing.  (No counterpart in the paper.)
 */
int32_t impact_loss_static_scratch_status(int32_t* flag_out, int32_t clear, void* stream);

/* ---- circular buffer C(N, K) ---------------------------------------------------------- */

/*
 * The paper's circular buffer (Algorithm 1 "Initialize circular buffer C(N,K)"; Section
 * 3.2): N slots, each holding one train batch; a batch is handed to the learner at most K
 * times and is then discarded, freeing its slot for a new worker batch.  When every slot
 * is live a push is refused (IMPACT_ERR_FULL) -- nothing is overwritten.
 *
 * A batch is `n_fields` opaque byte blobs (for example actions, rewards, discounts,
 * worker_logp, target_logits), field f taking field_bytes[f] bytes per slot.  Storage is
 * one device allocation owned by the handle (slot-major; every field starts on a 256-byte
 * boundary), or caller memory when `storage` is non-NULL (then it must hold
 * impact_buffer_storage_bytes() bytes, 256-byte aligned, and outlive the handle).
 * Slot bookkeeping (validity, traversal counts, cursors, draw counter) lives on the host.
 * A handle is not thread-safe.
 */
typedef struct impact_buffer impact_buffer;

/* Bytes of device storage a buffer with these fields needs; 0 on invalid arguments. */
size_t impact_buffer_storage_bytes(int32_t N, int32_t n_fields, const size_t* field_bytes);

/*
 * Creates a buffer.  field_bytes is a HOST array of n_fields (1..16) positive sizes.
 * sample_mode: IMPACT_SAMPLE_*.  Allocates device memory (cudaMalloc) unless `storage`
 * is given.  *out receives the handle.  Errors: INVALID_ARG, CUDA.
 */
int32_t impact_buffer_create(int32_t N, int32_t K, int32_t n_fields, const size_t* field_bytes,
                             uint64_t seed, int32_t sample_mode, void* storage,
                             impact_buffer** out);
/* Frees the handle and the storage it owns.  Synchronises the device first. */
int32_t impact_buffer_destroy(impact_buffer* h);

/*
 * A worker sends a batch (Worker-i, "Send B_i to C(N,K)").  Takes the first free slot at
 * or after the write cursor in ring order, copies every non-NULL field_src[f] (HOST array
 * of n_fields pointers; a NULL entry leaves that field for a later impact_buffer_append)
 * into it on `stream`, sets its traversal count to 0 and returns the slot in *slot_out.
 * src_location: IMPACT_SRC_DEVICE (one fused copy kernel) or IMPACT_SRC_HOST (one
 * cudaMemcpyAsync per field; use pinned memory to stay asynchronous).
 * Returns IMPACT_ERR_FULL, with nothing copied, when no slot is free.
 */
int32_t impact_buffer_push(impact_buffer* h, const void* const* field_src, int32_t src_location,
                           int32_t* slot_out, void* stream);

/*
 * The learner obtains a batch (Algorithm 1, "Obtain batch B ... traversed k times").
 * Picks a live slot (uniform seeded draw or round robin), returns it in *slot_out and
 * its traversal count BEFORE this call in *k_before_out (0 means the target network's
 * output still has to be appended), then counts the traversal; after the K-th the slot is
 * discarded (Algorithm 1, "If k = K, discard batch").
 * gather_dst: NULL for zero-copy use through impact_buffer_slot_ptr, else a HOST array of
 * n_fields device pointers (NULL entries skipped) that receive copies of the slot's
 * fields, enqueued on `stream` as one kernel.
 * A discarded slot may be overwritten by a later push: readers of a zero-copy slot must
 * be ordered before that push (same stream, or an event).
 * Returns IMPACT_ERR_EMPTY when no slot is live.
 */
int32_t impact_buffer_sample(impact_buffer* h, int32_t* slot_out, int32_t* k_before_out,
                             void* const* gather_dst, void* stream);

/*
 * Stores `src` (device, field_bytes[field] bytes) into one field of a slot: Algorithm 1,
 * "If k = 0, evaluate B on target, append target output to B".
 */
int32_t impact_buffer_append(impact_buffer* h, int32_t slot, int32_t field, const void* src,
                             void* stream);

/* Device address of a field of a slot (NULL on bad arguments). */
void* impact_buffer_slot_ptr(impact_buffer* h, int32_t slot, int32_t field);

/* Number of live slots, or a negative status. */
int32_t impact_buffer_live(const impact_buffer* h);

/*
 * Bookkeeping checkpoint: writes the host-side state (slot validity and counts, cursors,
 * draw counter, seed, shape) into `blob` (HOST).  impact_buffer_state_bytes gives the size.
 * Import requires a buffer created with the same N, K and fields.  Payload is not included.
 */
size_t impact_buffer_state_bytes(const impact_buffer* h);
int32_t impact_buffer_export_state(const impact_buffer* h, void* blob, size_t blob_bytes);
int32_t impact_buffer_import_state(impact_buffer* h, const void* blob, size_t blob_bytes);

/*
 * ---- bookkeeping on the device -------------------------------------------------------------------------------
 * Algorithm 1's "Obtain batch B ... traversed k times" / "If k = K, discard batch" and the workers' "Send B_i to
 * C(N,K)" (Section 3.2) with the slot bookkeeping kept in device memory: a learner iteration is then enqueued --
 * or captured into a CUDA graph and replayed -- without the host ever learning a slot number.  The protocol and the
 * draw are exactly those of impact_buffer_push / impact_buffer_sample (same trace for the same seed).
 *
 *   impact_buffer_device_begin   uploads the handle's bookkeeping (allocating a few kilobytes of device memory the
 *                                first time) and switches the handle to device mode: impact_buffer_push, _sample and
 *                                _import_state are refused until impact_buffer_device_end, which brings the
 *                                bookkeeping back to the host (synchronises `stream`).  impact_buffer_live and
 *                                _export_state keep working (they fetch the device's copy; synchronising).
 *   impact_buffer_device_step    one step on `stream`, in this order:
 *     (1) if push_sources != NULL: the next of n_candidates worker batches goes into the first free slot at or after
 *         the write cursor; with every slot live nothing happens (IMPACT_ERR_FULL in the event log).  push_sources is
 *         a DEVICE array of n_candidates x (n_fields + 1) pointers: for each candidate its n_fields field sources
 *         (NULL = leave the field for the append) and one extra pointer that is remembered with the slot -- the
 *         target network's output for that batch.  Candidates are taken in turn (pushes so far mod n_candidates).
 *         The copy itself is a second kernel enqueued by this call.
 *     (2) if inputs_out != NULL: a live slot is drawn, its count goes up, after the K-th traversal it is discarded,
 *         and *inputs_out (DEVICE memory, 16-byte aligned) receives the arguments of the loss call for that batch:
 *         the slot's fields named by `map` (-1 = not kept in the ring: NULL), learner_logits / values /
 *         bootstrap_values as passed here (the learner network's outputs for the batch), and for the target logits
 *         either the slot's field or -- at the batch's first traversal, when an extra pointer came with the batch --
 *         that pointer with the slot's field as target_logits_copy (Algorithm 1, "If k = 0, evaluate B on target,
 *         append target output to B", done by the loss call).  With no live slot status is IMPACT_ERR_EMPTY and the
 *         pointers of the previous draw stay in place.
 *     A loss call reads the record through impact_loss_call.inputs_on_device.  All steps and the loss calls that
 *     use their records belong on ONE stream.
 *   impact_buffer_device_events  the most recent outcomes, oldest first, as (op, status, slot, k_before) quadruples
 *                                of int32 (op 1 = push, 2 = sample; up to 4096 are kept); synchronises `stream`.
 */
typedef struct impact_ring_field_map {
    int32_t actions, rewards, discounts, worker_logp, target_logits; /* index of the ring field, or -1 */
} impact_ring_field_map;

typedef struct impact_loss_inputs { /* lives in DEVICE memory */
    const void* learner_logits;
    const void* target_logits;
    const float* worker_logp;
    const int32_t* actions;
    const float* rewards;
    const float* discounts;
    const float* values;
    const float* bootstrap_values;
    void* target_logits_copy;
    int32_t status, slot, k_before, pad;
} impact_loss_inputs;

int32_t impact_buffer_device_begin(impact_buffer* h, void* stream);
int32_t impact_buffer_device_end(impact_buffer* h, void* stream);
int32_t impact_buffer_device_step(impact_buffer* h, const impact_ring_field_map* map, const void* learner_logits,
                                  const float* values, const float* bootstrap_values,
                                  const void* const* push_sources, int32_t n_candidates,
                                  impact_loss_inputs* inputs_out, void* stream);
int32_t impact_buffer_device_events(impact_buffer* h, int32_t* events_out, int32_t max_events, int32_t* n_out,
                                    void* stream);

/*
 * Index gather of rows: dst[i, :] = src[idx[i], :] for i in [0, n), rows of row_bytes
 * bytes.  src, dst, idx are device pointers; idx is int32 with every entry in
 * [0, n_src_rows) (entries outside are clamped).  Bit-exact copy; src and dst must not
 * overlap.  row_bytes > 0; rows are copied with 16-byte accesses when src, dst and
 * row_bytes allow it, else with narrower ones.
 */
int32_t impact_gather_rows(const void* src, const int32_t* idx, int64_t n, int64_t n_src_rows,
                           size_t row_bytes, void* dst, void* stream);

/*
 * Measurement aid (no counterpart in the paper): reads read_bytes from src and writes the first write_bytes of
 * them to dst with plain 16-byte loads and stores -- the byte mix of a loss launch with no arithmetic in between,
 * launched the way the loss kernels are.  The benchmark times it beside the loss kernel to show what a batch of
 * that size allows at all.  src, dst device, 16-byte aligned; sizes multiples of 16, 16 <= write_bytes <=
 * read_bytes; the ranges must not overlap.
 */
int32_t impact_stream_copy(const void* src, size_t read_bytes, void* dst, size_t write_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* IMPACT_H_ */
