/*
 * dppo.h — C ABI of libdppo: the hot path of DPPO's pruned GRPO training step on one B200.
 *
 * DPPO ("Unbiased Dynamic Pruning for Efficient Group-Based Policy Optimization") prunes prompts
 * and completions of a GRPO batch at random, reweights what is retained by importance-sampling
 * factors so that the gradient stays unbiased, packs the retained sequences densely and trains on
 * them.  This library does, per batch:  group advantages -> candidate sets, pruning masks and
 * rescaling factors -> Dense Prompt Packing -> one sweep over the LM-head logits that yields the
 * loss and dlogits.
 *
 * Conventions (all entry points)
 *  - Return value: 0 (DPPO_OK) or a negative dppo_error.  Nothing throws, aborts or prints.
 *    dppo_last_error() gives the message of the calling thread's last failure.
 *  - Unless a parameter says "host", array pointers are DEVICE pointers owned by the caller.  The
 *    library allocates no memory and keeps no state between calls; scratch comes from a caller
 *    workspace sized by the matching *_workspace_bytes() (a pure host function).  The one exception is
 *    dppo_pack_prompts_static, whose scratch is an array inside the library that all its calls on a device
 *    share (see there).
 *  - Work is enqueued on `stream` (a cudaStream_t passed as void*); there is no host
 *    synchronisation inside.  Outputs are valid once the stream reaches that point.
 *  - Host-visible arguments are validated before anything is launched.  Problems only the device
 *    can see (a unit longer than a row, a target id outside the vocabulary, a wait that ran out)
 *    are recorded in the caller's `status` word (device int32, first error wins, caller zeroes it)
 *    as a positive dppo_status; the kernel then finishes without trapping.
 *  - Every output is a deterministic function of the inputs (no floating-point atomics).
 *  - Each entry point that enqueues work opens an NVTX range of its own name around its host side, so
 *    its launches are grouped under it in a timeline profiler.
 */
#ifndef DPPO_H_
#define DPPO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    DPPO_OK = 0,
    DPPO_ERR_INVALID_ARG = -1,          /* NULL where data is required, negative size, bad enum       */
    DPPO_ERR_BAD_SHAPE = -2,            /* sizes inconsistent with each other or above a stated limit */
    DPPO_ERR_MISALIGNED = -3,           /* base pointer or row stride not a multiple of 16 bytes      */
    DPPO_ERR_WORKSPACE_TOO_SMALL = -4,
    DPPO_ERR_UNSUPPORTED = -5,          /* dtype / option this build does not implement               */
    DPPO_ERR_CUDA = -6                  /* a CUDA runtime call failed (message has the CUDA error)    */
} dppo_error;

typedef enum {                          /* values of the device status word */
    DPPO_STATUS_OK = 0,
    DPPO_STATUS_BAD_LENGTH = 1,         /* pack: a retained unit has length < 1 or > L_row            */
    DPPO_STATUS_BAD_TARGET = 2,         /* loss: a target id outside [0, V)                           */
    DPPO_STATUS_TIMEOUT = 3,            /* a bounded device-side wait ran out                         */
    DPPO_STATUS_BAD_SEGMENTS = 4,       /* loss: cu_seqlens does not cover a token                    */
    DPPO_STATUS_BAD_INDEX = 5,          /* history: a prompt id outside the table                     */
    DPPO_STATUS_RANGE = 6               /* fused LM-head backward: a sampled token whose log-prob under the
                                           current policy is below about -66 (see dppo_lmhead_grpo_loss)  */
} dppo_status;

int dppo_version(void);                 /* major*10000 + minor*100 + patch */
const char* dppo_last_error(void);      /* host string, valid until the thread's next failing call */

/* ------------------------------------------------------------------------------------------------
 * Group-relative advantages — Eq. 2 (A_i = (r_i - mean)/std over the G completions of a prompt) and
 * the per-prompt threshold of Eq. 14 (Abar = mean_i |A_i|).
 *   rewards       f32 [P*G], row-major by prompt
 *   std_ddof      0 population std (default reading of "std"), 1 sample std
 *   std_eps       added to std before dividing (1e-6 by default; 0 allowed)
 *   adv           f32 [P*G] out;  mean_abs_adv f32 [P] out
 * A group whose rewards are all bitwise equal gets A = 0.  Arithmetic is binary64, one rounded
 * operation at a time in ascending i, rounded once to f32 — results are reproducible bit for bit.
 * Errors: INVALID_ARG (NULL, P<0, G<1, ddof not 0/1, eps<0).  P == 0 is a no-op.
 */
int dppo_group_advantages(const float* rewards, int P, int G, int std_ddof, double std_eps,
                          float* adv, float* mean_abs_adv, int32_t* status, void* stream);

/* ------------------------------------------------------------------------------------------------
 * Candidate sets, dynamic pruning masks, importance rescaling, history update —
 * Eq. 15 (completion policy), Eq. 17 (prompt policy), Eq. 18 (discrete rescaling), Eq. 16 (history).
 */
typedef struct {
    int32_t P, G;
    double r_q, r_o;        /* pruning probabilities in [0,1): a candidate is pruned when u < r      */
    int32_t mode;           /* 0: independent Bernoulli draws (Eq. 15, 17).
                               1: fixed fraction (Appendix A / Algorithm 1): prune the floor(r*|C|)
                                  candidates with the smallest u, ties to the lower index           */
    int32_t reverse;        /* 0: low-|A| completions / low-H prompts are the candidates (the paper's
                               rule); 1: the opposite sets (the ablation of Table 5)                 */
    uint64_t seed, step;    /* Philox4x32-10 key / counter words when u_q,u_o are NULL:
                               key=(seed lo,hi), counter=(index, domain, step lo, step hi),
                               domain 1 prompts (index k), 2 completions (index k*G+i);
                               u = ((out0 | out1<<32) >> 11) * 2^-53                                 */
} dppo_prune_params;

/*   adv, mean_abs_adv   outputs of dppo_group_advantages
 *   H_prev   f32 [P] history scores H_{t-1}(q_k); NULL in the first epoch: no prompt is a candidate
 *   u_q      f64 [P],  u_o f64 [P*G]: explicit draws in [0,1) replacing the generator (NULL: generate)
 *   cand_q   u8 [P]    the floor(P/2) prompts with the lowest H_prev (ties: lower index)
 *   cand_o   u8 [P*G]  |A_i| <= Abar_k, taken as G*|A_i| <= (sum_j |A_j|)*(1+1e-12) in binary64
 *   keep_q   u8 [P];  keep_o u8 [P*G] (all 0 for a pruned prompt)
 *   n_keep_q i32 [1] = |S^q|;  n_keep_o i32 [P] = |S^o(q_k)|
 *   gamma_q  f32 [P]   (|S^q|/P)/(1-P^q);  gamma_o f32 [P*G] (|S^o_k|/G)/(1-P^o); 0 where pruned
 *   w_seq    f32 [P*G] weight of a completion in the pruned objective read as the mean over retained
 *                      prompts of gamma_q x mean over retained completions of gamma_o x term:
 *                      1/(P*G*(1-P^q)*(1-P^o)); 0 where pruned
 *   H_next   f32 [P]   Abar_k if the prompt was retained (or H_prev is NULL), else H_prev[k]
 * In mode 1, P^q and P^o in these formulas are the realised fractions floor(r|C|)/|C| (the true
 * inclusion probabilities), so the weights stay unbiased.
 * Errors: INVALID_ARG (NULL outputs, r outside [0,1), bad mode), BAD_SHAPE (P*G >= 2^31).
 */
int dppo_prune_and_rescale(const dppo_prune_params* p, const float* adv, const float* mean_abs_adv,
                           const float* H_prev, const double* u_q, const double* u_o,
                           uint8_t* cand_q, uint8_t* cand_o, uint8_t* keep_q, uint8_t* keep_o,
                           int32_t* n_keep_q, int32_t* n_keep_o, float* gamma_q, float* gamma_o,
                           float* w_seq, float* H_next, int32_t* status, void* stream);

/* ------------------------------------------------------------------------------------------------
 * History scores across epochs — Eq. 16 keeps one score H_t(q) per DATASET prompt; Algorithm 1 starts
 * from H_0 = 0 and skips prompt pruning in the first epoch.  A batch gathers the scores of its prompts
 * before dppo_prune_and_rescale (H_prev) and scatters H_next back afterwards: retained prompts get
 * their fresh mean |A|, pruned ones keep their old score (the carry-forward).
 *   H_table     f32 [N] one score per dataset prompt (caller zero-initialises it)
 *   prompt_ids  i32 [P] dataset index of each prompt of the batch (distinct within a batch)
 *   H_batch     f32 [P] out of gather;  H_next f32 [P] in to scatter
 * An id outside [0, N) sets status DPPO_STATUS_BAD_INDEX (gather returns 0 for it, scatter skips it).
 */
int dppo_history_gather(const float* H_table, int N, const int32_t* prompt_ids, int P, float* H_batch,
                        int32_t* status, void* stream);
int dppo_history_scatter(float* H_table, int N, const int32_t* prompt_ids, int P, const float* H_next,
                         int32_t* status, void* stream);

/* ------------------------------------------------------------------------------------------------
 * Dense Prompt Packing — Section 4.3 (window-based greedy selection from a candidate pool W of
 * size N_win, refilled from the stream, into rows of capacity L_row).
 */
typedef struct {
    int32_t n_max;          /* units offered (retained or not)                                       */
    int32_t L_row;          /* row capacity in tokens                                                */
    int32_t N_win;          /* pool size, >= 1                                                       */
    int32_t policy;         /* 0 first unit in pool order that fits; 1 longest that fits (ties: oldest) */
} dppo_pack_params;

size_t dppo_pack_workspace_bytes(const dppo_pack_params* p);

/*   len        i32 [n_max] tokens of each unit (prompt + response)
 *   keep       u8  [n_max] or NULL: units with keep == 0 are not in the stream
 *   loss_len   i32 [n_max] or NULL: loss (response) tokens of each unit; NULL: = len
 *   order      i32 [n_max] out: order[p] = unit placed p-th, for p < n_units; -1 beyond
 *   row_of, off_in_row  i32 [n_max] out, indexed by unit; -1 for units not in the stream
 *   row_fill   i32 [n_max] out: tokens used in row r, for r < n_rows; 0 beyond
 *   cu_seqlens i32 [n_max+1] out: exclusive scan of loss_len in placement order; entries past
 *              n_units repeat the total, so the array is non-decreasing over its whole length
 *   counts     i32 [4] out: n_units, n_rows, total tokens, total loss tokens
 * A retained unit with length < 1 or > L_row sets status DPPO_STATUS_BAD_LENGTH and packs nothing
 * (counts = 0); so does a stream whose tokens add up to 2^31 or more (the counts are i32).  The limit is
 * n_max <= 2,097,152 units (a dataset-sized stream, packed once at set-up; one warp places about a million units
 * per second).  Errors: INVALID_ARG, BAD_SHAPE (n_max above the limit: the workspace query reports 0 bytes),
 * WORKSPACE_TOO_SMALL.
 */
int dppo_pack_prompts(const dppo_pack_params* p, const int32_t* len, const uint8_t* keep,
                      const int32_t* loss_len, int32_t* order, int32_t* row_of, int32_t* off_in_row,
                      int32_t* row_fill, int32_t* cu_seqlens, int32_t* counts,
                      void* workspace, size_t workspace_bytes, int32_t* status, void* stream);

/* ------------------------------------------------------------------------------------------------
 * Packing without a caller workspace.  (The paper has no counterpart: this entry point exists for the
 * sake of callers, not of the method.)
 *
 * Same operation, same arguments and same results as dppo_pack_prompts, minus `workspace`: the
 * scratch is a fixed 32 KB array inside the library's device image.  It is meant for callers that
 * have no way to hand over device scratch at the point of the call: host code that is given only
 * its input and output buffers by a framework and owns no allocator, or a training loop whose
 * device memory is entirely reserved by a pool, where a cudaMalloc would fail or would stall every
 * stream while it runs.  The call itself allocates nothing (no cudaMalloc / cudaFree, no library
 * allocation).
 *
 *  - Limit: n_max <= dppo_pack_static_max_units() (8192 units); larger requests return
 *    DPPO_ERR_BAD_SHAPE and launch nothing.  Every GPU that loads the library holds the 32 KB until
 *    the process ends, used or not.
 *  - The first call on each device looks up the array's device address (cudaGetSymbolAddress, with
 *    that device current) and caches it; make that first call before starting any stream capture.
 *    The cached address belongs to the device's context at that time: after cudaDeviceReset (or any
 *    other way of replacing that context) this entry point must not be used again in the process.
 *  - All calls on a device share the one array.  It keeps whatever the previous call left there;
 *    the kernel never reads a slot before writing it, so nothing needs clearing.  Two calls whose
 *    kernels can overlap on the GPU (different streams, no ordering between them) race on it:
 *    keep calls on one stream or order them yourself.
 */
int dppo_pack_static_max_units(void);
int dppo_pack_prompts_static(const dppo_pack_params* p, const int32_t* len, const uint8_t* keep,
                             const int32_t* loss_len, int32_t* order, int32_t* row_of,
                             int32_t* off_in_row, int32_t* row_fill, int32_t* cu_seqlens,
                             int32_t* counts, int32_t* status, void* stream);

/* ------------------------------------------------------------------------------------------------
 * Fused loss sweep over the logits — Eq. 1 (clipped surrogate minus beta x KL, 1/|o_i| per sequence,
 * KL estimator rho_hat - log rho_hat - 1) with the sequence weights of dppo_prune_and_rescale, and
 * its gradient with respect to the logits.
 *
 * For token t of sequence s (cu_seqlens[s] <= t < cu_seqlens[s+1]), target y, A = adv[s], W =
 * w[s]/|o_s|:  z = logits[t,:]/temperature;  lse = log sum_v exp z_v;  logp = z_y - lse;
 * rho = exp(logp - logp_old);  d = logp_ref - logp;  kl = e^d - d - 1;
 * surr = min(rho A, clip(rho, 1-eps_lo, 1+eps_hi) A);  loss = -sum_t W (surr - beta kl);
 * g = dloss/dlogp = -W (A rho [clipped branch not strictly smaller] + beta (e^d - 1));
 * dlogits[t,v] = g ([v == y] - exp(z_v - lse)) / temperature.
 */
typedef enum { DPPO_F32 = 0, DPPO_BF16 = 1 } dppo_dtype;

typedef struct {
    int64_t T_max;          /* rows of logits / upper bound of loss tokens                           */
    int32_t V;              /* vocabulary size                                                       */
    int32_t dtype;          /* dppo_dtype of logits and dlogits                                      */
    int64_t row_stride;     /* elements between consecutive rows (>= V; bytes a multiple of 16)      */
    int32_t S_max;          /* cu_seqlens has S_max+1 entries, non-decreasing, last >= true T        */
    int32_t variant;        /* 0: the library picks the kernel.  Tuning aid: 1 forces the general two-pass
                               kernel, 2 the warp-per-row kernel (rows up to 8 KB), 3 the streaming kernel (forward-only
                               calls), 4 the tile kernel (dense rows of up to 32 KB),
                               C*10000+threads the shared-memory kernel with C = 1, 2, 4 or 8
                               CTAs per row and 128 / 256 / 512 / 1024 threads per CTA.
                               Self-test of the bounded waits: 1000000 + (0, 3, 4 or a C*10000+threads code) runs
                               the shared-memory, streaming or tile kernel with a barrier expecting a few bytes
                               more than are ever sent and a wait limit of 1 ms: every row then ends as a
                               timed-out row does (status DPPO_STATUS_TIMEOUT; the row's dlogits, logp_out,
                               lse_out and loss terms are zero) and nothing hangs                    */
    double eps_lo, eps_hi;  /* clip range 1-eps_lo .. 1+eps_hi (the paper: both 0.2)                 */
    double beta;            /* KL coefficient                                                        */
    double temperature;     /* > 0 (the paper: 1)                                                    */
    /* Variants for the other objectives the paper combines the method with (Section 5.2); zero / NULL
       give Eq. 1 as printed. */
    int32_t no_length_norm; /* 1: W = w[s] instead of w[s]/|o_s| (a token-level mean is then up to the w
                               the caller passes)                                                    */
    int32_t reserved2;      /* 0                                                                     */
    const float* seq_log_ratio; /* device f32 [S_max] or NULL.  Given: every token of sequence s uses the
                               sequence-level ratio rho = exp(seq_log_ratio[s]) (from
                               dppo_sequence_log_ratio on the current log-probs, i.e. after a forward-only
                               call) in place of exp(logp - logp_old); requires no_length_norm == 0     */
} dppo_loss_params;

size_t dppo_grpo_loss_workspace_bytes(const dppo_loss_params* p);

/*   logits       [T_max x row_stride] of dtype, read-only unless dlogits aliases it
 *   target       i32 [T_max] sampled token ids
 *   logp_old, logp_ref  f32 [T_max] log-probs of the target under the old / reference policy
 *   cu_seqlens   i32 [S_max+1]
 *   n_tokens_dev i32 [1] true number of tokens T <= T_max on the device, or NULL (T = T_max);
 *                rows >= T are neither read nor written
 *   adv, w       f32: advantage and sequence weight of each sequence, read at index seg_map[s]
 *                when seg_map (i32 [S_max], e.g. the packer's `order`) is given, else at index s
 *   dlogits      same dtype/stride as logits; may alias logits (in place); NULL: forward only
 *   logp_out, lse_out   f32 [T_max] or NULL
 *   loss_out     f32 [5]: loss, policy-gradient part -sum W surr, sum W kl, clipped fraction, T
 * Errors: INVALID_ARG, BAD_SHAPE, MISALIGNED (logits/dlogits base or row stride), UNSUPPORTED
 * (dtype), WORKSPACE_TOO_SMALL.  Device status: BAD_TARGET, BAD_SEGMENTS (a row below T that cu_seqlens does not
 * cover): such a row's dlogits are zero, its logp_out is 0 (its lse_out is still the row's log-sum-exp) and it adds
 * nothing to the loss; the other rows are not affected.
 */
int dppo_grpo_loss_fwd_bwd(const dppo_loss_params* p, const void* logits, const int32_t* target,
                           const float* logp_old, const float* logp_ref, const int32_t* cu_seqlens,
                           const int32_t* n_tokens_dev, const float* adv, const float* w,
                           const int32_t* seg_map, void* dlogits, float* logp_out, float* lse_out,
                           float* loss_out, void* workspace, size_t workspace_bytes,
                           int32_t* status, void* stream);

/* Which kernel a dppo_grpo_loss_fwd_bwd call with these parameters runs on the current device (a host-side query:
 * it makes the same choice and the same device checks as the call and launches nothing).  Dense rows (V a whole
 * number of 16-byte vectors) of up to 16 KB go to the tile kernel.  Other rows of
 * up to 8 KB go to the warp-per-row kernel, rows that fit eight shared-memory slices to the shared-memory
 * kernel, longer ones to the general two-pass kernel; a forward-only call (forward_only != 0: the call will pass
 * dlogits = NULL) on rows of 128 KB and more goes to the streaming kernel.  fell_back = 1 says that the device refused the kernel the
 * row length asked for (its shared memory or cluster size) and the slower general kernel runs instead.
 * Errors: INVALID_ARG; UNSUPPORTED when params.variant forces a kernel that cannot take the shape.
 */
typedef enum { DPPO_KERNEL_GENERAL = 0, DPPO_KERNEL_WARP = 1, DPPO_KERNEL_SHARED = 2, DPPO_KERNEL_STREAM = 3, DPPO_KERNEL_TILE = 4 } dppo_loss_kernel;
typedef struct {
    int32_t kernel;         /* dppo_loss_kernel                                                      */
    int32_t ctas_per_row;   /* cluster size of the shared-memory kernel, else 1                      */
    int32_t threads;        /* threads that work on one row at a time in each CTA                    */
    int32_t fell_back;      /* 1: general kernel in place of the one the row length asked for        */
} dppo_loss_kernel_choice;
int dppo_grpo_loss_kernel_choice(const dppo_loss_params* p, int forward_only, dppo_loss_kernel_choice* out);

/* Mean token log-ratio of each sequence, out[s] = mean_t (logp[t] - logp_old[t]) over cu_seqlens[s] <= t <
 * cu_seqlens[s+1] (0 for an empty sequence): the log of the length-normalised sequence-level likelihood
 * ratio of sequence-level objectives (Section 5.2).  logp, logp_old f32 [T]; out f32 [S_max].  Binary64
 * accumulation in a fixed order.  Errors: INVALID_ARG.
 */
int dppo_sequence_log_ratio(const float* logp, const float* logp_old, const int32_t* cu_seqlens, int S_max,
                            float* out, int32_t* status, void* stream);

/* ------------------------------------------------------------------------------------------------
 * Fused LM-head + loss: the same loss as dppo_grpo_loss_fwd_bwd with the logits z = hidden W^T
 * produced on the fly by the tensor cores; the [T x V] logits of the batch are never written to memory
 * (Eq. 1's pi_theta is the log-softmax of exactly these logits).
 *
 *   loss     the loss parameters; dtype must be DPPO_BF16; row_stride and variant are ignored
 *   H        hidden width, a multiple of 64
 *   hidden   bf16 [T_max x H] row-major, one row per loss token in packed order
 *   W        bf16 [V x H] row-major LM-head weight
 *   backward 0: forward only (loss_out, logp_out, lse_out; dhidden and dW must be NULL).
 *            1: also the gradients, dhidden = D W and dW = D^T hidden with D = dlogits.  The tokens are taken 9472
 *            at a time.  A chunk's exponentials are kept in workspace scratch as bf16, relative to each row's own
 *            reference, the sampled token's logit (never the full [T x V], and never the logits themselves); D is
 *            that scratch times one factor per row, so the two contractions read the scratch directly and no
 *            dlogits array is formed.  The reference bounds the representable rows: a sampled token whose log-prob
 *            under the current policy is below about -66 sets status DPPO_STATUS_RANGE; that row adds nothing to
 *            the loss and its gradient is zero
 *   dhidden  bf16 [T_max x H] out (rows at or past the true token count are zero)
 *   dW       [V x H] out, f32 or (params.dW_dtype = DPPO_BF16) bf16; overwritten, or added to when
 *            params.accumulate_dW = 1.  It is summed over the chunks in f32 either way (for bf16 in a workspace
 *            buffer, rounded once at the end).  Each element receives one add per chunk, in stream order: the
 *            result does not vary from run to run
 *   other arguments as in dppo_grpo_loss_fwd_bwd.  The workspace (dppo_lmhead_workspace_bytes, which
 *   depends on `backward`) must be 1024-byte aligned.
 * Errors: INVALID_ARG, BAD_SHAPE (H not a multiple of 64), MISALIGNED, UNSUPPORTED, WORKSPACE_TOO_SMALL,
 * CUDA (tensor-map creation).  Device status: BAD_TARGET, BAD_SEGMENTS, RANGE, TIMEOUT.
 */
typedef struct {
    dppo_loss_params loss;
    int32_t H;
    int32_t backward;
    int32_t variant;        /* 0: CTA pairs (cta_group::2) share each B tile; 1: one CTA per tile (tuning aid).
                               100 / 101: the same two with the self-test of the bounded waits: the first pipeline
                               stage of every CTA expects 16 bytes more than are ever copied and the wait limit
                               is 1 ms, so every CTA gives up, frees its tensor memory and returns; the call
                               reports DPPO_STATUS_TIMEOUT and its other outputs are unspecified    */
    int32_t dW_dtype;       /* DPPO_F32 (0) or DPPO_BF16: element type of dW */
    int32_t accumulate_dW;  /* 0: dW is overwritten; 1: the gradient is added to what dW holds (micro-batches) */
    int32_t reserved;       /* 0 */
} dppo_lmhead_params;

size_t dppo_lmhead_workspace_bytes(const dppo_lmhead_params* p);

int dppo_lmhead_grpo_loss(const dppo_lmhead_params* p, const void* hidden, const void* W,
                          const int32_t* target, const float* logp_old, const float* logp_ref,
                          const int32_t* cu_seqlens, const int32_t* n_tokens_dev, const float* adv,
                          const float* w, const int32_t* seg_map, void* dhidden, void* dW,
                          float* logp_out, float* lse_out, float* loss_out, void* workspace,
                          size_t workspace_bytes, int32_t* status, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* DPPO_H_ */
