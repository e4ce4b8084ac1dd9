/*
 * fork_dllm.h — C ABI of the Fork-dLLM confidence pass for NVIDIA B200 (sm_100a).
 *
 * One sampling step of a masked diffusion language model, as Fork-dLLM defines it
 * (Algorithm 2 of the paper; Section 2, "Sampling in masked dLLMs"):
 *   M_t   = still-masked positions (here: mask[b,k] != 0 inside the sequence's active block),
 *   x_0^k = candidate token; at temperature 0 the arg-max of the position's distribution,
 *   c_t^k = q_theta^k(x_0^k | x_t) = its softmax probability (the largest one at temperature 0),
 *   U_t   = {k in M_t : c_t^k > lambda}; if U_t is empty, U_t = {leftmost(M_t)}   (the Fork fallback),
 *   x_{t-1}^k = x_0^k for k in U_t.
 * Besides the commit, the step emits per position the confidence, candidate, token entropy
 * (Section 3.1) and log-probability, and per sequence whether the step was a fallback step
 * (the set F_i of Section 3.2), which is what ForkGRPO scores.
 *
 * Entry points: fork_step (one step), fork_decode_loop (steps until nothing is masked),
 * fork_logprob (log-likelihood scoring of Section 3.2), fork_step_host (host buffers),
 * fork_step_static (no workspace argument), fork_step_fused_head (the step fused into the LM-head
 * product: hidden states and weight in, no logits in memory) and fork_decode_loop_fused_head (the
 * loop on hidden states); the variants the paper compares with or trains with:
 * candidates drawn at temperature tau > 0 and the other fallback orders (fields of fork_step_args),
 * fork_select_top_entropy (JustGRPO-Fast's position selection), fork_grpo_loss (Eq. 2),
 * fork_logprob_backward (its log-softmax backward) and fork_grpo_fused (the three in one pass); fork_vp_reduce / fork_vp_reduce_peers /
 * fork_vp_select (the step with the vocabulary sharded over ranks).
 *
 * Conventions for every entry point
 *   - All data pointers are DEVICE pointers owned by the caller unless a comment says "host".
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  fork_step and
 *     fork_logprob only enqueue work on it and return; results are in device memory once the
 *     stream reaches that point.  They never synchronise, and never allocate or free device
 *     memory (the first call with a new workspace address adds an entry to a small host table).
 *   - `workspace` is device scratch of at least fork_workspace_bytes(B, Lt) bytes, 256-byte
 *     aligned, private to one call at a time on one stream; its contents need not be kept
 *     between calls (fork_decode_loop keeps its block cursors there while it runs) and need
 *     not be initialised.  State that must be clean when a kernel starts (the one-kernel step,
 *     see FORK_TUNE_ONE_KERNEL) lives in control blocks inside the library, one per workspace
 *     address and device, up to 1024 at a time (fork_workspace_release gives one back); workspace
 *     addresses beyond that run the two-kernel step.
 *   - Argument errors are found on the host before anything is launched and return
 *     FORK_ERR_INVALID_ARG / FORK_ERR_WORKSPACE; a failed launch returns FORK_ERR_CUDA.
 *   - Logits rows are contiguous in V.  Row (b,k) starts at element
 *       b*stride_b + (k - pos0)*stride_l
 *     of `logits`; the buffer covers positions pos0 .. pos0+Ll-1 (pos0 = 0 and Ll = Lt for a
 *     full [B,Lt,V] tensor, or one block's window).  Rows that are not live are never read, so
 *     they may hold anything.  The fast path needs the base pointer and both strides to be
 *     multiples of 16 bytes; otherwise a slower scalar path runs (same results).
 *   - Vocabulary ties go to the lowest index.  A logit of -inf has probability 0.  A row that
 *     holds NaN or +inf, or only -inf, gets FORK_ROW_NONFINITE in row_status, confidence 0,
 *     NaN entropy / log-probability, and as candidate the lowest index of the maximum over
 *     its non-NaN entries (0 if it has none).
 */
#ifndef FORK_DLLM_H
#define FORK_DLLM_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum fork_status {
  FORK_OK = 0,
  FORK_ERR_INVALID_ARG = -1,
  FORK_ERR_CUDA = -2,
  FORK_ERR_WORKSPACE = -3,
  FORK_ERR_MAX_STEPS = -4,
  FORK_ERR_PROVIDER = -5
} fork_status;

typedef enum fork_dtype { FORK_BF16 = 0, FORK_F32 = 1 } fork_dtype;

/* bits of row_status[b,k] */
#define FORK_ROW_NONFINITE 1u /* NaN or +inf in the row, or nothing but -inf */
#define FORK_ROW_BAD_TOKEN 2u /* fork_logprob: token id outside [0,V) */

/* bits of the device status word (fork_device_status) */
#define FORK_DEV_WINDOW_CLAMPED 1u /* a block [lo,hi) reached outside [pos0,pos0+Ll) or [0,Lt) and was clipped */
#define FORK_DEV_TIMEOUT 2u        /* a bounded in-kernel wait gave up; the results of that call are not valid.  Reading
                                      this bit with fork_device_status also puts the library's control block of that
                                      workspace back to its initial state; do that before the next step on it. */

/*
 * Arguments of one sampling step (Algorithm 2; inputs x_t, q_theta, lambda -> x_{t-1}).
 * Output pointers marked "optional" may be NULL.
 */
/*
 * Which position a fallback step (no confidence above lambda) commits.
 *   LEFTMOST    Fork-dLLM: the leftmost masked position of the block (Algorithm 2, highlighted line)
 *   MAX_CONF    Fast-dLLM: arg-max_k c_t^k (Algorithm 1)
 *   MIN_CONF, MAX_ENTROPY, RANDOM   the fallback ablations of Section 4.1 (lowest confidence,
 *               highest token entropy, a random masked position)
 * Equal keys go to the lower position.  Rows flagged FORK_ROW_NONFINITE are passed over unless every
 * live row of the block is flagged, in which case the leftmost is taken.  A step with a non-empty
 * threshold set is the same under every mode.
 */
typedef enum fork_fallback_mode {
  FORK_FALLBACK_LEFTMOST = 0,
  FORK_FALLBACK_MAX_CONF = 1,
  FORK_FALLBACK_MIN_CONF = 2,
  FORK_FALLBACK_MAX_ENTROPY = 3,
  FORK_FALLBACK_RANDOM = 4
} fork_fallback_mode;

typedef struct fork_step_args {
  const void* logits;        /* model output q_theta(.|x_t) as logits; see the layout rule above */
  int64_t stride_b, stride_l;/* in elements; stride_l >= V */
  int32_t pos0;              /* sequence position of logits row 0 */
  int32_t B, Lt, Ll, V;      /* sequences, sequence-buffer length, logits rows per sequence, vocabulary */
  int32_t dtype;             /* fork_dtype of the logits */
  int32_t* tokens;           /* [B,Lt] in/out: x_t -> x_{t-1}; written only at committed positions */
  uint8_t* mask;             /* [B,Lt] in/out: 1 = still [MASK]; cleared at committed positions */
  const int32_t* blk_lo;     /* [B] active block, half open [lo,hi), absolute positions; */
  const int32_t* blk_hi;     /*     lo == hi means the sequence takes no part in this step */
  float threshold;           /* lambda; commit iff confidence > lambda (strict) */
  int32_t step;              /* id written into commit_step */
  /* per position, written for every live position (masked and inside the block); all optional */
  float* conf;               /* [B,Lt] c_t^k */
  int32_t* cand;             /* [B,Lt] x_0^k */
  float* entropy;            /* [B,Lt] token entropy of q_theta^k in nats */
  float* logp;               /* [B,Lt] log q_theta^k(x_0^k | x_t) = ln conf */
  uint32_t* row_status;      /* [B,Lt] FORK_ROW_* bits */
  /* per position, written only at positions committed by this step; all optional.
     (conf/entropy/logp are last written at the step that commits the position, so after a
     decode loop they hold the values at commit time.) */
  int32_t* commit_step;      /* [B,Lt] */
  uint8_t* commit_fallback;  /* [B,Lt] 1 if committed by a fallback step (a step in F_i) */
  float* commit_logp;        /* [B,Lt] log-probability of the committed token (old-policy term of the ForkGRPO ratio) */
  /* per sequence; all optional */
  int32_t* n_unmasked;       /* [B] |U_t| (0 if the sequence had no live position) */
  uint8_t* is_fallback;      /* [B] 1 if U_t was empty and the fallback position was taken */
  int32_t* fallback_pos;     /* [B] that position, else -1 */
  int32_t* nfe;              /* [B] += 1 if the sequence had a live position (model evaluations used) */
  int32_t* n_fallback;       /* [B] += is_fallback */
  /* variants the paper compares with; all zero = Algorithm 2 with arg-max candidates */
  int32_t fallback_mode;     /* fork_fallback_mode: which position a fallback step commits */
  const uint32_t* fallback_rand; /* [B] FORK_FALLBACK_RANDOM only: the step takes live position number
                                (fallback_rand[b] mod live count) of the block, counted from the left;
                                read at every step, so a loop's provider may refresh it */
  float temperature;         /* tau >= 0 of Algorithm 2 line 4; 0 = arg-max candidates */
  uint64_t sample_seed;      /* stream of uniform variates that draws the candidates when tau > 0 */
  void* sample_scratch;      /* tau > 0 only: DEVICE scratch of at least fork_sample_scratch_bytes(B, Lt) bytes, 256-byte
                                aligned, private to one call at a time like the workspace (FORK_ERR_WORKSPACE if missing).
                                Unlike the workspace it must be ZERO-FILLED before its first use (its first 4*B*Lt
                                bytes hold per-row arrival counters that every call leaves at zero again; after a call
                                that reported FORK_DEV_TIMEOUT, zero them once more). */
  size_t sample_scratch_bytes;
} fork_step_args;

/*
 * Arguments of the log-likelihood scoring used by ForkGRPO (Section 3.2): for every selected
 * position (select[b,k] != 0, normally the fallback steps' positions k_{i,t}) the log-probability
 * of the given token under the given logits, log q_theta^k(x^k | .) = x_tok - max - ln sum exp.
 */
typedef struct fork_logprob_args {
  const void* logits; int64_t stride_b, stride_l; int32_t pos0;
  int32_t B, Lt, Ll, V; int32_t dtype;
  const int32_t* tokens;     /* [B,Lt] token whose likelihood is wanted */
  const uint8_t* select;     /* [B,Lt] */
  float* logp;               /* [B,Lt] out: log-probability where selected, 0 elsewhere */
  float* seq_sum;            /* [B] out, optional: sum of logp over the sequence's selected positions */
  int32_t* seq_cnt;          /* [B] out, optional: number of selected positions (|F_i|) */
  uint32_t* row_status;      /* [B,Lt] out, optional: FORK_ROW_* bits at selected positions.
                                A token outside [0,V) sets FORK_ROW_BAD_TOKEN and scores 0. */
  float* lse;                /* [B,Lt] out, optional: log-sum-exp (max + ln sum exp) of every selected row,
                                which fork_logprob_backward takes back; untouched elsewhere */
} fork_logprob_args;

/*
 * The ForkGRPO objective (Eq. 2) on B = prompts * group rollouts, rollout i = prompt * group + j:
 *     rho_{i,t} = exp(logp_new - logp_old) at the selected positions (the fallback steps F_i),
 *     A_i       = (r_i - mean of its group) / (population standard deviation of its group);
 *                 a group whose rewards are all equal is skipped (A_i = 0 for its rollouts),
 *     obj_i     = 1/|F_i| * sum_t min(rho A_i, clip(rho, 1 - eps_lo, 1 + eps_hi) A_i), 0 if F_i is empty,
 *     J         = 1/B * sum_i obj_i,
 *     dlogp     = dJ/dlogp_new = rho A_i / (B |F_i|) where the unclipped term is the minimum, else 0.
 * All pointers are device memory.
 */
typedef struct fork_grpo_args {
  int32_t B, Lt, group;      /* B must be a multiple of group */
  const float* logp_new;     /* [B,Lt] log q_theta(token) at the selected positions (fork_logprob) */
  const float* logp_old;     /* [B,Lt] log q_theta_old(token) there (commit_logp of the rollout) */
  const uint8_t* select;     /* [B,Lt] non-zero at the positions of F_i */
  const float* reward;       /* [B] */
  float eps_lo, eps_hi;      /* clip range [1 - eps_lo, 1 + eps_hi] */
  float* seq_obj;            /* [B] out: obj_i */
  float* objective;          /* [1] out, optional: J */
  float* adv;                /* [B] out, optional: A_i */
  float* ratio;              /* [B,Lt] out, optional: rho at selected positions, 0 elsewhere */
  float* dlogp;              /* [B,Lt] out, optional: dJ/dlogp_new, 0 where not selected */
  uint8_t* skipped;          /* [B/group] out, optional: 1 for a group with equal rewards */
} fork_grpo_args;

/*
 * Derivative of the scored log-likelihoods with respect to the logits (the log-softmax backward
 * of Section 3.2's likelihood terms): for every selected position with a token inside [0,V),
 *     grad[b,k,v] = dlogp[b,k] * (1[v == token] - exp(logits[b,k,v] - lse[b,k])),
 * written over the whole row in the logits' dtype (bf16: round to nearest even).  Rows of
 * positions that are not selected, or whose token is outside [0,V), are not touched.
 */
typedef struct fork_logprob_bwd_args {
  const void* logits; int64_t stride_b, stride_l; int32_t pos0;
  int32_t B, Lt, Ll, V; int32_t dtype;
  const int32_t* tokens;     /* [B,Lt] */
  const uint8_t* select;     /* [B,Lt] */
  const float* lse;          /* [B,Lt] from fork_logprob on the same logits */
  const float* dlogp;        /* [B,Lt] upstream derivative (fork_grpo_loss) */
  void* grad;                /* out: same dtype and row addressing as logits, with its own strides */
  int64_t grad_stride_b, grad_stride_l;   /* in elements; grad_stride_l >= V */
} fork_logprob_bwd_args;

/*
 * ForkGRPO's pass over the new policy's logits in one call (Section 3.2, Eq. 2): for every selected
 * position (the fallback steps F_i; logits are [B, Lt, V], the window is the whole buffer) the
 * log-likelihood of the given token as fork_logprob computes it, the ratio and dJ/dlogp_new as
 * fork_grpo_loss computes them, and the gradient row of fork_logprob_backward for that dlogp -- with
 * every selected row read from HBM once and its gradient written once (the three calls in a row read
 * it twice).  Same results as the three calls.  `logp`, `lse`, `row_status`, `ratio` and `dlogp` are
 * written at the selected positions only; rows of `grad` that belong to unselected positions, or to
 * tokens outside [0,V), are not touched.  All pointers are device memory.
 */
typedef struct fork_grpo_fused_args {
  const void* logits; int64_t stride_b, stride_l;
  int32_t B, Lt, V; int32_t dtype;
  const int32_t* tokens;     /* [B,Lt] */
  const uint8_t* select;     /* [B,Lt] non-zero at the positions of F_i */
  int32_t group;             /* B must be a multiple of group; rollout i = prompt * group + j */
  const float* logp_old;     /* [B,Lt] log q_theta_old(token) at the selected positions */
  const float* reward;       /* [B] */
  float eps_lo, eps_hi;      /* clip range [1 - eps_lo, 1 + eps_hi] */
  void* grad;                /* out: d J / d logits, same dtype and row addressing as logits, with its own strides */
  int64_t grad_stride_b, grad_stride_l;   /* in elements; grad_stride_l >= V */
  float* logp;               /* [B,Lt] out: log q_theta(token) */
  float* lse;                /* [B,Lt] out, optional */
  uint32_t* row_status;      /* [B,Lt] out, optional: FORK_ROW_* bits */
  float* seq_obj;            /* [B] out: obj_i of Eq. 2 */
  float* objective;          /* [1] out, optional: J */
  float* adv;                /* [B] out, optional: A_i */
  float* ratio;              /* [B,Lt] out, optional: rho */
  float* dlogp;              /* [B,Lt] out, optional: dJ/dlogp_new */
  uint8_t* skipped;          /* [B/group] out, optional: 1 for a group with equal rewards */
} fork_grpo_fused_args;

/* Device scratch needed by any entry point for a batch of B sequences of buffer length Lt. */
size_t fork_workspace_bytes(int32_t B, int32_t Lt);

/* Additional device scratch of a step that draws its candidates (temperature > 0): 1060 bytes per
   position plus 2 MB; zero-filled once by the caller (see fork_step_args.sample_scratch).  How the draw works (Algorithm 2 line 4 fixes its distribution, softmax(x / tau),
   not the method): by inversion.  The vocabulary is laid out in a fixed order -- 16-byte vectors of
   logits dealt round robin to 256 lanes, lane after lane, the fewer-than-a-vector trailing entries last
   --, the weights exp((x - max) / tau) are summed along it in the same pass that computes the soft-max
   statistics (one more exponential per logit), and the candidate is the first entry at which the
   running sum reaches U times the total, U one uniform variate per position and step from a
   counter-based generator keyed by sample_seed.  The scratch holds the per-lane sums of every partial
   result of a row; the warp that delivers a row's last partial result locates the entry from them and
   re-reads the few dozen vectors of the row it can be in. */
size_t fork_sample_scratch_bytes(int32_t B, int32_t Lt);

/* One sampling step (Algorithm 2) for all B sequences.  Asynchronous on `stream`. */
fork_status fork_step(const fork_step_args* args, void* workspace, size_t workspace_bytes, void* stream);

/* Log-likelihood of given tokens at selected positions (Section 3.2).  Asynchronous on `stream`. */
fork_status fork_logprob(const fork_logprob_args* args, void* workspace, size_t workspace_bytes, void* stream);

/* The ForkGRPO objective and its derivative with respect to the new log-likelihoods.  Asynchronous. */
fork_status fork_grpo_loss(const fork_grpo_args* args, void* stream);

/* Log-softmax backward at the selected rows.  Asynchronous; uses the workspace like fork_logprob. */
fork_status fork_logprob_backward(const fork_logprob_bwd_args* args, void* workspace, size_t workspace_bytes, void* stream);

/* Scoring, Eq. 2 and the backward in one pass over the logits.  Asynchronous; uses the workspace like fork_logprob. */
fork_status fork_grpo_fused(const fork_grpo_fused_args* args, void* workspace, size_t workspace_bytes, void* stream);

/*
 * The step with the vocabulary sharded over N ranks (a vocabulary-parallel LM head): rank j holds
 * logits [B, Ll, V_j], the entries [offset_j, offset_j + V_j) of every row, offsets ascending with
 * the rank.  tokens / mask / block bounds are replicated.  The paper runs on one GPU and has no
 * counterpart; the merge is the associative one the single-GPU kernels already use between CTAs.
 *
 *   1. fork_vp_reduce on every rank: args as for fork_step with logits = the slice and V = V_j; nothing
 *      is committed.  For every live position it writes part_out[b,k] = (m, s, t2, index) as four
 *      32-bit words (float, float, float, int32: slice maximum, sum 2^((x-m) log2 e), sum of
 *      (x-m) log2 e * 2^(...), GLOBAL index of the lowest arg-max; s = NaN if the slice holds NaN or
 *      +inf; m = -inf, s = t2 = 0 if it holds nothing but -inf), and with temperature > 0 also
 *      key_out[b,k] = (sum of the slice's tempered weights against its own maximum, global index of
 *      the entry the slice would contribute, its logit, 0).  The draw is two-stage: every rank draws
 *      inside its slice with one uniform variate (the same on all ranks), the select phase picks
 *      the slice, with probability proportional to its tempered total, with a second one; the
 *      result is a sample of softmax(x / tau) over the whole vocabulary, and which sample depends
 *      on how the vocabulary is cut.
 *      part_out / key_out: device, [B,Lt] x 16 bytes, 16-byte aligned; other positions untouched.
 *   2. the caller gathers the N buffers (e.g. one all-gather) into [N][B,Lt] in rank order.
 *   3. fork_vp_select on every rank: merges the N parts of each live row in rank order, derives
 *      confidence, candidate, entropy, log-probability, and applies the unmask rule exactly as
 *      fork_step does (all of its outputs, all fallback orders).  args->logits is not read; Ll and
 *      pos0 must be those given to fork_vp_reduce (Ll = 0 means the whole sequence).
 */
fork_status fork_vp_reduce(const fork_step_args* args, int32_t vocab_offset, void* part_out, void* key_out,
                           void* workspace, size_t workspace_bytes, void* stream);
fork_status fork_vp_select(const fork_step_args* args, const void* parts, const void* keys, int32_t n_ranks,
                           void* workspace, size_t workspace_bytes, void* stream);

/*
 * Steps 1 and 2 in one kernel: fork_vp_reduce with the exchange fused in.  Instead of filling one
 * local [B,Lt] buffer for the caller to all-gather, the kernel stores each live position's 16 bytes,
 * as soon as the slice's reduction of that sequence is complete, straight into the gather buffer of
 * EVERY rank at [rank][b,k] -- plain 16-byte stores, the remote ones travelling over NVLink while
 * the rest of the slice is still being reduced.  Nothing is ever loaded from another GPU's memory.
 *   - peer_parts: HOST array of n_ranks device addresses, valid on THIS GPU: entry j is rank j's
 *     gather buffer [n_ranks][B,Lt] x 16 bytes (this GPU's own buffer for j == rank; for the others
 *     memory of GPU j mapped here: CUDA IPC, cuMem with peer access, or symmetric memory), 16-byte
 *     aligned.  peer_keys: the same for the perturbed keys, needed when temperature > 0, else NULL.
 *     n_ranks <= FORK_VP_MAX_RANKS.  The arrays are read during the call only.
 *   - Ordering is the caller's: fork_vp_select on any rank must not start before the kernels of
 *     this call have COMPLETED on all ranks (e.g. synchronise the stream, then a barrier among the
 *     ranks; or a stream-ordered collective on one word).  Positions that are not live are not
 *     written: fork_vp_select reads live positions only.
 */
#define FORK_VP_MAX_RANKS 16
fork_status fork_vp_reduce_peers(const fork_step_args* args, int32_t vocab_offset, int32_t rank, int32_t n_ranks,
                                 void* const* peer_parts, void* const* peer_keys,
                                 void* workspace, size_t workspace_bytes, void* stream);

/*
 * The step fused into the LM-head product (the paper's model "predicts a distribution
 * q_theta^k(.|x_t) for every k in M_t", Section 2: the logits of a step are hidden states times the
 * output embedding).  Instead of reading logits from memory, this entry point takes the hidden
 * states of the logits window and the LM-head weight, forms logits = hidden x weight^T tile by tile
 * on the tensor cores (bf16 inputs, fp32 accumulation) and reduces every tile to the step's per-row
 * statistics while it is still in tensor memory; the logits are never written anywhere.  Then the
 * unmask rule runs exactly as in fork_step (all outputs, all fallback orders).
 *   - hidden: device, bf16, [B * Ll, d]: row b * Ll + (k - pos0) is the final hidden state of position
 *     k of sequence b (every position of the window, masked or not), rows hidden_stride elements apart.
 *   - weight: device, bf16, [V, d], rows weight_stride elements apart: logit v = <hidden row, weight row v>.
 *   - d a multiple of 64; both base addresses 16-byte aligned and both strides multiples of 8 elements.
 *   - args->logits, stride_b, stride_l and dtype are ignored.
 *   - temperature > 0 draws the candidates (Algorithm 2 line 4) in two stages, with the two uniforms of the
 *     row that fork_step uses: the vocabulary is cut into chunks of 32 consecutive entries; the chunk is
 *     drawn with probability proportional to its tempered weight (by inversion, chunks ascending), and the
 *     token inside it by inversion in index order -- i.e. the draw fork_step_vocab_parallel makes with one
 *     slice per chunk.  args->sample_scratch must then hold fork_head_sample_scratch_bytes(B, Ll, V) bytes
 *     (device, 256-byte aligned; it needs no initialisation).
 *   - The logits are the fp32-accumulated products themselves (not rounded to bf16 on the way), so
 *     results agree with fork_step on materialised bf16 logits only up to that rounding.  A row whose
 *     logits hold NaN or an infinity is flagged FORK_ROW_NONFINITE.
 *   - row_pos0 (optional): the window of every sequence starts at its own position, row b * Ll + l is
 *     position row_pos0[b] + l of sequence b (args->pos0 is then ignored).  This is how a caller whose
 *     sequences sit in different blocks hands over just each sequence's active block.
 * Asynchronous on `stream`; four kernels (active set, product + reduction, merge of the column
 * splits, unmask rule).
 */
typedef struct fork_head_args {
  const void* hidden;        /* [B*Ll, d] bf16 */
  int64_t hidden_stride;     /* elements between rows, >= d */
  const void* weight;        /* [V, d] bf16 */
  int64_t weight_stride;     /* elements between rows, >= d */
  int32_t d;                 /* hidden size */
  const int32_t* row_pos0;   /* device [B], optional: first position of each sequence's window */
} fork_head_args;
fork_status fork_step_fused_head(const fork_step_args* args, const fork_head_args* head, void* workspace,
                                 size_t workspace_bytes, void* stream);
size_t fork_head_sample_scratch_bytes(int32_t B, int32_t Ll, int32_t V);

/*
 * fork_step without a workspace argument, for callers that have no device memory to give and
 * cannot allocate any.  (The paper has no counterpart of this entry point; it exists for
 * deployment.)  Typical callers: an inference server whose memory pool already owns the whole
 * device, so that a cudaMalloc made on its behalf would fail or fragment the pool; and code on a
 * latency-critical path, where the implicit device synchronisation of cudaMalloc / cudaFree is not
 * acceptable.  This call allocates nothing and frees nothing, neither with the CUDA runtime nor
 * through any library: the scratch is a fixed array of FORK_STATIC_SCRATCH_BYTES inside the library's
 * device image (every GPU that loads the library holds that much until the process exits).
 *
 *   - Same arguments, results and asynchrony as fork_step.
 *   - Batches whose scratch need, fork_workspace_bytes(B, Lt), exceeds FORK_STATIC_SCRATCH_BYTES are
 *     rejected with FORK_ERR_WORKSPACE before anything is launched (B*Lt up to about 30,000
 *     positions fits).
 *   - The first call on each device looks up the array's device address (one cudaGetSymbolAddress,
 *     with that device current) and caches it; make that first call outside any stream capture.
 *   - All calls on a device share the one array (and one control block reserved for it), which
 *     simply keep what the previous call left: a step reads nothing there that it has not written
 *     itself, and leaves the counters of the control block as it found them, so back-to-back calls
 *     on one stream are fine, but two calls that can overlap on the GPU (different streams, or
 *     different threads without ordering) race on it.
 *   - fork_device_status(NULL, ...) reads the device status word of the last call.
 */
#define FORK_STATIC_SCRATCH_BYTES (2u * 1024u * 1024u)
fork_status fork_step_static(const fork_step_args* args, void* stream);

/*
 * Model-forward callback of the decode loop: must enqueue on `stream` the work that fills
 * `logits_out` (the buffer given as proto->logits) for the live positions of step `step`,
 * given the current device-side tokens / mask / block cursors.  Returns 0 on success.
 * One call = one model evaluation (NFE, Section 4.1).
 */
typedef int (*fork_logits_fn)(void* ctx, int32_t step, const int32_t* tokens, const uint8_t* mask,
                              const int32_t* blk_lo, const int32_t* blk_hi, void* logits_out, void* stream);

/*
 * Semi-autoregressive decoding (Section 2: repeat sampling steps until nothing is masked;
 * Section 4.1: blocks of block_len inside the generation window [gen_lo,gen_hi)).
 * Every sequence keeps its own block cursor: the first block that still holds a masked
 * position.  Each iteration calls provider once and runs fork_step on every unfinished sequence's
 * block (step ids proto->step, proto->step+1, ...); the step itself moves the cursors on (the
 * finaliser of a sequence whose block is complete looks for the next block that holds a masked
 * position) and its last finaliser reports how many sequences are unfinished in eight bytes of
 * pinned host memory, which the host polls: no kernel besides the step's own, no stream
 * synchronisation.  (The first call in a process allocates 2 KB of pinned host memory for these
 * reports; up to 32 loops may run at the same time.)
 * By default the host waits for the report of a step before it calls the provider for the next
 * one.  With FORK_TUNE_LOOP_AHEAD = d > 0 it runs up to d steps ahead of the reports, so the GPU
 * never waits for the host; the price is up to d provider calls (and steps, which then find nothing
 * to do: they change neither sequences nor records nor evaluation counts, only n_unmasked /
 * is_fallback / fallback_pos, which describe the last step enqueued, an empty one) after the batch
 * is in fact complete.
 * proto->blk_lo / blk_hi are ignored.  *steps_taken (host) receives the number of steps after
 * which nothing was masked (= provider calls when d = 0).  Returns FORK_ERR_MAX_STEPS if masked
 * positions remain after max_steps steps, and FORK_ERR_PROVIDER if the callback fails; device state
 * then reflects the steps completed and *steps_taken the steps enqueued.
 */
fork_status fork_decode_loop(const fork_step_args* proto, int32_t block_len, int32_t gen_lo, int32_t gen_hi,
                             fork_logits_fn provider, void* ctx, int32_t max_steps, int32_t* steps_taken,
                             void* workspace, size_t workspace_bytes, void* stream);

/*
 * fork_decode_loop on hidden states: every step, `provider` fills head->hidden with the final hidden
 * states of each sequence's ACTIVE BLOCK -- row b * Ll + l is position blk_lo[b] + l of sequence b,
 * where blk_lo is the cursor array the provider is called with (Ll = proto->Ll >= block_len) -- and
 * the step is fork_step_fused_head on them; the logits are never stored.  Everything else (cursors
 * advanced on the device, outcomes read from pinned host memory, FORK_TUNE_LOOP_AHEAD, steps_taken,
 * the error codes) is as for fork_decode_loop.  head->row_pos0 is ignored (the loop supplies its
 * cursors); proto->pos0, logits, strides and dtype are ignored.
 */
fork_status fork_decode_loop_fused_head(const fork_step_args* proto, const fork_head_args* head, int32_t block_len,
                                        int32_t gen_lo, int32_t gen_hi, fork_logits_fn provider, void* ctx,
                                        int32_t max_steps, int32_t* steps_taken, void* workspace,
                                        size_t workspace_bytes, void* stream);

/*
 * fork_step for callers whose buffers live in HOST memory (pinned memory recommended): every
 * pointer in `host_args` is a host pointer.  The call copies the logits window, tokens, mask
 * and block bounds into `staging` (device, at least fork_staging_bytes(host_args) bytes), runs
 * fork_step, copies every non-NULL output back and synchronises `stream` before returning.
 */
size_t fork_staging_bytes(const fork_step_args* host_args);
fork_status fork_step_host(const fork_step_args* host_args, void* staging, size_t staging_bytes,
                           void* workspace, size_t workspace_bytes, void* stream);

/*
 * Position selection of JustGRPO-Fast (Section 3.2, last paragraph; Section 4.2 Setup): of the
 * eligible positions of each rollout, mark the fraction `ratio` with the highest token entropy, as
 * the `select` input of fork_logprob.  The count is floor(ratio * n), n = eligible positions of the
 * rollout, and at least 1 when n > 0 and ratio > 0; equal entropies go to the lower position; NaN
 * entropies rank last.  All pointers are device memory: entropy [B,Lt] (e.g. the `entropy` output of
 * the decode loop), eligible [B,Lt] (non-zero = may be selected), select [B,Lt] out (0/1 at every
 * position), n_selected [B] out, optional.  0 <= ratio <= 1, Lt <= 32768.  Asynchronous on `stream`.
 */
fork_status fork_select_top_entropy(const float* entropy, const uint8_t* eligible, int32_t B, int32_t Lt,
                                    float ratio, uint8_t* select, int32_t* n_selected, void* stream);

/* Benchmark aid: reads `bytes` of device memory once with the kernels' own streaming loads and does
   nothing else (buffer 16-byte aligned; sink4 = 4 bytes of device memory).  Its rate is the
   read-only ceiling that bench.py reports beside the measured copy rate.  Asynchronous. */
fork_status fork_read_probe(const void* buffer, size_t bytes, void* sink4, void* stream);

/* One-kernel steps keep a small control block inside the library for every workspace address they
   have seen on the current device (see "Conventions").  Call this when a workspace is done with --
   every call that used it has completed, and no CUDA graph that captured such a call will be
   launched again -- to give its block back; addresses that are never released simply keep theirs.
   Releasing an address the library has not seen is not an error. */
fork_status fork_workspace_release(const void* workspace);

/* Copies the device status word of the last call that used `workspace` to *host_out
   (FORK_DEV_* bits) and synchronises `stream`.  workspace = NULL asks about the scratch inside the
   library, i.e. about the last fork_step_static call on the current device (and, like for any
   workspace, a reported FORK_DEV_TIMEOUT puts the control block reserved for it back to its
   initial state). */
fork_status fork_device_status(const void* workspace, uint32_t* host_out, void* stream);

/* Human-readable name of a status code. */
const char* fork_status_string(int status);

/*
 * Tuning knobs (process wide; intended for benchmarking).  Keys:
 *   FORK_TUNE_VARIANT       0 = automatic, 1 = direct vector loads, 2 = bulk-copy shared-memory ring
 *   FORK_TUNE_CTAS_PER_SM   0 = automatic, else resident CTAs per SM used to size the grid of variant 1
 *                           (variant 2 always runs two per SM)
 *   FORK_TUNE_PDL           0 = launch the kernels of a step with programmatic dependent launch (each
 *                           waits on-device for its predecessor before touching memory), -1 = plain launches
 *   FORK_TUNE_STAGES        0 = automatic, else shared-memory stages (16 KB each) per CTA of variant 2
 *   FORK_TUNE_ONE_KERNEL    0 = a step of at most 256 sequences whose logits cover at most 2048 positions
 *                           per sequence and 32768 over all sequences runs as ONE kernel on variant 2
 *                           (every CTA derives the active set itself), -1 = always the set-up kernel first
 *   FORK_TUNE_LATE_CTA      testing only: g + 1 makes virtual CTA g of a one-kernel step start about
 *                           0.1 ms late (exercises the hand-over of mask updates), 0 = off.  A non-zero
 *                           value selects an instance of the kernel compiled with that hook; the
 *                           instances that run otherwise do not contain it.
 *   FORK_TUNE_L2_EVICT_FIRST 0 = the bulk copies of logits carry the L2 "evict first" hint (a row is read
 *                           once; what a step re-reads stays cached), -1 = no hint
 *   FORK_TUNE_LOOP_AHEAD    fork_decode_loop: how many steps the host may enqueue beyond the last step whose
 *                           outcome it has read (0..6, default 0); see fork_decode_loop
 *   FORK_TUNE_MIN_UNITS     0 = automatic (8), else how many units of 2048 logits a participating CTA gets at
 *                           least, on average: a step with few live rows then runs on fewer CTAs, which
 *                           leaves fewer partial results to hand over and merge
 * Returns the previous value, or -1 for an unknown key.
 */
enum { FORK_TUNE_VARIANT = 0, FORK_TUNE_CTAS_PER_SM = 1, FORK_TUNE_PDL = 2, FORK_TUNE_STAGES = 3,
       FORK_TUNE_ONE_KERNEL = 4, FORK_TUNE_LATE_CTA = 5, FORK_TUNE_L2_EVICT_FIRST = 6, FORK_TUNE_MIN_UNITS = 7,
       FORK_TUNE_LOOP_AHEAD = 8, FORK_TUNE_COUNT_ = 9 };
int32_t fork_set_tuning(int32_t key, int32_t value);

/* Profiling hook: the next fork_step / fork_logprob call made by this host thread records the two
   CUDA events (cudaEvent_t passed as void*) on its stream immediately before and after its
   streaming kernel (not around the active-set kernel), then forgets them. */
void fork_set_timing_events(void* start, void* stop);

/* Number of kernels this library has launched since it was loaded (all entry points). */
int64_t fork_kernel_launches(void);

/* One-kernel steps: how many times, since the library was loaded on the current device, a sequence's
   mask update was handed on because a CTA of the launch had not yet read the mask (see
   FORK_TUNE_LATE_CTA).  Synchronises the device; -1 on a CUDA error.  For tests. */
int64_t fork_mask_handovers(void);

/* For tests: the host-side arithmetic of the work partition as the kernels use it (the paper has no
   counterpart).  A step's live rows are cut into units of fork_debug_chunk() logits, numbered row by
   row (C units per row, U in all); fork_debug_effective_grid gives how many of G CTAs take part when
   every one of them should get at least min_units units; CTA g of those owns the units from
   fork_debug_part_begin(U, G, g) up to fork_debug_part_begin(U, G, g + 1); fork_debug_part_owner is the
   CTA that owns unit x, fork_debug_row_parts the number of CTAs that share row r.  Pure functions of
   their arguments; no GPU is touched. */
int64_t fork_debug_part_begin(int64_t U, int32_t G, int32_t g);
int32_t fork_debug_part_owner(int64_t U, int32_t G, int64_t x);
int32_t fork_debug_row_parts(int64_t U, int32_t G, int32_t C, int64_t r);
int32_t fork_debug_chunk(void);
int32_t fork_debug_effective_grid(int64_t U, int32_t G, int32_t min_units);

#ifdef __cplusplus
}
#endif
#endif /* FORK_DLLM_H */
