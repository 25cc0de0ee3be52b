/*
 * nat.h - C ABI of the partial-token GRPO policy-gradient step (NAT, "Not All
 * Tokens are Needed") for NVIDIA B200 (sm_100a).
 *
 * Notation (the paper's): P prompts, G responses per prompt, B = P*G
 * responses; response i has length T_i and belongs to prompt i / G; the
 * responses are packed back to back, cu_seqlens[i] is the index of the first
 * token of response i and cu_seqlens[B] = N_tot.  Token n of the packed
 * stream sits at 1-based position t = n - cu_seqlens[resp(n)] + 1.
 * m is the selection mask, pi the inclusion probability, L_i the RPC cut,
 * A_i the group-relative advantage, d the hidden size, V the vocabulary.
 *
 * Conventions for every entry point
 *   - Pointers are DEVICE pointers owned by the caller unless the comment says
 *     "host".  Nothing is retained after the call returns.
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).
 *     Calls enqueue work on it and return without synchronising.
 *   - The library allocates no device memory: kernels that need scratch take
 *     a caller-provided `workspace` whose size the matching *_workspace_bytes
 *     function returns.  The workspace must be 256-byte aligned.
 *   - Return value: NAT_OK, or a negative nat_status.  Arguments are validated
 *     (and the tensor maps of the bf16 path encoded) before the first
 *     enqueue, so NAT_ERR_INVALID_ARG, NAT_ERR_UNSUPPORTED and NAT_ERR_CAPACITY
 *     mean that nothing was enqueued; NAT_ERR_CUDA (a launch or memset refused
 *     by the runtime) may leave earlier work of the same call on the stream.
 *     nat_last_error() gives a thread-local message.
 *   - Device-side conditions that cannot be known at launch (a bounded wait
 *     that ran out, n_sel above the stated capacity, a target outside the
 *     vocabulary) are recorded in the 32-bit status word at the start of the
 *     loss workspace (see NAT_DEV_* bits, nat_poll_status); kernels never trap.
 *   - Alignment: mask, pi, surv and q arrays, the compacted lists and every
 *     matrix must start on a 16-byte boundary (the kernels use 16-byte
 *     accesses); a misaligned pointer is refused with NAT_ERR_INVALID_ARG.
 */
#ifndef NAT_H_
#define NAT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  NAT_OK = 0,
  NAT_ERR_INVALID_ARG = -1, /* null pointer, negative size, p outside (0,1], ... */
  NAT_ERR_UNSUPPORTED = -2, /* dtype/shape the kernels do not cover, wrong GPU architecture */
  NAT_ERR_CAPACITY = -3,    /* workspace or output capacity too small */
  NAT_ERR_CUDA = -4         /* a CUDA runtime/driver call failed; see nat_last_error() */
} nat_status;

/* Bits of the device status word (first 4 bytes of a loss workspace). */
#define NAT_DEV_TIMEOUT 1u  /* a bounded mbarrier wait gave up; outputs are invalid */
#define NAT_DEV_CAPACITY 2u /* *n_sel exceeded n_sel_cap; surplus rows were ignored */
#define NAT_DEV_FALLBACK 4u /* informational: nat_policy_loss_fwd_bwd redid some row chunk with
                               the two-pass kernels (results are valid) */
#define NAT_DEV_BAD_TARGET 8u /* some selected token's target lies outside [0, V): that token
                                 was left out (zero loss term and gradient, logp = NaN) */

const char* nat_status_string(int status);
const char* nat_last_error(void); /* host string, valid until the thread's next failing call */
int nat_version(void);

/* Copies the device status word at the head of a loss workspace to *host_word (host
 * pointer) and waits for `stream`, i.e. for the loss calls enqueued on it so far.  (A
 * convenience of this library; the paper has no counterpart.)  The word is the OR of the
 * NAT_DEV_* bits raised by the last loss call that used the workspace. */
int nat_poll_status(const void* workspace, void* stream, uint32_t* host_word);

/* ---------------------------------------------------------------------------
 * Group-relative advantage (Eq. grpo-adv, Section 2.2):
 *   A_i = (R_i - mu) / (sigma + eps), mu and sigma the population mean and
 *   standard deviation (1/G) of the G rewards of response i's prompt.
 * rewards, adv: float32 [P*G].  Arithmetic is double in index order and the
 * result is rounded once to float32, so it is reproducible bit for bit.
 * A group with equal rewards gets A = 0.
 * ------------------------------------------------------------------------- */
int nat_grpo_adv(int32_t P, int32_t G, const float* rewards, float eps, float* adv, void* stream);

/* ---------------------------------------------------------------------------
 * Token selection (Section 3.1 "Random masking", URS; Section 4 RPC with the
 * uniform and minimum-cutoff laws; deterministic truncation as the biased
 * comparison).  Random draws are Philox4x32-10 outputs, a pure function of
 * (seed, offset, response index, position); below i stands for resp_base + the
 * response's index in cu_seqlens:
 *   key     = (seed_lo, seed_hi ^ offset_hi)
 *   URS     token t uses word (t-1)%4 of counter ((t-1)/4, i, 0, offset_lo);
 *           m = [x < thr], thr = clamp(floor(p 2^32), 1, 2^32), pi = thr/2^32.
 *   RPC     response i draws counter (0, i, 1, offset_lo), u = x1 2^32 + x0,
 *           C_i = min(max(min_cut,1), T_i), n = T_i - C_i + 1,
 *           L_i = C_i + floor(u n / 2^64); m_t = [t <= L_i];
 *           pi_t = 1 (t <= C_i), (T_i-t+1)/(T_i-C_i+1) otherwise (one float32
 *           division, Eq. rpc-survival under the uniform law).
 *   DET     K_i = max(1, floor(beta T_i)); m_t = [t <= K_i]; pi_t = 1.
 * Outputs: mask uint8 [n_tot] (0/1), pi float32 [n_tot], cut_len int32 [B]
 * (L_i or K_i, 0 for an empty response; may be NULL for URS, which leaves it
 * untouched).  cu_seqlens int32 [B+1] on the device; n_tot is the host's copy
 * of cu_seqlens[B].  T_i = 0 is allowed.
 * resp_base: index, in the whole job's batch, of the first response of cu_seqlens.  A
 * data-parallel rank that holds responses [lo, hi) of the batch passes its own cu_seqlens
 * and resp_base = lo and realises exactly the masks the whole batch would (masks of
 * different responses are independent, Section 3.1); 0 for an unsharded batch.
 * Errors: NAT_ERR_INVALID_ARG for p outside (0,1], beta outside (0,1],
 * min_cut < 0, B < 0, n_tot < 0, resp_base < 0, null or misaligned pointers.
 * ------------------------------------------------------------------------- */
typedef enum { NAT_SEL_URS = 0, NAT_SEL_RPC = 1, NAT_SEL_DET = 2 } nat_sel_mode;

typedef struct {
  int32_t mode;    /* nat_sel_mode */
  int32_t min_cut; /* RPC: C (0 and 1 both mean the plain uniform cutoff) */
  double p;        /* URS: inclusion probability in (0,1] */
  double beta;     /* DET: kept fraction in (0,1] */
  uint64_t seed;
  uint64_t offset; /* caller's step counter: a new offset gives fresh draws */
  int32_t resp_base; /* global index of the first response (0 unless the batch is a shard) */
  int32_t reserved;  /* set to 0 */
} nat_select_params;

int nat_select(const nat_select_params* params /* host */, int32_t B, const int32_t* cu_seqlens,
               int64_t n_tot, uint8_t* mask, float* pi, int32_t* cut_len, void* stream);

/* ---------------------------------------------------------------------------
 * Random Prefix Cutting under a caller-given survival schedule (Section 4:
 * Eq. rpc-mask and Eq. rpc-survival for a general cut law q_i; Appendix B.3
 * discusses schedules other than the uniform one).
 *   surv float32 [n_tot]: p_{i,t} = Pr(L_i >= t) for every packed token; inside a
 *   response it must start at 1, never increase and stay positive (not checked).
 * Response i draws u = (x0 >> 8) 2^-24 from the Philox block with counter
 * (0, resp_base + i, 2, offset_lo), key as in nat_select; m_t = [u < surv], a prefix of
 * length L_i because surv is monotone, and Pr(L_i >= t) = ceil(surv 2^24) / 2^24.
 * Outputs: mask uint8 [n_tot], cut_len int32 [B] (L_i; 0 for an empty response).
 * The inclusion probabilities are the schedule: pass `surv` as `pi` to the loss.
 * surv and mask must be 16-byte aligned.
 * ------------------------------------------------------------------------- */
int nat_select_survival(int32_t B, const int32_t* cu_seqlens, int64_t n_tot, const float* surv,
                        uint64_t seed, uint64_t offset, int32_t resp_base, uint8_t* mask,
                        int32_t* cut_len, void* stream);

/* ---------------------------------------------------------------------------
 * Random Prefix Cutting under a caller-given cut law (Section 4: Eq. rpc-mask; the
 * survival function is the suffix sum of the law, Eq. rpc-survival; Appendix B.3 on laws
 * other than the uniform one).
 *   q float32 [n_tot]: the mass q_i(l) the law of token n's response puts on cutting right
 *   after that token, up to a common positive factor per response.  Masses enter in
 *   32-bit fixed point, k = min(floor(q 2^32), 2^32 - 1) for q > 0 and 0 otherwise, so that
 *   every sum below is an exact 64-bit integer, independent of the order of summation:
 *     S_t  = sum_{l >= t} k_l       (a scan over the packed stream on the device)
 *     u    = x1 2^32 + x0 of the Philox block with counter (0, resp_base + i, 3, offset_lo),
 *     r    = floor(u S_1 / 2^64),  m_t = [S_t > r]:  L_i = max{t : S_t > r},
 *            Pr(L_i >= t) = S_t / S_1 to within S_1 2^-64
 *     pi_t = float32(double(S_t) * (1 / double(S_1))), every operation rounded to nearest:
 *            pi_1 = 1 and pi never increases, by construction; pi_t > 0 wherever the law
 *            still has mass at or after t.
 *   A response whose masses are all zero is kept whole with pi = 1.  Tokens after the
 *   last positive mass get pi = 0 and are never selected.
 * Outputs: mask uint8 [n_tot], pi float32 [n_tot], cut_len int32 [B].
 * workspace: nat_select_cutlaw_workspace_bytes(B, n_tot) bytes, 256-byte aligned.
 * ------------------------------------------------------------------------- */
size_t nat_select_cutlaw_workspace_bytes(int32_t B, int64_t n_tot);
int nat_select_cutlaw(int32_t B, const int32_t* cu_seqlens, int64_t n_tot, const float* q,
                      uint64_t seed, uint64_t offset, int32_t resp_base, uint8_t* mask, float* pi,
                      int32_t* cut_len, void* workspace, size_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------------------
 * Compaction of the selected tokens (Section 1: tokens that were not selected take no
 * part in the backward pass; Eq. ht-estimator sums over m = 1 only).
 *   sel_idx  int32 [cap]   ascending packed indices n with mask[n] != 0
 *   sel_resp int32 [cap]   resp(sel_idx[k])
 *   sel_offsets int32 [B+1] number of selected tokens in responses < i
 *   n_sel    int32 device scalar = sel_offsets[B]
 * cap is the number of elements the two lists can hold; if more tokens are
 * selected the surplus is not written and *n_sel still reports the true count.
 * workspace: nat_compact_workspace_bytes(n_tot) bytes.
 * ------------------------------------------------------------------------- */
size_t nat_compact_workspace_bytes(int64_t n_tot);
int nat_compact(int32_t B, const int32_t* cu_seqlens, int64_t n_tot, const uint8_t* mask,
                int32_t* sel_idx, int32_t* sel_resp, int32_t* sel_offsets, int32_t* n_sel,
                int64_t cap, void* workspace, size_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------------------
 * Compaction under a prefix mask (Eq. rpc-mask: m_t = 1[t <= L_i]; also the deterministic
 * truncation).  The selected tokens of response i are the packed indices
 * [cu_seqlens[i], cu_seqlens[i] + L_i), so the lists follow from cut_len alone: the mask
 * is not read and nothing but the lists is written (8 bytes per selected token).
 *   cut_len int32 [B]: L_i as written by nat_select (RPC, DET), nat_select_survival or
 *   nat_select_cutlaw; values are clamped to [0, T_i].
 * Outputs and capacity rule as for nat_compact; the results are identical to
 * nat_compact on the corresponding mask.  n_tot (host copy of cu_seqlens[B]) bounds the
 * launch.  No workspace.
 * ------------------------------------------------------------------------- */
int nat_compact_prefix(int32_t B, const int32_t* cu_seqlens, int64_t n_tot,
                       const int32_t* cut_len, int32_t* sel_idx, int32_t* sel_resp,
                       int32_t* sel_offsets, int32_t* n_sel, int64_t cap, void* stream);

/* ---------------------------------------------------------------------------
 * Packing for prefix-truncated computation (Section 4, the paragraph on compute
 * savings: under RPC the model only has to process the prefix 1..L_i of each
 * response, forward as well as backward).
 *   nat_gather_rows   dst[k, :] = src[sel_idx[k], :]  for k < min(*n_sel, cap)
 *   nat_scatter_rows  dst = 0 over [n_tot, row_bytes], then
 *                     dst[sel_idx[k], :] = src[k, :]   (e.g. compact dHidden back
 *                     to the packed stream; unselected tokens get zero gradient)
 * Rows are row_bytes bytes (a positive multiple of 16) of any element type;
 * src and dst are 16-byte aligned and must not overlap.  After nat_compact under
 * RPC or truncation, sel_offsets is the cu_seqlens of the packed prefixes.
 * ------------------------------------------------------------------------- */
int nat_gather_rows(const void* src, int64_t row_bytes, const int32_t* sel_idx,
                    const int32_t* n_sel, int64_t cap, void* dst, void* stream);
int nat_scatter_rows(const void* src, int64_t row_bytes, const int32_t* sel_idx,
                     const int32_t* n_sel, int64_t cap, int64_t n_tot, void* dst, void* stream);

/* ---------------------------------------------------------------------------
 * nat_compact_static: nat_compact without a workspace argument.  (An addition
 * of this library; the paper has no counterpart.)
 *
 * For callers that cannot obtain device memory at the point of the call: code
 * running under a framework that has reserved the whole GPU for its own pool,
 * plugin or callback contexts where cudaMalloc is forbidden or would
 * synchronise the device, and tight inner loops that must not touch an
 * allocator.  The scan scratch lives in a fixed array inside the library
 * (64 KB of device memory per GPU that loads the library, held until the
 * process exits), so the call allocates and frees nothing.
 *
 * Arguments, outputs and results are those of nat_compact.  Differences:
 *   - n_tot may not exceed nat_compact_static_max_tokens() (67,108,864 tokens);
 *     larger inputs return NAT_ERR_CAPACITY and enqueue nothing.
 *   - The first call on each device looks up the array's device address (a
 *     runtime query, not an allocation).  Make that first call outside any
 *     stream capture.
 *   - All calls on one GPU share the one array.  Calls whose kernels could run
 *     at the same time (different streams without ordering) race on it and
 *     give wrong results; order them on one stream or with events.  Nothing in
 *     the array needs clearing between calls: each call overwrites what it
 *     reads.
 * ------------------------------------------------------------------------- */
int64_t nat_compact_static_max_tokens(void);
int nat_compact_static(int32_t B, const int32_t* cu_seqlens, int64_t n_tot, const uint8_t* mask,
                       int32_t* sel_idx, int32_t* sel_resp, int32_t* sel_offsets, int32_t* n_sel,
                       int64_t cap, void* stream);

/* ---------------------------------------------------------------------------
 * Policy loss over the selected tokens (ratio Eq. ratio, clipped surrogate
 * Eq. grpo-surrogate, sequence/group mean Eq. grpo-obj, Horvitz-Thompson
 * weights Eq. ht-estimator and Eq. rpc-ht; KL coefficient 0 as in the paper's
 * experiments).  For selected token k (packed index n = sel_idx[k],
 * response i = sel_resp[k], hidden row h):
 *   z = W h (V logits, fp32 accumulation), lse = log sum_v exp z_v,
 *   logp = z[targets[n]] - lse,  r = exp(logp - old_logp[n]),
 *   S = min(r A_i, clip(r, 1-clip_lo, 1+clip_hi) A_i),
 *   L = S - kl_beta (logp - ref_logp[n])   (Eq. grpo-token-loss; the per-token KL in the
 *       sampled-token form of the paper's footnote; kl_beta = 0 by default),
 *   w = 1 / (pi[n] T_i B),   loss = - sum_k w L.
 * The logits are never written to memory.
 *
 * dtype NAT_BF16: hidden, W, dHidden are bfloat16 and the projection runs on
 * the tensor cores; requires d % 64 == 0.  dtype NAT_F32: float32 operands,
 * plain fp32 arithmetic, any V and d <= 1024 (meant for small problems; a larger d is
 * refused with NAT_ERR_UNSUPPORTED and has workspace size 0).
 * hidden is [n_tot, d] row-major (row sel_idx[k] is used) or, with
 * hidden_is_compact, [>= n_sel, d] with row k belonging to sel_idx[k].
 * W is [V, d] row-major.  targets int32 [n_tot] in [0, V); old_logp, pi
 * float32 [n_tot]; adv float32 [number of responses in cu_seqlens].  params->B is the
 * divisor of the batch mean: the number of responses of the WHOLE job's batch, which
 * exceeds the number of responses passed here when the batch is sharded over
 * data-parallel ranks (the ranks' losses and dW then add up to the job's).
 * A target outside [0, V) raises NAT_DEV_BAD_TARGET and its token is left out.
 * n_sel is the device scalar written by
 * nat_compact; n_sel_cap is a host upper bound on it (grid and workspace are
 * sized from it; rows beyond it are ignored and NAT_DEV_CAPACITY is raised).
 * Outputs: loss float32 device scalar; logp, lse float32 [n_sel_cap] (entries
 * k < n_sel are written).  The reduction order is fixed, so the loss is
 * reproducible run to run.
 * workspace: nat_policy_loss_workspace_bytes(params, n_sel_cap); it is shared
 * by forward and backward and holds nothing that must survive between them.
 * ------------------------------------------------------------------------- */
#define NAT_F32 0
#define NAT_BF16 1

typedef struct {
  int32_t d;
  int32_t V;
  int32_t dtype; /* NAT_F32 | NAT_BF16 */
  int32_t B;     /* number of responses of the whole batch (the batch mean's divisor) */
  float clip_lo; /* ratio is clipped to [1-clip_lo, 1+clip_hi] */
  float clip_hi;
  int32_t hidden_is_compact;
  int32_t accumulate_dW; /* backward: 0 overwrite dW, 1 add to it */
  float kl_beta;         /* coefficient of the KL term of Eq. grpo-token-loss; 0 (the paper's
                            experimental setting) leaves the term out */
  int32_t reserved;      /* set to 0 */
  const float* ref_logp; /* device float32 [n_tot]: log-probability of each token under the
                            reference policy; read only when kl_beta != 0 (else may be NULL) */
} nat_loss_params;

size_t nat_policy_loss_workspace_bytes(const nat_loss_params* params /* host */,
                                       int64_t n_sel_cap);

int nat_policy_loss_fwd(const nat_loss_params* params /* host */, const void* hidden,
                        const void* W, const int32_t* targets, const float* old_logp,
                        const float* adv, const float* pi, const int32_t* cu_seqlens,
                        const int32_t* sel_idx, const int32_t* sel_resp, const int32_t* n_sel,
                        int64_t n_sel_cap, float* loss, float* logp, float* lse,
                        void* workspace, size_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------------------
 * Backward of the loss above (the gradient of Eq. ht-estimator, Appendix A).
 * With g_k = -dloss w (A r 1[surrogate not saturated] - kl_beta) (saturated: A > 0 and
 * r > 1+clip_hi, or A < 0 and r < 1-clip_lo; A = 0 gives 0 for the first term):
 *   dz[k, v] = g_k (1[v = y_k] - exp(z_v - lse_k))      (z recomputed)
 *   dHidden[k, :] = sum_v dz[k, v] W[v, :]     compact: row k <-> sel_idx[k]
 *   dW[v, :]      = sum_k dz[k, v] h_k          float32 [V, d]
 * logp and lse are the forward's outputs.  dloss is a device float scalar
 * (NULL means 1).  dHidden has hidden's dtype, [n_sel_cap, d]; rows >= n_sel
 * are not written.  With accumulate_dW the product is added to dW's contents.
 * Every element of dHidden and dW is summed in a fixed order (tokens that share a target
 * are added to that row of dW in ascending order), so a call repeated on the same inputs
 * reproduces its outputs bit for bit.
 * ------------------------------------------------------------------------- */
int nat_policy_loss_bwd(const nat_loss_params* params /* host */, const void* hidden,
                        const void* W, const int32_t* targets, const float* old_logp,
                        const float* adv, const float* pi, const int32_t* cu_seqlens,
                        const int32_t* sel_idx, const int32_t* sel_resp, const int32_t* n_sel,
                        int64_t n_sel_cap, const float* logp, const float* lse,
                        const float* dloss, void* dHidden, float* dW, void* workspace,
                        size_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------------------
 * Forward and backward in one call (same definitions and outputs as
 * nat_policy_loss_fwd followed by nat_policy_loss_bwd: Eq. ratio,
 * Eq. grpo-surrogate, Eq. grpo-obj, Eq. ht-estimator / Eq. rpc-ht and their
 * gradient, Appendix A).  The bf16 path evaluates the projection S = H W^T once
 * per block of rows instead of twice: it keeps the softmax numerators
 * exp(S - mref) of at most 8192 rows in the workspace (mref = the row's largest
 * logit over the first 256 vocabulary entries), and the per-row factors
 * (1/sum, g) are applied outside the two gradient contractions.  If some logit
 * exceeds its row's mref by more than 60 the block is redone by the two-pass
 * kernels and NAT_DEV_FALLBACK is set; results are the same either way within
 * the rounding of bf16 staging.  Arguments as in the two separate calls;
 * outputs loss, logp, lse, dHidden, dW.
 * ------------------------------------------------------------------------- */
int nat_policy_loss_fwd_bwd(const nat_loss_params* params /* host */, const void* hidden,
                            const void* W, const int32_t* targets, const float* old_logp,
                            const float* adv, const float* pi, const int32_t* cu_seqlens,
                            const int32_t* sel_idx, const int32_t* sel_resp,
                            const int32_t* n_sel, int64_t n_sel_cap, const float* dloss,
                            float* loss, float* logp, float* lse, void* dHidden, float* dW,
                            void* workspace, size_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------------------
 * Per-kernel timing of the bf16 loss kernels (a measurement aid of this library;
 * the paper has no counterpart).  Between nat_trace_begin() and nat_trace_end()
 * every tensor-core kernel launch made by the loss entry points is bracketed by
 * a pair of CUDA events on the caller's stream.  nat_trace_end() waits for those
 * events (it synchronises with the work traced so far), adds up the elapsed
 * milliseconds and the launch counts per kernel kind into two HOST arrays of
 * NAT_TRACE_KINDS entries (either may be NULL), releases the events and stops
 * tracing.  Tracing creates CUDA events; leave it off in allocation-free code.
 * ------------------------------------------------------------------------- */
#define NAT_TRACE_KINDS 5
#define NAT_TRACE_FWD 0 /* S = H W^T with online log-sum-exp (forward; also the row references) */
#define NAT_TRACE_DZ 1  /* recomputed S -> softmax gradient (two-pass backward) */
#define NAT_TRACE_DH 2  /* dHidden contraction */
#define NAT_TRACE_DW 3  /* dW contraction */
#define NAT_TRACE_E 4   /* single-pass S -> softmax numerators */
int nat_trace_begin(void);
int nat_trace_end(float* ms_by_kind /* host */, int32_t* launches_by_kind /* host */);

#ifdef __cplusplus
}
#endif
#endif /* NAT_H_ */
