/*
 * hass.h - C ABI of the B200 (sm_100a) fused LM-head + Top-K distillation library.
 *
 * The library computes, for N rows of target features H_t and draft features H_d and the
 * frozen LM head W that both share, the Top-K distillation loss of HASS and its gradient
 * with respect to H_d. No N x V logit matrix is ever held in memory: logits exist tile by tile in
 * tensor memory. What does pass through the workspace, between the forward sweep and the
 * back-projection of the fused call, is a bounded chunk of un-normalised bf16 draft probabilities
 * (chunk rows x V, chunk rows = 128 x a quarter of the SM count, 4736 on a 148-SM device whatever
 * N is: 1.2 GB for V = 128256); see hass_topk_distill_fwd_bwd.
 *
 * Notation follows the paper (Section 3.1): q = softmax(H_t W^T) is the target LLM's
 * next-token distribution, p = softmax(H_d W^T) the draft model's, Omega the vocabulary
 * (size V), Omega_hat the K tokens with the highest q.
 *
 * Common conventions
 *   - Every pointer is DEVICE memory owned by the caller unless a parameter says "host".
 *     The library allocates nothing, frees nothing and (except hass_check and the *_host
 *     entry) never synchronises: work is enqueued on `cuda_stream` (a cudaStream_t passed as
 *     void*; NULL = the default stream) and outputs are valid once the stream reaches that point.
 *   - Matrices are dense row-major: H_t, H_d [N, d], W [V, d], bf16 (raw 16-bit patterns).
 *     All pointers must be 16-byte aligned; d must be a multiple of 8 (a row is then a whole
 *     number of 16-byte units, which the TMA engine requires).
 *   - 1 <= K <= min(V, HASS_K_MAX). N >= 1 and V >= 1 are otherwise arbitrary; ragged row and
 *     vocabulary tiles are handled inside.
 *   - The return value is a hass_status. Argument errors are found on the host before anything
 *     is launched. A device-side problem (a bounded wait that gave up) is recorded in a status
 *     word at the start of the workspace and reported by hass_check. Nothing traps or aborts.
 *   - The device must be compute capability 10.x; anything else returns HASS_ERR_ARCH. There is
 *     no fallback path.
 *   - `workspace` is scratch the caller provides (hass_topk_distill_workspace_bytes gives the
 *     size; 256-byte aligned). The same workspace may be reused by successive calls on one
 *     stream; calls that may overlap on the GPU need separate workspaces.
 */
#ifndef HASS_H_
#define HASS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define HASS_K_MAX 256

typedef enum {
    HASS_OK = 0,
    HASS_ERR_INVALID_ARG = -1, /* null / misaligned pointer, size out of range */
    HASS_ERR_UNSUPPORTED = -2, /* legal but not implemented (e.g. N too large for one call) */
    HASS_ERR_WORKSPACE = -3,   /* workspace missing or too small */
    HASS_ERR_CUDA = -4,        /* a CUDA runtime/driver call failed, or no CUDA device */
    HASS_ERR_TIMEOUT = -5,     /* a bounded device-side wait expired (see hass_check) */
    HASS_ERR_ARCH = -6,        /* device is not sm_100 */
    HASS_ERR_RANGE = -7        /* fused path: a row's logits spread too far (see hass_topk_distill_fwd_bwd) */
} hass_status;

typedef enum { HASS_BF16 = 0, HASS_FP32 = 1 } hass_dtype; /* element type of dH_d */

/* Human-readable name of a status code (static string, never NULL). */
const char* hass_status_string(int status);

/* Library version, major * 10000 + minor * 100 + patch. */
int hass_version(void);

/*
 * Bytes of workspace that every entry point below accepts for this problem size.
 * The figure covers: a status block, per-CTA partial softmax statistics and Top-K candidate
 * buffers of the forward sweep, the index-sorted Top-K lists of the split backward, and two
 * bounded scratch areas for one chunk of rows (a fixed number of 128-row tiles that does not grow
 * with N): the bf16 un-normalised draft probabilities (fused call) or dz_d (split backward),
 * chunk_rows x V, and the fp32 Omega_hat term of dH_d, chunk_rows x d. A smaller workspace is
 * accepted down to room for one 128-row tile of scratch; the calls then work in smaller chunks.
 * Needs no GPU (assumes 148 SMs if none is present).
 */
int hass_topk_distill_workspace_bytes(int64_t N, int64_t d, int64_t V, int32_t K, size_t* bytes);

/*
 * Forward: Eq. 1 of the paper, L_i = - sum_{x in Omega_hat_i} q_i(x) log p_i(x), per row.
 *
 * Steps (Section 3.1 and the training listing of the appendix,
 * "Implementation of Harmonized Context Alignment": lm_head(hidden_states_target),
 * lm_head(predict), logit loss): target logits z_t = H_t W^T and draft logits z_d = H_d W^T over
 * the whole vocabulary (computed tile by tile, never stored), their log-sum-exp, the K largest
 * target logits per row (= K most probable tokens under q), and the loss.
 * q and p are full-vocabulary softmaxes; they are not renormalised over Omega_hat.
 *
 *   loss      [N]    out  per-row loss, unweighted
 *   topk_idx  [N,K]  out  Omega_hat, in descending q; equal logits: lower token id first
 *   topk_q    [N,K]  out  q(x) for those tokens
 *   lse_t     [N]    out  log sum_v exp z_t[v]
 *   lse_d     [N]    out  log sum_v exp z_d[v]
 */
int hass_topk_distill_fwd(const void* H_t, const void* H_d, const void* W, int64_t N, int64_t d,
                          int64_t V, int32_t K, float* loss, int32_t* topk_idx, float* topk_q,
                          float* lse_t, float* lse_d, void* workspace, size_t workspace_bytes,
                          void* cuda_stream);

/*
 * Forward for aligning steps j >= 2 of harmonized context alignment (Section 3.2): the target
 * side (q, Omega_hat) does not change between steps - the paper counts it in the "constant
 * part" of the cost (Appendix, Training Overhead) - so topk_idx / topk_q from an earlier
 * hass_topk_distill_fwd are INPUTS here and only the draft projection is computed.
 *
 *   topk_idx [N,K] in, topk_q [N,K] in;  loss [N] out, lse_d [N] out.
 */
int hass_topk_distill_fwd_draft(const void* H_d, const void* W, int64_t N, int64_t d, int64_t V,
                                int32_t K, const int32_t* topk_idx, const float* topk_q, float* loss,
                                float* lse_d, void* workspace, size_t workspace_bytes,
                                void* cuda_stream);

/*
 * Backward: gradient of sum_i grad_loss[i] * L_i with respect to H_d (the loss.backward() of the
 * training listing; the target side and the LM head receive no gradient - Section 2 says the
 * head is the target LLM's, and the Appendix says the constant part needs no gradient).
 *
 *   dz_d[i,v] = grad_loss[i] * ( S_q,i * p_i(v) - q_i(v) * [v in Omega_hat_i] ),  S_q = sum of topk_q
 *   dH_d      = dz_d W
 *
 * dz_d is formed one bounded chunk of rows at a time (recomputing z_d tile by tile from H_d, W
 * and lse_d) in bf16 inside the workspace and contracted with W on the tensor cores.
 *
 *   topk_idx, topk_q, lse_d   in   as written by the forward
 *   grad_loss [N]             in   upstream weight per row (loss weight w, step re-weighting
 *                                  beta^(j-1), masks, 1/N ...), or NULL for all ones
 *   dH_d      [N,d]           out  bf16 or fp32 according to dH_dtype (a hass_dtype)
 */
int hass_topk_distill_bwd(const void* H_d, const void* W, int64_t N, int64_t d, int64_t V, int32_t K,
                          const int32_t* topk_idx, const float* topk_q, const float* lse_d,
                          const float* grad_loss, void* dH_d, int dH_dtype, void* workspace,
                          size_t workspace_bytes, void* cuda_stream);

/*
 * Forward and backward in one call (the whole hot path of one aligning step): the same results as
 * hass_topk_distill_fwd followed by hass_topk_distill_bwd, up to rounding, but no logit is
 * computed twice and no row of W is gathered. Rows are processed in bounded chunks. Per chunk the
 * target rows are swept first (statistics and Top-K candidates), Omega_hat is selected, then the
 * draft rows are swept: their statistics, their logits at the row's Omega_hat (copied out of the
 * fp32 accumulator for Eq. 1), and the tile itself, written to the workspace as bf16 values
 * 2^(z_d log2(e) - ref2), ref2 a per-row exponent fixed from the row's largest logit among the
 * first 256 tokens. With coef = g S_q 2^ref2 / sum_v e^{z_d},
 *     dz_d(v) = coef ( spill(v) - [v in Omega_hat] g q(v) / coef ),
 * so the K entries of a row at its Omega_hat tokens are lowered in place (in bf16) and
 * dH_d = coef (spill W) is formed by the second GEMM, whose epilogue applies the row scale.
 * Precision: every entry of dz_d, the Omega_hat entries included, reaches the tensor cores in bf16
 * (2^-9 relative); the loss uses fp32 logits throughout.
 * Range condition: the fixed exponent holds as long as no draft logit of a row exceeds that
 * row's largest logit among tokens 0..255 by more than about 130 (natural-log units; a probability
 * ratio of e^130). The sweep detects a violation; the call therefore also enqueues the separate
 * forward and the recomputing backward as conditional launches that return at once unless a
 * violation was detected, in which case they redo the whole call exactly. The result is correct
 * either way; the conditional launches cost about 0.3 % when they have nothing to do. The _draft
 * form and the Top-P variant work the same way.
 * hass_combined_distill_fwd_bwd and the Bi-directional variant handle a violation differently: their
 * sweep records every row's largest logit, and the whole sequence is enqueued a second time as
 * conditional launches that take each row's exponent from that record (no logit of the row can
 * exceed it); a violation therefore costs one more pass and the result is correct either way.
 * HASS_ERR_RANGE is what hass_check reports if a violation was detected and nothing redid the call
 * (none of the entry points of this version leaves it at that).
 */
int hass_topk_distill_fwd_bwd(const void* H_t, const void* H_d, const void* W, int64_t N, int64_t d,
                              int64_t V, int32_t K, const float* grad_loss, float* loss,
                              int32_t* topk_idx, float* topk_q, float* lse_t, float* lse_d,
                              void* dH_d, int dH_dtype, void* workspace, size_t workspace_bytes,
                              void* cuda_stream);

/*
 * hass_topk_distill_fwd_bwd for aligning steps j >= 2: topk_idx / topk_q are inputs (as for
 * hass_topk_distill_fwd_draft), only the draft projection, its loss and dH_d are computed.
 */
int hass_topk_distill_fwd_bwd_draft(const void* H_d, const void* W, int64_t N, int64_t d, int64_t V,
                                    int32_t K, const int32_t* topk_idx, const float* topk_q,
                                    const float* grad_loss, float* loss, float* lse_d, void* dH_d,
                                    int dH_dtype, void* workspace, size_t workspace_bytes,
                                    void* cuda_stream);

/*
 * Combined training objective of one aligning step (Section 3.2: the cross-entropy between the
 * target's and the draft's next-token distributions plus the Top-K loss of Section 3.1 with
 * weight w, Section 4.1 uses w = 1.0), forward and backward in one call:
 *
 *   loss_ce[i]   = - sum_{v in Omega}     q_i(v) log p_i(v)        (full vocabulary)
 *   loss_topk[i] = - sum_{x in Omega_hat} q_i(x) log p_i(x)        (Eq. 1)
 *   dz_d[i,v]    = grad_loss[i] * ( (1 + w S_q) p(v) - q(v) - w q(v) [v in Omega_hat] )
 *   dH_d         = dz_d W
 *
 * i.e. the gradient of sum_i grad_loss[i] (loss_ce[i] + w loss_topk[i]) with respect to H_d. The
 * sweep spills the target tiles as well, a second GEMM forms q W per row, from which both the
 * cross-entropy, lse_d - <H_d[i], (q W)[i]>, and its gradient term follow; 8 N d V tensor FLOPs
 * are executed. Range condition as for hass_topk_distill_fwd_bwd, for target and draft logits
 * alike; a violation is repaired by a second pass of the same sequence (see there). The other
 * outputs are those of hass_topk_distill_fwd.
 * Workspace: hass_combined_distill_workspace_bytes (the normal workspace plus the target spill and
 * a q W buffer for one chunk of rows).
 */
int hass_combined_distill_workspace_bytes(int64_t N, int64_t d, int64_t V, int32_t K, size_t* bytes);
int hass_combined_distill_fwd_bwd(const void* H_t, const void* H_d, const void* W, int64_t N, int64_t d,
                                  int64_t V, int32_t K, float w_topk, const float* grad_loss,
                                  float* loss_ce, float* loss_topk, int32_t* topk_idx, float* topk_q,
                                  float* lse_t, float* lse_d, void* dH_d, int dH_dtype, void* workspace,
                                  size_t workspace_bytes, void* cuda_stream);

/*
 * Loss variants that the paper compares with the Top-K loss (Section 4.3, one sentence each; the exact
 * formulas below are this library's readings), forward and backward in one call:
 *
 *   HASS_LOSS_TOPK         Eq. 1; the same as hass_topk_distill_fwd_bwd.
 *   HASS_LOSS_TOP_P        Omega_hat = the shortest prefix of the tokens sorted by descending q whose
 *                          cumulative probability is larger than param = P, at most K tokens; loss and
 *                          gradient as Eq. 1 on that set. topk_idx / topk_q beyond the prefix are -1 / 0.
 *   HASS_LOSS_NORMED_TOPK  q and p both renormalised over Omega_hat (the K most probable tokens):
 *                          L = - sum qn log pn, qn = q / S_q, pn = p / S_p (a softmax of the draft
 *                          logits restricted to Omega_hat), dz_d = g (pn - qn) on Omega_hat, 0 elsewhere.
 *                          Only the target rows are swept; lse_d is not written (may be NULL).
 *   HASS_LOSS_BIDIR_TOPK   Omega_hat = the K most probable tokens under q united with the K most probable
 *                          under p (taken as a constant set); loss and gradient as Eq. 1 on the union.
 *                          topk_idx / topk_q must hold 2K entries per row: the target's K in descending q,
 *                          then the draft's tokens not among them in descending p, then -1 / 0. K <= HASS_K_MAX / 2.
 *
 * topk_n [N] (nullable) receives |Omega_hat| per row; for HASS_LOSS_TOP_P the count is negated (-K) on a row
 * whose K most probable tokens together still do not exceed P, i.e. whose prefix was cut by the cap of K
 * tokens rather than by P (K may be as large as HASS_K_MAX). The other arguments are those of
 * hass_topk_distill_fwd_bwd. The Recall@k surrogate and BiLD losses of that section are not built (the
 * paper does not define them).
 */
typedef enum {
    HASS_LOSS_TOPK = 0,
    HASS_LOSS_TOP_P = 1,
    HASS_LOSS_NORMED_TOPK = 2,
    HASS_LOSS_BIDIR_TOPK = 3
} hass_loss_variant;
int hass_variant_distill_fwd_bwd(const void* H_t, const void* H_d, const void* W, int64_t N, int64_t d,
                                 int64_t V, int32_t K, int variant, float param, const float* grad_loss,
                                 float* loss, int32_t* topk_idx, float* topk_q, int32_t* topk_n,
                                 float* lse_t, float* lse_d, void* dH_d, int dH_dtype, void* workspace,
                                 size_t workspace_bytes, void* cuda_stream);

/*
 * The same forward + backward for callers whose features live in HOST memory (the training
 * listing reads precomputed target hidden states per batch): H_t_host, H_d_host [N,d] bf16 are
 * copied to the device, the path runs, and loss_host [N] (fp32) and dH_d_host [N,d] (dH_dtype)
 * are copied back; topk_idx_host / topk_q_host may be NULL to skip their copy. W stays a DEVICE
 * pointer: the LM head is frozen and shared, so it is uploaded once, not per step.
 * grad_loss_host is a host pointer or NULL. Host buffers should be page-locked for the copies
 * to be asynchronous. The call returns after the stream has been synchronised (the host results
 * are then valid) and reports device-side errors like hass_check.
 * `workspace` must hold hass_topk_distill_host_workspace_bytes(...) bytes: the normal workspace
 * plus device staging for the inputs and outputs.
 * The copies overlap the computation: the call works in row chunks, the rows of chunk c + 1 travel to the
 * device while chunk c computes and the dH_d rows of chunk c travel back while chunk c + 1 computes. For this
 * the library keeps, per device, two copy streams and a pool of events of its own (created by the first call
 * on that device; no device memory); they are ordered after `cuda_stream` at the start of the call and
 * `cuda_stream` is ordered after them at its end.
 */
int hass_topk_distill_host_workspace_bytes(int64_t N, int64_t d, int64_t V, int32_t K, int dH_dtype,
                                           size_t* bytes);
int hass_topk_distill_fwd_bwd_host(const void* H_t_host, const void* H_d_host, const void* W,
                                   int64_t N, int64_t d, int64_t V, int32_t K,
                                   const float* grad_loss_host, float* loss_host,
                                   int32_t* topk_idx_host, float* topk_q_host, void* dH_d_host,
                                   int dH_dtype, void* workspace, size_t workspace_bytes,
                                   void* cuda_stream);

/*
 * HCA attention of the draft layer (Section 3.2 "Harmonized Context Alignment" and the attention
 * listing of the appendix), forward. In aligning step m + 1 the query at position t attends
 * causally to positions s <= t; the key and value of the pair (t, s) come from the target LLM's
 * features, except for t - s = i < m, where they come from the i-th most recent earlier draft
 * pass (i = 0: the latest pass, on the main diagonal):
 *     w[t, .] = softmax_{s <= t}( scale * <Q[t], k(t, s)> ),   O[t] = sum_s w[t, s] v(t, s).
 * The weights that multiply the draft values are the normalised ones (the text's concatenated
 * key/value sequence); m = 0 is plain causal attention (the first aligning step).
 * The projections q_proj/k_proj/v_proj/o_proj are ordinary GEMMs outside this call.
 *
 *   Q            [B, T, H, D]     bf16  projected queries (of the latest draft features, or of the
 *                                       target features when m = 0)
 *   K_t, V_t     [B, T, Hkv, D]   bf16  projected target features; H a multiple of Hkv, query head
 *                                       h reads key/value head h / (H / Hkv)
 *   K_d, V_d     HOST arrays of m DEVICE pointers, each [B, T, Hkv, D] bf16: entry i replaces the
 *                i-th sub-diagonal. Read during the call only. 0 <= m <= HASS_HCA_MAX_DRAFTS.
 *   D            must be 128 (HASS_ERR_UNSUPPORTED otherwise); scale > 0, normally 1/sqrt(D)
 *   O            [B, T, H, D]     bf16  out (32-byte aligned; inputs 16-byte aligned)
 *   lse          [B, H, T]        fp32  out, optional: natural-log normaliser of each query row
 *   workspace    at least hass_hca_attention_workspace_bytes (256) bytes, 256-byte aligned; holds
 *                the status word hass_check reads
 * One kernel is enqueued on cuda_stream. Errors as for the other entries: argument problems are
 * returned before anything is launched; a bounded device wait that gave up is reported by
 * hass_check as HASS_ERR_TIMEOUT and O is then undefined.
 */
#define HASS_HCA_MAX_DRAFTS 8
int hass_hca_attention_workspace_bytes(size_t* bytes);
int hass_hca_attention_fwd(const void* Q, const void* K_t, const void* V_t, const void* const* K_d,
                           const void* const* V_d, int32_t m, int64_t B, int64_t T, int64_t H,
                           int64_t Hkv, int64_t D, float scale, void* O, float* lse, void* workspace,
                           size_t workspace_bytes, void* cuda_stream);

/*
 * Backward of hass_hca_attention_fwd (Section 3.2; the paper prints the forward only, the gradients are the
 * chain rule through it): given dO = d(loss)/dO it returns the gradients with respect to every projected
 * input. With P the softmax weights (recomputed from lse), Dt = <dO[t], O[t]> and
 * dS[t,s] = P[t,s] (<dO[t], v(t,s)> - Dt) scale:
 *     dQ[t] = sum_s dS[t,s] k(t,s);   dK_t[s], dV_t[s] collect the pairs with t - s >= m;
 *     dK_d[i][s], dV_d[i][s] collect the single pair t = s + i of every query head of the group.
 *
 *   Q, K_t, V_t, K_d, V_d, m, B, T, H, Hkv, D, scale   as in the forward call
 *   O [B, T, H, D] bf16, lse [B, H, T] fp32              the forward's outputs (lse is required here)
 *   dO [B, T, H, D] bf16
 *   dQ [B, T, H, D], dK_t, dV_t [B, T, Hkv, D] bf16      out (32-byte aligned)
 *   dK_d, dV_d   HOST arrays of m DEVICE pointers, each [B, T, Hkv, D] bf16, out
 *   workspace    hass_hca_attention_bwd_workspace_bytes(B, T, H, m) bytes, 256-byte aligned: the status
 *                word, Dt, and dQ in fp32 (4 B T H D bytes)
 * Three kernels are enqueued on cuda_stream: a row kernel (Dt, the substituted entries with the draft passes'
 * gradients and their share of dQ), one tensor-core kernel for dK_t, dV_t and the key tiles' shares of dQ, which
 * it adds into the fp32 copy with atomic reductions (their order is not fixed, so dQ may differ between two
 * runs in the last bits of that fp32 sum), and the conversion of dQ to bf16. Errors as for the forward.
 */
int hass_hca_attention_bwd_workspace_bytes(int64_t B, int64_t T, int64_t H, int32_t m, size_t* bytes);
int hass_hca_attention_bwd(const void* Q, const void* K_t, const void* V_t, const void* const* K_d,
                           const void* const* V_d, int32_t m, int64_t B, int64_t T, int64_t H,
                           int64_t Hkv, int64_t D, float scale, const void* O, const float* lse,
                           const void* dO, void* dQ, void* dK_t, void* dV_t, void* const* dK_d,
                           void* const* dV_d, void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Synchronises `cuda_stream` and returns the status word of `workspace`: HASS_OK, or
 * HASS_ERR_TIMEOUT if a kernel gave up on a bounded wait (its outputs are then undefined), or
 * HASS_ERR_CUDA if the stream reports an error. Clears the status word.
 */
int hass_check(void* workspace, void* cuda_stream);

/*
 * Self-test of the library's failure detection (no counterpart in the paper). Every device-side wait of
 * the kernels above is bounded: a wait that runs out records a code in the workspace's status word,
 * raises a flag that ends the other waits of its CTA, and the kernel returns; hass_check then reports
 * HASS_ERR_TIMEOUT. This call exercises exactly that path without making any real kernel wait: it enqueues
 * one small kernel (one CTA of 128 threads, no copies, no tensor memory) whose threads wait on a barrier
 * that nothing completes, the first thread for limit_ns nanoseconds (1000 .. 100000000), the others until
 * the first one's give-up flag reaches them. Afterwards hass_check(workspace) must return
 * HASS_ERR_TIMEOUT once and HASS_OK from then on.
 *   workspace  at least 256 bytes, 256-byte aligned; word 0 is the status word; the kernel also writes
 *              word 16 = number of threads whose wait gave up (128) and word 17 = nanoseconds waited.
 */
int hass_selftest_wait_expiry(void* workspace, size_t workspace_bytes, uint64_t limit_ns, void* cuda_stream);

/*
 * Number of kernels of this library launched by the calling process so far (all entry points).
 * Lets a benchmark report how many of the library's own kernels ran in a timed region.
 */
int64_t hass_kernel_launch_count(void);

/*
 * hass_topk_distill_fwd with no workspace argument. The paper has no counterpart to this entry:
 * it exists for callers that cannot obtain device memory at the time of the call. Typical cases:
 * a process whose framework reserved the whole GPU at start-up, so any later cudaMalloc fails; a
 * plug-in interface that hands the callee its input and output buffers and nothing else; a
 * latency-critical loop that must not run into the device-wide synchronisation cudaMalloc and
 * cudaFree imply. For them the partial softmax statistics and Top-K candidates of the forward
 * sweep live in an array built into the library's device image instead of a caller workspace.
 *
 *   - The array is HASS_STATIC_SCRATCH_MAX_BYTES (32 MiB) and every GPU that loads the library
 *     holds it until the process exits. The forward scratch of a problem is about
 *     slots * 128 * (8 * cap(K) + 16) bytes: slots = the partial-result slots of its tile schedule
 *     (the number of SMs for up to 128 rows, about three times that for thousands of rows) and
 *     cap(K) = 16 for K <= 16, else K + max(2 K, 96) + 32 rounded up to a multiple of 32.
 *     hass_topk_distill_fwd_static_scratch_bytes returns the exact figure. On a 148-SM device
 *     N = 8192, V = 128256 needs 7.7 MiB for K <= 16 and 69.6 MiB for K = 17, so it is accepted up
 *     to K = 16; N = 128 fits up to K = 53. A problem that does not fit is refused with
 *     HASS_ERR_UNSUPPORTED before anything is launched; use hass_topk_distill_fwd with a workspace.
 *   - The call allocates and frees nothing, in this library or through any other.
 *   - The first call on each device looks up the array's device address (a CUDA runtime query,
 *     with that device current). Make that first call outside any stream capture.
 *   - All calls on a device share the one array, and it keeps whatever the previous call left.
 *     The call itself clears the only word that has to start at zero. Two calls that can overlap
 *     on the GPU (different streams, no ordering between them) race on the array: serialise them.
 *   - Arguments and outputs are those of hass_topk_distill_fwd. device_status is optional
 *     (NULL to skip): a caller-owned DEVICE word that receives, in stream order, 0 or the
 *     non-zero code of a bounded device-side wait that gave up (outputs are then undefined);
 *     it replaces hass_check, which needs a workspace pointer.
 */
#define HASS_STATIC_SCRATCH_MAX_BYTES (32u << 20)
int hass_topk_distill_fwd_static_scratch_bytes(int64_t N, int64_t d, int64_t V, int32_t K, size_t* bytes);
int hass_topk_distill_fwd_static(const void* H_t, const void* H_d, const void* W, int64_t N, int64_t d,
                                 int64_t V, int32_t K, float* loss, int32_t* topk_idx, float* topk_q,
                                 float* lse_t, float* lse_d, unsigned int* device_status,
                                 void* cuda_stream);

/*
 * Optional per-kernel timing for benchmarks (no counterpart in the paper). While enabled, each
 * kernel launch of the library is bracketed by CUDA events on its stream (the events are created
 * on the first enable). hass_profile_summary waits for the recorded events, adds the elapsed
 * milliseconds and launch counts per kernel kind into arrays of at least HASS_PROFILE_KINDS
 * entries, and clears the records. Kinds: 0 logits+statistics GEMM (forward), 1 dz_d GEMM
 * (backward, recompute), 2 dH_d GEMM (backward), 3 finalize, 4 backward preparation, 5 the conditional
 * launches of the exact route behind a fused call (they return at once unless it is needed),
 * 6 HCA attention forward, 7 / 8 / 9 HCA attention backward: conversion of dQ to bf16, the tensor-core kernel,
 * the row kernel (row sums, substituted entries, the draft passes' gradients), 10 the sweep of the draft rows in hass_topk_distill_fwd_bwd, its
 * _draft form and the Top-P variant (kind 0 is then the sweep of the target rows alone).
 * At most 8192 launches are recorded between summaries. Not thread-safe.
 */
#define HASS_PROFILE_KINDS 11
int hass_profile_enable(int on);
int hass_profile_summary(double* ms_by_kind, int64_t* launches_by_kind, int n_kinds);

#ifdef __cplusplus
}
#endif
#endif /* HASS_H_ */
