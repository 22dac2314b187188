/*
 * heart.h -- C ABI of the B200 (sm_100a) HEART sparse-attention hot path.
 *
 * One layer-step of head-wise adaptive block-sparse attention for video
 * diffusion transformers:
 *   (a) Temporal Mask Reuse: mean-pooled query/key drift of every head against
 *       its cached anchor step and the refresh-or-reuse decision
 *       (Temporal Mask Reuse section, Eq. mean-pooled drift; Algorithm 1);
 *   (b) block-importance mask prediction for the refreshed heads: block-pooled
 *       Q.K^T scores, row softmax, cumulative top-p selection with each head's
 *       own threshold tau_h (Observation II; the minimal cumulative-mass set of
 *       Observation I; tau_h is the output of the offline calibration, an input
 *       here);
 *   (c) block-sparse attention over the retained (query block, key block) pairs
 *       with online softmax.
 *
 * Conventions
 *   - Every pointer below is a DEVICE pointer owned by the caller unless it is
 *     marked "host".  The library never allocates or frees device memory, and
 *     everything the method carries from step to step lives in heart_state and
 *     the caller's workspace.  What the library itself keeps, per device and
 *     until the process exits: the two internal streams and the events of
 *     heart_step_host (created by its first call), and the built-in scratch
 *     array of heart_drift_static with its cached device address.
 *   - Every call except heart_get_status is asynchronous on `stream` and never
 *     synchronises.  Arguments are validated on the host before any launch;
 *     on a host-detected error nothing is launched and no state changes.
 *   - R = B*H "head rows"; n_b = ceil(N / block); W = ceil(n_b / 32).
 *   - Q, K, V, O are bf16 with head_dim contiguous; the element strides of the
 *     other three dimensions are given in heart_config (0,0,0 selects the
 *     contiguous [B,H,N,D] layout).  Base pointers must be 16-byte aligned and
 *     strides multiples of 8 elements.
 *   - Return value: HEART_OK or one of the HEART_ERR_* codes (never throws,
 *     never traps, never exits).
 */
#ifndef HEART_H_
#define HEART_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef void *heart_stream_t; /* a cudaStream_t (NULL = the legacy default stream) */

enum {
  HEART_OK = 0,
  HEART_ERR_INVALID = 1,      /* null pointer, bad size/stride/alignment               */
  HEART_ERR_UNSUPPORTED = 2,  /* D != 128, block not in {64,128}, n_b > 1024            */
  HEART_ERR_CUDA = 3,         /* a CUDA call or launch failed (see heart_strerror)      */
  HEART_ERR_DEVICE_CHECK = 4, /* a device-side check failed: bad index-list entry or a  */
                              /* bounded wait ran out; only via heart_get_status        */
  HEART_ERR_TOO_LARGE = 5,    /* heart_drift_static: the shape needs more scratch than   */
                              /* HEART_STATIC_SCRATCH_BYTES                              */
  HEART_ERR_INFEASIBLE = 6    /* heart_assign_thresholds: no assignment meets the budget */
};

#define HEART_FORCE_REFRESH 1u /* every head refreshes this step (decision overridden)  */
#define HEART_FORCE_DENSE 2u   /* dense warm-up step (the baselines' first denoising    */
                               /* steps): attention over all blocks, TMR state untouched */
#define HEART_BLOCK_MEANS_VALID 4u /* heart_predict_mask only: the workspace already holds */
                               /* the block means of these Q, K (see that call)          */
#define HEART_ESTIMATOR_ANTIDIAG 8u /* mask prediction ranks blocks with the strided       */
                               /* antidiagonal estimator instead of mean pooling (see    */
                               /* heart_predict_mask); needs a larger workspace          */
#define HEART_ANTIDIAG_STRIDE 16   /* tokens per sampled group of that estimator          */

#define HEART_MAX_BLOCKS 1024  /* largest supported n_b */

typedef struct {
  int32_t B, H, N, D;      /* D must be 128                                                */
  int32_t block;           /* 64 or 128 tokens; query and key blocks are equal             */
  int64_t stride_b, stride_h, stride_n; /* elements; all 0 = contiguous [B,H,N,D]          */
  double scale;            /* logit scale; <= 0 selects 1/sqrt(D) (query-key interaction   */
                           /* of the appendix)                                             */
  double gate_lo, gate_hi; /* layer gate on the refreshed-head fraction (0.4 / 0.8 in the  */
                           /* appendix); lo = 0, hi = 1 disables it                        */
  int32_t idx_stride;      /* row pitch of kv_idx in entries, >= n_b                       */
  uint32_t flags;          /* HEART_FORCE_*                                                */
} heart_config;

/* TMR state of one layer (Algorithm 1: cached anchor features and anchor mask). */
typedef struct {
  double *anchor_q, *anchor_k; /* [R, D]  token-mean Q and K at each head's anchor step    */
  uint8_t *has_anchor;         /* [R]     0 = "no cached anchor exists"                    */
  uint32_t *mask_bits;         /* [R, n_b, W] bit J%32 of word J/32 = pair (I,J) retained  */
  int32_t *kv_idx;             /* [R, n_b, idx_stride] retained key blocks, ascending      */
  int32_t *kv_cnt;             /* [R, n_b] number of retained key blocks per query block   */
} heart_state;

/* Bytes of scratch every compute call needs (block means, token means, flags, status
 * word, and the pooled scores of the mask predictor: 8 * R * n_b * roundup(n_b, 32) bytes,
 * by far the largest part; with HEART_ESTIMATOR_ANTIDIAG in cfg->flags another
 * 8 * R * floor(N / 16) * n_b bytes).  Host-only; returns 0 for an invalid or unsupported config.
 * The caller allocates it once (256-byte aligned) and zero-fills it before first use. */
size_t heart_workspace_bytes(const heart_config *cfg /* host */);

/* The leading part of that workspace which heart_drift alone reads and writes (everything
 * but the pooled scores).  A caller that only ever calls heart_drift may allocate just this
 * much.  Host-only; 0 for an invalid or unsupported config. */
size_t heart_drift_workspace_bytes(const heart_config *cfg /* host */);

/* Clears has_anchor (and zeroes kv_cnt) so the next step refreshes every head
 * (Algorithm 1, "no cached anchor exists"). */
int heart_state_reset(const heart_config *cfg, heart_state *st /* host struct */, heart_stream_t stream);

/* (a) Temporal Mask Reuse decision -- Eq. mean-pooled drift, Algorithm 1, layer gate.
 *   mean_q[r,:] = (1/N) sum_i Q[r,i,:]  (same for K), fp64;
 *   drift[r]    = ||anchor_q[r]-mean_q[r]||_1 + ||anchor_k[r]-mean_k[r]||_1   (+inf if no anchor);
 *   refresh[r]  = !has_anchor[r] || drift[r] > delta[r]   (strict; then the gate per batch entry:
 *                 fraction < gate_lo -> anchored heads reuse, fraction > gate_hi -> all refresh);
 *   refreshed heads: anchor <- current means, has_anchor <- 1.
 * delta [R] fp64 (a negative entry always refreshes).  drift_out [R] fp64 and refresh_out [R] u8
 * may each be NULL.  Also leaves the per-block means of Q and K in the workspace. */
int heart_drift(const heart_config *cfg, const void *Q, const void *K, const double *delta,
                heart_state *st, double *drift_out, uint8_t *refresh_out, void *workspace,
                heart_stream_t stream);

/* (b) Mask prediction for the heads with refresh[r] != 0 (NULL = all heads) -- Observation II.
 *   Qp[r,I,:] = mean of the real tokens of block I (same for Kp), fp64;
 *   P[r,I,:]  = softmax_J( scale * <Qp[r,I], Kp[r,J]> );
 *   keep the first k* blocks in (P descending, J ascending) order, k* = min{k>=1: cum mass >= tau[r]};
 *   tau[r] >= 1 (or NaN, or a mass that never reaches tau) keeps all n_b blocks; at least one is
 *   kept: tau[r] <= 0 keeps exactly the largest block (the lowest index among equals).
 * Writes mask_bits, kv_idx (ascending), kv_cnt of those heads; other heads are untouched.
 * tau [R] fp64.
 * With HEART_ESTIMATOR_ANTIDIAG in cfg->flags the importances come from the strided antidiagonal
 * estimator instead (the estimator family of the paper's main sparse-attention backbone, appendix
 * "XAttention and SVG2 Configurations": anti-diagonal scoring with stride 16; the paper states the
 * stride and the block size only, so the definition is this library's):
 *   tokens are taken in groups of s = HEART_ANTIDIAG_STRIDE; only the floor(N / s) full groups are
 *   sampled;  S'(a, c) = (scale / s) * sum_{t<s} <q_{a s + t}, k_{c s + s-1-t}>;  P'(a, .) = softmax over
 *   the groups c;  P[r,I,J] = sum of P'(a, c) over the groups of blocks I and J / groups in I;
 *   a query block without a full group gets uniform P, a key block without one gets P = 0;
 *   then the same selection rule.  The contraction runs in bf16 with fp32 accumulation on the tensor
 *   cores, the exponentials in fp32, the block sums and the selection in fp64.  The workspace must
 *   have been sized with the flag set.  heart_step and heart_step_host honour the flag too.
 * (Pooled estimator:) the call first repeats heart_drift's pass over Q and K for the block means.  A caller that has just
 * run heart_drift (or heart_predict_mask) on the same Q and K pointers, the same cfg shape and the
 * same workspace, with no heart_full_token_drift and no change of the tensors' contents in between,
 * sets HEART_BLOCK_MEANS_VALID in cfg->flags: the pass is skipped and the means in the workspace are
 * used.  The kernels compare a signature of (pointers, shape, strides) that the pass left in the
 * workspace; on a mismatch nothing is predicted and heart_get_status reports
 * HEART_ERR_DEVICE_CHECK.  The contents of the tensors are the caller's promise. */
int heart_predict_mask(const heart_config *cfg, const void *Q, const void *K, const double *tau,
                       const uint8_t *refresh, heart_state *st, void *workspace,
                       heart_stream_t stream);

/* (c) Block-sparse attention with online softmax over the listed pairs.
 *   For query token i of block I:  o_i = sum_j softmax_j(scale * <q_i,k_j>) v_j over the real keys
 *   (j < N) of the key blocks kv_idx[r,I,0..kv_cnt[r,I]).  bf16 in, fp32 accumulate, bf16 out (RNE).
 *   An empty list gives zeros (lse = -inf).  Rows i >= N are never written.
 *   lse [R, N] fp32 natural-log sum-exp of the scaled logits, or NULL.
 *   Lists must hold distinct block indices in [0, n_b); entries out of range are skipped and
 *   reported as HEART_ERR_DEVICE_CHECK through heart_get_status. */
int heart_block_sparse_attn(const heart_config *cfg, const void *Q, const void *K, const void *V,
                            const int32_t *kv_idx, const int32_t *kv_cnt, void *O, float *lse,
                            void *workspace, heart_stream_t stream);

/* One whole layer-step: heart_drift, then heart_predict_mask for the refreshed heads, then
 * heart_block_sparse_attn with the (cached or new) lists -- all on `stream`, no host round trip
 * (Algorithm 1 followed by the sparse attention it feeds).  Results equal the three calls made
 * one after the other.  With HEART_FORCE_DENSE only dense attention runs (state untouched,
 * refresh_out = 0, drift_out = +inf). */
int heart_step(const heart_config *cfg, const void *Q, const void *K, const void *V,
               const double *delta, const double *tau, heart_state *st, void *O, float *lse,
               double *drift_out, uint8_t *refresh_out, void *workspace, heart_stream_t stream);

/* heart_step for callers whose tensors live in HOST memory (the end-to-end path).
 *   Q_host, K_host, V_host: bf16, contiguous [B,H,N,D] (cfg strides must be 0,0,0), ideally pinned;
 *   O_host: bf16 [B,H,N,D] result; drift_host [R] fp64 and refresh_host [R] u8 may be NULL.
 *   Q_dev, K_dev, V_dev, O_dev: caller-owned DEVICE staging buffers of B*H*N*D bf16 each.
 * Enqueues the uploads of Q and K and the drift / mask kernels on `stream`; V goes up, one group of
 * heads at a time, on an internal stream while those run, the attention of a head group starts on
 * `stream` when its V has landed, and its O goes down on a second internal stream while the next
 * group computes; drift and refresh follow.  `stream` finally waits for the last download.  Does
 * not synchronise: the host results are valid once `stream` has drained, and later work on `stream`
 * is ordered after everything this call enqueued.  Results equal heart_step on the same data.
 * The two internal streams and a few events are created on the first call on each device and kept
 * (no device memory is allocated); calls on one device are serialised on a host mutex while they
 * enqueue.  delta, tau, st, workspace are device-side exactly as in heart_step. */
int heart_step_host(const heart_config *cfg, const void *Q_host, const void *K_host, const void *V_host,
                    const double *delta, const double *tau, heart_state *st, void *O_host,
                    double *drift_host, uint8_t *refresh_host, void *Q_dev, void *K_dev, void *V_dev,
                    void *O_dev, void *workspace, heart_stream_t stream);

/* Built-in scratch of heart_drift_static: 16 MiB, enough for B*H*n_b <= ~8100 head-row blocks
 * (e.g. 12 heads x 512 blocks; the 40-head and 720P shapes need the caller-allocated path). */
#define HEART_STATIC_SCRATCH_BYTES (16u << 20)

/* heart_drift without a workspace argument, for callers that cannot allocate device memory.
 * (No counterpart in the paper: this is a packaging variant of call (a) above.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a host framework's
 * allocator-managed region where foreign allocations are forbidden or would fragment a fully
 * reserved GPU, in a real-time or callback context that must not block on the driver's allocator,
 * or a plugin that is handed Q/K and the TMR state but no way to obtain scratch.  Such a caller
 * still passes its inputs, outputs and state; only the scratch (block means, token means, flags) comes
 * from a fixed HEART_STATIC_SCRATCH_BYTES array compiled into the library.  The call makes no
 * cudaMalloc / cudaFree and calls no allocating routine.
 *
 * Same arguments, results and error codes as heart_drift (an invalid cfg gives heart_drift's code), except:
 *   - no `workspace`; st->mask_bits / kv_idx / kv_cnt may be NULL (they are not touched);
 *   - a shape whose heart_drift_workspace_bytes exceeds HEART_STATIC_SCRATCH_BYTES is rejected with
 *     HEART_ERR_TOO_LARGE before anything is launched;
 *   - the per-block means it leaves behind are in the built-in array, not in a caller workspace,
 *     so a following heart_predict_mask recomputes them (it always does).
 * The array is part of the library image: every GPU that loads the library holds those 16 MiB
 * until the process exits.  The first call on each device looks the array's device address up
 * (with that device current) and caches it; make that first call outside any stream capture.
 * All calls on a device share the one array and it keeps the previous call's contents.  Every
 * value the kernels read from it is rewritten by the same call first, except one counter that the
 * kernels expect to find at zero (the layer gate's ticket); each call clears it on `stream` before
 * its kernels run.  Two calls that overlap on the GPU (different streams, no ordering between
 * them) race on the array and give undefined results for both -- serialise them; calls after the
 * race are sound again, because of that clearing. */
int heart_drift_static(const heart_config *cfg, const void *Q, const void *K, const double *delta,
                       heart_state *st, double *drift_out, uint8_t *refresh_out, heart_stream_t stream);

/* ---- Analysis quantities (not on the layer-step path; nothing else reads their results) ---- */

/* Full-token drift between two steps of the same layer -- Eq. full-token drift, the costly
 * reference that the mean-pooled drift of heart_drift approximates (TMR section):
 *   drift_out[r] = (1/N) sum_i ( ||Qa[r,i]-Qb[r,i]||_1 + ||Ka[r,i]-Kb[r,i]||_1 ),  fp64 [R].
 * Qa, Ka (the cached step) and Qb, Kb (the current step) are bf16 with the layout cfg gives.
 * One streaming pass over the four tensors; uses the workspace as scratch (a later heart_drift or
 * heart_predict_mask rewrites what it needs); reads and writes no TMR state. */
int heart_full_token_drift(const heart_config *cfg, const void *Qa, const void *Ka, const void *Qb,
                           const void *Kb, double *drift_out, void *workspace, heart_stream_t stream);

/* Block-mask IoU between two steps -- Observation I (adjacent-step mask similarity), taken over the
 * retained (query block, key block) pairs of each head:
 *   iou_out[r] = |A_r AND B_r| / |A_r OR B_r|   (1 when both masks are empty), fp64 [R].
 * mask_a, mask_b: [R, n_b, W] bit masks in the mask_bits layout of heart_state (bits at J >= n_b
 * must be zero, as heart_predict_mask leaves them).  counts_out: optional int64 [R, 2] =
 * (intersection, union) pair counts, or NULL. */
int heart_mask_iou(const heart_config *cfg, const uint32_t *mask_a, const uint32_t *mask_b,
                   double *iou_out, int64_t *counts_out, heart_stream_t stream);

/* Frequency-aware velocity error of the offline calibration -- Eq. calibration error and the
 * appendix paragraph "Frequency-aware velocity error" (an offline quantity: not on the layer-step path).
 *   err = y_sparse - y_dense;  3-D DFT over (t, y, x) of every channel;  along an axis of length n a
 *   frequency is low when it lies within floor(n/4) of the zero frequency (after fftshift);
 *   LL = low t, low y and low x;  LH = low t, high on at least one spatial axis;
 *   HL = high t, low on both spatial axes;  HH = the rest;
 *   e = sum_q w_q * (spectral energy of err in band q) / (spectral energy of y_dense + eps).
 * y_sparse, y_dense: fp32 [C, T, H, W], contiguous, device.  weights: host, (w_LL, w_LH, w_HL, w_HH)
 * (the paper uses 1.0, 0.5, 0.01, 0.01 and eps = 1e-10).  out: device, fp64 [6] =
 * (e, E_LL, E_LH, E_HL, E_HH, denominator), energies of the unnormalised DFT, summed over channels.
 * workspace: heart_band_error_workspace_bytes(C, T, H, W) bytes of device scratch (four fp64 copies of
 * the tensor), 256-byte aligned; it need not be cleared. */
size_t heart_band_error_workspace_bytes(int32_t C, int32_t T, int32_t H, int32_t W);
int heart_band_error(const float *y_sparse, const float *y_dense, int32_t C, int32_t T, int32_t H, int32_t W,
                     const double *weights /* host [4] */, double eps, double *out, void *workspace,
                     heart_stream_t stream);

/* Threshold assignment of the offline calibration -- the one-choice-per-head assignment problem of the
 * section "Error-guided Budgeted Calibration" (the last step of Algorithm 2; appendix "Optimization
 * and budget": three candidate thresholds 0.85 / 0.90 / 0.95 per head):
 *     minimise   sum_i E[i][k_i]
 *     subject to one candidate k_i per head i  and  (1/M) sum_i S[i][k_i] >= S_min.
 * An offline problem on M * K numbers: it runs on the HOST (every pointer here is a host pointer, no
 * GPU is touched) as an exact multiple-choice-knapsack search.
 *   E, S: [n_heads, n_candidates] row-major fp64, the measured error and realised sparsity of each
 *   candidate of each head (the heads of all layers flattened); finite values.
 *   choice_out [n_heads]: the chosen candidate index per head.  objective_out, mean_sparsity_out
 *   (optional): the plain left-to-right sums of the chosen entries (the second divided by n_heads) --
 *   the same arithmetic that decides feasibility.  proved_optimal_out (optional): 1 when the search
 *   ran to the end (always, short of pathological tables with tens of millions of undominated
 *   partial sums), 0 when it stopped early and returns the best assignment found.
 * Among assignments of exactly equal objective any one may be returned.
 * Returns HEART_ERR_INFEASIBLE (outputs untouched) when even the sparsest candidate of every head
 * misses the budget. */
int heart_assign_thresholds(const double *E /* host */, const double *S /* host */, int32_t n_heads,
                            int32_t n_candidates, double S_min, int32_t *choice_out /* host */,
                            double *objective_out /* host */, double *mean_sparsity_out /* host */,
                            int32_t *proved_optimal_out /* host */);

/* Synchronises `stream`, reads the workspace status word into *code_out (host) and clears it.
 * The only call that blocks. */
int heart_get_status(void *workspace, heart_stream_t stream, int32_t *code_out /* host */);

/* Static description of a return code; for HEART_ERR_CUDA includes the last CUDA error text
 * seen by the calling thread. */
const char *heart_strerror(int code);

/* Number of kernels the last compute call on this thread launched (for accounting). */
int heart_last_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* HEART_H_ */
