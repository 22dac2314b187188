// Shared host/device helpers of the HEART CUDA library (geometry, workspace layout, status word).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "heart.h"

namespace heart {

constexpr int kD = 128;  // head_dim (fixed)

// Geometry derived from a validated heart_config.
struct Geom {
  int B, H, R, N, block, nb, W, idx_stride;
  long long sb, sh, sn;  // element strides of Q/K/V/O
  double scale, gate_lo, gate_hi;
  unsigned flags;
  int bpc, nchunks;  // block-sum kernel: key/query blocks per CTA and CTAs per (head row, tensor)
};

// Chunking of the block-sum pass: at most one wave of 5 CTAs per SM (48 registers x 256 threads) on a 148-SM part, whatever the
// device (the split fixes the summation order, so it must depend on the shape only).  Never a little
// more than one wave: the few CTAs of a second wave would each run as long as the whole first one.
#ifndef HEART_CHUNK_TARGET
#define HEART_CHUNK_TARGET (148 * 5)
#endif
__host__ inline void set_chunks(Geom &g) {
  const int target = HEART_CHUNK_TARGET;
  int per_pair = target / (2 * g.R);
  if (per_pair < 1) per_pair = 1;
  g.bpc = (g.nb + per_pair - 1) / per_pair;
  if (g.bpc < 1) g.bpc = 1;
  g.nchunks = (g.nb + g.bpc - 1) / g.bpc;
}

// Workspace layout (all offsets 256-byte aligned).
struct Workspace {
  int32_t *status;    // [64]   word 0: sticky device-check code; word 1: detail; word 8: ticket counter
                      //        of the drift kernel (zero between launches); words 10-11: signature of
                      //        the (Q, K, shape) whose block means the workspace holds (0: none)
  double *bmean;      // [2][R][nb][D]  per-block (pooled) means of Q (0) and K (1)
  double *psum;       // [2][R][nchunks][D]  per-CTA partial token sums
  double *mean;       // [2][R][D]      token means of the current step
  uint8_t *pre;       // [R]            head-wise decision before the gate
  uint8_t *refresh;   // [R]            final decision of the current step
  double *drift;      // [R]
  int32_t *order;     // [R * ceil(N / 128)] order in which an attention launch takes the tiles of each head
  double *scores;     // [R][nb][pitch] pooled scores of the refreshed heads, pitch = nb rounded up to 32
  void *pairs;        // strided antidiagonal estimator only (HEART_ESTIMATOR_ANTIDIAG in the flags):
                      // float2 [R][N/16][nb], a (max, sum) pair per (query group, key block)
  size_t bytes_drift;  // what heart_drift alone touches (everything above `scores`)
  size_t bytes;
};

__host__ inline size_t align256(size_t x) { return (x + 255) & ~size_t(255); }

__host__ inline Workspace carve(const Geom &g, void *base) {
  Workspace w;
  char *p = static_cast<char *>(base);
  size_t off = 0;
  w.status = reinterpret_cast<int32_t *>(p + off);
  off += align256(64 * sizeof(int32_t));
  w.bmean = reinterpret_cast<double *>(p + off);
  off += align256(sizeof(double) * 2 * (size_t)g.R * g.nb * kD);
  w.psum = reinterpret_cast<double *>(p + off);
  off += align256(sizeof(double) * 2 * (size_t)g.R * g.nchunks * kD);
  w.mean = reinterpret_cast<double *>(p + off);
  off += align256(sizeof(double) * 2 * (size_t)g.R * kD);
  w.pre = reinterpret_cast<uint8_t *>(p + off);
  off += align256((size_t)g.R);
  w.refresh = reinterpret_cast<uint8_t *>(p + off);
  off += align256((size_t)g.R);
  w.drift = reinterpret_cast<double *>(p + off);
  off += align256(sizeof(double) * (size_t)g.R);
  w.order = reinterpret_cast<int32_t *>(p + off);
  off += align256(sizeof(int32_t) * (size_t)g.R * (size_t)((g.N + 127) / 128));
  w.bytes_drift = off;
  w.scores = reinterpret_cast<double *>(p + off);
  off += align256(sizeof(double) * (size_t)g.R * g.nb * (size_t)(((g.nb + 31) / 32) * 32));
  w.pairs = p + off;
  if (g.flags & HEART_ESTIMATOR_ANTIDIAG)
    off += align256(8 * (size_t)g.R * (size_t)(g.N / HEART_ANTIDIAG_STRIDE) * (size_t)g.nb);
  w.bytes = off;
  return w;
}

constexpr int kStatusTicketWord = 8, kStatusSigWord = 10;

#ifdef __CUDACC__
// Programmatic dependent launch: a kernel launched with the stream-serialisation attribute may be
// scheduled while the kernel before it on the stream drains; it must not touch that kernel's results
// before pdl_wait().  pdl_launch_dependents() in the earlier kernel lets the later one be scheduled
// once every CTA has issued it (or exited).
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// exp(x) for x <= 0 in about a third of the instructions of the library routine, which spends most of
// its time on ranges that cannot occur here: n = rint(x log2 e) by the magic-number add, r = x - n ln 2
// in two steps, the Taylor polynomial of degree 13 on |r| <= ln 2 / 2 (truncation 4e-18), 2^n by an
// integer add into the exponent field.  Below -708 (weights under 1e-307 of the row maximum) it
// returns 0.  Within an ulp or two of the correctly rounded value, like the library routine.
__device__ __forceinline__ double exp_nonpositive(double x) {
  if (!(x >= -708.0)) return 0.0;  // also NaN
  const double t = fma(x, 1.4426950408889634, 6755399441055744.0);
  const int n = __double2loint(t);
  const double fn = t - 6755399441055744.0;
  double r = fma(fn, -6.93147180369123816490e-01, x);
  r = fma(fn, -1.90821492927058770002e-10, r);
  double q = 1.6059043836821613e-10;            // 1/13!
  q = fma(q, r, 2.08767569878681e-09);          // 1/12!
  q = fma(q, r, 2.505210838544172e-08);         // 1/11!
  q = fma(q, r, 2.755731922398589e-07);         // 1/10!
  q = fma(q, r, 2.7557319223985893e-06);        // 1/9!
  q = fma(q, r, 2.48015873015873e-05);          // 1/8!
  q = fma(q, r, 1.984126984126984e-04);         // 1/7!
  q = fma(q, r, 1.388888888888889e-03);         // 1/6!
  q = fma(q, r, 8.333333333333333e-03);         // 1/5!
  q = fma(q, r, 4.1666666666666664e-02);        // 1/4!
  q = fma(q, r, 1.6666666666666666e-01);        // 1/3!
  q = fma(q, r, 0.5);
  q = fma(q, r, 1.0);
  q = fma(q, r, 1.0);
  return __hiloint2double(__double2hiint(q) + (n << 20), __double2loint(q));
}

template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

// Validates the shape part of a config and derives the geometry: HEART_OK or an error code.
int make_geom(const heart_config *c, Geom *g);
// What the block means in a workspace belong to (tensor addresses, shape, strides), never 0.
unsigned long long block_means_signature(const Geom &g, const void *Q, const void *K);

// Launchers (defined in the kernel files). Each returns the cudaError_t of its launches and
// adds the number of kernels it launched to *launches.
cudaError_t launch_block_sums(const Geom &g, const void *Q, const void *K, const Workspace &w,
                              cudaStream_t s, int *launches);
cudaError_t launch_decide(const Geom &g, const Workspace &w, const double *delta, heart_state st,
                          double *drift_out, uint8_t *refresh_out, cudaStream_t s, int *launches);
// expect_sig != 0: the block means were left by an earlier call; the kernels check the workspace's
// signature against it and report HEART_ERR_DEVICE_CHECK (masks untouched) on a mismatch.
cudaError_t launch_predict_mask(const Geom &g, const Workspace &w, const double *tau,
                                const uint8_t *refresh, heart_state st, cudaStream_t s, int *launches,
                                unsigned long long expect_sig = 0);
// The two halves of it: pooled scores into w.scores, then the top-p rows over w.scores.
cudaError_t launch_pooled_scores(const Geom &g, const Workspace &w, const uint8_t *refresh, cudaStream_t s,
                                 int *launches, unsigned long long expect_sig);
cudaError_t launch_top_p(const Geom &g, const Workspace &w, const double *tau, const uint8_t *refresh,
                         heart_state st, cudaStream_t s, int *launches, unsigned long long expect_sig);
// Strided antidiagonal estimator: log block importances of the refreshed heads into w.scores.
cudaError_t launch_antidiag_scores(const Geom &g, const Workspace &w, const void *Q, const void *K,
                                   const uint8_t *refresh, cudaStream_t s, int *launches);
// h0/hcount select the heads [h0, h0 + hcount) of every batch entry (hcount <= 0: all heads).
cudaError_t launch_attention(const Geom &g, const void *Q, const void *K, const void *V,
                             const int32_t *kv_idx, const int32_t *kv_cnt, bool dense, void *O,
                             float *lse, int32_t *status, int32_t *order, cudaStream_t s, int *launches,
                             int h0 = 0, int hcount = 0);

cudaError_t launch_token_drift(const Geom &g, const void *Qa, const void *Ka, const void *Qb,
                               const void *Kb, double *partial, double *drift_out, cudaStream_t s,
                               int *launches);
int token_drift_chunks(const Geom &g, int *rows_per_cta);
cudaError_t launch_mask_iou(const Geom &g, const uint32_t *A, const uint32_t *B, double *iou,
                            long long *counts, cudaStream_t s, int *launches);

size_t band_error_workspace_bytes(int C, int T, int H, int W);
cudaError_t launch_band_error(const float *ys, const float *yd, int C, int T, int H, int W, const double *weights,
                              double eps, double *out, void *workspace, cudaStream_t s, int *launches);

}  // namespace heart
