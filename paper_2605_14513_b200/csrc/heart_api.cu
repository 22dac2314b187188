// C ABI of the HEART hot path: argument validation, workspace carving and kernel sequencing.
// No device memory is allocated here and nothing synchronises except heart_get_status.
#include <math.h>

#include <mutex>
#include <stdio.h>
#include <string.h>

#include "common.cuh"

using namespace heart;

namespace {

thread_local char g_errbuf[256] = "";
thread_local int g_launches = 0;

int cuda_fail(cudaError_t e, const char *where) {
  snprintf(g_errbuf, sizeof g_errbuf, "CUDA error in %s: %s", where, cudaGetErrorString(e));
  return HEART_ERR_CUDA;
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

// Validates the shape part of a config and derives the geometry. Returns HEART_OK or an error.
int heart::make_geom(const heart_config *c, Geom *g) {
  if (c == nullptr) return HEART_ERR_INVALID;
  if (c->B <= 0 || c->H <= 0 || c->N <= 0) return HEART_ERR_INVALID;
  if (c->D != kD) return HEART_ERR_UNSUPPORTED;
  if (c->block != 64 && c->block != 128) return HEART_ERR_UNSUPPORTED;
  g->B = c->B;
  g->H = c->H;
  g->R = c->B * c->H;
  g->N = c->N;
  g->block = c->block;
  g->nb = (c->N + c->block - 1) / c->block;
  if (g->nb > HEART_MAX_BLOCKS) return HEART_ERR_UNSUPPORTED;
  g->W = (g->nb + 31) / 32;
  if (c->stride_b == 0 && c->stride_h == 0 && c->stride_n == 0) {
    g->sn = kD;
    g->sh = (long long)c->N * kD;
    g->sb = g->sh * c->H;
  } else {
    g->sb = c->stride_b;
    g->sh = c->stride_h;
    g->sn = c->stride_n;
    if (g->sn < kD || g->sh <= 0 || g->sb <= 0) return HEART_ERR_INVALID;
    if ((g->sn % 8) || (g->sh % 8) || (g->sb % 8)) return HEART_ERR_INVALID;
  }
  g->idx_stride = c->idx_stride;
  if (g->idx_stride < g->nb) return HEART_ERR_INVALID;
  g->scale = (c->scale > 0.0) ? c->scale : 1.0 / sqrt((double)kD);
  g->gate_lo = c->gate_lo;
  g->gate_hi = c->gate_hi;
  if (isnan(g->gate_lo) || isnan(g->gate_hi)) return HEART_ERR_INVALID;
  g->flags = c->flags;
  set_chunks(*g);
  return HEART_OK;
}

namespace {

bool state_ok(const heart_state *st) {
  return st && st->anchor_q && st->anchor_k && st->has_anchor && st->mask_bits && st->kv_idx && st->kv_cnt;
}

// Mask prediction inside a layer-step (the refresh flags are the ones the decision kernel just wrote).
cudaError_t predict_for_step(const Geom &g, const Workspace &w, const void *Q, const void *K, const double *tau,
                             heart_state st, cudaStream_t s) {
  if (g.flags & HEART_ESTIMATOR_ANTIDIAG) {
    cudaError_t e = launch_antidiag_scores(g, w, Q, K, w.refresh, s, &g_launches);
    if (e != cudaSuccess) return e;
    return launch_top_p(g, w, tau, w.refresh, st, s, &g_launches, 0);
  }
  return launch_predict_mask(g, w, tau, w.refresh, st, s, &g_launches);
}

__global__ void fill_dense_outputs_kernel(int R, double *drift_out, uint8_t *refresh_out, uint8_t *refresh_ws) {
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r < R) {
    if (drift_out) drift_out[r] = __longlong_as_double(0x7ff0000000000000LL);
    if (refresh_out) refresh_out[r] = 0;
    refresh_ws[r] = 0;
  }
}

}  // namespace

extern "C" {

size_t heart_workspace_bytes(const heart_config *cfg) {
  Geom g;
  if (make_geom(cfg, &g) != HEART_OK) return 0;
  return carve(g, nullptr).bytes;
}

size_t heart_drift_workspace_bytes(const heart_config *cfg) {
  Geom g;
  if (make_geom(cfg, &g) != HEART_OK) return 0;
  return carve(g, nullptr).bytes_drift;
}

int heart_state_reset(const heart_config *cfg, heart_state *st, heart_stream_t stream) {
  Geom g;
  int rc = make_geom(cfg, &g);
  if (rc != HEART_OK) return rc;
  if (!state_ok(st)) return HEART_ERR_INVALID;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaError_t e = cudaMemsetAsync(st->has_anchor, 0, (size_t)g.R, s);
  if (e != cudaSuccess) return cuda_fail(e, "heart_state_reset");
  e = cudaMemsetAsync(st->kv_cnt, 0, sizeof(int32_t) * (size_t)g.R * g.nb, s);
  if (e != cudaSuccess) return cuda_fail(e, "heart_state_reset");
  return HEART_OK;
}

int heart_drift(const heart_config *cfg, const void *Q, const void *K, const double *delta,
                heart_state *st, double *drift_out, uint8_t *refresh_out, void *workspace,
                heart_stream_t stream) {
  Geom g;
  int rc = make_geom(cfg, &g);
  if (rc != HEART_OK) return rc;
  if (!Q || !K || !delta || !workspace || !state_ok(st)) return HEART_ERR_INVALID;
  if (!aligned16(Q) || !aligned16(K) || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return HEART_ERR_INVALID;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  Workspace w = carve(g, workspace);
  g_launches = 0;
  cudaError_t e = launch_block_sums(g, Q, K, w, s, &g_launches);
  if (e != cudaSuccess) return cuda_fail(e, "block_sums");
  e = launch_decide(g, w, delta, *st, drift_out, refresh_out, s, &g_launches);
  if (e != cudaSuccess) return cuda_fail(e, "decide");
  return HEART_OK;
}

int heart_predict_mask(const heart_config *cfg, const void *Q, const void *K, const double *tau,
                       const uint8_t *refresh, heart_state *st, void *workspace, heart_stream_t stream) {
  Geom g;
  int rc = make_geom(cfg, &g);
  if (rc != HEART_OK) return rc;
  if (!Q || !K || !tau || !workspace || !state_ok(st)) return HEART_ERR_INVALID;
  if (!aligned16(Q) || !aligned16(K) || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return HEART_ERR_INVALID;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  Workspace w = carve(g, workspace);
  g_launches = 0;
  cudaError_t e;
  unsigned long long expect_sig = 0;
  if (g.flags & HEART_ESTIMATOR_ANTIDIAG) {
    // this estimator works on the tokens themselves: no block means needed
    e = launch_antidiag_scores(g, w, Q, K, refresh, s, &g_launches);
    if (e != cudaSuccess) return cuda_fail(e, "antidiag_scores");
    e = launch_top_p(g, w, tau, refresh, *st, s, &g_launches, 0);
    if (e != cudaSuccess) return cuda_fail(e, "top_p");
    return HEART_OK;
  }
  if (g.flags & HEART_BLOCK_MEANS_VALID) {
    // the caller vouches that a heart_drift (or heart_predict_mask) on these very tensors left the block
    // means in this workspace: no second pass over Q and K; the kernels verify the workspace's signature
    expect_sig = block_means_signature(g, Q, K);
  } else {
    e = launch_block_sums(g, Q, K, w, s, &g_launches);
    if (e != cudaSuccess) return cuda_fail(e, "block_sums");
  }
  e = launch_predict_mask(g, w, tau, refresh, *st, s, &g_launches, expect_sig);
  if (e != cudaSuccess) return cuda_fail(e, "predict_mask");
  return HEART_OK;
}

int heart_block_sparse_attn(const heart_config *cfg, const void *Q, const void *K, const void *V,
                            const int32_t *kv_idx, const int32_t *kv_cnt, void *O, float *lse,
                            void *workspace, heart_stream_t stream) {
  Geom g;
  int rc = make_geom(cfg, &g);
  if (rc != HEART_OK) return rc;
  const bool dense = (g.flags & HEART_FORCE_DENSE) != 0;
  if (!Q || !K || !V || !O || !workspace) return HEART_ERR_INVALID;
  if (!dense && (!kv_idx || !kv_cnt)) return HEART_ERR_INVALID;
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) ||
      (reinterpret_cast<uintptr_t>(workspace) & 255u))
    return HEART_ERR_INVALID;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  Workspace w = carve(g, workspace);
  g_launches = 0;
  cudaError_t e = launch_attention(g, Q, K, V, kv_idx, kv_cnt, dense, O, lse, w.status, w.order, s, &g_launches);
  if (e != cudaSuccess) return cuda_fail(e, "attention");
  return HEART_OK;
}

int heart_step(const heart_config *cfg, const void *Q, const void *K, const void *V,
               const double *delta, const double *tau, heart_state *st, void *O, float *lse,
               double *drift_out, uint8_t *refresh_out, void *workspace, heart_stream_t stream) {
  Geom g;
  int rc = make_geom(cfg, &g);
  if (rc != HEART_OK) return rc;
  if (!Q || !K || !V || !O || !delta || !tau || !workspace || !state_ok(st)) return HEART_ERR_INVALID;
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) ||
      (reinterpret_cast<uintptr_t>(workspace) & 255u))
    return HEART_ERR_INVALID;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  Workspace w = carve(g, workspace);
  g_launches = 0;
  cudaError_t e;
  if (g.flags & HEART_FORCE_DENSE) {
    fill_dense_outputs_kernel<<<(g.R + 127) / 128, 128, 0, s>>>(g.R, drift_out, refresh_out, w.refresh);
    ++g_launches;
    if ((e = cudaGetLastError()) != cudaSuccess) return cuda_fail(e, "fill_dense_outputs");
    e = launch_attention(g, Q, K, V, nullptr, nullptr, true, O, lse, w.status, w.order, s, &g_launches);
    if (e != cudaSuccess) return cuda_fail(e, "attention");
    return HEART_OK;
  }
  e = launch_block_sums(g, Q, K, w, s, &g_launches);
  if (e != cudaSuccess) return cuda_fail(e, "block_sums");
  e = launch_decide(g, w, delta, *st, drift_out, refresh_out, s, &g_launches);
  if (e != cudaSuccess) return cuda_fail(e, "decide");
  e = predict_for_step(g, w, Q, K, tau, *st, s);
  if (e != cudaSuccess) return cuda_fail(e, "predict_mask");
  e = launch_attention(g, Q, K, V, st->kv_idx, st->kv_cnt, false, O, lse, w.status, w.order, s, &g_launches);
  if (e != cudaSuccess) return cuda_fail(e, "attention");
  return HEART_OK;
}

namespace {

// Streams and events of heart_step_host, created on first use on each device and kept.
constexpr int kHostGroups = 16;  // head groups the V copy, the attention and the O copy are pipelined over
struct HostPipe {
  bool ready = false;
  cudaStream_t s_in = nullptr, s_out = nullptr;
  cudaEvent_t ev_qk = nullptr, ev_join = nullptr, ev_v[kHostGroups] = {}, ev_o[kHostGroups] = {};
};
constexpr int kMaxPipeDevices = 64;
std::mutex g_pipe_mu;
HostPipe g_pipe[kMaxPipeDevices];

cudaError_t pipe_for_current_device(HostPipe **out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxPipeDevices) return cudaErrorInvalidDevice;
  HostPipe &p = g_pipe[dev];
  if (!p.ready) {
    if ((e = cudaStreamCreateWithFlags(&p.s_in, cudaStreamNonBlocking)) != cudaSuccess) return e;
    if ((e = cudaStreamCreateWithFlags(&p.s_out, cudaStreamNonBlocking)) != cudaSuccess) return e;
    if ((e = cudaEventCreateWithFlags(&p.ev_qk, cudaEventDisableTiming)) != cudaSuccess) return e;
    if ((e = cudaEventCreateWithFlags(&p.ev_join, cudaEventDisableTiming)) != cudaSuccess) return e;
    for (int i = 0; i < kHostGroups; ++i) {
      if ((e = cudaEventCreateWithFlags(&p.ev_v[i], cudaEventDisableTiming)) != cudaSuccess) return e;
      if ((e = cudaEventCreateWithFlags(&p.ev_o[i], cudaEventDisableTiming)) != cudaSuccess) return e;
    }
    p.ready = true;
  }
  *out = &p;
  return cudaSuccess;
}

}  // namespace

// Pipeline: Q and K go up on `stream`, then drift and mask prediction run there while V goes up on
// an internal stream, one group of heads at a time; the attention of a head group starts when its V
// has landed and its O goes down on a second internal stream while the next group computes.  `stream`
// finally waits for the last download, so everything is ordered before later work on `stream`.
int heart_step_host(const heart_config *cfg, const void *Q_host, const void *K_host, const void *V_host,
                    const double *delta, const double *tau, heart_state *st, void *O_host,
                    double *drift_host, uint8_t *refresh_host, void *Q_dev, void *K_dev, void *V_dev,
                    void *O_dev, void *workspace, heart_stream_t stream) {
  Geom g;
  int rc = make_geom(cfg, &g);
  if (rc != HEART_OK) return rc;
  if (cfg->stride_b != 0 || cfg->stride_h != 0 || cfg->stride_n != 0) return HEART_ERR_INVALID;
  if (!Q_host || !K_host || !V_host || !O_host || !Q_dev || !K_dev || !V_dev || !O_dev || !delta || !tau ||
      !workspace || !state_ok(st))
    return HEART_ERR_INVALID;
  if (!aligned16(Q_dev) || !aligned16(K_dev) || !aligned16(V_dev) || !aligned16(O_dev) ||
      (reinterpret_cast<uintptr_t>(workspace) & 255u))
    return HEART_ERR_INVALID;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  Workspace w = carve(g, workspace);
  std::lock_guard<std::mutex> lock(g_pipe_mu);  // the events are shared by the calls on a device
  HostPipe *pp = nullptr;
  cudaError_t e = pipe_for_current_device(&pp);
  if (e != cudaSuccess) return cuda_fail(e, "heart_step_host (streams)");
  const size_t head_bytes = sizeof(uint16_t) * (size_t)g.N * kD;
  const size_t bytes = head_bytes * g.R;
  g_launches = 0;
  e = cudaMemcpyAsync(Q_dev, Q_host, bytes, cudaMemcpyHostToDevice, s);
  if (e == cudaSuccess) e = cudaMemcpyAsync(K_dev, K_host, bytes, cudaMemcpyHostToDevice, s);
  if (e == cudaSuccess) e = cudaEventRecord(pp->ev_qk, s);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(pp->s_in, pp->ev_qk, 0);  // V queues behind Q and K
  if (e != cudaSuccess) return cuda_fail(e, "heart_step_host (host to device)");
  const bool dense = (g.flags & HEART_FORCE_DENSE) != 0;
  if (dense) {
    fill_dense_outputs_kernel<<<(g.R + 127) / 128, 128, 0, s>>>(g.R, w.drift, nullptr, w.refresh);
    ++g_launches;
    if ((e = cudaGetLastError()) != cudaSuccess) return cuda_fail(e, "fill_dense_outputs");
  } else {
    e = launch_block_sums(g, Q_dev, K_dev, w, s, &g_launches);
    if (e != cudaSuccess) return cuda_fail(e, "block_sums");
    e = launch_decide(g, w, delta, *st, w.drift, nullptr, s, &g_launches);
    if (e != cudaSuccess) return cuda_fail(e, "decide");
    e = predict_for_step(g, w, Q_dev, K_dev, tau, *st, s);
    if (e != cudaSuccess) return cuda_fail(e, "predict_mask");
  }
  const int groups = g.H < kHostGroups ? g.H : kHostGroups;
  for (int gi = 0; gi < groups; ++gi) {
    const int h0 = (int)((long long)g.H * gi / groups), h1 = (int)((long long)g.H * (gi + 1) / groups);
    for (int b = 0; b < g.B && e == cudaSuccess; ++b) {  // one copy per batch entry: its heads h0..h1 are contiguous
      const size_t off = ((size_t)b * g.H + h0) * head_bytes;
      e = cudaMemcpyAsync(static_cast<char *>(V_dev) + off, static_cast<const char *>(V_host) + off,
                          head_bytes * (h1 - h0), cudaMemcpyHostToDevice, pp->s_in);
    }
    if (e == cudaSuccess) e = cudaEventRecord(pp->ev_v[gi], pp->s_in);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(s, pp->ev_v[gi], 0);
    if (e != cudaSuccess) return cuda_fail(e, "heart_step_host (host to device)");
    e = launch_attention(g, Q_dev, K_dev, V_dev, dense ? nullptr : st->kv_idx, dense ? nullptr : st->kv_cnt, dense,
                         O_dev, nullptr, w.status, w.order, s, &g_launches, h0, h1 - h0);
    if (e != cudaSuccess) return cuda_fail(e, "attention");
    e = cudaEventRecord(pp->ev_o[gi], s);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(pp->s_out, pp->ev_o[gi], 0);
    for (int b = 0; b < g.B && e == cudaSuccess; ++b) {
      const size_t off = ((size_t)b * g.H + h0) * head_bytes;
      e = cudaMemcpyAsync(static_cast<char *>(O_host) + off, static_cast<const char *>(O_dev) + off,
                          head_bytes * (h1 - h0), cudaMemcpyDeviceToHost, pp->s_out);
    }
    if (e != cudaSuccess) return cuda_fail(e, "heart_step_host (device to host)");
  }
  // drift and refresh were final before the first attention launch: ev_o[0] on s_out covers them
  if (drift_host)
    e = cudaMemcpyAsync(drift_host, w.drift, sizeof(double) * (size_t)g.R, cudaMemcpyDeviceToHost, pp->s_out);
  if (e == cudaSuccess && refresh_host)
    e = cudaMemcpyAsync(refresh_host, w.refresh, (size_t)g.R, cudaMemcpyDeviceToHost, pp->s_out);
  if (e == cudaSuccess) e = cudaEventRecord(pp->ev_join, pp->s_out);
  if (e == cudaSuccess) e = cudaStreamWaitEvent(s, pp->ev_join, 0);
  if (e != cudaSuccess) return cuda_fail(e, "heart_step_host (device to host)");
  return HEART_OK;
}

int heart_full_token_drift(const heart_config *cfg, const void *Qa, const void *Ka, const void *Qb,
                           const void *Kb, double *drift_out, void *workspace, heart_stream_t stream) {
  Geom g;
  int rc = make_geom(cfg, &g);
  if (rc != HEART_OK) return rc;
  if (!Qa || !Ka || !Qb || !Kb || !drift_out || !workspace) return HEART_ERR_INVALID;
  if (!aligned16(Qa) || !aligned16(Ka) || !aligned16(Qb) || !aligned16(Kb) ||
      (reinterpret_cast<uintptr_t>(workspace) & 255u))
    return HEART_ERR_INVALID;
  Workspace w = carve(g, workspace);
  int rows = 0;
  const size_t need = (size_t)g.R * token_drift_chunks(g, &rows);  // partials live in the block-sum area
  if (need > 2 * (size_t)g.R * g.nb * kD) return HEART_ERR_INVALID;
  g_launches = 0;
  // the partials overwrite the block means: the workspace no longer holds any
  cudaError_t e = cudaMemsetAsync(w.status + kStatusSigWord, 0, 8, static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return cuda_fail(e, "token_drift");
  e = launch_token_drift(g, Qa, Ka, Qb, Kb, w.bmean, drift_out, static_cast<cudaStream_t>(stream), &g_launches);
  if (e != cudaSuccess) return cuda_fail(e, "token_drift");
  return HEART_OK;
}

int heart_mask_iou(const heart_config *cfg, const uint32_t *mask_a, const uint32_t *mask_b,
                   double *iou_out, int64_t *counts_out, heart_stream_t stream) {
  Geom g;
  int rc = make_geom(cfg, &g);
  if (rc != HEART_OK) return rc;
  if (!mask_a || !mask_b || !iou_out) return HEART_ERR_INVALID;
  g_launches = 0;
  cudaError_t e = launch_mask_iou(g, mask_a, mask_b, iou_out, reinterpret_cast<long long *>(counts_out),
                                  static_cast<cudaStream_t>(stream), &g_launches);
  if (e != cudaSuccess) return cuda_fail(e, "mask_iou");
  return HEART_OK;
}

size_t heart_band_error_workspace_bytes(int32_t C, int32_t T, int32_t H, int32_t W) {
  if (C < 1 || T < 1 || H < 1 || W < 1 || (long long)C * T * H * W > (1LL << 31)) return 0;
  return band_error_workspace_bytes(C, T, H, W);
}

int heart_band_error(const float *y_sparse, const float *y_dense, int32_t C, int32_t T, int32_t H, int32_t W,
                     const double *weights, double eps, double *out, void *workspace, heart_stream_t stream) {
  if (heart_band_error_workspace_bytes(C, T, H, W) == 0) return HEART_ERR_INVALID;
  if (!y_sparse || !y_dense || !weights || !out || !workspace || !(eps >= 0.0)) return HEART_ERR_INVALID;
  if (reinterpret_cast<uintptr_t>(workspace) & 255u) return HEART_ERR_INVALID;
  g_launches = 0;
  cudaError_t e = launch_band_error(y_sparse, y_dense, C, T, H, W, weights, eps, out, workspace,
                                    static_cast<cudaStream_t>(stream), &g_launches);
  if (e != cudaSuccess) return cuda_fail(e, "band_error");
  return HEART_OK;
}

int heart_get_status(void *workspace, heart_stream_t stream, int32_t *code_out) {
  if (!workspace || !code_out) return HEART_ERR_INVALID;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int32_t words[2] = {0, 0};
  cudaError_t e = cudaMemcpyAsync(words, workspace, sizeof words, cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) return cuda_fail(e, "heart_get_status");
  *code_out = words[0];
  if (words[0] != 0) {
    e = cudaMemsetAsync(workspace, 0, sizeof words, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return cuda_fail(e, "heart_get_status");
  }
  return HEART_OK;
}

const char *heart_strerror(int code) {
  switch (code) {
    case HEART_OK: return "ok";
    case HEART_ERR_INVALID: return "invalid argument (null pointer, size, stride or alignment)";
    case HEART_ERR_UNSUPPORTED: return "unsupported shape (head_dim must be 128, block 64 or 128, at most 1024 blocks)";
    case HEART_ERR_CUDA: return g_errbuf[0] ? g_errbuf : "CUDA error";
    case HEART_ERR_TOO_LARGE: return "shape needs more scratch than the built-in HEART_STATIC_SCRATCH_BYTES array holds";
    case HEART_ERR_INFEASIBLE: return "no assignment of one candidate per head meets the sparsity budget";
    case HEART_ERR_DEVICE_CHECK: return "device-side check failed (index-list entry out of range or a bounded wait ran out)";
    default: return "unknown code";
  }
}

int heart_last_launch_count(void) { return g_launches; }

}  // extern "C"
