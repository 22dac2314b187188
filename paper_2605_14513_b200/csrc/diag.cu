// Analysis quantities of the Temporal Mask Reuse study, computed on the device so that a caller can
// monitor a running model without a host round trip over the tensors:
//   - the full-token drift of Eq. full-token drift (the costly reference that the mean-pooled
//     drift approximates), one streaming pass over the current and the cached Q and K;
//   - the block-mask IoU between two steps (Observation I, adjacent-step mask similarity).
// Neither is on the layer-step path; nothing else in the library reads their results.
//
// Numerics of the drift: |a - b| of two bf16 values is formed in fp32 (exact unless the exponents
// differ by more than 16), the 16 differences of one thread's 128-bit chunks (8 of Q, 8 of K) are
// added in fp32, and every sum after that is fp64 in an order fixed by the shape alone.
#include "common.cuh"

namespace heart {

namespace {

__device__ __forceinline__ uint4 ldg_stream_v4(const void *p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

__device__ __forceinline__ float absdiff2(uint32_t a, uint32_t b) {
  const float lo = fabsf(__uint_as_float(a << 16) - __uint_as_float(b << 16));
  const float hi = fabsf(__uint_as_float(a & 0xffff0000u) - __uint_as_float(b & 0xffff0000u));
  return lo + hi;
}

__device__ __forceinline__ float absdiff8(const uint4 &a, const uint4 &b) {
  return (absdiff2(a.x, b.x) + absdiff2(a.y, b.y)) + (absdiff2(a.z, b.z) + absdiff2(a.w, b.w));
}

constexpr int kRowsPerIter = 16;  // 256 threads = 16 rows x 16 chunks of 8 dims

// One CTA per (range of rows_per_cta tokens, head row r).  Two rows per thread are in flight
// (8 independent 128-bit loads) before anything is reduced.
__global__ void __launch_bounds__(256) token_drift_partial_kernel(
    const uint16_t *__restrict__ Qa, const uint16_t *__restrict__ Ka, const uint16_t *__restrict__ Qb,
    const uint16_t *__restrict__ Kb, long long sb, long long sh, long long sn, int H, int N,
    int rows_per_cta, double *__restrict__ partial) {
  const int chunk = blockIdx.x, r = blockIdx.y;
  const int c = threadIdx.x & 15, g = threadIdx.x >> 4;
  const long long head = (long long)(r / H) * sb + (long long)(r % H) * sh + c * 8;
  const int i0 = chunk * rows_per_cta, i1 = min(N, i0 + rows_per_cta);
  double acc = 0.0;
  for (int row = i0 + g; row < i1; row += 2 * kRowsPerIter) {
    const long long o0 = head + (long long)row * sn;
    const bool two = row + kRowsPerIter < i1;
    const long long o1 = two ? o0 + (long long)kRowsPerIter * sn : o0;
    const uint4 qa0 = ldg_stream_v4(Qa + o0), qb0 = ldg_stream_v4(Qb + o0);
    const uint4 ka0 = ldg_stream_v4(Ka + o0), kb0 = ldg_stream_v4(Kb + o0);
    const uint4 qa1 = ldg_stream_v4(Qa + o1), qb1 = ldg_stream_v4(Qb + o1);
    const uint4 ka1 = ldg_stream_v4(Ka + o1), kb1 = ldg_stream_v4(Kb + o1);
    acc += (double)(absdiff8(qa0, qb0) + absdiff8(ka0, kb0));
    if (two) acc += (double)(absdiff8(qa1, qb1) + absdiff8(ka1, kb1));
  }
  __shared__ double red[256];
  red[threadIdx.x] = acc;
  __syncthreads();
  for (int w = 128; w > 0; w >>= 1) {  // fixed-shape tree: deterministic
    if (threadIdx.x < w) red[threadIdx.x] += red[threadIdx.x + w];
    __syncthreads();
  }
  if (threadIdx.x == 0) partial[(size_t)r * gridDim.x + chunk] = red[0];
}

// One CTA per head row: d[r] = (sum of the per-CTA partials) / N.
__global__ void __launch_bounds__(256) token_drift_final_kernel(const double *__restrict__ partial,
                                                                int nchunks, int N,
                                                                double *__restrict__ drift) {
  const int r = blockIdx.x;
  double s = 0.0;
  for (int i = threadIdx.x; i < nchunks; i += 256) s += partial[(size_t)r * nchunks + i];
  __shared__ double red[256];
  red[threadIdx.x] = s;
  __syncthreads();
  for (int w = 128; w > 0; w >>= 1) {
    if (threadIdx.x < w) red[threadIdx.x] += red[threadIdx.x + w];
    __syncthreads();
  }
  if (threadIdx.x == 0) drift[r] = red[0] / (double)N;
}

// One CTA per head row: popcounts of A&B and A|B over the nb*W mask words of the head.
__global__ void __launch_bounds__(256) mask_iou_kernel(const uint32_t *__restrict__ A,
                                                       const uint32_t *__restrict__ B, int words,
                                                       double *__restrict__ iou,
                                                       long long *__restrict__ counts) {
  const int r = blockIdx.x;
  const uint32_t *a = A + (size_t)r * words, *b = B + (size_t)r * words;
  unsigned long long inter = 0, uni = 0;
  for (int i = threadIdx.x; i < words; i += 256) {
    const uint32_t x = a[i], y = b[i];
    inter += __popc(x & y);
    uni += __popc(x | y);
  }
  __shared__ unsigned long long s_inter, s_uni;
  if (threadIdx.x == 0) s_inter = s_uni = 0;
  __syncthreads();
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    inter += __shfl_xor_sync(0xffffffffu, inter, o);
    uni += __shfl_xor_sync(0xffffffffu, uni, o);
  }
  if ((threadIdx.x & 31) == 0) {
    atomicAdd(&s_inter, inter);
    atomicAdd(&s_uni, uni);
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    iou[r] = s_uni ? (double)s_inter / (double)s_uni : 1.0;
    if (counts) {
      counts[2 * r] = (long long)s_inter;
      counts[2 * r + 1] = (long long)s_uni;
    }
  }
}

}  // namespace

int token_drift_chunks(const Geom &g, int *rows_per_cta) {
  int per_head = (HEART_CHUNK_TARGET + g.R - 1) / g.R;
  if (per_head < 1) per_head = 1;
  int rows = (g.N + per_head - 1) / per_head;
  rows = (rows + 2 * kRowsPerIter - 1) / (2 * kRowsPerIter) * (2 * kRowsPerIter);
  *rows_per_cta = rows;
  return (g.N + rows - 1) / rows;
}

cudaError_t launch_token_drift(const Geom &g, const void *Qa, const void *Ka, const void *Qb,
                               const void *Kb, double *partial, double *drift_out, cudaStream_t s,
                               int *launches) {
  int rows = 0;
  const int nchunks = token_drift_chunks(g, &rows);
  token_drift_partial_kernel<<<dim3(nchunks, g.R), 256, 0, s>>>(
      static_cast<const uint16_t *>(Qa), static_cast<const uint16_t *>(Ka),
      static_cast<const uint16_t *>(Qb), static_cast<const uint16_t *>(Kb), g.sb, g.sh, g.sn, g.H, g.N,
      rows, partial);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  ++*launches;
  token_drift_final_kernel<<<g.R, 256, 0, s>>>(partial, nchunks, g.N, drift_out);
  e = cudaGetLastError();
  if (e == cudaSuccess) ++*launches;
  return e;
}

cudaError_t launch_mask_iou(const Geom &g, const uint32_t *A, const uint32_t *B, double *iou,
                            long long *counts, cudaStream_t s, int *launches) {
  mask_iou_kernel<<<g.R, 256, 0, s>>>(A, B, g.nb * g.W, iou, counts);
  cudaError_t e = cudaGetLastError();
  if (e == cudaSuccess) ++*launches;
  return e;
}

}  // namespace heart
