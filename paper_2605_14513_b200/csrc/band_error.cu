// Frequency-aware velocity error of the offline calibration (Eq. calibration error; appendix
// "Frequency-aware velocity error"): the spectral energy of err = y_sparse - y_dense in four bands
// of its 3-D DFT over (t, y, x), weighted and divided by the energy of y_dense.
//
// No transform is formed.  Keeping the low frequencies of one axis is an orthogonal projection,
// L = F^H diag(low) F / n, a real symmetric circulant n x n matrix, and the bands are products of
// such projections and their complements, so by Parseval (with N = T*H*W, unnormalised DFT)
//   E_LL = N |L_t L_y L_x err|^2          E_LH = N |L_t err       - L_t L_y L_x err|^2
//   E_HL = N |L_y L_x err - L_t L_y L_x err|^2
//   E_HH = N |(err - L_t err) - (L_y L_x err - L_t L_y L_x err)|^2
// -- three small dense contractions along the axes and five sums of squares, all in fp64, every
// band from a direct norm (no subtraction of energies).  Off the layer-step path; sized for latents
// of a few million elements.
#include <math.h>

#include "common.cuh"

namespace heart {

namespace {

// L[d] for d = (i - j) mod n:  (1/n) sum over the low frequencies k of cos(2 pi k d / n);
// k is low iff its fftshift-ed index lies within floor(n/4) of the centre, i.e. min(k, n-k) <= n/4.
__global__ void projection_kernel(int n, double *__restrict__ L) {
  const int d = blockIdx.x * blockDim.x + threadIdx.x;
  if (d >= n) return;
  const int radius = n / 4;
  double s = 0.0;
  for (int k = 0; k < n; ++k) {
    if (min(k, n - k) > radius) continue;
    const long long kd = ((long long)k * d) % n;  // exact argument reduction
    s += cospi(2.0 * (double)kd / (double)n);
  }
  L[d] = s / (double)n;
}

// dst[..., i, ...] = sum_j L[(i - j) mod n] src[..., j, ...] along one axis of a [outer, n, inner] view.
// FROM_FLOATS: src is the pair (a, b) of fp32 tensors and the contraction runs over a - b.
template <bool FROM_FLOATS>
__global__ void __launch_bounds__(256) project_axis_kernel(const double *__restrict__ src, const float *__restrict__ a,
                                                           const float *__restrict__ b, const double *__restrict__ L,
                                                           long long outer, int n, long long inner,
                                                           double *__restrict__ dst) {
  const long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= outer * n * inner) return;
  const long long in = e % inner, i = (e / inner) % n, o = e / (inner * n);
  const long long base = o * n * inner + in;
  double s = 0.0;
  for (int j = 0; j < n; ++j) {
    const long long at = base + (long long)j * inner;
    const double v = FROM_FLOATS ? ((double)a[at] - (double)b[at]) : src[at];
    int d = (int)i - j;
    d += d < 0 ? n : 0;
    s = fma(L[d], v, s);
  }
  dst[e] = s;
}

// Per-CTA partial sums of squares of: err, L_t err - C, B - C, (err - L_t err) - (B - C), C, y_dense
// (B = L_y L_x err, C = L_t B), fixed-shape tree per CTA: deterministic.
__global__ void __launch_bounds__(256) band_partials_kernel(const float *__restrict__ ys, const float *__restrict__ yd,
                                                            const double *__restrict__ Z, const double *__restrict__ Bm,
                                                            const double *__restrict__ Cm, long long total,
                                                            double *__restrict__ partial) {
  double acc[5] = {0.0, 0.0, 0.0, 0.0, 0.0};  // LL, LH, HL, HH, |y_dense|^2
  for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (long long)gridDim.x * blockDim.x) {
    const double y = (double)yd[e], x = (double)ys[e] - y;
    const double z = Z[e], bb = Bm[e], c = Cm[e];
    const double lh = z - c, hl = bb - c, hh = (x - z) - hl;
    acc[0] = fma(c, c, acc[0]);
    acc[1] = fma(lh, lh, acc[1]);
    acc[2] = fma(hl, hl, acc[2]);
    acc[3] = fma(hh, hh, acc[3]);
    acc[4] = fma(y, y, acc[4]);
  }
  __shared__ double red[5][256];
#pragma unroll
  for (int q = 0; q < 5; ++q) red[q][threadIdx.x] = acc[q];
  __syncthreads();
  for (int w = 128; w > 0; w >>= 1) {
    if (threadIdx.x < w) {
#pragma unroll
      for (int q = 0; q < 5; ++q) red[q][threadIdx.x] += red[q][threadIdx.x + w];
    }
    __syncthreads();
  }
  if (threadIdx.x < 5) partial[(size_t)blockIdx.x * 5 + threadIdx.x] = red[threadIdx.x][0];
}

// out = (e, E_LL, E_LH, E_HL, E_HH, denominator)
__global__ void band_final_kernel(const double *__restrict__ partial, int nparts, double n_freq, double w0, double w1,
                                  double w2, double w3, double eps, double *__restrict__ out) {
  __shared__ double tot[5];
  if (threadIdx.x < 5) {
    double s = 0.0;
    for (int i = 0; i < nparts; ++i) s += partial[(size_t)i * 5 + threadIdx.x];
    tot[threadIdx.x] = s * n_freq;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const double denom = tot[4] + eps;
    out[0] = (w0 * tot[0] + w1 * tot[1] + w2 * tot[2] + w3 * tot[3]) / denom;
    out[1] = tot[0];
    out[2] = tot[1];
    out[3] = tot[2];
    out[4] = tot[3];
    out[5] = denom;
  }
}

constexpr int kBandParts = 148 * 4;

}  // namespace

size_t band_error_workspace_bytes(int C, int T, int H, int W) {
  const size_t n = (size_t)C * T * H * W;
  return align256(sizeof(double) * ((size_t)T + H + W)) + 4 * align256(sizeof(double) * n) +
         align256(sizeof(double) * kBandParts * 5);
}

cudaError_t launch_band_error(const float *ys, const float *yd, int C, int T, int H, int W, const double *weights,
                              double eps, double *out, void *workspace, cudaStream_t s, int *launches) {
  const long long n = (long long)C * T * H * W;
  char *p = static_cast<char *>(workspace);
  double *Lt = reinterpret_cast<double *>(p), *Lh = Lt + T, *Lw = Lh + H;
  p += align256(sizeof(double) * ((size_t)T + H + W));
  double *A = reinterpret_cast<double *>(p);
  p += align256(sizeof(double) * n);
  double *Bm = reinterpret_cast<double *>(p);
  p += align256(sizeof(double) * n);
  double *Cm = reinterpret_cast<double *>(p);
  p += align256(sizeof(double) * n);
  double *Z = reinterpret_cast<double *>(p);
  p += align256(sizeof(double) * n);
  double *partial = reinterpret_cast<double *>(p);
  projection_kernel<<<(T + 127) / 128, 128, 0, s>>>(T, Lt);
  projection_kernel<<<(H + 127) / 128, 128, 0, s>>>(H, Lh);
  projection_kernel<<<(W + 127) / 128, 128, 0, s>>>(W, Lw);
  const unsigned blocks = (unsigned)((n + 255) / 256);
  // A = L_x err ; B = L_y A ; C = L_t B ; Z = L_t err
  project_axis_kernel<true><<<blocks, 256, 0, s>>>(nullptr, ys, yd, Lw, (long long)C * T * H, W, 1, A);
  project_axis_kernel<false><<<blocks, 256, 0, s>>>(A, nullptr, nullptr, Lh, (long long)C * T, H, W, Bm);
  project_axis_kernel<false><<<blocks, 256, 0, s>>>(Bm, nullptr, nullptr, Lt, C, T, (long long)H * W, Cm);
  project_axis_kernel<true><<<blocks, 256, 0, s>>>(nullptr, ys, yd, Lt, C, T, (long long)H * W, Z);
  band_partials_kernel<<<kBandParts, 256, 0, s>>>(ys, yd, Z, Bm, Cm, n, partial);
  band_final_kernel<<<1, 32, 0, s>>>(partial, kBandParts, (double)T * H * W, weights[0], weights[1], weights[2],
                                    weights[3], eps, out);
  *launches += 9;
  return cudaGetLastError();
}

}  // namespace heart
