// Streaming statistics of one layer-step: per-block means of Q and K in a single pass over HBM
// (token-mean pooling of Algorithm 1 line 1 and the block pooling of the mask predictor share the
// pass), then the mean-pooled L1 drift, the refresh-or-reuse decision, the layer gate and the
// anchor update (Eq. mean-pooled drift; Algorithm 1; layer-level gating of the TMR section).
//
// Numerics: each thread adds at most block/16 (4 or 8) bf16 values in fp32 -- exact unless an
// addend lies more than 2^16 below the running sum -- and everything after that (the 16-way
// combine inside the CTA, the sum over the CTA's blocks, the sum over CTAs, means, drift) is fp64 in
// an order fixed by the shape alone, so the result is bit-reproducible run to run: identical inputs
// give a drift of exactly 0.
#include "common.cuh"

namespace heart {

__device__ __forceinline__ uint4 ldg_nc_v4(const void *p) {
  uint4 v;
  asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// One CTA per (chunk of consecutive blocks, head row r, tensor z).  256 threads: 16 row groups x 16
// chunks of 8 dims.  The 128-bit loads of block i+1 are issued before block i is reduced, so every
// thread keeps BLOCK/16 loads in flight across the shared-memory combine; the combine is double-
// buffered (fp32, the precision the partials have anyway), so a block costs one barrier.
template <int BLOCK>
__global__ void __launch_bounds__(256) block_sums_kernel(const uint16_t *__restrict__ Q,
                                                         const uint16_t *__restrict__ K, long long sb,
                                                         long long sh, long long sn, int H, int N,
                                                         int nb, int bpc, double *__restrict__ bmean,
                                                         double *__restrict__ psum) {
  constexpr int ITERS = BLOCK / 16;
  const int chunk = blockIdx.x, r = blockIdx.y, z = blockIdx.z, R = gridDim.y;
  const int c = threadIdx.x & 15, g = threadIdx.x >> 4;
  const uint16_t *X = (z ? K : Q) + (long long)(r / H) * sb + (long long)(r % H) * sh + c * 8;
  const int i0 = chunk * bpc, i1 = min(nb, i0 + bpc);
  __shared__ float sm[2][16][kD];

  uint4 cur[ITERS], nxt[ITERS];
  auto load_block = [&](int I, uint4 (&v)[ITERS]) {
    const int rows = min(BLOCK, N - I * BLOCK);
    const uint16_t *base = X + (long long)I * BLOCK * sn;
#pragma unroll
    for (int it = 0; it < ITERS; ++it) {
      const int row = it * 16 + g;
      v[it] = (row < rows) ? ldg_nc_v4(base + (long long)row * sn) : make_uint4(0, 0, 0, 0);
    }
  };
  // threads 0..127: sum of dim threadIdx.x over the 16 row groups of block I (staged in sm[buf])
  auto finish_block = [&](int I, int buf, double &total) {
    double s = 0.0;
#pragma unroll
    for (int k = 0; k < 16; ++k) s += (double)sm[buf][k][threadIdx.x];
    // the pooled mean of the block (what the mask predictor contracts); a full block divides by a
    // power of two, exactly
    const int rows = min(BLOCK, N - I * BLOCK);
    bmean[(((size_t)z * R + r) * nb + I) * kD + threadIdx.x] = (rows == BLOCK) ? s * (1.0 / BLOCK) : s / (double)rows;
    total += s;
  };
  load_block(i0, cur);
  double total = 0.0;  // threads 0..127: running token sum of dim threadIdx.x over this CTA's blocks
  int buf = 0;
  for (int I = i0; I < i1; ++I, buf ^= 1) {
    if (I + 1 < i1) load_block(I + 1, nxt);
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int it = 0; it < ITERS; ++it) {
      acc[0] += bf16_lo(cur[it].x);
      acc[1] += bf16_hi(cur[it].x);
      acc[2] += bf16_lo(cur[it].y);
      acc[3] += bf16_hi(cur[it].y);
      acc[4] += bf16_lo(cur[it].z);
      acc[5] += bf16_hi(cur[it].z);
      acc[6] += bf16_lo(cur[it].w);
      acc[7] += bf16_hi(cur[it].w);
    }
    // sm[buf] was last read two blocks ago, before the barrier of the previous block
    *reinterpret_cast<float4 *>(&sm[buf][g][c * 8]) = make_float4(acc[0], acc[1], acc[2], acc[3]);
    *reinterpret_cast<float4 *>(&sm[buf][g][c * 8 + 4]) = make_float4(acc[4], acc[5], acc[6], acc[7]);
    __syncthreads();
    if (threadIdx.x < kD) finish_block(I, buf, total);
#pragma unroll
    for (int it = 0; it < ITERS; ++it) cur[it] = nxt[it];
  }
  if (threadIdx.x < kD) psum[(((size_t)z * R + r) * gridDim.x + chunk) * kD + threadIdx.x] = total;
}

// Decision inputs that the last CTA of mean_drift_kernel needs.
struct DecideArgs {
  int B, H;
  const double *delta;
  double gate_lo, gate_hi;
  unsigned flags;
  double *anchor_q, *anchor_k;
  uint8_t *has_anchor, *refresh_ws;
  double *drift_out;
  uint8_t *refresh_out;
  int *ticket;  // zero between launches
};

// Head-wise rule, gate over the H heads of batch entry b, anchor update.  One CTA, any block size.
// `part` and `mean` were written by other CTAs of the same launch: read them past L1.
__device__ void decide_batch_entry(int b, int R, const double *part, const double *mean, const DecideArgs &a,
                                   uint8_t *sh_flags /* [2*H] */, int *cnt /* shared */) {
  const int H = a.H;
  if (threadIdx.x == 0) *cnt = 0;
  __syncthreads();
  for (int h = threadIdx.x; h < H; h += blockDim.x) {
    const int r = b * H + h;
    const bool had = a.has_anchor[r] != 0;
    const double dr = had ? (__ldcg(&part[r]) + __ldcg(&part[R + r])) : __longlong_as_double(0x7ff0000000000000LL);
    bool rf = !had || (dr > a.delta[r]);
    if (a.flags & HEART_FORCE_REFRESH) rf = true;
    sh_flags[h] = rf;
    sh_flags[H + h] = had;
    if (a.drift_out) a.drift_out[r] = dr;
    if (rf) atomicAdd(cnt, 1);
  }
  __syncthreads();
  const double f = (double)*cnt / (double)H;
  for (int h = threadIdx.x; h < H; h += blockDim.x) {
    bool rf = sh_flags[h];
    if (f < a.gate_lo) {
      if (sh_flags[H + h]) rf = false;
    } else if (f > a.gate_hi) {
      rf = true;
    }
    sh_flags[h] = rf;
    const int r = b * H + h;
    a.refresh_ws[r] = rf;
    if (a.refresh_out) a.refresh_out[r] = rf;
    if (rf) a.has_anchor[r] = 1;
  }
  __syncthreads();
  for (int e = threadIdx.x; e < H * kD; e += blockDim.x) {
    const int h = e / kD, r = b * H + h;
    if (sh_flags[h]) {
      a.anchor_q[(size_t)r * kD + (e % kD)] = __ldcg(&mean[(size_t)r * kD + (e % kD)]);
      a.anchor_k[(size_t)r * kD + (e % kD)] = __ldcg(&mean[((size_t)R + r) * kD + (e % kD)]);
    }
  }
  __syncthreads();
}

// One CTA per (head row r, tensor z), 1024 threads = 8 ranges of partial sums x 128 dims.
// mean[z][r][d] = (sum over the per-CTA partials, ascending) / N;  part[z][r] = sum_d |anchor - mean|.
// The CTA that finishes last (a ticket counter) then takes the decisions of Algorithm 1 for every
// batch entry, so drift and decision are one launch.
__global__ void __launch_bounds__(1024) mean_drift_kernel(const double *__restrict__ psum, int R, int N,
                                                          int nchunks, double *__restrict__ mean,
                                                          double *__restrict__ part, const DecideArgs a) {
  extern __shared__ uint8_t sh_flags[];  // [2*H]: decision, had_anchor
  const int r = blockIdx.x, z = blockIdx.y;
  const int d = threadIdx.x & (kD - 1), grp = threadIdx.x >> 7;  // 8 groups
  const int per = (nchunks + 7) / 8;
  const int i0 = grp * per, i1 = min(nchunks, i0 + per);
  const double *src = psum + ((size_t)z * R + r) * nchunks * kD + d;
  double s = 0.0;
#pragma unroll 8
  for (int i = i0; i < i1; ++i) s += src[(size_t)i * kD];
  __shared__ double sm[8][kD];
  __shared__ double red[kD];
  __shared__ int last, cnt;
  sm[grp][d] = s;
  __syncthreads();
  if (threadIdx.x < kD) {
    double t = 0.0;
#pragma unroll
    for (int k = 0; k < 8; ++k) t += sm[k][d];
    const double m = t / (double)N;
    mean[((size_t)z * R + r) * kD + d] = m;
    const double anc = (z ? a.anchor_k : a.anchor_q)[(size_t)r * kD + d];
    red[d] = fabs(anc - m);
  }
  __syncthreads();
  for (int w = kD / 2; w > 0; w >>= 1) {  // fixed-shape tree: deterministic
    if (threadIdx.x < w) red[threadIdx.x] += red[threadIdx.x + w];
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    part[(size_t)z * R + r] = red[0];
    __threadfence();
    last = (atomicAdd(a.ticket, 1) == (int)(gridDim.x * gridDim.y) - 1);
  }
  __syncthreads();
  if (!last) return;
  // Every other CTA has read the old anchors and published its mean and drift part.
  __threadfence();
  for (int b = 0; b < a.B; ++b) decide_batch_entry(b, R, part, mean, a, sh_flags, &cnt);
  if (threadIdx.x == 0) *a.ticket = 0;
}

cudaError_t launch_block_sums(const Geom &g, const void *Q, const void *K, const Workspace &w,
                              cudaStream_t s, int *launches) {
  dim3 grid(g.nchunks, g.R, 2);
  const uint16_t *q = static_cast<const uint16_t *>(Q), *k = static_cast<const uint16_t *>(K);
  if (g.block == 64)
    block_sums_kernel<64><<<grid, 256, 0, s>>>(q, k, g.sb, g.sh, g.sn, g.H, g.N, g.nb, g.bpc, w.bmean, w.psum);
  else
    block_sums_kernel<128><<<grid, 256, 0, s>>>(q, k, g.sb, g.sh, g.sn, g.H, g.N, g.nb, g.bpc, w.bmean, w.psum);
  ++*launches;
  return cudaGetLastError();
}

cudaError_t launch_decide(const Geom &g, const Workspace &w, const double *delta, heart_state st,
                          double *drift_out, uint8_t *refresh_out, cudaStream_t s, int *launches) {
  DecideArgs a;
  a.B = g.B;
  a.H = g.H;
  a.delta = delta;
  a.gate_lo = g.gate_lo;
  a.gate_hi = g.gate_hi;
  a.flags = g.flags;
  a.anchor_q = st.anchor_q;
  a.anchor_k = st.anchor_k;
  a.has_anchor = st.has_anchor;
  a.refresh_ws = w.refresh;
  a.drift_out = drift_out;
  a.refresh_out = refresh_out;
  a.ticket = w.status + 8;
  mean_drift_kernel<<<dim3(g.R, 2), 1024, 2 * g.H, s>>>(w.psum, g.R, g.N, g.nchunks, w.mean, w.part, a);
  ++*launches;
  return cudaGetLastError();
}

}  // namespace heart
