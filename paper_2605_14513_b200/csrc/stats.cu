// Streaming statistics of one layer-step: per-block means of Q and K in a single pass over HBM
// (token-mean pooling of Algorithm 1 line 1 and the block pooling of the mask predictor share the
// pass), then the mean-pooled L1 drift, the refresh-or-reuse decision, the layer gate and the
// anchor update (Eq. mean-pooled drift; Algorithm 1; layer-level gating of the TMR section).
//
// Numerics: each thread adds 4 bf16 values in fp32 -- exact unless an addend lies more than 2^16
// below the running sum -- and everything after that (the 16-way combine inside the CTA, the two
// halves of a 128-token block, the sum over the CTA's blocks, the sum over CTAs, means, drift) is fp64 in
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
// chunks of 8 dims.  The pass moves in units of 64 tokens (a 128-token block is two units): the
// 128-bit loads of unit u+1 are issued before unit u is reduced, so every thread keeps 4 loads in
// flight across the shared-memory combine; the combine is double-buffered (fp32, the precision the
// partials have anyway), so a unit costs one barrier.  48 registers: five CTAs per SM.
template <int BLOCK>
__global__ void __launch_bounds__(256, 5) block_sums_kernel(const uint16_t *__restrict__ Q,
                                                         const uint16_t *__restrict__ K, long long sb,
                                                         long long sh, long long sn, int H, int N,
                                                         int nb, int bpc, double *__restrict__ bmean,
                                                         double *__restrict__ psum,
                                                         unsigned long long *__restrict__ sig_word,
                                                         unsigned long long sig) {
  constexpr int UNIT = 64, ITERS = UNIT / 16, UPB = BLOCK / UNIT;  // units per block
  const int chunk = blockIdx.x, r = blockIdx.y, z = blockIdx.z, R = gridDim.y;
  const int c = threadIdx.x & 15, g = threadIdx.x >> 4;
  const uint16_t *X = (z ? K : Q) + (long long)(r / H) * sb + (long long)(r % H) * sh + c * 8;
  const int i0 = chunk * bpc, i1 = min(nb, i0 + bpc);
  const int u0 = i0 * UPB, u1 = i1 * UPB;
  __shared__ float sm[2][16][kD];
  // Launched with programmatic stream serialisation: when the kernel before it on the stream allows it
  // (the library's own kernels do), these CTAs are scheduled while that kernel drains and wait here until
  // it has completed and its writes are visible; after any other kernel this returns at once.
  pdl_wait();
  // The grid is one wave, so every CTA is past this point right after that: the follow-up kernel's CTAs
  // are scheduled as soon as the first CTAs of this one leave, and wait there for the rest.
  pdl_launch_dependents();
  if (chunk == 0 && r == 0 && z == 0 && threadIdx.x == 0) *sig_word = sig;  // whose means these are

  uint4 cur[ITERS], nxt[ITERS];
  auto load_unit = [&](int u, uint4 (&v)[ITERS]) {
    const int rows = min(UNIT, N - u * UNIT);  // <= 0 for the padded half of a ragged last block
    const uint16_t *base = X + (long long)u * UNIT * sn;
#pragma unroll
    for (int it = 0; it < ITERS; ++it) {
      const int row = it * 16 + g;
      v[it] = (row < rows) ? ldg_nc_v4(base + (long long)row * sn) : make_uint4(0, 0, 0, 0);
    }
  };
  load_unit(u0, cur);
  double total = 0.0;  // threads 0..127: running token sum of dim threadIdx.x over this CTA's blocks
  double blk = 0.0;    // threads 0..127: sum of the current block so far
  int buf = 0;
  for (int u = u0; u < u1; ++u, buf ^= 1) {
    if (u + 1 < u1) load_unit(u + 1, nxt);
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
    // sm[buf] was last read two units ago, before the barrier of the previous unit
    *reinterpret_cast<float4 *>(&sm[buf][g][c * 8]) = make_float4(acc[0], acc[1], acc[2], acc[3]);
    *reinterpret_cast<float4 *>(&sm[buf][g][c * 8 + 4]) = make_float4(acc[4], acc[5], acc[6], acc[7]);
    __syncthreads();
    if (threadIdx.x < kD) {  // sum of dim threadIdx.x over the 16 row groups of this unit
      double s = 0.0;
#pragma unroll
      for (int k = 0; k < 16; ++k) s += (double)sm[buf][k][threadIdx.x];
      blk += s;
      if ((u + 1) % UPB == 0) {
        // the pooled mean of the block (what the mask predictor contracts); a full block divides by a
        // power of two, exactly
        const int I = u / UPB, rows = min(BLOCK, N - I * BLOCK);
        bmean[(((size_t)z * R + r) * nb + I) * kD + threadIdx.x] =
            (rows == BLOCK) ? blk * (1.0 / BLOCK) : blk / (double)rows;
        total += blk;
        blk = 0.0;
      }
    }
#pragma unroll
    for (int it = 0; it < ITERS; ++it) cur[it] = nxt[it];
  }
  if (threadIdx.x < kD) psum[(((size_t)z * R + r) * gridDim.x + chunk) * kD + threadIdx.x] = total;
}

// Decision inputs of mean_drift_kernel.
struct DecideArgs {
  int B, H;
  const double *delta;
  double gate_lo, gate_hi;
  unsigned flags;
  double *anchor_q, *anchor_k;
  uint8_t *has_anchor, *refresh_ws, *pre_ws;
  double *drift_out;
  uint8_t *refresh_out;
  int *ticket;  // zero between launches (used only when the layer gate is on)
};

// Layer gate over the H heads of batch entry b and the anchor update of its refreshed heads.  One
// CTA, any block size.  The head-wise decisions, the drifts and the means were written by other CTAs
// of the same launch: read them past L1.
__device__ void gate_batch_entry(int b, int R, const double *mean, const DecideArgs &a,
                                 uint8_t *sh_flags /* [2*H] */, int *cnt /* shared */) {
  const int H = a.H;
  if (threadIdx.x == 0) *cnt = 0;
  __syncthreads();
  for (int h = threadIdx.x; h < H; h += blockDim.x) {
    const int r = b * H + h;
    const bool rf = __ldcg(&a.pre_ws[r]) != 0;
    sh_flags[h] = rf;
    sh_flags[H + h] = a.has_anchor[r] != 0;
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

// One CTA per head row r, 1024 threads = 2 tensors x 4 ranges of partial sums x 128 dims.
//   mean[z][r][d] = (sum over the per-CTA partials: four ascending ranges, then the four in order) / N
//   drift[r]      = sum_d |anchor_q - mean_q| + sum_d |anchor_k - mean_k|   (fixed-shape reductions)
// and the head-wise rule of Algorithm 1.  With the layer gate off (the usual case) that is the final
// decision and the CTA moves its own anchor; with the gate on, the CTA that finishes last (a ticket
// counter) applies the gate for every batch entry.
__global__ void __launch_bounds__(1024) mean_drift_kernel(const double *__restrict__ psum, int R, int N,
                                                          int nchunks, double *__restrict__ mean,
                                                          const DecideArgs a) {
  extern __shared__ uint8_t sh_flags[];  // [2*H]: decision, had_anchor (gate path)
  __shared__ double sm[2][4][kD];
  __shared__ double wsum[8];
  __shared__ int last, cnt, sh_rf;
  const int r = blockIdx.x;
  const int z = threadIdx.x >> 9, grp = (threadIdx.x >> 7) & 3, d = threadIdx.x & (kD - 1);
  const int per = (nchunks + 3) / 4;
  const int i0 = grp * per, i1 = min(nchunks, i0 + per);
  const double *src = psum + ((size_t)z * R + r) * nchunks * kD + d;
  const bool gate_on = a.gate_lo > 0.0 || a.gate_hi < 1.0;
  // What does not come from the block-sum pass is fetched while that pass drains.
  double anc = 0.0, dl = 0.0;
  bool had = false;
  if (threadIdx.x < 2 * kD) anc = ((threadIdx.x >> 7) ? a.anchor_k : a.anchor_q)[(size_t)r * kD + d];
  if (threadIdx.x == 0) {
    had = a.has_anchor[r] != 0;
    dl = a.delta[r];
  }
  pdl_wait();  // the partial sums come from the kernel before this one
  pdl_launch_dependents();
  double s = 0.0;
#pragma unroll 8
  for (int i = i0; i < i1; ++i) s += src[(size_t)i * kD];
  sm[z][grp][d] = s;
  __syncthreads();
  double m = 0.0;
  if (threadIdx.x < 2 * kD) {
    const int zz = threadIdx.x >> 7;
    m = (((sm[zz][0][d] + sm[zz][1][d]) + sm[zz][2][d]) + sm[zz][3][d]) / (double)N;
    mean[((size_t)zz * R + r) * kD + d] = m;
    double v = fabs(anc - m);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);  // same tree in every lane
    if ((threadIdx.x & 31) == 0) wsum[threadIdx.x >> 5] = v;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const double pq = (wsum[0] + wsum[1]) + (wsum[2] + wsum[3]), pk = (wsum[4] + wsum[5]) + (wsum[6] + wsum[7]);
    const double dr = had ? (pq + pk) : __longlong_as_double(0x7ff0000000000000LL);
    bool rf = !had || (dr > dl);
    if (a.flags & HEART_FORCE_REFRESH) rf = true;
    if (a.drift_out) a.drift_out[r] = dr;
    if (!gate_on) {
      a.refresh_ws[r] = rf;
      if (a.refresh_out) a.refresh_out[r] = rf;
      if (rf) a.has_anchor[r] = 1;
      sh_rf = rf;
    } else {
      a.pre_ws[r] = rf;
      __threadfence();
      last = (atomicAdd(a.ticket, 1) == (int)gridDim.x - 1);
    }
  }
  __syncthreads();
  if (!gate_on) {
    if (sh_rf && threadIdx.x < 2 * kD) ((threadIdx.x >> 7) ? a.anchor_k : a.anchor_q)[(size_t)r * kD + d] = m;
    return;
  }
  if (!last) return;
  // Every other CTA has read its old anchor and published its means and head-wise decision.
  __threadfence();
  for (int b = 0; b < a.B; ++b) gate_batch_entry(b, R, mean, a, sh_flags, &cnt);
  if (threadIdx.x == 0) *a.ticket = 0;
}

unsigned long long block_means_signature(const Geom &g, const void *Q, const void *K) {
  // A 64-bit mix of everything the block means depend on besides the tensors' contents.
  unsigned long long h = 0x9E3779B97F4A7C15ull;
  auto mix = [&h](unsigned long long v) {
    h ^= v + 0x9E3779B97F4A7C15ull + (h << 6) + (h >> 2);
    h *= 0xBF58476D1CE4E5B9ull;
    h ^= h >> 29;
  };
  mix(reinterpret_cast<uintptr_t>(Q));
  mix(reinterpret_cast<uintptr_t>(K));
  mix((unsigned long long)g.B << 40 | (unsigned long long)g.H << 20 | (unsigned long long)g.block);
  mix((unsigned long long)g.N);
  mix((unsigned long long)g.sb);
  mix((unsigned long long)g.sh);
  mix((unsigned long long)g.sn);
  return h | 1ull;  // never 0: a zeroed workspace holds no means
}

cudaError_t launch_block_sums(const Geom &g, const void *Q, const void *K, const Workspace &w,
                              cudaStream_t s, int *launches) {
  dim3 grid(g.nchunks, g.R, 2);
  const uint16_t *q = static_cast<const uint16_t *>(Q), *k = static_cast<const uint16_t *>(K);
  unsigned long long *sig_word = reinterpret_cast<unsigned long long *>(w.status + kStatusSigWord);
  const unsigned long long sig = block_means_signature(g, Q, K);
  ++*launches;
  if (g.block == 64)
    return launch_pdl(block_sums_kernel<64>, grid, dim3(256), 0, s, q, k, g.sb, g.sh, g.sn, g.H, g.N, g.nb, g.bpc,
                      w.bmean, w.psum, sig_word, sig);
  return launch_pdl(block_sums_kernel<128>, grid, dim3(256), 0, s, q, k, g.sb, g.sh, g.sn, g.H, g.N, g.nb, g.bpc,
                    w.bmean, w.psum, sig_word, sig);
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
  a.pre_ws = w.pre;
  a.drift_out = drift_out;
  a.refresh_out = refresh_out;
  a.ticket = w.status + kStatusTicketWord;
  ++*launches;
  return launch_pdl(mean_drift_kernel, dim3(g.R), dim3(1024), (size_t)2 * g.H, s, (const double *)w.psum, g.R, g.N,
                    g.nchunks, w.mean, a);
}

}  // namespace heart
