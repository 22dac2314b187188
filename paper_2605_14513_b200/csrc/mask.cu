// Block-importance mask prediction for the refreshed heads (Observation II: rank candidate blocks by
// importance, retain until the accumulated importance reaches the head's threshold; the minimal
// cumulative-mass set of Observation I).  Importance = row softmax of the block-pooled Q.K^T scores.
//
// One CTA owns TI = 16 query blocks of one head.  Phase 1 is a register-tiled fp64 contraction of
// the pooled means (each thread 8 query blocks x 4 key blocks, key means staged through shared
// memory 512 blocks x 16 dims at a time with the next stage's loads in flight) into a shared-memory
// tile of scores.  Phase 2 gives each
// warp two rows: two-pass softmax, then top-p WITHOUT a sort: the kept set is {p > theta} plus the
// lowest-index ties at theta, where theta is the largest element value whose ">= theta" mass still
// reaches tau -- found by a search over the IEEE-754 pattern of p (positive doubles order like
// their bit patterns): the top 14 bits two at a time over all blocks, the rest directly over the
// few blocks that share that prefix.  Everything is fp64 so the integer outputs (bit mask,
// ascending index list, count) agree with a plain fp64 sort-and-accumulate reference except when
// the cumulative mass is within rounding (1e-15) of tau.
#include <type_traits>

#include "common.cuh"

namespace heart {

constexpr int TI = 16;    // query blocks per CTA
constexpr int TJ = 512;   // key blocks per staged pass
constexpr int TD = 16;    // dims per staged chunk
constexpr int KLD = TD + 1;

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;  // identical in every lane (each level adds the same two numbers in both partners)
}
__device__ __forceinline__ double warp_max(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmax(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

template <int NJ>  // NJ*32 >= n_b
__global__ void __launch_bounds__(256) predict_mask_kernel(const double *__restrict__ bsum, int R, int N,
                                                           int block, int nb, double scale,
                                                           const double *__restrict__ tau,
                                                           const uint8_t *__restrict__ refresh,
                                                           unsigned flags, uint32_t *__restrict__ mask_bits,
                                                           int32_t *__restrict__ kv_idx,
                                                           int32_t *__restrict__ kv_cnt, int idx_stride,
                                                           int W) {
  constexpr int NBP = NJ * 32;
  const int r = blockIdx.y;
  if (refresh != nullptr && refresh[r] == 0) return;  // reuse branch of Algorithm 1: mask untouched
  const int I0 = blockIdx.x * TI;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  double *S = reinterpret_cast<double *>(smem_raw);  // [TI][NBP]
  double *Qs = S + TI * NBP;                         // [TI][kD]
  double *Ks = Qs + TI * kD;                         // [TJ][KLD]
  const double *bq = bsum + ((size_t)r * nb) * kD;
  const double *bk = bsum + (((size_t)R + r) * nb) * kD;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int last_cnt = N - (nb - 1) * block;
  const double inv_block = 1.0 / (double)block;

  for (int e = tid; e < TI * kD; e += 256) {
    const int i = e / kD, I = I0 + i;
    double v = 0.0;
    if (I < nb) v = (I == nb - 1) ? bq[(size_t)I * kD + (e % kD)] / (double)last_cnt : bq[(size_t)I * kD + (e % kD)] * inv_block;
    Qs[e] = v;
  }

  // ---- phase 1: S[i][J] = scale * <Qp[I0+i], Kp[J]>.  Each thread owns 8 query blocks x 4 key blocks;
  // the key means are staged 512 blocks x 16 dims at a time, and the loads of the next stage are in
  // flight (in registers) while the current one is multiplied.
  const int rg = tid >> 7, cl = tid & 127;
  constexpr int PER = (TJ * TD) / 256;  // staged values per thread = 32
  const int n_jc = (nb + TJ - 1) / TJ, n_stage = n_jc * (kD / TD);
  double pre[PER];
  auto fetch = [&](int stage) {
    const int jc = (stage / (kD / TD)) * TJ, dc = (stage % (kD / TD)) * TD;
#pragma unroll
    for (int k = 0; k < PER; ++k) {
      const int e = tid + 256 * k, J = jc + e / TD;
      pre[k] = (J < nb) ? bk[(size_t)J * kD + dc + (e % TD)] : 0.0;
    }
  };
  fetch(0);
  double acc[8][4];
  for (int stage = 0; stage < n_stage; ++stage) {
    const int jc = (stage / (kD / TD)) * TJ, dc = (stage % (kD / TD)) * TD;
    if (dc == 0) {
#pragma unroll
      for (int a = 0; a < 8; ++a)
#pragma unroll
        for (int m = 0; m < 4; ++m) acc[a][m] = 0.0;
    }
    __syncthreads();  // the previous stage has been consumed
#pragma unroll
    for (int k = 0; k < PER; ++k) {
      const int e = tid + 256 * k, row = e / TD, J = jc + row;
      // full blocks: 1/block is a power of two, so the product equals the division exactly
      Ks[row * KLD + (e % TD)] = (J == nb - 1) ? pre[k] / (double)last_cnt : pre[k] * inv_block;
    }
    __syncthreads();
    if (stage + 1 < n_stage) fetch(stage + 1);
    // column groups of 128 key blocks that exist in this pass (the last pass is usually short)
    const int nm = min(4, (nb - jc + 127) >> 7);
    auto multiply = [&](auto NM) {
      constexpr int kNm = decltype(NM)::value;
#pragma unroll 4
      for (int dd = 0; dd < TD; ++dd) {
        double q[8], k4[kNm];
#pragma unroll
        for (int a = 0; a < 8; ++a) q[a] = Qs[(rg * 8 + a) * kD + dc + dd];
#pragma unroll
        for (int m = 0; m < kNm; ++m) k4[m] = Ks[(cl + 128 * m) * KLD + dd];
#pragma unroll
        for (int a = 0; a < 8; ++a)
#pragma unroll
          for (int m = 0; m < kNm; ++m) acc[a][m] = fma(q[a], k4[m], acc[a][m]);
      }
    };
    if (nm == 4)
      multiply(std::integral_constant<int, 4>{});
    else if (nm == 3)
      multiply(std::integral_constant<int, 3>{});
    else if (nm == 2)
      multiply(std::integral_constant<int, 2>{});
    else
      multiply(std::integral_constant<int, 1>{});
    if (dc == kD - TD) {
#pragma unroll
      for (int a = 0; a < 8; ++a)
#pragma unroll
        for (int m = 0; m < 4; ++m) {
          const int J = jc + cl + 128 * m;
          if (J < NBP) S[(rg * 8 + a) * NBP + J] = acc[a][m] * scale;
        }
    }
  }
  __syncthreads();

  // ---- phase 2: per-row softmax and top-p; warp w owns rows 2w and 2w+1
  const unsigned lt_mask = (1u << lane) - 1u;
  for (int i = warp * 2; i < warp * 2 + 2; ++i) {
    const int I = I0 + i;
    if (I >= nb) continue;
    const size_t row = (size_t)r * nb + I;
    double p[NJ];
    const double neg_inf = __longlong_as_double(0xfff0000000000000LL);
    double mx = neg_inf;
#pragma unroll
    for (int j = 0; j < NJ; ++j) {
      const int J = j * 32 + lane;
      p[j] = (J < nb) ? S[i * NBP + J] : neg_inf;
      mx = fmax(mx, p[j]);
    }
    mx = warp_max(mx);
    double z = 0.0;
#pragma unroll
    for (int j = 0; j < NJ; ++j) {
      const int J = j * 32 + lane;
      p[j] = (J < nb) ? exp(p[j] - mx) : 0.0;
      z += p[j];
    }
    z = warp_sum(z);
    double total = 0.0;
#pragma unroll
    for (int j = 0; j < NJ; ++j) {
      p[j] = p[j] / z;
      total += p[j];
    }
    total = warp_sum(total);

    const double t = (flags & HEART_FORCE_DENSE) ? 1.0 : tau[r];
    const bool keep_all = !(t < 1.0) || !(total >= t);
    long long theta = 0;
    int m_ties = 0;
    if (!keep_all) {
      // Full-width rounds for the exponent and the top mantissa bits ...
      auto mass_at_least = [&](long long cand) -> double {
        double g0 = 0.0, g1 = 0.0, g2 = 0.0, g3 = 0.0;  // fixed 4-way split: same order on every run
#pragma unroll
        for (int j = 0; j < NJ; j += 4) {
          if (__double_as_longlong(p[j]) >= cand) g0 += p[j];
          if (j + 1 < NJ && __double_as_longlong(p[j + 1]) >= cand) g1 += p[j + 1];
          if (j + 2 < NJ && __double_as_longlong(p[j + 2]) >= cand) g2 += p[j + 2];
          if (j + 3 < NJ && __double_as_longlong(p[j + 3]) >= cand) g3 += p[j + 3];
        }
        return warp_sum((g0 + g1) + (g2 + g3));
      };
      constexpr int kSplit = 48;  // bits [kSplit, 62) are searched over all blocks, two bits a round
      // (three trial thresholds per round: their three reductions run side by side)
      auto masses_at_least = [&](long long c1, long long c2, long long c3, double &m1, double &m2, double &m3) {
        double a1 = 0.0, a2 = 0.0, a3 = 0.0, b1 = 0.0, b2 = 0.0, b3 = 0.0;  // fixed split: same order on every run
#pragma unroll
        for (int j = 0; j < NJ; j += 2) {
          const long long k0 = __double_as_longlong(p[j]), k1 = __double_as_longlong(p[j + 1]);
          if (k0 >= c1) a1 += p[j];
          if (k0 >= c2) a2 += p[j];
          if (k0 >= c3) a3 += p[j];
          if (k1 >= c1) b1 += p[j + 1];
          if (k1 >= c2) b2 += p[j + 1];
          if (k1 >= c3) b3 += p[j + 1];
        }
        m1 = a1 + b1;
        m2 = a2 + b2;
        m3 = a3 + b3;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          m1 += __shfl_xor_sync(0xffffffffu, m1, o);
          m2 += __shfl_xor_sync(0xffffffffu, m2, o);
          m3 += __shfl_xor_sync(0xffffffffu, m3, o);
        }
      };
      static_assert((62 - kSplit) % 2 == 0 && NJ % 2 == 0, "two bits per round, two blocks per step");
      for (int bit = 60; bit >= kSplit; bit -= 2) {
        // trial patterns theta | 01, 10, 11 at bits (bit+1, bit): the mass is non-increasing in them
        const long long c1 = theta | (1LL << bit), c2 = theta | (2LL << bit), c3 = theta | (3LL << bit);
        double m1, m2, m3;
        masses_at_least(c1, c2, c3, m1, m2, m3);
        theta = (m3 >= t) ? c3 : (m2 >= t) ? c2 : (m1 >= t) ? c1 : theta;
      }
      // ... then only the blocks whose pattern shares that prefix can still decide the remaining bits:
      // they are compacted (through this row's no longer needed score slots) and the other 48 rounds
      // run on at most two candidates per lane.  Blocks above the prefix enter as one constant.
      const long long hi = theta >> kSplit;
      double *scr = S + i * NBP;
      double ab0 = 0.0, ab1 = 0.0;
      int n_cand = 0;
      __syncwarp();
#pragma unroll
      for (int j = 0; j < NJ; ++j) {
        const long long kh = __double_as_longlong(p[j]) >> kSplit;
        if (kh > hi) {
          if (j & 1) ab1 += p[j]; else ab0 += p[j];
        }
        const bool is_c = (kh == hi) && (j * 32 + lane < nb);
        const unsigned bal = __ballot_sync(0xffffffffu, is_c);
        if (is_c) scr[n_cand + __popc(bal & lt_mask)] = p[j];
        n_cand += __popc(bal);
      }
      const double mass_above = warp_sum(ab0 + ab1);
      __syncwarp();
      if (n_cand <= 64) {
        // Few candidates: each lane takes two of them and adds up, over all candidates, the mass at
        // or above its own value; theta is the largest candidate whose mass still reaches tau (the
        // smallest candidate always does: that is what the prefix search established).
        const double c0 = (lane < n_cand) ? scr[lane] : 0.0, c1 = (lane + 32 < n_cand) ? scr[lane + 32] : 0.0;
        const long long k0 = __double_as_longlong(c0), k1 = __double_as_longlong(c1);
        double g0 = mass_above, g1 = mass_above;
        long long k_min = 0x7fffffffffffffffLL;
        for (int n = 0; n < n_cand; ++n) {
          const double v = scr[n];
          const long long kv = __double_as_longlong(v);
          if (kv >= k0) g0 += v;
          if (kv >= k1) g1 += v;
          k_min = kv < k_min ? kv : k_min;
        }
        long long best = k_min;
        if (lane < n_cand && g0 >= t && k0 > best) best = k0;
        if (lane + 32 < n_cand && g1 >= t && k1 > best) best = k1;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          const long long other = __shfl_xor_sync(0xffffffffu, best, o);
          best = other > best ? other : best;
        }
        theta = best;
      } else {  // many near-equal blocks: keep searching over all of them
        for (int bit = kSplit - 1; bit >= 0; --bit) {
          const long long cand = theta | (1LL << bit);
          if (mass_at_least(cand) >= t) theta = cand;
        }
      }
      double above = 0.0;
      int nties = 0;
#pragma unroll
      for (int j = 0; j < NJ; ++j) {
        const long long b = __double_as_longlong(p[j]);
        if (b > theta) above += p[j];
        nties += (b == theta && j * 32 + lane < nb) ? 1 : 0;
      }
      above = warp_sum(above);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) nties += __shfl_xor_sync(0xffffffffu, nties, o);
      const double th = __longlong_as_double(theta);
      double c = above;
      do {  // ties enter in ascending index order, one at a time, until the mass reaches tau
        c += th;
        ++m_ties;
      } while (c < t && m_ties < nties);
    }

    int base = 0, tie_seen = 0;
#pragma unroll
    for (int j = 0; j < NJ; ++j) {
      const int J = j * 32 + lane;
      const long long b = __double_as_longlong(p[j]);
      const bool valid = J < nb;
      const bool is_tie = valid && !keep_all && b == theta;
      const unsigned tie_ballot = __ballot_sync(0xffffffffu, is_tie);
      const int tie_rank = tie_seen + __popc(tie_ballot & lt_mask);
      tie_seen += __popc(tie_ballot);
      const bool keep = valid && (keep_all || b > theta || (is_tie && tie_rank < m_ties));
      const unsigned word = __ballot_sync(0xffffffffu, keep);
      if (lane == 0 && j < W) mask_bits[row * W + j] = word;
      if (keep) kv_idx[row * idx_stride + base + __popc(word & lt_mask)] = J;
      base += __popc(word);
    }
    if (lane == 0) kv_cnt[row] = base;
  }
}

template <int NJ>
static cudaError_t launch_nj(const Geom &g, const Workspace &w, const double *tau, const uint8_t *refresh,
                             heart_state st, cudaStream_t s) {
  const size_t smem = sizeof(double) * ((size_t)TI * NJ * 32 + TI * kD + TJ * KLD);
  cudaError_t e = cudaFuncSetAttribute(predict_mask_kernel<NJ>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)smem);
  if (e != cudaSuccess) return e;
  dim3 grid((g.nb + TI - 1) / TI, g.R);
  predict_mask_kernel<NJ><<<grid, 256, smem, s>>>(w.bsum, g.R, g.N, g.block, g.nb, g.scale, tau, refresh,
                                                 g.flags, st.mask_bits, st.kv_idx, st.kv_cnt,
                                                 g.idx_stride, g.W);
  return cudaGetLastError();
}

cudaError_t launch_predict_mask(const Geom &g, const Workspace &w, const double *tau,
                                const uint8_t *refresh, heart_state st, cudaStream_t s, int *launches) {
  ++*launches;
  const int nj = (g.nb + 31) / 32;
  if (nj <= 8) return launch_nj<8>(g, w, tau, refresh, st, s);
  if (nj <= 16) return launch_nj<16>(g, w, tau, refresh, st, s);
  if (nj <= 24) return launch_nj<24>(g, w, tau, refresh, st, s);
  return launch_nj<32>(g, w, tau, refresh, st, s);
}

}  // namespace heart
