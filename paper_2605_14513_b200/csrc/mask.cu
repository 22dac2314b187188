// Block-importance mask prediction for the refreshed heads (Observation II: rank candidate blocks by
// importance, retain until the accumulated importance reaches the head's threshold; the minimal
// cumulative-mass set of Observation I).  Importance = row softmax of the block-pooled Q.K^T scores.
//
// Two kernels.  pooled_scores_kernel is a register-tiled fp64 contraction of the pooled means: a CTA
// owns 64 query blocks x 128 key blocks of one head (each thread 8 x 4), the means arrive 16 dims at
// a time by cp.async into a double-buffered shared-memory tile, and every score accumulates over the
// 128 dims in ascending order in one fma chain.  The scores go to the workspace (they stay in L2).
// top_p_kernel gives each warp one row (its weights in shared memory, the loops over them rolled):
// row max, unnormalised weights e = exp(s - max), then top-p WITHOUT a sort and without dividing by
// the row sum z: the kept set is {e > theta} plus the lowest-index ties at theta, where theta is the
// largest element value whose ">= theta" mass still reaches tau * z -- found by a search over the
// IEEE-754 pattern of e (positive doubles order like their bit patterns): starting below the leading
// bits that the largest and the smallest weight share, two bits a round over all blocks down to bit
// 48, the rest directly over the few blocks that share that prefix.  Everything is fp64 so the
// integer outputs (bit mask, ascending index list, count) agree with a plain fp64
// sort-and-accumulate reference except when the cumulative mass is within rounding (1e-15) of tau.
#include "common.cuh"

namespace heart {

constexpr int SI = 64;    // query blocks per CTA of the score kernel
constexpr int SJ = 128;   // key blocks per CTA
constexpr int TD = 16;    // dims per staged chunk
constexpr int KLD = TD + 1;
constexpr int kRowsPerCta = 8;  // rows (warps) per CTA of the top-p kernel
constexpr int kMaxCand = 64;    // candidates the direct threshold evaluation takes

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

// 8-byte asynchronous copy global -> shared; src_bytes = 0 writes zeros instead
__device__ __forceinline__ void cp_async8(double *smem_dst, const double *src, int src_bytes) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 8, %2;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)),
               "l"(src), "r"(src_bytes)
               : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// scores[r][I][J] = scale * <mean_q[r][I], mean_k[r][J]> for the refreshed heads r.
__global__ void __launch_bounds__(256, 2) pooled_scores_kernel(const double *__restrict__ bmean, int R, int nb,
                                                               int pitch, double scale,
                                                               const uint8_t *__restrict__ refresh,
                                                               double *__restrict__ scores,
                                                               int32_t *__restrict__ status,
                                                               unsigned long long expect_sig) {
  const int r = blockIdx.z;
  pdl_wait();  // refresh flags and block means come from the kernels before this one
  pdl_launch_dependents();
  if (expect_sig != 0 && *reinterpret_cast<const unsigned long long *>(status + kStatusSigWord) != expect_sig) {
    // the caller vouched for block means that this workspace does not hold: report, predict nothing
    if (threadIdx.x == 0) atomicExch(status, HEART_ERR_DEVICE_CHECK);
    return;
  }
  if (refresh != nullptr && refresh[r] == 0) return;  // reuse branch of Algorithm 1: nothing to predict
  const int I0 = blockIdx.y * SI, J0 = blockIdx.x * SJ;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  double *tile = reinterpret_cast<double *>(smem_raw);  // [2][SI + SJ][KLD]: query rows, then key rows
  const double *bq = bmean + ((size_t)r * nb) * kD;
  const double *bk = bmean + (((size_t)R + r) * nb) * kD;
  const int tid = threadIdx.x;
  constexpr int kRows = SI + SJ, kPer = kRows * TD / 256;  // 12 copies per thread and stage
  auto stage_in = [&](int stage, int buf) {
    const int dc = stage * TD;
    double *dst = tile + (size_t)buf * kRows * KLD;
#pragma unroll
    for (int k = 0; k < kPer; ++k) {
      const int e = tid + 256 * k, row = e / TD, dd = e % TD;
      const int blk = row < SI ? I0 + row : J0 + row - SI;
      const double *src = (row < SI ? bq : bk) + (size_t)min(blk, nb - 1) * kD + dc + dd;
      cp_async8(dst + row * KLD + dd, src, blk < nb ? 8 : 0);
    }
    cp_async_commit();
  };
  const int rg = tid >> 5, cl = tid & 31;  // rows rg*8 .. rg*8+7, key columns cl + 32 m
  double acc[8][4];
#pragma unroll
  for (int a = 0; a < 8; ++a)
#pragma unroll
    for (int m = 0; m < 4; ++m) acc[a][m] = 0.0;
  stage_in(0, 0);
  for (int stage = 0; stage < kD / TD; ++stage) {
    const int buf = stage & 1;
    if (stage + 1 < kD / TD) {
      stage_in(stage + 1, buf ^ 1);  // its buffer was released by the barrier that ended stage - 1
      cp_async_wait<1>();
    } else {
      cp_async_wait<0>();
    }
    __syncthreads();
    const double *Qs = tile + (size_t)buf * kRows * KLD, *Ks = Qs + SI * KLD;
#pragma unroll 4
    for (int dd = 0; dd < TD; ++dd) {
      double q[8], k4[4];
#pragma unroll
      for (int a = 0; a < 8; ++a) q[a] = Qs[(rg * 8 + a) * KLD + dd];
#pragma unroll
      for (int m = 0; m < 4; ++m) k4[m] = Ks[(cl + 32 * m) * KLD + dd];
#pragma unroll
      for (int a = 0; a < 8; ++a)
#pragma unroll
        for (int m = 0; m < 4; ++m) acc[a][m] = fma(q[a], k4[m], acc[a][m]);
    }
    __syncthreads();  // this stage's buffer may be refilled
  }
#pragma unroll
  for (int a = 0; a < 8; ++a) {
    const int I = I0 + rg * 8 + a;
    if (I >= nb) continue;
#pragma unroll
    for (int m = 0; m < 4; ++m) {
      const int J = J0 + cl + 32 * m;
      if (J < pitch) scores[((size_t)r * nb + I) * pitch + J] = acc[a][m] * scale;
    }
  }
}

template <int NJ>  // NJ*32 >= n_b
__global__ void __launch_bounds__(32 * kRowsPerCta) top_p_kernel(const double *__restrict__ scores, int nb, int pitch,
                                                                 const double *__restrict__ tau,
                                                                 const uint8_t *__restrict__ refresh,
                                                                 unsigned flags, uint32_t *__restrict__ mask_bits,
                                                                 int32_t *__restrict__ kv_idx,
                                                                 int32_t *__restrict__ kv_cnt, int idx_stride,
                                                                 int W, const int32_t *__restrict__ status,
                                                                 unsigned long long expect_sig) {
  const int r = blockIdx.y;
  pdl_wait();  // the scores come from the kernel before this one
  if (expect_sig != 0 && *reinterpret_cast<const unsigned long long *>(status + kStatusSigWord) != expect_sig)
    return;  // reported by the score kernel
  if (refresh != nullptr && refresh[r] == 0) return;  // reuse branch of Algorithm 1: mask untouched
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  extern __shared__ __align__(16) unsigned char smem_top[];
  double *weights = reinterpret_cast<double *>(smem_top);  // [kRowsPerCta][NJ * 32]
  __shared__ double cand[kRowsPerCta][kMaxCand];
  const unsigned lt_mask = (1u << lane) - 1u;
  {
    const int I = blockIdx.x * kRowsPerCta + warp;
    if (I >= nb) return;
    const size_t row = (size_t)r * nb + I;
    const double *srow = scores + row * pitch;
    // The weights of the row live in shared memory (lane-major, conflict-free): rolled loops over the
    // NJ blocks of a lane keep the kernel small enough for the instruction cache -- fully unrolled
    // over registers it was several times slower at n_b > 512.
    double *pw = weights + (size_t)warp * NJ * 32 + lane;
    const double neg_inf = __longlong_as_double(0xfff0000000000000LL);
    double mx = neg_inf;
#pragma unroll 4
    for (int j = 0; j < NJ; ++j) {
      const int J = j * 32 + lane;
      pw[(j) * 32] = (J < nb) ? srow[J] : neg_inf;
      mx = fmax(mx, pw[(j) * 32]);
    }
    mx = warp_max(mx);
    double z = 0.0;
#pragma unroll 4
    for (int j = 0; j < NJ; ++j) {
      const int J = j * 32 + lane;
      pw[(j) * 32] = (J < nb) ? exp_nonpositive(pw[(j) * 32] - mx) : 0.0;
      z += pw[(j) * 32];
    }
    z = warp_sum(z);
    // From here on p holds the unnormalised weights e = exp(s - max) <= 1 and every mass is compared
    // with tau * z instead of dividing the row by z: the same ranking, the same ties and the same
    // cumulative-mass test up to rounding, at 1/3 fewer fp64 instructions per block.
    const double tau_r = (flags & HEART_FORCE_DENSE) ? 1.0 : tau[r];
    // tau <= 0: every prefix reaches it, so the minimal one is the single largest block (lowest index
    // on ties): the smallest positive threshold gives exactly that
    const double t = (tau_r > 0.0 ? tau_r : 2.2250738585072014e-308) * z;
    const bool keep_all = !(tau_r < 1.0) || !(z >= t);
    long long theta = 0;
    int m_ties = 0, n_ties = 0;
    if (!keep_all) {
      // Rounds over all blocks, two bits of theta each: three trial thresholds per round, their three
      // reductions side by side (fixed split of the sums: same order on every run).
      auto round2 = [&](int bit) {
        // trial patterns theta | 01, 10, 11 at bits (bit+1, bit): the mass is non-increasing in them
        // (bit >= 32: the low words of the patterns are zero, so comparing the high words decides)
        const long long c1 = theta | (1LL << bit), c2 = theta | (2LL << bit), c3 = theta | (3LL << bit);
        const int h1 = (int)(c1 >> 32), h2 = (int)(c2 >> 32), h3 = (int)(c3 >> 32);
        double a1 = 0.0, a2 = 0.0, a3 = 0.0, b1 = 0.0, b2 = 0.0, b3 = 0.0;
#pragma unroll 2
        for (int j = 0; j < NJ; j += 2) {
          const int k0 = __double2hiint(pw[(j) * 32]), k1 = __double2hiint(pw[(j + 1) * 32]);
          if (k0 >= h1) a1 += pw[(j) * 32];
          if (k0 >= h2) a2 += pw[(j) * 32];
          if (k0 >= h3) a3 += pw[(j) * 32];
          if (k1 >= h1) b1 += pw[(j + 1) * 32];
          if (k1 >= h2) b2 += pw[(j + 1) * 32];
          if (k1 >= h3) b3 += pw[(j + 1) * 32];
        }
        double m1 = a1 + b1, m2 = a2 + b2, m3 = a3 + b3;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          m1 += __shfl_xor_sync(0xffffffffu, m1, o);
          m2 += __shfl_xor_sync(0xffffffffu, m2, o);
          m3 += __shfl_xor_sync(0xffffffffu, m3, o);
        }
        theta = (m3 >= t) ? c3 : (m2 >= t) ? c2 : (m1 >= t) ? c1 : theta;
      };
      static_assert(NJ % 2 == 0, "two blocks per step");
      // The exponent and the top four mantissa bits first (bits 61..48; bit 62 is clear for p <= 1) ...
      constexpr int low = 48;  // bits [low, 62) of theta are decided over all blocks
      static_assert(low >= 32, "the full-width rounds compare high words only");
      // theta is the value of one of the blocks, so it shares the leading bits that the largest and
      // the smallest weight of the row have in common: the rounds start below them.
      int first_bit = 60;
      {
        int hmax = 0, hmin = 0x7fffffff;
#pragma unroll 4
        for (int j = 0; j < NJ; ++j) {
          const int h = __double2hiint(pw[(j) * 32]);
          hmax = max(hmax, h);
          if (j * 32 + lane < nb) hmin = min(hmin, h);
        }
        hmax = __reduce_max_sync(0xffffffffu, hmax);
        hmin = __reduce_min_sync(0xffffffffu, hmin);
        const int top = 63 - __clz(hmax ^ hmin);  // highest bit (of the 64) in which they differ; 31 if none in the high word
        first_bit = min(60, top & ~1);            // the round at `bit` decides bits (bit + 1, bit)
        if (first_bit + 2 < 62) theta = ((long long)hmax << 32) & ~((1LL << (first_bit + 2)) - 1);
      }
      for (int bit = first_bit; bit >= low; bit -= 2) round2(bit);
      if (first_bit < low) theta &= ~((1LL << low) - 1);  // the whole searched prefix is common
      // ... then only the blocks whose pattern shares that prefix can still decide the remaining bits:
      // they are compacted into shared memory (the first kMaxCand of them; more than that takes the
      // slow path below, which does not read the list).  Blocks above the prefix enter as one constant.
      const long long hi = theta >> low;
      double *scr = cand[warp];
      double ab0 = 0.0, ab1 = 0.0;
      int n_cand = 0;
      __syncwarp();
#pragma unroll 4
      for (int j = 0; j < NJ; ++j) {
        const long long kh = __double_as_longlong(pw[(j) * 32]) >> low;
        if (kh > hi) {
          if (j & 1) ab1 += pw[(j) * 32]; else ab0 += pw[(j) * 32];
        }
        const bool is_c = (kh == hi) && (j * 32 + lane < nb);
        const unsigned bal = __ballot_sync(0xffffffffu, is_c);
        if (is_c) {
          const int pos = n_cand + __popc(bal & lt_mask);
          if (pos < kMaxCand) scr[pos] = pw[(j) * 32];
        }
        n_cand += __popc(bal);
      }
      const double mass_above = warp_sum(ab0 + ab1);
      __syncwarp();
      if (n_cand <= kMaxCand) {
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
      } else {  // many near-equal blocks: keep searching over all of them, a bit at a time
        for (int bit = low - 1; bit >= 0; --bit) {
          const long long cnd = theta | (1LL << bit);
          double g0 = 0.0, g1 = 0.0, g2 = 0.0, g3 = 0.0;  // fixed 4-way split: same order on every run
#pragma unroll 1
          for (int j = 0; j < NJ; j += 4) {
            if (__double_as_longlong(pw[(j) * 32]) >= cnd) g0 += pw[(j) * 32];
            if (j + 1 < NJ && __double_as_longlong(pw[(j + 1) * 32]) >= cnd) g1 += pw[(j + 1) * 32];
            if (j + 2 < NJ && __double_as_longlong(pw[(j + 2) * 32]) >= cnd) g2 += pw[(j + 2) * 32];
            if (j + 3 < NJ && __double_as_longlong(pw[(j + 3) * 32]) >= cnd) g3 += pw[(j + 3) * 32];
          }
          if (warp_sum((g0 + g1) + (g2 + g3)) >= t) theta = cnd;
        }
      }
      double above = 0.0;
      int nties = 0;
#pragma unroll 4
      for (int j = 0; j < NJ; ++j) {
        const long long b = __double_as_longlong(pw[(j) * 32]);
        if (b > theta) above += pw[(j) * 32];
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
      n_ties = nties;
    }

    int base = 0, tie_seen = 0;
    // the usual case: every block equal to theta is kept (theta = 0 when all blocks are kept)
    const bool all_ties_kept = keep_all || m_ties == n_ties;
    // The mask words are gathered in registers (lane l keeps word l) and leave in one store.
    uint32_t my_word = 0u;
#pragma unroll 4
    for (int j = 0; j < NJ; ++j) {
      const int J = j * 32 + lane;
      const long long b = __double_as_longlong(pw[(j) * 32]);
      const bool valid = J < nb;
      bool keep;
      if (all_ties_kept) {
        keep = valid && b >= theta;
      } else {
        const bool is_tie = valid && b == theta;
        const unsigned tie_ballot = __ballot_sync(0xffffffffu, is_tie);
        const int tie_rank = tie_seen + __popc(tie_ballot & lt_mask);
        tie_seen += __popc(tie_ballot);
        keep = valid && (b > theta || (is_tie && tie_rank < m_ties));
      }
      const unsigned word = __ballot_sync(0xffffffffu, keep);
      if (lane == j) my_word = word;
      if (keep) kv_idx[row * idx_stride + base + __popc(word & lt_mask)] = J;
      base += __popc(word);
    }
    if (lane < W) mask_bits[row * W + lane] = my_word;
    if (lane == 0) kv_cnt[row] = base;
  }
}

template <int NJ>
static cudaError_t launch_nj(const Geom &g, const Workspace &w, const double *tau, const uint8_t *refresh,
                             heart_state st, int pitch, cudaStream_t s, unsigned long long expect_sig) {
  dim3 grid((g.nb + kRowsPerCta - 1) / kRowsPerCta, g.R);
  const size_t smem = sizeof(double) * kRowsPerCta * NJ * 32;
  cudaError_t e = cudaFuncSetAttribute(top_p_kernel<NJ>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  return launch_pdl(top_p_kernel<NJ>, grid, dim3(32 * kRowsPerCta), smem, s, (const double *)w.scores, g.nb, pitch, tau,
                    refresh, g.flags, st.mask_bits, st.kv_idx, st.kv_cnt, g.idx_stride, g.W, (const int32_t *)w.status,
                    expect_sig);
}

cudaError_t launch_pooled_scores(const Geom &g, const Workspace &w, const uint8_t *refresh, cudaStream_t s,
                                 int *launches, unsigned long long expect_sig) {
  ++*launches;
  const int nj = (g.nb + 31) / 32, pitch = nj * 32;
  const size_t smem = sizeof(double) * 2 * (SI + SJ) * KLD;
  cudaError_t e = cudaFuncSetAttribute(pooled_scores_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  dim3 grid((g.nb + SJ - 1) / SJ, (g.nb + SI - 1) / SI, g.R);
  return launch_pdl(pooled_scores_kernel, grid, dim3(256), smem, s, (const double *)w.bmean, g.R, g.nb, pitch, g.scale,
                    refresh, w.scores, w.status, expect_sig);
}

cudaError_t launch_top_p(const Geom &g, const Workspace &w, const double *tau, const uint8_t *refresh,
                         heart_state st, cudaStream_t s, int *launches, unsigned long long expect_sig) {
  ++*launches;
  const int nj = (g.nb + 31) / 32, pitch = nj * 32;
  if (nj <= 8) return launch_nj<8>(g, w, tau, refresh, st, pitch, s, expect_sig);
  if (nj <= 16) return launch_nj<16>(g, w, tau, refresh, st, pitch, s, expect_sig);
  if (nj <= 24) return launch_nj<24>(g, w, tau, refresh, st, pitch, s, expect_sig);
  return launch_nj<32>(g, w, tau, refresh, st, pitch, s, expect_sig);
}

cudaError_t launch_predict_mask(const Geom &g, const Workspace &w, const double *tau,
                                const uint8_t *refresh, heart_state st, cudaStream_t s, int *launches,
                                unsigned long long expect_sig) {
  cudaError_t e = launch_pooled_scores(g, w, refresh, s, launches, expect_sig);
  if (e != cudaSuccess) return e;
  return launch_top_p(g, w, tau, refresh, st, s, launches, expect_sig);
}

}  // namespace heart
