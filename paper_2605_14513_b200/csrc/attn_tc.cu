// Block-sparse attention with online softmax on the sm_100a tensor cores.
//
// One CTA owns one 128-row query tile of one head: one query block of 128 tokens, or two query
// blocks of 64 whose lists are merged into an ascending union (one flag bit per query block; rows of
// the half that does not list a key block see -inf there).  Keys are processed 128 at a time: a key
// tile is one 128-token block or two 64-token blocks of the union.
//
// The key tiles are dealt to two independent streams (even / odd tile index).  Each stream keeps its
// own running max, row sum and output accumulator and the two are merged at the end, so the softmax of
// one stream overlaps the MMAs of the other (ping-pong) although both work for the same query rows.
//
// Warp roles (320 threads):
//   warp 0      TMA producer: the Q tile once, then the listed K and V blocks through shared-memory
//               rings (cp.async.bulk.tensor, 128-byte swizzle, completion on mbarriers).
//   warp 1      MMA issuer (one lane): S_t = Q K^T into tensor memory (tcgen05.mma, operands in shared
//               memory), O_t += P_t V with P_t read from tensor memory.
//   warps 2-9   softmax: both warpgroups work on the stream whose scores are ready, warpgroup a on key
//               columns [64a, 64a+64); thread = (query row, column half).  It reads its half of the S
//               row from tensor memory, the two halves exchange their row maxima through shared
//               memory, it keeps the running max / partial sum, writes P (bf16) back over S,
//               rescales its half of O only when the max grew by more than 2^8, and at the end merges
//               the two streams and writes its half of O (and lse).
// Tensor memory (512 columns): S0 | S1 | O0 | O1, 128 fp32 columns each; P_t aliases S_t.
//
// Every wait is bounded; a wait that runs out raises a CTA-wide abort flag and the status word, the
// roles drain, tensor memory is freed and the CTA exits.
#include <cuda.h>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace heart {
using namespace tc;

constexpr int kAttnThreads = 320;
constexpr int kMaxNb = HEART_MAX_BLOCKS;

// Shared-memory plan.  A key tile always holds 128 keys = SUBS key blocks of B tokens.
template <int B>
struct AttnSmem {
  static constexpr int SUBS = 128 / B;          // key blocks per 128-key tile (1 or 2)
  static constexpr int QBT = 128 / B;           // query blocks per CTA (1 or 2)
  static constexpr int TILE_BYTES = 128 * 256;  // [2 dim halves][128 rows][64] bf16, 128-byte swizzle
  static constexpr int OFF_Q = 0;
  static constexpr int OFF_K = OFF_Q + TILE_BYTES;      // 2 stages: stream t uses stage t
  static constexpr int OFF_V = OFF_K + 2 * TILE_BYTES;  // 2 stages
  static constexpr int OFF_UNI = OFF_V + 2 * TILE_BYTES;  // int32[kMaxNb]: J | flags << 16
  static constexpr int OFF_TBL = OFF_UNI + 4 * kMaxNb;    // uint32[kMaxNb]: flags per key block
  static constexpr int OFF_XCH = OFF_TBL + 4 * kMaxNb;    // float[2 uses][2 streams][2 halves][128 rows]: row max, row sum
  static constexpr int OFF_BAR = OFF_XCH + 4096;          // mbarriers and scalars
  static constexpr int TOTAL = OFF_BAR + 512;
};

struct AttnBars {
  uint64_t q_full;
  uint64_t k_full[2], k_empty[2], v_full[2], v_empty[2];
  uint64_t s_full[2], p_full[2], pv_done[2];
  uint64_t x_full[2][4];  // [stream][lane quarter]: the two column halves of the same 32 rows meet here
  uint32_t tmem_base;
  int n_union;
  int abort;
  int bad;
};

struct AttnParams {
  const int32_t *kv_idx, *kv_cnt;
  uint16_t *O;
  float *lse;
  int32_t *status;
  long long sb, sh, sn;
  int H, N, nb, idx_stride, n_ctas_per_head, dense;
  float scale_log2;
};

__device__ __forceinline__ float fmax3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}

template <int B>
__global__ void __launch_bounds__(kAttnThreads, 1)
    attn_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_kv,
                   const __grid_constant__ CUtensorMap map_v, const AttnParams p) {
  using L = AttnSmem<B>;
  constexpr int SUBS = L::SUBS;
  extern __shared__ unsigned char smem_dyn[];
  unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) &
                                                          ~static_cast<uintptr_t>(1023));
  unsigned char *Qs = smem + L::OFF_Q, *Ks = smem + L::OFF_K, *Vs = smem + L::OFF_V;
  int32_t *uni = reinterpret_cast<int32_t *>(smem + L::OFF_UNI);
  uint32_t *tbl = reinterpret_cast<uint32_t *>(smem + L::OFF_TBL);
  float *xch = reinterpret_cast<float *>(smem + L::OFF_XCH);
  AttnBars *bars = reinterpret_cast<AttnBars *>(smem + L::OFF_BAR);
  volatile int *abort = &bars->abort;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int r = blockIdx.x / p.n_ctas_per_head, cta_in_head = blockIdx.x % p.n_ctas_per_head;
  const int bidx = r / p.H, hidx = r % p.H;
  const int row0 = cta_in_head * 128;  // first query token of this CTA
  const int nb = p.nb;

  // ------------------------------------------------------------------ set-up
  if (tid == 0) {
    mbar_init(&bars->q_full, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(&bars->s_full[i], 1);
      mbar_init(&bars->p_full[i], 8);  // one arrival per softmax warp
      for (int qq = 0; qq < 4; ++qq) mbar_init(&bars->x_full[i][qq], 2);
      mbar_init(&bars->pv_done[i], 1);
      mbar_init(&bars->k_full[i], 1);
      mbar_init(&bars->k_empty[i], 1);
      mbar_init(&bars->v_full[i], 1);
      mbar_init(&bars->v_empty[i], 1);
    }
    bars->abort = 0;
    bars->bad = 0;
    bars->n_union = 0;
    mbar_fence_init();
  }
  for (int j = tid; j < nb; j += kAttnThreads) tbl[j] = 0u;
  __syncthreads();
  for (int qb = 0; qb < L::QBT; ++qb) {  // scatter: flag bit qb of every key block listed by query block qb
    const int I = cta_in_head * L::QBT + qb;
    if (I >= nb) break;
    const size_t row = (size_t)r * nb + I;
    int cnt = p.dense ? nb : p.kv_cnt[row];
    if (cnt < 0 || cnt > p.idx_stride) {
      bars->bad = 1;
      cnt = cnt < 0 ? 0 : p.idx_stride;
    }
    const int32_t *list = p.kv_idx + row * p.idx_stride;
    for (int t = tid; t < cnt; t += kAttnThreads) {
      const int J = p.dense ? t : list[t];
      if (J < 0 || J >= nb)
        bars->bad = 1;  // skipped, reported
      else
        atomicOr(&tbl[J], 1u << qb);
    }
  }
  if (warp == 1) {
    tmem_alloc(&bars->tmem_base, 512);
    tmem_relinquish();
  }
  __syncthreads();
  if (warp == 0) {  // ascending compaction of the flagged key blocks
    int count = 0;
    for (int base = 0; base < nb; base += 32) {
      const int J = base + lane;
      const uint32_t f = (J < nb) ? tbl[J] : 0u;
      const unsigned ballot = __ballot_sync(0xffffffffu, f != 0u);
      if (f != 0u) uni[count + __popc(ballot & ((1u << lane) - 1u))] = J | (int)(f << 16);
      count += __popc(ballot);
    }
    if (lane == 0) {
      bars->n_union = count;
      if (bars->bad) atomicExch(p.status, HEART_ERR_DEVICE_CHECK);
      tma_prefetch_desc(&map_q);
      tma_prefetch_desc(&map_kv);
      tma_prefetch_desc(&map_v);
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_base;
  const int U = bars->n_union;
  const int NT = (U + SUBS - 1) / SUBS;  // 128-key tiles; tile k belongs to stream k & 1

  // ------------------------------------------------------------------ roles
  if (warp < 2) {
    if (warp == 0 && lane == 0) {  // ===== TMA producer
      mbar_expect_tx(&bars->q_full, L::TILE_BYTES);
      tma_load_4d(Qs, &map_q, &bars->q_full, 0, row0, hidx, bidx);
      tma_load_4d(Qs + 128 * 128, &map_q, &bars->q_full, 64, row0, hidx, bidx);
      int n_k = 0, n_v = 0;  // K and V tiles issued so far
      for (int k = 0; k < NT; ++k) {
        const int s = k & 1, ph = (k >> 1) & 1;
        const int nsub = min(SUBS, U - k * SUBS);
        if (k >= 2 && !mbar_wait(&bars->k_empty[s], ph ^ 1, abort)) break;
        mbar_expect_tx(&bars->k_full[s], nsub * B * 256);
        for (int sub = 0; sub < nsub; ++sub) {
          const int J = uni[k * SUBS + sub] & 0xffff;
          unsigned char *dst = Ks + s * L::TILE_BYTES + sub * (B * 128);
          tma_load_4d(dst, &map_kv, &bars->k_full[s], 0, J * B, hidx, bidx);
          tma_load_4d(dst + 128 * 128, &map_kv, &bars->k_full[s], 64, J * B, hidx, bidx);
        }
        n_k = k + 1;
        if (k >= 2 && !mbar_wait(&bars->v_empty[s], ph ^ 1, abort)) break;
        mbar_expect_tx(&bars->v_full[s], nsub * B * 256);
        for (int sub = 0; sub < nsub; ++sub) {
          const int J = uni[k * SUBS + sub] & 0xffff;
          unsigned char *dst = Vs + s * L::TILE_BYTES + sub * (B * 128);
          tma_load_4d(dst, &map_v, &bars->v_full[s], 0, J * B, hidx, bidx);
          tma_load_4d(dst + 128 * 128, &map_v, &bars->v_full[s], 64, J * B, hidx, bidx);
        }
        n_v = k + 1;
      }
      // Shared memory must not be released under a copy in flight: the Q tile is always awaited here
      // (nobody else does when the union is empty), and after an abort so are the last K/V copies.
      auto settle = [&](uint64_t *bar, uint32_t parity) {
        const long long t0 = clock64();
        while (!mbar_try_wait(bar, parity) && clock64() - t0 < 40000000LL) {
        }
      };
      settle(&bars->q_full, 0);
      if (*abort) {
        for (int k = (n_k > 2 ? n_k - 2 : 0); k < n_k; ++k) settle(&bars->k_full[k & 1], (k >> 1) & 1);
        for (int k = (n_v > 2 ? n_v - 2 : 0); k < n_v; ++k) settle(&bars->v_full[k & 1], (k >> 1) & 1);
      }
    } else if (warp == 1 && lane == 0 && NT > 0) {  // ===== MMA issuer
      constexpr uint32_t idesc_qk_full = idesc_bf16_f32(128, 128, false, false);
      constexpr uint32_t idesc_qk_half = idesc_bf16_f32(128, 64, false, false);
      constexpr uint32_t idesc_pv = idesc_bf16_f32(128, 128, false, true);
      // descriptors differ only in the 14-bit start-address field: base + constant per k-step
      const uint64_t q_desc = smem_desc_sw128(smem_u32(Qs), 16, 1024);
      const uint64_t k_desc = smem_desc_sw128(smem_u32(Ks), 16, 1024);
      const uint64_t v_desc = smem_desc_sw128(smem_u32(Vs), 128 * 128, 1024);
      bool ok = true;
      auto keys_in = [&](int k) -> int { return min(SUBS, U - k * SUBS) * B; };
      // every descriptor is formed once, outside the loop: issuing a tile is 8 back-to-back MMAs
      uint64_t qd[8], kd[2][8], vd[2][8];
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        qd[ks] = q_desc + ((ks >> 2) * 1024 + (ks & 3) * 2);
        kd[0][ks] = k_desc + ((ks >> 2) * 1024 + (ks & 3) * 2);
        kd[1][ks] = kd[0][ks] + (L::TILE_BYTES >> 4);
        vd[0][ks] = v_desc + ks * 128;
        vd[1][ks] = vd[0][ks] + (L::TILE_BYTES >> 4);
      }
      auto issue_qk = [&](int k) {  // S_t = Q K_k^T, t = k & 1; K_k sits in stage t
        const int t = k & 1;
        const uint32_t d = tmem + t * 128;
        const uint32_t idesc = keys_in(k) == 128 ? idesc_qk_full : idesc_qk_half;
        if (t == 0) {
          mma_ss(d, qd[0], kd[0][0], idesc, 0u);
#pragma unroll
          for (int ks = 1; ks < 8; ++ks) mma_ss(d, qd[ks], kd[0][ks], idesc, 1u);
        } else {
          mma_ss(d, qd[0], kd[1][0], idesc, 0u);
#pragma unroll
          for (int ks = 1; ks < 8; ++ks) mma_ss(d, qd[ks], kd[1][ks], idesc, 1u);
        }
        tc_commit(&bars->s_full[t]);
        tc_commit(&bars->k_empty[t]);
      };
      auto issue_pv = [&](int k) {  // O_t (+)= P_t V_k
        const int t = k & 1;
        const uint32_t d = tmem + 256 + t * 128, pa = tmem + t * 128;
        const int ksteps = keys_in(k) / 16;
        if (t == 0) {
          mma_ts(d, pa, vd[0][0], idesc_pv, k >= 2 ? 1u : 0u);
#pragma unroll
          for (int ks = 1; ks < 8; ++ks)
            if (ks < ksteps) mma_ts(d, pa + ks * 8, vd[0][ks], idesc_pv, 1u);
        } else {
          mma_ts(d, pa, vd[1][0], idesc_pv, k >= 2 ? 1u : 0u);
#pragma unroll
          for (int ks = 1; ks < 8; ++ks)
            if (ks < ksteps) mma_ts(d, pa + ks * 8, vd[1][ks], idesc_pv, 1u);
        }
        tc_commit(&bars->pv_done[t]);
        tc_commit(&bars->v_empty[t]);
      };
      ok = mbar_wait(&bars->q_full, 0, abort);
      for (int k = 0; k < 2 && k < NT && ok; ++k) {
        ok = mbar_wait(&bars->k_full[k], 0, abort);
        if (ok) {
          tc_fence_after();
          issue_qk(k);
        }
      }
      for (int k = 0; k < NT && ok; ++k) {
        const int t = k & 1, ph = (k >> 1) & 1;
        ok = mbar_wait(&bars->v_full[t], ph, abort);
        if (ok) ok = mbar_wait(&bars->p_full[t], ph, abort);
        if (!ok) break;
        tc_fence_after();
        issue_pv(k);
        if (k + 2 < NT) {
          ok = mbar_wait(&bars->k_full[t], ph ^ 1, abort);
          if (!ok) break;
          tc_fence_after();
          issue_qk(k + 2);
        }
      }
    }
  } else {
    // ===== softmax / correction / epilogue: thread = (query row, half of the key columns), both streams
    // The stream index t is a run-time value on purpose: one compact copy of this code serves both
    // streams, which keeps the loop inside the instruction cache.
    const int a = (warp - 2) >> 2;  // column half: S columns [64a, 64a+64), O columns [64a, 64a+64)
    const int q = warp & 3;         // TMEM lane quarter this warp may touch
    const int row = q * 32 + lane;  // row inside the 128-row query tile
    const uint32_t lane_addr = tmem + ((uint32_t)(q * 32) << 16);
    const float c = p.scale_log2;
    float m_ref0 = -INFINITY, m_ref1 = -INFINITY, l_part0 = 0.f, l_part1 = 0.f;
    bool ok = true;
    const int my_sub = (a * 64) / B;             // key sub-block this thread's columns belong to
    const int col_in_sub = a * 64 - my_sub * B;  // first of its columns inside that sub-block
    const uint32_t my_bit = 1u << (row / B);     // query block of this row (uniform within a warp)
    for (int k = 0; k < NT && ok; ++k) {
      const int t = k & 1, n_act = k >> 1;
      const int nsub = min(SUBS, U - k * SUBS);
      // valid key columns, for this row, of the thread's two 32-column chunks
      int lim0 = 0, lim1 = 0;
      if (my_sub < nsub) {
        const uint32_t e = (uint32_t)uni[k * SUBS + my_sub];
        if ((e >> 16) & my_bit) {
          const int v = min(B, p.N - (int)(e & 0xffff) * B) - col_in_sub;
          lim0 = max(0, min(32, v));
          lim1 = max(0, min(32, v - 32));
        }
      }
      float m_ref = t ? m_ref1 : m_ref0;
      const uint32_t s_addr = lane_addr + t * 128 + a * 64;
      const uint32_t o_addr = lane_addr + 256 + t * 128 + a * 64;
      float *xrow = xch + (t * 2) * 128 + row;  // [t][half][row]
      ok = __all_sync(0xffffffffu, mbar_wait(&bars->s_full[t], n_act & 1, abort));
      if (!ok) break;
      tc_fence_after();
      uint32_t sreg[64];
      if (lim0 > 0) tmem_ld32(s_addr, *reinterpret_cast<uint32_t(*)[32]>(&sreg[0]));
      if (lim1 > 0) tmem_ld32(s_addr + 32, *reinterpret_cast<uint32_t(*)[32]>(&sreg[32]));
      tmem_wait_ld();
      if (lim0 < 32 || lim1 < 32) {  // rare: ragged last block or a sub-block this row does not list
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          if (i >= lim0) sreg[i] = 0xff800000u;  // -inf: ignored by the max, 2^-inf = 0
          if (i >= lim1) sreg[32 + i] = 0xff800000u;
        }
      }
      float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
      for (int i = 0; i < 64; i += 8) {
        mx0 = fmax3(mx0, __uint_as_float(sreg[i]), __uint_as_float(sreg[i + 1]));
        mx1 = fmax3(mx1, __uint_as_float(sreg[i + 2]), __uint_as_float(sreg[i + 3]));
        mx2 = fmax3(mx2, __uint_as_float(sreg[i + 4]), __uint_as_float(sreg[i + 5]));
        mx3 = fmax3(mx3, __uint_as_float(sreg[i + 6]), __uint_as_float(sreg[i + 7]));
      }
      // the two column halves of a row exchange their maxima
      const float mx_mine = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
      xrow[a * 128] = mx_mine;
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->x_full[t][q]);
      ok = __all_sync(0xffffffffu, mbar_wait(&bars->x_full[t][q], n_act & 1, abort));
      if (!ok) break;
      const float x_max = fmaxf(mx_mine, xrow[(1 - a) * 128]) * c;  // -inf stays -inf (c > 0)
      float alpha = 1.f;
      bool grow = false;
      if (m_ref == -INFINITY) {
        m_ref = x_max;  // nothing accumulated for this row yet: no rescale needed
      } else if (x_max > m_ref + 8.f) {
        alpha = ex2(m_ref - x_max);
        m_ref = x_max;
        grow = true;
      }
      if (__any_sync(0xffffffffu, grow) && n_act > 0) {
        // O_t must be quiescent: the latest PV of this stream has to be complete
        ok = __all_sync(0xffffffffu, mbar_wait(&bars->pv_done[t], (n_act - 1) & 1, abort));
        if (!ok) break;
        tc_fence_after();
#pragma unroll 1
        for (int ch = 0; ch < 2; ++ch) {
          uint32_t v[32];
          tmem_ld32(o_addr + ch * 32, v);
          tmem_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) * alpha);
          tmem_st32(o_addr + ch * 32, v);
        }
        tmem_wait_st();
      }
      const float neg_m = (m_ref == -INFINITY) ? 0.f : -m_ref;
      // p = 2^(s*c - m), packed to bf16 over columns [32a, 32a+32) of S_t
      float sum0 = 0.f, sum1 = 0.f;
      if (a * 64 < nsub * B) {  // else: sub-block absent from this tile, the PV product skips its keys
#pragma unroll
        for (int ch = 0; ch < 2; ++ch) {
          uint32_t pk[16];
          if ((ch ? lim1 : lim0) == 0) {  // this row lists nothing here: zeros, no exponentials
#pragma unroll
            for (int i = 0; i < 16; ++i) pk[i] = 0u;
          } else
#pragma unroll
          for (int i = 0; i < 32; i += 2) {
            const float p0 = ex2(fmaf(__uint_as_float(sreg[ch * 32 + i]), c, neg_m));
            const float p1 = ex2(fmaf(__uint_as_float(sreg[ch * 32 + i + 1]), c, neg_m));
            // the row sum is taken over the bf16-rounded weights, the ones the PV product really
            // uses, so numerator and denominator carry the same rounding: O stays a weighted mean
            const uint32_t w = pack_bf16x2(p0, p1);
            pk[i >> 1] = w;
            sum0 += __uint_as_float(w << 16);
            sum1 += __uint_as_float(w & 0xffff0000u);
          }
          tmem_st16(lane_addr + t * 128 + a * 32 + ch * 16, pk);
        }
      }
      const float l_new = (t ? l_part1 : l_part0) * alpha + (sum0 + sum1);
      tmem_wait_st();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->p_full[t]);
      if (t) {
        m_ref1 = m_ref;
        l_part1 = l_new;
      } else {
        m_ref0 = m_ref;
        l_part0 = l_new;
      }
    }
    // epilogue: merge the two streams; each warpgroup writes its 64-dim half of the output rows
    const int n0 = (NT + 1) >> 1, n1 = NT >> 1;  // tiles per stream
    const int tok = row0 + row;
    const bool valid_row = tok < p.N;
    float l0 = l_part0, l1 = l_part1;
    if (ok && n0 > 0) {  // the column halves add their partial row sums (stream 0, then stream 1)
      // (own slots, not the ones of the row maxima: a slow partner may still be reading those)
      xch[512 + row + a * 128] = l_part0;
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->x_full[0][q]);
      ok = __all_sync(0xffffffffu, mbar_wait(&bars->x_full[0][q], n0 & 1, abort));
      if (ok) l0 += xch[512 + row + (1 - a) * 128];
      if (ok) ok = __all_sync(0xffffffffu, mbar_wait(&bars->pv_done[0], (n0 - 1) & 1, abort));
    }
    if (ok && n1 > 0) {
      xch[768 + row + a * 128] = l_part1;
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->x_full[1][q]);
      ok = __all_sync(0xffffffffu, mbar_wait(&bars->x_full[1][q], n1 & 1, abort));
      if (ok) l1 += xch[768 + row + (1 - a) * 128];
      if (ok) ok = __all_sync(0xffffffffu, mbar_wait(&bars->pv_done[1], (n1 - 1) & 1, abort));
    }
    if (ok) {
      tc_fence_after();
      const float m = fmaxf(m_ref0, m_ref1);
      const float w0 = (n0 > 0 && m_ref0 > -INFINITY) ? ex2(m_ref0 - m) : 0.f;
      const float w1 = (n1 > 0 && m_ref1 > -INFINITY) ? ex2(m_ref1 - m) : 0.f;
      const float l = l0 * w0 + l1 * w1;
      const float inv = l > 0.f ? 1.f / l : 0.f;
      const float f0 = w0 * inv, f1 = w1 * inv;
      uint16_t *orow = p.O + (long long)bidx * p.sb + (long long)hidx * p.sh + (long long)tok * p.sn + a * 64;
      const uint32_t o_addr = lane_addr + 256 + a * 64;
#pragma unroll 1
      for (int ch = 0; ch < 4; ++ch) {  // 16 output dims at a time
        uint32_t v0[16], v1[16];
        if (n0 > 0) tmem_ld16(o_addr + ch * 16, v0);
        if (n1 > 0) tmem_ld16(o_addr + 128 + ch * 16, v1);
        tmem_wait_ld();
        float o[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          o[i] = 0.f;
          if (n0 > 0) o[i] = __uint_as_float(v0[i]) * f0;
          if (n1 > 0) o[i] = fmaf(__uint_as_float(v1[i]), f1, o[i]);
        }
        if (valid_row) {
#pragma unroll
          for (int g4 = 0; g4 < 2; ++g4) {
            uint4 w;
            w.x = pack_bf16x2(o[g4 * 8 + 0], o[g4 * 8 + 1]);
            w.y = pack_bf16x2(o[g4 * 8 + 2], o[g4 * 8 + 3]);
            w.z = pack_bf16x2(o[g4 * 8 + 4], o[g4 * 8 + 5]);
            w.w = pack_bf16x2(o[g4 * 8 + 6], o[g4 * 8 + 7]);
            *reinterpret_cast<uint4 *>(orow + ch * 16 + g4 * 8) = w;
          }
        }
      }
      if (a == 0 && valid_row && p.lse != nullptr)
        p.lse[(size_t)r * p.N + tok] = l > 0.f ? (m + log2f(l)) * 0.6931471805599453f : -INFINITY;
    }
  }

  // ------------------------------------------------------------------ tear-down
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
  if (tid == 0 && bars->abort) atomicExch(p.status, HEART_ERR_DEVICE_CHECK);
}

// ---------------------------------------------------------------------- host side
namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = []() -> EncodeTiledFn {
    void *sym = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      return nullptr;
    return reinterpret_cast<EncodeTiledFn>(sym);
  }();
  return fn;
}

// bf16 [B,H,N,128] with element strides (sb, sh, sn, 1): box = 64 dims x `rows` tokens, 128-byte swizzle,
// out-of-range rows read as zero.
bool make_map(CUtensorMap *m, const void *base, const Geom &g, int rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[4] = {(cuuint64_t)kD, (cuuint64_t)g.N, (cuuint64_t)g.H, (cuuint64_t)g.B};
  cuuint64_t strides[3] = {(cuuint64_t)g.sn * 2, (cuuint64_t)g.sh * 2, (cuuint64_t)g.sb * 2};
  cuuint32_t box[4] = {64, (cuuint32_t)rows, 1, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int B>
cudaError_t launch_bk(const Geom &g, const CUtensorMap &mq, const CUtensorMap &mk, const CUtensorMap &mv,
                      const AttnParams &prm, cudaStream_t s) {
  const int smem = AttnSmem<B>::TOTAL + 1024;
  cudaError_t e = cudaFuncSetAttribute(attn_tc_kernel<B>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  attn_tc_kernel<B><<<g.R * prm.n_ctas_per_head, kAttnThreads, smem, s>>>(mq, mk, mv, prm);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_attention(const Geom &g, const void *Q, const void *K, const void *V,
                             const int32_t *kv_idx, const int32_t *kv_cnt, bool dense, void *O,
                             float *lse, int32_t *status, cudaStream_t s, int *launches) {
  CUtensorMap mq, mk, mv;
  if (!make_map(&mq, Q, g, 128) || !make_map(&mk, K, g, g.block) || !make_map(&mv, V, g, g.block))
    return cudaErrorInvalidValue;
  AttnParams prm;
  prm.kv_idx = kv_idx;
  prm.kv_cnt = kv_cnt;
  prm.O = static_cast<uint16_t *>(O);
  prm.lse = lse;
  prm.status = status;
  prm.sb = g.sb;
  prm.sh = g.sh;
  prm.sn = g.sn;
  prm.H = g.H;
  prm.N = g.N;
  prm.nb = g.nb;
  prm.idx_stride = g.idx_stride;
  prm.n_ctas_per_head = (g.N + 127) / 128;
  prm.dense = dense ? 1 : 0;
  prm.scale_log2 = (float)(g.scale * 1.4426950408889634);
  ++*launches;
  return g.block == 64 ? launch_bk<64>(g, mq, mk, mv, prm, s) : launch_bk<128>(g, mq, mk, mv, prm, s);
}

}  // namespace heart
