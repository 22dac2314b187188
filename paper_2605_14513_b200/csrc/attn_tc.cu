// Block-sparse attention with online softmax on the sm_100a tensor cores.
//
// One CTA owns 256 consecutive query rows of one head = two 128-row MMA tiles (tile t = rows
// [128t, 128t+128)).  With 128-token blocks a tile is one query block; with 64-token blocks it is two
// query blocks whose lists are merged (rows of the half that does not list a key block see -inf).
// The lists of the CTA's 2 or 4 query blocks are merged once into an ascending union; each union
// entry carries one flag bit per query block.  K/V blocks are fetched once per CTA and shared by
// both tiles; a tile skips the MMAs of union entries none of its query blocks lists.
//
// Warp roles (384 threads):
//   warp 0      TMA producer: Q tiles once, then the listed K and V blocks through shared-memory
//               rings (cp.async.bulk.tensor, 128-byte swizzle, completion on mbarriers).
//   warp 1      MMA issuer (one lane): S_t = Q_t K^T into tensor memory (tcgen05.mma, operands in
//               shared memory), O_t += P_t V with P_t read from tensor memory; the two tiles are
//               interleaved so one tile's softmax overlaps the other tile's MMAs.
//   warps 4-7   softmax of tile 0, warps 8-11 softmax of tile 1: thread = query row; reads its S
//               row from tensor memory, keeps the running max / sum, writes P (bf16) back over S,
//               rescales O only when the max grew by more than 2^8, and writes O / lse at the end.
// Tensor memory (512 columns): S0 | S1 | O0 | O1, 128 fp32 columns each; P_t aliases S_t.
//
// Every wait is bounded; a wait that runs out raises a CTA-wide abort flag and the status word, the
// roles drain, tensor memory is freed and the CTA exits.
#include <cuda.h>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace heart {
using namespace tc;

constexpr int kAttnThreads = 384;
constexpr int kMaxNb = HEART_MAX_BLOCKS;

template <int BK>
struct AttnSmem {
  static constexpr int NQB = 256 / BK;            // query blocks per CTA
  static constexpr int QBT = 128 / BK;            // query blocks per 128-row tile
  static constexpr int NS = (BK == 128) ? 2 : 4;  // ring depth of K and of V
  static constexpr int Q_BYTES = 128 * 256;       // one Q tile  [2 halves][128 rows][64] bf16
  static constexpr int KV_BYTES = BK * 256;       // one K/V tile [2 halves][BK rows][64] bf16
  static constexpr int OFF_Q = 0;
  static constexpr int OFF_K = OFF_Q + 2 * Q_BYTES;
  static constexpr int OFF_V = OFF_K + NS * KV_BYTES;
  static constexpr int OFF_UNI = OFF_V + NS * KV_BYTES;  // int32[kMaxNb]: J | flags << 16
  static constexpr int OFF_TBL = OFF_UNI + 4 * kMaxNb;   // uint32[kMaxNb]: flags per key block
  static constexpr int OFF_BAR = OFF_TBL + 4 * kMaxNb;   // mbarriers and scalars
  static constexpr int TOTAL = OFF_BAR + 512;
};

struct AttnBars {
  uint64_t q_full[2];
  uint64_t k_full[4], k_empty[4], v_full[4], v_empty[4];
  uint64_t s_full[2], p_full[2], pv_done[2];
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

template <int BK>
__global__ void __launch_bounds__(kAttnThreads, 1)
    attn_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_kv,
                   const __grid_constant__ CUtensorMap map_v, const AttnParams p) {
  using L = AttnSmem<BK>;
  extern __shared__ unsigned char smem_dyn[];
  unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) &
                                                          ~static_cast<uintptr_t>(1023));
  unsigned char *Qs = smem + L::OFF_Q, *Ks = smem + L::OFF_K, *Vs = smem + L::OFF_V;
  int32_t *uni = reinterpret_cast<int32_t *>(smem + L::OFF_UNI);
  uint32_t *tbl = reinterpret_cast<uint32_t *>(smem + L::OFF_TBL);
  AttnBars *bars = reinterpret_cast<AttnBars *>(smem + L::OFF_BAR);
  volatile int *abort = &bars->abort;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int r = blockIdx.x / p.n_ctas_per_head, cta_in_head = blockIdx.x % p.n_ctas_per_head;
  const int bidx = r / p.H, hidx = r % p.H;
  const int row0 = cta_in_head * 256;  // first query token of this CTA
  const int nb = p.nb;

  // ------------------------------------------------------------------ set-up
  if (tid == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(&bars->q_full[i], 1);
      mbar_init(&bars->s_full[i], 1);
      mbar_init(&bars->p_full[i], 128);
      mbar_init(&bars->pv_done[i], 1);
    }
    for (int i = 0; i < 4; ++i) {
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
  for (int qb = 0; qb < L::NQB; ++qb) {  // scatter: flag bit qb of every key block listed by query block qb
    const int I = cta_in_head * L::NQB + qb;
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
  const uint32_t tile_mask0 = (1u << L::QBT) - 1u;

  // ------------------------------------------------------------------ roles
  if (warp == 0) {
    if (lane == 0) {  // ===== TMA producer
      for (int t = 0; t < 2; ++t) {
        const int tr = row0 + t * 128;
        if (tr < p.N) {
          mbar_expect_tx(&bars->q_full[t], L::Q_BYTES);
          tma_load_4d(Qs + t * L::Q_BYTES, &map_q, &bars->q_full[t], 0, tr, hidx, bidx);
          tma_load_4d(Qs + t * L::Q_BYTES + 128 * 128, &map_q, &bars->q_full[t], 64, tr, hidx, bidx);
        }
      }
      int n_k = 0, n_v = 0;  // K and V loads issued so far
      for (int u = 0; u < U; ++u) {
        const int s = u % L::NS, ph = (u / L::NS) & 1;
        const int J = uni[u] & 0xffff;
        if (u >= L::NS && !mbar_wait(&bars->k_empty[s], ph ^ 1, abort)) break;
        mbar_expect_tx(&bars->k_full[s], L::KV_BYTES);
        tma_load_4d(Ks + s * L::KV_BYTES, &map_kv, &bars->k_full[s], 0, J * BK, hidx, bidx);
        tma_load_4d(Ks + s * L::KV_BYTES + BK * 128, &map_kv, &bars->k_full[s], 64, J * BK, hidx, bidx);
        n_k = u + 1;
        if (u >= L::NS && !mbar_wait(&bars->v_empty[s], ph ^ 1, abort)) break;
        mbar_expect_tx(&bars->v_full[s], L::KV_BYTES);
        tma_load_4d(Vs + s * L::KV_BYTES, &map_v, &bars->v_full[s], 0, J * BK, hidx, bidx);
        tma_load_4d(Vs + s * L::KV_BYTES + BK * 128, &map_v, &bars->v_full[s], 64, J * BK, hidx, bidx);
        n_v = u + 1;
      }
      // Shared memory must not be released under a copy in flight: the Q tiles are always awaited here
      // (nobody else does when the union is empty), and after an abort so are the last K/V copies.
      auto settle = [&](uint64_t *bar, uint32_t parity) {
        const long long t0 = clock64();
        while (!mbar_try_wait(bar, parity) && clock64() - t0 < 40000000LL) {
        }
      };
      for (int t = 0; t < 2; ++t)
        if (row0 + t * 128 < p.N) settle(&bars->q_full[t], 0);
      if (*abort) {
        for (int u = (n_k > L::NS ? n_k - L::NS : 0); u < n_k; ++u) settle(&bars->k_full[u % L::NS], (u / L::NS) & 1);
        for (int u = (n_v > L::NS ? n_v - L::NS : 0); u < n_v; ++u) settle(&bars->v_full[u % L::NS], (u / L::NS) & 1);
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && U > 0) {  // ===== MMA issuer
      constexpr uint32_t idesc_qk = idesc_bf16_f32(128, BK, false, false);
      constexpr uint32_t idesc_pv = idesc_bf16_f32(128, 128, false, true);
      const uint32_t q_addr = smem_u32(Qs), k_addr = smem_u32(Ks), v_addr = smem_u32(Vs);
      uint32_t fresh_mask = 3u;  // bit t: O_t has not been written yet
      int n_pv0 = 0, n_pv1 = 0;
      bool ok = true;
      auto active = [&](int u, int t) -> bool {
        return (((uint32_t)uni[u] >> 16) & (tile_mask0 << (t * L::QBT))) != 0u;
      };
      auto issue_qk = [&](int t, int u) {
        const int s = u % L::NS;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          const uint64_t a = smem_desc_sw128(q_addr + t * L::Q_BYTES + (ks >> 2) * (128 * 128) + (ks & 3) * 32, 16, 1024);
          const uint64_t b = smem_desc_sw128(k_addr + s * L::KV_BYTES + (ks >> 2) * (BK * 128) + (ks & 3) * 32, 16, 1024);
          mma_ss(tmem + t * 128, a, b, idesc_qk, ks > 0 ? 1u : 0u);
        }
        tc_commit(&bars->s_full[t]);
      };
      auto issue_pv = [&](int t, int u) {
        const int s = u % L::NS;
#pragma unroll
        for (int ks = 0; ks < BK / 16; ++ks) {
          const uint64_t b = smem_desc_sw128(v_addr + s * L::KV_BYTES + ks * 2048, BK * 128, 1024);
          mma_ts(tmem + 256 + t * 128, tmem + t * 128 + ks * 8, b, idesc_pv, (((fresh_mask >> t) & 1u) && ks == 0) ? 0u : 1u);
        }
        fresh_mask &= ~(1u << t);
        tc_commit(&bars->pv_done[t]);
      };
      for (int t = 0; t < 2 && ok; ++t)
        if (row0 + t * 128 < p.N) ok = mbar_wait(&bars->q_full[t], 0, abort);
      if (ok) ok = mbar_wait(&bars->k_full[0], 0, abort);
      if (ok) {
        tc_fence_after();
        if (active(0, 0)) issue_qk(0, 0);
        if (active(0, 1)) issue_qk(1, 0);
        tc_commit(&bars->k_empty[0]);
      }
      for (int u = 0; u < U && ok; ++u) {
        const int s = u % L::NS, ph = (u / L::NS) & 1;
        const bool more = (u + 1 < U);
        ok = mbar_wait(&bars->v_full[s], ph, abort);
        if (ok && more) ok = mbar_wait(&bars->k_full[(u + 1) % L::NS], ((u + 1) / L::NS) & 1, abort);
        if (!ok) break;
        tc_fence_after();
        for (int t = 0; t < 2 && ok; ++t) {
          if (active(u, t)) {
            int &n_pv = t ? n_pv1 : n_pv0;
            ok = mbar_wait(&bars->p_full[t], n_pv & 1, abort);
            if (!ok) break;
            ++n_pv;
            tc_fence_after();
            issue_pv(t, u);
          }
          if (more && active(u + 1, t)) issue_qk(t, u + 1);
        }
        if (!ok) break;
        tc_commit(&bars->v_empty[s]);
        if (more) tc_commit(&bars->k_empty[(u + 1) % L::NS]);
      }
    }
  } else if (warp >= 4) {
    // ===== softmax / correction / epilogue: warpgroup t handles tile t, thread = query row
    const int t = (warp - 4) >> 2;
    const int q = warp & 3;                 // TMEM lane quarter this warp may touch
    const int row_in_tile = q * 32 + lane;
    const int tok = row0 + t * 128 + row_in_tile;
    const bool valid_row = tok < p.N;
    const uint32_t my_bit = 1u << (t * L::QBT + row_in_tile / BK);
    const uint32_t my_tile_mask = tile_mask0 << (t * L::QBT);
    const uint32_t s_addr = tmem + ((uint32_t)(q * 32) << 16) + t * 128;
    const uint32_t o_addr = tmem + ((uint32_t)(q * 32) << 16) + 256 + t * 128;
    const float c = p.scale_log2;
    float m_ref = -INFINITY, l = 0.f;
    int n_act = 0;
    bool ok = true;
    for (int u = 0; u < U && ok; ++u) {
      const uint32_t e = (uint32_t)uni[u];
      if (((e >> 16) & my_tile_mask) == 0u) continue;
      const int J = e & 0xffff;
      const bool row_has = ((e >> 16) & my_bit) != 0u;
      const int kv_valid = row_has ? min(BK, p.N - J * BK) : 0;
      ok = __all_sync(0xffffffffu, mbar_wait(&bars->s_full[t], n_act & 1, abort));
      if (!ok) break;
      tc_fence_after();
      // pass 1: row maximum of the raw scores
      float mx = -INFINITY;
#pragma unroll
      for (int ch = 0; ch < BK / 32; ++ch) {
        uint32_t v[32];
        tmem_ld32(s_addr + ch * 32, v);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 32; ++i)
          if (ch * 32 + i < kv_valid) mx = fmaxf(mx, __uint_as_float(v[i]));
      }
      const float x_max = mx * c;  // -inf stays -inf (c > 0)
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
        // O_t must be quiescent: the latest PV of this tile has to be complete
        ok = __all_sync(0xffffffffu, mbar_wait(&bars->pv_done[t], (n_act - 1) & 1, abort));
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) {
          uint32_t v[32];
          tmem_ld32(o_addr + ch * 32, v);
          tmem_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) * alpha);
          tmem_st32(o_addr + ch * 32, v);
        }
        tmem_wait_st();
      }
      l *= alpha;
      const float m_use = (m_ref == -INFINITY) ? 0.f : m_ref;
      // pass 2: p = 2^(s*c - m), packed to bf16 over the first BK/2 columns of S_t
      float sum = 0.f;
#pragma unroll
      for (int ch = 0; ch < BK / 32; ++ch) {
        uint32_t v[32], pk[16];
        tmem_ld32(s_addr + ch * 32, v);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
          const float p0 = (ch * 32 + i < kv_valid) ? ex2(fmaf(__uint_as_float(v[i]), c, -m_use)) : 0.f;
          const float p1 = (ch * 32 + i + 1 < kv_valid) ? ex2(fmaf(__uint_as_float(v[i + 1]), c, -m_use)) : 0.f;
          // the row sum is taken over the bf16-rounded weights, the ones the PV product really uses,
          // so numerator and denominator carry the same rounding and O stays a true weighted mean
          const uint32_t w = pack_bf16x2(p0, p1);
          pk[i >> 1] = w;
          sum += __uint_as_float(w << 16) + __uint_as_float(w & 0xffff0000u);
        }
        tmem_st16(s_addr + ch * 16, pk);
      }
      l += sum;
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(&bars->p_full[t]);
      ++n_act;
    }
    // epilogue
    if (ok && n_act > 0) ok = __all_sync(0xffffffffu, mbar_wait(&bars->pv_done[t], (n_act - 1) & 1, abort));
    if (ok) {
      tc_fence_after();
      const float inv = l > 0.f ? 1.f / l : 0.f;
      uint16_t *orow = p.O + (long long)bidx * p.sb + (long long)hidx * p.sh + (long long)tok * p.sn;
#pragma unroll
      for (int ch = 0; ch < 4; ++ch) {
        uint32_t v[32];
        if (n_act > 0) {
          tmem_ld32(o_addr + ch * 32, v);
          tmem_wait_ld();
        } else {
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] = 0u;
        }
        if (valid_row) {
#pragma unroll
          for (int g4 = 0; g4 < 4; ++g4) {
            uint4 o;
            o.x = pack_bf16x2(__uint_as_float(v[g4 * 8 + 0]) * inv, __uint_as_float(v[g4 * 8 + 1]) * inv);
            o.y = pack_bf16x2(__uint_as_float(v[g4 * 8 + 2]) * inv, __uint_as_float(v[g4 * 8 + 3]) * inv);
            o.z = pack_bf16x2(__uint_as_float(v[g4 * 8 + 4]) * inv, __uint_as_float(v[g4 * 8 + 5]) * inv);
            o.w = pack_bf16x2(__uint_as_float(v[g4 * 8 + 6]) * inv, __uint_as_float(v[g4 * 8 + 7]) * inv);
            *reinterpret_cast<uint4 *>(orow + ch * 32 + g4 * 8) = o;
          }
        }
      }
      if (valid_row && p.lse != nullptr)
        p.lse[(size_t)r * p.N + tok] = l > 0.f ? (m_ref + log2f(l)) * 0.6931471805599453f : -INFINITY;
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

template <int BK>
cudaError_t launch_bk(const Geom &g, const CUtensorMap &mq, const CUtensorMap &mk, const CUtensorMap &mv,
                      const AttnParams &prm, cudaStream_t s) {
  const int smem = AttnSmem<BK>::TOTAL + 1024;
  cudaError_t e = cudaFuncSetAttribute(attn_tc_kernel<BK>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  attn_tc_kernel<BK><<<g.R * prm.n_ctas_per_head, kAttnThreads, smem, s>>>(mq, mk, mv, prm);
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
  prm.n_ctas_per_head = (g.N + 255) / 256;
  prm.dense = dense ? 1 : 0;
  prm.scale_log2 = (float)(g.scale * 1.4426950408889634);
  ++*launches;
  return g.block == 64 ? launch_bk<64>(g, mq, mk, mv, prm, s) : launch_bk<128>(g, mq, mk, mv, prm, s);
}

}  // namespace heart
