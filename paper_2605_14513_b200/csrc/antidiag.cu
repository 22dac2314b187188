// Strided antidiagonal block-importance estimator on the sm_100a tensor cores -- the estimator
// family of the paper's main backbone (appendix "XAttention and SVG2 Configurations": anti-diagonal
// scoring with stride 16; the paper gives the stride and the block size only, the definition is
// this library's):
//   groups of s = 16 consecutive tokens; only the Ns = floor(N / s) full groups are sampled;
//   S'(a, c) = (scale / s) * sum_t <q_{a s + t}, k_{c s + s-1-t}>      (antidiagonal mean of a tile)
//   P'(a, .) = softmax over the groups c;  importance(I, J) = sum of P' over the groups of the two
//   blocks / number of groups in I;  then the same top-p selection as the pooled estimator.
//
// The contraction is a bf16 GEMM per head on the very memory of Q and K: row a of the left operand
// is the 16 tokens of group a laid end to end (16 x 128 values), row c of the right operand the 16
// tokens of group c in reverse order.  A 5-D tensor map (dim, token in group, group, head, batch)
// lets one TMA box fetch "token t of 128 (or 256) consecutive groups", which is exactly a K-major
// operand tile; reversing the key tokens is a change of one box coordinate.
//
// antidiag_scores_kernel: one CTA per (128 groups of queries, head); it walks over all key groups,
// 256 at a time.  Warp 0 issues the TMA loads into a four-stage ring (one stage = 64 dims of one
// token position: 16 KB of Q + 32 KB of K), warp 1 issues tcgen05.mma (M = 128, N = 256, 4 x K = 16
// per stage, 32 stages per tile) into one of two 256-column accumulators in tensor memory, warps
// 2-5 drain the other accumulator: one thread per query group, and for every key block of the tile
// the pair (max, sum of 2^(x - max)) over the block's 4 or 8 groups goes to the workspace.
// antidiag_reduce_kernel (fp64) turns the pairs of the groups of one query block into the log of
// the block importances, which top_p_kernel consumes like pooled scores.
#include <cuda.h>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace heart {
using namespace tc;

namespace {

constexpr int kS = HEART_ANTIDIAG_STRIDE;  // tokens per group
constexpr int kMt = 128;                   // query groups per CTA
constexpr int kNt = 256;                   // key groups per accumulator tile
constexpr int kStagesAd = 4;
constexpr int kABytes = kMt * 128, kBBytes = kNt * 128, kStageBytes = kABytes + kBBytes;
constexpr int kKSteps = kS * 2;            // ring stages per tile: 16 token positions x 2 halves of the head dim
constexpr int kThreadsAd = 192;

struct AdBars {
  uint64_t full[kStagesAd], empty[kStagesAd];
  uint64_t acc_full[2], acc_empty[2];
  uint64_t drain;
  uint32_t tmem_base;
  int abort;
};

struct AdParams {
  float2 *pairs;          // [R][Ns][nb]: (max, sum) in the log2 domain per (query group, key block)
  const uint8_t *refresh;
  int32_t *status;
  int H, Ns, nb, g;       // g = groups per block
  float c2;               // (scale / s) * log2(e)
};

__device__ __forceinline__ void tma_load_5d(void *smem_dst, const CUtensorMap *map, uint64_t *bar, int c0, int c1,
                                            int c2, int c3, int c4) {
  asm volatile(
      "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];"
      ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2),
      "r"(c3), "r"(c4)
      : "memory");
}

template <int G>  // groups per block: 4 (64-token blocks) or 8 (128-token blocks)
__global__ void __launch_bounds__(kThreadsAd, 1)
    antidiag_scores_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                           const AdParams p) {
  const int r = blockIdx.y;
  if (p.refresh != nullptr && p.refresh[r] == 0) return;  // reuse branch of Algorithm 1: nothing to predict
  extern __shared__ unsigned char smem_dyn[];
  unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) &
                                                          ~static_cast<uintptr_t>(1023));
  AdBars *bars = reinterpret_cast<AdBars *>(smem + kStagesAd * kStageBytes);
  volatile int *abort = &bars->abort;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int bidx = r / p.H, hidx = r % p.H;
  const int a0 = blockIdx.x * kMt;
  // The key groups are dealt to gridDim.z CTAs per (row tile, head): every key block's pair is written
  // by exactly one of them, so nothing has to be combined.  This CTA takes tiles [tile0, tile0 + n_tiles).
  const int all_tiles = (p.Ns + kNt - 1) / kNt;
  const int tile0 = (int)((long long)all_tiles * blockIdx.z / gridDim.z);
  const int n_tiles = (int)((long long)all_tiles * (blockIdx.z + 1) / gridDim.z) - tile0;
  const int n_steps = n_tiles * kKSteps;

  if (tid == 0) {
    for (int i = 0; i < kStagesAd; ++i) {
      mbar_init(&bars->full[i], 1);
      mbar_init(&bars->empty[i], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&bars->acc_full[i], 1);
      mbar_init(&bars->acc_empty[i], 4);  // one arrival per draining warp
    }
    mbar_init(&bars->drain, 1);
    bars->abort = 0;
    mbar_fence_init();
  }
  if (warp == 1) {
    tmem_alloc(&bars->tmem_base, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_base;
  auto settle = [&](uint64_t *bar, uint32_t parity) {
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity) && clock64() - t0 < 40000000LL) {
    }
  };

  if (warp == 0) {
    if (lane == 0) {  // ===== TMA producer
      tma_prefetch_desc(&map_q);
      tma_prefetch_desc(&map_k);
      int issued = 0;
      for (int it = 0; it < n_steps; ++it) {
        const int st = it % kStagesAd, n = it / kStagesAd;
        if (n >= 1 && !mbar_wait_relaxed(&bars->empty[st], (n - 1) & 1, abort)) break;
        const int tile = it / kKSteps, ks = it % kKSteps, t = ks >> 1, dh = ks & 1;
        unsigned char *dst = smem + st * kStageBytes;
        mbar_expect_tx(&bars->full[st], kStageBytes);
        // token t of the query groups a0 .. a0+127; token s-1-t of the key groups of this tile
        tma_load_5d(dst, &map_q, &bars->full[st], dh * 64, t, a0, hidx, bidx);
        tma_load_5d(dst + kABytes, &map_k, &bars->full[st], dh * 64, kS - 1 - t, (tile0 + tile) * kNt, hidx, bidx);
        issued = it + 1;
      }
      if (*abort)  // shared memory must not be released under a copy in flight
        for (int it = (issued > kStagesAd ? issued - kStagesAd : 0); it < issued; ++it)
          settle(&bars->full[it % kStagesAd], (it / kStagesAd) & 1);
    }
  } else if (warp == 1) {
    // ===== MMA issuer: the whole warp runs the loop, one elected lane issues
    constexpr uint32_t idesc = idesc_bf16_f32(kMt, kNt, false, false);
    auto at = [](uint64_t desc, uint32_t off16) -> uint64_t {
      return (desc & 0xffffffff00000000ull) | (uint32_t)((uint32_t)desc + off16);
    };
    const bool leader = elect_one();
    const uint64_t a_desc0 = smem_desc_sw128(smem_u32(smem), 16, 1024);
    const uint64_t b_desc0 = smem_desc_sw128(smem_u32(smem + kABytes), 16, 1024);
    bool ok = true;
    int it = 0;
    for (int tile = 0; tile < n_tiles && ok; ++tile) {
      const int buf = tile & 1, m = tile >> 1;
      if (m >= 1) ok = mbar_wait(&bars->acc_empty[buf], (m - 1) & 1, abort);
      if (!ok) break;
      tc_fence_after();
      const uint32_t d = tmem + buf * kNt;
      for (int ks = 0; ks < kKSteps && ok; ++ks, ++it) {
        const int st = it % kStagesAd, n = it / kStagesAd;
        ok = mbar_wait(&bars->full[st], n & 1, abort);
        if (!ok) break;
        tc_fence_after();
        const uint64_t a_desc = at(a_desc0, st * (kStageBytes >> 4)), b_desc = at(b_desc0, st * (kStageBytes >> 4));
        if (leader) {
#pragma unroll
          for (int k = 0; k < 4; ++k) mma_ss(d, at(a_desc, k * 2), at(b_desc, k * 2), idesc, (ks > 0 || k > 0) ? 1u : 0u);
          tc_commit(&bars->empty[st]);
          if (ks == kKSteps - 1) tc_commit(&bars->acc_full[buf]);
        }
        __syncwarp();
      }
    }
    if (*abort) {  // tensor memory must not be released under a product in flight
      if (leader) tc_commit(&bars->drain);
      __syncwarp();
      settle(&bars->drain, 0);
    }
  } else {
    // ===== drain: thread = one query group; per key block of the tile a (max, sum) pair
    const int q = warp & 3;  // the lane quarter of tensor memory this warp may read
    const int a = a0 + q * 32 + lane;
    const uint32_t lane_addr = tmem + ((uint32_t)(q * 32) << 16);
    float2 *out = p.pairs + ((size_t)r * p.Ns + (a < p.Ns ? a : 0)) * p.nb;
    bool ok = true;
    for (int tile = 0; tile < n_tiles && ok; ++tile) {
      const int buf = tile & 1, m = tile >> 1;
      ok = __all_sync(0xffffffffu, mbar_wait(&bars->acc_full[buf], m & 1, abort));
      if (!ok) break;
      tc_fence_after();
      const int c0 = (tile0 + tile) * kNt;
#pragma unroll 1
      for (int ch = 0; ch < kNt / 32; ++ch) {
        if (c0 + ch * 32 >= p.Ns) break;  // (uniform) nothing but padding from here on
        uint32_t v[32];
        tmem_ld32(lane_addr + buf * kNt + ch * 32, v);
        tmem_wait_ld();
#pragma unroll
        for (int j = 0; j < 32 / G; ++j) {
          const int cb = c0 + ch * 32 + j * G;  // first group of this key block
          float mx = -INFINITY;
#pragma unroll
          for (int i = 0; i < G; ++i)
            if (cb + i < p.Ns) mx = fmaxf(mx, __uint_as_float(v[j * G + i]));
          float l = 0.f;
          const float mc = mx * p.c2;
#pragma unroll
          for (int i = 0; i < G; ++i)
            if (cb + i < p.Ns) l += ex2(fmaf(__uint_as_float(v[j * G + i]), p.c2, -mc));
          if (cb < p.Ns && a < p.Ns) out[cb / G] = make_float2(mc, l);
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->acc_empty[buf]);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
  if (tid == 0 && bars->abort) atomicExch(p.status, HEART_ERR_DEVICE_CHECK);
}

// One CTA per (query block I, head r), fp64: the (max, sum) pairs of the block's groups become
// scores[r][I][J] = ln(importance(I, J)) (-inf for importance 0), which the top-p kernel reads like
// pooled scores.  A query block without a full group gets equal scores (uniform importance).
// One warp per group of the block (at most 8): row maximum and row sum by shuffles, the weights of
// the lane's key blocks stay in registers in between; the groups are then added into the block's
// weights one after the other.  Every reduction has a fixed shape: bit-reproducible.
template <int NJ>  // NJ * 32 >= n_b
__global__ void __launch_bounds__(256, 2) antidiag_reduce_kernel(const float2 *__restrict__ pairs, int Ns, int nb,
                                                                 int g, int pitch, const uint8_t *__restrict__ refresh,
                                                                 double *__restrict__ scores) {
  const int I = blockIdx.x, r = blockIdx.y;
  if (refresh != nullptr && refresh[r] == 0) return;
  __shared__ double wgt[HEART_MAX_BLOCKS];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int a0 = I * g, a1 = min(a0 + g, Ns);
  const int nJ = (Ns + g - 1) / g;  // key blocks that hold at least one full group
  double *srow = scores + ((size_t)r * nb + I) * pitch;
  if (a1 <= a0) {
    for (int J = tid; J < pitch; J += 256) srow[J] = 0.0;
    return;
  }
  for (int J = tid; J < nb; J += 256) wgt[J] = 0.0;
  constexpr int kPerLane = NJ;
  const double ln2 = 0.6931471805599453;
  double e[kPerLane];
  double inv_z = 0.0;
  const int a = a0 + warp;  // this warp's group (g <= 8 warps have one)
  if (warp < g && a < a1) {
    const float2 *prow = pairs + ((size_t)r * Ns + a) * nb;
    float mxf = -INFINITY;
#pragma unroll
    for (int k = 0; k < kPerLane; ++k)
      if (lane + 32 * k < nJ) mxf = fmaxf(mxf, prow[lane + 32 * k].x);
    double mx = (double)mxf;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmax(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    double z = 0.0;
#pragma unroll
    for (int k = 0; k < kPerLane; ++k) {
      e[k] = 0.0;
      if (lane + 32 * k < nJ) {  // (the row is in L1 / L2 from the pass above)
        const float2 pr = prow[lane + 32 * k];
        e[k] = exp_nonpositive(((double)pr.x - mx) * ln2) * (double)pr.y;
      }
      z += e[k];
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
    inv_z = 1.0 / z;
  }
  __syncthreads();
  for (int aa = 0; aa < g; ++aa) {  // groups in ascending order: a fixed summation order
    if (warp == aa && a < a1) {
#pragma unroll
      for (int k = 0; k < kPerLane; ++k)
        if (lane + 32 * k < nJ) wgt[lane + 32 * k] += e[k] * inv_z;
    }
    __syncthreads();
  }
  const double inv = 1.0 / (double)(a1 - a0);
  for (int J = tid; J < pitch; J += 256) {
    const double w = (J < nJ) ? wgt[J] * inv : 0.0;
    srow[J] = (w > 0.0) ? log(w) : -INFINITY;
  }
}

// bf16 [B,H,N,128] seen as (dim, token in group, group, head, batch); box = 64 dims of one token
// position of `rows` consecutive groups, 128-byte swizzle, groups past Ns read as zero.
bool make_group_map(CUtensorMap *m, const void *base, const Geom &g, int Ns, int rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  cuuint64_t dims[5] = {(cuuint64_t)kD, (cuuint64_t)kS, (cuuint64_t)Ns, (cuuint64_t)g.H, (cuuint64_t)g.B};
  cuuint64_t strides[4] = {(cuuint64_t)g.sn * 2, (cuuint64_t)g.sn * 2 * kS, (cuuint64_t)g.sh * 2, (cuuint64_t)g.sb * 2};
  cuuint32_t box[5] = {64, 1, (cuuint32_t)rows, 1, 1};
  cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void *>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

size_t antidiag_pairs_bytes(const Geom &g) {
  return sizeof(float2) * (size_t)g.R * (size_t)(g.N / kS) * (size_t)g.nb;
}

cudaError_t launch_antidiag_scores(const Geom &g, const Workspace &w, const void *Q, const void *K,
                                   const uint8_t *refresh, cudaStream_t s, int *launches) {
  const int Ns = g.N / kS, grp = g.block / kS, pitch = ((g.nb + 31) / 32) * 32;
  if (Ns > 0) {
    CUtensorMap mq, mk;
    if (!make_group_map(&mq, Q, g, Ns, kMt) || !make_group_map(&mk, K, g, Ns, kNt)) return cudaErrorInvalidValue;
    AdParams prm;
    prm.pairs = reinterpret_cast<float2 *>(w.pairs);
    prm.refresh = refresh;
    prm.status = w.status;
    prm.H = g.H;
    prm.Ns = Ns;
    prm.nb = g.nb;
    prm.g = grp;
    prm.c2 = (float)(g.scale / (double)kS * 1.4426950408889634);
    const int smem = kStagesAd * kStageBytes + 1024 + 256;
    // Split the key range over up to four CTAs per (row tile, head) when that fills the 148 SMs' waves
    // better (one CTA per SM); a shape-only rule.
    const int row_tiles = (Ns + kMt - 1) / kMt, col_tiles = (Ns + kNt - 1) / kNt;
    int split = 1;
    double best_eff = 0.0;
    for (int c = 1; c <= 4 && c <= col_tiles; ++c) {
      const long long ctas = (long long)row_tiles * g.R * c;
      const double waves = (double)((ctas + 147) / 148);
      const int longest = (col_tiles + c - 1) / c;  // column tiles of the busiest CTA
      const double eff = (double)ctas / (148.0 * waves) * ((double)col_tiles / c) / longest;
      if (eff > best_eff + 0.02) {
        best_eff = eff;
        split = c;
      }
    }
    dim3 grid(row_tiles, g.R, split);
    cudaError_t e;
    if (grp == 4) {
      e = cudaFuncSetAttribute(antidiag_scores_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
      if (e != cudaSuccess) return e;
      antidiag_scores_kernel<4><<<grid, kThreadsAd, smem, s>>>(mq, mk, prm);
    } else {
      e = cudaFuncSetAttribute(antidiag_scores_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
      if (e != cudaSuccess) return e;
      antidiag_scores_kernel<8><<<grid, kThreadsAd, smem, s>>>(mq, mk, prm);
    }
    ++*launches;
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
  }
  const float2 *pairs = reinterpret_cast<const float2 *>(w.pairs);
  const dim3 rgrid(g.nb, g.R);
  const int nj = (g.nb + 31) / 32;
  if (nj <= 8)
    antidiag_reduce_kernel<8><<<rgrid, 256, 0, s>>>(pairs, Ns, g.nb, grp, pitch, refresh, w.scores);
  else if (nj <= 16)
    antidiag_reduce_kernel<16><<<rgrid, 256, 0, s>>>(pairs, Ns, g.nb, grp, pitch, refresh, w.scores);
  else if (nj <= 24)
    antidiag_reduce_kernel<24><<<rgrid, 256, 0, s>>>(pairs, Ns, g.nb, grp, pitch, refresh, w.scores);
  else
    antidiag_reduce_kernel<32><<<rgrid, 256, 0, s>>>(pairs, Ns, g.nb, grp, pitch, refresh, w.scores);
  ++*launches;
  return cudaGetLastError();
}

}  // namespace heart
