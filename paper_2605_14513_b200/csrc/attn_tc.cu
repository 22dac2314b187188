// Block-sparse attention with online softmax on the sm_100a tensor cores.
//
// One CTA owns one 128-row query tile of one head: one query block of 128 tokens, or two query
// blocks of 64 whose lists are merged into an ascending union (one flag bit per query block; rows of
// the half that does not list a key block see -inf there).  Keys are processed 64 at a time: a "key
// step" is one 64-token block, or one half of a 128-token block.
//
// Two CTAs share an SM (256 threads, 105 KB of shared memory and 256 of the 512 tensor-memory
// columns each).  They work on different query tiles and drift out of phase, so while the softmax
// warps of one compute exponentials -- the special-function unit is the scarcest resource of this
// kernel -- those of the other wait, load scores or take maxima, and the set-up and the epilogue of
// one tile hide behind the key steps of the other.  Inside a CTA the scores are double-buffered in
// tensor memory: S of step h+1 is complete before the softmax of step h ends, so the serial chain
// softmax -> P V -> Q K^T -> softmax is off the critical path.
//
// Warp roles (registers are moved from the helper warps to the softmax warps at start):
//   warps 0-3   softmax, one thread per query row (lane quarter = warp).  Per key step a thread reads
//               its row of S (64 columns), takes the max, rescales its row of O only when the max
//               grew by more than 2^8, writes P = 2^(s*scale*log2e - m) as bf16 over the first half
//               of the S buffer and adds the row sum; at the end it writes O / l (and lse).
//   warps 4-7   one helper role each, rotated with the CTA index so that the two CTAs of an SM
//               rarely put the same role on the same sub-partition:
//               K producer  TMA loads of Q (once) and of the listed K blocks into a two-stage ring
//                           (cp.async.bulk.tensor, 128-byte swizzle, completion on mbarriers);
//               V producer  the same for V (its own ring: V_h is needed two key steps after K_h);
//               QK issuer   S_h = Q K_h^T (tcgen05.mma, operands in shared memory), one elected lane;
//               PV issuer   O += P_h V_h with P_h read from tensor memory.
// Tensor memory (256 columns per CTA): O | S[2]  =  128 + 2 x 64; key step h uses S[h & 1] and
// shared-memory stage h & 1; P_h aliases S[h & 1].
//
// CTAs run head-major (the K/V of one or two heads stay in L2).  Within a head the tiles are taken in
// an order that tile_order_kernel writes just before the launch: by the first key block of their
// lists, so that the ~300 tiles in flight together read neighbouring key blocks (a head's K and V no
// longer fit one die's half of the L2 at 75 000 tokens and more), except for the last two heads of the
// launch, whose tiles go longest-list-first so that the launch does not end on a long tile that
// started late.  The K tile of the first listed key block is requested during set-up, before the step
// list is complete, and that block is put first.
//
// Every wait is bounded; a wait that runs out raises a CTA-wide abort flag and the status word, the
// roles drain, tensor memory is freed and the CTA exits.
#include <cuda.h>

#include "common.cuh"
#include "tc_ptx.cuh"

namespace heart {
using namespace tc;

constexpr int kAttnThreads = 256;
// warp roles: 0-3 softmax (lane quarter = warp), then one helper per SM sub-partition
constexpr int kRoleKProd = 0, kRoleVProd = 1, kRolePV = 2, kRoleQK = 3;  // helper warp 4 + ((role + CTA index) & 3)
constexpr int kRegsSoftmax = 176, kRegsHelper = 80;  // (176 + 80) * 128 threads = the CTA's 256 x 128
constexpr int kStep = 64;   // keys per key step
constexpr int kStages = 2;  // K / V ring depth = number of S buffers
constexpr int kTmemCols = 256;  // O (128) + S[2] (2 x 64): two CTAs share the 512 columns of an SM
constexpr int kMaxNb = HEART_MAX_BLOCKS;

// Shared-memory plan.
template <int B>
struct AttnSmem {
  static constexpr int HPB = B / kStep;         // key steps per key block (1 or 2)
  static constexpr int QBT = 128 / B;           // query blocks per CTA (1 or 2)
  static constexpr int Q_BYTES = 128 * 256;     // [2 dim halves][128 rows][64] bf16, 128-byte swizzle
  static constexpr int KV_BYTES = kStep * 256;  // [2 dim halves][64 rows][64] bf16, 128-byte swizzle
  static constexpr int OFF_Q = 0;
  static constexpr int OFF_K = OFF_Q + Q_BYTES;
  static constexpr int OFF_V = OFF_K + kStages * KV_BYTES;
  static constexpr int OFF_UNI = OFF_V + kStages * KV_BYTES;  // int32[kMaxNb]: J | flags << 16
  static constexpr int OFF_TBL = OFF_UNI + 4 * kMaxNb;        // uint32[kMaxNb]: flags per key block
  static constexpr int OFF_BAR = OFF_TBL + 4 * kMaxNb;        // mbarriers and scalars
  static constexpr int TOTAL = OFF_BAR + 512;
};

struct AttnBars {
  uint64_t q_full;
  uint64_t k_full[kStages], v_full[kStages];  // TMA -> MMA issuer
  uint64_t qk_done[kStages];                  // S_h complete: softmax may read it, K stage is free
  uint64_t pv_done[kStages];                  // P_h V_h complete: V stage and S/P buffer are free
  uint64_t p_full[kStages];                   // P_h written (one arrival per warp of the stream)
  uint64_t drain[2];                          // abort path: the issuers' products in flight have landed
  uint32_t tmem_base;
  int chunk_cnt[32];  // flagged key blocks per 32-block chunk (set-up)
  int n_union;
  int abort;
  int bad;
  int first_j;  // key block whose K tile was requested before the step list existed (-1: none)
};

struct AttnParams {
  const int32_t *kv_idx, *kv_cnt;
  uint16_t *O;
  float *lse;
  int32_t *status;
  long long sb, sh, sn;
  int H, N, nb, idx_stride, n_ctas_per_head, dense;
  int h0, hcount, R_all;  // this launch covers heads [h0, h0 + hcount) of every batch entry; R_all = B*H
  const int32_t *order;   // [heads of the launch][n_ctas_per_head]: tile of the head that CTA i takes (NULL: i)
  float scale_log2;
  int test_skip_v;  // test-hook builds only: CTA 0 leaves out the V copy of its second key step
};

// Clock-stamp trace (compile with -DHEART_TRACE; the caller's lse buffer must then have one extra
// row of N >= 4096 floats behind its R*N entries): CTA 0 records clock64() at the marked points of
// its first 64 key steps.  Slots: 0-7 softmax warp 2, 16-23 softmax warp 6, 8-15 the MMA issuer.
#ifdef HEART_TRACE
#define HEART_TR(h, slot)                                                             \
  do {                                                                                \
    if (trace_base != nullptr && (h) < 64) trace_base[(h) * 32 + (slot)] = clock64(); \
  } while (0)
#else
#define HEART_TR(h, slot) \
  do {                    \
  } while (0)
#endif

__device__ __forceinline__ float fmax3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}

template <int B>
__global__ void __launch_bounds__(kAttnThreads, 2)
    attn_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_kv,
                   const __grid_constant__ CUtensorMap map_v, const AttnParams p) {
  using L = AttnSmem<B>;
  constexpr int HPB = L::HPB;
  extern __shared__ unsigned char smem_dyn[];
  unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) &
                                                          ~static_cast<uintptr_t>(1023));
  unsigned char *Qs = smem + L::OFF_Q, *Ks = smem + L::OFF_K, *Vs = smem + L::OFF_V;
  int32_t *uni = reinterpret_cast<int32_t *>(smem + L::OFF_UNI);
  uint32_t *tbl = reinterpret_cast<uint32_t *>(smem + L::OFF_TBL);
  AttnBars *bars = reinterpret_cast<AttnBars *>(smem + L::OFF_BAR);
  volatile int *abort = &bars->abort;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // The helper roles rotate with the CTA index: the two CTAs that share an SM then rarely have the
  // same role (above all the issuer of the score products) on the same sub-partition.
  const int kWarpKProd = 4 + ((kRoleKProd + blockIdx.x) & 3), kWarpVProd = 4 + ((kRoleVProd + blockIdx.x) & 3),
            kWarpPV = 4 + ((kRolePV + blockIdx.x) & 3), kWarpQK = 4 + ((kRoleQK + blockIdx.x) & 3);
  // Tiles run head-major, which keeps the K/V of one or two heads in L2; within a head in the order
  // of the table (tiles whose lists start at the same key block together; the last two heads
  // longest-first, so that the launch ends on short tiles).
  const int rr = blockIdx.x / p.n_ctas_per_head;
  const int cta_in_head = p.order ? __ldg(&p.order[blockIdx.x]) : (int)(blockIdx.x % p.n_ctas_per_head);
  const int bidx = rr / p.hcount, hidx = p.h0 + rr % p.hcount;
  const int r = bidx * p.H + hidx;
  const int row0 = cta_in_head * 128;  // first query token of this CTA
  const int nb = p.nb;
#ifdef HEART_TRACE
  long long *trace_base = (blockIdx.x == 0 && p.lse != nullptr)
                              ? reinterpret_cast<long long *>(p.lse + (size_t)p.R_all * p.N)
                              : nullptr;
#endif

  // ------------------------------------------------------------------ set-up
  // A kernel that follows on the stream under programmatic stream serialisation (the next layer-step's
  // block-sum pass) may be scheduled once every tile of this launch has started: its CTAs then fill the
  // SMs that the last tiles leave behind and wait there for this launch to complete.
  pdl_launch_dependents();
  if (tid == 0) HEART_TR(0, 28);
  // The lists of this tile's query blocks come from global memory: their loads are issued first
  // (speculatively, inside the row pitch) so that their latency overlaps the rest of the set-up.
  constexpr int kPre = kMaxNb / kAttnThreads;  // entries per thread held in registers
  int cnt_q[L::QBT];
  int32_t ent[L::QBT][kPre];
#pragma unroll
  for (int qb = 0; qb < L::QBT; ++qb) {
    const int I = cta_in_head * L::QBT + qb;
    const size_t row = (size_t)r * nb + I;
    cnt_q[qb] = (I < nb) ? (p.dense ? nb : p.kv_cnt[row]) : 0;
#pragma unroll
    for (int k = 0; k < kPre; ++k) {
      const int t = tid + k * kAttnThreads;
      ent[qb][k] = (I < nb && !p.dense && t < p.idx_stride) ? p.kv_idx[row * p.idx_stride + t] : t;
    }
  }
  if (tid == 0) {
    mbar_init(&bars->q_full, 1);
    for (int i = 0; i < kStages; ++i) {
      mbar_init(&bars->k_full[i], 1);
      mbar_init(&bars->v_full[i], 1);
      mbar_init(&bars->qk_done[i], 1);
      mbar_init(&bars->pv_done[i], 1);
      mbar_init(&bars->p_full[i], 4);  // one arrival per softmax warp
    }
    mbar_init(&bars->drain[0], 1);
    mbar_init(&bars->drain[1], 1);
    bars->abort = 0;
    bars->bad = 0;
    bars->n_union = 0;
    mbar_fence_init();
  }
  for (int j = tid; j < nb; j += kAttnThreads) tbl[j] = 0u;
  __syncthreads();
  if (tid == 0) HEART_TR(1, 28);
  if (warp == kWarpKProd && lane == 0) {  // the Q tile does not depend on the lists: start it now
    tma_prefetch_desc(&map_q);
    tma_prefetch_desc(&map_kv);
    tma_prefetch_desc(&map_v);
    mbar_expect_tx(&bars->q_full, L::Q_BYTES);
    tma_load_4d(Qs, &map_q, &bars->q_full, 0, row0, hidx, bidx);
    tma_load_4d(Qs + 128 * 128, &map_q, &bars->q_full, 64, row0, hidx, bidx);
  }
  if (tid == 0) {
    // Thread 0 holds the first entry of each list.  Whatever the union turns out to be, that key
    // block is in it: its K tile is requested now, ~2000 clocks before the step list is ready, and
    // the compaction below puts the block first (for ascending lists it is the first anyway).
    int j0 = 0x7fffffff;
#pragma unroll
    for (int qb = 0; qb < L::QBT; ++qb)
      if (cnt_q[qb] > 0 && p.idx_stride > 0) j0 = min(j0, ent[qb][0] < 0 ? 0x7fffffff : ent[qb][0]);
    if (j0 < nb) {
      mbar_expect_tx(&bars->k_full[0], L::KV_BYTES);
      tma_load_4d(Ks, &map_kv, &bars->k_full[0], 0, j0 * B, hidx, bidx);
      tma_load_4d(Ks + kStep * 128, &map_kv, &bars->k_full[0], 64, j0 * B, hidx, bidx);
      bars->first_j = j0;
    } else {
      bars->first_j = -1;
    }
  }
#pragma unroll
  for (int qb = 0; qb < L::QBT; ++qb) {  // scatter: flag bit qb of every key block listed by query block qb
    const int I = cta_in_head * L::QBT + qb;
    int cnt = cnt_q[qb];
    if (cnt < 0 || cnt > p.idx_stride) {
      bars->bad = 1;
      cnt = cnt < 0 ? 0 : p.idx_stride;
    }
#pragma unroll
    for (int k = 0; k < kPre; ++k) {
      const int t = tid + k * kAttnThreads;
      if (t < cnt) {
        const int J = ent[qb][k];
        if (J < 0 || J >= nb)
          bars->bad = 1;  // skipped, reported
        else
          atomicOr(&tbl[J], 1u << qb);
      }
    }
    if (cnt > kPre * kAttnThreads) {  // longer than any list of distinct blocks: the slow way
      const int32_t *list = p.kv_idx + ((size_t)r * nb + I) * p.idx_stride;
      for (int t = kPre * kAttnThreads + tid; t < cnt; t += kAttnThreads) {
        const int J = list[t];
        if (J < 0 || J >= nb)
          bars->bad = 1;
        else
          atomicOr(&tbl[J], 1u << qb);
      }
    }
  }
  if (tid == 0) HEART_TR(1, 29);
  if (warp == kWarpQK) {
    tmem_alloc(&bars->tmem_base, kTmemCols);
    tmem_relinquish();
  }
  __syncthreads();
  if (tid == 0) HEART_TR(1, 30);
  {  // ascending compaction of the flagged key blocks: warp w takes the 32-block chunks w, w+16
    constexpr int kChunksPerWarp = kMaxNb / 32 / (kAttnThreads / 32);
    uint32_t f[kChunksPerWarp];
    unsigned ballot[kChunksPerWarp];
#pragma unroll
    for (int i = 0; i < kChunksPerWarp; ++i) {
      const int J = (warp + i * (kAttnThreads / 32)) * 32 + lane;
      f[i] = (J < nb) ? tbl[J] : 0u;
      ballot[i] = __ballot_sync(0xffffffffu, f[i] != 0u);
      if (lane == 0) bars->chunk_cnt[warp + i * (kAttnThreads / 32)] = __popc(ballot[i]);
    }
    __syncthreads();
    // exclusive prefix over the 32 chunk counts (every warp computes it: lane = chunk)
    const int mine = bars->chunk_cnt[lane];
    int incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    // the block whose K tile is already on its way goes first: p0 = its ascending rank
    const int first_j = bars->first_j;
    int p0 = 0;
    if (first_j >= 0) {
      const unsigned in_chunk = __ballot_sync(0xffffffffu, tbl[(first_j & ~31) + lane] != 0u);
      p0 = __shfl_sync(0xffffffffu, incl - mine, first_j >> 5) + __popc(in_chunk & ((1u << (first_j & 31)) - 1u));
    }
#pragma unroll
    for (int i = 0; i < kChunksPerWarp; ++i) {
      const int chunk = warp + i * (kAttnThreads / 32);
      const int base = __shfl_sync(0xffffffffu, incl - mine, chunk);
      if (f[i] != 0u) {
        const int J = chunk * 32 + lane, q = base + __popc(ballot[i] & ((1u << lane) - 1u));
        uni[J == first_j ? 0 : (q < p0 ? q + 1 : q)] = J | (int)(f[i] << 16);
      }
    }
    const int total = __shfl_sync(0xffffffffu, incl, 31);
    if (tid == 0) {
      bars->n_union = total;
      if (bars->bad) atomicExch(p.status, HEART_ERR_DEVICE_CHECK);
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (tid == 0) HEART_TR(0, 29);
  const uint32_t tmem = bars->tmem_base;
  const int U = bars->n_union;
  const int NH = U * HPB;  // key steps; step h uses S buffer and shared-memory stage h & 1
  // first key token of step h
  auto key0_of = [&](int h) -> int { return (uni[h / HPB] & 0xffff) * B + (h % HPB) * kStep; };

  // ------------------------------------------------------------------ roles
  // Shared memory must not be released under a copy in flight: a producer that stops early (abort)
  // waits, bounded, for the copies it has issued.
  auto settle = [&](uint64_t *bar, uint32_t parity) {
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity) && clock64() - t0 < 40000000LL) {
    }
  };
  if (warp >= 4) setmaxnreg_dec<kRegsHelper>();
  if (warp == kWarpKProd) {
    if (lane == 0) {  // ===== TMA producer (Q was started during set-up): K_h into stage h & 1
      int issued = 0;
      for (int h = 0; h < NH; ++h) {
        const int s = h % kStages, ph = (h / kStages) & 1;
        if (h == 0 && bars->first_j >= 0) {  // requested during set-up
          issued = 1;
          continue;
        }
        // the stage is free once S_{h-4} = Q K_{h-4}^T is complete
        if (h >= kStages && !mbar_wait_relaxed(&bars->qk_done[s], ph ^ 1, abort)) break;
        const int key0 = key0_of(h);
        unsigned char *dst = Ks + s * L::KV_BYTES;
        mbar_expect_tx(&bars->k_full[s], L::KV_BYTES);
        tma_load_4d(dst, &map_kv, &bars->k_full[s], 0, key0, hidx, bidx);
        tma_load_4d(dst + kStep * 128, &map_kv, &bars->k_full[s], 64, key0, hidx, bidx);
        issued = h + 1;
      }
      settle(&bars->q_full, 0);  // nobody else waits for Q when the union is empty
      if (*abort)
        for (int h = (issued > kStages ? issued - kStages : 0); h < issued; ++h) settle(&bars->k_full[h % kStages], (h / kStages) & 1);
    }
  } else if (warp == kWarpVProd) {
    if (lane == 0) {  // ===== TMA producer: V_h into stage h & 1
      int issued = 0;
      for (int h = 0; h < NH; ++h) {
        const int s = h % kStages, ph = (h / kStages) & 1;
        if (h >= kStages && !mbar_wait_relaxed(&bars->pv_done[s], ph ^ 1, abort)) break;
#ifdef HEART_TEST_HOOKS
        // Test-only library: one V tile is never requested (neither the byte count nor the copy), so the
        // waits that depend on it run out and the abort path below is taken.
        if (p.test_skip_v && blockIdx.x == 0 && h == 1) continue;
#endif
        const int key0 = key0_of(h);
        unsigned char *dst = Vs + s * L::KV_BYTES;
        mbar_expect_tx(&bars->v_full[s], L::KV_BYTES);
        tma_load_4d(dst, &map_v, &bars->v_full[s], 0, key0, hidx, bidx);
        tma_load_4d(dst + kStep * 128, &map_v, &bars->v_full[s], 64, key0, hidx, bidx);
        issued = h + 1;
      }
      if (*abort)
        for (int h = (issued > kStages ? issued - kStages : 0); h < issued; ++h) settle(&bars->v_full[h % kStages], (h / kStages) & 1);
    }
  } else if (warp == kWarpPV || warp == kWarpQK) {
    // ===== MMA issuers: warp 7 issues S_h = Q K_h^T, warp 6 issues O += P_h V_h.  Two warps, so that
    // the barrier round trips of one overlap the issue of the other.  The whole warp runs the loop
    // (uniform control flow keeps the descriptors in uniform registers), one elected lane issues.
    if (NH > 0) {
      constexpr uint32_t idesc_qk = idesc_bf16_f32(128, kStep, false, false);
      constexpr uint32_t idesc_pv = idesc_bf16_f32(128, 128, false, true);
      // Descriptors of one key step differ only in the start-address field (low word, no carry out
      // of it): base + a compile-time offset per 16-element k-step.
      //   Q, K (K-major): 64 dims = one 128-byte row; dim halves Q: 128*128 B apart, K: 64*128 B.
      //   V (MN-major):   64 dims = one 128-byte row; dim halves 64*128 B apart (the LBO);
      //                   16 keys = 16 rows = 2048 B per k-step.
      auto at = [](uint64_t desc, uint32_t off16) -> uint64_t {
        return (desc & 0xffffffff00000000ull) | (uint32_t)((uint32_t)desc + off16);
      };
      const bool leader = elect_one();  // the same lane every time: commits track its MMAs
      bool ok = true;
      if (warp == kWarpQK) {
        const uint64_t q_desc = smem_desc_sw128(smem_u32(Qs), 16, 1024);
        const uint64_t k_desc = smem_desc_sw128(smem_u32(Ks), 16, 1024);
        auto issue_qk = [&](int s) {  // S[s] = Q K^T with the K tile that sits in stage s
          const uint32_t d = tmem + 128 + s * kStep;
          const uint64_t ks_desc = at(k_desc, s * (L::KV_BYTES >> 4));
          if (leader) {
#pragma unroll
            for (int ks = 0; ks < 8; ++ks)
              mma_ss(d, at(q_desc, (ks >> 2) * 1024 + (ks & 3) * 2), at(ks_desc, (ks >> 2) * 512 + (ks & 3) * 2),
                     idesc_qk, ks > 0 ? 1u : 0u);
            tc_commit(&bars->qk_done[s]);
          }
          __syncwarp();
        };
        ok = mbar_wait(&bars->q_full, 0, abort);
        for (int h = 0; h < kStages && h < NH && ok; ++h) {
          ok = mbar_wait(&bars->k_full[h], 0, abort);
          if (ok) {
            tc_fence_after();
            issue_qk(h);
          }
        }
        for (int h = 0; h + kStages < NH && ok; ++h) {
          const int s = h % kStages, ph = (h / kStages) & 1;
          // S[s] holds P_h until the product P_h V_h has read it
          ok = mbar_wait(&bars->k_full[s], ph ^ 1, abort);
          if (ok) ok = mbar_wait(&bars->pv_done[s], ph, abort);
          if (!ok) break;
          HEART_TR(h, 10);
          tc_fence_after();
          issue_qk(s);
          HEART_TR(h, 11);
        }
      } else {
        const uint64_t v_desc = smem_desc_sw128(smem_u32(Vs), kStep * 128, 1024);
        for (int h = 0; h < NH && ok; ++h) {  // O (+)= P_h V_h; P_h sits over S[h & 1]
          const int s = h % kStages, ph = (h / kStages) & 1;
          ok = mbar_wait(&bars->v_full[s], ph, abort);
          HEART_TR(h, 12);
          if (ok) ok = mbar_wait(&bars->p_full[s], ph, abort);
          if (!ok) break;
          HEART_TR(h, 8);
          tc_fence_after();
          const uint32_t d = tmem, pa = tmem + 128 + s * kStep;
          const uint64_t vs_desc = at(v_desc, s * (L::KV_BYTES >> 4));
          if (leader) {
#pragma unroll
            for (int ks = 0; ks < 4; ++ks)
              mma_ts(d, pa + ks * 8, at(vs_desc, ks * 128), idesc_pv, (h > 0 || ks > 0) ? 1u : 0u);
            tc_commit(&bars->pv_done[s]);
          }
          __syncwarp();
          HEART_TR(h, 9);
        }
      }
      if (*abort) {
        // Tensor memory must not be released under a product in flight: a commit arrives once
        // everything this lane has issued is complete; the wait for it is bounded like the others.
        uint64_t *bar = &bars->drain[warp == kWarpQK ? 0 : 1];
        if (leader) tc_commit(bar);
        __syncwarp();
        settle(bar, 0);
      }
    }
  } else {
    // ===== softmax / correction / epilogue: thread = one query row
    setmaxnreg_inc<kRegsSoftmax>();
    const int q = warp;             // TMEM lane quarter this warp may touch
    const int row = q * 32 + lane;  // row inside the 128-row query tile
    const uint32_t lane_addr = tmem + ((uint32_t)(q * 32) << 16);
    const uint32_t o_addr = lane_addr;
    const float c = p.scale_log2;
    float m_ref = -INFINITY, l_run = 0.f;
    bool ok = true;
    const uint32_t my_bit = 1u << (row / B);  // query block of this row (uniform within a warp)
#ifdef HEART_TRACE
    const int tr0 = 0;
    const bool trw = warp == 0 && lane == 0;
#define HEART_TRS(slot)                   \
  do {                                    \
    if (trw) HEART_TR(h, tr0 + (slot));   \
  } while (0)
#else
#define HEART_TRS(slot) \
  do {                  \
  } while (0)
#endif
    for (int h = 0; h < NH && ok; ++h) {
      const int s = h % kStages, ph = (h / kStages) & 1;
      HEART_TRS(0);
      // key columns of this step that are real keys this row attends to
      int lim = 0;
      {
        const uint32_t e = (uint32_t)uni[h / HPB];
        if ((e >> 16) & my_bit) lim = max(0, min(kStep, p.N - ((int)(e & 0xffff) * B + (h % HPB) * kStep)));
      }
      const int lim0 = min(lim, 32), lim1 = max(lim - 32, 0);
      const uint32_t s_addr = lane_addr + 128 + s * kStep;
      ok = __all_sync(0xffffffffu, mbar_wait(&bars->qk_done[s], ph, abort));
      if (!ok) break;
      HEART_TRS(1);
      tc_fence_after();
      uint32_t sreg[64];
      if (lim0 > 0) tmem_ld32(s_addr, *reinterpret_cast<uint32_t(*)[32]>(&sreg[0]));
      if (lim1 > 0) tmem_ld32(s_addr + 32, *reinterpret_cast<uint32_t(*)[32]>(&sreg[32]));
      tmem_wait_ld();
      HEART_TRS(2);
      if (lim < kStep) {  // rare: ragged last block, or a block this row's query block does not list
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
      const float x_max = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * c;  // -inf stays -inf (c > 0)
      HEART_TRS(3);
      float alpha = 1.f;
      bool grow = false;
      if (m_ref == -INFINITY) {
        m_ref = x_max;  // nothing accumulated for this row yet: no rescale needed
      } else if (x_max > m_ref + 8.f) {
        alpha = ex2(m_ref - x_max);
        m_ref = x_max;
        grow = true;
      }
      if (__any_sync(0xffffffffu, grow) && h >= 1) {
        // O must be quiescent: the previous product has to be complete
        ok = __all_sync(0xffffffffu, mbar_wait(&bars->pv_done[(h - 1) % kStages], ((h - 1) / kStages) & 1, abort));
        if (!ok) break;
        tc_fence_after();
        const uint64_t alpha2 = pack_f32x2(alpha, alpha);
#pragma unroll 1
        for (int ch = 0; ch < 4; ++ch) {
          uint32_t v[32];
          tmem_ld32(o_addr + ch * 32, v);
          tmem_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; i += 2) {
            float lo, hi;
            unpack_f32x2(mul_f32x2(pack_f32x2(__uint_as_float(v[i]), __uint_as_float(v[i + 1])), alpha2), lo, hi);
            v[i] = __float_as_uint(lo);
            v[i + 1] = __float_as_uint(hi);
          }
          tmem_st32(o_addr + ch * 32, v);
        }
        tmem_wait_st();
      }
      HEART_TRS(4);
      const float neg_m = (m_ref == -INFINITY) ? 0.f : -m_ref;
      const uint64_t c2 = pack_f32x2(c, c), neg_m2 = pack_f32x2(neg_m, neg_m);
      // p = 2^(s*c - m), packed to bf16 over columns [0, 32) of S[h & 1]; the product reads all 64
      // keys of the step, so every column is written (zeros where the row has no key)
      float sum0 = 0.f, sum1 = 0.f, sum2 = 0.f, sum3 = 0.f;
#pragma unroll
      for (int ch = 0; ch < 2; ++ch) {
        uint32_t pk[16];
        if ((ch ? lim1 : lim0) == 0) {
#pragma unroll
          for (int i = 0; i < 16; ++i) pk[i] = 0u;
        } else {
#pragma unroll
          for (int i = 0; i < 32; i += 4) {
            float x0, x1, x2, x3;
            unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(sreg[ch * 32 + i]), __uint_as_float(sreg[ch * 32 + i + 1])), c2, neg_m2), x0, x1);
            unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(sreg[ch * 32 + i + 2]), __uint_as_float(sreg[ch * 32 + i + 3])), c2, neg_m2), x2, x3);
            // the row sum is taken over the bf16-rounded weights, the ones the PV product really
            // uses, so numerator and denominator carry the same rounding: O stays a weighted mean
            const uint32_t w0 = pack_bf16x2(ex2(x0), ex2(x1));
            const uint32_t w1 = pack_bf16x2(ex2(x2), ex2(x3));
            pk[i >> 1] = w0;
            pk[(i >> 1) + 1] = w1;
            add_bf16x2_to_f32(sum0, sum1, w0);
            add_bf16x2_to_f32(sum2, sum3, w1);
          }
        }
        tmem_st16(s_addr + ch * 16, pk);
      }
      l_run = l_run * alpha + ((sum0 + sum1) + (sum2 + sum3));
      HEART_TRS(5);
      tmem_wait_st();
      HEART_TRS(6);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->p_full[s]);
      HEART_TRS(7);
#ifdef HEART_TRACE
      if (lane == 0) HEART_TR(h, 24 + q);  // arrival time of each warp of the warpgroup
#endif
    }
    // epilogue: O / l, one row per thread
    const int tok = row0 + row;
    const bool valid_row = tok < p.N;
    // the products complete in issue order: the last one covers them all
    if (ok && NH > 0)
      ok = __all_sync(0xffffffffu, mbar_wait(&bars->pv_done[(NH - 1) % kStages], ((NH - 1) / kStages) & 1, abort));
    if (ok) {
      tc_fence_after();
      const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
      uint16_t *orow = p.O + (long long)bidx * p.sb + (long long)hidx * p.sh + (long long)tok * p.sn;
#pragma unroll 1
      for (int ch = 0; ch < 4; ++ch) {  // 32 output dims at a time
        uint32_t v[32];
        if (NH > 0) {
          tmem_ld32(o_addr + ch * 32, v);
          tmem_wait_ld();
        }
        if (valid_row) {
#pragma unroll
          for (int g4 = 0; g4 < 4; ++g4) {
            float o[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) o[i] = NH > 0 ? __uint_as_float(v[g4 * 8 + i]) * inv : 0.f;
            uint4 w;
            w.x = pack_bf16x2(o[0], o[1]);
            w.y = pack_bf16x2(o[2], o[3]);
            w.z = pack_bf16x2(o[4], o[5]);
            w.w = pack_bf16x2(o[6], o[7]);
            *reinterpret_cast<uint4 *>(orow + ch * 32 + g4 * 8) = w;
          }
        }
      }
      if (valid_row && p.lse != nullptr)
        p.lse[(size_t)r * p.N + tok] = l_run > 0.f ? (m_ref + log2f(l_run)) * 0.6931471805599453f : -INFINITY;
    }
  }

  // ------------------------------------------------------------------ tear-down
  if (tid == 0) HEART_TR(0, 30);
  tc_fence_before();
  __syncthreads();
  if (tid == 0) HEART_TR(0, 31);
  if (warp == kWarpQK) {
    tc_fence_after();
    tmem_dealloc(tmem, kTmemCols);
  }
  if (tid == 0 && bars->abort) atomicExch(p.status, HEART_ERR_DEVICE_CHECK);
}

// Order of the tiles of every head of a launch.  One CTA per head; rank by counting over at most 1024
// keys, so the result is a permutation whatever the lists hold.  Heads before the last two: index order
// while a head's K and V fit the L2 comfortably; beyond that ascending by the first key block that the
// tile's lists name (ties by tile index) -- tiles that read the same region of K and V run together.
// The last two heads: descending by the number of listed key blocks.
__global__ void __launch_bounds__(256) tile_order_kernel(const int32_t *__restrict__ kv_idx,
                                                         const int32_t *__restrict__ kv_cnt, int nb, int qbt, int ncph,
                                                         int idx_stride, int H, int h0, int hcount, int n_heads,
                                                         int by_first_key, int32_t *__restrict__ order) {
  __shared__ int key[1024];
  const int rr = blockIdx.x, r = (rr / hcount) * H + h0 + rr % hcount;
  const bool by_length = rr >= n_heads - 2;
  for (int t = threadIdx.x; t < ncph; t += blockDim.x) {
    int len = 0, first = 0x3fffffff;
    for (int qb = 0; qb < qbt; ++qb) {
      const int I = t * qbt + qb;
      if (I >= nb) break;
      const int c = min(max(__ldg(&kv_cnt[(size_t)r * nb + I]), 0), idx_stride);
      len += c;
      if (c > 0) first = min(first, max(__ldg(&kv_idx[((size_t)r * nb + I) * idx_stride]), 0));
    }
    key[t] = by_length ? -len : (by_first_key ? first : t);
  }
  __syncthreads();
  for (int t = threadIdx.x; t < ncph; t += blockDim.x) {
    const int mine = key[t];
    int rank = 0;
    for (int u = 0; u < ncph; ++u) rank += (key[u] < mine || (key[u] == mine && u < t)) ? 1 : 0;
    order[(size_t)rr * ncph + rank] = t;
  }
}

// ---------------------------------------------------------------------- host side
namespace {

// bf16 [B,H,N,128] with element strides (sb, sh, sn, 1): box = 64 dims x `rows` tokens, 128-byte swizzle,
// out-of-range rows read as zero.
bool make_map(CUtensorMap *m, const void *base, const Geom &g, int rows) {
  EncodeTiledFn fn = encode_tiled_fn();
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
  // two CTAs per SM: all of the configurable shared memory
  e = cudaFuncSetAttribute(attn_tc_kernel<B>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
  if (e != cudaSuccess) return e;
  attn_tc_kernel<B><<<g.B * prm.hcount * prm.n_ctas_per_head, kAttnThreads, smem, s>>>(mq, mk, mv, prm);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_attention(const Geom &g, const void *Q, const void *K, const void *V,
                             const int32_t *kv_idx, const int32_t *kv_cnt, bool dense, void *O,
                             float *lse, int32_t *status, int32_t *order, cudaStream_t s, int *launches, int h0,
                             int hcount) {
  if (hcount <= 0) {
    h0 = 0;
    hcount = g.H;
  }
  CUtensorMap mq, mk, mv;
  if (!make_map(&mq, Q, g, 128) || !make_map(&mk, K, g, kStep) || !make_map(&mv, V, g, kStep))
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
  prm.h0 = h0;
  prm.hcount = hcount;
  prm.R_all = g.R;
  prm.scale_log2 = (float)(g.scale * 1.4426950408889634);
  prm.test_skip_v = 0;
#ifdef HEART_TEST_HOOKS
  prm.test_skip_v = (g.flags & 0x80000000u) ? 1 : 0;
#endif
  prm.order = nullptr;
  if (!dense && order != nullptr && prm.n_ctas_per_head <= 1024) {
    const int rows = g.B * hcount;
    // K + V of one head beyond 32 MB (about half of one die's share of the L2): order by key locality
    const int by_first_key = (size_t)g.N * kD * 2 * 2 > (size_t)(32u << 20) ? 1 : 0;
    tile_order_kernel<<<rows, 256, 0, s>>>(kv_idx, kv_cnt, g.nb, 128 / g.block, prm.n_ctas_per_head, g.idx_stride, g.H,
                                           h0, hcount, rows, by_first_key, order);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    prm.order = order;
    ++*launches;
  }
  ++*launches;
  return g.block == 64 ? launch_bk<64>(g, mq, mk, mv, prm, s) : launch_bk<128>(g, mq, mk, mv, prm, s);
}

}  // namespace heart
