// Block-sparse attention with online softmax over the retained (query block, key block) pairs.
// CUDA-core version: one CTA per query block, fp32 FMA tiles in shared memory.
#include <cuda_bf16.h>

#include "common.cuh"

namespace heart {

constexpr int QLD = kD + 8;  // padded bf16 row (elements)

template <int BLOCK>
__global__ void __launch_bounds__(256) attn_fma_kernel(const uint16_t *__restrict__ Q,
                                                       const uint16_t *__restrict__ K,
                                                       const uint16_t *__restrict__ V, long long sb,
                                                       long long sh, long long sn, int H, int N, int nb,
                                                       float scale_log2, const int32_t *__restrict__ kv_idx,
                                                       const int32_t *__restrict__ kv_cnt, int idx_stride,
                                                       int dense, uint16_t *__restrict__ O,
                                                       float *__restrict__ lse, int32_t *status) {
  constexpr int TM = BLOCK / 16;
  constexpr int PLD = BLOCK + 1;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint16_t *Qs = reinterpret_cast<uint16_t *>(smem_raw);
  uint16_t *Ks = Qs + BLOCK * QLD;
  uint16_t *Vs = Ks + BLOCK * QLD;
  float *Ps = reinterpret_cast<float *>(Vs + BLOCK * QLD);
  float *alpha_s = Ps + BLOCK * PLD;
  float *m_s = alpha_s + BLOCK;
  float *l_s = m_s + BLOCK;

  const int I = blockIdx.x, r = blockIdx.y;
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4, lane = tid & 31, warp = tid >> 5;
  const long long head = (long long)(r / H) * sb + (long long)(r % H) * sh;
  const size_t row = (size_t)r * nb + I;
  const int cnt = dense ? nb : kv_cnt[row];
  const int32_t *list = kv_idx + row * idx_stride;

  for (int e = tid; e < BLOCK * 16; e += 256) {
    const int i = e >> 4, c = e & 15, tok = I * BLOCK + i;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (tok < N) v = *reinterpret_cast<const uint4 *>(Q + head + (long long)tok * sn + c * 8);
    *reinterpret_cast<uint4 *>(Qs + i * QLD + c * 8) = v;
  }
  for (int i = tid; i < BLOCK; i += 256) {
    m_s[i] = -INFINITY;
    l_s[i] = 0.f;
  }
  float acc[TM][8];
#pragma unroll
  for (int a = 0; a < TM; ++a)
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[a][e] = 0.f;

  for (int t = 0; t < cnt; ++t) {
    const int J = dense ? t : list[t];
    if (J < 0 || J >= nb) {  // bad entry: skip, report
      if (tid == 0) atomicExch(status, HEART_ERR_DEVICE_CHECK);
      continue;
    }
    __syncthreads();  // previous tile fully consumed
    for (int e = tid; e < BLOCK * 16; e += 256) {
      const int j = e >> 4, c = e & 15, tok = J * BLOCK + j;
      uint4 kv = make_uint4(0, 0, 0, 0), vv = make_uint4(0, 0, 0, 0);
      if (tok < N) {
        kv = *reinterpret_cast<const uint4 *>(K + head + (long long)tok * sn + c * 8);
        vv = *reinterpret_cast<const uint4 *>(V + head + (long long)tok * sn + c * 8);
      }
      *reinterpret_cast<uint4 *>(Ks + j * QLD + c * 8) = kv;
      *reinterpret_cast<uint4 *>(Vs + j * QLD + c * 8) = vv;
    }
    __syncthreads();
    {  // S = Q K^T (log2 domain)
      float s[TM][TM];
#pragma unroll
      for (int a = 0; a < TM; ++a)
#pragma unroll
        for (int c = 0; c < TM; ++c) s[a][c] = 0.f;
      for (int d2 = 0; d2 < kD / 2; ++d2) {
        float q0[TM], q1[TM];
#pragma unroll
        for (int a = 0; a < TM; ++a) {
          const uint32_t w = *reinterpret_cast<const uint32_t *>(Qs + (ty + 16 * a) * QLD + 2 * d2);
          q0[a] = __uint_as_float(w << 16);
          q1[a] = __uint_as_float(w & 0xffff0000u);
        }
#pragma unroll
        for (int c = 0; c < TM; ++c) {
          const uint32_t w = *reinterpret_cast<const uint32_t *>(Ks + (tx + 16 * c) * QLD + 2 * d2);
          const float k0 = __uint_as_float(w << 16), k1 = __uint_as_float(w & 0xffff0000u);
#pragma unroll
          for (int a = 0; a < TM; ++a) s[a][c] = fmaf(q1[a], k1, fmaf(q0[a], k0, s[a][c]));
        }
      }
#pragma unroll
      for (int a = 0; a < TM; ++a)
#pragma unroll
        for (int c = 0; c < TM; ++c) {
          const int j = tx + 16 * c;
          Ps[(ty + 16 * a) * PLD + j] = (J * BLOCK + j < N) ? s[a][c] * scale_log2 : -INFINITY;
        }
    }
    __syncthreads();
    for (int i = warp * (BLOCK / 8); i < (warp + 1) * (BLOCK / 8); ++i) {  // online softmax per row
      float v[BLOCK / 32], mx = -INFINITY;
#pragma unroll
      for (int k = 0; k < BLOCK / 32; ++k) {
        v[k] = Ps[i * PLD + lane + 32 * k];
        mx = fmaxf(mx, v[k]);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      const float m_old = m_s[i], m_new = fmaxf(m_old, mx);
      float sum = 0.f;
#pragma unroll
      for (int k = 0; k < BLOCK / 32; ++k) {
        const float p = exp2f(v[k] - m_new);
        Ps[i * PLD + lane + 32 * k] = p;
        sum += p;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
      if (lane == 0) {
        const float al = (m_old == -INFINITY) ? 0.f : exp2f(m_old - m_new);
        alpha_s[i] = al;
        m_s[i] = m_new;
        l_s[i] = l_s[i] * al + sum;
      }
    }
    __syncthreads();
#pragma unroll
    for (int a = 0; a < TM; ++a) {
      const float al = alpha_s[ty + 16 * a];
#pragma unroll
      for (int e = 0; e < 8; ++e) acc[a][e] *= al;
    }
    for (int j = 0; j < BLOCK; ++j) {  // O += P V
      const uint4 vv = *reinterpret_cast<const uint4 *>(Vs + j * QLD + tx * 8);
      float vf[8] = {__uint_as_float(vv.x << 16), __uint_as_float(vv.x & 0xffff0000u),
                     __uint_as_float(vv.y << 16), __uint_as_float(vv.y & 0xffff0000u),
                     __uint_as_float(vv.z << 16), __uint_as_float(vv.z & 0xffff0000u),
                     __uint_as_float(vv.w << 16), __uint_as_float(vv.w & 0xffff0000u)};
#pragma unroll
      for (int a = 0; a < TM; ++a) {
        const float p = Ps[(ty + 16 * a) * PLD + j];
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[a][e] = fmaf(p, vf[e], acc[a][e]);
      }
    }
  }
  __syncthreads();
#pragma unroll
  for (int a = 0; a < TM; ++a) {
    const int i = ty + 16 * a, tok = I * BLOCK + i;
    if (tok >= N) continue;
    const float l = l_s[i], inv = l > 0.f ? 1.f / l : 0.f;
    __nv_bfloat162 o2[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) o2[e] = __floats2bfloat162_rn(acc[a][2 * e] * inv, acc[a][2 * e + 1] * inv);
    *reinterpret_cast<uint4 *>(O + head + (long long)tok * sn + tx * 8) = *reinterpret_cast<uint4 *>(o2);
    if (lse != nullptr && tx == 0)
      lse[(size_t)r * N + tok] = l > 0.f ? (m_s[i] + log2f(l)) * 0.6931471805599453f : -INFINITY;
  }
}

cudaError_t launch_attention(const Geom &g, const void *Q, const void *K, const void *V,
                             const int32_t *kv_idx, const int32_t *kv_cnt, bool dense, void *O,
                             float *lse, int32_t *status, cudaStream_t s, int *launches) {
  const float scale_log2 = (float)(g.scale * 1.4426950408889634);
  const uint16_t *q = static_cast<const uint16_t *>(Q), *k = static_cast<const uint16_t *>(K),
                 *v = static_cast<const uint16_t *>(V);
  dim3 grid(g.nb, g.R);
  ++*launches;
  if (g.block == 64) {
    const size_t smem = 3 * 64 * QLD * 2 + 64 * 65 * 4 + 3 * 64 * 4;
    cudaError_t e = cudaFuncSetAttribute(attn_fma_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    attn_fma_kernel<64><<<grid, 256, smem, s>>>(q, k, v, g.sb, g.sh, g.sn, g.H, g.N, g.nb, scale_log2, kv_idx,
                                                kv_cnt, g.idx_stride, dense ? 1 : 0, static_cast<uint16_t *>(O),
                                                lse, status);
  } else {
    const size_t smem = 3 * 128 * QLD * 2 + 128 * 129 * 4 + 3 * 128 * 4;
    cudaError_t e = cudaFuncSetAttribute(attn_fma_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    attn_fma_kernel<128><<<grid, 256, smem, s>>>(q, k, v, g.sb, g.sh, g.sn, g.H, g.N, g.nb, scale_log2, kv_idx,
                                                 kv_cnt, g.idx_stride, dense ? 1 : 0, static_cast<uint16_t *>(O),
                                                 lse, status);
  }
  return cudaGetLastError();
}

}  // namespace heart
