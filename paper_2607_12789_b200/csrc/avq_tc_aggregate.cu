// Value aggregation for the bf16 path (Eq. "aggregates"; the scatter steps of Algorithm 1).
//
// leaf_scatter_kernel  one warp per key: the key's V row is added to the sum of its leaf
//                      codeword (parent, child) with vector reductions to global memory, and
//                      the leaf's count is bumped.  Only the leaf level is scattered.
// finalize_kernel      per parent: Vp = sum over its children (every key sits in exactly one
//                      child, so the parent sum is the sum of its leaves), np likewise, and
//                      the bf16 operand copies the attention kernel stages with TMA:
//                        VpT [B,H,d,M]    value sums with the codeword index fastest
//                        VcT [B,H,M,d,C]  per parent a contiguous d x C block, child fastest
#include "avq_tc_common.cuh"

namespace avq {
namespace {

constexpr int kScatterThreads = 256;
constexpr int kKeysPerCta = 256;

template <int D>
__global__ void __launch_bounds__(kScatterThreads)
leaf_scatter_kernel(const __nv_bfloat16* __restrict__ V, const int32_t* __restrict__ pidx,
                    const int32_t* __restrict__ cidx, float* __restrict__ Vc, float* __restrict__ nc,
                    int Nk, int M, int C) {
  const int bh = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int j0 = blockIdx.x * kKeysPerCta;
  const int j1 = min(Nk, j0 + kKeysPerCta);
  const size_t kb = (size_t)bh * Nk;
  for (int j = j0 + warp; j < j1; j += kScatterThreads / 32) {
    const int a = __ldg(pidx + kb + j);
    const int c = __ldg(cidx + kb + j);
    const size_t leaf = ((size_t)bh * M + a) * C + c;
    float* dst = Vc + leaf * D;
    const __nv_bfloat16* v = V + (kb + j) * D;
    if constexpr (D == 128) {
      const uint2 u = __ldg(reinterpret_cast<const uint2*>(v) + lane);
      float4 f = make_float4(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xFFFF0000u),
                             __uint_as_float(u.y << 16), __uint_as_float(u.y & 0xFFFF0000u));
      atomicAdd(reinterpret_cast<float4*>(dst) + lane, f);
    } else {
      const uint32_t u = __ldg(reinterpret_cast<const uint32_t*>(v) + lane);
      float2 f = make_float2(__uint_as_float(u << 16), __uint_as_float(u & 0xFFFF0000u));
      atomicAdd(reinterpret_cast<float2*>(dst) + lane, f);
    }
    if (lane == 0) atomicAdd(nc + leaf, 1.0f);
  }
}

// One CTA: 8 consecutive parents of one (batch, head); thread k owns head-dimension index k.
template <int D>
__global__ void __launch_bounds__(D)
finalize_kernel(const float* __restrict__ Vc, const float* __restrict__ nc, float* __restrict__ Vp,
                float* __restrict__ np_, __nv_bfloat16* __restrict__ VpT, __nv_bfloat16* __restrict__ VcT,
                int M, int C) {
  const int bh = blockIdx.y, m0 = blockIdx.x * 8, k = threadIdx.x;
  __align__(16) __nv_bfloat16 pk[8];
#pragma unroll
  for (int mm = 0; mm < 8; ++mm) {
    const int m = m0 + mm;
    const float* src = Vc + (((size_t)bh * M + m) * C) * D + k;
    __align__(16) __nv_bfloat16 ck[8];
    float s = 0.f;
    for (int c = 0; c < C; ++c) {
      const float x = src[(size_t)c * D];
      s += x;
      ck[c] = __float2bfloat16_rn(x);
    }
    Vp[((size_t)bh * M + m) * D + k] = s;
    pk[mm] = __float2bfloat16_rn(s);
    if (VcT) {
      __nv_bfloat16* dst = VcT + (((size_t)bh * M + m) * D + k) * C;
      if (C == 8) *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(ck);
      else *reinterpret_cast<uint2*>(dst) = *reinterpret_cast<const uint2*>(ck);
    }
  }
  if (VpT) *reinterpret_cast<uint4*>(VpT + ((size_t)bh * D + k) * M + m0) = *reinterpret_cast<const uint4*>(pk);
  if (k < 8) {
    const int m = m0 + k;
    float s = 0.f;
    for (int c = 0; c < C; ++c) s += nc[((size_t)bh * M + m) * C + c];
    np_[(size_t)bh * M + m] = s;
  }
}

template <int D>
avq_status run(const avq_problem& p, const void* V, const int32_t* pidx, const int32_t* cidx, float* Vp,
               float* np_, float* Vc, float* nc, void* VpT, void* VcT, cudaStream_t st) {
  const unsigned BH = (unsigned)(p.B * p.H);
  if (cudaMemsetAsync(Vc, 0, sizeof(float) * (size_t)BH * p.M * p.C * D, st) != cudaSuccess) return AVQ_ERR_CUDA;
  if (cudaMemsetAsync(nc, 0, sizeof(float) * (size_t)BH * p.M * p.C, st) != cudaSuccess) return AVQ_ERR_CUDA;
  dim3 g1((p.Nk + kKeysPerCta - 1) / kKeysPerCta, BH);
  leaf_scatter_kernel<D><<<g1, kScatterThreads, 0, st>>>(static_cast<const __nv_bfloat16*>(V), pidx, cidx, Vc,
                                                         nc, p.Nk, p.M, p.C);
  if (cudaGetLastError() != cudaSuccess) return AVQ_ERR_CUDA;
  dim3 g2(p.M / 8, BH);
  finalize_kernel<D><<<g2, D, 0, st>>>(Vc, nc, Vp, np_, static_cast<__nv_bfloat16*>(VpT),
                                       static_cast<__nv_bfloat16*>(VcT), p.M, p.C);
  return cuda_ok(cudaGetLastError());
}

}  // namespace

avq_status tc_aggregate(const avq_problem& p, const void* V, const int32_t* parent_idx,
                        const int32_t* child_idx, float* Vp, float* np_, float* Vc, float* nc, void* VpT,
                        void* VcT, cudaStream_t st) {
  return p.d == 64 ? run<64>(p, V, parent_idx, child_idx, Vp, np_, Vc, nc, VpT, VcT, st)
                   : run<128>(p, V, parent_idx, child_idx, Vp, np_, Vc, nc, VpT, VcT, st);
}

}  // namespace avq
