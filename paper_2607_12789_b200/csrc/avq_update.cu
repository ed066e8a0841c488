// avq_codebook_update: one training-time update of the hierarchical codebook from a batch of keys
// (appendix "Codeword Clustering During Training").
//
// The data-parallel part reuses the forward's own kernels: avq_assign gives every key its parent and
// child under the current codebooks, and the aggregation kernels, fed the KEYS as values, give the
// per-(batch, head) key sums and counts of every parent and child.  ema_project_kernel then folds the
// batch into the per-head EMA statistics, moves each parent to its EMA mean, and places the children at
// the mass-weighted projection of their EMA means onto  mean_c C_{p,c} = C_p
// (Eq. "child_constraint_solve").
#include <cuda_bf16.h>

#include "avq_internal.h"

namespace avq {
namespace {

constexpr float kMassFloor = 1e-6f;   // a code without EMA mass keeps its position and absorbs the residual

template <typename T> __device__ __forceinline__ float ld_code(const T* p);
template <> __device__ __forceinline__ float ld_code<float>(const float* p) { return *p; }
template <> __device__ __forceinline__ float ld_code<__nv_bfloat16>(const __nv_bfloat16* p) { return __bfloat162float(*p); }
template <typename T> __device__ __forceinline__ void st_code(T* p, float v);
template <> __device__ __forceinline__ void st_code<float>(float* p, float v) { *p = v; }
template <> __device__ __forceinline__ void st_code<__nv_bfloat16>(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

// One CTA per (head, parent); thread k owns head-dimension index k (strided when d > blockDim).
// Kp [B,H,M,d], np [B,H,M], Kc [B,H,M,C,d], nc [B,H,M,C]: this batch's key sums and counts.
template <typename T>
__global__ void __launch_bounds__(128)
ema_project_kernel(const float* __restrict__ Kp, const float* __restrict__ np_, const float* __restrict__ Kc,
                   const float* __restrict__ nc, const T* __restrict__ Cp, const T* __restrict__ Cc,
                   float* __restrict__ Sp, float* __restrict__ Np, float* __restrict__ Sc, float* __restrict__ Nc,
                   T* __restrict__ Cp_out, T* __restrict__ Cc_out, int B, int H, int M, int C, int d, float decay) {
  const int m = blockIdx.x, h = blockIdx.y;
  const size_t hm = (size_t)h * M + m;
  __shared__ float s_np, s_nc[16];
  if (threadIdx.x <= C) {
    // counts: thread 0 the parent, threads 1..C the children (summed over the batch, then the EMA step)
    float cnt = 0.f;
    for (int b = 0; b < B; ++b) {
      const size_t bhm = ((size_t)b * H + h) * M + m;
      cnt += threadIdx.x == 0 ? np_[bhm] : nc[bhm * C + (threadIdx.x - 1)];
    }
    if (threadIdx.x == 0) {
      const float v = decay * Np[hm] + (1.f - decay) * cnt;
      Np[hm] = v;
      s_np = v;
    } else {
      const size_t i = hm * C + (threadIdx.x - 1);
      const float v = decay * Nc[i] + (1.f - decay) * cnt;
      Nc[i] = v;
      s_nc[threadIdx.x - 1] = v;
    }
  }
  __syncthreads();
  float sigma = 0.f;
  for (int c = 0; c < C; ++c) sigma += 1.f / fmaxf(s_nc[c], kMassFloor);
  for (int k = threadIdx.x; k < d; k += blockDim.x) {
    float sum = 0.f;
    for (int b = 0; b < B; ++b) sum += Kp[(((size_t)b * H + h) * M + m) * d + k];
    const float sp = decay * Sp[hm * d + k] + (1.f - decay) * sum;
    Sp[hm * d + k] = sp;
    const float cp = s_np > kMassFloor ? sp / s_np : ld_code(Cp + hm * d + k);
    st_code(Cp_out + hm * d + k, cp);
    float mc[16], delta = -(float)C * cp;
    for (int c = 0; c < C; ++c) {
      float cs = 0.f;
      for (int b = 0; b < B; ++b) cs += Kc[((((size_t)b * H + h) * M + m) * C + c) * d + k];
      const size_t i = (hm * C + c) * d + k;
      const float sc = decay * Sc[i] + (1.f - decay) * cs;
      Sc[i] = sc;
      mc[c] = s_nc[c] > kMassFloor ? sc / s_nc[c] : ld_code(Cc + i);
      delta += mc[c];
    }
    for (int c = 0; c < C; ++c)
      st_code(Cc_out + (hm * C + c) * d + k, mc[c] - delta / (fmaxf(s_nc[c], kMassFloor) * sigma));
  }
}

struct UpdateLayout {
  size_t pidx, cidx, Kp, np, Kc, nc, total;
};
UpdateLayout update_layout(const avq_problem& p) {
  UpdateLayout L;
  const size_t BH = (size_t)p.B * p.H;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = (off + bytes + 255) / 256 * 256; return o; };
  L.pidx = take(4 * BH * p.Nk);
  L.cidx = take(4 * BH * p.Nk);
  L.Kp = take(4 * BH * p.M * p.d);
  L.np = take(4 * BH * p.M);
  L.Kc = take(4 * BH * p.M * p.C * p.d);
  L.nc = take(4 * BH * p.M * p.C);
  L.total = off;
  return L;
}

}  // namespace
}  // namespace avq

using namespace avq;

extern "C" {

size_t avq_codebook_update_workspace_bytes(const avq_problem* prob) {
  if (validate_problem(prob) != AVQ_OK) return 0;
  return update_layout(*prob).total;
}

avq_status avq_codebook_update(const avq_problem* prob, const void* K, const void* Cp, const void* Cc, float decay,
                               float* Sp, float* Np, float* Sc, float* Nc, void* Cp_out, void* Cc_out,
                               void* workspace, size_t workspace_bytes, void* stream) {
  avq_status s = validate_problem(prob);
  if (s != AVQ_OK) return s;
  if (!(decay >= 0.f && decay <= 1.f)) return AVQ_ERR_SHAPE;
  if (prob->C > 16) return AVQ_ERR_UNSUPPORTED;
  if (!K || !Cp || !Cc || !Sp || !Np || !Sc || !Nc || !Cp_out || !Cc_out) return AVQ_ERR_NULL;
  if (!workspace) return AVQ_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(workspace) & 255u) return AVQ_ERR_ALIGN;
  const UpdateLayout L = update_layout(*prob);
  if (workspace_bytes < L.total) return AVQ_ERR_WORKSPACE;
  char* ws = static_cast<char*>(workspace);
  int32_t* pidx = reinterpret_cast<int32_t*>(ws + L.pidx);
  int32_t* cidx = reinterpret_cast<int32_t*>(ws + L.cidx);
  float* Kp = reinterpret_cast<float*>(ws + L.Kp);
  float* np_ = reinterpret_cast<float*>(ws + L.np);
  float* Kc = reinterpret_cast<float*>(ws + L.Kc);
  float* nc = reinterpret_cast<float*>(ws + L.nc);
  // the keys' assignment under the current codebooks, then their sums and counts per codeword
  s = avq_assign(prob, K, Cp, Cc, pidx, cidx, stream);
  if (s != AVQ_OK) return s;
  s = avq_aggregate(prob, K, pidx, cidx, Kp, np_, Kc, nc, stream);
  if (s != AVQ_OK) return s;
  const dim3 grid((unsigned)prob->M, (unsigned)prob->H);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (prob->dtype == AVQ_F32)
    ema_project_kernel<float><<<grid, 128, 0, st>>>(Kp, np_, Kc, nc, static_cast<const float*>(Cp),
                                                    static_cast<const float*>(Cc), Sp, Np, Sc, Nc,
                                                    static_cast<float*>(Cp_out), static_cast<float*>(Cc_out),
                                                    prob->B, prob->H, prob->M, prob->C, prob->d, decay);
  else
    ema_project_kernel<__nv_bfloat16><<<grid, 128, 0, st>>>(
        Kp, np_, Kc, nc, static_cast<const __nv_bfloat16*>(Cp), static_cast<const __nv_bfloat16*>(Cc), Sp, Np, Sc,
        Nc, static_cast<__nv_bfloat16*>(Cp_out), static_cast<__nv_bfloat16*>(Cc_out), prob->B, prob->H, prob->M,
        prob->C, prob->d, decay);
  return cuda_ok(cudaGetLastError());
}

}  // extern "C"
