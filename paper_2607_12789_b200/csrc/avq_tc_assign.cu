// Tensor-core key assignment (Algorithm 1, parent and child argmin) for bf16 inputs.
//
// One CTA takes 128 consecutive keys of one (batch, head).  TMA stages the key tile and the
// head's parent codebook in shared memory (K-major, 128-byte swizzle); one elected thread
// issues the tcgen05 MMA chain  D[128 x M] = K_tile . Cp^T  into TMEM.  Each of the 128
// threads then owns one key (one TMEM lane): it reads its row of dot products, forms
// ||c||^2 - 2 k.c, keeps the best and the runner-up, and - only when those two are closer
// than the MMA's rounding can separate - re-evaluates all M distances in float64 in the direct
// form.  The child argmin over the C children of the winner runs on CUDA cores (2 C d
// flops per key; a second MMA over all M C children would cost C times the parent GEMM).
#include "avq_tc_common.cuh"

namespace avq {
namespace {

using namespace tc;

constexpr int kKeys = 128;

__device__ __forceinline__ float bf_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf_hi(uint32_t u) { return __uint_as_float(u & 0xFFFF0000u); }

template <int D>
__device__ double exact_dist_regs(const uint32_t (&kreg)[D / 2], const __nv_bfloat16* c) {
  double s = 0.0;
#pragma unroll 4
  for (int q = 0; q < D / 2; ++q) {
    const double a = (double)bf_lo(kreg[q]) - (double)__bfloat162float(c[2 * q]);
    const double b = (double)bf_hi(kreg[q]) - (double)__bfloat162float(c[2 * q + 1]);
    s += a * a;
    s += b * b;
  }
  return s;
}

template <int D>
__device__ float direct_dist_regs(const uint32_t (&kreg)[D / 2], const __nv_bfloat16* c) {
  const uint4* c4 = reinterpret_cast<const uint4*>(c);
  float s = 0.f;
#pragma unroll
  for (int q = 0; q < D / 8; ++q) {
    const uint4 v = __ldg(c4 + q);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float a = bf_lo(kreg[4 * q + e]) - bf_lo(w[e]);
      const float b = bf_hi(kreg[4 * q + e]) - bf_hi(w[e]);
      s = fmaf(a, a, s);
      s = fmaf(b, b, s);
    }
  }
  return s;
}

template <int D>
__global__ void __launch_bounds__(kKeys)
tc_assign_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmCp,
                 const __nv_bfloat16* __restrict__ Cp, const __nv_bfloat16* __restrict__ Cc,
                 int32_t* __restrict__ pidx, int32_t* __restrict__ cidx, int H, int Nk, int M, int C,
                 uint32_t tmem_cols, int32_t* status_word) {
  // 1024-byte alignment (swizzle atoms) is requested from the launch, not computed from the pointer, so
  // that the compiler keeps every access in the shared address space.
  extern __shared__ __align__(1024) unsigned char smem[];
  constexpr int kSub = D / 64;                       // 64-column sub-tiles along the head dimension
  unsigned char* Ks = smem;                          // kSub x [128 x 128 B]
  unsigned char* Cs = Ks + kSub * kKeys * 128;       // kSub x [M x 128 B]
  float* cnorm = reinterpret_cast<float*>(Cs + kSub * M * 128);   // [M]
  uint64_t* bars = reinterpret_cast<uint64_t*>(cnorm + M);        // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int tid = threadIdx.x, warp = tid >> 5;
  const int bh = blockIdx.y, h = bh % H;
  const int j0 = blockIdx.x * kKeys, j = j0 + tid;

  if (tid == 0) {
    mbar_init(&bars[0], 1);
    mbar_init(&bars[1], 1);
    mbar_fence_init();
    *abort_flag = 0;
    prefetch_tmap(&tmK);
    prefetch_tmap(&tmCp);
  }
  if (warp == 0) {
    tmem_alloc(tmem_slot, tmem_cols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (tid == 0) {
    mbar_expect_tx(&bars[0], (uint32_t)(kSub * (kKeys + M) * 128));
#pragma unroll
    for (int s = 0; s < kSub; ++s) {
      tma_load_3d(Ks + s * kKeys * 128, &tmK, s * 64, j0, bh, &bars[0]);
      tma_load_2d(Cs + s * M * 128, &tmCp, s * 64, h * M, &bars[0]);
    }
  }
  const bool loaded = mbar_wait(&bars[0], 0, abort_flag, status_word, DEV_TIMEOUT_ASSIGN);

  if (tid == 0 && loaded) {
    tc_fence_after();
    const uint32_t idesc = umma_idesc_bf16(kKeys, M);
    const uint32_t ka = smem_u32(Ks), ca = smem_u32(Cs);
#pragma unroll
    for (int k = 0; k < D / 16; ++k) {
      const uint64_t ad = umma_desc_sw128(ka + (k / 4) * kKeys * 128 + (k % 4) * 32);
      const uint64_t bd = umma_desc_sw128(ca + (k / 4) * M * 128 + (k % 4) * 32);
      umma_bf16(tmem_base, ad, bd, idesc, k > 0);
    }
    umma_commit(&bars[1]);
  }

  // ||c_m||^2 from the staged codebook, and this thread's key row into registers
  for (int m = tid; m < M; m += kKeys) {
    float s = 0.f;
#pragma unroll
    for (int sub = 0; sub < kSub; ++sub) {
      const unsigned char* row = Cs + sub * M * 128;
#pragma unroll
      for (int ch = 0; ch < 8; ++ch) {
        const uint4 v = *reinterpret_cast<const uint4*>(row + sw128_offset(m, ch * 8));
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          s = fmaf(bf_lo(w[e]), bf_lo(w[e]), s);
          s = fmaf(bf_hi(w[e]), bf_hi(w[e]), s);
        }
      }
    }
    cnorm[m] = s;
  }
  uint32_t kreg[D / 2];
  float knorm = 0.f;
#pragma unroll
  for (int sub = 0; sub < kSub; ++sub) {
#pragma unroll
    for (int ch = 0; ch < 8; ++ch) {
      const uint4 v = *reinterpret_cast<const uint4*>(Ks + sub * kKeys * 128 + sw128_offset(tid, ch * 8));
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        kreg[sub * 32 + ch * 4 + e] = w[e];
        knorm = fmaf(bf_lo(w[e]), bf_lo(w[e]), knorm);
        knorm = fmaf(bf_hi(w[e]), bf_hi(w[e]), knorm);
      }
    }
  }
  __syncthreads();   // cnorm visible

  const bool done = mbar_wait(&bars[1], 0, abort_flag, status_word, DEV_TIMEOUT_ASSIGN);
  tc_fence_after();

  float d1 = INFINITY, d2 = INFINITY, cmax = 0.f;
  int i1 = 0;
  if (done) {
    const uint32_t trow = tmem_base + ((uint32_t)(warp * 32) << 16);
    for (int c0 = 0; c0 < M; c0 += 16) {
      float dot[16];
      tmem_ld16(trow + c0, dot);
#pragma unroll
      for (int e = 0; e < 16; ++e) {
        const float cn = cnorm[c0 + e];
        const float dist = fmaf(-2.f, dot[e], cn);
        cmax = fmaxf(cmax, cn);
        if (dist < d1) { d2 = d1; d1 = dist; i1 = c0 + e; }
        else if (dist < d2) { d2 = dist; }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, tmem_cols);
  if (j >= Nk || !done) return;

  const __nv_bfloat16* Cph = Cp + (size_t)h * M * D;
  // The MMA accumulates k.c in fp32: its error is a small multiple of 2^-24 * ||k|| * ||c||, which
  // 2e-4 * (||k||^2 + max ||c||^2) bounds with a wide margin.
  if (M > 1 && !(d2 - d1 > 2e-4f * (knorm + cmax))) {
    double best = INFINITY;
    int bi = 0;
    for (int m = 0; m < M; ++m) {
      const double s = exact_dist_regs<D>(kreg, Cph + (size_t)m * D);
      if (s < best) { best = s; bi = m; }
    }
    i1 = bi;
  }

  const __nv_bfloat16* Cch = Cc + ((size_t)h * M + i1) * C * D;
  float e1 = INFINITY, e2 = INFINITY;
  int c1 = 0;
  for (int c = 0; c < C; ++c) {
    const float s = direct_dist_regs<D>(kreg, Cch + (size_t)c * D);
    if (s < e1) { e2 = e1; e1 = s; c1 = c; }
    else if (s < e2) { e2 = s; }
  }
  if (C > 1 && !(e2 - e1 > 1e-4f * e2)) {
    double best = INFINITY;
    int bi = 0;
    for (int c = 0; c < C; ++c) {
      const double s = exact_dist_regs<D>(kreg, Cch + (size_t)c * D);
      if (s < best) { best = s; bi = c; }
    }
    c1 = bi;
  }
  pidx[(size_t)bh * Nk + j] = i1;
  cidx[(size_t)bh * Nk + j] = c1;
}

uint32_t pow2_cols(int n) {
  uint32_t c = 32;
  while ((int)c < n) c <<= 1;
  return c;
}

template <int D>
avq_status launch(const avq_problem& p, const void* K, const void* Cp, const void* Cc, int32_t* pidx,
                  int32_t* cidx, int32_t* status_word, cudaStream_t st) {
  CUtensorMap tmK, tmCp;
  const uint64_t BH = (uint64_t)p.B * p.H;
  {
    const uint64_t dims[3] = {(uint64_t)D, (uint64_t)p.Nk, BH};
    const uint32_t box[3] = {64, (uint32_t)kKeys, 1};
    avq_status s = make_tmap_bf16(&tmK, K, 3, dims, box);
    if (s != AVQ_OK) return s;
  }
  {
    const uint64_t dims[2] = {(uint64_t)D, (uint64_t)p.H * p.M};
    const uint32_t box[2] = {64, (uint32_t)p.M};
    avq_status s = make_tmap_bf16(&tmCp, Cp, 2, dims, box);
    if (s != AVQ_OK) return s;
  }
  const size_t smem = 1024 + (size_t)(D / 64) * (kKeys + p.M) * 128 + sizeof(float) * p.M + 64;
  auto kern = tc_assign_kernel<D>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return AVQ_ERR_CUDA;
  dim3 grid((p.Nk + kKeys - 1) / kKeys, (unsigned)BH);
  kern<<<grid, kKeys, smem, st>>>(tmK, tmCp, static_cast<const __nv_bfloat16*>(Cp),
                                  static_cast<const __nv_bfloat16*>(Cc), pidx, cidx, p.H, p.Nk, p.M, p.C,
                                  pow2_cols(p.M), status_word);
  return cuda_ok(cudaGetLastError());
}

}  // namespace

avq_status tc_assign(const avq_problem& p, const void* K, const void* Cp, const void* Cc,
                     int32_t* parent_idx, int32_t* child_idx, int32_t* status_word, cudaStream_t st) {
  return p.d == 64 ? launch<64>(p, K, Cp, Cc, parent_idx, child_idx, status_word, st)
                   : launch<128>(p, K, Cp, Cc, parent_idx, child_idx, status_word, st);
}

}  // namespace avq
