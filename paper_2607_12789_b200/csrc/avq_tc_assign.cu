// Tensor-core key assignment (Algorithm 1, parent and child argmin) for bf16 inputs.
//
// One CTA takes 128 consecutive keys of one (batch, head), 8 warps.  TMA stages the key tile and the
// head's parent codebook in shared memory (K-major, 128-byte swizzle); one elected thread issues the
// tcgen05 MMA chain  D[128 x M] = K_tile . Cp^T  into TMEM.
//   parent   two threads per key (column halves) read their TMEM lane, form ||c||^2 - 2 k.c and keep
//            the best and the runner-up; the halves are merged in shared memory.  Only when best and
//            runner-up are closer than the MMA's rounding can separate are all M distances redone in
//            float64 in the direct form (lowest index wins ties).
//   child    fp32 direct form sum (k - c)^2 on CUDA cores (2 C d flops per key; a second MMA over all
//            M C children would cost C times the parent GEMM), float64 recheck for near-ties.
//            Four lanes per key, each over a quarter of the head dimension for all C children of the
//            key's parent (one running sum per child); a transposing butterfly merges the four lanes.
#include "avq_tc_common.cuh"

namespace avq {
namespace {

using namespace tc;

constexpr int kKeys = 128;
constexpr int kThreadsA = 256;
// CTAs per SM the register budget is set for: the d = 64 kernels are small enough (24-48 KB of shared
// memory, at most 128 TMEM columns up to M = 128) for four to share an SM.
constexpr int assign_min_ctas(int D, int NL) { return D == 64 ? 4 : 2; }

__device__ __forceinline__ float bf_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf_hi(uint32_t u) { return __uint_as_float(u & 0xFFFF0000u); }

// Two packed bf16 widened to a pair of fp32 in one 64-bit register (for the f32x2 instructions).
__device__ __forceinline__ uint64_t bf2_to_f32x2(uint32_t u) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(u << 16), "r"(u & 0xFFFF0000u));
  return r;
}
struct KeyChunk { uint64_t p[4]; };   // 8 key elements as four fp32 pairs
__device__ __forceinline__ KeyChunk widen8(const uint4& a) {
  KeyChunk k;
  k.p[0] = bf2_to_f32x2(a.x); k.p[1] = bf2_to_f32x2(a.y); k.p[2] = bf2_to_f32x2(a.z); k.p[3] = bf2_to_f32x2(a.w);
  return k;
}
// sum over 8 elements of (k - c)^2, two lanes of packed fp32 arithmetic (sub.f32x2 / fma.f32x2)
__device__ __forceinline__ float sqdiff8(const KeyChunk& k, const uint4& c) {
  const uint32_t y[4] = {c.x, c.y, c.z, c.w};
  uint64_t acc = 0;   // {0.f, 0.f}
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    uint64_t d;
    const uint64_t cw = bf2_to_f32x2(y[e]);
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(k.p[e]), "l"(cw));
    asm("fma.rn.f32x2 %0, %1, %1, %0;" : "+l"(acc) : "l"(d));
  }
  float lo, hi;
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(acc));
  return lo + hi;
}

// element `col` (0..D-1) of key row `row` in the swizzled key tile
template <int D>
__device__ __forceinline__ float key_elem(const unsigned char* Ks, int row, int col) {
  const unsigned char* sub = Ks + (col >> 6) * (kKeys * 128);
  return __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(sub + sw128_offset(row, col & 63)));
}

template <int D>
__device__ double exact_dist_smem(const unsigned char* Ks, int row, const __nv_bfloat16* c) {
  double s = 0.0;
  for (int k = 0; k < D; ++k) {
    const double t = (double)key_elem<D>(Ks, row, k) - (double)__bfloat162float(c[k]);
    s += t * t;
  }
  return s;
}

// ||c||^2 of every parent codeword of every head, once per call: a per-head constant that otherwise each of
// the Nk / 128 assign CTAs of every (batch, head) recomputes.  Eight lanes per codeword row.
template <int D>
__global__ void __launch_bounds__(256) code_norms_kernel(const __nv_bfloat16* __restrict__ Cp, float* __restrict__ cnorm,
                                                         int rows) {
  pdl_launch_dependents();   // the assign grid may start its set-up and loads
  const int row = (blockIdx.x * 256 + threadIdx.x) >> 3, part = threadIdx.x & 7;
  float s = 0.f;
  if (row < rows) {
    const uint4* src = reinterpret_cast<const uint4*>(Cp + (size_t)row * D) + part;
#pragma unroll
    for (int t = 0; t < D / 64; ++t) {
      const uint4 v = __ldg(src + 8 * t);
      const uint32_t wv[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        s = fmaf(bf_lo(wv[e]), bf_lo(wv[e]), s);
        s = fmaf(bf_hi(wv[e]), bf_hi(wv[e]), s);
      }
    }
  }
  s += __shfl_xor_sync(0xffffffffu, s, 1);
  s += __shfl_xor_sync(0xffffffffu, s, 2);
  s += __shfl_xor_sync(0xffffffffu, s, 4);
  if (row < rows && part == 0) cnorm[row] = s;
}

// NL = 16-byte loads per lane that cover one parent's C x d block of children: C * d / 256.
// STAYS: Algorithm 1's masked scatter - a key moves to its nearest child only if that child is strictly
// closer than the parent (child index -1 otherwise).
template <int D, int NL, bool STAYS>
__global__ void __launch_bounds__(kThreadsA, assign_min_ctas(D, NL))
tc_assign_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmCp,
                 const __nv_bfloat16* __restrict__ Cp, const __nv_bfloat16* __restrict__ Cc,
                 int32_t* __restrict__ pidx, int32_t* __restrict__ cidx, int H, int Nk, int M, int C,
                 uint32_t tmem_cols, int32_t* status_word, uint4* __restrict__ zero_base, uint32_t zero_units,
                 const float* cnorm_g) {
  // 1024-byte alignment (swizzle atoms) is requested from the launch, not computed from the pointer, so
  // that the compiler keeps every access in the shared address space.
  extern __shared__ __align__(1024) unsigned char smem[];
  constexpr int kSub = D / 64;                       // 64-column sub-tiles along the head dimension
  unsigned char* Ks = smem;                          // kSub x [128 x 128 B]
  unsigned char* Cs = Ks + kSub * kKeys * 128;       // kSub x [M x 128 B]
  float* cnorm = reinterpret_cast<float*>(Cs + kSub * M * 128);   // [M]
  float* xd1 = cnorm + M;                            // [2][128] best distance of each column half
  float* xd2 = xd1 + 2 * kKeys;                      // [2][128] runner-up
  float* xkn = xd2 + 2 * kKeys;                      // [2][128] halves of ||k||^2
  int* xi1 = reinterpret_cast<int*>(xkn + 2 * kKeys);   // [2][128] index of the best
  int* par = xi1 + 2 * kKeys;                        // [128] final parent of each key
  int* chi = par + kKeys;                            // [128] final child of each key
  uint32_t* cmax_bits = reinterpret_cast<uint32_t*>(chi + kKeys);   // max ||c||^2 (non-negative float bits)
  uint32_t* tmem_slot = cmax_bits + 1;
  uint64_t* bars = reinterpret_cast<uint64_t*>(tmem_slot + 1);      // [2]
  volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + 2);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int q = warp & 3, hf = warp >> 2, r = q * 32 + lane;
  const int bh = blockIdx.y, h = bh % H;
  const int j0 = blockIdx.x * kKeys;
  const int MH = M >> 1;                             // columns per half (multiple of 16: M % 32 == 0)
  pdl_launch_dependents();   // the next kernel of the call may begin its set-up
  // Inside avq_forward the grid also clears the accumulators of the aggregation that follows (status
  // header, leaf sums, leaf counts: zero_units 16-byte words), each CTA an equal slice; the stores drain
  // while the tile loads.  A bounded wait that expires does so long after CTA 0 has cleared the header.
  if (zero_units) {
    const uint32_t ncta = gridDim.x * gridDim.y, cta = blockIdx.y * gridDim.x + blockIdx.x;
    const uint32_t per = (zero_units + ncta - 1) / ncta;
    const uint32_t u0 = cta * per, u1 = min(zero_units, u0 + per);
    for (uint32_t u = u0 + tid; u < u1; u += kThreadsA) zero_base[u] = make_uint4(0u, 0u, 0u, 0u);
  }
  if (tid == 0) {
    prefetch_tmap(&tmK);
    prefetch_tmap(&tmCp);
    mbar_init(&bars[0], 1);
    mbar_init(&bars[1], 1);
    mbar_fence_init();
    *abort_flag = 0;
    *cmax_bits = 0;
    mbar_expect_tx(&bars[0], (uint32_t)(kSub * (kKeys + M) * 128));
#pragma unroll
    for (int s = 0; s < kSub; ++s) {
      tma_load_3d(Ks + s * kKeys * 128, &tmK, s * 64, j0, bh, &bars[0]);
      tma_load_2d(Cs + s * M * 128, &tmCp, s * 64, h * M, &bars[0]);
    }
  }
  // tcgen05.alloc blocks while the SM's columns are taken (four CTAs of 256 columns share an SM at d = 64,
  // M > 128: two run, two wait here).  The holders need nothing from the waiters and free their columns
  // before they end, so the wait is finite; it is the one device-side wait without a time limit of its own.
  if (warp == 1) {                                   // not the warp whose lane 0 is busy issuing the loads
    tmem_alloc(tmem_slot, tmem_cols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const bool loaded = mbar_wait(&bars[0], 0, abort_flag, status_word, DEV_TIMEOUT_ASSIGN);
  if (tid == 0 && loaded) {
    tc_fence_after();
    const uint32_t idesc = umma_idesc_bf16(kKeys, M);
    const uint32_t ka = smem_u32(Ks), ca = smem_u32(Cs);
#pragma unroll
    for (int k = 0; k < D / 16; ++k)
      umma_bf16(tmem_base, umma_desc_sw128(ka + (k / 4) * kKeys * 128 + (k % 4) * 32),
                umma_desc_sw128(ca + (k / 4) * M * 128 + (k % 4) * 32), idesc, k > 0);
    umma_commit(&bars[1]);
  }

  // ||c_m||^2 (and its maximum): from the array the kernel ahead of this one filled, or from the staged
  // codebook; half of ||k||^2 per thread
  if (cnorm_g) {
    pdl_wait();
    for (int m = tid; m < M; m += kThreadsA) {
      const float s = ld_after_wait(cnorm_g + (size_t)h * M + m);
      cnorm[m] = s;
      atomicMax(cmax_bits, __float_as_uint(s));
    }
  } else
  for (int m = tid; m < M; m += kThreadsA) {
    float s = 0.f;
#pragma unroll
    for (int sub = 0; sub < kSub; ++sub) {
#pragma unroll
      for (int ch = 0; ch < 8; ++ch) {
        const uint4 v = *reinterpret_cast<const uint4*>(Cs + sub * M * 128 + sw128_offset(m, ch * 8));
        const uint32_t wv[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          s = fmaf(bf_lo(wv[e]), bf_lo(wv[e]), s);
          s = fmaf(bf_hi(wv[e]), bf_hi(wv[e]), s);
        }
      }
    }
    cnorm[m] = s;
    atomicMax(cmax_bits, __float_as_uint(s));
  }
  {
    float s = 0.f;
    constexpr int kChunksHalf = D / 16;              // 16-byte chunks in half a row
#pragma unroll
    for (int cc = 0; cc < kChunksHalf; ++cc) {
      const int ch = hf * kChunksHalf + cc;          // chunk index in the row, 0 .. D/8-1
      const uint4 v = *reinterpret_cast<const uint4*>(Ks + (ch >> 3) * kKeys * 128 + sw128_offset(r, (ch & 7) * 8));
      const uint32_t wv[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        s = fmaf(bf_lo(wv[e]), bf_lo(wv[e]), s);
        s = fmaf(bf_hi(wv[e]), bf_hi(wv[e]), s);
      }
    }
    xkn[hf * kKeys + r] = s;
  }
  __syncthreads();   // cnorm, cmax visible

  const bool done = mbar_wait(&bars[1], 0, abort_flag, status_word, DEV_TIMEOUT_ASSIGN);
  tc_fence_after();

  // ---- parent argmin over this thread's half of the columns
  {
    float d1 = INFINITY, d2 = INFINITY;
    int i1 = 0;
    const uint32_t trow = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(hf * MH);
    for (int c0 = 0; c0 < MH; c0 += 16) {
      float dot[16];
      tmem_ld16(trow + c0, dot);                     // warp-collective: executed by every lane
      const float4* cn4 = reinterpret_cast<const float4*>(cnorm + hf * MH + c0);
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const float4 cn = cn4[u];
        const float dist[4] = {fmaf(-2.f, dot[4 * u], cn.x), fmaf(-2.f, dot[4 * u + 1], cn.y),
                               fmaf(-2.f, dot[4 * u + 2], cn.z), fmaf(-2.f, dot[4 * u + 3], cn.w)};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          d2 = fminf(d2, fmaxf(dist[e], d1));        // runner-up: second smallest so far
          if (dist[e] < d1) { d1 = dist[e]; i1 = hf * MH + c0 + 4 * u + e; }
        }
      }
    }
    xd1[hf * kKeys + r] = d1;
    xd2[hf * kKeys + r] = d2;
    xi1[hf * kKeys + r] = i1;
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, tmem_cols);

  // ---- merge the halves (the lower half holds the lower indices, so it wins ties); recheck near-ties
  const __nv_bfloat16* Cph = Cp + (size_t)h * M * D;
  if (hf == 0) {
    const float a1 = xd1[r], a2 = xd2[r], b1 = xd1[kKeys + r], b2 = xd2[kKeys + r];
    int i1 = (b1 < a1) ? xi1[kKeys + r] : xi1[r];
    const float d1 = fminf(a1, b1);
    const float d2 = fminf(fmaxf(a1, b1), fminf(a2, b2));
    const float knorm = xkn[r] + xkn[kKeys + r];
    const float cmax = __uint_as_float(*cmax_bits);
    // The MMA accumulates k.c in fp32: its error is a small multiple of 2^-24 * ||k|| * ||c||, which
    // 2e-4 * (||k||^2 + max ||c||^2) bounds with a wide margin.
    if (done && j0 + r < Nk && !(d2 - d1 > 2e-4f * (knorm + cmax))) {
      double best = INFINITY;
      int bi = 0;
      for (int m = 0; m < M; ++m) {
        const double s = exact_dist_smem<D>(Ks, r, Cph + (size_t)m * D);
        if (s < best) { best = s; bi = m; }
      }
      i1 = bi;
    }
    par[r] = i1;
  }
  __syncthreads();

  {
    // ---- child argmin, four lanes per key: a warp takes 8 keys at a time (two passes over its 16 keys).
    // Lane s of a key's group covers the 16-byte chunks s, s + 4, ... of the key row and of each of the
    // parent's C children (the group reads 64 contiguous bytes of a child row per load), keeps one running
    // sum per child, and a transposing butterfly over the four lanes leaves child s (and s + 4) in lane s.
    // The loads of the next chunk column are in flight while the current one is squared.
    constexpr int kC = NL * 256 / D;                   // children per parent (4 or 8)
    constexpr int kChunks = D / 8;                     // 16-byte chunks per row
    constexpr int kT = kChunks / 4;                    // chunk columns per lane (2 or 4)
    constexpr int kSteps = 2 * kT;                     // (pass, chunk column) pairs
    const int s4 = lane & 3, grp = lane >> 2;
    const size_t head_base = (size_t)h * M;
    uint4 buf[2][kC];
    auto issue = [&](int step, uint4 (&dst)[kC]) {
      const int key = warp * 16 + (step / kT) * 8 + grp;
      const uint4* src = reinterpret_cast<const uint4*>(Cc + (head_base + par[key]) * kC * D) + (s4 + 4 * (step % kT));
  #pragma unroll
      for (int c = 0; c < kC; ++c) dst[c] = __ldg(src + c * kChunks);
    };
    float sum[kC];
    float sum_p = 0.f;                                   // STAYS: direct-form distance to the parent itself
    issue(0, buf[0]);
  #pragma unroll
    for (int step = 0; step < kSteps; ++step) {
      const int pass = step / kT, t = step % kT;
      const int key = warp * 16 + pass * 8 + grp;
      if (step + 1 < kSteps) issue(step + 1, buf[(step + 1) & 1]);
      if (t == 0) {
  #pragma unroll
        for (int c = 0; c < kC; ++c) sum[c] = 0.f;
        sum_p = 0.f;
      }
      const int ch = s4 + 4 * t;
      const KeyChunk kv = widen8(*reinterpret_cast<const uint4*>(Ks + (ch >> 3) * (kKeys * 128) + sw128_offset(key, (ch & 7) * 8)));
  #pragma unroll
      for (int c = 0; c < kC; ++c) sum[c] += sqdiff8(kv, buf[step & 1][c]);
      if constexpr (STAYS)
        sum_p += sqdiff8(kv, __ldg(reinterpret_cast<const uint4*>(Cp + (head_base + par[key]) * D) + ch));
      if (t == kT - 1) {
        // transpose-reduce over the group: after the two exchanges lane s holds the total of child s
        // (and of child s + 4 when C = 8)
        const bool hi1 = (s4 & 1) != 0, hi2 = (s4 & 2) != 0;
        float r[kC / 2];
  #pragma unroll
        for (int i = 0; i < kC / 2; ++i) {
          const float send = hi1 ? sum[2 * i] : sum[2 * i + 1];
          const float keep = hi1 ? sum[2 * i + 1] : sum[2 * i];
          r[i] = keep + __shfl_xor_sync(0xffffffffu, send, 1);
        }
        float tot[kC / 4];
  #pragma unroll
        for (int i = 0; i < kC / 4; ++i) {
          const float send = hi2 ? r[2 * i] : r[2 * i + 1];
          const float keep = hi2 ? r[2 * i + 1] : r[2 * i];
          tot[i] = keep + __shfl_xor_sync(0xffffffffu, send, 2);
        }
        float e1 = tot[0], e2 = INFINITY;
        int c1 = s4;
        if constexpr (kC == 8) {
          e2 = fmaxf(tot[0], tot[1]);
          if (tot[1] < tot[0]) { e1 = tot[1]; c1 = s4 + 4; }
        }
  #pragma unroll
        for (int o = 1; o < 4; o <<= 1) {
          const float b1 = __shfl_xor_sync(0xffffffffu, e1, o);
          const float b2 = __shfl_xor_sync(0xffffffffu, e2, o);
          const int cb = __shfl_xor_sync(0xffffffffu, c1, o);
          e2 = fminf(fmaxf(e1, b1), fminf(e2, b2));
          if (b1 < e1 || (b1 == e1 && cb < c1)) { e1 = b1; c1 = cb; }
        }
        float dp = 0.f;
        if constexpr (STAYS) {
          dp = sum_p + __shfl_xor_sync(0xffffffffu, sum_p, 1);
          dp += __shfl_xor_sync(0xffffffffu, dp, 2);
        }
        if (s4 == 0) {
          bool rechecked = false;
          double best = INFINITY;
          if (done && j0 + key < Nk && !(e2 - e1 > 1e-4f * e2)) {
            const __nv_bfloat16* Cch = Cc + (head_base + par[key]) * kC * D;
            int bi = 0;
            for (int c = 0; c < kC; ++c) {
              const double sd = exact_dist_smem<D>(Ks, key, Cch + (size_t)c * D);
              if (sd < best) { best = sd; bi = c; }
            }
            c1 = bi;
            rechecked = true;
          }
          if constexpr (STAYS) {
            // strict '<' against the parent distance; float64 when the two are closer than fp32 separates
            bool moved = e1 < dp;
            if (done && j0 + key < Nk && (rechecked || !(fabsf(e1 - dp) > 1e-4f * fmaxf(e1, dp)))) {
              if (!rechecked) best = exact_dist_smem<D>(Ks, key, Cc + ((head_base + par[key]) * kC + c1) * D);
              moved = best < exact_dist_smem<D>(Ks, key, Cp + (head_base + par[key]) * D);
            }
            if (!moved) c1 = -1;
          }
          chi[key] = c1;
        }
      }
    }
  }
  __syncthreads();
  // When a wait above gave up the indices are meaningless, but they are in range (both argmins start
  // from index 0 and only take loop indices), so the kernels behind this one read nothing out of bounds;
  // they see the recorded status word and skip their work.
  if (tid < kKeys && j0 + tid < Nk) {
    pidx[(size_t)bh * Nk + j0 + tid] = par[tid];
    cidx[(size_t)bh * Nk + j0 + tid] = chi[tid];
  }
}

uint32_t pow2_cols(int n) {
  uint32_t c = 32;
  while ((int)c < n) c <<= 1;
  return c;
}

template <int D, int NL, bool STAYS>
avq_status launch(const avq_problem& p, const void* K, const void* Cp, const void* Cc, int32_t* pidx,
                  int32_t* cidx, int32_t* status_word, void* zero_base, size_t zero_bytes, float* cnorm, cudaStream_t st) {
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
  const size_t smem = (size_t)(D / 64) * (kKeys + p.M) * 128 +
                      sizeof(float) * (p.M + 6 * kKeys) +
                      sizeof(int) * (4 * kKeys) + 64 + 1024;
  auto kern = tc_assign_kernel<D, NL, STAYS>;
  // The limit is set once per device and instantiation (setting it again is harmless if two threads race).
  static size_t configured[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return AVQ_ERR_CUDA;
  if (dev < 0 || dev >= 64 || smem > configured[dev]) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return AVQ_ERR_CUDA;
    if (dev >= 0 && dev < 64) configured[dev] = smem;
  }
  dim3 grid((p.Nk + kKeys - 1) / kKeys, (unsigned)BH);
  if (cnorm) {
    const int rows = p.H * p.M;
    code_norms_kernel<D><<<(rows * 8 + 255) / 256, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(Cp), cnorm, rows);
    if (cudaGetLastError() != cudaSuccess) return AVQ_ERR_CUDA;
  }
  // launched as a dependent of the norms kernel when there is one: set-up, loads and the MMA overlap it
  return cuda_ok(launch_pdl(kern, grid, dim3(kThreadsA), smem, st, cnorm != nullptr, tmK, tmCp,
                            static_cast<const __nv_bfloat16*>(Cp), static_cast<const __nv_bfloat16*>(Cc), pidx, cidx,
                            p.H, p.Nk, p.M, p.C, pow2_cols(p.M), status_word, static_cast<uint4*>(zero_base),
                            (uint32_t)(zero_bytes / 16), static_cast<const float*>(cnorm)));
}

}  // namespace

avq_status tc_assign(const avq_problem& p, const void* K, const void* Cp, const void* Cc,
                     int32_t* parent_idx, int32_t* child_idx, int32_t* status_word, void* zero_base,
                     size_t zero_bytes, float* cnorm, cudaStream_t st) {
  if (zero_bytes % 16 != 0 || (zero_bytes / 16) >> 31) return AVQ_ERR_WORKSPACE;
  const bool stays = (p.flags & AVQ_FLAG_PARENT_STAYS) != 0;
#define AVQ_ASSIGN(DD, NN)                                                                                     \
  (stays ? launch<DD, NN, true>(p, K, Cp, Cc, parent_idx, child_idx, status_word, zero_base, zero_bytes, cnorm, st) \
         : launch<DD, NN, false>(p, K, Cp, Cc, parent_idx, child_idx, status_word, zero_base, zero_bytes, cnorm, st))
  if (p.d == 64) return p.C == 4 ? AVQ_ASSIGN(64, 1) : AVQ_ASSIGN(64, 2);
  return p.C == 4 ? AVQ_ASSIGN(128, 2) : AVQ_ASSIGN(128, 4);
#undef AVQ_ASSIGN
}

}  // namespace avq
