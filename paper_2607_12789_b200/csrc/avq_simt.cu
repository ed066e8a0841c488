// Plain CUDA-core (FFMA) kernels for the three stages of the AVQ-attention forward.
// They carry the float32 path (tensor-core inputs are 16-bit, too coarse for a 1e-4
// output tolerance) and any shape outside the tensor-core envelope, for either dtype.
//
//   assign_simt_kernel     Algorithm 1, parent and child argmin, one thread per key
//   aggregate_simt_kernel  Eq. "aggregates": value sums and counts, one warp per key
//   attend_simt_kernel     Algorithm 2 in its masked form: parent pass, Eq. "importance",
//                          top-P, then one softmax over {unrefined parents} U {children of the
//                          refined parents} with the maximum taken over non-empty codewords
#include <cuda_bf16.h>
#include <math.h>

#include "avq_internal.h"

namespace avq {
namespace {

template <typename T> __device__ __forceinline__ float ldf(const T* p);
template <> __device__ __forceinline__ float ldf<float>(const float* p) { return __ldg(p); }
template <> __device__ __forceinline__ float ldf<__nv_bfloat16>(const __nv_bfloat16* p) {
  return __bfloat162float(*p);
}
template <typename T> __device__ __forceinline__ void stf(T* p, float v);
template <> __device__ __forceinline__ void stf<float>(float* p, float v) { *p = v; }
template <> __device__ __forceinline__ void stf<__nv_bfloat16>(__nv_bfloat16* p, float v) {
  *p = __float2bfloat16_rn(v);
}

constexpr int kAssignKeys = 128;   // keys (= threads) per CTA
constexpr int kAssignCodes = 16;   // parent codewords staged in shared memory at a time
// Two distances closer than this (relative) are re-evaluated in float64.  The float32 direct
// form carries about d * 2^-24 relative error, far below it.
constexpr float kNearTie = 1e-4f;

template <typename T>
__device__ double exact_dist(const float* krow, const T* c, int d) {
  double s = 0.0;
  for (int k = 0; k < d; ++k) {
    double t = (double)krow[k] - (double)ldf(c + k);
    s += t * t;
  }
  return s;
}

// ------------------------------------------------------------------------------- assign
template <typename T>
__global__ void __launch_bounds__(kAssignKeys)
assign_simt_kernel(const T* __restrict__ K, const T* __restrict__ Cp, const T* __restrict__ Cc,
                   int32_t* __restrict__ pidx, int32_t* __restrict__ cidx, int H, int Nk, int d, int M,
                   int C, int parent_stays) {
  extern __shared__ float smem[];
  const int ldk = d + 1;
  float* ks = smem;                        // [kAssignKeys][d+1]
  float* cs = smem + kAssignKeys * ldk;    // [kAssignCodes][d]
  const int bh = blockIdx.y, h = bh % H;
  const int j0 = blockIdx.x * kAssignKeys, t = threadIdx.x, j = j0 + t;
  const int rows = min(kAssignKeys, Nk - j0);
  const T* Kb = K + ((size_t)bh * Nk + j0) * d;
  for (int e = t; e < rows * d; e += kAssignKeys) ks[(e / d) * ldk + (e % d)] = ldf(Kb + e);
  const float* kr = ks + t * ldk;
  const T* Cph = Cp + (size_t)h * M * d;

  float d1 = INFINITY, d2 = INFINITY;
  int i1 = 0;
  for (int m0 = 0; m0 < M; m0 += kAssignCodes) {
    const int mc = min(kAssignCodes, M - m0);
    __syncthreads();
    for (int e = t; e < mc * d; e += kAssignKeys) cs[e] = ldf(Cph + (size_t)m0 * d + e);
    __syncthreads();
    if (j < Nk) {
      for (int mm = 0; mm < mc; ++mm) {
        const float* c = cs + mm * d;
        float s = 0.f;
        for (int k = 0; k < d; ++k) {
          float df = kr[k] - c[k];
          s = fmaf(df, df, s);
        }
        if (s < d1) { d2 = d1; d1 = s; i1 = m0 + mm; }
        else if (s < d2) { d2 = s; }
      }
    }
  }
  if (j >= Nk) return;

  double dp64 = -1.0;   // exact parent distance, if it had to be computed
  if (M > 1 && !(d2 - d1 > kNearTie * d2)) {
    double best = INFINITY;
    int bi = 0;
    for (int m = 0; m < M; ++m) {
      double s = exact_dist(kr, Cph + (size_t)m * d, d);
      if (s < best) { best = s; bi = m; }
    }
    i1 = bi;
    dp64 = best;
    d1 = (float)best;
  }

  const T* Cch = Cc + ((size_t)h * M + i1) * C * d;
  float e1 = INFINITY, e2 = INFINITY;
  int c1 = 0;
  for (int c = 0; c < C; ++c) {
    const T* cc = Cch + (size_t)c * d;
    float s = 0.f;
    for (int k = 0; k < d; ++k) {
      float df = kr[k] - ldf(cc + k);
      s = fmaf(df, df, s);
    }
    if (s < e1) { e2 = e1; e1 = s; c1 = c; }
    else if (s < e2) { e2 = s; }
  }
  double dc64 = -1.0;
  if (C > 1 && !(e2 - e1 > kNearTie * e2)) {
    double best = INFINITY;
    int bi = 0;
    for (int c = 0; c < C; ++c) {
      double s = exact_dist(kr, Cch + (size_t)c * d, d);
      if (s < best) { best = s; bi = c; }
    }
    c1 = bi;
    dc64 = best;
    e1 = (float)best;
  }
  if (parent_stays) {
    bool moved = e1 < d1;
    float hi = fmaxf(e1, d1);
    if (!(fabsf(e1 - d1) > kNearTie * hi)) {
      if (dp64 < 0.0) dp64 = exact_dist(kr, Cph + (size_t)i1 * d, d);
      if (dc64 < 0.0) dc64 = exact_dist(kr, Cch + (size_t)c1 * d, d);
      moved = dc64 < dp64;
    }
    if (!moved) c1 = -1;
  }
  pidx[(size_t)bh * Nk + j] = i1;
  cidx[(size_t)bh * Nk + j] = c1;
}

// ------------------------------------------------------------------------------- aggregate
template <typename T>
__global__ void __launch_bounds__(256)
aggregate_simt_kernel(const T* __restrict__ V, const int32_t* __restrict__ pidx,
                      const int32_t* __restrict__ cidx, float* __restrict__ Vp, float* __restrict__ np_,
                      float* __restrict__ Vc, float* __restrict__ nc, int Nk, int d, int M, int C,
                      int keys_per_cta) {
  const int bh = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
  const int j0 = blockIdx.x * keys_per_cta;
  const int j1 = min(Nk, j0 + keys_per_cta);
  for (int j = j0 + warp; j < j1; j += nwarps) {
    const int a = pidx[(size_t)bh * Nk + j];
    const int c = cidx[(size_t)bh * Nk + j];
    const T* v = V + ((size_t)bh * Nk + j) * d;
    float* vp = Vp + ((size_t)bh * M + a) * d;
    float* vc = (c >= 0) ? Vc + (((size_t)bh * M + a) * C + c) * d : nullptr;
    for (int k = lane; k < d; k += 32) {
      float x = ldf(v + k);
      atomicAdd(vp + k, x);
      if (vc) atomicAdd(vc + k, x);
    }
    if (lane == 0) {
      atomicAdd(np_ + (size_t)bh * M + a, 1.0f);
      if (c >= 0) atomicAdd(nc + ((size_t)bh * M + a) * C + c, 1.0f);
    }
  }
}

// ------------------------------------------------------------------------------- attend
struct AttendArgs {
  const void *Q, *Cp, *Cc;
  const float *Vp, *np_, *Vc, *nc;
  void* Y;
  int32_t* topp_out;
  float* importance_out;
  int H, Nq, d, M, C, P, block_q, nblk, stays;
  int correcting; // Algorithm 2's literal child pass: mean-recovered parent logit and Delta A = A_c - A_p
  int tile_m;     // 0: exact importance; else parents visited in tiles of tile_m (Eq. "aproxdenom")
  int Nk;
  float scale;
};

template <typename T>
__device__ __forceinline__ float logit(const float* q, const T* c, int d, float scale) {
  float s = 0.f;
  for (int k = 0; k < d; ++k) s = fmaf(q[k], ldf(c + k), s);
  return s * scale;
}

__device__ __forceinline__ float warp_max(float v) {
  for (int o = 16; o; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
  for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

constexpr int kAttendThreads = 256;
constexpr int kMaxDPerLane = 8;   // d <= 256

template <typename T>
__global__ void __launch_bounds__(kAttendThreads) attend_simt_kernel(AttendArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int d = a.d, M = a.M, C = a.C, P = a.P;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, nwarps = kAttendThreads / 32;
  const int blk = blockIdx.x, bh = blockIdx.y, h = bh % a.H;
  const int i0 = blk * a.block_q;
  const int rows = min(a.block_q, a.Nq - i0);
  const int ncols = M + P * C;

  // shared memory carve-up (doubles first for alignment)
  double* w = reinterpret_cast<double*>(smem_raw);                 // [M]
  float* qs = reinterpret_cast<float*>(w + M);                     // [block_q][d]
  float* rm = qs + (size_t)a.block_q * d;                          // [block_q]
  float* rz = rm + a.block_q;                                      // [block_q]
  float* npS = rz + a.block_q;                                     // [M]
  float* nstay = npS + M;                                          // [M]
  float* sbuf = nstay + M;                                         // [nwarps][ncols]
  int* sel = reinterpret_cast<int*>(sbuf + (size_t)nwarps * ncols);   // [M]
  int* sel_list = sel + M;                                         // [max(P,1)]
  const int ntiles = a.tile_m > 0 ? (M + a.tile_m - 1) / a.tile_m : 0;
  float* zt = reinterpret_cast<float*>(sel_list + (P > 0 ? P : 1));   // [block_q][ntiles] denominators seen up to a tile
  float* nseen = zt + (size_t)a.block_q * ntiles;                  // [ntiles] keys of the tiles seen up to a tile

  const T* Qb = static_cast<const T*>(a.Q) + ((size_t)bh * a.Nq + i0) * d;
  const T* Cph = static_cast<const T*>(a.Cp) + (size_t)h * M * d;
  const T* Cch = static_cast<const T*>(a.Cc) + (size_t)h * M * C * d;
  const float* Vp = a.Vp + (size_t)bh * M * d;
  const float* Vc = a.Vc + (size_t)bh * M * C * d;
  const float* np_ = a.np_ + (size_t)bh * M;
  const float* nc = a.nc + (size_t)bh * M * C;

  for (int e = tid; e < rows * d; e += kAttendThreads) qs[e] = ldf(Qb + e);
  for (int j = tid; j < M; j += kAttendThreads) {
    float n = np_[j], s = 0.f;
    for (int c = 0; c < C; ++c) s += nc[j * C + c];
    npS[j] = n;
    nstay[j] = n - s;
  }
  __syncthreads();

  // ---- parent pass: row maximum over non-empty parents and z_i = sum_j A_ij n_j
  float* sb = sbuf + (size_t)warp * ncols;
  for (int i = warp; i < rows; i += nwarps) {
    float mx = -INFINITY;
    for (int j = lane; j < M; j += 32) {
      float s = logit(qs + (size_t)i * d, Cph + (size_t)j * d, d, a.scale);
      sb[j] = s;
      if (npS[j] > 0.f) mx = fmaxf(mx, s);
    }
    mx = warp_max(mx);
    float z = 0.f;
    for (int j = lane; j < M; j += 32)
      if (npS[j] > 0.f) z += expf(sb[j] - mx) * npS[j];
    z = warp_sum(z);
    if (lane == 0) { rm[i] = mx; rz[i] = z; }
    // tiled importance: the part of the denominator contributed by the tiles visited so far
    float prefix = 0.f;
    for (int t = 0; t < ntiles; ++t) {
      float zp = 0.f;
      const int j1 = min(M, (t + 1) * a.tile_m);
      for (int j = t * a.tile_m + lane; j < j1; j += 32)
        if (npS[j] > 0.f) zp += expf(sb[j] - mx) * npS[j];
      prefix += warp_sum(zp);
      if (lane == 0) zt[(size_t)i * ntiles + t] = prefix;
    }
  }
  if (tid == 0) {
    float seen = 0.f;
    for (int t = 0; t < ntiles; ++t) {
      const int j1 = min(M, (t + 1) * a.tile_m);
      for (int j = t * a.tile_m; j < j1; ++j) seen += npS[j];
      nseen[t] = seen;
    }
  }
  __syncthreads();

  // ---- importance w_j = n_j * sum_i exp(s_ij - m_i) / z_i, fixed summation order, float64 sum
  for (int j = tid; j < M; j += kAttendThreads) {
    double acc = 0.0;
    if (npS[j] > 0.f) {
      // exact: the row's full denominator.  Tiled (appendix "Computing Importance with Tiled Codewords"):
      // the denominator seen up to this codeword's tile, extrapolated by N / N_seen (Eq. "aproxdenom").
      const int t = ntiles ? j / a.tile_m : 0;
      for (int i = 0; i < rows; ++i) {
        float s = logit(qs + (size_t)i * d, Cph + (size_t)j * d, d, a.scale);
        acc += (double)expf(s - rm[i]) / (double)(ntiles ? zt[(size_t)i * ntiles + t] : rz[i]);
      }
      acc *= (double)npS[j];
      if (ntiles) acc *= (double)nseen[t] / (double)a.Nk;
    }
    w[j] = acc;
  }
  __syncthreads();
  if (a.importance_out) {
    float* io = a.importance_out + ((size_t)bh * a.nblk + blk) * M;
    for (int j = tid; j < M; j += kAttendThreads) io[j] = (float)w[j];
  }

  // ---- top-P by rank (ties -> lower index), then an ascending list
  for (int j = tid; j < M; j += kAttendThreads) {
    int rank = 0;
    const double wj = w[j];
    for (int k = 0; k < M; ++k) {
      const double wk = w[k];
      rank += (wk > wj) || (wk == wj && k < j);
    }
    sel[j] = rank < P;
  }
  __syncthreads();
  for (int j = tid; j < M; j += kAttendThreads) {
    if (sel[j]) {
      int pos = 0;
      for (int k = 0; k < j; ++k) pos += sel[k];
      sel_list[pos] = j;
    }
  }
  __syncthreads();
  if (a.topp_out) {
    int32_t* to = a.topp_out + ((size_t)bh * a.nblk + blk) * P;
    for (int r = tid; r < P; r += kAttendThreads) to[r] = sel_list[r];
  }

  // ---- merged softmax over unrefined parents, stay residuals and children of refined parents
  T* Yb = static_cast<T*>(a.Y) + ((size_t)bh * a.Nq + i0) * d;
  for (int i = warp; i < rows; i += nwarps) {
    const float* q = qs + (size_t)i * d;
    float mx = -INFINITY;
    for (int j = lane; j < M; j += 32) {
      float s = logit(q, Cph + (size_t)j * d, d, a.scale);
      sb[j] = s;
      const float cnt = (sel[j] && !a.correcting) ? (a.stays ? nstay[j] : 0.f) : npS[j];
      if (cnt > 0.f) mx = fmaxf(mx, s);
    }
    for (int e = lane; e < P * C; e += 32) {
      const int p = sel_list[e / C], c = e % C;
      float s = logit(q, Cch + ((size_t)p * C + c) * d, d, a.scale);
      sb[M + e] = s;
      if (nc[p * C + c] > 0.f) mx = fmaxf(mx, s);
    }
    mx = warp_max(mx);
    __syncwarp();
    float x[kMaxDPerLane];
#pragma unroll
    for (int u = 0; u < kMaxDPerLane; ++u) x[u] = 0.f;
    float z = 0.f;
    for (int j = 0; j < M; ++j) {
      // correcting form: every parent keeps its full term here, the children add differences below
      const bool s_ = sel[j] != 0 && !a.correcting;
      const float cnt = s_ ? (a.stays ? nstay[j] : 0.f) : npS[j];
      if (!(cnt > 0.f)) continue;
      const float av = expf(sb[j] - mx);
      z += av * cnt;
#pragma unroll
      for (int u = 0; u < kMaxDPerLane; ++u) {
        const int k = lane + 32 * u;
        if (k < d) {
          float v = Vp[(size_t)j * d + k];
          if (s_)
            for (int c = 0; c < C; ++c) v -= Vc[((size_t)j * C + c) * d + k];
          x[u] = fmaf(av, v, x[u]);
        }
      }
    }
    for (int e = 0; e < P * C; ++e) {
      const int p = sel_list[e / C], c = e % C;
      const float cnt = nc[p * C + c];
      if (!(cnt > 0.f)) continue;
      float av = expf(sb[M + e] - mx);
      if (a.correcting) {
        // Eq. "parent_recovery": under parent = mean(children) the parent's logit is the mean of its
        // children's; Eq. "correcting_attention": the child's keys trade the parent's weight for their own
        float sp = 0.f;
        for (int c2 = 0; c2 < C; ++c2) sp += sb[M + (e / C) * C + c2];
        av -= expf(sp / (float)C - mx);
      }
      z += av * cnt;
#pragma unroll
      for (int u = 0; u < kMaxDPerLane; ++u) {
        const int k = lane + 32 * u;
        if (k < d) x[u] = fmaf(av, Vc[((size_t)p * C + c) * d + k], x[u]);
      }
    }
    const float inv = 1.f / z;
#pragma unroll
    for (int u = 0; u < kMaxDPerLane; ++u) {
      const int k = lane + 32 * u;
      if (k < d) stf(Yb + (size_t)i * d + k, x[u] * inv);
    }
    __syncwarp();
  }
}

}  // namespace (the size below is also used by the host-side validation)

size_t simt_attend_smem_bytes(int d, int M, int C, int P, int block_q, int tile_m) {
  const size_t ncols = (size_t)M + (size_t)P * C;
  size_t b = sizeof(double) * M;
  b += sizeof(float) * ((size_t)block_q * d + 2 * (size_t)block_q + 2 * (size_t)M +
                        (kAttendThreads / 32) * ncols);
  b += sizeof(int) * ((size_t)M + (size_t)(P > 0 ? P : 1));
  if (tile_m > 0) b += sizeof(float) * ((size_t)block_q + 1) * ((M + tile_m - 1) / tile_m);
  return b;
}

namespace {

template <typename T>
avq_status launch_assign(const avq_problem& p, const void* K, const void* Cp, const void* Cc,
                         int32_t* pidx, int32_t* cidx, cudaStream_t st) {
  const size_t smem = sizeof(float) * ((size_t)kAssignKeys * (p.d + 1) + (size_t)kAssignCodes * p.d);
  auto kern = assign_simt_kernel<T>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return AVQ_ERR_CUDA;
  dim3 grid((p.Nk + kAssignKeys - 1) / kAssignKeys, p.B * p.H);
  kern<<<grid, kAssignKeys, smem, st>>>(static_cast<const T*>(K), static_cast<const T*>(Cp),
                                        static_cast<const T*>(Cc), pidx, cidx, p.H, p.Nk, p.d, p.M, p.C,
                                        (p.flags & AVQ_FLAG_PARENT_STAYS) ? 1 : 0);
  return cuda_ok(cudaGetLastError());
}

template <typename T>
avq_status launch_aggregate(const avq_problem& p, const void* V, const int32_t* pidx, const int32_t* cidx,
                            float* Vp, float* np_, float* Vc, float* nc, cudaStream_t st) {
  const int keys_per_cta = 256;
  dim3 grid((p.Nk + keys_per_cta - 1) / keys_per_cta, p.B * p.H);
  aggregate_simt_kernel<T><<<grid, 256, 0, st>>>(static_cast<const T*>(V), pidx, cidx, Vp, np_, Vc, nc,
                                                p.Nk, p.d, p.M, p.C, keys_per_cta);
  return cuda_ok(cudaGetLastError());
}

template <typename T>
avq_status launch_attend(const AttendArgs& a, int B, cudaStream_t st) {
  const size_t smem = simt_attend_smem_bytes(a.d, a.M, a.C, a.P, a.block_q, a.tile_m);
  if (smem > kSimtAttendSmemLimit) return AVQ_ERR_UNSUPPORTED;   // validate_forward rejects these up front
  auto kern = attend_simt_kernel<T>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return AVQ_ERR_CUDA;
  dim3 grid(a.nblk, B * a.H);
  kern<<<grid, kAttendThreads, smem, st>>>(a);
  return cuda_ok(cudaGetLastError());
}

}  // namespace

avq_status simt_assign(const avq_problem& p, const void* K, const void* Cp, const void* Cc,
                       int32_t* parent_idx, int32_t* child_idx, cudaStream_t st) {
  return p.dtype == AVQ_F32 ? launch_assign<float>(p, K, Cp, Cc, parent_idx, child_idx, st)
                            : launch_assign<__nv_bfloat16>(p, K, Cp, Cc, parent_idx, child_idx, st);
}

avq_status simt_aggregate(const avq_problem& p, const void* V, const int32_t* parent_idx,
                          const int32_t* child_idx, float* Vp, float* np_, float* Vc, float* nc,
                          cudaStream_t st) {
  const size_t BH = (size_t)p.B * p.H;
  cudaError_t e = cudaMemsetAsync(Vp, 0, sizeof(float) * BH * p.M * p.d, st);
  if (e == cudaSuccess) e = cudaMemsetAsync(np_, 0, sizeof(float) * BH * p.M, st);
  if (e == cudaSuccess) e = cudaMemsetAsync(Vc, 0, sizeof(float) * BH * p.M * p.C * p.d, st);
  if (e == cudaSuccess) e = cudaMemsetAsync(nc, 0, sizeof(float) * BH * p.M * p.C, st);
  if (e != cudaSuccess) return AVQ_ERR_CUDA;
  return p.dtype == AVQ_F32
             ? launch_aggregate<float>(p, V, parent_idx, child_idx, Vp, np_, Vc, nc, st)
             : launch_aggregate<__nv_bfloat16>(p, V, parent_idx, child_idx, Vp, np_, Vc, nc, st);
}

avq_status simt_attend(const avq_problem& p, const void* Q, const void* Cp, const void* Cc,
                       const float* Vp, const float* np_, const float* Vc, const float* nc, int32_t P,
                       int32_t block_q, void* Y, int32_t* topp_out, float* importance_out,
                       int32_t tile_m, cudaStream_t st) {
  AttendArgs a;
  a.tile_m = tile_m;
  a.Nk = p.Nk;
  a.Q = Q; a.Cp = Cp; a.Cc = Cc; a.Vp = Vp; a.np_ = np_; a.Vc = Vc; a.nc = nc; a.Y = Y;
  a.topp_out = topp_out; a.importance_out = importance_out;
  a.H = p.H; a.Nq = p.Nq; a.d = p.d; a.M = p.M; a.C = p.C; a.P = P; a.block_q = block_q;
  a.nblk = (p.Nq + block_q - 1) / block_q;
  a.stays = (p.flags & AVQ_FLAG_PARENT_STAYS) ? 1 : 0;
  a.correcting = (p.flags & AVQ_FLAG_CORRECTING) ? 1 : 0;
  a.scale = p.scale;
  return p.dtype == AVQ_F32 ? launch_attend<float>(a, p.B, st) : launch_attend<__nv_bfloat16>(a, p.B, st);
}

}  // namespace avq
