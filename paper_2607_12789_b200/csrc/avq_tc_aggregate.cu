// Value aggregation for the bf16 path (Eq. "aggregates"; the scatter steps of Algorithm 1).
//
// (After a bounded wait has expired in the assign kernel its indices are meaningless but in range, so these
// kernels run on regardless - they only flag indices that are out of range - and the attention kernel,
// which reads the status word, leaves without writing.)
//
// leaf_scatter_kernel  one warp per 8 keys: each key's V row is added to the sum of its leaf
//                      codeword (parent, child) with vector reductions to global memory, and
//                      the leaf's count is bumped.  Only the leaf level is scattered; a key whose
//                      child index is -1 (it stays with its parent, Algorithm 1's masked scatter)
//                      goes to its parent's "stay" leaf, which is the parent's own row of Vp / np.
// finalize_kernel      per parent: Vp = stay part + sum over its children (every key sits in
//                      exactly one leaf, so the parent sum is the sum of its leaves), np likewise, and
//                      the bf16 operands the attention kernel stages (rows = codewords, the
//                      MN-major B operand of its value MMAs), as per-codeword MEANS (sum / count, zero
//                      for an empty codeword):
//                        Vpb [B,H,M,d]    parent value means
//                        Vcb [B,H,M,C,d]  leaf value means: a parent's C children are C consecutive rows
#include <type_traits>

#include "avq_tc_common.cuh"

namespace avq {
namespace {

constexpr int kScatterThreads = 256;
constexpr int kKeysPerWarp = 8;
constexpr int kKeysPerCta = kKeysPerWarp * (kScatterThreads / 32);

// One warp = 8 consecutive keys: their indices are read with one coalesced load and broadcast by
// shuffle, the 8 value rows are loaded before the first reduction is issued.
template <int D>
__global__ void __launch_bounds__(kScatterThreads)
leaf_scatter_kernel(const __nv_bfloat16* __restrict__ V, const int32_t* __restrict__ pidx,
                    const int32_t* __restrict__ cidx, float* __restrict__ Vc, float* __restrict__ nc,
                    float* __restrict__ Vp, float* __restrict__ np_, int Nk, int M, int C,
                    int32_t* status_word) {
  tc::pdl_launch_dependents();
  const int bh = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int j0 = blockIdx.x * kKeysPerCta + warp * kKeysPerWarp;
  const size_t kb = (size_t)bh * Nk;
  // Every lane adds four floats with one 16-byte reduction: a full warp covers a 128-wide row, a
  // half warp a 64-wide one (two keys per step).  The value rows are the caller's: their loads go out
  // before the wait for the kernel that writes the indices.
  constexpr int kLanesPerRow = D / 4;
  constexpr int kRowsPerStep = 32 / kLanesPerRow;
  constexpr int kSteps = kKeysPerWarp / kRowsPerStep;
  const int sub = lane / kLanesPerRow, col = lane % kLanesPerRow;
  uint2 v[kSteps];
#pragma unroll
  for (int t = 0; t < kSteps; ++t) {
    const int j = j0 + t * kRowsPerStep + sub;
    v[t] = make_uint2(0u, 0u);
    if (j < Nk) v[t] = __ldg(reinterpret_cast<const uint2*>(V + (kb + j) * D) + col);
  }
  tc::pdl_wait();                                    // the indices come from the kernel before
  if (j0 >= Nk) return;
  // leaf_l: a * C + c for a key that moved to child c, kStayBit | a for a key that stays, -1 = nothing to add
  constexpr int kStayBit = 1 << 30;
  int leaf_l = -1;
  if (lane < kKeysPerWarp && j0 + lane < Nk) {
    const int a = tc::ld_after_wait(pidx + kb + j0 + lane);   // ordered behind the dependency wait
    const int c = tc::ld_after_wait(cidx + kb + j0 + lane);
    if (a < 0 || a >= M || c < -1 || c >= C) {       // caller-supplied index out of range: skip the key, flag it
      if (status_word) atomicCAS(status_word, 0, DEV_BAD_INDEX);
    } else {
      leaf_l = c < 0 ? (kStayBit | a) : a * C + c;
    }
  }
#pragma unroll
  for (int t = 0; t < kSteps; ++t) {
    const int leaf = __shfl_sync(0xffffffffu, leaf_l, t * kRowsPerStep + sub);
    if (leaf >= 0) {
      float* dst = (leaf & kStayBit) ? Vp + ((size_t)bh * M + (leaf & ~kStayBit)) * D
                                     : Vc + ((size_t)bh * M * C + leaf) * D;
      const uint2 u = v[t];
      atomicAdd(reinterpret_cast<float4*>(dst) + col,
                make_float4(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xFFFF0000u),
                            __uint_as_float(u.y << 16), __uint_as_float(u.y & 0xFFFF0000u)));
    }
  }
  if (leaf_l >= 0) {
    if (leaf_l & kStayBit) atomicAdd(np_ + (size_t)bh * M + (leaf_l & ~kStayBit), 1.0f);
    else atomicAdd(nc + (size_t)bh * M * C + leaf_l, 1.0f);
  }
}

// Long sequences over few codewords put hundreds of keys on every leaf, and the reductions above then
// queue on the same addresses.  This variant gives one CTA a contiguous chunk of a head's keys, orders
// the chunk by leaf with a counting sort in shared memory (integer atomics only) and lets every warp walk
// an equal share of the ordered list, summing in registers: a leaf costs one global reduction per CTA
// (one more where a leaf straddles two warps' shares) instead of one per key.
constexpr int kSortThreads = 512;
constexpr int kSortKeysPerThread = 16;
constexpr int kSortMaxKeys = kSortThreads * kSortKeysPerThread;   // keys per CTA (16-bit key field of the order list)
constexpr int kSortMaxLeaves = 256 * 9;                           // M * (C + 1) <= 256 * 9: C children + the stay leaf
// The chunked variant is chosen for heads of at least kSortMinKeys keys when a CTA's chunk holds at least
// 0.8 keys per leaf (measured: faster from there on; short heads leave its 512-thread CTAs idle).
constexpr int kSortRatio10 = 8;
constexpr int kSortMinKeys = 2048;

template <int D>
__global__ void __launch_bounds__(kSortThreads, 2)
leaf_sorted_kernel(const __nv_bfloat16* __restrict__ V, const int32_t* __restrict__ pidx,
                   const int32_t* __restrict__ cidx, float* __restrict__ Vc, float* __restrict__ nc,
                   float* __restrict__ Vp, float* __restrict__ np_, int Nk, int M, int C, int chunk,
                   int32_t* status_word) {
  // leaves: (parent, child) pairs at a * C + c, then one "stay" leaf per parent at M * C + a
  const int MC = M * C, L = MC + M;
  extern __shared__ __align__(16) unsigned char sort_smem[];
  int* hist = reinterpret_cast<int*>(sort_smem);        // [L] keys per leaf
  int* offs = hist + L;                                 // [L] first slot of each leaf in `order`
  int* wsum = offs + L;                                 // [16] per-warp totals of the scan
  uint32_t* order = reinterpret_cast<uint32_t*>(wsum + 16);   // [chunk] leaf << 16 | key (relative to the chunk)
  tc::pdl_launch_dependents();
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int bh = blockIdx.y;
  const int j0 = blockIdx.x * chunk;
  const int n = min(chunk, Nk - j0);
  for (int l = tid; l < L; l += kSortThreads) hist[l] = 0;
  __syncthreads();
  tc::pdl_wait();                                      // the indices come from the kernel before
  if (n <= 0) return;
  const size_t kb = (size_t)bh * Nk + j0;

  // ---- leaf of every key and its rank among the chunk's keys of that leaf
  uint32_t lr[kSortKeysPerThread];                     // leaf << 16 | rank
  // all index loads first: they are ordered statements (behind the dependency wait) that the compiler will
  // not move across the shared-memory atomics below, so issued one key at a time each would cost a round trip
  int av[kSortKeysPerThread], cv[kSortKeysPerThread];
#pragma unroll
  for (int t = 0; t < kSortKeysPerThread; ++t) {
    const int j = tid + t * kSortThreads;
    av[t] = cv[t] = 0;
    if (j < n) {
      av[t] = tc::ld_after_wait(pidx + kb + j);
      cv[t] = tc::ld_after_wait(cidx + kb + j);
    }
  }
#pragma unroll
  for (int t = 0; t < kSortKeysPerThread; ++t) {
    const int j = tid + t * kSortThreads;
    lr[t] = 0xFFFFFFFFu;
    if (j < n) {
      const int a = av[t], c = cv[t];
      if (a < 0 || a >= M || c < -1 || c >= C) {       // caller-supplied index out of range: skip the key, flag it
        if (status_word) atomicCAS(status_word, 0, DEV_BAD_INDEX);
      } else {
        const int leaf = c < 0 ? MC + a : a * C + c;
        lr[t] = ((uint32_t)leaf << 16) | (uint32_t)atomicAdd(&hist[leaf], 1);
      }
    }
  }
  __syncthreads();

  // ---- exclusive scan of the histogram: thread t owns entries [t * E, (t + 1) * E); key counts go out
  {
    const int E = (L + kSortThreads - 1) / kSortThreads;   // <= 5
    int c[5] = {0, 0, 0, 0, 0}, tot = 0;
#pragma unroll
    for (int e = 0; e < 5; ++e)
      if (e < E && tid * E + e < L) {
        c[e] = hist[tid * E + e];
        tot += c[e];
        if (c[e] > 0) {
          const int leaf = tid * E + e;
          atomicAdd(leaf < MC ? nc + (size_t)bh * MC + leaf : np_ + (size_t)bh * M + (leaf - MC), (float)c[e]);
        }
      }
    int inc = tot;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int up = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += up;
    }
    if (lane == 31) wsum[warp] = inc;
    __syncthreads();
    int base = inc - tot;
    for (int u = 0; u < warp; ++u) base += wsum[u];
#pragma unroll
    for (int e = 0; e < 5; ++e)
      if (e < E && tid * E + e < L) { offs[tid * E + e] = base; base += c[e]; }
  }
  __syncthreads();
#pragma unroll
  for (int t = 0; t < kSortKeysPerThread; ++t)
    if (lr[t] != 0xFFFFFFFFu)
      order[offs[lr[t] >> 16] + (int)(lr[t] & 0xFFFFu)] = (lr[t] & 0xFFFF0000u) | (uint32_t)(tid + t * kSortThreads);
  __syncthreads();

  // ---- every warp walks an equal share of the ordered list, 16 rows in flight (lane = 2 or 4 consecutive
  // head dimensions), and flushes its register sum whenever the leaf changes
  using Word = typename std::conditional<D == 64, uint32_t, uint2>::type;
  const Word* Vw = reinterpret_cast<const Word*>(V + kb * D) + lane;   // row j at Vw + j * 32
  constexpr int kWarps = kSortThreads / 32, kBatch = 16;
  const int listed = offs[L - 1] + hist[L - 1];         // keys in the ordered list (= n unless some were skipped)
  const int share = (listed + kWarps - 1) / kWarps;
  const int s0 = warp * share, s1 = min(listed, s0 + share);
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  int cur = -1;
  auto flush = [&]() {
    if (cur < 0) return;
    float* dst = cur < MC ? Vc + ((size_t)bh * MC + cur) * D : Vp + ((size_t)bh * M + (cur - MC)) * D;
    if constexpr (D == 64) atomicAdd(reinterpret_cast<float2*>(dst) + lane, make_float2(acc[0], acc[1]));
    else atomicAdd(reinterpret_cast<float4*>(dst) + lane, make_float4(acc[0], acc[1], acc[2], acc[3]));
    acc[0] = acc[1] = acc[2] = acc[3] = 0.f;
  };
  auto add_row = [&](uint32_t e, const Word& w) {
    const int leaf = (int)(e >> 16);
    if (leaf != cur) { flush(); cur = leaf; }          // warp-uniform
    if constexpr (D == 64) {
      acc[0] += __uint_as_float(w << 16);
      acc[1] += __uint_as_float(w & 0xFFFF0000u);
    } else {
      acc[0] += __uint_as_float(w.x << 16);
      acc[1] += __uint_as_float(w.x & 0xFFFF0000u);
      acc[2] += __uint_as_float(w.y << 16);
      acc[3] += __uint_as_float(w.y & 0xFFFF0000u);
    }
  };
  int i = s0;
  for (; i + kBatch <= s1; i += kBatch) {               // full batches: one list read per batch, no guards
    const uint32_t ev = order[i + (lane & (kBatch - 1))];
    Word w[kBatch];
#pragma unroll
    for (int u = 0; u < kBatch; ++u)
      w[u] = __ldg(Vw + (size_t)(__shfl_sync(0xffffffffu, ev, u) & 0xFFFFu) * 32);
#pragma unroll
    for (int u = 0; u < kBatch; ++u) add_row(__shfl_sync(0xffffffffu, ev, u), w[u]);
  }
  if (i < s1) {                                         // ragged tail of the share
    const uint32_t ev = order[min(i + (lane & (kBatch - 1)), s1 - 1)];
    Word w[kBatch];
#pragma unroll
    for (int u = 0; u < kBatch; ++u)
      w[u] = __ldg(Vw + (size_t)(__shfl_sync(0xffffffffu, ev, u) & 0xFFFFu) * 32);
#pragma unroll
    for (int u = 0; u < kBatch; ++u)
      if (i + u < s1) add_row(__shfl_sync(0xffffffffu, ev, u), w[u]);
  }
  flush();
}

// One CTA: kPer consecutive parents of one (batch, head) (8 with four children each, 4 with eight: 32 leaf
// rows); thread k owns head-dimension index k.  Every load is issued before the first use.
// 1 / n for a key count (a small positive integer held in a float): the approximate reciprocal (one XU
// instruction, within an ulp or two) is far inside what the bf16 rounding of the mean leaves of it.  The
// correctly rounded __frcp_rn is a long dependent sequence, 40 of which per thread were most of this kernel's
// time on the few warps it runs with.
__device__ __forceinline__ float fast_rcp(float x) {
  float y;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

template <int D, int C>
__global__ void __launch_bounds__(D * ((C == 4) ? 8 : 4))
finalize_kernel(const float* __restrict__ Vc, const float* __restrict__ nc, float* __restrict__ Vp,
                float* __restrict__ np_, __nv_bfloat16* __restrict__ Vpb, __nv_bfloat16* __restrict__ Vcb,
                __nv_bfloat16* __restrict__ Vsb, float* __restrict__ rho, int M) {
  // One CTA = kPer consecutive parents of one (batch, head); thread (k, mm) owns head-dimension index k of
  // parent mm: C + 1 row loads, C + 2 counts, a handful of stores.  The kernel is a load round trip followed
  // by a little arithmetic, so it wants many short threads, not few long ones.
  constexpr int kPer = (C == 4) ? 8 : 4;
  tc::pdl_launch_dependents();
  tc::pdl_wait();                                    // the leaf sums come from the kernel before
  const int bh = blockIdx.y, k = threadIdx.x, mm = threadIdx.y;
  const size_t row = (size_t)bh * M + blockIdx.x * kPer + mm;
  // Everything read here is written by the kernel before this one: the loads are statements the compiler
  // cannot move ahead of the dependency wait above (an ordinary load of np_ was seen to be scheduled ahead of
  // it, reading counts the scatter had not finished).
  float x[C], cn[C];
#pragma unroll
  for (int c = 0; c < C; ++c) {
    x[c] = tc::ld_after_wait(Vc + (row * C + c) * D + k);
    cn[c] = tc::ld_after_wait(nc + row * C + c);
  }
  const float stay = tc::ld_after_wait(Vp + row * D + k);   // zero unless keys stay
  const float nstay = tc::ld_after_wait(np_ + row);         // keys that stay
  float s = stay, n = nstay;
#pragma unroll
  for (int c = 0; c < C; ++c) {
    s += x[c];
    n += cn[c];
    // the attention kernel takes per-codeword MEANS: the count rides in its softmax weights
    if (Vcb) Vcb[(row * C + c) * D + k] = __float2bfloat16_rn(cn[c] > 0.f ? x[c] * fast_rcp(cn[c]) : 0.f);
  }
  Vp[row * D + k] = s;
  const float rn = n > 0.f ? fast_rcp(n) : 0.f;
  if (Vpb) Vpb[row * D + k] = __float2bfloat16_rn(s * rn);
  // what a refined parent keeps under the PARENT_STAYS rule, per key of the parent: its weight in the
  // attention kernel is A n_p, so the row is Vbar_stay / n_p and the count n_stay / n_p
  if (Vsb) Vsb[row * D + k] = __float2bfloat16_rn(stay * rn);
  if (rho && k == 0) rho[row] = nstay * rn;
  __syncthreads();                                     // every thread has read its parent's stay count
  if (k == 0) np_[row] = n;
}

// Zeroes the four accumulator arrays of a stand-alone avq_aggregate in one launch (inside avq_forward the
// assign grid clears them on the side).
__global__ void __launch_bounds__(256) clear_accumulators_kernel(float* a, size_t na, float* b, size_t nb, float* c,
                                                                 size_t nc_, float* d, size_t nd) {
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < na; i += stride) a[i] = 0.f;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < nb; i += stride) b[i] = 0.f;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < nc_; i += stride) c[i] = 0.f;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < nd; i += stride) d[i] = 0.f;
}

template <int D, int C>
avq_status run(const avq_problem& p, const void* V, const int32_t* pidx, const int32_t* cidx, float* Vp,
               float* np_, float* Vc, float* nc, void* Vpb, void* Vcb, void* Vsb, float* rho, bool pre_zeroed,
               int32_t* status_word, cudaStream_t st) {
  const unsigned BH = (unsigned)(p.B * p.H);
  if (!pre_zeroed) {                                   // the stand-alone call: one launch clears the four accumulators
    const size_t n_c = (size_t)BH * p.M * C, n_p = (size_t)BH * p.M;
    const size_t total = (n_c + n_p) * (D + 1);
    const unsigned blocks = (unsigned)((total + 4 * 256 - 1) / (4 * 256) < 2048 ? (total + 4 * 256 - 1) / (4 * 256) : 2048);
    clear_accumulators_kernel<<<blocks, 256, 0, st>>>(Vc, n_c * D, nc, n_c, Vp, n_p * D, np_, n_p);
    if (cudaGetLastError() != cudaSuccess) return AVQ_ERR_CUDA;
  }
  // `pre_zeroed` marks the chained call from avq_forward: the kernel before in the stream is the assign
  // kernel, so the scatter may be launched as its programmatic dependent.
  // Chunked variant when a CTA's share of a long head holds about a key per leaf or more: two CTAs per SM.
  const int L = p.M * C;
  int sms = 148;
  {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return AVQ_ERR_CUDA;
    static int cached_sms[64] = {};
    if (dev >= 0 && dev < 64 && cached_sms[dev] > 0) sms = cached_sms[dev];
    else {
      if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return AVQ_ERR_CUDA;
      if (dev >= 0 && dev < 64) cached_sms[dev] = sms;
    }
  }
  int per_head = 2 * sms / (int)BH;                      // rounded down: the grid must fit in one wave
  if (per_head < 1) per_head = 1;
  int chunk = (p.Nk + per_head - 1) / per_head;
  if (chunk > kSortMaxKeys) chunk = kSortMaxKeys;
  chunk = (chunk + 31) & ~31;
  if (L <= kSortMaxLeaves && p.Nk >= kSortMinKeys && chunk * 10 >= kSortRatio10 * L) {
    dim3 g1((p.Nk + chunk - 1) / chunk, BH);
    const size_t smem = sizeof(int) * (2 * (size_t)p.M * (C + 1) + 16) + sizeof(uint32_t) * (size_t)chunk;
    // above the default limit only for the largest leaf count and chunk: opt in once per device
    static bool configured[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return AVQ_ERR_CUDA;
    if (dev < 0 || dev >= 64 || !configured[dev]) {
      const int max_smem = (int)(sizeof(int) * (2 * kSortMaxLeaves + 16) + sizeof(uint32_t) * kSortMaxKeys);
      if (cudaFuncSetAttribute(leaf_sorted_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem) !=
          cudaSuccess)
        return AVQ_ERR_CUDA;
      if (dev >= 0 && dev < 64) configured[dev] = true;
    }
    if (tc::launch_pdl(leaf_sorted_kernel<D>, g1, dim3(kSortThreads), smem, st, pre_zeroed,
                       static_cast<const __nv_bfloat16*>(V), pidx, cidx, Vc, nc, Vp, np_, p.Nk, p.M, C, chunk,
                       status_word) != cudaSuccess)
      return AVQ_ERR_CUDA;
  } else {
    dim3 g1((p.Nk + kKeysPerCta - 1) / kKeysPerCta, BH);
    if (tc::launch_pdl(leaf_scatter_kernel<D>, g1, dim3(kScatterThreads), 0, st, pre_zeroed,
                       static_cast<const __nv_bfloat16*>(V), pidx, cidx, Vc, nc, Vp, np_, p.Nk, p.M, C,
                       status_word) != cudaSuccess)
      return AVQ_ERR_CUDA;
  }
  dim3 g2(p.M / (C == 4 ? 8 : 4), BH);
  return cuda_ok(tc::launch_pdl(finalize_kernel<D, C>, g2, dim3(D, C == 4 ? 8 : 4), 0, st, true, static_cast<const float*>(Vc),
                                static_cast<const float*>(nc), Vp, np_, static_cast<__nv_bfloat16*>(Vpb),
                                static_cast<__nv_bfloat16*>(Vcb), static_cast<__nv_bfloat16*>(Vsb), rho, p.M));
}

}  // namespace

avq_status tc_aggregate(const avq_problem& p, const void* V, const int32_t* parent_idx,
                        const int32_t* child_idx, float* Vp, float* np_, float* Vc, float* nc, void* Vpb,
                        void* Vcb, void* Vsb, float* rho, bool pre_zeroed, int32_t* status_word, cudaStream_t st) {
  if (p.d == 64)
    return p.C == 4 ? run<64, 4>(p, V, parent_idx, child_idx, Vp, np_, Vc, nc, Vpb, Vcb, Vsb, rho, pre_zeroed, status_word, st)
                    : run<64, 8>(p, V, parent_idx, child_idx, Vp, np_, Vc, nc, Vpb, Vcb, Vsb, rho, pre_zeroed, status_word, st);
  return p.C == 4 ? run<128, 4>(p, V, parent_idx, child_idx, Vp, np_, Vc, nc, Vpb, Vcb, Vsb, rho, pre_zeroed, status_word, st)
                  : run<128, 8>(p, V, parent_idx, child_idx, Vp, np_, Vc, nc, Vpb, Vcb, Vsb, rho, pre_zeroed, status_word, st);
}

}  // namespace avq
