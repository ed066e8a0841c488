// Tensor-core attention pass of AVQ-attention (Algorithm 2 in its masked form) for bf16 inputs.
//
// One CTA = one query tile of 128 rows of one (batch, head), 8 warps.  The codeword columns are
// walked as tiles: tile 0 holds the M parents, later tiles hold the children of the selected
// parents in chunks.  Per tile:
//   codes [n x d] in shared memory (TMA for parents, gathered rows for children)
//   S = Q . codes^T          tcgen05.mma, fp32 accumulator in TMEM columns [0, n)
//   softmax weights          each query row is split over two threads (column halves); the
//                            row maximum runs over non-empty codewords only; weights of empty
//                            codewords are zero (appendix on numerical stability)
//   A (bf16) -> shared       K-major, 128-byte swizzle, in place of the codes
//   O += A . Vbar            tcgen05.mma into TMEM columns [CT, CT + d)
// Tile 0 additionally forms the importance w_j = n_j sum_i A_ij / z_i (Eq. "importance") from
// the fp32 weights, picks the P largest (ties to the lower index) and zeroes the selected
// parents' columns before they reach the second MMA: their keys are represented by the
// children instead.  When a later tile raises a row's maximum, that row of O is rescaled in
// TMEM.  The denominator uses the same bf16-rounded weights as the numerator.
#include "avq_tc_common.cuh"

namespace avq {
namespace {

using namespace tc;

constexpr int kRows = 128;
constexpr int kThreads = 256;

struct AttendParams {
  const __nv_bfloat16* Cc;    // [H, M, C, d]
  const __nv_bfloat16* VcT;   // [B*H, M, d, C]
  const float* np_;           // [B*H, M]
  const float* nc;            // [B*H, M, C]
  __nv_bfloat16* Y;           // [B*H, Nq, d]
  int32_t* topp_out;          // optional
  float* importance_out;      // optional
  int32_t* status_word;
  int H, Nq, M, C, P, nblk;
  int CT;                     // columns per tile (two halves of CT/2), multiple of 32, >= M
  uint32_t tmem_cols;
  float scale_log2e;
};

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float bf16_round(float x) { return __bfloat162float(__float2bfloat16_rn(x)); }

// Column sums over the 32 lanes of a warp of V values per lane.  Returns, in every lane, the
// sum of column (lane >> (5 - log2 V)).  V = 32: 31 shuffles instead of 160.
template <int V>
__device__ __forceinline__ float transpose_reduce(float (&v)[V], int lane) {
  int n = V;
#pragma unroll
  for (int b = 16; b >= 1; b >>= 1) {
    if (n > 1) {
      n >>= 1;
      const bool hi = (lane & b) != 0;
#pragma unroll
      for (int i = 0; i < V / 2; ++i) {
        if (i < n) {
          const float send = hi ? v[i] : v[i + n];
          const float keep = hi ? v[i + n] : v[i];
          v[i] = keep + __shfl_xor_sync(0xffffffffu, send, b);
        }
      }
    } else {
      v[0] += __shfl_xor_sync(0xffffffffu, v[0], b);
    }
  }
  return v[0];
}

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
tc_attend_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmCp,
                 const __grid_constant__ CUtensorMap tmVpT, const AttendParams p) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023u) & ~(uintptr_t)1023u);
  constexpr int kSubD = D / 64;
  const int CT = p.CT, MH = CT >> 1, M = p.M, C = p.C, P = p.P;
  const int subA = (CT + 63) >> 6;                       // 64-column sub-tiles of an A / value tile
  const int ca_bytes = max(CT * D * 2, subA * kRows * 128);
  unsigned char* Qs = smem;                              // kSubD x [128 x 128 B]
  unsigned char* CA = Qs + kSubD * kRows * 128;          // codes, later the bf16 weights
  unsigned char* Vs = CA + ca_bytes;                     // subA x [D x 128 B]
  float* cnt = reinterpret_cast<float*>(Vs + subA * D * 128);   // [CT] counts of the tile's codewords
  float* w = cnt + CT;                                   // [256] importance
  float* wpart = w + 256;                                // [4][CT]
  float* xm = wpart + 4 * CT;                            // [2][128] pair exchange: maxima
  float* xz = xm + 2 * kRows;                            // [2][128] pair exchange: sums
  float* xz2 = xz + 2 * kRows;                           // [2][128]
  int* sel_list = reinterpret_cast<int*>(xz2 + 2 * kRows);   // [256]
  uint32_t* wmask = reinterpret_cast<uint32_t*>(sel_list + 256);   // [8]
  uint64_t* bars = reinterpret_cast<uint64_t*>(wmask + 8);         // [4]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  unsigned char* selS = reinterpret_cast<unsigned char*>(tmem_slot + 2);   // [256]

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int q = warp & 3, hf = warp >> 2, r = q * 32 + lane;
  const int blk = blockIdx.x, bh = blockIdx.y, h = bh % p.H;
  const int i0 = blk * kRows;
  const int rows_valid = min(kRows, p.Nq - i0);
  uint64_t* bar_ld0 = &bars[0];
  uint64_t* bar_ld1 = &bars[1];
  uint64_t* bar_s = &bars[2];
  uint64_t* bar_pv = &bars[3];

  // A wait that expired in an earlier CTA of this launch: do not start more work.
  __shared__ int early_exit;
  if (tid == 0) early_exit = (p.status_word != nullptr && *reinterpret_cast<volatile int32_t*>(p.status_word) != 0);
  __syncthreads();
  if (early_exit) return;

  if (tid == 0) {
    mbar_init(bar_ld0, 1);
    mbar_init(bar_ld1, 1);
    mbar_init(bar_s, 1);
    mbar_init(bar_pv, 1);
    mbar_fence_init();
    *abort_flag = 0;
    prefetch_tmap(&tmQ);
    prefetch_tmap(&tmCp);
    prefetch_tmap(&tmVpT);
  }
  if (warp == 0) {
    tmem_alloc(tmem_slot, p.tmem_cols);
    tmem_relinquish();
  }
  for (int j = tid; j < CT; j += kThreads) cnt[j] = j < M ? p.np_[(size_t)bh * M + j] : 0.f;
  selS[tid] = 0;
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t t_s = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(hf * MH);
  const uint32_t t_o = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(CT + hf * (D / 2));
  const uint32_t idesc_o = umma_idesc_bf16(kRows, D);

  // ---- stage Q, the parent codebook and the parents' value sums; S = Q . Cp^T
  if (tid == 0) {
    mbar_expect_tx(bar_ld0, (uint32_t)(kSubD * (kRows + M) * 128));
#pragma unroll
    for (int s = 0; s < kSubD; ++s) {
      tma_load_3d(Qs + s * kRows * 128, &tmQ, s * 64, i0, bh, bar_ld0);
      tma_load_2d(CA + s * M * 128, &tmCp, s * 64, h * M, bar_ld0);
    }
    const int subM = (M + 63) >> 6;
    mbar_expect_tx(bar_ld1, (uint32_t)(subM * D * 128));
    for (int s = 0; s < subM; ++s) tma_load_2d(Vs + s * D * 128, &tmVpT, s * 64, bh * D, bar_ld1);
    if (mbar_wait(bar_ld0, 0, abort_flag, p.status_word, DEV_TIMEOUT_ATTEND)) {
      tc_fence_after();
      const uint32_t idesc = umma_idesc_bf16(kRows, M);
      const uint32_t qa = smem_u32(Qs), ca = smem_u32(CA);
#pragma unroll
      for (int k = 0; k < D / 16; ++k)
        umma_bf16(tmem_base, umma_desc_sw128(qa + (k / 4) * kRows * 128 + (k % 4) * 32),
                  umma_desc_sw128(ca + (k / 4) * M * 128 + (k % 4) * 32), idesc, k > 0);
      umma_commit(bar_s);
    }
  }

  float m_run = -INFINITY, z_run = 0.f;
  uint32_t ph_s = 0, ph_pv = 0;
  const int PC = P * C;
  int e0 = 0;           // first child column of the current child tile
  int ncols = M;        // valid columns of the current tile (tile 0: parents)
  for (int tile = 0;; ++tile) {
    const int ncols_pad = (ncols + 15) & ~15;
    const int my_cols = min(max(ncols_pad - hf * MH, 0), MH);   // multiple of 16

    // ---- wait for S, row maximum over non-empty codewords
    const bool s_ok = mbar_wait(bar_s, ph_s, abort_flag, p.status_word, DEV_TIMEOUT_ATTEND);
    ph_s ^= 1;
    tc_fence_after();
    float mloc = -INFINITY;
    if (s_ok) {
      for (int c0 = 0; c0 < my_cols; c0 += 16) {
        float s[16];
        tmem_ld16(t_s + c0, s);
#pragma unroll
        for (int e = 0; e < 16; ++e)
          if (cnt[hf * MH + c0 + e] > 0.f) mloc = fmaxf(mloc, s[e] * p.scale_log2e);
      }
    }
    xm[hf * kRows + r] = mloc;
    __syncthreads();
    const float m_new = fmaxf(m_run, fmaxf(xm[r], xm[kRows + r]));
    // m_new is finite from tile 0 on: at least one parent holds a key.

    if (tile == 0) {
      // ---- fp32 weights back into TMEM, exact denominator of the parent pass
      float zloc = 0.f;
      for (int c0 = 0; c0 < my_cols; c0 += 16) {
        float s[16];
        tmem_ld16(t_s + c0, s);
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          const float n = cnt[hf * MH + c0 + e];
          s[e] = n > 0.f ? ex2(fmaf(s[e], p.scale_log2e, -m_new)) : 0.f;
          zloc = fmaf(s[e], n, zloc);
        }
        tmem_st16(t_s + c0, s);
      }
      tmem_st_wait();
      xz[hf * kRows + r] = zloc;
      __syncthreads();
      const float zfull = xz[r] + xz[kRows + r];
      const float inv = (r < rows_valid) ? 1.f / zfull : 0.f;
      // ---- importance: column sums of A_ij / z_i over the 128 rows
      for (int c0 = 0; c0 < my_cols; c0 += 32) {
        float v[32];
        {
          float a[16];
          tmem_ld16(t_s + c0, a);
#pragma unroll
          for (int e = 0; e < 16; ++e) v[e] = a[e] * inv;
          if (c0 + 16 < my_cols) {
            tmem_ld16(t_s + c0 + 16, a);
#pragma unroll
            for (int e = 0; e < 16; ++e) v[16 + e] = a[e] * inv;
          } else {
#pragma unroll
            for (int e = 0; e < 16; ++e) v[16 + e] = 0.f;
          }
        }
        const float colsum = transpose_reduce<32>(v, lane);
        if (c0 + lane < my_cols) wpart[q * CT + hf * MH + c0 + lane] = colsum;
      }
      __syncthreads();
      if (tid < M) {
        const float wj = cnt[tid] * (wpart[tid] + wpart[CT + tid] + wpart[2 * CT + tid] + wpart[3 * CT + tid]);
        w[tid] = wj;
        if (p.importance_out) p.importance_out[((size_t)bh * p.nblk + blk) * M + tid] = wj;
      }
      __syncthreads();
      // ---- top-P by rank, ties to the lower index; ascending list
      bool mine = false;
      if (tid < M) {
        const float wj = w[tid];
        int rank = 0;
        for (int k = 0; k < M; ++k) {
          const float wk = w[k];
          rank += (wk > wj) || (wk == wj && k < tid);
        }
        mine = rank < P;
        selS[tid] = mine ? 1 : 0;
      }
      const uint32_t bal = __ballot_sync(0xffffffffu, mine);
      if (lane == 0) wmask[warp] = bal;
      __syncthreads();
      if (mine) {
        int pos = __popc(bal & ((1u << lane) - 1u));
        for (int u = 0; u < warp; ++u) pos += __popc(wmask[u]);
        sel_list[pos] = tid;
        if (p.topp_out) p.topp_out[((size_t)bh * p.nblk + blk) * P + pos] = tid;
      }
      // ---- masked bf16 weights into shared memory (over the dead codebook), denominator
      zloc = 0.f;
      for (int c0 = 0; c0 < my_cols; c0 += 16) {
        float a[16];
        tmem_ld16(t_s + c0, a);
        uint32_t pk[8];
#pragma unroll
        for (int e = 0; e < 16; e += 2) {
          const int col = hf * MH + c0 + e;
          const float a0 = selS[col] ? 0.f : bf16_round(a[e]);
          const float a1 = selS[col + 1] ? 0.f : bf16_round(a[e + 1]);
          zloc = fmaf(a0, cnt[col], zloc);
          zloc = fmaf(a1, cnt[col + 1], zloc);
          pk[e >> 1] = pack_bf16(a0, a1);
        }
        const int col0 = hf * MH + c0;
        unsigned char* sub = CA + (col0 >> 6) * (kRows * 128);
        *reinterpret_cast<uint4*>(sub + sw128_offset(r, col0 & 63)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
        *reinterpret_cast<uint4*>(sub + sw128_offset(r, (col0 & 63) + 8)) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
      }
      xz2[hf * kRows + r] = zloc;
      m_run = m_new;
    } else {
      // ---- child tile: rescale what has been accumulated if this row's maximum moved
      const float alpha = ex2(m_run - m_new);
      if (__any_sync(0xffffffffu, alpha < 1.f)) {
        for (int c0 = 0; c0 < D / 2; c0 += 16) {
          float o[16];
          tmem_ld16(t_o + c0, o);
#pragma unroll
          for (int e = 0; e < 16; ++e) o[e] *= alpha;
          tmem_st16(t_o + c0, o);
        }
        tmem_st_wait();
      }
      z_run *= alpha;
      m_run = m_new;
      float zloc = 0.f;
      for (int c0 = 0; c0 < my_cols; c0 += 16) {
        float a[16];
        if (s_ok) tmem_ld16(t_s + c0, a);
        uint32_t pk[8];
#pragma unroll
        for (int e = 0; e < 16; e += 2) {
          const int col = hf * MH + c0 + e;
          const float n0 = cnt[col], n1 = cnt[col + 1];
          const float a0 = n0 > 0.f ? bf16_round(ex2(fmaf(a[e], p.scale_log2e, -m_new))) : 0.f;
          const float a1 = n1 > 0.f ? bf16_round(ex2(fmaf(a[e + 1], p.scale_log2e, -m_new))) : 0.f;
          zloc = fmaf(a0, n0, zloc);
          zloc = fmaf(a1, n1, zloc);
          pk[e >> 1] = pack_bf16(a0, a1);
        }
        const int col0 = hf * MH + c0;
        unsigned char* sub = CA + (col0 >> 6) * (kRows * 128);
        *reinterpret_cast<uint4*>(sub + sw128_offset(r, col0 & 63)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
        *reinterpret_cast<uint4*>(sub + sw128_offset(r, (col0 & 63) + 8)) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
      }
      xz2[hf * kRows + r] = zloc;
    }
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    z_run += xz2[r] + xz2[kRows + r];

    // ---- O (+)= A . Vbar for this tile
    if (tid == 0) {
      tc_fence_after();
      const bool v_ok = tile > 0 || mbar_wait(bar_ld1, 0, abort_flag, p.status_word, DEV_TIMEOUT_ATTEND);
      if (v_ok) {
        const uint32_t aa = smem_u32(CA), va = smem_u32(Vs);
        for (int k = 0; k < ncols_pad / 16; ++k)
          umma_bf16(tmem_base + CT, umma_desc_sw128(aa + (k / 4) * kRows * 128 + (k % 4) * 32),
                    umma_desc_sw128(va + (k / 4) * D * 128 + (k % 4) * 32), idesc_o, tile > 0 || k > 0);
      }
      umma_commit(bar_pv);
    }

    // ---- next child tile, if any
    if (e0 >= PC) break;
    const int e1 = min(PC, e0 + CT);
    ncols = e1 - e0;
    const int np16 = (ncols + 15) & ~15;
    // The second MMA reads A (in CA) and the values (in Vs): both must be done before they are rewritten.
    mbar_wait(bar_pv, ph_pv, abort_flag, p.status_word, DEV_TIMEOUT_ATTEND);
    ph_pv ^= 1;
    tc_fence_after();
    // child codes: row e (local column) = Cc[h, sel_list[(e0+e)/C], (e0+e)%C, :], zero rows as padding
    {
      const __nv_bfloat16* Cch = p.Cc + (size_t)h * M * C * D;
      const int chunks = D / 8;                              // 16-byte chunks per row
      for (int u = tid; u < np16 * chunks; u += kThreads) {
        const int row = u / chunks, ch = u % chunks;
        uint4 val = make_uint4(0, 0, 0, 0);
        if (row < ncols) {
          const int e = e0 + row;
          const int par = sel_list[e / C];
          val = __ldg(reinterpret_cast<const uint4*>(Cch + ((size_t)par * C + (e % C)) * D) + ch);
        }
        unsigned char* sub = CA + (ch >> 3) * (np16 * 128);
        *reinterpret_cast<uint4*>(sub + sw128_offset(row, (ch & 7) * 8)) = val;
      }
    }
    // child values: Vs[k][e] = VcT[bh, par, k, c]; one parent's C children are contiguous per k
    {
      const __nv_bfloat16* Vch = p.VcT + (size_t)bh * M * D * C;
      const int npar = (ncols + C - 1) / C;                  // e0 and ncols are multiples of C
      const int par0 = e0 / C;
      for (int u = tid; u < npar * D; u += kThreads) {
        const int pr = u / D, k = u % D;
        const int par = sel_list[par0 + pr];
        const int col = pr * C;
        unsigned char* dst = Vs + (col >> 6) * (D * 128) + sw128_offset(k, col & 63);
        const __nv_bfloat16* src = Vch + ((size_t)par * D + k) * C;
        if (C == 8) *reinterpret_cast<uint4*>(dst) = __ldg(reinterpret_cast<const uint4*>(src));
        else *reinterpret_cast<uint2*>(dst) = __ldg(reinterpret_cast<const uint2*>(src));
      }
      // zero the padding columns [ncols, np16) of the value tile (they meet zero weights, but 0 * NaN is NaN)
      const int padc = np16 - ncols;
      for (int u = tid; u < padc * D; u += kThreads) {
        const int col = ncols + u / D, k = u % D;
        *reinterpret_cast<__nv_bfloat16*>(Vs + (col >> 6) * (D * 128) + sw128_offset(k, col & 63)) =
            __float2bfloat16_rn(0.f);
      }
      const float* ncb = p.nc + (size_t)bh * M * C;
      for (int e = tid; e < CT; e += kThreads)
        cnt[e] = e < ncols ? ncb[(size_t)sel_list[(e0 + e) / C] * C + ((e0 + e) % C)] : 0.f;
    }
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    if (tid == 0) {
      tc_fence_after();
      const uint32_t idesc = umma_idesc_bf16(kRows, np16);
      const uint32_t qa = smem_u32(Qs), ca = smem_u32(CA);
#pragma unroll
      for (int k = 0; k < D / 16; ++k)
        umma_bf16(tmem_base, umma_desc_sw128(qa + (k / 4) * kRows * 128 + (k % 4) * 32),
                  umma_desc_sw128(ca + (k / 4) * np16 * 128 + (k % 4) * 32), idesc, k > 0);
      umma_commit(bar_s);
    }
    e0 = e1;
  }

  // ---- epilogue: Y = O / z
  const bool o_ok = mbar_wait(bar_pv, ph_pv, abort_flag, p.status_word, DEV_TIMEOUT_ATTEND);
  tc_fence_after();
  if (o_ok) {
    // tcgen05.ld is warp-collective: every lane loads, only rows inside the tensor store.
    const float inv = 1.f / z_run;
    __nv_bfloat16* yrow = p.Y + ((size_t)bh * p.Nq + i0 + r) * D + hf * (D / 2);
    for (int c0 = 0; c0 < D / 2; c0 += 16) {
      float o[16];
      tmem_ld16(t_o + c0, o);
      uint32_t pk[8];
#pragma unroll
      for (int e = 0; e < 16; e += 2) pk[e >> 1] = pack_bf16(o[e] * inv, o[e + 1] * inv);
      if (r < rows_valid) {
        *reinterpret_cast<uint4*>(yrow + c0) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
        *reinterpret_cast<uint4*>(yrow + c0 + 8) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem_base, p.tmem_cols);
}

size_t attend_smem(int D, int CT) {
  const int subA = (CT + 63) / 64;
  const size_t ca = (size_t)max(CT * D * 2, subA * kRows * 128);
  size_t b = 1024 + (size_t)(D / 64) * kRows * 128 + ca + (size_t)subA * D * 128;
  b += sizeof(float) * ((size_t)CT + 256 + 4 * (size_t)CT + 6 * kRows);
  b += sizeof(int) * 256 + sizeof(uint32_t) * 8 + sizeof(uint64_t) * 4 + 2 * sizeof(uint32_t) + 256;
  return b + 64;
}

template <int D>
avq_status launch(const avq_problem& p, const void* Q, const void* Cp, const void* Cc, const float* np_,
                  const float* nc, const void* VpT, const void* VcT, int32_t P, void* Y, int32_t* topp_out,
                  float* importance_out, int32_t* status_word, cudaStream_t st) {
  const uint64_t BH = (uint64_t)p.B * p.H;
  CUtensorMap tmQ, tmCp, tmVpT;
  {
    const uint64_t dims[3] = {(uint64_t)D, (uint64_t)p.Nq, BH};
    const uint32_t box[3] = {64, (uint32_t)kRows, 1};
    avq_status s = make_tmap_bf16(&tmQ, Q, 3, dims, box);
    if (s != AVQ_OK) return s;
  }
  {
    const uint64_t dims[2] = {(uint64_t)D, (uint64_t)p.H * p.M};
    const uint32_t box[2] = {64, (uint32_t)p.M};
    avq_status s = make_tmap_bf16(&tmCp, Cp, 2, dims, box);
    if (s != AVQ_OK) return s;
  }
  {
    const uint64_t dims[2] = {(uint64_t)p.M, BH * D};
    const uint32_t box[2] = {64, (uint32_t)D};
    avq_status s = make_tmap_bf16(&tmVpT, VpT, 2, dims, box);
    if (s != AVQ_OK) return s;
  }
  AttendParams a;
  a.Cc = static_cast<const __nv_bfloat16*>(Cc);
  a.VcT = static_cast<const __nv_bfloat16*>(VcT);
  a.np_ = np_;
  a.nc = nc;
  a.Y = static_cast<__nv_bfloat16*>(Y);
  a.topp_out = topp_out;
  a.importance_out = importance_out;
  a.status_word = status_word;
  a.H = p.H; a.Nq = p.Nq; a.M = p.M; a.C = p.C; a.P = P;
  a.nblk = (p.Nq + kRows - 1) / kRows;
  int CT = 32;
  while (CT < p.M) CT <<= 1;
  a.CT = CT;
  uint32_t cols = 32;
  while ((int)cols < CT + D) cols <<= 1;
  a.tmem_cols = cols;
  a.scale_log2e = p.scale * 1.4426950408889634f;
  const size_t smem = attend_smem(D, CT);
  auto kern = tc_attend_kernel<D>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return AVQ_ERR_CUDA;
  dim3 grid(a.nblk, (unsigned)BH);
  kern<<<grid, kThreads, smem, st>>>(tmQ, tmCp, tmVpT, a);
  return cuda_ok(cudaGetLastError());
}

}  // namespace

avq_status tc_attend(const avq_problem& p, const void* Q, const void* Cp, const void* Cc, const float* np_,
                     const float* nc, const void* VpT, const void* VcT, int32_t P, void* Y, int32_t* topp_out,
                     float* importance_out, int32_t* status_word, cudaStream_t st) {
  return p.d == 64 ? launch<64>(p, Q, Cp, Cc, np_, nc, VpT, VcT, P, Y, topp_out, importance_out, status_word, st)
                   : launch<128>(p, Q, Cp, Cc, np_, nc, VpT, VcT, P, Y, topp_out, importance_out, status_word, st);
}

}  // namespace avq
