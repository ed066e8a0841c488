// Tensor-core attention pass of AVQ-attention (Algorithm 2 in its masked form) for bf16 inputs.
//
// One CTA = one query tile of 128 rows of one (batch, head) at a time; each row is handled by NQ threads
// (column slices).  Values enter as per-codeword MEANS with the key counts multiplied into the weights.
// Flow of a tile:
//   parents   S = Q . Cp^T                 tcgen05.mma, fp32 accumulator in TMEM columns [0, M)
//             read once into registers: row maximum over non-empty parents, exp2, exact
//             denominator z                                         (Eq. "vqflashattention");
//             in the same loop the bf16 weights A_ij n_j -> shared memory (over the dead codebook)
//             importance w_j = n_j sum_i A_ij / z_i from the fp32 weights  (Eq. "importance")
//             top-P by rank, ties to the lower index                ("Child spawning")
//             a refined parent's row of the value tile becomes its stay row (zeros by default) and its
//             rounded weights leave the denominator
//             O = (A n) . mean_p           tcgen05.mma into TMEM columns [CT, CT + d)
//   children  of the selected parents, in chunks of <= CHW columns: gathered codeword rows,
//             S_c = Q . Cc_sel^T, running maximum (non-empty children only), O rescaled in TMEM if a
//             row's maximum moved, bf16 weights, O += A_c . Vbar_c   (Algorithm 2, child loop)
//   Y = O / z, z accumulated from the same bf16-rounded weights as the numerator.
// Empty codewords are excluded from every maximum and contribute nothing (their count and value sum
// are zero; their weight is clamped so that it stays finite) - appendix on numerical stability.
// The gathers of the first child chunk are issued as soon as the selection is known.
#include "avq_tc_common.cuh"

namespace avq {
namespace {

using namespace tc;

constexpr int kRows = 128;

struct AttendParams {
  const __nv_bfloat16* Cc;    // [H, M, C, d]
  const __nv_bfloat16* Vcb;   // [B*H, M, C, d]
  const __nv_bfloat16* Vsb;   // [B*H, M, d]  PARENT_STAYS: value sum of the keys that stay / all keys of the parent
  const float* rho;           // [B*H, M]     PARENT_STAYS: keys that stay / all keys of the parent (else nullptr)
  const float* np_;           // [B*H, M]
  const float* nc;            // [B*H, M, C]
  __nv_bfloat16* Y;           // [B*H, Nq, d]
  int32_t* topp_out;          // optional
  float* importance_out;      // optional
  int32_t* status_word;
  int H, Nq, M, C, P, nblk;
  int total_tiles;            // nblk * B * H
  int logC;                   // log2(C)
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

// The NQ warps that share a quarter of the rows (warp % 4 == q) exchange per-row values through shared
// memory; they synchronise among themselves on named barrier q + 1 instead of stalling the whole CTA.
template <int NQ>
__device__ __forceinline__ void row_sync(int q) {
  asm volatile("bar.sync %0, %1;" ::"r"(q + 1), "r"(32 * NQ) : "memory");
}

// Multiplies 16 fp32 weights by their codewords' key counts, rounds the products to bf16, stores them at
// (row r, columns col0..col0+15) of the K-major swizzled A tile, and returns the sum of the rounded
// products (the denominator is built from exactly what the value MMA multiplies).  KEEP: each product
// enters that sum times keep16[] (the share of its own term a parent keeps once it is refined).
template <bool KEEP>
__device__ __forceinline__ float store_weights16(unsigned char* A, int r, int col0, const float* cnt16,
                                                 const float* keep16, const float (&a)[16]) {
  const float4* n4 = reinterpret_cast<const float4*>(cnt16);
  const float4* k4 = reinterpret_cast<const float4*>(keep16);
  uint32_t pk[8];
  float z0 = 0.f, z1 = 0.f, z2 = 0.f, z3 = 0.f;         // independent partial sums: no 16-deep add chain
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    const float4 n = n4[u];
    const uint32_t p0 = pack_bf16(a[4 * u] * n.x, a[4 * u + 1] * n.y);
    const uint32_t p1 = pack_bf16(a[4 * u + 2] * n.z, a[4 * u + 3] * n.w);
    if constexpr (KEEP) {
      const float4 k = k4[u];
      z0 = fmaf(__uint_as_float(p0 << 16), k.x, z0);
      z1 = fmaf(__uint_as_float(p0 & 0xFFFF0000u), k.y, z1);
      z2 = fmaf(__uint_as_float(p1 << 16), k.z, z2);
      z3 = fmaf(__uint_as_float(p1 & 0xFFFF0000u), k.w, z3);
    } else {
      z0 += __uint_as_float(p0 << 16);
      z1 += __uint_as_float(p0 & 0xFFFF0000u);
      z2 += __uint_as_float(p1 << 16);
      z3 += __uint_as_float(p1 & 0xFFFF0000u);
    }
    pk[2 * u] = p0;
    pk[2 * u + 1] = p1;
  }
  const float z = (z0 + z1) + (z2 + z3);
  unsigned char* sub = A + (col0 >> 6) * (kRows * 128);
  *reinterpret_cast<uint4*>(sub + sw128_offset(r, col0 & 63)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
  *reinterpret_cast<uint4*>(sub + sw128_offset(r, (col0 & 63) + 8)) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
  return z;
}

// NQ = threads per query row: 1, 2 or 4.  Small tiles take NQ = 1 so that four CTAs share an SM and
// overlap each other's load / MMA / softmax phases; the largest take NQ = 4.
// CT = parent tile width (64, 128 or 256, >= M), a compile-time constant so that every shared-memory
// offset folds into the instruction stream instead of occupying a register.
// FUSE = the weight conversion runs inside the exponential loop (chosen by the launcher from CT, P and M).
template <int D, int NQ, int CT, bool FUSE>
__global__ void __launch_bounds__(128 * NQ, 4 / NQ)
tc_attend_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmCp,
                 const __grid_constant__ CUtensorMap tmVpb, const __grid_constant__ CUtensorMap tmY,
                 const AttendParams p) {
  // 1024-byte alignment (swizzle atoms) is requested from the launch, not computed from the pointer, so
  // that the compiler keeps every access in the shared address space.
  extern __shared__ __align__(1024) unsigned char smem[];
  constexpr int kThreads = 128 * NQ;
  constexpr int kScLane = kThreads / 2;                  // lane 0 of a warp in the other half of the CTA
  constexpr int kSubD = D / 64;
  constexpr int kLogD = (D == 128) ? 7 : 6;
  constexpr int kLogChunks = kLogD - 3;                  // 16-byte chunks per codeword row
  constexpr int CHW = CT < 128 ? CT : 128;               // child chunk width
  constexpr int QW = CT / NQ, QWC = CHW / NQ;
  constexpr int subA = CT >> 6;                          // 64-column sub-tiles of an A / value tile
  constexpr int ca_bytes = (CT * D * 2 > subA * kRows * 128) ? CT * D * 2 : subA * kRows * 128;
  const int M = p.M, C = p.C, P = p.P, logC = p.logC;
  unsigned char* Qs = smem;                              // kSubD x [128 x 128 B]
  unsigned char* CA = Qs + kSubD * kRows * 128;          // parent codes, later the bf16 weights
  unsigned char* Vs = CA + ca_bytes;                     // value rows: kSubD x [rows x 128 B], rows = M or a chunk's children
  unsigned char* CC = Vs + subA * D * 128;               // kSubD x [CHW x 128 B] gathered child codes
  float* cnt = reinterpret_cast<float*>(CC + CHW * D * 2);   // [CT] key counts of the parents
  float* bias = cnt + CT;                                // [CT] 0 for non-empty parents, -inf for empty
  float* cntk = bias + CT;                               // [CT] share of its own term a parent keeps: 1, or once refined 0 / its stay share
  float* cntc = cntk + CT;                               // [CHW] key counts of the child chunk
  float* biasc = cntc + CHW;                             // [CHW]
  float* w = biasc + CHW;                                // [CT] importance
  float* wpart = w + CT;                                 // [4][CT]
  float* xm = wpart + 4 * CT;                            // [NQ][128] exchange between the threads of a row
  float* xz = xm + NQ * kRows;                           // [NQ][128]
  float* xz2 = xz + NQ * kRows;                          // [NQ][128]
  float* ncs = xz2 + NQ * kRows;                         // [M * C] key counts of every child of this (b, h)
  int* sel_list = reinterpret_cast<int*>(ncs + p.M * p.C);    // [CT]
  uint32_t* wmask = reinterpret_cast<uint32_t*>(sel_list + CT);    // [16]
  uint64_t* bars = reinterpret_cast<uint64_t*>(wmask + 18);        // [5]  (wmask[16] is a scratch word)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 5);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int q = warp & 3, cq = warp >> 2, r = q * 32 + lane;
  const int colbase = cq * QW;
  uint64_t* bar_q = &bars[0];                            // query tile landed
  uint64_t* bar_ld1 = &bars[1];                          // parent value rows landed
  uint64_t* bar_s = &bars[2];
  uint64_t* bar_pv = &bars[3];
  uint64_t* bar_cp = &bars[4];                           // parent codebook landed
  // A CTA works through the tiles blockIdx.x, blockIdx.x + gridDim.x, ... (the grid is one wave of CTAs).
  // The next tile's Q is loaded as soon as this tile's last logits are done, its codebook as soon as this
  // tile's last value MMA is done, so the set-up, the loads and the first MMA of a tile hide behind the tail
  // of the tile before.  The output is staged where the next tile's first loads do not go: in the child-code
  // buffer when that is as large as a Q tile (CT >= 128), else across the value tile and the child-code
  // buffer, which are adjacent and together as large (the next tile's value rows then load a little later).
  constexpr bool kChain = true;
  constexpr bool kStageInCC = CT >= 128;
  // weight conversion inside the exponential loop (see there): pays where few CTAs share the SM and P is small
  // against M; measured slower for the 64-column tiles (four CTAs per SM already fill each other's gaps) and
  // for P near M (the P look-ups per row cost more than the overlap gains)
  constexpr bool fuse = FUSE;
  auto issue_q = [&](int t) {                            // thread 0 only
    const int tb = t / p.nblk, ti0 = (t - tb * p.nblk) * kRows;
    mbar_expect_tx(bar_q, (uint32_t)(kSubD * kRows * 128));
#pragma unroll
    for (int s = 0; s < kSubD; ++s) tma_load_3d(Qs + s * kRows * 128, &tmQ, s * 64, ti0, tb, bar_q);
  };
  auto issue_cp = [&](int t) {
    const int th = (t / p.nblk) % p.H;
    mbar_expect_tx(bar_cp, (uint32_t)(kSubD * M * 128));
#pragma unroll
    for (int s = 0; s < kSubD; ++s) tma_load_2d(CA + s * M * 128, &tmCp, s * 64, th * M, bar_cp);
  };
  auto issue_vp = [&](int t) {
    const int tb = t / p.nblk;
    mbar_expect_tx(bar_ld1, (uint32_t)(kSubD * M * 128));
#pragma unroll
    for (int s = 0; s < kSubD; ++s) tma_load_2d(Vs + s * M * 128, &tmVpb, s * 64, tb * M, bar_ld1);
  };

  auto issue_s = [&](uint32_t tmem_d, uint32_t parity) {  // one thread: S = Q . Cp^T once both tiles have landed
    const bool q_ok = mbar_wait(bar_q, parity, abort_flag, p.status_word, DEV_TIMEOUT_ATTEND);
    const bool c_ok = mbar_wait(bar_cp, parity, abort_flag, p.status_word, DEV_TIMEOUT_ATTEND);
    if (q_ok && c_ok) {
      tc_fence_after();
      const uint32_t idesc = umma_idesc_bf16(kRows, M);
      const uint32_t qa = smem_u32(Qs), ca = smem_u32(CA);
#pragma unroll
      for (int k = 0; k < D / 16; ++k)
        umma_bf16(tmem_d, umma_desc_sw128(qa + (k / 4) * kRows * 128 + (k % 4) * 32),
                  umma_desc_sw128(ca + (k / 4) * M * 128 + (k % 4) * 32), idesc, k > 0);
    }
    umma_commit(bar_s);
  };

  __shared__ int early_exit;

  // ---- Part 1 touches only the caller's Q and Cp, so it may run while the kernel that produces the
  // aggregates is still finishing (programmatic dependent launch): barriers, TMEM, the Q / Cp loads and
  // S = Q . Cp^T.
  if (tid == 0) {
    prefetch_tmap(&tmQ);
    prefetch_tmap(&tmCp);
    prefetch_tmap(&tmVpb);
    mbar_init(bar_q, 1);
    mbar_init(bar_cp, 1);
    mbar_init(bar_ld1, 1);
    mbar_init(bar_s, 1);
    mbar_init(bar_pv, 1);
    mbar_fence_init();
    *abort_flag = 0;
    issue_q(blockIdx.x);
    issue_cp(blockIdx.x);
  }
  // TMEM is allocated before the dependency wait.  tcgen05.alloc blocks until the columns are free and the
  // wait returns only when the kernels before this one have finished; neither can hold the other up: the
  // columns an earlier kernel's CTAs own are released when those CTAs end, which needs nothing from this
  // kernel, and CTAs of this kernel release theirs on every path (including the early exit below).
  if (warp == 1) {                                   // not the warp whose lane 0 is busy issuing the loads
    tmem_alloc(tmem_slot, p.tmem_cols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16);
  const uint32_t t_s = t_row + (uint32_t)colbase;
  const uint32_t t_sc = t_row + (uint32_t)(cq * QWC);
  const uint32_t t_o = t_row + (uint32_t)(CT + cq * (D / NQ));
  const uint32_t idesc_o = umma_idesc_bf16(kRows, D) | (1u << 16);   // B (the value rows) is MN-major
  const float sc = p.scale_log2e;
  uint32_t ph_s = 0, ph_pv = 0, ph_in = 0;               // ph_in: parity of the three load barriers (once per tile)
  const int PC = P * C;
  const int my_cols = min(max(M - colbase, 0), QW);      // multiple of 16 (M % 32 == 0, QW % 16 == 0)
  bool first = true;
  bool store_pending = false;                            // thread 0: a TMA store may still be reading CC
  for (int tile = blockIdx.x; tile < p.total_tiles; tile += gridDim.x) {
  const int bh = tile / p.nblk, blk = tile - bh * p.nblk, h = bh % p.H;
  const int i0 = blk * kRows;
  const int rows_valid = min(kRows, p.Nq - i0);
  const int next_tile = tile + gridDim.x;
  const bool has_next = kChain && next_tile < p.total_tiles;
  // Key counts of this (b, h): one parent count and one 16-byte group of child counts per thread.  Their loads
  // are started before thread 0 turns to the MMA issue so that its warp is not a load latency behind the
  // others at the next barrier (first tile: only after the dependency wait below - the kernel before this
  // one writes them, so they are loaded with statements the compiler cannot move ahead of that wait).
  static_assert(CT <= kThreads && 2 * CT <= 4 * kThreads, "one count load per thread");
  float n_reg = 0.f;
  float4 nc_reg = make_float4(0.f, 0.f, 0.f, 0.f);
  auto load_counts = [&]() {
    if (tid < M) n_reg = ld_after_wait(p.np_ + (size_t)bh * M + tid);
    if (PC > 0 && tid < ((M * C) >> 2))
      nc_reg = ld_after_wait(reinterpret_cast<const float4*>(p.nc + (size_t)bh * M * C) + tid);
  };
  if (!first) load_counts();
  if (tid == 0) {
    issue_s(tmem_base, ph_in);
    if (!kStageInCC && !first) {
      // the value tile was the staging area of the tile before: reload it once that store has read it
      tma_store_wait_read();
      store_pending = false;
      issue_vp(tile);
    }
  }

  // ---- Part 2 reads what the earlier kernels of this call wrote: status word, counts, value sums.
  if (first) {
    pdl_wait();
    load_counts();                                     // in flight before thread 0 blocks on the status word
    if (tid == 0) {
      issue_vp(tile);
      // a wait that expired in an earlier CTA or kernel of this call: do not start more work
      early_exit = (p.status_word != nullptr && *reinterpret_cast<volatile int32_t*>(p.status_word) != 0);
    }
  }
  if (tid < CT) {
    cnt[tid] = n_reg;
    bias[tid] = n_reg > 0.f ? 0.f : -INFINITY;
    cntk[tid] = 1.f;
  }
  // every child's key count: the gathers below pick theirs from shared memory instead of waiting for a
  // dependent global load once the selection is known
  if (PC > 0 && tid < ((M * C) >> 2)) reinterpret_cast<float4*>(ncs)[tid] = nc_reg;
  __syncthreads();
  if (first && early_exit) {
    // let the MMA and the load already in flight finish, then leave cleanly
    mbar_wait(bar_s, 0, abort_flag, nullptr, 0);
    mbar_wait(bar_ld1, 0, abort_flag, nullptr, 0);
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, p.tmem_cols);
    return;
  }
  first = false;

  // ---- parents: row maximum over non-empty codewords (empty ones carry a -inf bias)
  mbar_wait(bar_s, ph_s, abort_flag, p.status_word, DEV_TIMEOUT_ATTEND);
  ph_s ^= 1;
  tc_fence_after();
  if (tid == 0 && has_next && PC == 0) issue_q(next_tile);   // no child logits will read this Q tile
  // This thread's QW (<= 64) parent logits are read from TMEM once and stay in registers through the
  // maximum, the exponentials, the importance sums and the conversion to bf16.
  float a[QW];
  float mx = -INFINITY, mx2 = -INFINITY;
#pragma unroll
  for (int c0 = 0; c0 < QW; c0 += 16) {
    if (c0 < my_cols) {                                  // warp-uniform
      float s[16];
      tmem_ld16(t_s + c0, s);
      const float4* b4 = reinterpret_cast<const float4*>(bias + colbase + c0);
      // the biased logit stays in the register: an empty parent's -inf becomes a weight of exactly 0
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const float4 b = b4[u];
        a[c0 + 4 * u] = s[4 * u] + b.x;
        a[c0 + 4 * u + 1] = s[4 * u + 1] + b.y;
        a[c0 + 4 * u + 2] = s[4 * u + 2] + b.z;
        a[c0 + 4 * u + 3] = s[4 * u + 3] + b.w;
        mx = fmaxf(mx, fmaxf(a[c0 + 4 * u], a[c0 + 4 * u + 1]));
        mx2 = fmaxf(mx2, fmaxf(a[c0 + 4 * u + 2], a[c0 + 4 * u + 3]));
      }
    } else {
#pragma unroll
      for (int e = 0; e < 16; ++e) a[c0 + e] = 0.f;
    }
  }
  float m_run = fmaxf(mx, mx2) * sc;                    // scale > 0: the maximum commutes with it
  if (NQ > 1) {
    xm[cq * kRows + r] = m_run;
    row_sync<NQ>(q);
#pragma unroll
    for (int u = 0; u < NQ; ++u) m_run = fmaxf(m_run, xm[u * kRows + r]);
  }
  // m_run is finite: at least one parent holds a key.

  // ---- fp32 weights; exact denominator of the parent pass.  Empty parents carry a logit of -inf, hence
  // a weight of exactly zero; every other logit is at most the maximum (up to one rounding).
  float zfull = 0.f, zall = 0.f;                          // zall: sum of this thread's bf16-rounded weights x counts
  {
    float zf0 = 0.f, zf1 = 0.f, zf2 = 0.f, zf3 = 0.f;
    const float negm = -m_run;
#pragma unroll
    for (int c0 = 0; c0 < QW; c0 += 16) {
      if (c0 < my_cols) {
        const float4* n4 = reinterpret_cast<const float4*>(cnt + colbase + c0);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const float4 n = n4[u];
          a[c0 + 4 * u] = ex2(fmaf(a[c0 + 4 * u], sc, negm));
          a[c0 + 4 * u + 1] = ex2(fmaf(a[c0 + 4 * u + 1], sc, negm));
          a[c0 + 4 * u + 2] = ex2(fmaf(a[c0 + 4 * u + 2], sc, negm));
          a[c0 + 4 * u + 3] = ex2(fmaf(a[c0 + 4 * u + 3], sc, negm));
          zf0 = fmaf(a[c0 + 4 * u], n.x, zf0);
          zf1 = fmaf(a[c0 + 4 * u + 1], n.y, zf1);
          zf2 = fmaf(a[c0 + 4 * u + 2], n.z, zf2);
          zf3 = fmaf(a[c0 + 4 * u + 3], n.w, zf3);
        }
        // Large tiles with few parents to refine: the bf16 weights go to shared memory (over the dead
        // codebook) right here - the exponentials keep the XU pipe busy and the conversion (ALU pipe, stores)
        // fills the issue slots they leave empty.  The selection is not known yet; what it removes is taken
        // out of the denominator afterwards (P look-ups per row).
        if constexpr (fuse) {
          float am[16];
#pragma unroll
          for (int e = 0; e < 16; ++e) am[e] = a[c0 + e];
          zall += store_weights16<false>(CA, r, colbase + c0, cnt + colbase + c0, nullptr, am);
        }
      }
    }
    zfull = (zf0 + zf1) + (zf2 + zf3);
    if (NQ > 1) {
      xz[cq * kRows + r] = zfull;
      row_sync<NQ>(q);
      zfull = 0.f;
#pragma unroll
      for (int u = 0; u < NQ; ++u) zfull += xz[u * kRows + r];
    }
  }
  // The importances are needed only to choose which parents to refine: with P = 0 (nothing refined) or
  // P >= M (everything refined) the choice is fixed and the pass is skipped unless the caller wants them.
  const bool need_w = (P > 0 && P < M) || p.importance_out != nullptr;
  if (need_w) {
    const float inv = (r < rows_valid) ? 1.f / zfull : 0.f;
    // ---- importance: column sums of A_ij / z_i over the 128 rows (32 per warp, then 4 warps)
    if constexpr ((QW & 31) == 0) {
#pragma unroll
      for (int c0 = 0; c0 < QW; c0 += 32) {
        if (c0 < my_cols) {
          float v[32];
#pragma unroll
          for (int e = 0; e < 32; ++e) v[e] = a[c0 + e] * inv;
          const float colsum = transpose_reduce<32>(v, lane);
          wpart[q * CT + colbase + c0 + lane] = colsum;
        }
      }
    } else {
#pragma unroll
      for (int c0 = 0; c0 < QW; c0 += 16) {
        if (c0 < my_cols) {
          float v[16];
#pragma unroll
          for (int e = 0; e < 16; ++e) v[e] = a[c0 + e] * inv;
          const float colsum = transpose_reduce<16>(v, lane);
          if ((lane & 1) == 0) wpart[q * CT + colbase + c0 + (lane >> 1)] = colsum;
        }
      }
    }
  }
  if (need_w) {
    __syncthreads();
    if (tid < M) {
      const float wj = cnt[tid] * ((wpart[tid] + wpart[CT + tid]) + (wpart[2 * CT + tid] + wpart[3 * CT + tid]));
      w[tid] = wj;
      if (p.importance_out) p.importance_out[((size_t)bh * p.nblk + blk) * M + tid] = wj;
    }
    __syncthreads();
  }

  // ---- top-P by rank.  Non-negative floats order like their bit patterns, so the comparisons run on
  // integers.  gt_j = number of strictly larger importances; parent j is selected if gt_j < P, except
  // that when a group of EQUAL importances straddles the boundary only its lowest indices are kept.
  // kT threads share one parent's scan.
  {
    const int kT = (kThreads >= 2 * M) ? 2 : 1;          // threads that share one parent's scan
    const int j = (kT == 2) ? (tid >> 1) : tid, part = (kT == 2) ? (tid & 1) : 0;
    const uint32_t* keys = reinterpret_cast<const uint32_t*>(w);
    int* gstar = reinterpret_cast<int*>(&wmask[16]);
    bool mine = false;
    if (P >= M) {
      mine = (j < M) && (part == 0);
    } else if (P > 0) {
      int gt = 0;
      if (j < M) {
        const uint32_t kj = keys[j];
        const int span = M / kT, kb = part * span;
        int g0 = 0, g1 = 0, g2 = 0, g3 = 0;              // four independent counters: no serial add chain
        // 16 keys per trip (span is a multiple of 16): the four 16-byte loads are in flight together
        // instead of one load -> compare -> add chain per trip
        for (int k = kb; k < kb + span; k += 16) {
          uint4 kq[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) kq[u] = *reinterpret_cast<const uint4*>(keys + k + 4 * u);
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            asm("{\n\t.reg .pred p0, p1, p2, p3;\n\t"
                "setp.gt.u32 p0, %4, %8;\n\tsetp.gt.u32 p1, %5, %8;\n\t"
                "setp.gt.u32 p2, %6, %8;\n\tsetp.gt.u32 p3, %7, %8;\n\t"
                "@p0 add.s32 %0, %0, 1;\n\t@p1 add.s32 %1, %1, 1;\n\t"
                "@p2 add.s32 %2, %2, 1;\n\t@p3 add.s32 %3, %3, 1;\n\t}"
                : "+r"(g0), "+r"(g1), "+r"(g2), "+r"(g3)
                : "r"(kq[u].x), "r"(kq[u].y), "r"(kq[u].z), "r"(kq[u].w), "r"(kj));
          }
        }
        gt = (g0 + g1) + (g2 + g3);
      }
      if (kT == 2) gt += __shfl_xor_sync(0xffffffffu, gt, 1);
      const bool cand = (j < M) && (part == 0) && (gt < P);
      if (tid == 0) *gstar = 0;
      const int ncand = __syncthreads_count(cand);
      mine = cand;
      if (ncand > P) {                                   // uniform: equal importances straddle the boundary
        if (cand) atomicMax(gstar, gt);                  // the tied group has the largest gt among candidates
        __syncthreads();
        const int g = *gstar;
        const bool tied = cand && gt == g;
        const uint32_t beq = __ballot_sync(0xffffffffu, tied);
        if (lane == 0) wmask[warp] = beq;
        __syncthreads();
        int epos = __popc(beq & ((1u << lane) - 1u));
        for (int u = 0; u < warp; ++u) epos += __popc(wmask[u]);
        mine = cand && (gt < g || epos < P - g);
        __syncthreads();
      }
    }
    const uint32_t bal = __ballot_sync(0xffffffffu, mine);
    if (lane == 0) wmask[warp] = bal;
    __syncthreads();
    if (mine) {
      int pos = __popc(bal & ((1u << lane) - 1u));
      for (int u = 0; u < warp; ++u) pos += __popc(wmask[u]);
      sel_list[pos] = j;
      cntk[j] = p.rho ? __ldg(p.rho + (size_t)bh * M + j) : 0.f;   // the share of its keys that stays with it
      if (p.topp_out) p.topp_out[((size_t)bh * p.nblk + blk) * P + pos] = j;
    }
  }
  // the output tile of the tile before must have left the child-code buffer before it is refilled (its
  // store was issued a whole parent pass ago, so this does not wait in practice)
  if (tid == 0 && store_pending) {
    tma_store_wait_read();
    store_pending = false;
  }
  __syncthreads();

  // ---- first child chunk: start the asynchronous gather of its codeword rows now; it lands while the
  // weight conversion below runs
  const __nv_bfloat16* Cch = p.Cc + (size_t)h * M * C * D;
  int ncols = min(PC, CHW);
  int np16 = (ncols + 15) & ~15;
  // Rows of a chunk, gathered into a K-major / row-per-codeword tile of np16 rows (kSubD sub-tiles of 64
  // columns): local row e = src[sel_list[(e_first+e)/C] * C + (e_first+e)%C, :]; padding rows are zero.
  // A thread keeps its 16-byte chunk column and walks down the rows (kThreads is a multiple of the chunks
  // per row).
  auto gather_rows = [&](unsigned char* tile, const __nv_bfloat16* src, int e_first) {
    constexpr int kRowsPerPass = kThreads >> kLogChunks;   // a multiple of 8: a thread's swizzle phase is fixed
    constexpr int kPasses = (CHW + kRowsPerPass - 1) / kRowsPerPass;
    const int ch = tid & ((1 << kLogChunks) - 1), row0 = tid >> kLogChunks;
    const uint32_t dst0 = smem_u32(tile) + (uint32_t)((ch >> 3) * (np16 * 128)) + sw128_offset(row0, (ch & 7) * 8);
    const __nv_bfloat16* src_col = src + ch * 8;
    int sel[kPasses];
#pragma unroll
    for (int it = 0; it < kPasses; ++it) {                 // the list look-ups first, all in flight together
      const int e = e_first + row0 + it * kRowsPerPass;
      sel[it] = (row0 + it * kRowsPerPass < ncols) ? sel_list[e >> logC] : 0;
    }
#pragma unroll
    for (int it = 0; it < kPasses; ++it) {
      const int row = row0 + it * kRowsPerPass;
      const uint32_t dst = dst0 + (uint32_t)(it * kRowsPerPass * 128);
      if (row < ncols) {
        const int e = e_first + row;
        const uint32_t off = (uint32_t)(((sel[it] << logC) + (e & (C - 1))) << kLogD);   // elements: < 2^31
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src_col + off) : "memory");
      } else if (row < np16) {
        asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(dst), "r"(0) : "memory");
      }
    }
  };
  auto gather_codes = [&](int e_first) {
    float n_child = 0.f;
    if (tid < ncols) {                                   // CHW <= 128 <= kThreads
      const int e = e_first + tid;
      n_child = ncs[(sel_list[e >> logC] << logC) + (e & (C - 1))];
    }
    gather_rows(CC, Cch, e_first);
    if (tid < CHW) {
      cntc[tid] = n_child;
      biasc[tid] = n_child > 0.f ? 0.f : -INFINITY;
    }
  };
  gather_codes(0);

  // ---- bf16 weights into shared memory (over the dead codebook) + their denominator.  A refined parent
  // is removed from the numerator by clearing its row of the value tile (d / 8 16-byte stores) and from the
  // denominator by its zeroed count, so the weights themselves need no mask.
  mbar_wait(bar_ld1, ph_in, abort_flag, p.status_word, DEV_TIMEOUT_ATTEND);   // value sums have landed
  for (int u = tid; u < (min(P, M) << kLogChunks); u += kThreads) {
    const int row = sel_list[u >> kLogChunks], ch = u & ((1 << kLogChunks) - 1);
    // a refined parent keeps only the keys that stayed with it (Algorithm 1's masked scatter): its value row
    // becomes the stay residual, Vbar_stay = Vbar_p - sum_c Vbar_c, in the same per-n_p units (all zero under
    // the default rule, where every key moves to a child)
    uint4 stay = make_uint4(0, 0, 0, 0);
    if (p.Vsb) stay = __ldg(reinterpret_cast<const uint4*>(p.Vsb + ((size_t)bh * M + row) * D) + ch);
    *reinterpret_cast<uint4*>(Vs + (ch >> 3) * (M * 128) + sw128_offset(row, (ch & 7) * 8)) = stay;
  }
  if constexpr (!fuse) {
    // bf16 weights into shared memory (over the dead codebook) + their denominator; a refined parent's
    // rounded weight enters the denominator with the share of its own term that it keeps (cntk)
    float zloc = 0.f;
#pragma unroll
    for (int c0 = 0; c0 < QW; c0 += 16) {
      if (c0 < my_cols) {
        float am[16];
#pragma unroll
        for (int e = 0; e < 16; ++e) am[e] = a[c0 + e];
        zloc += store_weights16<true>(CA, r, colbase + c0, cnt + colbase + c0, cntk + colbase + c0, am);
      }
    }
    xz2[cq * kRows + r] = zloc;
  } else {
    // denominator of the parent pass from the rounded weights, less what the refined parents no longer carry
    // (all of it under the default rule, the share of the keys that moved to children under PARENT_STAYS);
    // the row's NQ threads split the P look-ups
    float fix = 0.f;
    const int nsel = min(P, M);
    for (int u0 = cq; u0 < nsel; u0 += 4 * NQ) {         // four look-ups in flight per trip
      int jj[4];
#pragma unroll
      for (int t = 0; t < 4; ++t) jj[t] = sel_list[min(u0 + t * NQ, nsel - 1)];
      float wv[4], kv[4];
#pragma unroll
      for (int t = 0; t < 4; ++t) {
        const uint16_t hv =
            *reinterpret_cast<const uint16_t*>(CA + (jj[t] >> 6) * (kRows * 128) + sw128_offset(r, jj[t] & 63));
        wv[t] = __uint_as_float((uint32_t)hv << 16);
        kv[t] = (u0 + t * NQ < nsel) ? 1.f - cntk[jj[t]] : 0.f;
      }
#pragma unroll
      for (int t = 0; t < 4; ++t) fix = fmaf(wv[t], kv[t], fix);
    }
    xz2[cq * kRows + r] = zall - fix;
  }
  cp_async_wait_all();
  fence_proxy_async();
  tc_fence_before();
  __syncthreads();
  float z_run = 0.f;
#pragma unroll
  for (int u = 0; u < NQ; ++u) z_run += xz2[u * kRows + r];

  // ---- O = A . Vbar_p, and right behind it the first child chunk's logits
  if (tid == 0) {
    tc_fence_after();
    if (mbar_wait(bar_ld1, ph_in, abort_flag, p.status_word, DEV_TIMEOUT_ATTEND)) {
      const uint32_t aa = smem_u32(CA), va = smem_u32(Vs);
      for (int k = 0; k < M / 16; ++k)
        umma_bf16(tmem_base + CT, umma_desc_sw128(aa + (k / 4) * kRows * 128 + (k % 4) * 32),
                  umma_desc_sw128_mn(va + k * 2048, (uint32_t)(M * 128)), idesc_o, k > 0);
    }
    umma_commit(bar_pv);
  }
  // The child-score MMAs are issued by a lane of another warp: an issuing lane stalls at the tensor pipe's
  // pace, and two short stalls side by side delay the next CTA-wide barrier less than one long one.
  if (tid == kScLane && PC > 0) {
    tc_fence_after();
    const uint32_t idesc = umma_idesc_bf16(kRows, np16);
    const uint32_t qa = smem_u32(Qs), ca = smem_u32(CC);
#pragma unroll
    for (int k = 0; k < D / 16; ++k)
      umma_bf16(tmem_base, umma_desc_sw128(qa + (k / 4) * kRows * 128 + (k % 4) * 32),
                umma_desc_sw128(ca + (k / 4) * np16 * 128 + (k % 4) * 32), idesc, k > 0);
    umma_commit(bar_s);
  }

  // ---- child chunks
  const __nv_bfloat16* Vch = p.Vcb + (size_t)bh * M * C * D;
  for (int e0 = 0; e0 < PC; e0 += CHW) {
    // The previous second MMA must have released A and Vs before they are rewritten.
    mbar_wait(bar_pv, ph_pv, abort_flag, p.status_word, DEV_TIMEOUT_ATTEND);
    ph_pv ^= 1;
    tc_fence_after();
    // value rows of this chunk (the same gather as for its codeword rows).  Asynchronous copies: they land
    // while the chunk's logits are turned into weights.  Padding rows are zero: they meet finite weights.
    gather_rows(Vs, Vch, e0);

    // ---- child logits: running maximum over non-empty children
    mbar_wait(bar_s, ph_s, abort_flag, p.status_word, DEV_TIMEOUT_ATTEND);
    ph_s ^= 1;
    tc_fence_after();
    if (tid == 0 && has_next && e0 + CHW >= PC) issue_q(next_tile);   // the last logits are done: Q is dead
    const int my_c = min(max(np16 - cq * QWC, 0), QWC);
    // With 32 child columns per thread the chunk's logits are read from TMEM once and stay in registers with
    // their bias (an empty child's -inf becomes a weight of exactly 0); with 64 per thread they are read twice
    // (the register copy measured slower there: N=16384 M=64 P=16 attend 43.4 -> 46.5 us; c3 179.7 -> 176.2).
    constexpr bool kChildRegs = QWC <= 32;
    float cl[kChildRegs ? QWC : 1];
    float mxc = -INFINITY;
    if constexpr (kChildRegs) {
#pragma unroll
      for (int c0 = 0; c0 < QWC; c0 += 16) {
        if (c0 < my_c) {                                 // warp-uniform
          float s[16];
          tmem_ld16(t_sc + c0, s);
          const float4* b4 = reinterpret_cast<const float4*>(biasc + cq * QWC + c0);
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const float4 b = b4[u];
            cl[c0 + 4 * u] = s[4 * u] + b.x;
            cl[c0 + 4 * u + 1] = s[4 * u + 1] + b.y;
            cl[c0 + 4 * u + 2] = s[4 * u + 2] + b.z;
            cl[c0 + 4 * u + 3] = s[4 * u + 3] + b.w;
            mxc = fmaxf(mxc, fmaxf(cl[c0 + 4 * u], cl[c0 + 4 * u + 1]));
            mxc = fmaxf(mxc, fmaxf(cl[c0 + 4 * u + 2], cl[c0 + 4 * u + 3]));
          }
        } else {
#pragma unroll
          for (int e = 0; e < 16; ++e) cl[c0 + e] = -INFINITY;
        }
      }
    } else {
      for (int c0 = 0; c0 < my_c; c0 += 16) {
        float s[16];
        tmem_ld16(t_sc + c0, s);
        const float4* b4 = reinterpret_cast<const float4*>(biasc + cq * QWC + c0);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const float4 b = b4[u];
          mxc = fmaxf(mxc, fmaxf(s[4 * u] + b.x, s[4 * u + 1] + b.y));
          mxc = fmaxf(mxc, fmaxf(s[4 * u + 2] + b.z, s[4 * u + 3] + b.w));
        }
      }
    }
    float m_c = mxc * sc;
    if (NQ > 1) {
      xm[cq * kRows + r] = m_c;
      row_sync<NQ>(q);
#pragma unroll
      for (int u = 0; u < NQ; ++u) m_c = fmaxf(m_c, xm[u * kRows + r]);
    }
    // Any reference value works as long as numerator and denominator share it.  The running one is
    // kept unless the children exceed it by more than 2^kLazyLog2 (weights up to that factor above 1 are
    // harmless in fp32 and bf16), which spares most rows the rescaling of O and z.
    constexpr float kLazyLog2 = 8.f;
    const float m_new = (m_c > m_run + kLazyLog2) ? m_c : m_run;
    const float negm = -m_new;
    // ---- rescale what has been accumulated if this row's maximum moved
    const float alpha = ex2(m_run + negm);
    if (__any_sync(0xffffffffu, alpha < 1.f)) {
      for (int c0 = 0; c0 < D / NQ; c0 += 16) {
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
    // ---- bf16 weights of the children over the parents' (consumed) weights
    {
      float zloc = 0.f;
      if constexpr (kChildRegs) {
#pragma unroll
        for (int c0 = 0; c0 < QWC; c0 += 16) {
          if (c0 < my_c) {
            float a[16];
#pragma unroll
            for (int e = 0; e < 16; ++e) a[e] = ex2(fmaf(cl[c0 + e], sc, negm));
            zloc += store_weights16<false>(CA, r, cq * QWC + c0, cntc + cq * QWC + c0, nullptr, a);
          }
        }
      } else {
        for (int c0 = 0; c0 < my_c; c0 += 16) {
          float a[16];
          tmem_ld16(t_sc + c0, a);
#pragma unroll
          for (int e = 0; e < 16; ++e) a[e] = ex2(fminf(fmaf(a[e], sc, negm), kLazyLog2));   // clamp: empty children
          zloc += store_weights16<false>(CA, r, cq * QWC + c0, cntc + cq * QWC + c0, nullptr, a);
        }
      }
      xz2[cq * kRows + r] = zloc;
    }
    cp_async_wait_all();
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
#pragma unroll
    for (int u = 0; u < NQ; ++u) z_run += xz2[u * kRows + r];

    // ---- O += A_c . Vbar_c; then stage the next chunk's codes (the logits MMA of this chunk is done)
    const int e_next = e0 + CHW;
    if (tid == 0) {
      tc_fence_after();
      const uint32_t aa = smem_u32(CA), va = smem_u32(Vs);
      for (int k = 0; k < np16 / 16; ++k)
        umma_bf16(tmem_base + CT, umma_desc_sw128(aa + (k / 4) * kRows * 128 + (k % 4) * 32),
                  umma_desc_sw128_mn(va + k * 2048, (uint32_t)(np16 * 128)), idesc_o, true);
      umma_commit(bar_pv);
    }
    if (e_next < PC) {
      ncols = min(PC - e_next, CHW);
      np16 = (ncols + 15) & ~15;
      gather_codes(e_next);
      cp_async_wait_all();
      fence_proxy_async();
      tc_fence_before();
      __syncthreads();
      if (tid == kScLane) {
        tc_fence_after();
        const uint32_t idesc = umma_idesc_bf16(kRows, np16);
        const uint32_t qa = smem_u32(Qs), ca = smem_u32(CC);
#pragma unroll
        for (int k = 0; k < D / 16; ++k)
          umma_bf16(tmem_base, umma_desc_sw128(qa + (k / 4) * kRows * 128 + (k % 4) * 32),
                    umma_desc_sw128(ca + (k / 4) * np16 * 128 + (k % 4) * 32), idesc, k > 0);
        umma_commit(bar_s);
      }
    }
  }

  // ---- epilogue: Y = O / z
  const bool o_ok = mbar_wait(bar_pv, ph_pv, abort_flag, p.status_word, DEV_TIMEOUT_ATTEND);
  ph_pv ^= 1;
  tc_fence_after();
  // the last value MMA has released the weight tile and the value tile: the next tile's codebook and
  // parent value rows load while this tile's output is written
  if (tid == 0 && has_next) {
    issue_cp(next_tile);
    if (kStageInCC) issue_vp(next_tile);
  }
  // The output tile is staged in shared memory in the layout of the Q load and written with TMA tile
  // stores; rows past Nq are clipped by the tensor map.  Staging area: see the top of the tile loop.
  unsigned char* stage = kStageInCC ? CC : Vs;
  if (o_ok) {
    const float inv = 1.f / z_run;
    for (int c0 = 0; c0 < D / NQ; c0 += 16) {
      float o[16];
      tmem_ld16(t_o + c0, o);
      uint32_t pk[8];
#pragma unroll
      for (int e = 0; e < 16; e += 2) pk[e >> 1] = pack_bf16(o[e] * inv, o[e + 1] * inv);
      const int col0 = cq * (D / NQ) + c0;
      unsigned char* sub = stage + (col0 >> 6) * (kRows * 128);
      *reinterpret_cast<uint4*>(sub + sw128_offset(r, col0 & 63)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
      *reinterpret_cast<uint4*>(sub + sw128_offset(r, (col0 & 63) + 8)) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
    }
    fence_proxy_async();
  }
  tc_fence_before();
  __syncthreads();
  if (tid == 0 && o_ok) {
#pragma unroll
    for (int s2 = 0; s2 < kSubD; ++s2) tma_store_3d(&tmY, stage + s2 * kRows * 128, s2 * 64, i0, bh);
    tma_store_commit();
    if (has_next) store_pending = true;                // waited for before the next tile refills CC
    else tma_store_wait_read();                        // before the CTA may leave
  }
  ph_in ^= 1;
  }   // tiles
  if (warp == 1) tmem_dealloc(tmem_base, p.tmem_cols);
}

size_t attend_smem(int D, int CT, int CHW, int NQ, int MC) {
  const int subA = CT / 64;
  const size_t ca = (size_t)max(CT * D * 2, subA * kRows * 128);
  size_t b = (size_t)(D / 64) * kRows * 128 + ca + (size_t)subA * D * 128 + (size_t)CHW * D * 2;
  b += sizeof(float) * (3 * (size_t)CT + 2 * (size_t)CHW + (size_t)CT + 4 * (size_t)CT + 3 * (size_t)NQ * kRows);
  b += sizeof(int) * (size_t)CT + sizeof(uint32_t) * 18 + sizeof(uint64_t) * 5 + 2 * sizeof(uint32_t);
  return b + 64 + sizeof(float) * (size_t)MC;
}

template <int D, int NQ, int CT, bool FUSE>
avq_status launch_nq_f(const CUtensorMap& tmQ, const CUtensorMap& tmCp, const CUtensorMap& tmVpb,
                     const CUtensorMap& tmY, const AttendParams& a, unsigned BH, size_t smem, bool chained,
                     cudaStream_t st) {
  auto kern = tc_attend_kernel<D, NQ, CT, FUSE>;
  // The limit is set once per device and instantiation (setting it again is harmless if two threads race).
  static size_t configured[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return AVQ_ERR_CUDA;
  if (dev < 0 || dev >= 64 || smem > configured[dev]) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return AVQ_ERR_CUDA;
    if (dev >= 0 && dev < 64) configured[dev] = smem;
  }
  // Grid: one wave of CTAs (4 / NQ per SM), each taking every gridDim.x-th tile.
  static int sm_count[64] = {};
  int sms = (dev >= 0 && dev < 64) ? sm_count[dev] : 0;
  if (sms <= 0) {
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return AVQ_ERR_CUDA;
    if (dev >= 0 && dev < 64) sm_count[dev] = sms;
  }
  int ctas = a.total_tiles;
  if (ctas > (4 / NQ) * sms) ctas = (4 / NQ) * sms;
  const dim3 grid((unsigned)ctas);
  // Inside avq_forward (`chained`) the kernel before it in the stream is the aggregate's finalize kernel
  // and Q was complete before the call, so the attention kernel may start as its programmatic dependent.
  // A stand-alone avq_attend is launched plainly: the work before it in the stream may be producing Q.
  return cuda_ok(launch_pdl(kern, grid, dim3(128 * NQ), smem, st, chained, tmQ, tmCp, tmVpb, tmY, a));
}

template <int D, int NQ, int CT>
avq_status launch_nq(const CUtensorMap& tmQ, const CUtensorMap& tmCp, const CUtensorMap& tmVpb,
                     const CUtensorMap& tmY, const AttendParams& a, unsigned BH, size_t smem, bool chained,
                     cudaStream_t st) {
  // conversion inside the exponential loop: measured to pay for the larger tiles when P is small against M
  // (c2 45.1 -> 43.3 us, c3 188 -> 184 us) and to cost for 64-column tiles (N=16384 M=64 P=16: 43 -> 47 us)
  // and for P near M (N=65536 M=128 P=128: 615 -> 649 us)
  if constexpr (CT >= 128) {
    if (4 * a.P <= a.M) return launch_nq_f<D, NQ, CT, true>(tmQ, tmCp, tmVpb, tmY, a, BH, smem, chained, st);
  }
  return launch_nq_f<D, NQ, CT, false>(tmQ, tmCp, tmVpb, tmY, a, BH, smem, chained, st);
}

template <int D>
avq_status launch(const avq_problem& p, const void* Q, const void* Cp, const void* Cc, const float* np_,
                  const float* nc, const void* Vpb, const void* Vcb, const void* Vsb, const float* rho, int32_t P, void* Y, int32_t* topp_out,
                  float* importance_out, int32_t* status_word, bool chained, cudaStream_t st) {
  const uint64_t BH = (uint64_t)p.B * p.H;
  CUtensorMap tmQ, tmCp, tmVpb, tmY;
  {
    const uint64_t dims[3] = {(uint64_t)D, (uint64_t)p.Nq, BH};
    const uint32_t box[3] = {64, (uint32_t)kRows, 1};
    avq_status s = make_tmap_bf16(&tmQ, Q, 3, dims, box);
    if (s != AVQ_OK) return s;
    s = make_tmap_bf16(&tmY, Y, 3, dims, box);
    if (s != AVQ_OK) return s;
  }
  {
    const uint64_t dims[2] = {(uint64_t)D, (uint64_t)p.H * p.M};
    const uint32_t box[2] = {64, (uint32_t)p.M};
    avq_status s = make_tmap_bf16(&tmCp, Cp, 2, dims, box);
    if (s != AVQ_OK) return s;
  }
  {
    const uint64_t dims[2] = {(uint64_t)D, BH * p.M};
    const uint32_t box[2] = {64, (uint32_t)p.M};
    avq_status s = make_tmap_bf16(&tmVpb, Vpb, 2, dims, box);
    if (s != AVQ_OK) return s;
  }
  AttendParams a;
  a.Cc = static_cast<const __nv_bfloat16*>(Cc);
  a.Vcb = static_cast<const __nv_bfloat16*>(Vcb);
  a.Vsb = static_cast<const __nv_bfloat16*>(Vsb);
  a.rho = rho;
  a.np_ = np_;
  a.nc = nc;
  a.Y = static_cast<__nv_bfloat16*>(Y);
  a.topp_out = topp_out;
  a.importance_out = importance_out;
  a.status_word = status_word;
  a.H = p.H; a.Nq = p.Nq; a.M = p.M; a.C = p.C; a.P = P;
  a.nblk = (p.Nq + kRows - 1) / kRows;
  if ((uint64_t)a.nblk * BH > 0x7fffffffull) return AVQ_ERR_UNSUPPORTED;
  a.total_tiles = (int)(a.nblk * BH);
  const int CT = p.M <= 64 ? 64 : (p.M <= 128 ? 128 : 256);
  const int CHW = CT < 128 ? CT : 128;
  a.logC = p.C == 8 ? 3 : 2;
  uint32_t cols = 32;
  while ((int)cols < CT + D) cols <<= 1;
  a.tmem_cols = cols;
  a.scale_log2e = p.scale * 1.4426950408889634f;
  const int NQ = (D == 64) ? (CT == 64 ? 1 : (CT == 128 ? 2 : 4)) : (CT == 64 ? 2 : 4);
  const size_t smem = attend_smem(D, CT, CHW, NQ, p.M * p.C);
  // Threads per query row follow from how many CTAs can share an SM (TMEM columns, shared memory):
  // four small CTAs of 128 threads, two of 256, or one of 512.
  const unsigned bh = (unsigned)BH;
  if (D == 64) {
    if (CT == 64) return launch_nq<D, 1, 64>(tmQ, tmCp, tmVpb, tmY, a, bh, smem, chained, st);
    if (CT == 128) return launch_nq<D, 2, 128>(tmQ, tmCp, tmVpb, tmY, a, bh, smem, chained, st);
    return launch_nq<D, 4, 256>(tmQ, tmCp, tmVpb, tmY, a, bh, smem, chained, st);
  }
  if (CT == 64) return launch_nq<D, 2, 64>(tmQ, tmCp, tmVpb, tmY, a, bh, smem, chained, st);
  if (CT == 128) return launch_nq<D, 4, 128>(tmQ, tmCp, tmVpb, tmY, a, bh, smem, chained, st);
  return launch_nq<D, 4, 256>(tmQ, tmCp, tmVpb, tmY, a, bh, smem, chained, st);
}

}  // namespace

avq_status tc_attend(const avq_problem& p, const void* Q, const void* Cp, const void* Cc, const float* np_,
                     const float* nc, const void* Vpb, const void* Vcb, const void* Vsb, const float* rho, int32_t P, void* Y, int32_t* topp_out,
                     float* importance_out, int32_t* status_word, bool chained, cudaStream_t st) {
  return p.d == 64 ? launch<64>(p, Q, Cp, Cc, np_, nc, Vpb, Vcb, Vsb, rho, P, Y, topp_out, importance_out, status_word, chained, st)
                   : launch<128>(p, Q, Cp, Cc, np_, nc, Vpb, Vcb, Vsb, rho, P, Y, topp_out, importance_out, status_word, chained, st);
}

}  // namespace avq
