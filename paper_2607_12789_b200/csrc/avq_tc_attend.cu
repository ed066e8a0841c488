// Tensor-core attention pass of AVQ-attention (Algorithm 2 in its masked form) for bf16 inputs.
//
// One persistent CTA per SM works through a contiguous run of query tiles (128 rows of one (batch, head)).
// Its 14 warps have fixed roles, and two tiles are in flight: while the parent pass of tile n+1 runs on
// the CUDA cores, the child pass and the output of tile n run beside it and the tensor pipe serves both.
//
//   issuer (1 warp, one lane)  TMA loads (Q tiles, the head's codebook, the value tile) and every
//                              tcgen05.mma: S = Q.Cp^T, O = W.Vp, S_c = Q.Cc_sel^T, O += W_c.Vc, and the
//                              denominators Z = W.1 through a one-column "ones" operand.
//   parent warps (8)           two threads per query row: count-weighted logits t = scale*s + log2 n_j
//                              (empty parents: -inf), row maximum, p = 2^(t - m), z = sum p  (Eq.
//                              "vqflashattention": p_ij = A_ij n_j), importance partial sums of p / z
//                              (Eq. "importance"), bf16 weights written back to TMEM where the value MMA
//                              reads them as its A operand.
//   selector (1 warp)          importance -> top-P by bisection on the bit pattern, ties to the lower index
//                              ("Child spawning"); removes the refined parents from the value tile and from
//                              the ones operand; gathers the selected parents' child codewords and child
//                              value rows (Algorithm 2, child loop).
//   child warps (4)            one thread per row: child logits -> running maximum (rescaling O and Z only
//                              when it moves by more than 2^8), weights to TMEM; then Y = O / Z.
//
// Values enter as per-codeword MEANS (value sum / count, written by the aggregation's finalize kernel) and
// the counts ride in the weights, so numerator and denominator are plain sums over the same bf16 weights:
//   Y_i = sum_j p_ij mean_j / sum_j p_ij,   p_ij = n_j exp(s_ij - m_i)      (same value as Eq. "aggregates" form).
// Every wait is a bounded mbarrier wait; a wait that gives up records a code in the status word, every
// role leaves its loop, and the CTA frees its TMEM and returns.
#include "avq_tc_common.cuh"

namespace avq {
namespace {

using namespace tc;

constexpr int kRows = 128;
constexpr int kParentWarps = 8;
// warps 8..11 are the child warps (a warp reaches the TMEM lane quarter warp % 4)
constexpr int kIssuerWarp = 12;
constexpr int kSelectWarp = 13;
constexpr int kLoaderWarp = 14;
constexpr int kAttendThreads = 15 * 32;
constexpr float kLazyLog2 = 8.f;        // a child maximum within 2^8 of the running one does not move it

struct AttendParams {
  const __nv_bfloat16* Cc;    // [H, M, C, d]
  const __nv_bfloat16* Vcb;   // [B*H, M, C, d]  child value means
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

// Barrier indices (one uint64_t each).
enum Bar : int {
  B_QFULL = 0,      // [2] query tile landed (per Q buffer)
  B_CPFULL = 2,     // parent codebook landed
  B_VPFULL = 3,     // value tile landed
  B_SFULL = 4,      // [2] S = Q.Cp^T done (per tile parity)
  B_WREADY = 6,     // [2] parent weights in TMEM (256 arrivals)
  B_IMP = 8,        // [2] importance partial sums in shared memory (256 arrivals)
  B_VCLR = 10,      // refined parents removed from the value tile / ones operand (32 arrivals)
  B_PVDONE = 11,    // O = W.Vp done
  B_CCREADY = 12,   // [2] child codes and values of a chunk gathered (TMA bytes + one arrival, per slot)
  B_SCFULL = 14,    // child logits done
  B_WCREADY = 15,   // child weights in TMEM (128 arrivals)
  B_CPVDONE = 16,   // [2] O += W_c.Vc done (per slot)
  B_OFREE = 18,     // output accumulators read (128 arrivals)
  B_PAIR = 19,      // [4] the two parent warps of a row quarter exchange (64 arrivals)
  B_PSYNC = 23,     // all parent threads (256 arrivals)
  B_DRAIN = 24,
  B_QFREE = 25,     // [2] every MMA that read this Q buffer has completed (issuer -> loader)
  B_XFREE = 27,     // the value tile's memory may take the next tile's values (issuer -> loader)
  B_COUNT = 28
};

template <int D, int CT, int CHW, bool ALIAS>
struct Smem {
  static constexpr int kQ = kRows * D * 2;                   // one query tile
  static constexpr int kCp = CT * D * 2;
  static constexpr int kX = CT * D * 2;                      // value tile (rows = parents)
  static constexpr int kSlot = 2 * CHW * D * 2;              // child codes + child values of one chunk
  static constexpr int kOnesP = (CT / 64) * 2048;
  static constexpr int kOnesC = (CHW / 64) * 2048;
  static constexpr int oQ = 0;
  static constexpr int oCp = oQ + 2 * kQ;
  static constexpr int oX = oCp + kCp;
  static constexpr int oSlots = ALIAS ? oX : oX + kX;
  static constexpr int oOnesP = ALIAS ? oX + kX : oSlots + 2 * kSlot;
  static constexpr int oOnesC = oOnesP + kOnesP;
  static constexpr int oLb = oOnesC + kOnesC;                // float [2][CT]
  static constexpr int oLbc = oLb + 2 * CT * 4;              // float [2][CHW]
  static constexpr int oWpart = oLbc + 2 * CHW * 4;          // float [2][4][CT]
  static constexpr int oXm = oWpart + 8 * CT * 4;            // float [2][128]
  static constexpr int oXz = oXm + 2 * kRows * 4;            // float [2][128]
  static constexpr int oMrow = oXz + 2 * kRows * 4;          // float [2][128]
  static constexpr int oSel = oMrow + 2 * kRows * 4;         // int [CT]
  static constexpr int oBars = oSel + CT * 4;                // uint64 [B_COUNT]
  static constexpr int oMisc = oBars + B_COUNT * 8;          // tmem slot, abort flag, early exit
  static constexpr int kTotal = oMisc + 16;
  static_assert(!ALIAS || 2 * kSlot <= kX, "child slots must fit the value tile");
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
__device__ __forceinline__ float max3(float a, float b, float c) { return fmaxf(a, fmaxf(b, c)); }

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

// Walks `ncols` (a multiple of 16) TMEM columns of this thread's lane, starting at `t`, in chunks of 32 and
// one closing chunk of 16 if needed (a TMEM round trip costs a few hundred cycles: wide chunks amortise it,
// and the other warps of the scheduler work meanwhile).  The functors get the raw registers and the chunk's
// first column.
template <typename F32, typename F16>
__device__ __forceinline__ void tmem_walk(uint32_t t, int ncols, F32&& f32, F16&& f16) {
  const int nfull = ncols >> 5;
  for (int i = 0; i < nfull; ++i) {
    uint32_t a[32];
    tmem_ld32_issue(t + (uint32_t)(i * 32), a);
    tmem_ld_wait32(a);
    f32(a, i * 32);
  }
  if (ncols & 16) {
    uint32_t tl[16];
    tmem_ld16_issue(t + (uint32_t)(nfull * 32), tl);
    tmem_ld_wait16(tl);
    f16(tl, nfull * 32);
  }
}
__device__ __forceinline__ float u2f(uint32_t u) { return __uint_as_float(u); }
__device__ __forceinline__ uint32_t f2u(float f) { return __float_as_uint(f); }

// D: head dimension; CT: parent tile width (>= M); CHW: child chunk width; SB: TMEM buffers for the parent
// logits (2 where the columns allow it: the next tile's logits are then computed before this tile's value
// MMA); ALIAS: the child chunk slots live inside the value tile's shared memory (used between a tile's
// value MMA and the reload of the value tile for the next tile).
template <int D, int CT, int CHW, int SB, bool ALIAS>
__global__ void __launch_bounds__(kAttendThreads, 1)
tc_attend_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmCp,
                 const __grid_constant__ CUtensorMap tmVpb, const __grid_constant__ CUtensorMap tmCc,
                 const __grid_constant__ CUtensorMap tmVcb, const AttendParams p) {
  // 1024-byte alignment (swizzle atoms) is requested from the launch, not computed from the pointer, so
  // that the compiler keeps every access in the shared address space.
  extern __shared__ __align__(1024) unsigned char smem[];
  using L = Smem<D, CT, CHW, ALIAS>;
  constexpr int kSubD = D / 64;
  constexpr int kLogChunks = (D == 128) ? 4 : 3;         // log2 of the 16-byte chunks per codeword row
  constexpr int kChunks = 1 << kLogChunks;
  constexpr uint32_t kColS = 0, kColSc = SB * CT, kColO = kColSc + CHW, kColZ = kColO + D;
  static_assert(kColZ + 16 <= 512, "TMEM columns");

  unsigned char* Qs = smem + L::oQ;
  unsigned char* Cps = smem + L::oCp;
  unsigned char* Xs = smem + L::oX;
  unsigned char* slots = smem + L::oSlots;
  unsigned char* ones_p = smem + L::oOnesP;
  unsigned char* ones_c = smem + L::oOnesC;
  float* lb = reinterpret_cast<float*>(smem + L::oLb);
  float* lbc = reinterpret_cast<float*>(smem + L::oLbc);
  float* wpart = reinterpret_cast<float*>(smem + L::oWpart);
  float* xm = reinterpret_cast<float*>(smem + L::oXm);
  float* xz = reinterpret_cast<float*>(smem + L::oXz);
  float* m_row = reinterpret_cast<float*>(smem + L::oMrow);
  int* sel_list = reinterpret_cast<int*>(smem + L::oSel);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::oBars);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::oMisc);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::oMisc + 4);
  volatile int* early_exit = reinterpret_cast<volatile int*>(smem + L::oMisc + 8);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int M = p.M, C = p.C, P = p.P, logC = p.logC;
  const int PC = P * C;
  const int nchunks = (PC + CHW - 1) / CHW;
  const float sc = p.scale_log2e;
  const bool need_w = (P > 0 && P < M) || p.importance_out != nullptr;

  // This CTA's run of tiles.
  const int t_begin = (int)(((long long)p.total_tiles * blockIdx.x) / gridDim.x);
  const int t_end = (int)(((long long)p.total_tiles * (blockIdx.x + 1)) / gridDim.x);
  const int T = t_end - t_begin;

#define AVQ_WAIT(bar_index, parity) \
  mbar_wait(&bars[bar_index], (uint32_t)(parity), abort_flag, p.status_word, DEV_TIMEOUT_ATTEND)

  // ------------------------------------------------------------------ set-up
  auto issue_q = [&](int n) {                            // issuer lane only
    const int tile = t_begin + n, tb = tile / p.nblk, ti0 = (tile - tb * p.nblk) * kRows;
    uint64_t* bar = &bars[B_QFULL + (n & 1)];
    mbar_expect_tx(bar, (uint32_t)L::kQ);
#pragma unroll
    for (int s = 0; s < kSubD; ++s)
      tma_load_3d(Qs + (n & 1) * L::kQ + s * kRows * 128, &tmQ, s * 64, ti0, tb, bar);
  };
  auto prefetch_q = [&](int n) {
    const int tile = t_begin + n, tb = tile / p.nblk, ti0 = (tile - tb * p.nblk) * kRows;
#pragma unroll
    for (int s = 0; s < kSubD; ++s) tma_prefetch_l2_3d(&tmQ, s * 64, ti0, tb);
  };
  auto issue_cp = [&](int h) {
    mbar_expect_tx(&bars[B_CPFULL], (uint32_t)(kSubD * M * 128));
#pragma unroll
    for (int s = 0; s < kSubD; ++s) tma_load_2d(Cps + s * M * 128, &tmCp, s * 64, h * M, &bars[B_CPFULL]);
  };
  auto issue_vp = [&](int bh) {
    mbar_expect_tx(&bars[B_VPFULL], (uint32_t)(kSubD * M * 128));
#pragma unroll
    for (int s = 0; s < kSubD; ++s) tma_load_2d(Xs + s * M * 128, &tmVpb, s * 64, bh * M, &bars[B_VPFULL]);
  };

  if (warp == kIssuerWarp && lane == 0) {
    prefetch_tmap(&tmQ);
    prefetch_tmap(&tmCp);
    prefetch_tmap(&tmVpb);
    prefetch_tmap(&tmCc);
    prefetch_tmap(&tmVcb);
    auto init = [&](int i, int n, uint32_t count) {
      for (int u = 0; u < n; ++u) mbar_init(&bars[i + u], count);
    };
    init(B_QFULL, 2, 1);
    init(B_CPFULL, 1, 1);
    init(B_VPFULL, 1, 1);
    init(B_SFULL, 2, 1);
    init(B_WREADY, 2, 32 * kParentWarps);
    init(B_IMP, 2, 32 * kParentWarps);
    init(B_VCLR, 1, 32);
    init(B_PVDONE, 1, 1);
    init(B_CCREADY, 2, 1);
    init(B_SCFULL, 1, 1);
    init(B_WCREADY, 1, 128);
    init(B_CPVDONE, 2, 1);
    init(B_OFREE, 1, 128);
    init(B_PAIR, 4, 64);
    init(B_PSYNC, 1, 32 * kParentWarps);
    init(B_DRAIN, 1, 1);
    init(B_QFREE, 2, 1);
    init(B_XFREE, 1, 1);
    mbar_fence_init();
    *abort_flag = 0;
    *early_exit = 0;
    // Q and the codebook are the caller's: their loads may go out while the kernel that produces the
    // aggregates is still finishing (programmatic dependent launch).
    issue_q(0);
    if (T > 1) issue_q(1);
    if (T > 2) prefetch_q(2);
    issue_cp(((t_begin / p.nblk)) % p.H);
  }
  if (warp == kSelectWarp) {
    tmem_alloc(tmem_slot, p.tmem_cols);
    tmem_relinquish();
  }
  // Constant operands: the ones tiles are [16 rows x 64 k] K-major swizzled sub-tiles, row 0 carries the
  // ones (the other 15 output columns of the denominator MMA stay zero and are never read).
  for (int u = tid; u < (L::kOnesP + L::kOnesC) / 16; u += kAttendThreads)
    reinterpret_cast<uint4*>(ones_p)[u] = make_uint4(0u, 0u, 0u, 0u);
  __syncthreads();
  for (int u = tid; u < (CHW / 64) * 8; u += kAttendThreads)      // row 0 of every child sub-tile: 128 bytes of 1.0
    *reinterpret_cast<uint4*>(ones_c + (u >> 3) * 2048 + (u & 7) * 16) =
        make_uint4(0x3F803F80u, 0x3F803F80u, 0x3F803F80u, 0x3F803F80u);
  fence_proxy_async();
  pdl_wait();          // from here on the aggregates of this call may be read
  if (tid == 0)
    *early_exit = (p.status_word != nullptr && *reinterpret_cast<volatile int32_t*>(p.status_word) != 0);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (*early_exit) {
    // a wait expired in an earlier kernel of this call: let the loads already in flight land, then leave
    if (warp == kIssuerWarp && lane == 0) {
      AVQ_WAIT(B_QFULL, 0);
      if (T > 1) AVQ_WAIT(B_QFULL + 1, 0);
      AVQ_WAIT(B_CPFULL, 0);
    }
  } else if (warp == kIssuerWarp) {
    // ================================================================ issuer
    if (lane == 0) {
      const uint32_t idesc_o = umma_idesc_bf16(kRows, D) | (1u << 16);   // B (value rows) is MN-major
      const uint32_t idesc_z = umma_idesc_bf16(kRows, 16);
      const uint32_t idesc_s = umma_idesc_bf16(kRows, M);
      const uint32_t cps = smem_u32(Cps), xs = smem_u32(Xs), onesp = smem_u32(ones_p), onesc = smem_u32(ones_c);
      uint32_t ph_q[2] = {0, 0}, ph_cp = 0, ph_vclr = 0, ph_pv = 0, ph_cc[2] = {0, 0}, ph_wc = 0,
               ph_cpv[2] = {0, 0}, ph_of = 0;
      int g = 0;                                           // child chunks issued so far (slot = g & 1)
      bool ok = true;
      auto mma_s = [&](int n) {
        const uint32_t qa = smem_u32(Qs + (n & 1) * L::kQ);
        const uint32_t d = tmem_base + kColS + (uint32_t)((n % SB) * CT);
#pragma unroll
        for (int k = 0; k < D / 16; ++k)
          umma_bf16(d, umma_desc_sw128(qa + (k / 4) * kRows * 128 + (k % 4) * 32),
                    umma_desc_sw128(cps + (k / 4) * M * 128 + (k % 4) * 32), idesc_s, k > 0);
        umma_commit(&bars[B_SFULL + (n & 1)]);
      };
      ok = AVQ_WAIT(B_QFULL, ph_q[0]) && AVQ_WAIT(B_CPFULL, ph_cp);
      ph_q[0] ^= 1;
      ph_cp ^= 1;
      if (ok) {
        tc_fence_after();
        mma_s(0);
      }
      for (int n = 0; ok && n < T; ++n) {
        const int tile = t_begin + n, bh = tile / p.nblk;
        const bool has_next = n + 1 < T;
        const int bh_next = (tile + 1) / p.nblk;
        auto next_logits = [&]() -> bool {                 // S(n+1): codebook of its head, its Q tile
          if ((bh_next % p.H) != (bh % p.H)) {
            // the logits MMA of tile n is the last reader of the resident codebook
            if (!AVQ_WAIT(B_SFULL + (n & 1), (n >> 1) & 1)) return false;
            issue_cp(bh_next % p.H);
            if (!AVQ_WAIT(B_CPFULL, ph_cp)) return false;
            ph_cp ^= 1;
          }
          if (!AVQ_WAIT(B_QFULL + ((n + 1) & 1), ph_q[(n + 1) & 1])) return false;
          ph_q[(n + 1) & 1] ^= 1;
          tc_fence_after();
          mma_s(n + 1);
          return true;
        };
        // With two logit buffers the next tile's logits go first: its buffer was released by the value
        // MMA of tile n-1, and every MMA that read the codebook has completed (waited for below).
        if (SB == 2 && has_next && !(ok = next_logits())) break;

        // ---- O = W.Vp, Z = W.1   (parents)
        ok = AVQ_WAIT(B_WREADY + (n & 1), (n >> 1) & 1) && AVQ_WAIT(B_VCLR, ph_vclr);
        ph_vclr ^= 1;
        if (ok && n > 0) {
          ok = AVQ_WAIT(B_OFREE, ph_of);
          ph_of ^= 1;
        }
        if (!ok) break;
        tc_fence_after();
        {
          const uint32_t wbase = tmem_base + kColS + (uint32_t)((n % SB) * CT);
          const int half_steps = M / 32;                   // K steps (16 parents) per column half
          // descriptors advance by adding to their 14-bit address field (units of 16 bytes; shared memory
          // addresses stay below 2^18, so the field cannot carry into the next one)
          const uint64_t dv = umma_desc_sw128_mn(xs, (uint32_t)(M * 128)), dz = umma_desc_sw128(onesp);
#pragma unroll 4
          for (int k = 0; k < M / 16; ++k) {
            const uint32_t a = wbase + (uint32_t)(k < half_steps ? k * 8 : M / 2 + (k - half_steps) * 8);
            umma_bf16_ts(tmem_base + kColO, a, dv + (uint64_t)(k * 128), idesc_o, k > 0);
            umma_bf16_ts(tmem_base + kColZ, a, dz + (uint64_t)((k >> 2) * 128 + (k & 3) * 2), idesc_z, k > 0);
          }
          umma_commit(&bars[B_PVDONE]);
        }
        // The value MMA must be complete before the value tile is reloaded, before the logit buffer it
        // read its weights from is overwritten, and (no children) before the Q buffer is reused.
        ok = AVQ_WAIT(B_PVDONE, ph_pv);
        ph_pv ^= 1;
        if (!ok) break;
        if (!ALIAS && has_next) mbar_arrive(&bars[B_XFREE]);
        if (SB == 1 && has_next && !(ok = next_logits())) break;

        // ---- children of tile n
        const uint32_t qa = smem_u32(Qs + (n & 1) * L::kQ);
        for (int k = 0; ok && k < nchunks; ++k, ++g) {
          const int slot = g & 1;
          const int ncols = min(PC - k * CHW, CHW), np16 = (ncols + 15) & ~15;
          const uint32_t cc = smem_u32(slots + slot * L::kSlot), vc = cc + CHW * D * 2;
          ok = AVQ_WAIT(B_CCREADY + slot, ph_cc[slot]);
          ph_cc[slot] ^= 1;
          if (!ok) break;
          tc_fence_after();
          const uint32_t idesc_c = umma_idesc_bf16(kRows, np16);
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk)
            umma_bf16(tmem_base + kColSc, umma_desc_sw128(qa + (kk / 4) * kRows * 128 + (kk % 4) * 32),
                      umma_desc_sw128(cc + (kk / 4) * np16 * 128 + (kk % 4) * 32), idesc_c, kk > 0);
          umma_commit(&bars[B_SCFULL]);
          ok = AVQ_WAIT(B_WCREADY, ph_wc);
          ph_wc ^= 1;
          if (!ok) break;
          tc_fence_after();
          const uint64_t dvc = umma_desc_sw128_mn(vc, (uint32_t)(np16 * 128)), dzc = umma_desc_sw128(onesc);
#pragma unroll 4
          for (int kk = 0; kk < np16 / 16; ++kk) {
            const uint32_t a = tmem_base + kColSc + (uint32_t)(kk * 8);
            umma_bf16_ts(tmem_base + kColO, a, dvc + (uint64_t)(kk * 128), idesc_o, true);
            umma_bf16_ts(tmem_base + kColZ, a, dzc + (uint64_t)((kk >> 2) * 128 + (kk & 3) * 2), idesc_z, true);
          }
          umma_commit(&bars[B_CPVDONE + slot]);
          // the child weights alias the child logits: the next chunk's logits wait for this MMA
          ok = AVQ_WAIT(B_CPVDONE + slot, ph_cpv[slot]);
          ph_cpv[slot] ^= 1;
        }
        if (!ok) break;
        if (ALIAS && has_next) mbar_arrive(&bars[B_XFREE]);   // the child slots inside the value tile are free again
        if (n + 2 < T) mbar_arrive(&bars[B_QFREE + (n & 1)]);  // every MMA that read Q(n) has completed
      }
      // every MMA issued above has completed on the normal path; after a failed wait give the ones in
      // flight (and the loads) time to finish before the CTA's shared memory and TMEM are released
      umma_commit(&bars[B_DRAIN]);
      mbar_wait(&bars[B_DRAIN], 0, abort_flag, nullptr, 0);
      if (*abort_flag) {
        const unsigned long long t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 100000ull) { }
      }
    }
  } else if (warp == kLoaderWarp) {
    // ================================================================ loader: the Q tiles and the value tiles
    // (a TMA issue costs its thread several hundred cycles, which the MMA issuer cannot spare)
    if (lane == 0) {
      issue_vp(t_begin / p.nblk);
      uint32_t ph_qf[2] = {0, 0}, ph_xf = 0;
      bool ok = true;
      for (int n = 0; ok && n < T; ++n) {
        if (n + 1 < T) {
          ok = AVQ_WAIT(B_XFREE, ph_xf);
          ph_xf ^= 1;
          if (!ok) break;
          issue_vp((t_begin + n + 1) / p.nblk);
        }
        if (n + 2 < T) {
          ok = AVQ_WAIT(B_QFREE + (n & 1), ph_qf[n & 1]);
          ph_qf[n & 1] ^= 1;
          if (!ok) break;
          issue_q(n + 2);
          if (n + 3 < T) prefetch_q(n + 3);
        }
      }
    }
  } else if (warp < kParentWarps) {
    // ================================================================ parent warps
    const int q = warp & 3, hf = warp >> 2, r = q * 32 + lane;
    const int Mh = M >> 1;                                // columns per thread (multiple of 16)
    const uint32_t t_lane = tmem_base + ((uint32_t)(q * 32) << 16);
    uint32_t ph_pair = 0, ph_psync = 0;
    int prev_bh = -1, lsel = 1;
    auto pair_sync = [&]() -> bool {
      mbar_arrive(&bars[B_PAIR + q]);
      const bool ok = AVQ_WAIT(B_PAIR + q, ph_pair);
      ph_pair ^= 1;
      return ok;
    };
    for (int n = 0; n < T; ++n) {
      const int tile = t_begin + n, bh = tile / p.nblk, blk = tile - bh * p.nblk;
      const int rows_valid = min(kRows, p.Nq - blk * kRows);
      if (bh != prev_bh) {
        // log2 of the parents' key counts (-inf for an empty parent and for the padding columns): added to the
        // scaled logit it puts the count into the weight and keeps empty parents out of the maximum
        lsel ^= 1;
        for (int j = tid; j < CT; j += 32 * kParentWarps)
          lb[lsel * CT + j] = j < M ? log2f(p.np_[(size_t)bh * M + j]) : -INFINITY;
        mbar_arrive(&bars[B_PSYNC]);
        const bool ok = AVQ_WAIT(B_PSYNC, ph_psync);
        ph_psync ^= 1;
        if (!ok) break;
        prev_bh = bh;
      }
      const float* lbt = lb + lsel * CT + hf * Mh;
      const uint32_t t_s = t_lane + kColS + (uint32_t)((n % SB) * CT + hf * Mh);
      if (!AVQ_WAIT(B_SFULL + (n & 1), (n >> 1) & 1)) break;
      tc_fence_after();

      // ---- pass 0: t = scale * s + log2 n_j, row maximum; t replaces s in TMEM
      float mx0 = -INFINITY, mx1 = -INFINITY;
      auto pass0 = [&](auto& rg, int c0) __attribute__((always_inline)) {
        constexpr int W = sizeof(rg) / 4;
        const float4* l4 = reinterpret_cast<const float4*>(lbt + c0);
#pragma unroll
        for (int u = 0; u < W / 4; ++u) {
          const float4 l = l4[u];
          const float t0 = fmaf(u2f(rg[4 * u]), sc, l.x), t1 = fmaf(u2f(rg[4 * u + 1]), sc, l.y);
          const float t2 = fmaf(u2f(rg[4 * u + 2]), sc, l.z), t3 = fmaf(u2f(rg[4 * u + 3]), sc, l.w);
          mx0 = max3(mx0, t0, t1);
          mx1 = max3(mx1, t2, t3);
          rg[4 * u] = f2u(t0); rg[4 * u + 1] = f2u(t1); rg[4 * u + 2] = f2u(t2); rg[4 * u + 3] = f2u(t3);
        }
        if constexpr (W == 32) tmem_st32(t_s + (uint32_t)c0, rg);
        else tmem_st16u(t_s + (uint32_t)c0, rg);
      };
      tmem_walk(t_s, Mh, pass0, pass0);
      tmem_st_wait();
      xm[hf * kRows + r] = fmaxf(mx0, mx1);
      if (!pair_sync()) break;
      const float m = fmaxf(xm[r], xm[kRows + r]);         // finite: at least one parent holds a key

      // ---- pass 1: p = 2^(t - m) (exactly 0 for empty parents), z = sum p; p replaces t in TMEM
      float z0 = 0.f, z1 = 0.f;
      auto pass1 = [&](auto& rg, int c0) __attribute__((always_inline)) {
        constexpr int W = sizeof(rg) / 4;
#pragma unroll
        for (int u = 0; u < W; u += 2) {
          const float e0 = ex2(u2f(rg[u]) - m), e1 = ex2(u2f(rg[u + 1]) - m);
          z0 += e0;
          z1 += e1;
          rg[u] = f2u(e0); rg[u + 1] = f2u(e1);
        }
        if constexpr (W == 32) tmem_st32(t_s + (uint32_t)c0, rg);
        else tmem_st16u(t_s + (uint32_t)c0, rg);
      };
      tmem_walk(t_s, Mh, pass1, pass1);
      tmem_st_wait();
      xz[hf * kRows + r] = z0 + z1;
      if (!pair_sync()) break;
      const float z = xz[r] + xz[kRows + r];
      if (hf == 0) m_row[(n & 1) * kRows + r] = m;

      // ---- pass 2, one read of p: bf16 weights, packed two per column over this thread's own (already
      // consumed) columns [hf * Mh, hf * Mh + Mh / 2) - the A operand of the value MMA - and the importance
      // partial sums: column sums of p_ij / z_i over the tile's valid rows (32 per warp; the selector adds
      // the four row quarters)                                       (Eq. "importance")
      const float inv = (r < rows_valid) ? 1.f / z : 0.f;
      float* wp = wpart + ((n & 1) * 4 + q) * CT + hf * Mh;
      auto pass2 = [&](auto& rg, int c0) __attribute__((always_inline)) {
        constexpr int W = sizeof(rg) / 4;
        uint32_t pk[W / 2];
#pragma unroll
        for (int u = 0; u < W / 2; ++u) pk[u] = pack_bf16(u2f(rg[2 * u]), u2f(rg[2 * u + 1]));
        if constexpr (W == 32) tmem_st16u(t_s + (uint32_t)(c0 >> 1), pk);
        else tmem_st8(t_s + (uint32_t)(c0 >> 1), pk);
        if (need_w) {
          float (&v)[W] = reinterpret_cast<float (&)[W]>(rg);   // in place: the registers are dead after this
#pragma unroll
          for (int e = 0; e < W; ++e) v[e] *= inv;
          const float colsum = transpose_reduce<W>(v, lane);
          if constexpr (W == 32) wp[c0 + lane] = colsum;
          else if ((lane & 1) == 0) wp[c0 + (lane >> 1)] = colsum;
        }
      };
      tmem_walk(t_s, Mh, pass2, pass2);
      mbar_arrive(&bars[B_IMP + (n & 1)]);
      tmem_st_wait();
      tc_fence_before();
      mbar_arrive(&bars[B_WREADY + (n & 1)]);
    }
  } else if (warp == kSelectWarp) {
    // ================================================================ selector
    constexpr int NI = CT / 32;                            // parents per lane (j = lane + 32 i)
    uint32_t ph_vp = 0, ph_pv = 0;
    int g = 0;
    bool ok = true;
    for (int n = 0; ok && n < T; ++n) {
      const int tile = t_begin + n, bh = tile / p.nblk, blk = tile - bh * p.nblk, h = bh % p.H;
      if (!AVQ_WAIT(B_IMP + (n & 1), (n >> 1) & 1)) break;
      uint32_t key[NI];
#pragma unroll
      for (int i = 0; i < NI; ++i) {
        const int j = lane + 32 * i;
        float w = 0.f;
        if (need_w && j < M) {
          const float* wp = wpart + (n & 1) * 4 * CT + j;
          w = (wp[0] + wp[CT]) + (wp[2 * CT] + wp[3 * CT]);
          if (p.importance_out) p.importance_out[((size_t)bh * p.nblk + blk) * M + j] = w;
        }
        key[i] = __float_as_uint(w);                       // non-negative floats order like their bit patterns
      }
      // ---- the P largest importances.  T climbs bit by bit to the largest value that at least P keys
      // reach; the search stops early when exactly P keys reach the candidate.  Keys equal to the final T
      // fill the remaining places in ascending index order (ties to the lower index).
      int n_sel = 0;
      if (P > 0) {
        uint32_t thr = 0;
        bool exact = P >= M;                               // P = M: every parent (threshold 0, all keys reach it)
        if (!exact) {
          // every lane forms the same count from ballots (no cross-lane reduction on the dependent path)
          for (int bit = 30; bit >= 0; --bit) {
            const uint32_t cand = thr | (1u << bit);
            int c = 0;
#pragma unroll
            for (int i = 0; i < NI; ++i) c += __popc(__ballot_sync(0xffffffffu, key[i] >= cand));
            if (c >= P) {
              thr = cand;
              if (c == P) { exact = true; break; }
            }
          }
        }
        int need = 0;
        if (!exact) {
          int c = 0;
#pragma unroll
          for (int i = 0; i < NI; ++i) c += __popc(__ballot_sync(0xffffffffu, key[i] > thr));
          need = P - c;                                    // places left for keys equal to the threshold
        }
#pragma unroll
        for (int i = 0; i < NI; ++i) {
          const int j = lane + 32 * i;
          const bool valid = j < M;
          uint32_t m_sel = __ballot_sync(0xffffffffu, valid && (exact ? key[i] >= thr : key[i] > thr));
          if (!exact) {
            uint32_t m_eq = __ballot_sync(0xffffffffu, valid && key[i] == thr);
            const int have = __popc(m_eq);
            if (have > need) {                              // keep the `need` lowest lanes of this group
              const uint32_t pos = need > 0 ? __fns(m_eq, 0, need + 1) : (uint32_t)__ffs(m_eq) - 1u;
              m_eq &= (pos >= 32u) ? 0xffffffffu : ((1u << pos) - 1u);
            }
            need -= __popc(m_eq);
            m_sel |= m_eq;
          }
          if (m_sel & (1u << lane)) {
            const int pos = n_sel + __popc(m_sel & ((1u << lane) - 1u));
            sel_list[pos] = j;
            if (p.topp_out) p.topp_out[((size_t)bh * p.nblk + blk) * P + pos] = j;
          }
          n_sel += __popc(m_sel);
        }
      }
      __syncwarp();

      // ---- the value tile of this tile has landed: remove the refined parents from it and from the ones
      // operand (row 0 of the ones tile is rewritten first: the tile before cleared other entries)
      if (!AVQ_WAIT(B_VPFULL, ph_vp)) break;
      ph_vp ^= 1;
      if (lane * 8 < CT) {
        uint32_t one[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int j = lane * 8 + 2 * u;
          one[u] = (j < M ? 0x3F80u : 0u) | (j + 1 < M ? 0x3F800000u : 0u);
        }
        *reinterpret_cast<uint4*>(ones_p + ((lane * 8) >> 6) * 2048 + ((lane * 8) & 63) * 2) =
            make_uint4(one[0], one[1], one[2], one[3]);
      }
      __syncwarp();
      for (int u = lane; u < n_sel; u += 32) {
        const int j = sel_list[u];
        *reinterpret_cast<unsigned short*>(ones_p + (j >> 6) * 2048 + (j & 63) * 2) = 0;
      }
      for (int u = lane; u < (n_sel << kLogChunks); u += 32) {
        const int row = sel_list[u >> kLogChunks], ch = u & (kChunks - 1);
        *reinterpret_cast<uint4*>(Xs + (ch >> 3) * (M * 128) + sw128_offset(row, (ch & 7) * 8)) =
            make_uint4(0u, 0u, 0u, 0u);
      }
      fence_proxy_async();
      mbar_arrive(&bars[B_VCLR]);

      // ---- child chunks of this tile: codeword rows and value-mean rows of the selected parents' children
      if (nchunks > 0 && ALIAS) {
        // the slots lie inside the value tile: wait until this tile's value MMA has read it
        if (!AVQ_WAIT(B_PVDONE, ph_pv)) break;
        ph_pv ^= 1;
      }
      const __nv_bfloat16* Cch = p.Cc + (size_t)h * M * C * D;
      const __nv_bfloat16* Vch = p.Vcb + (size_t)bh * M * C * D;
      const float* ncb = p.nc + (size_t)bh * M * C;
      for (int k = 0; k < nchunks; ++k, ++g) {
        const int slot = g & 1;
        if (g >= 2) {                                      // the chunk that used this slot before must be consumed
          if (!(ok = AVQ_WAIT(B_CPVDONE + slot, ((g >> 1) - 1) & 1))) break;
        }
        const int e_first = k * CHW;
        const int ncols = min(PC - e_first, CHW), np16 = (ncols + 15) & ~15;
        unsigned char* cc = slots + slot * L::kSlot;
        unsigned char* vc = cc + CHW * D * 2;
        float* lbs = lbc + slot * CHW;
        for (int i = lane; i < CHW; i += 32) {
          float l = -INFINITY;
          if (i < ncols) {
            const int e = e_first + i;
            l = log2f(__ldg(ncb + ((size_t)sel_list[e >> logC] << logC) + (e & (C - 1))));
          }
          lbs[i] = l;
        }
        // Rows of the chunk as K-major / row-per-codeword tiles of np16 rows (sub-tiles of 64 columns).  The
        // C children of a selected parent are C consecutive rows in global memory and in the tile: one TMA box
        // per (parent, sub-tile) for the codes and one for the value means, a lane per parent.  Padding rows
        // (a chunk that ends off a multiple of 16) are zeroed by hand.
        const int npar = ncols >> logC;                    // selected parents in this chunk
        const int p_first = e_first >> logC;
        uint64_t* bar = &bars[B_CCREADY + slot];
        if (np16 > ncols) {
          for (int u = lane; u < ((np16 - ncols) << kLogChunks); u += 32) {
            const int row = ncols + (u >> kLogChunks), ch = u & (kChunks - 1);
            const uint32_t off = (uint32_t)((ch >> 3) * (np16 * 128)) + sw128_offset(row, (ch & 7) * 8);
            *reinterpret_cast<uint4*>(cc + off) = make_uint4(0u, 0u, 0u, 0u);
            *reinterpret_cast<uint4*>(vc + off) = make_uint4(0u, 0u, 0u, 0u);
          }
          fence_proxy_async();
        }
        __syncwarp();
        if (lane == 0) mbar_expect_tx(bar, (uint32_t)(ncols * D * 2 * 2));   // the one arrival + all the bytes
        __syncwarp();
        for (int i = lane; i < npar; i += 32) {
          const int par = sel_list[p_first + i];
          const int row_c = (h * M + par) << logC, row_v = (bh * M + par) << logC;
#pragma unroll
          for (int sd = 0; sd < kSubD; ++sd) {
            const uint32_t off = (uint32_t)(sd * (np16 * 128) + ((i << logC) * 128));
            tma_load_2d(cc + off, &tmCc, sd * 64, row_c, bar);
            tma_load_2d(vc + off, &tmVcb, sd * 64, row_v, bar);
          }
        }
      }
    }
    cp_async_wait_all();
  } else {
    // ================================================================ child warps
    const int q = warp & 3, r = q * 32 + lane;
    const uint32_t t_lane = tmem_base + ((uint32_t)(q * 32) << 16);
    const uint32_t t_sc = t_lane + kColSc, t_o = t_lane + kColO, t_z = t_lane + kColZ;
    uint32_t ph_sc = 0, ph_pv = 0;
    int g = 0;
    bool ok = true;
    for (int n = 0; ok && n < T; ++n) {
      const int tile = t_begin + n, bh = tile / p.nblk, blk = tile - bh * p.nblk;
      const int i0 = blk * kRows;
      const int rows_valid = min(kRows, p.Nq - i0);
      if (nchunks == 0) {
        ok = AVQ_WAIT(B_PVDONE, ph_pv);
        ph_pv ^= 1;
        if (!ok) break;
        tc_fence_after();
      }
      float m_run = 0.f;
      for (int k = 0; k < nchunks; ++k, ++g) {
        const int slot = g & 1;
        const int ncols = min(PC - k * CHW, CHW), np16 = (ncols + 15) & ~15;
        // the logits of this chunk are done; so is every MMA issued before them (the parents' value MMA,
        // the chunk before): O and Z may be rescaled
        ok = AVQ_WAIT(B_SCFULL, ph_sc);
        ph_sc ^= 1;
        if (!ok) break;
        tc_fence_after();
        if (k == 0) m_run = m_row[(n & 1) * kRows + r];
        const float* lbs = lbc + slot * CHW;
        float mx0 = -INFINITY, mx1 = -INFINITY;
        auto cpass0 = [&](auto& rg, int c0) __attribute__((always_inline)) {
          constexpr int W = sizeof(rg) / 4;
          const float4* l4 = reinterpret_cast<const float4*>(lbs + c0);
#pragma unroll
          for (int u = 0; u < W / 4; ++u) {
            const float4 l = l4[u];
            const float t0 = fmaf(u2f(rg[4 * u]), sc, l.x), t1 = fmaf(u2f(rg[4 * u + 1]), sc, l.y);
            const float t2 = fmaf(u2f(rg[4 * u + 2]), sc, l.z), t3 = fmaf(u2f(rg[4 * u + 3]), sc, l.w);
            mx0 = max3(mx0, t0, t1);
            mx1 = max3(mx1, t2, t3);
            rg[4 * u] = f2u(t0); rg[4 * u + 1] = f2u(t1); rg[4 * u + 2] = f2u(t2); rg[4 * u + 3] = f2u(t3);
          }
          if constexpr (W == 32) tmem_st32(t_sc + (uint32_t)c0, rg);
          else tmem_st16u(t_sc + (uint32_t)c0, rg);
        };
        tmem_walk(t_sc, np16, cpass0, cpass0);
        tmem_st_wait();
        // Any reference value works as long as numerator and denominator share it.  The running one is kept
        // unless the children exceed it by more than 2^kLazyLog2 (weights up to that factor above 1 are
        // harmless in fp32 and bf16), which spares most rows the rescaling of O and Z.
        const float m_c = fmaxf(mx0, mx1);
        const float m_new = (m_c > m_run + kLazyLog2) ? m_c : m_run;
        const float alpha = ex2(m_run - m_new);
        if (__any_sync(0xffffffffu, alpha < 1.f)) {
          for (int c0 = 0; c0 < D; c0 += 16) {
            float o[16];
            tmem_ld16(t_o + c0, o);
#pragma unroll
            for (int e = 0; e < 16; ++e) o[e] *= alpha;
            tmem_st16(t_o + c0, o);
          }
          float zz[16];
          tmem_ld16(t_z, zz);
#pragma unroll
          for (int e = 0; e < 16; ++e) zz[e] *= alpha;
          tmem_st16(t_z, zz);
          tmem_st_wait();
        }
        m_run = m_new;
        auto cpass1 = [&](auto& rg, int c0) __attribute__((always_inline)) {
          constexpr int W = sizeof(rg) / 4;
          uint32_t pk[W / 2];
#pragma unroll
          for (int u = 0; u < W / 2; ++u)
            pk[u] = pack_bf16(ex2(u2f(rg[2 * u]) - m_new), ex2(u2f(rg[2 * u + 1]) - m_new));
          if constexpr (W == 32) tmem_st16u(t_sc + (uint32_t)(c0 >> 1), pk);
          else tmem_st8(t_sc + (uint32_t)(c0 >> 1), pk);
        };
        tmem_walk(t_sc, np16, cpass1, cpass1);
        tmem_st_wait();
        tc_fence_before();
        mbar_arrive(&bars[B_WCREADY]);
      }
      if (!ok) break;
      if (nchunks > 0) {
        // last chunk of the tile: its value MMA completes the accumulators
        const int gl = g - 1;
        if (!AVQ_WAIT(B_CPVDONE + (gl & 1), (gl >> 1) & 1)) break;
        tc_fence_after();
      }
      // ---- Y = O / Z, written row by row (a thread owns one query row: D * 2 contiguous bytes)
      float zz[16];
      tmem_ld16(t_z, zz);
      const float inv = 1.f / zz[0];
      uint4* yrow = reinterpret_cast<uint4*>(p.Y + ((size_t)bh * p.Nq + i0 + r) * D);
      auto epi = [&](auto& rg, int c0) __attribute__((always_inline)) {
        constexpr int W = sizeof(rg) / 4;
        uint32_t pk[W / 2];
#pragma unroll
        for (int e = 0; e < W / 2; ++e) pk[e] = pack_bf16(u2f(rg[2 * e]) * inv, u2f(rg[2 * e + 1]) * inv);
        if (r < rows_valid) {
#pragma unroll
          for (int e = 0; e < W / 8; ++e)
            yrow[c0 / 8 + e] = make_uint4(pk[4 * e], pk[4 * e + 1], pk[4 * e + 2], pk[4 * e + 3]);
        }
      };
      tmem_walk(t_o, D, epi, epi);
      tc_fence_before();
      mbar_arrive(&bars[B_OFREE]);
    }
  }
#undef AVQ_WAIT

  tc_fence_before();
  __syncthreads();
  if (warp == kSelectWarp) tmem_dealloc(tmem_base, p.tmem_cols);
}

template <int D, int CT, int CHW, int SB, bool ALIAS>
avq_status launch_variant(const CUtensorMap& tmQ, const CUtensorMap& tmCp, const CUtensorMap& tmVpb,
                          const CUtensorMap& tmCc, const CUtensorMap& tmVcb, AttendParams a, bool chained,
                          cudaStream_t st) {
  auto kern = tc_attend_kernel<D, CT, CHW, SB, ALIAS>;
  constexpr size_t smem = Smem<D, CT, CHW, ALIAS>::kTotal;
  static_assert(smem <= 227 * 1024, "shared memory");
  // The limit is set once per device and instantiation (setting it again is harmless if two threads race).
  static bool configured[64] = {};
  static int sm_count[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return AVQ_ERR_CUDA;
  const bool cached = dev >= 0 && dev < 64;
  if (!cached || !configured[dev]) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return AVQ_ERR_CUDA;
    if (cached) configured[dev] = true;
  }
  int sms = cached ? sm_count[dev] : 0;
  if (sms <= 0) {
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return AVQ_ERR_CUDA;
    if (cached) sm_count[dev] = sms;
  }
  constexpr uint32_t kCols = SB * CT + CHW + D + 16;
  uint32_t cols = 32;
  while (cols < kCols) cols <<= 1;
  a.tmem_cols = cols;
  // One CTA per SM, each with a contiguous run of tiles (a head's codebook then stays resident).
  const int ctas = a.total_tiles < sms ? a.total_tiles : sms;
  // Inside avq_forward (`chained`) the kernel before it in the stream is the aggregate's finalize kernel
  // and Q was complete before the call, so the attention kernel may start as its programmatic dependent.
  // A stand-alone avq_attend is launched plainly: the work before it in the stream may be producing Q.
  return cuda_ok(launch_pdl(kern, dim3((unsigned)ctas), dim3(kAttendThreads), smem, st, chained, tmQ, tmCp, tmVpb, tmCc,
                            tmVcb, a));
}

template <int D>
avq_status launch(const avq_problem& p, const void* Q, const void* Cp, const void* Cc, const float* np_,
                  const float* nc, const void* Vpb, const void* Vcb, int32_t P, void* Y, int32_t* topp_out,
                  float* importance_out, int32_t* status_word, bool chained, cudaStream_t st) {
  const uint64_t BH = (uint64_t)p.B * p.H;
  CUtensorMap tmQ, tmCp, tmVpb, tmCc, tmVcb;
  {
    // child codewords and child value means as [rows = (head, parent, child), d]: a box is one parent's C rows
    const uint32_t box[2] = {64, (uint32_t)p.C};
    const uint64_t dims_c[2] = {(uint64_t)D, (uint64_t)p.H * p.M * p.C};
    const uint64_t dims_v[2] = {(uint64_t)D, BH * p.M * p.C};
    avq_status s = make_tmap_bf16(&tmCc, Cc, 2, dims_c, box);
    if (s != AVQ_OK) return s;
    s = make_tmap_bf16(&tmVcb, Vcb, 2, dims_v, box);
    if (s != AVQ_OK) return s;
  }
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
    const uint64_t dims[2] = {(uint64_t)D, BH * p.M};
    const uint32_t box[2] = {64, (uint32_t)p.M};
    avq_status s = make_tmap_bf16(&tmVpb, Vpb, 2, dims, box);
    if (s != AVQ_OK) return s;
  }
  AttendParams a;
  a.Cc = static_cast<const __nv_bfloat16*>(Cc);
  a.Vcb = static_cast<const __nv_bfloat16*>(Vcb);
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
  a.logC = p.C == 8 ? 3 : 2;
  a.tmem_cols = 0;
  a.scale_log2e = p.scale * 1.4426950408889634f;
  const int CT = p.M <= 64 ? 64 : (p.M <= 128 ? 128 : 256);
  // Variants by TMEM columns (SB*CT + CHW + D + 16 <= 512) and shared memory: two logit buffers up to
  // CT = 128; at d = 128 the child chunks are 64 columns wide, and with CT = 256 their slots share the
  // value tile's memory.
  if constexpr (D == 64) {
    if (CT == 64) return launch_variant<D, 64, 128, 2, false>(tmQ, tmCp, tmVpb, tmCc, tmVcb, a, chained, st);
    if (CT == 128) return launch_variant<D, 128, 128, 2, false>(tmQ, tmCp, tmVpb, tmCc, tmVcb, a, chained, st);
    return launch_variant<D, 256, 128, 1, false>(tmQ, tmCp, tmVpb, tmCc, tmVcb, a, chained, st);
  } else {
    if (CT == 64) return launch_variant<D, 64, 64, 2, false>(tmQ, tmCp, tmVpb, tmCc, tmVcb, a, chained, st);
    if (CT == 128) return launch_variant<D, 128, 64, 2, false>(tmQ, tmCp, tmVpb, tmCc, tmVcb, a, chained, st);
    return launch_variant<D, 256, 64, 1, true>(tmQ, tmCp, tmVpb, tmCc, tmVcb, a, chained, st);
  }
}

}  // namespace

// Parent tiles of up to 128 codewords leave room for several small CTAs per SM (avq_tc_attend_small.cu);
// larger ones take the whole SM and run the warp-specialised kernel above.
avq_status tc_attend(const avq_problem& p, const void* Q, const void* Cp, const void* Cc, const float* np_,
                     const float* nc, const void* Vpb, const void* Vcb, int32_t P, void* Y, int32_t* topp_out,
                     float* importance_out, int32_t* status_word, bool chained, cudaStream_t st) {
  if (p.M <= 128)
    return tc_attend_small(p, Q, Cp, Cc, np_, nc, Vpb, Vcb, P, Y, topp_out, importance_out, status_word, chained, st);
  return p.d == 64 ? launch<64>(p, Q, Cp, Cc, np_, nc, Vpb, Vcb, P, Y, topp_out, importance_out, status_word, chained, st)
                   : launch<128>(p, Q, Cp, Cc, np_, nc, Vpb, Vcb, P, Y, topp_out, importance_out, status_word, chained, st);
}

}  // namespace avq
