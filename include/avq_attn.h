/*
 * avq_attn.h - C ABI of the AVQ-attention forward library for NVIDIA B200 (sm_100a).
 *
 * AVQ-attention ("Adaptive Vector-Quantized Attention") replaces the N keys of an
 * attention layer by M parent codewords, measures per query tile how much attention
 * mass each parent receives, and refines the P most important parents with their C
 * pre-learned child codewords.  This library implements the inference forward pass:
 *
 *   avq_assign     nearest parent, then nearest child of that parent, per key
 *                  (Sec. "Vector-Quantized Attention", a(K_j) = argmin_a ||C_a - K_j||^2;
 *                   Algorithm 1, parent-assignment and child-assignment steps)
 *   avq_aggregate  per-codeword value sums and key counts
 *                  (Eq. "aggregates"; Algorithm 1, the two scatter steps)
 *   avq_forward    assign + aggregate + the attention pass: parent logits and softmax
 *                  weights (Eq. "vqflashattention"), per-parent importance
 *                  (Eq. "importance"), top-P selection and child refinement
 *                  ("Child spawning", "Child attention", Algorithm 2), with the
 *                  non-empty-only running maximum of the appendix "Numerical Stability
 *                  of Online Softmax in VQ-Attention".
 *
 * Conventions
 *   - Every pointer is a DEVICE pointer unless the argument is documented as host.
 *     The caller owns every buffer.  The library allocates no device memory and keeps
 *     no state that can change a result (it caches encoded TMA descriptors and one-time
 *     kernel attributes); calls on different streams with different workspaces may overlap.
 *   - All tensors are dense, row-major, last index fastest:
 *       Q  [B, H, Nq, d]     K, V [B, H, Nk, d]     Y [B, H, Nq, d]
 *       Cp [H, M, d]         parent codebook, one per head, shared over the batch
 *       Cc [H, M, C, d]      child codebook; children of parent m are rows Cc[h, m, 0..C-1]
 *     (the paper's single [H, M(1+C), d] buffer is the case Cc = Cp + M*d per head, with
 *     child (m, c) at flat index M + m*C + c).
 *   - dtype is the element type of Q, K, V, Cp, Cc and Y: float32 or bfloat16.
 *     Indices are int32, aggregates and importances float32 (counts are exact integers).
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *     Calls are asynchronous with respect to the host unless stated otherwise.
 *   - The logit scale is explicit (the paper drops the customary 1/sqrt(d) "for clarity").
 *   - Ties: the lowest index wins in both argmins and in the top-P selection.
 *   - Query tiles ("Block_N" of Algorithm 2) are contiguous runs of block_q queries inside
 *     one (batch, head); the last one may be shorter.  block_q changes the result, since
 *     each tile selects its own P parents.
 *
 * Errors: every entry point validates its arguments on the host and returns a status
 * without launching anything when they are unusable.  Shapes outside the supported
 * envelope give AVQ_ERR_UNSUPPORTED; there is no silent fallback.  Device-side waits on
 * barriers (loads, tensor-core completion) are bounded; a kernel that gives up records a
 * code in the workspace header which avq_check() reports as AVQ_ERR_DEVICE_TIMEOUT.  Two
 * hardware waits carry no limit of their own and end when the work ahead of them on the
 * GPU ends: the allocation of tensor memory by a thread block and the dependency wait
 * between the kernels of one call.
 */
#ifndef AVQ_ATTN_H_
#define AVQ_ATTN_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define AVQ_API __attribute__((visibility("default")))
#else
#define AVQ_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  AVQ_OK = 0,
  AVQ_ERR_NULL = 1,           /* a required pointer is NULL                               */
  AVQ_ERR_SHAPE = 2,          /* a size is non-positive or inconsistent (e.g. P > M)      */
  AVQ_ERR_UNSUPPORTED = 3,    /* valid problem, but outside what the kernels handle       */
  AVQ_ERR_ALIGN = 4,          /* a pointer is not 16-byte aligned                          */
  AVQ_ERR_WORKSPACE = 5,      /* workspace missing or smaller than avq_workspace_bytes()  */
  AVQ_ERR_CUDA = 6,           /* a CUDA runtime / driver call failed                      */
  AVQ_ERR_DEVICE_TIMEOUT = 7, /* a bounded device-side wait expired (see avq_check)       */
  AVQ_ERR_INDEX = 8           /* a kernel met a parent/child index out of range (avq_check) */
} avq_status;

typedef enum { AVQ_F32 = 0, AVQ_BF16 = 1 } avq_dtype;

enum {
  /* Algorithm 1's masked scatter: a key moves to its nearest child only if that child is
   * strictly closer than the parent; otherwise it stays with the parent (child index -1).
   * Default (flag clear): every key is represented by the nearest child of its parent.
   * A refined parent then keeps the keys that stayed with it (value sum Vbar_p - sum_c Vbar_c). */
  AVQ_FLAG_PARENT_STAYS = 1u,
  /* Use the plain CUDA-core (FFMA) kernels even where a tensor-core kernel exists.
   * float32 problems always use them.  Meant for cross-checks and for shapes outside the
   * tensor-core envelope. */
  AVQ_FLAG_SIMT = 2u,
  /* Algorithm 2's child pass as printed: the parent's logit is recovered as the mean of its children's
   * logits (Eq. "parent_recovery") and the children add the differences Delta A = A_c - A_p to accumulators
   * that keep every parent's full term (Eq. "correcting_attention").  Equal to the default (masked) form only
   * for codebooks that satisfy parent = mean(children); CUDA-core kernels only (with bfloat16 inputs set
   * AVQ_FLAG_SIMT too: rounding the codebook to bfloat16 already breaks the constraint by an ulp). */
  AVQ_FLAG_CORRECTING = 4u
};

typedef struct {
  int32_t B, H;        /* batch, heads                                                   */
  int32_t Nq, Nk;      /* queries and keys per (batch, head)                             */
  int32_t d;           /* head dimension                                                 */
  int32_t M, C;        /* parents per head, children per parent                          */
  int32_t dtype;       /* avq_dtype of Q, K, V, Cp, Cc, Y                                */
  float scale;         /* logits are scale * <q, c>                                      */
  uint32_t flags;      /* AVQ_FLAG_*                                                     */
} avq_problem;

/* Supported envelope.
 *   CUDA-core kernels (float32, or AVQ_FLAG_SIMT): d % 4 == 0, 4 <= d <= 256; 1 <= M <= 1024;
 *     1 <= C <= 16; 0 <= P <= M; 1 <= block_q <= 256; M + P*C <= 8192; and the attention kernel's
 *     shared memory, 4*block_q*(d + 2) + 20*M + 32*(M + P*C) + 4*max(P, 1) bytes, at most 200 KiB
 *     (e.g. d = 256 with block_q = 256 does not fit; d = 128 with block_q = 256 does).
 *   Tensor-core kernels (bfloat16, no flags): d in {64, 128}; M a multiple of 32, 32..256;
 *     C in {4, 8}; 0 <= P <= M; block_q = 128; scale > 0.
 */

/* Bytes of device scratch avq_forward needs for this problem (0 if the problem is invalid).
 * The workspace holds a 256-byte header (device status word), the key indices and the
 * aggregates between the three stages.  Host function, no CUDA calls. */
AVQ_API size_t avq_workspace_bytes(const avq_problem* prob, int32_t P, int32_t block_q);

/* Stage 1.  parent_idx[b,h,j] = argmin_m ||Cp[h,m] - K[b,h,j]||^2  (int32, [B,H,Nk]);
 * child_idx[b,h,j] = argmin_c ||Cc[h,parent,c] - K[b,h,j]||^2 in [0,C), or -1 when
 * AVQ_FLAG_PARENT_STAYS is set and no child is strictly closer than the parent.
 * Distances that are closer than the kernels' arithmetic can separate are re-evaluated
 * in float64 in the direct form sum_k (K_k - C_k)^2, so the result equals the exact argmin
 * with lowest-index tie-break.  Uses Nk, d, M, C, B, H, dtype, flags of `prob`. */
AVQ_API avq_status avq_assign(const avq_problem* prob, const void* K, const void* Cp, const void* Cc,
                      int32_t* parent_idx, int32_t* child_idx, void* stream);

/* Stage 2.  Vp[b,h,m,:] = sum of V rows whose parent is m, np_[b,h,m] their number;
 * Vc[b,h,m,c,:], nc[b,h,m,c] the same over keys with (parent, child) = (m, c); keys with
 * child index -1 enter the parent sums only.  All four outputs are float32 and are
 * overwritten (the call zeroes them first).  Summation order is not fixed, so the last
 * bits of the sums may differ from run to run; counts are exact.
 * Indices are the caller's here: a key whose parent index is outside [0, M) or whose child
 * index is outside [-1, C) is left out of every sum (no out-of-range access is made). */
AVQ_API avq_status avq_aggregate(const avq_problem* prob, const void* V, const int32_t* parent_idx,
                         const int32_t* child_idx, float* Vp, float* np_, float* Vc, float* nc,
                         void* stream);

/* The whole forward: stages 1 and 2 into the workspace, then per query tile
 *   s = scale * Q_I Cp^T;  m_i = max over non-empty parents;  A = exp(s - m), 0 for empty;
 *   z_i = sum_j A_ij n_j;  w_j = sum_{i in I} A_ij n_j / z_i          (importance)
 *   S = the P parents with largest w (ties -> lower index)
 *   Y_I = [ sum_{p not in S} A_p Vp_p + sum_{p in S} ( A_p Vstay_p + sum_c A_pc Vc_pc ) ]
 *         / [ the same with counts ],   Vstay = Vp - sum_c Vc (zero unless PARENT_STAYS),
 * evaluated with one running maximum over all non-empty columns.
 *   Y              [B,H,Nq,d], dtype of Q
 *   topp_out       optional (may be NULL): int32 [B,H,ceil(Nq/block_q),P], ascending indices
 *   importance_out optional (may be NULL): float32 [B,H,ceil(Nq/block_q),M]
 *   workspace      device scratch of at least avq_workspace_bytes() bytes, 256-byte aligned;
 *                  its contents are overwritten; after the call it holds, at the offsets
 *                  avq_workspace_layout() reports, the indices and aggregates of this call.
 */
AVQ_API avq_status avq_forward(const avq_problem* prob, const void* Q, const void* K, const void* V,
                       const void* Cp, const void* Cc, int32_t P, int32_t block_q, void* Y,
                       int32_t* topp_out, float* importance_out, void* workspace,
                       size_t workspace_bytes, void* stream);

/* avq_forward over query tiles that follow a caller-supplied token order (Sec. "Vector Quantization for
 * (A)VQ-Attention": tokens of an image are reordered along a space-filling curve so that a query tile holds
 * neighbouring tokens; building the curve is the caller's business).  perm: int32 [Nq], a permutation of
 * 0..Nq-1 shared by every (batch, head): tile t holds the queries perm[t*block_q .. (t+1)*block_q).  Only
 * the grouping of the queries changes the result (sums and counts over keys do not depend on their order),
 * so K and V are used as given.  Y, topp_out and importance_out as in avq_forward, with Y rows in the
 * caller's ORIGINAL order and tile t of the optional outputs referring to the permuted tile t.
 * Needs avq_workspace_bytes_permuted() bytes (the forward's workspace plus two [B,H,Nq,d] buffers).  An
 * entry of perm outside [0, Nq) is skipped and reported by avq_check() as AVQ_ERR_INDEX. */
AVQ_API size_t avq_workspace_bytes_permuted(const avq_problem* prob, int32_t P, int32_t block_q);
AVQ_API avq_status avq_forward_permuted(const avq_problem* prob, const void* Q, const void* K, const void* V,
                                const void* Cp, const void* Cc, int32_t P, int32_t block_q,
                                const int32_t* perm, void* Y, int32_t* topp_out, float* importance_out,
                                void* workspace, size_t workspace_bytes, void* stream);

/* avq_forward with the parents visited in tiles of tile_m codewords, for codebooks too large to score in one
 * tile (appendix "Computing Importance with Tiled Codewords").  The codewords of tile J get their importance
 * from the part of the softmax denominator seen up to that tile, extrapolated by key counts:
 *     Ztilde_i(J) = Nk / N_seen(J) * sum_{t<=J} sum_{j in t} A_ij n_j          (Eq. "aproxdenom")
 *     w_j = sum_i A_ij n_j / Ztilde_i(J),  j in J                              (Eq. "codewordimportance")
 * and the P parents with the largest w are refined.  The output is the exact refined attention for that
 * selection; only the selection (and importance_out) differs from avq_forward.  tile_m: a multiple of 32;
 * tile_m >= M reproduces avq_forward.  Runs the CUDA-core kernels for either dtype (M up to 1024); the
 * workspace is that of avq_forward for the same problem with AVQ_FLAG_SIMT set. */
AVQ_API avq_status avq_forward_tiled(const avq_problem* prob, const void* Q, const void* K, const void* V,
                             const void* Cp, const void* Cc, int32_t P, int32_t block_q, int32_t tile_m,
                             void* Y, int32_t* topp_out, float* importance_out, void* workspace,
                             size_t workspace_bytes, void* stream);

/* One training-time update of the codebooks from a batch of keys (appendix "Codeword Clustering During
 * Training").  The keys are assigned under the current codebooks (as in avq_assign, honouring
 * AVQ_FLAG_PARENT_STAYS); every parent and child adds the sum and the number of its keys, over the whole batch,
 * to its exponential-moving-average statistics,  S <- decay*S + (1-decay)*sum,  N <- decay*N + (1-decay)*count;
 * a parent moves to Sp/Np; the children of a parent move to
 *     Cc' = Mc - delta / (Nc * sigma),   Mc = Sc/Nc,  delta = sum_c Mc - C*Cp',  sigma = sum_c 1/Nc
 * (Eq. "child_constraint_solve"), the mass-weighted least-squares projection onto  mean_c Cc' = Cp'.
 * A code whose EMA mass is below 1e-6 keeps its previous position as its mean and enters the projection
 * with that floor as its mass (the appendix does not say; with no data it absorbs the residual).
 *   K [B,H,Nk,d];  Cp [H,M,d], Cc [H,M,C,d] current codebooks (read only)
 *   Sp [H,M,d], Np [H,M], Sc [H,M,C,d], Nc [H,M,C]   float32 EMA statistics, updated in place
 *   Cp_out, Cc_out   the new codebooks, dtype of K (bfloat16 rounding perturbs the constraint by an ulp)
 *   workspace        avq_codebook_update_workspace_bytes() bytes, 256-byte aligned
 * C <= 16.  Uses B, H, Nk, d, M, C, dtype, flags of `prob`. */
AVQ_API size_t avq_codebook_update_workspace_bytes(const avq_problem* prob);
AVQ_API avq_status avq_codebook_update(const avq_problem* prob, const void* K, const void* Cp, const void* Cc,
                               float decay, float* Sp, float* Np, float* Sc, float* Nc, void* Cp_out,
                               void* Cc_out, void* workspace, size_t workspace_bytes, void* stream);

/* Stage 3 alone: the attention pass of avq_forward over a workspace that a previous
 * avq_forward call with the same `prob`, P and block_q (and the same K, V, Cp, Cc) filled.
 * Reads the aggregates from the workspace, recomputes Y (and the optional outputs) for Q.
 * Lets a caller reuse one set of keys for several query tensors, and lets a profiler time
 * the attention kernel by itself.  Arguments as in avq_forward. */
AVQ_API avq_status avq_attend(const avq_problem* prob, const void* Q, const void* Cp, const void* Cc,
                      int32_t P, int32_t block_q, void* Y, int32_t* topp_out, float* importance_out,
                      void* workspace, size_t workspace_bytes, void* stream);

/* Same computation for callers whose Q, K, V and Y live in HOST memory (pinned memory lets
 * the copies overlap; pageable memory works but serialises).  dQ, dK, dV, dY are device
 * staging buffers of the tensors' sizes, supplied by the caller.  The call enqueues
 * host->device copies of Q, K, V, the forward, and the device->host copy of Y on `stream`
 * and returns; synchronise the stream before reading hY.  Cp, Cc stay device pointers
 * (they are model parameters). */
AVQ_API avq_status avq_forward_host(const avq_problem* prob, const void* hQ, const void* hK, const void* hV,
                            const void* Cp, const void* Cc, int32_t P, int32_t block_q, void* hY,
                            void* dQ, void* dK, void* dV, void* dY, void* workspace,
                            size_t workspace_bytes, void* stream);

/* Size of the built-in scratch array avq_forward_static works in. */
#define AVQ_STATIC_WORKSPACE_BYTES (24u * 1024u * 1024u)

/* avq_forward for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a packaging variant of avq_forward, not a step of the method.)
 *
 * Who needs it: code that must not call cudaMalloc where it runs the forward pass - a
 * plugin given only its input and output buffers, a serving loop whose memory is planned
 * up front, a real-time path that bans allocator calls after start-up.  avq_forward asks
 * such callers for a workspace they cannot produce; this entry point uses a fixed
 * AVQ_STATIC_WORKSPACE_BYTES array inside the library's device image instead, so it makes
 * no cudaMalloc/cudaFree call and calls no allocating library routine.  Every GPU on which
 * the library is loaded holds that array until the process exits.
 *
 * Arguments and results are those of avq_forward without workspace/workspace_bytes.
 *   - Problems whose avq_workspace_bytes() exceeds AVQ_STATIC_WORKSPACE_BYTES are rejected
 *     with AVQ_ERR_WORKSPACE before anything is launched (the three large benchmark
 *     configurations fit; e.g. B = 4, H = 16, N = 65536 does not).
 *   - The first call on a device resolves the array's device address (once per device, with
 *     that device current) and should therefore happen before any stream capture begins.
 *   - All calls share the one array.  Each call clears what it accumulates into, so calls
 *     that run one after another are independent; calls that overlap on the GPU (different
 *     streams, or several host threads) race on it and give wrong results.
 *   - avq_check_static() is avq_check() on the built-in array. */
AVQ_API avq_status avq_forward_static(const avq_problem* prob, const void* Q, const void* K, const void* V,
                              const void* Cp, const void* Cc, int32_t P, int32_t block_q, void* Y,
                              int32_t* topp_out, float* importance_out, void* stream);
AVQ_API avq_status avq_check_static(void* stream);
AVQ_API size_t avq_static_workspace_bytes(void);

/* Byte offsets inside the workspace of what avq_forward leaves there.  Any pointer may be
 * NULL.  parent/child: int32 [B,H,Nk]; Vp f32 [B,H,M,d]; np f32 [B,H,M]; Vc f32 [B,H,M,C,d];
 * nc f32 [B,H,M,C].  Host function. */
AVQ_API avq_status avq_workspace_layout(const avq_problem* prob, int32_t P, int32_t block_q,
                                size_t* parent_idx_off, size_t* child_idx_off, size_t* Vp_off,
                                size_t* np_off, size_t* Vc_off, size_t* nc_off);

/* Waits for `stream`, reads the status word in the workspace header and clears it.
 * AVQ_OK, AVQ_ERR_DEVICE_TIMEOUT (a bounded wait inside a kernel expired; outputs of that
 * call are not valid), AVQ_ERR_INDEX (a kernel skipped a key whose index was out of range)
 * or AVQ_ERR_CUDA.  Blocks the host. */
AVQ_API avq_status avq_check(void* workspace, void* stream);

/* Static, NUL-terminated description of a status code. */
AVQ_API const char* avq_status_string(avq_status s);

/* Library version as major*10000 + minor*100 + patch. */
AVQ_API int32_t avq_version(void);

#ifdef __cplusplus
}
#endif
#endif /* AVQ_ATTN_H_ */
