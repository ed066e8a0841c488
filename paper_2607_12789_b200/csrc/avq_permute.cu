// avq_forward_permuted: the forward pass over query tiles that follow a caller-supplied token order
// (Sec. "Vector Quantization for (A)VQ-Attention": image tokens are reordered along a space-filling curve
// so that a tile holds neighbouring tokens; the curve itself is the caller's business).
//
// Only the grouping of QUERIES into tiles changes the result: per-codeword sums and counts do not depend
// on the order of the keys.  So the call gathers Q into tile order, runs avq_forward on it, and scatters
// the output rows back:  Qp[i] = Q[perm[i]],  Y[perm[i]] = Yp[i].  Two extra passes over Q and Y.
#include "avq_internal.h"

namespace avq {
namespace {

// rows of `row_vec` 16-byte vectors; one warp copies a row.  gather: dst[i] = src[perm[i]];
// scatter: dst[perm[i]] = src[i].  An index outside [0, N) is flagged; its row is gathered as zeros and not
// scattered at all.
__global__ void __launch_bounds__(256)
permute_rows_kernel(uint4* __restrict__ dst, const uint4* __restrict__ src, const int32_t* __restrict__ perm,
                    int N, int row_vec, long long rows_total, int scatter, int32_t* status_word) {
  const int lane = threadIdx.x & 31;
  const long long row = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (row >= rows_total) return;
  const long long bh = row / N;
  const int i = (int)(row - bh * N);
  const int j = __ldg(perm + i);
  if (j < 0 || j >= N) {
    if (lane == 0 && status_word) atomicCAS(status_word, 0, DEV_BAD_INDEX);
    if (!scatter)                                     // the tile still needs a defined query row: zeros
      for (int v = lane; v < row_vec; v += 32) dst[row * row_vec + v] = make_uint4(0u, 0u, 0u, 0u);
    return;
  }
  const long long from = scatter ? row : bh * N + j, to = scatter ? bh * N + j : row;
  for (int v = lane; v < row_vec; v += 32) dst[to * row_vec + v] = __ldg(src + from * row_vec + v);
}

avq_status permute_rows(void* dst, const void* src, const int32_t* perm, const avq_problem& p, bool scatter,
                        int32_t* status_word, cudaStream_t st) {
  const size_t es = p.dtype == AVQ_F32 ? 4 : 2;
  const int row_vec = (int)(p.d * es / 16);
  const long long rows = (long long)p.B * p.H * p.Nq;
  const unsigned blocks = (unsigned)((rows + 7) / 8);
  permute_rows_kernel<<<blocks, 256, 0, st>>>(static_cast<uint4*>(dst), static_cast<const uint4*>(src), perm,
                                             p.Nq, row_vec, rows, scatter ? 1 : 0, status_word);
  return cuda_ok(cudaGetLastError());
}

inline size_t align256(size_t x) { return (x + 255) / 256 * 256; }

}  // namespace
}  // namespace avq

using namespace avq;

extern "C" {

size_t avq_workspace_bytes_permuted(const avq_problem* prob, int32_t P, int32_t block_q) {
  const size_t base = avq_workspace_bytes(prob, P, block_q);
  if (base == 0) return 0;
  const size_t es = prob->dtype == AVQ_F32 ? 4 : 2;
  if ((prob->d * es) % 16 != 0) return 0;
  const size_t qb = align256(es * (size_t)prob->B * prob->H * prob->Nq * prob->d);
  return align256(base) + 2 * qb;
}

avq_status avq_forward_permuted(const avq_problem* prob, const void* Q, const void* K, const void* V,
                                const void* Cp, const void* Cc, int32_t P, int32_t block_q,
                                const int32_t* perm, void* Y, int32_t* topp_out, float* importance_out,
                                void* workspace, size_t workspace_bytes, void* stream) {
  avq_status s = validate_forward(prob, P, block_q);
  if (s != AVQ_OK) return s;
  if (!perm || !Q || !Y) return AVQ_ERR_NULL;
  if (reinterpret_cast<uintptr_t>(perm) & 3u) return AVQ_ERR_ALIGN;
  const size_t es = prob->dtype == AVQ_F32 ? 4 : 2;
  if ((prob->d * es) % 16 != 0) return AVQ_ERR_UNSUPPORTED;
  if (!workspace) return AVQ_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(workspace) & 255u) return AVQ_ERR_ALIGN;
  const size_t need = avq_workspace_bytes_permuted(prob, P, block_q);
  if (need == 0 || workspace_bytes < need) return AVQ_ERR_WORKSPACE;
  const size_t base = align256(avq_workspace_bytes(prob, P, block_q));
  const size_t qb = align256(es * (size_t)prob->B * prob->H * prob->Nq * prob->d);
  char* ws = static_cast<char*>(workspace);
  void* Qp = ws + base;
  void* Yp = ws + base + qb;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // avq_forward clears the status header at offset 0 at its start, so an index flagged by the gather would be
  // lost: the gather runs first without a status word, the scatter (same indices) reports.
  s = permute_rows(Qp, Q, perm, *prob, false, nullptr, st);
  if (s != AVQ_OK) return s;
  s = avq_forward(prob, Qp, K, V, Cp, Cc, P, block_q, Yp, topp_out, importance_out, workspace, base, stream);
  if (s != AVQ_OK) return s;
  return permute_rows(Y, Yp, perm, *prob, true, static_cast<int32_t*>(workspace), st);
}

}  // extern "C"
