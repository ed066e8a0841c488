// Internal declarations shared by the translation units of libavq_attn (not part of the ABI).
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "avq_attn.h"

namespace avq {

// Byte offsets of the regions of an avq_forward workspace.
struct Layout {
  size_t header = 0;       // 256 bytes; int32 status word at offset 0
  size_t Vc = 0;           // f32 [B,H,M,C,d]   header, Vc, nc, Vp and np are adjacent: one pass clears them
  size_t nc = 0;           // f32 [B,H,M,C]
  size_t Vp = 0;           // f32 [B,H,M,d]     (accumulates the keys that stay with their parent)
  size_t np = 0;           // f32 [B,H,M]
  size_t zero_end = 0;     // end of the region that must be zero before aggregation
  size_t parent_idx = 0;   // int32 [B,H,Nk]
  size_t child_idx = 0;    // int32 [B,H,Nk]
  size_t Vpb = 0;          // bf16 [B,H,M,d]      copy of Vp (tensor-core path only)
  size_t Vcb = 0;          // bf16 [B,H,M,C,d]    copy of Vc (tensor-core path only)
  size_t Vsb = 0;          // bf16 [B,H,M,d]      stay residual rows (tensor-core path, PARENT_STAYS)
  size_t rho = 0;          // f32 [B,H,M]         share of a parent's keys that stay
  size_t cnorm = 0;        // f32 [H,M]           squared norms of the parent codewords (tensor-core path)
  size_t total = 0;
};

// Device status codes written to the workspace header by kernels that give up on a wait.
enum DeviceCode : int32_t {
  DEV_OK = 0,
  DEV_TIMEOUT_ASSIGN = 101,
  DEV_TIMEOUT_ATTEND = 102,
  DEV_TIMEOUT_TEST = 103,      // the self-test wait of avq_selftest_wait_expiry
  DEV_BAD_INDEX = 201,         // a caller-supplied parent / child index was out of range (the key was skipped)
};

bool use_tensor_path(const avq_problem& p);
avq_status validate_problem(const avq_problem* p);
avq_status validate_forward(const avq_problem* p, int32_t P, int32_t block_q);
Layout make_layout(const avq_problem& p, int32_t P, int32_t block_q);

// ---- plain CUDA-core kernels (avq_simt.cu) ----
avq_status simt_assign(const avq_problem& p, const void* K, const void* Cp, const void* Cc,
                       int32_t* parent_idx, int32_t* child_idx, cudaStream_t st);
avq_status simt_aggregate(const avq_problem& p, const void* V, const int32_t* parent_idx,
                          const int32_t* child_idx, float* Vp, float* np_, float* Vc, float* nc,
                          cudaStream_t st);
avq_status simt_attend(const avq_problem& p, const void* Q, const void* Cp, const void* Cc,
                       const float* Vp, const float* np_, const float* Vc, const float* nc, int32_t P,
                       int32_t block_q, void* Y, int32_t* topp_out, float* importance_out,
                       int32_t tile_m, cudaStream_t st);   // tile_m: 0 = exact importance

// Shared memory the CUDA-core attention kernel needs for a problem, and the most it may ask for.
size_t simt_attend_smem_bytes(int d, int M, int C, int P, int block_q, int tile_m);
constexpr size_t kSimtAttendSmemLimit = 200 * 1024;

// ---- tensor-core kernels (avq_tc_*.cu) ----
// zero_base / zero_bytes: a region (multiple of 16 bytes, or none) the assign grid clears on the side
// cnorm: scratch for [H, M] squared codeword norms, filled by a small kernel ahead of the assign grid; when
// null every assign CTA computes the norms of its head itself
avq_status tc_assign(const avq_problem& p, const void* K, const void* Cp, const void* Cc,
                     int32_t* parent_idx, int32_t* child_idx, int32_t* status_word, void* zero_base,
                     size_t zero_bytes, float* cnorm, cudaStream_t st);
avq_status tc_aggregate(const avq_problem& p, const void* V, const int32_t* parent_idx,
                        const int32_t* child_idx, float* Vp, float* np_, float* Vc, float* nc,
                        void* Vpb, void* Vcb, void* Vsb, float* rho, bool pre_zeroed, int32_t* status_word,
                        cudaStream_t st);   // Vsb, rho: stay rows and stay shares (PARENT_STAYS), may be null
avq_status tc_attend(const avq_problem& p, const void* Q, const void* Cp, const void* Cc,
                     const float* np_, const float* nc, const void* Vpb, const void* Vcb, const void* Vsb,
                     const float* rho, int32_t P,
                     void* Y, int32_t* topp_out, float* importance_out, int32_t* status_word,
                     bool chained, cudaStream_t st);   // chained: launched right behind tc_aggregate

inline avq_status cuda_ok(cudaError_t e) { return e == cudaSuccess ? AVQ_OK : AVQ_ERR_CUDA; }

}  // namespace avq
