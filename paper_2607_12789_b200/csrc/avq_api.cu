// C ABI of libavq_attn: argument validation, workspace layout and stage dispatch.
// Every entry point checks its arguments on the host and launches nothing when they are
// unusable; the kernels themselves live in avq_simt.cu (CUDA cores) and avq_tc_*.cu
// (tcgen05 tensor cores).
#include <math.h>
#include <string.h>

#include "avq_internal.h"

namespace avq {

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
static inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

bool use_tensor_path(const avq_problem& p) {
  return p.dtype == AVQ_BF16 && !(p.flags & AVQ_FLAG_SIMT);
}

avq_status validate_problem(const avq_problem* p) {
  if (!p) return AVQ_ERR_NULL;
  if (p->B <= 0 || p->H <= 0 || p->Nq <= 0 || p->Nk <= 0 || p->d <= 0 || p->M <= 0 || p->C <= 0)
    return AVQ_ERR_SHAPE;
  if (p->dtype != AVQ_F32 && p->dtype != AVQ_BF16) return AVQ_ERR_SHAPE;
  if (!isfinite(p->scale)) return AVQ_ERR_SHAPE;
  if (p->flags & ~(uint32_t)(AVQ_FLAG_PARENT_STAYS | AVQ_FLAG_SIMT | AVQ_FLAG_CORRECTING)) return AVQ_ERR_SHAPE;
  if ((int64_t)p->B * p->H > 65535) return AVQ_ERR_UNSUPPORTED;
  if ((int64_t)p->B * p->H * (int64_t)(p->Nq > p->Nk ? p->Nq : p->Nk) * p->d >= ((int64_t)1 << 40))
    return AVQ_ERR_UNSUPPORTED;
  if (use_tensor_path(*p)) {
    if (p->flags & AVQ_FLAG_CORRECTING) return AVQ_ERR_UNSUPPORTED;   // the tensor-core kernel is the masked form
    if (p->d != 64 && p->d != 128) return AVQ_ERR_UNSUPPORTED;
    if (p->M % 32 != 0 || p->M < 32 || p->M > 256) return AVQ_ERR_UNSUPPORTED;
    if (p->C != 4 && p->C != 8) return AVQ_ERR_UNSUPPORTED;
    if (!(p->scale > 0.f)) return AVQ_ERR_UNSUPPORTED;
  } else {
    if (p->d % 4 != 0 || p->d < 4 || p->d > 256) return AVQ_ERR_UNSUPPORTED;
    if (p->M > 1024 || p->C > 16) return AVQ_ERR_UNSUPPORTED;
  }
  return AVQ_OK;
}

avq_status validate_forward(const avq_problem* p, int32_t P, int32_t block_q) {
  avq_status s = validate_problem(p);
  if (s != AVQ_OK) return s;
  if (P < 0 || P > p->M || block_q <= 0) return AVQ_ERR_SHAPE;
  if (use_tensor_path(*p)) {
    if (block_q != 128) return AVQ_ERR_UNSUPPORTED;
  } else {
    if (block_q > 256) return AVQ_ERR_UNSUPPORTED;
    if ((int64_t)p->M + (int64_t)P * p->C > 8192) return AVQ_ERR_UNSUPPORTED;
    if (simt_attend_smem_bytes(p->d, p->M, p->C, P, block_q, 0) > kSimtAttendSmemLimit) return AVQ_ERR_UNSUPPORTED;
  }
  return AVQ_OK;
}

Layout make_layout(const avq_problem& p, int32_t /*P*/, int32_t /*block_q*/) {
  Layout L;
  const size_t BH = (size_t)p.B * p.H;
  size_t off = 256;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  L.header = 0;
  L.Vc = take(sizeof(float) * BH * p.M * p.C * p.d);
  L.nc = take(sizeof(float) * BH * p.M * p.C);
  L.Vp = take(sizeof(float) * BH * p.M * p.d);
  L.np = take(sizeof(float) * BH * p.M);
  L.zero_end = off;
  L.parent_idx = take(sizeof(int32_t) * BH * p.Nk);
  L.child_idx = take(sizeof(int32_t) * BH * p.Nk);
  if (use_tensor_path(p)) {
    L.Vpb = take(2 * BH * p.M * p.d);
    L.Vcb = take(2 * BH * p.M * p.C * p.d);
    if (p.flags & AVQ_FLAG_PARENT_STAYS) {
      L.Vsb = take(2 * BH * p.M * p.d);
      L.rho = take(sizeof(float) * BH * p.M);
    }
    L.cnorm = take(sizeof(float) * (size_t)p.H * p.M);
  }
  L.total = off;
  return L;
}

}  // namespace avq

using namespace avq;

extern "C" {

size_t avq_workspace_bytes(const avq_problem* prob, int32_t P, int32_t block_q) {
  if (validate_forward(prob, P, block_q) != AVQ_OK) return 0;
  return make_layout(*prob, P, block_q).total;
}

avq_status avq_workspace_layout(const avq_problem* prob, int32_t P, int32_t block_q,
                                size_t* parent_idx_off, size_t* child_idx_off, size_t* Vp_off,
                                size_t* np_off, size_t* Vc_off, size_t* nc_off) {
  avq_status s = validate_forward(prob, P, block_q);
  if (s != AVQ_OK) return s;
  Layout L = make_layout(*prob, P, block_q);
  if (parent_idx_off) *parent_idx_off = L.parent_idx;
  if (child_idx_off) *child_idx_off = L.child_idx;
  if (Vp_off) *Vp_off = L.Vp;
  if (np_off) *np_off = L.np;
  if (Vc_off) *Vc_off = L.Vc;
  if (nc_off) *nc_off = L.nc;
  return AVQ_OK;
}

avq_status avq_assign(const avq_problem* prob, const void* K, const void* Cp, const void* Cc,
                      int32_t* parent_idx, int32_t* child_idx, void* stream) {
  avq_status s = validate_problem(prob);
  if (s != AVQ_OK) return s;
  if (!K || !Cp || !Cc || !parent_idx || !child_idx) return AVQ_ERR_NULL;
  if (!aligned16(K) || !aligned16(Cp) || !aligned16(Cc) || !aligned16(parent_idx) || !aligned16(child_idx))
    return AVQ_ERR_ALIGN;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (use_tensor_path(*prob)) return tc_assign(*prob, K, Cp, Cc, parent_idx, child_idx, nullptr, nullptr, 0, nullptr, st);
  return simt_assign(*prob, K, Cp, Cc, parent_idx, child_idx, st);
}

avq_status avq_aggregate(const avq_problem* prob, const void* V, const int32_t* parent_idx,
                         const int32_t* child_idx, float* Vp, float* np_, float* Vc, float* nc,
                         void* stream) {
  avq_status s = validate_problem(prob);
  if (s != AVQ_OK) return s;
  if (!V || !parent_idx || !child_idx || !Vp || !np_ || !Vc || !nc) return AVQ_ERR_NULL;
  if (!aligned16(V) || !aligned16(parent_idx) || !aligned16(child_idx) || !aligned16(Vp) ||
      !aligned16(np_) || !aligned16(Vc) || !aligned16(nc))
    return AVQ_ERR_ALIGN;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (use_tensor_path(*prob))
    return tc_aggregate(*prob, V, parent_idx, child_idx, Vp, np_, Vc, nc, nullptr, nullptr, nullptr, nullptr, false, nullptr, st);
  return simt_aggregate(*prob, V, parent_idx, child_idx, Vp, np_, Vc, nc, st);
}

namespace {
struct Regions {
  int32_t *status_word, *pidx, *cidx;
  float *Vp, *np_, *Vc, *nc;
  void *Vpb, *Vcb, *Vsb;
  float* rho;
  float* cnorm;
};
Regions carve(void* workspace, const Layout& L) {
  char* ws = static_cast<char*>(workspace);
  Regions r;
  r.status_word = reinterpret_cast<int32_t*>(ws + L.header);
  r.pidx = reinterpret_cast<int32_t*>(ws + L.parent_idx);
  r.cidx = reinterpret_cast<int32_t*>(ws + L.child_idx);
  r.Vp = reinterpret_cast<float*>(ws + L.Vp);
  r.np_ = reinterpret_cast<float*>(ws + L.np);
  r.Vc = reinterpret_cast<float*>(ws + L.Vc);
  r.nc = reinterpret_cast<float*>(ws + L.nc);
  r.Vpb = ws + L.Vpb;
  r.Vcb = ws + L.Vcb;
  r.Vsb = L.Vsb ? ws + L.Vsb : nullptr;
  r.rho = L.rho ? reinterpret_cast<float*>(ws + L.rho) : nullptr;
  r.cnorm = L.cnorm ? reinterpret_cast<float*>(ws + L.cnorm) : nullptr;
  return r;
}
avq_status attend_stage(const avq_problem& p, const Regions& r, const void* Q, const void* Cp, const void* Cc,
                        int32_t P, int32_t block_q, void* Y, int32_t* topp_out, float* importance_out,
                        bool chained, cudaStream_t st) {
  if (use_tensor_path(p))
    return tc_attend(p, Q, Cp, Cc, r.np_, r.nc, r.Vpb, r.Vcb, r.Vsb, r.rho, P, Y, topp_out, importance_out, r.status_word,
                     chained, st);
  return simt_attend(p, Q, Cp, Cc, r.Vp, r.np_, r.Vc, r.nc, P, block_q, Y, topp_out, importance_out, 0, st);
}
avq_status check_workspace(const avq_problem* prob, int32_t P, int32_t block_q, void* workspace,
                           size_t workspace_bytes, Layout* L) {
  if (!workspace) return AVQ_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(workspace) & 255u) return AVQ_ERR_ALIGN;
  *L = make_layout(*prob, P, block_q);
  if (workspace_bytes < L->total) return AVQ_ERR_WORKSPACE;
  return AVQ_OK;
}
}  // namespace

avq_status avq_forward(const avq_problem* prob, const void* Q, const void* K, const void* V,
                       const void* Cp, const void* Cc, int32_t P, int32_t block_q, void* Y,
                       int32_t* topp_out, float* importance_out, void* workspace,
                       size_t workspace_bytes, void* stream) {
  avq_status s = validate_forward(prob, P, block_q);
  if (s != AVQ_OK) return s;
  if (!Q || !K || !V || !Cp || !Cc || !Y) return AVQ_ERR_NULL;
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(Cp) || !aligned16(Cc) || !aligned16(Y) ||
      !aligned16(topp_out) || !aligned16(importance_out))
    return AVQ_ERR_ALIGN;
  Layout L;
  s = check_workspace(prob, P, block_q, workspace, workspace_bytes, &L);
  if (s != AVQ_OK) return s;
  const avq_problem& p = *prob;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const Regions r = carve(workspace, L);
  if (use_tensor_path(p)) {
    // status header, leaf sums and leaf counts are adjacent: the assign grid clears them on the side
    // The codeword norms as a pass of their own pay once many CTAs share them and a codebook is large: measured
    // c3 (128 CTAs per head, M d = 32768) -4 us, c2 (M d = 8192) +-0, c1 +1.4 us (the extra launch).
    const bool norms_pass = (size_t)p.M * p.d >= 16384 && (size_t)p.B * p.H * ((p.Nk + 127) / 128) >= 592;
    s = tc_assign(p, K, Cp, Cc, r.pidx, r.cidx, r.status_word, workspace, L.zero_end, norms_pass ? r.cnorm : nullptr, st);
    if (s != AVQ_OK) return s;
    s = tc_aggregate(p, V, r.pidx, r.cidx, r.Vp, r.np_, r.Vc, r.nc, r.Vpb, r.Vcb, r.Vsb, r.rho, true, r.status_word, st);
  } else {
    if (cudaMemsetAsync(r.status_word, 0, 256, st) != cudaSuccess) return AVQ_ERR_CUDA;
    s = simt_assign(p, K, Cp, Cc, r.pidx, r.cidx, st);
    if (s != AVQ_OK) return s;
    s = simt_aggregate(p, V, r.pidx, r.cidx, r.Vp, r.np_, r.Vc, r.nc, st);
  }
  if (s != AVQ_OK) return s;
  return attend_stage(p, r, Q, Cp, Cc, P, block_q, Y, topp_out, importance_out, true, st);
}

avq_status avq_forward_tiled(const avq_problem* prob, const void* Q, const void* K, const void* V,
                             const void* Cp, const void* Cc, int32_t P, int32_t block_q, int32_t tile_m,
                             void* Y, int32_t* topp_out, float* importance_out, void* workspace,
                             size_t workspace_bytes, void* stream) {
  if (!prob) return AVQ_ERR_NULL;
  avq_problem p = *prob;
  p.flags |= AVQ_FLAG_SIMT;                        // the tiled importance lives in the CUDA-core attention kernel
  avq_status s = validate_forward(&p, P, block_q);
  if (s != AVQ_OK) return s;
  if (tile_m < 32 || tile_m % 32 != 0) return AVQ_ERR_SHAPE;
  if (simt_attend_smem_bytes(p.d, p.M, p.C, P, block_q, tile_m) > kSimtAttendSmemLimit) return AVQ_ERR_UNSUPPORTED;
  if (!Q || !K || !V || !Cp || !Cc || !Y) return AVQ_ERR_NULL;
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(Cp) || !aligned16(Cc) || !aligned16(Y) ||
      !aligned16(topp_out) || !aligned16(importance_out))
    return AVQ_ERR_ALIGN;
  Layout L;
  s = check_workspace(&p, P, block_q, workspace, workspace_bytes, &L);
  if (s != AVQ_OK) return s;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const Regions r = carve(workspace, L);
  if (cudaMemsetAsync(r.status_word, 0, 256, st) != cudaSuccess) return AVQ_ERR_CUDA;
  s = simt_assign(p, K, Cp, Cc, r.pidx, r.cidx, st);
  if (s != AVQ_OK) return s;
  s = simt_aggregate(p, V, r.pidx, r.cidx, r.Vp, r.np_, r.Vc, r.nc, st);
  if (s != AVQ_OK) return s;
  return simt_attend(p, Q, Cp, Cc, r.Vp, r.np_, r.Vc, r.nc, P, block_q, Y, topp_out, importance_out, tile_m, st);
}

avq_status avq_attend(const avq_problem* prob, const void* Q, const void* Cp, const void* Cc, int32_t P,
                      int32_t block_q, void* Y, int32_t* topp_out, float* importance_out, void* workspace,
                      size_t workspace_bytes, void* stream) {
  avq_status s = validate_forward(prob, P, block_q);
  if (s != AVQ_OK) return s;
  if (!Q || !Cp || !Cc || !Y) return AVQ_ERR_NULL;
  if (!aligned16(Q) || !aligned16(Cp) || !aligned16(Cc) || !aligned16(Y) || !aligned16(topp_out) ||
      !aligned16(importance_out))
    return AVQ_ERR_ALIGN;
  Layout L;
  s = check_workspace(prob, P, block_q, workspace, workspace_bytes, &L);
  if (s != AVQ_OK) return s;
  return attend_stage(*prob, carve(workspace, L), Q, Cp, Cc, P, block_q, Y, topp_out, importance_out, false,
                      static_cast<cudaStream_t>(stream));
}

avq_status avq_forward_host(const avq_problem* prob, const void* hQ, const void* hK, const void* hV,
                            const void* Cp, const void* Cc, int32_t P, int32_t block_q, void* hY,
                            void* dQ, void* dK, void* dV, void* dY, void* workspace,
                            size_t workspace_bytes, void* stream) {
  avq_status s = validate_forward(prob, P, block_q);
  if (s != AVQ_OK) return s;
  if (!hQ || !hK || !hV || !hY || !dQ || !dK || !dV || !dY) return AVQ_ERR_NULL;
  const avq_problem& p = *prob;
  const size_t es = p.dtype == AVQ_F32 ? 4 : 2;
  const size_t qb = es * (size_t)p.B * p.H * p.Nq * p.d;
  const size_t kb = es * (size_t)p.B * p.H * p.Nk * p.d;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(dQ, hQ, qb, cudaMemcpyHostToDevice, st) != cudaSuccess) return AVQ_ERR_CUDA;
  if (cudaMemcpyAsync(dK, hK, kb, cudaMemcpyHostToDevice, st) != cudaSuccess) return AVQ_ERR_CUDA;
  if (cudaMemcpyAsync(dV, hV, kb, cudaMemcpyHostToDevice, st) != cudaSuccess) return AVQ_ERR_CUDA;
  s = avq_forward(prob, dQ, dK, dV, Cp, Cc, P, block_q, dY, nullptr, nullptr, workspace, workspace_bytes,
                  stream);
  if (s != AVQ_OK) return s;
  if (cudaMemcpyAsync(hY, dY, qb, cudaMemcpyDeviceToHost, st) != cudaSuccess) return AVQ_ERR_CUDA;
  return AVQ_OK;
}

avq_status avq_check(void* workspace, void* stream) {
  if (!workspace) return AVQ_ERR_NULL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int32_t word = 0;
  if (cudaMemcpyAsync(&word, workspace, sizeof(word), cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return AVQ_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return AVQ_ERR_CUDA;
  if (word != 0) {
    if (cudaMemsetAsync(workspace, 0, sizeof(word), st) != cudaSuccess) return AVQ_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return AVQ_ERR_CUDA;
    return word == DEV_BAD_INDEX ? AVQ_ERR_INDEX : AVQ_ERR_DEVICE_TIMEOUT;
  }
  return AVQ_OK;
}

const char* avq_status_string(avq_status s) {
  switch (s) {
    case AVQ_OK: return "ok";
    case AVQ_ERR_NULL: return "a required pointer is NULL";
    case AVQ_ERR_SHAPE: return "a size, dtype, flag or P is invalid";
    case AVQ_ERR_UNSUPPORTED: return "problem is outside the supported envelope of the selected kernels";
    case AVQ_ERR_ALIGN: return "a pointer is not sufficiently aligned";
    case AVQ_ERR_WORKSPACE: return "workspace is NULL or too small";
    case AVQ_ERR_CUDA: return "a CUDA call failed";
    case AVQ_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait expired";
    case AVQ_ERR_INDEX: return "a parent or child index read by a kernel was out of range";
  }
  return "unknown status";
}

int32_t avq_version(void) { return 100; }

}  // extern "C"
