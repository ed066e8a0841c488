// Placeholder until the tcgen05 kernels land.
#include "avq_internal.h"
namespace avq {
avq_status tc_assign(const avq_problem&, const void*, const void*, const void*, int32_t*, int32_t*, int32_t*,
                     cudaStream_t) { return AVQ_ERR_UNSUPPORTED; }
avq_status tc_aggregate(const avq_problem&, const void*, const int32_t*, const int32_t*, float*, float*, float*,
                        float*, void*, void*, cudaStream_t) { return AVQ_ERR_UNSUPPORTED; }
avq_status tc_attend(const avq_problem&, const void*, const void*, const void*, const float*, const float*,
                     const void*, const void*, int32_t, void*, int32_t*, float*, int32_t*, cudaStream_t) {
  return AVQ_ERR_UNSUPPORTED;
}
}  // namespace avq
