// Tensor-core (tcgen05) kernel family -- placeholder until the kernels land.
#include "mrp_internal.cuh"

namespace mrp {
bool tc_supported(const mrp_config &, const mrp_head_weights *, const void *) { return false; }
cudaError_t tc_create(Ctx *) { return cudaErrorNotSupported; }
void tc_destroy(Ctx *) {}
cudaError_t tc_draft(Ctx *, const void *, const float *, const int32_t *, int, int,
                     const mrp_draft_out &, cudaStream_t) { return cudaErrorNotSupported; }
}  // namespace mrp
