// BF16 tensor-core gradient path (placeholder until the tcgen05 kernels land).
#include "common.cuh"

namespace dbw {
int grad_bf16_alloc(dbw_handle*) { return DBW_ERR_BAD_MODEL; }
void grad_bf16_free(dbw_handle*) {}
int launch_grad_bf16(dbw_handle*, const float*, const int32_t*, float*, float*, cudaStream_t) {
    return DBW_ERR_BAD_MODEL;
}
}  // namespace dbw
