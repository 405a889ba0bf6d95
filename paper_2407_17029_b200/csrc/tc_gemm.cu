// Tensor-core path (placeholder until the tcgen05 kernels land): reports "not supported" so the
// general path is used.
#include "common.cuh"
namespace qb {
bool tc_supported(const QwView&, const AdView*, int64_t) { return false; }
size_t tc_ws_bytes(int, const QwView&, const AdView*, int64_t) { return kStatusBytes; }
int tc_linear_fwd(const QwView&, const AdView*, const __nv_bfloat16*, int64_t, void*, int, char*, cudaStream_t) { return QBLORA_ERR_UNSUPPORTED; }
int tc_linear_bwd(const QwView&, const AdView*, const __nv_bfloat16*, const __nv_bfloat16*, int64_t, void*, int, float*, float*, char*, cudaStream_t) { return QBLORA_ERR_UNSUPPORTED; }
}  // namespace qb
