// Placeholder until the tensor-core kernels land: reports every shape as unsupported so
// that the generic path runs.
#include "ta_common.cuh"
namespace ta {
bool fast_fwd_supported(const tucker_attn_desc&) { return false; }
size_t fast_fwd_workspace(const tucker_attn_desc&) { return 0; }
int fast_fwd(Problem&) { return TA_ERR_UNSUPPORTED_SHAPE; }
bool fast_decode_supported(const tucker_attn_desc&, int32_t) { return false; }
size_t fast_decode_workspace(const tucker_attn_desc&, int32_t) { return 0; }
int fast_decode(Problem&) { return TA_ERR_UNSUPPORTED_SHAPE; }
}  // namespace ta
