#include "kvp_host.h"
namespace kvp {
int attn_bwd_read_status() { return 0; }
size_t attn_bwd_workspace(const kvp_shape*, const int32_t*) { return 0; }
int attn_bwd_all(const kvp_shape*, const int32_t*, int, float, const void* const*, const void* const*,
                 const void* const*, const void* const*, const void* const*, const float* const*, void* const*,
                 float* const*, float* const*, void*, size_t, cudaStream_t) { return KVP_ERR_UNSUPPORTED; }
}  // namespace kvp
