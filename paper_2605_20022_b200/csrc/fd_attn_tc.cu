// placeholder: the tensor-core attention kernel is added in a later step
#include "fd_internal.cuh"
namespace fd {
bool attn_tc_supported(int, int, int) { return false; }
cudaError_t attn_tc_prepare(void**, const AttnParams&) { return cudaErrorNotSupported; }
void launch_attn_tc(void*, const AttnParams&, cudaStream_t) {}
void attn_tc_free(void*) {}
}  // namespace fd
