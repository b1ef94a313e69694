// placeholder until the tcgen05 kernel lands
#include "moga_internal.cuh"
namespace moga {
moga_status launch_attn_bf16(const moga_shape&, const WsLayout&, const void*, const void*,
                             const void*, const int32_t*, void*, float*, char*, cudaStream_t) {
  return MOGA_ERR_UNSUPPORTED;
}
}  // namespace moga
