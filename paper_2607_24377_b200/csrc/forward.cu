// placeholder, replaced by the fused attention kernel
#include "common.cuh"
namespace mxattn {
int launch_forward(const void*, const void*, const void*, const void*, const void*, const void*, void*,
                   int, int, int64_t, int64_t, float, unsigned, int*, cudaStream_t) {
  return MXATTN_EUNSUPPORTED;
}
}
