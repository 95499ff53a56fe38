// placeholder, replaced by the backward kernels
#include "pk_common.cuh"
extern "C" int pk_attn_bwd(const void*, const void*, const void*, const void*, const void*, int32_t,
                           const float*, const int32_t*, int32_t, int32_t, int32_t, int32_t, float,
                           float, void*, void*, void*, int32_t, int32_t, void*, size_t, void*) {
  return PK_ERR_UNSUPPORTED;
}
