// Small device helpers shared by the attention kernels: vector reductions to global memory
// and row-chunk stores with an optional cast to bf16.
#pragma once

#include <cuda_bf16.h>

#include "sm100_ptx.cuh"

namespace pk {
namespace {

using ptx::pack_bf16x2;

__device__ __forceinline__ void red_add_v4(float* addr, float a, float b, float c, float d) {
  asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};"
               ::"l"(addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}

template <typename GradT>
__device__ __forceinline__ void store_chunk32(GradT* dst, const float* x);
template <>
__device__ __forceinline__ void store_chunk32<float>(float* dst, const float* x) {
#pragma unroll
  for (int c = 0; c < 32; c += 4)
    *reinterpret_cast<float4*>(dst + c) = make_float4(x[c], x[c + 1], x[c + 2], x[c + 3]);
}
template <>
__device__ __forceinline__ void store_chunk32<__nv_bfloat16>(__nv_bfloat16* dst, const float* x) {
#pragma unroll
  for (int c = 0; c < 32; c += 8) {
    uint4 o;
    o.x = pack_bf16x2(x[c], x[c + 1]);
    o.y = pack_bf16x2(x[c + 2], x[c + 3]);
    o.z = pack_bf16x2(x[c + 4], x[c + 5]);
    o.w = pack_bf16x2(x[c + 6], x[c + 7]);
    *reinterpret_cast<uint4*>(dst + c) = o;
  }
}


}  // namespace
}  // namespace pk
