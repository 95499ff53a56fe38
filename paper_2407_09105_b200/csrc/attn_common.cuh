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

// 32 bytes per store where the address allows it: the epilogues write one row per thread, so a
// warp's store touches 32 different rows, and the load/store unit's time goes with the number
// of (row, instruction) pairs; full 32-byte sectors also spare L2 the partial writes.
__device__ __forceinline__ void st_global_v8(void* p, const uint32_t* v) {
  asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
               ::"l"(p), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]),
                 "r"(v[6]), "r"(v[7]) : "memory");
}

// eight reduced rotation angles per load (rows of the angle table are 32-byte aligned), turned
// into (cos, sin) with the fast intrinsics: the angles lie in [-pi, pi], where those are accurate
// to 4e-7
__device__ __forceinline__ void ld_angles8(const float* p, float2* t) {
  float v[8];
  asm volatile("ld.global.nc.v8.f32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]), "=f"(v[4]), "=f"(v[5]), "=f"(v[6]),
                 "=f"(v[7])
               : "l"(p));
#pragma unroll
  for (int e = 0; e < 8; ++e) __sincosf(v[e], &t[e].y, &t[e].x);
}

template <typename GradT>
__device__ __forceinline__ void store_chunk32(GradT* dst, const float* x);
template <>
__device__ __forceinline__ void store_chunk32<float>(float* dst, const float* x) {
  if ((reinterpret_cast<uintptr_t>(dst) & 31) == 0) {
#pragma unroll
    for (int c = 0; c < 32; c += 8) {
      uint32_t v[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) v[e] = __float_as_uint(x[c + e]);
      st_global_v8(dst + c, v);
    }
    return;
  }
#pragma unroll
  for (int c = 0; c < 32; c += 4)
    *reinterpret_cast<float4*>(dst + c) = make_float4(x[c], x[c + 1], x[c + 2], x[c + 3]);
}
// 32 bf16 values, already packed in pairs
__device__ __forceinline__ void store_packed32(__nv_bfloat16* dst, const uint32_t* v) {
  if ((reinterpret_cast<uintptr_t>(dst) & 31) == 0) {
    st_global_v8(dst, v);
    st_global_v8(dst + 16, v + 8);
    return;
  }
#pragma unroll
  for (int c = 0; c < 16; c += 4)
    *reinterpret_cast<uint4*>(dst + 2 * c) = make_uint4(v[c], v[c + 1], v[c + 2], v[c + 3]);
}
template <>
__device__ __forceinline__ void store_chunk32<__nv_bfloat16>(__nv_bfloat16* dst, const float* x) {
  uint32_t v[16];
#pragma unroll
  for (int c = 0; c < 16; ++c) v[c] = pack_bf16x2(x[2 * c], x[2 * c + 1]);
  store_packed32(dst, v);
}


}  // namespace
}  // namespace pk
