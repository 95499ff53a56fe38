// Rotary embedding indexed by position_ids: the standalone in-place kernel and the
// (cos, sin) table the attention kernels read while they rotate Q/K tiles in shared
// memory.  The paper requires only that position ids reach the attention (end of
// Sec. 3.5); the rotation is the usual half-split one.  Angles are formed in fp64 so
// that ids up to 2^17 lose nothing before the fp32 cos/sin are taken.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "pk_common.cuh"

namespace pk {
namespace {

__device__ __forceinline__ void angle_cos_sin(int pos, int i, int D, double log2_theta,
                                              float* c, float* s) {
  const double inv_freq = exp2(-2.0 * (double)i / (double)D * log2_theta);
  double sd, cd;
  sincos((double)pos * inv_freq, &sd, &cd);
  *c = (float)cd;
  *s = (float)sd;
}

// table[t][i] = (cos, sin)(pos[t] * theta^(-2i/D))
__global__ void rope_table_kernel(const int32_t* __restrict__ pos, int T, int D, double log2_theta,
                                  float2* __restrict__ table) {
  const int half = D / 2;
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)T * half) return;
  const int t = (int)(idx / half), i = (int)(idx % half);
  float c, s;
  angle_cos_sin(pos[t], i, D, log2_theta, &c, &s);
  table[idx] = make_float2(c, s);
}

// angle[t][i] = pos[t] * theta^(-2i/D) reduced to [-pi, pi] (in fp64, then rounded to fp32): what the
// epilogues of the rotated-copies path read.  Half the bytes of a (cos, sin) pair per entry, which
// is what their row-per-thread loads are bound by; they take sine and cosine with the fast
// intrinsics, accurate to 4e-7 on that range.
__global__ void rope_angle_kernel(const int32_t* __restrict__ pos, int T, int D, int row,
                                  double log2_theta, float* __restrict__ angle) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)T * row) return;
  const int t = (int)(idx / row), i = (int)(idx % row);
  if (i >= D / 2) {       // columns a padded head does not have
    angle[idx] = 0.f;
    return;
  }
  const double a = (double)pos[t] * exp2(-2.0 * (double)i / (double)D * log2_theta);
  const double two_pi = 6.283185307179586476925286766559;
  angle[idx] = (float)(a - two_pi * rint(a / two_pi));
}

// One thread per (token, pair index); loops over heads so cos/sin are formed once.
__global__ void rope_apply_kernel(__nv_bfloat16* __restrict__ x, const int32_t* __restrict__ pos,
                                  int T, int H, int D, double log2_theta, int inverse) {
  const int half = D / 2;
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)T * half) return;
  const int t = (int)(idx / half), i = (int)(idx % half);
  float c, s;
  angle_cos_sin(pos[t], i, D, log2_theta, &c, &s);
  if (inverse) s = -s;
  __nv_bfloat16* row = x + (int64_t)t * H * D;
  for (int h = 0; h < H; ++h) {
    const float a = __bfloat162float(row[h * D + i]);
    const float b = __bfloat162float(row[h * D + i + half]);
    row[h * D + i] = __float2bfloat16_rn(a * c - b * s);
    row[h * D + i + half] = __float2bfloat16_rn(b * c + a * s);
  }
}

// y = rotate(x) stored as fp16: one thread per (token, pair index), looping over the heads.
__global__ void rope_rotate_f16_kernel(const __nv_bfloat16* __restrict__ x,
                                       const int32_t* __restrict__ pos, int T, int H, int D,
                                       double log2_theta, __half* __restrict__ y) {
  const int half = D / 2;
  if ((D & 15) == 0) {
    // 16-byte accesses: a thread owns 8 consecutive pair indices of one token; its 8 (cos, sin)
    // are formed once and reused for every head.  HBM-bound: 2 B read + 2 B written per element.
    const int chunks = half / 8;
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (int64_t)T * chunks) return;
    const int t = (int)(idx / chunks), i0 = (int)(idx % chunks) * 8;
    float c[8], s[8];
    const int p = pos[t];
#pragma unroll
    for (int e = 0; e < 8; ++e) angle_cos_sin(p, i0 + e, D, log2_theta, &c[e], &s[e]);
    const __nv_bfloat16* xr = x + (int64_t)t * H * D + i0;
    __half* yr = y + (int64_t)t * H * D + i0;
    for (int h = 0; h < H; ++h) {
      const uint4 a4 = *reinterpret_cast<const uint4*>(xr + h * D);
      const uint4 b4 = *reinterpret_cast<const uint4*>(xr + h * D + half);
      const __nv_bfloat162* av = reinterpret_cast<const __nv_bfloat162*>(&a4);
      const __nv_bfloat162* bv = reinterpret_cast<const __nv_bfloat162*>(&b4);
      uint4 o1, o2;
      __half2* o1v = reinterpret_cast<__half2*>(&o1);
      __half2* o2v = reinterpret_cast<__half2*>(&o2);
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float2 a = __bfloat1622float2(av[e]), b = __bfloat1622float2(bv[e]);
        o1v[e] = __floats2half2_rn(a.x * c[2 * e] - b.x * s[2 * e],
                                   a.y * c[2 * e + 1] - b.y * s[2 * e + 1]);
        o2v[e] = __floats2half2_rn(b.x * c[2 * e] + a.x * s[2 * e],
                                   b.y * c[2 * e + 1] + a.y * s[2 * e + 1]);
      }
      *reinterpret_cast<uint4*>(yr + h * D) = o1;
      *reinterpret_cast<uint4*>(yr + h * D + half) = o2;
    }
    return;
  }
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)T * half) return;
  const int t = (int)(idx / half), i = (int)(idx % half);
  float c, s;
  angle_cos_sin(pos[t], i, D, log2_theta, &c, &s);
  const __nv_bfloat16* xr = x + (int64_t)t * H * D;
  __half* yr = y + (int64_t)t * H * D;
  for (int h = 0; h < H; ++h) {
    const float a = __bfloat162float(xr[h * D + i]);
    const float b = __bfloat162float(xr[h * D + i + half]);
    yr[h * D + i] = __float2half_rn(a * c - b * s);
    yr[h * D + i + half] = __float2half_rn(b * c + a * s);
  }
}

}  // namespace

int g_rope_mode = 0;

int rope_rotate_f16_launch(const void* x, const int32_t* position_ids, int32_t T, int32_t H,
                           int32_t D, float theta, void* y, cudaStream_t stream) {
  if (T == 0) return PK_OK;
  const int64_t n = (int64_t)T * ((D & 15) == 0 ? D / 16 : D / 2);
  const int threads = 128;
  const unsigned blocks = (unsigned)((n + threads - 1) / threads);
  rope_rotate_f16_kernel<<<blocks, threads, 0, stream>>>(
      static_cast<const __nv_bfloat16*>(x), position_ids, T, H, D, log2((double)theta),
      static_cast<__half*>(y));
  return launch_status();
}

int rope_angle_launch(const int32_t* position_ids, int32_t T, int32_t D, float theta,
                      float* angle, cudaStream_t stream, int32_t row) {
  if (T == 0) return PK_OK;
  if (row <= 0) row = D / 2;
  const int64_t n = (int64_t)T * row;
  const int threads = 256;
  const unsigned blocks = (unsigned)((n + threads - 1) / threads);
  rope_angle_kernel<<<blocks, threads, 0, stream>>>(position_ids, T, D, row, log2((double)theta),
                                                    angle);
  return launch_status();
}

int rope_table_launch(const int32_t* position_ids, int32_t T, int32_t D, float theta,
                      float* table, cudaStream_t stream) {
  if (T == 0) return PK_OK;
  const int64_t n = (int64_t)T * (D / 2);
  const int threads = 256;
  const unsigned blocks = (unsigned)((n + threads - 1) / threads);
  rope_table_kernel<<<blocks, threads, 0, stream>>>(position_ids, T, D, log2((double)theta),
                                                    reinterpret_cast<float2*>(table));
  return launch_status();
}

}  // namespace pk

extern "C" int pk_rope_apply(void* x, const int32_t* position_ids, int32_t T, int32_t H,
                             int32_t D, float theta, int32_t inverse, void* stream) {
  if (T < 0 || H <= 0) return PK_ERR_INVALID_ARG;
  if (D <= 0 || D > 256 || (D & 1)) return PK_ERR_UNSUPPORTED;
  if (!(theta > 0.0f)) return PK_ERR_INVALID_ARG;
  if (T == 0) return PK_OK;
  if (x == nullptr || position_ids == nullptr) return PK_ERR_INVALID_ARG;
  const int64_t n = (int64_t)T * (D / 2);
  const int threads = 256;
  const unsigned blocks = (unsigned)((n + threads - 1) / threads);
  pk::rope_apply_kernel<<<blocks, threads, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<__nv_bfloat16*>(x), position_ids, T, H, D, log2((double)theta), inverse);
  return pk::launch_status();
}

extern "C" int pk_set_rope_mode(int32_t mode) {
  if (mode != PK_ROPE_ROTATED_COPIES && mode != PK_ROPE_IN_TILE) return PK_ERR_INVALID_ARG;
  pk::g_rope_mode = mode;
  return PK_OK;
}
