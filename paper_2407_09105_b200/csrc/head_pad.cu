// Head sizes other than 64 and 128 (multiples of 16 up to 128: 80 and 96 among the model list of
// Sec. 3.5's closing paragraph): the attention kernels are built for 64 and 128 columns, so such a
// call runs on zero-padded copies.  Zero columns change neither Q K^T nor the softmax, and the
// columns of O, dQ, dK, dV they produce are dropped again.
//
// Layout of a padded head row (P = padded size, D = the caller's): the two halves of the row stay
// halves, [x[0 : D/2], 0 ..., x[D/2 : D], 0 ...] with the second half at column P/2, so that the
// rotary pairs (i, i + D/2) remain (i, i + P/2).  With RoPE the padded copies of q and k are the
// rotated fp16 copies the warp-specialised kernels work on anyway (angles pos * theta^(-2i/D),
// for the caller's D), and the backward's epilogues rotate dQ and dK back from an angle table
// that is zero in the pad columns.
//
// Cost: one streaming pass over every tensor each way, and contractions at the padded size.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "pk_common.cuh"
#include "tensor_map.cuh"

namespace pk {
namespace {

__device__ __forceinline__ void load8(const __nv_bfloat16* p, float* x) {
  const uint4 r = *reinterpret_cast<const uint4*>(p);
  const __nv_bfloat162* v = reinterpret_cast<const __nv_bfloat162*>(&r);
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const float2 f = __bfloat1622float2(v[e]);
    x[2 * e] = f.x;
    x[2 * e + 1] = f.y;
  }
}
__device__ __forceinline__ void load8(const float* p, float* x) {
  const float4 a = *reinterpret_cast<const float4*>(p), b = *reinterpret_cast<const float4*>(p + 4);
  x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w;
  x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
}
__device__ __forceinline__ void store8(__nv_bfloat16* p, const float* x) {
  uint4 r;
  __nv_bfloat162* v = reinterpret_cast<__nv_bfloat162*>(&r);
#pragma unroll
  for (int e = 0; e < 4; ++e) v[e] = __floats2bfloat162_rn(x[2 * e], x[2 * e + 1]);
  *reinterpret_cast<uint4*>(p) = r;
}
__device__ __forceinline__ void store8(__half* p, const float* x) {
  uint4 r;
  __half2* v = reinterpret_cast<__half2*>(&r);
#pragma unroll
  for (int e = 0; e < 4; ++e) v[e] = __floats2half2_rn(x[2 * e], x[2 * e + 1]);
  *reinterpret_cast<uint4*>(p) = r;
}
__device__ __forceinline__ void store8(float* p, const float* x) {
  *reinterpret_cast<float4*>(p) = make_float4(x[0], x[1], x[2], x[3]);
  *reinterpret_cast<float4*>(p + 4) = make_float4(x[4], x[5], x[6], x[7]);
}

// Copies [T][H] head rows between two layouts of the same D-column content: rows of src_row
// columns with the second half at column src_half, to rows of dst_row columns with the second
// half at dst_half; columns of the destination beyond the content are zeroed.  rotate = +1 / -1
// applies the rotation by +/- pos * theta^(-2i/D) to the pairs (i, i + D/2) on the way (fp32
// arithmetic, angles in fp64), 0 copies.  One thread per (token, 8 consecutive columns of a
// half), looping over the heads so that the angles are formed once.
template <typename SrcT, typename DstT>
__global__ void __launch_bounds__(128)
head_repack_kernel(const SrcT* __restrict__ src, int src_row, int src_half, DstT* __restrict__ dst,
                   int dst_row, int dst_half, const int32_t* __restrict__ pos, int T, int H, int D,
                   double log2_theta, int rotate) {
  const int chunks = dst_half / 8;                  // dst_half >= D/2 always
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)T * chunks) return;
  const int t = (int)(idx / chunks), i0 = (int)(idx % chunks) * 8;
  const bool content = i0 < D / 2;
  float c[8], s[8];
  if (content && rotate != 0) {
    const int p = pos[t];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const double inv_freq = exp2(-2.0 * (double)(i0 + e) / (double)D * log2_theta);
      double sd, cd;
      sincos((double)p * inv_freq, &sd, &cd);
      c[e] = (float)cd;
      s[e] = rotate > 0 ? (float)sd : -(float)sd;
    }
  }
  const SrcT* sr = src + (int64_t)t * H * src_row + i0;
  DstT* dr = dst + (int64_t)t * H * dst_row + i0;
  for (int h = 0; h < H; ++h) {
    float a[8], b[8];
    if (content) {
      load8(sr + (int64_t)h * src_row, a);
      load8(sr + (int64_t)h * src_row + src_half, b);
      if (rotate != 0) {
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const float x = a[e], y = b[e];
          a[e] = x * c[e] - y * s[e];
          b[e] = y * c[e] + x * s[e];
        }
      }
    } else {
#pragma unroll
      for (int e = 0; e < 8; ++e) a[e] = b[e] = 0.f;
    }
    store8(dr + (int64_t)h * dst_row, a);
    store8(dr + (int64_t)h * dst_row + dst_half, b);
  }
}

template <typename SrcT, typename DstT>
int repack(const void* src, int src_row, void* dst, int dst_row, const int32_t* pos, int T, int H,
           int D, float theta, int rotate, cudaStream_t stream) {
  const int dst_half = dst_row / 2;
  const int64_t n = (int64_t)T * (dst_half / 8);
  const unsigned blocks = (unsigned)((n + 127) / 128);
  head_repack_kernel<SrcT, DstT><<<blocks, 128, 0, stream>>>(
      static_cast<const SrcT*>(src), src_row, src_row / 2, static_cast<DstT*>(dst), dst_row,
      dst_half, pos, T, H, D, rotate != 0 ? log2((double)theta) : 0.0, rotate);
  return launch_status();
}

// caller's layout -> padded copy of the same element type (bf16 or fp32); rotate = 1: bf16 ->
// rotated fp16
int pad(const void* src, void* dst, int dtype, const int32_t* pos, int T, int H, int D, int P,
        float theta, int rotate, cudaStream_t stream) {
  if (rotate)
    return repack<__nv_bfloat16, __half>(src, D, dst, P, pos, T, H, D, theta, 1, stream);
  return dtype == PK_F32
             ? repack<float, float>(src, D, dst, P, pos, T, H, D, theta, 0, stream)
             : repack<__nv_bfloat16, __nv_bfloat16>(src, D, dst, P, pos, T, H, D, theta, 0, stream);
}

// padded result -> caller's layout, same element type
int unpad(const void* src, void* dst, int dtype, int T, int H, int D, int P, cudaStream_t stream) {
  return dtype == PK_F32
             ? repack<float, float>(src, P, dst, D, nullptr, T, H, D, 0.f, 0, stream)
             : repack<__nv_bfloat16, __nv_bfloat16>(src, P, dst, D, nullptr, T, H, D, 0.f, 0,
                                                    stream);
}

// The padded copies behind the sections of the padded-size layout.
struct PadBuffers {
  char *q, *dout, *out, *dq, *k, *v, *dk, *dv;
};
PadBuffers pad_buffers(char* ws, const WorkspaceLayout& lay, int64_t T, int64_t Hq, int64_t Hkv,
                       int64_t P) {
  const size_t Tn = (size_t)(T > 0 ? T : 1);
  const size_t per_q = align_up(Tn * (size_t)Hq * (size_t)P * 2, 256);
  const size_t per_kv = align_up(Tn * (size_t)Hkv * (size_t)P * 2, 256);
  PadBuffers b;
  char* cur = ws + lay.off_pad;
  b.q = cur;    cur += per_q;
  b.dout = cur; cur += per_q;
  b.out = cur;  cur += 2 * per_q;
  b.dq = cur;   cur += 2 * per_q;
  b.k = cur;    cur += per_kv;
  b.v = cur;    cur += per_kv;
  b.dk = cur;   cur += 2 * per_kv;
  b.dv = cur;
  return b;
}

}  // namespace

int attn_fwd_padded(const void* q, const void* k, const void* v, const int32_t* position_ids,
                    int32_t T, int32_t Hq, int32_t Hkv, int32_t D, float softmax_scale,
                    float rope_theta, int32_t window, void* out, int32_t out_dtype, float* lse,
                    int32_t reuse_plan, void* workspace, size_t workspace_bytes, void* stream_) {
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  (void)workspace_bytes;                         // checked by the caller
  const int P = padded_head_dim(D);
  const WorkspaceLayout lay = workspace_layout(T, Hq, Hkv, D);     // sections sized for P
  char* ws = static_cast<char*>(workspace);
  const PadBuffers b = pad_buffers(ws, lay, T, Hq, Hkv, P);
  const int rot = rope_theta > 0.f ? 1 : 0;
  int rc;
  if (!(reuse_plan & PK_REUSE_PLAN) &&
      (rc = plan_launch(position_ids, T, nullptr, nullptr, nullptr, workspace, lay, stream)) != PK_OK)
    return rc;
  if ((rc = pad(q, b.q, PK_BF16, position_ids, T, Hq, D, P, rope_theta, rot, stream)) != PK_OK ||
      (rc = pad(k, b.k, PK_BF16, position_ids, T, Hkv, D, P, rope_theta, rot, stream)) != PK_OK ||
      (rc = pad(v, b.v, PK_BF16, position_ids, T, Hkv, D, P, 0.f, 0, stream)) != PK_OK)
    return rc;
  CUtensorMap tq, tk, tv;
  if (!make_tile_map_bf16(&tq, b.q, T, Hq * P) || !make_tile_map_bf16(&tk, b.k, T, Hkv * P) ||
      !make_tile_map_bf16(&tv, b.v, T, Hkv * P))
    return PK_ERR_CUDA;
  rc = launch_fwd_ws(tq, tk, tv, ws, lay, b.out, lse, T, Hq, Hkv, P, out_dtype, softmax_scale,
                     window, rot != 0, stream);
  if (rc != PK_OK) return rc;
  return unpad(b.out, out, out_dtype, T, Hq, D, P, stream);
}

int attn_bwd_padded(const void* dout, const void* q, const void* k, const void* v, const void* out,
                    int32_t out_dtype, const float* lse, const int32_t* position_ids, int32_t T,
                    int32_t Hq, int32_t Hkv, int32_t D, float softmax_scale, float rope_theta,
                    int32_t window, void* dq, void* dk, void* dv, int32_t grad_dtype,
                    int32_t reuse_plan, void* workspace, size_t workspace_bytes, void* stream_) {
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  (void)workspace_bytes;
  const int P = padded_head_dim(D);
  const WorkspaceLayout lay = workspace_layout(T, Hq, Hkv, D);
  char* ws = static_cast<char*>(workspace);
  const PadBuffers b = pad_buffers(ws, lay, T, Hq, Hkv, P);
  const int rot = rope_theta > 0.f ? 1 : 0;
  int rc;
  if (!(reuse_plan & PK_REUSE_PLAN) &&
      (rc = plan_launch(position_ids, T, nullptr, nullptr, nullptr, workspace, lay, stream)) != PK_OK)
    return rc;
  // PK_REUSE_ROTATED: the forward's padded (and rotated) q, k, v are still in place
  if (!(reuse_plan & PK_REUSE_ROTATED)) {
    if ((rc = pad(q, b.q, PK_BF16, position_ids, T, Hq, D, P, rope_theta, rot, stream)) != PK_OK ||
        (rc = pad(k, b.k, PK_BF16, position_ids, T, Hkv, D, P, rope_theta, rot, stream)) != PK_OK ||
        (rc = pad(v, b.v, PK_BF16, position_ids, T, Hkv, D, P, 0.f, 0, stream)) != PK_OK)
      return rc;
  }
  if ((rc = pad(dout, b.dout, PK_BF16, position_ids, T, Hq, D, P, 0.f, 0, stream)) != PK_OK)
    return rc;
  // delta from the caller's own tensors (the pad columns would add nothing)
  float* delta = reinterpret_cast<float*>(ws + lay.off[PK_WS_DELTA]);
  if ((D & (D - 1)) == 0) {
    rc = delta_launch(dout, out, out_dtype, delta, T, Hq, D, stream);
  } else {   // the pre-pass wants a power-of-two row: give it the padded copies
    if ((rc = pad(out, b.out, out_dtype, position_ids, T, Hq, D, P, 0.f, 0, stream)) != PK_OK)
      return rc;
    rc = delta_launch(b.dout, b.out, out_dtype, delta, T, Hq, P, stream);
  }
  if (rc != PK_OK) return rc;
  if (rot && (rc = rope_angle_launch(position_ids, T, D, rope_theta,
                                     reinterpret_cast<float*>(ws + lay.off[PK_WS_ROPE_TABLE]),
                                     stream, P / 2)) != PK_OK)
    return rc;
  CUtensorMap tq, tk, tv, tdo;
  if (!make_tile_map_bf16(&tq, b.q, T, Hq * P) || !make_tile_map_bf16(&tk, b.k, T, Hkv * P) ||
      !make_tile_map_bf16(&tv, b.v, T, Hkv * P) || !make_tile_map_bf16(&tdo, b.dout, T, Hq * P))
    return PK_ERR_CUDA;
  rc = launch_bwd_ws(tq, tk, tv, tdo, ws, lay, lse, b.dq, b.dk, b.dv, T, Hq, Hkv, P, grad_dtype,
                     softmax_scale, window, rot != 0, stream);
  if (rc != PK_OK) return rc;
  if ((rc = unpad(b.dq, dq, grad_dtype, T, Hq, D, P, stream)) != PK_OK ||
      (rc = unpad(b.dk, dk, grad_dtype, T, Hkv, D, P, stream)) != PK_OK)
    return rc;
  return unpad(b.dv, dv, grad_dtype, T, Hkv, D, P, stream);
}

}  // namespace pk
