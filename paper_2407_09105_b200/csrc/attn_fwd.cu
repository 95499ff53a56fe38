// Forward of packed (block-diagonal causal) attention on sm_100a: the entry point pk_attn_fwd
// (bottom of the file) and the single-tile kernel with RoPE applied inside the tile.
//
// pk_attn_fwd plans (or reuses the plan), then runs the warp-specialised two-tile kernel of
// attn_fwd_ws.cu: directly on q and k without RoPE, on rotated fp16 copies with it (the default
// RoPE mode).  Only the in-tile RoPE mode (pk_set_rope_mode) runs the kernel of this file:
//
// Work comes from the plan's forward list: one unit = (a block of <= 128 query rows of one
// example, one query head).  Only the key tiles between the example start and the block's
// last row are visited, so tiles outside an example's causal block are never touched
// (Table 1, "Correct Cross-Attention"; boundaries from position_ids, paragraph after
// Table 1).  Per key tile: TMA brings K and V into 128B-swizzled shared memory (Q once per
// unit), tcgen05.mma forms S = Q K^T in tensor memory, 128 threads (one per query row) run
// the online softmax in fp32 straight out of tensor memory, write P back to tensor memory
// as bf16, and a second tcgen05.mma accumulates O += P V with P read from tensor memory.
// The Q and K tiles are rotated in shared memory right after they land.
#include <cuda_bf16.h>

#include "pk_common.cuh"
#include "sm100_ptx.cuh"
#include "tensor_map.cuh"

namespace pk {
namespace {

using namespace ptx;

constexpr int kFwdThreads = 128;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

template <int D>
struct FwdSmem {
  static constexpr int kBoxBytes = 128 * 128;           // 128 rows x 64 bf16
  static constexpr int kBoxes = D / 64;
  static constexpr int kTileBytes = kBoxBytes * kBoxes;
  static constexpr int kQ = 0;
  static constexpr int kK = kTileBytes;
  static constexpr int kV = 2 * kTileBytes;
  static constexpr int kBars = 3 * kTileBytes;          // 3 mbarriers
  static constexpr int kMisc = kBars + 32;              // tmem address, abort flag, unit
  static constexpr int kTotal = kMisc + 32;
  static constexpr int kDynamic = kTotal + 1024;        // slack for 1024-byte alignment
};

// Rotate the rows of one 128-row tile held as kBoxes swizzled boxes: pairs (i, i + D/2).
template <int D>
__device__ __forceinline__ void rope_tile_inplace(uint8_t* tile, const float2* __restrict__ table,
                                                  int first_token, int T, int tid) {
  constexpr int kHalfChunks = D / 16;   // 16-byte chunks in half a row
#pragma unroll 1
  for (int idx = tid; idx < 128 * kHalfChunks; idx += kFwdThreads) {
    const int row = idx / kHalfChunks, ch = idx % kHalfChunks;
    const int tok = first_token + row;
    if (tok >= T) continue;
    uint8_t *p1, *p2;
    if (D == 128) {
      const int off = row * 128 + ((ch ^ (row & 7)) << 4);
      p1 = tile + off;
      p2 = tile + FwdSmem<D>::kBoxBytes + off;
    } else {
      p1 = tile + row * 128 + ((ch ^ (row & 7)) << 4);
      p2 = tile + row * 128 + (((ch + kHalfChunks) ^ (row & 7)) << 4);
    }
    uint4 a = *reinterpret_cast<uint4*>(p1);
    uint4 b = *reinterpret_cast<uint4*>(p2);
    const float4* cs = reinterpret_cast<const float4*>(table + (size_t)tok * (D / 2) + ch * 8);
    __nv_bfloat162* av = reinterpret_cast<__nv_bfloat162*>(&a);
    __nv_bfloat162* bv = reinterpret_cast<__nv_bfloat162*>(&b);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float4 c01 = __ldg(cs + e);     // (cos0, sin0, cos1, sin1)
      const float2 x = __bfloat1622float2(av[e]);
      const float2 y = __bfloat1622float2(bv[e]);
      // the rotated values are kept as fp16 (11-bit significand): the score contraction then
      // runs fp16 x fp16, which loses 8x less to rounding than re-rounding to bf16
      reinterpret_cast<uint32_t*>(&a)[e] =
          pack_f16x2(x.x * c01.x - y.x * c01.y, x.y * c01.z - y.y * c01.w);
      reinterpret_cast<uint32_t*>(&b)[e] =
          pack_f16x2(y.x * c01.x + x.x * c01.y, y.y * c01.z + x.y * c01.w);
    }
    *reinterpret_cast<uint4*>(p1) = a;
    *reinterpret_cast<uint4*>(p2) = b;
  }
}

template <typename OutT>
__device__ __forceinline__ void store_row32(OutT* dst, const uint32_t* r, float scale);

template <>
__device__ __forceinline__ void store_row32<float>(float* dst, const uint32_t* r, float scale) {
#pragma unroll
  for (int c = 0; c < 32; c += 4) {
    float4 o;
    o.x = __uint_as_float(r[c]) * scale;
    o.y = __uint_as_float(r[c + 1]) * scale;
    o.z = __uint_as_float(r[c + 2]) * scale;
    o.w = __uint_as_float(r[c + 3]) * scale;
    *reinterpret_cast<float4*>(dst + c) = o;
  }
}
template <>
__device__ __forceinline__ void store_row32<__nv_bfloat16>(__nv_bfloat16* dst, const uint32_t* r,
                                                           float scale) {
#pragma unroll
  for (int c = 0; c < 32; c += 8) {
    uint4 o;
    o.x = pack_bf16x2(__uint_as_float(r[c]) * scale, __uint_as_float(r[c + 1]) * scale);
    o.y = pack_bf16x2(__uint_as_float(r[c + 2]) * scale, __uint_as_float(r[c + 3]) * scale);
    o.z = pack_bf16x2(__uint_as_float(r[c + 4]) * scale, __uint_as_float(r[c + 5]) * scale);
    o.w = pack_bf16x2(__uint_as_float(r[c + 6]) * scale, __uint_as_float(r[c + 7]) * scale);
    *reinterpret_cast<uint4*>(dst + c) = o;
  }
}

template <int D, bool kRope, typename OutT>
__global__ void __launch_bounds__(kFwdThreads, 2)
attn_fwd_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                const __grid_constant__ CUtensorMap tm_v, const int4* __restrict__ items,
                const int32_t* __restrict__ order, int32_t* hdr, OutT* __restrict__ out,
                float* __restrict__ lse, const float2* __restrict__ rope_table, int T, int Hq,
                int Hkv, float scale_log2) {
  using L = FwdSmem<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  const uint32_t sbase = smem_u32(smem);
  const uint32_t sQ = sbase + L::kQ, sK = sbase + L::kK, sV = sbase + L::kV;
  const uint32_t bar_q = sbase + L::kBars, bar_kv = bar_q + 8, bar_mma = bar_q + 16;
  volatile int* s_tmem = reinterpret_cast<volatile int*>(smem + L::kMisc);
  volatile int* s_abort = s_tmem + 1;
  volatile int* s_unit = s_tmem + 2;

  const int tid = threadIdx.x, warp = tid >> 5;

  if (tid == 0) {
    mbar_init(bar_q, 1);
    mbar_init(bar_kv, 1);
    mbar_init(bar_mma, 1);
    fence_mbar_init();
    *s_abort = 0;
    prefetch_tensormap(&tm_q);
    prefetch_tensormap(&tm_k);
    prefetch_tensormap(&tm_v);
  }
  if (warp == 0) {
    tmem_alloc(smem_u32(const_cast<int*>(s_tmem)), 256);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = static_cast<uint32_t>(*s_tmem);
  const uint32_t tS = tmem;            // 128 fp32 columns; P (bf16) reuses the first 64
  const uint32_t tO = tmem + 128;      // D fp32 columns
  const uint32_t lane_off = static_cast<uint32_t>(warp * 32) << 16;

  constexpr uint32_t kQKFmt = kRope ? kFmtF16 : kFmtBF16;   // rotated tiles are fp16
  constexpr uint32_t kIdescQK = make_idesc(128, 128, kQKFmt, kQKFmt, 0, 0);
  constexpr uint32_t kIdescPV = make_idesc(128, D, kFmtBF16, kFmtBF16, 0, 1);

  const int G = Hq / Hkv;
  const int n_items = (hdr[PK_HDR_PLAN_T] == T) ? hdr[PK_HDR_N_ITEMS] : 0;
  if (hdr[PK_HDR_PLAN_T] != T && blockIdx.x == 0 && tid == 0) set_status(hdr, PK_ERR_NO_PLAN, T);
  const int n_units = n_items * Hq;

  uint32_t ph_q = 0, ph_kv = 0, ph_mma = 0;

  while (true) {
    if (tid == 0) *s_unit = atomicAdd(&hdr[kHdrFwdTicket], 1);
    __syncthreads();
    const int unit = *s_unit;
    const bool aborted = (*s_abort != 0);
    __syncthreads();
    if (unit >= n_units || aborted) break;

    const int4 it = items[order[unit / Hq]];
    const int h = unit % Hq, g = h / G;
    const int q_start = it.x, q_len = it.y, kv_start = it.z, kv_len = it.w;
    const int n_kv = (kv_len + kBN - 1) / kBN;

    if (tid == 0) {
      mbar_expect_tx(bar_q, L::kTileBytes);
#pragma unroll
      for (int b = 0; b < L::kBoxes; ++b)
        tma_load_2d(sQ + b * L::kBoxBytes, &tm_q, h * D + b * 64, q_start, bar_q);
    }

    float m_run = -INFINITY, l_run = 0.f;

    for (int j = 0; j < n_kv; ++j) {
      const int kv0 = kv_start + j * kBN;
      if (tid == 0) {
        mbar_expect_tx(bar_kv, 2 * L::kTileBytes);
#pragma unroll
        for (int b = 0; b < L::kBoxes; ++b) {
          tma_load_2d(sK + b * L::kBoxBytes, &tm_k, g * D + b * 64, kv0, bar_kv);
          tma_load_2d(sV + b * L::kBoxBytes, &tm_v, g * D + b * 64, kv0, bar_kv);
        }
      }
      if (j == 0) {
        mbar_wait(bar_q, ph_q, s_abort);
        ph_q ^= 1;
        if (kRope) rope_tile_inplace<D>(smem + L::kQ, rope_table, q_start, T, tid);
      }
      mbar_wait(bar_kv, ph_kv, s_abort);
      ph_kv ^= 1;
      if (kRope) {
        rope_tile_inplace<D>(smem + L::kK, rope_table, kv0, T, tid);
        fence_proxy_async_smem();
      }
      tc_fence_before();
      __syncthreads();

      // ---- S = Q K^T -------------------------------------------------------------
      if (tid == 0) {
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t off = (kk / 4) * L::kBoxBytes + (kk % 4) * 32;
          mma_ss(tS, smem_desc_sw128(sQ + off, 16, 1024), smem_desc_sw128(sK + off, 16, 1024),
                 kIdescQK, kk > 0);
        }
        mma_commit(bar_mma);
      }
      mbar_wait(bar_mma, ph_mma, s_abort);
      ph_mma ^= 1;
      tc_fence_after();

      // ---- online softmax: this thread owns query row `tid` ---------------------
      uint32_t s[128];
#pragma unroll
      for (int c = 0; c < 4; ++c) tmem_ld32(tS + lane_off + c * 32, s + c * 32);
      tmem_wait_ld();

      const bool diagonal = (j == n_kv - 1);
      float mx = -INFINITY;
#pragma unroll
      for (int c = 0; c < 128; ++c) {
        float x = __uint_as_float(s[c]);
        if (diagonal && c > tid) x = -INFINITY;
        s[c] = __float_as_uint(x);
        mx = fmaxf(mx, x);
      }
      const float m_new = fmaxf(m_run, mx * scale_log2);
      const float alpha = fast_exp2(m_run - m_new);   // 0 on the first tile
      float sum = 0.f;
      uint32_t p[64];
#pragma unroll
      for (int c = 0; c < 128; c += 2) {
        const float p0 = fast_exp2(fmaf(__uint_as_float(s[c]), scale_log2, -m_new));
        const float p1 = fast_exp2(fmaf(__uint_as_float(s[c + 1]), scale_log2, -m_new));
        sum += p0 + p1;
        p[c >> 1] = pack_bf16x2(p0, p1);
      }
      l_run = l_run * alpha + sum;
      const bool changed = (m_new > m_run);
      m_run = m_new;

      // rescale the running O only when some row of this warp moved its maximum
      if (j > 0 && __any_sync(0xffffffffu, changed)) {
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
          uint32_t o[32];
          tmem_ld32(tO + lane_off + c * 32, o);
          tmem_wait_ld();
#pragma unroll
          for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
          tmem_st32(tO + lane_off + c * 32, o);
        }
      }
      tmem_st32(tS + lane_off, p);
      tmem_st32(tS + lane_off + 32, p + 32);
      tmem_wait_st();
      tc_fence_before();
      __syncthreads();

      // ---- O += P V --------------------------------------------------------------
      if (tid == 0) {
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < kBN / 16; ++kk)
          mma_ts(tO, tS + kk * 8, smem_desc_sw128(sV + kk * 2048, L::kBoxBytes, 1024), kIdescPV,
                 (j > 0 || kk > 0));
        mma_commit(bar_mma);
      }
      mbar_wait(bar_mma, ph_mma, s_abort);
      ph_mma ^= 1;
      tc_fence_after();
    }

    // ---- epilogue: O / l and lse ------------------------------------------------------
    const bool live = (*s_abort == 0);
    const float inv_l = 1.f / l_run;
    if (tid < q_len && live) {
      lse[(size_t)h * T + q_start + tid] = (m_run + log2f(l_run)) * kLn2;
    }
    OutT* orow = out + ((size_t)(q_start + tid) * Hq + h) * D;
#pragma unroll
    for (int c = 0; c < D / 32; ++c) {
      uint32_t o[32];
      tmem_ld32(tO + lane_off + c * 32, o);
      tmem_wait_ld();
      if (tid < q_len && live) store_row32<OutT>(orow + c * 32, o, inv_l);
    }
    tc_fence_before();
  }

  if (*s_abort != 0 && tid == 0) set_status(hdr, PK_ERR_TIMEOUT, 1);
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, 256);
}

template <int D, bool kRope, typename OutT>
int launch_fwd(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, char* ws,
               const WorkspaceLayout& lay, void* out, float* lse, int T, int Hq, int Hkv,
               float scale, cudaStream_t stream) {
  auto kern = attn_fwd_kernel<D, kRope, OutT>;
  const int smem_bytes = FwdSmem<D>::kDynamic;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes) !=
      cudaSuccess)
    return PK_ERR_CUDA;
  int32_t* hdr = reinterpret_cast<int32_t*>(ws + lay.off[PK_WS_HEADER]);
  if (cudaMemsetAsync(hdr + kHdrFwdTicket, 0, sizeof(int32_t), stream) != cudaSuccess)
    return PK_ERR_CUDA;
  const int grid = 2 * sm_count();
  TimedLaunch timed(PK_KERNEL_FWD, stream);
  kern<<<grid, kFwdThreads, smem_bytes, stream>>>(
      tq, tk, tv, reinterpret_cast<const int4*>(ws + lay.off[PK_WS_FWD_ITEMS]),
      reinterpret_cast<const int32_t*>(ws + lay.off[PK_WS_FWD_ORDER]), hdr,
      static_cast<OutT*>(out), lse,
      reinterpret_cast<const float2*>(ws + lay.off[PK_WS_ROPE_TABLE]), T, Hq, Hkv,
      scale * kLog2e);
  return launch_status();
}

}  // namespace
}  // namespace pk

extern "C" int pk_attn_fwd(const void* q, const void* k, const void* v,
                           const int32_t* position_ids, int32_t T, int32_t Hq, int32_t Hkv,
                           int32_t D, float softmax_scale, float rope_theta, int32_t window,
                           void* out, int32_t out_dtype, float* lse, int32_t reuse_plan,
                           void* workspace,
                           size_t workspace_bytes, void* stream_) {
  using namespace pk;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  if (T < 0 || Hq <= 0 || Hkv <= 0 || !(softmax_scale > 0.f) || window < 0)
    return PK_ERR_INVALID_ARG;
  if (!shape_supported(T, Hq, Hkv, D)) return PK_ERR_UNSUPPORTED;
  // the sliding window lives in the warp-specialised kernels only
  if (window > 0 && rope_theta > 0.f && g_rope_mode != PK_ROPE_ROTATED_COPIES)
    return PK_ERR_UNSUPPORTED;
  if (out_dtype != PK_BF16 && out_dtype != PK_F32) return PK_ERR_UNSUPPORTED;
  if (workspace == nullptr || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0)
    return PK_ERR_INVALID_ARG;
  const WorkspaceLayout lay = workspace_layout(T, Hq, Hkv, D);
  if (workspace_bytes < lay.total) return PK_ERR_WORKSPACE;
  if (T == 0) return PK_OK;
  if (!q || !k || !v || !position_ids || !out || !lse) return PK_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out))
    return PK_ERR_INVALID_ARG;
  if (D != padded_head_dim(D))
    return attn_fwd_padded(q, k, v, position_ids, T, Hq, Hkv, D, softmax_scale, rope_theta, window,
                           out, out_dtype, lse, reuse_plan, workspace, workspace_bytes, stream_);

  char* ws = static_cast<char*>(workspace);
  if (!(reuse_plan & PK_REUSE_PLAN)) {
    int rc = plan_launch(position_ids, T, nullptr, nullptr, nullptr, workspace, lay, stream);
    if (rc != PK_OK) return rc;
  }
  const bool use_rope = rope_theta > 0.f;
  if (use_rope && g_rope_mode == PK_ROPE_ROTATED_COPIES) {
    // rotated fp16 copies of q and k in the (otherwise unused) dQ accumulator section
    char* qr = ws + lay.off[PK_WS_DQ_ACC];
    char* kr = qr + align_up((size_t)T * Hq * D * 2, 256);
    int rc = rope_rotate_f16_launch(q, position_ids, T, Hq, D, rope_theta, qr, stream);
    if (rc != PK_OK) return rc;
    rc = rope_rotate_f16_launch(k, position_ids, T, Hkv, D, rope_theta, kr, stream);
    if (rc != PK_OK) return rc;
    CUtensorMap tqr, tkr, tvv;
    if (!make_tile_map_bf16(&tqr, qr, T, Hq * D) || !make_tile_map_bf16(&tkr, kr, T, Hkv * D) ||
        !make_tile_map_bf16(&tvv, v, T, Hkv * D))
      return PK_ERR_CUDA;
    return launch_fwd_ws(tqr, tkr, tvv, ws, lay, out, lse, T, Hq, Hkv, D, out_dtype, softmax_scale,
                         window, true, stream);
  }
  if (use_rope) {
    int rc = rope_table_launch(position_ids, T, D, rope_theta,
                               reinterpret_cast<float*>(ws + lay.off[PK_WS_ROPE_TABLE]), stream);
    if (rc != PK_OK) return rc;
  }
  CUtensorMap tq, tk, tv;
  if (!make_tile_map_bf16(&tq, q, T, Hq * D) || !make_tile_map_bf16(&tk, k, T, Hkv * D) ||
      !make_tile_map_bf16(&tv, v, T, Hkv * D))
    return PK_ERR_CUDA;

  if (!use_rope)   // two tiles per CTA (two heads of a kv head, or two query blocks), warp-specialised
    return launch_fwd_ws(tq, tk, tv, ws, lay, out, lse, T, Hq, Hkv, D, out_dtype, softmax_scale,
                         window, false, stream);
#define PK_FWD(DD, RR, TT) \
  return launch_fwd<DD, RR, TT>(tq, tk, tv, ws, lay, out, lse, T, Hq, Hkv, softmax_scale, stream)
  if (D == 128) {
    if (use_rope) {
      if (out_dtype == PK_BF16) PK_FWD(128, true, __nv_bfloat16); else PK_FWD(128, true, float);
    } else {
      if (out_dtype == PK_BF16) PK_FWD(128, false, __nv_bfloat16); else PK_FWD(128, false, float);
    }
  } else {
    if (use_rope) {
      if (out_dtype == PK_BF16) PK_FWD(64, true, __nv_bfloat16); else PK_FWD(64, true, float);
    } else {
      if (out_dtype == PK_BF16) PK_FWD(64, false, __nv_bfloat16); else PK_FWD(64, false, float);
    }
  }
#undef PK_FWD
}
