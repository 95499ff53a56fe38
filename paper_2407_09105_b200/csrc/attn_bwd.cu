// Backward of packed (block-diagonal causal) attention on sm_100a: the entry point pk_attn_bwd
// (bottom of the file), the row-sum pre-pass delta = sum_d dO*O, and the single-kernel backward
// with RoPE applied inside the tile.
//
// pk_attn_bwd plans (or reuses the plan), runs the pre-pass and then the two warp-specialised
// kernels of attn_bwd_ws.cu (dK/dV, then dQ; no reductions through memory): directly on q and k
// without RoPE, on rotated fp16 copies with it (the default RoPE mode).  Only the in-tile RoPE
// mode (pk_set_rope_mode) runs the main kernel of this file:
//
// It is key-tile stationary: one unit = (a block of <= 128 key rows of one example, one kv head); it
// walks the query tiles from the diagonal to the end of the example for each of the G query
// heads of the group, keeps dK and dV in tensor memory for the whole unit (fixed accumulation
// order, so their rows are bitwise reproducible) and sends each query tile's dQ contribution
// to an fp32 accumulator with vector reductions; a last pass scales, un-rotates and casts
// dQ.  Query tiles outside the example are never visited (Table 1, "Correct Cross-Attention").
//
// Per step, with the key rows on the tensor-memory lanes:
//   S^T = K Q^T, dP^T = V dO^T            (both operands from swizzled shared memory)
//   P^T = exp2(S^T*scale*log2e - lse*log2e), masked;  dS^T = P^T o (dP^T - delta)
//   dV += P^T dO                           (P^T read from tensor memory as bf16)
//   dK += dS^T Q,   dQ = dS K              (dS^T staged once in shared memory, read K-major
//                                           for dK and MN-major for dQ)
#include <cuda_bf16.h>

#include "attn_common.cuh"
#include "pk_common.cuh"
#include "sm100_ptx.cuh"
#include "tensor_map.cuh"

namespace pk {
namespace {

using namespace ptx;

constexpr int kBwdThreads = 128;
constexpr float kLog2e = 1.4426950408889634f;

// ------------------------------------------------------------------ delta pre-pass
// D/16 lanes per (token, head) row, 32 bytes of dO per lane; shuffles reduce inside the lane
// group (a warp covers 32*16/D rows).  HBM-bound: reads dO and O once.  With 256-bit loads it runs
// at 6.9 TB/s (c4: 2.07 GB in 0.30 ms) where 128-bit loads gave 4.3 TB/s; buffers that are only
// 16-byte aligned take two 128-bit loads instead.
__device__ __forceinline__ void ld_nc_v8(const void* p, uint32_t* v, bool aligned32) {
  if (aligned32) {
    asm volatile("ld.global.nc.L1::no_allocate.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]),
                   "=r"(v[6]), "=r"(v[7])
                 : "l"(p));
  } else {
    const uint4 a = __ldg(static_cast<const uint4*>(p)), b = __ldg(static_cast<const uint4*>(p) + 1);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
    v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
  }
}
template <typename OutT>
__global__ void delta_kernel(const __nv_bfloat16* __restrict__ dout, const OutT* __restrict__ out,
                             float* __restrict__ delta, int T, int Hq, int D, bool aligned32) {
  const int lanes_per_row = D >> 4;                       // 8 (D = 128), 4 (D = 64), ...
  const int rows_per_warp = 32 / lanes_per_row;
  const int lane = threadIdx.x & 31;
  const int64_t warp_id = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int64_t row = warp_id * rows_per_warp + lane / lanes_per_row;
  const int c = (lane % lanes_per_row) * 16;
  float acc = 0.f;
  if (row < (int64_t)T * Hq) {
    uint32_t a[8];
    ld_nc_v8(dout + row * D + c, a, aligned32);
    float y[16];
    if (sizeof(OutT) == 2) {
      uint32_t b[8];
      ld_nc_v8(out + row * D + c, b, aligned32);
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        y[2 * e] = __uint_as_float(b[e] << 16);
        y[2 * e + 1] = __uint_as_float(b[e] & 0xffff0000u);
      }
    } else {
      uint32_t b0[8], b1[8];
      ld_nc_v8(out + row * D + c, b0, aligned32);
      ld_nc_v8(out + row * D + c + 8, b1, aligned32);
#pragma unroll
      for (int e = 0; e < 8; ++e) { y[e] = __uint_as_float(b0[e]); y[8 + e] = __uint_as_float(b1[e]); }
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      acc = fmaf(__uint_as_float(a[e] << 16), y[2 * e], acc);
      acc = fmaf(__uint_as_float(a[e] & 0xffff0000u), y[2 * e + 1], acc);
    }
  }
  for (int o = lanes_per_row >> 1; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if ((lane % lanes_per_row) == 0 && row < (int64_t)T * Hq) {
    const int t = (int)(row / Hq), h = (int)(row % Hq);
    delta[(size_t)h * T + t] = acc;
  }
}

// ------------------------------------------------------------------ dQ finishing pass
template <typename GradT>
__device__ __forceinline__ void store_grad(GradT* p, float v);
template <>
__device__ __forceinline__ void store_grad<float>(float* p, float v) { *p = v; }
template <>
__device__ __forceinline__ void store_grad<__nv_bfloat16>(__nv_bfloat16* p, float v) {
  *p = __float2bfloat16_rn(v);
}

// dq = scale * acc, rotated back by -angle when RoPE was fused.  One thread per pair (i, i+D/2).
template <typename GradT>
__global__ void dq_finish_kernel(const float* __restrict__ acc, GradT* __restrict__ dq,
                                 const float2* __restrict__ table, int64_t n_pairs, int Hq, int D,
                                 float scale, int use_rope) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= n_pairs) return;
  const int half = D / 2;
  const int i = (int)(idx % half);
  const int64_t row = idx / half;          // token * Hq + head
  const int64_t base = row * D;
  float a = acc[base + i] * scale, b = acc[base + i + half] * scale;
  if (use_rope) {
    const float2 cs = table[(row / Hq) * half + i];
    const float a2 = a * cs.x + b * cs.y;
    const float b2 = b * cs.x - a * cs.y;
    a = a2; b = b2;
  }
  store_grad<GradT>(dq + base + i, a);
  store_grad<GradT>(dq + base + i + half, b);
}

// ------------------------------------------------------------------ main kernel
template <int D>
struct BwdSmem {
  static constexpr int kBoxBytes = 128 * 128;
  static constexpr int kBoxes = D / 64;
  static constexpr int kTileBytes = kBoxBytes * kBoxes;
  static constexpr int kK = 0;
  static constexpr int kV = kTileBytes;
  static constexpr int kQ = 2 * kTileBytes;
  static constexpr int kdO = 3 * kTileBytes;
  static constexpr int kdS = 4 * kTileBytes;               // always 2 boxes (128 q columns)
  static constexpr int kLse = kdS + 2 * kBoxBytes;         // 128 floats
  static constexpr int kDelta = kLse + 512;                // 128 floats
  static constexpr int kBars = kDelta + 512;
  static constexpr int kMisc = kBars + 32;
  static constexpr int kTotal = kMisc + 32;
  static constexpr int kDynamic = kTotal + 1024;
};

template <int D>
__device__ __forceinline__ void rope_tile_inplace_bwd(uint8_t* tile, const float2* __restrict__ table,
                                                      int first_token, int T, int tid) {
  constexpr int kHalfChunks = D / 16;
#pragma unroll 1
  for (int idx = tid; idx < 128 * kHalfChunks; idx += kBwdThreads) {
    const int row = idx / kHalfChunks, ch = idx % kHalfChunks;
    const int tok = first_token + row;
    if (tok >= T) continue;
    uint8_t *p1, *p2;
    if (D == 128) {
      const int off = row * 128 + ((ch ^ (row & 7)) << 4);
      p1 = tile + off;
      p2 = tile + BwdSmem<D>::kBoxBytes + off;
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
      const float4 c01 = __ldg(cs + e);
      const float2 x = __bfloat1622float2(av[e]);
      const float2 y = __bfloat1622float2(bv[e]);
      // rotated values stay fp16 (see the forward kernel)
      reinterpret_cast<uint32_t*>(&a)[e] =
          pack_f16x2(x.x * c01.x - y.x * c01.y, x.y * c01.z - y.y * c01.w);
      reinterpret_cast<uint32_t*>(&b)[e] =
          pack_f16x2(y.x * c01.x + x.x * c01.y, y.y * c01.z + x.y * c01.w);
    }
    *reinterpret_cast<uint4*>(p1) = a;
    *reinterpret_cast<uint4*>(p2) = b;
  }
}

template <int D, bool kRope, typename GradT>
__global__ void __launch_bounds__(kBwdThreads, 1)
attn_bwd_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_do,
                const int4* __restrict__ items, const int32_t* __restrict__ order, int32_t* hdr,
                const float* __restrict__ lse, const float* __restrict__ delta,
                float* __restrict__ dq_acc, GradT* __restrict__ dk, GradT* __restrict__ dv,
                const float2* __restrict__ rope_table, int T, int Hq, int Hkv, float scale,
                float scale_log2) {
  using L = BwdSmem<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>(
      (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  const uint32_t sbase = smem_u32(smem);
  const uint32_t sK = sbase + L::kK, sV = sbase + L::kV, sQ = sbase + L::kQ, sdO = sbase + L::kdO,
                 sdS = sbase + L::kdS;
  float* s_lse = reinterpret_cast<float*>(smem + L::kLse);
  float* s_delta = reinterpret_cast<float*>(smem + L::kDelta);
  const uint32_t bar_kv = sbase + L::kBars, bar_q = bar_kv + 8, bar_mma = bar_kv + 16;
  volatile int* s_tmem = reinterpret_cast<volatile int*>(smem + L::kMisc);
  volatile int* s_abort = s_tmem + 1;
  volatile int* s_unit = s_tmem + 2;

  const int tid = threadIdx.x, warp = tid >> 5;

  if (tid == 0) {
    mbar_init(bar_kv, 1);
    mbar_init(bar_q, 1);
    mbar_init(bar_mma, 1);
    fence_mbar_init();
    *s_abort = 0;
    prefetch_tensormap(&tm_q);
    prefetch_tensormap(&tm_k);
    prefetch_tensormap(&tm_v);
    prefetch_tensormap(&tm_do);
  }
  if (warp == 0) {
    tmem_alloc(smem_u32(const_cast<int*>(s_tmem)), 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = static_cast<uint32_t>(*s_tmem);
  const uint32_t tS = tmem;           // S^T fp32 [128 cols]; P^T bf16 reuses cols [0, 64)
  const uint32_t tdP = tmem + 128;    // dP^T fp32 [128 cols]; then dQ [D cols]
  const uint32_t tdV = tmem + 256;    // D cols
  const uint32_t tdK = tmem + 384;    // D cols
  const uint32_t lane_off = static_cast<uint32_t>(warp * 32) << 16;

  constexpr uint32_t kQKFmt = kRope ? kFmtF16 : kFmtBF16;   // rotated Q, K tiles are fp16
  constexpr uint32_t kIdescS = make_idesc(128, 128, kQKFmt, kQKFmt, 0, 0);      // K Q^T
  constexpr uint32_t kIdescDP = make_idesc(128, 128, kFmtBF16, kFmtBF16, 0, 0);  // V dO^T
  constexpr uint32_t kIdescDV = make_idesc(128, D, kFmtBF16, kFmtBF16, 0, 1);    // P^T dO
  // dS^T takes the format of the tiles it is multiplied with (fp16 when they were rotated)
  constexpr uint32_t kIdescDK = make_idesc(128, D, kQKFmt, kQKFmt, 0, 1);        // dS^T Q
  constexpr uint32_t kIdescDQ = make_idesc(128, D, kQKFmt, kQKFmt, 1, 1);        // dS K

  const int G = Hq / Hkv;
  const int n_items = (hdr[PK_HDR_PLAN_T] == T) ? hdr[PK_HDR_N_ITEMS] : 0;
  if (hdr[PK_HDR_PLAN_T] != T && blockIdx.x == 0 && tid == 0) set_status(hdr, PK_ERR_NO_PLAN, T);
  const int n_units = n_items * Hkv;
  const float lse_scale = kLog2e;

  uint32_t ph_kv = 0, ph_q = 0, ph_mma = 0;

  while (true) {
    if (tid == 0) *s_unit = atomicAdd(&hdr[kHdrBwdTicket], 1);
    __syncthreads();
    const int unit = *s_unit;
    const bool aborted = (*s_abort != 0);
    __syncthreads();
    if (unit >= n_units || aborted) break;

    const int4 it = items[order[unit / Hkv]];
    const int g = unit % Hkv;
    const int kv_start = it.x, kv_len = it.y, q_start = it.z, q_len = it.w;
    const int n_q = (q_len + kBM - 1) / kBM;

    if (tid == 0) {
      mbar_expect_tx(bar_kv, 2 * L::kTileBytes);
#pragma unroll
      for (int b = 0; b < L::kBoxes; ++b) {
        tma_load_2d(sK + b * L::kBoxBytes, &tm_k, g * D + b * 64, kv_start, bar_kv);
        tma_load_2d(sV + b * L::kBoxBytes, &tm_v, g * D + b * 64, kv_start, bar_kv);
      }
    }
    mbar_wait(bar_kv, ph_kv, s_abort);
    ph_kv ^= 1;
    if (kRope) rope_tile_inplace_bwd<D>(smem + L::kK, rope_table, kv_start, T, tid);

    bool first_step = true;
    for (int hh = 0; hh < G; ++hh) {
      const int h = g * G + hh;
      for (int i = 0; i < n_q; ++i) {
        const int q0 = q_start + i * kBM;
        if (tid == 0) {
          mbar_expect_tx(bar_q, 2 * L::kTileBytes);
#pragma unroll
          for (int b = 0; b < L::kBoxes; ++b) {
            tma_load_2d(sQ + b * L::kBoxBytes, &tm_q, h * D + b * 64, q0, bar_q);
            tma_load_2d(sdO + b * L::kBoxBytes, &tm_do, h * D + b * 64, q0, bar_q);
          }
        }
        {
          const int tok = q0 + tid;
          const bool in = tok < T;
          s_lse[tid] = in ? lse[(size_t)h * T + tok] * lse_scale : 0.f;
          s_delta[tid] = in ? delta[(size_t)h * T + tok] : 0.f;
        }
        mbar_wait(bar_q, ph_q, s_abort);
        ph_q ^= 1;
        if (kRope) rope_tile_inplace_bwd<D>(smem + L::kQ, rope_table, q0, T, tid);
        if (kRope) fence_proxy_async_smem();
        tc_fence_before();
        __syncthreads();

        // ---- S^T = K Q^T and dP^T = V dO^T ------------------------------------------
        if (tid == 0) {
          tc_fence_after();
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk) {
            const uint32_t off = (kk / 4) * L::kBoxBytes + (kk % 4) * 32;
            mma_ss(tS, smem_desc_sw128(sK + off, 16, 1024), smem_desc_sw128(sQ + off, 16, 1024),
                   kIdescS, kk > 0);
          }
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk) {
            const uint32_t off = (kk / 4) * L::kBoxBytes + (kk % 4) * 32;
            mma_ss(tdP, smem_desc_sw128(sV + off, 16, 1024), smem_desc_sw128(sdO + off, 16, 1024),
                   kIdescDP, kk > 0);
          }
          mma_commit(bar_mma);
        }
        mbar_wait(bar_mma, ph_mma, s_abort);
        ph_mma ^= 1;
        tc_fence_after();

        // ---- this thread owns key row `tid`; columns are the tile's query rows -------
        const int q_left = q_len - i * kBM;          // query rows of the tile inside the example
        const int col_min = (i == 0) ? tid : 0;      // causal: query index >= key index
        uint8_t* ds_row = smem + L::kdS + tid * 128;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint32_t s[32], dp[32];
          tmem_ld32(tS + lane_off + c * 32, s);
          tmem_ld32(tdP + lane_off + c * 32, dp);
          tmem_wait_ld();
          uint32_t pp[16], dd[16];
#pragma unroll
          for (int e = 0; e < 32; e += 2) {
            float p0, p1, d0, d1;
            {
              const int col = c * 32 + e;
              const bool ok = (col >= col_min) && (col < q_left);
              const float x = fast_exp2(fmaf(__uint_as_float(s[e]), scale_log2, -s_lse[col]));
              p0 = ok ? x : 0.f;
              d0 = p0 * (__uint_as_float(dp[e]) - s_delta[col]);
            }
            {
              const int col = c * 32 + e + 1;
              const bool ok = (col >= col_min) && (col < q_left);
              const float x = fast_exp2(fmaf(__uint_as_float(s[e + 1]), scale_log2, -s_lse[col]));
              p1 = ok ? x : 0.f;
              d1 = p1 * (__uint_as_float(dp[e + 1]) - s_delta[col]);
            }
            pp[e >> 1] = pack_bf16x2(p0, p1);
            dd[e >> 1] = kRope ? pack_f16x2(d0, d1) : pack_bf16x2(d0, d1);
          }
          tmem_st16(tS + lane_off + c * 16, pp);
          // dS^T row `tid`, query columns [32c, 32c+32): box c/2, chunks (c%2)*4 .. +3
          uint8_t* box = ds_row + (c >> 1) * L::kBoxBytes;
#pragma unroll
          for (int ch = 0; ch < 4; ++ch) {
            const int chunk = ((c & 1) * 4 + ch) ^ (tid & 7);
            *reinterpret_cast<uint4*>(box + (chunk << 4)) =
                make_uint4(dd[ch * 4], dd[ch * 4 + 1], dd[ch * 4 + 2], dd[ch * 4 + 3]);
          }
        }
        tmem_wait_st();
        fence_proxy_async_smem();
        tc_fence_before();
        __syncthreads();

        // ---- dV += P^T dO,  dK += dS^T Q,  dQ = dS K ---------------------------------
        if (tid == 0) {
          tc_fence_after();
          const uint32_t acc = first_step ? 0u : 1u;
#pragma unroll
          for (int kk = 0; kk < kBM / 16; ++kk)
            mma_ts(tdV, tS + kk * 8, smem_desc_sw128(sdO + kk * 2048, L::kBoxBytes, 1024),
                   kIdescDV, acc | (kk > 0));
#pragma unroll
          for (int kk = 0; kk < kBM / 16; ++kk) {
            const uint32_t off = (kk / 4) * L::kBoxBytes + (kk % 4) * 32;
            mma_ss(tdK, smem_desc_sw128(sdS + off, 16, 1024),
                   smem_desc_sw128(sQ + kk * 2048, L::kBoxBytes, 1024), kIdescDK, acc | (kk > 0));
          }
#pragma unroll
          for (int kk = 0; kk < kBN / 16; ++kk)
            mma_ss(tdP, smem_desc_sw128(sdS + kk * 2048, L::kBoxBytes, 1024),
                   smem_desc_sw128(sK + kk * 2048, L::kBoxBytes, 1024), kIdescDQ, kk > 0);
          mma_commit(bar_mma);
        }
        first_step = false;
        mbar_wait(bar_mma, ph_mma, s_abort);
        ph_mma ^= 1;
        tc_fence_after();

        // ---- dQ tile: this thread owns query row `tid` --------------------------------
        {
          const bool live = (tid < q_left) && (*s_abort == 0);
          float* dst = dq_acc + ((size_t)(q0 + tid) * Hq + h) * D;
#pragma unroll
          for (int c = 0; c < D / 32; ++c) {
            uint32_t x[32];
            tmem_ld32(tdP + lane_off + c * 32, x);
            tmem_wait_ld();
            if (live) {
#pragma unroll
              for (int e = 0; e < 32; e += 4)
                red_add_v4(dst + c * 32 + e, __uint_as_float(x[e]), __uint_as_float(x[e + 1]),
                           __uint_as_float(x[e + 2]), __uint_as_float(x[e + 3]));
            }
          }
        }
        tc_fence_before();
        __syncthreads();
      }
    }

    // ---- epilogue: dV and dK rows of this key block ------------------------------------
    {
      const bool live = (tid < kv_len) && (*s_abort == 0);
      const int tok = kv_start + tid;
      GradT* dv_row = dv + ((size_t)tok * Hkv + g) * D;
      GradT* dk_row = dk + ((size_t)tok * Hkv + g) * D;
#pragma unroll
      for (int c = 0; c < D / 32; ++c) {
        uint32_t x[32];
        float y[32];
        tmem_ld32(tdV + lane_off + c * 32, x);
        tmem_wait_ld();
#pragma unroll
        for (int e = 0; e < 32; ++e) y[e] = __uint_as_float(x[e]);
        if (live) store_chunk32<GradT>(dv_row + c * 32, y);
      }
      if (!kRope) {
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
          uint32_t x[32];
          float y[32];
          tmem_ld32(tdK + lane_off + c * 32, x);
          tmem_wait_ld();
#pragma unroll
          for (int e = 0; e < 32; ++e) y[e] = __uint_as_float(x[e]) * scale;
          if (live) store_chunk32<GradT>(dk_row + c * 32, y);
        }
      } else {
        // rotate back: pairs (i, i + D/2) sit in chunks c and c + D/64
#pragma unroll
        for (int c = 0; c < D / 64; ++c) {
          uint32_t x1[32], x2[32];
          float y1[32], y2[32];
          tmem_ld32(tdK + lane_off + c * 32, x1);
          tmem_ld32(tdK + lane_off + (c + D / 64) * 32, x2);
          tmem_wait_ld();
          if (live) {
            const float2* cs = rope_table + (size_t)tok * (D / 2) + c * 32;
#pragma unroll
            for (int e = 0; e < 32; ++e) {
              const float2 t = __ldg(cs + e);
              const float a = __uint_as_float(x1[e]) * scale, b = __uint_as_float(x2[e]) * scale;
              y1[e] = a * t.x + b * t.y;
              y2[e] = b * t.x - a * t.y;
            }
            store_chunk32<GradT>(dk_row + c * 32, y1);
            store_chunk32<GradT>(dk_row + (c + D / 64) * 32, y2);
          }
        }
      }
    }
    tc_fence_before();
  }

  if (*s_abort != 0 && tid == 0) set_status(hdr, PK_ERR_TIMEOUT, 2);
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, 512);
}

template <int D, bool kRope, typename GradT>
int launch_bwd(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
               const CUtensorMap& tdo, char* ws, const WorkspaceLayout& lay, const float* lse,
               void* dk, void* dv, int T, int Hq, int Hkv, float scale, cudaStream_t stream) {
  auto kern = attn_bwd_kernel<D, kRope, GradT>;
  const int smem_bytes = BwdSmem<D>::kDynamic;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes) !=
      cudaSuccess)
    return PK_ERR_CUDA;
  int32_t* hdr = reinterpret_cast<int32_t*>(ws + lay.off[PK_WS_HEADER]);
  if (cudaMemsetAsync(hdr + kHdrBwdTicket, 0, sizeof(int32_t), stream) != cudaSuccess)
    return PK_ERR_CUDA;
  TimedLaunch timed(PK_KERNEL_BWD, stream);
  kern<<<sm_count(), kBwdThreads, smem_bytes, stream>>>(
      tq, tk, tv, tdo, reinterpret_cast<const int4*>(ws + lay.off[PK_WS_BWD_ITEMS]),
      reinterpret_cast<const int32_t*>(ws + lay.off[PK_WS_BWD_ORDER]), hdr, lse,
      reinterpret_cast<const float*>(ws + lay.off[PK_WS_DELTA]),
      reinterpret_cast<float*>(ws + lay.off[PK_WS_DQ_ACC]), static_cast<GradT*>(dk),
      static_cast<GradT*>(dv), reinterpret_cast<const float2*>(ws + lay.off[PK_WS_ROPE_TABLE]), T,
      Hq, Hkv, scale, scale * kLog2e);
  return launch_status();
}

}  // namespace

int delta_launch(const void* dout, const void* out, int out_dtype, float* delta, int T, int Hq, int D,
                 cudaStream_t stream) {
  const int64_t rows = (int64_t)T * Hq;
  const int warps = 8;
  const int64_t rows_per_block = (int64_t)warps * (32 / (D >> 4));
  const unsigned blocks = (unsigned)((rows + rows_per_block - 1) / rows_per_block);
  // rows are multiples of 32 bytes (D >= 16), so the base addresses decide the alignment
  const bool aligned32 =
      ((reinterpret_cast<uintptr_t>(dout) | reinterpret_cast<uintptr_t>(out)) & 31u) == 0;
  TimedLaunch timed(PK_KERNEL_DELTA, stream);
  if (out_dtype == PK_BF16)
    delta_kernel<__nv_bfloat16><<<blocks, warps * 32, 0, stream>>>(
        static_cast<const __nv_bfloat16*>(dout), static_cast<const __nv_bfloat16*>(out), delta, T,
        Hq, D, aligned32);
  else
    delta_kernel<float><<<blocks, warps * 32, 0, stream>>>(
        static_cast<const __nv_bfloat16*>(dout), static_cast<const float*>(out), delta, T, Hq, D,
        aligned32);
  return launch_status();
}

}  // namespace pk

extern "C" int pk_attn_bwd(const void* dout, const void* q, const void* k, const void* v,
                           const void* out, int32_t out_dtype, const float* lse,
                           const int32_t* position_ids, int32_t T, int32_t Hq, int32_t Hkv,
                           int32_t D, float softmax_scale, float rope_theta, int32_t window,
                           void* dq, void* dk, void* dv, int32_t grad_dtype,
                           int32_t reuse_plan, void* workspace,
                           size_t workspace_bytes, void* stream_) {
  using namespace pk;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  if (T < 0 || Hq <= 0 || Hkv <= 0 || !(softmax_scale > 0.f) || window < 0)
    return PK_ERR_INVALID_ARG;
  if (!shape_supported(T, Hq, Hkv, D)) return PK_ERR_UNSUPPORTED;
  if (window > 0 && rope_theta > 0.f && g_rope_mode != PK_ROPE_ROTATED_COPIES)
    return PK_ERR_UNSUPPORTED;
  if ((out_dtype != PK_BF16 && out_dtype != PK_F32) ||
      (grad_dtype != PK_BF16 && grad_dtype != PK_F32))
    return PK_ERR_UNSUPPORTED;
  if (workspace == nullptr || (reinterpret_cast<uintptr_t>(workspace) & 255u) != 0)
    return PK_ERR_INVALID_ARG;
  const WorkspaceLayout lay = workspace_layout(T, Hq, Hkv, D);
  if (workspace_bytes < lay.total) return PK_ERR_WORKSPACE;
  if (T == 0) return PK_OK;
  if (!dout || !q || !k || !v || !out || !lse || !position_ids || !dq || !dk || !dv)
    return PK_ERR_INVALID_ARG;
  if (!aligned16(dout) || !aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out) ||
      !aligned16(dq) || !aligned16(dk) || !aligned16(dv))
    return PK_ERR_INVALID_ARG;
  if (D != padded_head_dim(D))
    return attn_bwd_padded(dout, q, k, v, out, out_dtype, lse, position_ids, T, Hq, Hkv, D,
                           softmax_scale, rope_theta, window, dq, dk, dv, grad_dtype, reuse_plan,
                           workspace, workspace_bytes, stream_);

  char* ws = static_cast<char*>(workspace);
  int rc;
  if (!(reuse_plan & PK_REUSE_PLAN)) {
    rc = plan_launch(position_ids, T, nullptr, nullptr, nullptr, workspace, lay, stream);
    if (rc != PK_OK) return rc;
  }
  const bool use_rope = rope_theta > 0.f;
  const bool rotated_copies = use_rope && g_rope_mode == PK_ROPE_ROTATED_COPIES;
  float* table = reinterpret_cast<float*>(ws + lay.off[PK_WS_ROPE_TABLE]);
  if (use_rope) {   // reduced angles for the warp-specialised kernels' epilogues, (cos, sin) in-tile
    rc = rotated_copies ? rope_angle_launch(position_ids, T, D, rope_theta, table, stream)
                        : rope_table_launch(position_ids, T, D, rope_theta, table, stream);
    if (rc != PK_OK) return rc;
  }
  float* delta = reinterpret_cast<float*>(ws + lay.off[PK_WS_DELTA]);
  float* dq_acc = reinterpret_cast<float*>(ws + lay.off[PK_WS_DQ_ACC]);

  // (1) delta pre-pass and a cleared dQ accumulator
  if ((rc = delta_launch(dout, out, out_dtype, delta, T, Hq, D, stream)) != PK_OK) return rc;
  // only the in-tile RoPE kernel accumulates dQ with reductions and needs a cleared buffer
  if (use_rope && !rotated_copies &&
      cudaMemsetAsync(dq_acc, 0, sizeof(float) * (size_t)T * Hq * D, stream) != cudaSuccess)
    return PK_ERR_CUDA;

  // (2) main kernel
  CUtensorMap tq, tk, tv, tdo;
  if (!make_tile_map_bf16(&tq, q, T, Hq * D) || !make_tile_map_bf16(&tk, k, T, Hkv * D) ||
      !make_tile_map_bf16(&tv, v, T, Hkv * D) || !make_tile_map_bf16(&tdo, dout, T, Hq * D))
    return PK_ERR_CUDA;
  if (rotated_copies) {
    // rotated fp16 copies of q and k in the dQ accumulator section (not needed otherwise here)
    char* qr = ws + lay.off[PK_WS_DQ_ACC];
    char* kr = qr + align_up((size_t)T * Hq * D * 2, 256);
    // PK_REUSE_ROTATED: the forward left exactly these copies there and the caller vouches that
    // nothing touched them
    const bool have_copies = (reuse_plan & PK_REUSE_ROTATED) != 0;
    if (!have_copies) {
      rc = rope_rotate_f16_launch(q, position_ids, T, Hq, D, rope_theta, qr, stream);
      if (rc != PK_OK) return rc;
      rc = rope_rotate_f16_launch(k, position_ids, T, Hkv, D, rope_theta, kr, stream);
      if (rc != PK_OK) return rc;
    }
    CUtensorMap tqr, tkr;
    if (!make_tile_map_bf16(&tqr, qr, T, Hq * D) || !make_tile_map_bf16(&tkr, kr, T, Hkv * D))
      return PK_ERR_CUDA;
    return launch_bwd_ws(tqr, tkr, tv, tdo, ws, lay, lse, dq, dk, dv, T, Hq, Hkv, D, grad_dtype,
                         softmax_scale, window, true, stream);
  }
  if (!use_rope) {
    // two warp-specialised kernels (dK/dV, then dQ); dQ is final, no finishing pass
    return launch_bwd_ws(tq, tk, tv, tdo, ws, lay, lse, dq, dk, dv, T, Hq, Hkv, D, grad_dtype,
                         softmax_scale, window, false, stream);
  } else {
#define PK_BWD(DD, RR, TT)                                                                      \
  rc = launch_bwd<DD, RR, TT>(tq, tk, tv, tdo, ws, lay, lse, dk, dv, T, Hq, Hkv, softmax_scale, \
                              stream)
  if (D == 128) {
    if (use_rope) {
      if (grad_dtype == PK_BF16) PK_BWD(128, true, __nv_bfloat16); else PK_BWD(128, true, float);
    } else {
      if (grad_dtype == PK_BF16) PK_BWD(128, false, __nv_bfloat16); else PK_BWD(128, false, float);
    }
  } else {
    if (use_rope) {
      if (grad_dtype == PK_BF16) PK_BWD(64, true, __nv_bfloat16); else PK_BWD(64, true, float);
    } else {
      if (grad_dtype == PK_BF16) PK_BWD(64, false, __nv_bfloat16); else PK_BWD(64, false, float);
    }
  }
#undef PK_BWD
  }
  if (rc != PK_OK) return rc;

  // (3) dQ: scale, rotate back, cast
  {
    const int64_t n_pairs = (int64_t)T * Hq * (D / 2);
    const int threads = 256;
    const unsigned blocks = (unsigned)((n_pairs + threads - 1) / threads);
    TimedLaunch timed(PK_KERNEL_DQ_FINISH, stream);
    if (grad_dtype == PK_BF16)
      dq_finish_kernel<__nv_bfloat16><<<blocks, threads, 0, stream>>>(
          dq_acc, static_cast<__nv_bfloat16*>(dq), reinterpret_cast<const float2*>(table), n_pairs,
          Hq, D, softmax_scale, use_rope ? 1 : 0);
    else
      dq_finish_kernel<float><<<blocks, threads, 0, stream>>>(
          dq_acc, static_cast<float*>(dq), reinterpret_cast<const float2*>(table), n_pairs, Hq, D,
          softmax_scale, use_rope ? 1 : 0);
  }
  return launch_status();
}
