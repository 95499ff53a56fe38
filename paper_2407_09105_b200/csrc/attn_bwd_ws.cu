// Warp-specialised backward kernels (no fused RoPE) for sm_100a.
//
// The backward is split into two kernels so that no gradient needs floating-point atomics
// (fp32 reductions into a dQ accumulator ran at about 2 TB/s here and took longer than all
// the tensor-core work together; a TMA reduce-add reached 2.7 TB/s, still not enough):
//
//   attn_bwd_dkv_kernel  key-block stationary, unit = (<=128 key rows of one example, kv head):
//       for each of the G query heads and each query tile from the diagonal to the example end
//         S^T = K Q^T, dP^T = V dO^T, P^T = exp2(..), dS^T = P^T o (dP^T - delta),
//         dV += P^T dO, dK += dS^T Q            (dK, dV stay in tensor memory for the unit)
//   attn_bwd_dq_kernel   query-block stationary, unit = (<=128 query rows of one example, q head):
//       for each key tile from the example start to the diagonal
//         S = Q K^T, dP = dO V^T, dS = P o (dP - delta), dQ += dS K   (dQ stays in tensor memory)
//
// Both recompute S and dP (7 contractions per tile pair instead of 5), both are bitwise
// reproducible, and both never visit a tile outside an example's causal block.
//
// Roles: 8 compute warps (lane = tensor-memory row; warp w works on columns [64*(w/4), +64) of
// the rows of lane quarter w%4; 16 warps of 32 columns measured slightly slower because they
// take issue slots from the warp that feeds the tensor pipe), one warp that walks the MMA
// schedule with one elected lane issuing every tcgen05.mma, one warp that drives TMA.
// Units are assigned statically: CTA c takes positions c, 2P-1-c, 2P+c, ... of the plan's
// longest-first order, so the roles enumerate the same sequence without talking to each other.
// Every wait is bounded; on expiry an abort flag makes all later waits return at once.
#include <cuda_bf16.h>

#include "attn_common.cuh"
#include "pk_common.cuh"
#include "sm100_ptx.cuh"
#include "tensor_map.cuh"

namespace pk {
namespace {

using namespace ptx;

#ifndef PK_BWD_COMPUTE_THREADS
#define PK_BWD_COMPUTE_THREADS 256
#endif
constexpr int kComputeThreads = PK_BWD_COMPUTE_THREADS;   // 256 or 512
constexpr int kNQ = kComputeThreads / 128;                // column groups per tile row
constexpr int kCW = 128 / kNQ;                            // columns per compute thread
constexpr int kWsThreads = kComputeThreads + 64;
constexpr int kMmaWarp = kComputeThreads / 32;
constexpr int kLoadWarp = kMmaWarp + 1;
static_assert(kNQ == 2, "the dK/dV kernel assigns two 32-column pieces per compute thread");
constexpr float kLog2eWs = 1.4426950408889634f;

// position in the longest-first order of the r-th unit of this CTA (snake over the rounds)
__device__ __forceinline__ int snake_unit(int r, int cta, int n_cta) {
  return r * n_cta + ((r & 1) ? (n_cta - 1 - cta) : cta);
}
__device__ __forceinline__ void compute_bar_sync() {
  asm volatile("bar.sync 1, %0;" ::"n"(kComputeThreads) : "memory");
}

// =========================================================================================
// dK / dV kernel
// =========================================================================================
template <int D>
struct DkvSmem {
  static constexpr int kBoxBytes = 128 * 128;
  static constexpr int kBoxes = D / 64;
  static constexpr int kTileBytes = kBoxBytes * kBoxes;
  static constexpr int kK = 0;
  static constexpr int kV = kTileBytes;
  static constexpr int kQ0 = 2 * kTileBytes;                 // stage s: Q at kQ0 + s*2*tile
  static constexpr int kStageBytes = 2 * kTileBytes;         // Q then dO
  static constexpr int kdS = kQ0 + 2 * kStageBytes;          // 2 boxes
  static constexpr int kLse = kdS + 2 * kBoxBytes;           // [2][128] floats
  static constexpr int kDelta = kLse + 1024;                 // [2][128] floats
  static constexpr int kBars = kDelta + 1024;
  static constexpr int kMisc = kBars + 16 * 8;
  static constexpr int kTotal = kMisc + 16;
};

enum DkvBar {
  kvKvFull = 0, kvKvEmpty, kvQFull0, kvQFull1, kvDoFull0, kvDoFull1, kvQdoEmpty0, kvQdoEmpty1,
  kvSFull, kvDpFull, kvPReady, kvPReadyA, kvDsReady, kvUnitDone, kvDkvRead, kvNumBars
};

template <int D, bool kRot, typename GradT>
__global__ void __launch_bounds__(kWsThreads, 1)
attn_bwd_dkv_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                    const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_do,
                    const int4* __restrict__ items, const int32_t* __restrict__ order, int32_t* hdr,
                    const float* __restrict__ lse, const float* __restrict__ delta,
                    GradT* __restrict__ dk, GradT* __restrict__ dv,
                    const float2* __restrict__ rope_table,
                    int T, int Hq, int Hkv, float scale, float scale_log2) {
  using L = DkvSmem<D>;
  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t sbase = smem_u32(smem);
  const uint32_t sK = sbase + L::kK, sV = sbase + L::kV, sdS = sbase + L::kdS;
  float* s_lse = reinterpret_cast<float*>(smem + L::kLse);
  float* s_delta = reinterpret_cast<float*>(smem + L::kDelta);
  const uint32_t bars = sbase + L::kBars;
  auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };
  volatile int* s_tmem = reinterpret_cast<volatile int*>(smem + L::kMisc);
  volatile int* s_abort = s_tmem + 1;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (tid == 0) {
    mbar_init(bar(kvKvFull), 1);
    mbar_init(bar(kvKvEmpty), 1);
    mbar_init(bar(kvQFull0), 33);
    mbar_init(bar(kvQFull1), 33);
    mbar_init(bar(kvDoFull0), 1);
    mbar_init(bar(kvDoFull1), 1);
    mbar_init(bar(kvQdoEmpty0), 1);
    mbar_init(bar(kvQdoEmpty1), 1);
    mbar_init(bar(kvSFull), 1);
    mbar_init(bar(kvDpFull), 1);
    mbar_init(bar(kvPReady), kComputeThreads);
    mbar_init(bar(kvPReadyA), kComputeThreads);
    mbar_init(bar(kvDsReady), kComputeThreads);
    mbar_init(bar(kvUnitDone), 1);
    mbar_init(bar(kvDkvRead), kComputeThreads);
    fence_mbar_init();
    *s_abort = ((sbase & 1023u) != 0) ? 1 : 0;   // swizzled tiles need a 1024-byte aligned base
  }
  if (warp == kMmaWarp) {
    tmem_alloc(smem_u32(const_cast<int*>(s_tmem)), 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = static_cast<uint32_t>(*s_tmem);
  const uint32_t tS = tmem, tdP = tmem + 128, tdV = tmem + 256, tdK = tmem + 384;

  const int G = Hq / Hkv;
  const bool plan_ok = (hdr[PK_HDR_PLAN_T] == T);
  if (!plan_ok && blockIdx.x == 0 && tid == 0) set_status(hdr, PK_ERR_NO_PLAN, T);
  const int n_units = plan_ok ? hdr[PK_HDR_N_ITEMS] * Hkv : 0;
  const int n_cta = gridDim.x, cta = blockIdx.x;

  if (warp == kLoadWarp) {
    // =============================== loader ===============================================
    if (lane == 0) {
      prefetch_tensormap(&tm_q);
      prefetch_tensormap(&tm_k);
      prefetch_tensormap(&tm_v);
      prefetch_tensormap(&tm_do);
    }
    int gs = 0, uc = 0;
    for (int r = 0;; ++r, ++uc) {
      const int u = snake_unit(r, cta, n_cta);
      if (u >= n_units || *s_abort) break;
      const int4 it = items[order[u / Hkv]];
      const int g = u % Hkv;
      const int kv_start = it.x, q_start = it.z, q_len = it.w;
      const int n_q = (q_len + kBM - 1) / kBM;
      mbar_wait(bar(kvKvEmpty), (uc & 1) ^ 1, s_abort);
      if (lane == 0) {
        mbar_expect_tx(bar(kvKvFull), 2 * L::kTileBytes);
#pragma unroll
        for (int b = 0; b < L::kBoxes; ++b) {
          tma_load_2d(sK + b * L::kBoxBytes, &tm_k, g * D + b * 64, kv_start, bar(kvKvFull));
          tma_load_2d(sV + b * L::kBoxBytes, &tm_v, g * D + b * 64, kv_start, bar(kvKvFull));
        }
      }
      for (int hh = 0; hh < G; ++hh) {
        const int h = g * G + hh;
        for (int i = 0; i < n_q; ++i, ++gs) {
          const int st = gs & 1;
          const int q0 = q_start + i * kBM;
          mbar_wait(bar(kvQdoEmpty0 + st), ((gs >> 1) & 1) ^ 1, s_abort);
          const uint32_t sQ = sbase + L::kQ0 + st * L::kStageBytes, sdO = sQ + L::kTileBytes;
          if (lane == 0) {
            mbar_expect_tx(bar(kvQFull0 + st), L::kTileBytes);
#pragma unroll
            for (int b = 0; b < L::kBoxes; ++b)
              tma_load_2d(sQ + b * L::kBoxBytes, &tm_q, h * D + b * 64, q0, bar(kvQFull0 + st));
            mbar_expect_tx(bar(kvDoFull0 + st), L::kTileBytes);
#pragma unroll
            for (int b = 0; b < L::kBoxes; ++b)
              tma_load_2d(sdO + b * L::kBoxBytes, &tm_do, h * D + b * 64, q0, bar(kvDoFull0 + st));
          }
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int row = lane * 4 + e, tok = q0 + row;
            const bool in = tok < T;
            s_lse[st * 128 + row] = in ? lse[(size_t)h * T + tok] * kLog2eWs : 0.f;
            s_delta[st * 128 + row] = in ? delta[(size_t)h * T + tok] : 0.f;
          }
          mbar_arrive(bar(kvQFull0 + st));
        }
      }
    }
  } else if (warp == kMmaWarp) {
    // =============================== MMA issuer ===========================================
    // The whole warp walks the schedule (so that addresses and descriptors stay warp-uniform);
    // one elected lane issues the tensor-core instructions.
    {
      // kRot: q and k are the rotated fp16 copies; dS then follows their format (operands of one
      // contraction must share a format), everything touching V, dO and P stays bf16
      constexpr uint32_t kQKFmt = kRot ? kFmtF16 : kFmtBF16;
      constexpr uint32_t kIdescS = make_idesc(128, 128, kQKFmt, kQKFmt, 0, 0);
      constexpr uint32_t kIdescDP = make_idesc(128, 128, kFmtBF16, kFmtBF16, 0, 0);
      constexpr uint32_t kIdescDV = make_idesc(128, D, kFmtBF16, kFmtBF16, 0, 1);
      constexpr uint32_t kIdescDK = make_idesc(128, D, kQKFmt, kQKFmt, 0, 1);
      const bool leader = elect_one();
      const uint32_t k_lo = desc_lo(sK, 16), v_lo = desc_lo(sV, 16), ds_lo = desc_lo(sdS, 16);
      int gs = 0, uc = 0;
      auto issue_s = [&](int st) {
        const uint32_t q_lo = desc_lo(sbase + L::kQ0 + st * L::kStageBytes, 16);
        if (leader) {
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk) {
            const uint32_t off = ((kk / 4) * L::kBoxBytes + (kk % 4) * 32) >> 4;
            mma_ss(tS, desc_from_lo(k_lo + off), desc_from_lo(q_lo + off), kIdescS, kk > 0);
          }
          mma_commit(bar(kvSFull));
        }
        __syncwarp();
      };
      auto issue_dp = [&](int st) {
        const uint32_t do_lo = desc_lo(sbase + L::kQ0 + st * L::kStageBytes + L::kTileBytes, 16);
        if (leader) {
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk) {
            const uint32_t off = ((kk / 4) * L::kBoxBytes + (kk % 4) * 32) >> 4;
            mma_ss(tdP, desc_from_lo(v_lo + off), desc_from_lo(do_lo + off), kIdescDP, kk > 0);
          }
          mma_commit(bar(kvDpFull));
        }
        __syncwarp();
      };
      for (int r = 0;; ++r, ++uc) {
        const int u = snake_unit(r, cta, n_cta);
        if (u >= n_units || *s_abort) break;
        const int4 it = items[order[u / Hkv]];
        const int n_q = (it.w + kBM - 1) / kBM;
        const int n_steps = G * n_q;
        mbar_wait(bar(kvKvFull), uc & 1, s_abort);
        // prologue: S(0), dP(0).  The compute warps finished reading S and dP of the previous
        // unit's last step before they signalled its dS, which the last dK waited for.
        mbar_wait(bar(kvQFull0 + (gs & 1)), (gs >> 1) & 1, s_abort);
        tc_fence_after();
        issue_s(gs & 1);
        mbar_wait(bar(kvDoFull0 + (gs & 1)), (gs >> 1) & 1, s_abort);
        tc_fence_after();
        issue_dp(gs & 1);
        for (int s = 0; s < n_steps; ++s, ++gs) {
          const int st = gs & 1;
          const uint32_t stage = sbase + L::kQ0 + st * L::kStageBytes;
          const uint32_t qT_lo = desc_lo(stage, L::kBoxBytes);                      // Q, MN-major
          const uint32_t doT_lo = desc_lo(stage + L::kTileBytes, L::kBoxBytes);     // dO, MN-major
          const uint32_t acc = s > 0 ? 1u : 0u;
          mbar_wait(bar(kvPReadyA), gs & 1, s_abort);   // first 64 query columns of P
          if (s == 0 && uc > 0) mbar_wait(bar(kvDkvRead), (uc - 1) & 1, s_abort);
          tc_fence_after();
          if (leader) {
#pragma unroll
            for (int kk = 0; kk < kBM / 32; ++kk)   // dV += P^T dO, first half of the query rows
              mma_ts(tdV, tS + kk * 8, desc_from_lo(doT_lo + ((kk * 2048) >> 4)), kIdescDV,
                     acc | (kk > 0));
          }
          __syncwarp();
          mbar_wait(bar(kvPReady), gs & 1, s_abort);    // second half
          tc_fence_after();
          if (leader) {
#pragma unroll
            for (int kk = kBM / 32; kk < kBM / 16; ++kk)
              mma_ts(tdV, tS + kk * 8, desc_from_lo(doT_lo + ((kk * 2048) >> 4)), kIdescDV, 1u);
          }
          __syncwarp();
          const bool more = (s + 1 < n_steps);
          const int g1 = gs + 1;
          if (more) {                              // S(s+1): P(s) was consumed by dV(s) above
            mbar_wait(bar(kvQFull0 + (g1 & 1)), (g1 >> 1) & 1, s_abort);
            tc_fence_after();
            issue_s(g1 & 1);
          }
          mbar_wait(bar(kvDsReady), gs & 1, s_abort);
          tc_fence_after();
          if (leader) {
#pragma unroll
            for (int kk = 0; kk < kBM / 16; ++kk) {   // dK += dS^T Q
              const uint32_t off = ((kk / 4) * L::kBoxBytes + (kk % 4) * 32) >> 4;
              mma_ss(tdK, desc_from_lo(ds_lo + off), desc_from_lo(qT_lo + ((kk * 2048) >> 4)),
                     kIdescDK, acc | (kk > 0));
            }
            mma_commit(bar(kvQdoEmpty0 + st));
          }
          __syncwarp();
          if (more) {                              // dP(s+1): dP(s) was read before dS(s) was signalled
            mbar_wait(bar(kvDoFull0 + (g1 & 1)), (g1 >> 1) & 1, s_abort);
            tc_fence_after();
            issue_dp(g1 & 1);
          }
        }
        if (leader) {
          mma_commit(bar(kvUnitDone));
          mma_commit(bar(kvKvEmpty));
        }
        __syncwarp();
      }
    }
  } else {
    // =============================== compute ===============================================
    const int row = tid & 127;              // key row inside the block
    const int qd = tid >> 7;                // which group of kCW query columns
    const uint32_t lane_off = static_cast<uint32_t>((warp & 3) * 32) << 16;
    int gs = 0, uc = 0;
    for (int r = 0;; ++r, ++uc) {
      const int u = snake_unit(r, cta, n_cta);
      if (u >= n_units || *s_abort) break;
      const int4 it = items[order[u / Hkv]];
      const int g = u % Hkv;
      const int kv_start = it.x, kv_len = it.y, q_len = it.w;
      const int n_q = (q_len + kBM - 1) / kBM;
      for (int hh = 0; hh < G; ++hh) {
        for (int i = 0; i < n_q; ++i, ++gs) {
          const int st = gs & 1;
          const int q_left = q_len - i * kBM;
          const int col_min = (i == 0) ? row : 0;
          // This thread's 64 query columns are taken in two pieces, [32*qd, +32) of the first 64
          // and of the second 64, so that all warps finish the first half of P together and dV
          // can start on it while the second half is still being exponentiated.
          const int col_a = qd * 32, col_b = 64 + qd * 32;
          mbar_wait(bar(kvQFull0 + st), (gs >> 1) & 1, s_abort);   // lse / delta rows visible
          mbar_wait(bar(kvSFull), gs & 1, s_abort);
          tc_fence_after();
          float p[64];
          uint32_t sv[64];
          tmem_ld32(tS + lane_off + col_a, sv);
          tmem_ld32(tS + lane_off + col_b, sv + 32);
          tmem_wait_ld();
          const bool edge = (i == 0 || q_left < kBM);   // diagonal tile or last, partial tile
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            const int col0 = half == 0 ? col_a : col_b;
            const float4* lse4 = reinterpret_cast<const float4*>(s_lse + st * 128 + col0);
#pragma unroll
            for (int c = 0; c < 32; c += 4) {
              const float4 l4 = lse4[c >> 2];
              const int k = half * 32 + c;
              p[k] = fast_exp2(fmaf(__uint_as_float(sv[k]), scale_log2, -l4.x));
              p[k + 1] = fast_exp2(fmaf(__uint_as_float(sv[k + 1]), scale_log2, -l4.y));
              p[k + 2] = fast_exp2(fmaf(__uint_as_float(sv[k + 2]), scale_log2, -l4.z));
              p[k + 3] = fast_exp2(fmaf(__uint_as_float(sv[k + 3]), scale_log2, -l4.w));
            }
            if (edge) {   // interior tiles skip the compares
#pragma unroll
              for (int c = 0; c < 32; ++c) {
                const int col = col0 + c;
                if (!((col >= col_min) && (col < q_left))) p[half * 32 + c] = 0.f;
              }
            }
            if (half == 0) {   // every thread has loaded S: P may overwrite its columns
              tc_fence_before();
              compute_bar_sync();
              tc_fence_after();
            }
            uint32_t pp[16];
#pragma unroll
            for (int c = 0; c < 16; ++c) pp[c] = pack_bf16x2(p[half * 32 + 2 * c], p[half * 32 + 2 * c + 1]);
            tmem_st16(tS + lane_off + half * 32 + qd * 16, pp);
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(bar(half == 0 ? kvPReadyA : kvPReady));
          }

          mbar_wait(bar(kvDpFull), gs & 1, s_abort);
          tc_fence_after();
#pragma unroll
          for (int c2 = 0; c2 < 2; ++c2) {
            const int col0 = c2 == 0 ? col_a : col_b;
            // dS^T row `row`, query columns [col0, +32): box c2, 16-byte chunks 4*qd .. 4*qd+3
            uint8_t* ds_row = smem + L::kdS + c2 * L::kBoxBytes + row * 128;
            const float4* dl4 = reinterpret_cast<const float4*>(s_delta + st * 128 + col0);
            uint32_t dp[32], dd[16];
            tmem_ld32(tdP + lane_off + col0, dp);
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < 32; e += 4) {
              const float4 d4 = dl4[e >> 2];
              const float d0 = p[c2 * 32 + e] * (__uint_as_float(dp[e]) - d4.x);
              const float d1 = p[c2 * 32 + e + 1] * (__uint_as_float(dp[e + 1]) - d4.y);
              const float d2 = p[c2 * 32 + e + 2] * (__uint_as_float(dp[e + 2]) - d4.z);
              const float d3 = p[c2 * 32 + e + 3] * (__uint_as_float(dp[e + 3]) - d4.w);
              dd[e >> 1] = kRot ? pack_f16x2(d0, d1) : pack_bf16x2(d0, d1);
              dd[(e >> 1) + 1] = kRot ? pack_f16x2(d2, d3) : pack_bf16x2(d2, d3);
            }
#pragma unroll
            for (int ch = 0; ch < 4; ++ch) {
              const int chunk = (qd * 4 + ch) ^ (row & 7);
              *reinterpret_cast<uint4*>(ds_row + (chunk << 4)) =
                  make_uint4(dd[ch * 4], dd[ch * 4 + 1], dd[ch * 4 + 2], dd[ch * 4 + 3]);
            }
          }
          fence_proxy_async_smem();
          tc_fence_before();
          mbar_arrive(bar(kvDsReady));
        }
      }
      // ---- unit epilogue: the first half of the column groups writes dV, the second dK ------
      mbar_wait(bar(kvUnitDone), uc & 1, s_abort);
      tc_fence_after();
      {
        constexpr int kHalfGroups = kNQ / 2;               // groups per output tensor
        constexpr int kEpiCols = D / kHalfGroups;          // columns each thread writes
        const bool is_dv = qd < kHalfGroups;
        const int col0 = (qd % kHalfGroups) * kEpiCols;
        const bool live = (row < kv_len) && (*s_abort == 0);
        const int tok = kv_start + row;
        GradT* dst = (is_dv ? dv : dk) + ((size_t)tok * Hkv + g) * D + col0;
        const uint32_t src = (is_dv ? tdV : tdK) + lane_off + col0;
        const float mul = is_dv ? 1.f : scale;
        if (kRot && !is_dv) {
          // dK was formed against the rotated k: rotate back by -angle, pairs (i, i + D/2)
          static_assert(!kRot || (D == 128 && kEpiCols == 128), "rotated path is built for D = 128");
#pragma unroll
          for (int c = 0; c < 2; ++c) {
            uint32_t x1[32], x2[32];
            float y1[32], y2[32];
            tmem_ld32(src + c * 32, x1);
            tmem_ld32(src + 64 + c * 32, x2);
            tmem_wait_ld();
            if (live) {
              const float2* cs = rope_table + (size_t)tok * (D / 2) + c * 32;
#pragma unroll
              for (int e = 0; e < 32; ++e) {
                const float2 t = __ldg(cs + e);
                const float a = __uint_as_float(x1[e]) * mul, b = __uint_as_float(x2[e]) * mul;
                y1[e] = a * t.x + b * t.y;
                y2[e] = b * t.x - a * t.y;
              }
              store_chunk32<GradT>(dst + c * 32, y1);
              store_chunk32<GradT>(dst + 64 + c * 32, y2);
            }
          }
        } else {
#pragma unroll
          for (int c = 0; c < kEpiCols / 32; ++c) {
            uint32_t x[32];
            float y[32];
            tmem_ld32(src + c * 32, x);
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < 32; ++e) y[e] = __uint_as_float(x[e]) * mul;
            if (live) store_chunk32<GradT>(dst + c * 32, y);
          }
        }
      }
      tc_fence_before();
      mbar_arrive(bar(kvDkvRead));
    }
  }

  tc_fence_before();
  __syncthreads();
  if (*s_abort != 0 && tid == 0) set_status(hdr, PK_ERR_TIMEOUT, 3);
  if (warp == kMmaWarp) tmem_dealloc(tmem, 512);
}

// =========================================================================================
// dQ kernel
// =========================================================================================
template <int D>
struct DqSmem {
  static constexpr int kBoxBytes = 128 * 128;
  static constexpr int kBoxes = D / 64;
  static constexpr int kTileBytes = kBoxBytes * kBoxes;
  static constexpr int kQ = 0;
  static constexpr int kdO = kTileBytes;
  // K tiles live from S(j) to dQ(j), V tiles only for dP(j): separate rings, K one stage
  // deeper, so that the loads run two steps ahead of the contractions
  static constexpr int kKStages = 3;
  static constexpr int kVStages = 2;
  static constexpr int kK0 = 2 * kTileBytes;
  static constexpr int kV0 = kK0 + kKStages * kTileBytes;
  static constexpr int kBars = kV0 + kVStages * kTileBytes;
  static constexpr int kMisc = kBars + 24 * 8;
  static constexpr int kTotal = kMisc + 16;
};

enum DqBar {
  dqQFull = 0, dqQEmpty, dqQtReady, dqKFull0, dqKFull1, dqKFull2, dqKEmpty0, dqKEmpty1, dqKEmpty2,
  dqVFull0, dqVFull1, dqVEmpty0, dqVEmpty1, dqSFull, dqSRead, dqDpFull, dqDsReady, dqDone, dqRead,
  dqNumBars
};

// The query-side tiles Q and dO are the stationary A operands of S = Q K^T and dP = dO V^T.
// They are copied once per unit from shared memory into tensor memory, so that those two
// contractions read only K / V from shared memory (the shared-memory port, not the tensor
// pipe, was the bound when all four operands came from there).
template <int D, bool kRot, typename GradT>
__global__ void __launch_bounds__(kWsThreads, 1)
attn_bwd_dq_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                   const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_do,
                   const int4* __restrict__ items, const int32_t* __restrict__ order, int32_t* hdr,
                   const float* __restrict__ lse, const float* __restrict__ delta,
                   GradT* __restrict__ dq, const float2* __restrict__ rope_table, int T, int Hq,
                   int Hkv, float scale, float scale_log2) {
  using L = DqSmem<D>;
  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t sbase = smem_u32(smem);
  const uint32_t bars = sbase + L::kBars;
  auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };
  volatile int* s_tmem = reinterpret_cast<volatile int*>(smem + L::kMisc);
  volatile int* s_abort = s_tmem + 1;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (tid == 0) {
    mbar_init(bar(dqQFull), 1);
    mbar_init(bar(dqQEmpty), kComputeThreads);
    mbar_init(bar(dqQtReady), kComputeThreads);
    for (int i = dqKFull0; i <= dqVEmpty1; ++i) mbar_init(bar(i), 1);
    mbar_init(bar(dqSFull), 1);
    mbar_init(bar(dqSRead), kComputeThreads);
    mbar_init(bar(dqDpFull), 1);
    mbar_init(bar(dqDsReady), kComputeThreads);
    mbar_init(bar(dqDone), 1);
    mbar_init(bar(dqRead), kComputeThreads);
    fence_mbar_init();
    *s_abort = ((sbase & 1023u) != 0) ? 1 : 0;
  }
  if (warp == kMmaWarp) {
    tmem_alloc(smem_u32(const_cast<int*>(s_tmem)), 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = static_cast<uint32_t>(*s_tmem);
  // [0,128) S, [128,256) dP (dS as bf16 reuses its first 64 columns), [256,256+D) dQ,
  // [384,384+D/2) Q as bf16 pairs, then D/2 columns of dO
  const uint32_t tS = tmem, tdP = tmem + 128, tdQ = tmem + 256, tQ = tmem + 384,
                 tdO = tmem + 384 + D / 2;

  const int G = Hq / Hkv;
  const bool plan_ok = (hdr[PK_HDR_PLAN_T] == T);
  const int n_units = plan_ok ? hdr[PK_HDR_N_ITEMS] * Hq : 0;
  const int n_cta = gridDim.x, cta = blockIdx.x;

  if (warp == kLoadWarp) {
    // =============================== loader ===============================================
    if (lane == 0) {
      prefetch_tensormap(&tm_q);
      prefetch_tensormap(&tm_k);
      prefetch_tensormap(&tm_v);
      prefetch_tensormap(&tm_do);
      int gk = 0, uc = 0;
      for (int r = 0;; ++r, ++uc) {
        const int u = snake_unit(r, cta, n_cta);
        if (u >= n_units || *s_abort) break;
        const int4 it = items[order[u / Hq]];
        const int h = u % Hq, g = h / G;
        const int q_start = it.x, kv_start = it.z, kv_len = it.w;
        const int n_kv = (kv_len + kBN - 1) / kBN;
        mbar_wait(bar(dqQEmpty), (uc & 1) ^ 1, s_abort);
        mbar_expect_tx(bar(dqQFull), 2 * L::kTileBytes);
#pragma unroll
        for (int b = 0; b < L::kBoxes; ++b) {
          tma_load_2d(sbase + L::kQ + b * L::kBoxBytes, &tm_q, h * D + b * 64, q_start, bar(dqQFull));
          tma_load_2d(sbase + L::kdO + b * L::kBoxBytes, &tm_do, h * D + b * 64, q_start, bar(dqQFull));
        }
        for (int j = 0; j < n_kv; ++j, ++gk) {
          const int ks = gk % L::kKStages, vs = gk % L::kVStages;
          const uint32_t sK = sbase + L::kK0 + ks * L::kTileBytes;
          const uint32_t sV = sbase + L::kV0 + vs * L::kTileBytes;
          mbar_wait(bar(dqKEmpty0 + ks), ((gk / L::kKStages) & 1) ^ 1, s_abort);
          mbar_expect_tx(bar(dqKFull0 + ks), L::kTileBytes);
#pragma unroll
          for (int b = 0; b < L::kBoxes; ++b)
            tma_load_2d(sK + b * L::kBoxBytes, &tm_k, g * D + b * 64, kv_start + j * kBN,
                        bar(dqKFull0 + ks));
          mbar_wait(bar(dqVEmpty0 + vs), ((gk / L::kVStages) & 1) ^ 1, s_abort);
          mbar_expect_tx(bar(dqVFull0 + vs), L::kTileBytes);
#pragma unroll
          for (int b = 0; b < L::kBoxes; ++b)
            tma_load_2d(sV + b * L::kBoxBytes, &tm_v, g * D + b * 64, kv_start + j * kBN,
                        bar(dqVFull0 + vs));
        }
      }
    }
    __syncwarp();
  } else if (warp == kMmaWarp) {
    // =============================== MMA issuer ===========================================
    // The whole warp walks the schedule (so that addresses and descriptors stay warp-uniform);
    // one elected lane issues the tensor-core instructions.
    {
      constexpr uint32_t kQKFmt = kRot ? kFmtF16 : kFmtBF16;   // rotated q, k copies are fp16
      constexpr uint32_t kIdescS = make_idesc(128, 128, kQKFmt, kQKFmt, 0, 0);
      constexpr uint32_t kIdescDP = make_idesc(128, 128, kFmtBF16, kFmtBF16, 0, 0);
      constexpr uint32_t kIdescDQ = make_idesc(128, D, kQKFmt, kQKFmt, 0, 1);   // dS follows k
      const bool leader = elect_one();
      int gk = 0, uc = 0;
      auto issue_s = [&](int g_idx) {       // S = Q K^T, Q from tensor memory
        const int ks = g_idx % L::kKStages;
        const uint32_t k_lo = desc_lo(sbase + L::kK0 + ks * L::kTileBytes, 16);
        mbar_wait(bar(dqKFull0 + ks), (g_idx / L::kKStages) & 1, s_abort);
        tc_fence_after();
        if (leader) {
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk) {
            const uint32_t off = (kk / 4) * L::kBoxBytes + (kk % 4) * 32;
            mma_ts(tS, tQ + kk * 8, desc_from_lo(k_lo + (off >> 4)), kIdescS, kk > 0);
          }
          mma_commit(bar(dqSFull));
        }
        __syncwarp();
      };
      auto issue_dp = [&](int g_idx) {      // dP = dO V^T; the V stage is free once it completes
        const int vs = g_idx % L::kVStages;
        const uint32_t v_lo = desc_lo(sbase + L::kV0 + vs * L::kTileBytes, 16);
        mbar_wait(bar(dqVFull0 + vs), (g_idx / L::kVStages) & 1, s_abort);
        tc_fence_after();
        if (leader) {
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk) {
            const uint32_t off = (kk / 4) * L::kBoxBytes + (kk % 4) * 32;
            mma_ts(tdP, tdO + kk * 8, desc_from_lo(v_lo + (off >> 4)), kIdescDP, kk > 0);
          }
          mma_commit(bar(dqDpFull));
          mma_commit(bar(dqVEmpty0 + vs));
        }
        __syncwarp();
      };
      for (int r = 0;; ++r, ++uc) {
        const int u = snake_unit(r, cta, n_cta);
        if (u >= n_units || *s_abort) break;
        const int4 it = items[order[u / Hq]];
        const int n_kv = (it.w + kBN - 1) / kBN;
        mbar_wait(bar(dqQtReady), uc & 1, s_abort);
        if (gk > 0) mbar_wait(bar(dqSRead), (gk - 1) & 1, s_abort);   // S of the previous step read
        tc_fence_after();
        issue_s(gk);
        issue_dp(gk);
        for (int j = 0; j < n_kv; ++j, ++gk) {
          const int ks = gk % L::kKStages;
          const uint32_t k_lo = desc_lo(sbase + L::kK0 + ks * L::kTileBytes, L::kBoxBytes);
          const bool more = (j + 1 < n_kv);
          if (more) {   // the single S buffer is free as soon as the compute warps have loaded S(j)
            mbar_wait(bar(dqSRead), gk & 1, s_abort);
            issue_s(gk + 1);
          }
          mbar_wait(bar(dqDsReady), gk & 1, s_abort);
          if (j == 0 && uc > 0) mbar_wait(bar(dqRead), (uc - 1) & 1, s_abort);
          tc_fence_after();
          if (leader) {
#pragma unroll
            for (int kk = 0; kk < kBN / 16; ++kk)   // dQ += dS K   (dS from tensor memory)
              mma_ts(tdQ, tdP + kk * 8, desc_from_lo(k_lo + ((kk * 2048) >> 4)), kIdescDQ,
                     (j > 0) | (kk > 0));
            mma_commit(bar(dqKEmpty0 + ks));
          }
          __syncwarp();
          if (more) issue_dp(gk + 1);   // overwrites dP/dS(j) after dQ(j) (same pipe, in order)
        }
        if (leader) mma_commit(bar(dqDone));
        __syncwarp();
      }
    }
  } else {
    // =============================== compute ===============================================
    const int row = tid & 127;              // query row inside the tile
    const int qd = tid >> 7;                // which group of kCW key columns
    const uint32_t lane_off = static_cast<uint32_t>((warp & 3) * 32) << 16;
    // Q and dO rows of unit number `n`: shared memory (128B-swizzled) -> tensor memory, half a
    // row per thread; then the shared-memory copies may be overwritten by the next load.
    auto copy_q_do = [&](int n) {
      mbar_wait(bar(dqQFull), n & 1, s_abort);
      if (qd < 2) {
        constexpr int kElems = D / 2;                       // elements per thread
        const int box = (qd * kElems) / 64, chunk0 = ((qd * kElems) % 64) / 8;
#pragma unroll
        for (int which = 0; which < 2; ++which) {
          const uint8_t* src = smem + (which == 0 ? L::kQ : L::kdO) + box * L::kBoxBytes + row * 128;
          uint32_t v[kElems / 2];
#pragma unroll
          for (int c = 0; c < kElems / 8; ++c) {
            const uint4 x = *reinterpret_cast<const uint4*>(src + (((chunk0 + c) ^ (row & 7)) << 4));
            v[4 * c] = x.x; v[4 * c + 1] = x.y; v[4 * c + 2] = x.z; v[4 * c + 3] = x.w;
          }
          const uint32_t dst = (which == 0 ? tQ : tdO) + lane_off + qd * (kElems / 2);
          if (kElems == 64) tmem_st32(dst, v);
          else tmem_st16(dst, v);
        }
        tmem_wait_st();
      }
      tc_fence_before();
      mbar_arrive(bar(dqQtReady));
      mbar_arrive(bar(dqQEmpty));
    };
    int gk = 0, uc = 0;
    if (snake_unit(0, cta, n_cta) < n_units && !*s_abort) copy_q_do(0);
    for (int r = 0;; ++r, ++uc) {
      const int u = snake_unit(r, cta, n_cta);
      if (u >= n_units || *s_abort) break;
      const int4 it = items[order[u / Hq]];
      const int h = u % Hq;
      const int q_start = it.x, q_len = it.y, kv_len = it.w;
      const int n_kv = (kv_len + kBN - 1) / kBN;
      const int tok = q_start + row;
      const float lse2 = (tok < T) ? lse[(size_t)h * T + tok] * kLog2eWs : 0.f;
      const float dl = (tok < T) ? delta[(size_t)h * T + tok] : 0.f;

      for (int j = 0; j < n_kv; ++j, ++gk) {
        mbar_wait(bar(dqSFull), gk & 1, s_abort);
        tc_fence_after();
        float p[kCW];
        {
          uint32_t sv[kCW];
#pragma unroll
          for (int c0 = 0; c0 < kCW; c0 += 32) tmem_ld32(tS + lane_off + qd * kCW + c0, sv + c0);
          tmem_wait_ld();
          tc_fence_before();
          mbar_arrive(bar(dqSRead));
#pragma unroll
          for (int c = 0; c < kCW; ++c)
            p[c] = fast_exp2(fmaf(__uint_as_float(sv[c]), scale_log2, -lse2));
          if (j == n_kv - 1) {   // only the diagonal tile needs the causal mask
#pragma unroll
            for (int c = 0; c < kCW; ++c)
              if (qd * kCW + c > row) p[c] = 0.f;
          }
        }
        mbar_wait(bar(dqDpFull), gk & 1, s_abort);
        tc_fence_after();
        uint32_t dd[kCW / 2];
#pragma unroll
        for (int c2 = 0; c2 < kCW / 32; ++c2) {
          uint32_t dp[32];
          tmem_ld32(tdP + lane_off + qd * kCW + c2 * 32, dp);
          tmem_wait_ld();
#pragma unroll
          for (int e = 0; e < 32; e += 2) {
            const float d0 = p[c2 * 32 + e] * (__uint_as_float(dp[e]) - dl);
            const float d1 = p[c2 * 32 + e + 1] * (__uint_as_float(dp[e + 1]) - dl);
            dd[c2 * 16 + (e >> 1)] = kRot ? pack_f16x2(d0, d1) : pack_bf16x2(d0, d1);
          }
        }
        // every thread must have read dP before dS overwrites its columns
        tc_fence_before();
        compute_bar_sync();
        tc_fence_after();
        if (kCW == 64) tmem_st32(tdP + lane_off + qd * (kCW / 2), dd);
        else tmem_st16(tdP + lane_off + qd * (kCW / 2), dd);
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(bar(dqDsReady));
      }
      // The last S and dP of this unit have been consumed, so Q/dO of the NEXT unit can move into
      // tensor memory now; the issuing warp then starts that unit while this one's dQ is written.
      if (snake_unit(r + 1, cta, n_cta) < n_units && !*s_abort) copy_q_do(uc + 1);
      // ---- unit epilogue: dQ rows, scaled (column groups 0 and 1 write half a row each) -----
      mbar_wait(bar(dqDone), uc & 1, s_abort);
      tc_fence_after();
      if (qd < 2) {
        const bool live = (row < q_len) && (*s_abort == 0);
        if (kRot) {
          // rotate back by -angle: this thread owns pairs i in [32*qd, +32) and i + 64
          static_assert(!kRot || D == 128, "rotated path is built for D = 128");
          GradT* dst = dq + ((size_t)tok * Hq + h) * D + qd * 32;
          uint32_t x1[32], x2[32];
          float y1[32], y2[32];
          tmem_ld32(tdQ + lane_off + qd * 32, x1);
          tmem_ld32(tdQ + lane_off + 64 + qd * 32, x2);
          tmem_wait_ld();
          if (live) {
            const float2* cs = rope_table + (size_t)tok * (D / 2) + qd * 32;
#pragma unroll
            for (int e = 0; e < 32; ++e) {
              const float2 t = __ldg(cs + e);
              const float a = __uint_as_float(x1[e]) * scale, b = __uint_as_float(x2[e]) * scale;
              y1[e] = a * t.x + b * t.y;
              y2[e] = b * t.x - a * t.y;
            }
            store_chunk32<GradT>(dst, y1);
            store_chunk32<GradT>(dst + 64, y2);
          }
        } else {
          GradT* dst = dq + ((size_t)tok * Hq + h) * D + qd * (D / 2);
#pragma unroll
          for (int c = 0; c < D / 64; ++c) {
            uint32_t x[32];
            float y[32];
            tmem_ld32(tdQ + lane_off + qd * (D / 2) + c * 32, x);
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < 32; ++e) y[e] = __uint_as_float(x[e]) * scale;
            if (live) store_chunk32<GradT>(dst + c * 32, y);
          }
        }
      }
      tc_fence_before();
      mbar_arrive(bar(dqRead));
    }
  }

  tc_fence_before();
  __syncthreads();
  if (*s_abort != 0 && tid == 0) set_status(hdr, PK_ERR_TIMEOUT, 4);
  if (warp == kMmaWarp) tmem_dealloc(tmem, 512);
}

template <int D, bool kRot, typename GradT>
int launch_ws(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
              const CUtensorMap& tdo, char* ws, const WorkspaceLayout& lay, const float* lse,
              void* dq, void* dk, void* dv, int T, int Hq, int Hkv, float scale,
              cudaStream_t stream) {
  auto kern_kv = attn_bwd_dkv_kernel<D, kRot, GradT>;
  auto kern_q = attn_bwd_dq_kernel<D, kRot, GradT>;
  if (cudaFuncSetAttribute(kern_kv, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           DkvSmem<D>::kTotal) != cudaSuccess ||
      cudaFuncSetAttribute(kern_q, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           DqSmem<D>::kTotal) != cudaSuccess)
    return PK_ERR_CUDA;
  int32_t* hdr = reinterpret_cast<int32_t*>(ws + lay.off[PK_WS_HEADER]);
  const float* delta = reinterpret_cast<const float*>(ws + lay.off[PK_WS_DELTA]);
  const float2* table = reinterpret_cast<const float2*>(ws + lay.off[PK_WS_ROPE_TABLE]);
  const int grid = sm_count();
  {
    TimedLaunch timed(PK_KERNEL_BWD, stream);
    kern_kv<<<grid, kWsThreads, DkvSmem<D>::kTotal, stream>>>(
        tq, tk, tv, tdo, reinterpret_cast<const int4*>(ws + lay.off[PK_WS_BWD_ITEMS]),
        reinterpret_cast<const int32_t*>(ws + lay.off[PK_WS_BWD_ORDER]), hdr, lse, delta,
        static_cast<GradT*>(dk), static_cast<GradT*>(dv), table, T, Hq, Hkv, scale,
        scale * kLog2eWs);
  }
  if (launch_status() != PK_OK) return PK_ERR_CUDA;
  {
    TimedLaunch timed(PK_KERNEL_BWD_DQ, stream);
    kern_q<<<grid, kWsThreads, DqSmem<D>::kTotal, stream>>>(
        tq, tk, tv, tdo, reinterpret_cast<const int4*>(ws + lay.off[PK_WS_FWD_ITEMS]),
        reinterpret_cast<const int32_t*>(ws + lay.off[PK_WS_FWD_ORDER]), hdr, lse, delta,
        static_cast<GradT*>(dq), table, T, Hq, Hkv, scale, scale * kLog2eWs);
  }
  return launch_status();
}

}  // namespace

int launch_bwd_ws(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                  const CUtensorMap& tdo, char* ws, const WorkspaceLayout& lay, const float* lse,
                  void* dq, void* dk, void* dv, int T, int Hq, int Hkv, int D, int grad_dtype,
                  float scale, bool rotated, cudaStream_t stream) {
#define PK_BWS(DD, RR, TT)                                                                     \
  return launch_ws<DD, RR, TT>(tq, tk, tv, tdo, ws, lay, lse, dq, dk, dv, T, Hq, Hkv, scale, \
                               stream)
  if (D == 128) {
    if (rotated) {
      if (grad_dtype == PK_BF16) PK_BWS(128, true, __nv_bfloat16); else PK_BWS(128, true, float);
    } else {
      if (grad_dtype == PK_BF16) PK_BWS(128, false, __nv_bfloat16); else PK_BWS(128, false, float);
    }
  }
  if (grad_dtype == PK_BF16) PK_BWS(64, false, __nv_bfloat16);
  PK_BWS(64, false, float);
#undef PK_BWS
}

}  // namespace pk
