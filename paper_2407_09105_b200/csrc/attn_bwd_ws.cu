// Warp-specialised backward kernels for sm_100a (with RoPE they run on rotated fp16 copies of q
// and k and rotate dQ / dK back in their epilogues: kRot).
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
// reproducible, and both never visit a tile outside an example's causal block (or, with a
// sliding window, outside the band of tiles the window reaches).
//
// Roles: 8 compute warps (lane = tensor-memory row; warp w works on columns [64*(w/4), +64) of
// the rows of lane quarter w%4; 16 warps of 32 columns measured slightly slower because they
// take issue slots from the warp that feeds the tensor pipe), one warp that walks the MMA
// schedule with one elected lane issuing every tcgen05.mma, one warp that drives TMA, and four
// writer warps (one thread per row) that scale, rotate back and store a unit's accumulators
// while the compute warps are already in the next unit.  512 threads start with 128 registers
// each; setmaxnreg moves them to the compute warps at the top of each warpgroup's branch.
// Units are drawn from a counter (see kUnitRing below) in the plan's order.
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
constexpr int kComputeThreads = PK_BWD_COMPUTE_THREADS;
constexpr int kNQ = kComputeThreads / 128;                // column groups per tile row
constexpr int kCW = 128 / kNQ;                            // columns per compute thread
// warps 0-7 compute, 8 issues the contractions, 9 loads, 10-11 idle, 12-15 write the results
constexpr int kBwdThreads = 512;
constexpr int kWriterWarp0 = 12;
constexpr int kWriterThreads = 128;
constexpr int kMmaWarp = kComputeThreads / 32;
constexpr int kLoadWarp = kMmaWarp + 1;
static_assert(kNQ == 2, "the dK/dV kernel gives each compute thread 64 query columns");
constexpr float kLog2eWs = 1.4426950408889634f;

// Units are handed out dynamically: the TMA warp draws the next position of the plan's order
// from a counter in the workspace header and publishes it to the other roles through a small
// ring in shared memory (one mbarrier per slot).  The order keeps the units of an example next
// to each other, so the CTAs that run at the same time share tiles in L2, and drawing from it
// keeps every CTA busy to the end (dealt out statically, the slowest CTA of the dK/dV kernel
// carried a fifth more steps than the mean on 8k-token packs).  A slot is rewritten four units
// later; no role can fall that far behind the TMA warp, which waits for the previous unit's
// tiles to be released before it loads the next one's.
constexpr int kUnitRing = 4;

// =========================================================================================
// dK / dV kernel
// =========================================================================================
template <int D>
struct DkvSmem {
  static constexpr int kBoxBytes = 128 * 128;
  static constexpr int kBoxes = D / 64;
  static constexpr int kTileBytes = kBoxBytes * kBoxes;
  static constexpr int kQStages = 3;                         // Q is needed until dK of its step
  static constexpr int kDoStages = 2;
  static constexpr int kK = 0;
  static constexpr int kV = kTileBytes;
  static constexpr int kQ0 = 2 * kTileBytes;                 // Q ring
  static constexpr int kDo0 = kQ0 + kQStages * kTileBytes;   // dO ring
  static constexpr int kLse = kDo0 + kDoStages * kTileBytes; // [2][128] floats, slot = step & 1
  static constexpr int kDelta = kLse + 1024;                 // [2][128] floats
  static constexpr int kBars = kDelta + 1024;
  static constexpr int kMisc = kBars + 24 * 8;               // tmem base, abort flag, unit ring
  static constexpr int kTotal = kMisc + 16 + 4 * kUnitRing;
};

enum DkvBar {
  kvKvFull = 0, kvKvEmpty,
  kvQFull0, kvQFull1, kvQFull2, kvDoFull0, kvDoFull1, kvQEmpty0, kvQEmpty1, kvQEmpty2,
  kvSFull, kvDpFull, kvPReady, kvDsReady, kvDpRead, kvUnitDone, kvDkvRead,
  kvUnitFull0, kvUnitFull1, kvUnitFull2, kvUnitFull3, kvNumBars
};
static_assert(kvNumBars <= 24, "barrier area");

// Tensor memory of the dK/dV kernel: two 128-column regions that trade roles every step, then
// the dV and dK accumulators.  Step n keeps S^T in region n & 1; each compute thread overwrites
// its own 64 columns of it with P^T (first 32 columns, 64 bf16) and dS^T (last 32), so no thread
// ever writes a column another thread still has to read.  dP^T of step n sits in the other
// region, and S^T of step n+1 is written there as soon as every thread holds dP^T(n) in
// registers: the next step's scores never wait for the tensor pipe to consume P^T or dS^T.
template <int D, bool kRot, typename GradT>
__global__ void __launch_bounds__(kBwdThreads, 1)
attn_bwd_dkv_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                    const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_do,
                    const int4* __restrict__ items, const int32_t* __restrict__ order, int32_t* hdr,
                    const float* __restrict__ lse, const float* __restrict__ delta,
                    GradT* __restrict__ dk, GradT* __restrict__ dv,
                    const float* __restrict__ rope_angle,
                    int T, int Hq, int Hkv, float scale, float scale_log2, int window) {
  using L = DkvSmem<D>;
  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t sbase = smem_u32(smem);
  const uint32_t sK = sbase + L::kK, sV = sbase + L::kV;
  float* s_lse = reinterpret_cast<float*>(smem + L::kLse);
  float* s_delta = reinterpret_cast<float*>(smem + L::kDelta);
  const uint32_t bars = sbase + L::kBars;
  auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };
  volatile int* s_tmem = reinterpret_cast<volatile int*>(smem + L::kMisc);
  volatile int* s_abort = s_tmem + 1;
  volatile int* s_unit = s_tmem + 4;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (tid == 0) {
    mbar_init(bar(kvKvFull), 1);
    mbar_init(bar(kvKvEmpty), 1);
    for (int i = 0; i < L::kQStages; ++i) {
      mbar_init(bar(kvQFull0 + i), 1);
      mbar_init(bar(kvQEmpty0 + i), 1);
    }
    for (int i = 0; i < L::kDoStages; ++i) mbar_init(bar(kvDoFull0 + i), 33);
    mbar_init(bar(kvSFull), 1);
    mbar_init(bar(kvDpFull), 1);
    mbar_init(bar(kvPReady), kComputeThreads);
    mbar_init(bar(kvDsReady), kComputeThreads);
    mbar_init(bar(kvDpRead), kComputeThreads);
    mbar_init(bar(kvUnitDone), 1);
    mbar_init(bar(kvDkvRead), kWriterThreads);
    for (int i = 0; i < kUnitRing; ++i) mbar_init(bar(kvUnitFull0 + i), 1);
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
  const uint32_t tdV = tmem + 256, tdK = tmem + 384;
  auto region_s = [&](int n) { return tmem + static_cast<uint32_t>(n & 1) * 128u; };
  auto region_dp = [&](int n) { return tmem + static_cast<uint32_t>((n & 1) ^ 1) * 128u; };

  const int G = Hq / Hkv;
  const bool plan_ok = (hdr[PK_HDR_PLAN_T] == T);
  if (!plan_ok && blockIdx.x == 0 && tid == 0) set_status(hdr, PK_ERR_NO_PLAN, T);
  const int n_units = plan_ok ? hdr[PK_HDR_N_ITEMS] * Hkv : 0;
  // query tiles of a key block: to the example's end, or (sliding window) to the last query that
  // still sees the block's last key, window - 1 rows further down
  auto query_tiles = [&](int kv_len, int q_len) {
    const int n = (q_len + kBM - 1) / kBM;
    return window > 0 ? min(n, (kv_len - 1 + window - 1) / kBM + 1) : n;
  };

  // Register budget: 512 threads start with 128 each; every warpgroup changes its allowance at the
  // top of its own branch.  The two decreases free 128 * (88 + 32) = 15 360 registers without
  // waiting for anything, the increases take 256 * 48 = 12 288: they cannot block for good.
  if ((warp >> 2) == (kMmaWarp >> 2)) {
  setmaxnreg_dec<40>();
  if (warp == kLoadWarp) {
    // =============================== loader ===============================================
    // Steps are numbered globally (gs) across this CTA's units.  Q(gs) goes to Q stage gs % 3 once
    // dK of step gs-3 has retired; dO(gs) and the lse / delta rows go to slot gs & 1 once dK of step
    // gs-2 has retired (dV(gs-2) precedes it on the tensor pipe, and the compute warps are done
    // with that step's lse / delta before they hand over its dS).
    if (lane == 0) {
      prefetch_tensormap(&tm_q);
      prefetch_tensormap(&tm_k);
      prefetch_tensormap(&tm_v);
      prefetch_tensormap(&tm_do);
    }
    int gs = 0, uc = 0;
    for (;; ++uc) {
      int u = 0;
      if (lane == 0) {
        u = atomicAdd(&hdr[kHdrBwdTicket], 1);
        s_unit[uc % kUnitRing] = u;
        mbar_arrive(bar(kvUnitFull0 + uc % kUnitRing));
      }
      u = __shfl_sync(0xffffffffu, u, 0);
      if (u >= n_units || *s_abort) break;
      const int4 it = items[order[u / Hkv]];
      const int g = u % Hkv;
      const int kv_start = it.x, q_start = it.z, q_len = it.w;
      const int n_q = query_tiles(it.y, q_len);
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
          const int qs = gs % L::kQStages, sl = gs & 1;
          const int q0 = q_start + i * kBM;
          mbar_wait(bar(kvQEmpty0 + qs), ((gs / L::kQStages) & 1) ^ 1, s_abort);
          if (lane == 0) {
            const uint32_t sQ = sbase + L::kQ0 + qs * L::kTileBytes;
            mbar_expect_tx(bar(kvQFull0 + qs), L::kTileBytes);
#pragma unroll
            for (int b = 0; b < L::kBoxes; ++b)
              tma_load_2d(sQ + b * L::kBoxBytes, &tm_q, h * D + b * 64, q0, bar(kvQFull0 + qs));
          }
          if (gs >= 2) {
            const int e = gs - 2;
            mbar_wait(bar(kvQEmpty0 + e % L::kQStages), (e / L::kQStages) & 1, s_abort);
          }
          if (lane == 0) {
            const uint32_t sdO = sbase + L::kDo0 + sl * L::kTileBytes;
            mbar_expect_tx(bar(kvDoFull0 + sl), L::kTileBytes);
#pragma unroll
            for (int b = 0; b < L::kBoxes; ++b)
              tma_load_2d(sdO + b * L::kBoxBytes, &tm_do, h * D + b * 64, q0, bar(kvDoFull0 + sl));
          }
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int row = lane * 4 + e, tok = q0 + row;
            const bool in = tok < T;
            s_lse[sl * 128 + row] = in ? lse[(size_t)h * T + tok] * kLog2eWs : 0.f;
            s_delta[sl * 128 + row] = in ? delta[(size_t)h * T + tok] : 0.f;
          }
          mbar_arrive(bar(kvDoFull0 + sl));
        }
      }
    }
  } else if (warp == kMmaWarp) {
    // =============================== MMA issuer ===========================================
    // The whole warp walks the schedule (so that addresses and descriptors stay warp-uniform);
    // one elected lane issues the tensor-core instructions.  Per step, in tensor-pipe order:
    //   S^T(s+1) | dV += P^T(s) dO | dK += dS^T(s) Q | dP^T(s+1)
    {
      // kRot: q and k are the rotated fp16 copies; dS then follows their format (operands of one
      // contraction must share a format), everything touching V, dO and P stays bf16
      constexpr uint32_t kQKFmt = kRot ? kFmtF16 : kFmtBF16;
      constexpr uint32_t kIdescS = make_idesc(128, 128, kQKFmt, kQKFmt, 0, 0);
      constexpr uint32_t kIdescDP = make_idesc(128, 128, kFmtBF16, kFmtBF16, 0, 0);
      constexpr uint32_t kIdescDV = make_idesc(128, D, kFmtBF16, kFmtBF16, 0, 1);
      constexpr uint32_t kIdescDK = make_idesc(128, D, kQKFmt, kQKFmt, 0, 1);
      const bool leader = elect_one();
      const uint32_t k_lo = desc_lo(sK, 16), v_lo = desc_lo(sV, 16);
      int gs = 0, uc = 0;
      auto issue_s = [&](int n) {   // S^T(n) = K Q(n)^T into region_s(n)
        const int qs = n % L::kQStages;
        mbar_wait(bar(kvQFull0 + qs), (n / L::kQStages) & 1, s_abort);
        tc_fence_after();
        const uint32_t q_lo = desc_lo(sbase + L::kQ0 + qs * L::kTileBytes, 16);
        const uint32_t dst = region_s(n);
        if (leader) {
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk) {
            const uint32_t off = ((kk / 4) * L::kBoxBytes + (kk % 4) * 32) >> 4;
            mma_ss(dst, desc_from_lo(k_lo + off), desc_from_lo(q_lo + off), kIdescS, kk > 0);
          }
          mma_commit(bar(kvSFull));
        }
        __syncwarp();
      };
      auto issue_dp = [&](int n) {  // dP^T(n) = V dO(n)^T into region_dp(n)
        const int sl = n & 1;
        mbar_wait(bar(kvDoFull0 + sl), (n >> 1) & 1, s_abort);
        tc_fence_after();
        const uint32_t do_lo = desc_lo(sbase + L::kDo0 + sl * L::kTileBytes, 16);
        const uint32_t dst = region_dp(n);
        if (leader) {
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk) {
            const uint32_t off = ((kk / 4) * L::kBoxBytes + (kk % 4) * 32) >> 4;
            mma_ss(dst, desc_from_lo(v_lo + off), desc_from_lo(do_lo + off), kIdescDP, kk > 0);
          }
          mma_commit(bar(kvDpFull));
        }
        __syncwarp();
      };
      for (;; ++uc) {
        mbar_wait(bar(kvUnitFull0 + uc % kUnitRing), (uc / kUnitRing) & 1, s_abort);
        const int u = s_unit[uc % kUnitRing];
        if (u >= n_units || *s_abort) break;
        const int4 it = items[order[u / Hkv]];
        const int n_q = query_tiles(it.y, it.w);
        const int n_steps = G * n_q;
        mbar_wait(bar(kvKvFull), uc & 1, s_abort);
        // prologue: S(0) goes where dP of the previous unit's last step was, so that one must
        // have been read; dP(0) goes where P / dS of that step were, which its dV / dK consumed
        // earlier on the tensor pipe
        if (gs > 0) mbar_wait(bar(kvDpRead), (gs - 1) & 1, s_abort);
        tc_fence_after();
        issue_s(gs);
        issue_dp(gs);
        // K and V are read for the last time by the unit's last S^T and dP^T, which are issued one
        // step before its end: releasing them there lets the next unit's K and V arrive while this
        // unit's last dV and dK still run
        if (n_steps == 1 && leader) mma_commit(bar(kvKvEmpty));
        for (int s = 0; s < n_steps; ++s, ++gs) {
          const uint32_t tA = region_s(gs);
          const uint32_t doT_lo = desc_lo(sbase + L::kDo0 + (gs & 1) * L::kTileBytes, L::kBoxBytes);
          const uint32_t qT_lo =
              desc_lo(sbase + L::kQ0 + (gs % L::kQStages) * L::kTileBytes, L::kBoxBytes);
          const uint32_t acc = s > 0 ? 1u : 0u;
          const bool more = (s + 1 < n_steps);
          if (more) {                             // S(s+1) over dP(s), which sits in registers now
            // (the TMA barrier first: it completed long ago, and polling it costs time best
            // spent while dP(s) is still being read)
            mbar_wait(bar(kvQFull0 + (gs + 1) % L::kQStages), ((gs + 1) / L::kQStages) & 1, s_abort);
            mbar_wait(bar(kvDpRead), gs & 1, s_abort);
            tc_fence_after();
            issue_s(gs + 1);
          } else {
            mbar_wait(bar(kvPReady), gs & 1, s_abort);
          }
          // every thread hands over P^T before it reads dP^T, so the wait above covers P^T as well
          if (s == 0 && uc > 0) mbar_wait(bar(kvDkvRead), (uc - 1) & 1, s_abort);
          tc_fence_after();
          if (leader) {
#pragma unroll
            for (int kk = 0; kk < kBM / 16; ++kk)   // dV += P^T dO; P^T of queries 16kk.. : see compute
              mma_ts(tdV, tA + (kk / 4) * 64 + (kk % 4) * 8, desc_from_lo(doT_lo + ((kk * 2048) >> 4)),
                     kIdescDV, acc | (kk > 0));
          }
          __syncwarp();
          mbar_wait(bar(kvDsReady), gs & 1, s_abort);
          tc_fence_after();
          if (leader) {
#pragma unroll
            for (int kk = 0; kk < kBM / 16; ++kk)   // dK += dS^T Q
              mma_ts(tdK, tA + (kk / 4) * 64 + 32 + (kk % 4) * 8,
                     desc_from_lo(qT_lo + ((kk * 2048) >> 4)), kIdescDK, acc | (kk > 0));
            mma_commit(bar(kvQEmpty0 + gs % L::kQStages));
          }
          __syncwarp();
          if (more) issue_dp(gs + 1);             // over P / dS(s), consumed just above
          if (s + 2 == n_steps && leader) mma_commit(bar(kvKvEmpty));
        }
        if (leader) mma_commit(bar(kvUnitDone));
        __syncwarp();
      }
    }
  }
  } else if (warp < kMmaWarp) {
    // =============================== compute ===============================================
    setmaxnreg_inc<176>();
    const int row = tid & 127;              // key row inside the block
    const int qd = tid >> 7;                // this thread's query columns: [64*qd, +64)
    const uint32_t lane_off = static_cast<uint32_t>((warp & 3) * 32) << 16;
    const int col0 = qd * kCW;
    int gs = 0, uc = 0;
    for (;; ++uc) {
      mbar_wait(bar(kvUnitFull0 + uc % kUnitRing), (uc / kUnitRing) & 1, s_abort);
      const int u = s_unit[uc % kUnitRing];
      if (u >= n_units || *s_abort) break;
      const int4 it = items[order[u / Hkv]];
      const int g = u % Hkv;
      const int kv_start = it.x, kv_len = it.y, q_len = it.w;
      const int n_q = query_tiles(kv_len, q_len);
      for (int hh = 0; hh < G; ++hh) {
        for (int i = 0; i < n_q; ++i, ++gs) {
          const int sl = gs & 1;
          // queries [i*128, ..) of the unit: up to the example's end and, with a sliding window,
          // less than `window` rows below this thread's key
          const int q_rows = q_len - i * kBM;
          const int q_left = window > 0 ? min(q_rows, row + window - i * kBM) : q_rows;
          const bool win_edge = window > 0 && (i + 1) * kBM > window;
          const int col_min = (i == 0) ? row : 0;
          const uint32_t tA = region_s(gs) + lane_off + col0;    // S^T, then P^T | dS^T
          const uint32_t tB = region_dp(gs) + lane_off + col0;   // dP^T
          mbar_wait(bar(kvDoFull0 + sl), (gs >> 1) & 1, s_abort);   // lse / delta rows visible
          mbar_wait(bar(kvSFull), gs & 1, s_abort);
          tc_fence_after();
          float p[64];
          {
            uint32_t sv[64];
            tmem_ld32(tA, sv);
            tmem_ld32(tA + 32, sv + 32);
            tmem_wait_ld();
            const float4* lse4 = reinterpret_cast<const float4*>(s_lse + sl * 128 + col0);
#pragma unroll
            for (int c = 0; c < 64; c += 4) {
              const float4 l4 = lse4[c >> 2];
              p[c] = fast_exp2(fmaf(__uint_as_float(sv[c]), scale_log2, -l4.x));
              p[c + 1] = fast_exp2(fmaf(__uint_as_float(sv[c + 1]), scale_log2, -l4.y));
              p[c + 2] = fast_exp2(fmaf(__uint_as_float(sv[c + 2]), scale_log2, -l4.z));
              p[c + 3] = fast_exp2(fmaf(__uint_as_float(sv[c + 3]), scale_log2, -l4.w));
            }
          }
          if (i == 0 || q_rows < kBM || win_edge) {   // diagonal, last partial or window-edge tile; interior tiles skip this
#pragma unroll
            for (int c = 0; c < 64; ++c) {
              const int col = col0 + c;
              if (!((col >= col_min) && (col < q_left))) p[c] = 0.f;
            }
          }
          {
            uint32_t pp[32];
#pragma unroll
            for (int c = 0; c < 32; ++c) pp[c] = pack_bf16x2(p[2 * c], p[2 * c + 1]);
            tmem_st32(tA, pp);            // over this thread's own S^T columns
          }
          tmem_wait_st();
          tc_fence_before();
          mbar_arrive(bar(kvPReady));

          mbar_wait(bar(kvDpFull), gs & 1, s_abort);
          tc_fence_after();
          {
            uint32_t dp[64], dd[32];
            tmem_ld32(tB, dp);
            tmem_ld32(tB + 32, dp + 32);
            tmem_wait_ld();
            tc_fence_before();
            mbar_arrive(bar(kvDpRead));   // the next S^T may be written over dP^T
            const float4* dl4 = reinterpret_cast<const float4*>(s_delta + sl * 128 + col0);
#pragma unroll
            for (int e = 0; e < 64; e += 4) {
              const float4 d4 = dl4[e >> 2];
              const float d0 = p[e] * (__uint_as_float(dp[e]) - d4.x);
              const float d1 = p[e + 1] * (__uint_as_float(dp[e + 1]) - d4.y);
              const float d2 = p[e + 2] * (__uint_as_float(dp[e + 2]) - d4.z);
              const float d3 = p[e + 3] * (__uint_as_float(dp[e + 3]) - d4.w);
              dd[e >> 1] = kRot ? pack_f16x2(d0, d1) : pack_bf16x2(d0, d1);
              dd[(e >> 1) + 1] = kRot ? pack_f16x2(d2, d3) : pack_bf16x2(d2, d3);
            }
            tmem_st32(tA + 32, dd);
          }
          tmem_wait_st();
          tc_fence_before();
          mbar_arrive(bar(kvDsReady));
        }
      }
    }
  } else if (warp >= kWriterWarp0) {
    // =============================== dK / dV writer ========================================
    // One thread per key row: waits for the unit's last contraction, pulls the rows of dV and dK
    // out of tensor memory 32 columns at a time, scales dK (and rotates it back), stores.  The
    // accumulators are released as soon as the last columns are in registers.
    setmaxnreg_dec<96>();
    const int row = tid & 127;
    const uint32_t lane_off = static_cast<uint32_t>((warp & 3) * 32) << 16;
    for (int uc = 0;; ++uc) {
      mbar_wait(bar(kvUnitFull0 + uc % kUnitRing), (uc / kUnitRing) & 1, s_abort);
      const int u = s_unit[uc % kUnitRing];
      if (u >= n_units || *s_abort) break;
      const int4 it = items[order[u / Hkv]];
      const int g = u % Hkv;
      const int tok = it.x + row;
      mbar_wait(bar(kvUnitDone), uc & 1, s_abort);
      tc_fence_after();
      const bool live = (row < it.y) && (*s_abort == 0);
      GradT* dv_row = dv + ((size_t)tok * Hkv + g) * D;
      GradT* dk_row = dk + ((size_t)tok * Hkv + g) * D;
#pragma unroll
      for (int c = 0; c < D; c += 32) {
        uint32_t x[32];
        tmem_ld32(tdV + lane_off + c, x);
        tmem_wait_ld();
        if (live) {
          float y[32];
#pragma unroll
          for (int e = 0; e < 32; ++e) y[e] = __uint_as_float(x[e]);
          store_chunk32<GradT>(dv_row + c, y);
        }
      }
      if (kRot) {
        // dK was formed against the rotated k: rotate back by -angle, pairs (i, i + D/2)
        const float* cs = rope_angle + (size_t)tok * (D / 2);
#pragma unroll
        for (int c = 0; c < D / 2; c += 32) {
          uint32_t x1[32], x2[32];
          tmem_ld32(tdK + lane_off + c, x1);
          tmem_ld32(tdK + lane_off + D / 2 + c, x2);
          tmem_wait_ld();
          if (c + 32 >= D / 2) {
            tc_fence_before();
            mbar_arrive(bar(kvDkvRead));
          }
          if (live) {
            float y1[32], y2[32];
#pragma unroll
            for (int e4 = 0; e4 < 32; e4 += 8) {
              float2 t4[8];
              ld_angles8(cs + c + e4, t4);
#pragma unroll
              for (int k = 0; k < 8; ++k) {
                const int e = e4 + k;
                const float p = __uint_as_float(x1[e]) * scale, q = __uint_as_float(x2[e]) * scale;
                y1[e] = p * t4[k].x + q * t4[k].y;
                y2[e] = q * t4[k].x - p * t4[k].y;
              }
            }
            store_chunk32<GradT>(dk_row + c, y1);
            store_chunk32<GradT>(dk_row + D / 2 + c, y2);
          }
        }
      } else {
#pragma unroll
        for (int c = 0; c < D; c += 32) {
          uint32_t x[32];
          tmem_ld32(tdK + lane_off + c, x);
          tmem_wait_ld();
          if (c + 32 >= D) {
            tc_fence_before();
            mbar_arrive(bar(kvDkvRead));
          }
          if (live) {
            float y[32];
#pragma unroll
            for (int e = 0; e < 32; ++e) y[e] = __uint_as_float(x[e]) * scale;
            store_chunk32<GradT>(dk_row + c, y);
          }
        }
      }
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
  static constexpr int kMisc = kBars + 24 * 8;               // tmem base, abort flag, unit ring
  static constexpr int kTotal = kMisc + 16 + 4 * kUnitRing;
};

enum DqBar {
  dqQFull = 0, dqQEmpty, dqQtReady, dqKFull0, dqKFull1, dqKFull2, dqKEmpty0, dqKEmpty1, dqKEmpty2,
  dqVFull0, dqVFull1, dqVEmpty0, dqVEmpty1, dqSFull, dqSRead, dqDpFull, dqDsReady, dqDone, dqRead,
  dqUnitFull0, dqUnitFull1, dqUnitFull2, dqUnitFull3, dqNumBars
};

// The query-side tiles Q and dO are the stationary A operands of S = Q K^T and dP = dO V^T.
// They are copied once per unit from shared memory into tensor memory, so that those two
// contractions read only K / V from shared memory (the shared-memory port, not the tensor
// pipe, was the bound when all four operands came from there).
// Warps as in the dK/dV kernel: 12-15 write each unit's dQ (one thread per query row).
constexpr int kDqThreads = kBwdThreads;
constexpr int kDqEpiWarp0 = kWriterWarp0;
constexpr int kDqEpiThreads = kWriterThreads;
template <int D, bool kRot, typename GradT>
__global__ void __launch_bounds__(kDqThreads, 1)
attn_bwd_dq_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                   const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_do,
                   const int4* __restrict__ items, const int32_t* __restrict__ order, int32_t* hdr,
                   const float* __restrict__ lse, const float* __restrict__ delta,
                   GradT* __restrict__ dq, const float* __restrict__ rope_angle, int T, int Hq,
                   int Hkv, float scale, float scale_log2, int window) {
  using L = DqSmem<D>;
  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t sbase = smem_u32(smem);
  const uint32_t bars = sbase + L::kBars;
  auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };
  volatile int* s_tmem = reinterpret_cast<volatile int*>(smem + L::kMisc);
  volatile int* s_abort = s_tmem + 1;
  volatile int* s_unit = s_tmem + 4;

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
    mbar_init(bar(dqRead), kDqEpiThreads);
    for (int i = 0; i < kUnitRing; ++i) mbar_init(bar(dqUnitFull0 + i), 1);
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
  // [0,128) S, [128,256) dP (dS as bf16 goes over each thread's own dP columns), [256,256+D) dQ,
  // [384,384+D/2) Q as bf16 pairs, then D/2 columns of dO
  const uint32_t tS = tmem, tdP = tmem + 128, tdQ = tmem + 256, tQ = tmem + 384,
                 tdO = tmem + 384 + D / 2;

  const int G = Hq / Hkv;
  const bool plan_ok = (hdr[PK_HDR_PLAN_T] == T);
  const int n_units = plan_ok ? hdr[PK_HDR_N_ITEMS] * Hq : 0;
  // first key tile of a query block: 0, or (sliding window) the tile holding the key window - 1
  // positions before the block's first row
  auto first_key_tile = [&](int q_start, int kv_start) {
    const int reach = q_start - (window - 1) - kv_start;
    return (window > 0 && reach > 0) ? reach / kBN : 0;
  };

  // Register budget: 512 threads start with 128 each; the compute warps need more, the rest less.
  // Each warpgroup changes its allowance at the top of its own branch (the decreases free 15 360
  // registers unconditionally, the increases take 12 288).
  if ((warp >> 2) == (kMmaWarp >> 2)) {
  setmaxnreg_dec<40>();
  if (warp == kLoadWarp) {
    // =============================== loader ===============================================
    if (lane == 0) {
      prefetch_tensormap(&tm_q);
      prefetch_tensormap(&tm_k);
      prefetch_tensormap(&tm_v);
      prefetch_tensormap(&tm_do);
      int gk = 0, uc = 0;
      for (;; ++uc) {
        const int u = atomicAdd(&hdr[kHdrDqTicket], 1);
        s_unit[uc % kUnitRing] = u;
        mbar_arrive(bar(dqUnitFull0 + uc % kUnitRing));
        if (u >= n_units || *s_abort) break;
        const int4 it = items[order[u / Hq]];
        const int h = u % Hq, g = h / G;
        const int q_start = it.x, kv_start = it.z, kv_len = it.w;
        const int n_kv = (kv_len + kBN - 1) / kBN;
        const int j0 = first_key_tile(q_start, kv_start);
        mbar_wait(bar(dqQEmpty), (uc & 1) ^ 1, s_abort);
        mbar_expect_tx(bar(dqQFull), 2 * L::kTileBytes);
#pragma unroll
        for (int b = 0; b < L::kBoxes; ++b) {
          tma_load_2d(sbase + L::kQ + b * L::kBoxBytes, &tm_q, h * D + b * 64, q_start, bar(dqQFull));
          tma_load_2d(sbase + L::kdO + b * L::kBoxBytes, &tm_do, h * D + b * 64, q_start, bar(dqQFull));
        }
        for (int j = j0; j < n_kv; ++j, ++gk) {
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
      for (;; ++uc) {
        mbar_wait(bar(dqUnitFull0 + uc % kUnitRing), (uc / kUnitRing) & 1, s_abort);
        const int u = s_unit[uc % kUnitRing];
        if (u >= n_units || *s_abort) break;
        const int4 it = items[order[u / Hq]];
        const int n_kv = (it.w + kBN - 1) / kBN;
        const int j0 = first_key_tile(it.x, it.z);
        mbar_wait(bar(dqQtReady), uc & 1, s_abort);
        if (gk > 0) mbar_wait(bar(dqSRead), (gk - 1) & 1, s_abort);   // S of the previous step read
        tc_fence_after();
        issue_s(gk);
        issue_dp(gk);
        for (int j = j0; j < n_kv; ++j, ++gk) {
          const int ks = gk % L::kKStages;
          const uint32_t k_lo = desc_lo(sbase + L::kK0 + ks * L::kTileBytes, L::kBoxBytes);
          const bool more = (j + 1 < n_kv);
          if (more) {   // the single S buffer is free as soon as the compute warps have loaded S(j)
            mbar_wait(bar(dqSRead), gk & 1, s_abort);
            issue_s(gk + 1);
          }
          mbar_wait(bar(dqDsReady), gk & 1, s_abort);
          if (j == j0 && uc > 0) mbar_wait(bar(dqRead), (uc - 1) & 1, s_abort);
          tc_fence_after();
          if (leader) {
#pragma unroll
            for (int kk = 0; kk < kBN / 16; ++kk)   // dQ += dS K   (dS of keys 16kk.. : see compute)
              mma_ts(tdQ, tdP + (kk / (kCW / 16)) * kCW + (kk % (kCW / 16)) * 8,
                     desc_from_lo(k_lo + ((kk * 2048) >> 4)), kIdescDQ, (j > j0) | (kk > 0));
            mma_commit(bar(dqKEmpty0 + ks));
          }
          __syncwarp();
          if (more) issue_dp(gk + 1);   // overwrites dP/dS(j) after dQ(j) (same pipe, in order)
        }
        if (leader) mma_commit(bar(dqDone));
        __syncwarp();
      }
    }
  }
  } else if (warp < kMmaWarp) {
    // =============================== compute ===============================================
    setmaxnreg_inc<176>();
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
    auto unit_at = [&](int n) {   // position drawn for this CTA's n-th unit (>= n_units: none)
      mbar_wait(bar(dqUnitFull0 + n % kUnitRing), (n / kUnitRing) & 1, s_abort);
      return static_cast<int>(s_unit[n % kUnitRing]);
    };
    if (unit_at(0) < n_units && !*s_abort) copy_q_do(0);
    for (;; ++uc) {
      const int u = unit_at(uc);
      if (u >= n_units || *s_abort) break;
      const int4 it = items[order[u / Hq]];
      const int h = u % Hq;
      const int q_start = it.x, q_len = it.y, kv_len = it.w;
      const int n_kv = (kv_len + kBN - 1) / kBN;
      const int j0 = first_key_tile(q_start, it.z);
      const int tok = q_start + row;
      const float lse2 = (tok < T) ? lse[(size_t)h * T + tok] * kLog2eWs : 0.f;
      const float dl = (tok < T) ? delta[(size_t)h * T + tok] : 0.f;

      for (int j = j0; j < n_kv; ++j, ++gk) {
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
          // sliding window: keys more than window - 1 before the row
          const int lo = (window > 0) ? (q_start + row - (window - 1) - it.z - j * kBN) : 0;
          if (lo > 0) {
#pragma unroll
            for (int c = 0; c < kCW; ++c)
              if (qd * kCW + c < lo) p[c] = 0.f;
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
        // dS (bf16 pairs, kCW / 2 columns) goes over the first half of this thread's own dP columns:
        // nobody else reads those, so no block-wide barrier is needed
        if (kCW == 64) tmem_st32(tdP + lane_off + qd * kCW, dd);
        else tmem_st16(tdP + lane_off + qd * kCW, dd);
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(bar(dqDsReady));
      }
      // The last S and dP of this unit have been consumed, so Q/dO of the NEXT unit can move into
      // tensor memory now; the issuing warp then starts that unit while this one's dQ is written.
      if (unit_at(uc + 1) < n_units && !*s_abort) copy_q_do(uc + 1);
    }
  } else if (warp >= kDqEpiWarp0) {
    // =============================== dQ writer =============================================
    // One thread per query row: waits for the unit's last contraction, pulls the row of dQ out of
    // tensor memory 32 columns at a time, scales (and rotates back), stores.  The accumulator is
    // released as soon as the last columns are in registers.
    setmaxnreg_dec<96>();
    const int row = tid & 127;
    const uint32_t lane_off = static_cast<uint32_t>((warp & 3) * 32) << 16;
    for (int uc = 0;; ++uc) {
      mbar_wait(bar(dqUnitFull0 + uc % kUnitRing), (uc / kUnitRing) & 1, s_abort);
      const int u = static_cast<int>(s_unit[uc % kUnitRing]);
      if (u >= n_units || *s_abort) break;
      const int4 it = items[order[u / Hq]];
      const int h = u % Hq;
      const int tok = it.x + row;
      mbar_wait(bar(dqDone), uc & 1, s_abort);
      tc_fence_after();
      const bool live = (row < it.y) && (*s_abort == 0);
      GradT* dst = dq + ((size_t)tok * Hq + h) * D;
      if (kRot) {
        // rotate back by -angle: pairs (i, i + D/2), 32 of them at a time
        static_assert(!kRot || D == 128 || D == 64, "rotated path is built for D = 64 and 128");
        const float* cs = rope_angle + (size_t)tok * (D / 2);
#pragma unroll
        for (int c = 0; c < D / 2; c += 32) {
          uint32_t x1[32], x2[32];
          tmem_ld32(tdQ + lane_off + c, x1);
          tmem_ld32(tdQ + lane_off + D / 2 + c, x2);
          tmem_wait_ld();
          if (c + 32 >= D / 2) {
            tc_fence_before();
            mbar_arrive(bar(dqRead));
          }
          if (live) {
            float y1[32], y2[32];
#pragma unroll
            for (int e4 = 0; e4 < 32; e4 += 8) {
              float2 t4[8];
              ld_angles8(cs + c + e4, t4);
#pragma unroll
              for (int k = 0; k < 8; ++k) {
                const int e = e4 + k;
                const float a = __uint_as_float(x1[e]) * scale, bb = __uint_as_float(x2[e]) * scale;
                y1[e] = a * t4[k].x + bb * t4[k].y;
                y2[e] = bb * t4[k].x - a * t4[k].y;
              }
            }
            store_chunk32<GradT>(dst + c, y1);
            store_chunk32<GradT>(dst + D / 2 + c, y2);
          }
        }
      } else {
#pragma unroll
        for (int c = 0; c < D; c += 32) {
          uint32_t x[32];
          tmem_ld32(tdQ + lane_off + c, x);
          tmem_wait_ld();
          if (c + 32 >= D) {
            tc_fence_before();
            mbar_arrive(bar(dqRead));
          }
          if (live) {
            float y[32];
#pragma unroll
            for (int e = 0; e < 32; ++e) y[e] = __uint_as_float(x[e]) * scale;
            store_chunk32<GradT>(dst + c, y);
          }
        }
      }
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
              void* dq, void* dk, void* dv, int T, int Hq, int Hkv, float scale, int window,
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
  const float* table = reinterpret_cast<const float*>(ws + lay.off[PK_WS_ROPE_TABLE]);   // reduced angles
  const int grid = sm_count();
  // the two unit counters (adjacent header slots) start every call at zero
  static_assert(kHdrDqTicket == kHdrBwdTicket + 1, "one memset covers both counters");
  if (cudaMemsetAsync(hdr + kHdrBwdTicket, 0, 2 * sizeof(int32_t), stream) != cudaSuccess)
    return PK_ERR_CUDA;
  {
    TimedLaunch timed(PK_KERNEL_BWD, stream);
    kern_kv<<<grid, kBwdThreads, DkvSmem<D>::kTotal, stream>>>(
        tq, tk, tv, tdo, reinterpret_cast<const int4*>(ws + lay.off[PK_WS_BWD_ITEMS]),
        reinterpret_cast<const int32_t*>(ws + lay.off[PK_WS_BWD_ORDER]), hdr, lse, delta,
        static_cast<GradT*>(dk), static_cast<GradT*>(dv), table, T, Hq, Hkv, scale,
        scale * kLog2eWs, window);
  }
  if (launch_status() != PK_OK) return PK_ERR_CUDA;
  {
    TimedLaunch timed(PK_KERNEL_BWD_DQ, stream);
    kern_q<<<grid, kDqThreads, DqSmem<D>::kTotal, stream>>>(
        tq, tk, tv, tdo, reinterpret_cast<const int4*>(ws + lay.off[PK_WS_FWD_ITEMS]),
        reinterpret_cast<const int32_t*>(ws + lay.off[PK_WS_FWD_ORDER]), hdr, lse, delta,
        static_cast<GradT*>(dq), table, T, Hq, Hkv, scale, scale * kLog2eWs, window);
  }
  return launch_status();
}

}  // namespace

int launch_bwd_ws(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                  const CUtensorMap& tdo, char* ws, const WorkspaceLayout& lay, const float* lse,
                  void* dq, void* dk, void* dv, int T, int Hq, int Hkv, int D, int grad_dtype,
                  float scale, int window, bool rotated, cudaStream_t stream) {
#define PK_BWS(DD, RR, TT)                                                                     \
  return launch_ws<DD, RR, TT>(tq, tk, tv, tdo, ws, lay, lse, dq, dk, dv, T, Hq, Hkv, scale, \
                               window, stream)
  if (D == 128) {
    if (rotated) {
      if (grad_dtype == PK_BF16) PK_BWS(128, true, __nv_bfloat16); else PK_BWS(128, true, float);
    } else {
      if (grad_dtype == PK_BF16) PK_BWS(128, false, __nv_bfloat16); else PK_BWS(128, false, float);
    }
  }
  if (rotated) {
    if (grad_dtype == PK_BF16) PK_BWS(64, true, __nv_bfloat16); else PK_BWS(64, true, float);
  }
  if (grad_dtype == PK_BF16) PK_BWS(64, false, __nv_bfloat16);
  PK_BWS(64, false, float);
#undef PK_BWS
}

}  // namespace pk
