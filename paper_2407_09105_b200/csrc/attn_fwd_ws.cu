// Warp-specialised forward kernel for sm_100a.  Q and K are read as given (no RoPE, or the caller's
// rotated fp16 copies); any number of query heads per kv head.
//
// One CTA per SM works on TWO query tiles at a time: the same block of <= 128 query rows for two
// adjacent query heads of one kv head (or two query blocks of one head: see FwdUnit).  Both tiles read the same K and V tiles, so each K/V
// tile is brought into shared memory once for both, and while the softmax warps of one tile
// are busy the tensor pipe runs the contractions of the other (ping-pong):
//   warps 0-3   softmax of tile 0 (one thread per query row, whole row in registers)
//   warps 4-7   softmax of tile 1
//   warp  8     issues every tcgen05.mma:  S_t = Q_t K^T  and  O_t += P_t V  (P_t from tensor memory)
//   warp  9     TMA: the two Q tiles per unit, K/V tiles through a 2-stage ring
//   warps 12-15 write O_0 and then O_1 of each unit (one thread per row) while the softmax warps
//               are already in the next unit; warps 10-11 idle.  Registers move from the small
//               roles to the softmax warps at the start (setmaxnreg).
// Tensor memory: [0,128) S_0 / P_0, [128,256) S_1 / P_1, [256,384) O_0, [384,512) O_1.
// The commit that announces S_t(j) also covers O_t += P_t V of step j-1 (same pipe, in order), so
// the softmax warps may rescale O_t in tensor memory as soon as they see S_t(j).
// Units (forward item x head pair, or pair of query blocks x head: see FwdUnit) are drawn from a
// counter in the plan's order (kFwsUnitRing).
// Every wait is bounded.
#include <cuda_bf16.h>

#include "attn_common.cuh"
#include "pk_common.cuh"
#include "sm100_ptx.cuh"
#include "tensor_map.cuh"

namespace pk {
namespace {

using namespace ptx;

constexpr int kFwsThreads = 512;
constexpr int kFwsEpiWarp0 = 12;
constexpr int kFwsMmaWarp = 8;
constexpr int kFwsLoadWarp = 9;
constexpr float kLog2eF = 1.4426950408889634f;
constexpr float kLn2F = 0.6931471805599453f;

// Units are handed out dynamically: the TMA warp draws the next position of the plan's order
// from a counter in the workspace header and publishes it to the other roles through a ring of
// four slots in shared memory (one mbarrier per slot).  The order keeps an example's units
// together (they share K/V tiles in L2) and drawing from it keeps every CTA busy to the end.
// No role can fall four units behind the TMA warp: it waits for the previous unit's Q tiles to
// be released before it loads the next one's.
constexpr int kFwsUnitRing = 4;

template <int D>
struct FwsSmem {
  static constexpr int kBoxBytes = 128 * 128;
  static constexpr int kBoxes = D / 64;
  static constexpr int kTileBytes = kBoxBytes * kBoxes;
  static constexpr int kQ0 = 0;                              // Q tile of head pair member 0, then 1
  static constexpr int kKV0 = 2 * kTileBytes;                // stage s: K then V
  static constexpr int kStageBytes = 2 * kTileBytes;
  static constexpr int kBars = kKV0 + 2 * kStageBytes;
  static constexpr int kMisc = kBars + 24 * 8;               // tmem base, abort flag, unit ring
  static constexpr int kInvL = kMisc + 16 + 4 * kFwsUnitRing;   // [2][128] floats: 1 / row sum
  static constexpr int kTotal = kInvL + 1024;
};

enum FwsBar {
  fQFull = 0, fQEmpty, fKvFull0, fKvFull1, fKvEmpty0, fKvEmpty1, fSFull0, fSFull1, fPReady0,
  fPReady1, fOFull0, fOFull1, fORead0, fORead1, fUnitFull0, fUnitFull1, fUnitFull2, fUnitFull3,
  fLReady0, fLReady1,
  fNumBars
};

template <typename OutT>
__device__ __forceinline__ void store_out32(OutT* dst, const uint32_t* r, float scale) {
  float y[32];
#pragma unroll
  for (int e = 0; e < 32; ++e) y[e] = __uint_as_float(r[e]) * scale;
  store_chunk32<OutT>(dst, y);
}

// What the two tiles of a unit are.  With an even number of query heads per kv head they are two
// query heads of one kv head over the same query block.  Otherwise (multi-head attention, odd
// group sizes) they are two consecutive query blocks b-1 and b of one example and one head, which
// also share every K/V tile: the unit runs the b+1 key steps of block b, and block b-1 sees its
// diagonal one step earlier and nothing in the last step.  Blocks are paired from the end of the
// example, so a block is left over only when the count is odd, and then it is block 0 (one key
// step), which runs with a copy of itself as tile 0 whose results are not stored.
struct FwdUnit {
  int h[2], q_start[2], q_len[2], diag[2];   // per tile: head, rows, rows to store, diagonal step
  int g, kv_start, n_kv;
  int j0;                                    // first key step (> 0 only with a sliding window)
};
__device__ __forceinline__ FwdUnit decode_fwd_unit(int u, const int4* __restrict__ items,
                                                   const int32_t* __restrict__ order, int Hq,
                                                   int G, bool pair_blocks, int window) {
  FwdUnit w;
  if (!pair_blocks) {
    const int pairs = Hq / 2;
    const int4 it = items[order[u / pairs]];
    const int h0 = (u % pairs) * 2;
    w.n_kv = (it.w + kBN - 1) / kBN;
    w.kv_start = it.z;
    w.g = h0 / G;
#pragma unroll
    for (int t = 0; t < 2; ++t) {
      w.h[t] = h0 + t; w.q_start[t] = it.x; w.q_len[t] = it.y; w.diag[t] = w.n_kv - 1;
    }
  } else {
    const int4 it = items[order[u / Hq]];
    const int h = u % Hq;
    const int b = (it.x - it.z) / kBM;          // block index inside the example
    w.n_kv = b + 1;
    w.kv_start = it.z;
    w.g = h / G;
    w.h[0] = w.h[1] = h;
    w.q_start[1] = it.x; w.q_len[1] = it.y; w.diag[1] = b;
    if (b >= 1) { w.q_start[0] = it.x - kBM; w.q_len[0] = kBM; w.diag[0] = b - 1; }
    else        { w.q_start[0] = it.x;       w.q_len[0] = 0;   w.diag[0] = 0; }
  }
  // sliding window: the first row of tile 0 reaches back window - 1 keys; whole key tiles
  // before that are skipped (rows further down see even less of them: masked in the softmax)
  const int reach = w.q_start[0] - (window - 1) - w.kv_start;
  w.j0 = (window > 0 && reach > 0) ? reach / kBN : 0;
  return w;
}
// block-pair mode: item n leads a unit when an even number of blocks follows it in its example
// (the backward item of the same index holds the rows from this block to the example's end)
__device__ __forceinline__ bool leads_block_pair(int u, const int4* __restrict__ bwd_items,
                                                 const int32_t* __restrict__ order, int Hq) {
  const int4 bi = bwd_items[order[u / Hq]];
  return (((bi.w + kBM - 1) / kBM - 1) & 1) == 0;
}

template <int D, bool kRot, typename OutT>
__global__ void __launch_bounds__(kFwsThreads, 1)
attn_fwd_ws_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                   const __grid_constant__ CUtensorMap tm_v, const int4* __restrict__ items,
                   const int4* __restrict__ bwd_items, const int32_t* __restrict__ order,
                   int32_t* hdr, OutT* __restrict__ out, float* __restrict__ lse, int T, int Hq,
                   int Hkv, float scale_log2, int window) {
  using L = FwsSmem<D>;
  extern __shared__ __align__(1024) uint8_t smem[];
  const uint32_t sbase = smem_u32(smem);
  const uint32_t bars = sbase + L::kBars;
  auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };
  volatile int* s_tmem = reinterpret_cast<volatile int*>(smem + L::kMisc);
  volatile int* s_abort = s_tmem + 1;
  volatile int* s_unit = s_tmem + 4;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (tid == 0) {
    mbar_init(bar(fQFull), 1);
    mbar_init(bar(fQEmpty), 1);
    mbar_init(bar(fKvFull0), 1);
    mbar_init(bar(fKvFull1), 1);
    mbar_init(bar(fKvEmpty0), 1);
    mbar_init(bar(fKvEmpty1), 1);
    mbar_init(bar(fSFull0), 1);
    mbar_init(bar(fSFull1), 1);
    mbar_init(bar(fPReady0), 128);
    mbar_init(bar(fPReady1), 128);
    mbar_init(bar(fOFull0), 1);
    mbar_init(bar(fOFull1), 1);
    mbar_init(bar(fORead0), 128);
    mbar_init(bar(fORead1), 128);
    mbar_init(bar(fLReady0), 128);
    mbar_init(bar(fLReady1), 128);
    for (int i = 0; i < kFwsUnitRing; ++i) mbar_init(bar(fUnitFull0 + i), 1);
    fence_mbar_init();
    *s_abort = ((sbase & 1023u) != 0) ? 1 : 0;
  }
  if (warp == kFwsMmaWarp) {
    tmem_alloc(smem_u32(const_cast<int*>(s_tmem)), 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = static_cast<uint32_t>(*s_tmem);

  const int G = Hq / Hkv;
  const bool pair_blocks = (G % 2) != 0;
  const bool plan_ok = (hdr[PK_HDR_PLAN_T] == T);
  if (!plan_ok && blockIdx.x == 0 && tid == 0) set_status(hdr, PK_ERR_NO_PLAN, T);
  const int n_units = plan_ok ? hdr[PK_HDR_N_ITEMS] * (pair_blocks ? Hq : Hq / 2) : 0;

  float* s_invl = reinterpret_cast<float*>(smem + L::kInvL);
  // Register budget: 512 threads start with 128 each; every warpgroup changes its allowance at the
  // top of its own branch.  The two decreases free 128 * (88 + 32) = 15 360 registers without
  // waiting for anything, the increases take 256 * 56 = 14 336: they cannot block for good.
  if ((warp >> 2) == (kFwsMmaWarp >> 2)) {
  setmaxnreg_dec<40>();
  if (warp == kFwsLoadWarp) {
    // =============================== loader ===============================================
    if (lane == 0) {
      prefetch_tensormap(&tm_q);
      prefetch_tensormap(&tm_k);
      prefetch_tensormap(&tm_v);
      int gk = 0, uc = 0;
      for (;; ++uc) {
        int u;
        do {   // in block-pair mode only the leading block of a pair becomes a unit
          u = atomicAdd(&hdr[kHdrFwdTicket], 1);
        } while (u < n_units && pair_blocks && !leads_block_pair(u, bwd_items, order, Hq));
        s_unit[uc % kFwsUnitRing] = u;
        mbar_arrive(bar(fUnitFull0 + uc % kFwsUnitRing));
        if (u >= n_units || *s_abort) break;
        const FwdUnit w = decode_fwd_unit(u, items, order, Hq, G, pair_blocks, window);
        const int g = w.g, kv_start = w.kv_start, n_kv = w.n_kv, j0 = w.j0;
        mbar_wait(bar(fQEmpty), (uc & 1) ^ 1, s_abort);
        mbar_expect_tx(bar(fQFull), 2 * L::kTileBytes);
#pragma unroll
        for (int t = 0; t < 2; ++t)
#pragma unroll
          for (int b = 0; b < L::kBoxes; ++b)
            tma_load_2d(sbase + L::kQ0 + t * L::kTileBytes + b * L::kBoxBytes, &tm_q,
                        w.h[t] * D + b * 64, w.q_start[t], bar(fQFull));
        for (int j = j0; j < n_kv; ++j, ++gk) {
          const int st = gk & 1;
          const uint32_t sK = sbase + L::kKV0 + st * L::kStageBytes, sV = sK + L::kTileBytes;
          mbar_wait(bar(fKvEmpty0 + st), ((gk >> 1) & 1) ^ 1, s_abort);
          mbar_expect_tx(bar(fKvFull0 + st), 2 * L::kTileBytes);
#pragma unroll
          for (int b = 0; b < L::kBoxes; ++b) {
            tma_load_2d(sK + b * L::kBoxBytes, &tm_k, g * D + b * 64, kv_start + j * kBN,
                        bar(fKvFull0 + st));
            tma_load_2d(sV + b * L::kBoxBytes, &tm_v, g * D + b * 64, kv_start + j * kBN,
                        bar(fKvFull0 + st));
          }
        }
      }
    }
    __syncwarp();
  } else if (warp == kFwsMmaWarp) {
    // =============================== MMA issuer ===========================================
    // The whole warp walks the schedule (so that addresses and descriptors stay warp-uniform);
    // one elected lane issues the tensor-core instructions.
    {
      // kRot: q and k are the rotated fp16 copies in the workspace
      constexpr uint32_t kQKFmt = kRot ? kFmtF16 : kFmtBF16;
      constexpr uint32_t kIdescQK = make_idesc(128, 128, kQKFmt, kQKFmt, 0, 0);
      constexpr uint32_t kIdescPV = make_idesc(128, D, kFmtBF16, kFmtBF16, 0, 1);
      const bool leader = elect_one();
      int gk = 0, uc = 0;
      auto issue_s = [&](int t, int st) {
        const uint32_t q_lo = desc_lo(sbase + L::kQ0 + t * L::kTileBytes, 16);
        const uint32_t k_lo = desc_lo(sbase + L::kKV0 + st * L::kStageBytes, 16);
        if (leader) {
#pragma unroll
          for (int kk = 0; kk < D / 16; ++kk) {
            const uint32_t off = ((kk / 4) * L::kBoxBytes + (kk % 4) * 32) >> 4;
            mma_ss(tmem + t * 128, desc_from_lo(q_lo + off), desc_from_lo(k_lo + off), kIdescQK,
                   kk > 0);
          }
          mma_commit(bar(fSFull0 + t));
        }
        __syncwarp();
      };
      for (;; ++uc) {
        mbar_wait(bar(fUnitFull0 + uc % kFwsUnitRing), (uc / kFwsUnitRing) & 1, s_abort);
        const int u = s_unit[uc % kFwsUnitRing];
        if (u >= n_units || *s_abort) break;
        const FwdUnit w = decode_fwd_unit(u, items, order, Hq, G, pair_blocks, window);
        const int n_kv = w.n_kv, j0 = w.j0;
        mbar_wait(bar(fQFull), uc & 1, s_abort);
        mbar_wait(bar(fKvFull0 + (gk & 1)), (gk >> 1) & 1, s_abort);
        tc_fence_after();
        issue_s(0, gk & 1);
        issue_s(1, gk & 1);
        // the Q tiles are read for the last time by the unit's last S, issued one step before its
        // end: releasing them there lets the next unit's Q arrive while the last P V still run
        if (j0 + 1 == n_kv && leader) mma_commit(bar(fQEmpty));
        for (int j = j0; j < n_kv; ++j, ++gk) {
          const int st = gk & 1;
          const uint32_t v_lo =
              desc_lo(sbase + L::kKV0 + st * L::kStageBytes + L::kTileBytes, L::kBoxBytes);
          const bool more = (j + 1 < n_kv);
#pragma unroll
          for (int t = 0; t < 2; ++t) {
            mbar_wait(bar(fPReady0 + t), gk & 1, s_abort);
            if (j == j0 && uc > 0) mbar_wait(bar(fORead0 + t), (uc - 1) & 1, s_abort);
            tc_fence_after();
            if (leader) {
#pragma unroll
              for (int kk = 0; kk < kBN / 16; ++kk)   // O_t += P_t V
                mma_ts(tmem + 256 + t * 128, tmem + t * 128 + kk * 8,
                       desc_from_lo(v_lo + ((kk * 2048) >> 4)), kIdescPV, (j > j0) | (kk > 0));
              if (t == 1) mma_commit(bar(fKvEmpty0 + st));
              if (!more) mma_commit(bar(fOFull0 + t));
            }
            __syncwarp();
            if (more) {                              // S_t(j+1): P_t(j) was consumed just above
              if (t == 0) {
                mbar_wait(bar(fKvFull0 + ((gk + 1) & 1)), ((gk + 1) >> 1) & 1, s_abort);
                tc_fence_after();
              }
              issue_s(t, (gk + 1) & 1);
              if (t == 1 && j + 2 == n_kv && leader) mma_commit(bar(fQEmpty));
            }
          }
        }
        __syncwarp();
      }
    }
  }
  } else if (warp < kFwsMmaWarp) {
    // =============================== softmax (warps 0-3: tile 0, warps 4-7: tile 1) =======
    setmaxnreg_inc<184>();
    const int t = tid >> 7;
    const int row = tid & 127;
    const uint32_t lane_off = static_cast<uint32_t>((warp & 3) * 32) << 16;
    const uint32_t tS = tmem + t * 128 + lane_off;
    const uint32_t tO = tmem + 256 + t * 128 + lane_off;
    int gk = 0, uc = 0;
    for (;; ++uc) {
      mbar_wait(bar(fUnitFull0 + uc % kFwsUnitRing), (uc / kFwsUnitRing) & 1, s_abort);
      const int u = s_unit[uc % kFwsUnitRing];
      if (u >= n_units || *s_abort) break;
      const FwdUnit w = decode_fwd_unit(u, items, order, Hq, G, pair_blocks, window);
      const int h = w.h[t], q_start = w.q_start[t], q_len = w.q_len[t], diag = w.diag[t];
      const int n_kv = w.n_kv, j0 = w.j0;
      float m_run = -INFINITY, l_run = 0.f;
      for (int j = j0; j < n_kv; ++j, ++gk) {
        mbar_wait(bar(fSFull0 + t), gk & 1, s_abort);
        tc_fence_after();
        uint32_t s[128];
#pragma unroll
        for (int c = 0; c < 4; ++c) tmem_ld32(tS + c * 32, s + c * 32);
        tmem_wait_ld();
        // sliding window: keys more than window - 1 before the row are masked too
        const int lo = (window > 0) ? (q_start + row - (window - 1) - w.kv_start - j * kBN) : 0;
        if (j >= diag || lo > 0) {   // diagonal tile: keys after the query row are masked; a tile
                                     // past the diagonal (block-pair mode, tile 0, last step) entirely
          const int first_masked = (j == diag) ? row + 1 : (j > diag ? 0 : 128);
#pragma unroll
          for (int c = 0; c < 128; ++c)
            if (c >= first_masked || c < lo) s[c] = 0xff800000u;   // -inf
        }
        float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};   // independent chains
#pragma unroll
        for (int c = 0; c < 128; c += 4) {
#pragma unroll
          for (int e = 0; e < 4; ++e) mx4[e] = fmaxf(mx4[e], __uint_as_float(s[c + e]));
        }
        const float row_m = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * scale_log2;
        // the reference maximum only moves when the row maximum exceeds it by more than 2^8, so
        // that the running O rarely needs rescaling; P then stays below 2^8
        const bool changed = row_m > m_run + 8.f;          // true on the first tile (m_run = -inf)
        const float m_new = changed ? row_m : m_run;
        const float alpha = changed ? fast_exp2(m_run - m_new) : 1.f;   // 0 on the first tile
        // a row that has seen nothing yet (possible only with a sliding window) keeps the maximum
        // at -inf; the exponentials then use 0 so that they come out as exp2(-inf) = 0, not NaN
        const float m_sub = (m_new == -INFINITY) ? 0.f : m_new;
        float sum4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int half = 0; half < 2; ++half) {   // P leaves in two 64-column pieces to bound registers
          uint32_t p[32];
#pragma unroll
          for (int c = 0; c < 64; c += 4) {
            const float p0 = fast_exp2(fmaf(__uint_as_float(s[half * 64 + c]), scale_log2, -m_sub));
            const float p1 = fast_exp2(fmaf(__uint_as_float(s[half * 64 + c + 1]), scale_log2, -m_sub));
            const float p2 = fast_exp2(fmaf(__uint_as_float(s[half * 64 + c + 2]), scale_log2, -m_sub));
            const float p3 = fast_exp2(fmaf(__uint_as_float(s[half * 64 + c + 3]), scale_log2, -m_sub));
            sum4[0] += p0; sum4[1] += p1; sum4[2] += p2; sum4[3] += p3;
            p[c >> 1] = pack_bf16x2(p0, p1);
            p[(c >> 1) + 1] = pack_bf16x2(p2, p3);
          }
          tmem_st32(tS + half * 32, p);
        }
        l_run = l_run * alpha + ((sum4[0] + sum4[1]) + (sum4[2] + sum4[3]));
        m_run = m_new;
        // O_t of step j-1 is complete (its contraction precedes S_t(j) on the tensor pipe)
        if (j > j0 && __any_sync(0xffffffffu, changed)) {
#pragma unroll
          for (int c = 0; c < D / 32; ++c) {
            uint32_t o[32];
            tmem_ld32(tO + c * 32, o);
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < 32; ++e) o[e] = __float_as_uint(__uint_as_float(o[e]) * alpha);
            tmem_st32(tO + c * 32, o);
          }
        }
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(bar(fPReady0 + t));
      }
      // ---- lse from here; O_t / l is written by the writer warps, which get 1 / l ------------
      if ((row < q_len) && (*s_abort == 0))
        lse[(size_t)h * T + q_start + row] = (m_run + log2f(l_run)) * kLn2F;
      s_invl[t * 128 + row] = 1.f / l_run;
      mbar_arrive(bar(fLReady0 + t));
    }
  } else if (warp >= kFwsEpiWarp0) {
    // =============================== O writer ==============================================
    // One thread per query row, tile 0 then tile 1 of every unit: waits for the tile's last
    // contraction, pulls the row out of tensor memory 32 columns at a time, scales by 1 / l,
    // stores.  The accumulator is released as soon as its last columns are in registers.
    setmaxnreg_dec<96>();
    const int row = tid & 127;
    const uint32_t lane_off = static_cast<uint32_t>((warp & 3) * 32) << 16;
    for (int uc = 0;; ++uc) {
      mbar_wait(bar(fUnitFull0 + uc % kFwsUnitRing), (uc / kFwsUnitRing) & 1, s_abort);
      const int u = s_unit[uc % kFwsUnitRing];
      if (u >= n_units || *s_abort) break;
      const FwdUnit w = decode_fwd_unit(u, items, order, Hq, G, pair_blocks, window);
#pragma unroll
      for (int t = 0; t < 2; ++t) {
        mbar_wait(bar(fLReady0 + t), uc & 1, s_abort);
        const float inv_l = s_invl[t * 128 + row];
        mbar_wait(bar(fOFull0 + t), uc & 1, s_abort);
        tc_fence_after();
        const bool live = (row < w.q_len[t]) && (*s_abort == 0);
        const uint32_t tO = tmem + 256 + t * 128 + lane_off;
        OutT* orow = out + ((size_t)(w.q_start[t] + row) * Hq + w.h[t]) * D;
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
          uint32_t o[32];
          tmem_ld32(tO + c * 32, o);
          tmem_wait_ld();
          if (c == D / 32 - 1) {
            tc_fence_before();
            mbar_arrive(bar(fORead0 + t));
          }
          if (live) store_out32<OutT>(orow + c * 32, o, inv_l);
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (*s_abort != 0 && tid == 0) set_status(hdr, PK_ERR_TIMEOUT, 5);
  if (warp == kFwsMmaWarp) tmem_dealloc(tmem, 512);
}

template <int D, bool kRot, typename OutT>
int launch_fws(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, char* ws,
               const WorkspaceLayout& lay, void* out, float* lse, int T, int Hq, int Hkv,
               float scale, int window, cudaStream_t stream) {
  auto kern = attn_fwd_ws_kernel<D, kRot, OutT>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           FwsSmem<D>::kTotal) != cudaSuccess)
    return PK_ERR_CUDA;
  int32_t* hdr = reinterpret_cast<int32_t*>(ws + lay.off[PK_WS_HEADER]);
  if (cudaMemsetAsync(hdr + kHdrFwdTicket, 0, sizeof(int32_t), stream) != cudaSuccess)
    return PK_ERR_CUDA;
  TimedLaunch timed(PK_KERNEL_FWD, stream);
  kern<<<sm_count(), kFwsThreads, FwsSmem<D>::kTotal, stream>>>(
      tq, tk, tv, reinterpret_cast<const int4*>(ws + lay.off[PK_WS_FWD_ITEMS]),
      reinterpret_cast<const int4*>(ws + lay.off[PK_WS_BWD_ITEMS]),
      reinterpret_cast<const int32_t*>(ws + lay.off[PK_WS_FWD_ORDER]), hdr,
      static_cast<OutT*>(out), lse, T, Hq, Hkv, scale * kLog2eF, window);
  return launch_status();
}

}  // namespace

int launch_fwd_ws(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, char* ws,
                  const WorkspaceLayout& lay, void* out, float* lse, int T, int Hq, int Hkv, int D,
                  int out_dtype, float scale, int window, bool rotated, cudaStream_t stream) {
#define PK_FWS(DD, RR, TT) \
  return launch_fws<DD, RR, TT>(tq, tk, tv, ws, lay, out, lse, T, Hq, Hkv, scale, window, stream)
  if (D == 128) {
    if (rotated) {
      if (out_dtype == PK_BF16) PK_FWS(128, true, __nv_bfloat16); else PK_FWS(128, true, float);
    } else {
      if (out_dtype == PK_BF16) PK_FWS(128, false, __nv_bfloat16); else PK_FWS(128, false, float);
    }
  }
  if (rotated) {
    if (out_dtype == PK_BF16) PK_FWS(64, true, __nv_bfloat16); else PK_FWS(64, true, float);
  }
  if (out_dtype == PK_BF16) PK_FWS(64, false, __nv_bfloat16);
  PK_FWS(64, false, float);
#undef PK_FWS
}

}  // namespace pk
