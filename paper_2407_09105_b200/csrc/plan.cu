// Boundary recovery and planning: position_ids -> cu_seqlens, example count, longest
// example, per-tile forward/backward work lists and their longest-first orders.
// (Paragraph after Table 1: the example count and cu_seq_len come from position_ids.)
// Integer work only; one CTA walks the stream in chunks of 1024 tokens, so there is no
// host round trip and no inter-CTA dependency.
#include "pk_common.cuh"

namespace pk {
namespace {

constexpr int kPlanThreads = 1024;

// Exclusive prefix sum of v over the CTA; *total receives the CTA-wide sum.
__device__ __forceinline__ int block_exclusive_scan(int v, int* total, int* sm /* [33] */) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int x = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int y = __shfl_up_sync(0xffffffffu, x, o);
    if (lane >= o) x += y;
  }
  if (lane == 31) sm[warp] = x;
  __syncthreads();
  if (warp == 0) {
    int w = sm[lane], s = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int y = __shfl_up_sync(0xffffffffu, s, o);
      if (lane >= o) s += y;
    }
    sm[lane] = s - w;
    if (lane == 31) sm[32] = s;
  }
  __syncthreads();
  const int res = x - v + sm[warp];
  *total = sm[32];
  __syncthreads();
  return res;
}

__global__ void __launch_bounds__(kPlanThreads)
plan_kernel(const int32_t* __restrict__ pos, int T,
            int32_t* __restrict__ cu_out, int32_t* __restrict__ nex_out,
            int32_t* __restrict__ max_out,
            int32_t* hdr, int32_t* cu, int32_t* ex_base,
            int4* fwd_items, int4* bwd_items, int32_t* fwd_order, int32_t* bwd_order,
            int32_t* hist, int hist_stride) {
  __shared__ int sscan[33];
  __shared__ int s_max, s_bad;
  const int tid = threadIdx.x;
  const int lane = tid & 31, warp = tid >> 5;

  if (tid < kHeaderInts) hdr[tid] = (tid == PK_HDR_PLAN_T) ? -1 : 0;
  if (tid == 0) { s_max = 0; s_bad = 0; }
  __syncthreads();

  // ---- A: example starts -> cu ------------------------------------------------------
  // Eight consecutive tokens per thread and round: the loop is bound by the latency of its loads
  // and barriers, not by their number, so fewer, fatter rounds are what shortens it.
  constexpr int kPer = 8;
  int carry = 0;
  for (int base = 0; base < T; base += kPlanThreads * kPer) {
    const int t0 = base + tid * kPer;
    int p[kPer + 1];
    p[0] = (t0 > 0 && t0 - 1 < T) ? pos[t0 - 1] : 0;
#pragma unroll
    for (int i = 0; i < kPer; ++i) p[i + 1] = (t0 + i < T) ? pos[t0 + i] : 0;
    unsigned flags = 0;
#pragma unroll
    for (int i = 0; i < kPer; ++i) {
      const int t = t0 + i;
      if (t < T) {
        if (p[i + 1] < 0) { set_status(hdr, PK_ERR_BAD_POSIDS, t); s_bad = 1; }
        if (t == 0 || p[i + 1] <= p[i]) flags |= 1u << i;
      }
    }
    int tot;
    const int ex = block_exclusive_scan(__popc(flags), &tot, sscan);
    int o = carry + ex;
#pragma unroll
    for (int i = 0; i < kPer; ++i)
      if (flags & (1u << i)) cu[o++] = t0 + i;
    carry += tot;
  }
  const int E = carry;
  for (int i = E + tid; i <= T; i += kPlanThreads) cu[i] = T;
  __syncthreads();
  const bool bad = (s_bad != 0);

  // ---- B: items per example, longest example ---------------------------------------
  int my_max = 0;
  carry = 0;
  for (int base = 0; base < E; base += kPlanThreads) {
    const int e = base + tid;
    int n = 0;
    if (e < E) {
      const int L = cu[e + 1] - cu[e];
      my_max = max(my_max, L);
      n = (L + kBM - 1) / kBM;
    }
    int tot;
    const int ex = block_exclusive_scan(n, &tot, sscan);
    if (e < E) ex_base[e] = carry + ex;
    carry += tot;
  }
  const int N = carry;
  if (tid == 0) ex_base[E] = N;
  if (my_max > 0) atomicMax(&s_max, my_max);
  __syncthreads();
  const int max_len = s_max;
  const int kmax = (max_len + kBM - 1) / kBM;   // largest key of either list

  int32_t* hist_f = hist;
  int32_t* hist_b = hist + hist_stride;
  for (int i = tid; i <= kmax + 1; i += kPlanThreads) { hist_f[i] = 0; hist_b[i] = 0; }
  __syncthreads();

  // ---- C: the lists (one thread per item, example found by binary search) -----------
  for (int n = tid; n < N; n += kPlanThreads) {
    int lo = 0, hi = E - 1;
    while (lo < hi) {
      const int mid = (lo + hi + 1) >> 1;
      if (ex_base[mid] <= n) lo = mid; else hi = mid - 1;
    }
    const int e = lo;
    const int s = cu[e], L = cu[e + 1] - s;
    const int b = n - ex_base[e];
    const int blk_len = min(kBM, L - b * kBM);
    fwd_items[n] = make_int4(s + b * kBM, blk_len, s, b * kBM + blk_len);
    bwd_items[n] = make_int4(s + b * kBN, blk_len, s + b * kBN, L - b * kBN);
    // sort key of both lists: the tile count of the item's EXAMPLE (see phase E)
    atomicAdd(&hist_f[(L + kBM - 1) / kBM], 1);
    atomicAdd(&hist_b[(L + kBM - 1) / kBM], 1);
  }
  __syncthreads();

  // ---- D: cursors = number of items with a larger key (descending order) ------------
  for (int pass = 0; pass < 2; ++pass) {
    int32_t* h = pass == 0 ? hist_f : hist_b;
    int c = 0;
    for (int base = 0; base < kmax; base += kPlanThreads) {
      const int idx = base + tid;
      const int key = kmax - idx;
      const int v = (idx < kmax) ? h[key] : 0;
      int tot;
      const int ex = block_exclusive_scan(v, &tot, sscan);
      if (idx < kmax) h[key] = c + ex;
      c += tot;
    }
  }
  __syncthreads();

  // ---- E: stable placement: chunks in order, warps of a chunk in order --------------
  // Items are ordered by descending tile count of their example and, inside an example, by
  // block: long examples first (their items carry the most work) while the units that run at
  // the same time belong to the same example and share its K/V (or Q/dO) tiles in L2.
  for (int base = 0; base < N; base += kPlanThreads) {
    const int n = base + tid;
    int kf = 0, kb = 0;
    if (n < N) {
      int lo = 0, hi = E - 1;
      while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (ex_base[mid] <= n) lo = mid; else hi = mid - 1;
      }
      kf = kb = ex_base[lo + 1] - ex_base[lo];
    }
    for (int w = 0; w < kPlanThreads / 32; ++w) {
      if (warp == w) {
#pragma unroll
        for (int pass = 0; pass < 2; ++pass) {
          const int key = pass == 0 ? kf : kb;
          int32_t* h = pass == 0 ? hist_f : hist_b;
          int32_t* order = pass == 0 ? fwd_order : bwd_order;
          const unsigned peers = __match_any_sync(0xffffffffu, key);
          const int rank = __popc(peers & ((1u << lane) - 1u));
          const int leader = __ffs(peers) - 1;
          int first = 0;
          if (lane == leader && key > 0) first = atomicAdd(&h[key], __popc(peers));
          first = __shfl_sync(0xffffffffu, first, leader);
          if (key > 0) order[first + rank] = n;
        }
      }
      __syncthreads();
    }
  }

  // ---- F: results --------------------------------------------------------------------
  if (cu_out != nullptr)
    for (int i = tid; i <= T; i += kPlanThreads) cu_out[i] = cu[i];
  if (tid == 0) {
    hdr[PK_HDR_N_EXAMPLES] = E;
    hdr[PK_HDR_MAX_SEQLEN] = max_len;
    hdr[PK_HDR_N_ITEMS] = bad ? 0 : N;
    hdr[PK_HDR_PLAN_T] = T;
    if (nex_out != nullptr) *nex_out = E;
    if (max_out != nullptr) *max_out = max_len;
  }
}

}  // namespace

int plan_launch(const int32_t* position_ids, int32_t T, int32_t* cu_seqlens, int32_t* n_examples,
                int32_t* max_seqlen, void* workspace, const WorkspaceLayout& lay,
                cudaStream_t stream) {
  char* ws = static_cast<char*>(workspace);
  TimedLaunch timed(PK_KERNEL_PLAN, stream);
  plan_kernel<<<1, kPlanThreads, 0, stream>>>(
      position_ids, T, cu_seqlens, n_examples, max_seqlen,
      reinterpret_cast<int32_t*>(ws + lay.off[PK_WS_HEADER]),
      reinterpret_cast<int32_t*>(ws + lay.off_cu),
      reinterpret_cast<int32_t*>(ws + lay.off_ex_base),
      reinterpret_cast<int4*>(ws + lay.off[PK_WS_FWD_ITEMS]),
      reinterpret_cast<int4*>(ws + lay.off[PK_WS_BWD_ITEMS]),
      reinterpret_cast<int32_t*>(ws + lay.off[PK_WS_FWD_ORDER]),
      reinterpret_cast<int32_t*>(ws + lay.off[PK_WS_BWD_ORDER]),
      reinterpret_cast<int32_t*>(ws + lay.off_hist), (int)lay.hist_stride);
  return launch_status();
}

}  // namespace pk

extern "C" int pk_seqlens_from_posids(const int32_t* position_ids, int32_t T,
                                      int32_t* cu_seqlens, int32_t* n_examples,
                                      int32_t* max_seqlen, void* workspace,
                                      size_t workspace_bytes, void* stream) {
  if (T < 0 || workspace == nullptr || cu_seqlens == nullptr) return PK_ERR_INVALID_ARG;
  if (T > 0 && position_ids == nullptr) return PK_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return PK_ERR_INVALID_ARG;
  // the plan part of the layout does not depend on the head shape
  const pk::WorkspaceLayout lay = pk::workspace_layout(T, 1, 1, 64);
  if (workspace_bytes < lay.plan_total) return PK_ERR_WORKSPACE;
  return pk::plan_launch(position_ids, T, cu_seqlens, n_examples, max_seqlen, workspace, lay,
                         static_cast<cudaStream_t>(stream));
}

// ---------------------------------------------------------------------------------------
// Boundary recovery without a caller-provided workspace and without any allocation.
// ---------------------------------------------------------------------------------------
namespace pk {
namespace {

// Upper bound of WorkspaceLayout::plan_total for T <= PK_NOALLOC_MAX_TOKENS: header, two
// item lists (16 B per entry), two orders, cu_seqlens copy, per-example bases, sort cursors,
// plus one 256-byte alignment gap per section.
constexpr size_t kNoAllocBytes =
    (size_t)PK_NOALLOC_MAX_TOKENS * (16 + 16 + 4 + 4 + 4 + 4) + 8 * (PK_NOALLOC_MAX_TOKENS / 128 + 4) +
    16 + 10 * 256;

// Scratch of the no-allocation entry point.  One copy lives on every GPU that loads the
// library, from load until the process exits.  In host code this name is only a handle for
// cudaGetSymbolAddress; kernels must be given the address that call returns.
static __device__ __align__(256) unsigned char g_noalloc_plan_scratch[kNoAllocBytes];

constexpr int kMaxDevices = 64;
void* g_noalloc_ptr[kMaxDevices] = {};

// Device address of the scratch array on the current device (looked up once per device).
int noalloc_scratch(void** out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return PK_ERR_CUDA;
  if (g_noalloc_ptr[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_noalloc_plan_scratch) != cudaSuccess || p == nullptr)
      return PK_ERR_CUDA;
    g_noalloc_ptr[dev] = p;
  }
  *out = g_noalloc_ptr[dev];
  return PK_OK;
}

}  // namespace
}  // namespace pk

extern "C" int pk_seqlens_from_posids_noalloc(const int32_t* position_ids, int32_t T,
                                              int32_t* cu_seqlens, int32_t* n_examples,
                                              int32_t* max_seqlen, void* stream) {
  if (T < 0 || cu_seqlens == nullptr) return PK_ERR_INVALID_ARG;
  if (T > 0 && position_ids == nullptr) return PK_ERR_INVALID_ARG;
  if (T > PK_NOALLOC_MAX_TOKENS) return PK_ERR_TOO_LARGE;
  const pk::WorkspaceLayout lay = pk::workspace_layout(T, 1, 1, 64);
  if (lay.plan_total > pk::kNoAllocBytes) return PK_ERR_TOO_LARGE;
  void* scratch = nullptr;
  const int rc = pk::noalloc_scratch(&scratch);
  if (rc != PK_OK) return rc;
  // the kernel itself clears the header and the sort cursors it reads, so stale contents
  // of the shared array from an earlier call do not matter
  return pk::plan_launch(position_ids, T, cu_seqlens, n_examples, max_seqlen, scratch, lay,
                         static_cast<cudaStream_t>(stream));
}
