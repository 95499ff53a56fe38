// Steps around the attention path ("next" scope): the padding-free collator of Sec. 3.4 / 3.5 on
// the device (position ids restart per example, first label of an example is ignored), its
// fixed-length variant (the stream cut into packs of msl tokens, Sec. 3.3), and the
// sample-selection baselines of Sec. 3.3 on the host (first-fit-decreasing as in Multipack, and
// first-come-first-served filling).
#include <algorithm>
#include <numeric>
#include <vector>

#include "pk_common.cuh"

namespace pk {
namespace {

// cu[0] = 0, cu[e+1] = cu[e] + lengths[e]; one CTA, chunks of 1024 examples.
__global__ void __launch_bounds__(1024) lengths_scan_kernel(const int32_t* __restrict__ lengths,
                                                            int E, int32_t* __restrict__ cu) {
  __shared__ int warp_sums[33];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  int carry = 0;
  if (tid == 0) cu[0] = 0;
  for (int base = 0; base < E; base += 1024) {
    const int e = base + tid;
    const int v = e < E ? lengths[e] : 0;
    int x = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, x, o);
      if (lane >= o) x += y;
    }
    if (lane == 31) warp_sums[warp] = x;
    __syncthreads();
    if (warp == 0) {
      const int w = warp_sums[lane];
      int s = w;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int y = __shfl_up_sync(0xffffffffu, s, o);
        if (lane >= o) s += y;
      }
      warp_sums[lane] = s - w;
      if (lane == 31) warp_sums[32] = s;
    }
    __syncthreads();
    if (e < E) cu[e + 1] = carry + warp_sums[warp] + x;
    carry += warp_sums[32];
    __syncthreads();
  }
}

// msl > 0: the stream is also cut at every multiple of msl (fixed-length packing, Sec. 3.3): the
// fragment that opens a pack counts as a new example.
__global__ void collate_kernel(const int32_t* __restrict__ input_ids, const int32_t* __restrict__ cu,
                               int E, int T, int msl, int32_t ignore_index,
                               int32_t* __restrict__ position_ids, int32_t* __restrict__ labels) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= T) return;
  int lo = 0, hi = E - 1;                 // largest e with cu[e] <= t
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (cu[mid] <= t) lo = mid; else hi = mid - 1;
  }
  int start = cu[lo];
  if (msl > 0) start = max(start, t - t % msl);
  const int p = t - start;
  position_ids[t] = p;
  if (labels != nullptr) labels[t] = (p == 0) ? ignore_index : input_ids[t];
}


// Padded batch [B][l_max][row_bytes] <-> packed stream [T][row_bytes]; kVec bytes per access.
// kPack: packed[cu[b] + i] = padded[b][i].  Otherwise the reverse, padding rows zero-filled.
// One CTA per destination row (blockIdx.x) and slice of it (blockIdx.y): the row's source is
// looked up once per CTA, and the threads stream the bytes without any index arithmetic.
template <int kVec, bool kPack>
__global__ void __launch_bounds__(256)
rows_move_kernel(const uint8_t* __restrict__ src, const int32_t* __restrict__ cu, int B, int l_max,
                 long long row_bytes, uint8_t* __restrict__ dst) {
  const long long r = blockIdx.x;
  long long from;
  bool copy = true;
  if (kPack) {
    int lo = 0, hi = B - 1;                 // largest b with cu[b] <= r (uniform for the CTA)
    while (lo < hi) {
      const int mid = (lo + hi + 1) >> 1;
      if (cu[mid] <= r) lo = mid; else hi = mid - 1;
    }
    from = (long long)lo * l_max + (r - cu[lo]);
  } else {
    const int b = (int)(r / l_max), i = (int)(r % l_max);
    copy = i < cu[b + 1] - cu[b];
    from = (long long)cu[b] + i;
  }
  const uint8_t* s = src + from * row_bytes;
  uint8_t* d = dst + r * row_bytes;
  const long long chunks = row_bytes / kVec;
  constexpr int kPerThread = 4;
  const long long c0 = ((long long)blockIdx.y * kPerThread) * 256 + threadIdx.x;
#pragma unroll
  for (int k = 0; k < kPerThread; ++k) {
    const long long c = c0 + (long long)k * 256;
    if (c >= chunks) break;
    if (kVec == 16) {
      reinterpret_cast<uint4*>(d)[c] = copy ? reinterpret_cast<const uint4*>(s)[c] : make_uint4(0, 0, 0, 0);
    } else if (kVec == 4) {
      reinterpret_cast<uint32_t*>(d)[c] = copy ? reinterpret_cast<const uint32_t*>(s)[c] : 0u;
    } else {
      d[c] = copy ? s[c] : (uint8_t)0;
    }
  }
}

template <bool kPack>
int rows_move(const void* src, const int32_t* cu, int B, int l_max, int T, long long row_bytes,
              void* dst, cudaStream_t stream) {
  const long long n_rows = kPack ? (long long)T : (long long)B * l_max;
  if (n_rows == 0) return PK_OK;
  if (n_rows > 0x7fffffffLL) return PK_ERR_UNSUPPORTED;
  const uintptr_t a = reinterpret_cast<uintptr_t>(src) | reinterpret_cast<uintptr_t>(dst) |
                      (uintptr_t)row_bytes;
  const int vec = (a & 15) == 0 ? 16 : ((a & 3) == 0 ? 4 : 1);
  const long long slices = (row_bytes / vec + 4 * 256 - 1) / (4 * 256);
  if (slices > 65535) return PK_ERR_UNSUPPORTED;
  const dim3 grid((unsigned)n_rows, (unsigned)slices);
  const auto* s = static_cast<const uint8_t*>(src);
  auto* d = static_cast<uint8_t*>(dst);
  if (vec == 16) rows_move_kernel<16, kPack><<<grid, 256, 0, stream>>>(s, cu, B, l_max, row_bytes, d);
  else if (vec == 4) rows_move_kernel<4, kPack><<<grid, 256, 0, stream>>>(s, cu, B, l_max, row_bytes, d);
  else rows_move_kernel<1, kPack><<<grid, 256, 0, stream>>>(s, cu, B, l_max, row_bytes, d);
  return launch_status();
}

}  // namespace
}  // namespace pk

namespace pk {
namespace {
int collate(const int32_t* input_ids, const int32_t* lengths, int32_t E, int32_t T, int32_t msl,
            int32_t* position_ids, int32_t* labels, int32_t* cu_seqlens, int32_t ignore_index,
            void* stream_) {
  if (E < 0 || T < 0 || cu_seqlens == nullptr) return PK_ERR_INVALID_ARG;
  if ((E > 0 && lengths == nullptr) || (T > 0 && position_ids == nullptr)) return PK_ERR_INVALID_ARG;
  if (T > 0 && (E == 0 || (labels != nullptr && input_ids == nullptr))) return PK_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  pk::lengths_scan_kernel<<<1, 1024, 0, stream>>>(lengths, E, cu_seqlens);
  if (pk::launch_status() != PK_OK) return PK_ERR_CUDA;
  if (T == 0) return PK_OK;
  pk::collate_kernel<<<(T + 255) / 256, 256, 0, stream>>>(input_ids, cu_seqlens, E, T, msl,
                                                         ignore_index, position_ids, labels);
  return pk::launch_status();
}
}  // namespace
}  // namespace pk

extern "C" int pk_collate_padding_free(const int32_t* input_ids, const int32_t* lengths, int32_t E,
                                       int32_t T, int32_t* position_ids, int32_t* labels,
                                       int32_t* cu_seqlens, int32_t ignore_index, void* stream) {
  return pk::collate(input_ids, lengths, E, T, 0, position_ids, labels, cu_seqlens, ignore_index,
                     stream);
}

extern "C" int pk_collate_fixed_length(const int32_t* input_ids, const int32_t* lengths, int32_t E,
                                       int32_t T, int32_t msl, int32_t* position_ids,
                                       int32_t* labels, int32_t* cu_seqlens, int32_t ignore_index,
                                       void* stream) {
  if (msl <= 0) return PK_ERR_INVALID_ARG;
  return pk::collate(input_ids, lengths, E, T, msl, position_ids, labels, cu_seqlens, ignore_index,
                     stream);
}

extern "C" int pk_pack_first_fit_decreasing(const int32_t* lengths, int32_t n, int32_t capacity,
                                            int32_t* bin_of, int32_t* n_bins) {
  if (n < 0 || capacity <= 0 || n_bins == nullptr || (n > 0 && (!lengths || !bin_of)))
    return PK_ERR_INVALID_ARG;
  for (int i = 0; i < n; ++i)
    if (lengths[i] <= 0 || lengths[i] > capacity) return PK_ERR_INVALID_ARG;
  std::vector<int32_t> order(n);
  std::iota(order.begin(), order.end(), 0);
  std::stable_sort(order.begin(), order.end(),
                   [&](int32_t a, int32_t b) { return lengths[a] > lengths[b]; });
  std::vector<int32_t> room;
  for (int32_t i : order) {
    size_t b = 0;
    while (b < room.size() && room[b] < lengths[i]) ++b;
    if (b == room.size()) room.push_back(capacity);
    room[b] -= lengths[i];
    bin_of[i] = (int32_t)b;
  }
  *n_bins = (int32_t)room.size();
  return PK_OK;
}

extern "C" int pk_pack_next_fit(const int32_t* lengths, int32_t n, int32_t capacity,
                                int32_t sort_descending, int32_t* bin_of, int32_t* n_bins) {
  if (n < 0 || capacity <= 0 || n_bins == nullptr || (n > 0 && (!lengths || !bin_of)))
    return PK_ERR_INVALID_ARG;
  for (int i = 0; i < n; ++i)
    if (lengths[i] <= 0 || lengths[i] > capacity) return PK_ERR_INVALID_ARG;
  std::vector<int32_t> order(n);
  std::iota(order.begin(), order.end(), 0);
  if (sort_descending)
    std::stable_sort(order.begin(), order.end(),
                     [&](int32_t a, int32_t b) { return lengths[a] > lengths[b]; });
  int32_t b = 0, used = 0;
  bool started = false;
  for (int32_t i : order) {
    if (started && used + lengths[i] > capacity) { ++b; used = 0; }
    bin_of[i] = b;
    used += lengths[i];
    started = true;
  }
  *n_bins = started ? b + 1 : 0;
  return PK_OK;
}

extern "C" int pk_pack_rows(const void* padded, const int32_t* cu_seqlens, int32_t B, int32_t l_max,
                            int32_t T, int64_t row_bytes, void* packed, void* stream) {
  if (B < 0 || l_max < 0 || T < 0 || row_bytes <= 0) return PK_ERR_INVALID_ARG;
  if (T > 0 && (!padded || !packed || !cu_seqlens || B == 0)) return PK_ERR_INVALID_ARG;
  return pk::rows_move<true>(padded, cu_seqlens, B, l_max, T, row_bytes, packed,
                             static_cast<cudaStream_t>(stream));
}

extern "C" int pk_unpack_rows(const void* packed, const int32_t* cu_seqlens, int32_t B, int32_t l_max,
                              int32_t T, int64_t row_bytes, void* padded, void* stream) {
  if (B < 0 || l_max < 0 || T < 0 || row_bytes <= 0) return PK_ERR_INVALID_ARG;
  if ((long long)B * l_max > 0 && (!padded || !cu_seqlens || (T > 0 && !packed)))
    return PK_ERR_INVALID_ARG;
  return pk::rows_move<false>(packed, cu_seqlens, B, l_max, T, row_bytes, padded,
                              static_cast<cudaStream_t>(stream));
}
