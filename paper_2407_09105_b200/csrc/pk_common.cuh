// Shared host/device definitions of the packed-attention library: workspace layout,
// status word, launch-error helper.  No attention arithmetic lives here.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "pk.h"

namespace pk {

constexpr int kBM = 128;   // query rows per tile
constexpr int kBN = 128;   // key rows per tile
constexpr int kHeaderInts = 32;

// header slots beyond the public PK_HDR_* ones
constexpr int kHdrFwdTicket = 8;
constexpr int kHdrBwdTicket = 9;    // dK/dV kernel (and the single-kernel backward)
constexpr int kHdrDqTicket = 10;    // dQ kernel

struct WorkspaceLayout {
  size_t off[PK_WS_NUM_SECTIONS];
  size_t bytes[PK_WS_NUM_SECTIONS];
  size_t off_cu;         // int32 [T+1]   the plan's own copy of cu_seqlens
  size_t off_ex_base;    // int32 [T+2]   first item index of every example
  size_t off_hist;       // int32 [2][T/128 + 4] counting-sort cursors (fwd, bwd)
  size_t hist_stride;    // ints per histogram
  size_t plan_total;     // bytes of the part that depends on T only
  // head sizes that run zero-padded to 64 or 128 (see head_pad.cu): padded copies of the
  // tensors, behind everything else; 0 bytes when D is 64 or 128
  size_t off_pad;
  size_t total;
};

// Head sizes other than 64 and 128 run on zero-padded copies of this size.
__host__ inline int padded_head_dim(int64_t D) { return D <= 64 ? 64 : 128; }

__host__ __device__ inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

__host__ inline WorkspaceLayout workspace_layout(int64_t T, int64_t Hq, int64_t Hkv,
                                                 int64_t D_given) {
  const int64_t D = padded_head_dim(D_given);   // every section is laid out for the padded size
  WorkspaceLayout w;
  size_t cur = 0;
  auto put = [&](int which, size_t bytes) {
    w.off[which] = cur;
    w.bytes[which] = bytes;
    cur = align_up(cur + bytes, 256);
  };
  const size_t Tn = (size_t)(T > 0 ? T : 1);
  // plan part: depends on T only
  put(PK_WS_HEADER, sizeof(int32_t) * kHeaderInts);
  put(PK_WS_FWD_ITEMS, sizeof(int32_t) * 4 * Tn);
  put(PK_WS_BWD_ITEMS, sizeof(int32_t) * 4 * Tn);
  put(PK_WS_FWD_ORDER, sizeof(int32_t) * Tn);
  put(PK_WS_BWD_ORDER, sizeof(int32_t) * Tn);
  w.off_cu = cur;
  cur = align_up(cur + sizeof(int32_t) * (Tn + 1), 256);
  w.off_ex_base = cur;
  cur = align_up(cur + sizeof(int32_t) * (Tn + 2), 256);
  w.hist_stride = Tn / 128 + 4;
  w.off_hist = cur;
  cur = align_up(cur + sizeof(int32_t) * 2 * w.hist_stride, 256);
  w.plan_total = cur;
  // attention part: depends on the head shape
  put(PK_WS_DELTA, sizeof(float) * (size_t)Hq * Tn);
  put(PK_WS_DQ_ACC, sizeof(float) * (size_t)(T + 128) * (size_t)Hq * (size_t)D);
  put(PK_WS_ROPE_TABLE, sizeof(float) * 2 * Tn * (size_t)(D / 2));
  w.off_pad = cur;
  if (D != D_given) {
    // q, dout (2 B), out, dq (4 B: fp32 allowed) per query head; k, v (2 B), dk, dv (4 B) per kv head
    const size_t per_q = align_up(Tn * (size_t)Hq * (size_t)D * 2, 256);
    const size_t per_kv = align_up(Tn * (size_t)Hkv * (size_t)D * 2, 256);
    cur += 2 * per_q + 2 * (2 * per_q) + 2 * per_kv + 2 * (2 * per_kv);
  }
  w.total = cur;
  return w;
}

inline bool shape_supported(int32_t T, int32_t Hq, int32_t Hkv, int32_t D) {
  if (T < 0 || Hq <= 0 || Hkv <= 0) return false;
  if (D < 16 || D > 128 || D % 16 != 0) return false;   // 64 and 128 natively, the rest padded
  if (Hq % Hkv != 0) return false;
  if ((int64_t)T * Hq * padded_head_dim(D) >= ((int64_t)1 << 31)) return false;
  return true;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Records the first device-side error; later ones are dropped.
__device__ inline void set_status(int32_t* header, int32_t code, int32_t detail) {
  if (atomicCAS(&header[PK_HDR_STATUS], PK_OK, code) == PK_OK) header[PK_HDR_DETAIL] = detail;
}

inline int launch_status() { return cudaGetLastError() == cudaSuccess ? PK_OK : PK_ERR_CUDA; }

// Optional event pair recorded around one kernel's launches (pk_set_timing_events).
extern cudaEvent_t g_timing_events[PK_NUM_KERNELS][2];
struct TimedLaunch {
  int which;
  cudaStream_t stream;
  TimedLaunch(int w, cudaStream_t s) : which(w), stream(s) {
    if (g_timing_events[which][0]) cudaEventRecord(g_timing_events[which][0], stream);
  }
  ~TimedLaunch() {
    if (g_timing_events[which][1]) cudaEventRecord(g_timing_events[which][1], stream);
  }
};

// internal entry points shared between translation units
int plan_launch(const int32_t* position_ids, int32_t T, int32_t* cu_seqlens, int32_t* n_examples,
                int32_t* max_seqlen, void* workspace, const WorkspaceLayout& lay,
                cudaStream_t stream);
int launch_bwd_ws(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                  const CUtensorMap& tdo, char* ws, const WorkspaceLayout& lay, const float* lse,
                  void* dq, void* dk, void* dv, int T, int Hq, int Hkv, int D, int grad_dtype, float scale,
                  int window, bool rotated, cudaStream_t stream);
int launch_fwd_ws(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, char* ws,
                  const WorkspaceLayout& lay, void* out, float* lse, int T, int Hq, int Hkv, int D,
                  int out_dtype, float scale, int window, bool rotated, cudaStream_t stream);
// reduced angles fp32 for the epilogues of the rotated-copies path: [T][row] with the D/2 angles
// of a token in front and zeros behind them (row = D/2 unless the heads run padded)
int rope_angle_launch(const int32_t* position_ids, int32_t T, int32_t D, float theta, float* angle,
                      cudaStream_t stream, int32_t row = 0);
// delta[h][t] = sum_d dO * O
int delta_launch(const void* dout, const void* out, int out_dtype, float* delta, int T, int Hq, int D,
                 cudaStream_t stream);
// q, k -> rotated fp16 copies (pairs (i, i + D/2), angle pos * theta^(-2i/D))
int rope_rotate_f16_launch(const void* x, const int32_t* position_ids, int32_t T, int32_t H,
                           int32_t D, float theta, void* y, cudaStream_t stream);
// head sizes other than 64 / 128: pad, run the call at the padded size, unpad (head_pad.cu)
int attn_fwd_padded(const void* q, const void* k, const void* v, const int32_t* position_ids,
                    int32_t T, int32_t Hq, int32_t Hkv, int32_t D, float softmax_scale,
                    float rope_theta, int32_t window, void* out, int32_t out_dtype, float* lse,
                    int32_t reuse_plan, void* workspace, size_t workspace_bytes, void* stream);
int attn_bwd_padded(const void* dout, const void* q, const void* k, const void* v, const void* out,
                    int32_t out_dtype, const float* lse, const int32_t* position_ids, int32_t T,
                    int32_t Hq, int32_t Hkv, int32_t D, float softmax_scale, float rope_theta,
                    int32_t window, void* dq, void* dk, void* dv, int32_t grad_dtype,
                    int32_t reuse_plan, void* workspace, size_t workspace_bytes, void* stream);
// 0: rotated copies of q, k in the workspace + warp-specialised kernels (default);
// 1: rotate the tiles in shared memory inside the attention kernels
extern int g_rope_mode;
int rope_table_launch(const int32_t* position_ids, int32_t T, int32_t D, float theta,
                      float* table, cudaStream_t stream);

}  // namespace pk
