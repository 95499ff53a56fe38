// Loss of a packed stream ("next" scope, the step right after the model): shifted cross entropy
// over the labels of the padding-free collator (Sec. 3.4 / 3.5: the first label of every example
// is -100, so the last token of an example never predicts the first token of the next one).
//
//   target[t] = labels[t + 1] (none for the last row);   loss_t = logsumexp(logits[t]) - logits[t][target]
//   loss = sum_t loss_t / n_valid;   dlogits[t] = (softmax(logits[t]) - onehot(target)) * g / n_valid
//
// Streaming kernels, one CTA per row, every logit read once per pass with 16-byte loads: the
// forward is bound by HBM reads (2 B per logit for bf16) with the special-function unit close
// behind (one exp2 per logit), the backward by read + write.  The per-row losses are summed by a
// second, single-CTA kernel in a fixed order, so the scalar is bitwise reproducible.
#include <cuda_bf16.h>

#include "pk_common.cuh"

namespace pk {
namespace {

constexpr int kLossThreads = 256;
constexpr float kLog2eL = 1.4426950408889634f;
constexpr float kLn2L = 0.6931471805599453f;

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

template <typename T> struct Vec;             // 16-byte vectors of logits
template <> struct Vec<__nv_bfloat16> {
  static constexpr int kN = 8;
  __device__ static void load(const __nv_bfloat16* p, float* f) {
    const uint4 v = *reinterpret_cast<const uint4*>(p);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {             // bf16 -> fp32 is a shift
      f[2 * i] = __uint_as_float(w[i] << 16);
      f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
  __device__ static void store(__nv_bfloat16* p, const float* f) {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const __nv_bfloat162 h = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
      w[i] = *reinterpret_cast<const uint32_t*>(&h);
    }
    *reinterpret_cast<uint4*>(p) = make_uint4(w[0], w[1], w[2], w[3]);
  }
};
template <> struct Vec<float> {
  static constexpr int kN = 4;
  __device__ static void load(const float* p, float* f) {
    const float4 v = *reinterpret_cast<const float4*>(p);
    f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;
  }
  __device__ static void store(float* p, const float* f) {
    *reinterpret_cast<float4*>(p) = make_float4(f[0], f[1], f[2], f[3]);
  }
};
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }
__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ void from_f32(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }
__device__ __forceinline__ void from_f32(float* p, float x) { *p = x; }

__device__ __forceinline__ int target_of(const int32_t* labels, int t, int T) {
  return (t + 1 < T) ? labels[t + 1] : -1;
}

// (m, s): running maximum and sum of exp2(y - m), both in the log2 domain
__device__ __forceinline__ void combine(float& m, float& s, float m2, float s2) {
  const float mn = fmaxf(m, m2);
  const float a = (m == -INFINITY) ? 0.f : ex2f(m - mn);
  const float b = (m2 == -INFINITY) ? 0.f : ex2f(m2 - mn);
  s = s * a + s2 * b;
  m = mn;
}

template <typename T, bool kVector>
__global__ void __launch_bounds__(kLossThreads)
ce_fwd_kernel(const T* __restrict__ logits, const int32_t* __restrict__ labels, int n_rows, int V,
              long long stride, int ignore_index, float* __restrict__ token_loss,
              float* __restrict__ lse_out) {
  const int t = blockIdx.x;
  const int tid = threadIdx.x;
  const int tgt = target_of(labels, t, n_rows);
  const bool valid = (t + 1 < n_rows) && tgt != ignore_index && tgt >= 0 && tgt < V;
  if (!valid) {                                  // uniform for the CTA
    if (tid == 0) { token_loss[t] = 0.f; lse_out[t] = 0.f; }
    return;
  }
  const T* row = logits + (long long)t * stride;
  float m = -INFINITY, s = 0.f;
  if (kVector) {
    constexpr int N = Vec<T>::kN;
    const int nv = V / N;
    // two vectors per rescale: the rescale costs an exp2 of its own and the special-function
    // unit is nearly as busy as the memory system here
    for (int i = tid; i < nv; i += 2 * kLossThreads) {
      float f[2 * N];
      const bool two = (i + kLossThreads) < nv;
      Vec<T>::load(row + (long long)i * N, f);
      if (two) Vec<T>::load(row + (long long)(i + kLossThreads) * N, f + N);
      else {
#pragma unroll
        for (int k = 0; k < N; ++k) f[N + k] = -INFINITY;
      }
      float mx = f[0];
#pragma unroll
      for (int k = 1; k < 2 * N; ++k) mx = fmaxf(mx, f[k]);
      const float mn = fmaxf(m, mx * kLog2eL);
      float acc = 0.f;
#pragma unroll
      for (int k = 0; k < 2 * N; ++k) acc += ex2f(fmaf(f[k], kLog2eL, -mn));
      s = s * ex2f(m - mn) + acc;               // m = -inf on the first round: exp2(-inf) = 0
      m = mn;
    }
  } else {
    for (int i = tid; i < V; i += kLossThreads) {
      const float y = to_f32(row[i]) * kLog2eL;
      const float mn = fmaxf(m, y);
      s = s * ex2f(m - mn) + ex2f(y - mn);
      m = mn;
    }
  }
  // block combine: warp shuffles, then the 8 warp results through shared memory
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float m2 = __shfl_xor_sync(0xffffffffu, m, o);
    const float s2 = __shfl_xor_sync(0xffffffffu, s, o);
    combine(m, s, m2, s2);
  }
  __shared__ float sm[kLossThreads / 32], ss[kLossThreads / 32];
  if ((tid & 31) == 0) { sm[tid >> 5] = m; ss[tid >> 5] = s; }
  __syncthreads();
  if (tid == 0) {
    float M = sm[0], S = ss[0];
#pragma unroll
    for (int w = 1; w < kLossThreads / 32; ++w) combine(M, S, sm[w], ss[w]);
    const float lse = (M + log2f(S)) * kLn2L;
    lse_out[t] = lse;
    token_loss[t] = lse - to_f32(row[tgt]);
  }
}

// sum of the per-row losses and number of rows with a target, fixed order: thread i adds rows
// i, i + 1024, ..., then a tree over the 1024 partial sums
__global__ void __launch_bounds__(1024)
ce_finish_kernel(const float* __restrict__ token_loss, const int32_t* __restrict__ labels, int n_rows,
                 int V, int ignore_index, float* __restrict__ result, int32_t* __restrict__ n_valid) {
  __shared__ float ssum[1024];
  __shared__ int scnt[1024];
  const int tid = threadIdx.x;
  float a = 0.f;
  int c = 0;
  for (int t = tid; t < n_rows; t += 1024) {
    const int tgt = target_of(labels, t, n_rows);
    if ((t + 1 < n_rows) && tgt != ignore_index && tgt >= 0 && tgt < V) {
      a += token_loss[t];
      ++c;
    }
  }
  ssum[tid] = a;
  scnt[tid] = c;
  __syncthreads();
  for (int o = 512; o > 0; o >>= 1) {
    if (tid < o) { ssum[tid] += ssum[tid + o]; scnt[tid] += scnt[tid + o]; }
    __syncthreads();
  }
  if (tid == 0) {
    result[1] = ssum[0];
    result[0] = scnt[0] > 0 ? ssum[0] / (float)scnt[0] : 0.f;
    *n_valid = scnt[0];
  }
}

template <typename T, bool kVector>
__global__ void __launch_bounds__(kLossThreads)
ce_bwd_kernel(const T* __restrict__ logits, const int32_t* __restrict__ labels,
              const float* __restrict__ lse_in, const int32_t* __restrict__ n_valid, float grad_out,
              int n_rows, int V, long long stride, int ignore_index, T* __restrict__ dlogits) {
  const int t = blockIdx.x;
  const int tid = threadIdx.x;
  const int tgt = target_of(labels, t, n_rows);
  const bool valid = (t + 1 < n_rows) && tgt != ignore_index && tgt >= 0 && tgt < V;
  const T* row = logits + (long long)t * stride;
  T* out = dlogits + (long long)t * stride;
  const int nval = *n_valid;
  const float g = valid ? grad_out / (float)(nval > 0 ? nval : 1) : 0.f;
  // x - lse is formed first: for rows with a large common offset it is exact where the product
  // form would round twice
  const float lse_t = valid ? lse_in[t] : 0.f;
  if (kVector) {
    constexpr int N = Vec<T>::kN;
    const int nv = V / N;
    for (int i = tid; i < nv; i += kLossThreads) {
      float f[N];
      if (valid) {
        Vec<T>::load(row + (long long)i * N, f);
#pragma unroll
        for (int k = 0; k < N; ++k) f[k] = ex2f((f[k] - lse_t) * kLog2eL) * g;
        const int d = tgt - i * N;
        if (d >= 0 && d < N) {
#pragma unroll
          for (int k = 0; k < N; ++k)
            if (k == d) f[k] -= g;
        }
      } else {
#pragma unroll
        for (int k = 0; k < N; ++k) f[k] = 0.f;
      }
      Vec<T>::store(out + (long long)i * N, f);
    }
  } else {
    for (int i = tid; i < V; i += kLossThreads) {
      float x = 0.f;
      if (valid) x = ex2f((to_f32(row[i]) - lse_t) * kLog2eL) * g - (i == tgt ? g : 0.f);
      from_f32(out + i, x);
    }
  }
}

template <typename T>
bool vector_ok(const void* a, const void* b, int V, long long stride) {
  const int N = 16 / (int)sizeof(T);
  return V % N == 0 && stride % N == 0 && (reinterpret_cast<uintptr_t>(a) & 15) == 0 &&
         (b == nullptr || (reinterpret_cast<uintptr_t>(b) & 15) == 0);
}

}  // namespace
}  // namespace pk

extern "C" int pk_packed_loss_fwd(const void* logits, int32_t logits_dtype, const int32_t* labels,
                                  int32_t T, int32_t V, int64_t row_stride, int32_t ignore_index,
                                  float* token_loss, float* lse, float* result, int32_t* n_valid,
                                  void* stream_) {
  using namespace pk;
  if (T < 0 || V <= 0 || row_stride < V || result == nullptr || n_valid == nullptr)
    return PK_ERR_INVALID_ARG;
  if (logits_dtype != PK_BF16 && logits_dtype != PK_F32) return PK_ERR_INVALID_ARG;
  if (T > 0 && (!logits || !labels || !token_loss || !lse)) return PK_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  if (T > 0) {
    TimedLaunch timed(PK_KERNEL_LOSS_FWD, stream);
    if (logits_dtype == PK_BF16) {
      const auto* p = static_cast<const __nv_bfloat16*>(logits);
      if (vector_ok<__nv_bfloat16>(p, nullptr, V, row_stride))
        ce_fwd_kernel<__nv_bfloat16, true><<<T, kLossThreads, 0, stream>>>(
            p, labels, T, V, row_stride, ignore_index, token_loss, lse);
      else
        ce_fwd_kernel<__nv_bfloat16, false><<<T, kLossThreads, 0, stream>>>(
            p, labels, T, V, row_stride, ignore_index, token_loss, lse);
    } else {
      const auto* p = static_cast<const float*>(logits);
      if (vector_ok<float>(p, nullptr, V, row_stride))
        ce_fwd_kernel<float, true><<<T, kLossThreads, 0, stream>>>(p, labels, T, V, row_stride,
                                                                  ignore_index, token_loss, lse);
      else
        ce_fwd_kernel<float, false><<<T, kLossThreads, 0, stream>>>(p, labels, T, V, row_stride,
                                                                   ignore_index, token_loss, lse);
    }
  }
  if (launch_status() != PK_OK) return PK_ERR_CUDA;
  ce_finish_kernel<<<1, 1024, 0, stream>>>(token_loss, labels, T, V, ignore_index, result, n_valid);
  return launch_status();
}

extern "C" int pk_packed_loss_bwd(const void* logits, int32_t logits_dtype, const int32_t* labels,
                                  const float* lse, const int32_t* n_valid, float grad_out, int32_t T,
                                  int32_t V, int64_t row_stride, int32_t ignore_index, void* dlogits,
                                  void* stream_) {
  using namespace pk;
  if (T < 0 || V <= 0 || row_stride < V || n_valid == nullptr) return PK_ERR_INVALID_ARG;
  if (logits_dtype != PK_BF16 && logits_dtype != PK_F32) return PK_ERR_INVALID_ARG;
  if (T == 0) return PK_OK;
  if (!logits || !labels || !lse || !dlogits) return PK_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  TimedLaunch timed(PK_KERNEL_LOSS_BWD, stream);
  if (logits_dtype == PK_BF16) {
    const auto* p = static_cast<const __nv_bfloat16*>(logits);
    auto* o = static_cast<__nv_bfloat16*>(dlogits);
    if (vector_ok<__nv_bfloat16>(p, o, V, row_stride))
      ce_bwd_kernel<__nv_bfloat16, true><<<T, kLossThreads, 0, stream>>>(
          p, labels, lse, n_valid, grad_out, T, V, row_stride, ignore_index, o);
    else
      ce_bwd_kernel<__nv_bfloat16, false><<<T, kLossThreads, 0, stream>>>(
          p, labels, lse, n_valid, grad_out, T, V, row_stride, ignore_index, o);
  } else {
    const auto* p = static_cast<const float*>(logits);
    auto* o = static_cast<float*>(dlogits);
    if (vector_ok<float>(p, o, V, row_stride))
      ce_bwd_kernel<float, true><<<T, kLossThreads, 0, stream>>>(p, labels, lse, n_valid, grad_out, T,
                                                                V, row_stride, ignore_index, o);
    else
      ce_bwd_kernel<float, false><<<T, kLossThreads, 0, stream>>>(p, labels, lse, n_valid, grad_out,
                                                                 T, V, row_stride, ignore_index, o);
  }
  return launch_status();
}
