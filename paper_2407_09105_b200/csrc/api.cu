// Small host-only entry points of the C ABI: tile shape, workspace sizing and layout,
// status read-back.
#include "pk_common.cuh"
#include "sm100_ptx.cuh"

namespace pk {
cudaEvent_t g_timing_events[PK_NUM_KERNELS][2] = {};
}

extern "C" int pk_set_timing_events(int32_t which, void* start, void* stop) {
  if (which < 0 || which >= PK_NUM_KERNELS) return PK_ERR_INVALID_ARG;
  pk::g_timing_events[which][0] = static_cast<cudaEvent_t>(start);
  pk::g_timing_events[which][1] = static_cast<cudaEvent_t>(stop);
  return PK_OK;
}

extern "C" int pk_tile_shape(int32_t* bm, int32_t* bn) {
  if (bm) *bm = pk::kBM;
  if (bn) *bn = pk::kBN;
  return PK_OK;
}

extern "C" size_t pk_workspace_bytes(int32_t T, int32_t Hq, int32_t Hkv, int32_t D) {
  if (!pk::shape_supported(T, Hq, Hkv, D)) return 0;
  return pk::workspace_layout(T, Hq, Hkv, D).total;
}

extern "C" int pk_workspace_section(int32_t which, int32_t T, int32_t Hq, int32_t Hkv, int32_t D,
                                    size_t* offset, size_t* bytes) {
  if (which < 0 || which >= PK_WS_NUM_SECTIONS || offset == nullptr || bytes == nullptr)
    return PK_ERR_INVALID_ARG;
  if (!pk::shape_supported(T, Hq, Hkv, D)) return PK_ERR_UNSUPPORTED;
  const pk::WorkspaceLayout lay = pk::workspace_layout(T, Hq, Hkv, D);
  *offset = lay.off[which];
  *bytes = lay.bytes[which];
  return PK_OK;
}

extern "C" int pk_status_read(const void* workspace, void* stream, int32_t* code, int32_t* detail) {
  if (workspace == nullptr || code == nullptr || detail == nullptr) return PK_ERR_INVALID_ARG;
  int32_t host[2] = {0, 0};
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(host, workspace, sizeof(host), cudaMemcpyDeviceToHost, s) != cudaSuccess)
    return PK_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return PK_ERR_CUDA;
  *code = host[PK_HDR_STATUS];
  *detail = host[PK_HDR_DETAIL];
  return PK_OK;
}

namespace pk {
namespace {
// Waits on an mbarrier that nothing ever arrives at, with a small budget, and reports the
// expiry through the status word exactly as the attention kernels do.
__global__ void bounded_wait_selftest_kernel(int32_t* hdr, long long budget) {
  __shared__ __align__(8) unsigned long long s_bar;
  __shared__ int s_abort;
  const uint32_t bar = ptx::smem_u32(&s_bar);
  if (threadIdx.x == 0) {
    ptx::mbar_init(bar, 1);
    ptx::fence_mbar_init();
    s_abort = 0;
  }
  __syncthreads();
  const bool ok = ptx::mbar_wait_budget(bar, 0, &s_abort, budget);
  __syncthreads();
  if (threadIdx.x == 0 && !ok) set_status(hdr, PK_ERR_TIMEOUT, 99);
}
}  // namespace
}  // namespace pk

extern "C" int pk_selftest_bounded_wait(void* workspace, int64_t budget_cycles, void* stream) {
  if (workspace == nullptr || budget_cycles <= 0 || budget_cycles > 2000000000LL)
    return PK_ERR_INVALID_ARG;
  pk::bounded_wait_selftest_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<int32_t*>(workspace), (long long)budget_cycles);
  return pk::launch_status();
}
