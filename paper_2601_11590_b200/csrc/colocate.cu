// Sharing the GPU with another stage (Section 3.5 of the paper: Encode co-located with Prefill or Decode).
//   * an SM budget for the encoder's persistent kernels, so that the rest of the GPU stays free for the
//     co-located stage;
//   * a stream-ordered "features ready" flag a consumer can poll or wait on (asynchronous prefetch of
//     Section 3.2: the consumer learns that a request's features are complete without a host round trip);
//   * a memory-bound stand-in for a Decode step (a persistent kernel streaming a large buffer), used only
//     to measure the mutual slowdown of the two stages.
#include <atomic>

#include "common.cuh"

namespace epd {
namespace {

std::atomic<int> g_sm_limit{0};

__global__ void signal_kernel(uint32_t* flag, uint32_t value) {
  pdl_launch_dependents();
  pdl_wait();
  // everything ordered before this kernel on the stream is visible to whoever observes the flag
  __threadfence_system();
  asm volatile("st.release.sys.global.u32 [%0], %1;" ::"l"(flag), "r"(value) : "memory");
}

// Each CTA streams its share of the buffer `passes` times with 16-byte loads and keeps a checksum.
__global__ void __launch_bounds__(512)
stream_read_kernel(const uint4* __restrict__ data, int64_t n_vec, int passes, unsigned long long* __restrict__ sums) {
  unsigned long long acc = 0;
  const int64_t per_cta = (n_vec + gridDim.x - 1) / gridDim.x;
  const int64_t beg = per_cta * blockIdx.x, end = min(n_vec, beg + per_cta);
  for (int p = 0; p < passes; ++p) {
    for (int64_t i = beg + threadIdx.x; i < end; i += blockDim.x) {
      const uint4 v = data[i];
      acc += (unsigned long long)(v.x ^ v.y) + (v.z ^ v.w) + p;
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if ((threadIdx.x & 31) == 0) atomicAdd(&sums[blockIdx.x], acc);
}

}  // namespace

int sm_limit() { return g_sm_limit.load(std::memory_order_relaxed); }

}  // namespace epd

extern "C" {

int epd_set_sm_limit(int32_t n_sms) {
  if (n_sms < 0) return EPD_EINVAL;
  epd::g_sm_limit.store(n_sms, std::memory_order_relaxed);
  return EPD_OK;
}

int32_t epd_get_sm_limit(void) { return epd::sm_limit(); }

int epd_signal_ready(uint32_t* flag, uint32_t value, void* stream) {
  if (!flag || ((uintptr_t)flag & 3)) return EPD_EINVAL;
  if (epd::launch_pdl(epd::signal_kernel, dim3(1), dim3(1), 0, static_cast<cudaStream_t>(stream), flag, value) != cudaSuccess)
    return EPD_ECUDA;
  return EPD_OK;
}

int epd_op_stream_read(const void* data, int64_t bytes, int32_t passes, int32_t n_ctas, uint64_t* cta_sums, void* stream) {
  if (!data || !cta_sums || bytes < 16 || passes < 1 || n_ctas < 1 || n_ctas > 4096 || ((uintptr_t)data & 15)) return EPD_EINVAL;
  epd::stream_read_kernel<<<n_ctas, 512, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const uint4*>(data), bytes / 16, passes, reinterpret_cast<unsigned long long*>(cta_sums));
  return cudaGetLastError() == cudaSuccess ? EPD_OK : EPD_ECUDA;
}

}  // extern "C"
