// Rotary embedding + head split + block-diagonal attention for callers that must not allocate.
//
// Some users of this library run where device allocation is off limits: a serving process that
// has handed all of HBM to its own memory pool (cudaMalloc would fail or fragment it), or a
// latency-critical loop that cannot afford the implicit device synchronisation an allocation may
// cause.  The attention step needs room for the head-major q, k and v it builds from the packed
// qkv matrix.  This file provides that room as a fixed array in the library's own device image,
// so the entry point below needs no workspace argument and calls no allocator at all.
//
// Cost and limits: every GPU that loads the library carries the array (kStaticScratchBytes) until
// the process exits; batches whose q, k, v do not fit are rejected with EPD_ECAPACITY; all calls
// on one GPU share the same array, so two calls whose kernels may overlap on the device (different
// streams) race with each other.
#include <mutex>

#include "common.cuh"

namespace {

constexpr size_t kStaticScratchBytes = (size_t)16 << 20;
constexpr int kMaxDevices = 64;

// In host code this name is only a handle for cudaGetSymbolAddress(); it is not a device address.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

std::mutex g_lock;
void* g_scratch_addr[kMaxDevices] = {};  // device address of g_static_scratch, per device ordinal

// Looks up (once per device, with that device current) where the array lives on this GPU.
int scratch_on_current_device(unsigned char** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return EPD_ECUDA;
  std::lock_guard<std::mutex> guard(g_lock);
  if (g_scratch_addr[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return EPD_ECUDA;
    g_scratch_addr[dev] = p;
  }
  *out = static_cast<unsigned char*>(g_scratch_addr[dev]);
  return EPD_OK;
}

}  // namespace

extern "C" {

size_t epd_static_scratch_bytes(void) { return kStaticScratchBytes; }

int epd_op_rope_attention_static(int32_t dtype, const void* qkv, const int32_t* pos_row, const int32_t* pos_col,
                                 const int32_t* cu_seqlens, const int32_t* host_cu_seqlens, int32_t n_seg, void* out,
                                 int64_t T, int32_t heads, int32_t head_dim, float theta, void* stream) {
  using namespace epd;
  if (dtype != EPD_DTYPE_F32 && dtype != EPD_DTYPE_BF16) return EPD_EINVAL;
  if (T < 0 || T > (1 << 30) || n_seg < 0 || heads < 1 || heads > 65535 || head_dim < 4 || head_dim % 4 ||
      head_dim > kMaxHeadDim)
    return EPD_EINVAL;   // also keeps the size arithmetic below far from overflow
  if (T == 0 || n_seg == 0) return EPD_OK;
  if (!qkv || !pos_row || !pos_col || !cu_seqlens || !host_cu_seqlens || !out) return EPD_EINVAL;
  if (host_cu_seqlens[0] != 0 || host_cu_seqlens[n_seg] != T) return EPD_EINVAL;
  for (int i = 0; i < n_seg; ++i)
    if (host_cu_seqlens[i + 1] <= host_cu_seqlens[i]) return EPD_EINVAL;
  const size_t es = dtype == EPD_DTYPE_F32 ? 4 : 2;
  const size_t one = (size_t)heads * (size_t)T * (size_t)padded_head_dim(head_dim) * es;
  const size_t one_aligned = (one + 255) / 256 * 256;
  if (3 * one_aligned > kStaticScratchBytes) return EPD_ECAPACITY;
  unsigned char* base = nullptr;
  const int rc = scratch_on_current_device(&base);
  if (rc != EPD_OK) return rc;
  // q, k, v are fully rewritten (padding columns included) by the split kernel on every call, so
  // nothing left behind by an earlier call is ever read.
  void* q = base;
  void* k = base + one_aligned;
  void* v = base + 2 * one_aligned;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const float q_scale = 1.4426950408889634f / sqrtf((float)head_dim);
  if (rope_split(dtype, qkv, pos_row, pos_col, nullptr, 0, q, k, v, T, heads, head_dim, theta, q_scale, s) !=
      cudaSuccess)
    return EPD_ECUDA;
  if (attention_any(dtype, q, k, v, cu_seqlens, host_cu_seqlens, n_seg, out, T, heads, head_dim, 0, nullptr, s) !=
      cudaSuccess)
    return EPD_ECUDA;
  return EPD_OK;
}

}  // extern "C"
