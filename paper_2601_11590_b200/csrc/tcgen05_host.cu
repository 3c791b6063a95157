// Host helpers shared by the tcgen05 kernels: tensor-map encoding through the driver entry point, per-device
// properties, and the cycle limit of the kernels' bounded waits.
#include <mutex>

#include "tcgen05_common.cuh"

namespace epd {
namespace {

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  });
  return fn;
}

constexpr long long kDefaultWaitCycles = 4000000000LL;   // ~2 s at 2 GHz
std::atomic<long long> g_wait_cycles{kDefaultWaitCycles};
std::atomic<int> g_sm_count[64] = {};

}  // namespace

bool tensor_maps_available() { return encode_tiled_fn() != nullptr; }
bool tensor_core_path_available() { return tensor_maps_available(); }

bool make_tensor_map_2d(CUtensorMap* tm, const void* base, int64_t rows, int64_t cols, int64_t pitch_bytes,
                        int box_rows, int box_cols, int elem_bytes, CUtensorMapSwizzle swizzle) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  const CUtensorMapDataType dt = elem_bytes == 4   ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32
                                 : elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16
                                                   : CU_TENSOR_MAP_DATA_TYPE_UINT8;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)pitch_bytes};
  cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(tm, dt, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int device_sm_count() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 148;
  const bool cached = dev >= 0 && dev < 64;
  if (cached) {
    const int n = g_sm_count[dev].load(std::memory_order_relaxed);
    if (n > 0) return n;
  }
  int n = 0;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
  if (cached) g_sm_count[dev].store(n, std::memory_order_relaxed);
  return n;
}

long long wait_limit_cycles() { return g_wait_cycles.load(std::memory_order_relaxed); }

}  // namespace epd

extern "C" int epd_debug_set_wait_limit(int64_t cycles) {
  epd::g_wait_cycles.store(cycles > 0 ? (long long)cycles : epd::kDefaultWaitCycles, std::memory_order_relaxed);
  return EPD_OK;
}
