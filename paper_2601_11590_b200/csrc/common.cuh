// Internal declarations shared by the kernels of the Encode-stage library.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "epd_encoder.h"

namespace epd {

// Device status word values written by kernels whose bounded waits expire.
constexpr int kStatusTimeout = EPD_ETIMEOUT;

// Largest head_dim the attention kernels cover.
constexpr int kMaxHeadDim = 128;

// Padded head width of the head-major q/k/v buffers: a multiple of 16 elements so that every
// row starts on a 32-byte boundary and the contraction over head_dim splits into 16-wide steps.
__host__ __device__ inline int padded_head_dim(int dh) { return (dh + 15) / 16 * 16; }

template <typename T> __device__ __forceinline__ float to_float(T v);
template <> __device__ __forceinline__ float to_float<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_float<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename T> __device__ __forceinline__ T from_float(float v);
template <> __device__ __forceinline__ float from_float<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_float<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

__device__ __forceinline__ float gelu_tanh_f(float x) {
  const float c = 0.7978845608028654f;  // sqrt(2/pi)
  return 0.5f * x * (1.0f + tanhf(c * (x + 0.044715f * x * x * x)));
}
__device__ __forceinline__ float gelu_erf_f(float x) { return 0.5f * x * (1.0f + erff(x * 0.7071067811865476f)); }

// Internal flag of the linear kernels (above the public EPD_LINEAR_* bits): the weight matrix is not written by
// any kernel that may still be running when this one starts (an encoder's own weights), so its first tiles may
// be fetched before the wait for the previous kernel.
constexpr int kLinearStaticWeights = 1 << 20;

// ---- programmatic dependent launch ---------------------------------------------------------------
// The kernels of one encode run back to back on one stream.  Launched with the programmatic-stream-
// serialization attribute, a kernel's CTAs may become resident as soon as every CTA of the previous
// kernel has started (pdl_launch_dependents, called first thing) and SM resources are free; they run
// their set-up (barrier init, tensor-memory allocation, descriptor prefetch) and then block in
// pdl_wait() until the previous kernel has completed and its writes are visible.  No global memory is
// read or written before pdl_wait().  A kernel launched the ordinary way ignores both instructions.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                              Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}

// ---- SM budget ---------------------------------------------------------------------------------
// Upper bound on the CTAs of the persistent kernels (linear, attention): 0 = every SM.  Set through
// epd_set_sm_limit() by a process that shares the GPU with another stage (co-location).
int sm_limit();
inline int limited_sms(int device_sms) {
  const int lim = sm_limit();
  return (lim > 0 && lim < device_sms) ? lim : device_sms;
}

// ---- plain-FMA kernels (kernels_fma.cu) -----------------------------------------------------
cudaError_t linear_fma(int dtype, const void* x, int64_t ldx, const void* w, int64_t ldw, const void* bias,
                       void* out, int64_t ldo, int64_t M, int64_t N, int64_t K, int flags, cudaStream_t s);
cudaError_t rmsnorm(int dtype, const void* x, const void* gain, void* out, const int32_t* dst_row, int64_t T,
                    int hidden, float eps, cudaStream_t s);
cudaError_t rope_split(int dtype, const void* qkv, const int32_t* pos_row, const int32_t* pos_col,
                       const float2* table, int table_rows, void* q, void* k, void* v, int64_t T, int heads,
                       int head_dim, float theta, float q_scale, cudaStream_t s);
cudaError_t rope_table(float2* table, int rows, int head_dim, float theta, cudaStream_t s);
cudaError_t attention_fma(int dtype, const void* q, const void* k, const void* v, const int32_t* cu_seqlens,
                          int n_seg, void* out, int64_t T, int heads, int head_dim, cudaStream_t s);
// Chooses the attention kernel for the shape (see attention kernels); `status` may be NULL.
cudaError_t attention_any(int dtype, const void* q, const void* k, const void* v, const int32_t* cu_seqlens,
                          const int32_t* host_cu_seqlens, int n_seg, void* out, int64_t T, int heads, int head_dim,
                          int flags, int* status, cudaStream_t s);
cudaError_t patchify(int dtype, int frame_format, const void* frames, const int64_t* item_off, const int32_t* grid_thw,
                     const int32_t* cu_seqlens, int n_images, int64_t T, void* patches, int64_t ld, int C, int P, int Tp,
                     const float* mean, const float* inv_std, cudaStream_t s);
cudaError_t content_hash(const void* data, const int64_t* item_off, int n_items, uint64_t* hashes, cudaStream_t s);
cudaError_t merge_gather(int dtype, const void* y, const int32_t* merge_idx, void* out, int64_t Tm, int hidden,
                         cudaStream_t s);
cudaError_t token_layout(const int32_t* grid_thw, const int32_t* cu_seqlens, const int32_t* cu_out, int n_images,
                         int64_t T, int32_t* pos_row, int32_t* pos_col, int32_t* merge_slot, int32_t* merge_idx,
                         cudaStream_t s);


// Attention with two query tiles per CTA sharing every K / V tile (attention_pair_tcgen05.cu).
bool attention_pair_supported(const void* q, const void* k, const void* v, const void* out, int64_t T, int heads,
                              int head_dim);
cudaError_t attention_pair(const void* q, const void* k, const void* v, const int32_t* host_cu_seqlens, int n_seg,
                           void* out, int64_t T, int heads, int head_dim, int* status, cudaStream_t s);

// True if the driver offers the tensor-map encoder the tensor-core kernels need.
bool tensor_core_path_available();

// ---- tensor-core kernels (gemm_tcgen05.cu) ---------------------------------------------------
// bf16 x bf16 -> fp32 linear layer on tcgen05; `status` (device int, may be NULL) receives
// EPD_ETIMEOUT if a bounded wait expires.  forced_bn: 0 = choose the tile width automatically.
bool linear_tc_supported(const void* x, int64_t ldx, const void* w, int64_t ldw, const void* bias, const void* out,
                         int64_t ldo, int64_t M, int64_t N, int64_t K, int flags);
cudaError_t linear_tc(const void* x, int64_t ldx, const void* w, int64_t ldw, const void* bias, void* out, int64_t ldo,
                      int64_t M, int64_t N, int64_t K, int flags, int forced_bn, int* status, cudaStream_t s);

// Same contract on CTA pairs (256 x 256 tiles, tcgen05.mma.cta_group::2); gemm_tcgen05_pair.cu.  A large residual
// update runs as linear_tc_pair_slices() consecutive launches over slices of K.
int linear_tc_pair_slices(int64_t N, int64_t K, int flags);
// Kernel launches linear_tc() makes for a shape.
int linear_tc_launches(int64_t M, int64_t N, int64_t K, int flags, int forced_bn);
cudaError_t linear_tc_pair(const void* x, int64_t ldx, const void* w, int64_t ldw, const void* bias, void* out,
                           int64_t ldo, int64_t M, int64_t N, int64_t K, int flags, int* status, cudaStream_t s);


// 8-bit floating-point (E4M3) variant: row quantiser (kernels_fma.cu) and the layer itself (gemm_tcgen05_pair.cu).
cudaError_t quantize_rows_e4m3(const void* x, int64_t ldx, void* q, int64_t ldq, float* scale, int64_t M, int64_t K,
                               cudaStream_t s);
cudaError_t linear_tc_pair_e4m3(const void* xq, int64_t ldx, const float* row_scale, const void* wq, int64_t ldw,
                                const float* col_scale, const void* bias, void* out, int64_t ldo, int64_t M, int64_t N,
                                int64_t K, int flags, int* status, cudaStream_t s);

// QKV projection whose epilogue applies the rotary embedding and writes head-major q, k, v (the
// padding columns are left as the caller initialised them with qkv_pad_init).  w_perm / bias_perm come
// from qkv_permute (pair order inside each head of q and k).  static_w: see kLinearStaticWeights.
cudaError_t linear_tc_pair_qkv(const void* x, int64_t ldx, const void* w_perm, int64_t ldw, const void* bias_perm,
                               void* q, void* k, void* v, const int32_t* pos_row, const int32_t* pos_col,
                               const float2* table, int table_rows, int64_t M, int heads, int head_dim, float q_scale,
                               int static_w, int* status, cudaStream_t s);
cudaError_t qkv_permute(const void* w, int64_t ldw, const void* bias, void* w_out, void* bias_out, int heads,
                        int head_dim, cudaStream_t s);
cudaError_t qkv_pad_init(void* q, void* k, void* v, int64_t rows, int head_dim, cudaStream_t s);

}  // namespace epd
