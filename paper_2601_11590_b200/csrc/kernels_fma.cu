// Plain-FMA kernels of the Encode stage: the float path of every step, the bandwidth-bound
// steps of the bf16 path (RMSNorm, rotary + head split, merge), and the integer token layout.
// The dense contractions of the bf16 path run in gemm_tcgen05.cu / attention kernels instead.
#include "common.cuh"

namespace epd {

// =============================================================================================
// Token layout (integers): positions and 2x2-merge slots of every packed token.
// Token j of item i with local index f*h*w + r*w + c has pos_row = r, pos_col = c and goes to
// quarter q = 2*(r%2) + (c%2) of merged row o = cu_out[i] + f*(h/2)*(w/2) + (r/2)*(w/2) + c/2.
// =============================================================================================
__global__ void token_layout_kernel(const int32_t* __restrict__ grid_thw, const int32_t* __restrict__ cu,
                                    const int32_t* __restrict__ cu_out, int n, int64_t T,
                                    int32_t* __restrict__ pos_row, int32_t* __restrict__ pos_col,
                                    int32_t* __restrict__ merge_slot, int32_t* __restrict__ merge_idx) {
  for (int64_t j = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; j < T; j += (int64_t)gridDim.x * blockDim.x) {
    int lo = 0, hi = n;  // largest i with cu[i] <= j
    while (hi - lo > 1) {
      int mid = (lo + hi) >> 1;
      if (cu[mid] <= j) lo = mid; else hi = mid;
    }
    const int i = lo;
    const int h = grid_thw[3 * i + 1], w = grid_thw[3 * i + 2];
    const int local = (int)(j - cu[i]);
    const int f = local / (h * w);
    const int rem = local - f * h * w;
    const int r = rem / w, c = rem - r * w;
    pos_row[j] = r;
    pos_col[j] = c;
    const int o = cu_out[i] + f * (h / 2) * (w / 2) + (r / 2) * (w / 2) + (c / 2);
    const int slot = o * 4 + 2 * (r & 1) + (c & 1);
    merge_slot[j] = slot;
    merge_idx[slot] = (int32_t)j;
  }
}

cudaError_t token_layout(const int32_t* grid_thw, const int32_t* cu_seqlens, const int32_t* cu_out, int n_images,
                         int64_t T, int32_t* pos_row, int32_t* pos_col, int32_t* merge_slot, int32_t* merge_idx,
                         cudaStream_t s) {
  if (T == 0) return cudaSuccess;
  const int threads = 256;
  const int blocks = (int)((T + threads - 1) / threads);
  token_layout_kernel<<<blocks, threads, 0, s>>>(grid_thw, cu_seqlens, cu_out, n_images, T, pos_row, pos_col,
                                                 merge_slot, merge_idx);
  return cudaGetLastError();
}

// =============================================================================================
// Pixels -> patch vectors: token j = (item, frame f, row r, column c) gathers, from the item's frames
// [t*Tp, C, h*P, w*P] (uint8, or bf16 on the same 0..255 scale), the window rows r*P.., columns c*P.. of frames
// f*Tp.. in element order (channel, temporal, y, x); value = (pixel/255 - mean[channel]) * inv_std[channel].
// One thread per 8 consecutive elements of a token's patch vector: they are 8 consecutive pixels of one image
// row when P is a multiple of 8 (one 8-byte / 16-byte load), otherwise they are gathered one by one; either way
// the thread writes them with 16-byte stores, and neighbouring threads write neighbouring pieces of the same
// row of the patch matrix.  Bytes per token: K * sizeof(pixel) read + K * sizeof(T) written: HBM bound.
// =============================================================================================
struct PixelNorm {
  float mean[4], inv_std[4];
};

__device__ __forceinline__ float pixel_value(uint8_t v) { return (float)v; }
__device__ __forceinline__ float pixel_value(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename T, typename PixT>
__global__ void __launch_bounds__(256)
patchify_kernel(const PixT* __restrict__ frames, const int64_t* __restrict__ item_off,
                const int32_t* __restrict__ grid_thw, const int32_t* __restrict__ cu, int n, int64_t T_tokens,
                T* __restrict__ patches, int64_t ld, int C, int P, int Tp, PixelNorm norm) {
  const int pieces = (int)((ld + 7) / 8);                       // 8-element pieces per patch-matrix row
  const int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (v >= T_tokens * pieces) return;
  const int64_t j = v / pieces;
  const int k0 = (int)(v - j * pieces) * 8;
  int lo = 0, hi = n;  // largest i with cu[i] <= j
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (cu[mid] <= j) lo = mid; else hi = mid;
  }
  const int i = lo;
  const int h = grid_thw[3 * i + 1], w = grid_thw[3 * i + 2];
  const int local = (int)(j - cu[i]);
  const int f = local / (h * w);
  const int rem = local - f * h * w;
  const int r = rem / w, c = rem - r * w;
  const int64_t H = (int64_t)h * P, W = (int64_t)w * P;
  const int K = C * Tp * P * P;
  // item_off counts bytes
  const PixT* base = reinterpret_cast<const PixT*>(reinterpret_cast<const uint8_t*>(frames) + item_off[i]);
  float val[8];
  auto source = [&](int k) -> const PixT* {
    const int x = k % P, y = (k / P) % P, tp = (k / (P * P)) % Tp, ch = k / (P * P * Tp);
    return base + (((int64_t)(f * Tp + tp) * C + ch) * H + (int64_t)r * P + y) * W + (int64_t)c * P + x;
  };
  if (k0 + 8 <= K && P % 8 == 0) {
    // 8 pixels of one image row, one channel
    const PixT* src = source(k0);
    const int ch = k0 / (P * P * Tp);
    const float m = norm.mean[ch], is = norm.inv_std[ch];
    PixT px[8];
    if ((reinterpret_cast<uintptr_t>(src) & (8 * sizeof(PixT) - 1)) == 0) {
      if constexpr (sizeof(PixT) == 1) *reinterpret_cast<uint2*>(px) = *reinterpret_cast<const uint2*>(src);
      else *reinterpret_cast<uint4*>(px) = *reinterpret_cast<const uint4*>(src);
    } else {
#pragma unroll
      for (int e = 0; e < 8; ++e) px[e] = src[e];
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) val[e] = (pixel_value(px[e]) * (1.0f / 255.0f) - m) * is;
  } else {
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const int k = k0 + e;
      if (k < K) {
        const int ch = k / (P * P * Tp);
        val[e] = (pixel_value(*source(k)) * (1.0f / 255.0f) - norm.mean[ch]) * norm.inv_std[ch];
      } else {
        val[e] = 0.0f;   // padding columns of the row (leading dimension > K) are zeroed so that they are never garbage
      }
    }
  }
  T* out = patches + j * ld + k0;
  if (k0 + 8 <= ld && (reinterpret_cast<uintptr_t>(out) & 15) == 0) {
    if constexpr (sizeof(T) == 2) {
      uint32_t pk[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        __nv_bfloat162 b2 = __floats2bfloat162_rn(val[2 * e], val[2 * e + 1]);
        pk[e] = *reinterpret_cast<uint32_t*>(&b2);
      }
      *reinterpret_cast<uint4*>(out) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
    } else {
      reinterpret_cast<float4*>(out)[0] = make_float4(val[0], val[1], val[2], val[3]);
      reinterpret_cast<float4*>(out)[1] = make_float4(val[4], val[5], val[6], val[7]);
    }
  } else {
#pragma unroll
    for (int e = 0; e < 8; ++e)
      if (k0 + e < ld) out[e] = from_float<T>(val[e]);
  }
}

cudaError_t patchify(int dtype, int frame_format, const void* frames, const int64_t* item_off, const int32_t* grid_thw,
                     const int32_t* cu_seqlens, int n_images, int64_t T, void* patches, int64_t ld, int C, int P, int Tp,
                     const float* mean, const float* inv_std, cudaStream_t s) {
  if (T == 0) return cudaSuccess;
  PixelNorm norm;
  for (int c = 0; c < 4; ++c) {
    norm.mean[c] = c < C ? mean[c] : 0.0f;
    norm.inv_std[c] = c < C ? inv_std[c] : 1.0f;
  }
  const int64_t vectors = T * ((ld + 7) / 8);
  const unsigned blocks = (unsigned)((vectors + 255) / 256);
#define EPD_PATCHIFY(OUT, PIX)                                                                                   \
  patchify_kernel<OUT, PIX><<<blocks, 256, 0, s>>>(static_cast<const PIX*>(frames), item_off, grid_thw, cu_seqlens, \
                                                   n_images, T, static_cast<OUT*>(patches), ld, C, P, Tp, norm)
  if (frame_format == EPD_FRAMES_U8) {
    if (dtype == EPD_DTYPE_F32) EPD_PATCHIFY(float, uint8_t); else EPD_PATCHIFY(__nv_bfloat16, uint8_t);
  } else {
    if (dtype == EPD_DTYPE_F32) EPD_PATCHIFY(float, __nv_bfloat16); else EPD_PATCHIFY(__nv_bfloat16, __nv_bfloat16);
  }
#undef EPD_PATCHIFY
  return cudaGetLastError();
}

// =============================================================================================
// Row-wise quantisation to 8-bit floating point (E4M3) for the 8-bit variant of the linear layer:
//   scale[i] = max_j |x[i, j]| / 448 (1 for an all-zero row),  q[i, j] = e4m3(x[i, j] / scale[i])
// with round-to-nearest-even and saturation.  One warp per row; the row is read twice (the second pass hits
// L2), 16 bytes per load, 8 bytes per store.  Both divisions are IEEE float divisions: the quotient decides the
// 8-bit code, so it is formed the same way wherever the codes are checked.
// =============================================================================================
__device__ __forceinline__ uint16_t e4m3x2(float lo, float hi) {
  uint16_t d;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(d) : "f"(hi), "f"(lo));   // first source -> upper byte
  return d;
}

__global__ void __launch_bounds__(256)
quantize_rows_e4m3_kernel(const __nv_bfloat16* __restrict__ x, int64_t ldx, uint8_t* __restrict__ q, int64_t ldq,
                          float* __restrict__ scale, int64_t M, int K) {
  const int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= M) return;
  const __nv_bfloat16* xr = x + row * ldx;
  const int vecs = K / 8;
  float amax = 0.0f;
  for (int v = lane; v < vecs; v += 32) {
    const uint4 u = *reinterpret_cast<const uint4*>(xr + 8 * v);
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float2 f = __bfloat1622float2(h[e]);
      amax = fmaxf(amax, fmaxf(fabsf(f.x), fabsf(f.y)));
    }
  }
  for (int k = vecs * 8 + lane; k < K; k += 32) amax = fmaxf(amax, fabsf(__bfloat162float(xr[k])));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
  const float sc = amax > 0.0f ? __fdiv_rn(amax, 448.0f) : 1.0f;
  if (lane == 0) scale[row] = sc;
  uint8_t* qr = q + row * ldq;
  for (int v = lane; v < vecs; v += 32) {
    const uint4 u = *reinterpret_cast<const uint4*>(xr + 8 * v);
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
    uint16_t c[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float2 f = __bfloat1622float2(h[e]);
      c[e] = e4m3x2(__fdiv_rn(f.x, sc), __fdiv_rn(f.y, sc));
    }
    *reinterpret_cast<uint2*>(qr + 8 * v) = make_uint2((uint32_t)c[0] | ((uint32_t)c[1] << 16),
                                                       (uint32_t)c[2] | ((uint32_t)c[3] << 16));
  }
  for (int k = vecs * 8 + lane; k < K; k += 32)
    qr[k] = (uint8_t)(e4m3x2(__fdiv_rn(__bfloat162float(xr[k]), sc), 0.0f) & 0xFF);
  for (int64_t k = K + lane; k < ldq; k += 32) qr[k] = 0;     // padding bytes of the row: zero codes
}

cudaError_t quantize_rows_e4m3(const void* x, int64_t ldx, void* q, int64_t ldq, float* scale, int64_t M, int64_t K,
                               cudaStream_t s) {
  if (M == 0) return cudaSuccess;
  quantize_rows_e4m3_kernel<<<(unsigned)((M + 7) / 8), 256, 0, s>>>(static_cast<const __nv_bfloat16*>(x), ldx,
                                                                  static_cast<uint8_t*>(q), ldq, scale, M, (int)K);
  return cudaGetLastError();
}

// =============================================================================================
// Linear layer with plain FMAs: out = act(x . w^T + bias), 64x64 tile, 4x4 outputs per thread.
// =============================================================================================
constexpr int kFmaTile = 64;
constexpr int kFmaBK = 16;

template <typename TIn, typename TOut, int ACT, bool ACCUM>
__global__ void __launch_bounds__(256)
linear_fma_kernel(const TIn* __restrict__ x, int64_t ldx, const TIn* __restrict__ w, int64_t ldw,
                  const TIn* __restrict__ bias, TOut* __restrict__ out, int64_t ldo, int64_t M, int64_t N,
                  int64_t K) {
  __shared__ float sx[kFmaBK][kFmaTile + 1];
  __shared__ float sw[kFmaBK][kFmaTile + 1];
  const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
  const int64_t m0 = (int64_t)blockIdx.y * kFmaTile, n0 = (int64_t)blockIdx.x * kFmaTile;
  float acc[4][4] = {};
  for (int64_t k0 = 0; k0 < K; k0 += kFmaBK) {
    for (int e = threadIdx.x; e < kFmaTile * kFmaBK; e += 256) {
      const int row = e / kFmaBK, kk = e % kFmaBK;
      const int64_t gk = k0 + kk;
      sx[kk][row] = (m0 + row < M && gk < K) ? to_float<TIn>(x[(m0 + row) * ldx + gk]) : 0.0f;
      sw[kk][row] = (n0 + row < N && gk < K) ? to_float<TIn>(w[(n0 + row) * ldw + gk]) : 0.0f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < kFmaBK; ++kk) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { a[i] = sx[kk][ty * 4 + i]; b[i] = sw[kk][tx * 4 + i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int64_t m = m0 + ty * 4 + i;
    if (m >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int64_t n = n0 + tx * 4 + j;
      if (n >= N) continue;
      float v = acc[i][j] + (bias ? to_float<TIn>(bias[n]) : 0.0f);
      if (ACT == 1) v = gelu_tanh_f(v);
      if (ACT == 2) v = gelu_erf_f(v);
      if (ACCUM) out[m * ldo + n] = from_float<TOut>(to_float<TOut>(out[m * ldo + n]) + v);
      else out[m * ldo + n] = from_float<TOut>(v);
    }
  }
}

template <typename TIn, typename TOut>
static cudaError_t linear_fma_t(const void* x, int64_t ldx, const void* w, int64_t ldw, const void* bias, void* out,
                                int64_t ldo, int64_t M, int64_t N, int64_t K, int flags, cudaStream_t s) {
  dim3 grid((unsigned)((N + kFmaTile - 1) / kFmaTile), (unsigned)((M + kFmaTile - 1) / kFmaTile));
  const int act = (flags & EPD_LINEAR_GELU_TANH) ? 1 : (flags & EPD_LINEAR_GELU_ERF) ? 2 : 0;
  const bool accum = flags & EPD_LINEAR_ACCUMULATE;
#define EPD_LAUNCH(A, C)                                                                                      \
  linear_fma_kernel<TIn, TOut, A, C><<<grid, 256, 0, s>>>((const TIn*)x, ldx, (const TIn*)w, ldw,             \
                                                          (const TIn*)bias, (TOut*)out, ldo, M, N, K)
  if (accum) {
    if (act == 0) EPD_LAUNCH(0, true); else if (act == 1) EPD_LAUNCH(1, true); else EPD_LAUNCH(2, true);
  } else {
    if (act == 0) EPD_LAUNCH(0, false); else if (act == 1) EPD_LAUNCH(1, false); else EPD_LAUNCH(2, false);
  }
#undef EPD_LAUNCH
  return cudaGetLastError();
}

cudaError_t linear_fma(int dtype, const void* x, int64_t ldx, const void* w, int64_t ldw, const void* bias,
                       void* out, int64_t ldo, int64_t M, int64_t N, int64_t K, int flags, cudaStream_t s) {
  if (M == 0 || N == 0) return cudaSuccess;
  const bool out_f32 = (dtype == EPD_DTYPE_F32) || (flags & (EPD_LINEAR_OUT_F32 | EPD_LINEAR_ACCUMULATE));
  if (dtype == EPD_DTYPE_F32) return linear_fma_t<float, float>(x, ldx, w, ldw, bias, out, ldo, M, N, K, flags, s);
  if (out_f32) return linear_fma_t<__nv_bfloat16, float>(x, ldx, w, ldw, bias, out, ldo, M, N, K, flags, s);
  return linear_fma_t<__nv_bfloat16, __nv_bfloat16>(x, ldx, w, ldw, bias, out, ldo, M, N, K, flags, s);
}

// =============================================================================================
// RMSNorm: one warp per row of the float residual stream; optional scattered destination row.
// Bytes per row: 4h read + sizeof(T)h written.  When the row fits (hidden <= 128*NV) each lane keeps
// its NV float4 pieces in registers, so the row is read once and all loads are in flight together;
// longer or unaligned rows take the two-pass kernel, whose second pass re-reads from L1/L2.
// =============================================================================================
template <typename T>
__device__ __forceinline__ void store4(T* orow, int i, float r0, float r1, float r2, float r3) {
  if constexpr (sizeof(T) == 4) {
    reinterpret_cast<float4*>(orow)[i] = make_float4(r0, r1, r2, r3);
  } else {
    __nv_bfloat162 lo = __floats2bfloat162_rn(r0, r1), hi = __floats2bfloat162_rn(r2, r3);
    uint2 pk;
    pk.x = *reinterpret_cast<uint32_t*>(&lo);
    pk.y = *reinterpret_cast<uint32_t*>(&hi);
    reinterpret_cast<uint2*>(orow)[i] = pk;
  }
}

template <typename T>
__device__ __forceinline__ float4 load_gain4(const T* gain, int i) {
  if constexpr (sizeof(T) == 4) {
    return reinterpret_cast<const float4*>(gain)[i];
  } else {
    const uint2 pk = reinterpret_cast<const uint2*>(gain)[i];
    const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&pk.x));
    const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&pk.y));
    return make_float4(a.x, a.y, b.x, b.y);
  }
}

template <typename T, int NV>
__global__ void __launch_bounds__(256, NV <= 9 ? 5 : 1)
rmsnorm_reg_kernel(const float* __restrict__ x, const T* __restrict__ gain, T* __restrict__ out,
                   const int32_t* __restrict__ dst_row, int64_t rows, int hidden, float eps) {
  pdl_launch_dependents();
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (row >= rows) return;
  const int nvec = hidden >> 2;
  const float4* x4 = reinterpret_cast<const float4*>(x + row * hidden);
  float4 v[NV];
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    const int idx = lane + 32 * i;
    v[i] = idx < nvec ? x4[idx] : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
  }
  float ss = 0.0f;
#pragma unroll
  for (int i = 0; i < NV; ++i) ss += v[i].x * v[i].x + v[i].y * v[i].y + v[i].z * v[i].z + v[i].w * v[i].w;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  const float inv = 1.0f / sqrtf(ss / (float)hidden + eps);
  const int64_t drow = dst_row ? (int64_t)dst_row[row] : row;
  T* orow = out + drow * hidden;
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    const int idx = lane + 32 * i;
    if (idx < nvec) {
      const float4 g = load_gain4<T>(gain, idx);
      store4<T>(orow, idx, v[i].x * inv * g.x, v[i].y * inv * g.y, v[i].z * inv * g.z, v[i].w * inv * g.w);
    }
  }
}

template <typename T>
__global__ void __launch_bounds__(256)
rmsnorm_kernel(const float* __restrict__ x, const T* __restrict__ gain, T* __restrict__ out,
               const int32_t* __restrict__ dst_row, int64_t rows, int hidden, float eps) {
  pdl_launch_dependents();
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (row >= rows) return;
  const float* xr = x + row * hidden;
  float ss = 0.0f;
  for (int i = lane; i < hidden; i += 32) ss += xr[i] * xr[i];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  const float inv = 1.0f / sqrtf(ss / (float)hidden + eps);
  const int64_t drow = dst_row ? (int64_t)dst_row[row] : row;
  T* orow = out + drow * hidden;
  for (int i = lane; i < hidden; i += 32) orow[i] = from_float<T>(xr[i] * inv * to_float<T>(gain[i]));
}

template <typename T>
static cudaError_t rmsnorm_t(const float* x, const T* gain, T* out, const int32_t* dst_row, int64_t rows, int hidden,
                             float eps, cudaStream_t s) {
  const int warps = 8;
  const unsigned blocks = (unsigned)((rows + warps - 1) / warps);
  const bool vec_ok = (hidden % 4) == 0 && (((uintptr_t)x | (uintptr_t)out) & 15) == 0 &&
                      ((uintptr_t)gain & (sizeof(T) == 4 ? 15 : 7)) == 0;
  const int nv = (hidden / 4 + 31) / 32;
  if (vec_ok && nv <= 4)
    return launch_pdl(rmsnorm_reg_kernel<T, 4>, dim3(blocks), dim3(warps * 32), 0, s, x, gain, out, dst_row, rows, hidden, eps);
  else if (vec_ok && nv <= 9)   // hidden <= 1152: 48 registers, five blocks per SM
    return launch_pdl(rmsnorm_reg_kernel<T, 9>, dim3(blocks), dim3(warps * 32), 0, s, x, gain, out, dst_row, rows, hidden, eps);
  else if (vec_ok && nv <= 13)
    return launch_pdl(rmsnorm_reg_kernel<T, 13>, dim3(blocks), dim3(warps * 32), 0, s, x, gain, out, dst_row, rows, hidden, eps);
  else if (vec_ok && nv <= 26)
    return launch_pdl(rmsnorm_reg_kernel<T, 26>, dim3(blocks), dim3(warps * 32), 0, s, x, gain, out, dst_row, rows, hidden, eps);
  else
    return launch_pdl(rmsnorm_kernel<T>, dim3(blocks), dim3(warps * 32), 0, s, x, gain, out, dst_row, rows, hidden, eps);
}

cudaError_t rmsnorm(int dtype, const void* x, const void* gain, void* out, const int32_t* dst_row, int64_t T,
                    int hidden, float eps, cudaStream_t s) {
  if (T == 0) return cudaSuccess;
  if (dtype == EPD_DTYPE_F32)
    return rmsnorm_t<float>((const float*)x, (const float*)gain, (float*)out, dst_row, T, hidden, eps, s);
  return rmsnorm_t<__nv_bfloat16>((const float*)x, (const __nv_bfloat16*)gain, (__nv_bfloat16*)out, dst_row, T, hidden,
                                  eps, s);
}

// =============================================================================================
// Rotary table and rotary + head split.
// table[p * nf + f] = (cos(p w_f), sin(p w_f)), w_f = theta^(-2f/(head_dim/2)), nf = head_dim/4.
// =============================================================================================
__global__ void rope_table_kernel(float2* table, int rows, int nf, int d2, double theta) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= rows * nf) return;
  const int p = idx / nf, f = idx % nf;
  const double w = pow(theta, -2.0 * (double)f / (double)d2);
  double sn, cs;
  sincos((double)p * w, &sn, &cs);
  table[idx] = make_float2((float)cs, (float)sn);
}

cudaError_t rope_table(float2* table, int rows, int head_dim, float theta, cudaStream_t s) {
  const int nf = head_dim / 4;
  const int total = rows * nf;
  if (total == 0) return cudaSuccess;
  rope_table_kernel<<<(total + 127) / 128, 128, 0, s>>>(table, rows, nf, head_dim / 2, (double)theta);
  return cudaGetLastError();
}

// One block per token.  Threads walk the token's q|k|v row in units of 2 adjacent frequencies
// (so loads and stores are 2-element vectors for bf16): unit u of a head covers pairs
// (f, f+nf), (f+1, f+1+nf) of one half.
template <typename T>
__global__ void __launch_bounds__(128)
rope_split_kernel(const T* __restrict__ qkv, const int32_t* __restrict__ pos_row,
                  const int32_t* __restrict__ pos_col, const float2* __restrict__ table, int table_rows,
                  T* __restrict__ q, T* __restrict__ k, T* __restrict__ v, int64_t Tn, int heads, int dh, int dhp,
                  float theta, float q_scale) {
  const int64_t j = blockIdx.x;
  const int h = heads * dh;
  const int d2 = dh / 2, nf = dh / 4;
  const T* row = qkv + j * 3 * (int64_t)h;
  const int pr = pos_row[j], pc = pos_col[j];
  const bool rotate = theta > 0.0f;
  // q and k: heads * 2 halves * nf frequencies, for 2 tensors
  const int n_rot = 2 * heads * 2 * nf;
  for (int e = threadIdx.x; e < n_rot; e += blockDim.x) {
    const int f = e % nf;
    int rest = e / nf;
    const int half = rest & 1; rest >>= 1;
    const int hd = rest % heads;
    const int which = rest / heads;  // 0 = q, 1 = k
    const int p = half ? pc : pr;
    float cs = 1.0f, sn = 0.0f;
    if (rotate) {
      if (table != nullptr && p < table_rows) {
        const float2 t = table[p * nf + f];
        cs = t.x; sn = t.y;
      } else {
        const double w = pow((double)theta, -2.0 * (double)f / (double)d2);
        double s_, c_;
        sincos((double)p * w, &s_, &c_);
        cs = (float)c_; sn = (float)s_;
      }
    }
    const int i0 = half * d2 + f, i1 = i0 + nf;
    const T* src = row + which * h + hd * dh;
    const float a = to_float<T>(src[i0]), b = to_float<T>(src[i1]);
    float ra = a * cs - b * sn, rb = b * cs + a * sn;
    if (which == 0) { ra *= q_scale; rb *= q_scale; }
    T* dst = (which == 0 ? q : k) + ((int64_t)hd * Tn + j) * dhp;
    dst[i0] = from_float<T>(ra);
    dst[i1] = from_float<T>(rb);
  }
  // v copy and zero padding of all three
  for (int e = threadIdx.x; e < heads * dhp; e += blockDim.x) {
    const int d = e % dhp, hd = e / dhp;
    const int64_t o = ((int64_t)hd * Tn + j) * dhp + d;
    if (d < dh) {
      v[o] = row[2 * h + hd * dh + d];
    } else {
      v[o] = from_float<T>(d == dh ? 1.0f : 0.0f);   // column head_dim of v is 1: P V then also yields the row sums
      q[o] = from_float<T>(0.0f);
      k[o] = from_float<T>(0.0f);
    }
  }
}

// Vector form of the same step.  A block stages the q|k|v rows of a few consecutive tokens in shared
// memory with 16-byte loads (the rows are contiguous in global memory) together with the tokens'
// (cos, sin) values; rotates q and k in place there, two adjacent frequencies per thread (one
// 2-element load per side of the pair); then copies whole 16-byte pieces out to the head-major rows:
// consecutive threads write consecutive pieces of (tensor, head, token), so the stores cover runs of
// tokens * head_dim_padded elements.  Needs head_dim to be a multiple of the 16-byte vector width.
template <typename T> struct Pair;
template <> struct Pair<float> {
  using type = float2;
  static __device__ __forceinline__ float2 unpack(float2 v) { return v; }
  static __device__ __forceinline__ float2 pack(float a, float b) { return make_float2(a, b); }
};
template <> struct Pair<__nv_bfloat16> {
  using type = __nv_bfloat162;
  static __device__ __forceinline__ float2 unpack(__nv_bfloat162 v) { return __bfloat1622float2(v); }
  static __device__ __forceinline__ __nv_bfloat162 pack(float a, float b) { return __floats2bfloat162_rn(a, b); }
};

template <typename T>
__global__ void __launch_bounds__(512)
rope_split_vec_kernel(const T* __restrict__ qkv, const int32_t* __restrict__ pos_row,
                      const int32_t* __restrict__ pos_col, const float2* __restrict__ table, int table_rows,
                      T* __restrict__ q, T* __restrict__ k, T* __restrict__ v, int64_t Tn, int heads, int dh, int dhp,
                      int tok_per_block, float theta, float q_scale) {
  pdl_launch_dependents();
  pdl_wait();
  constexpr int VEC = 16 / (int)sizeof(T);
  using P2 = typename Pair<T>::type;
  extern __shared__ __align__(16) uint8_t rope_smem[];
  const int h = heads * dh, row_elems = 3 * h;
  const int d2 = dh / 2, nf = dh / 4, nf2 = nf / 2;
  const int64_t j0 = (int64_t)blockIdx.x * tok_per_block;
  const int ntok = (int)min((int64_t)tok_per_block, Tn - j0);
  T* s_in = reinterpret_cast<T*>(rope_smem);
  float2* s_cs = reinterpret_cast<float2*>(rope_smem + (size_t)tok_per_block * row_elems * sizeof(T));

  const uint4* src = reinterpret_cast<const uint4*>(qkv + j0 * row_elems);
  const int nvec = ntok * (row_elems / VEC);
  for (int i = threadIdx.x; i < nvec; i += blockDim.x) reinterpret_cast<uint4*>(s_in)[i] = src[i];
  for (int i = threadIdx.x; i < ntok * 2 * nf; i += blockDim.x) {
    const int f = i % nf, half = (i / nf) & 1, t = i / (2 * nf);
    const int p = half ? pos_col[j0 + t] : pos_row[j0 + t];
    float2 cs = make_float2(1.0f, 0.0f);
    if (theta > 0.0f) {
      if (table != nullptr && p < table_rows) {
        cs = table[p * nf + f];
      } else {
        const double w = pow((double)theta, -2.0 * (double)f / (double)d2);
        double s_, c_;
        sincos((double)p * w, &s_, &c_);
        cs = make_float2((float)c_, (float)s_);
      }
    }
    s_cs[i] = cs;
  }
  __syncthreads();

  // rotate q and k in place: unit i = (head, half, frequency pair); index arithmetic once per unit
  const int units = heads * 2 * nf2;
  for (int i = threadIdx.x; i < units; i += blockDim.x) {
    const int fp = i % nf2;
    const int rest = i / nf2;
    const int half = rest & 1, hd = rest >> 1;
    const int e0 = hd * dh + half * d2 + 2 * fp;   // element of the pair's first member inside q (or k)
    const int c0 = half * nf + 2 * fp;             // its (cos, sin) entry inside the token's list
    for (int t = 0; t < ntok; ++t) {
      const float4 cs = *reinterpret_cast<const float4*>(s_cs + t * 2 * nf + c0);  // cos0 sin0 cos1 sin1
#pragma unroll
      for (int which = 0; which < 2; ++which) {
        T* base = s_in + t * row_elems + which * h + e0;
        const float2 a = Pair<T>::unpack(*reinterpret_cast<const P2*>(base));
        const float2 b = Pair<T>::unpack(*reinterpret_cast<const P2*>(base + nf));
        const float sc = which == 0 ? q_scale : 1.0f;
        const float ra0 = (a.x * cs.x - b.x * cs.y) * sc, rb0 = (b.x * cs.x + a.x * cs.y) * sc;
        const float ra1 = (a.y * cs.z - b.y * cs.w) * sc, rb1 = (b.y * cs.z + a.y * cs.w) * sc;
        *reinterpret_cast<P2*>(base) = Pair<T>::pack(ra0, ra1);
        *reinterpret_cast<P2*>(base + nf) = Pair<T>::pack(rb0, rb1);
      }
    }
  }
  __syncthreads();

  // copy out: a warp takes whole (tensor, head) pairs; the ntok padded rows of a pair are contiguous in
  // global memory, so consecutive lanes write consecutive 16-byte pieces
  const int vec_per_row = dhp / VEC, data_vecs = dh / VEC;
  const int per_pair = ntok * vec_per_row;
  const unsigned inv_vpr = (65536u + vec_per_row - 1) / vec_per_row;   // r / vec_per_row for r < 4096
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
  for (int pair = warp; pair < 3 * heads; pair += nwarps) {
    const int which = pair / heads, hd = pair - which * heads;
    const T* sbase = s_in + which * h + hd * dh;
    T* gbase = (which == 0 ? q : which == 1 ? k : v) + ((int64_t)hd * Tn + j0) * dhp;
    for (int r = lane; r < per_pair; r += 32) {
      const int t = (int)((r * inv_vpr) >> 16), ov = r - t * vec_per_row;
      uint4 pk = make_uint4(0u, 0u, 0u, 0u);
      if (ov < data_vecs) pk = *reinterpret_cast<const uint4*>(sbase + t * row_elems + ov * VEC);
      // column head_dim of v is 1 (the rest of the padding 0): P V then also yields the row sums
      else if (which == 2 && ov == data_vecs) pk.x = sizeof(T) == 4 ? 0x3F800000u : 0x00003F80u;
      *reinterpret_cast<uint4*>(gbase + r * VEC) = pk;
    }
  }
}

template <typename T>
static cudaError_t rope_split_t(const T* qkv, const int32_t* pos_row, const int32_t* pos_col, const float2* table,
                                int table_rows, T* q, T* k, T* v, int64_t Tn, int heads, int dh, float theta,
                                float q_scale, cudaStream_t s) {
  constexpr int VEC = 16 / (int)sizeof(T);
  const int dhp = padded_head_dim(dh);
  const size_t row_bytes = (size_t)3 * heads * dh * sizeof(T);
  const bool aligned = ((((uintptr_t)qkv | (uintptr_t)q | (uintptr_t)k | (uintptr_t)v)) & 15) == 0;
  if (aligned && dh % 8 == 0 && row_bytes + 2 * (dh / 4) * sizeof(float2) <= 96 * 1024) {
    // 8 tokens per block (fewer for very wide rows); as many threads as there are rotation units
    // (head, half, frequency pair), so that the rotation takes whole passes
    int tok = (int)(65536 / row_bytes);
    tok = tok < 1 ? 1 : tok > 8 ? 8 : tok;
    const size_t smem = tok * (row_bytes + 2 * (dh / 4) * sizeof(float2));
    const int units = heads * 2 * (dh / 8);
    const int passes = (units + 511) / 512;
    int threads = ((units + passes - 1) / passes + 31) / 32 * 32;
    threads = threads < 128 ? 128 : threads;
    auto kern = rope_split_vec_kernel<T>;
    static size_t configured = 48 * 1024;
    if (smem > configured) {
      cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024);
      if (e != cudaSuccess) return e;
      configured = 100 * 1024;
    }
    return launch_pdl(kern, dim3((unsigned)((Tn + tok - 1) / tok)), dim3(threads), smem, s, qkv, pos_row, pos_col, table,
                      table_rows, q, k, v, Tn, heads, dh, dhp, tok, theta, q_scale);
  } else {
    rope_split_kernel<T><<<(unsigned)Tn, 128, 0, s>>>(qkv, pos_row, pos_col, table, table_rows, q, k, v, Tn, heads, dh,
                                                      dhp, theta, q_scale);
  }
  return cudaGetLastError();
}

cudaError_t rope_split(int dtype, const void* qkv, const int32_t* pos_row, const int32_t* pos_col,
                       const float2* table, int table_rows, void* q, void* k, void* v, int64_t T, int heads,
                       int head_dim, float theta, float q_scale, cudaStream_t s) {
  if (T == 0) return cudaSuccess;
  if (dtype == EPD_DTYPE_F32)
    return rope_split_t<float>((const float*)qkv, pos_row, pos_col, table, table_rows, (float*)q, (float*)k,
                               (float*)v, T, heads, head_dim, theta, q_scale, s);
  return rope_split_t<__nv_bfloat16>((const __nv_bfloat16*)qkv, pos_row, pos_col, table, table_rows,
                                     (__nv_bfloat16*)q, (__nv_bfloat16*)k, (__nv_bfloat16*)v, T, heads, head_dim,
                                     theta, q_scale, s);
}

// =============================================================================================
// Attention with plain FMAs: one warp per (query token, head).  Keys are visited 32 at a time:
// lane l scores key l of the chunk, the warp keeps a running max / sum (online softmax, base 2:
// q arrives multiplied by log2(e)/sqrt(head_dim)), and lane l accumulates output dims l, l+32, ...
// =============================================================================================
template <typename T>
__global__ void __launch_bounds__(256)
attention_fma_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                     const int32_t* __restrict__ cu, int n_seg, T* __restrict__ out, int64_t Tn, int heads, int dh,
                     int dhp) {
  __shared__ float sq[8][kMaxHeadDim];
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  const int64_t j = (int64_t)blockIdx.x * 8 + wid;
  const int hd = blockIdx.y;
  if (j >= Tn) return;
  int lo = 0, hi = n_seg;
  while (hi - lo > 1) {
    int mid = (lo + hi) >> 1;
    if (cu[mid] <= j) lo = mid; else hi = mid;
  }
  const int kbeg = cu[lo], kend = cu[lo + 1];
  const T* qrow = q + ((int64_t)hd * Tn + j) * dhp;
  for (int d = lane; d < dh; d += 32) sq[wid][d] = to_float<T>(qrow[d]);
  __syncwarp();
  float m = -INFINITY, l = 0.0f;
  float acc[kMaxHeadDim / 32] = {};
  for (int c0 = kbeg; c0 < kend; c0 += 32) {
    const int key = c0 + lane;
    float sc = -INFINITY;
    if (key < kend) {
      const T* krow = k + ((int64_t)hd * Tn + key) * dhp;
      float dot = 0.0f;
      for (int d = 0; d < dh; ++d) dot = fmaf(sq[wid][d], to_float<T>(krow[d]), dot);
      sc = dot;
    }
    float cmax = sc;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) cmax = fmaxf(cmax, __shfl_xor_sync(0xffffffffu, cmax, o));
    const float m_new = fmaxf(m, cmax);
    const float scale = exp2f(m - m_new);
    const float p = exp2f(sc - m_new);
    float psum = p;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) psum += __shfl_xor_sync(0xffffffffu, psum, o);
    l = l * scale + psum;
    m = m_new;
#pragma unroll
    for (int i = 0; i < kMaxHeadDim / 32; ++i) acc[i] *= scale;
    const int nk = min(32, kend - c0);
    for (int kk = 0; kk < nk; ++kk) {
      const float pk = __shfl_sync(0xffffffffu, p, kk);
      const T* vrow = v + ((int64_t)hd * Tn + c0 + kk) * dhp;
#pragma unroll
      for (int i = 0; i < kMaxHeadDim / 32; ++i) {
        const int d = lane + 32 * i;
        if (d < dh) acc[i] = fmaf(pk, to_float<T>(vrow[d]), acc[i]);
      }
    }
  }
  const float inv = 1.0f / l;
  T* orow = out + j * (int64_t)(heads * dh) + hd * dh;
#pragma unroll
  for (int i = 0; i < kMaxHeadDim / 32; ++i) {
    const int d = lane + 32 * i;
    if (d < dh) orow[d] = from_float<T>(acc[i] * inv);
  }
}

cudaError_t attention_fma(int dtype, const void* q, const void* k, const void* v, const int32_t* cu_seqlens,
                          int n_seg, void* out, int64_t T, int heads, int head_dim, cudaStream_t s) {
  if (T == 0) return cudaSuccess;
  const int dhp = padded_head_dim(head_dim);
  dim3 grid((unsigned)((T + 7) / 8), (unsigned)heads);
  if (dtype == EPD_DTYPE_F32)
    attention_fma_kernel<float><<<grid, 256, 0, s>>>((const float*)q, (const float*)k, (const float*)v, cu_seqlens,
                                                     n_seg, (float*)out, T, heads, head_dim, dhp);
  else
    attention_fma_kernel<__nv_bfloat16><<<grid, 256, 0, s>>>((const __nv_bfloat16*)q, (const __nv_bfloat16*)k,
                                                             (const __nv_bfloat16*)v, cu_seqlens, n_seg,
                                                             (__nv_bfloat16*)out, T, heads, head_dim, dhp);
  return cudaGetLastError();
}

// =============================================================================================
// 2x2 merge as a gather: slot s = 4*o + q of the merged matrix copies row merge_idx[s] of y.
// =============================================================================================
__global__ void __launch_bounds__(128)
merge_gather_kernel(const uint8_t* __restrict__ y, const int32_t* __restrict__ merge_idx, uint8_t* __restrict__ out,
                    int64_t slots, int row_bytes) {
  const int64_t s = blockIdx.x;
  if (s >= slots) return;
  const uint8_t* src = y + (int64_t)merge_idx[s] * row_bytes;
  uint8_t* dst = out + s * row_bytes;
  if ((row_bytes & 15) == 0) {
    for (int i = threadIdx.x; i < row_bytes / 16; i += blockDim.x)
      reinterpret_cast<uint4*>(dst)[i] = reinterpret_cast<const uint4*>(src)[i];
  } else {
    for (int i = threadIdx.x; i < row_bytes / 2; i += blockDim.x)
      reinterpret_cast<uint16_t*>(dst)[i] = reinterpret_cast<const uint16_t*>(src)[i];
  }
}

cudaError_t merge_gather(int dtype, const void* y, const int32_t* merge_idx, void* out, int64_t Tm, int hidden,
                         cudaStream_t s) {
  if (Tm == 0) return cudaSuccess;
  const int row_bytes = hidden * (dtype == EPD_DTYPE_F32 ? 4 : 2);
  merge_gather_kernel<<<(unsigned)(Tm * 4), 128, 0, s>>>((const uint8_t*)y, merge_idx, (uint8_t*)out, Tm * 4,
                                                         row_bytes);
  return cudaGetLastError();
}

}  // namespace epd
