// bf16 linear layer on the 5th-generation tensor cores:  out = act(x . w^T + bias) (+ out).
//
// One persistent CTA per SM walks output tiles of 128 x BN.  Warp roles:
//   warp 0      TMA producer: cp.async.bulk.tensor loads of 128x64 (x) and BNx64 (w) bf16 boxes,
//               128-byte swizzle, into a STAGES-deep shared-memory ring
//   warp 1      allocates tensor memory and issues tcgen05.mma (one thread), fp32 accumulators in
//               TMEM, two accumulator buffers so the epilogue of tile i overlaps the loop of tile i+1
//   warps 2..5  epilogue: tcgen05.ld the accumulators (warp w reads TMEM lanes 32*(w%4)..+32),
//               bias / GELU in registers, 32-row x 128-byte chunks staged in swizzled shared
//               memory and written with TMA: a plain tensor store, or for the residual update
//               a tensor reduce-add (out += tile) so the old values never travel to the SM
// Both operands are K-major (row-major [rows, K]), so one shared-memory descriptor form serves both.
// Ragged M, N and K are handled by TMA: zero fill on loads, clipping on stores.
// Every mbarrier wait is bounded: on expiry the kernel records EPD_ETIMEOUT and drains.
#include "tcgen05_common.cuh"

namespace epd {
namespace {

using namespace tc;

constexpr int BM = 128;
constexpr int BK = 64;          // 64 bf16 = 128 bytes = one swizzle row
constexpr int UMMA_K = 16;
constexpr int kEpiWarps = 4;
constexpr int kThreads = 32 * (2 + kEpiWarps);

// D[tmem] (+)= A[smem] . B[smem]^T, bf16 inputs, fp32 accumulation, issued by one thread.
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = BN.
__host__ __device__ constexpr uint32_t instr_desc_bf16(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}

template <int BN, int STAGES>
struct SmemLayout {
  static constexpr int kABytes = BM * BK * 2;
  static constexpr int kBBytes = BN * BK * 2;
  static constexpr int kStageBytes = kABytes + kBBytes;
  // output staging: per epilogue warp kOutBufs buffers of 32 rows x 128 bytes (1024-byte aligned)
  static constexpr int kOutBufs = BN >= 256 ? 1 : 2;
  static constexpr int kOutBufBytes = 32 * 128;
  static constexpr int kOutOffset = STAGES * kStageBytes;
  static constexpr int kBarOffset = kOutOffset + kEpiWarps * kOutBufs * kOutBufBytes;
  // full[STAGES], empty[STAGES], tmem_full[2], tmem_empty[2], drain, (spare), tmem base, abort flag,
  // bias[kEpiWarps][BN]
  static constexpr int kBiasOffset = kBarOffset + (2 * STAGES + 6) * 8 + 16;
  static constexpr int kTotal = kBiasOffset + kEpiWarps * BN * 4;
  static_assert(kTotal + 1024 <= 232448, "exceeds the shared memory of one CTA");
  static constexpr int kDynamic = kTotal + 1024;  // slack to align the ring to 1024 bytes
};

// ---------------------------------------------------------------------------------------------
// Kernel
// ---------------------------------------------------------------------------------------------
template <int BN, int STAGES, typename OutT, int ACT, bool ACCUM>
__global__ void __launch_bounds__(kThreads, 1)
linear_tc_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_w,
                 const __grid_constant__ CUtensorMap tm_out, const __nv_bfloat16* __restrict__ bias, int M, int N,
                 int K, int* __restrict__ status, long long wait_limit) {
  using L = SmemLayout<BN, STAGES>;
  static_assert(L::kDynamic > 116 * 1024, "one CTA per SM is assumed by the TMEM allocation");
  static_assert(BN % 16 == 0 && BN >= 32 && BN <= 256, "UMMA N");
  constexpr int kAccStride = BN <= 128 ? 128 : 256;  // TMEM columns between the two accumulators
  constexpr int kTmemCols = 2 * kAccStride;

  pdl_launch_dependents();
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + L::kBarOffset);
  uint64_t* empty = full + STAGES;
  uint64_t* tmem_full = empty + STAGES;
  uint64_t* tmem_empty = tmem_full + 2;
  uint64_t* drain_bar = tmem_empty + 2;    // after an abort: the issuing thread's MMAs have completed
  uint32_t* tmem_base_slot = reinterpret_cast<uint32_t*>(drain_bar + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_base_slot + 1);
  const WaitCtx wc{abort_flag, 0u, wait_limit};
  uint32_t loads_issued = 0;               // stage loads issued by the producer thread
  float* bias_s = reinterpret_cast<float*>(smem + L::kBiasOffset);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m_tiles = (M + BM - 1) / BM, n_tiles = (N + BN - 1) / BN;
  const int num_tiles = m_tiles * n_tiles;
  const int k_blocks = (K + BK - 1) / BK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&tmem_full[a], 1); mbar_init(&tmem_empty[a], kEpiWarps); }
    mbar_init(drain_bar, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc(tmem_base_slot, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_base_slot;
  pdl_wait();   // nothing above touches global memory

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    // The whole warp walks the loop and one elected lane issues (see elect_one()).
    {
      if (lane == 0) {
        prefetch_map(&tm_x);
        prefetch_map(&tm_w);
      }
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
        const int m0 = (tile % m_tiles) * BM, n0 = (tile / m_tiles) * BN;
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!mbar_wait_warp(&empty[stage], phase ^ 1, wc)) { ok = false; break; }
          uint8_t* sa = smem + stage * L::kStageBytes;
          if (elect_one()) {
            mbar_expect_tx(&full[stage], L::kStageBytes);
            tma_load_2d(sa, &tm_x, kb * BK, m0, &full[stage]);
            tma_load_2d(sa + L::kABytes, &tm_w, kb * BK, n0, &full[stage]);
          }
          __syncwarp();
          ++loads_issued;
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    // The whole warp walks the loop and one elected lane issues.
    {
      constexpr uint32_t idesc = instr_desc_bf16(BN);
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
        if (!mbar_wait_warp(&tmem_empty[acc], acc_phase ^ 1, wc)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * kAccStride;
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!mbar_wait_warp(&full[stage], phase, wc)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = smem_u32(smem + stage * L::kStageBytes);
          const uint64_t da = smem_desc_k_sw128(sa), db = smem_desc_k_sw128(sa + L::kABytes);
          if (elect_one()) {
#pragma unroll
            for (int k = 0; k < BK / UMMA_K; ++k) {
              // advancing 16 bf16 along K inside the swizzled row = 32 bytes = 2 descriptor units
              umma_bf16(d_tmem, da + 2 * k, db + 2 * k, idesc, (kb | k) != 0);
            }
            umma_commit(&empty[stage]);
          }
          __syncwarp();
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
        if (!ok) break;
        if (elect_one()) umma_commit(&tmem_full[acc]);
        __syncwarp();
        if (++acc == 2) { acc = 0; acc_phase ^= 1; }
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------------ epilogue
    constexpr int CC = sizeof(OutT) == 4 ? 32 : 64;  // columns per staged chunk: 128 bytes per row
    const int q = warp & 3;                          // TMEM lane quarter this warp may read
    float* bs = bias_s + (warp - 2) * BN;            // this warp's private copy of the tile's bias values
    uint8_t* stage_out = smem + L::kOutOffset + (warp - 2) * L::kOutBufs * L::kOutBufBytes;
    int obuf = 0;
    int acc = 0;
    uint32_t acc_phase = 0;
    if (lane == 0) prefetch_map(&tm_out);
    for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x) {
      const int m0 = (tile % m_tiles) * BM, n0 = (tile / m_tiles) * BN;
      __syncwarp();
      for (int i = lane; i < BN; i += 32)
        bs[i] = (bias != nullptr && n0 + i < N) ? __bfloat162float(bias[n0 + i]) : 0.0f;
      __syncwarp();
      if (!mbar_wait_warp(&tmem_full[acc], acc_phase, wc)) break;
      tc_fence_after();
      const int row0 = m0 + q * 32;
      const uint32_t taddr = tmem_base + acc * kAccStride + ((uint32_t)(q * 32) << 16);
#pragma unroll 1
      for (int c = 0; c < BN / CC; ++c) {
        uint32_t pk[32];  // this thread's row of the chunk, as stored: 32 floats or 64 bf16
        if constexpr (sizeof(OutT) == 4) {
          tmem_ld32(taddr + c * CC, pk);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            float t = __uint_as_float(pk[j]) + bs[c * CC + j];
            if (ACT == 1) t = gelu_tanh_fast(t);
            if (ACT == 2) t = gelu_erf_fast(t);
            pk[j] = __float_as_uint(t);
          }
        } else {
          uint32_t r0[32], r1[32];
          tmem_ld32(taddr + c * CC, r0);
          tmem_ld32(taddr + c * CC + 32, r1);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const uint32_t* src = j < 16 ? r0 : r1;
            const int jj = (2 * j) & 31;
            float t0 = __uint_as_float(src[jj]) + bs[c * CC + 2 * j];
            float t1 = __uint_as_float(src[jj + 1]) + bs[c * CC + 2 * j + 1];
            if (ACT == 1) { t0 = gelu_tanh_fast(t0); t1 = gelu_tanh_fast(t1); }
            if (ACT == 2) { t0 = gelu_erf_fast(t0); t1 = gelu_erf_fast(t1); }
            __nv_bfloat162 b = __floats2bfloat162_rn(t0, t1);
            pk[j] = *reinterpret_cast<uint32_t*>(&b);
          }
        }
        if (c == BN / CC - 1) {
          // all accumulator columns of this tile have been read: hand the buffer back
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&tmem_empty[acc]);
        }
        // the staging buffer is free once the bulk store issued from it has read it
        if (lane == 0) bulk_wait_read<L::kOutBufs - 1>();
        __syncwarp();
        uint8_t* sbuf = stage_out + obuf * L::kOutBufBytes;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          // 128-byte swizzle: 16-byte chunk j of row r lives at chunk position j ^ (r % 8)
          uint4* dst = reinterpret_cast<uint4*>(sbuf + lane * 128 + ((j ^ (lane & 7)) << 4));
          *dst = make_uint4(pk[4 * j], pk[4 * j + 1], pk[4 * j + 2], pk[4 * j + 3]);
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) {
          if (row0 < M && n0 + c * CC < N) {
            if (ACCUM) tma_reduce_add_2d(&tm_out, n0 + c * CC, row0, sbuf);
            else tma_store_2d(&tm_out, n0 + c * CC, row0, sbuf);
          }
          bulk_commit();
        }
        if (++obuf == L::kOutBufs) obuf = 0;
      }
      if (++acc == 2) { acc = 0; acc_phase ^= 1; }
    }
    if (lane == 0) bulk_wait_all();
    __syncwarp();
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    // A wait expired.  Every role has left its loop (the barrier above), so nothing new is issued.  What was
    // issued completes by itself: the producer waits for its last load of every stage, the issuing thread for
    // its last MMA (a commit arrives only after all earlier MMAs), the epilogue warps have waited for their
    // stores; a fixed pause on top, then shared and tensor memory are released.
    if (threadIdx.x == 0 && status != nullptr) atomicCAS(status, 0, kStatusTimeout);
    if (warp == 0 && lane == 0) drain_ring(full, STAGES, loads_issued);
    if (warp == 1 && elect_one()) {   // the lane that issued the products: a commit covers the products of its own thread
      umma_commit(drain_bar);
      mbar_wait_drain(drain_bar, 0);
    }
    for (int i = 0; i < 64; ++i) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ---------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------
// Tensor map of a row-major matrix [rows, cols] with leading dimension ld (elements of elem_bytes),
// box = box_rows x (128 bytes of columns), 128-byte swizzle.
bool make_map(CUtensorMap* tm, const void* base, int64_t rows, int64_t cols, int64_t ld, int box_rows,
              int elem_bytes) {
  return make_tensor_map_2d(tm, base, rows, cols, ld * elem_bytes, box_rows, 128 / elem_bytes, elem_bytes,
                            CU_TENSOR_MAP_SWIZZLE_128B);
}

template <int BN, int STAGES, typename OutT, int ACT, bool ACCUM>
cudaError_t launch(const CUtensorMap& tx, const CUtensorMap& tw, const CUtensorMap& to, const void* bias, int M, int N,
                   int K, int* status, cudaStream_t s) {
  using L = SmemLayout<BN, STAGES>;
  auto kern = linear_tc_kernel<BN, STAGES, OutT, ACT, ACCUM>;
  static PerDeviceOnce configured;
  cudaError_t e = once_per_device(configured, [&] {
    return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kDynamic);
  });
  if (e != cudaSuccess) return e;
  const int tiles = ((M + BM - 1) / BM) * ((N + BN - 1) / BN);
  const int sms_avail = limited_sms(device_sm_count());
  const int grid = tiles < sms_avail ? tiles : sms_avail;
  return launch_pdl(kern, dim3(grid), dim3(kThreads), L::kDynamic, s, tx, tw, to, (const __nv_bfloat16*)bias, M, N, K, status,
                    wait_limit_cycles());
}

template <int BN, int STAGES>
cudaError_t launch_bn(const CUtensorMap& tx, const CUtensorMap& tw, const CUtensorMap& to, const void* bias, int M,
                      int N, int K, int flags, int* status, cudaStream_t s) {
  const int act = (flags & EPD_LINEAR_GELU_TANH) ? 1 : (flags & EPD_LINEAR_GELU_ERF) ? 2 : 0;
  const bool accum = flags & EPD_LINEAR_ACCUMULATE;
  const bool out_f32 = accum || (flags & EPD_LINEAR_OUT_F32);
#define EPD_TC(OUT, A, C) return launch<BN, STAGES, OUT, A, C>(tx, tw, to, bias, M, N, K, status, s)
  if (accum) {
    if (act == 0) EPD_TC(float, 0, true);
    if (act == 1) EPD_TC(float, 1, true);
    EPD_TC(float, 2, true);
  }
  if (out_f32) {
    if (act == 0) EPD_TC(float, 0, false);
    if (act == 1) EPD_TC(float, 1, false);
    EPD_TC(float, 2, false);
  }
  if (act == 0) EPD_TC(__nv_bfloat16, 0, false);
  if (act == 1) EPD_TC(__nv_bfloat16, 1, false);
  EPD_TC(__nv_bfloat16, 2, false);
#undef EPD_TC
}

// Tile width: the candidate with the smallest estimated time = waves x tile width / efficiency.
// The efficiencies are the measured mainloop rates of each width relative to 256 (narrower tiles
// re-read the x operand from shared memory more often per flop).
int pick_bn(int M, int N) {
  const int cands[3] = {256, 192, 128};
  const double eff[3] = {1.0, 0.88, 0.65};
  const int sms = limited_sms(device_sm_count());
  const int m_tiles = (M + BM - 1) / BM;
  int best = 256;
  double best_cost = 1e300;
  for (int i = 0; i < 3; ++i) {
    const int bn = cands[i];
    const int tiles = m_tiles * ((N + bn - 1) / bn);
    const int waves = (tiles + sms - 1) / sms;
    const double cost = (double)waves * bn / eff[i];
    if (cost < best_cost) { best_cost = cost; best = bn; }
  }
  return best;
}

}  // namespace

bool linear_tc_supported(const void* x, int64_t ldx, const void* w, int64_t ldw, const void* bias, const void* out,
                         int64_t ldo, int64_t M, int64_t N, int64_t K, int flags) {
  (void)bias;
  const bool out_f32 = flags & (EPD_LINEAR_ACCUMULATE | EPD_LINEAR_OUT_F32);
  if (M < 1 || N < 8 || K < 8 || (N % 8) || M > (1 << 30) || N > (1 << 30) || K > (1 << 30)) return false;
  if (((uintptr_t)x & 15) || ((uintptr_t)w & 15) || ((uintptr_t)out & 15)) return false;
  if ((ldx % 8) || (ldw % 8) || (ldo % (out_f32 ? 4 : 8))) return false;
  return tensor_maps_available();
}

int linear_tc_launches(int64_t M, int64_t N, int64_t K, int flags, int forced_bn) {
  return (forced_bn == 0 && M > BM) ? linear_tc_pair_slices(N, K, flags) : 1;
}

cudaError_t linear_tc(const void* x, int64_t ldx, const void* w, int64_t ldw, const void* bias, void* out, int64_t ldo,
                      int64_t M, int64_t N, int64_t K, int flags, int forced_bn, int* status, cudaStream_t s) {
  // Without a forced tile width, anything taller than one 128-row tile goes to the CTA-pair kernel.
  if (forced_bn == 0 && M > BM) return linear_tc_pair(x, ldx, w, ldw, bias, out, ldo, M, N, K, flags, status, s);
  const int bn = forced_bn > 0 ? forced_bn : pick_bn((int)M, (int)N);
  const bool out_f32 = flags & (EPD_LINEAR_ACCUMULATE | EPD_LINEAR_OUT_F32);
  CUtensorMap tx, tw, to;
  if (!make_map(&tx, x, M, K, ldx, BM, 2) || !make_map(&tw, w, N, K, ldw, bn, 2) ||
      !make_map(&to, out, M, N, ldo, 32, out_f32 ? 4 : 2))
    return cudaErrorInvalidValue;
  switch (bn) {
    case 256: return launch_bn<256, 4>(tx, tw, to, bias, (int)M, (int)N, (int)K, flags, status, s);
    case 192: return launch_bn<192, 4>(tx, tw, to, bias, (int)M, (int)N, (int)K, flags, status, s);
    case 128: return launch_bn<128, 5>(tx, tw, to, bias, (int)M, (int)N, (int)K, flags, status, s);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace epd
