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
#include <cuda.h>

#include <mutex>

#include "common.cuh"

namespace epd {
namespace {

constexpr int BM = 128;
constexpr int BK = 64;          // 64 bf16 = 128 bytes = one swizzle row
constexpr int UMMA_K = 16;
constexpr int kEpiWarps = 4;
constexpr int kThreads = 32 * (2 + kEpiWarps);
constexpr long long kWaitCycles = 4000000000LL;  // ~2 s at 2 GHz

// ---------------------------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false (and raises *abort_flag) if the phase did not complete in time or
// another role already gave up.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  int spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 255) == 0) {
      if (*abort_flag) return false;
      if (clock64() - t0 > kWaitCycles) {
        *abort_flag = 1;
        return false;
      }
    }
  }
  return true;
}

__device__ __forceinline__ void tma_load_2d(void* smem_dst, const CUtensorMap* tm, int x, int y, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(smem_dst)), "l"(tm), "r"(smem_u32(bar)), "r"(x), "r"(y)
      : "memory");
}

// TMA tensor store / reduce-add of one staged box, tracked by the issuing thread's bulk group.
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* tm, int x, int y, const void* smem_src) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
               ::"l"(tm), "r"(smem_u32(smem_src)), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tma_reduce_add_2d(const CUtensorMap* tm, int x, int y, const void* smem_src) {
  asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%2, %3}], [%1];"
               ::"l"(tm), "r"(smem_u32(smem_src)), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void bulk_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t* smem_result, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_result)),
               "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t addr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(addr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

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
// mbarrier arrives once all tcgen05.mma issued so far by this thread have completed.
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}

// 32 lanes x 32 consecutive fp32 columns: thread i of the warp receives row (lane base + i).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major tile whose rows are 128 bytes, 128-byte swizzled
// (the layout a TMA box of 64 bf16 columns produces): 8-row groups are 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_k_sw128(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFF) >> 4);  // start address, 16-byte units
  d |= (uint64_t)1 << 16;                       // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;             // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                       // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                       // 128-byte swizzle
  return d;
}

// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = BN.
__host__ __device__ constexpr uint32_t instr_desc_bf16(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}

__device__ __forceinline__ float gelu_tanh_fast(float x) {
  const float u = 0.7978845608028654f * (x + 0.044715f * x * x * x);
  float t;
  asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(u));
  return 0.5f * x * (1.0f + t);
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
  // full[STAGES], empty[STAGES], tmem_full[2], tmem_empty[2], tmem base, abort flag, bias[kEpiWarps][BN]
  static constexpr int kBiasOffset = kBarOffset + (2 * STAGES + 4) * 8 + 16;
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
                 int K, int* __restrict__ status) {
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
  uint32_t* tmem_base_slot = reinterpret_cast<uint32_t*>(tmem_empty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_base_slot + 1);
  float* bias_s = reinterpret_cast<float*>(smem + L::kBiasOffset);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m_tiles = (M + BM - 1) / BM, n_tiles = (N + BN - 1) / BN;
  const int num_tiles = m_tiles * n_tiles;
  const int k_blocks = (K + BK - 1) / BK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&tmem_full[a], 1); mbar_init(&tmem_empty[a], kEpiWarps); }
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
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_x) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_w) : "memory");
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
        const int m0 = (tile % m_tiles) * BM, n0 = (tile / m_tiles) * BN;
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!mbar_wait(&empty[stage], phase ^ 1, abort_flag)) { ok = false; break; }
          uint8_t* sa = smem + stage * L::kStageBytes;
          mbar_expect_tx(&full[stage], L::kStageBytes);
          tma_load_2d(sa, &tm_x, kb * BK, m0, &full[stage]);
          tma_load_2d(sa + L::kABytes, &tm_w, kb * BK, n0, &full[stage]);
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = instr_desc_bf16(BN);
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
        if (!mbar_wait(&tmem_empty[acc], acc_phase ^ 1, abort_flag)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * kAccStride;
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!mbar_wait(&full[stage], phase, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = smem_u32(smem + stage * L::kStageBytes);
          const uint64_t da = smem_desc_k_sw128(sa), db = smem_desc_k_sw128(sa + L::kABytes);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            // advancing 16 bf16 along K inside the swizzled row = 32 bytes = 2 descriptor units
            umma_bf16(d_tmem, da + 2 * k, db + 2 * k, idesc, (kb | k) != 0);
          }
          umma_commit(&empty[stage]);
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
        if (!ok) break;
        umma_commit(&tmem_full[acc]);
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
    if (lane == 0) asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_out) : "memory");
    for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x) {
      const int m0 = (tile % m_tiles) * BM, n0 = (tile / m_tiles) * BN;
      __syncwarp();
      for (int i = lane; i < BN; i += 32)
        bs[i] = (bias != nullptr && n0 + i < N) ? __bfloat162float(bias[n0 + i]) : 0.0f;
      __syncwarp();
      if (!mbar_wait(&tmem_full[acc], acc_phase, abort_flag)) break;
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
            if (ACT == 2) t = gelu_erf_f(t);
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
            if (ACT == 2) { t0 = gelu_erf_f(t0); t1 = gelu_erf_f(t1); }
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
    // a wait expired: report it and give loads still in flight time to land before the CTA's
    // shared memory is released
    if (threadIdx.x == 0 && status != nullptr) atomicCAS(status, 0, kStatusTimeout);
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

// Tensor map of a row-major matrix [rows, cols] with leading dimension ld (elements of elem_bytes),
// box = box_rows x (128 bytes of columns), 128-byte swizzle.
bool make_map(CUtensorMap* tm, const void* base, int64_t rows, int64_t cols, int64_t ld, int box_rows,
              int elem_bytes) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)ld * elem_bytes};
  cuuint32_t box[2] = {(cuuint32_t)(128 / elem_bytes), (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(tm, elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2,
            const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int sm_count() {
  static int n = 0;
  if (n == 0) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
    if (n <= 0) n = 148;
  }
  return n;
}

template <int BN, int STAGES, typename OutT, int ACT, bool ACCUM>
cudaError_t launch(const CUtensorMap& tx, const CUtensorMap& tw, const CUtensorMap& to, const void* bias, int M, int N,
                   int K, int* status, cudaStream_t s) {
  using L = SmemLayout<BN, STAGES>;
  auto kern = linear_tc_kernel<BN, STAGES, OutT, ACT, ACCUM>;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kDynamic);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  const int tiles = ((M + BM - 1) / BM) * ((N + BN - 1) / BN);
  const int sms_avail = limited_sms(sm_count());
  const int grid = tiles < sms_avail ? tiles : sms_avail;
  return launch_pdl(kern, dim3(grid), dim3(kThreads), L::kDynamic, s, tx, tw, to, (const __nv_bfloat16*)bias, M, N, K, status);
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
  const int sms = limited_sms(sm_count());
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
  return encode_tiled_fn() != nullptr;
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
