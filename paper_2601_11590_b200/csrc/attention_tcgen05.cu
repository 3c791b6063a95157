// Block-diagonal bidirectional flash attention on the 5th-generation tensor cores.
//
// One CTA handles one (segment, head, 128-query tile) and streams the segment's keys/values in
// tiles of 128.  Per key tile:
//   S = Q K^T          tcgen05.mma, both operands K-major in shared memory, fp32 S in TMEM
//   online softmax     4 warps, one thread per query row: tcgen05.ld S, running max / sum in
//                      registers (base-2 exponentials; q arrives scaled by log2(e)/sqrt(head_dim)),
//                      P = exp2(S - m) written back over S in TMEM as bf16 (tcgen05.st)
//   O += P V           tcgen05.mma with P as the TMEM operand and V read MN-major from shared memory
// The running max is only advanced (and O rescaled in TMEM) when it grows by more than 2^8; until
// then the stale max is used for P, the row sum and O alike, so the result is unchanged.
// Warp roles: warp 0 TMA producer, warp 1 TMEM allocation + MMA issue, warps 2..5 softmax /
// rescale / epilogue.  Q, K and V tiles are single-buffered (K is reloaded while P V runs, V while
// the next Q K^T and softmax run); two CTAs share an SM so one CTA's softmax overlaps the other's
// MMAs.  head_dim 72 is stored padded to 80: columns 0..63 form a 128-byte-swizzled box, columns
// 64..79 a 32-byte-swizzled box, each fed to its own MMA.
// Every mbarrier wait is bounded: on expiry the kernel records EPD_ETIMEOUT and drains.
#include <cuda.h>

#include <mutex>

#include "common.cuh"

namespace epd {
namespace {

constexpr int BQ = 128;   // query rows per CTA
constexpr int BKV = 128;  // keys per tile
constexpr int kThreads = 192;
constexpr long long kWaitCycles = 4000000000LL;
constexpr float kRescaleThreshold = 8.0f;  // log2 of the largest P value tolerated before rescaling

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

// D[tmem] (+)= A[smem] . B[smem]
__device__ __forceinline__ void umma_ss(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                        uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
      : "memory");
}
// D[tmem] (+)= A[tmem] . B[smem]
__device__ __forceinline__ void umma_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t desc_b, uint32_t idesc,
                                        uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(tmem_d), "r"(tmem_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}

#define EPD_R16(r, o) "=r"(r[o + 0]), "=r"(r[o + 1]), "=r"(r[o + 2]), "=r"(r[o + 3]), "=r"(r[o + 4]), "=r"(r[o + 5]), \
    "=r"(r[o + 6]), "=r"(r[o + 7]), "=r"(r[o + 8]), "=r"(r[o + 9]), "=r"(r[o + 10]), "=r"(r[o + 11]),                \
    "=r"(r[o + 12]), "=r"(r[o + 13]), "=r"(r[o + 14]), "=r"(r[o + 15])
#define EPD_W16(r, o) "r"(r[o + 0]), "r"(r[o + 1]), "r"(r[o + 2]), "r"(r[o + 3]), "r"(r[o + 4]), "r"(r[o + 5]),       \
    "r"(r[o + 6]), "r"(r[o + 7]), "r"(r[o + 8]), "r"(r[o + 9]), "r"(r[o + 10]), "r"(r[o + 11]), "r"(r[o + 12]),       \
    "r"(r[o + 13]), "r"(r[o + 14]), "r"(r[o + 15])

// 32 lanes x 16 consecutive 32-bit columns: thread i of the warp owns lane (base + i).
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : EPD_R16(r, 0)
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* r) {
  tmem_ld16(taddr, r);
  tmem_ld16(taddr + 16, r + 16);
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), EPD_W16(r, 0)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Shared-memory matrix descriptor.  layout: 2 = 128-byte swizzle, 6 = 32-byte swizzle.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint32_t layout) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFF) >> 4);
  d |= (uint64_t)(lbo_bytes >> 4) << 16;
  d |= (uint64_t)(sbo_bytes >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)layout << 61;
  return d;
}
// bf16 x bf16 -> fp32, M = 128; b_mn = 1 when the B operand is MN-major (V: head_dim contiguous).
__device__ __forceinline__ uint32_t instr_desc(int n, int b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)b_mn << 16) | ((uint32_t)(n >> 3) << 17) |
         ((uint32_t)(128 >> 4) << 24);
}

// Shared-memory plan for a padded head width DHP (64, 80 or 128).
template <int DHP>
struct Plan {
  static constexpr int kMainBoxes = DHP / 64;          // 128-byte-swizzled boxes of 64 columns
  static constexpr int kTail = DHP % 64;               // 0 or 16 columns, 32-byte swizzle
  static_assert(kTail == 0 || kTail == 16, "padded head width must be 64*a or 64*a + 16");
  static constexpr int kMainBytes = BKV * 128;         // one main box: 128 rows x 128 bytes
  static constexpr int kTailBytes = kTail ? BKV * 32 : 0;
  static constexpr int kTileBytes = kMainBoxes * kMainBytes + kTailBytes;  // one of Q / K / V
  static constexpr int kQ = 0, kK = kTileBytes, kV = 2 * kTileBytes;
  static constexpr int kBar = 3 * kTileBytes;          // 9 mbarriers, tmem slot, abort flag, segment info
  static constexpr int kTotal = kBar + 9 * 8 + 32;
  // at most two CTAs per SM: each allocates 256 of the 512 TMEM columns
  static constexpr int kDynamic = (kTotal + 1024 > 78 * 1024) ? kTotal + 1024 : 78 * 1024;
  static constexpr int kOCols = DHP;                   // O accumulator columns, after the 128 S columns
};

struct Maps {
  CUtensorMap q_main, q_tail, k_main, k_tail, v_main, v_tail;
};

template <int DHP>
__global__ void __launch_bounds__(kThreads, 2)
attention_tc_kernel(const __grid_constant__ Maps maps, const int32_t* __restrict__ cu, int n_seg,
                    __nv_bfloat16* __restrict__ out, int T, int heads, int dh, int* __restrict__ status) {
  using P = Plan<DHP>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + P::kBar);
  uint64_t *q_full = bars, *k_full = bars + 1, *k_empty = bars + 2, *v_full = bars + 3, *v_empty = bars + 4,
           *s_full = bars + 5, *p_full = bars + 6, *o_done = bars + 7;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 9);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int head = blockIdx.y;

  // which segment and query tile: walk the segments (a few dozen at most)
  int tile = blockIdx.x, seg_beg = 0, seg_end = 0;
  for (int i = 0; i < n_seg; ++i) {
    const int b = cu[i], e = cu[i + 1];
    const int nt = (e - b + BQ - 1) / BQ;
    if (tile < nt) { seg_beg = b; seg_end = e; break; }
    tile -= nt;
  }
  const int q0 = seg_beg + tile * BQ;            // first query token of this CTA
  const int seg_len = seg_end - seg_beg;
  const int n_kv = (seg_len + BKV - 1) / BKV;
  const int row_base = head * T;                 // row of token 0 of this head in the [heads*T, DHP] matrices

  if (threadIdx.x == 0) {
    for (int i = 0; i < 8; ++i) mbar_init(&bars[i], i == 6 ? 4 : 1);  // p_full: one arrival per softmax warp
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, 256);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tmem_s = tmem_base;        // S (fp32, 128 columns), overwritten by P (bf16 pairs, 64 columns)
  const uint32_t tmem_o = tmem_base + 128;  // O (fp32, DHP columns)

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer
    if (lane == 0 && seg_len > 0) {
      auto load_tile = [&](uint8_t* dst, const CUtensorMap* mm, const CUtensorMap* mt, int row, uint64_t* bar) {
        mbar_expect_tx(bar, P::kTileBytes);
#pragma unroll
        for (int b = 0; b < P::kMainBoxes; ++b) tma_load_2d(dst + b * P::kMainBytes, mm, b * 64, row, bar);
        if (P::kTail) tma_load_2d(dst + P::kMainBoxes * P::kMainBytes, mt, P::kMainBoxes * 64, row, bar);
      };
      load_tile(smem + P::kQ, &maps.q_main, &maps.q_tail, row_base + q0, q_full);
      for (int j = 0; j < n_kv; ++j) {
        const int row = row_base + seg_beg + j * BKV;
        if (!mbar_wait(k_empty, (j & 1) ^ 1, abort_flag)) break;
        load_tile(smem + P::kK, &maps.k_main, &maps.k_tail, row, k_full);
        if (!mbar_wait(v_empty, (j & 1) ^ 1, abort_flag)) break;
        load_tile(smem + P::kV, &maps.v_main, &maps.v_tail, row, v_full);
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer
    if (lane == 0 && seg_len > 0) {
      const uint32_t sq = smem_u32(smem + P::kQ), sk = smem_u32(smem + P::kK), sv = smem_u32(smem + P::kV);
      bool ok = mbar_wait(q_full, 0, abort_flag);
      for (int j = 0; j < n_kv && ok; ++j) {
        const int kv_valid = min(BKV, seg_len - j * BKV);
        const int n16 = (kv_valid + 15) & ~15;  // keys taking part in this tile's MMAs
        // S and O of the previous tile must be complete before S is overwritten
        if (j > 0 && !mbar_wait(o_done, (j - 1) & 1, abort_flag)) { ok = false; break; }
        if (!mbar_wait(k_full, j & 1, abort_flag)) { ok = false; break; }
        tc_fence_after();
        {
          const uint32_t idesc = instr_desc(n16, 0);
          uint32_t accum = 0;
#pragma unroll
          for (int b = 0; b < P::kMainBoxes; ++b) {
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              umma_ss(tmem_s, smem_desc(sq + b * P::kMainBytes + k * 32, 16, 1024, 2),
                      smem_desc(sk + b * P::kMainBytes + k * 32, 16, 1024, 2), idesc, accum);
              accum = 1;
            }
          }
          if (P::kTail)
            umma_ss(tmem_s, smem_desc(sq + P::kMainBoxes * P::kMainBytes, 16, 256, 6),
                    smem_desc(sk + P::kMainBoxes * P::kMainBytes, 16, 256, 6), idesc, accum);
        }
        umma_commit(s_full);
        umma_commit(k_empty);
        if (!mbar_wait(p_full, j & 1, abort_flag)) { ok = false; break; }
        if (!mbar_wait(v_full, j & 1, abort_flag)) { ok = false; break; }
        tc_fence_after();
        {
          const uint32_t idesc_main = instr_desc(64, 1), idesc_tail = instr_desc(16, 1);
          for (int ks = 0; ks < n16 / 16; ++ks) {
            const uint32_t accum = (j | ks) != 0;
            const uint32_t a_tmem = tmem_s + ks * 8;  // 16 bf16 of P = 8 columns
#pragma unroll
            for (int b = 0; b < P::kMainBoxes; ++b)
              umma_ts(tmem_o + b * 64, a_tmem, smem_desc(sv + b * P::kMainBytes + ks * 2048, 16384, 1024, 2),
                      idesc_main, accum);
            if (P::kTail)
              umma_ts(tmem_o + P::kMainBoxes * 64, a_tmem,
                      smem_desc(sv + P::kMainBoxes * P::kMainBytes + ks * 512, 4096, 256, 6), idesc_tail, accum);
          }
        }
        umma_commit(v_empty);
        umma_commit(o_done);
      }
    }
    __syncwarp();
  } else if (seg_len > 0) {
    // ---------------------------------------------------------------- softmax / rescale / epilogue
    const int q = warp & 3;
    const int r = q * 32 + lane;                       // query row inside the tile
    const uint32_t lane_off = (uint32_t)(q * 32) << 16;
    float m = -INFINITY, l = 0.0f;
    bool ok = true;
    for (int j = 0; j < n_kv; ++j) {
      const int kv_valid = min(BKV, seg_len - j * BKV);
      const int n_chunks = (kv_valid + 31) >> 5;       // 32-column chunks that hold valid keys
      if (!mbar_wait(s_full, j & 1, abort_flag)) { ok = false; break; }
      tc_fence_after();
      // pass 1: row max over the valid keys
      float m_tile = -INFINITY;
      for (int c = 0; c < n_chunks; ++c) {
        uint32_t s[32];
        tmem_ld32(tmem_s + lane_off + c * 32, s);
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 32; ++i)
          if (c * 32 + i < kv_valid) m_tile = fmaxf(m_tile, __uint_as_float(s[i]));
      }
      // advance the running max only when it would grow by more than the threshold
      float scale = 1.0f;
      bool grow = false;
      if (j == 0) {
        m = m_tile;
      } else if (m_tile - m > kRescaleThreshold) {
        scale = ex2(m - m_tile);
        m = m_tile;
        l *= scale;
        grow = true;
      }
      if (__any_sync(0xffffffffu, grow)) {
        // O of the previous tiles is complete (the S we just read was issued after it): rescale it
#pragma unroll
        for (int c = 0; c < P::kOCols / 16; ++c) {
          uint32_t o[16];
          tmem_ld16(tmem_o + lane_off + c * 16, o);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 16; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * scale);
          tmem_st16(tmem_o + lane_off + c * 16, o);
        }
      }
      // pass 2: P = exp2(S - m) as bf16 pairs over the S columns already consumed
      for (int c = 0; c < n_chunks; ++c) {
        uint32_t s[32], pk[16];
        tmem_ld32(tmem_s + lane_off + c * 32, s);
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const int col = c * 32 + 2 * i;
          const float p0 = col < kv_valid ? ex2(__uint_as_float(s[2 * i]) - m) : 0.0f;
          const float p1 = col + 1 < kv_valid ? ex2(__uint_as_float(s[2 * i + 1]) - m) : 0.0f;
          l += p0 + p1;
          __nv_bfloat162 b = __floats2bfloat162_rn(p0, p1);
          pk[i] = *reinterpret_cast<uint32_t*>(&b);
        }
        tmem_st16(tmem_s + lane_off + c * 16, pk);
      }
      tmem_st_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(p_full);
    }
    // epilogue: O / l -> bf16 -> out[token, head*dh ..]
    if (ok && mbar_wait(o_done, (n_kv - 1) & 1, abort_flag)) {
      tc_fence_after();
      const float inv = 1.0f / l;
      const int token = q0 + r;
      __nv_bfloat16* orow = out + (int64_t)token * (heads * dh) + head * dh;
#pragma unroll
      for (int c = 0; c < P::kOCols / 16; ++c) {
        uint32_t o[16];
        tmem_ld16(tmem_o + lane_off + c * 16, o);
        tmem_ld_wait();
        if (token < seg_end) {
#pragma unroll
          for (int g = 0; g < 2; ++g) {
            if (c * 16 + g * 8 < dh) {  // dh is a multiple of 8
              uint4 pk;
              __nv_bfloat162 b0 = __floats2bfloat162_rn(__uint_as_float(o[8 * g]) * inv, __uint_as_float(o[8 * g + 1]) * inv);
              __nv_bfloat162 b1 = __floats2bfloat162_rn(__uint_as_float(o[8 * g + 2]) * inv, __uint_as_float(o[8 * g + 3]) * inv);
              __nv_bfloat162 b2 = __floats2bfloat162_rn(__uint_as_float(o[8 * g + 4]) * inv, __uint_as_float(o[8 * g + 5]) * inv);
              __nv_bfloat162 b3 = __floats2bfloat162_rn(__uint_as_float(o[8 * g + 6]) * inv, __uint_as_float(o[8 * g + 7]) * inv);
              pk.x = *reinterpret_cast<uint32_t*>(&b0);
              pk.y = *reinterpret_cast<uint32_t*>(&b1);
              pk.z = *reinterpret_cast<uint32_t*>(&b2);
              pk.w = *reinterpret_cast<uint32_t*>(&b3);
              *reinterpret_cast<uint4*>(orow + c * 16 + g * 8) = pk;
            }
          }
        }
      }
    }
  }

  // ---------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0 && status != nullptr) atomicCAS(status, 0, kStatusTimeout);
    for (int i = 0; i < 64; ++i) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 256);
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

// Map over a bf16 matrix [rows, dhp] (row pitch dhp*2 bytes): box = 128 rows x box_cols columns.
bool make_map(CUtensorMap* tm, const void* base, int64_t rows, int dhp, int box_cols, CUtensorMapSwizzle swz) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)dhp, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)dhp * 2};
  cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)BKV};
  cuuint32_t estr[2] = {1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int DHP>
cudaError_t launch(const Maps& maps, const int32_t* cu, int n_seg, int q_tiles, void* out, int T, int heads, int dh,
                   int* status, cudaStream_t s) {
  using P = Plan<DHP>;
  auto kern = attention_tc_kernel<DHP>;
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, P::kDynamic);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  dim3 grid((unsigned)q_tiles, (unsigned)heads);
  kern<<<grid, kThreads, P::kDynamic, s>>>(maps, cu, n_seg, (__nv_bfloat16*)out, T, heads, dh, status);
  return cudaGetLastError();
}

bool attention_tc_supported(const void* q, const void* k, const void* v, const void* out, int64_t T, int heads,
                            int head_dim) {
  const int dhp = padded_head_dim(head_dim);
  if (dhp != 64 && dhp != 80 && dhp != 128) return false;
  if (head_dim % 8) return false;
  if (((uintptr_t)q & 15) || ((uintptr_t)k & 15) || ((uintptr_t)v & 15) || ((uintptr_t)out & 15)) return false;
  if ((int64_t)heads * T > (1 << 30) || heads > 65535) return false;
  return encode_tiled_fn() != nullptr;
}

cudaError_t attention_tc(const void* q, const void* k, const void* v, const int32_t* cu_seqlens,
                         const int32_t* host_cu_seqlens, int n_seg, void* out, int64_t T, int heads, int head_dim,
                         int* status, cudaStream_t s) {
  const int dhp = padded_head_dim(head_dim);
  int q_tiles = 0;
  for (int i = 0; i < n_seg; ++i) q_tiles += (host_cu_seqlens[i + 1] - host_cu_seqlens[i] + BQ - 1) / BQ;
  if (q_tiles == 0) return cudaSuccess;
  const int64_t rows = (int64_t)heads * T;
  Maps maps;
  const void* ptr[3] = {q, k, v};
  CUtensorMap* mains[3] = {&maps.q_main, &maps.k_main, &maps.v_main};
  CUtensorMap* tails[3] = {&maps.q_tail, &maps.k_tail, &maps.v_tail};
  for (int i = 0; i < 3; ++i) {
    if (!make_map(mains[i], ptr[i], rows, dhp, 64, CU_TENSOR_MAP_SWIZZLE_128B)) return cudaErrorInvalidValue;
    if (!make_map(tails[i], ptr[i], rows, dhp, 16, CU_TENSOR_MAP_SWIZZLE_32B)) return cudaErrorInvalidValue;
  }
  switch (dhp) {
    case 64: return launch<64>(maps, cu_seqlens, n_seg, q_tiles, out, (int)T, heads, head_dim, status, s);
    case 80: return launch<80>(maps, cu_seqlens, n_seg, q_tiles, out, (int)T, heads, head_dim, status, s);
    case 128: return launch<128>(maps, cu_seqlens, n_seg, q_tiles, out, (int)T, heads, head_dim, status, s);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace

cudaError_t attention_any(int dtype, const void* q, const void* k, const void* v, const int32_t* cu_seqlens,
                          const int32_t* host_cu_seqlens, int n_seg, void* out, int64_t T, int heads, int head_dim,
                          int flags, int* status, cudaStream_t s) {
  if (dtype == EPD_DTYPE_BF16 && !(flags & EPD_ATTENTION_FORCE_FMA) &&
      attention_tc_supported(q, k, v, out, T, heads, head_dim))
    return attention_tc(q, k, v, cu_seqlens, host_cu_seqlens, n_seg, out, T, heads, head_dim, status, s);
  return attention_fma(dtype, q, k, v, cu_seqlens, n_seg, out, T, heads, head_dim, s);
}

}  // namespace epd
