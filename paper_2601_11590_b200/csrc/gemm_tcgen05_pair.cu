// bf16 linear layer on the 5th-generation tensor cores with CTA pairs:  out = act(x . w^T + bias) (+ out).
//
// Why pairs: with one CTA per tile the main loop is bound by shared-memory bandwidth, not by the
// tensor pipe.  Per 64-wide contraction block a 128 x 256 tile has TMA write 48 KB into shared
// memory and the MMAs read the same 48 KB back in the 512 clocks the MMAs need: 192 B/clk against
// the 128 B/clk an SM's shared memory moves (measured: ~63 % of the MMA rate, which alone reaches
// 8165 FLOP/clk/SM).  A pair of CTAs on neighbouring SMs (a cluster of 2) computes a 256 x 256 tile
// with tcgen05.mma.cta_group::2: each CTA stages its own 128 rows of x and only HALF of the w tile
// (128 of the 256 output columns); the hardware feeds both halves of w to both tensor cores.  That is
// 32 KB written + 32 KB read per SM per block = 128 B/clk.
//
// Roles per CTA (10 warps):
//   warp 0      TMA producer: loads its x tile and its half of the w tile into a STAGES-deep ring; the
//               bytes of both CTAs are counted on the LEADER's (cluster rank 0) "full" barrier
//   warp 1      allocates tensor memory (pair-wide allocation); in the leader one thread issues the MMAs
//               for both CTAs and commits to the "empty" / "accumulator full" barriers of both
//   warps 2..9  epilogue, two warps per TMEM lane quarter, each taking half of the tile's columns:
//               tcgen05.ld, bias / GELU, 32-row x 128-byte chunks staged in swizzled shared memory and
//               written with TMA (plain store, or reduce-add for the residual update)
// Each CTA holds the accumulator rows of its own 128 rows of x (two accumulators of 256 columns, so
// the epilogue of tile i overlaps the main loop of tile i+1).  Ragged M, N, K are handled by TMA
// (zero fill on loads, clipping on stores).  No load in this file is a multicast load.
//
// QKV variant (ROPE = true): the epilogue applies the 2-D rotary embedding to the q and k columns and
// writes q, k, v straight into the head-major padded buffers the attention kernel reads, so the
// [T, 3h] intermediate and a separate rotary pass disappear.  It expects the q and k rows of the weight
// (and bias) permuted inside each head so that the two members of a rotation pair are neighbours
// (qkv_pair_permutation below); q.k^T does not depend on the order of the head dimensions as long as q
// and k share it.
// Every mbarrier wait is bounded: on expiry the CTA records EPD_ETIMEOUT and drains; the two cluster
// barriers (start, end) are reached by both CTAs on every path.
#include "tcgen05_common.cuh"

namespace epd {
namespace {

using namespace tc;

constexpr int BM = 128;         // rows of x per CTA (256 per pair)
constexpr int BK = 64;          // 64 bf16 = 128 bytes = one swizzle row
constexpr int kEpiWarps = 8;
constexpr int kThreads = 32 * (2 + kEpiWarps);
constexpr int kMaxDynamicSmem = 232448;           // 227 KB: the most one CTA can have

__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// Address, in the cluster's shared-memory window, of the same variable in CTA `rank` of the pair.
__device__ __forceinline__ uint32_t map_to_rank(uint32_t smem_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Arrive on a barrier given by its cluster-window address (own CTA's or the peer's).  Relaxed: the
// arrival only says "my tcgen05.ld of this accumulator have completed" (tcgen05.wait::ld has returned),
// no memory written by this thread is handed over; a release here would also wait for the thread's
// output stores still in flight to L2 (measured ~2000 clocks per tile).
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// L2 eviction policies for the bulk copies: the operand a band of tiles keeps coming back to should stay in L2
// (evict last), what streams past once (the other operand, the output) should leave first.
__device__ __forceinline__ uint64_t policy_evict_last() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t policy_evict_normal() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(p));
  return p;
}
// Tensor load into this CTA's shared memory whose completion bytes are counted on a barrier that may
// live in the other CTA of the pair (given by its cluster-window address).
__device__ __forceinline__ void tma_load_2d_pair(void* smem_dst, const CUtensorMap* tm, int x, int y,
                                                 uint32_t bar_cluster_addr, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint "
      "[%0], [%1, {%3, %4}], [%2], %5;"
      ::"r"(smem_u32(smem_dst)), "l"(tm), "r"(bar_cluster_addr), "r"(x), "r"(y), "l"(policy)
      : "memory");
}
__device__ __forceinline__ void tma_store_2d_hint(const CUtensorMap* tm, int x, int y, const void* smem_src, uint64_t policy) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group.L2::cache_hint [%0, {%2, %3}], [%1], %4;"
               ::"l"(tm), "r"(smem_u32(smem_src)), "r"(x), "r"(y), "l"(policy) : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t* smem_result, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_result)),
               "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t addr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(addr), "r"(cols) : "memory");
}

// D[tmem, both CTAs] (+)= A[smem, 128 rows per CTA] . B[smem, half the columns per CTA]^T; issued by
// one thread of the leader CTA.  FP8: 8-bit floating-point operands (kind::f8f6f4, 32 elements per instruction)
// instead of 16-bit ones (kind::f16, 16 elements per instruction): 32 bytes of every row either way.
template <bool FP8>
__device__ __forceinline__ void umma_pair(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                          uint32_t accumulate) {
  if constexpr (FP8) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
        : "memory");
  } else {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
        : "memory");
  }
}
// Once all MMAs issued so far by this thread have completed, arrive on the barrier at this offset in
// both CTAs of the pair.
__device__ __forceinline__ void umma_commit_both(uint64_t* bar) {
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
      ::"r"(smem_u32(bar)), "h"((uint16_t)3)
      : "memory");
}

// Instruction descriptor: fp32 accumulation, both operands K-major, M = 256 over the pair, N = BN; operand format
// bf16 (code 1 of kind::f16) or E4M3 (code 0 of kind::f8f6f4).
__host__ __device__ constexpr uint32_t instr_desc_pair(int n, bool fp8) {
  return (1u << 4) | (fp8 ? 0u : ((1u << 7) | (1u << 10))) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
}

// Destination of the QKV variant's epilogue.
struct RopeSplitArgs {
  __nv_bfloat16* qkv[3];        // head-major [heads, T, dhp] each
  const int32_t* pos_row;       // [T]
  const int32_t* pos_col;       // [T]
  const float2* table;          // [table_rows, dh/4] (cos, sin) of position * frequency
  int table_in_smem;            // entries (float2) copied into shared memory behind the kernel's own layout; 0 = read from global
  int heads, dh, dhp;
  float q_scale;
  int stream_out;               // q, k, v together exceed the L2: write them with streaming stores
};

// Order in which the pairs walk the grid of output tiles.  The pairs resident at one time work on consecutive
// tiles, so the order decides what they share in L2: with `by_rows`, the tile grid is cut into bands of `group` tile
// rows, and inside a band the tiles are taken column by column (the band's rows of x stay in L2 while the whole of w
// streams past once per band); otherwise into bands of `group` tile columns taken row by row (the band's rows of w
// stay, x streams past once per band).  Row-major or column-major over the whole grid are the bands of full width.
struct TileOrder {
  int by_rows;
  int group;
  int stream_normal;   // the streamed operand is loaded with the ordinary L2 priority instead of evict-first
};
// Policy for the operand that streams past a band.  Its tiles are still shared by the pairs that work on the band's
// tiles at the same time: beside a small band (up to 24 MB) it does better with the ordinary priority (measured:
// 16384 x 3200 x 3200 1351 -> 1434 TFLOP/s, 22656 x 4304 x 1152 1375 -> 1497), beside a band that fills the L2's
// share (the 41 MB bands of the 6B-class fc1 and fc2) with evict-first (1607 against 1577).
__device__ __forceinline__ uint64_t policy_stream(const TileOrder& o) {
  return o.stream_normal ? policy_evict_normal() : policy_evict_first();
}
__device__ __forceinline__ void tile_coords(int tile, int m_tiles, int n_tiles, const TileOrder& o, int& mt, int& nt) {
  if (o.by_rows) {
    const int per = o.group * n_tiles, band = tile / per, r = tile - band * per;
    const int first = band * o.group, rows = min(o.group, m_tiles - first);
    nt = r / rows;
    mt = first + (r - nt * rows);
  } else {
    const int per = o.group * m_tiles, band = tile / per, r = tile - band * per;
    const int first = band * o.group, cols = min(o.group, n_tiles - first);
    mt = r / cols;
    nt = first + (r - mt * cols);
  }
}

template <int BN, int STAGES>
struct PairLayout {
  static constexpr int kABytes = BM * BK * 2;
  static constexpr int kBBytes = (BN / 2) * BK * 2;     // this CTA's half of the w tile
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kOutBufBytes = 32 * 128;         // one staging buffer per epilogue warp
  static constexpr int kOutOffset = STAGES * kStageBytes;
  static constexpr int kBarOffset = kOutOffset + kEpiWarps * kOutBufBytes;
  // full[STAGES], empty[STAGES], tmem_full[2], tmem_empty[2], drain, (spare), tmem base, abort flag,
  // bias[kEpiWarps][BN/2]
  static constexpr int kBiasOffset = kBarOffset + (2 * STAGES + 6) * 8 + 16;
  static constexpr int kScaleOffset = kBiasOffset + kEpiWarps * (BN / 2) * 4;   // column scales of the 8-bit variant
  static constexpr int kTotal = kScaleOffset + kEpiWarps * (BN / 2) * 4;
  static constexpr int kDynamic = kTotal + 1024;
  static_assert(kDynamic <= 232448, "exceeds the shared memory of one CTA");
  static_assert(kDynamic > 116 * 1024, "one CTA per SM is assumed by the TMEM allocation");
};

// ---------------------------------------------------------------------------------------------
// Kernel
// ---------------------------------------------------------------------------------------------
template <int BN, int STAGES, typename OutT, int ACT, bool ACCUM, bool ROPE, bool FP8>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
linear_pair_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_w,
                   const __grid_constant__ CUtensorMap tm_out, const __nv_bfloat16* __restrict__ bias, int M, int N,
                   int K, int* __restrict__ status, long long wait_limit, int static_w, const TileOrder order,
                   const RopeSplitArgs rs, const float* __restrict__ row_scale, const float* __restrict__ col_scale) {
  static_assert(!ROPE || (sizeof(OutT) == 2 && ACT == 0 && !ACCUM), "the QKV variant writes bf16, no activation");
  static_assert(!(ROPE && FP8), "the QKV variant takes bf16 operands");
  // elements per contraction block (128 bytes of a row) and per MMA (32 bytes)
  constexpr int BKE = FP8 ? 2 * BK : BK;
  using L = PairLayout<BN, STAGES>;
  static_assert(BN == 256 || BN == 128, "tile width");
  constexpr int kAccStride = BN;                 // TMEM columns between the two accumulators
  constexpr int kTmemCols = 2 * kAccStride;

  pdl_launch_dependents();
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + L::kBarOffset);   // used in the leader only
  uint64_t* empty = full + STAGES;                                      // one set per CTA
  uint64_t* tmem_full = empty + STAGES;                                 // one set per CTA
  uint64_t* tmem_empty = tmem_full + 2;                                 // used in the leader only
  uint64_t* drain_bar = tmem_empty + 2;     // one per CTA; after an abort: the pair's MMAs have completed
  uint32_t* tmem_base_slot = reinterpret_cast<uint32_t*>(drain_bar + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_base_slot + 1);
  uint32_t loads_issued = 0;                // stage loads issued by this CTA's producer thread
  float* bias_s = reinterpret_cast<float*>(smem + L::kBiasOffset);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_rank();          // 0 = leader
  // a wait that expires raises the abort flag of both CTAs of the pair
  const WaitCtx wc{abort_flag, map_to_rank(smem_u32(const_cast<int*>(abort_flag)), rank ^ 1u), wait_limit};
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int m_tiles = (M + 2 * BM - 1) / (2 * BM), n_tiles = (N + BN - 1) / BN;
  const int num_tiles = m_tiles * n_tiles;
  const int k_blocks = (K + BKE - 1) / BKE;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&tmem_full[a], 1); mbar_init(&tmem_empty[a], 2 * kEpiWarps); }
    mbar_init(drain_bar, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc_pair(tmem_base_slot, kTmemCols);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync();                                 // both CTAs' barriers exist before either signals the other
  tc_fence_after();
  const uint32_t tmem_base = *tmem_base_slot;
  // The weight tiles of the first stages do not depend on the previous kernel (static_w): the producer fetches
  // them before the wait below, so they arrive while the previous kernel is still finishing; the x tiles follow
  // after the wait, into the same stages, counted on the same barrier phase.
  int early = 0;
  if (static_w && warp == 0 && pair < num_tiles) {
    int mt, nt;
    tile_coords(pair, m_tiles, n_tiles, order, mt, nt);
    const int n0 = nt * BN + (int)rank * (BN / 2);
    const uint64_t pol_w = order.by_rows ? policy_stream(order) : policy_evict_last();
    early = k_blocks < STAGES ? k_blocks : STAGES;
    if (elect_one()) {
      prefetch_map(&tm_w);
      for (int kb = 0; kb < early; ++kb) {
        if (rank == 0) mbar_expect_tx(&full[kb], 2 * L::kStageBytes);
        tma_load_2d_pair(smem + kb * L::kStageBytes + L::kABytes, &tm_w, kb * BKE, n0,
                         map_to_rank(smem_u32(&full[kb]), 0), pol_w);
      }
    }
    __syncwarp();
    loads_issued = early;     // for the drain after an abort: these stages have loads in flight
  }
  pdl_wait();   // nothing above touches global memory that an earlier kernel of the stream writes

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (both CTAs)
    // The whole warp walks the loop and one elected lane issues (see elect_one()).
    {
      if (lane == 0) {
        prefetch_map(&tm_x);
        prefetch_map(&tm_w);
      }
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      loads_issued = 0;
      // the operand of the band stays in L2, the other one streams past
      const uint64_t pol_x = order.by_rows ? policy_evict_last() : policy_stream(order);
      const uint64_t pol_w = order.by_rows ? policy_stream(order) : policy_evict_last();
      for (int tile = pair; tile < num_tiles && ok; tile += n_pairs) {
        int mt, nt;
        tile_coords(tile, m_tiles, n_tiles, order, mt, nt);
        const int m0 = mt * (2 * BM) + (int)rank * BM;        // this CTA's rows of x
        const int n0 = nt * BN + (int)rank * (BN / 2);       // this CTA's half of the w tile
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!mbar_wait_warp<true>(&empty[stage], phase ^ 1, wc)) { ok = false; break; }
          uint8_t* sa = smem + stage * L::kStageBytes;
          const uint32_t bar = map_to_rank(smem_u32(&full[stage]), 0);
          const bool w_early = early > 0;             // this stage's bytes are expected and its w tile is on its way
          if (w_early) --early;
          if (elect_one()) {
            if (!w_early) {
              // the leader's barrier counts the bytes of both CTAs
              if (rank == 0) mbar_expect_tx(&full[stage], 2 * L::kStageBytes);
              tma_load_2d_pair(sa + L::kABytes, &tm_w, kb * BKE, n0, bar, pol_w);
            }
            tma_load_2d_pair(sa, &tm_x, kb * BKE, m0, bar, pol_x);
          }
          __syncwarp();
          ++loads_issued;
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (leader only)
    // The whole warp walks the loop and one elected lane issues (see elect_one()).
    if (rank == 0) {
      constexpr uint32_t idesc = instr_desc_pair(BN, FP8);
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int tile = pair; tile < num_tiles && ok; tile += n_pairs) {
        if (!mbar_wait_warp<true>(&tmem_empty[acc], acc_phase ^ 1, wc)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * kAccStride;
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!mbar_wait_warp<true>(&full[stage], phase, wc)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = smem_u32(smem + stage * L::kStageBytes);
          const uint64_t da = smem_desc_k_sw128(sa), db = smem_desc_k_sw128(sa + L::kABytes);
          if (elect_one()) {
#pragma unroll
            for (int k = 0; k < BK / 16; ++k)   // one MMA per 32 bytes along K inside the swizzled row = 2 descriptor units
              umma_pair<FP8>(d_tmem, da + 2 * k, db + 2 * k, idesc, (kb | k) != 0);
            umma_commit_both(&empty[stage]);
          }
          __syncwarp();
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
        if (!ok) break;
        if (elect_one()) umma_commit_both(&tmem_full[acc]);
        __syncwarp();
        if (++acc == 2) { acc = 0; acc_phase ^= 1; }
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------------ epilogue (both CTAs)
    constexpr int CC = sizeof(OutT) == 4 ? 32 : 64;  // columns per staged chunk: 128 bytes per row
    constexpr int kChunks = (BN / 2) / CC;           // chunks per warp: a warp owns half of the tile's columns
    const int q = warp & 3;                          // TMEM lane quarter this warp may read
    const int half = (warp - 2) >> 2;                // which half of the columns
    float* bs = bias_s + (warp - 2) * (BN / 2);
    float* cs = reinterpret_cast<float*>(smem + L::kScaleOffset) + (warp - 2) * (BN / 2);
    uint8_t* sbuf = smem + L::kOutOffset + (warp - 2) * L::kOutBufBytes;
    const uint32_t tmem_empty_leader0 = map_to_rank(smem_u32(&tmem_empty[0]), 0);
    int acc = 0;
    uint32_t acc_phase = 0;
    if (!ROPE && lane == 0) prefetch_map(&tm_out);
    const uint64_t pol_out = policy_evict_first();   // the output is not read again by this kernel
    const float2* rope_tab = rs.table;
    if constexpr (ROPE) {
      if (rs.table_in_smem > 0) {
        // the (cos, sin) table is small: keep it in shared memory (every epilogue warp reaches this
        // barrier before any wait that can give up)
        float4* dst = reinterpret_cast<float4*>(smem + L::kTotal);
        const float4* srcv = reinterpret_cast<const float4*>(rs.table);
        for (int i = threadIdx.x - 64; i < rs.table_in_smem / 2; i += 32 * kEpiWarps) dst[i] = srcv[i];
        asm volatile("bar.sync 1, %0;" ::"n"(32 * kEpiWarps) : "memory");
        rope_tab = reinterpret_cast<const float2*>(dst);
      }
    }
    for (int tile = pair; tile < num_tiles; tile += n_pairs) {
      int mt, nt;
      tile_coords(tile, m_tiles, n_tiles, order, mt, nt);
      const int m0 = mt * (2 * BM) + (int)rank * BM;
      const int n0 = nt * BN + half * (BN / 2);
      __syncwarp();
      for (int i = lane; i < BN / 2; i += 32) {
        bs[i] = (bias != nullptr && n0 + i < N) ? __bfloat162float(bias[n0 + i]) : 0.0f;
        if constexpr (FP8) cs[i] = n0 + i < N ? col_scale[n0 + i] : 0.0f;
      }
      __syncwarp();
      if (!mbar_wait_warp<true>(&tmem_full[acc], acc_phase, wc)) break;
      tc_fence_after();
      const int row0 = m0 + q * 32;
      float rscale = 1.0f;                              // 8-bit variant: this thread's row scale
      if constexpr (FP8) rscale = row0 + lane < M ? row_scale[row0 + lane] : 0.0f;
      const uint32_t taddr = tmem_base + acc * kAccStride + half * (BN / 2) + ((uint32_t)(q * 32) << 16);
      // QKV variant: this thread's row positions, and (tensor, head, dim) of its first column
      int prow = 0, pcol = 0, rt = 0, rhead = 0, rd = 0;
      if constexpr (ROPE) {
        if (row0 + lane < M) { prow = rs.pos_row[row0 + lane]; pcol = rs.pos_col[row0 + lane]; }
        const int hdim = rs.heads * rs.dh;
        rt = n0 / hdim;
        const int within = n0 - rt * hdim;
        rhead = within / rs.dh;
        rd = within - rhead * rs.dh;
      }
#pragma unroll 1
      for (int c = 0; c < kChunks; ++c) {
        uint32_t pk[32];  // this thread's row of the chunk, as stored: 32 floats or 64 bf16
        if constexpr (sizeof(OutT) == 4) {
          tmem_ld32(taddr + c * CC, pk);
          tmem_ld_wait();
          const float4* bs4 = reinterpret_cast<const float4*>(bs + c * CC);   // broadcast reads, 16 bytes each
#pragma unroll
          for (int j4 = 0; j4 < 8; ++j4) {
            const float4 bv = bs4[j4];
            const float bb[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              float t = __uint_as_float(pk[4 * j4 + e]);
              if constexpr (FP8) t *= rscale * cs[c * CC + 4 * j4 + e];
              t += bb[e];
              if (ACT == 1) t = gelu_tanh_fast(t);
              if (ACT == 2) t = gelu_erf_fast(t);
              pk[4 * j4 + e] = __float_as_uint(t);
            }
          }
        } else {
          uint32_t r0[32], r1[32];
          tmem_ld32(taddr + c * CC, r0);
          tmem_ld32(taddr + c * CC + 32, r1);
          tmem_ld_wait();
          if constexpr (ROPE) {
            // groups of 8 columns = 4 rotation pairs, never across a head; two pairs share one
            // 16-byte table read (pairs 2u, 2u+1 of a half use neighbouring frequencies)
            const int nf = rs.dh >> 2;
#pragma unroll
            for (int g = 0; g < 8; ++g) {
              const uint32_t* src = g < 4 ? r0 : r1;
              const int jj = (8 * g) & 31;
              const float4 ba = *reinterpret_cast<const float4*>(bs + c * CC + 8 * g);
              const float4 bb = *reinterpret_cast<const float4*>(bs + c * CC + 8 * g + 4);
              const float bias8[8] = {ba.x, ba.y, ba.z, ba.w, bb.x, bb.y, bb.z, bb.w};
              float v[8];
#pragma unroll
              for (int e = 0; e < 8; ++e) v[e] = __uint_as_float(src[jj + e]) + bias8[e];
              if (rt < 2) {
                const float sc = rt == 0 ? rs.q_scale : 1.0f;
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                  const int p2 = (rd >> 1) + 2 * u;                       // first pair of the unit inside the head
                  const int hf = p2 >= nf ? 1 : 0;
                  const int f = p2 - hf * nf;
                  const float4 cs = *reinterpret_cast<const float4*>(rope_tab + (hf ? pcol : prow) * nf + f);
                  const float a0 = v[4 * u], b0 = v[4 * u + 1], a1 = v[4 * u + 2], b1 = v[4 * u + 3];
                  v[4 * u] = (a0 * cs.x - b0 * cs.y) * sc;
                  v[4 * u + 1] = (b0 * cs.x + a0 * cs.y) * sc;
                  v[4 * u + 2] = (a1 * cs.z - b1 * cs.w) * sc;
                  v[4 * u + 3] = (b1 * cs.z + a1 * cs.w) * sc;
                }
              }
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                __nv_bfloat162 b = __floats2bfloat162_rn(v[2 * e], v[2 * e + 1]);
                pk[4 * g + e] = *reinterpret_cast<uint32_t*>(&b);
              }
              rd += 8;
              if (rd == rs.dh) { rd = 0; if (++rhead == rs.heads) { rhead = 0; ++rt; } }
            }
          } else {
            const float4* bs4 = reinterpret_cast<const float4*>(bs + c * CC);   // broadcast reads, 16 bytes each
#pragma unroll
            for (int j2 = 0; j2 < 16; ++j2) {
              const uint32_t* src = j2 < 8 ? r0 : r1;
              const int jj = (4 * j2) & 31;
              const float4 bv = bs4[j2];
              float t0 = __uint_as_float(src[jj]), t1 = __uint_as_float(src[jj + 1]);
              float t2 = __uint_as_float(src[jj + 2]), t3 = __uint_as_float(src[jj + 3]);
              if constexpr (FP8) {
                const float4 sv = *reinterpret_cast<const float4*>(cs + c * CC + 4 * j2);
                t0 *= rscale * sv.x; t1 *= rscale * sv.y; t2 *= rscale * sv.z; t3 *= rscale * sv.w;
              }
              t0 += bv.x; t1 += bv.y; t2 += bv.z; t3 += bv.w;
              if (ACT == 1) { t0 = gelu_tanh_fast(t0); t1 = gelu_tanh_fast(t1); t2 = gelu_tanh_fast(t2); t3 = gelu_tanh_fast(t3); }
              if (ACT == 2) { t0 = gelu_erf_fast(t0); t1 = gelu_erf_fast(t1); t2 = gelu_erf_fast(t2); t3 = gelu_erf_fast(t3); }
              __nv_bfloat162 b0 = __floats2bfloat162_rn(t0, t1), b1 = __floats2bfloat162_rn(t2, t3);
              pk[2 * j2] = *reinterpret_cast<uint32_t*>(&b0);
              pk[2 * j2 + 1] = *reinterpret_cast<uint32_t*>(&b1);
            }
          }
        }
        if (c == kChunks - 1) {
          // this warp has read all of its accumulator columns: tell the leader's MMA thread
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(tmem_empty_leader0 + acc * 8);
        }
        // the staging buffer is free once the bulk store issued from it has read it
        if (!ROPE && lane == 0) bulk_wait_read<0>();
        __syncwarp();
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          // 128-byte swizzle: 16-byte chunk j of row r lives at chunk position j ^ (r % 8)
          uint4* dst = reinterpret_cast<uint4*>(sbuf + lane * 128 + ((j ^ (lane & 7)) << 4));
          *dst = make_uint4(pk[4 * j], pk[4 * j + 1], pk[4 * j + 2], pk[4 * j + 3]);
        }
        if constexpr (ROPE) {
          // copy out with 8 lanes per row: 128 contiguous bytes of a head-major row per lane group
          __syncwarp();
          const int piece = lane & 7;
          const int col = n0 + c * CC + 8 * piece;
          const int hdim = rs.heads * rs.dh;
          const int t = col / hdim;
          const int within = col - t * hdim;
          const int head = within / rs.dh;
          const int d = within - head * rs.dh;
          if (col < N) {
            __nv_bfloat16* base = (t == 0 ? rs.qkv[0] : t == 1 ? rs.qkv[1] : rs.qkv[2]) + (int64_t)head * M * rs.dhp + d;
#pragma unroll
            for (int it = 0; it < 8; ++it) {
              const int r = it * 4 + (lane >> 3);
              if (row0 + r < M) {
                uint4* dst = reinterpret_cast<uint4*>(base + (int64_t)(row0 + r) * rs.dhp);
                const uint4 val = *reinterpret_cast<const uint4*>(sbuf + r * 128 + ((piece ^ (r & 7)) << 4));
                // Large outputs are streamed, so that they do not push the band of x out of L2 (16384 tokens x 25
                // heads x 128: 588 -> 327 MB read per launch); small ones stay in L2 for the attention kernel.
                if (rs.stream_out) __stcs(dst, val); else *dst = val;
              }
            }
          }
          continue;
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) {
          if (row0 < M && n0 + c * CC < N) {
            if (ACCUM) tma_reduce_add_2d(&tm_out, n0 + c * CC, row0, sbuf);
            else tma_store_2d_hint(&tm_out, n0 + c * CC, row0, sbuf, pol_out);
          }
          bulk_commit();
        }
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
    // A wait expired (here or in the other CTA of the pair).  Every role of this CTA has left its loop, so
    // nothing new is issued.  What was issued completes by itself: the leader's producer waits for the last
    // load of every stage (its barriers count the bytes of both CTAs), the leader's issuing thread commits
    // to the drain barrier of both CTAs (a commit arrives only after all earlier MMAs) and each CTA waits for
    // it, the epilogue warps have waited for their stores; a fixed pause on top, then the cluster barrier, after
    // which shared and tensor memory are released.
    if (threadIdx.x == 0 && status != nullptr) atomicCAS(status, 0, kStatusTimeout);
    if (warp == 0 && lane == 0 && rank == 0) drain_ring<true>(full, STAGES, loads_issued);
    if (warp == 1) {
      // the lane that issued the products commits (a commit covers the products of its own thread)
      if (elect_one()) {
        if (rank == 0) umma_commit_both(drain_bar);
        mbar_wait_drain<true>(drain_bar, 0);
      }
      __syncwarp();
    }
    for (int i = 0; i < 64; ++i) __nanosleep(1000);
    __syncthreads();
  }
  cluster_sync();   // neither CTA's shared memory or tensor memory goes away while the other may still touch it
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, kTmemCols);
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

// Tile order with the least modelled DRAM traffic.  The operand of a band (its rows of x, or its rows of w) is
// read once per band and kept in L2 (evict-last loads) while the other operand streams past (evict-first); a band
// may hold up to kL2Resident bytes.  Measured on the 6B-class fc1 shape (16384 x 12800 x 3200; operands 187 MB):
// with the whole grid taken column by column x was read from DRAM again for every tile column, 3.2 GB per launch
// at 1193 TFLOP/s; bands of 72 / 40 / 24 / 12 MB with the eviction hints: 1.8 / 0.48 / 1.1 / 1.9 GB, 1329 / 1453 /
// 1431 / 1401 TFLOP/s.  (The 126 MB L2 is two halves; 40 MB is what a band can count on.)
constexpr double kL2Resident = 40.0 * 1024 * 1024;
TileOrder choose_order(int M, int N, int K, int elem_bytes) {
  const int m_tiles = (M + 2 * BM - 1) / (2 * BM), n_tiles = (N + 255) / 256;
  const double tile_bytes = 256.0 * K * elem_bytes, x_bytes = (double)M * K * elem_bytes, w_bytes = (double)N * K * elem_bytes;
  const int cap = (int)(1.1 * kL2Resident / tile_bytes) > 1 ? (int)(1.1 * kL2Resident / tile_bytes) : 1;
  // bands of equal height: as few as the cap allows
  const int m_bands = (m_tiles + cap - 1) / cap, n_bands = (n_tiles + cap - 1) / cap;
  const double by_rows = x_bytes + w_bytes * m_bands;     // x once, w once per band of tile rows
  const double by_cols = w_bytes + x_bytes * n_bands;     // w once, x once per band of tile columns
  const int rows = (m_tiles + m_bands - 1) / m_bands, cols = (n_tiles + n_bands - 1) / n_bands;
  const double kSmallBand = 24.0 * 1024 * 1024;
  return by_rows <= by_cols ? TileOrder{1, rows, rows * tile_bytes <= kSmallBand ? 1 : 0}
                            : TileOrder{0, cols, cols * tile_bytes <= kSmallBand ? 1 : 0};
}

template <int BN, int STAGES, typename OutT, int ACT, bool ACCUM, bool ROPE = false, bool FP8 = false>
cudaError_t launch(const CUtensorMap& tx, const CUtensorMap& tw, const CUtensorMap& to, const void* bias, int M, int N,
                   int K, int* status, cudaStream_t s, int static_w, const RopeSplitArgs& rs = RopeSplitArgs{},
                   const float* row_scale = nullptr, const float* col_scale = nullptr) {
  using L = PairLayout<BN, STAGES>;
  auto kern = linear_pair_kernel<BN, STAGES, OutT, ACT, ACCUM, ROPE, FP8>;
  static PerDeviceOnce configured;
  cudaError_t e = once_per_device(configured, [&] {
    return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, ROPE ? kMaxDynamicSmem : L::kDynamic);
  });
  if (e != cudaSuccess) return e;
  const size_t smem_bytes = L::kDynamic + (ROPE ? (size_t)rs.table_in_smem * sizeof(float2) : 0);
  const int tiles = ((M + 2 * BM - 1) / (2 * BM)) * ((N + BN - 1) / BN);
  // pairs that can be resident at once on this device (SMs pair up inside a GPC, so this can be below SMs / 2)
  static PerDeviceInt resident;
  int dev = 0;
  cudaGetDevice(&dev);
  const int slot = dev >= 0 && dev < 64 ? dev : 0;
  int max_pairs = resident.v[slot].load(std::memory_order_relaxed);
  if (max_pairs == 0 || slot != dev) {
    const int sms = device_sm_count();
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(sms / 2 * 2);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = L::kDynamic;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2;
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess || n <= 0) {
      (void)cudaGetLastError();
      n = sms / 2;
    }
    max_pairs = n < sms / 2 ? n : sms / 2;
    if (slot == dev) resident.v[slot].store(max_pairs, std::memory_order_relaxed);
  }
  const int avail = limited_sms(2 * max_pairs) / 2 > 0 ? limited_sms(2 * max_pairs) / 2 : 1;   // pairs within the SM budget
  const int pairs = tiles < avail ? tiles : avail;
  return launch_pdl(kern, dim3(2 * pairs), dim3(kThreads), smem_bytes, s, tx, tw, to, (const __nv_bfloat16*)bias, M, N, K,
                    status, wait_limit_cycles(), static_w, choose_order(M, N, K, FP8 ? 1 : 2), rs, row_scale, col_scale);
}

template <int BN, int STAGES>
cudaError_t launch_bn(const CUtensorMap& tx, const CUtensorMap& tw, const CUtensorMap& to, const void* bias, int M,
                      int N, int K, int flags, int* status, cudaStream_t s) {
  const int act = (flags & EPD_LINEAR_GELU_TANH) ? 1 : (flags & EPD_LINEAR_GELU_ERF) ? 2 : 0;
  const bool accum = flags & EPD_LINEAR_ACCUMULATE;
  const bool out_f32 = accum || (flags & EPD_LINEAR_OUT_F32);
#define EPD_TC(OUT, A, C) \
  return launch<BN, STAGES, OUT, A, C>(tx, tw, to, bias, M, N, K, status, s, (flags & kLinearStaticWeights) ? 1 : 0)
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

}  // namespace

// Launches linear_tc_pair() makes for a shape (see there).
int linear_tc_pair_slices(int64_t N, int64_t K, int flags) {
  int slices = 1;
  if ((flags & EPD_LINEAR_ACCUMULATE) && !(flags & (EPD_LINEAR_GELU_TANH | EPD_LINEAR_GELU_ERF))) {
    const double w_bytes = (double)N * K * 2;
    while (slices < 4 && w_bytes / slices > 1.1 * kL2Resident) ++slices;
  }
  return slices;
}

// 256 x 256 tiles on CTA pairs.  Same argument contract as linear_tc().
// A residual update (out += ...) whose weight matrix is too large for any band of it to stay in L2 (the 6B-class
// fc2: 82 MB, 6.5 MB per tile row) is run as consecutive launches over slices of the contraction dimension, each
// adding its part to `out`: a slice's share of w then fits (41 MB), x is read once per slice instead of once per
// tile column.  The split depends on N and K only, so a row's result does not depend on the batch it is in.
cudaError_t linear_tc_pair(const void* x, int64_t ldx, const void* w, int64_t ldw, const void* bias, void* out,
                           int64_t ldo, int64_t M, int64_t N, int64_t K, int flags, int* status, cudaStream_t s) {
  const bool out_f32 = flags & (EPD_LINEAR_ACCUMULATE | EPD_LINEAR_OUT_F32);
  constexpr int BN = 256;
  const int slices = linear_tc_pair_slices(N, K, flags);
  const int64_t k_slice = slices > 1 ? ((K + slices - 1) / slices + BK - 1) / BK * BK : K;
  for (int64_t k0 = 0; k0 < K; k0 += k_slice) {
    const int64_t kc = K - k0 < k_slice ? K - k0 : k_slice;
    const char* xs = static_cast<const char*>(x) + k0 * 2;
    const char* wsl = static_cast<const char*>(w) + k0 * 2;
    CUtensorMap tx, tw, to;
    if (!make_map(&tx, xs, M, kc, ldx, BM, 2) || !make_map(&tw, wsl, N, kc, ldw, BN / 2, 2) ||
        !make_map(&to, out, M, N, ldo, 32, out_f32 ? 4 : 2))
      return cudaErrorInvalidValue;
    cudaError_t e = launch_bn<BN, 5>(tx, tw, to, k0 == 0 ? bias : nullptr, (int)M, (int)N, (int)kc, flags, status, s);
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

// The same layer with 8-bit floating-point operands (E4M3): xq [M, K] and wq [N, K] hold byte codes, row_scale [M] and
// col_scale [N] the factors they were divided by; out = act((xq . wq^T) * row_scale * col_scale^T + bias), bf16 or
// (EPD_LINEAR_OUT_F32) float.  K a multiple of 16 bytes, leading dimensions too.
cudaError_t linear_tc_pair_e4m3(const void* xq, int64_t ldx, const float* row_scale, const void* wq, int64_t ldw,
                                const float* col_scale, const void* bias, void* out, int64_t ldo, int64_t M, int64_t N,
                                int64_t K, int flags, int* status, cudaStream_t s) {
  constexpr int BN = 256;
  const bool out_f32 = flags & EPD_LINEAR_OUT_F32;
  const int act = (flags & EPD_LINEAR_GELU_TANH) ? 1 : (flags & EPD_LINEAR_GELU_ERF) ? 2 : 0;
  CUtensorMap tx, tw, to;
  if (!make_map(&tx, xq, M, K, ldx, BM, 1) || !make_map(&tw, wq, N, K, ldw, BN / 2, 1) ||
      !make_map(&to, out, M, N, ldo, 32, out_f32 ? 4 : 2))
    return cudaErrorInvalidValue;
#define EPD_F8(OUT, A) \
  return launch<BN, 5, OUT, A, false, false, true>(tx, tw, to, bias, (int)M, (int)N, (int)K, status, s, 0, RopeSplitArgs{}, \
                                                   row_scale, col_scale)
  if (out_f32) {
    if (act == 0) EPD_F8(float, 0);
    if (act == 1) EPD_F8(float, 1);
    EPD_F8(float, 2);
  }
  if (act == 0) EPD_F8(__nv_bfloat16, 0);
  if (act == 1) EPD_F8(__nv_bfloat16, 1);
  EPD_F8(__nv_bfloat16, 2);
#undef EPD_F8
}

// QKV projection with the rotary embedding and the head split in its epilogue.  w and bias hold the q
// and k rows in pair order (qkv_pair_permutation); q, k, v are head-major [heads, M, padded head_dim]
// whose padding columns the caller has initialised (they are not written here).
cudaError_t linear_tc_pair_qkv(const void* x, int64_t ldx, const void* w_perm, int64_t ldw, const void* bias_perm,
                               void* q, void* k, void* v, const int32_t* pos_row, const int32_t* pos_col,
                               const float2* table, int table_rows, int64_t M, int heads, int head_dim, float q_scale,
                               int static_w, int* status, cudaStream_t s) {
  constexpr int BN = 256;
  const int64_t hdim = (int64_t)heads * head_dim, N = 3 * hdim, K = hdim;
  if (head_dim % 8 || !table) return cudaErrorInvalidValue;
  CUtensorMap tx, tw;
  if (!make_map(&tx, x, M, K, ldx, BM, 2) || !make_map(&tw, w_perm, N, K, ldw, BN / 2, 2)) return cudaErrorInvalidValue;
  RopeSplitArgs rs;
  rs.qkv[0] = static_cast<__nv_bfloat16*>(q);
  rs.qkv[1] = static_cast<__nv_bfloat16*>(k);
  rs.qkv[2] = static_cast<__nv_bfloat16*>(v);
  rs.pos_row = pos_row;
  rs.pos_col = pos_col;
  rs.table = table;
  const int64_t entries = (int64_t)table_rows * (head_dim / 4);
  rs.table_in_smem =
      (entries % 2 == 0 && entries * (int64_t)sizeof(float2) <= kMaxDynamicSmem - PairLayout<BN, 5>::kDynamic) ? (int)entries : 0;
  rs.heads = heads;
  rs.dh = head_dim;
  rs.dhp = padded_head_dim(head_dim);
  rs.q_scale = q_scale;
  rs.stream_out = 3.0 * (double)heads * (double)M * rs.dhp * 2.0 > 96.0 * 1024 * 1024 ? 1 : 0;
  // the output tensor map is not used by this variant
  return launch<BN, 5, __nv_bfloat16, 0, false, true>(tx, tw, tx, bias_perm, (int)M, (int)N, (int)K, status, s, static_w, rs);
}

namespace {

// Row n of the permuted QKV weight is row qkv_source_row(n) of the original: inside each head of q and
// k, position 2p holds the first member of rotation pair p and 2p + 1 its partner (pairs counted over
// the row half, then the column half); v rows stay.
__global__ void qkv_permute_kernel(const __nv_bfloat16* __restrict__ w, const __nv_bfloat16* __restrict__ b,
                                   __nv_bfloat16* __restrict__ w_out, __nv_bfloat16* __restrict__ b_out, int heads,
                                   int dh, int64_t ldw) {
  const int hdim = heads * dh, n = blockIdx.x;
  int src = n;
  if (n < 2 * hdim) {
    const int j = n % dh, p = j >> 1, nf = dh >> 2;
    const int hf = p / nf, f = p - hf * nf;
    src = n - j + hf * (dh >> 1) + f + (j & 1) * nf;
  }
  const uint4* in = reinterpret_cast<const uint4*>(w + (int64_t)src * ldw);
  uint4* out = reinterpret_cast<uint4*>(w_out + (int64_t)n * hdim);
  for (int i = threadIdx.x; i < hdim / 8; i += blockDim.x) out[i] = in[i];
  if (threadIdx.x == 0) b_out[n] = b ? b[src] : __float2bfloat16(0.0f);
}

// Padding columns of the head-major buffers: zeros, and 1 in v's first padding column.
__global__ void qkv_pad_init_kernel(__nv_bfloat16* __restrict__ q, __nv_bfloat16* __restrict__ k,
                                    __nv_bfloat16* __restrict__ v, int64_t rows, int dh, int dhp) {
  const int pad = dhp - dh;
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= rows * pad) return;
  const int64_t r = i / pad;
  const int c = (int)(i - r * pad);
  const int64_t at = r * dhp + dh + c;
  q[at] = __float2bfloat16(0.0f);
  k[at] = __float2bfloat16(0.0f);
  v[at] = __float2bfloat16(c == 0 ? 1.0f : 0.0f);
}

}  // namespace

cudaError_t qkv_permute(const void* w, int64_t ldw, const void* bias, void* w_out, void* bias_out, int heads,
                        int head_dim, cudaStream_t s) {
  const int hdim = heads * head_dim;
  if (head_dim % 8 || (ldw % 8) || ((uintptr_t)w & 15) || ((uintptr_t)w_out & 15)) return cudaErrorInvalidValue;
  qkv_permute_kernel<<<3 * hdim, 128, 0, s>>>((const __nv_bfloat16*)w, (const __nv_bfloat16*)bias, (__nv_bfloat16*)w_out,
                                             (__nv_bfloat16*)bias_out, heads, head_dim, ldw);
  return cudaGetLastError();
}

cudaError_t qkv_pad_init(void* q, void* k, void* v, int64_t rows, int head_dim, cudaStream_t s) {
  const int dhp = padded_head_dim(head_dim), pad = dhp - head_dim;
  if (pad == 0 || rows == 0) return cudaSuccess;
  const int64_t n = rows * pad;
  qkv_pad_init_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>((__nv_bfloat16*)q, (__nv_bfloat16*)k, (__nv_bfloat16*)v,
                                                                 rows, head_dim, dhp);
  return cudaGetLastError();
}

}  // namespace epd
