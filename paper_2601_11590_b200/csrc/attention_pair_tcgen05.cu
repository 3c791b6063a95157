// Block-diagonal bidirectional flash attention on the 5th-generation tensor cores: two query tiles per CTA.
//
// Persistent kernel, one CTA per SM.  A work item is one (segment, head, 256 query rows): two tiles of 128
// query rows that walk the segment's keys / values together, so every K and V tile brought into shared
// memory serves both.  Each query tile w has two score buffers S_w[0], S_w[1] and an output accumulator O_w in
// tensor memory, its own running max and row sum, two issuing warps and eight softmax warps; there is nothing to
// merge at the end of an item.  The keys are walked in steps of 64; step t of query tile w uses score buffer t mod 2:
//   S_w[b] = Q_w K_t^T     tcgen05.mma, both operands K-major in shared memory, fp32 scores in TMEM
//   online softmax         the tile's softmax warps read S into registers (tcgen05.ld), take row maxima,
//                          P = exp2(S - m) as bf16 pairs, written back over the first half of the same buffer
//                          (tcgen05.st).  q arrives scaled by log2(e)/sqrt(head_dim): base-2 exponentials suffice
//   O_w += P_w V_t         one tcgen05.mma per 16 keys with P as the TMEM operand, V read MN-major from shared
//                          memory
// Issuing: one warp issues  P_w V_t  as soon as P is written, another issues  Q_w K_(t+2)^T  into the buffer P was
// read from as soon as that product is complete.  Each walks its loop as a whole warp and lets one elected lane
// issue (a product then costs the thread 40 to 50 clocks; issued from inside a branch that only lane 0 takes it
// cost ~130, and one thread per query tile was the kernel's bound).  While the softmax warps work on one buffer, the
// score product for the other one is already complete or under way.
// Softmax: a query tile's rows are spread over quads.  A warp reads 16 TMEM lanes in the 16x256b fragment shape:
// thread t holds rows t/4 and t/4 + 8 and two neighbouring columns of every 8-column block, 32 scores per step;
// the four softmax warps of an SM sub-partition are the two halves of a lane quarter for both query tiles.  The
// running max only advances (and O_w is rescaled in TMEM) when it grows by more than 2^8; until then the stale max
// serves P, the row sum and O_w alike, which leaves the result unchanged.  So after an item's first step the weights
// are computed against the running max as it stands, alongside the maxima of the thread's own quarter of its rows,
// and nothing is exchanged; only when some thread of the warp finds its quarter above the threshold do the quads
// exchange maxima (two shuffles), rescale the accumulator (after waiting for the previous step's P V, the only
// product that may still be adding to it) and compute the weights again from the scores, which are still in their
// buffer.  Where head_dim is below the padded width, column head_dim of V holds 1.0 and column head_dim of O_w is
// the row sum of P, summed by the tensor core from the same bf16 values as the numerator.  The bound at head width
// 72 is the softmax warps' step (~1600 clocks, against 1024 of the exponential unit at 16 results per clock per SM
// and 840 of products).
// Epilogue: four 8-column blocks at a time are transposed inside the quad, so that a thread writes 16 bytes and a
// quad 64 contiguous bytes of an output row.
// A segment whose length is not a multiple of 256 ends with an item whose second query tile is partly or
// wholly beyond the segment: rows beyond it are computed and not stored; a wholly empty second tile is
// skipped (its issuing warps only hand the K / V slots back, its softmax warps idle for that item).
// TMEM (512 columns): S_0[0] | S_0[1] | S_1[0] | S_1[1] | O_0 | O_1, 64 columns per score buffer and the
// padded head width per accumulator.
// Warp roles: warp 0 TMA producer of Q (per tile, NQ buffers) and the K ring, warp 3 TMA producer of the V
// ring, warps 1 / 2 the P V products of query tile 0 / 1 (warp 1 also allocates tensor memory), warps 4 / 5
// their score products, warps 6, 7 idle, warps 8..23 softmax (and epilogue): warps 8..15 query tile 0, 16..23 query
// tile 1, each half again split into the first and second 16 lanes of every TMEM lane quarter (warp & 3).  The
// softmax warps raise their register allowance at the expense of warps 0..7 (setmaxnreg).
// head_dim 72 is stored padded to 80.  Q and K tiles: columns 0..63 form a 128-byte-swizzled box, columns
// 64..79 a 32-byte-swizzled box, each contraction step its own MMA.  V tiles: five 32-byte-swizzled boxes of 16
// columns, so that one MMA covers all 80 output columns.
// Every mbarrier wait is bounded: on expiry the kernel records EPD_ETIMEOUT and drains.  No load is a
// multicast load.
#include <algorithm>
#include <vector>

#include "tcgen05_common.cuh"

namespace epd {
namespace {

using namespace tc;

constexpr int BQ = 128;          // query rows per tile; an item has two tiles
constexpr int BKV = 64;          // keys per step
constexpr int kThreads = 768;    // warps 0..7: loaders and issuing threads; warps 8..23: four softmax warpgroups
// Registers move between the warps of one SM sub-partition only (warp index mod 4), and setmaxnreg.inc waits until
// they are free: the plan must balance per sub-partition, where two warps of 0..7 and four softmax warps live:
// 2 x 64 + 4 x 88 = 6 x 80, the count the kernel is launched with.
constexpr int kRegsLow = 64, kRegsHigh = 88;
static_assert(2 * kRegsLow + 4 * kRegsHigh <= 6 * 80, "register plan does not balance per SM sub-partition");
constexpr int kMaxSegs = 128;    // segments one launch can describe
constexpr float kRescaleThreshold = 8.0f;  // log2 of the largest P value tolerated before rescaling

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

#define EPD_R8(r, o) "=r"(r[o + 0]), "=r"(r[o + 1]), "=r"(r[o + 2]), "=r"(r[o + 3]), "=r"(r[o + 4]), "=r"(r[o + 5]), \
    "=r"(r[o + 6]), "=r"(r[o + 7])
#define EPD_W8(r, o) "r"(r[o + 0]), "r"(r[o + 1]), "r"(r[o + 2]), "r"(r[o + 3]), "r"(r[o + 4]), "r"(r[o + 5]),       \
    "r"(r[o + 6]), "r"(r[o + 7])
#define EPD_R16(r, o) EPD_R8(r, o), EPD_R8(r, o + 8)
#define EPD_W16(r, o) EPD_W8(r, o), EPD_W8(r, o + 8)
#define EPD_R32(r, o) EPD_R16(r, o), EPD_R16(r, o + 16)

// tcgen05.ld / tcgen05.st in the 16-lane fragment shapes.  A warp moves 16 TMEM lanes starting at the address's
// lane (the first or second half of its lane quarter).  Shape 16x256b, per 8 columns: thread t holds rows
// t / 4 and t / 4 + 8, columns 2 (t % 4) and 2 (t % 4) + 1; register 4 k + 2 a + b = row t / 4 + 8 a, column
// 8 k + 2 (t % 4) + b.  Shape 16x128b, per 4 columns: register 2 k + a = row t / 4 + 8 a, column 4 k + t % 4.
// A row is spread over the four threads of a quad; two bf16 packed from neighbouring columns of the first shape
// land exactly on a column of the second.
__device__ __forceinline__ void ld_frag_x2(uint32_t taddr, uint32_t* r) {
  asm volatile("tcgen05.ld.sync.aligned.16x256b.x2.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : EPD_R8(r, 0) : "r"(taddr) : "memory");
}
__device__ __forceinline__ void ld_frag_x4(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.16x256b.x4.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : EPD_R16(r, 0) : "r"(taddr) : "memory");
}
__device__ __forceinline__ void ld_frag_x8(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.16x256b.x8.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : EPD_R32(r, 0) : "r"(taddr) : "memory");
}
// COLS columns (a multiple of 16) of 16 lanes: COLS / 2 registers.
template <int COLS>
__device__ __forceinline__ void ld_frag(uint32_t taddr, uint32_t* r) {
  if constexpr (COLS >= 64) { ld_frag_x8(taddr, r); ld_frag<COLS - 64>(taddr + 64, r + 32); }
  else if constexpr (COLS >= 32) { ld_frag_x4(taddr, r); ld_frag<COLS - 32>(taddr + 32, r + 16); }
  else if constexpr (COLS >= 16) { ld_frag_x2(taddr, r); ld_frag<COLS - 16>(taddr + 16, r + 8); }
}
__device__ __forceinline__ void st_frag16(uint32_t taddr, const uint32_t* r) {
  asm volatile("tcgen05.st.sync.aligned.16x256b.x2.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
               ::"r"(taddr), EPD_W8(r, 0) : "memory");
}
// KEYS bf16 weights per row as KEYS / 2 packed columns, shape 16x128b: KEYS / 4 registers.
template <int KEYS>
__device__ __forceinline__ void st_pairs(uint32_t taddr, const uint32_t* r) {
  static_assert(KEYS == 64, "one store of 32 columns");
  asm volatile(
      "tcgen05.st.sync.aligned.16x128b.x8.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), EPD_W16(r, 0) : "memory");
}

__device__ __forceinline__ float max3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}
// a_i for i in 0..3.
__device__ __forceinline__ uint32_t sel4(int i, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3) {
  const uint32_t lo = (i & 1) ? a1 : a0, hi = (i & 1) ? a3 : a2;
  return (i & 2) ? hi : lo;
}
// 2^x for x below ~100 on the FMA and integer pipes: x is rounded to the nearest integer n by adding 1.5 * 2^23
// (n lands in the low mantissa bits), 2^(x - n) is a cubic on [-0.5, 0.5] (relative error 7.5e-5, far inside the
// bf16 rounding of the weights it is used for), and n goes into the exponent field by an integer add.
__device__ __forceinline__ float ex2_fma(float x) {
  x = fmaxf(x, -125.0f);
  const float t = x + 12582912.0f;
  const float f = x - (t - 12582912.0f);
  float p = fmaf(0.05517167f, f, 0.24261113f);
  p = fmaf(p, f, 0.69326097f);
  p = fmaf(p, f, 0.99992806f);
  return __int_as_float(__float_as_int(p) + (__float_as_int(t) << 23));
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
template <int N> __device__ __forceinline__ void regs_dec() {
  asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N));
}
template <int N> __device__ __forceinline__ void regs_inc() {
  asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N));
}

// Shared-memory matrix descriptor.  layout: 2 = 128-byte swizzle, 6 = 32-byte swizzle.
// K-major operand: sbo = distance between 8-row groups.  MN-major operand: lbo = distance between
// swizzle-wide column groups, sbo = distance between 8-row (contraction) groups.
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
__host__ __device__ constexpr uint32_t instr_desc(int n, int b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)b_mn << 16) | ((uint32_t)(n >> 3) << 17) |
         ((uint32_t)(128 >> 4) << 24);
}

// Shared-memory and tensor-memory plan for a padded head width DHP (64, 80 or 128).
template <int DHP>
struct Plan {
  // score buffers S_w[b] at column (2 w + b) * BKV
  static constexpr int kO0 = 4 * BKV, kO1 = kO0 + DHP;
  static_assert(kO1 + DHP <= 512, "tensor memory plan does not fit");
  static constexpr int kMainBoxes = DHP / 64;          // Q, K: 128-byte-swizzled boxes of 64 columns
  static constexpr int kTail = DHP % 64;               // Q, K: 0 or 16 columns, 32-byte swizzle
  static_assert(kTail == 0 || kTail == 16, "padded head width must be 64*a or 64*a + 16");
  static constexpr bool kV32 = kTail != 0;             // V as 32-byte-swizzled boxes of 16 columns
  static constexpr int kQMain = BQ * 128;              // bytes of a main box of a Q tile
  static constexpr int kQTile = BQ * DHP * 2;          // bytes of a Q tile
  static constexpr int kKMain = BKV * 128;             // bytes of a main box of a K tile
  static constexpr int kKTile = BKV * DHP * 2;         // bytes of a K or V tile
  static_assert(kQTile % 1024 == 0 && kKTile % 1024 == 0, "tiles keep the 1024-byte alignment of the swizzled boxes");
  static constexpr int kVBox = kV32 ? BKV * 32 : BKV * 128;
  static constexpr int kVBoxes = kV32 ? DHP / 16 : DHP / 64;
  static_assert(kVBox * kVBoxes == kKTile, "V tile");
  static constexpr int NQ = DHP == 128 ? 1 : 2;        // buffers per query tile
  static constexpr int KS = DHP == 128 ? 4 : DHP == 80 ? 6 : 8;   // K ring depth
  static constexpr int VS = DHP == 128 ? 5 : DHP == 80 ? 6 : 8;   // V ring depth
  static constexpr int kQ = 0;                         // [tile w][buffer b]
  static constexpr int kK = 2 * NQ * kQTile;
  static constexpr int kV = kK + KS * kKTile;
  static constexpr int kBar = kV + VS * kKTile;
  // q_full[2][NQ] q_empty[2][NQ] k_full[KS] k_empty[KS] v_full[VS] v_empty[VS] s_full[2][2] p_full[2][2]
  // pv_done[2][2] o_done[2] o_free[2] drain[4]
  static constexpr int kNumBars = 4 * NQ + 2 * KS + 2 * VS + 20;
  static constexpr int kTotal = kBar + kNumBars * 8 + 32;
  static constexpr int kDynamic = kTotal + 1024;       // slack to align the tiles to 1024 bytes
  static_assert(kDynamic > 116 * 1024, "one CTA per SM is assumed by the TMEM allocation");
  static_assert(kDynamic <= 232448, "exceeds the shared memory of one CTA");
};

struct Maps {
  CUtensorMap q_main, q_tail, k_main, k_tail, v;   // q boxes are BQ rows high, k and v boxes BKV rows
};

// Segments of one launch, longest first (host-sorted).
struct SegList {
  int n;
  int beg[kMaxSegs];
  int len[kMaxSegs];
  int first[kMaxSegs];    // number of the segment's first item
};

struct Item {
  int head, seg_beg, seg_len, q0, n_kv;
  bool two;     // the second query tile holds rows of the segment
};

// Item i -> (segment, head, 256-row query block): segments in list order, then head, then query block, so
// that neighbouring items (which run at the same time on different SMs) share K and V in L2.
// A CTA's items come in ascending order: `seg` is the caller's cursor into the segment list (0 before its first item).
__device__ __forceinline__ Item decode_item(const SegList& segs, int i, int& seg) {
  while (seg + 1 < segs.n && i >= segs.first[seg + 1]) ++seg;
  Item it;
  it.seg_beg = segs.beg[seg];
  it.seg_len = segs.len[seg];
  const int qb = (it.seg_len + 2 * BQ - 1) / (2 * BQ);
  i -= segs.first[seg];
  it.head = i / qb;
  it.q0 = it.seg_beg + (i - it.head * qb) * 2 * BQ;
  it.n_kv = (it.seg_len + BKV - 1) / BKV;
  it.two = it.q0 + BQ < it.seg_beg + it.seg_len;
  return it;
}

// ONES: head_dim < DHP and column head_dim of every V row holds 1.0, so column head_dim of O_w is the row sum
// of P_w and the softmax threads need not add it up.
template <int DHP, bool ONES>
__global__ void __launch_bounds__(kThreads, 1)
attention_pair_kernel(const __grid_constant__ Maps maps, const __grid_constant__ SegList segs, int n_items,
                      __nv_bfloat16* __restrict__ out, int T, int heads, int dh, int* __restrict__ status,
                      long long wait_limit) {
  using P = Plan<DHP>;
  constexpr int NQ = P::NQ;
  pdl_launch_dependents();
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + P::kBar);
  uint64_t* q_full = bars;                    // [2][NQ]  Q tile w, buffer b loaded
  uint64_t* q_empty = q_full + 2 * NQ;        // [2][NQ]  its last score product is complete
  uint64_t* k_full = q_empty + 2 * NQ;        // [KS]
  uint64_t* k_empty = k_full + P::KS;         // [KS]  both issuing threads are done with the slot (2 arrivals)
  uint64_t* v_full = k_empty + P::KS;         // [VS]
  uint64_t* v_empty = v_full + P::VS;         // [VS]  (2 arrivals)
  uint64_t* s_full = v_empty + P::VS;         // [2][2]  S_w[b] complete
  uint64_t* p_full = s_full + 4;              // [2][2]  P written over S_w[b] (8 warp arrivals)
  uint64_t* pv_done = p_full + 4;             // [2][2]  the P_w V product that read P from S_w[b] is complete
  uint64_t* o_done = pv_done + 4;             // [2]  the item's last P_w V is complete: O_w final
  uint64_t* o_free = o_done + 2;              // [2]  O_w read out by its warps (8 warp arrivals)
  uint64_t* drain = o_free + 2;               // [4]  after an abort: the products of an issuing thread have completed
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + P::kNumBars);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const WaitCtx wc{abort_flag, 0u, wait_limit};
  uint32_t q_loads0 = 0, q_loads1 = 0, kv_loads = 0;   // loads issued by this thread (warp 0: Q and K tiles, warp 3: V tiles)

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int i = 0; i < P::kNumBars; ++i) mbar_init(&bars[i], 1);
    for (int i = 0; i < P::KS; ++i) mbar_init(&k_empty[i], 2);
    for (int i = 0; i < P::VS; ++i) mbar_init(&v_empty[i], 2);
    for (int i = 0; i < 4; ++i) mbar_init(&p_full[i], 8);
    for (int w = 0; w < 2; ++w) mbar_init(&o_free[w], 8);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  pdl_wait();   // nothing above touches global memory
  if (warp < 8) regs_dec<kRegsLow>();

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer of Q and K
    if (lane == 0) {
      uint32_t kc = 0, n = 0;
      bool ok = true;
      int seg_cur = 0;
      for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++n) {
        const Item it = decode_item(segs, item, seg_cur);
        const int row_base = it.head * T;
        const int qb = n % NQ;
        const uint32_t qphase = (n / NQ) & 1;
        // both query tiles are loaded even when the second holds no row of the segment: the barrier
        // counters then advance the same way for every item
        for (int w = 0; w < 2 && ok; ++w) {
          if (!mbar_wait(&q_empty[w * NQ + qb], qphase ^ 1, wc)) { ok = false; break; }
          uint8_t* dst = smem + P::kQ + (w * NQ + qb) * P::kQTile;
          uint64_t* full = &q_full[w * NQ + qb];
          const int row = row_base + it.q0 + w * BQ;
          mbar_expect_tx(full, P::kQTile);
#pragma unroll
          for (int b = 0; b < P::kMainBoxes; ++b) tma_load_2d(dst + b * P::kQMain, &maps.q_main, b * 64, row, full);
          if (P::kTail) tma_load_2d(dst + P::kMainBoxes * P::kQMain, &maps.q_tail, P::kMainBoxes * 64, row, full);
          if (w == 0) ++q_loads0; else ++q_loads1;
        }
        if (!ok) break;
        for (int j = 0; j < it.n_kv; ++j, ++kc) {
          const int row = row_base + it.seg_beg + j * BKV;
          const int ks = kc % P::KS;
          if (!mbar_wait(&k_empty[ks], ((kc / P::KS) & 1) ^ 1, wc)) { ok = false; break; }
          uint8_t* dk = smem + P::kK + ks * P::kKTile;
          mbar_expect_tx(&k_full[ks], P::kKTile);
#pragma unroll
          for (int b = 0; b < P::kMainBoxes; ++b) tma_load_2d(dk + b * P::kKMain, &maps.k_main, b * 64, row, &k_full[ks]);
          if (P::kTail) tma_load_2d(dk + P::kMainBoxes * P::kKMain, &maps.k_tail, P::kMainBoxes * 64, row, &k_full[ks]);
          ++kv_loads;
        }
      }
    }
    __syncwarp();
  } else if (warp == 3) {
    // ---------------------------------------------------------------- TMA producer of V
    if (lane == 0) {
      uint32_t vc = 0;
      bool ok = true;
      int seg_cur = 0;
      for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
        const Item it = decode_item(segs, item, seg_cur);
        const int row_base = it.head * T;
        for (int j = 0; j < it.n_kv; ++j, ++vc) {
          const int row = row_base + it.seg_beg + j * BKV;
          const int vs = vc % P::VS;
          if (!mbar_wait(&v_empty[vs], ((vc / P::VS) & 1) ^ 1, wc)) { ok = false; break; }
          uint8_t* dv = smem + P::kV + vs * P::kKTile;
          mbar_expect_tx(&v_full[vs], P::kKTile);
#pragma unroll
          for (int b = 0; b < P::kVBoxes; ++b)
            tma_load_2d(dv + b * P::kVBox, &maps.v, b * (P::kV32 ? 16 : 64), row, &v_full[vs]);
          ++kv_loads;
        }
      }
    }
    __syncwarp();
  } else if (warp == 1 || warp == 2) {
    // ---------------------------------------------------------------- P V products of query tile w
    // The whole warp walks the loop (so that addresses and descriptors are warp-uniform values); one elected lane
    // issues.
    {
      const int w = warp - 1;
      uint32_t vc = 0;                 // V tiles seen (all of them, also in skipped items)
      uint32_t c = 0;                  // steps of this query tile so far: step c uses score buffer c & 1
      uint32_t items_w = 0;            // items in which this query tile took part
      constexpr uint32_t idesc_pv = instr_desc(DHP, 1);
      constexpr uint32_t kVStep = P::kV32 ? 512 / 16 : 2048 / 16;   // 16 keys further down the V tile, 16-byte units
      const uint32_t tmem_o = tmem_base + (w ? P::kO1 : P::kO0);
      bool ok = true;
      int seg_cur = 0;
      for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
        const Item it = decode_item(segs, item, seg_cur);
        if (w == 1 && !it.two) {
          // nothing to compute for this query tile: hand every V slot back, each only once it has been filled
          // (so that an arrival can never be counted for a later use of the slot)
          for (int j = 0; j < it.n_kv; ++j, ++vc) {
            if (!mbar_wait_warp(&v_full[vc % P::VS], (vc / P::VS) & 1, wc)) { ok = false; break; }
            if (lane == 0) mbar_arrive(&v_empty[vc % P::VS]);
          }
          continue;
        }
        for (int t = 0; t < it.n_kv; ++t, ++vc, ++c) {
          const int vs = vc % P::VS;
          if (!mbar_wait_warp(&v_full[vs], (vc / P::VS) & 1, wc)) { ok = false; break; }
          if (t == 0) {
            // the accumulator of the query tile's previous item must have been read out
            if (items_w > 0 && !mbar_wait_warp(&o_free[w], (items_w - 1) & 1, wc)) { ok = false; break; }
            ++items_w;
          }
          // P of this step is in tensor memory
          if (!mbar_wait_warp(&p_full[2 * w + (c & 1)], (c >> 1) & 1, wc)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sv = smem_u32(smem + P::kV + vs * P::kKTile);
          // MN-major V: boxes (16 or 64 columns wide) are kVBox apart, 8-row groups 256 / 1024 bytes apart
          const uint64_t dv = P::kV32 ? smem_desc(sv, P::kVBox, 256, 6) : smem_desc(sv, P::kVBox, 1024, 2);
          const uint32_t tmem_p = tmem_base + (2 * w + (c & 1)) * BKV;
          const int kv_valid = min(BKV, it.seg_len - t * BKV);
          const int steps = (kv_valid + 15) >> 4;
          if (elect_one()) {
            if (steps == BKV / 16) {
#pragma unroll
              for (int s = 0; s < BKV / 16; ++s)       // 16 bf16 of P = 8 columns
                umma_ts(tmem_o, tmem_p + s * 8, dv + s * kVStep, idesc_pv, (t | s) != 0 ? 1u : 0u);
            } else {
              for (int s = 0; s < steps; ++s)
                umma_ts(tmem_o, tmem_p + s * 8, dv + s * kVStep, idesc_pv, (t | s) != 0 ? 1u : 0u);
            }
            umma_commit(&pv_done[2 * w + (c & 1)]);    // frees the score buffer, orders rescales
            umma_commit(&v_empty[vs]);
            if (t == it.n_kv - 1) umma_commit(&o_done[w]);
          }
          __syncwarp();
        }
      }
    }
    __syncwarp();
  } else if (warp == 4 || warp == 5) {
    // ---------------------------------------------------------------- score products of query tile w
    {
      const int w = warp - 4;
      uint32_t kc = 0, n = 0;          // K tiles / items seen (all of them, also in skipped items)
      uint32_t g = 0;                  // score tiles of this query tile so far: tile g goes to buffer g & 1
      bool ok = true;
      int seg_cur = 0;
      for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++n) {
        const Item it = decode_item(segs, item, seg_cur);
        const int qb = n % NQ;
        const uint32_t qphase = (n / NQ) & 1;
        if (!mbar_wait_warp(&q_full[w * NQ + qb], qphase, wc)) break;
        if (w == 1 && !it.two) {
          // nothing to compute for this query tile: hand the Q buffer and every K slot back, each only once it
          // has been filled
          if (lane == 0) mbar_arrive(&q_empty[w * NQ + qb]);
          for (int j = 0; j < it.n_kv; ++j, ++kc) {
            if (!mbar_wait_warp(&k_full[kc % P::KS], (kc / P::KS) & 1, wc)) { ok = false; break; }
            if (lane == 0) mbar_arrive(&k_empty[kc % P::KS]);
          }
          continue;
        }
        const uint32_t sq = smem_u32(smem + P::kQ + (w * NQ + qb) * P::kQTile);
        const uint64_t dq_main = smem_desc(sq, 16, 1024, 2);
        const uint64_t dq_tail = smem_desc(sq + P::kMainBoxes * P::kQMain, 16, 256, 6);
        for (int t = 0; t < it.n_kv; ++t, ++kc, ++g) {
          const int ks = kc % P::KS;
          if (!mbar_wait_warp(&k_full[ks], (kc / P::KS) & 1, wc)) { ok = false; break; }
          // the buffer's previous content (P of the step two before) must have been consumed by its P V product.
          // One barrier per buffer: the buffer's next product cannot complete before these scores exist, so the
          // barrier is at most one phase past the one waited for and the parity is unambiguous.
          if (g >= 2 && !mbar_wait_warp(&pv_done[2 * w + (g & 1)], ((g >> 1) - 1) & 1, wc)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sk = smem_u32(smem + P::kK + ks * P::kKTile);
          const uint64_t dk_main = smem_desc(sk, 16, 1024, 2);
          const uint64_t dk_tail = smem_desc(sk + P::kMainBoxes * P::kKMain, 16, 256, 6);
          const uint32_t tmem_s = tmem_base + (2 * w + (g & 1)) * BKV;
          const int kv_valid = min(BKV, it.seg_len - t * BKV);
          const uint32_t idesc = kv_valid == BKV ? instr_desc(BKV, 0) : instr_desc((kv_valid + 15) & ~15, 0);
          // descriptor addresses count 16-byte units: one 16-element step inside a swizzled row is +2
          if (elect_one()) {
#pragma unroll
            for (int b = 0; b < P::kMainBoxes; ++b) {
#pragma unroll
              for (int k = 0; k < 4; ++k)
                umma_ss(tmem_s, dq_main + (b * P::kQMain / 16 + 2 * k), dk_main + (b * P::kKMain / 16 + 2 * k), idesc,
                        (b | k) != 0);
            }
            if (P::kTail) umma_ss(tmem_s, dq_tail, dk_tail, idesc, 1);
            umma_commit(&s_full[2 * w + (g & 1)]);
            umma_commit(&k_empty[ks]);
            if (t == it.n_kv - 1) umma_commit(&q_empty[w * NQ + qb]);   // the query tile's last score product
          }
          __syncwarp();
        }
      }
    }
    __syncwarp();
  } else if (warp >= 8) {
    // ---------------------------------------------------------------- softmax / rescale / epilogue
    regs_inc<kRegsHigh>();
    const int grp = (warp - 8) >> 2;
    const int w = grp >> 1;                             // query tile of this warp
    const int hf = grp & 1;                             // which 16 rows of the warp's TMEM lane quarter
    const int qr = warp & 3;                            // TMEM lane quarter this warp may access
    const int quad = lane & 3;                          // the four threads of a quad share two rows
    const int r0 = qr * 32 + hf * 16 + (lane >> 2);     // this thread's query rows inside the tile: r0 and r0 + 8
    const uint32_t lane_off = (uint32_t)(qr * 32 + hf * 16) << 16;
    const uint32_t tmem_s0 = tmem_base + 2 * w * BKV + lane_off;   // S_w[0]; S_w[1] is BKV columns further
    const uint32_t tmem_o = tmem_base + (w ? P::kO1 : P::kO0) + lane_off;
    uint32_t c = 0, oc = 0;                             // steps / items processed by this warp
    bool ok = true;
    int seg_cur = 0;
    for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
      const Item it = decode_item(segs, item, seg_cur);
      if (w == 1 && !it.two) continue;                  // no row of the segment in this query tile
      float m[2] = {-INFINITY, -INFINITY}, l[2] = {0.0f, 0.0f};
      for (int t = 0; t < it.n_kv; ++t, ++c) {
        const int kv_valid = min(BKV, it.seg_len - t * BKV);
        const uint32_t tmem_s = tmem_s0 + (c & 1) * BKV;   // P lives in the buffer's first BKV / 2 columns
        if (!mbar_wait_warp(&s_full[2 * w + (c & 1)], (c >> 1) & 1, wc)) { ok = false; break; }
        tc_fence_after();
        // register 4 k + 2 a + b holds row r0 + 8 a, column 8 k + 2 quad + b
        uint32_t s[BKV / 2];
        ld_frag<BKV>(tmem_s, s);
        tmem_ld_wait();

        // P = exp2(S - m) as bf16 pairs, to be written over the first half of the score buffer: b32 column
        // 4 k + quad of row r0 + 8 a is register 2 k + a.  Keys beyond the segment get weight zero (the products
        // read P in whole groups of 16 keys).
        uint32_t pk[BKV / 4];
        float sum0 = 0.0f, sum1 = 0.0f;
        auto weights = [&](float neg_m0, float neg_m1) {
          sum0 = sum1 = 0.0f;
          if (kv_valid == BKV) {
#pragma unroll
            for (int k = 0; k < BKV / 8; ++k) {
              const float p0 = ex2(__uint_as_float(s[4 * k]) + neg_m0);
              const float p1 = ex2(__uint_as_float(s[4 * k + 1]) + neg_m0);
              const float p2 = ex2(__uint_as_float(s[4 * k + 2]) + neg_m1);
              // one exponential in eight is evaluated on the FMA pipe for head width 72 (padded to 80, row sums from
              // the ones column), where the exponential unit is the busiest one and the FMA pipe has room: measured
              // in one run +2.5 to +4 % there, -3 % at head width 128, -5 % at 64 and 80, where the row sums are added
              // on the FMA pipe as well; one in four or one in sixteen were slower than none
              const float p3 = (ONES && DHP == 80 && (k & 1)) ? ex2_fma(__uint_as_float(s[4 * k + 3]) + neg_m1)
                                                              : ex2(__uint_as_float(s[4 * k + 3]) + neg_m1);
              if (!ONES) { sum0 += p0 + p1; sum1 += p2 + p3; }
              __nv_bfloat162 b0 = __floats2bfloat162_rn(p0, p1), b1 = __floats2bfloat162_rn(p2, p3);
              pk[2 * k] = *reinterpret_cast<uint32_t*>(&b0);
              pk[2 * k + 1] = *reinterpret_cast<uint32_t*>(&b1);
            }
          } else {
#pragma unroll
            for (int k = 0; k < BKV / 8; ++k) {
              const int col = 8 * k + 2 * quad;
              const float p0 = col < kv_valid ? ex2(__uint_as_float(s[4 * k]) + neg_m0) : 0.0f;
              const float p1 = col + 1 < kv_valid ? ex2(__uint_as_float(s[4 * k + 1]) + neg_m0) : 0.0f;
              const float p2 = col < kv_valid ? ex2(__uint_as_float(s[4 * k + 2]) + neg_m1) : 0.0f;
              const float p3 = col + 1 < kv_valid ? ex2(__uint_as_float(s[4 * k + 3]) + neg_m1) : 0.0f;
              if (!ONES) { sum0 += p0 + p1; sum1 += p2 + p3; }
              __nv_bfloat162 b0 = __floats2bfloat162_rn(p0, p1), b1 = __floats2bfloat162_rn(p2, p3);
              pk[2 * k] = *reinterpret_cast<uint32_t*>(&b0);
              pk[2 * k + 1] = *reinterpret_cast<uint32_t*>(&b1);
            }
          }
        };
        // maximum over this thread's quarter of its two rows
        float mx[2] = {-INFINITY, -INFINITY};
        if (kv_valid == BKV) {
#pragma unroll
          for (int k = 0; k < BKV / 8; ++k) {
            mx[0] = max3(mx[0], __uint_as_float(s[4 * k]), __uint_as_float(s[4 * k + 1]));
            mx[1] = max3(mx[1], __uint_as_float(s[4 * k + 2]), __uint_as_float(s[4 * k + 3]));
          }
        } else {
#pragma unroll
          for (int i = 0; i < BKV / 2; ++i)
            if (8 * (i >> 2) + 2 * quad + (i & 1) < kv_valid) mx[(i >> 1) & 1] = fmaxf(mx[(i >> 1) & 1], __uint_as_float(s[i]));
        }
        // A row's running max only advances when it would grow by more than the threshold, so after an item's
        // first step the weights are almost always taken against the running max as it stands: they are computed
        // at once, alongside the maxima, and kept unless some thread of the warp finds its quarter of a row above
        // the threshold (if none does, no row is, and the threads of a quad still share their rows' running max
        // without having exchanged anything).  Otherwise, and in the first step, the quads exchange their
        // maxima, take the same decision per row, rescale what has been accumulated and compute the weights
        // against the new max.
        bool exact = t == 0;
        if (t != 0) {
          weights(-m[0], -m[1]);
          exact = __any_sync(0xffffffffu, mx[0] - m[0] > kRescaleThreshold || mx[1] - m[1] > kRescaleThreshold);
        }
        if (exact) {
          float scale[2] = {1.0f, 1.0f};
#pragma unroll
          for (int a = 0; a < 2; ++a) {
            mx[a] = fmaxf(mx[a], __shfl_xor_sync(0xffffffffu, mx[a], 1));
            mx[a] = fmaxf(mx[a], __shfl_xor_sync(0xffffffffu, mx[a], 2));
            if (t == 0) {
              m[a] = mx[a];
            } else if (mx[a] - m[a] > kRescaleThreshold) {
              scale[a] = ex2(m[a] - mx[a]);
              m[a] = mx[a];
              l[a] *= scale[a];
            }
          }
          if (t != 0) {
            // O_w must be quiescent: the product of step t-2 is complete (these scores were issued behind it); the
            // product of step t-1 is the only one that may still be adding to it
            if (!mbar_wait_warp(&pv_done[2 * w + ((c - 1) & 1)], ((c - 1) >> 1) & 1, wc)) { ok = false; break; }
            tc_fence_after();
#pragma unroll
            for (int q = 0; q < DHP / 16; ++q) {
              uint32_t o[8];
              ld_frag<16>(tmem_o + q * 16, o);
              tmem_ld_wait();
#pragma unroll
              for (int i = 0; i < 8; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * scale[(i >> 1) & 1]);
              st_frag16(tmem_o + q * 16, o);
            }
            // the scores are still in their buffer
            ld_frag<BKV>(tmem_s, s);
            tmem_ld_wait();
          }
          weights(-m[0], -m[1]);
        }
        st_pairs<BKV>(tmem_s, pk);
        if (!ONES) { l[0] += sum0; l[1] += sum1; }
        tmem_st_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&p_full[2 * w + (c & 1)]);
      }
      if (!ok) break;
      // ---- epilogue: O_w / l -> out
      if (!mbar_wait_warp(&o_done[w], oc & 1, wc)) { ok = false; break; }
      ++oc;
      tc_fence_after();
      // the accumulator rows go into registers (same fragment layout as the scores), then the accumulator is
      // handed back
      uint32_t o[DHP / 2];
      ld_frag<DHP>(tmem_o, o);
      tmem_ld_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&o_free[w]);
      if (ONES) {
        // head_dim = DHP - 8: the row sums sit in column head_dim, held by the first thread of the quad
        constexpr int kb = DHP / 8 - 1;
        l[0] = __shfl_sync(0xffffffffu, __uint_as_float(o[4 * kb]), lane & ~3);
        l[1] = __shfl_sync(0xffffffffu, __uint_as_float(o[4 * kb + 2]), lane & ~3);
      } else {
#pragma unroll
        for (int a = 0; a < 2; ++a) {
          l[a] += __shfl_xor_sync(0xffffffffu, l[a], 1);
          l[a] += __shfl_xor_sync(0xffffffffu, l[a], 2);
        }
      }
      // A thread holds two neighbouring columns of every 8-column block of its rows.  Four blocks at a time are
      // transposed inside the quad (three exchanges), after which thread q of the quad holds all 8 columns of
      // block 4 g + q and writes them as 16 bytes: a quad writes 64 contiguous bytes of a row.
      constexpr int kBlocks = DHP / 8;
#pragma unroll
      for (int a = 0; a < 2; ++a) {
        const int token = it.q0 + w * BQ + r0 + 8 * a;
        const bool row_ok = token < it.seg_beg + it.seg_len;
        const float inv = 1.0f / l[a];
        __nv_bfloat16* orow = out + (int64_t)token * (heads * dh) + it.head * dh;
        auto word = [&](int k) {
          __nv_bfloat162 b2 = __floats2bfloat162_rn(__uint_as_float(o[4 * k + 2 * a]) * inv,
                                                    __uint_as_float(o[4 * k + 2 * a + 1]) * inv);
          return *reinterpret_cast<uint32_t*>(&b2);
        };
#pragma unroll
        for (int g = 0; g < kBlocks / 4; ++g) {
          const uint32_t w0 = word(4 * g), w1 = word(4 * g + 1), w2 = word(4 * g + 2), w3 = word(4 * g + 3);
          // what lane q ^ r needs from this lane is this lane's word of block q ^ r
          const uint32_t r0w = sel4(quad, w0, w1, w2, w3);
          const uint32_t r1w = __shfl_xor_sync(0xffffffffu, sel4(quad ^ 1, w0, w1, w2, w3), 1);
          const uint32_t r2w = __shfl_xor_sync(0xffffffffu, sel4(quad ^ 2, w0, w1, w2, w3), 2);
          const uint32_t r3w = __shfl_xor_sync(0xffffffffu, sel4(quad ^ 3, w0, w1, w2, w3), 3);
          // word j of the block comes from lane j of the quad, i.e. from the exchange with distance j ^ q
          const uint4 v = make_uint4(sel4(quad, r0w, r1w, r2w, r3w), sel4(quad ^ 1, r0w, r1w, r2w, r3w),
                                     sel4(quad ^ 2, r0w, r1w, r2w, r3w), sel4(quad ^ 3, r0w, r1w, r2w, r3w));
          const int blk = 4 * g + quad;
          if (row_ok && blk * 8 < dh) *reinterpret_cast<uint4*>(orow + blk * 8) = v;   // head_dim is a multiple of 8
        }
#pragma unroll
        for (int k = kBlocks / 4 * 4; k < kBlocks; ++k)
          if (row_ok && k * 8 < dh) *reinterpret_cast<uint32_t*>(orow + k * 8 + 2 * quad) = word(k);
      }
    }
  }

  // ---------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    // A wait expired.  Every role has left its loop, so nothing new is issued.  What was issued completes by
    // itself: each loader waits for its last load of every ring slot, each issuing thread for its last product
    // (a commit arrives only after all earlier products); the softmax warps write their rows with ordinary
    // stores.  A fixed pause on top, then shared and tensor memory are released.
    if (threadIdx.x == 0 && status != nullptr) atomicCAS(status, 0, kStatusTimeout);
    if (lane == 0) {
      if (warp == 0) {
        drain_ring(q_full, NQ, q_loads0);
        drain_ring(q_full + NQ, NQ, q_loads1);
        drain_ring(k_full, P::KS, kv_loads);
      }
      if (warp == 3) drain_ring(v_full, P::VS, kv_loads);
    }
    if (warp == 1 || warp == 2 || warp == 4 || warp == 5) {
      // the lane that issued the warp's products commits (a commit covers the products of its own thread)
      if (elect_one()) {
        const int d = warp < 3 ? warp - 1 : warp - 2;
        umma_commit(&drain[d]);
        mbar_wait_drain(&drain[d], 0);
      }
      __syncwarp();
    }
    for (int i = 0; i < 64; ++i) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

// ---------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------

// Map over a bf16 matrix [rows, dhp] (row pitch dhp*2 bytes): box = box_rows rows x box_cols columns.
bool make_map(CUtensorMap* tm, const void* base, int64_t rows, int dhp, int box_rows, int box_cols,
              CUtensorMapSwizzle swz) {
  return make_tensor_map_2d(tm, base, rows, dhp, (int64_t)dhp * 2, box_rows, box_cols, 2, swz);
}

template <int DHP, bool ONES>
cudaError_t launch(const Maps& maps, const SegList& segs, int n_items, void* out, int T, int heads, int dh,
                   int* status, cudaStream_t s) {
  using P = Plan<DHP>;
  auto kern = attention_pair_kernel<DHP, ONES>;
  static PerDeviceOnce configured;
  cudaError_t e = once_per_device(configured, [&] {
    return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, P::kDynamic);
  });
  if (e != cudaSuccess) return e;
  const int sms = limited_sms(device_sm_count());
  const int grid = n_items < sms ? n_items : sms;
  return launch_pdl(kern, dim3(grid), dim3(kThreads), P::kDynamic, s, maps, segs, n_items, (__nv_bfloat16*)out, T, heads, dh,
                    status, wait_limit_cycles());
}

}  // namespace

bool attention_pair_supported(const void* q, const void* k, const void* v, const void* out, int64_t T, int heads,
                              int head_dim) {
  const int dhp = padded_head_dim(head_dim);
  if (dhp != 64 && dhp != 80 && dhp != 128) return false;
  if (head_dim % 8) return false;
  if (dhp != head_dim && dhp - head_dim != 8) return false;   // the row-sum column is read at padded width - 8
  if (((uintptr_t)q & 15) || ((uintptr_t)k & 15) || ((uintptr_t)v & 15) || ((uintptr_t)out & 15)) return false;
  if ((int64_t)heads * T > (1 << 30) || heads > 65535) return false;
  return tensor_maps_available();
}

cudaError_t attention_pair(const void* q, const void* k, const void* v, const int32_t* host_cu_seqlens, int n_seg,
                           void* out, int64_t T, int heads, int head_dim, int* status, cudaStream_t s) {
  const int dhp = padded_head_dim(head_dim);
  if (n_seg <= 0) return cudaSuccess;
  const int64_t rows = (int64_t)heads * T;
  Maps maps;
  if (!make_map(&maps.q_main, q, rows, dhp, BQ, 64, CU_TENSOR_MAP_SWIZZLE_128B) ||
      !make_map(&maps.q_tail, q, rows, dhp, BQ, 16, CU_TENSOR_MAP_SWIZZLE_32B) ||
      !make_map(&maps.k_main, k, rows, dhp, BKV, 64, CU_TENSOR_MAP_SWIZZLE_128B) ||
      !make_map(&maps.k_tail, k, rows, dhp, BKV, 16, CU_TENSOR_MAP_SWIZZLE_32B))
    return cudaErrorInvalidValue;
  if (dhp % 64 ? !make_map(&maps.v, v, rows, dhp, BKV, 16, CU_TENSOR_MAP_SWIZZLE_32B)
               : !make_map(&maps.v, v, rows, dhp, BKV, 64, CU_TENSOR_MAP_SWIZZLE_128B))
    return cudaErrorInvalidValue;
  // longest segments first: items are dealt round-robin, so the long ones spread evenly and the
  // short ones fill the tail
  std::vector<int> order(n_seg);
  for (int i = 0; i < n_seg; ++i) order[i] = i;
  std::stable_sort(order.begin(), order.end(), [&](int a, int b) {
    return host_cu_seqlens[a + 1] - host_cu_seqlens[a] > host_cu_seqlens[b + 1] - host_cu_seqlens[b];
  });
  for (int first = 0; first < n_seg; first += kMaxSegs) {
    SegList segs;
    segs.n = n_seg - first < kMaxSegs ? n_seg - first : kMaxSegs;
    int n_items = 0;
    for (int i = 0; i < segs.n; ++i) {
      const int sg = order[first + i];
      segs.beg[i] = host_cu_seqlens[sg];
      segs.len[i] = host_cu_seqlens[sg + 1] - host_cu_seqlens[sg];
      segs.first[i] = n_items;
      n_items += (segs.len[i] + 2 * BQ - 1) / (2 * BQ) * heads;
    }
    for (int i = segs.n; i < kMaxSegs; ++i) segs.beg[i] = segs.len[i] = segs.first[i] = 0;
    cudaError_t e;
    switch (dhp) {
#define EPD_ATT(D)                                                                                          \
  e = head_dim < D ? launch<D, true>(maps, segs, n_items, out, (int)T, heads, head_dim, status, s)          \
                   : launch<D, false>(maps, segs, n_items, out, (int)T, heads, head_dim, status, s)
      case 64: EPD_ATT(64); break;
      case 80: EPD_ATT(80); break;
      case 128: EPD_ATT(128); break;
#undef EPD_ATT
      default: return cudaErrorInvalidValue;
    }
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

}  // namespace epd
