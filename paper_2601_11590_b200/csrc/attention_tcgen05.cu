// Block-diagonal bidirectional flash attention on the 5th-generation tensor cores.
//
// Persistent kernel, one CTA per SM.  A work item is one (segment, head, 128-query tile); items are
// ordered longest segment first and dealt round-robin to the CTAs.  Inside an item the segment's
// keys/values stream through shared memory in tiles of BKV keys, and the two softmax warpgroups take
// alternate key tiles, each with its own running max / sum and its own output accumulator:
//   S_w = Q K^T        tcgen05.mma, both operands K-major in shared memory, fp32 S_w in TMEM (w = warpgroup)
//   online softmax     warpgroup w, one thread per query row: the S row is read once into registers
//                      (tcgen05.ld) and the S_w buffer handed back at once, so the next S_w is computed
//                      while this tile's exponentials run; P = exp2(S - m) goes to a separate bf16
//                      buffer P_w (tcgen05.st).  q arrives scaled by log2(e)/sqrt(head_dim), so base-2
//                      exponentials suffice
//   O_w += P_w V       one tcgen05.mma per 16 keys with P_w as the TMEM operand and V read MN-major
//                      from shared memory
// Two threads feed the tensor pipe, one issuing the score products and one the P V products (the
// waits and commits around a product cost more issue time than the product itself, so one thread
// cannot keep up).  Score tiles run ahead of the P V products by as much as the S_w buffers and the
// K ring allow, so a warpgroup does not wait for the tensor pipe in steady state and the exponential
// unit stays busy.  That unit delivers 16 results per clock per SM; evaluating part of the exponentials
// on the FMA pipe instead (cubic for 2^fraction, kFmaExpEvery) is implemented but off: measured on
// B200 the softmax warps are bound by instruction issue as much as by that unit, and the extra FMAs
// cost more than they save (16k-token segment: 660 TFLOP/s without, 622 with one in four, 517 with one in two).
// The running max only advances (and O_w is rescaled in TMEM) when it grows by more than 2^8; until
// then the stale max serves P, the row sum and O_w alike, which leaves the result unchanged.  At the
// end of an item the two partial results are merged:
//   m = max(m0, m1),  O = (2^(m0-m) O0 + 2^(m1-m) O1) / (2^(m0-m) l0 + 2^(m1-m) l1)
// by the warpgroup that owns the item's last key tile.  The other one publishes its (m, l) and starts on
// the next item's score tiles at once; the first key tile of the next item is given to it.  The merging
// warpgroup first copies the other accumulator into its (dead) score registers and hands it back, then
// its own, so the other warpgroup's P V products of the next item are not held up by the merge; each
// accumulator has its own "complete" (o_done) and "read out" (o_free) barrier.  With an odd number of
// key tiles (7 for a 784-token image) the extra tile and the merge alternate between the warpgroups.
// (Measured against both warpgroups waiting for each other and sharing the epilogue: 16384-token segment
// 726 -> 756 TFLOP/s, 8 x 784 tokens 361 -> 383, mixed lengths 569 -> 581, 16 x 1024 tokens 466 -> 457.)
// TMEM (512 columns): S0 | P0 | S1 | P1 | O0 | O1, with BKV chosen so that this fits: 112 keys for a
// padded head width of 80, 80 keys for 128, 128 keys for 64.
// Warp roles: warp 0 TMA producer of Q (double-buffered across items) and the K ring, warp 3 TMA
// producer of the V ring (a V tile stays resident much longer than a K tile, so the two rings must
// not throttle each other), warp 1 TMEM allocation + Q K^T issue, warp 2 P V issue, warps 4..7 and
// 8..11 the two softmax warpgroups (also merge + epilogue).
// head_dim 72 is stored padded to 80.  Q and K tiles: columns 0..63 form a 128-byte-swizzled box,
// columns 64..79 a 32-byte-swizzled box, each contraction step its own MMA.  V tiles: five
// 32-byte-swizzled boxes of 16 columns, so that one MMA covers all 80 output columns (an MMA costs
// max(45, N/2) clocks whatever its width, so few wide ones beat many narrow ones).
// Every mbarrier wait is bounded: on expiry the kernel records EPD_ETIMEOUT and drains.
#include <algorithm>
#include <vector>

#include "tcgen05_common.cuh"

namespace epd {
namespace {

using namespace tc;

constexpr int BQ = 128;          // query rows per work item
constexpr int kThreads = 384;    // warps 0..3: loaders and MMA issuers; warps 4..11: two softmax warpgroups
constexpr int kMaxSegs = 128;    // segments one launch can describe
constexpr int kFmaExpEvery = 0;            // 1 in this many exponentials is computed with FMAs (even; 0 = none)
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
#define EPD_W32(r, o) EPD_W16(r, o), EPD_W16(r, o + 16)
#define EPD_R64(r, o) EPD_R32(r, o), EPD_R32(r, o + 32)
#define EPD_W64(r, o) EPD_W32(r, o), EPD_W32(r, o + 32)

// tcgen05.ld / tcgen05.st, shape 32x32b: thread i of the warp owns TMEM lane (base + i) and moves
// N consecutive 32-bit columns.  One instruction per call; a wide form costs about the same issue
// time as a narrow one, so callers use the widest that fits.
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, uint32_t* r) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : EPD_R8(r, 0) : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : EPD_R16(r, 0) : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld32p(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : EPD_R32(r, 0) : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld64(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x64.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, "
      "%32, %33, %34, %35, %36, %37, %38, %39, %40, %41, %42, %43, %44, %45, %46, %47, "
      "%48, %49, %50, %51, %52, %53, %54, %55, %56, %57, %58, %59, %60, %61, %62, %63}, [%64];"
      : EPD_R64(r, 0) : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t* r) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
               ::"r"(taddr), EPD_W8(r, 0) : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), EPD_W16(r, 0) : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), EPD_W32(r, 0) : "memory");
}
__device__ __forceinline__ void tmem_st64(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x64.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32, "
      "%33, %34, %35, %36, %37, %38, %39, %40, %41, %42, %43, %44, %45, %46, %47, %48, "
      "%49, %50, %51, %52, %53, %54, %55, %56, %57, %58, %59, %60, %61, %62, %63, %64};"
      ::"r"(taddr), EPD_W64(r, 0) : "memory");
}
// N columns (a multiple of 8) with as few instructions as possible.
template <int N>
__device__ __forceinline__ void tmem_ld_cols(uint32_t taddr, uint32_t* r) {
  if constexpr (N >= 64) { tmem_ld64(taddr, r); tmem_ld_cols<N - 64>(taddr + 64, r + 64); }
  else if constexpr (N >= 32) { tmem_ld32p(taddr, r); tmem_ld_cols<N - 32>(taddr + 32, r + 32); }
  else if constexpr (N >= 16) { tmem_ld16(taddr, r); tmem_ld_cols<N - 16>(taddr + 16, r + 16); }
  else if constexpr (N >= 8) { tmem_ld8(taddr, r); tmem_ld_cols<N - 8>(taddr + 8, r + 8); }
}
template <int N>
__device__ __forceinline__ void tmem_st_cols(uint32_t taddr, const uint32_t* r) {
  if constexpr (N >= 64) { tmem_st64(taddr, r); tmem_st_cols<N - 64>(taddr + 64, r + 64); }
  else if constexpr (N >= 32) { tmem_st32(taddr, r); tmem_st_cols<N - 32>(taddr + 32, r + 32); }
  else if constexpr (N >= 16) { tmem_st16(taddr, r); tmem_st_cols<N - 16>(taddr + 16, r + 16); }
  else if constexpr (N >= 8) { tmem_st8(taddr, r); tmem_st_cols<N - 8>(taddr + 8, r + 8); }
}

__device__ __forceinline__ float max3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// 2^x for x <= 0 without the special-function unit: x = n + f with n integer and f in [-0.5, 0.5],
// 2^f from a cubic (relative error 1.2e-4, far below the bf16 rounding of P), and n added into the
// exponent field.
__device__ __forceinline__ float ex2_fma(float x) {
  x = fmaxf(x, -125.0f);
  const float t = x + 12582912.0f;     // 1.5 * 2^23: the sum's low mantissa bits hold round(x)
  const float f = x - (t - 12582912.0f);
  float p = 0.05459282547235489f;
  p = fmaf(p, f, 0.24221783876419067f);
  p = fmaf(p, f, 0.6933686137199402f);
  p = fmaf(p, f, 1.0f);
  return __int_as_float(__float_as_int(p) + (__float_as_int(t) << 23));
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
  static constexpr int BKV = DHP == 80 ? 112 : DHP == 128 ? 80 : 128;   // keys per tile
  static constexpr int kPCols = (BKV / 2 + 15) / 16 * 16;              // TMEM columns reserved for P_w
  static constexpr int kS0 = 0, kP0 = BKV, kS1 = BKV + kPCols, kP1 = kS1 + BKV;
  static constexpr int kO0 = 2 * (BKV + kPCols), kO1 = kO0 + DHP;
  static_assert(kO1 + DHP <= 512, "tensor memory plan does not fit");
  static constexpr int kMainBoxes = DHP / 64;          // Q, K: 128-byte-swizzled boxes of 64 columns
  static constexpr int kTail = DHP % 64;               // Q, K: 0 or 16 columns, 32-byte swizzle
  static_assert(kTail == 0 || kTail == 16, "padded head width must be 64*a or 64*a + 16");
  static constexpr bool kV32 = kTail != 0;             // V as 32-byte-swizzled boxes of 16 columns
  static constexpr int kQMain = BQ * 128, kQTail = kTail ? BQ * 32 : 0;
  static constexpr int kQBytes = kMainBoxes * kQMain + kQTail;
  static constexpr int kKMain = BKV * 128, kKTail = kTail ? BKV * 32 : 0;
  static constexpr int kKBytes = kMainBoxes * kKMain + kKTail;          // bytes TMA writes per K (or V) tile
  static constexpr int kKStride = (kKBytes + 1023) / 1024 * 1024;       // ring slot pitch (1024-byte aligned)
  static constexpr int kVBox = kV32 ? BKV * 32 : BKV * 128;             // one V box
  static constexpr int kVBoxes = kV32 ? DHP / 16 : DHP / 64;
  static_assert(kVBox * kVBoxes == kKBytes, "K and V tiles have the same size");
  static constexpr int KS = DHP == 128 ? 3 : 4;        // K ring depth
  static constexpr int VS = DHP == 128 ? 3 : 4;        // V ring depth
  static constexpr int kQ = 0;                         // two Q buffers
  static constexpr int kK = 2 * kQBytes;
  static constexpr int kV = kK + KS * kKStride;
  static constexpr int kMl = kV + VS * kKStride;       // (m, l) of both warpgroups, by item parity: float2[2][2][128]
  static constexpr int kBar = kMl + 4 * BQ * 8;
  // q_full[2] q_empty[2] k_full[KS] k_empty[KS] v_full[VS] v_empty[VS] s_full[2] s_free[2] p_full[2] p_free[2]
  // o_done[2] o_free[2] ml_pub[2] drain[2]
  static constexpr int kNumBars = 4 + 2 * KS + 2 * VS + 16;
  static constexpr int kTotal = kBar + kNumBars * 8 + 32;
  static constexpr int kDynamic = kTotal + 1024;       // slack to align the tiles to 1024 bytes
  static_assert(kQBytes % 1024 == 0, "Q buffers keep the rings 1024-byte aligned");
  static_assert(kDynamic > 116 * 1024, "one CTA per SM is assumed by the TMEM allocation");
  static_assert(kDynamic <= 232448, "exceeds the shared memory of one CTA");
  static constexpr int kOChunks = DHP / 16;            // 16-column pieces of an O accumulator
  static constexpr int kSChunks = BKV / 16;            // 16-column pieces of a score row
};

struct Maps {
  CUtensorMap q_main, q_tail, k_main, k_tail, v;
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
};

// Item i -> (segment, head, query tile): segments in list order, then head, then query tile, so
// that neighbouring items (which run at the same time on different SMs) share K and V in L2.
// A CTA's items come in ascending order: `seg` is the caller's cursor into the segment list (0 before its first item).
template <int BKV>
__device__ __forceinline__ Item decode_item(const SegList& segs, int i, int& seg) {
  while (seg + 1 < segs.n && i >= segs.first[seg + 1]) ++seg;
  Item it;
  it.seg_beg = segs.beg[seg];
  it.seg_len = segs.len[seg];
  const int qt = (it.seg_len + BQ - 1) / BQ;
  i -= segs.first[seg];
  it.head = i / qt;
  it.q0 = it.seg_beg + (i - it.head * qt) * BQ;
  it.n_kv = (it.seg_len + BKV - 1) / BKV;
  return it;
}

// Epilogue of one query row: columns [col0, col0 + N) of (f0 O0 + f1 O1) as bf16, 16 bytes per store.
// buf holds 2 MAXB registers; N columns are done in batches of at most MAXB.
template <int N, int MAXB>
__device__ __forceinline__ void write_output_cols(uint32_t tmem_o0, uint32_t tmem_o1, int col0, bool has1, bool row_ok,
                                                  float f0, float f1, int dh, __nv_bfloat16* orow, uint32_t* buf) {
  if constexpr (N > MAXB) {
    write_output_cols<MAXB, MAXB>(tmem_o0, tmem_o1, col0, has1, row_ok, f0, f1, dh, orow, buf);
    write_output_cols<N - MAXB, MAXB>(tmem_o0, tmem_o1, col0 + MAXB, has1, row_ok, f0, f1, dh, orow, buf);
    return;
  }
  tmem_ld_cols<N>(tmem_o0 + col0, buf);
  if (has1) tmem_ld_cols<N>(tmem_o1 + col0, buf + N);
  tmem_ld_wait();
  if (row_ok) {
#pragma unroll
    for (int g = 0; g < N / 8; ++g) {
      if (col0 + g * 8 < dh) {  // dh is a multiple of 8
        uint32_t pk[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          float v0 = __uint_as_float(buf[8 * g + 2 * e]) * f0, v1 = __uint_as_float(buf[8 * g + 2 * e + 1]) * f0;
          if (has1) {
            v0 = fmaf(__uint_as_float(buf[N + 8 * g + 2 * e]), f1, v0);
            v1 = fmaf(__uint_as_float(buf[N + 8 * g + 2 * e + 1]), f1, v1);
          }
          __nv_bfloat162 b = __floats2bfloat162_rn(v0, v1);
          pk[e] = *reinterpret_cast<uint32_t*>(&b);
        }
        *reinterpret_cast<uint4*>(orow + col0 + g * 8) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
      }
    }
  }
}

// Key tile j of an item goes to warpgroup (j & 1) ^ fw.  The warpgroup that owns the last key tile merges
// the item; the other one is free earlier, so it takes the first key tile of the next item.
__device__ __forceinline__ int merging_warpgroup(int fw, int n_kv) { return ((n_kv - 1) & 1) ^ fw; }
__device__ __forceinline__ int next_first_warpgroup(int fw, int n_kv) { return merging_warpgroup(fw, n_kv) ^ 1; }

// Order in which the two issuing threads walk an item's key tiles: 0, 2, 1, 4, 3, 6, 5, ... for items of
// at most 32 key tiles (and rings of four tiles), 0, 1, 2, ... otherwise.
// The warpgroup that takes tile 0 is the one that did not merge the previous item; giving it its first
// tiles one step early lets it work through three of them while the other warpgroup is still merging
// (with the plain order 0, 1, 2, ... it stalls after one, behind the first product the merging
// warpgroup is not ready for).  Each warpgroup still sees its own tiles in ascending order.  Measured:
// 8 x 784 tokens 378 -> 393 TFLOP/s, 16 x 1024 tokens 456 -> 471; a 16384-token segment, where item
// boundaries are rare, lost 1 % in that order and keeps the plain one.  It needs K and V rings of four
// tiles: with three (head width 128) taking tile 2 before tile 1 leaves the loaders no slack (16 x 1024
// tokens, 25 heads x 128: 788 -> 655 TFLOP/s), so those keep the plain order too.
__device__ __forceinline__ int issue_order(int i, int n_kv, bool deep_rings) {
  if (i == 0 || n_kv > 32 || !deep_rings) return i;
  const int j = (i & 1) ? i + 1 : i - 1;
  return j < n_kv ? j : i;
}

// ONES: head_dim < DHP and column head_dim of every V row holds 1.0, so column head_dim of O_w is the
// row sum of P_w (summed by the tensor core from the same bf16 values as the numerator) and the
// softmax threads need not add it up.
template <int DHP, bool ONES>
__global__ void __launch_bounds__(kThreads, 1)
attention_tc_kernel(const __grid_constant__ Maps maps, const __grid_constant__ SegList segs, int n_items,
                    __nv_bfloat16* __restrict__ out, int T, int heads, int dh, int* __restrict__ status,
                    long long wait_limit) {
  using P = Plan<DHP>;
  constexpr int BKV = P::BKV;
  pdl_launch_dependents();
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + P::kBar);
  uint64_t* q_full = bars;                    // [2]
  uint64_t* q_empty = bars + 2;               // [2]
  uint64_t* k_full = bars + 4;                // [KS]
  uint64_t* k_empty = k_full + P::KS;         // [KS]
  uint64_t* v_full = k_empty + P::KS;         // [VS]
  uint64_t* v_empty = v_full + P::VS;         // [VS]
  uint64_t* s_full = v_empty + P::VS;         // [2]  S_w complete
  uint64_t* s_free = s_full + 2;              // [2]  S_w copied to registers (4 warp arrivals)
  uint64_t* p_full = s_free + 2;              // [2]  P_w written (4 warp arrivals)
  uint64_t* p_free = p_full + 2;              // [2]  P_w consumed: the warpgroup's last P V is complete
  uint64_t* o_done = p_free + 2;              // [2]  warpgroup w's P V products of the item complete: O_w final
  uint64_t* o_free = o_done + 2;              // [2]  O_w read out by the merging warpgroup (4 warp arrivals)
  uint64_t* ml_pub = o_free + 2;              // [2]  warpgroup w published its (m, l) of the item (4 warp arrivals)
  uint64_t* drain = ml_pub + 2;               // [2]  after an abort: the MMAs of issuing thread 0 / 1 have completed
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + P::kNumBars);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const WaitCtx wc{abort_flag, 0u, wait_limit};
  uint32_t q_loads = 0, kv_loads = 0;         // loads issued by this thread (warp 0: Q and K tiles, warp 3: V tiles)
  float2* ml_all = reinterpret_cast<float2*>(smem + P::kMl);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int i = 0; i < P::kNumBars; ++i) mbar_init(&bars[i], 1);
    for (int w = 0; w < 2; ++w) { mbar_init(&s_free[w], 4); mbar_init(&p_full[w], 4); }
    for (int w = 0; w < 2; ++w) { mbar_init(&o_free[w], 4); mbar_init(&ml_pub[w], 4); }
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

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer of Q and K
    if (lane == 0) {
      uint32_t kc = 0, n = 0;
      bool ok = true;
      int seg_cur = 0;
      for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++n) {
        const Item it = decode_item<BKV>(segs, item, seg_cur);
        const int row_base = it.head * T;
        const int qb = n & 1;
        if (!mbar_wait(&q_empty[qb], ((n >> 1) & 1) ^ 1, wc)) break;
        {
          uint8_t* dst = smem + P::kQ + qb * P::kQBytes;
          mbar_expect_tx(&q_full[qb], P::kQBytes);
#pragma unroll
          for (int b = 0; b < P::kMainBoxes; ++b)
            tma_load_2d(dst + b * P::kQMain, &maps.q_main, b * 64, row_base + it.q0, &q_full[qb]);
          if (P::kTail)
            tma_load_2d(dst + P::kMainBoxes * P::kQMain, &maps.q_tail, P::kMainBoxes * 64, row_base + it.q0, &q_full[qb]);
          ++q_loads;
        }
        for (int j = 0; j < it.n_kv; ++j, ++kc) {
          const int row = row_base + it.seg_beg + j * BKV;
          const int ks = kc % P::KS;
          if (!mbar_wait(&k_empty[ks], ((kc / P::KS) & 1) ^ 1, wc)) { ok = false; break; }
          uint8_t* dk = smem + P::kK + ks * P::kKStride;
          mbar_expect_tx(&k_full[ks], P::kKBytes);
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
        const Item it = decode_item<BKV>(segs, item, seg_cur);
        const int row_base = it.head * T;
        for (int j = 0; j < it.n_kv; ++j, ++vc) {
          const int row = row_base + it.seg_beg + j * BKV;
          const int vs = vc % P::VS;
          if (!mbar_wait(&v_empty[vs], ((vc / P::VS) & 1) ^ 1, wc)) { ok = false; break; }
          uint8_t* dv = smem + P::kV + vs * P::kKStride;
          mbar_expect_tx(&v_full[vs], P::kKBytes);
#pragma unroll
          for (int b = 0; b < P::kVBoxes; ++b)
            tma_load_2d(dv + b * P::kVBox, &maps.v, b * (P::kV32 ? 16 : 64), row, &v_full[vs]);
          ++kv_loads;
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ---------------------------------------------------------------- Q K^T issuer:  S_w(j) = Q K_j^T
    // The whole warp walks the loop and one elected lane issues (see elect_one()).
    {
      uint32_t kc = 0, n = 0, sc0 = 0, sc1 = 0;        // sc_w: score tiles issued for warpgroup w
      int fw = 0;                                      // warpgroup that takes the item's first key tile
      bool ok = true;
      int seg_cur = 0;
      for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++n) {
        const Item it = decode_item<BKV>(segs, item, seg_cur);
        const int qb = n & 1;
        if (!mbar_wait_warp(&q_full[qb], (n >> 1) & 1, wc)) break;
        const uint32_t sq = smem_u32(smem + P::kQ + qb * P::kQBytes);
        const uint64_t dq_main = smem_desc(sq, 16, 1024, 2);
        const uint64_t dq_tail = smem_desc(sq + P::kMainBoxes * P::kQMain, 16, 256, 6);
        for (int i = 0; i < it.n_kv; ++i) {
          const int j = issue_order(i, it.n_kv, P::KS >= 4 && P::VS >= 4);
          const uint32_t kt = kc + j;                   // the tile's number in the K ring
          const int w = (j & 1) ^ fw;
          const int ks = kt % P::KS;
          if (!mbar_wait_warp(&k_full[ks], (kt / P::KS) & 1, wc)) { ok = false; break; }
          uint32_t& sc = w ? sc1 : sc0;
          // the warpgroup must have copied its previous score tile out of S_w
          if (sc > 0 && !mbar_wait_warp(&s_free[w], (sc - 1) & 1, wc)) { ok = false; break; }
          ++sc;
          tc_fence_after();
          const uint32_t sk = smem_u32(smem + P::kK + ks * P::kKStride);
          const uint64_t dk_main = smem_desc(sk, 16, 1024, 2);
          const uint64_t dk_tail = smem_desc(sk + P::kMainBoxes * P::kKMain, 16, 256, 6);
          const uint32_t tmem_s = tmem_base + (w ? P::kS1 : P::kS0);
          const int kv_valid = min(BKV, it.seg_len - j * BKV);
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
            umma_commit(&s_full[w]);
            umma_commit(&k_empty[ks]);
            if (i == it.n_kv - 1) umma_commit(&q_empty[qb]);
          }
          __syncwarp();
        }
        kc += it.n_kv;
        fw = next_first_warpgroup(fw, it.n_kv);
      }
    }
    __syncwarp();
  } else if (warp == 2) {
    // ---------------------------------------------------------------- P V issuer:  O_w += P_w(j) V_j
    // The whole warp walks the loop and one elected lane issues.
    {
      uint32_t vc = 0, n = 0, pc0 = 0, pc1 = 0;        // pc_w: P tiles consumed for warpgroup w
      uint32_t items0 = 0, items1 = 0;                 // items in which warpgroup 0 / 1 had key tiles
      int fw = 0;
      constexpr uint32_t idesc = instr_desc(DHP, 1);
      constexpr uint32_t kStep = P::kV32 ? 512 / 16 : 2048 / 16;   // 16 keys further down the V tile, 16-byte units
      bool ok = true;
      int seg_cur = 0;
      for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++n) {
        const Item it = decode_item<BKV>(segs, item, seg_cur);
        for (int i = 0; i < it.n_kv; ++i) {
          const int j = issue_order(i, it.n_kv, P::KS >= 4 && P::VS >= 4);
          const uint32_t vt = vc + j;                   // the tile's number in the V ring
          const int w = (j & 1) ^ fw;
          const int vs = vt % P::VS;
          uint32_t& pc = w ? pc1 : pc0;
          // V arrives long before P: take that wait first so that only P's is on the critical path
          if (!mbar_wait_warp(&v_full[vs], (vt / P::VS) & 1, wc)) { ok = false; break; }
          if (!mbar_wait_warp(&p_full[w], pc & 1, wc)) { ok = false; break; }
          ++pc;
          if (j < 2) {
            // the warpgroup's accumulator of its previous item must have been read out before it is overwritten
            uint32_t& items = w ? items1 : items0;
            if (items > 0 && !mbar_wait_warp(&o_free[w], (items - 1) & 1, wc)) { ok = false; break; }
            ++items;
          }
          tc_fence_after();
          const uint32_t sv = smem_u32(smem + P::kV + vs * P::kKStride);
          // MN-major V: boxes (16 or 64 columns wide) are kVBox apart, 8-row groups 256 / 1024 bytes apart
          const uint64_t dv = P::kV32 ? smem_desc(sv, P::kVBox, 256, 6) : smem_desc(sv, P::kVBox, 1024, 2);
          const uint32_t tmem_p = tmem_base + (w ? P::kP1 : P::kP0), tmem_o = tmem_base + (w ? P::kO1 : P::kO0);
          const uint32_t first = j >= 2 ? 1u : 0u;     // a warpgroup's first tile starts O_w afresh
          const int kv_valid = min(BKV, it.seg_len - j * BKV);
          if (elect_one()) {
            if (kv_valid == BKV) {
#pragma unroll
              for (int ks = 0; ks < BKV / 16; ++ks)       // 16 bf16 of P = 8 columns
                umma_ts(tmem_o, tmem_p + ks * 8, dv + ks * kStep, idesc, ks == 0 ? first : 1u);
            } else {
              const int steps = (kv_valid + 15) >> 4;
              for (int ks = 0; ks < steps; ++ks)
                umma_ts(tmem_o, tmem_p + ks * 8, dv + ks * kStep, idesc, ks == 0 ? first : 1u);
            }
            umma_commit(&v_empty[vs]);
            umma_commit(&p_free[w]);
            if (j >= it.n_kv - 2) umma_commit(&o_done[w]);   // the warpgroup's last key tile of the item
          }
          __syncwarp();
        }
        if (!ok) break;
        vc += it.n_kv;
        fw = next_first_warpgroup(fw, it.n_kv);
      }
    }
    __syncwarp();
  } else if (warp >= 4) {
    // ---------------------------------------------------------------- softmax / rescale / merge / epilogue
    const int w = (warp - 4) >> 2;                      // warpgroup; takes key tiles of parity w ^ (item count & 1)
    const int qr = warp & 3;                            // TMEM lane quarter this warp may access
    const int r = qr * 32 + lane;                       // query row inside the tile
    const uint32_t lane_off = (uint32_t)(qr * 32) << 16;
    const uint32_t tmem_s = tmem_base + (w ? P::kS1 : P::kS0) + lane_off;
    const uint32_t tmem_p = tmem_base + (w ? P::kP1 : P::kP0) + lane_off;
    const uint32_t tmem_o = tmem_base + (w ? P::kO1 : P::kO0) + lane_off;
    uint32_t tc = 0, n = 0;                             // score tiles processed, items processed
    uint32_t items_me = 0, items_other = 0;             // items in which this / the other warpgroup had key tiles
    uint32_t pubs_me = 0, pubs_other = 0;               // (m, l) publications of this / the other warpgroup
    int fw = 0;                                         // warpgroup that takes the item's first key tile
    bool ok = true;
    int seg_cur = 0;
    for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x, ++n) {
      const Item it = decode_item<BKV>(segs, item, seg_cur);
      float m = -INFINITY, l = 0.0f;
      uint32_t s[BKV];
      // The loop is software-pipelined: the tcgen05.ld of the next score tile is issued right after
      // the tcgen05.st of this tile's P, so the two TMEM round trips overlap.
      auto load_scores = [&](int j) -> bool {
        const int kv_valid = min(BKV, it.seg_len - j * BKV);
        if (!mbar_wait_warp(&s_full[w], tc & 1, wc)) return false;
        tc_fence_after();
        if (kv_valid == BKV) {
          tmem_ld_cols<BKV>(tmem_s, s);
        } else {
#pragma unroll
          for (int c = 0; c < P::kSChunks; ++c)
            if (c * 16 < kv_valid) tmem_ld16(tmem_s + c * 16, s + c * 16);
        }
        return true;
      };
      // The warpgroup that owns the item's last key tile merges the item and writes its rows.  The other
      // one does not wait: it publishes (m, l) and goes on to the next item, whose first key tile is
      // given to it.  With an odd number of key tiles (7 for a 784-token image) the extra tile and the
      // merge thus alternate between the warpgroups.
      const int j0 = w ^ fw;                            // this warpgroup's first key tile of the item
      const int merging = merging_warpgroup(fw, it.n_kv);
      const bool has_other = it.n_kv > 1;               // the other warpgroup has key tiles too
      // state of both warpgroups after this item (every path below leaves the item with it)
      const uint32_t my_items = items_me + (j0 < it.n_kv ? 1u : 0u);   // counts this item
      const uint32_t other_items = items_other + ((j0 ^ 1) < it.n_kv ? 1u : 0u);
      const uint32_t other_pubs = pubs_other;           // publications before this item
      const uint32_t my_pubs = pubs_me;
      items_me = my_items;
      items_other = other_items;
      if (has_other) { if (merging == w) ++pubs_other; else ++pubs_me; }
      fw = merging ^ 1;
      if (j0 < it.n_kv && !load_scores(j0)) { ok = false; break; }
      for (int j = j0; j < it.n_kv; j += 2) {
        const int kv_valid = min(BKV, it.seg_len - j * BKV);
        tmem_ld_wait();
        // S_w may be overwritten by the next score tile from here on
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&s_free[w]);

        float mx[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) mx[i] = -INFINITY;
        if (kv_valid == BKV) {
#pragma unroll
          for (int i = 0; i < BKV / 2; ++i)
            mx[i & 7] = max3(mx[i & 7], __uint_as_float(s[2 * i]), __uint_as_float(s[2 * i + 1]));
        } else {
#pragma unroll
          for (int i = 0; i < BKV; ++i)
            if (i < kv_valid) mx[i & 7] = fmaxf(mx[i & 7], __uint_as_float(s[i]));
        }
        const float m_tile = fmaxf(fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])),
                                   fmaxf(fmaxf(mx[4], mx[5]), fmaxf(mx[6], mx[7])));
        // advance the running max only when it would grow by more than the threshold
        float scale = 1.0f;
        bool grow = false;
        if (j == j0) {
          m = m_tile;
        } else if (m_tile - m > kRescaleThreshold) {
          scale = ex2(m - m_tile);
          m = m_tile;
          l *= scale;
          grow = true;
        }
        // P = exp2(S - m) as bf16 pairs
        const float neg_m = -m;
        float sum[4] = {0.0f, 0.0f, 0.0f, 0.0f};
        if (kv_valid == BKV) {
#pragma unroll
          for (int i = 0; i < BKV / 2; ++i) {
            // one exponential in kFmaExpEvery goes to the FMA pipe
            const float p0 = ex2(__uint_as_float(s[2 * i]) + neg_m);
            const float p1 = (kFmaExpEvery > 0 && i % (kFmaExpEvery > 0 ? kFmaExpEvery / 2 : 1) == kFmaExpEvery / 2 - 1)
                                 ? ex2_fma(__uint_as_float(s[2 * i + 1]) + neg_m)
                                 : ex2(__uint_as_float(s[2 * i + 1]) + neg_m);
            if (!ONES) sum[i & 3] += p0 + p1;
            __nv_bfloat162 b = __floats2bfloat162_rn(p0, p1);
            s[i] = *reinterpret_cast<uint32_t*>(&b);
          }
        } else {
#pragma unroll
          for (int i = 0; i < BKV / 2; ++i) {
            const float p0 = 2 * i < kv_valid ? ex2(__uint_as_float(s[2 * i]) + neg_m) : 0.0f;
            const float p1 = 2 * i + 1 < kv_valid ? ex2(__uint_as_float(s[2 * i + 1]) + neg_m) : 0.0f;
            if (!ONES) sum[i & 3] += p0 + p1;
            __nv_bfloat162 b = __floats2bfloat162_rn(p0, p1);
            s[i] = *reinterpret_cast<uint32_t*>(&b);
          }
        }
        if (!ONES) l += (sum[0] + sum[1]) + (sum[2] + sum[3]);
        // P_w and O_w are free once this warpgroup's previous P V has completed
        if (tc > 0 && !mbar_wait_warp(&p_free[w], (tc - 1) & 1, wc)) { ok = false; break; }
        ++tc;
        tc_fence_after();
        if (__any_sync(0xffffffffu, grow)) {
#pragma unroll
          for (int c = 0; c < P::kOChunks; ++c) {
            uint32_t o[16];
            tmem_ld16(tmem_o + c * 16, o);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 16; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * scale);
            tmem_st16(tmem_o + c * 16, o);
          }
        }
        // 8 packed columns hold 16 keys; a store reads its registers when it is issued
        if (kv_valid == BKV) {
          tmem_st_cols<BKV / 2>(tmem_p, s);
        } else {
#pragma unroll
          for (int c = 0; c < P::kSChunks; ++c)
            if (c * 16 < kv_valid) tmem_st8(tmem_p + c * 8, s + c * 8);
        }
        if (j + 2 < it.n_kv && !load_scores(j + 2)) { ok = false; break; }
        tmem_st_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&p_full[w]);
      }
      if (!ok) break;
      if (w != merging) {
        if (j0 >= it.n_kv) continue;                    // no key tile in this item: nothing to hand over
        // Publish (m, l) and go on.  The slot (double-buffered by item parity) and the barrier phase must
        // not overtake the reader of this warpgroup's previous publication: that reader has finished once
        // O_w of this warpgroup's previous item with key tiles was read out (with two or more key tiles
        // in this item that is already known through the P V products).
        if (my_pubs > 0 && my_items >= 2 && !mbar_wait_warp(&o_free[w], (my_items - 2) & 1, wc)) { ok = false; break; }
        ml_all[(n & 1) * 2 * BQ + w * BQ + r] = make_float2(m, l);
        __syncwarp();
        if (lane == 0) mbar_arrive(&ml_pub[w]);
        continue;
      }
      // ---- merge: "a" is this warpgroup's accumulator, "b" the other's
      const uint32_t tmem_oa = tmem_base + (w ? P::kO1 : P::kO0) + lane_off;
      const uint32_t tmem_ob = tmem_base + (w ? P::kO0 : P::kO1) + lane_off;
      float2 ml_a = make_float2(m, l), ml_b = make_float2(-INFINITY, 0.0f);
      // O_b fits the dead score registers next to a 32-column batch of O_a: read it first and hand the
      // accumulator back, so that the other warpgroup's next item is not held up by this merge
      constexpr bool kEarly = DHP + 32 <= BKV;
      if (has_other) {
        if (!mbar_wait_warp(&ml_pub[w ^ 1], other_pubs & 1, wc)) { ok = false; break; }
        if (!mbar_wait_warp(&o_done[w ^ 1], (other_items - 1) & 1, wc)) { ok = false; break; }
        tc_fence_after();
        ml_b = ml_all[(n & 1) * 2 * BQ + (w ^ 1) * BQ + r];
        if constexpr (kEarly) {
          tmem_ld_cols<DHP>(tmem_ob, s);
          tmem_ld_wait();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&o_free[w ^ 1]);
          // with a ones column head_dim is DHP - 8 (a multiple of 8 just below the padded width): the row
          // sum sits in column DHP - 8
          if (ONES) ml_b.y = __uint_as_float(s[DHP - 8]);
        } else if (ONES) {
          uint32_t t1[8];
          tmem_ld8(tmem_ob + (dh & ~7), t1);            // the row sum sits in column head_dim
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 8; ++i)
            if (i == (dh & 7)) ml_b.y = __uint_as_float(t1[i]);
        }
      }
      if (!mbar_wait_warp(&o_done[w], (my_items - 1) & 1, wc)) { ok = false; break; }
      tc_fence_after();
      const int token = it.q0 + r;
      const bool row_ok = token < it.seg_beg + it.seg_len;
      __nv_bfloat16* orow = out + (int64_t)token * (heads * dh) + it.head * dh;
      if constexpr (kEarly) {
        // O_a in batches of at most 32 columns behind O_b in the score registers, the last batch first:
        // it holds the row sum the factors need
        uint32_t* oa = s + DHP;
        constexpr int kLast = (DHP - 1) / 32 * 32;       // first column of the last batch
        float fa = 0.0f, fb = 0.0f;
#pragma unroll
        for (int b = 0; b < (DHP + 31) / 32; ++b) {
          const int c0 = b == 0 ? kLast : (b - 1) * 32;
          if (b == 0) tmem_ld_cols<DHP - kLast>(tmem_oa + kLast, oa);
          else tmem_ld_cols<32>(tmem_oa + c0, oa);
          tmem_ld_wait();
          if (b == (DHP + 31) / 32 - 1) {
            // O_a is in registers: the accumulator may be overwritten by this warpgroup's next item
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&o_free[w]);
          }
          if (b == 0) {
            if (ONES) ml_a.y = __uint_as_float(oa[DHP - 8 - kLast]);
            const float mm = fmaxf(ml_a.x, ml_b.x);
            const float ea = ex2(ml_a.x - mm), eb = has_other ? ex2(ml_b.x - mm) : 0.0f;
            const float inv = 1.0f / (ea * ml_a.y + eb * ml_b.y);
            fa = ea * inv;
            fb = eb * inv;
          }
          if (row_ok) {
#pragma unroll
            for (int g = 0; g < 4; ++g) {
              if (c0 + g * 8 < DHP && c0 + g * 8 < dh) {   // dh is a multiple of 8
                uint32_t pk[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                  float v0 = __uint_as_float(oa[8 * g + 2 * e]) * fa, v1 = __uint_as_float(oa[8 * g + 2 * e + 1]) * fa;
                  if (has_other) {
                    v0 = fmaf(__uint_as_float(s[c0 + 8 * g + 2 * e]), fb, v0);
                    v1 = fmaf(__uint_as_float(s[c0 + 8 * g + 2 * e + 1]), fb, v1);
                  }
                  __nv_bfloat162 b2 = __floats2bfloat162_rn(v0, v1);
                  pk[e] = *reinterpret_cast<uint32_t*>(&b2);
                }
                *reinterpret_cast<uint4*>(orow + c0 + g * 8) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
              }
            }
          }
        }
      } else {
        // both accumulators in batches through the score registers; handed back at the end
        if (ONES) {
          uint32_t t0[8];
          tmem_ld8(tmem_oa + (dh & ~7), t0);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 8; ++i)
            if (i == (dh & 7)) ml_a.y = __uint_as_float(t0[i]);
        }
        const float mm = fmaxf(ml_a.x, ml_b.x);
        const float ea = ex2(ml_a.x - mm), eb = has_other ? ex2(ml_b.x - mm) : 0.0f;
        const float inv = 1.0f / (ea * ml_a.y + eb * ml_b.y);
        const float fa = ea * inv, fb = eb * inv;
        constexpr int kMaxB = BKV / 2 / 16 * 16;   // columns of each accumulator that fit the score registers
        write_output_cols<DHP, kMaxB>(tmem_oa, tmem_ob, 0, has_other, row_ok, fa, fb, dh, orow, s);
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(&o_free[w]);
          if (has_other) mbar_arrive(&o_free[w ^ 1]);
        }
      }
    }
  }

  // ---------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    // A wait expired.  Every role has left its loop, so nothing new is issued.  What was issued completes by
    // itself: each loader waits for its last load of every ring slot, each issuing thread for its last MMA (a
    // commit arrives only after all earlier MMAs); the softmax warps write their rows with ordinary stores.  A
    // fixed pause on top, then shared and tensor memory are released.
    if (threadIdx.x == 0 && status != nullptr) atomicCAS(status, 0, kStatusTimeout);
    if (lane == 0) {
      if (warp == 0) { drain_ring(q_full, 2, q_loads); drain_ring(k_full, P::KS, kv_loads); }
      if (warp == 3) drain_ring(v_full, P::VS, kv_loads);
    }
    if ((warp == 1 || warp == 2) && elect_one()) {   // the lane that issued the products: a commit covers its own thread's
      umma_commit(&drain[warp - 1]);
      mbar_wait_drain(&drain[warp - 1], 0);
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
bool make_map(CUtensorMap* tm, const void* base, int64_t rows, int dhp, int box_cols, int box_rows,
              CUtensorMapSwizzle swz) {
  return make_tensor_map_2d(tm, base, rows, dhp, (int64_t)dhp * 2, box_rows, box_cols, 2, swz);
}

template <int DHP, bool ONES>
cudaError_t launch(const Maps& maps, const SegList& segs, int n_items, void* out, int T, int heads, int dh,
                   int* status, cudaStream_t s) {
  using P = Plan<DHP>;
  auto kern = attention_tc_kernel<DHP, ONES>;
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

bool attention_tc_supported(const void* q, const void* k, const void* v, const void* out, int64_t T, int heads,
                            int head_dim) {
  const int dhp = padded_head_dim(head_dim);
  if (dhp != 64 && dhp != 80 && dhp != 128) return false;
  if (head_dim % 8) return false;
  if (((uintptr_t)q & 15) || ((uintptr_t)k & 15) || ((uintptr_t)v & 15) || ((uintptr_t)out & 15)) return false;
  if ((int64_t)heads * T > (1 << 30) || heads > 65535) return false;
  return tensor_maps_available();
}

cudaError_t attention_tc(const void* q, const void* k, const void* v, const int32_t* host_cu_seqlens, int n_seg,
                         void* out, int64_t T, int heads, int head_dim, int* status, cudaStream_t s) {
  const int dhp = padded_head_dim(head_dim);
  if (n_seg <= 0) return cudaSuccess;
  const int64_t rows = (int64_t)heads * T;
  Maps maps;
  const int bkv = dhp == 80 ? Plan<80>::BKV : dhp == 128 ? Plan<128>::BKV : Plan<64>::BKV;
  if (!make_map(&maps.q_main, q, rows, dhp, 64, BQ, CU_TENSOR_MAP_SWIZZLE_128B) ||
      !make_map(&maps.q_tail, q, rows, dhp, 16, BQ, CU_TENSOR_MAP_SWIZZLE_32B) ||
      !make_map(&maps.k_main, k, rows, dhp, 64, bkv, CU_TENSOR_MAP_SWIZZLE_128B) ||
      !make_map(&maps.k_tail, k, rows, dhp, 16, bkv, CU_TENSOR_MAP_SWIZZLE_32B))
    return cudaErrorInvalidValue;
  if (dhp % 64 ? !make_map(&maps.v, v, rows, dhp, 16, bkv, CU_TENSOR_MAP_SWIZZLE_32B)
               : !make_map(&maps.v, v, rows, dhp, 64, bkv, CU_TENSOR_MAP_SWIZZLE_128B))
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
      n_items += (segs.len[i] + BQ - 1) / BQ * heads;
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

}  // namespace

cudaError_t attention_any(int dtype, const void* q, const void* k, const void* v, const int32_t* cu_seqlens,
                          const int32_t* host_cu_seqlens, int n_seg, void* out, int64_t T, int heads, int head_dim,
                          int flags, int* status, cudaStream_t s) {
  if (dtype == EPD_DTYPE_BF16 && !(flags & EPD_ATTENTION_FORCE_FMA)) {
    // Two tensor-core kernels.  Measured on B200 in one run (TFLOP/s, two-query-tile kernel / split-keys kernel), head
    // width 72: 16 x 1024 tokens 593 / 452, ten segments of 840..5208 tokens 686 / 633, a 16384-token segment plus
    // 8 x 784 tokens 749 / 718, mixed lengths 196..7056 678 / 662, 8 x 784 tokens 336 / 356; head width 128, 16 x 1024
    // tokens 953 / 700.  The two-query-tile kernel is the default wherever it applies.  The choice depends on the head
    // width only, never on what else is in the batch: an item's features must not change with the company it is
    // encoded in.
    const bool forced_pair = flags & EPD_ATTENTION_TWO_QUERY_TILES;
    const bool prefer_pair = true;
    if ((forced_pair || (prefer_pair && !(flags & EPD_ATTENTION_SPLIT_KEYS))) &&
        attention_pair_supported(q, k, v, out, T, heads, head_dim))
      return attention_pair(q, k, v, host_cu_seqlens, n_seg, out, T, heads, head_dim, status, s);
    if (attention_tc_supported(q, k, v, out, T, heads, head_dim))
      return attention_tc(q, k, v, host_cu_seqlens, n_seg, out, T, heads, head_dim, status, s);
  }
  return attention_fma(dtype, q, k, v, cu_seqlens, n_seg, out, T, heads, head_dim, s);
}

}  // namespace epd
