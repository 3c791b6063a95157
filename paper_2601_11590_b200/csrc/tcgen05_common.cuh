// What the tcgen05 kernels of this library share: PTX wrappers (mbarrier, TMA, tensor memory, MMA commit),
// the bounded wait with its abort / drain protocol, and the host helpers (tensor maps, per-device launch set-up).
#pragma once

#include <cuda.h>

#include <atomic>

#include "common.cuh"

namespace epd {

// ---------------------------------------------------------------------------------------------
// Host helpers (tcgen05_host.cu)
// ---------------------------------------------------------------------------------------------

// Row-major 2-D tensor map over [rows, cols] elements of elem_bytes (2 = bf16, 4 = float, 1 = byte) with
// row pitch pitch_bytes; box = box_rows x box_cols elements.  False if the driver entry point is missing or
// the encoding is rejected.
bool make_tensor_map_2d(CUtensorMap* tm, const void* base, int64_t rows, int64_t cols, int64_t pitch_bytes,
                        int box_rows, int box_cols, int elem_bytes, CUtensorMapSwizzle swizzle);
bool tensor_maps_available();

// SM count of the current device (cached per device ordinal).
int device_sm_count();

// Cycle limit of the kernels' bounded waits (default ~2 s at 2 GHz; epd_debug_set_wait_limit changes it).
long long wait_limit_cycles();

// Work that must happen once per device (a function attribute, an occupancy query): a bit per device ordinal.
struct PerDeviceOnce {
  std::atomic<uint64_t> done{0};
};
template <typename F>
inline cudaError_t once_per_device(PerDeviceOnce& o, F&& f) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const uint64_t bit = dev >= 0 && dev < 64 ? (uint64_t)1 << dev : 0;   // ordinals beyond 63: set up on every call
  if (bit && (o.done.load(std::memory_order_acquire) & bit)) return cudaSuccess;
  e = f();                                   // idempotent: two threads racing here both run it
  if (e == cudaSuccess && bit) o.done.fetch_or(bit, std::memory_order_release);
  return e;
}
// Per-device cached integer (e.g. resident clusters of a kernel); 0 = not yet computed.
struct PerDeviceInt {
  std::atomic<int> v[64] = {};
};

// ---------------------------------------------------------------------------------------------
// Device side
// ---------------------------------------------------------------------------------------------
namespace tc {

// Waits during the drain after an abort: long enough for any copy or MMA in flight (microseconds), short
// enough to return promptly if a barrier can no longer complete.
constexpr long long kDrainCycles = 2000000LL;

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
// kCluster: acquire at cluster scope (the barrier is also signalled from the other CTA of a pair).
template <bool kCluster = false>
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  if constexpr (kCluster) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  } else {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  }
  return ok != 0;
}

// State of a CTA's bounded waits.
struct WaitCtx {
  volatile int* abort_flag;   // this CTA's flag in shared memory: set by the first role whose wait expires
  uint32_t peer_flag;         // cluster-window address of the same flag in the other CTA of a pair; 0 = none
  long long limit;            // cycles a wait may take
};

__device__ __forceinline__ void raise_abort(const WaitCtx& wc) {
  *wc.abort_flag = 1;
  if (wc.peer_flag) asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(wc.peer_flag), "r"(1u) : "memory");
}

// Bounded wait.  Returns false if the phase did not complete within the limit (the abort flag is raised, in the
// peer CTA too) or another role has already given up.  The ordinary limit is checked every 256 polls.  A short
// limit (a test's) is checked on every poll, and once more when the phase has completed: a poll may itself
// suspend the thread for longer than such a limit, and the wait must count as expired all the same.
template <bool kCluster = false>
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, const WaitCtx& wc) {
  if (mbar_try_wait<kCluster>(bar, parity)) return true;
  const long long t0 = clock64();
  const bool short_limit = wc.limit < (1LL << 22);
  const int mask = short_limit ? 0 : 255;
  int spins = 0;
  while (!mbar_try_wait<kCluster>(bar, parity)) {
    if ((++spins & mask) == 0) {
      if (*wc.abort_flag) return false;
      if (clock64() - t0 > wc.limit) {
        raise_abort(wc);
        return false;
      }
    }
  }
  if (short_limit && clock64() - t0 > wc.limit) {
    raise_abort(wc);
    return false;
  }
  return true;
}
// The same wait made by all 32 lanes of a warp, with one outcome for the whole warp (false if any lane gave up):
// what follows such a wait is warp-synchronous (tcgen05.ld / st with .sync.aligned), so the lanes must not part.
template <bool kCluster = false>
__device__ __forceinline__ bool mbar_wait_warp(uint64_t* bar, uint32_t parity, const WaitCtx& wc) {
  return __all_sync(0xffffffffu, mbar_wait<kCluster>(bar, parity, wc));
}
// Wait used while draining after an abort: its own fixed limit, indifferent to the abort flag.
template <bool kCluster = false>
__device__ __forceinline__ bool mbar_wait_drain(uint64_t* bar, uint32_t parity) {
  const long long t0 = clock64();
  while (!mbar_try_wait<kCluster>(bar, parity))
    if (clock64() - t0 > kDrainCycles) return false;
  return true;
}
// After an abort, the thread that issued `issued` loads into a ring of `stages` barriers (load i on barrier
// i % stages, phase parity (i / stages) & 1) waits for the last load of every stage to land.
template <bool kCluster = false>
__device__ __forceinline__ void drain_ring(uint64_t* full, int stages, uint32_t issued) {
  const uint32_t first = issued > (uint32_t)stages ? issued - stages : 0;
  for (uint32_t i = first; i < issued; ++i) mbar_wait_drain<kCluster>(&full[i % stages], (i / stages) & 1);
}

// ---- TMA ------------------------------------------------------------------------------------------
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
__device__ __forceinline__ void prefetch_map(const CUtensorMap* tm) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(tm) : "memory");
}

// ---- tensor memory --------------------------------------------------------------------------------
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
// True in exactly one lane of a converged warp.  The issuing roles walk their loops with the whole warp and let the
// elected lane issue: addresses and descriptors are then warp-uniform values, which the tcgen05.mma and
// tcgen05.commit instructions take without a per-instruction transfer from the lane's own registers (measured:
// 130 -> 40-50 clocks per product for the issuing thread).
__device__ __forceinline__ bool elect_one() {
  uint32_t e;
  asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(e));
  return e != 0;
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// mbarrier arrives once all tcgen05.mma issued so far by this thread have completed.
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}

// 32 lanes x 32 consecutive 32-bit columns: thread i of the warp receives lane (base + i).
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
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major tile whose rows are 128 bytes, 128-byte swizzled (the layout a
// TMA box of 128 bytes of columns produces): 8-row groups are 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_k_sw128(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFF) >> 4);  // start address, 16-byte units
  d |= (uint64_t)1 << 16;                       // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;             // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                       // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                       // 128-byte swizzle
  return d;
}

__device__ __forceinline__ float gelu_tanh_fast(float x) {
  const float u = 0.7978845608028654f * (x + 0.044715f * x * x * x);
  float t;
  asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(u));
  return 0.5f * x * (1.0f + t);
}

// x Phi(x) with Phi(x) = erfc(-x / sqrt 2) / 2.  erfc(z), z >= 0, from the rational approximation 7.1.26 of
// Abramowitz & Stegun's handbook: erfc(z) = (a1 t + a2 t^2 + ... + a5 t^5) exp(-z^2), t = 1 / (1 + p z), absolute
// error <= 1.5e-7.  For x < 0 the product x erfc(|x| / sqrt 2) / 2 is formed directly (no 1 - ... cancellation).
// Against the exact function in double precision: relative Frobenius error 8e-8 on N(0, 1.5^2) inputs, far
// below the bf16 rounding of the output; two special-function operations and nine FMAs per value, no branch.
__device__ __forceinline__ float gelu_erf_fast(float x) {
  const float z = fabsf(x) * 0.70710678118654752f;
  float t, e;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(t) : "f"(fmaf(0.3275911f, z, 1.0f)));
  float poly = fmaf(1.061405429f, t, -1.453152027f);
  poly = fmaf(poly, t, 1.421413741f);
  poly = fmaf(poly, t, -0.284496736f);
  poly = fmaf(poly, t, 0.254829592f);
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(z * z * -1.4426950408889634f));
  const float half_erfc = 0.5f * poly * t * e;      // Phi(-|x|)
  return x * (x < 0.0f ? half_erfc : 1.0f - half_erfc);
}

}  // namespace tc
}  // namespace epd
