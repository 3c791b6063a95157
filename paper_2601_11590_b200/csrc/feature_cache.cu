// Feature keys and a device-resident feature cache: the step right after the Encode stage.
//
// The paper keeps encoder outputs in a "MM Store" keyed by a hash of the multimodal input, so that a
// repeated input is not encoded twice and only the key has to travel with the request (Section 3.2).
// This file provides the two pieces that belong to the encoder's side of that hand-off:
//   * content_hash: a 64-bit key per item, computed on the GPU from the item's input bytes
//       key = mix( (sum_k mix(w_k xor k*GOLDEN)) + 8n ),  w_1..w_n the bytes as little-endian 64-bit
//       words, mix = the SplitMix64 finalizer, arithmetic mod 2^64.  The sum is order independent, so
//       thousands of threads form it with integer atomics and the result is bit-exact.
//   * epd_feature_cache: an index (host) over a caller-provided pool of device memory holding feature
//       matrices by key, first-in-first-out eviction.
#include <cstring>
#include <new>
#include <unordered_map>
#include <vector>

#include "common.cuh"

namespace epd {
namespace {

constexpr unsigned long long kGolden = 0x9E3779B97F4A7C15ULL;

__host__ __device__ inline unsigned long long mix64(unsigned long long z) {
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
  return z ^ (z >> 31);
}

// grid (chunks, items): the item's words are read as 16-byte pairs from the first 16-byte boundary on;
// thread t of chunk c takes pairs c*blockDim.x + t, stepping by the grid's width.  k*GOLDEN advances
// by addition.  A leading or trailing single word is taken by the first thread of chunk 0.
__global__ void __launch_bounds__(256)
hash_accumulate_kernel(const uint8_t* __restrict__ data, const int64_t* __restrict__ item_off,
                       unsigned long long* __restrict__ acc) {
  const int i = blockIdx.y;
  const int64_t beg = item_off[i], words = (item_off[i + 1] - beg) >> 3;
  const unsigned long long* w = reinterpret_cast<const unsigned long long*>(data + beg);
  const int64_t head = (words > 0 && (reinterpret_cast<uintptr_t>(w) & 8)) ? 1 : 0;
  const int64_t pairs = (words - head) >> 1;
  const ulonglong2* w2 = reinterpret_cast<const ulonglong2*>(w + head);
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  unsigned long long c = (unsigned long long)(head + 2 * p + 1) * kGolden;   // (1-based index of the pair's first word) * GOLDEN
  const unsigned long long cstep = (unsigned long long)(2 * stride) * kGolden;
  unsigned long long sum = 0;
#pragma unroll 4
  for (; p < pairs; p += stride, c += cstep) {
    const ulonglong2 v = __ldg(w2 + p);
    sum += mix64(v.x ^ c) + mix64(v.y ^ (c + kGolden));
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    if (head) sum += mix64(w[0] ^ kGolden);
    if ((words - head) & 1) sum += mix64(w[words - 1] ^ ((unsigned long long)words * kGolden));
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  __shared__ unsigned long long part[8];
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = sum;
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned long long s = 0;
    for (int k = 0; k < (int)(blockDim.x >> 5); ++k) s += part[k];
    if (s != 0) atomicAdd(&acc[i], s);
  }
}

__global__ void hash_finalize_kernel(const int64_t* __restrict__ item_off, unsigned long long* __restrict__ acc, int n) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) acc[i] = mix64(acc[i] + (unsigned long long)(item_off[i + 1] - item_off[i]));
}

}  // namespace

cudaError_t content_hash(const void* data, const int64_t* item_off, int n_items, uint64_t* hashes, cudaStream_t s) {
  if (n_items == 0) return cudaSuccess;
  cudaError_t e = cudaMemsetAsync(hashes, 0, (size_t)n_items * sizeof(uint64_t), s);
  if (e != cudaSuccess) return e;
  hash_accumulate_kernel<<<dim3(64, (unsigned)n_items), 256, 0, s>>>(
      static_cast<const uint8_t*>(data), item_off, reinterpret_cast<unsigned long long*>(hashes));
  hash_finalize_kernel<<<(n_items + 127) / 128, 128, 0, s>>>(item_off, reinterpret_cast<unsigned long long*>(hashes),
                                                            n_items);
  return cudaGetLastError();
}

}  // namespace epd

// ---------------------------------------------------------------------------------------------
// Feature cache
// ---------------------------------------------------------------------------------------------
struct epd_feature_cache {
  struct Entry {
    uint64_t key;
    int64_t rows;
    size_t offset;   // bytes from the start of the pool
    size_t bytes;
  };
  uint8_t* pool = nullptr;
  size_t pool_bytes = 0, row_bytes = 0;
  std::vector<Entry> fifo;          // oldest first; entries occupy the ring [tail, head)
  size_t head = 0;                  // next free byte
  std::unordered_map<uint64_t, size_t> index;   // key -> position in fifo (rebuilt on eviction)
  int64_t hits = 0, misses = 0, evictions = 0;

  void reindex() {
    index.clear();
    for (size_t i = 0; i < fifo.size(); ++i) index[fifo[i].key] = i;
  }
  // Is [off, off+bytes) free of live entries?
  bool range_free(size_t off, size_t bytes) const {
    for (const Entry& e : fifo)
      if (off < e.offset + e.bytes && e.offset < off + bytes) return false;
    return true;
  }
};

extern "C" {

int epd_op_content_hash(const void* data, const int64_t* item_offsets, int32_t n_items, uint64_t* hashes,
                        void* stream) {
  if (n_items < 0) return EPD_EINVAL;
  if (n_items == 0) return EPD_OK;
  if (!data || !item_offsets || !hashes || ((uintptr_t)data & 7)) return EPD_EINVAL;
  if (epd::content_hash(data, item_offsets, n_items, hashes, static_cast<cudaStream_t>(stream)) != cudaSuccess)
    return EPD_ECUDA;
  return EPD_OK;
}

int epd_feature_cache_create(void* pool, size_t pool_bytes, size_t row_bytes, epd_feature_cache_t** out) {
  if (!out) return EPD_EINVAL;
  *out = nullptr;
  if (!pool || pool_bytes == 0 || row_bytes == 0 || ((uintptr_t)pool & 255)) return EPD_EINVAL;
  epd_feature_cache* c = new (std::nothrow) epd_feature_cache();
  if (!c) return EPD_ENOMEM;
  c->pool = static_cast<uint8_t*>(pool);
  c->pool_bytes = pool_bytes;
  c->row_bytes = row_bytes;
  *out = c;
  return EPD_OK;
}

int epd_feature_cache_destroy(epd_feature_cache_t* c) {
  delete c;
  return EPD_OK;
}

int epd_feature_cache_lookup(epd_feature_cache_t* c, uint64_t key, int64_t rows, void* dst, void* stream) {
  if (!c || rows < 0) return EPD_EINVAL;
  auto it = c->index.find(key);
  if (it == c->index.end() || c->fifo[it->second].rows != rows) {
    c->misses++;
    return 1;
  }
  c->hits++;
  if (dst && rows > 0) {
    const epd_feature_cache::Entry& e = c->fifo[it->second];
    if (cudaMemcpyAsync(dst, c->pool + e.offset, e.bytes, cudaMemcpyDeviceToDevice, static_cast<cudaStream_t>(stream)) !=
        cudaSuccess)
      return EPD_ECUDA;
  }
  return EPD_OK;
}

int epd_feature_cache_insert(epd_feature_cache_t* c, uint64_t key, int64_t rows, const void* src, void* stream) {
  if (!c || rows < 0 || (rows > 0 && !src)) return EPD_EINVAL;
  auto found = c->index.find(key);
  if (found != c->index.end()) {
    if (c->fifo[found->second].rows == rows) return EPD_OK;    // already cached
    // same key, other row count: the old entry could never be hit again (lookups require the row count to
    // match), so it is dropped and the new one stored
    c->fifo.erase(c->fifo.begin() + (long)found->second);
    c->evictions++;
    c->reindex();
  }
  const size_t bytes = ((size_t)rows * c->row_bytes + 255) / 256 * 256;
  if (bytes > c->pool_bytes) return EPD_ECAPACITY;
  // ring allocation: continue at head, wrap to 0 when the tail of the pool is too short, evict oldest
  // entries until the range is free
  size_t off = c->head;
  if (off + bytes > c->pool_bytes) off = 0;
  bool evicted = false;
  while (!c->range_free(off, bytes)) {
    c->fifo.erase(c->fifo.begin());
    c->evictions++;
    evicted = true;
  }
  if (evicted) c->reindex();
  if (rows > 0 && cudaMemcpyAsync(c->pool + off, src, (size_t)rows * c->row_bytes, cudaMemcpyDeviceToDevice,
                                  static_cast<cudaStream_t>(stream)) != cudaSuccess)
    return EPD_ECUDA;
  c->fifo.push_back({key, rows, off, bytes});
  c->index[key] = c->fifo.size() - 1;
  c->head = off + bytes;
  return EPD_OK;
}

int epd_feature_cache_stats(const epd_feature_cache_t* c, int64_t* hits, int64_t* misses, int64_t* evictions,
                            int64_t* entries) {
  if (!c) return EPD_EINVAL;
  if (hits) *hits = c->hits;
  if (misses) *misses = c->misses;
  if (evictions) *evictions = c->evictions;
  if (entries) *entries = (int64_t)c->fifo.size();
  return EPD_OK;
}

}  // extern "C"
