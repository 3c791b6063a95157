// C ABI of the Encode stage: the encoder object, host-side validation and integer layout,
// and the launch sequence of one forward pass.
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "common.cuh"

using namespace epd;

namespace {

// Step classes reported by epd_debug_profile_read().
enum { KC_LAYOUT = 0, KC_PATCH, KC_RMSNORM, KC_QKV, KC_ROPE, KC_ATTENTION, KC_OUT, KC_FC1, KC_FC2, KC_MERGE, KC_PROJ,
       KC_END, KC_COUNT = KC_END };

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Offsets of every activation buffer inside the caller's workspace.
struct Layout {
  size_t x, a, qkv, qh, kh, vh, u, merged, proj_hidden, stage_patches, stage_features, pix_patches;
  size_t grid, cu, cu_out, item_off, pos_row, pos_col, merge_slot, merge_idx, rope, status, aux, total;
  size_t qkv_perm_w, qkv_perm_b;   // per layer: QKV weight / bias with q and k rows in rotation-pair order
  size_t stage_patches2, stage_features2;   // second staging buffers of the pipelined host entry point
  size_t keys;                              // content keys of a batch's items (cached encode)
};

// The QKV projection can apply the rotary embedding and the head split in its epilogue.
bool fused_rope_possible(const epd_config_t& c) {
  return c.dtype == EPD_DTYPE_BF16 && c.head_dim % 8 == 0 && c.rope_theta > 0.0f && c.layers > 0;
}

bool config_ok(const epd_config_t* c) {
  if (!c) return false;
  if (c->dtype != EPD_DTYPE_F32 && c->dtype != EPD_DTYPE_BF16) return false;
  if (c->in_channels < 1 || c->patch < 1 || c->temporal_patch < 1) return false;
  if (c->hidden < 1 || c->layers < 0 || c->heads < 1 || c->head_dim < 4) return false;
  if (c->heads * c->head_dim != c->hidden || c->head_dim % 4 || c->head_dim > kMaxHeadDim) return false;
  if (c->mlp < 1 || (c->act != EPD_ACT_GELU_TANH && c->act != EPD_ACT_GELU_ERF)) return false;
  if (c->merge != 2 || !(c->eps >= 0.0f)) return false;
  if (c->proj_kind != EPD_PROJ_LINEAR && c->proj_kind != EPD_PROJ_MLP) return false;
  if (c->proj_kind == EPD_PROJ_MLP && c->proj_hidden < 1) return false;
  if (c->out_dim < 1 || c->max_tokens < 4 || c->max_tokens > (1 << 30) || c->max_images < 1 || c->max_grid < 2)
    return false;
  if (c->dtype == EPD_DTYPE_BF16 && (c->hidden % 8 || c->mlp % 8 || c->out_dim % 8 || c->proj_hidden % 8))
    return false;
  return true;
}

Layout make_layout(const epd_config_t& c) {
  Layout L{};
  const size_t es = c.dtype == EPD_DTYPE_F32 ? 4 : 2;
  const size_t T = (size_t)c.max_tokens, Tm = T / 4, h = c.hidden;
  const size_t dhp = padded_head_dim(c.head_dim);
  const size_t K = (size_t)c.in_channels * c.temporal_patch * c.patch * c.patch;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  L.x = take(T * h * 4);
  L.a = take(T * h * es);
  L.qkv = take(T * 3 * h * es);
  L.qh = take((size_t)c.heads * T * dhp * es);
  L.kh = take((size_t)c.heads * T * dhp * es);
  L.vh = take((size_t)c.heads * T * dhp * es);
  L.u = take(T * (size_t)c.mlp * es);
  L.merged = take(Tm * 4 * h * es);
  L.proj_hidden = take(c.proj_kind == EPD_PROJ_MLP ? Tm * (size_t)c.proj_hidden * es : 0);
  L.stage_patches = take(T * ((K + 7) / 8 * 8) * es);
  L.stage_features = take(Tm * (size_t)c.out_dim * es);
  L.stage_patches2 = take(T * ((K + 7) / 8 * 8) * es);
  L.stage_features2 = take(Tm * (size_t)c.out_dim * es);
  L.pix_patches = take(T * ((K + 7) / 8 * 8) * es);   // patch vectors built from raw frames
  L.grid = take((size_t)c.max_images * 3 * 4);
  L.cu = take(((size_t)c.max_images + 1) * 4);
  L.cu_out = take(((size_t)c.max_images + 1) * 4);
  L.item_off = take(((size_t)c.max_images + 1) * 8);
  L.keys = take((size_t)c.max_images * 8);
  L.pos_row = take(T * 4);
  L.pos_col = take(T * 4);
  L.merge_slot = take(T * 4);
  L.merge_idx = take(T * 4);
  L.rope = take((size_t)c.max_grid * (c.head_dim / 4) * sizeof(float2));
  L.status = take(256);
  const bool fused = fused_rope_possible(c);
  L.qkv_perm_w = take(fused ? (size_t)c.layers * 3 * h * h * es : 0);
  L.qkv_perm_b = take(fused ? (size_t)c.layers * align_up(3 * h * es, 256) : 0);
  L.aux = take(0);
  L.total = off;
  return L;
}

}  // namespace

struct epd_encoder {
  epd_config_t cfg;
  epd_weights_t w;
  std::vector<const void*> norm1_w, qkv_w, qkv_b, out_w, out_b, norm2_w, fc1_w, fc1_b, fc2_w, fc2_b;
  Layout lay;
  uint8_t* ws = nullptr;
  int32_t* pinned = nullptr;       // [3*max_images | max_images+1 | max_images+1]
  int64_t* pinned_off = nullptr;   // [max_images+1] byte offsets of the items' frames
  uint64_t* pinned_keys = nullptr; // [max_images] content keys read back by the cached encode
  cudaEvent_t staged_off = nullptr;
  bool staged_off_valid = false;
  cudaEvent_t staged = nullptr;    // recorded after the layout copy of the last batch
  bool staged_valid = false;
  cudaEvent_t last_launch = nullptr;   // recorded behind the encoder's most recent work on the caller's stream
  bool last_launch_valid = false;
  cudaStream_t aux_stream = nullptr;   // non-blocking stream of the encoder's own: reads the status word
  int32_t* pinned_status = nullptr;
  std::vector<int32_t> last_grid;  // grids of the batch whose layout is on the device
  std::vector<int32_t> host_cu;
  int64_t last_T = -1;
  std::vector<void*> taps;
  int64_t launches = 0;
  int64_t patch_dim = 0;
  // optional per-step timing: one event before every launch, one after the last
  bool profile = false;
  std::vector<cudaEvent_t> prof_events;
  std::vector<int> prof_class;
  std::vector<int> prof_launches;   // kernel launches behind each event (a sliced linear layer makes several)
  size_t prof_used = 0;
  bool use_tc = false;
  bool fused_rope = false;         // QKV epilogue does rotary + split (batches of more than 128 tokens)
  // Launch sequences captured as CUDA graphs, one per (batch geometry, buffers): a repeated request is one
  // graph launch instead of ~190 kernel launches (the host needs ~11 us per launch, which bounds the latency
  // of small batches).
  struct GraphEntry {
    const void* patches; int64_t ld; void* features; int sm_limit; std::vector<int32_t> grid;
    cudaGraphExec_t exec; int64_t launches;
  };
  std::vector<GraphEntry> graphs;
  bool use_graphs = true;
  // pipelined host entry point: copy streams of the library's own, double-buffered staging, and per slot
  // the events "patches on the device", "encode finished", "features on the host"
  cudaStream_t h2d_stream = nullptr, d2h_stream = nullptr;
  cudaEvent_t h2d_done[2] = {nullptr, nullptr}, compute_done[2] = {nullptr, nullptr}, d2h_done[2] = {nullptr, nullptr};
  bool compute_valid[2] = {false, false}, d2h_valid[2] = {false, false};
  uint64_t host_calls = 0;

  template <typename T> T* at(size_t off) const { return reinterpret_cast<T*>(ws + off); }
};

namespace {

// The CUDA error behind the most recent EPD_ECUDA of this thread (see epd_last_cuda_error()).
thread_local cudaError_t g_last_cuda_error = cudaSuccess;

#define EPD_CUDA(expr)                        \
  do {                                        \
    cudaError_t e__ = (expr);                 \
    if (e__ != cudaSuccess) {                 \
      g_last_cuda_error = e__;                \
      return EPD_ECUDA;                       \
    }                                         \
  } while (0)

// Counts a launch of step class `cls` and, in profiling mode, records an event before it.
int mark(epd_encoder* enc, int cls, cudaStream_t s) {
  enc->launches++;
  if (!enc->profile) return EPD_OK;
  if (enc->prof_used == enc->prof_events.size()) {
    cudaEvent_t ev;
    EPD_CUDA(cudaEventCreate(&ev));
    enc->prof_events.push_back(ev);
  }
  EPD_CUDA(cudaEventRecord(enc->prof_events[enc->prof_used], s));
  if (enc->prof_class.size() <= enc->prof_used) {
    enc->prof_class.resize(enc->prof_used + 1);
    enc->prof_launches.resize(enc->prof_used + 1);
  }
  enc->prof_class[enc->prof_used] = cls;
  enc->prof_launches[enc->prof_used] = 1;
  enc->prof_used++;
  return EPD_OK;
}
#define EPD_MARK(cls)                              \
  do {                                             \
    int rc__ = mark(enc, (cls), s);                \
    if (rc__) return rc__;                         \
  } while (0)

int linear_dispatch(epd_encoder* enc, int dtype, const void* x, int64_t ldx, const void* w, int64_t ldw,
                    const void* bias, void* out, int64_t ldo, int64_t M, int64_t N, int64_t K, int flags,
                    cudaStream_t s) {
  if (dtype == EPD_DTYPE_BF16 && !(flags & EPD_LINEAR_FORCE_FMA) &&
      linear_tc_supported(x, ldx, w, ldw, bias, out, ldo, M, N, K, flags)) {
    int* status = enc ? enc->at<int>(enc->lay.status) : nullptr;
    const int forced_bn = (flags >> EPD_LINEAR_TILE_N_SHIFT) & 0x1FF;
    if (forced_bn != 0 && forced_bn != 128 && forced_bn != 192 && forced_bn != 256) return EPD_EINVAL;
    EPD_CUDA(linear_tc(x, ldx, w, ldw, bias, out, ldo, M, N, K, enc ? (flags | kLinearStaticWeights) : flags, forced_bn,
                       status, s));
    if (enc) {
      const int extra = linear_tc_launches(M, N, K, flags, forced_bn) - 1;   // the caller counted one
      enc->launches += extra;
      if (enc->profile && enc->prof_used > 0) enc->prof_launches[enc->prof_used - 1] += extra;
    }
    return EPD_OK;
  }
  EPD_CUDA(linear_fma(dtype, x, ldx, w, ldw, bias, out, ldo, M, N, K, flags, s));
  return EPD_OK;
}

// Integer facts of a batch that follow from the grid list alone.
struct BatchShape {
  int64_t T = 0, Tm = 0;
  std::vector<int32_t> cu, cuo;    // prefix sums of tokens / merged tokens per item
};

// Host-only validation of a grid list against the encoder's capacities; nothing is enqueued.
int validate_grids(const epd_encoder* enc, const int32_t* grid_thw, int32_t n, int64_t capacity_rows, BatchShape* bs) {
  const epd_config_t& c = enc->cfg;
  if (n < 0 || (n > 0 && !grid_thw)) return EPD_EINVAL;
  if (n > c.max_images) return EPD_ECAPACITY;
  bs->T = bs->Tm = 0;
  bs->cu.assign(n + 1, 0);
  bs->cuo.assign(n + 1, 0);
  for (int i = 0; i < n; ++i) {
    const int64_t t = grid_thw[3 * i], h = grid_thw[3 * i + 1], w = grid_thw[3 * i + 2];
    if (t < 1 || h < 1 || w < 1 || (h & 1) || (w & 1)) return EPD_EINVAL;
    if (h > c.max_grid || w > c.max_grid) return EPD_ECAPACITY;
    if (t > c.max_tokens || t * h > c.max_tokens || t * h * w > c.max_tokens) return EPD_ECAPACITY;
    bs->T += t * h * w;
    bs->Tm += t * (h / 2) * (w / 2);
    if (bs->T > c.max_tokens) return EPD_ECAPACITY;
    bs->cu[i + 1] = (int32_t)bs->T;
    bs->cuo[i + 1] = (int32_t)bs->Tm;
  }
  if (capacity_rows >= 0 && bs->Tm > capacity_rows) return EPD_ECAPACITY;
  return EPD_OK;
}

// Validation of everything an encode of device buffers needs, before anything is enqueued.
int validate_encode(const epd_encoder* enc, const void* patches, int64_t patches_ld, const int32_t* grid_thw,
                    int32_t n, const void* features, int64_t cap_rows, BatchShape* bs) {
  if (cap_rows < 0) return EPD_EINVAL;
  const int rc = validate_grids(enc, grid_thw, n, cap_rows, bs);
  if (rc) return rc;
  if (bs->T == 0) return EPD_OK;
  if (!patches || !features) return EPD_EINVAL;
  if (((uintptr_t)patches & 15) || ((uintptr_t)features & 15)) return EPD_EINVAL;
  if (patches_ld < enc->patch_dim) return EPD_EINVAL;
  if (enc->cfg.dtype == EPD_DTYPE_BF16 && (patches_ld % 8)) return EPD_EINVAL;
  return EPD_OK;
}

void fill_host_outputs(const BatchShape& bs, int32_t n, int64_t* out_rows, int32_t* out_cu_rows) {
  if (out_rows) *out_rows = bs.Tm;
  if (out_cu_rows) std::memcpy(out_cu_rows, bs.cuo.data(), (n + 1) * sizeof(int32_t));
}

// Stages the integer layout of a validated batch on the device, unless it is the layout already there.
int stage_layout(epd_encoder* enc, const int32_t* grid_thw, int32_t n, const BatchShape& bs, cudaStream_t s,
                 bool* unchanged = nullptr) {
  const epd_config_t& c = enc->cfg;
  if (unchanged) *unchanged = false;
  if (n == 0) return EPD_OK;
  const int64_t T = bs.T;
  const bool same = enc->last_T == T && (int)enc->last_grid.size() == 3 * n &&
                    std::memcmp(enc->last_grid.data(), grid_thw, 3 * n * sizeof(int32_t)) == 0;
  if (same) {
    if (unchanged) *unchanged = true;
    return EPD_OK;
  }
  // The pinned staging buffer may still be the source of the previous batch's copy.
  if (enc->staged_valid) EPD_CUDA(cudaEventSynchronize(enc->staged));
  int32_t* pg = enc->pinned;
  int32_t* pcu = pg + 3 * (size_t)c.max_images;
  int32_t* pcuo = pcu + c.max_images + 1;
  std::memcpy(pg, grid_thw, 3 * n * sizeof(int32_t));
  std::memcpy(pcu, bs.cu.data(), (n + 1) * sizeof(int32_t));
  std::memcpy(pcuo, bs.cuo.data(), (n + 1) * sizeof(int32_t));
  EPD_CUDA(cudaMemcpyAsync(enc->at<int32_t>(enc->lay.grid), pg, 3 * n * sizeof(int32_t), cudaMemcpyHostToDevice, s));
  EPD_CUDA(cudaMemcpyAsync(enc->at<int32_t>(enc->lay.cu), pcu, (n + 1) * sizeof(int32_t), cudaMemcpyHostToDevice, s));
  EPD_CUDA(cudaMemcpyAsync(enc->at<int32_t>(enc->lay.cu_out), pcuo, (n + 1) * sizeof(int32_t),
                           cudaMemcpyHostToDevice, s));
  EPD_CUDA(cudaEventRecord(enc->staged, s));
  enc->staged_valid = true;
  EPD_MARK(KC_LAYOUT);
  EPD_CUDA(token_layout(enc->at<int32_t>(enc->lay.grid), enc->at<int32_t>(enc->lay.cu),
                        enc->at<int32_t>(enc->lay.cu_out), n, T, enc->at<int32_t>(enc->lay.pos_row),
                        enc->at<int32_t>(enc->lay.pos_col), enc->at<int32_t>(enc->lay.merge_slot),
                        enc->at<int32_t>(enc->lay.merge_idx), s));
  enc->last_grid.assign(grid_thw, grid_thw + 3 * n);
  enc->host_cu = bs.cu;
  enc->last_T = T;
  return EPD_OK;
}

// Marks the end of the encoder's work on stream s for epd_encoder_last_status (not while s is being captured:
// an event recorded into a capture cannot be waited for).
int note_last_launch(epd_encoder* enc, cudaStream_t s) {
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(s, &cap) != cudaSuccess) { (void)cudaGetLastError(); return EPD_OK; }
  if (cap != cudaStreamCaptureStatusNone) return EPD_OK;
  EPD_CUDA(cudaEventRecord(enc->last_launch, s));
  enc->last_launch_valid = true;
  return EPD_OK;
}

int attention_dispatch(epd_encoder* enc, int64_t T, int n_seg, cudaStream_t s) {
  const epd_config_t& c = enc->cfg;
  EPD_MARK(KC_ATTENTION);
  EPD_CUDA(attention_any(c.dtype, enc->at<void>(enc->lay.qh), enc->at<void>(enc->lay.kh), enc->at<void>(enc->lay.vh),
                         enc->at<int32_t>(enc->lay.cu), enc->host_cu.data(), n_seg, enc->at<void>(enc->lay.a), T,
                         c.heads, c.head_dim, 0, enc->at<int>(enc->lay.status), s));
  return EPD_OK;
}

// Steps RMSNorm .. MLP of block l on the float residual stream x.
int run_block(epd_encoder* enc, int l, float* x, int64_t T, int n_seg, cudaStream_t s) {
  const epd_config_t& c = enc->cfg;
  const int h = c.hidden, m = c.mlp;
  const int dt = c.dtype;
  void* a = enc->at<void>(enc->lay.a);
  void* qkv = enc->at<void>(enc->lay.qkv);
  void* u = enc->at<void>(enc->lay.u);
  const int gelu = c.act == EPD_ACT_GELU_TANH ? EPD_LINEAR_GELU_TANH : EPD_LINEAR_GELU_ERF;
  int rc;
  EPD_MARK(KC_RMSNORM);
  EPD_CUDA(rmsnorm(dt, x, enc->norm1_w[l], a, nullptr, T, h, c.eps, s));
  EPD_MARK(KC_QKV);
  const float q_scale = 1.4426950408889634f / sqrtf((float)c.head_dim);
  if (enc->fused_rope && T > 128) {
    // rotary embedding and head split in the projection's epilogue
    const size_t hh = (size_t)h;
    EPD_CUDA(linear_tc_pair_qkv(a, h, enc->ws + enc->lay.qkv_perm_w + (size_t)l * 3 * hh * hh * 2, h,
                                enc->ws + enc->lay.qkv_perm_b + (size_t)l * align_up(3 * hh * 2, 256),
                                enc->at<void>(enc->lay.qh), enc->at<void>(enc->lay.kh), enc->at<void>(enc->lay.vh),
                                enc->at<int32_t>(enc->lay.pos_row), enc->at<int32_t>(enc->lay.pos_col),
                                enc->at<float2>(enc->lay.rope), c.max_grid, T, c.heads, c.head_dim, q_scale, 1,
                                enc->at<int>(enc->lay.status), s));
  } else {
    if ((rc = linear_dispatch(enc, dt, a, h, enc->qkv_w[l], h, enc->qkv_b[l], qkv, 3 * h, T, 3 * h, h, 0, s)))
      return rc;
    EPD_MARK(KC_ROPE);
    EPD_CUDA(rope_split(dt, qkv, enc->at<int32_t>(enc->lay.pos_row), enc->at<int32_t>(enc->lay.pos_col),
                        enc->at<float2>(enc->lay.rope), c.max_grid, enc->at<void>(enc->lay.qh),
                        enc->at<void>(enc->lay.kh), enc->at<void>(enc->lay.vh), T, c.heads, c.head_dim, c.rope_theta,
                        q_scale, s));
  }
  if ((rc = attention_dispatch(enc, T, n_seg, s))) return rc;
  EPD_MARK(KC_OUT);
  if ((rc = linear_dispatch(enc, dt, a, h, enc->out_w[l], h, enc->out_b[l], x, h, T, h, h, EPD_LINEAR_ACCUMULATE, s)))
    return rc;
  EPD_MARK(KC_RMSNORM);
  EPD_CUDA(rmsnorm(dt, x, enc->norm2_w[l], a, nullptr, T, h, c.eps, s));
  EPD_MARK(KC_FC1);
  if ((rc = linear_dispatch(enc, dt, a, h, enc->fc1_w[l], h, enc->fc1_b[l], u, m, T, m, h, gelu, s))) return rc;
  EPD_MARK(KC_FC2);
  if ((rc = linear_dispatch(enc, dt, u, m, enc->fc2_w[l], m, enc->fc2_b[l], x, h, T, h, m, EPD_LINEAR_ACCUMULATE, s)))
    return rc;
  return EPD_OK;
}

// Closes the event list of a profiled pass.
int finish_profile(epd_encoder* enc, cudaStream_t s) {
  if (!enc->profile) return EPD_OK;
  enc->launches--;  // the closing event is not a launch
  return mark(enc, KC_END, s);
}

int launch_sequence(epd_encoder* enc, const void* patches, int64_t patches_ld, int32_t n, void* features, int64_t T,
                    cudaStream_t s);

// Encode of device buffers.  `bs` is the batch as validate_encode() left it: nothing here can fail validation.
int encode_validated(epd_encoder* enc, const void* patches, int64_t patches_ld, const int32_t* grid_thw, int32_t n,
                     void* features, const BatchShape& bs, cudaStream_t s);

int encode_device(epd_encoder* enc, const void* patches, int64_t patches_ld, const int32_t* grid_thw, int32_t n,
                  void* features, int64_t cap_rows, int64_t* out_rows, int32_t* out_cu_rows, cudaStream_t s) {
  enc->launches = 0;
  enc->prof_used = 0;
  BatchShape bs;
  const int rc = validate_encode(enc, patches, patches_ld, grid_thw, n, features, cap_rows, &bs);
  if (rc) return rc;
  fill_host_outputs(bs, n, out_rows, out_cu_rows);
  if (bs.T == 0) return EPD_OK;
  return encode_validated(enc, patches, patches_ld, grid_thw, n, features, bs, s);
}

int encode_validated(epd_encoder* enc, const void* patches, int64_t patches_ld, const int32_t* grid_thw, int32_t n,
                     void* features, const BatchShape& bs, cudaStream_t s) {
  const int64_t T = bs.T;
  bool unchanged = false;
  int rc = stage_layout(enc, grid_thw, n, bs, s, &unchanged);
  if (rc) return rc;
  rc = [&]() -> int {
  // A repeated request (same grids, same buffers) replays its captured launch sequence.  Capturing needs the
  // integer layout already on the device (no copies inside the capture), a stream that can be captured, and
  // no debugging hooks.
  if (enc->use_graphs && unchanged && s != nullptr && !enc->profile && enc->taps.empty()) {
    const int lim = sm_limit();
    for (const epd_encoder::GraphEntry& g : enc->graphs) {
      if (g.patches == patches && g.ld == patches_ld && g.features == features && g.sm_limit == lim &&
          (int)g.grid.size() == 3 * n && std::memcmp(g.grid.data(), grid_thw, 3 * n * sizeof(int32_t)) == 0) {
        enc->launches = g.launches;
        EPD_CUDA(cudaGraphLaunch(g.exec, s));
        return EPD_OK;
      }
    }
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(s, &cap) == cudaSuccess && cap == cudaStreamCaptureStatusNone &&
        cudaStreamBeginCapture(s, cudaStreamCaptureModeThreadLocal) == cudaSuccess) {
      rc = launch_sequence(enc, patches, patches_ld, n, features, T, s);
      cudaGraph_t graph = nullptr;
      const cudaError_t e_end = cudaStreamEndCapture(s, &graph);
      cudaGraphExec_t exec = nullptr;
      if (rc == EPD_OK && e_end == cudaSuccess && graph != nullptr &&
          cudaGraphInstantiate(&exec, graph, 0) == cudaSuccess) {
        cudaGraphDestroy(graph);
        if (enc->graphs.size() >= 8) {
          cudaGraphExecDestroy(enc->graphs.front().exec);
          enc->graphs.erase(enc->graphs.begin());
        }
        enc->graphs.push_back({patches, patches_ld, features, lim, std::vector<int32_t>(grid_thw, grid_thw + 3 * n), exec,
                               enc->launches});
        EPD_CUDA(cudaGraphLaunch(exec, s));
        return EPD_OK;
      }
      // capture did not work out: plain launches from now on
      if (graph) cudaGraphDestroy(graph);
      (void)cudaGetLastError();
      enc->use_graphs = false;
      enc->launches = 0;
    } else {
      (void)cudaGetLastError();
    }
  }
  return launch_sequence(enc, patches, patches_ld, n, features, T, s);
  }();
  if (rc) return rc;
  return note_last_launch(enc, s);
}

// The kernels of one encode, patch embedding to projector, on stream s.
int launch_sequence(epd_encoder* enc, const void* patches, int64_t patches_ld, int32_t n, void* features, int64_t T,
                    cudaStream_t s) {
  const epd_config_t& c = enc->cfg;
  const int dt = c.dtype;
  const int h = c.hidden;
  int rc;
  const int64_t Tm = T / 4;
  float* x = enc->at<float>(enc->lay.x);

  // patch embedding -> float residual stream
  EPD_MARK(KC_PATCH);
  if ((rc = linear_dispatch(enc, dt, patches, patches_ld, enc->w.patch_w, enc->w.patch_w_ld, enc->w.patch_b, x, h, T,
                            h, enc->patch_dim, EPD_LINEAR_OUT_F32, s)))
    return rc;
  for (int l = 0; l < c.layers; ++l) {
    if (!enc->taps.empty() && enc->taps[l])
      EPD_CUDA(cudaMemcpyAsync(enc->taps[l], x, (size_t)T * h * 4, cudaMemcpyDeviceToDevice, s));
    if ((rc = run_block(enc, l, x, T, n, s))) return rc;
  }
  if (!enc->taps.empty() && enc->taps[c.layers])
    EPD_CUDA(cudaMemcpyAsync(enc->taps[c.layers], x, (size_t)T * h * 4, cudaMemcpyDeviceToDevice, s));

  // final norm fused with the 2x2 merge: token j is written to slot merge_slot[j] of [4*Tm, h]
  void* merged = enc->at<void>(enc->lay.merged);
  if (c.final_norm) {
    EPD_MARK(KC_RMSNORM);
    EPD_CUDA(rmsnorm(dt, x, enc->w.final_norm_w, merged, enc->at<int32_t>(enc->lay.merge_slot), T, h, c.eps, s));
  } else if (dt == EPD_DTYPE_F32) {
    EPD_MARK(KC_MERGE);
    EPD_CUDA(merge_gather(dt, x, enc->at<int32_t>(enc->lay.merge_idx), merged, Tm, h, s));
  } else {
    return EPD_EUNSUPPORTED;  // bf16 without a final norm: the float stream has no bf16 copy to gather
  }
  if (c.proj_kind == EPD_PROJ_LINEAR) {
    EPD_MARK(KC_PROJ);
    if ((rc = linear_dispatch(enc, dt, merged, 4 * h, enc->w.proj_w1, 4 * h, enc->w.proj_b1, features, c.out_dim, Tm,
                              c.out_dim, 4 * h, 0, s)))
      return rc;
  } else {
    void* ph = enc->at<void>(enc->lay.proj_hidden);
    const int gelu = c.act == EPD_ACT_GELU_TANH ? EPD_LINEAR_GELU_TANH : EPD_LINEAR_GELU_ERF;
    EPD_MARK(KC_PROJ);
    if ((rc = linear_dispatch(enc, dt, merged, 4 * h, enc->w.proj_w1, 4 * h, enc->w.proj_b1, ph, c.proj_hidden, Tm,
                              c.proj_hidden, 4 * h, gelu, s)))
      return rc;
    EPD_MARK(KC_PROJ);
    if ((rc = linear_dispatch(enc, dt, ph, c.proj_hidden, enc->w.proj_w2, c.proj_hidden, enc->w.proj_b2, features,
                              c.out_dim, Tm, c.out_dim, c.proj_hidden, 0, s)))
      return rc;
  }
  return finish_profile(enc, s);
}

// Bytes of one item's raw frames: [t*Tp, C, h*P, w*P] pixels of 1 (uint8) or 2 (bf16) bytes.
int64_t item_frame_bytes(const epd_config_t& c, const int32_t* thw, int frame_format = EPD_FRAMES_U8) {
  return (int64_t)thw[0] * c.temporal_patch * c.in_channels * ((int64_t)thw[1] * c.patch) * ((int64_t)thw[2] * c.patch) *
         (frame_format == EPD_FRAMES_BF16 ? 2 : 1);
}

// Pixels of a validated batch -> patch vectors -> the stage.  item_off[i] is the byte offset of item i's frames
// inside `frames` (HOST array of n entries; the items need not be adjacent).
int encode_frames_at(epd_encoder* enc, const void* frames, int frame_format, const int64_t* item_off,
                     const int32_t* grid_thw, int32_t n,
                     const float* mean, const float* inv_std, void* features, const BatchShape& bs, cudaStream_t s) {
  const epd_config_t& c = enc->cfg;
  const int64_t ld = (enc->patch_dim + 7) / 8 * 8;
  if (enc->staged_off_valid) EPD_CUDA(cudaEventSynchronize(enc->staged_off));
  for (int i = 0; i < n; ++i) enc->pinned_off[i] = item_off[i];
  enc->pinned_off[n] = 0;
  enc->launches = 0;
  // the integer layout (grid, cu_seqlens) must be on the device before the patch kernel reads it
  int rc = stage_layout(enc, grid_thw, n, bs, s);
  if (rc) return rc;
  const int64_t launches_layout = enc->launches;
  EPD_CUDA(cudaMemcpyAsync(enc->at<int64_t>(enc->lay.item_off), enc->pinned_off, ((size_t)n + 1) * sizeof(int64_t),
                           cudaMemcpyHostToDevice, s));
  EPD_CUDA(cudaEventRecord(enc->staged_off, s));
  enc->staged_off_valid = true;
  EPD_CUDA(patchify(c.dtype, frame_format, frames, enc->at<int64_t>(enc->lay.item_off),
                    enc->at<int32_t>(enc->lay.grid), enc->at<int32_t>(enc->lay.cu), n, bs.T,
                    enc->at<void>(enc->lay.pix_patches), ld, c.in_channels, c.patch, c.temporal_patch, mean, inv_std, s));
  enc->launches = 0;
  rc = encode_validated(enc, enc->at<void>(enc->lay.pix_patches), ld, grid_thw, n, features, bs, s);
  enc->launches += launches_layout + 1;
  return rc;
}

// Frees everything the encoder object owns on the host side (events, streams, pinned buffers) and the object.
void release_host_side(epd_encoder* enc) {
  if (enc->staged) cudaEventDestroy(enc->staged);
  if (enc->staged_off) cudaEventDestroy(enc->staged_off);
  if (enc->last_launch) cudaEventDestroy(enc->last_launch);
  for (epd_encoder::GraphEntry& g : enc->graphs) cudaGraphExecDestroy(g.exec);
  for (int b = 0; b < 2; ++b) {
    if (enc->h2d_done[b]) cudaEventDestroy(enc->h2d_done[b]);
    if (enc->compute_done[b]) cudaEventDestroy(enc->compute_done[b]);
    if (enc->d2h_done[b]) cudaEventDestroy(enc->d2h_done[b]);
  }
  if (enc->h2d_stream) cudaStreamDestroy(enc->h2d_stream);
  if (enc->d2h_stream) cudaStreamDestroy(enc->d2h_stream);
  if (enc->aux_stream) cudaStreamDestroy(enc->aux_stream);
  if (enc->pinned_off) cudaFreeHost(enc->pinned_off);
  if (enc->pinned_status) cudaFreeHost(enc->pinned_status);
  if (enc->pinned_keys) cudaFreeHost(enc->pinned_keys);
  for (cudaEvent_t ev : enc->prof_events) cudaEventDestroy(ev);
  if (enc->pinned) cudaFreeHost(enc->pinned);
  delete enc;
}

}  // namespace

// =============================================================================================
// exported functions
// =============================================================================================
extern "C" {

size_t epd_encoder_workspace_bytes(const epd_config_t* cfg) {
  if (!config_ok(cfg)) return 0;
  return make_layout(*cfg).total;
}

int epd_encoder_create(const epd_config_t* cfg, const epd_weights_t* weights, void* workspace,
                       size_t workspace_bytes, epd_encoder_t** out) {
  if (!out) return EPD_EINVAL;
  *out = nullptr;
  if (!config_ok(cfg) || !weights || !workspace) return EPD_EINVAL;
  if ((uintptr_t)workspace & 255) return EPD_EINVAL;
  const Layout lay = make_layout(*cfg);
  if (workspace_bytes < lay.total) return EPD_ENOMEM;
  const int L = cfg->layers;
  const int64_t K = (int64_t)cfg->in_channels * cfg->temporal_patch * cfg->patch * cfg->patch;
  if (!weights->patch_w || weights->patch_w_ld < K || !weights->proj_w1) return EPD_EINVAL;
  if (cfg->final_norm && !weights->final_norm_w) return EPD_EINVAL;
  if (cfg->proj_kind == EPD_PROJ_MLP && !weights->proj_w2) return EPD_EINVAL;
  if (L > 0 && (!weights->norm1_w || !weights->qkv_w || !weights->out_w || !weights->norm2_w || !weights->fc1_w ||
                !weights->fc2_w))
    return EPD_EINVAL;
  if (cfg->dtype == EPD_DTYPE_BF16 && (weights->patch_w_ld % 8)) return EPD_EINVAL;

  epd_encoder* e = new (std::nothrow) epd_encoder();
  if (!e) return EPD_ENOMEM;
  e->cfg = *cfg;
  e->w = *weights;
  e->lay = lay;
  e->ws = static_cast<uint8_t*>(workspace);
  e->patch_dim = K;
  e->use_tc = cfg->dtype == EPD_DTYPE_BF16;
  auto copy_list = [&](std::vector<const void*>& dst, const void* const* src, bool required) -> bool {
    dst.assign(L, nullptr);
    if (!src) return !required || L == 0;
    for (int l = 0; l < L; ++l) {
      dst[l] = src[l];
      if (required && !src[l]) return false;
    }
    return true;
  };
  bool ok = copy_list(e->norm1_w, weights->norm1_w, true) && copy_list(e->qkv_w, weights->qkv_w, true) &&
            copy_list(e->qkv_b, weights->qkv_b, false) && copy_list(e->out_w, weights->out_w, true) &&
            copy_list(e->out_b, weights->out_b, false) && copy_list(e->norm2_w, weights->norm2_w, true) &&
            copy_list(e->fc1_w, weights->fc1_w, true) && copy_list(e->fc1_b, weights->fc1_b, false) &&
            copy_list(e->fc2_w, weights->fc2_w, true) && copy_list(e->fc2_b, weights->fc2_b, false);
  if (!ok) { delete e; return EPD_EINVAL; }
  // the struct's per-layer arrays belong to the caller: keep only our copies
  e->w.norm1_w = e->w.qkv_w = e->w.qkv_b = e->w.out_w = e->w.out_b = e->w.norm2_w = nullptr;
  e->w.fc1_w = e->w.fc1_b = e->w.fc2_w = e->w.fc2_b = nullptr;

  const size_t pinned_ints = 3 * (size_t)cfg->max_images + 2 * ((size_t)cfg->max_images + 1);
  if (cudaMallocHost(reinterpret_cast<void**>(&e->pinned), pinned_ints * sizeof(int32_t)) != cudaSuccess) {
    delete e;
    return EPD_ECUDA;
  }
  if (cudaEventCreateWithFlags(&e->staged, cudaEventDisableTiming) != cudaSuccess ||
      cudaEventCreateWithFlags(&e->staged_off, cudaEventDisableTiming) != cudaSuccess ||
      cudaEventCreateWithFlags(&e->last_launch, cudaEventDisableTiming) != cudaSuccess ||
      cudaStreamCreateWithFlags(&e->aux_stream, cudaStreamNonBlocking) != cudaSuccess ||
      cudaMallocHost(reinterpret_cast<void**>(&e->pinned_status), 64) != cudaSuccess ||
      cudaMallocHost(reinterpret_cast<void**>(&e->pinned_keys), (size_t)cfg->max_images * sizeof(uint64_t)) != cudaSuccess ||
      cudaMallocHost(reinterpret_cast<void**>(&e->pinned_off), ((size_t)cfg->max_images + 1) * sizeof(int64_t)) !=
          cudaSuccess) {
    release_host_side(e);
    return EPD_ECUDA;
  }
  cudaError_t err = cudaMemset(e->ws + lay.status, 0, 256);
  if (err == cudaSuccess && cfg->rope_theta > 0.0f)
    err = rope_table(e->at<float2>(lay.rope), cfg->max_grid, cfg->head_dim, cfg->rope_theta, 0);
  // permuted QKV weights and the padding columns of q, k, v for the fused rotary epilogue
  e->fused_rope = fused_rope_possible(*cfg);
  for (int l = 0; l < L && e->fused_rope; ++l)
    if (((uintptr_t)e->qkv_w[l] & 15) || (e->qkv_b[l] && ((uintptr_t)e->qkv_b[l] & 1))) e->fused_rope = false;
  if (e->fused_rope) {
    const size_t h = (size_t)cfg->hidden;
    for (int l = 0; l < L && err == cudaSuccess; ++l)
      err = qkv_permute(e->qkv_w[l], cfg->hidden, e->qkv_b[l], e->ws + lay.qkv_perm_w + (size_t)l * 3 * h * h * 2,
                        e->ws + lay.qkv_perm_b + (size_t)l * align_up(3 * h * 2, 256), cfg->heads, cfg->head_dim, 0);
    if (err == cudaSuccess)
      err = qkv_pad_init(e->at<void>(lay.qh), e->at<void>(lay.kh), e->at<void>(lay.vh),
                         (int64_t)cfg->heads * cfg->max_tokens, cfg->head_dim, 0);
  }
  if (err == cudaSuccess) err = cudaDeviceSynchronize();
  if (err != cudaSuccess) {
    release_host_side(e);
    return EPD_ECUDA;
  }
  *out = e;
  return EPD_OK;
}

int epd_encode(epd_encoder_t* enc, const void* patches, int64_t patches_ld, const int32_t* grid_thw,
               int32_t n_images, void* features, int64_t features_capacity_rows, int64_t* out_rows,
               int32_t* out_cu_rows, void* stream) {
  if (!enc) return EPD_EINVAL;
  return encode_device(enc, patches, patches_ld, grid_thw, n_images, features, features_capacity_rows, out_rows,
                       out_cu_rows, static_cast<cudaStream_t>(stream));
}

int epd_encode_host(epd_encoder_t* enc, const void* host_patches, const int32_t* grid_thw, int32_t n_images,
                    void* host_features, int64_t features_capacity_rows, int64_t* out_rows, int32_t* out_cu_rows,
                    void* stream) {
  if (!enc) return EPD_EINVAL;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const epd_config_t& c = enc->cfg;
  const size_t es = c.dtype == EPD_DTYPE_F32 ? 4 : 2;
  enc->launches = 0;
  enc->prof_used = 0;
  void* dp = enc->at<void>(enc->lay.stage_patches);
  void* df = enc->at<void>(enc->lay.stage_features);
  // the staged copy gets a leading dimension the tensor-core path accepts (a multiple of 8 elements)
  const int64_t ld = c.dtype == EPD_DTYPE_BF16 ? (enc->patch_dim + 7) / 8 * 8 : enc->patch_dim;
  // everything is validated before the first copy is enqueued
  if (features_capacity_rows < 0) return EPD_EINVAL;
  BatchShape bs;
  int rc = validate_grids(enc, grid_thw, n_images, features_capacity_rows, &bs);
  if (rc) return rc;
  if (bs.T > 0 && (!host_patches || !host_features)) return EPD_EINVAL;
  fill_host_outputs(bs, n_images, out_rows, out_cu_rows);
  if (bs.T == 0) return EPD_OK;
  EPD_CUDA(cudaMemcpy2DAsync(dp, (size_t)ld * es, host_patches, (size_t)enc->patch_dim * es,
                             (size_t)enc->patch_dim * es, (size_t)bs.T, cudaMemcpyHostToDevice, s));
  rc = encode_validated(enc, dp, ld, grid_thw, n_images, df, bs, s);
  if (rc) return rc;
  EPD_CUDA(cudaMemcpyAsync(host_features, df, (size_t)bs.Tm * c.out_dim * es, cudaMemcpyDeviceToHost, s));
  return note_last_launch(enc, s);
}

int epd_encode_host_async(epd_encoder_t* enc, const void* host_patches, const int32_t* grid_thw, int32_t n_images,
                          void* host_features, int64_t features_capacity_rows, int64_t* out_rows,
                          int32_t* out_cu_rows, void* stream) {
  if (!enc) return EPD_EINVAL;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const epd_config_t& c = enc->cfg;
  const size_t es = c.dtype == EPD_DTYPE_F32 ? 4 : 2;
  enc->launches = 0;
  enc->prof_used = 0;
  // everything is validated before the first copy is enqueued
  if (features_capacity_rows < 0) return EPD_EINVAL;
  BatchShape bs;
  int rc = validate_grids(enc, grid_thw, n_images, features_capacity_rows, &bs);
  if (rc) return rc;
  if (bs.T > 0 && (!host_patches || !host_features)) return EPD_EINVAL;
  fill_host_outputs(bs, n_images, out_rows, out_cu_rows);
  if (bs.T == 0) return EPD_OK;
  // lazily: two copy streams and six events
  if (!enc->h2d_stream) {
    EPD_CUDA(cudaStreamCreateWithFlags(&enc->h2d_stream, cudaStreamNonBlocking));
    EPD_CUDA(cudaStreamCreateWithFlags(&enc->d2h_stream, cudaStreamNonBlocking));
    for (int b = 0; b < 2; ++b) {
      EPD_CUDA(cudaEventCreateWithFlags(&enc->h2d_done[b], cudaEventDisableTiming));
      EPD_CUDA(cudaEventCreateWithFlags(&enc->compute_done[b], cudaEventDisableTiming));
      EPD_CUDA(cudaEventCreateWithFlags(&enc->d2h_done[b], cudaEventDisableTiming));
    }
  }
  const int b = (int)(enc->host_calls++ & 1);
  void* dp = enc->at<void>(b ? enc->lay.stage_patches2 : enc->lay.stage_patches);
  void* df = enc->at<void>(b ? enc->lay.stage_features2 : enc->lay.stage_features);
  const int64_t ld = c.dtype == EPD_DTYPE_BF16 ? (enc->patch_dim + 7) / 8 * 8 : enc->patch_dim;
  // patches -> staging slot b, once the encode that last read this slot (two calls ago) has finished
  if (enc->compute_valid[b]) EPD_CUDA(cudaStreamWaitEvent(enc->h2d_stream, enc->compute_done[b], 0));
  EPD_CUDA(cudaMemcpy2DAsync(dp, (size_t)ld * es, host_patches, (size_t)enc->patch_dim * es,
                             (size_t)enc->patch_dim * es, (size_t)bs.T, cudaMemcpyHostToDevice, enc->h2d_stream));
  EPD_CUDA(cudaEventRecord(enc->h2d_done[b], enc->h2d_stream));
  // the encode, on the caller's stream: after its patches have arrived and after the features this slot held
  // two calls ago have left for the host
  EPD_CUDA(cudaStreamWaitEvent(s, enc->h2d_done[b], 0));
  if (enc->d2h_valid[b]) EPD_CUDA(cudaStreamWaitEvent(s, enc->d2h_done[b], 0));
  rc = encode_validated(enc, dp, ld, grid_thw, n_images, df, bs, s);
  if (rc) return rc;
  EPD_CUDA(cudaEventRecord(enc->compute_done[b], s));
  enc->compute_valid[b] = true;
  // features -> host, behind the encode, while the caller's stream goes on with the next call
  EPD_CUDA(cudaStreamWaitEvent(enc->d2h_stream, enc->compute_done[b], 0));
  EPD_CUDA(cudaMemcpyAsync(host_features, df, (size_t)bs.Tm * c.out_dim * es, cudaMemcpyDeviceToHost, enc->d2h_stream));
  EPD_CUDA(cudaEventRecord(enc->d2h_done[b], enc->d2h_stream));
  enc->d2h_valid[b] = true;
  return EPD_OK;
}

int epd_encode_host_join(epd_encoder_t* enc, void* stream) {
  if (!enc) return EPD_EINVAL;
  for (int b = 0; b < 2; ++b)
    if (enc->d2h_valid[b]) EPD_CUDA(cudaStreamWaitEvent(static_cast<cudaStream_t>(stream), enc->d2h_done[b], 0));
  return EPD_OK;
}

int epd_encode_frames_fmt(epd_encoder_t* enc, const void* frames, int32_t frame_format, const int32_t* grid_thw,
                          int32_t n_images, const float* mean, const float* inv_std, void* features,
                          int64_t features_capacity_rows, int64_t* out_rows, int32_t* out_cu_rows, void* stream) {
  if (!enc) return EPD_EINVAL;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  enc->launches = 0;
  enc->prof_used = 0;
  // everything is validated before anything is enqueued
  if (frame_format != EPD_FRAMES_U8 && frame_format != EPD_FRAMES_BF16) return EPD_EINVAL;
  if (enc->cfg.in_channels > 4) return EPD_EUNSUPPORTED;
  BatchShape bs;
  int rc = validate_encode(enc, enc->at<void>(enc->lay.pix_patches), (enc->patch_dim + 7) / 8 * 8, grid_thw, n_images,
                           features, features_capacity_rows, &bs);
  if (rc) return rc;
  if (bs.T > 0 && (!frames || !mean || !inv_std)) return EPD_EINVAL;
  if (frame_format == EPD_FRAMES_BF16 && ((uintptr_t)frames & 1)) return EPD_EINVAL;
  fill_host_outputs(bs, n_images, out_rows, out_cu_rows);
  if (bs.T == 0) return EPD_OK;
  std::vector<int64_t> off(n_images);
  int64_t at = 0;
  for (int i = 0; i < n_images; ++i) {
    off[i] = at;
    at += item_frame_bytes(enc->cfg, grid_thw + 3 * i, frame_format);
  }
  return encode_frames_at(enc, frames, frame_format, off.data(), grid_thw, n_images, mean, inv_std, features, bs, s);
}

int epd_encode_frames(epd_encoder_t* enc, const void* frames, const int32_t* grid_thw, int32_t n_images,
                      const float* mean, const float* inv_std, void* features, int64_t features_capacity_rows,
                      int64_t* out_rows, int32_t* out_cu_rows, void* stream) {
  return epd_encode_frames_fmt(enc, frames, EPD_FRAMES_U8, grid_thw, n_images, mean, inv_std, features,
                               features_capacity_rows, out_rows, out_cu_rows, stream);
}

int epd_encode_frames_cached(epd_encoder_t* enc, epd_feature_cache_t* cache, const void* frames,
                             const int32_t* grid_thw, int32_t n_images, const float* mean, const float* inv_std,
                             void* features, int64_t features_capacity_rows, int64_t* out_rows, int32_t* out_cu_rows,
                             uint64_t* out_keys, uint8_t* out_hit, void* stream) {
  if (!enc || !cache) return EPD_EINVAL;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const epd_config_t& c = enc->cfg;
  const size_t row_bytes = (size_t)c.out_dim * (c.dtype == EPD_DTYPE_F32 ? 4 : 2);
  enc->launches = 0;
  enc->prof_used = 0;
  if (c.in_channels > 4) return EPD_EUNSUPPORTED;
  BatchShape bs;
  int rc = validate_encode(enc, enc->at<void>(enc->lay.pix_patches), (enc->patch_dim + 7) / 8 * 8, grid_thw, n_images,
                           features, features_capacity_rows, &bs);
  if (rc) return rc;
  if (bs.T > 0 && (!frames || !mean || !inv_std)) return EPD_EINVAL;
  fill_host_outputs(bs, n_images, out_rows, out_cu_rows);
  if (bs.T == 0) return EPD_OK;
  // content keys of all items: hashed on the device, read back (the one host wait of this call)
  if (enc->staged_off_valid) EPD_CUDA(cudaEventSynchronize(enc->staged_off));
  std::vector<int64_t> off(n_images + 1);
  off[0] = 0;
  for (int i = 0; i < n_images; ++i) off[i + 1] = off[i] + item_frame_bytes(c, grid_thw + 3 * i);
  for (int i = 0; i <= n_images; ++i) {
    if (off[i] % 8) return EPD_EUNSUPPORTED;   // the hash reads 8-byte words
    enc->pinned_off[i] = off[i];
  }
  EPD_CUDA(cudaMemcpyAsync(enc->at<int64_t>(enc->lay.item_off), enc->pinned_off, ((size_t)n_images + 1) * sizeof(int64_t),
                           cudaMemcpyHostToDevice, s));
  EPD_CUDA(cudaEventRecord(enc->staged_off, s));
  enc->staged_off_valid = true;
  EPD_CUDA(content_hash(frames, enc->at<int64_t>(enc->lay.item_off), n_images, enc->at<uint64_t>(enc->lay.keys), s));
  EPD_CUDA(cudaMemcpyAsync(enc->pinned_keys, enc->at<uint64_t>(enc->lay.keys), (size_t)n_images * sizeof(uint64_t),
                           cudaMemcpyDeviceToHost, s));
  EPD_CUDA(cudaStreamSynchronize(s));
  const int64_t hash_launches = 2;
  // hits are copied from the cache straight to their rows; the first occurrence of every missing key is encoded
  std::vector<int> todo;               // items to encode
  std::vector<int> source(n_images, -1);   // for a missing item: position in `todo` of the item that carries its key
  for (int i = 0; i < n_images; ++i) {
    const uint64_t key = enc->pinned_keys[i];
    const int64_t rows = bs.cuo[i + 1] - bs.cuo[i];
    if (out_keys) out_keys[i] = key;
    const int st = epd_feature_cache_lookup(cache, key, rows, static_cast<uint8_t*>(features) + (size_t)bs.cuo[i] * row_bytes,
                                            stream);
    if (st < 0) return st;
    if (out_hit) out_hit[i] = st == EPD_OK ? 1 : 0;
    if (st == EPD_OK) continue;
    for (size_t k = 0; k < todo.size() && source[i] < 0; ++k)
      if (enc->pinned_keys[todo[k]] == key && std::memcmp(grid_thw + 3 * todo[k], grid_thw + 3 * i, 12) == 0)
        source[i] = (int)k;
    if (source[i] < 0) {
      source[i] = (int)todo.size();
      todo.push_back(i);
    }
  }
  int64_t launches = hash_launches;
  if (!todo.empty()) {
    const int m = (int)todo.size();
    std::vector<int32_t> g(3 * m);
    std::vector<int64_t> sub_off(m);
    for (int k = 0; k < m; ++k) {
      std::memcpy(&g[3 * k], grid_thw + 3 * todo[k], 12);
      sub_off[k] = off[todo[k]];
    }
    BatchShape sub;
    if ((rc = validate_grids(enc, g.data(), m, -1, &sub))) return rc;
    // the missing items are encoded as a batch of their own into the staging buffer of the workspace
    uint8_t* scratch = enc->at<uint8_t>(enc->lay.stage_features);
    rc = encode_frames_at(enc, frames, EPD_FRAMES_U8, sub_off.data(), g.data(), m, mean, inv_std, scratch, sub, s);
    if (rc) return rc;
    launches += enc->launches;
    for (int i = 0; i < n_images; ++i) {
      if (source[i] < 0) continue;
      const int k = source[i];
      const size_t bytes = (size_t)(sub.cuo[k + 1] - sub.cuo[k]) * row_bytes;
      if (bytes)
        EPD_CUDA(cudaMemcpyAsync(static_cast<uint8_t*>(features) + (size_t)bs.cuo[i] * row_bytes,
                                 scratch + (size_t)sub.cuo[k] * row_bytes, bytes, cudaMemcpyDeviceToDevice, s));
    }
    for (int k = 0; k < m; ++k) {
      rc = epd_feature_cache_insert(cache, enc->pinned_keys[todo[k]], sub.cuo[k + 1] - sub.cuo[k],
                                    scratch + (size_t)sub.cuo[k] * row_bytes, stream);
      if (rc == EPD_ECAPACITY) rc = EPD_OK;      // an item larger than the whole pool is simply not cached
      if (rc) return rc;
    }
  }
  enc->launches = launches;
  return note_last_launch(enc, s);
}

int epd_encoder_last_status(epd_encoder_t* enc) {
  if (!enc) return EPD_EINVAL;
  // wait for the encoder's own most recent work only (an event behind its last launch), and read the word on
  // a non-blocking stream of the encoder's: other streams and processes sharing the GPU are not stalled
  if (enc->last_launch_valid) EPD_CUDA(cudaStreamWaitEvent(enc->aux_stream, enc->last_launch, 0));
  EPD_CUDA(cudaMemcpyAsync(enc->pinned_status, enc->ws + enc->lay.status, sizeof(int32_t), cudaMemcpyDeviceToHost,
                           enc->aux_stream));
  EPD_CUDA(cudaStreamSynchronize(enc->aux_stream));
  const int32_t st = *enc->pinned_status;
  if (st != 0) {
    EPD_CUDA(cudaMemsetAsync(enc->ws + enc->lay.status, 0, sizeof(int32_t), enc->aux_stream));
    EPD_CUDA(cudaStreamSynchronize(enc->aux_stream));
  }
  return st;
}

int64_t epd_encoder_last_launch_count(const epd_encoder_t* enc) { return enc ? enc->launches : 0; }

int epd_encoder_uses_tensor_cores(const epd_encoder_t* enc) { return enc && enc->use_tc ? 1 : 0; }

int epd_encoder_destroy(epd_encoder_t* enc) {
  if (!enc) return EPD_OK;
  // the encoder's work must be over before its buffers go away: its last launch on the caller's stream, and
  // the copies on its own streams
  if (enc->last_launch_valid) cudaEventSynchronize(enc->last_launch);
  for (int b = 0; b < 2; ++b)
    if (enc->d2h_valid[b]) cudaEventSynchronize(enc->d2h_done[b]);
  if (enc->h2d_stream) cudaStreamSynchronize(enc->h2d_stream);
  if (enc->aux_stream) cudaStreamSynchronize(enc->aux_stream);
  release_host_side(enc);
  return EPD_OK;
}

const char* epd_last_cuda_error(void) { return cudaGetErrorName(g_last_cuda_error); }

const char* epd_strerror(int status) {
  switch (status) {
    case EPD_OK: return "ok";
    case EPD_EINVAL: return "invalid argument";
    case EPD_ENOMEM: return "workspace too small or out of host memory";
    case EPD_ECUDA: return "CUDA call failed";
    case EPD_ECAPACITY: return "batch exceeds configured capacity";
    case EPD_EUNSUPPORTED: return "unsupported shape";
    case EPD_ETIMEOUT: return "bounded device-side wait expired";
    default: return "unknown status";
  }
}

int epd_debug_bookkeeping(epd_encoder_t* enc, int32_t* cu_seqlens, int32_t* pos_row, int32_t* pos_col,
                          int32_t* merge_idx) {
  if (!enc || enc->last_T < 0) return EPD_EINVAL;
  if (enc->last_launch_valid) EPD_CUDA(cudaEventSynchronize(enc->last_launch));
  const size_t n = enc->last_grid.size() / 3, T = (size_t)enc->last_T;
  if (cu_seqlens) EPD_CUDA(cudaMemcpy(cu_seqlens, enc->ws + enc->lay.cu, (n + 1) * 4, cudaMemcpyDeviceToHost));
  if (pos_row) EPD_CUDA(cudaMemcpy(pos_row, enc->ws + enc->lay.pos_row, T * 4, cudaMemcpyDeviceToHost));
  if (pos_col) EPD_CUDA(cudaMemcpy(pos_col, enc->ws + enc->lay.pos_col, T * 4, cudaMemcpyDeviceToHost));
  if (merge_idx) EPD_CUDA(cudaMemcpy(merge_idx, enc->ws + enc->lay.merge_idx, T * 4, cudaMemcpyDeviceToHost));
  return EPD_OK;
}

int epd_debug_set_taps(epd_encoder_t* enc, void* const* taps) {
  if (!enc) return EPD_EINVAL;
  enc->taps.clear();
  if (taps) enc->taps.assign(taps, taps + enc->cfg.layers + 1);
  return EPD_OK;
}

int epd_debug_run_block(epd_encoder_t* enc, int32_t layer, void* x, const int32_t* grid_thw, int32_t n_images,
                        void* stream) {
  if (!enc || !x || layer < 0 || layer >= enc->cfg.layers) return EPD_EINVAL;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  int64_t T = 0;
  enc->launches = 0;
  enc->prof_used = 0;
  BatchShape bs;
  int rc = validate_grids(enc, grid_thw, n_images, -1, &bs);
  if (rc) return rc;
  T = bs.T;
  if (T == 0) return EPD_OK;
  if ((rc = stage_layout(enc, grid_thw, n_images, bs, s))) return rc;
  if ((rc = run_block(enc, layer, static_cast<float*>(x), T, n_images, s))) return rc;
  if ((rc = finish_profile(enc, s))) return rc;
  return note_last_launch(enc, s);
}

int epd_debug_use_graphs(epd_encoder_t* enc, int32_t enable) {
  if (!enc) return EPD_EINVAL;
  enc->use_graphs = enable != 0;
  return EPD_OK;
}

int32_t epd_debug_graph_count(const epd_encoder_t* enc) { return enc ? (int32_t)enc->graphs.size() : 0; }

int epd_debug_profile(epd_encoder_t* enc, int32_t enable) {
  if (!enc) return EPD_EINVAL;
  enc->profile = enable != 0;
  enc->prof_used = 0;
  return EPD_OK;
}

int32_t epd_debug_profile_classes(void) { return KC_COUNT; }

const char* epd_debug_profile_class_name(int32_t cls) {
  static const char* names[KC_COUNT] = {"token_layout", "patch_embed", "rmsnorm", "qkv_linear", "rope_split",
                                        "attention", "out_linear", "fc1_linear", "fc2_linear", "merge", "projector"};
  return (cls >= 0 && cls < KC_COUNT) ? names[cls] : "";
}

int epd_debug_profile_read(epd_encoder_t* enc, float* ms, int64_t* launches) {
  if (!enc || !ms || !launches) return EPD_EINVAL;
  for (int i = 0; i < KC_COUNT; ++i) { ms[i] = 0.0f; launches[i] = 0; }
  if (enc->prof_used < 2) return EPD_OK;
  EPD_CUDA(cudaEventSynchronize(enc->prof_events[enc->prof_used - 1]));
  for (size_t i = 0; i + 1 < enc->prof_used; ++i) {
    float t = 0.0f;
    EPD_CUDA(cudaEventElapsedTime(&t, enc->prof_events[i], enc->prof_events[i + 1]));
    const int cls = enc->prof_class[i];
    if (cls >= 0 && cls < KC_COUNT) { ms[cls] += t; launches[cls] += enc->prof_launches[i]; }
  }
  return EPD_OK;
}

// ---- single steps ---------------------------------------------------------------------------

int epd_op_linear(int32_t dtype, const void* x, int64_t ldx, const void* w, int64_t ldw, const void* bias, void* out,
                  int64_t ldo, int64_t M, int64_t N, int64_t K, int32_t flags, void* stream) {
  if (dtype != EPD_DTYPE_F32 && dtype != EPD_DTYPE_BF16) return EPD_EINVAL;
  if (M < 0 || N < 0 || K < 1 || ldx < K || ldw < K || ldo < N) return EPD_EINVAL;
  if (M == 0 || N == 0) return EPD_OK;
  if (!x || !w || !out) return EPD_EINVAL;
  return linear_dispatch(nullptr, dtype, x, ldx, w, ldw, bias, out, ldo, M, N, K, flags,
                         static_cast<cudaStream_t>(stream));
}

int epd_op_rmsnorm(int32_t dtype, const void* x, const void* gain, void* out, const int32_t* dst_row, int64_t T,
                   int32_t hidden, float eps, void* stream) {
  if (dtype != EPD_DTYPE_F32 && dtype != EPD_DTYPE_BF16) return EPD_EINVAL;
  if (T < 0 || hidden < 1) return EPD_EINVAL;
  if (T == 0) return EPD_OK;
  if (!x || !gain || !out || ((uintptr_t)x & 15) || ((uintptr_t)out & 15)) return EPD_EINVAL;
  EPD_CUDA(rmsnorm(dtype, x, gain, out, dst_row, T, hidden, eps, static_cast<cudaStream_t>(stream)));
  return EPD_OK;
}

int epd_op_quantize_e4m3(const void* x, int64_t ldx, void* q, int64_t ldq, float* scale, int64_t M, int64_t K,
                         void* stream) {
  if (M < 0 || K < 1 || ldx < K || ldq < K) return EPD_EINVAL;
  if (M == 0) return EPD_OK;
  if (!x || !q || !scale) return EPD_EINVAL;
  if (((uintptr_t)x & 15) || ((uintptr_t)q & 15) || (ldx % 8) || (ldq % 16)) return EPD_EINVAL;
  EPD_CUDA(quantize_rows_e4m3(x, ldx, q, ldq, scale, M, K, static_cast<cudaStream_t>(stream)));
  return EPD_OK;
}

int epd_op_linear_e4m3(const void* xq, int64_t ldx, const float* x_scale, const void* wq, int64_t ldw,
                       const float* w_scale, const void* bias, void* out, int64_t ldo, int64_t M, int64_t N, int64_t K,
                       int32_t flags, void* stream) {
  if (M < 0 || N < 0 || K < 1 || ldx < K || ldw < K || ldo < N) return EPD_EINVAL;
  if (flags & (EPD_LINEAR_ACCUMULATE | EPD_LINEAR_FORCE_FMA)) return EPD_EUNSUPPORTED;
  if (M == 0 || N == 0) return EPD_OK;
  if (!xq || !wq || !x_scale || !w_scale || !out) return EPD_EINVAL;
  const bool out_f32 = flags & EPD_LINEAR_OUT_F32;
  if (((uintptr_t)xq | (uintptr_t)wq | (uintptr_t)out) & 15) return EPD_EINVAL;
  if ((ldx % 16) || (ldw % 16) || (ldo % (out_f32 ? 4 : 8)) || (N % 8) || M > (1 << 30) || N > (1 << 30) || K > (1 << 30))
    return EPD_EUNSUPPORTED;
  if (!tensor_core_path_available()) return EPD_EUNSUPPORTED;
  EPD_CUDA(linear_tc_pair_e4m3(xq, ldx, x_scale, wq, ldw, w_scale, bias, out, ldo, M, N, K, flags, nullptr,
                               static_cast<cudaStream_t>(stream)));
  return EPD_OK;
}

int32_t epd_padded_head_dim(int32_t head_dim) { return padded_head_dim(head_dim); }

int epd_op_rope_split(int32_t dtype, const void* qkv, const int32_t* pos_row, const int32_t* pos_col, void* q,
                      void* k, void* v, int64_t T, int32_t heads, int32_t head_dim, float theta, float q_scale,
                      void* stream) {
  if (dtype != EPD_DTYPE_F32 && dtype != EPD_DTYPE_BF16) return EPD_EINVAL;
  if (T < 0 || heads < 1 || head_dim < 4 || head_dim % 4 || head_dim > kMaxHeadDim) return EPD_EINVAL;
  if (T == 0) return EPD_OK;
  if (!qkv || !pos_row || !pos_col || !q || !k || !v) return EPD_EINVAL;
  EPD_CUDA(rope_split(dtype, qkv, pos_row, pos_col, nullptr, 0, q, k, v, T, heads, head_dim, theta, q_scale,
                      static_cast<cudaStream_t>(stream)));
  return EPD_OK;
}

int epd_op_qkv_prepare(const void* w, int64_t ldw, const void* bias, void* w_prepared, void* bias_prepared,
                       int32_t heads, int32_t head_dim, void* stream) {
  if (heads < 1 || head_dim < 8 || head_dim % 8 || head_dim > kMaxHeadDim) return EPD_EINVAL;
  if (!w || !w_prepared || !bias_prepared || ldw < (int64_t)heads * head_dim || ldw % 8) return EPD_EINVAL;
  if (((uintptr_t)w | (uintptr_t)w_prepared) & 15) return EPD_EINVAL;
  EPD_CUDA(qkv_permute(w, ldw, bias, w_prepared, bias_prepared, heads, head_dim, static_cast<cudaStream_t>(stream)));
  return EPD_OK;
}

int epd_op_rope_table(float* table, int32_t rows, int32_t head_dim, float theta, void* stream) {
  if (!table || rows < 1 || head_dim < 4 || head_dim % 4 || head_dim > kMaxHeadDim || !(theta > 0.0f)) return EPD_EINVAL;
  EPD_CUDA(rope_table(reinterpret_cast<float2*>(table), rows, head_dim, theta, static_cast<cudaStream_t>(stream)));
  return EPD_OK;
}

int epd_op_qkv_pad_init(void* q, void* k, void* v, int64_t rows, int32_t head_dim, void* stream) {
  if (rows < 0 || head_dim < 4 || head_dim > kMaxHeadDim) return EPD_EINVAL;
  if (rows == 0) return EPD_OK;
  if (!q || !k || !v) return EPD_EINVAL;
  EPD_CUDA(qkv_pad_init(q, k, v, rows, head_dim, static_cast<cudaStream_t>(stream)));
  return EPD_OK;
}

int epd_op_qkv_rope(const void* x, int64_t ldx, const void* w_prepared, const void* bias_prepared,
                    const int32_t* pos_row, const int32_t* pos_col, const float* table, int32_t table_rows,
                    void* q, void* k, void* v, int64_t T, int32_t heads, int32_t head_dim, float q_scale,
                    void* stream) {
  if (T < 0 || T > (1 << 30) || heads < 1 || head_dim < 8 || head_dim % 8 || head_dim > kMaxHeadDim) return EPD_EINVAL;
  if (T == 0) return EPD_OK;
  const int64_t h = (int64_t)heads * head_dim;
  if (!x || !w_prepared || !pos_row || !pos_col || !table || table_rows < 1 || !q || !k || !v) return EPD_EINVAL;
  if (ldx < h || ldx % 8) return EPD_EINVAL;
  if (((uintptr_t)x | (uintptr_t)w_prepared | (uintptr_t)q | (uintptr_t)k | (uintptr_t)v | (uintptr_t)table) & 15)
    return EPD_EINVAL;
  EPD_CUDA(linear_tc_pair_qkv(x, ldx, w_prepared, h, bias_prepared, q, k, v, pos_row, pos_col,
                              reinterpret_cast<const float2*>(table), table_rows, T, heads, head_dim, q_scale, 0, nullptr,
                              static_cast<cudaStream_t>(stream)));
  return EPD_OK;
}

int epd_op_attention(int32_t dtype, const void* q, const void* k, const void* v, const int32_t* cu_seqlens,
                     const int32_t* host_cu_seqlens, int32_t n_seg, void* out, int64_t T, int32_t heads,
                     int32_t head_dim, int32_t flags, void* stream) {
  if (dtype != EPD_DTYPE_F32 && dtype != EPD_DTYPE_BF16) return EPD_EINVAL;
  if (T < 0 || n_seg < 0 || heads < 1 || head_dim < 4 || head_dim > kMaxHeadDim) return EPD_EINVAL;
  if (T == 0 || n_seg == 0) return EPD_OK;
  if (!q || !k || !v || !cu_seqlens || !host_cu_seqlens || !out) return EPD_EINVAL;
  if (host_cu_seqlens[0] != 0 || host_cu_seqlens[n_seg] != T) return EPD_EINVAL;
  for (int i = 0; i < n_seg; ++i)
    if (host_cu_seqlens[i + 1] <= host_cu_seqlens[i]) return EPD_EINVAL;
  EPD_CUDA(attention_any(dtype, q, k, v, cu_seqlens, host_cu_seqlens, n_seg, out, T, heads, head_dim, flags, nullptr,
                         static_cast<cudaStream_t>(stream)));
  return EPD_OK;
}

int epd_op_patchify_fmt(int32_t dtype, int32_t frame_format, const void* frames, const int64_t* item_offsets,
                        const int32_t* grid_thw, const int32_t* cu_seqlens, int32_t n_images, int64_t T, void* patches,
                        int64_t ld, int32_t in_channels, int32_t patch, int32_t temporal_patch, const float* mean,
                        const float* inv_std, void* stream) {
  if (dtype != EPD_DTYPE_F32 && dtype != EPD_DTYPE_BF16) return EPD_EINVAL;
  if (frame_format != EPD_FRAMES_U8 && frame_format != EPD_FRAMES_BF16) return EPD_EINVAL;
  if (n_images < 0 || T < 0 || in_channels < 1 || in_channels > 4 || patch < 1 || temporal_patch < 1) return EPD_EINVAL;
  if (T == 0 || n_images == 0) return EPD_OK;
  if (!frames || !item_offsets || !grid_thw || !cu_seqlens || !patches || !mean || !inv_std) return EPD_EINVAL;
  if (ld < (int64_t)in_channels * temporal_patch * patch * patch) return EPD_EINVAL;
  EPD_CUDA(patchify(dtype, frame_format, frames, item_offsets, grid_thw, cu_seqlens, n_images, T, patches, ld, in_channels,
                    patch, temporal_patch, mean, inv_std, static_cast<cudaStream_t>(stream)));
  return EPD_OK;
}

int epd_op_patchify(int32_t dtype, const void* frames, const int64_t* item_offsets, const int32_t* grid_thw,
                    const int32_t* cu_seqlens, int32_t n_images, int64_t T, void* patches, int64_t ld,
                    int32_t in_channels, int32_t patch, int32_t temporal_patch, const float* mean, const float* inv_std,
                    void* stream) {
  return epd_op_patchify_fmt(dtype, EPD_FRAMES_U8, frames, item_offsets, grid_thw, cu_seqlens, n_images, T, patches, ld,
                             in_channels, patch, temporal_patch, mean, inv_std, stream);
}

int epd_op_merge(int32_t dtype, const void* y, const int32_t* merge_idx, void* out, int64_t Tm, int32_t hidden,
                 void* stream) {
  if (dtype != EPD_DTYPE_F32 && dtype != EPD_DTYPE_BF16) return EPD_EINVAL;
  if (Tm < 0 || hidden < 1) return EPD_EINVAL;
  if (Tm == 0) return EPD_OK;
  if (!y || !merge_idx || !out) return EPD_EINVAL;
  EPD_CUDA(merge_gather(dtype, y, merge_idx, out, Tm, hidden, static_cast<cudaStream_t>(stream)));
  return EPD_OK;
}

}  // extern "C"
