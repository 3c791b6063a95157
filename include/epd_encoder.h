/*
 * epd_encoder.h -- C ABI of the Encode stage  V_m = E(I_m)  (Section 3.1 "Encode Stage", Eq. 1).
 *
 * E is a Vision Transformer: a packed batch of images / video clips, given as pixel patches
 * plus one (t, h, w) patch grid per item, is turned into one contiguous [n, d] feature
 * matrix per item -- the tensor that crosses the Encode -> Prefill boundary (Section 3.1
 * "Cross-Stage Transmission"; the [n, 3584] tensors of the E-P prefetching table, Section 4).
 * The call is stateless per request, so the fault-tolerant recomputation of Section 3.2 is
 * simply calling it again.
 *
 * Conventions
 *   - Every function returns an epd_status_t (0 = OK, < 0 = error); nothing throws, aborts or
 *     prints.  epd_strerror() names a code.
 *   - "device" pointers are CUDA global-memory addresses on the current device, "HOST"
 *     pointers are ordinary process memory.  All matrices are row-major.  Weight matrices
 *     are [out_features, in_features] (the contraction dimension is contiguous).
 *   - dtype EPD_DTYPE_F32: activations, weights and features are float.
 *     dtype EPD_DTYPE_BF16: weights, patches and features are bfloat16, all contractions
 *     accumulate in float and the residual stream is kept in float.
 *   - All work is enqueued on the given cudaStream_t and the call returns without
 *     synchronising, unless stated otherwise.  The library never allocates device memory
 *     after epd_encoder_create(): activations live in the caller-provided workspace.
 *   - One encode may be in flight per encoder object (the workspace is per encoder).
 *   - The CUDA device current at create time must be current for every later call.
 */
#ifndef EPD_ENCODER_H_
#define EPD_ENCODER_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct epd_encoder epd_encoder_t;

typedef enum {
  EPD_OK = 0,
  EPD_EINVAL = -1,       /* NULL / misaligned pointer, bad size, inconsistent configuration */
  EPD_ENOMEM = -2,       /* workspace too small, host allocation failed */
  EPD_ECUDA = -3,        /* a CUDA runtime / driver call failed */
  EPD_ECAPACITY = -4,    /* batch exceeds max_tokens / max_images / the feature buffer */
  EPD_EUNSUPPORTED = -5, /* shape the kernels do not cover */
  EPD_ETIMEOUT = -6      /* a bounded device-side wait expired (reported by epd_encoder_last_status) */
} epd_status_t;

enum { EPD_DTYPE_F32 = 0, EPD_DTYPE_BF16 = 1 };
enum { EPD_ACT_GELU_TANH = 0, EPD_ACT_GELU_ERF = 1 };
enum { EPD_PROJ_LINEAR = 0, EPD_PROJ_MLP = 1 };
enum { EPD_FRAMES_U8 = 0, EPD_FRAMES_BF16 = 1 };   /* element type of raw frames; both on the 0..255 scale */

/* Static description of the encoder E of Eq. 1. */
typedef struct {
  int32_t dtype;          /* EPD_DTYPE_* */
  int32_t in_channels;    /* C */
  int32_t patch;          /* P: patch side in pixels */
  int32_t temporal_patch; /* Tp: frames folded into one patch; patch vector length K = C*Tp*P*P */
  int32_t hidden;         /* h */
  int32_t layers;         /* L */
  int32_t heads;          /* heads * head_dim == hidden */
  int32_t head_dim;       /* multiple of 4 (2-D rotary pairs), <= 128 */
  int32_t mlp;            /* MLP width m */
  int32_t act;            /* EPD_ACT_* (MLP and projector) */
  float eps;              /* RMSNorm epsilon (inside the square root) */
  float rope_theta;       /* rotary base; <= 0 disables the rotary embedding */
  int32_t merge;          /* spatial merge factor; must be 2 */
  int32_t final_norm;     /* 1: RMSNorm before the merge */
  int32_t proj_kind;      /* EPD_PROJ_* */
  int32_t proj_hidden;    /* width of the projector's hidden layer (EPD_PROJ_MLP) */
  int32_t out_dim;        /* d of Eq. 1 */
  int64_t max_tokens;     /* capacity: largest packed token count T of one call */
  int32_t max_images;     /* capacity: largest number of items of one call */
  int32_t max_grid;       /* capacity: largest h or w of any grid (rotary table rows) */
} epd_config_t;

/*
 * Encoder parameters: device pointers, borrowed for the lifetime of the encoder (the caller
 * keeps them alive and unchanged).  Per-layer entries are HOST arrays of `layers` device
 * pointers.  Any bias pointer may be NULL (no bias).  Matrix rows are contiguous
 * (leading dimension == in_features) except patch_w, whose leading dimension is patch_w_ld.
 * In EPD_DTYPE_BF16 every leading dimension must be a multiple of 8 elements.
 */
typedef struct {
  const void* patch_w;      /* [hidden, patch_w_ld], first K columns used */
  int64_t patch_w_ld;       /* >= K */
  const void* patch_b;      /* [hidden] */
  const void* const* norm1_w; /* [L] -> [hidden] gains */
  const void* const* qkv_w;   /* [L] -> [3*hidden, hidden]; rows 0..h-1 = q, h..2h-1 = k, 2h..3h-1 = v */
  const void* const* qkv_b;   /* [L] -> [3*hidden] */
  const void* const* out_w;   /* [L] -> [hidden, hidden] */
  const void* const* out_b;   /* [L] -> [hidden] */
  const void* const* norm2_w; /* [L] -> [hidden] */
  const void* const* fc1_w;   /* [L] -> [mlp, hidden] */
  const void* const* fc1_b;   /* [L] -> [mlp] */
  const void* const* fc2_w;   /* [L] -> [hidden, mlp] */
  const void* const* fc2_b;   /* [L] -> [hidden] */
  const void* final_norm_w;   /* [hidden]; ignored when final_norm == 0 */
  const void* proj_w1;        /* LINEAR: [out_dim, 4*hidden]; MLP: [proj_hidden, 4*hidden] */
  const void* proj_b1;
  const void* proj_w2;        /* MLP: [out_dim, proj_hidden]; LINEAR: NULL */
  const void* proj_b2;
} epd_weights_t;

/* ------------------------------------------------------------------------------------------
 * Encoder object
 * ---------------------------------------------------------------------------------------- */

/* Bytes of device workspace epd_encoder_create() needs for this configuration (0 on a bad config). */
size_t epd_encoder_workspace_bytes(const epd_config_t* cfg);

/*
 * Build an encoder.  `workspace` is device memory of at least epd_encoder_workspace_bytes(cfg)
 * bytes, 256-byte aligned, owned by the caller and reserved for this encoder until destroy.
 * Synchronous: builds the rotary table on the device and returns after it is ready.
 * Weights are borrowed (they must stay valid and unchanged until destroy) with one exception: for bf16
 * configurations whose head_dim is a multiple of 8 the encoder keeps, inside the workspace, its own copy
 * of every layer's QKV weight and bias with the q and k rows reordered for the rotary epilogue; changing
 * those weights afterwards needs a new encoder.
 * Errors: EPD_EINVAL (bad config / NULL / alignment), EPD_ENOMEM (workspace too small),
 * EPD_EUNSUPPORTED, EPD_ECUDA.
 */
int epd_encoder_create(const epd_config_t* cfg, const epd_weights_t* weights, void* workspace,
                       size_t workspace_bytes, epd_encoder_t** out);

/*
 * The Encode stage (Eq. 1) for one packed batch.
 *   patches      device [T, patches_ld], element type per dtype; row j is the patch vector of
 *                token j, element order inside a patch (channel, temporal, y, x).  Tokens of
 *                item i occupy rows cu[i]..cu[i+1], raster order (frame, row, col).
 *                16-byte aligned; in bf16 patches_ld must be a multiple of 8.
 *   grid_thw     HOST [n_images, 3] = (t, h, w) of each item in patch units; t,h,w >= 1 and
 *                h, w even.  An item with t > 1 is a clip: attention spans all its frames.
 *   features     device [features_capacity_rows, out_dim], caller-owned E->P buffer.  Item i's
 *                feature matrix V_m is rows out_cu_rows[i]..out_cu_rows[i+1], merged tokens in
 *                (frame, row/2, col/2) raster order, each row = projector(concat of the 2x2
 *                neighbours (dy,dx) = (0,0),(0,1),(1,0),(1,1)).
 *   out_rows     HOST, optional: total feature rows written (T/4).
 *   out_cu_rows  HOST [n_images+1], optional: prefix sums of per-item feature rows.
 *   stream       cudaStream_t (NULL = legacy default stream).
 * Every argument is validated on the host before anything is enqueued (no copy, no kernel): a call that
 * returns EPD_EINVAL or EPD_ECAPACITY has touched neither the stream nor the workspace, and
 * epd_encoder_last_launch_count() is 0 after it.  Host outputs are filled synchronously (they depend on
 * grid_thw only).  n_images == 0 is valid and launches nothing.  The same holds for the host-buffer and
 * raw-frame forms below.
 * Errors: EPD_EINVAL, EPD_ECAPACITY, EPD_ECUDA.
 */
int epd_encode(epd_encoder_t* enc, const void* patches, int64_t patches_ld, const int32_t* grid_thw,
               int32_t n_images, void* features, int64_t features_capacity_rows, int64_t* out_rows,
               int32_t* out_cu_rows, void* stream);

/*
 * Same stage with HOST patches and a HOST feature buffer (both should be page-locked for the
 * copies to be asynchronous): copies patches to a staging area inside the workspace, encodes,
 * copies the features back, all on `stream`.  Returns without synchronising; the features are
 * valid after the stream is synchronised.  patches_ld == K here.
 */
int epd_encode_host(epd_encoder_t* enc, const void* host_patches, const int32_t* grid_thw,
                    int32_t n_images, void* host_features, int64_t features_capacity_rows,
                    int64_t* out_rows, int32_t* out_cu_rows, void* stream);

/*
 * Pipelined form of epd_encode_host for a loop of requests: the host-to-device copy of the patches, the
 * encode and the device-to-host copy of the features of one call run on three streams (the copies on two
 * streams the encoder creates on first use, the encode on `stream`), with two staging slots in the
 * workspace, so that the copies of neighbouring calls overlap the encodes: H2D(i+1) and D2H(i-1) run during
 * encode(i).  Ordering is by events only; the call does not block the host.
 *   host_patches of a call must stay unchanged until its copy has run, host_features are valid once work
 *   enqueued after epd_encode_host_join(enc, stream) on `stream` runs (e.g. after joining and synchronising
 *   the stream), or after a device-wide synchronisation.  Both should be page-locked.
 * epd_encode_host_join makes `stream` wait for the feature copies of all earlier calls (no host wait).
 */
int epd_encode_host_async(epd_encoder_t* enc, const void* host_patches, const int32_t* grid_thw, int32_t n_images,
                          void* host_features, int64_t features_capacity_rows, int64_t* out_rows,
                          int32_t* out_cu_rows, void* stream);
int epd_encode_host_join(epd_encoder_t* enc, void* stream);

/*
 * The same stage fed with raw pixels: the step immediately in front of Eq. 1's E.  `frames` is a
 * device buffer holding the items back to back, item i as [t*Tp, C, h*P, w*P]
 * (frame, channel, y, x; t, h, w from grid_thw, Tp = temporal_patch, P = patch, C = in_channels <= 4), elements
 * uint8 (epd_encode_frames, and frame_format EPD_FRAMES_U8) or bfloat16 on the same 0..255 scale
 * (EPD_FRAMES_BF16, e.g. the output of a resize that keeps fractions).
 * Pixel v of channel c becomes (v/255 - mean[c]) * inv_std[c] (mean, inv_std: HOST arrays of C floats)
 * and token (frame f, row r, column c) gathers its patch in element order (channel, temporal, y, x)
 * -- the patch matrix epd_encode() takes -- in a buffer inside the workspace; then the stage runs as
 * in epd_encode().  Resizing images to a multiple of the patch size is preprocessing and stays with
 * the caller.  Errors as epd_encode(), plus EPD_EUNSUPPORTED for more than 4 channels.
 */
int epd_encode_frames(epd_encoder_t* enc, const void* frames, const int32_t* grid_thw, int32_t n_images,
                      const float* mean, const float* inv_std, void* features, int64_t features_capacity_rows,
                      int64_t* out_rows, int32_t* out_cu_rows, void* stream);
int epd_encode_frames_fmt(epd_encoder_t* enc, const void* frames, int32_t frame_format, const int32_t* grid_thw,
                          int32_t n_images, const float* mean, const float* inv_std, void* features,
                          int64_t features_capacity_rows, int64_t* out_rows, int32_t* out_cu_rows, void* stream);

/*
 * epd_encode_frames() behind a feature cache (Section 3.2: features are stored under a hash of the input, so a
 * repeated input is not encoded again).  The items' content keys are computed on the device
 * (epd_op_content_hash over each item's frame bytes, whose size must be a multiple of 8) and read back -- the
 * one point where this call waits for the stream; items whose key (with the same row count) is cached are
 * copied from the cache to their rows of `features`; the others are encoded as one batch, the first occurrence
 * of every distinct key only, copied to their rows and inserted into the cache (an item larger than the whole
 * pool is returned but not cached).  `features` ends up exactly as epd_encode_frames() would leave it.
 *   out_keys  HOST [n_images], optional: the content keys.
 *   out_hit   HOST [n_images], optional: 1 where the item came from the cache.
 * The cache must be used with this one stream (see epd_feature_cache_insert).
 */
typedef struct epd_feature_cache epd_feature_cache_t;
int epd_encode_frames_cached(epd_encoder_t* enc, epd_feature_cache_t* cache, const void* frames,
                             const int32_t* grid_thw, int32_t n_images, const float* mean, const float* inv_std,
                             void* features, int64_t features_capacity_rows, int64_t* out_rows, int32_t* out_cu_rows,
                             uint64_t* out_keys, uint8_t* out_hit, void* stream);

/* Reads the encoder's device status word: EPD_OK or the first device-side error (EPD_ETIMEOUT), then clears
 * it.  Blocks the calling host thread until the encoder's own most recent work has finished (an event recorded
 * behind its last launch) and reads the word on a non-blocking stream of the encoder's; it does not
 * synchronise the device, so other streams -- a co-located stage -- keep running. */
int epd_encoder_last_status(epd_encoder_t* enc);

/* Number of kernels the last epd_encode() call launched. */
int64_t epd_encoder_last_launch_count(const epd_encoder_t* enc);

/* 1 if the encoder runs its contractions on the tcgen05 tensor-core kernels, 0 if on the
 * plain-FMA kernels (EPD_DTYPE_F32 always does). */
int epd_encoder_uses_tensor_cores(const epd_encoder_t* enc);

int epd_encoder_destroy(epd_encoder_t* enc);

const char* epd_strerror(int status);

/* Name of the CUDA runtime error behind the calling thread's most recent EPD_ECUDA return
 * ("cudaSuccess" if there was none): a diagnostic aid, the string is static. */
const char* epd_last_cuda_error(void);

/* ------------------------------------------------------------------------------------------
 * Test hooks on an encoder
 * ---------------------------------------------------------------------------------------- */

/* Copies the integer layout of the LAST encoded batch back to HOST arrays (synchronises):
 * cu_seqlens [n+1], pos_row [T], pos_col [T], merge_idx [T/4, 4] (source token of each merged
 * slot).  Any pointer may be NULL. */
int epd_debug_bookkeeping(epd_encoder_t* enc, int32_t* cu_seqlens, int32_t* pos_row, int32_t* pos_col,
                          int32_t* merge_idx);

/* `taps` is a HOST array of layers+1 device pointers (or NULL to clear).  During later encodes,
 * a non-NULL taps[l] receives the float residual stream [T, hidden] entering block l
 * (l == layers: leaving the last block). */
int epd_debug_set_taps(epd_encoder_t* enc, void* const* taps);

/* Runs only block `layer` (steps RMSNorm..MLP of one layer) on a caller-supplied residual
 * stream x (device float [T, hidden], updated in place) for the given grids. */
int epd_debug_run_block(epd_encoder_t* enc, int32_t layer, void* x, const int32_t* grid_thw,
                        int32_t n_images, void* stream);

/* A repeated request - same grid list, same patch and feature buffers, same SM budget - replays the launch
 * sequence captured as a CUDA graph on its previous occurrence (up to 8 graphs are kept, oldest dropped):
 * one graph launch instead of ~190 kernel launches, which matters for small batches, whose latency is
 * otherwise bound by the host's launch rate.  Needs a capturable stream (not the legacy default stream) that
 * is not itself being captured; otherwise, and with taps or profiling on, the kernels are launched one by
 * one.  epd_debug_use_graphs(enc, 0) switches the mechanism off; epd_debug_graph_count returns how many graphs
 * the encoder holds. */
int epd_debug_use_graphs(epd_encoder_t* enc, int32_t enable);
int32_t epd_debug_graph_count(const epd_encoder_t* enc);

/* Cycle limit of every bounded device-side wait of kernels launched after the call (process-wide); cycles <= 0
 * restores the default (about 2 s).  A wait that exceeds the limit gives up: the kernel records EPD_ETIMEOUT in
 * the encoder's status word, lets what it has in flight complete, frees its tensor memory and returns; its
 * output is then undefined and epd_encoder_last_status() reports the code.  A test hook: a limit of a few
 * thousand cycles makes ordinary waits (a first tile still on its way from memory) expire, which exercises that
 * path without anything being made to hang or fault. */
int epd_debug_set_wait_limit(int64_t cycles);

/* Per-step timing of the next encodes: with enable != 0 every launch of epd_encode() is bracketed
 * by CUDA events on the launching stream (this costs a few microseconds per launch, so it is
 * meant for a separate measuring pass).  epd_debug_profile_read() synchronises on the last event
 * and fills ms[c] / launches[c] (HOST arrays of epd_debug_profile_classes() entries) with the
 * device time and launch count of step class c of the most recent encode;
 * epd_debug_profile_class_name(c) names the class ("qkv_linear", "attention", ...). */
int epd_debug_profile(epd_encoder_t* enc, int32_t enable);
int32_t epd_debug_profile_classes(void);
const char* epd_debug_profile_class_name(int32_t cls);
int epd_debug_profile_read(epd_encoder_t* enc, float* ms, int64_t* launches);

/* ------------------------------------------------------------------------------------------
 * Single steps of the path (each is what the encoder itself launches)
 * ---------------------------------------------------------------------------------------- */

enum {
  EPD_LINEAR_GELU_TANH = 1,  /* apply tanh-GELU after the bias */
  EPD_LINEAR_GELU_ERF = 2,   /* apply erf-GELU after the bias */
  EPD_LINEAR_ACCUMULATE = 4, /* out (float) += result: the residual update */
  EPD_LINEAR_OUT_F32 = 8,    /* out is float even when dtype is bf16 */
  EPD_LINEAR_FORCE_FMA = 16, /* use the plain-FMA kernel even where the tensor-core kernel applies */
  EPD_LINEAR_TILE_N_SHIFT = 8 /* bits 8..16: tensor-core tile width override (0 = automatic; 128, 192, 256) */
};

/* out[M,N] = act(x[M,K] . w[N,K]^T + bias[N]) (optionally accumulated into a float out).
 * x, w: element type per dtype, leading dimensions ldx, ldw (elements); out: leading dimension
 * ldo.  All device pointers, 16-byte aligned.  In bf16 the tcgen05 kernel is used when every
 * leading dimension and N are multiples of 8; other shapes run on the plain-FMA kernel. */
int epd_op_linear(int32_t dtype, const void* x, int64_t ldx, const void* w, int64_t ldw, const void* bias,
                  void* out, int64_t ldo, int64_t M, int64_t N, int64_t K, int32_t flags, void* stream);

/* The same layer with 8-bit floating-point operands, a variant beside the bf16 path (Section 3.5 names the
 * operator mix of the stages; the paper states no precision).  Format E4M3: 4 exponent bits with bias 7, 3
 * mantissa bits, largest finite value 448, no infinities.
 * epd_op_quantize_e4m3: x bf16 [M, K] (leading dimension ldx, a multiple of 8) -> q bytes [M, ldq] (ldq a multiple
 *   of 16, padding bytes zeroed) and scale float [M]:  scale[i] = max_j |x[i,j]| / 448 (1 for an all-zero row),
 *   q[i,j] = the E4M3 value nearest to x[i,j] / scale[i] (ties to even, saturating); both divisions are IEEE float
 *   divisions.  Used for activations (one scale per token) and, once, for weights (one scale per output feature).
 * epd_op_linear_e4m3: out[M,N] = act((xq . wq^T) * x_scale * w_scale^T + bias), xq [M, K] and wq [N, K] byte codes,
 *   products exact and summed in float on the tensor cores (tcgen05.mma kind::f8f6f4); bias bf16 or NULL; out bf16,
 *   or float with EPD_LINEAR_OUT_F32; the GELU flags apply; EPD_LINEAR_ACCUMULATE is not offered.  All pointers
 *   device, 16-byte aligned; N a multiple of 8. */
int epd_op_quantize_e4m3(const void* x, int64_t ldx, void* q, int64_t ldq, float* scale, int64_t M, int64_t K,
                         void* stream);
int epd_op_linear_e4m3(const void* xq, int64_t ldx, const float* x_scale, const void* wq, int64_t ldw,
                       const float* w_scale, const void* bias, void* out, int64_t ldo, int64_t M, int64_t N, int64_t K,
                       int32_t flags, void* stream);

/* out[j,:] = x[j,:] / sqrt(mean(x[j,:]^2) + eps) * gain, x float [T, hidden], out per dtype.
 * If dst_row != NULL (device int32 [T]) row j is written at element offset dst_row[j]*hidden
 * instead of j*hidden (used to fuse the 2x2 merge into the final norm). */
int epd_op_rmsnorm(int32_t dtype, const void* x, const void* gain, void* out, const int32_t* dst_row,
                   int64_t T, int32_t hidden, float eps, void* stream);

/* Rotary embedding + head split.  qkv [T, 3*hidden] per dtype -> q, k, v each
 * [heads, T, head_dim_padded] per dtype (head_dim_padded = epd_padded_head_dim(head_dim); pad
 * columns zero, except that column head_dim of v is 1 when there is padding: the attention
 * step's P.V product then also delivers the softmax row sums).  q and k are rotated by (pos_row, pos_col) (device int32 [T]); q is also
 * multiplied by q_scale.  theta <= 0 skips the rotation. */
int epd_op_rope_split(int32_t dtype, const void* qkv, const int32_t* pos_row, const int32_t* pos_col,
                      void* q, void* k, void* v, int64_t T, int32_t heads, int32_t head_dim, float theta,
                      float q_scale, void* stream);

int32_t epd_padded_head_dim(int32_t head_dim);

/* The fused form of "QKV projection, rotary embedding, head split" that the encoder uses for bf16
 * batches of more than 128 tokens (head_dim a multiple of 8): the rotation runs in the projection's
 * epilogue on the fp32 accumulators, so the [T, 3*hidden] intermediate is never written.
 *
 * epd_op_qkv_prepare: w [3*hidden, hidden] (leading dimension ldw, a multiple of 8), bias [3*hidden] or
 *   NULL -> w_prepared [3*hidden, hidden] contiguous, bias_prepared [3*hidden]: the q and k rows
 *   reordered inside each head so that position 2p holds the first member of rotation pair p and 2p+1
 *   its partner (pairs of the row half first, then the column half); v rows unchanged.  q.k^T does not
 *   depend on the order of the head dimensions as long as q and k share it.
 * epd_op_rope_table: table float [rows, head_dim/4, 2] = (cos, sin)(p * theta^(-2f/(head_dim/2))) for
 *   position p < rows and frequency f, evaluated in double precision.
 * epd_op_qkv_pad_init: writes the padding columns of q, k, v [rows, head_dim_padded] (zeros; 1 in v's
 *   first padding column).  Needed once per buffer: epd_op_qkv_rope never writes them.
 * epd_op_qkv_rope: x bf16 [T, hidden] (leading dimension ldx) -> q, k, v bf16
 *   [heads, T, head_dim_padded]; q additionally multiplied by q_scale; q and k keep the prepared
 *   (pair) order of their head dimensions, v the natural one.  pos_row / pos_col device int32 [T] with
 *   values < table_rows.  All pointers device, 16-byte aligned.  EPD_EINVAL for other dtypes or
 *   head_dim not a multiple of 8. */
int epd_op_qkv_prepare(const void* w, int64_t ldw, const void* bias, void* w_prepared, void* bias_prepared,
                       int32_t heads, int32_t head_dim, void* stream);
int epd_op_rope_table(float* table, int32_t rows, int32_t head_dim, float theta, void* stream);
int epd_op_qkv_pad_init(void* q, void* k, void* v, int64_t rows, int32_t head_dim, void* stream);
int epd_op_qkv_rope(const void* x, int64_t ldx, const void* w_prepared, const void* bias_prepared,
                    const int32_t* pos_row, const int32_t* pos_col, const float* table, int32_t table_rows,
                    void* q, void* k, void* v, int64_t T, int32_t heads, int32_t head_dim, float q_scale,
                    void* stream);

enum {
  EPD_ATTENTION_FORCE_FMA = 1,        /* use the plain-FMA kernel even where a tensor-core kernel applies */
  EPD_ATTENTION_SPLIT_KEYS = 2,       /* force the tensor-core kernel that gives one query tile to both softmax
                                         warpgroups (alternate key tiles, merged at the end) */
  EPD_ATTENTION_TWO_QUERY_TILES = 4   /* force the tensor-core kernel with two query tiles per CTA sharing every
                                         K / V tile; without either flag this kernel runs wherever it applies
                                         (the choice depends on the head width only, never on the batch) */
};

/* Block-diagonal bidirectional attention.  q, k, v [heads, T, head_dim_padded] per dtype as written
 * by epd_op_rope_split(): q already multiplied by log2(e)/sqrt(head_dim), pad columns zero except
 * v[.., head_dim] = 1 when head_dim_padded > head_dim (required by the tensor-core kernel); cu_seqlens device int32 [n_seg+1] and the same
 * values in HOST memory (host_cu_seqlens) for the launch geometry.  out [T, heads*head_dim] per
 * dtype: for each segment and head softmax over all keys of the segment.  In bf16 with head_dim 64,
 * 72 or 128 (a multiple of 8 whose padded width is 64, 80 or 128) the tcgen05 kernel runs; other
 * shapes, and flags & EPD_ATTENTION_FORCE_FMA, use the plain-FMA kernel. */
int epd_op_attention(int32_t dtype, const void* q, const void* k, const void* v, const int32_t* cu_seqlens,
                     const int32_t* host_cu_seqlens, int32_t n_seg, void* out, int64_t T, int32_t heads,
                     int32_t head_dim, int32_t flags, void* stream);

/* Pixels -> patch vectors (the front end of epd_encode_frames()).  frames: device uint8 as described
 * there (epd_op_patchify) or in the given frame_format (epd_op_patchify_fmt); item_offsets: device int64
 * [n_images+1] BYTE offsets of the items inside frames; grid_thw: device int32 [n_images, 3]; cu_seqlens: device
 * int32 [n_images+1]; patches: device [T, ld] per dtype, ld >= C*Tp*P*P (columns beyond are zeroed); mean,
 * inv_std: HOST arrays of in_channels floats. */
int epd_op_patchify(int32_t dtype, const void* frames, const int64_t* item_offsets, const int32_t* grid_thw,
                    const int32_t* cu_seqlens, int32_t n_images, int64_t T, void* patches, int64_t ld,
                    int32_t in_channels, int32_t patch, int32_t temporal_patch, const float* mean, const float* inv_std,
                    void* stream);
int epd_op_patchify_fmt(int32_t dtype, int32_t frame_format, const void* frames, const int64_t* item_offsets,
                        const int32_t* grid_thw, const int32_t* cu_seqlens, int32_t n_images, int64_t T, void* patches,
                        int64_t ld, int32_t in_channels, int32_t patch, int32_t temporal_patch, const float* mean,
                        const float* inv_std, void* stream);

/* out[o, q*hidden:(q+1)*hidden] = y[merge_idx[o*4+q], :], y [T, hidden], out [T/4, 4*hidden] per dtype. */
int epd_op_merge(int32_t dtype, const void* y, const int32_t* merge_idx, void* out, int64_t Tm,
                 int32_t hidden, void* stream);

/* ------------------------------------------------------------------------------------------
 * After the stage: feature keys and a feature cache (the encoder's side of the multimodal store of
 * Section 3.2, "Asynchronous Feature Prefetching": features are kept under a hash of the input so
 * that a repeated input is not encoded again and only the key travels with the request)
 * ---------------------------------------------------------------------------------------- */

/* 64-bit content key of each item.  data: device bytes (8-byte aligned); item_offsets: device int64
 * [n_items+1] byte offsets of the items inside data, multiples of 8; hashes: device uint64 [n_items].
 * With w_1..w_n the item's bytes as little-endian 64-bit words and mix the SplitMix64 finalizer,
 *   key = mix( (sum_k mix(w_k xor k*0x9E3779B97F4A7C15)) + 8n )  mod 2^64.
 * Enqueued on the stream (a memset and two kernels); bit-exact whatever the launch geometry. */
int epd_op_content_hash(const void* data, const int64_t* item_offsets, int32_t n_items, uint64_t* hashes,
                        void* stream);

/* A cache of feature matrices by key inside `pool` (device memory, 256-byte aligned, owned by the
 * caller and reserved for the cache until destroy).  row_bytes = out_dim * sizeof(element).  The index
 * lives on the host; entries are evicted first-in-first-out when the pool wraps.  Not thread-safe. */
int epd_feature_cache_create(void* pool, size_t pool_bytes, size_t row_bytes, epd_feature_cache_t** out);
int epd_feature_cache_destroy(epd_feature_cache_t* cache);
/* Returns EPD_OK on a hit (and, if dst != NULL, enqueues the copy of the `rows` feature rows to dst on
 * the stream), 1 on a miss (no entry with this key and row count), < 0 on error. */
int epd_feature_cache_lookup(epd_feature_cache_t* cache, uint64_t key, int64_t rows, void* dst, void* stream);
/* Enqueues the copy of `rows` feature rows from src (device) into the pool and records them under
 * key; evicts the oldest entries if room is needed.  A key that is already cached with the same row count is
 * left as it is; with another row count the old entry is dropped and the new one stored.  EPD_ECAPACITY if the
 * rows can never fit.  The copies are ordered by the stream only: use ONE stream for all lookups and inserts of a
 * cache (an eviction lets a later insert overwrite pool bytes that a lookup's copy on another stream may still
 * be reading). */
int epd_feature_cache_insert(epd_feature_cache_t* cache, uint64_t key, int64_t rows, const void* src, void* stream);
int epd_feature_cache_stats(const epd_feature_cache_t* cache, int64_t* hits, int64_t* misses, int64_t* evictions,
                            int64_t* entries);

/* ------------------------------------------------------------------------------------------
 * Sharing the GPU with another stage (Section 3.5 "Physical Co-location"; Section 3.2 asynchronous
 * prefetch)
 * ---------------------------------------------------------------------------------------- */

/* SM budget: the persistent kernels of this library (linear layers, attention) launch at most n_sms CTAs
 * (0 = every SM, the default), leaving the other SMs to kernels of a co-located stage on another stream or
 * in another process.  Process-wide; applies to launches made after the call.  Results do not depend on
 * it (the same tiles are computed, by fewer CTAs).  The short non-persistent kernels (RMSNorm, patchify,
 * layout) are not limited. */
int epd_set_sm_limit(int32_t n_sms);
int32_t epd_get_sm_limit(void);

/* Enqueues a one-thread kernel that stores `value` to *flag (device memory, or host memory mapped into the
 * device's address space) with system-scope release semantics once everything enqueued on the stream
 * before it has completed: a consumer that polls the flag, or waits on it with a stream memory
 * operation, may then read the features written by a preceding epd_encode* call. */
int epd_signal_ready(uint32_t* flag, uint32_t value, void* stream);

/* Memory-bound stand-in for a Decode step, for co-location measurements only: n_ctas persistent CTAs
 * stream `bytes` of device memory `passes` times with 16-byte loads; cta_sums (device uint64 [n_ctas],
 * zeroed by the caller) receives checksums so the loads cannot be elided. */
int epd_op_stream_read(const void* data, int64_t bytes, int32_t passes, int32_t n_ctas, uint64_t* cta_sums,
                       void* stream);

/* ------------------------------------------------------------------------------------------
 * Allocation-free variant (the paper has no counterpart: this is a convenience of this library)
 * ---------------------------------------------------------------------------------------- */

/*
 * Rotary embedding + head split + block-diagonal attention on a packed qkv matrix, for callers
 * that cannot allocate device memory: a process whose own pool already owns all of HBM (so
 * cudaMalloc fails), or a latency-critical loop that must avoid the device-wide synchronisation
 * an allocation can trigger.  It computes what epd_op_rope_split() followed by epd_op_attention()
 * computes (q scaled by log2(e)/sqrt(head_dim)), but the head-major q, k, v intermediates live in
 * a fixed array inside the library's device image instead of caller-provided buffers; the call
 * performs no cudaMalloc / cudaFree and uses no allocating library routine.
 *   qkv [T, 3*heads*head_dim], out [T, heads*head_dim] per dtype; pos_row, pos_col, cu_seqlens
 *   device int32; host_cu_seqlens the same prefix sums in HOST memory.
 * Limits and caveats:
 *   - 3 * heads * T * epd_padded_head_dim(head_dim) * sizeof(element) (each third rounded up to
 *     256 bytes) must not exceed epd_static_scratch_bytes() (16 MiB); larger batches return
 *     EPD_ECAPACITY and launch nothing.
 *   - Every GPU that loads the library holds the array until the process exits.
 *   - The first call on a device looks up the array's device address (which may make the CUDA runtime load
 *     the library's device code on that GPU: the moment the 16 MiB are backed); make that first call
 *     outside any stream capture and outside latency-critical code.
 *   - heads <= 65535.  A bounded device-side wait that expires inside the attention kernel leaves `out`
 *     undefined; this entry point has no status word, such an expiry is not reported.
 *   - All calls on a device share the array: calls whose kernels can overlap on the GPU
 *     (different streams without ordering) race.  Nothing has to be cleared between calls: every
 *     element that is read, padding included, is rewritten first by the same call.
 */
int epd_op_rope_attention_static(int32_t dtype, const void* qkv, const int32_t* pos_row, const int32_t* pos_col,
                                 const int32_t* cu_seqlens, const int32_t* host_cu_seqlens, int32_t n_seg, void* out,
                                 int64_t T, int32_t heads, int32_t head_dim, float theta, void* stream);
size_t epd_static_scratch_bytes(void);

#ifdef __cplusplus
}
#endif
#endif /* EPD_ENCODER_H_ */
