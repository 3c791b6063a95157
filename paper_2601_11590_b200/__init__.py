"""Python binding of the Encode-stage C library (libepd_encoder.so).

Argument marshalling only: every step of the path runs in the library's CUDA kernels.
PyTorch supplies device memory and streams.  There is no CPU fallback: importing works
without a GPU (so the exported symbols can be inspected), but creating an encoder or calling
an op requires the compiled library and a CUDA device.
"""
from __future__ import annotations

import ctypes
import os
from typing import Dict, List, Optional, Sequence

import numpy as np

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libepd_encoder.so")

EPD_OK, EPD_EINVAL, EPD_ENOMEM, EPD_ECUDA, EPD_ECAPACITY, EPD_EUNSUPPORTED, EPD_ETIMEOUT = 0, -1, -2, -3, -4, -5, -6
DTYPE_F32, DTYPE_BF16 = 0, 1
LINEAR_GELU_TANH, LINEAR_GELU_ERF, LINEAR_ACCUMULATE, LINEAR_OUT_F32, LINEAR_FORCE_FMA = 1, 2, 4, 8, 16
FRAMES_U8, FRAMES_BF16 = 0, 1
ATTENTION_FORCE_FMA = 1
ATTENTION_SPLIT_KEYS = 2
ATTENTION_TWO_QUERY_TILES = 4

EXPORTED_SYMBOLS = [
    "epd_encoder_workspace_bytes", "epd_encoder_create", "epd_encode", "epd_encode_host",
    "epd_encode_host_async", "epd_encode_host_join", "epd_debug_use_graphs", "epd_debug_graph_count",
    "epd_encoder_last_status", "epd_encoder_last_launch_count", "epd_encoder_uses_tensor_cores",
    "epd_encoder_destroy", "epd_strerror", "epd_debug_bookkeeping", "epd_debug_set_taps",
    "epd_debug_run_block", "epd_debug_profile", "epd_debug_profile_classes",
    "epd_debug_profile_class_name", "epd_debug_profile_read", "epd_op_linear", "epd_op_rmsnorm", "epd_op_rope_split",
    "epd_padded_head_dim", "epd_op_attention", "epd_op_merge", "epd_op_rope_attention_static",
    "epd_static_scratch_bytes", "epd_last_cuda_error", "epd_encode_frames", "epd_op_patchify",
    "epd_op_qkv_prepare", "epd_op_rope_table", "epd_op_qkv_pad_init", "epd_op_qkv_rope",
    "epd_set_sm_limit", "epd_get_sm_limit", "epd_signal_ready", "epd_op_stream_read", "epd_op_content_hash", "epd_feature_cache_create", "epd_feature_cache_destroy",
    "epd_feature_cache_lookup", "epd_feature_cache_insert", "epd_feature_cache_stats",
    "epd_encode_frames_cached", "epd_debug_set_wait_limit", "epd_encode_frames_fmt", "epd_op_patchify_fmt",
    "epd_op_quantize_e4m3", "epd_op_linear_e4m3",
]


class EpdError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        detail = ""
        if status == EPD_ECUDA and _lib is not None:
            detail = " [" + _lib.epd_last_cuda_error().decode() + "]"
        super().__init__(f"{what}: {strerror(status)} ({status}){detail}")


class ConfigStruct(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("dtype", "in_channels", "patch", "temporal_patch", "hidden", "layers", "heads",
                 "head_dim", "mlp", "act")] + \
               [("eps", ctypes.c_float), ("rope_theta", ctypes.c_float)] + \
               [(n, ctypes.c_int32) for n in ("merge", "final_norm", "proj_kind", "proj_hidden", "out_dim")] + \
               [("max_tokens", ctypes.c_int64), ("max_images", ctypes.c_int32), ("max_grid", ctypes.c_int32)]


_PP = ctypes.POINTER(ctypes.c_void_p)


class WeightsStruct(ctypes.Structure):
    _fields_ = [("patch_w", ctypes.c_void_p), ("patch_w_ld", ctypes.c_int64), ("patch_b", ctypes.c_void_p)] + \
               [(n, _PP) for n in ("norm1_w", "qkv_w", "qkv_b", "out_w", "out_b", "norm2_w",
                                   "fc1_w", "fc1_b", "fc2_w", "fc2_b")] + \
               [(n, ctypes.c_void_p) for n in ("final_norm_w", "proj_w1", "proj_b1", "proj_w2", "proj_b2")]


_lib = None


def load_library() -> ctypes.CDLL:
    """dlopen the compiled library; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2601_11590_b200.build`")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, f32 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_float
    i32p, i64p = ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_int64)
    lib.epd_encoder_workspace_bytes.restype = ctypes.c_size_t
    lib.epd_encoder_workspace_bytes.argtypes = [ctypes.POINTER(ConfigStruct)]
    lib.epd_encoder_create.restype = ctypes.c_int
    lib.epd_encoder_create.argtypes = [ctypes.POINTER(ConfigStruct), ctypes.POINTER(WeightsStruct), vp,
                                       ctypes.c_size_t, ctypes.POINTER(vp)]
    lib.epd_encode.restype = ctypes.c_int
    lib.epd_encode.argtypes = [vp, vp, i64, i32p, i32, vp, i64, i64p, i32p, vp]
    lib.epd_encode_host.restype = ctypes.c_int
    lib.epd_encode_host.argtypes = [vp, vp, i32p, i32, vp, i64, i64p, i32p, vp]
    lib.epd_encode_host_async.restype = ctypes.c_int
    lib.epd_encode_host_async.argtypes = [vp, vp, i32p, i32, vp, i64, i64p, i32p, vp]
    lib.epd_encode_host_join.restype = ctypes.c_int
    lib.epd_encode_host_join.argtypes = [vp, vp]
    lib.epd_debug_use_graphs.restype = ctypes.c_int
    lib.epd_debug_use_graphs.argtypes = [vp, i32]
    lib.epd_debug_graph_count.restype = i32
    lib.epd_debug_graph_count.argtypes = [vp]
    lib.epd_encoder_last_status.restype = ctypes.c_int
    lib.epd_encoder_last_status.argtypes = [vp]
    f32p = ctypes.POINTER(ctypes.c_float)
    lib.epd_encode_frames.restype = ctypes.c_int
    lib.epd_encode_frames.argtypes = [vp, vp, i32p, i32, f32p, f32p, vp, i64, i64p, i32p, vp]
    lib.epd_encode_frames_cached.restype = ctypes.c_int
    lib.epd_encode_frames_cached.argtypes = [vp, vp, vp, i32p, i32, f32p, f32p, vp, i64, i64p, i32p,
                                             ctypes.POINTER(ctypes.c_uint64), ctypes.POINTER(ctypes.c_uint8), vp]
    lib.epd_debug_set_wait_limit.restype = ctypes.c_int
    lib.epd_debug_set_wait_limit.argtypes = [i64]
    lib.epd_op_patchify.restype = ctypes.c_int
    lib.epd_op_patchify.argtypes = [i32, vp, vp, vp, vp, i32, i64, vp, i64, i32, i32, i32, f32p, f32p, vp]
    lib.epd_op_quantize_e4m3.restype = ctypes.c_int
    lib.epd_op_quantize_e4m3.argtypes = [vp, i64, vp, i64, vp, i64, i64, vp]
    lib.epd_op_linear_e4m3.restype = ctypes.c_int
    lib.epd_op_linear_e4m3.argtypes = [vp, i64, vp, vp, i64, vp, vp, vp, i64, i64, i64, i64, i32, vp]
    lib.epd_op_patchify_fmt.restype = ctypes.c_int
    lib.epd_op_patchify_fmt.argtypes = [i32, i32, vp, vp, vp, vp, i32, i64, vp, i64, i32, i32, i32, f32p, f32p, vp]
    lib.epd_encode_frames_fmt.restype = ctypes.c_int
    lib.epd_encode_frames_fmt.argtypes = [vp, vp, i32, i32p, i32, f32p, f32p, vp, i64, i64p, i32p, vp]
    lib.epd_op_qkv_prepare.restype = ctypes.c_int
    lib.epd_op_qkv_prepare.argtypes = [vp, i64, vp, vp, vp, i32, i32, vp]
    lib.epd_op_rope_table.restype = ctypes.c_int
    lib.epd_op_rope_table.argtypes = [vp, i32, i32, ctypes.c_float, vp]
    lib.epd_op_qkv_pad_init.restype = ctypes.c_int
    lib.epd_op_qkv_pad_init.argtypes = [vp, vp, vp, i64, i32, vp]
    lib.epd_op_qkv_rope.restype = ctypes.c_int
    lib.epd_op_qkv_rope.argtypes = [vp, i64, vp, vp, vp, vp, vp, i32, vp, vp, vp, i64, i32, i32, ctypes.c_float, vp]
    lib.epd_set_sm_limit.restype = ctypes.c_int
    lib.epd_set_sm_limit.argtypes = [i32]
    lib.epd_get_sm_limit.restype = i32
    lib.epd_get_sm_limit.argtypes = []
    lib.epd_signal_ready.restype = ctypes.c_int
    lib.epd_signal_ready.argtypes = [vp, ctypes.c_uint32, vp]
    lib.epd_op_stream_read.restype = ctypes.c_int
    lib.epd_op_stream_read.argtypes = [vp, i64, i32, i32, vp, vp]
    lib.epd_op_content_hash.restype = ctypes.c_int
    lib.epd_op_content_hash.argtypes = [vp, vp, i32, vp, vp]
    lib.epd_feature_cache_create.restype = ctypes.c_int
    lib.epd_feature_cache_create.argtypes = [vp, ctypes.c_size_t, ctypes.c_size_t, ctypes.POINTER(vp)]
    lib.epd_feature_cache_destroy.restype = ctypes.c_int
    lib.epd_feature_cache_destroy.argtypes = [vp]
    lib.epd_feature_cache_lookup.restype = ctypes.c_int
    lib.epd_feature_cache_lookup.argtypes = [vp, ctypes.c_uint64, i64, vp, vp]
    lib.epd_feature_cache_insert.restype = ctypes.c_int
    lib.epd_feature_cache_insert.argtypes = [vp, ctypes.c_uint64, i64, vp, vp]
    lib.epd_feature_cache_stats.restype = ctypes.c_int
    lib.epd_feature_cache_stats.argtypes = [vp, i64p, i64p, i64p, i64p]
    lib.epd_encoder_last_launch_count.restype = ctypes.c_int64
    lib.epd_encoder_last_launch_count.argtypes = [vp]
    lib.epd_encoder_uses_tensor_cores.restype = ctypes.c_int
    lib.epd_encoder_uses_tensor_cores.argtypes = [vp]
    lib.epd_encoder_destroy.restype = ctypes.c_int
    lib.epd_encoder_destroy.argtypes = [vp]
    lib.epd_strerror.restype = ctypes.c_char_p
    lib.epd_strerror.argtypes = [ctypes.c_int]
    lib.epd_last_cuda_error.restype = ctypes.c_char_p
    lib.epd_last_cuda_error.argtypes = []
    lib.epd_debug_bookkeeping.restype = ctypes.c_int
    lib.epd_debug_bookkeeping.argtypes = [vp, i32p, i32p, i32p, i32p]
    lib.epd_debug_set_taps.restype = ctypes.c_int
    lib.epd_debug_set_taps.argtypes = [vp, _PP]
    lib.epd_debug_run_block.restype = ctypes.c_int
    lib.epd_debug_run_block.argtypes = [vp, i32, vp, i32p, i32, vp]
    lib.epd_debug_profile.restype = ctypes.c_int
    lib.epd_debug_profile.argtypes = [vp, i32]
    lib.epd_debug_profile_classes.restype = i32
    lib.epd_debug_profile_classes.argtypes = []
    lib.epd_debug_profile_class_name.restype = ctypes.c_char_p
    lib.epd_debug_profile_class_name.argtypes = [i32]
    lib.epd_debug_profile_read.restype = ctypes.c_int
    lib.epd_debug_profile_read.argtypes = [vp, ctypes.POINTER(ctypes.c_float), i64p]
    lib.epd_op_linear.restype = ctypes.c_int
    lib.epd_op_linear.argtypes = [i32, vp, i64, vp, i64, vp, vp, i64, i64, i64, i64, i32, vp]
    lib.epd_op_rmsnorm.restype = ctypes.c_int
    lib.epd_op_rmsnorm.argtypes = [i32, vp, vp, vp, vp, i64, i32, f32, vp]
    lib.epd_op_rope_split.restype = ctypes.c_int
    lib.epd_op_rope_split.argtypes = [i32, vp, vp, vp, vp, vp, vp, i64, i32, i32, f32, f32, vp]
    lib.epd_padded_head_dim.restype = i32
    lib.epd_padded_head_dim.argtypes = [i32]
    lib.epd_op_attention.restype = ctypes.c_int
    lib.epd_op_attention.argtypes = [i32, vp, vp, vp, vp, i32p, i32, vp, i64, i32, i32, i32, vp]
    lib.epd_op_merge.restype = ctypes.c_int
    lib.epd_op_merge.argtypes = [i32, vp, vp, vp, i64, i32, vp]
    lib.epd_op_rope_attention_static.restype = ctypes.c_int
    lib.epd_op_rope_attention_static.argtypes = [i32, vp, vp, vp, vp, i32p, i32, vp, i64, i32, i32, f32, vp]
    lib.epd_static_scratch_bytes.restype = ctypes.c_size_t
    lib.epd_static_scratch_bytes.argtypes = []
    _lib = lib
    return lib


def strerror(status: int) -> str:
    return load_library().epd_strerror(int(status)).decode()


def _check(status: int, what: str) -> None:
    if status != EPD_OK:
        raise EpdError(status, what)


def _torch():
    import torch
    if not torch.cuda.is_available():
        raise RuntimeError("the Encode-stage library needs a CUDA device; there is no CPU path")
    return torch


def _stream_ptr(stream) -> int:
    torch = _torch()
    s = stream if stream is not None else torch.cuda.current_stream()
    return int(s.cuda_stream)


def _ptr(t) -> Optional[int]:
    return None if t is None else int(t.data_ptr())


def _i32_array(values: Sequence[int]):
    arr = np.ascontiguousarray(np.asarray(values, dtype=np.int32).reshape(-1))
    return arr, arr.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))


def torch_dtype(dtype: int):
    torch = _torch()
    return torch.float32 if dtype == DTYPE_F32 else torch.bfloat16


def to_device(arr: Optional[np.ndarray], dtype: int, device="cuda"):
    """float32 numpy values -> device tensor of the configuration's element type (exact for
    values already representable in it)."""
    if arr is None:
        return None
    torch = _torch()
    return torch.from_numpy(np.ascontiguousarray(arr, dtype=np.float32)).to(device=device, dtype=torch_dtype(dtype))


def make_config(cfg, max_tokens: int, max_images: int, max_grid: int) -> ConfigStruct:
    """cfg: any object with the fields of epd_config_t (e.g. synth.EncoderConfig)."""
    c = ConfigStruct()
    for name in ("dtype", "in_channels", "patch", "temporal_patch", "hidden", "layers", "heads", "head_dim",
                 "mlp", "act", "merge", "final_norm", "proj_kind", "proj_hidden", "out_dim"):
        setattr(c, name, int(getattr(cfg, name)))
    c.eps = float(cfg.eps)
    c.rope_theta = float(cfg.rope_theta)
    c.max_tokens, c.max_images, c.max_grid = int(max_tokens), int(max_images), int(max_grid)
    return c


class Encoder:
    """Owns one epd_encoder_t, its device weights (torch tensors) and its workspace."""

    def __init__(self, cfg, weights: Dict, max_tokens: int, max_images: int = 64, max_grid: int = 128,
                 device="cuda", patch_w_ld: Optional[int] = None):
        """weights: dict of float32 numpy arrays or device tensors laid out as synth.make_weights()."""
        torch = _torch()
        self.lib = load_library()
        self.cfg = cfg
        self.dtype = int(cfg.dtype)
        self.device = torch.device(device)
        self.max_tokens = int(max_tokens)
        self._c = make_config(cfg, max_tokens, max_images, max_grid)
        K = cfg.in_channels * cfg.temporal_patch * cfg.patch * cfg.patch
        self.patch_dim = K
        if patch_w_ld is None:
            patch_w_ld = K if self.dtype == DTYPE_F32 else (K + 7) // 8 * 8
        self.patch_w_ld = patch_w_ld

        def dev(a):
            if a is None:
                return None
            if isinstance(a, np.ndarray):
                return to_device(a, self.dtype, self.device)
            return a.to(device=self.device, dtype=torch_dtype(self.dtype)).contiguous()

        pw = dev(weights["patch_w"])
        if patch_w_ld != K:
            padded = torch.zeros((cfg.hidden, patch_w_ld), dtype=pw.dtype, device=self.device)
            padded[:, :K] = pw
            pw = padded
        self._keep = {"patch_w": pw, "patch_b": dev(weights["patch_b"]),
                      "final_norm_w": dev(weights.get("final_norm_w")),
                      "proj_w1": dev(weights["proj_w1"]), "proj_b1": dev(weights.get("proj_b1")),
                      "proj_w2": dev(weights.get("proj_w2")), "proj_b2": dev(weights.get("proj_b2"))}
        names = ("norm1_w", "qkv_w", "qkv_b", "out_w", "out_b", "norm2_w", "fc1_w", "fc1_b", "fc2_w", "fc2_b")
        self._layers: List[Dict] = [{n: dev(lw.get(n)) for n in names} for lw in weights["layers"]]
        assert len(self._layers) == cfg.layers
        w = WeightsStruct()
        w.patch_w, w.patch_w_ld, w.patch_b = _ptr(pw), patch_w_ld, _ptr(self._keep["patch_b"])
        self._arrays = {}
        for n in names:
            arr = (ctypes.c_void_p * max(1, cfg.layers))(*[_ptr(lw[n]) for lw in self._layers])
            self._arrays[n] = arr
            setattr(w, n, ctypes.cast(arr, _PP))
        for n in ("final_norm_w", "proj_w1", "proj_b1", "proj_w2", "proj_b2"):
            setattr(w, n, _ptr(self._keep[n]))
        nbytes = self.lib.epd_encoder_workspace_bytes(ctypes.byref(self._c))
        if nbytes == 0:
            raise EpdError(EPD_EINVAL, "epd_encoder_workspace_bytes")
        self.workspace_bytes = int(nbytes)
        self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
        base = (self.workspace.data_ptr() + 255) // 256 * 256
        handle = ctypes.c_void_p()
        with torch.cuda.device(self.device):
            _check(self.lib.epd_encoder_create(ctypes.byref(self._c), ctypes.byref(w), base, nbytes,
                                               ctypes.byref(handle)), "epd_encoder_create")
        self._h = handle
        self._taps = None

    # ---- the stage -------------------------------------------------------------------------
    def encode(self, patches, grid_thw, features=None, stream=None):
        """patches: device tensor [T, ld]; returns (features tensor [rows, out_dim], cu_rows ndarray)."""
        torch = _torch()
        g, gp = _i32_array(grid_thw)
        n = g.size // 3
        T = int(sum(int(g[3 * i]) * int(g[3 * i + 1]) * int(g[3 * i + 2]) for i in range(n)))
        if features is None:
            features = torch.empty((max(T // 4, 1), self.cfg.out_dim), dtype=torch_dtype(self.dtype),
                                   device=self.device)
        rows = ctypes.c_int64(0)
        cu_rows = np.zeros(n + 1, dtype=np.int32)
        ld = int(patches.stride(0)) if (patches is not None and patches.dim() == 2 and patches.shape[0] > 0) \
            else self.patch_dim
        _check(self.lib.epd_encode(self._h, _ptr(patches), ld, gp, n, _ptr(features), int(features.shape[0]),
                                   ctypes.byref(rows), cu_rows.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)),
                                   _stream_ptr(stream)), "epd_encode")
        return features[: rows.value], cu_rows

    def encode_frames(self, frames, grid_thw, mean, std, features=None, stream=None):
        """frames: device uint8 or bfloat16 tensor, the items' [t*Tp, C, H, W] frames back to back (flattened)."""
        torch = _torch()
        fmt = FRAMES_BF16 if frames.dtype == torch.bfloat16 else FRAMES_U8
        g, gp = _i32_array(grid_thw)
        n = g.size // 3
        T = int(sum(int(g[3 * i]) * int(g[3 * i + 1]) * int(g[3 * i + 2]) for i in range(n)))
        if features is None:
            features = torch.empty((max(T // 4, 1), self.cfg.out_dim), dtype=torch_dtype(self.dtype),
                                   device=self.device)
        rows = ctypes.c_int64(0)
        cu_rows = np.zeros(n + 1, dtype=np.int32)
        m = (ctypes.c_float * len(mean))(*[float(v) for v in mean])
        istd = (ctypes.c_float * len(std))(*[1.0 / float(v) for v in std])
        _check(self.lib.epd_encode_frames_fmt(self._h, _ptr(frames), fmt, gp, n, m, istd, _ptr(features),
                                              int(features.shape[0]), ctypes.byref(rows),
                                              cu_rows.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)),
                                              _stream_ptr(stream)), "epd_encode_frames_fmt")
        return features[: rows.value], cu_rows

    def encode_frames_cached(self, cache: "FeatureCache", frames, grid_thw, mean, std, features=None, stream=None):
        """encode_frames with a feature cache in front (epd_encode_frames_cached): items whose content key is
        cached are not encoded again.  Returns (list of per-item feature tensors, keys uint64 [n], hit mask)."""
        torch = _torch()
        g, gp = _i32_array(grid_thw)
        n = g.size // 3
        T = int(sum(int(g[3 * i]) * int(g[3 * i + 1]) * int(g[3 * i + 2]) for i in range(n)))
        if features is None:
            features = torch.empty((max(T // 4, 1), self.cfg.out_dim), dtype=torch_dtype(self.dtype),
                                   device=self.device)
        rows = ctypes.c_int64(0)
        cu_rows = np.zeros(n + 1, dtype=np.int32)
        keys = np.zeros(n, dtype=np.uint64)
        hit = np.zeros(n, dtype=np.uint8)
        m = (ctypes.c_float * len(mean))(*[float(v) for v in mean])
        istd = (ctypes.c_float * len(std))(*[1.0 / float(v) for v in std])
        _check(self.lib.epd_encode_frames_cached(
            self._h, cache._h, _ptr(frames), gp, n, m, istd, _ptr(features), int(features.shape[0]),
            ctypes.byref(rows), cu_rows.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)),
            keys.ctypes.data_as(ctypes.POINTER(ctypes.c_uint64)), hit.ctypes.data_as(ctypes.POINTER(ctypes.c_uint8)),
            _stream_ptr(stream)), "epd_encode_frames_cached")
        return [features[int(cu_rows[i]):int(cu_rows[i + 1])] for i in range(n)], keys, hit.astype(bool)

    def encode_host(self, host_patches, grid_thw, host_features, stream=None):
        """host_patches / host_features: CPU tensors (pinned for asynchronous copies)."""
        g, gp = _i32_array(grid_thw)
        n = g.size // 3
        rows = ctypes.c_int64(0)
        cu_rows = np.zeros(n + 1, dtype=np.int32)
        _check(self.lib.epd_encode_host(self._h, _ptr(host_patches), gp, n, _ptr(host_features),
                                        int(host_features.shape[0]), ctypes.byref(rows),
                                        cu_rows.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)),
                                        _stream_ptr(stream)), "epd_encode_host")
        return rows.value, cu_rows

    def encode_host_async(self, host_patches, grid_thw, host_features, stream=None):
        """Pipelined encode_host: copies on the encoder's own streams; call host_join() before reading."""
        g, gp = _i32_array(grid_thw)
        n = g.size // 3
        rows = ctypes.c_int64(0)
        cu_rows = np.zeros(n + 1, dtype=np.int32)
        _check(self.lib.epd_encode_host_async(self._h, _ptr(host_patches), gp, n, _ptr(host_features),
                                              int(host_features.shape[0]), ctypes.byref(rows),
                                              cu_rows.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)),
                                              _stream_ptr(stream)), "epd_encode_host_async")
        return rows.value, cu_rows

    def host_join(self, stream=None) -> None:
        _check(self.lib.epd_encode_host_join(self._h, _stream_ptr(stream)), "epd_encode_host_join")

    def use_graphs(self, enable: bool) -> None:
        _check(self.lib.epd_debug_use_graphs(self._h, 1 if enable else 0), "epd_debug_use_graphs")

    def graph_count(self) -> int:
        return int(self.lib.epd_debug_graph_count(self._h))

    def last_status(self) -> int:
        return int(self.lib.epd_encoder_last_status(self._h))

    def last_launch_count(self) -> int:
        return int(self.lib.epd_encoder_last_launch_count(self._h))

    def uses_tensor_cores(self) -> bool:
        return bool(self.lib.epd_encoder_uses_tensor_cores(self._h))

    # ---- test hooks ------------------------------------------------------------------------
    def debug_bookkeeping(self, n_images: int, T: int):
        cu = np.zeros(n_images + 1, np.int32)
        pr, pc, mi = np.zeros(T, np.int32), np.zeros(T, np.int32), np.zeros(T, np.int32)
        p = lambda a: a.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))
        _check(self.lib.epd_debug_bookkeeping(self._h, p(cu), p(pr), p(pc), p(mi)), "epd_debug_bookkeeping")
        return {"cu_seqlens": cu, "pos_row": pr, "pos_col": pc, "merge_idx": mi.reshape(-1, 4)}

    def set_taps(self, taps):
        """taps: list of layers+1 float32 device tensors or None entries; None clears."""
        if taps is None:
            self._taps = None
            _check(self.lib.epd_debug_set_taps(self._h, None), "epd_debug_set_taps")
            return
        assert len(taps) == self.cfg.layers + 1
        self._taps = list(taps)
        arr = (ctypes.c_void_p * len(taps))(*[_ptr(t) for t in taps])
        _check(self.lib.epd_debug_set_taps(self._h, ctypes.cast(arr, _PP)), "epd_debug_set_taps")

    def run_block(self, layer: int, x, grid_thw, stream=None):
        g, gp = _i32_array(grid_thw)
        _check(self.lib.epd_debug_run_block(self._h, int(layer), _ptr(x), gp, g.size // 3, _stream_ptr(stream)),
               "epd_debug_run_block")
        return x

    def profile(self, enable: bool):
        _check(self.lib.epd_debug_profile(self._h, 1 if enable else 0), "epd_debug_profile")

    def profile_read(self) -> Dict[str, Dict]:
        """Device time (ms) and launch count per step class of the most recent profiled encode."""
        n = int(self.lib.epd_debug_profile_classes())
        ms = (ctypes.c_float * n)()
        cnt = (ctypes.c_int64 * n)()
        _check(self.lib.epd_debug_profile_read(self._h, ms, cnt), "epd_debug_profile_read")
        return {self.lib.epd_debug_profile_class_name(i).decode(): {"ms": float(ms[i]), "launches": int(cnt[i])}
                for i in range(n)}

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            self.lib.epd_encoder_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


# ---- single steps ------------------------------------------------------------------------------

def op_linear(dtype, x, w, bias, out, M, N, K, flags=0, ldx=None, ldw=None, ldo=None, stream=None):
    lib = load_library()
    _check(lib.epd_op_linear(dtype, _ptr(x), ldx if ldx is not None else x.stride(0), _ptr(w),
                             ldw if ldw is not None else w.stride(0), _ptr(bias), _ptr(out),
                             ldo if ldo is not None else out.stride(0), M, N, K, flags, _stream_ptr(stream)),
           "epd_op_linear")
    return out


def op_quantize_e4m3(x, stream=None):
    """bf16 [M, K] -> (E4M3 byte codes [M, ldq] with ldq = K rounded up to 16, float scales [M])."""
    torch = _torch()
    lib = load_library()
    M, K = x.shape
    ldq = (K + 15) // 16 * 16
    q = torch.empty((M, ldq), dtype=torch.uint8, device=x.device)
    scale = torch.empty(M, dtype=torch.float32, device=x.device)
    _check(lib.epd_op_quantize_e4m3(_ptr(x), x.stride(0), _ptr(q), ldq, _ptr(scale), M, K, _stream_ptr(stream)),
           "epd_op_quantize_e4m3")
    return q, scale


def op_linear_e4m3(xq, x_scale, wq, w_scale, bias, out, K, flags=0, stream=None):
    lib = load_library()
    M, N = xq.shape[0], wq.shape[0]
    _check(lib.epd_op_linear_e4m3(_ptr(xq), xq.stride(0), _ptr(x_scale), _ptr(wq), wq.stride(0), _ptr(w_scale),
                                  _ptr(bias), _ptr(out), out.stride(0), M, N, K, flags, _stream_ptr(stream)),
           "epd_op_linear_e4m3")
    return out


def op_rmsnorm(dtype, x, gain, out, eps, dst_row=None, stream=None):
    lib = load_library()
    _check(lib.epd_op_rmsnorm(dtype, _ptr(x), _ptr(gain), _ptr(out), _ptr(dst_row), x.shape[0], x.shape[1],
                              eps, _stream_ptr(stream)), "epd_op_rmsnorm")
    return out


def padded_head_dim(head_dim: int) -> int:
    return int(load_library().epd_padded_head_dim(head_dim))


def op_rope_split(dtype, qkv, pos_row, pos_col, heads, head_dim, theta, q_scale, stream=None):
    torch = _torch()
    lib = load_library()
    T = qkv.shape[0]
    dhp = padded_head_dim(head_dim)
    q, k, v = (torch.empty((heads, T, dhp), dtype=qkv.dtype, device=qkv.device) for _ in range(3))
    _check(lib.epd_op_rope_split(dtype, _ptr(qkv), _ptr(pos_row), _ptr(pos_col), _ptr(q), _ptr(k), _ptr(v), T,
                                 heads, head_dim, theta, q_scale, _stream_ptr(stream)), "epd_op_rope_split")
    return q, k, v


def op_attention(dtype, q, k, v, cu_seqlens_dev, cu_seqlens_host, head_dim, flags=0, stream=None):
    torch = _torch()
    lib = load_library()
    heads, T, _ = q.shape
    out = torch.empty((T, heads * head_dim), dtype=q.dtype, device=q.device)
    hcu, hp = _i32_array(cu_seqlens_host)
    _check(lib.epd_op_attention(dtype, _ptr(q), _ptr(k), _ptr(v), _ptr(cu_seqlens_dev), hp, hcu.size - 1,
                                _ptr(out), T, heads, head_dim, flags, _stream_ptr(stream)), "epd_op_attention")
    return out


def op_merge(dtype, y, merge_idx, stream=None):
    torch = _torch()
    lib = load_library()
    T, h = y.shape
    out = torch.empty((T // 4, 4 * h), dtype=y.dtype, device=y.device)
    _check(lib.epd_op_merge(dtype, _ptr(y), _ptr(merge_idx), _ptr(out), T // 4, h, _stream_ptr(stream)),
           "epd_op_merge")
    return out


def pack_frames(frames: Sequence[np.ndarray], bf16: bool = False):
    """List of [t*Tp, C, H, W] arrays -> one flat device tensor (items back to back; uint8, or bfloat16 for
    float-valued frames) and the int64 BYTE offsets of the items."""
    torch = _torch()
    if bf16:
        flat = np.concatenate([np.ascontiguousarray(f, dtype=np.float32).reshape(-1) for f in frames]) if frames \
            else np.zeros(0, np.float32)
        off = np.concatenate([[0], np.cumsum([2 * f.size for f in frames])]).astype(np.int64)
        return torch.from_numpy(flat).cuda().to(torch.bfloat16), off
    flat = np.concatenate([np.ascontiguousarray(f, dtype=np.uint8).reshape(-1) for f in frames]) if frames \
        else np.zeros(0, np.uint8)
    off = np.concatenate([[0], np.cumsum([f.size for f in frames])]).astype(np.int64)
    return torch.from_numpy(flat).cuda(), off


def op_patchify(dtype, frames_dev, item_off, grid_thw, cu_seqlens, in_channels, patch, temporal_patch, mean, std,
                ld=None, stream=None):
    torch = _torch()
    lib = load_library()
    g = np.asarray(grid_thw, dtype=np.int32).reshape(-1, 3)
    n = g.shape[0]
    T = int(cu_seqlens[-1])
    K = in_channels * temporal_patch * patch * patch
    ld = K if ld is None else ld
    out = torch.full((T, ld), 7.0, dtype=torch_dtype(dtype), device="cuda")
    m = (ctypes.c_float * len(mean))(*[float(v) for v in mean])
    istd = (ctypes.c_float * len(std))(*[1.0 / float(v) for v in std])
    off_d = torch.from_numpy(np.asarray(item_off, dtype=np.int64)).cuda()
    g_d = torch.from_numpy(g.copy()).cuda()
    cu_d = torch.from_numpy(np.asarray(cu_seqlens, dtype=np.int32)).cuda()
    fmt = FRAMES_BF16 if frames_dev.dtype == torch.bfloat16 else FRAMES_U8
    _check(lib.epd_op_patchify_fmt(dtype, fmt, _ptr(frames_dev), _ptr(off_d), _ptr(g_d), _ptr(cu_d), n, T, _ptr(out),
                                   ld, in_channels, patch, temporal_patch, m, istd, _stream_ptr(stream)),
           "epd_op_patchify_fmt")
    return out


def op_qkv_rope(x, w, bias, pos_row, pos_col, heads, head_dim, theta, q_scale, table_rows, stream=None):
    """Fused QKV projection + rotary + head split (bf16).  Returns q, k, v [heads, T, padded]; q and k in
    the prepared (pair) order epd_op_qkv_prepare documents."""
    torch = _torch()
    lib = load_library()
    T, h = x.shape[0], heads * head_dim
    sp = _stream_ptr(stream)
    wp = torch.empty((3 * h, h), dtype=torch.bfloat16, device="cuda")
    bp = torch.empty(3 * h, dtype=torch.bfloat16, device="cuda")
    _check(lib.epd_op_qkv_prepare(_ptr(w), w.stride(0), _ptr(bias), _ptr(wp), _ptr(bp), heads, head_dim, sp),
           "epd_op_qkv_prepare")
    table = torch.empty((table_rows, head_dim // 4, 2), dtype=torch.float32, device="cuda")
    _check(lib.epd_op_rope_table(_ptr(table), table_rows, head_dim, theta, sp), "epd_op_rope_table")
    dhp = padded_head_dim(head_dim)
    q, k, v = (torch.full((heads, T, dhp), 7.0, dtype=torch.bfloat16, device="cuda") for _ in range(3))
    _check(lib.epd_op_qkv_pad_init(_ptr(q), _ptr(k), _ptr(v), heads * T, head_dim, sp), "epd_op_qkv_pad_init")
    _check(lib.epd_op_qkv_rope(_ptr(x), x.stride(0), _ptr(wp), _ptr(bp), _ptr(pos_row), _ptr(pos_col), _ptr(table),
                               table_rows, _ptr(q), _ptr(k), _ptr(v), T, heads, head_dim, q_scale, sp),
           "epd_op_qkv_rope")
    return q, k, v


def set_wait_limit(cycles: int) -> None:
    """Cycle limit of the kernels' bounded waits (test hook); 0 restores the default."""
    _check(load_library().epd_debug_set_wait_limit(int(cycles)), "epd_debug_set_wait_limit")


def set_sm_limit(n_sms: int) -> None:
    """At most n_sms CTAs for the persistent kernels (0 = every SM)."""
    _check(load_library().epd_set_sm_limit(n_sms), "epd_set_sm_limit")


def get_sm_limit() -> int:
    return int(load_library().epd_get_sm_limit())


def signal_ready(flag, value: int, stream=None) -> None:
    """Stream-ordered store of `value` to flag[0] (int32 device tensor)."""
    _check(load_library().epd_signal_ready(_ptr(flag), value, _stream_ptr(stream)), "epd_signal_ready")


def op_stream_read(data, passes: int, n_ctas: int, sums, stream=None) -> None:
    _check(load_library().epd_op_stream_read(_ptr(data), data.numel() * data.element_size(), passes, n_ctas,
                                             _ptr(sums), _stream_ptr(stream)), "epd_op_stream_read")


def op_content_hash(data_dev, item_off, stream=None) -> np.ndarray:
    """64-bit content keys of the items of a packed device byte buffer (item_off: byte offsets,
    multiples of 8, length n+1).  Returns uint64 [n] on the host."""
    torch = _torch()
    lib = load_library()
    off = np.asarray(item_off, dtype=np.int64).reshape(-1)
    n = off.size - 1
    if n <= 0:
        return np.zeros(0, dtype=np.uint64)
    if np.any(off % 8) or np.any(np.diff(off) < 0):
        raise ValueError("item offsets must be non-decreasing multiples of 8")
    off_d = torch.from_numpy(off).cuda()
    out = torch.empty(n, dtype=torch.int64, device="cuda")
    _check(lib.epd_op_content_hash(_ptr(data_dev), _ptr(off_d), n, _ptr(out), _stream_ptr(stream)),
           "epd_op_content_hash")
    return out.cpu().numpy().view(np.uint64)


class FeatureCache:
    """Feature matrices by content key in a device pool owned by this object (first-in-first-out)."""

    def __init__(self, pool_bytes: int, out_dim: int, dtype: int):
        torch = _torch()
        lib = load_library()
        self._lib = lib
        self.out_dim = out_dim
        self.tdtype = torch_dtype(dtype)
        self._pool = torch.empty(pool_bytes, dtype=torch.uint8, device="cuda")
        h = ctypes.c_void_p()
        row_bytes = out_dim * (4 if dtype == DTYPE_F32 else 2)
        _check(lib.epd_feature_cache_create(_ptr(self._pool), pool_bytes, row_bytes, ctypes.byref(h)),
               "epd_feature_cache_create")
        self._h = h

    def lookup(self, key: int, rows: int, stream=None):
        """The cached [rows, out_dim] features, or None."""
        torch = _torch()
        dst = torch.empty((rows, self.out_dim), dtype=self.tdtype, device="cuda")
        st = self._lib.epd_feature_cache_lookup(self._h, int(key), rows, _ptr(dst), _stream_ptr(stream))
        if st == 1:
            return None
        _check(st, "epd_feature_cache_lookup")
        return dst

    def insert(self, key: int, feats, stream=None) -> None:
        assert feats.is_contiguous() and feats.shape[1] == self.out_dim and feats.dtype == self.tdtype
        _check(self._lib.epd_feature_cache_insert(self._h, int(key), feats.shape[0], _ptr(feats),
                                                  _stream_ptr(stream)), "epd_feature_cache_insert")

    def stats(self) -> dict:
        v = [ctypes.c_int64() for _ in range(4)]
        _check(self._lib.epd_feature_cache_stats(self._h, *[ctypes.byref(x) for x in v]), "epd_feature_cache_stats")
        return dict(zip(("hits", "misses", "evictions", "entries"), (int(x.value) for x in v)))

    def close(self) -> None:
        if self._h:
            self._lib.epd_feature_cache_destroy(self._h)
            self._h = None
            self._pool = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def static_scratch_bytes() -> int:
    return int(load_library().epd_static_scratch_bytes())


def op_rope_attention_static(dtype, qkv, pos_row, pos_col, cu_seqlens_dev, cu_seqlens_host, heads, head_dim,
                             theta, out=None, stream=None):
    """Allocation-free rotary + split + attention: intermediates live in the library's fixed device
    array.  `out` may be passed in so that the call itself allocates nothing at all."""
    torch = _torch()
    lib = load_library()
    T = qkv.shape[0]
    if out is None:
        out = torch.empty((T, heads * head_dim), dtype=qkv.dtype, device=qkv.device)
    hcu, hp = _i32_array(cu_seqlens_host)
    _check(lib.epd_op_rope_attention_static(dtype, _ptr(qkv), _ptr(pos_row), _ptr(pos_col), _ptr(cu_seqlens_dev),
                                            hp, hcu.size - 1, _ptr(out), T, heads, head_dim, theta,
                                            _stream_ptr(stream)), "epd_op_rope_attention_static")
    return out
