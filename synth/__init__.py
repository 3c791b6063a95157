"""Seeded synthetic inputs for the ViT Encode stage (shared by the CPU oracle's tests and the CUDA path).

This module holds data only: the encoder configurations, a counter-based random
generator (Philox keyed by (seed, tensor id)), the bf16 rounding applied once to
generated values, and the image-grid lists of each workload.  It contains none of
the encoder's arithmetic and imports neither the oracle nor the CUDA package.

Recipe (all workloads): pixel patches i.i.d. N(0,1); matrices and biases N(0,0.02);
RMSNorm gains 1 + N(0,0.02); bf16 configurations round every generated value to bf16
(round-to-nearest-even) so both sides consume identical numbers.
"""
from __future__ import annotations

import dataclasses
import zlib
from typing import Dict, List, Sequence, Tuple

import numpy as np

DTYPE_FP32 = 0
DTYPE_BF16 = 1
ACT_GELU_TANH = 0
ACT_GELU_ERF = 1
PROJ_LINEAR = 0
PROJ_MLP = 1


@dataclasses.dataclass(frozen=True)
class EncoderConfig:
    """Static shape of one encoder; field names mirror epd_config_t."""
    name: str
    dtype: int
    in_channels: int
    patch: int
    temporal_patch: int
    hidden: int
    layers: int
    heads: int
    head_dim: int
    mlp: int
    act: int
    eps: float
    rope_theta: float
    merge: int
    final_norm: int
    proj_kind: int
    proj_hidden: int
    out_dim: int

    @property
    def patch_dim(self) -> int:
        return self.in_channels * self.temporal_patch * self.patch * self.patch

    def with_layers(self, layers: int) -> "EncoderConfig":
        return dataclasses.replace(self, layers=layers, name=f"{self.name}-L{layers}")


TINY_FP32 = EncoderConfig(
    name="tiny-fp32", dtype=DTYPE_FP32, in_channels=3, patch=14, temporal_patch=1,
    hidden=256, layers=2, heads=4, head_dim=64, mlp=1024, act=ACT_GELU_TANH,
    eps=1e-6, rope_theta=10000.0, merge=2, final_norm=1,
    proj_kind=PROJ_LINEAR, proj_hidden=0, out_dim=512)

VIT_06B = EncoderConfig(
    name="vit-0.6b-bf16", dtype=DTYPE_BF16, in_channels=3, patch=16, temporal_patch=1,
    hidden=1152, layers=27, heads=16, head_dim=72, mlp=4304, act=ACT_GELU_TANH,
    eps=1e-6, rope_theta=10000.0, merge=2, final_norm=1,
    proj_kind=PROJ_MLP, proj_hidden=4608, out_dim=4096)

VIT_06B_VIDEO = dataclasses.replace(VIT_06B, name="vit-0.6b-bf16-tp2", temporal_patch=2)

VIT_6B = EncoderConfig(
    name="vit-6b-bf16", dtype=DTYPE_BF16, in_channels=3, patch=14, temporal_patch=1,
    hidden=3200, layers=45, heads=25, head_dim=128, mlp=12800, act=ACT_GELU_ERF,
    eps=1e-6, rope_theta=10000.0, merge=2, final_norm=1,
    proj_kind=PROJ_MLP, proj_hidden=12800, out_dim=8192)


# A 0.7B-class encoder with the hand-off width the paper's E-P prefetching table prints (d = 3584, patch 14
# with the 2x2 merge: 280x280 -> [100, 3584]).  The paper gives no internal widths: 32 layers of 16 heads x 80
# with a 4x MLP are this repository's choice (0.63 G parameters in the blocks).
VIT_07B = EncoderConfig(
    name="vit-0.7b-bf16", dtype=DTYPE_BF16, in_channels=3, patch=14, temporal_patch=1,
    hidden=1280, layers=32, heads=16, head_dim=80, mlp=5120, act=ACT_GELU_TANH,
    eps=1e-6, rope_theta=10000.0, merge=2, final_norm=1,
    proj_kind=PROJ_MLP, proj_hidden=5120, out_dim=3584)


def tiny_variant(dtype: int = DTYPE_FP32, head_dim: int = 8, heads: int = 2, layers: int = 2,
                 mlp: int = 24, patch: int = 2, temporal_patch: int = 1, act: int = ACT_GELU_TANH,
                 proj_kind: int = PROJ_LINEAR, out_dim: int = 12) -> EncoderConfig:
    """A very small encoder for brute-force checks."""
    hidden = heads * head_dim
    return EncoderConfig(
        name="brute", dtype=dtype, in_channels=3, patch=patch, temporal_patch=temporal_patch,
        hidden=hidden, layers=layers, heads=heads, head_dim=head_dim, mlp=mlp, act=act,
        eps=1e-6, rope_theta=10000.0, merge=2, final_norm=1, proj_kind=proj_kind,
        proj_hidden=(4 * hidden if proj_kind == PROJ_MLP else 0), out_dim=out_dim)


# ----------------------------------------------------------------------------- random numbers

def _tensor_key(seed: int, tensor_id: str) -> List[int]:
    return [int(seed) & 0xFFFFFFFFFFFFFFFF, zlib.crc32(tensor_id.encode("utf-8"))]


def generator(seed: int, tensor_id: str) -> np.random.Generator:
    """Philox stream keyed by (seed, crc32(tensor id)); each tensor has its own stream."""
    return np.random.Generator(np.random.Philox(key=_tensor_key(seed, tensor_id)))


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bf16 (ties to even); result stays float32."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    r = (u + bias) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """The uint16 bit patterns of values that are already exactly representable in bf16."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    return (u >> np.uint32(16)).astype(np.uint16)


def normal(seed: int, tensor_id: str, shape: Sequence[int], std: float, mean: float,
           dtype: int) -> np.ndarray:
    """float32 array ~ N(mean, std²); bf16 configurations get values rounded to bf16."""
    g = generator(seed, tensor_id)
    x = g.standard_normal(size=tuple(shape), dtype=np.float32)
    x *= np.float32(std)
    if mean != 0.0:
        x += np.float32(mean)
    if dtype == DTYPE_BF16:
        x = round_to_bf16(x)
    return x


# ----------------------------------------------------------------------------- weights / inputs

def make_layer_weights(cfg: EncoderConfig, l: int, seed: int = 0, qkv_scale: float = 1.0) -> Dict:
    """Parameters of block l (each tensor has its own random stream, so blocks can be drawn one at a time)."""
    h, m, d = cfg.hidden, cfg.mlp, cfg.dtype
    p = f"layer{l}."

    def mat(tid, shape, scale=1.0):
        return normal(seed, p + tid, shape, 0.02 * scale, 0.0, d)

    def gain(tid, n):
        return normal(seed, p + tid, (n,), 0.02, 1.0, d)

    return {
        "norm1_w": gain("norm1_w", h),
        "qkv_w": mat("qkv_w", (3 * h, h), qkv_scale),
        "qkv_b": mat("qkv_b", (3 * h,)),
        "out_w": mat("out_w", (h, h)),
        "out_b": mat("out_b", (h,)),
        "norm2_w": gain("norm2_w", h),
        "fc1_w": mat("fc1_w", (m, h)),
        "fc1_b": mat("fc1_b", (m,)),
        "fc2_w": mat("fc2_w", (h, m)),
        "fc2_b": mat("fc2_b", (h,)),
    }


def make_weights(cfg: EncoderConfig, seed: int = 0, qkv_scale: float = 1.0, with_layers: bool = True) -> Dict:
    """All encoder parameters as float32 arrays ([out, in] row-major matrices).

    qkv_scale > 1 multiplies W_qkv so attention logits become sharply peaked (a stress case
    for the online-softmax rescaling; not one of the benchmark configurations).
    with_layers=False leaves "layers" empty (the caller draws the blocks with make_layer_weights).
    """
    h, K = cfg.hidden, cfg.patch_dim
    d = cfg.dtype

    def mat(tid, shape, scale=1.0):
        return normal(seed, tid, shape, 0.02 * scale, 0.0, d)

    def gain(tid, n):
        return normal(seed, tid, (n,), 0.02, 1.0, d)

    w = {"patch_w": mat("patch_w", (h, K)), "patch_b": mat("patch_b", (h,)), "layers": []}
    if with_layers:
        w["layers"] = [make_layer_weights(cfg, l, seed, qkv_scale) for l in range(cfg.layers)]
    w["final_norm_w"] = gain("final_norm_w", h)
    D4 = cfg.merge * cfg.merge * h
    if cfg.proj_kind == PROJ_LINEAR:
        w["proj_w1"] = mat("proj_w1", (cfg.out_dim, D4))
        w["proj_b1"] = mat("proj_b1", (cfg.out_dim,))
        w["proj_w2"] = None
        w["proj_b2"] = None
    else:
        w["proj_w1"] = mat("proj_w1", (cfg.proj_hidden, D4))
        w["proj_b1"] = mat("proj_b1", (cfg.proj_hidden,))
        w["proj_w2"] = mat("proj_w2", (cfg.out_dim, cfg.proj_hidden))
        w["proj_b2"] = mat("proj_b2", (cfg.out_dim,))
    return w


def num_tokens(grid_thw: Sequence[Sequence[int]]) -> int:
    return int(sum(int(t) * int(h) * int(w) for t, h, w in grid_thw))


def make_patches(cfg: EncoderConfig, grid_thw: Sequence[Sequence[int]], seed: int = 0,
                 tensor_id: str = "patches") -> np.ndarray:
    """Packed pixel patches [T, C*Tp*P*P], N(0,1); element order inside a patch is (c, tp, y, x)."""
    return normal(seed, tensor_id, (num_tokens(grid_thw), cfg.patch_dim), 1.0, 0.0, cfg.dtype)


PIXEL_MEAN = (0.5, 0.5, 0.5)
PIXEL_STD = (0.5, 0.5, 0.5)


def make_frames(cfg: EncoderConfig, grid_thw: Sequence[Sequence[int]], seed: int = 0) -> List[np.ndarray]:
    """Raw frames of every item: uint8 [t*Tp, C, h*P, w*P], pixel values uniform over 0..255."""
    out = []
    for i, (t, h, w) in enumerate(grid_thw):
        g = generator(seed, f"frames{i}")
        out.append(g.integers(0, 256, size=(t * cfg.temporal_patch, cfg.in_channels, h * cfg.patch, w * cfg.patch),
                              dtype=np.uint8))
    return out


# ----------------------------------------------------------------------------- workloads

def grid_batch_fixed(n_images: int, height: int, width: int, patch: int, frames_t: int = 1
                     ) -> List[Tuple[int, int, int]]:
    return [(frames_t, height // patch, width // patch)] * n_images


def grid_variable_resolution(n_images: int = 32, patch: int = 16, seed: int = 0,
                             lo: int = 224, hi: int = 1344, step: int = 32
                             ) -> List[Tuple[int, int, int]]:
    """H and W each uniform over multiples of `step` in [lo, hi], drawn in the order H0, W0, H1, ..."""
    g = generator(seed, "variable_resolution")
    draws = g.integers(lo // step, hi // step + 1, size=2 * n_images)
    return [(1, int(draws[2 * i]) * step // patch, int(draws[2 * i + 1]) * step // patch)
            for i in range(n_images)]


def grid_long_sequences(patch: int = 16) -> List[Tuple[int, int, int]]:
    """One 2048x2048 image and one 16-frame 448x448 clip with temporal patch 2."""
    return [(1, 2048 // patch, 2048 // patch), (16 // 2, 448 // patch, 448 // patch)]


def grid_prefetch_table() -> List[Tuple[int, int, int]]:
    """The image sizes of the paper's E-P prefetching table, snapped to multiples of 28 pixels (patch 14):
    280x280, 560x560, 720x1280, 1080x1920 and 4096x3112 -> 100, 400, 1196, 2691 and 16206 merged tokens."""
    return [(1, 20, 20), (1, 40, 40), (1, 52, 92), (1, 78, 138), (1, 292, 222)]


WORKLOADS = {
    # name: (config, grid list)
    "cfg0_tiny_fp32": (TINY_FP32, grid_batch_fixed(2, 224, 224, 14)),
    "cfg1_vit06b_b8_448": (VIT_06B, grid_batch_fixed(8, 448, 448, 16)),
    "cfg2_vit06b_var32": (VIT_06B, grid_variable_resolution(32, 16, 0)),
    "cfg3_vit06b_long": (VIT_06B_VIDEO, grid_long_sequences(16)),
    "cfg4_vit6b_b16_448": (VIT_6B, grid_batch_fixed(16, 448, 448, 14)),
    # beyond the five benchmark configurations: the hand-off shapes the paper prints
    "cfg5_vit07b_table42": (VIT_07B, grid_prefetch_table()),
}


def algorithmic_flops(cfg: EncoderConfig, grid_thw: Sequence[Sequence[int]]) -> float:
    """Floating-point operations one forward must perform (true head_dim, full bidirectional blocks)."""
    T = num_tokens(grid_thw)
    h, m, L = cfg.hidden, cfg.mlp, cfg.layers
    seg2 = float(sum((t * a * b) ** 2 for t, a, b in grid_thw))
    Tm = T // (cfg.merge * cfg.merge)
    D4 = cfg.merge * cfg.merge * h
    if cfg.proj_kind == PROJ_LINEAR:
        proj = D4 * cfg.out_dim
    else:
        proj = D4 * cfg.proj_hidden + cfg.proj_hidden * cfg.out_dim
    return 2.0 * T * cfg.patch_dim * h + L * (2.0 * T * (4 * h * h + 2 * h * m) + 4.0 * h * seg2) \
        + 2.0 * Tm * proj
