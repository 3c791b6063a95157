"""CPU fp64 oracle for the Encode stage  V_m = E(I_m)  (Section 3.1 "Encode Stage", Eq. 1).

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition the CUDA path is
checked against.  Only the tests, the smoke check and the benchmark's CPU-baseline leg
may import it; the product never does, and it shares no code with the CUDA path.

The paper fixes the stage's contract -- multimodal items in, one [n, d] feature matrix
per item out, consumed by Prefill (Eq. 1; the printed E->P tensors of the prefetching
table in Section 4) -- and says E is a Vision Transformer whose attention cost grows
quadratically with the visual sequence length (Section 1).  It gives no layer-level
formulae, so the encoder evaluated here is the standard pre-norm ViT the benchmark
configurations name, written out step by step in float64 with no blocking, fusion or
intermediate rounding:

  P0  (optional front end) raw uint8 frames -> patch vectors: per-channel normalisation and
      patch extraction, element order (channel, temporal, y, x)
  O0  packing: image i has grid (t, h, w); its tokens are raster-ordered (frame, row, col)
      and occupy rows cu[i]..cu[i+1] of every activation matrix; every frame reuses the
      image's (row, col) positions.
  O1  X = patches @ W_pe^T + b_pe
  per layer:
  O2  A = rmsnorm(X; g1)
  O3  [q|k|v] = A @ W_qkv^T + b_qkv, heads are consecutive head_dim-wide column groups
  O4  2-D rotary embedding on q and k: first half of each head rotates by the row index,
      second half by the column index, rotate-half pairing inside each half
  O5  per image, per head: softmax(q k^T / sqrt(head_dim)) v over ALL tokens of that image
      (bidirectional, block-diagonal across images)
  O6  X += O @ W_o^T + b_o
  O7  X += gelu(rmsnorm(X; g2) @ W_1^T + b_1) @ W_2^T + b_2
  O8  Y = rmsnorm(X; g_final)
  O9  2x2 spatial merge: merged token (f, R, C) concatenates Y at (2R+dy, 2C+dx) for
      (dy,dx) = (0,0),(0,1),(1,0),(1,1)
  O10 projector: linear, or linear-GELU-linear, producing the [n, d] hand-off features.

  Q   (variant, Section 3.5's operator mix at lower precision: not part of the bf16 path) a linear layer with
      8-bit floating-point operands: rows of x and rows of w are scaled to the E4M3 range, rounded to E4M3
      (4 exponent bits, bias 7, 3 mantissa bits, largest finite value 448, no infinities), multiplied exactly and
      rescaled: quantize_e4m3_rows, linear_e4m3.

Parity pins (tests/test_oracle_*.py): pure-Python brute force on tiny inputs, PyTorch CPU
float64 library routines for each step, closed forms and invariants, and the merged-row
counts the paper prints.  The numerical values of the features themselves are
"parity unpinned" by the paper (it prints none); they are pinned only by that chain.
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np
from scipy.special import erf as _erf

ACT_GELU_TANH = 0
ACT_GELU_ERF = 1


# ----------------------------------------------------------------------------- O0 / O9 integers

def bookkeeping(grid_thw: Sequence[Sequence[int]], merge: int = 2) -> Dict[str, np.ndarray]:
    """Integer layout of a packed batch (step O0 and the index side of step O9).

    Returns int32 arrays: cu_seqlens [n+1], pos_row [T], pos_col [T], cu_out [n+1] and
    merge_idx [Tm, merge*merge] with merge_idx[o, 2*dy+dx] = source token of merged row o.
    The contract is Eq. 1's V_m in R^{n x d}: rows cu_out[i]..cu_out[i+1] are image i's n rows.
    """
    n = len(grid_thw)
    cu = np.zeros(n + 1, dtype=np.int64)
    cu_out = np.zeros(n + 1, dtype=np.int64)
    pos_row: List[np.ndarray] = []
    pos_col: List[np.ndarray] = []
    idx: List[np.ndarray] = []
    for i, (t, h, w) in enumerate(grid_thw):
        t, h, w = int(t), int(h), int(w)
        if t < 1 or h < 1 or w < 1 or h % merge or w % merge:
            raise ValueError(f"bad grid {(t, h, w)}")
        cu[i + 1] = cu[i] + t * h * w
        cu_out[i + 1] = cu_out[i] + t * (h // merge) * (w // merge)
        r = np.repeat(np.arange(h), w)
        c = np.tile(np.arange(w), h)
        pos_row.append(np.tile(r, t))
        pos_col.append(np.tile(c, t))
        f, R, C = np.meshgrid(np.arange(t), np.arange(h // merge), np.arange(w // merge), indexing="ij")
        cols = []
        for dy in range(merge):
            for dx in range(merge):
                cols.append(cu[i] + f * h * w + (merge * R + dy) * w + (merge * C + dx))
        idx.append(np.stack([c_.reshape(-1) for c_ in cols], axis=1))
    cat = lambda xs, width=None: (np.concatenate(xs) if xs else np.zeros((0,) if width is None else (0, width)))
    return {
        "cu_seqlens": cu.astype(np.int32),
        "cu_out": cu_out.astype(np.int32),
        "pos_row": cat(pos_row).astype(np.int32),
        "pos_col": cat(pos_col).astype(np.int32),
        "merge_idx": cat(idx, merge * merge).astype(np.int32).reshape(-1, merge * merge),
    }


# ----------------------------------------------------------------------------- content hash (feature key)

_MASK64 = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15


def _mix64(z: int) -> int:
    """The finalizer of the SplitMix64 generator (Steele, Lea, Flood 2014; constants of Stafford's mix 13)."""
    z &= _MASK64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _MASK64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _MASK64
    return z ^ (z >> 31)


def content_hash(data: bytes) -> int:
    """64-bit key of one item's input bytes (the key under which its features are cached; the paper's
    MM Store keys features by a hash of the multimodal input, Section 3.2, without naming the hash).

    The bytes (length a multiple of 8) are read as little-endian 64-bit words w_1 .. w_n:
        key = mix( (sum_k mix(w_k xor k*GOLDEN)) + 8n )   (all arithmetic mod 2^64)
    The sum makes the key independent of evaluation order (it can be formed in parallel), the
    position salt k*GOLDEN makes it depend on word order, the length term on trailing zeros.
    Plain Python integers, one word at a time."""
    if len(data) % 8:
        raise ValueError("length must be a multiple of 8 bytes")
    acc = 0
    for k in range(len(data) // 8):
        w = int.from_bytes(data[8 * k: 8 * k + 8], "little")
        acc = (acc + _mix64(w ^ (((k + 1) * _GOLDEN) & _MASK64))) & _MASK64
    return _mix64((acc + len(data)) & _MASK64)


# ----------------------------------------------------------------------------- pixels -> patch vectors

def patchify(frames: Sequence[np.ndarray], grid_thw: Sequence[Sequence[int]], patch: int, temporal_patch: int,
             mean: Sequence[float], std: Sequence[float]) -> np.ndarray:
    """The step in front of the stage: raw frames -> the packed patch matrix [T, C*Tp*P*P] that O1 consumes.

    frames[i] is item i as uint8 [t*Tp, C, h*P, w*P] (frame, channel, y, x).  Pixel value v of channel c
    becomes (v/255 - mean[c]) / std[c]; token (f, r, c) of the item gathers frames f*Tp .. f*Tp+Tp-1,
    rows r*P .. r*P+P-1, columns c*P .. c*P+P-1 in element order (channel, temporal, y, x).
    Resizing an image to a multiple of the patch size is preprocessing and happens before this.
    """
    P, Tp = int(patch), int(temporal_patch)
    mean = np.asarray(mean, dtype=np.float64)
    std = np.asarray(std, dtype=np.float64)
    rows = []
    for fr, (t, h, w) in zip(frames, grid_thw):
        fr = np.asarray(fr)
        C = fr.shape[1]
        assert fr.shape == (t * Tp, C, h * P, w * P), (fr.shape, (t, h, w))
        x = (fr.astype(np.float64) / 255.0 - mean[None, :, None, None]) / std[None, :, None, None]
        x = x.reshape(t, Tp, C, h, P, w, P)              # f, tp, c, r, y, col, xx
        x = x.transpose(0, 3, 5, 2, 1, 4, 6)             # f, r, col, c, tp, y, xx
        rows.append(x.reshape(t * h * w, C * Tp * P * P))
    return np.concatenate(rows, axis=0) if rows else np.zeros((0, 0))


# ----------------------------------------------------------------------------- elementwise pieces

def rmsnorm(x: np.ndarray, g: np.ndarray, eps: float) -> np.ndarray:
    """Step O2/O8: x / sqrt(mean(x^2) + eps) * g, row-wise."""
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * g


def gelu(x: np.ndarray, act: int) -> np.ndarray:
    if act == ACT_GELU_TANH:
        return 0.5 * x * (1.0 + np.tanh(np.sqrt(2.0 / np.pi) * (x + 0.044715 * x ** 3)))
    if act == ACT_GELU_ERF:
        return 0.5 * x * (1.0 + _erf(x / np.sqrt(2.0)))
    raise ValueError("unknown activation")


def linear(x: np.ndarray, w: np.ndarray, b: Optional[np.ndarray]) -> np.ndarray:
    """y = x @ w^T + b with w stored [out, in]."""
    y = x @ w.T
    if b is not None:
        y = y + b
    return y


# ----------------------------------------------------------------------------- Q  8-bit floating-point variant

E4M3_MAX = 448.0


def round_to_e4m3(v: np.ndarray) -> np.ndarray:
    """Nearest E4M3 value (ties to the even mantissa), saturating at +-448; the result is returned as float64.

    E4M3: sign, 4 exponent bits with bias 7, 3 mantissa bits.  Normal values 2^e (1 + k/8), e = -6..8 (the top
    binade stops at 448 = 2^8 * 1.75: its last code is NaN); subnormals k * 2^-9, k = 0..7.  So the spacing of
    representable values around |v| is 2^(e-3) with e = max(floor(log2 |v|), -6).
    """
    v = np.asarray(v, dtype=np.float64)
    a = np.abs(v)
    e = np.floor(np.log2(np.where(a > 0, a, 1.0)))
    e = np.maximum(e, -6.0)
    quantum = np.exp2(e - 3.0)
    q = np.rint(a / quantum) * quantum          # rint: round half to even; a / quantum is exact (power of two)
    q = np.minimum(q, E4M3_MAX)
    return np.copysign(q, v)                    # the sign survives, for zeros too (the format has a negative zero)


def e4m3_bits(q: np.ndarray) -> np.ndarray:
    """The byte codes of values that are exactly representable in E4M3."""
    q = np.asarray(q, dtype=np.float64)
    a = np.abs(q)
    sign = (np.signbit(q)).astype(np.uint8) << 7
    e = np.floor(np.log2(np.where(a > 0, a, 1.0)))
    normal = a >= 2.0 ** -6
    exp_field = np.where(normal, e + 7, 0).astype(np.int64)
    mant = np.where(normal, a / np.exp2(e) * 8 - 8, a * 2.0 ** 9)
    assert np.all(mant == np.rint(mant)), "not an E4M3 value"
    return (sign | (exp_field.astype(np.uint8) << 3) | mant.astype(np.uint8)).astype(np.uint8)


def quantize_e4m3_rows(x: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """Per-row scaling to the E4M3 range and rounding: returns (q, scale) with x[i, :] ~ q[i, :] * scale[i].

    scale[i] = max_j |x[i, j]| / 448 (1 for an all-zero row), q[i, j] = round_to_e4m3(x[i, j] / scale[i]).
    The scale and the quotient decide which 8-bit code an element gets, so they are evaluated in float32
    arithmetic (one correctly rounded division each), the precision the CUDA path takes these decisions in;
    the rounding to E4M3 itself is exact.
    """
    x32 = np.ascontiguousarray(x, dtype=np.float32)
    amax = np.max(np.abs(x32), axis=1)
    scale = np.where(amax > 0, amax / np.float32(E4M3_MAX), np.float32(1.0)).astype(np.float32)
    t = (x32 / scale[:, None]).astype(np.float32)
    return round_to_e4m3(t), scale.astype(np.float64)


def linear_e4m3(x: np.ndarray, w: np.ndarray, b: Optional[np.ndarray]) -> np.ndarray:
    """y = (q_x @ q_w^T) * (s_x s_w^T) + b: both operands quantised row by row (a row of w is one output
    feature), the products and sums exact (float64), the two scales applied to the sum."""
    qx, sx = quantize_e4m3_rows(x)
    qw, sw = quantize_e4m3_rows(w)
    y = (qx @ qw.T) * sx[:, None] * sw[None, :]
    if b is not None:
        y = y + b
    return y


def rope_2d(x: np.ndarray, pos_row: np.ndarray, pos_col: np.ndarray, theta: float) -> np.ndarray:
    """Step O4 on x [T, heads, head_dim].

    With d2 = head_dim/2 and nf = head_dim/4, frequency f has omega_f = theta^(-2f/d2).
    Dims [0, d2) use p = row, dims [d2, head_dim) use p = col.  Inside a half, dims f and
    f+nf form a pair:  x'_f = x_f cos(p w_f) - x_{f+nf} sin(p w_f),
                       x'_{f+nf} = x_{f+nf} cos(p w_f) + x_f sin(p w_f).
    """
    T, nH, dh = x.shape
    assert dh % 4 == 0
    d2, nf = dh // 2, dh // 4
    omega = theta ** (-2.0 * np.arange(nf, dtype=np.float64) / d2)
    out = np.empty_like(x)
    for half, pos in ((0, pos_row), (1, pos_col)):
        ang = pos.astype(np.float64)[:, None] * omega[None, :]          # [T, nf]
        c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
        a = x[:, :, half * d2: half * d2 + nf]
        b = x[:, :, half * d2 + nf: (half + 1) * d2]
        out[:, :, half * d2: half * d2 + nf] = a * c - b * s
        out[:, :, half * d2 + nf: (half + 1) * d2] = b * c + a * s
    return out


def attention_block_diagonal(q: np.ndarray, k: np.ndarray, v: np.ndarray, cu_seqlens: np.ndarray,
                             return_probs: bool = False):
    """Step O5 on q, k, v [T, heads, head_dim]: per image and head, softmax(q k^T / sqrt(dh)) v."""
    T, nH, dh = q.shape
    o = np.zeros_like(q)
    probs = []
    for i in range(len(cu_seqlens) - 1):
        a, b = int(cu_seqlens[i]), int(cu_seqlens[i + 1])
        for hd in range(nH):
            s = (q[a:b, hd, :] @ k[a:b, hd, :].T) / np.sqrt(float(dh))
            s = s - s.max(axis=1, keepdims=True)
            p = np.exp(s)
            p = p / p.sum(axis=1, keepdims=True)
            o[a:b, hd, :] = p @ v[a:b, hd, :]
            if return_probs:
                probs.append(p)
    return (o, probs) if return_probs else o


def merge_2x2(y: np.ndarray, merge_idx: np.ndarray) -> np.ndarray:
    """Step O9: M[o, q*h:(q+1)*h] = Y[merge_idx[o, q], :]."""
    Tm, nq = merge_idx.shape
    return y[merge_idx.reshape(-1)].reshape(Tm, nq * y.shape[1])


# ----------------------------------------------------------------------------- blocks / whole stage

def _f64(a):
    return None if a is None else np.asarray(a, dtype=np.float64)


def attention_sublayer(cfg, lw: Dict, x: np.ndarray, bk: Dict) -> np.ndarray:
    """Steps O2-O6: returns x + out_proj(attn(rope(qkv(rmsnorm(x)))))."""
    T = x.shape[0]
    h, nH, dh = cfg.hidden, cfg.heads, cfg.head_dim
    a = rmsnorm(x, _f64(lw["norm1_w"]), cfg.eps)
    qkv = linear(a, _f64(lw["qkv_w"]), _f64(lw["qkv_b"]))
    q = qkv[:, 0:h].reshape(T, nH, dh)
    k = qkv[:, h:2 * h].reshape(T, nH, dh)
    v = qkv[:, 2 * h:3 * h].reshape(T, nH, dh)
    if cfg.rope_theta > 0:
        q = rope_2d(q, bk["pos_row"], bk["pos_col"], cfg.rope_theta)
        k = rope_2d(k, bk["pos_row"], bk["pos_col"], cfg.rope_theta)
    o = attention_block_diagonal(q, k, v, bk["cu_seqlens"]).reshape(T, h)
    return x + linear(o, _f64(lw["out_w"]), _f64(lw["out_b"]))


def mlp_sublayer(cfg, lw: Dict, x: np.ndarray) -> np.ndarray:
    """Step O7."""
    b = rmsnorm(x, _f64(lw["norm2_w"]), cfg.eps)
    u = gelu(linear(b, _f64(lw["fc1_w"]), _f64(lw["fc1_b"])), cfg.act)
    return x + linear(u, _f64(lw["fc2_w"]), _f64(lw["fc2_b"]))


def block(cfg, lw: Dict, x: np.ndarray, bk: Dict) -> np.ndarray:
    """One encoder block (O2-O7) applied to a given block input x [T, hidden]."""
    return mlp_sublayer(cfg, lw, attention_sublayer(cfg, lw, _f64(x), bk))


def block_rows(cfg, lw: Dict, x: np.ndarray, bk: Dict, rows: Sequence[int]) -> np.ndarray:
    """Rows `rows` of block(cfg, lw, x, bk): the same definition (O2-O7) evaluated only for the chosen
    query tokens.  Keys and values are still formed for every token of the images those rows belong
    to; everything after attention is row-wise.  Lets a large batch be checked on sampled rows."""
    x = _f64(x)
    rows = np.asarray(rows, dtype=np.int64)
    h, nH, dh = cfg.hidden, cfg.heads, cfg.head_dim
    cu = bk["cu_seqlens"]
    out = np.empty((len(rows), h), dtype=np.float64)
    seg_of = np.searchsorted(cu, rows, side="right") - 1
    for i in np.unique(seg_of):
        a, b = int(cu[i]), int(cu[i + 1])
        sel = np.nonzero(seg_of == i)[0]
        local = rows[sel] - a
        an = rmsnorm(x[a:b], _f64(lw["norm1_w"]), cfg.eps)
        qkv = linear(an, _f64(lw["qkv_w"]), _f64(lw["qkv_b"]))
        q = qkv[:, 0:h].reshape(b - a, nH, dh)
        k = qkv[:, h:2 * h].reshape(b - a, nH, dh)
        v = qkv[:, 2 * h:3 * h].reshape(b - a, nH, dh)
        if cfg.rope_theta > 0:
            q = rope_2d(q, bk["pos_row"][a:b], bk["pos_col"][a:b], cfg.rope_theta)
            k = rope_2d(k, bk["pos_row"][a:b], bk["pos_col"][a:b], cfg.rope_theta)
        o = np.empty((len(local), nH, dh), dtype=np.float64)
        for hd in range(nH):
            sc = (q[local, hd, :] @ k[:, hd, :].T) / np.sqrt(float(dh))
            sc = sc - sc.max(axis=1, keepdims=True)
            p = np.exp(sc)
            p = p / p.sum(axis=1, keepdims=True)
            o[:, hd, :] = p @ v[:, hd, :]
        x1 = x[rows[sel]] + linear(o.reshape(len(local), h), _f64(lw["out_w"]), _f64(lw["out_b"]))
        out[sel] = mlp_sublayer(cfg, lw, x1)
    return out


def head(cfg, weights: Dict, x: np.ndarray, bk: Dict) -> np.ndarray:
    """Steps O8-O10 on the residual stream after the last block."""
    y = rmsnorm(_f64(x), _f64(weights["final_norm_w"]), cfg.eps) if cfg.final_norm else _f64(x)
    m = merge_2x2(y, bk["merge_idx"])
    f = linear(m, _f64(weights["proj_w1"]), _f64(weights["proj_b1"]))
    if weights.get("proj_w2") is not None:
        f = linear(gelu(f, cfg.act), _f64(weights["proj_w2"]), _f64(weights["proj_b2"]))
    return f


def encode(cfg, weights: Dict, patches: np.ndarray, grid_thw: Sequence[Sequence[int]],
           return_taps: bool = False):
    """The whole stage (Eq. 1): packed patches [T, K] -> features [Tm, out_dim] in float64.

    With return_taps, also returns the residual stream entering block 0, 1, ..., L-1 and
    leaving the last block (L+1 arrays [T, hidden]).
    """
    bk = bookkeeping(grid_thw, cfg.merge)
    x = linear(_f64(patches), _f64(weights["patch_w"]), _f64(weights["patch_b"]))
    taps = [x]
    for l in range(cfg.layers):
        x = block(cfg, weights["layers"][l], x, bk)
        taps.append(x)
    f = head(cfg, weights, x, bk)
    return (f, taps) if return_taps else f
