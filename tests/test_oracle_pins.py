"""Pins for the CPU oracle: things fixed by the paper or by mathematics, not by the oracle itself.

* pure-Python brute force of the whole stage on tiny inputs (independent loops, math module only)
* each step against a PyTorch CPU float64 library routine
* closed forms and invariants (softmax rows, RoPE isometry and relative-position property,
  block-diagonal isolation, identity blocks, RMS of normalised rows, GELU identities)
* the merged-row counts printed in the paper's E-P prefetching table (tests/golden/)
"""
import math
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import synth
from oracle import encoder_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------------------- brute force

def brute_force_encode(cfg, w, patches, grids):
    """Whole stage with scalar loops only; written separately from the oracle."""
    h, nH, dh, K, m = cfg.hidden, cfg.heads, cfg.head_dim, cfg.patch_dim, cfg.mlp
    # token table: (image, frame, row, col)
    toks = []
    starts = []
    for i, (t, gh, gw) in enumerate(grids):
        starts.append(len(toks))
        for f in range(t):
            for r in range(gh):
                for c in range(gw):
                    toks.append((i, f, r, c))
    T = len(toks)

    def lin(x, W, b, nout, nin):
        y = [[0.0] * nout for _ in range(len(x))]
        for j in range(len(x)):
            for o in range(nout):
                acc = 0.0
                for k_ in range(nin):
                    acc += float(x[j][k_]) * float(W[o][k_])
                y[j][o] = acc + (float(b[o]) if b is not None else 0.0)
        return y

    def norm(x, g):
        out = []
        for row in x:
            ms = sum(v * v for v in row) / len(row)
            out.append([v / math.sqrt(ms + cfg.eps) * float(g[c]) for c, v in enumerate(row)])
        return out

    def act(v):
        if cfg.act == synth.ACT_GELU_TANH:
            return 0.5 * v * (1.0 + math.tanh(math.sqrt(2.0 / math.pi) * (v + 0.044715 * v * v * v)))
        return 0.5 * v * (1.0 + math.erf(v / math.sqrt(2.0)))

    def rot(vec, r, c):
        # vec: one head's dh values
        out = list(vec)
        d2, nf = dh // 2, dh // 4
        for half, p in ((0, r), (1, c)):
            for f in range(nf):
                w_f = cfg.rope_theta ** (-(2.0 * f) / d2)
                i0, i1 = half * d2 + f, half * d2 + f + nf
                cs, sn = math.cos(p * w_f), math.sin(p * w_f)
                out[i0] = vec[i0] * cs - vec[i1] * sn
                out[i1] = vec[i1] * cs + vec[i0] * sn
        return out

    x = lin(patches.tolist(), w["patch_w"], w["patch_b"], h, K)
    for lw in w["layers"]:
        a = norm(x, lw["norm1_w"])
        qkv = lin(a, lw["qkv_w"], lw["qkv_b"], 3 * h, h)
        o = [[0.0] * h for _ in range(T)]
        for hd in range(nH):
            qs, ks, vs = [], [], []
            for j in range(T):
                _, _, r, c = toks[j]
                qs.append(rot(qkv[j][hd * dh:(hd + 1) * dh], r, c))
                ks.append(rot(qkv[j][h + hd * dh: h + (hd + 1) * dh], r, c))
                vs.append(qkv[j][2 * h + hd * dh: 2 * h + (hd + 1) * dh])
            for j in range(T):
                same = [jj for jj in range(T) if toks[jj][0] == toks[j][0]]
                sc = [sum(qs[j][e] * ks[jj][e] for e in range(dh)) / math.sqrt(dh) for jj in same]
                mx = max(sc)
                ex = [math.exp(s - mx) for s in sc]
                z = sum(ex)
                for e in range(dh):
                    o[j][hd * dh + e] = sum(ex[n_] / z * vs[jj][e] for n_, jj in enumerate(same))
        proj = lin(o, lw["out_w"], lw["out_b"], h, h)
        x = [[x[j][c] + proj[j][c] for c in range(h)] for j in range(T)]
        b = norm(x, lw["norm2_w"])
        u = lin(b, lw["fc1_w"], lw["fc1_b"], m, h)
        u = [[act(v) for v in row] for row in u]
        d = lin(u, lw["fc2_w"], lw["fc2_b"], h, m)
        x = [[x[j][c] + d[j][c] for c in range(h)] for j in range(T)]
    y = norm(x, w["final_norm_w"])
    merged = []
    for i, (t, gh, gw) in enumerate(grids):
        for f in range(t):
            for R in range(gh // 2):
                for C in range(gw // 2):
                    row = []
                    for dy in (0, 1):
                        for dx in (0, 1):
                            j = starts[i] + f * gh * gw + (2 * R + dy) * gw + (2 * C + dx)
                            row.extend(y[j])
                    merged.append(row)
    if w["proj_w2"] is None:
        return np.array(lin(merged, w["proj_w1"], w["proj_b1"], cfg.out_dim, 4 * h))
    z = lin(merged, w["proj_w1"], w["proj_b1"], cfg.proj_hidden, 4 * h)
    z = [[act(v) for v in row] for row in z]
    return np.array(lin(z, w["proj_w2"], w["proj_b2"], cfg.out_dim, cfg.proj_hidden))


def _boost(w, scale=20.0):
    """Make tiny-model activations O(1) so every term matters (weights N(0,0.02) are too flat)."""
    out = {k: (v * scale if (v is not None and k.endswith(("_w", "_w1", "_w2")) and v.ndim == 2) else v)
           for k, v in w.items() if k != "layers"}
    out["layers"] = [{k: (v * scale if v.ndim == 2 else v) for k, v in lw.items()} for lw in w["layers"]]
    return out


@pytest.mark.parametrize("variant", [
    dict(grids=[(1, 2, 2), (2, 2, 4)], act=synth.ACT_GELU_TANH, proj_kind=synth.PROJ_LINEAR, layers=2),
    dict(grids=[(1, 4, 2), (1, 2, 2), (1, 2, 6)], act=synth.ACT_GELU_ERF, proj_kind=synth.PROJ_MLP, layers=1),
])
def test_whole_stage_matches_brute_force(variant):
    cfg = synth.tiny_variant(head_dim=8, heads=2, layers=variant["layers"], mlp=12, patch=1,
                             act=variant["act"], proj_kind=variant["proj_kind"], out_dim=6)
    w = _boost(synth.make_weights(cfg, seed=3))
    grids = variant["grids"]
    patches = synth.make_patches(cfg, grids, seed=4)
    got = O.encode(cfg, w, patches, grids)
    ref = brute_force_encode(cfg, w, patches, grids)
    assert got.shape == ref.shape == (synth.num_tokens(grids) // 4, cfg.out_dim)
    assert np.max(np.abs(got - ref)) <= 1e-12 * max(1.0, np.max(np.abs(ref)))
    assert np.std(ref) > 1e-3  # the comparison is not between two near-zero tensors


# ----------------------------------------------------------------------------- library routines per step

def _t(a):
    return torch.from_numpy(np.asarray(a, dtype=np.float64))


def test_rmsnorm_against_torch():
    rng = np.random.default_rng(0)
    x, g = rng.standard_normal((7, 40)), rng.standard_normal(40)
    ref = F.rms_norm(_t(x), (40,), _t(g), eps=1e-6).numpy()
    np.testing.assert_allclose(O.rmsnorm(x, g, 1e-6), ref, rtol=1e-13, atol=1e-13)


@pytest.mark.parametrize("act,approx", [(O.ACT_GELU_TANH, "tanh"), (O.ACT_GELU_ERF, "none")])
def test_gelu_against_torch(act, approx):
    x = np.linspace(-6, 6, 241)
    np.testing.assert_allclose(O.gelu(x, act), F.gelu(_t(x), approximate=approx).numpy(), rtol=1e-13, atol=1e-14)
    assert O.gelu(np.zeros(1), act)[0] == 0.0
    np.testing.assert_allclose(O.gelu(x, act) - O.gelu(-x, act), x, rtol=0, atol=1e-14)


def test_gelu_flavours_differ_and_printed_constants():
    # gelu_erf(1) = Phi(1) = 0.841344746...; the tanh flavour is a different function
    assert abs(O.gelu(np.array([1.0]), O.ACT_GELU_ERF)[0] - 0.8413447460685429) < 1e-15
    assert abs(O.gelu(np.array([1.0]), O.ACT_GELU_TANH)[0] - 0.8411919906082768) < 1e-12


def test_linear_against_torch():
    rng = np.random.default_rng(1)
    x, w, b = rng.standard_normal((5, 9)), rng.standard_normal((4, 9)), rng.standard_normal(4)
    np.testing.assert_allclose(O.linear(x, w, b), F.linear(_t(x), _t(w), _t(b)).numpy(), rtol=1e-13, atol=1e-13)


def test_attention_against_torch_sdpa_per_segment():
    rng = np.random.default_rng(2)
    cu = np.array([0, 5, 5 + 12, 5 + 12 + 3])
    T, nH, dh = int(cu[-1]), 3, 12
    q, k, v = (rng.standard_normal((T, nH, dh)) * 2 for _ in range(3))
    got = O.attention_block_diagonal(q, k, v, cu)
    for i in range(3):
        a, b = cu[i], cu[i + 1]
        ref = F.scaled_dot_product_attention(_t(q[a:b]).transpose(0, 1), _t(k[a:b]).transpose(0, 1),
                                             _t(v[a:b]).transpose(0, 1)).transpose(0, 1).numpy()
        np.testing.assert_allclose(got[a:b], ref, rtol=1e-12, atol=1e-13)


def test_rope_against_complex_multiplication():
    """Independent statement: the pair (x_f, x_{f+nf}) is the complex number x_f + i x_{f+nf} times e^{i p w_f}."""
    rng = np.random.default_rng(3)
    T, nH, dh, theta = 11, 2, 24, 10000.0
    x = rng.standard_normal((T, nH, dh))
    pr, pc = rng.integers(0, 90, T), rng.integers(0, 90, T)
    got = O.rope_2d(x, pr, pc, theta)
    d2, nf = dh // 2, dh // 4
    for half, p in ((0, pr), (1, pc)):
        z = x[:, :, half * d2: half * d2 + nf] + 1j * x[:, :, half * d2 + nf: (half + 1) * d2]
        w_f = np.array([theta ** (-2.0 * f / d2) for f in range(nf)])
        zr = z * np.exp(1j * p[:, None, None] * w_f[None, None, :])
        np.testing.assert_allclose(got[:, :, half * d2: half * d2 + nf], zr.real, rtol=1e-12, atol=1e-12)
        np.testing.assert_allclose(got[:, :, half * d2 + nf: (half + 1) * d2], zr.imag, rtol=1e-12, atol=1e-12)


def test_rope_frequencies_first_and_last():
    # omega_0 = 1 (angle = position), last frequency = theta^(-(2nf-2)/d2)
    dh, theta = 8, 10000.0
    x = np.zeros((1, 1, dh)); x[0, 0, 0] = 1.0; x[0, 0, 5] = 1.0   # row-half f=0, col-half f=1
    y = O.rope_2d(x, np.array([2]), np.array([3]), theta)[0, 0]
    assert abs(y[0] - math.cos(2.0)) < 1e-15 and abs(y[2] - math.sin(2.0)) < 1e-15
    w1 = theta ** (-2.0 / 4.0)
    assert abs(y[5] - math.cos(3 * w1)) < 1e-15 and abs(y[7] - math.sin(3 * w1)) < 1e-15


# ----------------------------------------------------------------------------- invariants

def test_softmax_rows_sum_to_one_and_convex_hull():
    rng = np.random.default_rng(4)
    cu = np.array([0, 9, 20])
    q, k, v = (rng.standard_normal((20, 2, 8)) * 3 for _ in range(3))
    o, probs = O.attention_block_diagonal(q, k, v, cu, return_probs=True)
    for p in probs:
        np.testing.assert_allclose(p.sum(axis=1), 1.0, rtol=0, atol=1e-14)
        assert (p >= 0).all()
    for i in range(2):
        a, b = cu[i], cu[i + 1]
        assert (o[a:b] <= v[a:b].max(axis=0, keepdims=True) + 1e-12).all()
        assert (o[a:b] >= v[a:b].min(axis=0, keepdims=True) - 1e-12).all()
    v_same = np.broadcast_to(v[:1], v.shape).copy()
    np.testing.assert_allclose(O.attention_block_diagonal(q, k, v_same, cu), v_same, atol=1e-14)


def test_rope_isometry_identity_and_relative_property():
    rng = np.random.default_rng(5)
    T, nH, dh = 16, 2, 16
    q, k = rng.standard_normal((T, nH, dh)), rng.standard_normal((T, nH, dh))
    pr, pc = rng.integers(0, 50, T), rng.integers(0, 50, T)
    qr = O.rope_2d(q, pr, pc, 10000.0)
    np.testing.assert_allclose(np.linalg.norm(qr, axis=-1), np.linalg.norm(q, axis=-1), rtol=1e-13)
    np.testing.assert_array_equal(O.rope_2d(q, np.zeros(T, int), np.zeros(T, int), 10000.0), q)
    kr = O.rope_2d(k, pr, pc, 10000.0)
    s0 = np.einsum("ihd,jhd->hij", qr, kr)
    s1 = np.einsum("ihd,jhd->hij", O.rope_2d(q, pr + 7, pc + 13, 10000.0), O.rope_2d(k, pr + 7, pc + 13, 10000.0))
    np.testing.assert_allclose(s0, s1, rtol=1e-11, atol=1e-11)
    # rows and columns are not interchangeable
    assert np.max(np.abs(O.rope_2d(q, pc, pr, 10000.0) - qr)) > 1e-3


def test_rmsnorm_unit_rms_and_scale_invariance():
    rng = np.random.default_rng(6)
    x = rng.standard_normal((5, 64)) * 3
    y = O.rmsnorm(x, np.ones(64), 1e-6)
    np.testing.assert_allclose(np.sqrt(np.mean(y * y, axis=1)), 1.0, rtol=1e-6)
    np.testing.assert_allclose(O.rmsnorm(4.0 * x, np.ones(64), 1e-12), O.rmsnorm(x, np.ones(64), 1e-12), rtol=1e-10)
    # eps sits inside the square root: a zero row maps to zero, a tiny row is damped by sqrt(eps)
    tiny = np.full((1, 4), 1e-6)
    np.testing.assert_allclose(O.rmsnorm(tiny, np.ones(4), 1e-6), tiny / math.sqrt(1e-12 + 1e-6), rtol=1e-12)


def _small_model(proj_kind=synth.PROJ_MLP):
    cfg = synth.tiny_variant(head_dim=8, heads=2, layers=2, mlp=24, patch=2, proj_kind=proj_kind, out_dim=10)
    return cfg, _boost(synth.make_weights(cfg, seed=11))


def test_block_diagonal_isolation_and_image_permutation():
    cfg, w = _small_model()
    grids = [(1, 4, 6), (2, 2, 2), (1, 6, 4)]
    patches = synth.make_patches(cfg, grids, seed=5)
    bk = O.bookkeeping(grids)
    cu, cuo = bk["cu_seqlens"], bk["cu_out"]
    full = O.encode(cfg, w, patches, grids)
    for i in range(3):
        alone = O.encode(cfg, w, patches[cu[i]:cu[i + 1]], [grids[i]])
        # BLAS may block rows differently for different batch sizes: equal up to fp64 rounding
        np.testing.assert_allclose(full[cuo[i]:cuo[i + 1]], alone, rtol=1e-11, atol=1e-12)
    # perturb the other images: image 1 must not move at all beyond rounding
    p2 = patches.copy(); p2[cu[0]:cu[1]] += 1.0; p2[cu[2]:cu[3]] *= -2.0
    np.testing.assert_allclose(O.encode(cfg, w, p2, grids)[cuo[1]:cuo[2]], full[cuo[1]:cuo[2]], rtol=1e-11, atol=1e-12)
    # permuting the image list permutes the feature blocks
    order = [2, 0, 1]
    pp = np.concatenate([patches[cu[i]:cu[i + 1]] for i in order])
    perm = O.encode(cfg, w, pp, [grids[i] for i in order])
    ref = np.concatenate([full[cuo[i]:cuo[i + 1]] for i in order])
    np.testing.assert_allclose(perm, ref, rtol=1e-11, atol=1e-12)
    # and attention really mixes tokens inside an image
    p3 = patches.copy(); p3[cu[1]] += 1.0
    assert np.max(np.abs(O.encode(cfg, w, p3, grids)[cuo[1]:cuo[2]] - full[cuo[1]:cuo[2]])) > 1e-6


def test_identity_blocks_reduce_to_closed_form():
    cfg, w = _small_model(proj_kind=synth.PROJ_LINEAR)
    for lw in w["layers"]:
        for k_ in ("out_w", "out_b", "fc2_w", "fc2_b"):
            lw[k_] = np.zeros_like(lw[k_])
    grids = [(1, 2, 4), (1, 4, 2)]
    patches = synth.make_patches(cfg, grids, seed=6)
    x = _t(patches) @ _t(w["patch_w"]).T + _t(w["patch_b"])
    y = F.rms_norm(x, (cfg.hidden,), _t(w["final_norm_w"]), eps=cfg.eps)
    idx = torch.from_numpy(O.bookkeeping(grids)["merge_idx"].astype(np.int64))
    m = y[idx.reshape(-1)].reshape(idx.shape[0], -1)
    ref = (m @ _t(w["proj_w1"]).T + _t(w["proj_b1"])).numpy()
    np.testing.assert_allclose(O.encode(cfg, w, patches, grids), ref, rtol=1e-12, atol=1e-13)


def test_taps_chain_blocks():
    cfg, w = _small_model()
    grids = [(1, 2, 2), (1, 4, 4)]
    patches = synth.make_patches(cfg, grids, seed=7)
    f, taps = O.encode(cfg, w, patches, grids, return_taps=True)
    assert len(taps) == cfg.layers + 1
    bk = O.bookkeeping(grids)
    for l in range(cfg.layers):
        np.testing.assert_array_equal(O.block(cfg, w["layers"][l], taps[l], bk), taps[l + 1])
    np.testing.assert_array_equal(O.head(cfg, w, taps[-1], bk), f)


# ----------------------------------------------------------------------------- bookkeeping

def _golden_rows():
    rows = []
    with open(os.path.join(GOLDEN, "e2p_feature_rows.txt")) as fh:
        for line in fh:
            if line.strip() and not line.startswith("#"):
                rows.append(tuple(int(v) for v in line.split()))
    return rows


def test_paper_feature_row_counts():
    rows = _golden_rows()
    assert len(rows) == 5
    for H, W, gh, gw, n in rows:
        assert gh == 2 * round(H / 28) and gw == 2 * round(W / 28)
        bk = O.bookkeeping([(1, gh, gw)])
        assert bk["merge_idx"].shape == (n, 4)
        assert bk["cu_out"].tolist() == [0, n]
        assert bk["cu_seqlens"].tolist() == [0, 4 * n]
    # as one packed batch: Eq. 1's n per image, stacked
    bk = O.bookkeeping([(1, r[2], r[3]) for r in rows])
    assert np.diff(bk["cu_out"]).tolist() == [r[4] for r in rows]


def test_bookkeeping_closed_forms_and_gather_index():
    grids = [(1, 4, 6), (3, 2, 4), (1, 2, 2)]
    bk = O.bookkeeping(grids)
    T = sum(t * h * w for t, h, w in grids)
    assert bk["cu_seqlens"][-1] == T and bk["cu_out"][-1] == T // 4
    # every token is gathered exactly once
    assert sorted(bk["merge_idx"].reshape(-1).tolist()) == list(range(T))
    # explicit small case: grid (1,2,4): tokens 0..7 = rows [0 1 2 3],[4 5 6 7]
    bk1 = O.bookkeeping([(1, 2, 4)])
    assert bk1["merge_idx"].tolist() == [[0, 1, 4, 5], [2, 3, 6, 7]]
    assert bk1["pos_row"].tolist() == [0, 0, 0, 0, 1, 1, 1, 1]
    assert bk1["pos_col"].tolist() == [0, 1, 2, 3, 0, 1, 2, 3]
    # frames reuse positions; second image starts at zero again
    bk2 = O.bookkeeping([(2, 2, 2), (1, 2, 2)])
    assert bk2["pos_row"].tolist() == [0, 0, 1, 1] * 3
    assert bk2["pos_col"].tolist() == [0, 1, 0, 1] * 3
    assert bk2["merge_idx"].tolist() == [[0, 1, 2, 3], [4, 5, 6, 7], [8, 9, 10, 11]]
    # Y[j,:] = j  =>  merged row holds its four source indices
    y = np.arange(T, dtype=np.float64)[:, None] * np.ones((1, 3))
    m = O.merge_2x2(y, bk["merge_idx"])
    assert m.shape == (T // 4, 12)
    np.testing.assert_array_equal(m[:, ::3], bk["merge_idx"].astype(np.float64))
    with pytest.raises(ValueError):
        O.bookkeeping([(1, 3, 4)])
    assert O.bookkeeping([])["cu_seqlens"].tolist() == [0]


def test_parameter_counts_match_paper_size_classes():
    """Table 1 of the paper lists 0.6 B and 6 B ViTs; the configurations are in those classes."""
    def count(cfg):
        h, m, K = cfg.hidden, cfg.mlp, cfg.patch_dim
        per_layer = 3 * h * h + 3 * h + h * h + h + 2 * h * m + m + h + 2 * h
        proj = 4 * h * cfg.proj_hidden + cfg.proj_hidden + cfg.proj_hidden * cfg.out_dim + cfg.out_dim
        return K * h + h + cfg.layers * per_layer + h + proj
    assert 0.40e9 < count(synth.VIT_06B) < 0.70e9
    assert 5.0e9 < count(synth.VIT_6B) < 6.5e9
    w = synth.make_weights(synth.tiny_variant(proj_kind=synth.PROJ_MLP))
    n = sum(v.size for v in w.values() if isinstance(v, np.ndarray)) + \
        sum(v.size for lw in w["layers"] for v in lw.values())
    assert n == count(synth.tiny_variant(proj_kind=synth.PROJ_MLP))


def test_synthetic_recipe():
    x = synth.normal(0, "a", (20000,), 0.02, 0.0, synth.DTYPE_FP32)
    assert abs(float(x.std()) - 0.02) < 1e-3 and abs(float(x.mean())) < 1e-3
    np.testing.assert_array_equal(x, synth.normal(0, "a", (20000,), 0.02, 0.0, synth.DTYPE_FP32))
    assert not np.array_equal(x, synth.normal(0, "b", (20000,), 0.02, 0.0, synth.DTYPE_FP32))
    b = synth.normal(0, "a", (1000,), 1.0, 0.0, synth.DTYPE_BF16)
    np.testing.assert_array_equal(torch.from_numpy(b).to(torch.bfloat16).float().numpy(), b)
    ref = torch.from_numpy(synth.normal(0, "a", (1000,), 1.0, 0.0, synth.DTYPE_FP32)).to(torch.bfloat16).float().numpy()
    np.testing.assert_array_equal(b, ref)
    g = synth.grid_variable_resolution(32, 16, 0)
    assert len(g) == 32 and all(t == 1 and 14 <= h <= 84 and h % 2 == 0 and 14 <= w <= 84 and w % 2 == 0 for t, h, w in g)
    assert synth.num_tokens(synth.WORKLOADS["cfg1_vit06b_b8_448"][1]) == 6272
    assert synth.num_tokens(synth.WORKLOADS["cfg3_vit06b_long"][1]) == 16384 + 6272
    assert synth.num_tokens(synth.WORKLOADS["cfg4_vit6b_b16_448"][1]) == 16384


def test_block_rows_is_block_restricted_to_rows():
    """The sampled-row form used for large batches equals the full block on those rows."""
    cfg = synth.tiny_variant(head_dim=8, heads=2, layers=1, mlp=24, patch=2)
    grids = [(1, 4, 6), (2, 2, 4), (1, 6, 2)]
    w = synth.make_weights(cfg, seed=11)
    bk = O.bookkeeping(grids)
    T = int(bk["cu_seqlens"][-1])
    x = synth.normal(12, "x", (T, cfg.hidden), 1.0, 0.0, synth.DTYPE_FP32).astype(np.float64)
    full = O.block(cfg, w["layers"][0], x, bk)
    rows = [0, 5, 23, 24, 30, 39, 40, T - 1]
    got = O.block_rows(cfg, w["layers"][0], x, bk, rows)
    assert np.allclose(got, full[rows], rtol=0, atol=1e-12)


# ----------------------------------------------------------------------------- pixels -> patches

def test_patchify_matches_brute_force_loops():
    cfg = synth.tiny_variant(patch=2, temporal_patch=2)
    grids = [(1, 2, 4), (2, 4, 2)]
    frames = synth.make_frames(cfg, grids, seed=3)
    mean, std = (0.4, 0.5, 0.6), (0.2, 0.25, 0.3)
    got = O.patchify(frames, grids, cfg.patch, cfg.temporal_patch, mean, std)
    P, Tp, C = cfg.patch, cfg.temporal_patch, cfg.in_channels
    want = []
    for fr, (t, h, w) in zip(frames, grids):
        for f in range(t):
            for r in range(h):
                for c in range(w):
                    vec = []
                    for ch in range(C):
                        for tp in range(Tp):
                            for y in range(P):
                                for x in range(P):
                                    v = float(fr[f * Tp + tp, ch, r * P + y, c * P + x])
                                    vec.append((v / 255.0 - mean[ch]) / std[ch])
                    want.append(vec)
    assert got.shape == (synth.num_tokens(grids), cfg.patch_dim)
    assert np.allclose(got, np.asarray(want), rtol=0, atol=1e-14)


def test_patchify_constant_and_position_coded_frames():
    P, Tp, C = 4, 1, 3
    grids = [(1, 2, 3)]
    # constant image: every element of every patch is (v/255 - mean)/std of its channel
    fr = np.full((1, C, 2 * P, 3 * P), 51, dtype=np.uint8)
    out = O.patchify([fr], grids, P, Tp, (0.2, 0.2, 0.2), (0.5, 1.0, 2.0))
    assert np.allclose(out[:, : P * P], 0.0) and np.allclose(out.reshape(6, C, P * P)[:, 1], 0.0)
    # pixel value codes (row, column): patch (r, c) must hold exactly its own window, row-major
    yy, xx = np.meshgrid(np.arange(2 * P), np.arange(3 * P), indexing="ij")
    fr = np.broadcast_to((yy * 12 + xx).astype(np.uint8), (1, C, 2 * P, 3 * P)).copy()
    out = O.patchify([fr], grids, P, Tp, (0.0,) * 3, (1.0 / 255.0,) * 3)     # identity scaling
    for r in range(2):
        for c in range(3):
            win = fr[0, 0, r * P:(r + 1) * P, c * P:(c + 1) * P].astype(np.float64).reshape(-1)
            assert np.allclose(out[r * 3 + c, : P * P], win)


# ----------------------------------------------------------------------------- content hash

def test_content_hash_against_vectorised_restatement_and_properties():
    rng = np.random.default_rng(5)
    data = rng.integers(0, 256, size=8 * 37, dtype=np.uint8).tobytes()
    h = O.content_hash(data)
    # an independent restatement with numpy's wrapping uint64 arithmetic
    w = np.frombuffer(data, dtype="<u8")
    with np.errstate(over="ignore"):
        z = w ^ (np.arange(1, w.size + 1, dtype=np.uint64) * np.uint64(0x9E3779B97F4A7C15))
        z = (z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
        z = z ^ (z >> np.uint64(31))
        acc = int(z.sum(dtype=np.uint64)) + len(data)
    assert h == O._mix64(acc)
    assert O.content_hash(b"") == 0                       # mix(0) = 0: the finalizer fixes zero
    # SplitMix64's published first output for seed 0 is mix(GOLDEN): pins the finalizer's constants
    assert O._mix64(0x9E3779B97F4A7C15) == 0xE220A8397B1DCDAF
    flipped = bytearray(data); flipped[100] ^= 0x10
    assert O.content_hash(bytes(flipped)) != h            # a single bit changes the key
    swapped = data[8:16] + data[0:8] + data[16:]
    assert O.content_hash(swapped) != h                   # word order matters
    assert O.content_hash(data + bytes(8)) != h           # trailing zeros matter
    with pytest.raises(ValueError):
        O.content_hash(b"abc")


# ----------------------------------------------------------------------------- 8-bit floating-point variant

def test_round_to_e4m3_hand_computed_values():
    """Values worked out by hand from the format's definition (sign, 4 exponent bits with bias 7, 3 mantissa
    bits, largest finite value 448, subnormal step 2^-9, ties to the even mantissa, saturation)."""
    cases = [
        (0.3, 0.3125),        # binade [0.25, 0.5): step 2^-5; 0.3 / 2^-5 = 9.6 -> 10
        (17.0, 16.0),         # binade [16, 32): step 2; 8.5 -> 8 (tie to even)
        (19.0, 20.0),         # 9.5 -> 10 (tie to even)
        (21.0, 20.0),         # 10.5 -> 10
        (448.0, 448.0), (449.0, 448.0), (1e6, 448.0), (-500.0, -448.0),     # saturation
        (464.0, 448.0),       # would round to 480, which the format does not have
        (2.0 ** -9, 2.0 ** -9), (0.001, 2.0 ** -9), (0.0009, 0.0),          # subnormals: step 2^-9
        (1.5 * 2.0 ** -9, 2.0 ** -8),                                        # tie between 1 and 2 steps -> 2 (even)
        (2.0 ** -6, 2.0 ** -6), (0.0, 0.0), (-1.0625, -1.0), (1.0625 + 1e-9, 1.125),
    ]
    for v, want in cases:
        assert float(O.round_to_e4m3(np.array([v]))[0]) == want, (v, want)
    # the sign of a zero survives (IEEE convention; the format has a negative zero, code 0x80)
    z = O.round_to_e4m3(np.array([-0.0, -1e-9, 0.0]))
    assert np.signbit(z).tolist() == [True, True, False] and O.e4m3_bits(z).tolist() == [0x80, 0x80, 0]
    # every one of the 2 x 127 finite codes maps to itself, and the codes come back
    codes = np.array([c for c in range(256) if (c & 0x7F) != 0x7F], dtype=np.uint8)
    sign = np.where(codes & 0x80, -1.0, 1.0)
    ef, mf = ((codes >> 3) & 0xF).astype(np.float64), (codes & 7).astype(np.float64)
    vals = sign * np.where(ef > 0, np.exp2(ef - 7) * (1 + mf / 8), mf * 2.0 ** -9)
    assert np.array_equal(O.round_to_e4m3(vals), vals)
    nonzero = vals != 0
    assert np.array_equal(O.e4m3_bits(vals[nonzero]), codes[nonzero])
    assert np.max(np.abs(vals)) == 448.0


def test_round_to_e4m3_agrees_with_the_library_conversion():
    """Inside the finite range PyTorch's CPU conversion to float8_e4m3fn is the same rounding."""
    torch = pytest.importorskip("torch")
    if not hasattr(torch, "float8_e4m3fn"):
        pytest.skip("no float8 in this torch")
    rng = np.random.default_rng(0)
    v = np.concatenate([rng.standard_normal(20000) * 30, rng.standard_normal(20000) * 0.01,
                        rng.uniform(-440, 440, 20000)]).astype(np.float32)
    lib = torch.from_numpy(v).to(torch.float8_e4m3fn).to(torch.float32).numpy().astype(np.float64)
    assert np.array_equal(O.round_to_e4m3(v), lib)


def test_quantize_rows_and_linear_e4m3_properties():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((7, 40)) * np.array([1e-3, 1, 5, 100, 0.2, 3, 1])[:, None]
    x[4, :] = 0.0
    q, s = O.quantize_e4m3_rows(x)
    assert s[4] == 1.0 and np.all(q[4] == 0)
    amax = np.max(np.abs(x.astype(np.float32)), axis=1)
    for i in (0, 1, 2, 3, 5, 6):
        assert np.max(np.abs(q[i])) == 448.0                         # the largest element of a row lands on 448
        assert abs(s[i] * 448.0 / amax[i] - 1) < 1e-6
    # relative error of an element at most half a step of its binade: 2^-4 of the value (normal range)
    big = np.abs(q) >= 2.0 ** -6
    rel = np.abs(q * s[:, None] - x)[big] / np.abs(x)[big]
    assert rel.max() <= 2.0 ** -4 + 1e-6
    # values that are already E4M3 multiples of the row scale pass through exactly: linear_e4m3 == plain product
    xs = O.round_to_e4m3(rng.uniform(-448, 448, (5, 16)))
    ws = O.round_to_e4m3(rng.uniform(-448, 448, (3, 16)))
    xs[:, 0], ws[:, 0] = 448.0, -448.0                               # every row's scale becomes exactly 1
    b = rng.standard_normal(3)
    assert np.allclose(O.linear_e4m3(xs, ws, b), xs @ ws.T + b, rtol=0, atol=1e-9)
    # scale invariance: scaling a row of x by a power of two scales its outputs by the same factor, exactly
    x2 = x.copy(); x2[1] *= 8.0
    w = rng.standard_normal((6, 40))
    y, y2 = O.linear_e4m3(x, w, None), O.linear_e4m3(x2, w, None)
    assert np.array_equal(y2[1], 8.0 * y[1]) and np.array_equal(y2[0], y[0])
