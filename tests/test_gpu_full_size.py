"""GPU parity at the benchmark configurations' full sizes, in the launch configuration bench.py times.

The oracle cannot evaluate these batches whole in reasonable time, so each case compares what it can
compute exactly:
  * an image's features do not depend on the rest of the batch (block-diagonal attention), so the
    features of one image of the full batch are compared with the oracle's encode of that image alone;
  * a block's output rows are compared, for sampled query rows, with the oracle's block evaluated on
    the GPU's own block input (keys and values of the whole image, every other step row-wise).
Tolerances: relative Frobenius error <= 1e-2 per block, <= 3e-2 on final features (bf16 configurations).
"""
import dataclasses

import numpy as np
import pytest
import torch

import synth
import paper_2601_11590_b200 as epd
from oracle import encoder_oracle as O
from tests.metrics import assert_parity, rel_err, worst_row_err

pytestmark = pytest.mark.gpu

TOL_BLOCK = 1e-2
TOL_FINAL = 3e-2


def to_np(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


@pytest.fixture(scope="module", autouse=True)
def _lib():
    from paper_2601_11590_b200 import build
    build.build_library()
    epd.load_library()


def _encode(cfg, grids, w, seed, taps=False):
    T = synth.num_tokens(grids)
    K = cfg.patch_dim
    ld = (K + 7) // 8 * 8
    enc = epd.Encoder(cfg, w, max_tokens=T, max_images=len(grids), max_grid=max(max(g[1], g[2]) for g in grids))
    patches = synth.make_patches(cfg, grids, seed=seed)
    p = torch.zeros((T, ld), dtype=torch.bfloat16, device="cuda")
    p[:, :K] = epd.to_device(patches, cfg.dtype)
    tap_bufs = None
    if taps:
        tap_bufs = [torch.zeros((T, cfg.hidden), dtype=torch.float32, device="cuda") for _ in range(cfg.layers + 1)]
        enc.set_taps(tap_bufs)
    feats, cu_rows = enc.encode(p, grids)
    torch.cuda.synchronize()
    assert enc.last_status() == epd.EPD_OK
    return enc, patches, feats, cu_rows, tap_bufs


def _sampled_rows(bk, images, per_image, seed):
    """Rows from the given images: first and last token, rows around tile boundaries, random rows."""
    rng = np.random.default_rng(seed)
    cu = bk["cu_seqlens"]
    rows = []
    for i in images:
        a, b = int(cu[i]), int(cu[i + 1])
        n = b - a
        fixed = [0, n - 1, min(111, n - 1), min(112, n - 1), min(127, n - 1), min(128, n - 1), n // 2]
        extra = rng.integers(0, n, size=max(0, per_image - len(fixed))).tolist()
        rows += [a + r for r in sorted(set(fixed + extra))]
    return np.asarray(rows, dtype=np.int64)


def _check_blocks_on_rows(cfg, w, grids, taps, images, per_image, seed):
    bk = O.bookkeeping(grids)
    rows = _sampled_rows(bk, images, per_image, seed)
    errs = []
    for l in range(cfg.layers):
        x_in = to_np(taps[l])
        want = O.block_rows(cfg, w["layers"][l], x_in, bk, rows)
        got = to_np(taps[l + 1][torch.from_numpy(rows).cuda()])
        errs.append(assert_parity(got, want, TOL_BLOCK, f"block {l}"))
    return errs


def test_cfg1_full_batch_one_image_end_to_end():
    """The benchmark's default workload (8 x 448x448, 27 layers): image 3's features against the oracle's
    encode of image 3 alone."""
    cfg, grids = synth.WORKLOADS["cfg1_vit06b_b8_448"]
    w = synth.make_weights(cfg, seed=0)
    enc, patches, feats, cu_rows, _ = _encode(cfg, grids, w, seed=0)
    bk = O.bookkeeping(grids)
    assert np.array_equal(cu_rows, bk["cu_out"])
    i = 3
    a, b = int(bk["cu_seqlens"][i]), int(bk["cu_seqlens"][i + 1])
    ref = O.encode(cfg, w, patches[a:b], [grids[i]])
    got = to_np(feats[cu_rows[i]:cu_rows[i + 1]])
    e = assert_parity(got, ref, TOL_FINAL, "cfg1 image 3")
    print("cfg1 image 3 final", e, "worst row", worst_row_err(got, ref))
    assert torch.isfinite(feats.float()).all()
    enc.close()


def test_cfg3_long_sequences_blocks_on_sampled_rows():
    """The long-sequence grid list (one 16384-token image + one 8-frame clip of 6272 tokens) at the
    encoder's full widths, two layers: every block on sampled rows of both items."""
    cfg0, grids = synth.WORKLOADS["cfg3_vit06b_long"]
    cfg = cfg0.with_layers(2)
    w = synth.make_weights(cfg, seed=1)
    enc, patches, feats, cu_rows, taps = _encode(cfg, grids, w, seed=1, taps=True)
    errs = _check_blocks_on_rows(cfg, w, grids, taps, images=[0, 1], per_image=40, seed=2)
    print("cfg3 blocks", errs)
    assert feats.shape[0] == synth.num_tokens(grids) // 4 and torch.isfinite(feats.float()).all()
    enc.close()


def test_cfg2_variable_resolution_blocks_on_sampled_rows():
    """The 32 variable-resolution images (seed 0) at full widths, one layer: the block on sampled rows
    of the largest, the smallest and two other images; bookkeeping of the whole batch bit-exact."""
    cfg0, grids = synth.WORKLOADS["cfg2_vit06b_var32"]
    cfg = cfg0.with_layers(1)
    w = synth.make_weights(cfg, seed=3)
    enc, patches, feats, cu_rows, taps = _encode(cfg, grids, w, seed=3, taps=True)
    bk = O.bookkeeping(grids)
    T = synth.num_tokens(grids)
    got = enc.debug_bookkeeping(len(grids), T)
    for key in ("cu_seqlens", "pos_row", "pos_col", "merge_idx"):
        assert np.array_equal(got[key], bk[key]), key
    assert np.array_equal(cu_rows, bk["cu_out"])
    lens = np.diff(bk["cu_seqlens"])
    images = sorted({int(np.argmax(lens)), int(np.argmin(lens)), 5, 17})
    errs = _check_blocks_on_rows(cfg, w, grids, taps, images=images, per_image=24, seed=4)
    print("cfg2 T", T, "blocks", errs)
    enc.close()


def test_cfg4_6b_widths_block_on_sampled_rows():
    """The 6B-class widths (hidden 3200, 25 heads x 128, MLP 12800, erf GELU) on the benchmark's 16
    images of 1024 tokens, one layer."""
    cfg0, grids = synth.WORKLOADS["cfg4_vit6b_b16_448"]
    cfg = cfg0.with_layers(1)
    w = synth.make_weights(cfg, seed=5)
    enc, patches, feats, cu_rows, taps = _encode(cfg, grids, w, seed=5, taps=True)
    errs = _check_blocks_on_rows(cfg, w, grids, taps, images=[0, 9], per_image=24, seed=6)
    print("cfg4 block", errs)
    assert feats.shape == (synth.num_tokens(grids) // 4, cfg.out_dim) and torch.isfinite(feats.float()).all()
    # the projector's two linear layers at their full widths, on a few rows
    rng_rows = 200
    x = synth.normal(7, "px", (rng_rows, 4 * cfg.hidden), 1.0, 0.0, cfg.dtype)
    ph = torch.empty((rng_rows, cfg.proj_hidden), dtype=torch.bfloat16, device="cuda")
    epd.op_linear(cfg.dtype, epd.to_device(x, cfg.dtype), enc._keep["proj_w1"], enc._keep["proj_b1"], ph, rng_rows,
                  cfg.proj_hidden, 4 * cfg.hidden, epd.LINEAR_GELU_ERF)
    ref = O.gelu(O.linear(x.astype(np.float64), w["proj_w1"].astype(np.float64), w["proj_b1"].astype(np.float64)),
                 O.ACT_GELU_ERF)
    assert_parity(to_np(ph), ref, 4e-3)
    enc.close()


def test_cfg5_prefetch_table_shapes_block_on_sampled_rows():
    """The image sizes of the paper's E-P prefetching table on a 0.7B-class encoder (head width 80: no padding
    column; a 292 x 222 patch grid: the rotary table does not fit shared memory and is read from global
    memory), one layer: feature row counts as printed in the paper, the block on sampled rows of the smallest,
    a middle and the 64824-token image."""
    cfg0, grids = synth.WORKLOADS["cfg5_vit07b_table42"]
    cfg = cfg0.with_layers(1)
    w = synth.make_weights(cfg, seed=8)
    enc, patches, feats, cu_rows, taps = _encode(cfg, grids, w, seed=8, taps=True)
    assert np.diff(cu_rows).tolist() == [100, 400, 1196, 2691, 16206]       # the paper's [n, 3584] row counts
    assert feats.shape == (20593, 3584) and torch.isfinite(feats.float()).all()
    errs = _check_blocks_on_rows(cfg, w, grids, taps, images=[0, 2, 4], per_image=12, seed=9)
    print("cfg5 block", errs)
    enc.close()


def test_cfg4_6b_widths_eight_layers_one_image_end_to_end():
    """The 6B-class widths on the benchmark's 16-image batch, eight of the 45 layers: image 5's features against
    the oracle's encode of image 5 alone (error growth over depth at these widths; the per-block figure is
    ~2.5e-3)."""
    cfg0, grids = synth.WORKLOADS["cfg4_vit6b_b16_448"]
    cfg = cfg0.with_layers(8)
    w = synth.make_weights(cfg, seed=11)
    enc, patches, feats, cu_rows, _ = _encode(cfg, grids, w, seed=11)
    bk = O.bookkeeping(grids)
    i = 5
    a, b = int(bk["cu_seqlens"][i]), int(bk["cu_seqlens"][i + 1])
    ref = O.encode(cfg, w, patches[a:b], [grids[i]])
    e = assert_parity(to_np(feats[cu_rows[i]:cu_rows[i + 1]]), ref, TOL_FINAL, "cfg4 8 layers image 5")
    print("cfg4 8 layers image 5 final", e)
    enc.close()


# ----------------------------------------------------------------------------- full batch, full depth

def _full_depth_one_item(workload, item, seed):
    """The whole batch of a benchmark configuration through every layer on the GPU; the features of one
    item against the oracle's encode of that item alone (exact: attention is block-diagonal and every
    other step is row-wise).  Returns (Frobenius ratio, worst-row ratio)."""
    cfg, grids = synth.WORKLOADS[workload]
    w = synth.make_weights(cfg, seed=seed)
    enc, patches, feats, cu_rows, _ = _encode(cfg, grids, w, seed=seed)
    bk = O.bookkeeping(grids)
    assert np.array_equal(cu_rows, bk["cu_out"])
    assert feats.shape == (synth.num_tokens(grids) // 4, cfg.out_dim) and torch.isfinite(feats.float()).all()
    a, b = int(bk["cu_seqlens"][item]), int(bk["cu_seqlens"][item + 1])
    got = to_np(feats[cu_rows[item]:cu_rows[item + 1]])
    enc.close()
    del enc, feats
    torch.cuda.empty_cache()
    ref = O.encode(cfg, w, patches[a:b], [grids[item]])
    e = assert_parity(got, ref, TOL_FINAL, f"{workload} item {item}")
    wr = worst_row_err(got, ref)
    print(workload, "layers", cfg.layers, "item", item, "tokens", b - a, "final", e, "worst row", wr)
    return e, wr


def test_cfg2_full_batch_full_depth_smallest_image():
    """32 variable-resolution images, all 27 layers: the smallest image of the batch."""
    _, grids = synth.WORKLOADS["cfg2_vit06b_var32"]
    lens = [t * h * w for t, h, w in grids]
    _full_depth_one_item("cfg2_vit06b_var32", int(np.argmin(lens)), seed=0)


def test_cfg3_full_batch_full_depth_clip():
    """The 16384-token image + the 8-frame clip, all 27 layers: the 6272-token clip (attention over all
    of its frames)."""
    _full_depth_one_item("cfg3_vit06b_long", 1, seed=0)


def test_cfg4_full_batch_full_depth_one_image():
    """The 6B-class encoder, 16 images, all 45 layers (11.6 GB of weights): image 11."""
    _full_depth_one_item("cfg4_vit6b_b16_448", 11, seed=0)


# ----------------------------------------------------------------------------- one batch split over replicas

def _device_weights(cfg, w):
    """The weight dictionary with every array already on the GPU in the encoder's element type (so that several
    encoders can borrow the same tensors)."""
    conv = lambda a: None if a is None else epd.to_device(a, cfg.dtype)
    out = {k: conv(v) for k, v in w.items() if k != "layers"}
    out["layers"] = [{k: conv(v) for k, v in lw.items()} for lw in w["layers"]]
    return out


def test_cfg2_batch_split_over_replicas_by_item_cost():
    """The 32 variable-resolution images dealt to 2, 3 and 8 replicas by the cost model (least-loaded first,
    costliest item first); every replica encodes its share with an encoder of its own (here: one after the
    other on the one GPU), and its rows go where the whole batch's layout puts them.  An item's features do
    not depend on what else is in the batch, so the reassembled buffer equals the whole-batch encode bit for
    bit; one item is also compared with the oracle."""
    from paper_2601_11590_b200 import replicas
    cfg, grids = synth.WORKLOADS["cfg2_vit06b_var32"]
    w = synth.make_weights(cfg, seed=0)
    wd = _device_weights(cfg, w)
    T, K = synth.num_tokens(grids), cfg.patch_dim
    patches = synth.make_patches(cfg, grids, seed=0)
    p_all = epd.to_device(patches, cfg.dtype)
    bk = O.bookkeeping(grids)
    cu = bk["cu_seqlens"]
    max_grid = max(max(g[1], g[2]) for g in grids)

    enc = epd.Encoder(cfg, wd, max_tokens=T, max_images=len(grids), max_grid=max_grid)
    whole, cu_rows = enc.encode(p_all, grids)
    torch.cuda.synchronize()
    assert enc.last_status() == epd.EPD_OK
    whole = whole.clone()
    enc.close()
    ranges = replicas.feature_row_ranges(grids)
    assert [r[0] for r in ranges] == cu_rows[:-1].tolist()

    for world in (2, 3, 8):
        shares = replicas.assign_items(grids, world, cfg.hidden, cfg.mlp)
        assert sorted(i for s in shares for i in s) == list(range(len(grids)))
        out = torch.full_like(whole, float("nan"))
        for items in shares:
            if not items:
                continue
            g = [grids[i] for i in items]
            p = torch.cat([p_all[int(cu[i]):int(cu[i + 1])] for i in items])
            e = epd.Encoder(cfg, wd, max_tokens=synth.num_tokens(g), max_images=len(g), max_grid=max_grid)
            f, cr = e.encode(p, g)
            torch.cuda.synchronize()
            assert e.last_status() == epd.EPD_OK
            for j, i in enumerate(items):
                out[ranges[i][0]:ranges[i][1]] = f[int(cr[j]):int(cr[j + 1])]
            e.close()
        assert torch.equal(out.view(torch.int16), whole.view(torch.int16)), world

    lens = np.diff(cu)
    i = int(np.argsort(lens)[1])                      # the second smallest image
    ref = O.encode(cfg, w, patches[int(cu[i]):int(cu[i + 1])], [grids[i]])
    e = assert_parity(to_np(whole[ranges[i][0]:ranges[i][1]]), ref, TOL_FINAL, f"cfg2 item {i}")
    print("cfg2 split: item", i, "tokens", int(lens[i]), "final", e)
