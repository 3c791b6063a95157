"""GPU parity: every step of the CUDA path and the whole stage against the CPU oracle,
through the C ABI, on the same seeded inputs.

Tolerances (relative Frobenius error ||G - O||_F / ||O||_F):
  float configurations     <= 1e-4 (whole stage and every step)
  bf16 configurations      <= 1e-2 per encoder block (block output for the GPU's own block input),
                           <= 3e-2 on the final features
  integer layout           bit-exact
"""
import ctypes

import numpy as np
import pytest
import torch

import synth
import paper_2601_11590_b200 as epd
from oracle import encoder_oracle as O
from tests.metrics import assert_parity, rel_err, worst_row_err

pytestmark = pytest.mark.gpu

TOL_F32 = 1e-4
TOL_BF16_BLOCK = 1e-2
TOL_BF16_FINAL = 3e-2
# a single bf16 step: inputs are exact, the only roundings are fp32 accumulation and one bf16 store (2^-9)
TOL_BF16_STEP = 4e-3


def to_np(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def dev(a, dtype):
    return epd.to_device(a, dtype)


def rnd(shape, seed, std, dtype):
    return synth.normal(seed, f"t{seed}", shape, std, 0.0, dtype)


@pytest.fixture(scope="module", autouse=True)
def _lib():
    from paper_2601_11590_b200 import build
    build.build_library()
    epd.load_library()


# ----------------------------------------------------------------------------- single steps

@pytest.mark.parametrize("dtype", [epd.DTYPE_F32, epd.DTYPE_BF16])
@pytest.mark.parametrize("M,N,K", [(1, 8, 8), (77, 40, 24), (200, 136, 72), (300, 1080, 288), (130, 288, 1080)])
@pytest.mark.parametrize("mode", ["plain", "gelu_tanh", "gelu_erf", "accum", "out_f32", "nobias"])
def test_linear(dtype, M, N, K, mode):
    x = rnd((M, K), 1, 1.0, dtype)
    w = rnd((N, K), 2, 1.0 / np.sqrt(K), dtype)
    b = None if mode == "nobias" else rnd((N,), 3, 0.5, dtype)
    flags = {"plain": 0, "nobias": 0, "gelu_tanh": epd.LINEAR_GELU_TANH, "gelu_erf": epd.LINEAR_GELU_ERF,
             "accum": epd.LINEAR_ACCUMULATE, "out_f32": epd.LINEAR_OUT_F32}[mode]
    ref = O.linear(x.astype(np.float64), w.astype(np.float64), None if b is None else b.astype(np.float64))
    if mode == "gelu_tanh":
        ref = O.gelu(ref, O.ACT_GELU_TANH)
    if mode == "gelu_erf":
        ref = O.gelu(ref, O.ACT_GELU_ERF)
    out_f32 = dtype == epd.DTYPE_F32 or mode in ("accum", "out_f32")
    r0 = rnd((M, N), 4, 1.0, epd.DTYPE_F32)
    out = torch.from_numpy(r0.copy()).cuda() if out_f32 else torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    if mode == "accum":
        ref = ref + r0.astype(np.float64)
    epd.op_linear(dtype, dev(x, dtype), dev(w, dtype), dev(b, dtype), out, M, N, K, flags)
    torch.cuda.synchronize()
    tol = TOL_F32 if dtype == epd.DTYPE_F32 else (1e-5 if out_f32 else TOL_BF16_STEP)
    assert_parity(to_np(out), ref, tol)


@pytest.mark.parametrize("tile_n", [0, 128, 192, 256])
@pytest.mark.parametrize("M,N,K,ldpad", [
    (1000, 1152, 1152, 0),     # several M tiles, K = 18 blocks
    (300, 4304, 1152, 0),      # ragged N (4304 = 33*128 + 80)
    (257, 1152, 4304, 0),      # ragged K (4304 = 67*64 + 16)
    (2000, 2304, 320, 0),      # more tiles than SMs: every CTA walks several tiles, both accumulators
    (130, 3200, 588, 4),       # K = 588 with leading dimensions padded to 592
    (64, 8, 8, 0),             # smaller than one tile in every direction
])
@pytest.mark.parametrize("mode", ["plain", "gelu_tanh", "accum"])
def test_linear_tensor_core_tiles(tile_n, M, N, K, ldpad, mode):
    """bf16 linear layer on the tcgen05 kernel, every tile width, against the oracle and the FMA kernel."""
    dtype = epd.DTYPE_BF16
    ld = K + ldpad
    x = np.zeros((M, ld), np.float32); x[:, :K] = rnd((M, K), 11, 1.0, dtype)
    w = np.zeros((N, ld), np.float32); w[:, :K] = rnd((N, K), 12, 1.0 / np.sqrt(K), dtype)
    if ldpad:   # the padding must be ignored, not multiplied in
        x[:, K:] = 7.0
        w[:, K:] = 7.0
    b = rnd((N,), 13, 0.5, dtype)
    flags = {"plain": 0, "gelu_tanh": epd.LINEAR_GELU_TANH, "accum": epd.LINEAR_ACCUMULATE}[mode]
    ref = O.linear(x[:, :K].astype(np.float64), w[:, :K].astype(np.float64), b.astype(np.float64))
    if mode == "gelu_tanh":
        ref = O.gelu(ref, O.ACT_GELU_TANH)
    r0 = rnd((M, N), 14, 1.0, epd.DTYPE_F32)
    if mode == "accum":
        ref = ref + r0.astype(np.float64)
        make_out = lambda: torch.from_numpy(r0.copy()).cuda()
    else:
        make_out = lambda: torch.full((M, N), 99.0, dtype=torch.bfloat16, device="cuda")
    xd, wd, bd = dev(x, dtype), dev(w, dtype), dev(b, dtype)
    out = epd.op_linear(dtype, xd, wd, bd, make_out(), M, N, K, flags | (tile_n << 8))
    torch.cuda.synchronize()
    tol = 1e-5 if mode == "accum" else TOL_BF16_STEP
    assert_parity(to_np(out), ref, tol)
    out_fma = epd.op_linear(dtype, xd, wd, bd, make_out(), M, N, K, flags | epd.LINEAR_FORCE_FMA)
    assert_parity(to_np(out), to_np(out_fma), tol)


@pytest.mark.parametrize("M,N,K", [(300, 1080, 1152), (130, 288, 4304), (700, 520, 80)])
def test_linear_e4m3_variant(M, N, K):
    """The 8-bit floating-point variant of the linear layer: the row quantiser's codes and scales bit for bit
    against the oracle (both take the rounding decisions from float32 quotients), then the layer on those codes
    (products exact, float accumulation: 2e-5 with float output, one bf16 rounding otherwise).  The distance to
    the unquantised layer is printed, not bounded: it is the format's error, not the kernel's."""
    dtype = epd.DTYPE_BF16
    x = rnd((M, K), 61, 1.0, dtype) * synth.round_to_bf16(np.exp2(np.arange(M) % 7 - 3).astype(np.float32))[:, None]
    x[M // 2, :] = 0.0                                           # an all-zero row: scale 1, zero codes
    w = rnd((N, K), 62, K ** -0.5, dtype)
    b = rnd((N,), 63, 0.5, dtype)
    xd, wd = dev(x, dtype), dev(w, dtype)
    xq, xs = epd.op_quantize_e4m3(xd)
    wq, ws = epd.op_quantize_e4m3(wd)
    for arr, q, sc in ((x, xq, xs), (w, wq, ws)):
        q_ref, s_ref = O.quantize_e4m3_rows(arr)
        assert np.array_equal(sc.cpu().numpy(), s_ref.astype(np.float32))
        assert np.array_equal(q.cpu().numpy()[:, :K], O.e4m3_bits(q_ref))
        assert not q.cpu().numpy()[:, K:].any()
    ref = O.linear_e4m3(x, w, b.astype(np.float64))
    out32 = torch.zeros((M, N), dtype=torch.float32, device="cuda")
    epd.op_linear_e4m3(xq, xs, wq, ws, dev(b, dtype), out32, K, epd.LINEAR_OUT_F32)
    assert_parity(to_np(out32), ref, 2e-5)
    out16 = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    epd.op_linear_e4m3(xq, xs, wq, ws, dev(b, dtype), out16, K, epd.LINEAR_GELU_TANH)
    assert_parity(to_np(out16), O.gelu(ref, O.ACT_GELU_TANH), TOL_BF16_STEP)
    exact = O.linear(x.astype(np.float64), w.astype(np.float64), b.astype(np.float64))
    print("e4m3 linear", (M, N, K), "distance to the unquantised layer", rel_err(ref, exact))


@pytest.mark.parametrize("dtype", [epd.DTYPE_F32, epd.DTYPE_BF16])
@pytest.mark.parametrize("T,h", [(1, 8), (37, 256), (100, 1152), (9, 3200), (5, 30)])
def test_rmsnorm(dtype, T, h):
    x = rnd((T, h), 5, 3.0, epd.DTYPE_F32)
    g = synth.normal(6, "g", (h,), 0.02, 1.0, dtype)
    ref = O.rmsnorm(x.astype(np.float64), g.astype(np.float64), 1e-6)
    out = torch.zeros((T, h), dtype=epd.torch_dtype(dtype), device="cuda")
    epd.op_rmsnorm(dtype, torch.from_numpy(x).cuda(), dev(g, dtype), out, 1e-6)
    assert_parity(to_np(out), ref, (1e-6 if dtype == epd.DTYPE_F32 else TOL_BF16_STEP))
    # scattered destination rows (the fused 2x2 merge)
    perm = np.random.default_rng(0).permutation(T).astype(np.int32)
    out2 = torch.zeros_like(out)
    epd.op_rmsnorm(dtype, torch.from_numpy(x).cuda(), dev(g, dtype), out2, 1e-6,
                   dst_row=torch.from_numpy(perm).cuda())
    assert torch.equal(out2[torch.from_numpy(perm.astype(np.int64)).cuda()], out)


@pytest.mark.parametrize("dtype", [epd.DTYPE_F32, epd.DTYPE_BF16])
@pytest.mark.parametrize("heads,dh", [(4, 64), (3, 72), (2, 128), (2, 8)])
def test_rope_split(dtype, heads, dh):
    T, h = 53, heads * dh
    qkv = rnd((T, 3 * h), 7, 1.0, dtype)
    rng = np.random.default_rng(1)
    pr, pc = rng.integers(0, 128, T).astype(np.int32), rng.integers(0, 128, T).astype(np.int32)
    scale = 0.37
    q, k, v = epd.op_rope_split(dtype, dev(qkv, dtype), torch.from_numpy(pr).cuda(), torch.from_numpy(pc).cuda(),
                                heads, dh, 10000.0, scale)
    x = qkv.astype(np.float64)
    qr = O.rope_2d(x[:, :h].reshape(T, heads, dh), pr, pc, 10000.0) * scale
    kr = O.rope_2d(x[:, h:2 * h].reshape(T, heads, dh), pr, pc, 10000.0)
    vr = x[:, 2 * h:].reshape(T, heads, dh)
    dhp = epd.padded_head_dim(dh)
    assert q.shape == (heads, T, dhp)
    tol = 1e-6 if dtype == epd.DTYPE_F32 else TOL_BF16_STEP
    for got, ref in ((q, qr), (k, kr), (v, vr)):
        g = to_np(got)
        assert_parity(g[:, :, :dh].transpose(1, 0, 2), ref, tol)
        if got is v and dhp > dh:   # v's first padding column is 1 (it makes P V deliver the row sums)
            assert np.all(g[:, :, dh] == 1.0) and np.all(g[:, :, dh + 1:] == 0.0)
        else:
            assert np.all(g[:, :, dh:] == 0.0)
    assert np.array_equal(to_np(v)[:, :, :dh].transpose(1, 0, 2), vr)  # v is a pure copy


def _prepared_order(heads, dh):
    """Order of the head dimensions of q and k after the fused projection, written out from its definition:
    inside a head, the rotation pairs (f, f + dh/4) of the row half come first, then those of the column
    half, the two members of a pair side by side."""
    nf = dh // 4
    inside = []
    for half in (0, 1):
        for f in range(nf):
            first = half * (dh // 2) + f
            inside += [first, first + nf]
    assert sorted(inside) == list(range(dh))
    return np.concatenate([a * dh + np.asarray(inside) for a in range(heads)])


@pytest.mark.parametrize("heads,dh,T", [(16, 72, 784), (3, 72, 300), (4, 64, 129), (25, 128, 260), (2, 8, 40), (16, 72, 1)])
def test_qkv_rope_fused(heads, dh, T):
    """Projection + rotary + head split in one kernel against the oracle's linear, rope_2d and split.
    Tile-ragged T, heads whose 72 columns straddle the 128-column halves and 256-column tiles, the
    q / k / v boundaries inside a tile (3 heads), padded and unpadded head widths."""
    dtype = epd.DTYPE_BF16
    h = heads * dh
    x = rnd((T, h), 31, 1.0, dtype)
    w = rnd((3 * h, h), 32, h ** -0.5, dtype)
    b = rnd((3 * h,), 33, 0.5, dtype)
    rng = np.random.default_rng(2)
    rows = 97
    pr, pc = rng.integers(0, rows, T).astype(np.int32), rng.integers(0, rows, T).astype(np.int32)
    scale = 0.21
    q, k, v = epd.op_qkv_rope(dev(x, dtype), dev(w, dtype), dev(b, dtype), torch.from_numpy(pr).cuda(),
                              torch.from_numpy(pc).cuda(), heads, dh, 10000.0, scale, rows)
    y = O.linear(x.astype(np.float64), w.astype(np.float64), b.astype(np.float64))
    qr = O.rope_2d(y[:, :h].reshape(T, heads, dh), pr, pc, 10000.0) * scale
    kr = O.rope_2d(y[:, h:2 * h].reshape(T, heads, dh), pr, pc, 10000.0)
    vr = y[:, 2 * h:].reshape(T, heads, dh)
    order = _prepared_order(heads, dh)              # q and k come back in the prepared order of head dims
    qr = qr.reshape(T, h)[:, order].reshape(T, heads, dh)
    kr = kr.reshape(T, h)[:, order].reshape(T, heads, dh)
    dhp = epd.padded_head_dim(dh)
    for got, ref in ((q, qr), (k, kr), (v, vr)):
        g = to_np(got)
        assert g.shape == (heads, T, dhp)
        assert_parity(g[:, :, :dh].transpose(1, 0, 2), ref, TOL_BF16_STEP)
        if got is v and dhp > dh:
            assert np.all(g[:, :, dh] == 1.0) and np.all(g[:, :, dh + 1:] == 0.0)
        else:
            assert np.all(g[:, :, dh:] == 0.0)
    # the scores do not depend on the order of the head dimensions
    s_fused = np.einsum("htd,hud->htu", to_np(q)[:, :, :dh], to_np(k)[:, :, :dh])
    s_ref = np.einsum("thd,uhd->htu", qr, kr)
    assert_parity(s_fused, s_ref, TOL_BF16_STEP)


def _attention_case(dtype, heads, dh, seglens, seed, logit_scale=1.0, flags=0):
    T = int(sum(seglens))
    cu = np.concatenate([[0], np.cumsum(seglens)]).astype(np.int32)
    dhp = epd.padded_head_dim(dh)
    qs = 1.4426950408889634 / np.sqrt(dh)
    q = rnd((heads, T, dh), seed, logit_scale, dtype)
    k = rnd((heads, T, dh), seed + 1, logit_scale, dtype)
    v = rnd((heads, T, dh), seed + 2, 1.0, dtype)
    # the kernel receives q already multiplied by log2(e)/sqrt(dh); round that product the way the
    # rotary step stores it so both sides start from the same numbers
    q_scaled = (q.astype(np.float64) * qs).astype(np.float32)
    if dtype == epd.DTYPE_BF16:
        q_scaled = synth.round_to_bf16(q_scaled)

    def pad(a, ones_column=False):
        out = np.zeros((heads, T, dhp), np.float32)
        out[:, :, :dh] = a
        if ones_column and dhp > dh:
            out[:, :, dh] = 1.0
        return dev(out, dtype)

    out = epd.op_attention(dtype, pad(q_scaled), pad(k), pad(v, True), torch.from_numpy(cu).cuda(), cu, dh, flags)
    q_eff = q_scaled.astype(np.float64) / qs
    ref = O.attention_block_diagonal(q_eff.transpose(1, 0, 2), k.astype(np.float64).transpose(1, 0, 2),
                                     v.astype(np.float64).transpose(1, 0, 2), cu).reshape(T, heads * dh)
    return to_np(out), ref


@pytest.mark.parametrize("dtype", [epd.DTYPE_F32, epd.DTYPE_BF16])
@pytest.mark.parametrize("heads,dh,seglens", [
    (2, 64, [256, 256]), (3, 72, [4, 196, 300, 33]), (2, 128, [129, 64, 1]), (2, 72, [784]), (1, 8, [5])])
def test_attention(dtype, heads, dh, seglens):
    got, ref = _attention_case(dtype, heads, dh, seglens, 10)
    assert_parity(got, ref, (1e-5 if dtype == epd.DTYPE_F32 else TOL_BF16_STEP))


@pytest.mark.parametrize("heads,dh,seglens", [
    (2, 72, [784, 784]),                 # the benchmark's segment length: 6 full key tiles + a 16-key tail
    (2, 72, [100, 1300, 128, 129, 4]),   # ragged tails on both the query and the key side
    (3, 64, [2000]),                     # 16 key tiles
    (2, 128, [700, 260]),
    (2, 72, [256, 257, 255, 512, 384]),  # query blocks of 256 rows: exactly full, one row over, one row short
    (1, 80, [1000, 130]),                # head width 80: no padding column, row sums in registers
    (3, 128, [1024, 1024]),              # the 6B-class encoder's images
    (2, 56, [300]),                      # padded width 64 with a ones column
    (148, 72, [300]),                    # more items than SMs: several items per CTA, second tile partly empty
])
def test_attention_tensor_core_long_segments(heads, dh, seglens):
    got, ref = _attention_case(epd.DTYPE_BF16, heads, dh, seglens, 40)
    assert_parity(got, ref, TOL_BF16_STEP)
    fma, _ = _attention_case(epd.DTYPE_BF16, heads, dh, seglens, 40, flags=epd.ATTENTION_FORCE_FMA)
    assert_parity(got, fma, TOL_BF16_STEP)
    for forced in (epd.ATTENTION_SPLIT_KEYS, epd.ATTENTION_TWO_QUERY_TILES):      # both tensor-core kernels
        other, _ = _attention_case(epd.DTYPE_BF16, heads, dh, seglens, 40, flags=forced)
        assert_parity(other, ref, TOL_BF16_STEP)


def test_attention_more_segments_than_one_launch_describes():
    """More segments than one launch of the tensor-core kernel can list (128): the segments are sorted by length and
    dealt to several launches, each of which must write exactly its own segments' rows."""
    rng = np.random.default_rng(5)
    seglens = rng.integers(2, 41, size=131).tolist()
    seglens[7], seglens[100] = 300, 129
    got, ref = _attention_case(epd.DTYPE_BF16, 2, 72, seglens, 50)
    assert_parity(got, ref, TOL_BF16_STEP)
    two, _ = _attention_case(epd.DTYPE_BF16, 2, 72, seglens, 50, flags=epd.ATTENTION_TWO_QUERY_TILES)
    assert_parity(two, ref, TOL_BF16_STEP)
    fma, _ = _attention_case(epd.DTYPE_BF16, 2, 72, seglens, 50, flags=epd.ATTENTION_FORCE_FMA)
    assert_parity(got, fma, TOL_BF16_STEP)


@pytest.mark.parametrize("dh", [64, 72, 80, 128])
def test_attention_segment_lengths_around_the_tile_edges(dh):
    """Segment lengths on both sides of every boundary the two-query-tile kernel has (the 16-key product group, the
    64-key step, the 128-row query tile, the 256-row item with its empty or ragged second tile), packed into one
    batch, against the oracle; both tensor-core kernels."""
    seglens = [1, 2, 15, 16, 17, 63, 64, 65, 127, 128, 129, 191, 193, 255, 256, 257, 300, 383, 385, 511, 513]
    for flags in (epd.ATTENTION_TWO_QUERY_TILES, epd.ATTENTION_SPLIT_KEYS):
        got, ref = _attention_case(epd.DTYPE_BF16, 2, dh, seglens, 70 + dh, flags=flags)
        assert np.isfinite(got).all()
        assert_parity(got, ref, TOL_BF16_STEP, f"attention, head width {dh}, flags {flags}")


@pytest.mark.parametrize("kernel", ["split_keys", "two_query_tiles"])
def test_attention_rescale_path(kernel):
    """Keys ordered so that the running maximum keeps growing from tile to tile by far more than the
    rescale threshold: every key tile forces a rescale of the accumulated output."""
    dtype, heads, dh, T = epd.DTYPE_BF16, 1, 64, 1024
    dhp = epd.padded_head_dim(dh)
    rng = np.random.default_rng(0)
    q = np.zeros((heads, T, dhp), np.float32); q[:, :, 0] = 1.0
    k = np.zeros((heads, T, dhp), np.float32)
    k[0, :, 0] = synth.round_to_bf16((np.arange(T) * 0.25).astype(np.float32))       # logits 0 .. 256 (base 2)
    k[0, :, 1:dh] = synth.round_to_bf16(rng.standard_normal((T, dh - 1)).astype(np.float32))
    v = np.zeros((heads, T, dhp), np.float32)
    v[:, :, :dh] = synth.round_to_bf16(rng.standard_normal((heads, T, dh)).astype(np.float32))
    cu = np.array([0, T], np.int32)
    flags = epd.ATTENTION_SPLIT_KEYS if kernel == "split_keys" else epd.ATTENTION_TWO_QUERY_TILES
    out = epd.op_attention(dtype, dev(q, dtype), dev(k, dtype), dev(v, dtype), torch.from_numpy(cu).cuda(), cu, dh, flags)
    # the kernel's q carries log2(e)/sqrt(dh); hand the oracle the unscaled q it implies
    q_eff = q[:, :, :dh].astype(np.float64) * np.log(2.0) * np.sqrt(dh)
    ref = O.attention_block_diagonal(q_eff.transpose(1, 0, 2), k[:, :, :dh].astype(np.float64).transpose(1, 0, 2),
                                     v[:, :, :dh].astype(np.float64).transpose(1, 0, 2), cu).reshape(T, heads * dh)
    assert_parity(to_np(out), ref, 1e-2)


@pytest.mark.parametrize("dtype", [epd.DTYPE_F32, epd.DTYPE_BF16])
def test_attention_peaked_logits(dtype):
    """Logit standard deviation ~ 50: exercises the running-max rescaling of the online softmax."""
    got, ref = _attention_case(dtype, 2, 72, [300, 520], 20, logit_scale=2.5)
    assert_parity(got, ref, (1e-4 if dtype == epd.DTYPE_F32 else 1e-2))
    if dtype == epd.DTYPE_BF16:
        for forced in (epd.ATTENTION_SPLIT_KEYS, epd.ATTENTION_TWO_QUERY_TILES):
            got, ref = _attention_case(dtype, 2, 72, [300, 520], 20, logit_scale=2.5, flags=forced)
            assert_parity(got, ref, 1e-2)


@pytest.mark.parametrize("dtype", [epd.DTYPE_F32, epd.DTYPE_BF16])
def test_merge(dtype):
    grids = [(1, 4, 6), (2, 2, 2), (1, 2, 8)]
    bk = O.bookkeeping(grids)
    T, h = int(bk["cu_seqlens"][-1]), 40
    y = rnd((T, h), 30, 1.0, dtype)
    out = epd.op_merge(dtype, dev(y, dtype), torch.from_numpy(bk["merge_idx"].reshape(-1).copy()).cuda())
    assert np.array_equal(to_np(out), O.merge_2x2(y.astype(np.float64), bk["merge_idx"]))


@pytest.mark.parametrize("dtype", [epd.DTYPE_F32, epd.DTYPE_BF16])
@pytest.mark.parametrize("P,Tp,grids,ldpad", [(16, 1, [(1, 4, 6), (1, 2, 2)], 0), (14, 1, [(1, 2, 4)], 4), (8, 1, [(1, 2, 6)], 3),
                                              (16, 2, [(3, 2, 4), (1, 6, 2)], 0), (2, 2, [(2, 2, 2)], 8)])
@pytest.mark.parametrize("pixels", ["u8", "bf16"])
def test_patchify(dtype, P, Tp, grids, ldpad, pixels):
    """Raw frames (uint8, or bf16 values with fractions on the same 0..255 scale) -> patch vectors against the
    oracle (one rounding to the element type)."""
    cfg = synth.tiny_variant(patch=P, temporal_patch=Tp)
    frames = synth.make_frames(cfg, grids, seed=21)
    if pixels == "bf16":
        rng = np.random.default_rng(3)
        frames = [synth.round_to_bf16((f.astype(np.float32) + rng.random(f.shape, dtype=np.float32)) * 0.97)
                  for f in frames]
    mean, std = (0.48, 0.46, 0.41), (0.27, 0.26, 0.28)
    ref = O.patchify(frames, grids, P, Tp, mean, std)
    bk = O.bookkeeping(grids)
    fd, off = epd.pack_frames(frames, bf16=pixels == "bf16")
    K = cfg.patch_dim
    got = epd.op_patchify(dtype, fd, off, grids, bk["cu_seqlens"], cfg.in_channels, P, Tp, mean, std, ld=K + ldpad)
    g = to_np(got)
    assert_parity(g[:, :K], ref, (1e-6 if dtype == epd.DTYPE_F32 else TOL_BF16_STEP))
    assert np.all(g[:, K:] == 0.0)


def test_stage_from_raw_frames():
    """epd_encode_frames: pixels in, features out, against the oracle's patchify + encode."""
    cfg = _small_bf16(tp=2)
    grids = [(2, 6, 8), (1, 10, 4)]
    w = synth.make_weights(cfg, seed=12)
    frames = synth.make_frames(cfg, grids, seed=12)
    T = synth.num_tokens(grids)
    enc = epd.Encoder(cfg, w, max_tokens=T, max_images=2, max_grid=16)
    fd, _ = epd.pack_frames(frames)
    feats, cu_rows = enc.encode_frames(fd, grids, synth.PIXEL_MEAN, synth.PIXEL_STD)
    torch.cuda.synchronize()
    assert enc.last_status() == epd.EPD_OK
    patches = O.patchify(frames, grids, cfg.patch, cfg.temporal_patch, synth.PIXEL_MEAN, synth.PIXEL_STD)
    ref = O.encode(cfg, w, patches, grids)
    assert np.array_equal(cu_rows, O.bookkeeping(grids)["cu_out"])
    assert_parity(to_np(feats), ref, TOL_BF16_FINAL)
    # a second call with the same grids (layout already staged) gives the same bits
    again, _ = enc.encode_frames(fd, grids, synth.PIXEL_MEAN, synth.PIXEL_STD)
    torch.cuda.synchronize()
    assert torch.equal(feats, again)
    # the same pixels handed over as bfloat16 (0..255 is exact in it): the same features, bit for bit
    fb, _ = epd.pack_frames([f.astype(np.float32) for f in frames], bf16=True)
    from_bf16, _ = enc.encode_frames(fb, grids, synth.PIXEL_MEAN, synth.PIXEL_STD)
    torch.cuda.synchronize()
    assert torch.equal(feats, from_bf16)
    enc.close()


# ----------------------------------------------------------------------------- integer layout

def _golden_grids():
    import os
    rows = []
    with open(os.path.join(os.path.dirname(__file__), "golden", "e2p_feature_rows.txt")) as fh:
        for line in fh:
            if line.strip() and not line.startswith("#"):
                rows.append(tuple(int(v) for v in line.split()))
    return rows


def test_bookkeeping_bit_exact_including_paper_shapes():
    cfg = synth.tiny_variant(head_dim=8, heads=2, layers=0, mlp=16, patch=1, out_dim=8)
    w = synth.make_weights(cfg, seed=1)
    golden = _golden_grids()
    cases = [
        [(1, 2, 2)],
        [(1, 4, 6), (3, 2, 4), (1, 2, 2)],
        [(2, 6, 2), (1, 16, 16), (1, 2, 30)],
        [(1, r[2], r[3]) for r in golden],
    ]
    maxT = max(synth.num_tokens(g) for g in cases)
    enc = epd.Encoder(cfg, w, max_tokens=maxT, max_images=8, max_grid=512)
    for grids in cases:
        T = synth.num_tokens(grids)
        patches = dev(synth.make_patches(cfg, grids, seed=2), cfg.dtype)
        feats, cu_rows = enc.encode(patches, grids)
        bk = O.bookkeeping(grids)
        got = enc.debug_bookkeeping(len(grids), T)
        for key in ("cu_seqlens", "pos_row", "pos_col", "merge_idx"):
            assert np.array_equal(got[key], bk[key]), key
        assert np.array_equal(cu_rows, bk["cu_out"])
        assert feats.shape == (T // 4, cfg.out_dim)
    assert np.diff(cu_rows).tolist() == [r[4] for r in golden]
    assert enc.last_status() == epd.EPD_OK
    enc.close()


# ----------------------------------------------------------------------------- whole stage

def _run_stage(cfg, grids, seed=0, qkv_scale=1.0, with_taps=True, max_grid=128):
    w = synth.make_weights(cfg, seed=seed, qkv_scale=qkv_scale)
    patches = synth.make_patches(cfg, grids, seed=seed)
    T = synth.num_tokens(grids)
    enc = epd.Encoder(cfg, w, max_tokens=T, max_images=max(1, len(grids)), max_grid=max_grid)
    taps = None
    if with_taps:
        taps = [torch.zeros((T, cfg.hidden), dtype=torch.float32, device="cuda") for _ in range(cfg.layers + 1)]
        enc.set_taps(taps)
    K = cfg.patch_dim
    ld = K if cfg.dtype == epd.DTYPE_F32 else (K + 7) // 8 * 8
    p = torch.zeros((T, ld), dtype=epd.torch_dtype(cfg.dtype), device="cuda")
    p[:, :K] = dev(patches, cfg.dtype)
    feats, cu_rows = enc.encode(p, grids)
    torch.cuda.synchronize()
    assert enc.last_status() == epd.EPD_OK
    assert enc.last_launch_count() >= 2
    return enc, w, patches, feats, cu_rows, taps


def _check_stage(cfg, grids, tol_final, tol_block, **kw):
    enc, w, patches, feats, cu_rows, taps = _run_stage(cfg, grids, **kw)
    ref, ref_taps = O.encode(cfg, w, patches, grids, return_taps=True)
    bk = O.bookkeeping(grids)
    assert np.array_equal(cu_rows, bk["cu_out"])
    # per-block error: oracle block applied to the GPU's own block input
    errs = []
    for l in range(cfg.layers):
        x_in = to_np(taps[l])
        want = O.block(cfg, w["layers"][l], x_in, bk)
        got = to_np(taps[l + 1])
        errs.append((assert_parity(got, want, tol_block, f"block {l}"), rel_err(got - x_in, want - x_in)))
    assert_parity(to_np(taps[0]), ref_taps[0], 1e-5, "patch embedding")
    e_final = assert_parity(to_np(feats), ref, tol_final, "final features")
    enc.close()
    return e_final, errs


def test_stage_tiny_fp32_config():
    cfg, grids = synth.WORKLOADS["cfg0_tiny_fp32"]
    e, errs = _check_stage(cfg, grids, TOL_F32, TOL_F32)
    print("cfg0 final", e, "blocks", errs)


def test_stage_fp32_ragged_grids_and_clip():
    cfg = synth.TINY_FP32
    _check_stage(cfg, [(1, 2, 2), (2, 6, 10), (1, 18, 14), (1, 4, 2)], TOL_F32, TOL_F32, seed=3)


def _small_bf16(layers=2, heads=4, dh=72, mlp=1080, act=synth.ACT_GELU_TANH, tp=1, patch=16):
    import dataclasses
    return dataclasses.replace(synth.VIT_06B, name="small-bf16", hidden=heads * dh, heads=heads, head_dim=dh,
                               layers=layers, mlp=mlp, act=act, temporal_patch=tp, patch=patch,
                               proj_hidden=4 * heads * dh, out_dim=512)


@pytest.mark.parametrize("variant", ["dh72", "dh128_erf", "dh64_video"])
def test_stage_small_bf16(variant):
    if variant == "dh72":
        cfg, grids = _small_bf16(), [(1, 28, 28), (1, 14, 20), (1, 2, 2), (1, 30, 8)]
    elif variant == "dh128_erf":
        import dataclasses
        cfg = dataclasses.replace(_small_bf16(heads=3, dh=128, mlp=1536, act=synth.ACT_GELU_ERF), patch=14)
        grids = [(1, 16, 16), (1, 32, 32)]
    else:
        cfg, grids = _small_bf16(heads=4, dh=64, mlp=1000, tp=2), [(4, 10, 12), (1, 22, 6)]
    e, errs = _check_stage(cfg, grids, TOL_BF16_FINAL, TOL_BF16_BLOCK, seed=5)
    print(variant, "final", e, "blocks", errs)


def test_stage_small_bf16_peaked_attention():
    """W_qkv scaled x8 (not a benchmark configuration): sharply peaked softmax rows."""
    cfg, grids = _small_bf16(), [(1, 20, 24), (1, 12, 12)]
    _check_stage(cfg, grids, TOL_BF16_FINAL, TOL_BF16_BLOCK, seed=6, qkv_scale=8.0)


def test_block_diagonal_isolation_on_gpu():
    """An item's features do not depend on the rest of the batch (bit-identical on the GPU when the
    launch geometry is the same; within tolerance against the item encoded alone)."""
    cfg = _small_bf16()
    grids = [(1, 12, 12), (1, 8, 16), (1, 20, 6)]
    w = synth.make_weights(cfg, seed=7)
    patches = synth.make_patches(cfg, grids, seed=7)
    T = synth.num_tokens(grids)
    enc = epd.Encoder(cfg, w, max_tokens=T, max_images=4)
    p = dev(patches, cfg.dtype)
    f0, cu_rows = enc.encode(p, grids)
    f0 = f0.clone()
    bk = O.bookkeeping(grids)
    cu = bk["cu_seqlens"]
    p2 = p.clone()
    p2[cu[0]:cu[1]] *= -1.5
    p2[cu[2]:cu[3]] += 1.0
    f1, _ = enc.encode(p2, grids)
    torch.cuda.synchronize()
    assert torch.equal(f0[cu_rows[1]:cu_rows[2]], f1[cu_rows[1]:cu_rows[2]])
    assert not torch.equal(f0[cu_rows[0]:cu_rows[1]], f1[cu_rows[0]:cu_rows[1]])
    alone, _ = enc.encode(p[cu[1]:cu[2]].contiguous(), [grids[1]])
    assert_parity(to_np(alone), to_np(f0[cu_rows[1]:cu_rows[2]]), TOL_BF16_FINAL)
    enc.close()


def test_one_encoder_alternating_small_and_large_batches():
    """The same encoder serves batches of at most 128 tokens (separate rotary kernel, single-CTA linear kernel)
    and larger ones (rotary embedding in the QKV epilogue, which relies on padding columns written once at
    create) in turn: every call matches the oracle, and a repeated batch gives the same bits as before."""
    cfg = _small_bf16()
    w = synth.make_weights(cfg, seed=31)
    batches = [[(1, 8, 8)], [(1, 20, 24), (1, 6, 6)], [(1, 4, 4), (1, 6, 8)], [(1, 30, 14)], [(1, 8, 8)],
               [(1, 20, 24), (1, 6, 6)]]
    enc = epd.Encoder(cfg, w, max_tokens=600, max_images=4, max_grid=32)
    seen = {}
    for i, grids in enumerate(batches):
        patches = synth.make_patches(cfg, grids, seed=40 + len(grids) + grids[0][1])
        feats, cu_rows = enc.encode(dev(patches, cfg.dtype), grids)
        torch.cuda.synchronize()
        assert enc.last_status() == epd.EPD_OK
        ref = O.encode(cfg, w, patches, grids)
        assert_parity(to_np(feats), ref, TOL_BF16_FINAL)
        key = tuple(grids)
        if key in seen:
            assert torch.equal(seen[key], feats), (i, grids)
        seen[key] = feats.clone()
    enc.close()


def test_sm_limit_ready_flag_and_stand_in():
    """Co-location helpers: an SM budget leaves the features bit-identical; the ready flag is written after
    the encode on its stream; the memory-bound stand-in's checksums match a host restatement."""
    cfg = _small_bf16()
    grids = [(1, 20, 24), (1, 12, 12)]
    enc, w, patches, feats, _, _ = _run_stage(cfg, grids, seed=9, with_taps=False)
    first = feats.clone()
    p = dev(patches, cfg.dtype)
    flag = torch.zeros(1, dtype=torch.int32, device="cuda")
    try:
        for limit in (40, 7, 0):
            epd.set_sm_limit(limit)
            assert epd.get_sm_limit() == limit
            again, _ = enc.encode(p, grids)
            epd.signal_ready(flag, 100 + limit)
            torch.cuda.synchronize()
            assert int(flag.item()) == 100 + limit
            assert torch.equal(first, again), limit
    finally:
        epd.set_sm_limit(0)
    enc.close()
    rng = np.random.default_rng(3)
    words = rng.integers(0, 2 ** 32, size=(4096 + 3) * 4, dtype=np.uint64)          # a ragged split over 5 CTAs
    data = torch.from_numpy(words.astype(np.uint32).view(np.int32)).cuda()
    sums = torch.zeros(5, dtype=torch.int64, device="cuda")
    passes = 3
    epd.op_stream_read(data, passes, 5, sums)
    torch.cuda.synchronize()
    v = words.reshape(-1, 4)
    per_vec = ((v[:, 0] ^ v[:, 1]) + (v[:, 2] ^ v[:, 3])).astype(np.uint64)
    want = (int(per_vec.sum()) * passes + sum(range(passes)) * len(per_vec)) % (1 << 64)
    got = int(sums.cpu().numpy().view(np.uint64).sum(dtype=np.uint64))
    assert got == want


def test_run_to_run_determinism():
    cfg = _small_bf16()
    grids = [(1, 16, 16), (1, 10, 30)]
    enc, w, patches, feats, _, _ = _run_stage(cfg, grids, seed=8, with_taps=False)
    first = feats.clone()
    p = dev(patches, cfg.dtype)
    for _ in range(3):
        again, _ = enc.encode(p, grids)
        torch.cuda.synchronize()
        assert torch.equal(first, again)
    enc.close()


def test_host_buffer_entry_point_matches_device_entry_point():
    cfg = _small_bf16()
    grids = [(1, 16, 16), (1, 6, 10)]
    enc, w, patches, feats, cu_rows, _ = _run_stage(cfg, grids, seed=9, with_taps=False)
    hp = dev(patches, cfg.dtype).cpu().pin_memory()
    hf = torch.zeros((feats.shape[0], cfg.out_dim), dtype=feats.dtype).pin_memory()
    rows, cu2 = enc.encode_host(hp, grids, hf)
    torch.cuda.synchronize()
    assert rows == feats.shape[0] and np.array_equal(cu2, cu_rows)
    assert torch.equal(hf, feats.cpu())
    enc.close()


def test_host_buffer_entry_point_with_patch_length_not_a_multiple_of_8():
    """patch 14 gives K = 588: the host entry point re-pitches the staged copy for the tensor-core path."""
    import dataclasses
    cfg = dataclasses.replace(_small_bf16(), patch=14)
    grids = [(1, 8, 8), (1, 4, 6)]
    enc, w, patches, feats, cu_rows, _ = _run_stage(cfg, grids, seed=10, with_taps=False)
    hp = dev(patches, cfg.dtype).cpu().pin_memory()
    hf = torch.zeros((feats.shape[0], cfg.out_dim), dtype=feats.dtype).pin_memory()
    rows, cu2 = enc.encode_host(hp, grids, hf)
    torch.cuda.synchronize()
    assert rows == feats.shape[0] and np.array_equal(cu2, cu_rows)
    assert torch.equal(hf, feats.cpu())
    enc.close()


def test_pipelined_host_entry_point_over_a_stream_of_requests():
    """Seven requests of different batches through epd_encode_host_async, each with host buffers of its own:
    after one join and a synchronisation of the stream every request's features equal those of the device entry
    point bit for bit (two staging slots are reused several times; the copies run on the encoder's streams)."""
    cfg = _small_bf16()
    w = synth.make_weights(cfg, seed=33)
    batches = [[(1, 16, 16), (1, 6, 10)], [(1, 8, 8)], [(1, 20, 24)], [(1, 16, 16), (1, 6, 10)], [(1, 4, 4), (1, 30, 14)],
               [(1, 8, 8)], [(1, 20, 24)]]
    enc = epd.Encoder(cfg, w, max_tokens=600, max_images=4, max_grid=32)
    want, hps, hfs = [], [], []
    for i, grids in enumerate(batches):
        patches = synth.make_patches(cfg, grids, seed=60 + i)
        feats, _ = enc.encode(dev(patches, cfg.dtype), grids)
        want.append(feats.cpu().clone())
        hps.append(dev(patches, cfg.dtype).cpu().pin_memory())
        hfs.append(torch.zeros((feats.shape[0], cfg.out_dim), dtype=feats.dtype).pin_memory())
    torch.cuda.synchronize()
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        for grids, hp, hf in zip(batches, hps, hfs):
            rows, _ = enc.encode_host_async(hp, grids, hf, stream=stream)
            assert rows == hf.shape[0]
        enc.host_join(stream=stream)
    stream.synchronize()                                 # only the caller's stream: the join covers the copies
    for i, (hf, ref) in enumerate(zip(hfs, want)):
        assert torch.equal(hf, ref), i
    assert enc.last_status() == epd.EPD_OK
    enc.close()


def test_repeated_requests_replay_a_captured_graph():
    """On a capturable stream the second identical request captures its launch sequence and later ones replay
    it: same bits as the plain launches, one graph per (batch, buffers); other batches in between, a changed
    SM budget and switching the mechanism off all keep the results identical."""
    cfg = _small_bf16()
    w = synth.make_weights(cfg, seed=35)
    ga, gb = [(1, 20, 24), (1, 6, 6)], [(1, 8, 8)]
    pa = dev(synth.make_patches(cfg, ga, seed=70), cfg.dtype)
    pb = dev(synth.make_patches(cfg, gb, seed=71), cfg.dtype)
    enc = epd.Encoder(cfg, w, max_tokens=600, max_images=4, max_grid=32)
    ref_a = enc.encode(pa, ga)[0].clone()                     # default stream: plain launches
    ref_b = enc.encode(pb, gb)[0].clone()
    torch.cuda.synchronize()
    assert enc.graph_count() == 0
    stream = torch.cuda.Stream()
    fa = torch.empty_like(ref_a)
    fb = torch.empty_like(ref_b)
    with torch.cuda.stream(stream):
        for i in range(4):                                    # a, a (capture), a (replay), a (replay)
            fa.zero_()
            enc.encode(pa, ga, features=fa, stream=stream)
            stream.synchronize()
            assert torch.equal(fa, ref_a), i
        assert enc.graph_count() == 1 and enc.last_launch_count() == 7 * cfg.layers + 4
        for i in range(3):                                    # alternate with another batch: layouts restaged
            fb.zero_()
            enc.encode(pb, gb, features=fb, stream=stream)
            fa.zero_()
            enc.encode(pa, ga, features=fa, stream=stream)
            stream.synchronize()
            assert torch.equal(fb, ref_b) and torch.equal(fa, ref_a), i
        for _ in range(2):
            fb.zero_()
            enc.encode(pb, gb, features=fb, stream=stream)    # b, b: the second one captures
        stream.synchronize()
        assert torch.equal(fb, ref_b) and enc.graph_count() == 2
        try:
            epd.set_sm_limit(24)                              # another budget: another graph
            for _ in range(3):
                fa.zero_()
                enc.encode(pa, ga, features=fa, stream=stream)
            stream.synchronize()
            assert torch.equal(fa, ref_a) and enc.graph_count() == 3
        finally:
            epd.set_sm_limit(0)
        enc.use_graphs(False)
        fa.zero_()
        enc.encode(pa, ga, features=fa, stream=stream)
        stream.synchronize()
        assert torch.equal(fa, ref_a) and enc.graph_count() == 3
    assert enc.last_status() == epd.EPD_OK
    enc.close()


@pytest.mark.parametrize("which", ["dh72", "dh128", "dh80"])
def test_random_batches_repeat_bit_identically(which):
    """Random item lists (1-6 items, stills and clips, grids of 2..64 patches a side) on two-layer encoders of
    the three head widths: every batch, encoded four more times on a side stream (plain, captured, replayed),
    gives the bits of its first encode and leaves the status word clean."""
    import dataclasses
    base = {"dh72": synth.VIT_06B, "dh128": synth.VIT_6B, "dh80": synth.VIT_07B}[which]
    cfg = dataclasses.replace(base, layers=2, name=which)
    w = synth.make_weights(cfg, seed=1)
    enc = epd.Encoder(cfg, w, max_tokens=12000, max_images=8, max_grid=64)
    rng = np.random.default_rng({"dh72": 5, "dh128": 6, "dh80": 7}[which])
    side = torch.cuda.Stream()
    K = cfg.patch_dim
    ld = (K + 7) // 8 * 8
    done = 0
    while done < 8:
        n = int(rng.integers(1, 7))
        grids = [(int(rng.integers(1, 3)), 2 * int(rng.integers(1, 33)), 2 * int(rng.integers(1, 33))) for _ in range(n)]
        T = synth.num_tokens(grids)
        if T > 12000:
            continue
        done += 1
        p = torch.zeros((T, ld), dtype=torch.bfloat16, device="cuda")
        p[:, :K] = epd.to_device(synth.normal(100 + done, "p", (T, K), 1.0, 0.0, cfg.dtype), cfg.dtype)
        ref = enc.encode(p, grids)[0].clone()
        torch.cuda.synchronize()
        assert enc.last_status() == epd.EPD_OK and torch.isfinite(ref.float()).all()
        out = torch.empty_like(ref)
        with torch.cuda.stream(side):
            for rep in range(4):
                out.zero_()
                enc.encode(p, grids, features=out, stream=side)
                side.synchronize()
                assert torch.equal(out, ref), (grids, rep)
        assert enc.last_status() == epd.EPD_OK
    enc.close()


# ----------------------------------------------------------------------------- edge cases / errors

def test_empty_and_invalid_batches():
    cfg = synth.tiny_variant(head_dim=8, heads=2, layers=1, mlp=16, patch=1, out_dim=8)
    w = synth.make_weights(cfg, seed=1)
    enc = epd.Encoder(cfg, w, max_tokens=64, max_images=2, max_grid=8)
    feats = torch.zeros((16, cfg.out_dim), device="cuda")
    out, cu_rows = enc.encode(None, [], features=feats)
    assert out.shape[0] == 0 and cu_rows.tolist() == [0]
    p = dev(synth.make_patches(cfg, [(1, 2, 2)]), cfg.dtype)
    enc.encode(p, [(1, 2, 2)], features=feats)
    assert enc.last_launch_count() > 0
    for bad in ([(1, 3, 2)], [(0, 2, 2)], [(1, 2, -2)]):
        with pytest.raises(epd.EpdError) as ei:
            enc.encode(p, bad, features=feats)
        assert ei.value.status == epd.EPD_EINVAL and enc.last_launch_count() == 0
    for too_big in ([(1, 2, 2)] * 3, [(1, 10, 2)], [(1, 8, 8), (1, 2, 2)]):
        with pytest.raises(epd.EpdError) as ei:
            enc.encode(p, too_big, features=feats)
        assert ei.value.status == epd.EPD_ECAPACITY and enc.last_launch_count() == 0
    with pytest.raises(epd.EpdError) as ei:   # feature buffer too small
        enc.encode(dev(synth.make_patches(cfg, [(1, 8, 8)]), cfg.dtype), [(1, 8, 8)], features=feats[:8])
    assert ei.value.status == epd.EPD_ECAPACITY and enc.last_launch_count() == 0
    # a rejected call enqueues nothing: not on the device entry point (a NULL / misaligned buffer is found before
    # the layout is staged), not on the host-buffer and raw-frame entry points (odd grid found before the copy)
    grids_new = [(1, 4, 4)]                      # a layout the device does not hold yet
    with pytest.raises(epd.EpdError) as ei:
        enc.encode(None, grids_new, features=feats)
    assert ei.value.status == epd.EPD_EINVAL and enc.last_launch_count() == 0
    with pytest.raises(epd.EpdError) as ei:
        raw = torch.zeros(16 * cfg.patch_dim + 4, device="cuda")
        enc.encode(raw[1:1 + 16 * cfg.patch_dim].view(16, cfg.patch_dim), grids_new, features=feats)   # 4-byte aligned only
    assert ei.value.status == epd.EPD_EINVAL and enc.last_launch_count() == 0
    hp = torch.zeros((64, cfg.patch_dim)).pin_memory()
    hf = torch.zeros((16, cfg.out_dim)).pin_memory()
    for call in (enc.encode_host, enc.encode_host_async):
        with pytest.raises(epd.EpdError) as ei:
            call(hp, [(1, 3, 2)], hf)
        assert ei.value.status == epd.EPD_EINVAL and enc.last_launch_count() == 0
    with pytest.raises(epd.EpdError) as ei:
        enc.encode_frames(torch.zeros(64, dtype=torch.uint8, device="cuda"), [(1, 3, 2)], synth.PIXEL_MEAN, synth.PIXEL_STD,
                          features=feats)
    assert ei.value.status == epd.EPD_EINVAL and enc.last_launch_count() == 0
    # the encoder still works afterwards, at its maximum size
    grids = [(1, 8, 8)]
    out, _ = enc.encode(dev(synth.make_patches(cfg, grids), cfg.dtype), grids, features=feats)
    ref = O.encode(cfg, w, synth.make_patches(cfg, grids), grids)
    assert_parity(to_np(out), ref, TOL_F32)
    enc.close()


def test_expired_wait_is_reported_and_the_encoder_recovers():
    """The bounded device-side waits, made to run out: with a limit of a thousand cycles the ordinary wait of an
    epilogue warp for its first accumulator (tiles still on their way from memory) counts as expired; the kernels
    record the timeout, let what they have in flight complete, free their tensor memory and return.  The status
    call reports EPD_ETIMEOUT once; with the limit restored, the next encode is bit-identical to the one before."""
    cfg = _small_bf16()
    grids = [(1, 16, 16), (1, 8, 12)]
    T = synth.num_tokens(grids)
    w = synth.make_weights(cfg, seed=40)
    enc = epd.Encoder(cfg, w, max_tokens=T, max_images=len(grids), max_grid=16)
    p = dev(synth.make_patches(cfg, grids, seed=40), cfg.dtype)
    ref, _ = enc.encode(p, grids)
    ref = ref.clone()
    torch.cuda.synchronize()
    assert enc.last_status() == epd.EPD_OK
    epd.set_wait_limit(1000)
    try:
        enc.encode(p, grids)
        torch.cuda.synchronize()
        st = enc.last_status()
    finally:
        epd.set_wait_limit(0)
    assert st == epd.EPD_ETIMEOUT
    assert enc.last_status() == epd.EPD_OK          # reading the status cleared it
    again, _ = enc.encode(p, grids)
    torch.cuda.synchronize()
    assert enc.last_status() == epd.EPD_OK
    assert torch.equal(again, ref)
    enc.close()


def test_create_rejects_small_workspace():
    lib = epd.load_library()
    c = epd.make_config(synth.TINY_FP32, 512, 2, 16)
    need = lib.epd_encoder_workspace_bytes(ctypes.byref(c))
    ws = torch.empty(need, dtype=torch.uint8, device="cuda")
    w = epd.WeightsStruct()
    handle = ctypes.c_void_p()
    w.patch_w = ws.data_ptr(); w.patch_w_ld = 588; w.proj_w1 = ws.data_ptr(); w.final_norm_w = ws.data_ptr()
    arr = (ctypes.c_void_p * 2)(ws.data_ptr(), ws.data_ptr())
    for n in ("norm1_w", "qkv_w", "out_w", "norm2_w", "fc1_w", "fc2_w"):
        setattr(w, n, ctypes.cast(arr, ctypes.POINTER(ctypes.c_void_p)))
    base = (ws.data_ptr() + 255) // 256 * 256
    assert lib.epd_encoder_create(ctypes.byref(c), ctypes.byref(w), base, need - 4096, ctypes.byref(handle)) \
        == epd.EPD_ENOMEM
    assert lib.epd_encoder_create(ctypes.byref(c), ctypes.byref(w), base + 8, need, ctypes.byref(handle)) \
        == epd.EPD_EINVAL


# ---------------------------------------------------------------------------------------------
# Feature keys and the feature cache
# ---------------------------------------------------------------------------------------------
def test_content_hash_bit_exact():
    """Keys of items of very different sizes (empty, one word, several blocks' worth, ragged against
    the launch width) equal the oracle's, bit for bit."""
    rng = np.random.default_rng(11)
    sizes = [0, 8, 16, 8 * 255, 8 * 256, 8 * 257, 8 * 64 * 256, 8 * (64 * 256 + 1), 8 * 150001, 1176 * 4 * 1024]
    items = [rng.integers(0, 256, size=s, dtype=np.uint8) for s in sizes]
    items[3][:] = 0                                     # an all-zero item still has a non-trivial key
    flat = np.concatenate(items)
    off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int64)
    got = epd.op_content_hash(torch.from_numpy(flat).cuda(), off)
    want = np.array([O.content_hash(it.tobytes()) for it in items], dtype=np.uint64)
    assert got.dtype == np.uint64 and np.array_equal(got, want), (got, want)
    assert epd.op_content_hash(torch.zeros(8, dtype=torch.uint8, device="cuda"), [0]).size == 0
    with pytest.raises(ValueError):
        epd.op_content_hash(torch.zeros(16, dtype=torch.uint8, device="cuda"), [0, 12])


def test_feature_cache_hits_misses_and_eviction():
    cache = epd.FeatureCache(pool_bytes=4096, out_dim=64, dtype=epd.DTYPE_BF16)   # 128 bytes per row
    mk = lambda rows, val: torch.full((rows, 64), float(val), dtype=torch.bfloat16, device="cuda")
    assert cache.lookup(1, 8) is None
    cache.insert(1, mk(8, 1))           # 1024 bytes
    cache.insert(2, mk(16, 2))          # 2048
    cache.insert(2, mk(16, 9))          # same key, same row count: kept as is
    assert torch.equal(cache.lookup(1, 8), mk(8, 1)) and torch.equal(cache.lookup(2, 16), mk(16, 2))
    assert cache.lookup(1, 4) is None   # same key, other row count: a miss
    cache.insert(3, mk(12, 3))          # 1536 bytes: does not fit behind key 2, wraps and evicts 1 and 2
    st = cache.stats()
    assert cache.lookup(1, 8) is None and torch.equal(cache.lookup(3, 12), mk(12, 3))
    assert st["evictions"] >= 1 and st["entries"] == cache.stats()["entries"]
    cache.insert(3, mk(4, 7))           # same key, other row count: replaces the entry
    assert cache.lookup(3, 12) is None and torch.equal(cache.lookup(3, 4), mk(4, 7))
    cache.insert(4, mk(0, 0))           # an item without rows
    assert cache.lookup(4, 0).shape == (0, 64)
    with pytest.raises(epd.EpdError):
        cache.insert(5, mk(64, 5))      # 8192 bytes can never fit
    torch.cuda.synchronize()
    cache.close()


def test_encode_frames_cached_matches_uncached():
    """A batch with a repeated image: the repeat is served from the cache, every item's features are
    bit-identical to the uncached encode of the same item, and a second call hits for every item."""
    cfg = _small_bf16()
    grids = [(1, 4, 6), (1, 8, 4), (1, 4, 6)]
    w = synth.make_weights(cfg, seed=21)
    frames = synth.make_frames(cfg, grids, seed=22)
    frames[2] = frames[0].copy()
    enc = epd.Encoder(cfg, w, max_tokens=synth.num_tokens(grids), max_images=len(grids), max_grid=8)
    dev, off = epd.pack_frames(frames)
    ref, cu = enc.encode_frames(dev, grids, synth.PIXEL_MEAN, synth.PIXEL_STD)
    ref = ref.clone()
    cache = epd.FeatureCache(pool_bytes=1 << 20, out_dim=cfg.out_dim, dtype=cfg.dtype)
    out, keys, hit = enc.encode_frames_cached(cache, dev, grids, synth.PIXEL_MEAN, synth.PIXEL_STD)
    assert keys[0] == keys[2] != keys[1] and not hit.any()
    assert [int(k) for k in keys] == [O.content_hash(f.tobytes()) for f in frames]
    for i in range(3):
        assert torch.equal(out[i], ref[cu[i]:cu[i + 1]]), i
    out2, _, hit2 = enc.encode_frames_cached(cache, dev, grids, synth.PIXEL_MEAN, synth.PIXEL_STD)
    assert hit2.all() and all(torch.equal(a, b) for a, b in zip(out, out2))
    assert cache.stats()["entries"] == 2
    cache.close()
    enc.close()
