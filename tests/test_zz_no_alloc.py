"""The allocation-free attention entry point against the ordinary entry points.

epd_op_rope_attention_static() serves callers that may not allocate device memory (their own pool
owns the GPU's memory, or they cannot tolerate the synchronisation an allocation may cause); it keeps
its q/k/v intermediates in a fixed array inside the library.  Here it is called twice in a row through
the C ABI -- the second batch smaller than the first, so anything the first call left in the shared
array would show up if it were read -- and each result is compared with epd_op_rope_split() +
epd_op_attention() on caller-provided buffers, and with the CPU oracle's rotary embedding + block-diagonal
attention on the same inputs.  This file sorts last so that a stop-at-first-failure
run has already executed every other test.
"""
import numpy as np
import pytest
import torch

import synth
import paper_2601_11590_b200 as epd
from oracle import encoder_oracle as O
from tests.metrics import assert_parity

pytestmark = pytest.mark.gpu

TOL = 4e-3   # the single-step bf16 tolerance of the parity tests; float results must agree to 1e-6


def _case(dtype, heads, dh, seglens, seed):
    T = int(sum(seglens))
    h = heads * dh
    cu = np.concatenate([[0], np.cumsum(seglens)]).astype(np.int32)
    qkv = epd.to_device(synth.normal(seed, "qkv", (T, 3 * h), 1.0, 0.0, dtype), dtype)
    rng = np.random.default_rng(seed)
    pr = torch.from_numpy(rng.integers(0, 64, T).astype(np.int32)).cuda()
    pc = torch.from_numpy(rng.integers(0, 64, T).astype(np.int32)).cuda()
    return qkv, pr, pc, cu, T, h


def _oracle(qkv, pr, pc, cu, heads, dh, theta):
    """Rotary embedding of q and k at the tokens' (row, column) positions, then softmax(q k^T / sqrt(dh)) v
    inside each segment, in float64 from the same input numbers."""
    x = qkv.float().cpu().numpy().astype(np.float64)
    T, h = x.shape[0], heads * dh
    pos_r, pos_c = pr.cpu().numpy(), pc.cpu().numpy()
    q = O.rope_2d(x[:, :h].reshape(T, heads, dh), pos_r, pos_c, theta)
    k = O.rope_2d(x[:, h:2 * h].reshape(T, heads, dh), pos_r, pos_c, theta)
    v = x[:, 2 * h:].reshape(T, heads, dh)
    return O.attention_block_diagonal(q, k, v, cu).reshape(T, h)


@pytest.mark.parametrize("dtype", [epd.DTYPE_BF16, epd.DTYPE_F32])
def test_static_scratch_entry_point_matches_ordinary_entry_points_twice(dtype):
    from paper_2601_11590_b200 import build
    build.build_library()
    heads, dh, theta = 4, 72, 10000.0
    q_scale = 1.4426950408889634 / np.sqrt(dh)
    for seglens, seed in (([300, 129, 64], 1), ([17, 40], 2)):
        qkv, pr, pc, cu, T, h = _case(dtype, heads, dh, seglens, seed)
        cu_dev = torch.from_numpy(cu).cuda()
        out = torch.full((T, h), 7.0, dtype=qkv.dtype, device="cuda")
        epd.op_rope_attention_static(dtype, qkv, pr, pc, cu_dev, cu, heads, dh, theta, out=out)
        q, k, v = epd.op_rope_split(dtype, qkv, pr, pc, heads, dh, theta, q_scale)
        ref = epd.op_attention(dtype, q, k, v, cu_dev, cu, dh)
        torch.cuda.synchronize()
        a, b = out.float().cpu().numpy().astype(np.float64), ref.float().cpu().numpy().astype(np.float64)
        err = np.linalg.norm(a - b) / np.linalg.norm(b)
        assert np.isfinite(a).all()
        assert err <= (TOL if dtype == epd.DTYPE_BF16 else 1e-6), err
        # against the oracle: two rounded steps in bf16 (rotated q, k stored as bf16, then the attention output)
        assert_parity(a, _oracle(qkv, pr, pc, cu, heads, dh, theta), 2 * TOL if dtype == epd.DTYPE_BF16 else 1e-5,
                      "static entry point against the oracle")


def test_static_scratch_rejects_oversized_batches():
    from paper_2601_11590_b200 import build
    build.build_library()
    limit = epd.static_scratch_bytes()
    assert limit == 16 << 20
    heads, dh = 16, 72
    per_token = 3 * heads * epd.padded_head_dim(dh) * 2
    T = limit // per_token + 64
    qkv = torch.zeros((T, 3 * heads * dh), dtype=torch.bfloat16, device="cuda")
    pos = torch.zeros(T, dtype=torch.int32, device="cuda")
    cu = np.array([0, T], dtype=np.int32)
    with pytest.raises(epd.EpdError) as ei:
        epd.op_rope_attention_static(epd.DTYPE_BF16, qkv, pos, pos, torch.from_numpy(cu).cuda(), cu, heads, dh, 1e4)
    assert ei.value.status == epd.EPD_ECAPACITY
