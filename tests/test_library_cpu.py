"""Host-side checks of the C library that need no GPU: it loads, exports every declared symbol,
and its pure-host entry points behave."""
import ctypes
import os
import re

import pytest

import synth
import paper_2601_11590_b200 as epd
from paper_2601_11590_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return epd.load_library()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "epd_encoder.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(epd_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert len(names) >= 15
    for name in names:
        assert hasattr(lib, name), name
    assert sorted(epd.EXPORTED_SYMBOLS) == names


def test_strerror_and_padded_head_dim(lib):
    assert epd.strerror(0) == "ok"
    assert "capacity" in epd.strerror(epd.EPD_ECAPACITY)
    assert "unknown" in epd.strerror(-99)
    assert [lib.epd_padded_head_dim(d) for d in (64, 72, 128, 8)] == [64, 80, 128, 16]


def test_workspace_bytes_scales_and_rejects_bad_configs(lib):
    c = epd.make_config(synth.VIT_06B, 6272, 8, 64)
    small = lib.epd_encoder_workspace_bytes(ctypes.byref(c))
    c2 = epd.make_config(synth.VIT_06B, 2 * 6272, 8, 64)
    big = lib.epd_encoder_workspace_bytes(ctypes.byref(c2))
    # at least the float residual stream, the qkv buffer and the MLP hidden buffer
    assert small >= 6272 * (1152 * 4 + 3 * 1152 * 2 + 4304 * 2)
    # the part that does not depend on the batch: the encoder's own copy of the QKV weights (q and k rows
    # reordered for the fused rotary epilogue), 27 layers x [3*1152, 1152] bf16, plus small tables
    fixed = 27 * 3 * 1152 * 1152 * 2
    assert fixed <= small
    assert 1.9 * (small - fixed) < big - fixed < 2.1 * (small - fixed)
    bad = epd.make_config(synth.VIT_06B, 6272, 8, 64)
    bad.heads = 15
    assert lib.epd_encoder_workspace_bytes(ctypes.byref(bad)) == 0
    bad = epd.make_config(synth.VIT_06B, 6272, 8, 64)
    bad.merge = 3
    assert lib.epd_encoder_workspace_bytes(ctypes.byref(bad)) == 0
    assert lib.epd_encoder_workspace_bytes(None) == 0


def test_null_arguments_are_rejected_without_a_device(lib):
    assert lib.epd_encoder_create(None, None, None, 0, None) == epd.EPD_EINVAL
    out = ctypes.c_void_p()
    c = epd.make_config(synth.TINY_FP32, 512, 2, 16)
    assert lib.epd_encoder_create(ctypes.byref(c), None, None, 0, ctypes.byref(out)) == epd.EPD_EINVAL
    assert lib.epd_encode(None, None, 0, None, 0, None, 0, None, None, None) == epd.EPD_EINVAL
    assert lib.epd_encoder_destroy(None) == epd.EPD_OK
    assert lib.epd_op_linear(7, None, 0, None, 0, None, None, 0, 1, 1, 1, 0, None) == epd.EPD_EINVAL


def test_binding_has_no_cpu_path():
    import torch
    if torch.cuda.is_available():
        pytest.skip("GPU present")
    with pytest.raises(RuntimeError, match="CUDA device"):
        epd.Encoder(synth.TINY_FP32, synth.make_weights(synth.TINY_FP32), 512)


def test_bench_reads_the_recorded_dram_traffic():
    """The roofline's `traffic` comes from the ncu summary under profiles/, which records the hash of the kernel
    source it was captured from: a kernel edit without a new capture must show up here, not as a silent null in
    the bench line."""
    import bench
    traffic = bench.linear_dram_traffic(bench.DEFAULT_WORKLOAD)
    assert traffic is not None, "profiles/linear_dram_traffic_per_workload.txt is stale for the current kernel source"
    assert 4e8 < traffic < 2e9          # bytes per launch: above the 510 MB of algorithmic bytes, far below the 3-5 GB of old
    assert bench.linear_dram_traffic("no_such_workload") is None
