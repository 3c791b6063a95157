"""The N > 1 path of bench.py on CPU: two gloo ranks launched the way the driver launches them."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _torchrun(extra, timeout=300):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", str(_free_port()), os.path.join(ROOT, "bench.py"), "--gpus", "2"] + extra
    env = dict(os.environ, CUDA_VISIBLE_DEVICES="", OMP_NUM_THREADS="2")
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=timeout, cwd=ROOT, env=env)
    assert r.returncode == 0, r.stderr[-2000:]
    return [json.loads(l) for l in r.stdout.splitlines() if l.startswith("{")]


def test_two_gloo_ranks_reduce_to_the_slowest_rank_and_rank0_prints():
    lines = _torchrun(["--dist-selftest"])
    assert len(lines) == 1
    d = lines[0]
    assert d["world"] == 2 and d["ms_max"] == 20.0          # rank r reported 10 (r + 1) ms
    assert d["distinct_batches"] == 2                       # every replica drew its own batch
    assert abs(d["value"] - 2 * 512 / 20e-3) < 1e-6         # all ranks' tokens over the slowest rank's time
    assert d["split_covers_batch_once"] is True             # --split: the ranks' shares partition the one batch


def test_reference_arm_under_two_ranks_prints_one_line():
    lines = _torchrun(["--impl", "reference", "--steps", "1", "--warmup", "0", "--workload", "cfg0_tiny_fp32"])
    assert len(lines) == 1 and lines[0]["impl"] == "reference" and lines[0]["n_gpus"] == 2
    assert lines[0]["cpu_baseline"]["kind"] == "oracle" and lines[0]["value"] > 0
