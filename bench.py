#!/usr/bin/env python
"""Throughput of the Encode stage (ViT forward) on synthetic data.

  python bench.py --gpus N --steps K --warmup W            # the CUDA path
  python bench.py --impl reference --steps K --warmup W    # the CPU oracle, as it stands

One step = one whole encode (every step of the path) of one packed batch.  The default workload
is the 0.6B-class bf16 encoder on 8 images of 448x448 (6272 image tokens).  With N > 1 (launched by
torch.distributed.run) every rank encodes its own batch of the same shape: independent replicas, no
collective on the data path ("weak" scaling); the value is all ranks' tokens over the slowest
rank's device time.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import synth  # noqa: E402

METRIC = "encoder image-tokens/s"
UNIT = "tokens/s"
DEFAULT_WORKLOAD = "cfg1_vit06b_b8_448"


def algorithmic_flops(cfg, grids) -> dict:
    """FLOPs one forward must perform: true head_dim, full bidirectional blocks per image."""
    T = synth.num_tokens(grids)
    h, m, L = cfg.hidden, cfg.mlp, cfg.layers
    seg2 = float(sum((t * a * b) ** 2 for t, a, b in grids))
    Tm = T // 4
    proj = 4 * h * cfg.out_dim if cfg.proj_kind == synth.PROJ_LINEAR else \
        4 * h * cfg.proj_hidden + cfg.proj_hidden * cfg.out_dim
    linear = 2.0 * T * cfg.patch_dim * h + L * 2.0 * T * (4 * h * h + 2 * h * m) + 2.0 * Tm * proj
    attention = L * 4.0 * h * seg2
    return {"linear": linear, "attention": attention, "total": linear + attention}


def load_peaks() -> dict:
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        return {"source": "measured", "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "hbm_gbs": float(p["hbm_gbs"])}
    return {"source": "fallback", "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu_index}", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------- CPU oracle legs

def oracle_sample(cfg, grids, seed=0):
    """A bounded, exact slice of the workload: the first image alone through every layer
    (block-diagonal attention makes its features independent of the rest of the batch)."""
    from oracle import encoder_oracle as O
    sample_grids = [grids[0]]
    w = synth.make_weights(cfg, seed=seed)
    patches = synth.make_patches(cfg, sample_grids, seed=seed)
    tokens = synth.num_tokens(sample_grids)

    def run():
        t0 = time.perf_counter()
        O.encode(cfg, w, patches, sample_grids)
        return time.perf_counter() - t0
    desc = (f"image 0 of {len(grids)} alone ({tokens} of {synth.num_tokens(grids)} tokens), all {cfg.layers} layers, "
            f"float64 numpy")
    return run, tokens, desc


def cpu_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 0) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return int(max(n))
    except Exception:
        pass
    return os.cpu_count() or 1


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg, grids = synth.WORKLOADS[args.workload]
    run, tokens, desc = oracle_sample(cfg, grids)
    for _ in range(args.warmup):
        run()
    times = [run() for _ in range(args.steps)]
    total = float(sum(times))
    value = tokens * args.steps / total
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "sample": desc},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ----------------------------------------------------------------------------- replicas (N > 1)

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the linear kernel, mean over the linear launches of one
# encode, from ncu captures of every linear shape of the workload (profiles/linear_pair_dram_traffic_cfg1_shapes.txt).
# Only for the workload whose shapes were captured; None elsewhere, and to be reset to None when that kernel changes.
LINEAR_DRAM_BYTES_PER_LAUNCH = {"cfg1_vit06b_b8_448": 58.26e6}


def weight_bytes(cfg) -> float:
    """Bytes of the encoder's weight matrices (the part a step streams from HBM)."""
    es = 2 if cfg.dtype == synth.DTYPE_BF16 else 4
    h, m = cfg.hidden, cfg.mlp
    per_layer = 3 * h * h + h * h + 2 * h * m
    proj = 4 * h * cfg.proj_hidden + cfg.proj_hidden * cfg.out_dim if cfg.proj_kind == synth.PROJ_MLP else 4 * h * cfg.out_dim
    return es * float(cfg.layers * per_layer + cfg.patch_dim * h + proj)


def rank_env():
    """(world size, rank, local rank) as torch.distributed.run exports them; (1, 0, 0) when run alone."""
    return (int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0")),
            int(os.environ.get("LOCAL_RANK", "0")))


def replica_seed(rank: int) -> int:
    """Every replica encodes its own batch: same shapes, pixels drawn from a stream of its own."""
    return rank


def max_over_ranks(ms: float, device) -> float:
    """The slowest rank's time (the job's time); a no-op without a process group."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(tokens_per_rank: int, world: int, steps: int, ms_total: float) -> float:
    """Aggregate image-tokens/s of `world` independent replicas over the slowest rank's time."""
    return world * tokens_per_rank * steps / (ms_total * 1e-3)


def run_dist_selftest(args):
    """CPU check of the N > 1 plumbing (gloo): per-rank seeds differ, the time is the max over ranks,
    rank 0 alone prints."""
    import torch
    import torch.distributed as dist
    world, rank, _ = rank_env()
    dist.init_process_group("gloo")
    cfg, grids = synth.WORKLOADS["cfg0_tiny_fp32"]
    patches = synth.make_patches(cfg, grids, seed=replica_seed(rank))
    digest = float(np.abs(patches).sum())
    digests = [None] * world
    dist.all_gather_object(digests, digest)
    ms = max_over_ranks(10.0 * (rank + 1), torch.device("cpu"))
    dist.barrier()
    if rank == 0:
        print(json.dumps({"selftest": "dist", "world": world, "ms_max": ms, "distinct_batches": len(set(digests)),
                          "value": whole_job_value(synth.num_tokens(grids), world, 1, ms)}))
    dist.destroy_process_group()


# ----------------------------------------------------------------------------- CUDA path

def run_cuda(args):
    import torch
    import torch.distributed as dist
    import paper_2601_11590_b200 as epd
    from paper_2601_11590_b200 import build

    world, rank, local_rank = rank_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the Encode-stage library has no CPU path")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if rank == 0:
        build.build_library()
    if world > 1:
        dist.barrier()
    epd.load_library()

    cfg, grids = synth.WORKLOADS[args.workload]
    T = synth.num_tokens(grids)
    Tm = T // 4
    K = cfg.patch_dim
    ld = (K + 7) // 8 * 8 if cfg.dtype == synth.DTYPE_BF16 else K
    tdt = epd.torch_dtype(cfg.dtype)

    w = synth.make_weights(cfg, seed=0)
    enc = epd.Encoder(cfg, w, max_tokens=T, max_images=len(grids), max_grid=max(max(g[1], g[2]) for g in grids))
    del w
    # every rank encodes its own batch (same shapes, different pixels)
    patches_np = synth.make_patches(cfg, grids, seed=replica_seed(rank))
    host_patches = torch.zeros((T, ld), dtype=tdt).pin_memory()
    host_patches[:, :K] = torch.from_numpy(patches_np).to(tdt)
    dev_patches = host_patches.cuda()
    feats = torch.empty((Tm, cfg.out_dim), dtype=tdt, device="cuda")
    host_feats = torch.empty((Tm, cfg.out_dim), dtype=tdt).pin_memory()
    host_patches_k = host_patches[:, :K].contiguous().pin_memory() if ld != K else host_patches
    stream = torch.cuda.current_stream()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps):
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(steps):
            fn()
        enc.host_join(stream=stream)    # the stream waits for every feature copy still on its way to the host
        e1.record(stream)
        barrier()
        return max_over_ranks(e0.elapsed_time(e1), "cuda")

    def step_device():
        enc.encode(dev_patches, grids, features=feats, stream=stream)

    def step_host():
        # the pipelined host entry point: H2D of step i+1 and D2H of step i-1 overlap the encode of step i
        enc.encode_host_async(host_patches_k, grids, host_feats, stream=stream)

    for _ in range(max(args.warmup, 3)):
        step_device()
    torch.cuda.synchronize()
    if enc.last_status() != epd.EPD_OK:
        raise SystemExit("device-side error during warm-up")
    launches_per_step = enc.last_launch_count()

    sampler = ClockSampler(local_rank) if rank == 0 else None
    if sampler:
        sampler.start()
        time.sleep(0.2)
    ms_total = timed(step_device, args.steps)
    clocks = sampler.stop() if sampler else None
    ms_e2e = timed(step_host, args.steps)

    # per-step-class device times, measured with events around every launch in a separate pass
    enc.profile(True)
    prof = {}
    prof_steps = min(args.steps, 5)
    for _ in range(prof_steps):
        step_device()
        for name, rec in enc.profile_read().items():
            acc = prof.setdefault(name, {"ms": 0.0, "launches": 0})
            acc["ms"] += rec["ms"]
            acc["launches"] += rec["launches"]
    enc.profile(False)
    status = enc.last_status()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = load_peaks()
    flops = algorithmic_flops(cfg, grids)
    ms_step = ms_total / args.steps
    value = whole_job_value(T, world, args.steps, ms_total)
    e2e_value = whole_job_value(T, world, args.steps, ms_e2e)
    es = 2 if cfg.dtype == synth.DTYPE_BF16 else 4

    # dominant kernel: the tcgen05 linear kernels (all linear launches of a step)
    lin_classes = ["patch_embed", "qkv_linear", "out_linear", "fc1_linear", "fc2_linear", "projector"]
    lin_ms = sum(prof[c]["ms"] for c in lin_classes) / prof_steps
    lin_launches = sum(prof[c]["launches"] for c in lin_classes) // prof_steps
    att_ms = prof["attention"]["ms"] / prof_steps
    peak_tf = peaks["bf16_tflops_sustained"]
    achieved_tf = flops["linear"] / (lin_ms * 1e-3) / 1e12 if lin_ms > 0 else 0.0
    roofline = {
        "bound": "tensor", "kernel": "linear_pair_kernel / linear_tc_kernel (all linear layers of a step)",
        "achieved": achieved_tf, "peak": peak_tf, "unit": "TFLOP/s", "frac": achieved_tf / peak_tf,
        "peak_source": f"{peaks['source']} sustained bf16 (kernel timed inside a long step)",
        "flops_per_launch": flops["linear"] / max(lin_launches, 1),
        "avg_launch_ms": lin_ms / max(lin_launches, 1), "launches_per_step": lin_launches,
        "traffic": LINEAR_DRAM_BYTES_PER_LAUNCH.get(args.workload),
        "attention": {"achieved": flops["attention"] / (att_ms * 1e-3) / 1e12 if att_ms > 0 else 0.0,
                      "unit": "TFLOP/s", "ms_per_step": att_ms},
        "whole_step": {"achieved": flops["total"] / (ms_step * 1e-3) / 1e12, "unit": "TFLOP/s",
                       "frac_of_sustained": flops["total"] / (ms_step * 1e-3) / 1e12 / peak_tf,
                       "frac_of_burst": flops["total"] / (ms_step * 1e-3) / 1e12 / peaks["bf16_tflops"],
                       "frac_of_nominal_2250": flops["total"] / (ms_step * 1e-3) / 1e12 / 2250.0},
        "step_breakdown_ms": {k: v["ms"] / prof_steps for k, v in prof.items() if v["launches"]},
    }

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        run, tokens, desc = oracle_sample(cfg, grids)
        t = run()
        cpu = {"value": tokens / t, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle", "sample": desc,
               "seconds": t}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16" if cfg.dtype == synth.DTYPE_BF16 else "f32", "data": "synthetic",
        "config": {"workload": args.workload, "encoder": cfg.name, "images_per_gpu": len(grids),
                   "tokens_per_gpu": T, "merged_tokens_per_gpu": Tm, "out_dim": cfg.out_dim,
                   "l2": f"weights ({weight_bytes(cfg) / 1e9:.1f} GB) and activations exceed the 126 MB L2; "
                         "no flush between steps",
                   "parallelism": f"replicas x{world}", "tflop_per_step": flops["total"] / 1e12},
        "images_per_s": world * len(grids) * args.steps / (ms_total * 1e-3),
        "e2e": {"value": e2e_value, "unit": UNIT, "ms_per_step": ms_e2e / args.steps,
                "h2d_bytes_per_step": T * K * es, "d2h_bytes_per_step": Tm * cfg.out_dim * es,
                "api": "epd_encode_host_async + epd_encode_host_join (pinned host patches in, pinned host features "
                       "out, every step; copies of neighbouring steps overlap the encodes)"},
        "gpu_launches": int(launches_per_step * args.steps),
        "tensor_cores": enc.uses_tensor_cores(),
        "device_status": status,
        "clocks": clocks,
        "roofline": roofline,
        "cpu_baseline": cpu,
    }
    print(json.dumps(line))
    enc.close()
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["cuda", "reference"], default="cuda")
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(synth.WORKLOADS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--dist-selftest", action="store_true", help="CPU/gloo check of the multi-rank plumbing")
    args = ap.parse_args()
    if args.dist_selftest:
        run_dist_selftest(args)
        return
    if args.impl == "reference":
        if args.steps == 20:
            args.steps = 3
        args.warmup = min(args.warmup, 1)
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
