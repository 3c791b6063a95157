#!/usr/bin/env python
"""Throughput of the Encode stage (ViT forward) on synthetic data.

  python bench.py --gpus N --steps K --warmup W            # the CUDA path
  python bench.py --impl reference --steps K --warmup W    # the CPU oracle, as it stands

One step = one whole encode (every step of the path) of one packed batch.  The default workload is the
largest single-GPU configuration: the 6B-class bf16 encoder on 16 images of 448x448 (16384 image tokens,
193 TFLOP per step, 11.6 GB of weights).  The three 0.6B-class configurations (8 x 448x448, 32
variable-resolution images, one 16384-token image + one 16-frame clip) are timed in the same process and
reported under config.other_workloads.  With N > 1 (launched by torch.distributed.run) every rank encodes
its own batch of the same shape: independent replicas, no collective on the data path ("weak" scaling); the
value is all ranks' tokens over the slowest rank's device time.  With --split the ranks instead share ONE
batch of the variable-resolution workload, each encoding the items a cost model assigns to it ("strong").
"""
from __future__ import annotations

import argparse
import dataclasses
import hashlib
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
DEFAULT_WORKLOAD = "cfg4_vit6b_b16_448"
OTHER_WORKLOADS = ["cfg1_vit06b_b8_448", "cfg2_vit06b_var32", "cfg3_vit06b_long"]
SPLIT_WORKLOAD = "cfg2_vit06b_var32"
# Layers of the oracle's timed sample for encoders too deep to run whole within the time allowed.
ORACLE_SAMPLE_LAYERS = 4
# A timed region shorter than this runs at burst clocks (the power cap has not yet pulled the clock down).
BURST_REGION_S = 2.0


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


def pick_peak(peaks: dict, region_s: float, clocks: dict) -> tuple:
    """Burst peak for a timed region under BURST_REGION_S or a median SM clock within 5 % of the maximum,
    the sustained one otherwise."""
    sm, mx = (clocks or {}).get("sm_mhz"), (clocks or {}).get("sm_max_mhz")
    near_max = bool(sm and mx and sm >= 0.95 * mx)
    if region_s < BURST_REGION_S or near_max:
        return peaks["bf16_tflops"], f"{peaks['source']} burst bf16 (timed region {region_s:.2f} s" + \
            (", SM clock within 5 % of max)" if near_max else ")")
    return peaks["bf16_tflops_sustained"], \
        f"{peaks['source']} sustained bf16 (timed region {region_s:.2f} s at a median {sm} MHz of {mx})"


def linear_dram_traffic(workload: str):
    """dram__bytes_read.sum + dram__bytes_write.sum per launch of the linear kernel (mean over the linear
    launches of one encode) from the ncu summary under profiles/, or None when there is no capture for this
    workload or the kernel's source has changed since (the summary records the source's hash)."""
    path = os.path.join(ROOT, "profiles", "linear_dram_traffic_per_workload.txt")
    src = os.path.join(ROOT, "paper_2601_11590_b200", "csrc", "gemm_tcgen05_pair.cu")
    if not (os.path.exists(path) and os.path.exists(src)):
        return None
    with open(src, "rb") as fh:
        digest = hashlib.sha256(fh.read()).hexdigest()[:16]
    with open(path) as fh:
        for line in fh:
            f = line.split()
            if len(f) >= 3 and f[0] == workload and f[2] == digest:
                return float(f[1])
    return None


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
    """A bounded, exact slice of the workload: the first image alone (block-diagonal attention makes its
    features independent of the rest of the batch), through every layer where that takes seconds, else
    through the first ORACLE_SAMPLE_LAYERS layers with the full-depth figure extrapolated by layer count.
    Returns (run() -> seconds, tokens of the sample, depth factor, description)."""
    from oracle import encoder_oracle as O
    sample_grids = [grids[0]]
    tokens = synth.num_tokens(sample_grids)
    per_token_layer = 2.0 * (4 * cfg.hidden ** 2 + 2 * cfg.hidden * cfg.mlp) + 4.0 * cfg.hidden * tokens
    whole = tokens * cfg.layers * per_token_layer <= 2.5e12       # ~30 s of float64 work on a host CPU
    run_cfg = cfg if whole else cfg.with_layers(ORACLE_SAMPLE_LAYERS)
    w = synth.make_weights(run_cfg, seed=seed)
    patches = synth.make_patches(cfg, sample_grids, seed=seed)

    def run():
        t0 = time.perf_counter()
        O.encode(run_cfg, w, patches, sample_grids)
        return time.perf_counter() - t0
    if whole:
        desc = (f"image 0 of {len(grids)} alone ({tokens} of {synth.num_tokens(grids)} tokens), all {cfg.layers} "
                f"layers, float64 numpy")
        return run, tokens, 1.0, desc
    desc = (f"image 0 of {len(grids)} alone ({tokens} of {synth.num_tokens(grids)} tokens), patch embedding + "
            f"{ORACLE_SAMPLE_LAYERS} of {cfg.layers} layers + projector, float64 numpy; value EXTRAPOLATED to full "
            f"depth by the layer count (time x {cfg.layers}/{ORACLE_SAMPLE_LAYERS})")
    return run, tokens, cfg.layers / ORACLE_SAMPLE_LAYERS, desc


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
    run, tokens, depth, desc = oracle_sample(cfg, grids)
    for _ in range(args.warmup):
        run()
    times = [run() for _ in range(args.steps)]
    total = float(sum(times)) * depth
    value = tokens * args.steps / total
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "sample": desc},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle", "sample": desc,
                         "measured_seconds_per_step": float(sum(times)) / args.steps, "depth_factor": depth},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ----------------------------------------------------------------------------- replicas (N > 1)

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


def split_share(cfg, grids, world: int, rank: int):
    """The items of one batch that rank `rank` of `world` encodes (cost-balanced, no overlap, no gap) and
    their positions in the batch."""
    from paper_2601_11590_b200 import replicas
    items = replicas.assign_items(grids, world, cfg.hidden, cfg.mlp)[rank]
    return [grids[i] for i in items], items


def run_dist_selftest(args):
    """CPU check of the N > 1 plumbing (gloo): per-rank seeds differ, the time is the max over ranks,
    rank 0 alone prints; the shares of a split batch cover it exactly once."""
    import torch
    import torch.distributed as dist
    world, rank, _ = rank_env()
    dist.init_process_group("gloo")
    cfg, grids = synth.WORKLOADS["cfg0_tiny_fp32"]
    patches = synth.make_patches(cfg, grids, seed=replica_seed(rank))
    digest = float(np.abs(patches).sum())
    digests = [None] * world
    dist.all_gather_object(digests, digest)
    split_cfg, split_grids = synth.WORKLOADS[SPLIT_WORKLOAD]
    _, mine = split_share(split_cfg, split_grids, world, rank)
    shares = [None] * world
    dist.all_gather_object(shares, list(mine))
    ms = max_over_ranks(10.0 * (rank + 1), torch.device("cpu"))
    dist.barrier()
    if rank == 0:
        covered = sorted(i for s in shares for i in s)
        print(json.dumps({"selftest": "dist", "world": world, "ms_max": ms, "distinct_batches": len(set(digests)),
                          "value": whole_job_value(synth.num_tokens(grids), world, 1, ms),
                          "split_covers_batch_once": covered == list(range(len(split_grids)))}))
    dist.destroy_process_group()


# ----------------------------------------------------------------------------- CUDA path

def streamed_weights(cfg, seed=0):
    """Weights whose blocks are drawn one at a time while the encoder uploads them (the 6B-class encoder's
    float32 host copy would otherwise take 23 GB per process)."""
    w = synth.make_weights(cfg, seed=seed, with_layers=False)
    w["layers"] = (synth.make_layer_weights(cfg, l, seed) for l in range(cfg.layers))
    return w


class Measured:
    """One workload on this rank's GPU: encoder, resident inputs, timing helpers."""

    def __init__(self, name, cfg, grids, seed, weights=None):
        import torch
        import paper_2601_11590_b200 as epd
        self.torch, self.epd = torch, epd
        self.name, self.cfg, self.grids = name, cfg, grids
        self.T = synth.num_tokens(grids)
        self.Tm = self.T // 4
        K = cfg.patch_dim
        self.K = K
        self.ld = (K + 7) // 8 * 8 if cfg.dtype == synth.DTYPE_BF16 else K
        tdt = epd.torch_dtype(cfg.dtype)
        self.enc = epd.Encoder(cfg, weights if weights is not None else streamed_weights(cfg), max_tokens=self.T,
                               max_images=len(grids), max_grid=max(max(g[1], g[2]) for g in grids))
        patches_np = synth.make_patches(cfg, grids, seed=seed)
        host = torch.zeros((self.T, self.ld), dtype=tdt).pin_memory()
        host[:, :K] = torch.from_numpy(patches_np).to(tdt)
        self.dev_patches = host.cuda()
        self.host_patches_k = host[:, :K].contiguous().pin_memory() if self.ld != K else host
        self.feats = torch.empty((self.Tm, cfg.out_dim), dtype=tdt, device="cuda")
        self.host_feats = torch.empty((self.Tm, cfg.out_dim), dtype=tdt).pin_memory()
        self.stream = torch.cuda.current_stream()

    def step_device(self):
        self.enc.encode(self.dev_patches, self.grids, features=self.feats, stream=self.stream)

    def step_host(self):
        # the pipelined host entry point: H2D of step i+1 and D2H of step i-1 overlap the encode of step i
        self.enc.encode_host_async(self.host_patches_k, self.grids, self.host_feats, stream=self.stream)

    def timed(self, fn, steps, barrier):
        torch = self.torch
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(self.stream)
        for _ in range(steps):
            fn()
        self.enc.host_join(stream=self.stream)    # the stream waits for every feature copy still on its way to the host
        e1.record(self.stream)
        barrier()
        return max_over_ranks(e0.elapsed_time(e1), "cuda")

    def profile(self, steps):
        """Device time per step class, events around every launch (a separate pass: the events cost the
        overlap between consecutive kernels that the timed region has)."""
        self.enc.profile(True)
        prof = {}
        for _ in range(steps):
            self.step_device()
            for name, rec in self.enc.profile_read().items():
                acc = prof.setdefault(name, {"ms": 0.0, "launches": 0})
                acc["ms"] += rec["ms"] / steps
                acc["launches"] += rec["launches"]
        self.enc.profile(False)
        for rec in prof.values():
            rec["launches"] //= steps
        return prof

    def close(self):
        self.enc.close()
        self.enc = None
        self.dev_patches = self.feats = None
        self.torch.cuda.empty_cache()


LIN_CLASSES = ["patch_embed", "qkv_linear", "out_linear", "fc1_linear", "fc2_linear", "projector"]


def summarise(m: Measured, ms_total, steps, world, prof, clocks, peaks):
    """Throughput and achieved rates of one workload from its timed region and its profiling pass."""
    flops = algorithmic_flops(m.cfg, m.grids)
    ms_step = ms_total / steps
    lin_ms = sum(prof[c]["ms"] for c in LIN_CLASSES if c in prof)
    lin_launches = sum(prof[c]["launches"] for c in LIN_CLASSES if c in prof)
    att_ms = prof.get("attention", {"ms": 0.0})["ms"]
    prof_sum = sum(v["ms"] for v in prof.values())
    peak, peak_source = pick_peak(peaks, ms_total * 1e-3, clocks)
    tf = lambda fl, ms: fl / (ms * 1e-3) / 1e12 if ms > 0 else 0.0
    return {
        "flops": flops, "ms_step": ms_step, "value": whole_job_value(m.T, world, steps, ms_total),
        "lin_ms": lin_ms, "lin_launches": lin_launches, "att_ms": att_ms, "prof_sum": prof_sum,
        "peak": peak, "peak_source": peak_source,
        "linear_tflops": tf(flops["linear"], lin_ms), "attention_tflops": tf(flops["attention"], att_ms),
        "whole_tflops": tf(flops["total"], ms_step),
    }


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

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    peaks = load_peaks()
    warmup = max(args.warmup, 3)
    workload = SPLIT_WORKLOAD if args.split else args.workload
    cfg, grids = synth.WORKLOADS[workload]
    batch_tokens = synth.num_tokens(grids)
    share_items = None
    if args.split:
        # one batch for the whole job: this rank encodes the items the cost model gives it
        grids, share_items = split_share(cfg, grids, world, rank)
    m = Measured(workload, cfg, grids, seed=0 if args.split else replica_seed(rank))

    for _ in range(warmup):
        m.step_device()
    torch.cuda.synchronize()
    if m.enc.last_status() != epd.EPD_OK:
        raise SystemExit("device-side error during warm-up")
    launches_per_step = m.enc.last_launch_count()

    sampler = ClockSampler(local_rank) if rank == 0 else None
    if sampler:
        sampler.start()
        time.sleep(0.2)
    ms_total = m.timed(m.step_device, args.steps, barrier)
    clocks = sampler.stop() if sampler else None
    ms_e2e = m.timed(m.step_host, args.steps, barrier)
    prof = m.profile(min(args.steps, 3))
    status = m.enc.last_status()
    uses_tc = m.enc.uses_tensor_cores()
    T, Tm, K = m.T, m.Tm, m.K
    n_items = len(grids)
    if args.split:
        # whole-job value: the one batch's tokens over the slowest rank's time
        value = batch_tokens * args.steps / (ms_total * 1e-3)
        e2e_value = batch_tokens * args.steps / (ms_e2e * 1e-3)
    s = summarise(m, ms_total, args.steps, world, prof, clocks, peaks)
    if not args.split:
        value = s["value"]
        e2e_value = whole_job_value(T, world, args.steps, ms_e2e)
    m.close()

    # the other benchmark configurations, same process, rank 0's GPU only (they are context for the line above)
    others = {}
    if rank == 0 and world == 1 and not args.no_other_workloads and not args.split and workload == DEFAULT_WORKLOAD:
        shared = {}
        for name in OTHER_WORKLOADS:
            ocfg, ogrids = synth.WORKLOADS[name]
            base = dataclasses.replace(ocfg, temporal_patch=1, name="")
            if base not in shared:
                shared[base] = synth.make_weights(ocfg, seed=0)
            w = dict(shared[base])
            if w["patch_w"].shape[1] != ocfg.patch_dim:    # same blocks, a patch embedding of its own width
                head = synth.make_weights(ocfg, seed=0, with_layers=False)
                w["patch_w"], w["patch_b"] = head["patch_w"], head["patch_b"]
            om = Measured(name, ocfg, ogrids, seed=0, weights=w)
            osteps = max(5, min(args.steps, int(1500.0 / max(1.0, 0.002 * om.T))))
            for _ in range(warmup):
                om.step_device()
            torch.cuda.synchronize()
            osampler = ClockSampler(local_rank)
            osampler.start()
            time.sleep(0.2)
            oms = om.timed(om.step_device, osteps, barrier)
            oclocks = osampler.stop()
            oprof = om.profile(2)
            ostatus = om.enc.last_status()
            os_ = summarise(om, oms, osteps, 1, oprof, oclocks, peaks)
            others[name] = {
                "tokens_per_s": os_["value"], "images_per_s": len(ogrids) * osteps / (oms * 1e-3),
                "ms_per_step": os_["ms_step"], "steps": osteps, "tokens": om.T,
                "tflop_per_step": os_["flops"]["total"] / 1e12,
                "attention_share_of_flops": os_["flops"]["attention"] / os_["flops"]["total"],
                "whole_step_tflops": os_["whole_tflops"], "attention_tflops": os_["attention_tflops"],
                "linear_tflops": os_["linear_tflops"], "attention_ms": os_["att_ms"],
                "profiled_step_ms": os_["prof_sum"],
                "peak": os_["peak"], "peak_source": os_["peak_source"],
                "whole_step_frac": os_["whole_tflops"] / os_["peak"],
                "attention_frac": os_["attention_tflops"] / os_["peak"],
                "clocks": oclocks, "device_status": ostatus,
            }
            om.close()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    es = 2 if cfg.dtype == synth.DTYPE_BF16 else 4
    peak_tf = s["peak"]
    whole_tf = s["whole_tflops"]
    scale = s["ms_step"] / s["prof_sum"] if s["prof_sum"] > 0 else 1.0
    roofline = {
        "bound": "tensor", "kernel": "linear_pair_kernel / linear_tc_kernel (all linear layers of a step)",
        "achieved": s["linear_tflops"], "peak": peak_tf, "unit": "TFLOP/s", "frac": s["linear_tflops"] / peak_tf,
        "peak_source": s["peak_source"],
        "peaks": {"burst": peaks["bf16_tflops"], "sustained": peaks["bf16_tflops_sustained"], "nominal": 2250.0},
        "frac_of_burst": s["linear_tflops"] / peaks["bf16_tflops"],
        "frac_of_sustained": s["linear_tflops"] / peaks["bf16_tflops_sustained"],
        "frac_of_nominal_2250": s["linear_tflops"] / 2250.0,
        "flops_per_launch": s["flops"]["linear"] / max(s["lin_launches"], 1),
        "avg_launch_ms": s["lin_ms"] / max(s["lin_launches"], 1), "launches_per_step": s["lin_launches"],
        "avg_launch_ms_source": "profiling pass: CUDA events around every launch on the launching stream; that pass "
                                "loses the overlap of consecutive kernels, so its classes sum to profiled_step_ms, "
                                "not to ms_per_step",
        "profiled_step_ms": s["prof_sum"], "timed_step_ms": s["ms_step"],
        "achieved_overlap_adjusted": s["linear_tflops"] / scale if scale > 0 else None,
        "traffic": linear_dram_traffic(workload),
        "attention": {"achieved": s["attention_tflops"], "unit": "TFLOP/s", "ms_per_step": s["att_ms"],
                      "frac": s["attention_tflops"] / peak_tf},
        "whole_step": {"achieved": whole_tf, "unit": "TFLOP/s", "frac": whole_tf / peak_tf,
                       "frac_of_sustained": whole_tf / peaks["bf16_tflops_sustained"],
                       "frac_of_burst": whole_tf / peaks["bf16_tflops"],
                       "frac_of_nominal_2250": whole_tf / 2250.0},
        "step_breakdown_ms": {k: v["ms"] for k, v in prof.items() if v["launches"]},
    }

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        run, tokens, depth, desc = oracle_sample(cfg, synth.WORKLOADS[workload][1])
        t = run()
        cpu = {"value": tokens / (t * depth), "unit": UNIT, "cores": cpu_threads(), "kind": "oracle", "sample": desc,
               "seconds": t, "depth_factor": depth}

    config = {"workload": workload, "encoder": cfg.name, "images_per_gpu": n_items,
              "tokens_per_gpu": T, "merged_tokens_per_gpu": Tm, "out_dim": cfg.out_dim,
              "l2": f"weights ({weight_bytes(cfg) / 1e9:.1f} GB) and activations exceed the 126 MB L2; "
                    "no flush between steps",
              "parallelism": (f"one batch split over {world} replicas by item cost" if args.split
                              else f"replicas x{world}"),
              "tflop_per_step": s["flops"]["total"] / 1e12}
    if share_items is not None:
        config["rank0_items"] = [int(i) for i in share_items]
        config["batch_tokens"] = batch_tokens
    if others:
        config["other_workloads"] = others
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": warmup, "ms_per_step": s["ms_step"], "higher_is_better": True,
        "scaling": "strong" if args.split else "weak",
        "vs_baseline": None, "dtype": "bf16" if cfg.dtype == synth.DTYPE_BF16 else "f32", "data": "synthetic",
        "config": config,
        "images_per_s": (len(synth.WORKLOADS[workload][1]) if args.split else world * n_items) * args.steps / (ms_total * 1e-3),
        "e2e": {"value": e2e_value, "unit": UNIT, "ms_per_step": ms_e2e / args.steps,
                "h2d_bytes_per_step": T * K * es, "d2h_bytes_per_step": Tm * cfg.out_dim * es,
                "api": "epd_encode_host_async + epd_encode_host_join (pinned host patches in, pinned host features "
                       "out, every step; copies of neighbouring steps overlap the encodes)"},
        "gpu_launches": int(launches_per_step * args.steps),
        "tensor_cores": uses_tc,
        "device_status": status,
        "clocks": clocks,
        "roofline": roofline,
        "cpu_baseline": cpu,
    }
    print(json.dumps(line))
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
    ap.add_argument("--no-other-workloads", action="store_true")
    ap.add_argument("--split", action="store_true",
                    help="strong scaling: the ranks share one variable-resolution batch, items assigned by cost")
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
