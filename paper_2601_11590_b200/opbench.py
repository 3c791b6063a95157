"""Time single steps of the Encode-stage library on random device data.

  python -m paper_2601_11590_b200.opbench linear --M 6272 --N 4304 --K 1152 --mode gelu_tanh
  python -m paper_2601_11590_b200.opbench attention --heads 16 --dh 72 --seglens 784x8
  python -m paper_2601_11590_b200.opbench rope --T 6272 --heads 16 --dh 72
  python -m paper_2601_11590_b200.opbench rmsnorm --T 6272 --hidden 1152
  python -m paper_2601_11590_b200.opbench hash --items 64 --item-bytes 4816896
  python -m paper_2601_11590_b200.opbench qkv --T 6272 --heads 16 --dh 72        (projection + rotary + split, fused)
  python -m paper_2601_11590_b200.opbench colocate --sm-limit 112 --standin-ctas 72   (encoder on an SM budget next to a
                                                                      memory-bound Decode stand-in on a second stream)

Each call goes through the C ABI (epd_op_*), is timed with CUDA events on the launching stream
after warm-up, and prints one JSON line: average device time, algorithmic FLOP/s or bytes/s.
Between timed launches a buffer larger than the L2 cache is overwritten unless --no-flush is given
(the in-pipeline condition, where operands come from the previous step, is closer to --no-flush).
The same command line with --iters 1 --warmup 1 is a convenient small target for a profiler.
"""
from __future__ import annotations

import argparse
import json

import numpy as np

import paper_2601_11590_b200 as epd


def parse_seglens(text: str):
    """'784x8,300,16384' -> [784]*8 + [300, 16384]"""
    out = []
    for part in text.split(","):
        if "x" in part:
            a, b = part.split("x")
            out += [int(a)] * int(b)
        else:
            out.append(int(part))
    return out


def time_op(torch, fn, iters: int, warmup: int, flush: bool) -> float:
    """Average device time of one launch.  With flushing, each launch is timed on its own after the
    L2 was overwritten; without, `iters` launches run back to back inside one pair of events."""
    stream = torch.cuda.current_stream()
    scratch = torch.empty(192 << 20, dtype=torch.uint8, device="cuda") if flush else None
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    if not flush:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        fn()
        e0.record(stream)
        for _ in range(iters):
            fn()
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / iters
    total = 0.0
    for _ in range(iters):
        scratch.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        fn()
        e1.record(stream)
        torch.cuda.synchronize()
        total += e0.elapsed_time(e1)
    return total / iters


def colocate(args, torch):
    """The default benchmark encode on an SM budget, a memory-bound stand-in for a Decode step on the other
    SMs, each alone and both at once on two streams: the mutual slowdown of co-locating the two stages."""
    import synth
    cfg, grids = synth.WORKLOADS["cfg1_vit06b_b8_448"]
    w = synth.make_weights(cfg, seed=0)
    T = synth.num_tokens(grids)
    enc = epd.Encoder(cfg, w, max_tokens=T, max_images=len(grids), max_grid=max(max(g[1], g[2]) for g in grids))
    patches = epd.to_device(synth.make_patches(cfg, grids, seed=0), cfg.dtype)
    n_bytes = int(args.standin_gb * (1 << 30)) // 16 * 16
    data = torch.randint(0, 255, (n_bytes,), dtype=torch.uint8, device="cuda")
    sums = torch.zeros(4096, dtype=torch.int64, device="cuda")
    sa, sb = torch.cuda.Stream(), torch.cuda.Stream()

    def run(encoder: bool, standin: bool, passes: int):
        torch.cuda.synchronize()
        ea0, ea1, eb0, eb1 = (torch.cuda.Event(enable_timing=True) for _ in range(4))
        if standin:
            eb0.record(sb)
            epd.op_stream_read(data, passes, args.standin_ctas, sums, stream=sb)
            eb1.record(sb)
        if encoder:
            ea0.record(sa)
            with torch.cuda.stream(sa):
                for _ in range(args.encodes):
                    enc.encode(patches, grids, stream=sa)
            ea1.record(sa)
        torch.cuda.synchronize()
        return (ea0.elapsed_time(ea1) / args.encodes if encoder else None,
                n_bytes * passes / (eb0.elapsed_time(eb1) * 1e-3) / 1e9 if standin else None)

    res = {"op": "colocate", "workload": "cfg1_vit06b_b8_448", "encodes": args.encodes, "standin_gb": args.standin_gb,
           "standin_ctas": args.standin_ctas}
    epd.set_sm_limit(0)
    run(True, False, 1)
    res["encode_ms_all_sms"] = run(True, False, 1)[0]
    epd.set_sm_limit(args.sm_limit)
    res["sm_limit"] = args.sm_limit
    run(True, False, 1)
    res["encode_ms_alone"] = run(True, False, 1)[0]
    run(False, True, 1)
    res["standin_gbs_alone"] = run(False, True, 4)[1]
    # size the stand-in to last about as long as the encodes
    passes = max(1, int(res["encode_ms_alone"] * args.encodes * 1e-3 * res["standin_gbs_alone"] * 1e9 / n_bytes))
    both = run(True, True, passes)
    res.update(encode_ms_together=both[0], standin_gbs_together=both[1], standin_passes=passes)
    res["encode_slowdown"] = both[0] / res["encode_ms_alone"]
    res["standin_slowdown"] = res["standin_gbs_alone"] / both[1]
    epd.set_sm_limit(0)
    enc.close()
    print(json.dumps(res))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("op", choices=["linear", "attention", "rope", "rmsnorm", "merge", "hash", "qkv", "colocate", "patchify"])
    ap.add_argument("--image", default="448x448", help="patchify: HxW of every image")
    ap.add_argument("--patch", type=int, default=16)
    ap.add_argument("--bf16-frames", action="store_true")
    ap.add_argument("--M", type=int, default=6272)
    ap.add_argument("--N", type=int, default=1152)
    ap.add_argument("--K", type=int, default=1152)
    ap.add_argument("--mode", default="plain", choices=["plain", "gelu_tanh", "gelu_erf", "accum", "out_f32"])
    ap.add_argument("--e4m3", action="store_true", help="linear: the 8-bit floating-point variant (operands quantised beforehand)")
    ap.add_argument("--tile-n", type=int, default=0)
    ap.add_argument("--T", type=int, default=6272)
    ap.add_argument("--hidden", type=int, default=1152)
    ap.add_argument("--heads", type=int, default=16)
    ap.add_argument("--dh", type=int, default=72)
    ap.add_argument("--seglens", default="784x8")
    ap.add_argument("--sm-limit", type=int, default=112)
    ap.add_argument("--standin-ctas", type=int, default=72)
    ap.add_argument("--standin-gb", type=float, default=2.0)
    ap.add_argument("--encodes", type=int, default=10)
    ap.add_argument("--items", type=int, default=64)
    ap.add_argument("--item-bytes", type=int, default=4816896)
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--no-flush", action="store_true")
    ap.add_argument("--fma", action="store_true", help="force the plain-FMA kernel")
    ap.add_argument("--two-query-tiles", action="store_true",
                    help="attention: force the kernel with two query tiles per CTA")
    ap.add_argument("--split-keys", action="store_true",
                    help="attention: the kernel with one query tile per CTA and key tiles split between the warpgroups")
    args = ap.parse_args()

    import torch
    from paper_2601_11590_b200 import build
    build.build_library()
    epd.load_library()
    dt = epd.DTYPE_BF16
    bf = torch.bfloat16
    g = torch.Generator(device="cuda").manual_seed(0)
    rnd = lambda *shape, std=1.0, dtype=bf: (torch.randn(*shape, generator=g, device="cuda") * std).to(dtype)
    res = {"op": args.op}

    if args.op == "colocate":
        colocate(args, torch)
        return

    if args.op == "linear":
        M, N, K = args.M, args.N, args.K
        x, w, b = rnd(M, K), rnd(N, K, std=K ** -0.5), rnd(N, std=0.5)
        flags = {"plain": 0, "gelu_tanh": epd.LINEAR_GELU_TANH, "gelu_erf": epd.LINEAR_GELU_ERF,
                 "accum": epd.LINEAR_ACCUMULATE, "out_f32": epd.LINEAR_OUT_F32}[args.mode]
        flags |= args.tile_n << 8
        if args.fma:
            flags |= epd.LINEAR_FORCE_FMA
        f32 = args.mode in ("accum", "out_f32")
        out = torch.zeros((M, N), dtype=torch.float32 if f32 else bf, device="cuda")
        fn = lambda: epd.op_linear(dt, x, w, b, out, M, N, K, flags)
        if args.e4m3:
            xq, xs = epd.op_quantize_e4m3(x)
            wq, ws = epd.op_quantize_e4m3(w)
            fn = lambda: epd.op_linear_e4m3(xq, xs, wq, ws, b, out, K, flags)
            res.update(e4m3=True)
        res.update(M=M, N=N, K=K, mode=args.mode, tile_n=args.tile_n, flops=2.0 * M * N * K,
                   bytes=2.0 * (M * K + N * K) + (8.0 if args.mode == "accum" else 4.0 if f32 else 2.0) * M * N)
    elif args.op == "attention":
        seg = parse_seglens(args.seglens)
        T = sum(seg)
        cu = np.concatenate([[0], np.cumsum(seg)]).astype(np.int32)
        cu_dev = torch.from_numpy(cu).cuda()
        dhp = epd.padded_head_dim(args.dh)
        q, k, v = (torch.zeros((args.heads, T, dhp), dtype=bf, device="cuda") for _ in range(3))
        for t in (q, k, v):
            t[:, :, :args.dh] = rnd(args.heads, T, args.dh, std=0.5)
        if dhp > args.dh:
            v[:, :, args.dh] = 1.0
        lib = epd.load_library()
        out = torch.empty((T, args.heads * args.dh), dtype=bf, device="cuda")
        hcu, hp = epd._i32_array(cu)
        flags = epd.ATTENTION_FORCE_FMA if args.fma else epd.ATTENTION_SPLIT_KEYS if args.split_keys else \
            epd.ATTENTION_TWO_QUERY_TILES if args.two_query_tiles else 0

        def fn():
            epd._check(lib.epd_op_attention(dt, epd._ptr(q), epd._ptr(k), epd._ptr(v), epd._ptr(cu_dev), hp,
                                            hcu.size - 1, epd._ptr(out), T, args.heads, args.dh, flags,
                                            epd._stream_ptr(None)), "epd_op_attention")
        res.update(heads=args.heads, dh=args.dh, T=T, n_seg=len(seg), split_keys=bool(args.split_keys),
                   flops=4.0 * args.heads * args.dh * float(sum(s * s for s in seg)),
                   bytes=2.0 * args.heads * T * (3 * dhp + args.dh))
    elif args.op == "rope":
        T, heads, dh = args.T, args.heads, args.dh
        h = heads * dh
        dhp = epd.padded_head_dim(dh)
        qkv = rnd(T, 3 * h)
        pr = torch.randint(0, 28, (T,), generator=g, device="cuda", dtype=torch.int32)
        pc = torch.randint(0, 28, (T,), generator=g, device="cuda", dtype=torch.int32)
        lib = epd.load_library()
        q, k, v = (torch.empty((heads, T, dhp), dtype=bf, device="cuda") for _ in range(3))

        def fn():
            epd._check(lib.epd_op_rope_split(dt, epd._ptr(qkv), epd._ptr(pr), epd._ptr(pc), epd._ptr(q), epd._ptr(k),
                                             epd._ptr(v), T, heads, dh, 10000.0, 0.17, epd._stream_ptr(None)),
                       "epd_op_rope_split")
        res.update(T=T, heads=heads, dh=dh, bytes=2.0 * T * 3 * h + 2.0 * 3 * heads * T * dhp + 8.0 * T)
    elif args.op == "patchify":
        H, W = (int(v) for v in args.image.split("x"))
        P, n = args.patch, args.items
        hh, ww = H // P, W // P
        T, K = n * hh * ww, 3 * P * P
        ld = (K + 7) // 8 * 8
        pix = torch.randint(0, 256, (n * 3 * hh * P * ww * P,), generator=g, device="cuda", dtype=torch.uint8)
        es = 1
        if args.bf16_frames:
            pix, es = pix.to(bf), 2
        item_bytes = 3 * hh * P * ww * P * es
        off = torch.arange(n + 1, device="cuda", dtype=torch.int64) * item_bytes
        grid = torch.tensor([[1, hh, ww]] * n, device="cuda", dtype=torch.int32)
        cu = torch.arange(n + 1, device="cuda", dtype=torch.int32) * (hh * ww)
        out = torch.empty((T, ld), dtype=bf, device="cuda")
        import ctypes
        mean = (ctypes.c_float * 3)(0.5, 0.5, 0.5)
        istd = (ctypes.c_float * 3)(2.0, 2.0, 2.0)
        lib = epd.load_library()

        def fn():
            epd._check(lib.epd_op_patchify_fmt(dt, epd.FRAMES_BF16 if args.bf16_frames else epd.FRAMES_U8, epd._ptr(pix),
                                               epd._ptr(off), epd._ptr(grid), epd._ptr(cu), n, T, epd._ptr(out), ld, 3, P, 1,
                                               mean, istd, epd._stream_ptr(None)), "epd_op_patchify_fmt")
        res.update(items=n, image=args.image, patch=P, T=T, K=K, bytes=float(T) * K * (es + 2))
    elif args.op == "rmsnorm":
        T, h = args.T, args.hidden
        x = rnd(T, h, dtype=torch.float32)
        gain = rnd(h, std=0.02) + 1
        out = torch.empty((T, h), dtype=bf, device="cuda")
        fn = lambda: epd.op_rmsnorm(dt, x, gain, out, 1e-6)
        res.update(T=T, hidden=h, bytes=6.0 * T * h)
    elif args.op == "qkv":
        T, heads, dh = args.T, args.heads, args.dh
        h = heads * dh
        dhp = epd.padded_head_dim(dh)
        x, w, b = rnd(T, h), rnd(3 * h, h, std=h ** -0.5), rnd(3 * h, std=0.5)
        pr = torch.randint(0, 28, (T,), generator=g, device="cuda", dtype=torch.int32)
        pc = torch.randint(0, 28, (T,), generator=g, device="cuda", dtype=torch.int32)
        lib = epd.load_library()
        sp = epd._stream_ptr(None)
        wp, bp = torch.empty_like(w), torch.empty_like(b)
        epd._check(lib.epd_op_qkv_prepare(epd._ptr(w), h, epd._ptr(b), epd._ptr(wp), epd._ptr(bp), heads, dh, sp),
                   "epd_op_qkv_prepare")
        table = torch.empty((28, dh // 4, 2), dtype=torch.float32, device="cuda")
        epd._check(lib.epd_op_rope_table(epd._ptr(table), 28, dh, 10000.0, sp), "epd_op_rope_table")
        q, k, v = (torch.zeros((heads, T, dhp), dtype=bf, device="cuda") for _ in range(3))

        def fn():
            epd._check(lib.epd_op_qkv_rope(epd._ptr(x), h, epd._ptr(wp), epd._ptr(bp), epd._ptr(pr), epd._ptr(pc),
                                           epd._ptr(table), 28, epd._ptr(q), epd._ptr(k), epd._ptr(v), T, heads, dh,
                                           0.17, sp), "epd_op_qkv_rope")
        res.update(T=T, heads=heads, dh=dh, flops=2.0 * T * 3 * h * h,
                   bytes=2.0 * (T * h + 3 * h * h) + 2.0 * 3 * T * h + 8.0 * T)
    elif args.op == "hash":
        n, nb = args.items, args.item_bytes // 8 * 8
        data = torch.randint(0, 256, (n * nb,), generator=g, device="cuda", dtype=torch.uint8)
        off = torch.arange(n + 1, device="cuda", dtype=torch.int64) * nb
        keys = torch.empty(n, dtype=torch.int64, device="cuda")
        lib = epd.load_library()

        def fn():
            epd._check(lib.epd_op_content_hash(epd._ptr(data), epd._ptr(off), n, epd._ptr(keys),
                                               epd._stream_ptr(None)), "epd_op_content_hash")
        res.update(items=n, item_bytes=nb, bytes=float(n) * nb + 16.0 * n)
    else:
        T, h = args.T // 4 * 4, args.hidden
        y = rnd(T, h)
        idx = torch.randperm(T, generator=g, device="cuda").to(torch.int32)
        lib = epd.load_library()
        out = torch.empty((T // 4, 4 * h), dtype=bf, device="cuda")

        def fn():
            epd._check(lib.epd_op_merge(dt, epd._ptr(y), epd._ptr(idx), epd._ptr(out), T // 4, h,
                                        epd._stream_ptr(None)), "epd_op_merge")
        res.update(T=T, hidden=h, bytes=4.0 * T * h + 4.0 * T)

    ms = time_op(torch, fn, args.iters, args.warmup, not args.no_flush)
    res["ms"] = ms
    res["l2_flush"] = not args.no_flush
    if "flops" in res:
        res["tflops"] = res["flops"] / (ms * 1e-3) / 1e12
    res["gbs"] = res["bytes"] / (ms * 1e-3) / 1e9
    print(json.dumps(res))


if __name__ == "__main__":
    main()
