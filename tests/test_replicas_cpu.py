"""Data-parallel item assignment: host logic on CPU, and a two-rank gloo run in which every rank
encodes its own items (with the oracle, on CPU) and the reassembled features equal the whole batch's."""
import os
import socket
import subprocess
import sys

import numpy as np

import synth
from paper_2601_11590_b200 import replicas

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_assignment_is_a_partition_and_balances_cost():
    _, grids = synth.WORKLOADS["cfg2_vit06b_var32"]
    h, m = synth.VIT_06B.hidden, synth.VIT_06B.mlp
    for world in (1, 2, 3, 8):
        a = replicas.assign_items(grids, world, h, m)
        assert sorted(i for r in a for i in r) == list(range(len(grids)))
        loads = replicas.rank_loads(grids, a, h, m)
        total, biggest = sum(loads), max(replicas.item_cost(g, h, m) for g in grids)
        # greedy longest-first bound: max load <= average + largest item
        assert max(loads) <= total / world + biggest + 1e-6
        if world > 1:
            naive = [sum(replicas.item_cost(grids[i], h, m) for i in range(r, len(grids), world)) for r in range(world)]
            assert max(loads) <= max(naive) + 1e-6     # never worse than round-robin on this batch
    # one huge item and many small ones: the huge one sits alone
    grids2 = [(1, 128, 128)] + [(1, 14, 14)] * 6
    a = replicas.assign_items(grids2, 2, h, m)
    assert [0] in a and sorted(a[0] + a[1]) == list(range(7))


def test_feature_row_ranges_match_the_oracle_layout():
    from oracle import encoder_oracle as O
    grids = [(1, 4, 6), (3, 2, 4), (1, 2, 2)]
    cu_out = O.bookkeeping(grids)["cu_out"]
    assert replicas.feature_row_ranges(grids) == [(int(cu_out[i]), int(cu_out[i + 1])) for i in range(3)]


_WORKER = r'''
import os, sys, numpy as np, torch.distributed as dist
sys.path.insert(0, sys.argv[1])
import synth
from oracle import encoder_oracle as O
from paper_2601_11590_b200 import replicas
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
cfg = synth.tiny_variant(head_dim=8, heads=2, layers=2, mlp=24, patch=2)
grids = [(1, 4, 6), (2, 2, 4), (1, 6, 2), (1, 8, 8), (1, 2, 2)]
w = synth.make_weights(cfg, seed=4)
patches = synth.make_patches(cfg, grids, seed=4)
bk = O.bookkeeping(grids)
mine = replicas.assign_items(grids, world, cfg.hidden, cfg.mlp)[rank]
cu = bk["cu_seqlens"]
my_patches = np.concatenate([patches[cu[i]:cu[i + 1]] for i in mine]) if mine else np.zeros((0, cfg.patch_dim))
my_feats = O.encode(cfg, w, my_patches, [grids[i] for i in mine]) if mine else np.zeros((0, cfg.out_dim))
gathered = [None] * world
dist.all_gather_object(gathered, (mine, my_feats))
if rank == 0:
    ranges = replicas.feature_row_ranges(grids)
    full = np.zeros((ranges[-1][1], cfg.out_dim))
    for items, feats in gathered:
        row = 0
        for i in items:
            a, b = ranges[i]
            full[a:b] = feats[row:row + (b - a)]
            row += b - a
    ref = O.encode(cfg, w, patches, grids)
    print("MAXDIFF", float(np.abs(full - ref).max()), "RANKS", sorted(len(g[0]) for g in gathered))
dist.destroy_process_group()
'''


def test_two_ranks_encode_their_items_and_reassemble(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(_WORKER)
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", str(port), str(script), ROOT]
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=300, cwd=ROOT,
                       env=dict(os.environ, CUDA_VISIBLE_DEVICES="", OMP_NUM_THREADS="2"))
    assert r.returncode == 0, r.stderr[-2000:]
    line = [l for l in r.stdout.splitlines() if l.startswith("MAXDIFF")][0].split()
    assert float(line[1]) < 1e-10          # block-diagonal isolation: identical up to summation order
    assert line[3:] and sum(int(v.strip("[],")) for v in line[3:]) == 5
