"""Multi-rank host logic on CPU (gloo, world size 2): contiguous sharding with global element
offsets reproduces the single-buffer result of Algorithm 1's shared random state, and the
rank-ordered squared-norm exchange gives identical bits on every rank."""

import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HP = dict(lr=6e-4, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.1)
N = 50_003


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import oracle
    from paper_2502_20566_b200 import synth
    from paper_2502_20566_b200.dist import global_sqnorm, max_over_ranks, partition
    p, g, m, v = synth.adamw_state(N, 77, "cpu", g_dtype=torch.float32, outlier_fraction=0.01)
    start, length = partition(N, world)[rank]
    sl = slice(start, start + length)
    g_loc = g[sl].numpy().copy()
    local = torch.tensor([oracle.sqnorm(g_loc)], dtype=torch.float64)
    total = global_sqnorm(local)
    gscale = oracle.clip_scale(float(total.item()), 0.125, 1.0)
    pb, mb, vb = (synth.bits16(t[sl]).copy() for t in (p, m, v))
    oracle.adamw_step(pb, g_loc, mb, vb, oracle.hparams(**HP), 1234, 10, 0, start, gscale)
    slowest = max_over_ranks(float(rank + 1), "cpu")
    np.savez(os.path.join(out_dir, f"rank{rank}.npz"), p=pb, m=mb, v=vb, total=total.numpy(), local=local.numpy(),
             start=start, length=length, slowest=slowest)
    dist.barrier()
    dist.destroy_process_group()


def test_partition_properties():
    sys.path.insert(0, ROOT)
    from paper_2502_20566_b200.dist import partition
    for n in (0, 1, 7, 8, 9, 1000, 6_658_404_352):
        for w in (1, 2, 3, 8):
            parts = partition(n, w)
            assert len(parts) == w and sum(l for _, l in parts) == n
            pos = 0
            for s, l in parts:
                assert (s == pos and s % 8 == 0) or l == 0
                pos += l
    assert partition(6_658_404_352, 8)[3] == (3 * 832_300_544, 832_300_544)


def test_two_ranks_reproduce_the_single_buffer(tmp_path):
    world, port = 2, _free_port()
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    sys.path.insert(0, ROOT)
    import oracle
    from paper_2502_20566_b200 import synth
    r = [np.load(tmp_path / f"rank{k}.npz") for k in range(world)]
    # identical global norm on both ranks, equal to the rank-ordered sum of the partials
    assert r[0]["total"].tobytes() == r[1]["total"].tobytes()
    assert float(r[0]["total"][0]) == float(r[0]["local"][0]) + float(r[1]["local"][0])
    assert r[0]["slowest"] == r[1]["slowest"] == 2.0
    # whole-buffer step with the same clip factor
    p, g, m, v = synth.adamw_state(N, 77, "cpu", g_dtype=torch.float32, outlier_fraction=0.01)
    gscale = oracle.clip_scale(float(r[0]["total"][0]), 0.125, 1.0)
    pb, mb, vb = (synth.bits16(t).copy() for t in (p, m, v))
    oracle.adamw_step(pb, g.numpy().copy(), mb, vb, oracle.hparams(**HP), 1234, 10, 0, 0, gscale)
    for name, whole in (("p", pb), ("m", mb), ("v", vb)):
        joined = np.concatenate([r[0][name], r[1][name]])
        assert np.array_equal(joined, whole)
    assert int(r[1]["start"]) % 8 == 0 and int(r[0]["length"]) + int(r[1]["length"]) == N
