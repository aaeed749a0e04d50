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


def _sharded_worker(rank, world, port, out_dir, grad_dtype_name="float32"):
    """sharded_clipped_step with the kernel calls replaced by the oracle (CPU tensors, gloo)."""
    grad_dtype = getattr(torch, grad_dtype_name)
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import oracle
    from paper_2502_20566_b200 import synth
    from paper_2502_20566_b200.dist import sharded_clipped_step
    n = 8 * world * 1500
    p, _, m, v = synth.adamw_state(n, 88, "cpu")
    g_local = synth.state_chunk(synth.ROLE_G, 500 + rank, 0, n, "cpu", g_dtype=grad_dtype, outlier_fraction=0.01)
    per = n // world
    sl = slice(rank * per, (rank + 1) * per)
    sp, sm, sv = (t[sl].clone() for t in (p, m, v))

    def as_host(t):      # FP32 values, or BF16 bit patterns
        return t.numpy().copy() if t.dtype == torch.float32 else synth.bits16(t).copy()

    class ops:
        @staticmethod
        def sqnorm(g, out):
            out[0] = oracle.sqnorm(as_host(g))

        @staticmethod
        def clip_scale(total, accum, mx, out):
            out[0] = oracle.clip_scale(float(total.item()), accum, mx)

        @staticmethod
        def step(pp, gg, mm, vv, gscale_dev, offset):
            pb, mb, vb = (synth.bits16(t) for t in (pp, mm, vv))       # views: updated in place
            oracle.adamw_step(pb, as_host(gg), mb, vb, oracle.hparams(**HP), 1234, 7, 0, offset, float(gscale_dev.item()))

    full = torch.empty(n, dtype=torch.bfloat16)
    # gloo has no reduce_scatter_tensor / all_gather_into_tensor on every build: fall back to the list forms
    if not hasattr(dist, "_orig_rs"):
        def rs(out, inp, op=dist.ReduceOp.SUM, group=None):
            t = inp.clone()
            dist.all_reduce(t, op=op, group=group)
            out.copy_(t[dist.get_rank(group) * out.numel():(dist.get_rank(group) + 1) * out.numel()])

        def ag(out, inp, group=None):
            parts = [torch.empty_like(inp) for _ in range(dist.get_world_size(group))]
            dist.all_gather(parts, inp, group=group)
            out.copy_(torch.cat(parts))
        dist._orig_rs = dist.reduce_scatter_tensor
        dist.reduce_scatter_tensor, dist.all_gather_into_tensor = rs, ag
    phases = []
    shard_g = torch.empty(per, dtype=grad_dtype)
    total = sharded_clipped_step(sp, sm, sv, g_local, HP, 1234, 7, max_norm=1.0, accum_scale=1.0 / world,
                                 full_param_out=full, ops=ops, phase_hook=phases.append, shard_grad_out=shard_g)
    np.savez(os.path.join(out_dir, f"s{rank}.npz"), full=synth.bits16(full), m=synth.bits16(sm), v=synth.bits16(sv),
             total=total.numpy(), g=g_local.float().numpy(), shard_g=shard_g.float().numpy(), phases=np.array(phases))
    dist.barrier()
    dist.destroy_process_group()


import pytest


@pytest.mark.parametrize("grad_dtype_name", ["float32", "bfloat16"])
def test_sharded_clipped_step_orchestration(tmp_path, grad_dtype_name):
    """reduce-scatter -> norm exchange -> clip -> shard step -> all-gather on two gloo ranks equals the
    single-process computation on the summed gradient, with the gradient communicated in FP32 (mixed
    precision) and in BF16 (the recipe of Section 3: the sum of the two ranks' BF16 gradients is itself
    rounded to BF16 by the collective, and everything downstream works on that BF16 slice)."""
    world, port = 2, _free_port()
    mp.spawn(_sharded_worker, args=(world, port, str(tmp_path), grad_dtype_name), nprocs=world, join=True)
    sys.path.insert(0, ROOT)
    import oracle
    from paper_2502_20566_b200 import synth
    from paper_2502_20566_b200.dist import wire_bytes
    r = [np.load(tmp_path / f"s{k}.npz") for k in range(world)]
    n = 8 * world * 1500
    per = n // world
    p, _, m, v = synth.adamw_state(n, 88, "cpu")
    assert list(r[0]["phases"]) == ["reduce_scatter", "sqnorm", "norm_exchange", "clip_scale", "step", "all_gather", "end"]
    exact = r[0]["g"].astype(np.float64) + r[1]["g"].astype(np.float64)
    g_sum = np.concatenate([r[k]["shard_g"] for k in range(world)])          # what the collective delivered
    if grad_dtype_name == "float32":
        assert np.array_equal(g_sum, r[0]["g"] + r[1]["g"])
    else:
        # a BF16 value next to the exact sum (8 significant bits), and exactly representable in BF16
        assert np.all(np.abs(g_sum - exact) <= np.abs(exact) * 2.0 ** -8 + 1e-30)
        assert np.array_equal(g_sum.view(np.uint32) & 0xFFFF, np.zeros(n, np.uint32))
        g_sum = (g_sum.view(np.uint32) >> 16).astype(np.uint16)                # BF16 bit patterns for the oracle
    b = {t: wire_bytes(n, world, getattr(torch, t)) for t in ("float32", "bfloat16")}
    assert b["float32"]["reduce_scatter"] == 2 * b["bfloat16"]["reduce_scatter"] == n * 4 // 2
    assert b["float32"]["all_gather"] == b["bfloat16"]["all_gather"] == n * 2 // 2
    assert wire_bytes(n, 1, torch.float32)["reduce_scatter"] == 0
    S = sum(oracle.sqnorm(np.ascontiguousarray(g_sum[k * per:(k + 1) * per])) for k in range(world))
    assert float(r[0]["total"][0]) == S and r[0]["total"].tobytes() == r[1]["total"].tobytes()
    gscale = oracle.clip_scale(S, 1.0 / world, 1.0)
    pb, mb, vb = (synth.bits16(t).copy() for t in (p, m, v))
    oracle.adamw_step(pb, g_sum.copy(), mb, vb, oracle.hparams(**HP), 1234, 7, 0, 0, gscale)
    assert np.array_equal(r[0]["full"], pb) and np.array_equal(r[1]["full"], pb)
    assert np.array_equal(np.concatenate([r[0]["m"], r[1]["m"]]), mb)
    assert np.array_equal(np.concatenate([r[0]["v"], r[1]["v"]]), vb)


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
