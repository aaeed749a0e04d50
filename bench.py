#!/usr/bin/env python
"""Benchmark of the fused SR-AdamW step (Algorithm 1) on the 6.7B-parameter flat buffer.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One step = one sr_adamw_step call over the whole buffer (6 658 404 352 BF16 elements of x, g, m, v
resident in HBM; 14 algorithmic bytes per element; the call enqueues 25 launches of one kernel).  Prints ONE JSON line: parameters updated per
second over all ranks, the HBM roofline of the kernel, an end-to-end figure with host-resident
state, and the CPU oracle timed on the same box.  With N > 1 (torchrun) every rank steps its own
full replica, as the data-parallel replicas of Algorithm 1 do; there is no collective in the path.
`--impl reference` times the CPU oracle (slow by construction) on a bounded sample per step.
"""

from __future__ import annotations

import argparse
import datetime as _dt
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "SR-AdamW params/sec and achieved HBM GB/s (% of B200 peak) at 6.7B, 1 GPU"
HP = dict(lr=6e-4, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.1)
SEED = 1234
FIRST_STEP = 1000
BYTES_PER_ELEMENT = 14          # read x, g, m, v (4 x 2 B) + write x, m, v (3 x 2 B)
FALLBACK_HBM_GBS = 6650.0       # used only when MEASURED_PEAKS.json is absent
NOMINAL_HBM_GBS = 7700.0        # data-sheet bandwidth of the HGX B200 (context beside the measured-peak fraction)
# DRAM bytes (read + write) of one launch of the headline kernel, from a profiler capture of the SAME kernel
# build and launch shape on a smaller case: (dram bytes read + written, elements of that case).  The traffic of
# a streaming kernel grows in proportion to the element count, so the full-size figure is bytes / elements * n.
# None whenever the kernel has changed since the capture was taken.  Current values: k_sr_adamw_flat_fast (BF16
# gradients, 384 x 1 blocks, 3 stages) on 2^28 elements (the length a flat call is cut into), dram__bytes_read.sum +
# dram__bytes_write.sum of one launch.
NCU_TRAFFIC_CAPTURE = (3_704_089_000, 268_435_456)


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--elements", type=int, default=0, help="override the buffer length (profiling on a small case)")
    ap.add_argument("--elem-offset", type=int, default=0,
                    help="global index of the buffer's first element (profiling the path for offsets that are not multiples of 8)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--e2e-elements", type=int, default=1 << 29)
    ap.add_argument("--no-extras", action="store_true", help="skip the secondary kernels (shard step, tensor list, cast)")
    ap.add_argument("--mode", choices=["replicas", "sharded"], default="replicas",
                    help="replicas: every rank steps its own full buffer (the paper's data parallelism); sharded: "
                         "reduce-scatter -> norm -> clip -> shard step -> all-gather over the ranks (torchrun)")
    ap.add_argument("--sustained-seconds", type=float, default=3.0,
                    help="length of the second timed region (back-to-back launches under the power cap); 0 skips it")
    ap.add_argument("--case", choices=EXTRA_CASES, default=None,
                    help="run one secondary call alone (with --elements: on a small case) instead of the headline step")
    return ap.parse_args()


# ---------------------------------------------------------------------------------------------
# clocks
# ---------------------------------------------------------------------------------------------

_SMI_FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
               "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
               "clocks_event_reasons.sw_power_cap")


class ClockSampler:
    """nvidia-smi polled in the background; samples are cut to the timed region afterwards."""

    def __init__(self, torch, device_index: int):
        self.proc = None
        self.path = None
        try:
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            f = tempfile.NamedTemporaryFile(prefix="clocks_", suffix=".csv", delete=False)
            self.path = f.name
            self.proc = subprocess.Popen(["nvidia-smi", "-i", uuid, f"--query-gpu={_SMI_FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "50"], stdout=f, stderr=subprocess.DEVNULL)
            f.close()
        except Exception:
            self.proc = None

    def stop(self) -> None:
        """End the poller and read its samples; `window` then cuts them to a timed region."""
        self.rows = []
        if self.proc is None:
            return
        time.sleep(0.12)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        try:
            with open(self.path) as f:
                for line in f:
                    parts = [x.strip() for x in line.split(",")]
                    if len(parts) != 8:
                        continue
                    try:
                        ts = _dt.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f")
                        self.rows.append((ts, float(parts[1]), float(parts[2]), float(parts[3]), parts[4:8]))
                    except ValueError:
                        continue
            os.unlink(self.path)
        except OSError:
            pass

    def window(self, t0: _dt.datetime, t1: _dt.datetime) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        rows = getattr(self, "rows", [])
        inside = [r for r in rows if t0 <= r[0] <= t1] or rows[-3:]
        if not inside:
            return out
        out["samples"] = len(inside)
        out["sm_mhz"] = statistics.median(r[1] for r in inside)
        out["sm_max_mhz"] = max(r[2] for r in inside)
        out["power_w_max"] = max(r[3] for r in inside)
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        out["reasons"] = [n for i, n in enumerate(names) if any(r[4][i].lower().startswith("active") for r in inside)]
        return out


# ---------------------------------------------------------------------------------------------
# CPU oracle legs
# ---------------------------------------------------------------------------------------------

def _oracle_sample(synth, torch, elements: int):
    import numpy as np
    p, g, m, v = synth.adamw_state(elements, SEED, "cpu")
    return [synth.bits16(t).copy() for t in (p, g, m, v)]


def time_oracle(sample_elements: int, budget_s: float = 15.0):
    """Oracle timed as it stands (OpenMP over elements) on `sample_elements` of the workload."""
    import torch
    import oracle
    from paper_2502_20566_b200 import synth
    arrs = _oracle_sample(synth, torch, sample_elements)
    hp = oracle.hparams(**HP)
    oracle.adamw_step(*[a[:1 << 16].copy() for a in arrs], hp, SEED, FIRST_STEP)      # load + warm
    times = []
    t_all = time.perf_counter()
    rep = 0
    while rep < 16 and (rep < 1 or time.perf_counter() - t_all < budget_s):   # about 13 s on 16 cores
        t0 = time.perf_counter()
        oracle.adamw_step(*arrs, hp, SEED, FIRST_STEP + rep)
        times.append(time.perf_counter() - t0)
        rep += 1
    mean = sum(times) / len(times)
    return {"value": sample_elements / mean, "unit": "params/s", "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"{len(times)} x sr_adamw_step on the first {sample_elements} elements of the workload "
                      f"(same distributions, step {FIRST_STEP}+), OpenMP threads = cores"}


def run_reference(args):
    """The reference arm: the CPU oracle, one bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import torch
    import oracle
    from paper_2502_20566_b200 import synth
    sample = 1 << 27
    arrs = _oracle_sample(synth, torch, sample)
    hp = oracle.hparams(**HP)
    for w in range(args.warmup):
        oracle.adamw_step(*arrs, hp, SEED, FIRST_STEP + w)
    t0 = time.perf_counter()
    for k in range(args.steps):
        oracle.adamw_step(*arrs, hp, SEED, FIRST_STEP + args.warmup + k)
    dt = time.perf_counter() - t0
    value = sample * args.steps / dt
    n = args.elements or synth.gpt_flat_numel()
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "params/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"6.7B flat buffer ({n} elements, bf16 x/g/m/v, step {FIRST_STEP}); each step runs "
                               f"the CPU oracle on a {sample}-element sample of it"},
        "cpu_baseline": {"value": value, "unit": "params/s", "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": f"{sample} elements per step"},
        "e2e": {"value": value, "unit": "params/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------------
# CUDA arm
# ---------------------------------------------------------------------------------------------

EXTRA_CASES = ("shard_fp32_grads", "fp32_master_recipe", "tensor_list", "tensor_list_6p7b", "offset_not_multiple_of_8",
               "cast_bf16", "cast_fp8", "cast_fp4", "accumulate")


def time_extras(torch, binding, synth, dev, peak, only=None, elements=0, reps=10, warmup=3):
    """The other calls of the library, each timed alone (half a second of idle, then CUDA events around
    3 warm-ups + 10 launches) on its own workload; bytes are the algorithmic ones.  Reported beside the headline, not part of it.
    `only` names one case of EXTRA_CASES (the others are skipped) and `elements` shrinks its buffers:
    the small single-kernel runs that profiler captures are taken on."""
    stream = torch.cuda.current_stream()
    want = lambda *cases: only is None or only in cases

    def timed(fn, reps=reps):
        torch.cuda.synchronize()
        time.sleep(0.5)          # every case starts from an idle GPU, like the headline's first timed region
        for _ in range(warmup):
            fn()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record(stream)
        for _ in range(reps):
            fn()
        b.record(stream)
        torch.cuda.synchronize()
        return a.elapsed_time(b) / reps

    out = {}
    if want("shard_fp32_grads", "fp32_master_recipe"):
        _extras_shard(torch, binding, synth, dev, peak, timed, out, want, elements)
    if want("offset_not_multiple_of_8"):
        _extras_offset(torch, binding, synth, dev, peak, timed, out, elements)
    if want("tensor_list"):
        _extras_list(torch, binding, synth, dev, peak, timed, out, compare_flat=only is None)
    if want("tensor_list_6p7b"):
        _extras_list_6p7b(torch, binding, synth, dev, peak, timed, out)
    if want("cast_bf16", "cast_fp8", "cast_fp4"):
        _extras_casts(torch, binding, synth, dev, peak, timed, out, want, elements)
    if want("accumulate"):
        _extras_accumulate(torch, binding, synth, dev, peak, timed, out, elements)
    return out


def _extras_shard(torch, binding, synth, dev, peak, timed, out, want, elements):
    # 1/8 shard with FP32 gradients: squared norm -> clip factor -> step (20 B per element over two passes)
    n = elements or synth.gpt_flat_numel() // 8
    p, g, m, v = synth.adamw_state(n, SEED, dev, g_dtype=torch.float32, outlier_fraction=0.01)
    if want("shard_fp32_grads"):
        _extras_shard_sr(torch, binding, dev, peak, timed, out, n, p, g, m, v)
    del p, m, v
    if want("fp32_master_recipe"):
        _extras_master(torch, binding, synth, dev, peak, timed, out, n, g)
    out.pop("sr_step_ms_same_shard", None)


def _extras_shard_sr(torch, binding, dev, peak, timed, out, n, p, g, m, v):
    ws = torch.empty(max(1, binding.grad_sqnorm_workspace_bytes(n) // 8), dtype=torch.float64, device=dev)
    S = torch.zeros(1, dtype=torch.float64, device=dev)
    gs = torch.zeros(1, dtype=torch.float32, device=dev)
    hp_clip = binding.hparams(**HP, grad_scale_dev=gs)
    t_norm = timed(lambda: binding.grad_sqnorm(g, S, ws))
    t_step = timed(lambda: binding.sr_adamw_step(p, g, m, v, hp_clip, SEED, FIRST_STEP, 0, 3 * n))

    def clipped():
        binding.grad_sqnorm(g, S, ws)
        binding.sr_clip_scale(S, 0.125, 1.0, gs)
        binding.sr_adamw_step(p, g, m, v, hp_clip, SEED, FIRST_STEP, 0, 3 * n)
    t_all = timed(clipped)
    out["sr_step_ms_same_shard"] = t_step
    out["shard_fp32_grads"] = {
        "elements": n,
        "grad_sqnorm": {"ms": t_norm, "gbs": 4 * n / t_norm / 1e6, "frac": 4 * n / t_norm / 1e6 / peak},
        "sr_adamw_step_f32g": {"ms": t_step, "gbs": 16 * n / t_step / 1e6, "frac": 16 * n / t_step / 1e6 / peak},
        "norm_clip_step": {"ms": t_all, "params_per_s": n / t_all * 1e3, "gbs": 20 * n / t_all / 1e6,
                           "frac": 20 * n / t_all / 1e6 / peak},
    }


def _extras_master(torch, binding, synth, dev, peak, timed, out, n, g):
    # the mixed-precision comparison recipe on the same shard: FP32 master weights and moments + BF16 copy
    p32, m32, v32 = (torch.empty(n, dtype=torch.float32, device=dev) for _ in range(3))
    for t, role in ((p32, synth.ROLE_P), (m32, synth.ROLE_M), (v32, synth.ROLE_V)):
        for c, start, length in synth.chunks(n):
            t[start:start + length] = synth.state_chunk(role, SEED, c, length, dev).float()
    p16 = torch.empty(n, dtype=torch.bfloat16, device=dev)
    hp_plain = binding.hparams(**HP)
    t_mp = timed(lambda: binding.sr_master_adamw_step(p32, p16, g, m32, v32, hp_plain, FIRST_STEP))
    out["fp32_master_recipe_same_shard"] = {
        "elements": n, "bytes_per_element": 30, "ms": t_mp, "params_per_s": n / t_mp * 1e3, "gbs": 30 * n / t_mp / 1e6,
        "frac": 30 * n / t_mp / 1e6 / peak, "state_bytes_per_param": 14, "sr_state_bytes_per_param": 6,
        "time_vs_sr_step": t_mp / out["sr_step_ms_same_shard"] if "sr_step_ms_same_shard" in out else None}


def _extras_list(torch, binding, synth, dev, peak, timed, out, compare_flat):
    # GPT-2 350M tensor list, one launch per step
    specs = synth.gpt2_param_list()
    P = [synth.init_param(sp, SEED, i, dev) for i, sp in enumerate(specs)]
    G = [synth.fresh_grad(sp, 4321, 1, i, dev) for i, sp in enumerate(specs)]
    M = [torch.zeros_like(t) for t in P]
    V = [torch.zeros_like(t) for t in P]
    plan = binding.sr_mt_plan_create(P, G, M, V)
    hp = binding.hparams(**HP)
    step = [0]

    def mt():
        step[0] += 1
        binding.sr_adamw_multi_tensor(plan, hp, SEED, step[0])
    t_mt = timed(mt)
    ne = plan.total_elements
    out["tensor_list_gpt2_350m"] = {"tensors": len(specs), "elements": ne, "ms": t_mt, "params_per_s": ne / t_mt * 1e3,
                                    "gbs": 14 * ne / t_mt / 1e6, "frac": 14 * ne / t_mt / 1e6 / peak}
    # global-norm clipping of the whole list on the device: list norm -> clip factor -> step (16 B per element)
    ws = torch.empty(max(1, binding.grad_sqnorm_multi_tensor_workspace_bytes(plan) // 8), dtype=torch.float64, device=dev)
    S = torch.zeros(1, dtype=torch.float64, device=dev)
    gs = torch.zeros(1, dtype=torch.float32, device=dev)
    hp_clip = binding.hparams(**HP, grad_scale_dev=gs)
    t_norm = timed(lambda: binding.grad_sqnorm_multi_tensor(plan, S, ws))

    def clipped():
        step[0] += 1
        binding.grad_sqnorm_multi_tensor(plan, S, ws)
        binding.sr_clip_scale(S, 1.0, 1.0, gs)
        binding.sr_adamw_multi_tensor(plan, hp_clip, SEED, step[0])
    t_clip = timed(clipped)
    out["tensor_list_gpt2_350m"]["grad_sqnorm_multi_tensor"] = {"ms": t_norm, "gbs": 2 * ne / t_norm / 1e6,
                                                                "frac": 2 * ne / t_norm / 1e6 / peak}
    out["tensor_list_gpt2_350m"]["norm_clip_step"] = {"ms": t_clip, "params_per_s": ne / t_clip * 1e3,
                                                      "gbs": 16 * ne / t_clip / 1e6, "frac": 16 * ne / t_clip / 1e6 / peak}
    plan.destroy()
    del P, G, M, V
    if not compare_flat:
        return
    # the flat kernel on a buffer of the same length, for comparison with the list launch
    fp, fg, fm, fv = synth.adamw_state(ne, SEED, dev)
    t_f = timed(lambda: binding.sr_adamw_step(fp, fg, fm, fv, hp, SEED, FIRST_STEP))
    out["flat_same_length_as_list"] = {"elements": ne, "ms": t_f, "gbs": 14 * ne / t_f / 1e6, "frac": 14 * ne / t_f / 1e6 / peak}


def _extras_offset(torch, binding, synth, dev, peak, timed, out, elements):
    # the 1/8 shard (BF16 gradients) placed at a global offset that is 3 modulo 8: every 16-byte vector then
    # straddles two noise groups; beside it the cast and the accumulation at the same offset
    n = elements or synth.gpt_flat_numel() // 8
    p, g, m, v = synth.adamw_state(n, SEED, dev)
    hp = binding.hparams(**HP)
    off = 3 * n + 3
    step = [FIRST_STEP]

    def one(offset):
        step[0] += 1
        binding.sr_adamw_step(p, g, m, v, hp, SEED, step[0], 0, offset)
    t_al = timed(lambda: one(3 * n))
    t_off = timed(lambda: one(off))
    res = {"elements": n, "elem_offset": off,
           "sr_adamw_step": {"ms": t_off, "gbs": 14 * n / t_off / 1e6, "frac": 14 * n / t_off / 1e6 / peak,
                             "ms_at_aligned_offset": t_al, "frac_at_aligned_offset": 14 * n / t_al / 1e6 / peak}}

    def acc():
        step[0] += 1
        binding.sr_accumulate_bf16(m, g, 0.125, SEED, step[0], 0, off)
    t_a = timed(acc)
    res["sr_accumulate_bf16"] = {"ms": t_a, "gbs": 6 * n / t_a / 1e6, "frac": 6 * n / t_a / 1e6 / peak}
    del p, m, v
    nc = min(n, 1 << 28)
    src = synth.downcast_mix(nc, 7, dev)
    dst = torch.empty(nc, dtype=torch.bfloat16, device=dev)
    t_c = timed(lambda: binding.sr_downcast_f32_bf16(src, dst, seed=7, elem_offset=off))
    res["sr_downcast_f32_bf16"] = {"elements": nc, "ms": t_c, "gbs": 6 * nc / t_c / 1e6, "frac": 6 * nc / t_c / 1e6 / peak}
    out["flat_offset_not_multiple_of_8"] = res


def _extras_list_6p7b(torch, binding, synth, dev, peak, timed, out):
    # the 6.7B model as a tensor list (388 tensors, each its own allocation; same element count as the flat buffer):
    # one sr_adamw_multi_tensor launch per step, and the list norm
    specs = synth.gpt2_param_list(layers=32, d=4096, vocab=50257, ctx=2048)
    P = [synth.init_param(sp, SEED, i, dev) for i, sp in enumerate(specs)]
    G = [synth.fresh_grad(sp, 4321, 1, i, dev) for i, sp in enumerate(specs)]
    M, V = [], []
    for i, sp in enumerate(specs):
        mm = torch.empty(sp.numel, dtype=torch.bfloat16, device=dev)
        vv = torch.empty(sp.numel, dtype=torch.bfloat16, device=dev)
        synth.fill_state(mm, synth.ROLE_M, SEED, stream_id=i)
        synth.fill_state(vv, synth.ROLE_V, SEED, stream_id=i)
        M.append(mm)
        V.append(vv)
    plan = binding.sr_mt_plan_create(P, G, M, V)
    hp = binding.hparams(**HP)
    step = [FIRST_STEP]

    def mt():
        step[0] += 1
        binding.sr_adamw_multi_tensor(plan, hp, SEED, step[0])
    t_mt = timed(mt)
    ne = plan.total_elements
    ws = torch.empty(max(1, binding.grad_sqnorm_multi_tensor_workspace_bytes(plan) // 8), dtype=torch.float64, device=dev)
    S = torch.zeros(1, dtype=torch.float64, device=dev)
    t_norm = timed(lambda: binding.grad_sqnorm_multi_tensor(plan, S, ws))
    out["tensor_list_6p7b"] = {"tensors": len(specs), "elements": ne, "ms": t_mt, "params_per_s": ne / t_mt * 1e3,
                               "gbs": 14 * ne / t_mt / 1e6, "frac": 14 * ne / t_mt / 1e6 / peak,
                               "grad_sqnorm_multi_tensor": {"ms": t_norm, "gbs": 2 * ne / t_norm / 1e6,
                                                            "frac": 2 * ne / t_norm / 1e6 / peak}}
    plan.destroy()


def _extras_casts(torch, binding, synth, dev, peak, timed, out, want, elements):
    # standalone stochastic-rounding casts of 2^28 FP32 values: BF16 (6 B per element), FP8 (5 B per element)
    nc = elements or 1 << 28
    src = synth.downcast_mix(nc, 7, dev)
    if want("cast_bf16"):
        dst = torch.empty(nc, dtype=torch.bfloat16, device=dev)
        t_c = timed(lambda: binding.sr_downcast_f32_bf16(src, dst, seed=7))
        out["sr_downcast_f32_bf16"] = {"elements": nc, "ms": t_c, "params_per_s": nc / t_c * 1e3,
                                       "gbs": 6 * nc / t_c / 1e6, "frac": 6 * nc / t_c / 1e6 / peak}
    if want("cast_fp8"):
        dst8 = torch.empty(nc, dtype=torch.uint8, device=dev).view(torch.float8_e4m3fn)
        t_8 = timed(lambda: binding.sr_downcast_f32_fp8(src, dst8, seed=7))
        out["sr_downcast_f32_fp8_e4m3"] = {"elements": nc, "ms": t_8, "params_per_s": nc / t_8 * 1e3,
                                           "gbs": 5 * nc / t_8 / 1e6, "frac": 5 * nc / t_8 / 1e6 / peak, "bound": "alu"}
    if want("cast_fp4"):
        dst4 = torch.empty(nc // 2, dtype=torch.uint8, device=dev)
        t_4 = timed(lambda: binding.sr_downcast_f32_fp4(src, dst4, seed=7))
        out["sr_downcast_f32_fp4_e2m1"] = {"elements": nc, "ms": t_4, "params_per_s": nc / t_4 * 1e3,
                                           "gbs": 4.5 * nc / t_4 / 1e6, "frac": 4.5 * nc / t_4 / 1e6 / peak, "bound": "alu"}


def _extras_accumulate(torch, binding, synth, dev, peak, timed, out, elements):
    # BF16 accumulator += BF16 term with stochastic rounding (6 B per element), on the 1/8 shard
    n = elements or synth.gpt_flat_numel() // 8
    _, g, acc, _ = synth.adamw_state(n, SEED, dev)
    step = [0]

    def accumulate():
        step[0] += 1
        binding.sr_accumulate_bf16(acc, g, 0.125, SEED, step[0])
    t_a = timed(accumulate)
    out["sr_accumulate_bf16"] = {"elements": n, "ms": t_a, "params_per_s": n / t_a * 1e3, "gbs": 6 * n / t_a / 1e6,
                                 "frac": 6 * n / t_a / 1e6 / peak}


def time_zero_cases(torch, binding, synth, bufs, hp, stream, reps=10, warmup=3):
    """Headline launch on the 6.7B buffers with (i) a tenth of the 1024-element rows holding zero gradient and zero
    moments, (ii) a zero gradient everywhere with the usual state, (iii) everything zero.  Leaves the buffers modified."""
    p, g, m, v = bufs
    n = p.numel()
    rows = n // 1024
    step = [FIRST_STEP + 10000]

    def timed():
        def one():
            step[0] += 1
            binding.sr_adamw_step(p, g, m, v, hp, SEED, step[0])
        for _ in range(warmup):
            one()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record(stream)
        for _ in range(reps):
            one()
        b.record(stream)
        torch.cuda.synchronize()
        return a.elapsed_time(b) / reps

    out = {}
    for t, role in zip(bufs, (synth.ROLE_P, synth.ROLE_G, synth.ROLE_M, synth.ROLE_V)):
        synth.fill_state(t, role, SEED)
    mask = torch.rand(rows, device=p.device, generator=torch.Generator(device=p.device).manual_seed(5)) < 0.10
    for t in (g, m, v):
        t[:rows * 1024].view(rows, 1024)[mask] = 0
    out["tenth_of_rows_zero_g_m_v"] = {"ms": timed()}
    for t, role in zip((m, v), (synth.ROLE_M, synth.ROLE_V)):
        synth.fill_state(t, role, SEED)
    g.zero_()
    out["zero_gradient"] = {"ms": timed()}
    for t in bufs:
        t.zero_()
    out["all_zero"] = {"ms": timed()}
    return out


def hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json, copy kernel)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (earlier measurement on this pool)"


def run_ours(args):
    import torch
    from paper_2502_20566_b200 import binding, synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    binding.lib()

    if args.case:   # one secondary call alone: the run a profiler capture of that kernel is taken on
        peak, peak_src = hbm_peak()
        res = time_extras(torch, binding, synth, dev, peak, only=args.case, elements=args.elements,
                          reps=args.steps, warmup=args.warmup)
        print(json.dumps({"case": args.case, "steps": args.steps, "warmup": args.warmup, "peak": peak,
                          "peak_source": peak_src, "result": res}), flush=True)
        return

    n = args.elements or synth.gpt_flat_numel()
    bufs = [torch.empty(n, dtype=torch.bfloat16, device=dev) for _ in range(4)]
    for t, role in zip(bufs, (synth.ROLE_P, synth.ROLE_G, synth.ROLE_M, synth.ROLE_V)):
        synth.fill_state(t, role, SEED)
    p, g, m, v = bufs
    hp = binding.hparams(**HP)
    stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    for w in range(args.warmup):
        binding.sr_adamw_step(p, g, m, v, hp, SEED, FIRST_STEP + w, 0, args.elem_offset)
    sampler = ClockSampler(torch, local) if rank == 0 and not os.environ.get("SRADAMW_NO_CLOCK_SAMPLER") else None
    if sampler is not None:
        time.sleep(0.3)          # let the poller start
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    barrier()
    t_begin = _dt.datetime.now()
    for k in range(args.steps):
        ev[k][0].record(stream)
        binding.sr_adamw_step(p, g, m, v, hp, SEED, FIRST_STEP + args.warmup + k, 0, args.elem_offset)
        ev[k][1].record(stream)
    barrier()
    t_end = _dt.datetime.now()
    total_ms = ev[0][0].elapsed_time(ev[-1][1])
    launch_ms = [a.elapsed_time(b) for a, b in ev]

    # second timed region: back-to-back launches for some seconds, long enough for the board to settle on its
    # power cap (the first region is over before it does); same call, same buffers, its own clock window
    sustained = None
    if args.sustained_seconds > 0 and world == 1 and not args.elements:
        reps = max(args.steps, int(args.sustained_seconds * 1e3 / (sum(launch_ms) / len(launch_ms))) + 1)
        sev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
        torch.cuda.synchronize()
        ts0 = _dt.datetime.now()
        for k in range(reps):
            sev[k][0].record(stream)
            binding.sr_adamw_step(p, g, m, v, hp, SEED, FIRST_STEP + args.warmup + args.steps + k)
            sev[k][1].record(stream)
        torch.cuda.synchronize()
        ts1 = _dt.datetime.now()
        sms = [a.elapsed_time(b) for a, b in sev]
        sustained = {"steps": reps, "seconds": sev[0][0].elapsed_time(sev[-1][1]) * 1e-3, "step_ms_avg": sum(sms) / reps,
                     "step_ms_last_quarter": sum(sms[-(reps // 4):]) / (reps // 4), "window": (ts0, ts1)}
    if sampler is not None:
        sampler.stop()
    clocks = sampler.window(t_begin, t_end) if sampler is not None else None
    if sustained is not None:
        w0, w1 = sustained.pop("window")
        sustained["clocks"] = sampler.window(w0, w1) if sampler is not None else None
    if dist is not None:
        tt = torch.tensor([total_ms], dtype=torch.float64, device=dev)
        dist.all_reduce(tt, op=dist.ReduceOp.MAX)
        total_ms = float(tt.item())

    # end to end: state in pinned host memory, staged through the device by sr_adamw_step_host
    e2e = None
    if not args.no_e2e:
        e = min(args.e2e_elements, n)
        chunk = 1 << 24
        host = [t[:e].cpu().pin_memory() for t in bufs]
        staging = torch.empty(binding.sr_adamw_step_host_staging_bytes(torch.bfloat16, chunk), dtype=torch.uint8, device=dev)
        reps = max(1, min(args.steps, 5))
        binding.sr_adamw_step_host(host[0], host[1], host[2], host[3], hp, SEED, 1, staging, chunk)
        barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for k in range(reps):
            binding.sr_adamw_step_host(host[0], host[1], host[2], host[3], hp, SEED, 2 + k, staging, chunk)
        b.record(stream)
        barrier()
        e2e_ms = a.elapsed_time(b)
        checksum = int(host[0][:1024].view(torch.int16).sum())      # the result is read on the host
        if dist is not None:
            tt = torch.tensor([e2e_ms], dtype=torch.float64, device=dev)
            dist.all_reduce(tt, op=dist.ReduceOp.MAX)
            e2e_ms = float(tt.item())
        e2e = {"value": world * e * reps / (e2e_ms * 1e-3), "unit": "params/s", "h2d_bytes_per_step": 8 * e,
               "d2h_bytes_per_step": 6 * e, "steps": reps, "ms_per_step": e2e_ms / reps,
               "sample": f"sr_adamw_step_host on {e} elements per rank held in pinned host memory "
                         f"(x, g, m, v up, x, m, v down every step; {chunk}-element chunks, two streams)",
               "host_checksum": checksum}
        del host, staging

    # the same launch on buffers with exact zeros (rows of 1024 elements): the cases in which the kernel's
    # branch-free arithmetic used to hand vectors to its reference path
    zero_cases = None
    if world == 1 and not args.no_extras and not args.elements:
        zero_cases = time_zero_cases(torch, binding, synth, bufs, hp, stream)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peak, peak_src = hbm_peak()
    # one call = launches_per_step launches of the same kernel back to back (the library cuts a flat call into launches
    # of 2^28 elements); the events bracket the call, so the per-launch figures below include the gaps between them
    launches_per_step = binding.sr_adamw_step_launch_count(n, args.elem_offset)
    avg_launch_ms = sum(launch_ms) / len(launch_ms)
    achieved = BYTES_PER_ELEMENT * n / (avg_launch_ms * 1e-3) / 1e9
    gbs = lambda ms: BYTES_PER_ELEMENT * n / (ms * 1e-3) / 1e9
    if sustained is not None:
        sustained.update(achieved=gbs(sustained["step_ms_avg"]), frac=gbs(sustained["step_ms_avg"]) / peak,
                         achieved_last_quarter=gbs(sustained["step_ms_last_quarter"]),
                         frac_last_quarter=gbs(sustained["step_ms_last_quarter"]) / peak, unit="GB/s")
    if zero_cases is not None:
        for c in zero_cases.values():
            c.update(gbs=gbs(c["ms"]), frac=gbs(c["ms"]) / peak)
    line = {
        "metric": METRIC,
        "value": world * n * args.steps / (total_ms * 1e-3),
        "unit": "params/s",
        "n_gpus": world,
        "steps": args.steps,
        "warmup": args.warmup,
        "ms_per_step": total_ms / args.steps,
        "higher_is_better": True,
        "scaling": "weak",
        "vs_baseline": None,
        "dtype": "f32",
        "data": "synthetic",
        "config": {
            "workload": f"6.7B flat buffer: {n} elements, bf16 x/g/m/v resident in HBM ({8 * n / 1e9:.1f} GB), "
                        f"one sr_adamw_step per step at step {FIRST_STEP}+, SR on x, m, v",
            "elements": n, "bytes_per_element": BYTES_PER_ELEMENT,
            "l2": "buffers are far larger than the 126 MB L2; no flush between iterations",
            "replicas": world,
        },
        "hbm_gbs": achieved,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": (NCU_TRAFFIC_CAPTURE[0] / NCU_TRAFFIC_CAPTURE[1] * n if NCU_TRAFFIC_CAPTURE else None),
                     "peak_source": peak_src, "frac_nominal": achieved / NOMINAL_HBM_GBS, "nominal_gbs": NOMINAL_HBM_GBS,
                     "kernel": "k_sr_adamw_flat_fast", "launches_per_step": launches_per_step,
                     "step_ms_avg": avg_launch_ms, "step_ms_min": min(launch_ms), "step_ms_median": statistics.median(launch_ms),
                     "launch_ms_avg": avg_launch_ms / launches_per_step,
                     "algorithmic_bytes_per_step": BYTES_PER_ELEMENT * n,
                     "algorithmic_bytes_per_launch": BYTES_PER_ELEMENT * n / launches_per_step,
                     "sustained": sustained},
        "gpu_launches": args.steps * launches_per_step,
        "clocks": clocks,
    }
    if e2e is not None:
        line["e2e"] = e2e
    if zero_cases is not None:
        line["zero_cases"] = zero_cases
    del bufs, p, g, m, v
    torch.cuda.empty_cache()
    if world == 1 and not args.no_extras and not args.elements:
        line["extras"] = time_extras(torch, binding, synth, dev, peak)
        torch.cuda.empty_cache()
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = time_oracle(1 << 28)
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()



# ---------------------------------------------------------------------------------------------
# sharded arm (ZeRO-1 shape): reduce-scatter -> norm -> clip -> shard step -> all-gather
# ---------------------------------------------------------------------------------------------

SHARDED_METRIC = "sharded SR-AdamW iteration (reduce-scatter, global-norm clip, shard step, all-gather) params/sec"
PHASES = ("reduce_scatter", "sqnorm", "norm_exchange", "clip_scale", "step", "all_gather")


def run_sharded(args):
    """One optimizer iteration with the optimizer state sharded over the ranks, timed phase by phase with the
    gradient communicated in BF16 (the recipe of Section 3) and in FP32 (mixed precision).  The collectives are
    plain NCCL calls through torch.distributed; every arithmetic step is a call of the library.  With one rank
    the collectives are copies; the arm exists so that a multi-GPU node measures the real thing."""
    import torch
    import torch.distributed as dist
    from paper_2502_20566_b200 import binding, synth
    from paper_2502_20566_b200 import dist as srdist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (there is no CPU fallback)")
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29555")
    # the communicator's own account of what it uses (rings / trees / NVLS), kept out of stdout
    nccl_log = os.path.join(tempfile.gettempdir(), f"sradamw_nccl_rank{rank}.log")
    if os.environ.get("NCCL_DEBUG", "VERSION").upper() in ("VERSION", "WARN"):      # the box presets VERSION
        os.environ["NCCL_DEBUG"] = "INFO"
    os.environ.setdefault("NCCL_DEBUG_FILE", nccl_log)
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist.init_process_group("nccl", rank=rank, world_size=world, device_id=dev)
    binding.lib()
    n = args.elements or synth.gpt_flat_numel()
    n -= n % (8 * world)
    per = n // world
    stream = torch.cuda.current_stream()
    results = {}
    for gname, gdtype in (("bf16", torch.bfloat16), ("fp32", torch.float32)):
        full_p = torch.empty(n, dtype=torch.bfloat16, device=dev)
        synth.fill_state(full_p, synth.ROLE_P, SEED)
        full_g = torch.empty(n, dtype=gdtype, device=dev)
        synth.fill_state(full_g, synth.ROLE_G, SEED + 100 * (rank + 1))          # every rank its own local gradient
        shard_p = full_p[rank * per:(rank + 1) * per].clone()
        shard_m = torch.empty(per, dtype=torch.bfloat16, device=dev)
        shard_v = torch.empty(per, dtype=torch.bfloat16, device=dev)
        synth.fill_state(shard_m, synth.ROLE_M, SEED, stream_id=rank)
        synth.fill_state(shard_v, synth.ROLE_V, SEED, stream_id=rank)
        shard_g = torch.empty(per, dtype=gdtype, device=dev)
        marks = []

        def hook(name):
            e = torch.cuda.Event(enable_timing=True)
            e.record(stream)
            marks.append((name, e))

        def iteration(k):
            srdist.sharded_clipped_step(shard_p, shard_m, shard_v, full_g, HP, SEED, FIRST_STEP + k, max_norm=1.0,
                                        accum_scale=1.0 / world, full_param_out=full_p, phase_hook=hook,
                                        shard_grad_out=shard_g)

        for w in range(args.warmup):
            iteration(w)
        torch.cuda.synchronize()
        dist.barrier()
        torch.cuda.synchronize()
        marks.clear()
        for k in range(args.steps):
            iteration(args.warmup + k)
        torch.cuda.synchronize()
        dist.barrier()
        torch.cuda.synchronize()
        per_iter = len(PHASES) + 1
        assert len(marks) == per_iter * args.steps
        total_ms = marks[0][1].elapsed_time(marks[-1][1])
        phase_ms = {ph: 0.0 for ph in PHASES}
        for k in range(args.steps):
            row = marks[k * per_iter:(k + 1) * per_iter]
            for (name, e0), (_, e1) in zip(row[:-1], row[1:]):
                phase_ms[name] += e0.elapsed_time(e1) / args.steps
        vals = torch.tensor([total_ms] + [phase_ms[ph] for ph in PHASES], dtype=torch.float64, device=dev)
        dist.all_reduce(vals, op=dist.ReduceOp.MAX)
        vals = vals.tolist()
        total_ms = vals[0]
        wire = srdist.wire_bytes(n, world, gdtype)
        results[gname] = {"ms_per_step": total_ms / args.steps, "params_per_s": n * args.steps / (total_ms * 1e-3),
                          "phase_ms": dict(zip(PHASES, vals[1:])), "wire_bytes_per_rank": wire,
                          "hbm_bytes_per_shard_element": {"sqnorm": wire["grad_bytes_per_element"],
                                                          "step": 12 + wire["grad_bytes_per_element"]}}
        del full_p, full_g, shard_p, shard_m, shard_v, shard_g
        torch.cuda.empty_cache()
    if rank == 0:
        nvls = None
        try:
            with open(os.environ["NCCL_DEBUG_FILE"]) as f:
                text = f.read()
            nvls = "NVLS" in text
        except OSError:
            pass
        rec = results["bf16"]
        line = {"metric": SHARDED_METRIC, "mode": "sharded", "value": rec["params_per_s"], "unit": "params/s",
                "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": rec["ms_per_step"],
                "higher_is_better": True, "scaling": "strong", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": {"workload": f"6.7B flat buffer sharded over {world} rank(s): {n} elements, {per} per rank; "
                                       "gradient reduce-scatter in BF16 (value) and in FP32 (beside it), FP64 norm exchange in "
                                       "rank order, clip to norm 1, shard step at elem_offset = rank * n / R, BF16 all-gather",
                           "elements": n, "per_rank": per},
                "gradient_communication": results,
                "reduce_scatter_bytes_bf16_over_fp32": (results["bf16"]["wire_bytes_per_rank"]["reduce_scatter"]
                                                        / results["fp32"]["wire_bytes_per_rank"]["reduce_scatter"]
                                                        if world > 1 else None),
                "nccl": {"debug": os.environ.get("NCCL_DEBUG"), "debug_file": os.environ["NCCL_DEBUG_FILE"], "nvls_in_log": nvls},
                "gpu_launches": args.steps * 4 * 2}
        print(json.dumps(line), flush=True)
    dist.destroy_process_group()


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.mode == "sharded":
        run_sharded(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
