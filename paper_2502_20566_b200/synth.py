"""Seeded synthetic inputs shaped like the workloads of the BF16+SR training recipe.

This module only draws numbers and lists shapes.  It contains none of the optimizer's arithmetic
(no rounding rule, no Philox, no AdamW) and is the one module that both the CUDA tests and the
CPU-oracle tests import, so that the two sides always see the same buffers.

All generators are chunk-addressable: a buffer of any length is the concatenation of chunks of
``CHUNK`` elements, chunk ``c`` being drawn from a ``torch.Generator`` seeded by
``(workload seed, role, c)``.  A buffer far larger than host memory can therefore be filled on the
device chunk by chunk, and any chunk can be drawn again later (for example to recover the state
before an in-place update).  CPU and CUDA generators produce different streams; a test draws on
one device and hands the same tensors to both implementations.

BF16 tensors are FP32 samples converted once with torch's round-to-nearest-even cast.
"""

from __future__ import annotations

from dataclasses import dataclass
from typing import Iterator, List, Tuple

import torch

CHUNK = 1 << 26

ROLE_P, ROLE_G, ROLE_M, ROLE_V, ROLE_SRC, ROLE_CLASS = range(6)

_MASK63 = (1 << 63) - 1


def _generator(device, *keys: int) -> torch.Generator:
    s = 0x9E3779B97F4A7C15
    for k in keys:
        s = ((s ^ (int(k) + 0x632BE59BD9B4E019)) * 0xD1342543DE82EF95 + 0x2545F4914F6CDD1D) & _MASK63
    g = torch.Generator(device=device)
    g.manual_seed(s)
    return g


def _normal(n: int, std: float, gen: torch.Generator, device) -> torch.Tensor:
    return torch.randn(n, generator=gen, device=device, dtype=torch.float32) * std


def chunks(n: int, chunk: int = CHUNK) -> Iterator[Tuple[int, int, int]]:
    """Yield (chunk index, start, length) over [0, n)."""
    c = 0
    start = 0
    while start < n:
        length = min(chunk, n - start)
        yield c, start, length
        c += 1
        start += length


# ---------------------------------------------------------------------------------------------
# optimizer state: p ~ N(0, 0.02), g ~ N(0, 1e-3), m ~ N(0, 1e-4), v = N(0, 1e-3)^2
# ---------------------------------------------------------------------------------------------

def state_chunk(role: int, seed: int, chunk_index: int, length: int, device,
                g_dtype: torch.dtype = torch.bfloat16, outlier_fraction: float = 0.0,
                stream_id: int = 0) -> torch.Tensor:
    """One chunk of p, g, m or v.  ``stream_id`` separates tensors of a list / steps of a run."""
    gen = _generator(device, seed, role, chunk_index, stream_id)
    if role == ROLE_P:
        return _normal(length, 0.02, gen, device).to(torch.bfloat16)
    if role == ROLE_M:
        return _normal(length, 1e-4, gen, device).to(torch.bfloat16)
    if role == ROLE_V:
        x = _normal(length, 1e-3, gen, device)
        return (x * x).to(torch.bfloat16)
    if role == ROLE_G:
        x = _normal(length, 1e-3, gen, device)
        if outlier_fraction > 0.0:
            pick = torch.rand(length, generator=gen, device=device) < outlier_fraction
            big = torch.randn(length, generator=gen, device=device, dtype=torch.float32)
            x = torch.where(pick, big, x)
        return x.to(g_dtype)
    raise ValueError("role")


def fill_state(out: torch.Tensor, role: int, seed: int, outlier_fraction: float = 0.0,
               stream_id: int = 0, chunk: int = CHUNK) -> None:
    """Fill a flat tensor in place, chunk by chunk (dtype of ``out`` decides the gradient type)."""
    n = out.numel()
    for c, start, length in chunks(n, chunk):
        out[start:start + length] = state_chunk(role, seed, c, length, out.device, out.dtype,
                                                outlier_fraction, stream_id)


def adamw_state(n: int, seed: int, device, g_dtype: torch.dtype = torch.bfloat16,
                outlier_fraction: float = 0.0):
    """(p, g, m, v) for a flat buffer of n elements."""
    p = torch.empty(n, dtype=torch.bfloat16, device=device)
    g = torch.empty(n, dtype=g_dtype, device=device)
    m = torch.empty(n, dtype=torch.bfloat16, device=device)
    v = torch.empty(n, dtype=torch.bfloat16, device=device)
    fill_state(p, ROLE_P, seed)
    fill_state(g, ROLE_G, seed, outlier_fraction)
    fill_state(m, ROLE_M, seed)
    fill_state(v, ROLE_V, seed)
    return p, g, m, v


# ---------------------------------------------------------------------------------------------
# FP32 mix for the standalone stochastic-rounding cast
# ---------------------------------------------------------------------------------------------

def downcast_mix_chunk(seed: int, chunk_index: int, length: int, device) -> torch.Tensor:
    """FP32 values: 60% N(0,1); 30% log-uniform magnitude in [1e-30, 1e30] with random sign; 2% each
    of signed zeros, FP32 subnormals, values already representable in BF16, values in the last BF16
    interval below FLT_MAX, and infinities / NaNs.  The class of each element is drawn
    independently, so the classes are interleaved."""
    gen = _generator(device, seed, ROLE_SRC, chunk_index)
    cls = torch.rand(length, generator=gen, device=device)
    normal = torch.randn(length, generator=gen, device=device, dtype=torch.float32)
    expo = torch.rand(length, generator=gen, device=device, dtype=torch.float64) * 60.0 - 30.0
    sign_bit = torch.randint(0, 2, (length,), generator=gen, device=device, dtype=torch.int64) << 31
    low = torch.randint(0, 1 << 23, (length,), generator=gen, device=device, dtype=torch.int64)

    def as_f32(bits64: torch.Tensor) -> torch.Tensor:
        b = bits64 & 0xFFFFFFFF
        b = torch.where(b >= (1 << 31), b - (1 << 32), b)
        return b.to(torch.int32).view(torch.float32)

    sign = torch.where(sign_bit != 0, -1.0, 1.0).to(torch.float64)
    loguni = (sign * torch.pow(torch.tensor(10.0, dtype=torch.float64, device=device), expo)).to(torch.float32)
    zeros = as_f32(sign_bit)
    subnormal = as_f32(sign_bit | torch.clamp(low, min=1))
    exact = normal.to(torch.bfloat16).to(torch.float32)
    near_max = as_f32(sign_bit | 0x7F7F0000 | (low & 0xFFFF))
    # a third each: infinity, quiet NaN with a payload, signalling NaN with a payload
    kind = low % 3
    nan_payload = torch.where(kind == 1, 0x400000 | (low >> 2), torch.clamp(low >> 2, min=1) & 0x3FFFFF)
    special = as_f32(sign_bit | 0x7F800000 | torch.where(kind == 0, torch.zeros_like(low), nan_payload))

    out = normal
    out = torch.where(cls >= 0.60, loguni, out)
    out = torch.where(cls >= 0.90, zeros, out)
    out = torch.where(cls >= 0.92, subnormal, out)
    out = torch.where(cls >= 0.94, exact, out)
    out = torch.where(cls >= 0.96, near_max, out)
    out = torch.where(cls >= 0.98, special, out)
    return out


def downcast_mix(n: int, seed: int, device, chunk: int = 1 << 22) -> torch.Tensor:
    out = torch.empty(n, dtype=torch.float32, device=device)
    for c, start, length in chunks(n, chunk):
        out[start:start + length] = downcast_mix_chunk(seed, c, length, device)
    return out


# ---------------------------------------------------------------------------------------------
# parameter lists
# ---------------------------------------------------------------------------------------------

@dataclass(frozen=True)
class TensorSpec:
    name: str
    shape: Tuple[int, ...]
    init: str  # "normal" (N(0, 0.02)), "ones", "zeros"

    @property
    def numel(self) -> int:
        n = 1
        for s in self.shape:
            n *= s
        return n


def gpt2_param_list(layers: int = 24, d: int = 1024, vocab: int = 50257, ctx: int = 1024) -> List[TensorSpec]:
    """GPT-2 style parameter list (350M by default): embeddings, then per layer LN / fused QKV /
    attention projection / LN / MLP up / MLP down with their biases, then the final LN."""
    out = [TensorSpec("wte", (vocab, d), "normal"), TensorSpec("wpe", (ctx, d), "normal")]
    for i in range(layers):
        pre = f"h{i}."
        out += [
            TensorSpec(pre + "ln1.w", (d,), "ones"), TensorSpec(pre + "ln1.b", (d,), "zeros"),
            TensorSpec(pre + "qkv.w", (d, 3 * d), "normal"), TensorSpec(pre + "qkv.b", (3 * d,), "zeros"),
            TensorSpec(pre + "proj.w", (d, d), "normal"), TensorSpec(pre + "proj.b", (d,), "zeros"),
            TensorSpec(pre + "ln2.w", (d,), "ones"), TensorSpec(pre + "ln2.b", (d,), "zeros"),
            TensorSpec(pre + "fc.w", (d, 4 * d), "normal"), TensorSpec(pre + "fc.b", (4 * d,), "zeros"),
            TensorSpec(pre + "mproj.w", (4 * d, d), "normal"), TensorSpec(pre + "mproj.b", (d,), "zeros"),
        ]
    out += [TensorSpec("lnf.w", (d,), "ones"), TensorSpec("lnf.b", (d,), "zeros")]
    return out


def init_param(spec: TensorSpec, seed: int, index: int, device) -> torch.Tensor:
    n = spec.numel
    if spec.init == "ones":
        return torch.ones(n, dtype=torch.bfloat16, device=device)
    if spec.init == "zeros":
        return torch.zeros(n, dtype=torch.bfloat16, device=device)
    out = torch.empty(n, dtype=torch.bfloat16, device=device)
    fill_state(out, ROLE_P, seed, stream_id=index)
    return out


def fresh_grad(spec: TensorSpec, grad_seed: int, step: int, index: int, device,
               dtype: torch.dtype = torch.bfloat16) -> torch.Tensor:
    """g ~ N(0, 1e-3) for tensor ``index`` at iteration ``step``."""
    out = torch.empty(spec.numel, dtype=dtype, device=device)
    fill_state(out, ROLE_G, grad_seed, stream_id=step * 100003 + index)
    return out


def gpt_flat_numel(layers: int = 32, d: int = 4096, vocab: int = 50257, ctx: int = 2048) -> int:
    """Element count of a GPT-style model with ffn = 4d as one flat buffer: per layer 12 d^2 weights
    and 13 d biases/LN entries, token and position embeddings, final LN.  Defaults: the 6.7B model
    (6 658 404 352 elements)."""
    return layers * (12 * d * d + 13 * d) + vocab * d + ctx * d + 2 * d


def bits16(t: torch.Tensor):
    """numpy uint16 view of a CPU BF16 tensor's bit patterns (no copy)."""
    import numpy as np

    return t.detach().view(torch.int16).numpy().view(np.uint16)
