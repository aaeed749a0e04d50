"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle, bit for bit on
the same seeded inputs.  Tolerance: 0 mismatching BF16 patterns, exact FP64 norm, exact FP32 scale."""

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

HP = dict(lr=6e-4, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.1)


@pytest.fixture(scope="module")
def env():
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    import oracle
    from paper_2502_20566_b200 import binding, synth
    binding.lib()   # raises if the CUDA library is missing: no fallback
    return oracle, binding, synth, torch.device("cuda", 0)


def bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().view(torch.int16).cpu().numpy().view(np.uint16).copy()


def host_g(g: torch.Tensor) -> np.ndarray:
    return g.cpu().numpy().copy() if g.dtype == torch.float32 else bits(g)


def mismatches(a: np.ndarray, b: np.ndarray) -> int:
    return int(np.count_nonzero(a != b))


def run_both(env, p, g, m, v, hp_kw, seed, step, tensor_id=0, elem_offset=0, gscale=1.0, flags=7):
    """Step the CUDA path in place on (p, m, v) and the oracle on host copies; return mismatch counts."""
    oracle, binding, _, _ = env
    hp_o = oracle.hparams(**hp_kw, flags=flags)
    pb, gb, mb, vb = bits(p), host_g(g), bits(m), bits(v)
    oracle.adamw_step(pb, gb, mb, vb, hp_o, seed, step, tensor_id, elem_offset, gscale)
    hp_g = binding.hparams(**hp_kw, grad_scale=gscale, flags=flags)
    binding.sr_adamw_step(p, g, m, v, hp_g, seed, step, tensor_id, elem_offset)
    torch.cuda.synchronize()
    return mismatches(bits(p), pb), mismatches(bits(m), mb), mismatches(bits(v), vb)


# ---------------------------------------------------------------------------------------------
# flat step
# ---------------------------------------------------------------------------------------------

def test_flat_step_2pow20(env):
    """One step on 2^20 elements, step 10, seed 1234, SR on x, m and v."""
    _, _, synth, dev = env
    p, g, m, v = synth.adamw_state(1 << 20, 1234, dev)
    p0 = bits(p)
    assert run_both(env, p, g, m, v, HP, seed=1234, step=10) == (0, 0, 0)
    assert mismatches(bits(p), p0) > (1 << 19)          # the step really changed the parameters


@pytest.mark.parametrize("n", [0, 1, 7, 8, 9, 255, 2047, 2048, 2049, 100003, (1 << 21) + 5])
@pytest.mark.parametrize("g_dtype", [torch.bfloat16, torch.float32])
def test_flat_step_ragged_sizes(env, n, g_dtype):
    _, _, synth, dev = env
    p, g, m, v = synth.adamw_state(n, 100 + n, dev, g_dtype=g_dtype)
    assert run_both(env, p, g, m, v, HP, seed=77, step=3, tensor_id=4) == (0, 0, 0)


@pytest.mark.parametrize("shift", [1, 3, 4])
def test_flat_step_unaligned_buffers(env, shift):
    """Buffers that start 2, 6 or 8 bytes past a 16-byte boundary take the element-wise path."""
    _, _, synth, dev = env
    n = 70001
    p, g, m, v = (t[shift:] for t in synth.adamw_state(n + shift, 5, dev))
    assert p.data_ptr() % 16 == (2 * shift) % 16
    assert run_both(env, p, g, m, v, HP, seed=1, step=2) == (0, 0, 0)


def test_flat_step_leaves_neighbouring_memory_alone(env):
    _, binding, synth, dev = env
    n, pad = 4099, 64
    bufs = synth.adamw_state(n + 2 * pad, 6, dev)
    before = [bits(t) for t in bufs]
    inner = [t[pad:pad + n] for t in bufs]
    binding.sr_adamw_step(*inner, binding.hparams(**HP), 9, 1)
    torch.cuda.synchronize()
    for t, b in zip(bufs, before):
        a = bits(t)
        assert np.array_equal(a[:pad], b[:pad]) and np.array_equal(a[pad + n:], b[pad + n:])
    assert np.array_equal(bits(bufs[1]), before[1])     # the gradient is read-only


@pytest.mark.parametrize("offset", [(1 << 32) - 1024, (1 << 32) - 1021, (1 << 33) + 8, (1 << 33) - 2048, (1 << 33) - 2045,
                                    3 * 832300544, (1 << 40) + 5])
def test_flat_step_index_offsets_cross_32_bits(env, offset):
    _, _, synth, dev = env
    p, g, m, v = synth.adamw_state(4096 + 3, 8, dev)
    assert run_both(env, p, g, m, v, HP, seed=(0xABCD << 32) | 17, step=1000, tensor_id=0xFFFFFFFF, elem_offset=offset) == (0, 0, 0)


@pytest.mark.parametrize("flags", range(8))
@pytest.mark.parametrize("g_dtype", [torch.bfloat16, torch.float32])
def test_flat_step_rounding_modes(env, flags, g_dtype):
    """Every choice of stochastic / nearest rounding for x, m, v (flags 1 = the paper's update-only SR)."""
    _, _, synth, dev = env
    p, g, m, v = synth.adamw_state(50000 + 1, 12, dev, g_dtype=g_dtype)
    assert run_both(env, p, g, m, v, HP, seed=3, step=10, gscale=0.125, flags=flags) == (0, 0, 0)


@pytest.mark.parametrize("eps", [0.0, 1e-8, 1e-4])
@pytest.mark.parametrize("flags", [15, 9, 8])
@pytest.mark.parametrize("g_dtype,n,offset", [(torch.bfloat16, (1 << 20) + 5, 0), (torch.float32, 50001, 24), (torch.bfloat16, 4099, 3)])
def test_flat_step_eps_inside(env, eps, flags, g_dtype, n, offset):
    """The other reading of the update step (epsilon under the square root, flag bit 3), with every rounding
    choice it is combined with here: bit-exact, and different from the default reading."""
    oracle, binding, synth, dev = env
    kw = dict(HP, eps=eps)
    p, g, m, v = synth.adamw_state(n, 14, dev, g_dtype=g_dtype)
    if n > 10000:                                   # special values take the same route as everything else
        mix = synth.downcast_mix(64, 5, dev)
        p[:64], m[64:128], v[128:192] = mix.bfloat16(), mix.bfloat16(), mix.abs().bfloat16()
    q = p.clone()
    assert run_both(env, p, g, m, v, kw, seed=21, step=10, elem_offset=offset, gscale=0.5, flags=flags) == (0, 0, 0)
    if eps > 1e-6 and n > 10000:
        p2, g2, m2, v2 = synth.adamw_state(n, 14, dev, g_dtype=g_dtype)
        binding.sr_adamw_step(p2, g2, m2, v2, binding.hparams(**kw, grad_scale=0.5, flags=flags & 7), 21, 10, 0, offset)
        torch.cuda.synchronize()
        assert mismatches(bits(p2)[192:], bits(p)[192:]) > n // 4


def test_eps_inside_list_and_master_recipe(env):
    oracle, binding, synth, dev = env
    kw = dict(HP, eps=1e-5)
    sizes = [5, 8192, 8193, 30000, 77, 2 * 8192 + 7]
    T = [synth.adamw_state(n, 700 + i, dev) for i, n in enumerate(sizes)]
    P, G, M, V = ([t[k] for t in T] for k in range(4))
    plan = binding.sr_mt_plan_create(P, G, M, V)
    host = [[bits(t) for t in P], [host_g(t) for t in G], [bits(t) for t in M], [bits(t) for t in V]]
    binding.sr_adamw_multi_tensor(plan, binding.hparams(**kw, flags=15), 4, 2, tensor_id_base=50)
    torch.cuda.synchronize()
    for i in range(len(sizes)):
        oracle.adamw_step(host[0][i], host[1][i], host[2][i], host[3][i], oracle.hparams(**kw, flags=15), 4, 2, 50 + i)
        assert mismatches(bits(P[i]), host[0][i]) + mismatches(bits(M[i]), host[2][i]) + mismatches(bits(V[i]), host[3][i]) == 0
    plan.destroy()
    n = 40003
    p0, g, m0, v0 = synth.adamw_state(n, 41, dev, g_dtype=torch.float32)
    p, m, v = p0.float(), m0.float(), v0.float()
    p16 = torch.zeros(n, dtype=torch.bfloat16, device=dev)
    ph, mh, vh = (t.cpu().numpy().copy() for t in (p, m, v))
    want16 = oracle.master_adamw_step(ph, host_g(g), mh, vh, oracle.hparams(**kw, flags=15), 3)
    binding.sr_master_adamw_step(p, p16, g, m, v, binding.hparams(**kw, flags=15), 3)
    torch.cuda.synchronize()
    for dev_t, host_t in ((p, ph), (m, mh), (v, vh)):
        assert np.array_equal(dev_t.cpu().numpy().view(np.uint32), host_t.view(np.uint32))
    assert mismatches(bits(p16), want16) == 0


@pytest.mark.parametrize("shift", [0, 4, 12])
def test_fp32_gradient_alignments(env, shift):
    """FP32 gradient buffers at 32-byte and at 16-byte-only alignment (shift counts 4-byte steps: 4 and 12 leave
    16-byte alignment only), flat and list."""
    oracle, binding, synth, dev = env
    n = 200003
    p, g, m, v = synth.adamw_state(n + 32, 77, dev, g_dtype=torch.float32)
    g = g[shift:shift + n]
    p, m, v = (t[:n] for t in (p, m, v))
    assert g.data_ptr() % 16 == 0 and (g.data_ptr() % 32 == 0) == (shift % 8 == 0)
    assert run_both(env, p, g, m, v, HP, seed=8, step=3, gscale=0.25) == (0, 0, 0)
    P, G, M, V = [p[:70000], p[70000:]], [g[:70000], g[70000:]], [m[:70000], m[70000:]], [v[:70000], v[70000:]]
    plan = binding.sr_mt_plan_create(P, G, M, V)
    host = [[bits(t) for t in P], [host_g(t) for t in G], [bits(t) for t in M], [bits(t) for t in V]]
    binding.sr_adamw_multi_tensor(plan, binding.hparams(**HP), 8, 4, tensor_id_base=3)
    torch.cuda.synchronize()
    for i in range(2):
        oracle.adamw_step(host[0][i], host[1][i], host[2][i], host[3][i], oracle.hparams(**HP), 8, 4, 3 + i)
        assert mismatches(bits(P[i]), host[0][i]) + mismatches(bits(M[i]), host[2][i]) + mismatches(bits(V[i]), host[3][i]) == 0
    plan.destroy()


@pytest.mark.parametrize("r", [1, 2, 3, 4, 5, 6, 7])
def test_offsets_that_split_noise_groups(env, r):
    """elem_offset = r mod 8 with aligned buffers: every 16-byte vector takes its noise from two groups.  Step, cast
    and accumulation, across a multiple of 2^33 in index space (where the high counter word changes)."""
    oracle, binding, synth, dev = env
    n = 40000 + r
    offset = (1 << 36) - 20000 + r - 8
    assert offset % 8 == r
    for g_dtype, flags in ((torch.bfloat16, 7), (torch.float32, 5)):
        p, g, m, v = synth.adamw_state(n, 60 + r, dev, g_dtype=g_dtype)
        assert run_both(env, p, g, m, v, HP, seed=(7 << 32) | 3, step=12, tensor_id=9, elem_offset=offset, flags=flags) == (0, 0, 0)
    src = synth.downcast_mix(n, 61, dev)
    dst = torch.empty(n, dtype=torch.bfloat16, device=dev)
    binding.sr_downcast_f32_bf16(src, dst, seed=(7 << 32) | 3, step=1, tensor_id=2, elem_offset=offset)
    torch.cuda.synchronize()
    assert mismatches(bits(dst), oracle.sr_downcast(src.cpu().numpy().copy(), (7 << 32) | 3, 1, 2, offset)) == 0
    _, g, acc, _ = synth.adamw_state(n, 62, dev)
    want = bits(acc)
    binding.sr_accumulate_bf16(acc, g, 0.5, seed=5, step=2, tensor_id=1, elem_offset=offset)
    oracle.sr_accumulate(want, bits(g), 0.5, 5, 2, 1, offset, True)
    torch.cuda.synchronize()
    assert mismatches(bits(acc), want) == 0


@pytest.mark.parametrize("n,r", [((1 << 25) + 77, 3), (200_000_013, 5)])
def test_offsets_that_split_noise_groups_over_many_runs(env, n, r):
    """The same at sizes where every warp walks several runs of consecutive vectors (short runs at 2^25 elements,
    the longest ones at 2e8), so that noise words cross from row to row, from run to run and from warp to warp:
    step with both gradient types, cast and accumulation, every element compared."""
    oracle, binding, synth, dev = env
    offset = (5 << 33) - 8 * 100_000 + r
    for g_dtype, flags in ((torch.bfloat16, 7), (torch.float32, 6)):
        p, g, m, v = synth.adamw_state(n, 70 + r, dev, g_dtype=g_dtype)
        assert run_both(env, p, g, m, v, HP, seed=(9 << 32) | 1, step=4, tensor_id=3, elem_offset=offset, flags=flags) == (0, 0, 0)
        del p, g, m, v
    src = synth.downcast_mix(n, 71, dev)
    dst = torch.empty(n, dtype=torch.bfloat16, device=dev)
    binding.sr_downcast_f32_bf16(src, dst, seed=11, step=1, tensor_id=2, elem_offset=offset)
    torch.cuda.synchronize()
    assert mismatches(bits(dst), oracle.sr_downcast(src.cpu().numpy().copy(), 11, 1, 2, offset)) == 0
    del src, dst
    _, g, acc, _ = synth.adamw_state(n, 72, dev)
    want = bits(acc)
    binding.sr_accumulate_bf16(acc, g, 0.5, seed=5, step=2, tensor_id=1, elem_offset=offset)
    oracle.sr_accumulate(want, bits(g), 0.5, 5, 2, 1, offset, True)
    torch.cuda.synchronize()
    assert mismatches(bits(acc), want) == 0


def test_offset_that_splits_noise_groups_long_launch(env):
    """2^29 elements and more take the long launch shape (staging and the table of head calls in dynamic shared
    memory) at offsets that are not multiples of 8 as well: every element compared, ragged end included."""
    _, _, synth, dev = env
    n = (1 << 29) + 8 * 37 + 5
    p, g, m, v = synth.adamw_state(n, 81, dev)
    assert run_both(env, p, g, m, v, HP, seed=3, step=7, tensor_id=1, elem_offset=(1 << 33) - 8 * 1000 + 3) == (0, 0, 0)


def test_flat_step_special_values(env):
    """NaN, infinities, zeros, subnormals and huge values in every input."""
    _, _, synth, dev = env
    n = 1 << 16
    p, g, m, v = synth.adamw_state(n, 13, dev, g_dtype=torch.float32)
    mix = synth.downcast_mix(4 * n, 99, dev)
    sel = torch.rand(4 * n, device=dev, generator=torch.Generator(device=dev).manual_seed(1)) < 0.3
    for k, t in enumerate((p, g, m, v)):
        s, x = sel[k * n:(k + 1) * n], mix[k * n:(k + 1) * n]
        if k == 3:
            x = x.abs()
        t[s] = x[s].to(t.dtype)
    assert run_both(env, p, g, m, v, HP, seed=5, step=2) == (0, 0, 0)
    assert run_both(env, p, g, m, v, HP, seed=5, step=3, flags=1) == (0, 0, 0)


def test_flat_step_hyperparameter_corners(env):
    _, _, synth, dev = env
    for kw, step in [(dict(lr=0.0, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.0), 1),
                     (dict(lr=1e-3, beta1=0.0, beta2=0.0, eps=0.0, weight_decay=0.0), 1),
                     (dict(lr=7e-4, beta1=0.9, beta2=0.999, eps=1e-6, weight_decay=0.2), 4_000_000_000),
                     (dict(lr=5.5e-4, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.1), 1)]:
        p, g, m, v = synth.adamw_state(30011, 14, dev)
        assert run_both(env, p, g, m, v, kw, seed=6, step=step) == (0, 0, 0)


@pytest.mark.parametrize("kw,step", [
    (dict(lr=1e-3, beta1=0.9, beta2=0.999999, eps=1.0, weight_decay=0.01), 1),      # 1/sqrt(1-beta2^t) = 1000, eps at its bound
    (dict(lr=1e-3, beta1=0.5, beta2=0.999, eps=0.0, weight_decay=0.0), 1),
    (dict(lr=3e-4, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.1), 1000),
    (dict(lr=1e-3, beta1=0.9, beta2=0.9999999, eps=1e-8, weight_decay=0.0), 1),     # beyond the gate: reference arithmetic
])
def test_in_range_arithmetic_over_its_whole_operand_range(env, kw, step):
    """Moments spread log-uniformly over and beyond the operand range of the branch-free square root
    and division (v, |m| from 2^-70 to 2^70, both gradient types), with the scalars at the limits
    under which that path is chosen: every vector inside the range must equal IEEE sqrt/div, every
    vector outside must have been redone."""
    _, _, synth, dev = env
    n = 1 << 20
    gen = torch.Generator(device=dev).manual_seed(1234 + step)
    for g_dtype in (torch.bfloat16, torch.float32):
        p, g, m, v = synth.adamw_state(n, 17, dev, g_dtype=g_dtype)
        span = 70.0 if g_dtype == torch.bfloat16 else 59.0      # second pass: (almost) every vector stays inside
        ev = (torch.rand(n, generator=gen, device=dev) * 2.0 - 1.0) * span
        em = (torch.rand(n, generator=gen, device=dev) * 2.0 - 1.0) * span
        sign = torch.where(torch.rand(n, generator=gen, device=dev) < 0.5, -1.0, 1.0)
        v.copy_(torch.exp2(ev).to(torch.bfloat16))
        m.copy_((sign * torch.exp2(em)).to(torch.bfloat16))
        g.mul_(0)                                   # m', v' are then beta * m, beta * v: the spread survives
        g[::7] = 1e-3
        assert run_both(env, p, g, m, v, kw, seed=8, step=step) == (0, 0, 0)


def test_in_range_arithmetic_equals_ieee_on_seeded_operands(env):
    """The branch-free square root and division against sqrt.rn / div.rn on 2^32 seeded operand sets per run
    (exponents over the whole range the kernels use them in; mantissas plain, just below a power of two, just
    above one; denominators also formed as root * factor + eps): no result may differ."""
    _, binding, _, dev = env
    bad = torch.full((2,), -1, dtype=torch.int64, device=dev)
    for seed in (1, (7 << 32) | 12345):
        binding.sr_selftest_in_range_arithmetic(seed, 1 << 31, bad)
        torch.cuda.synchronize()
        assert bad.tolist() == [0, 0], seed
    binding.sr_selftest_in_range_arithmetic(3, 0, bad)
    torch.cuda.synchronize()
    assert bad.tolist() == [0, 0]


def test_shards_equal_whole_and_runs_repeat(env):
    """Shared random state: 8 shards stepped separately equal the whole buffer; a second run repeats
    the first bit for bit; another seed does not."""
    _, binding, synth, dev = env
    n = 8 * 12500 + 4
    whole = synth.adamw_state(n, 15, dev)
    parts = [t.clone() for t in whole]
    again = [t.clone() for t in whole]
    other = [t.clone() for t in whole]
    hp = binding.hparams(**HP)
    binding.sr_adamw_step(*whole, hp, 21, 7, 3)
    binding.sr_adamw_step(*again, hp, 21, 7, 3)
    binding.sr_adamw_step(*other, hp, 22, 7, 3)
    bounds = np.linspace(0, n, 9).astype(int)
    for a, b in zip(bounds[:-1], bounds[1:]):
        binding.sr_adamw_step(*[t[a:b] for t in parts], hp, 21, 7, 3, elem_offset=int(a))
    torch.cuda.synchronize()
    for w, q, r in zip(whole, parts, again):
        assert torch.equal(w.view(torch.int16), q.view(torch.int16))
        assert torch.equal(w.view(torch.int16), r.view(torch.int16))
    assert not torch.equal(whole[0].view(torch.int16), other[0].view(torch.int16))


def test_checkpoint_resume_is_exact(env):
    """The random state is a function of (seed, step): 6 steps straight equal 3 steps, a copy out and
    back, and 3 more."""
    _, binding, synth, dev = env
    n = 40000
    a = synth.adamw_state(n, 16, dev)
    b = [t.clone() for t in a]
    hp = binding.hparams(**HP)
    grads = [synth.state_chunk(synth.ROLE_G, 1000 + s, 0, n, dev) for s in range(1, 7)]
    for s in range(1, 7):
        binding.sr_adamw_step(a[0], grads[s - 1], a[2], a[3], hp, 4, s)
    for s in range(1, 4):
        binding.sr_adamw_step(b[0], grads[s - 1], b[2], b[3], hp, 4, s)
    saved = [t.cpu() for t in b]
    b = [t.to(dev) for t in saved]
    for s in range(4, 7):
        binding.sr_adamw_step(b[0], grads[s - 1], b[2], b[3], hp, 4, s)
    torch.cuda.synchronize()
    for k in (0, 2, 3):
        assert torch.equal(a[k].view(torch.int16), b[k].view(torch.int16))


# ---------------------------------------------------------------------------------------------
# standalone stochastic-rounding cast
# ---------------------------------------------------------------------------------------------

def test_downcast_2pow26_mix(env):
    oracle, binding, synth, dev = env
    n = 1 << 26
    src = synth.downcast_mix(n, 7, dev)
    dst = torch.empty(n, dtype=torch.bfloat16, device=dev)
    binding.sr_downcast_f32_bf16(src, dst, seed=7)
    torch.cuda.synchronize()
    want = oracle.sr_downcast(src.cpu().numpy(), seed=7)
    got = bits(dst)
    assert mismatches(got, want) == 0
    b = src.cpu().numpy().view(np.uint32)
    nan = (b & 0x7FFFFFFF) > 0x7F800000
    assert nan.any() and np.all(got[nan] == 0x7FC0)
    rep = (b & 0xFFFF) == 0
    assert np.array_equal(got[rep & ~nan], (b[rep & ~nan] >> 16).astype(np.uint16))


@pytest.mark.parametrize("n,offset,shift", [(0, 0, 0), (1, 0, 0), (13, 5, 0), (4097, (1 << 32) - 9, 0), (5000, 16, 1), (5000, 3, 2)])
def test_downcast_ragged_and_unaligned(env, n, offset, shift):
    oracle, binding, synth, dev = env
    src = synth.downcast_mix(n + shift, 8, dev)[shift:]
    dst = torch.full((n + shift + 8,), -1.0, dtype=torch.bfloat16, device=dev)
    out = dst[shift:shift + n]
    binding.sr_downcast_f32_bf16(src, out, seed=(5 << 32) | 1, step=9, tensor_id=2, elem_offset=offset)
    torch.cuda.synchronize()
    want = oracle.sr_downcast(src.cpu().numpy().copy(), seed=(5 << 32) | 1, step=9, tensor_id=2, elem_offset=offset)
    assert mismatches(bits(out), want) == 0
    assert torch.all(dst[shift + n:] == -1.0) and torch.all(dst[:shift] == -1.0)


def test_downcast_unbiased_over_4096_seeds(env):
    """Mean over 4096 seeds of a 4096-element subset: within 6 sigma of x, sigma^2 = Delta^2 q(1-q)/4096
    (quantisation-error lemma), and the up-counts follow Binomial(4096, q)."""
    oracle, binding, synth, dev = env
    k = 4096
    src = synth.downcast_mix(1 << 16, 7, dev)
    b_all = src.cpu().numpy().view(np.uint32)
    ok = ((b_all & 0x7FFFFFFF) < 0x7F7F0000)                      # finite, below the last BF16 interval
    idx = np.flatnonzero(ok)[:k]
    sub = src[torch.from_numpy(idx).to(dev)].contiguous()
    outs = torch.empty((k, k), dtype=torch.bfloat16, device=dev)
    for s in range(k):
        binding.sr_downcast_f32_bf16(sub, outs[s], seed=s)
    torch.cuda.synchronize()
    sub_h = sub.cpu().numpy()
    for s in (0, 1, 4095):
        assert np.array_equal(bits(outs[s]), oracle.sr_downcast(sub_h, seed=s))
    x = sub_h.astype(np.float64)
    b = sub_h.view(np.uint32)
    lo = (b & 0xFFFF0000).view(np.float32).astype(np.float64)
    hi = ((b & 0xFFFF0000) + 0x10000).astype(np.uint32).view(np.float32).astype(np.float64)
    delta = hi - lo
    q = (b & 0xFFFF) / 65536.0
    vals = outs.float().double().cpu().numpy()
    mean = vals.mean(axis=0)
    sigma = np.abs(delta) * np.sqrt(q * (1 - q) / k)
    assert np.all(np.abs(mean - x) <= 6 * sigma + 0.0)
    ups = (bits(outs).reshape(k, k) != (b >> 16).astype(np.uint16)[None, :]).sum(axis=0)
    var = k * q * (1 - q)
    assert np.all(ups[var == 0] == 0)
    wide = var >= 25.0                                     # normal approximation is good there
    assert wide.sum() > k // 2
    z = (ups - k * q)[wide] / np.sqrt(var[wide])
    assert np.abs(z).max() < 6.0 and abs(z.mean()) < 0.1 and 0.9 < z.std() < 1.1


def test_random_walk_example_on_the_gpu(env):
    """Section 2.2, first example, run with the library's cast: walkers start on a BF16 level, take two
    half-level steps and then steps of epsilon levels.  P(T <= 2) = 3/4 and E[T] = 3/2 + 1/(4 eps)."""
    _, binding, _, dev = env
    walkers, eps, horizon = 1 << 20, 1.0 / 16.0, 400
    level, delta = 1.0, 2.0 ** -7                                   # 1.0 and 1 + 2^-7 are consecutive BF16 values
    x = torch.full((walkers,), level, dtype=torch.float32, device=dev)
    out = torch.empty(walkers, dtype=torch.bfloat16, device=dev)
    hit = torch.zeros(walkers, dtype=torch.int32, device=dev)
    for t in range(1, horizon + 1):
        u = delta / 2 if t <= 2 else delta * eps
        binding.sr_downcast_f32_bf16(x + u, out, seed=2024, step=t)
        x = out.float()
        hit = torch.where((hit == 0) & (x > level), torch.full_like(hit, t), hit)
        x = torch.where(hit > 0, torch.full_like(x, level + delta), x)   # absorbed at the upper level
    assert int((hit == 0).sum()) == 0                               # (15/16)^398 is far below 2^-20
    p_le_2 = float((hit <= 2).float().mean())
    assert abs(p_le_2 - 0.75) < 5 * (0.75 * 0.25 / walkers) ** 0.5
    mean_T = float(hit.double().mean())
    want = 1.5 + 0.25 / eps
    var_T = 0.25 * (1 - eps) / eps ** 2 + 5.0                        # generous bound on Var[T]
    assert abs(mean_T - want) < 5 * (var_T / walkers) ** 0.5
    for n in (3, 4, 6):
        p_n = float((hit == n).float().mean())
        assert abs(p_n - 0.25 * (1 - eps) ** (n - 3) * eps) < 5 * (0.02 / walkers) ** 0.5


def test_linear_loss_toy_qualitative(env):
    """Section 2.2, second example, run on the library: Adam on the linear loss f(x) = -(x - 2) + 1 for
    x < 3 (0 beyond), from x0 = 2, with a decaying learning rate.  The paper does not give the decay
    schedule, so only the qualitative statements are checked, with an assumed schedule (linear decay over
    5000 steps, chosen so that FP32 reaches x = 3 in about 4600 steps at minimum rate 1e-5): BF16 with
    stochastic rounding needs more steps than FP32 on average, and fewer when the minimum rate is higher."""
    _, binding, _, dev = env
    runs, horizon = 1024, 40000

    def schedule(t, lr_min):
        lr_max = 3.94e-4
        return max(lr_min, lr_max - (lr_max - 1e-5) * t / 5000.0)

    def steps_to_converge(lr_min, sr):
        kw = dict(beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0)
        x = torch.full((runs,), 2.0, device=dev, dtype=torch.bfloat16 if sr else torch.float32)
        m, v = torch.zeros_like(x), torch.zeros_like(x)
        x16 = torch.empty(runs, dtype=torch.bfloat16, device=dev)
        hit = torch.zeros(runs, dtype=torch.int32, device=dev)
        for t in range(1, horizon + 1):
            g = torch.where(x < 3.0, -1.0, 0.0).to(torch.bfloat16)
            hp = binding.hparams(lr=schedule(t - 1, lr_min), **kw)
            if sr:
                binding.sr_adamw_step(x, g, m, v, hp, seed=77, step=t)
            else:
                binding.sr_master_adamw_step(x, x16, g, m, v, hp, t)
            hit = torch.where((hit == 0) & (x >= 3.0), torch.full_like(hit, t), hit)
            if t % 500 == 0 and int((hit == 0).sum()) == 0:
                break
        # a run still short of x = 3 at the horizon counts as the horizon: its mean is then a lower bound
        return torch.where(hit == 0, torch.full_like(hit, horizon), hit).double()

    fp32 = steps_to_converge(1e-5, sr=False)
    assert float(fp32.min()) == float(fp32.max()) and 4500 <= float(fp32[0]) <= 4700
    assert float(fp32[0]) < horizon
    sr_slow = steps_to_converge(1e-5, sr=True)
    sr_fast = steps_to_converge(5e-5, sr=True)
    assert float(sr_slow.mean()) > 1.1 * float(fp32[0])          # stagnation at small learning rates
    assert float(sr_fast.mean()) < float(sr_slow.mean())          # a higher minimum rate closes the gap
    assert float(sr_slow.std()) > 0                               # runs differ: the rounding is stochastic


# ---------------------------------------------------------------------------------------------
# squared norm, clipping, and the clipped shard step
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("n", [0, 1, 5, 8191, 8192, 8193, 100000, 8192 * 8192 + 12345])
@pytest.mark.parametrize("g_dtype", [torch.float32, torch.bfloat16])
def test_sqnorm_bit_exact(env, n, g_dtype):
    oracle, binding, synth, dev = env
    g = torch.empty(n, dtype=g_dtype, device=dev)
    synth.fill_state(g, synth.ROLE_G, 17, outlier_fraction=0.01)
    ws = torch.empty(max(1, binding.grad_sqnorm_workspace_bytes(n) // 8), dtype=torch.float64, device=dev)
    out = torch.full((1,), -1.0, dtype=torch.float64, device=dev)
    binding.grad_sqnorm(g, out, ws)
    torch.cuda.synchronize()
    assert float(out.item()).hex() == oracle.sqnorm(host_g(g)).hex()


@pytest.mark.parametrize("g_dtype", [torch.float32, torch.bfloat16])
def test_sqnorm_unaligned(env, g_dtype):
    """A buffer that starts one element past a 16-byte boundary: every tree block goes element by element."""
    oracle, binding, synth, dev = env
    g = torch.empty(30000, dtype=g_dtype, device=dev)
    synth.fill_state(g, synth.ROLE_G, 18, outlier_fraction=0.01)
    g = g[1:]
    ws = torch.empty(16, dtype=torch.float64, device=dev)
    out = torch.zeros(1, dtype=torch.float64, device=dev)
    binding.grad_sqnorm(g, out, ws)
    torch.cuda.synchronize()
    assert float(out.item()).hex() == oracle.sqnorm(host_g(g)).hex()


@pytest.mark.parametrize("g_dtype", [torch.float32, torch.bfloat16])
def test_sqnorm_with_more_than_one_later_level(env, g_dtype):
    """More than 8192 tree blocks: the pass over the block sums also folds its own results, and the output cell counts
    its finished blocks first, whatever the cell held before the call.  Repeated, because the block that folds is the
    one that happens to finish last."""
    oracle, binding, synth, dev = env
    n = 3 * 8192 * 8192 + 777
    g = torch.empty(n, dtype=g_dtype, device=dev)
    synth.fill_state(g, synth.ROLE_G, 19, outlier_fraction=0.01)
    want = oracle.sqnorm(host_g(g)).hex()
    ws = torch.empty(binding.grad_sqnorm_workspace_bytes(n) // 8, dtype=torch.float64, device=dev)
    for before in (-1.0, float("nan"), 1e300, 0.0, 5e-324, float("inf")) * 3:
        out = torch.full((1,), before, dtype=torch.float64, device=dev)
        binding.grad_sqnorm(g, out, ws)
        torch.cuda.synchronize()
        assert float(out.item()).hex() == want


def test_clip_scale_bit_exact(env):
    oracle, binding, _, dev = env
    out = torch.zeros(1, dtype=torch.float32, device=dev)
    for S, acc, mx in [(4.0, 0.125, 1.0), (1e6, 0.125, 1.0), (0.0, 1.0, 1.0), (7.3e4, 0.25, 2.0), (832.3004, 0.125, 1.0),
                       (float("inf"), 1.0, 1.0), (float("nan"), 1.0, 1.0)]:
        binding.sr_clip_scale(torch.tensor([S], dtype=torch.float64, device=dev), acc, mx, out)
        got, want = float(out.item()), oracle.clip_scale(S, acc, mx)
        assert (np.isnan(got) and np.isnan(want)) or np.float32(got).tobytes() == np.float32(want).tobytes()


def _clipped_shard(env, n, rank):
    oracle, binding, synth, dev = env
    p, g, m, v = synth.adamw_state(n, 19, dev, g_dtype=torch.float32, outlier_fraction=0.01)
    ws = torch.empty(max(1, binding.grad_sqnorm_workspace_bytes(n) // 8), dtype=torch.float64, device=dev)
    S = torch.zeros(1, dtype=torch.float64, device=dev)
    gs = torch.zeros(1, dtype=torch.float32, device=dev)
    pb, gb, mb, vb = bits(p), host_g(g), bits(m), bits(v)
    binding.grad_sqnorm(g, S, ws)
    binding.sr_clip_scale(S, 0.125, 1.0, gs)
    binding.sr_adamw_step(p, g, m, v, binding.hparams(**HP, grad_scale_dev=gs), 1234, 1000, 0, rank * n)
    torch.cuda.synchronize()
    S_o = oracle.sqnorm(gb)
    gs_o = oracle.clip_scale(S_o, 0.125, 1.0)
    assert float(S.item()).hex() == S_o.hex()
    assert np.float32(gs.item()).tobytes() == np.float32(gs_o).tobytes()
    assert gs_o < 0.125                                       # the outliers make clipping active
    oracle.adamw_step(pb, gb, mb, vb, oracle.hparams(**HP), 1234, 1000, 0, rank * n, gs_o)
    return mismatches(bits(p), pb), mismatches(bits(m), mb), mismatches(bits(v), vb)


def test_clipped_shard_small(env):
    assert _clipped_shard(env, (1 << 22) + 13, 3) == (0, 0, 0)


def test_clipped_shard_full_size(env):
    """A 1/8 shard of the 6.7B buffer (832 300 544 elements, FP32 gradients with 1% outliers), rank 3."""
    _, _, synth, _ = env
    n = synth.gpt_flat_numel() // 8
    assert n == 832_300_544
    assert _clipped_shard(env, n, 3) == (0, 0, 0)


def test_clipped_sequence_in_a_cuda_graph(env):
    """accumulate -> norm -> clip factor -> step captured once on a stream and replayed: no call allocates,
    synchronises or reads back, so the whole sequence is capturable; every replay matches the oracle."""
    oracle, binding, synth, dev = env
    n = (1 << 21) + 24
    p, g, m, v = synth.adamw_state(n, 23, dev, g_dtype=torch.float32, outlier_fraction=0.01)
    acc = torch.zeros(n, dtype=torch.bfloat16, device=dev)
    ws = torch.empty(max(1, binding.grad_sqnorm_workspace_bytes(n) // 8), dtype=torch.float64, device=dev)
    S = torch.zeros(1, dtype=torch.float64, device=dev)
    gs = torch.zeros(1, dtype=torch.float32, device=dev)
    hp = binding.hparams(**HP, grad_scale_dev=gs)
    pb, gb, mb, vb, ab = bits(p), host_g(g), bits(m), bits(v), bits(acc)

    def sequence():
        binding.sr_accumulate_bf16(acc, g, 0.5, seed=1234, step=7, tensor_id=2)
        binding.grad_sqnorm(acc, S, ws)
        binding.sr_clip_scale(S, 1.0, 1.0, gs)
        binding.sr_adamw_step(p, acc, m, v, hp, 1234, 7, 2, 0)

    binding.lib()                                   # library and device info are set up before the capture
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        sequence()                                  # warm-up outside the capture (replayed on the oracle as well)
    torch.cuda.current_stream().wait_stream(side)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        sequence()
    replays = 3
    for _ in range(replays):
        graph.replay()
    torch.cuda.synchronize()
    for _ in range(1 + replays):
        oracle.sr_accumulate(ab, gb, 0.5, 1234, 7, 2, 0, True)
        S_o = oracle.sqnorm(ab)
        oracle.adamw_step(pb, ab, mb, vb, oracle.hparams(**HP), 1234, 7, 2, 0, oracle.clip_scale(S_o, 1.0, 1.0))
    assert float(S.item()).hex() == S_o.hex()
    assert mismatches(bits(acc), ab) == 0
    assert (mismatches(bits(p), pb), mismatches(bits(m), mb), mismatches(bits(v), vb)) == (0, 0, 0)


# ---------------------------------------------------------------------------------------------
# tensor list
# ---------------------------------------------------------------------------------------------

def _run_list(env, specs, steps, seed=1234, grad_seed=4321, shift=0):
    oracle, binding, synth, dev = env
    P = [synth.init_param(s, seed, i, dev) for i, s in enumerate(specs)]
    if shift:
        P = [torch.cat([t.new_zeros(shift), t])[shift:] if i % 3 == 1 else t for i, t in enumerate(P)]
    M = [torch.zeros_like(t) for t in P]
    V = [torch.zeros_like(t) for t in P]
    G = [torch.zeros_like(t) for t in P]
    plan = binding.sr_mt_plan_create(P, G, M, V)
    assert plan.total_elements == sum(s.numel for s in specs)
    hp_g, hp_o = binding.hparams(**HP), oracle.hparams(**HP)
    host = [[bits(t) for t in P], None, [bits(t) for t in M], [bits(t) for t in V]]
    total = [0, 0, 0]
    for step in range(1, steps + 1):
        for i, s in enumerate(specs):
            G[i].copy_(synth.fresh_grad(s, grad_seed, step, i, dev))
        binding.sr_adamw_multi_tensor(plan, hp_g, seed, step)
        torch.cuda.synchronize()
        for i in range(len(specs)):
            oracle.adamw_step(host[0][i], bits(G[i]), host[2][i], host[3][i], hp_o, seed, step, tensor_id=i)
        for k, dev_list in ((0, P), (2, M), (3, V)):
            for i in range(len(specs)):
                total[0 if k == 0 else k - 1] += mismatches(bits(dev_list[i]), host[k][i])
        assert total == [0, 0, 0], f"step {step}"
    plan.destroy()
    return total


def test_multi_tensor_small_list_with_odd_shapes(env):
    _, _, synth, _ = env
    T = synth.TensorSpec
    specs = [T("a", (1,), "normal"), T("b", (7,), "ones"), T("c", (16384,), "normal"), T("d", (16385,), "normal"),
             T("e", (3, 1111), "normal"), T("f", (0,), "zeros"), T("g", (100000,), "normal"), T("h", (8,), "zeros")]
    _run_list(env, specs, steps=3)
    _run_list(env, specs, steps=2, shift=1)      # every third tensor starts 2 bytes off alignment


@pytest.mark.parametrize("g_dtype,flags,gscale", [(torch.bfloat16, 7, 1.0), (torch.bfloat16, 1, 0.5), (torch.float32, 7, 1.0),
                                                 (torch.float32, 0, 0.125)])
def test_multi_tensor_random_lists(env, g_dtype, flags, gscale):
    """Lists of many tensors whose sizes straddle every boundary of the kernel: fewer vectors than a
    block has threads, one more than that, whole chunks, a chunk plus one element, runs of tiny tensors
    (threads that skip several chunks in a row), empty tensors, and a few unaligned ones."""
    oracle, binding, synth, dev = env
    rng = np.random.default_rng(int(flags) * 7 + (g_dtype == torch.float32))
    sizes = [1, 3, 8, 8 * 127, 8 * 128, 8 * 128 + 1, 8 * 129, 8191, 8192, 8193, 2 * 8192, 2 * 8192 + 7, 0, 5, 5, 5, 5, 5, 5, 16, 24,
             3 * 8192 + 8 * 64, 40, 100000] + [int(x) for x in rng.integers(1, 30000, 40)] + [int(x) for x in rng.integers(1, 64, 30)]
    order = rng.permutation(len(sizes))
    sizes = [sizes[i] for i in order]
    P, G, M, V = [], [], [], []
    for i, n in enumerate(sizes):
        shift = 1 if i % 11 == 3 else 0                 # some tensors start 2 bytes off a 16-byte boundary
        p, g, m, v = synth.adamw_state(n + shift, 900 + i, dev, g_dtype=g_dtype)
        P.append(p[shift:]); G.append(g[shift:]); M.append(m[shift:]); V.append(v[shift:])
    plan = binding.sr_mt_plan_create(P, G, M, V)
    assert plan.total_elements == sum(sizes)
    hp_o = oracle.hparams(**HP, flags=flags)
    hp_g = binding.hparams(**HP, grad_scale=gscale, flags=flags)
    host = [[bits(t) for t in P], [host_g(t) for t in G], [bits(t) for t in M], [bits(t) for t in V]]
    for step in (1, 2):
        binding.sr_adamw_multi_tensor(plan, hp_g, 99, step, tensor_id_base=1000)
        torch.cuda.synchronize()
        bad = 0
        for i in range(len(sizes)):
            oracle.adamw_step(host[0][i], host[1][i], host[2][i], host[3][i], hp_o, 99, step, 1000 + i, 0, gscale)
            bad += mismatches(bits(P[i]), host[0][i]) + mismatches(bits(M[i]), host[2][i]) + mismatches(bits(V[i]), host[3][i])
            assert np.array_equal(host_g(G[i]), host[1][i])
        assert bad == 0, f"step {step}"
    plan.destroy()


@pytest.mark.parametrize("flags,gscale", [(7, 1.0), (5, 0.25)])
def test_multi_tensor_long_list(env, flags, gscale):
    """A list of more than 2^29 elements (65 536 chunks and more): a few large tensors plus sizes around every
    boundary of a block's pass over a chunk and of a chunk itself, runs of tiny tensors, an empty and an unaligned
    one; every element compared."""
    oracle, binding, synth, dev = env
    sizes = [1 << 27, 5, 8 * 511, 8 * 512, 8 * 512 + 1, 8 * 513, 8191, 8192, 8193, (1 << 28) + 8 * 300 + 3, 0, 7, 7, 7, 16,
             8 * 255, 8 * 256, 8 * 257, 2 * 8192 + 8 * 512, 100003, (1 << 27) + 9, 12345, 8 * 1023, 3]
    P, G, M, V = [], [], [], []
    for i, n in enumerate(sizes):
        shift = 1 if i == 19 else 0
        p, g, m, v = synth.adamw_state(n + shift, 300 + i, dev)
        P.append(p[shift:]); G.append(g[shift:]); M.append(m[shift:]); V.append(v[shift:])
    assert sum((n + 8191) // 8192 for n in sizes) >= 1 << 16
    plan = binding.sr_mt_plan_create(P, G, M, V)
    hp_o = oracle.hparams(**HP, flags=flags)
    hp_g = binding.hparams(**HP, grad_scale=gscale, flags=flags)
    host = [[bits(t) for t in P], [bits(t) for t in G], [bits(t) for t in M], [bits(t) for t in V]]
    ws = torch.empty(max(1, binding.grad_sqnorm_multi_tensor_workspace_bytes(plan) // 8), dtype=torch.float64, device=dev)
    S = torch.zeros(1, dtype=torch.float64, device=dev)
    binding.grad_sqnorm_multi_tensor(plan, S, ws)
    binding.sr_adamw_multi_tensor(plan, hp_g, 17, 3, tensor_id_base=50)
    torch.cuda.synchronize()
    assert float(S.item()).hex() == oracle.sqnorm_list([host[1][i] for i in range(len(sizes))]).hex()
    for i in range(len(sizes)):
        oracle.adamw_step(host[0][i], host[1][i], host[2][i], host[3][i], hp_o, 17, 3, 50 + i, 0, gscale)
        assert mismatches(bits(P[i]), host[0][i]) + mismatches(bits(M[i]), host[2][i]) + mismatches(bits(V[i]), host[3][i]) == 0, i
        assert np.array_equal(bits(G[i]), host[1][i])
    plan.destroy()


def test_multi_tensor_large_tensors_keep_stream_order(env):
    """Five tensors of 2^24 elements and more (their launches alternate between the caller's stream and the plan's own)
    plus small ones, stepped three times on a stream of the caller's with no synchronisation: the gradients of every
    step are copied in on that stream just before the call and the parameters copied out just after it."""
    oracle, binding, synth, dev = env
    sizes = [1 << 24, 100, (1 << 24) + 8, 3 << 23, 4097, 1 << 24, (1 << 24) + 16]
    steps = 3
    P, G, M, V, Gsrc = [], [], [], [], []
    for i, n in enumerate(sizes):
        p, g, m, v = synth.adamw_state(n, 500 + i, dev)
        P.append(p); G.append(torch.zeros_like(g)); M.append(m); V.append(v)
        Gsrc.append([synth.adamw_state(n, 600 + 10 * i + t, dev)[1] for t in range(steps)])
    plan = binding.sr_mt_plan_create(P, G, M, V)
    hp_o, hp_g = oracle.hparams(**HP), binding.hparams(**HP)
    host = [[bits(t) for t in P], None, [bits(t) for t in M], [bits(t) for t in V]]
    host_g = [[bits(Gsrc[i][t]) for i in range(len(sizes))] for t in range(steps)]
    out = [[torch.empty_like(p) for p in P] for _ in range(steps)]
    torch.cuda.synchronize()
    s = torch.cuda.Stream(device=dev)
    with torch.cuda.stream(s):
        for t in range(steps):
            for i in range(len(sizes)):
                G[i].copy_(Gsrc[i][t], non_blocking=True)
            binding.sr_adamw_multi_tensor(plan, hp_g, 23, 5 + t, tensor_id_base=7, stream=s)
            for i in range(len(sizes)):
                out[t][i].copy_(P[i], non_blocking=True)
    s.synchronize()
    for t in range(steps):
        for i in range(len(sizes)):
            oracle.adamw_step(host[0][i], host_g[t][i], host[2][i], host[3][i], hp_o, 23, 5 + t, 7 + i, 0, 1.0)
            assert mismatches(bits(out[t][i]), host[0][i]) == 0, (t, i)
    for i in range(len(sizes)):
        assert mismatches(bits(M[i]), host[2][i]) + mismatches(bits(V[i]), host[3][i]) == 0, i
    plan.destroy()


def test_multi_tensor_with_large_tensors_in_a_cuda_graph(env):
    """The list step whose large tensors alternate between two streams, captured once and replayed: the fork and the
    join are events inside the call, so the capture takes the plan's stream in and releases it again."""
    oracle, binding, synth, dev = env
    sizes = [1 << 24, 300, (1 << 24) + 8, 1 << 24, 9000]
    P, G, M, V = [], [], [], []
    for i, n in enumerate(sizes):
        p, g, m, v = synth.adamw_state(n, 700 + i, dev)
        P.append(p); G.append(g); M.append(m); V.append(v)
    plan = binding.sr_mt_plan_create(P, G, M, V)
    hp_o, hp_g = oracle.hparams(**HP), binding.hparams(**HP)
    host = [[bits(t) for t in P], [bits(t) for t in G], [bits(t) for t in M], [bits(t) for t in V]]
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        binding.sr_adamw_multi_tensor(plan, hp_g, 29, 11, tensor_id_base=3)       # warm-up outside the capture
    torch.cuda.current_stream().wait_stream(side)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        binding.sr_adamw_multi_tensor(plan, hp_g, 29, 11, tensor_id_base=3)
    replays = 2
    for _ in range(replays):
        graph.replay()
    torch.cuda.synchronize()
    for i in range(len(sizes)):
        for _ in range(1 + replays):
            oracle.adamw_step(host[0][i], host[1][i], host[2][i], host[3][i], hp_o, 29, 11, 3 + i, 0, 1.0)
        assert mismatches(bits(P[i]), host[0][i]) + mismatches(bits(M[i]), host[2][i]) + mismatches(bits(V[i]), host[3][i]) == 0, i
    del graph
    plan.destroy()


def test_multi_tensor_gpt2_350m_ten_steps(env):
    """GPT-2 350M parameter list (292 tensors, 354 823 168 elements), 10 iterations with fresh
    gradients, zero mismatches after every iteration."""
    _, _, synth, _ = env
    specs = synth.gpt2_param_list()
    assert len(specs) == 292 and sum(s.numel for s in specs) == 354_823_168
    _run_list(env, specs, steps=10)


# ---------------------------------------------------------------------------------------------
# full-size flat buffer: sampled chunks
# ---------------------------------------------------------------------------------------------

def test_flat_6p7b_every_element(env):
    """The 6 658 404 352-element buffer stepped once (step 1000) in the launch shape the benchmark
    times.  Every chunk of 2^26 elements (the last one ragged, two of them around index 2^32) is drawn
    again from the seeded generator, stepped by the oracle and compared bit for bit: all elements
    are checked.  Guard elements past the end stay intact."""
    oracle, binding, synth, dev = env
    n = synth.gpt_flat_numel()
    assert n == 6_658_404_352
    guard = 64
    bufs = [torch.empty(n + guard, dtype=torch.bfloat16, device=dev) for _ in range(4)]
    roles = (synth.ROLE_P, synth.ROLE_G, synth.ROLE_M, synth.ROLE_V)
    for t, role in zip(bufs, roles):
        synth.fill_state(t[:n], role, 1234)
        t[n:] = 1.5
    p, g, m, v = (t[:n] for t in bufs)
    binding.sr_adamw_step(p, g, m, v, binding.hparams(**HP), 1234, 1000)
    torch.cuda.synchronize()
    for t in bufs:
        assert torch.all(t[n:] == 1.5)
    nchunks = (n + synth.CHUNK - 1) // synth.CHUNK
    hp_o = oracle.hparams(**HP)
    bad = 0
    for c in range(nchunks):
        start = c * synth.CHUNK
        length = min(synth.CHUNK, n - start)
        pre = [bits(synth.state_chunk(role, 1234, c, length, dev)) for role in roles]
        assert np.array_equal(pre[1], bits(g[start:start + length]))            # the gradient was not touched
        oracle.adamw_step(*pre, hp_o, 1234, 1000, 0, start)
        for k, t in ((0, p), (2, m), (3, v)):
            bad += mismatches(bits(t[start:start + length]), pre[k])
        assert bad == 0, f"chunk {c}"
    assert nchunks == 100


@pytest.mark.parametrize("flags,gscale,offset", [(7, 1.0, 0), (5, 0.25, (1 << 33) - (1 << 29))])
def test_long_launch_tiles_with_ragged_tail_and_special_values(env, flags, gscale, offset):
    """A launch long enough for the long-launch shape (2^30 elements) plus a ragged tail, with NaN / infinity /
    zero / tiny values sprinkled in (vectors that fall back to the reference arithmetic), a gradient scale,
    nearest rounding on m, and an offset that makes the buffer cross a multiple of 2^33 in index space.  Every
    element is compared."""
    oracle, binding, synth, dev = env
    n = (1 << 30) + 3 * 4096 + 1237
    guard = 64
    roles = (synth.ROLE_P, synth.ROLE_G, synth.ROLE_M, synth.ROLE_V)
    bufs = [torch.empty(n + guard, dtype=torch.bfloat16, device=dev) for _ in range(4)]
    for t, role in zip(bufs, roles):
        synth.fill_state(t[:n], role, 77)
        t[n:] = 1.5
    p, g, m, v = (t[:n] for t in bufs)
    special = torch.tensor([float("nan"), float("inf"), -float("inf"), 0.0, -0.0, 1e-30, 3e38, 1e-40], device=dev).bfloat16()
    for k, t in enumerate((p, g, m, v)):
        pos = torch.arange(8, device=dev) * 977 + 13 + 131071 * k
        t[pos] = special.abs() if k == 3 else special
        t[pos + (1 << 29)] = special.abs() if k == 3 else special
    before = [bits(t[c * synth.CHUNK:(c + 1) * synth.CHUNK]) for c in (0, 8) for t in (p, g, m, v)]
    binding.sr_adamw_step(p, g, m, v, binding.hparams(**HP, grad_scale=gscale, flags=flags), 4321, 17, 5, offset)
    torch.cuda.synchronize()
    for t in bufs:
        assert torch.all(t[n:] == 1.5)
    hp_o = oracle.hparams(**HP, flags=flags)
    nchunks = (n + synth.CHUNK - 1) // synth.CHUNK
    for c in range(nchunks):
        start = c * synth.CHUNK
        length = min(synth.CHUNK, n - start)
        if c in (0, 8):                               # the chunks that hold the special values
            pre = [a.copy() for a in before[(0 if c == 0 else 4):(4 if c == 0 else 8)]]
        else:
            pre = [bits(synth.state_chunk(role, 77, c, length, dev)) for role in roles]
        oracle.adamw_step(*pre, hp_o, 4321, 17, 5, offset + start, gscale)
        bad = sum(mismatches(bits(t[start:start + length]), pre[k]) for k, t in ((0, p), (2, m), (3, v)))
        assert bad == 0, f"chunk {c}"


# ---------------------------------------------------------------------------------------------
# host-resident state
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("g_dtype", [torch.bfloat16, torch.float32])
def test_host_resident_step_equals_oracle(env, g_dtype):
    """State in pinned host memory, staged through the device in chunks: same bits as the oracle
    (and therefore as the in-device step), including a ragged last chunk and a non-zero offset."""
    oracle, binding, synth, dev = env
    n, chunk = 5 * 65536 + 1237, 65536
    p, g, m, v = (t.pin_memory() for t in synth.adamw_state(n, 23, "cpu", g_dtype=g_dtype))
    pb, mb, vb = (synth.bits16(t).copy() for t in (p, m, v))
    gb = g.numpy().copy() if g_dtype == torch.float32 else synth.bits16(g).copy()
    oracle.adamw_step(pb, gb, mb, vb, oracle.hparams(**HP), 31, 5, 2, 1000)
    staging = torch.empty(binding.sr_adamw_step_host_staging_bytes(g_dtype, chunk), dtype=torch.uint8, device=dev)
    binding.sr_adamw_step_host(p, g, m, v, binding.hparams(**HP), 31, 5, staging, chunk, tensor_id=2, elem_offset=1000)
    torch.cuda.synchronize()
    assert mismatches(synth.bits16(p), pb) == 0 and mismatches(synth.bits16(m), mb) == 0 and mismatches(synth.bits16(v), vb) == 0


# ---------------------------------------------------------------------------------------------
# FP32-master comparison recipe
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("n,shift", [(0, 0), (5, 0), (8 * 4096 + 3, 0), ((1 << 22) + 11, 0), (9001, 1), (70003, 4)])
@pytest.mark.parametrize("g_dtype,gscale", [(torch.bfloat16, 1.0), (torch.float32, 0.125)])
def test_master_recipe_bit_exact(env, n, shift, g_dtype, gscale):
    """FP32 master weights and moments + nearest-rounded BF16 copy (the paper's mixed-precision
    comparison): two consecutive steps, every FP32 word and every BF16 pattern equal to the oracle's.
    shift moves every buffer by 4 * shift bytes: 1 = unaligned (element-wise path), 4 = 16-byte but not
    32-byte aligned (16-byte accesses), 0 = 32-byte accesses."""
    oracle, binding, synth, dev = env
    s16 = 2 * shift                                  # BF16 buffers: twice the elements for the same bytes
    p0, g, m0, v0 = synth.adamw_state(n + 2 * shift, 31 + n, dev, g_dtype=g_dtype)
    p, m, v = (t.float()[shift:shift + n] for t in (p0, m0, v0))
    g = g[shift:shift + n] if g_dtype == torch.float32 else g[s16:s16 + n]
    if n > 100:
        p[7], m[11], v[13], v[17] = float("nan"), float("inf"), 0.0, 1e-30      # vectors that leave the fast range
    p16 = torch.zeros(n + s16, dtype=torch.bfloat16, device=dev)[s16:]
    ph, mh, vh = (t.cpu().numpy().copy() for t in (p, m, v))
    gh = host_g(g)
    hp_kw = dict(HP)
    for step in (1, 2):
        want16 = oracle.master_adamw_step(ph, gh, mh, vh, oracle.hparams(**hp_kw), step, gscale)
        binding.sr_master_adamw_step(p, p16, g, m, v, binding.hparams(**hp_kw, grad_scale=gscale), step)
        torch.cuda.synchronize()
        for dev_t, host_t in ((p, ph), (m, mh), (v, vh)):
            got = dev_t.cpu().numpy().view(np.uint32)
            want = host_t.view(np.uint32)
            nan = (want & 0x7FFFFFFF) > 0x7F800000                      # NaN payloads may differ between platforms
            assert np.array_equal(got[~nan], want[~nan])
            assert np.all((got[nan] & 0x7FFFFFFF) > 0x7F800000)
            host_t[nan] = dev_t.cpu().numpy()[nan]                      # keep both sides on the same NaN bits
        assert mismatches(bits(p16), want16) == 0


# ---------------------------------------------------------------------------------------------
# sharded step through torch.distributed (one rank here; two ranks are covered on CPU with gloo)
# ---------------------------------------------------------------------------------------------

def test_sharded_clipped_step_single_rank_nccl(env):
    import os
    import socket
    import torch.distributed as dist
    oracle, binding, synth, dev = env
    from paper_2502_20566_b200.dist import sharded_clipped_step
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=dev)
    try:
        n = 8 * 40000
        p, g, m, v = synth.adamw_state(n, 91, dev, g_dtype=torch.float32, outlier_fraction=0.01)
        pb, gb, mb, vb = bits(p), host_g(g), bits(m), bits(v)
        full = torch.empty(n, dtype=torch.bfloat16, device=dev)
        total = sharded_clipped_step(p, m, v, g, HP, 1234, 3, max_norm=1.0, accum_scale=0.125, full_param_out=full)
        torch.cuda.synchronize()
        S = oracle.sqnorm(gb)
        assert float(total.item()).hex() == S.hex()
        oracle.adamw_step(pb, gb, mb, vb, oracle.hparams(**HP), 1234, 3, 0, 0, oracle.clip_scale(S, 0.125, 1.0))
        assert mismatches(bits(p), pb) == 0 and mismatches(bits(full), pb) == 0
        assert mismatches(bits(m), mb) == 0 and mismatches(bits(v), vb) == 0
    finally:
        dist.destroy_process_group()


# ---------------------------------------------------------------------------------------------
# FP8 stochastic-rounding cast
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("dtype", [torch.float8_e4m3fn, torch.float8_e5m2])
@pytest.mark.parametrize("n,offset,shift", [(0, 0, 0), (3, 0, 0), (1 << 22, 0, 0), ((1 << 20) + 13, 16 * 77, 0), (70001, 5, 0),
                                            (70001, 32, 1), (5000, (1 << 34) - 64, 0)])
def test_fp8_cast_bit_exact(env, dtype, n, offset, shift):
    oracle, binding, synth, dev = env
    e5m2 = dtype == torch.float8_e5m2
    src = synth.downcast_mix(n + shift, 21, dev)[shift:]
    if n > 1000:                                   # most of the mix lies outside the FP8 range: add in-range values
        k = n // 2
        scale = torch.pow(10.0, torch.rand(k, device=dev, generator=torch.Generator(device=dev).manual_seed(4)) * 8 - 6)
        src[:k] = torch.randn(k, device=dev, generator=torch.Generator(device=dev).manual_seed(3)) * scale
    dst = torch.zeros(n + shift + 16, dtype=torch.uint8, device=dev).view(dtype)
    out = dst[shift:shift + n]
    binding.sr_downcast_f32_fp8(src, out, seed=(9 << 32) | 5, step=2, tensor_id=7, elem_offset=offset)
    torch.cuda.synchronize()
    want = oracle.sr_downcast_fp8(src.cpu().numpy().copy(), e5m2, (9 << 32) | 5, 2, 7, offset)
    got = out.view(torch.uint8).cpu().numpy()
    assert int(np.count_nonzero(got != want)) == 0
    assert int(dst.view(torch.uint8)[shift + n:].sum()) == 0 and int(dst.view(torch.uint8)[:shift].sum()) == 0
    if n > 1000:
        assert len(np.unique(got)) > 100           # the cast really spreads over the grid


def test_fp8_cast_is_unbiased_over_seeds(env):
    """Mean over 2048 seeds of 4096 in-range values: within 6 sigma of x, sigma^2 = Delta^2 f (1 - f) / seeds."""
    _, binding, _, dev = env
    k, seeds = 4096, 2048
    gen = torch.Generator(device=dev).manual_seed(11)
    x = (torch.rand(k, device=dev, generator=gen) * 2 - 1) * torch.pow(2.0, torch.rand(k, device=dev, generator=gen) * 12 - 6)
    for dtype in (torch.float8_e4m3fn, torch.float8_e5m2):
        outs = torch.empty((seeds, k), dtype=torch.uint8, device=dev).view(dtype)
        for s in range(seeds):
            binding.sr_downcast_f32_fp8(x, outs[s], seed=s)
        torch.cuda.synchronize()
        vals = outs.to(torch.float32).double()
        M, bias = (2, 15) if dtype == torch.float8_e5m2 else (3, 7)
        a = x.double().abs()
        eq = torch.clamp(torch.floor(torch.log2(a)), min=1 - bias)            # binade that sets the spacing
        delta = torch.exp2(eq - M)
        lo = torch.floor(a / delta) * delta
        f = (a - lo) / delta
        assert torch.all((vals.abs() == lo) | (vals.abs() == lo + delta))      # the two neighbouring levels only
        sigma = delta * torch.sqrt(f * (1 - f) / seeds)
        assert torch.all((vals.mean(dim=0) - x.double()).abs() <= 6 * sigma + 1e-300)


# ---------------------------------------------------------------------------------------------
# FP4 (E2M1) stochastic-rounding cast
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("n,offset,shift", [(0, 0, 0), (1, 0, 0), (3, 0, 0), (1 << 22, 0, 0), ((1 << 20) + 13, 16 * 77, 0),
                                            (70001, 5, 0), (70002, 32, 4), (70001, 48, 3), (5000, (1 << 34) - 64, 0)])
def test_fp4_cast_bit_exact(env, n, offset, shift):
    """shift moves the source by `shift` floats and the destination by `shift` bytes (unaligned buffers)."""
    oracle, binding, synth, dev = env
    src = synth.downcast_mix(n + shift, 23, dev)[shift:]
    if n > 1000:                                   # most of the mix lies outside the E2M1 range: add in-range values
        k = 3 * n // 4
        scale = torch.pow(10.0, torch.rand(k, device=dev, generator=torch.Generator(device=dev).manual_seed(4)) * 5 - 4)
        src[:k] = torch.randn(k, device=dev, generator=torch.Generator(device=dev).manual_seed(3)) * scale
    nbytes = (n + 1) // 2
    dst = torch.full((nbytes + shift + 16,), 0xEE, dtype=torch.uint8, device=dev)
    out = dst[shift:shift + nbytes]
    binding.sr_downcast_f32_fp4(src, out, seed=(9 << 32) | 5, step=2, tensor_id=7, elem_offset=offset)
    torch.cuda.synchronize()
    want = oracle.sr_downcast_fp4(src.cpu().numpy().copy(), (9 << 32) | 5, 2, 7, offset)
    got = out.cpu().numpy()
    assert int(np.count_nonzero(got != want)) == 0
    assert bool((dst[shift + nbytes:] == 0xEE).all()) and bool((dst[:shift] == 0xEE).all())   # nothing written outside
    if n > 1000:
        codes = np.concatenate([got & 0xF, got >> 4])
        assert len(np.unique(codes)) == 16         # every code of the grid occurs


def test_fp4_cast_is_unbiased_over_seeds(env):
    """Mean over 2048 seeds of 4096 values inside (-6, 6): within 6 sigma of x, sigma^2 = Delta^2 f (1 - f) / seeds."""
    _, binding, _, dev = env
    k, seeds = 4096, 2048
    gen = torch.Generator(device=dev).manual_seed(12)
    x = (torch.rand(k, device=dev, generator=gen) * 2 - 1) * 5.9 * torch.pow(2.0, -torch.rand(k, device=dev, generator=gen) * 6)
    outs = torch.empty((seeds, k // 2), dtype=torch.uint8, device=dev)
    for s in range(seeds):
        binding.sr_downcast_f32_fp4(x, outs[s], seed=s)
    torch.cuda.synchronize()
    table = torch.tensor([0, .5, 1, 1.5, 2, 3, 4, 6, -0.0, -.5, -1, -1.5, -2, -3, -4, -6], dtype=torch.float64, device=dev)
    codes = torch.stack([outs & 0xF, outs >> 4], dim=2).reshape(seeds, k).long()
    vals = table[codes]
    a = x.double().abs()
    eq = torch.clamp(torch.floor(torch.log2(a)), min=0)                       # binade that sets the spacing (bias 1)
    delta = torch.exp2(eq - 1)
    lo = torch.floor(a / delta) * delta
    f = (a - lo) / delta
    assert torch.all((vals.abs() == lo) | (vals.abs() == lo + delta))
    sigma = delta * torch.sqrt(f * (1 - f) / seeds)
    assert torch.all((vals.mean(dim=0) - x.double()).abs() <= 6 * sigma + 1e-300)


# ---------------------------------------------------------------------------------------------
# BF16 accumulation with stochastic rounding
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("g_dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("stochastic", [True, False])
@pytest.mark.parametrize("n,offset,shift", [(0, 0, 0), (5, 0, 0), (1 << 22, 0, 0), ((1 << 20) + 11, 8 * 123, 0), (70001, 5, 0),
                                            (70001, 64, 1), (4096, (1 << 36) - 1024, 0)])
def test_accumulate_bit_exact(env, g_dtype, stochastic, n, offset, shift):
    oracle, binding, synth, dev = env
    p, g, m, v = synth.adamw_state(n + shift, 57, dev, g_dtype=g_dtype, outlier_fraction=0.01)
    acc, g = m[shift:], g[shift:]                   # a BF16 accumulator of gradient-like magnitude
    if n > 100:
        acc[:8] = torch.tensor([0.0, -0.0, float("inf"), float("-inf"), float("nan"), 3.3895e38, 1e-40, 1.0], device=dev).bfloat16()
        g[:8] = torch.tensor([-0.0, 0.0, 1.0, float("inf"), 1.0, 3e38, 1e-40, -1.0], device=dev).to(g_dtype)
    want = bits(acc)
    gh = host_g(g)
    for micro in range(3):
        binding.sr_accumulate_bf16(acc, g, 0.25, seed=(3 << 32) | 77, step=10 + micro, tensor_id=5, elem_offset=offset,
                                   stochastic=stochastic)
        oracle.sr_accumulate(want, gh, 0.25, (3 << 32) | 77, 10 + micro, 5, offset, stochastic)
    torch.cuda.synchronize()
    assert mismatches(bits(acc), want) == 0
    if shift:
        assert mismatches(bits(m[:shift]), bits(synth.adamw_state(n + shift, 57, dev, g_dtype=g_dtype, outlier_fraction=0.01)[2][:shift])) == 0


def test_accumulate_stagnation_and_mean(env):
    """Section 2.1 on the device: terms of a quarter spacing never move a nearest-rounded accumulator; under
    stochastic rounding the mean over many accumulators follows the exact sum."""
    _, binding, _, dev = env
    n, steps, u = 1 << 16, 256, 2.0 ** -9
    g = torch.full((n,), u, dtype=torch.float32, device=dev)
    near = torch.ones(n, dtype=torch.bfloat16, device=dev)
    sr = torch.ones(n, dtype=torch.bfloat16, device=dev)
    for t in range(1, steps + 1):
        binding.sr_accumulate_bf16(near, g, 1.0, seed=5, step=t, stochastic=False)
        binding.sr_accumulate_bf16(sr, g, 1.0, seed=5, step=t, stochastic=True)
    torch.cuda.synchronize()
    assert bool((near == 1.0).all())
    vals = sr.double()
    sigma = (steps * (2.0 ** -7) ** 2 / 4) ** 0.5
    assert abs(float(vals.mean()) - (1.0 + steps * u)) < 6 * sigma / n ** 0.5
    assert float(vals.std()) > 0.2 * sigma


def test_accumulate_noise_is_disjoint_from_the_step(env):
    """The accumulation draws rounding slot 3, the step slots 0..2: with the same (seed, step, tensor_id) the
    up/down decisions of the two calls on identical fractions are not the same."""
    oracle, binding, _, dev = env
    n = 1 << 16
    x = torch.full((n,), 1.0 + 2.0 ** -9, dtype=torch.float32, device=dev)    # fraction 1/4 of a BF16 spacing
    cast = torch.empty(n, dtype=torch.bfloat16, device=dev)
    binding.sr_downcast_f32_bf16(x, cast, seed=8, step=4, tensor_id=1)       # slot 0
    acc = torch.ones(n, dtype=torch.bfloat16, device=dev)
    binding.sr_accumulate_bf16(acc, torch.full((n,), 2.0 ** -9, dtype=torch.float32, device=dev), 1.0, seed=8, step=4, tensor_id=1)
    torch.cuda.synchronize()
    up_cast, up_acc = (cast > 1.0), (acc > 1.0)
    assert abs(float(up_cast.float().mean()) - 0.25) < 0.02 and abs(float(up_acc.float().mean()) - 0.25) < 0.02
    both = float((up_cast & up_acc).float().mean())
    assert abs(both - 0.0625) < 0.01                                           # independent: P(both) = 1/16


def test_decisions_that_share_a_philox_call_are_independent(env):
    """The 2x2 tables of the oracle's joint-noise pin, taken from the device's outputs: elements that share
    a word or a call of one slot (through the cast and through the step), and the three slots of one
    element (through the step), at P(up) = 1/4 over 2^20 indices."""
    import joint
    _, binding, _, dev = env
    n = 1 << 20
    src = torch.full((n,), joint.QUARTER_F32_BITS, dtype=torch.int32, device=dev).view(torch.float32)
    dst = torch.empty(n, dtype=torch.bfloat16, device=dev)
    binding.sr_downcast_f32_bf16(src, dst, seed=11, step=3, tensor_id=2)
    torch.cuda.synchronize()
    up = joint.up_decisions(bits(dst), joint.QUARTER_DOWN)
    assert abs(up.mean() - 0.25) < 4 * np.sqrt(0.1875 / n)
    for name, (a, b) in joint.pair_tables(up).items():
        assert joint.chi2_independent_quarters(a, b) < joint.CHI2_3DOF_LIMIT, name

    st = joint.QUARTER_STEP_STATE_BITS
    p, g, m, v = (torch.full((n,), st[k], dtype=torch.int16, device=dev).view(torch.bfloat16) for k in ("p", "g", "m", "v"))
    binding.sr_adamw_step(p, g, m, v, binding.hparams(**joint.QUARTER_STEP_HP), (5 << 32) | 9, 1, 4)
    torch.cuda.synchronize()
    ups = {k: joint.up_decisions(bits(t), joint.QUARTER_STEP_DOWN[k]) for k, t in (("p", p), ("m", m), ("v", v))}
    for k, u in ups.items():
        assert abs(u.mean() - 0.25) < 4 * np.sqrt(0.1875 / n), k
        for name, (a, b) in joint.pair_tables(u).items():
            assert joint.chi2_independent_quarters(a, b) < joint.CHI2_3DOF_LIMIT, (k, name)
    for a, b in (("p", "m"), ("m", "v"), ("p", "v")):
        assert joint.chi2_independent_quarters(ups[a], ups[b]) < joint.CHI2_3DOF_LIMIT, (a, b)


# ---------------------------------------------------------------------------------------------
# exact zeros
# ---------------------------------------------------------------------------------------------

def _plant_zero_patterns(p, g, m, v, row=1024, seed=3):
    """Rows of `row` elements with the zero patterns that occur in training: gradient and both moments zero
    (a row no batch has touched), everything zero (padding), only the gradient zero, only one moment zero,
    and negative zeros in every combination that decides the sign of a zero result."""
    dev = p.device
    n = p.numel()
    rows = n // row
    gen = torch.Generator(device=dev).manual_seed(seed)
    kind = torch.randint(0, 12, (rows,), generator=gen, device=dev)
    view = lambda t: t[:rows * row].view(rows, row)
    P, G, M, V = view(p), view(g), view(m), view(v)
    neg0 = lambda t, sel: t.__setitem__(sel, torch.tensor(-0.0, dtype=t.dtype, device=dev))
    for t in (G, M, V):
        t[kind == 0] = 0                      # untouched row, x arbitrary
    for t in (P, G, M, V):
        t[kind == 1] = 0                      # padding
    G[kind == 2] = 0                          # gradient zero, state alive
    M[kind == 3] = 0
    G[kind == 3] = 0                          # m' = 0, v' > 0
    V[kind == 4] = 0
    G[kind == 4] = 0                          # v' = 0, m' != 0
    for t in (P, G, M):                       # x = -0, g = -0, m = -0, v = 0: the sign of every zero matters
        neg0(t, kind == 5)
    V[kind == 5] = 0
    neg0(M, kind == 6)                        # m = -0, g = +0, x = -0
    G[kind == 6] = 0
    neg0(P, kind == 6)
    neg0(M, kind == 7)                        # m = -0, g = -0, x = +0, v alive
    neg0(G, kind == 7)
    P[kind == 7] = 0
    # zeros scattered inside otherwise ordinary vectors
    sel = torch.rand(n, generator=gen, device=dev) < 0.02
    g[sel] = 0
    m[sel] = 0
    v[sel] = 0
    return int((kind <= 7).sum())


@pytest.mark.parametrize("kw", [HP, dict(HP, eps=0.0), dict(HP, eps=1e-10), dict(HP, eps=1.0, weight_decay=0.0),
                                dict(HP, lr=0.0), dict(HP, beta1=0.0, beta2=0.0)])
@pytest.mark.parametrize("g_dtype,flags,gscale,offset", [(torch.bfloat16, 7, 1.0, 0), (torch.float32, 7, 0.125, 8 * 31),
                                                        (torch.bfloat16, 15, 1.0, 0), (torch.bfloat16, 1, 1.0, 5)])
def test_exact_zeros_stay_bit_exact(env, kw, g_dtype, flags, gscale, offset):
    """Zero rows run the branch-free arithmetic when epsilon allows it (default reading, eps >= 2^-30) and the
    reference arithmetic otherwise; either way every bit, signs of zeros included, equals the oracle's."""
    _, _, synth, dev = env
    n = 300 * 1024 + 5
    p, g, m, v = synth.adamw_state(n, 21, dev, g_dtype=g_dtype)
    assert _plant_zero_patterns(p, g, m, v) > 100
    assert run_both(env, p, g, m, v, kw, seed=12, step=7, tensor_id=1, elem_offset=offset, gscale=gscale, flags=flags) == (0, 0, 0)
    assert run_both(env, p, g, m, v, kw, seed=12, step=8, tensor_id=1, elem_offset=offset, gscale=gscale, flags=flags) == (0, 0, 0)


def test_exact_zeros_in_the_tensor_list_and_the_master_recipe(env):
    oracle, binding, synth, dev = env
    sizes = [64 * 1024, 8192 + 24, 1024, 40 * 1024 + 8]
    P, G, M, V = [], [], [], []
    for i, n in enumerate(sizes):
        p, g, m, v = synth.adamw_state(n, 30 + i, dev)
        _plant_zero_patterns(p, g, m, v, seed=i)
        P.append(p); G.append(g); M.append(m); V.append(v)
    want = [[bits(t) for t in L] for L in (P, G, M, V)]
    plan = binding.sr_mt_plan_create(P, G, M, V)
    binding.sr_adamw_multi_tensor(plan, binding.hparams(**HP), 99, 3, 10)
    torch.cuda.synchronize()
    plan.destroy()
    for i in range(len(sizes)):
        oracle.adamw_step(want[0][i], want[1][i], want[2][i], want[3][i], oracle.hparams(**HP), 99, 3, 10 + i)
        assert [mismatches(bits(t[i]), want[k][i]) for k, t in ((0, P), (2, M), (3, V))] == [0, 0, 0]
    # FP32 master recipe: results are kept in FP32, so every sign of zero is visible
    n = 100 * 1024 + 3
    p, g, m, v = synth.adamw_state(n, 41, dev)
    _plant_zero_patterns(p, g, m, v)
    p32, m32, v32 = p.float(), m.float(), v.float()
    p16 = torch.empty(n, dtype=torch.bfloat16, device=dev)
    hp, ho = binding.hparams(**HP), oracle.hparams(**HP)
    po, mo, vo = (t.cpu().numpy().copy() for t in (p32, m32, v32))
    p16o = oracle.master_adamw_step(po, bits(g), mo, vo, ho, 5)
    binding.sr_master_adamw_step(p32, p16, g, m32, v32, hp, 5)
    torch.cuda.synchronize()
    for got, ref in ((p32, po), (m32, mo), (v32, vo)):
        assert np.array_equal(got.cpu().numpy().view(np.uint32), ref.view(np.uint32))
    assert mismatches(bits(p16), p16o) == 0


def test_long_launch_with_zero_rows(env):
    """The long-launch shape (2^29 elements and more) with a tenth of its 1024-element rows holding zero
    gradient and moments and some all-zero rows: every element compared."""
    oracle, binding, synth, dev = env
    n = (1 << 29) + 5 * 1024 + 77
    p, g, m, v = synth.adamw_state(n, 55, dev)
    rows = n // 1024
    gen = torch.Generator(device=dev).manual_seed(8)
    r = torch.rand(rows, generator=gen, device=dev)
    for t in (g, m, v):
        t[:rows * 1024].view(rows, 1024)[r < 0.10] = 0
    p[:rows * 1024].view(rows, 1024)[r < 0.02] = 0
    pre = [bits(t) for t in (p, g, m, v)]
    binding.sr_adamw_step(p, g, m, v, binding.hparams(**HP), 2024, 1000)
    torch.cuda.synchronize()
    oracle.adamw_step(*pre, oracle.hparams(**HP), 2024, 1000)
    assert [mismatches(bits(t), pre[k]) for k, t in ((0, p), (2, m), (3, v))] == [0, 0, 0]
