"""Pins for the oracle's AdamW arithmetic (Algorithm 1): every FP32 intermediate against correctly
rounded exact rational arithmetic, the per-iteration scalars against exact powers, closed forms and
special cases, a library AdamW as a loose bound, and the array driver (noise words, offsets,
flags, sharding)."""

import math
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from exact import (bits_f32, f32_bits, frac_of_bf16_bits, frac_of_f32_bits, frac_of_float, is_nan_bits,
                   round_to_f32, round_to_f32_bits)
from paper_2502_20566_b200 import synth

HP = dict(lr=6e-4, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.1)


def f32(x):
    return float(np.float32(x))


def test_round_helper_is_nearest():
    """The exact-rational rounding helper used below is itself checked: its result is a nearest
    FP32 value by exact comparison, and a few known casts."""
    rng = np.random.default_rng(0)
    for _ in range(2000):
        a = Fraction(int(rng.integers(-10**12, 10**12)), int(rng.integers(1, 10**9)))
        a *= Fraction(2) ** int(rng.integers(-160, 130))
        got = round_to_f32(a)
        # nearest means: the error is at most half the gap to either FP32 neighbour, decided exactly
        if math.isinf(got):
            assert abs(a) >= frac_of_f32_bits(0x7F7FFFFF)
            continue
        gq = frac_of_float(got)
        gb = f32_bits(got)
        mag = gb & 0x7FFFFFFF
        up = frac_of_f32_bits(mag + 1) if mag + 1 < 0x7F800000 else None
        dn = frac_of_f32_bits(mag - 1) if mag > 0 else None
        err = abs(abs(a) - abs(gq))
        if up is not None:
            assert err <= (up - abs(gq)) / 2
        if dn is not None:
            assert err <= (abs(gq) - dn) / 2
    assert round_to_f32(Fraction(1, 3)) == f32(1 / 3)
    assert round_to_f32(Fraction(16777217)) == 16777216.0          # tie to even
    assert round_to_f32(Fraction(16777219)) == 16777220.0


# ---------------------------------------------------------------------------------------------
# scalars (bias corrections of the m-hat / v-hat steps)
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("step", [1, 2, 3, 10, 17, 1000, 65537, 4_000_000_000])
def test_scalars_against_exact_powers(step):
    hp = oracle.hparams(**HP)
    sc = oracle.adamw_scalars(hp, step)
    b1, b2 = frac_of_float(f32(HP["beta1"])), frac_of_float(f32(HP["beta2"]))
    lr, wd = frac_of_float(f32(HP["lr"])), frac_of_float(f32(HP["weight_decay"]))
    if step <= 1000:
        bc1, bc2 = 1 - b1 ** step, 1 - b2 ** step
    else:
        bc1 = bc2 = Fraction(1)          # beta^t underflows far below 2^-53
    assert sc.one_minus_beta1 == round_to_f32(1 - b1) and sc.one_minus_beta2 == round_to_f32(1 - b2)
    assert sc.lr_wd == round_to_f32(lr * wd)
    want_step = lr / bc1
    assert abs(frac_of_float(sc.step_size) - want_step) <= want_step * Fraction(1, 1 << 23)
    got_r = frac_of_float(sc.rsqrt_bc2)
    # 1/sqrt(bc2) checked without a square root: got^2 * bc2 is 1 to FP32 accuracy
    assert abs(got_r * got_r * bc2 - 1) <= Fraction(1, 1 << 22)
    assert sc.beta1 == f32(HP["beta1"]) and sc.eps == f32(HP["eps"])


def test_scalars_step_size_is_double_division_rounded_once():
    hp = oracle.hparams(**HP)
    for step in (1, 5, 10, 100):
        sc = oracle.adamw_scalars(hp, step)
        b1 = frac_of_float(f32(HP["beta1"]))
        exact = frac_of_float(f32(HP["lr"])) / (1 - b1 ** step)
        # double arithmetic first (relative error <= a few 2^-53), then one cast: at most 1 FP32 ulp
        # from the exact quotient, and equal to it unless the quotient sits within 2^-50 of a tie
        assert f32_bits(sc.step_size) in {round_to_f32_bits(exact) + d for d in (-1, 0, 1)}


def test_step_zero_is_rejected():
    with pytest.raises(ValueError):
        oracle.adamw_scalars(oracle.hparams(**HP), 0)


# ---------------------------------------------------------------------------------------------
# element function: one correctly rounded operation per line
# ---------------------------------------------------------------------------------------------

def _is_correct_sqrt(s: float, v: float) -> bool:
    """s == RN(sqrt(v)) decided exactly: v lies between the squares of the midpoints around s."""
    if v == 0.0:
        return s == 0.0
    sb = f32_bits(s)
    sq = frac_of_float(s)
    lo_mid = (sq + frac_of_f32_bits(sb - 1)) / 2
    hi_mid = (sq + frac_of_f32_bits(sb + 1)) / 2
    vq = frac_of_float(v)
    return lo_mid * lo_mid <= vq <= hi_mid * hi_mid


def _check_trace(x, g, m, v, gscale, sc, t):
    F = frac_of_float
    assert t.g == round_to_f32(F(gscale) * F(g))
    assert t.a == round_to_f32(F(sc.one_minus_beta1) * F(t.g))
    assert t.m_new == round_to_f32(F(sc.beta1) * F(m) + F(t.a))                  # one rounding: fused
    assert t.b1 == round_to_f32(F(sc.one_minus_beta2) * F(t.g))
    assert t.b2 == round_to_f32(F(t.b1) * F(t.g))
    assert t.v_new == round_to_f32(F(sc.beta2) * F(v) + F(t.b2))
    if sc.eps_inside:
        assert t.s == round_to_f32(F(t.v_new) * F(sc.inv_bc2) + F(sc.eps))
        assert _is_correct_sqrt(t.den, t.s)
    else:
        assert _is_correct_sqrt(t.s, t.v_new)
        assert t.den == round_to_f32(F(t.s) * F(sc.rsqrt_bc2) + F(sc.eps))
    assert t.u == round_to_f32(F(t.m_new) / F(t.den))
    assert t.w == round_to_f32(F(sc.lr_wd) * F(x))
    assert t.q == round_to_f32(F(sc.step_size) * F(t.u) + F(t.w))
    assert t.x_new == round_to_f32(F(x) - F(t.q))


def test_element_function_against_exact_rational_arithmetic():
    rng = np.random.default_rng(3)
    hp = oracle.hparams(**HP)
    for step in (1, 10, 1000):
        sc = oracle.adamw_scalars(hp, step)
        for _ in range(150):
            x = float(torch.tensor(rng.normal(0, 0.02)).to(torch.bfloat16))
            g = float(torch.tensor(rng.normal(0, 1e-3)).to(torch.bfloat16))
            m = float(torch.tensor(rng.normal(0, 1e-4)).to(torch.bfloat16))
            v = float(torch.tensor(rng.normal(0, 1e-3) ** 2).to(torch.bfloat16))
            gscale = f32(rng.choice([1.0, 0.125, 0.0371]))
            t = oracle.adamw_element(x, g, m, v, gscale, sc)
            _check_trace(x, g, m, v, gscale, sc, t)


def test_element_function_with_fp32_gradients_and_tiny_values():
    """FP32 gradients (not BF16-representable) and values whose products fall into the subnormal
    range: no flush to zero anywhere."""
    rng = np.random.default_rng(4)
    sc = oracle.adamw_scalars(oracle.hparams(**HP), 7)
    for _ in range(150):
        x = float(torch.tensor(rng.normal(0, 0.02)).to(torch.bfloat16))
        g = f32(rng.normal(0, 1.0) * 10.0 ** rng.uniform(-22, 0))
        m = float(torch.tensor(rng.normal(0, 1.0) * 10.0 ** rng.uniform(-30, -3)).to(torch.bfloat16))
        v = float(torch.tensor(10.0 ** rng.uniform(-44, -5)).to(torch.bfloat16))
        t = oracle.adamw_element(x, g, m, v, 1.0, sc)
        _check_trace(x, g, m, v, 1.0, sc, t)
    t = oracle.adamw_element(0.5, 1e-20, 0.0, 0.0, 1.0, sc)
    assert t.b2 != 0.0 and t.b2 < 1.1754944e-38            # subnormal square survives
    _check_trace(0.5, f32(1e-20), 0.0, 0.0, 1.0, sc, t)


def test_first_step_from_zero_state_closed_form():
    """t = 1, m = v = 0: m-hat = g and sqrt(v-hat) = |g|, so the argument of Q_SR is
    x - alpha (g / (|g| + eps) + lambda x)."""
    hp = oracle.hparams(**HP)
    sc = oracle.adamw_scalars(hp, 1)
    rng = np.random.default_rng(5)
    for _ in range(200):
        x = float(torch.tensor(rng.normal(0, 0.02)).to(torch.bfloat16))
        g = float(torch.tensor(rng.normal(0, 1e-3)).to(torch.bfloat16))
        t = oracle.adamw_element(x, g, 0.0, 0.0, 1.0, sc)
        want = x - HP["lr"] * (g / (abs(g) + HP["eps"]) + HP["weight_decay"] * x)
        assert t.x_new == pytest.approx(want, rel=2e-6, abs=1e-9)
        # the bias-corrected direction is g / (|g| + eps): magnitude just under 1, sign of g
        assert sc.step_size * t.u == pytest.approx(HP["lr"] * g / (abs(g) + HP["eps"]), rel=1e-6)


# ---------------------------------------------------------------------------------------------
# the other reading of the update step: epsilon under the square root
# ---------------------------------------------------------------------------------------------

def test_eps_inside_scalar_and_exact_intermediates():
    rng = np.random.default_rng(31)
    for eps in (1e-8, 1e-6, 1e-3):
        hp = oracle.hparams(lr=6e-4, beta1=0.9, beta2=0.95, eps=eps, weight_decay=0.1, flags=oracle.SR_ALL | oracle.EPS_INSIDE)
        for step in (1, 10, 1000):
            sc = oracle.adamw_scalars(hp, step)
            assert sc.eps_inside == 1
            b2 = frac_of_float(f32(0.95))
            exact = 1 / (1 - b2 ** step)
            assert abs(frac_of_float(sc.inv_bc2) - exact) <= exact * Fraction(1, 1 << 23)      # one FP32 rounding of 1/(1-beta2^t)
            for _ in range(100):
                x = float(torch.tensor(rng.normal(0, 0.02)).to(torch.bfloat16))
                g = f32(rng.normal(0, 1.0) * 10.0 ** rng.uniform(-8, 0))
                m = float(torch.tensor(rng.normal(0, 1e-4)).to(torch.bfloat16))
                v = float(torch.tensor(10.0 ** rng.uniform(-20, -2)).to(torch.bfloat16))
                t = oracle.adamw_element(x, g, m, v, 1.0, sc)
                _check_trace(x, g, m, v, 1.0, sc, t)
    assert oracle.adamw_scalars(oracle.hparams(**HP), 5).eps_inside == 0


def test_eps_inside_first_step_closed_form_and_difference_from_default():
    """t = 1, m = v = 0: v-hat = g^2, so the direction is g / sqrt(g^2 + eps); for |g| << sqrt(eps) that is
    g / sqrt(eps), whereas the default reading gives g / (|g| + eps): the two readings are told apart."""
    eps = 1e-6
    kw = dict(lr=6e-4, beta1=0.9, beta2=0.95, eps=eps, weight_decay=0.1)
    inside = oracle.adamw_scalars(oracle.hparams(**kw, flags=oracle.SR_ALL | oracle.EPS_INSIDE), 1)
    outside = oracle.adamw_scalars(oracle.hparams(**kw), 1)
    rng = np.random.default_rng(32)
    for _ in range(200):
        x = float(torch.tensor(rng.normal(0, 0.02)).to(torch.bfloat16))
        g = float(torch.tensor(rng.normal(0, 1e-3)).to(torch.bfloat16))
        t = oracle.adamw_element(x, g, 0.0, 0.0, 1.0, inside)
        want = x - kw["lr"] * (g / math.sqrt(g * g + eps) + kw["weight_decay"] * x)
        assert t.x_new == pytest.approx(want, rel=2e-6, abs=1e-9)
    g = f32(1e-5)                                                   # |g| = 0.01 sqrt(eps)
    ti = oracle.adamw_element(0.0, g, 0.0, 0.0, 1.0, inside)
    to = oracle.adamw_element(0.0, g, 0.0, 0.0, 1.0, outside)
    assert inside.step_size * ti.u == pytest.approx(kw["lr"] * g / math.sqrt(eps), rel=1e-3)
    assert outside.step_size * to.u == pytest.approx(kw["lr"] * g / (g + eps), rel=1e-5)
    assert abs(to.u) > 50 * abs(ti.u)


def test_eps_inside_with_zero_eps_agrees_with_the_default_to_rounding():
    kw = dict(lr=6e-4, beta1=0.9, beta2=0.95, eps=0.0, weight_decay=0.0)
    rng = np.random.default_rng(33)
    for step in (1, 7, 300):
        a = oracle.adamw_scalars(oracle.hparams(**kw, flags=oracle.SR_ALL | oracle.EPS_INSIDE), step)
        b = oracle.adamw_scalars(oracle.hparams(**kw), step)
        for _ in range(100):
            g, m, v = f32(rng.normal(0, 1e-3)), f32(rng.normal(0, 1e-4)), f32(rng.normal(0, 1e-3) ** 2)
            ta, tb = oracle.adamw_element(0.1, g, m, v, 1.0, a), oracle.adamw_element(0.1, g, m, v, 1.0, b)
            assert ta.den == pytest.approx(tb.den, rel=4e-7) and ta.m_new == tb.m_new and ta.v_new == tb.v_new


def test_eps_inside_array_step_uses_the_flag():
    n = 4096
    p, g, m, v = synth.adamw_state(n, 12, "cpu")
    kw = dict(lr=6e-4, beta1=0.9, beta2=0.95, eps=1e-4, weight_decay=0.1)
    outs = []
    for flags in (oracle.SR_ALL, oracle.SR_ALL | oracle.EPS_INSIDE):
        pb, gb, mb, vb = (synth.bits16(t).copy() for t in (p, g, m, v))
        hp = oracle.hparams(**kw, flags=flags)
        oracle.adamw_step(pb, gb, mb, vb, hp, seed=3, step=4)
        sc = oracle.adamw_scalars(hp, 4)
        for i in range(0, n, 97):
            t = oracle.adamw_element(float(p[i]), float(g[i]), float(m[i]), float(v[i]), 1.0, sc)
            r = oracle.noise(3, 4, 0, i)
            assert pb[i] == oracle.sr_bf16_bits(f32_bits(t.x_new), r[0])
        outs.append((pb, mb, vb))
    assert not np.array_equal(outs[0][0], outs[1][0])               # x differs between the readings
    assert np.array_equal(outs[0][1], outs[1][1]) and np.array_equal(outs[0][2], outs[1][2])   # m, v do not


def test_zero_gradient_only_decays():
    sc = oracle.adamw_scalars(oracle.hparams(**HP), 10)
    x, m, v = 0.0625, 3.0517578125e-05, 9.5367431640625e-07
    t = oracle.adamw_element(x, 0.0, m, v, 1.0, sc)
    assert t.m_new == round_to_f32(frac_of_float(sc.beta1) * frac_of_float(m))
    assert t.v_new == round_to_f32(frac_of_float(sc.beta2) * frac_of_float(v))
    hp0 = oracle.hparams(lr=6e-4, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.1)
    sc0 = oracle.adamw_scalars(hp0, 10)
    t0 = oracle.adamw_element(x, 0.0, 0.0, 0.0, 1.0, sc0)          # no direction at all: pure decay
    assert t0.u == 0.0 and t0.x_new == round_to_f32(frac_of_float(x) - frac_of_float(round_to_f32(frac_of_float(sc0.lr_wd) * frac_of_float(x))))


def test_zero_learning_rate_leaves_parameters_bit_identical():
    n = 4096
    p, g, m, v = synth.adamw_state(n, 11, "cpu")
    pb, gb, mb, vb = (synth.bits16(t).copy() for t in (p, g, m, v))
    keep = pb.copy()
    hp = oracle.hparams(lr=0.0, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.0)
    oracle.adamw_step(pb, gb, mb, vb, hp, seed=3, step=4)
    not_negzero = keep != 0x8000
    assert np.array_equal(pb[not_negzero], keep[not_negzero])
    assert not np.array_equal(mb, synth.bits16(m))


def test_against_library_adamw_before_rounding():
    """torch.optim.AdamW in FP32 (epsilon outside the square root, bias-corrected, decoupled decay)
    agrees with the un-rounded FP32 results to FP32 accuracy: pins signs, terms and the epsilon
    placement to the optimizer the paper cites."""
    n, step = 2048, 10
    p, g, m, v = synth.adamw_state(n, 21, "cpu")
    pf, gf, mf, vf = (t.float() for t in (p, g, m, v))
    param = torch.nn.Parameter(pf.clone())
    opt = torch.optim.AdamW([param], lr=HP["lr"], betas=(HP["beta1"], HP["beta2"]), eps=HP["eps"],
                            weight_decay=HP["weight_decay"])
    param.grad = gf.clone()
    opt.state[param] = {"step": torch.tensor(float(step - 1)), "exp_avg": mf.clone(), "exp_avg_sq": vf.clone()}
    opt.step()
    sc = oracle.adamw_scalars(oracle.hparams(**HP), step)
    tr = [oracle.adamw_element(float(pf[i]), float(gf[i]), float(mf[i]), float(vf[i]), 1.0, sc) for i in range(n)]
    x_new = np.array([t.x_new for t in tr]); m_new = np.array([t.m_new for t in tr]); v_new = np.array([t.v_new for t in tr])
    st = opt.state[param]
    np.testing.assert_allclose(m_new, st["exp_avg"].numpy(), rtol=3e-6, atol=3e-10)   # atol: cancellation between the two terms
    np.testing.assert_allclose(v_new, st["exp_avg_sq"].numpy(), rtol=3e-6, atol=1e-14)
    # the update itself (x - x_new) to 1e-5 relative: far tighter than any dropped or misplaced term
    np.testing.assert_allclose(pf.numpy() - x_new, pf.numpy() - param.detach().numpy(), rtol=2e-4, atol=1.5e-8)   # atol: two FP32 ulps of x
    np.testing.assert_allclose(x_new, param.detach().numpy(), rtol=1e-6, atol=1e-9)


# ---------------------------------------------------------------------------------------------
# array driver
# ---------------------------------------------------------------------------------------------

def _compose_expected(pb, g_f32, mb, vb, hp, seed, step, tensor_id, offset, gscale, flags):
    sc = oracle.adamw_scalars(hp, step)
    out = []
    for i in range(len(pb)):
        F = lambda h: bits_f32(int(h) << 16)
        t = oracle.adamw_element(F(pb[i]), float(g_f32[i]), F(mb[i]), F(vb[i]), gscale, sc)
        idx = offset + i
        res = []
        for k, val in enumerate((t.x_new, t.m_new, t.v_new)):
            fb = f32_bits(val)
            number = 4 * (idx >> 3) + k
            w = oracle.philox4x32_10([number & 0xFFFFFFFF, number >> 32, tensor_id, seed >> 32], [seed & 0xFFFFFFFF, step])
            word = w[(idx & 7) >> 1]
            r = (word >> 16) if idx & 1 else (word & 0xFFFF)
            res.append(oracle.sr_bf16_bits(fb, r) if flags & (1 << k) else oracle.rne_bf16_bits(fb))
        out.append(res)
    return np.array(out, dtype=np.uint16)


@pytest.mark.parametrize("flags", [7, 1, 0, 5])
@pytest.mark.parametrize("g_dtype", [torch.bfloat16, torch.float32])
def test_array_step_is_element_function_plus_rounding(flags, g_dtype):
    n = 777
    p, g, m, v = synth.adamw_state(n, 31, "cpu", g_dtype=g_dtype)
    pb, mb, vb = (synth.bits16(t).copy() for t in (p, m, v))
    g_arr = g.numpy().copy() if g_dtype == torch.float32 else synth.bits16(g).copy()
    seed, step, tid, off, gscale = 0xDEADBEEF_00C0FFEE, 10, 5, (1 << 32) - 300, f32(0.37)
    hp = oracle.hparams(**HP, flags=flags)
    want = _compose_expected(pb, g.float().numpy(), mb, vb, hp, seed, step, tid, off, gscale, flags)
    oracle.adamw_step(pb, g_arr, mb, vb, hp, seed, step, tid, off, gscale)
    assert np.array_equal(pb, want[:, 0]) and np.array_equal(mb, want[:, 1]) and np.array_equal(vb, want[:, 2])


def test_shards_reproduce_the_whole_buffer():
    """Same random state on every rank: a buffer stepped in 8 contiguous shards (each told its
    global offset) equals the buffer stepped whole."""
    n = 8 * 1000 + 8
    p, g, m, v = synth.adamw_state(n, 41, "cpu")
    hp = oracle.hparams(**HP)
    whole = [synth.bits16(t).copy() for t in (p, g, m, v)]
    oracle.adamw_step(*whole, hp, seed=9, step=3, tensor_id=2)
    parts = [synth.bits16(t).copy() for t in (p, g, m, v)]
    bounds = np.linspace(0, n, 9).astype(int)
    for a, b in zip(bounds[:-1], bounds[1:]):
        sl = [np.ascontiguousarray(x[a:b]) for x in parts]
        oracle.adamw_step(*sl, hp, seed=9, step=3, tensor_id=2, elem_offset=int(a))
        for dst, src in zip(parts, sl):
            dst[a:b] = src
    for w, q in zip(whole, parts):
        assert np.array_equal(w, q)
    other = [synth.bits16(t).copy() for t in (p, g, m, v)]
    oracle.adamw_step(*other, hp, seed=10, step=3, tensor_id=2)
    assert not np.array_equal(other[0], whole[0])          # another seed rounds differently


def test_outputs_are_neighbours_of_the_fp32_result():
    n = 3000
    p, g, m, v = synth.adamw_state(n, 51, "cpu")
    pb, gb, mb, vb = (synth.bits16(t).copy() for t in (p, g, m, v))
    hp = oracle.hparams(**HP)
    sc = oracle.adamw_scalars(hp, 10)
    before = [pb.copy(), mb.copy(), vb.copy()]
    oracle.adamw_step(pb, gb, mb, vb, hp, seed=1234, step=10)
    ups = np.zeros(3)
    for i in range(n):
        F = lambda h: bits_f32(int(h) << 16)
        t = oracle.adamw_element(F(before[0][i]), F(gb[i]), F(before[1][i]), F(before[2][i]), 1.0, sc)
        for k, (val, got) in enumerate(zip((t.x_new, t.m_new, t.v_new), (pb[i], mb[i], vb[i]))):
            fb = f32_bits(val)
            assert int(got) in ((fb >> 16), (fb >> 16) + 1)
            ups[k] += int(got) != (fb >> 16)
    assert np.all(ups > 0.3 * n) and np.all(ups < 0.7 * n)  # rounding really is stochastic


def test_sr_downcast_array_and_offsets():
    src = synth.downcast_mix(5000, 7, "cpu").numpy()
    out = oracle.sr_downcast(src, seed=7)
    b = src.view(np.uint32)
    for i in range(0, 5000, 7):
        w = oracle.philox4x32_10([4 * (i >> 3), 0, 0, 0], [7, 0])[(i & 7) >> 1]
        assert out[i] == oracle.sr_bf16_bits(int(b[i]), (w >> 16) if i & 1 else (w & 0xFFFF))
    shifted = oracle.sr_downcast(np.ascontiguousarray(src[1000:2000]), seed=7, elem_offset=1000)
    assert np.array_equal(shifted, out[1000:2000])
    nan = is_nan_bits_array(b)
    assert np.all(out[nan] == 0x7FC0)
    lo = (b >> 16).astype(np.int64)
    assert np.all((out[~nan].astype(np.int64) - lo[~nan] >= 0) & (out[~nan].astype(np.int64) - lo[~nan] <= 1))


def is_nan_bits_array(b):
    return (b & 0x7FFFFFFF) > 0x7F800000


def test_master_recipe_tracks_library_adamw_over_several_steps():
    """FP32-master recipe (the paper's mixed-precision comparison): eight consecutive steps stay within
    FP32 rounding of torch.optim.AdamW, and the BF16 copy is the nearest-rounded parameter."""
    n = 4096
    p0, _, _, _ = synth.adamw_state(n, 61, "cpu")
    p = p0.float().numpy().copy()
    m = np.zeros(n, dtype=np.float32)
    v = np.zeros(n, dtype=np.float32)
    param = torch.nn.Parameter(torch.from_numpy(p.copy()))
    opt = torch.optim.AdamW([param], lr=HP["lr"], betas=(HP["beta1"], HP["beta2"]), eps=HP["eps"],
                            weight_decay=HP["weight_decay"])
    hp = oracle.hparams(**HP)
    for step in range(1, 9):
        g = synth.state_chunk(synth.ROLE_G, 600 + step, 0, n, "cpu", g_dtype=torch.float32)
        param.grad = g.clone()
        opt.step()
        p16 = oracle.master_adamw_step(p, g.numpy().copy(), m, v, hp, step)
        np.testing.assert_allclose(p, param.detach().numpy(), rtol=2e-6, atol=2e-8)
        want16 = torch.from_numpy(p.copy()).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
        assert np.array_equal(p16, want16)
    st = opt.state[param]
    np.testing.assert_allclose(m, st["exp_avg"].numpy(), rtol=2e-5, atol=1e-9)
    np.testing.assert_allclose(v, st["exp_avg_sq"].numpy(), rtol=2e-5, atol=1e-13)


def test_master_recipe_is_the_element_function():
    n = 333
    p0, g, m0, v0 = synth.adamw_state(n, 62, "cpu")
    p, m, v = (t.float().numpy().copy() for t in (p0, m0, v0))
    before = (p.copy(), m.copy(), v.copy())
    hp = oracle.hparams(**HP)
    sc = oracle.adamw_scalars(hp, 5)
    gb = synth.bits16(g).copy()
    p16 = oracle.master_adamw_step(p, gb, m, v, hp, 5, gscale=f32(0.25))
    for i in range(n):
        t = oracle.adamw_element(float(before[0][i]), float(g[i]), float(before[1][i]), float(before[2][i]), f32(0.25), sc)
        assert (p[i], m[i], v[i]) == (t.x_new, t.m_new, t.v_new)
        assert p16[i] == oracle.rne_bf16_bits(f32_bits(t.x_new))


# ---------------------------------------------------------------------------------------------
# squared norm and clipping
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("n", [0, 1, 5, 1023, 8192, 8193, 100000, 8192 * 8192 // 64 + 77])
def test_sqnorm_is_exact_on_integer_data(n):
    rng = np.random.default_rng(n)
    g = rng.integers(-64, 65, n).astype(np.float32)          # squares and all partial sums are exact
    want = int((g.astype(np.int64) ** 2).sum())
    assert oracle.sqnorm(g) == float(want)
    gb = synth.bits16(torch.from_numpy(g).to(torch.bfloat16))
    assert oracle.sqnorm(gb.copy()) == float(want)


def test_sqnorm_is_accurate_on_random_data_and_order_sensitive_data():
    rng = np.random.default_rng(6)
    g = (rng.normal(0, 1e-3, 300001) * np.where(rng.random(300001) < 0.01, 1000.0, 1.0)).astype(np.float32)
    exact = math.fsum((g.astype(np.float64) ** 2).tolist())
    assert oracle.sqnorm(g) == pytest.approx(exact, rel=1e-14)
    # the first pass squares, later passes do not
    terms = rng.random(20000)
    assert oracle.tree_sum(terms) == pytest.approx(math.fsum(terms.tolist()), rel=1e-14)
    assert oracle.tree_sum(np.array([3.5])) == 3.5


def test_clip_scale_closed_forms():
    # below the threshold: only the accumulation factor remains
    assert oracle.clip_scale(4.0, 0.125, 1.0) == 0.125            # norm = 0.25 < 1
    # above: accum * max_norm / (accum * sqrt(S) + 1e-6)
    got = oracle.clip_scale(1.0e6, 0.125, 1.0)                    # norm = 125
    assert got == f32(0.125 * (1.0 / (125.0 + 1e-6)))
    assert oracle.clip_scale(0.0, 1.0, 1.0) == 1.0
    # scaled gradient has norm max_norm (up to the 1e-6 guard)
    S = 7.3e4
    gs = oracle.clip_scale(S, 0.25, 2.0)
    assert gs * math.sqrt(S) == pytest.approx(2.0, rel=1e-6)


def test_list_norm_reduces_to_the_flat_norm_and_is_exact_on_integers():
    """Pins for the list form of the squared norm: one tensor gives the flat routine's bits; tensors whose
    lengths are multiples of 8192 give the bits of their concatenation; integer data give the exact sum."""
    rng = np.random.default_rng(40)
    a = rng.normal(0, 1e-3, 3 * 8192).astype(np.float32)
    b = rng.normal(0, 1.0, 8192).astype(np.float32)
    c = rng.normal(0, 1e-2, 20000).astype(np.float32)
    assert oracle.sqnorm_list([c]).hex() == oracle.sqnorm(c).hex()
    assert oracle.sqnorm_list([a, b, c]).hex() == oracle.sqnorm(np.concatenate([a, b, c])).hex()
    ints = [rng.integers(-50, 50, n).astype(np.float32) for n in (5, 8192, 8193, 1, 0, 30000)]
    assert oracle.sqnorm_list(ints) == float(sum(int((x.astype(np.int64) ** 2).sum()) for x in ints))
    assert oracle.sqnorm_list([]) == 0.0 and oracle.sqnorm_list([np.zeros(0, np.float32)]) == 0.0
    bf = [(x.view(np.uint32) >> 16).astype(np.uint16) for x in (a, c)]
    want = sum(float(v) ** 2 for x in bf for v in (x.astype(np.uint32) << 16).view(np.float32).astype(np.float64))
    assert oracle.sqnorm_list(bf) == pytest.approx(want, rel=1e-12)
