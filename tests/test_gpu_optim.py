"""The torch.optim front end on a GPU: bit-exact against the oracle, the paper's qualitative claim on a
synthetic regression (BF16 + stochastic rounding follows FP32 AdamW where BF16 + nearest rounding stagnates,
Section 2.1), and bit-exact resume from a checkpoint."""

import copy

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    import oracle
    from paper_2502_20566_b200 import binding, optim, synth
    binding.lib()
    return oracle, binding, optim, synth, torch.device("cuda", 0)


def bits(t):
    return t.detach().view(torch.int16).cpu().numpy().view(np.uint16).copy()


def test_optimizer_step_is_the_oracle_step(env):
    oracle, binding, optim, synth, dev = env
    sizes = [(300, 70), (70,), (8192,), (1,), (129, 64)]
    gen = torch.Generator(device=dev).manual_seed(1)
    params = [torch.nn.Parameter((torch.randn(s, device=dev, generator=gen) * 0.05).bfloat16()) for s in sizes]
    groups = [dict(params=params[:3], weight_decay=0.1), dict(params=params[3:], weight_decay=0.0, lr=3e-4)]
    opt = optim.SRAdamW(groups, lr=6e-4, betas=(0.9, 0.95), eps=1e-8, seed=(5 << 32) | 9)
    host = [dict(p=bits(p).reshape(-1), m=np.zeros(p.numel(), np.uint16), v=np.zeros(p.numel(), np.uint16)) for p in params]
    for step in (1, 2, 3):
        for i, p in enumerate(params):
            p.grad = None if (step == 2 and i == 1) else (torch.randn(p.shape, device=dev, generator=gen) * 1e-3).bfloat16()
        opt.step(grad_scale=0.5)
        torch.cuda.synchronize()
        for i, p in enumerate(params):
            if p.grad is None:
                continue
            kw = dict(lr=6e-4 if i < 3 else 3e-4, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.1 if i < 3 else 0.0)
            h = host[i]
            oracle.adamw_step(h["p"], bits(p.grad).reshape(-1), h["m"], h["v"], oracle.hparams(**kw), (5 << 32) | 9, step, i, 0, 0.5)
            assert np.array_equal(bits(p).reshape(-1), h["p"])
            assert np.array_equal(bits(opt.state[p]["exp_avg"]).reshape(-1), h["m"])
            assert np.array_equal(bits(opt.state[p]["exp_avg_sq"]).reshape(-1), h["v"])


def _regression(dev):
    gen = torch.Generator(device=dev).manual_seed(7)
    d, n = 256, 2048
    X = torch.randn(n, d, device=dev, generator=gen)
    w_star = torch.randn(d, device=dev, generator=gen)
    w_star = torch.where(w_star.abs() < 0.5, w_star.sign() * 0.5 - w_star, w_star)      # |w*| >= 0.5: coarse BF16 spacing
    y = X @ w_star
    w0 = (w_star + 0.05 * torch.randn(d, device=dev, generator=gen)).bfloat16().float()
    return X, y, w_star, w0


def _train(make_opt, w0, X, y, dtype, steps=400):
    w = torch.nn.Parameter(w0.to(dtype).clone())
    opt = make_opt([w])
    for _ in range(steps):
        r = X @ w.detach().float() - y
        w.grad = (X.t() @ r / X.shape[0]).to(dtype)
        opt.step()
    return w.detach().float()


def test_sr_follows_fp32_where_nearest_rounding_stagnates(env):
    """Updates of about lr = 5e-4 per step are far below half a BF16 spacing (2^-9 .. 2^-8 for these weights):
    nearest rounding discards them, stochastic rounding applies them in expectation."""
    _, binding, optim, _, dev = env
    X, y, w_star, w0 = _regression(dev)
    kw = dict(lr=5e-4, betas=(0.9, 0.95), eps=1e-8, weight_decay=0.0)
    err = lambda w: float((w - w_star).norm())
    e0 = err(w0)
    e_fp32 = err(_train(lambda ps: torch.optim.AdamW(ps, **kw), w0, X, y, torch.float32))
    e_sr = err(_train(lambda ps: optim.SRAdamW(ps, seed=3, **kw), w0, X, y, torch.bfloat16))
    e_near = err(_train(lambda ps: optim.SRAdamW(ps, seed=3, sr_flags=0, **kw), w0, X, y, torch.bfloat16))
    assert e_fp32 < 0.2 * e0
    assert e_sr < 0.35 * e0                      # SR gets most of the way (its floor is the BF16 spacing)
    assert e_near > 0.8 * e0                     # nearest rounding hardly moves
    assert e_sr < 0.4 * e_near


def test_resume_from_checkpoint_is_bit_exact(env):
    _, binding, optim, _, dev = env
    gen = torch.Generator(device=dev).manual_seed(11)
    shapes = [(64, 33), (33,), (4097,)]
    init = [(torch.randn(s, device=dev, generator=gen) * 0.05).bfloat16() for s in shapes]
    grads = [[(torch.randn(s, device=dev, generator=gen) * 1e-3).bfloat16() for s in shapes] for _ in range(6)]

    def run(params, opt, steps):
        for t in steps:
            for p, g in zip(params, grads[t]):
                p.grad = g.clone()
            opt.step()

    a = [torch.nn.Parameter(t.clone()) for t in init]
    opt_a = optim.SRAdamW(a, lr=1e-3, betas=(0.9, 0.95), seed=42)
    run(a, opt_a, range(6))
    b = [torch.nn.Parameter(t.clone()) for t in init]
    opt_b = optim.SRAdamW(b, lr=1e-3, betas=(0.9, 0.95), seed=42)
    run(b, opt_b, range(3))
    saved = copy.deepcopy(opt_b.state_dict())
    weights = [p.detach().clone() for p in b]
    c = [torch.nn.Parameter(t.clone()) for t in weights]
    opt_c = optim.SRAdamW(c, lr=1e-3, betas=(0.9, 0.95), seed=0)          # the seed comes from the checkpoint
    opt_c.load_state_dict(saved)
    run(c, opt_c, range(3, 6))
    torch.cuda.synchronize()
    for pa, pc in zip(a, c):
        assert np.array_equal(bits(pa), bits(pc))
        assert np.array_equal(bits(opt_a.state[pa]["exp_avg_sq"]), bits(opt_c.state[pc]["exp_avg_sq"]))


@pytest.mark.parametrize("g_dtype", [torch.float32, torch.bfloat16])
def test_list_norm_bit_exact(env, g_dtype):
    """grad_sqnorm_multi_tensor against the oracle on lists with ragged, empty, tiny and unaligned tensors; a
    list of one tensor equals grad_sqnorm."""
    oracle, binding, _, synth, dev = env
    rng = np.random.default_rng(3)
    sizes = [1, 5, 8192, 8193, 0, 3 * 8192, 70001, 17, 2 * 8192 + 9] + [int(x) for x in rng.integers(1, 40000, 60)]
    P, G, M, V = [], [], [], []
    for i, n in enumerate(sizes):
        shift = 1 if i % 7 == 2 else 0
        p, g, m, v = synth.adamw_state(n + shift, 300 + i, dev, g_dtype=g_dtype, outlier_fraction=0.01)
        P.append(p[shift:]); G.append(g[shift:]); M.append(m[shift:]); V.append(v[shift:])
    plan = binding.sr_mt_plan_create(P, G, M, V)
    ws = torch.empty(max(1, binding.grad_sqnorm_multi_tensor_workspace_bytes(plan) // 8), dtype=torch.float64, device=dev)
    S = torch.zeros(1, dtype=torch.float64, device=dev)
    host = [g.cpu().numpy().copy() if g_dtype == torch.float32 else bits(g) for g in G]
    for _ in range(2):
        binding.grad_sqnorm_multi_tensor(plan, S, ws)
        torch.cuda.synchronize()
        assert float(S.item()).hex() == oracle.sqnorm_list(host).hex()
    plan.destroy()
    one = binding.sr_mt_plan_create(P[6:7], G[6:7], M[6:7], V[6:7])
    ws1 = torch.empty(max(1, binding.grad_sqnorm_multi_tensor_workspace_bytes(one) // 8), dtype=torch.float64, device=dev)
    S1, S2 = torch.zeros(1, dtype=torch.float64, device=dev), torch.zeros(1, dtype=torch.float64, device=dev)
    binding.grad_sqnorm_multi_tensor(one, S1, ws1)
    ws2 = torch.empty(max(1, binding.grad_sqnorm_workspace_bytes(sizes[6]) // 8), dtype=torch.float64, device=dev)
    binding.grad_sqnorm(G[6], S2, ws2)
    torch.cuda.synchronize()
    assert float(S1.item()).hex() == float(S2.item()).hex()
    one.destroy()
    empty = binding.sr_mt_plan_create([], [], [], [])
    binding.grad_sqnorm_multi_tensor(empty, S, None)
    torch.cuda.synchronize()
    assert float(S.item()) == 0.0


def test_clipped_optimizer_step_is_the_oracle_sequence(env):
    oracle, binding, optim, synth, dev = env
    gen = torch.Generator(device=dev).manual_seed(21)
    shapes = [(500, 40), (40,), (9000,), (3,)]
    params = [torch.nn.Parameter((torch.randn(s, device=dev, generator=gen) * 0.05).bfloat16()) for s in shapes]
    groups = [dict(params=params[:2], weight_decay=0.1), dict(params=params[2:], weight_decay=0.0)]
    opt = optim.SRAdamW(groups, lr=6e-4, betas=(0.9, 0.95), seed=77, max_norm=0.5)
    host = [dict(p=bits(p).reshape(-1), m=np.zeros(p.numel(), np.uint16), v=np.zeros(p.numel(), np.uint16)) for p in params]
    for step in (1, 2):
        for p in params:
            p.grad = (torch.randn(p.shape, device=dev, generator=gen) * (0.02 if step == 1 else 1e-4)).bfloat16()   # clipped, then not
        opt.step(grad_scale=0.25)
        torch.cuda.synchronize()
        gh = [bits(p.grad).reshape(-1) for p in params]
        S = oracle.sqnorm_list(gh)
        gscale = oracle.clip_scale(S, 0.25, 0.5)
        assert (gscale < 0.25) == (step == 1)
        for i, p in enumerate(params):
            kw = dict(lr=6e-4, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.1 if i < 2 else 0.0)
            h = host[i]
            oracle.adamw_step(h["p"], gh[i], h["m"], h["v"], oracle.hparams(**kw), 77, step, i, 0, gscale)
            assert np.array_equal(bits(p).reshape(-1), h["p"])
            assert np.array_equal(bits(opt.state[p]["exp_avg"]).reshape(-1), h["m"])


def test_flat_optimizer_is_the_oracle_on_the_flat_buffers_and_trains_through_autograd(env):
    """FlatSRAdamW: parameters and gradients become views of flat buffers; autograd writes into the flat gradient
    buffer; each step equals norm -> clip -> oracle step on the flat buffers (two groups, padding between tensors)."""
    oracle, binding, optim, synth, dev = env
    torch.manual_seed(0)
    model = torch.nn.Sequential(torch.nn.Linear(37, 53), torch.nn.Tanh(), torch.nn.Linear(53, 11)).to(dev).bfloat16()
    decay = [p for p in model.parameters() if p.dim() > 1]
    no_decay = [p for p in model.parameters() if p.dim() == 1]
    opt = optim.FlatSRAdamW([dict(params=decay, weight_decay=0.1), dict(params=no_decay, weight_decay=0.0)], lr=1e-3,
                            betas=(0.9, 0.95), seed=31, max_norm=0.05)
    for p in model.parameters():
        assert p.data_ptr() % 16 == 0 and p.grad is not None
    x = torch.randn(256, 37, device=dev).bfloat16()
    y = torch.randn(256, 11, device=dev).bfloat16()
    host = []
    for gi in range(2):
        fp, fg, fm, fv = opt.flat_buffers(gi)
        host.append([bits(fp), None, bits(fm), bits(fv)])
    losses = []
    for step in (1, 2, 3):
        opt.zero_grad()
        loss = torch.nn.functional.mse_loss(model(x).float(), y.float())
        loss.backward()
        losses.append(float(loss.detach()))
        g_all = np.concatenate([bits(opt.flat_buffers(gi)[1]) for gi in range(2)])
        assert np.count_nonzero(g_all) > g_all.size // 2                      # autograd really wrote into the flat buffer
        opt.step(grad_scale=1.0)
        torch.cuda.synchronize()
        gscale = oracle.clip_scale(oracle.sqnorm(g_all), 1.0, 0.05)
        for gi, wd in ((0, 0.1), (1, 0.0)):
            fp, fg, fm, fv = opt.flat_buffers(gi)
            h = host[gi]
            oracle.adamw_step(h[0], bits(fg), h[2], h[3], oracle.hparams(lr=1e-3, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=wd),
                              31, step, gi, 0, gscale)
            assert np.array_equal(bits(fp), h[0]) and np.array_equal(bits(fm), h[2]) and np.array_equal(bits(fv), h[3])
    assert losses[2] < losses[0]                                              # the model views see the updates
    # resume: parameters + state_dict saved after step 3; step 4 taken twice from that point gives the same bits
    saved = opt.state_dict()
    assert saved["sr"]["steps"] == 3
    params_saved = [opt.flat_buffers(gi)[0].clone() for gi in range(2)]

    def fourth_step():
        opt.zero_grad()
        torch.nn.functional.mse_loss(model(x).float(), y.float()).backward()
        opt.step()
        torch.cuda.synchronize()
        return [bits(opt.flat_buffers(gi)[k]) for gi in range(2) for k in (0, 2, 3)]

    first = fourth_step()
    for gi in range(2):
        opt.flat_buffers(gi)[0].copy_(params_saved[gi])
    opt.load_state_dict(saved)
    second = fourth_step()
    assert all(np.array_equal(a, b) for a, b in zip(first, second))


def test_flat_optimizer_survives_model_zero_grad(env):
    """``model.zero_grad()`` drops every ``p.grad``; the next backward pass allocates gradients outside the flat
    buffer.  The step must see them all the same: two models trained in lock-step, one cleared through the
    optimizer and one through the model, stay bit-identical, and the gradients are views of the flat buffer again."""
    _, _, optim, _, dev = env
    x = torch.randn(64, 19, device=dev).bfloat16()
    y = torch.randn(64, 5, device=dev).bfloat16()
    runs = []
    for clear_through_model in (False, True):
        torch.manual_seed(3)
        model = torch.nn.Sequential(torch.nn.Linear(19, 33), torch.nn.Tanh(), torch.nn.Linear(33, 5)).to(dev).bfloat16()
        opt = optim.FlatSRAdamW(model.parameters(), lr=1e-3, betas=(0.9, 0.95), seed=7, max_norm=1.0)
        for step in range(3):
            if clear_through_model:
                model.zero_grad()                       # set_to_none=True by default
                assert all(p.grad is None for p in model.parameters())
            else:
                opt.zero_grad()
            torch.nn.functional.mse_loss(model(x).float(), y.float()).backward()
            if clear_through_model and step == 2:
                list(model.parameters())[1].grad = None     # a parameter without a gradient counts as zero
            elif step == 2:
                list(model.parameters())[1].grad.zero_()
            opt.step()
        torch.cuda.synchronize()
        fp, fg, _, _ = opt.flat_buffers(0)
        for p in model.parameters():
            assert fg.data_ptr() <= p.grad.data_ptr() < fg.data_ptr() + 2 * fg.numel()
        runs.append([bits(t) for t in opt.flat_buffers(0)])
    assert all(np.array_equal(a, b) for a, b in zip(*runs))
    assert np.count_nonzero(runs[0][2]) > 0
