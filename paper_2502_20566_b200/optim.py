"""``torch.optim`` front end of the fused step: Algorithm 1 (AdamW on BF16 parameters with stochastically
rounded updates and a random state shared by all replicas) for a model whose parameters are BF16 CUDA tensors.

The class only marshals arguments: every parameter group becomes one tensor-list plan and one
``sr_adamw_multi_tensor`` launch per step.  Moments are BF16 (6 bytes of optimizer-side state per parameter
instead of the 14 of an FP32-master recipe).  The noise is a pure function of (seed, step, tensor id, element
index), so there is no generator state to fork, restore or checkpoint: replicas that hold the same seed stay
bit-identical, and ``state_dict`` / ``load_state_dict`` resume a run bit-exactly.
"""

from __future__ import annotations

from typing import Iterable, Optional

import torch

from . import binding


class SRAdamW(torch.optim.Optimizer):
    """AdamW with BF16 parameters, gradients and moments and stochastic rounding (Algorithm 1).

    params: BF16 CUDA parameters (or parameter groups); gradients may be BF16 or FP32, one type per group.
    sr_flags: which of x, m, v are rounded stochastically (``binding.SR_FLAG_SR_P | _M | _V``); 1 is the
        paper's update-only SR, 0 plain nearest rounding.
    eps_inside: the other reading of the update step, epsilon under the square root.
    seed: the shared random state; give every data-parallel replica the same value.
    max_norm: clip the global gradient norm (over all groups) to this value; the norm, the clipping factor and
        the step all stay on the device (``grad_sqnorm_multi_tensor`` -> ``sr_clip_scale`` -> step).
    Plans are cached by the data pointers of parameters, gradients and moments; creating one copies a table to
    the device and waits for it.  Keep gradient buffers in place between steps (``zero_grad(set_to_none=False)``)
    so that the plans are built once.
    ``step(grad_scale=...)`` multiplies the gradients by a host scalar (with clipping: the factor the norm is
    taken under, e.g. 1 / accumulation steps), ``step(grad_scale_dev=t)`` by a device scalar, without an extra
    pass over them.
    """

    def __init__(self, params: Iterable, lr: float = 1e-3, betas=(0.9, 0.999), eps: float = 1e-8,
                 weight_decay: float = 1e-2, seed: int = 0, sr_flags: int = binding.SR_FLAGS_DEFAULT,
                 eps_inside: bool = False, max_norm: Optional[float] = None):
        if lr < 0 or not 0 <= betas[0] < 1 or not 0 <= betas[1] < 1 or eps < 0:
            raise ValueError("invalid hyper-parameter")
        if sr_flags & ~7:
            raise ValueError("sr_flags: bits 0..2 only")
        defaults = dict(lr=lr, betas=tuple(betas), eps=eps, weight_decay=weight_decay)
        super().__init__(params, defaults)
        self.seed = int(seed)
        self.flags = int(sr_flags) | (binding.SR_FLAG_EPS_INSIDE if eps_inside else 0)
        self.max_norm = max_norm
        self._steps = 0
        self._plans = {}          # group index (or "all" for the norm) -> (key of data pointers, plan)
        self._clip = None         # device scalars and workspace of the clipped step
        binding.lib()             # fail here, not in the first step, when the CUDA library is missing
        for group in self.param_groups:
            for p in group["params"]:
                if not p.is_cuda or p.dtype != torch.bfloat16 or not p.is_contiguous():
                    raise TypeError("SRAdamW needs contiguous BF16 CUDA parameters")

    # the moments are created on first use so that load_state_dict can supply them instead
    def _moments(self, p: torch.Tensor):
        st = self.state[p]
        if "exp_avg" not in st:
            st["exp_avg"] = torch.zeros_like(p, memory_format=torch.contiguous_format)
            st["exp_avg_sq"] = torch.zeros_like(p, memory_format=torch.contiguous_format)
        return st["exp_avg"], st["exp_avg_sq"]

    def _plan(self, gi, group) -> Optional[binding.MtPlan]:
        P, G, M, V = [], [], [], []
        g_dtype = None
        for p in group["params"]:
            if p.grad is not None:
                if p.grad.is_sparse:
                    raise RuntimeError("SRAdamW does not support sparse gradients")
                g_dtype = g_dtype or p.grad.dtype
        if g_dtype is None:
            return None
        empty = None
        for p in group["params"]:
            g = p.grad
            if g is None:
                # keeps the tensor ids of the others unchanged: an entry of zero elements
                if empty is None:
                    empty = (torch.empty(0, dtype=torch.bfloat16, device=p.device), torch.empty(0, dtype=g_dtype, device=p.device))
                P.append(empty[0]); G.append(empty[1]); M.append(empty[0]); V.append(empty[0])
                continue
            m, v = self._moments(p)
            P.append(p.data); G.append(g if g.is_contiguous() else g.contiguous()); M.append(m); V.append(v)
        key = tuple(t.data_ptr() for ts in (P, G, M, V) for t in ts) + tuple(t.numel() for t in P)
        cached = self._plans.get(gi)
        if cached is None or cached[0] != key:
            if cached is not None:
                cached[1].destroy()
            cached = (key, binding.sr_mt_plan_create(P, G, M, V))
            self._plans[gi] = cached
        return cached[1]

    @torch.no_grad()
    def step(self, closure=None, grad_scale: float = 1.0, grad_scale_dev: Optional[torch.Tensor] = None):
        loss = None
        if closure is not None:
            with torch.enable_grad():
                loss = closure()
        self._steps += 1
        if self.max_norm is not None:
            if grad_scale_dev is not None:
                raise ValueError("max_norm computes the device scale itself")
            grad_scale_dev, grad_scale = self._clip_scale(grad_scale), 1.0
        base = 0
        for gi, group in enumerate(self.param_groups):
            plan = self._plan(gi, group)
            if plan is not None:
                hp = binding.hparams(lr=group["lr"], beta1=group["betas"][0], beta2=group["betas"][1], eps=group["eps"],
                                     weight_decay=group["weight_decay"], grad_scale=grad_scale,
                                     grad_scale_dev=grad_scale_dev, flags=self.flags)
                binding.sr_adamw_multi_tensor(plan, hp, self.seed, self._steps, tensor_id_base=base)
            base += len(group["params"])
        return loss

    def _clip_scale(self, accum_scale: float) -> Optional[torch.Tensor]:
        """Device scalar accum_scale * min(1, max_norm / (accum_scale * ||g|| + 1e-6)) over every gradient."""
        everything = dict(params=[p for group in self.param_groups for p in group["params"]])
        plan = self._plan("all", everything)
        if plan is None:
            return None
        need = binding.grad_sqnorm_multi_tensor_workspace_bytes(plan)
        if self._clip is None or self._clip[2].numel() * 8 < need:
            dev = plan.device
            self._clip = (torch.zeros(1, dtype=torch.float64, device=dev), torch.zeros(1, dtype=torch.float32, device=dev),
                          torch.empty(max(1, need // 8), dtype=torch.float64, device=dev))
        S, gs, ws = self._clip
        binding.grad_sqnorm_multi_tensor(plan, S, ws)
        binding.sr_clip_scale(S, accum_scale, self.max_norm, gs)
        return gs

    # ---- checkpointing: seed and step count are the whole random state -------------------------
    def state_dict(self):
        d = super().state_dict()
        d["sr"] = {"seed": self.seed, "steps": self._steps, "flags": self.flags}
        return d

    def load_state_dict(self, state_dict):
        sr = state_dict.get("sr")
        super().load_state_dict({k: v for k, v in state_dict.items() if k != "sr"})
        if sr is not None:
            self.seed, self._steps, self.flags = int(sr["seed"]), int(sr["steps"]), int(sr["flags"])
        for cached in self._plans.values():
            cached[1].destroy()
        self._plans = {}


class FlatSRAdamW(torch.optim.Optimizer):
    """The same update on flat buffers: every parameter group is packed into one contiguous BF16 buffer (each tensor
    starting on a multiple of 8 elements, the gaps zero), with flat buffers of the same layout for the gradients and
    both moments.  ``p.data`` and ``p.grad`` of every parameter become views into them, so autograd accumulates
    straight into the flat gradient buffer and one ``sr_adamw_step`` launch per group updates the whole model -- the
    launch shape the 6.7B-parameter measurement uses.  The groups' gradient buffers are slices of one buffer, so with
    ``max_norm`` the global norm is one ``grad_sqnorm`` call.

    Differences from ``SRAdamW``: the noise index runs over the flat buffer (tensor_id = group index), so the two
    classes round differently although both follow Algorithm 1; the class's ``zero_grad`` zeroes the flat buffer
    and keeps ``p.grad`` in place, and ``step`` repairs gradients that were moved or dropped by other code (one
    copy each; see ``_rebind``).
    """

    def __init__(self, params: Iterable, lr: float = 1e-3, betas=(0.9, 0.999), eps: float = 1e-8,
                 weight_decay: float = 1e-2, seed: int = 0, sr_flags: int = binding.SR_FLAGS_DEFAULT,
                 eps_inside: bool = False, max_norm: Optional[float] = None, grad_dtype: torch.dtype = torch.bfloat16):
        if lr < 0 or not 0 <= betas[0] < 1 or not 0 <= betas[1] < 1 or eps < 0:
            raise ValueError("invalid hyper-parameter")
        if sr_flags & ~7:
            raise ValueError("sr_flags: bits 0..2 only")
        if grad_dtype != torch.bfloat16:
            raise TypeError("autograd produces gradients of the parameters' type: BF16")
        super().__init__(params, dict(lr=lr, betas=tuple(betas), eps=eps, weight_decay=weight_decay))
        self.seed = int(seed)
        self.flags = int(sr_flags) | (binding.SR_FLAG_EPS_INSIDE if eps_inside else 0)
        self.max_norm = max_norm
        self._steps = 0
        binding.lib()
        self._flat = []           # per group: dict(p, g, m, v flat tensors, offsets)
        layouts = []
        for group in self.param_groups:
            ps = group["params"]
            for p in ps:
                if not p.is_cuda or p.dtype != torch.bfloat16 or not p.is_contiguous():
                    raise TypeError("FlatSRAdamW needs contiguous BF16 CUDA parameters")
            offsets, total = [], 0
            for p in ps:
                offsets.append(total)
                total += -(-p.numel() // 8) * 8          # every tensor starts on a multiple of 8 elements (16 bytes)
            layouts.append((offsets, total))
        dev = self.param_groups[0]["params"][0].device
        # one gradient buffer for all groups (each group a slice): the global norm is one grad_sqnorm call
        self._g_all = torch.zeros(sum(t for _, t in layouts), dtype=torch.bfloat16, device=dev)
        start = 0
        for group, (offsets, total) in zip(self.param_groups, layouts):
            flat = {k: torch.zeros(total, dtype=torch.bfloat16, device=dev) for k in ("p", "m", "v")}
            flat["g"] = self._g_all[start:start + total]
            start += total
            for p, off in zip(group["params"], offsets):
                n = p.numel()
                flat["p"][off:off + n].copy_(p.data.reshape(-1))
                p.data = flat["p"][off:off + n].view(p.shape)
                if p.grad is not None:
                    flat["g"][off:off + n].copy_(p.grad.reshape(-1))
                p.grad = flat["g"][off:off + n].view(p.shape)
            flat["offsets"] = offsets
            self._flat.append(flat)
        self._S = torch.zeros(1, dtype=torch.float64, device=dev)
        self._gs = torch.zeros(1, dtype=torch.float32, device=dev)
        need = binding.grad_sqnorm_workspace_bytes(self._g_all.numel())
        self._ws = torch.empty(max(1, need // 8), dtype=torch.float64, device=dev)

    def zero_grad(self, set_to_none: bool = False):
        self._g_all.zero_()

    def flat_buffers(self, group: int = 0):
        """(parameters, gradients, first moments, second moments) of one group as flat BF16 tensors."""
        f = self._flat[group]
        return f["p"], f["g"], f["m"], f["v"]

    def _rebind(self):
        """Host-side pointer check before every step (no synchronisation): the kernels read the flat buffers, so
        a gradient that autograd or user code put somewhere else (``model.zero_grad()`` sets ``p.grad`` to None
        and the next backward pass allocates a fresh tensor) is copied into its slice and ``p.grad`` is made a
        view of the slice again; a missing gradient counts as zero.  Parameters that no longer live in the flat
        buffer cannot be repaired silently and raise."""
        esize = 2
        for group, flat in zip(self.param_groups, self._flat):
            pbase, gbase = flat["p"].data_ptr(), flat["g"].data_ptr()
            for p, off in zip(group["params"], flat["offsets"]):
                n = p.numel()
                if p.data.data_ptr() != pbase + esize * off:
                    raise RuntimeError("FlatSRAdamW: a parameter's storage was replaced; it must stay a view of the flat buffer")
                g = p.grad
                if g is not None and g.data_ptr() == gbase + esize * off and g.dtype == torch.bfloat16:
                    continue
                piece = flat["g"][off:off + n]
                if g is None:
                    piece.zero_()
                else:
                    piece.copy_(g.reshape(-1))
                p.grad = piece.view(p.shape)

    @torch.no_grad()
    def step(self, closure=None, grad_scale: float = 1.0):
        loss = None
        if closure is not None:
            with torch.enable_grad():
                loss = closure()
        self._rebind()
        self._steps += 1
        gs_dev = None
        if self.max_norm is not None:
            binding.grad_sqnorm(self._g_all, self._S, self._ws)
            binding.sr_clip_scale(self._S, grad_scale, self.max_norm, self._gs)
            gs_dev, grad_scale = self._gs, 1.0
        for i, (group, flat) in enumerate(zip(self.param_groups, self._flat)):
            hp = binding.hparams(lr=group["lr"], beta1=group["betas"][0], beta2=group["betas"][1], eps=group["eps"],
                                 weight_decay=group["weight_decay"], grad_scale=grad_scale, grad_scale_dev=gs_dev,
                                 flags=self.flags)
            binding.sr_adamw_step(flat["p"], flat["g"], flat["m"], flat["v"], hp, self.seed, self._steps, tensor_id=i)
        return loss

    def state_dict(self):
        return {"sr": {"seed": self.seed, "steps": self._steps, "flags": self.flags},
                "flat": [{"m": f["m"].clone(), "v": f["v"].clone()} for f in self._flat],
                "param_groups": [{k: v for k, v in g.items() if k != "params"} for g in self.param_groups]}

    def load_state_dict(self, state_dict):
        sr = state_dict["sr"]
        self.seed, self._steps, self.flags = int(sr["seed"]), int(sr["steps"]), int(sr["flags"])
        for f, saved in zip(self._flat, state_dict["flat"]):
            f["m"].copy_(saved["m"])
            f["v"].copy_(saved["v"])
        for g, saved in zip(self.param_groups, state_dict["param_groups"]):
            g.update(saved)
