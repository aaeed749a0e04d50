"""B200-native fused SR-AdamW: BF16 parameters, gradients and moments, FP32 math in registers,
stochastic rounding on every downcast, behind the C-ABI library ``libsradamw.so``.

Submodules:
  binding  -- ctypes access to the C-ABI library (loads it on first use; fails loudly if absent)
  build    -- compiles the CUDA sources for sm_100a
  synth    -- seeded synthetic workloads (no optimizer arithmetic)
  dist     -- host-side helpers for several ranks (sharding, rank-ordered norm exchange)
  optim    -- SRAdamW, a torch.optim.Optimizer front end over the tensor-list step
"""

__all__ = ["binding", "build", "dist", "optim", "synth"]
