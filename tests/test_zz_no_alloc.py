"""grad_sqnorm_static: the squared norm for callers that are not allowed to allocate device memory
(their memory belongs to someone else's pool, or they sit in a loop where an allocation is
forbidden).  Its scratch is a fixed array inside the library, shared by all calls on a GPU and never
cleared, so this test calls it twice in a row, with different data and sizes, and requires the same
bits as grad_sqnorm with a caller-provided workspace each time.  Collected last on purpose."""

import ctypes

import pytest
import torch

pytestmark = pytest.mark.gpu


def test_static_scratch_norm_equals_workspace_norm_twice_in_a_row():
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    from paper_2502_20566_b200 import binding, synth
    dev = torch.device("cuda", 0)
    L = binding.lib()
    assert binding.grad_sqnorm_static_max_elements() == 1_073_610_752
    cases = [((1 << 26) + 12345, torch.float32, 71),     # 8194 block sums, then 2, then 1
             (3 * 8192 + 5, torch.bfloat16, 72),         # fewer block sums than the call before left behind
             (5000, torch.float32, 73)]                  # single block: scratch unused
    for n, dtype, seed in cases:
        g = torch.empty(n, dtype=dtype, device=dev)
        synth.fill_state(g, synth.ROLE_G, seed, outlier_fraction=0.01)
        ws = torch.empty(max(1, binding.grad_sqnorm_workspace_bytes(n) // 8), dtype=torch.float64, device=dev)
        want = torch.full((1,), -1.0, dtype=torch.float64, device=dev)
        got = torch.full((1,), -2.0, dtype=torch.float64, device=dev)
        binding.grad_sqnorm(g, want, ws)
        # through the C ABI, raw pointers only; the call itself must not allocate
        torch.cuda.synchronize()
        before = torch.cuda.memory_allocated(dev)
        st = L.grad_sqnorm_static(g.data_ptr(), binding.SR_DT_F32 if dtype == torch.float32 else binding.SR_DT_BF16,
                                  n, got.data_ptr(), ctypes.c_void_p(torch.cuda.current_stream().cuda_stream))
        assert st == binding.SR_OK
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated(dev) == before
        assert float(got.item()).hex() == float(want.item()).hex()      # bit-equal, the tolerance of the other tests
        assert float(want.item()) > 0.0
    # beyond the fixed capacity: refused before anything is launched
    too_big = binding.grad_sqnorm_static_max_elements() + 1
    out = torch.zeros(1, dtype=torch.float64, device=dev)
    small = torch.zeros(16, dtype=torch.float32, device=dev)
    assert L.grad_sqnorm_static(small.data_ptr(), binding.SR_DT_F32, too_big, out.data_ptr(), None) == binding.SR_ERR_WORKSPACE
    assert float(out.item()) == 0.0
    # empty input
    assert L.grad_sqnorm_static(None, binding.SR_DT_F32, 0, got.data_ptr(), None) == binding.SR_OK
    torch.cuda.synchronize()
    assert float(got.item()) == 0.0
