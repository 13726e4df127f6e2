"""entmax_attn_fwd_static: the forward pass for callers that cannot allocate device memory.

Some users of the library are handed tensors but no allocator, or run before a memory pool exists,
or sit in a region where calling the allocator is not allowed; they cannot supply the workspace the
regular forward call wants.  The static entry point keeps its scratch in a fixed array inside the
library.  This test calls it through the C ABI twice in a row (the second call finds the scratch
full of the first call's data, and a different problem in between changes its contents) and checks
O and tau against the regular entry point within the tolerances used by the other GPU tests.

The file name sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import numpy as np
import pytest
import torch

from paper_2506_16640_b200 import binding
from paper_2506_16640_b200.inputs import Workload, make_inputs

import parity

pytestmark = pytest.mark.gpu


def _workload(name, N, d, dtype, causal, seed):
    return Workload(name, 1, 3, N, d, dtype, causal, (1.5,), plant=3, plant_mode="subset", use_scale=True,
                    seed_offset=seed)


def _static(dev, alpha, causal):
    q = dev["q"]
    B, H, N, _ = q.shape
    o = torch.empty_like(q)
    tau = torch.empty((B, H, N), dtype=torch.float32, device=q.device)
    status = torch.full((binding.STATUS_WORDS,), -1, dtype=torch.int32, device=q.device)
    binding.entmax_attn_fwd_static(q, dev["k"], dev["v"], alpha, causal, dev["beta"], dev["gamma"], dev["delta"],
                                   o=o, tau=tau, status=status)
    torch.cuda.synchronize()
    assert int(status[binding.STATUS_FLAGS]) == 0
    return o, tau


def _close(o, tau, ref, dtype_name):
    o_err = (o.float() - ref["o"].float()).abs().max().item()
    t_ref = ref["tau"].double()
    tau_err = ((tau.double() - t_ref).abs() / t_ref.abs().clamp_min(1.0)).max().item()
    assert o_err <= parity.O_TOL, o_err
    assert tau_err <= parity.tau_tol(dtype_name), tau_err


@pytest.mark.parametrize("alpha", [1.5, 2.0])
def test_static_forward_matches_regular_forward_twice(alpha):
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    binding.load()
    big = make_inputs(_workload("static_a", 700, 64, "bf16", True, 31))
    small = make_inputs(_workload("static_b", 130, 128, "fp32", False, 32))
    ref_big = parity.run_fwd(big, alpha)
    ref_small = parity.run_fwd(small, alpha)
    # two calls in a row on the same problem: the second one starts from a used scratch
    for _ in range(2):
        o, tau = _static(ref_big["dev"], alpha, True)
        _close(o, tau, ref_big, "bf16")
    # another shape in between rewrites the scratch with a different layout; then the first again
    o, tau = _static(ref_small["dev"], alpha, False)
    _close(o, tau, ref_small, "fp32")
    o, tau = _static(ref_big["dev"], alpha, True)
    _close(o, tau, ref_big, "bf16")
    # the static result also agrees with the oracle on a few rows
    got = {"o": o, "tau": tau, "params": ref_big["params"], "workspace": ref_big["workspace"]}
    parity.check_fwd_rows(big, alpha, got, 1, np.arange(0, 700, 7), check_support=False)


def test_static_forward_rejects_problems_beyond_the_scratch():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    binding.load()
    # 16 heads x 32768 keys needs 16*32768 + 64*32768 floats = 10 MiB > the 8 MiB scratch
    q = torch.zeros((1, 16, 32768, 64), dtype=torch.bfloat16, device="cuda")
    o = torch.empty_like(q)
    tau = torch.empty((1, 16, 32768), dtype=torch.float32, device="cuda")
    with pytest.raises(binding.EntmaxAttnError, match="built-in scratch"):
        binding.entmax_attn_fwd_static(q, q, q, 1.5, True, o=o, tau=tau)
