"""Stand-ins for the memory checker: a bounded wait that is made to run out, and canary-padded buffers around
every output of the small-shape calls (tails, single rows, strided layouts) whose pads must come back untouched."""
import numpy as np
import pytest
import torch

from paper_2506_16640_b200 import binding
from paper_2506_16640_b200.inputs import Workload, make_inputs

import parity

pytestmark = pytest.mark.gpu

PAD = 4096          # bytes of canary on either side of every buffer


@pytest.fixture(scope="module", autouse=True)
def _need_cuda():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    binding.load()


def test_bounded_wait_runs_out_and_the_kernel_returns():
    # a barrier nothing arrives on, a limit of 3 ms: the wait gives up, the CTA flags it and returns; the context
    # stays usable (a forward call afterwards is clean)
    status = torch.full((binding.STATUS_WORDS,), -1, dtype=torch.int32, device="cuda")
    binding.entmax_attn_selftest_wait_expiry(3_000_000, status)
    torch.cuda.synchronize()
    st = status.cpu().tolist()
    assert st[binding.STATUS_FLAGS] == binding.FLAG_WAIT_EXPIRED
    assert 3000 <= st[1] <= 50_000, st            # microseconds the wait lasted
    with pytest.raises(binding.EntmaxAttnError):
        binding.entmax_attn_selftest_wait_expiry(10**9, status)      # limits beyond 100 ms are refused
    inp = make_inputs(Workload("after_expiry", 1, 2, 300, 64, "bf16", True, (1.5,), plant=2, plant_mode="subset", seed_offset=55))
    got = parity.run_fwd(inp, 1.5)
    parity.check_fwd_rows(inp, 1.5, got, 0, np.arange(0, 300, 7))


class Guarded:
    """A tensor carved out of a byte buffer with PAD bytes of a known pattern before and after it."""

    def __init__(self, shape, dtype, strides=None, fill=0x5A):
        self.dtype = dtype
        esize = torch.empty((), dtype=dtype).element_size()
        if strides is None:
            numel = int(np.prod(shape))
            span = numel
        else:
            span = 1 + sum((s - 1) * st for s, st in zip(shape, strides))
        self.nbytes = span * esize
        self.fill = fill
        self.raw = torch.full((PAD + self.nbytes + PAD,), fill, dtype=torch.uint8, device="cuda")
        body = self.raw[PAD: PAD + self.nbytes].view(dtype)
        self.t = body.view(shape) if strides is None else torch.as_strided(body, shape, strides)

    def check(self, name):
        head, tail = self.raw[:PAD], self.raw[PAD + self.nbytes:]
        assert bool((head == self.fill).all()) and bool((tail == self.fill).all()), "%s: write outside the buffer" % name


@pytest.mark.parametrize("alpha", [1.5, 2.0])
@pytest.mark.parametrize("strided", [False, True])
@pytest.mark.parametrize("N,d,dtype", [(1, 64, "bf16"), (127, 64, "bf16"), (129, 128, "bf16"), (257, 64, "bf16"),
                                       (257, 128, "bf16"), (129, 64, "fp32"), (600, 128, "bf16")])
def test_no_call_writes_outside_its_buffers(N, d, dtype, strided, alpha):
    # sigma 0.05 at N = 600 sends the rows through the dense-tile kernels as well
    sigma = 0.05 if N == 600 else 1.0
    w = Workload("canary", 2, 3, N, d, dtype, True, (alpha,), qk_sigma=sigma, plant=2 if 40 < N < 600 else 0,
                 plant_mode="subset" if 40 < N < 600 else "none", backward=True, seed_offset=N + d)
    inp = make_inputs(w)
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    shape = (w.B, w.H, N, d)
    strides = (N * w.H * d, d, w.H * d, 1) if strided else None       # [B, N, H, d] storage viewed as [B, H, N, d]

    def guarded_copy(src):
        g = Guarded(shape, tdt, strides)
        g.t.copy_(src.cuda())
        return g

    q, k, v, d_o = (guarded_copy(t) for t in (inp.q, inp.k, inp.v, inp.d_o))
    o, dq, dk, dv = (Guarded(shape, tdt, strides) for _ in range(4))
    tau = Guarded((w.B, w.H, N), torch.float32)
    st_f, st_b = Guarded((binding.STATUS_WORDS,), torch.int32), Guarded((binding.STATUS_WORDS,), torch.int32)
    params = binding.make_params(q.t, alpha, True)
    ws_f = Guarded((binding.entmax_attn_workspace_bytes(params, False),), torch.uint8)
    ws_b = Guarded((binding.entmax_attn_workspace_bytes(params, True),), torch.uint8)
    sc = [t.cuda() for t in (inp.beta, inp.gamma, inp.delta)]
    binding.entmax_attn_fwd(q.t, k.t, v.t, alpha, True, *sc, o=o.t, tau=tau.t, workspace=ws_f.t, status=st_f.t)
    binding.entmax_attn_bwd(q.t, k.t, v.t, tau.t, d_o.t, alpha, True, *sc, dq=dq.t, dk=dk.t, dv=dv.t, workspace=ws_b.t,
                            status=st_b.t)
    torch.cuda.synchronize()
    assert int(st_f.t[0]) == 0 and int(st_b.t[0]) == 0
    for name, g in (("q", q), ("k", k), ("v", v), ("dO", d_o), ("O", o), ("tau", tau), ("dQ", dq), ("dK", dk), ("dV", dv),
                    ("forward workspace", ws_f), ("backward workspace", ws_b), ("forward status", st_f),
                    ("backward status", st_b)):
        g.check(name)
    if strided:
        # the gaps between rows of the strided outputs belong to the other heads: all of them were written by this
        # call, so nothing of the fill pattern may be left inside, and the result must equal the contiguous call's
        ref_o, ref_tau = binding.entmax_attn_fwd(q.t.contiguous(), k.t.contiguous(), v.t.contiguous(), alpha, True, *sc)
        torch.cuda.synchronize()
        assert torch.equal(ref_tau, tau.t) and torch.equal(ref_o, o.t.contiguous())
    # and the guarded call computed the right thing
    got = {"o": o.t, "tau": tau.t, "params": params, "workspace": ws_f.t}
    parity.check_fwd_rows(inp, alpha, got, 1, np.arange(N), check_support=not strided)
    parity.check_bwd_head(inp, alpha, {"dq": dq.t, "dk": dk.t, "dv": dv.t}, 4) if alpha < 2.0 else None
