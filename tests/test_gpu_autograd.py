"""The torch.autograd wrapper (paper_2506_16640_b200.autograd) hands the C-ABI gradients to PyTorch unchanged:
input and parameter gradients against the oracle, with and without the forward call's supports kept."""
import numpy as np
import pytest
import torch

import oracle as oracle_mod
import parity
from paper_2506_16640_b200.autograd import entmax_attention
from paper_2506_16640_b200.inputs import Workload, make_inputs

pytestmark = pytest.mark.gpu


def _inputs(N=300, d=64, causal=True, seed=5):
    w = Workload("autograd", 1, 2, N, d, "bf16", causal, (1.5,), plant=2, plant_mode="subset", backward=True,
                 seed_offset=200 + seed)
    return make_inputs(w)


@pytest.mark.parametrize("keep_supports", [False, True])
@pytest.mark.parametrize("alpha", [1.5, 2.0])
def test_gradients_of_inputs_and_scale_parameters(alpha, keep_supports):
    inp = _inputs()
    w = inp.workload
    dev = torch.device("cuda")
    q, k, v = (t.to(dev).requires_grad_(True) for t in (inp.q, inp.k, inp.v))
    beta, gamma, delta = (t.to(dev).requires_grad_(True) for t in (inp.beta, inp.gamma, inp.delta))
    o, tau = entmax_attention(q, k, v, beta, gamma, delta, alpha=alpha, causal=w.causal, keep_supports=keep_supports,
                              return_tau=True)
    assert not tau.requires_grad
    o.backward(inp.d_o.to(dev))
    torch.cuda.synchronize()
    ref_params = np.zeros((w.H, 3))
    for h in range(w.H):
        qh, kh, vh, gh = (t[0, h].float().numpy() for t in (inp.q, inp.k, inp.v, inp.d_o))
        dq, dk, dv = oracle_mod.attn_bwd_head(qh, kh, vh, gh, alpha, inp.sm_scale, w.causal, scale=inp.head_scale(h))
        parity.grad_close("dQ", q.grad[0, h].float().cpu().numpy(), dq)
        parity.grad_close("dK", k.grad[0, h].float().cpu().numpy(), dk)
        parity.grad_close("dV", v.grad[0, h].float().cpu().numpy(), dv)
        _, ref_params[h] = oracle_mod.attn_bwd_scale_head(qh, kh, vh, gh, alpha, inp.sm_scale, w.causal,
                                                          scale=inp.head_scale(h))
    for idx, p in enumerate((beta, gamma, delta)):
        got = p.grad.double().cpu().numpy()
        tol = 2e-2 * max(1.0, np.abs(ref_params[:, idx]).max())
        assert np.abs(got - ref_params[:, idx]).max() <= tol, (idx, got, ref_params[:, idx])


def test_gradient_of_a_per_query_scale_table():
    inp = _inputs(N=260, seed=6)
    w = inp.workload
    dev = torch.device("cuda")
    q, k, v = (t.to(dev) for t in (inp.q, inp.k, inp.v))
    # the table the per-head parameters would give, as a leaf of its own
    rows = np.stack([[oracle_mod.asentmax_scale(*inp.head_scale(h), i + 1) for i in range(w.N)] for h in range(w.H)])
    c_rows = torch.tensor(rows[None], dtype=torch.float32, device=dev, requires_grad=True)
    o = entmax_attention(q, k, v, c_rows=c_rows, alpha=1.5, causal=True)
    o.backward(inp.d_o.to(dev))
    torch.cuda.synchronize()
    assert q.grad is None
    for h in range(w.H):
        qh, kh, vh, gh = (t[0, h].float().numpy() for t in (inp.q, inp.k, inp.v, inp.d_o))
        dc_ref, _ = oracle_mod.attn_bwd_scale_head(qh, kh, vh, gh, 1.5, inp.sm_scale, True, scale=inp.head_scale(h))
        parity.grad_close("dc rows", c_rows.grad[0, h].cpu().numpy(), dc_ref)
