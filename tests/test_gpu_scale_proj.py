"""The content-dependent ASEntmax scale (Sec. 4.1): the projection kernels against the fp64 oracle, alone and chained
with the per-query-scale attention calls."""
import numpy as np
import pytest
import torch

from paper_2506_16640_b200 import binding
from paper_2506_16640_b200.inputs import Workload, make_inputs

import oracle as oracle_mod
import parity

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _need_cuda():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    binding.load()


def _weights(H, dm, seed):
    gen = torch.Generator().manual_seed(seed)
    x_scale = 1.0 / np.sqrt(dm)
    wb = torch.randn((H, dm), generator=gen) * x_scale
    wg = torch.randn((H, dm), generator=gen) * x_scale
    delta = torch.rand((H,), generator=gen) + 0.5
    return wb, wg, delta


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("B,H,N,dm,causal,n_mode", [(2, 3, 70, 96, True, 0), (1, 12, 300, 768, True, 0), (2, 5, 129, 100, False, 0),
                                                    (1, 2, 65, 64, True, 1), (1, 1, 1, 32, True, 0)])
def test_projection_forward_and_backward_match_the_oracle(B, H, N, dm, causal, n_mode, dtype):
    gen = torch.Generator().manual_seed(1000 + N + dm)
    x = torch.randn((B, N, dm), generator=gen).to(dtype)
    wb, wg, delta = _weights(H, dm, N)
    dc = torch.randn((B, H, N), generator=gen)
    s = 1.5
    xd, wbd, wgd, dd, dcd = (t.cuda() for t in (x, wb, wg, delta, dc))
    c = binding.entmax_attn_scale_proj_fwd(xd, wbd, wgd, dd, s, causal, n_mode=n_mode)
    dwb, dwg, ddel, dx = binding.entmax_attn_scale_proj_bwd(xd, wbd, wgd, dcd, s, causal, n_mode=n_mode)
    torch.cuda.synchronize()
    xf = x.double().numpy()
    c_ref, _, _ = oracle_mod.scale_projection(xf, wb.numpy(), wg.numpy(), delta.numpy(), s, causal, n_mode)
    np.testing.assert_allclose(c.cpu().double().numpy(), c_ref, rtol=2e-5, atol=2e-6)
    rwb, rwg, rdd, rdx = oracle_mod.scale_projection_bwd(xf, wb.numpy(), wg.numpy(), dc.numpy(), s, causal, n_mode)
    for name, got, ref in (("dw_beta", dwb, rwb), ("dw_gamma", dwg, rwg), ("ddelta", ddel, rdd)):
        tol = 2e-4 * max(1.0, np.abs(ref).max())
        assert np.abs(got.cpu().double().numpy() - ref).max() <= tol, name
    dx_tol = (1e-2 if dtype == torch.bfloat16 else 2e-4) * max(1.0, np.abs(rdx).max())
    assert np.abs(dx.cpu().double().numpy() - rdx).max() <= dx_tol


def test_projection_chained_with_the_per_query_attention_calls():
    # x -> c (projection) -> attention with a per-query scale table -> dL/dc -> dL/dw_beta, dL/dw_gamma, dL/ddelta, dL/dx;
    # the oracle walks the same chain in fp64
    N, d, dm, H, alpha, s = 80, 64, 48, 2, 1.5, 1.0
    inp = make_inputs(Workload("proj_chain", 1, H, N, d, "fp32", True, (alpha,), use_scale=False, backward=True, seed_offset=131))
    gen = torch.Generator().manual_seed(77)
    x = torch.randn((1, N, dm), generator=gen)
    wb, wg, delta = _weights(H, dm, 5)
    dev = parity.to_device(inp)
    xd, wbd, wgd, dd = (t.cuda() for t in (x, wb, wg, delta))
    c = binding.entmax_attn_scale_proj_fwd(xd, wbd, wgd, dd, s, True)
    o, tau = binding.entmax_attn_fwd_rowscale(dev["q"], dev["k"], dev["v"], c, alpha, True)
    dq, dk, dv, dc = binding.entmax_attn_bwd_rowscale(dev["q"], dev["k"], dev["v"], c, tau, dev["d_o"], alpha, True)
    dwb, dwg, ddel, dx = binding.entmax_attn_scale_proj_bwd(xd, wbd, wgd, dc, s, True)
    torch.cuda.synchronize()
    c_ref, _, _ = oracle_mod.scale_projection(x.double().numpy(), wb.numpy(), wg.numpy(), delta.numpy(), s, True)
    dc_ref = np.zeros((1, H, N))
    for h in range(H):
        q, k, v, g = (t[0, h].float().numpy() for t in (inp.q, inp.k, inp.v, inp.d_o))
        for i in range(N):
            row_dc, _ = oracle_mod.attn_bwd_scale_head(q[: i + 1], k[: i + 1], v[: i + 1], g[: i + 1], alpha, inp.sm_scale, True,
                                                       scale=(0.0, 1.0, float(c_ref[0, h, i])))
            dc_ref[0, h, i] = row_dc[i]
    parity.grad_close("dc", dc[0].cpu().numpy(), dc_ref[0])
    rwb, rwg, rdd, rdx = oracle_mod.scale_projection_bwd(x.double().numpy(), wb.numpy(), wg.numpy(), dc_ref, s, True)
    for name, got, ref in (("dw_beta", dwb, rwb), ("dw_gamma", dwg, rwg), ("ddelta", ddel, rdd), ("dx", dx, rdx)):
        tol = 2e-3 * max(1.0, np.abs(ref).max())
        assert np.abs(got.cpu().double().numpy() - ref).max() <= tol, (name, np.abs(got.cpu().double().numpy() - ref).max())


def test_projection_rejects_bad_arguments():
    x = torch.zeros((1, 8, 16), device="cuda")
    w = torch.zeros((2, 16), device="cuda")
    d = torch.ones((2,), device="cuda")
    with pytest.raises(binding.EntmaxAttnError):
        binding.entmax_attn_scale_proj_fwd(x, w, w, d, 0.0, True)            # gamma_range must be positive
    with pytest.raises(binding.EntmaxAttnError):
        binding.entmax_attn_scale_proj_fwd(x.double(), w, w, d, 1.0, True)   # dtype
