"""The workspace-taking forward / backward entry points and the decode entry point only enqueue work on the caller's stream (no allocation, no
synchronisation), so a caller can record them into a CUDA graph and replay it on new data in the same buffers."""
import pytest
import torch

from paper_2506_16640_b200 import binding
from paper_2506_16640_b200.inputs import Workload, make_inputs

pytestmark = pytest.mark.gpu


def test_forward_and_backward_replay_from_a_cuda_graph():
    dev = torch.device("cuda")
    w = Workload("graph", 2, 4, 700, 64, "bf16", True, (1.5,), plant=2, plant_mode="subset", backward=True, seed_offset=301)
    first, second = make_inputs(w), make_inputs(Workload(**{**w.__dict__, "seed_offset": 302}))
    names = ("q", "k", "v", "d_o", "beta", "gamma", "delta")
    buf = {n: getattr(first, n).to(dev).clone() for n in names}
    params = binding.make_params(buf["q"], 1.5, True)
    ws = binding.alloc_workspace(params, True, dev)
    status = torch.zeros(binding.STATUS_WORDS, dtype=torch.int32, device=dev)
    o = torch.empty_like(buf["q"])
    tau = torch.empty((w.B, w.H, w.N), dtype=torch.float32, device=dev)
    dq, dk, dv = (torch.empty_like(buf["q"]) for _ in range(3))

    def step():
        binding.entmax_attn_fwd(buf["q"], buf["k"], buf["v"], 1.5, True, buf["beta"], buf["gamma"], buf["delta"], o=o,
                                tau=tau, workspace=ws, status=status)
        binding.entmax_attn_bwd(buf["q"], buf["k"], buf["v"], tau, buf["d_o"], 1.5, True, buf["beta"], buf["gamma"],
                                buf["delta"], dq=dq, dk=dk, dv=dv, workspace=ws, status=status)

    def eager(inp):
        for n in names:
            buf[n].copy_(getattr(inp, n))
        step()
        torch.cuda.synchronize()
        return [t.clone() for t in (o, tau, dq)], [dk.clone(), dv.clone()]

    exact_2, approx_2 = eager(second)
    exact_1, approx_1 = eager(first)           # also the warm-up before capture
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    for inp, exact, approx in ((second, exact_2, approx_2), (first, exact_1, approx_1)):
        for n in names:
            buf[n].copy_(getattr(inp, n))
        graph.replay()
        torch.cuda.synchronize()
        assert int(status[binding.STATUS_FLAGS]) == 0
        for got, ref in zip((o, tau, dq), exact):
            assert torch.equal(got, ref)
        # dK, dV are sums of unordered reductions: equal up to the order of fp32 additions
        for got, ref in zip((dk, dv), approx):
            assert (got.float() - ref.float()).abs().max().item() <= 2e-2 * max(1.0, ref.float().abs().max().item())


def test_decode_replays_from_a_cuda_graph():
    dev = torch.device("cuda")
    torch.manual_seed(5)
    B, H, N, d, QL = 2, 4, 3000, 128, 2
    k = torch.randn(B, H, N, d, device=dev).bfloat16()
    v = torch.randn(B, H, N, d, device=dev).bfloat16()
    q = torch.randn(B, H, QL, d, device=dev).bfloat16()
    kv_len = torch.tensor([N, 1234], dtype=torch.int32, device=dev)
    o_ref, tau_ref, supp_ref = binding.entmax_attn_decode_fwd(q, k, v, 1.5, kv_len)
    torch.cuda.synchronize()
    o, tau, supp = torch.empty_like(o_ref), torch.empty_like(tau_ref), torch.empty_like(supp_ref)
    import ctypes
    params = binding.DecodeParams(B, H, QL, N, d, 1.5, 0.0, 0, 0, 0)
    ws = torch.empty(binding.load().entmax_attn_decode_workspace_bytes(ctypes.byref(params)), dtype=torch.uint8, device=dev)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        binding.entmax_attn_decode_fwd(q, k, v, 1.5, kv_len, o=o, tau=tau, support_size=supp, workspace=ws)
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(o, o_ref) and torch.equal(tau, tau_ref) and torch.equal(supp, supp_ref)
