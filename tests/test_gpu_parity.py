"""GPU parity: the CUDA path, called through the C ABI, against the fp64 CPU oracle on the same seeded
inputs -- element by element at small sizes, on sampled rows (and invariants) at the full sizes."""
import math

import numpy as np
import pytest
import torch

from paper_2506_16640_b200 import binding, inputs
from paper_2506_16640_b200.inputs import WORKLOADS, Workload, make_inputs, sample_rows, scaled

import oracle as oracle_mod
import parity

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _need_cuda():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    binding.load()


def _small(name, N, d, causal, dtype="bf16", B=1, H=2, plant=0, use_scale=True, backward=False, sigma=1.0, seed=7):
    return Workload(name, B, H, N, d, dtype, causal, (1.5,), qk_sigma=sigma, plant=plant,
                    plant_mode="subset" if plant else "none", use_scale=use_scale, backward=backward, seed_offset=seed)


# ------------------------------------------------------------------ score tile engine (tcgen05 + TMA)
@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("N", [1, 100, 256, 700])
def test_score_tiles_match_fp64_dot_products(N, d, causal):
    inp = make_inputs(_small("scores", N, d, causal, H=3))
    dev = parity.to_device(inp)
    for bh in [0, 2]:
        status = torch.zeros(binding.STATUS_WORDS, dtype=torch.int32, device="cuda")
        s = binding.entmax_attn_scores_debug(dev["q"], dev["k"], bh, causal, status=status)
        torch.cuda.synchronize()
        assert int(status[0]) == 0
        ref = inp.q[0, bh].double() @ inp.k[0, bh].double().T
        got = s.cpu().double()
        keep = torch.ones(N, N, dtype=torch.bool).tril() if causal else torch.ones(N, N, dtype=torch.bool)
        assert torch.isnan(got[~keep]).all()          # masked entries were never written
        err = (got[keep] - ref[keep]).abs().max().item()
        assert err <= 1e-4 * max(1.0, ref.abs().max().item()), err


# ------------------------------------------------------------------ config 1: fp32, fixed temperature
def test_cfg1_fp32_all_rows():
    inp = make_inputs(WORKLOADS[1])
    got = parity.run_fwd(inp, 1.5)
    for bh in range(inp.workload.B * inp.workload.H):
        st = parity.check_fwd_rows(inp, 1.5, got, bh, np.arange(inp.workload.N))
        assert st["tau_err"] <= 1e-4


# ------------------------------------------------------------------ small shapes, every row
@pytest.mark.parametrize("alpha", [1.25, 1.5, 2.0, 1.7])
@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("N,d,dtype", [(1, 64, "bf16"), (2, 64, "bf16"), (127, 64, "bf16"), (128, 128, "bf16"),
                                       (129, 64, "bf16"), (257, 128, "bf16"), (600, 64, "bf16"), (130, 128, "fp32"),
                                       (33, 64, "fp32")])
def test_small_shapes_all_rows(N, d, dtype, causal, alpha):
    for use_scale in (True, False):
        inp = make_inputs(_small("small", N, d, causal, dtype=dtype, plant=3 if N > 40 else 0, use_scale=use_scale,
                                 seed=N + d))
        got = parity.run_fwd(inp, alpha)
        for bh in range(inp.workload.H):
            parity.check_fwd_rows(inp, alpha, got, bh, np.arange(N))


def test_dense_rows_fall_back_and_still_match():
    # tiny logits (sigma 0.05, no scale): almost every key is in the support, far beyond the list capacity
    inp = make_inputs(_small("dense", 900, 64, True, use_scale=False, sigma=0.05, seed=3))
    got = parity.run_fwd(inp, 1.5)
    st = parity.check_fwd_rows(inp, 1.5, got, 1, np.arange(900))
    assert st["dense_rows"] > 300 and int(got["status"][binding.STATUS_DENSE_ROWS]) > 600
    inp = make_inputs(_small("dense_nc", 700, 128, False, use_scale=False, sigma=0.05, backward=True, seed=4))
    got = parity.run_fwd(inp, 2.0)
    parity.check_fwd_rows(inp, 2.0, got, 0, np.arange(700))
    bwd = parity.run_bwd(inp, 2.0, got["tau"], got["dev"])
    parity.check_bwd_head(inp, 2.0, bwd, 0)


@pytest.mark.parametrize("alpha", [1.25, 1.5, 2.0, 1.7])
@pytest.mark.parametrize("N,d,causal", [(2100, 128, True), (1300, 64, False), (515, 128, False)])
def test_dense_tiles_on_tensor_cores(N, d, causal, alpha):
    # tiny logits: supports of hundreds to thousands of keys, so every row goes through the dense-tile path
    # (Newton sweeps of QK^T tiles, then P V on the tensor cores); several K tiles and a ragged tail
    inp = make_inputs(_small("dense_tiles", N, d, causal, use_scale=True, sigma=0.03, seed=N))
    got = parity.run_fwd(inp, alpha)
    rows = np.arange(0, N, 3)
    for bh in range(inp.workload.H):
        st = parity.check_fwd_rows(inp, alpha, got, bh, rows)
    assert int(got["status"][binding.STATUS_DENSE_ROWS]) > N


@pytest.mark.parametrize("sigma,expect", [(0.55, 200), (0.3, 1000), (0.18, 4000)])
def test_dense_path_at_supports_of_hundreds_to_thousands(sigma, expect):
    # long rows whose supports run to about 200, 1000 and 4000 keys (fixed temperature, logits of std sigma^2): forward
    # (tau, O and the support size the dense-tile kernel counted) on sampled rows, backward on sampled dQ rows, at
    # N = 8192 so that the dense-tile kernels take their sampled start
    N = 8192
    inp = make_inputs(Workload("dense_support_%d" % expect, 1, 2, N, 64, "bf16", True, (1.5,), qk_sigma=sigma, use_scale=False,
                               backward=True, seed_offset=140 + expect % 97))
    got = parity.run_fwd(inp, 1.5)
    bwd = parity.run_bwd(inp, 1.5, got["tau"], got["dev"])
    late = np.arange(N - 1536, N, 24)                        # rows that see the whole sequence, more or less
    rows = np.unique(np.concatenate([sample_rows(inp, 0, 64), late]))
    sizes = []
    for bh in range(2):
        st = parity.check_fwd_rows(inp, 1.5, got, bh, rows)
        parity.check_bwd_rows(inp, 1.5, bwd, bh, rows)
        sizes.append(st["supp_max"])
        assert st["dense_rows"] > len(late) // 2             # these rows went through the dense-tile kernels
    assert 0.4 * expect <= max(sizes) <= 2.5 * expect, sizes


def test_mixed_sparse_and_dense_rows_in_one_tile():
    # planted keys make some rows one-hot while the others stay dense: both paths write into the same Q tiles
    inp = make_inputs(_small("mixed", 1000, 128, True, plant=3, use_scale=False, sigma=0.05, seed=21))
    got = parity.run_fwd(inp, 1.5)
    for bh in range(inp.workload.H):
        st = parity.check_fwd_rows(inp, 1.5, got, bh, np.arange(1000))
    dense = int(got["status"][binding.STATUS_DENSE_ROWS])
    assert 0 < dense < 2 * 1000


@pytest.mark.parametrize("alpha", [1.25, 1.5, 2.0, 1.7])
@pytest.mark.parametrize("N,d,causal", [(900, 128, True), (700, 64, False), (515, 128, False), (130, 64, True)])
def test_dense_tiles_backward_on_tensor_cores(N, d, causal, alpha):
    # every row dense: the backward runs as two passes of tensor-core tiles per Q tile (sum u, sum u dP; then
    # P and dS tiles feeding dQ, dK, dV); several K tiles, a ragged tail, both head dims
    inp = make_inputs(_small("dense_tiles_bwd", N, d, causal, use_scale=True, sigma=0.01 if alpha == 2.0 else 0.04,
                             backward=True, seed=N + 7))
    got = parity.run_fwd(inp, alpha)
    bwd = parity.run_bwd(inp, alpha, got["tau"], got["dev"])
    dense, tiles = int(bwd["status"][binding.STATUS_DENSE_ROWS]), int(bwd["status"][binding.STATUS_TILES])
    assert dense > N // 8 and 1 <= tiles <= inp.workload.H * ((N + 127) // 128)
    for bh in range(inp.workload.H):
        parity.check_bwd_head(inp, alpha, bwd, bh)


def test_mixed_sparse_and_dense_rows_backward():
    # one-hot rows (list path) and dense rows (tile path) share Q tiles and key rows of dK, dV
    inp = make_inputs(_small("mixed_bwd", 1000, 128, True, plant=3, use_scale=False, sigma=0.05, backward=True, seed=22))
    got = parity.run_fwd(inp, 1.5)
    bwd = parity.run_bwd(inp, 1.5, got["tau"], got["dev"])
    dense = int(bwd["status"][binding.STATUS_DENSE_ROWS])
    assert 0 < dense < 2 * 1000
    for bh in range(inp.workload.H):
        parity.check_bwd_head(inp, 1.5, bwd, bh)


@pytest.mark.parametrize("alpha", [1.25, 1.5, 2.0])
@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
def test_all_logits_equal_gives_uniform_rows(alpha, dtype):
    # q = 0: every visible key ties, p_i is uniform over the i + 1 visible keys, tau_i = -(i + 1)^-(alpha-1) (Eq. 1 with
    # sum p = 1), O_i the running mean of V; rows grow from one key to a dense 600
    inp = make_inputs(_small("ties", 600, 64, True, dtype=dtype, use_scale=True, seed=31))
    inp.q.zero_()
    got = parity.run_fwd(inp, alpha)
    n = torch.arange(1, 601, dtype=torch.float64)
    tau_ref = -n.pow(-(alpha - 1.0))
    for bh in range(inp.workload.H):
        tau = got["tau"][0, bh].double().cpu()
        assert (tau - tau_ref).abs().max().item() <= parity.tau_tol(dtype)
        o_ref = inp.v[0, bh].double().cumsum(dim=0) / n[:, None]
        assert (got["o"][0, bh].double().cpu() - o_ref).abs().max().item() <= parity.O_TOL
        parity.check_fwd_rows(inp, alpha, got, bh, np.arange(0, 600, 7), check_support=False)


def test_n_mode_total_length_and_strided_layout():
    inp = make_inputs(_small("nmode", 300, 64, True, seed=11))
    got = parity.run_fwd(inp, 1.5, n_mode=1)
    parity.check_fwd_rows(inp, 1.5, got, 0, np.arange(300), n_mode=1)
    # [B, N, H, D] storage viewed as [B, H, N, D]
    dev = parity.to_device(inp)
    for name in ("q", "k", "v"):
        dev[name] = dev[name].permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    o = torch.empty_like(dev["q"])
    params = binding.make_params(dev["q"], 1.5, True)
    ws = binding.alloc_workspace(params, False, "cuda")
    status = torch.zeros(binding.STATUS_WORDS, dtype=torch.int32, device="cuda")
    o, tau = binding.entmax_attn_fwd(dev["q"], dev["k"], dev["v"], 1.5, True, dev["beta"], dev["gamma"], dev["delta"],
                                     o=o, workspace=ws, status=status)
    torch.cuda.synchronize()
    got2 = {"o": o, "tau": tau, "workspace": ws, "params": params, "status": status.cpu()}
    parity.check_fwd_rows(inp, 1.5, got2, 1, np.arange(300))


@pytest.mark.parametrize("d", [64, 128])
def test_dense_tiles_with_strided_layout_and_batches(d):
    # every row dense, two batch elements, tensors stored [B, N, H, D] and passed as [B, H, N, D] views: the tile
    # kernels' tensor maps, row addressing and the fp32 dK / dV accumulators all see the strides
    inp = make_inputs(_small("dense_strided", 700, d, True, B=2, H=3, use_scale=True, sigma=0.04, backward=True, seed=61))
    w = inp.workload
    dev = parity.to_device(inp)
    for name in ("q", "k", "v", "d_o"):
        dev[name] = dev[name].permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    status = torch.zeros(binding.STATUS_WORDS, dtype=torch.int32, device="cuda")
    o, tau = binding.entmax_attn_fwd(dev["q"], dev["k"], dev["v"], 1.5, True, dev["beta"], dev["gamma"], dev["delta"],
                                     status=status)
    dq, dk, dv = (torch.empty_like(dev["q"]) for _ in range(3))
    st2 = torch.zeros(binding.STATUS_WORDS, dtype=torch.int32, device="cuda")
    binding.entmax_attn_bwd(dev["q"], dev["k"], dev["v"], tau, dev["d_o"], 1.5, True, dev["beta"], dev["gamma"],
                            dev["delta"], dq=dq, dk=dk, dv=dv, status=st2)
    torch.cuda.synchronize()
    assert int(status[binding.STATUS_FLAGS]) == 0 and int(st2[binding.STATUS_FLAGS]) == 0
    assert int(status[binding.STATUS_DENSE_ROWS]) > w.B * w.H * 500 and int(st2[binding.STATUS_DENSE_ROWS]) > w.B * w.H * 500
    assert not dq.is_contiguous()
    got = {"o": o, "tau": tau}
    bwd = {"dq": dq, "dk": dk, "dv": dv}
    for bh in (0, 4, 5):
        parity.check_fwd_rows(inp, 1.5, got, bh, np.arange(0, 700, 5), check_support=False)
        parity.check_bwd_head(inp, 1.5, bwd, bh)


def test_right_padded_sequences_need_no_mask_under_the_causal_mask():
    # a batch of sequences of different lengths, right-padded to N: a valid row i < L sees only keys j <= i < L, so
    # whatever sits in the padding cannot reach it; with dO = 0 on the padding rows it cannot reach dK, dV either
    inp = make_inputs(_small("padded", 1000, 64, True, plant=2, backward=True, seed=71))
    L = 700
    dev = parity.to_device(inp)
    dev["d_o"][:, :, L:] = 0
    o1, tau1 = binding.entmax_attn_fwd(dev["q"], dev["k"], dev["v"], 1.5, True, dev["beta"], dev["gamma"], dev["delta"])
    g1 = binding.entmax_attn_bwd(dev["q"], dev["k"], dev["v"], tau1, dev["d_o"], 1.5, True, dev["beta"], dev["gamma"],
                                 dev["delta"])
    gen = torch.Generator(device="cuda").manual_seed(3)
    for name in ("q", "k", "v"):
        junk = torch.randn(dev[name][:, :, L:].shape, generator=gen, device="cuda") * 50.0
        dev[name][:, :, L:] = junk.to(dev[name].dtype)
    o2, tau2 = binding.entmax_attn_fwd(dev["q"], dev["k"], dev["v"], 1.5, True, dev["beta"], dev["gamma"], dev["delta"])
    g2 = binding.entmax_attn_bwd(dev["q"], dev["k"], dev["v"], tau2, dev["d_o"], 1.5, True, dev["beta"], dev["gamma"],
                                 dev["delta"])
    torch.cuda.synchronize()
    assert torch.equal(o1[:, :, :L], o2[:, :, :L]) and torch.equal(tau1[:, :, :L], tau2[:, :, :L])
    assert torch.equal(g1[0][:, :, :L], g2[0][:, :, :L])                       # dQ of the valid rows
    for a_, b_ in zip(g1[1:], g2[1:]):                                         # dK, dV of the valid keys
        ref = a_[:, :, :L].float()
        assert (ref - b_[:, :, :L].float()).abs().max().item() <= 1e-2 * max(1.0, ref.abs().max().item())


def test_two_calls_are_bitwise_identical():
    # the lists the sweep leaves vary from run to run (order, surplus candidates); O and tau must not
    for N, d, plant in [(513, 128, 4), (3000, 64, 0)]:
        inp = make_inputs(_small("det", N, d, True, plant=plant, seed=5))
        a = parity.run_fwd(inp, 1.5)
        for _ in range(4):
            b = parity.run_fwd(inp, 1.5, dev=a["dev"])
            assert torch.equal(a["tau"], b["tau"]) and torch.equal(a["o"], b["o"])


# ------------------------------------------------------------------ backward, small, full heads
@pytest.mark.parametrize("alpha", [1.25, 1.5, 2.0])
@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("N,d,dtype", [(1, 64, "bf16"), (130, 64, "bf16"), (300, 128, "bf16"), (97, 64, "fp32")])
def test_backward_small_full_heads(N, d, dtype, causal, alpha):
    inp = make_inputs(_small("bwd", N, d, causal, dtype=dtype, plant=2 if N > 40 else 0, backward=True, seed=N))
    got = parity.run_fwd(inp, alpha)
    bwd = parity.run_bwd(inp, alpha, got["tau"], got["dev"])
    for bh in range(inp.workload.H):
        parity.check_bwd_head(inp, alpha, bwd, bh)


# ------------------------------------------------------------------ alpha > 2 (the paper's retrieval runs use 4 ... 64)
@pytest.mark.parametrize("alpha", [3.0, 4.0])
@pytest.mark.parametrize("N,d,dtype,causal", [(1, 64, "bf16", True), (130, 64, "bf16", True), (300, 128, "bf16", False),
                                              (600, 64, "bf16", True), (97, 64, "fp32", True)])
def test_alpha_above_two_small_shapes(N, d, dtype, causal, alpha):
    # e = 1/(alpha-1) < 1: every solver runs its bracketed iteration; forward on every row, backward on whole heads
    inp = make_inputs(_small("alpha_gt2", N, d, causal, dtype=dtype, plant=2 if N > 40 else 0, backward=True, seed=N + 11))
    got = parity.run_fwd(inp, alpha)
    bwd = parity.run_bwd(inp, alpha, got["tau"], got["dev"])
    for bh in range(inp.workload.H):
        parity.check_fwd_rows(inp, alpha, got, bh, np.arange(N))
        parity.check_bwd_head_banded(inp, alpha, bwd, bh)


@pytest.mark.parametrize("alpha", [3.0, 4.0])
def test_alpha_above_two_dense_tiles(alpha):
    # For alpha > 2 a support of hundreds of keys needs logits that agree to within n^-(alpha-1), i.e. ties: q = 0
    # makes every visible key tie, p_i uniform over the i + 1 visible keys and tau_i = -(i + 1)^-(alpha-1) (Eq. 1 with
    # sum p = 1).  Rows beyond the list capacity go through the dense-tile kernels and their bracketed sweeps.
    N = 700
    inp = make_inputs(_small("alpha_gt2_dense", N, 128, True, use_scale=True, backward=True, seed=93))
    inp.q.zero_()
    got = parity.run_fwd(inp, alpha)
    assert int(got["status"][binding.STATUS_DENSE_ROWS]) > N
    n = torch.arange(1, N + 1, dtype=torch.float64)
    tau_ref = -n.pow(-(alpha - 1.0))
    bwd = parity.run_bwd(inp, alpha, got["tau"], got["dev"])
    for bh in range(inp.workload.H):
        tau = got["tau"][0, bh].double().cpu()
        assert (tau - tau_ref).abs().max().item() <= parity.tau_tol("bf16")
        o_ref = inp.v[0, bh].double().cumsum(dim=0) / n[:, None]
        assert (got["o"][0, bh].double().cpu() - o_ref).abs().max().item() <= parity.O_TOL
        # every key of a row sits at the same distance above the threshold, so the gradients are well conditioned
        parity.check_bwd_head(inp, alpha, bwd, bh)


def test_alpha_above_two_long_rows():
    # one 8192-token shape (sampled pre-pass, list shrinks with the bisection bound), sampled rows of every head
    inp = make_inputs(Workload("alpha_gt2_8k", 1, 4, 8192, 64, "bf16", True, (3.0,), plant=4, plant_mode="subset",
                               backward=True, seed_offset=95))
    for alpha in (3.0, 4.0):
        got = parity.run_fwd(inp, alpha)
        bwd = parity.run_bwd(inp, alpha, got["tau"], got["dev"])
        for bh in range(4):
            rows = sample_rows(inp, bh, 192)
            parity.check_fwd_rows(inp, alpha, got, bh, rows)
        parity.check_bwd_head_banded(inp, alpha, bwd, 2)


def test_alpha_sixteen_on_rows_it_can_resolve():
    # alpha = 16: p = y^(1/15) cannot be normalised in floating point unless the row is one-hot or an exact tie
    # (a key at y = 1e-7 above the threshold already weighs 0.34); planted keys three units above the rest make
    # every planted row one-hot: tau = 15 s_max - 1, O = v of the planted key.  All other rows only have to be finite.
    inp = make_inputs(_small("alpha16", 400, 64, True, plant=1, use_scale=True, seed=97))
    got = parity.run_fwd(inp, 16.0)
    assert torch.isfinite(got["tau"]).all() and torch.isfinite(got["o"].float()).all()
    w = inp.workload
    checked = 0
    for bh in range(w.H):
        q, k, v = (t[0, bh].float().numpy() for t in (inp.q, inp.k, inp.v))
        rows = inp.planted_rows[bh]
        ref = oracle_mod.attn_fwd_rows(q, k, v, rows, 16.0, inp.sm_scale, True, scale=inp.head_scale(bh % w.H))
        one_hot = ref["supp"] == 1
        tau_g = got["tau"][0, bh].cpu().numpy()[rows]
        o_g = got["o"][0, bh].float().cpu().numpy()[rows]
        rel = np.abs(tau_g - ref["tau"]) / np.maximum(1.0, np.abs(ref["tau"]))
        assert rel[one_hot].max() <= parity.tau_tol("bf16")
        assert np.abs(o_g - ref["o"])[one_hot].max() <= parity.O_TOL
        checked += int(one_hot.sum())
    assert checked > 100


# ------------------------------------------------------------------ gradients of the ASEntmax scale
@pytest.mark.parametrize("alpha", [1.25, 1.5, 2.0])
@pytest.mark.parametrize("N,d,dtype,causal,sigma,plant", [(300, 64, "bf16", True, 1.0, 2), (700, 128, "bf16", False, 1.0, 0),
                                                          (260, 64, "bf16", True, 0.05, 0), (97, 64, "fp32", True, 1.0, 0)])
def test_scale_gradients(N, d, dtype, causal, sigma, plant, alpha):
    # sigma 0.05 makes every row dense (the dense backward path computes the same gradients)
    inp = make_inputs(_small("dscale", N, d, causal, dtype=dtype, plant=plant, backward=True, sigma=sigma, seed=N + 1))
    w = inp.workload
    got = parity.run_fwd(inp, alpha)
    dev = got["dev"]
    dq, dk, dv, dc, grads = binding.entmax_attn_bwd_scale(dev["q"], dev["k"], dev["v"], got["tau"], dev["d_o"], alpha,
                                                          causal, dev["beta"], dev["gamma"], dev["delta"])
    torch.cuda.synchronize()
    ref_g = np.zeros((w.H, 3))
    for h in range(w.H):
        q, k, v, g = (t[0, h].float().numpy() for t in (inp.q, inp.k, inp.v, inp.d_o))
        dc_ref, gr = oracle_mod.attn_bwd_scale_head(q, k, v, g, alpha, inp.sm_scale, causal, scale=inp.head_scale(h))
        ref_g[h] = gr
        parity.grad_close("dc rows", dc[0, h].cpu().numpy(), dc_ref)
    for idx, name in enumerate(("dbeta", "dgamma", "ddelta")):
        got_g = grads[idx].cpu().double().numpy()
        tol = 2e-2 * max(1.0, np.abs(ref_g[:, idx]).max())
        assert np.abs(got_g - ref_g[:, idx]).max() <= tol, (name, got_g, ref_g[:, idx])
    # the plain backward entry point is the same call without the extra outputs
    plain = parity.run_bwd(inp, alpha, got["tau"], dev)
    assert torch.equal(plain["dq"], dq)


def test_backward_from_compact_saved_supports():
    # sparse rows (compact lists hold them), rows with more than 32 support entries and dense rows (both recomputed
    # on the tensor cores): the compact saved state gives the gradients of the plain backward call
    for sigma, plant, N in [(1.0, 3, 900), (0.35, 0, 900), (0.05, 0, 600)]:
        inp = make_inputs(_small("compact", N, 128, True, plant=plant, backward=True, sigma=sigma, seed=81))
        got = parity.run_fwd(inp, 1.5)
        dev = got["dev"]
        saved = binding.entmax_attn_save_supports(dev["q"], 1.5, True, got["workspace"])
        status = torch.zeros(binding.STATUS_WORDS, dtype=torch.int32, device="cuda")
        dq, dk, dv, _, _ = binding.entmax_attn_bwd_ex(dev["q"], dev["k"], dev["v"], got["tau"], dev["d_o"], 1.5, True,
                                                      dev["beta"], dev["gamma"], dev["delta"], saved_supports=saved,
                                                      status=status)
        torch.cuda.synchronize()
        assert int(status[binding.STATUS_FLAGS]) == 0
        rows = inp.workload.H * N
        recomputed = int(status[binding.STATUS_DENSE_ROWS])
        if sigma == 1.0:
            assert recomputed == 0
        elif sigma == 0.35:
            assert recomputed < rows              # most supports fit the slots
        else:
            assert recomputed > rows // 2
        bwd = {"dq": dq, "dk": dk, "dv": dv}
        for bh in range(inp.workload.H):
            parity.check_bwd_head(inp, 1.5, bwd, bh)
        if sigma == 1.0:
            full = binding.entmax_attn_bwd_ex(dev["q"], dev["k"], dev["v"], got["tau"], dev["d_o"], 1.5, True, dev["beta"],
                                              dev["gamma"], dev["delta"], fwd_workspace=got["workspace"])
            assert torch.equal(full[0], dq)        # the same lists in the same order


# ------------------------------------------------------------------ per-query scale tables
def test_rowscale_equals_per_head_call_when_given_the_same_table():
    inp = make_inputs(_small("rowscale_same", 700, 128, True, plant=3, backward=True, B=2, seed=41))
    w = inp.workload
    got = parity.run_fwd(inp, 1.5)
    dev = got["dev"]
    lay = binding.entmax_attn_workspace_layout(got["params"])
    table = got["workspace"][lay.scale_offset: lay.scale_offset + 4 * w.H * w.N].view(torch.float32).view(w.H, w.N)
    c_rows = table.unsqueeze(0).expand(w.B, w.H, w.N).contiguous()
    o, tau = binding.entmax_attn_fwd_rowscale(dev["q"], dev["k"], dev["v"], c_rows, 1.5, True)
    torch.cuda.synchronize()
    assert torch.equal(o, got["o"]) and torch.equal(tau, got["tau"])
    ref = binding.entmax_attn_bwd_scale(dev["q"], dev["k"], dev["v"], tau, dev["d_o"], 1.5, True, dev["beta"],
                                        dev["gamma"], dev["delta"], want_param_grads=False)
    dq, dk, dv, dc = binding.entmax_attn_bwd_rowscale(dev["q"], dev["k"], dev["v"], c_rows, tau, dev["d_o"], 1.5, True)
    torch.cuda.synchronize()
    assert torch.equal(dq, ref[0]) and torch.equal(dc, ref[3])
    # dK, dV are sums of fp32 atomics: equal up to the order of the additions
    for a_, b_ in ((dk, ref[1]), (dv, ref[2])):
        assert (a_.float() - b_.float()).abs().max().item() <= 2e-2 * max(1.0, b_.float().abs().max().item())


@pytest.mark.parametrize("alpha", [1.5, 2.0])
@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
def test_rowscale_with_a_batch_dependent_table_matches_the_oracle(dtype, alpha):
    # c differs per batch element and per row; the oracle sees row i with beta = 0, delta = c_i
    N, d = 96, 64
    inp = make_inputs(_small("rowscale_rows", N, d, True, dtype=dtype, backward=True, B=2, use_scale=False, seed=43))
    w = inp.workload
    gen = torch.Generator().manual_seed(4343)
    c_host = torch.rand((w.B, w.H, N), generator=gen) * 6.0 + 0.5
    dev = parity.to_device(inp)
    c_rows = c_host.cuda()
    o, tau = binding.entmax_attn_fwd_rowscale(dev["q"], dev["k"], dev["v"], c_rows, alpha, True)
    dq, dk, dv, dc = binding.entmax_attn_bwd_rowscale(dev["q"], dev["k"], dev["v"], c_rows, tau, dev["d_o"], alpha, True)
    torch.cuda.synchronize()
    tol_tau = parity.tau_tol(dtype)
    for b in range(w.B):
        for h in range(w.H):
            q, k, v, g = (t[b, h].float().numpy() for t in (inp.q, inp.k, inp.v, inp.d_o))
            for i in range(0, N, 5):
                sc = (0.0, 1.0, float(c_host[b, h, i]))
                rows = np.array([i])
                f = oracle_mod.attn_fwd_rows(q, k, v, rows, alpha, inp.sm_scale, True, scale=sc)
                assert abs(float(tau[b, h, i]) - f["tau"][0]) <= tol_tau * max(1.0, abs(f["tau"][0]))
                assert np.abs(o[b, h, i].float().cpu().numpy() - f["o"][0]).max() <= parity.O_TOL
                dq_ref, _ = oracle_mod.attn_bwd_rows(q, k, v, g, rows, alpha, inp.sm_scale, True, scale=sc)
                parity.grad_close("dQ row", dq[b, h, i].float().cpu().numpy(), dq_ref[0])
                dc_ref, _ = oracle_mod.attn_bwd_scale_head(q, k, v, g, alpha, inp.sm_scale, True, scale=sc)
                parity.grad_close("dc row", np.array([float(dc[b, h, i])]), np.array([dc_ref[i]]))


# ------------------------------------------------------------------ ALiBi term (the paper's NAPE: half the heads)
def _check_alibi(inp, alpha, causal, slopes, dense_expected):
    w = inp.workload
    dev = parity.to_device(inp)
    sl = torch.tensor(slopes, dtype=torch.float32, device="cuda")
    status = torch.zeros(binding.STATUS_WORDS, dtype=torch.int32, device="cuda")
    o, tau = binding.entmax_attn_fwd_ex(dev["q"], dev["k"], dev["v"], alpha, causal, dev["beta"], dev["gamma"],
                                        dev["delta"], alibi_slopes=sl, status=status)
    dq, dk, dv, dc, grads = binding.entmax_attn_bwd_ex(dev["q"], dev["k"], dev["v"], tau, dev["d_o"], alpha, causal,
                                                       dev["beta"], dev["gamma"], dev["delta"], alibi_slopes=sl,
                                                       want_scale_rows=True, want_param_grads=inp.beta is not None)
    torch.cuda.synchronize()
    assert int(status[binding.STATUS_FLAGS]) == 0
    if dense_expected is not None:
        assert (int(status[binding.STATUS_DENSE_ROWS]) > 0) == dense_expected
    N = w.N
    rows = np.arange(N)
    for h in range(w.H):
        q, k, v, g = (t[0, h].float().numpy() for t in (inp.q, inp.k, inp.v, inp.d_o))
        sc = inp.head_scale(h)
        f = oracle_mod.attn_fwd_rows(q, k, v, rows, alpha, inp.sm_scale, causal, scale=sc, alibi=slopes[h])
        tau_err = np.abs(tau[0, h].cpu().double().numpy() - f["tau"]) / np.maximum(1.0, np.abs(f["tau"]))
        assert tau_err.max() <= parity.tau_tol(w.dtype), tau_err.max()
        assert np.abs(o[0, h].float().cpu().numpy() - f["o"]).max() <= parity.O_TOL
        rq, rk, rv = oracle_mod.attn_bwd_head(q, k, v, g, alpha, inp.sm_scale, causal, scale=sc, alibi=slopes[h])
        parity.grad_close("dQ", dq[0, h].float().cpu().numpy(), rq)
        parity.grad_close("dK", dk[0, h].float().cpu().numpy(), rk)
        parity.grad_close("dV", dv[0, h].float().cpu().numpy(), rv)
        dc_ref, gr = oracle_mod.attn_bwd_scale_head(q, k, v, g, alpha, inp.sm_scale, causal, scale=sc, alibi=slopes[h])
        parity.grad_close("dc rows", dc[0, h].cpu().numpy(), dc_ref)
        for idx in range(3 if grads is not None else 0):
            assert abs(float(grads[idx][h]) - gr[idx]) <= 2e-2 * max(1.0, abs(gr[idx])), (idx, float(grads[idx][h]), gr[idx])


@pytest.mark.parametrize("alpha", [1.25, 1.5, 2.0])
@pytest.mark.parametrize("N,d", [(700, 64), (4500, 128)])
def test_alibi_bf16_causal_sparse_rows(N, d, alpha):
    # head 0 without positional term, head 1 with a slope (NAPE); N = 4500 also runs the sampled pre-pass
    inp = make_inputs(_small("alibi", N, d, True, plant=2, backward=True, seed=N + 7))
    _check_alibi(inp, alpha, True, [0.0, 0.05], None)


def test_alibi_window_skips_far_tiles_and_keeps_parity():
    # NAPE-style heads at a length where the hard cutoff bites: slopes 0 (NoPE), 0.5, 0.1 and 0.02.  The sweep starts
    # every work item at the first K tile that can still hold a candidate (norm bound on the logits); forward and
    # backward (tau-only: its sweep has the exact threshold as its bound) must still match the oracle, which scores
    # every visible key
    N = 8192
    inp = make_inputs(Workload("alibi_window", 1, 4, N, 64, "bf16", True, (1.5,), plant=3, plant_mode="subset",
                               backward=True, seed_offset=83))
    slopes = [0.0, 0.5, 0.1, 0.02]
    dev = parity.to_device(inp)
    sl = torch.tensor(slopes, dtype=torch.float32, device="cuda")
    for alpha in (1.5, 2.0):
        st = torch.zeros(binding.STATUS_WORDS, dtype=torch.int32, device="cuda")
        o, tau = binding.entmax_attn_fwd_ex(dev["q"], dev["k"], dev["v"], alpha, True, dev["beta"], dev["gamma"],
                                            dev["delta"], alibi_slopes=sl, status=st)
        st2 = torch.zeros(binding.STATUS_WORDS, dtype=torch.int32, device="cuda")
        dq, dk, dv, _, _ = binding.entmax_attn_bwd_ex(dev["q"], dev["k"], dev["v"], tau, dev["d_o"], alpha, True,
                                                      dev["beta"], dev["gamma"], dev["delta"], alibi_slopes=sl, status=st2)
        torch.cuda.synchronize()
        assert int(st[binding.STATUS_FLAGS]) == 0 and int(st2[binding.STATUS_FLAGS]) == 0
        for status in (st, st2):
            skipped, scored = int(status[binding.STATUS_SKIPPED_STEPS]), int(status[binding.STATUS_SCORED_STEPS])
            # 4 heads x 32 items; an item at row r sees (r + 256) / 256 key tiles: 4 * (1 + ... + 32) steps in all
            assert skipped + scored == 4 * 32 * 33 // 2
            assert skipped > 0.4 * (skipped + scored), (skipped, scored)
        for h in range(4):
            q, k, v, g = (t[0, h].float().numpy() for t in (inp.q, inp.k, inp.v, inp.d_o))
            rows = sample_rows(inp, h, 160)
            f = oracle_mod.attn_fwd_rows(q, k, v, rows, alpha, inp.sm_scale, True, scale=inp.head_scale(h), alibi=slopes[h])
            rt = torch.from_numpy(rows)
            tau_err = np.abs(tau[0, h].cpu()[rt].double().numpy() - f["tau"]) / np.maximum(1.0, np.abs(f["tau"]))
            assert tau_err.max() <= parity.tau_tol("bf16"), (h, tau_err.max())
            assert np.abs(o[0, h].float().cpu()[rt].numpy() - f["o"]).max() <= parity.O_TOL
            if alpha < 2.0:
                rq, _ = oracle_mod.attn_bwd_rows(q, k, v, g, rows, alpha, inp.sm_scale, True, scale=inp.head_scale(h),
                                                 alibi=slopes[h])
                parity.grad_close("dQ rows", dq[0, h].float().cpu()[rt].numpy(), rq)
        # a whole head of dK, dV (every row contributes) on the steepest slope
        if alpha < 2.0:
            q, k, v, g = (t[0, 1].float().numpy() for t in (inp.q, inp.k, inp.v, inp.d_o))
            rq, rk, rv = oracle_mod.attn_bwd_head(q, k, v, g, alpha, inp.sm_scale, True, scale=inp.head_scale(1), alibi=slopes[1])
            parity.grad_close("dK", dk[0, 1].float().cpu().numpy(), rk)
            parity.grad_close("dV", dv[0, 1].float().cpu().numpy(), rv)


def test_alibi_bf16_causal_dense_rows():
    inp = make_inputs(_small("alibi_dense", 600, 128, True, backward=True, use_scale=False, sigma=0.05, seed=19))
    _check_alibi(inp, 1.5, True, [0.002, 0.0005], True)


@pytest.mark.parametrize("causal", [True, False])
def test_alibi_fp32_both_masks(causal):
    inp = make_inputs(_small("alibi32", 150, 64, causal, dtype="fp32", backward=True, seed=23))
    _check_alibi(inp, 1.5, causal, [0.1, 0.02], None)


def test_alibi_bf16_noncausal_is_rejected():
    inp = make_inputs(_small("alibi_nc", 128, 64, False, seed=29))
    dev = parity.to_device(inp)
    sl = torch.tensor([0.1, 0.1], dtype=torch.float32, device="cuda")
    with pytest.raises(binding.EntmaxAttnError, match="sm_100|unsupported|needs"):
        binding.entmax_attn_fwd_ex(dev["q"], dev["k"], dev["v"], 1.5, False, alibi_slopes=sl)


# ------------------------------------------------------------------ backward from the forward call's saved supports
@pytest.mark.parametrize("alpha", [1.25, 1.5, 2.0])
@pytest.mark.parametrize("N,d,sigma,plant", [(1300, 64, 1.0, 3), (700, 128, 1.0, 0), (400, 128, 0.05, 0)])
def test_backward_with_saved_forward_workspace(N, d, sigma, plant, alpha):
    # sigma 0.05: every row dense (row_count -2 in the saved workspace -> dense backward path)
    inp = make_inputs(_small("saved", N, d, True, plant=plant, backward=True, sigma=sigma, seed=N + 3))
    got = parity.run_fwd(inp, alpha)
    dev = got["dev"]
    ref = binding.entmax_attn_bwd_scale(dev["q"], dev["k"], dev["v"], got["tau"], dev["d_o"], alpha, True, dev["beta"],
                                        dev["gamma"], dev["delta"])
    dq, dk, dv, dc, grads = binding.entmax_attn_bwd_ex(dev["q"], dev["k"], dev["v"], got["tau"], dev["d_o"], alpha, True,
                                                       dev["beta"], dev["gamma"], dev["delta"],
                                                       fwd_workspace=got["workspace"], want_scale_rows=True,
                                                       want_param_grads=True)
    torch.cuda.synchronize()
    for name, a_, b_ in (("dq", dq, ref[0]), ("dk", dk, ref[1]), ("dv", dv, ref[2]), ("dc", dc, ref[3])):
        parity.grad_close(name, a_.float().cpu().numpy(), b_.float().cpu().numpy())
    for idx in range(3):
        parity.grad_close("param grad", grads[idx].cpu().numpy(), ref[4][idx].cpu().numpy())
    # and against the oracle directly
    bwd = {"dq": dq, "dk": dk, "dv": dv}
    parity.check_bwd_head(inp, alpha, bwd, 1)


# ------------------------------------------------------------------ the benchmark workloads
def test_cfg2_all_rows():
    inp = make_inputs(WORKLOADS[2])
    got = parity.run_fwd(inp, 1.5)
    w = inp.workload
    supp = []
    for bh in range(w.B * w.H):
        st = parity.check_fwd_rows(inp, 1.5, got, bh, np.arange(w.N))
        supp.append(st["supp_mean"])
    assert np.mean(supp) < 64      # planted keys make the rows sparse


def test_cfg3_forward_and_backward():
    inp = make_inputs(WORKLOADS[3])
    w = inp.workload
    got = parity.run_fwd(inp, 1.5)
    bwd = parity.run_bwd(inp, 1.5, got["tau"], got["dev"])
    full = [0, 21, 42, 63]
    for bh in range(w.B * w.H):
        if bh in full:
            parity.check_fwd_rows(inp, 1.5, got, bh, np.arange(w.N))
            parity.check_bwd_head(inp, 1.5, bwd, bh)
        elif bh % 4 == 1:
            rows = sample_rows(inp, bh, 256)
            parity.check_fwd_rows(inp, 1.5, got, bh, rows)
            parity.check_bwd_rows(inp, 1.5, bwd, bh, rows)
    _gradient_invariants(inp, bwd)


def _gradient_invariants(inp, bwd):
    # rows of P sum to one, so sum_j dV_j = sum_i dO_i; rows of dS sum to zero, so sum_j dK_j = 0 when
    # every row of a head shares one scale... (not the case with per-row c_i), hence only the dV identity.
    dv = bwd["dv"].float().sum(dim=2).cpu()
    do = inp.d_o.float().sum(dim=2)
    tol = 2e-2 * math.sqrt(inp.workload.N) * 4
    assert (dv - do).abs().max().item() <= tol


@pytest.mark.parametrize("alpha", [1.25, 1.5, 2.0])
def test_cfg4_sampled_rows(alpha, cfg4_inputs):
    inp = cfg4_inputs
    w = inp.workload
    got = parity.run_fwd(inp, alpha, dev=_cfg4_dev(inp))
    supp = []
    for bh in range(w.B * w.H):
        rows = sample_rows(inp, bh, 256)
        st = parity.check_fwd_rows(inp, alpha, got, bh, rows)
        supp.append(st["supp_mean"])
    # every row's probabilities sum to one: with V = 1 ... checked through O on sampled rows above; the
    # cheap global invariant is that tau is finite everywhere and no row was left unwritten
    assert torch.isfinite(got["tau"]).all() and torch.isfinite(got["o"].float()).all()
    print("cfg4 alpha=%g mean support %.1f dense rows %d" % (alpha, np.mean(supp), int(got["status"][1])))


@pytest.mark.parametrize("alpha", [1.25, 1.5, 2.0])
def test_cfg4_backward_at_size(alpha, cfg4_inputs):
    # the benchmark's own timed backward call: the long-context tensors plus the benchmark's seeded dO, through
    # entmax_attn_bwd (tau only), then the two saved-state variants compared with it
    inp = cfg4_inputs
    w = inp.workload
    if inp.d_o is None:
        inp.d_o = inputs.seeded_d_o(w)
    dev = _cfg4_dev(inp)
    if dev.get("d_o") is None:
        dev["d_o"] = inp.d_o.cuda()
    got = parity.run_fwd(inp, alpha, dev=dev)
    bwd = parity.run_bwd(inp, alpha, got["tau"], dev)
    for bh in range(w.B * w.H):
        rows = sample_rows(inp, bh, 256)
        parity.check_bwd_rows(inp, alpha, bwd, bh, rows)
    _gradient_invariants(inp, bwd)
    if alpha == 1.5:
        # one whole head against the oracle: dK and dV need every query row
        parity.check_bwd_head(inp, alpha, bwd, 5)
    # backward fed with the forward call's workspace, and with the compact copy of its supports
    st = torch.zeros(binding.STATUS_WORDS, dtype=torch.int32, device="cuda")
    full = binding.entmax_attn_bwd_ex(dev["q"], dev["k"], dev["v"], got["tau"], dev["d_o"], alpha, True, dev["beta"],
                                      dev["gamma"], dev["delta"], fwd_workspace=got["workspace"], status=st)
    saved = binding.entmax_attn_save_supports(dev["q"], alpha, True, got["workspace"])
    st2 = torch.zeros(binding.STATUS_WORDS, dtype=torch.int32, device="cuda")
    comp = binding.entmax_attn_bwd_ex(dev["q"], dev["k"], dev["v"], got["tau"], dev["d_o"], alpha, True, dev["beta"],
                                      dev["gamma"], dev["delta"], saved_supports=saved, status=st2)
    torch.cuda.synchronize()
    assert int(st[binding.STATUS_FLAGS]) == 0 and int(st2[binding.STATUS_FLAGS]) == 0
    for other in (full, comp):
        # dQ is row-local: the same supports give the same sums up to their order; dK, dV are sums over rows.
        # alpha = 2: u = 1 on the whole support, so a key within rounding of the threshold (the saved lists and
        # the recomputed scores differ by one rounding) flips a row's gradient: such rows must be few and each
        # must have a key inside the don't-care band of the threshold
        for bh in (0, 7, 15):
            a_dq, b_dq = other[0][0, bh].float().cpu().numpy(), bwd["dq"][0, bh].float().cpu().numpy()
            bad = parity.grad_mismatch_rows(a_dq, b_dq)
            if alpha < 2.0:
                assert len(bad) == 0, ("dq (saved state vs tau-only)", bh, bad[:8])
            else:
                assert len(bad) <= 8, ("dq (saved state vs tau-only): too many rows differ", bh, len(bad))
                for i in bad:
                    assert parity.threshold_margin(inp, alpha, bh, int(i)) <= parity.BAND, (bh, int(i))
            if alpha < 2.0 or len(bad) == 0:
                for name, a_, b_ in (("dk", other[1], bwd["dk"]), ("dv", other[2], bwd["dv"])):
                    parity.grad_close(name + " (saved state vs tau-only)", a_[0, bh].float().cpu().numpy(),
                                      b_[0, bh].float().cpu().numpy())
    del full, comp, saved, bwd, got
    torch.cuda.empty_cache()


_CFG4_DEV = {}


def _cfg4_dev(inp):
    if "dev" not in _CFG4_DEV:
        _CFG4_DEV["dev"] = parity.to_device(inp)
    return _CFG4_DEV["dev"]


@pytest.fixture(scope="module")
def cfg4_inputs():
    yield make_inputs(WORKLOADS[4])
    _CFG4_DEV.clear()


def test_cfg5_noncausal_retrieval():
    inp = make_inputs(WORKLOADS[5])
    w = inp.workload
    got = parity.run_fwd(inp, 1.5)
    bwd = parity.run_bwd(inp, 1.5, got["tau"], got["dev"])
    supp = []
    for bh in range(w.B * w.H):
        rows = sample_rows(inp, bh, 128)
        st = parity.check_fwd_rows(inp, 1.5, got, bh, rows)
        supp.append(st["supp_mean"])
        parity.check_bwd_rows(inp, 1.5, bwd, bh, rows)
    assert np.mean(supp) < 4
    _gradient_invariants(inp, bwd)


def test_long_sequences_with_byte_offsets_beyond_32_bits():
    # 18 heads x 131072 rows: 2.36 M rows, so the candidate lists span 4.8 GB and the row index times the list pitch
    # no longer fits 32 bits; the longest sequence any test runs.  Sampled rows of three heads, forward and dQ.
    inp = make_inputs(Workload("long_rows", 1, 18, 131072, 64, "bf16", True, (1.5,), backward=True, seed_offset=77))
    w = inp.workload
    got = parity.run_fwd(inp, 1.5)
    bwd = parity.run_bwd(inp, 1.5, got["tau"], got["dev"])
    for bh in (0, 9, 17):
        rows = sample_rows(inp, bh, 48)
        parity.check_fwd_rows(inp, 1.5, got, bh, rows)
        parity.check_bwd_rows(inp, 1.5, bwd, bh, rows)
    _gradient_invariants(inp, bwd)
    del got, bwd
    torch.cuda.empty_cache()


def test_cfg5_one_full_head_backward_at_size():
    # dK and dV need every query row: one seeded head of the retrieval workload at its real length (the oracle
    # spends about a minute on it), forward rows on a stride
    inp = make_inputs(WORKLOADS[5])
    w = inp.workload
    got = parity.run_fwd(inp, 1.5)
    bwd = parity.run_bwd(inp, 1.5, got["tau"], got["dev"])
    bh = int(np.random.default_rng(20250616 + 5).integers(w.B * w.H))
    parity.check_fwd_rows(inp, 1.5, got, bh, np.arange(0, w.N, 97))
    parity.check_bwd_head(inp, 1.5, bwd, bh)
    del got, bwd
    torch.cuda.empty_cache()


def test_cfg5_shape_reduced_full_backward():
    # same recipe at N = 4096 so that dK and dV of a whole head can be checked against the oracle
    inp = make_inputs(scaled(WORKLOADS[5], N=4096, H=2, name="cfg5_reduced"))
    got = parity.run_fwd(inp, 1.5)
    bwd = parity.run_bwd(inp, 1.5, got["tau"], got["dev"])
    parity.check_fwd_rows(inp, 1.5, got, 1, np.arange(4096))
    parity.check_bwd_head(inp, 1.5, bwd, 1)
