"""Decode-shape forward (entmax_attn_decode_fwd) against the CPU oracle.

A decode problem is cut out of a seeded full problem [B,H,N,d]: sequence b keeps its first kv_len[b] keys
and values as the cache, and its q_len query rows are the full problem's rows kv_len[b]-q_len .. kv_len[b]-1.
The oracle then answers with those rows of the causal problem of length kv_len[b] (Eq. 1 on the ASEntmax-scaled
logits, n_i = position + 1), which is what the entry point defines.  Tolerances as in tests/parity.py.
"""
import numpy as np
import pytest
import torch

import oracle as oracle_mod
import parity
from paper_2506_16640_b200 import binding
from paper_2506_16640_b200.inputs import Workload, make_inputs

pytestmark = pytest.mark.gpu


def _problem(B, H, N, d, plant=0, use_scale=True, sigma=1.0, seed=0):
    w = Workload("decode", B, H, N, d, "bf16", True, (1.5,), qk_sigma=sigma, plant=plant,
                 plant_mode="subset" if plant else "none", use_scale=use_scale, seed_offset=100 + seed)
    return make_inputs(w)


def _lengths(B, N, q_len, seed, ragged):
    if not ragged:
        return np.full(B, N, dtype=np.int32)
    rng = np.random.default_rng(seed)
    lens = rng.integers(q_len, N + 1, size=B).astype(np.int32)
    lens[0] = N                      # one sequence fills the cache
    if B > 1:
        lens[-1] = q_len             # one holds nothing but the new rows
    return lens


def _run(inp, lens, q_len, alpha, slopes=None, cache_layout="bhnd"):
    w = inp.workload
    dev = torch.device("cuda")
    idx = torch.from_numpy(np.stack([np.arange(int(L) - q_len, int(L)) for L in lens]))          # [B, q_len]
    q = torch.stack([inp.q[b][:, idx[b]] for b in range(w.B)]).contiguous().to(dev)                # [B,H,q_len,d]
    if cache_layout == "bnhd":
        k = inp.k.permute(0, 2, 1, 3).contiguous().to(dev).permute(0, 2, 1, 3)                     # a view, d innermost
        v = inp.v.permute(0, 2, 1, 3).contiguous().to(dev).permute(0, 2, 1, 3)
    else:
        k, v = inp.k.to(dev), inp.v.to(dev)
    kv_len = torch.from_numpy(lens).to(dev)
    sc = [t.to(dev) if t is not None else None for t in (inp.beta, inp.gamma, inp.delta)]
    al = torch.tensor(slopes, dtype=torch.float32, device=dev) if slopes is not None else None
    status = torch.full((binding.STATUS_WORDS,), -1, dtype=torch.int32, device=dev)
    o, tau, supp = binding.entmax_attn_decode_fwd(q, k, v, alpha, kv_len, sc[0], sc[1], sc[2], alibi_slopes=al,
                                                  status=status)
    torch.cuda.synchronize()
    return {"o": o.cpu(), "tau": tau.cpu(), "supp": supp.cpu(), "status": status.cpu()}


def _check(inp, lens, q_len, alpha, got, slopes=None, heads=None):
    w = inp.workload
    for b in range(w.B):
        L = int(lens[b])
        rows = np.arange(L - q_len, L)
        for h in (range(w.H) if heads is None else heads):
            q, k, v = (t[b, h, :L].float().numpy() for t in (inp.q, inp.k, inp.v))
            m = 0.0 if slopes is None else float(slopes[h])
            ref = oracle_mod.attn_fwd_rows(q, k, v, rows, alpha, inp.sm_scale, True, scale=inp.head_scale(h), want_p=True,
                                           alibi=m)
            tau_g = got["tau"][b, h].double().numpy()
            o_g = got["o"][b, h].double().numpy()
            tau_err = np.abs(tau_g - ref["tau"]) / np.maximum(1.0, np.abs(ref["tau"]))
            assert tau_err.max() <= parity.tau_tol("bf16"), (b, h, tau_g, ref["tau"])
            o_err = np.abs(o_g - ref["o"]).max(axis=1)
            # support size: exact unless keys sit within the band around the threshold
            sc = inp.head_scale(h)
            for t, i in enumerate(rows):
                c = oracle_mod.asentmax_scale(sc[0], sc[1], sc[2], int(i) + 1) if sc is not None else 1.0
                z = (k[: i + 1].astype(np.float64) @ q[i].astype(np.float64)) * inp.sm_scale - m * (i - np.arange(i + 1))
                y = (alpha - 1) * c * z
                in_band = int((np.abs(y - ref["tau"][t]) <= parity.BAND).sum())
                assert abs(int(got["supp"][b, h, t]) - int(ref["supp"][t])) <= in_band, (b, h, t)
                # alpha > 2: a key inside the band weighs up to BAND^(1/(alpha-1)); such a row is beyond float32
                assert o_err[t] <= parity.O_TOL or (alpha > 2.0 and in_band > 0), (b, h, t, o_err[t])


@pytest.mark.parametrize("alpha", [1.25, 1.5, 2.0, 1.7, 3.0])
@pytest.mark.parametrize("B,H,N,d,q_len,plant", [(2, 3, 700, 64, 1, 3), (2, 2, 1500, 128, 4, 0), (1, 2, 2100, 128, 8, 3),
                                                 (3, 2, 513, 64, 3, 0), (2, 2, 8, 64, 8, 0), (1, 1, 1, 128, 1, 0),
                                                 (2, 2, 1030, 128, 2, 2), (1, 2, 600, 64, 5, 0)])
def test_decode_matches_oracle_rows(B, H, N, d, q_len, plant, alpha):
    inp = _problem(B, H, N, d, plant=plant if N > 40 else 0, seed=N + q_len)
    for ragged in (False, True):
        lens = _lengths(B, N, q_len, N, ragged)
        got = _run(inp, lens, q_len, alpha)
        assert int(got["status"][binding.STATUS_FLAGS]) == 0
        _check(inp, lens, q_len, alpha, got)


def test_decode_fixed_temperature_and_strided_cache():
    # no scale parameters (c = 1); the cache is stored [B, N, H, d] and passed as a strided view
    inp = _problem(2, 4, 900, 128, plant=2, use_scale=False, seed=5)
    lens = _lengths(2, 900, 2, 9, True)
    got = _run(inp, lens, 2, 1.5, cache_layout="bnhd")
    _check(inp, lens, 2, 1.5, got)
    same = _run(inp, lens, 2, 1.5)
    assert torch.equal(got["o"], same["o"]) and torch.equal(got["tau"], same["tau"])


@pytest.mark.parametrize("alpha", [1.5, 2.0])
def test_decode_with_alibi_slopes(alpha):
    inp = _problem(2, 4, 800, 64, plant=2, seed=6)
    slopes = [0.0, 0.5, 0.0625, 0.0078125]          # one head without positional term
    lens = _lengths(2, 800, 3, 4, True)
    got = _run(inp, lens, 3, alpha, slopes=slopes)
    _check(inp, lens, 3, alpha, got, slopes=slopes)


@pytest.mark.parametrize("alpha", [1.25, 1.5, 2.0])
def test_decode_dense_rows_are_solved_on_the_score_row(alpha):
    # tiny logits: thousands of keys in every support, far beyond the on-chip candidate list
    inp = _problem(1, 2, 5000, 128, use_scale=False, sigma=0.01 if alpha == 2.0 else 0.03, seed=8)
    lens = _lengths(1, 5000, 4, 0, False)
    got = _run(inp, lens, 4, alpha)
    assert int(got["status"][binding.STATUS_DENSE_ROWS]) == 2 * 4
    assert int(got["supp"].min()) > 2048
    _check(inp, lens, 4, alpha, got)


def test_decode_is_bitwise_reproducible():
    inp = _problem(2, 4, 3000, 128, plant=3, seed=9)
    lens = _lengths(2, 3000, 4, 1, True)
    first = _run(inp, lens, 4, 1.5)
    for _ in range(3):
        again = _run(inp, lens, 4, 1.5)
        for name in ("o", "tau", "supp"):
            assert torch.equal(first[name], again[name]), name


def test_decode_flags_lengths_outside_the_cache():
    inp = _problem(2, 2, 300, 64, seed=10)
    lens = np.array([300, 2], dtype=np.int32)        # second sequence shorter than its 4 new rows
    got = _run(inp, lens, 4, 1.5)
    assert int(got["status"][binding.STATUS_FLAGS]) & binding.FLAG_BAD_LENGTH
    ok = _run(inp, np.array([300, 4], dtype=np.int32), 4, 1.5)
    assert int(ok["status"][binding.STATUS_FLAGS]) == 0


def test_decode_long_cache_sampled_heads():
    # the benchmark's long-context shape as a decode problem: 16 heads, 32768 cached keys, d = 128
    inp = make_inputs(Workload("decode_long", 2, 16, 32768, 128, "bf16", True, (1.5,), plant=8, plant_mode="subset",
                               seed_offset=111))
    lens = np.array([32768, 20011], dtype=np.int32)
    got = _run(inp, lens, 2, 1.5)
    assert int(got["status"][binding.STATUS_FLAGS]) == 0
    _check(inp, lens, 2, 1.5, got, heads=[0, 7, 15])
