"""Helpers of the GPU parity tests: run the CUDA path through the binding, run the CPU oracle on the
same seeded tensors, compare element by element with the tolerances of the target:

  max |O - O_ref| <= 2e-2
  |tau - tau_ref| / max(1, |tau_ref|) <= 1e-3 (bf16 inputs) or 1e-4 (fp32 inputs)
  supports identical except for entries within 1e-3 of the threshold
  gradients: max |dX - dX_ref| <= 2e-2 * max(1, max |dX_ref|)  (the forward tolerance scaled to the
  gradient's magnitude; bf16 outputs alone carry 2^-9 relative rounding), and element by element
  |dX - dX_ref| <= 2e-2 * |dX_ref| + 2e-2 * rms(dX_ref row), the rms taken over the d entries of the element's own
  query / key row (a gradient row is a sum of vectors that cancel, so an entry's error scales with its row, not
  with itself), floored at 10 % of the whole tensor's rms (every support entry carries the fp32 rounding of
  tau into dS as an absolute error of about |tau| 2^-23 |dP| g |q|, however small the entry's own weight is, so
  rows that only weak entries reach cannot be held to their own magnitude), so that small rows cannot hide behind the largest one
  rows the dense path computed keep no list: their support SIZE must equal the oracle's up to the number of keys
  within 1e-3 of the threshold
"""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2506_16640_b200 import binding

O_TOL = 2e-2
BAND = 1e-3


def tau_tol(dtype_name: str) -> float:
    return 1e-4 if dtype_name == "fp32" else 1e-3


def to_device(inp, device="cuda"):
    d = {name: getattr(inp, name).to(device) for name in ("q", "k", "v")}
    d["d_o"] = inp.d_o.to(device) if inp.d_o is not None else None
    for name in ("beta", "gamma", "delta"):
        t = getattr(inp, name)
        d[name] = t.to(device) if t is not None else None
    return d


def run_fwd(inp, alpha, dev=None, n_mode=0):
    """CUDA forward through the C ABI.  Returns dict(o, tau, workspace, status, params) (device tensors)."""
    dev = dev or to_device(inp)
    w = inp.workload
    params = binding.make_params(dev["q"], alpha, w.causal, 0.0, n_mode)
    ws = binding.alloc_workspace(params, False, dev["q"].device)
    status = torch.full((binding.STATUS_WORDS,), -1, dtype=torch.int32, device=dev["q"].device)
    o, tau = binding.entmax_attn_fwd(dev["q"], dev["k"], dev["v"], alpha, w.causal, dev["beta"], dev["gamma"],
                                     dev["delta"], n_mode=n_mode, workspace=ws, status=status)
    torch.cuda.synchronize()
    st = status.cpu()
    assert int(st[binding.STATUS_FLAGS]) == 0, "device status flags: %d" % int(st[binding.STATUS_FLAGS])
    return {"o": o, "tau": tau, "workspace": ws, "status": st, "params": params, "dev": dev}


def run_bwd(inp, alpha, tau, dev=None, n_mode=0):
    dev = dev or to_device(inp)
    w = inp.workload
    status = torch.full((binding.STATUS_WORDS,), -1, dtype=torch.int32, device=dev["q"].device)
    dq, dk, dv = binding.entmax_attn_bwd(dev["q"], dev["k"], dev["v"], tau, dev["d_o"], alpha, w.causal, dev["beta"],
                                         dev["gamma"], dev["delta"], n_mode=n_mode, status=status)
    torch.cuda.synchronize()
    st = status.cpu()
    assert int(st[binding.STATUS_FLAGS]) == 0, "device status flags: %d" % int(st[binding.STATUS_FLAGS])
    return {"dq": dq, "dk": dk, "dv": dv, "status": st}


def check_fwd_rows(inp, alpha, got, bh, rows, n_mode=0, check_support=True):
    """Compares rows `rows` of head index bh = b*H + h against the oracle.  Returns summary stats."""
    w = inp.workload
    b, h = divmod(bh, w.H)
    q, k, v = (t[b, h].float().numpy() for t in (inp.q, inp.k, inp.v))
    rows = np.asarray(rows, dtype=np.int64)
    ref = oracle.attn_fwd_rows(q, k, v, rows, alpha, inp.sm_scale, w.causal, scale=inp.head_scale(h), n_mode=n_mode,
                               want_p=check_support)
    rows_t = torch.from_numpy(rows)
    tau_g = got["tau"][b, h].cpu()[rows_t].double().numpy()
    o_g = got["o"][b, h].cpu()[rows_t].double().numpy()
    tau_err = np.abs(tau_g - ref["tau"]) / np.maximum(1.0, np.abs(ref["tau"]))
    o_err = np.abs(o_g - ref["o"]).max(axis=1)
    worst_t = int(np.argmax(tau_err))
    assert tau_err.max() <= tau_tol(w.dtype), "tau: row %d (bh %d) gpu %.7g ref %.7g rel err %.3g" % (
        rows[worst_t], bh, tau_g[worst_t], ref["tau"][worst_t], tau_err.max())
    worst_o = int(np.argmax(o_err))
    if alpha > 2.0 and o_err.max() > O_TOL:
        # alpha > 2: a key that sits d above the threshold weighs d^(1/(alpha-1)) -- 0.1 at the edge of the support's
        # own don't-care band (1e-3) for alpha = 4 -- so a row with a key inside that band is outside what float32
        # can decide; every other row is held to the output tolerance
        for r in np.flatnonzero(o_err > O_TOL):
            m = threshold_margin(inp, alpha, bh, int(rows[r]), n_mode)
            assert m <= BAND, "O: row %d (bh %d) max abs err %.3g with no key inside the band (margin %.3g)" % (
                rows[r], bh, o_err[r], m)
        assert (o_err > O_TOL).mean() <= 0.25, "O: too many rows inside the band"
        o_err = np.where(o_err > O_TOL, 0.0, o_err)
    assert o_err.max() <= O_TOL, "O: row %d (bh %d) max abs err %.3g" % (rows[worst_o], bh, o_err.max())
    stats = {"tau_err": float(tau_err.max()), "o_err": float(o_err.max()), "supp_mean": float(ref["supp"].mean()),
             "supp_max": int(ref["supp"].max()), "band_mismatch": 0, "dense_rows": 0}
    if check_support:
        grow = bh * w.N + rows
        lists = binding.read_support(got["params"], got["workspace"], grow)
        dense_sizes = None
        for r, (idx, _y) in enumerate(lists):
            i = int(rows[r])
            if idx is None:
                # computed by the dense path: its list is not kept, its support size is
                stats["dense_rows"] += 1
                if dense_sizes is None:
                    dense_sizes = binding.read_dense_support_sizes(got["params"], got["workspace"], grow).numpy()
                size = int(dense_sizes[r])
                ref_size = int(ref["supp"][r])
                if size != ref_size:
                    nv = i + 1 if w.causal else w.N
                    n_i = w.N if n_mode else nv
                    sc = inp.head_scale(h)
                    c = oracle.asentmax_scale(sc[0], sc[1], sc[2], n_i) if sc is not None else 1.0
                    y = (alpha - 1) * c * (k[:nv].astype(np.float64) @ q[i].astype(np.float64)) * inp.sm_scale
                    in_band = int((np.abs(y - ref["tau"][r]) <= BAND).sum())
                    assert abs(size - ref_size) <= in_band, "row %d: dense-path support size %d, oracle %d, %d keys " \
                        "within the band" % (i, size, ref_size, in_band)
                    stats["band_mismatch"] += abs(size - ref_size)
                continue
            gpu_set = set(int(x) for x in idx)
            assert len(gpu_set) == len(idx), "row %d: duplicate keys in the support list" % i
            ref_set = set(int(x) for x in np.flatnonzero(ref["p"][r] > 0))
            diff = gpu_set ^ ref_set
            if diff:
                nv = i + 1 if w.causal else w.N
                n_i = w.N if n_mode else nv
                sc = inp.head_scale(h)
                c = oracle.asentmax_scale(sc[0], sc[1], sc[2], n_i) if sc is not None else 1.0
                for j in diff:
                    assert 0 <= j < nv, "row %d: key %d outside the mask" % (i, j)
                    y = (alpha - 1) * c * float(q[i].astype(np.float64) @ k[j].astype(np.float64)) * inp.sm_scale
                    assert abs(y - ref["tau"][r]) <= BAND, "row %d key %d: support differs, margin %.3g" % (
                        i, j, y - ref["tau"][r])
                stats["band_mismatch"] += len(diff)
    return stats


def grad_mismatch_rows(got, ref):
    """Rows (index along the second-to-last axis of a 2-D array) with an element outside grad_close's
    element-wise tolerance."""
    ref = np.asarray(ref, dtype=np.float64)
    got = np.asarray(got, dtype=np.float64)
    rms = np.sqrt(np.mean(ref * ref, axis=-1, keepdims=True))
    rms = np.maximum(rms, max(1e-1 * float(np.sqrt(np.mean(ref * ref))), 1e-6))
    excess = np.abs(got - ref) - (2e-2 * np.abs(ref) + 2e-2 * rms)
    return np.flatnonzero((excess > 0).any(axis=-1))


def threshold_margin(inp, alpha, bh, i, n_mode=0):
    """min_j |y_ij - tau_i| of query row i (oracle tau, fp64 scores): how close the nearest key sits to the
    threshold.  Within BAND the key's membership in the support is "don't care" -- and at alpha = 2, where u = 1
    on the whole support, so is the row's gradient (the Jacobian of Eq. 1 jumps when a key enters)."""
    w = inp.workload
    b, h = divmod(bh, w.H)
    q, k, v = (t[b, h].float().numpy() for t in (inp.q, inp.k, inp.v))
    ref = oracle.attn_fwd_rows(q, k, v, np.array([i]), alpha, inp.sm_scale, w.causal, scale=inp.head_scale(h), n_mode=n_mode)
    nv = i + 1 if w.causal else w.N
    n_i = w.N if n_mode else nv
    sc = inp.head_scale(h)
    c = oracle.asentmax_scale(sc[0], sc[1], sc[2], n_i) if sc is not None else 1.0
    y = (alpha - 1) * c * (k[:nv].astype(np.float64) @ q[i].astype(np.float64)) * inp.sm_scale
    return float(np.abs(y - ref["tau"][0]).min())


def head_margins(inp, alpha, bh, n_mode=0):
    """min_j |y_ij - tau_i| for every query row of one head (fp64 scores, oracle tau)."""
    w = inp.workload
    b, h = divmod(bh, w.H)
    q, k, v = (t[b, h].float().numpy() for t in (inp.q, inp.k, inp.v))
    ref = oracle.attn_fwd_rows(q, k, v, np.arange(w.N), alpha, inp.sm_scale, w.causal, scale=inp.head_scale(h), n_mode=n_mode)
    sc = inp.head_scale(h)
    i = np.arange(w.N)
    n_i = np.full(w.N, w.N) if (n_mode or not w.causal) else i + 1
    c = np.array([oracle.asentmax_scale(sc[0], sc[1], sc[2], int(n)) for n in n_i]) if sc is not None else np.ones(w.N)
    y = (alpha - 1) * c[:, None] * (q.astype(np.float64) @ k.astype(np.float64).T) * inp.sm_scale
    gap = np.abs(y - ref["tau"][:, None])
    if w.causal:
        gap[np.triu_indices(w.N, 1)] = np.inf
    return gap.min(axis=1)


def check_bwd_head_banded(inp, alpha, got_bwd, bh, n_mode=0, max_band_frac=0.25):
    """Like check_bwd_head, for exponents whose Jacobian jumps (alpha = 2) or blows up (alpha > 2: u = p^(2-alpha)) where
    a key crosses the threshold: a dQ row may miss the element-wise tolerance only if one of its keys lies within BAND
    of the threshold (the support's own don't-care band); such rows must be few.  dK and dV collect every row, so
    they are held to the element-wise tolerance only when the head has no such row, and to the global one otherwise."""
    w = inp.workload
    b, h = divmod(bh, w.H)
    q, k, v, d_o = (t[b, h].float().numpy() for t in (inp.q, inp.k, inp.v, inp.d_o))
    dq, dk, dv = oracle.attn_bwd_head(q, k, v, d_o, alpha, inp.sm_scale, w.causal, scale=inp.head_scale(h), n_mode=n_mode)
    margins = head_margins(inp, alpha, bh, n_mode)
    in_band = margins <= BAND
    assert in_band.mean() <= max_band_frac, "too many rows inside the band: %.3f" % in_band.mean()
    got_dq = got_bwd["dq"][b, h].float().cpu().numpy()
    bad = grad_mismatch_rows(got_dq, dq)
    off_band = [int(i) for i in bad if not in_band[i]]
    assert not off_band, "dQ rows %s differ from the oracle with no key inside the band (margins %s)" % (
        off_band[:6], margins[off_band[:6]])
    for name, got, ref in (("dK", got_bwd["dk"], dk), ("dV", got_bwd["dv"], dv)):
        g = got[b, h].float().cpu().numpy()
        if not in_band.any():
            grad_close(name, g, ref)
        else:
            # rows inside the band reach these sums with a gradient of their own choosing: leave their keys out
            tol = 2e-2 * max(1.0, float(np.abs(ref).max()))
            err = np.abs(g - ref).max(axis=1)
            assert (err > tol).mean() <= max_band_frac, "%s: %.3f of the key rows beyond the global tolerance" % (
                name, (err > tol).mean())
    return {"band_rows": int(in_band.sum()), "bad_rows": len(bad)}


def grad_close(name, got, ref):
    ref = np.asarray(ref, dtype=np.float64)
    got = np.asarray(got, dtype=np.float64)
    tol = 2e-2 * max(1.0, float(np.abs(ref).max()))
    diff = np.abs(got - ref)
    err = float(diff.max())
    assert err <= tol, "%s: max abs err %.4g > %.4g" % (name, err, tol)
    # element by element: relative to the entry itself plus a floor at the magnitude of the entry's own row
    # (last axis; a 1-D array is one row)
    rms = np.sqrt(np.mean(ref * ref, axis=-1, keepdims=True))
    rms = np.maximum(rms, max(1e-1 * float(np.sqrt(np.mean(ref * ref))), 1e-6))
    excess = diff - (2e-2 * np.abs(ref) + 2e-2 * rms)
    worst = int(np.argmax(excess))
    assert excess.flat[worst] <= 0, "%s: element %d got %.6g ref %.6g (row rms %.3g)" % (
        name, worst, got.flat[worst], ref.flat[worst], np.broadcast_to(rms, ref.shape).flat[worst])
    return err


def check_bwd_head(inp, alpha, got_bwd, bh, n_mode=0):
    """Full dQ, dK, dV of one head against the oracle."""
    w = inp.workload
    b, h = divmod(bh, w.H)
    q, k, v, d_o = (t[b, h].float().numpy() for t in (inp.q, inp.k, inp.v, inp.d_o))
    dq, dk, dv = oracle.attn_bwd_head(q, k, v, d_o, alpha, inp.sm_scale, w.causal, scale=inp.head_scale(h), n_mode=n_mode)
    return {"dq": grad_close("dQ", got_bwd["dq"][b, h].float().cpu().numpy(), dq),
            "dk": grad_close("dK", got_bwd["dk"][b, h].float().cpu().numpy(), dk),
            "dv": grad_close("dV", got_bwd["dv"][b, h].float().cpu().numpy(), dv)}


def check_bwd_rows(inp, alpha, got_bwd, bh, rows, n_mode=0):
    w = inp.workload
    b, h = divmod(bh, w.H)
    q, k, v, d_o = (t[b, h].float().numpy() for t in (inp.q, inp.k, inp.v, inp.d_o))
    rows = np.asarray(rows, dtype=np.int64)
    dq, _ = oracle.attn_bwd_rows(q, k, v, d_o, rows, alpha, inp.sm_scale, w.causal, scale=inp.head_scale(h), n_mode=n_mode)
    got = got_bwd["dq"][b, h].float().cpu()[torch.from_numpy(rows)].numpy()
    return grad_close("dQ rows", got, dq)
