"""Small, named problems for profiling the kernels one at a time (e.g. under ncu):

    python -m paper_2506_16640_b200.profile_cases CASE [--iters K] [--alpha A]

    dense     16 heads x 4096 x d=128, causal, logits of sigma 0.03: every row takes the dense-tile kernels
    dense8k   the same at 8192 tokens
    sweep8k   16 heads x 8192 x d=128, causal, the long-context recipe (8 planted keys) at a quarter of its length
    cfg3      the 4 x 16 x 8192 x d=64 forward + backward workload
    cfg4      the long-context workload itself (1 x 16 x 32768 x d=128)

Each iteration is one forward and one backward call; the per-call device times are printed.  Marshalling only:
every step runs in the library's kernels.
"""
from __future__ import annotations

import argparse
import statistics

import torch

from . import binding
from .inputs import WORKLOADS, Workload, make_inputs, scaled, seeded_d_o

CASES = {
    "dense": Workload("profile_dense_16x4096x128", 1, 16, 4096, 128, "bf16", True, (1.5,), qk_sigma=0.03, backward=True,
                      seed_offset=301),
    "dense8k": Workload("profile_dense_16x8192x128", 1, 16, 8192, 128, "bf16", True, (1.5,), qk_sigma=0.03, backward=True,
                        seed_offset=303),
    "sweep8k": scaled(WORKLOADS[4], N=8192, name="profile_sweep_16x8192x128", backward=True, seed_offset=302),
    "cfg3": WORKLOADS[3],
    "cfg4": WORKLOADS[4],
}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("case", choices=sorted(CASES))
    ap.add_argument("--iters", type=int, default=3)
    ap.add_argument("--alpha", type=float, default=1.5)
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("needs a CUDA device")
    w = CASES[args.case]
    inp = make_inputs(w)
    if inp.d_o is None:
        inp.d_o = seeded_d_o(w)
    dev = torch.device("cuda")
    t = {n: getattr(inp, n).to(dev) for n in ("q", "k", "v", "d_o", "beta", "gamma", "delta")}
    params = binding.make_params(t["q"], args.alpha, w.causal)
    ws = binding.alloc_workspace(params, True, dev)
    st = torch.zeros(binding.STATUS_WORDS, dtype=torch.int32, device=dev)
    st_b = torch.zeros(binding.STATUS_WORDS, dtype=torch.int32, device=dev)
    o = torch.empty_like(t["q"])
    tau = torch.empty((w.B, w.H, w.N), dtype=torch.float32, device=dev)
    dq, dk, dv = (torch.empty_like(t["q"]) for _ in range(3))
    ev = lambda: torch.cuda.Event(enable_timing=True)
    tf, tb = [], []
    for it in range(args.iters + (1 if args.iters > 1 else 0)):
        e0, e1, e2 = ev(), ev(), ev()
        e0.record()
        binding.entmax_attn_fwd(t["q"], t["k"], t["v"], args.alpha, w.causal, t["beta"], t["gamma"], t["delta"], o=o, tau=tau,
                                workspace=ws, status=st)
        e1.record()
        binding.entmax_attn_bwd(t["q"], t["k"], t["v"], tau, t["d_o"], args.alpha, w.causal, t["beta"], t["gamma"],
                                t["delta"], dq=dq, dk=dk, dv=dv, workspace=ws, status=st_b)
        e2.record()
        torch.cuda.synchronize()
        if it > 0 or args.iters == 1:          # with more than one iteration the first is a warm-up
            tf.append(e0.elapsed_time(e1))
            tb.append(e1.elapsed_time(e2))
    f, b = st.tolist(), st_b.tolist()
    pairs = (w.N * (w.N + 1) // 2 if w.causal else w.N * w.N) * w.B * w.H
    fwd_ms, bwd_ms = statistics.median(tf), statistics.median(tb)
    print("%s alpha %g: fwd %.3f ms (%.1f dense-equivalent TFLOP/s) bwd %.3f ms (%.1f) | forward: flags %d dense rows %d "
          "tiles %d sweeps/tile %.2f | backward: flags %d dense rows %d tiles %d"
          % (w.name, args.alpha, fwd_ms, 4 * w.d * pairs / fwd_ms / 1e9, bwd_ms, 10 * w.d * pairs / bwd_ms / 1e9, f[0], f[1], f[3],
             f[2] / max(f[3], 1), b[0], b[1], b[3]))
    assert f[0] == 0 and b[0] == 0, "device status flags set"


if __name__ == "__main__":
    main()
