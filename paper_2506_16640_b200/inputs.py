"""Seeded synthetic inputs shared by the CPU oracle tests and the CUDA parity tests / benchmark.

This module holds no arithmetic of the attention method itself: it only draws Q, K, V, dO and the
per-head scale parameters, plants high-similarity keys, rounds once to the workload's dtype and
picks the query rows that get checked.  Everything is generated on the CPU from a seed.

The five workloads stand in for the paper's synthetic-task and language-model attention shapes
(12 heads x d=64 x n=1024 is the learned-scale study; d=64 with 1K-16K contexts is the 420M LM;
16 heads at 8K-65K is the retrieval extrapolation range); no item of any dataset is reproduced.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Optional

import numpy as np
import torch

BASE_SEED = 20250616


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    B: int
    H: int
    N: int
    d: int
    dtype: str            # "bf16" | "fp32"
    causal: bool
    alphas: tuple
    qk_sigma: float = 1.0
    plant: int = 0        # planted keys per planted query
    plant_mode: str = "none"   # "none" | "subset" (random free slots) | "shift" (cyclic shift, every query)
    use_scale: bool = True     # draw beta, gamma, delta ~ U[0.5, 1.5] per head
    backward: bool = False
    seed_offset: int = 0


WORKLOADS = {
    1: Workload("cfg1_fixed_temp_fp32_n128", 1, 2, 128, 64, "fp32", True, (1.5,), use_scale=False, seed_offset=1),
    2: Workload("cfg2_asentmax_bf16_n1024_planted4", 8, 12, 1024, 64, "bf16", True, (1.5,), plant=4,
                plant_mode="subset", seed_offset=2),
    3: Workload("cfg3_asentmax_bf16_n8192_fwd_bwd", 4, 16, 8192, 64, "bf16", True, (1.5,), backward=True,
                seed_offset=3),
    4: Workload("cfg4_asentmax_bf16_n32768_d128_planted8", 1, 16, 32768, 128, "bf16", True, (1.25, 1.5, 2.0),
                plant=8, plant_mode="subset", seed_offset=4),
    5: Workload("cfg5_noncausal_bf16_n65536_retrieval", 1, 8, 65536, 64, "bf16", False, (1.5,), qk_sigma=0.25,
                plant=1, plant_mode="shift", backward=True, seed_offset=5),
}


@dataclasses.dataclass
class Inputs:
    workload: Workload
    q: torch.Tensor            # [B,H,N,d] in the workload dtype (CPU)
    k: torch.Tensor
    v: torch.Tensor
    d_o: Optional[torch.Tensor]
    beta: Optional[torch.Tensor]    # [H] float32 or None (fixed temperature)
    gamma: Optional[torch.Tensor]
    delta: Optional[torch.Tensor]
    planted_rows: list          # per (b*H+h): np.ndarray of planted query indices
    sm_scale: float

    def head_scale(self, h: int):
        """(beta, gamma, delta) of head h as Python floats (exact fp32 values), or None."""
        if self.beta is None:
            return None
        return (float(self.beta[h]), float(self.gamma[h]), float(self.delta[h]))


def scaled(w: Workload, **kw) -> Workload:
    """A workload with some fields replaced (smaller shapes for tests)."""
    return dataclasses.replace(w, **kw)


def _torch_dtype(name: str):
    return {"bf16": torch.bfloat16, "fp32": torch.float32}[name]


def _plant_subset(q_h: torch.Tensor, k_h: torch.Tensor, p: int, causal: bool, gen: torch.Generator):
    """Planted queries are i with i mod (p+1) == p, taken in increasing order; each takes p key slots
    uniformly from the still-unassigned slots it can see and those K rows are overwritten with
    3*sqrt(d)*q_i/||q_i|| + N(0, sigma=0.1).  Returns the planted query indices."""
    N, d = q_h.shape
    planted = np.arange(p, N, p + 1, dtype=np.int64)
    R = planted.shape[0]
    if R == 0:
        return planted
    u = torch.rand((R, p), generator=gen, dtype=torch.float64).numpy()
    noise = torch.randn((R, p, d), generator=gen, dtype=torch.float32) * 0.1
    free: list = []
    nxt = 0
    if not causal:
        free = list(range(N))
        nxt = N
    slots = np.empty((R, p), dtype=np.int64)
    for r in range(R):
        i = int(planted[r])
        while nxt <= i and nxt < N:
            free.append(nxt)
            nxt += 1
        for t in range(p):
            m = len(free)
            x = min(int(u[r, t] * m), m - 1)
            slots[r, t] = free[x]
            free[x] = free[m - 1]
            free.pop()
    qi = q_h[torch.from_numpy(planted)]                      # [R, d]
    direction = qi / qi.norm(dim=1, keepdim=True).clamp_min(1e-20)
    rows = (3.0 * math.sqrt(d)) * direction[:, None, :] + noise   # [R, p, d]
    k_h[torch.from_numpy(slots.reshape(-1))] = rows.reshape(R * p, d)
    return planted


def _plant_shift(q_h: torch.Tensor, k_h: torch.Tensor, gen: torch.Generator):
    """Every query i gets one key at j = (i + shift) mod N, shift drawn per head."""
    N, d = q_h.shape
    shift = int(torch.randint(0, N, (1,), generator=gen).item())
    noise = torch.randn((N, d), generator=gen, dtype=torch.float32) * 0.1
    direction = q_h / q_h.norm(dim=1, keepdim=True).clamp_min(1e-20)
    j = (torch.arange(N) + shift) % N
    k_h[j] = (3.0 * math.sqrt(d)) * direction + noise
    return np.arange(N, dtype=np.int64)


def make_inputs(w: Workload, seed: Optional[int] = None) -> Inputs:
    """Draw the tensors of a workload.  Values are drawn in fp32, keys planted, then rounded ONCE to
    the workload dtype; the oracle and the CUDA path both start from these rounded tensors."""
    seed = BASE_SEED + w.seed_offset if seed is None else seed
    gen = torch.Generator(device="cpu")
    gen.manual_seed(seed)
    shape = (w.B, w.H, w.N, w.d)
    q = torch.randn(shape, generator=gen, dtype=torch.float32) * w.qk_sigma
    k = torch.randn(shape, generator=gen, dtype=torch.float32) * w.qk_sigma
    v = torch.randn(shape, generator=gen, dtype=torch.float32)
    d_o = torch.randn(shape, generator=gen, dtype=torch.float32) if w.backward else None
    beta = gamma = delta = None
    if w.use_scale:
        beta = torch.rand(w.H, generator=gen, dtype=torch.float32) + 0.5
        gamma = torch.rand(w.H, generator=gen, dtype=torch.float32) + 0.5
        delta = torch.rand(w.H, generator=gen, dtype=torch.float32) + 0.5
    dt = _torch_dtype(w.dtype)
    # planting uses the query values the kernels will see (rounded to the workload dtype)
    q = q.to(dt)
    planted_rows = []
    for b in range(w.B):
        for h in range(w.H):
            if w.plant_mode == "subset" and w.plant > 0:
                planted_rows.append(_plant_subset(q[b, h].float(), k[b, h], w.plant, w.causal, gen))
            elif w.plant_mode == "shift":
                planted_rows.append(_plant_shift(q[b, h].float(), k[b, h], gen))
            else:
                planted_rows.append(np.empty(0, dtype=np.int64))
    k = k.to(dt)
    v = v.to(dt)
    if d_o is not None:
        d_o = d_o.to(dt)
    return Inputs(w, q.contiguous(), k.contiguous(), v.contiguous(), d_o, beta, gamma, delta, planted_rows,
                  1.0 / math.sqrt(w.d))


def seeded_d_o(w: Workload, seed_offset: int = 404) -> torch.Tensor:
    """A seeded N(0,1) output gradient for a workload that has none of its own (the forward-only long-context
    workload when the benchmark and its parity test run a backward pass on it), rounded once to the workload dtype."""
    gen = torch.Generator(device="cpu")
    gen.manual_seed(BASE_SEED + seed_offset)
    return torch.randn((w.B, w.H, w.N, w.d), generator=gen, dtype=torch.float32).to(_torch_dtype(w.dtype))


def sample_rows(inp: Inputs, bh: int, count: int, seed: int = 0) -> np.ndarray:
    """`count` distinct query rows of head index bh = b*H + h; where the head has planted rows, half
    of the sample is forced to be planted rows.  Always contains row 0 and row N-1."""
    w = inp.workload
    rng = np.random.default_rng(BASE_SEED * 7 + w.seed_offset * 1000 + bh * 17 + seed)
    count = min(count, w.N)
    chosen = {0, w.N - 1}
    pl = inp.planted_rows[bh]
    if pl.shape[0] > 0 and pl.shape[0] < w.N:
        take = min(count // 2, pl.shape[0])
        chosen.update(int(x) for x in rng.choice(pl, size=take, replace=False))
    while len(chosen) < count:
        chosen.update(int(x) for x in rng.integers(0, w.N, size=count - len(chosen)))
    return np.array(sorted(chosen)[:count] if len(chosen) > count else sorted(chosen), dtype=np.int64)
