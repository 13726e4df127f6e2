"""torch.autograd wrapper around the C-ABI calls: argument marshalling only.

    o = entmax_attention(q, k, v, beta, gamma, delta, alpha=1.5, causal=True)

is differentiable with respect to q, k, v and the ASEntmax parameters beta, gamma, delta (Eq. "asentmax":
the temperature c_i = delta_h + beta_h (log n_i)^gamma_h is learnable), or with respect to a per-query
scale table ``c_rows`` [B,H,N] when the caller evaluates the paper's content-dependent beta, gamma itself
(Sec. 4.1) and wants dL/dc_i back.  Every number comes from entmax_attn_fwd_ex / entmax_attn_bwd_ex.

``keep_supports=True`` keeps a compact copy of every row's support (260 bytes per query row, made by
entmax_attn_save_supports) until the backward pass, which then skips its score sweep: no second Q K^T.
"""
from __future__ import annotations

from typing import Optional

import torch

from . import binding


class _EntmaxAttention(torch.autograd.Function):
    @staticmethod
    def forward(ctx, q, k, v, beta, gamma, delta, c_rows, alibi_slopes, alpha, causal, sm_scale, keep_supports):
        params = binding.make_params(q, alpha, causal, sm_scale, 0)
        ws = binding.alloc_workspace(params, False, q.device) if keep_supports and q.dtype == torch.bfloat16 else None
        keep_supports = ws is not None
        det = lambda t: None if t is None else t.detach()
        o, tau = binding.entmax_attn_fwd_ex(q.detach(), k.detach(), v.detach(), alpha, causal, det(beta), det(gamma),
                                            det(delta), c_rows=det(c_rows), alibi_slopes=det(alibi_slopes),
                                            sm_scale=sm_scale, workspace=ws)
        saved = binding.entmax_attn_save_supports(q, alpha, causal, ws, sm_scale=sm_scale) if keep_supports else None
        ctx.save_for_backward(q, k, v, beta, gamma, delta, c_rows, alibi_slopes, tau)
        ctx.alpha, ctx.causal, ctx.sm_scale, ctx.saved_supports = alpha, causal, sm_scale, saved
        ctx.mark_non_differentiable(tau)
        return o, tau

    @staticmethod
    def backward(ctx, d_o, _d_tau):
        q, k, v, beta, gamma, delta, c_rows, alibi_slopes, tau = ctx.saved_tensors
        det = lambda t: None if t is None else t.detach()
        want_params = beta is not None and any(ctx.needs_input_grad[3:6])
        want_rows = c_rows is not None and ctx.needs_input_grad[6]
        dq, dk, dv, dc, grads = binding.entmax_attn_bwd_ex(
            q.detach(), k.detach(), v.detach(), tau, d_o.contiguous(), ctx.alpha, ctx.causal, det(beta), det(gamma),
            det(delta), c_rows=det(c_rows), alibi_slopes=det(alibi_slopes), saved_supports=ctx.saved_supports,
            want_scale_rows=want_rows, want_param_grads=want_params, sm_scale=ctx.sm_scale)
        ctx.saved_supports = None
        db, dg, dd = grads if grads is not None else (None, None, None)
        return dq, dk, dv, db, dg, dd, (dc if want_rows else None), None, None, None, None, None


def entmax_attention(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, beta: Optional[torch.Tensor] = None,
                     gamma: Optional[torch.Tensor] = None, delta: Optional[torch.Tensor] = None, *,
                     c_rows: Optional[torch.Tensor] = None, alibi_slopes: Optional[torch.Tensor] = None,
                     alpha: float = 1.5, causal: bool = True, sm_scale: float = 0.0, keep_supports: bool = False,
                     return_tau: bool = False):
    """alpha-entmax attention of q, k, v [B,H,N,d] (CUDA tensors, bf16 or fp32, one layout).

    beta, gamma, delta: float32 [H] (all three or none); c_rows: float32 [B,H,N] instead of them;
    alibi_slopes: float32 [H] (causal bf16 problems and fp32 problems).  Returns O, or (O, tau)."""
    o, tau = _EntmaxAttention.apply(q, k, v, beta, gamma, delta, c_rows, alibi_slopes, float(alpha), bool(causal),
                                    float(sm_scale), bool(keep_supports))
    return (o, tau) if return_tau else o
