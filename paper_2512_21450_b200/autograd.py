"""torch.autograd front end of the fused head.

The library computes the loss and both gradients in one call, so the autograd Function does all
the work in `forward` and only scales the stored gradients by the incoming gradient in
`backward`.  Marshalling only: the arithmetic is the C ABI's.
"""
from __future__ import annotations

import torch

from .binding import default_context


class _FusedHeadLoss(torch.autograd.Function):
    @staticmethod
    def forward(ctx, H, W, tokens, old_logp, ref_logp, adv, mask, eps_low, eps_high, beta, ent_coef, token_weight,
                agg_mode, sequence_level, seq_offsets):
        lib = default_context(W.device.index or 0)
        out = lib.rl_policy_loss_fwd_bwd(H.detach(), W.detach(), tokens, old_logp, ref_logp, adv, mask, eps_low,
                                         eps_high, beta, ent_coef=ent_coef, token_weight=token_weight,
                                         agg_mode=agg_mode, sequence_level=sequence_level, seq_offsets=seq_offsets)
        ctx.save_for_backward(out["dH"], out["dW"])
        ctx.mark_non_differentiable(out["logp"], out["entropy"], out["metrics"])
        return out["loss"].reshape(()).clone(), out["logp"], out["entropy"], out["metrics"]

    @staticmethod
    def backward(ctx, g_loss, *_):
        dH, dW = ctx.saved_tensors
        gH = (dH.float() * g_loss).to(dH.dtype) if ctx.needs_input_grad[0] else None
        gW = (dW * g_loss).to(torch.bfloat16) if ctx.needs_input_grad[1] else None
        return (gH, gW) + (None,) * 13


def fused_grpo_head_loss(H, W, tokens, old_logp, ref_logp, adv, mask, eps_low=0.2, eps_high=0.2, beta=0.04,
                         ent_coef=0.0, token_weight=None, agg_mode=0, sequence_level=False, seq_offsets=None):
    """Loss of Eq. 6 (negated) as a differentiable scalar in H [T,d] bf16 and W [V,d] bf16.

    Returns (loss, logp[T], entropy[T], metrics[8]); gradients reach H (bf16) and W (the fp32 dW
    rounded to W's dtype) through autograd.
    """
    return _FusedHeadLoss.apply(H, W, tokens, old_logp, ref_logp, adv, mask, eps_low, eps_high, beta, ent_coef,
                                token_weight, agg_mode, sequence_level, seq_offsets)
