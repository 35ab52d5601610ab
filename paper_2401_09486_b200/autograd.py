"""torch.autograd glue for the masked attention: argument marshalling and tensor bookkeeping only.

Every arithmetic step runs in the CUDA library (loma_masked_attn_fwd / loma_masked_attn_bwd through
the C ABI); this module allocates the outputs, keeps what the backward needs, and hands both calls
the same layout parameters.  There is no fallback: without the library the calls raise.
"""

from __future__ import annotations

import torch

from . import binding as L


class _MaskedAttention(torch.autograd.Function):
    @staticmethod
    def forward(ctx, q, k, v, n_chunks, c, t, tail_read, flags, softmax_scale):
        if not (q.is_cuda and k.is_cuda and v.is_cuda):
            raise RuntimeError("loma_masked_attention needs CUDA tensors (there is no CPU path)")
        q, k, v = q.contiguous(), k.contiguous(), v.contiguous()
        B, H, S, D = q.shape
        o = torch.empty_like(q)
        lse = torch.empty((B, H, S), dtype=torch.float32, device=q.device)
        L.loma_masked_attn_fwd(q, k, v, o, lse, n_chunks, c, t, tail_read, flags, softmax_scale)
        ctx.save_for_backward(q, k, v, o, lse)
        ctx.layout = (n_chunks, c, t, tail_read, flags, softmax_scale)
        return o

    @staticmethod
    def backward(ctx, d_o):
        q, k, v, o, lse = ctx.saved_tensors
        n_chunks, c, t, tail_read, flags, softmax_scale = ctx.layout
        B, H, S, D = q.shape
        d_o = d_o.contiguous()
        dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
        nbytes = L.loma_masked_attn_bwd_workspace_bytes(B, H, D, n_chunks, c, t, tail_read, flags)
        ws = torch.empty(max(256, nbytes), dtype=torch.uint8, device=q.device)
        L.loma_masked_attn_bwd(q, k, v, o, d_o, lse, dq, dk, dv, n_chunks, c, t, tail_read, flags, ws, softmax_scale)
        return dq, dk, dv, None, None, None, None, None, None


def loma_masked_attention(q, k, v, n_chunks: int, c: int, t: int, tail_read: int = 0, flags: int = 0,
                          softmax_scale: float = 0.0) -> torch.Tensor:
    """Zone-masked attention over the laid-out sequence (Eq. 1-3, Eq. 7) as a differentiable torch op.

    q, k, v: [B, H, S, D] CUDA tensors of one dtype (fp32 or bf16), S = n_chunks * chunk length + tail_read.
    Returns O [B, H, S, D]; gradients flow to q, k and v through the library's backward kernels.
    """
    return _MaskedAttention.apply(q, k, v, n_chunks, c, t, tail_read, flags, softmax_scale)


class _Rope(torch.autograd.Function):
    @staticmethod
    def forward(ctx, q, k, n_chunks, c, t, tail_read, flags, theta_base, position_type):
        q, k = q.contiguous().clone(), k.contiguous().clone()
        L.loma_rope_apply(q, k, n_chunks, c, t, tail_read, flags, theta_base, position_type)
        ctx.layout = (n_chunks, c, t, tail_read, flags, theta_base, position_type)
        return q, k

    @staticmethod
    def backward(ctx, dq, dk):
        n_chunks, c, t, tail_read, flags, theta_base, position_type = ctx.layout
        dq, dk = dq.contiguous().clone(), dk.contiguous().clone()
        L.loma_rope_apply(dq, dk, n_chunks, c, t, tail_read, flags, theta_base, position_type | L.LOMA_ROPE_INVERSE)
        return dq, dk, None, None, None, None, None, None, None


def loma_rope(q, k, n_chunks: int, c: int, t: int, tail_read: int = 0, flags: int = 0, theta_base: float = 0.0,
              position_type: int = 0):
    """Rotary embedding of q and k at the layout's position ids as a differentiable torch op (out of place;
    the gradient is the rotation by the opposite angle, run by the same kernel)."""
    return _Rope.apply(q, k, n_chunks, c, t, tail_read, flags, theta_base, position_type)
