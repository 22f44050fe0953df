"""Convolution layers through the same contraction (Appendix B.4, "For convolutions ..."): an image is
unfolded into one row per output position holding that position's receptive field, after which the layer is
the dense sequence-level layer of Section 2.3 with T = H_out * W_out "tokens" and d_in = C * K_h * K_w, and its
per-example weight gradient is G_b = dY_b^T X_b reshaped to [F, C, K_h, K_w].

Only the data layout happens here (torch's unfold and a transpose); the statistics are the library calls.
"""
from __future__ import annotations

import torch
import torch.nn.functional as F

from . import binding

__all__ = ["conv2d_operands", "pe_conv2d_stats"]


def conv2d_operands(x: torch.Tensor, grad_out: torch.Tensor, kernel_size, stride=1, padding=0, dilation=1):
    """x: [B, C, H, W] layer input, grad_out: [B, F, H_out, W_out] cotangent of the layer output.
    Returns (X [B, T, C*K_h*K_w], dY [B, T, F]) in bf16, T = H_out * W_out, ready for pe_linear_stats.
    The feature order of X is torch's unfold order (channel-major, then kernel row, then kernel column), i.e.
    the order of weight.view(F, -1)."""
    if x.dim() != 4 or grad_out.dim() != 4 or x.shape[0] != grad_out.shape[0]:
        raise ValueError("x must be [B, C, H, W] and grad_out [B, F, H_out, W_out]")
    cols = F.unfold(x.float(), kernel_size, dilation=dilation, padding=padding, stride=stride)      # [B, C*K*K, T]
    B, Fo = grad_out.shape[:2]
    T = cols.shape[2]
    if grad_out.shape[2] * grad_out.shape[3] != T:
        raise ValueError("grad_out's spatial size does not match the convolution's output size")
    X = cols.transpose(1, 2).contiguous().to(torch.bfloat16)
    dY = grad_out.reshape(B, Fo, T).transpose(1, 2).contiguous().to(torch.bfloat16)
    return X, dY


def pe_conv2d_stats(x, grad_out, weight_shape, phi, stride=1, padding=0, dilation=1):
    """sum_b G_b and sum_b phi(G_b) of a conv2d weight [F, C, K_h, K_w]; both returned in the weight's shape."""
    Fo, C, Kh, Kw = weight_shape
    X, dY = conv2d_operands(x, grad_out, (Kh, Kw), stride, padding, dilation)
    mean, stat = binding.pe_linear_stats(X, dY, phi)
    return mean.view(Fo, C, Kh, Kw), stat.view(Fo, C, Kh, Kw)
