"""Convolution weights through the unfolded contraction (Appendix B.4): the summed per-example gradient must be
autograd's conv weight gradient, and the per-example statistics must match the oracle on the unfolded operands
and the per-example gradients autograd gives one image at a time."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle
import paper_2510_00236_b200 as pe
from paper_2510_00236_b200 import conv_unfold, inputs
from parity_util import FROB_TOL, SIGN_REL, check_sign, rel_frob

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("B,C,Fo,H,W,K,stride,padding,dilation", [
    (6, 16, 24, 12, 12, 3, 1, 1, 1),        # "same" convolution: T = 144, d_in = 144
    (5, 8, 40, 17, 13, 5, 2, 2, 1),         # strided, rectangular image: T = 63, d_in = 200
    (4, 8, 16, 14, 14, 3, 1, 0, 2),         # dilated, no padding
    (3, 3, 8, 10, 10, 3, 1, 1, 1),          # d_in = 27: not a multiple of 8, served by the SIMT kernel
])
def test_conv2d_weight_statistics_via_unfold(B, C, Fo, H, W, K, stride, padding, dilation):
    g = torch.Generator(device="cpu").manual_seed(100 * B + C)
    # values already representable in bf16, so autograd (fp32) and the library see the same numbers
    # (the autograd side runs in fp64, so that it is a reference rather than a second fp32 / tf32 computation)
    x = torch.randn((B, C, H, W), generator=g).to(torch.bfloat16).double().to(DEV)
    w = (torch.randn((Fo, C, K, K), generator=g) / (C * K * K) ** 0.5).double().to(DEV).requires_grad_(True)
    out = F.conv2d(x, w, stride=stride, padding=padding, dilation=dilation)
    gy = (torch.randn(out.shape, generator=g) / 8).to(torch.bfloat16).double().to(DEV)     # cotangent of sum_b f_b
    (gw_batch,) = torch.autograd.grad(out, w, gy, retain_graph=True)
    # per-example weight gradients, one image at a time (the "compute-intensive" route of Section 2.1)
    per_ex = []
    for b in range(B):
        ob = F.conv2d(x[b:b + 1], w, stride=stride, padding=padding, dilation=dilation)
        per_ex.append(torch.autograd.grad(ob, w, gy[b:b + 1])[0].double())
    per_ex = torch.stack(per_ex)

    mean, sq = conv_unfold.pe_conv2d_stats(x, gy, w.shape, "square", stride, padding, dilation)
    _, sg = conv_unfold.pe_conv2d_stats(x, gy, w.shape, "sign", stride, padding, dilation)
    torch.cuda.synchronize()
    assert pe.pe_last_path() == (pe.PATH_TENSOR if (C * K * K) % 8 == 0 and Fo % 8 == 0 else pe.PATH_SIMT)
    # sum_b G_b is the ordinary conv weight gradient
    assert rel_frob(mean.cpu().numpy(), gw_batch.cpu().numpy()) <= FROB_TOL
    # sum_b G_b^2 against autograd's per-example gradients ...
    assert rel_frob(sq.cpu().numpy(), (per_ex ** 2).sum(0).cpu().numpy()) <= FROB_TOL
    # ... and everything against the oracle on the unfolded operands
    X, dY = conv_unfold.conv2d_operands(x, gy, (K, K), stride, padding, dilation)
    st = oracle.linear_stats(inputs.to_numpy_bits(X), inputs.to_numpy_bits(dY), small_rel=SIGN_REL)
    flat = lambda t: t.reshape(Fo, -1).cpu().numpy().astype(np.float64)
    assert rel_frob(flat(mean), st.sum_g) <= FROB_TOL and rel_frob(flat(sq), st.sum_g2) <= FROB_TOL
    check_sign(flat(sg), st)
    # the oracle's own per-example picture agrees with autograd's: the unfold harness is what it claims to be
    assert rel_frob(st.sum_g2, flat((per_ex ** 2).sum(0))) <= 1e-10
    assert pe.pe_get_async_status(DEV) == (0, 0)
