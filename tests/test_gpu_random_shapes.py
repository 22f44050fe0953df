"""Seeded random shapes through every statistics entry point, against the oracle.

The hand-picked shapes of the other files target known edges (tile and stage boundaries, odd batch slices); this
file draws shapes the author did not choose: batch sizes, sequence lengths and widths (multiples of 8, so the
tensor-core path is taken whenever the shape allows it) from fixed lists with a fixed seed, Gaussian and
heavy-tailed inputs in turn.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2510_00236_b200 as pe
from paper_2510_00236_b200 import inputs
from parity_util import FROB_TOL, check_sign, rel_frob

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _cases(n, seed):
    rng = np.random.default_rng(seed)
    out = []
    while len(out) < n:
        B = int(rng.choice([1, 2, 3, 5, 8, 17, 40, 75, 130]))
        T = int(rng.choice([1, 7, 16, 31, 32, 33, 48, 64, 65, 100, 128, 129, 200, 257, 600]))
        d_in = int(rng.choice([8, 16, 72, 128, 136, 256, 264, 392, 520]))
        d_out = int(rng.choice([8, 24, 128, 136, 256, 264, 384, 520, 776]))
        if B * T * d_in * d_out <= 6e8:            # keeps the oracle at a fraction of a second per case
            out.append((B, T, d_in, d_out, len(out) % 2))
    return out


@pytest.fixture(autouse=True)
def _auto_path():
    prev = pe.pe_set_path(pe.PATH_AUTO)
    yield
    pe.pe_set_path(prev)


@pytest.mark.parametrize("B,T,d_in,d_out,heavy", _cases(28, 20251))
def test_every_entry_point_on_a_random_shape(B, T, d_in, d_out, heavy):
    gen = inputs.heavy_tailed_layer if heavy else inputs.gaussian_layer
    li = gen(B, T, d_in, d_out, seed=9000 + B * T + d_in, device=DEV)
    Xh, Yh = inputs.to_numpy_bits(li.X), inputs.to_numpy_bits(li.dY)
    st = oracle.linear_stats(Xh, Yh, small_rel=1e-3)
    tok = oracle.token_sqstats(Xh, Yh)
    norms = oracle.example_sqnorms(Xh, Yh)
    nan = lambda: torch.full((d_out, d_in), float("nan"), device=DEV)
    for phi in ("square", "sign", "identity"):
        for both in (True, False):
            mean, stat = (nan() if both else None), nan()
            pe.pe_linear_stats(li.X, li.dY, phi, mean, stat)
            torch.cuda.synchronize()
            if both:
                assert rel_frob(mean.cpu().numpy(), st.sum_g) <= FROB_TOL
            if phi == "sign":
                check_sign(stat.cpu().numpy(), st)
            else:
                assert rel_frob(stat.cpu().numpy(), st.sum_g2 if phi == "square" else st.sum_g) <= FROB_TOL
    outs = [nan() for _ in range(3)]
    pe.pe_linear_stats_all(li.X, li.dY, *outs)
    acc = [torch.zeros((d_out, d_in), device=DEV) for _ in range(2)]
    for lo, hi in ((0, B // 2), (B // 2, B)):
        pe.pe_linear_stats_accumulate(li.X[lo:hi].clone(), li.dY[lo:hi].clone(), "square", acc[0], acc[1])
    n = pe.pe_example_sqnorms(li.X, li.dY)
    t1, t2 = nan(), pe.pe_token_sqstats_staged(li.X, li.dY)
    pe.pe_token_sqstats(li.X, li.dY, t1)
    torch.cuda.synchronize()
    assert pe.pe_get_async_status(DEV) == (0, 0)
    assert rel_frob(outs[0].cpu().numpy(), st.sum_g) <= FROB_TOL and rel_frob(outs[1].cpu().numpy(), st.sum_g2) <= FROB_TOL
    check_sign(outs[2].cpu().numpy(), st)
    assert rel_frob(acc[0].cpu().numpy(), st.sum_g) <= FROB_TOL and rel_frob(acc[1].cpu().numpy(), st.sum_g2) <= FROB_TOL
    assert np.max(np.abs(n.cpu().numpy() - norms) / np.maximum(norms, 1e-300)) <= 2e-3
    assert rel_frob(t1.cpu().numpy(), tok) <= FROB_TOL and rel_frob(t2.cpu().numpy(), tok) <= FROB_TOL
