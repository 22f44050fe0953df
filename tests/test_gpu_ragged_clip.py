"""GPU parity of the packed-batch (ragged) statistics and of the norm-clipped sum against the oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_2510_00236_b200 as pe
from paper_2510_00236_b200 import inputs
from parity_util import FROB_TOL, SIGN_REL, rel_frob

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _packed(lens, d_in, d_out, seed):
    """Packed rows of a batch whose sequences have the given lengths, with `pad` unowned rows before and after."""
    g = torch.Generator(device="cpu").manual_seed(seed)
    pad = 3
    rows = int(sum(lens)) + 2 * pad
    X = torch.randn((rows, d_in), generator=g).to(torch.bfloat16)
    dY = (torch.randn((rows, d_out), generator=g) / 8).to(torch.bfloat16)
    offs = np.concatenate([[pad], pad + np.cumsum(lens)]).astype(np.int32)
    return X.to(DEV), dY.to(DEV), torch.from_numpy(offs).to(DEV), offs


def _entrywise(a, ref, scale, what):
    """Per-entry bound beside the Frobenius one: no entry may be off by more than 1e-3 of the reference's rms."""
    assert np.max(np.abs(a - ref)) <= 1e-3 * scale, what


LENS = [
    [40, 7, 128, 0, 300, 16, 1, 95],                 # tails of every kind, an empty sequence, multi-stage sequences
    [16, 32, 48, 64],                                # whole 16-token groups only: no tail stage at all
    [5] * 9,                                         # all shorter than one MMA step
    [700, 3],                                        # very uneven pair
    [0, 0, 9],                                       # leading empty sequences
    list(np.random.default_rng(5).integers(0, 200, 37)),
]


@pytest.mark.parametrize("case", range(len(LENS)))
@pytest.mark.parametrize("d_in,d_out", [(136, 264), (384, 256)])
def test_ragged_statistics_match_the_oracle(case, d_in, d_out):
    lens = [int(v) for v in LENS[case]]
    X, dY, offs_d, offs = _packed(lens, d_in, d_out, 40 + case)
    st = oracle.linear_stats_ragged(inputs.to_numpy_bits(X), inputs.to_numpy_bits(dY), offs, small_rel=SIGN_REL)
    rms2 = float(np.sqrt(np.mean(st.sum_g2 ** 2))) + 1e-30
    rms1 = float(np.sqrt(np.mean(st.sum_g ** 2))) + 1e-30
    for path in (pe.PATH_TENSOR, pe.PATH_SIMT):
        prev = pe.pe_set_path(path)
        try:
            for phi, both in (("square", True), ("sign", True), ("square", False), ("sign", False), ("identity", True)):
                mean = torch.full((d_out, d_in), float("nan"), device=DEV) if both else None
                stat = torch.full((d_out, d_in), float("nan"), device=DEV)
                pe.pe_linear_stats_ragged(X, dY, offs_d, phi, mean, stat)
                torch.cuda.synchronize()
                s = stat.cpu().numpy().astype(np.float64)
                if both:
                    m = mean.cpu().numpy().astype(np.float64)
                    assert rel_frob(m, st.sum_g) <= FROB_TOL, (path, phi)
                    _entrywise(m, st.sum_g, rms1, (path, phi, "mean"))
                if phi == "square":
                    assert rel_frob(s, st.sum_g2) <= FROB_TOL, (path, phi, both)
                    _entrywise(s, st.sum_g2, rms2, (path, phi, "square"))
                elif phi == "sign":
                    assert np.all(np.abs(s - st.sum_sign) <= 2.0 * st.n_small + 1e-9), (path, phi, both)
                else:
                    assert rel_frob(s, st.sum_g) <= FROB_TOL
            norms = pe.pe_example_sqnorms_ragged(X, dY, offs_d).cpu().numpy().astype(np.float64)
            np.testing.assert_allclose(norms, st.sq_norms, rtol=2e-3, atol=1e-6 * float(st.sq_norms.max() + 1e-30))
            assert pe.pe_last_path() == path
        finally:
            pe.pe_set_path(prev)
    assert pe.pe_get_async_status(DEV) == (0, 0)


def test_ragged_with_equal_lengths_equals_the_fixed_length_call():
    B, T, d_in, d_out = 12, 80, 200, 264
    li = inputs.gaussian_layer(B, T, d_in, d_out, seed=71, device=DEV)
    offs = torch.arange(B + 1, dtype=torch.int32, device=DEV) * T
    m0, s0 = pe.pe_linear_stats(li.X, li.dY, "square")
    m1, s1 = pe.pe_linear_stats_ragged(li.X.view(B * T, d_in), li.dY.view(B * T, d_out), offs, "square")
    torch.cuda.synchronize()
    assert rel_frob(m1.cpu().numpy(), m0.cpu().numpy()) <= 1e-5
    assert rel_frob(s1.cpu().numpy(), s0.cpu().numpy()) <= 1e-5


def test_ragged_argument_errors():
    X, dY, offs_d, _ = _packed([8, 8], 64, 64, 1)
    out = torch.empty((64, 64), device=DEV)
    with pytest.raises(pe.PestatsError) as e:        # workspace too small
        pe.pe_linear_stats_ragged(X, dY, offs_d, "square", None, out, workspace=torch.empty(256, dtype=torch.uint8, device=DEV))
    assert e.value.status == 9
    m, s = pe.pe_linear_stats_ragged(X, dY, offs_d[:1], "square")        # B = 0: zeros
    torch.cuda.synchronize()
    assert float(m.abs().max()) == 0.0 and float(s.abs().max()) == 0.0


@pytest.mark.parametrize("B,T,d_in,d_out", [(12, 80, 200, 264), (5, 200, 136, 264), (40, 33, 384, 256), (3, 1, 64, 72), (6, 50, 60, 36)])
def test_clipped_sum_matches_the_oracle(B, T, d_in, d_out):
    li = inputs.heterogeneous_layer(B, T, d_in, d_out, seed=900 + B, device=DEV)      # some sequences 5 x larger: mixed clipping
    Xh, dYh = inputs.to_numpy_bits(li.X), inputs.to_numpy_bits(li.dY)
    own = oracle.example_sqnorms(Xh, dYh)
    C = float(np.sqrt(np.median(own)))
    ref, coef = oracle.clipped_sum(Xh, dYh, C)
    assert 0 < int((coef < 1).sum()) < B                                  # both branches of the min are exercised
    out, norms = pe.pe_linear_clipped_sum(li.X, li.dY, C)
    torch.cuda.synchronize()
    o = out.cpu().numpy().astype(np.float64)
    assert rel_frob(o, ref) <= FROB_TOL
    assert np.max(np.abs(o - ref)) <= 1e-3 * float(np.sqrt(np.mean(ref ** 2)))
    np.testing.assert_allclose(norms.cpu().numpy(), own, rtol=2e-3)
    # given (model-wide) norms: four times larger squared norms halve every clipped coefficient
    big = torch.from_numpy((own * 4.0).astype(np.float32)).to(DEV)
    ref2, _ = oracle.clipped_sum(Xh, dYh, C, sq_norms=big.cpu().numpy().astype(np.float64))
    out2, _ = pe.pe_linear_clipped_sum(li.X, li.dY, C, sq_norms=big)
    torch.cuda.synchronize()
    assert rel_frob(out2.cpu().numpy(), ref2) <= FROB_TOL
    # limits: nothing clipped = the batch gradient; clip_norm = 0 = zeros
    out3, _ = pe.pe_linear_clipped_sum(li.X, li.dY, 1e30)
    mean, _ = pe.pe_linear_stats(li.X, li.dY, "square")
    torch.cuda.synchronize()
    assert rel_frob(out3.cpu().numpy(), mean.cpu().numpy()) <= 1e-5
    out4, _ = pe.pe_linear_clipped_sum(li.X, li.dY, 0.0)
    assert float(out4.abs().max()) == 0.0
    assert pe.pe_get_async_status(DEV) == (0, 0)
