"""Pins of the oracle's packed-batch (ragged) statistics and of its clipped sum against what the paper and the
mathematics fix: reductions to the fixed-length call, zero padding, exact brute force on tiny inputs, and the
limits of the clipping coefficient.  CPU only."""
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from paper_2510_00236_b200 import inputs


def _rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape).astype(np.float32)


def _bf16_bits(a):
    return inputs.to_numpy_bits(torch.from_numpy(np.asarray(a, np.float32)).to(torch.bfloat16))


# ----------------------------------------------------------------------------- packed (ragged) batches

def test_equal_lengths_reduce_to_the_fixed_length_statistics():
    """Section 2.3: with every sequence T tokens long the packed form is the [B, T, d] form."""
    B, T, d_in, d_out = 5, 7, 6, 4
    X, dY = _rand((B, T, d_in), 1), _rand((B, T, d_out), 2)
    ref = oracle.linear_stats(X, dY)
    rg = oracle.linear_stats_ragged(X.reshape(B * T, d_in), dY.reshape(B * T, d_out), np.arange(B + 1) * T)
    for a, b in ((rg.sum_g, ref.sum_g), (rg.sum_g2, ref.sum_g2), (rg.sum_sign, ref.sum_sign), (rg.max_abs, ref.max_abs)):
        assert np.array_equal(a, b)
    assert np.array_equal(rg.n_small, ref.n_small)
    np.testing.assert_allclose(rg.sq_norms, oracle.example_sqnorms(X, dY), rtol=1e-13)


@pytest.mark.parametrize("bf16", [False, True])
def test_ragged_equals_zero_padded_fixed_length(bf16):
    """A token whose activation row and cotangent row are zero adds nothing to G_b: packing the sequences
    and padding them with zero rows to a common length give the same statistics."""
    lens = [3, 0, 7, 1, 5]
    B, Tmax, d_in, d_out = len(lens), 8, 5, 3
    offs = np.concatenate([[0], np.cumsum(lens)])
    Xp, dYp = _rand((offs[-1], d_in), 3), _rand((offs[-1], d_out), 4)
    if bf16:
        Xp = torch.from_numpy(Xp).to(torch.bfloat16).float().numpy()
        dYp = torch.from_numpy(dYp).to(torch.bfloat16).float().numpy()
    Xf, dYf = np.zeros((B, Tmax, d_in), np.float32), np.zeros((B, Tmax, d_out), np.float32)
    for b, n in enumerate(lens):
        Xf[b, :n], dYf[b, :n] = Xp[offs[b]:offs[b + 1]], dYp[offs[b]:offs[b + 1]]
    conv = _bf16_bits if bf16 else (lambda a: a)
    rg = oracle.linear_stats_ragged(conv(Xp), conv(dYp), offs)
    ref = oracle.linear_stats(conv(Xf), conv(dYf))
    np.testing.assert_allclose(rg.sum_g, ref.sum_g, rtol=1e-14, atol=1e-15)
    np.testing.assert_allclose(rg.sum_g2, ref.sum_g2, rtol=1e-14, atol=1e-15)
    assert np.array_equal(rg.sum_sign, ref.sum_sign)
    assert rg.sq_norms[1] == 0.0 and rg.max_abs[1] == 0.0        # the empty sequence


def test_ragged_brute_force_in_exact_rationals():
    lens = [2, 4, 1]
    d_in, d_out = 3, 2
    offs = np.concatenate([[0], np.cumsum(lens)])
    X, dY = _rand((offs[-1], d_in), 5), _rand((offs[-1], d_out), 6)
    sg = [[Fraction(0)] * d_in for _ in range(d_out)]
    sg2 = [[Fraction(0)] * d_in for _ in range(d_out)]
    ss = [[0] * d_in for _ in range(d_out)]
    norms = []
    for b in range(len(lens)):
        nb = Fraction(0)
        for o in range(d_out):
            for i in range(d_in):
                g = sum((Fraction(float(dY[r, o])) * Fraction(float(X[r, i])) for r in range(offs[b], offs[b + 1])), Fraction(0))
                sg[o][i] += g
                sg2[o][i] += g * g
                ss[o][i] += (g > 0) - (g < 0)
                nb += g * g
        norms.append(float(nb))
    f = lambda m: np.array([[float(v) for v in r] for r in m])
    rg = oracle.linear_stats_ragged(X, dY, offs)
    np.testing.assert_allclose(rg.sum_g, f(sg), rtol=1e-13, atol=1e-14)
    np.testing.assert_allclose(rg.sum_g2, f(sg2), rtol=1e-13, atol=1e-14)
    assert np.array_equal(rg.sum_sign, np.array(ss, np.float64))
    np.testing.assert_allclose(rg.sq_norms, norms, rtol=1e-13)


def test_ragged_rows_outside_every_sequence_are_ignored_and_the_sum_is_the_batch_gradient_of_the_owned_rows():
    """offsets need not start at 0 or cover all rows; sum_b G_b is the plain weight-gradient GEMM over the
    rows that belong to some sequence."""
    d_in, d_out = 4, 6
    X, dY = _rand((20, d_in), 7), _rand((20, d_out), 8)
    offs = np.array([2, 5, 5, 11, 17])
    rg = oracle.linear_stats_ragged(X, dY, offs)
    ref = dY[2:17].astype(np.float64).T @ X[2:17].astype(np.float64)
    np.testing.assert_allclose(rg.sum_g, ref, rtol=1e-12, atol=1e-13)
    with pytest.raises(RuntimeError):
        oracle.linear_stats_ragged(X, dY, np.array([0, 5, 3]))       # decreasing offsets


# ----------------------------------------------------------------------------- clipped sum

def _per_example_grads(X, dY):
    return np.einsum("bto,bti->boi", dY.astype(np.float64), X.astype(np.float64))


def test_clipping_limits():
    """C -> infinity: nothing is clipped and the result is the batch gradient.  C -> 0: every example is
    clipped and result / C is the sum of unit-norm gradients."""
    B, T, d_in, d_out = 6, 5, 4, 3
    X, dY = _rand((B, T, d_in), 9), _rand((B, T, d_out), 10)
    G = _per_example_grads(X, dY)
    out, coef = oracle.clipped_sum(X, dY, 1e30)
    assert np.all(coef == 1.0)
    np.testing.assert_allclose(out, G.sum(0), rtol=1e-13, atol=1e-14)
    C = 1e-9
    out, coef = oracle.clipped_sum(X, dY, C)
    unit = sum(G[b] / np.linalg.norm(G[b]) for b in range(B))
    np.testing.assert_allclose(out / C, unit, rtol=1e-12, atol=1e-13)
    out0, coef0 = oracle.clipped_sum(X, dY, 0.0)
    assert np.all(out0 == 0.0) and np.all(coef0 == 0.0)


def test_clipped_terms_have_norm_at_most_C_and_small_examples_pass_unchanged():
    B, T, d_in, d_out = 8, 4, 5, 5
    X, dY = _rand((B, T, d_in), 11), _rand((B, T, d_out), 12)
    dY[:3] *= 0.01                                   # three examples well below the threshold
    G = _per_example_grads(X, dY)
    norms = np.sqrt((G ** 2).sum((1, 2)))
    C = float(np.median(norms))
    out, coef = oracle.clipped_sum(X, dY, C)
    np.testing.assert_allclose(coef, np.minimum(1.0, C / norms), rtol=1e-13)
    assert np.all(coef[:3] == 1.0) and np.any(coef < 1.0)
    assert np.all(coef * norms <= C * (1 + 1e-12))
    np.testing.assert_allclose(out, np.einsum("b,boi->oi", np.minimum(1.0, C / norms), G), rtol=1e-12, atol=1e-14)
    # one example: the result is G rescaled to norm min(||G||, C)
    out1, _ = oracle.clipped_sum(X[5:6], dY[5:6], C)
    np.testing.assert_allclose(np.linalg.norm(out1), min(norms[5], C), rtol=1e-13)


def test_clipping_by_given_norms_and_by_own_norms_agree_and_model_wide_norms_clip_harder():
    B, T, d_in, d_out = 5, 6, 4, 4
    X, dY = _rand((B, T, d_in), 13), _rand((B, T, d_out), 14)
    own = oracle.example_sqnorms(X, dY)
    C = float(np.sqrt(np.median(own)))
    a, ca = oracle.clipped_sum(X, dY, C)
    b, cb = oracle.clipped_sum(X, dY, C, sq_norms=own)
    np.testing.assert_allclose(a, b, rtol=1e-13)
    # norms that include other layers are larger, so every coefficient can only shrink
    c, cc = oracle.clipped_sum(X, dY, C, sq_norms=own * 4.0)
    assert np.all(cc <= ca + 1e-15) and np.any(cc < ca)
    G = _per_example_grads(X, dY)
    np.testing.assert_allclose(c, np.einsum("b,boi->oi", np.minimum(1.0, C / (2.0 * np.sqrt(own))), G), rtol=1e-12, atol=1e-14)


def test_clipped_sum_brute_force_bf16():
    B, T, d_in, d_out = 3, 3, 2, 2
    X, dY = _rand((B, T, d_in), 15), _rand((B, T, d_out), 16)
    Xb, dYb = _bf16_bits(X), _bf16_bits(dY)
    Xv = torch.from_numpy(X).to(torch.bfloat16).double().numpy()
    dYv = torch.from_numpy(dY).to(torch.bfloat16).double().numpy()
    C = 0.8
    ref = np.zeros((d_out, d_in))
    for b in range(B):
        G = np.zeros((d_out, d_in))
        for o in range(d_out):
            for i in range(d_in):
                for t in range(T):
                    G[o, i] += dYv[b, t, o] * Xv[b, t, i]
        nrm = np.sqrt((G * G).sum())
        ref += G * (C / nrm if nrm > C else 1.0)
    out, _ = oracle.clipped_sum(Xb, dYb, C)
    np.testing.assert_allclose(out, ref, rtol=1e-12, atol=1e-14)
