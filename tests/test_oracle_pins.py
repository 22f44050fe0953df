"""Pins for the CPU oracle: each test ties one of its functions to something fixed by the paper
or by the mathematics, not to the oracle itself.  A dropped term, a wrong sign or index or a
transposed operand in the oracle must fail at least one of these."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from paper_2510_00236_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _bf16_bits(a: np.ndarray) -> np.ndarray:
    return inputs.to_numpy_bits(torch.from_numpy(np.asarray(a, np.float32)).to(torch.bfloat16))


def _bits_to_f64(bits: np.ndarray) -> np.ndarray:
    t = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16)
    return t.to(torch.float64).numpy()


def _rand(shape, seed, dtype=np.float32):
    return np.random.default_rng(seed).standard_normal(shape).astype(dtype)


# ----------------------------------------------------------------------------- input widening

def test_bf16_widening_matches_torch_for_every_bit_pattern():
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    ref = _bits_to_f64(bits)
    finite = np.isfinite(ref)
    # T=1, d_out=1, dY=1: sum_g[0, i] is X[i] widened.
    X = bits[finite].reshape(1, 1, -1)
    one = _bf16_bits(np.ones((1, 1, 1)))
    st = oracle.linear_stats(X, one)
    assert np.array_equal(st.sum_g[0], ref[finite])


# ----------------------------------------------------------------------------- paper's example

def test_appendix_a_worked_example():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "appendix_a_worked_example.txt"))
            if l.strip() and not l.startswith("#")]
    B, T, d_in, d_out = map(int, rows[0][:4])
    sum_g, mean_sq, sum_sign = map(float, rows[0][4:])
    X = np.ones((B, T, d_in), np.float32)
    dY = np.ones((B, T, d_out), np.float32)
    st = oracle.linear_stats(X, dY)
    assert np.all(st.sum_g == sum_g)
    assert np.all(st.sum_g2 / B == mean_sq)
    assert np.all(st.sum_sign == sum_sign)
    assert np.all(oracle.token_sqstats(X, dY) == B * T)


# ----------------------------------------------------------------------------- identities

@pytest.mark.parametrize("B,T,d_in,d_out", [(5, 7, 6, 9), (3, 16, 33, 10), (1, 4, 8, 8)])
def test_sum_of_per_example_gradients_is_the_batch_gradient(B, T, d_in, d_out):
    X, dY = _rand((B, T, d_in), 1), _rand((B, T, d_out), 2)
    st = oracle.linear_stats(X, dY)
    ref = dY.reshape(B * T, d_out).astype(np.float64).T @ X.reshape(B * T, d_in).astype(np.float64)
    np.testing.assert_allclose(st.sum_g, ref, rtol=1e-12, atol=1e-12)


def test_single_example_reduces_to_phi_of_batch_gradient():
    T, d_in, d_out = 12, 7, 5
    X, dY = _rand((1, T, d_in), 3), _rand((1, T, d_out), 4)
    G = dY[0].astype(np.float64).T @ X[0].astype(np.float64)
    st = oracle.linear_stats(X, dY)
    np.testing.assert_allclose(st.sum_g, G, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(st.sum_g2, G * G, rtol=1e-12, atol=1e-13)
    assert np.array_equal(st.sum_sign, np.sign(G))
    assert st.max_abs[0] == pytest.approx(np.abs(G).max(), rel=1e-12)


def test_rank_one_case_factorises():
    """T = 1: gradients are rank one, so square and sign factor through the operands
    (Section 2.3, dense layers in standard MLPs)."""
    B, d_in, d_out = 9, 6, 11
    X, dY = _rand((B, 1, d_in), 5), _rand((B, 1, d_out), 6)
    st = oracle.linear_stats(X, dY)
    x, y = X[:, 0].astype(np.float64), dY[:, 0].astype(np.float64)
    np.testing.assert_allclose(st.sum_g2, (y * y).T @ (x * x), rtol=1e-12)
    assert np.array_equal(st.sum_sign, np.sign(y).T @ np.sign(x))
    np.testing.assert_allclose(oracle.token_sqstats(X, dY), st.sum_g2, rtol=1e-12)


def _brute(X, dY):
    """Five nested loops in exact rational arithmetic."""
    B, T, d_in = X.shape
    d_out = dY.shape[2]
    sg = [[Fraction(0)] * d_in for _ in range(d_out)]
    sg2 = [[Fraction(0)] * d_in for _ in range(d_out)]
    ss = [[0] * d_in for _ in range(d_out)]
    tok = [[Fraction(0)] * d_in for _ in range(d_out)]
    for b in range(B):
        for o in range(d_out):
            for i in range(d_in):
                g = Fraction(0)
                for t in range(T):
                    y, x = Fraction(float(dY[b, t, o])), Fraction(float(X[b, t, i]))
                    g += y * x
                    tok[o][i] += y * y * x * x
                sg[o][i] += g
                sg2[o][i] += g * g
                ss[o][i] += (g > 0) - (g < 0)
    f = lambda m: np.array([[float(v) for v in r] for r in m])
    return f(sg), f(sg2), f(ss), f(tok)


@pytest.mark.parametrize("B,T,d_in,d_out,bf16", [(3, 4, 5, 2, False), (2, 3, 4, 5, True), (4, 1, 3, 3, False)])
def test_brute_force_tiny(B, T, d_in, d_out, bf16):
    X, dY = _rand((B, T, d_in), 7), _rand((B, T, d_out), 8)
    if bf16:
        Xb, dYb = _bf16_bits(X), _bf16_bits(dY)
        Xv, dYv = _bits_to_f64(Xb), _bits_to_f64(dYb)
    else:
        Xb, dYb, Xv, dYv = X, dY, X, dY
    sg, sg2, ss, tok = _brute(Xv, dYv)
    st = oracle.linear_stats(Xb, dYb)
    np.testing.assert_allclose(st.sum_g, sg, rtol=1e-13, atol=1e-14)
    np.testing.assert_allclose(st.sum_g2, sg2, rtol=1e-13, atol=1e-14)
    assert np.array_equal(st.sum_sign, ss)
    np.testing.assert_allclose(oracle.token_sqstats(Xb, dYb), tok, rtol=1e-13)


def test_sign_of_exact_zero_is_zero_and_padding_tokens_do_not_count():
    B, T, d_in, d_out = 4, 3, 3, 2
    X, dY = _rand((B, T, d_in), 9), _rand((B, T, d_out), 10)
    X[:, :, 1] = 0.0          # an input feature that is always zero -> G_b[:, 1] == 0 exactly
    st = oracle.linear_stats(X, dY)
    assert np.all(st.sum_sign[:, 1] == 0)
    assert np.all(st.sum_g2[:, 1] == 0)
    # zero rows (padding) change nothing
    Xp = np.concatenate([X, np.zeros((B, 2, d_in), np.float32)], 1)
    dYp = np.concatenate([dY, _rand((B, 2, d_out), 11)], 1)
    stp = oracle.linear_stats(Xp, dYp)
    np.testing.assert_allclose(stp.sum_g2, st.sum_g2, rtol=1e-13)
    assert np.array_equal(stp.sum_sign, st.sum_sign)


def test_invariants():
    B, T, d_in, d_out = 12, 9, 10, 7
    X, dY = _rand((B, T, d_in), 12), _rand((B, T, d_out), 13)
    st = oracle.linear_stats(X, dY)
    tok = oracle.token_sqstats(X, dY)
    # Cauchy-Schwarz over examples: nu_adam <= nu_micro (Eq. (3))
    assert np.all(st.sum_g ** 2 <= B * st.sum_g2 * (1 + 1e-12))
    # Cauchy-Schwarz over tokens: G_b^2 <= T * sum_t (dy x)^2
    assert np.all(st.sum_g2 <= T * tok * (1 + 1e-12))
    assert np.all(np.abs(st.sum_sign) <= B)
    assert np.all((st.sum_sign.astype(np.int64) - B) % 2 == 0)    # no exact zeros here
    # scaling: dY -> c dY scales sum_g by c, sum_g2 by c^2, token stat by c^2, sign unchanged
    st2 = oracle.linear_stats(X, (2.0 * dY).astype(np.float32))
    np.testing.assert_allclose(st2.sum_g, 2 * st.sum_g, rtol=1e-12)
    np.testing.assert_allclose(st2.sum_g2, 4 * st.sum_g2, rtol=1e-12)
    assert np.array_equal(st2.sum_sign, st.sum_sign)
    # negating X flips signs
    st3 = oracle.linear_stats(-X, dY)
    assert np.array_equal(st3.sum_sign, -st.sum_sign)
    np.testing.assert_allclose(st3.sum_g2, st.sum_g2, rtol=1e-12)


def test_permuting_examples_or_tokens_changes_nothing_but_mixing_them_does():
    B, T, d_in, d_out = 5, 6, 4, 3
    X, dY = _rand((B, T, d_in), 14), _rand((B, T, d_out), 15)
    st = oracle.linear_stats(X, dY)
    pb = np.random.default_rng(0).permutation(B)
    pt = np.random.default_rng(1).permutation(T)
    st_b = oracle.linear_stats(X[pb], dY[pb])
    st_t = oracle.linear_stats(X[:, pt], dY[:, pt])
    np.testing.assert_allclose(st_b.sum_g2, st.sum_g2, rtol=1e-12)
    np.testing.assert_allclose(st_t.sum_g2, st.sum_g2, rtol=1e-12)
    # regrouping the same B*T rows into different sequences keeps the batch gradient and the
    # per-token statistic but changes the per-example square statistic
    Xr, dYr = X.reshape(B * T, d_in), dY.reshape(B * T, d_out)
    st_r = oracle.linear_stats(Xr.reshape(T, B, d_in), dYr.reshape(T, B, d_out))
    np.testing.assert_allclose(st_r.sum_g, st.sum_g, rtol=1e-11, atol=1e-12)
    assert not np.allclose(st_r.sum_g2, st.sum_g2, rtol=1e-3)
    np.testing.assert_allclose(oracle.token_sqstats(Xr.reshape(T, B, d_in), dYr.reshape(T, B, d_out)),
                               oracle.token_sqstats(X, dY), rtol=1e-12)


def test_max_abs_and_small_counts():
    B, T, d_in, d_out = 6, 5, 4, 3
    X, dY = _rand((B, T, d_in), 16), _rand((B, T, d_out), 17)
    rel = 0.2
    st = oracle.linear_stats(X, dY, small_rel=rel)
    G = np.einsum("bto,bti->boi", dY.astype(np.float64), X.astype(np.float64))
    mx = np.abs(G).reshape(B, -1).max(1)
    np.testing.assert_allclose(st.max_abs, mx, rtol=1e-12)
    ref = (np.abs(G) <= rel * mx[:, None, None] * (1 + 1e-9)).sum(0)
    ref_lo = (np.abs(G) <= rel * mx[:, None, None] * (1 - 1e-9)).sum(0)
    assert np.all(st.n_small <= ref) and np.all(st.n_small >= ref_lo)
    assert st.n_small.sum() > 0


# ----------------------------------------------------------------------------- statistics

def test_second_moment_of_iid_gaussian_inputs():
    """Eq. (5) with mu = 0: per-example gradients of i.i.d. N(0,1) operands have variance T, so
    E[sum_g2 / B] = T; the per-token statistic has E[S'/(B T)] = 1; E[sum_sign] = 0."""
    B, T, d = 64, 8, 48
    X, dY = _rand((B, T, d), 18), _rand((B, T, d), 19)
    st = oracle.linear_stats(X, dY)
    n = d * d
    # var of G^2 for a sum of T products of normals is T^2*(2 + 6/T); standard error over B*n samples
    se = T * math.sqrt((2 + 6 / T) / (B * n))
    assert abs((st.sum_g2 / B).mean() - T) < 6 * se
    tok = oracle.token_sqstats(X, dY)
    assert abs(tok.mean() / (B * T) - 1.0) < 6 * math.sqrt(8.0 / (B * T * n))
    assert abs(st.sum_sign.mean()) < 6 * math.sqrt(B / n) + 1e-9


def test_mean_sign_with_planted_mean_follows_2p_minus_1():
    """Appendix C.1: sign(N(r,1)) has mean 2p-1 with p = Phi(r).  T = 1, X = 1 makes
    G_b = dY_b ~ N(r, 1) exactly."""
    B, d_out, r = 4096, 8, 0.5
    dY = (_rand((B, 1, d_out), 20) + r).astype(np.float32)
    X = np.ones((B, 1, 1), np.float32)
    st = oracle.linear_stats(X, dY)
    p = 0.5 * (1 + math.erf(r / math.sqrt(2)))
    se = 2 * math.sqrt(p * (1 - p) / (B * d_out))
    assert abs(st.sum_sign.mean() / B - (2 * p - 1)) < 5 * se


def test_example_norms_equal_the_gram_matrix_contraction_and_close_the_sum_of_squares():
    """Per-example squared norms against three things the mathematics fixes: the "ghost" identity
    ||dY_b^T X_b||_F^2 = sum_{t,t'} (X_b X_b^T)[t,t'] (dY_b dY_b^T)[t,t'] (Section 2.3's remark on norms from
    Gram matrices; numpy's matmul, a different contraction order), the rank-one closed form ||x||^2 ||dy||^2 at
    T = 1, and sum_b N_b = the sum of all entries of sum_b G_b^2."""
    rng = np.random.default_rng(41)
    B, T, d_in, d_out = 5, 7, 9, 6
    X = rng.standard_normal((B, T, d_in)).astype(np.float32)
    dY = rng.standard_normal((B, T, d_out)).astype(np.float32)
    n = oracle.example_sqnorms(X, dY)
    Xd, Yd = X.astype(np.float64), dY.astype(np.float64)
    ghost = np.array([np.sum((Xd[b] @ Xd[b].T) * (Yd[b] @ Yd[b].T)) for b in range(B)])
    np.testing.assert_allclose(n, ghost, rtol=1e-12)
    np.testing.assert_allclose(n.sum(), oracle.linear_stats(X, dY).sum_g2.sum(), rtol=1e-12)
    n1 = oracle.example_sqnorms(X[:, :1], dY[:, :1])
    np.testing.assert_allclose(n1, (Xd[:, 0] ** 2).sum(1) * (Yd[:, 0] ** 2).sum(1), rtol=1e-12)
    # bf16 bit patterns widen as everywhere else; scaling one example's cotangents by 3 scales its norm by 9
    Xb = inputs.to_numpy_bits(torch.tensor(X).to(torch.bfloat16))
    Yb = inputs.to_numpy_bits(torch.tensor(dY).to(torch.bfloat16))
    nb = oracle.example_sqnorms(Xb, Yb)
    Y3 = torch.tensor(dY).to(torch.bfloat16)
    Y3[2] *= 2                                                    # exact in bf16
    n3 = oracle.example_sqnorms(Xb, inputs.to_numpy_bits(Y3))
    np.testing.assert_allclose(n3[2], 4 * nb[2], rtol=1e-12)
    np.testing.assert_array_equal(np.delete(n3, 2), np.delete(nb, 2))


# ----------------------------------------------------------------------------- optimizer steps

def test_microadam_with_one_example_is_adam():
    """With B = 1 nu_micro = nu_adam (Eq. (3)), so MicroAdam is Adam; torch's Adam is the library
    cross-check (eps outside the square root, no weight decay)."""
    n, steps = 37, 4
    lr, b1, b2, eps = 1e-2, 0.9, 0.95, 1e-8
    rng = np.random.default_rng(21)
    theta0 = rng.standard_normal(n)
    p = torch.nn.Parameter(torch.tensor(theta0, dtype=torch.float64))
    opt = torch.optim.Adam([p], lr=lr, betas=(b1, b2), eps=eps)
    th, m, v = theta0.copy(), np.zeros(n), np.zeros(n)
    for t in range(1, steps + 1):
        g = rng.standard_normal(n)
        p.grad = torch.tensor(g, dtype=torch.float64)
        opt.step()
        th, m, v = oracle.microadam_step(th, m, v, g, g * g, 1, lr=lr, beta1=b1, beta2=b2, eps=eps, step=t)
        np.testing.assert_allclose(th, p.detach().numpy(), rtol=1e-12, atol=1e-14)


def test_microadam_hand_computed_step():
    # B = 2, two parameters.  sum_g = (3, -1), sum_g2 = (5, 1)  (e.g. g = {1,2} and {-1,0}).
    th, m, v = oracle.microadam_step([1.0, 2.0], [0.0, 0.0], [0.0, 0.0], [3.0, -1.0], [5.0, 1.0], 2,
                                     lr=0.1, beta1=0.9, beta2=0.99, eps=0.0, step=1)
    # mu = (1.5, -0.5); nu = (2.5, 0.5); m = 0.1 mu; v = 0.01 nu; mh = mu; vh = nu; u = mu/sqrt(nu)
    np.testing.assert_allclose(m, [0.15, -0.05], rtol=1e-14)
    np.testing.assert_allclose(v, [0.025, 0.005], rtol=1e-14)
    np.testing.assert_allclose(th, [1.0 - 0.1 * 1.5 / math.sqrt(2.5), 2.0 + 0.1 * 0.5 / math.sqrt(0.5)], rtol=1e-14)


def test_microadam_first_step_closed_form_and_bound():
    n, B = 50, 8
    rng = np.random.default_rng(22)
    G = rng.standard_normal((B, n))
    sg, sg2 = G.sum(0), (G * G).sum(0)
    th0 = rng.standard_normal(n)
    for inside in (False, True):
        eps = 1e-3
        th, m, v = oracle.microadam_step(th0, np.zeros(n), np.zeros(n), sg, sg2, B, lr=1.0, beta1=0.9,
                                         beta2=0.999, eps=eps, eps_inside_sqrt=inside, step=1)
        mu, nu = sg / B, sg2 / B
        u = mu / np.sqrt(eps + nu) if inside else mu / (np.sqrt(nu) + eps)
        np.testing.assert_allclose(th0 - th, u, rtol=1e-10)
        assert np.all(np.abs(th0 - th) <= 1.0)          # |mean| <= sqrt(mean of squares)
    # grad_scale: G -> s G is the same as passing s
    s = 3.0
    a = oracle.microadam_step(th0, np.zeros(n), np.zeros(n), sg, sg2, B, grad_scale=s, lr=0.1, beta1=0.9,
                              beta2=0.99, eps=1e-8, step=1)
    b = oracle.microadam_step(th0, np.zeros(n), np.zeros(n), s * sg, s * s * sg2, B, lr=0.1, beta1=0.9,
                              beta2=0.99, eps=1e-8, step=1)
    for x, y in zip(a, b):
        np.testing.assert_allclose(x, y, rtol=1e-12)
    # weight decay is independent of the learning rate
    th_wd, _, _ = oracle.microadam_step(th0, np.zeros(n), np.zeros(n), sg, sg2, B, lr=0.0, beta1=0.9,
                                        beta2=0.99, eps=1e-8, weight_decay=0.25, step=1)
    np.testing.assert_allclose(th_wd, 0.75 * th0, rtol=1e-14)


def test_microadam_bias_correction_uses_step_index():
    n, B = 5, 4
    sg, sg2 = np.full(n, 2.0), np.full(n, 4.0)
    m0, v0 = np.full(n, 0.3), np.full(n, 0.2)
    t, b1, b2 = 3, 0.9, 0.99
    th, m, v = oracle.microadam_step(np.zeros(n), m0, v0, sg, sg2, B, lr=1.0, beta1=b1, beta2=b2, eps=0.0, step=t)
    m_ref = b1 * 0.3 + (1 - b1) * 0.5
    v_ref = b2 * 0.2 + (1 - b2) * 1.0
    u = (m_ref / (1 - b1 ** t)) / math.sqrt(v_ref / (1 - b2 ** t))
    np.testing.assert_allclose(m, m_ref, rtol=1e-14)
    np.testing.assert_allclose(v, v_ref, rtol=1e-14)
    np.testing.assert_allclose(th, -u, rtol=1e-13)


def test_adam_family_original_variant_is_adam_on_the_mean_gradient():
    """Algorithm 1, "Original": nu = mu^2 at any batch size; torch's Adam fed the average gradient is the library check."""
    n, B, steps = 23, 5, 3
    lr, b1, b2, eps = 3e-3, 0.9, 0.99, 1e-8
    rng = np.random.default_rng(31)
    theta0 = rng.standard_normal(n)
    p = torch.nn.Parameter(torch.tensor(theta0, dtype=torch.float64))
    opt = torch.optim.Adam([p], lr=lr, betas=(b1, b2), eps=eps)
    th, m, v = theta0.copy(), np.zeros(n), np.zeros(n)
    for t in range(1, steps + 1):
        g = rng.standard_normal((B, n))
        p.grad = torch.tensor(g.mean(0), dtype=torch.float64)
        opt.step()
        th, m, v = oracle.adam_family_step(th, m, v, g.sum(0), (g * g).sum(0), B, "adam", lr=lr, beta1=b1, beta2=b2, eps=eps, step=t)
        np.testing.assert_allclose(th, p.detach().numpy(), rtol=1e-12, atol=1e-14)


def test_adam_family_preconditioners_are_the_textbook_unbiased_estimators():
    """Eq. (6): sigma2_hat is the sample variance with Bessel's correction (numpy's var with ddof=1), mu2_hat is
    mean^2 - var/B, and mu2_hat + sigma2_hat/B = nu_adam.  With beta2 = 0 the returned v IS the preconditioner."""
    n, B = 41, 7
    rng = np.random.default_rng(32)
    g = rng.standard_normal((B, n)) * 0.7 + 0.3
    kw = dict(lr=0.0, beta1=0.9, beta2=0.0, eps=1e-8, step=1)
    zeros = np.zeros(n)
    out = {k: oracle.adam_family_step(zeros, zeros, zeros, g.sum(0), (g * g).sum(0), B, k, **kw)[2] for k in oracle.ADAM_VARIANTS}
    np.testing.assert_allclose(out["adam"], g.mean(0) ** 2, rtol=1e-13)
    np.testing.assert_allclose(out["microadam"], (g * g).mean(0), rtol=1e-13)
    np.testing.assert_allclose(out["microadam_var"], g.var(0, ddof=1), rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(out["microadam_msq"], g.mean(0) ** 2 - g.var(0, ddof=1) / B, rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(out["microadam_msq"] + out["microadam_var"] / B, out["adam"], rtol=1e-12, atol=1e-15)
    # grad_scale s: sums of G_b = g_b / s give the same estimators
    s = 4.0
    v2 = oracle.adam_family_step(zeros, zeros, zeros, g.sum(0) / s, (g * g).sum(0) / s**2, B, "microadam_var", grad_scale=s, **kw)[2]
    np.testing.assert_allclose(v2, out["microadam_var"], rtol=1e-12, atol=1e-15)


def test_adam_family_estimators_are_unbiased_in_expectation():
    """E[mu2_hat] = mu^2 and E[sigma2_hat] = sigma^2 (Eq. (6)); nu_adam and nu_micro are not (Eq. (5))."""
    B, n, mu, sigma = 4, 200_000, 0.5, 2.0
    rng = np.random.default_rng(33)
    g = rng.standard_normal((B, n)) * sigma + mu
    kw = dict(lr=0.0, beta1=0.0, beta2=0.0, eps=1e-8, step=1)
    zeros = np.zeros(n)
    est = {k: oracle.adam_family_step(zeros, zeros, zeros, g.sum(0), (g * g).sum(0), B, k, **kw)[2].mean() for k in oracle.ADAM_VARIANTS}
    tol = 6 * 3 * sigma**2 / math.sqrt(n)
    assert abs(est["microadam_msq"] - mu**2) < tol
    assert abs(est["microadam_var"] - sigma**2) < tol
    assert abs(est["adam"] - (mu**2 + sigma**2 / B)) < tol          # Eq. (5): nu_adam carries sigma^2 / B
    assert abs(est["microadam"] - (mu**2 + sigma**2)) < tol          # nu_micro carries all of sigma^2


def test_adam_family_msq_clamps_a_negative_second_moment_only_when_it_is_used():
    # B = 2, g = {2, -1}: mu = 0.5, nu_adam = 0.25, nu_micro = 2.5, mu2_hat = 2 (0.25 - 1.25) = -2.
    th, m, v = oracle.adam_family_step([1.0], [0.0], [0.0], [1.0], [5.0], 2, "microadam_msq",
                                       lr=1e-3, beta1=0.9, beta2=0.99, eps=1e-6, step=1)
    np.testing.assert_allclose(v, [0.01 * -2.0], rtol=1e-14)          # the EMA keeps the negative value
    np.testing.assert_allclose(m, [0.05], rtol=1e-14)
    np.testing.assert_allclose(th, [1.0 - 1e-3 * 0.5 / 1e-6], rtol=1e-12)   # vh clamped to 0: u = mh / eps
    th_in, _, _ = oracle.adam_family_step([1.0], [0.0], [0.0], [1.0], [5.0], 2, "microadam_msq",
                                          lr=1e-3, beta1=0.9, beta2=0.99, eps=1e-6, eps_inside_sqrt=True, step=1)
    np.testing.assert_allclose(th_in, [1.0 - 1e-3 * 0.5 / 1e-3], rtol=1e-12)  # u = mh / sqrt(eps + 0)
    # the variance needs two examples
    for k in ("microadam_var", "microadam_msq"):
        with pytest.raises(RuntimeError):
            oracle.adam_family_step([1.0], [0.0], [0.0], [1.0], [1.0], 1, k, lr=1e-3, beta1=0.9, beta2=0.99, eps=1e-8)
    # and the MicroAdam member is the MicroAdam step
    a = oracle.adam_family_step([1.0, 2.0], [0.1, 0.0], [0.2, 0.3], [3.0, -1.0], [5.0, 1.0], 2, "microadam", lr=0.1, beta1=0.9, beta2=0.99, eps=1e-8, step=3)
    b = oracle.microadam_step([1.0, 2.0], [0.1, 0.0], [0.2, 0.3], [3.0, -1.0], [5.0, 1.0], 2, lr=0.1, beta1=0.9, beta2=0.99, eps=1e-8, step=3)
    for x, y in zip(a, b):
        np.testing.assert_array_equal(x, y)


def test_microsignsgd_reductions():
    n = 20
    rng = np.random.default_rng(23)
    g = rng.standard_normal(n)
    th0 = rng.standard_normal(n)
    # B = 1, beta = 0: plain SignSGD, theta - lr * sign(g)
    th, m = oracle.microsignsgd_step(th0, np.zeros(n), np.sign(g), 1, lr=0.01, beta=0.0)
    np.testing.assert_allclose(th, th0 - 0.01 * np.sign(g), rtol=1e-14)
    # EMA form and |m| <= 1
    B = 6
    ss = rng.integers(-B, B + 1, n).astype(np.float64)
    m0 = rng.uniform(-1, 1, n)
    th, m = oracle.microsignsgd_step(th0, m0, ss, B, lr=0.1, beta=0.9, weight_decay=0.01)
    np.testing.assert_allclose(m, 0.9 * m0 + 0.1 * ss / B, rtol=1e-13, atol=1e-15)
    assert np.all(np.abs(m) <= 1.0)
    np.testing.assert_allclose(th, th0 - 0.1 * m - 0.01 * th0, rtol=1e-13)


# ----------------------------------------------------------------------------- plumbing

def test_inputs_are_deterministic_and_shaped():
    a, b = inputs.config1(), inputs.config1()
    assert a.shape == (8, 16, 64, 64) and a.X.dtype == torch.float32
    assert torch.equal(a.X, b.X) and torch.equal(a.dY, b.dY) and torch.equal(a.W, b.W)
    h = inputs.heterogeneous_layer(16, 8, 8, 16, seed=5)
    assert h.X.dtype == torch.bfloat16 and len(h.meta["boosted"]) == 2
    norms = h.dY.float().pow(2).mean((1, 2)).sqrt()
    boosted = set(h.meta["boosted"])
    for b_ in range(16):
        assert (norms[b_] > 2.5 * 8 ** -0.5) == (b_ in boosted)
    t = inputs.heavy_tailed_layer(4, 16, 8, 8, seed=6)
    assert t.dY.dtype == torch.bfloat16 and torch.isfinite(t.dY.float()).all()
    sub = inputs.gather_columns(a, [3, 5], [0, 7, 9])
    full = oracle.linear_stats(inputs.to_numpy_bits(a.X), inputs.to_numpy_bits(a.dY))
    part = oracle.linear_stats(inputs.to_numpy_bits(sub.X), inputs.to_numpy_bits(sub.dY))
    np.testing.assert_array_equal(part.sum_g2, full.sum_g2[[3, 5]][:, [0, 7, 9]])
