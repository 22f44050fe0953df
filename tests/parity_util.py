"""Helpers shared by the GPU parity tests: run the CUDA library and the CPU oracle on the same
seeded inputs and compare at the stated tolerances."""
from __future__ import annotations

import numpy as np
import torch

import oracle
import paper_2510_00236_b200 as pe
from paper_2510_00236_b200 import inputs

# Relative Frobenius tolerance for the mean, square and per-token statistics and for updated
# parameters; the sign statistic must agree exactly wherever |G_b| > SIGN_REL * max|G_b|.
FROB_TOL = 2e-3
SIGN_REL = 1e-3


def rel_frob(a: np.ndarray, ref: np.ndarray) -> float:
    a = np.asarray(a, np.float64)
    ref = np.asarray(ref, np.float64)
    den = np.linalg.norm(ref)
    num = np.linalg.norm(a - ref)
    return float(num / den) if den > 0 else float(num)


def assert_entries_close(a, ref, what, rel_rms=1e-3):
    """Per-entry bound beside the Frobenius one: no single entry may be off by more than rel_rms times the
    reference's rms (observed deviations are around 1e-7 of it; one wrong entry among millions is of order 1)."""
    a = np.asarray(a, np.float64)
    ref = np.asarray(ref, np.float64)
    scale = float(np.sqrt(np.mean(ref ** 2)))
    worst = float(np.max(np.abs(a - ref))) if a.size else 0.0
    assert worst <= rel_rms * scale + 1e-30, f"{what}: an entry is off by {worst:.3e} (rms of the reference {scale:.3e})"


def assert_token_entries_close(a, ref, what):
    """Per-token statistic: all terms are non-negative and each squared operand is rounded to 11 bits, so every
    entry must be within 2e-3 of its own exact value."""
    a = np.asarray(a, np.float64)
    ref = np.asarray(ref, np.float64)
    assert np.all(np.abs(a - ref) <= 2e-3 * np.abs(ref) + 1e-30), f"{what}: an entry is off by more than 2e-3 of its value"


def boundary_and_random(n: int, k: int, seed: int, tile: int = 128) -> list[int]:
    """Sample of indices in [0, n): tile edges (first/last element of the first, second and last tile)
    plus seeded random ones."""
    edges = {0, n - 1, min(tile - 1, n - 1), min(tile, n - 1), ((n - 1) // tile) * tile, max(0, ((n - 1) // tile) * tile - 1)}
    rng = np.random.default_rng(seed)
    extra = set(int(x) for x in rng.choice(n, size=min(n, k), replace=False))
    out = sorted(edges | extra)
    return out[: max(k, len(edges))] if len(out) > max(k, len(edges)) else out


def gpu_stats(li: inputs.LayerInputs, phi: str, poison: bool = True):
    """Runs pe_linear_stats (bf16) or pe_linear_stats_f32 on li; returns (mean, stat) as numpy."""
    B, T, d_in, d_out = li.shape
    mean = torch.full((d_out, d_in), float("nan"), device=li.X.device) if poison else torch.empty((d_out, d_in), device=li.X.device)
    stat = torch.full((d_out, d_in), float("nan"), device=li.X.device) if poison else torch.empty((d_out, d_in), device=li.X.device)
    fn = pe.pe_linear_stats if li.X.dtype == torch.bfloat16 else pe.pe_linear_stats_f32
    fn(li.X, li.dY, phi, mean, stat)
    torch.cuda.synchronize()
    return mean.cpu().numpy(), stat.cpu().numpy()


def gpu_token(li: inputs.LayerInputs):
    B, T, d_in, d_out = li.shape
    out = torch.full((d_out, d_in), float("nan"), device=li.X.device)
    if li.X.dtype == torch.bfloat16:
        pe.pe_token_sqstats(li.X, li.dY, out)
    else:
        pe.pe_token_sqstats_f32(li.X, li.dY, out)
    torch.cuda.synchronize()
    return out.cpu().numpy()


def oracle_on(li: inputs.LayerInputs):
    Xh, dYh = inputs.to_numpy_bits(li.X), inputs.to_numpy_bits(li.dY)
    return oracle.linear_stats(Xh, dYh, small_rel=SIGN_REL), oracle.token_sqstats(Xh, dYh)


def check_sign(gpu_sign: np.ndarray, st: oracle.LinearStats) -> int:
    """Sign rule: every contribution with |G_b| above the threshold must agree, so an entry's sum may
    differ by at most 2 per below-threshold example.  Returns the number of disagreeing entries."""
    diff = np.abs(gpu_sign.astype(np.float64) - st.sum_sign)
    assert np.all(diff <= 2.0 * st.n_small + 1e-9), (
        f"sign statistic differs above the threshold at {int((diff > 2.0 * st.n_small).sum())} entries")
    assert np.all(gpu_sign == np.round(gpu_sign)), "sign statistic must be integer valued"
    return int((diff > 0).sum())


def check_all(li_full: inputs.LayerInputs, rows=None, cols=None, phis=("square", "sign"), token=True, tol=FROB_TOL,
              bench_calls=False):
    """Full comparison when rows/cols are None, otherwise on the sampled output rows x cols: the GPU runs
    the full layer, the oracle the column-gathered sub-layer (each output entry depends on one column
    of dY and one of X only)."""
    li_or = li_full if rows is None else inputs.gather_columns(li_full, rows, cols)
    st, tok = oracle_on(li_or)
    pick = (lambda a: a) if rows is None else (lambda a: a[np.asarray(rows)][:, np.asarray(cols)])
    report = {}
    for phi in phis:
        mean, stat = gpu_stats(li_full, phi)
        mean, stat = pick(mean), pick(stat)
        assert np.isfinite(mean).all() and np.isfinite(stat).all(), "unwritten or non-finite outputs"
        e = rel_frob(mean, st.sum_g)
        assert e <= tol, f"sum_b G_b: rel. Frobenius error {e:.3e} > {tol}"
        assert_entries_close(mean, st.sum_g, f"sum_b G_b ({phi})")
        report[f"mean_err_{phi}"] = e
        if phi == "square":
            e = rel_frob(stat, st.sum_g2)
            assert e <= tol, f"sum_b G_b^2: rel. Frobenius error {e:.3e} > {tol}"
            assert_entries_close(stat, st.sum_g2, "sum_b G_b^2")
            report["square_err"] = e
        elif phi == "sign":
            report["sign_disagreements"] = check_sign(stat, st)
        else:
            e = rel_frob(stat, st.sum_g)
            assert e <= tol
            assert_entries_close(stat, st.sum_g, "sum_b G_b (identity)")
    if token:
        t = pick(gpu_token(li_full))
        assert np.isfinite(t).all()
        e = rel_frob(t, tok)
        assert e <= tol, f"per-token statistic: rel. Frobenius error {e:.3e} > {tol}"
        assert_token_entries_close(t, tok, "per-token statistic")
        report["token_err"] = e
    if bench_calls:
        # the calls the benchmark step makes: all three statistics in one pass, the two-pass per-token statistic
        dev = li_full.X.device
        B, T, d_in, d_out = li_full.shape
        outs = [torch.full((d_out, d_in), float("nan"), device=dev) for _ in range(3)]
        pe.pe_linear_stats_all(li_full.X, li_full.dY, *outs)
        torch.cuda.synchronize()
        mean, sq, sgn = (pick(o.cpu().numpy()) for o in outs)
        del outs
        assert np.isfinite(mean).all() and np.isfinite(sq).all() and np.isfinite(sgn).all()
        report["one_pass_mean_err"], report["one_pass_square_err"] = rel_frob(mean, st.sum_g), rel_frob(sq, st.sum_g2)
        assert report["one_pass_mean_err"] <= tol and report["one_pass_square_err"] <= tol
        assert_entries_close(mean, st.sum_g, "one-pass sum_b G_b")
        assert_entries_close(sq, st.sum_g2, "one-pass sum_b G_b^2")
        report["one_pass_sign_disagreements"] = check_sign(sgn, st)
        t = pick(pe.pe_token_sqstats_staged(li_full.X, li_full.dY).cpu().numpy())
        assert np.isfinite(t).all()
        report["token_two_pass_err"] = rel_frob(t, tok)
        assert report["token_two_pass_err"] <= tol
        assert_token_entries_close(t, tok, "two-pass per-token statistic")
        report["oracle_stats"] = st
    status, detail = pe.pe_get_async_status(li_full.X.device)
    assert status == 0, f"device status {status} detail {detail}"
    return report
