"""GPU parity of the statistics + parameter update fused into one launch against the oracle's composition
linear_stats -> adam_family_step / microsignsgd_step (Algorithm 1; Section 3.1)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2510_00236_b200 as pe
from paper_2510_00236_b200 import inputs
from parity_util import FROB_TOL, SIGN_REL, check_sign, rel_frob

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
ADAM = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8)


@pytest.fixture(autouse=True, params=[pe.FUSED_ALWAYS, pe.FUSED_AUTO], ids=["fused_kernel", "auto"])
def _fused_mode(request):
    """Every test runs with the fused kernel forced and with the default choice (fused launch only when no
    statistic buffers are given, otherwise the two-kernel sequence)."""
    prev = pe.pe_set_fused_update(request.param)
    yield request.param
    pe.pe_set_fused_update(prev)


def _state(li, seed):
    g = torch.Generator(device="cpu").manual_seed(seed)
    d_out, d_in = li.shape[3], li.shape[2]
    W = (torch.randn((d_out, d_in), generator=g) / d_in ** 0.5)
    m = torch.randn((d_out, d_in), generator=g) * 1e-3
    v = torch.rand((d_out, d_in), generator=g) * 1e-4
    return W, m, v


def _upd_err(new, old, ref_new):
    """Relative Frobenius error of the UPDATE (new - old), the quantity the step actually computes."""
    num = np.linalg.norm((new - old) - (ref_new - old))
    return float(num / (np.linalg.norm(ref_new - old) + 1e-300))


def _adam_kw(variant):
    """The squared-mean member runs with eps = 1e-6, as in Section 3.2.3: its second moment is clamped at zero
    where it is used, and with eps = 1e-8 an entry whose fp32 state sits within 1e-9 of the clamp moves by
    percents between fp32 and fp64 state, which is a property of that hyper-parameter, not of the kernels."""
    return dict(ADAM, eps=1e-6) if variant == "microadam_msq" else ADAM


def _run_adam(li, variant, eps_inside, step, with_outputs, with_workspace, W, m, v, lp=True):
    B, T, d_in, d_out = li.shape
    th, mm, vv = W.to(DEV), m.to(DEV), v.to(DEV)
    tlp = torch.empty((d_out, d_in), dtype=torch.bfloat16, device=DEV) if lp else None
    om = torch.full((d_out, d_in), float("nan"), device=DEV) if with_outputs else None
    os_ = torch.full((d_out, d_in), float("nan"), device=DEV) if with_outputs else None
    ws = torch.empty(pe.pe_linear_fused_workspace_bytes(d_in, d_out), dtype=torch.uint8, device=DEV) if with_workspace else None
    before = pe.pe_launch_count()
    pe.pe_linear_microadam_step(li.X, li.dY, th, mm, vv, step=step, variant=variant, eps_inside_sqrt=eps_inside, theta_lp=tlp,
                                out_mean=om, out_stat=os_, workspace=ws, **_adam_kw(variant))
    torch.cuda.synchronize()
    return th, mm, vv, tlp, om, os_, pe.pe_launch_count() - before


@pytest.mark.parametrize("B,T,d_in,d_out", [
    (64, 256, 512, 2048),    # the transformer-MLP-shaped layer: batch split over two blocks per tile
    (12, 80, 200, 264),      # ragged tiles, 256 x 128 tile (d_in pads badly to 192)
    (70, 48, 136, 264),      # 256 x 192 tile, short sequences, batch split
    (3, 300, 392, 520),      # unsplit-capable small batch
    (9, 16, 320, 192),
])
@pytest.mark.parametrize("variant,eps_inside", [("microadam", False), ("adam", True), ("microadam_var", False), ("microadam_msq", True)])
def test_fused_adam_family_matches_stats_then_step(B, T, d_in, d_out, variant, eps_inside):
    li = inputs.heterogeneous_layer(B, T, d_in, d_out, seed=4000 + B, device=DEV)
    W, m, v = _state(li, 7)
    step = 3
    rows = list(range(d_out)) if d_out <= 600 else sorted(set(np.linspace(0, d_out - 1, 96).astype(int)))
    cols = list(range(d_in)) if d_out <= 600 else sorted(set(np.linspace(0, d_in - 1, 96).astype(int)))
    sub = li if d_out <= 600 else inputs.gather_columns(li, rows, cols)
    st = oracle.linear_stats(inputs.to_numpy_bits(sub.X), inputs.to_numpy_bits(sub.dY), small_rel=SIGN_REL)
    pick = lambda a: a.cpu().numpy().astype(np.float64)[np.ix_(rows, cols)]
    W0, m0, v0 = (pick(t) for t in (W, m, v))
    th_ref, m_ref, v_ref = oracle.adam_family_step(W0, m0, v0, st.sum_g, st.sum_g2, B, variant, step=step, eps_inside_sqrt=eps_inside,
                                                   **_adam_kw(variant))
    for with_outputs, with_ws in ((True, True), (False, False), (True, False)):
        th, mm, vv, tlp, om, os_, launches = _run_adam(li, variant, eps_inside, step, with_outputs, with_ws, W, m, v)
        assert _upd_err(pick(th), W0, th_ref) <= FROB_TOL, (with_outputs, with_ws)
        assert _upd_err(pick(mm), m0, m_ref) <= FROB_TOL
        assert _upd_err(pick(vv), v0, v_ref) <= FROB_TOL
        assert torch.equal(tlp, th.to(torch.bfloat16))
        if with_outputs:
            assert rel_frob(pick(om), st.sum_g) <= FROB_TOL and rel_frob(pick(os_), st.sum_g2) <= FROB_TOL
        assert launches <= 3, launches                 # statistics kernel (+ zeroing kernel of a split batch) (+ update kernel)
    assert pe.pe_get_async_status(DEV) == (0, 0)
    assert pe.pe_last_path() == pe.PATH_TENSOR


def _close(a, b):
    return torch.allclose(a, b, rtol=2e-6, atol=1e-10)


def test_fused_update_equals_the_two_call_sequence_on_an_unsplit_schedule():
    """Same sums in the same order: with the batch unsplit the statistics are bit-identical to
    pe_linear_stats and the update equals microadam_step of them up to the compiler's choice of fused
    multiply-adds in the two kernels."""
    li = inputs.gaussian_layer(4, 128, 1024, 4096, seed=5, device=DEV)      # many tiles, few examples: never split
    W, m, v = _state(li, 9)
    th, mm, vv, tlp, om, os_, launches = _run_adam(li, "microadam", False, 2, True, True, W, m, v)
    assert launches <= 2
    mean, sq = pe.pe_linear_stats(li.X, li.dY, "square")
    th2, m2, v2 = W.to(DEV), m.to(DEV), v.to(DEV)
    pe.microadam_step(th2, m2, v2, mean, sq, 4, step=2, **ADAM)
    torch.cuda.synchronize()
    assert torch.equal(om, mean) and torch.equal(os_, sq)
    assert _close(th, th2) and _close(mm, m2) and _close(vv, v2)


def test_fused_adam_fp32_inputs_config1():
    """Config 1 (fp32, B=8, T=16, 64 x 64): statistics and one MicroAdam step in one SIMT launch."""
    li = inputs.config1(DEV)
    B, T, d_in, d_out = li.shape
    W = li.W.clone()
    th, mm, vv = W.clone(), torch.zeros_like(W), torch.zeros_like(W)
    before = pe.pe_launch_count()
    pe.pe_linear_microadam_step_f32(li.X, li.dY, th, mm, vv, step=1, **ADAM)
    torch.cuda.synchronize()
    assert pe.pe_launch_count() - before == 1 and pe.pe_last_path() == pe.PATH_SIMT
    st = oracle.linear_stats(li.X.cpu().numpy(), li.dY.cpu().numpy())
    W0 = W.cpu().numpy().astype(np.float64)
    th_ref, m_ref, v_ref = oracle.microadam_step(W0, np.zeros_like(W0), np.zeros_like(W0), st.sum_g, st.sum_g2, B, step=1, **ADAM)
    assert _upd_err(th.cpu().numpy().astype(np.float64), W0, th_ref) <= FROB_TOL
    assert rel_frob(mm.cpu().numpy(), m_ref) <= FROB_TOL and rel_frob(vv.cpu().numpy(), v_ref) <= FROB_TOL


@pytest.mark.parametrize("B,T,d_in,d_out", [(64, 256, 512, 2048), (12, 80, 200, 264), (70, 48, 136, 264), (5, 600, 264, 520)])
def test_fused_microsignsgd_matches_sign_stats_then_step(B, T, d_in, d_out):
    li = inputs.heterogeneous_layer(B, T, d_in, d_out, seed=4100 + B, device=DEV)
    W, m, _ = _state(li, 11)
    rows = list(range(d_out)) if d_out <= 600 else sorted(set(np.linspace(0, d_out - 1, 96).astype(int)))
    cols = list(range(d_in)) if d_out <= 600 else sorted(set(np.linspace(0, d_in - 1, 96).astype(int)))
    sub = li if d_out <= 600 else inputs.gather_columns(li, rows, cols)
    st = oracle.linear_stats(inputs.to_numpy_bits(sub.X), inputs.to_numpy_bits(sub.dY), small_rel=SIGN_REL)
    pick = lambda a: a.cpu().numpy().astype(np.float64)[np.ix_(rows, cols)]
    kw = dict(lr=3.47e-3, beta=0.9)
    for with_out, with_ws in ((True, True), (False, False)):
        th, mm = W.to(DEV), m.to(DEV)
        tlp = torch.empty((d_out, d_in), dtype=torch.bfloat16, device=DEV)
        sg = torch.full((d_out, d_in), float("nan"), device=DEV) if with_out else None
        ws = torch.empty(pe.pe_linear_fused_workspace_bytes(d_in, d_out), dtype=torch.uint8, device=DEV) if with_ws else None
        pe.pe_linear_microsignsgd_step(li.X, li.dY, th, mm, theta_lp=tlp, out_sign=sg, workspace=ws, **kw)
        # the same statistic from the separate call: the update must be exactly microsignsgd_step of it
        _, sg2 = pe.pe_linear_stats(li.X, li.dY, "sign", None, torch.empty((d_out, d_in), device=DEV))
        th2, m2 = W.to(DEV), m.to(DEV)
        pe.microsignsgd_step(th2, m2, sg2, B, **kw)
        torch.cuda.synchronize()
        check_sign(pick(sg2), st)
        if with_out:
            assert torch.equal(sg, sg2)
        assert _close(th, th2) and _close(mm, m2) and torch.equal(tlp, th.to(torch.bfloat16))
        # and against the oracle wherever no example sits below the sign threshold
        th_ref, m_ref = oracle.microsignsgd_step(pick(W), pick(m), st.sum_sign, B, **kw)
        exact = st.n_small == 0
        np.testing.assert_allclose(pick(mm)[exact], m_ref[exact], rtol=1e-5, atol=1e-7)
        np.testing.assert_allclose(pick(th)[exact], th_ref[exact], rtol=1e-5, atol=1e-7)
    assert pe.pe_get_async_status(DEV) == (0, 0)
