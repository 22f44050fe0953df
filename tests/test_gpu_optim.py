"""GPU parity of the fused optimizer-update kernels against the fp64 oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_2510_00236_b200 as pe
from paper_2510_00236_b200 import inputs
from parity_util import FROB_TOL, rel_frob

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _state(n, seed):
    g = torch.Generator().manual_seed(seed)
    theta = torch.randn(n, generator=g)
    m = torch.randn(n, generator=g) * 0.1
    v = torch.rand(n, generator=g) * 0.1
    sg = torch.randn(n, generator=g) * 3
    sg2 = sg * sg / 4 + torch.rand(n, generator=g)
    return theta, m, v, sg, sg2


@pytest.mark.parametrize("n", [1, 3, 4, 1023, 4096, 1 << 20, (1 << 20) + 5])
@pytest.mark.parametrize("inside", [False, True])
def test_microadam_matches_oracle(n, inside):
    theta, m, v, sg, sg2 = _state(n, n)
    B, kw = 8, dict(lr=1e-2, beta1=0.9, beta2=0.95, eps=1e-6, step=3, grad_scale=2.0, weight_decay=1e-3)
    ref = oracle.microadam_step(theta.numpy(), m.numpy(), v.numpy(), sg.numpy(), sg2.numpy(), B, eps_inside_sqrt=inside, **kw)
    d = [t.to(DEV).contiguous() for t in (theta, m, v, sg, sg2)]
    lp = torch.empty(n, dtype=torch.bfloat16, device=DEV)
    pe.microadam_step(d[0], d[1], d[2], d[3], d[4], B, eps_inside_sqrt=inside, theta_lp=lp, **kw)
    torch.cuda.synchronize()
    for got, want in zip(d[:3], ref):
        assert rel_frob(got.cpu().numpy(), want) <= 1e-5 <= FROB_TOL
    assert torch.equal(lp, d[0].to(torch.bfloat16))


@pytest.mark.parametrize("variant", ["adam", "microadam", "microadam_var", "microadam_msq"])
@pytest.mark.parametrize("n,inside", [(3, False), (4099, False), ((1 << 19) + 1, True)])
def test_adam_family_matches_oracle(variant, n, inside):
    """Every member of the extended Adam family (Section 3.2.3) against the fp64 oracle.  The sums are built so
    that the squared-mean estimator is clearly positive on even entries and clearly negative on odd ones (there
    MicroAdamMSQ must clamp), never near zero where fp32 and fp64 could take different sides."""
    g = torch.Generator().manual_seed(n + len(variant))
    B = 8
    theta = torch.randn(n, generator=g)
    m = torch.randn(n, generator=g) * 0.1
    sg = (torch.rand(n, generator=g) + 0.5) * torch.where(torch.rand(n, generator=g) < 0.5, -1.0, 1.0) * 3
    odd = (torch.arange(n) % 2 == 1)
    sg2 = torch.where(odd, 4 * sg * sg + 1, 0.25 * sg * sg)
    if variant == "microadam_var":
        sg2 = sg * sg / B * (1.5 + torch.rand(n, generator=g))         # a variance estimate is never negative
    v = torch.zeros(n) if variant == "microadam_msq" else torch.rand(n, generator=g) * 0.1
    kw = dict(lr=1e-2, beta1=0.9, beta2=0.95, eps=1e-6, step=2, grad_scale=0.5, weight_decay=1e-3, eps_inside_sqrt=inside)
    ref = oracle.adam_family_step(theta.numpy(), m.numpy(), v.numpy(), sg.numpy(), sg2.numpy(), B, variant, **kw)
    d = [t.to(DEV).contiguous() for t in (theta, m, v, sg, sg2)]
    lp = torch.empty(n, dtype=torch.bfloat16, device=DEV)
    pe.microadam_family_step(d[0], d[1], d[2], d[3], d[4], B, variant, theta_lp=lp, **kw)
    torch.cuda.synchronize()
    if variant == "microadam_msq" and n > 1:
        assert (ref[2][1::2] < 0).all() and (ref[2][0::2] > 0).all()    # both branches of the clamp are exercised
    for got, want in zip(d[:3], ref):
        assert rel_frob(got.cpu().numpy(), want) <= 1e-5 <= FROB_TOL
    assert rel_frob((d[0].cpu() - theta).numpy(), ref[0] - theta.numpy().astype(np.float64)) <= FROB_TOL
    assert torch.equal(lp, d[0].to(torch.bfloat16))


def test_adam_family_rejects_what_it_cannot_compute():
    t = [torch.zeros(8, device=DEV) for _ in range(5)]
    kw = dict(lr=1e-3, beta1=0.9, beta2=0.99, eps=1e-8, step=1)
    for variant in ("microadam_var", "microadam_msq"):
        with pytest.raises(pe.PestatsError) as e:
            pe.microadam_family_step(*t, 1, variant, **kw)                 # a variance needs two examples
        assert e.value.status == 2
    with pytest.raises(pe.PestatsError) as e:
        pe.microadam_family_step(*t, 4, 7, **kw)
    assert e.value.status == 5


def test_config1_statistics_then_microadam_step():
    li = inputs.config1(DEV)
    mean, stat = pe.pe_linear_stats_f32(li.X, li.dY, "square")
    theta = li.W.clone()
    m = torch.zeros_like(theta)
    v = torch.zeros_like(theta)
    kw = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, step=1)
    pe.microadam_step(theta, m, v, mean, stat, 8, **kw)
    torch.cuda.synchronize()
    st = oracle.linear_stats(inputs.to_numpy_bits(li.X), inputs.to_numpy_bits(li.dY))
    th_ref, m_ref, v_ref = oracle.microadam_step(li.W.cpu().numpy(), np.zeros((64, 64)), np.zeros((64, 64)), st.sum_g, st.sum_g2, 8, **kw)
    assert rel_frob(theta.cpu().numpy(), th_ref) <= FROB_TOL
    assert rel_frob(m.cpu().numpy(), m_ref) <= FROB_TOL and rel_frob(v.cpu().numpy(), v_ref) <= FROB_TOL
    # the update itself (not just theta, which barely moves) must match too
    assert rel_frob(theta.cpu().numpy() - li.W.cpu().numpy(), th_ref - li.W.cpu().numpy().astype(np.float64)) <= FROB_TOL


@pytest.mark.parametrize("n", [2, 4, 1000, (1 << 18) + 3])
def test_microsignsgd_matches_oracle(n):
    g = torch.Generator().manual_seed(n)
    B = 16
    theta = torch.randn(n, generator=g)
    m = torch.rand(n, generator=g) * 2 - 1
    ss = torch.randint(-B, B + 1, (n,), generator=g).float()
    kw = dict(lr=3.47e-3, beta=0.9, weight_decay=1e-4)
    th_ref, m_ref = oracle.microsignsgd_step(theta.numpy(), m.numpy(), ss.numpy(), B, **kw)
    d = [t.to(DEV).contiguous() for t in (theta, m, ss)]
    lp = torch.empty(n, dtype=torch.bfloat16, device=DEV)
    pe.microsignsgd_step(d[0], d[1], d[2], B, theta_lp=lp, **kw)
    torch.cuda.synchronize()
    assert rel_frob(d[0].cpu().numpy(), th_ref) <= 1e-6
    assert rel_frob(d[1].cpu().numpy(), m_ref) <= 1e-6
    assert torch.equal(lp, d[0].to(torch.bfloat16))
    assert rel_frob((d[0].cpu() - theta).numpy(), th_ref - theta.numpy().astype(np.float64)) <= FROB_TOL


def test_multi_step_microadam_trajectory():
    n, B, steps = 5000, 4, 5
    g = torch.Generator().manual_seed(5)
    theta = torch.randn(n, generator=g)
    th_r, m_r, v_r = theta.numpy().astype(np.float64), np.zeros(n), np.zeros(n)
    th_d, m_d, v_d = theta.to(DEV), torch.zeros(n, device=DEV), torch.zeros(n, device=DEV)
    for t in range(1, steps + 1):
        G = torch.randn(B, n, generator=g)
        sg, sg2 = G.sum(0), (G * G).sum(0)
        kw = dict(lr=1e-2, beta1=0.9, beta2=0.95, eps=1e-8, step=t)
        th_r, m_r, v_r = oracle.microadam_step(th_r, m_r, v_r, sg.numpy(), sg2.numpy(), B, **kw)
        pe.microadam_step(th_d, m_d, v_d, sg.to(DEV), sg2.to(DEV), B, **kw)
    torch.cuda.synchronize()
    assert rel_frob(th_d.cpu().numpy(), th_r) <= 1e-5
    assert rel_frob((th_d.cpu() - theta).numpy(), th_r - theta.numpy().astype(np.float64)) <= FROB_TOL


def test_launch_counter_counts_kernels():
    pe.pe_reset_launch_count()
    n = 256
    z = [torch.zeros(n, device=DEV) for _ in range(4)]
    pe.microsignsgd_step(z[0], z[1], z[2], 4, lr=0.1, beta=0.9)
    pe.microsignsgd_step(z[0], z[1], z[2], 4, lr=0.1, beta=0.9)
    assert pe.pe_launch_count() == 2
