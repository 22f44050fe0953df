"""The give-up path of the tensor-core kernels: every wait on an on-chip barrier has a cycle budget; when one
runs out the kernel skips its outputs, exits normally and latches PE_ERR_TIMEOUT with the identity of the wait.
The budget is lowered to one cycle here, so that the first wait that does not succeed at once gives up (no
kernel is broken and nothing hangs: all waits still end, just unsuccessfully); afterwards the default budget
is restored and the same call must be correct."""
import numpy as np
import pytest
import torch

import oracle
import paper_2510_00236_b200 as pe
from paper_2510_00236_b200 import inputs
from parity_util import FROB_TOL, rel_frob

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
PE_ERR_TIMEOUT = 8


@pytest.fixture()
def short_waits():
    pe.pe_set_path(pe.PATH_TENSOR)
    pe.pe_set_wait_limit_cycles(1, DEV)
    yield
    pe.pe_set_wait_limit_cycles(0, DEV)
    pe.pe_set_path(pe.PATH_AUTO)


def test_waits_that_run_out_are_reported_and_the_library_stays_usable(short_waits):
    li = inputs.gaussian_layer(8, 512, 256, 512, seed=31, device=DEV, with_weights=True)
    B, T, d_in, d_out = li.shape
    sentinel = 7.0
    mean = torch.full((d_out, d_in), sentinel, device=DEV)
    stat = torch.full((d_out, d_in), sentinel, device=DEV)
    pe.pe_linear_stats(li.X, li.dY, "square", mean, stat)               # returns PE_OK: the give-up happens on the device
    status, detail = pe.pe_get_async_status(DEV)
    assert status == PE_ERR_TIMEOUT and 1 <= detail <= 4, (status, detail)
    assert pe.pe_get_async_status(DEV) == (0, 0)                        # reading the status clears it

    tok = torch.full((d_out, d_in), sentinel, device=DEV)
    pe.pe_token_sqstats(li.X, li.dY, tok)                               # the one-kernel per-token statistic
    status, detail = pe.pe_get_async_status(DEV)
    assert status == PE_ERR_TIMEOUT and detail > 0, (status, detail)

    # the fused statistics + update call must leave the parameters alone when it gives up
    W = li.W.clone()
    th, mm, vv = W.clone(), torch.zeros_like(W), torch.zeros_like(W)
    ws = torch.zeros(pe.pe_linear_fused_workspace_bytes(d_in, d_out), dtype=torch.uint8, device=DEV)
    pe.pe_linear_microadam_step(li.X, li.dY, th, mm, vv, lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, step=1, out_mean=mean, out_stat=stat,
                                workspace=ws)
    status, detail = pe.pe_get_async_status(DEV)
    assert status == PE_ERR_TIMEOUT, (status, detail)
    assert torch.equal(th, W) and float(mm.abs().max()) == 0.0 and float(vv.abs().max()) == 0.0

    # default budget back: the same calls are correct
    pe.pe_set_wait_limit_cycles(0, DEV)
    st = oracle.linear_stats(inputs.to_numpy_bits(li.X), inputs.to_numpy_bits(li.dY))
    tok_ref = oracle.token_sqstats(inputs.to_numpy_bits(li.X), inputs.to_numpy_bits(li.dY))
    pe.pe_linear_stats(li.X, li.dY, "square", mean, stat)
    pe.pe_token_sqstats(li.X, li.dY, tok)
    assert pe.pe_get_async_status(DEV) == (0, 0)
    assert rel_frob(mean.cpu().numpy(), st.sum_g) <= FROB_TOL and rel_frob(stat.cpu().numpy(), st.sum_g2) <= FROB_TOL
    assert rel_frob(tok.cpu().numpy(), tok_ref) <= FROB_TOL
    pe.pe_linear_microadam_step(li.X, li.dY, th, mm, vv, lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, step=1, workspace=ws)
    assert pe.pe_get_async_status(DEV) == (0, 0)
    W0 = W.cpu().numpy().astype(np.float64)
    th_ref, _, _ = oracle.microadam_step(W0, np.zeros_like(W0), np.zeros_like(W0), st.sum_g, st.sum_g2, B, lr=1e-3, beta1=0.9, beta2=0.999,
                                         eps=1e-8, step=1)
    assert np.linalg.norm((th.cpu().numpy() - W0) - (th_ref - W0)) <= FROB_TOL * np.linalg.norm(th_ref - W0)
