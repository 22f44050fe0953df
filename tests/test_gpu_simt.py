"""GPU parity of the SIMT kernels (fp32 inputs, and bf16 shapes forced onto the SIMT path) against the oracle."""
import numpy as np
import pytest
import torch

import paper_2510_00236_b200 as pe
from paper_2510_00236_b200 import inputs
from parity_util import check_all, gpu_stats

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(autouse=True)
def _auto_path():
    prev = pe.pe_set_path(pe.PATH_AUTO)
    yield
    pe.pe_set_path(prev)


def test_config1_fp32_all_statistics():
    li = inputs.config1(DEV)
    rep = check_all(li, phis=("identity", "square", "sign"))
    assert pe.pe_last_path() == pe.PATH_SIMT
    assert rep["square_err"] < 1e-5


@pytest.mark.parametrize("B,T,d_in,d_out", [(3, 40, 136, 200), (5, 17, 72, 9), (1, 1, 1, 1), (7, 33, 65, 129), (4, 5, 8, 300)])
def test_simt_fp32_ragged_shapes(B, T, d_in, d_out):
    li = inputs.gaussian_layer(B, T, d_in, d_out, dtype=torch.float32, seed=100 + B, device=DEV)
    check_all(li, phis=("identity", "square", "sign"))


@pytest.mark.parametrize("B,T,d_in,d_out", [(6, 48, 136, 72), (64, 16, 100, 60), (2, 300, 64, 64)])
def test_simt_bf16_forced(B, T, d_in, d_out):
    pe.pe_set_path(pe.PATH_SIMT)
    li = inputs.gaussian_layer(B, T, d_in, d_out, seed=200 + B, device=DEV)
    check_all(li)
    assert pe.pe_last_path() == pe.PATH_SIMT


def test_bf16_shape_not_multiple_of_8_takes_simt_automatically():
    li = inputs.gaussian_layer(4, 20, 36, 50, seed=7, device=DEV)
    check_all(li)
    assert pe.pe_last_path() == pe.PATH_SIMT
    pe.pe_set_path(pe.PATH_TENSOR)
    with pytest.raises(pe.PestatsError) as e:
        pe.pe_linear_stats(li.X, li.dY, "square")
    assert e.value.status == 4        # PE_ERR_UNSUPPORTED_SHAPE


def test_empty_batch_and_empty_sequence_give_zeros():
    for B, T in ((0, 5), (3, 0)):
        X = torch.zeros((B, T, 16), dtype=torch.float32, device=DEV)
        dY = torch.zeros((B, T, 24), dtype=torch.float32, device=DEV)
        mean, stat = gpu_stats(inputs.LayerInputs("e", X, dY), "square")
        assert np.all(mean == 0) and np.all(stat == 0)
        Xb, dYb = X.to(torch.bfloat16), dY.to(torch.bfloat16)
        mean, stat = gpu_stats(inputs.LayerInputs("e", Xb, dYb), "sign")
        assert np.all(mean == 0) and np.all(stat == 0)
        out = pe.pe_token_sqstats(Xb, dYb)
        assert torch.all(out == 0)


def test_only_one_output_requested():
    li = inputs.gaussian_layer(3, 10, 24, 40, dtype=torch.float32, seed=9, device=DEV)
    mean_ref, stat_ref = gpu_stats(li, "square")
    stat = torch.full((40, 24), float("nan"), device=DEV)
    pe.pe_linear_stats_f32(li.X, li.dY, "square", None, stat)
    mean = torch.full((40, 24), float("nan"), device=DEV)
    pe.pe_linear_stats_f32(li.X, li.dY, "square", mean, None)
    torch.cuda.synchronize()
    assert np.array_equal(stat.cpu().numpy(), stat_ref) and np.array_equal(mean.cpu().numpy(), mean_ref)


def test_three_statistics_call_on_a_shape_the_tensor_cores_do_not_take():
    """pe_linear_stats_all falls back to the two separate calls (here both on the SIMT kernel: widths that are
    not multiples of 8)."""
    from parity_util import FROB_TOL, check_sign, oracle_on, rel_frob
    li = inputs.gaussian_layer(6, 40, 36, 20, seed=1500, device=DEV)
    mean, sq, sgn = pe.pe_linear_stats_all(li.X, li.dY)
    torch.cuda.synchronize()
    assert pe.pe_last_path() == pe.PATH_SIMT
    st, _ = oracle_on(li)
    assert rel_frob(mean.cpu().numpy(), st.sum_g) <= FROB_TOL and rel_frob(sq.cpu().numpy(), st.sum_g2) <= FROB_TOL
    check_sign(sgn.cpu().numpy(), st)


def test_accumulate_on_the_simt_path():
    from parity_util import FROB_TOL, oracle_on, rel_frob
    li = inputs.gaussian_layer(7, 33, 36, 20, seed=1700, device=DEV)
    mean = torch.zeros((20, 36), device=DEV)
    stat = torch.zeros((20, 36), device=DEV)
    for lo, hi in ((0, 3), (3, 7)):
        pe.pe_linear_stats_accumulate(li.X[lo:hi].clone(), li.dY[lo:hi].clone(), "square", mean, stat)
    torch.cuda.synchronize()
    assert pe.pe_last_path() == pe.PATH_SIMT
    st, _ = oracle_on(li)
    assert rel_frob(mean.cpu().numpy(), st.sum_g) <= FROB_TOL and rel_frob(stat.cpu().numpy(), st.sum_g2) <= FROB_TOL


def test_per_example_squared_norms_on_the_simt_path():
    import oracle
    li = inputs.gaussian_layer(9, 33, 36, 20, seed=1900, device=DEV)
    norms = pe.pe_example_sqnorms(li.X, li.dY)
    torch.cuda.synchronize()
    assert pe.pe_last_path() == pe.PATH_SIMT
    want = oracle.example_sqnorms(inputs.to_numpy_bits(li.X), inputs.to_numpy_bits(li.dY))
    assert np.max(np.abs(norms.cpu().numpy() - want) / want) <= 2e-3
    assert pe.pe_example_sqnorms(li.X[:0], li.dY[:0]).numel() == 0
