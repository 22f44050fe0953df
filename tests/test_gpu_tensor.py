"""GPU parity of the tcgen05 tensor-core kernel against the oracle: small shapes that span several
tiles with ragged tails, and the benchmark configurations at full size on sampled outputs."""
import numpy as np
import pytest
import torch

import oracle
import paper_2510_00236_b200 as pe
from paper_2510_00236_b200 import inputs
from parity_util import SIGN_REL, boundary_and_random, check_all, check_sign, gpu_stats, rel_frob

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(autouse=True)
def _tensor_path():
    prev = pe.pe_set_path(pe.PATH_TENSOR)
    yield
    pe.pe_set_path(prev)


def test_structured_single_tile_catches_layout_mistakes():
    """Every (token, feature) pair gets a distinct small integer, exactly representable in bf16, so
    a wrong swizzle, stride or operand orientation changes the result by whole numbers."""
    B, T, d_in, d_out = 2, 64, 128, 128
    t = torch.arange(T, dtype=torch.float32).view(1, T, 1)
    X = ((t % 5) - 2 + (torch.arange(d_in).view(1, 1, d_in) % 7 - 3) + torch.arange(B).view(B, 1, 1)).to(torch.bfloat16)
    dY = ((t % 3) - 1 + (torch.arange(d_out).view(1, 1, d_out) % 11 - 5) * 0.5 - torch.arange(B).view(B, 1, 1)).to(torch.bfloat16)
    li = inputs.LayerInputs("structured", X.to(DEV).contiguous(), dY.to(DEV).contiguous())
    rep = check_all(li, phis=("identity", "square", "sign"), token=False, tol=1e-6)
    assert pe.pe_last_path() == pe.PATH_TENSOR
    assert rep["sign_disagreements"] == 0
    check_all(li, phis=(), token=True)          # 128 rows: too few for bf16 squares, runs on the SIMT kernel


@pytest.mark.parametrize("B,T,d_in,d_out", [
    (3, 64, 128, 128),      # one tile, one stage per example
    (5, 200, 136, 264),     # ragged tiles, T not a multiple of 16 or 64
    (9, 16, 320, 192),      # short sequences: epilogue-bound regime
    (2, 1, 64, 72),         # rank-one gradients
    (1, 1000, 256, 128),    # single example
    (70, 48, 8, 8),         # smallest widths the path takes, batch split across blocks
    (40, 96, 384, 256),
    (130, 32, 264, 392),    # many short sequences: 32-token stages, batch split
    (21, 64, 136, 520),     # half-filled stages
    (11, 33, 128, 256),     # just above the short-stage limit
    (13, 32, 264, 136),     # exactly one short stage per example
    (2, 4100, 136, 264),    # very long sequences on the 256 x 192 tile
    (2, 4100, 200, 264),    # d_in pads badly to 192: sum_b G_b kept in tensor memory beside a 256 x 256 tile
])
def test_tensor_small_shapes_full_comparison(B, T, d_in, d_out):
    li = inputs.gaussian_layer(B, T, d_in, d_out, seed=300 + 7 * B + T, device=DEV)
    check_all(li, phis=("identity", "square", "sign"), token=False)
    assert pe.pe_last_path() == pe.PATH_TENSOR
    check_all(li, phis=(), token=True)
    assert pe.pe_last_path() == (pe.PATH_TENSOR if B * T >= 256 else pe.PATH_SIMT)


@pytest.mark.parametrize("B,T,d_in,d_out", [(5, 200, 136, 264), (9, 16, 320, 192), (33, 300, 520, 264), (2, 1, 64, 72), (75, 40, 520, 264)])
def test_single_output_calls_use_the_wide_tile_and_match(B, T, d_in, d_out):
    """Asking for only sum_b phi(G_b) (or only sum_b G_b) takes the 256 x 256 pair tile (or the plain
    contraction); both must agree with the oracle like the two-output call does."""
    from parity_util import FROB_TOL, check_sign, oracle_on, rel_frob
    li = inputs.gaussian_layer(B, T, d_in, d_out, seed=900 + B, device=DEV)
    st, _ = oracle_on(li)
    for phi in ("square", "sign"):
        stat = torch.full((d_out, d_in), float("nan"), device=DEV)
        pe.pe_linear_stats(li.X, li.dY, phi, None, stat)
        mean = torch.full((d_out, d_in), float("nan"), device=DEV)
        pe.pe_linear_stats(li.X, li.dY, phi, mean, None)
        torch.cuda.synchronize()
        assert rel_frob(mean.cpu().numpy(), st.sum_g) <= FROB_TOL
        if phi == "square":
            assert rel_frob(stat.cpu().numpy(), st.sum_g2) <= FROB_TOL
        else:
            check_sign(stat.cpu().numpy(), st)
    assert pe.pe_get_async_status(DEV) == (0, 0)


def test_odd_batch_slices_and_long_sequences_single_output():
    """An odd number of examples per slice ends on an unpaired example whose stages run through both
    issuers' slots; long sequences make that tail many stages long."""
    from parity_util import FROB_TOL, check_sign, oracle_on, rel_frob
    li = inputs.gaussian_layer(3, 2000, 264, 520, seed=77, device=DEV)
    st, tok = oracle_on(li)
    for both in (True, False):
        stat = torch.full((520, 264), float("nan"), device=DEV)
        mean = torch.full((520, 264), float("nan"), device=DEV) if both else None
        pe.pe_linear_stats(li.X, li.dY, "square", mean, stat)
        torch.cuda.synchronize()
        assert rel_frob(stat.cpu().numpy(), st.sum_g2) <= FROB_TOL
    assert rel_frob(pe.pe_token_sqstats(li.X, li.dY).cpu().numpy(), tok) <= FROB_TOL
    assert pe.pe_get_async_status(DEV) == (0, 0)


@pytest.mark.parametrize("B,T,d_in,d_out", [(5, 200, 136, 264), (40, 96, 384, 256), (3, 2000, 264, 520), (7, 128, 256, 512)])
def test_register_mean_kernel_at_any_sequence_length(B, T, d_in, d_out):
    """Long sequences normally keep sum_b G_b in tensor memory; the 256 x 128 kernel with both running
    sums in registers must give the same statistics when forced."""
    pe.pe_set_path(pe.PATH_TENSOR_NARROW)
    li = inputs.gaussian_layer(B, T, d_in, d_out, seed=500 + T, device=DEV)
    check_all(li, phis=("square", "sign"), token=False)
    assert pe.pe_last_path() == pe.PATH_TENSOR


@pytest.mark.parametrize("B,T,d_in,d_out", [(5, 200, 136, 264), (40, 96, 384, 256), (3, 2000, 264, 520), (33, 300, 776, 264),
                                            (9, 48, 320, 192), (1, 1000, 200, 128), (70, 64, 8, 8)])
def test_three_statistics_on_the_wide_tile(B, T, d_in, d_out):
    """The one-pass mean + square + sign kernel on the 256 x 192 tile (two thirds of sum_b G_b in tensor memory,
    a third in registers), forced on shapes with ragged tiles, one and many examples per block, split batches."""
    from parity_util import FROB_TOL, assert_entries_close, check_sign, oracle_on, rel_frob
    pe.pe_set_path(pe.PATH_TENSOR_WIDE)
    li = inputs.heterogeneous_layer(B, T, d_in, d_out, seed=1700 + B, device=DEV, with_weights=False)
    outs = [torch.full((d_out, d_in), float("nan"), device=DEV) for _ in range(3)]
    launches0 = pe.pe_launch_count()
    pe.pe_linear_stats_all(li.X, li.dY, *outs)
    torch.cuda.synchronize()
    assert pe.pe_get_async_status(DEV) == (0, 0) and pe.pe_last_path() == pe.PATH_TENSOR
    assert pe.pe_launch_count() - launches0 <= 2
    mean, sq, sgn = (o.cpu().numpy() for o in outs)
    assert np.isfinite(mean).all() and np.isfinite(sq).all() and np.isfinite(sgn).all()
    st, _ = oracle_on(li)
    assert rel_frob(mean, st.sum_g) <= FROB_TOL and rel_frob(sq, st.sum_g2) <= FROB_TOL
    assert_entries_close(mean, st.sum_g, "sum_b G_b")
    assert_entries_close(sq, st.sum_g2, "sum_b G_b^2")
    check_sign(sgn, st)


def test_wide_tile_structured_inputs_catch_layout_mistakes():
    """The 256 x 192 tile loads X in 64-byte rows with the 64-byte swizzle.  Distinct small integers per
    (token, feature), exactly representable in bf16: a wrong swizzle, stride or column offset of that
    layout changes results by whole numbers.  d_in = 400 spans three 192-column tiles, the last ragged."""
    pe.pe_set_path(pe.PATH_TENSOR_WIDE)
    B, T, d_in, d_out = 3, 144, 400, 264
    t = torch.arange(T, dtype=torch.float32).view(1, T, 1)
    X = ((t % 5) - 2 + (torch.arange(d_in).view(1, 1, d_in) % 13 - 6) + torch.arange(B).view(B, 1, 1)).to(torch.bfloat16)
    dY = ((t % 3) - 1 + (torch.arange(d_out).view(1, 1, d_out) % 11 - 5) * 0.5 - torch.arange(B).view(B, 1, 1)).to(torch.bfloat16)
    li = inputs.LayerInputs("structured", X.to(DEV).contiguous(), dY.to(DEV).contiguous())
    rep = check_all(li, phis=("square", "sign"), token=False, tol=1e-6)
    assert pe.pe_last_path() == pe.PATH_TENSOR
    assert rep["sign_disagreements"] == 0


@pytest.mark.parametrize("B,T,d_in,d_out", [(5, 200, 136, 264), (40, 96, 384, 256), (3, 2000, 264, 520), (7, 128, 192, 512),
                                            (9, 16, 320, 192), (2, 1, 64, 72), (70, 48, 8, 8), (33, 300, 776, 264)])
def test_wide_tile_kernel_at_any_shape(B, T, d_in, d_out):
    """The 256 x 192 kernel (both running sums in registers, 96 columns per thread), forced on shapes
    with ragged 192-column tiles, short and long sequences and split batches."""
    pe.pe_set_path(pe.PATH_TENSOR_WIDE)
    li = inputs.gaussian_layer(B, T, d_in, d_out, seed=1500 + T, device=DEV)
    check_all(li, phis=("square", "sign"), token=False)
    assert pe.pe_last_path() == pe.PATH_TENSOR


@pytest.mark.parametrize("B,T,d_in,d_out", [(5, 200, 136, 264), (64, 64, 512, 256), (3, 1000, 520, 776), (1, 257, 8, 8), (16, 512, 1024, 1024)])
def test_token_stat_fused_staged_and_oracle_agree(B, T, d_in, d_out):
    """The one-kernel per-token statistic, the two-pass one and the oracle give the same matrix; the two
    GPU routes round the squares to the same 11 significant bits (tf32 there, column-scaled half here),
    so they differ only by the order of the fp32 sums."""
    from parity_util import FROB_TOL, oracle_on, rel_frob
    li = inputs.heavy_tailed_layer(B, T, d_in, d_out, seed=1200 + B, device=DEV, with_weights=False)
    fused = torch.full((d_out, d_in), float("nan"), device=DEV)
    pe.pe_token_sqstats(li.X, li.dY, fused)
    assert pe.pe_last_path() == pe.PATH_TENSOR
    staged = pe.pe_token_sqstats_staged(li.X, li.dY)
    torch.cuda.synchronize()
    assert pe.pe_get_async_status(DEV) == (0, 0)
    f, s_ = fused.cpu().numpy(), staged.cpu().numpy()
    assert np.isfinite(f).all()
    assert rel_frob(f, s_) <= 1e-5
    if B * T * d_in * d_out <= 3e9:
        _, tok = oracle_on(li)
        assert rel_frob(f, tok) <= FROB_TOL


def test_staged_token_stat_keeps_every_column_accurate_over_a_wide_range_of_magnitudes():
    """The two-pass route stores the squares as IEEE half with one power-of-two scale per column.  Columns
    whose magnitudes differ by up to 2^50 (far outside half's range without the scales) must each come
    out right: the check is entry by entry, not a norm over the matrix."""
    from parity_util import oracle_on
    B, T, d_in, d_out = 6, 96, 136, 264
    li = inputs.gaussian_layer(B, T, d_in, d_out, seed=1300, device=DEV, with_weights=False)
    gen = torch.Generator().manual_seed(1301)
    kx = torch.randint(-20, 21, (d_in,), generator=gen).to(DEV)
    ky = torch.randint(-30, 11, (d_out,), generator=gen).to(DEV)
    li.X.mul_(torch.pow(2.0, kx.float()).to(torch.bfloat16))          # powers of two: exact in bf16
    li.dY.mul_(torch.pow(2.0, ky.float()).to(torch.bfloat16))
    staged = pe.pe_token_sqstats_staged(li.X, li.dY)
    assert pe.pe_last_path() == pe.PATH_TENSOR
    torch.cuda.synchronize()
    assert pe.pe_get_async_status(DEV) == (0, 0)
    _, tok = oracle_on(li)
    got = staged.cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all() and (tok > 0).all()
    assert np.max(np.abs(got - tok) / tok) <= 2e-3


@pytest.mark.parametrize("B,T,d_in,d_out,tensor_one_pass", [
    (5, 200, 136, 264, True),      # ragged tiles, ragged T
    (70, 96, 8, 8, True),          # one tile, batch split across blocks: partial sign counts are added
    (33, 300, 520, 264, True),     # odd slices
    (1, 1000, 256, 128, True),     # single example
    (2, 4100, 136, 264, True),     # very long sequences stay on the one-pass kernel
    (64, 256, 512, 2048, True),    # the benchmark layer, sampled below
    (9, 16, 320, 192, True),       # short sequences: the one-pass kernel on 32-token stages
    (21, 32, 136, 520, True),      # exactly one short stage per example
    (130, 32, 264, 392, True),     # many short sequences, batch split
    (2, 1, 64, 72, True),          # rank-one gradients
    (21, 64, 136, 520, True),      # half-filled stages
])
def test_three_statistics_in_one_pass(B, T, d_in, d_out, tensor_one_pass):
    """pe_linear_stats_all: sum_b G_b, sum_b G_b^2 and sum_b sign(G_b) from one pass over the examples, against
    the oracle (full comparison on the small shapes, sampled rows x columns on the benchmark layer)."""
    from parity_util import FROB_TOL, boundary_and_random, check_sign, oracle_on, rel_frob
    li = inputs.heterogeneous_layer(B, T, d_in, d_out, seed=1400 + B, device=DEV, with_weights=False)
    outs = [torch.full((d_out, d_in), float("nan"), device=DEV) for _ in range(3)]
    launches0 = pe.pe_launch_count()
    pe.pe_linear_stats_all(li.X, li.dY, *outs)
    torch.cuda.synchronize()
    assert pe.pe_get_async_status(DEV) == (0, 0)
    if tensor_one_pass:
        assert pe.pe_last_path() == pe.PATH_TENSOR
        assert pe.pe_launch_count() - launches0 <= 2            # the statistics kernel, plus the zeroing kernel when split
    mean, sq, sgn = (o.cpu().numpy() for o in outs)
    assert np.isfinite(mean).all() and np.isfinite(sq).all() and np.isfinite(sgn).all()
    if B * T * d_in * d_out <= 3e9:
        st, _ = oracle_on(li)
    else:
        rows, cols = boundary_and_random(d_out, 40, 11), boundary_and_random(d_in, 24, 12)
        st, _ = oracle_on(inputs.gather_columns(li, rows, cols))
        mean, sq, sgn = (a[np.asarray(rows)][:, np.asarray(cols)] for a in (mean, sq, sgn))
    assert rel_frob(mean, st.sum_g) <= FROB_TOL
    assert rel_frob(sq, st.sum_g2) <= FROB_TOL
    check_sign(sgn, st)
    # and the same numbers as the two calls it replaces (signs can differ only where an accumulator is within
    # rounding of zero: the two kernels use different tile widths)
    m2, s2 = pe.pe_linear_stats(li.X, li.dY, "square")
    _, g2 = pe.pe_linear_stats(li.X, li.dY, "sign", None, torch.empty((d_out, d_in), device=DEV))
    torch.cuda.synchronize()
    assert float((g2 != outs[2]).float().mean()) <= 1e-3
    assert rel_frob(outs[0].cpu().numpy(), m2.cpu().numpy()) <= 1e-5 and rel_frob(outs[1].cpu().numpy(), s2.cpu().numpy()) <= 1e-5


@pytest.mark.parametrize("B,T,d_in,d_out,phi", [(11, 200, 136, 264, "square"), (70, 96, 8, 8, "sign"), (6, 4100, 136, 264, "square"),
                                                  (9, 16, 320, 192, "sign"), (5, 300, 264, 136, "identity")])
def test_accumulating_over_micro_batches_gives_the_statistics_of_the_batch(B, T, d_in, d_out, phi):
    """pe_linear_stats_accumulate over three unequal micro-batches (one of them empty) into outputs zeroed once,
    against the oracle on the whole batch."""
    from parity_util import FROB_TOL, check_sign, oracle_on, rel_frob
    li = inputs.gaussian_layer(B, T, d_in, d_out, seed=1600 + B, device=DEV)
    mean = torch.zeros((d_out, d_in), device=DEV)
    stat = torch.zeros((d_out, d_in), device=DEV)
    cuts = [0, B // 3, B // 3, B - 2, B]                     # micro-batches of B//3, 0, B-2-B//3 and 2 examples
    for lo, hi in zip(cuts[:-1], cuts[1:]):
        pe.pe_linear_stats_accumulate(li.X[lo:hi].clone(), li.dY[lo:hi].clone(), phi, mean, stat)
    torch.cuda.synchronize()
    assert pe.pe_get_async_status(DEV) == (0, 0)
    st, _ = oracle_on(li)
    assert rel_frob(mean.cpu().numpy(), st.sum_g) <= FROB_TOL
    if phi == "square":
        assert rel_frob(stat.cpu().numpy(), st.sum_g2) <= FROB_TOL
    elif phi == "sign":
        check_sign(stat.cpu().numpy(), st)
    else:
        assert rel_frob(stat.cpu().numpy(), st.sum_g) <= FROB_TOL
    # a single output works too, and what is already there is kept
    only = torch.full((d_out, d_in), 3.0, device=DEV)
    pe.pe_linear_stats_accumulate(li.X, li.dY, phi, None, only)
    torch.cuda.synchronize()
    ref = {"square": st.sum_g2, "sign": st.sum_sign, "identity": st.sum_g}[phi]
    if phi == "sign":
        check_sign(only.cpu().numpy() - 3.0, st)
    else:
        assert rel_frob(only.cpu().numpy().astype(np.float64) - 3.0, ref) <= FROB_TOL + 1e-4


@pytest.mark.parametrize("B,T,d_in,d_out", [(5, 200, 136, 264), (70, 48, 8, 8), (33, 300, 520, 264), (9, 16, 320, 192),
                                              (3, 2000, 264, 520), (64, 256, 512, 2048)])
def test_per_example_squared_norms(B, T, d_in, d_out):
    """pe_example_sqnorms against the oracle (on the benchmark layer: on a sample of the examples)."""
    li = inputs.heterogeneous_layer(B, T, d_in, d_out, seed=1800 + B, device=DEV, with_weights=False)
    norms = torch.full((B,), float("nan"), device=DEV)
    pe.pe_example_sqnorms(li.X, li.dY, norms)
    torch.cuda.synchronize()
    assert pe.pe_last_path() == pe.PATH_TENSOR and pe.pe_get_async_status(DEV) == (0, 0)
    got = norms.cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    picked = list(range(B)) if B * T * d_in * d_out <= 3e9 else [0, 1, B // 2, B - 1]      # the oracle is slow: sample examples
    want = oracle.example_sqnorms(inputs.to_numpy_bits(li.X[picked]), inputs.to_numpy_bits(li.dY[picked]))
    assert np.max(np.abs(got[picked] - want) / want) <= 2e-3          # every example, not a norm over the batch
    # the norms add up to the sum of all entries of sum_b G_b^2
    _, sq = pe.pe_linear_stats(li.X, li.dY, "square")
    assert abs(float(sq.double().sum()) - got.sum()) <= 1e-4 * got.sum()
    # a second call overwrites, it does not add
    pe.pe_example_sqnorms(li.X, li.dY, norms)
    torch.cuda.synchronize()
    assert np.max(np.abs(norms.cpu().numpy() - got) / got) <= 1e-5


def test_three_statistics_of_an_empty_batch_are_zero():
    outs = [torch.full((72, 64), float("nan"), device=DEV) for _ in range(3)]
    X = torch.empty((0, 128, 64), dtype=torch.bfloat16, device=DEV)
    dY = torch.empty((0, 128, 72), dtype=torch.bfloat16, device=DEV)
    pe.pe_linear_stats_all(X, dY, *outs)
    torch.cuda.synchronize()
    assert all(bool((o == 0).all()) for o in outs)


def test_three_statistics_need_all_three_outputs():
    li = inputs.gaussian_layer(2, 128, 64, 64, seed=1, device=DEV)
    out = torch.empty((64, 64), device=DEV)
    lib = pe.load_library()
    assert lib.pe_linear_stats_all(li.X.data_ptr(), li.dY.data_ptr(), 2, 128, 64, 64, out.data_ptr(), out.data_ptr(), None, None) == 1


@pytest.mark.parametrize("B,T", [(2, 64), (3, 16), (5, 80)])
def test_launches_of_several_waves_full_comparison(B, T):
    """10 pair rows x 9-17 column tiles: more thread-block pairs than the GPU holds at once, so the order in which
    tiles are handed out matters, and the host picks it per launch (bands of 1, 6 or 8 pair rows here, depending on
    the tile width and the batch split); every output entry is compared."""
    d_in, d_out = 2112, 2560
    li = inputs.gaussian_layer(B, T, d_in, d_out, seed=77 + B, device=DEV)
    check_all(li, phis=("identity", "square", "sign"), token=False)
    assert pe.pe_last_path() == pe.PATH_TENSOR
    st = oracle.linear_stats(inputs.to_numpy_bits(li.X), inputs.to_numpy_bits(li.dY), small_rel=SIGN_REL)
    outs = [torch.full((d_out, d_in), float("nan"), device=DEV) for _ in range(3)]
    pe.pe_linear_stats_all(li.X, li.dY, *outs)
    stat_only = torch.full((d_out, d_in), float("nan"), device=DEV)
    pe.pe_linear_stats(li.X, li.dY, "square", None, stat_only)
    torch.cuda.synchronize()
    mean, sq, sg = (o.cpu().numpy() for o in outs)
    assert np.isfinite(mean).all() and np.isfinite(sq).all() and np.isfinite(sg).all()
    assert rel_frob(mean, st.sum_g) <= 1e-5 and rel_frob(sq, st.sum_g2) <= 1e-5
    assert rel_frob(stat_only.cpu().numpy(), st.sum_g2) <= 1e-5
    check_sign(sg, st)


@pytest.mark.parametrize("exponent", [-10, -60, -68, -72])
def test_sign_statistic_of_tiny_denormal_and_zero_gradients(exponent):
    """Gradients as small as fp32 denormals keep their sign, and exact zeros of either sign count as zero: every
    example repeats one token of entries +-2^e (bf16 holds them exactly), so G_b = +-T 2^(2e), down to 2^-139; a block
    of zero columns in dY with negative X next to it gives -0 products and +0 sums."""
    B, T, d_in, d_out = 5, 32, 264, 136
    g = torch.Generator().manual_seed(17 - exponent)
    sx = (torch.randint(0, 2, (B, 1, d_in), generator=g) * 2 - 1).float()
    sy = (torch.randint(0, 2, (B, 1, d_out), generator=g) * 2 - 1).float()
    sy[:, :, 40:56] = 0.0                              # zero gradient columns: G_b[40:56, :] = +-0
    X = (sx * 2.0 ** exponent).expand(B, T, d_in).to(torch.bfloat16).contiguous().to(DEV)
    dY = (sy * 2.0 ** exponent).expand(B, T, d_out).to(torch.bfloat16).contiguous().to(DEV)
    li = inputs.LayerInputs("tiny", X, dY)
    st = oracle.linear_stats(inputs.to_numpy_bits(X), inputs.to_numpy_bits(dY))
    want = np.einsum("bo,bi->oi", sy[:, 0, :].numpy(), sx[:, 0, :].numpy())
    assert np.array_equal(st.sum_sign, want)           # the oracle keeps every sign, whatever the magnitude
    for path in (pe.PATH_TENSOR, pe.PATH_SIMT):
        pe.pe_set_path(path)
        _, stat = gpu_stats(li, "sign")
        assert pe.pe_last_path() == path
        assert np.array_equal(stat, want), f"path {path}: {int((stat != want).sum())} entries differ"
        outs = [torch.full((d_out, d_in), float("nan"), device=DEV) for _ in range(3)]
        pe.pe_linear_stats_all(X, dY, *outs)
        torch.cuda.synchronize()
        assert np.array_equal(outs[2].cpu().numpy(), want)
        assert np.all(outs[2].cpu().numpy()[40:56] == 0)


def test_heavy_tailed_and_heterogeneous_small():
    check_all(inputs.heavy_tailed_layer(12, 128, 256, 384, seed=41, device=DEV))
    check_all(inputs.heterogeneous_layer(20, 64, 128, 256, seed=42, device=DEV))


def test_unsplit_schedule_is_bit_reproducible():
    li = inputs.gaussian_layer(4, 128, 2048, 2048, seed=43, device=DEV)     # 256 tiles >= SM count: no batch split
    a = gpu_stats(li, "square")
    b = gpu_stats(li, "square")
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])


def test_config2_full_size_sampled_outputs():
    li = inputs.config2(DEV)
    rows = boundary_and_random(2048, 40, 1)
    cols = boundary_and_random(512, 32, 2)
    rep = check_all(li, rows, cols, bench_calls=True)
    rep.pop("oracle_stats", None)
    assert pe.pe_last_path() == pe.PATH_TENSOR
    print("config2", rep)


def test_config4_full_size_sampled_outputs():
    li = inputs.config4(DEV)
    rows = boundary_and_random(8192, 24, 3)
    cols = boundary_and_random(2048, 24, 4)
    rep = check_all(li, rows, cols, bench_calls=True)
    st = rep.pop("oracle_stats")
    print("config4", rep)
    # ... followed by the MicroSignSGD step on the fp32 master weights (beta = 0.9, lr = 3.47e-3, m_0 = 0), with the
    # bf16 copy: once as the separate update kernel on the sign statistic, once fused into the statistics kernel
    B, d_out, d_in = li.shape[0], 8192, 2048
    kw = dict(lr=3.47e-3, beta=0.9)
    pick = lambda t: t.float().cpu().numpy().astype(np.float64)[np.ix_(rows, cols)]
    W0 = pick(li.W)
    th_ref, m_ref = oracle.microsignsgd_step(W0, np.zeros_like(W0), st.sum_sign, B, **kw)
    slack = 2.0 * st.n_small / B * (1.0 - kw["beta"])            # what the examples below the sign threshold may move m by
    sgn = torch.empty((d_out, d_in), device=DEV)
    pe.pe_linear_stats(li.X, li.dY, "sign", None, sgn)
    for fused in (False, True):
        th, m = li.W.clone(), torch.zeros((d_out, d_in), device=DEV)
        lp = torch.empty((d_out, d_in), dtype=torch.bfloat16, device=DEV)
        if fused:
            ws = torch.empty(pe.pe_linear_fused_workspace_bytes(d_in, d_out), dtype=torch.uint8, device=DEV)
            pe.pe_linear_microsignsgd_step(li.X, li.dY, th, m, theta_lp=lp, out_sign=sgn, workspace=ws, **kw)
        else:
            pe.microsignsgd_step(th, m, sgn, B, theta_lp=lp, **kw)
        torch.cuda.synchronize()
        assert np.all(np.abs(pick(m) - m_ref) <= slack + 1e-7), fused
        assert np.all(np.abs(pick(th) - th_ref) <= kw["lr"] * slack + 1e-7), fused
        exact = st.n_small == 0
        # the update itself (fp32 master weights hold it to about 1e-4 of its size), at the tolerance for updated parameters
        from parity_util import FROB_TOL
        assert rel_frob((pick(th) - W0)[exact], (th_ref - W0)[exact]) <= FROB_TOL
        assert torch.equal(lp, th.to(torch.bfloat16))
        del th, m, lp
    assert pe.pe_get_async_status(DEV) == (0, 0)
    del li, sgn
    torch.cuda.empty_cache()


@pytest.mark.parametrize("d", inputs.SWEEP_D)
@pytest.mark.parametrize("B,T", inputs.SWEEP_BT)
def test_config5_points_sampled_outputs(B, T, d):
    li = inputs.config5_point(B, T, d, DEV)
    rows = boundary_and_random(d, 16, 5)
    cols = boundary_and_random(d, 16, 6)
    check_all(li, rows, cols)
    del li
    torch.cuda.empty_cache()


def test_sign_counters_force_a_batch_split_beyond_32767_examples_per_block():
    """The one-pass kernel counts sign(G_b) + 1 in 16-bit halves of a register, good for 32767 examples per
    block; with more examples than 16 x 32767 the host must split the batch further than it otherwise would."""
    B, T, d = 16 * 32767 + 40, 33, 8
    li = inputs.gaussian_layer(B, T, d, d, seed=123, device=DEV)
    outs = [torch.full((d, d), float("nan"), device=DEV) for _ in range(3)]
    pe.pe_linear_stats_all(li.X, li.dY, *outs)
    torch.cuda.synchronize()
    assert pe.pe_last_path() == pe.PATH_TENSOR and pe.pe_get_async_status(DEV) == (0, 0)
    from parity_util import check_sign, oracle_on, rel_frob, FROB_TOL
    st, _ = oracle_on(li)
    assert rel_frob(outs[0].cpu().numpy(), st.sum_g) <= FROB_TOL and rel_frob(outs[1].cpu().numpy(), st.sum_g2) <= FROB_TOL
    check_sign(outs[2].cpu().numpy(), st)
    assert float(outs[2].abs().max()) <= B


def test_staged_token_stat_requires_workspace():
    li = inputs.gaussian_layer(4, 64, 64, 64, seed=44, device=DEV)
    out = torch.empty((64, 64), device=DEV)
    lib = pe.load_library()
    st = lib.pe_token_sqstats_staged(li.X.data_ptr(), li.dY.data_ptr(), 4, 64, 64, 64, out.data_ptr(), None, 0, None)
    assert st == 9      # PE_ERR_WORKSPACE
