"""CPU-only checks of the C-ABI boundary: the library builds, loads without a GPU, exports every
function the header declares, and its host-side helpers behave."""
import ctypes
import os
import re

import pytest

import paper_2510_00236_b200 as pe
from paper_2510_00236_b200 import build as pe_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    pe_build.build_library()
    return pe.load_library()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "pestats.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = re.findall(r"\b([a-z_0-9]+)\s*\([^;{]*\)\s*;", text)
    return sorted(set(names))


def test_header_functions_are_all_exported_and_bound(lib):
    declared = _declared_functions()
    assert "pe_linear_stats" in declared and "microsignsgd_step" in declared
    for name in declared:
        assert hasattr(lib, name), f"{name} declared in pestats.h but not exported"
    assert sorted(pe.EXPORTED_SYMBOLS) == declared
    for name in declared:
        assert hasattr(pe, name), f"binding lacks {name}"


def test_status_strings_and_path_switch(lib):
    assert pe.pe_status_string(0) == "PE_OK"
    assert pe.pe_status_string(8) == "PE_ERR_TIMEOUT"
    assert pe.pe_status_string(9) == "PE_ERR_WORKSPACE"
    assert pe.pe_status_string(1234) == "PE_ERR_UNKNOWN"
    prev = pe.pe_set_path(pe.PATH_SIMT)
    assert pe.pe_set_path(prev) == pe.PATH_SIMT
    assert pe.pe_set_path(77) == -1


def test_host_side_validation_needs_no_gpu(lib):
    # argument errors are reported before any CUDA call
    assert lib.pe_linear_stats(None, None, 1, 1, 8, 8, 1, None, None, None) == 1          # PE_ERR_NULL
    buf = ctypes.create_string_buffer(4096)
    p = ctypes.addressof(buf)
    p16 = (p + 15) & ~15
    assert lib.pe_linear_stats(p16, p16, 1, 1, 8, 8, 1, None, None, None) == 1            # both outputs NULL
    assert lib.pe_linear_stats(p16, p16, -1, 1, 8, 8, 1, p16, p16, None) == 2             # PE_ERR_DIM
    assert lib.pe_linear_stats(None, None, 1, 1, 0, 8, 1, p16, p16, None) == 2
    assert lib.pe_linear_stats(p16 + 2, p16, 1, 1, 8, 8, 1, p16, p16, None) == 3          # PE_ERR_ALIGN
    assert lib.pe_linear_stats(p16, p16, 1, 1, 8, 8, 7, p16, p16, None) == 5              # PE_ERR_PHI
    assert lib.microadam_step(p16, None, p16, p16, p16, p16, 4, 0, 1.0, 1e-3, 0.9, 0.99, 1e-8, 0, 0.0, 1, None) == 2
    assert lib.microadam_step(p16, None, p16, p16, p16, p16, 4, 1, 1.0, 1e-3, 0.9, 0.99, 1e-8, 0, 0.0, 0, None) == 2
    assert lib.microsignsgd_step(p16, None, None, p16, 4, 1, 1e-3, 0.9, 0.0, None) == 1


def test_workspace_size_formula(lib):
    prev = pe.pe_set_path(pe.PATH_AUTO)
    try:
        # column maxima (4 B per column), then the squares as half (2 B each); every part a multiple of 256 B
        assert pe.pe_token_sqstats_staged_workspace_bytes(64, 256, 512, 2048) == (512 + 2048) * 4 + 64 * 256 * (512 + 2048) * 2
        assert pe.pe_token_sqstats_staged_workspace_bytes(30, 10, 8, 8) == 256 + 4864 + 4864   # 64 B and 4800 B rounded up
        assert pe.pe_token_sqstats_staged_workspace_bytes(3, 5, 8, 8) == 0                  # too few rows for bf16 squares
        assert pe.pe_token_sqstats_staged_workspace_bytes(3, 5, 7, 8) == 0                  # SIMT shape: no workspace
        pe.pe_set_path(pe.PATH_SIMT)
        assert pe.pe_token_sqstats_staged_workspace_bytes(64, 256, 512, 2048) == 0
    finally:
        pe.pe_set_path(prev)


def test_other_workspace_sizes_and_mode_switches(lib):
    prev = pe.pe_set_path(pe.PATH_AUTO)
    try:
        # packed batches: the zero-padded last partial 16-token group of every sequence, X's then dY's, bf16
        assert pe.pe_linear_stats_ragged_workspace_bytes(10, 64, 128) == 10 * 16 * 64 * 2 + 10 * 16 * 128 * 2
        assert pe.pe_linear_stats_ragged_workspace_bytes(3, 8, 8) == 768 + 768          # 3 * 16 * 8 * 2 = 768, already a multiple of 256
        assert pe.pe_linear_stats_ragged_workspace_bytes(3, 7, 8) == 0                  # SIMT shape: no workspace
        assert pe.pe_linear_stats_ragged_workspace_bytes(0, 8, 8) == 0
        # fused update: one counter per thread block of the widest grid (256 x 128 tiles, two blocks per pair)
        assert pe.pe_linear_fused_workspace_bytes(2048, 8192) == 2 * 32 * 16 * 4
        assert pe.pe_linear_fused_workspace_bytes(8, 8) == 256
        # fp8 staging: one byte per element when both widths are multiples of 16, the half layout otherwise
        assert pe.pe_token_sqstats_fp8_workspace_bytes(64, 256, 512, 2048) == (512 + 2048) * 4 + 64 * 256 * (512 + 2048)
        assert pe.pe_token_sqstats_fp8_workspace_bytes(64, 256, 520, 2048) == pe.pe_token_sqstats_staged_workspace_bytes(64, 256, 520, 2048)
    finally:
        pe.pe_set_path(prev)
    prev = pe.pe_set_fused_update(pe.FUSED_ALWAYS)
    assert pe.pe_set_fused_update(prev) == pe.FUSED_ALWAYS
    assert pe.pe_set_fused_update(9) == -1
    assert pe.pe_set_path(pe.PATH_TENSOR_WIDE) == pe.PATH_AUTO and pe.pe_set_path(pe.PATH_AUTO) == pe.PATH_TENSOR_WIDE


def test_new_entry_points_validate_on_the_host(lib):
    buf = ctypes.create_string_buffer(8192)
    p16 = (ctypes.addressof(buf) + 255) & ~255
    vp, ll, f = ctypes.c_void_p, ctypes.c_longlong, ctypes.c_float
    # packed batches: offsets required, sizes checked, outputs required
    assert lib.pe_linear_stats_ragged(p16, p16, None, 2, ll(32), 8, 8, 1, p16, p16, p16, 4096, None) == 1
    assert lib.pe_linear_stats_ragged(p16, p16, p16, -1, ll(32), 8, 8, 1, p16, p16, p16, 4096, None) == 2
    assert lib.pe_linear_stats_ragged(p16, p16, p16, 2, ll(1 << 31), 8, 8, 1, p16, p16, p16, 4096, None) == 2
    assert lib.pe_linear_stats_ragged(p16, p16, p16, 2, ll(32), 8, 8, 1, None, None, p16, 4096, None) == 1
    assert lib.pe_linear_stats_ragged(p16, p16, p16, 2, ll(32), 8, 8, 9, p16, p16, p16, 4096, None) == 5
    # clipped sum: negative or NaN threshold, missing norms buffer
    assert lib.pe_linear_clipped_sum(p16, p16, 2, 4, 8, 8, f(-1.0), p16, 0, p16, None) == 2
    assert lib.pe_linear_clipped_sum(p16, p16, 2, 4, 8, 8, f(float("nan")), p16, 0, p16, None) == 2
    assert lib.pe_linear_clipped_sum(p16, p16, 2, 4, 8, 8, f(1.0), None, 0, p16, None) == 1
    # statistics + update: parameters required, step and variant checked, a variance needs two examples
    adam = (1, f(1.0), f(1e-3), f(0.9), f(0.99), f(1e-8), 0, f(0.0))
    assert lib.pe_linear_microadam_step(p16, p16, 2, 4, 8, 8, None, None, p16, p16, None, None, *adam, 1, None, 0, None) == 1
    assert lib.pe_linear_microadam_step(p16, p16, 2, 4, 8, 8, p16, None, p16, p16, None, None, *adam, 0, None, 0, None) == 2
    assert lib.pe_linear_microadam_step(p16, p16, 2, 4, 8, 8, p16, None, p16, p16, None, None, 7, *adam[1:], 1, None, 0, None) == 5
    assert lib.pe_linear_microadam_step(p16, p16, 1, 4, 8, 8, p16, None, p16, p16, None, None, 2, *adam[1:], 1, None, 0, None) == 2
    assert lib.pe_linear_microsignsgd_step(p16, p16, 0, 4, 8, 8, p16, None, p16, None, f(1e-3), f(0.9), f(0.0), None, 0, None) == 2


def test_cpu_tensors_are_rejected_loudly():
    import torch
    X = torch.zeros(1, 2, 8, dtype=torch.bfloat16)
    with pytest.raises(pe.PestatsError):
        pe.pe_linear_stats(X, X, "square")


def _wave_columns(pairs_m, tiles_n, tile_cols, band, slices, slots):
    """Operand columns the waves of a launch stream: thread-block pairs start in index order, `slots` at a time, one
    batch slice after the other; within a slice consecutive pairs walk `band` pair rows, then the next column tile."""
    order = []
    for first in range(0, pairs_m, band):
        rows = min(band, pairs_m - first)
        order += [(first + r, n) for n in range(tiles_n) for r in range(rows)]
    units = (order * slices)[: 1 << 14]
    total = 0
    for w in range(0, len(units), slots):
        wave = units[w:w + slots]
        total += 256 * len({m for m, _ in wave}) + tile_cols * len({n for _, n in wave})
    return total


def test_tile_order_band_follows_the_wave_model(lib):
    band = pe.pe_tile_order_band
    # out-of-range arguments
    assert band(0, 256, 192, 1, 148) == 0 and band(256, 256, 100, 1, 148) == 0 and band(256, 256, 192, 0, 148) == 0
    # launches of a single wave keep the default: 8 pair rows, or all of them
    assert band(512, 2048, 192, 3, 148) == 8 and band(1024, 1024, 256, 1, 148) == 4
    # the large layer (32 pair rows x 11 column tiles of 192, five batch slices): bands of one pair row
    assert band(2048, 8192, 192, 5, 148) == 1
    # 16 x 22 tiles: the default is the cheapest
    assert band(4096, 4096, 192, 1, 148) == 8
    # whatever it returns costs, by the model, no more than the default, and is within 3 % of the best candidate
    for (d_in, d_out, cols, slices) in [(2048, 8192, 192, 5), (2048, 8192, 256, 2), (2112, 2560, 192, 1), (2112, 2560, 256, 1),
                                        (512, 32768, 192, 1), (8192, 2048, 192, 1), (4096, 4096, 256, 2), (1152, 4096, 128, 1)]:
        pairs_m, tiles_n = -(-d_out // 256), -(-d_in // cols)
        got = band(d_in, d_out, cols, slices, 148)
        assert 1 <= got <= pairs_m
        cost = {b: _wave_columns(pairs_m, tiles_n, cols, min(b, pairs_m), slices, 74) for b in (1, 2, 3, 4, 6, 8, 12, 16)}
        mine = _wave_columns(pairs_m, tiles_n, cols, got, slices, 74)
        assert mine <= cost[8]
        assert mine <= min(cost.values()) / 0.97 + 1
