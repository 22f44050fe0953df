"""ctypes binding of ``libpestats.so``: same names as the C ABI, argument marshalling only.

Tensors are passed as raw device pointers (``tensor.data_ptr()``) together with the current CUDA
stream; every computation happens in the library's kernels.  There is no fallback: if the library
has not been built, or a call returns an error status, a :class:`PestatsError` is raised.
"""
from __future__ import annotations

import ctypes
import os

import torch

__all__ = [
    "PestatsError", "PHI_IDENTITY", "PHI_SQUARE", "PHI_SIGN", "PATH_AUTO", "PATH_SIMT", "PATH_TENSOR", "PATH_TENSOR_NARROW", "PATH_TENSOR_WIDE",
    "EXPORTED_SYMBOLS", "library_path", "load_library", "pe_linear_stats", "pe_linear_stats_f32",
    "pe_token_sqstats", "pe_token_sqstats_f32", "pe_token_sqstats_staged", "pe_token_sqstats_staged_workspace_bytes",
    "microadam_step", "microsignsgd_step", "pe_status_string", "pe_get_async_status", "pe_set_path", "pe_last_path",
    "pe_launch_count", "pe_reset_launch_count", "pe_token_sqstats_static", "STATIC_SCRATCH_BYTES",
    "microadam_family_step", "ADAM_VARIANTS", "pe_linear_stats_all", "pe_linear_stats_accumulate", "pe_example_sqnorms",
    "pe_linear_stats_ragged", "pe_linear_stats_ragged_workspace_bytes", "pe_example_sqnorms_ragged", "pe_linear_clipped_sum",
    "pe_linear_microadam_step", "pe_linear_microadam_step_f32", "pe_linear_microsignsgd_step", "pe_linear_fused_workspace_bytes",
    "pe_token_sqstats_fp8", "pe_token_sqstats_fp8_workspace_bytes", "pe_set_wait_limit_cycles", "pe_tile_order_band",
    "pe_set_fused_update", "FUSED_AUTO", "FUSED_ALWAYS", "FUSED_NEVER",
]

PHI_IDENTITY, PHI_SQUARE, PHI_SIGN = 0, 1, 2
PATH_AUTO, PATH_SIMT, PATH_TENSOR, PATH_TENSOR_NARROW, PATH_TENSOR_WIDE = 0, 1, 2, 3, 4
FUSED_AUTO, FUSED_ALWAYS, FUSED_NEVER = 0, 1, 2      # pe_fused_mode_t
_PHI_NAMES = {"identity": PHI_IDENTITY, "square": PHI_SQUARE, "sign": PHI_SIGN}

# every symbol include/pestats.h declares
EXPORTED_SYMBOLS = [
    "pe_linear_stats", "pe_linear_stats_f32", "pe_token_sqstats", "pe_token_sqstats_f32", "pe_token_sqstats_staged",
    "pe_token_sqstats_staged_workspace_bytes", "microadam_step", "microsignsgd_step", "pe_status_string",
    "pe_get_async_status", "pe_set_path", "pe_last_path", "pe_launch_count", "pe_reset_launch_count",
    "pe_token_sqstats_static", "microadam_family_step", "pe_linear_stats_all", "pe_linear_stats_accumulate", "pe_example_sqnorms",
    "pe_linear_stats_ragged", "pe_linear_stats_ragged_workspace_bytes", "pe_example_sqnorms_ragged", "pe_linear_clipped_sum",
    "pe_linear_microadam_step", "pe_linear_microadam_step_f32", "pe_linear_microsignsgd_step", "pe_linear_fused_workspace_bytes",
    "pe_token_sqstats_fp8", "pe_token_sqstats_fp8_workspace_bytes", "pe_set_wait_limit_cycles", "pe_tile_order_band",
    "pe_set_fused_update",
]
ADAM_VARIANTS = {"adam": 0, "microadam": 1, "microadam_var": 2, "microadam_msq": 3}      # pe_adam_variant_t
STATIC_SCRATCH_BYTES = 32 * 1024 * 1024      # PE_STATIC_SCRATCH_BYTES of pestats.h

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "csrc", "libpestats.so")
_lib = None


class PestatsError(RuntimeError):
    """A libpestats call failed; ``status`` holds the pe_status_t code."""

    def __init__(self, fn: str, status: int, text: str):
        super().__init__(f"{fn} failed: {text} ({status})")
        self.status = status


def library_path() -> str:
    return _LIB_PATH


def load_library() -> ctypes.CDLL:
    """Loads the in-tree CUDA library; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise PestatsError("load_library", -1,
                           f"{_LIB_PATH} not found; build it with `python -m paper_2510_00236_b200.build`")
    lib = ctypes.CDLL(_LIB_PATH)
    vp, i, f, ll, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_longlong, ctypes.c_size_t
    lib.pe_linear_stats.argtypes = [vp, vp, i, i, i, i, i, vp, vp, vp]
    lib.pe_linear_stats_f32.argtypes = [vp, vp, i, i, i, i, i, vp, vp, vp]
    lib.pe_linear_stats_all.argtypes = [vp, vp, i, i, i, i, vp, vp, vp, vp]
    lib.pe_linear_stats_accumulate.argtypes = [vp, vp, i, i, i, i, i, vp, vp, vp]
    lib.pe_example_sqnorms.argtypes = [vp, vp, i, i, i, i, vp, vp]
    lib.pe_token_sqstats.argtypes = [vp, vp, i, i, i, i, vp, vp]
    lib.pe_linear_stats_ragged.argtypes = [vp, vp, vp, i, ll, i, i, i, vp, vp, vp, sz, vp]
    lib.pe_linear_stats_ragged_workspace_bytes.argtypes = [i, i, i]
    lib.pe_linear_stats_ragged_workspace_bytes.restype = sz
    lib.pe_example_sqnorms_ragged.argtypes = [vp, vp, vp, i, ll, i, i, vp, vp, sz, vp]
    lib.pe_linear_clipped_sum.argtypes = [vp, vp, i, i, i, i, f, vp, i, vp, vp]
    lib.pe_linear_microadam_step.argtypes = [vp, vp, i, i, i, i, vp, vp, vp, vp, vp, vp, i, f, f, f, f, f, i, f, i, vp, sz, vp]
    lib.pe_linear_microadam_step_f32.argtypes = [vp, vp, i, i, i, i, vp, vp, vp, vp, vp, vp, i, f, f, f, f, f, i, f, i, vp]
    lib.pe_linear_microsignsgd_step.argtypes = [vp, vp, i, i, i, i, vp, vp, vp, vp, f, f, f, vp, sz, vp]
    lib.pe_linear_fused_workspace_bytes.argtypes = [i, i]
    lib.pe_linear_fused_workspace_bytes.restype = sz
    lib.pe_token_sqstats_staged.argtypes = [vp, vp, i, i, i, i, vp, vp, sz, vp]
    lib.pe_token_sqstats_fp8.argtypes = [vp, vp, i, i, i, i, vp, vp, sz, vp]
    lib.pe_token_sqstats_fp8_workspace_bytes.argtypes = [i, i, i, i]
    lib.pe_token_sqstats_fp8_workspace_bytes.restype = sz
    lib.pe_token_sqstats_f32.argtypes = [vp, vp, i, i, i, i, vp, vp]
    lib.pe_token_sqstats_static.argtypes = [vp, vp, i, i, i, i, vp, vp]
    lib.pe_token_sqstats_staged_workspace_bytes.argtypes = [i, i, i, i]
    lib.pe_token_sqstats_staged_workspace_bytes.restype = sz
    lib.microadam_step.argtypes = [vp, vp, vp, vp, vp, vp, ll, i, f, f, f, f, f, i, f, i, vp]
    lib.microadam_family_step.argtypes = [vp, vp, vp, vp, vp, vp, ll, i, i, f, f, f, f, f, i, f, i, vp]
    lib.microsignsgd_step.argtypes = [vp, vp, vp, vp, ll, i, f, f, f, vp]
    lib.pe_status_string.argtypes = [i]
    lib.pe_status_string.restype = ctypes.c_char_p
    lib.pe_get_async_status.argtypes = [vp, ctypes.POINTER(ctypes.c_int)]
    lib.pe_set_path.argtypes = [i]
    lib.pe_set_fused_update.argtypes = [i]
    lib.pe_set_fused_update.restype = i
    lib.pe_set_wait_limit_cycles.argtypes = [ll]
    lib.pe_set_wait_limit_cycles.restype = i
    lib.pe_last_path.argtypes = []
    lib.pe_tile_order_band.argtypes = [ctypes.c_int] * 5
    lib.pe_tile_order_band.restype = ctypes.c_int
    lib.pe_launch_count.argtypes = []
    lib.pe_launch_count.restype = ll
    lib.pe_reset_launch_count.argtypes = []
    lib.pe_reset_launch_count.restype = None
    for name in ("pe_linear_stats", "pe_linear_stats_f32", "pe_linear_stats_all", "pe_linear_stats_accumulate", "pe_example_sqnorms", "pe_token_sqstats", "pe_token_sqstats_f32", "pe_token_sqstats_static",
                 "pe_token_sqstats_staged", "pe_token_sqstats_fp8",
                 "pe_linear_stats_ragged", "pe_example_sqnorms_ragged", "pe_linear_clipped_sum",
                 "pe_linear_microadam_step", "pe_linear_microadam_step_f32", "pe_linear_microsignsgd_step",
                 "microadam_step", "microadam_family_step", "microsignsgd_step", "pe_get_async_status", "pe_set_path", "pe_last_path"):
        getattr(lib, name).restype = i
    _lib = lib
    return lib


def pe_status_string(status: int) -> str:
    return load_library().pe_status_string(int(status)).decode()


def _check(fn: str, status: int):
    if status != 0:
        raise PestatsError(fn, status, pe_status_string(status))


def _stream(t: torch.Tensor) -> int:
    return torch.cuda.current_stream(t.device).cuda_stream


def _ptr(t):
    return None if t is None else t.data_ptr()


def _phi(phi) -> int:
    return _PHI_NAMES[phi] if isinstance(phi, str) else int(phi)


def _dev_ctx(t: torch.Tensor):
    if not t.is_cuda:
        raise PestatsError("binding", -1, "tensors must live on a CUDA device (there is no CPU path)")
    return torch.cuda.device(t.device)


def _io_check(X, dY, dtype):
    if X.dtype != dtype or dY.dtype != dtype:
        raise TypeError(f"X and dY must be {dtype}")
    if X.dim() != 3 or dY.dim() != 3 or X.shape[:2] != dY.shape[:2]:
        raise ValueError("X must be [B,T,d_in] and dY [B,T,d_out] with equal B and T")
    if not (X.is_contiguous() and dY.is_contiguous()):
        raise ValueError("X and dY must be contiguous")
    B, T, d_in = X.shape
    return B, T, d_in, dY.shape[2]


def _out_check(name, t, d_out, d_in):
    if t is not None and (t.dtype != torch.float32 or tuple(t.shape) != (d_out, d_in) or not t.is_contiguous()):
        raise ValueError(f"{name} must be a contiguous float32 [d_out, d_in] tensor")


def pe_linear_stats(X, dY, phi, out_mean=None, out_stat=None):
    """out_mean = sum_b G_b, out_stat = sum_b phi(G_b) with G_b = dY_b^T X_b (bf16 inputs).
    Buffers are allocated when both are omitted; returns (out_mean, out_stat)."""
    B, T, d_in, d_out = _io_check(X, dY, torch.bfloat16)
    if out_mean is None and out_stat is None:
        out_mean = torch.empty((d_out, d_in), dtype=torch.float32, device=X.device)
        out_stat = torch.empty((d_out, d_in), dtype=torch.float32, device=X.device)
    _out_check("out_mean", out_mean, d_out, d_in)
    _out_check("out_stat", out_stat, d_out, d_in)
    with _dev_ctx(X):
        _check("pe_linear_stats", load_library().pe_linear_stats(
            X.data_ptr(), dY.data_ptr(), B, T, d_in, d_out, _phi(phi), _ptr(out_mean), _ptr(out_stat), _stream(X)))
    return out_mean, out_stat


def pe_example_sqnorms(X, dY, out_norms=None):
    """Per-example squared gradient norms ||dY_b^T X_b||_F^2 as a float32 [B] tensor (bf16 inputs)."""
    B, T, d_in, d_out = _io_check(X, dY, torch.bfloat16)
    if out_norms is None:
        out_norms = torch.empty((B,), dtype=torch.float32, device=X.device)
    if out_norms.dtype != torch.float32 or tuple(out_norms.shape) != (B,) or not out_norms.is_contiguous():
        raise ValueError("out_norms must be a contiguous float32 [B] tensor")
    with _dev_ctx(X):
        _check("pe_example_sqnorms", load_library().pe_example_sqnorms(
            X.data_ptr(), dY.data_ptr(), B, T, d_in, d_out, out_norms.data_ptr() if B > 0 else None, _stream(X)))
    return out_norms


def _ragged_check(X, dY, seq_offsets):
    if X.dtype != torch.bfloat16 or dY.dtype != torch.bfloat16:
        raise TypeError("X and dY must be torch.bfloat16")
    if X.dim() != 2 or dY.dim() != 2 or X.shape[0] != dY.shape[0]:
        raise ValueError("X must be [rows, d_in] and dY [rows, d_out] with equal row counts")
    if not (X.is_contiguous() and dY.is_contiguous()):
        raise ValueError("X and dY must be contiguous")
    if seq_offsets.dtype != torch.int32 or seq_offsets.dim() != 1 or seq_offsets.numel() < 1 or not seq_offsets.is_contiguous() \
            or seq_offsets.device != X.device:
        raise ValueError("seq_offsets must be a contiguous int32 [B+1] tensor on the inputs' device")
    return seq_offsets.numel() - 1, X.shape[0], X.shape[1], dY.shape[1]


def pe_linear_stats_ragged_workspace_bytes(B, d_in, d_out) -> int:
    return int(load_library().pe_linear_stats_ragged_workspace_bytes(int(B), int(d_in), int(d_out)))


def _ragged_workspace(workspace, B, d_in, d_out, device):
    need = pe_linear_stats_ragged_workspace_bytes(B, d_in, d_out)
    if workspace is None and need > 0:
        workspace = torch.empty(need, dtype=torch.uint8, device=device)
    return workspace, (workspace.numel() * workspace.element_size() if workspace is not None else 0)


def pe_linear_stats_ragged(X, dY, seq_offsets, phi, out_mean=None, out_stat=None, workspace=None):
    """pe_linear_stats for a packed batch: X [rows, d_in], dY [rows, d_out], example b owns rows
    seq_offsets[b] .. seq_offsets[b+1]-1 (int32 device tensor).  Returns (out_mean, out_stat)."""
    B, rows, d_in, d_out = _ragged_check(X, dY, seq_offsets)
    if out_mean is None and out_stat is None:
        out_mean = torch.empty((d_out, d_in), dtype=torch.float32, device=X.device)
        out_stat = torch.empty((d_out, d_in), dtype=torch.float32, device=X.device)
    _out_check("out_mean", out_mean, d_out, d_in)
    _out_check("out_stat", out_stat, d_out, d_in)
    workspace, wbytes = _ragged_workspace(workspace, B, d_in, d_out, X.device)
    with _dev_ctx(X):
        _check("pe_linear_stats_ragged", load_library().pe_linear_stats_ragged(
            X.data_ptr(), dY.data_ptr(), seq_offsets.data_ptr(), B, rows, d_in, d_out, _phi(phi), _ptr(out_mean), _ptr(out_stat),
            _ptr(workspace), wbytes, _stream(X)))
    return out_mean, out_stat


def pe_example_sqnorms_ragged(X, dY, seq_offsets, out_norms=None, workspace=None):
    """Per-example squared gradient norms of a packed batch, float32 [B]."""
    B, rows, d_in, d_out = _ragged_check(X, dY, seq_offsets)
    if out_norms is None:
        out_norms = torch.empty((B,), dtype=torch.float32, device=X.device)
    if out_norms.dtype != torch.float32 or tuple(out_norms.shape) != (B,) or not out_norms.is_contiguous():
        raise ValueError("out_norms must be a contiguous float32 [B] tensor")
    workspace, wbytes = _ragged_workspace(workspace, B, d_in, d_out, X.device)
    with _dev_ctx(X):
        _check("pe_example_sqnorms_ragged", load_library().pe_example_sqnorms_ragged(
            X.data_ptr(), dY.data_ptr(), seq_offsets.data_ptr(), B, rows, d_in, d_out, out_norms.data_ptr() if B > 0 else None,
            _ptr(workspace), wbytes, _stream(X)))
    return out_norms


def pe_linear_clipped_sum(X, dY, clip_norm, sq_norms=None, out_sum=None):
    """sum_b min(1, clip_norm / sqrt(N_b)) * G_b.  sq_norms None: this layer's own squared norms are computed
    (and returned); otherwise the given float32 [B] tensor is used.  Returns (out_sum, sq_norms)."""
    B, T, d_in, d_out = _io_check(X, dY, torch.bfloat16)
    given = sq_norms is not None
    if sq_norms is None:
        sq_norms = torch.empty((B,), dtype=torch.float32, device=X.device)
    if sq_norms.dtype != torch.float32 or tuple(sq_norms.shape) != (B,) or not sq_norms.is_contiguous():
        raise ValueError("sq_norms must be a contiguous float32 [B] tensor")
    if out_sum is None:
        out_sum = torch.empty((d_out, d_in), dtype=torch.float32, device=X.device)
    _out_check("out_sum", out_sum, d_out, d_in)
    with _dev_ctx(X):
        _check("pe_linear_clipped_sum", load_library().pe_linear_clipped_sum(
            X.data_ptr(), dY.data_ptr(), B, T, d_in, d_out, float(clip_norm), sq_norms.data_ptr() if B > 0 else None, int(given),
            out_sum.data_ptr(), _stream(X)))
    return out_sum, sq_norms


def pe_linear_fused_workspace_bytes(d_in, d_out) -> int:
    return int(load_library().pe_linear_fused_workspace_bytes(int(d_in), int(d_out)))


def _param_check(name, t, d_out, d_in, dtype=torch.float32):
    if t.dtype != dtype or tuple(t.shape) != (d_out, d_in) or not t.is_contiguous():
        raise ValueError(f"{name} must be a contiguous {dtype} [d_out, d_in] tensor")


def pe_linear_microadam_step(X, dY, theta, m, v, *, lr, beta1, beta2, eps, step, variant="microadam", grad_scale=1.0,
                             eps_inside_sqrt=False, weight_decay=0.0, theta_lp=None, out_mean=None, out_stat=None, workspace=None):
    """Per-example statistics (phi = square) and the Adam-family update of theta, m, v in one launch.
    X, dY bf16 (tensor-core / SIMT kernel) or float32 (SIMT kernel).  `workspace`: uint8 tensor of
    pe_linear_fused_workspace_bytes(d_in, d_out) bytes; with it and both outputs the batch may be split."""
    B, T, d_in, d_out = _io_check(X, dY, X.dtype)
    for name, t in (("theta", theta), ("m", m), ("v", v)):
        _param_check(name, t, d_out, d_in)
    if theta_lp is not None:
        _param_check("theta_lp", theta_lp, d_out, d_in, torch.bfloat16)
    _out_check("out_mean", out_mean, d_out, d_in)
    _out_check("out_stat", out_stat, d_out, d_in)
    common = (B, T, d_in, d_out, theta.data_ptr(), _ptr(theta_lp), m.data_ptr(), v.data_ptr(), _ptr(out_mean), _ptr(out_stat),
              ADAM_VARIANTS[variant] if isinstance(variant, str) else int(variant), float(grad_scale), float(lr), float(beta1),
              float(beta2), float(eps), int(bool(eps_inside_sqrt)), float(weight_decay), int(step))
    with _dev_ctx(X):
        if X.dtype == torch.float32:
            _check("pe_linear_microadam_step_f32", load_library().pe_linear_microadam_step_f32(X.data_ptr(), dY.data_ptr(), *common, _stream(X)))
        else:
            wb = workspace.numel() * workspace.element_size() if workspace is not None else 0
            _check("pe_linear_microadam_step", load_library().pe_linear_microadam_step(X.data_ptr(), dY.data_ptr(), *common, _ptr(workspace), wb, _stream(X)))
    return theta, m, v


def pe_linear_microadam_step_f32(X, dY, theta, m, v, **kw):
    """pe_linear_microadam_step for float32 inputs (the C entry point of the same name)."""
    if X.dtype != torch.float32:
        raise TypeError("X and dY must be torch.float32")
    return pe_linear_microadam_step(X, dY, theta, m, v, **kw)


def pe_linear_microsignsgd_step(X, dY, theta, m, *, lr, beta, weight_decay=0.0, theta_lp=None, out_sign=None, workspace=None):
    """Per-example sign statistic and the MicroSignSGD update of theta, m in one launch (bf16 inputs)."""
    B, T, d_in, d_out = _io_check(X, dY, torch.bfloat16)
    _param_check("theta", theta, d_out, d_in)
    _param_check("m", m, d_out, d_in)
    if theta_lp is not None:
        _param_check("theta_lp", theta_lp, d_out, d_in, torch.bfloat16)
    _out_check("out_sign", out_sign, d_out, d_in)
    wb = workspace.numel() * workspace.element_size() if workspace is not None else 0
    with _dev_ctx(X):
        _check("pe_linear_microsignsgd_step", load_library().pe_linear_microsignsgd_step(
            X.data_ptr(), dY.data_ptr(), B, T, d_in, d_out, theta.data_ptr(), _ptr(theta_lp), m.data_ptr(), _ptr(out_sign), float(lr),
            float(beta), float(weight_decay), _ptr(workspace), wb, _stream(X)))
    return theta, m


def pe_linear_stats_accumulate(X, dY, phi, out_mean, out_stat):
    """Adds this micro-batch's sum_b G_b / sum_b phi(G_b) to out_mean / out_stat (either may be None)."""
    B, T, d_in, d_out = _io_check(X, dY, torch.bfloat16)
    _out_check("out_mean", out_mean, d_out, d_in)
    _out_check("out_stat", out_stat, d_out, d_in)
    with _dev_ctx(X):
        _check("pe_linear_stats_accumulate", load_library().pe_linear_stats_accumulate(
            X.data_ptr(), dY.data_ptr(), B, T, d_in, d_out, _phi(phi), _ptr(out_mean), _ptr(out_stat), _stream(X)))
    return out_mean, out_stat


def pe_linear_stats_all(X, dY, out_mean=None, out_square=None, out_sign=None):
    """sum_b G_b, sum_b G_b^2 and sum_b sign(G_b) in one pass (bf16 inputs); returns the three [d_out, d_in]
    float32 tensors.  Missing outputs are allocated."""
    B, T, d_in, d_out = _io_check(X, dY, torch.bfloat16)
    outs = []
    for name, t in (("out_mean", out_mean), ("out_square", out_square), ("out_sign", out_sign)):
        if t is None:
            t = torch.empty((d_out, d_in), dtype=torch.float32, device=X.device)
        _out_check(name, t, d_out, d_in)
        outs.append(t)
    with _dev_ctx(X):
        _check("pe_linear_stats_all", load_library().pe_linear_stats_all(
            X.data_ptr(), dY.data_ptr(), B, T, d_in, d_out, outs[0].data_ptr(), outs[1].data_ptr(), outs[2].data_ptr(), _stream(X)))
    return tuple(outs)


def pe_linear_stats_f32(X, dY, phi, out_mean=None, out_stat=None):
    """fp32-input variant of :func:`pe_linear_stats`."""
    B, T, d_in, d_out = _io_check(X, dY, torch.float32)
    if out_mean is None and out_stat is None:
        out_mean = torch.empty((d_out, d_in), dtype=torch.float32, device=X.device)
        out_stat = torch.empty((d_out, d_in), dtype=torch.float32, device=X.device)
    _out_check("out_mean", out_mean, d_out, d_in)
    _out_check("out_stat", out_stat, d_out, d_in)
    with _dev_ctx(X):
        _check("pe_linear_stats_f32", load_library().pe_linear_stats_f32(
            X.data_ptr(), dY.data_ptr(), B, T, d_in, d_out, _phi(phi), _ptr(out_mean), _ptr(out_stat), _stream(X)))
    return out_mean, out_stat


def pe_token_sqstats(X, dY, out_stat=None):
    """Per-token second moment sum_{b,t} dY^2 X^2 (bf16 inputs), squared and contracted in one kernel."""
    B, T, d_in, d_out = _io_check(X, dY, torch.bfloat16)
    if out_stat is None:
        out_stat = torch.empty((d_out, d_in), dtype=torch.float32, device=X.device)
    _out_check("out_stat", out_stat, d_out, d_in)
    with _dev_ctx(X):
        _check("pe_token_sqstats", load_library().pe_token_sqstats(
            X.data_ptr(), dY.data_ptr(), B, T, d_in, d_out, out_stat.data_ptr(), _stream(X)))
    return out_stat


def pe_token_sqstats_staged_workspace_bytes(B, T, d_in, d_out) -> int:
    return int(load_library().pe_token_sqstats_staged_workspace_bytes(int(B), int(T), int(d_in), int(d_out)))


def pe_token_sqstats_staged(X, dY, out_stat=None, workspace=None):
    """The same statistic in two passes through a workspace holding the squares as column-scaled IEEE
    half (as large as the inputs); the faster form on large layers.  ``workspace`` is a uint8 CUDA tensor
    of at least pe_token_sqstats_staged_workspace_bytes(...) bytes; allocated when omitted."""
    B, T, d_in, d_out = _io_check(X, dY, torch.bfloat16)
    if out_stat is None:
        out_stat = torch.empty((d_out, d_in), dtype=torch.float32, device=X.device)
    _out_check("out_stat", out_stat, d_out, d_in)
    need = pe_token_sqstats_staged_workspace_bytes(B, T, d_in, d_out)
    if workspace is None and need > 0:
        workspace = torch.empty(need, dtype=torch.uint8, device=X.device)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    with _dev_ctx(X):
        _check("pe_token_sqstats_staged", load_library().pe_token_sqstats_staged(
            X.data_ptr(), dY.data_ptr(), B, T, d_in, d_out, out_stat.data_ptr(), _ptr(workspace), ws_bytes, _stream(X)))
    return out_stat


def pe_set_wait_limit_cycles(cycles: int, device=None) -> None:
    """Cycle budget of the waits inside the tensor-core kernels on `device` (default: the current one);
    cycles <= 0 restores the default.  For tests of the PE_ERR_TIMEOUT path."""
    dev = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
    with torch.cuda.device(dev):
        torch.cuda.synchronize()
        _check("pe_set_wait_limit_cycles", load_library().pe_set_wait_limit_cycles(int(cycles)))


def pe_token_sqstats_fp8_workspace_bytes(B, T, d_in, d_out) -> int:
    return int(load_library().pe_token_sqstats_fp8_workspace_bytes(int(B), int(T), int(d_in), int(d_out)))


def pe_token_sqstats_fp8(X, dY, out_stat=None, workspace=None):
    """The two-pass per-token statistic with the squares staged as e4m3 and contracted at the 8-bit tensor-core
    rate: an approximation with about 0.0375 * sqrt(sum w^2) / sum w relative error per entry (see pestats.h)."""
    B, T, d_in, d_out = _io_check(X, dY, torch.bfloat16)
    if out_stat is None:
        out_stat = torch.empty((d_out, d_in), dtype=torch.float32, device=X.device)
    _out_check("out_stat", out_stat, d_out, d_in)
    need = pe_token_sqstats_fp8_workspace_bytes(B, T, d_in, d_out)
    if workspace is None and need > 0:
        workspace = torch.empty(need, dtype=torch.uint8, device=X.device)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    with _dev_ctx(X):
        _check("pe_token_sqstats_fp8", load_library().pe_token_sqstats_fp8(
            X.data_ptr(), dY.data_ptr(), B, T, d_in, d_out, out_stat.data_ptr(), _ptr(workspace), ws_bytes, _stream(X)))
    return out_stat


def pe_token_sqstats_static(X, dY, out_stat):
    """Per-token second moment for callers that cannot supply (or allocate) a workspace: the library's
    built-in device array of STATIC_SCRATCH_BYTES stages the squared operands, and neither this
    wrapper nor the library allocates anything, so ``out_stat`` (float32 [d_out, d_in]) is required.
    Shapes whose staging does not fit raise PestatsError (PE_ERR_WORKSPACE).  Calls that may overlap on
    the GPU share that array and race; keep them on one stream.  Make the first call on a device
    outside stream capture (it looks up the array's address)."""
    B, T, d_in, d_out = _io_check(X, dY, torch.bfloat16)
    if out_stat is None:
        raise ValueError("out_stat is required: this entry point allocates nothing")
    _out_check("out_stat", out_stat, d_out, d_in)
    with _dev_ctx(X):
        _check("pe_token_sqstats_static", load_library().pe_token_sqstats_static(
            X.data_ptr(), dY.data_ptr(), B, T, d_in, d_out, out_stat.data_ptr(), _stream(X)))
    return out_stat


def pe_token_sqstats_f32(X, dY, out_stat=None):
    B, T, d_in, d_out = _io_check(X, dY, torch.float32)
    if out_stat is None:
        out_stat = torch.empty((d_out, d_in), dtype=torch.float32, device=X.device)
    _out_check("out_stat", out_stat, d_out, d_in)
    with _dev_ctx(X):
        _check("pe_token_sqstats_f32", load_library().pe_token_sqstats_f32(
            X.data_ptr(), dY.data_ptr(), B, T, d_in, d_out, out_stat.data_ptr(), _stream(X)))
    return out_stat


def _flat_f32(name, t, n=None):
    if t.dtype != torch.float32 or not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous float32")
    if n is not None and t.numel() != n:
        raise ValueError(f"{name} has {t.numel()} elements, expected {n}")
    return t.numel()


def microadam_step(theta, m, v, sum_g, sum_g2, B, *, lr, beta1, beta2, eps, step, grad_scale=1.0,
                   eps_inside_sqrt=False, weight_decay=0.0, theta_lp=None):
    """In-place MicroAdam update of (theta, m, v) from sum_b G_b and sum_b G_b^2."""
    n = _flat_f32("theta", theta)
    for name, t in (("m", m), ("v", v), ("sum_g", sum_g), ("sum_g2", sum_g2)):
        _flat_f32(name, t, n)
    if theta_lp is not None and (theta_lp.dtype != torch.bfloat16 or theta_lp.numel() != n or not theta_lp.is_contiguous()):
        raise ValueError("theta_lp must be contiguous bfloat16 with theta's element count")
    with _dev_ctx(theta):
        _check("microadam_step", load_library().microadam_step(
            theta.data_ptr(), _ptr(theta_lp), m.data_ptr(), v.data_ptr(), sum_g.data_ptr(), sum_g2.data_ptr(), n, int(B),
            float(grad_scale), float(lr), float(beta1), float(beta2), float(eps), int(bool(eps_inside_sqrt)),
            float(weight_decay), int(step), _stream(theta)))


def microadam_family_step(theta, m, v, sum_g, sum_g2, B, variant, *, lr, beta1, beta2, eps, step, grad_scale=1.0,
                          eps_inside_sqrt=False, weight_decay=0.0, theta_lp=None):
    """In-place update by a member of the extended Adam family: variant is "adam", "microadam",
    "microadam_var" or "microadam_msq" (or the integer code)."""
    n = _flat_f32("theta", theta)
    for name, t in (("m", m), ("v", v), ("sum_g", sum_g), ("sum_g2", sum_g2)):
        _flat_f32(name, t, n)
    if theta_lp is not None and (theta_lp.dtype != torch.bfloat16 or theta_lp.numel() != n or not theta_lp.is_contiguous()):
        raise ValueError("theta_lp must be contiguous bfloat16 with theta's element count")
    code = ADAM_VARIANTS[variant] if isinstance(variant, str) else int(variant)
    with _dev_ctx(theta):
        _check("microadam_family_step", load_library().microadam_family_step(
            theta.data_ptr(), _ptr(theta_lp), m.data_ptr(), v.data_ptr(), sum_g.data_ptr(), sum_g2.data_ptr(), n, int(B), code,
            float(grad_scale), float(lr), float(beta1), float(beta2), float(eps), int(bool(eps_inside_sqrt)),
            float(weight_decay), int(step), _stream(theta)))


def microsignsgd_step(theta, m, sum_sign, B, *, lr, beta, weight_decay=0.0, theta_lp=None):
    """In-place MicroSignSGD update of (theta, m) from sum_b sign(G_b)."""
    n = _flat_f32("theta", theta)
    _flat_f32("m", m, n)
    _flat_f32("sum_sign", sum_sign, n)
    if theta_lp is not None and (theta_lp.dtype != torch.bfloat16 or theta_lp.numel() != n or not theta_lp.is_contiguous()):
        raise ValueError("theta_lp must be contiguous bfloat16 with theta's element count")
    with _dev_ctx(theta):
        _check("microsignsgd_step", load_library().microsignsgd_step(
            theta.data_ptr(), _ptr(theta_lp), m.data_ptr(), sum_sign.data_ptr(), n, int(B), float(lr), float(beta),
            float(weight_decay), _stream(theta)))


def pe_get_async_status(device=None):
    """Synchronises the current stream of ``device``; returns (status, detail). status 0 = OK."""
    dev = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
    detail = ctypes.c_int(0)
    with torch.cuda.device(dev):
        st = load_library().pe_get_async_status(torch.cuda.current_stream(dev).cuda_stream, ctypes.byref(detail))
    return int(st), int(detail.value)


def pe_set_fused_update(mode: int) -> int:
    """Chooses how the statistics + update calls run (FUSED_AUTO / FUSED_ALWAYS / FUSED_NEVER); returns the previous mode."""
    return int(load_library().pe_set_fused_update(int(mode)))


def pe_set_path(path: int) -> int:
    return int(load_library().pe_set_path(int(path)))


def pe_tile_order_band(d_in: int, d_out: int, tile_cols: int, batch_slices: int, sm_count: int) -> int:
    """Pair rows per band of the tile order a tensor-core launch of this shape would use (host-side query)."""
    return int(load_library().pe_tile_order_band(int(d_in), int(d_out), int(tile_cols), int(batch_slices), int(sm_count)))


def pe_last_path() -> int:
    return int(load_library().pe_last_path())


def pe_launch_count() -> int:
    return int(load_library().pe_launch_count())


def pe_reset_launch_count() -> None:
    load_library().pe_reset_launch_count()
