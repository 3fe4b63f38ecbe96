"""Thin ctypes binding over the C ABI in include/awq_b200.h (argument marshalling only).

torch supplies device memory and the current stream; every step of the layer runs in the
CUDA library.  There is no fallback: if the library has not been built, or a call returns
an error status, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libawq_b200.so")

PATH_AUTO, PATH_GEMV, PATH_GEMM, PATH_GEMV_SPLITK, PATH_GEMM_1SM, PATH_GEMV_MID, PATH_GEMM_SKINNY = 0, 1, 2, 3, 4, 5, 6

EXPORTS = (
    "awq_qweight_bytes", "awq_scales_bytes", "awq_zeros_bytes", "awq_quantize_pack",
    "awq_channel_scale", "awq_linear", "awq_linear_path", "awq_workspace_bytes",
    "awq_set_workspace", "awq_unpack_canonical", "awq_poll_status", "awq_status_string",
    "awq_last_cuda_error", "awq_layout_version", "awq_launch_count", "awq_linear_gemv_static",
    "awq_linear_multi", "awq_search_scratch_bytes", "awq_search_alpha",
    "awq_quantize_pack_ex", "awq_search_clip", "awq_static_scratch_fill",
    "awq_set_wait_limit_us", "awq_test_stall_next_gemv",
    "awq_linear_scaled", "awq_linear_multi_scaled", "awq_linear_scaled_needs_scratch",
    "awq_inverse_channel_scale", "awq_qweight_bytes_int3", "awq_pack_int3", "awq_unpack_int3", "awq_linear_int3",
)


class _Problem(ctypes.Structure):
    _fields_ = [("qweight", ctypes.c_void_p), ("scales", ctypes.c_void_p), ("zeros", ctypes.c_void_p),
                ("y", ctypes.c_void_p), ("N", ctypes.c_int)]

_lib = None
_workspace: dict = {}          # device index -> torch tensor registered with the library


class AwqError(RuntimeError):
    pass


def lib() -> ctypes.CDLL:
    """Loads the library on first use; raises if it is missing (no CPU or eager fallback)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise AwqError(f"{LIB_PATH} not found: build it with `python -m paper_2306_00978_b200.build`")
    L = ctypes.CDLL(LIB_PATH)
    vp, i, f, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
    L.awq_qweight_bytes.restype, L.awq_qweight_bytes.argtypes = sz, [i, i]
    L.awq_scales_bytes.restype, L.awq_scales_bytes.argtypes = sz, [i, i, i]
    L.awq_zeros_bytes.restype, L.awq_zeros_bytes.argtypes = sz, [i, i, i]
    L.awq_quantize_pack.restype, L.awq_quantize_pack.argtypes = i, [vp, vp, f, i, vp, vp, vp, i, i, vp]
    L.awq_quantize_pack_ex.restype, L.awq_quantize_pack_ex.argtypes = i, [vp, vp, f, i, i, i, vp, vp, vp, vp, i, i, vp]
    L.awq_search_clip.restype, L.awq_search_clip.argtypes = i, [vp, vp, f, i, i, vp, i, vp, i, i, vp]
    L.awq_channel_scale.restype, L.awq_channel_scale.argtypes = i, [vp, f, vp, i, vp]
    L.awq_linear.restype, L.awq_linear.argtypes = i, [vp, vp, vp, vp, vp, i, i, i, i, vp]
    L.awq_linear_path.restype, L.awq_linear_path.argtypes = i, [vp, vp, vp, vp, vp, i, i, i, i, i, vp]
    L.awq_linear_gemv_static.restype, L.awq_linear_gemv_static.argtypes = i, [vp, vp, vp, vp, vp, i, i, i, i, vp]
    L.awq_static_scratch_fill.restype, L.awq_static_scratch_fill.argtypes = i, [i, vp]
    L.awq_set_wait_limit_us.restype, L.awq_set_wait_limit_us.argtypes = i, [ctypes.c_uint]
    L.awq_test_stall_next_gemv.restype, L.awq_test_stall_next_gemv.argtypes = i, []
    L.awq_linear_scaled.restype, L.awq_linear_scaled.argtypes = i, [vp, vp, vp, vp, vp, vp, vp, i, i, i, i, vp]
    L.awq_linear_multi_scaled.restype, L.awq_linear_multi_scaled.argtypes = i, [vp, vp, vp, vp, i, i, i, i, vp]
    L.awq_inverse_channel_scale.restype, L.awq_inverse_channel_scale.argtypes = i, [vp, f, vp, i, vp]
    L.awq_qweight_bytes_int3.restype, L.awq_qweight_bytes_int3.argtypes = sz, [i, i]
    L.awq_pack_int3.restype, L.awq_pack_int3.argtypes = i, [vp, vp, i, i, vp]
    L.awq_unpack_int3.restype, L.awq_unpack_int3.argtypes = i, [vp, vp, i, i, vp]
    L.awq_linear_int3.restype, L.awq_linear_int3.argtypes = i, [vp, vp, vp, vp, vp, vp, i, i, i, i, vp]
    L.awq_linear_scaled_needs_scratch.restype, L.awq_linear_scaled_needs_scratch.argtypes = i, [i, i, i, i]
    L.awq_linear_multi.restype, L.awq_linear_multi.argtypes = i, [vp, vp, i, i, i, i, vp]
    L.awq_search_scratch_bytes.restype, L.awq_search_scratch_bytes.argtypes = sz, [i, i, i, i]
    L.awq_search_alpha.restype, L.awq_search_alpha.argtypes = i, [vp, vp, vp, i, i, i, i, vp, i, vp, vp, vp, sz, vp]
    L.awq_workspace_bytes.restype, L.awq_workspace_bytes.argtypes = sz, [i, i, i, i]
    L.awq_set_workspace.restype, L.awq_set_workspace.argtypes = i, [vp, sz]
    L.awq_unpack_canonical.restype, L.awq_unpack_canonical.argtypes = i, [vp, vp, vp, i, i, i, vp, vp, vp, vp]
    L.awq_poll_status.restype, L.awq_poll_status.argtypes = i, []
    L.awq_status_string.restype, L.awq_status_string.argtypes = ctypes.c_char_p, [i]
    L.awq_last_cuda_error.restype, L.awq_last_cuda_error.argtypes = ctypes.c_char_p, []
    L.awq_layout_version.restype, L.awq_layout_version.argtypes = i, []
    L.awq_launch_count.restype, L.awq_launch_count.argtypes = ctypes.c_ulonglong, []
    _lib = L
    return L


def _check(rc: int, what: str) -> None:
    if rc != 0:
        L = lib()
        msg = L.awq_status_string(rc).decode()
        extra = L.awq_last_cuda_error().decode()
        raise AwqError(f"{what}: status {rc} ({msg}){' - ' + extra if extra and rc == 8 else ''}")


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _dev(t: torch.Tensor, dtype: torch.dtype, name: str) -> int:
    if not t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise AwqError(f"{name}: expected a contiguous CUDA tensor of dtype {dtype}")
    return t.data_ptr()


def launch_count() -> int:
    return int(lib().awq_launch_count())


def packed_sizes(N: int, K: int, group: int) -> Tuple[int, int, int]:
    L = lib()
    sizes = (L.awq_qweight_bytes(N, K), L.awq_scales_bytes(N, K, group), L.awq_zeros_bytes(N, K, group))
    if 0 in sizes:
        raise AwqError(f"shape N={N}, K={K}, group={group} is not accepted")
    return sizes


def channel_scale(act_mean_abs: Optional[torch.Tensor], alpha: float, K: int) -> torch.Tensor:
    """s = act_mean_abs ** alpha as the quantizer computes it (Eq. 5); fp32 [K] on the device."""
    s = torch.empty(K, dtype=torch.float32, device="cuda")
    a = 0 if act_mean_abs is None else _dev(act_mean_abs, torch.float32, "act_mean_abs")
    _check(lib().awq_channel_scale(a, float(alpha), s.data_ptr(), K, _stream()), "awq_channel_scale")
    return s


def inverse_channel_scale(act_mean_abs: Optional[torch.Tensor], alpha: float, K: int) -> torch.Tensor:
    """1 / s as awq_linear_scaled wants it (the correctly rounded reciprocal of channel_scale)."""
    inv = torch.empty(K, dtype=torch.float32, device="cuda")
    a = 0 if act_mean_abs is None else _dev(act_mean_abs, torch.float32, "act_mean_abs")
    _check(lib().awq_inverse_channel_scale(a, float(alpha), inv.data_ptr(), K, _stream()), "awq_inverse_channel_scale")
    return inv


def quantize_pack(W: torch.Tensor, act_mean_abs: Optional[torch.Tensor], alpha: float, group: int,
                  clip_ratio: Optional[torch.Tensor] = None, bits: int = 4, symmetric: bool = False):
    """awq_quantize_pack / awq_quantize_pack_ex: returns (qweight u8 [N*K/2],
    scales fp16 [N/16][K/g][16], zeros u8 [N/32][K/g][16]), g = min(group, 128)."""
    N, K = W.shape
    qb, sb, zb = packed_sizes(N, K, group)
    dev = W.device
    qweight = torch.empty(qb, dtype=torch.uint8, device=dev)
    stored = min(int(group), 128)                  # groups above 128 columns are stored once per 128 columns
    scales = torch.empty((N // 16, K // stored, 16), dtype=torch.float16, device=dev)
    zeros = torch.empty((N // 32, K // stored, 16), dtype=torch.uint8, device=dev)
    a = 0 if act_mean_abs is None else _dev(act_mean_abs, torch.float32, "act_mean_abs")
    if clip_ratio is None and bits == 4 and not symmetric:
        rc = lib().awq_quantize_pack(_dev(W, torch.float16, "W"), a, float(alpha), int(group),
                                     qweight.data_ptr(), scales.data_ptr(), zeros.data_ptr(), N, K, _stream())
        _check(rc, "awq_quantize_pack")
        return qweight, scales, zeros
    c = 0
    if clip_ratio is not None:
        if tuple(clip_ratio.shape) != (N, K // group):
            raise AwqError(f"clip_ratio: expected shape {(N, K // group)}")
        c = _dev(clip_ratio, torch.float32, "clip_ratio")
    rc = lib().awq_quantize_pack_ex(_dev(W, torch.float16, "W"), a, float(alpha), int(group), int(bits),
                                    int(bool(symmetric)), c,
                                    qweight.data_ptr(), scales.data_ptr(), zeros.data_ptr(), N, K, _stream())
    _check(rc, "awq_quantize_pack_ex")
    return qweight, scales, zeros


def search_clip(W: torch.Tensor, act_mean_abs: Optional[torch.Tensor], alpha: float, group: int,
                ratios, bits: int = 4) -> torch.Tensor:
    """awq_search_clip: per-group range ratios (fp32 [N][K/group], device) of least squared
    quantization error, each one of `ratios` (a sequence of floats in (0, 1])."""
    N, K = W.shape
    out = torch.empty((N, K // group), dtype=torch.float32, device=W.device)
    arr = (ctypes.c_float * len(ratios))(*[float(r) for r in ratios])
    a = 0 if act_mean_abs is None else _dev(act_mean_abs, torch.float32, "act_mean_abs")
    rc = lib().awq_search_clip(_dev(W, torch.float16, "W"), a, float(alpha), int(group), int(bits),
                               ctypes.cast(arr, ctypes.c_void_p), len(ratios), out.data_ptr(), N, K, _stream())
    _check(rc, "awq_search_clip")
    return out


def ensure_workspace(nbytes: int) -> None:
    """Registers (growing if needed) a torch-allocated scratch buffer for the current device."""
    if nbytes <= 0:
        return
    dev = torch.cuda.current_device()
    cur = _workspace.get(dev)
    if cur is not None and cur.numel() >= nbytes:
        return
    torch.cuda.synchronize()
    buf = torch.empty(max(nbytes, 1 << 22), dtype=torch.uint8, device=f"cuda:{dev}")
    _check(lib().awq_set_workspace(buf.data_ptr(), buf.numel()), "awq_set_workspace")
    _workspace[dev] = buf


def workspace_bytes(M: int, N: int, K: int, group: int) -> int:
    return int(lib().awq_workspace_bytes(M, N, K, group))


def linear(x: torch.Tensor, qweight: torch.Tensor, scales: torch.Tensor, zeros: torch.Tensor,
           N: int, K: int, group: int, out: Optional[torch.Tensor] = None,
           path: int = PATH_AUTO) -> torch.Tensor:
    """awq_linear / awq_linear_path: y = x . dequant(Wq)^T, x fp16 [M][K] already divided by s."""
    M = x.shape[0]
    if x.shape[1] != K:
        raise AwqError("x must be [M][K]")
    y = out if out is not None else torch.empty((M, N), dtype=torch.float16, device=x.device)
    ensure_workspace(workspace_bytes(M, N, K, group))         # required (split-K GEMV) or optional (GEMM)
    args = (_dev(x, torch.float16, "x"), _dev(qweight, torch.uint8, "qweight"),
            _dev(scales, torch.float16, "scales"), _dev(zeros, torch.uint8, "zeros"),
            _dev(y, torch.float16, "y"), M, N, K, int(group))
    if path == PATH_AUTO:
        rc = lib().awq_linear(*args, _stream())
    else:
        rc = lib().awq_linear_path(*args, int(path), _stream())
    _check(rc, "awq_linear")
    return y


def linear_multi(x: torch.Tensor, mats, K: int, group: int, outs=None):
    """awq_linear_multi: several packed matrices that read the same x (fused q/k/v or gate/up), one
    call.  `mats` is a list of (qweight, scales, zeros, N); returns the list of outputs."""
    M = x.shape[0]
    if x.shape[1] != K:
        raise AwqError("x must be [M][K]")
    if outs is None:
        outs = [torch.empty((M, m[3]), dtype=torch.float16, device=x.device) for m in mats]
    if M <= 16:
        ensure_workspace(max(workspace_bytes(M, m[3], K, group) for m in mats))
    arr = (_Problem * len(mats))()
    for k, ((qw, sc, zp, N), y) in enumerate(zip(mats, outs)):
        arr[k] = _Problem(_dev(qw, torch.uint8, "qweight"), _dev(sc, torch.float16, "scales"),
                          _dev(zp, torch.uint8, "zeros"), _dev(y, torch.float16, "y"), int(N))
    rc = lib().awq_linear_multi(_dev(x, torch.float16, "x"), ctypes.byref(arr), len(mats), M, K, int(group),
                                _stream())
    _check(rc, "awq_linear_multi")
    return outs


def linear_multi_scaled(x: torch.Tensor, inv_s: torch.Tensor, mats, K: int, group: int, outs=None,
                        x_scratch: Optional[torch.Tensor] = None):
    """awq_linear_multi_scaled (awq_linear_scaled for one matrix): x is NOT scaled; the product
    fp16(fp32(x) * inv_s) is folded into the matrix-vector kernel where it can be, else formed
    by a small kernel into `x_scratch` (allocated here if it is needed and not given)."""
    M = x.shape[0]
    s = inv_s
    if x.shape[1] != K or s.numel() != K:
        raise AwqError("x must be [M][K] and inv_s [K]")
    if outs is None:
        outs = [torch.empty((M, m[3]), dtype=torch.float16, device=x.device) for m in mats]
    if x_scratch is None and lib().awq_linear_scaled_needs_scratch(M, sum(m[3] for m in mats), K, int(group)):
        x_scratch = torch.empty_like(x)
    ensure_workspace(max(workspace_bytes(M, m[3], K, group) for m in mats))
    arr = (_Problem * len(mats))()
    for k, ((qw, sc, zp, N), y) in enumerate(zip(mats, outs)):
        arr[k] = _Problem(_dev(qw, torch.uint8, "qweight"), _dev(sc, torch.float16, "scales"),
                          _dev(zp, torch.uint8, "zeros"), _dev(y, torch.float16, "y"), int(N))
    rc = lib().awq_linear_multi_scaled(_dev(x, torch.float16, "x"), _dev(s, torch.float32, "s"),
                                       0 if x_scratch is None else _dev(x_scratch, torch.float16, "x_scratch"),
                                       ctypes.byref(arr), len(mats), M, K, int(group), _stream())
    _check(rc, "awq_linear_multi_scaled")
    return outs


def pack_int3(qweight: torch.Tensor, N: int, K: int) -> torch.Tensor:
    """awq_pack_int3: the 4-bit layout holding 3-bit codes -> the 3-bit storage (u8 [N*K*3/8])."""
    out = torch.empty(int(lib().awq_qweight_bytes_int3(N, K)), dtype=torch.uint8, device=qweight.device)
    _check(lib().awq_pack_int3(_dev(qweight, torch.uint8, "qweight"), out.data_ptr(), N, K, _stream()), "awq_pack_int3")
    return out


def unpack_int3(qweight3: torch.Tensor, N: int, K: int) -> torch.Tensor:
    out = torch.empty(N * K // 2, dtype=torch.uint8, device=qweight3.device)
    _check(lib().awq_unpack_int3(_dev(qweight3, torch.uint8, "qweight3"), out.data_ptr(), N, K, _stream()),
           "awq_unpack_int3")
    return out


def linear_int3(x: torch.Tensor, qweight3: torch.Tensor, scales: torch.Tensor, zeros: torch.Tensor,
                N: int, K: int, group: int, out: Optional[torch.Tensor] = None,
                scratch: Optional[torch.Tensor] = None) -> torch.Tensor:
    """awq_linear_int3: the layer on the 3-bit storage (`scratch`, N*K/2 bytes, is allocated here
    when the shape needs the expansion and none is given)."""
    M = x.shape[0]
    y = out if out is not None else torch.empty((M, N), dtype=torch.float16, device=x.device)
    ensure_workspace(workspace_bytes(M, N, K, group))
    if scratch is None:
        scratch = torch.empty(N * K // 2, dtype=torch.uint8, device=x.device)
    rc = lib().awq_linear_int3(_dev(x, torch.float16, "x"), _dev(qweight3, torch.uint8, "qweight3"),
                               _dev(scales, torch.float16, "scales"), _dev(zeros, torch.uint8, "zeros"),
                               _dev(y, torch.float16, "y"), scratch.data_ptr(), M, N, K, int(group), _stream())
    _check(rc, "awq_linear_int3")
    return y


def linear_gemv_static(x: torch.Tensor, qweight: torch.Tensor, scales: torch.Tensor, zeros: torch.Tensor,
                       N: int, K: int, group: int, out: torch.Tensor) -> torch.Tensor:
    """awq_linear_gemv_static: the matrix-vector kernel on the library's built-in scratch.

    For callers that must not allocate device memory: nothing is allocated here either,
    so the output tensor `out` (fp16 [M][N]) has to be passed in.  M <= 8."""
    M = x.shape[0]
    if x.shape[1] != K or tuple(out.shape) != (M, N):
        raise AwqError("x must be [M][K] and out [M][N]")
    rc = lib().awq_linear_gemv_static(
        _dev(x, torch.float16, "x"), _dev(qweight, torch.uint8, "qweight"),
        _dev(scales, torch.float16, "scales"), _dev(zeros, torch.uint8, "zeros"),
        _dev(out, torch.float16, "out"), M, N, K, int(group), _stream())
    _check(rc, "awq_linear_gemv_static")
    return out


def set_wait_limit_us(us: int) -> None:
    """awq_set_wait_limit_us: limit of a device-side wait (0 = default)."""
    _check(lib().awq_set_wait_limit_us(int(us)), "awq_set_wait_limit_us")


def static_scratch_fill(value: int) -> None:
    """awq_static_scratch_fill: test aid, dirties the built-in scratch's arrival counters."""
    _check(lib().awq_static_scratch_fill(int(value), _stream()), "awq_static_scratch_fill")


def search_alpha(W: torch.Tensor, act_mean_abs: torch.Tensor, X: torch.Tensor, group: int, alphas):
    """awq_search_alpha (Sec. 3.2): returns (losses as a list of floats, index of the first least loss)."""
    N, K = W.shape
    M = X.shape[0]
    n = len(alphas)
    need = int(lib().awq_search_scratch_bytes(M, N, K, int(group)))
    if need == 0:
        raise AwqError(f"shape N={N}, K={K}, group={group} is not accepted")
    scratch = torch.empty(need, dtype=torch.uint8, device=W.device)
    ensure_workspace(workspace_bytes(M, N, K, group))
    a = (ctypes.c_float * n)(*[float(v) for v in alphas])
    losses = (ctypes.c_float * n)()
    best = ctypes.c_int(0)
    rc = lib().awq_search_alpha(_dev(W, torch.float16, "W"), _dev(act_mean_abs, torch.float32, "act_mean_abs"),
                                _dev(X, torch.float16, "X"), M, N, K, int(group), a, n, losses,
                                ctypes.byref(best), scratch.data_ptr(), need, _stream())
    _check(rc, "awq_search_alpha")
    return [float(v) for v in losses], int(best.value)


def unpack_canonical(qweight, scales, zeros, N: int, K: int, group: int):
    """Expands the packed arrays: (codes u8 [N][K], scales fp16 [N][K/group], zeros u8 [N][K/group])."""
    ng = K // group
    codes = torch.empty((N, K), dtype=torch.uint8, device=qweight.device)
    sc = torch.empty((N, ng), dtype=torch.float16, device=qweight.device)
    zp = torch.empty((N, ng), dtype=torch.uint8, device=qweight.device)
    rc = lib().awq_unpack_canonical(qweight.data_ptr(), scales.data_ptr(), zeros.data_ptr(), N, K, int(group),
                                    codes.data_ptr(), sc.data_ptr(), zp.data_ptr(), _stream())
    _check(rc, "awq_unpack_canonical")
    return codes, sc, zp


def poll_status() -> None:
    """Synchronizes and raises if a kernel gave up a bounded wait since the last poll."""
    _check(lib().awq_poll_status(), "awq_poll_status")
