"""ctypes binding of ``libslim.so`` with the same names as ``include/slim.h``.

Argument marshalling only: tensors are torch CUDA tensors (torch supplies device
memory and streams), every step of the computation runs in the library's
kernels.  If the library is missing or a call fails, a :class:`SlimError` is
raised; there is no fallback path.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libslim.so")

(SLIM_OK, SLIM_ERR_INVALID_ARG, SLIM_ERR_UNSUPPORTED_SHAPE, SLIM_ERR_BAD_MASK, SLIM_ERR_CODE_RANGE,
 SLIM_ERR_WORKSPACE, SLIM_ERR_CUDA, SLIM_ERR_TIMEOUT, SLIM_ERR_ARCH) = range(9)
KERNEL_AUTO, KERNEL_SIMPLE, KERNEL_DECODE, KERNEL_PREFILL, KERNEL_PREFILL_PAIR = range(5)
KERNEL_NAMES = {KERNEL_AUTO: "auto", KERNEL_SIMPLE: "simple", KERNEL_DECODE: "decode", KERNEL_PREFILL: "prefill", KERNEL_PREFILL_PAIR: "prefill_pair"}
WORKSPACE_SYNC_BYTES = 256
NOALLOC_SCRATCH_BYTES = 16 << 20
LAYOUT_DECODE_TILED = 1

# every symbol include/slim.h declares, with (restype, argtypes)
_P, _I, _F, _SZ = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
SIGNATURES = {
    "slim_pack": (_I, [_P, _P, _I, _I, _P, _P, _P, _P]),
    "slim_unpack": (_I, [_P, _P, _I, _I, _P, _P, _P]),
    "slim_workspace_bytes": (_SZ, [_I, _I, _I, _I]),
    "slim_workspace_reset": (_I, [_P, _SZ, _P]),
    "slim_linear_fwd": (_I, [_P, _I, _P, _P, _F, _P, _P, _I, _I, _I, _P, _P, _SZ, _P, _P]),
    "slim_linear_fwd_ex": (_I, [_P, _I, _P, _P, _F, _P, _P, _I, _I, _I, _P, _P, _SZ, _P, _P, _I]),
    "slim_linear_fwd_host": (_I, [_P, _I, _P, _P, _F, _P, _P, _I, _I, _I, _P, _P, _P, _P, _SZ, _P, _P]),
    "slim_linear_fwd_noalloc": (_I, [_P, _I, _P, _P, _F, _P, _P, _I, _I, _I, _P, _P, _P]),
    "slim_tiled_bytes": (_SZ, [_I, _I, _I]),
    "slim_repack_tiled": (_I, [_P, _P, _I, _I, _I, _P, _P]),
    "slim_linear_fwd_tiled": (_I, [_P, _I, _P, _I, _F, _P, _P, _I, _I, _I, _P, _P, _SZ, _P, _P]),
    "slim_linear_fwd_tiled_host": (_I, [_P, _I, _P, _I, _F, _P, _P, _I, _I, _I, _P, _P, _P, _P, _SZ, _P, _P]),
    "slim_noalloc_scratch_needed": (_SZ, [_I, _I, _I, _I]),
    "slim_mask_top2": (_I, [_P, _P, _I, _I, _P, _P, _P]),
    "slim_quant_workspace_bytes": (_SZ, [_I, _I]),
    "slim_quant": (_I, [_P, _I, _I, _P, _P, _P, _SZ, _P, _P]),
    "slim_adapter_code_bytes": (_SZ, [_I, _I]),
    "slim_adapter_scale_bytes": (_SZ, [_I, _I]),
    "slim_pack_adapter": (_I, [_P, _I, _I, _P, _P, _P]),
    "slim_unpack_adapter": (_I, [_P, _P, _I, _I, _P, _P]),
    "slim_workspace_bytes_q": (_SZ, [_I, _I, _I, _I]),
    "slim_linear_fwd_q": (_I, [_P, _I, _P, _P, _F, _P, _P, _P, _P, _I, _I, _I, _P, _P, _SZ, _P, _P]),
    "slim_select_kernel": (_I, [_I, _I, _I, _I]),
    "slim_decode_layout_hint": (_I, [_I, _I, _I, _I]),
    "slim_last_launch_count": (_I, []),
    "slim_last_token_tile": (_I, []),
    "slim_strerror": (ctypes.c_char_p, [_I]),
    "slim_version": (ctypes.c_char_p, []),
}


class SlimError(RuntimeError):
    def __init__(self, code: int, where: str, text: str = ""):
        super().__init__(f"{where}: {text or code} (status {code})")
        self.code = code


_lib = None


def lib() -> ctypes.CDLL:
    """Load ``libslim.so`` (built in-tree by ``build.py``); raise if it is absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise SlimError(-1, "load", f"{LIB_PATH} not found: run paper_2410_09615_b200/build.py")
        l = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(l, name)
            fn.restype, fn.argtypes = res, args
        _lib = l
    return _lib


def strerror(code: int) -> str:
    return lib().slim_strerror(code).decode()


def _check(code: int, where: str):
    if code != SLIM_OK:
        raise SlimError(code, where, strerror(code))


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _dev(t, dtype, name):
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise TypeError(f"{name}: expected a contiguous CUDA tensor of {dtype}")
    return t


def bf16_from_bits(bits: np.ndarray, device="cuda") -> torch.Tensor:
    """uint16 bfloat16 bit patterns (host) -> torch.bfloat16 tensor on ``device``."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).to(device)


def bits_from_bf16(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def read_status(status: torch.Tensor) -> int:
    return int(status.item()) & 0xFFFFFFFF


def raise_on_status(bits: int, where: str):
    for code in (SLIM_ERR_BAD_MASK, SLIM_ERR_CODE_RANGE, SLIM_ERR_TIMEOUT):
        if bits & (1 << code):
            raise SlimError(code, where, strerror(code))


def slim_pack(codes: torch.Tensor, mask: torch.Tensor, vals=None, meta=None, status=None, check=True):
    """codes int8 [d_out, d_in], mask uint8 [d_out, d_in] -> (vals, meta) uint8 tensors."""
    _dev(codes, torch.int8, "codes"), _dev(mask, torch.uint8, "mask")
    d_out, d_in = codes.shape
    if vals is None:
        vals = torch.empty((d_out, d_in // 4), dtype=torch.uint8, device=codes.device)
    if meta is None:
        meta = torch.empty((d_out, d_in // 8), dtype=torch.uint8, device=codes.device)
    own_status = status is None and check
    if own_status:
        status = torch.zeros(1, dtype=torch.int32, device=codes.device)
    _check(lib().slim_pack(_ptr(codes), _ptr(mask), d_out, d_in, _ptr(vals), _ptr(meta), _ptr(status), _stream()),
           "slim_pack")
    if own_status:
        raise_on_status(read_status(status), "slim_pack")
    return vals, meta


def slim_unpack(vals: torch.Tensor, meta: torch.Tensor, want_mask=True):
    _dev(vals, torch.uint8, "vals"), _dev(meta, torch.uint8, "meta")
    d_out, d_in = vals.shape[0], vals.shape[1] * 4
    codes = torch.empty((d_out, d_in), dtype=torch.int8, device=vals.device)
    mask = torch.empty((d_out, d_in), dtype=torch.uint8, device=vals.device) if want_mask else None
    _check(lib().slim_unpack(_ptr(vals), _ptr(meta), d_out, d_in, _ptr(codes), _ptr(mask), _stream()), "slim_unpack")
    return codes, mask


def slim_workspace_bytes(b: int, d_out: int, d_in: int, r: int) -> int:
    return int(lib().slim_workspace_bytes(b, d_out, d_in, r))


def slim_noalloc_scratch_needed(b: int, d_out: int, d_in: int, r: int) -> int:
    return int(lib().slim_noalloc_scratch_needed(b, d_out, d_in, r))


def slim_select_kernel(b: int, d_out: int, d_in: int, r: int) -> int:
    return int(lib().slim_select_kernel(b, d_out, d_in, r))


def slim_decode_layout_hint(b: int, d_out: int, d_in: int, r: int) -> int:
    return int(lib().slim_decode_layout_hint(b, d_out, d_in, r))


def slim_last_launch_count() -> int:
    return int(lib().slim_last_launch_count())


def slim_last_token_tile() -> int:
    return int(lib().slim_last_token_tile())


def new_workspace(b: int, d_out: int, d_in: int, r: int, device="cuda") -> torch.Tensor:
    """Allocate a workspace of the required size and initialise it (slim_workspace_reset)."""
    n = slim_workspace_bytes(b, d_out, d_in, r)
    if n == 0:
        raise SlimError(SLIM_ERR_UNSUPPORTED_SHAPE, "slim_workspace_bytes", "illegal shape")
    ws = torch.empty(n, dtype=torch.uint8, device=device)
    with torch.cuda.device(ws.device):
        slim_workspace_reset(ws)
    return ws


def slim_workspace_reset(workspace: torch.Tensor):
    _check(lib().slim_workspace_reset(_ptr(workspace), workspace.numel(), _stream()), "slim_workspace_reset")


def slim_linear_fwd(X, vals, meta, s: float, L, R, Y=None, workspace=None, status=None,
                    kernel: int = KERNEL_AUTO):
    """Y = X (s Q)^T + (X R^T) L^T on the current stream.  Returns Y (bf16 [b, d_out])."""
    _dev(X, torch.bfloat16, "X"), _dev(vals, torch.uint8, "vals"), _dev(meta, torch.uint8, "meta")
    b, d_in = X.shape
    d_out = vals.shape[0]
    r = 0 if L is None else L.shape[1]
    if r:
        _dev(L, torch.bfloat16, "L"), _dev(R, torch.bfloat16, "R")
        if tuple(L.shape) != (d_out, r) or tuple(R.shape) != (r, d_in):
            raise ValueError("adapter shapes do not match the weight")
    if vals.shape[1] * 4 != d_in or tuple(meta.shape) != (d_out, d_in // 8):
        raise ValueError("packed weight does not match X")
    if Y is None:
        Y = torch.empty((b, d_out), dtype=torch.bfloat16, device=X.device)
    if workspace is None:
        workspace = new_workspace(b, d_out, d_in, r, X.device)
    fn = lib().slim_linear_fwd_ex
    _check(fn(_ptr(X), b, _ptr(vals), _ptr(meta), float(s), _ptr(L) if r else None, _ptr(R) if r else None,
              r, d_out, d_in, _ptr(Y), _ptr(workspace), workspace.numel(), _ptr(status), _stream(), int(kernel)),
           "slim_linear_fwd")
    return Y


def slim_tiled_bytes(d_out: int, d_in: int, layout: int = LAYOUT_DECODE_TILED) -> int:
    return int(lib().slim_tiled_bytes(d_out, d_in, layout))


def slim_repack_tiled(vals: torch.Tensor, meta: torch.Tensor, layout: int = LAYOUT_DECODE_TILED, out=None) -> torch.Tensor:
    """(vals, meta) of slim_pack -> the decode-tiled copy (uint8, one flat buffer)."""
    _dev(vals, torch.uint8, "vals"), _dev(meta, torch.uint8, "meta")
    d_out, d_in = vals.shape[0], vals.shape[1] * 4
    n = slim_tiled_bytes(d_out, d_in, layout)
    if n == 0 or tuple(meta.shape) != (d_out, d_in // 8):
        raise SlimError(SLIM_ERR_UNSUPPORTED_SHAPE, "slim_repack_tiled", "shape cannot be tiled")
    if out is None:
        out = torch.empty(n, dtype=torch.uint8, device=vals.device)
    _check(lib().slim_repack_tiled(_ptr(vals), _ptr(meta), d_out, d_in, layout, _ptr(out), _stream()), "slim_repack_tiled")
    return out


def slim_linear_fwd_tiled(X, tiled, d_out: int, s: float, L, R, Y=None, workspace=None, status=None,
                          layout: int = LAYOUT_DECODE_TILED):
    """Small-batch forward on a decode-tiled weight.  Returns Y (bf16 [b, d_out])."""
    _dev(X, torch.bfloat16, "X"), _dev(tiled, torch.uint8, "tiled")
    b, d_in = X.shape
    r = 0 if L is None else L.shape[1]
    if r:
        _dev(L, torch.bfloat16, "L"), _dev(R, torch.bfloat16, "R")
        if tuple(L.shape) != (d_out, r) or tuple(R.shape) != (r, d_in):
            raise ValueError("adapter shapes do not match the weight")
    if tiled.numel() != slim_tiled_bytes(d_out, d_in, layout):
        raise ValueError("tiled weight does not match the shape")
    if Y is None:
        Y = torch.empty((b, d_out), dtype=torch.bfloat16, device=X.device)
    if workspace is None:
        workspace = new_workspace(b, d_out, d_in, r, X.device)
    _check(lib().slim_linear_fwd_tiled(_ptr(X), b, _ptr(tiled), layout, float(s), _ptr(L) if r else None,
                                       _ptr(R) if r else None, r, d_out, d_in, _ptr(Y), _ptr(workspace),
                                       workspace.numel(), _ptr(status), _stream()), "slim_linear_fwd_tiled")
    return Y


def slim_linear_fwd_tiled_host(X_host: torch.Tensor, tiled, d_out: int, s: float, L, R, Y_host: torch.Tensor,
                               x_dev, y_dev, workspace, status=None, layout: int = LAYOUT_DECODE_TILED):
    """Host-buffer form of :func:`slim_linear_fwd_tiled` (copies inside the call, stream synchronised)."""
    b, d_in = X_host.shape
    r = 0 if L is None else L.shape[1]
    _check(lib().slim_linear_fwd_tiled_host(ctypes.c_void_p(X_host.data_ptr()), b, _ptr(tiled), layout, float(s),
                                            _ptr(L) if r else None, _ptr(R) if r else None, r, d_out, d_in,
                                            ctypes.c_void_p(Y_host.data_ptr()), _ptr(x_dev), _ptr(y_dev),
                                            _ptr(workspace), workspace.numel(), _ptr(status), _stream()),
           "slim_linear_fwd_tiled_host")
    return Y_host


def slim_linear_fwd_host(X_host: torch.Tensor, vals, meta, s: float, L, R, Y_host: torch.Tensor,
                         x_dev, y_dev, workspace, status=None):
    """Host-buffer form: X_host / Y_host are (pinned) CPU bf16 tensors; copies
    run inside the call and the stream is synchronised before it returns."""
    b, d_in = X_host.shape
    d_out = vals.shape[0]
    r = 0 if L is None else L.shape[1]
    _check(lib().slim_linear_fwd_host(ctypes.c_void_p(X_host.data_ptr()), b, _ptr(vals), _ptr(meta), float(s),
                                      _ptr(L) if r else None, _ptr(R) if r else None, r, d_out, d_in,
                                      ctypes.c_void_p(Y_host.data_ptr()), _ptr(x_dev), _ptr(y_dev),
                                      _ptr(workspace), workspace.numel(), _ptr(status), _stream()),
           "slim_linear_fwd_host")
    return Y_host


def slim_linear_fwd_noalloc(X, vals, meta, s: float, L, R, Y, status=None):
    """Small-batch forward for callers that must not allocate device memory:
    the library's built-in scratch array replaces the workspace, and ``Y`` has
    to be supplied.  Calls on one device share that scratch, so keep them on one
    stream (or order them); overlapping calls corrupt each other."""
    _dev(X, torch.bfloat16, "X"), _dev(vals, torch.uint8, "vals"), _dev(meta, torch.uint8, "meta")
    _dev(Y, torch.bfloat16, "Y")
    b, d_in = X.shape
    d_out = vals.shape[0]
    r = 0 if L is None else L.shape[1]
    if tuple(Y.shape) != (b, d_out) or vals.shape[1] * 4 != d_in or tuple(meta.shape) != (d_out, d_in // 8):
        raise ValueError("shapes do not match")
    if r and (tuple(L.shape) != (d_out, r) or tuple(R.shape) != (r, d_in)):
        raise ValueError("adapter shapes do not match the weight")
    _check(lib().slim_linear_fwd_noalloc(_ptr(X), b, _ptr(vals), _ptr(meta), float(s), _ptr(L) if r else None,
                                         _ptr(R) if r else None, r, d_out, d_in, _ptr(Y), _ptr(status), _stream()),
           "slim_linear_fwd_noalloc")
    return Y


def slim_pack_adapter(A: torch.Tensor):
    """bf16 adapter [rows, cols] -> (codes uint8 [rows, cols / 2], scales bf16 [rows, ceil(cols / 128)])."""
    _dev(A, torch.bfloat16, "A")
    rows, cols = A.shape
    if lib().slim_adapter_code_bytes(rows, cols) == 0:
        raise SlimError(SLIM_ERR_INVALID_ARG, "slim_pack_adapter", "illegal adapter shape")
    codes = torch.empty((rows, cols // 2), dtype=torch.uint8, device=A.device)
    scales = torch.empty((rows, (cols + 127) // 128), dtype=torch.bfloat16, device=A.device)
    _check(lib().slim_pack_adapter(_ptr(A), rows, cols, _ptr(codes), _ptr(scales), _stream()), "slim_pack_adapter")
    return codes, scales


def slim_unpack_adapter(codes: torch.Tensor, scales: torch.Tensor) -> torch.Tensor:
    """The bf16 matrix nearest to what codes and scales stand for."""
    _dev(codes, torch.uint8, "codes"), _dev(scales, torch.bfloat16, "scales")
    rows, cols = codes.shape[0], codes.shape[1] * 2
    out = torch.empty((rows, cols), dtype=torch.bfloat16, device=codes.device)
    _check(lib().slim_unpack_adapter(_ptr(codes), _ptr(scales), rows, cols, _ptr(out), _stream()), "slim_unpack_adapter")
    return out


def slim_workspace_bytes_q(b: int, d_out: int, d_in: int, r: int) -> int:
    return int(lib().slim_workspace_bytes_q(b, d_out, d_in, r))


def slim_linear_fwd_q(X, vals, meta, s: float, Lq, Ls, Rq, Rs, Y=None, workspace=None, status=None):
    """Layer forward with quantized adapters.  Returns Y (bf16 [b, d_out])."""
    _dev(X, torch.bfloat16, "X"), _dev(vals, torch.uint8, "vals"), _dev(meta, torch.uint8, "meta")
    for name, t, dt in (("Lq", Lq, torch.uint8), ("Ls", Ls, torch.bfloat16), ("Rq", Rq, torch.uint8), ("Rs", Rs, torch.bfloat16)):
        _dev(t, dt, name)
    b, d_in = X.shape
    d_out, r = vals.shape[0], Lq.shape[1] * 2
    if tuple(Lq.shape) != (d_out, r // 2) or tuple(Rq.shape) != (r, d_in // 2):
        raise ValueError("adapter code shapes do not match the weight")
    if Y is None:
        Y = torch.empty((b, d_out), dtype=torch.bfloat16, device=X.device)
    if workspace is None:
        n = slim_workspace_bytes_q(b, d_out, d_in, r)
        if n == 0:
            raise SlimError(SLIM_ERR_UNSUPPORTED_SHAPE, "slim_workspace_bytes_q", "illegal shape")
        workspace = torch.empty(n, dtype=torch.uint8, device=X.device)
        with torch.cuda.device(X.device):
            slim_workspace_reset(workspace)
    _check(lib().slim_linear_fwd_q(_ptr(X), b, _ptr(vals), _ptr(meta), float(s), _ptr(Lq), _ptr(Ls), _ptr(Rq), _ptr(Rs), r,
                                   d_out, d_in, _ptr(Y), _ptr(workspace), workspace.numel(), _ptr(status), _stream()),
           "slim_linear_fwd_q")
    return Y


def slim_quant(W: torch.Tensor, status=None):
    """SLiM-Quant on a float32 matrix: (codes int8 like W, scale_alpha float32[2] on the device = (s, alpha*),
    table float64 [29, 2] of the candidates tried, alpha* as float64)."""
    _dev(W, torch.float32, "W")
    d_out, d_in = W.shape
    n = int(lib().slim_quant_workspace_bytes(d_out, d_in))
    ws = torch.empty(n, dtype=torch.uint8, device=W.device)
    codes = torch.empty((d_out, d_in), dtype=torch.int8, device=W.device)
    sa = torch.empty(4, dtype=torch.float32, device=W.device)
    _check(lib().slim_quant(_ptr(W), d_out, d_in, _ptr(codes), _ptr(sa), _ptr(ws), n, _ptr(status), _stream()), "slim_quant")
    bins = max(512, min(d_out * d_in // 1000, 20000))
    off = 256 + (bins * 4 + 255) // 256 * 256
    tab = ws[off:off + 59 * 8].view(torch.float64)
    return codes, sa[:2], tab[:58].view(29, 2), tab[58]


def slim_mask_top2(codes: torch.Tensor, xbar=None, status=None) -> torch.Tensor:
    """2:4 mask (uint8, like codes) of int8 codes; xbar: float32 [d_in] average input magnitudes, or None."""
    _dev(codes, torch.int8, "codes")
    d_out, d_in = codes.shape
    if xbar is not None:
        _dev(xbar, torch.float32, "xbar")
    mask = torch.empty((d_out, d_in), dtype=torch.uint8, device=codes.device)
    _check(lib().slim_mask_top2(_ptr(codes), _ptr(xbar), d_out, d_in, _ptr(mask), _ptr(status), _stream()), "slim_mask_top2")
    return mask
