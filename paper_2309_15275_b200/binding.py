"""ctypes binding of liblbp.so: argument marshalling only.

Every function mirrors one entry point of include/lbp.h.  Tensors are torch
CUDA tensors used as device-memory handles (data_ptr) -- all arithmetic runs in
the library's kernels.  There is no CPU or eager fallback: if the shared library
is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Sequence, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# LBP_LIBRARY selects another build of the same library (a diagnostic variant)
LIB_PATH = os.environ.get("LBP_LIBRARY") or os.path.join(_HERE, "liblbp.so")

LBP_F32, LBP_BF16 = 0, 1
SEL_L1, SEL_LINF, SEL_PREFIX = 0, 1, 2
LBP_OK = 0


class LbpError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = _lib().lbp_status_string(status).decode()
        if status == 9:
            msg += f" (cudaError {_lib().lbp_last_cuda_error()})"
        super().__init__(f"{where}: {msg} [status {status}]")


class Basis(C.Structure):
    _fields_ = [("i", C.c_int32), ("j", C.c_int32)]


class Layer(C.Structure):
    _fields_ = [("B", C.c_int32), ("H", C.c_int32), ("W", C.c_int32),
                ("Cin", C.c_int32), ("Cout", C.c_int32), ("k", C.c_int32),
                ("dtype", C.c_int32), ("gw_dtype", C.c_int32)]


class View(C.Structure):
    _fields_ = [("image", C.c_int64), ("row", C.c_int64), ("token", C.c_int64)]


class Extras(C.Structure):
    _fields_ = [("beta", C.c_float), ("g_bias", C.c_void_p), ("n_extra", C.c_int32),
                ("x_extra", C.c_void_p), ("gy_extra", C.c_void_p), ("gx_extra", C.c_void_p),
                ("x_view", View), ("gy_view", View), ("gx_view", View),
                ("x_extra_pitch", C.c_int64), ("gy_extra_pitch", C.c_int64),
                ("gx_extra_pitch", C.c_int64)]


_LIB = None


def _lib() -> C.CDLL:
    global _LIB
    if _LIB is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with "
                "`python -m paper_2309_15275_b200.build` (there is no fallback path)")
        lib = C.CDLL(LIB_PATH)
        vp, sz, i32 = C.c_void_p, C.c_size_t, C.c_int
        lib.lbp_select_bases.argtypes = [i32, i32, i32, C.POINTER(Basis), i32, C.POINTER(i32)]
        lib.lbp_select_bases.restype = i32
        lib.lbp_basis_matrix.argtypes = [i32, C.POINTER(Basis), i32, C.POINTER(C.c_int8)]
        lib.lbp_basis_matrix.restype = i32
        lib.lbp_flops.argtypes = [i32, i32, C.c_longlong, i32, i32]
        lib.lbp_flops.restype = C.c_double
        lib.lbp_status_string.argtypes = [i32]
        lib.lbp_status_string.restype = C.c_char_p
        lib.lbp_last_cuda_error.argtypes = []
        lib.lbp_last_cuda_error.restype = i32
        lib.lbp_workspace_bytes.argtypes = [C.POINTER(Layer), i32]
        lib.lbp_workspace_bytes.restype = sz
        lib.lbp_status_bytes.argtypes = []
        lib.lbp_status_bytes.restype = sz
        lib.lbp_select_lhe.argtypes = [C.POINTER(C.c_double), i32, i32, C.POINTER(Basis)]
        lib.lbp_select_lhe.restype = i32
        lib.lbp_spectrum_workspace_bytes.argtypes = [i32, i32, i32, i32, i32, i32]
        lib.lbp_spectrum_workspace_bytes.restype = sz
        lib.lbp_spectrum.argtypes = [vp, vp, i32, i32, i32, i32, i32, i32, vp, sz, vp]
        lib.lbp_spectrum.restype = i32
        for name in ("lbp_project", "lbp_expand"):
            f = getattr(lib, name)
            f.argtypes = [vp, vp, i32, i32, i32, i32, i32, C.POINTER(Basis), i32, i32, vp, sz, vp]
            f.restype = i32
        lib.lbp_backward.argtypes = [vp, vp, vp, vp, vp, C.POINTER(Layer), C.POINTER(Basis), i32,
                                     vp, sz, vp]
        lib.lbp_backward.restype = i32
        lib.lbp_workspace_bytes_ex.argtypes = [C.POINTER(Layer), i32, C.POINTER(Extras)]
        lib.lbp_workspace_bytes_ex.restype = sz
        lib.lbp_backward_ex.argtypes = [vp, vp, vp, vp, vp, vp, C.POINTER(Layer), C.POINTER(Basis),
                                        i32, C.POINTER(Extras), vp, sz, vp]
        lib.lbp_backward_ex.restype = i32
        lib.lbp_backward_projected.argtypes = [vp, vp, vp, vp, vp, C.POINTER(Layer),
                                               C.POINTER(Basis), i32, vp, sz, vp]
        lib.lbp_backward_projected.restype = i32
        lib.lbp_backward_batch.argtypes = [i32, C.POINTER(vp), C.POINTER(vp), C.POINTER(vp),
                                           C.POINTER(vp), C.POINTER(vp), C.POINTER(Layer),
                                           C.POINTER(Basis), i32, C.POINTER(vp), C.POINTER(sz),
                                           C.POINTER(vp), vp]
        lib.lbp_backward_batch.restype = i32
        lib.lbp_backward_fullrank.argtypes = [vp, vp, vp, vp, vp, C.POINTER(Layer), vp, sz, vp]
        lib.lbp_backward_fullrank.restype = i32
        lib.lbp_poll_status.argtypes = [vp, vp]
        lib.lbp_poll_status.restype = i32
        lib.lbp_backward_static.argtypes = [vp, vp, vp, vp, vp, C.POINTER(Layer), C.POINTER(Basis),
                                            i32, vp]
        lib.lbp_backward_static.restype = i32
        lib.lbp_test_tile_plan.argtypes = [i32] * 9 + [C.POINTER(C.c_int32), C.POINTER(C.c_uint16),
                                                       C.POINTER(C.c_uint16)]
        lib.lbp_test_tile_plan.restype = i32
        lib.lbp_test_reload_env.argtypes = []
        lib.lbp_test_reload_env.restype = i32
        lib.lbp_test_struct_size.argtypes = [i32]
        lib.lbp_test_struct_size.restype = sz
        lib.lbp_test_stall_products.argtypes = [i32]
        lib.lbp_test_stall_products.restype = i32
        lib.lbp_launch_count.argtypes = []
        lib.lbp_launch_count.restype = C.c_longlong
        lib.lbp_set_phase_events.argtypes = [C.POINTER(vp), i32]
        lib.lbp_set_phase_events.restype = i32
        lib.lbp_phase_count.argtypes = []
        lib.lbp_phase_count.restype = i32
        lib.lbp_phase_name.argtypes = [i32]
        lib.lbp_phase_name.restype = C.c_char_p
        _LIB = lib
    return _LIB


EXPORTED = ("lbp_select_bases", "lbp_basis_matrix", "lbp_flops", "lbp_status_string",
            "lbp_last_cuda_error", "lbp_workspace_bytes", "lbp_status_bytes", "lbp_project",
            "lbp_expand", "lbp_backward", "lbp_backward_fullrank", "lbp_poll_status",
            "lbp_backward_static", "lbp_launch_count", "lbp_set_phase_events", "lbp_phase_count",
            "lbp_phase_name", "lbp_select_lhe", "lbp_spectrum_workspace_bytes", "lbp_spectrum",
            "lbp_backward_batch", "lbp_test_stall_products",
            "lbp_test_reload_env", "lbp_workspace_bytes_ex", "lbp_backward_ex",
            "lbp_backward_projected", "lbp_test_tile_plan", "lbp_test_struct_size")


def _check(status: int, where: str) -> None:
    if status != LBP_OK:
        raise LbpError(status, where)


def _bases(bases: Sequence[Tuple[int, int]]):
    arr = (Basis * max(len(bases), 1))()
    for q, (i, j) in enumerate(bases):
        arr[q].i, arr[q].j = int(i), int(j)
    return arr


def _dtype_code(t: torch.dtype) -> int:
    if t == torch.float32:
        return LBP_F32
    if t == torch.bfloat16:
        return LBP_BF16
    raise TypeError(f"unsupported dtype {t}")


def _dev(t: torch.Tensor, name: str) -> int:
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor (the library has no CPU path)")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    return t.data_ptr()


def _dev_view(t: torch.Tensor, name: str):
    """Pointer and element strides of a (B,H,W,C) tensor that may be a view of a
    larger one (channels contiguous); (0, 0, 0) stands for dense."""
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor (the library has no CPU path)")
    if t.is_contiguous():
        return t.data_ptr(), (0, 0, 0)
    B, H, Wd, Cc = t.shape
    if Cc > 1 and t.stride(3) != 1:
        raise ValueError(f"{name}: the channels of a token must be contiguous")
    tok = t.stride(2) if Wd > 1 else Cc
    row = t.stride(1) if H > 1 else Wd * tok
    img = t.stride(0) if B > 1 else H * row
    return t.data_ptr(), (img, row, tok)


def _dev_rows(t: torch.Tensor, name: str):
    """Pointer and row pitch (elements; 0 = dense) of an (n, C) matrix."""
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor (the library has no CPU path)")
    if t.is_contiguous():
        return t.data_ptr(), 0
    if t.shape[1] > 1 and t.stride(1) != 1:
        raise ValueError(f"{name}: the channels of a token must be contiguous")
    return t.data_ptr(), (t.stride(0) if t.shape[0] > 1 else 0)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


# ------------------------------------------------------------ host helpers ----
def lbp_select_bases(k: int, rule: int, param: int) -> List[Tuple[int, int]]:
    out = (Basis * 256)()
    r = C.c_int(0)
    _check(_lib().lbp_select_bases(k, rule, param, out, 256, C.byref(r)), "lbp_select_bases")
    return [(out[q].i, out[q].j) for q in range(r.value)]


def lbp_basis_matrix(k: int, bases: Sequence[Tuple[int, int]]):
    import numpy as np
    r = len(bases)
    buf = (C.c_int8 * (k * k * max(r, 1)))()
    _check(_lib().lbp_basis_matrix(k, _bases(bases), r, buf), "lbp_basis_matrix")
    return np.frombuffer(buf, dtype=np.int8).reshape(k * k, r).copy()


def lbp_flops(Cin: int, Cout: int, L: int, r: int, which: int) -> float:
    return float(_lib().lbp_flops(Cin, Cout, L, r, which))


def lbp_status_string(status: int) -> str:
    return _lib().lbp_status_string(status).decode()


def lbp_status_bytes() -> int:
    return int(_lib().lbp_status_bytes())


def _layer(B, H, W, Cin, Cout, k, dtype, gw_dtype) -> Layer:
    return Layer(B, H, W, Cin, Cout, k, dtype, gw_dtype)


def lbp_workspace_bytes(B, H, W, Cin, Cout, k, dtype: int, gw_dtype: int, r: int) -> int:
    lay = _layer(B, H, W, Cin, Cout, k, dtype, gw_dtype)
    return int(_lib().lbp_workspace_bytes(C.byref(lay), r))


# ---------------------------------------------------------- device calls ----
def _status_ws(device) -> torch.Tensor:
    return torch.empty(lbp_status_bytes(), dtype=torch.uint8, device=device)


def lbp_project(t: torch.Tensor, k: int, bases, out: torch.Tensor | None = None,
                ws: torch.Tensor | None = None) -> torch.Tensor:
    """t (B,H,W,C) -> t_hat (B,ceil(H/k),ceil(W/k),r,C)."""
    B, H, W, Cc = t.shape
    r = len(bases)
    if out is None:
        kk = max(k, 1)
        out = torch.empty((B, -(-H // kk), -(-W // kk), r, Cc), dtype=t.dtype, device=t.device)
    if ws is None:
        ws = _status_ws(t.device)
    _check(_lib().lbp_project(_dev(t, "t"), _dev(out, "t_hat"), B, H, W, Cc, k, _bases(bases), r,
                              _dtype_code(t.dtype), _dev(ws, "ws"), ws.numel(), _stream()),
           "lbp_project")
    return out


def lbp_select_lhe(energy, k: int, r: int) -> List[Tuple[int, int]]:
    """The r bases with the largest energy (k x k array as returned by lbp_spectrum)."""
    flat = [float(v) for v in (energy.reshape(-1).tolist() if hasattr(energy, "reshape") else energy)]
    if len(flat) != k * k:
        raise ValueError("energy must hold k*k values")
    buf = (C.c_double * (k * k))(*flat)
    out = (Basis * max(r, 1))()
    _check(_lib().lbp_select_lhe(buf, k, r, out), "lbp_select_lhe")
    return [(out[q].i, out[q].j) for q in range(r)]


def lbp_spectrum_workspace_bytes(B: int, H: int, W: int, Cc: int, k: int, dtype_code: int) -> int:
    return int(_lib().lbp_spectrum_workspace_bytes(B, H, W, Cc, k, dtype_code))


def lbp_spectrum(t: torch.Tensor, k: int, out: torch.Tensor | None = None,
                 ws: torch.Tensor | None = None) -> torch.Tensor:
    """t (B,H,W,C) -> energy (k, k) float64 on the device: sum of squares of every basis response."""
    B, H, W, Cc = t.shape
    if out is None:
        out = torch.empty((k, k), dtype=torch.float64, device=t.device)
    if ws is None:
        n = lbp_spectrum_workspace_bytes(B, H, W, Cc, k, _dtype_code(t.dtype))
        if n == 0:
            raise ValueError("invalid shape for lbp_spectrum_workspace_bytes")
        ws = torch.empty(n, dtype=torch.uint8, device=t.device)
    _check(_lib().lbp_spectrum(_dev(t, "t"), _dev(out, "energy"), B, H, W, Cc, k,
                               _dtype_code(t.dtype), _dev(ws, "ws"), ws.numel(), _stream()),
           "lbp_spectrum")
    return out


def lbp_expand(t_hat: torch.Tensor, k: int, bases, out: torch.Tensor | None = None,
               ws: torch.Tensor | None = None, grid: Tuple[int, int] | None = None) -> torch.Tensor:
    """t_hat (B,ceil(H/k),ceil(W/k),r,C) -> t (B,H,W,C).  grid = (H, W) when the
    grid sides are not multiples of k (default: Hb * k, Wb * k)."""
    B, Hb, Wb, r, Cc = t_hat.shape
    H, W = grid if grid is not None else (Hb * k, Wb * k)
    if -(-H // max(k, 1)) != Hb or -(-W // max(k, 1)) != Wb:
        raise ValueError("grid does not match the block grid of t_hat")
    if out is None:
        out = torch.empty((B, H, W, Cc), dtype=t_hat.dtype, device=t_hat.device)
    if ws is None:
        ws = _status_ws(t_hat.device)
    _check(_lib().lbp_expand(_dev(t_hat, "t_hat"), _dev(out, "t"), B, H, W, Cc, k,
                             _bases(bases), len(bases), _dtype_code(t_hat.dtype),
                             _dev(ws, "ws"), ws.numel(), _stream()),
           "lbp_expand")
    return out


def alloc_workspace(x: torch.Tensor, g_y: torch.Tensor, k: int, r: int,
                    gw_dtype: torch.dtype = torch.float32) -> torch.Tensor:
    B, H, W, Cin = x.shape
    n = lbp_workspace_bytes(B, H, W, Cin, g_y.shape[-1], k, _dtype_code(x.dtype),
                            _dtype_code(gw_dtype), r)
    if n == 0:
        raise ValueError("invalid layer for lbp_workspace_bytes")
    return torch.empty(n, dtype=torch.uint8, device=x.device)


def _check_layer_tensors(g_y, W, g_x, g_W, Cin: int, x=None, x_hat=None, k=None, r=None):
    """Shapes, dtypes and devices of one backward problem, before the C call: the
    library sees raw pointers and would read a short or mistyped buffer as it is."""
    if g_y.dim() != 4:
        raise ValueError("g_y must be (B, H, W, Cout)")
    B, H, Wd, Cout = g_y.shape
    dt, dev = g_y.dtype, g_y.device
    if x is not None and tuple(x.shape) != (B, H, Wd, Cin):
        raise ValueError(f"x {tuple(x.shape)} does not match g_y {tuple(g_y.shape)} and Cin {Cin}")
    if x_hat is not None:
        want = (B, -(-H // max(k, 1)), -(-Wd // max(k, 1)), r, Cin)
        if tuple(x_hat.shape) != want:
            raise ValueError(f"x_hat {tuple(x_hat.shape)} must be {want}")
    if tuple(W.shape) != (Cout, Cin):
        raise ValueError(f"W {tuple(W.shape)} must be (Cout, Cin) = ({Cout}, {Cin})")
    if g_x is not None and tuple(g_x.shape) != (B, H, Wd, Cin):
        raise ValueError(f"g_x {tuple(g_x.shape)} must be {(B, H, Wd, Cin)}")
    if g_W is not None and tuple(g_W.shape) != (Cout, Cin):
        raise ValueError(f"g_W {tuple(g_W.shape)} must be ({Cout}, {Cin})")
    for name, t in (("x", x), ("x_hat", x_hat), ("W", W), ("g_x", g_x)):
        if t is not None and t.dtype != dt:
            raise ValueError(f"{name} is {t.dtype}, g_y is {dt}: one dtype per layer")
    for name, t in (("x", x), ("x_hat", x_hat), ("W", W), ("g_x", g_x), ("g_W", g_W)):
        if t is not None and t.device != dev:
            raise ValueError(f"{name} is on {t.device}, g_y on {dev}")
    if dev.type == "cuda" and dev.index is not None and dev.index != torch.cuda.current_device():
        raise ValueError(f"tensors are on {dev}, the current device is cuda:{torch.cuda.current_device()}")


def lbp_backward(x, g_y, W, k: int, bases, *, gw_dtype: torch.dtype = torch.float32,
                 g_x=None, g_W=None, ws=None):
    """Algorithm 1.  Returns (g_x (B,H,W,Cin), g_W (Cout,Cin))."""
    if x.dim() != 4:
        raise ValueError("x must be (B, H, W, Cin)")
    B, H, Wd, Cin = x.shape
    Cout = g_y.shape[-1]
    r = len(bases)
    _check_layer_tensors(g_y, W, g_x, g_W, Cin, x=x)
    if g_x is None:
        g_x = torch.empty_like(x)
    if g_W is None:
        g_W = torch.empty((Cout, Cin), dtype=gw_dtype, device=x.device)
    if ws is None:
        ws = alloc_workspace(x, g_y, k, r, g_W.dtype)
    lay = _layer(B, H, Wd, Cin, Cout, k, _dtype_code(x.dtype), _dtype_code(g_W.dtype))
    _check(_lib().lbp_backward(_dev(x, "x"), _dev(g_y, "g_y"), _dev(W, "W"), _dev(g_x, "g_x"),
                               _dev(g_W, "g_W"), C.byref(lay), _bases(bases), r,
                               _dev(ws, "ws"), ws.numel(), _stream()),
           "lbp_backward")
    return g_x, g_W


def _extras(g_y, Cin, beta, g_bias, x_extra, gy_extra, gx_extra):
    Cout = g_y.shape[-1]
    ex = Extras()
    ex.beta = float(beta)
    if g_bias is not None:
        if g_bias.dtype != torch.float32 or tuple(g_bias.shape) != (Cout,):
            raise ValueError("g_bias must be fp32 of shape (Cout,)")
        ex.g_bias = _dev(g_bias, "g_bias")
    n = 0
    if x_extra is not None or gy_extra is not None:
        if x_extra is None or gy_extra is None or gx_extra is None:
            raise ValueError("x_extra, gy_extra and gx_extra go together")
        n = x_extra.shape[0]
        if (tuple(x_extra.shape) != (n, Cin) or tuple(gy_extra.shape) != (n, Cout)
                or tuple(gx_extra.shape) != (n, Cin)):
            raise ValueError("extra tokens must be (n, Cin), (n, Cout), (n, Cin)")
        for t in (x_extra, gy_extra, gx_extra):
            if t.dtype != g_y.dtype or t.device != g_y.device:
                raise ValueError("extra tokens must have the layer's dtype and device")
        if n > 0:
            ex.x_extra, ex.x_extra_pitch = _dev_rows(x_extra, "x_extra")
            ex.gy_extra, ex.gy_extra_pitch = _dev_rows(gy_extra, "gy_extra")
            ex.gx_extra, ex.gx_extra_pitch = _dev_rows(gx_extra, "gx_extra")
    ex.n_extra = n
    return ex


def lbp_workspace_bytes_ex(B, H, W, Cin, Cout, k, dtype: int, gw_dtype: int, r: int, *, beta=0.0,
                           bias=False, n_extra=0, x_view=None, gy_view=None, gx_view=None,
                           extra_pitches=None) -> int:
    """Scratch of lbp_backward_ex.  Views are (image, row, token) element strides,
    extra_pitches the (x, g_y, g_x) row pitches of the extra tokens."""
    lay = _layer(B, H, W, Cin, Cout, k, dtype, gw_dtype)
    ex = Extras()
    ex.beta, ex.n_extra = float(beta), 0
    # sizes only: the pointers are not looked at beyond NULL / non-NULL
    ex.g_bias = 16 if bias else None
    if n_extra:
        ex.n_extra, ex.x_extra, ex.gy_extra, ex.gx_extra = int(n_extra), 16, 16, 16
        if extra_pitches is not None:
            ex.x_extra_pitch, ex.gy_extra_pitch, ex.gx_extra_pitch = (int(v) for v in extra_pitches)
    for name, v in (("x_view", x_view), ("gy_view", gy_view), ("gx_view", gx_view)):
        if v is not None:
            setattr(ex, name, View(*[int(a) for a in v]))
    return int(_lib().lbp_workspace_bytes_ex(C.byref(lay), r, C.byref(ex)))


def lbp_backward_ex(x, g_y, W, k: int, bases, *, x_hat=None, beta: float = 0.0, g_bias=None,
                    x_extra=None, gy_extra=None, gx_extra=None,
                    gw_dtype: torch.dtype = torch.float32, g_x=None, g_W=None, ws=None):
    """Algorithm 1 with what a ViT layer needs around it: accumulation into g_W
    (beta), the bias gradient, tokens outside the grid (Eq. 2), and x_hat = p(x)
    handed in instead of x (pass x=None).  Returns (g_x, g_W)."""
    if (x is None) == (x_hat is None):
        raise ValueError("give exactly one of x and x_hat")
    B, H, Wd, Cout = g_y.shape
    r = len(bases)
    Cin = (x if x is not None else x_hat).shape[-1]
    _check_layer_tensors(g_y, W, g_x, g_W, Cin, x=x, x_hat=x_hat, k=k, r=r)
    if g_x is None:
        g_x = torch.empty((B, H, Wd, Cin), dtype=g_y.dtype, device=g_y.device)
    if g_W is None:
        if beta != 0.0:
            raise ValueError("beta != 0 accumulates into g_W: pass it")
        g_W = torch.empty((Cout, Cin), dtype=gw_dtype, device=g_y.device)
    ex = _extras(g_y, Cin, beta, g_bias, x_extra, gy_extra, gx_extra)
    # x, g_y and g_x may be views of larger tensors (the tokens behind a class
    # token, a channel slice): their strides go to the library as they are
    px = None
    if x is not None:
        px, v = _dev_view(x, "x")
        ex.x_view = View(*v)
    pgy, v = _dev_view(g_y, "g_y")
    ex.gy_view = View(*v)
    pgx, v = _dev_view(g_x, "g_x")
    ex.gx_view = View(*v)
    lay = _layer(B, H, Wd, Cin, Cout, k, _dtype_code(g_y.dtype), _dtype_code(g_W.dtype))
    if ws is None:
        n = int(_lib().lbp_workspace_bytes_ex(C.byref(lay), r, C.byref(ex)))
        if n == 0:
            raise ValueError("invalid layer, strides or extras for lbp_workspace_bytes_ex")
        ws = torch.empty(n, dtype=torch.uint8, device=g_y.device)
    _check(_lib().lbp_backward_ex(px, None if x_hat is None else _dev(x_hat, "x_hat"),
                                  pgy, _dev(W, "W"), pgx, _dev(g_W, "g_W"),
                                  C.byref(lay), _bases(bases), r, C.byref(ex), _dev(ws, "ws"),
                                  ws.numel(), _stream()),
           "lbp_backward_ex")
    return g_x, g_W


def lbp_backward_projected(x_hat, g_y, W, k: int, bases, *, gw_dtype: torch.dtype = torch.float32,
                           g_x=None, g_W=None, ws=None):
    """Algorithm 1 from its second step on: x_hat = lbp_project(x, k, bases) was
    taken at forward time (Eq. 3).  Returns (g_x, g_W)."""
    B, H, Wd, Cout = g_y.shape
    r = len(bases)
    Cin = x_hat.shape[-1]
    _check_layer_tensors(g_y, W, g_x, g_W, Cin, x_hat=x_hat, k=k, r=r)
    if g_x is None:
        g_x = torch.empty((B, H, Wd, Cin), dtype=g_y.dtype, device=g_y.device)
    if g_W is None:
        g_W = torch.empty((Cout, Cin), dtype=gw_dtype, device=g_y.device)
    lay = _layer(B, H, Wd, Cin, Cout, k, _dtype_code(g_y.dtype), _dtype_code(g_W.dtype))
    if ws is None:
        n = int(_lib().lbp_workspace_bytes(C.byref(lay), r))
        if n == 0:
            raise ValueError("invalid layer for lbp_workspace_bytes")
        ws = torch.empty(n, dtype=torch.uint8, device=g_y.device)
    _check(_lib().lbp_backward_projected(_dev(x_hat, "x_hat"), _dev(g_y, "g_y"), _dev(W, "W"),
                                         _dev(g_x, "g_x"), _dev(g_W, "g_W"), C.byref(lay),
                                         _bases(bases), r, _dev(ws, "ws"), ws.numel(), _stream()),
           "lbp_backward_projected")
    return g_x, g_W


def lbp_backward_batch(xs, g_ys, Ws, k: int, bases, *, g_xs, g_Ws, wss, done_events=None):
    """Algorithm 1 for several independent layers in one call (same k and bases).
    Every argument is a list with one tensor per layer; outputs and workspaces are
    the caller's and must not overlap anything of another layer.  done_events: an
    optional list of torch.cuda.Event (or None entries), one per layer, recorded
    behind that layer's last kernel."""
    n = len(xs)
    lays = (Layer * n)()
    for i in range(n):
        _check_layer_tensors(g_ys[i], Ws[i], g_xs[i], g_Ws[i], xs[i].shape[-1], x=xs[i])
        B, H, Wd, Cin = xs[i].shape
        lays[i] = _layer(B, H, Wd, Cin, g_ys[i].shape[-1], k, _dtype_code(xs[i].dtype),
                         _dtype_code(g_Ws[i].dtype))

    def ptrs(ts, name):
        return (C.c_void_p * n)(*[_dev(t, name) for t in ts])
    sizes = (C.c_size_t * n)(*[w.numel() for w in wss])
    evs = None
    if done_events is not None:
        if len(done_events) != n:
            raise ValueError("done_events needs one entry per layer")
        for e in done_events:
            if e is not None and not e.cuda_event:
                e.record()          # a torch event has no handle before its first record
        evs = (C.c_void_p * n)(*[None if e is None else e.cuda_event for e in done_events])
    _check(_lib().lbp_backward_batch(n, ptrs(xs, "x"), ptrs(g_ys, "g_y"), ptrs(Ws, "W"),
                                     ptrs(g_xs, "g_x"), ptrs(g_Ws, "g_W"), lays, _bases(bases),
                                     len(bases), ptrs(wss, "ws"), sizes, evs, _stream()),
           "lbp_backward_batch")
    return g_xs, g_Ws


def lbp_backward_fullrank(x, g_y, W, k: int, *, gw_dtype: torch.dtype = torch.float32,
                          g_x=None, g_W=None, ws=None):
    """Eq. 2, exact backpropagation (the r = k*k mode)."""
    B, H, Wd, Cin = x.shape
    Cout = g_y.shape[-1]
    _check_layer_tensors(g_y, W, g_x, g_W, Cin, x=x)
    if g_x is None:
        g_x = torch.empty_like(x)
    if g_W is None:
        g_W = torch.empty((Cout, Cin), dtype=gw_dtype, device=x.device)
    if ws is None:
        ws = alloc_workspace(x, g_y, k, k * k, g_W.dtype)
    lay = _layer(B, H, Wd, Cin, Cout, k, _dtype_code(x.dtype), _dtype_code(g_W.dtype))
    _check(_lib().lbp_backward_fullrank(_dev(x, "x"), _dev(g_y, "g_y"), _dev(W, "W"),
                                        _dev(g_x, "g_x"), _dev(g_W, "g_W"), C.byref(lay),
                                        _dev(ws, "ws"), ws.numel(), _stream()),
           "lbp_backward_fullrank")
    return g_x, g_W


STATIC_SCRATCH_BYTES = 32 * 1024 * 1024


def lbp_backward_static(x, g_y, W, k: int, bases, *, g_x, g_W):
    """lbp_backward on the scratch array built into the library: no workspace
    argument and no allocation inside the call.  The caller passes the output
    tensors g_x (B,H,W,Cin) and g_W (Cout,Cin); layers whose scratch need exceeds
    STATIC_SCRATCH_BYTES raise LbpError (status 7)."""
    B, H, Wd, Cin = x.shape
    Cout = g_y.shape[-1]
    _check_layer_tensors(g_y, W, g_x, g_W, Cin, x=x)
    lay = _layer(B, H, Wd, Cin, Cout, k, _dtype_code(x.dtype), _dtype_code(g_W.dtype))
    _check(_lib().lbp_backward_static(_dev(x, "x"), _dev(g_y, "g_y"), _dev(W, "W"),
                                      _dev(g_x, "g_x"), _dev(g_W, "g_W"), C.byref(lay),
                                      _bases(bases), len(bases), _stream()),
           "lbp_backward_static")
    return g_x, g_W


def lbp_poll_status(ws: torch.Tensor) -> int:
    """Synchronises the current stream and returns the device status (0 = ok)."""
    return int(_lib().lbp_poll_status(_dev(ws, "ws"), _stream()))


def lbp_test_tile_plan(Cin, Cout, G, bpt, k, units, pair, max_splits=1, epi_kind=0):
    """Test hook: the host-side tile plan of the products kernel.  Returns
    (dict of tile sizes, list of per-unit tile-id lists or None when not listed)."""
    out = (C.c_int32 * 6)()
    first = (C.c_uint16 * 161)()
    ids = (C.c_uint16 * 1536)()
    _check(_lib().lbp_test_tile_plan(Cin, Cout, G, bpt, k, units, 1 if pair else 0, max_splits,
                                     epi_kind, out, first, ids), "lbp_test_tile_plan")
    info = {"BNw": out[0], "BNx": out[1], "splits": out[2], "kbps": out[3], "listed": bool(out[4])}
    if not info["listed"]:
        return info, None
    return info, [[ids[j] for j in range(first[u], first[u + 1])] for u in range(units)]


def lbp_test_reload_env() -> None:
    """Test hook: the library reads its LBP_* tuning switches from the environment again."""
    _check(_lib().lbp_test_reload_env(), "lbp_test_reload_env")


def lbp_test_stall_products(on, projection: bool = False) -> None:
    """Test hook (include/lbp_test_hooks.h): while on, the products kernel's TMA
    producers (with `projection`: those of the tcgen05 projection kernel) issue
    nothing, so the call ends in LBP_ERR_TIMEOUT (lbp_poll_status)."""
    mode = (2 if projection else 1) if on else 0
    _check(_lib().lbp_test_stall_products(mode), "lbp_test_stall_products")


# ------------------------------------------------------ measurement hooks ----
def lbp_launch_count() -> int:
    return int(_lib().lbp_launch_count())


def lbp_phase_count() -> int:
    return int(_lib().lbp_phase_count())


def lbp_phase_name(i: int) -> str:
    return _lib().lbp_phase_name(i).decode()


_PHASE_KEEPALIVE = None


def lbp_set_phase_events(events) -> None:
    """events: list of torch.cuda.Event (already created with enable_timing=True
    and recorded once so their handles exist; an entry may be None to skip that
    phase boundary), or None to switch the hook off."""
    global _PHASE_KEEPALIVE
    if events is None:
        _check(_lib().lbp_set_phase_events(None, 0), "lbp_set_phase_events")
        _PHASE_KEEPALIVE = None
        return
    arr = (C.c_void_p * len(events))(*[None if e is None else e.cuda_event for e in events])
    _check(_lib().lbp_set_phase_events(arr, len(events)), "lbp_set_phase_events")
    _PHASE_KEEPALIVE = (arr, list(events))
