"""Thin ctypes binding over the C ABI of ``libdeer_b200.so`` (see include/deer.h).

Argument marshalling only: every step of the path runs in the library's CUDA
kernels.  PyTorch supplies device memory and streams.  Loading fails loudly
if the CUDA library has not been built; there is no CPU fallback.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdeer_b200.so")

DEER_OK, DEER_NOT_CONVERGED, DEER_NONFINITE = 0, 1, 2
DEER_ERR_INVALID_ARG, DEER_ERR_UNSUPPORTED_N, DEER_ERR_WORKSPACE = -1, -2, -3
DEER_ERR_CUDA, DEER_ERR_DEVICE_TIMEOUT = -4, -5
DEER_OP_EVAL, DEER_OP_SCAN, DEER_OP_VJP, DEER_OP_CLASSIFIER, DEER_OP_ODE, DEER_OP_LSTM = 0, 1, 2, 3, 4, 5
DEER_FLAG_WARM_START, DEER_FLAG_GENERIC, DEER_FLAG_MATERIALIZE, DEER_FLAG_TCGEN05 = 1, 2, 4, 8
DEER_FLAG_EXPIRE_WAITS, DEER_FLAG_COEF_ROWS = 16, 32

NOALLOC_SCRATCH_BYTES = 8 << 20
EXPORTS = ["deer_workspace_bytes", "deer_linrec_scan", "deer_linrec_scan_noalloc", "deer_gru_eval",
           "deer_gru_eval_diag", "deer_gru_eval_host", "deer_gru_vjp",
           "deer_gru_classifier_step", "deer_status_string", "deer_last_error", "deer_launch_count",
           "deer_workspace_status", "deer_noalloc_status", "deer_scan_geometry", "deer_gru_eval_host_chunk", "deer_gru_eval_host_chunks", "deer_gru_cell_jac",
           "deer_multihead_workspace_bytes", "deer_gru_multihead_eval", "deer_gru_multihead_vjp", "deer_gru_jvp",
           "deer_ode_linear_solve", "deer_lstm_eval"]


class _Params(ctypes.Structure):
    _fields_ = [("n", ctypes.c_int), ("m", ctypes.c_int), ("W_i", ctypes.c_void_p),
                ("W_h", ctypes.c_void_p), ("b_i", ctypes.c_void_p), ("b_h", ctypes.c_void_p)]


class _LstmParams(ctypes.Structure):
    _fields_ = [("k", ctypes.c_int), ("m", ctypes.c_int), ("W_i", ctypes.c_void_p), ("W_h", ctypes.c_void_p),
                ("b", ctypes.c_void_p)]


class _Grads(ctypes.Structure):
    _fields_ = [("dW_i", ctypes.c_void_p), ("dW_h", ctypes.c_void_p), ("db_i", ctypes.c_void_p),
                ("db_h", ctypes.c_void_p)]


_lib = None


def lib():
    """Load the CUDA library; raise if it is missing (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with "
                               "`python -m paper_2309_12252_b200.build` (needs nvcc, sm_100a)")
        L = ctypes.CDLL(LIB_PATH)
        L.deer_workspace_bytes.restype = ctypes.c_size_t
        L.deer_workspace_bytes.argtypes = [ctypes.c_int] * 6
        vp, ci, cf, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
        L.deer_linrec_scan.restype = ci
        L.deer_linrec_scan.argtypes = [vp, vp, vp, ci, ci, ci, ci, vp, vp, sz, ci, vp]
        L.deer_linrec_scan_noalloc.restype = ci
        L.deer_linrec_scan_noalloc.argtypes = [vp, vp, vp, ci, ci, ci, ci, vp, vp]
        L.deer_gru_eval.restype = ci
        L.deer_gru_eval.argtypes = [ctypes.POINTER(_Params), vp, vp, ci, ci, cf, ci, vp,
                                    ctypes.POINTER(ci), ctypes.POINTER(cf), vp, vp, sz, ci, vp]
        L.deer_gru_eval_diag.restype = ci
        L.deer_gru_eval_diag.argtypes = [ctypes.POINTER(_Params), vp, vp, ci, ci, cf, ci, vp,
                                         ctypes.POINTER(ci), ctypes.POINTER(cf), vp, vp,
                                         ctypes.POINTER(ctypes.c_ulonglong), vp, sz, ci, vp]
        L.deer_gru_eval_host.restype = ci
        L.deer_gru_eval_host.argtypes = [ctypes.POINTER(_Params), vp, vp, ci, ci, cf, ci, vp,
                                         ctypes.POINTER(ci), ctypes.POINTER(cf), vp, vp, vp, sz, ci, vp]
        L.deer_gru_vjp.restype = ci
        L.deer_gru_vjp.argtypes = [ctypes.POINTER(_Params), vp, vp, vp, vp, ci, ci,
                                   ctypes.POINTER(_Grads), vp, vp, vp, sz, ci, vp]
        L.deer_gru_classifier_step.restype = ci
        L.deer_gru_classifier_step.argtypes = [ctypes.POINTER(_Params), ctypes.POINTER(_Params), vp, vp,
                                               ci, vp, vp, ci, ci, cf, ci, ctypes.POINTER(cf),
                                               ctypes.POINTER(ci), ctypes.POINTER(_Grads),
                                               ctypes.POINTER(_Grads), vp, vp, vp, sz, ci, vp]
        L.deer_workspace_status.restype = ci
        L.deer_workspace_status.argtypes = [vp, vp]
        L.deer_noalloc_status.restype = ci
        L.deer_noalloc_status.argtypes = [vp]
        L.deer_gru_eval_host_chunk.restype = ci
        L.deer_gru_eval_host_chunk.argtypes = [ci, ci]
        L.deer_gru_eval_host_chunks.restype = ci
        L.deer_gru_eval_host_chunks.argtypes = [ci, ci, ctypes.POINTER(ci)]
        L.deer_scan_geometry.restype = ci
        L.deer_scan_geometry.argtypes = [ci, ci, ci, ci, ctypes.POINTER(ci)]
        L.deer_gru_cell_jac.restype = ci
        L.deer_gru_cell_jac.argtypes = [ctypes.POINTER(_Params), vp, vp, vp, ci, ci, vp, vp, vp, sz, ci, vp]
        L.deer_multihead_workspace_bytes.restype = sz
        L.deer_multihead_workspace_bytes.argtypes = [ctypes.POINTER(ci), ci, ci, ci, ci, ci, ci]
        L.deer_gru_multihead_eval.restype = ci
        L.deer_gru_multihead_eval.argtypes = [ctypes.POINTER(_Params), ctypes.POINTER(ci), ci, vp, vp, ci, ci, cf, ci, vp,
                                              ctypes.POINTER(ci), vp, sz, ci, vp]
        L.deer_gru_multihead_vjp.restype = ci
        L.deer_gru_multihead_vjp.argtypes = [ctypes.POINTER(_Params), ctypes.POINTER(ci), ci, vp, vp, vp, vp, ci, ci,
                                             ctypes.POINTER(_Grads), vp, vp, vp, sz, ci, vp]
        L.deer_lstm_eval.restype = ci
        L.deer_lstm_eval.argtypes = [ctypes.POINTER(_LstmParams), vp, vp, ci, ci, cf, ci, vp, ctypes.POINTER(ci),
                                     ctypes.POINTER(cf), vp, sz, ci, vp]
        L.deer_ode_linear_solve.restype = ci
        L.deer_ode_linear_solve.argtypes = [vp, vp, vp, vp, ci, ci, ci, vp, vp, sz, ci, vp]
        L.deer_gru_jvp.restype = ci
        L.deer_gru_jvp.argtypes = [ctypes.POINTER(_Params), ctypes.POINTER(_Params), vp, vp, vp, vp, vp, ci, ci, vp, vp, sz, ci, vp]
        L.deer_status_string.restype = ctypes.c_char_p
        L.deer_status_string.argtypes = [ci]
        L.deer_last_error.restype = ctypes.c_char_p
        L.deer_launch_count.restype = ctypes.c_longlong
        _lib = L
    return _lib


class DeerError(RuntimeError):
    def __init__(self, status: int):
        self.status = status
        msg = lib().deer_status_string(status).decode()
        if status in (DEER_ERR_CUDA, DEER_ERR_WORKSPACE):
            extra = lib().deer_last_error().decode()
            if extra:
                msg += ": " + extra
        super().__init__(f"deer status {status}: {msg}")


def _ptr(t):
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device-resident contiguous tensors only"
    return ctypes.c_void_p(t.data_ptr())


def _hptr(t):
    """Pointer to a contiguous HOST tensor (pinned for asynchronous copies)."""
    assert not t.is_cuda and t.is_contiguous() and t.dtype == torch.float32
    return ctypes.c_void_p(t.data_ptr())


def _f32(t):
    assert t.dtype == torch.float32
    return t


def _stream(stream):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


@dataclass
class GruParamsDev:
    """GRU parameters resident on the device (gate order r, z, n)."""
    n: int
    m: int
    W_i: torch.Tensor
    W_h: torch.Tensor
    b_i: torch.Tensor
    b_h: torch.Tensor

    @staticmethod
    def from_numpy(p, device="cuda"):
        mk = lambda a: torch.from_numpy(np.ascontiguousarray(a, np.float32)).to(device)
        return GruParamsDev(p.n, p.m, mk(p.W_i), mk(p.W_h), mk(p.b_i), mk(p.b_h))

    def c_struct(self):
        for t, shape in ((self.W_i, (3 * self.n, self.m)), (self.W_h, (3 * self.n, self.n)),
                         (self.b_i, (3 * self.n,)), (self.b_h, (3 * self.n,))):
            assert tuple(t.shape) == shape and t.dtype == torch.float32 and t.is_cuda and t.is_contiguous()
        return _Params(self.n, self.m, self.W_i.data_ptr(), self.W_h.data_ptr(), self.b_i.data_ptr(),
                       self.b_h.data_ptr())


def deer_status_string(status: int) -> str:
    return lib().deer_status_string(int(status)).decode()


def deer_launch_count() -> int:
    return int(lib().deer_launch_count())


def deer_workspace_bytes(op: int, B: int, T: int, n: int, m: int = 1, flags: int = 0) -> int:
    return int(lib().deer_workspace_bytes(op, B, T, n, m, flags))


def alloc_workspace(op: int, B: int, T: int, n: int, m: int = 1, flags: int = 0, device="cuda"):
    nbytes = deer_workspace_bytes(op, B, T, n, m, flags)
    if nbytes == 0:
        raise DeerError(DEER_ERR_UNSUPPORTED_N)
    return torch.empty(nbytes, dtype=torch.uint8, device=device)   # torch allocations are 512-B aligned


def deer_linrec_scan(J, b, y0=None, reverse=False, y=None, ws=None, flags=0, stream=None, check=True):
    """y = scan(J, b, y0); see include/deer.h.  Returns y (asynchronous)."""
    B, T, n = b.shape
    assert tuple(J.shape) == (B, T, n, n)
    if y is None:
        y = torch.empty_like(b)
    if ws is None:
        ws = alloc_workspace(DEER_OP_SCAN, B, T, n, 1, flags, b.device)
    rc = lib().deer_linrec_scan(_ptr(_f32(J)), _ptr(_f32(b)), _ptr(y0), B, T, n, int(bool(reverse)),
                                _ptr(y), _ptr(ws), ws.numel(), flags, _stream(stream))
    if check and rc != DEER_OK:
        raise DeerError(rc)
    return y if check else (y, rc)


def deer_workspace_status(ws, stream=None) -> int:
    """Outcome of the last asynchronous call on workspace ``ws`` (synchronises the stream)."""
    return int(lib().deer_workspace_status(_ptr(ws), _stream(stream)))


def deer_noalloc_status(stream=None) -> int:
    return int(lib().deer_noalloc_status(_stream(stream)))


def deer_gru_eval_host_chunk(B: int, T: int) -> int:
    """Sequences of the largest chunk of deer_gru_eval_host (B when the batch is not split)."""
    return int(lib().deer_gru_eval_host_chunk(int(B), int(T)))


def deer_gru_eval_host_chunks(B: int, T: int) -> list:
    """First sequence of every chunk of deer_gru_eval_host, then B: [0, ..., B] ([] for invalid sizes)."""
    first = (ctypes.c_int * 9)()
    nc = int(lib().deer_gru_eval_host_chunks(int(B), int(T), first))
    return [int(first[k]) for k in range(nc + 1)] if nc > 0 else []


def deer_scan_geometry(B: int, T: int, n: int, flags: int = 0) -> dict:
    """Launch geometry of the scan for these sizes on the current device; see include/deer.h."""
    out = (ctypes.c_int * 6)()
    rc = lib().deer_scan_geometry(B, T, n, flags, out)
    if rc != DEER_OK:
        raise DeerError(rc)
    return dict(single_pass=bool(out[0]), tile_len=out[1], chain_len=out[2], tiles_per_seq=out[3],
                resolver_ctas=out[4], sms=out[5])


def deer_gru_cell_jac(params: "GruParamsDev", x, y0, y, flags=0, ws=None, stream=None):
    """Cell Jacobians (or coefficient rows with DEER_FLAG_COEF_ROWS) and rhs at the guess y; see include/deer.h."""
    B, T, m = x.shape
    n = params.n
    J = torch.empty((B, T, n, 4 if flags & DEER_FLAG_COEF_ROWS else n), dtype=torch.float32, device=x.device)
    rhs = torch.empty((B, T, n), dtype=torch.float32, device=x.device)
    if ws is None:
        ws = alloc_workspace(DEER_OP_EVAL, B, T, n, m, 0, x.device)
    ps = params.c_struct()
    rc = lib().deer_gru_cell_jac(ctypes.byref(ps), _ptr(_f32(x)), _ptr(_f32(y0)), _ptr(_f32(y)), B, T, _ptr(J),
                                 _ptr(rhs), _ptr(ws), ws.numel(), flags, _stream(stream))
    if rc != DEER_OK:
        raise DeerError(rc)
    return J, rhs


def deer_linrec_scan_noalloc(J, b, y0=None, reverse=False, y=None, stream=None, check=True):
    """deer_linrec_scan for callers that may not allocate: the library's built-in
    scratch array is used instead of a workspace (see include/deer.h for the limits)."""
    B, T, n = b.shape
    assert tuple(J.shape) == (B, T, n, n)
    if y is None:
        y = torch.empty_like(b)
    rc = lib().deer_linrec_scan_noalloc(_ptr(_f32(J)), _ptr(_f32(b)), _ptr(y0), B, T, n, int(bool(reverse)),
                                        _ptr(y), _stream(stream))
    if check and rc != DEER_OK:
        raise DeerError(rc)
    return y if check else (y, rc)


@dataclass
class EvalResult:
    y: torch.Tensor
    iters: int
    err: float
    status: int
    err_trace: np.ndarray


def deer_gru_eval(params: GruParamsDev, x, y0, tol=1e-4, max_iter=100, y=None, ws=None, flags=0,
                  stream=None, check=True) -> EvalResult:
    """DEER evaluation of the GRU over x [B,T,m]; see include/deer.h."""
    B, T, m = x.shape
    n = params.n
    assert m == params.m and tuple(y0.shape) == (B, n)
    if y is None:
        assert not (flags & DEER_FLAG_WARM_START)
        y = torch.empty((B, T, n), dtype=torch.float32, device=x.device)
    if ws is None:
        ws = alloc_workspace(DEER_OP_EVAL, B, T, n, m, flags, x.device)
    iters = ctypes.c_int(0)
    err = ctypes.c_float(0.0)
    trace = np.full((max(int(max_iter), 1),), np.nan, np.float32)
    ps = params.c_struct()
    rc = lib().deer_gru_eval(ctypes.byref(ps), _ptr(_f32(x)), _ptr(_f32(y0)), B, T, float(tol),
                             int(max_iter), _ptr(y), ctypes.byref(iters), ctypes.byref(err),
                             trace.ctypes.data_as(ctypes.c_void_p), _ptr(ws), ws.numel(), flags,
                             _stream(stream))
    if check and rc < 0:
        raise DeerError(rc)
    return EvalResult(y, iters.value, err.value, rc, trace[:iters.value])


def deer_gru_eval_diag(params: GruParamsDev, x, y0, tol=1e-4, max_iter=100, y=None, ws=None, flags=0, stream=None):
    """deer_gru_eval plus the diagnostics of the last body: returns (EvalResult, err_b [B] numpy, err_argmax int)."""
    B, T, m = x.shape
    n = params.n
    if y is None:
        y = torch.empty((B, T, n), dtype=torch.float32, device=x.device)
    if ws is None:
        ws = alloc_workspace(DEER_OP_EVAL, B, T, n, m, flags, x.device)
    iters = ctypes.c_int(0)
    err = ctypes.c_float(0.0)
    trace = np.full((max(int(max_iter), 1),), np.nan, np.float32)
    err_b = np.full((B,), np.nan, np.float32)
    argmax = ctypes.c_ulonglong(0)
    ps = params.c_struct()
    rc = lib().deer_gru_eval_diag(ctypes.byref(ps), _ptr(_f32(x)), _ptr(_f32(y0)), B, T, float(tol), int(max_iter),
                                  _ptr(y), ctypes.byref(iters), ctypes.byref(err),
                                  trace.ctypes.data_as(ctypes.c_void_p), err_b.ctypes.data_as(ctypes.c_void_p),
                                  ctypes.byref(argmax), _ptr(ws), ws.numel(), flags, _stream(stream))
    if rc < 0:
        raise DeerError(rc)
    return EvalResult(y, iters.value, err.value, rc, trace[:iters.value]), err_b, int(argmax.value)


def deer_gru_eval_host(params: GruParamsDev, x_host, y0_dev, y_host, x_dev, y_dev, ws, tol=1e-4,
                       max_iter=100, flags=0, stream=None) -> EvalResult:
    """End-to-end call with HOST buffers (x_host, y_host: pinned host tensors; x_dev, y_dev: device
    staging buffers): the library copies x to the device, evaluates, copies y back; see include/deer.h."""
    B, T, m = x_host.shape
    n = params.n
    assert m == params.m and not x_host.is_cuda and not y_host.is_cuda and x_dev.is_cuda and y_dev.is_cuda
    assert tuple(y_host.shape) == (B, T, n) == tuple(y_dev.shape) and tuple(x_dev.shape) == (B, T, m)
    iters = ctypes.c_int(0)
    err = ctypes.c_float(0.0)
    ps = params.c_struct()
    rc = lib().deer_gru_eval_host(ctypes.byref(ps), _hptr(x_host), _ptr(_f32(y0_dev)), B, T, float(tol),
                                  int(max_iter), _hptr(y_host), ctypes.byref(iters), ctypes.byref(err),
                                  _ptr(x_dev), _ptr(y_dev), _ptr(ws), ws.numel(), flags, _stream(stream))
    if rc < 0:
        raise DeerError(rc)
    return EvalResult(y_dev, iters.value, err.value, rc, np.zeros((0,), np.float32))


def deer_gru_vjp(params: GruParamsDev, x, y0, y, gy, want_dx=True, want_dy0=True, ws=None, flags=0,
                 stream=None):
    """Gradients of L (dL/dy = gy) w.r.t. parameters, x and y0; see include/deer.h."""
    B, T, m = x.shape
    n = params.n
    dev = x.device
    g = dict(dW_i=torch.empty((3 * n, m), device=dev), dW_h=torch.empty((3 * n, n), device=dev),
             db_i=torch.empty((3 * n,), device=dev), db_h=torch.empty((3 * n,), device=dev))
    dx = torch.empty_like(x) if want_dx else None
    dy0 = torch.empty((B, n), device=dev) if want_dy0 else None
    if ws is None:
        ws = alloc_workspace(DEER_OP_VJP, B, T, n, m, flags, dev)
    ps = params.c_struct()
    gs = _Grads(g["dW_i"].data_ptr(), g["dW_h"].data_ptr(), g["db_i"].data_ptr(), g["db_h"].data_ptr())
    rc = lib().deer_gru_vjp(ctypes.byref(ps), _ptr(_f32(x)), _ptr(_f32(y0)), _ptr(_f32(y)), _ptr(_f32(gy)),
                            B, T, ctypes.byref(gs), _ptr(dx), _ptr(dy0), _ptr(ws), ws.numel(), flags,
                            _stream(stream))
    if rc != DEER_OK:
        raise DeerError(rc)
    g["dx"], g["dy0"] = dx, dy0
    return g


def deer_gru_classifier_step(layer1: GruParamsDev, layer2: GruParamsDev, W_o, b_o, x, labels, tol=1e-4,
                             max_iter=100, ws=None, flags=0, stream=None):
    """Loss and all gradients of the 2-layer GRU classifier; see include/deer.h."""
    B, T, m = x.shape
    n = layer1.n
    ncls = W_o.shape[0]
    dev = x.device
    mk = lambda p: dict(dW_i=torch.empty((3 * n, p.m), device=dev), dW_h=torch.empty((3 * n, n), device=dev),
                        db_i=torch.empty((3 * n,), device=dev), db_h=torch.empty((3 * n,), device=dev))
    g1, g2 = mk(layer1), mk(layer2)
    cs = lambda g: _Grads(g["dW_i"].data_ptr(), g["dW_h"].data_ptr(), g["db_i"].data_ptr(), g["db_h"].data_ptr())
    dW_o = torch.empty_like(W_o); db_o = torch.empty_like(b_o)
    if ws is None:
        ws = alloc_workspace(DEER_OP_CLASSIFIER, B, T, n, m, flags, dev)
    loss = ctypes.c_float(0.0)
    iters = (ctypes.c_int * 2)()
    p1, p2 = layer1.c_struct(), layer2.c_struct()
    s1, s2 = cs(g1), cs(g2)
    assert labels.dtype == torch.int32
    rc = lib().deer_gru_classifier_step(ctypes.byref(p1), ctypes.byref(p2), _ptr(_f32(W_o)), _ptr(_f32(b_o)),
                                        ncls, _ptr(_f32(x)), _ptr(labels), B, T, float(tol), int(max_iter),
                                        ctypes.byref(loss), iters, ctypes.byref(s1), ctypes.byref(s2),
                                        _ptr(dW_o), _ptr(db_o), _ptr(ws), ws.numel(), flags, _stream(stream))
    if rc < 0:
        raise DeerError(rc)
    return dict(loss=loss.value, iters=(iters[0], iters[1]), status=rc, g1=g1, g2=g2, dW_o=dW_o, db_o=db_o)


def _mh_args(heads, strides):
    H = len(heads)
    ps = (_Params * H)(*[h.c_struct() for h in heads])
    st = (ctypes.c_int * H)(*[int(v) for v in strides])
    return H, ps, st


def alloc_multihead_workspace(heads, strides, B, T, device="cuda"):
    H, _, st = _mh_args(heads, strides)
    nbytes = int(lib().deer_multihead_workspace_bytes(st, H, B, T, heads[0].n, heads[0].m, 0))
    if nbytes == 0:
        raise DeerError(DEER_ERR_INVALID_ARG)
    return torch.empty(nbytes, dtype=torch.uint8, device=device)


def deer_gru_multihead_eval(heads, strides, x, y0, tol=1e-4, max_iter=100, y=None, ws=None, flags=0, stream=None):
    """Multi-head GRU unit: heads = list of GruParamsDev, strides = list of ints, x [B,T,m], y0 [B,H,n].
    Returns (y [B,T,H,n], iters per head, status); see include/deer.h."""
    B, T, m = x.shape
    H, ps, st = _mh_args(heads, strides)
    n = heads[0].n
    assert tuple(y0.shape) == (B, H, n)
    if y is None:
        y = torch.empty((B, T, H, n), dtype=torch.float32, device=x.device)
    if ws is None:
        ws = alloc_multihead_workspace(heads, strides, B, T, x.device)
    iters = (ctypes.c_int * H)()
    rc = lib().deer_gru_multihead_eval(ps, st, H, _ptr(_f32(x)), _ptr(_f32(y0)), B, T, float(tol), int(max_iter), _ptr(y),
                                       iters, _ptr(ws), ws.numel(), flags, _stream(stream))
    if rc < 0:
        raise DeerError(rc)
    return y, list(iters), rc


def deer_gru_multihead_vjp(heads, strides, x, y0, y, gy, ws=None, flags=0, stream=None):
    """Gradients of the multi-head unit: dict with per-head lists dW_i, dW_h, db_i, db_h and dx, dy0."""
    B, T, m = x.shape
    H, ps, st = _mh_args(heads, strides)
    n = heads[0].n
    dev = x.device
    g = dict(dW_i=[torch.empty((3 * n, m), device=dev) for _ in range(H)], dW_h=[torch.empty((3 * n, n), device=dev) for _ in range(H)],
             db_i=[torch.empty((3 * n,), device=dev) for _ in range(H)], db_h=[torch.empty((3 * n,), device=dev) for _ in range(H)])
    gs = (_Grads * H)(*[_Grads(g["dW_i"][h].data_ptr(), g["dW_h"][h].data_ptr(), g["db_i"][h].data_ptr(),
                               g["db_h"][h].data_ptr()) for h in range(H)])
    dx = torch.empty_like(x)
    dy0 = torch.empty_like(y0)
    if ws is None:
        ws = alloc_multihead_workspace(heads, strides, B, T, dev)
    rc = lib().deer_gru_multihead_vjp(ps, st, H, _ptr(_f32(x)), _ptr(_f32(y0)), _ptr(_f32(y)), _ptr(_f32(gy)), B, T, gs,
                                      _ptr(dx), _ptr(dy0), _ptr(ws), ws.numel(), flags, _stream(stream))
    if rc != DEER_OK:
        raise DeerError(rc)
    g["dx"], g["dy0"] = dx, dy0
    return g


def deer_gru_jvp(params, dparams, x, dx, y0, dy0, y, ws=None, flags=0, stream=None):
    """Forward-mode derivative dy [B,T,n] of the trajectory y along (dparams, dx, dy0); any of the three may be
    None.  dparams: a GruParamsDev holding the direction; see include/deer.h."""
    B, T, m = x.shape
    n = params.n
    dy = torch.empty((B, T, n), dtype=torch.float32, device=x.device)
    if ws is None:
        ws = alloc_workspace(DEER_OP_VJP, B, T, n, m, flags, x.device)
    ps = params.c_struct()
    dps = None if dparams is None else dparams.c_struct()
    rc = lib().deer_gru_jvp(ctypes.byref(ps), None if dps is None else ctypes.byref(dps), _ptr(_f32(x)), _ptr(dx),
                            _ptr(_f32(y0)), _ptr(dy0), _ptr(_f32(y)), B, T, _ptr(dy), _ptr(ws), ws.numel(), flags,
                            _stream(stream))
    if rc != DEER_OK:
        raise DeerError(rc)
    return dy


def deer_ode_linear_solve(G, z, t, y0, ws=None, flags=0, stream=None):
    """y = L_G^{-1}[z] for dy/dt + G(t) y = z(t), y(t_0) = y0, mid-point values per interval; see include/deer.h."""
    B, T, n = z.shape
    assert tuple(G.shape) == (B, T, n, n) and tuple(t.shape) == (T,) and tuple(y0.shape) == (B, n)
    y = torch.empty_like(z)
    if ws is None:
        ws = alloc_workspace(DEER_OP_ODE, B, T, n, 1, flags, z.device)
    rc = lib().deer_ode_linear_solve(_ptr(_f32(G)), _ptr(_f32(z)), _ptr(_f32(t)), _ptr(_f32(y0)), B, T, n, _ptr(y), _ptr(ws),
                                     ws.numel(), flags, _stream(stream))
    if rc != DEER_OK:
        raise DeerError(rc)
    return y


def deer_lstm_eval(p, x, s0, tol=1e-4, max_iter=100, s=None, ws=None, flags=0, stream=None) -> EvalResult:
    """DEER evaluation of an LSTM (p: synth.LstmParams-like with numpy arrays; moved to the device here);
    returns EvalResult with y = states [B,T,2k] = [h; c]; see include/deer.h."""
    B, T, m = x.shape
    k = p.k
    mk = lambda a: torch.from_numpy(np.ascontiguousarray(a, np.float32)).to(x.device)
    W_i, W_h, b = mk(p.W_i), mk(p.W_h), mk(p.b)
    if s is None:
        assert not (flags & DEER_FLAG_WARM_START)
        s = torch.empty((B, T, 2 * k), dtype=torch.float32, device=x.device)
    if ws is None:
        ws = alloc_workspace(DEER_OP_LSTM, B, T, k, m, flags, x.device)
    ps = _LstmParams(k, m, W_i.data_ptr(), W_h.data_ptr(), b.data_ptr())
    iters = ctypes.c_int(0)
    err = ctypes.c_float(0.0)
    rc = lib().deer_lstm_eval(ctypes.byref(ps), _ptr(_f32(x)), _ptr(_f32(s0)), B, T, float(tol), int(max_iter), _ptr(s),
                              ctypes.byref(iters), ctypes.byref(err), _ptr(ws), ws.numel(), flags, _stream(stream))
    if rc < 0:
        raise DeerError(rc)
    return EvalResult(s, iters.value, err.value, rc, np.zeros((0,), np.float32))
