"""CPU oracle for the DEER-GRU hot path: TEST INFRASTRUCTURE ONLY.

Thin ctypes/numpy marshalling around ``deer_oracle.c`` (plain sequential C,
fp64 and fp32 instantiations).  Only ``tests/``, the smoke check and the
benchmark's ``cpu_baseline`` / reference arm may import this package; the
CUDA library and its Python binding never do, and this package imports
nothing from them.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "libdeer_oracle.so")
_SRC = [os.path.join(_HERE, "deer_oracle.c"), os.path.join(_HERE, "deer_oracle_impl.h")]
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math, no FMA contraction)."""
    stale = (not os.path.exists(_SO)) or any(os.path.getmtime(s) > os.path.getmtime(_SO) for s in _SRC)
    if force or stale:
        cmd = ["gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-fPIC", "-shared",
               "-o", _SO, _SRC[0], "-lm"]
        subprocess.run(cmd, check=True, cwd=_HERE)
    return _SO


def lib():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_SO)
        _lib.oracle_classifier_f64.restype = ctypes.c_double
        _lib.oracle_classifier_f32.restype = ctypes.c_float
    return _lib


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def _sfx(dtype):
    dtype = np.dtype(dtype)
    if dtype == np.float64:
        return "f64", ctypes.c_double
    if dtype == np.float32:
        return "f32", ctypes.c_float
    raise TypeError("oracle supports float64 and float32 only")


def _c(a, dtype):
    return np.ascontiguousarray(a, dtype=dtype)


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _params(p, dtype):
    return (_c(p.W_i, dtype), _c(p.W_h, dtype), _c(p.b_i, dtype), _c(p.b_h, dtype))


def gru_seq(p, x, y0, dtype=np.float64):
    """O-1: sequential GRU trajectory y[B,T,n]."""
    sfx, _ = _sfx(dtype)
    W_i, W_h, b_i, b_h = _params(p, dtype)
    x = _c(x, dtype); y0 = _c(y0, dtype)
    B, T, m = x.shape
    y = np.empty((B, T, p.n), dtype)
    getattr(lib(), f"oracle_gru_seq_{sfx}")(p.n, m, _p(W_i), _p(W_h), _p(b_i), _p(b_h), _p(x),
                                            _p(y0), B, T, _p(y))
    return y


def gru_cell_jac(p, hprev, x, dtype=np.float64, want_J=True):
    """Cell value f[N,n] and Jacobian J[N,n,n] at N given (h_prev, x) rows."""
    sfx, _ = _sfx(dtype)
    W_i, W_h, b_i, b_h = _params(p, dtype)
    hprev = _c(hprev, dtype).reshape(-1, p.n); x = _c(x, dtype).reshape(-1, p.m)
    N = hprev.shape[0]
    f = np.empty((N, p.n), dtype)
    J = np.empty((N, p.n, p.n), dtype) if want_J else None
    getattr(lib(), f"oracle_gru_cell_jac_{sfx}")(p.n, p.m, _p(W_i), _p(W_h), _p(b_i), _p(b_h),
                                                 _p(hprev), _p(x), ctypes.c_long(N), _p(f), _p(J))
    return f, J


def linrec(J, b, y0=None, reverse=False, dtype=np.float64):
    """O-2: sequential linear recurrence, forward or reverse (adjoint)."""
    sfx, _ = _sfx(dtype)
    J = _c(J, dtype); b = _c(b, dtype)
    B, T, n = b.shape
    assert J.shape == (B, T, n, n)
    y0c = None if y0 is None else _c(y0, dtype)
    y = np.empty((B, T, n), dtype)
    getattr(lib(), f"oracle_linrec_{sfx}")(_p(J), _p(b), _p(y0c), B, T, n, int(bool(reverse)), _p(y))
    return y


def deer(p, x, y0, tol=None, max_iter=100, y_guess=None, dtype=np.float64, form=0,
         cell="gru", want_history=False):
    """O-3: DEER/Newton iteration.  Returns dict(y, iters, err, trace[, history]).

    ``cell='affine'`` uses f(h, x) = W_h[:n] h + x (W_h's first n rows); ``cell='lstm'`` takes
    synth.LstmParams and states [h; c] of 2k components."""
    sfx, cty = _sfx(dtype)
    if tol is None:
        tol = 1e-7 if np.dtype(dtype) == np.float64 else 1e-4
    x = _c(x, dtype); y0 = _c(y0, dtype)
    B, T, m = x.shape
    n = 2 * p.k if cell == "lstm" else p.n
    if cell == "affine":
        assert m == n
        W_h = _c(p.W_h[:n], dtype); W_i = b_i = b_h = W_h
        cell_id = 1
    elif cell == "lstm":
        n = 2 * p.k
        W_i, W_h, b_i = _c(p.W_i, dtype), _c(p.W_h, dtype), _c(p.b, dtype)
        b_h = b_i
        cell_id = 2
    else:
        W_i, W_h, b_i, b_h = _params(p, dtype)
        cell_id = 0
    y = np.zeros((B, T, n), dtype) if y_guess is None else _c(y_guess, dtype).copy()
    err = cty(0)
    trace = np.full((max_iter,), np.nan, dtype)
    hist = np.empty((max_iter, B, T, n), dtype) if want_history else None
    fn = getattr(lib(), f"oracle_deer_{sfx}")
    iters = fn(cell_id, int(form), n, m, _p(W_i), _p(W_h), _p(b_i), _p(b_h), _p(x), _p(y0), B, T,
               cty(tol), int(max_iter), _p(y), ctypes.byref(err), _p(trace), _p(hist))
    out = dict(y=y, iters=int(iters), err=float(err.value), trace=trace[:iters])
    if want_history:
        out["history"] = hist[:iters]
    return out


def _grad_call(name, p, x, y0, y, gy, dtype, want_lam=False):
    sfx, _ = _sfx(dtype)
    W_i, W_h, b_i, b_h = _params(p, dtype)
    x = _c(x, dtype); y0 = _c(y0, dtype); y = _c(y, dtype); gy = _c(gy, dtype)
    B, T, m = x.shape
    n = p.n
    g = dict(dW_i=np.empty((3 * n, m), dtype), dW_h=np.empty((3 * n, n), dtype),
             db_i=np.empty((3 * n,), dtype), db_h=np.empty((3 * n,), dtype),
             dx=np.empty((B, T, m), dtype), dy0=np.empty((B, n), dtype))
    args = [n, m, _p(W_i), _p(W_h), _p(b_i), _p(b_h), _p(x), _p(y0), _p(y), _p(gy), B, T,
            _p(g["dW_i"]), _p(g["dW_h"]), _p(g["db_i"]), _p(g["db_h"]), _p(g["dx"]), _p(g["dy0"])]
    if want_lam:
        g["lam"] = np.empty((B, T, n), dtype)
        args.append(_p(g["lam"]))
    getattr(lib(), f"{name}_{sfx}")(*args)
    return g


def gru_bptt(p, x, y0, y, gy, dtype=np.float64):
    """O-4: textbook BPTT at trajectory ``y`` for dL/dy = gy."""
    return _grad_call("oracle_gru_bptt", p, x, y0, y, gy, dtype)


def deer_grad(p, x, y0, y, gy, dtype=np.float64):
    """DEER gradient: one reverse linear solve, then the cell VJP (Eq. 7)."""
    return _grad_call("oracle_deer_grad", p, x, y0, y, gy, dtype, want_lam=True)


def classifier(layers, W_o, b_o, x, labels, dtype=np.float64, want_grad=True, want_states=False):
    """O-5: 2-layer GRU + mean-pool + linear head + softmax-CE; loss and grads."""
    sfx, _ = _sfx(dtype)
    l1, l2 = layers
    P1 = _params(l1, dtype); P2 = _params(l2, dtype)
    W_o = _c(W_o, dtype); b_o = _c(b_o, dtype)
    x = _c(x, dtype); labels = np.ascontiguousarray(labels, np.int32)
    B, T, m = x.shape
    n = l1.n
    ncls = W_o.shape[0]
    g = {}
    for tag, lp in (("1", l1), ("2", l2)):
        g["dW_i" + tag] = np.zeros((3 * n, lp.m), dtype); g["dW_h" + tag] = np.zeros((3 * n, n), dtype)
        g["db_i" + tag] = np.zeros((3 * n,), dtype); g["db_h" + tag] = np.zeros((3 * n,), dtype)
    g["dW_o"] = np.zeros((ncls, n), dtype); g["db_o"] = np.zeros((ncls,), dtype)
    y1 = np.empty((B, T, n), dtype) if want_states else None
    y2 = np.empty((B, T, n), dtype) if want_states else None
    loss = getattr(lib(), f"oracle_classifier_{sfx}")(
        n, m, ncls, *[_p(a) for a in P1], *[_p(a) for a in P2], _p(W_o), _p(b_o), _p(x),
        _p(labels), B, T, int(want_grad),
        _p(g["dW_i1"]), _p(g["dW_h1"]), _p(g["db_i1"]), _p(g["db_h1"]),
        _p(g["dW_i2"]), _p(g["dW_h2"]), _p(g["db_i2"]), _p(g["db_h2"]),
        _p(g["dW_o"]), _p(g["db_o"]), _p(y1), _p(y2))
    g["loss"] = float(loss)
    if want_states:
        g["y1"], g["y2"] = y1, y2
    return g


def _stack_heads(heads, dtype):
    return (_c(np.stack([h.W_i for h in heads]), dtype), _c(np.stack([h.W_h for h in heads]), dtype),
            _c(np.stack([h.b_i for h in heads]), dtype), _c(np.stack([h.b_h for h in heads]), dtype))


def multihead_seq(heads, strides, x, y0, dtype=np.float64):
    """O-6: sequential multi-head GRU.  heads: list of H parameter sets (same n, m); strides [H];
    x [B,T,m]; y0 [B,H,n].  Returns y [B,T,H,n]."""
    sfx, _ = _sfx(dtype)
    H, n, m = len(heads), heads[0].n, heads[0].m
    W_i, W_h, b_i, b_h = _stack_heads(heads, dtype)
    st = np.ascontiguousarray(strides, np.int32)
    x = _c(x, dtype); y0 = _c(y0, dtype)
    B, T, _m = x.shape
    assert _m == m and y0.shape == (B, H, n) and st.shape == (H,) and np.all(st >= 1)
    y = np.empty((B, T, H, n), dtype)
    getattr(lib(), f"oracle_multihead_seq_{sfx}")(H, n, m, _p(W_i), _p(W_h), _p(b_i), _p(b_h), _p(st), _p(x),
                                                  _p(y0), B, T, _p(y))
    return y


def multihead_bptt(heads, strides, x, y0, y, gy, dtype=np.float64):
    """BPTT through the multi-head unit at trajectory y for dL/dy = gy [B,T,H,n]: dict of
    dW_i [H,3n,m], dW_h [H,3n,n], db_i, db_h [H,3n], dx [B,T,m], dy0 [B,H,n]."""
    sfx, _ = _sfx(dtype)
    H, n, m = len(heads), heads[0].n, heads[0].m
    W_i, W_h, b_i, b_h = _stack_heads(heads, dtype)
    st = np.ascontiguousarray(strides, np.int32)
    x = _c(x, dtype); y0 = _c(y0, dtype); y = _c(y, dtype); gy = _c(gy, dtype)
    B, T, _m = x.shape
    g = dict(dW_i=np.empty((H, 3 * n, m), dtype), dW_h=np.empty((H, 3 * n, n), dtype),
             db_i=np.empty((H, 3 * n), dtype), db_h=np.empty((H, 3 * n), dtype),
             dx=np.empty((B, T, m), dtype), dy0=np.empty((B, H, n), dtype))
    getattr(lib(), f"oracle_multihead_bptt_{sfx}")(H, n, m, _p(W_i), _p(W_h), _p(b_i), _p(b_h), _p(st), _p(x),
                                                   _p(y0), _p(y), _p(gy), B, T, _p(g["dW_i"]), _p(g["dW_h"]),
                                                   _p(g["db_i"]), _p(g["db_h"]), _p(g["dx"]), _p(g["dy0"]))
    return g


def gru_jvp(p, dp, x, dx, y0, dy0, y, dtype=np.float64):
    """O-7: forward-mode derivative of the trajectory along (dp, dx, dy0); dp is a parameter-shaped
    object (W_i, W_h, b_i, b_h) or None, dx / dy0 arrays or None.  Returns dy [B,T,n]."""
    sfx, _ = _sfx(dtype)
    W_i, W_h, b_i, b_h = _params(p, dtype)
    x = _c(x, dtype); y0 = _c(y0, dtype); y = _c(y, dtype)
    B, T, m = x.shape
    t = (None,) * 4 if dp is None else _params(dp, dtype)
    dxc = None if dx is None else _c(dx, dtype)
    dy0c = None if dy0 is None else _c(dy0, dtype)
    dy = np.empty((B, T, p.n), dtype)
    getattr(lib(), f"oracle_gru_jvp_{sfx}")(p.n, m, _p(W_i), _p(W_h), _p(b_i), _p(b_h), _p(t[0]), _p(t[1]), _p(t[2]),
                                            _p(t[3]), _p(x), _p(dxc), _p(y0), _p(dy0c), _p(y), B, T, _p(dy))
    return dy


def ode_linear(G, z, t, y0, dtype=np.float64, want_discrete=False):
    """O-8: y = L_G^{-1}[z] for dy/dt + G(t) y = z(t), y(t_0) = y0 (Sec. 3.3): G [B,T,n,n], z [B,T,n] at the
    time points t [T], mid-point values per interval.  Returns y [B,T,n] (and Gbar, zbar if asked)."""
    sfx, _ = _sfx(dtype)
    G = _c(G, dtype); z = _c(z, dtype); t = _c(t, dtype); y0 = _c(y0, dtype)
    B, T, n = z.shape
    assert G.shape == (B, T, n, n) and t.shape == (T,) and y0.shape == (B, n)
    y = np.empty((B, T, n), dtype)
    Gb = np.empty((B, max(T - 1, 0), n, n), dtype) if want_discrete else None
    zb = np.empty((B, max(T - 1, 0), n), dtype) if want_discrete else None
    getattr(lib(), f"oracle_ode_linear_{sfx}")(_p(G), _p(z), _p(t), _p(y0), B, T, n, _p(y), _p(Gb), _p(zb))
    return (y, Gb, zb) if want_discrete else y


def lstm_seq(p, x, s0, dtype=np.float64):
    """Sequential LSTM trajectory [B,T,2k] of states [h; c] (p: synth.LstmParams; gate order i, f, g, o)."""
    sfx, _ = _sfx(dtype)
    W_i, W_h, b = _c(p.W_i, dtype), _c(p.W_h, dtype), _c(p.b, dtype)
    x = _c(x, dtype); s0 = _c(s0, dtype)
    B, T, m = x.shape
    y = np.empty((B, T, 2 * p.k), dtype)
    getattr(lib(), f"oracle_lstm_seq_{sfx}")(p.k, m, _p(W_i), _p(W_h), _p(b), _p(x), _p(s0), B, T, _p(y))
    return y


def lstm_cell_jac(p, sprev, x, dtype=np.float64, want_J=True):
    """LSTM cell value f [N,2k] and state Jacobian J [N,2k,2k] at N given (s_prev, x) rows."""
    sfx, _ = _sfx(dtype)
    W_i, W_h, b = _c(p.W_i, dtype), _c(p.W_h, dtype), _c(p.b, dtype)
    sprev = _c(sprev, dtype).reshape(-1, 2 * p.k); x = _c(x, dtype).reshape(-1, p.m)
    N = sprev.shape[0]
    f = np.empty((N, 2 * p.k), dtype)
    J = np.empty((N, 2 * p.k, 2 * p.k), dtype) if want_J else None
    getattr(lib(), f"oracle_lstm_cell_jac_{sfx}")(p.k, p.m, _p(W_i), _p(W_h), _p(b), _p(sprev), _p(x), ctypes.c_long(N),
                                                  _p(f), _p(J))
    return f, J
