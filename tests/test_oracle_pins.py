"""Pins for the CPU oracle: every oracle function is checked against something
other than itself -- closed forms, brute-force matrix products, finite
differences, the fixed-point property, values the paper prints.  None of the
expected values below comes from the oracle or from the CUDA path."""
import math
import os

import numpy as np
import pytest

import oracle
from paper_2309_12252_b200 import synth

GOLD = {}
with open(os.path.join(os.path.dirname(__file__), "golden", "paper_values.txt")) as fh:
    for line in fh:
        line = line.split("#")[0].split()
        if len(line) == 2:
            GOLD[line[0]] = float(line[1])


def small(n, m, B, T, seed=1, scale_y0=0.5):
    p = synth.gru_params(n, m, seed, tag="t/gru")
    x = synth.x_gaussian(B, T, m, seed, tag="t/x")
    y0 = synth.normal(seed, "t/y0", (B, n)) * scale_y0
    return p, x, y0


# -- independent numpy restatement of the cell used ONLY as a finite-difference
#    target: f is evaluated through the oracle itself (gru_cell_jac with
#    want_J=False), so that J, BPTT and the DEER gradient are pinned by
#    differencing the oracle's own forward map, and the forward map is pinned
#    separately by hand-computed values below.

def test_cell_hand_computed_n1():
    """n = m = 1 GRU step written out with scalar math (Sec. 4.1 cell)."""
    p = synth.GruParams(1, 1, np.array([[0.3], [-0.2], [0.7]]), np.array([[0.5], [0.1], [-0.4]]),
                        np.array([0.05, -0.1, 0.2]), np.array([0.0, 0.3, -0.25]))
    h, x = 0.6, -1.5
    sig = lambda a: 1.0 / (1.0 + math.exp(-a))
    r = sig(0.3 * x + 0.05 + 0.5 * h + 0.0)
    z = sig(-0.2 * x - 0.1 + 0.1 * h + 0.3)
    q = -0.4 * h - 0.25
    c = math.tanh(0.7 * x + 0.2 + r * q)
    want = (1 - z) * c + z * h
    f, _ = oracle.gru_cell_jac(p, [[h]], [[x]])
    assert abs(f[0, 0] - want) < 1e-15
    y = oracle.gru_seq(p, np.array([[[x], [x]]]), np.array([[h]]))
    # second step by hand from the first
    h2 = want
    r = sig(0.3 * x + 0.05 + 0.5 * h2); z = sig(-0.2 * x - 0.1 + 0.1 * h2 + 0.3)
    c = math.tanh(0.7 * x + 0.2 + r * (-0.4 * h2 - 0.25))
    assert abs(y[0, 0, 0] - want) < 1e-15
    assert abs(y[0, 1, 0] - ((1 - z) * c + z * h2)) < 1e-15


def test_cell_gate_layout_vs_numpy():
    """Vector case against a numpy restatement with explicit gate slices
    (catches a transposed weight or a wrong gate order)."""
    p, x, y0 = small(5, 3, 1, 1)
    W_i, W_h, b_i, b_h = (a.astype(np.float64) for a in (p.W_i, p.W_h, p.b_i, p.b_h))
    h = y0[0].astype(np.float64); xv = x[0, 0].astype(np.float64)
    u = W_i @ xv + b_i; g = W_h @ h + b_h
    n = 5
    r = 1 / (1 + np.exp(-(u[:n] + g[:n]))); z = 1 / (1 + np.exp(-(u[n:2 * n] + g[n:2 * n])))
    c = np.tanh(u[2 * n:] + r * g[2 * n:])
    want = (1 - z) * c + z * h
    f, _ = oracle.gru_cell_jac(p, h[None], xv[None])
    np.testing.assert_allclose(f[0], want, rtol=0, atol=1e-15)


def test_P7_jacobian_vs_central_differences():
    p, x, y0 = small(6, 4, 1, 7)
    h = (synth.normal(3, "t/h", (7, 6)) * 0.8).astype(np.float64)
    xs = x[0].astype(np.float64)
    _, J = oracle.gru_cell_jac(p, h, xs)
    eps = 1e-6
    for j in range(6):
        hp = h.copy(); hp[:, j] += eps
        hm = h.copy(); hm[:, j] -= eps
        fp, _ = oracle.gru_cell_jac(p, hp, xs, want_J=False)
        fm, _ = oracle.gru_cell_jac(p, hm, xs, want_J=False)
        np.testing.assert_allclose(J[:, :, j], (fp - fm) / (2 * eps), rtol=0, atol=1e-8)


def test_P3_scan_closed_form_scalar_times_identity():
    """J_t = a I: y_t = a^{t+1} y0 + sum_k a^{t-k} b_k; constant b: geometric sum."""
    B, T, n, a = 2, 40, 3, 0.83
    J = np.tile(a * np.eye(n), (B, T, 1, 1))
    b = synth.normal(5, "t/b", (B, T, n)).astype(np.float64)
    y0 = synth.normal(5, "t/y0b", (B, n)).astype(np.float64)
    y = oracle.linrec(J, b, y0)
    for t in (0, 1, 17, T - 1):
        want = a ** (t + 1) * y0 + sum(a ** (t - k) * b[:, k] for k in range(t + 1))
        np.testing.assert_allclose(y[:, t], want, rtol=1e-13, atol=1e-13)
    bc = np.broadcast_to(np.array([0.3, -1.0, 2.0]), (B, T, n)).copy()
    yc = oracle.linrec(J, bc, y0)
    t = T - 1
    want = a ** (t + 1) * y0 + bc[:, 0] * (1 - a ** (t + 1)) / (1 - a)
    np.testing.assert_allclose(yc[:, t], want, rtol=1e-13, atol=1e-13)


def test_P4_scan_brute_force_products():
    """T <= 8: y_t = (prod J) y0 + sum (prod J) b_k with explicit products
    (Eq. 9's cumulative operator written out)."""
    B, T, n = 2, 8, 4
    J = synth.uniform(9, "t/J", (B, T, n, n), -0.7, 0.7, dtype=np.float64)
    b = synth.normal(9, "t/bb", (B, T, n)).astype(np.float64)
    y0 = synth.normal(9, "t/y0c", (B, n)).astype(np.float64)
    y = oracle.linrec(J, b, y0)
    for s in range(B):
        for t in range(T):
            P = np.eye(n)
            acc = np.zeros(n)
            for k in range(t, -1, -1):      # P = J_t ... J_{k+1}
                acc += P @ b[s, k]
                P = P @ J[s, k]
            acc += P @ y0[s]
            np.testing.assert_allclose(y[s, t], acc, rtol=1e-12, atol=1e-12)
    # y0 = None means a zero start
    np.testing.assert_allclose(oracle.linrec(J, b, None), oracle.linrec(J, b, np.zeros((B, n))),
                               rtol=0, atol=0)


def test_P6_associativity_and_chunked_evaluation():
    """Combine (A2,b2) o (A1,b1) = (A2 A1, A2 b1 + b2) is associative, and a
    chunked evaluation with numpy carries equals the oracle's sequential one."""
    rng_J = synth.uniform(2, "t/J3", (3, 4, 4), -0.9, 0.9, dtype=np.float64)
    rng_b = synth.normal(2, "t/b3", (3, 4)).astype(np.float64)
    comb = lambda c2, c1: (c2[0] @ c1[0], c2[0] @ c1[1] + c2[1])
    c1, c2, c3 = [(rng_J[i], rng_b[i]) for i in range(3)]
    left = comb(comb(c3, c2), c1); right = comb(c3, comb(c2, c1))
    np.testing.assert_allclose(left[0], right[0], rtol=1e-14, atol=1e-14)
    np.testing.assert_allclose(left[1], right[1], rtol=1e-14, atol=1e-14)
    B, T, n = 1, 37, 3
    J = synth.uniform(4, "t/J4", (B, T, n, n), -0.6, 0.6, dtype=np.float64)
    b = synth.normal(4, "t/b4", (B, T, n)).astype(np.float64)
    y0 = synth.normal(4, "t/y04", (B, n)).astype(np.float64)
    y = oracle.linrec(J, b, y0)
    for L in (1, 5, 16, 37, 64):
        state = y0[0].copy()
        for c0 in range(0, T, L):
            A = np.eye(n); beta = np.zeros(n)
            for t in range(c0, min(T, c0 + L)):
                A, beta = comb((J[0, t], b[0, t]), (A, beta))
            state = A @ state + beta
            np.testing.assert_allclose(state, y[0, min(T, c0 + L) - 1], rtol=1e-12, atol=1e-12)


def test_P8_reverse_scan_is_adjoint_of_forward():
    """<S(J,b,0), g> == <b, S^T(J,g)> (dual operator, Sec. 3.1.1)."""
    B, T, n = 2, 23, 5
    J = synth.uniform(6, "t/J5", (B, T, n, n), -0.5, 0.5, dtype=np.float64)
    b = synth.normal(6, "t/b5", (B, T, n)).astype(np.float64)
    g = synth.normal(6, "t/g5", (B, T, n)).astype(np.float64)
    lhs = np.sum(oracle.linrec(J, b, None) * g)
    rhs = np.sum(b * oracle.linrec(J, g, None, reverse=True))
    assert abs(lhs - rhs) <= 1e-12 * max(1.0, abs(lhs))
    # brute force of the reverse recurrence on the last three positions
    lam = oracle.linrec(J, g, None, reverse=True)
    np.testing.assert_allclose(lam[:, T - 1], g[:, T - 1], rtol=0, atol=0)
    want = g[:, T - 2] + np.einsum("bki,bk->bi", J[:, T - 1], g[:, T - 1])
    np.testing.assert_allclose(lam[:, T - 2], want, rtol=1e-14, atol=1e-14)
    # terminal term is added at t = T-1 only and propagates linearly
    term = synth.normal(6, "t/term", (B, n)).astype(np.float64)
    lam2 = oracle.linrec(J, g, term, reverse=True)
    np.testing.assert_allclose(lam2[:, T - 1], g[:, T - 1] + term, rtol=0, atol=1e-15)
    g2 = g.copy(); g2[:, T - 1] += term
    np.testing.assert_allclose(lam2, oracle.linrec(J, g2, None, reverse=True), rtol=1e-13, atol=1e-13)


def test_P10_n1_matches_cumprod_form():
    """n = 1: y_t = P_t (y0 + sum_k b_k / P_k), P_t = prod_{k<=t} a_k
    (integrating-factor form, App. A.5) on well-conditioned coefficients."""
    T = 60
    a = synth.uniform(8, "t/a", (1, T, 1, 1), 0.7, 1.1, dtype=np.float64)
    b = synth.normal(8, "t/b1", (1, T, 1)).astype(np.float64)
    y0 = np.array([[0.4]])
    y = oracle.linrec(a, b, y0)[0, :, 0]
    P = np.cumprod(a[0, :, 0, 0])
    want = P * (y0[0, 0] + np.cumsum(b[0, :, 0] / P))
    np.testing.assert_allclose(y, want, rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("form", [0, 1])
def test_P1_deer_returns_sequential_trajectory(form):
    """The iteration's fixed point is the sequential trajectory (Sec. 4.1)."""
    p, x, y0 = small(4, 2, 3, 300)
    seq = oracle.gru_seq(p, x, y0, np.float64)
    out = oracle.deer(p, x, y0, dtype=np.float64, form=form)
    assert out["iters"] < 30 and out["err"] <= GOLD["default_tol_fp64"]
    assert np.max(np.abs(out["y"] - seq)) <= 1e-12
    seq32 = oracle.gru_seq(p, x, y0, np.float32)
    out32 = oracle.deer(p, x, y0, dtype=np.float32, form=form)
    assert out32["err"] <= GOLD["default_tol_fp32"]
    assert np.max(np.abs(out32["y"] - seq32)) <= 2e-6
    assert np.max(np.abs(seq32 - seq)) <= 5e-6


def test_forms_agree_iterate_by_iterate():
    """Eq. 3 form and the Newton-update form of App. A.1 give the same iterates."""
    p, x, y0 = small(3, 3, 2, 120)
    a = oracle.deer(p, x, y0, tol=-1.0, max_iter=5, form=0, want_history=True)
    b = oracle.deer(p, x, y0, tol=-1.0, max_iter=5, form=1, want_history=True)
    assert a["iters"] == b["iters"] == 5
    np.testing.assert_allclose(a["history"], b["history"], rtol=0, atol=1e-11)


def test_P2_affine_cell_is_solved_by_one_body():
    """Newton on an affine f is exact after one body; the second body only
    confirms (iters == 2 with the paper's loop condition)."""
    n, B, T = 4, 2, 50
    M = synth.uniform(3, "t/M", (n, n), -0.45, 0.45, dtype=np.float64)
    p = synth.GruParams(n, n, np.zeros((3 * n, n)), np.vstack([M, M, M]), np.zeros(3 * n), np.zeros(3 * n))
    x = synth.normal(3, "t/xa", (B, T, n)).astype(np.float64)
    y0 = synth.normal(3, "t/y0a", (B, n)).astype(np.float64)
    out = oracle.deer(p, x, y0, cell="affine", want_history=True)
    want = np.empty((B, T, n))
    for s in range(B):
        h = y0[s]
        for t in range(T):
            h = M @ h + x[s, t]
            want[s, t] = h
    assert out["iters"] == 2
    np.testing.assert_allclose(out["history"][0], want, rtol=1e-12, atol=1e-12)
    assert out["trace"][1] <= 1e-12


def test_P4_P5_prefix_exact_after_k_bodies_and_T_bodies_suffice():
    """After k bodies the first k positions equal the sequential values, so
    max_iter = T with a negative tol reproduces the whole trajectory."""
    p, x, y0 = small(3, 2, 2, 8, seed=11, scale_y0=1.5)
    seq = oracle.gru_seq(p, x, y0)
    out = oracle.deer(p, x, y0, tol=-1.0, max_iter=8, want_history=True)
    assert out["iters"] == 8
    for k in range(1, 9):
        np.testing.assert_allclose(out["history"][k - 1][:, :k], seq[:, :k], rtol=0, atol=1e-14)
    np.testing.assert_allclose(out["y"], seq, rtol=0, atol=1e-14)


def test_P11_quadratic_convergence():
    """Near the solution the error roughly squares per body (App. A.3)."""
    p, x, y0 = small(4, 2, 1, 200, seed=5)
    seq = oracle.gru_seq(p, x, y0)
    guess = seq + 1e-3 * synth.normal(5, "t/noise", seq.shape).astype(np.float64)
    out = oracle.deer(p, x, y0, tol=-1.0, max_iter=3, y_guess=guess, want_history=True)
    e = [np.max(np.abs(h - seq)) for h in out["history"]]
    e0 = np.max(np.abs(guess - seq))
    assert e[0] < 50 * e0 ** 2 and e[0] < 1e-4
    assert e[1] < 50 * max(e[0] ** 2, 1e-16)
    assert e[1] < 1e-10


def test_loop_semantics_tol_and_max_iter():
    """err0 = 1e10, loop while err > tol and k < max_iter; iters counts bodies."""
    p, x, y0 = small(4, 2, 1, 50)
    assert oracle.deer(p, x, y0, max_iter=1)["iters"] == 1
    out = oracle.deer(p, x, y0, tol=1e30)
    # err0 = 1e10 < 1e30 means no body runs at all: the guess is returned
    assert out["iters"] == 0 and np.all(out["y"] == 0)
    full = oracle.deer(p, x, y0)
    assert full["trace"][-1] <= 1e-7 and (len(full["trace"]) == 1 or full["trace"][-2] > 1e-7)
    # T = 1: one body gives f(y0, x0); the second confirms
    p1, x1, y01 = small(4, 2, 2, 1)
    o1 = oracle.deer(p1, x1, y01)
    assert o1["iters"] == 2
    f, _ = oracle.gru_cell_jac(p1, y01, x1[:, 0])
    np.testing.assert_allclose(o1["y"][:, 0], f, rtol=0, atol=1e-15)


def test_nan_propagates_to_err():
    p, x, y0 = small(2, 2, 1, 20)
    x = x.copy(); x[0, 7, 1] = np.nan
    out = oracle.deer(p, x, y0, max_iter=10)
    assert math.isnan(out["err"]) and out["iters"] == 1


def test_P12_fp32_magnitude_and_tolerance_insensitivity():
    """fp32 DEER vs fp32 sequential differs by a few ulp at unit scale (the
    paper prints 1.788e-7 for GRU n=2, T=10k), and the iteration count moves by
    at most one between tol 1e-4 and 3e-7 (App. C.1)."""
    p = synth.gru_params(2, 2, 0, tag="p12/gru")
    x = synth.x_gaussian(1, 10000, 2, 0, tag="p12/x")
    y0 = np.zeros((1, 2), np.float32)
    seq = oracle.gru_seq(p, x, y0, np.float32)
    a = oracle.deer(p, x, y0, tol=1e-4, dtype=np.float32)
    b = oracle.deer(p, x, y0, tol=3e-7, dtype=np.float32)
    printed = GOLD["fp32_deer_vs_sequential_max_abs_err"]
    for o in (a, b):
        err = float(np.max(np.abs(o["y"] - seq)))
        assert err <= 8 * printed, err            # same order of magnitude as the printed value
    assert 0 <= b["iters"] - a["iters"] <= 1
    assert a["iters"] <= 12


def fd_grad(loss_fn, arr, idxs, eps=1e-6):
    out = []
    for idx in idxs:
        old = arr[idx]
        arr[idx] = old + eps; lp = loss_fn()
        arr[idx] = old - eps; lm = loss_fn()
        arr[idx] = old
        out.append((lp - lm) / (2 * eps))
    return np.array(out)


def test_P9_bptt_vs_finite_differences_and_deer_gradient():
    """BPTT equals central differences of the sequential loss; the DEER
    gradient (one reverse solve + cell VJP, Eq. 7) equals BPTT."""
    n, m, B, T = 3, 2, 2, 25
    p, x, y0 = small(n, m, B, T, seed=21)
    p = p.astype(np.float64); x = x.astype(np.float64); y0 = y0.astype(np.float64)
    gy = synth.normal(21, "t/gy", (B, T, n)).astype(np.float64)
    loss = lambda: float(np.sum(oracle.gru_seq(p, x, y0) * gy))
    y = oracle.gru_seq(p, x, y0)
    g = oracle.gru_bptt(p, x, y0, y, gy)
    checks = [
        (p.W_i, "dW_i", [(0, 0), (4, 1), (8, 0)]),
        (p.W_h, "dW_h", [(0, 2), (3, 1), (7, 0), (8, 2)]),
        (p.b_i, "db_i", [(0,), (4,), (8,)]),
        (p.b_h, "db_h", [(1,), (5,), (6,)]),
        (x, "dx", [(0, 0, 0), (1, 12, 1), (0, 24, 1)]),
        (y0, "dy0", [(0, 0), (1, 2)]),
    ]
    for arr, key, idxs in checks:
        fd = fd_grad(loss, arr, idxs)
        got = np.array([g[key][i] for i in idxs])
        np.testing.assert_allclose(got, fd, rtol=2e-7, atol=2e-8, err_msg=key)
    d = oracle.deer_grad(p, x, y0, y, gy)
    for key in ("dW_i", "dW_h", "db_i", "db_h", "dx", "dy0"):
        np.testing.assert_allclose(d[key], g[key], rtol=1e-11, atol=1e-12, err_msg=key)
    # gy only at the last position (loss = sum(y_T * w)) exercises the same path
    gy2 = np.zeros_like(gy); gy2[:, -1] = gy[:, -1]
    g2 = oracle.gru_bptt(p, x, y0, y, gy2); d2 = oracle.deer_grad(p, x, y0, y, gy2)
    loss2 = lambda: float(np.sum(oracle.gru_seq(p, x, y0)[:, -1] * gy[:, -1]))
    fd = fd_grad(loss2, p.W_h, [(2, 1), (6, 0)])
    np.testing.assert_allclose([g2["dW_h"][2, 1], g2["dW_h"][6, 0]], fd, rtol=2e-7, atol=2e-9)
    np.testing.assert_allclose(d2["dW_h"], g2["dW_h"], rtol=1e-11, atol=1e-13)


def test_classifier_loss_and_gradients():
    """O-5 against a numpy restatement of pool/head/loss on the oracle's
    states, and its gradients against central differences."""
    w = synth.config4(seed=3, B=3, T=12, n=4, m=2, n_classes=3)
    l1, l2 = [l.astype(np.float64) for l in w.layers]
    W_o = w.W_o.astype(np.float64); b_o = w.b_o.astype(np.float64)
    x = w.x.astype(np.float64)
    out = oracle.classifier([l1, l2], W_o, b_o, x, w.labels, want_states=True)
    z0 = np.zeros((3, 4))
    y1 = oracle.gru_seq(l1, x, z0); y2 = oracle.gru_seq(l2, y1, z0)
    np.testing.assert_allclose(out["y2"], y2, rtol=0, atol=0)
    logits = y2.mean(axis=1) @ W_o.T + b_o
    lse = np.log(np.sum(np.exp(logits), axis=1))
    want = float(np.mean(lse - logits[np.arange(3), w.labels]))
    assert abs(out["loss"] - want) < 1e-13
    loss = lambda: oracle.classifier([l1, l2], W_o, b_o, x, w.labels, want_grad=False)["loss"]
    for arr, key, idxs in [
        (l1.W_i, "dW_i1", [(0, 0), (9, 1)]), (l1.W_h, "dW_h1", [(2, 3), (11, 0)]),
        (l1.b_i, "db_i1", [(5,)]), (l1.b_h, "db_h1", [(10,)]),
        (l2.W_i, "dW_i2", [(1, 2), (8, 3)]), (l2.W_h, "dW_h2", [(0, 0), (7, 1)]),
        (l2.b_i, "db_i2", [(3,)]), (l2.b_h, "db_h2", [(9,)]),
        (W_o, "dW_o", [(0, 1), (2, 3)]), (b_o, "db_o", [(1,)]),
    ]:
        fd = fd_grad(loss, arr, idxs)
        got = np.array([out[key][i] for i in idxs])
        np.testing.assert_allclose(got, fd, rtol=5e-7, atol=2e-9, err_msg=key)


def test_synth_is_deterministic_and_distributed_as_documented():
    a = synth.normal(0, "s/a", (200000,), dtype=np.float64)
    assert abs(a.mean()) < 0.01 and abs(a.std() - 1.0) < 0.01
    np.testing.assert_array_equal(a[:100], synth.normal(0, "s/a", (100,), dtype=np.float64))
    u = synth.uniform(0, "s/u", (100000,), -0.5, 0.5, dtype=np.float64)
    assert u.min() > -0.5 and u.max() < 0.5 and abs(u.mean()) < 0.01
    # first SplitMix64 output for state 0 (published test vector of the generator)
    assert int(synth._mix(np.array([0x9E3779B97F4A7C15], dtype=np.uint64))[0]) == 0xE220A8397B1DCDAF
    w = synth.config(2, B=2, T=50)
    assert w.x.shape == (2, 50, 4) and w.params.W_h.shape == (24, 8)
    assert np.all(np.abs(w.params.W_h) <= 1 / math.sqrt(8))
    rw = synth.x_random_walk(2, 500, 3, 0)
    np.testing.assert_allclose(rw.mean(axis=1), 0, atol=1e-5)
    np.testing.assert_allclose(rw.std(axis=1), 1, atol=1e-4)


# ----------------------------------------------------------------------------- multi-head GRU (Sec. 4.4, App. B.4)
def mh_case(H, n, m, B, T, strides, seed=5):
    heads = synth.multihead_params(H, n, m, seed, tag="t/mh")
    x = synth.x_gaussian(B, T, m, seed, tag="t/mhx")
    y0 = synth.normal(seed, "t/mhy0", (B, H, n)) * 0.5
    return heads, np.asarray(strides, np.int32), x, y0


def test_multihead_reading_reproduces_the_papers_parameter_count():
    """The paper prints the model's parameter count (App. B.4) but not how a head is wired.  The reading
    taken here -- every head is a GRU of 8 channels that reads ALL 256 input channels, with the
    parameters of the cited GRU cell (input kernels with biases for r, z, n; hidden kernels without bias
    for r, z and with bias for n) -- gives exactly that count; heads reading only a 1/32 slice of the
    input would not."""
    H, n, m, layers = 32, 8, 256, 4
    head = 3 * (m * n + n) + 3 * n * n + n
    composite = H * head + (256 * 512 + 512) + 2 * 256          # multi-head GRU, linear 256 -> 512 (GLU has none), layer norm
    total = (3 * 256 + 256) + layers * composite + (256 * 10 + 10)
    assert total == int(GOLD["multihead_model_trainable_parameters"])
    sliced = 3 * ((m // H) * n + n) + 3 * n * n + n
    assert (3 * 256 + 256) + layers * (H * sliced + 256 * 512 + 512 + 512) + 2570 != total


def test_multihead_one_head_stride_one_is_the_plain_gru():
    heads, st, x, y0 = mh_case(1, 4, 3, 2, 50, [1])
    y = oracle.multihead_seq(heads, st, x, y0)
    assert np.array_equal(y[:, :, 0], oracle.gru_seq(heads[0], x, y0[:, 0]))


def test_multihead_strided_head_is_interleaved_sequences_and_heads_are_independent():
    """Head h with stride s is s independent GRU runs over x[:, p::s], each from y0 (Sec. 4.4)."""
    strides = [1, 2, 4, 3]
    heads, st, x, y0 = mh_case(4, 3, 5, 2, 41, strides)
    y = oracle.multihead_seq(heads, st, x, y0)
    for h, s in enumerate(strides):
        for p in range(s):
            want = oracle.gru_seq(heads[h], x[:, p::s], y0[:, h])
            assert np.array_equal(y[:, p::s, h], want), (h, p)
    for dtype in (np.float32,):
        y32 = oracle.multihead_seq(heads, st, x, y0, dtype)
        assert np.max(np.abs(y32 - y)) <= 2e-6


def test_multihead_bptt_matches_finite_differences():
    strides = [2, 1, 3]
    heads, st, x, y0 = mh_case(3, 2, 2, 2, 9, strides)
    gy = synth.normal(9, "t/mhgy", (2, 9, 3, 2)).astype(np.float64)
    loss = lambda hd, xx, yy0: float(np.sum(gy * oracle.multihead_seq(hd, st, xx, yy0)))
    y = oracle.multihead_seq(heads, st, x, y0)
    g = oracle.multihead_bptt(heads, st, x, y0, y, gy)
    eps = 1e-6
    x64, y064 = x.astype(np.float64), y0.astype(np.float64)
    h64 = [h.astype(np.float64) for h in heads]
    for hh in range(3):
        for name in ("W_i", "W_h", "b_i", "b_h"):
            arr = getattr(h64[hh], name)
            for idx in list(np.ndindex(arr.shape))[::3]:
                old = arr[idx]
                arr[idx] = old + eps; lp = loss(h64, x64, y064)
                arr[idx] = old - eps; lm = loss(h64, x64, y064)
                arr[idx] = old
                assert abs((lp - lm) / (2 * eps) - g["d" + name][(hh,) + idx]) <= 1e-7, (hh, name, idx)
    for arr, key in ((x64, "dx"), (y064, "dy0")):
        for idx in list(np.ndindex(arr.shape))[::2]:
            old = arr[idx]
            arr[idx] = old + eps; lp = loss(h64, x64, y064)
            arr[idx] = old - eps; lm = loss(h64, x64, y064)
            arr[idx] = old
            assert abs((lp - lm) / (2 * eps) - g[key][idx]) <= 1e-7, (key, idx)


def test_multihead_bptt_reduces_to_plain_bptt_per_phase():
    """One head of stride s: its gradient is the sum of plain BPTT over the s interleaved sequences."""
    s = 3
    heads, st, x, y0 = mh_case(1, 3, 2, 2, 20, [s])
    y = oracle.multihead_seq(heads, st, x, y0)
    gy = synth.normal(4, "t/mhgy2", y.shape).astype(np.float64)
    g = oracle.multihead_bptt(heads, st, x, y0, y, gy)
    acc = None
    for p in range(s):
        gp = oracle.gru_bptt(heads[0], x[:, p::s], y0[:, 0], y[:, p::s, 0], gy[:, p::s, 0])
        assert np.allclose(g["dx"][:, p::s], gp["dx"], atol=1e-13)
        gp = {k: gp[k] for k in ("dW_i", "dW_h", "db_i", "db_h", "dy0")}
        acc = gp if acc is None else {k: acc[k] + gp[k] for k in gp}
    for k in ("dW_i", "dW_h", "db_i", "db_h"):
        assert np.allclose(g[k][0], acc[k], atol=1e-12), k
    assert np.allclose(g["dy0"][:, 0], acc["dy0"], atol=1e-13)


# ----------------------------------------------------------------------------- forward-mode derivative (Sec. 3.1.1)
def test_jvp_matches_central_differences_of_the_sequential_trajectory():
    """dy = L_G^{-1}[df/dtheta dtheta] (+ the x and y0 directions): the tangent recurrence against the
    difference quotient of the sequential evaluation along the same direction."""
    p, x, y0 = small(3, 2, 2, 25, seed=8)
    p64 = p.astype(np.float64); x64 = x.astype(np.float64); y064 = y0.astype(np.float64)
    dp = synth.GruParams(3, 2, *(synth.normal(8, f"t/dp{i}", a.shape).astype(np.float64)
                                 for i, a in enumerate((p.W_i, p.W_h, p.b_i, p.b_h))))
    dx = synth.normal(8, "t/dx", x.shape).astype(np.float64)
    dy0 = synth.normal(8, "t/dy0", y0.shape).astype(np.float64)
    y = oracle.gru_seq(p64, x64, y064)
    eps = 1e-6

    def shifted(sign, use_p, use_x, use_y0):
        q = synth.GruParams(3, 2, *((a + sign * eps * d) if use_p else a for a, d in
                                    ((p64.W_i, dp.W_i), (p64.W_h, dp.W_h), (p64.b_i, dp.b_i), (p64.b_h, dp.b_h))))
        return oracle.gru_seq(q, x64 + (sign * eps * dx if use_x else 0.0), y064 + (sign * eps * dy0 if use_y0 else 0.0))

    for use_p, use_x, use_y0 in ((True, False, False), (False, True, False), (False, False, True), (True, True, True)):
        fd = (shifted(+1, use_p, use_x, use_y0) - shifted(-1, use_p, use_x, use_y0)) / (2 * eps)
        got = oracle.gru_jvp(p64, dp if use_p else None, x64, dx if use_x else None, y064,
                             dy0 if use_y0 else None, y)
        assert np.max(np.abs(got - fd)) <= 2e-8, (use_p, use_x, use_y0)


def test_jvp_is_the_transpose_of_the_gradient():
    """<gy, dy> = <dL/dtheta, dtheta> + <dL/dx, dx> + <dL/dy0, dy0>: the forward derivative paired with any
    gy equals the backward derivative (Sec. 3.1.1, both equations) paired with the direction."""
    p, x, y0 = small(4, 3, 2, 30, seed=9)
    p64 = p.astype(np.float64)
    y = oracle.gru_seq(p64, x, y0)
    dp = synth.GruParams(4, 3, *(synth.normal(9, f"t/dq{i}", a.shape).astype(np.float64)
                                 for i, a in enumerate((p.W_i, p.W_h, p.b_i, p.b_h))))
    dx = synth.normal(9, "t/dx2", x.shape).astype(np.float64)
    dy0 = synth.normal(9, "t/dy02", y0.shape).astype(np.float64)
    gy = synth.normal(9, "t/gy2", y.shape).astype(np.float64)
    dy = oracle.gru_jvp(p64, dp, x, dx, y0, dy0, y)
    g = oracle.gru_bptt(p64, x, y0, y, gy)
    rhs = sum(float(np.sum(g["d" + k] * getattr(dp, k))) for k in ("W_i", "W_h", "b_i", "b_h"))
    rhs += float(np.sum(g["dx"] * dx)) + float(np.sum(g["dy0"] * dy0))
    assert abs(float(np.sum(gy * dy)) - rhs) <= 1e-10 * max(1.0, abs(rhs))


# ----------------------------------------------------------------------------- ODE instantiation of L_G^{-1} (Sec. 3.3)
def test_ode_scalar_closed_form():
    """n = 1, constant g and z: y_{i+1} = e^{-g D} y_i + (1 - e^{-g D}) z / g exactly."""
    g, zc, T = 0.7, -0.4, 40
    t = np.cumsum(synth.uniform(1, "o/dt", (T,), 0.01, 0.3, dtype=np.float64))
    y = oracle.ode_linear(np.full((1, T, 1, 1), g), np.full((1, T, 1), zc), t, np.array([[1.5]]))
    want = zc / g + (1.5 - zc / g) * np.exp(-g * (t - t[0]))
    assert np.max(np.abs(y[0, :, 0] - want)) <= 1e-13


def test_ode_discretisation_against_a_library_exponential():
    scipy_linalg = pytest.importorskip("scipy.linalg")
    B, T, n = 2, 6, 4
    G = synth.normal(2, "o/G", (B, T, n, n)).astype(np.float64)
    z = synth.normal(2, "o/z", (B, T, n)).astype(np.float64)
    t = np.cumsum(synth.uniform(2, "o/dt2", (T,), 0.05, 0.5, dtype=np.float64))
    y0 = synth.normal(2, "o/y0", (B, n)).astype(np.float64)
    y, Gb, zb = oracle.ode_linear(G, z, t, y0, want_discrete=True)
    for b in range(B):
        for k in range(T - 1):
            Gm = 0.5 * (G[b, k] + G[b, k + 1]); zm = 0.5 * (z[b, k] + z[b, k + 1]); D = t[k + 1] - t[k]
            E = scipy_linalg.expm(-Gm * D)
            assert np.max(np.abs(Gb[b, k] - E)) <= 1e-12 * max(1.0, np.max(np.abs(E)))
            zbar = np.linalg.solve(Gm, (np.eye(n) - E) @ zm)           # G^{-1}(I - Gbar) z as printed in Sec. 3.3
            assert np.max(np.abs(zb[b, k] - zbar)) <= 1e-10 * max(1.0, np.max(np.abs(zbar)))
            assert np.allclose(y[b, k + 1], E @ y[b, k] + zbar, atol=1e-10)


def test_ode_constant_coefficients_are_exact_and_singular_G_is_fine():
    scipy_linalg = pytest.importorskip("scipy.linalg")
    n, T = 3, 30
    G0 = synth.normal(3, "o/G0", (n, n)).astype(np.float64) * 0.8 + 1.5 * np.eye(n)
    z0 = synth.normal(3, "o/z0", (n,)).astype(np.float64)
    t = np.linspace(0.0, 3.0, T)
    y0 = np.array([[0.5, -1.0, 2.0]])
    y = oracle.ode_linear(np.broadcast_to(G0, (1, T, n, n)), np.broadcast_to(z0, (1, T, n)), t, y0)
    yinf = np.linalg.solve(G0, z0)
    for k in range(T):
        want = scipy_linalg.expm(-G0 * t[k]) @ (y0[0] - yinf) + yinf
        assert np.max(np.abs(y[0, k] - want)) <= 1e-11
    # G = 0: dy/dt = z(t), mid-point rule = trapezoid
    zt = np.sin(t)[None, :, None] * np.ones((1, T, n))
    y = oracle.ode_linear(np.zeros((1, T, n, n)), zt, t, y0)
    trap = np.concatenate([[0.0], np.cumsum(0.5 * (np.sin(t[1:]) + np.sin(t[:-1])) * np.diff(t))])
    assert np.max(np.abs(y[0] - (y0[0][None, :] + trap[:, None]))) <= 1e-13


def test_ode_midpoint_rule_converges_with_second_order():
    """App. A.5: local truncation error O(D^3) with mid-point values, hence global O(D^2):
    halving the step divides the error by about four (reference: a very fine grid)."""
    n = 2
    Gf = lambda tt: np.array([[1.0 + 0.5 * np.sin(tt), 0.3 * tt], [-0.4, 0.8 + 0.2 * np.cos(2 * tt)]])
    zf = lambda tt: np.array([np.cos(tt), 0.5 * tt])
    y0 = np.array([[1.0, -0.5]])

    def solve(T):
        t = np.linspace(0.0, 2.0, T)
        G = np.stack([Gf(v) for v in t])[None]; z = np.stack([zf(v) for v in t])[None]
        return oracle.ode_linear(G, z, t, y0)[0, -1]

    ref = solve(20001)
    e1, e2, e3 = (np.max(np.abs(solve(T) - ref)) for T in (21, 41, 81))
    assert 3.5 <= e1 / e2 <= 4.5 and 3.5 <= e2 / e3 <= 4.5


# ----------------------------------------------------------------------------- a second cell: LSTM (Sec. 3.4: any f)
def test_lstm_matches_a_library_lstm():
    """The oracle's LSTM against torch.nn.LSTM on CPU with the same weights (gate order i, f, g, o)."""
    torch = pytest.importorskip("torch")
    k, m, B, T = 5, 3, 2, 40
    p = synth.lstm_params(k, m, 3, tag="t/lstm")
    x = synth.x_gaussian(B, T, m, 3, tag="t/lx").astype(np.float64)
    s0 = synth.normal(3, "t/ls0", (B, 2 * k)).astype(np.float64) * 0.5
    net = torch.nn.LSTM(m, k, batch_first=True).double()
    with torch.no_grad():
        net.weight_ih_l0.copy_(torch.from_numpy(p.W_i.astype(np.float64)))
        net.weight_hh_l0.copy_(torch.from_numpy(p.W_h.astype(np.float64)))
        net.bias_ih_l0.copy_(torch.from_numpy(p.b.astype(np.float64)))
        net.bias_hh_l0.zero_()
        h0 = torch.from_numpy(s0[:, :k].copy())[None]; c0 = torch.from_numpy(s0[:, k:].copy())[None]
        hs = []
        state = (h0, c0)
        for t in range(T):                        # step by step to read c as well
            out, state = net(torch.from_numpy(x[:, t:t + 1]), state)
            hs.append(np.concatenate([state[0][0].numpy(), state[1][0].numpy()], axis=1))
    want = np.stack(hs, axis=1)
    got = oracle.lstm_seq(p, x, s0)
    assert np.max(np.abs(got - want)) <= 1e-12


def test_lstm_jacobian_matches_central_differences_and_deer_returns_the_sequence():
    k, m, B, T = 3, 2, 2, 60
    p = synth.lstm_params(k, m, 4, tag="t/lstm2")
    x = synth.x_gaussian(B, T, m, 4, tag="t/lx2").astype(np.float64)
    s0 = synth.normal(4, "t/ls02", (B, 2 * k)).astype(np.float64) * 0.5
    sp = synth.normal(4, "t/lsp", (7, 2 * k)).astype(np.float64)
    xs = synth.normal(4, "t/lxs", (7, m)).astype(np.float64)
    f, J = oracle.lstm_cell_jac(p, sp, xs)
    eps = 1e-6
    for j in range(2 * k):
        d = np.zeros(2 * k); d[j] = eps
        fp, _ = oracle.lstm_cell_jac(p, sp + d, xs, want_J=False)
        fm, _ = oracle.lstm_cell_jac(p, sp - d, xs, want_J=False)
        assert np.max(np.abs((fp - fm) / (2 * eps) - J[:, :, j])) <= 1e-8
    seq = oracle.lstm_seq(p, x, s0)
    o = oracle.deer(p, x, s0, tol=1e-9, dtype=np.float64, cell="lstm")
    assert o["iters"] < 30 and np.max(np.abs(o["y"] - seq)) <= 1e-11
    o32 = oracle.deer(p, x, s0, tol=1e-4, dtype=np.float32, cell="lstm")
    assert np.max(np.abs(o32["y"] - seq)) <= 5e-6
