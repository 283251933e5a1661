"""Parity of the CUDA path (through the C ABI) with the CPU oracle, element by
element on the same seeded inputs.  Tolerances (stated by the benchmark
definition): trajectories within 1e-4 max-abs of the sequential fp32
trajectory; gradients within 1e-3 relative (inf-norm per tensor) of BPTT;
the stand-alone scan within 1e-5 * max|y| of the fp64 sequential solve."""
import numpy as np
import pytest
import torch

import oracle
from paper_2309_12252_b200 import synth

pytestmark = pytest.mark.gpu

TOL_Y = 1e-4
TOL_GRAD = 1e-3
TOL_SCAN = 1e-5


@pytest.fixture(scope="module")
def bd():
    from paper_2309_12252_b200 import binding
    binding.lib()
    return binding


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def rel_inf(a, b):
    return float(np.max(np.abs(a - b)) / max(np.max(np.abs(b)), 1e-30))


# ----------------------------------------------------------------------------- scan
SCAN_CASES = [  # (n, B, T)
    (1, 3, 1), (1, 2, 2), (1, 4, 4097), (2, 3, 1000), (3, 2, 257), (4, 1, 1000), (4, 5, 2049),
    (5, 2, 130), (8, 2, 1), (8, 3, 2), (8, 16, 1111), (8, 1, 5000), (16, 3, 515), (32, 2, 300),
    (64, 2, 70), (7, 1, 63), (1, 3, 20001), (1, 1, 40000), (2, 2, 6001), (2, 3, 1001), (4, 1, 10000),
    (8, 2, 193), (8, 2, 192), (8, 5, 191), (4, 3, 769),
    # more sequences than resolver warps (several sequences per warp), and sequences with more tiles than
    # one resolver visit looks at
    (4, 40, 1500), (2, 70, 5000), (1, 70, 15000), (8, 40, 700), (4, 2, 30001), (2, 1, 50000), (1, 1, 150000),
    # tiny T and tile boundaries of the n = 4 and n = 2 kernels (640 and 2304 positions per tile)
    (4, 2, 1), (4, 3, 2), (4, 2, 5), (4, 1, 640), (4, 2, 641), (4, 1, 1279), (2, 2, 1), (2, 1, 2304), (2, 2, 2305),
]


@pytest.mark.parametrize("n,B,T", SCAN_CASES)
@pytest.mark.parametrize("reverse", [False, True])
@pytest.mark.parametrize("flags", [0, 2])
def test_linrec_scan_vs_oracle(bd, n, B, T, reverse, flags):
    J = synth.contractive_J(B, T, n, seed=n + T, tag="g/J", scale=1.0)
    b = synth.normal(n + T, "g/b", (B, T, n))
    y0 = synth.normal(n + T, "g/y0", (B, n))
    for y0_used in (y0, None):
        want = oracle.linrec(J, b, y0_used, reverse=reverse, dtype=np.float64)
        got = bd.deer_linrec_scan(dev(J), dev(b), None if y0_used is None else dev(y0), reverse=reverse,
                                  flags=flags).cpu().numpy()
        scale = max(1.0, float(np.max(np.abs(want))))
        assert np.max(np.abs(got - want)) <= TOL_SCAN * scale


@pytest.mark.parametrize("B,T", [(2, 70), (3, 64), (2, 1), (4, 1000), (16, 333)])
@pytest.mark.parametrize("reverse", [False, True])
def test_linrec_scan_n64_tcgen05_path(bd, B, T, reverse):
    """The n = 64 chain product on tcgen05 (tensor-memory accumulator) gives the same scan."""
    n = 64
    J = synth.contractive_J(B, T, n, seed=7 + T, tag="g/J64", scale=1.0)
    b = synth.normal(7 + T, "g/b64", (B, T, n))
    y0 = synth.normal(7 + T, "g/y064", (B, n))
    want = oracle.linrec(J, b, y0, reverse=reverse, dtype=np.float64)
    got = bd.deer_linrec_scan(dev(J), dev(b), dev(y0), reverse=reverse, flags=bd.DEER_FLAG_TCGEN05).cpu().numpy()
    assert np.max(np.abs(got - want)) <= TOL_SCAN * max(1.0, float(np.max(np.abs(want))))


def test_linrec_scan_growing_products(bd):
    """Non-contractive J (norm > 1 over short stretches): error relative to max|y|."""
    n, B, T = 4, 2, 60
    J = synth.uniform(3, "g/Jbig", (B, T, n, n), -0.6, 0.6)
    b = synth.normal(3, "g/bbig", (B, T, n))
    want = oracle.linrec(J, b, None, dtype=np.float64)
    got = bd.deer_linrec_scan(dev(J), dev(b)).cpu().numpy()
    assert np.max(np.abs(got - want)) <= TOL_SCAN * max(1.0, np.max(np.abs(want)))


def test_scan_is_bit_reproducible(bd):
    n, B, T = 8, 4, 3000
    J = dev(synth.contractive_J(B, T, n, seed=1, tag="g/Jr")); b = dev(synth.normal(1, "g/br", (B, T, n)))
    a = bd.deer_linrec_scan(J, b).clone()
    for _ in range(3):
        assert torch.equal(a, bd.deer_linrec_scan(J, b))


# ----------------------------------------------------------------------------- forward evaluation
def run_eval(bd, w, **kw):
    p = bd.GruParamsDev.from_numpy(w.params)
    return bd.deer_gru_eval(p, dev(w.x), dev(w.y0), **kw)


@pytest.mark.parametrize("n,m,B,T", [(1, 1, 2, 50), (2, 3, 3, 333), (3, 2, 2, 100), (4, 2, 1, 1000),
                                     (8, 4, 4, 2500), (16, 16, 2, 700), (32, 32, 2, 400),
                                     (64, 6, 2, 150), (5, 7, 3, 129),
                                     # input-projection shapes: tensor-core path with ragged position tiles
                                     # (m % 8 == 0, m >= 16), tiled path otherwise
                                     (8, 16, 3, 77), (16, 24, 1, 131), (32, 8, 2, 200), (64, 64, 1, 300)])
@pytest.mark.parametrize("flags", [0, 2, 4])
def test_eval_matches_sequential(bd, n, m, B, T, flags):
    p = synth.gru_params(n, m, seed=7, tag="e/gru")
    x = synth.x_gaussian(B, T, m, seed=7, tag="e/x")
    y0 = synth.normal(7, "e/y0", (B, n)) * 0.5
    w = synth.Workload("t", B, T, n, m, p, x, y0)
    r = run_eval(bd, w, flags=flags)
    seq32 = oracle.gru_seq(p, x, y0, np.float32)
    seq64 = oracle.gru_seq(p, x, y0, np.float64)
    got = r.y.cpu().numpy()
    assert r.status == 0 and r.err <= 1e-4
    assert np.max(np.abs(got - seq32)) <= TOL_Y
    assert np.max(np.abs(got - seq64)) <= TOL_Y
    o = oracle.deer(p, x, y0, tol=1e-4, dtype=np.float32)
    assert abs(r.iters - o["iters"]) <= 1


def test_first_iterate_matches_oracle_iteration(bd):
    """One body from the zero guess equals the oracle's first Newton iterate
    (checks cell, Jacobian, rhs and scan together before convergence hides them)."""
    w = synth.config(2, B=3, T=800)
    r = run_eval(bd, w, tol=-1.0, max_iter=1)
    o = oracle.deer(w.params, w.x, w.y0, tol=-1.0, max_iter=1, dtype=np.float64)
    assert r.iters == 1 and r.status == 0
    assert np.max(np.abs(r.y.cpu().numpy() - o["y"])) <= 2e-5
    assert abs(r.err - o["err"]) <= 1e-5 * max(1.0, o["err"])


def test_config1_full(bd):
    w = synth.config(1)
    r = run_eval(bd, w)
    seq32 = oracle.gru_seq(w.params, w.x, w.y0, np.float32)
    assert r.status == 0 and np.max(np.abs(r.y.cpu().numpy() - seq32)) <= TOL_Y
    o = oracle.deer(w.params, w.x, w.y0, tol=1e-4, dtype=np.float32)
    assert abs(r.iters - o["iters"]) <= 1


def test_config2_full_and_scan_on_generated_J(bd):
    w = synth.config(2)
    r = run_eval(bd, w)
    seq32 = oracle.gru_seq(w.params, w.x, w.y0, np.float32)
    got = r.y.cpu().numpy()
    assert r.status == 0 and np.max(np.abs(got - seq32)) <= TOL_Y
    # scan alone on the J, b of the converged trajectory (oracle generates them in fp64)
    yprev = np.concatenate([w.y0[:, None], seq32[:, :-1]], axis=1).astype(np.float64)
    f, J = oracle.gru_cell_jac(w.params, yprev.reshape(-1, 8), w.x.reshape(-1, 4))
    J = J.reshape(16, 10000, 8, 8); f = f.reshape(16, 10000, 8)
    rhs = f - np.einsum("btij,btj->bti", J, yprev)
    want = oracle.linrec(J, rhs, w.y0, dtype=np.float64)
    y = bd.deer_linrec_scan(dev(J.astype(np.float32)), dev(rhs.astype(np.float32)), dev(w.y0)).cpu().numpy()
    assert np.max(np.abs(y - want)) <= TOL_SCAN * max(1.0, np.max(np.abs(want)))


def test_config3_forward_sampled_sequences(bd):
    """Full-size config 3 on the GPU; the oracle checks every element (it is sequential and fast)."""
    w = synth.config(3)
    r = run_eval(bd, w)
    assert r.status == 0
    seq32 = oracle.gru_seq(w.params, w.x, w.y0, np.float32)
    assert np.max(np.abs(r.y.cpu().numpy() - seq32)) <= TOL_Y


def test_edge_T1_T2_and_status_codes(bd):
    for T in (1, 2):
        w = synth.config(1, B=3, T=T)
        r = run_eval(bd, w)
        seq = oracle.gru_seq(w.params, w.x, w.y0, np.float32)
        assert np.max(np.abs(r.y.cpu().numpy() - seq)) <= 1e-6
        assert 2 <= r.iters <= T + 1 and r.status == 0
    w = synth.config(2, B=2, T=500)
    r = run_eval(bd, w, max_iter=1)
    assert r.status == bd.DEER_NOT_CONVERGED and r.iters == 1
    r = run_eval(bd, w, tol=-1.0, max_iter=3)
    assert r.status == 0 and r.iters == 3
    x = w.x.copy(); x[1, 77, 2] = np.nan
    r = run_eval(bd, synth.Workload("nan", 2, 500, 8, 4, w.params, x, w.y0))
    assert r.status == bd.DEER_NONFINITE
    # invalid arguments are refused, nothing runs
    p = bd.GruParamsDev.from_numpy(w.params)
    xd, y0d = dev(w.x), dev(w.y0)
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    r = bd.deer_gru_eval(p, xd, y0d, ws=small, check=False)
    assert r.status == bd.DEER_ERR_WORKSPACE
    r = bd.deer_gru_eval(p, xd, y0d, max_iter=0, check=False)
    assert r.status == bd.DEER_ERR_INVALID_ARG
    r = bd.deer_gru_eval(p, xd, y0d, tol=float("nan"), check=False)
    assert r.status == bd.DEER_ERR_INVALID_ARG
    assert bd.deer_workspace_bytes(bd.DEER_OP_SCAN, 1, 10, 65) == 0
    J = torch.zeros((1, 4, 65, 65), device="cuda"); b = torch.zeros((1, 4, 65), device="cuda")
    _, rc = bd.deer_linrec_scan(J, b, ws=small, check=False)
    assert rc == bd.DEER_ERR_UNSUPPORTED_N


def test_eval_is_bit_reproducible_and_warm_start(bd):
    w = synth.config(2, B=4, T=3000)
    a = run_eval(bd, w)
    b = run_eval(bd, w)
    assert a.iters == b.iters and torch.equal(a.y, b.y) and a.err == b.err
    assert np.array_equal(a.err_trace, b.err_trace)
    # warm start from the solution: converges in the confirming body (plus at most one)
    p = bd.GruParamsDev.from_numpy(w.params)
    y = a.y.clone()
    r = bd.deer_gru_eval(p, dev(w.x), dev(w.y0), y=y, flags=bd.DEER_FLAG_WARM_START)
    assert r.iters <= 2 and r.status == 0
    assert torch.max(torch.abs(r.y - a.y)).item() <= 1e-5


@pytest.mark.parametrize("max_iter,tol", [(100, 1e-4), (3, 1e-4), (5, -1.0), (7, -1.0)])
def test_eval_with_host_buffers_matches_device_call(bd, max_iter, tol):
    """deer_gru_eval_host (copies inside the library, result selected on the device) returns exactly what
    deer_gru_eval returns, for even and odd body counts and for more bodies than the first group."""
    w = synth.config(2, B=3, T=1200)
    p = bd.GruParamsDev.from_numpy(w.params)
    ref = bd.deer_gru_eval(p, dev(w.x), dev(w.y0), tol=tol, max_iter=max_iter, check=False)
    x_host = torch.from_numpy(np.ascontiguousarray(w.x)).pin_memory()
    y_host = torch.empty((3, 1200, 8), dtype=torch.float32).pin_memory()
    x_dev = torch.empty((3, 1200, 4), device="cuda"); y_dev = torch.empty((3, 1200, 8), device="cuda")
    ws = bd.alloc_workspace(bd.DEER_OP_EVAL, 3, 1200, 8, 4, 0, x_dev.device)
    r = bd.deer_gru_eval_host(p, x_host, dev(w.y0), y_host, x_dev, y_dev, ws, tol=tol, max_iter=max_iter)
    assert (r.iters, r.status) == (ref.iters, ref.status) and r.err == ref.err
    assert torch.equal(y_host, ref.y.cpu()) and torch.equal(y_dev, ref.y)


@pytest.mark.parametrize("n,m,B,T", [(8, 4, 5, 200_000), (32, 32, 3, 300_000)])
def test_eval_with_host_buffers_in_chunks_of_sequences(bd, n, m, B, T):
    """A batch that deer_gru_eval_host splits (copies of the neighbouring chunks overlap an evaluation): every chunk
    holds exactly what deer_gru_eval returns for those sequences alone, iters / err are the largest over the chunks, and
    the whole agrees with the unsplit device call within the tolerance the iteration is solved to."""
    first = bd.deer_gru_eval_host_chunks(B, T)
    assert len(first) >= 3 and first[0] == 0 and first[-1] == B
    p_np = synth.gru_params(n, m, 5, tag="hc/gru")
    x_np = synth.x_gaussian(B, T, m, 5, tag="hc/x")
    y0_np = (synth.normal(5, "hc/y0", (B, n)) * 0.3).astype(np.float32)
    p = bd.GruParamsDev.from_numpy(p_np)
    x_host = torch.from_numpy(np.ascontiguousarray(x_np)).pin_memory()
    y_host = torch.empty((B, T, n), dtype=torch.float32).pin_memory()
    x_dev = torch.empty((B, T, m), device="cuda"); y_dev = torch.empty((B, T, n), device="cuda")
    ws = bd.alloc_workspace(bd.DEER_OP_EVAL, B, T, n, m, 0, x_dev.device)
    r = bd.deer_gru_eval_host(p, x_host, dev(y0_np), y_host, x_dev, y_dev, ws)
    assert r.status == 0 and torch.equal(y_dev.cpu(), y_host)
    its, errs = [], []
    for b0, b1 in zip(first[:-1], first[1:]):
        rc = bd.deer_gru_eval(p, dev(x_np[b0:b1]), dev(y0_np[b0:b1]))
        assert torch.equal(rc.y.cpu(), y_host[b0:b1])
        its.append(rc.iters); errs.append(rc.err)
    assert r.iters == max(its) and r.err == max(errs)
    whole = bd.deer_gru_eval(p, dev(x_np), dev(y0_np))
    assert torch.max(torch.abs(whole.y.cpu() - y_host)).item() <= 1e-4
    # the second call on the same buffers (copy streams and events are reused)
    y_host.zero_()
    r2 = bd.deer_gru_eval_host(p, x_host, dev(y0_np), y_host, x_dev, y_dev, ws)
    assert (r2.iters, r2.err) == (r.iters, r.err) and torch.equal(y_dev.cpu(), y_host)


@pytest.mark.parametrize("n,m,B,T,k", [(8, 4, 5, 700, 3), (8, 4, 5, 700, 4), (4, 2, 3, 1000, 2), (32, 32, 2, 300, 3),
                                       (2, 2, 4, 50, 1)])
def test_eval_diagnostics_of_the_last_body(bd, n, m, B, T, k):
    """err_b and err_argmax describe max |y_k - y_{k-1}|: checked against the two iterates themselves
    (exactly k and k - 1 bodies from the same start are bit-reproducible), ties to the smallest index,
    identical across runs."""
    p_np = synth.gru_params(n, m, 3, tag="d/gru")
    x = dev(synth.x_gaussian(B, T, m, 3, tag="d/x"))
    y0 = dev(synth.normal(3, "d/y0", (B, n)) * 0.3)
    p = bd.GruParamsDev.from_numpy(p_np)
    r, err_b, amax = bd.deer_gru_eval_diag(p, x, y0, tol=-1.0, max_iter=k)
    r2, err_b2, amax2 = bd.deer_gru_eval_diag(p, x, y0, tol=-1.0, max_iter=k)
    assert r.iters == k and amax == amax2 and np.array_equal(err_b, err_b2) and torch.equal(r.y, r2.y)
    prev = (bd.deer_gru_eval(p, x, y0, tol=-1.0, max_iter=k - 1, check=False).y if k > 1
            else torch.zeros_like(r.y))
    d = (r.y - prev).abs().cpu().numpy()
    assert np.array_equal(err_b, d.reshape(B, -1).max(axis=1))
    assert float(err_b.max()) == r.err
    assert amax == int(np.argmax(d.reshape(-1)))          # numpy: first occurrence of the maximum


@pytest.mark.parametrize("n,m,B,T", [(16, 16, 3, 900), (32, 32, 2, 700), (16, 5, 2, 333), (32, 8, 1, 65), (64, 6, 2, 500),
                                     (64, 64, 1, 130)])
def test_generated_and_materialised_jacobians_agree(bd, n, m, B, T):
    """n = 16, 32 (64: forward only): by default the cell writes coefficient rows
    and the scans build J_t / J_{t+1}^T from them (the forward evaluation in the Newton-update form with
    reduced-precision chain products); with DEER_FLAG_MATERIALIZE the cell writes J itself and the scan is 3 x TF32.
    Two implementations of the same path: they agree to rounding, and both match the oracle."""
    p_np = synth.gru_params(n, m, 11, tag="f/gru")
    x_np = synth.x_gaussian(B, T, m, 11, tag="f/x")
    y0_np = synth.normal(11, "f/y0", (B, n)) * 0.3
    p = bd.GruParamsDev.from_numpy(p_np)
    x, y0 = dev(x_np), dev(y0_np)
    a = bd.deer_gru_eval(p, x, y0)
    b = bd.deer_gru_eval(p, x, y0, flags=bd.DEER_FLAG_MATERIALIZE)
    seq = oracle.gru_seq(p_np, x_np, y0_np, np.float32)
    assert a.status == 0 and b.status == 0 and abs(a.iters - b.iters) <= 1
    assert np.max(np.abs(a.y.cpu().numpy() - seq)) <= TOL_Y and np.max(np.abs(b.y.cpu().numpy() - seq)) <= TOL_Y
    assert float((a.y - b.y).abs().max()) <= 2e-6
    gy = dev(synth.normal(11, "f/gy", (B, T, n)))
    ga = bd.deer_gru_vjp(p, x, y0, a.y, gy)
    gb = bd.deer_gru_vjp(p, x, y0, a.y, gy, flags=bd.DEER_FLAG_MATERIALIZE)
    for k in ga:
        ref = gb[k].cpu().numpy()
        assert np.max(np.abs(ga[k].cpu().numpy() - ref)) <= 1e-4 * max(1e-30, float(np.max(np.abs(ref)))), k


def test_batch_with_sequences_converging_at_different_bodies(bd):
    """One global err: a sequence that is easy (zero input, tiny weights effect)
    next to a hard one still ends at the sequential values for both."""
    w = synth.config(2, B=2, T=2000)
    x = w.x.copy(); x[0] = 0.0
    w2 = synth.Workload("mix", 2, 2000, 8, 4, w.params, x, w.y0)
    r = run_eval(bd, w2)
    seq = oracle.gru_seq(w.params, x, w.y0, np.float32)
    assert np.max(np.abs(r.y.cpu().numpy() - seq)) <= TOL_Y


# ----------------------------------------------------------------------------- gradients
def grad_case(bd, n, m, B, T, dense, seed=5, flags=0, want_dx=True):
    p = synth.gru_params(n, m, seed, tag="v/gru")
    x = synth.x_gaussian(B, T, m, seed, tag="v/x")
    y0 = synth.normal(seed, "v/y0", (B, n)) * 0.3
    y32 = oracle.gru_seq(p, x, y0, np.float32)
    gy = synth.normal(seed, "v/gy", (B, T, n))
    if not dense:                      # L = sum_b y[b, T-1] . w[b]
        last = gy[:, -1].copy(); gy = np.zeros_like(gy); gy[:, -1] = last
    want = oracle.gru_bptt(p, x, y0, y32.astype(np.float64), gy, np.float64)
    pd = bd.GruParamsDev.from_numpy(p)
    got = bd.deer_gru_vjp(pd, dev(x), dev(y0), dev(y32), dev(gy), want_dx=want_dx, flags=flags)
    for k in ("dW_i", "dW_h", "db_i", "db_h", "dx", "dy0"):
        if k == "dx" and not want_dx:
            continue
        assert rel_inf(got[k].cpu().numpy().astype(np.float64), want[k]) <= TOL_GRAD, k
    return got


@pytest.mark.parametrize("n,m,B,T", [(1, 1, 2, 40), (2, 2, 3, 300), (4, 2, 2, 1000), (8, 4, 3, 1500),
                                     (16, 8, 2, 600), (32, 32, 2, 500), (64, 6, 2, 200), (3, 5, 2, 77),
                                     (16, 40, 1, 131), (64, 64, 1, 260)])
@pytest.mark.parametrize("dense", [True, False])
def test_vjp_matches_bptt(bd, n, m, B, T, dense):
    grad_case(bd, n, m, B, T, dense)


@pytest.mark.parametrize("n,m,B,T", [(8, 8, 2, 900), (4, 8, 3, 333), (2, 1, 2, 50), (1, 4, 3, 211), (8, 4, 16, 5000),
                                     (8, 1, 5, 77), (4, 4, 1, 1)])
def test_vjp_small_fused_path(bd, n, m, B, T):
    """The one-pass gradient kernel for n, m in {1,2,4,8}: more shapes (positions beyond one pass of the
    grid, ragged warps, T = 1), without dx, and against the separate kernels it replaces."""
    a = grad_case(bd, n, m, B, T, True)
    grad_case(bd, n, m, B, T, False, want_dx=False)
    b = grad_case(bd, n, m, B, T, True, flags=bd.DEER_FLAG_GENERIC)
    for k in ("dW_i", "dW_h", "db_i", "db_h", "dx", "dy0"):
        ref = b[k].cpu().numpy()
        assert np.max(np.abs(a[k].cpu().numpy() - ref)) <= 1e-4 * max(1.0, float(np.max(np.abs(ref)))), k


def test_vjp_is_bit_reproducible(bd):
    a = grad_case(bd, 8, 4, 4, 2000, True)
    b = grad_case(bd, 8, 4, 4, 2000, True)
    for k in a:
        assert torch.equal(a[k], b[k]), k


def test_config3_gradient_reduced_T(bd):
    """Config 3's loss L = sum(y_T . w): forward by DEER on the GPU, gradient by
    the reverse scan, against BPTT (T reduced so that the fp64 oracle is quick)."""
    w = synth.config(3, B=4, T=20000)
    r = run_eval(bd, w)
    assert r.status == 0
    wv = synth.normal(0, "c3/w", (4, 32))
    gy = np.zeros((4, 20000, 32), np.float32); gy[:, -1] = wv
    y32 = oracle.gru_seq(w.params, w.x, w.y0, np.float32)
    want = oracle.gru_bptt(w.params, w.x, w.y0, y32.astype(np.float64), gy, np.float64)
    got = bd.deer_gru_vjp(bd.GruParamsDev.from_numpy(w.params), dev(w.x), dev(w.y0), r.y, dev(gy))
    for k in ("dW_i", "dW_h", "db_i", "db_h", "dx", "dy0"):
        assert rel_inf(got[k].cpu().numpy().astype(np.float64), want[k]) <= TOL_GRAD, k


def test_config3_gradient_full_size(bd):
    """Config 3 at its full size (B=16, T=1e5, n=m=32), in the launch configuration the benchmark
    uses: both losses of the benchmark definition (terminal L = sum(y_T . w), and a dense gy)."""
    w = synth.config(3)
    r = run_eval(bd, w)
    assert r.status == 0
    y32 = oracle.gru_seq(w.params, w.x, w.y0, np.float32)
    p = bd.GruParamsDev.from_numpy(w.params)
    wv = synth.normal(0, "c3/w", (16, 32))
    gy_last = np.zeros((16, 100000, 32), np.float32); gy_last[:, -1] = wv
    gy_dense = synth.normal(0, "c3/gy", (16, 100000, 32)).astype(np.float32)
    for gy in (gy_last, gy_dense):
        want = oracle.gru_bptt(w.params, w.x, w.y0, y32.astype(np.float64), gy, np.float64)
        got = bd.deer_gru_vjp(p, dev(w.x), dev(w.y0), r.y, dev(gy))
        for k in ("dW_i", "dW_h", "db_i", "db_h", "dx", "dy0"):
            assert rel_inf(got[k].cpu().numpy().astype(np.float64), want[k]) <= TOL_GRAD, k


# ----------------------------------------------------------------------------- classifier
@pytest.mark.parametrize("B,T,n,m", [(3, 200, 8, 3), (4, 1500, 64, 6), (32, 17984, 64, 6), (2, 300, 16, 5), (2, 150, 32, 4)])
def test_classifier_step_matches_oracle(bd, B, T, n, m):
    w = synth.config4(seed=2, B=B, T=T, n=n, m=m)
    want = oracle.classifier(w.layers, w.W_o, w.b_o, w.x, w.labels, np.float64)
    l1 = bd.GruParamsDev.from_numpy(w.layers[0]); l2 = bd.GruParamsDev.from_numpy(w.layers[1])
    got = bd.deer_gru_classifier_step(l1, l2, dev(w.W_o), dev(w.b_o), dev(w.x), dev(w.labels))
    assert got["status"] == 0
    assert abs(got["loss"] - want["loss"]) <= 1e-4 * max(1.0, abs(want["loss"]))
    for tag, g in (("1", got["g1"]), ("2", got["g2"])):
        for k in ("dW_i", "dW_h", "db_i", "db_h"):
            assert rel_inf(g[k].cpu().numpy().astype(np.float64), want[k + tag]) <= TOL_GRAD, k + tag
    assert rel_inf(got["dW_o"].cpu().numpy().astype(np.float64), want["dW_o"]) <= TOL_GRAD
    assert rel_inf(got["db_o"].cpu().numpy().astype(np.float64), want["db_o"]) <= TOL_GRAD
