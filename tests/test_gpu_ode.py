"""The ODE instantiation of L_G^{-1} (Sec. 3.3) on the GPU against the oracle (fp64): batched matrix exponential of
the mid-point values, then the scan.  Tolerance: 1e-5 relative to max|y|, as for the stand-alone scan, for
well-conditioned problems; stiff intervals (|G D| up to ~30) at 1e-4."""
import numpy as np
import pytest
import torch

import oracle
from paper_2309_12252_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def bd():
    from paper_2309_12252_b200 import binding
    binding.lib()
    return binding


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a, np.float32)).cuda()


def problem(B, T, n, seed, stiff=1.0):
    G = synth.normal(seed, "ode/G", (B, T, n, n)) * (0.5 * stiff) + stiff * np.eye(n, dtype=np.float32)
    z = synth.normal(seed, "ode/z", (B, T, n))
    dt = synth.uniform(seed, "ode/dt", (T,), 0.01, 0.2, dtype=np.float64)
    t = np.cumsum(dt).astype(np.float32)
    y0 = synth.normal(seed, "ode/y0", (B, n))
    return G, z, t, y0


@pytest.mark.parametrize("B,T,n", [(1, 1, 2), (2, 2, 1), (3, 257, 2), (2, 1000, 4), (4, 5000, 8), (1, 40000, 8), (16, 3000, 3),
                                   (2, 777, 5), (2, 300, 7)])
def test_ode_linear_solve_matches_oracle(bd, B, T, n):
    G, z, t, y0 = problem(B, T, n, seed=B + T + n)
    want = oracle.ode_linear(G, z, t, y0, np.float64)
    ws = bd.alloc_workspace(bd.DEER_OP_ODE, B, T, n)
    got = bd.deer_ode_linear_solve(dev(G), dev(z), dev(t), dev(y0), ws=ws)
    assert bd.deer_workspace_status(ws) == bd.DEER_OK
    assert float(np.max(np.abs(got.cpu().numpy() - want))) <= 1e-5 * max(1.0, float(np.max(np.abs(want))))


def test_ode_stiff_intervals_singular_G_and_constant_coefficients(bd):
    scipy_linalg = pytest.importorskip("scipy.linalg")
    B, T, n = 2, 400, 4
    G, z, t, y0 = problem(B, T, n, seed=9, stiff=150.0)             # |G D| up to ~30: many squarings
    want = oracle.ode_linear(G, z, t, y0, np.float64)
    got = bd.deer_ode_linear_solve(dev(G), dev(z), dev(t), dev(y0)).cpu().numpy()
    assert np.max(np.abs(got - want)) <= 1e-4 * max(1.0, np.max(np.abs(want)))
    # G = 0: dy/dt = z, the mid-point rule is the trapezoid rule
    zt = np.sin(t)[None, :, None] * np.ones((1, T, n), np.float32)
    got = bd.deer_ode_linear_solve(dev(np.zeros((1, T, n, n))), dev(zt), dev(t), dev(y0[:1])).cpu().numpy()
    trap = np.concatenate([[0.0], np.cumsum(0.5 * (np.sin(t[1:].astype(np.float64)) + np.sin(t[:-1].astype(np.float64))) * np.diff(t.astype(np.float64)))])
    assert np.max(np.abs(got[0] - (y0[0][None, :] + trap[:, None]))) <= 2e-5
    # constant coefficients: the exact solution of the linear ODE at every time point
    G0 = (synth.normal(5, "ode/G0", (n, n)) * 0.5 + 1.5 * np.eye(n)).astype(np.float64)
    z0 = synth.normal(5, "ode/z0", (n,)).astype(np.float64)
    got = bd.deer_ode_linear_solve(dev(np.broadcast_to(G0, (1, T, n, n))), dev(np.broadcast_to(z0, (1, T, n))), dev(t),
                                   dev(y0[:1])).cpu().numpy()
    yinf = np.linalg.solve(G0, z0)
    for k in (0, 1, 57, T - 1):
        exact = scipy_linalg.expm(-G0 * float(t[k] - t[0])) @ (y0[0].astype(np.float64) - yinf) + yinf
        assert np.max(np.abs(got[0, k] - exact)) <= 2e-5 * max(1.0, np.max(np.abs(exact)))


def test_ode_refuses_large_n(bd):
    G = torch.zeros((1, 4, 9, 9), device="cuda"); z = torch.zeros((1, 4, 9), device="cuda")
    assert bd.deer_workspace_bytes(bd.DEER_OP_ODE, 1, 4, 9) == 0
    small = torch.empty(4096, dtype=torch.uint8, device="cuda")
    with pytest.raises(bd.DeerError):
        bd.deer_ode_linear_solve(G, z, torch.arange(4, device="cuda", dtype=torch.float32), torch.zeros((1, 9), device="cuda"), ws=small)
