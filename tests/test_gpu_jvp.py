"""Forward-mode derivative (Sec. 3.1.1) on the GPU against the oracle's tangent recurrence in fp64 and against
the gradient (the two derivatives are transposes of one another).  Tolerance: 1e-3 relative, as for gradients."""
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
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def rel_inf(a, b):
    return float(np.max(np.abs(a - b)) / max(np.max(np.abs(b)), 1e-30))


@pytest.mark.parametrize("n,m,B,T", [(1, 1, 2, 60), (2, 3, 3, 333), (4, 2, 2, 1000), (8, 4, 3, 1500), (16, 16, 2, 700),
                                     (32, 32, 2, 500), (64, 6, 2, 200), (5, 7, 2, 129), (32, 32, 4, 20000)])
@pytest.mark.parametrize("which", ["params", "x", "y0", "all"])
def test_jvp_matches_oracle(bd, n, m, B, T, which):
    p = synth.gru_params(n, m, 31, tag="j/gru")
    x = synth.x_gaussian(B, T, m, 31, tag="j/x")
    y0 = synth.normal(31, "j/y0", (B, n)) * 0.3
    dp = synth.GruParams(n, m, *(synth.normal(31, f"j/dp{i}", a.shape) for i, a in enumerate((p.W_i, p.W_h, p.b_i, p.b_h))))
    dx = synth.normal(31, "j/dx", x.shape)
    dy0 = synth.normal(31, "j/dy0", y0.shape)
    use_p, use_x, use_y0 = which in ("params", "all"), which in ("x", "all"), which in ("y0", "all")
    y32 = oracle.gru_seq(p, x, y0, np.float32)
    want = oracle.gru_jvp(p, dp if use_p else None, x, dx if use_x else None, y0, dy0 if use_y0 else None,
                          y32.astype(np.float64), np.float64)
    pd = bd.GruParamsDev.from_numpy(p)
    dpd = bd.GruParamsDev.from_numpy(dp) if use_p else None
    ws = bd.alloc_workspace(bd.DEER_OP_VJP, B, T, n, m)
    got = bd.deer_gru_jvp(pd, dpd, dev(x), dev(dx) if use_x else None, dev(y0), dev(dy0) if use_y0 else None, dev(y32), ws=ws)
    assert bd.deer_workspace_status(ws) == bd.DEER_OK
    assert rel_inf(got.cpu().numpy().astype(np.float64), want) <= 1e-3


def test_jvp_is_the_transpose_of_vjp_on_the_gpu(bd):
    n, m, B, T = 8, 4, 3, 2000
    p = synth.gru_params(n, m, 32, tag="j2/gru")
    x = synth.x_gaussian(B, T, m, 32, tag="j2/x")
    y0 = synth.normal(32, "j2/y0", (B, n)) * 0.3
    dp = synth.GruParams(n, m, *(synth.normal(32, f"j2/dp{i}", a.shape) for i, a in enumerate((p.W_i, p.W_h, p.b_i, p.b_h))))
    dx = synth.normal(32, "j2/dx", x.shape)
    dy0 = synth.normal(32, "j2/dy0", y0.shape)
    gy = synth.normal(32, "j2/gy", (B, T, n))
    pd, dpd = bd.GruParamsDev.from_numpy(p), bd.GruParamsDev.from_numpy(dp)
    y = bd.deer_gru_eval(pd, dev(x), dev(y0)).y
    dy = bd.deer_gru_jvp(pd, dpd, dev(x), dev(dx), dev(y0), dev(dy0), y)
    g = bd.deer_gru_vjp(pd, dev(x), dev(y0), y, dev(gy))
    lhs = float((dev(gy).double() * dy.double()).sum())
    rhs = sum(float((g["d" + k].double() * dev(getattr(dp, k)).double()).sum()) for k in ("W_i", "W_h", "b_i", "b_h"))
    rhs += float((g["dx"].double() * dev(dx).double()).sum()) + float((g["dy0"].double() * dev(dy0).double()).sum())
    assert abs(lhs - rhs) <= 1e-3 * max(1.0, abs(rhs))
