"""A second cell behind the same iteration (Sec. 3.4): the LSTM evaluated by DEER on the GPU against the oracle's
sequential LSTM (fp32: 1e-4, as for the GRU) and the oracle's Newton iteration (body count within one)."""
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


# state sizes 2k on the single-pass kernels (2, 4, 8, 16, 32, 64) and on the three-kernel path (6, 10)
@pytest.mark.parametrize("k,m,B,T", [(1, 1, 2, 50), (2, 3, 3, 500), (4, 2, 2, 2000), (8, 8, 4, 1500), (16, 5, 2, 700),
                                     (32, 16, 2, 300), (3, 2, 2, 333), (5, 7, 1, 129)])
def test_lstm_eval_matches_sequential(bd, k, m, B, T):
    p = synth.lstm_params(k, m, 41, tag="g/lstm")
    x = synth.x_gaussian(B, T, m, 41, tag="g/lx")
    s0 = synth.normal(41, "g/ls0", (B, 2 * k)) * 0.3
    r = bd.deer_lstm_eval(p, dev(x), dev(s0))
    seq32 = oracle.lstm_seq(p, x, s0, np.float32)
    assert r.status == 0 and r.err <= 1e-4
    assert float(np.max(np.abs(r.y.cpu().numpy() - seq32))) <= 1e-4
    o = oracle.deer(p, x, s0, tol=1e-4, dtype=np.float32, cell="lstm")
    assert abs(r.iters - o["iters"]) <= 1
    r2 = bd.deer_lstm_eval(p, dev(x), dev(s0))
    assert r2.iters == r.iters and torch.equal(r.y, r2.y)


def test_lstm_first_iterate_status_codes_and_warm_start(bd):
    k, m, B, T = 8, 4, 3, 800
    p = synth.lstm_params(k, m, 42, tag="g/lstm2")
    x = synth.x_gaussian(B, T, m, 42, tag="g/lx2")
    s0 = synth.normal(42, "g/ls02", (B, 2 * k)) * 0.3
    r = bd.deer_lstm_eval(p, dev(x), dev(s0), tol=-1.0, max_iter=1)
    o = oracle.deer(p, x, s0, tol=-1.0, max_iter=1, dtype=np.float64, cell="lstm")
    assert r.iters == 1 and float(np.max(np.abs(r.y.cpu().numpy() - o["y"]))) <= 2e-5 * max(1.0, float(np.max(np.abs(o["y"]))))
    r = bd.deer_lstm_eval(p, dev(x), dev(s0), max_iter=1)
    assert r.status == bd.DEER_NOT_CONVERGED
    full = bd.deer_lstm_eval(p, dev(x), dev(s0))
    warm = bd.deer_lstm_eval(p, dev(x), dev(s0), s=full.y.clone(), flags=bd.DEER_FLAG_WARM_START)
    assert warm.status == 0 and warm.iters <= 2
    assert bd.deer_workspace_bytes(bd.DEER_OP_LSTM, 1, 10, 33, 4) == 0
