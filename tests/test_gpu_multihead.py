"""Multi-head GRU unit (Sec. 4.4, App. B.4) on the GPU against the oracle's sequential evaluation and BPTT:
independent heads on the same input, strides as interleaved sequences.  Tolerances as for the single GRU
(trajectory 1e-4 against the sequential fp32 loop, gradients 1e-3 relative per tensor)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2309_12252_b200 import synth

pytestmark = pytest.mark.gpu

TOL_Y = 1e-4
TOL_GRAD = 1e-3


@pytest.fixture(scope="module")
def bd():
    from paper_2309_12252_b200 import binding
    binding.lib()
    return binding


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def rel_inf(a, b):
    return float(np.max(np.abs(a - b)) / max(np.max(np.abs(b)), 1e-30))


def case(H, n, m, B, T, strides, seed):
    heads = synth.multihead_params(H, n, m, seed, tag="g/mh")
    x = synth.x_gaussian(B, T, m, seed, tag="g/mhx")
    y0 = synth.normal(seed, "g/mhy0", (B, H, n)) * 0.3
    return heads, np.asarray(strides, np.int32), x, y0


# (H, n, m, B, T, strides): ragged phases (T not a multiple of the stride), a stride beyond T, other n,
# and the shape of the paper's sequential-CIFAR model (32 heads of 8 channels on 256 inputs, T = 1024)
CASES = [
    (6, 8, 16, 3, 203, [1, 2, 4, 8, 1, 2]),
    (3, 4, 3, 2, 50, [3, 1, 64]),
    (2, 16, 16, 2, 300, [2, 5]),
    (32, 8, 256, 2, 1024, list(synth.multihead_strides(32))),
]


@pytest.mark.parametrize("H,n,m,B,T,strides", CASES)
def test_multihead_eval_matches_sequential(bd, H, n, m, B, T, strides):
    heads, st, x, y0 = case(H, n, m, B, T, strides, seed=H + T)
    hd = [bd.GruParamsDev.from_numpy(h) for h in heads]
    y, iters, status = bd.deer_gru_multihead_eval(hd, st, dev(x), dev(y0))
    assert status == 0 and all(2 <= k <= 100 for k in iters)
    want32 = oracle.multihead_seq(heads, st, x, y0, np.float32)
    assert float(np.max(np.abs(y.cpu().numpy() - want32))) <= TOL_Y
    # a head's evaluation is the single-GRU evaluation of its interleaved sequences: same body count
    h = 0
    s = int(st[h])
    xs = np.concatenate([x[:, p::s][:, :T // s] for p in range(s)], axis=0) if T % s == 0 else None
    if xs is not None:
        y0s = np.concatenate([y0[:, h]] * s, axis=0)
        o = oracle.deer(heads[h], xs, y0s, tol=1e-4, dtype=np.float32)
        assert abs(iters[h] - o["iters"]) <= 1
    # bit-reproducible
    y2, iters2, _ = bd.deer_gru_multihead_eval(hd, st, dev(x), dev(y0))
    assert iters2 == iters and torch.equal(y, y2)


@pytest.mark.parametrize("H,n,m,B,T,strides", CASES)
def test_multihead_vjp_matches_bptt(bd, H, n, m, B, T, strides):
    heads, st, x, y0 = case(H, n, m, B, T, strides, seed=H + T + 1)
    y32 = oracle.multihead_seq(heads, st, x, y0, np.float32)
    gy = synth.normal(H + T, "g/mhgy", y32.shape)
    want = oracle.multihead_bptt(heads, st, x, y0, y32.astype(np.float64), gy, np.float64)
    hd = [bd.GruParamsDev.from_numpy(h) for h in heads]
    g = bd.deer_gru_multihead_vjp(hd, st, dev(x), dev(y0), dev(y32), dev(gy))
    for k in ("dW_i", "dW_h", "db_i", "db_h"):
        got = np.stack([t.cpu().numpy() for t in g[k]]).astype(np.float64)
        for h in range(H):
            assert rel_inf(got[h], want[k][h]) <= TOL_GRAD, (k, h)
    assert rel_inf(g["dx"].cpu().numpy().astype(np.float64), want["dx"]) <= TOL_GRAD
    assert rel_inf(g["dy0"].cpu().numpy().astype(np.float64), want["dy0"]) <= TOL_GRAD


def test_multihead_warm_start_and_argument_checks(bd):
    H, n, m, B, T = 4, 8, 8, 2, 400
    heads, st, x, y0 = case(H, n, m, B, T, [1, 2, 4, 8], seed=3)
    hd = [bd.GruParamsDev.from_numpy(h) for h in heads]
    y, iters, status = bd.deer_gru_multihead_eval(hd, st, dev(x), dev(y0))
    guess = y.clone()
    y2, iters2, status2 = bd.deer_gru_multihead_eval(hd, st, dev(x), dev(y0), y=guess, flags=bd.DEER_FLAG_WARM_START)
    assert status2 == 0 and all(k <= 2 for k in iters2)
    assert float((y2 - y).abs().max()) <= 1e-5
    with pytest.raises(bd.DeerError):
        bd.deer_gru_multihead_eval(hd, [1, 2, 0, 8], dev(x), dev(y0))
    small = torch.empty(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(bd.DeerError):
        bd.deer_gru_multihead_eval(hd, st, dev(x), dev(y0), ws=small)
