"""The allocation-free scan entry point, for hosts that only hand the library
their input and output buffers (no workspace, no device allocation allowed at
the call site): it must give the same answer as deer_linrec_scan -- and as the
oracle's sequential solve -- twice in a row on the shared built-in scratch,
also when consecutive calls use different sizes (the scratch then holds words
of another layout), allocate nothing, and refuse sizes the scratch cannot hold.
Collected last on purpose, so that a failure here cannot hide other results."""
import numpy as np
import pytest
import torch

import oracle
from paper_2309_12252_b200 import synth

pytestmark = pytest.mark.gpu

TOL_SCAN = 1e-5      # same bound as the other scan tests: relative to max |y|


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


# (n, B, T, reverse, y0 given): every scan kernel family, the three-kernel path (n = 3) and a missing y0;
# the order alternates the layouts of the words kept in the scratch (64-bit words for n <= 4, flags +
# floats for n >= 8, chunk carries for the three-kernel path)
CASES = [(8, 4, 3000, False, True), (2, 3, 9001, False, True), (8, 4, 3000, True, True), (1, 5, 20000, True, True),
         (32, 2, 300, False, True), (4, 3, 7000, False, False), (3, 2, 2000, True, True), (4, 3, 7000, True, True),
         (16, 2, 700, False, False), (64, 1, 200, True, True), (1, 5, 20000, False, False)]


def test_noalloc_scan_matches_workspace_scan_and_oracle_twice_in_a_row():
    from paper_2309_12252_b200 import binding as bd
    bd.lib()
    data = []
    for i, (n, B, T, reverse, with_y0) in enumerate(CASES):
        assert bd.deer_workspace_bytes(bd.DEER_OP_SCAN, B, T, n) <= bd.NOALLOC_SCRATCH_BYTES
        J = synth.contractive_J(B, T, n, seed=40 + i, tag="na/J")
        b = synth.normal(40 + i, "na/b", (B, T, n))
        y0 = synth.normal(40 + i, "na/y0", (B, n)) if with_y0 else None
        want64 = oracle.linrec(J, b, y0, reverse=reverse, dtype=np.float64)
        data.append((dev(J), dev(b), None if y0 is None else dev(y0), reverse, want64))
    # first call on this device (looks up the scratch address), before the memory readings below
    J, b, y0, reverse, _ = data[0]
    bd.deer_linrec_scan_noalloc(J, b, y0, reverse=reverse)
    torch.cuda.synchronize()
    for rnd in range(2):
        for (J, b, y0, reverse, want64), case in zip(data, CASES):
            want = bd.deer_linrec_scan(J, b, y0, reverse=reverse)
            out = torch.empty_like(b)
            torch.cuda.synchronize()
            for call in range(2):                  # second call reuses whatever the first left in the scratch
                out.zero_()
                free0 = torch.cuda.mem_get_info()[0]
                bd.deer_linrec_scan_noalloc(J, b, y0, reverse=reverse, y=out)
                assert bd.deer_noalloc_status() == bd.DEER_OK
                assert torch.cuda.mem_get_info()[0] == free0, "the call must not allocate device memory"
                scale = max(1.0, float(np.max(np.abs(want64))))
                assert float((out - want).abs().max()) <= TOL_SCAN * scale, (case, rnd, call)
                assert float(np.max(np.abs(out.cpu().numpy() - want64))) <= TOL_SCAN * scale, (case, rnd, call)


def test_noalloc_scan_refuses_what_does_not_fit():
    from paper_2309_12252_b200 import binding as bd
    n, B, T = 8, 16, 400000
    assert bd.deer_workspace_bytes(bd.DEER_OP_SCAN, B, T, n) > bd.NOALLOC_SCRATCH_BYTES
    # no compute happens for a refused call, so tiny stand-in buffers are enough to pass the pointer checks
    J = torch.zeros(16, device="cuda"); b = torch.zeros(16, device="cuda"); y = torch.zeros(16, device="cuda")
    rc = bd.lib().deer_linrec_scan_noalloc(J.data_ptr(), b.data_ptr(), None, B, T, n, 0, y.data_ptr(), None)
    assert rc == bd.DEER_ERR_WORKSPACE
    assert b"scratch" in bd.lib().deer_last_error()
