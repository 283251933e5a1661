"""Host-side checks that need no GPU: the C-ABI library loads, exports every
symbol the header declares, sizes workspaces sanely and refuses bad arguments
before touching the device."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    from paper_2309_12252_b200 import build
    path = build.build()
    return ctypes.CDLL(path)


def declared_functions():
    src = open(os.path.join(ROOT, "include", "deer.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(deer_[a-z0-9_]+)\s*\(", src)))


def test_header_symbols_are_exported(L):
    names = declared_functions()
    assert {"deer_gru_eval", "deer_linrec_scan", "deer_gru_vjp", "deer_workspace_bytes"} <= set(names)
    for name in names:
        assert hasattr(L, name), name
    from paper_2309_12252_b200 import binding
    assert set(binding.EXPORTS) <= set(names)


def test_workspace_sizes(L):
    L.deer_workspace_bytes.restype = ctypes.c_size_t
    f = lambda *a: int(L.deer_workspace_bytes(*a))
    ev = f(0, 16, 10000, 8, 4, 0)
    sc = f(1, 16, 10000, 8, 1, 0)
    vj = f(2, 16, 10000, 8, 4, 0)
    assert 0 < sc < ev and 0 < vj
    assert ev % 256 == 0 and sc % 256 == 0
    assert ev < 16 * 10000 * 8 * (8 + 3 + 2 + 2) * 4 * 2      # no gross over-allocation
    assert f(0, 0, 10, 8, 4, 0) == 0 and f(0, 1, 10, 65, 4, 0) == 0 and f(9, 1, 10, 8, 4, 0) == 0
    assert f(0, 16, 10000, 8, 4, 0) == ev                       # pure function of the sizes


def test_status_strings_and_argument_validation(L):
    L.deer_status_string.restype = ctypes.c_char_p
    seen = {L.deer_status_string(s) for s in (0, 1, 2, -1, -2, -3, -4, -5)}
    assert len(seen) == 8 and all(seen)
    assert L.deer_linrec_scan(None, None, None, 1, 1, 1, 0, None, None, 0, 0, None) == -1
    assert L.deer_gru_eval(None, None, None, 1, 1, ctypes.c_float(1e-4), 100, None, None, None, None,
                           None, 0, 0, None) == -1
    assert L.deer_gru_vjp(None, None, None, None, None, 1, 1, None, None, None, None, 0, 0, None) == -1
    L.deer_launch_count.restype = ctypes.c_longlong
    assert L.deer_launch_count() == 0


def test_scan_geometry_bounds_the_resolver_ctas(L):
    """The single-pass scans give the first role tickets to resolver CTAs, which only spin: a batch
    that would need more of them than a quarter of the SMs must take the three-kernel path instead
    (host logic only; with no device the SM count falls back to 148)."""
    geo = (ctypes.c_int * 6)()
    for n in (1, 2, 4, 8, 16, 32, 64):
        last_single = 0
        for B in (1, 16, 100, 500, 1000, 1184, 1185, 2368, 2369, 5000, 20000, 100000):
            assert L.deer_scan_geometry(B, 3, n, 0, geo) == 0
            single, tile, chain, tiles, res, sms = list(geo)
            assert sms > 0 and tile > 0 and tiles == (3 + tile - 1) // tile
            if single:
                assert 1 <= res and 4 * res <= sms, (n, B, res)
                last_single = B
            else:
                assert res == 0
        assert last_single >= 500                       # ordinary batches stay on the single-pass kernels
        assert L.deer_scan_geometry(100000, 3, n, 0, geo) == 0 and geo[0] == 0
    assert L.deer_scan_geometry(16, 1000, 5, 0, geo) == 0 and geo[0] == 0      # other n: three-kernel path
    assert L.deer_scan_geometry(16, 1000, 8, 2, geo) == 0 and geo[0] == 0      # DEER_FLAG_GENERIC
    assert L.deer_scan_geometry(0, 1000, 8, 0, geo) == -1 and L.deer_scan_geometry(1, 1, 65, 0, geo) == -2
    # chain lengths the n = 8 kernel takes at benchmark sizes (148 SMs)
    if geo[5] == 148:
        for T, want in ((10000, 40), (40000, 64), (80000, 128), (120000, 256), (1000000, 256)):
            assert L.deer_scan_geometry(16, T, 8, 0, geo) == 0 and geo[2] == want, (T, list(geo))


def test_host_call_chunking_rule(L):
    """deer_gru_eval_host splits a batch into chunks of whole sequences of about 2^19 positions, at most eight, the
    first and the last about half as long as the others from three chunks on, and leaves small batches and single
    sequences whole (host logic only)."""
    import ctypes
    f = L.deer_gru_eval_host_chunk
    fs = L.deer_gru_eval_host_chunks
    fs.restype = ctypes.c_int
    fs.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.POINTER(ctypes.c_int)]

    def chunks(B, T):
        first = (ctypes.c_int * 9)()
        nc = fs(B, T, first)
        return [first[k] for k in range(nc + 1)] if nc else []

    assert f(0, 10) == 0 and f(3, 0) == 0 and fs(0, 10, None) == 0 and fs(3, 0, None) == 0
    assert f(3, 1200) == 3 and f(1, 10_000_000) == 1 and f(16, 10_000) == 16
    assert chunks(3, 1200) == [0, 3] and chunks(16, 10_000) == [0, 16] and fs(16, 100_000, None) == 3
    assert chunks(16, 100_000) == [0, 4, 12, 16] and f(16, 100_000) == 8      # three chunks: 4, 8 and 4 sequences
    assert chunks(2, 600_000) == [0, 1, 2] and chunks(3, 600_000) == [0, 1, 2, 3]
    for B, T in ((5, 200_000), (3, 300_000), (32, 17_984), (16, 1_000_000), (7, 123_457), (1000, 1000), (9, 2_000_000)):
        first = chunks(B, T)
        nc = len(first) - 1
        sizes = [b - a for a, b in zip(first[:-1], first[1:])]
        assert 1 <= nc <= 8 and first[0] == 0 and first[-1] == B and min(sizes) >= 1
        assert f(B, T) == max(sizes)
        if nc >= 3:                                                  # the edges are the short ones
            assert max(sizes[0], sizes[-1]) <= min(sizes[1:-1]) and min(sizes[0], sizes[-1]) * 2 + 1 >= max(sizes[1:-1]) - 1
        if nc == 2:
            assert abs(sizes[0] - sizes[1]) <= 1
