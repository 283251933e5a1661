"""The device-side input generator draws the same streams as the host generator (checked here with
CPU tensors: the integer arithmetic is the same on either device)."""
import numpy as np
import torch

from paper_2309_12252_b200 import synth, synth_device


def test_uniform_is_bit_identical_to_the_host_generator():
    for seed, name, shape, lo, hi in [(0, "a/J", (3, 1001, 4, 4), -0.225, 0.225), (7, "b", (5, 13), 0.001, 0.1),
                                      (123456789, "c/long name", (70001,), -1.0, 1.0)]:
        want = synth.uniform(seed, name, shape, lo, hi)
        got = synth_device.uniform(seed, name, shape, lo, hi, device="cpu").numpy()
        assert got.dtype == np.float32 and np.array_equal(got, want)
    J = synth_device.contractive_J(2, 50, 8, seed=3, tag="t/J", scale=1.0, device="cpu").numpy()
    assert np.array_equal(J, synth.contractive_J(2, 50, 8, seed=3, tag="t/J", scale=1.0))


def test_normal_matches_the_host_generator_to_the_last_place():
    want = synth.normal(5, "n/x", (4, 999, 3))
    got = synth_device.normal(5, "n/x", (4, 999, 3), device="cpu").numpy()
    ulp = np.spacing(np.abs(want).astype(np.float32))
    assert np.all(np.abs(got - want) <= ulp)
    assert np.mean(got == want) > 0.999


def test_chunked_generation_is_seamless():
    a = synth_device.uniform(1, "chunk", ((1 << 24) + 5,), 0.0, 1.0, device="cpu")
    tail = synth.uniform01(1, "chunk", 10, offset=(1 << 24) - 5).astype(np.float32)
    assert np.array_equal(a[-10:].numpy(), tail)
