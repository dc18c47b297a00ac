"""Pins for the oracle's number formats and its one summation routine.

Each check compares the oracle with something that is not the oracle: numpy's
and torch's own conversion routines, exact integer arithmetic, binary64 sums.
"""
import numpy as np
import torch

from paper_2609_38166_b200 import synth


def _edge_f32():
    vals = [0.0, -0.0, 1.0, -1.0, 65504.0, 65519.99, 65520.0, 70000.0, -70000.0, 1e-8, 2.0 ** -24, 2.0 ** -25,
            2.0 ** -25 * 1.0000001, 2.0 ** -14, 2.0 ** -14 * 0.9999, 6.1e-5, 5.96e-8, 3.0e-8, 1.0009765625,
            1.00048828125, 1.00146484375, 0.333333, 2047.5, 2048.5, 2049.0, 1023.75]
    return np.array(vals, np.float32)


def test_f16_conversion_matches_numpy(oracle):
    rng = np.random.default_rng(0)
    # random bit patterns cover every exponent, including fp16's subnormal and overflow ranges
    bits = rng.integers(0, 2 ** 32, size=50000, dtype=np.uint64).astype(np.uint32)
    x = bits.view(np.float32)
    x = x[np.isfinite(x)]
    x = np.concatenate([x, _edge_f32(), rng.standard_normal(20000).astype(np.float32),
                        (rng.standard_normal(20000) * 1e-5).astype(np.float32)])
    with np.errstate(over="ignore"):
        want = x.astype(np.float16).view(np.uint16)
    got = np.array([oracle.f32_to_f16(float(v)) for v in x], np.uint16)
    assert np.array_equal(got, want)


def test_f16_widening_matches_numpy(oracle):
    h = np.arange(0, 65536, dtype=np.uint32).astype(np.uint16)
    want = h.view(np.float16).astype(np.float32)
    got = np.array([oracle.f16_to_f32(int(v)) for v in h], np.float32)
    fin = np.isfinite(want)
    assert np.array_equal(got[fin].view(np.uint32), want[fin].view(np.uint32))
    assert np.array_equal(np.isnan(got), np.isnan(want))
    assert np.array_equal(np.isinf(got), np.isinf(want))


def test_bf16_rounding_matches_torch(oracle):
    rng = np.random.default_rng(1)
    x = np.concatenate([rng.standard_normal(50000).astype(np.float32),
                        np.array([1.00390625, 1.01171875, 1.0, 3.0e38, 1e-40, -2.5], np.float32)])
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = np.array([oracle.f32_to_bf16(float(v)) for v in x], np.uint16)
    assert np.array_equal(got, want)
    # the input generator's rounding is the same function
    assert np.array_equal(synth.f32_to_bf16_bits(x), want)
    assert np.array_equal(synth.bf16_bits_to_f32(want), torch.from_numpy(x).to(torch.bfloat16).float().numpy())


def test_csum_is_exact_on_integers(oracle):
    # small integers: every partial sum is exactly representable, so any correct order gives the exact sum
    rng = np.random.default_rng(2)
    for n in (0, 1, 5, 8, 9, 16, 64, 100, 128, 131, 1000):
        a = rng.integers(-50, 50, n).astype(np.float32)
        b = rng.integers(-50, 50, n).astype(np.float32)
        assert oracle.csum_dot(a, b) == float(np.dot(a.astype(np.int64), b.astype(np.int64)))
        assert oracle.csum_abs(a) == float(np.abs(a.astype(np.int64)).sum())


def test_csum_close_to_binary64_sum(oracle, oracle_wide):
    rng = np.random.default_rng(3)
    for n in (7, 128, 129, 333):
        for _ in range(20):
            a = rng.standard_normal(n).astype(np.float32)
            b = rng.standard_normal(n).astype(np.float32)
            exact = float(np.dot(a.astype(np.float64), b.astype(np.float64)))
            bound = (np.log2(max(n, 2)) + 9) * 2.0 ** -24 * float(np.abs(a.astype(np.float64) * b).sum())
            assert abs(oracle.csum_dot(a, b) - exact) <= bound
            assert abs(oracle_wide.csum_dot(a, b) - exact) <= 2.0 ** -24 * abs(exact) + 1e-30
            exact_abs = float(np.abs(a.astype(np.float64)).sum())
            assert abs(oracle.csum_abs(a) - exact_abs) <= (np.log2(n) + 9) * 2.0 ** -24 * exact_abs


def test_csum_order_is_blocks_of_eight_then_neighbour_tree(oracle):
    """Terms chosen so that only the stated order reproduces the result: inside a block of eight the even
    and the odd terms are summed separately and then added; blocks are combined neighbours first."""
    a = np.ones(32, np.float32)
    b = np.zeros(32, np.float32)
    # block 0: even terms 2^30, 1, 1, 1 (the ones vanish next to 2^30, spacing 128); odd terms -2^30, 1, 1, 1
    b[0] = 2.0 ** 30; b[1] = -(2.0 ** 30); b[2:8] = 1.0
    b[8:16] = 1.0                            # block 1: 4 + 4
    b[16:32] = 1.0                           # blocks 2, 3: 8 each
    # blocks: [2^30 + (-2^30) = 0, 8, 8, 8] -> tree: (0 + 8) + (8 + 8) = 24
    assert oracle.csum_dot(a, b) == 24.0
    # even terms 2^24, 1, 1, 1 stay 2^24 (ties to even); odd terms 1+1+1+1 = 4 survive
    assert oracle.csum_abs(np.array([2.0 ** 24, 1, 1, 1, 1, 1, 1, 1], np.float32)) == float(2.0 ** 24 + 4)
    # a left-to-right sum would give 2^30 - 2^30 + 6 + 24 = 30, which is also the exact value
    assert float(np.sum(b.astype(np.float64))) == 30.0
