"""Pins for the oracle's quantizer and Philox generator (no GPU)."""
import os

import numpy as np
import pytest

import oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def test_philox_known_answers():
    # Published known-answer vectors of Philox4x32-10 (Random123 kat file).
    rows = [l.split() for l in open(os.path.join(GOLD, "philox4x32_10_kat.txt"))
            if l.strip() and not l.startswith("#")]
    assert len(rows) == 2
    for r in rows:
        v = [int(t, 16) for t in r if t != "->"]
        out = oracle.philox4x32_10(v[0:4], v[4:6])
        assert [int(o) for o in out] == v[6:10]


def test_philox_bijection_and_uniformity():
    # A counter-mode generator is a bijection on the counter for a fixed key:
    # distinct counters give distinct blocks; words look uniform.
    outs = np.stack([oracle.philox4x32_10([i, 0, 0, 0], [7, 9]) for i in range(4096)])
    assert len({tuple(o) for o in outs}) == 4096
    u = (outs >> 8).astype(np.float64) * 2.0 ** -24
    assert abs(u.mean() - 0.5) < 4 * (1 / np.sqrt(12 * u.size))
    bits = np.unpackbits(outs.view(np.uint8))
    assert abs(bits.mean() - 0.5) < 4 * 0.5 / np.sqrt(bits.size)


def test_sym_hand_examples():
    # scale exactly 1 (amax = 127): ties go to the even integer.
    x = np.array([[0.5, 1.5, 2.5, -0.5, -1.5, 127.0]], np.float32)
    q, s = oracle.quantize_sym_s8(x)
    assert s[0] == 1.0
    assert q.tolist() == [[0, 2, 2, 0, -2, 127]]
    # amax = 1.27 -> grid step 0.01
    x = np.array([[-1.0, 0.5, 0.25, 1.27]], np.float32)
    q, s = oracle.quantize_sym_s8(x)
    assert q.tolist() == [[-100, 50, 25, 127]]
    assert s[0] == np.float32(1.27) / np.float32(127.0)


def test_sym_invariants():
    rng = np.random.default_rng(1)
    x = (rng.standard_normal((5, 4099)) * rng.uniform(1e-3, 1e3, (5, 1))).astype(np.float32)
    q, s = oracle.quantize_sym_s8(x)
    xd = x.astype(np.float64)
    # error bound: half a grid step (plus fp32 rounding of x*inv)
    err = np.abs(xd - s[:, None].astype(np.float64) * q)
    assert np.all(err <= 0.5 * s[:, None] * (1 + 2.0 ** -20))
    # the extreme element maps to +-127, per node, independently
    amax_pos = np.abs(x).argmax(axis=1)
    for n in range(5):
        assert abs(int(q[n, amax_pos[n]])) == 127
        assert s[n] == np.abs(x[n]).max() / np.float32(127)
    assert q.min() >= -127
    # idempotent on the grid
    xg = oracle.dequantize(q, s)
    q2, s2 = oracle.quantize_sym_s8(xg)
    assert np.array_equal(q2, q)
    # dequantize is scale * q in fp32
    assert np.array_equal(xg, q.astype(np.float32) * s[:, None])


def test_sym_zero_tensor_and_node_independence():
    x = np.zeros((2, 16), np.float32)
    x[1, 3] = -2.0
    q, s = oracle.quantize_sym_s8(x)
    assert s[0] == 1.0 and not q[0].any()
    assert q[1, 3] == -127 and s[1] == np.float32(2.0) / np.float32(127)


def test_sym_matches_numpy_rint():
    # special case that reduces to a library routine: np.rint is round-half-even
    rng = np.random.default_rng(2)
    x = rng.standard_normal((3, 1000)).astype(np.float32)
    q, s = oracle.quantize_sym_s8(x)
    amax = np.abs(x).max(axis=1, keepdims=True)
    inv = np.float32(127.0) / amax
    ref = np.clip(np.rint(x * inv), -127, 127).astype(np.int8)
    assert np.array_equal(q, ref)


def test_affine_properties():
    rng = np.random.default_rng(3)
    x = rng.uniform(-1.0, 3.0, (2, 1001)).astype(np.float32)
    x[0, 0] = 0.0
    q, s, zp = oracle.quantize_affine_u8(x)
    # real zero maps exactly onto the zero point
    assert q[0, 0] == zp[0]
    # range endpoints map to the ends of the code range
    for n in range(2):
        assert q[n, x[n].argmin()] == 0 and q[n, x[n].argmax()] == 255
    xd = oracle.dequantize(q, s, zp)
    assert np.all(np.abs(xd - x) <= s[:, None] * (0.5 + 1e-3) + 1e-7)
    # one-sided tensor: the range is extended to contain zero
    x = rng.uniform(2.0, 3.0, (1, 64)).astype(np.float32)
    q, s, zp = oracle.quantize_affine_u8(x)
    assert zp[0] == 0 and s[0] == x.max() / np.float32(255)


def test_stochastic_rounding_properties():
    rng = np.random.default_rng(4)
    x = rng.standard_normal((2, 4096)).astype(np.float32)
    q, s = oracle.quantize_sym_s8(x, rounding=1, seed=123, ctr_offset=5)
    qn, _ = oracle.quantize_sym_s8(x, rounding=0)
    # strictly less than one grid step away, and a neighbour of the real value
    err = np.abs(x.astype(np.float64) - s[:, None].astype(np.float64) * q)
    assert np.all(err < s[:, None] * (1 + 2.0 ** -20))
    assert np.all(np.abs(q.astype(int) - qn.astype(int)) <= 1)
    # deterministic in (seed, offset); different offsets give different draws
    q2, _ = oracle.quantize_sym_s8(x, rounding=1, seed=123, ctr_offset=5)
    q3, _ = oracle.quantize_sym_s8(x, rounding=1, seed=123, ctr_offset=6)
    assert np.array_equal(q, q2) and not np.array_equal(q, q3)
    # grid values never move
    xg = oracle.dequantize(qn, s)
    qg, _ = oracle.quantize_sym_s8(xg, rounding=1, seed=9)
    assert np.array_equal(qg, qn)


def test_stochastic_rounding_unbiased():
    # E[scale*q] = x: a constant tensor with one pinning element; compare the
    # mean code with x*inv within 4 sigma.
    n = 1 << 18
    x = np.full((1, n), 0.3, np.float32)
    x[0, 0] = 1.27  # fixes scale = 0.01, so 0.3 -> 30.0000x
    x[0, 1:] = np.float32(0.3037)
    q, s = oracle.quantize_sym_s8(x, rounding=1, seed=42)
    t = float(np.float32(0.3037) * (np.float32(127.0) / np.float32(1.27)))
    frac = t - np.floor(t)
    mean = q[0, 1:].astype(np.float64).mean()
    sigma = np.sqrt(frac * (1 - frac) / (n - 1))
    assert abs(mean - t) < 4 * sigma
    assert set(np.unique(q[0, 1:]).tolist()) == {int(np.floor(t)), int(np.floor(t)) + 1}


def test_stochastic_uses_the_documented_counter_layout():
    # element i draws word i%4 of block (i//4, 0, node, ctr_offset), key = seed halves
    x = np.full((2, 8), 0.5, np.float32)
    x[:, 0] = 127.0  # inv = 1 -> t = 0.5, f = 0.5: rounds up iff u < 0.5
    seed = (77 << 32) | 5
    q, _ = oracle.quantize_sym_s8(x, rounding=1, seed=seed, ctr_offset=11)
    for node in range(2):
        for i in range(1, 8):
            r = oracle.philox4x32_10([i // 4, 0, node, 11], [5, 77])
            u = float(int(r[i % 4]) >> 8) * 2.0 ** -24
            assert q[node, i] == (1 if u < 0.5 else 0)
