"""Pins for the oracle's gossip/top-k step and glue ops (no GPU)."""
import os

import numpy as np
import pytest

import oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def ring(n):
    W = np.zeros((n, n), np.float32)
    for i in range(n):
        for j in (i - 1, i, i + 1):
            W[i, j % n] += np.float32(1.0 / 3.0)
    return W


def test_ring4_hand_case():
    rows = {l.split()[0]: np.array(l.split()[1:], np.float32)
            for l in open(os.path.join(GOLD, "gossip_ring4_hand_case.txt"))
            if l.strip() and not l.startswith("#")}
    xh = rows["x_half"].reshape(4, 1)
    x, xhat, q = oracle.gossip_mix(xh, np.zeros((4, 1), np.float32), ring(4), 1.0)
    assert np.allclose(x.ravel(), rows["x_out"], atol=1e-6)
    assert np.array_equal(xhat.ravel(), rows["x_hat_new"])
    assert np.array_equal(q, xh)


@pytest.mark.parametrize("k_frac", [1.0, 0.1, 0.01])
def test_average_is_preserved(k_frac):
    # doubly-stochastic W: sum_i x_i = sum_i x_half_i for any x_hat, gamma, k
    rng = np.random.default_rng(0)
    n, d = 8, 1000
    xh = rng.standard_normal((n, d)).astype(np.float32)
    xhat = rng.standard_normal((n, d)).astype(np.float32)
    k = max(1, int(k_frac * d))
    x, _, _ = oracle.gossip_mix(xh, xhat, ring(n), 0.37, [0, d], [k])
    assert np.allclose(x.astype(np.float64).sum(0), xh.astype(np.float64).sum(0),
                       atol=1e-6 * n * np.abs(xh).max())


def test_no_compression_is_plain_mixing():
    # k = d, gamma = 1, x_hat = anything: x_hat_new = x_half, and x = W @ x_half (D-PSGD)
    rng = np.random.default_rng(1)
    n, d = 6, 257
    xh = rng.standard_normal((n, d)).astype(np.float32)
    xhat0 = np.zeros((n, d), np.float32)
    W = ring(n)
    x, xhat, q = oracle.gossip_mix(xh, xhat0, W, 1.0)
    assert np.array_equal(xhat, xh)
    assert np.allclose(x, W.astype(np.float64) @ xh.astype(np.float64), atol=1e-6)
    # asymmetric row-stochastic W: row i holds the weights node i applies (not the transpose)
    Wa = rng.uniform(0, 1, (n, n)); Wa /= Wa.sum(1, keepdims=True)
    x, _, _ = oracle.gossip_mix(xh, xhat0, Wa.astype(np.float32), 1.0)
    assert np.allclose(x, Wa.astype(np.float32).astype(np.float64) @ xh, atol=2e-6)


def test_consensus_fixed_point_and_gamma():
    n, d = 5, 33
    row = np.linspace(-1, 1, d, dtype=np.float32)
    xh = np.tile(row, (n, 1))
    x, xhat, _ = oracle.gossip_mix(xh, xh.copy(), ring(n), 0.7)
    assert np.array_equal(x, xh) and np.array_equal(xhat, xh)
    # gamma scales the consensus term linearly
    rng = np.random.default_rng(2)
    xh = rng.standard_normal((n, d)).astype(np.float32)
    xhat = rng.standard_normal((n, d)).astype(np.float32)
    x1, _, _ = oracle.gossip_mix(xh, xhat, ring(n), 1.0, [0, d], [3])
    x2, _, _ = oracle.gossip_mix(xh, xhat, ring(n), 0.25, [0, d], [3])
    assert np.allclose((x2 - xh), 0.25 * (x1 - xh).astype(np.float64), atol=1e-6)


def test_topk_selection_rules():
    rng = np.random.default_rng(3)
    n, d, k = 3, 500, 17
    xh = rng.standard_normal((n, d)).astype(np.float32)
    xhat0 = rng.standard_normal((n, d)).astype(np.float32)
    _, xhat, q = oracle.gossip_mix(xh, xhat0, ring(n), 0.5, [0, d], [k])
    delta = xh - xhat0
    for i in range(n):
        nz = np.flatnonzero(q[i])
        assert len(nz) == k
        assert np.array_equal(q[i, nz], delta[i, nz])
        dropped = np.setdiff1d(np.arange(d), nz)
        assert np.abs(delta[i, nz]).min() >= np.abs(delta[i, dropped]).max()
    assert np.array_equal(xhat, xhat0 + q)                       # error feedback update
    # brute force: the kept set equals the k largest by (|delta| desc, index asc)
    for i in range(n):
        order = sorted(range(d), key=lambda e: (-abs(float(delta[i, e])), e))
        assert sorted(order[:k]) == np.flatnonzero(q[i]).tolist()


def test_topk_ties_keep_lower_index_and_segments():
    xh = np.array([[1, -1, 1, -1, 0.5, 2, 2, 2]], np.float32)
    xhat0 = np.zeros_like(xh)
    W1 = np.ones((1, 1), np.float32)
    _, _, q = oracle.gossip_mix(xh, xhat0, W1, 1.0, [0, 8], [3])
    assert q.tolist() == [[0, 0, 0, 0, 0, 2, 2, 2]]
    _, _, q = oracle.gossip_mix(xh, xhat0, W1, 1.0, [0, 5, 8], [2, 1])   # layer-wise top-k
    assert q.tolist() == [[1, -1, 0, 0, 0, 2, 0, 0]]
    _, _, q = oracle.gossip_mix(xh, xhat0, W1, 1.0, [0, 5, 8], [5, 2])   # k == len: dense segment
    assert q.tolist() == [[1, -1, 1, -1, 0.5, 2, 2, 0]]


def test_uses_updated_public_copies():
    # 2 nodes, W = 1/2 everywhere, k = d: x_i = xh_i + (1/2)(xh_j - xh_i) needs x_hat AFTER the update
    xh = np.array([[2.0], [6.0]], np.float32)
    W = np.full((2, 2), 0.5, np.float32)
    x, _, _ = oracle.gossip_mix(xh, np.array([[100.0], [-50.0]], np.float32), W, 1.0)
    assert x.ravel().tolist() == [4.0, 4.0]


def test_sgd_update():
    x = np.array([1.0, 2.0, -3.0], np.float32); g = np.array([0.5, -4.0, 0.25], np.float32)
    assert oracle.sgd_update(x, g, 0.1).tolist() == [np.float32(1.0) - np.float32(0.1) * np.float32(0.5),
                                                      np.float32(2.0) + np.float32(0.1) * np.float32(4.0),
                                                      np.float32(-3.0) - np.float32(0.1) * np.float32(0.25)]


def test_residual_add_and_adjoint():
    rng = np.random.default_rng(4)
    a = rng.standard_normal((2, 2, 4, 4, 3)).astype(np.float32)
    r = rng.standard_normal((2, 2, 4, 4, 3)).astype(np.float32)
    assert np.array_equal(oracle.residual_add(r, a), r + a)
    # projection shortcut: spatial subsample by 2, channels placed at offset 2 of 7
    r2 = rng.standard_normal((2, 2, 2, 2, 7)).astype(np.float32)
    y = oracle.residual_add(r2, a, stride=2, ch_off=2)
    want = r2.copy(); want[..., 2:5] += a[:, :, ::2, ::2, :]
    assert np.array_equal(y, want)
    dy = rng.standard_normal(r2.shape).astype(np.float32)
    gm = rng.standard_normal(a.shape).astype(np.float32)
    da = oracle.residual_add_bwd(dy, gm, stride=2, ch_off=2)
    want = gm.copy(); want[:, :, ::2, ::2, :] += dy[..., 2:5]
    assert np.array_equal(da, want)


def test_pools():
    rng = np.random.default_rng(5)
    x = rng.standard_normal((2, 3, 4, 6, 5)).astype(np.float32)
    assert np.allclose(oracle.avgpool(x), x.astype(np.float64).mean(axis=(2, 3)), atol=1e-7)
    dy = rng.standard_normal((2, 3, 5)).astype(np.float32)
    dx = oracle.avgpool_bwd(dy, 4, 6)
    assert np.array_equal(dx, np.broadcast_to((dy / np.float32(24))[:, :, None, None, :], dx.shape))
    y, idx = oracle.maxpool2x2(x)
    want = x.reshape(2, 3, 2, 2, 3, 2, 5).max(axis=(3, 5))
    assert np.array_equal(y, want)
    g = rng.standard_normal(y.shape).astype(np.float32)
    dxm = oracle.maxpool2x2_bwd(g, idx, 4, 6)
    assert np.allclose(dxm.sum(), g.sum(), atol=1e-4)
    assert np.array_equal(dxm.reshape(2, 3, 2, 2, 3, 2, 5).sum(axis=(3, 5)), g)
    assert np.all((dxm != 0) <= (x == np.repeat(np.repeat(y, 2, 2), 2, 3)))


def test_softmax_ce():
    from scipy.special import log_softmax, softmax
    rng = np.random.default_rng(6)
    z = (3 * rng.standard_normal((2, 5, 10))).astype(np.float32)
    lab = rng.integers(0, 10, (2, 5)).astype(np.int32)
    loss, dz = oracle.softmax_ce(z, lab)
    ls = log_softmax(z.astype(np.float64), axis=-1)
    want_loss = -np.take_along_axis(ls, lab[..., None].astype(np.int64), -1).mean(axis=(1, 2))
    assert np.allclose(loss, want_loss, atol=1e-6)
    onehot = np.eye(10)[lab]
    assert np.allclose(dz, (softmax(z.astype(np.float64), axis=-1) - onehot) / 5, atol=1e-7)
    assert np.allclose(dz.sum(-1), 0, atol=1e-6)


def test_colsum():
    x = np.arange(24, dtype=np.float32).reshape(2, 3, 4)
    assert np.array_equal(oracle.colsum(x), x.sum(1))


# ---- 8-bit messages (the quantized exchange behind the Data column's factor of four) ----
def test_q8_messages_on_the_grid_and_error_bound():
    rng = np.random.default_rng(3)
    n, d = 4, 3000
    xh = rng.standard_normal((n, d)).astype(np.float32)
    xhat = (xh - rng.standard_normal((n, d)) * rng.choice([1.0, 0.01], (n, d))).astype(np.float32)
    so, sk = [0, 1000, 3000], [50, 2000]                    # second segment dense
    x, xhat2, q, codes, scales = oracle.gossip_mix_q8(xh, xhat, ring(n), 0.4, so, sk)
    delta = xh - xhat
    for i in range(n):
        for s, (lo, hi) in enumerate(zip(so[:-1], so[1:])):
            k = min(sk[s], hi - lo)
            kept = codes[i, lo:hi] != 0
            sent = q[i, lo:hi] != 0
            assert sent.sum() <= k and np.array_equal(kept, sent)
            amax = np.abs(delta[i, lo:hi]).max()
            assert scales[i, s] == np.float32(amax) / np.float32(127.0)          # one range per (node, segment)
            assert np.abs(codes[i, lo:hi]).max() == 127                           # the largest entry maps to +-127
            # the message is code*scale exactly, within half a step of the difference on the entries sent
            assert np.array_equal(q[i, lo:hi], codes[i, lo:hi].astype(np.float32) * scales[i, s])
            err = np.abs(q[i, lo:hi][sent].astype(np.float64) - delta[i, lo:hi][sent])
            assert err.max() <= 0.5 * float(scales[i, s]) * (1 + 1e-6)
            # selection is the fp32-message one: same support as top-k of |delta| (up to codes that round to 0)
            _, _, q32 = oracle.gossip_mix(xh, xhat, ring(n), 0.4, so, sk)
            assert not (sent & (q32[i, lo:hi] == 0)).any()
    assert np.array_equal(xhat2, xhat + q)


def test_q8_average_is_preserved_and_error_feedback():
    # doubly-stochastic W: sum_i x_i = sum_i x_half_i for any public copies, quantized or not
    rng = np.random.default_rng(4)
    n, d = 6, 500
    xh = rng.standard_normal((n, d)).astype(np.float32)
    xhat = np.zeros((n, d), np.float32)
    x, xhat2, q, codes, scales = oracle.gossip_mix_q8(xh, xhat, ring(n), 0.7, [0, d], [25])
    np.testing.assert_allclose(x.sum(0, dtype=np.float64), xh.sum(0, dtype=np.float64), atol=1e-5)
    # what was not sent (dropped entries and rounding) stays in the next difference
    np.testing.assert_allclose((xh - xhat2).astype(np.float64), (xh - xhat).astype(np.float64) - q, atol=1e-6)


def test_q8_exact_when_differences_sit_on_the_grid():
    # differences that are integer multiples of amax/127 are sent without error: same result as fp32 messages
    n, d = 3, 254
    codes = np.tile(np.arange(-127, 127, dtype=np.float32), (n, 1))
    codes[:, 0] = 127                                          # the range is set by an entry equal to amax
    xh = (codes * np.float32(0.5)).astype(np.float32)          # amax = 63.5, scale = 0.5 exactly
    xhat = np.zeros((n, d), np.float32)
    x8, xhat8, q8, c8, s8 = oracle.gossip_mix_q8(xh, xhat, ring(n), 1.0)
    x32, xhat32, q32 = oracle.gossip_mix(xh, xhat, ring(n), 1.0)
    assert np.all(s8 == np.float32(0.5))
    assert np.array_equal(q8, q32) and np.array_equal(xhat8, xhat32) and np.array_equal(x8, x32)
    assert np.array_equal(c8, codes.astype(np.int8))


def test_q8_hand_case_and_zero_difference():
    # one node pair, d = 4: delta = [1.27, -0.635, 0.004, 0] -> scale 0.01, codes [127, -64 (63.5 -> even), 0, 0]
    xh = np.array([[1.27, -0.635, 0.004, 0.0], [0, 0, 0, 0]], np.float32)
    W = np.array([[0.5, 0.5], [0.5, 0.5]], np.float32)
    x, xhat, q, codes, scales = oracle.gossip_mix_q8(xh, np.zeros_like(xh), W, 1.0)
    assert codes[0].tolist()[0] == 127 and codes[0].tolist()[2:] == [0, 0] and codes[0, 1] in (-63, -64)
    t = np.float32(-0.635) * (np.float32(127.0) / np.float32(1.27))
    assert codes[0, 1] == int(np.rint(t))                     # ties resolved as rint does (half to even)
    assert scales[1, 0] == 1.0 and not codes[1].any()         # all-zero difference: scale 1, nothing sent
    np.testing.assert_allclose(x[1], 0.5 * xhat[0], rtol=1e-6)


# ---- Deep-Squeeze mixing (supplementary Algorithm 2) ----
def test_deepsqueeze_without_compression_is_plain_mixing():
    # k = d, zero error buffer, eta = 1: x = x_half + (W x_half - x_half) = W x_half, a matrix product
    rng = np.random.default_rng(7)
    n, d = 5, 64
    xh = rng.standard_normal((n, d)).astype(np.float32)
    x, delta, c, _ = oracle.deepsqueeze_mix(xh, np.zeros((n, d), np.float32), ring(n), 1.0)
    np.testing.assert_allclose(x, ring(n).astype(np.float64) @ xh.astype(np.float64), rtol=1e-6, atol=1e-6)
    assert not delta.any() and np.array_equal(c, xh)


@pytest.mark.parametrize("bits", [32, 8])
def test_deepsqueeze_error_feedback_and_average(bits):
    rng = np.random.default_rng(8)
    n, d, k = 6, 400, 20
    xh = rng.standard_normal((n, d)).astype(np.float32)
    delta0 = (0.1 * rng.standard_normal((n, d))).astype(np.float32)
    x, delta, c, scales = oracle.deepsqueeze_mix(xh, delta0, ring(n), 0.5, [0, d], [k], bits)
    v = xh + delta0
    assert all(np.count_nonzero(c[i]) <= k for i in range(n))
    # what is sent plus what is carried over is the compensated update (v - c is exact or within an ulp)
    np.testing.assert_allclose((c + delta).astype(np.float64), v.astype(np.float64), rtol=2e-7, atol=1e-7)
    # the kept entries are the largest of |v|
    for i in range(n):
        sent = c[i] != 0
        if bits == 32:
            assert sent.sum() == k and np.array_equal(c[i][sent], v[i][sent])
        assert np.abs(v[i][sent]).min() >= np.abs(v[i][~sent]).max() - 1e-7
        if bits == 8:
            codes = c[i][sent] / scales[i, 0]
            assert np.allclose(codes, np.rint(codes)) and np.abs(codes).max() <= 127
            assert scales[i, 0] == np.float32(np.abs(v[i]).max()) / np.float32(127.0)
    # doubly-stochastic W: the node average moves only by the local updates
    np.testing.assert_allclose(x.sum(0, dtype=np.float64), xh.sum(0, dtype=np.float64), atol=1e-5)


def test_deepsqueeze_hand_case():
    # ring of 4, d = 1, W = 1/3, k = 1 (everything sent), delta = [1, 0, 0, -1], x_half = [0, 3, 6, 9], eta = 1:
    # v = c = [1, 3, 6, 8]; x_i = x_half_i + (c_{i-1} + c_i + c_{i+1})/3 - c_i
    xh = np.array([[0.0], [3.0], [6.0], [9.0]], np.float32)
    d0 = np.array([[1.0], [0.0], [0.0], [-1.0]], np.float32)
    x, delta, c, _ = oracle.deepsqueeze_mix(xh, d0, ring(4), 1.0, [0, 1], [1])
    assert c[:, 0].tolist() == [1.0, 3.0, 6.0, 8.0] and not delta.any()
    want = [0 + (8 + 1 + 3) / 3 - 1, 3 + (1 + 3 + 6) / 3 - 3, 6 + (3 + 6 + 8) / 3 - 6, 9 + (6 + 8 + 1) / 3 - 8]
    np.testing.assert_allclose(x[:, 0], want, rtol=1e-6)
    # k = 0: nothing is sent, the whole compensated update is carried over and x = x_half
    x, delta, c, _ = oracle.deepsqueeze_mix(xh, d0, ring(4), 1.0, [0, 1], [0])
    assert not c.any() and np.array_equal(delta, xh + d0) and np.array_equal(x, xh)


# ---- push-sum bias weights (supplementary Algorithms 4-5) ----
def _column_stochastic(n, seed):
    rng = np.random.default_rng(seed)
    W = rng.random((n, n)) * (rng.random((n, n)) < 0.5)
    W[np.arange(n), np.arange(n)] += 0.5                      # every node keeps part of its own mass
    return (W / W.sum(0, keepdims=True)).astype(np.float32)   # columns sum to one: mass is conserved


def test_pushsum_mass_conservation_and_debias():
    n, d = 7, 33
    W = _column_stochastic(n, 1)
    rng = np.random.default_rng(2)
    u = np.ones(n, np.float32)
    x = rng.standard_normal((n, d)).astype(np.float32)
    for _ in range(5):
        u2, z = oracle.pushsum_debias(x, u, W, 1.0)
        # eta = 1: u_new = W u, a matrix-vector product; column-stochastic W keeps sum(u) = n
        np.testing.assert_allclose(u2, W.astype(np.float64) @ u.astype(np.float64), rtol=1e-6)
        np.testing.assert_allclose(u2.sum(dtype=np.float64), n, rtol=1e-6)
        np.testing.assert_allclose(z * u2[:, None], x, rtol=3e-7, atol=1e-30)     # z = x / u_new
        u = u2
    assert np.abs(u - 1).max() > 1e-3                         # a directed graph does move the weights


def test_pushsum_trivial_on_doubly_stochastic_ring():
    n, d = 6, 10
    x = np.random.default_rng(3).standard_normal((n, d)).astype(np.float32)
    u2, z = oracle.pushsum_debias(x, np.ones(n, np.float32), ring(n), 0.7)
    np.testing.assert_allclose(u2, 1.0, rtol=1e-6)            # rows also sum to one: weights stay at 1
    np.testing.assert_allclose(z, x, rtol=1e-6)


def test_pushsum_average_consensus_through_debiasing():
    # uncompressed push-sum gossip with zero gradients converges to the average of the initial models
    # although W is only column-stochastic: x <- W x, u <- W u, z = x / u
    n, d = 5, 4
    W = _column_stochastic(n, 4)
    x = np.random.default_rng(5).standard_normal((n, d)).astype(np.float32)
    mean = x.mean(0, dtype=np.float64)
    u = np.ones(n, np.float32)
    for _ in range(200):
        x, _, _, _ = oracle.deepsqueeze_mix(x, np.zeros_like(x), W, 1.0)        # k = d: x <- W x
        u, z = oracle.pushsum_debias(x, u, W, 1.0)
    np.testing.assert_allclose(z, np.tile(mean, (n, 1)), atol=1e-4)
