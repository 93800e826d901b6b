"""Pins for the oracle's synchronisation rules (Algorithms 2-4): closed forms, conservation laws,
hand-computed fixtures.  CPU only."""
import os

import numpy as np
import pytest

from oracle import shadowsync_oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    out = []
    for line in open(os.path.join(GOLD, name)):
        line = line.strip()
        if line and not line.startswith("#"):
            out.append([float(x) for x in line.split()])
    return out


def _vecs(R, n, seed=0):
    rng = np.random.default_rng(seed)
    return [rng.normal(0, 0.02, n).astype(np.float32) for _ in range(R)]


# ---------------------------------------------------------------- EASGD (Algorithm 2)
def test_easgd_golden_single_trainer():
    rows = _rows("easgd_single_trainer.txt")
    w = np.array([rows[0][1]], dtype=np.float32)
    c = np.array([rows[0][2]], dtype=np.float32)
    for k, wk, ck in rows[1:]:
        O.sync_easgd([w], c, 0.25)
        assert w[0] == np.float32(wk) and c[0] == np.float32(ck)


def test_easgd_golden_literal_order():
    a, w0, c0, wl, cl, ws, cs = _rows("easgd_literal_order.txt")[0]
    w, c = np.array([w0], np.float32), np.array([c0], np.float32)
    O.sync_easgd([w], c, a, literal=True)
    assert (w[0], c[0]) == (wl, cl)
    w, c = np.array([w0], np.float32), np.array([c0], np.float32)
    O.sync_easgd([w], c, a)
    assert (w[0], c[0]) == (ws, cs)


def test_easgd_alpha0_is_identity_bitwise():
    ws = _vecs(4, 1000)
    c = _vecs(1, 1000, 9)[0]
    ws0, c0 = [w.copy() for w in ws], c.copy()
    O.sync_easgd(ws, c, 0.0)
    assert all(np.array_equal(a, b) for a, b in zip(ws, ws0)) and np.array_equal(c, c0)


@pytest.mark.parametrize("R", [1, 2, 4, 16])
def test_easgd_conserves_centre_plus_replicas(R):
    ws = _vecs(R, 4096)
    c = _vecs(1, 4096, 5)[0]
    before = c.astype(np.float64) + sum(w.astype(np.float64) for w in ws)
    O.sync_easgd(ws, c, 0.1)
    after = c.astype(np.float64) + sum(w.astype(np.float64) for w in ws)
    np.testing.assert_allclose(after, before, rtol=0, atol=(R + 1) * 4e-9)


def test_easgd_all_equal_is_fixed_point():
    w = _vecs(1, 512)[0]
    ws = [w.copy() for _ in range(3)]
    c = w.copy()
    O.sync_easgd(ws, c, 0.3)
    for x in ws + [c]:
        np.testing.assert_allclose(x, w, rtol=1e-7)


def test_easgd_closed_form_single_trainer():
    # w_k - c_k = (1-2a)^k (w_0 - c_0) and w_k + c_k constant
    a, k = 0.1, 7
    w = _vecs(1, 256, 1)[0]
    c = _vecs(1, 256, 2)[0]
    diff0 = w.astype(np.float64) - c
    sum0 = w.astype(np.float64) + c
    for _ in range(k):
        O.sync_easgd([w], c, a)
    np.testing.assert_allclose(w.astype(np.float64) - c, (1 - 2 * a) ** k * diff0, atol=2e-8)
    np.testing.assert_allclose(w.astype(np.float64) + c, sum0, atol=2e-8)


def test_easgd_half_alpha_meets_in_the_middle():
    w = _vecs(1, 64, 1)[0]
    c = _vecs(1, 64, 2)[0]
    mid = (0.5 * (w.astype(np.float64) + c)).astype(np.float32)
    O.sync_easgd([w], c, 0.5)
    assert np.array_equal(w, c) and np.array_equal(w, mid)


def test_easgd_literal_differs_by_alpha_squared():
    a = 0.2
    w0 = _vecs(1, 300, 1)[0]
    c0 = _vecs(1, 300, 2)[0]
    w1, c1 = w0.copy(), c0.copy()
    w2, c2 = w0.copy(), c0.copy()
    O.sync_easgd([w1], c1, a)
    O.sync_easgd([w2], c2, a, literal=True)
    assert np.array_equal(c1, c2)
    np.testing.assert_allclose(w2.astype(np.float64) - w1, a * a * (w0.astype(np.float64) - c0), atol=1e-8)


def test_easgd_round_robin_order_matters_and_is_sequential():
    # the second replica sees the centre already moved by the first (trainers visit the PS in turn)
    w1, w2, c = (np.array([x], np.float32) for x in (1.0, 1.0, 0.0))
    O.sync_easgd([w1, w2], c, 0.5)
    # visit 1: d=.5 -> w1=.5, c=.5 ; visit 2: d=.25 -> w2=.75, c=.75
    assert (w1[0], w2[0], c[0]) == (0.5, 0.75, 0.75)


# ---------------------------------------------------------------- MA (Algorithm 3)
def test_ma_golden():
    r = _rows("ma_scalar.txt")[0]
    ws = [np.array([x], np.float32) for x in r[1:4]]
    O.sync_ma(ws, r[0])
    assert [float(w[0]) for w in ws] == r[4:7]


@pytest.mark.parametrize("R", [2, 4, 8, 16])
def test_ma_identical_replicas_identity_bitwise(R):
    w = _vecs(1, 2048)[0]
    ws = [w.copy() for _ in range(R)]
    O.sync_ma(ws, 0.37)
    # (1-a)w + a*w in double rounds back to w for R a power of two (the mean is exact)
    for x in ws:
        np.testing.assert_allclose(x, w, rtol=1.2e-7)
    ws = [w.copy() for _ in range(R)]
    O.sync_ma(ws, 1.0)
    assert all(np.array_equal(x, w) for x in ws)


def test_ma_sum_conserved_and_alpha_limits():
    ws = _vecs(5, 1024)
    ws0 = [w.copy() for w in ws]
    tot = sum(w.astype(np.float64) for w in ws)
    O.sync_ma(ws, 0.25)
    np.testing.assert_allclose(sum(w.astype(np.float64) for w in ws), tot, atol=5 * 4e-9)
    ws = [w.copy() for w in ws0]
    O.sync_ma(ws, 0.0)
    assert all(np.array_equal(a, b) for a, b in zip(ws, ws0))
    g = np.zeros(1024, np.float32)
    O.sync_ma(ws, 1.0, g)
    mean = (tot / 5).astype(np.float32)
    assert all(np.array_equal(w, mean) for w in ws) and np.array_equal(g, mean)


def test_ma_contracts_spread_by_one_minus_alpha():
    ws = _vecs(4, 512)
    spread0 = ws[0].astype(np.float64) - ws[3]
    O.sync_ma(ws, 0.3)
    np.testing.assert_allclose(ws[0].astype(np.float64) - ws[3], 0.7 * spread0, atol=1e-8)


# ---------------------------------------------------------------- BMUF (Algorithm 4)
def test_bmuf_golden():
    for mu, d0, g1, d1, w1, w2 in _rows("bmuf_scalar.txt"):
        ws = [np.array([1.0], np.float32), np.array([3.0], np.float32)]
        g, d = np.array([0.0], np.float32), np.array([d0], np.float32)
        O.sync_bmuf(ws, g, d, alpha=0.25, eta=0.5, mu=mu)
        assert (g[0], d[0], ws[0][0], ws[1][0]) == (g1, d1, w1, w2)


def test_bmuf_nesterov_golden_and_limits():
    for mu, d0, g1, d1, w1, w2 in _rows("bmuf_nesterov_scalar.txt"):
        ws = [np.array([1.0], np.float32), np.array([3.0], np.float32)]
        g, d = np.array([0.0], np.float32), np.array([d0], np.float32)
        O.sync_bmuf(ws, g, d, alpha=0.25, eta=0.5, mu=mu, nesterov=True)
        assert (g[0], d[0], ws[0][0], ws[1][0]) == (g1, d1, w1, w2)
    # without momentum the look-ahead point is the global model itself
    a, b = _vecs(3, 500), _vecs(3, 500)
    ga, gb = _vecs(1, 500, 4)[0], _vecs(1, 500, 4)[0]
    da, db = np.zeros(500, np.float32), np.zeros(500, np.float32)
    O.sync_bmuf(a, ga, da, 0.1, 0.7, 0.0, nesterov=True)
    O.sync_bmuf(b, gb, db, 0.1, 0.7, 0.0, nesterov=False)
    assert all(np.array_equal(x, y) for x, y in zip(a, b)) and np.array_equal(ga, gb)
    # the global model and the momentum do not depend on the variant; replicas differ by alpha*mu*delta
    a, b = _vecs(3, 500), _vecs(3, 500)
    ga, gb = _vecs(1, 500, 4)[0], _vecs(1, 500, 4)[0]
    da, db = _vecs(1, 500, 6)[0], _vecs(1, 500, 6)[0]
    O.sync_bmuf(a, ga, da, 0.2, 1.0, 0.9, nesterov=True)
    O.sync_bmuf(b, gb, db, 0.2, 1.0, 0.9, nesterov=False)
    assert np.array_equal(ga, gb) and np.array_equal(da, db)
    np.testing.assert_allclose(a[1].astype(np.float64) - b[1], 0.2 * 0.9 * da.astype(np.float64), atol=1e-8)


def test_bmuf_mu0_eta1_equals_ma():
    ws_a = _vecs(8, 3000)
    ws_b = [w.copy() for w in ws_a]
    g = _vecs(1, 3000, 7)[0]
    d = np.zeros(3000, np.float32)
    gm = np.zeros(3000, np.float32)
    O.sync_ma(ws_a, 0.05, gm)
    O.sync_bmuf(ws_b, g, d, alpha=0.05, eta=1.0, mu=0.0)
    # g + (m - g) can differ from m by one rounding of the difference
    np.testing.assert_allclose(g, gm, atol=1e-8)
    for a, b in zip(ws_a, ws_b):
        np.testing.assert_allclose(a, b, atol=1e-9)


def test_bmuf_fixed_point():
    g = _vecs(1, 100)[0]
    ws = [g.copy() for _ in range(4)]
    d = np.zeros(100, np.float32)
    O.sync_bmuf(ws, g.copy(), d, 0.1, 1.0, 0.9)
    assert all(np.array_equal(w, g) for w in ws) and not d.any()


def test_bmuf_momentum_second_order_recurrence():
    # with the replicas held at a constant mean m (alpha=0), e_k = g_k - m obeys
    # e_{k+1} = (1 + mu - eta) e_k - mu e_{k-1}
    mu, eta = 0.9, 0.3
    ws = _vecs(4, 50)
    m = np.mean(np.stack(ws).astype(np.float64), axis=0)
    g = _vecs(1, 50, 3)[0]
    d = np.zeros(50, np.float32)
    e = [g.astype(np.float64) - m]
    for _ in range(6):
        O.sync_bmuf(ws, g, d, 0.0, eta, mu)
        e.append(g.astype(np.float64) - m)
    # first step has e_{-1} = e_0 (delta_0 = 0)
    np.testing.assert_allclose(e[1], (1 - eta) * e[0], atol=1e-8)
    for k in range(1, 6):
        np.testing.assert_allclose(e[k + 1], (1 + mu - eta) * e[k] - mu * e[k - 1], atol=2e-8)


def test_bmuf_eta_geometric_without_momentum():
    ws = _vecs(2, 40)
    m = np.mean(np.stack(ws).astype(np.float64), axis=0)
    g = _vecs(1, 40, 3)[0]
    e0 = g.astype(np.float64) - m
    d = np.zeros(40, np.float32)
    for _ in range(5):
        O.sync_bmuf(ws, g, d, 0.0, 0.5, 0.0)
    np.testing.assert_allclose(g.astype(np.float64) - m, 0.5 ** 5 * e0, atol=1e-8)


# ---------------------------------------------------------------- metrics (Section 4)
def test_ne_of_constant_predictor_is_one():
    y = (np.arange(1000) % 25 == 0).astype(np.float32)
    assert abs(O.normalized_entropy(np.full(1000, y.mean()), y) - 1.0) < 1e-12


def test_avg_sync_gap_definition():
    # 5.21 iterations per sync when a trainer runs 521 iterations/s and syncs 100 times/s (Table 2's value)
    assert abs(O.avg_sync_gap(521.0, 100.0) - 5.21) < 1e-12


def test_round_bf16():
    x = np.array([1.0, 1.00390625, 1.01171875, -3.0e-40, 65504.0, 1.0 + 2 ** -9], np.float32)
    # 1+2^-8 is a tie -> even (1.0); 1+3*2^-8 is a tie -> even (1+2^-6); 1+2^-9 rounds down
    got = O.round_bf16(x)
    import torch
    ref = torch.from_numpy(x).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(got, ref)
    assert got[1] == 1.0 and got[2] == 1.015625
    rng = np.random.default_rng(0)
    r = rng.normal(0, 1, 10000).astype(np.float32)
    assert np.array_equal(O.round_bf16(r), torch.from_numpy(r).to(torch.bfloat16).to(torch.float64).numpy())
