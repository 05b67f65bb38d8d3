"""Pins for the oracle's embedding predictor (LSTM + graph convolution + skip) and cache ring."""
import numpy as np
import pytest
import torch

from oracle import sat_ref as orc
from tests.dense_pins import csr_from_edges, dense_P, random_graph


def test_five_node_predictor_numbers(five_node):
    g = five_node
    pr = g["pred"]
    rowptr, col = csr_from_edges(5, g["edges"])
    dtil, _ = orc.degrees(rowptr)
    P = orc.build_partition(rowptr, col, np.array(g["part"], dtype=np.int32), 2)
    old = np.array([[pr["history_old_new"][str(v)][0]] for v in g["C"]], dtype=np.float32)
    new = np.array([[pr["history_old_new"][str(v)][1]] for v in g["C"]], dtype=np.float32)
    Wx, Uh, b = np.array(pr["Wx"]), np.array(pr["Uh"]), np.array(pr["b"])
    Wg, bg = np.array(pr["Wg"]), np.array(pr["bg"])
    S1 = orc.lstm_state([old], 1, 1, Wx, Uh, b, 3)
    assert abs(S1[0, 0] - pr["node1_step1"]["s"]) < 2e-6
    S = orc.lstm_state([old, new], 1, 1, Wx, Uh, b, 3)
    np.testing.assert_allclose(S[:, 0], pr["S"], atol=2e-6)
    out0 = orc.predict_halo(P, 0, dtil, S, new, Wg, bg)
    out1 = orc.predict_halo(P, 1, dtil, S, new, Wg, bg)
    np.testing.assert_allclose(out0[:, 0], pr["Hhat_part0"], atol=3e-6)
    np.testing.assert_allclose(out1[:, 0], pr["Hhat_part1"], atol=3e-6)
    # the gate values of the first step, from the textbook cell written out
    x = 1.0
    a = x * Wx[0]
    sig = lambda t: 1 / (1 + np.exp(-t))
    a = a + b
    i, f, gg, o = sig(a[0]), sig(a[1]), np.tanh(a[2]), sig(a[3])
    assert abs(i - pr["node1_step1"]["i"]) < 1e-6 and abs(f - pr["node1_step1"]["f"]) < 1e-6
    assert abs(gg - pr["node1_step1"]["g"]) < 1e-6 and abs(o - pr["node1_step1"]["o"]) < 1e-6
    assert abs(i * gg - pr["node1_step1"]["c"]) < 1e-6


@pytest.mark.parametrize("k,d,h", [(1, 5, 3), (4, 9, 6), (8, 16, 16)])
def test_lstm_against_library_cell(k, d, h):
    """Same weights through torch.nn.LSTM in float64 (gate order i, f, g, o; zero initial state)."""
    rng = np.random.default_rng(k * 100 + d)
    n = 11
    snaps = [rng.standard_normal((n, d)).astype(np.float32) for _ in range(k)]
    Wx = (rng.standard_normal((d, 4 * h)) * 0.4).astype(np.float32)
    Uh = (rng.standard_normal((h, 4 * h)) * 0.4).astype(np.float32)
    b = (rng.standard_normal(4 * h) * 0.2).astype(np.float32)
    S = orc.lstm_state(snaps, d, h, Wx, Uh, b, n)
    lstm = torch.nn.LSTM(d, h, batch_first=False).double()
    with torch.no_grad():
        lstm.weight_ih_l0.copy_(torch.tensor(Wx.T, dtype=torch.float64))
        lstm.weight_hh_l0.copy_(torch.tensor(Uh.T, dtype=torch.float64))
        lstm.bias_ih_l0.copy_(torch.tensor(b, dtype=torch.float64))
        lstm.bias_hh_l0.zero_()
        x = torch.tensor(np.stack(snaps), dtype=torch.float64)      # [k, n, d]
        _, (hn, _) = lstm(x)
    np.testing.assert_allclose(S, hn[0].numpy(), atol=1e-6)
    # a subset of slots gives the same rows
    sel = np.array([7, 2], dtype=np.int32)
    S2 = orc.lstm_state(snaps, d, h, Wx, Uh, b, n, slots_sel=sel)
    assert np.array_equal(S2[sel], S[sel])


def test_lstm_degenerate_cases():
    rng = np.random.default_rng(0)
    n, d, h = 5, 4, 3
    snaps = [rng.standard_normal((n, d)).astype(np.float32) for _ in range(3)]
    z = lambda *s: np.zeros(s, dtype=np.float32)
    # all-zero parameters: gates are 1/2, g = 0 -> c = 0 -> s = 0
    assert np.all(orc.lstm_state(snaps, d, h, z(d, 4 * h), z(h, 4 * h), z(4 * h), n) == 0)
    # no snapshot: zero state
    assert np.all(orc.lstm_state([], d, h, z(d, 4 * h), z(h, 4 * h), z(4 * h), n) == 0)
    # k = 1, U = 0: s = sigm(a_o) tanh(sigm(a_i) tanh(a_g))
    Wx = (rng.standard_normal((d, 4 * h)) * 0.5).astype(np.float32)
    b = (rng.standard_normal(4 * h) * 0.5).astype(np.float32)
    S = orc.lstm_state(snaps[:1], d, h, Wx, z(h, 4 * h), b, n)
    a = snaps[0].astype(np.float64) @ Wx.astype(np.float64) + b
    sig = lambda t: 1 / (1 + np.exp(-t))
    want = sig(a[:, 3 * h:]) * np.tanh(sig(a[:, :h]) * np.tanh(a[:, 2 * h:3 * h]))
    np.testing.assert_allclose(S, want, atol=1e-7)


def test_predictor_graph_conv_against_dense_and_identity():
    rng = np.random.default_rng(9)
    n, M, h, d = 30, 3, 4, 6
    rowptr, col = random_graph(rng, n, 0.2)
    dtil, _ = orc.degrees(rowptr)
    part = rng.integers(0, M, size=n).astype(np.int32)
    P = orc.build_partition(rowptr, col, part, M)
    S = rng.standard_normal((P.n_slots, h)).astype(np.float32)
    newest = rng.standard_normal((P.n_slots, d)).astype(np.float32)
    Wg = rng.standard_normal((h, d)).astype(np.float32)
    bg = rng.standard_normal(d).astype(np.float32)
    Pm = dense_P(rowptr, col)
    Sfull = np.zeros((n, h))
    Sfull[P.slot >= 0] = S[P.slot[P.slot >= 0]]
    for m in range(M):
        out = orc.predict_halo(P, m, dtil, S, newest, Wg, bg)
        halo = P.halo_gid[m]
        # dense statement: rows of P restricted to (u itself) + (neighbours inside V_m)
        keep = (part == m)[None, :] | (np.arange(n)[None, :] == halo[:, None])
        a = (Pm[halo] * keep) @ Sfull
        want = newest[P.slot[halo]].astype(np.float64) + a @ Wg.astype(np.float64) + bg
        np.testing.assert_allclose(out, want, atol=2e-6)
        # zero output weights: the predictor is the identity on the newest snapshot
        ident = orc.predict_halo(P, m, dtil, S, newest, np.zeros_like(Wg), np.zeros_like(bg))
        assert np.array_equal(ident, newest[P.slot[halo]])
        assert np.array_equal(ident, orc.historical_halo(P, m, newest, d))
        # linear in S
        out2 = orc.predict_halo(P, m, dtil, 2 * S, newest, Wg, np.zeros_like(bg))
        out1 = orc.predict_halo(P, m, dtil, S, newest, Wg, np.zeros_like(bg))
        np.testing.assert_allclose(out2 - newest[P.slot[halo]], 2 * (out1 - newest[P.slot[halo]]), atol=5e-6)
        # all-zero LSTM state: prediction = newest + b_g
        outz = orc.predict_halo(P, m, dtil, np.zeros_like(S), newest, Wg, bg)
        np.testing.assert_allclose(outz, newest[P.slot[halo]] + bg, atol=1e-6)
        # no committed snapshot
        outn = orc.predict_halo(P, m, dtil, np.zeros_like(S), None, Wg, bg)
        np.testing.assert_allclose(outn, np.broadcast_to(bg, outn.shape), atol=1e-7)


def test_cache_ring_window():
    tau, n, w = 3, 4, 2
    ring = orc.CacheRing(n, [w], tau)
    assert ring.snapshots(1) == [] and ring.newest(1) is None
    for t in range(1, 8):
        ring.push(1, np.arange(n), np.full((n, w), float(t), dtype=np.float32))
        # a push is invisible until the commit
        if t > 1:
            assert ring.newest(1)[0, 0] == float(t - 1)
        ring.commit()
        vals = [float(s[0, 0]) for s in ring.snapshots(1)]
        assert vals == [float(x) for x in range(max(1, t - tau + 1), t + 1)]   # a snapshot leaves after tau commits
        assert ring.n_valid == min(t, tau)
        assert ring.write_idx == t % (tau + 1)


@pytest.mark.parametrize("k,d,h", [(1, 5, 3), (4, 9, 6), (7, 16, 8)])
def test_gru_against_library_cell(k, d, h):
    """Same weights through torch.nn.GRU in float64 (gate order r, z, n; the hidden-side bias only on the candidate)."""
    rng = np.random.default_rng(k * 10 + d)
    n = 9
    snaps = [rng.standard_normal((n, d)).astype(np.float32) for _ in range(k)]
    Wx = (rng.standard_normal((d, 3 * h)) * 0.4).astype(np.float32)
    Uh = (rng.standard_normal((h, 3 * h)) * 0.4).astype(np.float32)
    b = (rng.standard_normal(4 * h) * 0.3).astype(np.float32)
    S = orc.gru_state(snaps, d, h, Wx, Uh, b, n)
    gru = torch.nn.GRU(d, h, batch_first=False).double()
    with torch.no_grad():
        gru.weight_ih_l0.copy_(torch.tensor(Wx.T, dtype=torch.float64))
        gru.weight_hh_l0.copy_(torch.tensor(Uh.T, dtype=torch.float64))
        gru.bias_ih_l0.copy_(torch.tensor(b[:3 * h], dtype=torch.float64))
        bh = np.zeros(3 * h)
        bh[2 * h:] = b[3 * h:]
        gru.bias_hh_l0.copy_(torch.tensor(bh, dtype=torch.float64))
        _, hn = gru(torch.tensor(np.stack(snaps), dtype=torch.float64))
    np.testing.assert_allclose(S, hn[0].numpy(), atol=1e-6)
    sel = np.array([4, 1], dtype=np.int32)
    S2 = orc.gru_state(snaps, d, h, Wx, Uh, b, n, slots_sel=sel)
    assert np.array_equal(S2[sel], S[sel])


def test_gru_degenerate_cases():
    rng = np.random.default_rng(1)
    n, d, h = 5, 4, 3
    snaps = [rng.standard_normal((n, d)).astype(np.float32) for _ in range(3)]
    z = lambda *s: np.zeros(s, dtype=np.float32)
    # all-zero parameters: z = 1/2, n = 0 -> the state halves from zero: stays zero; no snapshot: zero state
    assert np.all(orc.gru_state(snaps, d, h, z(d, 3 * h), z(h, 3 * h), z(4 * h), n) == 0)
    assert np.all(orc.gru_state([], d, h, z(d, 3 * h), z(h, 3 * h), z(4 * h), n) == 0)
    # one step from the zero state: s = (1 - sigm(a_z)) tanh(a_n + sigm(a_r) b_hn)
    Wx = (rng.standard_normal((d, 3 * h)) * 0.5).astype(np.float32)
    Uh = (rng.standard_normal((h, 3 * h)) * 0.5).astype(np.float32)
    b = (rng.standard_normal(4 * h) * 0.5).astype(np.float32)
    S = orc.gru_state(snaps[:1], d, h, Wx, Uh, b, n)
    a = snaps[0].astype(np.float64) @ Wx.astype(np.float64) + b[:3 * h]
    sig = lambda t: 1 / (1 + np.exp(-t))
    want = (1 - sig(a[:, h:2 * h])) * np.tanh(a[:, 2 * h:] + sig(a[:, :h]) * b[3 * h:])
    np.testing.assert_allclose(S, want, atol=1e-7)
    # a saturated update gate (b_z large) freezes the state: it stays at its initial zero whatever the inputs
    b2 = b.copy()
    b2[h:2 * h] = 40.0
    assert np.abs(orc.gru_state(snaps, d, h, Wx, Uh, b2, n)).max() < 1e-12
