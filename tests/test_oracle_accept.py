"""Pins for the oracle's speculative acceptance (Eq. 1 and the resampling rule): the losslessness identity
measured from the oracle's own decisions on a tiny vocabulary (exactly, by locating its decision
boundaries, and empirically over a million seeded draws), plus special cases.  CPU only."""
import numpy as np
from scipy.special import softmax

import oracle


def run1(tl, dl, x, ua, ur):
    n, out, _, _ = oracle.accept(tl[None], dl[None], np.asarray(x, np.int32)[None], np.asarray(ua, np.float32)[None],
                                 np.asarray([ur], np.float32))
    return int(n[0]), out[0].tolist()


def accept_measure(tl, dl, x):
    """Lebesgue measure of {u in [0,1): the oracle accepts draft token x at row 0}, by bisection."""
    if run1(tl, dl, [x], [np.nextafter(np.float32(1), np.float32(0))], 0.5)[0] == 1:
        return 1.0
    lo, hi = 0.0, 1.0   # accepted at lo (u=0 accepts whenever P[x] > 0), rejected at hi
    if run1(tl, dl, [x], [0.0], 0.5)[0] == 0:
        return 0.0
    for _ in range(40):
        mid = np.float32((lo + hi) / 2)
        if mid == np.float32(lo) or mid == np.float32(hi):
            break
        if run1(tl, dl, [x], [mid], 0.5)[0] == 1:
            lo = float(mid)
        else:
            hi = float(mid)
    return (lo + hi) / 2


def resample_measures(tl, dl, x_rej, V, n_grid=4001):
    """Measure of u_res mapped to each token after a rejection of x_rej: boundaries located by bisection."""
    def tok(u):
        n, out = run1(tl, dl, [x_rej], [np.nextafter(np.float32(1), np.float32(0))], u)
        assert n == 0
        return out[0]
    edges, cur, lo = [0.0], tok(0.0), 0.0
    toks = [cur]
    while True:
        # find the first grid point where the token changes, then bisect
        us = np.linspace(lo, 1.0, n_grid, dtype=np.float64)[1:]
        nxt = None
        for u in us:
            if u < 1.0 and tok(np.float32(u)) != cur:
                nxt = float(np.float32(u))
                break
        if nxt is None:
            break
        a, b = lo, nxt
        for _ in range(40):
            m = np.float32((a + b) / 2)
            if m == np.float32(a) or m == np.float32(b):
                break
            if tok(m) == cur:
                a = float(m)
            else:
                b = float(m)
        edges.append((a + b) / 2)
        cur, lo = tok(np.float32(b)), b
        toks.append(cur)
    edges.append(1.0)
    meas = np.zeros(V)
    for i, t in enumerate(toks):
        meas[t] += edges[i + 1] - edges[i]
    assert toks == sorted(toks)   # inverse CDF in ascending token id
    return meas


def test_lossless_identity_by_enumeration():
    """sum_x Q[x] * (a_x * [t = x] + (1 - a_x) * r_x[t]) = P[t], with a_x and r_x measured from the oracle."""
    rng = np.random.default_rng(0)
    V = 6
    for trial in range(3):
        tl = (rng.standard_normal((2, V)) * 1.5).astype(np.float32)
        dl = (rng.standard_normal((1, V)) * 1.5).astype(np.float32)
        P = softmax(tl[0].astype(np.float64))
        Q = softmax(dl[0].astype(np.float64))
        law = np.zeros(V)
        acc_total = 0.0
        for x in range(V):
            a = accept_measure(tl, dl, x)
            law[x] += Q[x] * a
            acc_total += Q[x] * a
            if a < 1.0:
                r = resample_measures(tl, dl, x, V)
                law += Q[x] * (1 - a) * r
        np.testing.assert_allclose(law, P, atol=3e-6)
        # per-position acceptance probability = sum min(P, Q) = 1 - TV(P, Q)
        np.testing.assert_allclose(acc_total, np.minimum(P, Q).sum(), atol=1e-6)


def test_lossless_identity_empirical_chain():
    """A million seeded draws, V = 6, gamma = 3: the token emitted at each reached position follows P_j."""
    rng = np.random.default_rng(1)
    V, g, N = 6, 3, 1_000_000
    tl = (rng.standard_normal((g + 1, V)) * 1.2).astype(np.float32)
    dl = (tl[:g] + 0.8 * rng.standard_normal((g, V))).astype(np.float32)
    P, Q = softmax(tl.astype(np.float64), axis=1), softmax(dl.astype(np.float64), axis=1)
    x = np.stack([rng.choice(V, size=N, p=Q[j]) for j in range(g)], axis=1).astype(np.int32)
    ua = rng.random((N, g), dtype=np.float32)
    ur = rng.random(N, dtype=np.float32)
    n, out, _, _ = oracle.accept(np.broadcast_to(tl, (N, g + 1, V)), np.broadcast_to(dl, (N, g, V)), x, ua, ur)
    assert n.min() >= 0 and n.max() == g
    reach = 1.0
    for j in range(g + 1):
        sel = n >= j                      # position j was reached (all earlier drafts accepted)
        cnt = np.bincount(out[sel, j], minlength=V).astype(np.float64)
        m = sel.sum()
        np.testing.assert_allclose(m / N, reach, atol=4 * np.sqrt(reach * (1 - reach) / N) + 1e-9)
        sigma = np.sqrt(P[j] * (1 - P[j]) / m)
        assert np.all(np.abs(cnt / m - P[j]) <= 4.5 * sigma), (j, cnt / m, P[j])
        chi2 = ((cnt - m * P[j]) ** 2 / (m * P[j])).sum()
        assert chi2 < 30.0                # 5 degrees of freedom: P(chi2 > 30) ~ 1.5e-5
        if j < g:
            reach *= np.minimum(P[j], Q[j]).sum()
    # accepted prefix is copied verbatim, the tail is -1
    for j in range(g):
        assert np.all(out[n > j, j] == x[n > j, j])
        assert np.all(out[n < j, j] == -1)


def test_special_cases():
    rng = np.random.default_rng(2)
    V, g = 8, 4
    tl = rng.standard_normal((g + 1, V)).astype(np.float32)
    # p = q: always accepted (u < 1), bonus follows the CDF of P_gamma
    x = rng.integers(0, V, g)
    n, out = run1(tl, tl[:g].copy(), x, [0.999999] * g, 0.0)
    assert n == g and out[:g] == x.tolist() and out[g] == 0
    Pg = softmax(tl[g].astype(np.float64))
    c = np.cumsum(Pg)
    for u in (0.05, 0.3, 0.77, 0.999):
        n, out = run1(tl, tl[:g].copy(), x, [0.5] * g, u)
        assert out[g] == int(np.searchsorted(c, np.float64(np.float32(u)) * c[-1], side="right"))
    # draft one-hot on a token the target gives ~0: rejected at row 0, resample ~ P_0 restricted to t != x
    dl = np.full((g, V), -200.0, np.float32)
    dl[:, 3] = 0.0
    tl2 = tl.copy()
    tl2[:, 3] = -200.0
    n, out = run1(tl2, dl, [3] * g, [1e-6] * g, 0.4)
    assert n == 0 and out[1:] == [-1] * g and out[0] != 3
    P0 = softmax(tl2[0].astype(np.float64))
    c = np.cumsum(P0)
    assert out[0] == int(np.searchsorted(c, np.float64(np.float32(0.4)) * c[-1], side="right"))
    # u_acc = 0 accepts whenever P[x] > 0
    dl = (tl[:g] + 3 * rng.standard_normal((g, V))).astype(np.float32)
    n, _ = run1(tl, dl, x, [0.0] * g, 0.5)
    assert n == g
    # mid-chain rejection: rows before it accepted, emitted token never equals a token with P <= Q
    ua = [0.0, 0.0, 0.99999, 0.0]
    xs = [0, 1, int(np.argmax(softmax(dl[2].astype(np.float64)) - softmax(tl[2].astype(np.float64)))), 2]
    n, out = run1(tl, dl, xs, ua, 0.5)
    assert n == 2 and out[:2] == [0, 1] and out[3:] == [-1, -1]
    Pn, Qn = softmax(tl[2].astype(np.float64)), softmax(dl[2].astype(np.float64))
    assert Pn[out[2]] > Qn[out[2]]
    # gamma = 0: only the bonus token
    n, out, _, _ = oracle.accept(tl[None, :1], np.zeros((1, 0, V), np.float32), np.zeros((1, 0), np.int32),
                                 np.zeros((1, 0), np.float32), np.asarray([0.0], np.float32))
    assert n[0] == 0 and out.shape == (1, 1) and out[0, 0] == 0


def test_resample_sweep_reproduces_residual_cdf():
    rng = np.random.default_rng(4)
    V = 7
    tl = rng.standard_normal((2, V)).astype(np.float32)
    dl = rng.standard_normal((1, V)).astype(np.float32)
    P, Q = softmax(tl[0].astype(np.float64)), softmax(dl[0].astype(np.float64))
    x = int(np.argmax(Q - P))
    w = np.maximum(0.0, P - Q)
    us = (np.arange(2000) + 0.5) / 2000
    toks = np.array([run1(tl, dl, [x], [0.9999999], u)[1][0] for u in us])
    np.testing.assert_allclose(np.bincount(toks, minlength=V) / 2000, w / w.sum(), atol=1.5e-3)
    assert w[x] == 0 and not np.any(toks == x)


# ---- greedy verification (the decoding mode of the paper's experiments) ---------------------------------------------

def test_greedy_matches_library_argmax_and_hand_cases():
    rng = np.random.default_rng(5)
    B, g, V = 6, 4, 37
    tl = rng.standard_normal((B, g + 1, V)).astype(np.float32)
    am = tl.argmax(axis=-1).astype(np.int32)                 # numpy's arg-max: first maximum, an independent routine
    x = am[:, :g].copy()
    x[1, 0] = (x[1, 0] + 1) % V                              # first token wrong
    x[2, 2] = (x[2, 2] + 5) % V                              # third token wrong
    x[3, 3] = (x[3, 3] + 1) % V                              # last token wrong
    n, out = oracle.accept_greedy(tl, x)
    assert n.tolist() == [4, 0, 2, 3, 4, 4]
    for b in range(B):
        k = int(n[b])
        assert out[b, :k].tolist() == x[b, :k].tolist()      # kept draft tokens
        assert out[b, k] == am[b, k]                         # the target's own token at the first mismatch / bonus
        assert (out[b, k + 1:] == -1).all()


def test_greedy_ties_take_the_lowest_token_id():
    tl = np.zeros((1, 2, 9), np.float32)
    tl[0, 0, [3, 7]] = 2.0                                   # two equal maxima
    tl[0, 1, [8, 1]] = 5.0
    n, out = oracle.accept_greedy(tl, np.array([[3]], np.int32))
    assert n.tolist() == [1] and out.tolist() == [[3, 1]]
    n, out = oracle.accept_greedy(tl, np.array([[7]], np.int32))      # 7 ties with 3 but is not the arg-max
    assert n.tolist() == [0] and out.tolist() == [[3, -1]]


def test_greedy_is_the_zero_temperature_limit_of_the_sampling_rule():
    """With logits scaled until both softmaxes are one-hot, Eq. 1 accepts exactly the draft tokens that equal the
    target's arg-max and the residual puts all its mass on that arg-max: the sampling oracle (pinned above by the
    losslessness identity) and the greedy oracle must agree for every uniform."""
    rng = np.random.default_rng(11)
    B, g, V = 40, 5, 23
    tl = rng.standard_normal((B, g + 1, V)).astype(np.float32)
    dl = tl[:, :g].copy()
    flip = rng.random((B, g)) < 0.3
    dl[flip] = rng.standard_normal((int(flip.sum()), V)).astype(np.float32)   # some draft rows disagree
    x = dl.argmax(axis=-1).astype(np.int32)                 # greedy draft
    ua = rng.random((B, g), dtype=np.float32)
    ur = rng.random(B, dtype=np.float32)
    n_s, out_s, _, _ = oracle.accept(tl * 1e4, dl * 1e4, x, ua, ur)
    n_g, out_g = oracle.accept_greedy(tl, x)
    assert n_s.tolist() == n_g.tolist()
    assert out_s.tolist() == out_g.tolist()
    assert len(set(n_g.tolist())) >= 3


# ---- the two margins the oracle reports (the GPU parity test reads them to classify a disagreement) -----------------

def margins1(tl, dl, x, ua, ur):
    n, out, ma, mc = oracle.accept(tl[None], dl[None], np.asarray(x, np.int32)[None], np.asarray(ua, np.float32)[None],
                                   np.asarray([ur], np.float32))
    return int(n[0]), out[0].tolist(), float(ma[0]), float(mc[0])


def test_margins_on_cases_worked_by_hand():
    """V = 2 and V = 3 with probabilities that are quarters and halves (logits 0, ln 2, ln 3), so |u Q - P| / P and the
    distance of u_res Z to the chosen token's CDF edges over Z are numbers written out below."""
    ln2, ln3 = np.float32(np.log(2.0)), np.float32(np.log(3.0))
    # P_0 = (1/4, 3/4), Q_0 = (1/2, 1/2), bonus row P_1 = (1/4, 3/4)
    tl = np.array([[0, ln3], [0, ln3]], np.float32)
    dl = np.array([[0, 0]], np.float32)
    # x = 0, u = 1/4: u Q = 1/8 < 1/4 accepted, margin |1/8 - 1/4| / (1/4) = 1/2.  Bonus from P_1 with u_res = 1/2:
    # CDF edges 1/4, 1 -> token 1, distances 1/4 and 1/2, Z = 1 -> 1/4
    n, out, ma, mc = margins1(tl, dl, [0], [0.25], 0.5)
    assert (n, out) == (1, [0, 1])
    np.testing.assert_allclose([ma, mc], [0.5, 0.25], rtol=0, atol=1e-6)
    # x = 0, u = 3/4: u Q = 3/8 >= 1/4 rejected, margin (3/8 - 1/4) / (1/4) = 1/2.  Residual (0, 1/4), Z = 1/4,
    # u_res = 3/8 -> target 3/32 in token 1's interval (0, 1/4]: distances 3/32 and 5/32 -> (3/32) / (1/4) = 3/8
    n, out, ma, mc = margins1(tl, dl, [0], [0.75], 0.375)
    assert (n, out) == (0, [1, -1])
    np.testing.assert_allclose([ma, mc], [0.5, 0.375], rtol=0, atol=1e-6)
    # x = 1: P/Q = 3/2, always accepted; u = 1/2: |1/4 - 3/4| / (3/4) = 2/3.  Bonus with u_res = 1/8: token 0,
    # interval [0, 1/4): distances 1/8 and 1/8 -> 1/8
    n, out, ma, mc = margins1(tl, dl, [1], [0.5], 0.125)
    assert (n, out) == (1, [1, 0])
    np.testing.assert_allclose([ma, mc], [2.0 / 3.0, 0.125], rtol=0, atol=1e-6)
    # V = 3, two draft rows: the accept margin is the minimum over the tests made.  P = (1/2, 1/4, 1/4) in every row,
    # Q = (1/4, 1/4, 1/2).  Row 0: x = 2, u = 1/4: u Q = 1/8 < 1/4 accepted, margin 1/2.  Row 1: x = 2, u = 7/16:
    # u Q = 7/32 < 1/4 accepted, margin 1/8.  Bonus from P with u_res = 5/8: CDF 1/2, 3/4, 1 -> token 1,
    # distances 1/8 and 1/8 -> 1/8
    tl3 = np.array([[ln2, 0, 0]] * 3, np.float32)
    dl3 = np.array([[0, 0, ln2]] * 2, np.float32)
    n, out, ma, mc = margins1(tl3, dl3, [2, 2], [0.25, 0.4375], 0.625)
    assert (n, out) == (2, [2, 2, 1])
    np.testing.assert_allclose([ma, mc], [0.125, 0.125], rtol=0, atol=1e-6)
    # row 1 rejected instead (u = 3/4: u Q = 3/8 >= 1/4, margin 1/2): the minimum stays row 0's 1/2; the second row's
    # test is the last one made.  Residual (1/4, 0, 0), Z = 1/4, u_res = 1/2: token 0, distances 1/8 and 1/8 -> 1/2
    n, out, ma, mc = margins1(tl3, dl3, [2, 2], [0.25, 0.75], 0.5)
    assert (n, out) == (1, [2, 0, -1])
    np.testing.assert_allclose([ma, mc], [0.5, 0.5], rtol=0, atol=1e-6)
    # a rejection at row 0 makes no test at row 1: a uniform there that sits almost on its boundary must not show
    n, out, ma, mc = margins1(tl3, dl3, [2, 2], [0.75, 0.5], 0.5)
    assert n == 0
    np.testing.assert_allclose(ma, 0.5, rtol=0, atol=1e-6)


def test_margins_vanish_at_the_measured_decision_boundaries():
    """The accept margin at u is |u - u*| / u* for the boundary u* = P/Q that the oracle's own decisions flip at (located
    by bisection over fp32 uniforms), and the CDF margin is the distance of u_res to the nearer measured edge of the
    emitted token's interval: both go to zero there, and nowhere else."""
    rng = np.random.default_rng(21)
    V = 6
    tl = (rng.standard_normal((2, V)) * 1.5).astype(np.float32)
    dl = (rng.standard_normal((1, V)) * 1.5).astype(np.float32)
    P, Q = softmax(tl[0].astype(np.float64)), softmax(dl[0].astype(np.float64))
    x = int(np.argmax(Q / P))                     # a token the draft over-weights: P/Q < 1, the boundary is inside (0, 1)
    u_star = accept_measure(tl, dl, x)
    np.testing.assert_allclose(u_star, P[x] / Q[x], atol=1e-6)
    for u in (0.1 * u_star, 0.5 * u_star, 0.999 * u_star, 1.001 * u_star, min(0.999, 1.5 * u_star)):
        u32 = float(np.float32(u))
        _, _, ma, _ = margins1(tl, dl, [x], [u32], 0.5)
        np.testing.assert_allclose(ma, abs(u32 - u_star) / u_star, atol=2e-6)
    below, above = np.nextafter(np.float32(u_star), np.float32(0)), np.nextafter(np.float32(u_star), np.float32(1))
    assert margins1(tl, dl, [x], [below], 0.5)[2] < 1e-6 and margins1(tl, dl, [x], [above], 0.5)[2] < 1e-6
    # CDF margin after a rejection: edges of the residual distribution measured from the emitted tokens
    w = np.maximum(0.0, P - Q)
    edges = np.concatenate([[0.0], np.cumsum(w) / w.sum()])
    for u_res in (0.03, 0.2, 0.41, 0.77, 0.96):
        u32 = float(np.float32(u_res))
        n, out, _, mc = margins1(tl, dl, [x], [np.nextafter(np.float32(1), np.float32(0))], u32)
        assert n == 0
        t = out[0]
        assert edges[t] <= u32 < edges[t + 1]
        np.testing.assert_allclose(mc, min(u32 - edges[t], edges[t + 1] - u32), atol=1e-7)
    # approaching an interior edge from both sides
    e = float(edges[np.flatnonzero(w > 0)[0] + 1])
    if 0.0 < e < 1.0:
        for u_res in (np.float32(e) - np.float32(1e-6), np.float32(e) + np.float32(1e-6)):
            assert margins1(tl, dl, [x], [0.9999999], float(u_res))[3] < 3e-6
