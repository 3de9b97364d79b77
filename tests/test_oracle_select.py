"""Pins for the oracle's selection (Eq. 3-7 and the top-k rule): closed forms, invariants, a hand-worked
case and library routines.  CPU only."""
import os

import numpy as np
import pytest

import oracle
from paper_2601_08273_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "select_hand_worked.txt")


def unit(angle_units):
    a = np.asarray(angle_units, dtype=np.float64) * (np.pi / 4)
    return np.stack([np.cos(a), np.sin(a)], axis=-1).astype(np.float32)


def test_hand_worked_case_matches_golden():
    rows = [l.split() for l in open(GOLDEN) if l.strip() and not l.startswith("#")]
    ang = [int(r[2]) for r in rows]
    mass = np.array([float(r[3]) for r in rows], dtype=np.float32)
    want_t, want_s, want_f = (np.array([float(r[c]) for r in rows]) for c in (4, 5, 6))
    fused, st, ss = oracle.select_scores(unit(ang), mass, 2, 2, 2, 2)
    # the unit vectors are rounded to fp32, so agreement is to ~1e-7, not to the 10 printed digits
    np.testing.assert_allclose(st, want_t, atol=5e-7)
    np.testing.assert_allclose(ss, want_s, atol=5e-7)
    np.testing.assert_allclose(fused, want_f, atol=5e-6)
    idx, kth = oracle.topk(fused, 2)
    assert idx.tolist() == [3, 4]
    assert abs(kth - 1.4797164608) < 5e-6


def test_spatial_closed_forms():
    # one frame, 5x5 grid, one 5x5 crop (M = 25)
    M, d = 25, 32
    ortho = np.zeros((M, d), dtype=np.float32)
    ortho[np.arange(M), np.arange(M)] = np.linspace(0.5, 3.0, M)  # mutually orthogonal, different norms
    mass = np.full(M, 1.0 / M, dtype=np.float32)
    _, _, ss = oracle.select_scores(ortho, mass, 5, 5)
    np.testing.assert_allclose(ss, (M - 1) / M**2, rtol=0, atol=1e-15)  # S = I  ->  (M-1)/M^2 = 0.0384
    same = np.tile(np.arange(1, d + 1, dtype=np.float32), (M, 1)) * np.linspace(1, 2, M, dtype=np.float32)[:, None]
    _, _, ss = oracle.select_scores(same, mass, 5, 5)
    np.testing.assert_allclose(ss, 0.0, atol=1e-14)  # all tokens parallel -> S = 1 everywhere -> variance 0


def test_spatial_clipped_crops_use_their_own_M():
    # 8x8 grid with 5x5 crops -> crops of 25, 15, 15 and 9 tokens; orthogonal tokens inside every crop
    gh = gw = 8
    d = 64
    E = np.zeros((gh * gw, d), dtype=np.float32)
    E[np.arange(64), np.arange(64)] = 1.0
    _, _, ss = oracle.select_scores(E, np.full(64, 1 / 64, np.float32), gh, gw)
    ss = ss.reshape(gh, gw)
    for (ys, xs, M) in ((slice(0, 5), slice(0, 5), 25), (slice(0, 5), slice(5, 8), 15),
                        (slice(5, 8), slice(0, 5), 15), (slice(5, 8), slice(5, 8), 9)):
        np.testing.assert_allclose(ss[ys, xs], (M - 1) / M**2, atol=1e-15)
    # 16x16 grid: the last crop column/row is 1 wide; the corner crop has a single token -> s_spa = 0
    E = np.zeros((256, 256), dtype=np.float32)
    E[np.arange(256), np.arange(256)] = 1.0
    _, _, ss = oracle.select_scores(E, np.full(256, 1 / 256, np.float32), 16, 16)
    ss = ss.reshape(16, 16)
    assert ss[15, 15] == 0.0
    np.testing.assert_allclose(ss[0:5, 15], 4 / 25, atol=1e-15)  # 5x1 crop, M = 5
    np.testing.assert_allclose(ss[0:5, 0:5], 24 / 625, atol=1e-15)


def test_temporal_closed_forms():
    # 3 frames of a 1x2 grid; cell 0: f1 = f0, f2 = -f1; cell 1: all mutually orthogonal
    d = 4
    e = np.eye(d, dtype=np.float32)
    E = np.stack([3 * e[0], e[1],      # frame 0
                  5 * e[0], e[2],      # frame 1
                  -2 * e[0], e[3]])    # frame 2
    _, st, _ = oracle.select_scores(E, np.full(6, 1 / 6, np.float32), 1, 2, 1, 2)
    # cell 0: frame0 has one neighbour (cos 1) -> 0; frame1: mean(1, -1) = 0 -> 1; frame2: cos -1 -> 2
    np.testing.assert_allclose(st[[0, 2, 4]], [0.0, 1.0, 2.0], atol=1e-15)
    np.testing.assert_allclose(st[[1, 3, 5]], 1.0, atol=1e-15)  # orthogonal -> 1
    # a single frame has no neighbour: s' = 0 -> s_temp = 1
    _, st, _ = oracle.select_scores(E[:2], np.full(2, 0.5, np.float32), 1, 2, 1, 2)
    np.testing.assert_allclose(st, 1.0, atol=0)


def test_partial_last_frame_neighbours_and_stats():
    # 2x2 grid, 3 frames, last frame has a single token: cells 1..3 of frame 1 have only frame 0 as neighbour
    rng = np.random.default_rng(5)
    E = rng.standard_normal((9, 8)).astype(np.float32)
    E[4:8] = E[0:4]          # frame 1 = frame 0
    E[8] = -E[4]             # frame 2 cell 0 = -frame 1 cell 0
    mass = rng.random(9).astype(np.float32)
    fused, st, ss = oracle.select_scores(E, mass, 2, 2, 2, 2)
    np.testing.assert_allclose(st[0:4], 0.0, atol=1e-15)
    np.testing.assert_allclose(st[4], 1.0, atol=1e-15)       # mean(cos 1, cos -1) = 0
    np.testing.assert_allclose(st[5:8], 0.0, atol=1e-15)     # only frame 0 contains these cells
    np.testing.assert_allclose(st[8], 2.0, atol=1e-15)
    assert ss[8] == 0.0                                       # single-token crop
    assert fused[8] == 0.0                                    # single-token frame: every standardised score is 0


def test_identical_embeddings_reduce_to_standardised_attention():
    cfg = W.CONFIGS[0]
    n = 256
    E = np.tile(np.linspace(-1, 1, 16, dtype=np.float32), (n, 1))
    mass = W.attention_mass(cfg, n)
    fused, st, ss = oracle.select_scores(E, mass, 8, 8)
    np.testing.assert_allclose(st, 0.0, atol=1e-14)
    np.testing.assert_allclose(ss, 0.0, atol=1e-14)
    m = mass.astype(np.float64).reshape(4, 64)
    z = (m - m.mean(axis=1, keepdims=True)) / m.std(axis=1, keepdims=True)  # numpy's population std
    np.testing.assert_allclose(fused, z.reshape(-1), rtol=1e-12, atol=1e-12)


def test_attention_only_single_frame_is_plain_topk():
    rng = np.random.default_rng(11)
    n = 64
    E = rng.standard_normal((n, 8)).astype(np.float32)
    mass = rng.random(n).astype(np.float32)
    idx, fused, _ = oracle.select_tokens(E, mass, 9, 8, 8, score_mask=1)
    want = np.sort(np.argsort(-mass.astype(np.float64), kind="stable")[:9])
    assert idx.tolist() == want.tolist()


def test_invariants():
    cfg = W.CONFIGS[0]
    inp = W.select_inputs(cfg)
    E, mass = inp["embeds"], inp["attn_mass"]
    fused, st, ss = oracle.select_scores(E, mass, 8, 8)
    # positive rescaling of any embedding changes nothing (cosines only)
    scale = np.exp2(np.random.default_rng(1).integers(-3, 4, size=(256, 1))).astype(np.float32)
    f2, st2, ss2 = oracle.select_scores(E * scale, mass, 8, 8)
    np.testing.assert_allclose(st2, st, atol=1e-13)
    np.testing.assert_allclose(ss2, ss, atol=1e-13)
    np.testing.assert_allclose(f2, fused, atol=1e-9)
    # per-frame affine change (positive slope) of the attention mass changes nothing; masses are first
    # quantised to multiples of 2^-20 so that the transformed values stay exact in fp32
    mq = np.round(mass.astype(np.float64) * 2**20) / 2**20
    m2 = mq.reshape(4, 64) * np.array([[1.0], [2.0], [0.5], [4.0]]) + np.array([[0.0], [1.0], [2.0], [0.25]]) / 1024
    assert np.all(m2.astype(np.float32).astype(np.float64) == m2)
    fa, _, _ = oracle.select_scores(E, mq.astype(np.float32), 8, 8, score_mask=1)
    fb, _, _ = oracle.select_scores(E, m2.reshape(-1).astype(np.float32), 8, 8, score_mask=1)
    np.testing.assert_allclose(fb, fa, atol=1e-11)
    # each standardised score type has mean 0 and mean square 1 in every frame
    for mask in (1, 2, 4):
        z, _, _ = oracle.select_scores(E, mass, 8, 8, score_mask=mask)
        z = z.reshape(4, 64)
        np.testing.assert_allclose(z.mean(axis=1), 0.0, atol=1e-12)
        np.testing.assert_allclose((z**2).mean(axis=1), 1.0, atol=1e-12)
    # the three masks add up (Eq. 7)
    parts = sum(oracle.select_scores(E, mass, 8, 8, score_mask=m)[0] for m in (1, 2, 4))
    np.testing.assert_allclose(parts, fused, atol=1e-12)
    # reversing the frame order permutes s_spa and z(attn) and leaves s_temp per token unchanged
    perm = np.arange(256).reshape(4, 64)[::-1].reshape(-1)
    _, st3, ss3 = oracle.select_scores(E[perm], mass[perm], 8, 8)
    np.testing.assert_allclose(ss3, ss[perm], atol=1e-15)
    np.testing.assert_allclose(st3, st[perm], atol=1e-15)


def test_scores_against_numpy_matrix_form():
    # Eq. 5 as a library matrix product on normalised rows, Eq. 6 as numpy's population variance.
    cfg = W.CONFIGS[0]
    inp = W.select_inputs(cfg)
    E = inp["embeds"].astype(np.float64)
    _, st, ss = oracle.select_scores(inp["embeds"], inp["attn_mass"], 8, 8)
    Eh = E / np.linalg.norm(E, axis=1, keepdims=True)
    G = Eh.reshape(4, 8, 8, -1)
    want = np.zeros((4, 8, 8))
    for f in range(4):
        for ys in (slice(0, 5), slice(5, 8)):
            for xs in (slice(0, 5), slice(5, 8)):
                X = G[f, ys, xs].reshape(-1, E.shape[1])
                S = X @ X.T
                np.fill_diagonal(S, 1.0)
                want[f, ys, xs] = S.var(axis=1).reshape(want[f, ys, xs].shape)
    np.testing.assert_allclose(ss, want.reshape(-1), rtol=1e-10, atol=1e-14)
    Ef = Eh.reshape(4, 64, -1)
    cos = np.einsum("fcd,fcd->fc", Ef[:-1], Ef[1:])  # cos between frame f and f+1
    sp = np.zeros((4, 64))
    sp[0], sp[3] = cos[0], cos[2]
    sp[1], sp[2] = (cos[0] + cos[1]) / 2, (cos[1] + cos[2]) / 2
    np.testing.assert_allclose(st, (1 - sp).reshape(-1), rtol=1e-10, atol=1e-13)


def test_topk_ties_and_order():
    s = np.array([1.0, 3.0, 3.0, 2.0, 3.0, 0.5])
    idx, kth = oracle.topk(s, 2)
    assert idx.tolist() == [1, 2] and kth == 3.0   # equal scores: lower index wins
    idx, kth = oracle.topk(s, 4)
    assert idx.tolist() == [1, 2, 3, 4] and kth == 2.0
    assert oracle.topk(s, 0)[0].tolist() == []
    assert oracle.topk(s, 6)[0].tolist() == [0, 1, 2, 3, 4, 5]
    rng = np.random.default_rng(3)
    s = rng.standard_normal(5000)
    idx, kth = oracle.topk(s, 500)
    want = np.sort(np.argsort(-s, kind="stable")[:500])
    assert idx.tolist() == want.tolist() and kth == np.sort(s)[-500]
    with pytest.raises(ValueError):
        oracle.topk(s, 5001)


def test_config0_keep_count_and_boundary_share():
    cfg = W.CONFIGS[0]
    inp = W.select_inputs(cfg)
    assert inp["k"] == 26
    assert [W.keep_count(n, 10) for n in (6272, 32768, 65536)] == [627, 3277, 6554]
    idx, fused, kth = oracle.select_tokens(inp["embeds"], inp["attn_mass"], inp["k"], 8, 8)
    assert len(idx) == 26 and np.all(np.diff(idx) > 0)
    assert np.all(fused[idx] >= kth) and np.sum(fused > kth) <= 26


# ---- the other selection rules (uniform per-frame budget, random keys, whole frames) --------------------------------

def test_policy_per_frame_budgets_and_in_frame_order():
    """Uniform pruning across frames: budgets worked by hand, and inside each frame numpy's stable arg-sort."""
    rng = np.random.default_rng(31)
    T = 12
    # 5 complete frames, k = 17: 17 // 5 = 3 each, the first 17 % 5 = 2 frames one more
    s = rng.standard_normal(5 * T)
    kept, budget = oracle.select_policy(oracle.POLICY_UNIFORM_PER_FRAME, s, 17, T)
    assert budget.tolist() == [4, 4, 3, 3, 3]
    want = np.concatenate([f * T + np.sort(np.argsort(-s[f * T:(f + 1) * T], kind="stable")[:budget[f]]) for f in range(5)])
    assert kept.tolist() == want.tolist()
    assert np.all(np.diff(kept) > 0)
    # k divisible by the frame count: the same share everywhere; k = 0; k = n keeps everything
    assert oracle.select_policy(1, s, 20, T)[1].tolist() == [4] * 5
    assert oracle.select_policy(1, s, 0, T)[0].size == 0
    assert oracle.select_policy(1, s, 5 * T, T)[0].tolist() == list(range(5 * T))
    # a partial last frame of 2 tokens with k = 16 over 4 frames: 4 each, the last can give 2, the shortfall of 2 goes
    # to frames 0 and 1 in order
    s2 = rng.standard_normal(3 * T + 2)
    kept, budget = oracle.select_policy(1, s2, 16, T)
    assert budget.tolist() == [5, 5, 4, 2]
    assert kept[-2:].tolist() == [3 * T, 3 * T + 1]
    # shortfall larger than one round: frames 0..2 of 12, a partial frame of 1 token, k = 34 -> 9, 9, 8, 8 wanted;
    # the last gives 1, 7 missing: +1 each to frames 0, 1, 2 twice (12 = full for none yet), then +1 to frame 0
    s3 = rng.standard_normal(3 * T + 1)
    assert oracle.select_policy(1, s3, 34, T)[1].tolist() == [12, 11, 10, 1]
    # one frame: the per-frame rule is the global rule
    one = rng.standard_normal(T)
    assert oracle.select_policy(1, one, 5, T)[0].tolist() == oracle.select_policy(0, one, 5, T)[0].tolist()
    # ties inside a frame: the lowest indices win
    flat = np.zeros(2 * T)
    assert oracle.select_policy(1, flat, 6, T)[0].tolist() == [0, 1, 2, T, T + 1, T + 2]


def test_policy_random_is_the_top_k_of_the_callers_keys():
    rng = np.random.default_rng(32)
    keys = rng.random(500).astype(np.float32)
    keys[[7, 300]] = keys[11]                                           # equal keys: the lower index first
    for k in (0, 1, 50, 499, 500):
        kept, _ = oracle.select_policy(oracle.POLICY_RANDOM, keys, k, 25)
        want = np.sort(np.lexsort((np.arange(500), -keys.astype(np.float64)))[:k])
        assert kept.tolist() == want.tolist()


def test_policy_whole_frames_at_a_regular_stride():
    T = 4
    none = np.zeros(8 * T)
    # 8 frames, keep 2 whole frames: frames 0 and 4; keep 4: frames 0, 2, 4, 6
    assert oracle.select_policy(oracle.POLICY_FRAME, none, 2 * T, T)[0].tolist() == [0, 1, 2, 3, 16, 17, 18, 19]
    kept = oracle.select_policy(3, none, 4 * T, T)[0]
    assert sorted(set((kept // T).tolist())) == [0, 2, 4, 6] and kept.size == 16
    # 3 frames out of 8: floor(i * 8 / 3) = 0, 2, 5
    assert sorted(set((oracle.select_policy(3, none, 3 * T, T)[0] // T).tolist())) == [0, 2, 5]
    # k not a multiple of the frame size: ceil(10 / 4) = 3 frames 0, 2, 5, the last one cut to its first 2 cells
    assert oracle.select_policy(3, none, 10, T)[0].tolist() == [0, 1, 2, 3, 8, 9, 10, 11, 20, 21]
    # every complete frame and more: a prefix of the sequence (partial last frame of 3 cells)
    part = np.zeros(2 * T + 3)
    assert oracle.select_policy(3, part, 2 * T + 1, T)[0].tolist() == list(range(9))
    assert oracle.select_policy(3, part, 5, T)[0].tolist() == [0, 1, 2, 3, 4]      # ceil(5/4) = 2 frames of 2: 0 and 1, second cut
    # no complete frame at all
    assert oracle.select_policy(3, np.zeros(3), 2, T)[0].tolist() == [0, 1]
    # ascending, exactly k, for a sweep
    for k in range(0, 8 * T + 1):
        kept = oracle.select_policy(3, none, k, T)[0]
        assert kept.size == k and np.all(np.diff(kept) > 0)
