"""Pins of the oracle's global-semantic-relevance score (Section 5.1, Eq. 2) against facts that do not come
from the oracle: a hand-worked case, closed forms, a library softmax, and invariants of the definition."""
import numpy as np
import pytest
from scipy.special import softmax

import oracle


def rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape).astype(np.float32)


def test_hand_worked_two_rows_two_keys():
    # one layer, one head, D = 1, scale 1.  Keys (0, ln 3).  Row q = 1: logits (0, ln 3) -> (1/4, 3/4);
    # row q = 0: logits (0, 0) -> (1/2, 1/2).  Mean over the two rows: (3/8, 5/8).
    q = np.array([1.0, 0.0], dtype=np.float32).reshape(1, 1, 2, 1, 1)
    k = np.array([0.0, np.log(3.0)], dtype=np.float32).reshape(1, 1, 2, 1, 1)
    m = oracle.attention_mass(q, k, [2], scale=1.0)
    # ln 3 is rounded to fp32 on input: 3/4 is reached to ~1e-8
    assert np.allclose(m[0], [0.375, 0.625], atol=2e-8)


def test_identical_keys_give_uniform_mass():
    q = rand((2, 1, 5, 4, 8), 1)
    k = np.broadcast_to(rand((2, 1, 1, 2, 8), 2), (2, 1, 37, 2, 8)).copy()
    m = oracle.attention_mass(q, k, [37])
    assert np.allclose(m[0], 1.0 / 37, rtol=0, atol=1e-15)


def test_mass_sums_to_one_and_is_zero_past_the_end():
    q = rand((3, 2, 6, 4, 16), 3)
    k = rand((3, 2, 50, 2, 16), 4)
    m = oracle.attention_mass(q, k, [50, 23])
    assert np.allclose(m.sum(axis=1), 1.0, atol=1e-13)
    assert np.all(m[1, 23:] == 0.0) and np.all(m[1, :23] > 0.0)


def test_matches_library_softmax_with_grouped_heads():
    nl, B, L, Hq, Hkv, D, nv = 2, 2, 7, 6, 2, 16, 41
    q = rand((nl, B, L, Hq, D), 5)
    k = rand((nl, B, nv, Hkv, D), 6)
    scale = 0.3
    kq = np.repeat(k.astype(np.float64), Hq // Hkv, axis=3)          # head h reads KV head h // G
    logits = scale * np.einsum("lbihd,lbjhd->lbhij", q.astype(np.float64), kq)
    ref = softmax(logits, axis=-1).mean(axis=(0, 2, 3))               # layers, heads, text rows
    m = oracle.attention_mass(q, k, [nv, nv], scale=scale)
    assert np.allclose(m, ref, rtol=1e-12, atol=1e-15)
    # the interleaved grouping (h % H_kv) is a different function on these inputs
    kq_wrong = np.tile(k.astype(np.float64), (1, 1, 1, Hq // Hkv, 1))
    wrong = softmax(scale * np.einsum("lbihd,lbjhd->lbhij", q.astype(np.float64), kq_wrong), axis=-1).mean(axis=(0, 2, 3))
    assert np.abs(wrong - ref).max() > 1e-4


def test_ragged_lengths_equal_separate_calls():
    nl, L, Hq, Hkv, D = 2, 4, 4, 2, 8
    q = rand((nl, 2, L, Hq, D), 7)
    k = rand((nl, 2, 30, Hkv, D), 8)
    both = oracle.attention_mass(q, k, [30, 11])
    one = oracle.attention_mass(q[:, 1:2], k[:, 1:2, :11], [11])
    assert np.array_equal(both[1, :11], one[0])


def test_dominant_key_takes_all_mass():
    q = np.ones((1, 1, 3, 2, 4), dtype=np.float32)
    k = np.zeros((1, 1, 9, 1, 4), dtype=np.float32)
    k[0, 0, 5] = 50.0     # logit 200 * scale above the rest
    m = oracle.attention_mass(q, k, [9], scale=1.0)
    assert m[0, 5] == pytest.approx(1.0, abs=1e-12) and m[0].sum() == pytest.approx(1.0, abs=1e-12)


def test_invariants_key_shift_scale_trade_and_layer_mean():
    nl, L, Hq, Hkv, D, nv = 2, 5, 4, 2, 8, 19
    q = rand((nl, 1, L, Hq, D), 9)
    k = rand((nl, 1, nv, Hkv, D), 10)
    base = oracle.attention_mass(q, k, [nv], scale=0.5)
    # adding one vector to every key shifts each row's logits by a constant
    shift = np.float32(0.25) * np.ones((1, 1, 1, 1, D), dtype=np.float32)
    assert np.allclose(oracle.attention_mass(q, k + shift, [nv], scale=0.5), base, rtol=1e-6)
    # scale and query magnitude trade off exactly (powers of two)
    assert np.array_equal(oracle.attention_mass(q * np.float32(2.0), k, [nv], scale=0.25), base)
    # the score over two layers is the mean of the per-layer scores
    l0 = oracle.attention_mass(q[:1], k[:1], [nv], scale=0.5)
    l1 = oracle.attention_mass(q[1:], k[1:], [nv], scale=0.5)
    assert np.allclose(base, 0.5 * (l0 + l1), rtol=1e-14)
    # a head whose queries are zero spreads its mass evenly whatever its keys are
    qz = q.copy(); qz[:, :, :, 2:] = 0.0
    k2 = k.copy(); k2[:, :, :, 1] = rand((nl, 1, nv, D), 11)
    assert np.allclose(oracle.attention_mass(qz, k, [nv]), oracle.attention_mass(qz, k2, [nv]), rtol=1e-13)
