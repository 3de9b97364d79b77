"""GPU parity: hippo_verify_attention / hippo_draft_attention (through the C ABI) against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import TOL, assert_close, dev, host, paged_cache
from paper_2601_08273_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def hb():
    from paper_2601_08273_b200 import binding
    return binding


def run_case(hb, fn, q, k, v, lens, dtype, shuffle_seed=None, num_splits=0, want_lse=True, fill=0.0, spare=0):
    kv, _, _ = paged_cache(hb, k, v, lens, dtype, shuffle_seed=shuffle_seed, fill=fill, spare=spare)
    qd = dev(q, dtype)
    kvl = dev(np.asarray(lens, np.int32))
    lse = torch.full(q.shape[:3], float("nan"), dtype=torch.float32, device="cuda") if want_lse else None
    out = fn(qd, kv, kvl, max(lens), num_splits=num_splits, lse=lse)
    torch.cuda.synchronize()
    return host(out), (None if lse is None else host(lse))


def check_full(hb, fn, q, k, v, lens, dtype, **kw):
    got, lse = run_case(hb, fn, q, k, v, lens, dtype, **kw)
    ref, ref_lse = oracle.attention(q, k, v, lens)
    assert_close(got, ref, TOL[dtype], "attention out")
    if lse is not None:
        assert_close(lse, ref_lse, TOL[dtype] if dtype == "fp32" else 2e-3, "lse")
    return got


def test_c0_verify_and_draft_fp32(hb):
    cfg = W.CONFIGS[0]
    n_v = W.visual_lengths(cfg)[0]
    q_len = cfg.gamma + 1
    lens = [n_v + cfg.n_text + q_len]
    inp = W.attention_inputs(cfg, "target", lens, q_len)
    check_full(hb, hb.hippo_verify_attention, inp["q"], inp["k"], inp["v"], lens, "fp32")
    # draft: pruned context (26 kept + 32 text) plus the tokens drafted so far, one query token
    for step in range(cfg.gamma):
        lens_d = [W.keep_count(n_v, cfg.keep_pct) + cfg.n_text + step + 1]
        inp = W.attention_inputs(cfg, "draft", lens_d, 1, layer=step)
        check_full(hb, hb.hippo_draft_attention, inp["q"], inp["k"], inp["v"], lens_d, "fp32")


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("D", [64, 128])
def test_ragged_batch_paged_several_tiles(hb, dtype, D):
    rng = np.random.default_rng(17)
    B, q_len, Hq, Hkv = 3, 6, 8, 2
    lens = [333, 6, 129]          # several tiles + ragged tail, kv_len == q_len, one key past a page boundary
    q = W.round_to_storage(rng.standard_normal((B, q_len, Hq, D)).astype(np.float32), dtype)
    k = W.round_to_storage(rng.standard_normal((B, max(lens), Hkv, D)).astype(np.float32), dtype)
    v = W.round_to_storage(rng.standard_normal((B, max(lens), Hkv, D)).astype(np.float32), dtype)
    a = check_full(hb, hb.hippo_verify_attention, q, k, v, lens, dtype, shuffle_seed=5, spare=3)
    # slots past each length hold NaN: they must never be read into a result
    b = check_full(hb, hb.hippo_verify_attention, q, k, v, lens, dtype, shuffle_seed=5, spare=3, fill=np.nan)
    np.testing.assert_array_equal(a, b)
    # different physical page order, same result bit for bit
    c = check_full(hb, hb.hippo_verify_attention, q, k, v, lens, dtype, shuffle_seed=6)
    np.testing.assert_array_equal(a, c)
    # split count does not matter beyond rounding
    for s in (1, 2, 5):
        check_full(hb, hb.hippo_verify_attention, q, k, v, lens, dtype, shuffle_seed=5, num_splits=s)
    check_full(hb, hb.hippo_draft_attention, q[:, :1], k, v, lens, dtype, shuffle_seed=5)


@pytest.mark.parametrize("rows", [(1, 7), (9, 8), (6, 7), (8, 4), (16, 8)])
def test_packed_row_shapes_bf16(hb, rows):
    q_len, G = rows
    rng = np.random.default_rng(q_len * 100 + G)
    Hkv, D, lens = 2, 128, [1000]
    q = W.round_to_storage(rng.standard_normal((1, q_len, Hkv * G, D)).astype(np.float32), "bf16")
    k = W.round_to_storage(rng.standard_normal((1, lens[0], Hkv, D)).astype(np.float32), "bf16")
    v = W.round_to_storage(rng.standard_normal((1, lens[0], Hkv, D)).astype(np.float32), "bf16")
    check_full(hb, hb.hippo_verify_attention, q, k, v, lens, "bf16")



@pytest.mark.parametrize("q_len,Hq,Hkv", [(6, 8, 2), (6, 14, 2), (9, 16, 2), (16, 16, 2)])
def test_reference_maxima_keep_growing(hb, q_len, Hq, Hkv):
    """Keys grow along the sequence, so that in tile after tile some scores exceed the rows' running maxima by far
    more than the lazy-rescale threshold: the rescale path (and the repeated probability sweep) runs mid-sequence,
    for 24, 42, 72 and 128 packed rows (with and without the spare row-sum columns, even and odd group counts)."""
    rng = np.random.default_rng(23)
    D, lens = 128, [1500, 700]
    q = W.round_to_storage(2.0 * rng.standard_normal((2, q_len, Hq, D)).astype(np.float32), "bf16")
    k = rng.standard_normal((2, max(lens), Hkv, D)).astype(np.float32)
    k *= (1.0 + 2.0 * (np.arange(max(lens)) // 100))[None, :, None, None]
    k[1, :, :, :] *= np.where(np.arange(max(lens)) % 257 == 0, 3.0, 1.0)[:, None, None]    # isolated spikes as well
    k = W.round_to_storage(k, "bf16")
    v = W.round_to_storage(rng.standard_normal((2, max(lens), Hkv, D)).astype(np.float32), "bf16")
    check_full(hb, hb.hippo_verify_attention, q, k, v, lens, "bf16", shuffle_seed=3)
    check_full(hb, hb.hippo_verify_attention, q, k, v, lens, "bf16", shuffle_seed=3, num_splits=3)


@pytest.mark.parametrize("D", [64, 128])
def test_more_units_than_sms(hb, D):
    """200 (sequence, kv head) units: more than one per SM, so CTAs walk several units and units straddle CTAs."""
    rng = np.random.default_rng(23)
    B, q_len, Hq, Hkv = 50, 3, 8, 4
    lens = [int(x) for x in rng.integers(q_len, 900, size=B)]
    lens[7], lens[8] = 1, 2                       # shorter than q_len: skipped, zero output
    q = W.round_to_storage(rng.standard_normal((B, q_len, Hq, D)).astype(np.float32), "bf16")
    k = W.round_to_storage(rng.standard_normal((B, max(lens), Hkv, D)).astype(np.float32), "bf16")
    v = W.round_to_storage(rng.standard_normal((B, max(lens), Hkv, D)).astype(np.float32), "bf16")
    got, lse = run_case(hb, hb.hippo_verify_attention, q, k, v, lens, "bf16", shuffle_seed=9)
    live = [b for b in range(B) if lens[b] >= q_len]
    ref, ref_lse = oracle.attention(q[live], k[live], v[live], [lens[b] for b in live])
    assert_close(got[live], ref, TOL["bf16"], "many units")
    assert_close(lse[live], ref_lse, 2e-3, "many units lse")
    assert np.all(got[7:9] == 0) and np.all(np.isneginf(lse[7:9]))


def test_short_sequence_is_skipped_and_zeroed(hb):
    rng = np.random.default_rng(3)
    B, q_len, Hq, Hkv, D = 2, 4, 4, 2, 64
    lens = [2, 70]               # first sequence shorter than q_len
    q = rng.standard_normal((B, q_len, Hq, D)).astype(np.float32)
    k = rng.standard_normal((B, 70, Hkv, D)).astype(np.float32)
    v = rng.standard_normal((B, 70, Hkv, D)).astype(np.float32)
    got, lse = run_case(hb, hb.hippo_verify_attention, q, k, v, lens, "fp32", shuffle_seed=1)
    assert np.all(got[0] == 0) and np.all(np.isneginf(lse[0]))
    ref, _ = oracle.attention(q[1:], k[1:], v[1:], lens[1:])
    assert_close(got[1:], ref, 1e-5)


def test_short_sequence_in_a_bf16_batch(hb):
    """bf16 path, few units (one cluster or one group of CTAs per unit): a sequence shorter than q_len gives zeros."""
    rng = np.random.default_rng(4)
    B, q_len, Hq, Hkv, D = 3, 4, 8, 2, 128
    lens = [700, 3, 260]
    q = W.round_to_storage(rng.standard_normal((B, q_len, Hq, D)).astype(np.float32), "bf16")
    k = W.round_to_storage(rng.standard_normal((B, max(lens), Hkv, D)).astype(np.float32), "bf16")
    v = W.round_to_storage(rng.standard_normal((B, max(lens), Hkv, D)).astype(np.float32), "bf16")
    for splits in (0, 3):
        got, lse = run_case(hb, hb.hippo_verify_attention, q, k, v, lens, "bf16", shuffle_seed=2, num_splits=splits)
        assert np.all(got[1] == 0) and np.all(np.isneginf(lse[1]))
        ref, _ = oracle.attention(q[[0, 2]], k[[0, 2]], v[[0, 2]], [lens[0], lens[2]])
        assert_close(got[[0, 2]], ref, TOL["bf16"], "neighbours of a skipped sequence")


def sampled_rows(rng, B, q_len, Hq, n):
    rows = {(0, 0, 0), (B - 1, q_len - 1, Hq - 1)}
    while len(rows) < n:
        rows.add((int(rng.integers(B)), int(rng.integers(q_len)), int(rng.integers(Hq))))
    return sorted(rows)


@pytest.mark.parametrize("ci", [1, 2, 4])
def test_full_size_verify(hb, ci):
    """The verification shapes at full size.  Every (token, head) row is compared with the oracle at c1, c2 and at the
    64k configuration's largest gamma; its other two gammas compare 48 sampled rows."""
    cfg = W.CONFIGS[ci]
    n_v = W.visual_lengths(cfg)[0]
    gammas = W.C4_GAMMA_SWEEP if ci == 4 else (cfg.gamma,)
    for g in gammas:
        q_len = g + 1
        lens = [n_v + cfg.n_text + q_len]
        inp = W.attention_inputs(cfg, "target", lens, q_len)
        got, lse = run_case(hb, hb.hippo_verify_attention, inp["q"], inp["k"], inp["v"], lens, cfg.dtype)
        assert np.isfinite(got).all()
        if ci != 4 or g == max(gammas):
            ref, ref_lse = oracle.attention(inp["q"], inp["k"], inp["v"], lens)
            assert_close(got, ref, TOL[cfg.dtype], "c%d gamma %d, all rows" % (ci, g))
            assert_close(lse, ref_lse, 2e-3, "lse")
            continue
        rows = sampled_rows(np.random.default_rng(ci), 1, q_len, cfg.tgt_q_heads, 48)
        ref, ref_lse = oracle.attention(inp["q"], inp["k"], inp["v"], lens, rows=rows)
        sel = np.array(rows)
        assert_close(got[sel[:, 0], sel[:, 1], sel[:, 2]], ref, TOL[cfg.dtype], "c%d gamma %d" % (ci, g))
        assert_close(lse[sel[:, 0], sel[:, 1], sel[:, 2]], ref_lse, 2e-3, "lse")


def test_c3_batched_paged_verify_and_draft(hb):
    cfg = W.CONFIGS[3]
    q_len = cfg.gamma + 1
    n_vs = W.visual_lengths(cfg)
    lens = [n + cfg.n_text + q_len for n in n_vs]
    inp = W.attention_inputs(cfg, "target", lens, q_len)
    got, _ = run_case(hb, hb.hippo_verify_attention, inp["q"], inp["k"], inp["v"], lens, cfg.dtype, shuffle_seed=33)
    ref, _ = oracle.attention(inp["q"], inp["k"], inp["v"], lens)       # all 8 x 6 x 28 rows
    assert_close(got, ref, TOL[cfg.dtype], "c3 verify")
    lens_d = [W.keep_count(n, cfg.keep_pct) + cfg.n_text + 1 for n in n_vs]
    inp = W.attention_inputs(cfg, "draft", lens_d, 1)
    got, _ = run_case(hb, hb.hippo_draft_attention, inp["q"], inp["k"], inp["v"], lens_d, cfg.dtype, shuffle_seed=34)
    ref, _ = oracle.attention(inp["q"], inp["k"], inp["v"], lens_d)
    assert_close(got, ref, TOL[cfg.dtype], "c3 draft")


@pytest.mark.parametrize("ci", [1, 2, 4])
def test_full_size_draft(hb, ci):
    cfg = W.CONFIGS[ci]
    n_v = W.visual_lengths(cfg)[0]
    pcts = W.C4_KEEP_PCT_SWEEP if ci == 4 else (cfg.keep_pct,)
    for pct in pcts:
        lens = [W.keep_count(n_v, pct) + cfg.n_text + cfg.gamma]
        inp = W.attention_inputs(cfg, "draft", lens, 1)
        got, _ = run_case(hb, hb.hippo_draft_attention, inp["q"], inp["k"], inp["v"], lens, cfg.dtype)
        ref, _ = oracle.attention(inp["q"], inp["k"], inp["v"], lens)
        assert_close(got, ref, TOL[cfg.dtype], "c%d draft keep %d%%" % (ci, pct))


@pytest.mark.parametrize("dtype,q_len,kvl", [("bf16", 6, 700), ("bf16", 1, 500), ("fp32", 3, 200)])
def test_lengths_known_on_the_host(hb, dtype, q_len, kvl):
    """kv_len = NULL: every sequence has max_kv_len keys; same result as with the length array."""
    rng = np.random.default_rng(31)
    B, Hq, Hkv, D = 2, 8, 2, 64
    lens = [kvl, kvl]
    q = W.round_to_storage(rng.standard_normal((B, q_len, Hq, D)).astype(np.float32), dtype)
    k = W.round_to_storage(rng.standard_normal((B, kvl, Hkv, D)).astype(np.float32), dtype)
    v = W.round_to_storage(rng.standard_normal((B, kvl, Hkv, D)).astype(np.float32), dtype)
    kv, _, _ = paged_cache(hb, k, v, lens, dtype, shuffle_seed=2)
    with_array = host(hb.hippo_verify_attention(dev(q, dtype), kv, dev(np.asarray(lens, np.int32)), kvl))
    without = host(hb.hippo_verify_attention(dev(q, dtype), kv, None, kvl))
    draft = host(hb.hippo_draft_attention(dev(q, dtype), kv, None, kvl))
    torch.cuda.synchronize()
    np.testing.assert_array_equal(with_array, without)
    ref, _ = oracle.attention(q, k, v, lens)
    assert_close(without, ref, TOL[dtype], "host lengths")
    assert_close(draft, ref, TOL[dtype], "host lengths, draft")


def test_workspace_status_is_clean(hb):
    ws = hb.new_workspace(hb.hippo_attention_workspace_bytes(1, 2, 4, 2, 64))
    rng = np.random.default_rng(0)
    q = dev(rng.standard_normal((1, 2, 4, 64)).astype(np.float32), "bf16")
    k = rng.standard_normal((1, 100, 2, 64)).astype(np.float32)
    kv, _, _ = paged_cache(hb, k, k, [100], "bf16")
    hb.hippo_verify_attention(q, kv, dev(np.asarray([100], np.int32)), 100, workspace=ws)
    assert hb.hippo_workspace_status(ws) == hb.HIPPO_OK


def test_same_bits_on_repeated_calls(hb):
    """Full long-video shape: the result does not depend on timing (which CTA finishes first, what ran before)."""
    cfg = W.CONFIGS[2]
    q_len = cfg.gamma + 1
    lens = [W.visual_lengths(cfg)[0] + cfg.n_text + q_len]
    inp = W.attention_inputs(cfg, "target", lens, q_len)
    kv, _, _ = paged_cache(hb, inp["k"], inp["v"], lens, "bf16")
    qd, kvl = dev(inp["q"], "bf16"), dev(np.asarray(lens, np.int32))
    ws = hb.new_workspace(hb.hippo_attention_workspace_bytes(1, q_len, cfg.tgt_q_heads, cfg.tgt_kv_heads, cfg.tgt_head_dim))
    outs = []
    for rep in range(3):
        if rep:
            torch.randn(1 << 24, device="cuda").sum().item()      # disturb caches and clocks in between
        outs.append(host(hb.hippo_verify_attention(qd, kv, kvl, lens[0], workspace=ws)).copy())
    np.testing.assert_array_equal(outs[0], outs[1])
    np.testing.assert_array_equal(outs[0], outs[2])
    assert hb.hippo_workspace_status(ws) == 0
