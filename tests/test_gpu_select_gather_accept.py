"""GPU parity: hippo_select_tokens, hippo_gather_kv and hippo_accept (through the C ABI) against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import dev, host
from paper_2601_08273_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def hb():
    from paper_2601_08273_b200 import binding
    return binding


# ---- selection ----------------------------------------------------------------------------------------------------

def check_kept(got_idx, got_fused, ref_idx, ref_fused, kth, what):
    """Kept sets must agree bit for bit, except for tokens whose oracle score lies within 1e-6 (relative) of the
    k-th threshold; the fused scores agree to fp32 rounding."""
    np.testing.assert_allclose(got_fused, ref_fused, rtol=0, atol=2e-6, err_msg=what)
    assert len(got_idx) == len(ref_idx), what
    assert np.all(np.diff(got_idx) > 0), what + ": not ascending / duplicates"
    diff = np.setxor1d(got_idx, ref_idx)
    if diff.size:
        band = np.abs(ref_fused[diff] - kth) <= 1e-6 * abs(kth)
        assert band.all(), "%s: %d kept-set differences outside the near-tie band" % (what, (~band).sum())


def run_select(hb, embeds_list, mass_list, ks, cfg, dtype, mask=7, crop=(5, 5)):
    n_visual = [e.shape[0] for e in embeds_list]
    E = dev(np.concatenate(embeds_list, axis=0), dtype)
    m = dev(np.concatenate(mass_list))
    kept, fused = hb.hippo_select_tokens(E, m, n_visual, ks, cfg.grid_h, cfg.grid_w, crop[0], crop[1], score_mask=mask)
    torch.cuda.synchronize()
    kept, fused = host(kept), host(fused)
    out, ko, so = [], 0, 0
    for n, k in zip(n_visual, ks):
        out.append((kept[ko:ko + k], fused[so:so + n]))
        ko, so = ko + k, so + n
    return out


@pytest.mark.parametrize("mask", [7, 1, 2, 4, 6])
def test_c0_select(hb, mask):
    cfg = W.CONFIGS[0]
    inp = W.select_inputs(cfg)
    (kept, fused), = run_select(hb, [inp["embeds"]], [inp["attn_mass"]], [inp["k"]], cfg, "fp32", mask=mask)
    ref_idx, ref_fused, kth = oracle.select_tokens(inp["embeds"], inp["attn_mass"], inp["k"], 8, 8, score_mask=mask)
    check_kept(kept, fused, ref_idx, ref_fused, kth, "c0 mask %d" % mask)
    if mask == 7:
        assert kept.tolist() == ref_idx.tolist()


def test_select_partial_frame_ragged_batch_bf16(hb):
    cfg = W.CONFIGS[3].replace(embed_dim=256)
    lens = [14 * 14 * 3 + 57, 14 * 14 * 2, 14 * 14 + 1, 9]
    embeds = [W.select_inputs(cfg, b, n)["embeds"] for b, n in enumerate(lens)]
    masses = [W.attention_mass(cfg, n, b) for b, n in enumerate(lens)]
    ks = [W.keep_count(n, 10) for n in lens]
    got = run_select(hb, embeds, masses, ks, cfg, "bf16")
    for b, (kept, fused) in enumerate(got):
        ref_idx, ref_fused, kth = oracle.select_tokens(embeds[b], masses[b], ks[b], 14, 14)
        check_kept(kept, fused, ref_idx, ref_fused, kth, "seq %d" % b)


def test_select_ties_lowest_index_wins(hb):
    cfg = W.CONFIGS[0]
    n = 256
    E = np.tile(np.linspace(-1, 1, 64, dtype=np.float32), (n, 1))     # identical embeddings: only attention matters
    mass = np.tile(np.array([4, 1, 4, 2, 4, 4, 1, 3], np.float32), n // 8) / 1000
    for k in (0, 1, 5, 100, 128, 129, 256):
        (kept, fused), = run_select(hb, [E], [mass], [k], cfg, "fp32")
        ref_idx, ref_fused, kth = oracle.select_tokens(E, mass, k, 8, 8)
        assert kept.tolist() == ref_idx.tolist(), k


@pytest.mark.parametrize("ci", [1, 2])
def test_full_size_select(hb, ci):
    cfg = W.CONFIGS[ci]
    inp = W.select_inputs(cfg)
    (kept, fused), = run_select(hb, [inp["embeds"]], [inp["attn_mass"]], [inp["k"]], cfg, cfg.dtype)
    ref_idx, ref_fused, kth = oracle.select_tokens(inp["embeds"], inp["attn_mass"], inp["k"], cfg.grid_h, cfg.grid_w)
    check_kept(kept, fused, ref_idx, ref_fused, kth, cfg.name)


def test_c3_batched_select(hb):
    cfg = W.CONFIGS[3]
    lens = W.visual_lengths(cfg)
    inps = [W.select_inputs(cfg, b) for b in range(cfg.batch)]
    ks = [i["k"] for i in inps]
    got = run_select(hb, [i["embeds"] for i in inps], [i["attn_mass"] for i in inps], ks, cfg, "bf16")
    for b in range(cfg.batch):
        ref_idx, ref_fused, kth = oracle.select_tokens(inps[b]["embeds"], inps[b]["attn_mass"], ks[b], 14, 14)
        check_kept(got[b][0], got[b][1], ref_idx, ref_fused, kth, "c3 seq %d" % b)


def test_c4_select_whole_sequence(hb):
    """Full c4 shape (65,536 tokens, d = 8192): the oracle scores the whole sequence once; for every kept share of the
    sweep (50 / 25 / 10 / 5 %) the GPU's fused scores and kept set are compared with it under the near-tie rule."""
    cfg = W.CONFIGS[4]
    inp = W.select_inputs(cfg)
    E, mass, n = inp["embeds"], inp["attn_mass"], inp["n_visual"]
    ref_fused, _, _ = oracle.select_scores(E, mass, cfg.grid_h, cfg.grid_w)
    Ed, md = dev(E, "bf16"), dev(mass)
    for pct in W.C4_KEEP_PCT_SWEEP:
        k = W.keep_count(n, pct)
        kept, fused = hb.hippo_select_tokens(Ed, md, [n], [k], cfg.grid_h, cfg.grid_w)
        torch.cuda.synchronize()
        ref_idx, kth = oracle.topk(ref_fused, k)
        check_kept(host(kept), host(fused), ref_idx, ref_fused, kth, "c4 keep %d%%" % pct)


# ---- the other selection rules ------------------------------------------------------------------------------------

def check_kept_per_frame(got_idx, ref_fused, k, tpf, what):
    """Uniform per-frame budget: per frame the kept sets agree except for tokens whose oracle score lies within 1e-6
    (relative) of that frame's own threshold; the budgets agree exactly."""
    ref_idx, budget = oracle.select_policy(oracle.POLICY_UNIFORM_PER_FRAME, ref_fused, k, tpf)
    assert len(got_idx) == k and np.all(np.diff(got_idx) > 0), what
    assert np.bincount(got_idx // tpf, minlength=len(budget)).tolist() == budget.tolist(), what + ": per-frame counts"
    diff = np.setxor1d(got_idx, ref_idx)
    for j in diff:
        f = j // tpf
        kth = np.sort(ref_fused[f * tpf:(f + 1) * tpf])[::-1][budget[f] - 1]
        assert abs(ref_fused[j] - kth) <= 1e-6 * abs(kth), "%s: token %d differs outside the near-tie band of frame %d" % (what, j, f)


@pytest.mark.parametrize("ci,mask", [(0, 7), (0, 1), (1, 7), (1, 1)])
def test_select_uniform_per_frame(hb, ci, mask):
    cfg = W.CONFIGS[ci]
    inp = W.select_inputs(cfg)
    E, m = dev(inp["embeds"], cfg.dtype), dev(inp["attn_mass"])
    ref_fused, _, _ = oracle.select_scores(inp["embeds"], inp["attn_mass"], cfg.grid_h, cfg.grid_w, score_mask=mask)
    for k in (inp["k"], 0, 1, cfg.frames - 1, inp["n_visual"] - 3, inp["n_visual"]):
        kept, fused = hb.hippo_select_tokens(E, m, [inp["n_visual"]], [k], cfg.grid_h, cfg.grid_w, score_mask=mask,
                                             policy=hb.HIPPO_SELECT_UNIFORM_PER_FRAME)
        torch.cuda.synchronize()
        np.testing.assert_allclose(host(fused), ref_fused, rtol=0, atol=2e-6)
        check_kept_per_frame(host(kept), ref_fused, k, cfg.tokens_per_frame, "c%d mask %d k %d" % (ci, mask, k))


def test_select_policies_ragged_batch_with_partial_frames(hb):
    """Four sequences, three with a partial last frame (one of them a single frame of 9 tokens): per-frame budgets with
    a shortfall, random keys, whole frames; kept lists written at explicit offsets."""
    cfg = W.CONFIGS[3].replace(embed_dim=128)
    tpf = cfg.tokens_per_frame
    lens = [tpf * 3 + 57, tpf * 2, tpf + 1, 9]
    embeds = [W.select_inputs(cfg, b, n)["embeds"] for b, n in enumerate(lens)]
    masses = [W.attention_mass(cfg, n, b) for b, n in enumerate(lens)]
    E, m = dev(np.concatenate(embeds), "bf16"), dev(np.concatenate(masses))
    rng = np.random.default_rng(5)
    keys = rng.random(sum(lens)).astype(np.float32)
    ks = [tpf * 2 + 100, 30, tpf, 4]            # sequence 0: 4 frames, the last (57 tokens) cannot take its 123
    offs = [0, 1000, 2000, 3000]
    starts = np.concatenate([[0], np.cumsum(lens)])
    for policy in (hb.HIPPO_SELECT_UNIFORM_PER_FRAME, hb.HIPPO_SELECT_RANDOM, hb.HIPPO_SELECT_FRAMES):
        kept = torch.full((3300,), -1, dtype=torch.int32, device="cuda")
        _, fused = hb.hippo_select_tokens(E, m, lens, ks, 14, 14, policy=policy, random_keys=dev(keys) if policy == hb.HIPPO_SELECT_RANDOM else None,
                                          kept_idx=kept, kept_offsets=offs)
        torch.cuda.synchronize()
        kept = host(kept)
        for b, n in enumerate(lens):
            got = kept[offs[b]:offs[b] + ks[b]]
            if policy == hb.HIPPO_SELECT_UNIFORM_PER_FRAME:
                ref_fused, _, _ = oracle.select_scores(embeds[b], masses[b], 14, 14)
                check_kept_per_frame(got, ref_fused, ks[b], tpf, "seq %d" % b)
            else:
                score = keys[starts[b]:starts[b + 1]]
                want, _ = oracle.select_policy(policy, score, ks[b], tpf)
                assert got.tolist() == want.tolist(), "policy %d seq %d" % (policy, b)
            assert np.all(kept[offs[b] + ks[b]:(offs[b + 1] if b + 1 < len(offs) else None)] == -1)   # nothing beyond k[b]
        if policy == hb.HIPPO_SELECT_RANDOM:
            np.testing.assert_array_equal(host(fused), keys)


def test_select_random_and_frames_need_no_embeddings(hb):
    cfg = W.CONFIGS[2]
    n, tpf = W.visual_lengths(cfg)[0], cfg.tokens_per_frame
    keys = np.random.default_rng(6).random(n).astype(np.float32)
    keys[100:140] = keys[7]                                        # a run of equal keys across the threshold region
    for k in (W.keep_count(n, 10), 1, n):
        kept, _ = hb.hippo_select_tokens(None, None, [n], [k], cfg.grid_h, cfg.grid_w, policy=hb.HIPPO_SELECT_RANDOM, random_keys=dev(keys))
        torch.cuda.synchronize()
        assert host(kept).tolist() == oracle.select_policy(oracle.POLICY_RANDOM, keys, k, tpf)[0].tolist()
    for k in (W.keep_count(n, 10), tpf * 13, 5, n - 1, n):
        kept, _ = hb.hippo_select_tokens(None, None, [n], [k], cfg.grid_h, cfg.grid_w, policy=hb.HIPPO_SELECT_FRAMES)
        torch.cuda.synchronize()
        assert host(kept).tolist() == oracle.select_policy(oracle.POLICY_FRAME, np.zeros(n), k, tpf)[0].tolist()


def test_topk_all_three_key_tiers(hb):
    """100,352 tokens: keys in registers, in shared memory and re-read from memory; many equal scores (attention term
    only, mass quantised to 64 levels) so that the index tie-break decides most of the threshold."""
    rng = np.random.default_rng(11)
    n, d = 512 * 196, 8
    E = dev(rng.standard_normal((n, d)).astype(np.float32))
    mass = dev((rng.integers(0, 64, size=n) / 64.0).astype(np.float32))
    for k in (1, 5000, 50177, n):
        kept, fused = hb.hippo_select_tokens(E, mass, [n], [k], 14, 14, score_mask=1)
        torch.cuda.synchronize()
        kept, fused = host(kept), host(fused)
        want = np.sort(np.lexsort((np.arange(n), -fused.astype(np.float64)))[:k])
        assert kept.tolist() == want.tolist()


# ---- gather -------------------------------------------------------------------------------------------------------

def run_gather(hb, cfg, n_layers, src_lens, keeps, dtype, shuffle=(None, None)):
    """src logical [L][B][T][H][D]; returns GPU dst as logical [L][B][max_keep][H][D] and the oracle's."""
    from gpu_util import paged_cache  # noqa
    H, D = cfg.dft_kv_heads, cfg.dft_head_dim
    B, T = len(src_lens), max(src_lens)
    rng = W.rng_for(cfg, W.TAG_GATHER)
    k = W.round_to_storage(rng.standard_normal((n_layers, B, T, H, D), dtype=np.float32), dtype)
    v = W.round_to_storage(rng.standard_normal((n_layers, B, T, H, D), dtype=np.float32), dtype)
    keep_lens = [len(x) for x in keeps]
    st, sp = W.make_page_table(src_lens, None if shuffle[0] is None else np.random.default_rng(shuffle[0]))
    dt, dp = W.make_page_table(keep_lens, None if shuffle[1] is None else np.random.default_rng(shuffle[1]), spare_pages=1)
    src_k = dev(np.stack([W.pack_paged(k[l], src_lens, st, sp) for l in range(n_layers)]), dtype)
    src_v = dev(np.stack([W.pack_paged(v[l], src_lens, st, sp) for l in range(n_layers)]), dtype)
    dst_k = torch.zeros((n_layers, dp, H, 64, D), dtype=src_k.dtype, device="cuda")
    dst_v = torch.zeros_like(dst_k)
    src = hb.KVCache(src_k[0], src_v[0], dev(st))
    dst = hb.KVCache(dst_k[0], dst_v[0], dev(dt))
    es = src_k.element_size()
    offs = np.concatenate([[0], np.cumsum(keep_lens)]).astype(np.int32)
    hb.hippo_gather_kv(n_layers, src, sp * H * 64 * D * es, dst, dp * H * 64 * D * es, B,
                       dev(np.concatenate(keeps).astype(np.int32)), dev(offs), int(offs[-1]))
    torch.cuda.synchronize()
    view = (lambda t: t.view(torch.int16).cpu().numpy().view(np.uint16)) if dtype == "bf16" else (lambda t: t.cpu().numpy())
    bits = (lambda a: W.to_bf16_bits(a)) if dtype == "bf16" else (lambda a: a)
    for name, dst_t, src_a in (("K", dst_k, k), ("V", dst_v, v)):
        g = view(dst_t)
        for l in range(n_layers):
            got = W.unpack_paged(g[l], keep_lens, dt)
            for b in range(B):
                ref = oracle.gather_kv(bits(src_a[l, b][None]), keeps[b])[0]
                np.testing.assert_array_equal(got[b, :keep_lens[b]], ref, err_msg="%s layer %d seq %d" % (name, l, b))
    return dst_k


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_gather_small_paged(hb, dtype):
    cfg = W.CONFIGS[0]
    rng = np.random.default_rng(8)
    src_lens = [288, 70, 1]
    keeps = [np.sort(rng.choice(288, 58, replace=False)), np.arange(70), np.array([0])]
    run_gather(hb, cfg, 3, src_lens, keeps, dtype, shuffle=(1, 2))


@pytest.mark.parametrize("ci,keep_pct", [(1, None), (2, None), (3, None), (4, 50), (4, 25), (4, 10), (4, 5)])
def test_gather_config_shapes(hb, ci, keep_pct):
    """Keep list = the oracle-independent random kept visual tokens + every text position, as the step does; the
    64k configuration at each kept share of its sweep."""
    cfg = W.CONFIGS[ci]
    pct = cfg.keep_pct if keep_pct is None else keep_pct
    rng = np.random.default_rng(ci)
    n_vs = W.visual_lengths(cfg)
    src_lens = [n + cfg.n_text for n in n_vs]
    keeps = [np.concatenate([np.sort(rng.choice(n, W.keep_count(n, pct), replace=False)),
                             np.arange(n, n + cfg.n_text)]) for n in n_vs]
    run_gather(hb, cfg, 2, src_lens, keeps, cfg.dtype, shuffle=(3, 4) if cfg.paged_shuffle else (None, None))


def test_gather_skips_out_of_range_entries_and_says_so(hb):
    """A keep index beyond the source's pages, a negative one, a page id outside the pool and a sequence that keeps more
    than its destination holds: nothing is read or written for those entries, the flag word is raised, every valid entry is
    still copied."""
    cfg = W.CONFIGS[0]
    H, D = cfg.dft_kv_heads, cfg.dft_head_dim
    rng = np.random.default_rng(3)
    src_lens = [200, 100]
    k = rng.standard_normal((2, 200, H, D)).astype(np.float32)
    st, sp = W.make_page_table(src_lens, np.random.default_rng(1))
    src_pool = dev(W.pack_paged(k, src_lens, st, sp))
    src = hb.KVCache(src_pool, src_pool.clone(), dev(st))

    def run(keeps, dst_table, n_dst_pages, src_cache=src):
        dst_k = torch.full((n_dst_pages, H, 64, D), -7.0, dtype=torch.float32, device="cuda")
        dst = hb.KVCache(dst_k, dst_k.clone(), dev(dst_table))
        offs = np.concatenate([[0], np.cumsum([len(x) for x in keeps])]).astype(np.int32)
        flag = torch.zeros(1, dtype=torch.int32, device="cuda")
        hb.hippo_gather_kv(1, src_cache, 0, dst, 0, len(keeps), dev(np.concatenate(keeps).astype(np.int32)), dev(offs),
                           int(offs[-1]), bad_index=flag)
        torch.cuda.synchronize()
        return host(dst_k), int(flag.item())

    dt, dp = W.make_page_table([64, 64], None)
    good = [np.array([5, 17, 199]), np.array([0, 99])]
    got, flag = run(good, dt, dp)
    assert flag == 0
    assert np.array_equal(got[dt[0, 0], :, :3], np.transpose(k[0, good[0]], (1, 0, 2)))
    # one entry past the source's page capacity (4 pages = 256 positions), one negative
    bad = [np.array([5, 256, 199]), np.array([-1, 99])]
    got, flag = run(bad, dt, dp)
    assert flag == 1
    assert np.array_equal(got[dt[0, 0], :, 0], k[0, 5]) and np.array_equal(got[dt[0, 0], :, 2], k[0, 199])
    assert np.all(got[dt[0, 0], :, 1] == -7.0) and np.all(got[dt[1, 0], :, 0] == -7.0)      # skipped: destination untouched
    assert np.array_equal(got[dt[1, 0], :, 1], k[1, 99])
    # a page id outside the source pool
    st_bad = st.copy()
    st_bad[0, 0] = sp + 5
    got, flag = run(good, dt, dp, hb.KVCache(src_pool, src_pool.clone(), dev(st_bad)))
    assert flag == 1 and np.all(got[dt[0, 0], :, :2] == -7.0) and np.array_equal(got[dt[0, 0], :, 2], k[0, 199])
    # sequence 0 keeps 70 tokens but its destination row holds one page: entries 64.. are skipped, not spilled into sequence 1
    many = [np.arange(70), np.array([3])]
    got, flag = run(many, dt, dp)
    assert flag == 1
    assert np.array_equal(got[dt[0, 0]], np.transpose(k[0, :64], (1, 0, 2)))
    assert np.array_equal(got[dt[1, 0], :, 0], k[1, 3]) and np.all(got[dt[1, 0], :, 1:] == -7.0)
    # more entries than the destination can hold at all: refused on the host
    with pytest.raises(hb.HippoError) as e:
        run([np.arange(100), np.arange(100)], dt, dp)
    assert e.value.status == hb.HIPPO_ERR_INVALID_ARG


# ---- acceptance -----------------------------------------------------------------------------------------------------

def check_accept(hb, inp, what, forgiven_allowed=0):
    """Accepted lengths and emitted tokens bit for bit.  A differing sequence is forgiven only when the oracle reports
    that a uniform sat within 1e-12 (relative) of a decision boundary, and the number forgiven is itself checked:
    none on the benchmark configurations."""
    rn, rout, ma, mc = oracle.accept(inp["target_logits"], inp["draft_logits"], inp["draft_tokens"], inp["u_accept"],
                                     inp["u_resample"])
    # the margins themselves must be usable: positive and finite wherever a test / a draw was made
    assert np.all(mc >= 0) and np.all(np.isfinite(mc)), what
    assert np.all(ma >= 0), what
    args = [dev(inp[k]) for k in ("target_logits", "draft_logits", "draft_tokens", "u_accept", "u_resample")]
    # both launch forms of the sampling acceptance (one kernel / three chained kernels), and the library's own choice
    for form, flag in (("chain", hb.HIPPO_ACCEPT_THREE_LAUNCHES), ("one launch", hb.HIPPO_ACCEPT_ONE_LAUNCH), ("auto", 0)):
        ws = hb.new_workspace(hb.hippo_accept_workspace_bytes(*rout.shape[:1], rout.shape[1] - 1, inp["target_logits"].shape[2]))
        n, out = hb.hippo_accept(*args, mode=hb.HIPPO_ACCEPT_SAMPLE | flag, workspace=ws)
        torch.cuda.synchronize()
        assert hb.hippo_workspace_status(ws) == hb.HIPPO_OK
        n, out = host(n), host(out)
        bad = np.where((n != rn) | (out != rout).any(axis=1))[0]
        forgiven = 0
        for b in bad:
            assert min(ma[b], mc[b]) < 1e-12, "%s (%s): sequence %d differs (n %d vs %d, tokens %s vs %s), margins %.3e %.3e" % (
                what, form, b, n[b], rn[b], out[b], rout[b], ma[b], mc[b])
            forgiven += 1
        assert forgiven <= forgiven_allowed, "%s (%s): %d of %d sequences forgiven by the near-boundary rule" % (what, form, forgiven, len(rn))
    return rn


def test_accept_c0(hb):
    cfg = W.CONFIGS[0]
    check_accept(hb, W.accept_inputs(cfg), "c0")
    lens = []
    for eps in (0.0, 0.1, 1.0):
        rn = check_accept(hb, W.accept_inputs(cfg, batch=64, corr_eps=eps), "c0 eps %g" % eps)
        lens.append(rn)
    assert np.all(lens[0] == cfg.gamma)                 # draft == target: everything accepted, bonus drawn
    assert len(set(lens[2].tolist())) >= 3              # mid-chain rejections occur


@pytest.mark.parametrize("ci", [1, 2, 3, 4])
def test_accept_full_vocab(hb, ci):
    cfg = W.CONFIGS[ci]
    gammas = W.C4_GAMMA_SWEEP if ci == 4 else (cfg.gamma,)
    for g in gammas:
        check_accept(hb, W.accept_inputs(cfg, gamma=g), "%s gamma %d" % (cfg.name, g))
    check_accept(hb, W.accept_inputs(cfg, batch=4, corr_eps=0.3, sub=1), cfg.name + " correlated")
    check_accept(hb, W.accept_inputs(cfg, batch=2, corr_eps=0.0, sub=2), cfg.name + " identical")


def test_accept_odd_vocab_and_gamma0(hb):
    cfg = W.CONFIGS[0]
    check_accept(hb, W.accept_inputs(cfg, batch=5, gamma=3, vocab=4099, corr_eps=0.5), "V=4099")
    check_accept(hb, W.accept_inputs(cfg, batch=3, gamma=0, vocab=777), "gamma 0")
    check_accept(hb, W.accept_inputs(cfg, batch=3, gamma=1, vocab=3, corr_eps=2.0), "V=3")


def test_accept_draft_token_outside_the_vocabulary_is_rejected(hb):
    """A draft token id that is not in [0, vocab) is never used as an index: it counts as rejected and the replacement is
    drawn from the residual of its row, exactly as the oracle does for a token whose acceptance test fails."""
    cfg = W.CONFIGS[0]
    inp = W.accept_inputs(cfg, batch=6, gamma=4, vocab=777, corr_eps=0.0)       # draft == target: all accepted otherwise
    x = inp["draft_tokens"].copy()
    x[1, 2], x[2, 0], x[4, 3] = 777, -5, 1 << 30
    n, out = hb.hippo_accept(dev(inp["target_logits"]), dev(inp["draft_logits"]), dev(x), dev(inp["u_accept"]),
                             dev(inp["u_resample"]))
    torch.cuda.synchronize()
    n, out = host(n), host(out)
    assert n.tolist() == [4, 2, 0, 4, 3, 4]
    for b, j in ((1, 2), (2, 0), (4, 3)):
        assert out[b, :j].tolist() == x[b, :j].tolist() and 0 <= out[b, j] < 777 and (out[b, j + 1:] == -1).all()
    # the untouched sequences still match the oracle
    rn, rout, _, _ = oracle.accept(inp["target_logits"], inp["draft_logits"], inp["draft_tokens"], inp["u_accept"], inp["u_resample"])
    for b in (0, 3, 5):
        assert n[b] == rn[b] and out[b].tolist() == rout[b].tolist()


@pytest.mark.parametrize("ci", [0, 1, 3])
def test_accept_greedy(hb, ci):
    """Greedy verification: bit-exact against the oracle; draft tokens = arg-max of draft rows that partly agree."""
    cfg = W.CONFIGS[ci]
    B = max(cfg.batch, 6)
    inp = W.accept_inputs(cfg, batch=B, corr_eps=0.0, sub=5)
    tl = inp["target_logits"]
    x = tl[:, :cfg.gamma].argmax(axis=-1).astype(np.int32)
    rng = np.random.default_rng(ci)
    wrong = rng.random(x.shape) < 0.25
    x[wrong] = rng.integers(0, cfg.vocab, size=int(wrong.sum()))
    x[0] = tl[0, :cfg.gamma].argmax(axis=-1)                 # one sequence accepts everything
    tl[1, 0, 5] = tl[1, 0, 9] = tl[1, 0].max() + 1.0          # a tie: the lowest id wins
    n, out = hb.hippo_accept(dev(tl), None, dev(x), None, None, mode=hb.HIPPO_ACCEPT_GREEDY)
    torch.cuda.synchronize()
    rn, rout = oracle.accept_greedy(tl, x)
    np.testing.assert_array_equal(host(n), rn)
    np.testing.assert_array_equal(host(out), rout)
    assert rn[0] == cfg.gamma and len(set(rn.tolist())) >= 2
