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


# ---- acceptance -----------------------------------------------------------------------------------------------------

def check_accept(hb, inp, what, forgiven_allowed=0):
    """Accepted lengths and emitted tokens bit for bit.  A differing sequence is forgiven only when the oracle reports
    that a uniform sat within 1e-12 (relative) of a decision boundary, and the number forgiven is itself checked:
    none on the benchmark configurations."""
    n, out = hb.hippo_accept(dev(inp["target_logits"]), dev(inp["draft_logits"]), dev(inp["draft_tokens"]),
                             dev(inp["u_accept"]), dev(inp["u_resample"]))
    torch.cuda.synchronize()
    rn, rout, ma, mc = oracle.accept(inp["target_logits"], inp["draft_logits"], inp["draft_tokens"], inp["u_accept"],
                                     inp["u_resample"])
    # the margins themselves must be usable: positive and finite wherever a test / a draw was made
    assert np.all(mc >= 0) and np.all(np.isfinite(mc)), what
    assert np.all(ma >= 0), what
    n, out = host(n), host(out)
    bad = np.where((n != rn) | (out != rout).any(axis=1))[0]
    forgiven = 0
    for b in bad:
        assert min(ma[b], mc[b]) < 1e-12, "%s: sequence %d differs (n %d vs %d, tokens %s vs %s), margins %.3e %.3e" % (
            what, b, n[b], rn[b], out[b], rout[b], ma[b], mc[b])
        forgiven += 1
    assert forgiven <= forgiven_allowed, "%s: %d of %d sequences forgiven by the near-boundary rule" % (what, forgiven, len(rn))
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
