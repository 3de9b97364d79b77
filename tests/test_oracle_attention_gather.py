"""Pins for the oracle's attention (library softmax attention, closed forms, masking invariants) and
gather (copy identities).  CPU only."""
import numpy as np
import torch

import oracle
from paper_2601_08273_b200 import workloads as W


def torch_reference(q, k, v, kv_len, scale=None):
    """Library routine: torch's scaled_dot_product_attention in fp64 with an explicit boolean mask."""
    B, q_len, Hq, D = q.shape
    Hkv = k.shape[2]
    G = Hq // Hkv
    out = np.zeros((B, q_len, Hq, D))
    for b in range(B):
        n = kv_len[b]
        qq = torch.from_numpy(q[b].astype(np.float64)).permute(1, 0, 2)            # [Hq][q_len][D]
        kk = torch.from_numpy(k[b, :n].astype(np.float64)).permute(1, 0, 2).repeat_interleave(G, dim=0)
        vv = torch.from_numpy(v[b, :n].astype(np.float64)).permute(1, 0, 2).repeat_interleave(G, dim=0)
        j = torch.arange(n)[None, :]
        t = torch.arange(q_len)[:, None]
        mask = j <= (n - q_len + t)
        o = torch.nn.functional.scaled_dot_product_attention(qq, kk, vv, attn_mask=mask, scale=scale)
        out[b] = o.permute(1, 0, 2).numpy()
    return out


def test_matches_library_attention_c0_shapes():
    cfg = W.CONFIGS[0]
    n_v = W.visual_lengths(cfg)[0]
    q_len = cfg.gamma + 1
    kv_len = [n_v + cfg.n_text + q_len]
    inp = W.attention_inputs(cfg, "target", kv_len, q_len)
    out, lse = oracle.attention(inp["q"], inp["k"], inp["v"], kv_len)
    want = torch_reference(inp["q"], inp["k"], inp["v"], kv_len)
    np.testing.assert_allclose(out, want, rtol=1e-11, atol=1e-12)
    # lse against a direct logsumexp of one row
    b, t, h = 0, 2, 3
    n = kv_len[0] - q_len + t + 1
    a = (inp["k"][0, :n, 0].astype(np.float64) @ inp["q"][0, t, h].astype(np.float64)) / 8.0
    np.testing.assert_allclose(lse[b, t, h], np.log(np.exp(a - a.max()).sum()) + a.max(), rtol=1e-13)


def test_matches_library_attention_ragged_gqa():
    rng = np.random.default_rng(7)
    B, q_len, Hq, Hkv, D = 3, 3, 6, 2, 16
    kv_len = [5, 37, 20]
    q = rng.standard_normal((B, q_len, Hq, D)).astype(np.float32)
    k = rng.standard_normal((B, 37, Hkv, D)).astype(np.float32)
    v = rng.standard_normal((B, 37, Hkv, D)).astype(np.float32)
    out, _ = oracle.attention(q, k, v, kv_len, scale=0.3)
    np.testing.assert_allclose(out, torch_reference(q, k, v, kv_len, scale=0.3), rtol=1e-11, atol=1e-12)
    rows = [(0, 0, 0), (1, 2, 5), (2, 1, 3)]
    sub, _ = oracle.attention(q, k, v, kv_len, scale=0.3, rows=rows)
    for i, (b, t, h) in enumerate(rows):
        np.testing.assert_array_equal(sub[i], out[b, t, h])


def test_closed_forms():
    rng = np.random.default_rng(9)
    D = 8
    # all keys equal -> output = mean of the visible values
    q = rng.standard_normal((1, 2, 2, D)).astype(np.float32)
    k = np.tile(rng.standard_normal((1, 1, 1, D)).astype(np.float32), (1, 6, 1, 1))
    v = rng.standard_normal((1, 6, 1, D)).astype(np.float32)
    out, lse = oracle.attention(q, k, v, [6])
    np.testing.assert_allclose(out[0, 0, 0], v[0, :5, 0].astype(np.float64).mean(axis=0), rtol=1e-13)
    np.testing.assert_allclose(out[0, 1, 1], v[0, :6, 0].astype(np.float64).mean(axis=0), rtol=1e-13)
    # one key with a logit 50 above the rest -> output ~ that key's value
    k = np.zeros((1, 6, 1, D), dtype=np.float32)
    k[0, 3, 0, 0] = 50.0
    q = np.zeros((1, 1, 1, D), dtype=np.float32)
    q[0, 0, 0, 0] = 1.0
    out, _ = oracle.attention(q, k, v, [6], scale=1.0)
    np.testing.assert_allclose(out[0, 0, 0], v[0, 3, 0], atol=1e-20 + 6 * np.exp(-50.0) * 4)
    # a single key: output = its value, lse = its logit
    out, lse = oracle.attention(q, k[:, 3:4], v[:, 3:4], [1], scale=1.0)
    np.testing.assert_array_equal(out[0, 0, 0], v[0, 3, 0].astype(np.float64))
    assert lse[0, 0, 0] == 50.0


def test_masking_and_grouping_invariants():
    rng = np.random.default_rng(13)
    B, q_len, Hq, Hkv, D, T = 1, 4, 4, 2, 16, 50
    q = rng.standard_normal((B, q_len, Hq, D)).astype(np.float32)
    q[0, :, 1] = q[0, :, 0]          # heads 0 and 1 share KV head 0 and now the same query
    k = rng.standard_normal((B, T, Hkv, D)).astype(np.float32)
    v = rng.standard_normal((B, T, Hkv, D)).astype(np.float32)
    out, _ = oracle.attention(q, k, v, [T])
    np.testing.assert_array_equal(out[0, :, 0], out[0, :, 1])
    assert np.abs(out[0, :, 2] - out[0, :, 0]).max() > 1e-3          # other KV head: different result
    # keys past a row's causal limit do not influence that row
    k2, v2 = k.copy(), v.copy()
    k2[0, T - 2:] += 5.0
    v2[0, T - 2:] -= 3.0
    out2, _ = oracle.attention(q, k2, v2, [T])
    np.testing.assert_array_equal(out2[0, :2], out[0, :2])           # rows 0,1 see keys <= T-4, T-3
    assert np.abs(out2[0, 3] - out[0, 3]).max() > 1e-3
    # entries past kv_len are never read
    out3, _ = oracle.attention(q, k2, v2, [T - 2])
    out4, _ = oracle.attention(q, k, v, [T - 2])
    np.testing.assert_array_equal(out3, out4)


def test_gather_identities():
    rng = np.random.default_rng(21)
    L, T, H, D = 3, 40, 2, 8
    src = W.to_bf16_bits(rng.standard_normal((L, T, H, D)).astype(np.float32))
    ident = oracle.gather_kv(src, np.arange(T))
    np.testing.assert_array_equal(ident, src)
    keep = np.sort(rng.choice(T, 17, replace=False)).astype(np.int32)
    g = oracle.gather_kv(src, keep)
    np.testing.assert_array_equal(g, src[:, keep])                   # numpy fancy indexing is the library routine
    keep2 = np.sort(rng.choice(17, 5, replace=False)).astype(np.int32)
    np.testing.assert_array_equal(oracle.gather_kv(g, keep2), oracle.gather_kv(src, keep[keep2]))
    assert oracle.gather_kv(src, np.zeros(0, np.int32)).shape == (L, 0, H, D)


def test_paged_layout_roundtrip():
    rng = np.random.default_rng(2)
    lens = [70, 64, 1, 130]
    x = rng.standard_normal((4, 130, 2, 8)).astype(np.float32)
    table, n_pool = W.make_page_table(lens, np.random.default_rng(3), spare_pages=2)
    pool = W.pack_paged(x, lens, table, n_pool)
    back = W.unpack_paged(pool, lens, table)
    for b, n in enumerate(lens):
        np.testing.assert_array_equal(back[b, :n], x[b, :n])
    used = table[table >= 0]
    assert len(set(used.tolist())) == len(used) == 2 + 1 + 1 + 3
