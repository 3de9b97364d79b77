"""GPU parity: hippo_attention_mass (Section 5.1, Eq. 2; through the C ABI) against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import dev, host, paged_cache
from paper_2601_08273_b200 import workloads as W

pytestmark = pytest.mark.gpu

# |got - ref| <= RTOL * ref + 1e-12.  bf16 path: fp32 tensor-core accumulation of exact products (~1e-6 on a logit),
# ex2.approx (2^-22), fp32 row and column sums over up to 65,536 / 2,048 terms: a few 1e-5 at worst.
RTOL = {"fp32": 1e-5, "bf16": 1e-4}


@pytest.fixture(scope="module")
def hb():
    from paper_2601_08273_b200 import binding
    return binding


def gpu_mass(hb, q_layers, k_layers, n_visual, dtype, scale=0.0, shuffle_seed=None, fill=0.0, caps=None):
    """q_layers[l] [B][L][Hq][D], k_layers[l] [B][T][Hkv][D] -> mass [sum n_visual] after all layers."""
    total = int(sum(n_visual))
    mass = torch.zeros(max(total, 1), dtype=torch.float32, device="cuda")
    B, L, Hq, _ = q_layers[0].shape
    weight = 1.0 / (len(q_layers) * Hq * L)
    for q, k in zip(q_layers, k_layers):
        lens = [max(int(n), 1) for n in n_visual]
        kv, _, _ = paged_cache(hb, k, k, lens, dtype, shuffle_seed=shuffle_seed, fill=fill, caps=caps)
        hb.hippo_attention_mass(dev(q, dtype), kv, n_visual, weight, mass, softmax_scale=scale)
    torch.cuda.synchronize()
    return host(mass)[:total]


def oracle_mass(q_layers, k_layers, n_visual, scale=None):
    m = oracle.attention_mass(np.stack(q_layers), np.stack(k_layers), n_visual, scale=scale)
    return np.concatenate([m[b, :n] for b, n in enumerate(n_visual)]) if sum(n_visual) else np.zeros(0)


def check(got, ref, dtype, what):
    err = np.abs(got.astype(np.float64) - ref)
    bound = RTOL[dtype] * np.abs(ref) + 1e-12
    bad = err > bound
    assert not bad.any(), "%s: %d / %d off, worst rel %.3e" % (what, bad.sum(), bad.size, (err / np.maximum(ref, 1e-300)).max())


def rand_case(seed, B, L, Hq, Hkv, D, T, dtype, n_layers=1):
    rng = np.random.default_rng(seed)
    qs = [W.round_to_storage(rng.standard_normal((B, L, Hq, D)).astype(np.float32), dtype) for _ in range(n_layers)]
    ks = [W.round_to_storage(rng.standard_normal((B, T, Hkv, D)).astype(np.float32), dtype) for _ in range(n_layers)]
    return qs, ks


def test_c0_tiny_fp32(hb):
    cfg = W.CONFIGS[0]
    nv = W.visual_lengths(cfg)
    inp = W.mass_inputs(cfg, nv)
    got = gpu_mass(hb, [inp["q_txt"]], [inp["k_vid"]], nv, "fp32")
    check(got, oracle_mass([inp["q_txt"]], [inp["k_vid"]], nv), "fp32", "c0")
    assert abs(got.sum() - 1.0) < 1e-5


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
def test_ragged_batch_paged_two_layers(hb, D, dtype):
    n_visual = [333, 1, 200]     # several key tiles with a ragged tail, one key, a length that ends inside a page
    qs, ks = rand_case(3, 3, 20, 8, 2, D, 400, dtype, n_layers=2)
    ref = oracle_mass(qs, ks, n_visual)
    a = gpu_mass(hb, qs, ks, n_visual, dtype, shuffle_seed=5, caps=[400, 400, 400])
    check(a, ref, dtype, "ragged")
    # positions past the visual tokens hold NaN: never read into a result; other page order: same bits
    ks_nan = [k.copy() for k in ks]
    for k in ks_nan:
        for b, n in enumerate(n_visual):
            k[b, n:] = np.nan
    b = gpu_mass(hb, qs, ks_nan, n_visual, dtype, shuffle_seed=6, caps=[400, 400, 400])
    np.testing.assert_array_equal(a, b)


def test_group_of_seven_and_partial_row_block(hb):
    # G = 7: 18 text rows (126 packed rows) per block; 40 text rows = two full blocks and one of four rows
    n_visual = [700, 130]
    qs, ks = rand_case(4, 2, 40, 14, 2, 128, 700, "bf16")
    check(gpu_mass(hb, qs, ks, n_visual, "bf16", scale=0.2, shuffle_seed=1), oracle_mass(qs, ks, n_visual, scale=0.2), "bf16", "G=7")


def test_empty_sequences_and_accumulation(hb):
    n_visual = [0, 150, 0]
    qs, ks = rand_case(5, 3, 8, 4, 4, 64, 150, "bf16")
    got = gpu_mass(hb, qs, ks, n_visual, "bf16")
    check(got, oracle_mass(qs, ks, n_visual), "bf16", "empty")
    # a second call with the same layer adds the same amount
    mass = torch.zeros(150, dtype=torch.float32, device="cuda")
    kv, _, _ = paged_cache(hb, ks[0], ks[0], [1, 150, 1], "bf16", shuffle_seed=2)
    for _ in range(2):
        hb.hippo_attention_mass(dev(qs[0], "bf16"), kv, n_visual, 1.0 / (4 * 8), mass)
    torch.cuda.synchronize()
    np.testing.assert_allclose(host(mass), 2.0 * got, rtol=1e-6)
    all_empty = torch.full((4,), 7.0, dtype=torch.float32, device="cuda")
    hb.hippo_attention_mass(dev(qs[0], "bf16"), kv, [0, 0, 0], 1.0, all_empty)
    torch.cuda.synchronize()
    assert (host(all_empty) == 7.0).all()


@pytest.mark.parametrize("ci", [1, 2, 3, 4])
def test_configs_one_layer_full_size(hb, ci):
    cfg = W.CONFIGS[ci]
    nv = W.visual_lengths(cfg)
    inp = W.mass_inputs(cfg, nv, layer=ci)
    got = gpu_mass(hb, [inp["q_txt"]], [inp["k_vid"]], nv, cfg.dtype, shuffle_seed=ci if cfg.paged_shuffle else None)
    ref = oracle_mass([inp["q_txt"]], [inp["k_vid"]], nv)
    check(got, ref, cfg.dtype, cfg.name)
    # each sequence's mass sums to one
    off = 0
    for n in nv:
        assert abs(got[off:off + n].sum() - 1.0) < 1e-4
        off += n


def test_feeds_the_selection(hb):
    """Mass computed on the GPU, handed to hippo_select_tokens: the kept set equals the oracle's on the oracle's mass,
    outside the near-tie band of the k-th score."""
    cfg = W.CONFIGS[1].replace(frames=4)
    nv = W.visual_lengths(cfg)
    inp = W.mass_inputs(cfg, nv)
    got = gpu_mass(hb, [inp["q_txt"]], [inp["k_vid"]], nv, cfg.dtype)
    ref = oracle_mass([inp["q_txt"]], [inp["k_vid"]], nv)
    check(got, ref, cfg.dtype, "mass")
    sel = W.select_inputs(cfg)
    k = sel["k"]
    kept, fused = hb.hippo_select_tokens(dev(sel["embeds"], cfg.dtype), dev(got.astype(np.float32)), nv, [k], cfg.grid_h, cfg.grid_w)
    torch.cuda.synchronize()
    ref_kept, scores, kth = oracle.select_tokens(sel["embeds"], ref, k, cfg.grid_h, cfg.grid_w)
    # the mass differs from the oracle's by ~1e-5 relative, which moves standardised scores by ~1e-4: tokens within that
    # distance of the threshold may differ, all others must agree
    band = np.abs(scores - kth) <= 1e-3 * max(1.0, abs(kth))
    diff = np.setxor1d(host(kept)[:k], ref_kept)
    assert band[diff].all()
    assert len(diff) <= 8


def test_reproducible_bits(hb):
    """The sums run in a fixed order: the same call gives the same bits, whatever else the GPU did in between."""
    cfg = W.CONFIGS[1]
    nv = W.visual_lengths(cfg)
    inp = W.mass_inputs(cfg, nv, layer=3)
    a = gpu_mass(hb, [inp["q_txt"]], [inp["k_vid"]], nv, cfg.dtype)
    torch.randn(1 << 22, device="cuda").sum().item()
    b = gpu_mass(hb, [inp["q_txt"]], [inp["k_vid"]], nv, cfg.dtype)
    np.testing.assert_array_equal(a, b)


def test_bounded_wait_runs_out_and_the_workspace_recovers(hb):
    """The same exercise as for the attention kernels: a 200 ns wait limit makes the first wait of the tensor-core
    mass kernel give up while every load still lands; the kernel returns, the status word says so, a reset clears it
    and the next call matches the oracle."""
    rng = np.random.default_rng(8)
    B, L, Hq, Hkv, D, nv = 1, 16, 8, 2, 128, [1500]
    q = W.round_to_storage(rng.standard_normal((B, L, Hq, D)).astype(np.float32), "bf16")
    k = W.round_to_storage(rng.standard_normal((B, nv[0], Hkv, D)).astype(np.float32), "bf16")
    kv, _, _ = paged_cache(hb, k, k, nv, "bf16")
    qd = dev(q, "bf16")
    ws = hb.new_workspace(hb.hippo_attention_mass_workspace_bytes(nv, L, Hq, Hkv, D, hb.HIPPO_DTYPE_BF16))
    mass = torch.zeros(nv[0], dtype=torch.float32, device="cuda")
    w = 1.0 / (Hq * L)
    hb.hippo_workspace_set_wait_limit(ws, 200)
    hb.hippo_attention_mass(qd, kv, nv, w, mass, workspace=ws)
    assert hb.hippo_workspace_status(ws) == hb.HIPPO_ERR_TIMEOUT
    hb.hippo_workspace_reset(ws)
    assert hb.hippo_workspace_status(ws) == hb.HIPPO_OK
    mass.zero_()
    hb.hippo_attention_mass(qd, kv, nv, w, mass, workspace=ws)
    assert hb.hippo_workspace_status(ws) == hb.HIPPO_OK
    ref = oracle.attention_mass(q[None], k[None], nv)[0][:nv[0]]
    got = host(mass)
    assert np.all(np.abs(got - ref) <= RTOL["bf16"] * ref + 1e-12)
