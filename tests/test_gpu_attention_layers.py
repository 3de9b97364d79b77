"""GPU parity: hippo_verify_attention_layers (several layers of verification attention in one launch) against the CPU
oracle, layer by layer, and the bounded-wait time-out path of the tensor-core kernels."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import TOL, assert_close, dev, host
from paper_2601_08273_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def hb():
    from paper_2601_08273_b200 import binding
    return binding


def layer_inputs(rng, n_layers, B, q_len, Hq, Hkv, D, lens, dtype):
    T = max(lens)
    q = W.round_to_storage(rng.standard_normal((n_layers, B, q_len, Hq, D)).astype(np.float32), dtype)
    k = W.round_to_storage(rng.standard_normal((n_layers, B, T, Hkv, D)).astype(np.float32), dtype)
    v = W.round_to_storage(rng.standard_normal((n_layers, B, T, Hkv, D)).astype(np.float32), dtype)
    return q, k, v


def layer_caches(hb, k, v, lens, dtype, shuffle_seed, fill=0.0):
    """One page table shared by all layers, one pool pair per layer."""
    rng = None if shuffle_seed is None else np.random.default_rng(shuffle_seed)
    table, n_pool = W.make_page_table(lens, rng, spare_pages=2)
    tab = None if (shuffle_seed is None and len(lens) == 1) else dev(table)
    caches = []
    for l in range(k.shape[0]):
        kp = dev(W.pack_paged(k[l], lens, table, n_pool, fill=fill), dtype)
        vp = dev(W.pack_paged(v[l], lens, table, n_pool, fill=fill), dtype)
        caches.append(hb.KVCache(kp, vp, tab, table.shape[1]))
    return caches


def run_layers(hb, q, k, v, lens, dtype, shuffle_seed=7, host_lens=False, want_lse=True, fill=0.0):
    n_layers = q.shape[0]
    caches = layer_caches(hb, k, v, lens, dtype, shuffle_seed, fill)
    qs = [dev(q[l], dtype) for l in range(n_layers)]
    outs = [torch.full_like(t, float("nan")) for t in qs]
    lses = [torch.full(q.shape[1:4], float("nan"), dtype=torch.float32, device="cuda") for _ in range(n_layers)] if want_lse else None
    ws = hb.new_workspace(hb.hippo_verify_attention_layers_workspace_bytes(n_layers, q.shape[1], q.shape[2], q.shape[3],
                                                                           k.shape[3], q.shape[4]))
    hb.hippo_verify_attention_layers(qs, caches, dev(np.asarray(lens, np.int32)), max(lens), outs, lse_layers=lses,
                                     workspace=ws, kv_len_host=lens if host_lens else None)
    torch.cuda.synchronize()
    assert hb.hippo_workspace_status(ws) == hb.HIPPO_OK
    return [host(o) for o in outs], (None if lses is None else [host(x) for x in lses])


def check_layers(hb, q, k, v, lens, dtype, **kw):
    outs, lses = run_layers(hb, q, k, v, lens, dtype, **kw)
    for l in range(q.shape[0]):
        live = [b for b in range(len(lens)) if lens[b] >= q.shape[2]]
        ref, ref_lse = oracle.attention(q[l][live], k[l][live], v[l][live], [lens[b] for b in live])
        assert_close(outs[l][live], ref, TOL[dtype], "layer %d" % l)
        if lses is not None:
            assert_close(lses[l][live], ref_lse, TOL[dtype] if dtype == "fp32" else 2e-3, "layer %d lse" % l)
        for b in range(len(lens)):
            if lens[b] < q.shape[2]:      # skipped sequence: zeros, lse = -inf
                assert np.all(outs[l][b] == 0)
                assert lses is None or np.all(np.isneginf(lses[l][b]))
    return outs


@pytest.mark.parametrize("D", [64, 128])
def test_layers_ragged_batch_more_layers_than_slot_sets(hb, D):
    """Seven layers (the partial-result slot sets are reused twice), ragged paged batch with several tiles per unit, a
    sequence equal to q_len and one shorter than q_len; slots past each length hold NaN."""
    rng = np.random.default_rng(101 + D)
    B, q_len, Hq, Hkv = 4, 6, 8, 2
    lens = [2333, 6, 1290, 3]
    q, k, v = layer_inputs(rng, 7, B, q_len, Hq, Hkv, D, lens, "bf16")
    check_layers(hb, q, k, v, lens, "bf16", fill=np.nan)
    # the host copy of the lengths only plans the launch (grid, work split): another summation order, the same result
    check_layers(hb, q, k, v, lens, "bf16", host_lens=True, want_lse=False)


def test_layers_one_unit_per_cta_and_more(hb):
    """40 units (one table warp is not enough: the block-wide partition) and 200 units (more than CTAs: the flat split,
    CTAs walk several units per layer and units straddle CTAs)."""
    for B, Hkv, n_layers in ((10, 4, 4), (50, 4, 5)):
        rng = np.random.default_rng(B)
        q_len, G, D = 3, 2, 128
        lens = [int(x) for x in rng.integers(q_len, 1200, size=B)]
        lens[1] = 2
        q, k, v = layer_inputs(rng, n_layers, B, q_len, Hkv * G, Hkv, D, lens, "bf16")
        check_layers(hb, q, k, v, lens, "bf16", shuffle_seed=B)


@pytest.mark.parametrize("D", [64, 128])
def test_layers_one_unit_with_more_contributors_than_a_merge_batch(hb, D):
    """One (sequence, KV head) unit of 14,000 keys is split over some 30 CTAs: a row's merge takes more partials than the
    merge warp fetches in one batch (24), so the running maximum and the rescaling across batches are exercised; values of
    K are scaled so that the row maxima differ from partial to partial."""
    rng = np.random.default_rng(240 + D)
    B, q_len, Hq, Hkv = 1, 4, 4, 1
    lens = [14000]
    q, k, v = layer_inputs(rng, 3, B, q_len, Hq, Hkv, D, lens, "bf16")
    k *= 4.0                                  # exact in bf16
    check_layers(hb, q, k, v, lens, "bf16", host_lens=True)


def test_layers_more_than_one_launch(hb):
    """70 layers: the per-layer operands travel as kernel parameters, 64 layers per launch."""
    rng = np.random.default_rng(70)
    B, q_len, Hq, Hkv, D = 1, 4, 4, 1, 64
    lens = [1500]
    q, k, v = layer_inputs(rng, 70, B, q_len, Hq, Hkv, D, lens, "bf16")
    check_layers(hb, q, k, v, lens, "bf16", shuffle_seed=None)


def test_layers_shapes_outside_the_kernel_run_layer_by_layer(hb):
    rng = np.random.default_rng(5)
    lens = [300, 77]
    q, k, v = layer_inputs(rng, 3, 2, 5, 4, 2, 64, lens, "fp32")        # fp32: CUDA-core path per layer
    check_layers(hb, q, k, v, lens, "fp32")
    q, k, v = layer_inputs(rng, 3, 2, 1, 8, 2, 64, lens, "bf16")        # few rows, short cache: the low-latency path
    check_layers(hb, q, k, v, lens, "bf16")


def test_layers_full_size_long_video(hb):
    """c2 at full size, five layers: every (token, head) row of every layer against the oracle."""
    cfg = W.CONFIGS[2]
    q_len = cfg.gamma + 1
    lens = [W.visual_lengths(cfg)[0] + cfg.n_text + q_len]
    n_layers = 5
    inps = [W.attention_inputs(cfg, "target", lens, q_len, layer=l) for l in range(n_layers)]
    q, k, v = (np.stack([i[x] for i in inps]) for x in ("q", "k", "v"))
    check_layers(hb, q, k, v, lens, "bf16", shuffle_seed=None)


def test_layers_c3_batched_paged(hb):
    cfg = W.CONFIGS[3]
    q_len = cfg.gamma + 1
    lens = [n + cfg.n_text + q_len for n in W.visual_lengths(cfg)]
    n_layers = 4
    inps = [W.attention_inputs(cfg, "target", lens, q_len, layer=l) for l in range(n_layers)]
    q, k, v = (np.stack([i[x] for i in inps]) for x in ("q", "k", "v"))
    check_layers(hb, q, k, v, lens, "bf16", shuffle_seed=33, host_lens=True, want_lse=False)


def test_layers_argument_validation(hb):
    rng = np.random.default_rng(1)
    lens = [200]
    q, k, v = layer_inputs(rng, 2, 1, 4, 4, 2, 64, lens, "bf16")
    caches = layer_caches(hb, k, v, lens, "bf16", 3)
    other_table = hb.KVCache(caches[1].k_pages, caches[1].v_pages, caches[1].page_table.clone())
    qs = [dev(q[l], "bf16") for l in range(2)]
    outs = [torch.empty_like(t) for t in qs]
    with pytest.raises(hb.HippoError) as e:
        hb.hippo_verify_attention_layers(qs, [caches[0], other_table], dev(np.asarray(lens, np.int32)), 200, outs)
    assert e.value.status == hb.HIPPO_ERR_INVALID_ARG
    with pytest.raises(hb.HippoError) as e:
        hb.hippo_verify_attention_layers(qs, caches, dev(np.asarray(lens, np.int32)), 200, outs,
                                         workspace=hb.new_workspace(4096))
    assert e.value.status == hb.HIPPO_ERR_WORKSPACE_TOO_SMALL


# ---- the time-out path ----------------------------------------------------------------------------------------------

def small_case(rng, B, q_len, Hq, Hkv, D, lens):
    q = W.round_to_storage(rng.standard_normal((B, q_len, Hq, D)).astype(np.float32), "bf16")
    k = W.round_to_storage(rng.standard_normal((B, max(lens), Hkv, D)).astype(np.float32), "bf16")
    v = W.round_to_storage(rng.standard_normal((B, max(lens), Hkv, D)).astype(np.float32), "bf16")
    return q, k, v


@pytest.mark.parametrize("mode", ["cluster", "split", "layers"])
def test_bounded_wait_runs_out_and_the_workspace_recovers(hb, mode):
    """The wait limit of the workspace is set to 200 ns, less than any load from memory takes: the first wait of a
    healthy kernel gives up.  Nothing is stuck - every load still lands and the exit waits keep their own limit - so the
    kernel returns, the status word says HIPPO_ERR_TIMEOUT, a reset clears it and the next call matches the oracle."""
    from gpu_util import paged_cache
    rng = np.random.default_rng(12)
    B, q_len, Hq, Hkv, D = 2, 6, 8, 2, 128
    lens = [3000, 2100]
    q, k, v = small_case(rng, B, q_len, Hq, Hkv, D, lens)
    kvl = dev(np.asarray(lens, np.int32))
    if mode == "layers":
        n_layers = 4
        qs, ks, vs = (np.stack([x] * n_layers) for x in (q, k, v))
        caches = layer_caches(hb, ks, vs, lens, "bf16", 5)
        q_d = [dev(q, "bf16") for _ in range(n_layers)]
        outs = [torch.empty_like(t) for t in q_d]
        ws = hb.new_workspace(hb.hippo_verify_attention_layers_workspace_bytes(n_layers, B, q_len, Hq, Hkv, D))
        call = lambda: hb.hippo_verify_attention_layers(q_d, caches, kvl, max(lens), outs, workspace=ws)
        result = lambda: host(outs[-1])
    else:
        kv, _, _ = paged_cache(hb, k, v, lens, "bf16", shuffle_seed=5)
        q_d = dev(q, "bf16")
        out = torch.empty_like(q_d)
        ws = hb.new_workspace(hb.hippo_attention_workspace_bytes(B, q_len, Hq, Hkv, D))
        splits = 0 if mode == "cluster" else 3
        call = lambda: hb.hippo_verify_attention(q_d, kv, kvl, max(lens), num_splits=splits, out=out, workspace=ws)
        result = lambda: host(out)
    call()
    assert hb.hippo_workspace_status(ws) == hb.HIPPO_OK
    hb.hippo_workspace_set_wait_limit(ws, 200)
    call()
    assert hb.hippo_workspace_status(ws) == hb.HIPPO_ERR_TIMEOUT
    assert b"gave up" in hb.lib.hippo_last_error()
    call()                                                  # the status word is sticky until the reset
    assert hb.hippo_workspace_status(ws) == hb.HIPPO_ERR_TIMEOUT
    hb.hippo_workspace_reset(ws)
    assert hb.hippo_workspace_status(ws) == hb.HIPPO_OK
    call()
    assert hb.hippo_workspace_status(ws) == hb.HIPPO_OK
    ref, _ = oracle.attention(q, k, v, lens)
    assert_close(result(), ref, TOL["bf16"], "after the reset")


def test_bf16_batch_beyond_the_tensor_core_limit(hb):
    """bf16 with more than 256 sequences is outside the tensor-core kernel's tables and runs on the CUDA-core path."""
    from gpu_util import paged_cache
    rng = np.random.default_rng(77)
    B, q_len, Hq, Hkv, D = 300, 2, 4, 2, 64
    lens = [int(x) for x in rng.integers(q_len, 200, size=B)]
    q, k, v = small_case(rng, B, q_len, Hq, Hkv, D, lens)
    kv, _, _ = paged_cache(hb, k, v, lens, "bf16", shuffle_seed=1)
    out = hb.hippo_verify_attention(dev(q, "bf16"), kv, dev(np.asarray(lens, np.int32)), max(lens))
    torch.cuda.synchronize()
    ref, _ = oracle.attention(q, k, v, lens)
    assert_close(host(out), ref, TOL["bf16"], "batch 300")


def test_host_lengths_only_plan_the_launch(hb):
    """A ragged batch with and without the host copy of its lengths: a different work split may be chosen, the results
    match the oracle either way."""
    from gpu_util import paged_cache
    rng = np.random.default_rng(9)
    B, q_len, Hq, Hkv, D = 8, 6, 28, 4, 128
    lens = [int(x) for x in rng.integers(3000, 9000, size=B)]
    q, k, v = small_case(rng, B, q_len, Hq, Hkv, D, lens)
    kv, _, _ = paged_cache(hb, k, v, lens, "bf16", shuffle_seed=4)
    qd, kvl = dev(q, "bf16"), dev(np.asarray(lens, np.int32))
    ref, _ = oracle.attention(q, k, v, lens)
    for hl in (None, lens):
        out = hb.hippo_verify_attention(qd, kv, kvl, max(lens), kv_len_host=hl)
        torch.cuda.synchronize()
        assert_close(host(out), ref, TOL["bf16"], "host lengths %s" % (hl is not None))
