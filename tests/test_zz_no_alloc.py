"""hippo_accept_noalloc: the acceptance step for callers that cannot allocate a workspace.

Such callers exist: a serving engine that took all device memory for its own pool, a decode loop in which a
cudaMalloc would stall every stream, a plug-in that only receives the logits.  The entry point keeps its scratch in
an array built into the library, so the only thing to check is that it decides exactly as hippo_accept does - on
two calls in a row with different inputs, because the second call finds the first call's leftovers in the array -
and that it refuses problems whose scratch would not fit instead of overrunning the array.

This file is named so that pytest collects it last.
"""
import numpy as np
import pytest
import torch

from gpu_util import dev, host
from paper_2601_08273_b200 import workloads as W

pytestmark = pytest.mark.gpu


def test_noalloc_matches_hippo_accept_twice_in_a_row():
    from paper_2601_08273_b200 import binding as hb
    cfg = W.CONFIGS[1]
    # two different problems, the second smaller than the first so that stale words of the first stay in the array
    cases = [W.accept_inputs(cfg, batch=3, corr_eps=0.3, sub=11), W.accept_inputs(cfg, batch=2, gamma=3, vocab=40001, corr_eps=0.1, sub=12)]
    names = ("target_logits", "draft_logits", "draft_tokens", "u_accept", "u_resample")
    for inp in cases:
        args = [dev(inp[k]) for k in names]
        B, g1, _ = inp["target_logits"].shape
        want_n, want_tok = hb.hippo_accept(*args)
        got_n = torch.full((B,), -7, dtype=torch.int32, device="cuda")
        got_tok = torch.full((B, g1), -7, dtype=torch.int32, device="cuda")
        torch.cuda.synchronize()
        before = torch.cuda.memory_allocated()
        hb.hippo_accept_noalloc(*args, got_n, got_tok)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == before
        # integer results: bit-exact agreement with the workspace variant
        np.testing.assert_array_equal(host(got_n), host(want_n))
        np.testing.assert_array_equal(host(got_tok), host(want_tok))
        assert (host(got_n) >= 0).all() and (host(got_n) <= g1 - 1).all()


def test_noalloc_calls_back_to_back_on_one_stream():
    """Three different problems enqueued on one stream with no synchronisation in between - sampling, no draft tokens at
    all (gamma = 0), greedy - all sharing the built-in array: stream order alone must keep them apart.  Checked after a
    single synchronisation against hippo_accept with its own workspaces."""
    from paper_2601_08273_b200 import binding as hb
    cfg = W.CONFIGS[1]
    names = ("target_logits", "draft_logits", "draft_tokens", "u_accept", "u_resample")
    a = W.accept_inputs(cfg, batch=4, corr_eps=0.2, sub=21)
    b = W.accept_inputs(cfg, batch=3, gamma=0, vocab=9001, sub=22)
    c = W.accept_inputs(cfg, batch=5, gamma=4, vocab=50001, corr_eps=0.0, sub=23)
    c["draft_tokens"] = c["target_logits"][:, :4].argmax(axis=-1).astype(np.int32)
    c["draft_tokens"][2, 1] += 1
    dev_in = [[dev(x[k]) for k in names] for x in (a, b, c)]
    modes = (hb.HIPPO_ACCEPT_SAMPLE, hb.HIPPO_ACCEPT_SAMPLE, hb.HIPPO_ACCEPT_GREEDY)
    want = [hb.hippo_accept(*args, mode=m) for args, m in zip(dev_in, modes)]
    got = [(torch.full((x["target_logits"].shape[0],), -7, dtype=torch.int32, device="cuda"),
            torch.full(x["target_logits"].shape[:2], -7, dtype=torch.int32, device="cuda")) for x in (a, b, c)]
    torch.cuda.synchronize()
    for rep in range(2):
        for args, m, (gn, gt) in zip(dev_in, modes, got):
            hb.hippo_accept_noalloc(*args, gn, gt, mode=m)
    torch.cuda.synchronize()
    for (wn, wt), (gn, gt) in zip(want, got):
        np.testing.assert_array_equal(host(gn), host(wn))
        np.testing.assert_array_equal(host(gt), host(wt))
    assert host(got[2][0]).tolist() == [4, 4, 1, 4, 4]


def test_noalloc_refuses_sizes_beyond_its_array():
    from paper_2601_08273_b200 import binding as hb
    B, g, V = 64, 8, 152064
    assert hb.hippo_accept_workspace_bytes(B, g, V) > hb.ACCEPT_NOALLOC_SCRATCH_BYTES
    # validation happens on the host before anything is launched, so small stand-in buffers are enough
    tiny = torch.zeros(16, dtype=torch.float32, device="cuda")
    tok = torch.zeros(16, dtype=torch.int32, device="cuda")
    rc = hb.lib.hippo_accept_noalloc(B, g, V, tiny.data_ptr(), tiny.data_ptr(), tok.data_ptr(), tiny.data_ptr(),
                                     tiny.data_ptr(), 0, tok.data_ptr(), tok.data_ptr(), None)
    assert rc == hb.HIPPO_ERR_WORKSPACE_TOO_SMALL
    assert b"built-in array" in hb.lib.hippo_last_error()
    # the largest batched configuration of the workloads fits
    assert hb.hippo_accept_workspace_bytes(8, 8, V) <= hb.ACCEPT_NOALLOC_SCRATCH_BYTES
