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
