"""GPU: the decoding loop (Section 5.2 schedule over the real kernels) behaves as the schedule oracle says when the
oracle is fed the verdicts the acceptance kernel produced, and those verdicts equal the acceptance oracle's."""
import numpy as np
import pytest
import torch

import oracle
from oracle import vpsd as O
from paper_2601_08273_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def loop():
    from paper_2601_08273_b200.vpsd import VpsdLoop
    cfg = W.CONFIGS[1].replace(frames=8, vocab=4096)
    return VpsdLoop(cfg, target_layers=2, draft_layers=2, buffered=9, pool=6, draft_noise=1.5)


def test_loop_follows_the_schedule(loop):
    g = loop.cfg.gamma
    for buffered in (0, 9):
        res = loop.run(24, buffered=buffered)
        tr = res["trace"]
        ref = O.vpsd(g, 1.0, 3.0, [t["accepted"] for t in tr], buffered=buffered)
        assert [(t["mode"], t["batch"], t["emitted"]) for t in tr] == [(r["mode"], r["batch"], r["emitted"]) for r in ref.rounds]
        assert res["tokens"] == ref.tokens
        # an aborted conservative round drafted less than planned only when x_1 was rejected
        for t in tr:
            if t["mode"] == O.CONSERVATIVE and t["accepted"] == 1:
                assert t["drafted_during"] == g - 1
        assert any(t["mode"] == O.OPTIMISTIC for t in tr) and any(t["mode"] == O.CONSERVATIVE for t in tr)


def test_verdicts_equal_the_acceptance_oracle(loop):
    for idx, c in ((0, 5), (1, 1), (2, 9), (3, 3)):
        a = loop.pool[idx]
        loop.verify_and_accept(c, idx, torch.cuda.current_stream())
        torch.cuda.synchronize()
        n_ref, tok_ref, _, _ = oracle.accept(a["target_logits"][:, :c + 1].cpu().numpy(), a["draft_logits"][:, :c].cpu().numpy(),
                                             a["draft_tokens"][:, :c].cpu().numpy(), a["u_accept"][:, :c].cpu().numpy(),
                                             a["u_resample"].cpu().numpy())[:4]
        assert int(loop.n_accepted.item()) == int(n_ref[0])
        np.testing.assert_array_equal(loop.out_tokens[:, :c + 1].cpu().numpy(), tok_ref)


def test_serial_loop_counts_tokens(loop):
    res = loop.run_serial(6)
    assert 6 <= res["tokens"] <= 6 * (loop.cfg.gamma + 1)
