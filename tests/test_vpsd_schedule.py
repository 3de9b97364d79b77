"""The library's host-side schedule (hippo_vpsd_*, Section 5.2) against the schedule oracle, round by round, on
seeded outcome streams; runs without a GPU (the functions are host-only)."""
import numpy as np
import pytest

from oracle import vpsd as O


@pytest.fixture(scope="module")
def hb():
    from paper_2601_08273_b200 import binding
    return binding


def run_library(hb, gamma, t_d, t_t, raw, buffered):
    st = hb.hippo_vpsd_init(gamma, buffered)
    rounds, total = [], 0.0
    for r in raw:
        rd = hb.hippo_vpsd_plan(st)
        n = min(int(r), rd.verify_tokens)
        # a conservative round whose x_1 is rejected stops drafting; how far it got does not change the outcome
        drafted = rd.draft_during if n == rd.verify_tokens else (rd.draft_during // 2 if rd.abort_on_reject else rd.draft_during)
        dt = hb.hippo_vpsd_round_time(rd, n, t_d, t_t)
        out = hb.hippo_vpsd_commit(st, rd, n, drafted)
        rounds.append({"mode": rd.mode, "batch": rd.verify_tokens, "accepted": n, "emitted": out.emitted, "time": dt})
        total += dt
    return st, rounds, total


@pytest.mark.parametrize("gamma,t_d,t_t,buffered,seed", [(3, 1.0, 3.0, 0, 1), (5, 1.0, 3.0, 12, 2), (8, 0.7, 2.0, 3, 3),
                                                         (1, 1.0, 3.0, 0, 4), (4, 2.0, 3.0, 0, 5), (7, 1.0, 9.0, 20, 6)])
def test_matches_oracle_round_by_round(hb, gamma, t_d, t_t, buffered, seed):
    rng = np.random.default_rng(seed)
    # geometric-like outcomes: long accepted runs and early rejections both occur
    raw = [int(x) for x in rng.geometric(0.25, size=400) - 1]
    ref = O.vpsd(gamma, t_d, t_t, raw, buffered=buffered)
    st, rounds, total = run_library(hb, gamma, t_d, t_t, raw, buffered)
    assert rounds == ref.rounds
    assert st.tokens_emitted == ref.tokens and total == pytest.approx(ref.time)
    assert st.rounds == len(raw)
    # every drafted token is emitted, discarded or still waiting; target tokens are the rest of the output
    assert st.tokens_drafted >= st.tokens_discarded + st.batch


def test_paper_numbers_through_the_library(hb):
    assert hb.hippo_vpsd_prefill_buffer(0.8, 0.2, 0.05) == 12                      # Section 5.2
    assert hb.hippo_vpsd_serial_round_time(3, 1.0, 3.0) == 6.0                     # Section 4.2: 4 tokens -> x2, 1 token -> x0.5
    st, rounds, total = run_library(hb, 3, 1.0, 3.0, [9] * 1000, 3)
    assert st.tokens_emitted * 3.0 / total == pytest.approx(3.0)


def test_argument_errors(hb):
    with pytest.raises(hb.HippoError):
        hb.hippo_vpsd_init(0)
    st = hb.hippo_vpsd_init(4)
    rd = hb.hippo_vpsd_plan(st)
    with pytest.raises(hb.HippoError):
        hb.hippo_vpsd_commit(st, rd, 2)            # more accepted than verified
    with pytest.raises(hb.HippoError):
        hb.hippo_vpsd_commit(st, rd, 1, 1)         # all accepted but drafting stopped early
    out = hb.hippo_vpsd_commit(st, rd, 1)
    assert (out.emitted, out.keep_drafted, out.next_mode) == (1, 3, hb.HIPPO_VPSD_OPTIMISTIC)
    with pytest.raises(hb.HippoError):
        hb.hippo_vpsd_commit(st, rd, 0)            # stale round: the state has moved on
