"""Pins of the schedule oracle: the paper's own worked numbers (Sections 4.2 and 5.2) and timelines worked by hand
from the text of Section 5.2."""
import pytest

from oracle import vpsd as O


def test_paper_example_serial_speculative_decoding():
    # Section 4.2: target three times slower than the draft model, three draft tokens per round.
    all_ok = O.serial_sd(3, 1.0, 3.0, [3])
    assert all_ok.tokens == 4 and all_ok.time == 6.0
    assert all_ok.speedup_over_autoregressive(3.0) == pytest.approx(2.0)          # the paper's "2"
    first_bad = O.serial_sd(3, 1.0, 3.0, [0])
    assert first_bad.tokens == 1
    assert first_bad.speedup_over_autoregressive(3.0) == pytest.approx(0.5)      # the paper's "0.5"


def test_paper_example_prefill_buffer():
    # Section 5.2: 0.8 s target prefill, 0.2 s draft prefill, 50 ms per draft token: about 12 tokens
    assert O.prefill_buffer(0.8, 0.2, 0.05) == 12
    assert O.prefill_buffer(0.2, 0.8, 0.05) == 0


def test_all_accepted_hides_the_draft_model():
    # hand timeline, T_d = 1, T_t = 3, gamma = 3:
    #   round 1 (conservative): draft x1 [0,1]; verify x1 [1,4] || draft x2,x3 [1,3]  -> t = 4, emits x1
    #   round 2 (optimistic, batch x2,x3): verify [4,7] || draft 3 more [4,7]          -> t = 7, emits 2
    #   rounds 3.. (optimistic, batch 3): 3 time units, 3 tokens each
    tr = O.vpsd(3, 1.0, 3.0, [9] * 6)
    assert [r["mode"] for r in tr.rounds] == [O.CONSERVATIVE] + [O.OPTIMISTIC] * 5
    assert [r["emitted"] for r in tr.rounds] == [1, 2, 3, 3, 3, 3]
    assert [r["time"] for r in tr.rounds] == [4.0, 3.0, 3.0, 3.0, 3.0, 3.0]
    # steady state: 3 tokens per 3 units = one token per T_d: speedup T_t / T_d = 3 over autoregressive (serial SD: 2)
    steady = O.vpsd(3, 1.0, 3.0, [9] * 1000, buffered=3)
    assert steady.speedup_over_autoregressive(3.0) == pytest.approx(3.0)


def test_always_rejected_never_worse_than_one_draft_pass():
    # every x1 rejected: each round is one draft pass and one target pass, one token: 3 / 4 of autoregressive speed
    # (serial speculative decoding with gamma = 3 would be at 0.5)
    tr = O.vpsd(3, 1.0, 3.0, [0] * 50)
    assert all(r["mode"] == O.CONSERVATIVE and r["time"] == 4.0 and r["emitted"] == 1 for r in tr.rounds)
    assert tr.speedup_over_autoregressive(3.0) == pytest.approx(0.75)


def test_rejection_in_optimistic_mode_drops_the_speculative_batch():
    # batch of 3, two accepted: emits 2 + the target's replacement, next round conservative
    tr = O.vpsd(3, 1.0, 3.0, [2, 1, 3], buffered=3)
    assert [(r["mode"], r["batch"], r["accepted"], r["emitted"]) for r in tr.rounds] == [
        (O.OPTIMISTIC, 3, 2, 3), (O.CONSERVATIVE, 1, 1, 1), (O.OPTIMISTIC, 2, 2, 2)]
    assert tr.tokens == 6 and tr.time == 3.0 + 4.0 + 3.0


def test_slow_draft_model_bounds_the_round():
    # gamma * T_d > T_t: the optimistic round lasts gamma * T_d; the conservative one T_d + (gamma - 1) * T_d
    tr = O.vpsd(4, 2.0, 3.0, [1, 9], buffered=0)
    assert [r["time"] for r in tr.rounds] == [2.0 + 6.0, 8.0]


def test_prefill_buffer_is_the_first_batch_and_gamma_one():
    tr = O.vpsd(5, 1.0, 3.0, [12, 5], buffered=12)
    assert (tr.rounds[0]["mode"], tr.rounds[0]["batch"], tr.rounds[0]["emitted"]) == (O.OPTIMISTIC, 12, 12)
    assert (tr.rounds[1]["batch"], tr.rounds[1]["emitted"]) == (5, 5)
    one = O.vpsd(1, 1.0, 3.0, [1, 0])
    assert [(r["emitted"], r["time"]) for r in one.rounds] == [(2, 4.0), (1, 4.0)]
