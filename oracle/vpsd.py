"""CPU oracle of the decoding schedules (Sections 3.2, 4.2 and 5.2).  TEST INFRASTRUCTURE ONLY.

Plain event-by-event simulation, in abstract time units, of
  * serial speculative decoding (Section 4.2's worked example): gamma draft passes, then one target pass;
  * video parallel speculative decoding (Section 5.2): synchronous draft-target prefill and the adaptive
    switch between the optimistic (post-verification) and the conservative (pre-verification) mode.
It shares nothing with the CUDA library or its host-side scheduler; only the tests may import it.

A verification outcome is the number of leading draft tokens the target accepts.  Outcomes are passed in as a
list `raw`: the k-th verification of c draft tokens accepts n = min(raw[k], c) of them.

Readings of Section 5.2 taken here (the paper gives no pseudo-code):
  * Optimistic round, current batch of c tokens: the target verifies the batch while the draft model produces the
    next gamma tokens; the round lasts max(T_t, gamma * T_d).  All accepted: the c tokens are emitted (the target's
    bonus token is not, the draft has already continued past it), the freshly drafted batch becomes current, the
    mode stays optimistic.  Rejection after n < c tokens: n + 1 tokens are emitted (the accepted ones and the
    target's replacement), the speculative batch is dropped, the mode becomes conservative.
  * Conservative round: the draft model produces x_1 (T_d); then the target verifies x_1 while the draft model
    produces x_2..x_gamma.  x_1 rejected: drafting is aborted when the verdict arrives, the round lasts
    T_d + T_t, one token (the replacement) is emitted, the mode stays conservative.  x_1 accepted: the round
    lasts T_d + max(T_t, (gamma - 1) * T_d), x_1 is emitted, x_2..x_gamma become the current batch of an
    optimistic round ("proceed to standard verification"); with gamma = 1 nothing is left, the target's bonus
    token is emitted too and the mode stays conservative.
  * Synchronous prefill: the draft model decodes while the target prefills, floor((P_t - P_d) / T_d) tokens; a
    non-empty buffer is the current batch of a first optimistic round.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Sequence

OPTIMISTIC, CONSERVATIVE = 0, 1


def prefill_buffer(p_target: float, p_draft: float, t_draft: float) -> int:
    """Draft tokens decoded while the target model is still prefilling."""
    if p_target <= p_draft:
        return 0
    return int(math.floor((p_target - p_draft) / t_draft + 1e-9))


@dataclass
class Trace:
    time: float = 0.0
    tokens: int = 0
    rounds: List[dict] = field(default_factory=list)

    def speedup_over_autoregressive(self, t_target: float) -> float:
        return self.tokens * t_target / self.time


def serial_sd(gamma: int, t_draft: float, t_target: float, raw: Sequence[int]) -> Trace:
    """gamma draft passes, one target pass, n + 1 tokens per round (accepted tokens and the target's own)."""
    tr = Trace()
    for r in raw:
        n = min(int(r), gamma)
        tr.time += gamma * t_draft + t_target
        tr.tokens += n + 1
        tr.rounds.append({"mode": None, "batch": gamma, "accepted": n, "emitted": n + 1,
                          "time": gamma * t_draft + t_target})
    return tr


def vpsd(gamma: int, t_draft: float, t_target: float, raw: Sequence[int], buffered: int = 0) -> Trace:
    """The adaptive schedule; one entry of `raw` is consumed per round."""
    tr = Trace()
    mode, batch = (OPTIMISTIC, buffered) if buffered > 0 else (CONSERVATIVE, 0)
    for r in raw:
        if mode == OPTIMISTIC:
            n = min(int(r), batch)
            dt = max(t_target, gamma * t_draft)
            if n == batch:
                emitted, nxt_mode, nxt_batch = batch, OPTIMISTIC, gamma
            else:
                emitted, nxt_mode, nxt_batch = n + 1, CONSERVATIVE, 0
            tr.rounds.append({"mode": OPTIMISTIC, "batch": batch, "accepted": n, "emitted": emitted, "time": dt})
        else:
            n = min(int(r), 1)
            if n == 0:
                dt, emitted, nxt_mode, nxt_batch = t_draft + t_target, 1, CONSERVATIVE, 0
            elif gamma == 1:
                dt, emitted, nxt_mode, nxt_batch = t_draft + t_target, 2, CONSERVATIVE, 0
            else:
                dt = t_draft + max(t_target, (gamma - 1) * t_draft)
                emitted, nxt_mode, nxt_batch = 1, OPTIMISTIC, gamma - 1
            tr.rounds.append({"mode": CONSERVATIVE, "batch": 1, "accepted": n, "emitted": emitted, "time": dt})
        tr.time += dt
        tr.tokens += emitted
        mode, batch = nxt_mode, nxt_batch
    return tr
