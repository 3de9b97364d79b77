"""Decoding rounds of video parallel speculative decoding (Section 5.2) over the library's kernels.

The schedule comes from the library's host-side scheduler (`hippo_vpsd_plan` / `hippo_vpsd_commit`); this module
only launches what a round's plan says: draft attention calls on one CUDA stream, verification attention and
`hippo_accept` on another, then one device-to-host read of the accepted count.  There are no models here: the query
tensors and the logits are synthetic (seeded), positions do not advance (every round reads the same caches), and a
"draft token" is `draft_layers` draft-attention calls.  What is real is the overlap pattern, the per-round
verification length, the abort of a conservative round, and the acceptance kernel's verdicts that drive the mode
switch.  Batch size 1, as in the paper.
"""
from __future__ import annotations

import dataclasses
import time
from typing import Dict, List, Optional

import torch

from . import binding as hb
from . import workloads as W
from .step import HippoStep, _randn


class VpsdLoop:
    def __init__(self, cfg: W.HippoConfig, target_layers: Optional[int] = None, draft_layers: Optional[int] = None,
                 buffered: int = 0, pool: int = 8, draft_noise: float = 1.0, use_graphs: bool = True, device="cuda",
                 verify_max_ctas: int = 0, gamma: Optional[int] = None, draft_num_splits: Optional[int] = None):
        assert cfg.batch == 1, "the schedule is per sequence; the driver runs one sequence"
        if gamma is not None:
            cfg = dataclasses.replace(cfg, gamma=gamma)
        self.cfg = cfg
        # Sharing one GPU between the two legs of a round.  The verification kernel keeps its CTAs for the whole pass and a
        # draft call is a wave of CTAs of its own, so the legs overlap only when both fit: verify_max_ctas > 0 bounds the
        # verification grid, and draft_num_splits (CTAs per (sequence, KV head) of a draft call over a long pruned cache)
        # sizes a draft call for the SMs that leaves free.  Left alone, a 148-CTA verification pass makes the draft
        # stream wait for its end and the round costs the sum of the legs.
        self.verify_max_ctas = verify_max_ctas
        self.st = HippoStep(cfg, device=device, target_layers=target_layers, draft_layers=draft_layers)
        if draft_num_splits is not None:
            self.st.draft_num_splits = draft_num_splits
        st, g = self.st, cfg.gamma
        self.dev = st.device
        self.max_batch = max(g, buffered)
        G = cfg.tgt_q_heads // cfg.tgt_kv_heads
        assert (self.max_batch + 1) * G <= 128, "verification batch exceeds the packed-row limit"
        assert st.ctx[0] + self.max_batch + 1 <= st.tgt_cache[0].struct.max_pages_per_seq * hb.PAGE_SIZE, \
            "the target cache has no room for the largest verification batch"
        gen = torch.Generator(device=self.dev)
        gen.manual_seed(3000 + cfg.seed)
        mb = self.max_batch
        # verification queries for up to max_batch + 1 rows; kv_len per batch size
        self.q_t = _randn((st.Lt, 1, mb + 1, cfg.tgt_q_heads, cfg.tgt_head_dim), st.tdt, gen, self.dev)
        self.out_t = torch.empty_like(self.q_t)
        self.kv_len_t = {c: torch.tensor([st.ctx[0] + c + 1], dtype=torch.int32, device=self.dev) for c in range(1, mb + 1)}
        self.verify_ws = hb.new_workspace(hb.hippo_verify_attention_layers_workspace_bytes(
            st.Lt, 1, mb + 1, cfg.tgt_q_heads, cfg.tgt_kv_heads, cfg.tgt_head_dim), self.dev)
        # acceptance inputs: a pool of rounds; draft logits = target logits + noise, draft tokens drawn from them
        V = cfg.vocab
        self.pool = []
        for _ in range(pool):
            tl = torch.randn((1, mb + 1, V), device=self.dev, generator=gen) * cfg.logit_sigma
            dl = tl[:, :mb] + draft_noise * torch.randn((1, mb, V), device=self.dev, generator=gen)
            tok = torch.multinomial(torch.softmax(dl[0], dim=-1), 1, generator=gen).to(torch.int32).reshape(1, mb)
            self.pool.append({"target_logits": tl.contiguous(), "draft_logits": dl.contiguous(), "draft_tokens": tok.contiguous(),
                              "u_accept": torch.rand((1, mb), device=self.dev, generator=gen),
                              "u_resample": torch.rand((1,), device=self.dev, generator=gen)})
        self.n_accepted = torch.zeros(1, dtype=torch.int32, device=self.dev)
        self.n_host = torch.zeros(1, dtype=torch.int32).pin_memory()
        self.out_tokens = torch.empty((1, mb + 1), dtype=torch.int32, device=self.dev)
        self.accept_ws = hb.new_workspace(hb.hippo_accept_workspace_bytes(1, mb, V), self.dev)
        self.stream_d, self.stream_v = st.stream_d, st.stream_v
        # One draft token (draft_layers launches) is launch-bound when issued call by call from one host thread, which
        # would serialise the two streams on the host: it is captured once into a CUDA graph and replayed, and so is the
        # verification pass of each batch size.
        self.g_draft = {}
        self.g_verify = {}
        if use_graphs:
            for jj in range(g):
                self.g_draft[jj] = self._capture(lambda s, jj=jj: self._draft_token_eager(jj, s))
            for c in range(1, mb + 1):
                self.g_verify[c] = self._capture(lambda s, c=c: self._verify_eager(c, s))

    def _capture(self, fn):
        side = torch.cuda.Stream(device=self.dev)
        side.wait_stream(torch.cuda.current_stream(self.dev))
        with torch.cuda.stream(side):
            fn(side)                                   # warm-up: one-time set-up inside the library happens here
        torch.cuda.current_stream(self.dev).wait_stream(side)
        torch.cuda.synchronize(self.dev)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            fn(torch.cuda.current_stream(self.dev))
        return graph

    # ---- launches -------------------------------------------------------------------------------------------------
    def _draft_token_eager(self, jj: int, stream) -> None:
        st = self.st
        for l in range(st.Ld):
            hb.hippo_draft_attention(st.q_d[l, jj], st.dst_cache[l], st.kv_len_d[jj], st.max_kv_d[jj],
                                     out=st.out_d[l, jj], workspace=st.draft_ws, stream=stream,
                                     num_splits=st.draft_num_splits)

    def _verify_eager(self, c: int, stream) -> None:
        st = self.st
        # the verification pass: every target layer's attention in one launch
        hb.hippo_verify_attention_layers([self.q_t[l][:, :c + 1] for l in range(st.Lt)], st.tgt_cache, self.kv_len_t[c],
                                         st.ctx[0] + c + 1, [self.out_t[l][:, :c + 1] for l in range(st.Lt)],
                                         workspace=self.verify_ws, stream=stream, kv_len_host=[st.ctx[0] + c + 1],
                                         max_ctas=self.verify_max_ctas)

    def draft_token(self, j: int, stream) -> None:
        jj = j % self.cfg.gamma
        if jj in self.g_draft:
            with torch.cuda.stream(stream):
                self.g_draft[jj].replay()
        else:
            self._draft_token_eager(jj, stream)

    def verify_and_accept(self, c: int, pool_idx: int, stream) -> None:
        if c in self.g_verify:
            with torch.cuda.stream(stream):
                self.g_verify[c].replay()
        else:
            self._verify_eager(c, stream)
        a = self.pool[pool_idx % len(self.pool)]
        hb.hippo_accept(a["target_logits"][:, :c + 1], a["draft_logits"][:, :c], a["draft_tokens"][:, :c],
                        a["u_accept"][:, :c], a["u_resample"], n_accepted=self.n_accepted,
                        out_tokens=self.out_tokens[:, :c + 1], workspace=self.accept_ws, stream=stream)

    # ---- the loops ----------------------------------------------------------------------------------------------------
    def _verdict(self, c: int, pool_idx: int, stream, event) -> None:
        """Verification of c draft tokens, acceptance, and the accepted count on its way to pinned host memory."""
        self.verify_and_accept(c, pool_idx, stream)
        with torch.cuda.stream(stream):
            self.n_host.copy_(self.n_accepted, non_blocking=True)
        event.record(stream)

    def run(self, rounds: int, buffered: int = 0) -> Dict[str, object]:
        """`rounds` rounds of the adaptive schedule.  Returns counters, the per-round trace and the wall time.

        The host touches a round twice: it launches what the plan says on the two streams, and it waits for the
        verdict (one event, four bytes in pinned memory).  The verification stream waits on the device for the draft
        tokens it verifies; nothing else is joined."""
        state = hb.hippo_vpsd_init(self.cfg.gamma, buffered)
        sd, sv = self.stream_d, self.stream_v
        verdict, batch_ready = torch.cuda.Event(), torch.cuda.Event()
        trace: List[dict] = []
        torch.cuda.synchronize(self.dev)
        t0 = time.perf_counter()
        batch_ready.record(sd)                      # a prefill buffer is there from the start
        for r in range(rounds):
            rd = hb.hippo_vpsd_plan(state)
            for j in range(rd.draft_before):
                self.draft_token(j, sd)
            if rd.draft_before:
                batch_ready.record(sd)
            sv.wait_event(batch_ready)              # the tokens to verify have been drafted
            self._verdict(rd.verify_tokens, r, sv, verdict)
            drafted, n = 0, None
            for j in range(rd.draft_during):
                if rd.abort_on_reject:
                    # the host follows the drafting token by token and stops at a rejecting verdict
                    if verdict.query():
                        n = int(self.n_host[0])
                        if n < rd.verify_tokens:
                            break
                self.draft_token(rd.draft_before + j, sd)
                drafted += 1
                if rd.abort_on_reject:
                    sd.synchronize()
            batch_ready.record(sd)
            if n is None:
                verdict.synchronize()               # the verdict is needed to plan the next round
                n = int(self.n_host[0])
            out = hb.hippo_vpsd_commit(state, rd, n, drafted)
            trace.append({"mode": rd.mode, "batch": rd.verify_tokens, "accepted": n, "emitted": out.emitted,
                          "drafted_during": drafted})
        torch.cuda.synchronize(self.dev)
        wall = time.perf_counter() - t0
        return {"rounds": rounds, "tokens": int(state.tokens_emitted), "drafted": int(state.tokens_drafted),
                "discarded": int(state.tokens_discarded), "wall_ms": wall * 1e3, "trace": trace}

    def run_serial(self, rounds: int) -> Dict[str, object]:
        """Serial speculative decoding for comparison: gamma draft tokens, then verification, on one stream."""
        g = self.cfg.gamma
        main = torch.cuda.current_stream(self.dev)
        verdict = torch.cuda.Event()
        tokens = 0
        torch.cuda.synchronize(self.dev)
        t0 = time.perf_counter()
        for r in range(rounds):
            for j in range(g):
                self.draft_token(j, main)
            self._verdict(g, r, main, verdict)
            verdict.synchronize()
            tokens += int(self.n_host[0]) + 1
        torch.cuda.synchronize(self.dev)
        return {"rounds": rounds, "tokens": tokens, "wall_ms": (time.perf_counter() - t0) * 1e3}

    def unit_times_ms(self, reps: int = 5) -> Dict[str, float]:
        """One draft token and one verification pass (gamma tokens), each timed alone with CUDA events."""
        main = torch.cuda.current_stream(self.dev)
        def timed(fn):
            fn()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize(self.dev)
            e0.record(main)
            for _ in range(reps):
                fn()
            e1.record(main)
            torch.cuda.synchronize(self.dev)
            return e0.elapsed_time(e1) / reps
        return {"t_draft": timed(lambda: self.draft_token(0, main)),
                "t_target": timed(lambda: self.verify_and_accept(self.cfg.gamma, 0, main))}

    def shared_times_ms(self, reps: int = 5) -> Dict[str, float]:
        """The same two times with both legs of an optimistic round in flight: gamma draft tokens on the draft stream
        beside one verification pass on the other.  On one GPU the legs share the SMs and, above all, the memory system:
        a draft call is a chain of dependent memory round trips whose latency grows severalfold while the verification
        kernel keeps HBM saturated, so a round costs max(t_target, gamma * t_draft) of THESE times, not of the times
        each leg shows alone."""
        g = self.cfg.gamma
        sd, sv = self.stream_d, self.stream_v
        td, tv = [], []
        for _ in range(reps + 1):
            torch.cuda.synchronize(self.dev)
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
            go = torch.cuda.Event()
            go.record(torch.cuda.current_stream(self.dev))
            sv.wait_event(go)
            sd.wait_event(go)
            ev[0].record(sv)
            self.verify_and_accept(g, 0, sv)
            ev[1].record(sv)
            ev[2].record(sd)
            for j in range(g):
                self.draft_token(j, sd)
            ev[3].record(sd)
            torch.cuda.synchronize(self.dev)
            tv.append(ev[0].elapsed_time(ev[1]))
            td.append(ev[2].elapsed_time(ev[3]) / g)
        td, tv = sorted(td[1:]), sorted(tv[1:])
        return {"t_draft": td[len(td) // 2], "t_target": tv[len(tv) // 2]}
