#!/usr/bin/env python
"""Benchmark of the HIPPO hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 1] [--impl ours|reference] [--no-graph] [--no-extra]

A step is one pass of the whole hot path over one batch of synthetic input: select -> gather -> (gamma x draft
layers of draft attention on one stream || target layers of verify attention on another) -> accept.  The metric
is the verification leg's KV-read bandwidth: target-KV bytes attended per step / device time of the step's
verify launches (CUDA events on the stream that launches them).  One JSON line is printed by rank 0.

N > 1 (launched by torch.distributed.run) runs N independent replicas, one per GPU: the path has no exchange
step, so there is no data-path collective; only the barrier and the max-over-ranks of the timings use NCCL.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "verify_kv_read_gbps"
UNIT = "GB/s"


# DRAM traffic of the dominant kernel per launch (dram__bytes_read.sum + dram__bytes_write.sum from one ncu capture of
# the workload named by the key); valid only for the kernel source it was taken on, identified by its hash.
NCU_TRAFFIC = {"source": "paper_2601_08273_b200/csrc/attn_tc.cu", "sha1_12": "a4d33593d3d2",
               "bytes_per_launch": {"c1_7b_video_6k": 13384704, "c2_long_video_32k": 139255552}}


def measured_traffic(workload):
    import hashlib
    try:
        with open(os.path.join(ROOT, NCU_TRAFFIC["source"]), "rb") as f:
            h = hashlib.sha1(f.read()).hexdigest()[:12]
    except OSError:
        return None
    if h != NCU_TRAFFIC["sha1_12"]:
        return None   # the kernel has changed since the counters were taken
    return NCU_TRAFFIC["bytes_per_launch"].get(workload)


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), "measured (MEASURED_PEAKS.json copy probe)"
    return 6650.0, "fallback (earlier measurement on this pool)"


# ---- clocks ---------------------------------------------------------------------------------------------------------

class ClockSampler:
    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_uuid: str):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", gpu_uuid, "--query-gpu=" + self.Q, "--format=csv,noheader,nounits",
                                       "-lms", "100"], stdout=self.f, stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None
        self.marks = []

    def mark(self):
        self.marks.append(time.time())

    def stop(self):
        if self.p is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        rows = [l.strip().split(", ") for l in self.f if l.strip()]
        self.f.close()
        os.unlink(self.f.name)
        import datetime
        sm, mx, power, reasons = [], [], [], set()
        lo, hi = (self.marks[0], self.marks[-1]) if len(self.marks) >= 2 else (0, float("inf"))
        for r in rows:
            if len(r) < 9:
                continue
            try:
                ts = datetime.datetime.strptime(r[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                if not (lo - 0.05 <= ts <= hi + 0.05):
                    continue
                sm.append(float(r[1])); mx.append(float(r[2])); power.append(float(r[3]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[5:9]):
                if val.strip() == "Active":
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples inside the timed region"], "samples": 0}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "power_w_max": max(power),
                "reasons": sorted(reasons), "samples": len(sm)}


# ---- reference arm: the CPU oracle on the host cores ------------------------------------------------------------------

def oracle_verify_sample(cfg, layers):
    """Times the oracle's verify attention on `layers` layers of the config (all rows). Returns (seconds, bytes)."""
    import oracle
    from paper_2601_08273_b200 import workloads as W
    n_v = W.visual_lengths(cfg)
    q_len = cfg.gamma + 1
    lens = [n + cfg.n_text + q_len for n in n_v]
    elem = 4 if cfg.dtype == "fp32" else 2
    total_s, total_b = 0.0, 0
    for l in range(layers):
        inp = W.attention_inputs(cfg, "target", lens, q_len, layer=l)
        t0 = time.perf_counter()
        oracle.attention(inp["q"], inp["k"], inp["v"], lens)
        total_s += time.perf_counter() - t0
        total_b += sum(lens) * 2 * cfg.tgt_kv_heads * cfg.tgt_head_dim * elem
    return total_s, total_b


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2601_08273_b200 import workloads as W
    cfg = W.CONFIGS[args.config]
    steps = args.steps if args.steps is not None else 5
    warmup = args.warmup if args.warmup is not None else 1
    for _ in range(warmup):
        oracle_verify_sample(cfg, 1)
    secs, nbytes = 0.0, 0
    for _ in range(steps):
        s, b = oracle_verify_sample(cfg, 1)
        secs += s
        nbytes += b
    val = nbytes / secs / 1e9
    sample = "oracle verify attention, 1 of %d target layers of %s per step (all %d rows), fp64" % (
        cfg.tgt_layers, cfg.name, (cfg.gamma + 1) * cfg.tgt_q_heads)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
        "warmup": warmup, "ms_per_step": secs / steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": {"workload": cfg.name},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": oracle.max_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


# ---- our arm --------------------------------------------------------------------------------------------------------

def timed(fn, n, stream, torch):
    """n back-to-back calls of fn bracketed by events on `stream`; returns total milliseconds."""
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record(stream)
    for _ in range(n):
        fn()
    e1.record(stream)
    torch.cuda.synchronize()
    return e0.elapsed_time(e1)


def try_graph(fn, torch):
    """Capture fn() into a CUDA graph; returns a replay callable or None."""
    try:
        g = torch.cuda.CUDAGraph()
        s = torch.cuda.Stream()
        s.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(s):
            fn()
        torch.cuda.current_stream().wait_stream(s)
        torch.cuda.synchronize()
        with torch.cuda.graph(g):
            fn()
        torch.cuda.synchronize()
        g.replay()
        torch.cuda.synchronize()
        return g.replay
    except Exception as e:  # noqa: BLE001 - capture is an optimisation; eager launches are the fallback
        sys.stderr.write("graph capture failed (%s); timing eager launches\n" % e)
        torch.cuda.synchronize()
        return None


def kernel_sweep(cfg, torch, hb, HippoStep, peak, passes=3, max_gb=24.0):
    """Per-call timings and the whole step of one configuration (distinct KV buffers per layer)."""
    from paper_2601_08273_b200 import workloads as W
    per_layer = sum(n + cfg.n_text + cfg.gamma + 1 for n in W.visual_lengths(cfg)) * 2 * cfg.tgt_kv_heads * cfg.tgt_head_dim * 2
    layers = max(1, min(cfg.tgt_layers, int(max_gb * 1e9 / per_layer)))
    st = HippoStep(cfg, target_layers=layers, draft_layers=min(cfg.dft_layers, 28))
    cur = torch.cuda.current_stream()
    for _ in range(3):
        st.verify(cur)
    replay = try_graph(lambda: st.verify(torch.cuda.current_stream()), torch)
    run = replay if replay is not None else (lambda: st.verify(cur))
    ms = timed(run, passes, cur, torch) / (passes * layers)
    out = {"workload": cfg.name, "verify_layers_timed": layers, "verify_us_per_layer": ms * 1e3,
           "verify_kv_mb_per_layer": st.verify_kv_bytes_per_layer() / 1e6,
           "verify_gbps": st.verify_kv_bytes_per_layer() / ms / 1e6,
           "verify_frac_of_measured_peak": st.verify_kv_bytes_per_layer() / ms / 1e6 / peak}
    st.select(cur); st.gather(cur)
    for _ in range(3):
        st.gather(cur)
    gms = timed(lambda: st.gather(cur), 10, cur, torch) / 10
    out.update({"gather_us": gms * 1e3, "gather_mb_per_launch": st.gather_bytes() / 1e6,
                "gather_gbps": st.gather_bytes() / gms / 1e6, "gather_frac_of_measured_peak": st.gather_bytes() / gms / 1e6 / peak})
    sms = timed(lambda: st.select(cur), 3, cur, torch) / 3
    out.update({"select_us": sms * 1e3, "select_embed_mb": st.select_bytes() / 1e6})
    dreplay = try_graph(lambda: st.draft(torch.cuda.current_stream()), torch)
    drun = dreplay if dreplay is not None else (lambda: st.draft(cur))
    drun()
    dms = timed(drun, passes, cur, torch) / (passes * cfg.gamma * st.Ld)
    out.update({"draft_us_per_call": dms * 1e3, "draft_kv_mb_per_call": st.draft_kv_bytes_per_call(cfg.gamma // 2) / 1e6})
    st.accept(cur)
    out["accept_us"] = timed(lambda: st.accept(cur), 10, cur, torch) / 10 * 1e3
    # global semantic relevance (Eq. 2) over the timed target layers: bound by the exponentials (MUFU: 16 / clk / SM)
    st.attention_mass(cur)
    mms = timed(lambda: st.attention_mass(cur), 2, cur, torch) / (2 * layers)
    mufu_peak = 148 * 16 * 1.965e9
    out.update({"mass_us_per_layer": mms * 1e3, "mass_gexp_per_s": st.mass_exps_per_layer() / mms / 1e6,
                "mass_frac_of_mufu_peak": st.mass_exps_per_layer() / (mms * 1e-3) / mufu_peak})
    # the whole step: select -> gather -> (draft || verify on two streams) -> accept, all target layers if they fit
    st.run()
    torch.cuda.synchronize()
    out["step_ms"] = timed(st.run, passes, cur, torch) / passes
    out["step_target_layers"] = layers
    out["step_draft_layers"] = st.Ld
    del st
    torch.cuda.empty_cache()
    return out


def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2601_08273_b200 import binding as hb
    from paper_2601_08273_b200 import workloads as W
    from paper_2601_08273_b200.step import HippoStep

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    steps = args.steps if args.steps is not None else 300
    warmup = max(3, args.warmup if args.warmup is not None else 10)
    peak, peak_src = load_peaks()
    cfg = W.CONFIGS[args.config]
    st = HippoStep(cfg)
    cur = torch.cuda.current_stream()

    from paper_2601_08273_b200 import replicas
    dev0 = torch.device("cuda", local)

    def barrier():
        replicas.barrier(dev0)

    def max_over_ranks(x: float) -> float:
        return replicas.max_over_ranks(x, dev0)

    # warm-up (eager), counting this library's launches per step
    c0 = hb.hippo_launch_count()
    st.run()
    torch.cuda.synchronize()
    launches_per_step = hb.hippo_launch_count() - c0
    c0 = hb.hippo_launch_count()
    st.verify(cur)
    torch.cuda.synchronize()
    launches_per_verify_leg = hb.hippo_launch_count() - c0
    assert hb.hippo_workspace_status(st.verify_ws) == 0 and hb.hippo_workspace_status(st.draft_ws) == 0
    use_graph = not args.no_graph
    step_fn, verify_fn = st.run, (lambda: st.verify(cur))
    if use_graph:
        r1 = try_graph(st.run, torch)
        r2 = try_graph(lambda: st.verify(torch.cuda.current_stream()), torch)
        if r1 is not None and r2 is not None:
            step_fn, verify_fn = r1, r2
        else:
            use_graph = False
    for _ in range(warmup):
        step_fn()
    for _ in range(3):
        verify_fn()

    sampler = ClockSampler("GPU-" + str(torch.cuda.get_device_properties(local).uuid)) if rank == 0 else None
    barrier()
    if sampler:
        sampler.mark()
    # timed region 1: K whole steps
    step_ms = max_over_ranks(timed(step_fn, steps, cur, torch))
    barrier()
    # timed region 2: the verification leg of K steps (same buffers, same launches), timed alone on its stream
    verify_ms = max_over_ranks(timed(verify_fn, steps, cur, torch))
    barrier()
    if sampler:
        sampler.mark()
    clocks = sampler.stop() if sampler else None

    kv_bytes_step = st.verify_kv_bytes_per_layer() * st.Lt
    value = world * kv_bytes_step * steps / (verify_ms * 1e-3) / 1e9
    per_launch_ms = verify_ms / (steps * st.Lt)

    # e2e: the verification leg through the public API with HOST buffers: per step, H2D of q / K / V / kv_len of every
    # layer from pinned memory, the launches, and D2H of the outputs
    e2e = None
    if not args.no_e2e:
        hk = [t.cpu().pin_memory() for t in (st.tgt_k, st.tgt_v, st.q_t)]
        h_len = st.kv_len_t.cpu().pin_memory()
        h_out = torch.empty(st.out_t.shape, dtype=st.out_t.dtype).pin_memory()
        m = max(st.kv_len_t_host)

        def e2e_step():
            st.kv_len_t.copy_(h_len, non_blocking=True)
            for l in range(st.Lt):
                st.tgt_k[l].copy_(hk[0][l], non_blocking=True)
                st.tgt_v[l].copy_(hk[1][l], non_blocking=True)
                st.q_t[l].copy_(hk[2][l], non_blocking=True)
                hb.hippo_verify_attention(st.q_t[l], st.tgt_cache[l], st.kv_len_t, m, out=st.out_t[l], workspace=st.verify_ws, stream=cur)
            h_out.copy_(st.out_t, non_blocking=True)

        n_e2e = max(3, min(20, steps))
        for _ in range(2):
            e2e_step()
        barrier()
        e2e_ms = max_over_ranks(timed(e2e_step, n_e2e, cur, torch))
        h2d = sum(t.numel() * t.element_size() for t in hk) + h_len.numel() * 4
        d2h = h_out.numel() * h_out.element_size()
        e2e = {"value": world * kv_bytes_step * n_e2e / (e2e_ms * 1e-3) / 1e9, "unit": UNIT,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": n_e2e, "ms_per_step": e2e_ms / n_e2e}
        del hk, h_out

    # per-call breakdown of one step (eager launches, each call timed alone)
    breakdown = {}
    if rank == 0:
        for name, fn, reps in (("select", lambda: st.select(cur), 5), ("gather", lambda: st.gather(cur), 20),
                               ("draft_all", (try_graph(lambda: st.draft(torch.cuda.current_stream()), torch) if use_graph else None) or (lambda: st.draft(cur)), 5),
                               ("accept", lambda: st.accept(cur), 20)):
            fn()
            breakdown[name + "_us"] = timed(fn, reps, cur, torch) / reps * 1e3
        breakdown["verify_all_us"] = verify_ms / steps * 1e3
        st.attention_mass(cur)
        breakdown["mass_all_layers_us"] = timed(lambda: st.attention_mass(cur), 3, cur, torch) / 3 * 1e3
        breakdown["mass_gexp_per_s"] = st.mass_exps_per_layer() * st.Lt / breakdown["mass_all_layers_us"] / 1e3
        breakdown["draft_us_per_call"] = breakdown["draft_all_us"] / (cfg.gamma * st.Ld)
        breakdown["gather_gbps"] = st.gather_bytes() / breakdown["gather_us"] / 1e3
        breakdown["draft_gbps"] = st.draft_kv_bytes_per_call(cfg.gamma // 2) / breakdown["draft_us_per_call"] / 1e3

    extra = []
    if rank == 0 and world == 1 and not args.no_extra:
        del st
        torch.cuda.empty_cache()
        for ci in (2, 3, 4):
            try:
                extra.append(kernel_sweep(W.CONFIGS[ci], torch, hb, HippoStep, peak))
            except Exception as e:  # noqa: BLE001
                extra.append({"workload": W.CONFIGS[ci].name, "error": str(e)[:200]})
        # the 64k configuration's sweep of gamma and of the pruning ratio (kept share 50/25/10/5 %)
        base, sweep = W.CONFIGS[4], []
        keys = ("verify_us_per_layer", "verify_frac_of_measured_peak", "draft_us_per_call", "gather_us",
                "gather_frac_of_measured_peak", "select_us", "accept_us", "step_ms")
        for g in W.C4_GAMMA_SWEEP:
            for pct in W.C4_KEEP_PCT_SWEEP:
                try:
                    r = kernel_sweep(base.replace(gamma=g, keep_pct=pct), torch, hb, HippoStep, peak, passes=2)
                    sweep.append({"gamma": g, "keep_pct": pct, **{k: round(r[k], 4) for k in keys}})
                except Exception as e:  # noqa: BLE001
                    sweep.append({"gamma": g, "keep_pct": pct, "error": str(e)[:200]})
        extra.append({"workload": base.name + " sweep", "points": sweep})
        # what the fused score does to the border bias of the attention mass: share of frame-border tokens among the
        # kept ones, attention term alone against all three terms (synthetic analogue of the paper's token-distribution figure)
        try:
            import numpy as np
            stb = HippoStep(cfg, target_layers=1, draft_layers=1)
            nv0, k0 = stb.n_visual[0], stb.k[0]
            border = W.is_boundary(cfg, nv0)
            shares = {}
            for name, mask in (("attention_only", 1), ("all_terms", 7)):
                kept, _ = hb.hippo_select_tokens(stb.embeds, stb.attn_mass, stb.n_visual, stb.k, cfg.grid_h, cfg.grid_w,
                                                 cfg.crop_h, cfg.crop_w, score_mask=mask)
                torch.cuda.synchronize()
                shares[name] = float(border[kept[:k0].cpu().numpy()].mean())
            extra.append({"workload": cfg.name + " kept-token border share", "border_share_of_all_tokens": float(border.mean()),
                          "kept": k0, **shares})
            del stb
        except Exception as e:  # noqa: BLE001
            extra.append({"workload": cfg.name + " kept-token border share", "error": str(e)[:200]})
        # the adaptive decoding schedule (Section 5.2) over the kernels, against the serial schedule, on the bench workload
        try:
            from paper_2601_08273_b200.vpsd import VpsdLoop
            torch.cuda.empty_cache()
            loop = VpsdLoop(cfg, buffered=0, pool=8, draft_noise=0.5)
            unit = loop.unit_times_ms()
            loop.run(4); loop.run_serial(2)
            par, ser = loop.run(60), loop.run_serial(30)
            st8 = hb.hippo_vpsd_init(cfg.gamma, 0)
            model_ms = 0.0
            for t in par["trace"]:
                rd = hb.hippo_vpsd_plan(st8)
                model_ms += hb.hippo_vpsd_round_time(rd, t["accepted"], unit["t_draft"], unit["t_target"])
                hb.hippo_vpsd_commit(st8, rd, t["accepted"], t["drafted_during"])
            extra.append({"workload": cfg.name + " decoding schedule", "gamma": cfg.gamma, "rounds": par["rounds"],
                          "t_draft_token_ms": unit["t_draft"], "t_verify_ms": unit["t_target"],
                          "parallel_tokens": par["tokens"], "parallel_ms": par["wall_ms"],
                          "parallel_tokens_per_s": par["tokens"] / par["wall_ms"] * 1e3,
                          "parallel_model_ms": model_ms,
                          "optimistic_rounds": sum(1 for t in par["trace"] if t["mode"] == 0),
                          "mean_accepted": sum(t["accepted"] for t in par["trace"]) / par["rounds"],
                          "serial_tokens": ser["tokens"], "serial_ms": ser["wall_ms"],
                          "serial_tokens_per_s": ser["tokens"] / ser["wall_ms"] * 1e3,
                          "note": "attention and acceptance kernels only, synthetic logits; host wall clock"})
            del loop
            torch.cuda.empty_cache()
        except Exception as e:  # noqa: BLE001
            extra.append({"workload": cfg.name + " decoding schedule", "error": str(e)[:200]})

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        import oracle
        # bounded sample: whole layers of the same workload (four distinct layers' inputs, cycled) until about 12 s
        # of CPU work have been timed
        from paper_2601_08273_b200 import workloads as W2
        lens = [n + cfg.n_text + cfg.gamma + 1 for n in W2.visual_lengths(cfg)]
        layers_in = [W2.attention_inputs(cfg, "target", lens, cfg.gamma + 1, layer=l) for l in range(min(4, cfg.tgt_layers))]
        per_layer_bytes = sum(lens) * 2 * cfg.tgt_kv_heads * cfg.tgt_head_dim * (4 if cfg.dtype == "fp32" else 2)
        s_tot, b_tot, n_layers = 0.0, 0, 0
        while s_tot < 12.0:
            inp = layers_in[n_layers % len(layers_in)]
            t0 = time.perf_counter()
            oracle.attention(inp["q"], inp["k"], inp["v"], lens)
            s_tot += time.perf_counter() - t0
            b_tot += per_layer_bytes
            n_layers += 1
        cpu = {"value": b_tot / s_tot / 1e9, "unit": UNIT, "cores": oracle.max_threads(), "kind": "oracle",
               "sample": "oracle verify attention (fp64, OpenMP over rows) on %d layer passes of %s (of %d layers per step), all %d rows per layer; %.1f s"
                         % (n_layers, cfg.name, cfg.tgt_layers, (cfg.gamma + 1) * cfg.tgt_q_heads, s_tot)}

    if rank == 0:
        achieved = (kv_bytes_step / cfg.tgt_layers) / (per_launch_ms * 1e-3) / 1e9
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
            "ms_per_step": step_ms / steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if cfg.dtype == "bf16" else "f32", "data": "synthetic",
            "config": {"workload": cfg.name, "visual_tokens": W.visual_lengths(cfg), "gamma": cfg.gamma,
                       "target_layers": cfg.tgt_layers, "draft_layers": cfg.dft_layers, "keep_pct": cfg.keep_pct,
                       "l2": "inputs larger than L2: every layer has its own KV buffers (%.0f MB of target KV per step)" % (kv_bytes_step / 1e6),
                       "cuda_graph": use_graph, "parallelism": "replicas" if world > 1 else "single"},
            "verify_us_per_layer": per_launch_ms * 1e3,
            "roofline": {"bound": "hbm", "kernel": "verify attention (%d launches per step)" % cfg.tgt_layers,
                         "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "peak_source": peak_src, "traffic": measured_traffic(cfg.name),
                         "algorithmic_bytes_per_launch": kv_bytes_step // cfg.tgt_layers,
                         # the same kernel (and the gather) on the longer workloads timed in this run, same peak
                         "other_workloads": {e["workload"]: {"verify_gbps": round(e["verify_gbps"], 1),
                                                             "verify_frac": round(e["verify_frac_of_measured_peak"], 3),
                                                             "gather_frac": round(e["gather_frac_of_measured_peak"], 3)}
                                             for e in extra if "verify_frac_of_measured_peak" in e}},
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches_per_step * steps + launches_per_verify_leg * steps),
            "gpu_launches_per_step": int(launches_per_step), "step_breakdown": breakdown, "extra": extra, "cpu_baseline": cpu,
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--config", type=int, default=1, help="index into the five configurations (default 1: 7B-class single video)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-graph", action="store_true")
    ap.add_argument("--no-extra", action="store_true", help="skip the per-call timings and whole-step times of the other configurations (c2, c3, c4)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
