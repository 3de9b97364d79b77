#!/usr/bin/env python
"""Benchmark of the HIPPO hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 2] [--impl ours|reference] [--no-graph] [--no-extra] [--no-breakdown]

A step is one pass of the whole hot path over one batch of synthetic input: select -> (verify attention of all target
layers on one stream || gather -> gamma x draft layers of draft attention on another) -> accept.  The metric is the
verification leg's KV-read bandwidth: target-KV bytes attended per step / device time of the step's verification
launches (CUDA events on the stream that launches them).  One JSON line is printed by rank 0.

Every figure is taken from `repeats` event-bracketed repetitions and printed as min / median / max; every GB/s figure
is given three ways: of the nominal 8,000 GB/s, of the measured copy bandwidth (MEASURED_PEAKS.json) and of a
read-only streaming probe run here (hippo_read_probe over 4 GiB).

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
NOMINAL_HBM_GBS = 8000.0
# 64 fp64 multiply-adds per clock and SM; a register-only probe of mma.sync.m8n8k4.f64 on this part measured 63.7 with
# constant operands and 47 with operands that change every instruction
FP64_PEAK_FLOPS = 148 * 64 * 2 * 1.965e9
MUFU_PEAK_PER_S = 148 * 16 * 1.965e9          # 16 ex2 per clock per SM


# DRAM traffic of the dominant kernel per launch (dram__bytes_read.sum + dram__bytes_write.sum from one ncu capture of
# the workload named by the key); valid only for the kernel source it was taken on, identified by its hash.
NCU_TRAFFIC = {"source": "paper_2601_08273_b200/csrc/attn_tc.cu", "sha1_12": "3f5bfa3f1be8",
               # 8 layers of the same workload captured (1,084.9 MB read + 4.0 MB written), scaled by 36 / 8: traffic grows
               # in proportion to the layers
               "bytes_per_launch": {"c2_long_video_32k": int((1084878000 + 4028928) * 36 / 8)}}


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

def timed_reps(fn, reps, stream, torch):
    """`reps` back-to-back calls of fn, each bracketed by its own events on `stream`.  Returns (total ms between the first
    and the last event, list of per-call ms)."""
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(reps + 1)]
    torch.cuda.synchronize()
    ev[0].record(stream)
    for i in range(reps):
        fn()
        ev[i + 1].record(stream)
    torch.cuda.synchronize()
    return ev[0].elapsed_time(ev[reps]), [ev[i].elapsed_time(ev[i + 1]) for i in range(reps)]


def spread(ms_list, scale=1.0, digits=3):
    """min / median / max of a list of milliseconds, scaled (e.g. 1e3 / launches for microseconds per launch)."""
    xs = sorted(x * scale for x in ms_list)
    return {"min": round(xs[0], digits), "median": round(statistics.median(xs), digits), "max": round(xs[-1], digits), "n": len(xs)}


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


class Peaks:
    """The three denominators of every bandwidth figure."""

    def __init__(self, torch, hb, reps=20):
        self.copy, self.copy_src = load_peaks()
        self.nominal = NOMINAL_HBM_GBS
        # read-only streaming probe: one pass of 16-byte loads over 4 GiB (larger than L2 by far), nothing written
        buf = torch.empty(1 << 30, dtype=torch.int32, device="cuda")
        buf.random_(0, 1 << 20)
        sink = torch.zeros(64, dtype=torch.int32, device="cuda")
        cur = torch.cuda.current_stream()
        for _ in range(3):
            hb.hippo_read_probe(buf, sink, stream=cur)
        _, per = timed_reps(lambda: hb.hippo_read_probe(buf, sink, stream=cur), reps, cur, torch)
        nbytes = buf.numel() * 4
        self.read = nbytes / (statistics.median(per) * 1e-3) / 1e9
        self.read_spread = spread([nbytes / (x * 1e-3) / 1e9 for x in per], digits=1)
        del buf
        torch.cuda.empty_cache()

    def fracs(self, gbps):
        return {"of_nominal_8000": round(gbps / self.nominal, 4), "of_measured_copy": round(gbps / self.copy, 4),
                "of_read_probe": round(gbps / self.read, 4)}

    def describe(self):
        return {"nominal_gbs": self.nominal, "measured_copy_gbs": self.copy, "measured_copy_source": self.copy_src,
                "read_probe_gbs": round(self.read, 1), "read_probe_spread_gbs": self.read_spread,
                "read_probe": "hippo_read_probe over 4 GiB, median of 20"}


def bandwidth_entry(nbytes, per_ms, launches, peaks):
    """A GB/s figure with its spread and the three fractions.  per_ms: list of ms per repetition of `launches` launches."""
    med = statistics.median(per_ms)
    gbps = nbytes * launches / (med * 1e-3) / 1e9
    return {"us_per_launch": spread(per_ms, 1e3 / launches), "mb_per_launch": round(nbytes / 1e6, 3),
            "gbps": round(gbps, 1), "frac": peaks.fracs(gbps)}


def kernel_sweep(cfg, torch, hb, HippoStep, peaks, uuid, reps=20, max_gb=24.0, brief=False):
    """Per-call timings and the whole step of one configuration (distinct KV buffers per layer), with its own clock
    record.  brief: fewer repetitions of the small calls (the sweep points)."""
    from paper_2601_08273_b200 import workloads as W
    per_layer = sum(n + cfg.n_text + cfg.gamma + 1 for n in W.visual_lengths(cfg)) * 2 * cfg.tgt_kv_heads * cfg.tgt_head_dim * 2
    layers = max(1, min(cfg.tgt_layers, int(max_gb * 1e9 / per_layer)))
    st = HippoStep(cfg, target_layers=layers, draft_layers=min(cfg.dft_layers, 28))
    cur = torch.cuda.current_stream()
    sampler = ClockSampler(uuid)
    out = {"workload": cfg.name, "target_layers_timed": layers, "repeats": reps}
    kvb = st.verify_kv_bytes_per_layer()
    # verification leg, all layers in one launch / one launch per layer: graph replay of the leg, per-replay events
    for name, leg in (("verify_layers_call", st.verify_layers), ("verify_per_layer_calls", st.verify)):
        for _ in range(3):
            leg(cur)
        replay = try_graph(lambda leg=leg: leg(torch.cuda.current_stream()), torch)
        run = replay if replay is not None else (lambda leg=leg: leg(cur))
        run()
        sampler.mark()
        _, per = timed_reps(run, reps, cur, torch)
        sampler.mark()
        out[name] = bandwidth_entry(kvb, per, layers, peaks)
        assert hb.hippo_workspace_status(st.verify_ws) == 0 and hb.hippo_workspace_status(st.verify_layers_ws) == 0
    n_small = 5 if brief else reps
    st.select(cur); st.gather(cur)
    for _ in range(3):
        st.gather(cur)
    _, per = timed_reps(lambda: st.gather(cur), n_small, cur, torch)
    out["gather"] = bandwidth_entry(st.gather_bytes(), per, 1, peaks)
    _, per = timed_reps(lambda: st.select(cur), max(3, n_small // 2), cur, torch)
    med = statistics.median(per)
    out["select"] = {"us": spread(per, 1e3), "embed_mb": round(st.select_bytes() / 1e6, 1),
                     "fp64_gflop": round(st.select_flops() / 1e9, 2),
                     "tflops": round(st.select_flops() / (med * 1e-3) / 1e12, 2),
                     "frac_of_fp64_peak": round(st.select_flops() / (med * 1e-3) / FP64_PEAK_FLOPS, 4)}
    dreplay = try_graph(lambda: st.draft(torch.cuda.current_stream()), torch)
    drun = dreplay if dreplay is not None else (lambda: st.draft(cur))
    drun()
    _, per = timed_reps(drun, n_small, cur, torch)
    calls = cfg.gamma * st.Ld
    out["draft"] = bandwidth_entry(st.draft_kv_bytes_per_call(cfg.gamma // 2), per, calls, peaks)
    st.accept(cur)
    _, per = timed_reps(lambda: st.accept(cur), n_small, cur, torch)
    out["accept"] = {"us": spread(per, 1e3), "logits_mb": round(st.accept_bytes() / 1e6, 2)}
    if not brief:
        # global semantic relevance (Eq. 2) over the timed target layers: bound by the exponentials
        st.attention_mass(cur)
        _, per = timed_reps(lambda: st.attention_mass(cur), 5, cur, torch)
        med = statistics.median(per) / layers
        out["attention_mass"] = {"us_per_layer": spread(per, 1e3 / layers), "gexp_per_s": round(st.mass_exps_per_layer() / med / 1e6, 1),
                                 "frac_of_mufu_peak": round(st.mass_exps_per_layer() / (med * 1e-3) / MUFU_PEAK_PER_S, 4)}
    # the whole step: select -> (verify || gather -> draft) -> accept, replayed from a graph like the headline step
    st.run()
    torch.cuda.synchronize()
    step_replay = try_graph(st.run, torch)
    step_run = step_replay if step_replay is not None else st.run
    step_run()
    sampler.mark()
    _, per = timed_reps(step_run, n_small, cur, torch)
    sampler.mark()
    out["step_ms"] = spread(per)
    out["step_draft_layers"] = st.Ld
    out["clocks"] = sampler.stop()
    del st
    torch.cuda.empty_cache()
    return out


def schedule_entry(cfg, torch, hb, rounds=40, draft_noise=0.5, verify_max_ctas=0, gamma=None, draft_num_splits=None):
    """The adaptive decoding schedule (Section 5.2) over the kernels against the serial schedule.  draft_noise sets how far
    the synthetic draft logits are from the target's (the acceptance rate); verify_max_ctas > 0 leaves SMs to the draft
    stream while the verification kernel runs."""
    from paper_2601_08273_b200.vpsd import VpsdLoop
    torch.cuda.empty_cache()
    loop = VpsdLoop(cfg, buffered=0, pool=8, draft_noise=draft_noise, verify_max_ctas=verify_max_ctas, gamma=gamma,
                    draft_num_splits=draft_num_splits)
    cfg = loop.cfg
    unit = loop.unit_times_ms()
    shared = loop.shared_times_ms()
    loop.run(4); loop.run_serial(2)
    par, ser = loop.run(rounds), loop.run_serial(rounds // 2)
    state = hb.hippo_vpsd_init(cfg.gamma, 0)
    # the round-time model twice: with each leg's time measured alone (the paper's setting: the legs do not share a
    # memory system) and with the times the legs show side by side on this one GPU
    model_ms, shared_model_ms = 0.0, 0.0
    for t in par["trace"]:
        rd = hb.hippo_vpsd_plan(state)
        model_ms += hb.hippo_vpsd_round_time(rd, t["accepted"], unit["t_draft"], unit["t_target"])
        u = shared if rd.draft_during > 0 else unit
        shared_model_ms += hb.hippo_vpsd_round_time(rd, t["accepted"], u["t_draft"], u["t_target"])
        hb.hippo_vpsd_commit(state, rd, t["accepted"], t["drafted_during"])
    serial_model = sum(hb.hippo_vpsd_serial_round_time(cfg.gamma, unit["t_draft"], unit["t_target"]) for _ in range(ser["rounds"]))
    out = {"workload": cfg.name + " decoding schedule", "gamma": cfg.gamma, "rounds": par["rounds"],
           "draft_noise": draft_noise, "verify_max_ctas": verify_max_ctas, "draft_num_splits": loop.st.draft_num_splits,
           "t_draft_token_ms": round(unit["t_draft"], 4), "t_verify_ms": round(unit["t_target"], 4),
           "target_over_draft": round(unit["t_target"] / unit["t_draft"], 2),
           "parallel_tokens": par["tokens"], "parallel_ms": round(par["wall_ms"], 3),
           "parallel_tokens_per_s": round(par["tokens"] / par["wall_ms"] * 1e3, 1),
           "parallel_model_ms": round(model_ms, 3), "parallel_measured_over_model": round(par["wall_ms"] / model_ms, 3),
           "t_draft_token_beside_verify_ms": round(shared["t_draft"], 4), "t_verify_beside_draft_ms": round(shared["t_target"], 4),
           "parallel_shared_gpu_model_ms": round(shared_model_ms, 3),
           "parallel_measured_over_shared_gpu_model": round(par["wall_ms"] / shared_model_ms, 3),
           "optimistic_rounds": sum(1 for t in par["trace"] if t["mode"] == 0),
           "mean_accepted": round(sum(t["accepted"] for t in par["trace"]) / par["rounds"], 2),
           "serial_tokens": ser["tokens"], "serial_ms": round(ser["wall_ms"], 3),
           "serial_tokens_per_s": round(ser["tokens"] / ser["wall_ms"] * 1e3, 1), "serial_model_ms": round(serial_model, 3),
           "note": "attention and acceptance kernels only, synthetic logits; host wall clock"}
    del loop
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
    steps = args.steps if args.steps is not None else 30
    warmup = max(3, args.warmup if args.warmup is not None else 5)
    reps = max(20, steps)
    uuid = "GPU-" + str(torch.cuda.get_device_properties(local).uuid)
    peaks = Peaks(torch, hb)
    cfg = W.CONFIGS[args.config]
    if args.layers is not None:
        cfg = cfg.replace(tgt_layers=max(1, args.layers))
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
    st.verify_layers(cur)
    torch.cuda.synchronize()
    launches_per_verify_leg = hb.hippo_launch_count() - c0
    c0 = hb.hippo_launch_count()
    st.verify(cur)
    torch.cuda.synchronize()
    launches_per_single_leg = hb.hippo_launch_count() - c0
    for ws in (st.verify_ws, st.verify_layers_ws, st.draft_ws):
        assert hb.hippo_workspace_status(ws) == 0
    use_graph = not args.no_graph
    step_fn, leg_fn, single_fn = st.run, (lambda: st.verify_layers(cur)), (lambda: st.verify(cur))
    if use_graph:
        r1 = try_graph(st.run, torch)
        r2 = try_graph(lambda: st.verify_layers(torch.cuda.current_stream()), torch)
        r3 = try_graph(lambda: st.verify(torch.cuda.current_stream()), torch)
        if r1 is not None and r2 is not None and r3 is not None:
            step_fn, leg_fn, single_fn = r1, r2, r3
        else:
            use_graph = False
    for _ in range(warmup):
        step_fn()
    for _ in range(3):
        leg_fn()
        single_fn()

    sampler = ClockSampler(uuid) if rank == 0 else None
    barrier()
    if sampler:
        sampler.mark()
    # timed region 1: K whole steps
    step_total, step_per = timed_reps(step_fn, steps, cur, torch)
    step_ms = max_over_ranks(step_total)
    barrier()
    # timed region 2: the verification leg of K steps (same buffers, same launches), timed alone on its stream
    leg_total, leg_per = timed_reps(leg_fn, steps, cur, torch)
    verify_ms = max_over_ranks(leg_total)
    barrier()
    # timed region 3: the same leg issued as one call per layer
    _, single_per = timed_reps(single_fn, reps, cur, torch)
    barrier()
    if sampler:
        sampler.mark()
    clocks = sampler.stop() if sampler else None

    kv_layer = st.verify_kv_bytes_per_layer()
    kv_bytes_step = kv_layer * st.Lt
    value = world * kv_bytes_step * steps / (verify_ms * 1e-3) / 1e9
    kernel_launches_per_leg = max(1, -(-st.Lt // 64))       # one kernel per 64 layers (plus one memset)
    per_launch_ms = verify_ms / (steps * kernel_launches_per_leg)

    # e2e: the verification leg through the public API with HOST buffers: per step, H2D of q / K / V / kv_len of every
    # layer from pinned memory, the launch, and D2H of the outputs
    e2e = None
    if not args.no_e2e:
        hk = [t.cpu().pin_memory() for t in (st.tgt_k, st.tgt_v, st.q_t)]
        h_len = st.kv_len_t.cpu().pin_memory()
        h_out = torch.empty(st.out_t.shape, dtype=st.out_t.dtype).pin_memory()

        def e2e_step():
            st.kv_len_t.copy_(h_len, non_blocking=True)
            st.tgt_k.copy_(hk[0], non_blocking=True)
            st.tgt_v.copy_(hk[1], non_blocking=True)
            st.q_t.copy_(hk[2], non_blocking=True)
            st.verify_layers(cur)
            h_out.copy_(st.out_t, non_blocking=True)

        n_e2e = max(3, min(10, steps))
        for _ in range(2):
            e2e_step()
        barrier()
        e2e_total, _ = timed_reps(e2e_step, n_e2e, cur, torch)
        e2e_ms = max_over_ranks(e2e_total)
        h2d = sum(t.numel() * t.element_size() for t in hk) + h_len.numel() * 4
        d2h = h_out.numel() * h_out.element_size()
        e2e = {"value": world * kv_bytes_step * n_e2e / (e2e_ms * 1e-3) / 1e9, "unit": UNIT,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": n_e2e, "ms_per_step": e2e_ms / n_e2e}
        del hk, h_out

    # per-call breakdown of one step (each call timed alone, `reps` event-bracketed repetitions)
    breakdown, other_kernels = {}, {}
    if rank == 0 and not args.no_breakdown:
        st.select(cur); st.gather(cur)
        _, per = timed_reps(lambda: st.gather(cur), reps, cur, torch)
        other_kernels["gather_kv"] = {"bound": "hbm", **bandwidth_entry(st.gather_bytes(), per, 1, peaks)}
        breakdown["gather_us"] = spread(per, 1e3)
        _, per = timed_reps(lambda: st.select(cur), reps, cur, torch)
        med = statistics.median(per)
        breakdown["select_us"] = spread(per, 1e3)
        other_kernels["select_tokens"] = {
            "bound": "alu", "unit": "TFLOP/s (fp64)", "achieved": round(st.select_flops() / (med * 1e-3) / 1e12, 3),
            "peak": round(FP64_PEAK_FLOPS / 1e12, 2), "frac": round(st.select_flops() / (med * 1e-3) / FP64_PEAK_FLOPS, 4),
            "peak_source": "148 SMs x 64 fp64 FMA per clock x 1.965 GHz", "fp64_gflop_per_launch_set": round(st.select_flops() / 1e9, 2),
            "us": spread(per, 1e3)}
        dfn = (try_graph(lambda: st.draft(torch.cuda.current_stream()), torch) if use_graph else None) or (lambda: st.draft(cur))
        dfn()
        _, per = timed_reps(dfn, reps, cur, torch)
        calls = cfg.gamma * st.Ld
        breakdown["draft_all_us"] = spread(per, 1e3)
        other_kernels["draft_attention"] = {"bound": "latency", **bandwidth_entry(st.draft_kv_bytes_per_call(cfg.gamma // 2), per, calls, peaks)}
        st.accept(cur)
        _, per = timed_reps(lambda: st.accept(cur), reps, cur, torch)
        breakdown["accept_us"] = spread(per, 1e3)
        breakdown["verify_leg_us"] = spread(leg_per, 1e3)
        breakdown["verify_leg_per_layer_calls_us"] = spread(single_per, 1e3)
        st.attention_mass(cur)
        _, per = timed_reps(lambda: st.attention_mass(cur), 5, cur, torch)
        med = statistics.median(per)
        breakdown["mass_all_layers_us"] = spread(per, 1e3)
        other_kernels["attention_mass"] = {
            "bound": "alu", "unit": "Gexp/s (MUFU ex2)", "achieved": round(st.mass_exps_per_layer() * st.Lt / med / 1e6, 1),
            "peak": round(MUFU_PEAK_PER_S / 1e9, 1), "frac": round(st.mass_exps_per_layer() * st.Lt / (med * 1e-3) / MUFU_PEAK_PER_S, 4),
            "peak_source": "148 SMs x 16 ex2 per clock x 1.965 GHz"}

    extra = []
    if rank == 0 and world == 1 and not args.no_extra:
        del st
        torch.cuda.empty_cache()
        for ci in (1, 2, 3, 4):
            if ci == args.config:
                continue
            try:
                extra.append(kernel_sweep(W.CONFIGS[ci], torch, hb, HippoStep, peaks, uuid))
            except Exception as e:  # noqa: BLE001
                extra.append({"workload": W.CONFIGS[ci].name, "error": str(e)[:200]})
        # the 64k configuration's sweep of gamma and of the pruning ratio (kept share 50/25/10/5 %)
        base, sweep = W.CONFIGS[4], []
        for g in W.C4_GAMMA_SWEEP:
            for pct in W.C4_KEEP_PCT_SWEEP:
                try:
                    r = kernel_sweep(base.replace(gamma=g, keep_pct=pct), torch, hb, HippoStep, peaks, uuid, reps=10, brief=True)
                    sweep.append({"gamma": g, "keep_pct": pct,
                                  "verify_layers_us_per_layer": r["verify_layers_call"]["us_per_launch"]["median"],
                                  "verify_layers_frac_of_measured_copy": r["verify_layers_call"]["frac"]["of_measured_copy"],
                                  "verify_per_layer_us": r["verify_per_layer_calls"]["us_per_launch"]["median"],
                                  "verify_per_layer_frac_of_measured_copy": r["verify_per_layer_calls"]["frac"]["of_measured_copy"],
                                  "draft_us_per_call": r["draft"]["us_per_launch"]["median"],
                                  "gather_us": r["gather"]["us_per_launch"]["median"],
                                  "gather_frac_of_measured_copy": r["gather"]["frac"]["of_measured_copy"],
                                  "select_us": r["select"]["us"]["median"], "accept_us": r["accept"]["us"]["median"],
                                  "step_ms": r["step_ms"]["median"], "clocks": r["clocks"]})
                except Exception as e:  # noqa: BLE001
                    sweep.append({"gamma": g, "keep_pct": pct, "error": str(e)[:200]})
        extra.append({"workload": base.name + " sweep", "points": sweep})
        # what the selection rule does to the border bias of the attention mass: share of frame-border tokens among the
        # kept ones (synthetic analogue of the paper's token-distribution figure), per policy
        try:
            import numpy as np
            stb = HippoStep(cfg, target_layers=1, draft_layers=1)
            nv0, k0 = stb.n_visual[0], stb.k[0]
            border = W.is_boundary(cfg, nv0)
            shares = {}
            for name, kw in stb.policy_variants().items():
                kept, _ = stb.select_with(**kw)
                torch.cuda.synchronize()
                shares[name] = round(float(border[kept[:k0].cpu().numpy()].mean()), 4)
            extra.append({"workload": cfg.name + " kept-token border share", "border_share_of_all_tokens": round(float(border.mean()), 4),
                          "kept": k0, **shares})
            del stb
        except Exception as e:  # noqa: BLE001
            extra.append({"workload": cfg.name + " kept-token border share", "error": str(e)[:200]})
        # at two acceptance rates (a draft far from / close to the target), with all SMs for the verification kernel and
        # with 32 of them left to the draft stream
        for ci in (1, 2, 4):
            for noise, ctas in ((0.5, 0), (0.1, 0), (0.1, 116)):
                try:
                    extra.append(schedule_entry(W.CONFIGS[ci], torch, hb, draft_noise=noise, verify_max_ctas=ctas))
                except Exception as e:  # noqa: BLE001
                    extra.append({"workload": W.CONFIGS[ci].name + " decoding schedule", "error": str(e)[:200]})

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        import oracle
        # bounded sample: whole layers of the same workload (distinct layers' inputs, cycled) until about 12 s
        # of CPU work have been timed
        from paper_2601_08273_b200 import workloads as W2
        lens = [n + cfg.n_text + cfg.gamma + 1 for n in W2.visual_lengths(cfg)]
        layers_in = [W2.attention_inputs(cfg, "target", lens, cfg.gamma + 1, layer=l) for l in range(min(2, cfg.tgt_layers))]
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
        layers_per_launch = min(cfg.tgt_layers, 64)
        alg_bytes_per_launch = kv_layer * layers_per_launch
        achieved = alg_bytes_per_launch / (per_launch_ms * 1e-3) / 1e9
        single = bandwidth_entry(kv_layer, single_per, cfg.tgt_layers, peaks)
        leg = bandwidth_entry(kv_layer, leg_per, cfg.tgt_layers, peaks)
        others = {}
        for e in extra:
            if "verify_layers_call" in e:
                others[e["workload"]] = {
                    "verify_layers_call": {"gbps": e["verify_layers_call"]["gbps"], "us_per_layer": e["verify_layers_call"]["us_per_launch"],
                                           "frac": e["verify_layers_call"]["frac"]},
                    "verify_per_layer_calls": {"gbps": e["verify_per_layer_calls"]["gbps"], "us_per_layer": e["verify_per_layer_calls"]["us_per_launch"],
                                               "frac": e["verify_per_layer_calls"]["frac"]},
                    "gather_kv": {"gbps": e["gather"]["gbps"], "frac": e["gather"]["frac"]}, "clocks": e["clocks"]}
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
            "ms_per_step": step_ms / steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if cfg.dtype == "bf16" else "f32", "data": "synthetic",
            "config": {"workload": cfg.name, "visual_tokens": W.visual_lengths(cfg), "gamma": cfg.gamma,
                       "target_layers": cfg.tgt_layers, "draft_layers": cfg.dft_layers, "keep_pct": cfg.keep_pct,
                       "l2": "inputs larger than L2: every layer has its own KV buffers (%.0f MB of target KV per step)" % (kv_bytes_step / 1e6),
                       "verify_leg": "hippo_verify_attention_layers: all %d target layers in %d launch(es)" % (cfg.tgt_layers, kernel_launches_per_leg),
                       "cuda_graph": use_graph, "parallelism": "replicas" if world > 1 else "single"},
            "step_ms": spread(step_per), "verify_us_per_layer": leg["us_per_launch"],
            "roofline": {"bound": "hbm", "kernel": "attn_tc_kernel, multi-layer (%d layers per launch, %d launch(es) per step)" % (layers_per_launch, kernel_launches_per_leg),
                         "achieved": achieved, "peak": peaks.copy, "unit": "GB/s", "frac": achieved / peaks.copy,
                         "peak_source": peaks.copy_src, "fracs": peaks.fracs(achieved), "peaks": peaks.describe(),
                         "traffic": measured_traffic(cfg.name) if args.layers is None else None,
                         "algorithmic_bytes_per_launch": alg_bytes_per_launch,
                         "algorithmic_bytes_per_layer": kv_layer, "per_layer": leg,
                         # the same layers as one hippo_verify_attention call per layer (two kernels each)
                         "per_layer_calls": single,
                         "other_kernels": other_kernels,
                         # the same kernels on the other workloads timed in this run
                         "other_workloads": others},
            "clocks": clocks, "e2e": e2e,
            "gpu_launches": int(launches_per_step * steps + launches_per_verify_leg * steps + launches_per_single_leg * reps),
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
    ap.add_argument("--config", type=int, default=2,
                    help="index into the five configurations (default 2: long video, 32,768 visual tokens, the smallest size the bandwidth target is stated for)")
    ap.add_argument("--layers", type=int, default=None,
                    help="time this many target layers instead of the configuration's (a small case for profiler captures)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-graph", action="store_true")
    ap.add_argument("--no-extra", action="store_true", help="skip the per-call timings and whole-step times of the other configurations")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-breakdown", action="store_true",
                    help="skip the per-call timings of the step's parts (a launch list of the run then holds whole steps only)")
    ap.add_argument("--no-cpu", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
