#!/usr/bin/env python
"""Benchmark of the ActQKV per-window retrieval path on B200.

One "step" = the whole hot path (bias+probe -> score -> cut-off/select -> attention -> append)
for one window of W queries of one layer at the last window of a 32k-token prefill of the
LLaMA3-8B-shaped workload.  Metric: prefill retrieval tokens/s/layer = W / step time.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

Cold L2: consecutive steps run on different, physically distinct copies of the layer state
(caches, tables, inputs; > 2x L2 in total), so nothing a step reads is left in L2 by the
previous one.  Under torchrun every rank runs its own copies (independent layers: weak
scaling, no collective on the data path); rank 0 prints one JSON line.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "prefill retrieval tokens/sec/layer at 32k ctx"
UNIT = "tokens/s/layer"


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return dict(hbm_gbs=d["hbm_gbs"], bf16_tflops=d["bf16_tflops"],
                    bf16_tflops_sustained=d.get("bf16_tflops_sustained", d["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index: int, period=0.004):
        super().__init__(daemon=True)
        self.index, self.period = index, period
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def sample(self):
        if self.nv is None:
            return
        nv = self.nv
        try:
            self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
            r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h) if hasattr(
                nv, "nvmlDeviceGetCurrentClocksEventReasons") else nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
            names = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
                     0x4: "sw_power_cap", 0x80: "hw_power_brake"}
            for bit, name in names.items():
                if r & bit:
                    self.reasons.add(name)
        except Exception:
            pass

    def run(self):
        while not self._stop_evt.is_set():
            self.sample()
            time.sleep(self.period)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2)
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# DRAM traffic of one launch of the attention kernel (dram__bytes_read.sum + dram__bytes_write.sum of one
# ncu capture of this workload), valid only for the kernel source it was taken on: the figure is
# reported while the sha256 of the kernel file still starts with the recorded digits, else null.
ATTENTION_TRAFFIC = {"source_sha256_16": "57ab1a5a6294688a", "bytes_per_launch": 23685248}


def attention_traffic():
    import hashlib
    path = os.path.join(ROOT, "paper_2502_13542_b200", "csrc", "attention_tc2.cu")
    try:
        with open(path, "rb") as f:
            digest = hashlib.sha256(f.read()).hexdigest()[:16]
    except OSError:
        return None
    return ATTENTION_TRAFFIC["bytes_per_launch"] if digest == ATTENTION_TRAFFIC["source_sha256_16"] else None


def attention_flops(spec, p0, c_blocks):
    """Causal-counted useful flops of one window's attention (4*D per query-key pair)."""
    from paper_2502_13542_b200 import workloads as wl
    n = wl.n_candidates(spec, p0)
    n_past = (spec.n_init + c_blocks * spec.block + (p0 - (spec.n_init + n * spec.block))) if p0 > spec.n_init else p0
    W = spec.window
    pairs = W * n_past + W * (W + 1) // 2
    return 4.0 * spec.head_dim * spec.n_q_heads * pairs


def stage_bytes(spec, p0):
    """Algorithmic HBM bytes of the memory-bound stages of one window (dtype bf16 = 2 B)."""
    from paper_2502_13542_b200 import workloads as wl
    e = 2 if spec.dtype == "bf16" else 4
    n = wl.n_candidates(spec, p0)
    W, Hq, Hkv, D, r = spec.window, spec.n_q_heads, spec.n_kv_heads, spec.head_dim, spec.n_repr
    return {
        "bias_probe": W * Hq * D * e + 3 * Hq * D * 4 + Hq * W * 4,
        "score": n * Hkv * r * D * e + n * Hkv * r * 4 + n * Hkv * 4,
        "select": n * Hkv * 4 + spec.cap_blocks * Hkv * 4,
        "append": 2 * 2 * W * Hkv * D * e,
    }


def stage_free_step_us(stage_all) -> float:
    """Sum of the median stage times of one step (an upper bound of the overlapped step)."""
    return float(sum(np.median(v) for v in stage_all.values()))


def max_over_ranks(x: float, device=None) -> float:
    """The slowest rank's value (all ranks get it); the identity when there is one process."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(x)
    t = torch.tensor([x], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(units_per_rank_step: int, world: int, ms_per_step: float) -> float:
    """Whole-job units per second: every rank processes its own units (independent layers, no
    collective on the data path), the step time is the slowest rank's."""
    return world * units_per_rank_step / (ms_per_step * 1e-3)


# ------------------------------------------------------------------------------------------
def l2_flusher(device, mbytes=512):
    """Returns a function that reads a buffer several times the L2 size: afterwards nothing a
    kernel reads is in L2, and the lines it leaves behind are clean (no write-back traffic lands in
    the next timed launch)."""
    import torch
    scratch = torch.zeros(mbytes << 20, dtype=torch.uint8, device=device)
    return lambda: scratch.view(torch.int32).sum()


def build_states(spec, n_copies, device, sweep_times=None, flush=None):
    """Prefills one layer up to the last window on the GPU, then clones the state into
    n_copies physically distinct copies.  Returns (cfg, states, inputs of the last window).
    With sweep_times (a list) every window's step is timed with CUDA events after an L2 flush and
    its microseconds are appended: the prefill sweep itself is the measurement."""
    import torch
    from paper_2502_13542_b200 import binding as B
    from paper_2502_13542_b200 import workloads as wl

    cfg = B.make_config(spec, out_dtype=B.BF16)
    base = B.RetrievalState(cfg, page_table=wl.shuffled_page_table(spec, spec.context)[None, :], device=device)
    out = torch.zeros(spec.window, spec.n_q_heads, spec.head_dim, dtype=torch.bfloat16, device=device)
    T = spec.n_windows
    evs = []
    if sweep_times is not None:
        # first launches of every kernel (module load, shared-memory opt-in) on a scratch state
        warm = B.RetrievalState(cfg, page_table=wl.shuffled_page_table(spec, spec.context)[None, :], device=device)
        for t in range(2):
            kw, vw = wl.gen_kv(spec, 0, t)
            warm.step(wl.to_device(wl.gen_q(spec, 0, t)[None], spec, device), wl.to_device(kw[None], spec, device),
                      wl.to_device(vw[None], spec, device), out, overlap_append=True)
        torch.cuda.synchronize()
        del warm
    for t in range(T - 1):
        q = wl.to_device(wl.gen_q(spec, 0, t)[None], spec, device)
        k, v = wl.gen_kv(spec, 0, t)
        k, v = wl.to_device(k[None], spec, device), wl.to_device(v[None], spec, device)
        if sweep_times is not None:
            flush()
            e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
            e0.record(); base.step(q, k, v, out, overlap_append=True); e1.record()
            evs.append((e0, e1))
        else:
            base.step(q, k, v, out)
    torch.cuda.synchronize()
    if sweep_times is not None:
        sweep_times.extend(1e3 * a.elapsed_time(b) for a, b in evs)
    q = wl.to_device(wl.gen_q(spec, 0, T - 1)[None], spec, device)
    k, v = wl.gen_kv(spec, 0, T - 1)
    k, v = wl.to_device(k[None], spec, device), wl.to_device(v[None], spec, device)
    states, inputs = [], []
    names = ["stats_count", "stats_mean", "stats_m2", "repr_k", "repr_inv_norm", "budget_state", "k_pages",
             "v_pages", "probe_kv", "probe_qh"]
    for i in range(n_copies):
        st = B.RetrievalState(cfg, page_table=base.page_table.cpu().numpy(), device=device)
        for nme in names:
            getattr(st, nme).copy_(getattr(base, nme))
        st.set_positions(base.host_pos0)
        states.append(st)
        inputs.append((q.clone(), k.clone(), v.clone(), torch.zeros_like(out)))
    return cfg, states, inputs


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2502_13542_b200 import binding as B
    from paper_2502_13542_b200 import workloads as wl

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)

    spec = wl.llama3_8b_layer().replace(page_tokens=args.page_tokens)
    p0 = (spec.n_windows - 1) * spec.window
    n_copies = args.copies
    extras = world == 1 and not args.headline_only
    sweep_us = [] if extras else None
    cfg, states, inputs = build_states(spec, n_copies, device, sweep_times=sweep_us,
                                       flush=l2_flusher(device) if extras else None)
    peaks = load_peaks()
    # One untimed step on the first copy, kept for the comparison with the oracle (the copies stand
    # exactly where the prefill sweep left the layer, so this is the sweep's last window).
    parity_sample = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        st0 = states[0]
        q0, k0, v0, out0 = inputs[0]
        st0.step(q0, k0, v0, out0, advance=False)
        torch.cuda.synchronize()
        parity_sample = {"out": out0.float().cpu().numpy(), "sel": st0.sel_idx[0].cpu().numpy().astype(np.int64),
                         "c": int(st0.sel_count.item())}

    side = torch.cuda.Stream(device=device)
    ev_fork, ev_join = torch.cuda.Event(), torch.cuda.Event()

    def one_step(i, events=None, overlap=True):
        """One window through the six stages.  In the timed loop the append runs on a second stream,
        concurrent with the attention of the same step (it reads the step's own K / V only and
        writes pages / table rows the attention does not read; started earlier it would compete
        with the short kernels that produce the selection, which the attention waits for); the
        instrumented pass (events given) runs everything in order on one stream to time each stage
        alone."""
        st = states[i % n_copies]
        q, k, v, out = inputs[i % n_copies]
        b = st.batch
        append = lambda stream=None: B.append_window(cfg, b, k, v, spec.window, st.pos0, st.k_pages, st.v_pages,
                                                     st.page_table, st.repr_k, st.repr_inv_norm, st.status,
                                                     stream=stream)
        calls = (
            ("bias_probe", lambda: B.bias_probe(cfg, b, q, spec.window, st.stats_count, st.stats_mean, st.stats_m2,
                                                st.phi_l1, None, st.probe_qh, st.probe_kv, st.status)),
            ("score_select", lambda: B.score_select(cfg, b, st.probe_kv, st.repr_k, st.repr_inv_norm, st.n_cand,
                                                    st.budget_state, st.scores, st.theta, st.sel_idx, st.sel_count,
                                                    st.budget_real, st.status)),
            ("attention", lambda: B.retrieval_attention(cfg, b, q, k, v, spec.window, st.k_pages, st.v_pages,
                                                        st.page_table, st.pos0, st.sel_idx, st.sel_count, out, None,
                                                        st.status)),
        )
        if events is not None:
            for name, fn in calls + (("append", append),):
                e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
                e0.record(); fn(); e1.record()
                events.setdefault(name, []).append((e0, e1))
            return
        if not overlap:
            for name, fn in calls + (("append", append),):
                fn()
            return
        main = torch.cuda.current_stream()

        def fork_append():
            ev_fork.record(main)
            side.wait_event(ev_fork)
            append(side)
            ev_join.record(side)

        # Replayed from a graph the append starts with the attention, once the selection is done
        # (earlier it competes with the short kernels the attention waits for); with plain
        # launches an event recorded between two kernels of the chain would cost the second one
        # its early start, so the fork sits in front of the step.
        late = torch.cuda.is_current_stream_capturing()
        if not late:
            fork_append()
        for name, fn in calls:
            if late and name == "attention":
                fork_append()
            fn()
        main.wait_event(ev_join)

    launches_per_step = 5   # bias_probe, score, cut-off + select, attention, append

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(args.warmup):
        one_step(i)
    barrier()
    # The K steps of the timed region are captured once into a CUDA graph (the launch pattern of a
    # prefill: one window through a run of layers, here the rotated layer states) and each
    # repetition replays it: enqueueing a step's five launches from Python takes about as long as
    # the step runs, so eager launches reach the GPU too late for the step's kernels to be
    # resident ahead of their turn (programmatic dependent launch).  --eager times the plain
    # launches instead.
    step_graph = None
    if not args.eager:
        step_graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(step_graph):
            for i in range(args.steps):
                one_step(args.warmup + i)
        for _ in range(2):
            step_graph.replay()
        barrier()
    sampler = ClockSampler(local)
    sampler.start()
    if args.profile_region:
        torch.cuda.profiler.start()          # cudaProfilerStart: lets a profiler capture the timed region only
    # The timed region of K steps is repeated `reps` times (each bracketed by a barrier and a device
    # synchronisation): a K-step region lasts a millisecond or two, so one sample would say little.
    # ms_per_step is the median repetition; min and max are reported beside it.
    rep_ms, step_idx = [], args.warmup
    for _ in range(max(1, args.reps)):
        barrier()
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        e0.record()
        if step_graph is not None:
            step_graph.replay()
        else:
            for i in range(args.steps):
                one_step(step_idx + i)
        e1.record()
        step_idx += args.steps
        barrier()
        rep_ms.append(max_over_ranks(e0.elapsed_time(e1), device) / args.steps)
    if args.profile_region:
        torch.cuda.profiler.stop()
    sampler.sample()
    clocks = sampler.stop()
    ms_step = float(np.median(rep_ms))
    value = job_throughput(spec.window, world, ms_step)
    step_stats = {"reps": len(rep_ms), "steps_per_rep": args.steps, "median_ms": ms_step,
                  "min_ms": float(np.min(rep_ms)), "max_ms": float(np.max(rep_ms))}

    # instrumented pass: per-stage device time with events around each call
    events = {}
    for i in range(max(args.steps, 20)):
        one_step(args.warmup + i, events)
    torch.cuda.synchronize()
    stage_all = {k: [1e3 * a.elapsed_time(b) for a, b in v] for k, v in events.items()}
    stage_us = {k: float(np.mean(v)) for k, v in stage_all.items()}
    assert all(int(st.status.item()) == 0 for st in states), "device status set during the bench"

    # The dominant kernel alone: `att_batch` launches back to back on the rotated (cold) copies between
    # two events, repeated; the duration of one launch is the batch time / launches.  (An event pair
    # around a single launch also counts the idle gap before the kernel starts: stages["attention"].)
    att_batch, att_reps = max(args.steps, 20), []
    for _ in range(5):
        a0 = torch.cuda.Event(enable_timing=True); a1 = torch.cuda.Event(enable_timing=True)
        a0.record()
        for i in range(att_batch):
            st = states[i % n_copies]
            q_, k_, v_, o_ = inputs[i % n_copies]
            B.retrieval_attention(cfg, st.batch, q_, k_, v_, spec.window, st.k_pages, st.v_pages, st.page_table,
                                  st.pos0, st.sel_idx, st.sel_count, o_, None, st.status)
        a1.record()
        torch.cuda.synchronize()
        att_reps.append(1e3 * a0.elapsed_time(a1) / att_batch)
    att_us = float(np.median(att_reps))
    c_sel = int(states[0].sel_count.item())
    flops = attention_flops(spec, p0, c_sel)
    att_tflops = flops / (att_us * 1e-6) / 1e12
    peak = peaks["bf16_tflops"]
    roofline = {"bound": "tensor", "kernel": "retrieval_attention", "achieved": att_tflops, "peak": peak,
                "unit": "TFLOP/s", "frac": att_tflops / peak, "traffic": attention_traffic(),
                "peak_source": peaks["source"] + " burst bf16 (cuBLAS)", "flops_per_launch": flops,
                "us_per_launch": att_us, "launches_timed": att_batch * len(att_reps),
                "timing": f"CUDA events around {att_batch} back-to-back launches on rotated cold copies, median of {len(att_reps)} batches",
                "us_single_launch_between_events": float(np.median(stage_all["attention"]))}
    sb = stage_bytes(spec, p0)
    stages = {k: {"us": v, "median_us": float(np.median(stage_all[k])), "min_us": float(np.min(stage_all[k]))}
              for k, v in stage_us.items()}
    stages["bias_probe"]["GBps"] = sb["bias_probe"] / stage_us["bias_probe"] / 1e3
    stages["score_select"]["GBps"] = (sb["score"] + sb["select"]) / stage_us["score_select"] / 1e3
    stages["append"]["GBps"] = sb["append"] / stage_us["append"] / 1e3
    stages["attention"]["TFLOPs"] = flops / (stage_us["attention"] * 1e-6) / 1e12

    # end to end through the public API with host buffers (pinned), copies inside the timed region
    q, k, v, out = inputs[0]
    hq, hk, hv = (x.cpu().pin_memory() for x in (q, k, v))
    ho = torch.empty_like(out, device="cpu").pin_memory()
    e2e_steps = max(3, min(args.steps, 200))

    def e2e_step(i):
        st = states[i % n_copies]
        dq, dk, dv, dout = inputs[i % n_copies]
        dq.copy_(hq, non_blocking=True); dk.copy_(hk, non_blocking=True); dv.copy_(hv, non_blocking=True)
        one_step(i, overlap=False)      # a synchronous step is bound by host latency: one stream is quicker
        ho.copy_(dout, non_blocking=True)
        torch.cuda.current_stream().synchronize()

    for i in range(3):
        e2e_step(i)
    barrier()
    t0 = time.perf_counter()
    for i in range(e2e_steps):
        e2e_step(3 + i)
    t_sync = max_over_ranks(time.perf_counter() - t0, device)

    # The same work as a pipeline over the rotated device buffers: the inputs of step i + 1 go up and
    # the result of step i - 1 comes down on copy streams of their own while step i computes.  Every
    # step's copies are inside the timed region; the host waits once, at the end.
    s_up, s_down = torch.cuda.Stream(device=device), torch.cuda.Stream(device=device)
    ev_up = [torch.cuda.Event() for _ in range(n_copies)]
    ev_done = [torch.cuda.Event() for _ in range(n_copies)]
    ev_down = [torch.cuda.Event() for _ in range(n_copies)]

    def pipelined(n, first, host_wait=True):
        main = torch.cuda.current_stream()
        for c in range(n_copies):
            ev_done[c].record(main); ev_down[c].record(main)
        for i in range(first, first + n):
            c = i % n_copies
            dq, dk, dv, dout = inputs[c]
            s_up.wait_event(ev_done[c])                 # the step that last read these input buffers
            with torch.cuda.stream(s_up):
                dq.copy_(hq, non_blocking=True); dk.copy_(hk, non_blocking=True); dv.copy_(hv, non_blocking=True)
                ev_up[c].record(s_up)
            main.wait_event(ev_up[c])
            main.wait_event(ev_down[c])                 # the result that last sat in this output buffer is on the host
            one_step(i)
            ev_done[c].record(main)
            s_down.wait_event(ev_done[c])
            with torch.cuda.stream(s_down):
                ho.copy_(dout, non_blocking=True)
                ev_down[c].record(s_down)
        if host_wait:
            s_down.synchronize(); main.synchronize(); s_up.synchronize()
        else:                                           # under capture: the copy streams join the capturing one
            main.wait_stream(s_up); main.wait_stream(s_down)

    pipelined(n_copies, 0)
    barrier()
    t0 = time.perf_counter()
    pipelined(e2e_steps, n_copies)
    t_eager = max_over_ranks(time.perf_counter() - t0, device)
    t_e2e, e2e_launch = t_eager, "eager calls"
    if not args.eager:
        # the same pipeline (copies, kernels, events) captured once and replayed: the host enqueues
        # a step's copies and launches more slowly than the GPU works through them
        e2e_graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(e2e_graph):
            pipelined(e2e_steps, n_copies, host_wait=False)
        e2e_graph.replay()
        barrier()
        t0 = time.perf_counter()
        e2e_graph.replay()
        torch.cuda.synchronize()
        t_e2e = max_over_ranks(time.perf_counter() - t0, device)
        e2e_launch = "one CUDA graph of the steps with their copies, launched and awaited inside the timed region"
    e2e = {"value": world * spec.window * e2e_steps / t_e2e, "unit": UNIT,
           "h2d_bytes_per_step": int(hq.numel() + hk.numel() + hv.numel()) * 2,
           "d2h_bytes_per_step": int(ho.numel()) * 2, "steps": e2e_steps,
           "mode": "copies of neighbouring steps overlap the step's kernels (three streams, one host wait at the end)",
           "launch": e2e_launch, "eager_calls": world * spec.window * e2e_steps / t_eager,
           "one_step_at_a_time": world * spec.window * e2e_steps / t_sync}

    secondary = {}
    if extras:
        # ---- sustained: the same step loop for about two seconds with the clock sampler running, and
        # the attention alone for about one second (its fraction is then taken against the sustained peak)
        def sustained(fn, seconds, est_ms):
            n = max(50, int(seconds / (est_ms * 1e-3)))
            smp = ClockSampler(local, period=0.02)
            torch.cuda.synchronize()
            smp.start()
            a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
            a.record()
            for i in range(n):
                fn(i)
            b.record()
            torch.cuda.synchronize()
            ck = smp.stop()
            ms = a.elapsed_time(b) / n
            return ms, n, ck

        if step_graph is not None:      # the timed region's graph of K steps, replayed for two seconds
            ms_g, n_g, ck_s = sustained(lambda i: step_graph.replay(), 2.0, ms_step * args.steps)
            ms_s, n_s = ms_g / args.steps, n_g * args.steps
        else:
            ms_s, n_s, ck_s = sustained(lambda i: one_step(i), 2.0, ms_step)

        def att_only(i):
            st = states[i % n_copies]
            q_, k_, v_, o_ = inputs[i % n_copies]
            B.retrieval_attention(cfg, st.batch, q_, k_, v_, spec.window, st.k_pages, st.v_pages, st.page_table,
                                  st.pos0, st.sel_idx, st.sel_count, o_, None, st.status)
        ms_a, n_a, ck_a = sustained(att_only, 1.0, stage_us["attention"] * 1e-3)
        tf_a = flops / (ms_a * 1e-3) / 1e12
        secondary["sustained"] = {
            "step": {"seconds": ms_s * n_s * 1e-3, "steps": n_s, "ms_per_step": ms_s, "tokens_per_s_layer": spec.window / (ms_s * 1e-3),
                     "launch": "graph replays" if step_graph is not None else "eager calls",
                     "sm_mhz_median": ck_s["sm_mhz"], "ms_x_mhz": ms_s * (ck_s["sm_mhz"] or 0), "reasons": ck_s["reasons"]},
            "attention": {"seconds": ms_a * n_a * 1e-3, "launches": n_a, "us_per_launch": ms_a * 1e3, "TFLOPs": tf_a,
                          "frac_of_sustained_bf16_peak": tf_a / peaks["bf16_tflops_sustained"],
                          "sm_mhz_median": ck_a["sm_mhz"], "reasons": ck_a["reasons"]}}
        # ---- the whole 32k prefill sweep, window by window (timed while the states were built)
        sweep_all = list(sweep_us) + [stage_free_step_us(stage_all)]
        secondary["sweep_32k"] = {"windows": len(sweep_all), "sum_ms": float(np.sum(sweep_all)) * 1e-3,
                                  "tokens_per_s_layer": spec.context / (float(np.sum(sweep_all)) * 1e-6),
                                  "first_window_us": sweep_all[0], "last_window_us": sweep_all[-1],
                                  "note": "every window timed alone with CUDA events after an L2 flush; the last one is the headline step"}
        sweep_all[-1] = ms_step * 1e3
        secondary["sweep_32k"]["sum_ms"] = float(np.sum(sweep_all)) * 1e-3
        secondary["sweep_32k"]["tokens_per_s_layer"] = spec.context / (float(np.sum(sweep_all)) * 1e-6)
        secondary["sweep_32k"]["last_window_us"] = sweep_all[-1]
        # ---- batched shapes of the memory-bound stages, the full-size score launch, the 131k sweep
        del states, inputs
        torch.cuda.empty_cache()
        iters = 20
        s32 = measure_stack32(iters, device)
        torch.cuda.empty_cache()
        d16 = measure_decode16(iters, device)
        torch.cuda.empty_cache()
        sfull = measure_score_full(iters, device)
        torch.cuda.empty_cache()

        def pick(d, name, alias=None):
            x = d["stages"][name]
            return {"us": x["us"], "min_us": x["min_us"], "bytes": x["bytes"], "GBps": x["GBps"],
                    "frac_of_measured_hbm": x["frac_of_measured_hbm"]}
        secondary["stages_batched"] = {
            "stack32": {"workload": s32["workload"], "bias_probe": pick(s32, "bias_probe"),
                        "score_select": pick(s32, "score_select"), "score_blocks": pick(s32, "score_blocks"),
                        "select_cutoff": pick(s32, "select_cutoff"), "append": pick(s32, "append")},
            "decode16": {"workload": d16["workload"], "score_select": pick(d16, "score_select"),
                         "score_blocks": pick(d16, "score_blocks"), "select_cutoff": pick(d16, "select_cutoff"),
                         "attention_decode": pick(d16, "attention_decode"), "keys_per_head": d16["keys_per_head"],
                         "model_step_32_layers": d16["stages"]["model_step_32_layers"]},
            "score_full_decode_step": sfull, "hbm_peak_gbs": peaks["hbm_gbs"], "peak_source": peaks["source"],
            "cold_l2": "512 MB read through L2 before every timed launch; median of 20 launches"}
        secondary["long131k"] = measure_long131k(device, peaks)
        torch.cuda.empty_cache()

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "llama3_8b_layer_32k: last window (p0=32256) of a 32768-token prefill, "
                               f"Hq=32 Hkv=8 D=128 W=512 B=128 r=4 n_init=128 k=cap=32, bf16 {spec.page_tokens}-token pages",
                   "cold_l2": f"{n_copies} distinct layer-state copies rotated (inputs larger than L2)",
                   "selected_blocks": c_sel, "parallelism": f"independent layers x{world}", "streams": "append on a second stream beside the attention, joined every step",
                   "launch": "eager calls" if args.eager else f"one CUDA graph of the {args.steps} steps, replayed per repetition"},
        "clocks": clocks, "e2e": e2e, "gpu_launches": launches_per_step * args.steps * len(rep_ms),
        "roofline": roofline, "stages": stages, "step_stats": step_stats,
    }
    line.update(secondary)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"], line["parity"] = cpu_baseline(spec, budget_s=args.cpu_budget, gpu=parity_sample)
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------------
def _oracle_sample(spec, st_cache, q, k, v, heads):
    """Times the oracle on one window: steps 1-4 in full, attention for `heads` KV heads."""
    from oracle import actqkv_oracle as orc
    state, chain, table = st_cache
    t0 = time.perf_counter()
    s2 = state.stats.copy()
    s2.update(q)
    phi, a = orc.activation_bias(q, s2.mean, s2.variance())
    pq = orc.probe_query(q, a)
    pkv = orc.kv_head_probe(pq, spec.n_kv_heads)
    p0 = state.k_cache.shape[0]
    n = orc.n_candidate_blocks(p0, spec.n_init, spec.block, spec.n_local_prev)
    s = orc.block_scores(pkv, table[:, :n])
    theta = orc.information_density(s)
    c = min(spec.k_blocks, n)
    sel = [orc.select_blocks(s[g], c)[0] for g in range(spec.n_kv_heads)]
    t1 = time.perf_counter()
    G = spec.group
    for g in heads:
        orc.retrieval_attention(q[:, g * G:(g + 1) * G], k[:, g:g + 1], v[:, g:g + 1], state.k_cache[:, g:g + 1],
                                state.v_cache[:, g:g + 1], p0, [sel[g]], spec.n_init, spec.block, spec.n_local_prev)
    t2 = time.perf_counter()
    return t1 - t0, t2 - t1


def _oracle_state(spec):
    from oracle import actqkv_oracle as orc
    from paper_2502_13542_b200 import workloads as wl
    from oracle.runner import OracleRunner
    run = OracleRunner(spec)
    T = spec.n_windows
    for t in range(T - 1):
        run.state.stats.update(wl.gen_q(spec, 0, t))
        k, v = wl.gen_kv(spec, 0, t)
        run.state.k_cache, run.state.v_cache = orc.append_window(run.state.k_cache, run.state.v_cache, k, v)
    run._extend_table(run.complete_blocks())
    q = wl.gen_q(spec, 0, T - 1)
    k, v = wl.gen_kv(spec, 0, T - 1)
    return (run.state, run.chain, run.table), q, k, v


def oracle_parity(spec, st_cache, q, k, v, gpu, head=3):
    """The timed configuration against the oracle: the selected block sets of every KV head, and the
    bf16-stored attention output of the query heads of one KV head, element by element."""
    from oracle import actqkv_oracle as orc
    state, chain, table = st_cache
    s2 = state.stats.copy()
    s2.update(q)
    _, a = orc.activation_bias(q, s2.mean, s2.variance())
    pkv = orc.kv_head_probe(orc.probe_query(q, a), spec.n_kv_heads)
    p0 = state.k_cache.shape[0]
    n = orc.n_candidate_blocks(p0, spec.n_init, spec.block, spec.n_local_prev)
    sc = orc.block_scores(pkv, table[:, :n])
    c = min(spec.k_blocks, n)
    picks = [orc.select_blocks(sc[g], c) for g in range(spec.n_kv_heads)]
    set_diffs = sum(len(set(gpu["sel"][g][:gpu["c"]].tolist()) ^ set(picks[g][0].tolist())) for g in range(spec.n_kv_heads))
    G = spec.group
    o, _ = orc.retrieval_attention(q[:, head * G:(head + 1) * G], k[:, head:head + 1], v[:, head:head + 1],
                                   state.k_cache[:, head:head + 1], state.v_cache[:, head:head + 1], p0,
                                   [gpu["sel"][head][:gpu["c"]]], spec.n_init, spec.block, spec.n_local_prev)
    d = np.abs(gpu["out"][:, head * G:(head + 1) * G].astype(np.float64) - o)
    return {"max_abs": float(d.max()), "mean_abs": float(d.mean()), "count_matches": bool(gpu["c"] == c),
            "selected_set_differences": int(set_diffs), "out_dtype": "bf16",
            "sample": f"attention output of the {G} query heads of KV head {head} at the last window (all {spec.window} tokens), "
                      f"block sets of all {spec.n_kv_heads} KV heads"}


def cpu_baseline(spec, budget_s=12.0, gpu=None):
    """The oracle as it stands on the host cores: whole windows (steps 1-4 and the attention of all
    KV heads) repeated until about `budget_s` seconds of work have been timed.  Returns the baseline
    record and, when a device result is given, its comparison with the oracle."""
    import torch
    st, q, k, v = _oracle_state(spec)
    parity = oracle_parity(spec, st, q, k, v, gpu) if gpu is not None else None
    heads = list(range(spec.n_kv_heads))
    _oracle_sample(spec, st, q, k, v, heads=heads[:1])        # page in BLAS
    times = []
    t_start = time.perf_counter()
    while len(times) < 3 or time.perf_counter() - t_start < budget_s:
        t14, tatt = _oracle_sample(spec, st, q, k, v, heads=heads)
        times.append(t14 + tatt)
    est = float(np.mean(times))
    return {"value": spec.window / est, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
            "sample": f"{len(times)} whole windows of the bench workload (steps 1-4 + attention of all "
                      f"{spec.n_kv_heads} KV heads), {sum(times):.1f} s of oracle time, mean {est:.3f} s per window; "
                      "NumPy fp64, its matrix products on the BLAS thread pool"}, parity


def blas_threads() -> int:
    """Threads the oracle's matrix products actually use: the size of NumPy's BLAS pool."""
    try:
        from threadpoolctl import threadpool_info
        n = [p["num_threads"] for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return int(max(n))
    except Exception:
        pass
    return int(os.environ.get("OMP_NUM_THREADS", 0)) or (os.cpu_count() or 1)


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2502_13542_b200 import workloads as wl
    spec = wl.llama3_8b_layer()
    st, q, k, v = _oracle_state(spec)
    times = []
    heads = list(range(spec.n_kv_heads))
    for i in range(args.warmup + args.steps):
        t14, tatt = _oracle_sample(spec, st, q, k, v, heads=heads)
        if i >= args.warmup:
            times.append(t14 + tatt)
    ms = 1e3 * float(np.mean(times))
    val = spec.window / (ms * 1e-3)
    cores = blas_threads()
    sample = "each step: one whole window of the bench workload through the oracle (steps 1-4 + attention of all 8 KV heads)"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "llama3_8b_layer_32k: last window (p0=32256) of a 32768-token prefill (CPU oracle)"},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))

# ------------------------------------------------------------------------------------------
# Secondary workloads (not the default headline line): the memory-bound stages on batched shapes
def _device_activations(spec, shape_heads, device, gen, n_tokens):
    """Seeded N(0,1) activations with the workload's outlier channels, drawn on the device
    (bench-only inputs: the parity tests use the host generator of workloads.py)."""
    import torch
    x = torch.randn(*shape_heads[:-1], n_tokens, shape_heads[-1], spec.head_dim, device=device, generator=gen)
    x[..., : spec.n_outlier] *= spec.outlier_scale
    return x.to(torch.bfloat16)


def _time_stage(fn, iters, flush):
    import torch
    evs = []
    for _ in range(iters):
        flush()
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        e0.record(); fn(); e1.record()
        evs.append((e0, e1))
    torch.cuda.synchronize()
    t = sorted(a.elapsed_time(b) for a, b in evs)
    return 1e3 * t[len(t) // 2], 1e3 * t[0]          # median and minimum, microseconds


def measure_stack32(iters, dev, n_layers=32):
    """All 32 layers of the LLaMA3-8B shape batched in one launch per stage at the last window of a
    32k prefill: Q = 134 MB, representative table = 66 MB per launch (larger than or comparable
    to L2; L2 is flushed before every timed launch)."""
    import torch
    from paper_2502_13542_b200 import binding as B
    from paper_2502_13542_b200 import workloads as wl
    spec = wl.llama3_8b_stack32().replace(n_layers=n_layers)
    L = spec.n_layers
    cfg = B.make_config(spec, out_dtype=B.BF16)
    st = B.RetrievalState(cfg, n_seq=1, n_layers=L, page_table=wl.shuffled_page_table(spec, spec.context)[None, :], device=dev)
    gen = torch.Generator(device=dev).manual_seed(spec.seed)
    out = torch.zeros(L, spec.window, spec.n_q_heads, spec.head_dim, dtype=torch.bfloat16, device=dev)
    W = spec.window
    for t in range(spec.n_windows - 1):
        q = _device_activations(spec, (L, spec.n_q_heads), dev, gen, W)
        k = _device_activations(spec, (L, spec.n_kv_heads), dev, gen, W)
        v = _device_activations(spec, (L, spec.n_kv_heads), dev, gen, W)
        st.step(q, k, v, out)
    q = _device_activations(spec, (L, spec.n_q_heads), dev, gen, W)
    k = _device_activations(spec, (L, spec.n_kv_heads), dev, gen, W)
    v = _device_activations(spec, (L, spec.n_kv_heads), dev, gen, W)
    torch.cuda.synchronize()
    scratch = torch.zeros(512 << 20, dtype=torch.uint8, device=dev)
    flush = lambda: scratch.view(torch.int32).sum()      # reading leaves clean lines: no write-back traffic in the timed launch
    b = st.batch
    p0 = (spec.n_windows - 1) * W
    sb = stage_bytes(spec, p0)
    stages = {
        "bias_probe": (lambda: B.bias_probe(cfg, b, q, W, st.stats_count, st.stats_mean, st.stats_m2, st.phi_l1, None,
                                            st.probe_qh, st.probe_kv, st.status), L * sb["bias_probe"]),
        "score_select": (lambda: B.score_select(cfg, b, st.probe_kv, st.repr_k, st.repr_inv_norm, st.n_cand,
                                                st.budget_state, st.scores, st.theta, st.sel_idx, st.sel_count,
                                                st.budget_real, st.status), L * (sb["score"] + sb["select"])),
        "append": (lambda: B.append_window(cfg, b, k, v, W, st.pos0, st.k_pages, st.v_pages, st.page_table,
                                           st.repr_k, st.repr_inv_norm, st.status), L * sb["append"]),
        "score_blocks": (lambda: B.score_blocks(cfg, b, st.probe_kv, st.repr_k, st.repr_inv_norm, st.n_cand, st.scores,
                                                st.theta, st.status), L * sb["score"]),
        "select_cutoff": (lambda: B.select_cutoff(cfg, b, st.scores, st.theta, st.n_cand, st.budget_state, st.sel_idx,
                                                  st.sel_count, st.budget_real, st.status), L * sb["select"]),
    }
    peaks = load_peaks()
    res = {}
    for name, (fn, nbytes) in stages.items():
        for _ in range(3):
            fn()
        us, us_min = _time_stage(fn, iters, flush)
        res[name] = {"us": us, "min_us": us_min, "bytes": nbytes, "GBps": nbytes / us / 1e3,
                     "frac_of_measured_hbm": nbytes / us / 1e3 / peaks["hbm_gbs"]}
    assert int(st.status.item()) == 0
    return {"workload": f"llama3_8b_stack32_32k: {L} layers batched per launch, last window", "stages": res,
            "hbm_peak_gbs": peaks["hbm_gbs"], "peak_source": peaks["source"],
            "cold_l2": "512 MB read through L2 before every timed launch"}


def measure_decode16(iters, dev, decode_splits=1):
    """Decode, 16 sequences with contexts ~ U[32768, 131072], one token per step, one layer per
    launch, probes fixed: score + cut-off/select over every sequence's table, then the decode
    attention over [128 initial | 32 selected blocks | >= 512 local] keys per KV head."""
    import torch
    from paper_2502_13542_b200 import binding as B
    from paper_2502_13542_b200 import workloads as wl
    spec = wl.decode_batch16().replace(n_layers=1, cap_blocks=32)
    S = spec.n_seq
    ctx = (wl.decode_contexts(spec) // spec.window) * spec.window
    n_pools = 2                                             # distinct physical layer copies, rotated
    max_ctx = int(ctx.max()) + spec.window
    pages_per_seq = -(-max_ctx // 16)
    cfg = B.make_config(spec, out_dtype=B.BF16, max_context=max_ctx, n_phys_pages=S * pages_per_seq)
    gen = torch.Generator(device=dev).manual_seed(spec.seed)
    rng = np.random.default_rng(spec.seed)
    table = rng.permutation(S * pages_per_seq).astype(np.int32).reshape(S, pages_per_seq)[:, : cfg.max_pages]
    states = []
    pre_spec = spec.replace(n_local_prev=0)
    pre_cfg = B.make_config(pre_spec, out_dtype=B.BF16, max_context=max_ctx, n_phys_pages=S * pages_per_seq)
    for pool in range(n_pools):
        st = B.RetrievalState(cfg, n_seq=S, n_layers=1, page_table=table, device=dev)
        outw = torch.zeros(1, spec.window, spec.n_q_heads, spec.head_dim, dtype=torch.bfloat16, device=dev)
        for s_i in range(S):
            ps = B.RetrievalState(pre_cfg, n_seq=1, n_layers=1, page_table=table[s_i:s_i + 1], device=dev,
                                  shared_pages=(st.k_pages, st.v_pages))
            for t in range(int(ctx[s_i]) // spec.window):
                qw = _device_activations(spec, (1, spec.n_q_heads), dev, gen, spec.window)
                kw = _device_activations(spec, (1, spec.n_kv_heads), dev, gen, spec.window)
                vw = _device_activations(spec, (1, spec.n_kv_heads), dev, gen, spec.window)
                ps.step(qw, kw, vw, outw)
            for name in ("repr_k", "repr_inv_norm", "probe_kv", "probe_qh"):
                getattr(st, name)[s_i:s_i + 1].copy_(getattr(ps, name))
            st.budget_state[s_i].copy_(ps.budget_state[0])
            del ps
        st.set_positions([int(c) for c in ctx])
        states.append(st)
    torch.cuda.synchronize()
    q = _device_activations(spec, (S, spec.n_q_heads), dev, gen, 1)
    k = _device_activations(spec, (S, spec.n_kv_heads), dev, gen, 1)
    v = _device_activations(spec, (S, spec.n_kv_heads), dev, gen, 1)
    out = torch.zeros(S, 1, spec.n_q_heads, spec.head_dim, dtype=torch.bfloat16, device=dev)
    scratch = torch.zeros(512 << 20, dtype=torch.uint8, device=dev)
    flush = lambda: scratch.view(torch.int32).sum()      # reading leaves clean lines: no write-back traffic in the timed launch
    it = {"i": 0}

    def cur():
        return states[it["i"] % n_pools]

    def score_select():
        st = cur()
        B.score_select(cfg, st.batch, st.probe_kv, st.repr_k, st.repr_inv_norm, st.n_cand, st.budget_state, st.scores,
                       st.theta, st.sel_idx, st.sel_count, st.budget_real, st.status)

    ws = None
    if decode_splits > 1:           # split form of the decode kernel, with a caller-owned workspace
        ws = torch.zeros(B.decode_workspace_bytes(cfg, states[0].batch, 1, decode_splits), dtype=torch.uint8, device=dev)

    def attention():
        st = cur()
        if ws is None:
            B.retrieval_attention(cfg, st.batch, q, k, v, 1, st.k_pages, st.v_pages, st.page_table, st.pos0, st.sel_idx,
                                  st.sel_count, out, None, st.status)
        else:
            B.decode_attention(cfg, st.batch, q, k, v, 1, st.k_pages, st.v_pages, st.page_table, st.pos0, st.sel_idx,
                               st.sel_count, out, None, decode_splits, ws, st.status)
        it["i"] += 1
    e = 2
    n_blocks = [wl.n_candidates(spec, int(c)) for c in ctx]
    score_bytes = sum(n * spec.n_kv_heads * spec.n_repr * (spec.head_dim * e + 4) + n * spec.n_kv_heads * 4 for n in n_blocks)
    for st in states:
        score_select_st = st
    score_select(); torch.cuda.synchronize()
    c_sel = cur().sel_count.cpu().numpy()
    keys = [spec.n_init + int(c_sel[i]) * spec.block + (int(ctx[i]) - (spec.n_init + n_blocks[i] * spec.block)) + 1 for i in range(S)]
    att_bytes = sum(kk * spec.n_kv_heads * spec.head_dim * e * 2 for kk in keys)
    peaks = load_peaks()
    res = {}
    def score_only():
        st = cur()
        B.score_blocks(cfg, st.batch, st.probe_kv, st.repr_k, st.repr_inv_norm, st.n_cand, st.scores, st.theta, st.status)

    def select_only():
        st = cur()
        B.select_cutoff(cfg, st.batch, st.scores, st.theta, st.n_cand, st.budget_state, st.sel_idx, st.sel_count,
                        st.budget_real, st.status)

    for name, fn, nbytes in (("score_select", score_select, score_bytes), ("attention_decode", attention, att_bytes),
                             ("score_blocks", score_only, score_bytes), ("select_cutoff", select_only, 0)):
        for _ in range(3):
            fn()
        us, us_min = _time_stage(fn, iters, flush)
        res[name] = {"us": us, "min_us": us_min, "bytes": nbytes, "GBps": nbytes / us / 1e3,
                     "frac_of_measured_hbm": nbytes / us / 1e3 / peaks["hbm_gbs"]}
    # ---- a whole decode step of a 32-layer model with the paper's decode probe q^t (Sec. 4.2): per
    # layer probe -> score -> cut-off / select -> decode attention -> append of the token, the layers
    # rotating over the physical pools; enqueued call by call, and captured once into a CUDA graph.
    n_model_layers = 32

    def layer_step(l):
        st = states[l % n_pools]
        B.probe_query(cfg, st.batch, q, 1, None, st.probe_qh, st.probe_kv, st.status)
        B.score_select(cfg, st.batch, st.probe_kv, st.repr_k, st.repr_inv_norm, st.n_cand, st.budget_state, st.scores,
                       st.theta, st.sel_idx, st.sel_count, st.budget_real, st.status)
        if ws is None:
            B.retrieval_attention(cfg, st.batch, q, k, v, 1, st.k_pages, st.v_pages, st.page_table, st.pos0, st.sel_idx,
                                  st.sel_count, out, None, st.status)
        else:
            B.decode_attention(cfg, st.batch, q, k, v, 1, st.k_pages, st.v_pages, st.page_table, st.pos0, st.sel_idx,
                               st.sel_count, out, None, decode_splits, ws, st.status)
        B.append_window(cfg, st.batch, k, v, 1, st.pos0, st.k_pages, st.v_pages, st.page_table, st.repr_k,
                        st.repr_inv_norm, st.status)

    def model_step():
        for l in range(n_model_layers):
            layer_step(l)

    def time_model_step(fn):
        for _ in range(2):
            fn()
        ts = []
        for _ in range(max(5, iters // 2)):
            a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            a.record(); fn(); b.record()
            torch.cuda.synchronize()
            ts.append(1e3 * a.elapsed_time(b))
        return float(np.median(ts)), float(np.min(ts))

    eager_us, eager_min = time_model_step(model_step)
    step_graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(step_graph):
        model_step()
    graph_us, graph_min = time_model_step(step_graph.replay)
    step_bytes = n_model_layers * (score_bytes + att_bytes)
    res["model_step_32_layers"] = {
        "us_graph": graph_us, "min_us_graph": graph_min, "us_eager": eager_us, "min_us_eager": eager_min,
        "us_per_layer_graph": graph_us / n_model_layers, "tokens_per_s": S / (graph_us * 1e-6),
        "bytes": step_bytes, "GBps": step_bytes / graph_us / 1e3,
        "frac_of_measured_hbm": step_bytes / graph_us / 1e3 / peaks["hbm_gbs"],
        "note": "probe q^t -> score -> cut-off / select -> decode attention -> append per layer, 32 layers over "
                f"{n_pools} physical pools (their tables and pages are larger than L2), no flush between layers"}
    assert all(int(st.status.item()) == 0 for st in states)
    return {"workload": f"decode16: 16 sequences, contexts {int(ctx.min())}..{int(ctx.max())}, 1 token per step, "
                        f"one layer per launch, {n_pools} layer pools rotated",
            "keys_per_head": {"min": min(keys), "max": max(keys)}, "stages": res,
            "hbm_peak_gbs": peaks["hbm_gbs"], "peak_source": peaks["source"],
            "cold_l2": "512 MB read through L2 before every timed launch"}


def measure_score_full(iters, dev):
    """Step 3 at the size of a whole decode step: 16 sequences x 32 layers scored in ONE launch, as
    Algorithm 1 does when every layer's scores are taken before any budget.  The table holds
    contexts ~ U[32768, 131072] (n = 251..1019 candidate blocks per sequence), filled with seeded
    random keys and their true inverse norms (the kernel's traffic does not depend on the values);
    algorithmic bytes = the candidate rows, their inverse norms and the scores written."""
    import torch
    from paper_2502_13542_b200 import binding as B
    from paper_2502_13542_b200 import workloads as wl
    spec = wl.decode_batch16()
    S, L, Hkv, D, r = spec.n_seq, spec.n_layers, spec.n_kv_heads, spec.head_dim, spec.n_repr
    ctx = (wl.decode_contexts(spec) // spec.window) * spec.window
    n_blocks = [wl.n_candidates(spec, int(c)) for c in ctx]
    n_cap = max(n_blocks)
    cfg = B.make_config(spec, out_dtype=B.BF16, n_cap=n_cap, max_context=int(ctx.max()) + spec.window)
    gen = torch.Generator(device=dev).manual_seed(spec.seed)
    U = S * L
    repr_k = torch.empty(U, Hkv, n_cap, r, D, dtype=torch.bfloat16, device=dev)
    inv = torch.empty(U, Hkv, n_cap, r, dtype=torch.float32, device=dev)
    for u0 in range(0, U, 32):                       # filled in slices: the fp32 temporaries stay small
        x = torch.randn(32, Hkv, n_cap, r, D, device=dev, generator=gen)
        repr_k[u0:u0 + 32] = x.to(torch.bfloat16)
        inv[u0:u0 + 32] = 1.0 / repr_k[u0:u0 + 32].float().norm(dim=-1)
        del x
    probe = torch.randn(U, Hkv, D, device=dev, generator=gen)
    scores = torch.zeros(U, Hkv, n_cap, device=dev)
    theta = torch.zeros(U, Hkv, device=dev)
    n_cand = torch.tensor(n_blocks, dtype=torch.int32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    batch = B.Batch(S, L, 0)
    nbytes = L * sum(n * Hkv * r * (D * 2 + 4) + n * Hkv * 4 for n in n_blocks)
    fn = lambda: B.score_blocks(cfg, batch, probe, repr_k, inv, n_cand, scores, theta, status)
    for _ in range(3):
        fn()
    flush = l2_flusher(dev)
    us, us_min = _time_stage(fn, iters, flush)
    assert int(status.item()) == 0
    peaks = load_peaks()
    return {"workload": f"score_blocks over 16 sequences x 32 layers in one launch ({nbytes / 1e9:.2f} GB of table rows)",
            "us": us, "min_us": us_min, "bytes": nbytes, "GBps": nbytes / us / 1e3,
            "frac_of_measured_hbm": nbytes / us / 1e3 / peaks["hbm_gbs"]}


def measure_long131k(dev, peaks):
    """The 131072-token prefill of one layer (k = cap = 128 blocks): every one of the 256 windows is
    timed as it is prefilled (L2 flushed before each), which gives the sweep average
    131072 / sum_t t_window(t); the last window (17,024 keys per query) is then repeated for the
    step time and the attention's tensor-core fraction at that length."""
    import torch
    from paper_2502_13542_b200 import binding as B
    from paper_2502_13542_b200 import workloads as wl
    spec = wl.long_131k()
    flush = l2_flusher(dev)
    sweep = []
    cfg, states, inputs = build_states(spec, 1, dev, sweep_times=sweep, flush=flush)
    st = states[0]
    q, k, v, out = inputs[0]
    W = spec.window
    p0 = (spec.n_windows - 1) * W
    att, step = [], []
    for i in range(23):
        flush()
        e0, e1, e2, e3 = (torch.cuda.Event(enable_timing=True) for _ in range(4))
        e0.record()
        st.step(q, k, v, out, advance=False, overlap_append=True)
        e1.record()
        flush()
        e2.record()
        B.retrieval_attention(cfg, st.batch, q, k, v, W, st.k_pages, st.v_pages, st.page_table, st.pos0, st.sel_idx,
                              st.sel_count, out, None, st.status)
        e3.record()
        torch.cuda.synchronize()
        if i >= 3:
            step.append(1e3 * e0.elapsed_time(e1)); att.append(1e3 * e2.elapsed_time(e3))
    assert int(st.status.item()) == 0
    sweep.append(float(np.median(step)))               # the last window, which the prefill loop leaves out
    c_sel = int(st.sel_count.item())
    flops = attention_flops(spec, p0, c_sel)
    att_us = float(np.median(att))
    tf = flops / (att_us * 1e-6) / 1e12
    return {"workload": "llama3_8b_layer_131k: 256 windows of 512 tokens, k = cap = 128 blocks",
            "last_window": {"step_us": float(np.median(step)), "step_min_us": float(np.min(step)),
                            "tokens_per_s_layer": W / (float(np.median(step)) * 1e-6), "selected_blocks": c_sel,
                            "attention_us": att_us, "attention_min_us": float(np.min(att)),
                            "attention_TFLOPs": tf, "attention_frac_of_measured_bf16": tf / peaks["bf16_tflops"],
                            "attention_flops": flops},
            "sweep": {"windows": len(sweep), "sum_ms": float(np.sum(sweep)) * 1e-3,
                      "tokens_per_s_layer": spec.context / (float(np.sum(sweep)) * 1e-6),
                      "first_window_us": sweep[0], "window_64_us": sweep[63], "window_128_us": sweep[127]}}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=400)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--copies", type=int, default=8)
    ap.add_argument("--cpu-budget", type=float, default=12.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--workload", default="layer32k", choices=["layer32k", "stack32", "decode16", "long131k", "scorefull"],
                    help="layer32k = the headline line (which also carries the others' figures unless --headline-only); "
                         "the others print one secondary measurement alone")
    ap.add_argument("--stack-layers", type=int, default=32, help="stack32 workload: layers batched per launch")
    ap.add_argument("--reps", type=int, default=20, help="repetitions of the timed K-step region (median reported)")
    ap.add_argument("--page-tokens", type=int, default=16, choices=[16, 32, 64, 128],
                    help="tokens per cache page of the layer32k workload (the headline workload has 16)")
    ap.add_argument("--eager", action="store_true",
                    help="enqueue the timed steps call by call from Python instead of replaying a CUDA graph of them")
    ap.add_argument("--headline-only", action="store_true",
                    help="skip the secondary measurements (batched stages, 131k sweep, sustained loop)")
    ap.add_argument("--decode-splits", type=int, default=1,
                    help="decode16 workload: key-stream splits per (sequence, KV head) of the decode attention")
    ap.add_argument("--profile-region", action="store_true",
                    help="bracket the timed region with cudaProfilerStart/Stop (for ncu --profile-from-start off)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.gpus != world:
        if "WORLD_SIZE" in os.environ or args.gpus < 1:
            sys.exit(f"bench.py: --gpus {args.gpus} does not match WORLD_SIZE={world} of the launcher")
        # started as a plain process with --gpus N > 1: become N ranks, one per GPU, under torchrun
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", os.environ.get("MASTER_PORT", "29517"),
               os.path.abspath(__file__)] + sys.argv[1:]
        os.execv(sys.executable, cmd)
    if args.impl == "reference":
        args.steps = min(args.steps, 30)
        args.warmup = min(args.warmup, 2)
        run_reference(args)
    elif args.workload == "layer32k":
        run_ours(args)
    else:
        import torch
        torch.cuda.set_device(0)
        dev = torch.device("cuda", 0)
        iters = args.steps if args.steps < 100 else 30
        if args.workload == "stack32":
            print(json.dumps(measure_stack32(iters, dev, args.stack_layers)))
        elif args.workload == "decode16":
            print(json.dumps(measure_decode16(iters, dev, args.decode_splits)))
        elif args.workload == "scorefull":
            print(json.dumps(measure_score_full(iters, dev)))
        else:
            print(json.dumps(measure_long131k(dev, load_peaks())))


if __name__ == "__main__":
    main()
