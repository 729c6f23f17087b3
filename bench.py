#!/usr/bin/env python
"""Benchmark of the routing-aware EP hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload C4] [--impl ours|reference]

One step = layout -> dispatch -> combine over one batch of seeded synthetic routing
(combine reads T*K independent expert-output rows in the pair space). Prints ONE
JSON line on rank 0. The headline workload is C4 (the largest configuration); the
same line carries, under `configs`, the step and per-kernel figures of the other
configurations (C1, C2, C3 and the host-staged C5 with its host-link roofline).
With N > 1 every rank runs an independent replica of the workload (the path has no
exchange between GPUs); the time is the max over ranks.
`--impl reference` times the CPU oracle on the host cores on the same batch.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time
from concurrent.futures import ThreadPoolExecutor

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

METRIC = "ep_layout_dispatch_combine_tokens_per_s"
UNIT = "tokens/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
# DRAM bytes per launch of the dominant kernels from the committed ncu captures (profiles/).
NCU_TRAFFIC_BYTES = {("C4", "combine_rows_kernel"): 1038.7e6, ("C4", "dispatch_rows_kernel"): 680.9e6}
L2_BYTES = 126e6
CONTEXT = ("paper reports 2.00x (dispatch) / 1.53x (combine) over NCCL for its dense all-gather/"
           "reduce-scatter on RTX 4090/5090 PCIe boxes; no number for the routing-aware path")


class L2Flush:
    """Evicts the working set from the 126 MB L2 between timed steps: writes a 256 MB buffer, then
    reads a second one, so that L2 ends up holding clean lines of a foreign buffer. (After the write
    alone, ~126 MB of dirty lines would be written back during the next timed kernel and be charged to it.)"""

    def __init__(self, dev, nbytes=256 << 20):
        self.w = torch.empty(nbytes, dtype=torch.uint8, device=dev)
        self.r = torch.zeros(nbytes // 4, dtype=torch.int32, device=dev)
        self.i = 0

    def __call__(self):
        self.i += 1
        self.w.fill_(self.i & 0xff)
        torch.sum(self.r)


def stats_us(ms_values):
    a = np.asarray(ms_values, dtype=np.float64) * 1e3
    return {"us": float(a.mean()), "median_us": float(np.median(a)), "best_us": float(a.min())}


def workload_text(cfg):
    routing = {"uniform": "uniform routing", "zipf": "Zipf(1.1) expert popularity, seeded permutation",
               "burst": "uniform routing + 10% hot-expert burst on expert 0"}[cfg.routing]
    return (f"{cfg.name}: T={cfg.T} H={cfg.H} E={cfg.E} K={cfg.K} R={cfg.R}, {routing}, bf16 N(0,1) rows, "
            f"softmax weights" + (", receive buffer in mapped pinned host memory" if cfg.host_staged else ""))


def step_bytes_estimate(cfg):
    return 2 * cfg.H * (2 * cfg.T + cfg.T * min(cfg.K, cfg.R) + cfg.T * cfg.K)


def is_small(cfg):
    """The step's data could (partly) stay in L2 from one step to the next."""
    return step_bytes_estimate(cfg) < 4 * L2_BYTES and not cfg.host_staged


def config_object(cfg, world, n_recv, n_pairs):
    """The `config` of the JSON line: a function of the workload alone, identical in both arms."""
    l2 = ("step data would fit L2: before every timed step 256 MB are written and then another 256 MB read "
          "(L2 left holding clean foreign lines); each step timed by its own event pair") if is_small(cfg) else \
        "working set per step exceeds L2 several times over (no flush needed)"
    return {"workload": workload_text(cfg), "parallelism": f"{world} independent replica(s)", "l2": l2,
            "n_recv": int(n_recv), "n_pairs": int(n_pairs)}


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


def algorithmic_bytes(cfg, n_recv, n_pairs):
    row = 2 * cfg.H
    return {
        "layout": 4 * cfg.T * cfg.K * 6 + 4 * (2 * cfg.E + cfg.R * cfg.R + n_recv),
        "dispatch": row * cfg.T + row * n_recv + 4 * cfg.T * cfg.K,
        "combine": row * n_pairs + row * cfg.T + 8 * cfg.T * cfg.K,
    }


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML while a region runs."""

    def __init__(self, device_index: int, period_s: float = 0.002):
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        self._h = None
        self.period = period_s
        try:
            import pynvml
            self.nv = pynvml
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            try:
                self._h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + uuid).encode())
            except Exception:
                self._h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._h = None

    def _loop(self):
        nv = self.nv
        names = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "sw_thermal_slowdown": 0x20,
                 "hw_thermal_slowdown": 0x40, "hw_power_brake_slowdown": 0x80, "sync_boost": 0x10}
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                try:
                    bits = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
                except Exception:
                    bits = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
                for n, b in names.items():
                    if bits & b:
                        self.reasons.add(n)
            except Exception:
                pass
            self._stop.wait(self.period)

    def __enter__(self):
        if self._h is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["unavailable"], "samples": 0}
        return {"sm_mhz": int(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


# --------------------------------------------------------------------------- CPU oracle legs

def oracle_step(oracle, cfg, idx, w, x, out):
    """One whole step of the oracle as it stands, one thread."""
    lay = oracle.layout(idx, cfg.E, cfg.R)
    oracle.dispatch(x, lay.recv_slot, lay.n_recv)
    oracle.combine_f32(out, lay.pair_slot, w)


def oracle_step_all_cores(oracle, pool, n_threads, cfg, idx, w, x, out):
    """The same step with the token range cut statically into one contiguous part per thread for
    dispatch and combine (independent per token once the slots exist); the layout stays serial.
    The oracle's C functions are called unchanged on row slices; ctypes releases the GIL."""
    lay = oracle.layout(idx, cfg.E, cfg.R)
    T = cfg.T
    cuts = [T * i // n_threads for i in range(n_threads + 1)]
    recv = np.empty((max(1, lay.n_recv), cfg.H), dtype=np.uint16)
    y = np.empty((T, cfg.H), dtype=np.uint16)
    parts = [(a, b) for a, b in zip(cuts[:-1], cuts[1:]) if b > a]
    list(pool.map(lambda ab: oracle.dispatch_into(x[ab[0]:ab[1]], lay.recv_slot[ab[0]:ab[1]], recv), parts))
    list(pool.map(lambda ab: oracle.combine_f32_into(out, lay.pair_slot[ab[0]:ab[1]], w[ab[0]:ab[1]], y[ab[0]:ab[1]]),
                  parts))


def usable_cores():
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count() or 1


def time_oracle(cfg, idx, w, x, out, min_seconds, max_steps):
    """Whole oracle steps on the given batch: one thread, then all usable cores."""
    import oracle
    oracle.build()

    def run(fn):
        fn()                                            # page in
        steps, t0 = 0, time.perf_counter()
        while True:
            fn()
            steps += 1
            el = time.perf_counter() - t0
            if el >= min_seconds or steps >= max_steps:
                return cfg.T * steps / el, steps, el

    v1, n1, el1 = run(lambda: oracle_step(oracle, cfg, idx, w, x, out))
    cores = usable_cores()
    with ThreadPoolExecutor(max_workers=cores) as pool:
        vn, nn, eln = run(lambda: oracle_step_all_cores(oracle, pool, cores, cfg, idx, w, x, out))
    return {"value": v1, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"{n1} whole step(s) of the same {cfg.name} batch in {el1:.1f} s, one thread",
            "all_cores": {"value": vn, "unit": UNIT, "cores": cores,
                          "sample": f"{nn} whole step(s) of the same batch in {eln:.1f} s; layout serial, dispatch and "
                                    f"combine split statically over {cores} threads by token range"},
            "host_cores_available": os.cpu_count()}


def run_reference(args, cfg):
    """The CPU oracle as the reference arm, on the same batch and generators as the GPU arm: each step
    is one whole oracle step (layout + dispatch + combine, one thread) over all T tokens."""
    from paper_2609_40093_b200 import inputs
    import oracle
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    oracle.build()
    d = inputs.make_inputs(cfg, args.seed)
    idx, w, x = d["topk_idx"], d["topk_weights"], d["x"]
    out = inputs.make_out(cfg, cfg.T * cfg.K, args.seed)
    lay = oracle.layout(idx, cfg.E, cfg.R)
    # every step is the whole batch unless the requested number of steps would then run for more than ~3 minutes
    # (the driver's --steps 20 --warmup 5 takes ~25 s at C4); only then each step is the first `sample` tokens
    sample = cfg.T
    t0 = time.perf_counter()
    oracle_step(oracle, cfg, idx, w, x, out)
    est = time.perf_counter() - t0
    while est * (args.steps + args.warmup) > 180 and sample > 8 * cfg.R:
        sample = max(cfg.R, (sample // 2) - (sample // 2) % cfg.R)
        est /= 2
    sub = cfg if sample == cfg.T else inputs.custom_config(sample, cfg.H, cfg.E, cfg.K, cfg.R, name=cfg.name)
    idx, w, x, out = idx[:sample], w[:sample], x[:sample], out[:sample * cfg.K]
    for _ in range(args.warmup):
        oracle_step(oracle, sub, idx, w, x, out)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_step(oracle, sub, idx, w, x, out)
    el = time.perf_counter() - t0
    value = sample * args.steps / el
    desc = (f"every step is one whole oracle step on the full {cfg.name} batch ({cfg.T} tokens), one thread" if sample == cfg.T
            else f"every step is one oracle step on the first {sample} tokens of the {cfg.name} batch (all K picks, all R ranks), "
                 f"one thread: the full batch would take {est * cfg.T / sample * (args.steps + args.warmup):.0f} s for this many steps")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": el / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic", "config": config_object(cfg, max(1, args.gpus), lay.n_recv, lay.n_pairs),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# --------------------------------------------------------------------------- GPU measurement

class Workload:
    """Device buffers and the step of one configuration."""

    def __init__(self, ep, inputs, cfg, rcfg, dev, seed, serial_layout=False, separate_calls=False, one_call=False, force_split=False):
        self.ep, self.cfg, self.dev = ep, cfg, dev
        T, K, H, E, R = cfg.T, cfg.K, cfg.H, cfg.E, cfg.R
        d = inputs.make_inputs(rcfg, seed)
        self.host = d
        self.idx_h = torch.from_numpy(d["topk_idx"]).pin_memory()
        self.w_h = torch.from_numpy(d["topk_weights"]).pin_memory()
        self.x_h = torch.from_numpy(d["x"].view(np.int16)).view(torch.bfloat16).pin_memory()
        self.idx, self.w, self.x = self.idx_h.to(dev), self.w_h.to(dev), self.x_h.to(dev)
        self.out_h = inputs.make_out(rcfg, T * K, seed)              # expert outputs, pair space (seeded, host)
        self.out = torch.from_numpy(self.out_h.view(np.int16)).view(torch.bfloat16).to(dev)
        self.lay = ep.alloc_layout(T, K, E, R, device=dev)
        self.ws = torch.empty(max(16, ep.ep_layout_workspace_bytes(T, K, E, R)), dtype=torch.uint8, device=dev)
        self.ws2 = torch.empty_like(self.ws)
        self.ws_both = torch.empty(2 * self.ws.numel() + 256, dtype=torch.uint8, device=dev)
        if cfg.host_staged:
            self.recv = torch.empty(T * min(K, R), H, dtype=torch.bfloat16).pin_memory()
        else:
            self.recv = torch.empty(T * min(K, R), H, dtype=torch.bfloat16, device=dev)
        self.y = torch.empty(T, H, dtype=torch.bfloat16, device=dev)
        # prefill-size batches (T >= 4096): the pair half of the layout runs beside dispatch; smaller ones keep one call
        self.split_layout = (not serial_layout) and (T >= 4096 or force_split) and not cfg.host_staged
        self.side = torch.cuda.Stream()
        self.fork_ev, self.join_ev = torch.cuda.Event(), torch.cuda.Event()
        self.separate_calls = separate_calls
        # batches far larger than L2: one ep_layout_dispatch call with the side stream (C4: 289.5 against 291.2 us
        # per step with separate calls); at C3 the early-resident dispatch CTAs delay the pair half (59.8 against 56.7 us)
        self.one_call_split = self.split_layout and not separate_calls and not is_small(cfg)
        # decode-size batches: layout and dispatch in one call (ep_layout_dispatch: the lean layout kernel and a dispatch
        # launched behind it; the one-launch form only for shapes the lean kernels do not cover)
        self.fused = (not separate_calls) and T <= 1024 and not cfg.host_staged
        self.one_call = one_call and not self.fused and not cfg.host_staged
        if self.one_call:
            self.split_layout = self.one_call_split = False

    def step(self, ev=None):
        """layout -> dispatch -> combine. Dispatch needs only the receive-row half of the layout, so for big
        batches the pair half (what combine needs) runs on a side stream while dispatch moves rows.
        ev: optional dict of timing events recorded between the calls."""
        ep, cfg, lay = self.ep, self.cfg, self.lay
        E, R = cfg.E, cfg.R
        main = torch.cuda.current_stream()
        if ev:
            ev["t0"].record()
        if self.one_call_split and ev is None:
            # one call: receive-row half, dispatch launched behind it, pair half on the side stream, joined at the end
            ep.ep_layout_dispatch(self.idx, self.x, self.recv, E, R, lay, self.ws_both, stream_pairs=self.side)
            ep.ep_combine(self.out, lay.pair_slot, self.w, self.y, E, R, status=lay.status)
            return
        if self.fused or self.one_call:
            ep.ep_layout_dispatch(self.idx, self.x, self.recv, E, R, lay, self.ws)    # small batches: one call for both
        elif not self.split_layout:
            ep.ep_layout(self.idx, E, R, out=lay, workspace=self.ws)
        else:
            self.fork_ev.record(main)                     # the side stream starts after everything queued so far
            ep.ep_layout_ranks(self.idx, E, R, lay, self.ws)      # critical path first
            self.side.wait_event(self.fork_ev)
            if ev:
                ev["p0"].record(self.side)
            ep.ep_layout_pairs(self.idx, E, R, lay, self.ws2, stream=self.side)
            if ev:
                ev["p1"].record(self.side)
            self.join_ev.record(self.side)
        if ev:
            ev["t1"].record()
        if not (self.fused or self.one_call):
            ep.ep_dispatch(self.x, lay.recv_slot, self.recv, E, R, status=lay.status)
        if ev:
            ev["t2"].record()
        if self.split_layout:
            main.wait_event(self.join_ev)
        if ev:
            ev["t3"].record()
        ep.ep_combine(self.out, lay.pair_slot, self.w, self.y, E, R, status=lay.status)
        if ev:
            ev["t4"].record()

    @staticmethod
    def new_events(external=False):
        kw = {"external": True} if external else {}
        return {k: torch.cuda.Event(enable_timing=True, **kw) for k in ["t0", "t1", "t2", "t3", "t4", "p0", "p1"]}


def small_direct(ep, wl, steps, flusher, rep, clocks, launches0):
    """Small workloads, direct launches: every step after an L2 flush, timed by its own event pair."""
    s_ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    e_ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps)]
    rep.barrier()
    if clocks:
        clocks.__enter__()
    for i in range(steps):
        flusher()
        s_ev[i].record()
        wl.step()
        e_ev[i].record()
    torch.cuda.synchronize()
    if clocks:
        clocks.__exit__()
    rep.barrier()
    launches = ep.ep_launch_count() - launches0
    evs = [wl.new_events() for _ in range(min(steps, 50))]
    for e in evs:
        flusher()
        wl.step(e)
    torch.cuda.synchronize()
    return [s.elapsed_time(e) for s, e in zip(s_ev, e_ev)], evs, launches, "direct launches"


def small_in_graph(ep, wl, steps, flusher, rep, clocks, per_graph=10):
    """Small workloads, the deployment form of a decode step: a CUDA graph holds `per_graph` repetitions
    of [L2 flush, event, step, event]; the events are recorded inside the graph, so the times are device
    times of the step's kernels with neither host launch cost nor the flush in them. Per-kernel figures
    come from a second graph with events between the calls. Also measures the floor of this protocol:
    the same bracket around one and around three kernels that do nothing."""
    def ext():
        return torch.cuda.Event(enable_timing=True, external=True)

    side = torch.cuda.Stream()
    with torch.cuda.stream(side):                        # per-device set-up of the calls outside any capture
        flusher()
        wl.step()
    torch.cuda.synchronize()
    n0 = ep.ep_launch_count()
    wl.step()
    torch.cuda.synchronize()
    per_step_launches = ep.ep_launch_count() - n0

    def build(body, n):
        pairs = [(ext(), ext()) for _ in range(n)]
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for s, e in pairs:
                flusher()
                s.record()
                body()
                e.record()
        return g, pairs

    g_step, pairs = build(wl.step, per_graph)
    warm_pairs = [(ext(), ext()) for _ in range(per_graph)]     # the same steps with nothing evicted in between
    g_warm = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g_warm):
        for s, e in warm_pairs:
            s.record()
            wl.step()
            e.record()
    ops_evs = [wl.new_events(external=True) for _ in range(per_graph)]
    g_ops = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g_ops):
        for e in ops_evs:
            flusher()
            wl.step(e)
    tiny = torch.zeros(64, dtype=torch.int32, device=wl.dev)
    g_one, p_one = build(lambda: ep.ep_post_flags(tiny, 0, 1, 1), per_graph)
    g_three, p_three = build(lambda: [ep.ep_post_flags(tiny, 0, 1, 1) for _ in range(3)], per_graph)
    for g in (g_step, g_ops, g_one, g_three):            # warm replays
        g.replay()
    torch.cuda.synchronize()
    step_ms = []
    rep.barrier()
    if clocks:
        clocks.__enter__()
    while len(step_ms) < steps:
        g_step.replay()
        torch.cuda.synchronize()
        step_ms += [s.elapsed_time(e) for s, e in pairs]
    if clocks:
        clocks.__exit__()
    rep.barrier()
    step_ms = step_ms[:steps]

    evs = []                                              # event times, read out after each replay
    for _ in range(max(1, min(steps, 50) // per_graph)):
        g_ops.replay()
        torch.cuda.synchronize()
        for e in ops_evs:
            spans = [("t0", "t1"), ("t1", "t2"), ("t0", "t2"), ("t2", "t3"), ("t3", "t4"), ("t0", "t4")]
            if wl.split_layout:
                spans.append(("p0", "p1"))
            evs.append(FrozenEvents({(a, b): e[a].elapsed_time(e[b]) for a, b in spans}))
    floor = {}
    for name, (g, ps) in [("one_empty_kernel_us", (g_one, p_one)), ("three_empty_kernels_us", (g_three, p_three))]:
        ts = []
        for _ in range(3):
            g.replay()
            torch.cuda.synchronize()
            ts += [s.elapsed_time(e) * 1e3 for s, e in ps]
        floor[name] = float(np.median(ts))
    warm = []
    for _ in range(4):
        g_warm.replay()
        torch.cuda.synchronize()
        warm += [s.elapsed_time(e) for s, e in warm_pairs]
    floor["step_without_flush"] = dict(stats_us(warm[per_graph:]),
                                       what="the same step replayed with L2 left warm (code and batch resident, as in a "
                                            "decode loop); not the protocol figure")
    floor["what"] = ("the same in-graph bracket [flush, event, kernels, event] around kernels that do nothing: after the "
                     "flush every kernel starts with cold instruction and parameter fetches; the event timer ticks in ~2 us steps")
    return step_ms, evs, steps * per_step_launches, f"CUDA graph of {per_graph} x [flush, event, step, event]", floor


class FrozenEvents:
    """Event-pair durations read out earlier, behind the interface `measure` uses for live events."""

    def __init__(self, spans):
        self.spans = spans

    def __getitem__(self, name):
        return _FrozenEvent(self, name)


class _FrozenEvent:
    def __init__(self, owner, name):
        self.owner, self.name = owner, name

    def elapsed_time(self, other):
        return self.owner.spans[(self.name, other.name)]


def measure(ep, wl, steps, warmup, rep, no_graph=False, sample_clocks=True):
    """Times `steps` steps of a workload. Big workloads: back to back from a CUDA graph (or direct launches), then
    once more as direct launches with per-kernel events. Small workloads: every step after an L2 flush, timed by its own event pair
    recorded inside a CUDA graph (small_in_graph), or with direct launches (small_direct)."""
    cfg, lay = wl.cfg, wl.lay
    small = is_small(cfg)
    dev_index = torch.cuda.current_device()
    clocks = ClockSampler(dev_index) if sample_clocks else None      # NVML set-up before the warm-up, not after it
    wl.step()
    torch.cuda.synchronize()
    assert ep.ep_status(lay.status) == 0
    n_recv, n_pairs = int(lay.rank_row_offsets[-1]), int(lay.expert_offsets[-1])
    alg = algorithmic_bytes(cfg, n_recv, n_pairs)
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for _ in range(warmup):                               # the W warm-up steps run right before the timed region
        wl.step()
    torch.cuda.synchronize()
    launches0 = ep.ep_launch_count()
    if not small:
        # pass A, the timed region: K steps back to back, one event before and one after. The steps are replayed
        # from a CUDA graph that holds G of them (G = the largest divisor of K up to 25): the same kernels with the
        # same dependencies, without the host's launch gaps (C4: 282-285 us per step against 288-289 with direct
        # launches, which --no-graph times instead; host-staged workloads always use direct launches).
        graph, per_graph, n_replays = None, 0, 0
        if not no_graph and not cfg.host_staged:
            in_graph = max(g for g in range(1, 26) if steps % g == 0)
            n_replays = steps // in_graph
            graph = torch.cuda.CUDAGraph()
            l0 = ep.ep_launch_count()
            with torch.cuda.graph(graph):
                for _ in range(in_graph):
                    wl.step()
            per_graph = ep.ep_launch_count() - l0
            graph.replay()                                # uploads the graph: untimed, part of the warm-up
            torch.cuda.synchronize()
            launches0 = ep.ep_launch_count()
        rep.barrier()
        if clocks:
            clocks.__enter__()
        start.record()
        if graph is not None:
            for i in range(n_replays):
                graph.replay()
        else:
            for i in range(steps):
                wl.step()
        stop.record()
        torch.cuda.synchronize()
        rep.barrier()
        launches = per_graph * n_replays if graph is not None else ep.ep_launch_count() - launches0
        total_ms = rep.max_over_ranks(start.elapsed_time(stop))
        direct_us = None
        if graph is not None:                             # the same K steps as direct launches, for comparison only
            a_d, b_d = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a_d.record()
            for i in range(steps):
                wl.step()
            b_d.record()
            torch.cuda.synchronize()
            direct_us = a_d.elapsed_time(b_d) / steps * 1e3
        # pass B, the same K steps again with events between the calls: per-kernel durations (the seven event
        # records per step cost a few microseconds of stream time, which is why they are kept out of pass A).
        # Replayed from a graph like pass A (events recorded inside it), or direct launches.
        start_b, stop_b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        if graph is not None:
            ops_evs = [wl.new_events(external=True) for _ in range(steps // n_replays)]
            g_ops = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g_ops):
                for e in ops_evs:
                    wl.step(e)
            g_ops.replay()
            torch.cuda.synchronize()
            spans = [("t0", "t1"), ("t1", "t2"), ("t0", "t2"), ("t2", "t3"), ("t3", "t4"), ("t0", "t4")]
            if wl.split_layout:
                spans.append(("p0", "p1"))
            evs, pass_b_ms = [], 0.0
            for _ in range(n_replays):
                start_b.record()
                g_ops.replay()
                stop_b.record()
                torch.cuda.synchronize()
                pass_b_ms += start_b.elapsed_time(stop_b)
                evs += [FrozenEvents({(a, b): e[a].elapsed_time(e[b]) for a, b in spans}) for e in ops_evs]
        else:
            evs = [wl.new_events() for _ in range(steps)]
            start_b.record()
            for i in range(steps):
                wl.step(evs[i])
            stop_b.record()
            torch.cuda.synchronize()
            pass_b_ms = start_b.elapsed_time(stop_b)
        if clocks:
            clocks.__exit__()
        rep.barrier()
        step_ms = [e["t0"].elapsed_time(e["t4"]) for e in evs]
        how = (f"a CUDA graph of {steps // n_replays} step(s) replayed {n_replays} time(s) back to back "
               f"(the same {steps} steps as direct launches: {direct_us:.1f} us per step)") if graph is not None else \
            "direct launches"
        launch_note = (f"{how}; value from {steps} steps with no events inside; per-kernel durations from the "
                       f"same {steps} steps repeated in the same way with events between the calls "
                       f"({pass_b_ms / steps * 1e3:.1f} us per step)")
    else:
        flusher = L2Flush(wl.dev)
        floor = None
        if no_graph:
            step_ms, evs, launches, launch_note = small_direct(ep, wl, steps, flusher, rep, clocks, launches0)
        else:
            step_ms, evs, launches, launch_note, floor = small_in_graph(ep, wl, steps, flusher, rep, clocks)
        total_ms = rep.max_over_ranks(sum(step_ms))
        del flusher

    def span(a, b):
        return [e[a].elapsed_time(e[b]) for e in evs]

    ops = {"layout": dict(stats_us(span("t0", "t1")),
                          what="layout and dispatch in one call (ep_layout_dispatch)" if wl.fused else
                          "whole layout" if not wl.split_layout else "receive-row half (critical path)"),
           "dispatch": dict(stats_us(span("t0", "t2") if wl.fused else span("t1", "t2")), bytes=alg["dispatch"]),
           "combine": dict(stats_us(span("t3", "t4")), bytes=alg["combine"])}
    if wl.split_layout:
        ops["layout_pair_half"] = dict(stats_us(span("p0", "p1")), what="ep_layout_pairs on the side stream, beside dispatch")
        ops["join_wait"] = dict(stats_us(span("t2", "t3")), what="main stream waiting for the pair half after dispatch")
    for name in ("dispatch", "combine"):
        o = ops[name]
        o["GB/s"] = o["bytes"] / (o["us"] * 1e-6) / 1e9
        o["best_GB/s"] = o["bytes"] / (o["best_us"] * 1e-6) / 1e9
        o["tokens/s"] = cfg.T / (o["us"] * 1e-6)
    if small:
        ops["note"] = ("per-kernel figures: events between the calls of a step" +
                       (", direct launches after a flush (launch latency included)" if no_graph else
                        " inside a graph, each step after a flush"))
    return {"total_ms": total_ms, "step": stats_us(step_ms), "ops": ops, "launches": int(launches), "floor": floor if small else None,
            "n_recv": n_recv, "n_pairs": n_pairs, "alg": alg, "launch": launch_note,
            "layout": "ep_layout_dispatch (layout kernel and a dependent dispatch launch, one call)" if wl.fused else
            "one ep_layout call" if not wl.split_layout else
            ("ep_layout_dispatch with a second stream (receive-row half, dispatch launched behind it, pair half on the "
             "side stream); the per-kernel pass issues the same work as separate calls" if wl.one_call_split else
             "ep_layout_ranks before dispatch, ep_layout_pairs on a side stream beside dispatch"),
            "clocks": clocks.summary() if clocks else None}


def ops_alone(ep, wl, alg, per_graph=8, replays=4):
    """Each call of the step by itself: [L2 flush, event, call, event] recorded inside a CUDA graph, so that a
    kernel is charged neither launch latency nor the write-back of the previous kernel's dirty L2 lines (inside
    the step, combine pays for up to ~60 MB of dispatch's output still sitting in L2)."""
    cfg, lay = wl.cfg, wl.lay
    E, R = cfg.E, cfg.R
    flusher = L2Flush(wl.dev)
    calls = {"layout": lambda: ep.ep_layout(wl.idx, E, R, out=lay, workspace=wl.ws),
             "dispatch": lambda: ep.ep_dispatch(wl.x, lay.recv_slot, wl.recv, E, R, status=lay.status),
             "combine": lambda: ep.ep_combine(wl.out, lay.pair_slot, wl.w, wl.y, E, R, status=lay.status)}
    if wl.split_layout:
        calls["layout_receive_row_half"] = lambda: ep.ep_layout_ranks(wl.idx, E, R, lay, wl.ws)
    if wl.fused:
        calls["layout_dispatch_one_call"] = lambda: ep.ep_layout_dispatch(wl.idx, wl.x, wl.recv, E, R, lay, wl.ws)
    res = {}
    side = torch.cuda.Stream()
    for name, fn in calls.items():
        with torch.cuda.stream(side):
            fn()
        torch.cuda.synchronize()
        pairs = [(torch.cuda.Event(enable_timing=True, external=True), torch.cuda.Event(enable_timing=True, external=True))
                 for _ in range(per_graph)]
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for s_, e_ in pairs:
                flusher()
                s_.record()
                fn()
                e_.record()
        ts = []
        for i in range(replays + 1):
            g.replay()
            torch.cuda.synchronize()
            if i:
                ts += [s_.elapsed_time(e_) for s_, e_ in pairs]
        o = stats_us(ts)
        if name in ("dispatch", "combine"):
            o["GB/s"] = alg[name] / (o["us"] * 1e-6) / 1e9
        res[name] = o
        del g
    del flusher
    return res


def time_variants(ep, wl, n_recv, n_pairs, iters=20):
    """Median device time of the variants around the path on the same batch: local grouping,
    expanded dispatch, combine with per-rank partial outputs, dense all-gather / reduce-scatter."""
    cfg, dev, lay = wl.cfg, wl.dev, wl.lay
    T, K, H, E, R = cfg.T, cfg.K, cfg.H, cfg.E, cfg.R
    row = 2 * H
    flush = L2Flush(dev)
    recv = torch.empty(max(1, n_recv), H, dtype=torch.bfloat16, device=dev)
    ep.ep_dispatch(wl.x, lay.recv_slot, recv, E, R)
    y = torch.empty(T, H, dtype=torch.bfloat16, device=dev)
    res = {"rows": {"routed_receive": n_recv, "pairs": n_pairs, "dense": R * T}}

    def timed(fn, nbytes):
        ts = []
        for _ in range(iters + 2):
            flush()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            fn()
            b.record()
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b))
        ms = float(np.median(ts[2:]))
        return {"us": ms * 1e3, "GB/s": nbytes / (ms * 1e-3) / 1e9, "bytes": nbytes}

    grouped = torch.empty(max(1, n_pairs), H, dtype=torch.bfloat16, device=dev)
    res["group (recv -> pair rows)"] = timed(lambda: ep.ep_group(recv, lay, grouped, E, R), 2 * row * n_pairs + 4 * n_pairs)
    res["expanded dispatch (x -> pair rows)"] = timed(lambda: ep.ep_dispatch(wl.x, lay.pair_slot, grouped, E, R),
                                                      row * T + row * n_pairs + 4 * T * K)
    del grouped
    partial = torch.empty(max(1, n_recv), H, dtype=torch.bfloat16, device=dev)
    res["combine with partial outputs (2 kernels)"] = timed(
        lambda: ep.ep_combine_partial(wl.out, lay, wl.w, partial, y, E, R),
        row * n_pairs + 2 * row * n_recv + row * T + 16 * T * K)
    del partial
    gathered = torch.empty(R * T, H, dtype=torch.bfloat16, device=dev)
    res["dense all-gather"] = timed(lambda: ep.ep_dense_allgather(wl.x, gathered, K, E, R), row * T + row * R * T)
    if R <= 32:
        res["dense reduce-scatter (2 kernels)"] = timed(
            lambda: ep.ep_dense_reduce_scatter(wl.idx, wl.out, lay.pair_slot, wl.w, gathered, y, E, R),
            row * n_pairs + 2 * row * R * T + row * T + 12 * T * K)
    del gathered, flush
    return res


def duplex_link_probe(dev, nbytes=256 << 20, reps=5):
    """One host-to-device and one device-to-host cudaMemcpyAsync of `nbytes` each (pinned), on two streams at the
    same time: GB/s per direction, best of `reps`. What the host link gives when both directions are busy."""
    h_up, h_dn = torch.empty(nbytes, dtype=torch.uint8).pin_memory(), torch.empty(nbytes, dtype=torch.uint8).pin_memory()
    d_up, d_dn = torch.empty(nbytes, dtype=torch.uint8, device=dev), torch.zeros(nbytes, dtype=torch.uint8, device=dev)
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    best = 1e30
    for _ in range(reps + 1):
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e1, e2 = torch.cuda.Event(), torch.cuda.Event()
        a.record()
        s1.wait_event(a), s2.wait_event(a)
        with torch.cuda.stream(s1):
            d_up.copy_(h_up, non_blocking=True)
        with torch.cuda.stream(s2):
            h_dn.copy_(d_dn, non_blocking=True)
        e1.record(s1), e2.record(s2)
        torch.cuda.current_stream().wait_event(e1), torch.cuda.current_stream().wait_event(e2)
        b.record()
        torch.cuda.synchronize()
        best = min(best, a.elapsed_time(b))
    return nbytes / (best * 1e-3) / 1e9


def host_staged_arms(ep, wl, iters=10, sweep=True):
    """Receive buffer in mapped pinned host memory: (i) the dispatch kernel stores straight
    into it; (ii) dispatch packs into device staging and the copy engine moves each rank's
    partition; plus the host-link probe both are measured against, and the round trips."""
    cfg, dev, lay, x, recv_host = wl.cfg, wl.dev, wl.lay, wl.x, wl.recv
    E, R = cfg.E, cfg.R
    n_recv = int(lay.rank_row_offsets[-1])
    row = 2 * cfg.H
    staging = torch.empty(recv_host.shape[0], cfg.H, dtype=torch.bfloat16, device=dev)
    probe_src = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    probe_dst = torch.empty(256 << 20, dtype=torch.uint8).pin_memory()
    d2h = ep.ep_probe_bandwidth(ep.PROBE_MEMCPY, probe_dst, probe_src, 256 << 20, iters=10)
    h2d = ep.ep_probe_bandwidth(ep.PROBE_MEMCPY, probe_src, probe_dst, 256 << 20, iters=10)
    del probe_src, probe_dst

    def timed(fn):
        best = 1e30
        for _ in range(iters + 1):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            fn()
            b.record()
            torch.cuda.synchronize()
            best = min(best, a.elapsed_time(b))
        return best

    def arm_kernel():
        ep.ep_dispatch(x, lay.recv_slot, recv_host, E, R)

    offs_pinned = torch.zeros(R + 1, dtype=torch.int32).pin_memory()

    def arm_copy_known():           # the offsets first travel to the host: one small copy and a stream sync, timed
        offs_pinned.copy_(lay.rank_row_offsets, non_blocking=True)
        torch.cuda.current_stream().synchronize()
        ep.ep_dispatch_copy_engine(x, lay.recv_slot, staging, recv_host, E, R, rank_row_offsets_host=offs_pinned)

    def arm_copy_blind():           # no count reaches the host: one copy of the worst-case T*min(K,R) rows
        ep.ep_dispatch_copy_engine(x, lay.recv_slot, staging, recv_host, E, R, rank_row_offsets_host=None)

    res = {"host_link_d2h_GB/s": d2h, "host_link_h2d_GB/s": h2d,
           "host_link_duplex_GB/s_each_way": duplex_link_probe(dev), "rows": n_recv, "bytes_over_link": n_recv * row}
    for name, fn, nbytes in [("kernel_store", arm_kernel, n_recv * row),
                             ("copy_engine_per_rank", arm_copy_known, n_recv * row),
                             ("copy_engine_worst_case", arm_copy_blind, recv_host.shape[0] * row)]:
        ms = timed(fn)
        res[name] = {"us": ms * 1e3, "GB/s": nbytes / (ms * 1e-3) / 1e9, "useful_GB/s": n_recv * row / (ms * 1e-3) / 1e9,
                     "frac_of_d2h_probe": n_recv * row / (ms * 1e-3) / 1e9 / d2h, "tokens/s": cfg.T / (ms * 1e-3)}
    # dispatch round trip through the bounce buffer on two streams: all uploads then all downloads, or chunk-wise duplex
    cap = recv_host.shape[0]
    bounce = torch.empty(2 * cap, cfg.H, dtype=torch.bfloat16).pin_memory()
    back = torch.empty(cap, cfg.H, dtype=torch.bfloat16, device=dev)
    up, down = torch.cuda.Stream(), torch.cuda.Stream()
    offs_host = lay.rank_row_offsets.cpu()
    torch.cuda.synchronize()
    trips = {}
    for duplex, chunks in ([(0, 1), (1, 1), (1, 2), (1, 4), (1, 8)] if sweep else [(0, 1), (1, 1)]):
        best = 1e30
        for rnd in range(iters + 1):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(down)
            ep.ep_host_roundtrip(x, lay.recv_slot, offs_host, staging, bounce, back, E, R, round=rnd,
                                 chunks_per_rank=chunks, duplex=bool(duplex), stream_up=up, stream_down=down)
            b.record(down)
            torch.cuda.synchronize()
            best = min(best, a.elapsed_time(b))
        trips[("duplex" if duplex else "serial") + f", {chunks} chunk(s) per rank"] = {
            "us": best * 1e3, "GB/s_each_way": n_recv * row / (best * 1e-3) / 1e9, "tokens/s": cfg.T / (best * 1e-3)}
    res["roundtrip"] = trips
    # cost of one completion check: the wait kernel on flags that are already posted
    n_s = max(1, R - 1)
    flags_dev = torch.full((64,), 3, dtype=torch.int32, device=dev)
    flags_pin = torch.full((64,), 3, dtype=torch.int32).pin_memory()
    waits = {}
    for name, fl in [("flags in device memory", flags_dev), ("flags in pinned host memory", flags_pin)]:
        waits[name] = {"us": timed(lambda: ep.ep_wait_senders(fl, n_s, 3, 100_000_000)) * 1e3, "senders": n_s}
    res["flag_wait_posted"] = waits

    # combine return leg: per-rank partial rows up, down to the owner, summed on the SMs
    so_host = lay.src_row_offsets.cpu()
    son = so_host.numpy()
    local_rows = int(sum(son[r, r + 1] - son[r, r] for r in range(R)))
    y = torch.empty(cfg.T, cfg.H, dtype=torch.bfloat16, device=dev)
    D, P, L = ep.HOST_DUPLEX, ep.HOST_PER_PEER, ep.HOST_LOCAL_ON_DEVICE
    legs = {}
    for name, fl in [("serial, one reduction behind the last download", 0), ("duplex, one reduction", D),
                     ("duplex, reduction per owner", D | P),
                     ("duplex, reduction per owner, local blocks stay on the device", D | P | L)]:
        best = 1e30
        for rnd in range(iters + 1):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(up)
            ep.ep_host_combine(wl.out, lay, wl.w, so_host, staging, back, bounce, y, E, R, round=rnd, flags=fl,
                               stream_up=up, stream_down=down)
            b.record(down)
            torch.cuda.synchronize()
            best = min(best, a.elapsed_time(b))
        rows = n_recv - (local_rows if fl & L else 0)
        legs[name] = {"us": best * 1e3, "rows_over_link": rows, "GB/s_each_way": rows * row / (best * 1e-3) / 1e9,
                      "frac_of_d2h_probe": rows * row / (best * 1e-3) / 1e9 / d2h,
                      "frac_of_h2d_probe": rows * row / (best * 1e-3) / 1e9 / h2d, "tokens/s": cfg.T / (best * 1e-3)}
    res["combine_return_leg"] = legs

    # dispatch with one consumer per sender: when is the first sender's data in use, when the last
    grouped = torch.empty(cfg.T * cfg.K, cfg.H, dtype=torch.bfloat16, device=dev)
    stamps = torch.zeros(R + 1, dtype=torch.int64, device=dev)
    cons = torch.cuda.Stream()
    t0 = time.perf_counter()
    so_timed = lay.src_row_offsets.cpu()                 # the segment table's trip to the host, timed once
    fetch_us = (time.perf_counter() - t0) * 1e6
    per_sender = {"src_row_offsets_to_host_us": fetch_us}
    for name, fl in [("consumer per sender", D | P), ("consumers behind the last download", D)]:
        firsts, lasts = [], []
        for rnd in range(iters + 1):
            ep.ep_host_dispatch_per_sender(x, lay, so_timed, staging, back, bounce, grouped, E, R, round=rnd, flags=fl,
                                           stamps_ns=stamps, stream_up=up, stream_down=down, stream_consume=cons)
            torch.cuda.synchronize()
            st = stamps.cpu().numpy()
            firsts.append((st[1] - st[0]) * 1e-3)
            lasts.append((st[-1] - st[0]) * 1e-3)
        per_sender[name] = {"first_sender_consumed_us": float(np.median(firsts[1:])),
                            "all_senders_consumed_us": float(np.median(lasts[1:]))}
    res["dispatch_per_sender"] = per_sender
    del grouped

    # consecutive rounds (dispatch round trip, then combine return leg): with the caller's per-half events
    # round n+1's uploads overlap round n's downloads; without, every call waits for the download stream
    bounce2 = torch.empty(2 * cap, cfg.H, dtype=torch.bfloat16).pin_memory()
    back2 = torch.empty(cap, cfg.H, dtype=torch.bfloat16, device=dev)
    send2 = torch.empty(cap, cfg.H, dtype=torch.bfloat16, device=dev)
    n_rounds = 6
    rounds = {}
    for name, overlap in [("rounds ordered by the download stream", False), ("rounds overlapped (per-half events)", True)]:
        best = 1e30
        for _ in range(3):
            hf1, hf2 = (ep.HalfFreeEvents(), ep.HalfFreeEvents()) if overlap else (None, None)
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(up)
            for rnd in range(n_rounds):
                ep.ep_host_roundtrip(x, lay.recv_slot, offs_host, staging, bounce, back, E, R, round=rnd, chunks_per_rank=1,
                                     duplex=True, stream_up=up, stream_down=down, half_free=hf1)
                ep.ep_host_combine(wl.out, lay, wl.w, so_host, send2, back2, bounce2, y, E, R, round=rnd, flags=D | P,
                                   stream_up=up, stream_down=down, half_free=hf2)
            b.record(down)
            torch.cuda.synchronize()
            best = min(best, a.elapsed_time(b))
        rounds[name] = {"us_per_round": best * 1e3 / n_rounds, "rounds": n_rounds,
                        "GB/s_each_way": 2 * n_recv * row * n_rounds / (best * 1e-3) / 1e9}
    res["dispatch_plus_combine_rounds"] = rounds
    # independent dispatch round trips back to back: what the two alternating bounce halves are for
    n_trips = 8
    trips_b2b = {}
    for name, overlap in [("ordered by the download stream", False), ("overlapped (per-half events)", True)]:
        best = 1e30
        for _ in range(3):
            hf = ep.HalfFreeEvents() if overlap else None
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(up)
            for rnd in range(n_trips):
                ep.ep_host_roundtrip(x, lay.recv_slot, offs_host, staging, bounce, back, E, R, round=rnd, chunks_per_rank=1,
                                     duplex=True, stream_up=up, stream_down=down, half_free=hf)
            b.record(down)
            torch.cuda.synchronize()
            best = min(best, a.elapsed_time(b))
        trips_b2b[name] = {"us_per_trip": best * 1e3 / n_trips, "trips": n_trips,
                           "GB/s_each_way": n_recv * row * n_trips / (best * 1e-3) / 1e9}
    res["dispatch_roundtrips_back_to_back"] = trips_b2b
    return res


def roofline_object(cfg, name, achieved, peak, peak_kind, probes=None):
    r = {"bound": "hbm", "kernel": name, "achieved": achieved, "peak": peak, "peak_kind": peak_kind + " copy peak",
         "unit": "GB/s", "frac": achieved / peak, "frac_of_nominal_8000": achieved / NOMINAL_HBM_GBS,
         "traffic": NCU_TRAFFIC_BYTES.get((cfg.name, name))}
    if probes:
        r["frac_of_own_copy_probe"] = achieved / probes["copy_GB/s"]
    return r


def summarize_config(cfg, m, peak, host=None):
    """The entry of one extra configuration under `configs`."""
    ops = m["ops"]
    e = {"workload": workload_text(cfg), "step": m["step"], "tokens/s": cfg.T / (m["step"]["us"] * 1e-6),
         "launch": m["launch"], "layout_call": m["layout"], "n_recv": m["n_recv"], "n_pairs": m["n_pairs"], "ops": ops}
    if m.get("floor"):
        e["floor"] = m["floor"]
    for name in ("dispatch", "combine"):
        ops[name]["frac_of_measured_peak"] = ops[name]["GB/s"] / peak
        ops[name]["frac_of_nominal_8000"] = ops[name]["GB/s"] / NOMINAL_HBM_GBS
    if step_bytes_estimate(cfg) < L2_BYTES:
        e["note"] = "launch-latency-bound: the whole step moves less than L2 holds; HBM fractions are not meaningful"
    if host is not None:
        link = host["host_link_d2h_GB/s"]
        e["host_link"] = {"bound": "host-link", "peak": link, "peak_kind": "cudaMemcpyAsync D2H probe, 256 MB pinned, same run",
                          "unit": "GB/s", "kernel_store": {"achieved": host["kernel_store"]["useful_GB/s"],
                                                           "frac": host["kernel_store"]["frac_of_d2h_probe"]},
                          "copy_engine_per_rank": {"achieved": host["copy_engine_per_rank"]["useful_GB/s"],
                                                   "frac": host["copy_engine_per_rank"]["frac_of_d2h_probe"]}}
        e["host_staged"] = host
    return e


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--workload", default="C4")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=20)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="time direct launches, not graph replays")
    ap.add_argument("--serial-layout", action="store_true",
                    help="one ep_layout call instead of the receive-row half before dispatch and the pair half beside it")
    ap.add_argument("--separate-calls", action="store_true",
                    help="ep_layout (or its halves) and ep_dispatch as separate calls instead of ep_layout_dispatch")
    ap.add_argument("--force-split", action="store_true", help="split layout (pair half on a side stream) also for small batches")
    ap.add_argument("--one-call", action="store_true",
                    help="big batches: ep_layout_dispatch (whole layout, dispatch launched behind it with programmatic "
                         "stream serialisation) instead of the split layout")
    ap.add_argument("--variants", action="store_true",
                    help="also time the variants around the path (grouping, partial-output combine, dense baseline)")
    ap.add_argument("--no-configs", action="store_true", help="skip the extra configurations under `configs`")
    ap.add_argument("--config-steps", type=int, default=50, help="timed steps of each extra configuration")
    ap.add_argument("--seed", type=int, default=0)
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3

    from paper_2609_40093_b200 import inputs
    cfg = inputs.CONFIGS[args.workload]
    if args.impl == "reference":
        run_reference(args, cfg)
        return

    import __graft_entry__ as entry
    from paper_2609_40093_b200 import ep
    from paper_2609_40093_b200.replicas import Replicas
    rep = Replicas()
    rank, world = rep.rank, rep.world
    if rank == 0:
        entry.build()
    rep.barrier()
    dev = torch.device("cuda", torch.cuda.current_device())
    rcfg = inputs.shard_config(cfg, rank)            # replica `rank`: same shapes, its own seed stream
    T, K, H, E, R = cfg.T, cfg.K, cfg.H, cfg.E, cfg.R

    wl = Workload(ep, inputs, cfg, rcfg, dev, args.seed, serial_layout=args.serial_layout,
                  separate_calls=args.separate_calls, one_call=args.one_call, force_split=args.force_split)
    m = measure(ep, wl, args.steps, args.warmup, rep, no_graph=args.no_graph)
    n_recv, n_pairs, alg = m["n_recv"], m["n_pairs"], m["alg"]
    value = world * T * args.steps / (m["total_ms"] * 1e-3)

    alone = ops_alone(ep, wl, alg) if not cfg.host_staged else None
    host = host_staged_arms(ep, wl) if cfg.host_staged else None
    variants = time_variants(ep, wl, n_recv, n_pairs) if args.variants else None

    # ---- end to end: one C-ABI call per step, host buffers in, host buffer out
    arena = torch.empty(ep.ep_host_step_arena_bytes(T, K, H, E, R), dtype=torch.uint8, device=dev)
    y_h = torch.empty(T, H, dtype=torch.bfloat16).pin_memory()
    st_h = torch.zeros(1, dtype=torch.int32).pin_memory()
    n_e2e = max(1, args.e2e_steps)
    e2e_chunks = 2 if T >= 2048 else 1       # C4, steps back to back: 2.61 ms with 2 chunks, 2.64 with 4, 2.78 with 8
    s_in, s_comp, s_out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()

    step_events, e2e_round = ep.StepEvents(), [0]

    def e2e_step():
        # consecutive steps alternate between two copies of the arena's transfer buffers: a step's uploads run
        # while the previous step's results are still on their way back
        ep.ep_host_step_pipelined(wl.x_h, wl.idx_h, wl.w_h, y_h, arena, E, R, e2e_chunks, s_in, s_comp, s_out,
                                  status_host=st_h, round=e2e_round[0], step_events=step_events)
        e2e_round[0] += 1

    torch.cuda.synchronize()
    for _ in range(3 if args.e2e_steps > 0 else 0):
        e2e_step()
    torch.cuda.synchronize()
    rep.barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(s_in)                      # the first thing a step does is an upload on s_in ...
    for _ in range(args.e2e_steps):
        e2e_step()
    e1.record(s_out)                     # ... and the last a download on s_out
    torch.cuda.synchronize()
    e2e_ms = rep.max_over_ranks(e0.elapsed_time(e1))
    assert int(st_h[0]) == 0
    e2e_value = world * T * args.e2e_steps / (e2e_ms * 1e-3) if args.e2e_steps > 0 else None
    h2d = wl.x_h.numel() * 2 + wl.idx_h.numel() * 4 + wl.w_h.numel() * 4
    d2h = y_h.numel() * 2 + 4
    del arena
    duplex = duplex_link_probe(dev) if args.e2e_steps > 0 else None    # both directions busy: the ceiling of the e2e step

    # the library's own stream probes on this GPU, beside the measured copy peak
    probes = None
    if not cfg.host_staged:
        pa = torch.empty(1 << 30, dtype=torch.uint8, device=dev)
        pb = torch.empty(1 << 30, dtype=torch.uint8, device=dev)
        pa.zero_(), pb.zero_()
        probes = {name + "_GB/s": ep.ep_probe_bandwidth(kind, pb, pa, 1 << 30, iters=8)
                  for name, kind in [("read", ep.PROBE_READ), ("write", ep.PROBE_WRITE), ("copy", ep.PROBE_COPY)]}
        probes["what"] = "ep_probe_bandwidth, 1 GiB, best of 8; copy counts read + write bytes"
        del pa, pb

    peak, peak_kind = measured_peak()

    # ---- the other configurations, same protocol, fewer steps (one GPU only: they are not part of `value`)
    configs = None
    if world == 1 and not args.no_configs:
        configs = {}
        for name in ["C1", "C2", "C3", "C5"]:
            if name == cfg.name:
                continue
            c = inputs.CONFIGS[name]
            w2 = Workload(ep, inputs, c, c, dev, args.seed)
            m2 = measure(ep, w2, args.config_steps, max(5, args.warmup), rep, sample_clocks=False)
            h2 = host_staged_arms(ep, w2, iters=6, sweep=False) if c.host_staged else None
            configs[name] = summarize_config(c, m2, peak, h2)
            if not c.host_staged:
                al = ops_alone(ep, w2, m2["alg"])
                for op in ("dispatch", "combine"):
                    al[op]["frac_of_measured_peak"] = al[op]["GB/s"] / peak
                configs[name]["ops_alone"] = al
            del w2
            torch.cuda.empty_cache()

    if rank != 0:
        rep.close()
        return
    ops = m["ops"]
    com_gbs, dis_gbs = ops["combine"]["GB/s"], ops["dispatch"]["GB/s"]
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": m["total_ms"] / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": config_object(cfg, world, n_recv, n_pairs),
        "protocol": {"launch": m["launch"], "layout": m["layout"], "step": m["step"], "floor": m["floor"]},
        "ops": ops,
        "ops_alone": alone,
        "roofline": roofline_object(cfg, "combine_rows_kernel", com_gbs, peak, peak_kind, probes),
        "roofline_dispatch": roofline_object(cfg, "dispatch_rows_kernel", dis_gbs, peak, peak_kind, probes),
        "probes": probes,
        "clocks": m["clocks"],
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": e2e_ms / n_e2e, "steps": args.e2e_steps,
                "call": f"ep_host_step_pipelined (layout+dispatch+group+combine, pinned host in/out, {e2e_chunks} token "
                        "chunk(s) on upload/compute/download streams; consecutive steps alternate between two copies "
                        "of the arena's transfer buffers, so a step's uploads overlap the previous step's downloads)",
                "link_GB/s_each_way": (h2d / (e2e_ms / n_e2e * 1e-3) / 1e9) if args.e2e_steps > 0 else None,
                "link_duplex_probe_GB/s_each_way": duplex if args.e2e_steps > 0 else None,
                "frac_of_duplex_probe": (h2d / (e2e_ms / n_e2e * 1e-3) / 1e9 / duplex) if args.e2e_steps > 0 else None},
        "gpu_launches": m["launches"],
        "context": CONTEXT,
    }
    if variants is not None:
        line["variants"] = variants
    if host is not None:
        line["host_staged"] = host
        link = host["host_link_d2h_GB/s"]
        line["roofline_dispatch"] = {"bound": "host-link", "kernel": "dispatch_rows_kernel (stores to mapped pinned memory)",
                                     "achieved": host["kernel_store"]["GB/s"], "peak": link,
                                     "peak_kind": "cudaMemcpyAsync D2H probe, 256 MB pinned, same run", "unit": "GB/s",
                                     "frac": host["kernel_store"]["GB/s"] / link, "traffic": None}
    if configs is not None:
        line["configs"] = configs
    if not args.no_cpu_baseline:
        line["cpu_baseline"] = time_oracle(cfg, wl.host["topk_idx"], wl.host["topk_weights"], wl.host["x"], wl.out_h,
                                           min_seconds=8.0, max_steps=20)
    print(json.dumps(line))
    rep.close()


if __name__ == "__main__":
    main()
