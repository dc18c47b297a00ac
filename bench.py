#!/usr/bin/env python
"""Benchmark of the per-window 8-bit GDN decode step on B200.

One "step" is one lq_decode_step call over the whole batch: every (sequence, value head) decodes one
token from its 8-bit window representation, and the 1/W of the sequences whose window becomes full are
taken through the window boundary (reconstruct, refit compensators, smooth, requantize) in the same call.

Workload (config.workload = "gdn_b256"): 256 sequences x 32 value heads (16 q/k heads), d_k = d_v = 128,
bf16 inputs, W = 16, r = 4; states pre-filled by 512 warm-up tokens of the same random recurrence and
window offsets staggered uniformly over [0, W), so that every step costs the same.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

Prints ONE JSON line (rank 0).  value = state-GB/s = (head-steps per second) x 19456 bytes of quantized
state per head; tokens_heads_per_s and the roofline object say the rest.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2609_38166_b200 import synth  # noqa: E402

WARM_TOKENS = 512
STATE_BYTES = 128 * 128 + 4 * 128 + 4 * 128 + 2 * 4 * (128 + 128)       # 19456 per head at r = 4
METRIC = "GDN decode state-GB/s at bs256 (8-bit per-window state, W=16, r=4)"


def state_bytes(r: int) -> int:
    """Bytes of the quantized state of one head: codes, two fp32 scale vectors, r fp16 compensator pairs."""
    return 128 * 128 + 4 * 128 + 4 * 128 + 2 * r * (128 + 128)


def metric_name(wl) -> str:
    """The headline metric's name; other shapes (flags --gate/--batch/--W/--r) are named after themselves."""
    if wl.gate == synth.GATE_SCALAR and wl.batch == 256 and wl.W == 16 and wl.r == 4 and not wl.rec16:
        return METRIC
    return "%s decode state-GB/s at bs%d (8-bit per-window state, W=%d, r=%d%s)" % (
        "GDN" if wl.gate == synth.GATE_SCALAR else "KDA", wl.batch, wl.W, wl.r, ", fp16 records" if wl.rec16 else "")

# DRAM bytes per launch from the ncu captures summarised under profiles/ (dram__bytes_read.sum +
# dram__bytes_write.sum of one full-batch launch of the gdn_b256 workload, W = 16), or None when not captured.
NCU_CAPTURE_N_ITER = 1                                # (the captures were taken with the default number of rounds)
NCU_TRAFFIC_BYTES_PER_LAUNCH = {"decode_kernel": 232.9e6, "boundary_kernel": 18.5e6}
# The same two counters from a launch list taken with --cache-control none (the caches are left as the kernel ahead
# left them, as in a real step): what the L2 serves - the records written by the last tokens, the token vectors, and
# for the boundary kernel the heads the decode kernel asked the L2 to keep - no longer comes from DRAM.
NCU_TRAFFIC_WARM_BYTES_PER_LAUNCH = {"decode_kernel": 195.1e6, "boundary_kernel": 2.2e6}


def record_bytes(diag: bool, rec16: int) -> int:
    """One buffered record (kt, u, decay): fp32 rows, or fp16 rows whose scalar-gate decay stays fp32."""
    if rec16:
        return 2 * 384 if diag else 2 * 256 + 4
    return 4 * (256 + (128 if diag else 1))


def algorithmic_bytes_per_head_step(W: int, r: int, diag: bool, group: int, launches_fused: bool, rec16: int = 0) -> float:
    """Bytes that must move per (head, token): quantized state + average record buffer + inputs + appended
    record + output + the window boundary amortised over W tokens."""
    g = 128 if diag else 1
    state = 128 * 128 + 512 + 512 + 512 * r
    rec = record_bytes(diag, rec16)
    buf_read = (W - 1) / 2.0 * rec
    inputs = 512 / group + 256 + 2 + 2 * g
    flush = state + (0 if launches_fused else state + W * rec)      # write back (+ re-read when a second kernel does it)
    return state + buf_read + inputs + rec + 512 + flush / W


L2_BYTES = 126e6


def l2_note(wl) -> str:
    """Whether the window representation of the whole batch (what a step streams) exceeds the L2."""
    heads = wl.batch * wl.heads_v
    rec = record_bytes(wl.gate == synth.GATE_DIAG, wl.rec16)
    mb = heads * (state_bytes(wl.r) + wl.W * rec) / 1e6
    if mb * 1e6 > 2 * L2_BYTES:
        return "working set %.0f MB per step exceeds the 126 MB L2; no flush needed" % mb
    return ("working set %.0f MB per step is below twice the 126 MB L2: this point is (partly) L2-resident and says "
            "nothing about HBM" % mb)


def config_dict(wl, world: int) -> dict:
    """The workload, the same for both arms (what differs between runs - warm-up length, steps - is not here)."""
    return {"workload": wl.name, "batch": wl.batch, "heads_v": wl.heads_v, "heads_qk": wl.heads_qk,
            "d_k": wl.d_k, "d_v": wl.d_v, "W": wl.W, "r": wl.r, "n_iter": wl.n_iter,
            "gate": "scalar (GDN)" if wl.gate == synth.GATE_SCALAR else "diagonal (KDA)",
            "state_dtype": "int8 + fp32 scales + fp16 compensators", "record_buffer_dtype": "f16" if wl.rec16 else "f32",
            "inputs_dtype": "bf16", "window_offsets": "uniform over [0,W)", "l2": l2_note(wl),
            "parallelism": "dp%d (independent batches, no collective)" % world}


def captured_traffic(wl, table):
    """The ncu DRAM bytes per launch of `table`, if this run's workload is the one they were captured on."""
    same = (wl.name == "gdn_b256" and wl.batch == 256 and wl.W == 16 and wl.r == 4 and wl.n_iter == NCU_CAPTURE_N_ITER and
            wl.gate == synth.GATE_SCALAR and not wl.rec16 and not wl.state_bf16 and wl.smooth == 1 and wl.delta == 1)
    return dict(table) if same else {k: None for k in table}


def shard_workload(wl, rank: int):
    """Every rank owns its own batch of the same shape (weak scaling): only the seed differs."""
    return wl.with_(seed=wl.seed + 1000 * rank)


def max_over_ranks(value_ms: float, dist_mod=None, device=None) -> float:
    """Slowest rank's time; `dist_mod` is torch.distributed when a process group is up, else None."""
    if dist_mod is None or not dist_mod.is_initialized() or dist_mod.get_world_size() == 1:
        return value_ms
    import torch
    t = torch.tensor([value_ms], dtype=torch.float64, device=device if device is not None else "cpu")
    dist_mod.all_reduce(t, op=dist_mod.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(heads_per_rank: int, world: int, steps: int, ms: float, r: int = 4) -> float:
    """state-GB/s of the whole job: all ranks' head-steps over the slowest rank's time."""
    return world * heads_per_rank * steps / (ms / 1e3) * state_bytes(r) / 1e9


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        return float(json.load(open(path))["hbm_gbs"]), "measured (MEASURED_PEAKS.json)"
    return 6650.0, "fallback"


# --------------------------------------------------------------------------------------------------
# clocks: NVML samples taken by a thread while the timed region runs (read-only queries)
# --------------------------------------------------------------------------------------------------
class ClockSampler:
    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, index: int):
        self.samples, self.reasons, self.power = [], set(), []
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h) if hasattr(
                    nv, "nvmlDeviceGetCurrentClocksEventReasons") else nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
                self.power.append(nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0)
            except Exception:
                pass
            time.sleep(0.005)

    def start(self):
        if self.nv:
            self._stop.clear()
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        if self._thread:
            self._stop.set()
            self._thread.join()
            self._thread = None

    def summary(self, source: str):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0, "source": source}
        return {"sm_mhz": statistics.median(self.samples), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples),
                "power_w_max": max(self.power) if self.power else None, "source": source}


# --------------------------------------------------------------------------------------------------
# reference arm: the CPU oracle, as it stands, on a bounded sample of the same workload
# --------------------------------------------------------------------------------------------------
def oracle_sample_state(oracle, wl, seed_tokens: int = 48):
    """Window representation of `wl.batch` sequences warmed by a short run of the oracle's own fp32
    recurrence, window offsets spread over [0, W)."""
    from oracle.lq_oracle import Shape, State
    sh = Shape(wl.batch, wl.heads_v, wl.heads_qk, wl.d_k, wl.d_v, wl.W, wl.r, wl.n_iter, wl.gate, wl.smooth)
    S = np.zeros((wl.batch, wl.heads_v, wl.d_k, wl.d_v), np.float32)
    for t in range(seed_tokens):
        oracle.ref_step_f32(sh, S, **synth.token_inputs(wl, t))
    st = State(sh)
    oracle.quantize_state(sh, S, st)
    st.win_pos[:] = (np.arange(wl.batch) * wl.W // max(wl.batch, 1)) % wl.W
    st.buf_a[...] = 1.0
    return sh, st


def time_oracle(wl, steps: int, warmup: int, limit_s: float):
    """Times oracle.decode_step on a sub-batch sized to fit `limit_s`; returns (head-steps/s, cores, sample)."""
    from oracle.lq_oracle import Oracle
    oracle = Oracle()
    probe = wl.with_(batch=2)
    sh, st = oracle_sample_state(oracle, probe, seed_tokens=8)
    toks = [synth.token_inputs(probe, 1000 + t) for t in range(4)]
    t0 = time.perf_counter()
    for t in range(4):
        oracle.decode_step(sh, st, **toks[t])
    rate = 4 * probe.batch * probe.heads_v / (time.perf_counter() - t0)          # head-steps per second, rough
    nb = int(max(1, min(wl.batch, limit_s * rate / ((steps + warmup) * wl.heads_v))))
    sub = wl.with_(batch=nb)
    sh, st = oracle_sample_state(oracle, sub)
    toks = [synth.token_inputs(sub, 2000 + t) for t in range(wl.W)]
    for t in range(warmup):
        oracle.decode_step(sh, st, **toks[t % wl.W])
    t0 = time.perf_counter()
    for t in range(steps):
        oracle.decode_step(sh, st, **toks[t % wl.W])
    dt = time.perf_counter() - t0
    sample = (f"oracle.decode_step on {nb} of {wl.batch} sequences x {wl.heads_v} heads, {steps} steps "
              f"(window offsets staggered, boundaries included), {dt:.1f} s")
    return nb * wl.heads_v * steps / dt, oracle.threads(), sample, dt / steps


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    hs, cores, sample, s_per_step = time_oracle(wl, args.steps, args.warmup, limit_s=150.0)
    value = hs * state_bytes(wl.r) / 1e9
    line = {"impl": "reference", "metric": metric_name(wl), "value": value, "unit": "GB/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": s_per_step * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "tokens_heads_per_s": hs,
            "config": config_dict(wl, args.gpus),
            "cpu_baseline": {"value": value, "unit": "GB/s", "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------------------------------
# CUDA arm
# --------------------------------------------------------------------------------------------------
SCRATCH_WORDS = True      # --no-scratch-words: states without lq_state.work (every decode CTA takes an equal share of heads)


def to_dev(tok, torch):
    return {k: torch.from_numpy(v.view(np.int16)).cuda(non_blocking=False) for k, v in tok.items()}


def prepare_state(wl, lq, torch, log, WARM_TOKENS=WARM_TOKENS):
    """512 warm-up tokens on the fp32-state kernel, quantized group by group so that at the end group g
    (a contiguous slice of the batch) holds g buffered records: window offsets uniform over [0, W)."""
    sh = lq.Shape(wl.batch, wl.heads_v, wl.heads_qk, wl.d_k, wl.d_v, wl.W, wl.r, wl.n_iter, wl.gate, wl.smooth, wl.delta,
                  wl.rec16, wl.state_bf16)
    B, W = wl.batch, wl.W
    st = lq.State(sh, work=SCRATCH_WORDS)
    S = torch.zeros((B, wl.heads_v, wl.d_k, wl.d_v), dtype=torch.float32, device="cuda")
    o = torch.empty((B, wl.heads_v, wl.d_v), dtype=torch.float32, device="cuda")
    per = max(B // W, 1)
    groups = (B + per - 1) // per                       # number of distinct offsets actually used (<= W)
    t0 = time.time()
    for t in range(WARM_TOKENS + 1):
        g = WARM_TOKENS - t                             # the group that is quantized after t tokens
        b_lq = min(B, g * per) if g < groups else B     # sequences [b_lq, B) already run quantized
        if g < groups:
            lo, hi = g * per, (B if g == groups - 1 else (g + 1) * per)
            lq.quantize_state(sh, S, st, b0=lo, nb=hi - lo)
            b_lq = lo
        if t == WARM_TOKENS:
            break
        d = to_dev(synth.token_inputs(wl, t), torch)
        if b_lq > 0:
            lq.ref_decode_step_f32(sh, S, d["q"], d["k"], d["v"], d["beta"], d["alpha"], o, b0=0, nb=b_lq)
        if b_lq < B:
            lq.decode_step(sh, st, d["q"], d["k"], d["v"], d["beta"], d["alpha"], o, b0=b_lq, nb=B - b_lq)
    torch.cuda.synchronize()
    log(f"warm-up of {WARM_TOKENS} tokens took {time.time() - t0:.1f} s; window offsets "
        f"{sorted(set(st.win_pos.tolist()))}")
    del S
    return sh, st, o


def run_cuda(args, wl):
    import torch
    import torch.distributed as dist
    from paper_2609_38166_b200 import build, lq

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    log = (lambda m: print(f"[bench] {m}", file=sys.stderr, flush=True)) if rank == 0 else (lambda m: None)
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        build.build()
    if world > 1:
        dist.barrier()
    lq.lib()                                             # raises if the CUDA library is missing

    wl = shard_workload(wl, rank)                        # every rank owns its own batch (weak scaling, no exchange)
    sh, st, o = prepare_state(wl, lq, torch, log, args.warm_tokens)
    WARM_TOKENS = args.warm_tokens
    toks = [to_dev(synth.token_inputs(wl, WARM_TOKENS + t), torch) for t in range(wl.W)]
    stream = torch.cuda.current_stream()

    def step(t):
        d = toks[t % wl.W]
        lq.decode_step(sh, st, d["q"], d["k"], d["v"], d["beta"], d["alpha"], o, stream)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for t in range(max(args.warmup, 3)):
        step(t)

    # The timed steps are launched the way a serving loop launches a decode step: W consecutive steps captured once
    # in a CUDA graph and replayed (every sequence passes exactly one window boundary per replay); steps beyond a
    # multiple of W are plain launches.  --no-graph times plain launches only.
    graph = None
    if not args.no_graph and args.steps >= wl.W:
        try:
            gs = torch.cuda.Stream()
            with torch.cuda.stream(gs):
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph, stream=gs):
                    for t in range(wl.W):
                        d = toks[t]
                        lq.decode_step(sh, st, d["q"], d["k"], d["v"], d["beta"], d["alpha"], o, gs)
            torch.cuda.synchronize()
            graph.replay()                               # uploads the graph to the device (untimed)
            torch.cuda.synchronize()
        except Exception as exc:                         # reported, never hidden
            log(f"CUDA-graph capture failed, timing plain launches: {exc!r}")
            graph = None

    def run_steps(k, use_graph=True):
        reps = k // wl.W if (graph is not None and use_graph) else 0
        for _ in range(reps):
            graph.replay()
        for t in range(reps * wl.W, k):
            step(t)

    sampler = ClockSampler(local)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    sampler.start()
    ev0.record(stream)
    run_steps(args.steps)
    ev1.record(stream)
    barrier()
    sampler.stop()
    ms = ev0.elapsed_time(ev1)
    clock_source = "timed region"
    if len(sampler.samples) < 5:                         # region too short to sample: repeat the same loop, untimed
        sampler.start()
        t_end = time.time() + 0.6
        t = 0
        while time.time() < t_end:
            step(t); t += 1
            if t % 256 == 0:
                torch.cuda.synchronize()
        torch.cuda.synchronize()
        sampler.stop()
        clock_source = "identical loop run right after the timed region (timed region shorter than the sampling period)"
    ms = max_over_ranks(ms, dist if world > 1 else None, "cuda")

    # the same K steps as plain launches (two kernel launches per step from the host), for comparison
    plain_ms = None
    if graph is not None and not args.only_timed:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record(stream)
        run_steps(args.steps, use_graph=False)
        e1.record(stream)
        barrier()
        plain_ms = max_over_ranks(e0.elapsed_time(e1), dist if world > 1 else None, "cuda") / args.steps
    graph_ms = ms / args.steps if graph is not None else None

    # end to end through the host-buffer entry point: inputs in pinned host memory, output read back
    e2e = None
    try:
        if args.only_timed:
            raise RuntimeError("skipped (--only-timed)")
        pin = [{k: torch.from_numpy(v.view(np.int16)).pin_memory() for k, v in
                synth.token_inputs(wl, WARM_TOKENS + t).items()} for t in range(wl.W)]
        o_h = torch.empty((wl.batch, wl.heads_v, wl.d_v), dtype=torch.float32).pin_memory()
        stage = torch.empty((lq.decode_stage_bytes(sh),), dtype=torch.uint8, device="cuda")
        # at least 256 calls, after a warm-up of two windows: consecutive calls chain onto each other (the inputs of
        # a call are fetched next to the previous call's boundary kernels), and a handful of calls is not that regime
        n_e2e = max(min(args.steps, 2000), 256)

        def step_host(t):
            d = pin[t % wl.W]
            lq.decode_step_host_pipelined(sh, st, d["q"], d["k"], d["v"], d["beta"], d["alpha"], o_h, stage, stream)

        for t in range(2 * wl.W + max(args.warmup, 3)):
            step_host(t)
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for t in range(n_e2e):
            step_host(t)
        e1.record(stream)
        barrier()
        e2e_ms = max_over_ranks(e0.elapsed_time(e1), dist if world > 1 else None, "cuda")
        h2d = sum(v.numel() * v.element_size() for v in pin[0].values())
        e2e = {"value": whole_job_value(wl.batch * wl.heads_v, world, n_e2e, e2e_ms, wl.r), "unit": "GB/s",
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": o_h.numel() * 4, "steps": n_e2e,
               "ms_per_step": e2e_ms / n_e2e,
               "api": "lq_decode_step_host_pipelined, one call per step: pinned host q,k,v,beta,alpha in (read over the "
                      "bus by a gather launch per half batch, which may start while the step before is still at its "
                      "window boundaries), o out to pinned host memory (copied while the window-boundary kernel runs)"}
    except Exception as exc:
        log(f"end-to-end timing failed: {exc!r}")

    # The two kernels of a step timed separately: a second loop, with an event between the kernels
    kern = None
    try:
        n_k = min(args.steps, 256)
        evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(n_k)]
        for trio in evs:
            for e in trio:
                e.record(stream)               # materialises the CUDA handles
        torch.cuda.synchronize()
        for t in range(n_k):
            d = toks[t % wl.W]
            evs[t][0].record(stream)
            lq.decode_step_profiled(sh, st, d["q"], d["k"], d["v"], d["beta"], d["alpha"], o, evs[t][1], stream)
            evs[t][2].record(stream)
        torch.cuda.synchronize()
        kern = {"decode_ms": statistics.mean(e[0].elapsed_time(e[1]) for e in evs),
                "boundary_ms": statistics.mean(e[1].elapsed_time(e[2]) for e in evs), "steps": n_k}
    except Exception as exc:
        log(f"per-kernel timing failed: {exc!r}")

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    heads = wl.batch * wl.heads_v
    ms_per_step = ms / args.steps
    hs = world * heads * args.steps / (ms / 1e3)
    launches = lq.decode_launches(sh)
    peak, peak_src = peaks()
    group = wl.heads_v // wl.heads_qk
    bytes_hs = algorithmic_bytes_per_head_step(wl.W, wl.r, wl.gate == synth.GATE_DIAG, group, launches == 1, wl.rec16)
    achieved = heads * bytes_hs / (ms_per_step / 1e3) / 1e9
    rec = record_bytes(wl.gate == synth.GATE_DIAG, wl.rec16)
    # what each kernel has to move per launch: the decode kernel everything but the boundary; the boundary
    # kernel, for the 1/W of the heads whose window is full, the window representation in and the head block out
    decode_bytes = heads * (bytes_hs - (2 * state_bytes(wl.r) + wl.W * rec) / wl.W)
    boundary_bytes = heads / wl.W * (2 * state_bytes(wl.r) + wl.W * rec)
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": None, "peak_source": peak_src,
                "kernel": "one step = decode_kernel + boundary_kernel (algorithmic bytes of both over the step time "
                          "of the timed region; the decode kernel carries 93 % of the bytes)",
                "algorithmic_bytes_per_head_step": bytes_hs, "algorithmic_bytes_per_step": heads * bytes_hs,
                "frac_of_nominal_8TBps": achieved / 8000.0}
    cold, warm = captured_traffic(wl, NCU_TRAFFIC_BYTES_PER_LAUNCH), captured_traffic(wl, NCU_TRAFFIC_WARM_BYTES_PER_LAUNCH)
    if kern:
        dk, bk = kern["decode_ms"], kern["boundary_ms"]
        roofline["kernels"] = {
            "decode_kernel": {"ms": dk, "algorithmic_bytes": decode_bytes, "achieved": decode_bytes / dk / 1e6,
                              "frac": decode_bytes / dk / 1e6 / peak, "bound": "hbm",
                              "traffic": cold["decode_kernel"]},
            "boundary_kernel": {"ms": bk, "algorithmic_bytes": boundary_bytes, "achieved": boundary_bytes / bk / 1e6,
                                "frac": boundary_bytes / bk / 1e6 / peak,
                                "bound": "fp32 issue and dependency latency, not hbm",
                                "traffic": cold["boundary_kernel"]},
            "how": "CUDA events on the launching stream around each kernel, mean of %d steps in a second loop" %
                   kern["steps"]}
    # ncu's DRAM bytes of one step: only for the workload the capture was taken on (profiles/), else null
    t_d, t_b = cold["decode_kernel"], cold["boundary_kernel"]
    roofline["traffic"] = (t_d + t_b) if (t_d and t_b) else None
    roofline["traffic_warm_caches"] = sum(warm.values()) if all(warm.values()) else None

    # speed baselines in the same run: dense fp32 / bf16 state, read and written every token
    base = {}
    try:
        if args.only_timed:
            raise RuntimeError("skipped (--only-timed)")
        S = torch.zeros((wl.batch, wl.heads_v, 128, 128), dtype=torch.float32, device="cuda")
        S16 = torch.zeros((wl.batch, wl.heads_v, 128, 128), dtype=torch.int16, device="cuda")
        for name, fn, buf in (("fp32_state", lq.ref_decode_step_f32, S), ("bf16_state", lq.ref_decode_step_bf16, S16)):
            nrep = 200
            for t in range(5):
                d = toks[t % wl.W]
                fn(sh, buf, d["q"], d["k"], d["v"], d["beta"], d["alpha"], o)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record(stream)
            for t in range(nrep):
                d = toks[t % wl.W]
                fn(sh, buf, d["q"], d["k"], d["v"], d["beta"], d["alpha"], o)
            e1.record(stream)
            torch.cuda.synchronize()
            bms = e0.elapsed_time(e1) / nrep
            nbytes = heads * (2 * 128 * 128 * (4 if name == "fp32_state" else 2) + 1028)
            base[name] = {"ms_per_step": bms, "speedup_of_8bit_path": bms / ms_per_step,
                          "GBps": nbytes / (bms / 1e3) / 1e9}
        del S, S16
    except Exception as exc:
        log(f"baseline kernels failed: {exc!r}")

    cpu = None
    if not args.only_timed:
        hs_cpu, cores, sample, _ = time_oracle(wl.with_(seed=wl.seed), steps=8 * wl.W, warmup=2, limit_s=25.0)
        cpu = {"value": hs_cpu * state_bytes(wl.r) / 1e9, "unit": "GB/s", "cores": cores, "kind": "oracle",
               "sample": sample, "tokens_heads_per_s": hs_cpu}

    line = {"metric": metric_name(wl), "value": hs * state_bytes(wl.r) / 1e9, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": config_dict(wl, world), "warmup_tokens": args.warm_tokens,
            "tokens_heads_per_s": hs, "pct_hbm_peak_measured": 100 * achieved / peak,
            "pct_hbm_peak_nominal_8TBps": 100 * achieved / 8000.0,
            "launch_mode": ("CUDA graph of W = %d steps replayed %d times + %d plain steps" %
                            (wl.W, args.steps // wl.W, args.steps % wl.W)) if graph is not None else "plain launches",
            "cuda_graph_ms_per_step": graph_ms, "plain_launch_ms_per_step": plain_ms,
            "gpu_launches": launches * args.steps,
            "clocks": sampler.summary(clock_source), "roofline": roofline, "baselines": base,
            "e2e": e2e, "cpu_baseline": cpu}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


# --------------------------------------------------------------------------------------------------
# Throughput sweep: GDN and KDA, batch x W x r, uniform window offsets; one JSON line per point
# --------------------------------------------------------------------------------------------------
def run_sweep(args):
    import torch
    from paper_2609_38166_b200 import build, lq

    log = lambda m: print(f"[sweep] {m}", file=sys.stderr, flush=True)
    torch.cuda.set_device(0)
    build.build()
    lq.lib()
    peak, peak_src = peaks()
    l2 = torch.cuda.get_device_properties(0).L2_cache_size
    stream = torch.cuda.current_stream()
    batches = [int(x) for x in args.sweep_batches.split(",")]
    windows = [int(x) for x in args.sweep_W.split(",")]
    ranks = [int(x) for x in args.sweep_r.split(",")]
    gates = [g for g in args.sweep_gates.split(",")]
    rec16s = [int(x) for x in args.sweep_rec16.split(",")]
    warm = max(windows) + 8
    rows = []
    for gate_name in gates:
        diag = gate_name == "kda"
        for B in batches:
            base_wl = synth.Workload(f"sweep_{gate_name}", B, 32, 32 if diag else 16, 128, 128, 16, 4,
                                     gate=synth.GATE_DIAG if diag else synth.GATE_SCALAR, seed=5)
            cache = {}

            def tok(t, base_wl=base_wl, cache=cache):
                if t not in cache:
                    cache[t] = to_dev(synth.token_inputs(base_wl, t), torch)
                return cache[t]

            def timed(fn, nrep, cycle):
                for t in range(cycle + 3):                     # also draws every token of the cycle (CPU work)
                    fn(t)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                torch.cuda.synchronize()
                e0.record(stream)
                for t in range(nrep):
                    fn(t)
                e1.record(stream)
                torch.cuda.synchronize()
                return e0.elapsed_time(e1) / nrep

            # the two dense-state baselines of this (gate, batch)
            sh0 = lq.Shape(B, 32, base_wl.heads_qk, 128, 128, 16, 4, 2, base_wl.gate, 1)
            o = torch.empty((B, 32, 128), dtype=torch.float32, device="cuda")
            S = torch.zeros((B, 32, 128, 128), dtype=torch.float32, device="cuda")
            ms32 = timed(lambda t: lq.ref_decode_step_f32(sh0, S, *[tok(t % 16)[k] for k in
                                                                    ("q", "k", "v", "beta", "alpha")], o), 100, 16)
            del S
            S16 = torch.zeros((B, 32, 128, 128), dtype=torch.int16, device="cuda")
            ms16 = timed(lambda t: lq.ref_decode_step_bf16(sh0, S16, *[tok(t % 16)[k] for k in
                                                                       ("q", "k", "v", "beta", "alpha")], o), 100, 16)
            del S16
            for W in windows:
                for r in ranks:
                  for rec16 in rec16s:
                    wl = base_wl.with_(W=W, r=r, rec16=rec16)
                    # same staggering as the headline run, with a short pre-fill (speed does not depend on it)
                    sh = lq.Shape(B, 32, wl.heads_qk, 128, 128, W, r, wl.n_iter, wl.gate, 1, 1, rec16)
                    st = lq.State(sh)
                    S = torch.zeros((B, 32, 128, 128), dtype=torch.float32, device="cuda")
                    per = max(B // W, 1)
                    groups = (B + per - 1) // per
                    for t in range(warm + 1):
                        g = warm - t
                        b_lq = B
                        if g < groups:
                            lo, hi = g * per, (B if g == groups - 1 else (g + 1) * per)
                            lq.quantize_state(sh, S, st, b0=lo, nb=hi - lo)
                            b_lq = lo
                        if t == warm:
                            break
                        d = tok(t)
                        if b_lq > 0:
                            lq.ref_decode_step_f32(sh, S, d["q"], d["k"], d["v"], d["beta"], d["alpha"], o, b0=0,
                                                   nb=b_lq)
                        if b_lq < B:
                            lq.decode_step(sh, st, d["q"], d["k"], d["v"], d["beta"], d["alpha"], o, b0=b_lq,
                                           nb=B - b_lq)
                    del S
                    nrep = max(args.sweep_steps // W, 1) * W      # every sequence flushes the same number of times
                    ms = timed(lambda t: lq.decode_step(sh, st, *[tok(warm + t % W)[k] for k in
                                                                  ("q", "k", "v", "beta", "alpha")], o, stream), nrep, W)
                    flags = lq.check_device()
                    heads = B * 32
                    bytes_hs = algorithmic_bytes_per_head_step(W, r, diag, wl.heads_v // wl.heads_qk, False, rec16)
                    foot = st.heads.numel() + st.records.numel() * st.records.element_size()
                    state_b = 128 * 128 + 4 * 128 + 4 * 128 + 2 * r * 256
                    row = {"sweep": True, "gate": gate_name, "batch": B, "W": W, "r": r, "n_iter": wl.n_iter,
                           "records": "f16" if rec16 else "f32",
                           "steps": nrep, "ms_per_step": ms, "tokens_heads_per_s": heads / (ms / 1e3),
                           "state_GBps": heads * state_b / (ms / 1e3) / 1e9,
                           "total_GBps": heads * bytes_hs / (ms / 1e3) / 1e9,
                           "pct_hbm_peak_measured": 100 * heads * bytes_hs / (ms / 1e3) / 1e9 / peak,
                           "speedup_vs_fp32_state": ms32 / ms, "speedup_vs_bf16_state": ms16 / ms,
                           "fp32_state_ms": ms32, "bf16_state_ms": ms16,
                           "l2": "L2-resident (window representation %.0f MB < 2 x %.0f MB L2)" % (foot / 1e6, l2 / 1e6)
                                 if foot < 2 * l2 else "exceeds L2", "device_error_flags": flags}
                    rows.append(row)
                    print(json.dumps(row), flush=True)
                    del st
            cache.clear()
            torch.cuda.empty_cache()
    log("gate  batch   W   r  rec   us/step   state GB/s  total GB/s  %peak   x fp32   x bf16")
    for x in rows:
        log(f"{x['gate']:4s} {x['batch']:6d} {x['W']:3d} {x['r']:3d}  {x['records']} {1e3 * x['ms_per_step']:9.1f} "
            f"{x['state_GBps']:11.0f} {x['total_GBps']:11.0f} {x['pct_hbm_peak_measured']:6.1f} "
            f"{x['speedup_vs_fp32_state']:8.2f} {x['speedup_vs_bf16_state']:8.2f}"
            f"{'  (L2-resident)' if x['l2'].startswith('L2-res') else ''}")


# --------------------------------------------------------------------------------------------------
# Ablation ladder (the structure of the paper's component ablation, on synthetic decode inputs): speed of
# every rung on the benchmark batch, and its error against the fp32 recurrence fed the same tokens.
# Everything runs on the GPU through the library; no oracle involved.
# --------------------------------------------------------------------------------------------------
def run_ladder(args):
    import torch
    from paper_2609_38166_b200 import build, lq

    log = lambda m: print(f"[ladder] {m}", file=sys.stderr, flush=True)
    torch.cuda.set_device(0)
    build.build()
    lq.lib()
    stream = torch.cuda.current_stream()
    rungs = [("fp32 state, every token", None),
             ("bf16 state, every token", "bf16"),
             ("bf16 per window (W=16): the -w baseline", dict(W=16, r=0, smooth=0, state_bf16=1)),
             ("int8 every token (W=1, no compensators, no smoothing)", dict(W=1, r=0, smooth=0)),
             ("int8 per window (W=16), no compensators, no smoothing", dict(W=16, r=0, smooth=0)),
             ("+ 4 Compensator Tokens", dict(W=16, r=4, smooth=0)),
             ("+ residual smoothing (the full method)", dict(W=16, r=4, smooth=1))]
    rows = []
    for base_name in ("gdn_b256", "kda_b128_outlier"):
        base = synth.config(base_name)
        small = base.with_(batch=16)                     # error: 16 sequences x 32 heads, 64 + 256 tokens
        n_warm, n_err = 64, 256
        toks_small = [to_dev(synth.token_inputs(small, t), torch) for t in range(n_warm + n_err)]
        toks_big = [to_dev(synth.token_inputs(base, 1000 + t), torch) for t in range(16)]
        keys = ("q", "k", "v", "beta", "alpha")
        for label, var in rungs:
            # ---- error against the fp32 recurrence ----
            wl = small if not isinstance(var, dict) else small.with_(**var)
            sh = lq.Shape(wl.batch, 32, wl.heads_qk, 128, 128, wl.W, wl.r, wl.n_iter, wl.gate, wl.smooth,
                          state_bf16=wl.state_bf16)
            S = torch.zeros((wl.batch, 32, 128, 128), dtype=torch.float32, device="cuda")
            o_ref = torch.empty((wl.batch, 32, 128), dtype=torch.float32, device="cuda")
            o_var = torch.empty_like(o_ref)
            for t in range(n_warm):
                lq.ref_decode_step_f32(sh, S, *[toks_small[t][k] for k in keys], o_ref)
            st = S16 = None
            if var == "bf16":
                S16 = S.to(torch.bfloat16).view(torch.int16).contiguous()
            elif isinstance(var, dict):
                st = lq.State(sh)
                lq.quantize_state(sh, S, st)
            errs = []
            for t in range(n_warm, n_warm + n_err):
                d = [toks_small[t][k] for k in keys]
                lq.ref_decode_step_f32(sh, S, *d, o_ref)
                if var is None:
                    o_var.copy_(o_ref)
                elif var == "bf16":
                    lq.ref_decode_step_bf16(sh, S16, *d, o_var)
                else:
                    lq.decode_step(sh, st, *d, o_var)
                num = (o_var - o_ref).flatten(1).norm(dim=1)
                den = o_ref.flatten(1).norm(dim=1)
                errs.append((num / den).mean())
            err = float(torch.stack(errs).mean())
            del S, S16, st
            # ---- speed on the full batch, windows staggered as in the headline run ----
            wlb = base if not isinstance(var, dict) else base.with_(**var)
            shb = lq.Shape(wlb.batch, 32, wlb.heads_qk, 128, 128, wlb.W, wlb.r, wlb.n_iter, wlb.gate, wlb.smooth,
                           state_bf16=wlb.state_bf16)
            ob = torch.empty((wlb.batch, 32, 128), dtype=torch.float32, device="cuda")
            if isinstance(var, dict):
                _, stb, ob = prepare_state(wlb, lq, torch, lambda m: None, 32)
                fn = lambda t: lq.decode_step(shb, stb, *[toks_big[t % 16][k] for k in keys], ob, stream)
                state_b = 2 * 128 * 128 if wlb.state_bf16 else 128 * 128 + 1024 + 2 * wlb.r * 256
            elif var == "bf16":
                Sb = torch.zeros((wlb.batch, 32, 128, 128), dtype=torch.int16, device="cuda")
                fn = lambda t: lq.ref_decode_step_bf16(shb, Sb, *[toks_big[t % 16][k] for k in keys], ob, stream)
                state_b = 2 * 128 * 128
            else:
                Sb = torch.zeros((wlb.batch, 32, 128, 128), dtype=torch.float32, device="cuda")
                fn = lambda t: lq.ref_decode_step_f32(shb, Sb, *[toks_big[t % 16][k] for k in keys], ob, stream)
                state_b = 4 * 128 * 128
            for t in range(48):
                fn(t)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record(stream)
            nrep = 512
            for t in range(nrep):
                fn(t)
            e1.record(stream)
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / nrep
            row = {"ladder": True, "workload": base_name, "rung": label, "ms_per_step": ms,
                   "state_bytes_per_head": state_b, "rel_err_o_vs_fp32": err,
                   "error_run": "16 sequences x 32 heads, 64 fp32 warm-up tokens, mean over 256 tokens and heads of |o - o_fp32| / |o_fp32|"}
            rows.append(row)
            print(json.dumps(row), flush=True)
            stb = Sb = None
            torch.cuda.empty_cache()
    t32 = {r["workload"]: r["ms_per_step"] for r in rows if r["rung"].startswith("fp32")}
    log("workload           rung                                                      us/step  x fp32   B/head   rel.err(o)")
    for r in rows:
        log(f"{r['workload']:18s} {r['rung']:56s} {1e3 * r['ms_per_step']:8.1f} {t32[r['workload']] / r['ms_per_step']:7.2f} "
            f"{r['state_bytes_per_head']:8d}   {r['rel_err_o_vs_fp32']:.3e}")


# --------------------------------------------------------------------------------------------------
# --timeline: where a step's time goes.  Runs the headline workload on the library variant with per-CTA time
# stamps (python -m paper_2609_38166_b200.build --stamps; thread 0 of every CTA reads the GPU's global timer when it
# becomes resident, when its wait for the kernel ahead ends, when its first head's data is there and when it leaves)
# and prints, for three consecutive steps, the spread of those moments over the CTAs of both kernels.  Not a
# measurement of throughput: the stamps cost a little, and nothing here is timed from the host.
# --------------------------------------------------------------------------------------------------
def run_timeline(args):
    import ctypes
    import torch
    from paper_2609_38166_b200 import build, lq

    torch.cuda.set_device(0)
    log = lambda m: print(f"[timeline] {m}", file=sys.stderr, flush=True)
    lq._LIB_PATH = build.build(stamps=True)
    L = lq.lib()
    wl = synth.config("gdn_b256").with_(W=args.W, batch=args.batch, r=args.r, rec16=args.rec16)
    if args.gate == "kda":
        wl = wl.with_(gate=synth.GATE_DIAG, heads_qk=wl.heads_v)
    sh, st, o = prepare_state(wl, lq, torch, log, min(args.warm_tokens, 64))
    toks = [to_dev(synth.token_inputs(wl, 64 + t), torch) for t in range(wl.W)]
    for t in range(4 * wl.W + 4):                       # (the stamps of the last four steps are kept)
        d = toks[t % wl.W]
        lq.decode_step(sh, st, d["q"], d["k"], d["v"], d["beta"], d["alpha"], o)
    torch.cuda.synchronize()
    buf = np.zeros((4, 2, 6, 1024), dtype=np.uint64)
    if L.lq_debug_timeline(buf.ctypes.data_as(ctypes.c_void_p)) != 0:
        raise RuntimeError("lq_debug_timeline failed")
    tl = buf.astype(np.int64)
    gd, gb = int((tl[0, 0, 1] != 0).sum()), int((tl[0, 1, 1] != 0).sum())
    pct = lambda a, t0: [round(float(np.percentile((a - t0) / 1e3, q)), 2) for q in (0, 10, 50, 90, 100)]
    steps = []
    order = sorted(range(4), key=lambda g_: tl[g_, 0, 1, :gd].min())       # the four generations, oldest first
    for g, g_next in zip(order[:3], order[1:]):
        t0 = tl[g, 0, 1, :gd].min()
        steps.append({
            "decode_resident": pct(tl[g, 0, 0, :gd], t0), "decode_first_head_there": pct(tl[g, 0, 2, :gd], t0),
            "decode_leaves": pct(tl[g, 0, 3, :gd], t0),
            "boundary_resident": pct(tl[g, 1, 0, :gb], t0), "boundary_wait_over": pct(tl[g, 1, 1, :gb], t0),
            "boundary_first_head_staged": pct(tl[g, 1, 2, :gb], t0), "boundary_first_head_done": pct(tl[g, 1, 3, :gb], t0),
            "boundary_leaves": pct(tl[g, 1, 4, :gb], t0),
            "next_decode_wait_over": round(float(tl[g_next, 0, 1, :gd].min() - t0) / 1e3, 2)})
    print(json.dumps({"timeline": True, "workload": wl.name, "gate": args.gate, "batch": wl.batch, "W": wl.W, "r": wl.r,
                      "unit": "us after the decode kernel's wait for the kernel ahead is over; "
                              "[min, 10 %, median, 90 %, max] over the CTAs",
                      "decode_ctas": gd, "boundary_ctas": gb, "steps": steps,
                      "device_error_flags": lq.check_device()}))


# --------------------------------------------------------------------------------------------------
# Long-chain drift: GDN, 64 x 16 heads, heavy-tailed values, 4096 consecutive tokens, W = 16.  Error of o of
# the 8-bit per-window path (and of the bf16-state baseline) against the fp32 recurrence fed the same tokens,
# per block of 256 steps.  All on the GPU through the library; the code parity of the same chain against the
# oracle is a test (tests/test_gpu_parity.py, tests/test_gpu_fullsize.py).
# --------------------------------------------------------------------------------------------------
def run_drift(args):
    import torch
    from paper_2609_38166_b200 import build, lq

    torch.cuda.set_device(0)
    build.build()
    lq.lib()
    wl = synth.config("gdn_drift")
    sh = lq.Shape(wl.batch, wl.heads_v, wl.heads_qk, 128, 128, wl.W, wl.r, wl.n_iter, wl.gate, wl.smooth)
    st = lq.State(sh)
    S = torch.zeros((wl.batch, wl.heads_v, 128, 128), dtype=torch.float32, device="cuda")
    S16 = torch.zeros((wl.batch, wl.heads_v, 128, 128), dtype=torch.int16, device="cuda")
    lq.quantize_state(sh, S, st)
    # the paper's -w baseline beside it: bfloat16 boundary state, rounded once per window
    shw = lq.Shape(wl.batch, wl.heads_v, wl.heads_qk, 128, 128, wl.W, 0, wl.n_iter, wl.gate, 0, state_bf16=1)
    stw = lq.State(shw)
    lq.quantize_state(shw, S, stw)
    o_ref = torch.empty((wl.batch, wl.heads_v, 128), dtype=torch.float32, device="cuda")
    o_q, o_b, o_w = torch.empty_like(o_ref), torch.empty_like(o_ref), torch.empty_like(o_ref)
    steps, block = args.drift_steps, 256
    acc = {"8bit": [], "bf16": [], "bf16_w": []}
    rows = []
    for t in range(steps):
        d = to_dev(synth.token_inputs(wl, t), torch)
        a = (d["q"], d["k"], d["v"], d["beta"], d["alpha"])
        lq.ref_decode_step_f32(sh, S, *a, o_ref)
        lq.decode_step(sh, st, *a, o_q)
        lq.ref_decode_step_bf16(sh, S16, *a, o_b)
        lq.decode_step(shw, stw, *a, o_w)
        den = o_ref.flatten(2).norm(dim=2)                       # per (sequence, head)
        acc["8bit"].append((o_q - o_ref).flatten(2).norm(dim=2) / den)
        acc["bf16"].append((o_b - o_ref).flatten(2).norm(dim=2) / den)
        acc["bf16_w"].append((o_w - o_ref).flatten(2).norm(dim=2) / den)
        if (t + 1) % block == 0:
            row = {"drift": True, "workload": wl.name, "steps": [t + 1 - block, t + 1]}
            for k in acc:
                e = torch.stack(acc[k])                           # [block, B, H]
                row[k] = {"mean": float(e.mean()), "max_over_heads_of_block_mean": float(e.mean(dim=0).max())}
                acc[k] = []
            rows.append(row)
            print(json.dumps(row), flush=True)
    flags = lq.check_device()
    print(f"[drift] device error flags {flags}", file=sys.stderr)
    print("[drift] steps            8-bit per window: mean   max head     bf16 per window: mean   max head     "
          "bf16 every token: mean   max head", file=sys.stderr)
    for r_ in rows:
        print(f"[drift] {r_['steps'][0]:5d}-{r_['steps'][1]:5d}        {r_['8bit']['mean']:.3e}  "
              f"{r_['8bit']['max_over_heads_of_block_mean']:.3e}           {r_['bf16_w']['mean']:.3e}  "
              f"{r_['bf16_w']['max_over_heads_of_block_mean']:.3e}            {r_['bf16']['mean']:.3e}  "
              f"{r_['bf16']['max_over_heads_of_block_mean']:.3e}", file=sys.stderr)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=4000)
    ap.add_argument("--warmup", type=int, default=64)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--W", type=int, default=16)
    ap.add_argument("--batch", type=int, default=256)
    ap.add_argument("--warm-tokens", type=int, default=WARM_TOKENS,
                    help="tokens of the fp32 recurrence that pre-fill the states (512 in the headline workload)")
    ap.add_argument("--no-graph", action="store_true", help="time plain launches instead of CUDA-graph replays")
    ap.add_argument("--no-scratch-words", action="store_true",
                    help="states without lq_state.work: every CTA of the decode kernel takes an equal share of the heads")
    ap.add_argument("--only-timed", action="store_true",
                    help="skip the CUDA-graph, end-to-end, baseline-kernel and CPU legs (for profiler runs)")
    ap.add_argument("--r", type=int, default=4, help="Compensator Tokens per state")
    ap.add_argument("--n-iter", type=int, default=None, help="power-iteration steps (default: the library's)")
    ap.add_argument("--gate", default="gdn", choices=["gdn", "kda"])
    ap.add_argument("--sweep", action="store_true",
                    help="throughput sweep over gate x batch x W x r (one JSON line per point) instead of the headline run")
    ap.add_argument("--ladder", action="store_true",
                    help="ablation ladder: fp32 / bf16 / int8 per token / int8 per window / + compensators / + smoothing, "
                         "speed and error against the fp32 recurrence (one JSON line per rung)")
    ap.add_argument("--drift", action="store_true",
                    help="long-chain drift of the 8-bit path and of the bf16-state baseline against the fp32 recurrence, "
                         "per 256 steps (GDN 64 x 16 heads, Student-t values)")
    ap.add_argument("--drift-steps", type=int, default=4096)
    ap.add_argument("--timeline", action="store_true",
                    help="per-CTA time stamps of both kernels over three steps (library variant built with --stamps)")
    ap.add_argument("--sweep-batches", default="32,128,256,512,1024")
    ap.add_argument("--sweep-W", default="8,16,32,64")
    ap.add_argument("--sweep-r", default="4,8")
    ap.add_argument("--sweep-gates", default="gdn,kda")
    ap.add_argument("--sweep-steps", type=int, default=512)
    ap.add_argument("--sweep-rec16", default="0", help="record buffer: 0 fp32, 1 fp16, or 0,1 for both")
    ap.add_argument("--rec16", type=int, default=0, choices=[0, 1],
                    help="1: fp16 record buffer (the paper's storage) instead of the fp32 buffer of the headline")
    args = ap.parse_args()
    global SCRATCH_WORDS
    SCRATCH_WORDS = not args.no_scratch_words
    if args.sweep:
        run_sweep(args)
        return
    if args.ladder:
        run_ladder(args)
        return
    if args.drift:
        run_drift(args)
        return
    if args.timeline:
        run_timeline(args)
        return
    wl = synth.config("gdn_b256").with_(W=args.W, batch=args.batch, r=args.r)
    if args.gate == "kda":
        wl = wl.with_(name="kda_b%d" % args.batch, gate=synth.GATE_DIAG, heads_qk=wl.heads_v)
    if args.n_iter is not None:
        wl = wl.with_(n_iter=args.n_iter)
    if args.rec16:
        wl = wl.with_(rec16=1, name=wl.name + "_rec16")
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        run_cuda(args, wl)


if __name__ == "__main__":
    main()
