#!/usr/bin/env python
"""Benchmark of the speculative-verification hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl native|reference]

One "step" is one pass of the whole hot path over one batch of synthetic input:
``fef_spec_verify`` (streaming softmax statistics, acceptance scan, residual
draw, confidences) followed by ``fef_remask_select`` (LowConf_k).  The workload
is the headline configuration: B = 64 windows of K = 32 draft positions,
V = 126464 (LLaDA-8B vocabulary), bf16 logits, temperature 1, peaked synthetic
logits with target = draft + N(0, 0.7^2); the re-mask selection runs on a
[64, 1024] confidence state with k = 8.

Prints ONE JSON line (rank 0).  ``--impl reference`` times the CPU oracle on the
host cores instead (a deliberately slow program; context, not a target).
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2605_14305_b200 import synth  # noqa: E402

METRIC = "verified draft positions/sec"
UNIT = "positions/s"
REMASK_L = 1024
FALLBACK_HBM_GBS = 6650.0
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "verify_kernels_B16_bf16_ncu.md")


# ------------------------------------------------------------------ helpers ----
def _workload(args) -> synth.Workload:
    w = synth.CONFIGS[args.workload]
    over = {}
    for name in ("B", "K", "V"):
        if getattr(args, name) is not None:
            over[name] = getattr(args, name)
    if args.dtype is not None:
        over["dtype"] = torch.float32 if args.dtype == "f32" else torch.bfloat16
    if args.temperature is not None:
        over["temperature"] = args.temperature
    if args.noise is not None:
        over["noise_std"] = args.noise
    return w.with_(**over) if over else w


L2_BYTES = 126 << 20


def _input_sets(w: synth.Workload) -> int:
    """Distinct input sets the timed steps rotate over: two when one step's logits exceed L2, else
    enough that the rotation covers twice the L2 (at most 32 sets: tiny workloads stay L2-resident)."""
    per_step = synth.algorithmic_bytes(w)
    if per_step > L2_BYTES:
        return 2
    return int(min(32, max(2, -(-2 * L2_BYTES // per_step))))


def _config_dict(w: synth.Workload, extra=None):
    cfg = {
        "workload": "%s: B=%d windows x K=%d draft positions, V=%d, %s logits, T=%g, %s draft logits, "
                    "target = draft + N(0, %g^2); re-mask select on [%d, %d] confidences, k=%d"
                    % (w.name, w.B, w.K, w.V, "bf16" if w.dtype == torch.bfloat16 else "fp32", w.temperature,
                       w.family, w.noise_std, w.B, REMASK_L, w.remask_k),
        "B": w.B, "K": w.K, "V": w.V, "temperature": w.temperature, "remask_k": w.remask_k,
        "l2": ("inputs of one step (%s) exceed the 126 MB L2 and two input sets alternate"
               % synth.human_bytes(synth.algorithmic_bytes(w))) if synth.algorithmic_bytes(w) > L2_BYTES else
              ("%d input sets of %s rotate (%s in all; L2 is 126 MB)"
               % (_input_sets(w), synth.human_bytes(synth.algorithmic_bytes(w)),
                  synth.human_bytes(_input_sets(w) * synth.algorithmic_bytes(w)))),
    }
    if extra:
        cfg.update(extra)
    return cfg


def _measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json, copy bandwidth)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (earlier measurement on this pool)"


def _ncu_traffic():
    """DRAM bytes per launch of the streaming kernel from the committed ncu summary, or None."""
    try:
        with open(TRAFFIC_FILE) as f:
            for line in f:
                if line.startswith("traffic_bytes_per_launch:"):
                    return float(line.split(":", 1)[1].split()[0])
    except Exception:
        pass
    return None


class ClockSampler(threading.Thread):
    """Samples SM clock and clock-event reasons of one GPU through NVML while the timed region runs."""

    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting", 0x10: "sync_boost"}

    def __init__(self, device_index: int, period_s: float = 0.02):
        super().__init__(daemon=True)
        self.period = period_s
        self.samples, self.reasons, self.power = [], set(), []
        self.max_mhz = None
        self._halt = threading.Event()
        self.ok = False
        try:
            import pynvml

            self.nv = pynvml
            pynvml.nvmlInit()
            handle = None
            try:
                uuid = str(torch.cuda.get_device_properties(device_index).uuid)
                if not uuid.startswith("GPU-"):
                    uuid = "GPU-" + uuid
                handle = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                handle = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.handle = handle
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(handle, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.ok = False

    def sample(self):
        if not self.ok:
            return
        nv = self.nv
        try:
            self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.handle, nv.NVML_CLOCK_SM)))
            try:
                bits = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.handle))
            except Exception:
                bits = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.handle))
            for bit, name in self.REASONS.items():
                if bits & bit:
                    self.reasons.add(name)
            self.power.append(nv.nvmlDeviceGetPowerUsage(self.handle) / 1000.0)
        except Exception:
            pass

    def run(self):
        while not self._halt.is_set():
            self.sample()
            self._halt.wait(self.period)

    def stop(self):
        self.sample()
        self._halt.set()

    def result(self):
        if not self.ok or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["nvml unavailable"], "samples": 0}
        return {"sm_mhz": int(statistics.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples),
                "power_w_max": round(max(self.power), 1) if self.power else None}


# ------------------------------------------------------------- native arm ----
def run_native(args):
    import torch.distributed as dist

    import paper_2605_14305_b200 as fef
    from paper_2605_14305_b200 import dist_util

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the native arm has no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    fef.load(build_if_missing=True)

    w = _workload(args)
    steps, warmup = args.steps, max(args.warmup, 3)
    nbuf = _input_sets(w)
    seed = dist_util.rank_seed(args.seed, rank)
    sets = [synth.make_call(w, seed=1000 * (rank + 1) + i, device=dev) for i in range(nbuf)]
    g = torch.Generator(device=dev).manual_seed(77 + rank)
    conf_state = torch.rand((w.B, REMASK_L), generator=g, device=dev)
    mask_state = (torch.rand((w.B, REMASK_L), generator=g, device=dev) < 0.5).to(torch.uint8)
    out = fef.VerifyResult(torch.empty(w.B, dtype=torch.int32, device=dev),
                           torch.empty((w.B, w.K), dtype=torch.int32, device=dev),
                           torch.empty((w.B, w.K), dtype=torch.float32, device=dev),
                           torch.zeros(1, dtype=torch.int32, device=dev))
    ws = torch.empty(max(fef.fef_spec_verify_workspace_bytes(w.B, w.K, w.V, w.dtype), 256), dtype=torch.uint8,
                     device=dev)
    positions = torch.empty((w.B, w.remask_k), dtype=torch.int32, device=dev)
    count = torch.empty(w.B, dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream()

    stage_ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(steps)]
    for evs in stage_ev:
        for e in evs:
            e.record(stream)  # creates the underlying CUDA event

    def step(i, stages=None):
        q, p, tok = sets[i % nbuf]
        fef.fef_spec_verify(q, p, tok, w.temperature, seed, i, out=out, workspace=ws, stage_events=stages)
        fef.fef_remask_select(conf_state, mask_state, w.remask_k, positions=positions, count=count)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(warmup):
        step(i)
    barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    # timed region 1: the K steps as a user runs them
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record(stream)
    for i in range(steps):
        step(warmup + i)
    t1.record(stream)
    barrier()
    elapsed_ms = t0.elapsed_time(t1)
    # timed region 2: each of the two calls alone, K times back to back between two CUDA events
    # (events between the calls would sit inside their dependent-launch chains)
    call_ms = [0.0, 0.0]
    if not args.no_call_events:
        c0, c1, c2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        c0.record(stream)
        for i in range(steps):
            q, p, tok = sets[(warmup + i) % nbuf]
            fef.fef_spec_verify(q, p, tok, w.temperature, seed, warmup + i, out=out, workspace=ws)
        c1.record(stream)
        for i in range(steps):
            fef.fef_remask_select(conf_state, mask_state, w.remask_k, positions=positions, count=count)
        c2.record(stream)
        barrier()
        call_ms = [c0.elapsed_time(c1) / steps, c1.elapsed_time(c2) / steps]
    # timed region 3: once more with events at the kernel boundaries inside the verification call
    # (fef_spec_verify_profiled), for the duration of each kernel alone
    stage_ms = [0.0, 0.0]
    if not args.no_call_events:
        for i in range(steps):
            step(warmup + i, stage_ev[i])
        barrier()
        for evs in stage_ev:
            for j in range(2):
                stage_ms[j] += evs[j].elapsed_time(evs[j + 1])
        stage_ms = [x / steps for x in stage_ms]
    # timed region 4 (not part of the step): the draft-token draws that precede a verification call
    draft_ms = norm_ms = both_ms = round_ms = None
    if not args.no_call_events:
        dws = torch.empty(max(fef.fef_draft_sample_workspace_bytes(w.B, w.K, w.V, w.dtype), 256), dtype=torch.uint8,
                          device=dev)
        dout = fef.fef_draft_sample(sets[0][0], w.temperature, seed, 0, workspace=dws)
        d0, d1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        d0.record(stream)
        for i in range(steps):
            fef.fef_draft_sample(sets[i % nbuf][0], w.temperature, seed, i, out=dout, workspace=dws)
        d1.record(stream)
        barrier()
        draft_ms = d0.elapsed_time(d1) / steps
        # ... and the verification that reuses their normalisers (streams the target rows only)
        douts = [fef.fef_draft_sample(sets[i][0], w.temperature, seed, 0) for i in range(nbuf)]
        barrier()
        d0.record(stream)
        for i in range(steps):
            q, p, _ = sets[i % nbuf]
            fef.fef_spec_verify(q, p, douts[i % nbuf].tokens, w.temperature, seed, 0, out=out, workspace=ws,
                                draft_log2_norm=douts[i % nbuf].log2_norm)
        d1.record(stream)
        barrier()
        norm_ms = d0.elapsed_time(d1) / steps
        # ... and a whole round with both tensors read once: draft draws that also reduce the target rows, then
        # the verification that takes both normalisers (it streams nothing)
        dboth = fef.fef_draft_sample(sets[0][0], w.temperature, seed, 0, workspace=dws, target_logits=sets[0][1])
        barrier()
        d0.record(stream)
        for i in range(steps):
            q, p, _ = sets[i % nbuf]
            fef.fef_draft_sample(q, w.temperature, seed, i, out=dboth, workspace=dws, target_logits=p)
        d1.record(stream)
        for i in range(steps):
            q, p, _ = sets[i % nbuf]
            fef.fef_draft_sample(q, w.temperature, seed, i, out=dboth, workspace=dws, target_logits=p)
            fef.fef_spec_verify(q, p, dboth.tokens, w.temperature, seed, i, out=out, workspace=ws,
                                draft_log2_norm=dboth.log2_norm, target_log2_norm=dboth.target_log2_norm)
        d2 = torch.cuda.Event(enable_timing=True)
        d2.record(stream)
        barrier()
        both_ms = d0.elapsed_time(d1) / steps
        round_ms = d1.elapsed_time(d2) / steps
    sampler.stop()
    status = int(out.device_status.item())
    accept_mean = float(out.accept_len.float().mean().item())
    rejected = int((out.accept_len < w.K).sum().item())

    # ---- end to end through the host-buffer entry points (copies inside the timed region)
    e2e_steps = max(1, min(steps, args.e2e_steps))
    hq, hp, htok = (t.cpu().pin_memory() for t in sets[0])
    hconf, hmask = conf_state.cpu().pin_memory(), mask_state.cpu().pin_memory()
    arena = torch.empty(fef.fef_spec_verify_host_arena_bytes(w.B, w.K, w.V, w.V, w.dtype), dtype=torch.uint8, device=dev)
    arena2 = torch.empty(fef.fef_remask_select_host_arena_bytes(w.B, REMASK_L, w.remask_k), dtype=torch.uint8, device=dev)
    hout = fef.HostVerifyResult(torch.empty(w.B, dtype=torch.int32).pin_memory(),
                                torch.empty((w.B, w.K), dtype=torch.int32).pin_memory(),
                                torch.empty((w.B, w.K), dtype=torch.float32).pin_memory(), 0)
    hpos = torch.empty((w.B, w.remask_k), dtype=torch.int32).pin_memory()
    hcnt = torch.empty(w.B, dtype=torch.int32).pin_memory()

    def host_step(i):
        fef.fef_spec_verify_host(hq, hp, htok, w.temperature, seed, i, arena, out=hout)
        fef.fef_remask_select_host(hconf, hmask, w.remask_k, arena2, positions=hpos, count=hcnt)

    host_step(0)
    barrier()
    h0, h1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    h0.record(stream)
    for i in range(e2e_steps):
        host_step(1 + i)
    h1.record(stream)
    barrier()
    e2e_ms = h0.elapsed_time(h1)

    elapsed_ms, e2e_ms = dist_util.max_over_ranks([elapsed_ms, e2e_ms], device=dev)

    logits_bytes = hq.numel() * hq.element_size() * (2 if w.temperature > 0 else 1)
    h2d = logits_bytes + htok.numel() * 4 + hconf.numel() * 4 + hmask.numel()
    d2h = w.B * 4 + w.B * w.K * 8 + 4 + w.B * w.remask_k * 4 + w.B * 4

    # ---- CPU baseline: the oracle as it stands, on rank 0 at N = 1 only
    cpu_baseline, parity = None, None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        from oracle.compare import compare_verify

        nwin = min(w.B, args.cpu_windows)
        q, p, tok = (t[:nwin].cpu() for t in sets[0])
        reps, t_cpu, ref = 0, 0.0, None
        while t_cpu < args.cpu_seconds and reps < 8:
            c0 = time.perf_counter()
            ref = oracle.spec_verify(q, p, tok, w.temperature, args.seed, 424242)
            t_cpu += time.perf_counter() - c0
            reps += 1
        cpu_baseline = {"value": reps * nwin * w.K / t_cpu, "unit": UNIT, "cores": 1, "kind": "oracle",
                        "host_cores": os.cpu_count(),
                        "sample": "%d call(s) over the first %d of %d windows of the same batch (%d positions each), "
                                  "%.1f s of single-thread CPU time" % (reps, nwin, w.B, nwin * w.K, t_cpu)}
        got = fef.fef_spec_verify(sets[0][0], sets[0][1], sets[0][2], w.temperature, args.seed, 424242)
        torch.cuda.synchronize()
        rep = compare_verify(got.accept_len[:nwin].cpu().numpy(), got.tokens[:nwin].cpu().numpy(),
                             got.conf[:nwin].cpu().numpy(), ref)
        parity = {"windows": rep.windows, "draws": rep.draws, "near_margin": rep.near_margin,
                  "excused": rep.excused, "mismatches": len(rep.mismatches),
                  "max_conf_rel_err": rep.max_conf_rel_err}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    positions_per_step = w.B * w.K * world
    value = dist_util.aggregate_rate(w.B * w.K, steps, elapsed_ms, world)
    peak, peak_src = _measured_peak()
    row_bytes = (2 if w.temperature > 0 else 1) * w.V * w.logit_bytes
    stream_bytes = w.B * w.K * row_bytes
    roof = {"bound": "hbm", "kernel": "stream_kernel", "unit": "GB/s", "peak": peak, "peak_source": peak_src,
            "traffic": _ncu_traffic(), "algorithmic_bytes_per_launch": stream_bytes}
    if not args.no_call_events and stage_ms[0] > 0:
        roof["achieved"] = stream_bytes / (stage_ms[0] * 1e-3) / 1e9
        roof["frac"] = roof["achieved"] / peak
        roof["frac_of_8TBs"] = roof["achieved"] / 8000.0
        roof["ms_per_launch"] = stage_ms[0]
        roof["kernel_ms"] = {"stream_kernel": stage_ms[0],
                             ("tail_kernel" if w.temperature > 0 else "scan_kernel"): stage_ms[1]}
        roof["timed"] = ("third pass over the same K steps with CUDA events at the kernel boundaries "
                         "(fef_spec_verify_profiled)")
        # the whole verification call (three kernels chained with dependent launches), K calls back to back,
        # every row counted once although the rejected rows are read a second time
        roof["call_ms"] = {"fef_spec_verify": call_ms[0], "fef_remask_select": call_ms[1]}
        roof["call_achieved"] = stream_bytes / (call_ms[0] * 1e-3) / 1e9
        roof["call_frac"] = roof["call_achieved"] / peak
        roof["call_frac_of_8TBs"] = roof["call_achieved"] / 8000.0
    else:
        roof["achieved"], roof["frac"] = None, None
    call_bytes = synth.algorithmic_bytes(w, rejected_rows=rejected)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
        "ms_per_step": elapsed_ms / steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic", "config": _config_dict(w),
        "parallelism": "replicas x%d (windows are independent; no collective)" % world,
        "impl": "native",
        "hbm_gbs_whole_step": call_bytes / (elapsed_ms / steps * 1e-3) / 1e9,
        "frac_of_8TBs_whole_step": call_bytes / (elapsed_ms / steps * 1e-3) / 8e12,
        "roofline": roof,
        "e2e": {"value": positions_per_step * e2e_steps / (e2e_ms * 1e-3), "unit": UNIT, "steps": e2e_steps,
                "ms_per_step": e2e_ms / e2e_steps, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "api": "fef_spec_verify_host + fef_remask_select_host (pinned host buffers)"},
        "draft_sample": None if draft_ms is None else {
            "ms_per_call": draft_ms, "positions_per_s": w.B * w.K / (draft_ms * 1e-3),
            "gbs": w.B * w.K * w.V * w.logit_bytes / (draft_ms * 1e-3) / 1e9,
            "note": "fef_draft_sample on the draft logits of the same workload; bound by Philox arithmetic, not "
                    "by HBM; not part of the step",
            "verify_with_draft_norm_ms": norm_ms,
            "verify_with_draft_norm_positions_per_s": w.B * w.K / (norm_ms * 1e-3),
            "draft_sample_with_target_ms": both_ms,
            "round_ms": round_ms,
            "round_note": "fef_draft_sample with the target logits + fef_spec_verify with both normalisers: one "
                          "whole round of Algorithm 2 (draws, verification), both tensors read once",
            "round_positions_per_s": w.B * w.K / (round_ms * 1e-3),
            "round_gbs": 2 * w.B * w.K * w.V * w.logit_bytes / (round_ms * 1e-3) / 1e9},
        # per step: begin-call, streaming, tail (acceptance tests + residual draw; greedy: scan), re-mask kernels
        "gpu_launches": steps * 4,
        "clocks": sampler.result(),
        "cpu_baseline": cpu_baseline,
        "parity_vs_oracle": parity,
        "device_status": status, "mean_accept_len": accept_mean,
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


# ---------------------------------------------------------- reference arm ----
def run_reference(args):
    """The CPU oracle, as it stands, on the host cores: each step verifies a bounded sample
    (the first n windows) of the same workload."""
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if rank != 0:
        return
    import oracle

    w = _workload(args)
    steps, warmup = args.steps, args.warmup
    # about 0.07 s of CPU time per headline-shaped window; keep the whole run near two minutes
    per_window_s = 0.07 * (w.V / 126464.0) * (w.K / 32.0)
    nwin = int(max(1, min(w.B, math.floor(120.0 / ((steps + warmup) * per_window_s)))))
    q, p, tok = synth.make_call(w.with_(B=nwin), seed=1000, device="cpu")
    for i in range(warmup):
        oracle.spec_verify(q, p, tok, w.temperature, args.seed, i)
    c0 = time.perf_counter()
    for i in range(steps):
        ref = oracle.spec_verify(q, p, tok, w.temperature, args.seed, warmup + i)
        conf = ref["conf"].astype("float32")
        oracle.remask_select(conf, (conf >= 0).astype("uint8"), w.remask_k)
    elapsed = time.perf_counter() - c0
    value = nwin * w.K * steps / elapsed
    sample = "each step: the first %d of %d windows (%d positions) of the workload" % (nwin, w.B, nwin * w.K)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps,
        "warmup": warmup, "ms_per_step": elapsed / steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": _config_dict(w), "parallelism": "one host thread",
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample,
                         "host_cores": os.cpu_count()},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ------------------------------------------------------------- loop sweep ----
def run_loop_sweep(args):
    """Extra mode (not the contract's line): the long-generation sweep.  The full decoding loop
    (window, logits, draft draws that also reduce the target rows, verification with both
    normalisers, commit; LowConf and re-masking between the denoising steps) on a device-resident
    state of L = 1024 positions per sequence until nothing is masked, at B in {1, 8, 64} x
    K in {8, 32, 64}, bf16 and fp32.  The logits of every round are made on the device from a seeded
    Philox stream (target = draft + N(0, 0.7^2)) inside the round; the generator's own time per
    round is measured separately and reported beside the round time.  "eager": the host drives the
    rounds and reads one integer per round; "graph": the whole loop is one graph launch
    (fef_loop_run_synthetic: a WHILE node around the round, no host in between)."""
    import paper_2605_14305_b200 as fef
    from paper_2605_14305_b200.decode_loop import run_decode_loop_device

    fef.load(build_if_missing=True)
    torch.cuda.set_device(0)
    L, remask_k, steps, V, T = 1024, 8, 2, synth.HEADLINE.V, 1.0
    points = []
    for dtype in (torch.bfloat16, torch.float32):
        for B in (1, 8, 64):
            for K in (8, 32, 64):
                def logits_fn(rnd, window, row_len, inputs):
                    return fef.fef_synth_logits(B, K, V, dtype, 2.0, 0.7, args.seed, rnd, boost_fraction=0.01, boost=8.0)

                # the generator alone
                buf = logits_fn(0, None, None, None)
                torch.cuda.synchronize()
                g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                g0.record()
                for r in range(10):
                    fef.fef_synth_logits(B, K, V, dtype, 2.0, 0.7, args.seed, r, boost_fraction=0.01, boost=8.0, out=buf)
                g1.record()
                torch.cuda.synchronize()
                gen_us = g0.elapsed_time(g1) * 1e3 / 10
                del buf
                run_decode_loop_device(fef, B, L, K, steps, remask_k, logits_fn, T, args.seed, reuse_target_norm=True, V=V)
                eager = run_decode_loop_device(fef, B, L, K, steps, remask_k, logits_fn, T, args.seed,
                                               reuse_target_norm=True, V=V)
                fef.fef_loop_run_synthetic(B, L, K, V, dtype, T, args.seed, steps, remask_k, 2.0, 0.7, 0.01, 8.0)
                torch.cuda.synchronize()
                t0 = time.perf_counter()
                graph = fef.fef_loop_run_synthetic(B, L, K, V, dtype, T, args.seed, steps, remask_k, 2.0, 0.7, 0.01, 8.0)
                torch.cuda.synchronize()
                graph_s = time.perf_counter() - t0
                same = bool((graph["tokens"] == eager["tokens"]).all().item()) and graph["rounds"] == eager["rounds"]
                rounds = eager["rounds"]
                points.append({
                    "B": B, "K": K, "dtype": "bf16" if dtype == torch.bfloat16 else "f32", "rounds": rounds,
                    "generator_us_per_round": gen_us,
                    "eager_us_per_round": eager["loop_seconds"] * 1e6 / rounds,
                    "graph_us_per_round": graph_s * 1e6 / rounds,
                    "graph_us_per_round_without_generator": graph_s * 1e6 / rounds - gen_us,
                    "committed_positions_per_s_graph": (B * L + B * remask_k) / graph_s,
                    "graph_equals_eager": same})
    print(json.dumps({"mode": "loop sweep", "L": L, "V": V, "denoising_steps": steps, "remask_k": remask_k,
                      "round": "fef_synth_logits + fef_draft_sample_with_target + fef_spec_verify_with_norms + bookkeeping",
                      "note": "graph time includes building and instantiating the graph (once per loop)",
                      "data": "synthetic", "points": points}))


# ------------------------------------------------------- from hidden states ----
def run_lmhead(args):
    """Extra mode (not the contract's line): verification straight from hidden states
    (``fef_lmhead_verify``: output-layer product on the tensor cores with the softmax partials in its
    epilogue) at the headline window shape with a hidden width of ``--d`` (default 4096), against a
    tensor-core roofline; beside it the unfused path: two library products that write bfloat16 logits,
    then ``fef_spec_verify`` on them."""
    import paper_2605_14305_b200 as fef

    fef.load(build_if_missing=True)
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    w = _workload(args)
    B, K, V, d, T = w.B, w.K, w.V, args.d, w.temperature if w.temperature > 0 else 1.0
    g = torch.Generator(device=dev).manual_seed(args.seed)
    Hq = torch.randn((B * K, d), generator=g, device=dev)
    Hp = (Hq + 0.35 * torch.randn((B * K, d), generator=g, device=dev)).to(torch.bfloat16)
    Hq = Hq.to(torch.bfloat16)
    W = (torch.randn((V, d), generator=g, device=dev) * (2.0 / math.sqrt(d))).to(torch.bfloat16)
    lq = Hq @ W.T
    tok = synth.sample_draft_tokens(lq.view(B, K, V), T, args.seed + 1)
    ws = torch.empty(fef.fef_lmhead_verify_workspace_bytes(B, K, V, d), dtype=torch.uint8, device=dev)
    out = fef.fef_lmhead_verify(Hq, Hp, W, tok, T, args.seed, 0, workspace=ws)
    ws2 = torch.empty(fef.fef_spec_verify_workspace_bytes(B, K, V, torch.bfloat16), dtype=torch.uint8, device=dev)
    lp = torch.empty_like(lq)
    out2 = fef.fef_spec_verify(lq.view(B, K, V), lq.view(B, K, V), tok, T, args.seed, 0, workspace=ws2)
    steps, warmup = min(args.steps, 50), max(3, min(args.warmup, 5))
    sampler = ClockSampler(0)
    sampler.start()

    def unfused(i):
        torch.matmul(Hq, W.T, out=lq)
        torch.matmul(Hp, W.T, out=lp)
        fef.fef_spec_verify(lq.view(B, K, V), lp.view(B, K, V), tok, T, args.seed, i, out=out2, workspace=ws2)

    arms = [lambda i: fef.fef_lmhead_verify(Hq, Hp, W, tok, T, args.seed, i, out=out, workspace=ws),
            unfused,
            lambda i: (torch.matmul(Hq, W.T, out=lq), torch.matmul(Hp, W.T, out=lp))]
    # The three arms take turns in blocks of a few steps, so that all of them see the same clocks: a dense
    # product runs under the power cap, and an arm timed alone, minutes after another, is not comparable.
    block = 5
    for fn in arms:
        for i in range(warmup):
            fn(i)
    torch.cuda.synchronize()
    total = [0.0, 0.0, 0.0]
    done = 0
    while done < steps:
        n = min(block, steps - done)
        marks = []
        for fn in arms:
            t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            t0.record()
            for i in range(n):
                fn(warmup + done + i)
            t1.record()
            marks.append((t0, t1))
        torch.cuda.synchronize()
        for k, (t0, t1) in enumerate(marks):
            total[k] += t0.elapsed_time(t1)
        done += n
    fused_ms, unfused_ms, gemm_ms = (t / steps for t in total)
    sampler.stop()
    status = int(out.device_status.item())
    same = bool((out.accept_len == out2.accept_len).float().mean().item() > 0.9)
    flops_stats = 2.0 * 2 * B * K * d * V
    flops_all = flops_stats + 2.0 * 2 * B * d * V
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            peak, src = float(json.load(f)["bf16_tflops_sustained"]), "measured (MEASURED_PEAKS.json, sustained bf16 GEMM)"
    except Exception:
        peak, src = 1400.0, "fallback (earlier measurement on this pool, sustained)"
    line = {
        "mode": "verification from hidden states", "metric": METRIC, "unit": UNIT, "data": "synthetic", "dtype": "bf16",
        "config": {"workload": "B=%d windows x K=%d positions, hidden width %d, V=%d, bf16 hidden states and weight, T=%g"
                               % (B, K, d, V, T)},
        "value": B * K / (fused_ms * 1e-3), "ms_per_step": fused_ms, "steps": steps, "warmup": warmup,
        "roofline": {"bound": "tensor", "kernel": "lmhead_gemm_kernel", "unit": "TFLOP/s", "peak": peak, "peak_source": src,
                     "achieved": flops_all / (fused_ms * 1e-3) / 1e12, "frac": flops_all / (fused_ms * 1e-3) / 1e12 / peak,
                     "flops_per_call": flops_all, "traffic": None,
                     "note": "whole call (both products, acceptance, the rejected rows' product, residual draw)"},
        "unfused": {"ms_per_step": unfused_ms, "library_products_ms": gemm_ms,
                    "library_tflops": flops_stats / (gemm_ms * 1e-3) / 1e12,
                    "note": "torch.matmul to bfloat16 logits twice, then fef_spec_verify; the arms alternate in blocks "
                            "of %d steps" % block},
        "device_status": status, "accept_len_mostly_equal_to_unfused": same, "clocks": sampler.result(),
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=500)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", choices=["native", "reference"], default="native")
    ap.add_argument("--workload", default="headline", choices=sorted(synth.CONFIGS))
    ap.add_argument("--B", type=int)
    ap.add_argument("--K", type=int)
    ap.add_argument("--V", type=int)
    ap.add_argument("--dtype", choices=["bf16", "f32"])
    ap.add_argument("--temperature", type=float)
    ap.add_argument("--noise", type=float)
    ap.add_argument("--seed", type=int, default=20260514)
    ap.add_argument("--e2e-steps", type=int, default=20)
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--cpu-windows", type=int, default=64)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-call-events", action="store_true")
    ap.add_argument("--loop-sweep", action="store_true", help="time the full decoding loop at the sweep points instead")
    ap.add_argument("--lmhead", action="store_true", help="time verification from hidden states (tensor-core product) instead")
    ap.add_argument("--d", type=int, default=4096, help="hidden width for --lmhead")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and not args.loop_sweep:
        # started by hand for several GPUs: become one rank per GPU (the same launch the driver uses)
        port = str(29500 + os.getpid() % 2000)
        os.execvp(sys.executable, [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node",
                                   str(args.gpus), "--master-addr", "127.0.0.1", "--master-port", port,
                                   os.path.abspath(__file__)] + sys.argv[1:])
    if args.lmhead:
        run_lmhead(args)
    elif args.loop_sweep:
        run_loop_sweep(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_native(args)


if __name__ == "__main__":
    main()
