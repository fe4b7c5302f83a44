#!/usr/bin/env python
"""Benchmark of the MtPC head on B200: window log-likelihood positions/s on the training-shaped CP workload
(8192 positions, d=4096, n=8, r=16, v=320), plus draft windows/s on one decode cell.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 1|2|3|5|6] [--impl reference]

One step = one mtpc_window_logprob call over the whole batch (projection GEMM with fused softmax/gather
epilogue + circuit evaluation). Prints ONE JSON line on rank 0. With N > 1 (launched by torchrun, one process
per GPU) every rank runs an independent replica: the head has no exchange step, so there is no collective on
the data path; ranks meet only at the timing barrier and `value` sums the replicas' work over the slowest
rank's time. `--impl reference` times the fp64 CPU oracle on the host cores instead (rank 0 only).
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
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2511_11346_b200 import inputs as I          # noqa: E402
from paper_2511_11346_b200 import replicas             # noqa: E402

METRIC = "window_loglik_positions_per_s"
UNIT = "positions/s"
FALLBACK_PEAKS = {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0}
# dram__bytes_read.sum + dram__bytes_write.sum of one projection-kernel launch, from the ncu captures
# summarised in profiles/ (captured on the full configuration). None = not captured, or the kernel has changed since.
NCU_TRAFFIC_BYTES = {1: 1_094_800_000, 2: 2_533_300_000, 3: 1_196_800_000, 5: None, 6: None}   # profiles/gemm_logprob_cfg1_cfg2_cfg3_ncu.txt
BURST_REGION_S = 1.0      # a timed loop shorter than this runs at boost clocks: its tensor roofline is the burst peak
SUSTAINED_LOOP_S = 2.5    # length of the second, power-capped loop whose roofline is the sustained peak


def workload_name(idx: int, wl) -> str:
    s = wl.shape
    return (f"configs[{idx}] {wl.name}: T={wl.T} d={s.d} n={s.n} r={s.r} v={s.v} "
            f"{'bf16' if s.io_dtype == I.BF16 else 'fp32'} io")


def algorithmic_flops(wl) -> float:
    """2 d (n r v + S r) per position: the method's own projection work (Table 3's 'MTP head linear')."""
    s = wl.shape
    return 2.0 * s.d * (s.n * s.r * s.symbols + s.sum_rows) * wl.T      # padding symbols earn no credit


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs (read-only)."""

    def __init__(self, index: int, period_s: float = 0.001):
        self.period_s = period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
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
        names = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "sw_thermal_slowdown": 0x20, "hw_thermal_slowdown": 0x40,
                 "hw_power_brake_slowdown": 0x80}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(self.period_s)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join(timeout=2)
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def oracle_positions_per_s(wl, sample_positions: int, chunk: int = 256):
    """The oracle as it stands, on the first `sample_positions` positions, in chunks (memory)."""
    from oracle import mtpc_oracle as orc
    s = wl.shape
    t0 = time.perf_counter()
    done = 0
    while done < sample_positions:
        rows = slice(done, min(done + chunk, sample_positions))
        orc.window_logprob(s.family, wl.hidden_q[rows], wl.W_emit_q, wl.W_sum_q, wl.T_static, wl.targets[rows])
        done = rows.stop
    dt = time.perf_counter() - t0
    return sample_positions / dt, dt


def host_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = max((p.get("num_threads", 1) for p in threadpool_info()), default=1)
        return int(n)
    except Exception:
        return os.cpu_count() or 1


def run_reference(args):
    rank, _, world = replicas.rank_env()
    if rank != 0:
        return
    wl = I.config_workload(args.workload)
    for _ in range(max(args.warmup, 1)):
        rate, _ = oracle_positions_per_s(wl, 64, chunk=64)
    # bounded sample: the whole run should take about two minutes whatever K is
    budget_s = 120.0
    sample = int(max(16, min(wl.T, args.ref_positions, rate * budget_s / max(args.steps, 1))))
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_positions_per_s(wl, sample)
    dt = time.perf_counter() - t0
    value = sample * args.steps / dt
    cores = host_threads()
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_block(args.workload, wl, world),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": f"first {sample} of {wl.T} positions per step, {args.steps} steps"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def circuit_bytes(wl) -> int:
    """Algorithmic bytes of one circuit-evaluation launch: it reads G [T, n, r] and log omega [T, S r] and writes [T]."""
    s = wl.shape
    return 4 * wl.T * (s.n * s.r + s.sum_rows + 1)


def graph_replay_times(torch, enqueue, outputs, steps: int, warmup: int):
    """Capture enqueue(stream) once into a CUDA graph on a side stream, zero `outputs`, replay it `warmup` times untimed
    and `steps` times timed (CUDA events on that stream, one replay each): the per-replay times in ms. The outputs hold
    the last replay's results when it returns."""
    side = torch.cuda.Stream()
    times = []
    with torch.cuda.stream(side):
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            enqueue(side)
        for t in outputs:
            t.zero_()
        for _ in range(warmup):
            graph.replay()
        side.synchronize()
        for _ in range(steps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            graph.replay()
            e1.record()
            e1.synchronize()
            times.append(e0.elapsed_time(e1))
    del graph
    return times


def measure_decode_cell(torch, cell, steps: int, warmup: int, with_graph: bool = True):
    """Draft windows/s and p50 latency on one decode cell (family, n, P) with 16 windows per position. Every call
    is timed on its own (CUDA events on the launching stream); the library's event ring gives the per-kernel split."""
    from paper_2511_11346_b200.runner import DeviceHead
    wl = I.config_workload(4, cell=cell)
    dh = DeviceHead(wl)
    h = dh.hidden_device()
    u = torch.from_numpy(wl.uniforms).cuda()
    W = wl.T * wl.wpp
    ob = torch.empty((W, wl.shape.n), dtype=torch.int32, device="cuda")
    ol = torch.empty(W, dtype=torch.float32, device="cuda")
    for _ in range(warmup):
        dh.head.mtpc_draft_sample(h, wl.wpp, u, ob, ol)
    torch.cuda.synchronize()
    # latency of the call as a user makes it (per-kernel events off: the kernels of a call overlap their launches)
    lat = []
    for _ in range(steps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        dh.head.mtpc_draft_sample(h, wl.wpp, u, ob, ol)
        e1.record()
        e1.synchronize()
        lat.append(e0.elapsed_time(e1))
    # the same call captured once into a CUDA graph and replayed: what a serving loop pays once the host side of the
    # three launches (tensor-map encode, launch attributes, the binding) is out of the way; results must be identical
    ref_b, ref_l = ob.clone(), ol.clone()
    graph_lat, graph_identical = [], None
    if with_graph:
        graph_lat = graph_replay_times(torch, lambda st: dh.head.mtpc_draft_sample(h, wl.wpp, u, ob, ol, stream=st),
                                       (ob, ol), steps, warmup)
        graph_identical = bool((ob == ref_b).all()) and bool(((ol == ref_l) | (ol.isnan() & ref_l.isnan())).all())
    # per-kernel split from the library's event ring (a second pass: the events serialise the kernels)
    ksteps = min(steps, 50)
    dh.head.mtpc_set_timing(ksteps)
    for _ in range(ksteps):
        dh.head.mtpc_draft_sample(h, wl.wpp, u, ob, ol)
    phases = [dh.head.mtpc_get_timing(i) for i in range(ksteps)]
    phase_p50 = [statistics.median(p[k] for p in phases) for k in range(len(phases[0]))]
    launches = len(phases[0])
    dh.head.mtpc_set_timing(0)
    # draft with prefix marginals + acceptance stage (Algorithm 3) against synthetic target-model rows
    s = wl.shape
    tp = torch.from_numpy(I.target_rows(I.BASE_SEED + 77, 9, (W, s.n + 1, s.v))).cuda()
    ua = torch.from_numpy(I.uniforms(I.BASE_SEED + 78, 10, (W, s.n + 1))).cuda()
    opre = torch.empty((W, s.n), dtype=torch.float32, device="cuda")
    oacc = torch.empty(W, dtype=torch.int32, device="cuda")
    onxt = torch.empty(W, dtype=torch.int32, device="cuda")
    cyc = []
    for it in range(warmup + steps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        dh.head.mtpc_draft_sample_prefix(h, wl.wpp, u, ob, opre)
        dh.head.mtpc_speculative_accept(wl.T, wl.wpp, ob, opre, tp, ua, oacc, onxt)
        e1.record()
        e1.synchronize()
        if it >= warmup:
            cyc.append(e0.elapsed_time(e1))
    mean_accepted = float(oacc.float().mean().cpu())
    ref_acc, ref_nxt = oacc.clone(), onxt.clone()
    graph_cyc, cycle_identical = [], None
    if with_graph:
        def cycle(st):
            dh.head.mtpc_draft_sample_prefix(h, wl.wpp, u, ob, opre, stream=st)
            dh.head.mtpc_speculative_accept(wl.T, wl.wpp, ob, opre, tp, ua, oacc, onxt, stream=st)
        graph_cyc = graph_replay_times(torch, cycle, (oacc, onxt), steps, warmup)
        cycle_identical = bool((oacc == ref_acc).all()) and bool((onxt == ref_nxt).all())
    status = dh.head.mtpc_get_status()
    p50 = statistics.median(lat)
    weight_bytes = (s.n * s.r * s.v + s.sum_rows) * s.d * 2
    peaks, src = load_peaks()
    gbs = weight_bytes / (p50 * 1e-3) / 1e9
    graph_p50 = statistics.median(graph_lat) if with_graph else None
    gemm_gbs = weight_bytes / (phase_p50[0] * 1e-3) / 1e9
    out = {"workload": f"configs[4] {wl.name}: P={wl.T} wpp={wl.wpp} d={s.d} n={s.n} r={s.r} v={s.v}",
           "windows_per_s": W / (p50 * 1e-3), "p50_ms": p50, "calls": steps, "kernels_per_call": launches,
           "kernel_p50_ms": phase_p50, "device_status": status,
           "cuda_graph_replay": None if graph_p50 is None else {
                                 "p50_ms": graph_p50, "hbm_frac": weight_bytes / (graph_p50 * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                 "results_identical_to_plain_call": graph_identical,
                                 "note": "mtpc_draft_sample captured once by the caller (torch.cuda.graph), replayed"},
           "draft_plus_accept": {"p50_ms": statistics.median(cyc), "kernels_per_call": launches + 1,
                                 "mean_accepted_bytes_vs_synthetic_target": mean_accepted,
                                 "calls": "mtpc_draft_sample_prefix + mtpc_speculative_accept",
                                 "cuda_graph_replay_p50_ms": statistics.median(graph_cyc) if with_graph else None,
                                 "cuda_graph_results_identical": cycle_identical},
           "hbm_roofline": {"algorithmic_bytes": weight_bytes, "note": "one pass over the emission and sum-unit weights",
                            "achieved_gbs": gbs, "peak_gbs": peaks["hbm_gbs"], "frac": gbs / peaks["hbm_gbs"],
                            "weight_pass_kernel_gbs": gemm_gbs, "weight_pass_kernel_frac": gemm_gbs / peaks["hbm_gbs"],
                            "peak_source": src}}
    dh.close()
    calls = (steps + warmup) + ((steps + warmup + 1) if with_graph else 0)        # plain loop; capture + replays
    return out, launches * (calls + min(steps, 50)) + (launches + 1) * calls


def measure_backward(torch, dh, wl, hidden, targets, steps: int, peaks):
    """One training step of the head = mtpc_window_logprob_backward (forward value + all gradients): ms per call,
    the per-phase split from the library's event ring, and the tensor throughput over the three weight-sized
    contractions it runs (forward, d hidden, dW): 3 x the forward's algorithmic FLOPs."""
    s = wl.shape
    f32 = dict(dtype=torch.float32, device="cuda")
    weight = torch.full((wl.T,), -1.0 / wl.T, **f32)
    out = (torch.empty(wl.T, **f32), torch.empty((wl.T, s.d), **f32), torch.empty((s.n, s.r, s.v, s.d), **f32),
           torch.empty((s.sum_rows, s.d), **f32), torch.empty((max(s.n - 1, 1), s.r, s.r), **f32) if s.family == I.HMM else None)
    call = lambda: dh.head.mtpc_window_logprob_backward(hidden, targets, weight, *out)
    for _ in range(3):
        call()
    torch.cuda.synchronize()
    dh.head.mtpc_set_timing(steps)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        call()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    phases = [dh.head.mtpc_get_timing(i) for i in range(steps)]
    phase_ms = [statistics.mean(p[k] for p in phases) for k in range(len(phases[0]))]
    dh.head.mtpc_set_timing(0)
    flops = 3.0 * algorithmic_flops(wl)
    tf = flops / (ms * 1e-3) / 1e12
    eq6 = measure_eq6_step(torch, dh, wl, hidden, targets, out, steps)
    lowrank = measure_lowrank(torch, wl, out[2], steps, peaks) if s.v <= 1536 else None
    return {"eq6_training_step": eq6, "lowrank_unembeddings": lowrank, "call": "mtpc_window_logprob_backward", "ms_per_call": ms, "positions_per_s": wl.T / (ms * 1e-3),
            "phase_ms": {"forward_projection": phase_ms[0], "circuit_backward": phase_ms[1],
                         "logit_gradient": phase_ms[2], "plain_gemms": phase_ms[3]},
            "flops_per_call": flops, "achieved_tflops": tf, "frac_of_sustained_peak": tf / peaks["bf16_tflops_sustained"],
            "device_status": dh.head.mtpc_get_status()}


def measure_lowrank(torch, wl, dW_emit, steps: int, peaks, k: int = 16):
    """Shared unembeddings with rank-k adaptors (App. G) on the workload's head shape: the composition
    U_ij = W_i + A_ij B_ij and the gradient carried back from dW_emit, each against one pass over its tensors in HBM."""
    from paper_2511_11346_b200.runner import lowrank_backward, lowrank_compose, to_device_bf16
    s = wl.shape
    Wb, A, Bm = I.lowrank_parameters(s.n, s.r, s.v, s.d, k, seed=97)
    Wb, A, Bm = to_device_bf16(Wb), to_device_bf16(A), to_device_bf16(Bm)
    units = s.n * s.r
    nU = units * s.v * s.d
    small = s.n * s.v * s.d + units * s.v * k + units * k * s.d

    def timed(call):
        for _ in range(3):
            call()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            call()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / steps

    ms_c = timed(lambda: lowrank_compose(Wb, A, Bm))
    ms_b = timed(lambda: lowrank_backward(A, Bm, dW_emit))
    bytes_c = 2 * nU + 2 * small                       # write U (bf16), read W, A, B once
    bytes_b = 4 * nU + 2 * small + 4 * small            # read dW_emit (fp32) once, read A, B, write the three gradients
    hbm = peaks["hbm_gbs"]
    out = {"rank": k, "compose_ms": ms_c, "compose_algorithmic_bytes": bytes_c,
           "compose_frac_of_hbm": bytes_c / (ms_c * 1e-3) / 1e9 / hbm, "backward_ms": ms_b, "backward_kernels": 3,
           "backward_algorithmic_bytes": bytes_b, "backward_frac_of_hbm": bytes_b / (ms_b * 1e-3) / 1e9 / hbm,
           "note": "CUDA-core kernels: k multiply-adds per element keep the fp32 pipes, not HBM, busiest; the three "
                   "gradient kernels each stream dW_emit once"}
    if wl.shape.io_dtype == I.BF16 and s.v % 16 == 0:
        out["factored_forward"] = measure_factored_forward(torch, wl, (Wb, A, Bm), steps)
        out["factored_draft"] = measure_factored_draft(torch, wl, (Wb, A, Bm), peaks)
        out["factored_backward"] = measure_factored_backward(torch, wl, (Wb, A, Bm), steps)
    return out


def measure_factored_backward(torch, wl, lowrank, steps: int):
    """mtpc_lowrank_window_logprob_backward: the training call of a head that keeps the shared unembeddings factored
    (value + gradients with respect to the hidden states, W_base, A, B and the sum-unit weights), per call and per phase."""
    from paper_2511_11346_b200 import binding as B
    from paper_2511_11346_b200.runner import to_device_bf16
    s = wl.shape
    k = lowrank[1].shape[-1]
    ctx = s.family == I.HMM_CTX
    W_sum = to_device_bf16(wl.W_sum_q)
    Ts = torch.from_numpy(np.ascontiguousarray(wl.T_static)).cuda() if wl.T_static is not None else None
    head = B.MtpcHead(B.MTPC_HMM if ctx else s.family, s.n, s.r, s.v, s.d, B.MTPC_BF16, wl.T, 1, None, W_sum, Ts,
                      flags=B.MTPC_FLAG_HMM_CONTEXTUAL if ctx else 0, v_valid=s.v_valid, lowrank=lowrank)
    hidden = to_device_bf16(wl.hidden_q)
    targets = torch.from_numpy(wl.targets).cuda()
    f32 = dict(dtype=torch.float32, device="cuda")
    weight = torch.full((wl.T,), -1.0 / wl.T, **f32)
    out = [torch.empty(wl.T, **f32), torch.empty((wl.T, s.d), **f32), torch.empty((s.n, s.v, s.d), **f32),
           torch.empty((s.n, s.r, s.v, k), **f32), torch.empty((s.n, s.r, k, s.d), **f32), torch.empty((s.sum_rows, s.d), **f32),
           torch.empty((max(s.n - 1, 1), s.r, s.r), **f32) if s.family == I.HMM else None]
    call = lambda: head.mtpc_lowrank_window_logprob_backward(hidden, targets, weight, *out)
    for _ in range(3):
        call()
    torch.cuda.synchronize()
    fwd = torch.empty(wl.T, **f32)
    head.mtpc_window_logprob(hidden, targets, fwd)
    same_value = bool(torch.equal(fwd, out[0]))
    head.mtpc_set_timing(steps)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        call()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    phases = [head.mtpc_get_timing(i) for i in range(steps)]
    phase_ms = [statistics.mean(p[q] for p in phases) for q in range(len(phases[0]))]
    head.mtpc_set_timing(0)
    # the paper's training loss (Eq. 6): sequences of 1024 positions, windows past the end of a sequence masked
    L = 1024 if wl.T % 1024 == 0 else wl.T
    N = wl.T // L
    t6 = targets.clone().view(N, L, s.n)
    for j in range(1, s.n):
        t6[:, L - j:, j] = -1
    t6 = t6.view(wl.T, s.n).contiguous()
    gamma = 0.8 if s.n <= 8 else 0.9
    slot, loss = torch.empty(s.n, **f32), torch.empty(1, **f32)
    call6 = lambda: head.mtpc_lowrank_window_loss_backward(hidden, t6, N, L, gamma, slot, loss, *out[1:])
    for _ in range(3):
        call6()
    torch.cuda.synchronize()
    e0.record()
    for _ in range(steps):
        call6()
    e1.record()
    torch.cuda.synchronize()
    ms6 = e0.elapsed_time(e1) / steps
    status = head.mtpc_get_status()
    head.mtpc_destroy()
    return {"call": "mtpc_lowrank_window_logprob_backward", "ms_per_call": ms, "phase_ms": phase_ms,
            "eq6_call": "mtpc_lowrank_window_loss_backward", "eq6_ms_per_call": ms6, "eq6_loss": float(loss.cpu()[0]),
            "phases": "factored forward keeping the logits, circuit backward, logit gradients + their sums + operand "
                      "copies, GEMMs (g A, d hidden, dW_base, dB, dW_sum, dA)",
            "value_equals_forward_call": same_value, "device_status": status,
            "note": "the route through the composed tensor costs compose_ms + the dense backward call + backward_ms"}


def measure_factored_draft(torch, wl, lowrank, peaks, P: int = 8, wpp: int = 16, calls: int = 200):
    """mtpc_draft_sample for a few positions on a head that keeps the shared unembeddings factored: the weight pass streams
    W_base and B (and the sum-unit weights) instead of the composed tensor, so "one pass over the weights" is
    2 d (n v + n r k + sum rows) + 2 n r v k bytes."""
    from paper_2511_11346_b200 import binding as B
    from paper_2511_11346_b200.runner import to_device_bf16
    s = wl.shape
    k = lowrank[1].shape[-1]
    ctx = s.family == I.HMM_CTX
    W_sum = to_device_bf16(wl.W_sum_q)
    Ts = torch.from_numpy(np.ascontiguousarray(wl.T_static)).cuda() if wl.T_static is not None else None
    head = B.MtpcHead(B.MTPC_HMM if ctx else s.family, s.n, s.r, s.v, s.d, B.MTPC_BF16, P, wpp, None, W_sum, Ts,
                      flags=B.MTPC_FLAG_HMM_CONTEXTUAL if ctx else 0, v_valid=s.v_valid, lowrank=lowrank)
    hidden = to_device_bf16(np.ascontiguousarray(wl.hidden_q[:P]))
    W = P * wpp
    u = torch.from_numpy(I.uniforms(I.BASE_SEED + 91, 7, (W, 2 * s.n))).cuda()
    ob = torch.empty((W, s.n), dtype=torch.int32, device="cuda")
    ol = torch.empty(W, dtype=torch.float32, device="cuda")
    for _ in range(5):
        head.mtpc_draft_sample(hidden, wpp, u, ob, ol)
    torch.cuda.synchronize()
    lat = []
    for _ in range(calls):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        head.mtpc_draft_sample(hidden, wpp, u, ob, ol)
        e1.record()
        e1.synchronize()
        lat.append(e0.elapsed_time(e1))
    ref_b = ob.clone()
    graph_lat = graph_replay_times(torch, lambda st: head.mtpc_draft_sample(hidden, wpp, u, ob, ol, stream=st), (ob, ol), calls, 5)
    identical = bool((ob == ref_b).all())
    status = head.mtpc_get_status()
    head.mtpc_destroy()
    # the whole batch of the workload, one window per position
    big = B.MtpcHead(B.MTPC_HMM if ctx else s.family, s.n, s.r, s.v, s.d, B.MTPC_BF16, wl.T, 1, None, W_sum, Ts,
                     flags=B.MTPC_FLAG_HMM_CONTEXTUAL if ctx else 0, v_valid=s.v_valid, lowrank=lowrank)
    hid_all = to_device_bf16(wl.hidden_q)
    u_all = torch.from_numpy(I.uniforms(I.BASE_SEED + 92, 7, (wl.T, 2 * s.n))).cuda()
    ob_all = torch.empty((wl.T, s.n), dtype=torch.int32, device="cuda")
    ol_all = torch.empty(wl.T, dtype=torch.float32, device="cuda")
    for _ in range(2):
        big.mtpc_draft_sample(hid_all, 1, u_all, ob_all, ol_all)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(5):
        big.mtpc_draft_sample(hid_all, 1, u_all, ob_all, ol_all)
    e1.record()
    torch.cuda.synchronize()
    whole_ms = e0.elapsed_time(e1) / 5
    # draft (with prefix marginals) + acceptance stage against synthetic target-model rows, whole batch
    tp_all = torch.from_numpy(I.target_rows(I.BASE_SEED + 93, 9, (wl.T, s.n + 1, s.v))).cuda()
    ua_all = torch.from_numpy(I.uniforms(I.BASE_SEED + 94, 10, (wl.T, s.n + 1))).cuda()
    pre_all = torch.empty((wl.T, s.n), dtype=torch.float32, device="cuda")
    acc_all = torch.empty(wl.T, dtype=torch.int32, device="cuda")
    nxt_all = torch.empty(wl.T, dtype=torch.int32, device="cuda")

    def cycle():
        big.mtpc_draft_sample_prefix(hid_all, 1, u_all, ob_all, pre_all)
        big.mtpc_speculative_accept(wl.T, 1, ob_all, pre_all, tp_all, ua_all, acc_all, nxt_all)
    for _ in range(2):
        cycle()
    torch.cuda.synchronize()
    e0.record()
    for _ in range(5):
        cycle()
    e1.record()
    torch.cuda.synchronize()
    cycle_ms = e0.elapsed_time(e1) / 5
    status |= big.mtpc_get_status()
    big.mtpc_destroy()
    p50, g50 = statistics.median(lat), statistics.median(graph_lat)
    weight_bytes = 2 * s.d * (s.n * s.v + s.n * s.r * k + s.sum_rows) + 2 * s.n * s.r * s.v * k
    dense_bytes = 2 * s.d * (s.n * s.r * s.v + s.sum_rows)
    return {"call": f"mtpc_draft_sample on a factored head, P={P} wpp={wpp}", "p50_ms": p50, "cuda_graph_replay_p50_ms": g50,
            "graph_results_identical": identical, "windows_per_s": W / (p50 * 1e-3), "kernels_per_call": 4,
            "weight_bytes": weight_bytes, "dense_weight_bytes": dense_bytes,
            "hbm_frac": weight_bytes / (g50 * 1e-3) / 1e9 / peaks["hbm_gbs"], "device_status": status,
            "whole_batch": {"windows": wl.T, "ms_per_call": whole_ms, "windows_per_s": wl.T / (whole_ms * 1e-3),
                            "draft_plus_accept_ms": cycle_ms,
                            "note": "mtpc_draft_sample over all positions of the workload, one window each: log omega, latent draws, one unit's "
                                    "logits per (window, slot) from W_base h and B h, evidence by the factored projection, circuit"},
            "note": "weight pass (W_base, B, sum units) + logits from the two small products + per-slot kernel + circuit; "
                    "at these sizes the call is a chain of four short kernels, not a bandwidth problem"}


def measure_factored_forward(torch, wl, lowrank, steps: int):
    """mtpc_window_logprob on a head that keeps the shared unembeddings factored (no composed tensor): time per call, the
    projection phase alone, and its own (smaller) FLOP count 2 d (n v + n r k) + 4 n r v k per position."""
    from paper_2511_11346_b200 import binding as B
    from paper_2511_11346_b200.runner import to_device_bf16
    s = wl.shape
    k = lowrank[1].shape[-1]
    ctx = s.family == I.HMM_CTX
    W_sum = to_device_bf16(wl.W_sum_q)
    Ts = torch.from_numpy(np.ascontiguousarray(wl.T_static)).cuda() if wl.T_static is not None else None
    head = B.MtpcHead(B.MTPC_HMM if ctx else s.family, s.n, s.r, s.v, s.d, B.MTPC_BF16, wl.T, 1, None, W_sum, Ts,
                      flags=B.MTPC_FLAG_HMM_CONTEXTUAL if ctx else 0, v_valid=s.v_valid, lowrank=lowrank)
    hidden = to_device_bf16(wl.hidden_q)
    targets = torch.from_numpy(wl.targets).cuda()
    out = torch.empty(wl.T, dtype=torch.float32, device="cuda")
    for _ in range(3):
        head.mtpc_window_logprob(hidden, targets, out)
    torch.cuda.synchronize()
    head.mtpc_set_timing(steps)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        head.mtpc_window_logprob(hidden, targets, out)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    phases = [head.mtpc_get_timing(i) for i in range(steps)]
    proj_ms = statistics.mean(p[0] for p in phases)
    head.mtpc_set_timing(0)
    status = head.mtpc_get_status()
    head.mtpc_destroy()
    flops = (2.0 * s.d * (s.n * s.symbols + s.n * s.r * k + s.sum_rows) + 4.0 * s.n * s.r * s.symbols * k) * wl.T
    return {"call": "mtpc_window_logprob on a factored head", "ms_per_call": ms, "projection_phase_ms": proj_ms,
            "positions_per_s": wl.T / (ms * 1e-3), "flops_per_call": flops, "achieved_tflops": flops / (proj_ms * 1e-3) / 1e12,
            "dense_flops_per_call": algorithmic_flops(wl), "device_status": status,
            "note": "projection phase = sum-unit tiles + z = B h (a plain GEMM that writes z as two bf16 halves) + factored kernel; the softmax over "
                    "n r v logits per position is the same as in the dense head and now dominates"}


def measure_eq6_step(torch, dh, wl, hidden, targets, grads, steps: int):
    """The paper's training loss (Eq. 6, discount 0.8, or 0.9 for n > 8) and its gradients in one call: sequences of 1024
    positions, windows that run past the end of their sequence masked."""
    s = wl.shape
    L = 1024 if wl.T % 1024 == 0 else wl.T
    N = wl.T // L
    t = targets.clone().view(N, L, s.n)
    for j in range(1, s.n):
        t[:, L - j:, j] = -1
    t = t.view(wl.T, s.n).contiguous()
    gamma = 0.9 if s.n > 8 else 0.8
    f32 = dict(dtype=torch.float32, device="cuda")
    slot, loss = torch.empty(s.n, **f32), torch.empty(1, **f32)
    call = lambda: dh.head.mtpc_window_loss_backward(hidden, t, N, L, gamma, slot, loss, *grads[1:])
    for _ in range(3):
        call()
    torch.cuda.synchronize()
    dh.head.mtpc_set_timing(steps)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        call()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    phases = [dh.head.mtpc_get_timing(i) for i in range(steps)]
    phase_ms = [statistics.mean(p[k] for p in phases) for k in range(len(phases[0]))]
    dh.head.mtpc_set_timing(0)
    return {"call": "mtpc_window_loss_backward", "sequences": N, "sequence_length": L, "gamma": gamma, "ms_per_call": ms,
            "positions_per_s": wl.T / (ms * 1e-3), "loss": float(loss.cpu()[0]),
            "phase_ms": {"forward_prefix_loss": phase_ms[0], "circuit_backward_passes": phase_ms[1],
                         "logit_gradient": phase_ms[2], "plain_gemms": phase_ms[3]}}


CIRCUIT_KERNEL = {I.CP: "circuit_cp_kernel", I.HMM: "circuit_hmm_stream_kernel", I.BTREE: "circuit_btree_kernel",
                  I.HMM_CTX: "circuit_hmm_stream_kernel (per-position tables)"}


def config_block(idx: int, wl, world: int) -> dict:
    """The `config` object of the JSON line; the same for this arm and for the reference arm."""
    s = wl.shape
    in_bytes = ((s.n * s.r * s.v + s.sum_rows) * s.d + wl.T * s.d) * 2
    return {"workload": workload_name(idx, wl), "parallelism": f"replicas x{world} (no collective)",
            "l2": f"inputs larger than L2: {in_bytes / 1e6:.0f} MB of weights and hidden states per step against 126 MB, "
                  "no flush between steps",
            "step": "one mtpc_window_logprob call: projection GEMM + fused epilogue, then circuit evaluation"}


def timed_logprob_loop(torch, head, hidden, targets, out, steps: int, dev_index: int, sync_ranks: bool = False):
    """`steps` back-to-back mtpc_window_logprob calls between two CUDA events on the launching stream, the SM clock
    sampled meanwhile; per-kernel means from the library's event ring (recorded on the same stream in the same loop)."""
    kept = min(steps, 4096)
    head.mtpc_set_timing(kept)
    launches0 = head.mtpc_launch_count()
    sampler = ClockSampler(dev_index)
    stream = torch.cuda.current_stream()
    if sync_ranks:
        replicas.barrier()
    torch.cuda.synchronize()
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(steps):
        head.mtpc_window_logprob(hidden, targets, out)
    e1.record(stream)
    torch.cuda.synchronize()
    clocks = sampler.stop()
    if sync_ranks:
        replicas.barrier()
    elapsed_s = e0.elapsed_time(e1) * 1e-3
    phases = [head.mtpc_get_timing(i) for i in range(kept)]
    head.mtpc_set_timing(0)
    return {"elapsed_s": elapsed_s, "steps": steps, "gemm_ms": statistics.mean(p[0] for p in phases),
            "circuit_ms": statistics.mean(p[1] for p in phases), "clocks": clocks, "timed_launches": kept,
            "launches": head.mtpc_launch_count() - launches0}


def tensor_roofline(flops: float, loop: dict, peaks: dict, peak_src: str) -> dict:
    """Projection kernel against the measured cuBLAS bf16 peak that matches the loop it was timed in: the burst figure
    for a loop shorter than BURST_REGION_S (boost clocks), the sustained one for a longer, power-capped loop."""
    achieved = flops / (loop["gemm_ms"] * 1e-3) / 1e12
    burst = loop["elapsed_s"] < BURST_REGION_S
    key = "bf16_tflops" if burst else "bf16_tflops_sustained"
    peak = peaks[key]
    c = loop["clocks"]
    return {"achieved": achieved, "peak": peak, "frac": achieved / peak,
            "peak_source": f"{peak_src}: {key} ({'burst' if burst else 'sustained'} figure: the kernel was timed inside a "
                           f"{loop['elapsed_s']:.3f} s loop of {loop['steps']} back-to-back steps)",
            "avg_launch_ms": loop["gemm_ms"], "timed_launches": loop["timed_launches"], "loop_s": loop["elapsed_s"],
            "sm_mhz_median": c["sm_mhz"], "clock_samples": c["samples"], "reasons": c["reasons"]}


def sustained_steps(ms_per_step: float) -> int:
    return int(max(20, min(4096, SUSTAINED_LOOP_S / (ms_per_step * 1e-3))))


def circuit_roofline(wl, circuit_ms: float, peaks: dict) -> dict:
    cbytes = circuit_bytes(wl)
    gbs = cbytes / (circuit_ms * 1e-3) / 1e9
    return {"kernel": CIRCUIT_KERNEL[wl.shape.family], "avg_ms": circuit_ms, "bound": "hbm", "algorithmic_bytes": cbytes,
            "achieved_gbs": gbs, "peak_gbs": peaks["hbm_gbs"], "frac": gbs / peaks["hbm_gbs"]}


def oracle_parity(wl, out, k: int = 256) -> dict:
    """The timed launches' own output against the fp64 oracle on the first k positions."""
    from oracle import mtpc_oracle as orc
    k = min(wl.T, k)
    ref = orc.window_logprob(wl.shape.family, wl.hidden_q[:k], wl.W_emit_q, wl.W_sum_q, wl.T_static, wl.targets[:k])
    return {"positions": k, "tolerance": 2e-3,
            "max_abs_err": float(np.abs(out[:k].cpu().numpy().astype(np.float64) - ref).max())}


def measure_draft_whole_batch(torch, head, wl, hidden, steps: int) -> dict:
    """configs[3]: draft one window per position over the whole batch (the many-position path)."""
    s = wl.shape
    u = torch.from_numpy(wl.uniforms).cuda()
    W = wl.T * wl.wpp
    ob = torch.empty((W, s.n), dtype=torch.int32, device="cuda")
    ol = torch.empty(W, dtype=torch.float32, device="cuda")
    for _ in range(3):
        head.mtpc_draft_sample(hidden, wl.wpp, u, ob, ol)
    torch.cuda.synchronize()
    head.mtpc_set_timing(steps)
    d0, d1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    d0.record()
    for _ in range(steps):
        head.mtpc_draft_sample(hidden, wl.wpp, u, ob, ol)
    d1.record()
    torch.cuda.synchronize()
    dms = d0.elapsed_time(d1) / steps
    dph = [head.mtpc_get_timing(i) for i in range(steps)]
    head.mtpc_set_timing(0)
    res = {"call": "mtpc_draft_sample over the whole batch", "windows": W, "ms_per_call": dms,
           "windows_per_s": W / (dms * 1e-3),
           "phase_ms": [statistics.mean(p[k] for p in dph) for k in range(len(dph[0]))],
           "phases": "sum-unit GEMM, latent draws, byte draws (sorted by unit: sort + staging + GEMM), GEMM + gather "
                     "epilogue on the drafted bytes, circuit"}
    # draft with prefix marginals + acceptance stage (Algorithm 3) on the whole batch, synthetic target-model rows
    tp = torch.from_numpy(I.target_rows(I.BASE_SEED + 77, 9, (W, s.n + 1, s.v))).cuda()
    ua = torch.from_numpy(I.uniforms(I.BASE_SEED + 78, 10, (W, s.n + 1))).cuda()
    opre = torch.empty((W, s.n), dtype=torch.float32, device="cuda")
    oacc = torch.empty(W, dtype=torch.int32, device="cuda")
    onxt = torch.empty(W, dtype=torch.int32, device="cuda")
    cyc = []
    for it in range(3 + steps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        head.mtpc_draft_sample_prefix(hidden, wl.wpp, u, ob, opre)
        head.mtpc_speculative_accept(wl.T, wl.wpp, ob, opre, tp, ua, oacc, onxt)
        e1.record()
        e1.synchronize()
        if it >= 3:
            cyc.append(e0.elapsed_time(e1))
    res["draft_plus_accept"] = {"ms_per_cycle": statistics.median(cyc),
                                "mean_accepted_bytes_vs_synthetic_target": float(oacc.float().mean().cpu()),
                                "calls": "mtpc_draft_sample_prefix + mtpc_speculative_accept"}
    res["device_status"] = head.mtpc_get_status()
    return res


def measure_other_workload(torch, idx: int, dev_index: int, peaks: dict, peak_src: str, with_oracle: bool,
                           steps: int = 20) -> dict:
    """configs[2] / configs[3] measured like the headline workload: a burst loop of `steps` calls after five warm-up
    calls (the headline's --steps: a 60-call loop already runs into the power cap, 1.5 GHz against 1.97 for 20 calls,
    and would be compared with a peak taken at full clock), a seconds-long sustained loop, the circuit kernel against HBM
    and the parity of the timed output."""
    from paper_2511_11346_b200.runner import DeviceHead
    wl = I.config_workload(idx)
    dh = DeviceHead(wl)
    head = dh.head
    hidden = dh.hidden_device()
    targets = torch.from_numpy(wl.targets).cuda()
    out = torch.empty(wl.T, dtype=torch.float32, device="cuda")
    for _ in range(5):
        head.mtpc_window_logprob(hidden, targets, out)
    torch.cuda.synchronize()
    flops = algorithmic_flops(wl)
    burst = timed_logprob_loop(torch, head, hidden, targets, out, steps, dev_index)
    ms = burst["elapsed_s"] / burst["steps"] * 1e3
    sus = timed_logprob_loop(torch, head, hidden, targets, out, sustained_steps(ms), dev_index)
    res = {"workload": workload_name(idx, wl), "positions_per_s": wl.T * burst["steps"] / burst["elapsed_s"],
           "ms_per_step": ms, "steps": burst["steps"],
           "positions_per_s_sustained": wl.T * sus["steps"] / sus["elapsed_s"],
           "roofline": dict(bound="tensor", kernel="mtpc_gemm_kernel<logprob>", unit="TFLOP/s", flops_per_launch=flops,
                            traffic=NCU_TRAFFIC_BYTES.get(idx), **tensor_roofline(flops, burst, peaks, peak_src)),
           "roofline_sustained": tensor_roofline(flops, sus, peaks, peak_src),
           "circuit_kernel": circuit_roofline(wl, burst["circuit_ms"], peaks),
           "device_status": head.mtpc_get_status()}
    if with_oracle:
        res["parity"] = oracle_parity(wl, out)
    if wl.wpp:
        res["draft_whole_batch"] = measure_draft_whole_batch(torch, head, wl, hidden, 20)
    res["gpu_launches"] = int(burst["launches"] + sus["launches"])
    dh.close()
    del dh, hidden, targets, out
    torch.cuda.empty_cache()
    return res


def run_ours(args):
    import torch
    from paper_2511_11346_b200.runner import DeviceHead

    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the MtPC head has no CPU path (use --impl reference for the oracle)")
    rank, local_rank, world = replicas.rank_env()
    torch.cuda.set_device(local_rank if world > 1 else 0)
    replicas.init_process_group("nccl")
    dev_index = torch.cuda.current_device()

    wl = I.config_workload(args.workload, T=args.positions)
    s = wl.shape
    dh = DeviceHead(wl)
    head = dh.head
    hidden = dh.hidden_device()
    targets = torch.from_numpy(wl.targets).cuda()
    out = torch.empty(wl.T, dtype=torch.float32, device="cuda")

    # ---------------- device-resident throughput: K steps back to back, per-kernel events kept by the library
    for _ in range(args.warmup):
        head.mtpc_window_logprob(hidden, targets, out)
    torch.cuda.synchronize()
    main = timed_logprob_loop(torch, head, hidden, targets, out, args.steps, dev_index, sync_ranks=True)
    elapsed_s = replicas.max_over_ranks(main["elapsed_s"], device="cuda")
    main["elapsed_s"] = elapsed_s
    status = head.mtpc_get_status()
    value = replicas.aggregate_throughput(wl.T, args.steps, world, elapsed_s)
    gemm_ms, circuit_ms = main["gemm_ms"], main["circuit_ms"]

    # ---------------- the same call in a loop long enough to sit under the power cap (sustained clocks)
    sus = None
    if not args.no_sustained:
        sus = timed_logprob_loop(torch, head, hidden, targets, out, sustained_steps(elapsed_s / args.steps * 1e3), dev_index,
                                 sync_ranks=True)
    out_main = out.clone()

    # ---------------- end to end through the host-buffer entry point (pinned host memory, copies timed)
    hh = dh.hidden_host()
    th = torch.from_numpy(wl.targets).pin_memory()
    oh = torch.empty(wl.T, dtype=torch.float32).pin_memory()
    e2e_steps = max(3, min(args.steps, 50))
    for _ in range(3):
        head.mtpc_window_logprob_host(hh, th, oh)
    replicas.barrier()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        head.mtpc_window_logprob_host(hh, th, oh)      # returns after the result is in host memory
    torch.cuda.synchronize()
    e2e_s = replicas.max_over_ranks(time.perf_counter() - t0, device="cuda")
    e2e_value = replicas.aggregate_throughput(wl.T, e2e_steps, world, e2e_s)
    h2d = hh.numel() * hh.element_size() + th.numel() * 4
    d2h = oh.numel() * 4

    if rank != 0:
        return

    peaks, peak_src = load_peaks()
    flops = algorithmic_flops(wl)
    roofline = dict(bound="tensor", kernel="mtpc_gemm_kernel<logprob>", unit="TFLOP/s", flops_per_launch=flops,
                    traffic=NCU_TRAFFIC_BYTES.get(args.workload), **tensor_roofline(flops, main, peaks, peak_src))
    roofline["frac_of_burst_peak"] = roofline["achieved"] / peaks["bf16_tflops"]
    roofline["frac_of_sustained_peak"] = roofline["achieved"] / peaks["bf16_tflops_sustained"]
    roofline["circuit_kernel_avg_ms"] = circuit_ms
    if sus is not None:
        roofline["sustained"] = tensor_roofline(flops, sus, peaks, peak_src)
        roofline["sustained"]["positions_per_s"] = wl.T * sus["steps"] / sus["elapsed_s"]
    achieved = roofline["achieved"]
    ck = circuit_roofline(wl, circuit_ms, peaks)
    ck["share_of_step"] = circuit_ms / (gemm_ms + circuit_ms)
    kernels = [
        {"kernel": "mtpc_gemm_kernel<logprob>", "avg_ms": gemm_ms, "bound": "tensor", "achieved_tflops": achieved,
         "frac": roofline["frac"], "share_of_step": gemm_ms / (gemm_ms + circuit_ms)},
        ck,
    ]

    # CPU baseline: the oracle as it stands on a bounded sample of the same workload
    cpu_baseline = None
    parity = None
    with_oracle = not args.no_cpu_baseline and world == 1          # rank 0 of a single-GPU run only
    if with_oracle:
        if args.ref_positions:
            sample = min(wl.T, args.ref_positions)
        else:                                                                # about 15 s of CPU work, sized by a short probe
            probe_rate, _ = oracle_positions_per_s(wl, min(wl.T, 256))
            sample = int(min(wl.T, max(256, (probe_rate * 15.0) // 256 * 256)))
        cpu_value, cpu_s = oracle_positions_per_s(wl, sample)
        cpu_baseline = {"value": cpu_value, "unit": UNIT, "cores": host_threads(), "kind": "oracle",
                        "sample": f"first {sample} of {wl.T} positions, one pass, {cpu_s:.1f} s"}
        # the timed launches' own output (device path and host-buffer path) against the oracle on the first positions
        parity = oracle_parity(wl, out_main)
        parity["max_abs_err_device_call"] = parity.pop("max_abs_err")
        parity["max_abs_err_host_call"] = oracle_parity(wl, oh)["max_abs_err"]

    backward = None
    if args.backward and world == 1:
        backward = measure_backward(torch, dh, wl, hidden, targets, steps=max(5, min(args.steps, 30)), peaks=peaks)

    draft_many = None
    if wl.wpp and world == 1:       # configs[3]: draft one window per position over the whole batch (many-position path)
        draft_many = measure_draft_whole_batch(torch, head, wl, hidden, max(3, min(args.steps, 30)))

    launches = main["launches"] + (sus["launches"] if sus else 0)
    dh.close()
    del dh, hidden, targets, out
    torch.cuda.empty_cache()

    # ---------------- the other heads the throughput target names (default run: configs[2] and configs[3])
    others = []
    if world == 1 and args.workload == 1 and args.positions is None and not args.no_other_workloads:
        for idx in (2, 3):
            others.append(measure_other_workload(torch, idx, dev_index, peaks, peak_src, with_oracle, steps=args.steps))
            launches += others[-1]["gpu_launches"]

    draft, sweep = None, None
    if not args.no_draft and world == 1:
        if args.decode_cells == "all":
            cells = I.DECODE_CELLS
        elif args.decode_cells == "one":
            cells = [(I.CP, 8, 64)]
        else:                                   # "cp:8:64", "hmm:16:1", ...
            fam, n_, p_ = args.decode_cells.split(":")
            cells = [({"cp": I.CP, "hmm": I.HMM}[fam], int(n_), int(p_))]
        sweep = []
        for cell in cells:
            res, cell_launches = measure_decode_cell(torch, cell, steps=200, warmup=5, with_graph=not args.no_graph)
            sweep.append(res)
            launches += cell_launches
        draft = next((c for c in sweep if "decode_cp_n8_P64" in c["workload"]), sweep[0])

    c = main["clocks"]
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": elapsed_s / args.steps * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": config_block(args.workload, wl, world),
        "clocks": {"sm_mhz": c["sm_mhz"], "sm_max_mhz": c["sm_max_mhz"], "reasons": c["reasons"], "samples": c["samples"],
                   "region": f"the {args.steps} timed steps ({elapsed_s * 1e3:.1f} ms); the sustained loop has its own record "
                             "under roofline.sustained"},
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": e2e_steps, "ms_per_step": e2e_s / e2e_steps * 1e3,
                "call": "mtpc_window_logprob_host (pinned host buffers, copies inside the call)"},
        "gpu_launches": int(main["launches"]),
        "gpu_launches_all_loops": int(launches),
        "roofline": roofline,
        "kernels": kernels,
        "cpu_baseline": cpu_baseline,
        "parity": parity,
        "device_status": status,
    }
    if others:
        line["workloads"] = others
    if backward is not None:
        line["backward"] = backward
    if draft_many is not None:
        line["draft_whole_batch"] = draft_many
    if draft is not None:
        line["draft"] = draft
        line["decode_sweep"] = sweep
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", type=int, default=1, choices=[1, 2, 3, 5, 6],
                    help="1 CP (the metric's configuration), 2 HMM, 3 binary tree, 5 HMM with contextual transitions, "
                         "6 CP with the byte-level Llama shape (d=3072, 268 symbols padded to 272)")
    ap.add_argument("--ref-positions", type=int, default=None,
                    help="positions the CPU oracle processes per step (reference arm: default 1024) or for the "
                         "cpu_baseline sample (default: sized to about 15 s by a short probe)")
    ap.add_argument("--no-draft", action="store_true", help="skip the decode-cell draft measurement")
    ap.add_argument("--decode-cells", default="all",
                    help="draft measurement: 'all' twelve cells of the decode sweep, 'one' (CP n=8 P=64), or a single "
                         "cell as family:n:P, e.g. hmm:16:1")
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip timing the CPU oracle (profiling runs)")
    ap.add_argument("--no-graph", action="store_true", help="skip the CUDA-graph replay of the draft calls (profiling runs)")
    ap.add_argument("--no-sustained", action="store_true", help="skip the second, seconds-long loop (profiling runs)")
    ap.add_argument("--no-other-workloads", action="store_true",
                    help="default run only: skip configs[2] and configs[3] after the headline workload")
    ap.add_argument("--backward", action="store_true", help="also time mtpc_window_logprob_backward on the workload")
    ap.add_argument("--positions", type=int, default=None,
                    help="override the number of positions (scaled-down profiler captures; not a bench value)")
    args = ap.parse_args()
    if args.impl == "reference":
        args.steps = 3 if args.steps is None else args.steps
        args.warmup = 1 if args.warmup is None else args.warmup
        args.ref_positions = args.ref_positions or 1024
        run_reference(args)
    else:
        args.steps = 400 if args.steps is None else args.steps
        args.warmup = max(3, 5 if args.warmup is None else args.warmup)
        run_ours(args)


if __name__ == "__main__":
    main()
