#!/usr/bin/env python
"""Benchmark of the CAMERA analysis hot path on B200.

One step = one MoE layer analysed end to end: camera_score_layer (router, permutation, W_down
norms, fused gate/up scoring, energy), then the prune masks at 20/40/60 % and the bit-widths of a 2.25-bit budget
(camera_select_all: the results of camera_select_prune x 3 and camera_alloc_bits from one set of radix passes), on
synthetic calibration tokens of the Qwen2-57B-A14B layer shape.

    python bench.py --gpus N --steps K --warmup W            (N > 1: launched by torch.distributed.run)
    python bench.py --impl reference ...                      (the float64 CPU oracle on a bounded sample)

Prints one JSON line.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "micro-expert scoring tokens/s per MoE layer"
UNIT = "tokens/s"
PRUNE_RATIOS = (0.2, 0.4, 0.6)
BIT_RATIOS, BIT_LEVELS = (0.2, 0.6, 0.2), (3, 2, 1)     # average 2 bits + 0.25 group overhead
ALPHA = 0.95
PAPER_CONTEXT = "paper: <5 min for the full Qwen2-57B-A14B analysis on one A100-40GB (incl. model forwards)"
# kernels launched by one step: score = router, block scan, plan, permute, pad, norms, scoring, combine;
# the selections = one kernel (radix passes, tie break and labels behind one cooperative launch)
LAUNCHES_PER_STEP = 8 + 1
# DRAM bytes (read + write) of one launch of the scoring kernel on the full Qwen2-57B-A14B-shaped layer (262144 tokens,
# single pass): the one-pass ncu capture of profiles/k_score_umma_pair_qwen2_full_dram.md.
SCORE_KERNEL_DRAM_BYTES_FULL_LAYER = 33036971776 + 344499712


def shard_layers(n_layers: int, world: int, rank: int):
    """Layers of the model a rank analyses when the layers are spread over `world` ranks."""
    return list(range(rank, n_layers, world))


def shard_tokens(n_tokens: int, world: int, rank: int):
    """[t0, t1) of the calibration tokens a rank scores when one layer's tokens are spread over `world` ranks."""
    base, extra = divmod(n_tokens, world)
    t0 = rank * base + min(rank, extra)
    return t0, t0 + base + (1 if rank < extra else 0)


def reduce_components(phi2, phi_inf_sq, dist=None):
    """The one exchange of token-sharded scoring: column sums add over the shards, column maxima take the maximum
    (Algorithm 1's ColumnSum and ColumnMax).  In place; a no-op without a process group."""
    if dist is not None and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(phi2, op=dist.ReduceOp.SUM)
        dist.all_reduce(phi_inf_sq, op=dist.ReduceOp.MAX)
    return phi2, phi_inf_sq


def max_over_ranks(ms: float, dist=None, device="cpu") -> float:
    """Largest per-rank time; a collective only when a process group exists."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return ms
    import torch
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"source": "measured", "hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"])}
    return {"source": "fallback", "hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for l in self.lines:
            f = [x.strip() for x in l.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def blas_threads() -> int:
    """Threads the oracle's numpy BLAS runs on."""
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 0) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return int(max(n))
    except Exception:
        pass
    return len(os.sched_getaffinity(0))


def oracle_prepare(L, X):
    """Widens the stored weights and tokens to float64 for the oracle (not timed)."""
    from oracle import f64, to_oracle_layer
    return to_oracle_layer(L), f64(X)


def oracle_step(ol, Xd):
    """One step of the CPU oracle, as it stands: scores, three prune masks, one bit allocation.  Returns seconds."""
    import oracle as O
    t0 = time.perf_counter()
    E = O.energy(*O.camera_components(ol, Xd), ALPHA)
    for r in PRUNE_RATIOS:
        O.select_prune(E, r)
    O.alloc_bits(E, BIT_RATIOS, BIT_LEVELS)
    return time.perf_counter() - t0


def run_reference(args):
    """--impl reference: the float64 oracle on host cores, bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2508_02322_b200 import workloads as W
    cfg = W.CONFIGS[args.config]
    n_sample = args.oracle_tokens or 512
    L = W.make_layer(cfg, seed=0, layer_id=0, device="cpu")
    X = W.make_tokens(W.scaled(cfg, n_tokens=n_sample), seed=0, layer_id=0, device="cpu")
    ol, Xd = oracle_prepare(L, X)
    for _ in range(args.warmup):
        oracle_step(ol, Xd)
    dt = sum(oracle_step(ol, Xd) for _ in range(args.steps))
    value = n_sample * args.steps / dt
    cores = blas_threads()
    sample = f"first {n_sample} tokens of one {cfg.name} layer, all {cfg.n_micro_experts} micro-experts, per step"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{cfg.name} layer (sample)", "n_tokens": n_sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def run_stack(args):
    """--stack: Algorithm 2's layer loop on a synthetic stack of MoE layers.  Per layer: output of the layer on the
    calibration tokens and scores from one pass over the gate/up weights
    (camera_score_forward_layer; every batch keeps its workspace, so Phi stays in HBM as h), selection and slicing,
    output of the retained micro-experts from the stored h and W_down with the pruned columns zeroed
    (camera_pruned_output: Phi[:,S] W[S,:] of Eq. 7 without a second pass over the gate/up weights),
    which -- added to the residual and rescaled to RMS 1, the stand-in for the rest of a decoder layer --
    becomes the next layer's input ("I <- O").  Prints one JSON line of its own."""
    import torch
    import paper_2508_02322_b200 as P
    from paper_2508_02322_b200 import workloads as W
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(dev)
    cfg = W.CONFIGS[args.config]
    if args.tokens:
        cfg = W.scaled(cfg, n_tokens=args.tokens)
    T, d = cfg.n_tokens, cfg.d_model
    n_layers = args.stack_layers or cfg.n_layers
    ratio = PRUNE_RATIOS[1]
    B = min(T, 65536)
    spans = [(t0, min(T, t0 + B)) for t0 in range(0, T, B)]
    X = W.make_tokens(cfg, seed=0, layer_id=0, device=dev)
    Y = torch.empty((T, d), dtype=torch.float32, device=dev)
    Yh = torch.empty_like(Y)
    probe = P.Layer.from_workload(W.make_layer(W.scaled(cfg, n_tokens=B), seed=0, layer_id=0, device=dev))
    n_me = probe.n_me
    ws_f = [P.alloc_workspace(P.camera_forward_workspace_bytes(probe, B), dev) for _ in spans]
    w_masked = [torch.empty_like(w) for w in probe.tensors["w_down"]]
    ws_sel = P.alloc_workspace(P.camera_select_workspace_bytes(n_me, 1, 2), dev)
    ws_c = P.alloc_workspace(int(P.lib.camera_compact_workspace_bytes(probe.n_experts)), dev)
    energy = torch.empty(n_me, dtype=torch.float32, device=dev)
    phi2, phi_inf, omega2 = torch.empty_like(energy), torch.empty_like(energy), torch.empty_like(energy)
    keep = torch.empty(n_me, dtype=torch.uint8, device=dev)
    outw = {k: [torch.empty_like(w) for w in probe.tensors[k]] for k in ("w_gate", "w_up", "w_down")}
    del probe
    stream = torch.cuda.current_stream()
    names = ("forward_and_score", "select_slice", "pruned_output", "error_next_input")
    tot = {k: 0.0 for k in names}
    errors = []
    for l in range(n_layers):
        L = W.make_layer(cfg, seed=0, layer_id=l, device=dev)        # weights of the layer: not timed
        layer = P.Layer.from_workload(L)
        off = P.expert_offsets_tensor(layer)
        torch.cuda.synchronize()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(len(names) + 1)]
        ev[0].record(stream)
        for i, (t0, t1) in enumerate(spans):
            P.camera_score_forward_layer(layer, X[t0:t1], ALPHA, energy=energy, y=Y[t0:t1], workspace=ws_f[i], phi2=phi2,
                                         phi_inf_sq=phi_inf, accumulate=i > 0, omega2=omega2, omega_given=i > 0)
        ev[1].record(stream)
        P.camera_select_prune(energy, ratio, workspace=ws_sel, keep_mask=keep)
        sub, counts = P.camera_sub_index(keep, off, [1])
        P.camera_compact_weights(layer, sub, counts, 1, out=outw, workspace=ws_c)
        ev[2].record(stream)
        P.camera_mask_down_columns(layer, keep, out=w_masked)
        for i, (t0, t1) in enumerate(spans):
            P.camera_pruned_output(layer, w_masked, t1 - t0, ws_f[i], y=Yh[t0:t1])
        ev[3].record(stream)
        err = P.camera_output_error(Y, Yh)
        P.camera_residual_norm(X, Yh, out=X)
        ev[4].record(stream)
        torch.cuda.synchronize()
        if any(P.camera_read_status(w) != 0 for w in ws_f):
            raise RuntimeError("device status set in the stack run")
        for i, k in enumerate(names):
            tot[k] += ev[i].elapsed_time(ev[i + 1])
        e = err.cpu().tolist()
        errors.append(e[0] / e[1] if e[1] > 0 else 0.0)
        del L, layer
    total_s = sum(tot.values()) * 1e-3
    print(json.dumps({
        "mode": "stack", "what": "Algorithm 2 over a synthetic stack of MoE layers (layer outputs, CAMERA scores, prune, slice, "
                                 "retained micro-experts' outputs fed to the next layer)",
        "config": {"workload": f"{cfg.name} x {n_layers} layers", "tokens": T, "prune_ratio": ratio, "alpha": ALPHA},
        "seconds": total_s, "tokens_per_s_per_layer": T * n_layers / total_s,
        "ms_per_layer": {k: v / n_layers for k, v in tot.items()},
        "relative_output_error": {"first_layer": errors[0], "last_layer": errors[-1], "mean": sum(errors) / len(errors)},
        "context": PAPER_CONTEXT}))


def time_steps(P, torch, cfg, layer, Xs, steps, warmup, dev, stream, ws_score, ws_sel, energy, keep, bits, sampler_index,
               cta_pair=None):
    """`steps` whole steps (score + every selection) of one layer after `warmup`, timed with CUDA events on the
    launching stream; the SM clock is sampled meanwhile.  Returns (ms in total, per-stage mean ms, clocks, flushed)."""
    def step(i, events=None):
        P.camera_score_layer(layer, Xs[i % 2], ALPHA, energy=energy, workspace=ws_score, stage_events=events, cta_pair=cta_pair)
        P.camera_select_all(energy, PRUNE_RATIOS, BIT_RATIOS, BIT_LEVELS, workspace=ws_sel, keep_masks=keep, bits_out=bits)
    for i in range(warmup):
        step(i)
    torch.cuda.synchronize()
    status = P.camera_read_status(ws_score)
    if status != 0:
        raise RuntimeError(f"device status {status} after warm-up ({cfg.name})")
    stage_ev = [{s: (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for s in P.binding.STAGES}
                for _ in range(steps)]
    for evs in stage_ev:            # events must exist before their handles are passed down
        for e0, e1 in evs.values():
            e0.record(stream); e1.record(stream)
    # inputs of the large configs exceed the 126 MB L2 several times over; a small config gets its L2 flushed between
    # steps (a 256 MiB write outside the per-step event pairs)
    esz = 2 if cfg.dtype == "bf16" else 4
    footprint = esz * (3 * layer.n_me * cfg.d_model + 2 * cfg.n_tokens * cfg.d_model)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if footprint < (512 << 20) else None
    sampler = ClockSampler(sampler_index)
    torch.cuda.synchronize()
    sampler.start()
    if flush is None:
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record(stream)
        for i in range(steps):
            step(i, stage_ev[i])
        ev1.record(stream)
        torch.cuda.synchronize()
        ms = ev0.elapsed_time(ev1)
    else:
        per_step = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for i in range(steps):
            flush.zero_()
            per_step[i][0].record(stream)
            step(i, stage_ev[i])
            per_step[i][1].record(stream)
        torch.cuda.synchronize()
        ms = sum(e0.elapsed_time(e1) for e0, e1 in per_step)
    clocks = sampler.stop()
    stage_ms = {s: statistics.mean(e[s][0].elapsed_time(e[s][1]) for e in stage_ev) for s in P.binding.STAGES}
    status = P.camera_read_status(ws_score)
    if status != 0:
        raise RuntimeError(f"device status {status} in the timed region ({cfg.name})")
    return ms, stage_ms, clocks, flush is not None


def time_e2e(P, torch, cfg, layer, Xs, n_steps, dev, stream):
    """The same step through camera_analyze_layer_host: pinned host tokens in, host energies / masks / bit-widths out,
    every step.  Returns (ms per step, bytes in per step, bytes out per step)."""
    n_me = layer.n_me
    ws_an = P.alloc_workspace(P.camera_analyze_workspace_bytes(layer, cfg.n_tokens, len(BIT_LEVELS)), dev)
    xh = [x.cpu().pin_memory() for x in Xs]
    eh = torch.empty(n_me, dtype=torch.float32).pin_memory()
    kh = torch.empty((len(PRUNE_RATIOS), n_me), dtype=torch.uint8).pin_memory()
    bh = torch.empty(n_me, dtype=torch.uint8).pin_memory()
    def run(i):
        P.camera_analyze_layer_host(layer, xh[i % 2], ALPHA, PRUNE_RATIOS, BIT_RATIOS, BIT_LEVELS, energy_host=eh,
                                    keep_host=kh, bits_host=bh, workspace=ws_an)
    for i in range(2):
        run(i)
    torch.cuda.synchronize()
    a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a0.record(stream)
    for i in range(n_steps):
        run(i)
    a1.record(stream)
    torch.cuda.synchronize()
    return a0.elapsed_time(a1) / n_steps, xh[0].numel() * xh[0].element_size(), eh.numel() * 4 + kh.numel() + bh.numel()


def bench_other_config(P, torch, W, name, dev, stream, local, peaks):
    """One of the smaller workload configs, measured like the headline one: whole steps with the inputs resident,
    the scoring stage's rate, and the end-to-end step through the host-buffer entry point."""
    cfg = W.CONFIGS[name]
    L = W.make_layer(cfg, seed=0, layer_id=0, device=dev)
    layer = P.Layer.from_workload(L)
    Xs = [W.make_tokens(cfg, seed=0, layer_id=i, device=dev) for i in range(2)]
    n_me, T = layer.n_me, cfg.n_tokens
    ws_score = P.alloc_workspace(P.camera_score_workspace_bytes(layer, T), dev)
    ws_sel = P.alloc_workspace(P.camera_select_workspace_bytes(n_me, 1, len(PRUNE_RATIOS) + len(BIT_LEVELS)), dev)
    energy = torch.empty(n_me, dtype=torch.float32, device=dev)
    keep = torch.empty((len(PRUNE_RATIOS), n_me), dtype=torch.uint8, device=dev)
    bits = torch.empty(n_me, dtype=torch.uint8, device=dev)
    bufs = (ws_score, ws_sel, energy, keep, bits, local)
    ms, _, _, _ = time_steps(P, torch, cfg, layer, Xs, 10, 3, dev, stream, *bufs)
    steps = int(min(2000, max(50, 1500.0 / max(ms / 10, 1e-3))))          # about a second and a half of steps
    ms, stage_ms, clocks, flushed = time_steps(P, torch, cfg, layer, Xs, steps, 3, dev, stream, *bufs)
    del ws_score, bufs
    e2e_ms, h2d, d2h = time_e2e(P, torch, cfg, layer, Xs, min(steps, 200), dev, stream)
    out = {"workload": f"{cfg.name} layer: d_model {cfg.d_model}, {cfg.n_routed}x{cfg.d_ff_routed} top-{cfg.top_k} + shared "
                       f"{list(cfg.d_ff_shared)}, {T} tokens, {cfg.dtype}", "steps": steps, "ms_per_step": ms / steps,
           "tokens_per_s": T * steps / (ms * 1e-3), "stage_ms": stage_ms, "clocks": clocks,
           "l2": "L2 flushed between steps (256 MiB write, not timed)" if flushed else "inputs larger than L2",
           "e2e_tokens_per_s": T / (e2e_ms * 1e-3), "e2e_ms_per_step": e2e_ms, "h2d_bytes_per_step": h2d,
           "d2h_bytes_per_step": d2h}
    if cfg.dtype == "bf16":
        tf = cfg.gate_up_flop / (stage_ms["score"] * 1e-3) / 1e12
        # these runs last a second or two: the burst peak is the denominator
        out.update({"score_tflops": tf, "score_frac_of_burst_peak": tf / peaks["bf16_tflops"], "peak": "measured burst bf16"
                    if peaks["source"] == "measured" else "fallback burst bf16"})
    else:
        out.update({"score_kernel": "fp32 FMA kernel; the step is launch bound at this size: no roofline claim"})
    return out


def bench_decode(P, torch, W, name, dev, stream, peaks, batch=64, score_tokens=16384):
    """A batch of `batch` tokens through one MoE layer (camera_layer_forward), unpruned and sliced at each prune ratio
    by the masks CAMERA-P gives on `score_tokens` calibration tokens.  The step is timed three ways: as the plain call
    (tables and tensor maps rebuilt by every call), with a prepared layer (camera_layer_prepare), and replayed from a
    CUDA graph of the prepared call; on the device with events, and on the host around launch + synchronise."""
    cfg = W.scaled(W.CONFIGS[name], n_tokens=score_tokens)
    L = W.make_layer(cfg, seed=0, layer_id=0, device=dev)
    layer = P.Layer.from_workload(L)
    X = W.make_tokens(cfg, seed=0, layer_id=0, device=dev)
    energy = P.camera_score_layer(layer, X, ALPHA)
    keep, _ = P.camera_select_all(energy, PRUNE_RATIOS)
    off = P.expert_offsets_tensor(layer)
    xd = X[:batch].contiguous()
    yd = torch.empty((batch, cfg.d_model), dtype=torch.float32, device=dev)
    ws_d = P.alloc_workspace(P.camera_forward_workspace_bytes(layer, batch), dev)
    ws_c = P.alloc_workspace(int(P.lib.camera_compact_workspace_bytes(layer.n_experts)), dev)

    def timed(fn, reps=50):
        for _ in range(5):
            fn()
        torch.cuda.synchronize()
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0 = time.perf_counter()
        f0.record(stream)
        for _ in range(reps):
            fn()
        f1.record(stream)
        torch.cuda.synchronize()
        host_us = 1e6 * (time.perf_counter() - t0) / reps
        return 1e3 * f0.elapsed_time(f1) / reps, host_us

    def three_ways(lay_plain, make_prepared):
        plain_us, plain_host = timed(lambda: P.camera_layer_forward(lay_plain, xd, y=yd, workspace=ws_d))
        lay = make_prepared()
        prep_us, prep_host = timed(lambda: P.camera_layer_forward(lay, xd, y=yd, workspace=ws_d))
        graph_us = graph_host = None
        try:
            side = torch.cuda.Stream()
            side.wait_stream(stream)
            g = torch.cuda.CUDAGraph()
            with torch.cuda.stream(side):
                P.camera_layer_forward(lay, xd, y=yd, workspace=ws_d)
                with torch.cuda.graph(g, stream=side):
                    P.camera_layer_forward(lay, xd, y=yd, workspace=ws_d)
            stream.wait_stream(side)
            graph_us, graph_host = timed(g.replay)
        except Exception as exc:          # a capture that fails leaves the plain numbers
            graph_us, graph_host = None, f"capture failed: {type(exc).__name__}"
        return {"us": prep_us, "host_us": prep_host, "unprepared_us": plain_us, "unprepared_host_us": plain_host,
                "graph_us": graph_us, "graph_host_us": graph_host}

    wbytes = 3 * layer.n_me * cfg.d_model * 2
    full = three_ways(layer, lambda: P.camera_layer_prepare(P.Layer.from_workload(L)))
    best = min(v for v in (full["us"], full["graph_us"]) if v is not None)
    out = {"workload": f"{cfg.name} layer, {batch} tokens", "weight_gb": wbytes / 1e9, "full_layer": full,
           "full_layer_us": best, "full_layer_weight_gbs": wbytes / 1e9 / (best * 1e-6),
           "frac_of_hbm_peak": wbytes / 1e9 / (best * 1e-6) / peaks["hbm_gbs"], "pruned": []}
    outd = {k: [torch.empty_like(w) for w in layer.tensors[k]] for k in ("w_gate", "w_up", "w_down")}
    for j, r in enumerate(PRUNE_RATIOS):
        sub, cnt = P.camera_sub_index(keep[j], off, [1])
        P.camera_compact_weights(layer, sub, cnt, 1, out=outd, workspace=ws_c)
        mj = cnt[:, 0].cpu().tolist()
        def sliced():
            return P.Layer(L["w_router"], [outd["w_gate"][e][:mj[e]] for e in range(layer.n_experts)],
                           [outd["w_up"][e][:mj[e]] for e in range(layer.n_experts)], outd["w_down"], cfg.top_k,
                           cfg.n_shared, L["router_bias"], L["w_shared_gate"], cfg.norm_topk, "hf", down_ld=layer.d_ff)
        t = three_ways(sliced(), lambda: P.camera_layer_prepare(sliced()))
        b = min(v for v in (t["us"], t["graph_us"]) if v is not None)
        out["pruned"].append({"prune_ratio": r, "us": b, "speedup": best / b, "ways": t})
    return out


def bench_whole_model(P, torch, W, cfg, dev, stream):
    """Every MoE layer of the model with weights and calibration tokens of its own (seeded by the layer's number):
    camera_score_layer per layer, then the prune masks and bit-widths of all layers from one camera_select_all call
    with one segment per layer.  Generating a layer's weights and tokens is outside the event pairs and reported
    beside the analysis time."""
    nl, T = cfg.n_layers, cfg.n_tokens
    probe = P.Layer.from_workload(W.make_layer(W.scaled(cfg, n_tokens=1), seed=0, layer_id=0, device=dev))
    n_me = probe.n_me
    ws_score = P.alloc_workspace(P.camera_score_workspace_bytes_single_pass(probe, T), dev)
    del probe
    ws_all = P.alloc_workspace(P.camera_select_workspace_bytes(nl * n_me, nl, len(PRUNE_RATIOS) + len(BIT_LEVELS)), dev)
    E_all = torch.empty((nl, n_me), dtype=torch.float32, device=dev)
    keep_all = torch.empty((len(PRUNE_RATIOS), nl * n_me), dtype=torch.uint8, device=dev)
    bits_all = torch.empty(nl * n_me, dtype=torch.uint8, device=dev)
    score_ms, gen_s = 0.0, 0.0
    for l in range(nl):
        t0 = time.perf_counter()
        L = W.make_layer(cfg, seed=0, layer_id=l, device=dev)
        X = W.make_tokens(cfg, seed=0, layer_id=l, device=dev)
        layer = P.Layer.from_workload(L)
        torch.cuda.synchronize()
        gen_s += time.perf_counter() - t0
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        P.camera_score_layer(layer, X, ALPHA, energy=E_all[l], workspace=ws_score, single_pass=True)
        e1.record(stream)
        torch.cuda.synchronize()
        if P.camera_read_status(ws_score) != 0:
            raise RuntimeError("device status set in the whole-model run")
        score_ms += e0.elapsed_time(e1)
        del L, X, layer
    seg = [i * n_me for i in range(nl + 1)]
    s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s0.record(stream)
    P.camera_select_all(E_all.view(-1), PRUNE_RATIOS, BIT_RATIOS, BIT_LEVELS, seg_offsets=seg, workspace=ws_all,
                        keep_masks=keep_all, bits_out=bits_all)
    s1.record(stream)
    torch.cuda.synchronize()
    sel_ms = s0.elapsed_time(s1)
    kept = keep_all.view(len(PRUNE_RATIOS), nl, n_me).sum(dim=2)
    ok = all(int(kept[j, l]) == n_me - int(PRUNE_RATIOS[j] * n_me + 1e-9) for j in range(len(PRUNE_RATIOS)) for l in range(nl))
    return {"what": f"{nl} layers, each with its own seeded weights and {T} tokens: camera_score_layer per layer, one "
                    f"camera_select_all over {nl} segments", "seconds": (score_ms + sel_ms) * 1e-3,
            "score_seconds": score_ms * 1e-3, "select_ms": sel_ms, "input_generation_seconds_not_timed": gen_s,
            "kept_counts_as_expected": bool(ok)}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=28)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="qwen2_57b_a14b")
    ap.add_argument("--tokens", type=int, default=0, help="override the tokens per layer (profiling small cases)")
    ap.add_argument("--routed", type=int, default=0, help="override the number of routed experts (profiling slices)")
    ap.add_argument("--topk", type=int, default=0, help="override top-k (with --routed and --tokens: a slice that keeps the full layer's tokens per expert)")
    ap.add_argument("--oracle-tokens", type=int, default=0, help="tokens of the CPU-oracle sample (default 512 for --impl reference, 2048 for the cpu_baseline leg)")
    ap.add_argument("--shard", default="layers", choices=["layers", "tokens"],
                    help="with --gpus N: every rank its own layer (weak scaling, no exchange), or one layer's tokens "
                         "spread over the ranks with an all-reduce of the 2 x N_e score components (strong scaling)")
    ap.add_argument("--cta-pair", action="store_true", help="force scoring on CTA pairs (tcgen05 cta_group::2)")
    ap.add_argument("--single-cta", action="store_true", help="force scoring with one CTA per MMA")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-compact", action="store_true")
    ap.add_argument("--no-forward", action="store_true")
    ap.add_argument("--no-configs", action="store_true", help="skip the other workload configs")
    ap.add_argument("--no-model", action="store_true", help="skip the measured loop over all layers of the model")
    ap.add_argument("--stack", action="store_true", help="run Algorithm 2's layer loop over a synthetic stack instead of the step benchmark")
    ap.add_argument("--decode-only", action="store_true", help="run only the 64-token decode leg of --config and print its record")
    ap.add_argument("--stack-layers", type=int, default=0, help="layers of the stack (default: the config's)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        return run_reference(args)
    if args.stack:
        return run_stack(args)
    if args.decode_only:
        import torch
        import paper_2508_02322_b200 as P
        from paper_2508_02322_b200 import workloads as W
        torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
        dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
        print(json.dumps({"mode": "decode", "decode": bench_decode(P, torch, W, args.config, dev, torch.cuda.current_stream(),
                                                                   load_peaks())}))
        return

    import torch
    import torch.distributed as dist
    import paper_2508_02322_b200 as P
    from paper_2508_02322_b200 import workloads as W

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    cfg = W.CONFIGS[args.config]
    if args.tokens:
        cfg = W.scaled(cfg, n_tokens=args.tokens)
    if args.routed:
        cfg = W.scaled(cfg, n_routed=args.routed, top_k=min(args.topk or cfg.top_k, args.routed))
    elif args.topk:
        cfg = W.scaled(cfg, top_k=args.topk)
    by_tokens = args.shard == "tokens"
    if by_tokens:
        # one layer for all ranks; a rank scores its share of the tokens, then the components are all-reduced
        t0, t1 = shard_tokens(cfg.n_tokens, world, rank)
        cfg = W.scaled(cfg, n_tokens=t1 - t0)
    T = cfg.n_tokens
    # layers mode: every rank analyses its own layer (weights and tokens seeded by the layer id): no data-path collective
    L = W.make_layer(cfg, seed=0, layer_id=0 if by_tokens else rank, device=dev)
    layer = P.Layer.from_workload(L)
    Xs = [W.make_tokens(cfg, seed=0, layer_id=rank + world * i, device=dev) for i in range(2)]
    n_me = layer.n_me
    # the timed step scores all tokens of the layer in one pass (one launch of the scoring kernel per step); the walk in
    # batches of 65536 tokens through a quarter of the scratch, the library's default, is timed beside it below
    ws_score = P.alloc_workspace(P.camera_score_workspace_bytes_single_pass(layer, T), dev)
    ws_sel = P.alloc_workspace(P.camera_select_workspace_bytes(n_me, 1, len(PRUNE_RATIOS) + len(BIT_LEVELS)), dev)
    energy = torch.empty(n_me, dtype=torch.float32, device=dev)
    keep = torch.empty((len(PRUNE_RATIOS), n_me), dtype=torch.uint8, device=dev)
    bits = torch.empty(n_me, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()

    phi2 = torch.empty(n_me, dtype=torch.float32, device=dev)
    phi_inf = torch.empty_like(phi2)
    x_none = Xs[0][:0]

    def step(i, events=None):
        if by_tokens:
            P.camera_score_layer(layer, Xs[i % 2], ALPHA, energy=energy, workspace=ws_score, stage_events=events, single_pass=True,
                                 cta_pair=(True if args.cta_pair else (False if args.single_cta else None)), phi2=phi2, phi_inf_sq=phi_inf)
            reduce_components(phi2, phi_inf, dist if world > 1 else None)
            # no tokens, accumulate: folds nothing in and turns the reduced components into the energies
            P.camera_score_layer(layer, x_none, ALPHA, energy=energy, workspace=ws_score, phi2=phi2, phi_inf_sq=phi_inf,
                                 accumulate=True)
        else:
            P.camera_score_layer(layer, Xs[i % 2], ALPHA, energy=energy, workspace=ws_score, stage_events=events, single_pass=True,
                                 cta_pair=(True if args.cta_pair else (False if args.single_cta else None)))
        P.camera_select_all(energy, PRUNE_RATIOS, BIT_RATIOS, BIT_LEVELS, workspace=ws_sel, keep_masks=keep, bits_out=bits)

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    for i in range(args.warmup):
        step(i)
    torch.cuda.synchronize()
    status = P.camera_read_status(ws_score)
    if status != 0:
        raise RuntimeError(f"device status {status} after warm-up")

    stage_ev = [{s: (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for s in P.binding.STAGES}
                for _ in range(args.steps)]
    for evs in stage_ev:            # events must exist before their handles are passed down
        for e0, e1 in evs.values():
            e0.record(stream); e1.record(stream)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local)
    sync_all()
    sampler.start()
    # inputs of the large configs exceed the 126 MB L2 several times over; a small config gets its L2 flushed between
    # steps (a 256 MiB write outside the per-step event pairs)
    esz = 2 if cfg.dtype == "bf16" else 4
    footprint = esz * (3 * n_me * cfg.d_model + 2 * T * cfg.d_model)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if footprint < (512 << 20) else None
    if flush is None:
        ev0.record(stream)
        for i in range(args.steps):
            step(i, stage_ev[i])
        ev1.record(stream)
        sync_all()
        ms_local = ev0.elapsed_time(ev1)
    else:
        per_step = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
        for i in range(args.steps):
            flush.zero_()
            per_step[i][0].record(stream)
            step(i, stage_ev[i])
            per_step[i][1].record(stream)
        sync_all()
        ms_local = sum(e0.elapsed_time(e1) for e0, e1 in per_step)
    clocks = sampler.stop()
    ms = max_over_ranks(ms_local, dist if world > 1 else None, dev)
    stage_ms = {s: statistics.mean(e[s][0].elapsed_time(e[s][1]) for e in stage_ev) for s in P.binding.STAGES}
    status = P.camera_read_status(ws_score)
    if status != 0:
        raise RuntimeError(f"device status {status} in the timed region")

    value = world * T * args.steps / (ms * 1e-3)
    ms_per_step = ms / args.steps

    # ---- the same step with the library's default for long token sets: batches of 65536 tokens through one batch's scratch
    batched = None
    if not by_tokens and T > 65536:
        small = P.camera_score_workspace_bytes(layer, T)
        ws_small = ws_score[:small]
        def step_batched(i):
            P.camera_score_layer(layer, Xs[i % 2], ALPHA, energy=energy, workspace=ws_small)
            P.camera_select_all(energy, PRUNE_RATIOS, BIT_RATIOS, BIT_LEVELS, workspace=ws_sel, keep_masks=keep, bits_out=bits)
        for i in range(2):
            step_batched(i)
        sync_all()
        b0, b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n_b = max(4, min(args.steps, 10))
        b0.record(stream)
        for i in range(n_b):
            step_batched(i)
        b1.record(stream)
        sync_all()
        if P.camera_read_status(ws_small) != 0:
            raise RuntimeError("device status set in the batched steps")
        batched = {"what": "the step with camera_score_layer walking the tokens in batches of 65536 (the default when no "
                           "single pass is asked for)", "steps": n_b, "ms_per_step": b0.elapsed_time(b1) / n_b,
                   "workspace_gib": small / 2 ** 30, "single_pass_workspace_gib": ws_score.numel() / 2 ** 30}

    # ---- the selection applied to the weights (Algorithm 2, TopSelect to the slicing), timed on its own after the step loop
    compact = forward = decode = None
    if not args.no_compact:
        off = P.expert_offsets_tensor(layer)
        outw = {k: [torch.empty_like(w) for w in layer.tensors[k]] for k in ("w_gate", "w_up", "w_down")}
        ws_c = P.alloc_workspace(int(P.lib.camera_compact_workspace_bytes(layer.n_experts)), dev)
        c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        def apply_mask():
            sub, counts = P.camera_sub_index(keep[1], off, [1])
            P.camera_compact_weights(layer, sub, counts, 1, out=outw, workspace=ws_c)
            return counts
        counts = apply_mask()
        for _ in range(3):
            apply_mask()
        sync_all()
        c0.record(stream)
        for _ in range(5):
            apply_mask()
        c1.record(stream)
        sync_all()
        c_ms = c0.elapsed_time(c1) / 5
        kept = int(keep[1].sum().item())
        esz = 2 if cfg.dtype == "bf16" else 4
        c_bytes = 3 * 2 * kept * cfg.d_model * esz       # kept rows/columns of three matrices, read once and written once
        compact = {"what": f"sub-index + gather of W_gate, W_up, W_down at prune ratio {PRUNE_RATIOS[1]}", "ms": c_ms,
                   "algorithmic_gb": c_bytes / 1e9, "achieved_gbs": c_bytes / 1e9 / (c_ms * 1e-3),
                   "frac_of_hbm_peak": c_bytes / 1e9 / (c_ms * 1e-3) / load_peaks()["hbm_gbs"]}
        # ---- the output of the full and of the sliced layer on one batch of tokens, and their distance (Eq. 7)
        if not args.no_forward and cfg.dtype == "bf16":
            Tb = min(T, 65536)
            xb = Xs[0][:Tb]
            m = counts[:, 0].cpu().tolist()
            sliced = P.Layer(L["w_router"], [outw["w_gate"][e][:m[e]] for e in range(layer.n_experts)],
                             [outw["w_up"][e][:m[e]] for e in range(layer.n_experts)], outw["w_down"], cfg.top_k,
                             cfg.n_shared, L["router_bias"], L["w_shared_gate"], cfg.norm_topk, "hf", down_ld=layer.d_ff)
            ws_f = P.alloc_workspace(P.camera_forward_workspace_bytes(layer, Tb), dev)
            yb = torch.empty((Tb, cfg.d_model), dtype=torch.float32, device=dev)
            yh = torch.empty_like(yb)
            def timed(fn, reps=3):
                fn(); sync_all()
                f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                f0.record(stream)
                for _ in range(reps):
                    fn()
                f1.record(stream); sync_all()
                return f0.elapsed_time(f1) / reps
            full_ms = timed(lambda: P.camera_layer_forward(layer, xb, y=yb, workspace=ws_f))
            sl_ms = timed(lambda: P.camera_layer_forward(sliced, xb, y=yh, workspace=ws_f))
            e_tmp = torch.empty(n_me, dtype=torch.float32, device=dev)
            both_ms = timed(lambda: P.camera_score_forward_layer(layer, xb, ALPHA, energy=e_tmp, y=yb, workspace=ws_f))
            err = P.camera_output_error(yb, yh).cpu().tolist()
            flop_full = 1.5 * cfg.gate_up_flop * Tb / T
            forward = {"tokens": Tb, "full_layer_ms": full_ms, "full_layer_tflops": flop_full / (full_ms * 1e-3) / 1e12,
                       "sliced_layer_ms": sl_ms, "full_layer_and_scores_ms": both_ms, "prune_ratio": PRUNE_RATIOS[1],
                       "relative_output_error": err[0] / err[1] if err[1] > 0 else None, "mean_cosine": err[2]}
            del ws_f, yb, yh
        del outw

        # ---- decode through the layer, batch of 64 tokens, full and sliced at each prune ratio (the paper's speed table:
        # a DeepSeek-MoE-16B layer; the Qwen2 shape beside it)
        if not args.no_forward and cfg.dtype == "bf16":
            decode = {"batch_tokens": 64, "shapes": {}}
            for name in ([args.config] if args.config != "qwen2_57b_a14b" else ["qwen2_57b_a14b", "deepseek_moe_16b"]):
                decode["shapes"][name] = bench_decode(P, torch, W, name, dev, stream, load_peaks())

    # ---- the selections of all layers of the model in one call (one segment per layer): where a6/a7 see real bytes
    select_model = None
    if not args.no_compact:
        nl = cfg.n_layers
        Eall = energy.repeat(nl) * (1.0 + torch.arange(nl * n_me, device=dev) // n_me).float()
        seg = [i * n_me for i in range(nl + 1)]
        keep_all = torch.empty((len(PRUNE_RATIOS), nl * n_me), dtype=torch.uint8, device=dev)
        bits_all = torch.empty(nl * n_me, dtype=torch.uint8, device=dev)
        ws_all = P.alloc_workspace(P.camera_select_workspace_bytes(nl * n_me, nl, len(PRUNE_RATIOS) + len(BIT_LEVELS)), dev)
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        def select_all():
            P.camera_select_all(Eall, PRUNE_RATIOS, BIT_RATIOS, BIT_LEVELS, seg_offsets=seg, workspace=ws_all,
                                keep_masks=keep_all, bits_out=bits_all)
        for _ in range(3):
            select_all()
        sync_all()
        s0.record(stream)
        for _ in range(10):
            select_all()
        s1.record(stream); sync_all()
        sel_ms = s0.elapsed_time(s1) / 10
        sel_bytes = 4 * nl * n_me + 4 * nl * n_me           # algorithmic: every energy read once, four label bytes per key out
        ws_one = P.alloc_workspace(P.camera_select_workspace_bytes(n_me, 1, len(PRUNE_RATIOS) + len(BIT_LEVELS)), dev)
        def select_one():
            P.camera_select_all(energy, PRUNE_RATIOS, BIT_RATIOS, BIT_LEVELS, workspace=ws_one, keep_masks=keep, bits_out=bits)
        for _ in range(3):
            select_one()
        sync_all()
        s0.record(stream)
        for _ in range(20):
            select_one()
        s1.record(stream); sync_all()
        one_us = 1e3 * s0.elapsed_time(s1) / 20
        select_model = {"what": f"3 prune masks + bit allocation for {nl} layers as segments of one camera_select_all call", "ms": sel_ms,
                        "one_layer_call_us": one_us, "launches_per_call": 1,
                        "algorithmic_gb": sel_bytes / 1e9, "achieved_gbs": sel_bytes / 1e9 / (sel_ms * 1e-3),
                        "frac_of_hbm_peak": sel_bytes / 1e9 / (sel_ms * 1e-3) / load_peaks()["hbm_gbs"]}
        del Eall, keep_all, bits_all, ws_all

    # ---- end to end through the host-buffer entry point: H2D of the tokens, D2H of the results, every step
    e2e = None
    if not args.no_e2e and not by_tokens:
        del ws_score
        torch.cuda.empty_cache()
        ws_an = P.alloc_workspace(P.camera_analyze_workspace_bytes(layer, T, len(BIT_LEVELS)), dev)
        xh = [x.cpu().pin_memory() for x in Xs]
        eh = torch.empty(n_me, dtype=torch.float32).pin_memory()
        kh = torch.empty((len(PRUNE_RATIOS), n_me), dtype=torch.uint8).pin_memory()
        bh = torch.empty(n_me, dtype=torch.uint8).pin_memory()
        n_e2e = max(2, min(args.steps, 4))
        for i in range(2):
            P.camera_analyze_layer_host(layer, xh[i % 2], ALPHA, PRUNE_RATIOS, BIT_RATIOS, BIT_LEVELS, energy_host=eh,
                                        keep_host=kh, bits_host=bh, workspace=ws_an)
        sync_all()
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a0.record(stream)
        for i in range(n_e2e):
            P.camera_analyze_layer_host(layer, xh[i % 2], ALPHA, PRUNE_RATIOS, BIT_RATIOS, BIT_LEVELS, energy_host=eh,
                                        keep_host=kh, bits_host=bh, workspace=ws_an)
        a1.record(stream)
        sync_all()
        e2e_ms = max_over_ranks(a0.elapsed_time(a1), dist if world > 1 else None, dev)
        e2e = {"value": world * T * n_e2e / (e2e_ms * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": xh[0].numel() * xh[0].element_size(),
               "d2h_bytes_per_step": eh.numel() * 4 + kh.numel() + bh.numel(), "steps": n_e2e,
               "ms_per_step": e2e_ms / n_e2e}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = load_peaks()
    # ---- the other workload configs and the measured loop over the model's layers (one GPU; not part of the step loop)
    configs = model_measured = None
    default_run = world == 1 and args.config == "qwen2_57b_a14b" and not (args.tokens or args.routed or args.topk)
    if default_run and not args.no_configs:
        torch.cuda.empty_cache()
        configs = {name: bench_other_config(P, torch, W, name, dev, stream, local, peaks)
                   for name in ("tiny_fp32", "mixtral_8x7b", "qwen15_moe_a27b", "deepseek_moe_16b")}
    if default_run and not args.no_model:
        torch.cuda.empty_cache()
        model_measured = bench_whole_model(P, torch, W, cfg, dev, stream)
    flop = cfg.gate_up_flop
    score_ms = stage_ms["score"]
    achieved = flop / (score_ms * 1e-3) / 1e12
    roofline = {"kernel": "k_score_umma" if args.single_cta else "k_score_umma_pair / k_score_umma (library's choice)", "bound": "tensor", "achieved": achieved,
                "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s", "frac": achieved / peaks["bf16_tflops_sustained"],
                "frac_of_burst_peak": achieved / peaks["bf16_tflops"], "burst_peak": peaks["bf16_tflops"],
                "peak_source": peaks["source"] + " (cuBLAS bf16 sustained in a seconds-long loop: the kernel is timed inside "
                                                 "a multi-second step loop; the burst figure is beside it)",
                "flop_per_launch": flop, "ms_per_launch": score_ms,
                "traffic": SCORE_KERNEL_DRAM_BYTES_FULL_LAYER
                if (args.config == "qwen2_57b_a14b" and not args.single_cta and not by_tokens
                    and not (args.tokens or args.routed or args.topk)) else None}

    # the HBM-bound stages of the step against their algorithmic bytes (X once for the router; X once in and k copies
    # out for the permutation; W_down once for its norms) and the measured copy peak
    esz = 2 if cfg.dtype == "bf16" else 4
    x_bytes = T * cfg.d_model * esz
    stage_bytes = {"router": x_bytes, "permute": (1 + cfg.top_k) * x_bytes, "rownorm": n_me * cfg.d_model * esz}
    stage_roofline = {s: {"bound": "hbm", "algorithmic_gb": b / 1e9, "achieved_gbs": b / 1e9 / (stage_ms[s] * 1e-3),
                          "frac": b / 1e9 / (stage_ms[s] * 1e-3) / peaks["hbm_gbs"]}
                      for s, b in stage_bytes.items() if stage_ms[s] > 0}

    cpu = None
    if not args.no_cpu_baseline:
        n_s = min(args.oracle_tokens or 2048, T)
        Lc = {k: ([t.cpu() for t in v] if isinstance(v, list) else (v.cpu() if hasattr(v, "cpu") else v)) for k, v in L.items()}
        ol, Xd = oracle_prepare(Lc, Xs[0][:n_s].cpu())
        secs = oracle_step(ol, Xd)
        tps = n_s / secs
        cpu = {"value": tps, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
               "sample": f"first {n_s} tokens of the same layer, all {n_me} micro-experts, {secs:.1f} s"}

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "strong" if by_tokens else "weak", "vs_baseline": None,
        "dtype": "bf16" if cfg.dtype == "bf16" else "f32", "data": "synthetic",
        "config": {"workload": f"{cfg.name} layer: d_model {cfg.d_model}, {cfg.n_routed}x{cfg.d_ff_routed} top-{cfg.top_k}"
                               f" + shared {list(cfg.d_ff_shared)}, {T} tokens", "tokens_per_layer": T,
                   "micro_experts": n_me, "alpha": ALPHA, "prune_ratios": list(PRUNE_RATIOS),
                   "bit_levels": list(BIT_LEVELS), "bit_ratios": list(BIT_RATIOS),
                   "l2": "inputs larger than L2" if flush is None else "L2 flushed between steps (256 MiB write, not timed)",
                   "parallelism": (f"tokens x{world}" if by_tokens else f"layers x{world}") if world > 1 else "single GPU"},
        "model_seconds": cfg.n_layers * ms_per_step * 1e-3 / world,     # extrapolated: layers x the step on one layer
        "model_seconds_measured": model_measured, "configs": configs, "batched_scoring": batched,
        "stage_ms": stage_ms, "stage_roofline": stage_roofline, "clocks": clocks, "e2e": e2e, "gpu_launches": (LAUNCHES_PER_STEP + (3 if by_tokens else 0)) * args.steps,
        "roofline": roofline, "compact": compact, "forward": forward, "decode": decode, "select_model": select_model, "cpu_baseline": cpu, "context": PAPER_CONTEXT,
    }
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
