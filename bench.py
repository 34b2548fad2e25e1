#!/usr/bin/env python
"""Benchmark of the GDN tail-replay hot path on B200.

A step is one pass of the whole path (scheduler + chunkwise GDN forward, outputs and final
states) over one batch of synthetic input: the 32-request concurrent-cache-hit workload
(tails ~U{400..3300}, 16 q/k heads shared by 32 v heads, dk = dv = 128, bf16 io, fp32 state).
Prints ONE JSON line.  `--impl reference` times the fp64 CPU oracle on a bounded sample of the
same workload instead.  Launch with torchrun for --gpus N > 1 (one rank per GPU, weak scaling:
every rank replays its own batch; the path has no exchange step, so no data-path collective).
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

from gdn_workloads import (config_concurrent_hits, config_budget_sweep_layer,  # noqa: E402
                           config_budget_sweep_tails)

METRIC = "gdn_tail_replay_throughput"
UNIT = "tokens*heads/s"
WORKLOAD = "concurrent_hits_32req_tails_U400-3300_Hq16_Hv32_d128_bf16_chunk64"
BYTES_PER_TOKEN_HEAD = 776.0        # q,k shared by 2 v-heads + v + o in bf16, g and beta in fp32
FLOPS_PER_TOKEN_HEAD = 139264.0     # 6 dk dv + C (3 dk + 2 dv), triangular products at half cost
STATE_BYTES_PER_CHAIN = 128 * 128 * 4
# DRAM bytes per token*head of the dominant kernel, from the committed ncu capture of the 8-request case
# (profiles/gdn_tc_kernel_concurrent_hits_8req.md: dram read + write = 278.2 MB for 346,944 token*heads,
# final states included); traffic grows in proportion to the units a launch processes.
NCU_TRAFFIC_BYTES_PER_TOKEN_HEAD = 801.8


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons through NVML (read-only) in a thread while the timed region runs."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown"}

    def __init__(self, cuda_index: int):
        self.cuda_index = cuda_index
        self.sm = []
        self.reasons = set()
        self.sm_max = None
        self.stop_flag = False
        self.thread = None
        self.handle = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            self.nv = pynvml
            try:
                uuid = str(torch.cuda.get_device_properties(cuda_index).uuid)
                if not uuid.startswith("GPU-"):
                    uuid = "GPU-" + uuid
                self.handle = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                self.handle = pynvml.nvmlDeviceGetHandleByIndex(cuda_index)
            self.sm_max = float(pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.handle = None

    def _poll(self):
        nv = self.nv
        while not self.stop_flag:
            try:
                self.sm.append(float(nv.nvmlDeviceGetClockInfo(self.handle, nv.NVML_CLOCK_SM)))
                mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.handle))
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.001)

    def start(self):
        if self.handle is None:
            return
        self.thread = threading.Thread(target=self._poll, daemon=True)
        self.thread.start()

    def stop(self):
        self.stop_flag = True
        if self.thread is not None:
            self.thread.join(timeout=2)
        return {"sm_mhz": statistics.median(self.sm) if self.sm else None, "sm_max_mhz": self.sm_max,
                "reasons": sorted(self.reasons), "samples": len(self.sm)}


def to_device(inp, device):
    import torch

    def bf(bits):
        return torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16)
    q, k, v = bf(inp.q_bits), bf(inp.k_bits), bf(inp.v_bits)
    g, beta, cu = torch.from_numpy(inp.g), torch.from_numpy(inp.beta), torch.from_numpy(inp.cu_tail_lens)
    host = [x.contiguous() for x in (q, k, v, g, beta, cu)]
    if device is None:
        return [x.pin_memory() for x in host]
    return [x.to(device) for x in host]


def oracle_timed(inp, budget_s=20.0):
    """Times the oracle, as it stands, on a bounded sample of the workload: whole requests in
    order until about budget_s of CPU work (all of them if they fit)."""
    import oracle
    threads = oracle.default_threads()
    probe = inp.take_chain(0, 0)
    t0 = time.perf_counter()
    oracle.gdn_forward_inputs(probe, threads=1)
    per_th = (time.perf_counter() - t0) / max(1, probe.total_tokens)       # s per token*head, one thread
    lens = inp.tail_lens()
    Hv = inp.num_v_heads
    est_rate = threads / per_th * 0.8
    take, tok = 0, 0
    for L in lens:
        if take > 0 and (tok + int(L)) * Hv / est_rate > budget_s:
            break
        take += 1
        tok += int(L)
    from gdn_workloads import GdnInputs
    sub = GdnInputs(q=inp.q[:tok], k=inp.k[:tok], v=inp.v[:tok], g=inp.g[:tok], beta=inp.beta[:tok],
                    cu_tail_lens=inp.cu_tail_lens[:take + 1].copy(), num_qk_heads=inp.num_qk_heads,
                    num_v_heads=Hv, head_k_dim=inp.head_k_dim, head_v_dim=inp.head_v_dim, io_dtype=inp.io_dtype)
    t0 = time.perf_counter()
    oracle.gdn_forward_inputs(sub, threads=threads)
    dt = time.perf_counter() - t0
    sample = "first %d of %d requests (%d tokens x %d heads), fp64 token-by-token, %.1f s" % (
        take, len(lens), tok, Hv, dt)
    return {"value": tok * Hv / dt, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample}, dt


def reduce_over_ranks(elapsed_ms: float, units: float, device="cpu"):
    """Whole-job view of one timed region: MAX of the elapsed time and SUM of the processed units over all
    ranks (identity when torch.distributed is not initialised).  The path has no exchange step, so this
    reduction of two scalars is the only collective of a multi-GPU run and it sits outside the timed region."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(elapsed_ms), float(units)
    t = torch.tensor([float(elapsed_ms)], dtype=torch.float64, device=device)
    u = torch.tensor([float(units)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def run_reference(args, rank):
    if rank != 0:
        return
    inp = config_concurrent_hits()
    per_step = []
    last = None
    # each step is a bounded sample; keep the whole run within a few minutes
    budget = max(2.0, min(20.0, 150.0 / max(1, args.steps + args.warmup)))
    for i in range(args.warmup + args.steps):
        res, dt = oracle_timed(inp, budget_s=budget)
        if i >= args.warmup:
            per_step.append((res, dt))
        last = res
    value = statistics.mean(r["value"] for r, _ in per_step) if per_step else last["value"]
    ms = statistics.mean(dt for _, dt in per_step) * 1e3 if per_step else None
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "note": "each step is a bounded sample of the workload"},
        "cpu_baseline": dict(last, value=value),
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def run_sweep(args, dev, gdn):
    """Timings of the other named configurations on one GPU (CUDA events, 3 warm-ups + 10 repetitions, 256 MB
    L2 flush before every repetition, 4 rotating seeded input sets where a configuration has layers)."""
    import torch
    from gdn_workloads import config_single_layer, config_full_prefill
    stream = torch.cuda.current_stream()
    ws = gdn.Workspace(dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

    def timed(call, reps=10, warm=3):
        ts = []
        for r in range(warm + reps):
            flush.zero_()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            call()
            b.record(stream)
            torch.cuda.synchronize()
            if r >= warm:
                ts.append(a.elapsed_time(b) * 1e3)
        return {"us_mean": statistics.mean(ts), "us_min": min(ts)}

    def layer_sets(make, n=4):
        return [to_device(make(i), dev) for i in range(n)]

    out = {}
    sets = layer_sets(lambda i: config_single_layer(seed_offset=i))
    L = 1638
    oo = torch.empty((L, 32, 128), dtype=torch.bfloat16, device=dev)
    ss = torch.empty((1, 32, 128, 128), dtype=torch.float32, device=dev)
    it = [0]

    def one_layer():
        x = sets[it[0] % 4]
        it[0] += 1
        gdn.gdn_tail_replay(x[0], x[1], x[2], x[3], x[4], x[5], 64, oo, ss, workspace=ws, kernel=args.kernel, stream=stream)
    r = timed(one_layer)
    r["tokens_heads_per_s"] = L * 32 / (r["us_mean"] * 1e-6)
    out["single_layer_tail_1638"] = r
    del sets
    for cfg in config_budget_sweep_tails():
        L = cfg["tail"]
        sets = layer_sets(lambda i: config_budget_sweep_layer(L, layer=i))
        oo = torch.empty((L, 32, 128), dtype=torch.bfloat16, device=dev)

        def rebuild():
            for layer in range(36):
                x = sets[layer % 4]
                gdn.gdn_tail_replay(x[0], x[1], x[2], x[3], x[4], x[5], 64, oo, ss, workspace=ws, kernel=args.kernel, stream=stream)
        r = timed(rebuild)
        r["layers"] = 36
        out["rebuild_prefix_%d_budget_%d%%_tail_%d" % (cfg["prefix"], cfg["budget_pct"], L)] = r
        del sets
    for m in (32768, 131072):
        x = to_device(config_full_prefill(m), dev)
        oo = torch.empty((m, 32, 128), dtype=torch.bfloat16, device=dev)

        def prefill():
            gdn.gdn_full_prefill(x[0], x[1], x[2], x[3], x[4], x[5], 64, oo, ss, workspace=ws, kernel=args.kernel, stream=stream)
        r = timed(prefill, reps=5)
        r["tokens_heads_per_s"] = m * 32 / (r["us_mean"] * 1e-6)
        out["full_prefill_%d" % m] = r
        del x, oo
    # the 32-request workload from raw projection outputs (input stage fused into the kernel) and from start states
    from gdn_workloads import config_concurrent_hits, make_raw_inputs
    c3 = config_concurrent_hits()
    lens = [int(b - a) for a, b in zip(c3.cu_tail_lens[:-1], c3.cu_tail_lens[1:])]
    ready = to_device(c3, dev)
    raw = to_device(make_raw_inputs(lens, 16, 32, 128, 128, "bf16", seed=2608030310 + 3500), dev)
    T, N = c3.total_tokens, c3.num_seqs
    oo = torch.empty((T, 32, 128), dtype=torch.bfloat16, device=dev)
    ss = torch.empty((N, 32, 128, 128), dtype=torch.float32, device=dev)
    st0 = torch.randn((N, 32, 128, 128), dtype=torch.float32, device=dev)
    for name, x, kw in (("ready_inputs", ready, {}), ("raw_inputs_fused_stage", raw, {"raw_inputs": True}),
                        ("ready_inputs_with_start_states", ready, {"init_state": st0})):
        def call():
            gdn.gdn_tail_replay(x[0], x[1], x[2], x[3], x[4], x[5], 64, oo, ss, workspace=ws, kernel=args.kernel,
                                stream=stream, **kw)
        r = timed(call)
        r["tokens_heads_per_s"] = T * 32 / (r["us_mean"] * 1e-6)
        out["concurrent_hits_32req_" + name] = r
    print(json.dumps({"sweep": out, "unit": "us", "n_gpus": 1, "dtype": "bf16", "data": "synthetic"}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--kernel", type=int, default=0, help="0 auto, 1 fp32 SIMT path, 2 tcgen05 path")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--requests", type=int, default=32, help="requests in the batch (32 = the named workload)")
    ap.add_argument("--sweep", action="store_true",
                    help="instead of the benchmark line, time the other named configurations (single layer, "
                         "budget sweep x 36 layers, full prefill 32K / 128K) and print them as one JSON line")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        run_reference(args, rank)
        return

    import torch
    import torch.distributed as dist
    import paper_2608_30310_b200 as gdn

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    gdn.load_library()

    if args.sweep:
        run_sweep(args, dev, gdn)
        return

    # every rank replays its own batch (weak scaling); seeds differ per rank
    inp = config_concurrent_hits(num_seqs=args.requests, seed_offset=rank)
    T, Hv, N = inp.total_tokens, inp.num_v_heads, inp.num_seqs
    q, k, v, g, beta, cu = to_device(inp, dev)
    out_o = torch.empty((T, Hv, 128), dtype=torch.bfloat16, device=dev)
    out_state = torch.empty((N, Hv, 128, 128), dtype=torch.float32, device=dev)
    ws = gdn.Workspace(dev)
    stream = torch.cuda.current_stream()

    def step():
        gdn.gdn_tail_replay(q, k, v, g, beta, cu, 64, out_o, out_state, workspace=ws, kernel=args.kernel,
                            stream=stream)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    launches_per_step = gdn.last_launch_count()
    barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    # inputs (1.5 GB per step) are far larger than the 126 MB L2: no flush needed between steps
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for a, b in evs:
        a.record(stream)
        step()
        b.record(stream)
    e1.record(stream)
    barrier()
    total_ms = e0.elapsed_time(e1)
    call_ms = [a.elapsed_time(b) for a, b in evs]
    clocks = sampler.stop()
    units_per_step = T * Hv
    total_ms, units_all = reduce_over_ranks(total_ms, units_per_step, dev)
    ms_per_step = total_ms / args.steps
    value = units_all / (ms_per_step * 1e-3)

    # roofline of the dominant kernel (the chunkwise forward); each call = a ~2 us scheduler kernel
    # + this kernel, timed together with events on the launching stream, so `achieved` is a floor
    peaks = load_peaks()
    kern_ms = statistics.mean(call_ms)
    alg_bytes = units_per_step * BYTES_PER_TOKEN_HEAD + N * Hv * STATE_BYTES_PER_CHAIN
    alg_flops = units_per_step * FLOPS_PER_TOKEN_HEAD
    t_hbm = alg_bytes / (peaks["hbm_gbs"] * 1e9)
    t_tc = alg_flops / (peaks["bf16_tflops"] * 1e12)
    achieved_gbs = alg_bytes / (kern_ms * 1e-3) / 1e9
    roofline = {
        "bound": "hbm" if t_hbm >= t_tc else "tensor",
        "achieved": achieved_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
        "frac": achieved_gbs / peaks["hbm_gbs"], "peak_source": peaks["source"],
        "traffic": (NCU_TRAFFIC_BYTES_PER_TOKEN_HEAD * units_per_step
                    if NCU_TRAFFIC_BYTES_PER_TOKEN_HEAD else None),
        "kernel_ms": kern_ms, "algorithmic_bytes": alg_bytes, "algorithmic_flops": alg_flops,
        "achieved_tflops": alg_flops / (kern_ms * 1e-3) / 1e12, "roofline_ms": max(t_hbm, t_tc) * 1e3,
        "frac_of_nominal_8000_gbs": achieved_gbs / 8000.0,      # context: the nominal HBM3e figure, not the denominator
    }

    # end to end through the same C-ABI call with HOST buffers: pinned inputs copied H2D and
    # outputs + states copied D2H inside the timed region, every step
    e2e = None
    if not args.no_e2e:
        hq, hk, hv_, hg, hb, hcu = to_device(inp, None)
        ho = torch.empty((T, Hv, 128), dtype=torch.bfloat16).pin_memory()
        hs = torch.empty((N, Hv, 128, 128), dtype=torch.float32).pin_memory()
        ws_h = gdn.Workspace(dev)
        h2d = sum(x.numel() * x.element_size() for x in (hq, hk, hv_, hg, hb, hcu))
        d2h = ho.numel() * ho.element_size() + hs.numel() * hs.element_size()

        def step_host():
            gdn.gdn_tail_replay(hq, hk, hv_, hg, hb, hcu, 64, ho, hs, workspace=ws_h, kernel=args.kernel,
                                stream=stream)
        e2e_steps = max(3, min(args.steps, 10))
        for _ in range(2):
            step_host()
        barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(e2e_steps):
            step_host()
        b.record(stream)
        barrier()
        te, _ = reduce_over_ranks(a.elapsed_time(b), units_per_step, dev)
        e2e = {"value": units_all / (te / e2e_steps * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps,
               "ms_per_step": te / e2e_steps}
        # context for the number above: the same input bytes copied host -> device with nothing else on the link
        # (the floor of any schedule that has to bring the inputs in)
        if rank == 0:
            dv_ = torch.empty_like(hv_, device=dev)
            dq_ = torch.empty_like(hq, device=dev)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            for rep in range(3):
                if rep == 1:
                    a.record(stream)
                with torch.cuda.stream(stream):
                    dv_.copy_(hv_, non_blocking=True); dq_.copy_(hq, non_blocking=True); dq_.copy_(hk, non_blocking=True)
            b.record(stream)
            torch.cuda.synchronize()
            cbytes = (hv_.numel() + hq.numel() + hk.numel()) * 2
            rate = cbytes / (a.elapsed_time(b) / 2 * 1e-3)
            e2e["h2d_only_gbs"] = rate / 1e9
            e2e["h2d_only_ms_for_step_inputs"] = h2d / rate * 1e3
            del dv_, dq_
        del hq, hk, hv_, ho, hs

    # us per 32K-hit state rebuild: 36 GDN layers back to back, batch 1, 5 % and 10 % budgets
    rebuild = {}
    if rank == 0:
        for cfg in config_budget_sweep_tails():
            if cfg["prefix"] != 32768:
                continue
            sets = [to_device(config_budget_sweep_layer(cfg["tail"], layer=l), dev) for l in range(4)]
            L = cfg["tail"]
            oo = torch.empty((L, Hv, 128), dtype=torch.bfloat16, device=dev)
            ss = torch.empty((1, Hv, 128, 128), dtype=torch.float32, device=dev)
            flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
            times = []
            for rep in range(3 + 10):
                flush.zero_()                                  # 256 MB write: evicts the 126 MB L2
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream)
                for layer in range(36):
                    x = sets[layer % 4]
                    gdn.gdn_tail_replay(x[0], x[1], x[2], x[3], x[4], x[5], 64, oo, ss, workspace=ws,
                                        kernel=args.kernel, stream=stream)
                b.record(stream)
                torch.cuda.synchronize()
                if rep >= 3:
                    times.append(a.elapsed_time(b) * 1e3)
            rebuild["budget_%d%%_tail_%d" % (cfg["budget_pct"], L)] = {
                "us_mean": statistics.mean(times), "us_min": min(times), "layers": 36,
                "note": "4 rotating input sets, L2 flushed before each rebuild"}
            # the same 36 calls captured once in a CUDA graph and replayed (the calls enqueue kernels only: no
            # allocation, no synchronisation), which removes most of the gap between consecutive launches
            try:
                side = torch.cuda.Stream(device=dev)
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.stream(side):
                    with torch.cuda.graph(graph, stream=side):
                        for layer in range(36):
                            x = sets[layer % 4]
                            gdn.gdn_tail_replay(x[0], x[1], x[2], x[3], x[4], x[5], 64, oo, ss, workspace=ws,
                                                kernel=args.kernel, stream=side)
                    gtimes = []
                    for rep in range(3 + 10):
                        flush.zero_()
                        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                        a.record(side)
                        graph.replay()
                        b.record(side)
                        torch.cuda.synchronize()
                        if rep >= 3:
                            gtimes.append(a.elapsed_time(b) * 1e3)
                rebuild["cuda_graph_budget_%d%%_tail_%d" % (cfg["budget_pct"], L)] = {
                    "us_mean": statistics.mean(gtimes), "us_min": min(gtimes), "layers": 36,
                    "note": "the 36 calls above replayed from one CUDA graph, L2 flushed before each rebuild"}
                del graph
            except Exception as exc:                           # capture is a convenience of the caller's, not a promise
                rebuild["cuda_graph_budget_%d%%_tail_%d" % (cfg["budget_pct"], L)] = {"error": str(exc)[:200]}
            del sets, flush

    # the same 32K-hit rebuild with the paper's independent groups packed into one call per layer position: the
    # current layer of every group goes in as one pseudo-request (group size is a model property the paper does not
    # fix: 3 linear-attention layers per group here, i.e. 12 groups and 3 calls per rebuild)
    if rank == 0:
        GROUP_LAYERS = 3
        groups = 36 // GROUP_LAYERS
        for cfg in config_budget_sweep_tails():
            if cfg["prefix"] != 32768:
                continue
            L = cfg["tail"]
            sets = []
            for pos in range(GROUP_LAYERS):
                layers = [config_budget_sweep_layer(L, layer=pos * groups + gi) for gi in range(groups)]
                packed = config_budget_sweep_layer(L, layer=0)
                for name in ("q_bits", "k_bits", "v_bits", "g", "beta"):
                    setattr(packed, name, np.ascontiguousarray(np.concatenate([getattr(x, name) for x in layers], axis=0)))
                packed.cu_tail_lens = (np.arange(groups + 1) * L).astype(np.int32)
                sets.append(to_device(packed, dev))
            oo = torch.empty((groups * L, Hv, 128), dtype=torch.bfloat16, device=dev)
            ss = torch.empty((groups, Hv, 128, 128), dtype=torch.float32, device=dev)
            flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
            times = []
            for rep in range(3 + 10):
                flush.zero_()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream)
                for pos in range(GROUP_LAYERS):
                    x = sets[pos]
                    gdn.gdn_tail_replay(x[0], x[1], x[2], x[3], x[4], x[5], 64, oo, ss, workspace=ws,
                                        kernel=args.kernel, stream=stream)
                b.record(stream)
                torch.cuda.synchronize()
                if rep >= 3:
                    times.append(a.elapsed_time(b) * 1e3)
            rebuild["group_parallel_budget_%d%%_tail_%d" % (cfg["budget_pct"], L)] = {
                "us_mean": statistics.mean(times), "us_min": min(times), "layers": 36, "calls": GROUP_LAYERS,
                "groups_per_call": groups, "note": "independent groups packed as pseudo-requests, L2 flushed before each rebuild"}
            del sets, flush, oo, ss

    # decoding step from the rebuilt states: 256 requests x 32 heads, one token each, states updated in place
    decode = None
    if rank == 0:
        ND = 256
        gq = torch.randn((ND, inp.num_qk_heads, 128), device=dev).to(torch.bfloat16)
        gk = torch.nn.functional.normalize(torch.randn((ND, inp.num_qk_heads, 128), device=dev), dim=-1).to(torch.bfloat16)
        gv = torch.randn((ND, Hv, 128), device=dev).to(torch.bfloat16)
        gg = -torch.rand((ND, Hv), device=dev) * 0.1
        gb = torch.sigmoid(torch.randn((ND, Hv), device=dev))
        st = torch.randn((ND, Hv, 128, 128), device=dev)
        do = torch.empty((ND, Hv, 128), dtype=torch.bfloat16, device=dev)
        ts = []
        for rep in range(3 + 10):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            gdn.gdn_decode_step(gq, gk, gv, gg, gb, st, do, st, stream=stream)
            b.record(stream)
            torch.cuda.synchronize()
            if rep >= 3:
                ts.append(a.elapsed_time(b) * 1e3)
        dbytes = 2.0 * st.numel() * 4 + (gq.numel() + gk.numel() + gv.numel() + do.numel()) * 2 + (gg.numel() + gb.numel()) * 4
        decode = {"requests": ND, "us_mean": statistics.mean(ts), "us_min": min(ts),
                  "achieved_gbs": dbytes / (statistics.mean(ts) * 1e-6) / 1e9, "peak_gbs": peaks["hbm_gbs"],
                  "frac": dbytes / (statistics.mean(ts) * 1e-6) / 1e9 / peaks["hbm_gbs"],
                  "note": "1 GiB of states read and written per step (larger than L2), bf16 io"}
        del st, gq, gk, gv, do

    # transfer/replay overlap (the paper's second optimisation): a pinned host buffer standing in for the
    # full-attention KV cache of a 32K-token hit goes host -> device while the 36-layer replay runs, serialised on
    # one stream (SER) or on a copy stream of its own (OVL); a synchronisation point follows, as before the query forward
    overlap = None
    if rank == 0:
        cfg = [c for c in config_budget_sweep_tails() if c["prefix"] == 32768 and c["budget_pct"] == 5][0]
        L = cfg["tail"]
        sets = [to_device(config_budget_sweep_layer(L, layer=l), dev) for l in range(4)]
        oo = torch.empty((L, Hv, 128), dtype=torch.bfloat16, device=dev)
        ss = torch.empty((1, Hv, 128, 128), dtype=torch.float32, device=dev)
        kv_bytes = 256 << 20                                   # 32,768 tokens x 8 KiB of K and V per token
        kv_host = torch.empty(kv_bytes, dtype=torch.uint8).pin_memory()
        kv_dev = torch.empty(kv_bytes, dtype=torch.uint8, device=dev)
        copy_stream = torch.cuda.Stream(device=dev)

        def replay():
            for layer in range(36):
                x = sets[layer % 4]
                gdn.gdn_tail_replay(x[0], x[1], x[2], x[3], x[4], x[5], 64, oo, ss, workspace=ws,
                                    kernel=args.kernel, stream=stream)

        def run(ovl):
            ts = []
            for rep in range(2 + 8):
                torch.cuda.synchronize()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream)
                if ovl:
                    copy_stream.wait_stream(stream)
                    with torch.cuda.stream(copy_stream):
                        kv_dev.copy_(kv_host, non_blocking=True)
                    replay()
                    stream.wait_stream(copy_stream)
                else:
                    kv_dev.copy_(kv_host, non_blocking=True)
                    replay()
                b.record(stream)
                torch.cuda.synchronize()
                if rep >= 2:
                    ts.append(a.elapsed_time(b) * 1e3)
            return statistics.mean(ts)
        ser, ovl = run(False), run(True)
        overlap = {"kv_bytes": kv_bytes, "tail": L, "layers": 36, "serialized_us": ser, "overlapped_us": ovl,
                   "saved_frac": 1.0 - ovl / ser}
        del sets, kv_host, kv_dev

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu_baseline, _ = oracle_timed(inp, budget_s=20.0)

    if world > 1:
        dist.barrier()
    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic",
            "config": {"workload": WORKLOAD, "requests": N, "tokens": T, "v_heads": Hv, "qk_heads": inp.num_qk_heads,
                       "chunk": 64, "state": "fp32", "l2": "inputs per step (1.5 GB) exceed L2, no flush",
                       "kernel": {0: "auto", 1: "fp32_simt", 2: "tcgen05"}[args.kernel]},
            "roofline": roofline, "cpu_baseline": cpu_baseline, "e2e": e2e, "clocks": clocks,
            "gpu_launches": launches_per_step * args.steps,
            "rebuild_32k_us": rebuild, "decode_step": decode, "transfer_replay_overlap": overlap,
            "paper_context": "paper reports only whole-model TTFT on H100 (9.1-14.3x over full prefill at 32K); no kernel-level number",
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
