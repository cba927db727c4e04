#!/usr/bin/env python
"""Benchmark of the block-sparse attention path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload wan14b|wan1p3b] [--no-e2e] [--no-cpu] [--sweep]

One "step" is one pass of the whole path over one batch of synthetic input
resident in HBM: block selection (pool + top-k kernels) followed by the
block-sparse attention forward, bf16, on the Wan2.1-14B-720P attention shape
(B=1, H=40, N=75600, d=128, 128x128 blocks) at 97 % block sparsity.  The
headline value is kept-block TFLOP/s = 4*d*sum(valid q rows * valid k rows
over kept tiles) / step time.  The same JSON line also carries the FP8 leg
(3 quantise launches + FP8 forward), per-kernel times, the roofline of the
dominant kernel, the end-to-end number through the host-buffer C-ABI call and
the CPU oracle timed on a bounded sample.

With N > 1 (torchrun, one rank per GPU) every rank runs the same-shaped
problem on its own seeded batch: batches are independent, so there is no
data-path collective; the value is the aggregate over ranks ("weak" scaling).

``--impl reference`` times the CPU oracle as it stands on the host cores.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import workloads  # noqa: E402

METRIC = "block-sparse attn effective TFLOP/s (kept FLOPs), select+fwd, 97% sparse"
UNIT = "TFLOP/s"
# DRAM bytes (read + write) of one bf16 forward launch on the default workload (wan14b, 97 %),
# from the one-pass ncu capture summarised in profiles/launch_list_wan14b_s97.md.
# bricks (frames x rows x columns of the token grid) that tile the grid of each workload; one 128-token block each
BRICKS = {"wan14b": (3, 5, 8), "wan1p3b": (3, 5, 4)}
FWD_DRAM_TRAFFIC_BYTES = {"wan14b": 2580123136 + 761104384}   # ncu one-pass capture of the full-size fwd_pipe_kernel launch


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"bf16": float(p["bf16_tflops"]), "bf16_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "hbm": float(p["hbm_gbs"]), "source": "measured"}
    return {"bf16": 1590.0, "bf16_sustained": 1400.0, "hbm": 6650.0, "source": "fallback"}


def kept_flops(w, kept_idx_cpu, kept_cnt_cpu, items=None):
    """4*d*sum over kept (query block, key block) tiles of valid rows x valid keys."""
    nb, blk, N = w.nb, w.block, w.N
    valid = torch.full((nb,), blk, dtype=torch.int64)
    valid[nb - 1] = w.tail
    idx = kept_idx_cpu.reshape(-1, nb, kept_idx_cpu.shape[-1]).long()
    cnt = kept_cnt_cpu.reshape(-1, nb).long()
    mask = torch.arange(idx.shape[-1])[None, None, :] < cnt[..., None]
    keys = (valid[idx.clamp(0, nb - 1)] * mask).sum(-1)           # [BH, nb] valid keys per query block
    per_item = keys * valid[None, :]
    if items is not None:
        return 4 * w.d * int(sum(per_item[h, i] for h, i in items))
    return 4 * w.d * int(per_item.sum())


class ClockSampler:
    """Samples SM clock, power and clock-event reasons while a region runs: NVML polled every few milliseconds
    from a thread (read-only queries), or `nvidia-smi -lms 100` when the NVML binding is missing."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")
    # NVML clock-event reason bits
    BITS = {"sw_power_cap": 0x4, "hw_slowdown": 0x8, "sw_thermal_slowdown": 0x20, "hw_thermal_slowdown": 0x40}

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []
        self.nvml, self.samples, self.stop = None, [], threading.Event()

    def __enter__(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            self.handle = pynvml.nvmlDeviceGetHandleByIndex(self.index)
            self.max_sm = float(pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM))
            self.nvml = pynvml
            self.thread = threading.Thread(target=self._poll, daemon=True)
            self.thread.start()
            return self
        except Exception:
            self.nvml = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def _poll(self):
        n = self.nvml
        get_reasons = getattr(n, "nvmlDeviceGetCurrentClocksEventReasons", None) or n.nvmlDeviceGetCurrentClocksThrottleReasons
        while not self.stop.is_set():
            try:
                self.samples.append((float(n.nvmlDeviceGetClockInfo(self.handle, n.NVML_CLOCK_SM)), int(get_reasons(self.handle)),
                                     n.nvmlDeviceGetPowerUsage(self.handle) / 1000.0))
            except Exception:
                pass
            time.sleep(0.004)

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def __exit__(self, *exc):
        if self.nvml is not None:
            self.stop.set()
            self.thread.join(timeout=2)
            return
        if self.proc is not None:
            time.sleep(0.15)
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()

    def summary(self):
        if self.nvml is not None and self.samples:
            sm = [c for c, _, _ in self.samples]
            reasons = sorted(name for name, bit in self.BITS.items() if any(r & bit for _, r, _ in self.samples))
            return {"sm_mhz": statistics.median(sm), "sm_min_mhz": min(sm), "sm_max_mhz": self.max_sm, "reasons": reasons,
                    "power_w_max": max(pw for _, _, pw in self.samples), "samples": len(sm), "source": "nvml"}
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons), "samples": len(sm),
                "source": "nvidia-smi"}


# --------------------------------------------------------------------------- CPU oracle legs

def cpu_oracle_sample(w, target_seconds: float, nheads: int = 4):
    """Times the CPU oracle (selection of `nheads` heads in full + attention on a sample of
    those heads' query blocks) and returns kept-FLOP throughput of the sample."""
    import oracle
    cores = oracle.num_threads()
    nheads = min(nheads, w.H)
    w1 = w.with_heads(nheads)
    q, k, v = workloads.structured_qkv(w, heads=list(range(nheads)), device="cpu")
    q, k, v = q[0], k[0], v[0]
    t0 = time.perf_counter()
    idx, cnt = oracle.select(q, k, w.block, w.topk)
    t_sel = time.perf_counter() - t0
    # calibrate on one batch of `cores` items, then size the sample for the time target
    g = torch.Generator().manual_seed(1234)
    order = [(int(x) // w.nb, int(x) % w.nb) for x in torch.randperm(nheads * w.nb, generator=g)]
    first = order[:cores]
    t0 = time.perf_counter()
    oracle.attention(q, k, v, idx, cnt, w.block, items=first)
    t_first = time.perf_counter() - t0
    n_more = int(max(0, min(len(order) - cores, (target_seconds - t_first - t_sel) / max(t_first, 1e-6) * cores)))
    rest = order[cores:cores + n_more]
    t_rest = 0.0
    if rest:
        t0 = time.perf_counter()
        oracle.attention(q, k, v, idx, cnt, w.block, items=rest)
        t_rest = time.perf_counter() - t0
    items = first + rest
    flops = kept_flops(w1, idx, cnt, items)
    t_total = t_first + t_rest + t_sel * len(items) / (nheads * w.nb)
    return {"value": flops / t_total / 1e12, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": (f"heads 0-{nheads - 1} of {w.name}: oracle selection of those heads ({t_sel:.2f} s, charged pro rata) + "
                       f"fp64 oracle attention on {len(items)} of their {nheads * w.nb} query blocks ({t_first + t_rest:.2f} s)"),
            "seconds": t_total, "items": len(items)}


def run_reference(args, w):
    """--impl reference: the CPU oracle on the host cores, one bounded sample per step."""
    import oracle
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cores = oracle.num_threads()
    q, k, v = workloads.structured_qkv(w, heads=[0], device="cpu")
    q, k, v = q[0], k[0], v[0]
    idx, cnt = oracle.select(q, k, w.block, w.topk)
    w1 = w.with_heads(1)
    g = torch.Generator().manual_seed(99)
    per_step = 8 * max(1, cores)
    times, flops = [], []
    for step in range(args.warmup + args.steps):
        items = [(0, int(i)) for i in torch.randint(0, w.nb, (per_step,), generator=g)]
        t0 = time.perf_counter()
        oracle.attention(q, k, v, idx, cnt, w.block, items=items)
        dt = time.perf_counter() - t0
        if step >= args.warmup:
            times.append(dt); flops.append(kept_flops(w1, idx, cnt, items))
    total_t, total_f = sum(times), sum(flops)
    value = total_f / total_t / 1e12
    sample = (f"each step: fp64 oracle attention on {per_step} random query blocks of head 0 of {w.name} "
              f"(kept lists from the oracle's own selection); throughput = kept FLOPs / time")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * total_t / max(1, len(times)), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_dict(w, "bf16"),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def config_dict(w, dtype):
    return {"workload": f"{w.name}: B={w.B} H={w.H} N={w.N} d={w.d} grid={'x'.join(map(str, w.grid))} "
                        f"block={w.block} sparsity={w.sparsity} (kept {w.topk} of {w.nb} key blocks per query block)",
            "dtype_inputs": dtype, "selection": "pooled-score top-k (sparkattn_select)",
            "l2": "inputs (3 x 774 MB) exceed the 126 MB L2; no explicit flush",
            "parallelism": "independent batch per GPU, no collective"}


# --------------------------------------------------------------------------- GPU leg

def max_over_ranks(value: float, device) -> float:
    """Largest value over all ranks of the default process group (identity without one)."""
    if not (torch.distributed.is_available() and torch.distributed.is_initialized()):
        return value
    t = torch.tensor([value], device=device, dtype=torch.float64)
    torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(flops_per_rank: float, ms: float, world: int) -> float:
    """Whole-job TFLOP/s when every rank did `flops_per_rank` in `ms` (the max over ranks)."""
    return world * flops_per_rank / (ms * 1e-3) / 1e12


def time_region(fn, steps, warmup, stream, dist_on):
    """warmup untimed calls, then `steps` timed calls between barrier+sync; returns max-over-ranks ms."""
    for _ in range(warmup):
        fn(-1)
    if dist_on:
        torch.distributed.barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(steps):
        fn(i)
    e1.record(stream)
    torch.cuda.synchronize()
    if dist_on:
        torch.distributed.barrier()
    return max_over_ranks(e0.elapsed_time(e1), "cuda")


def run_ours(args, w):
    import paper_2609_23153_b200 as sa
    from paper_2609_23153_b200 import build as sa_build
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dist_on = world > 1
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    if dist_on:
        torch.distributed.init_process_group("nccl", device_id=torch.device(dev))
    if rank == 0:
        sa_build.build()
    if dist_on:
        torch.distributed.barrier()
    sa.lib()
    peaks = load_peaks()
    stream = torch.cuda.current_stream()

    # every rank owns an independent batch of the same shape (different seed)
    wr = workloads.Workload(w.name, w.cfg_id + 1000 * rank, w.B, w.H, w.d, w.grid, w.block, w.sparsity)
    q, k, v = workloads.structured_qkv(wr, device=dev)
    topk, nb = w.topk, w.nb
    shape = sa.make_shape(q, w.block)
    ws_sel = sa.alloc_workspace(shape, 0, topk, dev)
    ws_fwd = sa.alloc_workspace(shape, 1, nb if args.sweep else topk, dev)
    kept_idx = torch.empty((w.B, w.H, nb, topk), dtype=torch.int32, device=dev)
    kept_cnt = torch.empty((w.B, w.H, nb), dtype=torch.int32, device=dev)
    out = torch.empty_like(q)

    K = args.steps
    ev = {name: [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
          for name in ("select", "fwd")}

    def step(i):
        if i >= 0:
            ev["select"][i][0].record(stream)
        sa.select(q, k, w.block, topk, kept_idx=kept_idx, kept_cnt=kept_cnt, workspace=ws_sel)
        if i >= 0:
            ev["select"][i][1].record(stream); ev["fwd"][i][0].record(stream)
        sa.fwd(q, k, v, kept_idx, kept_cnt, w.block, out=out, workspace=ws_fwd)
        if i >= 0:
            ev["fwd"][i][1].record(stream)

    with ClockSampler(local) as clk:
        ms_total = time_region(step, K, args.warmup, stream, dist_on)
    clocks = clk.summary()
    for wsb, name in ((ws_sel, "select"), (ws_fwd, "fwd")):
        st = sa.read_status(wsb)
        if st != sa.OK:
            raise RuntimeError(f"device status after {name}: {sa.status_string(st)}")
    ms_step = ms_total / K
    ms_sel = statistics.mean(a.elapsed_time(b) for a, b in ev["select"])
    ms_fwd = statistics.mean(a.elapsed_time(b) for a, b in ev["fwd"])
    idx_cpu, cnt_cpu = kept_idx.cpu(), kept_cnt.cpu()
    flops = kept_flops(w, idx_cpu, cnt_cpu)
    value = aggregate_throughput(flops, ms_step, world)
    fwd_tflops = flops / (ms_fwd * 1e-3) / 1e12
    elems = w.B * w.H * w.N * w.d
    sel_bytes = 2 * elems * 2 + kept_idx.numel() * 4 + kept_cnt.numel() * 4
    kernels = {
        "select": {"ms": ms_sel, "launches_per_step": 2, "algorithmic_bytes": sel_bytes,
                   "GBps": sel_bytes / (ms_sel * 1e-3) / 1e9, "frac_of_hbm_peak": sel_bytes / (ms_sel * 1e-3) / 1e9 / peaks["hbm"]},
        "fwd_bf16": {"ms": ms_fwd, "launches_per_step": 2 if (w.d == 128 and w.block in (64, 128)) else 1, "TFLOPs": fwd_tflops},
    }
    pipelined = w.d == 128 and w.block in (64, 128)   # d = 128 runs the persistent pipelined kernel (+ list pre-pass)
    roofline = {"kernel": f"fwd_pipe_kernel (bf16, d=128, {w.block}x{w.block} blocks)" if pipelined else f"fwd_kernel<{w.d},{w.block},bf16>", "bound": "tensor", "achieved": fwd_tflops, "peak": peaks["bf16"],
                "unit": "TFLOP/s", "frac": fwd_tflops / peaks["bf16"], "traffic": FWD_DRAM_TRAFFIC_BYTES.get(w.name) if w.sparsity == 0.97 else None,
                "peak_source": f"{peaks['source']} bf16 burst (sustained {peaks['bf16_sustained']})",
                "flops_per_launch": flops, "ms_per_launch": ms_fwd}

    # ---- FP8 leg: 3 quantise launches + FP8 forward (selection reuses the bf16 lists)
    fp8 = None
    if not args.no_fp8:
        codes = [torch.empty(q.shape, dtype=torch.uint8, device=dev) for _ in range(3)]
        scales = [torch.empty((w.B, w.H, nb), dtype=torch.float32, device=dev) for _ in range(3)]
        evq = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
        evf = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]

        def step8(i):
            if i >= 0:
                evq[i][0].record(stream)
            for t, c, s in zip((q, k, v), codes, scales):
                sa.quant_fp8(t, w.block, codes=c, scales=s)
            if i >= 0:
                evq[i][1].record(stream); evf[i][0].record(stream)
            sa.fwd(codes[0], codes[1], codes[2], kept_idx, kept_cnt, w.block, scales=tuple(scales), out=out,
                   workspace=ws_fwd)
            if i >= 0:
                evf[i][1].record(stream)

        ms8 = time_region(step8, K, args.warmup, stream, dist_on) / K
        if sa.read_status(ws_fwd) != sa.OK:
            raise RuntimeError("device status after fp8 fwd")
        ms_q = statistics.mean(a.elapsed_time(b) for a, b in evq)
        ms_f8 = statistics.mean(a.elapsed_time(b) for a, b in evf)
        qbytes = 3 * (elems * 3 + scales[0].numel() * 4)
        fp8 = {"kernel": "fwd_pipe_kernel (FP8)" if pipelined else f"fwd_kernel<{w.d},{w.block},fp8>", "ms_per_step_quant_plus_fwd": ms8, "quant_ms_3_tensors": ms_q, "quant_GBps": qbytes / (ms_q * 1e-3) / 1e9,
               "quant_frac_of_hbm_peak": qbytes / (ms_q * 1e-3) / 1e9 / peaks["hbm"],
               "fwd_ms": ms_f8, "fwd_TFLOPs": flops / (ms_f8 * 1e-3) / 1e12,
               "fwd_frac_of_nominal_fp8_peak_4500": flops / (ms_f8 * 1e-3) / 1e12 / 4500.0,
               "fwd_frac_of_2x_measured_bf16_peak": flops / (ms_f8 * 1e-3) / 1e12 / (2 * peaks["bf16"]),
               "note": "FP8 peak = measured bf16 peak x 2 (nominal ratio); torch._scaled_mm 8192^3 measured 3122 TFLOP/s on this pool"}
        # per-token activation quantisation (the paper's fused scale-and-cast kernel), one tensor, outside the step
        tok_scales = torch.empty((w.B, w.H, w.N), dtype=torch.float32, device=dev)
        evt = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]

        def step_tok(i):
            if i >= 0:
                evt[i][0].record(stream)
            sa.quant_fp8_per_token(v if i % 2 else k, codes=codes[0], scales=tok_scales)
            if i >= 0:
                evt[i][1].record(stream)

        time_region(step_tok, K, args.warmup, stream, dist_on)
        ms_tok = statistics.mean(a.elapsed_time(b) for a, b in evt)
        tbytes = elems * 3 + tok_scales.numel() * 4
        fp8["quant_per_token_ms"] = ms_tok
        fp8["quant_per_token_GBps"] = tbytes / (ms_tok * 1e-3) / 1e9
        fp8["quant_per_token_frac_of_hbm_peak"] = tbytes / (ms_tok * 1e-3) / 1e9 / peaks["hbm"]
        del codes, tok_scales

    # ---- compensation branch + gate fusion (d = 128 only): state pass over K, V, then the fused apply pass
    comp = None
    if not args.no_comp and w.d == 128:
        pq, pk, gate = workloads.compensation_params(wr, 64, device=dev)
        axis, freq = workloads.rope_schedule(w.d, 64)
        ws_c = torch.empty(sa.comp_workspace_bytes(shape, w.grid), dtype=torch.uint8, device=dev)
        state = torch.empty((w.B, w.H, 64, w.d), dtype=torch.float32, device=dev)
        fused = torch.empty_like(q)
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
        eva = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]

        def stepc(i):
            if i >= 0:
                evs[i][0].record(stream)
            sa.comp_state(k, v, pk, w.grid, axis, freq, state=state, workspace=ws_c)
            if i >= 0:
                evs[i][1].record(stream); eva[i][0].record(stream)
            sa.comp_apply(q, pq, state, gate, out, w.grid, axis, freq, out=fused, workspace=ws_c)
            if i >= 0:
                eva[i][1].record(stream)

        msc = time_region(stepc, K, args.warmup, stream, dist_on) / K
        if sa.read_status(ws_c) != sa.OK:
            raise RuntimeError("device status after compensation")
        ms_s = statistics.mean(a.elapsed_time(b) for a, b in evs)
        ms_a = statistics.mean(a.elapsed_time(b) for a, b in eva)
        sbytes = 2 * elems * 2
        abytes = 3 * elems * 2 + gate.numel() * 4
        comp = {"rank": 64, "ms_per_step": msc, "state_ms": ms_s, "state_GBps": sbytes / (ms_s * 1e-3) / 1e9,
                "state_frac_of_hbm_peak": sbytes / (ms_s * 1e-3) / 1e9 / peaks["hbm"],
                "apply_ms": ms_a, "apply_GBps": abytes / (ms_a * 1e-3) / 1e9,
                "apply_frac_of_hbm_peak": abytes / (ms_a * 1e-3) / 1e9 / peaks["hbm"],
                "launches_per_step": 3}
        del fused, state, ws_c, pq, pk, gate

    # ---- brick token order (d = 128, 128-token blocks): gather into bricks padded to whole blocks, selection and
    # forward with per-block token counts, and how much of the attention mass the kept blocks hold in either order
    bricks = None
    if not args.no_bricks and w.d == 128 and w.block == 128 and not args.block:
        brick = BRICKS.get(w.name)
        gather, valid, scatter = sa.brick_layout(w.grid, brick, w.block, device=dev)
        nbr = valid.numel()
        topk_b = max(1, int((1.0 - w.sparsity) * nbr + 0.5))
        qb_ = sa.gather_tokens(q, gather); kb_ = sa.gather_tokens(k, gather); vb_ = sa.gather_tokens(v, gather)
        shape_b = sa.make_shape(qb_, w.block)
        ws_sb = sa.alloc_workspace(shape_b, 0, topk_b, dev); ws_fb = sa.alloc_workspace(shape_b, 1, topk_b, dev)
        idx_b, cnt_b = sa.select(qb_, kb_, w.block, topk_b, block_valid=valid, workspace=ws_sb)
        out_b = torch.empty_like(qb_)
        evg = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
        evs_b = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
        evf_b = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]

        def step_b(i):
            if i >= 0:
                evg[i][0].record(stream)
            sa.gather_tokens(q, gather, out=qb_)
            if i >= 0:
                evg[i][1].record(stream); evs_b[i][0].record(stream)
            sa.select(qb_, kb_, w.block, topk_b, block_valid=valid, kept_idx=idx_b, kept_cnt=cnt_b, workspace=ws_sb)
            if i >= 0:
                evs_b[i][1].record(stream); evf_b[i][0].record(stream)
            sa.fwd(qb_, kb_, vb_, idx_b, cnt_b, w.block, out=out_b, workspace=ws_fb, block_valid=valid)
            if i >= 0:
                evf_b[i][1].record(stream)

        time_region(step_b, K, args.warmup, stream, dist_on)
        if sa.read_status(ws_fb) != sa.OK:
            raise RuntimeError("device status after the brick-order forward")
        ms_g = statistics.mean(a.elapsed_time(b) for a, b in evg)
        gbytes = elems * 2 + qb_.numel() * 2
        # attention mass held by the kept blocks, raster order against brick order, on sampled query rows
        gen = torch.Generator().manual_seed(11)
        heads = list(range(min(w.H, 4)))
        rows = torch.randint(0, w.N, (64,), generator=gen).to(dev)
        mass_r = mass_b = 0.0
        for hh in heads:
            logits = (q[0, hh, rows].float() @ k[0, hh].float().T) / math.sqrt(w.d)
            pr = torch.softmax(logits, dim=-1)                                         # [rows, N]
            blk_of_key = torch.arange(w.N, device=dev) // w.block
            keep_r = torch.zeros((rows.numel(), nb), dtype=torch.bool, device=dev)
            keep_r.scatter_(1, kept_idx[0, hh, rows // w.block].long(), True)
            mass_r += float((pr * keep_r[:, blk_of_key]).sum()) / rows.numel()
            pos = scatter[rows].long()                                                 # the rows' positions in brick order
            keep_b = torch.zeros((rows.numel(), nbr), dtype=torch.bool, device=dev)
            keep_b.scatter_(1, idx_b[0, hh, pos // w.block].long(), True)
            mass_b += float((pr * keep_b[:, scatter.long() // w.block]).sum()) / rows.numel()
        bricks = {"brick": list(brick), "blocks": nbr, "real_rows_per_block": [int(valid.min()), int(valid.max())], "topk": topk_b,
                  "gather_ms_per_tensor": ms_g, "gather_GBps": gbytes / (ms_g * 1e-3) / 1e9,
                  "gather_frac_of_hbm_peak": gbytes / (ms_g * 1e-3) / 1e9 / peaks["hbm"],
                  "select_ms": statistics.mean(a.elapsed_time(b) for a, b in evs_b),
                  "fwd_ms": statistics.mean(a.elapsed_time(b) for a, b in evf_b),
                  "attention_mass_in_kept_blocks": {"raster": mass_r / len(heads), "bricks": mass_b / len(heads),
                                                    "sample": f"{rows.numel()} query rows of heads {heads[0]}-{heads[-1]}, equal budget ({w.topk} of {nb} / {topk_b} of {nbr} blocks)"}}
        del qb_, kb_, vb_, out_b, ws_sb, ws_fb

    # ---- sparsity sweep (optional): fwd only, lists from sparkattn_select
    sweep = None
    if args.sweep:
        sweep = []
        for s in (0.0, 0.5, 0.75, 0.9, 0.97):
            ws_ = w.with_sparsity(s)
            ki, kc = sa.select(q, k, w.block, ws_.topk, workspace=ws_sel)
            reps = 2 if s < 0.6 else 5
            sa.fwd(q, k, v, ki, kc, w.block, out=out, workspace=ws_fwd)
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for _ in range(reps):
                sa.fwd(q, k, v, ki, kc, w.block, out=out, workspace=ws_fwd)
            b.record(stream); torch.cuda.synchronize()
            ms = a.elapsed_time(b) / reps
            fl = kept_flops(w, ki.cpu(), kc.cpu())
            sweep.append({"sparsity": s, "kept": ws_.topk, "dtype": "bf16", "ms": ms, "TFLOPs": fl / ms / 1e9,
                          "frac_of_bf16_peak": fl / ms / 1e9 / peaks["bf16"]})
            del ki, kc

    # ---- end to end through the host-buffer C-ABI call (H2D of Q,K,V and D2H of O inside the timed region)
    e2e = None
    if not args.no_e2e:
        del out
        torch.cuda.empty_cache()
        hq, hk, hv = (t.cpu().pin_memory() for t in (q, k, v))
        ho = torch.empty_like(hq).pin_memory()
        arena = torch.empty(sa.arena_bytes(shape, sa.BF16, topk), dtype=torch.uint8, device=dev)
        ke = max(1, min(K, args.e2e_steps))

        def step_e2e(i):
            sa.attention_host(hq, hk, hv, w.block, topk, out=ho, arena=arena)

        ms_e = time_region(step_e2e, ke, 1, stream, dist_on) / ke
        e2e = {"value": world * flops / (ms_e * 1e-3) / 1e12, "unit": UNIT, "ms_per_step": ms_e, "steps": ke,
               "h2d_bytes_per_step": 3 * hq.numel() * 2, "d2h_bytes_per_step": ho.numel() * 2 + 8,
               "call": "sparkattn_attention_host (pinned host Q,K,V -> select -> fwd -> host O)"}
        del arena, hq, hk, hv, ho

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu:
        cpu = cpu_oracle_sample(w, target_seconds=args.cpu_seconds)

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": args.warmup,
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic", "config": config_dict(w, "bf16"),
            "kept_flops_per_step_per_gpu": flops, "clocks": clocks, "gpu_launches": (4 if pipelined else 3) * K,
            "kernels": kernels, "roofline": roofline, "fp8": fp8, "compensation": comp, "bricks": bricks, "e2e": e2e,
            "cpu_baseline": cpu,
        }
        if sweep is not None:
            line["sweep"] = sweep
        print(json.dumps(line), flush=True)
    if dist_on:
        torch.distributed.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", choices=["wan14b", "wan1p3b"], default="wan14b")
    ap.add_argument("--sparsity", type=float, default=None)
    ap.add_argument("--block", type=int, default=None, help="token block size (default: the workload's; 64 = the paper's trained size)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-fp8", action="store_true")
    ap.add_argument("--no-comp", action="store_true", help="skip the compensation-branch leg")
    ap.add_argument("--no-bricks", action="store_true", help="skip the brick-token-order leg")
    ap.add_argument("--sweep", action="store_true")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    w = workloads.WORKLOADS[args.workload]
    if args.sparsity is not None:
        w = w.with_sparsity(args.sparsity)
    if args.block is not None and args.block != w.block:
        w = workloads.Workload(f"{w.name}_b{args.block}", w.cfg_id, w.B, w.H, w.d, w.grid, args.block, w.sparsity)
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
