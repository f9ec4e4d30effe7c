#!/usr/bin/env python
"""Benchmark of the W4A4KV4 hot path.

A step is one pass of the Llama-3-8B-shaped linear set at prefill (M = 2048 tokens, 4 of them
prefixed outlier tokens that the W4A4 path skips): for each of the four distinct layer inputs one
fused rotate+quantize call, then the W4A4 GEMMs (q|k|v and gate|up concatenated along N, o, down).
The metric is integer tera-operations per second over the GEMM work of the step (2*M*N*K), the
rotate+quantize kernels included in the time. Extra sections report the decode-shaped GEMMs and
the KV4 decode attention in GB/s. `--impl reference` times the CPU oracle on a bounded sample.
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

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "w4a4_prefill_linear_set_tops"
UNIT = "TOPS"
M_TOKENS = 2048
N_PREFIX = 4
NOMINAL_INT8_TOPS = 4500.0
NOMINAL_HBM_GBS = 8000.0


def linear_launches():
    """(name, N, K, had_block, input id) of the launches of one step; logical layers in the name."""
    from paper_2410_05265_b200 import inputs

    c = inputs.LLAMA3_8B
    h, kv, f = c["hidden"], c["kv_dim"], c["ffn"]
    return [
        ("q|k|v", h + 2 * kv, h, h, 0),
        ("o", h, h, h, 1),
        ("gate|up", 2 * f, h, h, 2),
        ("down", h, f, 2048, 3),
    ]


def step_ops(m_rows: int) -> float:
    return sum(2.0 * m_rows * n * k for _, n, k, _, _ in linear_launches())


def read_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm=d["hbm_gbs"], bf16=d["bf16_tflops"], bf16_sus=d.get("bf16_tflops_sustained", d["bf16_tflops"]),
                    src="measured")
    return dict(hbm=6650.0, bf16=1590.0, bf16_sus=1400.0, src="fallback")


def sha256_of(path: str) -> str:
    import hashlib

    with open(path, "rb") as f:
        return hashlib.sha256(f.read()).hexdigest()


def recorded_traffic():
    """DRAM bytes per launch of the dominant kernel as an ncu capture recorded them (a text file beside the profile
    summaries), or None when there is no record or the kernel's source has changed since it was taken."""
    rec = os.path.join(ROOT, "profiles", "roofline_traffic.txt")
    if not os.path.exists(rec):
        return None, "no ncu record"
    kv = {}
    for line in open(rec):
        if ":" in line and not line.lstrip().startswith("#"):
            k, v = line.split(":", 1)
            kv[k.strip()] = v.strip()
    # the kernel's sources (comma-separated) and the SHA-256 of each, in the same order
    srcs = [os.path.join(ROOT, t.strip()) for t in kv.get("source", "").split(",") if t.strip()]
    shas = [t.strip() for t in kv.get("source_sha256", "").split(",") if t.strip()]
    if not srcs or len(srcs) != len(shas) or any(not os.path.isfile(f) or sha256_of(f) != h for f, h in zip(srcs, shas)):
        return None, "kernel source changed since the ncu capture"
    return int(kv["dram_bytes_per_launch"]), f"ncu capture of the {kv.get('launch', '?')} launch (not measured by this run)"


def free_port() -> int:
    import socket

    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        return sock.getsockname()[1]


def spawn_ranks(n: int, script: str, argv) -> int:
    """Starts `script` as n ranks of one node (one process per GPU) under torch.distributed.run and returns its
    exit code; rank 0 of the child prints the result line."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
           "--master-port", str(free_port()), script] + list(argv)
    return subprocess.call(cmd)


def job_throughput(ms_local: float, steps: int, units_per_step_per_rank: float, world: int, dist=None, device=None):
    """Whole-job figures of a replicated (weak-scaling) run: every rank processes the same number of
    units per step, the job's step time is the slowest rank's, the value is all ranks' units over it.
    Returns (ms_per_step, units_per_second). With dist given, the maximum is taken over the ranks."""
    ms = float(ms_local)
    if dist is not None and world > 1:
        import torch

        t = torch.tensor([ms], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
    ms_per_step = ms / steps
    return ms_per_step, world * units_per_step_per_rank / (ms_per_step * 1e-3)


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 6:
                continue
            try:
                sm.append(float(f[0])), mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------------------------------- GPU arm
def build_workload(ctx, device):
    """Synthetic Llama-3-8B-shaped tensors, weights quantized offline, static scales calibrated on
    the seed-1 batch over the non-prefix rows."""
    import torch

    from paper_2410_05265_b200 import inputs

    L = linear_launches()
    acts, scales, wqs, sws = [], [], [], []
    for i, (name, N, K, had, inp) in enumerate(L):
        x = inputs.activations(M_TOKENS, K, seed=0, n_prefix=N_PREFIX, layer=inp, device=device)
        cal = inputs.activations(M_TOKENS, K, seed=1, n_prefix=N_PREFIX, layer=inp, device=device)
        s_a = ctx.calib_act_scale(cal, had, N_PREFIX)
        del cal
        W = inputs.weights(N, K, seed=2 + i, device=device)
        wq, s_w = ctx.quant_weights(W)
        del W
        acts.append(x), scales.append(s_a), wqs.append(wq), sws.append(s_w)
    torch.cuda.synchronize()
    return L, acts, scales, wqs, sws


def ctx_sm_count(torch, index: int) -> int:
    return torch.cuda.get_device_properties(index).multi_processor_count


def run_gpu(args):
    import torch

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dist = None
    if world > 1:
        import torch.distributed as dist

        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    else:
        torch.cuda.set_device(local)
    device = torch.device("cuda", local)

    from paper_2410_05265_b200 import binding, build as pq_build

    if rank == 0:
        pq_build.build()
    if dist:
        dist.barrier()
    ctx = binding.Context()
    L, acts, scales, wqs, sws = build_workload(ctx, device)
    m_rows = M_TOKENS - N_PREFIX
    xqs = [torch.zeros((M_TOKENS, K // 2), dtype=torch.uint8, device=device) for _, _, K, _, _ in L]
    outs = [torch.zeros((M_TOKENS, N), dtype=torch.bfloat16, device=device) for _, N, _, _, _ in L]

    def step(gemm_events=None):
        for i, (name, N, K, had, inp) in enumerate(L):
            if gemm_events is not None:
                eh = torch.cuda.Event(enable_timing=True)
                eh.record()
            ctx.hadamard_quant_act(acts[i], had, scales[i], N_PREFIX, out=xqs[i])
            if gemm_events is not None:
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
            ctx.w4a4_gemm(xqs[i], wqs[i], scales[i], sws[i], N_PREFIX, out=outs[i])
            if gemm_events is not None:
                e1.record()
                gemm_events.append((i, e0, e1))
                rot_events.append((i, eh, e0))

    def barrier():
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    ctx.check()
    # ---- timed region: device-resident inputs -------------------------------------------------
    # Two passes of the same K steps. The first has nothing but the eight launches of a step in the stream and gives
    # `value`; the second brackets every launch with CUDA events for the per-kernel figures. An event record between
    # two launches keeps the second from being placed while the first drains (programmatic dependent launch), so
    # the bracketed pass is a few percent slower per step; its time is reported beside the other.
    sampler = ClockSampler(local)
    gemm_events = []
    rot_events = []
    barrier()
    sampler.start()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(args.steps):
        step()
    t1.record()
    barrier()
    t2, t3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t2.record()
    for _ in range(args.steps):
        step(gemm_events)
    t3.record()
    barrier()
    clocks = sampler.stop()
    ctx.check()
    ms_per_step, ops_per_s = job_throughput(t0.elapsed_time(t1), args.steps, step_ops(m_rows), world, dist, device)
    value = ops_per_s / 1e12
    bracketed_ms_per_step = t2.elapsed_time(t3) / args.steps

    gemm_ms = sum(e0.elapsed_time(e1) for _, e0, e1 in gemm_events)
    per_shape = {}
    for i, e0, e1 in gemm_events:
        per_shape.setdefault(L[i][0], []).append(e0.elapsed_time(e1))
    gemm_ops = args.steps * step_ops(m_rows)
    peaks = read_peaks()
    # the rotate+quantize launch in front of every GEMM, between its own event and the GEMM's: 2.5 bytes per element
    rot_shape = {}
    for i, e0, e1 in rot_events:
        rot_shape.setdefault(L[i][0], []).append(e0.elapsed_time(e1))
    rotate_quant = {}
    for k, v in rot_shape.items():
        kk = next(kk for nm, n, kk, _, _ in L if nm == k)
        gbs = 2.5 * m_rows * kk / (statistics.mean(v) * 1e-3) / 1e9
        rotate_quant[k + " input"] = {"ms": round(statistics.mean(v), 4), "GB/s": round(gbs, 1), "frac_measured_hbm": round(gbs / peaks["hbm"], 3)}
    # Denominator: dense INT8 is nominally 2x dense bf16 (4.5 vs 2.25 PFLOP/s); of the two measured bf16 figures the
    # burst one applies to a timed region shorter than a second (the chip does not reach its power-capped clock in
    # that time), the sustained one to a longer region.
    timed_s = t2.elapsed_time(t3) * 1e-3  # the pass the per-launch events come from
    peak_kind = "burst" if timed_s < 1.0 else "sustained"
    int8_peak = 2.0 * (peaks["bf16"] if timed_s < 1.0 else peaks["bf16_sus"])
    achieved = gemm_ops / (gemm_ms * 1e-3) / 1e12
    # attainable rate: resident-operand kind::i8 MMAs (no loads, no expansion), at the clock sampled during the step
    attainable = None
    try:
        iters = 8192
        cyc = ctx.probe_i8_mma(iters)
        torch.cuda.synchronize()
        cyc = cyc[cyc > 0].double()
        mac_per_clk = float((iters * 128.0 * 256.0 * 32.0 / cyc).median())
        mhz = clocks.get("sm_mhz") or clocks.get("sm_max_mhz") or 0.0
        att_tops = mac_per_clk * 2.0 * ctx_sm_count(torch, local) * mhz * 1e6 / 1e12
        attainable = {"mac_per_clk_per_sm": round(mac_per_clk, 1), "sm_mhz": mhz, "TOPS": round(att_tops, 1),
                      "frac": round(achieved / att_tops, 4) if att_tops else None,
                      "how": "8192 resident-operand tcgen05.mma kind::i8 128x256x32 per SM, median over SMs, at the step's median SM clock"}
    except Exception as e:  # the probe never takes the line down
        attainable = {"error": repr(e)}
    traffic, traffic_note = recorded_traffic()
    roofline = {
        "kernel": "gemm_w4a4_pair_kernel (the four GEMM launches of the step)", "bound": "tensor", "achieved": round(achieved, 1),
        "peak": round(int8_peak, 1), "unit": "TOPS", "frac": round(achieved / int8_peak, 4), "traffic": traffic, "traffic_note": traffic_note,
        "peak_source": f"2 x bf16 {peak_kind} GEMM of {peaks['src']} (timed region {timed_s:.2f} s)",
        "frac_of_nominal_4500": round(achieved / NOMINAL_INT8_TOPS, 4), "attainable_int8": attainable,
        "per_launch_pass_ms_per_step": round(bracketed_ms_per_step, 4),
        "per_launch": {k: {"ms": round(statistics.mean(v), 4),
                           "tops": round(2.0 * m_rows * next(n * kk for nm, n, kk, _, _ in L if nm == k) /
                                         (statistics.mean(v) * 1e-3) / 1e12, 1)} for k, v in per_shape.items()},
    }

    # ---- end to end: host buffers in, host buffers out, through the same calls ----------------------
    h_acts = [a.cpu().pin_memory() for a in acts]
    h_outs = [torch.empty(o.shape, dtype=o.dtype).pin_memory() for o in outs]
    d_acts = [torch.empty_like(a) for a in acts]
    h2d = sum(a.numel() * a.element_size() for a in h_acts)
    d2h = sum(o.numel() * o.element_size() for o in h_outs)

    # Three streams, as a caller with host buffers would run it: uploads, the library calls, and downloads
    # overlap across the four linears (PCIe is full duplex and has its own copy engines); events order each
    # buffer's upload -> use -> download, and its reuse in the next step.
    st_in, st_run, st_out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
    ev_in = [torch.cuda.Event() for _ in L]
    ev_run = [torch.cuda.Event() for _ in L]
    ev_out = [torch.cuda.Event() for _ in L]

    def e2e_step():
        for i, (name, N, K, had, inp) in enumerate(L):
            with torch.cuda.stream(st_in):
                st_in.wait_event(ev_run[i])          # the previous step's kernels are done with this input buffer
                d_acts[i].copy_(h_acts[i], non_blocking=True)
                ev_in[i].record(st_in)
            with torch.cuda.stream(st_run):
                st_run.wait_event(ev_in[i])
                st_run.wait_event(ev_out[i])         # the previous step's download of this output buffer is done
                ctx.hadamard_quant_act(d_acts[i], had, scales[i], N_PREFIX, out=xqs[i])
                ctx.w4a4_gemm(xqs[i], wqs[i], scales[i], sws[i], N_PREFIX, out=outs[i])
                ev_run[i].record(st_run)
            with torch.cuda.stream(st_out):
                st_out.wait_event(ev_run[i])
                h_outs[i].copy_(outs[i], non_blocking=True)
                ev_out[i].record(st_out)

    e2e_steps = max(2, min(args.steps, 10))
    e2e_step()
    barrier()
    w0 = time.perf_counter()
    for _ in range(e2e_steps):
        e2e_step()
    barrier()
    e2e_s = time.perf_counter() - w0
    if dist:
        tmax = torch.tensor([e2e_s], device=device)
        dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
        e2e_s = float(tmax.item())
    e2e_value = world * step_ops(m_rows) * e2e_steps / e2e_s / 1e12
    # the pipelined path delivers the same bytes as the device-resident step
    step()
    barrier()
    e2e_ok = all(torch.equal(h_outs[i], outs[i].cpu()) for i in (1, 3))

    sections, cpu_baseline = None, None
    if rank == 0 and world == 1 and not args.no_sections:
        sections = {}
        try:
            sections["config0_single_linear_256x4096x4096"] = section_config0(ctx, device, peaks)
            sections["w4a8_prefill_linear_set"] = section_w4a8(ctx, device, peaks, acts, wqs, sws)
            sections["w4a4_dynamic_per_token_linear_set"] = section_dynamic(ctx, device, peaks, acts, wqs, sws)
            sections["w4a4_byte_codes_linear_set"] = section_w4a4_byte_codes(ctx, device, peaks, acts, scales, wqs, sws)
            sections["decode_gemm"] = section_decode_gemm(ctx, device, peaks)
            sections["decode_attention"] = section_decode_attention(ctx, device, peaks)
            sections["block_llama3_70b_prefill4096"] = section_block(ctx, device, peaks)
        except Exception as e:  # sections never take the main line down
            sections["error"] = repr(e)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu_baseline = oracle_sample(1536)  # about 10-15 s of host work on 16 cores

    if rank == 0:
        line = {
            "metric": METRIC, "value": round(value, 2), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": round(ms_per_step, 4), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "s4 x s4 -> s32 (tcgen05 kind::i8 on 16*code), fp32 epilogue, bf16 out",
            "data": "synthetic",
            "config": {"workload": "configs[1]: Llama-3-8B linear set, prefill M=2048 (4 prefixed rows skipped), batch 1",
                       "launches_per_step": "4 x hadamard_quant_act + 4 x w4a4_gemm (q|k|v and gate|up concatenated along N)",
                       "l2": "inputs larger than L2: a step touches ~400 MB (weights 109 MB, activations 109 MB, outputs 176 MB) against 126 MB",
                       "parallelism": "replicas only" if world > 1 else "single GPU"},
            "clocks": clocks, "roofline": roofline,
            "e2e": {"value": round(e2e_value, 2), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "steps": e2e_steps, "pipeline": "uploads, library calls and downloads on three streams", "matches_device_step": e2e_ok},
            "gpu_launches": args.steps * 2 * len(L),
            "rotate_quant_per_launch": rotate_quant,
        }
        if cpu_baseline:
            line["cpu_baseline"] = cpu_baseline
        if sections:
            line["sections"] = sections
        print(json.dumps(line))
    if dist:
        dist.barrier()
        dist.destroy_process_group()


def _graph_time(torch, fn, n_inner, reps=5):
    """Captures n_inner calls of fn(i) in a CUDA graph and returns the best ms per call."""
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        for i in range(3):
            fn(i)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            for i in range(n_inner):
                fn(i)
        g.replay()
        torch.cuda.synchronize()
        best = float("inf")
        for _ in range(reps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            g.replay()
            e1.record()
            torch.cuda.synchronize()
            best = min(best, e0.elapsed_time(e1) / n_inner)
    torch.cuda.current_stream().wait_stream(s)
    return best


def section_config0(ctx, device, peaks):
    """configs[0]: one W4A4 linear, 256 tokens, 4096 -> 4096: rotate+quantize, GEMM, and both chained, each as 200
    calls in a CUDA graph. 8.6 GOP against ~13 MB: a ridge-point, launch-bound shape (16 pair tiles on 74 CTA pairs)."""
    import torch

    from paper_2410_05265_b200 import inputs

    M, K, N = 256, 4096, 4096
    x = inputs.activations(M, K, seed=0, device=device)
    cal = inputs.activations(M, K, seed=1, device=device)
    s_a = ctx.calib_act_scale(cal, K)
    wq, s_w = ctx.quant_weights(inputs.weights(N, K, seed=2, device=device))
    xq = torch.zeros((M, K // 2), dtype=torch.uint8, device=device)
    out = torch.zeros((M, N), dtype=torch.bfloat16, device=device)
    ms_q = _graph_time(torch, lambda i: ctx.hadamard_quant_act(x, K, s_a, out=xq), 200)
    ms_g = _graph_time(torch, lambda i: ctx.w4a4_gemm(xq, wq, s_a, s_w, out=out), 200)

    def both(i):
        ctx.hadamard_quant_act(x, K, s_a, out=xq)
        ctx.w4a4_gemm(xq, wq, s_a, s_w, out=out)

    ms_b = _graph_time(torch, both, 200)
    ctx.check()
    ops = 2.0 * M * N * K
    return {"rotate_quant_us": round(ms_q * 1e3, 3), "gemm_us": round(ms_g * 1e3, 3), "chained_us": round(ms_b * 1e3, 3),
            "gemm_TOPS": round(ops / (ms_g * 1e-3) / 1e12, 1), "chained_TOPS": round(ops / (ms_b * 1e-3) / 1e12, 1),
            "rotate_quant_GBs": round(2.5 * M * K / (ms_q * 1e-3) / 1e9, 1),
            "note": "launch-bound: 16 tiles of 256 x 256 on 74 CTA pairs, operands resident in L2 across the repeated calls"}


def section_decode_gemm(ctx, device, peaks):
    """configs[2]: M in {1,4,16} through the Llama-3-8B shapes; 8 distinct weight copies visited
    round-robin (872 MB > L2) so the weights stream from HBM; 1000 calls in a CUDA graph."""
    import torch

    from paper_2410_05265_b200 import inputs

    res = {}
    n_copies = 8
    for name, N, K, had, inp in linear_launches():
        wq = torch.randint(0, 256, (n_copies, N, K // 2), dtype=torch.uint8, device=device)
        s_w = torch.full((N,), 0.003, device=device)
        s_a = torch.full((1,), 0.05, device=device)
        for M in (1, 4, 16):
            xq = torch.randint(0, 256, (M, K // 2), dtype=torch.uint8, device=device)
            out = torch.zeros((M, N), dtype=torch.bfloat16, device=device)
            ms = _graph_time(torch, lambda i: ctx.w4a4_gemm(xq, wq[i % n_copies], s_a, s_w, out=out), 1000)
            by = N * K // 2 + N * 4 + M * K // 2 + M * N * 2
            gbs = by / (ms * 1e-3) / 1e9
            res[f"{name} M={M}"] = {"us": round(ms * 1e3, 3), "GB/s": round(gbs, 1), "frac_measured_hbm": round(gbs / peaks["hbm"], 3),
                                    "frac_nominal_8TBs": round(gbs / NOMINAL_HBM_GBS, 3)}
            if M == 1:  # the same call on one weight copy: after the first call the weights come from L2, not from HBM
                ms_l2 = _graph_time(torch, lambda i: ctx.w4a4_gemm(xq, wq[0], s_a, s_w, out=out), 1000)
                res[f"{name} M={M}"]["L2_resident_us"] = round(ms_l2 * 1e3, 3)
                res[f"{name} M={M}"]["L2_resident_GB/s (not an HBM figure)"] = round(by / (ms_l2 * 1e-3) / 1e9, 1)
        del wq
    ctx.check()
    for M in (1, 4, 16):  # the whole layer set of one decode step
        us = sum(v["us"] for k, v in res.items() if k.endswith(f"M={M}"))
        by = sum(N * K // 2 + N * 4 + M * K // 2 + M * N * 2 for _, N, K, _, _ in linear_launches())
        res[f"layer set M={M}"] = {"us": round(us, 3), "frac_measured_hbm": round(by / (us * 1e-6) / 1e9 / peaks["hbm"], 3)}
    return res


def section_decode_attention(ctx, device, peaks):
    """configs[3]: batch 8, 32 query / 8 KV heads, head_dim 128, 4 fp16 prefix entries + 4092 INT4
    entries; 32 distinct cache layers (1.07 GB) visited round-robin; one append + one attention per step."""
    import torch

    from paper_2410_05265_b200 import binding, inputs

    B, Hq, Hkv, D, P, T, Tmax, layers = 8, 32, 8, 128, 4, 4091, 4096, 32
    pk = inputs.prefix_kv(Hkv, P, D, 0, "k", 50.0, device=device)
    pv = inputs.prefix_kv(Hkv, P, D, 0, "v", 50.0, device=device)
    s_k = torch.full((Hkv,), 4.5 / 7, device=device)
    s_v = torch.full((Hkv,), 4.5 / 7, device=device)
    caches = []
    for _ in range(layers):
        kq = torch.randint(0, 256, (B, Hkv, Tmax, D // 2), dtype=torch.uint8, device=device)
        vq = torch.randint(0, 256, (B, Hkv, Tmax, D // 2), dtype=torch.uint8, device=device)
        length = torch.full((B,), T, dtype=torch.int32, device=device)
        caches.append(binding.KV4Cache(pk, pv, kq, vq, s_k, s_v, length, Hq))
    q = inputs.queries(B, Hq, D, 0, device=device)
    k1 = inputs.kv_tensor(B, 1, Hkv, D, 0, "k", device=device)
    v1 = inputs.kv_tensor(B, 1, Hkv, D, 0, "v", device=device)
    ws = ctx.decode_attn_workspace(caches[0])
    out = torch.empty_like(q)
    sm = 1 / math.sqrt(D)

    def reset():
        for c in caches:
            c.length.fill_(T)

    def both(i):
        c = caches[i % layers]
        ctx.kv4_append(c, k1, v1)
        ctx.decode_attn(c, q, sm, ws, out=out)

    def attn_only(i):
        ctx.decode_attn(caches[i % layers], q, sm, ws, out=out)

    def append_only(i):
        ctx.kv4_append(caches[i % layers], k1, v1)

    reset()
    ms_attn = _graph_time(torch, attn_only, 320)
    # each layer is appended to at most (3 + 32 * 7) / 32 + 1 < 9 times below: start low enough
    for c in caches:
        c.length.fill_(T - 40)
    ms_app = _graph_time(torch, append_only, 32, reps=3)
    for c in caches:
        c.length.fill_(T - 40)
    ms_both = _graph_time(torch, both, 32, reps=3)
    for c in caches:
        c.length.fill_(T - 40)

    def fused(i):
        ctx.kv4_append_decode_attn(caches[i % layers], k1, v1, q, sm, ws, out=out)

    ms_fused = _graph_time(torch, fused, 32, reps=3)
    ctx.check()
    # the comparison setting (Table 1, O1): group-wise dynamic KV, one step per cached vector, on the same codes
    dyn = [binding.KV4Cache(pk, pv, c.kq, c.vq, None, None, c.length, Hq, sk_tok=torch.rand((B, Hkv, Tmax), device=device) * 0.6 + 0.3,
                            sv_tok=torch.rand((B, Hkv, Tmax), device=device) * 0.6 + 0.3) for c in caches]
    for c in caches:
        c.length.fill_(T - 40)
    ms_dyn_attn = _graph_time(torch, lambda i: ctx.decode_attn(dyn[i % layers], q, sm, ws, out=out), 64, reps=3)
    ms_dyn_app = _graph_time(torch, lambda i: ctx.kv4_append(dyn[i % layers], k1, v1), 32, reps=3)
    ctx.check()
    del dyn
    # one long sequence (Llama-3-70B heads, 32K context): few (sequence, head) pairs, several clusters of splits each
    del caches
    Bl, Hql, Tl, Tmaxl, nl = 1, 64, 32764, 32768, 10
    long_caches = [binding.KV4Cache(pk, pv, torch.randint(0, 256, (Bl, Hkv, Tmaxl, D // 2), dtype=torch.uint8, device=device),
                                    torch.randint(0, 256, (Bl, Hkv, Tmaxl, D // 2), dtype=torch.uint8, device=device), s_k, s_v,
                                    torch.full((Bl,), Tl, dtype=torch.int32, device=device), Hql) for _ in range(nl)]
    ql = inputs.queries(Bl, Hql, D, 0, device=device)
    wsl = ctx.decode_attn_workspace(long_caches[0])
    outl = torch.empty_like(ql)
    ms_long = _graph_time(torch, lambda i: ctx.decode_attn(long_caches[i % nl], ql, sm, wsl, out=outl), 8 * nl)
    ctx.check()
    del long_caches
    by_long = Bl * Hkv * Tl * D
    by = B * Hkv * (T + 1) * (D // 2) * 2 + Hkv * P * D * 2 * 2 + 2 * B * Hq * D * 2 + 2 * Hkv * 4
    gbs = by / (ms_attn * 1e-3) / 1e9
    return {"attention_us": round(ms_attn * 1e3, 3), "append_us": round(ms_app * 1e3, 3), "append+attention_us": round(ms_both * 1e3, 3),
            "append+attention_one_launch_us": round(ms_fused * 1e3, 3),
            "groupwise_dynamic_kv (Table 1 O1)": {"attention_us": round(ms_dyn_attn * 1e3, 3), "append_us": round(ms_dyn_app * 1e3, 3),
                                                  "note": "per-vector steps (+2 MB of step reads), plain fp32 kernel: the setting the static path is compared with"},
            "append+attention_one_launch_frac_measured_hbm": round(by / (ms_fused * 1e-3) / 1e9 / peaks["hbm"], 3),
            "long_context_b1_hq64_t32764": {"attention_us": round(ms_long * 1e3, 3),
                                            "frac_measured_hbm": round(by_long / (ms_long * 1e-3) / 1e9 / peaks["hbm"], 3)},
            "GB/s": round(gbs, 1), "frac_measured_hbm": round(gbs / peaks["hbm"], 3), "frac_nominal_8TBs": round(gbs / NOMINAL_HBM_GBS, 3),
            "bytes_per_step": by}


def section_w4a8(ctx, device, peaks, acts, wqs, sws):
    """The linear set of configs[1] at the W4A8 precision (Sec. 5.1): 8-bit static per-tensor activation
    codes, the same packed 4-bit weights; timed like the main step (events around a loop of steps, GEMM
    launches timed on their own as well)."""
    import torch

    L = linear_launches()
    m_rows = M_TOKENS - N_PREFIX
    scales = [ctx.calib_act_scale8(acts[i], had, N_PREFIX) for i, (_, _, _, had, _) in enumerate(L)]
    xqs = [torch.zeros((M_TOKENS, K), dtype=torch.int8, device=device) for _, _, K, _, _ in L]
    outs = [torch.zeros((M_TOKENS, N), dtype=torch.bfloat16, device=device) for _, N, _, _, _ in L]
    ev = []

    def step(timed):
        for i, (name, N, K, had, inp) in enumerate(L):
            ctx.hadamard_quant_act8(acts[i], had, scales[i], N_PREFIX, out=xqs[i])
            if timed:
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
            ctx.w4a8_gemm(xqs[i], wqs[i], scales[i], sws[i], N_PREFIX, out=outs[i])
            if timed:
                e1.record()
                ev.append((name, e0, e1))

    steps = 50
    for _ in range(5):
        step(False)
    torch.cuda.synchronize()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(steps):
        step(False)  # the step's launches alone in the stream, as in the main timed pass
    t1.record()
    torch.cuda.synchronize()
    for _ in range(steps):
        step(True)   # per-launch events from a second pass
    torch.cuda.synchronize()
    ctx.check()
    ms = t0.elapsed_time(t1) / steps
    per = {}
    for name, e0, e1 in ev:
        per.setdefault(name, []).append(e0.elapsed_time(e1))
    gemm_ms = sum(statistics.mean(v) for v in per.values())
    int8_peak = 2.0 * peaks["bf16"]  # a region of a few milliseconds: the burst figure applies
    gemm_tops = step_ops(m_rows) / (gemm_ms * 1e-3) / 1e12
    return {"ms_per_step": round(ms, 4), "TOPS": round(step_ops(m_rows) / (ms * 1e-3) / 1e12, 1), "gemm_TOPS": round(gemm_tops, 1),
            "gemm_frac_of_2x_bf16_burst": round(gemm_tops / int8_peak, 4), "gemm_frac_of_nominal_4500": round(gemm_tops / NOMINAL_INT8_TOPS, 4),
            "per_launch": {k: {"ms": round(statistics.mean(v), 4),
                               "tops": round(2.0 * m_rows * next(n * kk for nm, n, kk, _, _ in L if nm == k) / (statistics.mean(v) * 1e-3) / 1e12, 1)}
                           for k, v in per.items()}}


def section_w4a4_byte_codes(ctx, device, peaks, acts, scales, wqs, sws):
    """The linear set of configs[1] with the 4-bit activation codes stored one per byte (pq_hadamard_quant_act_c8 +
    pq_w4a8_gemm): W4A4's codes, sums and outputs, without the expansion of the token operand in the GEMM and with
    twice the activation bytes. Beside the packed path of the scope table, which the headline measures."""
    import torch

    L = linear_launches()
    m_rows = M_TOKENS - N_PREFIX
    xqs = [torch.zeros((M_TOKENS, K), dtype=torch.int8, device=device) for _, _, K, _, _ in L]
    outs = [torch.zeros((M_TOKENS, N), dtype=torch.bfloat16, device=device) for _, N, _, _, _ in L]

    def step():
        for i, (name, N, K, had, inp) in enumerate(L):
            ctx.hadamard_quant_act_c8(acts[i], had, scales[i], N_PREFIX, out=xqs[i])
            ctx.w4a8_gemm(xqs[i], wqs[i], scales[i], sws[i], N_PREFIX, out=outs[i])

    steps = 50
    for _ in range(5):
        step()
    torch.cuda.synchronize()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(steps):
        step()
    t1.record()
    torch.cuda.synchronize()
    ctx.check()
    ms = t0.elapsed_time(t1) / steps
    return {"ms_per_step": round(ms, 4), "TOPS": round(step_ops(m_rows) / (ms * 1e-3) / 1e12, 1),
            "note": "same codes, sums and outputs as the packed path (asserted by the GPU tests); activations take M x K bytes instead of M x K / 2"}


def section_dynamic(ctx, device, peaks, acts, wqs, sws):
    """The linear set of configs[1] in the per-token dynamic setting (Table 1, O1): per linear one pass for the
    token steps, one for the codes, then the GEMM with the per-token epilogue. The paper's comparison
    setting: it reports the static path as the faster one."""
    import torch

    L = linear_launches()
    m_rows = M_TOKENS - N_PREFIX
    s_tok = [torch.zeros((M_TOKENS,), dtype=torch.float32, device=device) for _ in L]
    xqs = [torch.zeros((M_TOKENS, K // 2), dtype=torch.uint8, device=device) for _, _, K, _, _ in L]
    outs = [torch.zeros((M_TOKENS, N), dtype=torch.bfloat16, device=device) for _, N, _, _, _ in L]

    def step():
        for i, (name, N, K, had, inp) in enumerate(L):
            ctx.dyn_hadamard_quant_act(acts[i], had, 1.0, N_PREFIX, s_tok=s_tok[i], out=xqs[i])
            ctx.w4a4_gemm_rows(xqs[i], wqs[i], s_tok[i], sws[i], N_PREFIX, out=outs[i])

    steps = 50
    for _ in range(5):
        step()
    torch.cuda.synchronize()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(steps):
        step()
    t1.record()
    torch.cuda.synchronize()
    ctx.check()
    ms = t0.elapsed_time(t1) / steps
    return {"ms_per_step": round(ms, 4), "TOPS": round(step_ops(m_rows) / (ms * 1e-3) / 1e12, 1),
            "launches_per_step": "3 x (dyn_hadamard_quant_act in one pass + w4a4_gemm_rows) for the 4096-wide inputs, "
                                 "1 x (step pass + memset + code pass + w4a4_gemm_rows) for the down projection (7 blocks per row)"}


def section_block(ctx, device, peaks):
    """configs[4]: one Llama-3-70B-shaped W4A4KV4 block at prefill, 4096 ordinary tokens after 4 prefixed
    tokens whose K/V sit in the cache in fp16; static scales from a seed-1 calibration pass."""
    import torch

    from paper_2410_05265_b200 import block, inputs

    c = inputs.LLAMA3_70B
    T, P, D = 4096, 4, c["head_dim"]
    shape = block.BlockShape(hidden=c["hidden"], n_q_heads=c["n_q_heads"], n_kv_heads=c["n_kv_heads"], ffn=c["ffn"])
    qd, kvd = shape.q_dim, shape.kv_dim
    mk = lambda n, k, seed: inputs.weights(n, k, seed=seed, device=device)
    blk = block.Block(ctx, shape, mk(qd + 2 * kvd, shape.hidden, 2), mk(shape.hidden, qd, 3), mk(2 * shape.ffn, shape.hidden, 4),
                      mk(shape.hidden, shape.ffn, 5), torch.ones(shape.hidden, dtype=torch.bfloat16, device=device),
                      torch.ones(shape.hidden, dtype=torch.bfloat16, device=device),
                      inputs.prefix_kv(c["n_kv_heads"], P, D, 0, "k", 50.0, device=device),
                      inputs.prefix_kv(c["n_kv_heads"], P, D, 0, "v", 50.0, device=device), t_max=T)
    torch.cuda.synchronize()
    blk.forward(inputs.activations(T, shape.hidden, seed=1, device=device), calibrate=True)
    x = inputs.activations(T, shape.hidden, seed=0, device=device)
    for _ in range(3):
        blk.forward(x)
    ctx.check()
    reps = 10
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        blk.forward(x)
    e1.record()
    torch.cuda.synchronize()
    ctx.check()
    ms = e0.elapsed_time(e1) / reps
    # per-stage share: one more pass with an event after every stage
    marks = []

    def tap(name, t):
        ev = torch.cuda.Event(enable_timing=True)
        ev.record()
        marks.append((name, ev))

    start = torch.cuda.Event(enable_timing=True)
    start.record()
    blk.forward(x, tap=tap)
    torch.cuda.synchronize()
    stages, prev = {}, start
    for name, ev in marks:
        if name in ("vq", "y"):
            continue
        stages[name] = round(prev.elapsed_time(ev), 4)
        prev = ev
    # the SwiGLU + rotate + quantize launch of the un-tapped pass, on its own
    gu_buf = blk.buf["gu"]
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    f0.record()
    for _ in range(reps):
        ctx.swiglu_hadamard_quant_act(gu_buf[:, : shape.ffn], gu_buf[:, shape.ffn:], shape.had_block(shape.ffn), blk.s_a[3], out=blk.buf["xq_f"])
    f1.record()
    torch.cuda.synchronize()
    fused_ms = f0.elapsed_time(f1) / reps
    # the same block with the online head-wise rotation R3 of q and k fused into the rotary step
    shape.r3 = True
    blk.forward(inputs.activations(T, shape.hidden, seed=1, device=device), calibrate=True)
    for _ in range(2):
        blk.forward(x)
    marks.clear()
    r0, r1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    r0.record()
    for _ in range(reps):
        blk.forward(x)
    r1.record()
    torch.cuda.synchronize()
    ms_r3 = r0.elapsed_time(r1) / reps
    start3 = torch.cuda.Event(enable_timing=True)
    start3.record()
    blk.forward(x, tap=tap)
    torch.cuda.synchronize()
    prev3, rope_r3 = start3, None
    for name, ev in marks:
        if name == "qkv_rope":
            rope_r3 = round(prev3.elapsed_time(ev), 4)
        prev3 = ev
    shape.r3 = False
    ctx.check()
    gemm_ops = 2.0 * T * shape.hidden * (qd + 2 * kvd + qd + 2 * shape.ffn + shape.ffn)
    attn_flops = 4.0 * D * c["n_q_heads"] * (T * (T + 1) / 2 + T * P)
    gemm_ms = sum(stages[k] for k in ("qkv", "o", "gu", "d"))
    return {"tokens_per_s": round(T / (ms * 1e-3), 1), "ms": round(ms, 4), "tokens": T, "n_prefix": P,
            "gemm_TOPS": round(gemm_ops / (gemm_ms * 1e-3) / 1e12, 1), "gemm_share": round(gemm_ms / sum(stages.values()), 3),
            "attention_TFLOPS": round(attn_flops / (stages["attn"] * 1e-3) / 1e12, 1), "stage_ms": stages,
            "swiglu_rotate_quant_fused_ms": round(fused_ms, 4),
            "stage_note": "stage_ms comes from a pass that stops after every stage (SwiGLU as its own launch: act + xq4); the timed pass fuses them",
            "with_r3": {"ms": round(ms_r3, 4), "rope_rotate_ms": rope_r3},
            "launches": block.Block.LAUNCHES_PER_FORWARD}


# ------------------------------------------------------------------------------------- CPU oracle arms
def oracle_sample(rows: int):
    """Times the CPU oracle, as it stands, on `rows` non-prefix token rows of the same workload
    through all seven linears (rotation, quantizer, integer GEMM, dequantization)."""
    import numpy as np

    from oracle import pq_oracle as orc
    from paper_2410_05265_b200 import inputs

    L = linear_launches()
    prepared = []
    rng = np.random.default_rng(0)
    for i, (name, N, K, had, inp) in enumerate(L):
        x = inputs.activations(N_PREFIX + rows, K, seed=0, n_prefix=N_PREFIX, layer=inp)
        wq = rng.integers(0, 256, (N, K // 2)).astype(np.uint8)  # weight codes: offline work, not timed
        s_w = np.full((N,), 0.003, np.float32)
        prepared.append((inputs.bits(x), wq, s_w, K, had))
    t0 = time.perf_counter()
    for xb, wq, s_w, K, had in prepared:
        s_a = np.float32(0.25)
        xq = orc.quant_act(xb, had, s_a, N_PREFIX)
        acc = orc.gemm_i4(xq[N_PREFIX:], wq)
        orc.dequant_bf16(acc, s_a, s_w)
    dt = time.perf_counter() - t0
    return {"value": round(step_ops(rows) / dt / 1e12, 6), "unit": UNIT, "cores": orc.get_threads(), "kind": "oracle",
            "sample": f"{rows} of {M_TOKENS - N_PREFIX} non-prefix token rows through all 7 linears (rotate, quantize, int GEMM, dequant)",
            "seconds": round(dt, 2)}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    rows = 4
    for _ in range(args.warmup):
        oracle_sample(1)
    t0 = time.perf_counter()
    last = None
    for _ in range(args.steps):
        last = oracle_sample(rows)
    dt = time.perf_counter() - t0
    value = step_ops(rows) * args.steps / dt / 1e12
    line = {
        "impl": "reference", "metric": METRIC, "value": round(value, 6), "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(dt / args.steps * 1e3, 2), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64 / int64 (CPU oracle)", "data": "synthetic",
        "config": {"workload": "configs[1]: Llama-3-8B linear set, prefill M=2048 (4 prefixed rows skipped), batch 1",
                   "sample": f"each step = {rows} token rows through all 7 linears"},
        "cpu_baseline": {"value": round(value, 6), "unit": UNIT, "cores": last["cores"], "kind": "oracle", "sample": last["sample"]},
        "e2e": {"value": round(value, 6), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


def run_case(args):
    """Runs one kernel a few times on a small synthetic case (the command ncu captures are made with)."""
    import torch

    from paper_2410_05265_b200 import binding, inputs

    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    ctx = binding.Context()
    name, _, rest = args.case.partition(":")
    dims = [int(v) for v in rest.split(",")] if rest else []
    reps = args.steps
    if name == "gemm":
        M, N, K = dims or [2048, 28672, 4096]
        xq = torch.randint(0, 256, (M, K // 2), dtype=torch.uint8, device=dev)
        wq = torch.randint(0, 256, (N, K // 2), dtype=torch.uint8, device=dev)
        s_a, s_w = torch.full((1,), 0.05, device=dev), torch.full((N,), 0.003, device=dev)
        out = torch.zeros((M, N), dtype=torch.bfloat16, device=dev)
        fn = lambda: ctx.w4a4_gemm(xq, wq, s_a, s_w, out=out)
        work = 2.0 * M * N * K
    elif name == "gemm8":
        M, N, K = dims or [2048, 28672, 4096]
        xq8 = torch.randint(-128, 128, (M, K), dtype=torch.int8, device=dev)
        wq = torch.randint(0, 256, (N, K // 2), dtype=torch.uint8, device=dev)
        s_a, s_w = torch.full((1,), 0.003, device=dev), torch.full((N,), 0.003, device=dev)
        out = torch.zeros((M, N), dtype=torch.bfloat16, device=dev)
        fn = lambda: ctx.w4a8_gemm(xq8, wq, s_a, s_w, out=out)
        work = 2.0 * M * N * K
    elif name == "hadamard8":
        M, K, B = dims or [8192, 14336, 2048]
        x = inputs.activations(M, K, seed=0, device=dev)
        s_a = ctx.calib_act_scale8(x, B)
        out = torch.zeros((M, K), dtype=torch.int8, device=dev)
        fn = lambda: ctx.hadamard_quant_act8(x, B, s_a, out=out)
        work = 3.0 * M * K
    elif name == "hadamard":
        M, K, B = dims or [8192, 14336, 2048]
        x = inputs.activations(M, K, seed=0, device=dev)
        s_a = ctx.calib_act_scale(x, B)
        out = torch.zeros((M, K // 2), dtype=torch.uint8, device=dev)
        fn = lambda: ctx.hadamard_quant_act(x, B, s_a, out=out)
        work = 2.5 * M * K
    elif name == "attn":
        B, Hq, Hkv, T, layers = dims or [8, 32, 8, 4092, 8]
        D, P = 128, 4
        pk = inputs.prefix_kv(Hkv, P, D, 0, "k", 50.0, device=dev)
        pv = inputs.prefix_kv(Hkv, P, D, 0, "v", 50.0, device=dev)
        s = torch.full((Hkv,), 4.5 / 7, device=dev)
        caches = [binding.KV4Cache(pk, pv, torch.randint(0, 256, (B, Hkv, T + 4, D // 2), dtype=torch.uint8, device=dev),
                                   torch.randint(0, 256, (B, Hkv, T + 4, D // 2), dtype=torch.uint8, device=dev), s, s,
                                   torch.full((B,), T, dtype=torch.int32, device=dev), Hq) for _ in range(layers)]
        q = inputs.queries(B, Hq, D, 0, device=dev)
        ws = ctx.decode_attn_workspace(caches[0])
        out = torch.empty_like(q)
        it = iter(range(10**9))
        fn = lambda: ctx.decode_attn(caches[next(it) % layers], q, 1 / math.sqrt(D), ws, out=out)
        work = float(B * Hkv * T * D)
    elif name == "prefill":
        T, Hq, Hkv = dims or [4096, 64, 8]
        D, P = 128, 4
        pk = inputs.prefix_kv(Hkv, P, D, 0, "k", 50.0, device=dev)
        pv = inputs.prefix_kv(Hkv, P, D, 0, "v", 50.0, device=dev)
        s = torch.full((Hkv,), 4.5 / 7, device=dev)
        cache = binding.KV4Cache(pk, pv, torch.randint(0, 256, (1, Hkv, T, D // 2), dtype=torch.uint8, device=dev),
                                 torch.randint(0, 256, (1, Hkv, T, D // 2), dtype=torch.uint8, device=dev), s, s,
                                 torch.full((1,), T, dtype=torch.int32, device=dev), Hq)
        q = inputs.kv_tensor(1, T, Hq, D, 0, "k", device=dev)[0].contiguous()
        out = torch.empty_like(q)
        fn = lambda: ctx.prefill_attn(cache, 0, q, 1 / math.sqrt(D), out=out)
        work = 4.0 * D * Hq * (T * (T + 1) / 2 + T * P)
    else:
        raise SystemExit(f"unknown case {name}")
    for _ in range(3):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    ctx.check()
    ms = e0.elapsed_time(e1) / reps
    print(json.dumps({"case": args.case, "ms": round(ms, 5), "work_per_s": work / (ms * 1e-3)}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--case", default=None, help="run one kernel on a small case: gemm:M,N,K | hadamard:M,K,B | attn:B,Hq,Hkv,T,layers | prefill:T,Hq,Hkv")
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-sections", action="store_true", help="skip the decode GEMM / decode attention sections")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.case:
        run_case(args)
    elif args.impl == "reference":
        run_reference(args)
    elif args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started as a plain program: become N ranks, one per GPU (rank 0 prints the line)
        sys.exit(spawn_ranks(args.gpus, os.path.abspath(__file__), sys.argv[1:]))
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
