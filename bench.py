"""Benchmark of the FP8 SLA forward: one step = quantise Q, K, V + block plan + forward on one synthetic batch.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload vggt8] [--impl ours|reference]

Prints ONE JSON line (rank 0).  `value` is dense-equivalent TFLOP/s (4*B*H*N^2*D per step over the step time)
with the bf16 sources resident in HBM; `e2e` is the same metric with pinned-host sources copied in and the fp32
output copied out inside the timed region.  `--impl reference` times the CPU oracle on the host cores instead.
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
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2605_11354_b200 import dist as pdist  # noqa: E402
from paper_2605_11354_b200 import workloads as wk  # noqa: E402

METRIC = "sla_fwd_dense_equiv_tflops"
UNIT = "TFLOP/s"
L2_FLUSH_BYTES = 512 << 20
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0}
FP8_OVER_BF16 = 2.0  # nominal dense ratio (4.5 vs 2.25 PFLOP/s)
# DRAM bytes (read + write) of one launch, keyed by (workload, kernel), from the ncu captures summarised under
# profiles/; a kernel that changed since its capture has no entry.
DRAM_BYTES_PER_LAUNCH = {
    ("vggt8", "attention"): 87756288,
    ("vggt8", "plan"): 1485824,
    ("vggt8", "quantize_qkv"): 72396800,
    ("vggt8", "summary"): 24797952,
    ("vggt8", "aggregation"): 23398144,
}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            return json.load(fh), "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML (read-only) while the timed region runs."""

    REASONS = (("hw_slowdown", 0x8), ("hw_thermal_slowdown", 0x40), ("sw_thermal_slowdown", 0x20),
               ("sw_power_cap", 0x4))

    def __init__(self, index: int, period_s: float = 0.002):
        self.index, self.period_s = index, period_s
        self.sm, self.mask, self.max_mhz = [], 0, None
        self.stop_flag = threading.Event()
        self.thread = None
        self.error = None

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            visible = os.environ.get("CUDA_VISIBLE_DEVICES")
            phys = self.index
            if visible:
                ids = [v for v in visible.split(",") if v.strip()]
                if self.index < len(ids) and ids[self.index].strip().isdigit():
                    phys = int(ids[self.index])
            self.handle = pynvml.nvmlDeviceGetHandleByIndex(phys)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM))
            self.nvml = pynvml
        except Exception as exc:  # noqa: BLE001
            self.error = f"nvml unavailable: {exc}"
            return
        self.thread = threading.Thread(target=self._pump, daemon=True)
        self.thread.start()

    def _pump(self):
        while not self.stop_flag.is_set():
            try:
                self.sm.append(float(self.nvml.nvmlDeviceGetClockInfo(self.handle, self.nvml.NVML_CLOCK_SM)))
                self.mask |= int(self.nvml.nvmlDeviceGetCurrentClocksEventReasons(self.handle))
            except Exception as exc:  # noqa: BLE001
                self.error = str(exc)
                return
            time.sleep(self.period_s)

    def stop(self):
        self.stop_flag.set()
        if self.thread is not None:
            self.thread.join(timeout=2)
        reasons = [name for name, bit in self.REASONS if self.mask & bit]
        out = {"sm_mhz": statistics.median(self.sm) if self.sm else None, "sm_max_mhz": self.max_mhz,
               "samples": len(self.sm), "reasons": reasons}
        if self.error:
            out["note"] = self.error
        return out


def executed_critical_flops(wl, k_crit):
    return 4.0 * wl.batch * wl.heads * wl.n_blocks * k_crit * wl.block * wl.block * wl.head_dim


def kernel_work(wl, plan):
    """Algorithmic work of one launch of each kernel of the step: (bound, amount, unit of the amount).
    HBM kernels: compulsory bytes (inputs read once + outputs written once).  Tensor kernels: executed flops."""
    tiles = wl.batch * wl.heads * wl.n_blocks
    elems = tiles * wl.block * wl.head_dim          # padded element count of one tensor
    src_bytes = 2 if wl.src_dtype == "bf16" else 4
    valid_elems = wl.batch * wl.heads * wl.tokens * wl.head_dim
    nb = wl.n_blocks
    return {
        # one launch for Q, K and V: read the sources, write codes + scale per tile, 64 column sums per Q and K tile
        "quantize_qkv": ("hbm", 3 * (valid_elems * src_bytes + elems + tiles * 4) + 2 * tiles * 256),
        # fp64 FMAs of the pooled scores (the selection itself is integer work on top)
        "plan": ("alu_fp64", 2.0 * wl.batch * wl.heads * nb * nb * wl.head_dim),
        # read V codes, write fp16 operand (a pass of its own only without a linear branch)
        "prep": ("hbm", elems * 3),
        # read K and V codes, write one bf16 summary row per tile and, next to a sparse branch, the fp16 V operand
        "summary": ("hbm", 2 * elems + tiles * 4160 * 2 + (elems * 2 if plan.k_crit > 0 else 0)),
        # 0/1-mask GEMM over the summaries
        "aggregation": ("tensor_bf16", 2.0 * wl.batch * wl.heads * nb * nb * 4160),
        # QK^T and PV of every (query block, critical key block) pair
        "attention": ("tensor_fp8", executed_critical_flops(wl, plan.k_crit)),
    }


def fp8_gemm_probe(device):
    """Burst throughput of a library e4m3 x e4m3 GEMM (8192^3, best of 10, CUDA events) on this GPU, in TFLOP/s, or
    None when the library call is not there.  Context for the FP8 roofline; nothing on the timed path uses it."""
    try:
        n = 8192
        a = torch.randn(n, n, device=device).to(torch.float8_e4m3fn)
        b = torch.randn(n, n, device=device).to(torch.float8_e4m3fn).t()
        one = torch.ones((), device=device)
        best = float("inf")
        for it in range(13):
            start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            start.record()
            torch._scaled_mm(a, b, scale_a=one, scale_b=one, out_dtype=torch.bfloat16)
            end.record()
            end.synchronize()
            if it >= 3:
                best = min(best, start.elapsed_time(end))
        return 2.0 * n ** 3 / best / 1e9
    except Exception:  # noqa: BLE001 - a missing or changed private torch call only removes the context figure
        return None


def build_roofline(wl, plan, stage_ms, peaks, peak_kind, fp8_probe=None):
    """Roofline of the dominant kernel (largest share of the step) plus a per-kernel table."""
    work = kernel_work(wl, plan)
    hbm = peaks["hbm_gbs"]
    bf16 = peaks["bf16_tflops"]
    table = {}
    for name, (bound, amount) in work.items():
        ms = stage_ms[name]
        if ms <= 0:
            continue
        if bound == "hbm":
            ach, peak, unit, b = amount / (ms * 1e-3) / 1e9, hbm, "GB/s", "hbm"
        elif bound == "tensor_bf16":
            ach, peak, unit, b = amount / (ms * 1e-3) / 1e12, bf16, "TFLOP/s", "tensor"
        elif bound == "tensor_fp8":
            ach, peak, unit, b = amount / (ms * 1e-3) / 1e12, bf16 * FP8_OVER_BF16, "TFLOP/s", "tensor"
        else:  # fp64 FMA pipe: 64 lanes per SM per clock, 148 SMs, at the maximum SM clock
            ach, peak, unit, b = amount / (ms * 1e-3) / 1e12, 2 * 64 * 148 * 1.965e9 / 1e12, "TFLOP/s", "alu"
        table[name] = {"bound": b, "ms": ms, "achieved": ach, "peak": peak, "unit": unit, "frac": ach / peak,
                       "work_per_launch": amount}
    top = max(table, key=lambda n: table[n]["ms"])
    t = table[top]
    launches = 1
    return {"kernel": top, "bound": t["bound"], "achieved": t["achieved"], "peak": t["peak"], "unit": t["unit"],
            "frac": t["frac"],
            "peak_source": (f"{peak_kind} HBM copy" if t["bound"] == "hbm" else
                            f"{peak_kind} bf16 burst x {FP8_OVER_BF16:g} (nominal fp8/bf16 ratio; no fp8 figure measured)"
                            if top == "attention" else f"{peak_kind} bf16 burst" if t["bound"] == "tensor" else
                            "64 fp64 FMA lanes x 148 SMs x 1.965 GHz"),
            "fp8_gemm_probe_tflops": fp8_probe,
            "frac_of_fp8_gemm_probe": (t["achieved"] / fp8_probe) if (fp8_probe and top == "attention") else None,
            "traffic": DRAM_BYTES_PER_LAUNCH.get((wl.name, top)),
            "work_per_launch": t["work_per_launch"] / launches, "avg_launch_ms": t["ms"] / launches,
            "stage_ms": stage_ms, "kernels": table}


# ------------------------------------------------------------------------------------------------ every configuration
PER_CONFIG = (("tiny", None), ("vggt8", None), ("vggt32", None), ("da3l", None), ("frame32", None),
              ("stress100", (0.02, 0.60)), ("stress100", (0.05, 0.60)), ("stress100", (0.10, 0.60)),
              ("stress100", (0.25, 0.60)), ("stress100", (1.00, 0.00)))


def measure_config(lt, wl, crit, neg, dev, proj, device, flush, peaks, reps=5):
    """Step and stage times of one configuration (outside the headline's timed region): whole step with L2 flushed
    before every run and back to back (L2 as the previous run left it), quantiser / plan / forward stages from CUDA
    events, the forward again with bf16 output, and each kernel against its bound."""
    from dataclasses import replace
    wl = replace(wl, crit=crit, neg=neg)
    eng = lt.SlaForward(wl.batch, wl.heads, wl.tokens, wl.block, crit, neg, device=device)

    def timed_once(fn, flushed):
        if flushed:
            flush.fill_(1)
        start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        start.record()
        fn()
        end.record()
        end.synchronize()
        return start.elapsed_time(end)

    run = lambda: eng.run_graph(dev["q"], dev["k"], dev["v"], proj)  # noqa: E731
    for _ in range(3):
        run()
    torch.cuda.synchronize(device)
    cold = statistics.median(timed_once(run, True) for _ in range(reps))
    warm = statistics.median(timed_once(run, False) for _ in range(reps))
    lt.profile_enable(True)
    stages = []
    for _ in range(reps):
        timed_once(lambda: eng.run(dev["q"], dev["k"], dev["v"], proj), True)
        stages.append(lt.profile_stage_ms())
    lt.profile_enable(False)
    quant = statistics.median(timed_once(lambda: eng.quantize(dev["q"], dev["k"], dev["v"]), True) for _ in range(reps))
    plan = statistics.median(timed_once(eng.make_plan, True) for _ in range(reps))
    fwd32 = statistics.median(timed_once(lambda: eng.forward(proj), True) for _ in range(reps))
    out16 = torch.empty(eng.out.shape, dtype=torch.bfloat16, device=device)
    fwd16 = statistics.median(timed_once(lambda: eng.forward(proj, out=out16), True) for _ in range(reps))
    assert int(eng.status.item()) == 0
    stage = {"quantize_qkv": quant, "plan": plan, "prep": statistics.median(s[0] for s in stages),
             "summary": statistics.median(s[1] for s in stages), "aggregation": statistics.median(s[2] for s in stages),
             "attention": statistics.median(s[3] for s in stages)}
    table = build_roofline(wl, eng.plan, stage, peaks, "measured")["kernels"]
    res = {"workload": wl.name, "crit": crit, "neg": neg, "k_crit": eng.plan.k_crit, "k_marg": eng.plan.k_marg,
           "ms_l2_flushed": cold, "ms_l2_warm": warm, "ms_quantize": quant, "ms_plan": plan, "ms_forward": fwd32,
           "ms_forward_bf16_out": fwd16, "dense_equiv_tflops": wl.dense_equiv_flops / cold / 1e9,
           "stage_ms": stage, "roofline_frac": {k: round(v["frac"], 4) for k, v in table.items()},
           "attention_tflops_executed": table["attention"]["achieved"] if "attention" in table else None}
    del eng, out16
    return res


def measure_projection(lt, wl, device, flush, peaks, reps=5):
    """The qkv projection in front of the attention as an FP8 GEMM whose epilogue is the block quantiser (Algorithm 2
    in its deployed form): per-token quantiser of the activations, the fused GEMM, and the step it makes possible
    (projection + plan + forward, no separate pass over Q, K, V)."""
    d_model = wl.heads * wl.head_dim
    g = torch.Generator(device="cpu").manual_seed(wl.cfg_id)
    x = torch.randn((wl.batch * wl.tokens, d_model), generator=g).to(torch.bfloat16).to(device)
    w = (torch.randn((3 * d_model, d_model), generator=g) / d_model ** 0.5).to(device)
    proj = (torch.randn((wl.heads, 64, 64), generator=g) / 8).to(device)
    wc, ws = lt.lite3r_quantize_rows_fp8(w)  # weights are quantised once, offline
    eng = lt.SlaForward(wl.batch, wl.heads, wl.tokens, wl.block, wl.crit, wl.neg, device=device)
    state = {}

    def timed_once(fn):
        flush.fill_(1)
        start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        start.record()
        fn()
        end.record()
        end.synchronize()
        return start.elapsed_time(end)

    def rowq():
        state["xc"], state["xs"] = lt.lite3r_quantize_rows_fp8(x)

    def gemm():
        lt.lite3r_qkv_project_fp8(state["xc"], state["xs"], wc, ws, None, eng.shape, eng.q8, eng.k8, eng.v8, eng.status)

    def step():
        rowq()
        gemm()
        eng.make_plan()
        eng.forward(proj)

    for _ in range(3):
        step()
    torch.cuda.synchronize(device)
    t_rowq = statistics.median(timed_once(rowq) for _ in range(reps))
    t_gemm = statistics.median(timed_once(gemm) for _ in range(reps))
    t_step = statistics.median(timed_once(step) for _ in range(reps))
    assert int(eng.status.item()) == 0
    flops = 2.0 * wl.batch * wl.tokens * d_model * 3 * d_model
    fp8_peak = peaks["bf16_tflops"] * FP8_OVER_BF16
    rowq_bytes = wl.batch * wl.tokens * d_model * 3 + wl.batch * wl.tokens * 4
    return {"workload": wl.name + "+qkv_projection", "d_model": d_model, "ms_quantize_rows": t_rowq,
            "ms_qkv_gemm_fused_quantiser": t_gemm, "ms_step_from_activations": t_step,
            "gemm_tflops": flops / t_gemm / 1e9, "gemm_frac_of_fp8_peak": flops / t_gemm / 1e9 / fp8_peak,
            "quantize_rows_frac_of_hbm": rowq_bytes / (t_rowq * 1e-3) / 1e9 / peaks["hbm_gbs"]}


def per_config_table(lt, device, flush, peaks):
    """One entry per benchmark configuration (the five of the contract, the frame-attention shape and the sparsity
    sweep of the stress configuration)."""
    rows, cached, cached_name = [], None, None
    for name, fractions in PER_CONFIG:
        try:
            wl = wk.WORKLOADS[name]
            if cached_name != name:
                cached = None
                torch.cuda.empty_cache()
                inputs = wk.make_inputs(wl)
                dev = {}
                for n in ("q", "k", "v"):
                    if wl.src_dtype == "bf16":
                        dev[n] = torch.from_numpy(wk.bf16_bits(inputs[n]).view(np.int16)).to(device).view(torch.bfloat16)
                    else:
                        dev[n] = torch.from_numpy(inputs[n]).to(device)
                cached, cached_name = (dev, torch.from_numpy(inputs["proj"]).to(device)), name
                del inputs
            crit, neg = fractions if fractions is not None else (wl.crit, wl.neg)
            rows.append(measure_config(lt, wl, crit, neg, cached[0], cached[1], device, flush, peaks))
            if name in ("vggt8", "vggt32"):
                rows.append(measure_projection(lt, wl, device, flush, peaks))
        except Exception as exc:  # noqa: BLE001 - a failed configuration is reported, the others still run
            rows.append({"workload": name, "error": f"{type(exc).__name__}: {exc}"})
    return rows


# ------------------------------------------------------------------------------------------------ CPU oracle timing
def time_oracle(wl, inputs, n_heads, budget_blocks):
    """One bounded sample of the step on the host cores: quantiser and plan for the first `n_heads` heads of every
    batch entry, the forward on a seeded sample of their query blocks; both parts are extrapolated to the whole
    workload (heads are independent problems of equal size).  Returns (seconds per whole step, description)."""
    from oracle import sla_oracle as orc
    n_heads = min(n_heads, wl.heads)
    sub = {n: np.ascontiguousarray(inputs[n][:, :n_heads]) for n in ("q", "k", "v")}
    proj = inputs["proj"][:n_heads]
    t0 = time.perf_counter()
    r = orc.sla_forward_from_source(sub["q"], sub["k"], sub["v"], proj, wl.block, wl.crit, wl.neg, query_blocks=[])
    t_front = time.perf_counter() - t0
    total_sub = wl.batch * n_heads * wl.n_blocks
    total = wl.batch * wl.heads * wl.n_blocks
    g = np.random.default_rng(wl.cfg_id)
    n = min(budget_blocks, total_sub)
    flat = g.choice(total_sub, size=n, replace=False)
    qb = [(int(f // (n_heads * wl.n_blocks)), int((f // wl.n_blocks) % n_heads), int(f % wl.n_blocks)) for f in flat]
    t0 = time.perf_counter()
    orc.sla_forward(r["qhat"], r["khat"], r["vhat"], proj, r["cls"], wl.block, "softmax", qb)
    t_blocks = time.perf_counter() - t0
    seconds = t_front * wl.heads / n_heads + t_blocks * total / n
    sample = (f"quantise x3 + plan on {n_heads} of {wl.heads} heads ({t_front:.1f} s) + forward on {n} of {total} "
              f"query blocks ({t_blocks:.1f} s), each extrapolated to the whole step")
    return seconds, sample


def host_threads():
    try:
        from threadpoolctl import threadpool_info
        n = max((p.get("num_threads", 1) for p in threadpool_info()), default=1)
    except Exception:
        n = 1
    return int(n)


def run_reference(args, wl):
    rank, _, world = pdist.env_world()
    if rank != 0:
        return
    inputs = wk.make_inputs(wl)
    times = []
    sample = ""
    for _ in range(args.warmup):
        time_oracle(wl, inputs, 1, 8)
    for _ in range(args.steps):
        sec, sample = time_oracle(wl, inputs, 2, max(16, args.oracle_blocks // 8))
        times.append(sec)
    sec = sum(times) / len(times)
    value = wl.dense_equiv_flops / sec / 1e12
    cores = host_threads()
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic", "impl": "reference",
            "config": {"workload": wl.name, "batch": wl.batch, "heads": wl.heads, "tokens": wl.tokens,
                       "head_dim": wl.head_dim, "block": wl.block, "crit": wl.crit, "neg": wl.neg},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------ CUDA path
def run_ours(args, wl):
    from paper_2605_11354_b200 import binding as lt
    from paper_2605_11354_b200 import build as lb

    rank, local_rank, world = pdist.init()
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the SLA forward has no CPU path")
    device = torch.device("cuda", local_rank)
    torch.cuda.set_device(device)
    if rank == 0:
        lb.build()
    pdist.barrier(device)
    lt.lib()

    inputs = wk.make_inputs(wl)
    host = {}
    for name in ("q", "k", "v"):
        if wl.src_dtype == "bf16":
            t = torch.from_numpy(wk.bf16_bits(inputs[name]).view(np.int16)).view(torch.bfloat16)
        else:
            t = torch.from_numpy(inputs[name])
        host[name] = t.pin_memory()
    proj = torch.from_numpy(inputs["proj"]).to(device)
    dev = {n: host[n].to(device) for n in ("q", "k", "v")}
    eng = lt.SlaForward(wl.batch, wl.heads, wl.tokens, wl.block, wl.crit, wl.neg, device=device)
    out_host = torch.empty(eng.out.shape, dtype=torch.float32).pin_memory()
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=device)

    def step():
        # one CUDA graph per step: quantise, plan beside the plan-independent half of the forward on a side stream,
        # the rest of the forward
        return eng.run_graph(dev["q"], dev["k"], dev["v"], proj)

    def step_in_order():
        return eng.run(dev["q"], dev["k"], dev["v"], proj)

    def step_e2e():
        for n in ("q", "k", "v"):
            dev[n].copy_(host[n], non_blocking=True)
        out = eng.run(dev["q"], dev["k"], dev["v"], proj)
        out_host.copy_(out, non_blocking=True)

    def timed_e2e(steps):
        """`steps` steps through the public API, each with its sources copied in from pinned host memory and its
        result copied back to pinned host memory, everything inside one timed region.  Three streams (copy-in,
        compute, copy-out) and two sets of device sources and results: the copies of neighbouring steps overlap the
        kernels and each other (PCIe is full duplex).  L2 is not flushed inside the region; a step touches about
        0.2 GB (sources, codes, operands, result), more than the 126 MB of L2."""
        cur = torch.cuda.current_stream(device)
        s_in, s_out = torch.cuda.Stream(device), torch.cuda.Stream(device)
        srcs = [dev, {n: torch.empty_like(dev[n]) for n in dev}]
        outs = [eng.out, torch.empty_like(eng.out)]
        out_hosts = [out_host, torch.empty_like(out_host).pin_memory()]
        consumed, read_back = [None, None], [None, None]
        flush.fill_(1)
        start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        start.record(cur)
        s_in.wait_stream(cur)
        s_out.wait_stream(cur)
        for i in range(steps):
            b = i & 1
            with torch.cuda.stream(s_in):
                if consumed[b] is not None:
                    s_in.wait_event(consumed[b])  # the step that last used these source buffers has run
                for n in ("q", "k", "v"):
                    srcs[b][n].copy_(host[n], non_blocking=True)
                arrived = s_in.record_event()
            cur.wait_event(arrived)
            if read_back[b] is not None:
                cur.wait_event(read_back[b])  # this result buffer has reached the host
            eng.run(srcs[b]["q"], srcs[b]["k"], srcs[b]["v"], proj, out=outs[b], overlap=True)
            consumed[b] = cur.record_event()
            with torch.cuda.stream(s_out):
                s_out.wait_event(consumed[b])
                out_hosts[b].copy_(outs[b], non_blocking=True)
                read_back[b] = s_out.record_event()
        cur.wait_stream(s_out)  # the region ends when the last result is on the host
        end.record(cur)
        end.synchronize()
        return start.elapsed_time(end)

    def timed(fn, steps, collect_stages):
        total_ms, stages = 0.0, []
        for _ in range(steps):
            flush.fill_(1)  # evict L2 between timed iterations (not timed)
            start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            start.record()
            fn()
            end.record()
            end.synchronize()
            total_ms += start.elapsed_time(end)
            if collect_stages:
                stages.append(lt.profile_stage_ms())
        return total_ms, stages

    for _ in range(args.warmup):
        step()
        step_e2e()
    torch.cuda.synchronize(device)
    assert int(eng.status.item()) == 0

    sampler = ClockSampler(local_rank)
    sampler.start()
    pdist.barrier(device)
    torch.cuda.synchronize(device)
    # kernels of one step, counted on a stream-ordered run (the timed steps replay the same launches as a CUDA graph,
    # which the library's launch counter does not see)
    launches0 = lt.launch_count()
    step_in_order()
    launches = (lt.launch_count() - launches0) * args.steps
    torch.cuda.synchronize(device)
    ms_total, _ = timed(step, args.steps, False)  # the library's stage events are off inside the timed regions
    torch.cuda.synchronize(device)
    pdist.barrier(device)
    e2e_total = timed_e2e(args.steps)
    torch.cuda.synchronize(device)
    pdist.barrier(device)
    clocks = sampler.stop()
    assert int(eng.status.item()) == 0

    # Per-kernel breakdown (outside the timed region, L2 flushed before each sample): quantiser and plan with CUDA
    # events on the launching stream, the forward's four stages from the library's own event marks.
    def sample(fn, reps):
        acc = 0.0
        for _ in range(reps):
            flush.fill_(1)
            start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            start.record()
            fn()
            end.record()
            end.synchronize()
            acc += start.elapsed_time(end)
        return acc / reps

    reps = max(3, min(args.steps, 10))
    lt.profile_enable(True)
    _, stages = timed(step_in_order, reps, True)  # one kernel after the other, so that each stage time is its own
    lt.profile_enable(False)
    quant_ms = sample(lambda: eng.quantize(dev["q"], dev["k"], dev["v"]), reps)
    plan_ms = sample(eng.make_plan, reps)

    flops = wl.dense_equiv_flops
    value_flops, worst_s = pdist.aggregate_throughput(flops * args.steps, ms_total / 1e3, device)
    e2e_flops, _ = pdist.aggregate_throughput(flops * args.steps, e2e_total / 1e3, device)

    peaks, peak_kind = measured_peaks()
    stage = {"quantize_qkv": quant_ms, "plan": plan_ms,
             "prep": statistics.mean(s[0] for s in stages), "summary": statistics.mean(s[1] for s in stages),
             "aggregation": statistics.mean(s[2] for s in stages), "attention": statistics.mean(s[3] for s in stages)}
    roofline = build_roofline(wl, eng.plan, stage, peaks, peak_kind, fp8_gemm_probe(device) if rank == 0 else None)

    if rank != 0:
        pdist.shutdown()
        return
    in_bytes = sum(host[n].numel() * host[n].element_size() for n in ("q", "k", "v"))
    out_bytes = out_host.numel() * 4
    line = {"metric": METRIC, "value": value_flops / 1e12, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": worst_s * 1e3 / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "fp8_e4m3", "data": "synthetic",
            "config": {"workload": wl.name, "batch": wl.batch, "heads": wl.heads, "tokens": wl.tokens,
                       "head_dim": wl.head_dim, "block": wl.block, "crit": wl.crit, "neg": wl.neg,
                       "k_crit": eng.plan.k_crit, "k_marg": eng.plan.k_marg, "k_neg": eng.plan.k_neg,
                       "source_dtype": wl.src_dtype, "l2": f"flushed between timed steps ({L2_FLUSH_BYTES >> 20} MiB write)",
                       "e2e_pipeline": "copy-in, compute and copy-out streams over two buffer sets; no L2 flush inside",
                       "streams": "one CUDA graph per step; summaries of the forward on a side stream beside the plan kernel",
                       "parallelism": "independent replicas, no collective" if world > 1 else "single GPU"},
            "e2e": {"value": e2e_flops / 1e12, "unit": UNIT, "h2d_bytes_per_step": in_bytes,
                    "d2h_bytes_per_step": out_bytes},
            "gpu_launches": int(launches), "clocks": clocks, "roofline": roofline}
    if world == 1 and args.no_per_config and args.projection:
        # the qkv projection in front of this workload alone (what profiles of the FP8 GEMM are taken on)
        line["per_config"] = [measure_projection(lt, wl, device, flush, peaks)]
    if world == 1 and not args.no_per_config:
        del dev, eng
        clocks_all = ClockSampler(local_rank)
        clocks_all.start()
        line["per_config"] = per_config_table(lt, device, flush, peaks)
        line["per_config_clocks"] = clocks_all.stop()
    if world == 1 and not args.no_cpu_baseline:
        sec, sample = time_oracle(wl, inputs, wl.heads, args.oracle_blocks)
        line["cpu_baseline"] = {"value": flops / sec / 1e12, "unit": UNIT, "cores": host_threads(), "kind": "oracle",
                                "sample": sample}
    print(json.dumps(line))
    pdist.shutdown()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="vggt8", choices=sorted(wk.WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=("ours", "reference"))
    ap.add_argument("--oracle-blocks", type=int, default=512)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-per-config", action="store_true", help="skip the table over all configurations")
    ap.add_argument("--projection", action="store_true",
                    help="with --no-per-config: still measure the FP8 qkv projection in front of the workload")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    wl = wk.WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()
