#!/usr/bin/env python
"""Benchmark of the ternary mpGEMM hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Workload (config.workload = "sweep100b"): the 100B-shaped decode sweep at batch 1 -- 80 layers of
four ternary linears (8192->10240, 8192->8192, 8192->57344, 28672->8192), every tensor with its own
seeded weights resident in HBM in the I2_S encoding (17.1 GB), one fp32 activation vector per linear.
One step = one pass over all 320 linears: absmax int8 quantiser, then I2_S mpGEMV with the fused
rescale -- ONE bitnet_linear_group call, i.e. one persistent kernel over the whole list.  `value` = I2_S bytes
streamed per step / step time (GB/s), so it charges the quantisers and every gap to the weight stream.  The same
pass as 320 separate launches (CUDA graphs) is reported under "per_linear_launches".  The same sweep in the TL2
encoding and the prefill mpGEMM (2048 x 4096 x 14336, int8 tensor cores) are timed in the same run
and reported under "tl2" and "prefill".  Inputs (17 GB) exceed L2 (126 MB) many times over, so no L2
flush is needed between steps.

With --gpus N > 1 (under torchrun) every rank runs an independent replica of the sweep on its own
GPU (the path has no exchange step; weak scaling, no collective on the data path).

--impl reference times the CPU oracle on a bounded sample of the same workload on the host cores.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "mpgemv_weight_stream_batch1"
UNIT = "GB/s"


# dram__bytes_read.sum + dram__bytes_write.sum of one captured launch of the grouped decode kernel over 4 layers of
# the sweep (856.652 MB read + 4.546 MB written) over the packed weight bytes of that launch (855.638 MB).  Traffic
# grows in proportion to the weights streamed, so the same ratio scales it to the full launch.
NCU_TRAFFIC_PER_ALGORITHMIC_BYTE = (856.652 + 4.546) / 855.638

def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm=float(d["hbm_gbs"]), bf16=float(d["bf16_tflops"]), which="measured")
    return dict(hbm=6650.0, bf16=1590.0, which="fallback")


# ------------------------------------------------------------------------------------------------ reference arm
def oracle_layer(wl, layer=0):
    """The bounded CPU sample: the four linears of one layer of the sweep (213.9 MB as I2_S)."""
    import numpy as np
    out = []
    for j, lin in enumerate(wl.linears):
        w = np.ascontiguousarray(wl.weights(layer, j).numpy())
        x = np.ascontiguousarray(wl.activations(layer, j, 1).numpy())
        out.append((w, x))
    return out


def oracle_step(oracle, sample, w_scales=None):
    """Alg. 1 on the CPU for every linear of the sample: quantiser, definition, rescale."""
    ys = []
    for i, (w, x) in enumerate(sample):
        q, sc, _ = oracle.quant_act(x)
        acc = oracle.mpgemm_def(q, w)
        ys.append((acc, sc, oracle.dequant(acc, sc, 2.0 / 3.0 if w_scales is None else w_scales[i])))
    return ys


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2502_11880_b200 import synth
    oracle.build()
    wl = synth.CONFIGS["sweep100b"]
    sample = oracle_layer(wl)
    nbytes = sum(w.shape[0] * w.shape[1] // 4 for w, _ in sample)
    for _ in range(args.warmup):
        oracle_step(oracle, sample)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_step(oracle, sample)
    dt = (time.perf_counter() - t0) / args.steps
    val = nbytes / dt / 1e9
    desc = f"layer 0 of the sweep (4 linears, {nbytes / 1e6:.1f} MB as I2_S) per step: quantiser + definition + rescale"
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "config": {"workload": "sweep100b", "sample": desc},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": desc},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------ our arm
class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU every 10 ms while the timed region runs (NVML reads
    only; falls back to one-shot nvidia-smi if the NVML binding is missing)."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, gpu_index):
        import threading
        self.sm, self.mem, self.power, self.reasons, self.sm_max = [], [], [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(gpu_index)
            self.sm_max = float(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        except Exception:
            self._nv = None

    def _run(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                self.sm.append(float(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                self.mem.append(float(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_MEM)))
                self.power.append(nv.nvmlDeviceGetPowerUsage(self._h) / 1000.0)
                bits = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
                for bit, name in self.REASONS.items():
                    if bits & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(0.01)

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join(timeout=2)
        out = {"sm_mhz": None, "sm_max_mhz": self.sm_max, "reasons": sorted(self.reasons), "samples": len(self.sm)}
        if self.mem:
            out["mem_mhz"] = statistics.median(self.mem)
        if self.power:
            out["power_w"] = statistics.median(self.power)
        if self.sm:
            out["sm_mhz"] = statistics.median(self.sm)
        elif self._nv is None:
            try:
                txt = subprocess.run(["nvidia-smi", "--query-gpu=clocks.sm,clocks.max.sm", "--format=csv,noheader,nounits"],
                                     capture_output=True, text=True, timeout=10).stdout.split("\n")[0].split(",")
                out.update(sm_mhz=float(txt[0]), sm_max_mhz=float(txt[1]), samples=1)
            except Exception:
                pass
        return out


class Sweep:
    """The decode sweep resident on one GPU: packed blobs, activation buffers, outputs, workspaces."""

    def __init__(self, bn, torch, wl, fmts, layers, device):
        self.bn, self.torch, self.wl, self.layers = bn, torch, wl, layers
        self.lin = wl.linears
        self.fmts = fmts
        self.blobs = {f: [] for f in fmts}
        self.w_scale = []
        t0 = time.time()
        # one encoding after the other, so that the blobs of an encoding lie together in device memory as they would
        # in a deployment that keeps a single encoding
        for fi, f in enumerate(fmts):
            for layer in range(layers):
                for j, lin in enumerate(self.lin):
                    w = wl.weights(layer, j, device=device)
                    if fi == 0:
                        self.w_scale.append(bn.synth.absmean_scale(w))
                    self.blobs[f].append(bn.pack(f, w, check=False))
                    del w
        torch.cuda.synchronize()
        self.setup_s = time.time() - t0
        self.bytes = {f: sum(b.numel() for b in self.blobs[f]) for f in fmts}
        # activations: all vectors of the sweep in one pinned host buffer and one device buffer
        self.x_off, self.y_off = [], []
        xo = yo = 0
        for layer in range(layers):
            for lin in self.lin:
                self.x_off.append(xo)
                self.y_off.append(yo)
                xo += lin.K
                yo += lin.M
        self.x_host = torch.empty(xo, dtype=torch.float32).pin_memory()
        self.y_host = torch.empty(yo, dtype=torch.float32).pin_memory()
        i = 0
        for layer in range(layers):
            for j, lin in enumerate(self.lin):
                self.x_host[self.x_off[i]: self.x_off[i] + lin.K] = wl.activations(layer, j, 1)[0]
                i += 1
        self.x_dev = self.x_host.to(device)
        self.y_dev = torch.zeros(yo, dtype=torch.float32, device=device)
        self.q_dev = torch.empty(xo, dtype=torch.int8, device=device)
        self.sc_dev = torch.empty(len(self.x_off), dtype=torch.float32, device=device)
        kmax = max(l.K for l in self.lin)
        mmax = max(l.M for l in self.lin)
        self.ws = {}
        for f in fmts:
            n = max(bn.bitnet_mpgemm_workspace_bytes(f, 1, l.M, l.K) for l in self.lin)
            self.ws[f] = torch.zeros(max(n, 16), dtype=torch.uint8, device=device)
        self.kmax, self.mmax = kmax, mmax
        self._host_batch = {}
        self._groups = {}

    def n_linears(self):
        return len(self.x_off)

    def views(self, i):
        lin = self.lin[i % len(self.lin)]
        x = self.x_dev[self.x_off[i]: self.x_off[i] + lin.K].view(1, lin.K)
        q = self.q_dev[self.x_off[i]: self.x_off[i] + lin.K].view(1, lin.K)
        y = self.y_dev[self.y_off[i]: self.y_off[i] + lin.M].view(1, lin.M)
        sc = self.sc_dev[i: i + 1]
        return lin, x, q, sc, y

    def step_device(self, fmt, mode="linear", lo=0, hi=None):
        """One pass over linears [lo, hi), inputs resident.  mode "linear": bitnet_linear (quantiser + mpGEMV +
        rescale; one fused kernel per linear for I2_S, two kernels for TL2); "quant" / "gemv": that step alone."""
        bn = self.bn
        hi = self.n_linears() if hi is None else hi
        for i in range(lo, hi):
            lin, x, q, sc, y = self.views(i)
            if mode == "linear":
                bn.bitnet_linear(fmt, self.blobs[fmt][i], self.w_scale[i], lin.M, lin.K, x, q=q, act_scale=sc, y=y,
                                 workspace=self.ws[fmt])
            elif mode == "quant":
                bn.bitnet_quant_act(x, q=q, act_scale=sc, act_sum=self._sum)
            else:
                bn.bitnet_mpgemm(fmt, self.blobs[fmt][i], self.w_scale[i], lin.M, lin.K, q, sc, y=y,
                                 workspace=self.ws[fmt])

    def step_group(self, fmt, lo=0, hi=None):
        """The same pass as ONE bitnet_linear_group call (I2_S: one persistent kernel over all linears)."""
        bn = self.bn
        hi = self.n_linears() if hi is None else hi
        key = (fmt, lo, hi)
        if key not in self._groups:
            items = []
            for i in range(lo, hi):
                lin, x, q, sc, y = self.views(i)
                items.append(dict(fmt=fmt, packed=self.blobs[fmt][i], w_scale=self.w_scale[i], M=lin.M, K=lin.K, x=x, q=q,
                                  act_scale=sc, y=y, workspace=self.ws[fmt]))
            self._groups[key] = (bn.make_group(items), items)
        bn.bitnet_linear_group(self._groups[key][0])

    def step_host(self, fmt):
        """The same pass through the host-buffer entry point (one bitnet_linear_host_batch call per step):
        per linear, H2D of x from pinned memory, quantiser + mpGEMV, D2H of y to pinned memory; the library
        overlaps the copies of one linear with the kernels of its neighbours."""
        bn = self.bn
        if fmt not in self._host_batch:
            items = []
            for i in range(self.n_linears()):
                lin, x, q, sc, y = self.views(i)
                xh = self.x_host[self.x_off[i]: self.x_off[i] + lin.K].view(1, lin.K)
                yh = self.y_host[self.y_off[i]: self.y_off[i] + lin.M].view(1, lin.M)
                items.append(dict(fmt=fmt, packed=self.blobs[fmt][i], w_scale=self.w_scale[i], M=lin.M, K=lin.K,
                                  x_host=xh, y_host=yh, x_dev=x, q_dev=q, scale_dev=sc, y_dev=y, workspace=self.ws[fmt]))
            self._host_batch[fmt] = (bn.make_host_batch(items), items)
        bn.bitnet_linear_host_batch(self._host_batch[fmt][0])

    def make_graph(self, fmt, mode="linear", linears_per_graph=128):
        """Captures the step as CUDA graphs of at most `linears_per_graph` linears each (long chains of
        programmatically dependent kernel nodes in ONE graph replay pathologically slowly on this driver).
        Returns a callable that replays them in order."""
        torch = self.torch
        self._sum = torch.empty(1, dtype=torch.int32, device=self.x_dev.device)
        s = torch.cuda.Stream()
        s.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(s):
            if mode == "group":
                self.step_group(fmt)
            else:
                self.step_device(fmt, mode)        # warm every kernel variant before capture
        torch.cuda.current_stream().wait_stream(s)
        torch.cuda.synchronize()
        graphs = []
        for lo in range(0, self.n_linears(), linears_per_graph):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                if mode == "group":
                    self.step_group(fmt, lo, min(lo + linears_per_graph, self.n_linears()))
                else:
                    self.step_device(fmt, mode, lo, min(lo + linears_per_graph, self.n_linears()))
            graphs.append(g)

        def replay():
            for g in graphs:
                g.replay()
        replay.n_graphs = len(graphs)
        return replay


def bench_batched(sw, torch, T, steps, warmup, fmt="i2s"):
    """The same sweep with T tokens per linear through ONE bitnet_linear_group call per step: quantiser + mpGEMM +
    rescale.  Every linear keeps its own weights; the T activation rows of layer 0's four linears are reused by all
    layers.  I2_S: up to 8 tokens the whole list is one persistent kernel; 9 to 16 tokens its two-group form after one
    quantiser launch over the list; 17 to 128 tokens one quantiser launch, then the streaming tcgen05 kernel (160
    linears per launch).  TL1, TL2 (up to 8 tokens): the scan kernel over the whole list."""
    bn, dev = sw.bn, sw.x_dev.device
    nl = len(sw.lin)
    xs = [sw.wl.activations(0, j, T).to(dev) for j in range(nl)]
    qs = [torch.empty((T, l.K), dtype=torch.int8, device=dev) for l in sw.lin]
    scs = [torch.empty(T, dtype=torch.float32, device=dev) for l in sw.lin]
    ys = [torch.empty((T, l.M), dtype=torch.float32, device=dev) for l in sw.lin]
    ws = torch.zeros(max(16, max(bn.bitnet_mpgemm_workspace_bytes(fmt, T, l.M, l.K) for l in sw.lin)),
                     dtype=torch.uint8, device=dev)
    items = []
    for i in range(sw.n_linears()):
        j = i % nl
        lin = sw.lin[j]
        items.append(dict(fmt=fmt, packed=sw.blobs[fmt][i], w_scale=sw.w_scale[i], M=lin.M, K=lin.K, x=xs[j], q=qs[j],
                          act_scale=scs[j], y=ys[j], workspace=ws))
    grp = bn.make_group(items)
    ms = time_replays(torch, lambda: bn.bitnet_linear_group(grp), steps, warmup)
    weights = sw.bytes["i2s"] * 4.0          # four weights per packed byte of the I2_S blob
    if fmt != "i2s":
        return {"tokens": T, "ms_per_step": ms, "tokens_per_s": T / ms * 1e3, "weight_GBps": sw.bytes[fmt] / ms / 1e6,
                "frac_of_hbm_peak": sw.bytes[fmt] / ms / 1e6 / peaks()["hbm"], "int8_tops": 2.0 * T * weights / ms / 1e9}
    # roofline of the line: the weights once over HBM, or the multiply-adds on the int8 tensor cores (2 x the measured
    # bf16 rate), whichever takes longer
    pk = peaks()
    ms_hbm, ms_tensor = sw.bytes["i2s"] / pk["hbm"] / 1e6, 2.0 * T * weights / (2.0 * pk["bf16"]) / 1e9
    return {"tokens": T, "ms_per_step": ms, "tokens_per_s": T / ms * 1e3, "weight_GBps": sw.bytes["i2s"] / ms / 1e6,
            "frac_of_hbm_peak": sw.bytes["i2s"] / ms / 1e6 / pk["hbm"], "int8_tops": 2.0 * T * weights / ms / 1e9,
            "roofline_ms": max(ms_hbm, ms_tensor), "roofline_bound": "hbm" if ms_hbm >= ms_tensor else "tensor",
            "frac_of_roofline": max(ms_hbm, ms_tensor) / ms}


def bench_small_configs(bn, torch, synth, steps, warmup):
    """The three small workloads (1536 GEMV, 3B-shaped layer, 8B-shaped layer), I2_S and TL2, at their token counts:
    time per pass over the workload's linears, (a) L2-resident: the same blobs over and over, (b) cold: rotating over
    enough distinct copies of the blobs that the working set is at least 256 MB (twice the L2)."""
    out = []
    dev = torch.device("cuda")
    for name in ("gemv1536", "layer3b", "layer8b"):
        wl = synth.CONFIGS[name]
        for fmt in ("i2s", "tl2"):
            blobs, scales = [], []
            for j, lin in enumerate(wl.linears):
                w = wl.weights(0, j, device=dev)
                scales.append(synth.absmean_scale(w))
                blobs.append(bn.pack(fmt, w, check=False))
                del w
            packed = sum(b.numel() for b in blobs)
            copies = max(2, -(-(256 << 20) // packed))
            rot = [[b.clone() for b in blobs] for _ in range(copies)]
            for T in wl.tokens:
                xs = [wl.activations(0, j, T).to(dev) for j in range(len(wl.linears))]
                qs = [torch.empty((T, l.K), dtype=torch.int8, device=dev) for l in wl.linears]
                scs = [torch.empty(T, dtype=torch.float32, device=dev) for l in wl.linears]
                ys = [torch.empty((T, l.M), dtype=torch.float32, device=dev) for l in wl.linears]
                ws = torch.zeros(max(16, max(bn.bitnet_mpgemm_workspace_bytes(fmt, T, l.M, l.K) for l in wl.linears)),
                                 dtype=torch.uint8, device=dev)

                def group_over(sets):
                    items = []
                    for bl in sets:
                        for j, lin in enumerate(wl.linears):
                            items.append(dict(fmt=fmt, packed=bl[j], w_scale=scales[j], M=lin.M, K=lin.K, x=xs[j], q=qs[j],
                                              act_scale=scs[j], y=ys[j], workspace=ws))
                    return bn.make_group(items), items

                reps = max(8, min(copies, 64))
                g_hot, keep1 = group_over([blobs] * reps)
                g_cold, keep2 = group_over(rot)
                # one pass alone (what a caller pays for one layer when nothing else is queued)
                g_one, keep3 = group_over([blobs])
                ms_hot = time_replays(torch, lambda: bn.bitnet_linear_group(g_hot), steps, warmup) / reps
                ms_cold = time_replays(torch, lambda: bn.bitnet_linear_group(g_cold), steps, warmup) / copies
                ms_one = time_replays(torch, lambda: bn.bitnet_linear_group(g_one), steps, warmup)
                out.append({"workload": name, "format": fmt, "tokens": T, "packed_bytes": packed,
                            "us_per_pass_l2_resident": ms_hot * 1e3, "us_per_pass_cold": ms_cold * 1e3,
                            "us_single_call": ms_one * 1e3, "cold_copies": copies,
                            "cold_GBps": packed / ms_cold / 1e6, "l2_resident_GBps": packed / ms_hot / 1e6})
            del rot, blobs
            torch.cuda.empty_cache()
    return out


def max_over_ranks(torch, dist, ms, device):
    """The job's time for a region is the slowest rank's device time (every rank gets the same number back)."""
    if dist is None:
        return float(ms)
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.barrier()
    return float(t.item())


def whole_job_value(bytes_per_replica, world, ms_step):
    """Replicas only: every rank streams its own copy of the sweep, so the job moves world x the bytes."""
    return bytes_per_replica * world / ms_step / 1e6


def time_replays(torch, fn, steps, warmup, dist=None):
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    ms = max_over_ranks(torch, dist, e0.elapsed_time(e1), "cuda")
    return ms / steps


def bench_ceilings(bn, torch, sm_mhz):
    """Ceilings measured on this GPU with the decode kernels' own access pattern and instruction kinds: a read-only
    stream over 8 GiB (cp.async rings, no arithmetic), the issue rate of the instructions the decode loops are made
    of (warp-instructions per clock and SM at the SM clock sampled under load), and the library's dense int8 GEMM
    at 8192^3 (the prefill denominator next to 2 x the measured bf16 figure)."""
    dev = torch.device("cuda")
    out = {}
    sink = torch.zeros(4, dtype=torch.int32, device=dev)
    buf = torch.empty(8 << 30, dtype=torch.uint8, device=dev)
    buf.view(torch.int32).fill_(0x01010101)
    rs = {}
    for depth in (4, 6, 8):
        ms = time_replays(torch, lambda: bn.bitnet_microbench_read_stream(buf, depth, sink), 10, 3)
        rs[f"ring_{depth}"] = buf.numel() / ms / 1e6
    out["read_stream_GBps"] = rs
    del buf
    torch.cuda.empty_cache()
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    clock_hz = (sm_mhz or 1965.0) * 1e6
    iters = 20000
    rates = {}
    for kind in bn.MICROBENCH_KINDS:
        ms = time_replays(torch, lambda: bn.bitnet_microbench_issue(kind, iters, sink), 5, 3)
        rates[kind] = 16.0 * iters * 32 / (ms * 1e-3 * clock_hz)
    out["issue_warp_instr_per_clk_per_sm"] = rates
    out["issue_note"] = f"16 warps per SM, 32 independent instructions per thread and iteration, at {clock_hz / 1e6:.0f} MHz"
    try:
        a = torch.randint(-127, 128, (8192, 8192), dtype=torch.int8, device=dev)
        b = torch.randint(-1, 2, (8192, 8192), dtype=torch.int8, device=dev).t()
        ms = time_replays(torch, lambda: torch._int_mm(a, b), 10, 3)
        out["library_int8_gemm_8192cubed_tops"] = 2.0 * 8192 ** 3 / ms / 1e9
    except Exception as e:          # noqa: BLE001 - context only
        out["library_int8_gemm_8192cubed_tops"] = None
        out["library_int8_gemm_note"] = str(e)[:80]
    return out


def bench_prefill(bn, torch, synth, steps, warmup):
    wl = synth.CONFIGS["prefill"]
    lin, T = wl.linears[0], wl.tokens[0]
    w = wl.weights(0, 0, device="cuda")
    blob = bn.pack("i2s", w, check=False)
    w_scale = synth.absmean_scale(w)
    del w
    x = wl.activations(0, 0, T).cuda()
    q, sc, sm = bn.bitnet_quant_act(x)
    y = torch.empty((T, lin.M), dtype=torch.float32, device="cuda")

    def gemm():
        bn.bitnet_mpgemm("i2s", blob, w_scale, lin.M, lin.K, q, sc, y=y)

    def both():
        bn.bitnet_quant_act(x, q=q, act_scale=sc, act_sum=sm)
        gemm()

    ms_gemm = time_replays(torch, gemm, steps, warmup)
    ms_both = time_replays(torch, both, steps, warmup)
    ops = 2.0 * T * lin.K * lin.M
    out = {"workload": f"prefill {T}x{lin.K}x{lin.M}", "ms_gemm": ms_gemm, "ms_quant_plus_gemm": ms_both,
           "int8_tops": ops / ms_gemm / 1e9, "int8_tops_with_quant": ops / ms_both / 1e9}
    # context: the library's int8 GEMM on the same shape with BOTH operands already int8 in HBM (four times the
    # weight bytes of the packed form, no unpacking): what the tensor cores deliver here, not a comparison arm
    try:
        wi = torch.randint(-1, 2, (lin.M, lin.K), dtype=torch.int8, device="cuda").t()
        ms_lib = time_replays(torch, lambda: torch._int_mm(q, wi), steps, warmup)
        out["library_int8_gemm_tops"] = ops / ms_lib / 1e9
        out["frac_of_library_int8_gemm"] = out["int8_tops"] / out["library_int8_gemm_tops"]
    except Exception as e:          # noqa: BLE001 - the line is context only
        out["library_int8_gemm_tops"] = None
        out["library_int8_gemm_note"] = str(e)[:80]
    return out


def bench_elut(bn, torch, synth, wl, layers, card, steps, warmup, check):
    """The sweep's shapes with weights of cardinality `card` (App. A, Table 3) stored as pair indices: one
    bitnet_elut_linear_group call per step (quantiser + scan kernel in pair mode + rescale).  With `check`, sampled rows
    of every linear of layer 0 are compared with the oracle."""
    import numpy as np
    dev = torch.device("cuda")
    items, kept, nbytes = [], [], 0
    for layer in range(layers):
        for j, lin in enumerate(wl.linears):
            w = synth.uniform_alphabet(wl.seed, 1000 + layer * 8 + j, lin.M, lin.K, card, device=dev)
            x = wl.activations(layer, j, 1)
            if layer == 0:
                rows = np.unique(np.concatenate([[0, lin.M - 1], np.random.default_rng(j).integers(0, lin.M, 30)]))
                kept.append((rows, w[torch.as_tensor(rows, device=dev)].cpu().numpy(), x.numpy()))
            blob = bn.bitnet_pack_elut(card, 2, w, check=False)
            del w
            items.append(dict(C=card, g=2, packed=blob, w_scale=0.5, M=lin.M, K=lin.K, x=x.to(dev),
                              q=torch.empty((1, lin.K), dtype=torch.int8, device=dev),
                              act_scale=torch.empty(1, dtype=torch.float32, device=dev),
                              y=torch.empty((1, lin.M), dtype=torch.float32, device=dev)))
            nbytes += blob.numel()
    grp = bn.make_elut_group(items)
    ms = time_replays(torch, lambda: bn.bitnet_elut_linear_group(grp), steps, warmup)
    out = {"cardinality": card, "group": 2, "bits_per_weight": 8.0 * nbytes / sum(l.M * l.K for l in wl.linears) / layers,
           "packed_bytes": nbytes, "ms_per_step": ms, "value": nbytes / ms / 1e6, "unit": UNIT,
           "frac_of_hbm_peak": nbytes / ms / 1e6 / peaks()["hbm"],
           "kernel": "gemv_tl2_scan_kernel, " + ("mask mode" if card == 4 else "pair mode") + " (one bitnet_elut_linear_group call per step)"}
    if check:
        import oracle
        ok = True
        for (rows, w_rows, x), d in zip(kept, items):
            q, sc, _ = oracle.quant_act(x)
            acc = oracle.mpgemm_def(q, np.ascontiguousarray(w_rows))
            y_ref = oracle.dequant(acc, sc, 0.5)[0]
            y = d["y"].cpu().numpy()[0, rows].astype(np.float64)
            ok &= bool(np.all(np.abs(y - y_ref) <= 1e-6 * np.abs(y_ref)) and np.all(y[acc[0] == 0] == 0.0))
        out["verified"] = ok
    return out


def verify_against_oracle(oracle, sw, wl, torch, ys_layer0, rows_per_linear=8):
    """Part of the CPU-baseline leg: the y the GPU produced in the timed steps against the oracle -- every row of
    layer 0 (whose oracle results `ys_layer0` come from the timed CPU run) and `rows_per_linear` sampled rows of
    every other linear, their weights re-drawn on the host.  Returns (ok, rows checked)."""
    import numpy as np
    y_all = sw.y_dev.cpu().numpy()
    checked, ok, failures = 0, True, []

    def close(y, y_ref, acc):
        return bool(np.all(np.abs(y.astype(np.float64) - y_ref) <= 1e-6 * np.abs(y_ref)) and np.all(y[acc == 0] == 0.0))

    nl = len(sw.lin)
    for i in range(sw.n_linears()):
        layer, j = divmod(i, nl)
        lin = sw.lin[j]
        y = y_all[sw.y_off[i]: sw.y_off[i] + lin.M]
        if layer == 0:
            acc, sc, y_ref = ys_layer0[j]
            good = close(y, y_ref[0], acc[0])
            if not good:
                failures.append(i)
            ok &= good
            checked += lin.M
            continue
        rng = np.random.default_rng(1000 + i)
        rows = np.unique(np.concatenate([[0, lin.M - 1], rng.integers(0, lin.M, rows_per_linear)]))
        w_rows = np.stack([wl.weights(layer, j, row_start=int(r), rows=1).numpy()[0] for r in rows])
        q, sc, _ = oracle.quant_act(np.ascontiguousarray(wl.activations(layer, j, 1).numpy()))
        acc = oracle.mpgemm_def(q, np.ascontiguousarray(w_rows))
        y_ref = oracle.dequant(acc, sc, sw.w_scale[i])
        good = close(y[rows], y_ref[0], acc[0])
        if not good:
            failures.append(i)
        ok &= good
        checked += len(rows)
    return bool(ok), checked, failures[:16]


def run_ours(args):
    import torch
    import paper_2502_11880_b200 as bn
    from paper_2502_11880_b200 import synth

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    bn.lib()   # fail loudly here if the extension is missing
    if args.no_early_start:
        bn.bitnet_set_early_start(False)
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    pk = peaks()
    wl = synth.CONFIGS["sweep100b"]
    layers = args.layers or wl.layers
    fmts = ["i2s", "tl2", "tl1"] if not args.skip_tl2 else ["i2s"]
    sw = Sweep(bn, torch, wl, fmts, layers, torch.device("cuda", local))
    n_lin = sw.n_linears()

    # ---- headline: I2_S sweep, quantiser + GEMV + rescale, ONE bitnet_linear_group call per step
    sw.step_group("i2s")
    torch.cuda.synchronize()
    sampler = ClockSampler(local) if rank == 0 else None
    ms_step = time_replays(torch, lambda: sw.step_group("i2s"), args.steps, args.warmup, dist)
    clocks = sampler.stop() if sampler else None
    value = whole_job_value(sw.bytes["i2s"], world, ms_step)
    achieved = sw.bytes["i2s"] / ms_step / 1e6
    launches_per_step = -(-n_lin // 409)      # the grouped kernel takes up to 409 items per launch

    # ---- end to end through the host-buffer entry point
    ms_e2e = time_replays(torch, lambda: (sw.step_host("i2s"), torch.cuda.current_stream().synchronize()),
                          max(2, args.steps // 4), 3, dist)
    e2e_val = whole_job_value(sw.bytes["i2s"], world, ms_e2e)
    # leave the device-resident results of the grouped call in y_dev for the verification below
    sw.y_dev.zero_()
    sw.step_group("i2s")
    torch.cuda.synchronize()

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8",
        "data": "synthetic",
        "config": {"workload": "sweep100b", "layers": layers, "linears_per_layer": 4, "tokens": 1, "format": "i2s",
                   "packed_bytes": sw.bytes["i2s"], "parallelism": f"replicas x{world}",
                   "l2": "inputs (17 GB of weights) exceed L2; no flush needed",
                   "launch": f"one bitnet_linear_group call per step = {launches_per_step} persistent kernel launch(es) over "
                             f"{n_lin} linears (quantiser fused)",
                   "pct_of_8TBps": 100.0 * (value / world) / 8000.0},
        "e2e": {"value": e2e_val, "unit": UNIT, "ms_per_step": ms_e2e,
                "h2d_bytes_per_step": int(sw.x_host.numel() * 4), "d2h_bytes_per_step": int(sw.y_host.numel() * 4),
                "note": "one bitnet_linear_host_batch call per step: pinned fp32 x -> device, grouped kernels (quantiser + mpGEMV + rescale), fp32 y -> pinned host, in five groups (1, 4, 6, 4 and 1 sixteenths of the linears) whose copies overlap the neighbouring groups' kernels; weights resident"},
        "gpu_launches": launches_per_step * args.steps,
        "roofline": {"bound": "hbm", "kernel": "gemv_i2s_group_kernel (quantiser fused)", "achieved": achieved,
                     "peak": pk["hbm"], "unit": "GB/s", "frac": achieved / pk["hbm"], "peak_source": pk["which"],
                     "launches_per_step": launches_per_step,
                     "bytes_per_launch": sw.bytes["i2s"] / launches_per_step,
                     "us_per_launch": 1e3 * ms_step / launches_per_step,
                     "traffic": NCU_TRAFFIC_PER_ALGORITHMIC_BYTE * sw.bytes["i2s"] / launches_per_step,
                     "traffic_note": "dram read+write bytes of an ncu capture of the grouped kernel on 4 layers of the "
                                     "sweep over the packed weight bytes of that launch, scaled by bytes to the full launch"},
        "clocks": clocks,
    }

    if rank == 0:
        # ---- context: the same pass as one launch per linear (the fused single-linear kernel, CUDA graphs)
        g_full = sw.make_graph("i2s")
        ms_per_linear = time_replays(torch, g_full, max(5, args.steps // 2), args.warmup)
        line["per_linear_launches"] = {"ms_per_step": ms_per_linear, "value": sw.bytes["i2s"] / ms_per_linear / 1e6, "unit": UNIT,
                                       "launch": f"{g_full.n_graphs} CUDA graph replays per step, one fused kernel per linear"}
        del g_full
        if "tl2" in fmts:
            # the same sweep in the TL2 encoding: (a) the scan kernel (decode table + tensor cores, one persistent
            # kernel per step), (b) the activation-table kernel of Alg. 2 (three launches per linear)
            ms_tl = time_replays(torch, lambda: sw.step_group("tl2"), max(5, args.steps // 2), args.warmup)
            bn.bitnet_set_tl2_lookup(True)
            ms_lut = time_replays(torch, lambda: sw.step_group("tl2"), max(3, args.steps // 5), args.warmup)
            bn.bitnet_set_tl2_lookup(False)
            line["tl2"] = {"packed_bytes": sw.bytes["tl2"], "ms_per_step": ms_tl, "value": sw.bytes["tl2"] / ms_tl / 1e6,
                           "unit": UNIT, "frac_of_hbm_peak": sw.bytes["tl2"] / ms_tl / 1e6 / pk["hbm"],
                           "i2s_equivalent_GBps": sw.bytes["i2s"] / ms_tl / 1e6,
                           "kernel": "gemv_tl2_scan_kernel (one bitnet_linear_group call per step)",
                           "lookup_table_kernel": {"ms_per_step": ms_lut, "value": sw.bytes["tl2"] / ms_lut / 1e6,
                                                   "frac_of_hbm_peak": sw.bytes["tl2"] / ms_lut / 1e6 / pk["hbm"],
                                                   "kernel": "quantiser + tl_table_kernel + gemv_tl_kernel per linear"}}
            # TL1 (2 bits per weight, Table 4): the scan kernel's pair mode
            ms_tl1 = time_replays(torch, lambda: sw.step_group("tl1"), max(5, args.steps // 2), args.warmup)
            line["tl1"] = {"packed_bytes": sw.bytes["tl1"], "ms_per_step": ms_tl1, "value": sw.bytes["tl1"] / ms_tl1 / 1e6,
                           "unit": UNIT, "frac_of_hbm_peak": sw.bytes["tl1"] / ms_tl1 / 1e6 / pk["hbm"],
                           "kernel": "gemv_tl2_scan_kernel, arithmetic mode (one bitnet_linear_group call per step)"}
            if not args.skip_batched:
                nb = max(3, args.steps // 10)
                line["tl2"]["batched"] = [bench_batched(sw, torch, T, nb, 3, "tl2") for T in (2, 4, 8)]
                line["tl1"]["batched"] = [bench_batched(sw, torch, T, nb, 3, "tl1") for T in (2, 4, 8)]
            sw.step_group("tl2")        # the verification below sees the scan kernel's y
        if not args.skip_batched:
            line["batched_decode"] = {
                "note": "the same sweep with T tokens per linear, one bitnet_linear_group call per step, inputs resident",
                "runs": [bench_batched(sw, torch, T, max(3, args.steps // 5), 3) for T in (2, 4, 8, 16, 32, 64, 128)]}
        if world == 1 and not args.skip_cpu:
            # ---- CPU baseline leg: the oracle, as it stands, on one full layer of the sweep for about 10 s on the
            # host cores; its results then check the y the GPU left in device memory
            import oracle
            oracle.build()
            sample = oracle_layer(wl)
            nb = sum(w.shape[0] * w.shape[1] // 4 for w, _ in sample)
            reps, t0 = 0, time.perf_counter()
            while True:
                ys0 = oracle_step(oracle, sample, sw.w_scale[:len(sample)])
                reps += 1
                dt = time.perf_counter() - t0
                if dt > 10.0 or reps >= 50:
                    break
            line["cpu_baseline"] = {"value": nb * reps / dt / 1e9, "unit": UNIT, "cores": oracle.num_threads(),
                                    "kind": "oracle",
                                    "ms_per_step_extrapolated": dt / reps * 1e3 * layers,
                                    "sample": f"layer 0 of the sweep (4 linears, {nb / 1e6:.1f} MB as I2_S) x {reps} "
                                              f"repetitions in {dt:.1f} s: quantiser + definition + rescale; the step "
                                              f"time is that layer's time x {layers} layers (extrapolated)"}
            ok, rows, failures = verify_against_oracle(oracle, sw, wl, torch, ys0)
            line["verified"] = ok
            line["verified_rows"] = rows
            if failures:
                line["verify_failures"] = failures
        del sw
        torch.cuda.empty_cache()
        if not args.skip_elut:
            # beyond ternary (App. A): the same shapes with weights of cardinality 5 (2.5 bits per weight) and 4 (2 bits)
            line["elut"] = [bench_elut(bn, torch, synth, wl, layers, card, max(5, args.steps // 2), args.warmup,
                                       world == 1 and not args.skip_cpu) for card in (5, 4)]
            torch.cuda.empty_cache()
        if not args.skip_small:
            line["small_configs"] = bench_small_configs(bn, torch, synth, max(5, args.steps // 2), 3)
        if not args.skip_ceilings:
            line["ceilings"] = bench_ceilings(bn, torch, (clocks or {}).get("sm_mhz"))
        if not args.skip_prefill:
            pf = bench_prefill(bn, torch, synth, max(3, args.steps // 2), 3)
            pf["frac_of_int8_peak"] = pf["int8_tops"] / (2.0 * pk["bf16"])
            pf["int8_peak_used"] = f"2 x {pk['which']} bf16 dense ({pk['bf16']} TFLOP/s)"
            lib8 = (line.get("ceilings") or {}).get("library_int8_gemm_8192cubed_tops")
            if lib8:
                pf["frac_of_library_int8_gemm_8192cubed"] = pf["int8_tops"] / lib8
            line["prefill"] = pf
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--layers", type=int, default=0, help="fewer layers than the workload's 80 (debugging only)")
    ap.add_argument("--skip-tl2", action="store_true")
    ap.add_argument("--skip-prefill", action="store_true")
    ap.add_argument("--skip-cpu", action="store_true")
    ap.add_argument("--skip-batched", action="store_true")
    ap.add_argument("--skip-elut", action="store_true", help="skip the sweeps with weights of cardinality 5 and 4")
    ap.add_argument("--skip-small", action="store_true", help="skip the timings of the three small workloads")
    ap.add_argument("--skip-ceilings", action="store_true", help="skip the read-stream / issue-rate / int8 GEMM ceilings")
    ap.add_argument("--no-early-start", action="store_true",
                    help="launch every kernel in plain stream order (no programmatic dependent launch)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
