#!/usr/bin/env python
"""Benchmark of the N:M structured-binary linear layer on B200.

One pass = one decode pass (batch 1) over the three MLP linears of a LLaMA-2-7B decoder layer at
6:8: gate 11008x4096 and up 11008x4096 read the same fp16 input, down 4096x11008 reads gate's
fp16 output; the three GEMVs are queued by stb_layer_stack on one stream.  The layers are the
workload's own: dense synthetic weights put through the method's quantizer (the CPU oracle's, run
here to PREPARE the inputs; it is never on the timed path).  The headline value is the effective
HBM bandwidth: bytes of packed weights streamed per second.  Weights are resident in HBM; every
pass reads another copy of the packed layers so that no byte comes from L2.  A "step" of
--steps is as many passes as it takes for the timed region to last a quarter of a second.

  python bench.py [--gpus N] [--steps K] [--warmup W]          CUDA path, one JSON line
  python bench.py --impl reference ...                         the CPU oracle on the host cores

With N > 1 (launched by torch.distributed.run, one rank per GPU) every rank runs an independent
replica of the same workload: the layer is not sharded, there is no data-path collective.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

import stb_inputs as si

METRIC = "gemv_packed_weight_bandwidth"
UNIT = "GB/s"
WORKLOAD = ("llama2-7b-mlp gate/up 11008x4096 + down 4096x11008, 6:8, block 128, batch-1 decode GEMV, "
            "layers made by the oracle's quantizer from the dense synthetic weights")
MLP = ("gate", "up", "down")
L2_BYTES = 126 * 1024 * 1024
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
MIN_TIMED_S = 0.25
KERNEL_SOURCES = ("stb_stack.cu", "stb_decode.cuh", "stb_layout.cuh", "stb_ptx.cuh")
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "traffic_stack_kernel_llama7b_mlp_6of8_batch1.txt")


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        d["_source"] = "measured"
        return d
    d = dict(FALLBACK_PEAKS)
    d["_source"] = "fallback"
    return d


def kernel_source_hash() -> str:
    h = hashlib.sha256()
    for f in KERNEL_SOURCES:
        h.update(open(os.path.join(ROOT, "paper_2408_01803_b200", "csrc", f), "rb").read())
    return h.hexdigest()[:16]


def captured_traffic():
    """dram__bytes_read.sum + dram__bytes_write.sum per launch of the GEMV on this workload, from the ncu summary
    under profiles/ -- or None (with the reason) when there is none or the kernel's sources changed since."""
    if not os.path.exists(TRAFFIC_FILE):
        return None, "no capture on file"
    kv = {}
    for line in open(TRAFFIC_FILE):
        if "=" in line and not line.lstrip().startswith("#"):
            k, v = line.split("=", 1)
            kv[k.strip()] = v.split("#")[0].strip()
    if kv.get("source_sha256") != kernel_source_hash():
        return None, "kernel sources changed since the capture (%s)" % os.path.basename(TRAFFIC_FILE)
    return float(kv["dram_bytes_per_launch"]), os.path.basename(TRAFFIC_FILE)


def quantized(config, name, N=0, verbose=True):
    """The workload's layer as the method makes it (oracle quantizer, cached on disk): input preparation."""
    import oracle.workloads as wl
    n, m, NN, seed = si.workload_layer(config, name, N)
    return wl.quantized_layer(n, m, NN, seed, verbose=verbose)


def salient_histogram(d):
    import oracle.workloads as wl
    c = wl.salient_counts(d)
    return {"mean": round(float(c.mean()), 2), "max": int(c.max()),
            "blocks_by_count": {"1-4": int(((c >= 1) & (c <= 4)).sum()), "5-8": int(((c >= 5) & (c <= 8)).sum()),
                                "9-16": int(((c >= 9) & (c <= 16)).sum()), "17-32": int((c >= 17).sum()), "0": int((c == 0).sum())}}


# ------------------------------------------------------------------------------------------
# clocks: NVML polled from a thread while the timed region runs (read-only queries)
class ClockSampler:
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting",
               0x10: "sync_boost"}

    def __init__(self, torch_device_index: int):
        self.samples, self.h, self.nv, self._stop, self._thr = [], None, None, threading.Event(), None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            uuid = "GPU-" + str(torch.cuda.get_device_properties(torch_device_index).uuid)
            try:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid)
            self.nv = pynvml
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception as e:  # noqa: BLE001
            self.err = repr(e)

    def sample(self):
        if self.h is None:
            return
        nv = self.nv
        try:
            mhz = int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
            try:
                mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
            except Exception:
                mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
            self.samples.append((time.perf_counter(), mhz, mask))
        except Exception:
            pass

    def start(self, period=0.01):
        def loop():
            while not self._stop.is_set():
                self.sample()
                time.sleep(period)
        self._thr = threading.Thread(target=loop, daemon=True)
        self._thr.start()

    def stop(self, t0, t1):
        self._stop.set()
        if self._thr:
            self._thr.join()
        if self.h is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "note": "NVML unavailable: " + getattr(self, "err", "")}
        inside = [s for s in self.samples if t0 <= s[0] <= t1] or self.samples[-1:]
        mask = 0
        for s in inside:
            mask |= s[2]
        reasons = sorted(v for k, v in self.REASONS.items() if mask & k)
        return {"sm_mhz": float(np.median([s[1] for s in inside])) if inside else None,
                "sm_max_mhz": self.max_mhz, "reasons": reasons, "samples": len(inside)}


# ------------------------------------------------------------------------------------------
def oracle_pass(Ls, xs, rows, threads=0):
    """One decode pass of the oracle over the listed output rows of each layer (fp32 decode from
    the logical arrays + float64 multiply-accumulate).  Returns seconds."""
    import oracle
    t0 = time.perf_counter()
    for L, x, r in zip(Ls, xs, rows):
        oracle.layer_rows(L, r, x, nthreads=threads)
    return time.perf_counter() - t0


def reference_arm(args):
    """The CPU oracle, as it stands, on the host cores: same workload, metric and unit.  Each step
    is a bounded sample of output rows so that the run ends within minutes."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    import oracle.workloads as wl
    oracle.build()
    ds = [quantized(2, name, verbose=False) for name in MLP]
    Ls = [wl.as_logical(d) for d in ds]
    x0 = si.activations(1, 4096, si.seed_for(2, 8)).astype(np.float64)
    x1 = si.activations(1, 11008, si.seed_for(2, 9)).astype(np.float64)     # stands in for gate's output
    xs = [x0, x0, x1]
    cores = oracle.hardware_threads()
    # calibrate the row rate on a small sample, then size a step for ~60 s over all steps
    probe = [np.arange(0, d["n"], 16, dtype=np.int32) for d in ds]
    tp = oracle_pass(Ls, xs, probe)
    frac_probe = 1.0 / 16
    budget = 60.0 / max(1, args.steps + args.warmup)
    frac = min(1.0, frac_probe * budget / max(tp, 1e-6))
    stride = max(1, int(np.ceil(1.0 / frac)))
    rows = [np.arange(0, d["n"], stride, dtype=np.int32) for d in ds]
    bytes_step = sum(wl.stream_bytes(d) * len(r) / (-(-d["n"] // 32) * 32) for d, r in zip(ds, rows))
    for _ in range(args.warmup):
        oracle_pass(Ls, xs, rows)
    t = 0.0
    for _ in range(args.steps):
        t += oracle_pass(Ls, xs, rows)
    val = bytes_step * args.steps / t / 1e9
    sample = "every %d-th output row of gate, up and down per step (%d rows, %.2f MB of packed weights)" % (
        stride, sum(len(r) for r in rows), bytes_step / 1e6)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "batch": 1, "sample": sample},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


# ------------------------------------------------------------------------------------------
def clone_layer(stb, lay, used):
    return stb.PackedLayer(lay.n, lay.m, lay.N, lay.buf[:used].clone(), lay.dev_status)


class Workload:
    """The MLP layers packed on the device, `copies` times each at distinct addresses."""

    def __init__(self, stb, torch, copies, resident=True):
        self.stb, self.torch, self.resident = stb, torch, resident
        self.logical = [quantized(2, name) for name in MLP]
        self.layers = []          # [copy][k]
        first = [stb.pack_numpy(d) for d in self.logical]
        torch.cuda.synchronize()
        for lay in first:
            assert int(lay.dev_status.item()) == 0
        self.infos = [lay.info() for lay in first]
        for c in range(copies):
            self.layers.append(first if c == 0 else [clone_layer(stb, l, self.infos[k]["used_bytes"]) for k, l in enumerate(first)])
        self.status = torch.zeros(1, dtype=torch.int32, device="cuda")
        self.x_np = si.activations(1, 4096, si.seed_for(2, 8))
        self.x = torch.from_numpy(self.x_np).cuda()
        self.h_gate = torch.zeros(1, 11008, dtype=torch.float16, device="cuda")
        self.h_up = torch.zeros(1, 11008, dtype=torch.float16, device="cuda")
        self.y = torch.zeros(1, 4096, dtype=torch.float32, device="cuda")
        self.steps = [stb.make_steps([(ls[0], self.x, self.h_gate), (ls[1], self.x, self.h_up),
                                      (ls[2], self.h_gate, self.y)]) for ls in self.layers]
        self.bytes_step = sum(i["stream_bytes"] for i in self.infos)
        self.ws = stb.resident_workspace(self.steps[0])      # one pass and many passes need the same workspace: it is sized by the largest group

    def step(self, c):
        if self.resident:
            self.stb.layer_stack_resident(None, self.ws, dev_status=self.status, marshalled=self.steps[c % len(self.steps)])
        else:
            self.stb.layer_stack(None, dev_status=self.status, marshalled=self.steps[c % len(self.steps)])

    def step_host(self, c, xh, yh):
        if self.resident:
            self.stb.layer_stack_resident_host(self.steps[c % len(self.steps)], self.ws, xh, yh, dev_status=self.status)
        else:
            self.stb.layer_stack_host(self.steps[c % len(self.steps)], xh, yh, dev_status=self.status)

    def run_steps(self, first, count):
        """`count` consecutive passes (copies first, first + 1, ...) as ONE call, the way a model's whole stack of
        linears is queued: stb_layer_stack_resident (one resident kernel for the whole list) or stb_layer_stack
        (one launch per group of same-input layers, chained by programmatic dependent launches)."""
        trip = []
        for c in range(first, first + count):
            ls = self.layers[c % len(self.layers)]
            trip += [(ls[0], self.x, self.h_gate), (ls[1], self.x, self.h_up), (ls[2], self.h_gate, self.y)]
        arr = self.stb.make_steps(trip)
        self._keep = getattr(self, "_keep", []) + [arr]
        if self.resident:
            self.stb.layer_stack_resident(None, self.ws, dev_status=self.status, marshalled=arr)
        else:
            self.stb.layer_stack(None, dev_status=self.status, marshalled=arr)


def capture(torch, fns):
    """One CUDA graph that runs every callable of `fns` once, in order."""
    g = torch.cuda.CUDAGraph()
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        fns[0]()                           # warm: module load, attribute set-up happen outside capture
    torch.cuda.current_stream().wait_stream(s)
    torch.cuda.synchronize()
    with torch.cuda.graph(g):
        for f in fns:
            f()
    return g


def time_graph(torch, g, calls_per_replay, min_calls=2000, warm=3):
    """Average microseconds per call of a captured sequence, CUDA events on the replay stream."""
    reps = max(3, -(-min_calls // calls_per_replay))
    for _ in range(warm):
        g.replay()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(reps):
        g.replay()
    e1.record()
    torch.cuda.synchronize()
    return 1e3 * e0.elapsed_time(e1) / (reps * calls_per_replay)


def rotating_copies(stb, lay, min_bytes=3 * L2_BYTES, lo=4, hi=48):
    info = lay.info()
    k = max(lo, min(hi, -(-min_bytes // info["stream_bytes"])))
    return [lay] + [clone_layer(stb, lay, info["used_bytes"]) for _ in range(k - 1)], info


def gemv_table(stb, torch, wl, pk):
    """Isolated per-layer GEMV timings, cold L2 (rotating over distinct packed copies), for the
    decode batches of the workload; plus the other decode shapes (quantizer-made layers as well) and a
    dense bf16 cuBLAS GEMV (torch.matmul) of the same shape as context."""
    out = []

    def one(name, copies, n, m, N, sbytes, batches):
        for b in batches:
            x = torch.from_numpy(si.activations(b, m, si.seed_for(2, 10 + b))).cuda()
            y = torch.empty(b, n, dtype=torch.float32, device="cuda")
            fns = [(lambda lay=lay: stb.gemv(lay, x, out=y)) for lay in copies]
            g = capture(torch, fns)
            us = time_graph(torch, g, len(fns))
            out.append({"layer": name, "n": n, "m": m, "N": N, "batch": b, "us_per_layer": round(us, 3),
                        "packed_MB": round(sbytes / 1e6, 3), "GBps": round(sbytes / us / 1e3, 1),
                        "frac_of_measured_hbm": round(sbytes / us / 1e3 / pk["hbm_gbs"], 4),
                        "frac_of_nominal_hbm_8TBps": round(sbytes / us / 1e3 / 8000.0, 4)})
            del g

    ncopy = len(wl.layers)
    one("gate/up 11008x4096 (isolated launches)", [wl.layers[c][k] for c in range(ncopy) for k in (0, 1)], 11008, 4096, 6,
        wl.infos[0]["stream_bytes"], (1, 4, 8, 16))
    one("down 4096x11008 (isolated launches)", [wl.layers[c][2] for c in range(ncopy)], 4096, 11008, 6,
        wl.infos[2]["stream_bytes"], (1, 4, 8, 16))
    # other decode shapes of the workload list (batch 1): 7B attention at 4:8, 13B block shapes at 5:8
    for label, config, name in (("7B q_proj 4096x4096", 1, "q"), ("13B q 5120x5120", 3, "q"),
                                ("13B gate 13824x5120", 3, "gate"), ("13B down 5120x13824", 3, "down")):
        d = quantized(config, name)
        lay = stb.pack_numpy(d)
        copies, info = rotating_copies(stb, lay)
        one(label, copies, d["n"], d["m"], d["N"], info["stream_bytes"], (1,))
        del copies, lay
        torch.cuda.empty_cache()
    # dense bf16 context
    ctx = []
    for name, n, m in (("gate/up 11008x4096", 11008, 4096), ("down 4096x11008", 4096, 11008)):
        k = max(2, -(-3 * L2_BYTES // (2 * n * m)))
        Ws = [torch.randn(n, m, device="cuda", dtype=torch.bfloat16) for _ in range(k)]
        x = torch.randn(m, 1, device="cuda", dtype=torch.bfloat16)
        y = torch.empty(n, 1, device="cuda", dtype=torch.bfloat16)
        g = capture(torch, [(lambda W=W: torch.matmul(W, x, out=y)) for W in Ws])
        us = time_graph(torch, g, k, min_calls=400)
        ctx.append({"layer": name, "kind": "dense bf16 torch.matmul (cuBLAS), batch 1", "us_per_layer": round(us, 3),
                    "dense_MB": round(2 * n * m / 1e6, 2), "GBps": round(2 * n * m / us / 1e3, 1)})
        del g, Ws
        torch.cuda.empty_cache()
    return out, ctx


def gemm_table(stb, torch, pk, real_ffn, only=None):
    """Prefill GEMM (stb_gemm, tcgen05) on the LLaMA-2-70B linear shapes at 4:8, 2048 bf16 tokens, with a
    dense bf16 cuBLAS GEMM (torch.matmul) of the same shape beside it.  q/o and k/v come from the oracle's
    quantizer; the two tall / wide FFN layers (minutes on the CPU) from stb_quantize on the GPU, which the parity
    tests hold equal to the oracle bit for bit (--tiled-ffn: repeat the quantized q layer instead)."""
    T, N = 2048, 4
    views = {"keep": np.uint8, "sign": np.uint8, "region": np.int16, "sign2": np.int32, "salient": np.int64, "scale": np.int16}

    def up(d):
        return {k: torch.from_numpy(np.ascontiguousarray(d[k]).view(v)).cuda() for k, v in views.items()}

    def rows_x(t):             # 28672 = 3.5 x 8192 rows
        return {k: (v if k == "salient" else torch.cat([v] * 3 + [v[:4096]], 0).contiguous()) for k, v in t.items()}

    def cols_x(t):             # 28672 = 3.5 x 8192 columns (whole 128-column blocks)
        out = {}
        for k, v in t.items():
            if k == "salient":
                out[k] = torch.cat([v] * 3 + [v[:32]], 0).contiguous()
            else:
                half = v.shape[1] // 2
                out[k] = torch.cat([v] * 3 + [v[:, :half]], 1).contiguous()
        return out

    def on_gpu(name):
        # the workload's dense weights through stb_quantize (equal to the oracle's quantizer bit for bit in the parity tests)
        n, m, NN, seed = si.workload_layer(4, name)
        W = torch.from_numpy(si.dense_weight(n, m, seed)).cuda()
        xn = torch.from_numpy(si.calib_norms(m, seed)).cuda()
        t = stb.quantize(W, xn, NN)
        torch.cuda.synchronize()
        del W
        sal = t["salient"].cpu().numpy().view(np.uint64)
        return t, salient_histogram({"salient": sal})

    dq = quantized(4, "q")
    b = up(dq)
    cases = [("q/o 8192x8192", 8192, 8192, b, "oracle-quantized", salient_histogram(dq))]
    dk = quantized(4, "k")
    cases.append(("k/v 1024x8192", 1024, 8192, up(dk), "oracle-quantized", salient_histogram(dk)))
    if real_ffn:
        tg, hg = on_gpu("gate")
        cases.append(("gate/up 28672x8192", 28672, 8192, tg, "stb_quantize (GPU quantizer) of the workload's dense weights", hg))
        del tg
        td, hd = on_gpu("down")
        cases.append(("down 8192x28672", 8192, 28672, td, "stb_quantize (GPU quantizer) of the workload's dense weights", hd))
        del td
    else:
        cases += [("gate/up 28672x8192", 28672, 8192, rows_x(b), "rows of the quantized q layer repeated 3.5 times", None),
                  ("down 8192x28672", 8192, 28672, cols_x(b), "column blocks of the quantized q layer repeated 3.5 times", None)]
    out = []
    for name, n, m, t, how, hist in cases:
        if only and not name.startswith(only):
            continue
        lay = stb.pack(n, m, N, t["keep"], t["sign"], t["region"], t["sign2"], t["salient"], t["scale"])
        torch.cuda.synchronize()
        assert int(lay.dev_status.item()) == 0, name
        x = torch.randn(T, m, device="cuda").to(torch.bfloat16)
        y = torch.empty(T, n, dtype=torch.bfloat16, device="cuda")
        need = stb.gemm_workspace(n, m, N, T)
        ws = torch.empty(max(need, 16), dtype=torch.uint8, device="cuda")
        flush = torch.empty(160 << 20, dtype=torch.uint8, device="cuda")

        def timed(fn, reps=8):
            for _ in range(3):
                fn()
            ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
            for e0, e1 in ev:
                flush.zero_()                      # L2 flush between timed iterations
                e0.record(); fn(); e1.record()
            torch.cuda.synchronize()
            return 1e3 * float(np.median([e0.elapsed_time(e1) for e0, e1 in ev]))

        us = timed(lambda: stb.gemm(lay, x, out=y, ws=ws))
        assert int(lay.dev_status.item()) == 0
        W = torch.randn(n, m, device="cuda").to(torch.bfloat16)
        usd = timed(lambda: torch.matmul(x, W.t(), out=y))
        fl = 2.0 * n * m * T
        row = {"layer": name, "n": n, "m": m, "tokens": T, "N": N, "inputs": how, "us": round(us, 1), "dense_TFLOPs": round(fl / us / 1e6, 1),
               "frac_of_measured_bf16_burst": round(fl / us / 1e6 / pk["bf16_tflops"], 4),
               "frac_of_nominal_bf16_2250TF": round(fl / us / 1e6 / 2250.0, 4),
               "frac_of_measured_bf16_sustained": round(fl / us / 1e6 / pk["bf16_tflops_sustained"], 4),
               "useful_TFLOPs": round(fl * N / 8 / us / 1e6, 1), "split_k_workspace_MB": round(need / 1e6, 1),
               "cublas_bf16_us": round(usd, 1), "cublas_bf16_TFLOPs": round(fl / usd / 1e6, 1)}
        # the same in the form of the headline's roofline object: a dense contraction against the measured cuBLAS burst peak
        # (the kernel is timed alone); the whole call (gather, GEMM, sum of K parts) counts as the kernel's time
        row["roofline"] = {"bound": "tensor", "achieved": round(fl / us / 1e6, 1), "peak": pk["bf16_tflops"], "unit": "TFLOP/s",
                           "frac": round(fl / us / 1e6 / pk["bf16_tflops"], 4), "traffic": None, "kernel": "stb::gemm_kernel",
                           "peak_source": pk["_source"]}
        if hist:
            row["salient_columns_per_block"] = hist
        out.append(row)
        del lay, W, x, y, ws, flush
        torch.cuda.empty_cache()
    return out


CALL = {True: "stb_layer_stack_resident (one resident kernel)", False: "stb_layer_stack (per-layer launches)",
        "tc": "stb_gemm_f16 per linear (tcgen05, 64-token tile; gather + GEMM + sum of K parts = 3 launches each)"}


def decoder(h, f):
    return [("q", h, h), ("k", h, h), ("v", h, h), ("o", h, h), ("gate", f, h), ("up", f, h), ("down", h, f)]


def build_stack(stb, config, names_N):
    """Packed layers of a stack, every one at its own address; one quantizer-made layer per (shape, N) family."""
    cache, layers = {}, []
    for name, N in names_N:
        n, m, NN, seed = si.workload_layer(config, name, N)
        key = (n, m, NN)
        if key not in cache:
            fam = {"k": "q", "v": "q", "o": "q", "up": "gate"}.get(name, name)
            base = stb.pack_numpy(quantized(config, fam, N))
            cache[key] = (base, base.info())
        base, info = cache[key]
        layers.append((name, clone_layer(stb, base, info["used_bytes"]), info["stream_bytes"]))
    return layers


def run_stack(stb, torch, layers, h, f, batch, nl, min_calls, resident):
    """All linears of `nl` decoder layers as ONE stb_layer_stack_resident (or stb_layer_stack) call in a CUDA graph;
    microseconds per call."""
    x = torch.from_numpy(si.activations(batch, h, si.seed_for(5, 40))).cuda()
    hb = [torch.empty(batch, h, dtype=torch.float16, device="cuda") for _ in range(5)]     # q k v o + layer output
    fb = [torch.empty(batch, f, dtype=torch.float16, device="cuda") for _ in range(2)]
    steps, cur = [], x
    for l in range(nl):
        q, k, v, o, gate, up, down = [lay for _, lay, _ in layers[7 * l: 7 * l + 7]]
        steps += [(q, cur, hb[0]), (k, cur, hb[1]), (v, cur, hb[2]), (o, hb[0], hb[3]), (gate, hb[3], fb[0]),
                  (up, hb[3], fb[1]), (down, fb[0], hb[4])]
        cur = hb[4]      # (the data flow of attention / activation functions is not part of this path)
    arr = stb.make_steps(steps)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    if resident == "tc":
        need = max(stb.gemm_f16_workspace(lay.n, lay.m, lay.N, batch) for lay, _, _ in steps)
        wsb = torch.empty(max(need, 256), dtype=torch.uint8, device="cuda")
        def fn():
            for lay, xin, yout in steps:
                stb.gemm_f16(lay, xin, out=yout, ws=wsb)
        status = None
    elif resident:
        ws = stb.resident_workspace(arr)
        fn = lambda: stb.layer_stack_resident(None, ws, dev_status=status, marshalled=arr)
    else:
        fn = lambda: stb.layer_stack(None, dev_status=status, marshalled=arr)
    g = capture(torch, [fn])
    us = time_graph(torch, g, 1, min_calls=min_calls)
    if status is None:
        assert all(int(t.item()) == 0 for t in {id(lay.dev_status): lay.dev_status for lay, _, _ in steps}.values())
    else:
        assert int(status.item()) == 0
    return us


def stack_tables(stb, torch, pk):
    """Whole decoder stacks as single stb_layer_stack calls (the other decode workloads):
      * one LLaMA-2-13B decoder block at 5:8, batch 1 (q/k/v, o, gate/up, down chained on one stream);
      * all 224 linears of a 32-layer LLaMA-2-7B stack with N drawn per decoder layer from {4, 5, 6}
        (seeded), batch 1, 8 and 64 -- the largest decode workload; its batch-1 line carries its own roofline.
    One layer is quantized per (shape, N) family and packed once per use at its own address (the kernels'
    work does not depend on which layer of a family it is), so that the 2.5-3.1 GB of a 7B stack are all
    distinct memory."""
    out = []
    l13 = build_stack(stb, 3, [(nm, 5) for nm, _, _ in decoder(5120, 13824)])
    b13 = sum(b for _, _, b in l13)
    for resident in (True, False):
        us = run_stack(stb, torch, l13, 5120, 13824, 1, 1, 200, resident)
        out.append({"stack": "LLaMA-2-13B decoder block, 7 linears, 5:8, batch 1", "call": CALL[resident], "us": round(us, 1),
                    "packed_MB": round(b13 / 1e6, 1), "GBps": round(b13 / us / 1e3, 1),
                    "frac_of_measured_hbm": round(b13 / us / 1e3 / pk["hbm_gbs"], 4)})
    del l13
    torch.cuda.empty_cache()
    Nl = si.stack_N_per_layer(32)
    names_N = [(nm, Nl[l]) for l in range(32) for nm, _, _ in decoder(4096, 11008)]
    l7 = build_stack(stb, 5, names_N)
    b7 = sum(b for _, _, b in l7)
    for batch, resident in ((1, True), (1, False), (8, True), (8, False), (64, False), (64, "tc")):
        # resident: 128 groups of same-input linears = two launches of 64 groups; per-layer launches: q/k/v as one grid,
        # o, gate/up as one grid, down = 128 launches
        launches = 2 if resident is True else 32 * 4
        us = run_stack(stb, torch, l7, 4096, 11008, batch, 32, 20, resident)
        row = {"stack": "LLaMA-2-7B, 32 decoder layers x 7 linears, N per layer from {4,5,6} (%d/%d/%d layers)" % (
                   Nl.count(4), Nl.count(5), Nl.count(6)), "call": CALL[resident], "batch": batch, "us": round(us, 1),
               "packed_GB": round(b7 / 1e9, 3), "GBps": round(b7 / us / 1e3, 1),
               "frac_of_measured_hbm": round(b7 / us / 1e3 / pk["hbm_gbs"], 4), "us_per_linear": round(us / 224, 2)}
        if batch == 1 and resident is True:
            row["roofline"] = {"bound": "hbm", "achieved": round(b7 / us / 1e3, 1), "peak": pk["hbm_gbs"], "unit": "GB/s",
                               "frac": round(b7 / us / 1e3 / pk["hbm_gbs"], 4), "traffic": None,
                               "kernel": "stb::stack_kernel", "bytes_per_launch": round(b7 / launches),
                               "launch_us": round(us / launches, 3), "launches": launches, "peak_source": pk["_source"]}
        out.append(row)
    del l7
    torch.cuda.empty_cache()
    return out


def quantizer_timing(stb, torch):
    """stb_quantize on the dense gate layer of the workload (11008 x 4096, 6:8): milliseconds, with the oracle's time for
    the same layer beside it when it was measured in this run."""
    n, m, N, seed = si.workload_layer(2, "gate")
    W = torch.from_numpy(si.dense_weight(n, m, seed)).cuda()
    xn = torch.from_numpy(si.calib_norms(m, seed)).cuda()
    stb.quantize(W, xn, N)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(3):
        stb.quantize(W, xn, N)
    e1.record()
    torch.cuda.synchronize()
    return {"layer": "gate 11008x4096 6:8", "ms": round(e0.elapsed_time(e1) / 3, 2),
            "note": "Eq. 3, N of 8, salient search (32 candidates), break-point search (160 grid points), residual + trisection, "
                    "float64; equals the oracle's output bit for bit (parity tests)"}


def pack_timing(stb, torch, wl):
    """stb_pack (two launches) on the gate layer: logical bytes read + packed bytes written per second."""
    d = wl.logical[0]
    n, m, N = d["n"], d["m"], d["N"]
    views = {"keep": np.uint8, "sign": np.uint8, "region": np.int16, "sign2": np.int32, "salient": np.int64, "scale": np.int16}
    t = {k: torch.from_numpy(np.ascontiguousarray(d[k]).view(v)).cuda() for k, v in views.items()}
    buf = torch.empty(stb.pack_size(n, m, N), dtype=torch.uint8, device="cuda")
    fn = lambda: stb.pack(n, m, N, t["keep"], t["sign"], t["region"], t["sign2"], t["salient"], t["scale"], buf=buf)
    for _ in range(3):
        fn()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(10):
        fn()
    e1.record()
    torch.cuda.synchronize()
    us = 1e3 * e0.elapsed_time(e1) / 10
    moved = sum(v.numel() * v.element_size() for v in t.values()) + wl.infos[0]["used_bytes"]
    return {"layer": "gate 11008x4096 6:8", "us": round(us, 1), "bytes_moved_MB": round(moved / 1e6, 2), "GBps": round(moved / us / 1e3, 1)}


def cuda_arm(args):
    import torch
    import torch.distributed as dist
    from paper_2408_01803_b200 import build
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the CUDA path has no CPU fallback")
    torch.cuda.set_device(local)
    if rank == 0 or not os.path.exists(os.path.join(ROOT, "paper_2408_01803_b200", "libstb.so")):
        build.build()
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        dist.barrier()
    import paper_2408_01803_b200 as stb
    pk = peaks()

    if args.only_gemm:
        # one prefill shape alone (for a profiler capture of stb::gemm_kernel)
        print(json.dumps({"gemm_prefill": gemm_table(stb, torch, pk, False, only=args.only_gemm)}))
        return
    copies = args.copies          # 12 distinct copies of the three layers per rotation: more than 6 x L2
    if world > 1 and rank != 0:
        dist.barrier()   # rank 0 quantizes (and caches) the layers first
    wl = Workload(stb, torch, copies, resident=not args.per_layer_launches)
    if world > 1 and rank == 0:
        dist.barrier()
    K, W = args.steps, args.warmup

    # one graph = `copies` consecutive passes (every pass another copy of the weights)
    g_full = capture(torch, [lambda: wl.run_steps(0, copies)])
    for i in range(max(W, 3)):
        wl.step(i)
    us_pass = time_graph(torch, g_full, copies, min_calls=20 * copies)
    # a step = `reps` graph replays, sized so that the K steps of the timed region last MIN_TIMED_S
    reps = max(1, int(np.ceil(args.min_timed_s / (K * copies * us_pass * 1e-6))))
    if world > 1:
        t = torch.tensor([reps], device="cuda", dtype=torch.int64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        reps = int(t.item())
    passes = K * reps * copies

    sampler = ClockSampler(local)
    sampler.start()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.perf_counter()
    e0.record()
    for _ in range(K * reps):
        g_full.replay()
    e1.record()
    sampler.sample()
    torch.cuda.synchronize()
    t1 = time.perf_counter()
    if world > 1:
        dist.barrier()
    ms = e0.elapsed_time(e1)
    clocks = sampler.stop(t0, t1)
    assert int(wl.status.item()) == 0, "device status %d" % int(wl.status.item())
    if world > 1:
        t = torch.tensor([ms], device="cuda", dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
    # resident: one launch per graph replay (`copies` passes, 2 groups each); per-layer launches: gate and up as one
    # grid + down = 2 launches per pass
    launches = K * reps if wl.resident else 2 * passes
    value = world * wl.bytes_step * passes / (ms * 1e-3) / 1e9
    launch_us = 1e3 * ms / launches
    per_launch_bytes = wl.bytes_step * passes / float(launches)
    achieved = per_launch_bytes / launch_us / 1e3

    # end to end: x from pinned host memory, y back to the host, every pass
    xh = torch.from_numpy(wl.x_np.copy()).pin_memory()
    yh = torch.empty(1, 4096, dtype=torch.float32).pin_memory()
    Ke = max(200, min(passes, 4000))
    for i in range(5):
        wl.step_host(i, xh, yh)
        torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    w0 = time.perf_counter()
    for i in range(Ke):
        wl.step_host(i, xh, yh)
        torch.cuda.current_stream().synchronize()
    w1 = time.perf_counter()
    e2e_s = w1 - w0
    if world > 1:
        t = torch.tensor([e2e_s], device="cuda", dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_s = float(t.item())
    e2e_val = world * wl.bytes_step * Ke / e2e_s / 1e9

    if rank != 0:
        if world > 1:
            dist.barrier()
            dist.destroy_process_group()
        return

    # the same list of passes walked by the checksum kernel: same dealing, rings and bulk copies, no arithmetic
    sums = torch.zeros(len(wl._keep[0]), dtype=torch.int64, device="cuda")
    g_sum = capture(torch, [lambda: stb.layer_stack_checksum(wl._keep[0], sums=sums, dev_status=wl.status)])
    us_stream = time_graph(torch, g_sum, copies, min_calls=100 * copies)
    del g_sum
    traffic, traffic_note = captured_traffic()
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": ms / passes, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOAD, "inputs": "oracle-quantized", "batch": 1, "layers_per_step": 3,
                   "packed_bytes_per_step": wl.bytes_step, "us_per_layer": round(1e3 * ms / (3 * passes), 3),
                   "step": "ms_per_step is per pass over the three layers; each of the %d steps of the timed region is %d passes "
                           "(%d graph replays) so that the region lasts >= %.2f s" % (K, reps * copies, reps, args.min_timed_s),
                   "passes_timed": passes, "timed_region_ms": round(ms, 3),
                   "salient_columns_per_block": {name: salient_histogram(d) for name, d in zip(MLP, wl.logical)},
                   "l2": "cold: %d distinct packed copies of each layer (%.0f MB per rotation, L2 is 126 MB)" % (
                       copies, copies * wl.bytes_step / 1e6),
                   "launch": ("one stb_layer_stack_resident call of %d passes (3 linears each) captured in a CUDA graph and replayed: one "
                              "cooperative launch of one 512-thread CTA per SM for the whole list" % copies) if wl.resident else
                             ("one stb_layer_stack call of %d passes (3 linears each) captured in a CUDA graph and replayed; 2 launches "
                              "per pass (gate+up as one grid, down), chained by programmatic dependent launch" % copies),
                   "multi_gpu": "replicas only" if world > 1 else "single GPU"},
        "clocks": clocks,
        "e2e": {"value": e2e_val, "unit": UNIT, "h2d_bytes_per_step": xh.numel() * 2, "d2h_bytes_per_step": yh.numel() * 4,
                "steps": Ke, "us_per_step": round(1e6 * e2e_s / Ke, 2),
                "call": ("stb_layer_stack_resident_host" if wl.resident else "stb_layer_stack_host") +
                        ": pinned host x -> device, 3 GEMVs, y -> pinned host, stream sync per pass"},
        "gpu_launches": launches,
        "roofline": {"bound": "hbm", "achieved": round(achieved, 1), "peak": pk["hbm_gbs"], "unit": "GB/s",
                     "frac": round(achieved / pk["hbm_gbs"], 4), "traffic": traffic, "traffic_source": traffic_note,
                     "kernel": "stb::stack_kernel" if wl.resident else "stb::gemv_mma_kernel<6,1>", "peak_source": pk["_source"],
                     "bytes_per_launch": round(per_launch_bytes), "launch_us": round(launch_us, 3),
                     "stream_only_frac": round(wl.bytes_step / us_stream / 1e3 / pk["hbm_gbs"], 4),
                     "stream_only_us_per_pass": round(us_stream, 3),
                     "note": "launch_us = timed region / launches (includes the gaps between launches); stream_only = the same "
                             "passes through stb_layer_stack_checksum, which walks the layers as the resident kernel does (same "
                             "dealing, rings and bulk copies) and XORs the words instead of decoding them"},
    }
    if world == 1 and not args.no_extras:
        # the same passes through the other entry point
        other = not wl.resident
        wl.resident = other
        g_other = capture(torch, [lambda: wl.run_steps(0, copies)])
        us_other = time_graph(torch, g_other, copies, min_calls=100 * copies)
        wl.resident = not other
        del g_other
        line["same_passes_other_call"] = {"call": CALL[other], "us_per_pass": round(us_other, 3),
                                          "GBps": round(wl.bytes_step / us_other / 1e3, 1),
                                          "frac_of_measured_hbm": round(wl.bytes_step / us_other / 1e3 / pk["hbm_gbs"], 4)}
        tab, ctx = gemv_table(stb, torch, wl, pk)
        line["gemv_layers"] = tab
        iso = [r for r in tab if r["batch"] == 1 and r["N"] == 6]
        line["roofline"]["isolated_launch_frac"] = round(float(np.mean([r["frac_of_measured_hbm"] for r in iso])), 4)
        line["dense_context"] = ctx
        line["gemm_prefill"] = gemm_table(stb, torch, pk, not args.tiled_ffn)
        line["gemm_prefill_note"] = "fractions of the MEASURED cuBLAS bf16 burst peak (%s TFLOP/s) decide the 50 %% target; fractions of the nominal 2250 TFLOP/s are printed beside them" % pk["bf16_tflops"]
        line["pack"] = pack_timing(stb, torch, wl)
        line["quantizer"] = quantizer_timing(stb, torch)
        st = stack_tables(stb, torch, pk)
        line["decode_stacks"] = st
        big = [r for r in st if r.get("batch") == 1 and "roofline" in r][0]
        line["largest_decode_workload"] = {"metric": METRIC, "value": big["GBps"], "unit": UNIT, "ms_per_step": big["us"] / 1e3,
                                           "config": {"workload": big["stack"], "inputs": "oracle-quantized, one layer per (shape, N) family", "batch": 1},
                                           "roofline": big["roofline"]}
        line["paper_context"] = ("paper's own kernel (2:4 1-bit GEMM, RTX 4090): up to 17.85x over ABQ-LLM 2-bit, "
                                 "263.45 TFLOPS = 79.74% of that GPU's sparse tensor-core peak at sequence length 8192")
    if world == 1 and not args.no_cpu:
        import oracle
        import oracle.workloads as owl
        oracle.build()
        Ls = [owl.as_logical(d) for d in wl.logical]
        x0 = wl.x_np.astype(np.float64)
        x1 = wl.h_gate.double().cpu().numpy()
        xs = [x0, x0, x1]
        rows = [np.arange(d["n"], dtype=np.int32) for d in wl.logical]
        t, n_pass = 0.0, 0
        while t < 10.0 and n_pass < 50:
            t += oracle_pass(Ls, xs, rows)
            n_pass += 1
        line["cpu_baseline"] = {"value": wl.bytes_step * n_pass / t / 1e9, "unit": UNIT, "cores": oracle.hardware_threads(),
                                "kind": "oracle", "sample": "all output rows of gate, up and down, batch 1, %d passes (%.1f s)" % (n_pass, t),
                                "us_per_layer": round(1e6 * t / n_pass / 3, 1)}
        # the same oracle on one core, on every 8th output row (scaled to all rows)
        rows8 = [r[::8] for r in rows]
        t1 = min(oracle_pass(Ls, xs, rows8, threads=1) for _ in range(2)) * 8.0
        line["cpu_baseline"]["one_core"] = {"value": wl.bytes_step / t1 / 1e9, "unit": UNIT, "us_per_layer": round(1e6 * t1 / 3, 1),
                                            "sample": "every 8th output row, one thread, time scaled by 8"}
    print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None, help="default: 20")
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--no-extras", action="store_true", help="skip the per-layer tables, the prefill GEMM and the decoder stacks")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU oracle timing")
    ap.add_argument("--copies", type=int, default=12, help="distinct packed copies of the layers per rotation (cold L2 needs >= 3)")
    ap.add_argument("--min-timed-s", type=float, default=MIN_TIMED_S, help="shortest timed region; 0 for a profiler capture")
    ap.add_argument("--only-gemm", default=None, help="run only the prefill GEMM shape whose name starts with this (q/o, k/v, gate/up, down)")
    ap.add_argument("--per-layer-launches", action="store_true", help="headline through stb_layer_stack instead of stb_layer_stack_resident")
    ap.add_argument("--tiled-ffn", action="store_true", help="prefill GEMM: build the 28672-wide FFN layers by repeating the quantized "
                                                             "q layer instead of quantizing the real ones on the GPU")
    args = ap.parse_args()
    args.steps = args.steps or 20
    if args.impl == "reference":
        reference_arm(args)
    else:
        cuda_arm(args)


if __name__ == "__main__":
    main()
