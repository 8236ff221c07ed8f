#!/usr/bin/env python
"""Benchmark of the W4A4 linear hot path (rotate -> INT4 quantise -> INT4 GEMM -> dequant).

One step = one pass of the whole path (sq_linear) over one batch of synthetic activations of
the named workload.  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]
                  [--structured-r2] [--fuse-decode] [--no-sweep] [--no-cpu-baseline] [--quick]
                  [--variants-only [--grouped-tokens T]]

After the headline workload the default run also times every other benchmark workload briefly and
reports them under "per_workload" of the same line, and the weight-only variant (W4A16 / W3A16) and the
grouped mixture-of-experts layer under "variants" (all skipped with --no-sweep or N > 1).

N > 1: launched under torchrun, one process per GPU; the path shards over tokens with no
collective (each rank owns its own batch and a replica of the packed weights), so scaling is
"weak" and the only communication is the barrier / max-over-ranks of the timing.
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

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2511_22316_b200 import workloads as wl  # noqa: E402

METRIC = "w4a4_linear_tops"
UNIT = "TOPS"
DEFAULT_WORKLOAD = wl.L7B_QKVO.name
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
INT8_OVER_BF16 = 2.0      # nominal dense ratio (4.5 POPS int8 : 2.25 PFLOP/s bf16)

# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu captures summarised under
# profiles/ (bytes; None until a capture exists for that kernel and workload).
NCU_TRAFFIC = {
    ("gemm", "llama2_7b_qkvo_prefill"): 12632576,           # w4a4_gemm_pair_kernel: reads (Y stays in L2)
    ("rotate_quant", "llama2_7b_qkvo_prefill"): 16888320,   # rotate_quant_tc_kernel
    ("rotate_quant_st", "llama2_7b_qkvo_prefill"): 16873472,  # rotate_quant_st_kernel (--structured-r2)
    ("gemm", "llama3_8b_up_decode_m16"): 29457408,          # w4a4_gemm_decode_kernel, K not split
    ("gemm", "llama3_8b_down_decode_m16"): 29518592,        # w4a4_gemm_decode_kernel, K over clusters of 4
    ("gemm", "llama3_8b_up_decode_m1"): 29408768,           # w4a4_gemv_kernel
    ("rotate_quant", "llama2_7b_down_prefill"): 45464320,   # rotate_quant_pair_kernel
    ("rotate_quant", "llama2_70b_gateup_prefill"): 69889536,   # rotate_quant_tc_kernel, n2 = 128
    ("rotate_quant", "llama2_70b_down_prefill"): 275649024,    # rotate_quant_pair_kernel, n2 = 128
    ("wo_gemm", "llama3_8b_up_decode_m16"): 29558016,       # wo_gemm_tmem_kernel<16, 4, 8> (W4A16)
    ("wo_gemm", "llama2_7b_qkvo_prefill"): 25311744,        # wo_gemm_pair_kernel (W4A16; Y stayed in L2)
}


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "source": "measured"}
    except Exception:
        d = dict(FALLBACK_PEAKS)
        d["source"] = "fallback"
        return d


def ops_per_step(w):
    return 2.0 * w.M * w.N * w.K


def rotate_quant_bytes(w):
    """Algorithmic HBM bytes of steps 1+2 per launch: read fp16 row, write packed row + step."""
    return w.M * (2.0 * w.n + w.n / 2.0 + 2.0)


def gemm_bytes(w):
    return (w.M + w.N) * w.K / 2.0 + 2.0 * w.M * w.N + 2.0 * (w.M + w.N)


def gemm_kernel_name(w):
    """The kernel sq_w4a4_gemm picks for this shape (mirrors the library's dispatch)."""
    fast = w.K % 128 == 0 and w.N % 8 == 0
    decode = fast and w.M <= 64 and w.N >= 128 and w.K >= 256
    if w.M <= 4 and w.K % 32 == 0 and w.K <= 32768 and (w.M <= 2 or not decode):
        return "w4a4_gemv_kernel"
    if decode:
        return "w4a4_gemm_decode_kernel"
    if fast and w.M > 128 and w.N >= 128:
        return "w4a4_gemm_pair_kernel"
    return "w4a4_gemm_tc_kernel" if fast else "w4a4_gemm_simple_kernel"


def rotate_kernel_name(w, structured=False):
    if structured:
        return "rotate_quant_st_kernel"
    if w.n2 in (64, 128) and w.n1 <= 128:
        return "rotate_quant_tc_kernel"
    if w.n2 in (64, 128) and w.n1 <= 256:
        return "rotate_quant_pair_kernel"
    return "rotate_quant_kernel"


# ----------------------------------------------------------------------------------------------
# clock sampling during the timed region
# ----------------------------------------------------------------------------------------------
class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_id: str):
        self.gpu = gpu_id          # a UUID ("GPU-...") when it could be resolved, else an nvidia-smi index
        self.proc = None
        self.lines = []
        self.thread = None

    @staticmethod
    def resolve(torch, device_index: int) -> str:
        """The nvidia-smi id of the torch device: its UUID (CUDA_VISIBLE_DEVICES may renumber the
        devices, so the torch index is not nvidia-smi's)."""
        try:
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            return uuid if uuid.startswith("GPU-") else "GPU-" + uuid
        except Exception:
            return str(device_index)

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.perf_counter(), line.strip()))

    def stop(self):
        if self.proc is None:
            return
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()

    def window(self, t_begin=None, t_end=None):
        """Median SM clock and throttle reasons over the samples that arrived inside [t_begin, t_end]
        (a timed region); if fewer than three did, over every sample so far, and says so."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        inside = [ln for (t, ln) in self.lines if t_begin is not None and t_begin <= t <= t_end]
        scope = "timed region" if len(inside) >= 3 else "whole run (timed region shorter than three samples)"
        for ln in (inside if len(inside) >= 3 else [ln for (_, ln) in self.lines]):
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                smax.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(smax) if smax else None,
                "samples": len(sm), "scope": scope, "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------------------------
# CPU oracle arm (also `--impl reference`)
# ----------------------------------------------------------------------------------------------
class OracleArm:
    """The oracle, as it stands, on the first `rows` token rows of the workload against the full
    weight matrix.  The weights are rotated+quantised once, untimed: that is offline setup on the
    GPU side too.  One pass = rotate, quantise, pack, integer GEMM, dequantise."""

    def __init__(self, w, rows: int, X=None, W=None):
        from oracle import singlequant_oracle as ora
        self.ora = ora
        self.w = w
        X = wl.make_activations(w) if X is None else X
        W = wl.make_weights(w) if W is None else W
        self.R1, self.R2 = ora.build_rotation(X.astype(np.float32), w.n1, w.n2)
        Wq, self.sw, _ = ora.pack_weight(W, self.R1, self.R2)
        self.Wc = ora.unpack_int4(Wq)
        self.rows = min(rows, w.M)
        self.Xs = X[:self.rows]
        self.sample = (f"first {self.rows} of {w.M} token rows per pass against the full "
                       f"{w.N}x{w.K} weight matrix")

    def one_pass(self):
        ora = self.ora
        Xq, sx, _ = ora.rotate_quant(self.Xs, self.R1, self.R2)
        acc = ora.gemm_i32(ora.unpack_int4(Xq), self.Wc)
        return ora.dequant(acc, sx, self.sw)

    def timed_pass(self) -> float:
        t0 = time.perf_counter()
        self.one_pass()
        return time.perf_counter() - t0

    def tops(self, seconds: float) -> float:
        return 2.0 * self.rows * self.w.N * self.w.K / seconds / 1e12

    @staticmethod
    def threads() -> int:
        try:
            from threadpoolctl import threadpool_info
            return max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
        except Exception:
            return len(os.sched_getaffinity(0))


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    arm = OracleArm(w, rows=256)
    for _ in range(args.warmup):
        arm.one_pass()
    times = [arm.timed_pass() for _ in range(args.steps)]
    dt = statistics.mean(times)
    value = arm.tops(dt)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": w.name, "M": w.M, "N": w.N, "K": w.K, "sample": arm.sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": arm.threads(), "kind": "oracle",
                         "sample": arm.sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


# ----------------------------------------------------------------------------------------------
# CUDA arm
# ----------------------------------------------------------------------------------------------
class Layer:
    """One workload resident on the device: rotation handle, packed weights, and a ring of buffer sets
    larger than L2 so that no step finds its inputs cached."""

    def __init__(self, sq, torch, w, device_index, rank=0, structured_r2=False, fuse_decode=False, keep_host=False):
        import dataclasses
        self.sq, self.torch, self.w = sq, torch, w
        M, N, K = w.M, w.N, w.K
        w_rank = dataclasses.replace(w, seed=w.seed + 7919 * rank) if rank else w
        X = wl.make_activations(w_rank)
        W = wl.make_weights(w)
        flags = (sq.SQ_ROT_DEFAULT | (sq.SQ_ROT_APPLY_STRUCTURED if structured_r2 else 0) |
                 (sq.SQ_ROT_FUSE_DECODE if fuse_decode else 0))
        self.rot = sq.sq_build_rotation(X.astype(np.float32), w.n1, w.n2, flags=flags, seed=0)
        dW = torch.from_numpy(W).cuda()
        Wq = torch.empty((N, K // 2), dtype=torch.uint8, device="cuda")
        sw = torch.empty((N,), dtype=torch.float16, device="cuda")
        sq.sq_pack_weight(self.rot, dW, N, K, Wq, sw)
        torch.cuda.synchronize()
        del dW
        self.l2 = torch.cuda.get_device_properties(device_index).L2_cache_size
        self.per_set = M * K * 2 + M * K // 2 + M * N * 2 + N * K // 2
        self.nsets = max(2, int(np.ceil(1.5 * self.l2 / self.per_set)) + 1)
        self.ws_bytes = sq.sq_linear_workspace_bytes(M, K)
        self.Xh = torch.from_numpy(X).pin_memory()
        self.sets = []
        for _ in range(self.nsets):
            ws = torch.empty(self.ws_bytes + 256, dtype=torch.uint8, device="cuda")
            off = (-ws.data_ptr()) % 256
            st = {"X": self.Xh.cuda(non_blocking=False).clone(), "Wq": Wq.clone(), "sw": sw.clone(),
                  "Y": torch.empty((M, N), dtype=torch.float16, device="cuda"), "ws": ws, "ws_ptr": ws.data_ptr() + off,
                  "Xq": torch.empty((M, K // 2), dtype=torch.uint8, device="cuda"),
                  "sx": torch.empty((M,), dtype=torch.float16, device="cuda")}
            # device pointers resolved once: the timed loop passes plain integers through the C ABI
            st["ptrs"] = (st["X"].data_ptr(), st["Wq"].data_ptr(), st["sw"].data_ptr(), st["ws_ptr"], st["Y"].data_ptr())
            self.sets.append(st)
        self.X, self.W = (X, W) if keep_host else (None, None)

    def step(self, i):
        w = self.w
        x_, wq_, sw_, ws_, y_ = self.sets[i % self.nsets]["ptrs"]
        self.sq.sq_linear(self.rot, x_, w.M, wq_, sw_, w.N, w.K, ws_, self.ws_bytes, y_)

    def rotate_quant(self, i):
        s, w = self.sets[i % self.nsets], self.w
        self.sq.sq_rotate_quant_act(self.rot, s["X"], w.M, s["Xq"], s["sx"])

    def gemm(self, i):
        s, w = self.sets[i % self.nsets], self.w
        self.sq.sq_w4a4_gemm(s["Xq"], s["sx"], s["Wq"], s["sw"], w.M, w.N, w.K, s["Y"], None)

    def timed_steps(self, steps):
        """CUDA events on the launching stream around `steps` calls of sq_linear, launched one by one."""
        torch = self.torch
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(steps):
            self.step(i)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1)

    def graph_time(self, fn, count):
        """Milliseconds per call of `fn` replayed from a CUDA graph of `count` back-to-back calls (launch
        overhead taken out); None when capture is not possible."""
        torch = self.torch
        try:
            gstream = torch.cuda.Stream()
            gstream.wait_stream(torch.cuda.current_stream())
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.stream(gstream):
                with torch.cuda.graph(graph, stream=gstream):
                    for i in range(count):
                        fn(i)
                graph.replay()
                gstream.synchronize()
                g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                g0.record(gstream)
                for _ in range(5):
                    graph.replay()
                g1.record(gstream)
                gstream.synchronize()
                ms = g0.elapsed_time(g1) / (5 * count)
            torch.cuda.current_stream().wait_stream(gstream)
            torch.cuda.synchronize()
            return ms
        except Exception as exc:       # capture is optional: the event timings stand on their own
            sys.stderr.write(f"graph replay skipped: {exc}\n")
            torch.cuda.synchronize()
            return None

    def kernel_times(self, count):
        """(rotate+quant ms, GEMM ms, whole step from a graph ms, how): per-entry-point times from graph
        replays of back-to-back launches on the ring, else from events around single launches."""
        torch = self.torch
        graph_ms = self.graph_time(self.step, count)
        rq = self.graph_time(self.rotate_quant, count)
        ge = self.graph_time(self.gemm, count)
        how = "cuda events around graph replays of back-to-back launches"
        if rq is None or ge is None:
            ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(count)]
            for i in range(count):
                ev[i][0].record()
                self.rotate_quant(i)
                ev[i][1].record()
                self.gemm(i)
                ev[i][2].record()
            torch.cuda.synchronize()
            rq = statistics.mean(e[0].elapsed_time(e[1]) for e in ev)
            ge = statistics.mean(e[1].elapsed_time(e[2]) for e in ev)
            how = "cuda events around single launches"
        return rq, ge, graph_ms, how

    def close(self):
        self.rot.close()
        self.sets = []
        self.torch.cuda.empty_cache()


def int8_yardstick(torch, w, l2_bytes):
    """A library int8 GEMM (torch._int_mm: int8 x int8 -> int32) of the workload's shape, timed in the same
    run on buffers rotated through more than L2: what "the dense INT8 tensor peak" amounts to on this machine
    at this size.  None where the library does not take the shape."""
    try:
        M, N, K = w.M, w.N, w.K
        if M <= 16 or K % 8 or N % 8:
            return None
        per = M * K + K * N + 4 * M * N
        nsets = max(2, int(np.ceil(1.5 * l2_bytes / per)) + 1)
        A = [torch.randint(-8, 8, (M, K), dtype=torch.int8, device="cuda") for _ in range(nsets)]
        B = [torch.randint(-8, 8, (K, N), dtype=torch.int8, device="cuda") for _ in range(nsets)]
        for i in range(3):
            torch._int_mm(A[i % nsets], B[i % nsets])
        torch.cuda.synchronize()
        iters = 20
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(iters):
            torch._int_mm(A[i % nsets], B[i % nsets])
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / iters
        return {"name": "torch._int_mm (int8 x int8 -> int32, library GEMM)", "ms": ms,
                "tops": 2.0 * M * N * K / (ms * 1e-3) / 1e12}
    except Exception as exc:
        sys.stderr.write(f"int8 yardstick skipped: {exc}\n")
        return None


def link_yardstick(torch, in_bytes, out_bytes, iters=10):
    """Milliseconds for one pinned host->device copy of `in_bytes` and one device->host copy of `out_bytes`
    running concurrently on two streams, no computation: the floor of an end-to-end step on this link."""
    try:
        hin = torch.empty(in_bytes, dtype=torch.uint8).pin_memory()
        hout = torch.empty(out_bytes, dtype=torch.uint8).pin_memory()
        din = torch.empty(in_bytes, dtype=torch.uint8, device="cuda")
        dout = torch.empty(out_bytes, dtype=torch.uint8, device="cuda")
        s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
        torch.cuda.synchronize()
        best = None
        for rep in range(2):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            s1.wait_event(e0)
            s2.wait_event(e0)
            for _ in range(iters):
                with torch.cuda.stream(s1):
                    din.copy_(hin, non_blocking=True)
                with torch.cuda.stream(s2):
                    hout.copy_(dout, non_blocking=True)
            torch.cuda.current_stream().wait_stream(s1)
            torch.cuda.current_stream().wait_stream(s2)
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / iters
            best = ms if best is None else min(best, ms)
        return best
    except Exception as exc:
        sys.stderr.write(f"link yardstick skipped: {exc}\n")
        return None


def rooflines(w, rq_ms, gemm_ms, pk, structured, yard=None):
    """The two kernels' roofline entries: (GEMM, rotate+quant)."""
    gemm_tops = ops_per_step(w) / (gemm_ms * 1e-3) / 1e12
    rq_gbs = rotate_quant_bytes(w) / (rq_ms * 1e-3) / 1e9
    int8_peak = pk["bf16_tflops"] * INT8_OVER_BF16
    if w.M <= 64:       # decode: bound by reading the packed weights once
        gemm_gbs = gemm_bytes(w) / (gemm_ms * 1e-3) / 1e9
        roof_gemm = {"kernel": gemm_kernel_name(w), "bound": "hbm", "achieved": gemm_gbs, "peak": pk["hbm_gbs"],
                     "unit": "GB/s", "frac": gemm_gbs / pk["hbm_gbs"],
                     "traffic": NCU_TRAFFIC.get(("gemm", w.name)),
                     "peak_source": f"{pk['source']} copy bandwidth", "ms_per_launch": gemm_ms,
                     "algorithmic_bytes": gemm_bytes(w), "frac_of_spec_8000": gemm_gbs / 8000.0}
    else:
        roof_gemm = {"kernel": gemm_kernel_name(w), "bound": "tensor", "achieved": gemm_tops, "peak": int8_peak,
                     "unit": "TOP/s", "frac": gemm_tops / int8_peak,
                     "traffic": NCU_TRAFFIC.get(("gemm", w.name)),
                     "peak_source": f"{pk['source']} bf16 burst x{INT8_OVER_BF16:g} (nominal int8:bf16 ratio)",
                     "ms_per_launch": gemm_ms, "algorithmic_ops": ops_per_step(w),
                     "frac_of_spec_4500": gemm_tops / 4500.0}
        if yard is not None:
            roof_gemm["yardstick"] = dict(yard, frac=gemm_tops / yard["tops"])
    roof_rq = {"kernel": rotate_kernel_name(w, structured), "bound": "hbm", "achieved": rq_gbs, "peak": pk["hbm_gbs"],
               "unit": "GB/s", "frac": rq_gbs / pk["hbm_gbs"],
               "traffic": NCU_TRAFFIC.get(("rotate_quant_st" if structured else "rotate_quant", w.name)),
               "peak_source": f"{pk['source']} copy bandwidth", "ms_per_launch": rq_ms,
               "algorithmic_bytes": rotate_quant_bytes(w), "frac_of_spec_8000": rq_gbs / 8000.0}
    return roof_gemm, roof_rq


def _graph_ms(torch, fn, count):
    """Milliseconds per call of `fn(i)` replayed from a CUDA graph of `count` back-to-back calls."""
    gstream = torch.cuda.Stream()
    gstream.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(gstream):
        with torch.cuda.graph(graph, stream=gstream):
            for i in range(count):
                fn(i)
        graph.replay()
        gstream.synchronize()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record(gstream)
        for _ in range(5):
            graph.replay()
        g1.record(gstream)
        gstream.synchronize()
        ms = g0.elapsed_time(g1) / (5 * count)
    torch.cuda.current_stream().wait_stream(gstream)
    torch.cuda.synchronize()
    return ms


def _events_ms(torch, fn, count):
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(count):
        fn(i)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / count


def weight_only_entry(sq, torch, w, bits, pk, l2, quick=False):
    """The weight-only layer (fp16 rotated activations x b-bit weights) on one workload: the step through
    sq_linear_wo, its two kernels from graph replays, roofline fractions, and a library fp16 GEMM of the
    same shape (torch.matmul, no unpacking, no scaling) as the yardstick."""
    M, N, K = w.M, w.N, w.K
    X = wl.make_activations(w)
    W = wl.make_weights(w)
    rot = sq.sq_build_rotation(X.astype(np.float32), w.n1, w.n2, seed=0)
    dW = torch.from_numpy(W).cuda()
    Wq = torch.empty((N, K // 2), dtype=torch.uint8, device="cuda")
    sw = torch.empty((N,), dtype=torch.float16, device="cuda")
    sq.sq_pack_weight_wo(rot, dW, N, K, bits, Wq, sw)
    torch.cuda.synchronize()
    per_set = M * K * 2 * 2 + M * N * 2 + N * K // 2
    nsets = max(2, int(np.ceil(1.5 * l2 / per_set)) + 1)
    ws_bytes = sq.sq_linear_wo_workspace_bytes(M, K)
    dX = torch.from_numpy(X).cuda()
    sets = []
    for _ in range(nsets):
        ws = torch.empty(ws_bytes + 256, dtype=torch.uint8, device="cuda")
        sets.append({"X": dX.clone(), "Wq": Wq.clone(), "sw": sw.clone(), "ws": ws,
                     "ws_ptr": ws.data_ptr() + (-ws.data_ptr()) % 256,
                     "Y": torch.empty((M, N), dtype=torch.float16, device="cuda")})

    def step(i):
        t = sets[i % nsets]
        sq.sq_linear_wo(rot, t["X"], M, t["Wq"], t["sw"], N, K, t["ws_ptr"], ws_bytes, t["Y"])

    def rotate(i):
        t = sets[i % nsets]
        sq.sq_rotate_act_f16(rot, t["X"], M, t["ws_ptr"])

    def gemm(i):
        t = sets[i % nsets]
        sq.sq_w4a16_gemm(t["ws_ptr"], t["Wq"], t["sw"], M, N, K, t["Y"])

    for i in range(5):
        step(i)
    torch.cuda.synchronize()
    count = 4 if quick else min(100, 4 * nsets)
    step_ms = _events_ms(torch, step, 4 if quick else (100 if M <= 2048 else 30))
    rot_ms, gemm_ms = _graph_ms(torch, rotate, count), _graph_ms(torch, gemm, count)
    flops = 2.0 * M * N * K
    gemm_bytes_wo = N * K / 2.0 + 2.0 * M * K + 2.0 * M * N + 2.0 * N
    rot_bytes = 4.0 * M * K
    if M <= 64:
        gbs = gemm_bytes_wo / (gemm_ms * 1e-3) / 1e9
        roof = {"kernel": "wo_gemv_kernel" if M <= 2 else "wo_gemm_tmem_kernel", "bound": "hbm", "achieved": gbs, "peak": pk["hbm_gbs"], "unit": "GB/s",
                "frac": gbs / pk["hbm_gbs"], "traffic": NCU_TRAFFIC.get(("wo_gemm", w.name)) if bits == 4 else None,
                "ms_per_launch": gemm_ms,
                "algorithmic_bytes": gemm_bytes_wo}
    else:
        tf = flops / (gemm_ms * 1e-3) / 1e12
        tc_ok = N >= 128 and K % 64 == 0 and N % 8 == 0
        roof = {"kernel": ("wo_gemm_pair_kernel" if (M > 128 and N >= 256) else "wo_gemm_tmem_kernel") if tc_ok else "wo_gemm_tc_kernel",
                "bound": "tensor", "achieved": tf, "peak": pk["bf16_tflops"],
                "unit": "TFLOP/s", "frac": tf / pk["bf16_tflops"],
                "traffic": NCU_TRAFFIC.get(("wo_gemm", w.name)) if bits == 4 else None, "ms_per_launch": gemm_ms,
                "peak_source": f"{pk['source']} bf16 burst (fp16 runs at the same rate)", "algorithmic_flops": flops}
        try:
            if quick:
                raise RuntimeError("quick run")
            A = [torch.randn((M, K), dtype=torch.float16, device="cuda") for _ in range(nsets)]
            B = [torch.randn((N, K), dtype=torch.float16, device="cuda") for _ in range(min(nsets, 4))]
            lib_ms = _events_ms(torch, lambda i: torch.matmul(A[i % nsets], B[i % len(B)].t()), 20)
            lib_ms = _events_ms(torch, lambda i: torch.matmul(A[i % nsets], B[i % len(B)].t()), 20)
            roof["yardstick"] = {"name": "torch.matmul fp16 x fp16 (library GEMM, dense fp16 weights)", "ms": lib_ms,
                                 "tflops": flops / (lib_ms * 1e-3) / 1e12, "frac": lib_ms / gemm_ms}
            del A, B
        except Exception as exc:
            sys.stderr.write(f"fp16 yardstick skipped: {exc}\n")
    rgbs = rot_bytes / (rot_ms * 1e-3) / 1e9
    out = {"M": M, "N": N, "K": K, "bits": bits, "ms_per_step": step_ms, "value": flops / (step_ms * 1e-3) / 1e12,
           "unit": "TFLOP/s (2MNK per step)", "gemm": roof,
           "rotate": {"kernel": rotate_kernel_name(w) + " (rotation only, fp16 out)", "bound": "hbm", "achieved": rgbs,
                      "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": rgbs / pk["hbm_gbs"], "traffic": None,
                      "ms_per_launch": rot_ms, "algorithmic_bytes": rot_bytes},
           "device_status": sq.sq_last_device_status()}
    rot.close()
    del sets
    torch.cuda.empty_cache()
    return out


def grouped_entry(sq, torch, l2, T=2048):
    """A mixture-of-experts up-projection through sq_linear_grouped: 8 experts of 4096 -> 14336 (the shape of
    Mixtral 8x7B's expert layers), T tokens routed to two experts each by a seeded uniform draw, sorted
    by expert; one rotation handle shared by the experts (they see the same input), weights per expert."""
    E, K, N, n1, n2 = 8, 4096, 14336, 64, 64
    rng = np.random.default_rng(2024)
    choice = np.stack([rng.permutation(E)[:2] for _ in range(T)])          # two distinct experts per token
    counts = np.bincount(choice.reshape(-1), minlength=E)
    offsets = np.concatenate([[0], np.cumsum(counts)]).astype(np.int64)
    M = int(offsets[-1])
    base = wl.small("moe_up", max(T, 64), n1, n2, N, seed=88)
    Xcal = wl.make_activations(base)                                          # calibration batch: at least 64 tokens
    Xtok = Xcal[:T]
    order = np.argsort(choice.reshape(-1), kind="stable")
    X = Xtok[order // 2]                                                      # token rows, expert-sorted
    rot = sq.sq_build_rotation(Xcal.astype(np.float32), n1, n2, seed=0)
    wqs, sws = [], []
    for e in range(E):
        We = torch.from_numpy((0.02 * np.random.default_rng(100 + e).standard_normal((N, K))).astype(np.float16)).cuda()
        q = torch.empty((N, K // 2), dtype=torch.uint8, device="cuda")
        s_ = torch.empty((N,), dtype=torch.float16, device="cuda")
        sq.sq_pack_weight(rot, We, N, K, q, s_)
        wqs.append(q); sws.append(s_)
        del We
    torch.cuda.synchronize()
    dX = torch.from_numpy(X).cuda()
    Y = torch.empty((M, N), dtype=torch.float16, device="cuda")
    ws_bytes = sq.sq_linear_workspace_bytes(M, K)
    ws = torch.empty(ws_bytes + 256, dtype=torch.uint8, device="cuda")
    wsp = ws.data_ptr() + (-ws.data_ptr()) % 256
    rots = [rot] * E

    def step(i):
        sq.sq_linear_grouped(rots, offsets, dX, wqs, sws, N, K, wsp, ws_bytes, Y)

    for i in range(3):
        step(i)
    torch.cuda.synchronize()
    before = sq.sq_kernel_launch_count()
    ms = _events_ms(torch, step, 20)
    launches = (sq.sq_kernel_launch_count() - before) // 20
    ops = 2.0 * M * N * K
    wbytes = float(sum(1 for c in counts if c > 0)) * N * K / 2
    out = {"weight_gbs": wbytes / (ms * 1e-3) / 1e9, "experts": E, "tokens": T, "top_k": 2, "rows": M, "rows_per_expert": counts.tolist(), "N": N, "K": K,
           "ms_per_step": ms, "value": ops / (ms * 1e-3) / 1e12, "unit": UNIT, "kernels_per_step": int(launches),
           "note": "weights of the eight experts (235 MB packed) exceed L2, activations are re-read from L2",
           "device_status": sq.sq_last_device_status()}
    rot.close()
    torch.cuda.empty_cache()
    return out


def run_variants_only(args, w):
    import torch
    from paper_2511_22316_b200 import binding as sq
    from paper_2511_22316_b200 import build as sqbuild
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(0)
    sqbuild.build()
    sq.load()
    l2 = torch.cuda.get_device_properties(0).L2_cache_size
    if args.grouped_tokens:
        entry = grouped_entry(sq, torch, l2, T=args.grouped_tokens)
        print(json.dumps({"variants": {"grouped": entry}, "n_gpus": 1, "data": "synthetic"}))
        return 0
    entry = weight_only_entry(sq, torch, w, 4, peaks(), l2, quick=args.quick)
    print(json.dumps({"variants": {"weight_only": {f"{w.name}_w4a16": entry}}, "n_gpus": 1, "data": "synthetic"}))
    return 0


def run_ours(args, w):
    import torch
    from paper_2511_22316_b200 import binding as sq
    from paper_2511_22316_b200 import build as sqbuild

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    if rank == 0 or world == 1:
        sqbuild.build()
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist.barrier()
    sq.load()

    M, N, K = w.M, w.N, w.K
    # every rank draws its own batch (weak scaling over tokens); the weights are replicated
    layer = Layer(sq, torch, w, local_rank, rank=rank, structured_r2=args.structured_r2,
                  fuse_decode=args.fuse_decode, keep_host=True)
    nsets, per_set, l2 = layer.nsets, layer.per_set, layer.l2
    structured = layer.rot.structured

    def sync_all():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    # the clock sampler is up before the warm-up, so that nothing but the barrier and the synchronize
    # stands between the last warm-up step and the timed region (an idle GPU drops its clocks)
    sampler = ClockSampler(ClockSampler.resolve(torch, local_rank))
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    sync_all()

    warm = max(args.warmup, 3)
    for i in range(warm):
        layer.step(i)
    sync_all()

    # ---- timed region: exactly K steps of sq_linear ------------------------------------------
    launches0 = sq.sq_kernel_launch_count()
    sync_all()
    t_region0 = time.perf_counter()
    ms_total = layer.timed_steps(args.steps)
    sync_all()
    t_region1 = time.perf_counter()
    launches = sq.sq_kernel_launch_count() - launches0
    clocks = sampler.window(t_region0, t_region1) if rank == 0 else None

    # ---- the same step for at least half a second, so that several clock samples fall inside it:
    # the step time and the clocks it ran at (time x median SM MHz lets a reader normalise) -----------
    sustained = None
    if rank == 0 and world == 1 and not args.quick:
        n_sus = max(args.steps, int(np.ceil(600.0 / max(ms_total / args.steps, 1e-3))))
        n_sus = min(n_sus, 400000)
        t0 = time.perf_counter()
        ms_sus = layer.timed_steps(n_sus)
        t1 = time.perf_counter()
        sustained = {"steps": n_sus, "ms_per_step": ms_sus / n_sus,
                     "value": ops_per_step(w) / (ms_sus / n_sus * 1e-3) / 1e12, "unit": UNIT,
                     "clocks": sampler.window(t0, t1)}
        if sustained["clocks"].get("sm_mhz"):
            sustained["us_x_mhz"] = ms_sus / n_sus * 1e3 * sustained["clocks"]["sm_mhz"]

    # ---- attribution: the two entry points and the whole step replayed from CUDA graphs -------
    gsteps = min(max(args.steps, 8), 4 * nsets)
    rq_ms, gemm_ms, graph_ms, kernel_timing = layer.kernel_times(gsteps)

    # ---- end to end: host activations in, host outputs out, through sq_linear_host ------------
    hws_bytes = sq.sq_linear_host_workspace_bytes(M, N, K)
    hws = torch.empty(hws_bytes + 256, dtype=torch.uint8, device="cuda")
    hoff = (-hws.data_ptr()) % 256
    Yh = torch.empty((M, N), dtype=torch.float16).pin_memory()
    e2e_steps = max(3, min(args.steps, 20))
    sets = layer.sets
    for _ in range(2):
        sq.sq_linear_host(layer.rot, layer.Xh, M, sets[0]["Wq"], sets[0]["sw"], N, K, hws.data_ptr() + hoff, hws_bytes, Yh)
    sync_all()
    h0, h1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    h0.record()
    for i in range(e2e_steps):
        s = sets[i % nsets]
        sq.sq_linear_host(layer.rot, layer.Xh, M, s["Wq"], s["sw"], N, K, hws.data_ptr() + hoff, hws_bytes, Yh)
    h1.record()
    sync_all()
    e2e_ms = h0.elapsed_time(h1) / e2e_steps
    status = sq.sq_last_device_status()
    link_ms = link_yardstick(torch, M * K * 2, M * N * 2) if (rank == 0 and world == 1 and not args.quick) else None
    del hws

    # ---- max over ranks ---------------------------------------------------------------------
    t = torch.tensor([ms_total, e2e_ms, rq_ms, gemm_ms, graph_ms if graph_ms is not None else -1.0],
                     dtype=torch.float64, device="cuda")
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    ms_total, e2e_ms, rq_ms, gemm_ms, graph_ms = (float(x) for x in t.tolist())
    graph_ms = graph_ms if graph_ms > 0 else None
    ms_per_step = ms_total / args.steps

    if rank == 0:
        pk = peaks()
        value = world * ops_per_step(w) / (ms_per_step * 1e-3) / 1e12
        e2e_value = world * ops_per_step(w) / (e2e_ms * 1e-3) / 1e12
        yard = int8_yardstick(torch, w, l2) if (world == 1 and not args.quick) else None
        roof_gemm, roof_rq = rooflines(w, rq_ms, gemm_ms, pk, structured, yard)
        dominant, other = (roof_gemm, roof_rq) if gemm_ms >= rq_ms else (roof_rq, roof_gemm)

        cpu = None
        if world == 1 and not args.no_cpu_baseline:
            arm = OracleArm(w, rows=256, X=layer.X, W=layer.W)
            arm.one_pass()
            times, t_start = [], time.perf_counter()
            while time.perf_counter() - t_start < 10.0 or not times:
                times.append(arm.timed_pass())
            cpu = {"value": arm.tops(statistics.mean(times)), "unit": UNIT, "cores": arm.threads(),
                   "kind": "oracle", "sample": f"{arm.sample}; {len(times)} passes, "
                                               f"{statistics.mean(times):.3f} s per pass"}
            del arm
        layer.X = layer.W = None

        # ---- every other benchmark workload, briefly: step (launched and from a graph), the two
        # kernels, both roofline fractions and the clocks sampled while it ran ------------------
        per_workload = None
        if world == 1 and not args.no_sweep:
            per_workload = {w.name: {"M": M, "N": N, "K": K, "n1": w.n1, "n2": w.n2, "steps": args.steps,
                                     "ms_per_step": ms_per_step, "step_graph_replay_ms": graph_ms,
                                     "value": value, "unit": UNIT, "rotate_quant": roof_rq, "gemm": roof_gemm,
                                     "clocks": clocks}}
            layer.close()
            for ow in wl.ALL_WORKLOADS:
                if ow.name == w.name:
                    continue
                try:
                    ol = Layer(sq, torch, ow, local_rank, structured_r2=args.structured_r2,
                               fuse_decode=args.fuse_decode)
                    for i in range(5):
                        ol.step(i)
                    torch.cuda.synchronize()
                    ostep = 100
                    t0 = time.perf_counter()
                    oms = ol.timed_steps(ostep) / ostep
                    # keep the clocks' window at least 0.35 s long
                    extra = int(np.ceil(max(0.0, 0.35 - (time.perf_counter() - t0)) / max(oms * 1e-3, 1e-6)))
                    if extra > 0:
                        ol.timed_steps(min(extra, 200000))
                    t1 = time.perf_counter()
                    orq, oge, ogr, _ = ol.kernel_times(min(ostep, 4 * ol.nsets))
                    og, orr = rooflines(ow, orq, oge, pk, ol.rot.structured,
                                        int8_yardstick(torch, ow, l2))
                    per_workload[ow.name] = {
                        "M": ow.M, "N": ow.N, "K": ow.K, "n1": ow.n1, "n2": ow.n2, "steps": ostep,
                        "ms_per_step": oms, "step_graph_replay_ms": ogr,
                        "value": ops_per_step(ow) / (oms * 1e-3) / 1e12, "unit": UNIT,
                        "rotate_quant": orr, "gemm": og, "clocks": sampler.window(t0, t1),
                        "device_status": sq.sq_last_device_status()}
                    ol.close()
                    del ol
                except Exception as exc:
                    per_workload[ow.name] = {"error": str(exc)}
        # ---- the weight-only variant and the grouped layer, briefly ---------------------------------
        variants = None
        if world == 1 and not args.no_sweep:
            variants = {"weight_only": {}, "grouped": None}
            for ow, bits in ((wl.L7B_QKVO, 4), (wl.L7B_QKVO, 3), (wl.L7B_GATEUP, 4), (wl.L70B_GATEUP, 4),
                             (wl.decode_up(1), 4), (wl.decode_down(1), 4), (wl.decode_up(16), 4),
                             (wl.decode_down(16), 4)):
                try:
                    variants["weight_only"][f"{ow.name}_w{bits}a16"] = weight_only_entry(sq, torch, ow, bits, pk, l2)
                except Exception as exc:
                    variants["weight_only"][f"{ow.name}_w{bits}a16"] = {"error": str(exc)}
            try:
                variants["grouped"] = grouped_entry(sq, torch, l2)
                variants["grouped_decode"] = grouped_entry(sq, torch, l2, T=16)
            except Exception as exc:
                variants["grouped"] = {"error": str(exc)}
        sampler.stop()

        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": warm, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "int8",
            "data": "synthetic",
            "config": {"workload": w.name, "M_per_gpu": M, "N": N, "K": K, "n1": w.n1, "n2": w.n2,
                       "r2_application": "structured (butterflies + rotation chains)" if structured else "dense",
                       "parallelism": f"token-sharded x{world}, no collective",
                       "l2": f"ring of {nsets} buffer sets ({nsets * per_set / 1e6:.0f} MB > L2 "
                             f"{l2 / 1e6:.0f} MB)"},
            "roofline": dominant,
            "roofline_other": other,
            "kernel_ms": {"rotate_quant": rq_ms, "w4a4_gemm": gemm_ms, "sum": rq_ms + gemm_ms,
                          "step": ms_per_step, "step_graph_replay": graph_ms, "how": kernel_timing},
            "e2e": {"value": e2e_value, "unit": UNIT, "ms_per_step": e2e_ms, "h2d_bytes_per_step": M * K * 2,
                    "d2h_bytes_per_step": M * N * 2, "api": "sq_linear_host (pinned host X -> host Y)",
                    "link_yardstick_ms": link_ms,
                    "frac_of_link": (link_ms / e2e_ms) if link_ms else None},
            "gpu_launches": int(launches),
            "clocks": clocks,
            "device_status": status,
        }
        if sustained is not None:
            line["sustained"] = sustained
        if cpu is not None:
            line["cpu_baseline"] = cpu
        if per_workload is not None:
            line["per_workload"] = per_workload
        if variants is not None:
            line["variants"] = variants
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None,
                    help="timed steps (default: 20000, about a second of config 2, so that several clock samples "
                         "fall inside the timed region; 20 passes for --impl reference)")
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true",
                    help="skip the timed CPU oracle leg (for profiler runs)")
    ap.add_argument("--no-sweep", action="store_true",
                    help="time the named workload only (skip the per_workload table)")
    ap.add_argument("--fuse-decode", action="store_true",
                    help="build the rotation with SQ_ROT_FUSE_DECODE: batches of up to 64 tokens as one launch")
    ap.add_argument("--structured-r2", action="store_true",
                    help="build the rotation with SQ_ROT_APPLY_STRUCTURED: R2 = H R2^U applied piece by piece "
                         "in registers instead of as a dense matrix on the tensor cores")
    ap.add_argument("--quick", action="store_true",
                    help="the K timed steps and the per-kernel attribution only: no sustained pass, no yardsticks, "
                         "no per-workload table, no CPU baseline (for profiler runs)")
    ap.add_argument("--variants-only", action="store_true",
                    help="time only the weight-only variant of the named workload (W4A16) and print it under "
                         "\"variants\" (for profiler runs of those kernels)")
    ap.add_argument("--grouped-tokens", type=int, default=0,
                    help="with --variants-only: time the grouped (mixture-of-experts) layer on this many tokens "
                         "instead of the weight-only variant")
    args = ap.parse_args()
    if args.quick:
        args.no_sweep = args.no_cpu_baseline = True
    if args.steps is None:
        args.steps = 20 if args.impl == "reference" else 20000
    w = wl.by_name(args.workload)
    if args.impl == "reference":
        return run_reference(args, w)
    if args.variants_only:
        return run_variants_only(args, w)
    return run_ours(args, w)


if __name__ == "__main__":
    sys.exit(main())
