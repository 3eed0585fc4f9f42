#!/usr/bin/env python
"""Benchmark of the CDL quantized layer on B200.

A step is one pass of the whole hot path over one batch of synthetic input: quantize weights and activations
(soft value + hard index + histogram), entropy, forward index GEMM, quantize the arriving gradient, the two
backward index GEMMs, and the analytic quantizer backward for activations and weights.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl cdl|reference]

Prints ONE JSON line (rank 0).  `value` counts the tensor elements that went through a quantizer pass per
second of whole-step time, summed over ranks (each rank runs its own batch: weak scaling).  On one GPU the same
line also carries the rest of the metric: `sweep` (quantizer passes alone, 2^28 / 2^30 elements and the layer's own
tensor size), `gemm` (the index GEMMs alone on the tensor-bound shapes) and `network` (the whole ResNet-18 step).
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import re
import statistics
import subprocess
import sys
import tempfile
import time
from pathlib import Path

ROOT = Path(__file__).resolve().parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))

METRIC = "quantizer Gelem/s (% of HBM peak); CDL layer fwd+bwd ms and int8 TOPS"
UNIT = "Gelem/s"
G_STD = 1e-2                 # standard deviation of the synthetic dL/dY
CPU_BASELINE_SECONDS = 14.0   # host time the all-threads leg of cpu_baseline may spend (it samples the step to fit)
CPU_BASELINE_SECONDS_1T = 8.0  # and the one-thread leg
INT8_OVER_BF16 = 2.0         # nominal dense int8 : bf16 tensor throughput on B200 (4.5 : 2.25 PFLOP/s)
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
BURST_REGION_SECONDS = 1.0   # a timed region shorter than this runs at burst clocks: the burst tensor peak applies
BYTES_PER_ELEM = {"hard": 5, "hard_hist": 5, "soft": 8, "soft_idx_hist": 9, "sample_hist": 5, "backward": 12,
                  "backward_rate": 12}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3000)
    ap.add_argument("--warmup", type=int, default=50)
    ap.add_argument("--impl", default="cdl", choices=["cdl", "reference"])
    ap.add_argument("--workload", default="resnet18_layer3_conv",
                    choices=["resnet18_layer3_conv", "cifar_resnet20_conv", "tiny", "resnet18_b256"])
    ap.add_argument("--batch", type=int, default=256, help="batch size of the resnet18_b256 workload")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--conv-form", action="store_true",
                    help="resnet18_b256: run the layers that cdl_qconv_* supports in convolution form")
    ap.add_argument("--no-implicit", action="store_true", help="skip the extra measurement of the layer in convolution form")
    ap.add_argument("--no-extras", action="store_true",
                    help="default line without its sweep / gemm / network blocks (e.g. for a profiler capture)")
    ap.add_argument("--no-network", action="store_true", help="default line without the whole-network block")
    ap.add_argument("--call-steps", type=int, default=None,
                    help="steps of the call-by-call pass that times each kernel (default: --steps, at least 50, at most 500)")
    ap.add_argument("--no-graph", action="store_true", help="launch the calls of a step one by one instead of replaying a CUDA graph")
    ap.add_argument("--sweep", action="store_true",
                    help="quantizer-only bandwidth sweep (sizes x levels x alpha), one JSON line, 1 GPU")
    ap.add_argument("--sweep-max-log2n", type=int, default=30)
    ap.add_argument("--sweep-dist", default="mixture", choices=["normal", "laplace", "mixture"],
                    help="with --sweep: N(0,1), Laplace(0,1) or their element-wise 50/50 mixture")
    ap.add_argument("--sweep-point", type=float, nargs=3, metavar=("L", "ALPHA", "LOG2N"),
                    help="with --sweep: only this point of the grid (any L <= 127, any alpha), e.g. for a profiler capture")
    ap.add_argument("--gemm", type=int, nargs=3, metavar=("M", "K", "N"), action="append",
                    help="index-GEMM-only timing of the forward, dX and dW products for this shape (repeatable)")
    return ap.parse_args()


def peaks():
    f = ROOT / "MEASURED_PEAKS.json"
    if f.exists():
        p = json.loads(f.read_text())
        return p, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def int8_yardstick(torch, reps=10):
    """A library int8 matrix product timed the way the bf16 peak was measured (8192^3, best of `reps`, CUDA
    events): the int8 throughput cuBLASLt reaches on this device, in TOPS; None if the routine is unavailable."""
    try:
        n = 8192
        a = torch.randint(-8, 8, (n, n), dtype=torch.int8, device="cuda")
        b = torch.randint(-8, 8, (n, n), dtype=torch.int8, device="cuda")
        for _ in range(3):
            torch._int_mm(a, b)
        torch.cuda.synchronize()
        best = float("inf")
        stream = torch.cuda.current_stream()
        for _ in range(reps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            torch._int_mm(a, b)
            e1.record(stream)
            e1.synchronize()
            best = min(best, e0.elapsed_time(e1))
        return 2.0 * n ** 3 / (best * 1e-3) / 1e12
    except Exception:
        return None


def tensor_peaks(pk, pk_kind, yardstick, region_seconds):
    """int8 tensor peaks the fractions are quoted against.  `used`: 2 x the measured bf16 figure (nominal int8 : bf16
    ratio) - the burst one when the kernels were timed in a region shorter than a second or alone, the sustained
    one inside a long step.  `library_int8_8192`: the library int8 product measured in this run."""
    burst = region_seconds < BURST_REGION_SECONDS
    bf16 = float(pk["bf16_tflops"] if burst else pk.get("bf16_tflops_sustained", pk["bf16_tflops"]))
    return {"used": bf16 * INT8_OVER_BF16,
            "used_source": f"{pk_kind} {'burst' if burst else 'sustained'} bf16 x {INT8_OVER_BF16:g} (nominal int8:bf16)",
            "burst_x2": float(pk["bf16_tflops"]) * INT8_OVER_BF16,
            "sustained_x2": float(pk.get("bf16_tflops_sustained", pk["bf16_tflops"])) * INT8_OVER_BF16,
            "library_int8_8192": yardstick,
            "library_int8_note": "torch._int_mm 8192^3, best of 10, CUDA events (this run)" if yardstick else "unavailable"}


def git_blob_sha1(path: Path) -> str:
    data = path.read_bytes()
    return hashlib.sha1(b"blob %d\0" % len(data) + data).hexdigest()


def traffic_from_profiles(workload, call):
    """DRAM bytes per launch of `call` from the committed ncu summaries: a line
    `bench-traffic: workload=W call=C bytes=B source=<file> sha1=<git blob hash of that file when captured>`.
    Returns (bytes, note); bytes is None when there is no such line or the kernel's source has changed since."""
    pat = re.compile(r"bench-traffic:\s+workload=(\S+)\s+call=(\S+)\s+bytes=(\d+)\s+source=(\S+)\s+sha1=([0-9a-f]{40})")
    for f in sorted((ROOT / "profiles").glob("*.md")):
        for m in pat.finditer(f.read_text()):
            if m.group(1) == workload and m.group(2) == call:
                src = ROOT / m.group(4)
                if src.exists() and git_blob_sha1(src) == m.group(5):
                    return int(m.group(3)), f"ncu capture summarised in profiles/{f.name}, kernel source unchanged since"
                return None, f"profiles/{f.name} holds counters for an older version of {m.group(4)}"
    return None, "no ncu capture of this call committed"


def make_case(name, seed_offset=0):
    from paper_2501_09849_b200 import inputs
    if name == "resnet18_layer3_conv":
        case, w, x = inputs.resnet18_layer3_conv(seed=3 + seed_offset)
    elif name == "cifar_resnet20_conv":
        case, w, x = inputs.cifar_resnet20_conv(seed=2 + seed_offset)
    else:
        case, w, x = inputs.tiny_layer(seed=0 + seed_offset)
        case.aq.window = 5
    return case, w, x


def host_inputs(case, w, x, hist_x):
    """Remaining inputs of a step: im2col index matrix (drawn from the activations' own level histogram),
    gradient arriving at the output, gradient arriving at the quantized activations."""
    from paper_2501_09849_b200 import inputs
    A = inputs.indices_from_histogram((case.M, case.K), hist_x, case.aq.lo, seed=case.seed, stream=3)
    dY = inputs.normal((case.M, case.N), G_STD, seed=case.seed, stream=4)
    gx = inputs.normal((x.size,), 1.0, seed=case.seed, stream=5)
    return {"w": w.reshape(-1), "x": x.reshape(-1), "A_idx": A, "dY": dY, "gx_in": gx}


def call_model(case, n_x):
    """Algorithmic bytes and integer operations per call of a step (what the method must move / compute)."""
    M, K, N = case.M, case.K, case.N
    n_w = K * N
    return {
        "quantize_soft_w": {"bytes": n_w * 9, "elems": n_w},
        "entropy_w": {"bytes": case.wq.nlev * 12, "elems": 0},
        "quantize_soft_x": {"bytes": n_x * 9, "elems": n_x},
        "entropy_x": {"bytes": case.aq.nlev * 12, "elems": 0},
        "qlinear_fwd": {"bytes": M * K + K * N + 4 * M * N, "ops": 2 * M * K * N, "elems": 0},
        "quantize_hard_g": {"bytes": M * N * 5, "elems": M * N},
        "qlinear_bwd_dx": {"bytes": M * N + K * N + 4 * M * K, "ops": 2 * M * K * N, "elems": 0},
        "qlinear_bwd_dw": {"bytes": M * K + M * N + 4 * K * N, "ops": 2 * M * K * N, "elems": 0},
        "quantize_backward_x": {"bytes": n_x * 12, "elems": n_x},
        "quantize_backward_w": {"bytes": n_w * 12, "elems": n_w},
    }


def conv_call_model(case, n_x):
    """call_model for the convolution form: the products read the NHWC index tensor (n_x bytes) instead of the
    M x K patch matrix and dX is written in the layout of x."""
    M, K, N = case.M, case.K, case.N
    m = call_model(case, n_x)
    m["qlinear_fwd"]["bytes"] = n_x + K * N + 4 * M * N
    m["qlinear_bwd_dx"]["bytes"] = M * N + K * N + 4 * n_x
    m["qlinear_bwd_dw"]["bytes"] = n_x + M * N + 4 * K * N
    return m


def queue_ahead(torch, ms=8.0):
    """Keeps the device busy for about `ms` so that the host can enqueue the launches that follow before the device
    reaches them: the intervals between their events then hold device time only, not the host's launch path."""
    sleep = getattr(torch.cuda, "_sleep", None)
    if sleep is not None:
        sleep(int(ms * 1e-3 * 1.9e9))


def per_call_times(torch, step, calls, k_steps, stream, **run_kw):
    """Mean device time of each call of a step: k_steps steps launched call by call with one CUDA event between
    calls, the host kept ahead of the device (queue_ahead) in chunks that fit the launch queue."""
    events = [[torch.cuda.Event(enable_timing=True) for _ in range(len(calls) + 1)] for _ in range(k_steps)]
    chunk = 32
    for it0 in range(0, k_steps, chunk):
        torch.cuda.synchronize()
        queue_ahead(torch)
        for it in range(it0, min(k_steps, it0 + chunk)):
            ev = iter(events[it])
            step.run(mark=lambda name: next(ev).record(stream), **run_kw)
    torch.cuda.synchronize()
    return {name: sum(events[it][i].elapsed_time(events[it][i + 1]) for it in range(k_steps)) / k_steps
            for i, name in enumerate(calls)}


def kernel_table(calls, model, per_call_ms, hbm, tp):
    """Per call: time, algorithmic GB/s, and for the products int8 TOPS and the fraction of min(tensor, HBM) roofline
    (tensor peak: tp['used']; the fraction of the library int8 product is given beside it)."""
    kernels = {}
    for name in calls:
        m, ms = model[name], per_call_ms[name]
        k = {"ms": round(ms, 5), "GBps": round(m["bytes"] / (ms * 1e-3) / 1e9, 1)}
        if m["elems"]:
            k["Gelem_per_s"] = round(m["elems"] / (ms * 1e-3) / 1e9, 2)
            k["hbm_frac_measured"] = round(k["GBps"] / hbm, 4)
            k["hbm_frac_8TBps"] = round(k["GBps"] / 8000.0, 4)
        if "ops" in m:
            tops = m["ops"] / (ms * 1e-3) / 1e12
            k["int8_TOPS"] = round(tops, 1)
            t_tensor, t_hbm = m["ops"] / (tp["used"] * 1e12), m["bytes"] / (hbm * 1e9)
            k["bound"] = "tensor" if t_tensor >= t_hbm else "hbm"
            k["roofline_frac"] = round(max(t_tensor, t_hbm) / (ms * 1e-3), 4)
            k["int8_frac_of_peak"] = round(tops / tp["used"], 4)
            if tp.get("library_int8_8192"):
                k["int8_frac_of_library_int8"] = round(tops / tp["library_int8_8192"], 4)
        kernels[name] = k
    return kernels


def run_implicit_conv(torch, cdl, CdlLayerStep, CALLS, case, step, q_g, steps, peaks_hbm, tp, call_steps=None):
    """The same layer as a convolution computed straight from the NHWC index tensor (cdl_qconv_*): same w, x and
    dL/dY, the data gradient feeds the activation quantizer's backward pass directly.  Returns a dict of times."""
    n_img, H, W, C = case.a_shape
    taps = case.K // C
    R = S = int(round(taps ** 0.5))
    assert R * S * C == case.K and n_img * H * W == case.M
    shape = cdl.ConvShape(n_img, H, W, C, R, S)
    cs = CdlLayerStep(torch, case.M, case.K, case.N, step.n_x, case.wq, case.aq, q_g, conv=shape)
    cs.w.copy_(step.w)
    cs.x.copy_(step.x)
    cs.dY.copy_(step.dY)
    stream = torch.cuda.current_stream()
    for _ in range(3):
        cs.run()
    graph = cs.capture()
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(steps):
        graph.replay()
    e1.record(stream)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    k_steps = call_steps if call_steps else max(50, min(steps, 200))
    per = per_call_times(torch, cs, CALLS, k_steps, stream)
    model = conv_call_model(case, step.n_x)
    kern = kernel_table(CALLS, model, per, peaks_hbm, tp)
    quant_elems = sum(m["elems"] for m in model.values())
    # end to end: this form's inputs (w, x, dL/dY) from pinned host memory every step, scalars and dL/dw back
    pinned = {k: t.cpu().pin_memory() for k, t in cs.input_tensors().items()}
    out_host = {"scalars": torch.empty(6, dtype=torch.float64).pin_memory(),
                "dw": torch.empty(cs.n_w, dtype=torch.float32).pin_memory()}
    e_steps = max(4, min(steps, 10))
    cs_b = CdlLayerStep(torch, case.M, case.K, case.N, step.n_x, case.wq, case.aq, q_g, conv=shape)
    for k, t in cs_b.input_tensors().items():
        t.copy_(pinned[k], non_blocking=True)
    cs_b.run()
    graph_b = cs_b.capture()
    e2e_ms = e2e_pipelined(torch, (cs, cs_b), (graph, graph_b), pinned, out_host, e_steps)
    del cs_b, graph_b
    h2d = sum(v.numel() * v.element_size() for v in pinned.values())
    d2h = sum(v.numel() * v.element_size() for v in out_host.values())
    status = cdl.cdl_workspace_status(cs.ws, check=False)
    return {"ms_per_step": ms, "value": quant_elems / (ms * 1e-3) / 1e9, "unit": UNIT, "steps": steps,
            "e2e": {"value": quant_elems / (e2e_ms * 1e-3) / 1e9, "unit": UNIT, "ms_per_step": e2e_ms,
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e_steps,
                    "overlap": "two sets of device buffers: the copy of step i+1 overlaps the kernels of step i"},
            "gpu_launches": steps * cs.kernels_per_step(), "device_status": status, "kernels": kern,
            "step_hbm": {"bytes": int(sum(m["bytes"] for m in model.values())),
                         "frac_of_measured_per_gpu": round(sum(m["bytes"] for m in model.values()) / (ms * 1e-3) / 1e9 / peaks_hbm, 4)},
            "note": "same layer through cdl_qconv_fwd/bwd: no stored patch matrix, dX in the layout of x"}


def e2e_pipelined(torch, steps2, graphs2, pinned, out_host, e_steps, run_kw=None):
    """End-to-end steps from host buffers: every step copies its inputs from pinned host memory, runs, and reads
    the scalars and dL/dw back.  Two sets of device buffers alternate, so the copy of step i+1 (on a copy stream)
    overlaps the kernels of step i; the host-to-device copies themselves are the critical path.
    Returns milliseconds per step."""
    stream = torch.cuda.current_stream()
    copy_s = torch.cuda.Stream()
    in_ready = [torch.cuda.Event(), torch.cuda.Event()]
    done = [torch.cuda.Event(), torch.cuda.Event()]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record(stream)
    copy_s.wait_event(e0)
    for i in range(e_steps):
        b = i % 2
        st = steps2[b]
        with torch.cuda.stream(copy_s):
            if i >= 2:
                copy_s.wait_event(done[b])          # the step that last used these buffers has finished
            for k, t in st.input_tensors().items():
                t.copy_(pinned[k].view(t.shape), non_blocking=True)
            in_ready[b].record(copy_s)
        stream.wait_event(in_ready[b])
        if graphs2[b] is not None:
            graphs2[b].replay()
        else:
            st.run(**(run_kw or {}))
        out_host["scalars"].copy_(st.scalars, non_blocking=True)
        out_host["dw"].copy_(st.dw, non_blocking=True)
        done[b].record(stream)
    e1.record(stream)
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / e_steps


class ClockSampler:
    QUERY = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu_index = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu_index), f"--query-gpu={self.QUERY}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self, t0=None, t1=None):
        """Median SM clock and throttle reasons of the samples taken between wall-clock times t0 and t1 (the timed
        region); if the region was too short to contain a sample, of all samples since start()."""
        import datetime
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0, "window": "timed region"}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        rows = []
        try:
            for line in open(self.path):
                f = [c.strip() for c in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    ts = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                    rows.append((ts, float(f[1]), float(f[2]), [n for n, v in zip(names, f[5:9]) if v.lower().startswith("active")]))
                except ValueError:
                    continue
            os.unlink(self.path)
        except Exception:
            pass
        inside = [r for r in rows if t0 is not None and t0 <= r[0] <= t1]
        if not inside:
            inside, out["window"] = rows, "warm-up + timed region (timed region shorter than the sampling period)"
        if inside:
            out.update(sm_mhz=statistics.median(r[1] for r in inside), sm_max_mhz=max(r[2] for r in inside),
                       reasons=sorted({n for r in inside for n in r[3]}), samples=len(inside))
        return out


def oracle_step_sample(case, host, frac=1.0):
    """Times the CPU oracle, as it stands, on a fraction `frac` of one step (leading elements / rows of every
    tensor) and scales every part to the full step by the units it processed.
    Returns (estimated seconds of a full step, description, threads, wall seconds actually spent)."""
    import numpy as np
    import oracle
    f32 = np.float32
    wq, aq = case.wq, case.aq
    n_x, n_w = host["x"].size, host["w"].size
    ns = int(max(min(n_x, 1 << 10), min(n_x, round(frac * n_x))))
    nw = int(max(min(n_w, 1 << 10), min(n_w, round(frac * n_w))))
    r = int(max(2, min(case.M, round(frac * case.M))))
    xs, gs = host["x"][:ns], host["gx_in"][:ns]
    w, ws = host["w"], host["w"][:nw]
    t_total = 0.0
    t_wall0 = time.perf_counter()

    def timed(fn, scale):
        nonlocal t_total
        t0 = time.perf_counter()
        out = fn()
        t_total += (time.perf_counter() - t0) * scale
        return out

    sx, sw, sm = n_x / ns, n_w / nw, case.M / r
    timed(lambda: oracle.soft(ws, f32(wq.q), wq.lo, wq.hi, f32(wq.alpha), wq.window), sw)
    _, hw = timed(lambda: oracle.hard(ws, f32(wq.q), wq.lo, wq.hi), sw)
    _, pw, _ = timed(lambda: oracle.entropy(hw), 1.0)
    timed(lambda: oracle.soft(xs, f32(aq.q), aq.lo, aq.hi, f32(aq.alpha), aq.window), sx)
    _, hx = timed(lambda: oracle.hard(xs, f32(aq.q), aq.lo, aq.hi), sx)
    _, px, _ = timed(lambda: oracle.entropy(hx), 1.0)
    W8 = oracle.hard(w, f32(wq.q), wq.lo, wq.hi)[0].reshape(case.K, case.N).astype(np.int8)   # operand set-up, untimed
    A = host["A_idx"][:r]
    timed(lambda: oracle.gemm_fwd(A, W8), sm)
    q_g = 4.0 * G_STD / 127.0
    gi, _ = timed(lambda: oracle.hard(host["dY"][:r], f32(q_g), -127, 127), sm)
    G8 = gi.astype(np.int8)
    timed(lambda: oracle.gemm_dx(G8, W8), sm)
    dW = timed(lambda: oracle.gemm_dw(A, G8), sm)
    timed(lambda: oracle.backward(xs, gs, f32(aq.q), aq.lo, aq.hi, f32(aq.alpha), aq.window, f32(aq.rate_weight), px), sx)
    gw = (dW.astype(np.float64) * q_g * aq.q).astype(f32).reshape(-1)[:nw]
    timed(lambda: oracle.backward(ws, gw, f32(wq.q), wq.lo, wq.hi, f32(wq.alpha), wq.window, f32(wq.rate_weight), pw), sw)
    desc = (f"oracle on {ns} of {n_x} activations and {nw} of {n_w} weights (quantize, entropy, backward), "
            f"{r} of {case.M} GEMM rows (fwd, dX, dW); each part scaled to the full step")
    return t_total, desc, oracle.threads(), time.perf_counter() - t_wall0


def cpu_baseline_block(case, host, quant_elems):
    """The oracle, as it stands, on the host cores: at all threads and at one thread, each on a bounded sample."""
    import oracle
    oracle.build()
    all_threads = oracle.threads()

    def leg(seconds):
        cal = oracle_step_sample(case, host, 1.0 / 256)[3]
        frac = min(1.0, seconds / max(256.0 * cal, 1e-9))
        return oracle_step_sample(case, host, frac)

    t_cpu, desc, thr, _ = leg(CPU_BASELINE_SECONDS)
    out = {"value": quant_elems / t_cpu / 1e9, "unit": UNIT, "cores": thr, "kind": "oracle", "sample": desc,
           "ms_per_step_estimate": t_cpu * 1e3,
           "timing": "time.perf_counter around each oracle call, one run per part, parts scaled to a full step"}
    try:
        oracle.set_threads(1)
        t1, desc1, thr1, _ = leg(CPU_BASELINE_SECONDS_1T)
        out.update(value_1thread=quant_elems / t1 / 1e9, ms_per_step_estimate_1thread=t1 * 1e3, sample_1thread=desc1,
                   cores_1thread=thr1)
    finally:
        oracle.set_threads(all_threads)
    return out


def run_reference(args, rank):
    """Reference arm: the CPU oracle on a bounded sample of the same workload (rank 0 only)."""
    if rank != 0:
        return
    import numpy as np
    import oracle
    oracle.build()
    case, w, x = make_case(args.workload)
    f32 = np.float32
    _, hist_x = oracle.hard(x.reshape(-1)[: 1 << 20], f32(case.aq.q), case.aq.lo, case.aq.hi)
    host = host_inputs(case, w, x, hist_x)
    quant_elems = 2 * (w.size + x.size) + case.M * case.N
    # size the per-step sample so that warm-up + K steps take about 60 s of host time whatever K is
    _, _, _, wall_cal = oracle_step_sample(case, host, frac=1.0 / 256)
    budget = 60.0 / max(1, args.steps + args.warmup)
    frac = min(1.0, budget / max(256.0 * wall_cal, 1e-9))
    for _ in range(max(args.warmup, 0)):
        oracle_step_sample(case, host, frac)
    ts = []
    for _ in range(args.steps):
        t, desc, thr, _ = oracle_step_sample(case, host, frac)
        ts.append(t)
    t_step = sum(ts) / len(ts)
    value = quant_elems / t_step / 1e9
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": t_step * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.workload, "M": case.M, "K": case.K, "N": case.N},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": thr, "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------------------------- quantizer sweep
def draw(torch, gen, n, dist, scale=1.0):
    """n float32 values on the device: N(0,1), Laplace(0,1) (by inversion) or their element-wise 50/50 mixture."""
    if dist == "normal":
        x = torch.randn(n, device="cuda", generator=gen)
    else:
        u = torch.rand(n, device="cuda", generator=gen) - 0.5
        x = -torch.sign(u) * torch.log1p(-2.0 * u.abs().clamp_(max=0.49999997))      # (u = -0.5 would give an infinity)
        del u
        if dist == "mixture":
            pick = torch.rand(n, device="cuda", generator=gen) < 0.5
            x = torch.where(pick, torch.randn(n, device="cuda", generator=gen), x)
            del pick
    if scale != 1.0:
        x *= scale
    return x.contiguous()


class SweepBuffers:
    """Device buffers of the quantizer-only timings and the timing loop itself."""

    def __init__(self, torch, cdl, nmax, reps):
        self.torch, self.cdl, self.nmax, self.reps = torch, cdl, nmax, reps
        self.gen = torch.Generator(device="cuda").manual_seed(5)
        self.x = None
        self.g = torch.randn(nmax, device="cuda", generator=self.gen)
        self.y = torch.empty(nmax, dtype=torch.float32, device="cuda")
        self.idx = torch.empty(nmax, dtype=torch.int8, device="cuda")
        self.s = torch.zeros(2, dtype=torch.float64, device="cuda")
        self.flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
        self.stream = torch.cuda.current_stream()

    def set_data(self, dist, scale=1.0):
        self.x = None
        self.x = draw(self.torch, self.gen, self.nmax, dist, scale)

    def timed(self, make_fn, n):
        """Median time of one launch.  Launches are issued back to back on distinct slices of the big buffers
        (so that none finds its input in L2 and the CPU-side launch cost is hidden), one event pair around all."""
        torch = self.torch
        k = max(1, min(16, self.nmax // n))
        fns = [make_fn(i * n) for i in range(k)]
        for f in fns[:2]:
            f()
        ts = []
        for _ in range(self.reps):
            if k * n * 12 < (512 << 20):
                self.flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(self.stream)
            for f in fns:
                f()
            e1.record(self.stream)
            e1.synchronize()
            ts.append(e0.elapsed_time(e1) / k)
        return statistics.median(ts)

    def passes(self, n, P, Pr, hist, which=None):
        """{pass name: maker(offset) -> launcher} for n elements under quantizer P (Pr: the same with level
        probabilities, for the rate term)."""
        cdl, x, g, y, s = self.cdl, self.x, self.g, self.y, self.s
        ix_t = self.idx if P.lo < 0 else self.idx.view(self.torch.uint8)

        def mk(kind, PP=P):
            def make(o):
                xs, gs, ys, ix = x[o:o + n], g[o:o + n], y[o:o + n], ix_t[o:o + n]
                if kind == "hard":
                    return lambda: cdl.cdl_quantize_hard(xs, n, PP, ix, None)
                if kind == "hard_hist":
                    return lambda: cdl.cdl_quantize_hard(xs, n, PP, ix, hist)
                if kind == "soft":
                    return lambda: cdl.cdl_quantize_soft(xs, n, PP, ys, None, None)
                if kind == "soft_idx_hist":
                    return lambda: cdl.cdl_quantize_soft(xs, n, PP, ys, ix, hist)
                if kind == "sample_hist":
                    return lambda: cdl.cdl_quantize_sample(xs, n, PP, 7, o, ix, None, hist)
                return lambda: cdl.cdl_quantize_backward(xs, gs, n, PP, ys, s[0:1], s[1:2])
            return make
        out = {"hard": mk("hard"), "hard_hist": mk("hard_hist"), "soft": mk("soft"), "soft_idx_hist": mk("soft_idx_hist"),
               "sample_hist": mk("sample_hist"), "backward": mk("backward"), "backward_rate": mk("backward", Pr)}
        return out if which is None else {k: out[k] for k in which}

    def row(self, n, name, ms, hbm, **extra):
        gbs = n * BYTES_PER_ELEM[name] / (ms * 1e-3) / 1e9
        r = {"n": n, "pass": name, "ms": round(ms, 4), "Gelem_per_s": round(n / (ms * 1e-3) / 1e9, 2), "GBps": round(gbs, 1),
             "hbm_frac_measured": round(gbs / hbm, 4), "hbm_frac_8TBps": round(gbs / 8000.0, 4)}
        r.update(extra)
        return r


def entropy_pass_ms(torch, cdl, nlev, reps=200):
    """cdl_index_entropy on its own: mean device time of back-to-back launches (a latency, not a bandwidth)."""
    hist = torch.randint(1, 1 << 20, (nlev,), dtype=torch.int64, device="cuda")
    H = torch.zeros(1, dtype=torch.float64, device="cuda")
    lp = torch.zeros(nlev, dtype=torch.float32, device="cuda")
    stream = torch.cuda.current_stream()
    for _ in range(3):
        cdl.cdl_index_entropy(hist, nlev, H, lp)
    torch.cuda.synchronize()
    queue_ahead(torch, 2.0)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(reps):
        cdl.cdl_index_entropy(hist, nlev, H, lp)
    e1.record(stream)
    e1.synchronize()
    return e0.elapsed_time(e1) / reps


def sweep_compact(torch, cdl, hbm, reps, layer_n):
    """The part of the quantizer sweep the default line carries: hard / hard+hist / soft+idx+hist / backward / backward
    with rate term at L = 7, alpha = 100 (step 4/L) on 2^28 elements of N(0,1), Laplace(0,1) and their mixture and on
    2^30 elements of the mixture; the paper's own operating point (6 bits, alpha = 500, step from the mean magnitude,
    weight-like data) on 2^25 elements; the same passes at the bench layer's tensor size, launched back to back on
    distinct slices; the entropy pass on its own."""
    rows = []
    names = ("hard", "hard_hist", "soft_idx_hist", "backward", "backward_rate")

    def point(B, n, L, alpha, q, lo, hi, tag, which=names, window=0):
        nlev = hi - lo + 1
        hist = torch.zeros(nlev, dtype=torch.int64, device="cuda")
        lp = torch.full((nlev,), 1.0 / nlev, dtype=torch.float32, device="cuda")
        lp[nlev // 2] *= 1.5
        P = cdl.QuantParams(q, lo, hi, alpha, 0.01, None, window)
        Pr = cdl.QuantParams(q, lo, hi, alpha, 0.01, lp, window)
        for name, make in B.passes(n, P, Pr, hist, which).items():
            rows.append(B.row(n, name, B.timed(make, n), hbm, L=L, alpha=alpha, data=tag, levels=nlev, window=window))

    n28 = 1 << 28
    B = SweepBuffers(torch, cdl, n28, reps)
    for dist in ("normal", "laplace", "mixture"):
        B.set_data(dist)
        point(B, n28, 7, 100.0, 4.0 / 7, -7, 7, dist)
    # bench layer size (12.85 M elements), mixture data still loaded: 16 distinct slices back to back
    point(B, layer_n, 7, 100.0, 4.0 / 7, -7, 7, "mixture, layer-size tensors back to back")
    # the layer's own activation quantizer (16 unsigned levels, window of five) on half-normal data of that size
    B.x.abs_()
    q_act = float(2.0 * B.x[:layer_n].mean() / 8.0 ** 0.5)
    point(B, layer_n, None, 100.0, q_act, 0, 15, "half-normal, layer-size tensors back to back", window=5,
          which=("soft_idx_hist", "backward_rate"))
    # the paper's operating point: b = 6, alpha = 500, step 2 mean|w| / sqrt(2^(b-1)) on He-normal-like weights
    n25 = 1 << 25
    B.set_data("normal", scale=(2.0 / 2304.0) ** 0.5)
    q6 = float(2.0 * B.x[:n25].abs().mean() / 32.0 ** 0.5)
    point(B, n25, None, 500.0, q6, -32, 31, "He-normal weights, 6-bit paper point (Sec. VI-B.3)", which=("soft_idx_hist", "backward"))
    del B
    torch.cuda.empty_cache()
    n30 = 1 << 30
    B = SweepBuffers(torch, cdl, n30, max(3, reps // 2))
    B.set_data("mixture")
    point(B, n30, 7, 100.0, 4.0 / 7, -7, 7, "mixture", which=("hard", "soft_idx_hist", "backward"))
    del B
    torch.cuda.empty_cache()
    ent = {f"nlev_{k}": round(entropy_pass_ms(torch, cdl, k) * 1e3, 2) for k in (15, 16, 255)}
    return {"rows": rows, "entropy_pass_us": ent,
            "timing": "median over repetitions of back-to-back launches on distinct slices (one CUDA event pair around "
                      "up to 16 launches), inputs never L2-resident"}


def run_sweep(args):
    """Quantizer-only bandwidth sweep: fp32 tensors of 2^20 .. 2^max elements (N(0,1), Laplace(0,1) or their 50/50
    mixture, drawn on the device), L in {1,3,7,15,127}, alpha in {1,100,1e4}, step 4/L; hard, hard+hist, soft,
    soft+idx+hist, sampled index+hist, backward and backward+rate timed separately with CUDA events."""
    import torch

    import paper_2501_09849_b200 as cdl
    from paper_2501_09849_b200 import build as cdl_build
    cdl_build.build()
    cdl.load_library()
    torch.cuda.set_device(0)
    pk, pk_kind = peaks()
    hbm = float(pk["hbm_gbs"])
    grid_n = list(range(20, args.sweep_max_log2n + 1, 2))
    grid_L, grid_alpha = (1, 3, 7, 15, 127), (1.0, 100.0, 1e4)
    if args.sweep_point:
        grid_L, grid_alpha, grid_n = (int(args.sweep_point[0]),), (float(args.sweep_point[1]),), [int(args.sweep_point[2])]
        args.sweep_max_log2n = grid_n[0]
    nmax = 1 << args.sweep_max_log2n
    B = SweepBuffers(torch, cdl, nmax, max(3, args.steps // 4))
    B.set_data(args.sweep_dist)
    rows = []
    for log2n in grid_n:
        n = 1 << log2n
        for L in grid_L:
            hist = torch.zeros(2 * L + 1, dtype=torch.int64, device="cuda")
            lp = torch.full((2 * L + 1,), 1.0 / (2 * L + 1), dtype=torch.float32, device="cuda")
            lp[L] *= 1.5
            for alpha in grid_alpha:
                P = cdl.QuantParams(4.0 / L, -L, L, alpha, 0.01)
                Pr = cdl.QuantParams(4.0 / L, -L, L, alpha, 0.01, lp)
                passes = B.passes(n, P, Pr, hist)
                if alpha != grid_alpha[0]:
                    passes.pop("hard"), passes.pop("hard_hist")      # the hard passes do not depend on alpha
                for name, make in passes.items():
                    r = B.row(n, name, B.timed(make, n), hbm, L=L, alpha=alpha)
                    r["log2n"] = log2n
                    rows.append(r)
    ent = {f"nlev_{k}": round(entropy_pass_ms(torch, cdl, k) * 1e3, 2) for k in (3, 7, 15, 31, 255)}
    print(json.dumps({"metric": METRIC, "unit": UNIT, "sweep": rows, "entropy_pass_us": ent, "peak_hbm_gbs": hbm,
                      "peak_source": pk_kind, "data": "synthetic",
                      "config": {"workload": "quantizer_sweep", "max_log2n": args.sweep_max_log2n,
                                 "distribution": args.sweep_dist}}), flush=True)


# ----------------------------------------------------------------------------------------------- index GEMMs alone
def gemm_rows(torch, cdl, shapes, steps, hbm, tp):
    """Index GEMMs alone: forward, dX and dW for each (M, K, N), 4-bit activation / weight indices and 8-bit gradient
    indices drawn uniformly on the device, float outputs; operands are rotated over several buffer sets when one set
    would fit in L2; each product's pass over the buffer sets is replayed from a CUDA graph."""
    stream = torch.cuda.current_stream()
    gen = torch.Generator(device="cuda").manual_seed(7)
    a, w, g = cdl.IndexDesc(0.25, 0, 15), cdl.IndexDesc(0.02, -7, 7), cdl.IndexDesc(1e-3, -127, 127)
    out = []
    for M, K, N in shapes:
        set_bytes = M * K + K * N + M * N + 4 * (M * N + M * K + K * N)
        nset = max(1, min(4, (400 << 20) // set_bytes + 1))
        sets = []
        for _ in range(nset):
            A = torch.randint(0, 16, (M, K), device="cuda", generator=gen, dtype=torch.uint8)
            W = torch.randint(-7, 8, (K, N), device="cuda", generator=gen, dtype=torch.int8)
            G = torch.randint(-127, 128, (M, N), device="cuda", generator=gen, dtype=torch.int8)
            sets.append((A, W, G, torch.empty((M, N), dtype=torch.float32, device="cuda"),
                         torch.empty((M, K), dtype=torch.float32, device="cuda"),
                         torch.empty((K, N), dtype=torch.float32, device="cuda")))
        nb = max(cdl.cdl_workspace_bytes(cdl.CDL_OP_QLINEAR_FWD, M, N, K), cdl.cdl_workspace_bytes(cdl.CDL_OP_QLINEAR_BWD, M, N, K))
        ws = torch.empty(nb, dtype=torch.uint8, device="cuda")
        calls = {
            "fwd": lambda t: cdl.cdl_qlinear_fwd(t[0], K, a, t[1], N, w, M, N, K, None, t[3], None, ws, nb),
            "dx": lambda t: cdl.cdl_qlinear_bwd(t[2], N, g, None, K, None, t[1], N, w, M, N, K, None, t[4], None, None, ws, nb),
            "dw": lambda t: cdl.cdl_qlinear_bwd(t[2], N, g, t[0], K, a, None, N, None, M, N, K, None, None, None, t[5], ws, nb),
        }
        bytes_ = {"fwd": M * K + K * N + 4 * M * N, "dx": M * N + K * N + 4 * M * K, "dw": M * K + M * N + 4 * K * N}
        row = {"M": M, "K": K, "N": N, "buffer_sets": nset}
        for name, fn in calls.items():
            for t in sets:
                fn(t)
            torch.cuda.synchronize()
            side = torch.cuda.Stream()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.stream(side):
                with torch.cuda.graph(graph, stream=side):
                    for t in sets:
                        fn(t)
            rounds = max(2, min(40, steps) // nset)
            graph.replay()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for i in range(rounds):
                graph.replay()
            e1.record(stream)
            e1.synchronize()
            ms = e0.elapsed_time(e1) / (rounds * nset)
            ops = 2.0 * M * K * N
            tops = ops / (ms * 1e-3) / 1e12
            t_tensor, t_hbm = ops / (tp["burst_x2"] * 1e12), bytes_[name] / (hbm * 1e9)
            row[name] = {"ms": round(ms, 5), "int8_TOPS": round(tops, 1),
                         "int8_frac_of_peak": round(tops / tp["burst_x2"], 4),
                         "GBps": round(bytes_[name] / (ms * 1e-3) / 1e9, 1), "bound": "tensor" if t_tensor >= t_hbm else "hbm",
                         "roofline_frac": round(max(t_tensor, t_hbm) / (ms * 1e-3), 4)}
            if tp.get("library_int8_8192"):
                row[name]["int8_frac_of_library_int8"] = round(tops / tp["library_int8_8192"], 4)
        row["status"] = cdl.cdl_workspace_status(ws, check=False)
        out.append(row)
        del sets
    return out


def run_gemm(args):
    import torch

    import paper_2501_09849_b200 as cdl
    from paper_2501_09849_b200 import build as cdl_build
    cdl_build.build()
    cdl.load_library()
    torch.cuda.set_device(0)
    pk, pk_kind = peaks()
    hbm = float(pk["hbm_gbs"])
    tp = tensor_peaks(pk, pk_kind, int8_yardstick(torch), 0.0)       # kernels timed alone: burst figure
    rows = gemm_rows(torch, cdl, args.gemm, args.steps, hbm, tp)
    print(json.dumps({"metric": METRIC, "unit": "int8 TOPS", "gemm": rows, "int8_peak_tops": tp["burst_x2"],
                      "tensor_peaks": tp, "peak_hbm_gbs": hbm, "data": "synthetic",
                      "config": {"workload": "index_gemm"}}), flush=True)


# ----------------------------------------------------------------------------------------------- whole network
def network_step(torch, cdl, batch, conv_form, steps, warm, use_graph=True):
    """Whole ResNet-18 (224x224) as a sequence of CDL layer steps: every conv and the FC layer with its true im2col
    GEMM shape, 3-bit weights (step = std(w) / 3), 4-bit activations (step from the mean magnitude), window of 5.
    Inputs are drawn on the device (seeded); each layer owns its buffers, so a step touches ~40 GB at batch 256.
    Returns the fields of the network line."""
    from paper_2501_09849_b200 import inputs
    from paper_2501_09849_b200.layer import CALLS, CdlLayerStep
    gen = torch.Generator(device="cuda").manual_seed(4)
    stream = torch.cuda.current_stream()
    q_g = 4.0 * G_STD / 127.0
    layers = []
    for name, M, K, N, n_x in inputs.resnet18_layers(batch):
        Np = (N + 15) // 16 * 16                  # index matrices need 16-byte row pitches: fc's 1000 columns -> 1008
        w = torch.randn(K * Np, device="cuda", generator=gen) * (2.0 / K) ** 0.5
        x = torch.randn(n_x, device="cuda", generator=gen).abs_()
        wq = inputs.Quantizer(float(w.std()) / 3.0, -3, 3, 100.0, 0.01, 0)
        xq = inputs.Quantizer(float(2.0 * x.mean() / 8.0 ** 0.5), 0, 15, 100.0, 0.01, 5)
        geo = inputs.resnet18_conv_geometry(name) if conv_form else None
        shape = cdl.ConvShape(batch, geo[0], geo[1], geo[2], geo[3], geo[4], geo[5], geo[6], geo[6]) if geo else None
        st = CdlLayerStep(torch, M, K, Np, n_x, wq, xq, q_g, need_dx=(name != "conv1"), conv=shape)   # the image needs no gradient
        st.w.copy_(w)
        st.x.copy_(x)
        del w, x
        if shape is None:
            # im2col index matrix drawn from the quantized activations' own level histogram
            hist = torch.zeros(16, dtype=torch.int64, device="cuda")
            cdl.cdl_quantize_hard(st.x, n_x, cdl.QuantParams(xq.q, 0, 15), None, hist)
            cdf = torch.cumsum(hist.double() / float(n_x), 0).float()
            rows = max(1, (1 << 26) // K)
            for r0 in range(0, M, rows):
                r1 = min(M, r0 + rows)
                u = torch.rand((r1 - r0, K), device="cuda", generator=gen)
                st.A_idx[r0:r1, :K] = torch.searchsorted(cdf, u).clamp_(max=15).to(torch.uint8)
            st.gx_in.copy_(torch.randn(n_x, device="cuda", generator=gen))
        st.dY.copy_(torch.randn((M, Np), device="cuda", generator=gen) * G_STD)
        layers.append((name, M, K, N, n_x, st))
    torch.cuda.synchronize()

    def run_all(mark=None):
        for li, (_, _, _, _, _, st) in enumerate(layers):
            st.run(mark=(lambda nm, li=li: mark(li, nm)) if mark else None)

    for _ in range(warm):
        run_all()
    torch.cuda.synchronize()
    # the whole network step as one CUDA graph (each layer recorded on three streams), replayed `steps` times
    graph = None
    if use_graph:
        graph = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        side.wait_stream(stream)
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                for *_, st in layers:
                    st.run_forked()
        stream.wait_stream(side)
        graph.replay()
        torch.cuda.synchronize()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record(stream)
        for _ in range(steps):
            graph.replay()
        g1.record(stream)
        torch.cuda.synchronize()
        graph_ms = g0.elapsed_time(g1) / steps
    c_steps = min(steps, 5)
    ev = [[[torch.cuda.Event(enable_timing=True) for _ in range(len(CALLS) + 1)] for _ in layers] for _ in range(c_steps)]
    cnt = {}
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(0)
    sampler.start()
    time.sleep(0.3)
    wall0 = time.time()
    torch.cuda.synchronize()
    queue_ahead(torch)
    t0.record(stream)
    for it in range(c_steps):
        cnt.clear()

        def mark(li, nm, it=it):
            i = cnt.get(li, 0)
            ev[it][li][i].record(stream)
            cnt[li] = i + 1
        run_all(mark)
    t1.record(stream)
    torch.cuda.synchronize()
    clocks = sampler.stop(wall0, time.time())
    ms_step = t0.elapsed_time(t1) / c_steps
    call_by_call_ms = ms_step
    if graph is not None:
        ms_step = graph_ms
    table, tot_ops, tot_q, gemm_ms, quant_ms = [], 0.0, 0, 0.0, 0.0
    for li, (name, M, K, N, n_x, st) in enumerate(layers):
        per = {c: sum(ev[it][li][i].elapsed_time(ev[it][li][i + 1]) for it in range(c_steps)) / c_steps for i, c in enumerate(CALLS)}
        g_ms = per["qlinear_fwd"] + per["qlinear_bwd_dx"] + per["qlinear_bwd_dw"]
        q_ms = sum(v for c, v in per.items() if c.startswith("quantize"))
        ops = (6.0 if st.need_dx else 4.0) * M * K * N
        q_el = 2 * (n_x + K * N) + M * N
        table.append({"layer": name, "M": M, "K": K, "N": N, "form": "convolution" if st.conv is not None else "stored patch matrix",
                      "ms": round(sum(per.values()), 4), "gemm_ms": round(g_ms, 4),
                      "gemm_int8_TOPS": round(ops / (g_ms * 1e-3) / 1e12, 1), "quantizer_ms": round(q_ms, 4),
                      "quantizer_Gelem_per_s": round(q_el / (q_ms * 1e-3) / 1e9, 1),
                      "calls_us": {c: round(v * 1e3, 1) for c, v in per.items()},
                      "status": cdl.cdl_workspace_status(st.ws, check=False)})
        tot_ops += ops
        tot_q += q_el
        gemm_ms += g_ms
        quant_ms += q_ms
    n_conv = sum(1 for *_, st in layers if st.conv is not None)
    return {
        "value": tot_q / (ms_step * 1e-3) / 1e9, "unit": UNIT, "steps": steps, "warmup": warm, "ms_per_step": ms_step,
        "config": {"workload": "resnet18_b256", "batch": batch, "layers": len(layers),
                   "form": ("convolution form for %d layers, stored patch matrices for the rest" % n_conv) if conv_form
                   else "stored patch matrices (im2col GEMMs)",
                   "launch": "stream launches" if graph is None else "CUDA graph replay of the network step",
                   "call_by_call_ms": call_by_call_ms, "weight_levels": 7,
                   "activation_levels": 16, "window_x": 5, "l2": "every layer's tensors exceed the 126 MB L2"},
        "network_fwd_bwd_ms": ms_step, "gemm_ms": gemm_ms, "gemm_int8_tops": tot_ops / (gemm_ms * 1e-3) / 1e12,
        "quantizer_ms": quant_ms, "quantizer_Gelem_per_s": tot_q / (quant_ms * 1e-3) / 1e9,
        "layers": table, "clocks": clocks,
        "gpu_launches": steps * sum(st.kernels_per_step() for *_, st in layers)}


def run_network(args):
    import torch

    import paper_2501_09849_b200 as cdl
    from paper_2501_09849_b200 import build as cdl_build
    cdl_build.build()
    cdl.load_library()
    torch.cuda.set_device(0)
    pk, pk_kind = peaks()
    warm = max(3, min(args.warmup, 5))
    steps = max(3, min(args.steps, 20))
    net = network_step(torch, cdl, args.batch, args.conv_form, steps, warm, use_graph=not args.no_graph)
    line = {"metric": METRIC, "n_gpus": 1, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32+s8", "data": "synthetic", "peak_hbm_gbs": float(pk["hbm_gbs"]), "peak_source": pk_kind,
            "e2e": None, "e2e_note": "not measured for this workload (a step's inputs are ~11 GB); see the default workload"}
    line.update(net)
    print(json.dumps(line), flush=True)


def main():
    args = parse_args()
    if args.workload == "resnet18_b256" and args.impl == "cdl":
        run_network(args)
        return
    if args.sweep:
        run_sweep(args)
        return
    if args.gemm:
        run_gemm(args)
        return
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank)
        return

    import numpy as np
    import torch
    import torch.distributed as dist

    import paper_2501_09849_b200 as cdl
    from paper_2501_09849_b200 import build as cdl_build
    from paper_2501_09849_b200 import sharding
    from paper_2501_09849_b200.layer import CALLS, CdlLayerStep

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (the product path has no CPU fallback)")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if local_rank == 0:
        cdl_build.build()
    if world > 1:
        dist.barrier()
    cdl.load_library()

    # ---- inputs: seeded, host-generated, one independent batch per rank (weak scaling); the weights are replicated
    case, w, x = make_case(args.workload, seed_offset=100 * rank)
    if rank > 0:
        w = make_case(args.workload, seed_offset=0)[1]
    M, K, N, n_x = case.M, case.K, case.N, x.size
    q_g = float(np.float32(4.0 * G_STD / 127.0))
    step = CdlLayerStep(torch, M, K, N, n_x, case.wq, case.aq, q_g)
    xd = torch.from_numpy(x.reshape(-1)).cuda()
    hist = torch.zeros(case.aq.nlev, dtype=torch.int64, device="cuda")
    cdl.cdl_quantize_hard(xd, n_x, cdl.QuantParams(case.aq.q, case.aq.lo, case.aq.hi), None, hist)
    host = host_inputs(case, w, x, hist.cpu().numpy().view(np.uint64))
    del xd
    pinned = {k: torch.from_numpy(np.ascontiguousarray(v)).pin_memory() for k, v in host.items()}
    dev_in = step.input_tensors()
    for k, t in dev_in.items():
        t.copy_(pinned[k].view(t.shape), non_blocking=True)
    torch.cuda.synchronize()
    stream = torch.cuda.current_stream()

    # data-parallel ranks: the step runs with its exchange points (activation histogram before the entropy, integer
    # dW accumulators before the conversion, the activation quantizer's two scalars at the end), launched call by call
    run_kw = {"exchange": sharding.StepExchange(dist, world), "rows_global": M * world} if world > 1 else {}

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    for _ in range(max(args.warmup, 3)):
        step.run(**run_kw)
    torch.cuda.synchronize()

    # ---- timed region: device-resident inputs, the step replayed from a CUDA graph (launch gaps between the ten
    # short kernels of a step are a tenth of its time when they are launched one by one)
    graph = step.capture() if (not args.no_graph and world == 1) else None
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    wall0 = time.time()
    t_start.record(stream)
    for it in range(args.steps):
        if graph is not None:
            graph.replay()
        else:
            step.run(**run_kw)
    t_end.record(stream)
    torch.cuda.synchronize()
    wall1 = time.time()
    if world > 1:
        dist.barrier()
    clocks = sampler.stop(wall0, wall1) if rank == 0 else None
    total_ms = t_start.elapsed_time(t_end)

    # ---- per-call times: a second pass over the same steps, launched call by call with an event between calls
    k_steps = args.call_steps if args.call_steps else max(50, min(args.steps, 500))
    per_call_ms = per_call_times(torch, step, CALLS, k_steps, stream, **run_kw)
    status = cdl.cdl_workspace_status(step.ws, check=False)

    # ---- end to end: host buffers in, results out, every step
    h2d = sum(v.numel() * v.element_size() for v in pinned.values())
    out_host = {"scalars": torch.empty(6, dtype=torch.float64).pin_memory(),
                "dw": torch.empty(step.n_w, dtype=torch.float32).pin_memory()}
    d2h = sum(v.numel() * v.element_size() for v in out_host.values())
    e_steps = max(4, min(args.steps, 10))
    step_b = CdlLayerStep(torch, M, K, N, n_x, case.wq, case.aq, q_g)       # second set of device buffers
    for k, t in step_b.input_tensors().items():
        t.copy_(pinned[k].view(t.shape), non_blocking=True)
    step_b.run(**run_kw)
    graph_b = step_b.capture() if graph is not None else None
    if world > 1:
        dist.barrier()
    e2e_ms = e2e_pipelined(torch, (step, step_b), (graph, graph_b), pinned, out_host, e_steps, run_kw=run_kw)
    del step_b, graph_b

    ms_step = total_ms / args.steps
    if world > 1:
        t = torch.tensor([ms_step, e2e_ms], dtype=torch.float64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms_step, e2e_ms = float(t[0]), float(t[1])

    if rank == 0:
        pk, pk_kind = peaks()
        model = call_model(case, n_x)
        quant_elems = sum(m["elems"] for m in model.values())
        value = world * quant_elems / (ms_step * 1e-3) / 1e9
        e2e_value = world * quant_elems / (e2e_ms * 1e-3) / 1e9
        hbm = float(pk["hbm_gbs"])
        yard = int8_yardstick(torch) if world == 1 else None
        # the per-call times come from call-by-call launches in a region of k_steps steps
        tp = tensor_peaks(pk, pk_kind, yard, k_steps * ms_step * 1e-3)
        kernels = kernel_table(CALLS, model, per_call_ms, hbm, tp)
        dom = max(CALLS, key=lambda c: per_call_ms[c])
        dm, dms = model[dom], per_call_ms[dom]
        if "ops" in dm and dm["ops"] / (tp["used"] * 1e12) >= dm["bytes"] / (hbm * 1e9):
            roof = {"kernel": dom, "bound": "tensor", "achieved": dm["ops"] / (dms * 1e-3) / 1e12, "peak": tp["used"],
                    "unit": "TFLOP/s", "peak_source": tp["used_source"]}
        else:
            roof = {"kernel": dom, "bound": "hbm", "achieved": dm["bytes"] / (dms * 1e-3) / 1e9, "peak": hbm,
                    "unit": "GB/s", "peak_source": f"{pk_kind} copy bandwidth"}
        roof["frac"] = roof["achieved"] / roof["peak"]
        roof["traffic"], roof["traffic_note"] = traffic_from_profiles(args.workload, dom)
        gemm_ms = sum(per_call_ms[c] for c in ("qlinear_fwd", "qlinear_bwd_dx", "qlinear_bwd_dw"))
        quant_ms = sum(per_call_ms[c] for c in CALLS if model[c]["elems"])
        step_bytes = sum(model[c]["bytes"] for c in CALLS)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32+s8", "data": "synthetic",
            "config": {"workload": args.workload, "M": M, "K": K, "N": N, "activation_elems": n_x,
                       "weight_levels": case.wq.nlev, "activation_levels": case.aq.nlev,
                       "alpha": case.wq.alpha, "rate_weight": case.wq.rate_weight, "window_x": case.aq.window,
                       "l2": ("per-step working set is several times the 126 MB L2 (inputs larger than L2)"
                              if step_bytes > 2 * 126e6 else
                              "a step moves %.0f MB in all, of the order of the 126 MB L2: a parity-size workload, not a bandwidth figure" % (step_bytes / 1e6)),
                       "parallelism": (f"batch rows split over {world} ranks; all-reduce of the activation histogram (before "
                                       "the entropy), the int32 dW accumulators (before the conversion) and two scalars")
                       if world > 1 else "single GPU"},
            "layer_fwd_bwd_ms": ms_step, "gemm_ms": gemm_ms, "gemm_int8_tops": 6.0 * M * K * N / (gemm_ms * 1e-3) / 1e12,
            "quantizer_ms": quant_ms, "quantizer_Gelem_per_s": quant_elems / (quant_ms * 1e-3) / 1e9,
            "quantizer_hbm_frac_measured": sum(model[c]["bytes"] for c in CALLS if model[c]["elems"]) / (quant_ms * 1e-3) / 1e9 / hbm,
            # every call's algorithmic bytes over the step time: what the step as a whole makes of the memory system
            "step_hbm": {"bytes": int(sum(model[c]["bytes"] for c in CALLS)),
                         "GBps": round(sum(model[c]["bytes"] for c in CALLS) / (ms_step * 1e-3) / 1e9 * world, 1),
                         "frac_of_measured_per_gpu": round(sum(model[c]["bytes"] for c in CALLS) / (ms_step * 1e-3) / 1e9 / hbm, 4)},
            "kernels": kernels, "roofline": roof, "tensor_peaks": tp, "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": UNIT, "ms_per_step": e2e_ms, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "steps": e_steps,
                    "overlap": "two sets of device buffers: the copy of step i+1 overlaps the kernels of step i"},
            "gpu_launches": args.steps * (step.kernels_per_step() + (1 if world > 1 else 0)), "device_status": status,
            "launch": "stream launches" if graph is None else "CUDA graph replay of one step",
            "kernel_timing": (f"second pass of {k_steps} steps launched call by call, one CUDA event between calls, the "
                              "host kept ahead of the device"),
        }
        if world == 1 and args.workload == "resnet18_layer3_conv" and not args.no_implicit:
            line["implicit_conv"] = run_implicit_conv(torch, cdl, CdlLayerStep, CALLS, case, step, q_g, args.steps, hbm, tp,
                                                      args.call_steps)
        extras = world == 1 and args.workload == "resnet18_layer3_conv" and not args.no_extras
        if extras:
            del step, graph
            torch.cuda.empty_cache()
            tp_alone = tensor_peaks(pk, pk_kind, yard, 0.0)
            line["gemm"] = {"rows": gemm_rows(torch, cdl, [(12544, 4608, 512), (8192, 8192, 8192)], min(args.steps, 40), hbm, tp_alone),
                            "int8_peak_tops": tp_alone["burst_x2"], "peak_source": tp_alone["used_source"],
                            "note": "index GEMMs alone (ResNet-18 layer4 3x3 and a square 8192^3), graph replay over rotated buffer sets"}
            line["sweep"] = sweep_compact(torch, cdl, hbm, max(3, min(args.steps, 40) // 4), n_x)
            if not args.no_network:
                torch.cuda.empty_cache()
                net = network_step(torch, cdl, 256, True, 5, 3)
                net.pop("clocks", None)
                line["network"] = net
                torch.cuda.empty_cache()
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline_block(case, host, quant_elems)
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
