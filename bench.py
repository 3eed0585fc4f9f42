#!/usr/bin/env python
"""Benchmark of the CDL quantized layer on B200.

A step is one pass of the whole hot path over one batch of synthetic input: quantize weights and activations
(soft value + hard index + histogram), entropy, forward index GEMM, quantize the arriving gradient, the two
backward index GEMMs, and the analytic quantizer backward for activations and weights.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl cdl|reference]

Prints ONE JSON line (rank 0).  `value` counts the tensor elements that went through a quantizer pass per
second of whole-step time, summed over ranks (each rank runs its own batch: weak scaling).
"""
from __future__ import annotations

import argparse
import json
import os
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
CPU_BASELINE_SECONDS = 20.0   # host time the cpu_baseline leg may spend (it samples the step to fit)
INT8_OVER_BF16 = 2.0         # nominal dense int8 : bf16 tensor throughput on B200 (4.5 : 2.25 PFLOP/s)
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel from an ncu capture, keyed by
# (workload, call); None until captured for the current kernel.
NCU_TRAFFIC_BYTES = {
    # profiles/index_gemm_tc_resnet18_layer3_conv.md: 13.5 MB read + 402.6 MB written while the kernel ran (the
    # write-back of the 462 MB output continues after it ends)
    ("resnet18_layer3_conv", "qlinear_bwd_dx"): 416.1e6,
}


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
    ap.add_argument("--no-graph", action="store_true", help="launch the calls of a step one by one instead of replaying a CUDA graph")
    ap.add_argument("--sweep", action="store_true",
                    help="quantizer-only bandwidth sweep (sizes x levels x alpha), one JSON line, 1 GPU")
    ap.add_argument("--sweep-max-log2n", type=int, default=28)
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
    import numpy as np
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


def run_implicit_conv(torch, cdl, CdlLayerStep, CALLS, case, step, q_g, steps, peaks_hbm, int8_tops):
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
    k_steps = min(steps, 200)
    events = [[torch.cuda.Event(enable_timing=True) for _ in range(len(CALLS) + 1)] for _ in range(k_steps)]
    for it in range(k_steps):
        ev = iter(events[it])
        cs.run(mark=lambda name: next(ev).record(stream))
    torch.cuda.synchronize()
    per = {name: sum(events[it][i].elapsed_time(events[it][i + 1]) for it in range(k_steps)) / k_steps
           for i, name in enumerate(CALLS)}
    model = conv_call_model(case, step.n_x)
    kern = {}
    for name in CALLS:
        m, t = model[name], per[name]
        k = {"ms": round(t, 5), "GBps": round(m["bytes"] / (t * 1e-3) / 1e9, 1)}
        if "ops" in m:
            k["int8_TOPS"] = round(m["ops"] / (t * 1e-3) / 1e12, 1)
            t_tensor, t_hbm = m["ops"] / (int8_tops * 1e12), m["bytes"] / (peaks_hbm * 1e9)
            k["bound"] = "tensor" if t_tensor >= t_hbm else "hbm"
            k["roofline_frac"] = round(max(t_tensor, t_hbm) / (t * 1e-3), 4)
        kern[name] = k
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
            "note": "same layer through cdl_qconv_fwd/bwd: no stored patch matrix, dX in the layout of x"}


def e2e_pipelined(torch, steps2, graphs2, pinned, out_host, e_steps, after_step=None):
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
            st.run()
        if after_step is not None:
            after_step(st)
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


def run_sweep(args):
    """Quantizer-only bandwidth sweep: fp32 tensors of 2^20 .. 2^max elements (50/50 N(0,1) / Laplace(0,1) mixture
    drawn on the device), L in {1,3,7,15,127}, alpha in {1,100,1e4}, step 4/L; hard, hard+hist, soft, soft+idx+hist,
    sampled index+hist, backward and backward+rate timed separately with CUDA events."""
    import torch

    import paper_2501_09849_b200 as cdl
    from paper_2501_09849_b200 import build as cdl_build
    cdl_build.build()
    cdl.load_library()
    torch.cuda.set_device(0)
    pk, pk_kind = peaks()
    hbm = float(pk["hbm_gbs"])
    gen = torch.Generator(device="cuda").manual_seed(5)
    grid_n = list(range(20, args.sweep_max_log2n + 1, 2))
    grid_L, grid_alpha = (1, 3, 7, 15, 127), (1.0, 100.0, 1e4)
    if args.sweep_point:
        grid_L, grid_alpha, grid_n = (int(args.sweep_point[0]),), (float(args.sweep_point[1]),), [int(args.sweep_point[2])]
        args.sweep_max_log2n = grid_n[0]
    nmax = 1 << args.sweep_max_log2n
    pick = torch.rand(nmax, device="cuda", generator=gen) < 0.5
    xn = torch.randn(nmax, device="cuda", generator=gen)
    u = torch.rand(nmax, device="cuda", generator=gen) - 0.5
    xl = -torch.sign(u) * torch.log1p(-2.0 * u.abs())           # Laplace(0,1) by inversion
    x = torch.where(pick, xn, xl).contiguous()
    del pick, xn, xl, u
    g = torch.randn(nmax, device="cuda", generator=gen)
    y = torch.empty(nmax, dtype=torch.float32, device="cuda")
    idx = torch.empty(nmax, dtype=torch.int8, device="cuda")
    s = torch.zeros(2, dtype=torch.float64, device="cuda")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()
    reps = max(3, args.steps // 4)

    def timed(make_fn, n):
        """Median time of one launch.  Launches are issued back to back on distinct slices of the big buffers
        (so that none finds its input in L2 and the CPU-side launch cost is hidden), one event pair around all."""
        k = max(1, min(16, nmax // n))
        fns = [make_fn(i * n) for i in range(k)]
        for f in fns[:2]:
            f()
        ts = []
        for _ in range(reps):
            if k * n * 12 < (512 << 20):
                flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for f in fns:
                f()
            e1.record(stream)
            e1.synchronize()
            ts.append(e0.elapsed_time(e1) / k)
        return statistics.median(ts)

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

                def mk(kind, PP=P):
                    def make(o):
                        xs, gs, ys, ix = x[o:o + n], g[o:o + n], y[o:o + n], idx[o:o + n]
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
                passes = {"hard": (5, mk("hard")), "hard_hist": (5, mk("hard_hist")), "soft": (8, mk("soft")),
                          "soft_idx_hist": (9, mk("soft_idx_hist")), "sample_hist": (5, mk("sample_hist")),
                          "backward": (12, mk("backward")),
                          "backward_rate": (12, mk("backward", Pr))}
                if alpha != grid_alpha[0]:
                    passes.pop("hard"), passes.pop("hard_hist")      # the hard passes do not depend on alpha
                for name, (bpe, make) in passes.items():
                    ms = timed(make, n)
                    gbs = n * bpe / (ms * 1e-3) / 1e9
                    rows.append({"log2n": log2n, "L": L, "alpha": alpha, "pass": name, "ms": round(ms, 4),
                                 "Gelem_per_s": round(n / (ms * 1e-3) / 1e9, 2), "GBps": round(gbs, 1),
                                 "hbm_frac_measured": round(gbs / hbm, 4), "hbm_frac_8TBps": round(gbs / 8000.0, 4)})
    print(json.dumps({"metric": METRIC, "unit": UNIT, "sweep": rows, "peak_hbm_gbs": hbm, "peak_source": pk_kind,
                      "data": "synthetic", "config": {"workload": "quantizer_sweep", "max_log2n": args.sweep_max_log2n}}),
          flush=True)


def run_gemm(args):
    """Index GEMMs alone: forward, dX and dW for each requested (M, K, N), 4-bit activation / weight indices and
    8-bit gradient indices drawn uniformly on the device, float outputs; operands are rotated over several
    buffer sets when one set would fit in L2."""
    import torch

    import paper_2501_09849_b200 as cdl
    from paper_2501_09849_b200 import build as cdl_build
    cdl_build.build()
    cdl.load_library()
    torch.cuda.set_device(0)
    pk, pk_kind = peaks()
    hbm = float(pk["hbm_gbs"])
    int8_tops = float(pk["bf16_tflops"]) * INT8_OVER_BF16          # kernels timed alone: burst figure
    stream = torch.cuda.current_stream()
    gen = torch.Generator(device="cuda").manual_seed(7)
    a, w, g = cdl.IndexDesc(0.25, 0, 15), cdl.IndexDesc(0.02, -7, 7), cdl.IndexDesc(1e-3, -127, 127)
    out = []
    for M, K, N in args.gemm:
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
            # one pass over the buffer sets recorded as a graph: calls of a few microseconds would otherwise be
            # timed by the host's launch path, not by the device
            torch.cuda.synchronize()
            side = torch.cuda.Stream()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.stream(side):
                with torch.cuda.graph(graph, stream=side):
                    for t in sets:
                        fn(t)
            rounds = max(2, min(40, args.steps) // nset)
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
            t_tensor, t_hbm = ops / (int8_tops * 1e12), bytes_[name] / (hbm * 1e9)
            row[name] = {"ms": round(ms, 5), "int8_TOPS": round(ops / (ms * 1e-3) / 1e12, 1),
                         "int8_frac_of_peak": round(ops / (ms * 1e-3) / 1e12 / int8_tops, 4),
                         "GBps": round(bytes_[name] / (ms * 1e-3) / 1e9, 1), "bound": "tensor" if t_tensor >= t_hbm else "hbm",
                         "roofline_frac": round(max(t_tensor, t_hbm) / (ms * 1e-3), 4)}
        row["status"] = cdl.cdl_workspace_status(ws, check=False)
        out.append(row)
        del sets
    print(json.dumps({"metric": METRIC, "unit": "int8 TOPS", "gemm": out, "int8_peak_tops": int8_tops,
                      "peak_source": f"{pk_kind} burst bf16 x {INT8_OVER_BF16:g} (nominal int8:bf16)", "peak_hbm_gbs": hbm,
                      "data": "synthetic", "config": {"workload": "index_gemm"}}), flush=True)


def run_network(args):
    """Whole ResNet-18 (224x224) as a sequence of CDL layer steps: every conv and the FC layer with its true im2col
    GEMM shape, 3-bit weights (step = std(w) / 3), 4-bit activations (step from the mean magnitude), window of 5.
    Inputs are drawn on the device (seeded); each layer owns its buffers, so a step touches ~40 GB at batch 256."""
    import torch

    import paper_2501_09849_b200 as cdl
    from paper_2501_09849_b200 import build as cdl_build
    from paper_2501_09849_b200 import inputs
    from paper_2501_09849_b200.layer import CALLS, CdlLayerStep
    cdl_build.build()
    cdl.load_library()
    torch.cuda.set_device(0)
    gen = torch.Generator(device="cuda").manual_seed(4)
    stream = torch.cuda.current_stream()
    q_g = 4.0 * G_STD / 127.0
    layers = []
    for name, M, K, N, n_x in inputs.resnet18_layers(args.batch):
        Np = (N + 15) // 16 * 16                  # index matrices need 16-byte row pitches: fc's 1000 columns -> 1008
        w = torch.randn(K * Np, device="cuda", generator=gen) * (2.0 / K) ** 0.5
        x = torch.randn(n_x, device="cuda", generator=gen).abs_()
        wq = inputs.Quantizer(float(w.std()) / 3.0, -3, 3, 100.0, 0.01, 0)
        xq = inputs.Quantizer(float(2.0 * x.mean() / 8.0 ** 0.5), 0, 15, 100.0, 0.01, 5)
        geo = inputs.resnet18_conv_geometry(name) if args.conv_form else None
        shape = cdl.ConvShape(args.batch, geo[0], geo[1], geo[2], geo[3], geo[4]) if geo else None
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

    warm = max(3, min(args.warmup, 5))
    steps = max(3, min(args.steps, 20))
    for _ in range(warm):
        run_all()
    torch.cuda.synchronize()
    # the whole network step as one CUDA graph (each layer recorded on three streams), replayed `steps` times
    graph = None
    if not args.no_graph:
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
    ev = [[[torch.cuda.Event(enable_timing=True) for _ in range(len(CALLS) + 1)] for _ in layers] for _ in range(steps)]
    cnt = {}
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(0)
    sampler.start()
    time.sleep(0.3)
    wall0 = time.time()
    t0.record(stream)
    for it in range(steps):
        cnt.clear()

        def mark(li, nm, it=it):
            i = cnt.get(li, 0)
            ev[it][li][i].record(stream)
            cnt[li] = i + 1
        run_all(mark)
    t1.record(stream)
    torch.cuda.synchronize()
    clocks = sampler.stop(wall0, time.time())
    ms_step = t0.elapsed_time(t1) / steps
    call_by_call_ms = ms_step
    if graph is not None:
        ms_step = graph_ms
    pk, pk_kind = peaks()
    hbm = float(pk["hbm_gbs"])
    table, tot_ops, tot_q, gemm_ms, quant_ms = [], 0.0, 0, 0.0, 0.0
    for li, (name, M, K, N, n_x, st) in enumerate(layers):
        per = {c: sum(ev[it][li][i].elapsed_time(ev[it][li][i + 1]) for it in range(steps)) / steps for i, c in enumerate(CALLS)}
        g_ms = per["qlinear_fwd"] + per["qlinear_bwd_dx"] + per["qlinear_bwd_dw"]
        q_ms = sum(v for c, v in per.items() if c.startswith("quantize"))
        ops = (6.0 if st.need_dx else 4.0) * M * K * N
        q_el = 2 * (n_x + K * N) + M * N
        table.append({"layer": name, "M": M, "K": K, "N": N, "ms": round(sum(per.values()), 4), "gemm_ms": round(g_ms, 4),
                      "gemm_int8_TOPS": round(ops / (g_ms * 1e-3) / 1e12, 1), "quantizer_ms": round(q_ms, 4),
                      "quantizer_Gelem_per_s": round(q_el / (q_ms * 1e-3) / 1e9, 1),
                      "calls_us": {c: round(v * 1e3, 1) for c, v in per.items()},
                      "status": cdl.cdl_workspace_status(st.ws, check=False)})
        tot_ops += ops
        tot_q += q_el
        gemm_ms += g_ms
        quant_ms += q_ms
    print(json.dumps({
        "metric": METRIC, "value": tot_q / (ms_step * 1e-3) / 1e9, "unit": UNIT, "n_gpus": 1, "steps": steps, "warmup": warm,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32+s8",
        "data": "synthetic",
        "config": {"workload": "resnet18_b256", "batch": args.batch, "layers": len(layers),
                   "form": ("convolution form for the %d stride-1 3x3 layers, stored patch matrices "
                            "for the rest" % sum(1 for *_, st in layers if st.conv is not None)) if args.conv_form
                   else "stored patch matrices (im2col GEMMs)",
                   "launch": "stream launches" if graph is None else "CUDA graph replay of the network step",
                   "call_by_call_ms": call_by_call_ms, "weight_levels": 7,
                   "activation_levels": 16, "window_x": 5, "l2": "every layer's tensors exceed the 126 MB L2"},
        "network_fwd_bwd_ms": ms_step, "gemm_ms": gemm_ms, "gemm_int8_tops": tot_ops / (gemm_ms * 1e-3) / 1e12,
        "quantizer_ms": quant_ms, "quantizer_Gelem_per_s": tot_q / (quant_ms * 1e-3) / 1e9,
        "layers": table, "clocks": clocks, "peak_hbm_gbs": hbm, "peak_source": pk_kind,
        "e2e": None, "e2e_note": "not measured for this workload (a step's inputs are ~11 GB); see the default workload",
        "gpu_launches": steps * sum(st.kernels_per_step() for *_, st in layers)}), flush=True)


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

    # ---- inputs: seeded, host-generated, one independent batch per rank (weak scaling)
    case, w, x = make_case(args.workload, seed_offset=100 * rank)
    M, K, N, n_x = case.M, case.K, case.N, x.size
    q_g = float(np.float32(4.0 * G_STD / 127.0))
    step = CdlLayerStep(torch, M, K, N, n_x, case.wq, case.aq, q_g)
    xd = torch.from_numpy(x.reshape(-1)).cuda()
    hist = torch.zeros(case.aq.nlev, dtype=torch.int64, device="cuda")
    cdl.cdl_quantize_hard(xd, n_x, cdl.QuantParams(case.aq.q, case.aq.lo, case.aq.hi), None, hist)
    host = host_inputs(case, w, x, hist.cpu().numpy().view(np.uint64))
    pinned = {k: torch.from_numpy(np.ascontiguousarray(v)).pin_memory() for k, v in host.items()}
    dev_in = step.input_tensors()
    for k, t in dev_in.items():
        t.copy_(pinned[k].view(t.shape), non_blocking=True)
    torch.cuda.synchronize()
    stream = torch.cuda.current_stream()

    def exchange():
        # data-parallel exchange of a step: the weight-side results are sums over the global batch
        sharding.exchange(dist, world, step.dW, step.hist_x, step.scalars)

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    for _ in range(max(args.warmup, 3)):
        step.run()
        exchange()
    torch.cuda.synchronize()

    # ---- timed region: device-resident inputs, the step replayed from a CUDA graph (launch gaps between the ten
    # short kernels of a step are a tenth of its time when they are launched one by one)
    graph = step.capture() if not args.no_graph else None
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
            step.run()
        exchange()
    t_end.record(stream)
    torch.cuda.synchronize()
    wall1 = time.time()
    if world > 1:
        dist.barrier()
    clocks = sampler.stop(wall0, wall1) if rank == 0 else None
    total_ms = t_start.elapsed_time(t_end)

    # ---- per-call times: a second pass over the same steps, launched call by call with an event between calls
    k_steps = min(args.steps, 500)
    events = [[torch.cuda.Event(enable_timing=True) for _ in range(len(CALLS) + 1)] for _ in range(k_steps)]
    for it in range(k_steps):
        ev = iter(events[it])
        step.run(mark=lambda name: next(ev).record(stream))
        exchange()
    torch.cuda.synchronize()
    per_call_ms = {name: sum(events[it][i].elapsed_time(events[it][i + 1]) for it in range(k_steps)) / k_steps
                   for i, name in enumerate(CALLS)}
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
    step_b.run()
    graph_b = step_b.capture() if graph is not None else None
    if world > 1:
        dist.barrier()
    e2e_ms = e2e_pipelined(torch, (step, step_b), (graph, graph_b), pinned, out_host, e_steps,
                           after_step=(lambda st: sharding.exchange(dist, world, st.dW, st.hist_x, st.scalars)) if world > 1 else None)
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
        int8_tops = float(pk.get("bf16_tflops_sustained", pk["bf16_tflops"])) * INT8_OVER_BF16
        kernels = {}
        for name in CALLS:
            m, ms = model[name], per_call_ms[name]
            k = {"ms": round(ms, 5), "GBps": round(m["bytes"] / (ms * 1e-3) / 1e9, 1)}
            if m["elems"]:
                k["Gelem_per_s"] = round(m["elems"] / (ms * 1e-3) / 1e9, 2)
                k["hbm_frac_measured"] = round(k["GBps"] / hbm, 4)
                k["hbm_frac_8TBps"] = round(k["GBps"] / 8000.0, 4)
            if "ops" in m:
                k["int8_TOPS"] = round(m["ops"] / (ms * 1e-3) / 1e12, 1)
                t_tensor, t_hbm = m["ops"] / (int8_tops * 1e12), m["bytes"] / (hbm * 1e9)
                k["bound"] = "tensor" if t_tensor >= t_hbm else "hbm"
                k["roofline_frac"] = round(max(t_tensor, t_hbm) / (ms * 1e-3), 4)
            kernels[name] = k
        dom = max(CALLS, key=lambda c: per_call_ms[c])
        dm, dms = model[dom], per_call_ms[dom]
        if "ops" in dm and dm["ops"] / (int8_tops * 1e12) >= dm["bytes"] / (hbm * 1e9):
            roof = {"kernel": dom, "bound": "tensor", "achieved": dm["ops"] / (dms * 1e-3) / 1e12, "peak": int8_tops,
                    "unit": "TFLOP/s", "peak_source": f"{pk_kind} sustained bf16 x {INT8_OVER_BF16:g} (nominal int8:bf16)"}
        else:
            roof = {"kernel": dom, "bound": "hbm", "achieved": dm["bytes"] / (dms * 1e-3) / 1e9, "peak": hbm,
                    "unit": "GB/s", "peak_source": f"{pk_kind} copy bandwidth"}
        roof["frac"] = roof["achieved"] / roof["peak"]
        roof["traffic"] = NCU_TRAFFIC_BYTES.get((args.workload, dom))
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
                       "parallelism": f"replicas x{world}, all-reduce of dW / histogram / scalars" if world > 1 else "single GPU"},
            "layer_fwd_bwd_ms": ms_step, "gemm_ms": gemm_ms, "gemm_int8_tops": 6.0 * M * K * N / (gemm_ms * 1e-3) / 1e12,
            "quantizer_ms": quant_ms, "quantizer_Gelem_per_s": quant_elems / (quant_ms * 1e-3) / 1e9,
            "quantizer_hbm_frac_measured": sum(model[c]["bytes"] for c in CALLS if model[c]["elems"]) / (quant_ms * 1e-3) / 1e9 / hbm,
            "kernels": kernels, "roofline": roof, "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": UNIT, "ms_per_step": e2e_ms, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "steps": e_steps,
                    "overlap": "two sets of device buffers: the copy of step i+1 overlaps the kernels of step i"},
            "gpu_launches": args.steps * step.kernels_per_step(), "device_status": status,
            "launch": "stream launches" if graph is None else "CUDA graph replay of one step",
            "kernel_timing": f"second pass of {k_steps} steps launched call by call, one CUDA event between calls",
        }
        if world == 1 and args.workload == "resnet18_layer3_conv" and not args.no_implicit:
            line["implicit_conv"] = run_implicit_conv(torch, cdl, CdlLayerStep, CALLS, case, step, q_g, args.steps, hbm, int8_tops)
        if world == 1 and not args.no_cpu_baseline:
            import oracle
            oracle.build()
            t_cpu, desc, thr, _ = oracle_step_sample(case, host, frac=min(1.0, CPU_BASELINE_SECONDS / max(256.0 * oracle_step_sample(case, host, 1.0 / 256)[3], 1e-9)))
            line["cpu_baseline"] = {"value": quant_elems / t_cpu / 1e9, "unit": UNIT, "cores": thr, "kind": "oracle",
                                    "sample": desc, "ms_per_step_estimate": t_cpu * 1e3}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
