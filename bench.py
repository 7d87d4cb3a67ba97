#!/usr/bin/env python
"""Benchmark of the FP4 Direct-P attention forward hot path on B200.

One step = one pass of the whole hot path over one batch: quantize Q, K (MXFP4 or NVFP4) and V
(MXFP4, transposed) + the attention forward.  Prints ONE JSON line on rank 0.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg5_N32768] [--impl reference]

Default workload: the longest point of the sequence sweep (B=1, H=16, N=32768, d=128, MXFP4 operands), the
largest single-GPU configuration and inside the N >= 8K range the metric is stated for.  The other
configurations are timed (attention launch alone) as sub-records with a roofline fraction of their own.

Timing protocol: at least W steps and 300 ms of warm-up; then EXACTLY K steps, each bracketed by CUDA events
after an L2 flush (`value`, `ms_per_step`, `roofline.achieved` come from these); then a window of at least
`--window-s` seconds of further steps whose per-launch MEDIANS, SM clock and power are reported under
`window` (the paper's protocol is 300 ms warm-up and a median over a seconds-long window), with a
clock-normalised figure beside the raw one.

Rooflines: `roofline` holds the attention kernel against the tensor roof (measured bf16 burst x 4);
`roofline_softmax_arith` holds the same kernel against what its softmax arithmetic alone allows on this device
(the kernel's score -> code instruction stream run by itself, four warps per scheduler: with exact codes the
special-function unit binds it); `roofline_quantize` the quantizers against the measured copy bandwidth.

N > 1 is launched with torch.distributed.run (one rank per GPU); every rank runs the same
workload on its own batch (independent (batch, head) units, no data-path collective), so the
job is weak-scaled and `value` is the sum over ranks divided by the slowest rank's time.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2609_04105_b200 import inputs as I  # noqa: E402

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the attention kernel (exact map), from one ncu
# capture per workload; part of O is still in L2 when the kernel ends, so the figure can be below the
# algorithmic bytes.  Workloads without a capture report null.
NCU_TRAFFIC_BYTES = {
    "cfg2": {"attn": 53.5e6 + 24.2e6, "quant_rows": 67.12e6 + 3.08e6},
    "cfg3": {"attn": 114.6e6 + 97.6e6},
    "cfg4": {"attn": 107.3e6 + 95.9e6},
    "cfg5_N32768": {"attn": 107.4e6 + 96.0e6},
}

METRIC = "fp4_attention_fwd_tflops"
UNIT = "TFLOP/s"
NOMINAL_FP4_OVER_BF16 = 4.0          # dense 9 PFLOP/s fp4 : 2.25 PFLOP/s bf16
DEFAULT_WORKLOAD = "cfg5_N32768"
SUB_RECORDS = ("cfg5_N8192", "cfg5_N16384", "cfg4", "cfg3", "cfg3_N32768", "cfg2", "cfg5_N4096", "cfg5_N2048", "cfg5_N1024")


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained"), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def _workload_text(w):
    fmt = "MXFP4 Q,K,P,V" if w.qk_fmt == I.FMT_MXFP4 else "NVFP4 Q,K + MXFP4 P,V"
    return f"{w.name}: B={w.B},H={w.H},N={w.N},d={w.d}, noncausal, {fmt}" + (", outlier channels x20" if w.outliers else "")


# ----------------------------------------------------------------------------- clocks and power
class ClockSampler:
    """Samples SM clock, board power and throttle reasons of one GPU through NVML (read-only) while running."""

    def __init__(self, index: int, period_s: float = 0.002):
        self.index, self.period, self.samples, self.power, self.reasons = index, period_s, [], [], set()
        self.max_mhz, self._stop, self._thr = None, threading.Event(), None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
        }
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    self.power.append(nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0)
                except Exception:
                    pass
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def __enter__(self):
        if self.nv is not None:
            self._thr = threading.Thread(target=self._run, daemon=True)
            self._thr.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thr is not None:
            self._thr.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["unavailable"]}
        out = {"sm_mhz": statistics.median(self.samples), "sm_max_mhz": self.max_mhz,
               "sm_mhz_min": min(self.samples), "reasons": sorted(self.reasons), "samples": len(self.samples)}
        if self.power:
            out["power_w_median"] = statistics.median(self.power)
            out["power_w_max"] = max(self.power)
        return out


def _nvml_index(local: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES", "")
    ids = [t for t in vis.split(",") if t.strip()]
    if ids and all(t.strip().isdigit() for t in ids) and local < len(ids):
        return int(ids[local])
    return local


# ----------------------------------------------------------------------------- oracle legs
def _blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return None


def _host_cores():
    return len(os.sched_getaffinity(0))


HYBRID_PATTERNS = {"hybrid4": 0x1111, "hybrid8": 0x5555, "hybrid12": 0x7777}     # exact element pairs of 16


def oracle_operands_of_heads(w, q, k, v, amax_qk=None):
    """Oracle quantization of the (batch, head) units in `heads` (bf16 bit arrays q, k, v hold exactly these units,
    [1, n, N, d]).  NVFP4 takes the tensor-wide maxima `amax_qk` (the encode factor belongs to the whole tensor)."""
    from oracle import quantize as Qz
    if w.qk_fmt == I.FMT_NVFP4:
        Gq = Qz.nv_tensor_scale(np.asarray([amax_qk[0]], np.float64))
        Gk = Qz.nv_tensor_scale(np.asarray([amax_qk[1]], np.float64))
        nq, sq = Qz.nv_quantize_lastdim(Qz.bf16_bits_to_f64(q), Gq)
        nk, sk = Qz.nv_quantize_lastdim(Qz.bf16_bits_to_f64(k), Gk)
        qd = {"nib": nq, "sf": sq, "G": Gq, "fmt": "nv"}
        kd = {"nib": nk, "sf": sk, "G": Gk, "fmt": "nv"}
    else:
        qd, kd = Qz.quantize_qk(q, "mx"), Qz.quantize_qk(k, "mx")
    return qd, kd, Qz.quantize_v(v)


def oracle_sample(w, q, k, v, n_heads, rows, p_map="ideal", p_scale="ceil", amax_qk=None, fixed_reference=None):
    """Runs the oracle (as it stands) on a bounded sample: `n_heads` units (held by q, k, v) and the given query
    rows.  Returns seconds, equivalent TFLOP/s, its outputs and the quantized operands."""
    from oracle import attention as A
    t0 = time.perf_counter()
    qd, kd, vd = oracle_operands_of_heads(w, q, k, v, amax_qk)
    okw = dict(p_map="hybrid", exact_pairs=HYBRID_PATTERNS[p_map]) if p_map in HYBRID_PATTERNS else dict(p_map=p_map)
    O, lse = A.direct_p_forward(qd, kd, vd, rows=rows, heads=[(0, i) for i in range(n_heads)], p_scale=p_scale,
                                fixed_reference=fixed_reference, **okw)
    dt = time.perf_counter() - t0
    n_rows = w.N if rows is None else len(rows)
    flops = 4.0 * n_heads * n_rows * w.N * w.d
    return dt, flops / dt / 1e12, O, lse, (qd, kd, vd)


def accuracy_vs_fp64(q, k, v, ops, rows, O_gpu, O_oracle, O_gpu_fp8=None):
    """cos / rel-L2 against unquantised fp64 attention of: the CUDA path, the oracle, and O_exactP (quantised
    Q, K, V with an exact softmax - what is left when P is not quantised)."""
    from oracle import attention as A
    from oracle import quantize as Qz
    keys = ("gpu", "oracle", "exact_p") + (("gpu_fp8_pv", "oracle_fp8_pv") if O_gpu_fp8 is not None else ())
    num = {key: [0.0, 0.0, 0.0, 0.0] for key in keys}
    v8 = Qz.quantize_v_e4m3(v) if O_gpu_fp8 is not None else None
    for n in range(q.shape[1]):
        x = [Qz.bf16_bits_to_f64(a[0, n]) for a in (q, k, v)]
        Oe, _ = A.exact_attention(x[0], x[1], x[2], rows=rows)
        Op, _ = A.exact_p_attention(ops[0], ops[1], ops[2], 0, n, rows=rows)
        outs = [("gpu", O_gpu[n]), ("oracle", O_oracle[n]), ("exact_p", Op)]
        if O_gpu_fp8 is not None:
            O8, _ = A.fp8_pv_forward(ops[0], ops[1], v8, rows=rows, heads=[(0, n)])
            outs += [("gpu_fp8_pv", O_gpu_fp8[n]), ("oracle_fp8_pv", O8[0])]
        for key, O in outs:
            acc = num[key]
            acc[0] += (O * Oe).sum(); acc[1] += (O * O).sum(); acc[2] += (Oe * Oe).sum(); acc[3] += ((O - Oe) ** 2).sum()
    out = {}
    for key, (dot, oo, ee, dd) in num.items():
        out[key] = {"cos": float(dot / np.sqrt(oo * ee)), "rel_l2": float(np.sqrt(dd / ee))}
    return out


def run_reference(args, w):
    """`--impl reference`: the oracle timed on the host cores, one bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    n_rows = min(w.N, 512)
    rng = np.random.default_rng(7)
    rows = np.sort(rng.choice(w.N, size=n_rows, replace=False))
    amax = None
    if w.qk_fmt == I.FMT_MXFP4:
        # the seeded streams fill [B, H, N, d] in order, so unit (0, 0) of the full tensors is the one-unit draw
        q, k, v = I.make_qkv(I.shrink(w, B=1, H=1))
    else:
        qf, kf, vf = I.make_qkv(w)
        bf = lambda a: I.bf16_bits_to_f32(a)
        amax = (float(np.abs(bf(qf)).max()), float(np.abs(bf(kf)).max()))
        q, k, v = (np.ascontiguousarray(a[:1, :1]) for a in (qf, kf, vf))
    for _ in range(args.warmup):
        oracle_sample(w, q, k, v, 1, rows, amax_qk=amax)
    times = []
    for _ in range(args.steps):
        times.append(oracle_sample(w, q, k, v, 1, rows, amax_qk=amax)[0])
    flops = 4.0 * len(rows) * w.N * w.d
    total = sum(times)
    value = flops * len(times) / total / 1e12
    sample = f"1 (batch, head) unit x {len(rows)} seeded query rows of {w.name} per step (rows are independent)"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / len(times),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": {"workload": _workload_text(w), "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": _host_cores(), "blas_threads": _blas_threads(),
                         "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ----------------------------------------------------------------------------- CUDA arm
def device_qkv(w, dev):
    """The seeded recipe on the device: the float32 draws are made on the host (three streams, three threads),
    copied over and rounded to bfloat16 there (round to nearest even, the same bits as the host rounding of
    inputs.make_qkv; a GPU test pins that)."""
    import torch
    out = [None, None, None]

    def work(t):
        out[t] = I.make_operand_f32(w, t)

    th = [threading.Thread(target=work, args=(t,)) for t in range(3)]
    for t in th:
        t.start()
    for t in th:
        t.join()
    return [torch.from_numpy(x).to(dev).to(torch.bfloat16) for x in out]


def _bits(t):
    """CUDA / CPU bf16 tensor -> uint16 bit array on the host."""
    import torch
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def timed_launches(fn, n, flush, E, sync):
    """Milliseconds of n calls of fn, each timed by its own pair of CUDA events after an L2 flush."""
    pairs = [(E(), E()) for _ in range(n)]
    for i, (a, b) in enumerate(pairs):
        flush.fill_(i & 0xFF)
        a.record()
        fn()
        b.record()
    sync()
    return [a.elapsed_time(b) for a, b in pairs]


def roofline_record(w, ms, fp4_peak, peaks, kernel="attn_fwd_kernel"):
    tf = w.flops / (ms * 1e-3) / 1e12
    return {"kernel": kernel, "bound": "tensor", "achieved": tf, "peak": fp4_peak, "unit": "TFLOP/s",
            "frac": tf / fp4_peak, "traffic": NCU_TRAFFIC_BYTES.get(w.name, {}).get("attn"),
            "peak_source": f"{peaks['source']} bf16 burst {peaks['bf16_tflops']} TFLOP/s x nominal fp4:bf16 ratio 4"}


def run_cuda(args, w):
    import torch
    import torch.distributed as dist
    from paper_2609_04105_b200 import binding as Bd, build

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        build.build()
    if world > 1:
        dist.barrier()
    Bd.lib()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    peaks = _peaks()
    fp4_peak = peaks["bf16_tflops"] * NOMINAL_FP4_OVER_BF16
    dq, dk, dv = device_qkv(w, dev)
    B, H, N, d = w.B, w.H, w.N, w.d
    O = torch.empty((B, H, N, d), dtype=torch.bfloat16, device=dev)
    lse = torch.empty((B, H, N), dtype=torch.float32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    qws = torch.empty(max(16, Bd.lib().fp4attn_quantize_workspace_bytes(w.qk_fmt, 0, B, H, N, d)), dtype=torch.uint8, device=dev)
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)      # > 126 MB L2
    launches_per_step = 4 if w.qk_fmt == I.FMT_MXFP4 else 8          # NVFP4: amax pass + encode factor + codes, for Q and for K
    pmap = Bd.PMAP_AFFINE if args.p_map == "affine" else Bd.PMAP_HYBRID if args.p_map in HYBRID_PATTERNS else Bd.PMAP_IDEAL
    pairs = HYBRID_PATTERNS.get(args.p_map, 0)
    pscale = {"thr16": Bd.PSCALE_THR16, "mse": Bd.PSCALE_MSE}.get(args.p_scale, Bd.PSCALE_CEIL)
    sched = Bd.SCHEDULE_TWO_QUERY if args.schedule == "two-query" else Bd.SCHEDULE_ONE_QUERY
    state = {}
    E = lambda: torch.cuda.Event(enable_timing=True)

    def step(ev=None):
        qd = Bd.fp4attn_quantize(dq, w.qk_fmt, Bd.ROLE_Q, qws)
        kd = Bd.fp4attn_quantize(dk, w.qk_fmt, Bd.ROLE_K, qws)
        vd = Bd.fp4attn_quantize(dv, Bd.FMT_MXFP4, Bd.ROLE_V)
        if ev is not None:
            ev[0].record()
        Bd.fp4attn_fwd(qd, kd, vd, out=O, lse=lse, status=status, p_map=pmap, p_scale_rule=pscale, exact_pairs=pairs,
                       schedule=sched, fixed_reference=args.fixed_reference)
        if ev is not None:
            ev[1].record()
        state["ops"] = (qd, kd, vd)

    def run_timed(n):
        ev_step = [(E(), E()) for _ in range(n)]
        ev_attn = [(E(), E()) for _ in range(n)]
        for i in range(n):
            flush.fill_(i & 0xFF)                                   # evict L2 (outside the step's events)
            ev_step[i][0].record()
            step(ev_attn[i])
            ev_step[i][1].record()
        barrier()
        return [a.elapsed_time(b) for a, b in ev_step], [a.elapsed_time(b) for a, b in ev_attn]

    # ---- warm-up: at least W steps and at least 300 ms
    n_warm, t0 = 0, time.perf_counter()
    while n_warm < max(args.warmup, 3) or time.perf_counter() - t0 < 0.3:
        step()
        n_warm += 1
        if n_warm % 8 == 0:
            torch.cuda.synchronize()
    barrier()

    # ---- the timed region: exactly K steps
    with ClockSampler(_nvml_index(local)) as clk:
        barrier()
        step_ms, attn_ms = run_timed(args.steps)
    assert int(status.item()) == 0, "attention kernel reported a bounded-wait timeout"
    total_ms = sum(step_ms)
    t = torch.tensor([total_ms, sum(attn_ms)], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    total_ms, attn_total_ms = float(t[0]), float(t[1])
    value = world * w.flops * args.steps / (total_ms * 1e-3) / 1e12
    attn_tflops = w.flops * args.steps / (attn_total_ms * 1e-3) / 1e12
    attn_launch_ms = attn_total_ms / args.steps

    # ---- a seconds-long window of further steps: medians, clocks and power in the sustained regime
    window = None
    if args.window_s > 0:
        n_win = int(min(5000, max(20, math.ceil(args.window_s * 1e3 / statistics.median(step_ms)))))
        with ClockSampler(_nvml_index(local)) as wclk:
            barrier()
            w_step, w_attn = run_timed(n_win)
        wc = wclk.summary()
        med_attn, med_step = statistics.median(w_attn), statistics.median(w_step)
        srt = sorted(w_attn)
        window = {"steps": n_win, "seconds_in_steps": sum(w_step) * 1e-3, "step_ms_median": med_step, "attn_ms_median": med_attn,
                  "attn_ms_p10": srt[len(srt) // 10], "attn_ms_p90": srt[(9 * len(srt)) // 10],
                  "value_median": w.flops / (med_step * 1e-3) / 1e12, "attn_tflops_median": w.flops / (med_attn * 1e-3) / 1e12,
                  "roofline_frac_median": w.flops / (med_attn * 1e-3) / 1e12 / fp4_peak, "clocks": wc}
        if wc.get("sm_mhz"):
            # the same launch at another SM clock takes time in inverse proportion while it is not memory-bound:
            # time x clock is the clock-independent figure
            window["clock_normalised"] = {"attn_ms_x_ghz": med_attn * wc["sm_mhz"] / 1e3,
                                          "attn_tflops_at_max_clock": w.flops / (med_attn * 1e-3) / 1e12 * wc["sm_max_mhz"] / wc["sm_mhz"]}

    # ---- quantizer alone (kernel a), HBM roofline of its dominant launch (the rows kernel): twelve launches
    # replayed from a CUDA graph, so that the figure is the kernels' time and not the Python call overhead;
    # the launches rotate over the Q, K and V tensors (each > L2), so no launch finds its input in L2
    qgraph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        Bd.fp4attn_quantize(dq, w.qk_fmt, Bd.ROLE_Q, qws)
        Bd.fp4attn_quantize(dv, Bd.FMT_MXFP4, Bd.ROLE_V)
    torch.cuda.current_stream().wait_stream(side)
    quant = {}
    for key, role, fmt in (("rows", Bd.ROLE_Q, w.qk_fmt), ("v", Bd.ROLE_V, Bd.FMT_MXFP4)):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for r in range(12):
                state["q_only"] = Bd.fp4attn_quantize((dq, dk, dv)[r % 3], fmt, role, qws)
        qb = [E(), E()]
        g.replay()
        flush.fill_(1)
        qb[0].record()
        g.replay()
        qb[1].record()
        torch.cuda.synchronize()
        quant[key] = qb[0].elapsed_time(qb[1]) / 12
        del g
    # algorithmic bytes per element: bf16 in, 4-bit codes and scale bytes out; NVFP4 reads the tensor twice
    q_bpe = (2 + 0.5 + 1.0 / 32) if w.qk_fmt == I.FMT_MXFP4 else (2 + 2 + 0.5 + 1.0 / 16)
    q_kernel = "quant_mx_rows_kernel" if w.qk_fmt == I.FMT_MXFP4 else "amax_partials_kernel + nv_encode_factor_kernel + quant_nv_rows_kernel"
    q_bytes = B * H * N * d * q_bpe
    v_bytes = B * H * N * d * (2 + 0.5 + 1.0 / 32)

    # ---- end to end through the host-buffer entry point (pinned host in, host out)
    hq, hk, hv = (t.cpu().pin_memory() for t in (dq, dk, dv))
    ho = torch.empty((B, H, N, d), dtype=torch.bfloat16).pin_memory()
    hl = torch.empty((B, H, N), dtype=torch.float32).pin_memory()
    ws = torch.empty(Bd.fp4attn_attention_host_workspace_bytes(w.qk_fmt, B, H, N, d), dtype=torch.uint8, device=dev)
    e2e_steps = max(3, min(args.steps, 20))
    for _ in range(2):
        Bd.fp4attn_attention_host(hq, hk, hv, w.qk_fmt, ho, hl, ws)
    barrier()
    e0, e1 = E(), E()
    e0.record()
    for _ in range(e2e_steps):
        Bd.fp4attn_attention_host(hq, hk, hv, w.qk_fmt, ho, hl, ws)
    e1.record()
    barrier()
    e2e_ms = torch.tensor([e0.elapsed_time(e1)], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(e2e_ms, op=dist.ReduceOp.MAX)
    e2e_value = world * w.flops * e2e_steps / (float(e2e_ms[0]) * 1e-3) / 1e12
    h2d = 3 * B * H * N * d * 2
    d2h = B * H * N * d * 2 + B * H * N * 4
    del hq, hk, hv, ho, hl, ws

    # ---- the same workload's attention launch under the other code maps (context beside the timed map)
    other_maps = {}
    if world == 1:
        qd0, kd0, vd0 = state["ops"]
        O_alt = torch.empty_like(O)                                 # O keeps the timed map's result for the parity sample
        for name, kw in (("ideal", dict(p_map=Bd.PMAP_IDEAL)), ("hybrid8", dict(p_map=Bd.PMAP_HYBRID, exact_pairs=0x5555)),
                         ("affine", dict(p_map=Bd.PMAP_AFFINE)),
                         ("affine_shiftless", dict(p_map=Bd.PMAP_AFFINE, fixed_reference=0))):
            if name == args.p_map or ("fixed_reference" in kw and w.outliers):     # (outlier logits span more than a fixed reference holds)
                continue
            rule = pscale if (pscale != Bd.PSCALE_MSE or name == "ideal") else Bd.PSCALE_CEIL     # the MSE rule exists for the ideal map
            if "fixed_reference" in kw:
                rule = Bd.PSCALE_CEIL                                # the fixed reference comes with the ceiling rule
            fn = lambda: Bd.fp4attn_fwd(qd0, kd0, vd0, out=O_alt, status=status, p_scale_rule=rule, **kw)
            for _ in range(3):
                fn()
            ms_map = statistics.median(timed_launches(fn, 10, flush, E, torch.cuda.synchronize))
            cyc_m = torch.zeros(2, dtype=torch.int64, device=dev)
            Bd.fp4attn_softmax_arith_probe(kw["p_map"], kw.get("exact_pairs", 0), 8192, cyc_m)
            torch.cuda.synchronize()
            other_maps[name] = {"attn_ms": ms_map, "attn_tflops": w.flops / (ms_map * 1e-3) / 1e12,
                                "roofline_frac": w.flops / (ms_map * 1e-3) / 1e12 / fp4_peak,
                                "softmax_arith_clk_per_block": int(cyc_m[0].item()) / (4.0 * 8192)}
        # the FP8 P/V route on the same Q, K (E4M3 V with per-unit factors, E4M3 probabilities)
        v8 = Bd.fp4attn_quantize_v_e4m3(dv)
        fn = lambda: Bd.fp4attn_fwd(qd0, kd0, v8, out=O_alt, status=status)
        for _ in range(3):
            fn()
        ms_map = statistics.median(timed_launches(fn, 10, flush, E, torch.cuda.synchronize))
        other_maps["fp8_pv"] = {"attn_ms": ms_map, "attn_tflops": w.flops / (ms_map * 1e-3) / 1e12,
                                "roofline_frac": w.flops / (ms_map * 1e-3) / 1e12 / fp4_peak,
                                "note": "kind::f8f6f4 second product; its own denominator would be the FP8 roof, half the FP4 one"}
        state["O_fp8"] = O_alt
        del v8

    # ---- measured dense FP4 issue rate of this device (context for the roofline)
    cyc = torch.zeros(1, dtype=torch.int64, device=dev)
    iters = 20000
    Bd.fp4attn_mma_peak_probe(iters, cyc)
    p0, p1 = E(), E()
    p0.record()
    Bd.fp4attn_mma_peak_probe(iters, cyc)
    p1.record()
    torch.cuda.synchronize()
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    probe_tflops = sms * iters * 2.0 * 128 * 128 * 64 / (p0.elapsed_time(p1) * 1e-3) / 1e12
    probe_flop_per_clk_sm = iters * 2.0 * 128 * 128 * 64 / max(1, int(cyc.item()))

    # ---- the vendor library's BF16 attention forward on the same unquantized tensors (torch SDPA, cuDNN backend):
    # context for the paper's "x times BF16 attention" figures, not a target and not part of any path of this library
    bf16_lib = None
    if world == 1:
        try:
            import torch.nn.functional as Fnn
            from torch.nn.attention import SDPBackend, sdpa_kernel
            with sdpa_kernel(SDPBackend.CUDNN_ATTENTION):
                sd = lambda: Fnn.scaled_dot_product_attention(dq, dk, dv)
                for _ in range(3):
                    sd()
                ms_sd = statistics.median(timed_launches(sd, 10, flush, E, torch.cuda.synchronize))
            bf16_lib = {"attn_ms": ms_sd, "attn_tflops": w.flops / (ms_sd * 1e-3) / 1e12, "what": "torch SDPA, cuDNN backend, bf16, noncausal"}
        except Exception:
            bf16_lib = None

    # ---- the library's dense block-scaled FP4 GEMM (cuBLASLt through torch._scaled_mm, NVFP4 operands, 8192^3) as a
    # cross-check of the roofline denominator; context only, None where this torch build does not offer it
    lib_fp4_tflops = None
    try:
        Mg = 8192
        ga = torch.randint(0, 256, (Mg, Mg // 2), dtype=torch.uint8, device=dev).view(torch.float4_e2m1fn_x2)
        gb = torch.randint(0, 256, (Mg, Mg // 2), dtype=torch.uint8, device=dev).view(torch.float4_e2m1fn_x2)
        gs = torch.full((Mg * (Mg // 16),), 1.0, device=dev).to(torch.float8_e4m3fn)      # one scale per 16 elements
        gemm = lambda: torch._scaled_mm(ga, gb.t(), scale_a=gs, scale_b=gs, out_dtype=torch.bfloat16)
        for _ in range(3):
            gemm()
        g0, g1 = E(), E()
        g0.record()
        for _ in range(10):
            gemm()
        g1.record()
        torch.cuda.synchronize()
        lib_fp4_tflops = 10 * 2.0 * Mg ** 3 / (g0.elapsed_time(g1) * 1e-3) / 1e12
        del ga, gb, gs
    except Exception:
        lib_fp4_tflops = None

    # ---- measured ceiling of the softmax arithmetic alone (second roofline of the attention kernel)
    cyc2 = torch.zeros(2, dtype=torch.int64, device=dev)
    arith_iters = 8192
    Bd.fp4attn_softmax_arith_probe(pmap, pairs, arith_iters, cyc2)
    Bd.fp4attn_softmax_arith_probe(pmap, pairs, arith_iters, cyc2)
    torch.cuda.synchronize()
    arith_clk_per_block = int(cyc2[0].item()) / (4.0 * arith_iters)      # per scheduler, four warps each

    # ---- parity sample inputs of the headline workload, taken before its tensors are released
    sample = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        rng = np.random.default_rng(7)
        n_rows = min(N, 4096)
        # sized for roughly 10-30 s of host work: cost ~ heads * rows * N * d at about 0.015 TFLOP/s
        n_heads = int(max(1, min(B * H, round(2.2e11 / (4.0 * n_rows * N * d)))))
        rows = np.sort(rng.choice(N, size=n_rows, replace=False))
        all_heads = [(b, h) for b in range(B) for h in range(H)]
        heads = [all_heads[i] for i in np.linspace(0, len(all_heads) - 1, n_heads).astype(int)]
        pick = lambda t: np.ascontiguousarray(np.stack([_bits(t[b, h]) for b, h in heads])[None])
        amax = (float(dq.abs().max()), float(dk.abs().max())) if w.qk_fmt == I.FMT_NVFP4 else None
        sample = dict(rows=rows, heads=heads, q=pick(dq), k=pick(dk), v=pick(dv), amax=amax,
                      Og=np.stack([O[b, h].float().cpu().numpy().astype(np.float64)[rows] for b, h in heads]))
        if "O_fp8" in state:
            sample["Og8"] = np.stack([state["O_fp8"][b, h].float().cpu().numpy().astype(np.float64)[rows] for b, h in heads])
    state.pop("O_fp8", None)

    # ---- attention kernel alone on the other configurations, each with a roofline fraction of its own (seeded
    # inputs of that configuration; every timed launch follows an L2 flush; median of the launches)
    sweep = {}
    if world == 1 and not args.no_sweep:
        del dq, dk, dv, state["ops"], state["q_only"]
        torch.cuda.empty_cache()
        n_it = 20
        for name in SUB_RECORDS:
            if name == w.name:
                continue
            ww = I.WORKLOADS[name]
            xq, xk, xv = device_qkv(ww, dev)
            sq = Bd.fp4attn_quantize(xq, ww.qk_fmt, Bd.ROLE_Q)
            sk = Bd.fp4attn_quantize(xk, ww.qk_fmt, Bd.ROLE_K)
            sv = Bd.fp4attn_quantize(xv, Bd.FMT_MXFP4, Bd.ROLE_V)
            sv8 = Bd.fp4attn_quantize_v_e4m3(xv)
            del xq, xk, xv
            so = torch.empty((ww.B, ww.H, ww.N, ww.d), dtype=torch.bfloat16, device=dev)
            rec = {"workload": _workload_text(ww), "launches": n_it, "inputs": "seeded recipe of the configuration"}
            variants = [("", {}, 1.0), ("affine_", dict(p_map=Bd.PMAP_AFFINE), 1.0), ("causal_", dict(causal=True), 0.5)]
            if not ww.outliers:                                      # config 4's logits span more than a fixed reference holds
                variants.append(("affine_shiftless_", dict(p_map=Bd.PMAP_AFFINE, fixed_reference=0), 1.0))
            if ww.d == 64 and ww.N % 256 == 0:                       # the two-query schedule beside the one-query one
                variants += [("two_query_", dict(schedule=Bd.SCHEDULE_TWO_QUERY), 1.0),
                             ("two_query_affine_", dict(schedule=Bd.SCHEDULE_TWO_QUERY, p_map=Bd.PMAP_AFFINE), 1.0)]
            variants.append(("fp8_pv_", None, 1.0))
            if ww.B >= 4:                                            # padded sequences: a fixed mix of token counts
                mix = [ww.N, ww.N * 5 // 8 - 120, ww.N // 2 + 1, 300] + [ww.N] * (ww.B - 4)
                sl = torch.tensor(mix, dtype=torch.int32, device=dev)
                variants.append(("length_mix_", dict(seq_len=sl), sum(float(n) * n for n in mix) / (ww.B * float(ww.N) ** 2)))
                rec["length_mix_tokens"] = mix
            for key, kw, share in variants:
                fn = (lambda: Bd.fp4attn_fwd(sq, sk, sv8, out=so, status=status)) if kw is None else \
                     (lambda: Bd.fp4attn_fwd(sq, sk, sv, out=so, status=status, **kw))
                for _ in range(3):
                    fn()
                torch.cuda.synchronize()
                ms = statistics.median(timed_launches(fn, n_it, flush, E, torch.cuda.synchronize))
                # causal: flops counted as half of the full product (the usual convention); length mix: the scores of
                # the tokens that exist
                rec[key + "attn_ms"] = ms
                rec[key + "attn_tflops"] = share * ww.flops / (ms * 1e-3) / 1e12
                if not key:
                    rec["roofline"] = roofline_record(ww, ms, fp4_peak, peaks)
                else:
                    rec[key + "roofline_frac"] = share * ww.flops / (ms * 1e-3) / 1e12 / fp4_peak
            sweep[name] = rec
            del sq, sk, sv, sv8, so
            torch.cuda.empty_cache()
        assert int(status.item()) == 0, "attention kernel reported a bounded-wait timeout"

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    roof = roofline_record(w, attn_launch_ms, fp4_peak, peaks, "attn_fwd_2q_kernel" if args.schedule == "two-query" else "attn_fwd_kernel")
    roof.update({"fp4_gemm_library_tflops": lib_fp4_tflops, "fp4_issue_probe_tflops": probe_tflops, "fp4_issue_probe_flop_per_clk_per_sm": probe_flop_per_clk_sm,
                 "launch_ms_mean": attn_launch_ms, "launch_ms_median": statistics.median(attn_ms)})
    # Softmax-arithmetic roofline: an SM converts four 32x32 blocks (one per scheduler) in `arith_clk_per_block`
    # clocks when it does nothing else; a block carries 4*32*32*d flop of the two products.  Clock: the median SM
    # clock sampled during the timed steps (the nominal maximum where NVML gives no samples).
    sm_hz = clk.summary().get("sm_mhz") or clk.max_mhz or 0
    arith_peak = sms * 4 * (4.0 * 32 * 32 * w.d) / arith_clk_per_block * sm_hz * 1e6 / 1e12 if sm_hz else None
    roof_softmax = {"kernel": roof["kernel"], "bound": "alu", "achieved": attn_tflops, "peak": arith_peak, "unit": UNIT,
                    "frac": attn_tflops / arith_peak if arith_peak else None, "traffic": None,
                    "clk_per_32x32_block_per_scheduler": arith_clk_per_block,
                    "peak_source": "measured on this device: the kernel's score -> code arithmetic for map '%s' run alone, four "
                                   "warps per scheduler (fp4attn_softmax_arith_probe), at the median SM clock of the timed steps; "
                                   "for exact codes the SFU's 16 ex2/clk/SM (12 of 16 pairs -> 192 clk per block) is the unit "
                                   "that binds" % args.p_map}
    for rec in other_maps.values():                                  # the same arithmetic ceiling for the other code maps
        if "softmax_arith_clk_per_block" in rec and sm_hz:
            pk = sms * 4 * (4.0 * 32 * 32 * w.d) / rec["softmax_arith_clk_per_block"] * sm_hz * 1e6 / 1e12
            rec["softmax_arith_frac"] = rec["attn_tflops"] / pk
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": n_warm, "ms_per_step": total_ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "fp4_e2m1 (fp32 accumulate)", "data": "synthetic",
        "config": {"workload": _workload_text(w), "step": "quantize Q,K,V + attention forward", "p_map": args.p_map, "p_scale": args.p_scale, "row_reference": "running" if args.fixed_reference is None else f"fixed at {args.fixed_reference}",
                   "schedule": args.schedule, "l2": "flushed between steps (256 MiB fill, outside the step's events)",
                   "warmup": f"{n_warm} steps (at least --warmup and 300 ms)",
                   "flops": "4*B*H*N^2*d", "parallelism": f"replica x{world}, (batch, head) units, no collective"},
        "attn_only": {"value": attn_tflops, "unit": UNIT, "ms": attn_launch_ms,
                      "note": "attention kernel alone (the paper's timing boundary excludes quantization)",
                      "other_code_maps": other_maps, "bf16_attention_library": bf16_lib},
        "roofline": roof,
        "roofline_softmax_arith": roof_softmax,
        "window": window,
        "roofline_quantize": {"kernel": q_kernel, "bound": "hbm", "achieved": q_bytes / (quant["rows"] * 1e-3) / 1e9,
                              "peak": peaks["hbm_gbs"], "unit": "GB/s",
                              "frac": q_bytes / (quant["rows"] * 1e-3) / 1e9 / peaks["hbm_gbs"],
                              "traffic": NCU_TRAFFIC_BYTES.get(w.name, {}).get("quant_rows"),
                              "bytes_per_element": q_bpe,
                              "v_kernel": {"kernel": "quant_mx_v_kernel", "achieved": v_bytes / (quant["v"] * 1e-3) / 1e9,
                                           "frac": v_bytes / (quant["v"] * 1e-3) / 1e9 / peaks["hbm_gbs"]}},
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "steps": e2e_steps, "api": "fp4attn_attention_host (pinned host buffers)"},
        "attn_other_workloads": sweep,
        "gpu_launches": launches_per_step * args.steps,
        "clocks": clk.summary(),
    }
    # ---- oracle on the host cores: bounded sample of the same workload, plus accuracy vs fp64
    if sample is not None:
        rows, heads = sample["rows"], sample["heads"]
        dt, tf, Oo, Lo, ops = oracle_sample(w, sample["q"], sample["k"], sample["v"], len(heads), rows, args.p_map, args.p_scale,
                                            sample["amax"], fixed_reference=args.fixed_reference)
        Og = sample["Og"]
        rel = max(float(np.linalg.norm(Og[i] - Oo[i]) / np.linalg.norm(Oo[i])) for i in range(len(heads)))
        text = f"{len(heads)} (batch, head) units x {len(rows)} seeded query rows of {w.name}, {dt:.1f} s"
        out["cpu_baseline"] = {"value": tf, "unit": UNIT, "cores": _host_cores(), "blas_threads": _blas_threads(),
                               "kind": "oracle", "sample": text}
        row_abs = np.abs(Og - Oo).max(axis=2)
        out["parity_on_sample"] = {"rel_fro_max": rel, "max_abs": float(row_abs.max()), "rows": int(row_abs.size),
                                   "rows_above_max_abs": int((row_abs > 2e-2).sum()),
                                   "tolerance": {"rel_fro": 5e-3, "max_abs": 2e-2},
                                   "ok": bool(rel <= 5e-3 and row_abs.max() <= 2e-2)}
        out["accuracy_vs_fp64"] = accuracy_vs_fp64(sample["q"], sample["k"], sample["v"], ops, rows, Og, Oo, sample.get("Og8"))
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=250)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(I.WORKLOADS))
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--window-s", type=float, default=1.0,
                    help="length of the median window that follows the K timed steps (0 skips it)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sweep", action="store_true", help="skip the attention-only timings of the other configurations")
    ap.add_argument("--p-scale", default="ceil", choices=["ceil", "thr16", "mse"],
                    help="block-exponent rule of P: ceiling (default), floor(max y + log2 1.6), or per block the better of "
                         "the two neighbouring exponents by squared error (ideal map only)")
    ap.add_argument("--schedule", default="one-query", choices=["one-query", "two-query"],
                    help="query tiles per thread block in the timed step (two-query: d = 64 workloads only)")
    ap.add_argument("--fixed-reference", type=int, default=None,
                    help="time the step with this constant row reference (the shiftless path; ideal or affine map, ceiling rule)")
    ap.add_argument("--p-map", default="ideal", choices=["ideal", "affine", "hybrid4", "hybrid8", "hybrid12"],
                    help="score->code map of the timed path: exact codes (default), the paper's affine classifier, or "
                         "4 / 8 / 12 of every 16 element pairs exact and the rest affine (EX2-density control)")
    args = ap.parse_args()
    w = I.WORKLOADS[args.workload]
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_cuda(args, w)


if __name__ == "__main__":
    main()
