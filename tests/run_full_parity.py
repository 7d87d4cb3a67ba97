#!/usr/bin/env python
"""Every row of every (batch, head) unit of a configuration, CUDA path against the oracle.

The pytest suite compares whole heads of each configuration (a few units each) so that it stays within minutes;
this script is the same comparison (tests/parity.py: strict figures, and the protocol for rows with more than one
correct value) over ALL units, for the record.  One launch of the configuration as bench.py launches it, then the
oracle on a pool of host processes, one unit per task.

  python tests/run_full_parity.py cfg4 [--p-map affine] [--p-scale mse] [--route fp8] [--length-mix] [--workers 12] [--units 0:32]

Prints one JSON line per unit and a summary line.  Needs a B200; imports the oracle (test infrastructure).
"""
from __future__ import annotations

import argparse
import json
import multiprocessing as mp
import os
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

from paper_2609_04105_b200 import inputs as I  # noqa: E402

_G = {}


def _unit(task):
    """Oracle operands of one unit from its bf16 bits, then the whole-head comparison."""
    import parity
    from oracle import quantize as Qz
    try:                                                         # one BLAS thread per worker process
        from threadpoolctl import threadpool_limits
        threadpool_limits(1)
    except Exception:
        pass
    b, h = task
    w, q, k, v, Og, Lg, Gq, Gk, okw = (_G[x] for x in ("w", "q", "k", "v", "O", "L", "Gq", "Gk", "okw"))
    one = lambda a: np.ascontiguousarray(a[b, h][None, None])
    if w.qk_fmt == I.FMT_NVFP4:
        nq, sq = Qz.nv_quantize_lastdim(Qz.bf16_bits_to_f64(one(q)), Gq)
        nk, sk = Qz.nv_quantize_lastdim(Qz.bf16_bits_to_f64(one(k)), Gk)
        qd = {"nib": nq, "sf": sq, "G": Gq, "fmt": "nv"}
        kd = {"nib": nk, "sf": sk, "G": Gk, "fmt": "nv"}
    else:
        qd, kd = Qz.quantize_qk(one(q), "mx"), Qz.quantize_qk(one(k), "mx")
    t0 = time.perf_counter()
    try:
        n = None if _G["lens"] is None else int(_G["lens"][b])     # padded sequence: the rows and keys that exist
        if _G["route"] == "fp8":
            st = _fp8_head(Og[b, h].astype(np.float64), Lg[b, h].astype(np.float64), qd, kd, Qz.quantize_v_e4m3(one(v)), n=n)
        else:
            extra = {} if n is None else dict(rows=np.arange(n), kv_len=n)
            st = parity.compare_head(Og[b, h].astype(np.float64), Lg[b, h].astype(np.float64), qd, kd, Qz.quantize_v(one(v)), 0, 0,
                                     **extra, **okw)
        st["ok"] = True
    except AssertionError as e:
        st = {"ok": False, "error": str(e)[:400]}
    st["head"] = (b, h)
    st["oracle_s"] = round(time.perf_counter() - t0, 1)
    return st


def _fp8_head(Og, Lg, qd, kd, v8, chunk=1024, n=None):
    """FP8 P/V route: strict comparison of one unit, all rows (no alternative evaluations are defined for it); with
    n, the first n rows of a sequence of n tokens."""
    import parity
    from oracle import attention as A
    N = Og.shape[0] if n is None else n
    num = den = 0.0
    worst = lse_err = 0.0
    for r0 in range(0, N, chunk):
        rows = np.arange(r0, min(N, r0 + chunk))
        Oo, Lo = A.fp8_pv_forward(qd, kd, v8, rows=rows, heads=[(0, 0)], seq_len=None if n is None else [n])
        num += ((Og[rows] - Oo[0]) ** 2).sum()
        den += (Oo[0] ** 2).sum()
        worst = max(worst, float(np.abs(Og[rows] - Oo[0]).max()))
        lse_err = max(lse_err, float((np.abs(Lg[rows] - Lo[0]) - parity.LSE_REL * np.abs(Lo[0])).max()))
    st = {"rows": int(N), "rel_fro_strict": float(np.sqrt(num / den)), "max_abs_strict": worst, "lse_err": lse_err,
          "rows_failing_strict": 0, "accepted_with_flips": 0}
    assert st["rel_fro_strict"] <= parity.REL_FRO and worst <= parity.MAX_ABS and lse_err <= parity.LSE_ABS, st
    return st


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("workload", choices=sorted(I.WORKLOADS))
    ap.add_argument("--p-map", default="ideal", choices=["ideal", "affine"])
    ap.add_argument("--p-scale", default="ceil", choices=["ceil", "thr16", "mse"], help="block-exponent rule of P (mse: ideal map only)")
    ap.add_argument("--length-mix", action="store_true",
                    help="padded sequences: N, 5N/8 - 120, N/2 + 1 and 300 tokens in the first four batch entries (B >= 4)")
    ap.add_argument("--route", default="fp4", choices=["fp4", "fp8"], help="probability / value format: Direct-P FP4 or FP8 P/V")
    ap.add_argument("--workers", type=int, default=max(1, len(os.sched_getaffinity(0)) - 2))
    ap.add_argument("--units", default=None, help="begin:end slice of the (batch, head) units, default all")
    args = ap.parse_args()
    import torch
    from oracle import quantize as Qz
    from paper_2609_04105_b200 import binding as Bd
    w = I.WORKLOADS[args.workload]
    q, k, v = I.make_qkv(w)
    dev = lambda a: torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
    qg = Bd.fp4attn_quantize(dev(q), w.qk_fmt, Bd.ROLE_Q)
    kg = Bd.fp4attn_quantize(dev(k), w.qk_fmt, Bd.ROLE_K)
    vg = Bd.fp4attn_quantize_v_e4m3(dev(v)) if args.route == "fp8" else Bd.fp4attn_quantize(dev(v), Bd.FMT_MXFP4, Bd.ROLE_V)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    lens = None
    if args.length_mix:
        assert w.B >= 4, "the length mix needs four batch entries"
        lens = [w.N, w.N * 5 // 8 - 120, w.N // 2 + 1, 300] + [w.N] * (w.B - 4)
    rule = {"ceil": Bd.PSCALE_CEIL, "thr16": Bd.PSCALE_THR16, "mse": Bd.PSCALE_MSE}[args.p_scale]
    assert args.route == "fp4" or args.p_scale == "ceil", "the FP8 P/V route has one rule"
    O, L = Bd.fp4attn_fwd(qg, kg, vg, status=status, p_map=Bd.PMAP_AFFINE if args.p_map == "affine" else Bd.PMAP_IDEAL,
                          p_scale_rule=rule, seq_len=None if lens is None else torch.tensor(lens, dtype=torch.int32, device="cuda"))
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    _G.update(lens=lens, route=args.route, w=w, q=q, k=k, v=v, O=O.float().cpu().numpy(), L=L.cpu().numpy(), Gq=None, Gk=None,
              okw=dict(p_map=args.p_map, p_scale=args.p_scale))
    if w.qk_fmt == I.FMT_NVFP4:
        _G["Gq"] = Qz.nv_tensor_scale(Qz.bf16_bits_to_f64(q))
        _G["Gk"] = Qz.nv_tensor_scale(Qz.bf16_bits_to_f64(k))
    del qg, kg, vg, O, L
    torch.cuda.empty_cache()
    units = [(b, h) for b in range(w.B) for h in range(w.H)]
    if args.units:
        lo, hi = (int(x) for x in args.units.split(":"))
        units = units[lo:hi]
    t0 = time.perf_counter()
    with mp.get_context("fork").Pool(args.workers) as pool:        # workers inherit the arrays; they never touch CUDA
        res = []
        for st in pool.imap_unordered(_unit, units):
            print(json.dumps(st), flush=True)
            res.append(st)
    good = [r for r in res if r["ok"]]
    summary = {"workload": w.name, "route": args.route, "p_map": args.p_map, "p_scale": args.p_scale, "length_mix": lens, "units": len(res), "units_ok": len(good),
               "rows": int(sum(r["rows"] for r in good)), "wall_s": round(time.perf_counter() - t0, 1)}
    if good:
        summary.update(rel_fro_strict_max=max(r["rel_fro_strict"] for r in good), max_abs_strict=max(r["max_abs_strict"] for r in good),
                       lse_err_max=max(r["lse_err"] for r in good), rows_failing_strict=int(sum(r["rows_failing_strict"] for r in good)),
                       accepted_with_flips=int(sum(r["accepted_with_flips"] for r in good)))
    print("SUMMARY " + json.dumps(summary), flush=True)
    sys.exit(0 if len(good) == len(res) else 1)


if __name__ == "__main__":
    main()
