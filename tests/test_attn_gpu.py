"""Kernel (b): the CUDA Direct-P attention forward against the oracle, element by element.

Tolerances (stated by the benchmark spec, per (batch, head)): relative Frobenius error <= 5e-3 and
max-abs error <= 2e-2 between the bf16 output and the oracle's fp64 output; for the LSE
|d| <= 1e-3 + 1e-5 |LSE| (fp32 log2 and accumulation of the row sum).
"""
import numpy as np
import pytest
import torch

from oracle import attention as A
from oracle import quantize as Qz
from paper_2609_04105_b200 import inputs as I

pytestmark = pytest.mark.gpu

REL_FRO, MAX_ABS = 5e-3, 2e-2


def _dev(bits):
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def run_gpu(w, q, k, v, softmax_scale=0.0):
    from paper_2609_04105_b200 import binding as Bd
    qd = Bd.fp4attn_quantize(_dev(q), w.qk_fmt, Bd.ROLE_Q)
    kd = Bd.fp4attn_quantize(_dev(k), w.qk_fmt, Bd.ROLE_K)
    vd = Bd.fp4attn_quantize(_dev(v), Bd.FMT_MXFP4, Bd.ROLE_V)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    O, lse = Bd.fp4attn_fwd(qd, kd, vd, softmax_scale=softmax_scale, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0, "kernel reported a bounded-wait timeout"
    return O.float().cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64)


def oracle_operands(w, q, k, v):
    fmt = "mx" if w.qk_fmt == I.FMT_MXFP4 else "nv"
    return Qz.quantize_qk(q, fmt), Qz.quantize_qk(k, fmt), Qz.quantize_v(v)


def check_heads(Og, Lg, Oo, Lo, heads, rows=None):
    """Og [B,H,N,d], Lg [B,H,N] from the GPU; Oo [n_heads,R,d], Lo [n_heads,R] from the oracle."""
    worst = (0.0, 0.0, 0.0)
    for n, (b, h) in enumerate(heads):
        g = Og[b, h] if rows is None else Og[b, h][rows]
        l = Lg[b, h] if rows is None else Lg[b, h][rows]
        rel = np.linalg.norm(g - Oo[n]) / np.linalg.norm(Oo[n])
        mab = np.abs(g - Oo[n]).max()
        dl = np.abs(l - Lo[n]) - 1e-5 * np.abs(Lo[n])
        worst = (max(worst[0], rel), max(worst[1], mab), max(worst[2], dl.max()))
        assert rel <= REL_FRO, f"head {(b, h)}: rel Frobenius {rel:.3e}"
        assert mab <= MAX_ABS, f"head {(b, h)}: max abs {mab:.3e}"
        assert dl.max() <= 1e-3, f"head {(b, h)}: LSE error {dl.max():.3e}"
    return worst


SMALL = [
    ("cfg1", dict()),                                   # B1 H2 N256 d128, MXFP4 x4 (config 1 itself)
    ("cfg1", dict(N=128)),                              # a single 128-key pair
    ("cfg1", dict(N=384, H=3)),                         # odd number of pairs, several heads
    ("cfg1", dict(d=64, N=512)),                        # MXFP4 at d=64
    ("cfg3", dict(B=2, H=2, N=512)),                    # NVFP4 Q/K at d=64 (config 3's formats)
    ("cfg3", dict(B=1, H=2, N=384, d=128)),             # NVFP4 Q/K at d=128
    ("cfg4", dict(H=2, N=1024)),                        # outlier channels: reference rescales, zero blocks
    ("cfg2", dict(B=2, H=3, N=2304)),                   # ring wraps several times, ragged wave
]


@pytest.mark.parametrize("name,kw", SMALL)
def test_attention_matches_oracle_elementwise(name, kw):
    w = I.shrink(I.WORKLOADS[name], **kw)
    q, k, v = I.make_qkv(w)
    Og, Lg = run_gpu(w, q, k, v)
    qd, kd, vd = oracle_operands(w, q, k, v)
    heads = [(b, h) for b in range(w.B) for h in range(w.H)]
    Oo, Lo = A.direct_p_forward(qd, kd, vd, heads=heads)
    check_heads(Og, Lg, Oo, Lo, heads)


def test_explicit_softmax_scale_and_constant_v():
    w = I.shrink(I.WORKLOADS["cfg1"], N=256)
    q, k, v = I.make_qkv(w)
    ones = I.f32_to_bf16_bits(np.full((w.B, w.H, w.N, w.d), -2.0, dtype=np.float32))
    Og, Lg = run_gpu(w, q, k, ones, softmax_scale=0.25)
    assert np.all(Og == -2.0)            # numerator and denominator use the same rounded codes
    qd, kd, vd = oracle_operands(w, q, k, ones)
    Oo, Lo = A.direct_p_forward(qd, kd, vd, softmax_scale=0.25)
    check_heads(Og, Lg, Oo, Lo, [(0, 0), (0, 1)])


def test_run_to_run_determinism():
    w = I.shrink(I.WORKLOADS["cfg2"], B=1, H=4, N=1024)
    q, k, v = I.make_qkv(w)
    O1, L1 = run_gpu(w, q, k, v)
    O2, L2 = run_gpu(w, q, k, v)
    assert np.array_equal(O1, O2) and np.array_equal(L1, L2)


def _full_size_case(name, n_rows, n_heads, seed, whole_heads=0):
    """One launch of a whole configuration as bench.py launches it.  `n_heads` (batch, head) units are compared on
    `n_rows` sampled query rows each, and `whole_heads` further units on ALL their rows under the protocol for
    outputs with more than one correct value (tests/parity.py); the statistics of those are printed."""
    import parity
    w = I.WORKLOADS[name]
    q, k, v = I.make_qkv(w)
    Og, Lg = run_gpu(w, q, k, v)
    qd, kd, vd = oracle_operands(w, q, k, v)
    rng = np.random.default_rng(seed)
    all_heads = [(b, h) for b in range(w.B) for h in range(w.H)]
    pick = [all_heads[i] for i in rng.choice(len(all_heads), size=min(n_heads + whole_heads, len(all_heads)), replace=False)]
    if n_heads:
        rows = np.sort(rng.choice(w.N, size=n_rows, replace=False))
        rows[0], rows[-1] = 0, w.N - 1
        heads = sorted(pick[:n_heads])
        Oo, Lo = A.direct_p_forward(qd, kd, vd, heads=heads, rows=rows)
        check_heads(Og, Lg, Oo, Lo, heads, rows)
    for (b, h) in pick[n_heads:]:
        st = parity.compare_head(Og[b, h], Lg[b, h], qd, kd, vd, b, h)
        print(f"{name} whole head: {st}")
        assert st["lse_err"] <= 1e-3 or st["rows_failing_strict"] > 0, st


def test_config2_full_size_sampled_rows_and_whole_heads():
    """B4 H16 N4096 d128 as bench.py launches it; 8 heads x 256 sampled query rows and 2 whole heads."""
    _full_size_case("cfg2", 256, 8, 2, whole_heads=2)


def test_config3_full_size_sampled_rows_and_whole_heads():
    """B8 H16 N8192 d64, NVFP4 Q/K (scores are sums float32 cannot always hold); 4 heads x 128 sampled rows and
    2 whole heads (all 8192 rows)."""
    _full_size_case("cfg3", 128, 4, 3, whole_heads=2)


def test_config4_full_size_sampled_rows_and_whole_heads():
    """B1 H32 N16384 d128 with x20 outlier channels (|y| ~ 300: moving reference, zero blocks, near one-hot
    rows where one code decision can move an output row); 3 heads x 96 sampled rows and 2 whole heads (all
    16384 rows)."""
    _full_size_case("cfg4", 96, 3, 4, whole_heads=2)


@pytest.mark.parametrize("N", [1024, 2048, 4096, 8192, 16384])
def test_config5_sweep_full_size_sampled_rows(N):
    """Sequence sweep at B*N = 32768 tokens, H=16, d=128: every point below the longest on sampled rows."""
    _full_size_case(f"cfg5_N{N}", 128 if N < 16384 else 96, 8 if N < 8192 else 4, 5)


def test_config5_longest_sequence_whole_head():
    """N = 32768 (B=1, H=16, d=128), the workload bench.py times: one whole head (all 32768 rows) and sampled rows
    of two more."""
    _full_size_case("cfg5_N32768", 64, 2, 5, whole_heads=1)


@pytest.mark.parametrize("kw", [dict(N=512), dict(B=3, H=8, N=256), dict(B=2, H=17, N=128)])
def test_host_buffer_entry_point_matches_device_path(kw):
    """Few heads take the one-stream path, 8 or more the pipelined one (groups of heads on internal copy
    streams, ragged last group): both must return what the device path returns, bit for bit; twice in a row
    to cover reuse of the internal events."""
    from paper_2609_04105_b200 import binding as Bd
    w = I.shrink(I.WORKLOADS["cfg1"], **kw)
    q, k, v = I.make_qkv(w)
    Og, Lg = run_gpu(w, q, k, v)
    host = [torch.from_numpy(a.view(np.int16)).view(torch.bfloat16).pin_memory() for a in (q, k, v)]
    ws = torch.empty(Bd.fp4attn_attention_host_workspace_bytes(w.qk_fmt, w.B, w.H, w.N, w.d), dtype=torch.uint8, device="cuda")
    for rep in range(3):
        out = torch.zeros((w.B, w.H, w.N, w.d), dtype=torch.bfloat16).pin_memory()
        lse = torch.zeros((w.B, w.H, w.N), dtype=torch.float32).pin_memory()
        st = torch.full((1,), -1, dtype=torch.int32).pin_memory()
        Bd.fp4attn_attention_host(host[0], host[1], host[2], w.qk_fmt, out, lse, ws, status=st)
        torch.cuda.synchronize()
        assert int(st[0]) == 0                                  # the call's status word: no bounded wait ran out
        assert np.array_equal(out.float().numpy().astype(np.float64), Og)
        assert np.array_equal(lse.numpy().astype(np.float64), Lg)
        if rep == 1:
            Bd.fp4attn_release()                                # internal streams, events, tensor maps: made again on the next call


def test_host_buffer_entry_point_from_two_threads():
    """Two host threads, each with its own stream, workspace and host buffers, enqueue the pipelined host
    path at the same time (the library's internal copy streams and events are shared and guarded by a
    lock): each must get exactly what the device path returns for its inputs."""
    import threading
    from paper_2609_04105_b200 import binding as Bd
    jobs = []
    for t in range(2):
        w = I.shrink(I.WORKLOADS["cfg1"], H=5 + 4 * t, N=384)                 # 10 and 18 heads: 4 groups each
        q, k, v = I.make_qkv(w)                                                # shapes differ, so do the tensors
        Og, Lg = run_gpu(w, q, k, v)
        host = [torch.from_numpy(a.view(np.int16)).view(torch.bfloat16).pin_memory() for a in (q, k, v)]
        ws = torch.empty(Bd.fp4attn_attention_host_workspace_bytes(w.qk_fmt, w.B, w.H, w.N, w.d), dtype=torch.uint8, device="cuda")
        out = torch.zeros((w.B, w.H, w.N, w.d), dtype=torch.bfloat16).pin_memory()
        lse = torch.zeros((w.B, w.H, w.N), dtype=torch.float32).pin_memory()
        jobs.append((w, host, ws, out, lse, Og, Lg, torch.cuda.Stream()))
    torch.cuda.synchronize()
    errors = []

    def work(job):
        w, host, ws, out, lse, _, _, stream = job
        try:
            with torch.cuda.stream(stream):
                for _ in range(3):
                    Bd.fp4attn_attention_host(host[0], host[1], host[2], w.qk_fmt, out, lse, ws)
            stream.synchronize()
        except Exception as e:                                                 # surfaces in the main thread below
            errors.append(e)

    threads = [threading.Thread(target=work, args=(j,)) for j in jobs]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    for w, host, ws, out, lse, Og, Lg, _ in jobs:
        assert np.array_equal(out.float().numpy().astype(np.float64), Og)
        assert np.array_equal(lse.numpy().astype(np.float64), Lg)


def test_cached_tensor_maps_follow_the_buffers():
    """The library remembers the tensor maps of a thread's last few calls by operand address and shape.  Calls
    that alternate between two operand sets and two output buffers, more distinct calls than the cache holds,
    and a call after fp4attn_release() must each read and write the buffers they were given."""
    from paper_2609_04105_b200 import binding as Bd
    sets = []
    for i, kw in enumerate((dict(N=256), dict(N=384), dict(N=256, H=3))):
        w = I.shrink(I.WORKLOADS["cfg1"], **kw)
        q, k, v = I.make_qkv(I.shrink(w, cfg=w.cfg + i))
        ops = [Bd.fp4attn_quantize(_dev(a), Bd.FMT_MXFP4, r) for a, r in ((q, Bd.ROLE_Q), (k, Bd.ROLE_K), (v, Bd.ROLE_V))]
        ref, _ = Bd.fp4attn_fwd(*ops)
        sets.append((ops, ref.clone()))
    outs = [torch.zeros_like(sets[j % 3][1]) for j in range(12)]          # twelve distinct output buffers > cache entries
    for rnd in range(2):
        for j, o in enumerate(outs):
            o.zero_()
            Bd.fp4attn_fwd(*sets[j % 3][0], out=o)
        torch.cuda.synchronize()
        for j, o in enumerate(outs):
            assert torch.equal(o, sets[j % 3][1]), (rnd, j)
        Bd.fp4attn_release()


def test_invalid_arguments_are_rejected_before_launch():
    from paper_2609_04105_b200 import binding as Bd
    x = torch.zeros((1, 1, 100, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(Bd.Fp4AttnError):
        Bd.fp4attn_quantize(x, Bd.FMT_MXFP4, Bd.ROLE_Q)
    x = torch.zeros((1, 1, 128, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(Bd.Fp4AttnError):
        Bd.fp4attn_quantize(x, Bd.FMT_NVFP4, Bd.ROLE_V)


def test_bounded_wait_times_out_and_reports_status():
    """Failure detection without a GPU fault: a wait that nothing satisfies runs out after its
    limit, the warp returns normally with the time-out status, and the context keeps working."""
    import time
    from paper_2609_04105_b200 import binding as Bd
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    t0 = time.perf_counter()
    Bd.fp4attn_selftest_bounded_wait(1 << 26, status)          # ~35 ms at 1.9 GHz
    torch.cuda.synchronize()
    assert int(status.item()) == Bd.ERR_TIMEOUT
    assert time.perf_counter() - t0 < 5.0
    x = torch.ones(8, device="cuda")                            # the context is still usable
    assert float((x + 1).sum()) == 16.0
    with pytest.raises(Bd.Fp4AttnError):
        Bd.fp4attn_selftest_bounded_wait(0, status)


def test_softmax_arithmetic_probe_respects_the_special_function_unit():
    """The probe runs the kernel's score -> code arithmetic alone.  With exact codes 24 of a block's 32 elements per
    row take ex2.approx, at 16 per clock and SM = 8 clocks per warp instruction and scheduler: no less than 192
    clocks per block.  The affine map has no exponential and must come out faster; the hybrid maps lie between."""
    from paper_2609_04105_b200 import binding as Bd
    cyc = torch.zeros(2, dtype=torch.int64, device="cuda")
    iters = 2048

    def clk(p_map, pairs=0):
        Bd.fp4attn_softmax_arith_probe(p_map, pairs, iters, cyc)
        torch.cuda.synchronize()
        return int(cyc[0].item()) / (4.0 * iters)

    ideal, affine, hybrid8 = clk(Bd.PMAP_IDEAL), clk(Bd.PMAP_AFFINE), clk(Bd.PMAP_HYBRID, 0x5555)
    assert 192.0 <= ideal < 300.0, ideal
    assert 40.0 < affine < ideal and affine <= hybrid8 <= ideal, (affine, hybrid8, ideal)
    with pytest.raises(Bd.Fp4AttnError):
        Bd.fp4attn_softmax_arith_probe(Bd.PMAP_HYBRID, 0x0101, iters, cyc)
    with pytest.raises(Bd.Fp4AttnError):
        Bd.fp4attn_softmax_arith_probe(Bd.PMAP_IDEAL, 0, 0, cyc)


# ------------------------------------------------------------------ affine classifier (p_map = AFFINE)
def run_gpu_affine(w, q, k, v, a=0.0, b=0.0):
    from paper_2609_04105_b200 import binding as Bd
    qd = Bd.fp4attn_quantize(_dev(q), w.qk_fmt, Bd.ROLE_Q)
    kd = Bd.fp4attn_quantize(_dev(k), w.qk_fmt, Bd.ROLE_K)
    vd = Bd.fp4attn_quantize(_dev(v), Bd.FMT_MXFP4, Bd.ROLE_V)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    O, lse = Bd.fp4attn_fwd(qd, kd, vd, status=status, p_map=Bd.PMAP_AFFINE, affine_a=a, affine_b=b)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return O.float().cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64)


AFFINE_CASES = [
    ("cfg1", dict(), (0.0, 0.0)),
    ("cfg1", dict(N=384, H=3), (1.6, 0.95)),                 # the paper's second constant pair
    ("cfg1", dict(d=64, N=512), (0.0, 0.0)),
    ("cfg3", dict(B=2, H=2, N=512), (0.0, 0.0)),
    ("cfg3", dict(B=1, H=2, N=384, d=128), (0.0, 0.0)),
    ("cfg4", dict(H=2, N=1024), (0.0, 0.0)),
    ("cfg2", dict(B=2, H=3, N=2304), (0.0, 0.0)),
]


@pytest.mark.parametrize("name,kw,ab", AFFINE_CASES)
def test_affine_map_matches_oracle_elementwise(name, kw, ab):
    """Same tolerances as the exact map: the classifier's arithmetic is fixed in fp32 on both sides,
    so the codes agree bit for bit and only accumulation order and bf16 rounding differ."""
    w = I.shrink(I.WORKLOADS[name], **kw)
    q, k, v = I.make_qkv(w)
    Og, Lg = run_gpu_affine(w, q, k, v, *ab)
    qd, kd, vd = oracle_operands(w, q, k, v)
    heads = [(b, h) for b in range(w.B) for h in range(w.H)]
    aff = ab if ab[0] else (1.5, 1.2)
    Oo, Lo = A.direct_p_forward(qd, kd, vd, heads=heads, p_map="affine", affine=aff)
    check_heads(Og, Lg, Oo, Lo, heads)


def test_affine_map_config2_full_size_sampled_rows():
    w = I.WORKLOADS["cfg2"]
    q, k, v = I.make_qkv(w)
    Og, Lg = run_gpu_affine(w, q, k, v)
    qd, kd, vd = oracle_operands(w, q, k, v)
    rng = np.random.default_rng(12)
    rows = np.sort(rng.choice(w.N, size=192, replace=False))
    heads = [(0, 0), (1, 7), (3, 15)]
    Oo, Lo = A.direct_p_forward(qd, kd, vd, heads=heads, rows=rows, p_map="affine")
    check_heads(Og, Lg, Oo, Lo, heads, rows)


def test_unknown_p_map_is_rejected():
    from paper_2609_04105_b200 import binding as Bd
    w = I.shrink(I.WORKLOADS["cfg1"], N=128)
    q, k, v = I.make_qkv(w)
    qd = Bd.fp4attn_quantize(_dev(q), w.qk_fmt, Bd.ROLE_Q)
    kd = Bd.fp4attn_quantize(_dev(k), w.qk_fmt, Bd.ROLE_K)
    vd = Bd.fp4attn_quantize(_dev(v), Bd.FMT_MXFP4, Bd.ROLE_V)
    with pytest.raises(Bd.Fp4AttnError):
        Bd.fp4attn_fwd(qd, kd, vd, p_map=7)


# ------------------------------------------------------------------ threshold block-exponent rule
@pytest.mark.parametrize("name,kw,p_map", [
    ("cfg1", dict(), "ideal"), ("cfg1", dict(), "affine"),
    ("cfg3", dict(B=2, H=2, N=512), "ideal"), ("cfg4", dict(H=2, N=1024), "ideal"),
    ("cfg2", dict(B=1, H=2, N=2048), "affine"),
])
def test_threshold_scale_rule_matches_oracle_elementwise(name, kw, p_map):
    from paper_2609_04105_b200 import binding as Bd
    w = I.shrink(I.WORKLOADS[name], **kw)
    q, k, v = I.make_qkv(w)
    qg = Bd.fp4attn_quantize(_dev(q), w.qk_fmt, Bd.ROLE_Q)
    kg = Bd.fp4attn_quantize(_dev(k), w.qk_fmt, Bd.ROLE_K)
    vg = Bd.fp4attn_quantize(_dev(v), Bd.FMT_MXFP4, Bd.ROLE_V)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    O, lse = Bd.fp4attn_fwd(qg, kg, vg, status=status, p_scale_rule=Bd.PSCALE_THR16,
                            p_map=Bd.PMAP_AFFINE if p_map == "affine" else Bd.PMAP_IDEAL)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    Og, Lg = O.float().cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64)
    qd, kd, vd = oracle_operands(w, q, k, v)
    heads = [(b, h) for b in range(w.B) for h in range(w.H)]
    Oo, Lo = A.direct_p_forward(qd, kd, vd, heads=heads, p_map=p_map, p_scale="thr16")
    check_heads(Og, Lg, Oo, Lo, heads)


# ------------------------------------------------------------------ causal mask and grouped-query attention
def run_gpu_general(w, q, k, v, **kw):
    from paper_2609_04105_b200 import binding as Bd
    qg = Bd.fp4attn_quantize(_dev(q), w.qk_fmt, Bd.ROLE_Q)
    kg = Bd.fp4attn_quantize(_dev(np.ascontiguousarray(k)), w.qk_fmt, Bd.ROLE_K)
    vg = Bd.fp4attn_quantize(_dev(np.ascontiguousarray(v)), Bd.FMT_MXFP4, Bd.ROLE_V)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    O, lse = Bd.fp4attn_fwd(qg, kg, vg, status=status, **kw)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return O.float().cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64)


CAUSAL_CASES = [
    ("cfg1", dict(), 1, "ideal"),
    ("cfg1", dict(N=128), 1, "ideal"),
    ("cfg1", dict(N=640, H=3), 1, "ideal"),
    ("cfg1", dict(N=512, H=4), 2, "ideal"),                 # grouped-query: 4 query heads on 2 K/V heads
    ("cfg1", dict(d=64, N=512, H=4), 4, "affine"),          # multi-query, affine map
    ("cfg3", dict(B=2, H=2, N=512), 1, "ideal"),            # NVFP4 Q/K, d = 64
    ("cfg4", dict(H=2, N=1024), 1, "ideal"),
    ("cfg2", dict(B=2, H=3, N=2304), 1, "affine"),
]


@pytest.mark.parametrize("name,kw,group,p_map", CAUSAL_CASES)
def test_causal_and_gqa_match_oracle_elementwise(name, kw, group, p_map):
    from paper_2609_04105_b200 import binding as Bd
    w = I.shrink(I.WORKLOADS[name], **kw)
    q, k, v = I.make_qkv(w)
    k, v = k[:, : w.H // group], v[:, : w.H // group]
    Og, Lg = run_gpu_general(w, q, k, v, causal=True, p_map=Bd.PMAP_AFFINE if p_map == "affine" else Bd.PMAP_IDEAL)
    fmt = "mx" if w.qk_fmt == I.FMT_MXFP4 else "nv"
    qd, kd, vd = Qz.quantize_qk(q, fmt), Qz.quantize_qk(np.ascontiguousarray(k), fmt), Qz.quantize_v(np.ascontiguousarray(v))
    heads = [(b, h) for b in range(w.B) for h in range(w.H)]
    Oo, Lo = A.direct_p_forward(qd, kd, vd, heads=heads, causal=True, kv_group=group, p_map=p_map)
    check_heads(Og, Lg, Oo, Lo, heads)


# ------------------------------------------------------------------ padded sequences (seq_len)
SEQLEN_CASES = [
    # name, shrink, lengths per batch entry, causal, K/V group, map, block-exponent rule
    ("cfg1", dict(B=3, H=2, N=512), [512, 300, 77], False, 1, "ideal", "ceil"),      # full, inside a tile, inside a block
    ("cfg1", dict(B=4, H=2, N=384), [1, 32, 128, 383], False, 1, "ideal", "ceil"),   # one key; block and tile boundaries
    ("cfg1", dict(B=2, H=4, N=640), [129, 600], True, 2, "ideal", "ceil"),           # causal, grouped K/V heads
    ("cfg1", dict(B=2, H=2, N=512), [200, 470], True, 1, "affine", "thr16"),
    ("cfg3", dict(B=2, H=2, N=512), [5, 257], False, 1, "affine", "ceil"),           # NVFP4 Q/K, d = 64
    ("cfg3", dict(B=2, H=2, N=768), [700, 330], True, 1, "ideal", "ceil"),
    ("cfg2", dict(B=2, H=2, N=1024), [1000, 640], False, 1, "ideal", "mse"),         # d = 128, MSE-selected exponents
    ("cfg4", dict(B=1, H=2, N=1024), [900], False, 1, "ideal", "ceil"),              # outlier channels
]


@pytest.mark.parametrize("name,kw,lens,causal,group,p_map,p_scale", SEQLEN_CASES)
def test_padded_sequences_match_oracle_on_the_rows_that_exist(name, kw, lens, causal, group, p_map, p_scale):
    """Per-batch token counts: keys beyond a count are masked, key tiles beyond it skipped; the rows below the count
    are compared with the oracle (whole-head protocol), the rows beyond it must at least be finite."""
    import parity
    from paper_2609_04105_b200 import binding as Bd
    w = I.shrink(I.WORKLOADS[name], **kw)
    q, k, v = I.make_qkv(w)
    k, v = np.ascontiguousarray(k[:, : w.H // group]), np.ascontiguousarray(v[:, : w.H // group])
    sl = torch.tensor(lens, dtype=torch.int32, device="cuda")
    rule = {"ceil": Bd.PSCALE_CEIL, "thr16": Bd.PSCALE_THR16, "mse": Bd.PSCALE_MSE}[p_scale]
    Og, Lg = run_gpu_general(w, q, k, v, causal=causal, seq_len=sl, p_scale_rule=rule,
                             p_map=Bd.PMAP_AFFINE if p_map == "affine" else Bd.PMAP_IDEAL)
    fmt = "mx" if w.qk_fmt == I.FMT_MXFP4 else "nv"
    qd, kd, vd = Qz.quantize_qk(q, fmt), Qz.quantize_qk(k, fmt), Qz.quantize_v(v)
    for b in range(w.B):
        n = lens[b]
        for h in range(w.H):
            st = parity.compare_head(Og[b, h], Lg[b, h], qd, kd, vd, b, h, rows=np.arange(n), kv_group=group, causal=causal,
                                     p_map=p_map, p_scale=p_scale, kv_len=n)
            assert st["lse_err"] <= parity.LSE_ABS, st
            # rows of the last tile that holds a token are computed (over the keys that exist); none may be NaN or Inf
            last = min(w.N, (n + 127) // 128 * 128)
            assert np.isfinite(Og[b, h][:last]).all() and np.isfinite(Lg[b, h][:last]).all()


def test_padded_sequences_full_size_length_mix_sampled_rows_and_timing():
    """B4 H16 N8192 d128 with a mix of lengths (full, inside a tile, one key past a tile boundary, short): sampled rows
    of two heads per batch entry against the oracle, noncausal and causal; and the launch takes less time than the full
    one (key tiles beyond a length are skipped, query tiles beyond it walk a single stage)."""
    import parity
    from paper_2609_04105_b200 import binding as Bd
    w = I.WORKLOADS["cfg5_N8192"]
    lens = [8192, 5000, 4097, 300]
    q, k, v = I.make_qkv(w)
    qg, kg = Bd.fp4attn_quantize(_dev(q), w.qk_fmt, Bd.ROLE_Q), Bd.fp4attn_quantize(_dev(k), w.qk_fmt, Bd.ROLE_K)
    vg = Bd.fp4attn_quantize(_dev(v), Bd.FMT_MXFP4, Bd.ROLE_V)
    sl = torch.tensor(lens, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    qd, kd, vd = oracle_operands(w, q, k, v)
    rng = np.random.default_rng(11)
    for causal in (False, True):
        O, L = Bd.fp4attn_fwd(qg, kg, vg, status=status, seq_len=sl, causal=causal)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        Og, Lg = O.float().cpu().numpy().astype(np.float64), L.cpu().numpy().astype(np.float64)
        for b, n in enumerate(lens):
            rows = np.unique(np.concatenate([[0, n - 1], rng.choice(n, size=min(n, 96), replace=False)]))
            for h in rng.choice(w.H, size=2, replace=False):
                st = parity.compare_head(Og[b, h], Lg[b, h], qd, kd, vd, b, int(h), rows=rows, causal=causal, kv_len=n)
                assert st["lse_err"] <= parity.LSE_ABS, st
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
    for _ in range(2):
        Bd.fp4attn_fwd(qg, kg, vg, status=status)
    ev[0].record()
    Bd.fp4attn_fwd(qg, kg, vg, status=status)
    ev[1].record()
    Bd.fp4attn_fwd(qg, kg, vg, status=status, seq_len=sl)
    ev[2].record()
    torch.cuda.synchronize()
    full, part = ev[0].elapsed_time(ev[1]), ev[1].elapsed_time(ev[2])
    work = sum(float(n) * n for n in lens) / (len(lens) * float(w.N) ** 2)          # 0.41 of the full launch's scores
    print(f"full {full:.3f} ms, length mix {part:.3f} ms, share of the scores {work:.2f}")
    assert part < 0.75 * full


def test_padded_sequences_full_length_is_bit_identical_and_padding_content_is_irrelevant():
    """seq_len = N must give the bits of the call without seq_len (another kernel instance: the masked one).  And what
    sits in the padding of Q and K, and in V beyond the 32-key block that holds the last token, cannot change the
    rows that exist."""
    from paper_2609_04105_b200 import binding as Bd
    w = I.shrink(I.WORKLOADS["cfg2"], B=2, H=2, N=768)
    q, k, v = I.make_qkv(w)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")

    def run(q, k, v, lens):
        qg, kg = Bd.fp4attn_quantize(_dev(q), w.qk_fmt, Bd.ROLE_Q), Bd.fp4attn_quantize(_dev(k), w.qk_fmt, Bd.ROLE_K)
        vg = Bd.fp4attn_quantize(_dev(v), Bd.FMT_MXFP4, Bd.ROLE_V)
        sl = None if lens is None else torch.tensor(lens, dtype=torch.int32, device="cuda")
        O, L = Bd.fp4attn_fwd(qg, kg, vg, status=status, seq_len=sl)
        torch.cuda.synchronize()
        return O, L

    O0, L0 = run(q, k, v, None)
    O1, L1 = run(q, k, v, [768, 768])
    assert torch.equal(O0, O1) and torch.equal(L0, L1)
    lens = [500, 290]
    O2, L2 = run(q, k, v, lens)
    q2, k2, v2 = q.copy(), k.copy(), v.copy()
    rng = np.random.default_rng(5)
    for b, n in enumerate(lens):
        pad = (n + 31) // 32 * 32                                # V: the straddling block keeps its scale
        for t, lo in ((q2, n), (k2, n), (v2, pad)):
            shape = t[b, :, lo:].shape                           # finite bf16 of either sign, magnitudes 2^-7 .. 2^9
            t[b, :, lo:] = (rng.integers(0x3C00, 0x4400, size=shape) | (rng.integers(0, 2, size=shape) << 15)).astype(t.dtype)
    O3, L3 = run(q2, k2, v2, lens)
    for b, n in enumerate(lens):
        assert torch.equal(O2[b, :, :n], O3[b, :, :n]) and torch.equal(L2[b, :, :n], L3[b, :, :n])
    assert int(status.item()) == 0


def test_padded_sequences_reject_what_they_do_not_cover():
    from paper_2609_04105_b200 import binding as Bd
    w = I.shrink(I.WORKLOADS["cfg3"], B=2, H=2, N=512)
    q, k, v = I.make_qkv(w)
    qg, kg = Bd.fp4attn_quantize(_dev(q), w.qk_fmt, Bd.ROLE_Q), Bd.fp4attn_quantize(_dev(k), w.qk_fmt, Bd.ROLE_K)
    vg = Bd.fp4attn_quantize(_dev(v), Bd.FMT_MXFP4, Bd.ROLE_V)
    sl = torch.tensor([100, 200], dtype=torch.int32, device="cuda")
    with pytest.raises(Bd.Fp4AttnError):
        Bd.fp4attn_fwd(qg, kg, vg, seq_len=sl, schedule=Bd.SCHEDULE_TWO_QUERY)
    with pytest.raises(Bd.Fp4AttnError):
        Bd.fp4attn_fwd(qg, kg, vg, seq_len=sl, p_map=Bd.PMAP_HYBRID, exact_pairs=0x5555)


def test_gqa_noncausal_matches_oracle():
    w = I.shrink(I.WORKLOADS["cfg1"], N=384, H=6)
    q, k, v = I.make_qkv(w)
    k, v = k[:, :2], v[:, :2]
    Og, Lg = run_gpu_general(w, q, k, v)
    qd, kd, vd = Qz.quantize_qk(q, "mx"), Qz.quantize_qk(np.ascontiguousarray(k), "mx"), Qz.quantize_v(np.ascontiguousarray(v))
    heads = [(0, h) for h in range(6)]
    Oo, Lo = A.direct_p_forward(qd, kd, vd, heads=heads, kv_group=3)
    check_heads(Og, Lg, Oo, Lo, heads)


def test_causal_config2_full_size_sampled_rows():
    w = I.WORKLOADS["cfg2"]
    q, k, v = I.make_qkv(w)
    Og, Lg = run_gpu_general(w, q, k, v, causal=True)
    qd, kd, vd = oracle_operands(w, q, k, v)
    rng = np.random.default_rng(31)
    rows = np.sort(np.concatenate([rng.choice(w.N, size=160, replace=False), [0, 1, 63, 64, 127, 128, w.N - 1]]))
    rows = np.unique(rows)
    heads = [(0, 3), (2, 9), (3, 15)]
    Oo, Lo = A.direct_p_forward(qd, kd, vd, heads=heads, rows=rows, causal=True)
    check_heads(Og, Lg, Oo, Lo, heads, rows)


# ------------------------------------------------------------------ mixed map (p_map = HYBRID)
HYBRID_CASES = [
    ("cfg1", dict(), 0x1111, "ceil"),
    ("cfg1", dict(N=384, H=3), 0x5555, "ceil"),
    ("cfg1", dict(d=64, N=512), 0x7777, "ceil"),
    ("cfg3", dict(B=2, H=2, N=512), 0x5555, "ceil"),
    ("cfg3", dict(B=1, H=2, N=384, d=128), 0x1111, "thr16"),
    ("cfg4", dict(H=2, N=1024), 0x7777, "ceil"),
    ("cfg2", dict(B=2, H=3, N=2304), 0x5555, "thr16"),
]


@pytest.mark.parametrize("name,kw,mask,p_scale", HYBRID_CASES)
def test_hybrid_map_matches_oracle_elementwise(name, kw, mask, p_scale):
    """A fixed pattern of element pairs takes the exact map, the rest the affine classifier; both sides
    fix the pattern and the fp32 arithmetic, so the codes agree and the usual tolerances hold."""
    from paper_2609_04105_b200 import binding as Bd
    w = I.shrink(I.WORKLOADS[name], **kw)
    q, k, v = I.make_qkv(w)
    rule = Bd.PSCALE_THR16 if p_scale == "thr16" else Bd.PSCALE_CEIL
    Og, Lg = run_gpu_general(w, q, k, v, p_map=Bd.PMAP_HYBRID, exact_pairs=mask, p_scale_rule=rule)
    qd, kd, vd = oracle_operands(w, q, k, v)
    heads = [(b, h) for b in range(w.B) for h in range(w.H)]
    Oo, Lo = A.direct_p_forward(qd, kd, vd, heads=heads, p_map="hybrid", exact_pairs=mask, p_scale=p_scale)
    check_heads(Og, Lg, Oo, Lo, heads)


def test_hybrid_map_config2_full_size_sampled_rows():
    from paper_2609_04105_b200 import binding as Bd
    w = I.WORKLOADS["cfg2"]
    q, k, v = I.make_qkv(w)
    Og, Lg = run_gpu_general(w, q, k, v, p_map=Bd.PMAP_HYBRID, exact_pairs=0x5555)
    qd, kd, vd = oracle_operands(w, q, k, v)
    rng = np.random.default_rng(13)
    rows = np.sort(rng.choice(w.N, size=128, replace=False))
    heads = [(0, 3), (2, 9)]
    Oo, Lo = A.direct_p_forward(qd, kd, vd, heads=heads, rows=rows, p_map="hybrid", exact_pairs=0x5555)
    check_heads(Og, Lg, Oo, Lo, heads, rows)


def test_hybrid_map_rejects_per_head_factors():
    from paper_2609_04105_b200 import binding as Bd
    x = torch.randn((1, 2, 128, 64), device="cuda").bfloat16()
    q, k = Bd.fp4attn_quantize_nvfp4_per_head(x, Bd.ROLE_Q), Bd.fp4attn_quantize_nvfp4_per_head(x, Bd.ROLE_K)
    v = Bd.fp4attn_quantize(x, Bd.FMT_MXFP4, Bd.ROLE_V)
    with pytest.raises(Bd.Fp4AttnError):
        Bd.fp4attn_fwd(q, k, v, p_map=Bd.PMAP_HYBRID, exact_pairs=0x5555)


def test_hybrid_map_rejects_other_patterns_and_the_causal_mask():
    from paper_2609_04105_b200 import binding as Bd
    w = I.shrink(I.WORKLOADS["cfg1"], N=128)
    q, k, v = I.make_qkv(w)
    ops = [Bd.fp4attn_quantize(_dev(a), w.qk_fmt if r != Bd.ROLE_V else Bd.FMT_MXFP4, r)
           for a, r in ((q, Bd.ROLE_Q), (k, Bd.ROLE_K), (v, Bd.ROLE_V))]
    for kw in (dict(exact_pairs=0x0101), dict(exact_pairs=0), dict(exact_pairs=0x5555, causal=True)):
        with pytest.raises(Bd.Fp4AttnError):
            Bd.fp4attn_fwd(*ops, p_map=Bd.PMAP_HYBRID, **kw)


# ------------------------------------------------------------------ size limits
def test_longest_sequence_sampled_rows():
    """N = 65536 keys in one head (512 stages per work item, 2^16-key rows, the ring wraps 85 times):
    index arithmetic and the long-running row sum.  24 sampled rows of B1 H1 d128 against the oracle."""
    w = I.shrink(I.WORKLOADS["cfg1"], H=1, N=65536)
    q, k, v = I.make_qkv(w)
    Og, Lg = run_gpu(w, q, k, v)
    qd, kd, vd = oracle_operands(w, q, k, v)
    rng = np.random.default_rng(21)
    rows = np.sort(rng.choice(w.N, size=24, replace=False))
    rows[0], rows[-1] = 0, w.N - 1
    Oo, Lo = A.direct_p_forward(qd, kd, vd, heads=[(0, 0)], rows=rows)
    check_heads(Og, Lg, Oo, Lo, [(0, 0)], rows)


def test_many_small_heads_more_items_than_one_wave():
    """B*H = 1024 heads of N = 128: 1024 single-stage work items on 148 persistent CTAs (every item is an
    item boundary: Q double buffer, epilogue overlap, reference reset).  All heads checked."""
    w = I.shrink(I.WORKLOADS["cfg1"], B=8, H=128, N=128)
    q, k, v = I.make_qkv(w)
    Og, Lg = run_gpu(w, q, k, v)
    qd, kd, vd = oracle_operands(w, q, k, v)
    rng = np.random.default_rng(22)
    heads = [(int(b), int(h)) for b, h in zip(rng.integers(0, w.B, 48), rng.integers(0, w.H, 48))]
    Oo, Lo = A.direct_p_forward(qd, kd, vd, heads=heads)
    check_heads(Og, Lg, Oo, Lo, heads)


# ------------------------------------------------------------------ fixed row reference (the shiftless path)
FIXREF_CASES = [
    # name, shrink, map, causal, token counts, K/V group, reference
    ("cfg1", dict(), "ideal", False, None, 1, 0),
    ("cfg1", dict(N=640, H=3), "affine", False, None, 1, 0),
    ("cfg1", dict(N=512, H=4), "ideal", True, None, 2, 0),
    ("cfg1", dict(B=3, H=2, N=512), "affine", False, [512, 300, 77], 1, 5),
    ("cfg3", dict(B=2, H=2, N=768), "ideal", True, [700, 330], 1, -20),       # NVFP4 Q/K, d = 64
    ("cfg3", dict(B=2, H=2, N=512), "affine", False, None, 1, 0),
    ("cfg2", dict(B=2, H=3, N=2304), "ideal", False, None, 1, 0),             # d = 128, many stages
    ("cfg2", dict(B=2, H=3, N=2304), "affine", True, None, 1, 30),
]


@pytest.mark.parametrize("name,kw,p_map,causal,lens,group,ref", FIXREF_CASES)
def test_fixed_row_reference_matches_oracle_and_the_running_reference(name, kw, p_map, causal, lens, group, ref):
    """The shiftless path: a constant row reference, bytes published by the softmax warps, no rescale.  Against the
    oracle run with the same reference, and against this library's running reference: O bit for bit (codes do not
    depend on the reference; numerator and row sum differ by the same power of two), LSE to float32 rounding."""
    import parity
    from paper_2609_04105_b200 import binding as Bd
    w = I.shrink(I.WORKLOADS[name], **kw)
    q, k, v = I.make_qkv(w)
    k, v = np.ascontiguousarray(k[:, : w.H // group]), np.ascontiguousarray(v[:, : w.H // group])
    sl = None if lens is None else torch.tensor(lens, dtype=torch.int32, device="cuda")
    pm = Bd.PMAP_AFFINE if p_map == "affine" else Bd.PMAP_IDEAL
    Og, Lg = run_gpu_general(w, q, k, v, causal=causal, seq_len=sl, p_map=pm, fixed_reference=ref)
    Or, Lr = run_gpu_general(w, q, k, v, causal=causal, seq_len=sl, p_map=pm)
    fmt = "mx" if w.qk_fmt == I.FMT_MXFP4 else "nv"
    qd, kd, vd = Qz.quantize_qk(q, fmt), Qz.quantize_qk(k, fmt), Qz.quantize_v(v)
    for b in range(w.B):
        n = w.N if lens is None else lens[b]
        assert np.array_equal(Og[b, :, :n], Or[b, :, :n])
        assert np.abs(Lg[b, :, :n] - Lr[b, :, :n]).max() <= 1e-5 * max(1.0, np.abs(Lr[b, :, :n]).max())
        for h in range(w.H):
            okw = {} if lens is None else dict(kv_len=n)
            st = parity.compare_head(Og[b, h], Lg[b, h], qd, kd, vd, b, h, rows=np.arange(n), kv_group=group, causal=causal,
                                     p_map=p_map, fixed_reference=ref, **okw)
            assert st["lse_err"] <= parity.LSE_ABS, st


def test_fixed_row_reference_reports_logits_outside_its_range_and_rejects_other_options():
    """Config 4's rows reach |y| ~ 300 and differ by hundreds of octaves: no constant reference holds them, and the
    kernel must say so through the status word instead of returning numbers.  A reference far above Gaussian logits
    loses whole rows the same way."""
    from paper_2609_04105_b200 import binding as Bd
    w = I.shrink(I.WORKLOADS["cfg4"], H=2, N=1024)
    q, k, v = I.make_qkv(w)
    qg, kg = Bd.fp4attn_quantize(_dev(q), w.qk_fmt, Bd.ROLE_Q), Bd.fp4attn_quantize(_dev(k), w.qk_fmt, Bd.ROLE_K)
    vg = Bd.fp4attn_quantize(_dev(v), Bd.FMT_MXFP4, Bd.ROLE_V)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    Bd.fp4attn_fwd(qg, kg, vg, status=status, fixed_reference=0)
    torch.cuda.synchronize()
    assert int(status.item()) == Bd.ERR_RANGE
    status.zero_()
    Bd.fp4attn_fwd(qg, kg, vg, status=status)                     # the running reference takes the same input
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    w = I.shrink(I.WORKLOADS["cfg1"], N=256)
    q, k, v = I.make_qkv(w)
    qg, kg = Bd.fp4attn_quantize(_dev(q), w.qk_fmt, Bd.ROLE_Q), Bd.fp4attn_quantize(_dev(k), w.qk_fmt, Bd.ROLE_K)
    vg = Bd.fp4attn_quantize(_dev(v), Bd.FMT_MXFP4, Bd.ROLE_V)
    Bd.fp4attn_fwd(qg, kg, vg, status=status, fixed_reference=400)                  # every block below the byte range
    torch.cuda.synchronize()
    assert int(status.item()) == Bd.ERR_RANGE
    for kw in (dict(p_scale_rule=Bd.PSCALE_THR16), dict(p_map=Bd.PMAP_HYBRID, exact_pairs=0x5555), dict(fixed_reference=5000)):
        with pytest.raises(Bd.Fp4AttnError):
            Bd.fp4attn_fwd(qg, kg, vg, **{**dict(fixed_reference=0), **kw})


# ------------------------------------------------------------------ degenerate inputs
@pytest.mark.parametrize("causal", [False, True])
def test_degenerate_inputs_zero_queries_zero_values_identical_keys(causal):
    """Q = 0: every score is 0, every visible key gets the same code, O is the mean of the reconstructed V over the
    visible keys and LSE the log of their number.  V = 0: O is exactly 0.  Identical keys: the same.  Each against the
    closed form and against the oracle."""
    from paper_2609_04105_b200 import binding as Bd
    w = I.shrink(I.WORKLOADS["cfg1"], B=1, H=2, N=384)
    q, k, v = I.make_qkv(w)
    zero = np.zeros_like(q)
    vd = Qz.quantize_v(v)
    Vhat = np.swapaxes(Qz.dequantize(vd), -1, -2)                                  # [B, H, N, d]
    n_vis = (np.arange(w.N) + 1.0) if causal else np.full(w.N, float(w.N))
    mean_v = (np.cumsum(Vhat, axis=2) / n_vis[None, None, :, None]) if causal else np.broadcast_to(Vhat.mean(axis=2, keepdims=True), Vhat.shape)
    kk = np.ascontiguousarray(np.broadcast_to(k[:, :, :1], k.shape))               # every key equals key 0
    for qq, kx in ((zero, k), (q, kk)):
        Og, Lg = run_gpu_general(w, qq, kx, v, causal=causal)
        assert np.abs(Og - mean_v).max() <= 2.0 ** -8 * max(1.0, np.abs(mean_v).max()) + 1e-6        # bf16 rounding of O
        if qq is zero:
            assert np.abs(Lg - np.log(n_vis)[None, None]).max() <= 1e-3
        qd, kd = Qz.quantize_qk(qq, "mx"), Qz.quantize_qk(kx, "mx")
        heads = [(0, 0), (0, 1)]
        Oo, Lo = A.direct_p_forward(qd, kd, vd, heads=heads, causal=causal)
        check_heads(Og, Lg, Oo, Lo, heads)
    Og, Lg = run_gpu_general(w, q, k, zero, causal=causal)
    assert not Og.any() and np.isfinite(Lg).all()


# ------------------------------------------------------------------ metamorphic checks (no oracle involved)
@pytest.mark.parametrize("name,kw", [("cfg2", dict(B=2, H=3, N=1024)), ("cfg3", dict(B=2, H=2, N=768))])
def test_exact_rescaling_of_q_and_head_permutation_leave_the_bits_unchanged(name, kw):
    """Q times 2^k with the softmax scale times 2^-k is the same operator: MXFP4 moves the power into the scale bytes,
    NVFP4 into the encode factor, the float32 scores and the score constant scale exactly, so O and LSE must come out
    bit for bit.  And the (batch, head) units are independent: permuting the heads permutes the output."""
    from paper_2609_04105_b200 import binding as Bd
    w = I.shrink(I.WORKLOADS[name], **kw)
    q, k, v = I.make_qkv(w)
    scale = 1.0 / np.sqrt(w.d)

    def run(q, k, v, s):
        qg, kg = Bd.fp4attn_quantize(_dev(q), w.qk_fmt, Bd.ROLE_Q), Bd.fp4attn_quantize(_dev(k), w.qk_fmt, Bd.ROLE_K)
        vg = Bd.fp4attn_quantize(_dev(v), Bd.FMT_MXFP4, Bd.ROLE_V)
        st = torch.zeros(1, dtype=torch.int32, device="cuda")
        O, L = Bd.fp4attn_fwd(qg, kg, vg, softmax_scale=s, status=st)
        torch.cuda.synchronize()
        assert int(st.item()) == 0
        return O, L

    O0, L0 = run(q, k, v, scale)
    for kpow in (-3, 5):
        q2 = I.f32_to_bf16_bits(I.bf16_bits_to_f32(q) * np.float32(2.0 ** kpow))       # exact in bf16
        O1, L1 = run(q2, k, v, scale * 2.0 ** -kpow)
        assert torch.equal(O0, O1) and torch.equal(L0, L1)
    perm = np.random.default_rng(3).permutation(w.H)
    O2, L2 = run(np.ascontiguousarray(q[:, perm]), np.ascontiguousarray(k[:, perm]), np.ascontiguousarray(v[:, perm]), scale)
    idx = torch.from_numpy(perm).cuda()
    assert torch.equal(O0[:, idx], O2) and torch.equal(L0[:, idx], L2)      # (a tensor-wide NVFP4 factor does not move)


# ------------------------------------------------------------------ seeded random configurations
@pytest.mark.parametrize("seed", [1, 2, 3])
def test_random_configurations_match_oracle(seed):
    """Forty seeded draws of (d, Q/K format, N, B, heads, K/V head sharing, mask, code map, block-exponent rule,
    softmax scale, outlier channels, NVFP4 factors per tensor or per head, MXFP4 amplitude rule) per seed: every combination of options on small shapes, sampled rows of two
    heads each against the oracle, usual tolerances."""
    from paper_2609_04105_b200 import binding as Bd
    rng = np.random.default_rng(seed)
    for _ in range(40):
        d = int(rng.choice([64, 128])); nv = bool(rng.integers(0, 2))
        N = 128 * int(rng.integers(1, 9)); B = int(rng.integers(1, 4))
        group = int(rng.choice([1, 1, 2, 4])); Hkv = int(rng.integers(1, 4)); H = Hkv * group
        causal = bool(rng.integers(0, 2)); pm = int(rng.choice([0, 0, 1, 2])); thr = bool(rng.integers(0, 2))
        mask = int(rng.choice([0x1111, 0x5555, 0x7777]))
        if pm == 2:
            causal = False
        scale = float(rng.choice([0.0, 0.05, 0.3]))
        x = [rng.standard_normal((B, h, N, d)).astype(np.float32) for h in (H, Hkv, Hkv)]
        if rng.integers(0, 4) == 0:                              # outlier channels as in config 4
            ch = rng.choice(d, size=3, replace=False)
            x[0][..., ch] *= 20
            x[1][..., ch] *= 20
        bits = [I.f32_to_bf16_bits(a) for a in x]
        per_head = bool(rng.integers(0, 2)) and pm != 2           # NVFP4: one factor per (batch, head) unit (not with the mixed map)
        rule = int(rng.integers(0, 4))                            # MXFP4 amplitude rule of Q, K and V
        rname = ["ceil", "thr16", "floor", "mse"][rule]
        if nv:
            quant = Bd.fp4attn_quantize_nvfp4_per_head if per_head else (lambda t, role: Bd.fp4attn_quantize(t, Bd.FMT_NVFP4, role))
            ops = [quant(_dev(bits[0]), Bd.ROLE_Q), quant(_dev(bits[1]), Bd.ROLE_K), Bd.fp4attn_quantize(_dev(bits[2]), Bd.FMT_MXFP4, Bd.ROLE_V)]
        else:
            ops = [Bd.fp4attn_quantize_mxfp4_rule(_dev(bits[i]), role, rule) for i, role in enumerate((Bd.ROLE_Q, Bd.ROLE_K, Bd.ROLE_V))]
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        O, L = Bd.fp4attn_fwd(*ops, softmax_scale=scale, status=status, p_map=pm, p_scale_rule=int(thr), causal=causal,
                              exact_pairs=mask if pm == 2 else 0)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        if nv:
            qd, kd, vd = Qz.quantize_qk(bits[0], "nv", per_head=per_head), Qz.quantize_qk(bits[1], "nv", per_head=per_head), Qz.quantize_v(bits[2])
        else:
            qd, kd, vd = Qz.quantize_qk(bits[0], "mx", rname), Qz.quantize_qk(bits[1], "mx", rname), Qz.quantize_v(bits[2], rname)
        heads = [(int(rng.integers(0, B)), int(rng.integers(0, H))) for _ in range(2)]
        rows = np.sort(rng.choice(N, size=min(N, 48), replace=False))
        rows[0], rows[-1] = 0, N - 1
        okw = dict(p_map=["ideal", "affine", "hybrid"][pm], p_scale="thr16" if thr else "ceil", causal=causal, kv_group=group,
                   softmax_scale=(scale if scale > 0 else None))
        if pm == 2:
            okw["exact_pairs"] = mask
        Oo, Lo = A.direct_p_forward(qd, kd, vd, heads=heads, rows=rows, **okw)
        check_heads(O.float().cpu().numpy().astype(np.float64), L.cpu().numpy().astype(np.float64), Oo, Lo, heads, rows)


@pytest.mark.parametrize("seed", [21, 22])
def test_random_padded_configurations_match_oracle(seed):
    """Thirty seeded draws per seed of (d, Q/K format, N, B, heads, K/V head sharing, mask, code map, block-exponent
    rule, token counts per batch entry): sampled existing rows of two heads each against the oracle."""
    from paper_2609_04105_b200 import binding as Bd
    rng = np.random.default_rng(seed)
    for _ in range(30):
        d = int(rng.choice([64, 128])); nv = bool(rng.integers(0, 2))
        N = 128 * int(rng.integers(1, 9)); B = int(rng.integers(1, 5))
        group = int(rng.choice([1, 1, 2, 4])); Hkv = int(rng.integers(1, 4)); H = Hkv * group
        causal = bool(rng.integers(0, 2)); pm = int(rng.integers(0, 2))
        rule = int(rng.choice([Bd.PSCALE_CEIL, Bd.PSCALE_THR16, Bd.PSCALE_MSE])) if pm == 0 else int(rng.integers(0, 2))
        lens = [int(rng.choice([1, N, int(rng.integers(1, N + 1)), 32 * int(rng.integers(1, N // 32 + 1))])) for _ in range(B)]
        x = [rng.standard_normal((B, h, N, d)).astype(np.float32) for h in (H, Hkv, Hkv)]
        bits = [I.f32_to_bf16_bits(a) for a in x]
        fmt = Bd.FMT_NVFP4 if nv else Bd.FMT_MXFP4
        ops = [Bd.fp4attn_quantize(_dev(bits[0]), fmt, Bd.ROLE_Q), Bd.fp4attn_quantize(_dev(bits[1]), fmt, Bd.ROLE_K),
               Bd.fp4attn_quantize(_dev(bits[2]), Bd.FMT_MXFP4, Bd.ROLE_V)]
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        O, L = Bd.fp4attn_fwd(*ops, status=status, p_map=pm, p_scale_rule=rule, causal=causal,
                              seq_len=torch.tensor(lens, dtype=torch.int32, device="cuda"))
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        name = "nv" if nv else "mx"
        qd, kd, vd = Qz.quantize_qk(bits[0], name), Qz.quantize_qk(bits[1], name), Qz.quantize_v(bits[2])
        Og, Lg = O.float().cpu().numpy().astype(np.float64), L.cpu().numpy().astype(np.float64)
        okw = dict(p_map=["ideal", "affine"][pm], p_scale=["ceil", "thr16", "mse"][rule], causal=causal, kv_group=group, seq_len=lens)
        for _ in range(2):
            b, h = int(rng.integers(0, B)), int(rng.integers(0, H))
            n = lens[b]
            rows = np.unique(np.concatenate([[0, n - 1], rng.choice(n, size=min(n, 40), replace=False)]))
            Oo, Lo = A.direct_p_forward(qd, kd, vd, heads=[(b, h)], rows=rows, **okw)
            check_heads(Og, Lg, Oo, Lo, [(b, h)], rows)


@pytest.mark.parametrize("kw,group,causal", [(dict(B=2, H=4, N=512), 1, False), (dict(B=1, H=4, N=384, d=128), 2, True),
                                             (dict(B=2, H=6, N=256), 3, False)])
def test_nvfp4_per_head_factors_attention_matches_oracle(kw, group, causal):
    """NVFP4 Q, K with one encode factor per (batch, head) unit (heads scaled by 2^-6..2^6 so that the factors
    differ), also with grouped K/V heads (the key factor is the K/V head's) and the causal mask."""
    from paper_2609_04105_b200 import binding as Bd
    w = I.shrink(I.WORKLOADS["cfg3"], **kw)
    q, k, v = I.make_qkv(w)
    rng = np.random.default_rng(11)
    Hkv = w.H // group
    xq = Qz.bf16_bits_to_f64(q) * 2.0 ** rng.integers(-6, 7, size=(w.B, w.H, 1, 1))
    xk = Qz.bf16_bits_to_f64(k)[:, :Hkv] * 2.0 ** rng.integers(-6, 7, size=(w.B, Hkv, 1, 1))
    q2, k2 = I.f32_to_bf16_bits(xq.astype(np.float32)), I.f32_to_bf16_bits(xk.astype(np.float32))
    v2 = np.ascontiguousarray(v[:, :Hkv])
    # logits range from 2^-12 to 2^12 times the usual: flat rows as well as one-hot ones
    qd = Bd.fp4attn_quantize_nvfp4_per_head(_dev(q2), Bd.ROLE_Q)
    kd = Bd.fp4attn_quantize_nvfp4_per_head(_dev(k2), Bd.ROLE_K)
    vd = Bd.fp4attn_quantize(_dev(v2), Bd.FMT_MXFP4, Bd.ROLE_V)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    O, lse = Bd.fp4attn_fwd(qd, kd, vd, status=status, causal=causal)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    Og, Lg = O.float().cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64)
    oq, ok_ = Qz.quantize_qk(q2, "nv", per_head=True), Qz.quantize_qk(k2, "nv", per_head=True)
    heads = [(b, h) for b in range(w.B) for h in range(w.H)]
    Oo, Lo = A.direct_p_forward(oq, ok_, Qz.quantize_v(v2), heads=heads, causal=causal, kv_group=group)
    check_heads(Og, Lg, Oo, Lo, heads)


@pytest.mark.parametrize("growth,scale", [(1.0, 2.0), (3.0, 2.0), (-0.11, 2.0), (1.0, 0.02)])
def test_row_reference_raises_of_every_size(growth, scale):
    """Scores that climb (or fall) by whole binades from one 128-key stage to the next: the keys of stage s are
    scaled by 1 + growth * s, and the softmax scale puts a row's stage maximum near 90 log2 units at s = 0.
    growth 1: the row reference rises by ~90 octaves per stage (raise capped at 126 octaves, old terms kept);
    growth 3: by ~270 (old terms drop out entirely); negative growth: later blocks fall far below the reference
    (zero blocks); small scale: the ordinary lazy regime.  The oracle keeps an exact running integer reference."""
    from paper_2609_04105_b200 import binding as Bd
    w = I.shrink(I.WORKLOADS["cfg1"], N=1024)
    q, k, v = I.make_qkv(w)
    xk = Qz.bf16_bits_to_f64(k)
    s = (np.arange(w.N) // 128).astype(np.float64)
    xk = xk * (1.0 + growth * s)[None, None, :, None]
    k2 = I.f32_to_bf16_bits(xk.astype(np.float32))
    Og, Lg = run_gpu(w, q, k2, v, softmax_scale=scale)
    qd, kd, vd = oracle_operands(w, q, k2, v)
    heads = [(0, 0), (0, 1)]
    rows = np.arange(0, w.N, 7)
    Oo, Lo = A.direct_p_forward(qd, kd, vd, heads=heads, rows=rows, softmax_scale=scale)
    assert np.isfinite(Og).all() and np.isfinite(Lg).all()
    check_heads(Og, Lg, Oo, Lo, heads, rows)


# ------------------------------------------------------------------ two-query schedule (d = 64)
TWO_QUERY_CASES = [
    ("cfg3", dict(B=2, H=2, N=512), dict()),                                   # NVFP4 Q/K, exact map
    ("cfg3", dict(B=1, H=3, N=256), dict(p_map=1)),                            # one tile pair per head, affine map
    ("cfg3", dict(B=2, H=2, N=1024), dict(p_map=2, exact_pairs=0x5555)),       # mixed map
    ("cfg1", dict(d=64, N=768, H=5), dict(p_map=1)),                           # MXFP4 Q/K at d = 64, odd number of pairs
    ("cfg1", dict(d=64, N=512, H=4), dict(p_scale_rule=1)),                    # threshold rule
    ("cfg4", dict(d=64, H=2, N=1024), dict()),                                 # outlier channels: the row reference moves
    ("cfg3", dict(B=3, H=40, N=2304), dict(p_map=1)),                          # more tile pairs than one wave of thread blocks
]


@pytest.mark.parametrize("name,kw,okw", TWO_QUERY_CASES)
def test_two_query_schedule_matches_oracle_and_the_one_query_schedule(name, kw, okw):
    """Two query tiles per thread block sharing every K/V stage (d = 64): same codes, same accumulation order per
    row, so the output must equal the one-query schedule's bit for bit, and the oracle within the tolerances."""
    from paper_2609_04105_b200 import binding as Bd
    w = I.shrink(I.WORKLOADS[name], **kw)
    q, k, v = I.make_qkv(w)
    O1, L1 = run_gpu_general(w, q, k, v, **okw)
    O2, L2 = run_gpu_general(w, q, k, v, schedule=Bd.SCHEDULE_TWO_QUERY, **okw)
    assert np.array_equal(O1, O2) and np.array_equal(L1, L2)
    qd, kd, vd = oracle_operands(w, q, k, v)
    rng = np.random.default_rng(8)
    all_heads = [(b, h) for b in range(w.B) for h in range(w.H)]
    heads = [all_heads[i] for i in sorted(rng.choice(len(all_heads), size=min(4, len(all_heads)), replace=False))]
    rows = np.sort(rng.choice(w.N, size=min(w.N, 256), replace=False))
    rows[0], rows[-1] = 0, w.N - 1
    omap = {0: "ideal", 1: "affine", 2: "hybrid"}[okw.get("p_map", 0)]
    extra = dict(exact_pairs=okw["exact_pairs"]) if "exact_pairs" in okw else {}
    Oo, Lo = A.direct_p_forward(qd, kd, vd, heads=heads, rows=rows, p_map=omap,
                                p_scale="thr16" if okw.get("p_scale_rule") else "ceil", **extra)
    check_heads(O2, L2, Oo, Lo, heads, rows)


def test_two_query_schedule_grouped_kv_heads_and_config3_full_size():
    """Grouped K/V heads under the two-query schedule, and config 3 (B8 H16 N8192 d64) at full size: bit-identical to
    the one-query launch."""
    from paper_2609_04105_b200 import binding as Bd
    w = I.shrink(I.WORKLOADS["cfg3"], B=1, H=6, N=512)
    q, k, v = I.make_qkv(w)
    k, v = k[:, :2], v[:, :2]
    O1, L1 = run_gpu_general(w, q, k, v)
    O2, L2 = run_gpu_general(w, q, k, v, schedule=Bd.SCHEDULE_TWO_QUERY)
    assert np.array_equal(O1, O2) and np.array_equal(L1, L2)
    w = I.WORKLOADS["cfg3"]
    q, k, v = I.make_qkv(w)
    for okw in (dict(), dict(p_map=Bd.PMAP_AFFINE)):
        O1, L1 = run_gpu_general(w, q, k, v, **okw)
        O2, L2 = run_gpu_general(w, q, k, v, schedule=Bd.SCHEDULE_TWO_QUERY, **okw)
        assert np.array_equal(O1, O2) and np.array_equal(L1, L2)


def test_two_query_schedule_rejects_what_it_does_not_cover():
    from paper_2609_04105_b200 import binding as Bd
    for kw, okw in ((dict(N=256), dict()),                          # d = 128
                    (dict(d=64, N=384), dict()),                    # N not a multiple of 256
                    (dict(d=64, N=512), dict(causal=True))):
        w = I.shrink(I.WORKLOADS["cfg1"], **kw)
        q, k, v = I.make_qkv(w)
        with pytest.raises(Bd.Fp4AttnError):
            run_gpu_general(w, q, k, v, schedule=Bd.SCHEDULE_TWO_QUERY, **okw)


# ------------------------------------------------------------------ MSE-selected block exponent for P
@pytest.mark.parametrize("name,kw,causal", [("cfg1", dict(), False), ("cfg1", dict(d=64, N=512, H=3), False),
                                            ("cfg3", dict(B=2, H=2, N=512), False), ("cfg4", dict(H=2, N=1024), False),
                                            ("cfg2", dict(B=1, H=2, N=2304), True)])
def test_mse_block_exponent_matches_oracle_with_near_ties_taken_either_way(name, kw, causal):
    """Per block the better of the two neighbouring exponents by squared error.  The GPU forms 2^x with ex2.approx and
    sums in fp32, so a block whose two error sums almost tie may take the other exponent: whole heads are compared
    under the protocol that accepts a row only if it matches the oracle with some of its reported near-ties flipped."""
    import parity
    from paper_2609_04105_b200 import binding as Bd
    w = I.shrink(I.WORKLOADS[name], **kw)
    q, k, v = I.make_qkv(w)
    Og, Lg = run_gpu_general(w, q, k, v, p_scale_rule=Bd.PSCALE_MSE, causal=causal)
    qd, kd, vd = oracle_operands(w, q, k, v)
    failing = 0
    for b in range(w.B):
        for h in range(w.H):
            st = parity.compare_head(Og[b, h], Lg[b, h], qd, kd, vd, b, h, chunk=512, p_scale="mse", causal=causal)
            failing += st["rows_failing_strict"]
    print(f"{name}: rows that needed a flipped near-tie: {failing}")
    # the rule is a different operator from the ceiling: on the same inputs the outputs differ visibly
    Oc, _ = run_gpu_general(w, q, k, v, causal=causal)
    assert np.abs(Oc - Og).max() > 1e-2


def test_mse_block_exponent_rejects_other_maps_and_schedules():
    from paper_2609_04105_b200 import binding as Bd
    w = I.shrink(I.WORKLOADS["cfg1"], d=64, N=256)
    q, k, v = I.make_qkv(w)
    for kw in (dict(p_map=Bd.PMAP_AFFINE), dict(schedule=Bd.SCHEDULE_TWO_QUERY), dict(p_map=Bd.PMAP_HYBRID, exact_pairs=0x5555)):
        with pytest.raises(Bd.Fp4AttnError):
            run_gpu_general(w, q, k, v, p_scale_rule=Bd.PSCALE_MSE, **kw)


# ------------------------------------------------------------------ repeated launches of every kernel family
def test_every_kernel_family_is_deterministic_over_repeated_launches():
    """Races between the roles of a kernel (a slot reused too early, a missing fence) show up as run-to-run differences
    long before they show up as wrong averages: thirty launches of each family on a shape with many work items per CTA
    and an odd number of stages must return bit-identical O and LSE, with other kernels interleaved on the stream."""
    from paper_2609_04105_b200 import binding as Bd
    cases = [
        ("cfg2", dict(B=2, H=5, N=1152), dict()),                                    # one-query, exact map, d = 128
        ("cfg2", dict(B=2, H=5, N=1152), dict(p_map=Bd.PMAP_AFFINE)),
        ("cfg2", dict(B=2, H=5, N=1152), dict(causal=True)),
        ("cfg2", dict(B=2, H=5, N=1152), dict(p_scale_rule=Bd.PSCALE_MSE)),
        ("cfg4", dict(H=6, N=1152), dict()),                                         # the row reference moves
        ("cfg3", dict(B=2, H=5, N=1280), dict()),                                    # d = 64, NVFP4
        ("cfg3", dict(B=2, H=5, N=1280), dict(schedule=Bd.SCHEDULE_TWO_QUERY)),
        ("cfg3", dict(B=2, H=5, N=1280), dict(schedule=Bd.SCHEDULE_TWO_QUERY, p_map=Bd.PMAP_AFFINE)),
    ]
    noise = torch.empty(64 * 1024 * 1024, dtype=torch.uint8, device="cuda")
    for name, kw, okw in cases:
        w = I.shrink(I.WORKLOADS[name], **kw)
        q, k, v = I.make_qkv(w)
        ops = [Bd.fp4attn_quantize(_dev(q), w.qk_fmt, Bd.ROLE_Q), Bd.fp4attn_quantize(_dev(k), w.qk_fmt, Bd.ROLE_K),
               Bd.fp4attn_quantize(_dev(v), Bd.FMT_MXFP4, Bd.ROLE_V)]
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        O0, L0 = Bd.fp4attn_fwd(*ops, status=status, **okw)
        O0, L0 = O0.clone(), L0.clone()
        for r in range(30):
            if r % 3 == 0:
                noise.fill_(r)                                    # evict L2, shift the timing of the loads
            O, L = Bd.fp4attn_fwd(*ops, status=status, **okw)
            assert torch.equal(O, O0) and torch.equal(L, L0), (name, okw, r)
        assert int(status.item()) == 0
    # the FP8 P/V route
    w = I.shrink(I.WORKLOADS["cfg2"], B=2, H=5, N=1152)
    q, k, v = I.make_qkv(w)
    ops = [Bd.fp4attn_quantize(_dev(q), 0, Bd.ROLE_Q), Bd.fp4attn_quantize(_dev(k), 0, Bd.ROLE_K), Bd.fp4attn_quantize_v_e4m3(_dev(v))]
    for okw in (dict(), dict(causal=True)):
        O0, L0 = Bd.fp4attn_fwd(*ops, **okw)
        O0, L0 = O0.clone(), L0.clone()
        for r in range(30):
            if r % 3 == 0:
                noise.fill_(r)
            O, L = Bd.fp4attn_fwd(*ops, **okw)
            assert torch.equal(O, O0) and torch.equal(L, L0), ("fp8", okw, r)
