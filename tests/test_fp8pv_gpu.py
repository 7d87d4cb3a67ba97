"""FP8 P/V route on the GPU: the E4M3 quantizer of V byte for byte, the attention forward within the usual
tolerances (relative Frobenius error <= 5e-3 and max-abs <= 2e-2 per (batch, head); LSE 1e-3 + 1e-5 |LSE|)."""
import numpy as np
import pytest
import torch

from oracle import attention as A
from oracle import quantize as Qz
from paper_2609_04105_b200 import inputs as I

pytestmark = pytest.mark.gpu
REL_FRO, MAX_ABS = 5e-3, 2e-2


def _dev(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


@pytest.mark.parametrize("name,kw", [("cfg1", dict()), ("cfg1", dict(d=64, N=384, H=3)), ("cfg4", dict(H=2, N=640)),
                                     ("cfg2", dict(B=2, H=5, N=2304))])
def test_e4m3_v_quantizer_bytes_match_oracle(name, kw):
    from paper_2609_04105_b200 import binding as Bd
    w = I.shrink(I.WORKLOADS[name], **kw)
    _, _, v = I.make_qkv(w)
    x = I.bf16_bits_to_f32(v)
    x[0, 0, 3, :] = 0.0                                        # a zero row, tiny and huge values inside one unit
    x[0, 0, 5, 1] = 3.0e-6
    x[0, w.H - 1] *= 2.0 ** -20                                # a unit far smaller than the others keeps its precision
    v = I.f32_to_bf16_bits(x)
    got = Bd.fp4attn_quantize_v_e4m3(_dev(v))
    want = Qz.quantize_v_e4m3(v)
    assert np.array_equal(got.G.cpu().numpy().reshape(w.B, w.H), want["G"])
    g = got.packed.cpu().numpy().reshape(want["byte"].shape)
    strip = lambda b: np.where((b & 0x7F) == 0, 0, b)           # the sign of a zero does not matter
    assert np.array_equal(strip(g), strip(want["byte"]))
    z = Bd.fp4attn_quantize_v_e4m3(torch.zeros((1, 1, 128, 64), dtype=torch.bfloat16, device="cuda"))
    assert float(z.G[0]) == 1.0 and not z.packed.any()


def _run(w, q, k, v, causal=False, group=1, softmax_scale=0.0):
    from paper_2609_04105_b200 import binding as Bd
    qg = Bd.fp4attn_quantize(_dev(q), w.qk_fmt, Bd.ROLE_Q)
    kg = Bd.fp4attn_quantize(_dev(k), w.qk_fmt, Bd.ROLE_K)
    vg = Bd.fp4attn_quantize_v_e4m3(_dev(v))
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    O, L = Bd.fp4attn_fwd(qg, kg, vg, status=status, causal=causal, softmax_scale=softmax_scale)
    torch.cuda.synchronize()
    assert int(status.item()) == 0, "kernel reported a bounded-wait timeout"
    return O.float().cpu().numpy().astype(np.float64), L.cpu().numpy().astype(np.float64)


def _check(w, q, k, v, Og, Lg, heads, rows=None, causal=False, group=1, softmax_scale=None):
    fmt = "mx" if w.qk_fmt == I.FMT_MXFP4 else "nv"
    qd, kd, v8 = Qz.quantize_qk(q, fmt), Qz.quantize_qk(np.ascontiguousarray(k), fmt), Qz.quantize_v_e4m3(np.ascontiguousarray(v))
    Oo, Lo = A.fp8_pv_forward(qd, kd, v8, heads=heads, rows=rows, causal=causal, kv_group=group, softmax_scale=softmax_scale)
    for n, (b, h) in enumerate(heads):
        g = Og[b, h] if rows is None else Og[b, h][rows]
        l = Lg[b, h] if rows is None else Lg[b, h][rows]
        rel = np.linalg.norm(g - Oo[n]) / np.linalg.norm(Oo[n])
        assert rel <= REL_FRO, f"head {(b, h)}: rel Frobenius {rel:.3e}"
        assert np.abs(g - Oo[n]).max() <= MAX_ABS, f"head {(b, h)}: max abs {np.abs(g - Oo[n]).max():.3e}"
        assert (np.abs(l - Lo[n]) - 1e-5 * np.abs(Lo[n])).max() <= 1e-3, f"head {(b, h)}: LSE"


CASES = [
    ("cfg1", dict(N=128), False, 1),
    ("cfg1", dict(), False, 1),
    ("cfg1", dict(N=384, H=3), False, 1),                  # odd number of stages: the sweeps change step parity
    ("cfg1", dict(d=64, N=512), False, 1),
    ("cfg3", dict(B=2, H=2, N=512), False, 1),             # NVFP4 Q/K, d = 64
    ("cfg3", dict(B=1, H=2, N=384, d=128), False, 1),
    ("cfg4", dict(H=2, N=1024), False, 1),                 # outlier channels: near one-hot rows, most bytes flushed
    ("cfg2", dict(B=2, H=3, N=2304), False, 1),            # the ring wraps many times, ragged wave
    ("cfg1", dict(N=640, H=3), True, 1),                   # causal
    ("cfg1", dict(N=512, H=4, d=64), True, 2),             # causal, grouped K/V heads
    ("cfg1", dict(N=384, H=6), False, 3),
]


@pytest.mark.parametrize("name,kw,causal,group", CASES)
def test_fp8_pv_attention_matches_oracle_elementwise(name, kw, causal, group):
    w = I.shrink(I.WORKLOADS[name], **kw)
    q, k, v = I.make_qkv(w)
    k, v = k[:, : w.H // group], v[:, : w.H // group]
    Og, Lg = _run(w, q, k, v, causal=causal, group=group)
    heads = [(b, h) for b in range(w.B) for h in range(w.H)]
    _check(w, q, k, v, Og, Lg, heads, causal=causal, group=group)


def test_fp8_pv_constant_v_scale_and_determinism():
    w = I.shrink(I.WORKLOADS["cfg1"], N=512)
    q, k, v = I.make_qkv(w)
    c = I.f32_to_bf16_bits(np.full((w.B, w.H, w.N, w.d), 1.75, dtype=np.float32))
    Og, _ = _run(w, q, k, c, softmax_scale=0.3)
    assert np.all(Og == 1.75)                                # same rounded probabilities in numerator and denominator
    O1, L1 = _run(w, q, k, v, softmax_scale=0.3)
    O2, L2 = _run(w, q, k, v, softmax_scale=0.3)
    assert np.array_equal(O1, O2) and np.array_equal(L1, L2)
    _check(w, q, k, v, O1, L1, [(0, 0), (0, 1)], softmax_scale=0.3)


def test_fp8_pv_config2_full_size_sampled_rows_and_many_small_heads():
    w = I.WORKLOADS["cfg2"]
    q, k, v = I.make_qkv(w)
    Og, Lg = _run(w, q, k, v)
    rng = np.random.default_rng(41)
    rows = np.sort(rng.choice(w.N, size=192, replace=False))
    rows[0], rows[-1] = 0, w.N - 1
    _check(w, q, k, v, Og, Lg, [(0, 3), (1, 8), (3, 15)], rows)
    w = I.shrink(I.WORKLOADS["cfg1"], B=4, H=96, N=128)      # 384 single-stage items: every item is an item boundary
    q, k, v = I.make_qkv(w)
    Og, Lg = _run(w, q, k, v)
    heads = [(int(b), int(h)) for b, h in zip(rng.integers(0, w.B, 24), rng.integers(0, w.H, 24))]
    _check(w, q, k, v, Og, Lg, heads)


FP8_SEQLEN_CASES = [
    ("cfg1", dict(B=3, H=2, N=512), [512, 300, 77], False, 1),
    ("cfg1", dict(B=4, H=2, N=384), [1, 32, 128, 383], False, 1),
    ("cfg1", dict(B=2, H=4, N=640), [129, 600], True, 2),
    ("cfg3", dict(B=2, H=2, N=768), [700, 330], True, 1),
    ("cfg2", dict(B=2, H=2, N=1024), [1000, 640], False, 1),
]


@pytest.mark.parametrize("name,kw,lens,causal,group", FP8_SEQLEN_CASES)
def test_fp8_pv_padded_sequences_match_oracle_on_the_rows_that_exist(name, kw, lens, causal, group):
    from paper_2609_04105_b200 import binding as Bd
    w = I.shrink(I.WORKLOADS[name], **kw)
    q, k, v = I.make_qkv(w)
    k, v = np.ascontiguousarray(k[:, : w.H // group]), np.ascontiguousarray(v[:, : w.H // group])
    qg, kg = Bd.fp4attn_quantize(_dev(q), w.qk_fmt, Bd.ROLE_Q), Bd.fp4attn_quantize(_dev(k), w.qk_fmt, Bd.ROLE_K)
    vg = Bd.fp4attn_quantize_v_e4m3(_dev(v))
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    O, L = Bd.fp4attn_fwd(qg, kg, vg, status=status, causal=causal, seq_len=torch.tensor(lens, dtype=torch.int32, device="cuda"))
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    Og, Lg = O.float().cpu().numpy().astype(np.float64), L.cpu().numpy().astype(np.float64)
    fmt = "mx" if w.qk_fmt == I.FMT_MXFP4 else "nv"
    qd, kd, v8 = Qz.quantize_qk(q, fmt), Qz.quantize_qk(k, fmt), Qz.quantize_v_e4m3(v)
    for b, n in enumerate(lens):
        heads = [(b, h) for h in range(w.H)]
        Oo, Lo = A.fp8_pv_forward(qd, kd, v8, heads=heads, rows=np.arange(n), causal=causal, kv_group=group, seq_len=lens)
        for i, (_, h) in enumerate(heads):
            g, l = Og[b, h][:n], Lg[b, h][:n]
            assert np.linalg.norm(g - Oo[i]) / np.linalg.norm(Oo[i]) <= REL_FRO and np.abs(g - Oo[i]).max() <= MAX_ABS
            assert (np.abs(l - Lo[i]) - 1e-5 * np.abs(Lo[i])).max() <= 1e-3
            last = min(w.N, (n + 127) // 128 * 128)
            assert np.isfinite(Og[b, h][:last]).all() and np.isfinite(Lg[b, h][:last]).all()
    O1, L1 = Bd.fp4attn_fwd(qg, kg, vg, status=status, causal=causal)
    O2, L2 = Bd.fp4attn_fwd(qg, kg, vg, status=status, causal=causal, seq_len=torch.full((w.B,), w.N, dtype=torch.int32, device="cuda"))
    assert torch.equal(O1, O2) and torch.equal(L1, L2)           # full lengths: the bits of the call without seq_len


def test_fp8_pv_rejects_the_fp4_only_options():
    from paper_2609_04105_b200 import binding as Bd
    w = I.shrink(I.WORKLOADS["cfg1"], N=128)
    q, k, v = I.make_qkv(w)
    qg, kg = Bd.fp4attn_quantize(_dev(q), 0, 0), Bd.fp4attn_quantize(_dev(k), 0, 1)
    vg = Bd.fp4attn_quantize_v_e4m3(_dev(v))
    for kw in (dict(p_map=Bd.PMAP_AFFINE), dict(p_scale_rule=Bd.PSCALE_THR16), dict(schedule=Bd.SCHEDULE_TWO_QUERY)):
        with pytest.raises(Bd.Fp4AttnError):
            Bd.fp4attn_fwd(qg, kg, vg, **kw)


@pytest.mark.parametrize("seed", [1, 2])
def test_fp8_pv_random_configurations_match_oracle(seed):
    """Thirty seeded draws of (d, Q/K format, N, B, heads, K/V head sharing, mask, softmax scale, outlier channels)
    per seed: sampled rows of two heads each against the oracle."""
    from paper_2609_04105_b200 import binding as Bd
    rng = np.random.default_rng(100 + seed)
    for _ in range(30):
        d = int(rng.choice([64, 128])); nv = bool(rng.integers(0, 2))
        N = 128 * int(rng.integers(1, 9)); B = int(rng.integers(1, 4))
        group = int(rng.choice([1, 1, 2, 4])); Hkv = int(rng.integers(1, 4)); H = Hkv * group
        causal = bool(rng.integers(0, 2)); scale = float(rng.choice([0.0, 0.05, 0.3]))
        x = [rng.standard_normal((B, h, N, d)).astype(np.float32) for h in (H, Hkv, Hkv)]
        if rng.integers(0, 4) == 0:
            ch = rng.choice(d, size=3, replace=False)
            x[0][..., ch] *= 20
            x[1][..., ch] *= 20
        bits = [I.f32_to_bf16_bits(a) for a in x]
        w = I.Workload("rand", 0, B, H, N, d, I.FMT_NVFP4 if nv else I.FMT_MXFP4)
        Og, Lg = _run(w, bits[0], bits[1], bits[2], causal=causal, group=group, softmax_scale=scale)
        heads = [(int(rng.integers(0, B)), int(rng.integers(0, H))) for _ in range(2)]
        rows = np.sort(rng.choice(N, size=min(N, 48), replace=False))
        rows[0], rows[-1] = 0, N - 1
        _check(w, bits[0], bits[1], bits[2], Og, Lg, heads, rows, causal=causal, group=group,
               softmax_scale=(scale if scale > 0 else None))
