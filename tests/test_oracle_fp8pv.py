"""Pins for the FP8-P/V route of the oracle (oracle.formats.e4m3_encode, oracle.quantize.quantize_v_e4m3,
oracle.attention.fp8_pv_rows / fp8_pv_forward): the E4M3 grid itself, closed forms, brute force on inputs whose
probabilities are exactly representable, invariants, and the accuracy level the paper reports for FP8 P/V."""
import math

import numpy as np

from oracle import attention as A
from oracle import formats as F
from oracle import quantize as Qz
from paper_2609_04105_b200 import inputs as I


def _e4m3_values():
    """Table "fp4-formats": 1-4-3 float, bias 7, subnormals m * 2**-9, largest 448; written out independently."""
    vals = []
    for e in range(16):
        for m in range(8):
            if e == 15 and m == 7:
                continue                                    # the NaN code
            vals.append(m * 2.0 ** -9 if e == 0 else (1 + m / 8) * 2.0 ** (e - 7))
    return np.array(vals)


def test_e4m3_signed_coder_round_trips_the_grid_and_rounds_ties_to_even():
    vals = _e4m3_values()
    assert len(vals) == 127 and vals.max() == 448 and np.all(np.diff(vals) > 0)
    for s in (1.0, -1.0):
        byte = F.e4m3_encode(s * vals)
        assert np.array_equal(F.e4m3_decode(byte), s * vals + 0.0)
    assert F.e4m3_encode(np.array([-0.0, -1e-9]))[0] == 0 and F.e4m3_encode(np.array([-1e-9]))[0] == 0
    mid = (vals[:-1] + vals[1:]) / 2                         # exact ties: the neighbour with an even mantissa wins
    got = F.e4m3_decode(F.e4m3_encode(-mid))
    even = np.where((np.arange(126) % 2) == 0, vals[:-1], vals[1:])   # value k has mantissa parity k % 2 (k = 8e + m)
    assert np.array_equal(got, -even)
    just = np.nextafter(mid, np.inf)
    assert np.array_equal(F.e4m3_decode(F.e4m3_encode(just)), vals[1:])
    assert F.e4m3_decode(F.e4m3_encode(np.array([1e9, -1e9, 448.0, 465.0]))).tolist() == [448.0, -448.0, 448.0, 448.0]


def test_v_e4m3_quantizer_closed_forms_scaling_and_error_bound():
    w = I.shrink(I.WORKLOADS["cfg1"], H=3, N=256)
    _, _, v = I.make_qkv(w)
    vd = Qz.quantize_v_e4m3(v)
    x = Qz.bf16_bits_to_f64(v)
    assert vd["byte"].shape == (1, 3, w.d, w.N) and vd["G"].shape == (1, 3)
    for h in range(3):
        a = np.abs(x[0, h]).max()
        assert vd["G"][0, h] == np.float32(np.float32(448.0) / np.float32(a))
        i, j = np.unravel_index(np.abs(x[0, h]).argmax(), x[0, h].shape)
        assert vd["byte"][0, h, j, i] & 0x7F == 0x7E            # the unit's maximum lands on 448 (transposed position)
        vh = Qz.dequantize_v_e4m3(vd, 0, h).T
        err = np.abs(vh - x[0, h])
        assert np.all(err <= np.maximum(2.0 ** -4 * np.abs(x[0, h]), 2.0 ** -10 / vd["G"][0, h]) * (1 + 1e-6))
    # a unit scaled by a power of two: same bytes, the factor moves
    x2 = x.copy()
    x2[0, 1] *= 2.0 ** -9
    vd2 = Qz.quantize_v_e4m3(I.f32_to_bf16_bits(x2.astype(np.float32)))
    assert np.array_equal(vd2["byte"], vd["byte"]) and vd2["G"][0, 1] == vd["G"][0, 1] * 2.0 ** 9
    z = Qz.quantize_v_e4m3(np.zeros((1, 1, 128, 64), np.uint16))
    assert z["G"][0, 0] == 1 and not z["byte"].any()


def _brute(y, V):
    R, N = y.shape
    O = np.zeros((R, V.shape[1]))
    lse = np.zeros(R)
    for i in range(R):
        m = max(float(t) for t in y[i])
        den = sum(2.0 ** (float(t) - m) for t in y[i])
        for j in range(N):
            O[i] += 2.0 ** (float(y[i, j]) - m) / den * V[j]
        lse[i] = math.log(2.0) * (m + math.log2(den))
    return O, lse


def test_fp8_probabilities_that_are_representable_reproduce_exact_attention():
    """Scores mu - k - {0, log2 1.25, log2 1.5, log2 1.75} for k = 0..13 give 2**x on the E4M3 grid (up to the
    float32 rounding of the logarithms, far inside a rounding cell): FP8 P/V must equal base-2 softmax attention."""
    rng = np.random.default_rng(3)
    R, N, d = 5, 256, 6
    k = rng.integers(0, 14, size=(R, N))
    frac = np.log2(np.array([1.0, 1.25, 1.5, 1.75]))[rng.integers(0, 4, size=(R, N))]
    y = 7.0 - k - 1.0 + frac                                   # every value below the row maximum ...
    y[:, 17] = 7.0                                              # ... which is an integer, so mu = 7
    V = rng.standard_normal((N, d))
    O, lse, byte, mu = A.fp8_pv_rows(y.astype(np.float32), np.float32(1.0), V)
    Ob, lb = _brute(y.astype(np.float32).astype(np.float64), V)
    assert np.all(mu == 7) and np.abs(O - Ob).max() < 1e-6 and np.abs(lse - lb).max() < 1e-6
    assert np.array_equal(F.e4m3_decode(byte[:, 17]), np.full(R, 256.0))


def test_fp8_rows_constant_v_flush_order_independence_and_error_bound():
    rng = np.random.default_rng(4)
    R, N, d = 4, 512, 8
    y = (rng.standard_normal((R, N)) * 3).astype(np.float32)
    V = rng.standard_normal((N, d))
    O, lse, byte, mu = A.fp8_pv_rows(y, np.float32(1.0), np.full((N, d), -0.75))
    assert np.all(O == -0.75)                                   # same rounded values in numerator and denominator
    O, lse, byte, mu = A.fp8_pv_rows(y, np.float32(1.0), V)
    assert np.array_equal(mu, np.ceil(y.max(axis=1).astype(np.float64)))
    perm = rng.permutation(N)                                   # no tile order enters the definition
    O2, lse2, _, _ = A.fp8_pv_rows(y[:, perm], np.float32(1.0), V[perm])
    assert np.abs(O2 - O).max() < 1e-13 and np.abs(lse2 - lse).max() < 1e-13
    p = np.exp2(y.astype(np.float64) - mu[:, None])
    p8 = F.e4m3_decode(byte) / 256.0
    assert np.all(np.abs(p8 - p) <= np.maximum(2.0 ** -4 * p, 2.0 ** -18))     # three mantissa bits; subnormal step 2**-17
    y[0, :] = -30.0                                             # 2**(-30 - mu + 8) is far below 2**-10: flushed to zero
    y[0, 5] = 1.5
    O3, _, byte3, _ = A.fp8_pv_rows(y, np.float32(1.0), V)
    assert np.count_nonzero(byte3[0]) == 1 and np.abs(O3[0] - V[5]).max() < 1e-15
    O4, _, _, _ = A.fp8_pv_rows(y[:, :256], np.float32(1.0), V[:256], row_index=np.array([5, 40, 100, 255]))
    O5, _, _, _ = A.fp8_pv_rows(y[1:2, :41], np.float32(1.0), V[:41])              # causal row 40 sees keys 0..40
    assert np.abs(O4[1] - O5[0]).max() < 1e-13


def test_fp8_pv_accuracy_sits_where_the_paper_reports_it():
    """NVFP4 Q/K + FP8 P/V: the paper's controls report cosine 0.9897-0.9899 against its 16-bit reference; here,
    against unquantised fp64 attention on Gaussian inputs, it must land in that neighbourhood and well above the
    full-FP4 route on the same inputs."""
    w = I.shrink(I.WORKLOADS["cfg3"], B=1, H=2, N=1024, d=128)
    q, k, v = I.make_qkv(w)
    qd, kd = Qz.quantize_qk(q, "nv"), Qz.quantize_qk(k, "nv")
    O8, L8 = A.fp8_pv_forward(qd, kd, Qz.quantize_v_e4m3(v), heads=[(0, 1)])
    O4, _ = A.direct_p_forward(qd, kd, Qz.quantize_v(v), heads=[(0, 1)])
    x = [Qz.bf16_bits_to_f64(a[0, 1]) for a in (q, k, v)]
    O64, L64 = A.exact_attention(*x)
    cos = lambda a: float((a * O64).sum() / np.linalg.norm(a) / np.linalg.norm(O64))
    assert 0.985 < cos(O8[0]) < 0.995 and cos(O8[0]) > cos(O4[0]) + 0.01
    assert np.abs(L8[0] - L64).max() < 0.15                     # same normaliser up to the operand quantisation
    # grouped K/V heads read the shared head
    O2, _ = A.fp8_pv_forward(qd, {**kd, "nib": kd["nib"][:, 1:], "sf": kd["sf"][:, 1:]},
                             {**Qz.quantize_v_e4m3(v[:, 1:])}, heads=[(0, 1)], kv_group=2)
    assert np.abs(O2[0] - O8[0]).max() < 1e-13


def test_fp8_rows_of_a_padded_sequence_equal_the_rows_on_the_truncated_keys():
    """No block structure in this route: keys beyond the length are simply absent, for any length."""
    rng = np.random.default_rng(9)
    R, N, d = 5, 256, 8
    y = (rng.standard_normal((R, N)) * 2).astype(np.float32)
    V = rng.standard_normal((N, d))
    for n in (1, 31, 32, 100, 129, 256):
        O, lse, byte, mu = A.fp8_pv_rows(y, np.float32(1.0), V, kv_len=n)
        Ot, lt, bt, mt = A.fp8_pv_rows(y[:, :n], np.float32(1.0), V[:n])
        assert np.abs(O - Ot).max() < 1e-13 and np.abs(lse - lt).max() < 1e-13 and np.array_equal(mu, mt)
        assert np.array_equal(byte[:, :n], bt) and not byte[:, n:].any()
    w = I.shrink(I.WORKLOADS["cfg1"], B=2, H=1, N=256)
    q, k, v = I.make_qkv(w)
    qd, kd, v8 = Qz.quantize_qk(q, "mx"), Qz.quantize_qk(k, "mx"), Qz.quantize_v_e4m3(v)
    O, L = A.fp8_pv_forward(qd, kd, v8, seq_len=[256, 90], causal=True)
    O0, L0 = A.fp8_pv_forward(qd, kd, v8, causal=True)
    assert np.array_equal(O[0], O0[0]) and np.isnan(O[1, 90:]).all()
    assert np.array_equal(O[1, :90], O0[1, :90])                # causal rows below the length never saw the masked keys
