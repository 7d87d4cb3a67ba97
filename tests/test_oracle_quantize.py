"""Pins for oracle/quantize.py: closed forms, error bounds, fixed points, byte layouts."""
import numpy as np

from oracle import formats as F
from oracle import quantize as Qz
from paper_2609_04105_b200 import inputs as I


def _bits(x):
    return I.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def test_mx_power_of_two_blocks_closed_form():
    # a block whose maximum is 2**k stores u = 127 + k and codes 6*v/2**k exactly
    for k in (-20, -3, 0, 1, 7, 40):
        blk = np.ldexp(np.array([1, -0.5, 0.25, 0.75, 0, -1] + [0.125] * 26, dtype=np.float64), k)
        nib, u = Qz.mx_quantize_lastdim(blk[None, :])
        assert u[0, 0] == 127 + k
        assert list(F.e2m1_decode(nib[0, :6])) == [6, -3, 1.5, 4, 0, -6]   # 4.5 ties to 4 (even)
        assert np.all(F.e2m1_decode(nib[0, 6:]) == 1.0)                      # 0.75 -> tie -> 1
    nib, u = Qz.mx_quantize_lastdim(np.zeros((1, 32)))
    assert u[0, 0] == 0 and not nib.any()


def test_mx_never_saturates_and_error_bound():
    w = I.WORKLOADS["cfg1"]
    q, _, _ = I.make_qkv(w)
    x = Qz.bf16_bits_to_f64(q)
    nib, u = Qz.mx_quantize_lastdim(x)
    alpha = F.e8m0_decode(u)
    xb = x.reshape(x.shape[:-1] + (-1, 32))
    ratio = np.abs(xb).max(axis=-1) / alpha
    assert np.all((ratio > 0.5) & (ratio <= 1.0))           # ceil rule: 6a/alpha in (3, 6]
    xh = Qz.mx_dequantize_lastdim(nib, u).reshape(xb.shape)
    t = 6 * np.abs(xb) / alpha[..., None]
    half_step = np.where(t <= 2, 0.25, np.where(t <= 4, 0.5, 1.0))   # E2M1 spacing 0.5 / 1 / 2
    assert np.all(np.abs(xh - xb) <= alpha[..., None] * half_step / 6 + 1e-300)
    # representable values are a fixed point of quantize -> reconstruct
    nib2, u2 = Qz.mx_quantize_lastdim(xh.reshape(x.shape))
    assert np.array_equal(Qz.mx_dequantize_lastdim(nib2, u2), xh.reshape(x.shape))
    # hardware-facing value is 6x the reconstruction
    assert np.array_equal(Qz.mx_dequantize_lastdim(nib, u, hw=True), 6 * xh.reshape(x.shape))


def test_nv_closed_forms():
    x = np.zeros((2, 32))
    x[0, :16] = np.linspace(-4, 4, 16)          # holds the tensor maximum 4
    x[0, 16:] = 1e-9                            # G*a/6 far below 2**-10 -> zero scale
    x[1, :16] = 2.0
    x[1, 16:] = [0.5] * 8 + [-0.25] * 8
    G = Qz.nv_tensor_scale(x)
    assert G == np.float32(2688.0) / np.float32(4.0)
    nib, sb = Qz.nv_quantize_lastdim(x, G)
    assert sb[0, 0] == 0x7E                     # a_B == a_T  ->  S_B = 448
    assert sb[0, 1] == 0 and not nib[0, 16:].any()       # zero scale: the block vanishes
    assert F.e4m3_decode(sb[1, 0]) == 224.0 and np.all(F.e2m1_decode(nib[1, :16]) == 6.0)
    assert F.e4m3_decode(sb[1, 1]) == 56.0
    assert list(F.e2m1_decode(nib[1, 16:])) == [6.0] * 8 + [-3.0] * 8
    xh = Qz.nv_dequantize_lastdim(nib, sb, G)
    assert np.allclose(xh[1], x[1], rtol=0, atol=0)
    assert Qz.nv_tensor_scale(np.zeros(4)) == 1.0


def test_nv_error_bound_on_gaussian():
    w = I.shrink(I.WORKLOADS["cfg3"], B=1, H=2, N=256)
    q, _, _ = I.make_qkv(w)
    qd = Qz.quantize_qk(q, "nv")
    x = Qz.bf16_bits_to_f64(q)
    xh = Qz.dequantize(qd)
    S = F.e4m3_decode(qd["sf"]) / float(qd["G"])            # decoded block scale
    xb, xhb = x.reshape(x.shape[:-1] + (-1, 16)), xh.reshape(x.shape[:-1] + (-1, 16))
    # the E4M3 scale is within 1/16 (half a mantissa step) of a_B/6, so |t| <= 6*(1+1/15)
    assert np.all(np.abs(xhb - xb) <= S[..., None] * 1.0 + 1e-12)
    assert np.linalg.norm(xh - x) / np.linalg.norm(x) < 0.11
    assert qd["sf"].max() == 0x7E


def test_v_is_blocked_along_keys_and_transposed():
    w = I.shrink(I.WORKLOADS["cfg1"], H=1, N=128)
    _, _, v = I.make_qkv(w)
    vd = Qz.quantize_v(v)
    assert vd["nib"].shape == (1, 1, 128, 128) and vd["sf"].shape == (1, 1, 128, 4)
    x = Qz.bf16_bits_to_f64(v)[0, 0]                       # [N, d]
    c, kb = 17, 2
    a = np.abs(x[32 * kb:32 * kb + 32, c]).max()
    assert vd["sf"][0, 0, c, kb] == 127 + F.ceil_log2(a)


def test_byte_layouts():
    nib = np.arange(16, dtype=np.uint8)[None, :]
    assert list(Qz.pack_nibbles(nib)[0]) == [0x10, 0x32, 0x54, 0x76, 0x98, 0xBA, 0xDC, 0xFE]
    assert list(Qz.strip_negative_zero(np.array([0x88, 0x18, 0x81], dtype=np.uint8))) == [0x00, 0x10, 0x01]
    rng = np.random.default_rng(0)
    sf = rng.integers(1, 255, size=(1, 2, 200, 6), dtype=np.uint8)
    sw = Qz.swizzle_scales(sf)
    assert sw.shape == (1, 2, 2 * 2 * 512)
    for r, c in [(0, 0), (31, 3), (32, 0), (127, 5), (128, 4), (199, 5)]:
        off = ((r // 128) * 2 + c // 4) * 512 + (r % 32) * 16 + ((r % 128) // 32) * 4 + c % 4
        assert sw[0, 1, off] == sf[0, 1, r, c]
    assert sw[0, 0].astype(int).sum() == sf[0, 0].astype(int).sum()      # padding is zero


def test_mx_amplitude_rules_against_exact_rational_arithmetic():
    """Eq. "mx-scale": alpha is one of the two powers of two next to the block maximum.  The three rules'
    exponents are checked against their definitions in exact integer arithmetic on every positive normal
    bf16 value with exponent -20..20: ceil(log2 a), floor(log2 a), floor(log2(1.6 a)) (8 a >= 5 2^j)."""
    from fractions import Fraction
    pats = np.array([(e << 7) | m for e in range(107, 148) for m in range(128)], dtype=np.uint16)
    a = Qz.bf16_bits_to_f64(pats)
    got = {r: Qz.mx_amplitude_exponent(a, r) for r in ("ceil", "floor", "thr16")}
    for i, v in enumerate(a):
        f = Fraction(float(v))
        fl = f.numerator.bit_length() - f.denominator.bit_length()
        if Fraction(2) ** fl > f:
            fl -= 1
        assert Fraction(2) ** fl <= f < Fraction(2) ** (fl + 1)
        assert got["floor"][i] == fl
        assert got["ceil"][i] == (fl if f == Fraction(2) ** fl else fl + 1)
        j = fl + 1 if 8 * f >= 5 * Fraction(2) ** (fl + 1) else fl      # 1.6 a >= 2^(fl+1)
        assert got["thr16"][i] == j
    # the default quantizer is the ceiling rule
    x = np.random.default_rng(0).standard_normal((3, 64)) * 3
    xb = Qz.bf16_bits_to_f64(I.f32_to_bf16_bits(x.astype(np.float32)))
    n0, u0 = Qz.mx_quantize_lastdim(xb)
    n1, u1 = Qz.mx_quantize_lastdim(xb, "ceil")
    assert np.array_equal(n0, n1) and np.array_equal(u0, u1)


def test_mx_amplitude_rules_closed_forms_and_saturation():
    """Hand-computed blocks.  Maximum 1.25: ceil -> alpha 2 (6v/alpha = 3.75 -> value 4, code index 6), thr16 -> alpha 2,
    floor -> alpha 1 (7.5 saturates at 6).  Maximum 1.2421875: thr16 keeps alpha 1 and saturates.  The block
    maximum's code is 6 for every block under floor, never saturated under ceil, and reconstruction error on
    Gaussian blocks orders thr16 < ceil < floor (the threshold rule is the paper's lower-error choice)."""
    blk = np.zeros((1, 32)); blk[0, 0] = 1.25; blk[0, 1] = -0.5
    for rule, u, c0 in (("ceil", 128, 6), ("thr16", 128, 6), ("floor", 127, 7)):
        nib, ub = Qz.mx_quantize_lastdim(blk, rule)
        assert ub[0, 0] == u and nib[0, 0] == c0, rule
    blk[0, 0] = 1.2421875
    for rule, u, c0 in (("ceil", 128, 6), ("thr16", 127, 7), ("floor", 127, 7)):
        nib, ub = Qz.mx_quantize_lastdim(blk, rule)
        assert ub[0, 0] == u and nib[0, 0] == c0, rule
    assert Qz.mx_quantize_lastdim(blk, "thr16")[0][0, 1] == 8 + 5          # -0.5 * 6 / 1 = -3 -> code index 5 (value 3), sign bit
    rng = np.random.default_rng(2)
    x = Qz.bf16_bits_to_f64(I.f32_to_bf16_bits(rng.standard_normal((64, 256)).astype(np.float32)))
    err = {}
    for rule in ("ceil", "thr16", "floor"):
        nib, u = Qz.mx_quantize_lastdim(x, rule)
        xr = Qz.mx_dequantize_lastdim(nib, u)
        err[rule] = np.linalg.norm(xr - x) / np.linalg.norm(x)
        top = (nib & 7).reshape(64, 8, 32).max(axis=-1)
        if rule == "floor":
            assert np.all(top == 7)
        if rule == "ceil":
            xb = np.abs(x).reshape(64, 8, 32)
            assert np.all(np.abs(xr).reshape(64, 8, 32).max(axis=-1) <= 2.0 ** np.ceil(np.log2(xb.max(axis=-1))))
    assert err["thr16"] < err["ceil"] < err["floor"]
    assert 0.10 < err["thr16"] < 0.12 and 0.17 < err["floor"] < 0.19


def test_mx_mse_rule_against_exact_rational_errors():
    """The MSE rule keeps, per block, whichever of the two amplitudes Eq. "mx-scale" allows reconstructs the
    block better.  Pins: (1) the chosen (byte, codes) always equal the floor rule's or the ceiling rule's output
    for that block; (2) the choice agrees with the two reconstruction errors computed in exact rational
    arithmetic from the dequantized values, except where those are within 1e-5 relative of each other (the rule
    sums in fp32); (3) hand-made blocks; (4) on Gaussian data its error is below the threshold rule's."""
    from fractions import Fraction
    rng = np.random.default_rng(11)
    x = Qz.bf16_bits_to_f64(I.f32_to_bf16_bits((rng.standard_normal((40, 128)) * rng.choice([1e-3, 1.0, 37.0], (40, 1))).astype(np.float32)))
    out = {r: Qz.mx_quantize_lastdim(x, r) for r in ("mse", "floor", "ceil")}
    xr = {r: Qz.mx_dequantize_lastdim(*out[r]) for r in out}
    picked_floor = 0
    for r in range(40):
        for b in range(4):
            sl = slice(32 * b, 32 * b + 32)
            is_f = out["mse"][1][r, b] == out["floor"][1][r, b] and np.array_equal(out["mse"][0][r, sl], out["floor"][0][r, sl])
            is_c = out["mse"][1][r, b] == out["ceil"][1][r, b] and np.array_equal(out["mse"][0][r, sl], out["ceil"][0][r, sl])
            assert is_f or is_c
            ef = sum((Fraction(float(p)) - Fraction(float(q))) ** 2 for p, q in zip(xr["floor"][r, sl], x[r, sl]))
            ec = sum((Fraction(float(p)) - Fraction(float(q))) ** 2 for p, q in zip(xr["ceil"][r, sl], x[r, sl]))
            if abs(ef - ec) > Fraction(1, 100000) * max(ef, ec):
                assert is_f == (ef < ec) or (is_f and is_c), (r, b, float(ef), float(ec))
            picked_floor += bool(is_f and not is_c)
    assert 20 < picked_floor < 140                                   # both amplitudes are in use
    # maximum 1.0078125, eight values 0.25.  alpha 1: 6.046875 -> 6 (d^2 = 0.0022), 1.5 exact.  alpha 2:
    # 0.75 is a tie -> 1.0 (even code), d = 0.25 eight times: the floor is far better
    blk = np.zeros((1, 32)); blk[0, 0] = 1.0078125; blk[0, 1:9] = 0.25
    nib, u = Qz.mx_quantize_lastdim(blk, "mse")
    assert u[0, 0] == 127 and nib[0, 0] == 7 and nib[0, 1] == 3 and nib[0, 9] == 0
    # maximum 1.5, three values 0.5 (exact on both grids).  alpha 1: 9 saturates at 6, d = 3 -> 9 units;
    # alpha 2: 4.5 -> 4 (tie to the even code), d = 0.5 -> 4 * 0.25 = 1 in the same units: the ceiling is kept
    blk = np.zeros((1, 32)); blk[0, 0] = 1.5; blk[0, 1:4] = 0.5
    nib, u = Qz.mx_quantize_lastdim(blk, "mse")
    assert u[0, 0] == 128 and nib[0, 0] == 6 and nib[0, 1] == 3
    # equal errors keep the ceiling: maximum 1.25 alone -> alpha 1: 7.5 -> 6, 2.25; alpha 2: 3.75 -> 4, 4 * 0.0625
    blk = np.zeros((1, 32)); blk[0, 0] = 1.25
    assert Qz.mx_quantize_lastdim(blk, "mse")[1][0, 0] == 128
    blk = np.zeros((1, 32)); blk[0, 0] = 2.0; blk[0, 5] = 0.3125         # power of two: only one candidate
    assert Qz.mx_quantize_lastdim(blk, "mse")[1][0, 0] == Qz.mx_quantize_lastdim(blk, "floor")[1][0, 0] == 128
    xg = Qz.bf16_bits_to_f64(I.f32_to_bf16_bits(np.random.default_rng(2).standard_normal((64, 256)).astype(np.float32)))
    err = {}
    for rule in ("mse", "thr16"):
        nib, u = Qz.mx_quantize_lastdim(xg, rule)
        err[rule] = np.linalg.norm(Qz.mx_dequantize_lastdim(nib, u) - xg) / np.linalg.norm(xg)
    assert err["mse"] < err["thr16"] and 0.10 < err["mse"] < 0.12


def test_mx_mse_rule_error_sum_is_order_pinned():
    """mx_block_error32 against its definition written out with Python floats rounded through float32 one
    operation at a time (left to right within groups of eight, groups as (g0 + g1) + (g2 + g3))."""
    import struct
    f32 = lambda v: struct.unpack("f", struct.pack("f", v))[0]
    rng = np.random.default_rng(3)
    xb = Qz.bf16_bits_to_f64(I.f32_to_bf16_bits(rng.standard_normal((6, 32)).astype(np.float32)))
    u = np.full((6,), 128, dtype=np.uint8)
    err, codes = Qz.mx_block_error32(xb, u)
    grid = [0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0]
    for r in range(6):
        g = []
        for j in range(4):
            acc = None
            for i in range(8):
                t = 6.0 * float(xb[r, 8 * j + i]) / 2.0
                q = min(grid, key=lambda c: (abs(abs(t) - c), grid.index(c) % 2))     # nearest, ties to the even code
                assert grid[int(codes[r, 8 * j + i]) & 7] == q
                d = abs(t) - q
                s = f32(d * d)
                acc = s if acc is None else f32(acc + s)
            g.append(acc)
        assert float(err[r]) == f32(f32(g[0] + g[1]) + f32(g[2] + g[3]))


def test_nv_per_head_factors_power_of_two_invariance_and_error():
    """Per-(batch, head) encode factors (Section "Pass the forward quantization into backward": per-head
    Q-K global factors).  (1) Scaling a head by 2^k leaves its codes and scale bytes untouched and moves only
    its factor, by exactly 2^-k; the other heads do not change at all.  (2) The tensor maximum's block of every
    head gets the largest scale byte.  (3) With head magnitudes 1 : 2^-20 one tensor-wide factor flushes
    the small head's blocks to zero scale, per-head factors keep every head inside the NVFP4 error bound."""
    w = I.shrink(I.WORKLOADS["cfg3"], B=2, H=3, N=128)
    q, _, _ = I.make_qkv(w)
    base = Qz.quantize_qk(q, "nv", per_head=True)
    assert base["G"].shape == (2, 3) and base["G"].dtype == np.float32
    x = Qz.bf16_bits_to_f64(q)
    for b in range(2):
        for h in range(3):
            assert base["G"][b, h] == np.float32(2688.0) / np.float32(np.abs(x[b, h]).max())
            assert base["sf"][b, h].max() == 0x7E
    scaled = x.copy()
    scaled[1, 2] *= 2.0 ** 5
    sd = Qz.quantize_qk(I.f32_to_bf16_bits(scaled.astype(np.float32)), "nv", per_head=True)
    assert np.array_equal(sd["nib"], base["nib"]) and np.array_equal(sd["sf"], base["sf"])
    want_G = base["G"].copy()
    want_G[1, 2] /= np.float32(32.0)
    assert np.array_equal(sd["G"], want_G)
    assert np.array_equal(Qz.dequantize(sd)[1, 2], Qz.dequantize(base)[1, 2] * 32.0)
    small = x.copy()
    small[0, 1] *= 2.0 ** -20
    bits = I.f32_to_bf16_bits(small.astype(np.float32))
    xs = Qz.bf16_bits_to_f64(bits)
    one, per = Qz.quantize_qk(bits, "nv"), Qz.quantize_qk(bits, "nv", per_head=True)
    rel = lambda qd, b, h: np.linalg.norm(Qz.dequantize(qd)[b, h] - xs[b, h]) / np.linalg.norm(xs[b, h])
    assert rel(one, 0, 1) > 0.9 and not one["sf"][0, 1].any()          # a_B G / 6 < 2^-10: every scale byte is zero
    for b in range(2):
        for h in range(3):
            assert rel(per, b, h) < 0.11
