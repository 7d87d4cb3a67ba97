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
