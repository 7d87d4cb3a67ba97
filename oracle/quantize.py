"""Operand quantizers of the path (oracle side, test infrastructure only).

MXFP4 (Eq. "mx-scale", amplitude convention): a block of 32 values with maximum
magnitude a stores the power-of-two amplitude alpha = 2**ceil(log2 a) as the E8M0 byte
u = 127 + ceil(log2 a) and the codes q = Q_E2M1(6 v / alpha); a value is reconstructed
as alpha * q / 6.  Reading taken here: the ceiling of the two powers the paper allows,
so the block maximum lands in (3, 6] and never saturates; the floor and the threshold rule
alpha = 2**floor(log2(1.6 a)) are selectable (`rule`), and then maxima above alpha saturate.

NVFP4 (Table "fp4-formats", Eq. "nv-scale"): a block of 16 values stores
S_B = Q_E4M3(G a_B / 6) and q = Q_E2M1(G v / S_B); reconstruction S_B q / G.  Reading
taken here: one encode factor G = 448*6 / max|x| per tensor; the scale arithmetic is
carried in float32 in a fixed order so that a GPU can reproduce the bytes exactly.

Q and K are blocked along the head dimension (the contraction of QK^T); V is blocked
along the key index (the contraction of PV) and is emitted transposed, [.., d, N].

Layouts of the bytes handed to the attention kernel are restated at the end of the file
(packing two nibbles per byte, and the 128x4 scale atom the block-scaled tensor-core
instruction reads).
"""
from __future__ import annotations

import numpy as np

from .formats import (ceil_log2, e2m1_decode, e2m1_encode, e4m3_decode, e4m3_encode,
                      e4m3_encode_unsigned, e8m0_decode)

MX_BLOCK = 32
NV_BLOCK = 16


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    u = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


# --------------------------------------------------------------------------- MXFP4
def mx_amplitude_exponent(a: np.ndarray, rule: str) -> np.ndarray:
    """Exponent e of the amplitude alpha = 2**e for block maxima a > 0 (Eq. "mx-scale" allows either
    power of two next to a):  "ceil"  ceil(log2 a);  "floor"  floor(log2 a);
    "thr16"  floor(log2(1.6 a)), i.e. round up exactly when a / 2**floor(log2 a) >= 1.25.
    (The fourth rule of mx_quantize_lastdim, "mse", picks between floor and ceil per block.)"""
    m, k = np.frexp(a)                      # a = m 2**k, m in [0.5, 1): exact
    fl = k.astype(np.int64) - 1             # floor(log2 a)
    if rule == "floor":
        return fl
    if rule == "ceil":
        return fl + (m != 0.5)
    if rule == "thr16":
        return fl + (2.0 * m >= 1.25)
    raise ValueError(rule)


def mx_quantize_lastdim(x: np.ndarray, rule: str = "ceil"):
    """x float64 [..., L], L % 32 == 0, blocks of 32 along the last axis.

    Returns (nibbles uint8 [..., L], scale bytes uint8 [..., L/32]).  `rule` picks the amplitude
    (see mx_amplitude_exponent); values above it saturate at code 6.
    """
    L = x.shape[-1]
    assert L % MX_BLOCK == 0
    xb = x.reshape(x.shape[:-1] + (L // MX_BLOCK, MX_BLOCK))
    a = np.abs(xb).max(axis=-1)
    nz = a > 0
    a1 = np.where(nz, a, 1.0)
    if rule == "mse":
        # per block the better of the two neighbouring powers of two (Eq. "mx-scale" names both); the squared
        # error is taken in float32 in a fixed order (mx_block_error32) so that a GPU reproduces the choice;
        # the floor wins only if its error is strictly smaller
        uf = np.clip(mx_amplitude_exponent(a1, "floor") + 127, 1, 254).astype(np.uint8)
        uc = np.clip(mx_amplitude_exponent(a1, "ceil") + 127, 1, 254).astype(np.uint8)
        ef, cf = mx_block_error32(xb, uf)
        ec, cc = mx_block_error32(xb, uc)
        take_f = (uf != uc) & (ef < np.float32(4.0) * ec)       # ceil's error is in units four times larger
        u = np.where(take_f, uf, uc)
        codes = np.where(take_f[..., None], cf, cc)
    else:
        e = ceil_log2(a1) if rule == "ceil" else mx_amplitude_exponent(a1, rule)
        u = np.clip(e + 127, 1, 254).astype(np.uint8)
        codes = e2m1_encode(6.0 * xb / e8m0_decode(u)[..., None])
    u = np.where(nz, u, 0).astype(np.uint8)
    codes = np.where(nz[..., None], codes, 0).astype(np.uint8)
    return codes.reshape(x.shape), u


def mx_block_error32(xb: np.ndarray, u: np.ndarray):
    """Squared error of MXFP4 blocks [..., 32] under scale bytes u, in units of (alpha/6)**2, as float32 in
    a fixed order: d_i = 6 v_i/alpha - q_i (exact above the float32 subnormal range), s_i = fl32(d_i*d_i); the eight s_i of each group of eight
    consecutive elements are added left to right, then the four group sums as (g0 + g1) + (g2 + g3).
    Returns (error float32 [...], codes uint8 [..., 32])."""
    t = 6.0 * xb / e8m0_decode(u)[..., None]                   # exact, and exactly representable in float32
    codes = e2m1_encode(t)
    d = (t - e2m1_decode(codes)).astype(np.float32)
    inexact = d.astype(np.float64) != t - e2m1_decode(codes)    # only below the float32 normal range, where
    assert np.all(np.abs(t[inexact]) < 2.0 ** -126)             # fl32(d*d) is 0 whichever way d was rounded
    s = (d * d).astype(np.float32).reshape(d.shape[:-1] + (4, 8))
    g = s[..., 0]
    for i in range(1, 8):
        g = (g + s[..., i]).astype(np.float32)
    err = ((g[..., 0] + g[..., 1]).astype(np.float32) + (g[..., 2] + g[..., 3]).astype(np.float32)).astype(np.float32)
    return err, codes


def mx_dequantize_lastdim(nib: np.ndarray, u: np.ndarray, hw: bool = False) -> np.ndarray:
    """alpha*q/6 (hw=False) or the tensor-core-facing alpha*q (hw=True)."""
    L = nib.shape[-1]
    q = e2m1_decode(nib).reshape(nib.shape[:-1] + (L // MX_BLOCK, MX_BLOCK))
    alpha = np.where(u == 0, 0.0, e8m0_decode(u))
    v = q * alpha[..., None]
    if not hw:
        v = v / 6.0
    return v.reshape(nib.shape)


# --------------------------------------------------------------------------- NVFP4
def nv_tensor_scale(x: np.ndarray) -> np.float32:
    """Encode factor G = fl32(2688 / max|x|) (G = 1 for an all-zero tensor)."""
    aT = np.float32(np.abs(x).max())
    if aT == 0:
        return np.float32(1.0)
    return np.float32(np.float32(2688.0) / aT)


def nv_quantize_lastdim(x: np.ndarray, G: np.float32):
    """x float64 holding bf16 values, [..., L], L % 16 == 0.

    float32 steps, in this order:  t = fl32(fl32(a_B * G) / 6);  S_B = Q_E4M3(t);
    r = fl32(G / S_B);  q = Q_E2M1(fl32(|v| * r)).  S_B == 0 makes the block vanish.
    Returns (nibbles [..., L], scale bytes [..., L/16]).
    """
    L = x.shape[-1]
    assert L % NV_BLOCK == 0
    G = np.float32(G)
    xb = x.reshape(x.shape[:-1] + (L // NV_BLOCK, NV_BLOCK)).astype(np.float32)
    a = np.abs(xb).max(axis=-1)
    t = (a * G).astype(np.float32) / np.float32(6.0)
    sbyte = e4m3_encode_unsigned(t.astype(np.float64))
    S = e4m3_decode(sbyte).astype(np.float32)
    with np.errstate(divide="ignore"):
        r = np.where(S > 0, G / np.where(S > 0, S, np.float32(1)), np.float32(0)).astype(np.float32)
    scaled = (np.abs(xb) * r[..., None]).astype(np.float32)
    codes = e2m1_encode(np.copysign(scaled.astype(np.float64), xb.astype(np.float64)))
    codes = np.where((S > 0)[..., None], codes, 0).astype(np.uint8)
    return codes.reshape(x.shape), sbyte


def nv_dequantize_lastdim(nib: np.ndarray, sbyte: np.ndarray, G=None, hw: bool = False) -> np.ndarray:
    """S_B*q/G (hw=False) or the tensor-core-facing S_B*q (hw=True)."""
    L = nib.shape[-1]
    q = e2m1_decode(nib).reshape(nib.shape[:-1] + (L // NV_BLOCK, NV_BLOCK))
    v = q * e4m3_decode(sbyte)[..., None]
    if not hw:
        G = np.asarray(G, dtype=np.float64)                      # one factor, or one per (batch, head) [B, H]
        v = v / G.reshape(G.shape + (1,) * (v.ndim - G.ndim))
    return v.reshape(nib.shape)


# --------------------------------------------------------------------------- roles
def quantize_qk(bits: np.ndarray, fmt: str, rule: str = "ceil", per_head: bool = False):
    """Q or K, bf16 bit patterns [B,H,N,d] -> dict(nib [B,H,N,d], sf [B,H,N,d/blk], G).

    NVFP4: G is one encode factor for the whole tensor, or with per_head one per (batch, head) unit,
    float32 [B, H], each taken from that unit's own maximum (Section "Pass the forward quantization into
    backward" saves per-head Q-K global factors): every unit is then quantized as if it were a tensor."""
    x = bf16_bits_to_f64(bits)
    if fmt == "mx":
        nib, sf = mx_quantize_lastdim(x, rule)
        return {"nib": nib, "sf": sf, "G": None, "fmt": "mx"}
    if per_head:
        B, H = x.shape[:2]
        G = np.empty((B, H), dtype=np.float32)
        nib = np.empty(x.shape, dtype=np.uint8)
        sf = np.empty(x.shape[:-1] + (x.shape[-1] // NV_BLOCK,), dtype=np.uint8)
        for b in range(B):
            for h in range(H):
                G[b, h] = nv_tensor_scale(x[b, h])
                nib[b, h], sf[b, h] = nv_quantize_lastdim(x[b, h], G[b, h])
        return {"nib": nib, "sf": sf, "G": G, "fmt": "nv"}
    G = nv_tensor_scale(x)
    nib, sf = nv_quantize_lastdim(x, G)
    return {"nib": nib, "sf": sf, "G": G, "fmt": "nv"}


def quantize_v(bits: np.ndarray, rule: str = "ceil"):
    """V bf16 [B,H,N,d] -> MXFP4 of V^T: dict(nib [B,H,d,N], sf [B,H,d,N/32]), blocks of 32 keys."""
    xt = np.ascontiguousarray(np.swapaxes(bf16_bits_to_f64(bits), -1, -2))
    nib, sf = mx_quantize_lastdim(xt, rule)
    return {"nib": nib, "sf": sf, "G": None, "fmt": "mx"}


def quantize_v_e4m3(bits: np.ndarray):
    """V bf16 [B,H,N,d] -> E4M3 bytes of V^T, dict(byte [B,H,d,N] uint8, G float32 [B,H], fmt "e4m3").

    The FP8 value operand of the FP8-P/V route (Section "Training stability selects FP8 P/V": V is kept in E4M3 there); the
    paper gives no scale rule, reading taken here: one encode factor per (batch, head) unit, like the per-head
    NVFP4 factors, G = fl32(448 / max|V[b,h]|) (1 for an all-zero unit), byte = Q_E4M3(fl32(v * G)) round to nearest
    even; a value is reconstructed as decode(byte) / G."""
    x = bf16_bits_to_f64(bits)
    B, H = x.shape[:2]
    a = np.abs(x).reshape(B, H, -1).max(axis=2).astype(np.float32)
    with np.errstate(divide="ignore"):
        G = np.where(a > 0, np.float32(448.0) / np.where(a > 0, a, np.float32(1)), np.float32(1)).astype(np.float32)
    t = (x.astype(np.float32) * G[:, :, None, None]).astype(np.float32)
    byte = e4m3_encode(t.astype(np.float64))
    return {"byte": np.ascontiguousarray(np.swapaxes(byte, -1, -2)), "G": G, "fmt": "e4m3"}


def dequantize_v_e4m3(vd: dict, b: int, h: int) -> np.ndarray:
    """Reconstructed V^T of one unit, [d, N] float64."""
    return e4m3_decode(vd["byte"][b, h]) / np.float64(vd["G"][b, h])


def dequantize(qd: dict, hw: bool = False) -> np.ndarray:
    if qd["fmt"] == "mx":
        return mx_dequantize_lastdim(qd["nib"], qd["sf"], hw=hw)
    return nv_dequantize_lastdim(qd["nib"], qd["sf"], qd["G"], hw=hw)


# --------------------------------------------------------------------------- byte layouts
def pack_nibbles(nib: np.ndarray) -> np.ndarray:
    """[..., L] nibbles -> [..., L/2] bytes; element 2k in bits 0-3, element 2k+1 in bits 4-7."""
    return (nib[..., 0::2] | (nib[..., 1::2] << 4)).astype(np.uint8)


def strip_negative_zero(packed: np.ndarray) -> np.ndarray:
    """Map nibble 0x8 (-0) to 0x0 so that byte comparisons ignore the sign of a zero code."""
    lo = packed & 0x0F
    hi = packed >> 4
    lo = np.where(lo == 8, 0, lo)
    hi = np.where(hi == 8, 0, hi)
    return (lo | (hi << 4)).astype(np.uint8)


def swizzle_scales(sf: np.ndarray) -> np.ndarray:
    """Scale bytes [B,H,R,C] -> flat atoms [B,H, ceil(R/128)*ceil(C/4)*512].

    Atom (rt, ct) covers rows 128*rt..+127 and scale columns 4*ct..+3 and starts at byte
    (rt*ceil(C/4) + ct)*512; inside it row r, column c sits at (r%32)*16 + (r%128)//32*4 + c%4.
    Padding bytes are zero.
    """
    B, H, R, C = sf.shape
    RT, CT = -(-R // 128), -(-C // 4)
    pad = np.zeros((B, H, RT * 128, CT * 4), dtype=np.uint8)
    pad[:, :, :R, :C] = sf
    # [B,H,RT, r_hi(4), r_lo(32), CT, c(4)] -> [B,H,RT,CT, r_lo, r_hi, c]
    v = pad.reshape(B, H, RT, 4, 32, CT, 4).transpose(0, 1, 2, 5, 4, 3, 6)
    return np.ascontiguousarray(v).reshape(B, H, RT * CT * 512)
