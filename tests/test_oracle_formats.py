"""Pins for oracle/formats.py against what the paper prints and what the formats fix."""
import os

import numpy as np
import pytest
import torch

from oracle import formats as F

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _golden_codebook():
    mags = bnds = None
    for line in open(os.path.join(GOLD, "e2m1_codebook.txt")):
        t = line.split()
        if t and t[0] == "magnitudes":
            mags = [float(v) for v in t[1:]]
        if t and t[0] == "boundaries":
            bnds = [float(v) for v in t[1:]]
    return mags, bnds


def test_codebook_matches_printed_values():
    mags, bnds = _golden_codebook()
    assert list(F.E2M1_VALUES) == mags
    assert list(F.E2M1_BOUNDARIES) == bnds
    # every boundary is the midpoint of two neighbouring magnitudes
    assert bnds == [(a + b) / 2 for a, b in zip(mags[:-1], mags[1:])]


def test_rounding_at_and_around_printed_boundaries():
    mags, bnds = _golden_codebook()
    for k, t in enumerate(bnds):
        lo, hi = k, k + 1
        assert F.e2m1_encode_mag(np.nextafter(t, 0.0)) == lo
        assert F.e2m1_encode_mag(np.nextafter(t, 10.0)) == hi
        even = lo if lo % 2 == 0 else hi          # mantissa bit is the low bit of the code
        assert F.e2m1_encode_mag(t) == even
    assert F.e2m1_encode_mag(6.0) == 7 and F.e2m1_encode_mag(1e30) == 7   # saturation


def test_exhaustive_bf16_times_scale_vs_nearest_search():
    """All 65536 bf16 patterns x several power-of-two scales against a brute-force search."""
    mags, _ = _golden_codebook()
    bits = np.arange(65536, dtype=np.uint32) << 16
    v = bits.view(np.float32)
    v = v[np.isfinite(v)].astype(np.float64)
    book = np.array(mags)
    for sh in (-3, -1, 0, 1, 2, 5):
        x = np.ldexp(v, sh)
        dist = np.abs(np.minimum(np.abs(x), 8.0)[:, None] - book[None, :])   # beyond 6: saturation
        best = dist.min(axis=1)
        # among equally near codes take the even one
        cand = dist == best[:, None]
        idx = np.where(cand[:, ::2].any(axis=1), 2 * np.argmax(cand[:, ::2], axis=1),
                       2 * np.argmax(cand[:, 1::2], axis=1) + 1)
        got = F.e2m1_encode(x)
        assert np.array_equal(got & 7, idx.astype(np.uint8))
        assert np.array_equal((got >> 3) == 1, (x < 0) & (idx > 0))
        assert np.array_equal(np.abs(F.e2m1_decode(got)), book[idx])


def test_e8m0_closed_forms():
    for e in range(-126, 128):
        assert F.e8m0_decode(e + 127) == 2.0 ** e
        assert F.ceil_log2(2.0 ** e) == e
        assert F.ceil_log2(np.nextafter(2.0 ** e, np.inf)) == e + 1
        assert F.ceil_log2(np.nextafter(2.0 ** e, 0)) == e
    assert F.ceil_log2(3.0) == 2 and F.ceil_log2(0.75) == 0


def test_e4m3_against_library_type():
    """Decode of all finite bytes and RNE encode of a dense grid against torch.float8_e4m3fn."""
    b = torch.arange(0, 127, dtype=torch.uint8)
    ref = b.view(torch.float8_e4m3fn).to(torch.float64).numpy()
    assert np.array_equal(F.e4m3_decode(b.numpy()), ref)
    assert F.e4m3_decode(0x7E) == 448.0 and F.e4m3_decode(0x01) == 2.0 ** -9
    rng = np.random.default_rng(0)
    x = np.concatenate([np.exp(rng.uniform(np.log(1e-4), np.log(448.0), 200000)),
                        (ref[:-1] + ref[1:]) / 2, ref])            # includes every tie point
    lib = torch.from_numpy(x).to(torch.float32).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    x32 = x.astype(np.float32).astype(np.float64)                   # what the library saw
    assert np.array_equal(F.e4m3_encode_unsigned(x32), lib)
    assert F.e4m3_encode_unsigned(1e6) == 0x7E                       # saturating, never NaN
    assert F.e4m3_encode_unsigned(2.0 ** -10) == 0                   # tie to even -> zero scale
    assert F.e4m3_encode_unsigned(np.nextafter(2.0 ** -10, 1)) == 1


def _p_range_rows():
    rows = {}
    for line in open(os.path.join(GOLD, "p_range_table.txt")):
        if line.startswith("#") or not line.strip():
            continue
        t = line.split()
        rows[(int(t[0]), t[1])] = [float(v) for v in t[2:]]
    return rows


def _gaussian_softmax(S, rows, seed):
    rng = np.random.default_rng(seed)
    d = 128
    q = rng.standard_normal((rows, d))
    k = rng.standard_normal((S, d))
    z = q @ k.T / np.sqrt(d)
    p = np.exp(z - z.max(axis=1, keepdims=True))
    p /= p.sum(axis=1, keepdims=True)
    return p, rng.standard_normal((S, d))


def _report(p, phat, zero_scale_frac, V):
    zero_payload = np.mean(phat == 0)
    lost = np.mean((p * (phat == 0)).sum(axis=1))
    pn = phat / phat.sum(axis=1, keepdims=True)
    rel = np.linalg.norm(pn - p) / np.linalg.norm(p)
    o, oh = p @ V, pn @ V
    cos = (o * oh).sum() / np.linalg.norm(o) / np.linalg.norm(oh)
    return zero_scale_frac, zero_payload, lost, rel, cos


@pytest.mark.parametrize("S", [1024, 4096])
def test_table_p_range_mxfp4_rows(S):
    """Exact Gaussian softmax -> N32 blocks -> alpha in {2^floor, 2^ceil} (the two amplitudes of
    Eq. "mx-scale", chosen per block by squared error) -> alpha*Q_E2M1(6p/alpha)/6, renormalised.
    Pins the E2M1 coder and the amplitude convention to the printed MXFP4 rows."""
    want = _p_range_rows()[(S, "MXFP4")]
    p, V = _gaussian_softmax(S, 256 if S == 1024 else 96, 1)
    pb = p.reshape(p.shape[0], S // 32, 32)
    a = pb.max(axis=2)
    up = F.ceil_log2(a)
    best = None
    for e in (up - 1, up):
        alpha = np.ldexp(1.0, e)[..., None]
        cand = alpha * F.e2m1_decode(F.e2m1_encode(6 * pb / alpha)) / 6
        err = ((cand - pb) ** 2).sum(axis=2, keepdims=True)
        best = (cand, err) if best is None else (np.where(err < best[1], cand, best[0]), np.minimum(err, best[1]))
    got = _report(p, best[0].reshape(p.shape), 0.0, V)
    assert got[0] == want[0]
    assert got[1] == pytest.approx(want[1], rel=0.03)       # zero payload
    assert got[2] == pytest.approx(want[2], rel=0.05)       # lost mass
    assert got[3] == pytest.approx(want[3], rel=0.03)       # P rel-L2
    assert got[4] == pytest.approx(want[4], abs=2e-3)       # PV cosine


@pytest.mark.parametrize("S,G", [(1024, 448.0), (4096, 448.0), (1024, 1.0), (4096, 1.0)])
def test_table_p_range_nvfp4_rows(S, G):
    """Eq. "nv-scale": S_B = Q_E4M3(G a_B/6), q = Q_E2M1(G p / S_B), p^ = S_B q / G on the
    table's matched N32 blocks.  Pins the E4M3 coder (incl. its underflow to a zero scale)."""
    want = _p_range_rows()[(S, "NVFP4_G448" if G == 448.0 else "NVFP4_G1")]
    p, V = _gaussian_softmax(S, 256 if S == 1024 else 96, 2)
    pb = p.reshape(p.shape[0], S // 32, 32)
    a = pb.max(axis=2)
    SB = F.e4m3_decode(F.e4m3_encode_unsigned(G * a / 6))
    safe = np.where(SB > 0, SB, 1.0)[..., None]
    phat = np.where(SB[..., None] > 0, safe * F.e2m1_decode(F.e2m1_encode(G * pb / safe)) / G, 0.0)
    got = _report(p, phat.reshape(p.shape), np.mean(SB == 0), V)
    if G == 1.0:
        assert got[0] == pytest.approx(want[0], abs=0.02 if S == 1024 else 0.003)   # zero scales
        assert got[1] == pytest.approx(want[1], abs=0.02)
    else:
        assert got[0] == 0.0
        assert got[1] == pytest.approx(want[1], rel=0.05)
        assert got[2] == pytest.approx(want[2], rel=0.06)
        assert got[3] == pytest.approx(want[3], rel=0.03)
        assert got[4] == pytest.approx(want[4], abs=2e-3)
