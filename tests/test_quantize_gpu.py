"""Kernel (a): the CUDA quantizer must reproduce the oracle's bytes exactly (sign of zero aside)."""
import numpy as np
import pytest
import torch

from oracle import quantize as Qz
from paper_2609_04105_b200 import inputs as I

pytestmark = pytest.mark.gpu


def _dev(bits):
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def _check_operand(got, want, role):
    packed = got.packed.cpu().numpy()
    want_packed = Qz.pack_nibbles(want["nib"]).reshape(-1)
    assert np.array_equal(Qz.strip_negative_zero(packed), Qz.strip_negative_zero(want_packed)), "codes differ"
    want_sf = Qz.swizzle_scales(want["sf"]).reshape(-1)
    assert np.array_equal(got.scales.cpu().numpy(), want_sf), "scale bytes differ"
    if want["G"] is not None:
        assert got.G.cpu().numpy()[0] == want["G"]


CASES = [
    ("cfg1", dict()),
    ("cfg1", dict(d=64, N=384, H=3)),
    ("cfg3", dict(B=2, H=2, N=512)),
    ("cfg3", dict(B=1, H=2, N=256, d=128)),
    ("cfg4", dict(H=2, N=640)),
]


@pytest.mark.parametrize("name,kw", CASES)
def test_quantizer_bytes_match_oracle(name, kw):
    from paper_2609_04105_b200 import binding as Bd
    w = I.shrink(I.WORKLOADS[name], **kw)
    q, k, v = I.make_qkv(w)
    fmt = "mx" if w.qk_fmt == I.FMT_MXFP4 else "nv"
    for bits, role in ((q, Bd.ROLE_Q), (k, Bd.ROLE_K)):
        got = Bd.fp4attn_quantize(_dev(bits), w.qk_fmt, role)
        _check_operand(got, Qz.quantize_qk(bits, fmt), role)
    got = Bd.fp4attn_quantize(_dev(v), Bd.FMT_MXFP4, Bd.ROLE_V)
    _check_operand(got, Qz.quantize_v(v), Bd.ROLE_V)


def test_quantizer_edge_values():
    """Zero blocks, huge and tiny magnitudes, exact ties, negative zero."""
    from paper_2609_04105_b200 import binding as Bd
    rng = np.random.default_rng(3)
    x = rng.standard_normal((1, 1, 128, 128)).astype(np.float32)
    x[0, 0, 0, :32] = 0.0
    x[0, 0, 1, :32] = -0.0
    x[0, 0, 2, :] *= 1e30
    x[0, 0, 3, :] *= 1e-30
    x[0, 0, 4, :32] = np.array([1, 0.75, 0.625, 0.4375, 0.125, 1 / 24, -0.875, 0.5] * 4)   # ties of 6v
    x[0, 0, 5, 0] = 3.0e38
    x[0, 0, 6, :] = 2.0 ** -130
    bits = I.f32_to_bf16_bits(x)
    for fmt, name in ((Bd.FMT_MXFP4, "mx"), (Bd.FMT_NVFP4, "nv")):
        got = Bd.fp4attn_quantize(_dev(bits), fmt, Bd.ROLE_Q)
        _check_operand(got, Qz.quantize_qk(bits, name), Bd.ROLE_Q)
    got = Bd.fp4attn_quantize(_dev(bits), Bd.FMT_MXFP4, Bd.ROLE_V)
    _check_operand(got, Qz.quantize_v(bits), Bd.ROLE_V)
    z = np.zeros((1, 1, 128, 64), dtype=np.uint16)
    got = Bd.fp4attn_quantize(_dev(z), Bd.FMT_NVFP4, Bd.ROLE_K)
    _check_operand(got, Qz.quantize_qk(z, "nv"), Bd.ROLE_K)


def test_full_size_quantizer_sampled(tmp_path):
    """Config 2's full tensor: every scale byte and a random sample of rows against the oracle."""
    from paper_2609_04105_b200 import binding as Bd
    w = I.WORKLOADS["cfg2"]
    q, _, v = I.make_qkv(w)
    got = Bd.fp4attn_quantize(_dev(q), Bd.FMT_MXFP4, Bd.ROLE_Q)
    want = Qz.quantize_qk(q, "mx")
    _check_operand(got, want, Bd.ROLE_Q)
    got = Bd.fp4attn_quantize(_dev(v), Bd.FMT_MXFP4, Bd.ROLE_V)
    _check_operand(got, Qz.quantize_v(v), Bd.ROLE_V)


def test_full_size_nvfp4_quantizer_all_bytes():
    """Config 3's full Q tensor (B8 H16 N8192 d64: 2^26 elements, 2^23 sixteen-byte groups, so every block of
    the tensor-wide amax pass walks its strided loop several times): encode factor, every scale byte and
    every code against the oracle; then the per-(batch, head) variant on the same tensor."""
    from paper_2609_04105_b200 import binding as Bd
    w = I.WORKLOADS["cfg3"]
    q, _, _ = I.make_qkv(w)
    x = _dev(q)
    got = Bd.fp4attn_quantize(x, Bd.FMT_NVFP4, Bd.ROLE_Q)
    _check_operand(got, Qz.quantize_qk(q, "nv"), Bd.ROLE_Q)
    got = Bd.fp4attn_quantize_nvfp4_per_head(x, Bd.ROLE_Q)
    want = Qz.quantize_qk(q, "nv", per_head=True)
    assert np.array_equal(got.G.cpu().numpy().reshape(w.B, w.H), want["G"])
    assert np.array_equal(Qz.strip_negative_zero(got.packed.cpu().numpy()),
                          Qz.strip_negative_zero(Qz.pack_nibbles(want["nib"]).reshape(-1)))
    assert np.array_equal(got.scales.cpu().numpy(), Qz.swizzle_scales(want["sf"]).reshape(-1))


RULES = [("ceil", 0), ("thr16", 1), ("floor", 2), ("mse", 3)]


@pytest.mark.parametrize("rule,code", RULES)
@pytest.mark.parametrize("name,kw", [("cfg1", dict()), ("cfg1", dict(d=64, N=384, H=3)), ("cfg4", dict(H=2, N=640))])
def test_mx_amplitude_rules_match_oracle(name, kw, rule, code):
    """Eq. "mx-scale" with either neighbouring power of two: bytes and codes bit for bit, all three roles."""
    from paper_2609_04105_b200 import binding as Bd
    w = I.shrink(I.WORKLOADS[name], **kw)
    q, k, v = I.make_qkv(w)
    for bits, role in ((q, Bd.ROLE_Q), (k, Bd.ROLE_K)):
        got = Bd.fp4attn_quantize_mxfp4_rule(_dev(bits), role, code)
        _check_operand(got, Qz.quantize_qk(bits, "mx", rule), role)
    got = Bd.fp4attn_quantize_mxfp4_rule(_dev(v), Bd.ROLE_V, code)
    _check_operand(got, Qz.quantize_v(v, rule), Bd.ROLE_V)
    if rule == "ceil":                                      # the default entry point writes the same bytes
        ref = Bd.fp4attn_quantize(_dev(q), Bd.FMT_MXFP4, Bd.ROLE_Q)
        again = Bd.fp4attn_quantize_mxfp4_rule(_dev(q), Bd.ROLE_Q, code)
        assert torch.equal(ref.packed, again.packed) and torch.equal(ref.scales, again.scales)


@pytest.mark.parametrize("rule,code", RULES)
def test_mx_amplitude_rules_edge_values(rule, code):
    """Maxima exactly on the threshold (significand 1.25), just below it, powers of two, saturating values."""
    from paper_2609_04105_b200 import binding as Bd
    rng = np.random.default_rng(5)
    x = (rng.standard_normal((1, 1, 128, 128)) * 0.1).astype(np.float32)
    x[0, 0, 0, 0] = 1.25          # threshold: rounds up under thr16
    x[0, 0, 1, 0] = 1.2421875     # largest bf16 below it: stays
    x[0, 0, 2, 0] = -2.0          # power of two: amplitude 2 under every rule
    x[0, 0, 3, 0] = 1.9921875     # largest significand
    x[0, 0, 4, :32] = 0.0
    x[0, 0, 5, :] *= 1e30
    x[0, 0, 6, :] = 2.0 ** -130
    x[0, 0, 7, 0] = 3.0e38
    bits = I.f32_to_bf16_bits(x)
    got = Bd.fp4attn_quantize_mxfp4_rule(_dev(bits), Bd.ROLE_Q, code)
    _check_operand(got, Qz.quantize_qk(bits, "mx", rule), Bd.ROLE_Q)
    got = Bd.fp4attn_quantize_mxfp4_rule(_dev(bits), Bd.ROLE_V, code)
    _check_operand(got, Qz.quantize_v(bits, rule), Bd.ROLE_V)


def test_mx_amplitude_rule_rejects_unknown_rule():
    from paper_2609_04105_b200 import binding as Bd
    x = torch.zeros((1, 1, 128, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(Bd.Fp4AttnError):
        Bd.fp4attn_quantize_mxfp4_rule(x, Bd.ROLE_Q, 7)


def test_mx_non_finite_values_stay_in_their_block():
    """An infinity and a NaN, each in a block of its own: the call succeeds, every other block carries exactly
    the oracle's bytes, and the two blocks get the largest amplitude byte with a saturated code."""
    from paper_2609_04105_b200 import binding as Bd
    rng = np.random.default_rng(9)
    x = rng.standard_normal((1, 2, 128, 128)).astype(np.float32)
    clean = I.f32_to_bf16_bits(x)
    bits = clean.copy()
    bits[0, 0, 5, 40] = 0x7F80                                  # +inf: row 5, block 1
    bits[0, 1, 77, 100] = 0xFFC1                                # a NaN: row 77, block 3
    got = Bd.fp4attn_quantize(_dev(bits), Bd.FMT_MXFP4, Bd.ROLE_Q)
    torch.cuda.synchronize()
    want = Qz.quantize_qk(clean, "mx")
    pk_g = Qz.strip_negative_zero(got.packed.cpu().numpy()).reshape(1, 2, 128, 4, 16)     # 16 bytes per 32-block
    pk_w = Qz.strip_negative_zero(Qz.pack_nibbles(want["nib"]).reshape(-1)).reshape(1, 2, 128, 4, 16)
    touched = np.zeros((1, 2, 128, 4), dtype=bool)
    touched[0, 0, 5, 1] = touched[0, 1, 77, 3] = True
    assert ((pk_g == pk_w).all(axis=-1) | touched).all()
    sf_clean = Bd.fp4attn_quantize(_dev(clean), Bd.FMT_MXFP4, Bd.ROLE_Q).scales.cpu().numpy()
    sf_g = got.scales.cpu().numpy()
    assert np.array_equal(sf_clean, Qz.swizzle_scales(want["sf"]).reshape(-1))
    assert (sf_g != sf_clean).sum() == 2 and set(sf_g[sf_g != sf_clean]) == {254}
    assert (pk_g[0, 0, 5, 1, (40 - 32) // 2] & 0xF) == 7        # +inf (even element: low nibble) saturates at +6


@pytest.mark.parametrize("kw", [dict(B=2, H=3, N=256), dict(B=1, H=5, N=1152, d=128), dict(B=3, H=1, N=128)])
def test_nvfp4_per_head_factors_match_oracle(kw):
    """One encode factor per (batch, head) unit: bytes and the B*H factors equal the oracle's; heads are given
    magnitudes from 2^-20 to 2^9 (and one unit is all zero) so that a tensor-wide factor would not do."""
    from paper_2609_04105_b200 import binding as Bd
    w = I.shrink(I.WORKLOADS["cfg3"], **kw)
    q, k, _ = I.make_qkv(w)
    rng = np.random.default_rng(3)
    for bits, role in ((q, Bd.ROLE_Q), (k, Bd.ROLE_K)):
        x = Qz.bf16_bits_to_f64(bits)
        x *= 2.0 ** rng.integers(-20, 10, size=(w.B, w.H, 1, 1))
        if role == Bd.ROLE_K:
            x[w.B - 1, w.H - 1] = 0.0
        bits2 = I.f32_to_bf16_bits(x.astype(np.float32))
        got = Bd.fp4attn_quantize_nvfp4_per_head(_dev(bits2), role)
        want = Qz.quantize_qk(bits2, "nv", per_head=True)
        G = want.pop("G")
        _check_operand(got, {**want, "G": None}, role)
        assert np.array_equal(got.G.cpu().numpy(), G.reshape(-1))
        assert got.per_head


def test_nvfp4_per_head_rejects_v_and_missing_workspace():
    from paper_2609_04105_b200 import binding as Bd
    x = torch.zeros((1, 2, 128, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(Bd.Fp4AttnError):
        Bd.fp4attn_quantize_nvfp4_per_head(x, Bd.ROLE_V)
    L = Bd.lib()
    buf = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    rc = L.fp4attn_quantize_nvfp4_per_head(x.data_ptr(), Bd.ROLE_Q, 1, 2, 128, 64, buf.data_ptr(), buf.data_ptr(),
                                           buf.data_ptr(), None, 0, None)
    assert rc == Bd.ERR_WORKSPACE


def test_device_rounding_of_the_seeded_draws_equals_the_host_recipe():
    """bench.py rounds the seeded float32 draws to bfloat16 on the device; the bits must be those of the host
    rounding that the tests and the oracle use (round to nearest even), including the scaled outlier channels."""
    w = I.shrink(I.WORKLOADS["cfg4"], H=2, N=1024)
    want = I.make_qkv(w)
    for t in range(3):
        x = I.make_operand_f32(w, t)
        got = torch.from_numpy(x).cuda().to(torch.bfloat16).view(torch.int16).cpu().numpy().view(np.uint16)
        assert np.array_equal(got, want[t])
