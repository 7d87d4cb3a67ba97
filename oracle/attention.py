"""Tiled Direct-P attention forward (oracle side, test infrastructure only).

Follows, in the paper's order and notation:
  * the online recurrence over key tiles (Eq. "online-recurrence"),
  * Algorithm "direct-p-pack" for every N32 score fragment: block maximum -> power-of-two
    amplitude alpha_B = 2**e_B with byte u_B = e_B + 127 (a block whose byte would fall
    below 1 is a zero block) -> x = (z - m)*log2(e) - e_B + log2(6) -> q = Q_E2M1(2**x)
    (Eq. "ideal-code-path") -> code sum c_B,
  * the represented numerator / denominator (Eqs. "represented-contributions",
    "represented-output"), with the denominator term evaluated as alpha_B * (c_B / 6) in that
    association (Algorithm "sampled-guard", steps 4-5).

Readings where the paper leaves a choice:
  * row reference m_i: the running maximum rounded UP to an integer in the log2 domain,
    mu_i = max over tiles seen so far of ceil(max_j y_ij), y = z*log2(e).  With an integer
    reference every online rescale factor is an exact power of two and
    x = y - E_B + log2(6) no longer depends on the reference, so the represented
    probabilities do not depend on tile size, tile order or rescale policy;
  * block exponent: E_B = ceil(max_{j in B} y_ij) (absolute), e_B = E_B - mu_i;
  * "fp32 accumulate": the score handed to softmax is the exact block-scaled product rounded
    once to float32; y used for the integer decisions is the float32 product fl32(s32*c32).
  * LSE is the natural log of the represented denominator.

Everything else is float64.

Second code map (p_map="affine", Eq. "affine-code-map"): q = Q_E2M1(max(0, A x + B)) with the paper's
generic `fast` fit A = 1.50, B = 1.20 by default.  The paper folds the score transform, e_B and the
log2 6 term into the coefficients of one fused multiply-add; that arithmetic is fixed here in
float32 so that a GPU reproduces the codes bit for bit:
    cA = fl32(A * c32),  bA = fl32(A * fl32(log2 6 - E_B) + B)  (one fma),  u = fl32(s32 * cA + bA)  (one fma).
Block exponents, reference, denominator and output are unchanged.

Mixed map (p_map="hybrid", the paper's EX2-density control, Appendix "SM103 launch and EX2 controls"):
element pair k of a block (keys 2k, 2k+1) takes the ideal map where bit k of `exact_pairs` is set and the
affine map elsewhere; which pairs pay for an exponential is a fixed pattern, so a GPU reproduces it.

Third block-exponent rule (p_scale="mse"): per block the better of the two neighbouring powers by squared error of
the represented values (see mse_exponent_of inside direct_p_rows); it reproduces the MXFP4 rows of Table "p-range" and
is a near-decision wherever the two error sums almost tie.

Second block-exponent rule (p_scale="thr16"): Eq. "mx-scale" allows either neighbouring power of two
as the amplitude; besides the ceiling (default) the oracle offers the threshold rule
E_B = floor(fl32(max y + fl32(log2 1.6))), i.e. alpha_B = 2^floor(log2(1.6 a_B)): the block maximum then
lands in [3.75, 7.5) code units and values above 6 saturate.  It reproduces the MXFP4 rows of Table
"p-range" (pinned in the tests) and lowers the P error.

Causal mask and grouped-query attention (the forward the paper's training section builds on,
Section "Causal backward ..."): causal=True removes keys j > i from query row i before anything else
(their score is -inf: they never raise a block maximum and always code to 0; a block with no visible
key contributes nothing); kv_group = g lets g consecutive query heads share one K/V head.

Several results can be correct.  A code changes only where the converter input crosses one of the seven
boundaries of Eq. "e2m1-boundaries", and a block exponent only where the block maximum crosses an
integer.  An implementation whose score differs from fl32(exact product) by a rounding (a tensor core
accumulating a sum that float32 cannot hold) or whose 2**x is an approximation may legitimately land on
the other side.  `direct_p_rows(report={})` therefore also lists every such near-decision of a row that
carries visible weight, and `flips=` re-evaluates rows with chosen decisions taken the other way; a
checker accepts an output row that disagrees with the default evaluation only if it agrees with one of
those alternatives.
"""
from __future__ import annotations

import math

import numpy as np

from .formats import E2M1_VALUES, e2m1_encode_mag
from .quantize import dequantize

LOG2E_32 = np.float32(1.4426950408889634)
LOG2_6_32 = np.float32(math.log2(6.0))
LOG2_1P6_32 = np.float32(math.log2(1.6))
P_BLOCK = 32


def block_exponent(ymax32: np.ndarray, p_scale: str = "ceil") -> np.ndarray:
    """Integer block exponent E_B from the block maximum of y (float32), as float64 integers."""
    if p_scale == "ceil":
        return np.ceil(np.asarray(ymax32, np.float32).astype(np.float64))
    assert p_scale == "thr16"
    return np.floor((np.asarray(ymax32, np.float32) + LOG2_1P6_32).astype(np.float32).astype(np.float64))


def score_constant(qd: dict, kd: dict, d: int, softmax_scale=None, unit=None) -> np.float32:
    """c32: multiplies the tensor-core-facing score S_hw to give y = z*log2(e).

    MXFP4 x MXFP4: S_hw carries 6*6 (amplitude convention) -> c = fl32(fl32(log2e*scale)/36).
    NVFP4 x NVFP4: S_hw carries G_q*G_k              -> c = fl32(fl32(log2e*scale)/fl32(G_q*G_k)).
    With per-(batch, head) factors (G arrays [B, H]) `unit` = (b, h, hk) names the query unit and the
    K/V head it reads, and the constant is that pair's.
    """
    scale = np.float32(1.0 / math.sqrt(d)) if softmax_scale is None else np.float32(softmax_scale)
    base = np.float32(LOG2E_32 * scale)
    if qd["fmt"] == "mx" and kd["fmt"] == "mx":
        return np.float32(base / np.float32(36.0))
    assert qd["fmt"] == "nv" and kd["fmt"] == "nv"
    Gq, Gk = qd["G"], kd["G"]
    if np.ndim(Gq) or np.ndim(Gk):
        b, h, hk = unit
        Gq, Gk = np.asarray(Gq)[b, h], np.asarray(Gk)[b, hk]
    return np.float32(base / np.float32(np.float32(Gq) * np.float32(Gk)))


def scores_fp32(qd: dict, kd: dict, b: int, h: int, rows=None, hk=None) -> np.ndarray:
    """S_hw[i, j] = sum_k (scale*code)_Q[i,k] * (scale*code)_K[j,k], exact, rounded once to fp32."""
    A = dequantize({**qd, "nib": qd["nib"][b, h][None, None], "sf": qd["sf"][b, h][None, None]}, hw=True)[0, 0]
    hk = h if hk is None else hk
    Bm = dequantize({**kd, "nib": kd["nib"][b, hk][None, None], "sf": kd["sf"][b, hk][None, None]}, hw=True)[0, 0]
    if rows is not None:
        A = A[rows]
    return (A @ Bm.T).astype(np.float32)


def _fma32(a, b, c):
    """fl32(a*b + c) for float32 inputs: the product is exact in float64, the sum is rounded once more
    only when it needs more than 53 bits (not the case for the magnitudes used here)."""
    return (np.asarray(a, np.float32).astype(np.float64) * np.asarray(b, np.float32).astype(np.float64)
            + np.asarray(c, np.float32).astype(np.float64)).astype(np.float32)


def ulp32(v) -> np.ndarray:
    """Spacing of float32 at |v| (float64 result; the smallest normal spacing below 2**-126)."""
    a = np.abs(np.asarray(v, np.float64))
    _, e = np.frexp(np.maximum(a, 2.0 ** -126))
    return np.ldexp(1.0, e - 24)


AMBIGUITY = dict(rel=2.0 ** -18, ulps=4.0, share=1e-4)
"""Default near-decision thresholds.  rel: relative distance of the converter input (2**x, or the affine
classifier's u measured through its slope) from a code boundary; ulps: float32 spacings of the score y
that an implementation's score may differ by (this widens `rel` for large |y| and is the distance of a
block maximum from an integer); share: smallest part of the row's represented mass an element (or, for
an exponent decision, a block) must carry for its decision to be listed."""


def _boundary_neighbours(v: np.ndarray):
    """For decision values v >= 0: index j of the nearest E2M1 rounding boundary t_j and |v - t_j|."""
    t = np.asarray([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0])
    dist = np.abs(v[..., None] - t)
    j = dist.argmin(axis=-1)
    return j, np.take_along_axis(dist, j[..., None], axis=-1)[..., 0], t[j]


def direct_p_rows(s32: np.ndarray, c32: np.float32, Vhat: np.ndarray, tile: int = 128, tile_order=None,
                  p_map: str = "ideal", affine=(1.5, 1.2), p_scale: str = "ceil", row_index=None,
                  exact_pairs: int = 0xFFFF, report=None, flips=None, ambiguity=None, kv_len=None,
                  fixed_reference=None):
    """Direct-P online softmax + PV for a set of query rows of one (batch, head).

    s32  [R, N] float32 tensor-core-facing scores;  Vhat [N, d] float64 reconstructed V.
    Returns O [R, d] float64, LSE [R] float64, and the represented probabilities' pieces
    (codes [R, N] uint8, block exponents E_B [R, N/32] int64, final reference mu [R]).

    report : optional dict, filled with the near-decisions of every row (thresholds `ambiguity`, default
             AMBIGUITY): "code" bool [R, N] - the element's code could be its neighbour's; "eb" bool
             [R, N/32] - the block exponent could be the other integer; "row" bool [R] - any of the two.
    kv_len : optional number of keys that exist (sequences shorter than the padded N): keys kv_len..N-1 are masked
             like the keys a causal row does not see (score -inf: they enter no block maximum, get code 0 and no
             weight), so the result is that of the operator on the first kv_len keys.
    fixed_reference : optional integer: the row reference is this constant for every row and never moves (the
             shiftless path of Section "Fix 3: guard only extreme model logits"; the `fast` policy of Table
             "policy-definition" has no anchor, i.e. reference 0).  A block's E8M0 byte is then E_B - reference +
             127: a block whose byte would fall below 1 is a zero block, a byte above 254 or a row left without any
             live block is outside the policy's range and raises ValueError.  Inside the range the result is that of
             the running reference (codes do not depend on the reference, rescales are exact powers of two).
    flips  : optional dict with the same two keys: decisions to take the OTHER way.  A flipped code moves to
             the code across its nearest boundary; a flipped block exponent to the integer on the other side
             of the block maximum, and the block's codes follow from the new exponent.
    """
    R, N = s32.shape
    assert N % P_BLOCK == 0 and tile % P_BLOCK == 0 and N % tile == 0
    if row_index is not None:                                    # causal: query row i sees keys 0..i
        s32 = np.where(np.arange(N)[None, :] > np.asarray(row_index)[:, None], np.float32(-np.inf), s32).astype(np.float32)
    if kv_len is not None:                                       # padded sequence: keys kv_len.. do not exist
        assert 1 <= int(kv_len) <= N
        s32 = np.where(np.arange(N)[None, :] >= int(kv_len), np.float32(-np.inf), s32).astype(np.float32)
    y32 = (s32 * np.float32(c32)).astype(np.float32)             # decision variable, fp32
    yx = s32.astype(np.float64) * np.float64(c32)                # converter input, fp64
    mu = np.full(R, -np.inf) if fixed_reference is None else np.full(R, float(int(fixed_reference)))
    L = np.zeros(R)
    O = np.zeros((R, Vhat.shape[1]))
    codes_all = np.zeros((R, N), dtype=np.uint8)
    EB_all = np.zeros((R, N // P_BLOCK), dtype=np.int64)
    assert p_map in ("ideal", "affine", "hybrid")
    # hybrid: element pair k (keys 2k, 2k+1 of a block) takes the ideal map where bit k of exact_pairs is set,
    # the affine map elsewhere
    pair_exact = ((int(exact_pairs) >> (np.arange(P_BLOCK) // 2)) & 1).astype(bool)
    A32, B32 = np.float32(affine[0]), np.float32(affine[1])
    cA = np.float32(A32 * np.float32(c32))
    amb = dict(AMBIGUITY, **(ambiguity or {}))
    if report is not None:
        near_code = np.zeros((R, N), dtype=bool)
        near_eb = np.zeros((R, N // P_BLOCK), dtype=bool)
        cand = np.zeros((R, N))                                   # larger candidate value of a near code, in units of 2**E_B / 6
    flip_code = None if flips is None or flips.get("code") is None else np.asarray(flips["code"], bool)
    flip_eb = None if flips is None or flips.get("eb") is None else np.asarray(flips["eb"], bool)

    def exponent_of(bj):
        """Block exponent of keys bj..bj+31 (with its flip applied), and whether it is a near-decision."""
        ymax = y32[:, bj:bj + P_BLOCK].max(axis=1)
        if p_scale == "mse":
            return mse_exponent_of(bj, ymax)
        E = block_exponent(ymax, p_scale)
        w = ymax if p_scale == "ceil" else (ymax + LOG2_1P6_32).astype(np.float32)   # the value that is rounded to an integer
        w64 = w.astype(np.float64)
        with np.errstate(invalid="ignore"):
            near = np.isfinite(w64) & (np.abs(w64 - np.rint(w64)) < amb["ulps"] * ulp32(np.where(np.isfinite(w64), w64, 0.0)))
        if flip_eb is not None:
            n = np.rint(np.where(np.isfinite(w64), w64, 0.0))
            other = np.where(E == n, n + (1 if p_scale == "ceil" else -1), n)      # the integer on the other side of w
            E = np.where(flip_eb[:, bj // P_BLOCK] & np.isfinite(w64), other, E)
        return E, near

    def mse_exponent_of(bj, ymax):
        """Eq. "mx-scale" names both powers of two next to the block maximum; this rule takes, per block, the one
        with the smaller squared error of the 32 represented values: with v = 6 * 2**(y - E_c) under the ceiling
        E_c = ceil(max y), the floor E_c - 1 doubles every v (values above 6 saturate), and its error sum is in
        units four times smaller, so the floor wins iff sum (2v - q(2v))**2 < 4 sum (v - q(v))**2 (strictly; a
        block whose maximum is an integer has one candidate only).  Near-decision: the two sides within 1e-3 of
        each other relative to their sum (an implementation evaluates 2**x approximately and sums in float32)."""
        Ec = np.ceil(ymax.astype(np.float64))
        fin = np.isfinite(Ec)
        Ec0 = np.where(fin, Ec, 0.0)
        b32 = np.float32(LOG2_6_32 - Ec0.astype(np.float32))
        v = np.exp2(yx[:, bj:bj + P_BLOCK] + b32.astype(np.float64)[:, None])
        ec = ((v - E2M1_VALUES[e2m1_encode_mag(v)]) ** 2).sum(axis=1)
        ef = ((2 * v - E2M1_VALUES[e2m1_encode_mag(2 * v)]) ** 2).sum(axis=1)
        two = fin & (ymax.astype(np.float64) != Ec)                # two candidates
        take_f = two & (ef < 4.0 * ec)
        near = two & (np.abs(ef - 4.0 * ec) <= 1e-3 * (ef + 4.0 * ec))
        if flip_eb is not None:
            take_f = np.where(flip_eb[:, bj // P_BLOCK] & two, ~take_f, take_f)
        return np.where(fin, Ec0 - take_f, Ec), near

    order = range(N // tile) if tile_order is None else tile_order
    for t in order:
        j0 = t * tile
        exps = [exponent_of(bj) for bj in range(j0, j0 + tile, P_BLOCK)]
        m_tile = np.max(np.stack([e for e, _ in exps]), axis=0)
        mu_new = np.maximum(mu, m_tile) if fixed_reference is None else mu
        f = np.where(np.isinf(mu), 0.0, np.exp2(mu - mu_new))     # exact power of two
        L *= f
        O *= f[:, None]
        mu = mu_new
        for bj, (E_B, eb_near) in zip(range(j0, j0 + tile, P_BLOCK), exps):
            seen = np.isfinite(E_B)                              # False: every key of the block is masked
            E_B = np.where(seen, E_B, 0.0)
            e_B = np.where(seen, E_B - mu, -np.inf)
            live = (e_B + 127) >= 1
            if fixed_reference is not None and np.any(seen & (e_B + 127 > 254)):
                raise ValueError("a block exponent lies more than 127 octaves above the fixed reference")
            b_B32 = np.float32(LOG2_6_32 - E_B.astype(np.float32))
            sl = slice(bj, bj + P_BLOCK)
            if p_map in ("ideal", "hybrid"):
                x = yx[:, sl] + b_B32.astype(np.float64)[:, None]
                v = np.exp2(x)                                   # decision value of the ideal map
                slope = math.log(2.0) * v                        # d v / d x
                code = e2m1_encode_mag(v)
            if p_map in ("affine", "hybrid"):
                bA = _fma32(A32, b_B32, B32)
                u = _fma32(s32[:, sl], cA, bA[:, None])
                v_a = np.maximum(u, np.float32(0)).astype(np.float64)
                code_a = e2m1_encode_mag(v_a)
                if p_map == "affine":
                    code, v, slope = code_a, v_a, np.full(v_a.shape, float(A32))
                else:
                    code = np.where(pair_exact[None, :], code, code_a)
                    v = np.where(pair_exact[None, :], v, v_a)
                    slope = np.where(pair_exact[None, :], slope, float(A32))
            if report is not None or flip_code is not None:
                with np.errstate(invalid="ignore"):
                    jn, dist, tj = _boundary_neighbours(np.where(np.isfinite(v), v, 0.0))
                if report is not None:
                    tol_x = np.maximum(amb["rel"] / math.log(2.0), amb["ulps"] * ulp32(np.where(np.isfinite(yx[:, sl]), yx[:, sl], 0.0)))
                    near_code[:, sl] = np.isfinite(yx[:, sl]) & live[:, None] & (dist < slope * tol_x)
                    cand[:, sl] = E2M1_VALUES[jn + 1]
                    near_eb[:, bj // P_BLOCK] = eb_near & seen & live
                if flip_code is not None:
                    code = np.where(flip_code[:, sl], (2 * jn + 1) - code.astype(np.int64), code)   # neighbours of boundary j are codes j, j+1
            code = np.where(live[:, None], code, 0).astype(np.uint8)
            q = E2M1_VALUES[code]
            alpha = np.where(live, np.exp2(np.where(live, e_B, 0.0)), 0.0)
            c_B = q.sum(axis=1)
            L += alpha * (c_B / 6.0)
            O += (alpha / 6.0)[:, None] * (q @ Vhat[sl])
            codes_all[:, sl] = code
            EB_all[:, bj // P_BLOCK] = np.where(seen, E_B, -(1 << 40)).astype(np.int64)
    if fixed_reference is not None and np.any(L <= 0):
        raise ValueError("a row has no block within 126 octaves below the fixed reference")
    Oout = O / L[:, None]
    lse = math.log(2.0) * (mu + np.log2(L))
    if report is not None:
        # keep only decisions that carry visible weight: an element's (larger candidate) share of the row's
        # represented mass, a block's whole share for an exponent decision
        EBf = np.repeat(np.where(EB_all > -(1 << 39), EB_all, 0).astype(np.float64), P_BLOCK, axis=1)
        w_el = np.exp2(np.minimum(EBf - mu[:, None], 0.0)) / 6.0 / L[:, None]
        visible = EB_all > -(1 << 39)
        share_el = cand * w_el
        share_blk = (E2M1_VALUES[codes_all] * w_el).reshape(R, N // P_BLOCK, P_BLOCK).sum(axis=2)
        report["code"] = near_code & (share_el > amb["share"])
        report["eb"] = near_eb & visible & (share_blk > amb["share"])
        report["row"] = report["code"].any(axis=1) | report["eb"].any(axis=1)
    return Oout, lse, codes_all, EB_all, mu


def direct_p_forward(qd: dict, kd: dict, vd: dict, softmax_scale=None, tile: int = 128,
                     rows=None, heads=None, tile_order=None, p_map: str = "ideal", affine=(1.5, 1.2),
                     p_scale: str = "ceil", causal: bool = False, kv_group: int = 1, exact_pairs: int = 0xFFFF,
                     seq_len=None, fixed_reference=None):
    """Whole-operator oracle.  qd/kd/vd come from oracle.quantize.quantize_qk / quantize_v.
    fixed_reference: see direct_p_rows (the shiftless path: a constant row reference).

    seq_len : optional [B] integers, 1 <= seq_len[b] <= N: batch entry b is a sequence of seq_len[b] tokens padded
              to N.  Its keys beyond the length are masked; its query rows beyond the length carry no meaning and
              are returned as NaN (a caller compares rows below the length only).

    rows : optional 1-D index array of query rows evaluated for every (b, h) (rows are
           independent); heads : optional list of (b, h) pairs.  Returns O [n_heads, R, d]
           float64 and LSE [n_heads, R] float64 in the order of `heads`.
    """
    B, H, N, d = qd["nib"].shape
    assert H % kv_group == 0 and kd["nib"].shape[1] == H // kv_group and vd["nib"].shape[1] == H // kv_group
    heads = [(b, h) for b in range(B) for h in range(H)] if heads is None else list(heads)
    ridx = np.arange(N) if rows is None else np.asarray(rows)
    Os, Ls = [], []
    for (b, h) in heads:
        hk = h // kv_group                                       # K/V head shared by the group
        c32 = score_constant(qd, kd, d, softmax_scale, (b, h, hk))
        s32 = scores_fp32(qd, kd, b, h, rows, hk)
        Vhat = dequantize({**vd, "nib": vd["nib"][b, hk][None, None], "sf": vd["sf"][b, hk][None, None]})[0, 0].T
        O, lse, _, _, _ = direct_p_rows(s32, c32, np.ascontiguousarray(Vhat), tile, tile_order, p_map, affine, p_scale,
                                        ridx if causal else None, exact_pairs,
                                        kv_len=None if seq_len is None else int(seq_len[b]), fixed_reference=fixed_reference)
        if seq_len is not None:
            O[ridx >= int(seq_len[b])] = np.nan
            lse[ridx >= int(seq_len[b])] = np.nan
        Os.append(O)
        Ls.append(lse)
    return np.stack(Os), np.stack(Ls)


# ----------------------------------------------------------------------------------------------- FP8 P/V route
P8_SHIFT = 8      # probabilities are carried as 2**8 * p, so the largest (p = 1) is 256 <= 448, the E4M3 maximum


def fp8_pv_rows(s32: np.ndarray, c32: np.float32, V8hat: np.ndarray, row_index=None, kv_len=None):
    """FP8 probabilities and values for a set of query rows of one (batch, head) (the route the paper retains for
    training, Section "Training stability selects FP8 P/V"; it prints no algorithm, reading taken here).

    s32 [R, N] float32 scores facing the tensor core, V8hat [N, d] float64 reconstructed E4M3 V.
      mu_i  = ceil(max_j y_ij), y = fl32(s32 * c32): an integer row reference, the row maximum rounded up, known
              before any probability is formed, so that nothing depends on a tile order;
      p8_ij = Q_E4M3(2**(y_ij - mu_i + 8)), round to nearest even on the E4M3 grid (three mantissa bits, subnormals
              of 2**-9; below 2**-10 the value is 0): one 8-bit float per probability, NO block scales;
      O_i   = sum_j p8_ij V^_j / sum_j p8_ij (the same rounded values in numerator and denominator, Eq.
              "represented-output" carried over), LSE_i = ln2 (mu_i - 8 + log2 sum_j p8_ij).
    kv_len: optional number of keys that exist (padded sequence); the others are masked like a causal row's
    invisible keys.  Returns O [R, d], LSE [R], the E4M3 bytes [R, N] and mu [R]."""
    from .formats import e4m3_decode, e4m3_encode_unsigned
    R, N = s32.shape
    if row_index is not None:
        s32 = np.where(np.arange(N)[None, :] > np.asarray(row_index)[:, None], np.float32(-np.inf), s32).astype(np.float32)
    if kv_len is not None:
        assert 1 <= int(kv_len) <= N
        s32 = np.where(np.arange(N)[None, :] >= int(kv_len), np.float32(-np.inf), s32).astype(np.float32)
    y32 = (s32 * np.float32(c32)).astype(np.float32)
    mu = np.ceil(y32.max(axis=1).astype(np.float64))
    b32 = np.float32(np.float32(P8_SHIFT) - mu.astype(np.float32))
    x = s32.astype(np.float64) * np.float64(c32) + b32.astype(np.float64)[:, None]
    byte = e4m3_encode_unsigned(np.exp2(x))
    p8 = e4m3_decode(byte)
    L = p8.sum(axis=1)
    O = (p8 @ V8hat) / L[:, None]
    lse = math.log(2.0) * (mu - P8_SHIFT + np.log2(L))
    return O, lse, byte, mu


def fp8_pv_forward(qd: dict, kd: dict, v8: dict, softmax_scale=None, rows=None, heads=None, causal: bool = False,
                   kv_group: int = 1, seq_len=None):
    """Whole-operator oracle of the FP8-P/V route: FP4 Q, K as in direct_p_forward, v8 from quantize_v_e4m3;
    seq_len as in direct_p_forward (rows beyond a length come back as NaN)."""
    from .quantize import dequantize_v_e4m3
    B, H, N, d = qd["nib"].shape
    heads = [(b, h) for b in range(B) for h in range(H)] if heads is None else list(heads)
    ridx = np.arange(N) if rows is None else np.asarray(rows)
    Os, Ls = [], []
    for (b, h) in heads:
        hk = h // kv_group
        c32 = score_constant(qd, kd, d, softmax_scale, (b, h, hk))
        s32 = scores_fp32(qd, kd, b, h, rows, hk)
        O, lse, _, _ = fp8_pv_rows(s32, c32, np.ascontiguousarray(dequantize_v_e4m3(v8, b, hk).T), ridx if causal else None,
                                   kv_len=None if seq_len is None else int(seq_len[b]))
        if seq_len is not None:
            O[ridx >= int(seq_len[b])] = np.nan
            lse[ridx >= int(seq_len[b])] = np.nan
        Os.append(O)
        Ls.append(lse)
    return np.stack(Os), np.stack(Ls)


def exact_attention(Q: np.ndarray, K: np.ndarray, V: np.ndarray, softmax_scale=None, rows=None, causal=False):
    """Eq. "exact-attention" in float64 for one head: Q [N,d], K [N,d], V [N,d] -> O, LSE."""
    d = Q.shape[1]
    scale = 1.0 / math.sqrt(d) if softmax_scale is None else float(softmax_scale)
    Qr = Q if rows is None else Q[rows]
    z = (Qr @ K.T) * scale
    if causal:
        ridx = np.arange(Q.shape[0]) if rows is None else np.asarray(rows)
        z = np.where(np.arange(K.shape[0])[None, :] > ridx[:, None], -np.inf, z)
    m = z.max(axis=1, keepdims=True)
    p = np.exp(z - m)
    l = p.sum(axis=1, keepdims=True)
    return (p @ V) / l, (m + np.log(l))[:, 0]


def exact_p_attention(qd: dict, kd: dict, vd: dict, b: int, h: int, softmax_scale=None, rows=None, causal=False,
                      hk=None):
    """O_exactP for one (batch, head): the quantized operands as they are reconstructed (Q^, K^, V^), exact
    float64 softmax in between - what the path would return if P were not quantized."""
    hk = h if hk is None else hk
    one = lambda dd, i: dequantize({**dd, "nib": dd["nib"][b, i][None, None], "sf": dd["sf"][b, i][None, None],
                                    "G": (None if dd["G"] is None else (np.asarray(dd["G"])[b, i] if np.ndim(dd["G"]) else dd["G"]))})[0, 0]
    return exact_attention(one(qd, h), one(kd, hk), one(vd, hk).T, softmax_scale, rows, causal)


def bf16_round(x: np.ndarray) -> np.ndarray:
    """float64 -> nearest bfloat16 value (ties to even), returned as float64."""
    x = np.asarray(x, dtype=np.float64)
    _, e = np.frexp(x)                    # |x| in [2**(e-1), 2**e)
    step = np.ldexp(1.0, e - 8)           # 8 significant bits
    return np.rint(x / step) * step       # rint is round-half-even
