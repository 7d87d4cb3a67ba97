"""Seeded synthetic inputs shared by the CUDA path's tests/bench and by the oracle.

This module holds no arithmetic of the attention method: it only draws Gaussian
tensors, rounds them to bfloat16 bit patterns and names the five workload
configurations.  numpy has no bfloat16, so tensors travel as uint16 bit patterns
(``[B, H, N, d]``, C-contiguous) and are widened with :func:`bf16_bits_to_f32`.

The paper measures on Gaussian operator tensors produced by a factory that is not
available here (Section "Operator benchmark suites"); these seeded N(0,1) tensors
stand in for them.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, Tuple

import numpy as np

BASE_SEED = 260904105

FMT_MXFP4 = 0
FMT_NVFP4 = 1


@dataclass(frozen=True)
class Workload:
    """One attention workload: shapes, operand formats and the input recipe."""

    name: str
    cfg: int          # seed offset index
    B: int
    H: int
    N: int
    d: int
    qk_fmt: int       # FMT_MXFP4 or FMT_NVFP4 (P and V are always MXFP4)
    outliers: bool = False   # 2 % of head-dim channels of Q and K scaled x20

    @property
    def flops(self) -> float:
        # Eq. "hao-flops" with D_QK = D_VO = d:  4 * B * H * N^2 * d
        return 4.0 * self.B * self.H * float(self.N) ** 2 * self.d


def sweep_workload(N: int) -> Workload:
    """Config 5: sequence sweep at B*N = 32768 tokens, H=16, d=128."""
    assert 32768 % N == 0
    return Workload(f"cfg5_N{N}", 5, 32768 // N, 16, N, 128, FMT_MXFP4)


WORKLOADS: Dict[str, Workload] = {
    "cfg1": Workload("cfg1", 1, 1, 2, 256, 128, FMT_MXFP4),
    "cfg2": Workload("cfg2", 2, 4, 16, 4096, 128, FMT_MXFP4),
    "cfg3": Workload("cfg3", 3, 8, 16, 8192, 64, FMT_NVFP4),
    "cfg4": Workload("cfg4", 4, 1, 32, 16384, 128, FMT_MXFP4, outliers=True),
}
for _n in (1024, 2048, 4096, 8192, 16384, 32768):
    WORKLOADS[f"cfg5_N{_n}"] = sweep_workload(_n)
# configuration 3's formats and head dimension at the longest sequence (same token count per head as the sweep's
# longest point): the second shape on which the two schedules of d = 64 are timed side by side
WORKLOADS["cfg3_N32768"] = Workload("cfg3_N32768", 6, 2, 16, 32768, 64, FMT_NVFP4)


def shrink(w: Workload, **kw) -> Workload:
    """Same recipe at other sizes (used for parity cases the oracle finishes fast)."""
    return replace(w, **kw)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bfloat16 bit pattern, round to nearest even (finite inputs)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """bfloat16 bit pattern -> float32 (exact)."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _normal_bf16(seed: int, shape: Tuple[int, ...]) -> np.ndarray:
    rng = np.random.default_rng(seed)
    return rng.standard_normal(shape, dtype=np.float32)


def outlier_channels(w: Workload) -> np.ndarray:
    """[H, k] channel indices scaled x20 in Q and K: k = round(0.02 * d), fixed per head."""
    k = max(1, int(round(0.02 * w.d)))
    rng = np.random.default_rng(BASE_SEED + 10 * w.cfg + 3)
    return np.stack([np.sort(rng.choice(w.d, size=k, replace=False)) for _ in range(w.H)])


def make_operand_f32(w: Workload, t: int) -> np.ndarray:
    """The float32 draw of operand t (0 = Q, 1 = K, 2 = V) before rounding to bfloat16, [B, H, N, d].

    Streams: Q seed = BASE_SEED + 10*cfg, K = +1, V = +2, outlier channels = +3.
    """
    x = _normal_bf16(BASE_SEED + 10 * w.cfg + t, (w.B, w.H, w.N, w.d))
    if w.outliers and t < 2:
        ch = outlier_channels(w)
        for h in range(w.H):
            x[:, h, :, ch[h]] *= np.float32(20.0)
    return x


def make_qkv(w: Workload, heads=None) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """bf16 bit patterns of Q, K, V, each [B, H, N, d] (uint16): make_operand_f32 rounded to nearest even."""
    out = [f32_to_bf16_bits(make_operand_f32(w, t)) for t in range(3)]
    return out[0], out[1], out[2]


def shard_units(n_units: int, world_size: int, rank: int) -> Tuple[int, int]:
    """Contiguous [begin, end) slice of independent units ((batch, head) pairs) for a rank."""
    base, rem = divmod(n_units, world_size)
    begin = rank * base + min(rank, rem)
    return begin, begin + base + (1 if rank < rem else 0)
