"""Thin ctypes binding over libfp4attn.so: argument marshalling only.

PyTorch appears here for device memory and streams; every step of the path runs inside the
library's CUDA kernels.  Importing this module fails loudly when the library is missing.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional, Tuple

import torch

FMT_MXFP4, FMT_NVFP4 = 0, 1
ROLE_Q, ROLE_K, ROLE_V = 0, 1, 2
PMAP_IDEAL, PMAP_AFFINE, PMAP_HYBRID = 0, 1, 2
PSCALE_CEIL, PSCALE_THR16, PSCALE_MSE = 0, 1, 2
SCHEDULE_ONE_QUERY, SCHEDULE_TWO_QUERY = 0, 1
PV_MXFP4, PV_E4M3 = 0, 1
QSCALE_CEIL, QSCALE_THR16, QSCALE_FLOOR, QSCALE_MSE = 0, 1, 2, 3
(OK, ERR_INVALID_ARG, ERR_UNSUPPORTED_SHAPE, ERR_UNSUPPORTED_ARCH, ERR_ALIGNMENT, ERR_WORKSPACE, ERR_CUDA,
 ERR_TIMEOUT, ERR_RANGE) = range(9)

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libfp4attn.so")

EXPORTS = [
    "fp4attn_status_string", "fp4attn_version", "fp4attn_packed_bytes", "fp4attn_scale_bytes",
    "fp4attn_quantize_workspace_bytes", "fp4attn_quantize", "fp4attn_fwd",
    "fp4attn_attention_host_workspace_bytes", "fp4attn_attention_host", "fp4attn_mma_peak_probe", "fp4attn_softmax_arith_probe",
    "fp4attn_quantize_nvfp4_noalloc", "fp4attn_selftest_bounded_wait", "fp4attn_quantize_mxfp4_rule",
    "fp4attn_quantize_nvfp4_per_head_workspace_bytes", "fp4attn_quantize_nvfp4_per_head", "fp4attn_release",
    "fp4attn_quantize_v_e4m3_workspace_bytes", "fp4attn_quantize_v_e4m3",
]


class Fp4AttnError(RuntimeError):
    pass


class _Operands(ctypes.Structure):
    _fields_ = [("q", ctypes.c_void_p), ("k", ctypes.c_void_p), ("v", ctypes.c_void_p),
                ("q_sf", ctypes.c_void_p), ("k_sf", ctypes.c_void_p), ("v_sf", ctypes.c_void_p),
                ("q_G", ctypes.c_void_p), ("k_G", ctypes.c_void_p),
                ("qk_fmt", ctypes.c_int), ("softmax_scale", ctypes.c_float),
                ("p_map", ctypes.c_int), ("affine_a", ctypes.c_float), ("affine_b", ctypes.c_float),
                ("p_scale_rule", ctypes.c_int), ("causal", ctypes.c_int), ("kv_heads", ctypes.c_int),
                ("exact_pairs", ctypes.c_int), ("g_per_head", ctypes.c_int), ("schedule", ctypes.c_int),
                ("pv_fmt", ctypes.c_int), ("v_G", ctypes.c_void_p), ("row_reference", ctypes.c_int),
                ("fixed_reference", ctypes.c_int), ("seq_len", ctypes.c_void_p)]


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise Fp4AttnError(f"{LIB_PATH} is missing: build it with `python -m paper_2609_04105_b200.build` "
                           "(there is no fallback path)")
    lib = ctypes.CDLL(LIB_PATH)
    i, sz, vp = ctypes.c_int, ctypes.c_size_t, ctypes.c_void_p
    lib.fp4attn_status_string.restype = ctypes.c_char_p
    lib.fp4attn_status_string.argtypes = [i]
    lib.fp4attn_version.restype = i
    lib.fp4attn_packed_bytes.restype = sz
    lib.fp4attn_packed_bytes.argtypes = [i, i, i, i]
    lib.fp4attn_scale_bytes.restype = sz
    lib.fp4attn_scale_bytes.argtypes = [i, i, i, i, i, i]
    lib.fp4attn_quantize_workspace_bytes.restype = sz
    lib.fp4attn_quantize_workspace_bytes.argtypes = [i, i, i, i, i, i]
    lib.fp4attn_quantize.restype = i
    lib.fp4attn_quantize.argtypes = [vp, i, i, i, i, i, i, vp, vp, vp, vp, sz, vp]
    lib.fp4attn_fwd.restype = i
    lib.fp4attn_fwd.argtypes = [ctypes.POINTER(_Operands), i, i, i, i, vp, vp, vp, vp]
    lib.fp4attn_attention_host_workspace_bytes.restype = sz
    lib.fp4attn_attention_host_workspace_bytes.argtypes = [i, i, i, i, i]
    lib.fp4attn_attention_host.restype = i
    lib.fp4attn_attention_host.argtypes = [vp, vp, vp, i, ctypes.c_float, i, i, i, i, vp, vp, vp, vp, sz, vp]
    lib.fp4attn_release.restype = i
    lib.fp4attn_release.argtypes = []
    lib.fp4attn_quantize_v_e4m3_workspace_bytes.restype = sz
    lib.fp4attn_quantize_v_e4m3_workspace_bytes.argtypes = [i, i, i, i]
    lib.fp4attn_quantize_v_e4m3.restype = i
    lib.fp4attn_quantize_v_e4m3.argtypes = [vp, i, i, i, i, vp, vp, vp, sz, vp]
    lib.fp4attn_quantize_mxfp4_rule.restype = i
    lib.fp4attn_quantize_mxfp4_rule.argtypes = [vp, i, i, i, i, i, i, vp, vp, vp]
    lib.fp4attn_quantize_nvfp4_noalloc.restype = i
    lib.fp4attn_quantize_nvfp4_noalloc.argtypes = [vp, i, i, i, i, i, vp, vp, vp, vp]
    lib.fp4attn_quantize_nvfp4_per_head_workspace_bytes.restype = sz
    lib.fp4attn_quantize_nvfp4_per_head_workspace_bytes.argtypes = [i, i, i, i]
    lib.fp4attn_quantize_nvfp4_per_head.restype = i
    lib.fp4attn_quantize_nvfp4_per_head.argtypes = [vp, i, i, i, i, i, vp, vp, vp, vp, sz, vp]
    lib.fp4attn_selftest_bounded_wait.restype = i
    lib.fp4attn_selftest_bounded_wait.argtypes = [ctypes.c_longlong, vp, vp]
    lib.fp4attn_mma_peak_probe.restype = i
    lib.fp4attn_mma_peak_probe.argtypes = [i, vp, vp]
    lib.fp4attn_softmax_arith_probe.restype = i
    lib.fp4attn_softmax_arith_probe.argtypes = [i, i, i, vp, vp]
    return lib


_lib: Optional[ctypes.CDLL] = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = _load()
    return _lib


def _check(rc: int, what: str) -> None:
    if rc != 0:
        raise Fp4AttnError(f"{what}: {lib().fp4attn_status_string(rc).decode()} (status {rc})")


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


@dataclass
class QuantizedOperand:
    packed: torch.Tensor              # uint8
    scales: torch.Tensor              # uint8, 128x4 atoms
    G: Optional[torch.Tensor]         # fp32 [1] (NVFP4) or None
    fmt: int
    role: int
    shape: Tuple[int, int, int, int]  # (B, H, N, d) of the source tensor
    per_head: bool = False            # NVFP4: G holds one factor per (batch, head) unit


def fp4attn_quantize(x: torch.Tensor, fmt: int, role: int, workspace: Optional[torch.Tensor] = None) -> QuantizedOperand:
    """x: CUDA bf16 [B,H,N,d] contiguous -> packed E2M1 + scale factors (see include/fp4attn.h)."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.is_contiguous() and x.dim() == 4
    B, H, N, d = x.shape
    L = lib()
    nb = L.fp4attn_packed_bytes(B, H, N, d)
    ns = L.fp4attn_scale_bytes(fmt, role, B, H, N, d)
    if nb == 0 or ns == 0:
        _check(L.fp4attn_quantize(x.data_ptr(), fmt, role, B, H, N, d, 1, 1, None, None, 0, _stream()), "fp4attn_quantize")
        raise Fp4AttnError("fp4attn_quantize: unsupported arguments")
    packed = torch.empty(nb, dtype=torch.uint8, device=x.device)
    scales = torch.empty(ns, dtype=torch.uint8, device=x.device)
    G = torch.empty(1, dtype=torch.float32, device=x.device) if fmt == FMT_NVFP4 else None
    nw = L.fp4attn_quantize_workspace_bytes(fmt, role, B, H, N, d)
    if nw and workspace is None:
        workspace = torch.empty(nw, dtype=torch.uint8, device=x.device)
    _check(L.fp4attn_quantize(x.data_ptr(), fmt, role, B, H, N, d, packed.data_ptr(), scales.data_ptr(),
                              _ptr(G), _ptr(workspace), 0 if workspace is None else workspace.numel(), _stream()),
           "fp4attn_quantize")
    return QuantizedOperand(packed, scales, G, fmt, role, (B, H, N, d))


def fp4attn_quantize_mxfp4_rule(x: torch.Tensor, role: int, scale_rule: int) -> QuantizedOperand:
    """MXFP4 quantizer with a selectable amplitude rule (QSCALE_CEIL / QSCALE_THR16 / QSCALE_FLOOR)."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.is_contiguous() and x.dim() == 4
    B, H, N, d = x.shape
    L = lib()
    nb = L.fp4attn_packed_bytes(B, H, N, d)
    ns = L.fp4attn_scale_bytes(FMT_MXFP4, role, B, H, N, d)
    if nb == 0 or ns == 0:
        _check(L.fp4attn_quantize_mxfp4_rule(x.data_ptr(), role, scale_rule, B, H, N, d, 1, 1, _stream()),
               "fp4attn_quantize_mxfp4_rule")
        raise Fp4AttnError("fp4attn_quantize_mxfp4_rule: unsupported arguments")
    packed = torch.empty(nb, dtype=torch.uint8, device=x.device)
    scales = torch.empty(ns, dtype=torch.uint8, device=x.device)
    _check(L.fp4attn_quantize_mxfp4_rule(x.data_ptr(), role, scale_rule, B, H, N, d, packed.data_ptr(),
                                         scales.data_ptr(), _stream()), "fp4attn_quantize_mxfp4_rule")
    return QuantizedOperand(packed, scales, None, FMT_MXFP4, role, (B, H, N, d))


def fp4attn_quantize_nvfp4_per_head(x: torch.Tensor, role: int) -> QuantizedOperand:
    """NVFP4 quantizer with one encode factor per (batch, head) unit; G comes back as fp32 [B*H]."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.is_contiguous() and x.dim() == 4
    B, H, N, d = x.shape
    L = lib()
    nb = L.fp4attn_packed_bytes(B, H, N, d)
    ns = L.fp4attn_scale_bytes(FMT_NVFP4, role, B, H, N, d)
    nw = L.fp4attn_quantize_nvfp4_per_head_workspace_bytes(B, H, N, d)
    if nb == 0 or ns == 0 or nw == 0:
        _check(L.fp4attn_quantize_nvfp4_per_head(x.data_ptr(), role, B, H, N, d, 1, 1, 1, None, 0, _stream()),
               "fp4attn_quantize_nvfp4_per_head")
        raise Fp4AttnError("fp4attn_quantize_nvfp4_per_head: unsupported arguments")
    packed = torch.empty(nb, dtype=torch.uint8, device=x.device)
    scales = torch.empty(ns, dtype=torch.uint8, device=x.device)
    G = torch.empty(B * H, dtype=torch.float32, device=x.device)
    ws = torch.empty(nw, dtype=torch.uint8, device=x.device)
    _check(L.fp4attn_quantize_nvfp4_per_head(x.data_ptr(), role, B, H, N, d, packed.data_ptr(), scales.data_ptr(),
                                             G.data_ptr(), ws.data_ptr(), ws.numel(), _stream()),
           "fp4attn_quantize_nvfp4_per_head")
    return QuantizedOperand(packed, scales, G, FMT_NVFP4, role, (B, H, N, d), True)


def fp4attn_quantize_nvfp4_noalloc(x: torch.Tensor, role: int, packed: torch.Tensor, scales: torch.Tensor,
                                   G: torch.Tensor) -> QuantizedOperand:
    """NVFP4 quantizer that allocates nothing: the caller passes every output buffer and the library
    uses its built-in 4 KB scratch.  For callers that must not touch the CUDA allocator."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.is_contiguous() and x.dim() == 4
    B, H, N, d = x.shape
    _check(lib().fp4attn_quantize_nvfp4_noalloc(x.data_ptr(), role, B, H, N, d, packed.data_ptr(), scales.data_ptr(),
                                                G.data_ptr(), _stream()), "fp4attn_quantize_nvfp4_noalloc")
    return QuantizedOperand(packed, scales, G, FMT_NVFP4, role, (B, H, N, d))


FMT_E4M3 = 2          # QuantizedOperand.fmt of an E4M3 V (fp4attn_quantize_v_e4m3); not a format of the C quantize calls


def fp4attn_quantize_v_e4m3(x: torch.Tensor) -> QuantizedOperand:
    """E4M3 bytes of V^T [B,H,d,N] with one encode factor per (batch, head) unit (G fp32 [B*H]); `scales` is empty."""
    assert x.is_cuda and x.dtype == torch.bfloat16 and x.is_contiguous() and x.dim() == 4
    B, H, N, d = x.shape
    L = lib()
    nw = L.fp4attn_quantize_v_e4m3_workspace_bytes(B, H, N, d)
    if nw == 0:
        _check(L.fp4attn_quantize_v_e4m3(x.data_ptr(), B, H, N, d, 1, 1, None, 0, _stream()), "fp4attn_quantize_v_e4m3")
        raise Fp4AttnError("fp4attn_quantize_v_e4m3: unsupported arguments")
    out = torch.empty(B * H * d * N, dtype=torch.uint8, device=x.device)
    G = torch.empty(B * H, dtype=torch.float32, device=x.device)
    ws = torch.empty(nw, dtype=torch.uint8, device=x.device)
    _check(L.fp4attn_quantize_v_e4m3(x.data_ptr(), B, H, N, d, out.data_ptr(), G.data_ptr(), ws.data_ptr(), ws.numel(), _stream()),
           "fp4attn_quantize_v_e4m3")
    return QuantizedOperand(out, torch.empty(0, dtype=torch.uint8, device=x.device), G, FMT_E4M3, ROLE_V, (B, H, N, d), True)


def fp4attn_fwd(q: QuantizedOperand, k: QuantizedOperand, v: QuantizedOperand, softmax_scale: float = 0.0,
                out: Optional[torch.Tensor] = None, lse: Optional[torch.Tensor] = None,
                status: Optional[torch.Tensor] = None, p_map: int = PMAP_IDEAL, affine_a: float = 0.0,
                affine_b: float = 0.0, p_scale_rule: int = PSCALE_CEIL, causal: bool = False,
                exact_pairs: int = 0, schedule: int = SCHEDULE_ONE_QUERY,
                seq_len: Optional[torch.Tensor] = None, fixed_reference: Optional[int] = None) -> Tuple[torch.Tensor, torch.Tensor]:
    """Direct-P attention forward on quantized operands -> (O bf16 [B,H,N,d], LSE fp32 [B,H,N]).
    p_map selects the exact code map or the affine classifier (affine_a = 0: A = 1.5, B = 1.2).
    seq_len: optional CUDA int32 tensor [B], the token count of every batch entry (padded to N).
    fixed_reference: None - running row reference; an integer - that constant row reference (the shiftless path)."""
    B, H, N, d = q.shape
    Hkv = k.shape[1]                                   # grouped-query attention when Hkv < H
    assert k.shape == v.shape and k.shape == (B, Hkv, N, d) and H % Hkv == 0 and q.fmt == k.fmt and v.fmt in (FMT_MXFP4, FMT_E4M3)
    fp8 = v.fmt == FMT_E4M3
    assert q.per_head == k.per_head, "Q and K must both carry per-head factors, or neither"
    assert seq_len is None or (seq_len.is_cuda and seq_len.dtype == torch.int32 and seq_len.numel() == B and seq_len.is_contiguous())
    dev = q.packed.device
    if out is None:
        out = torch.empty((B, H, N, d), dtype=torch.bfloat16, device=dev)
    if lse is None:
        lse = torch.empty((B, H, N), dtype=torch.float32, device=dev)
    ops = _Operands(q.packed.data_ptr(), k.packed.data_ptr(), v.packed.data_ptr(),
                    q.scales.data_ptr(), k.scales.data_ptr(), None if fp8 else v.scales.data_ptr(),
                    _ptr(q.G), _ptr(k.G), q.fmt, float(softmax_scale), int(p_map), float(affine_a), float(affine_b), int(p_scale_rule), int(bool(causal)), int(Hkv),
                    int(exact_pairs), int(q.per_head), int(schedule), PV_E4M3 if fp8 else PV_MXFP4, _ptr(v.G) if fp8 else None,
                    0 if fixed_reference is None else 1, 0 if fixed_reference is None else int(fixed_reference), _ptr(seq_len))
    _check(lib().fp4attn_fwd(ctypes.byref(ops), B, H, N, d, out.data_ptr(), lse.data_ptr(), _ptr(status), _stream()),
           "fp4attn_fwd")
    return out, lse


def fp4attn_attention_host_workspace_bytes(qk_fmt: int, B: int, H: int, N: int, d: int) -> int:
    return lib().fp4attn_attention_host_workspace_bytes(qk_fmt, B, H, N, d)


def fp4attn_attention_host(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, qk_fmt: int, out: torch.Tensor,
                           lse: Optional[torch.Tensor], workspace: torch.Tensor, softmax_scale: float = 0.0,
                           status: Optional[torch.Tensor] = None) -> None:
    """Host (pinned) bf16 Q, K, V -> host O (and LSE); copies, quantizers and attention are enqueued
    on the current stream.  `workspace` is a CUDA uint8 tensor of the queried size; `status` an optional
    HOST int32 tensor that receives the call's status word (0, or ERR_TIMEOUT) once the stream is synchronised."""
    assert not q.is_cuda and not out.is_cuda and workspace.is_cuda and (status is None or not status.is_cuda)
    B, H, N, d = q.shape
    _check(lib().fp4attn_attention_host(q.data_ptr(), k.data_ptr(), v.data_ptr(), qk_fmt, float(softmax_scale),
                                        B, H, N, d, out.data_ptr(), _ptr(lse), _ptr(status), workspace.data_ptr(),
                                        workspace.numel(), _stream()), "fp4attn_attention_host")


def fp4attn_release() -> None:
    """Destroys the host path's internal streams and events and forgets cached tensor maps."""
    _check(lib().fp4attn_release(), "fp4attn_release")


def fp4attn_mma_peak_probe(iters: int, cycles_out: torch.Tensor) -> None:
    _check(lib().fp4attn_mma_peak_probe(iters, cycles_out.data_ptr(), _stream()), "fp4attn_mma_peak_probe")


def fp4attn_softmax_arith_probe(p_map: int, exact_pairs: int, iters: int, cycles_out: torch.Tensor) -> None:
    """cycles_out: two int64 words on the device; word 0 receives the slowest warp's clocks."""
    assert cycles_out.is_cuda and cycles_out.dtype == torch.int64 and cycles_out.numel() >= 2
    _check(lib().fp4attn_softmax_arith_probe(p_map, exact_pairs, iters, cycles_out.data_ptr(), _stream()),
           "fp4attn_softmax_arith_probe")


def fp4attn_selftest_bounded_wait(limit_cycles: int, status: torch.Tensor) -> None:
    """One warp waits (bounded) on a barrier nothing completes; `status` (int32 CUDA) receives the time-out code."""
    _check(lib().fp4attn_selftest_bounded_wait(int(limit_cycles), status.data_ptr(), _stream()), "fp4attn_selftest_bounded_wait")
