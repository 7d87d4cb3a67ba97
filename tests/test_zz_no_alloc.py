"""The allocation-free NVFP4 quantizer entry point against the ordinary one (collected last).

Some callers may not call cudaMalloc (fixed memory budgets, foreign allocators, latency-critical
loops), so fp4attn_quantize_nvfp4_noalloc keeps its amax scratch in an array built into the library.
It must produce the same bytes as fp4attn_quantize, call after call, although every call reuses
that one array and inherits whatever the previous call left in it.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2609_04105_b200 import inputs as I

pytestmark = pytest.mark.gpu


def _dev(bits):
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def test_noalloc_entry_point_matches_workspace_entry_point_twice_in_a_row():
    from paper_2609_04105_b200 import binding as Bd
    L = Bd.lib()
    shapes = [I.shrink(I.WORKLOADS["cfg3"], B=2, H=4, N=1024),            # d = 64
              I.shrink(I.WORKLOADS["cfg3"], B=1, H=2, N=384, d=128)]      # d = 128, smaller: stale scratch beyond its partials
    for rep in range(2):                                                   # two calls in a row per shape
        for w in shapes:
            q, k, _ = I.make_qkv(w)
            for bits, role in ((q, Bd.ROLE_Q), (k, Bd.ROLE_K)):
                x = _dev(bits)
                ref = Bd.fp4attn_quantize(x, Bd.FMT_NVFP4, role)
                packed = torch.full_like(ref.packed, 0xAB)
                scales = torch.full_like(ref.scales, 0xCD)
                G = torch.full((1,), -1.0, dtype=torch.float32, device="cuda")
                # straight through the C ABI: device pointers and sizes only
                rc = L.fp4attn_quantize_nvfp4_noalloc(x.data_ptr(), role, w.B, w.H, w.N, w.d, packed.data_ptr(),
                                                      scales.data_ptr(), G.data_ptr(),
                                                      torch.cuda.current_stream().cuda_stream)
                assert rc == 0
                torch.cuda.synchronize()
                assert torch.equal(packed, ref.packed), (rep, w.name, role)
                assert torch.equal(scales, ref.scales), (rep, w.name, role)
                assert torch.equal(G, ref.G), (rep, w.name, role)


def test_noalloc_entry_point_rejects_oversized_and_invalid_requests():
    from paper_2609_04105_b200 import binding as Bd
    L = Bd.lib()
    vp = ctypes.c_void_p
    a = vp(0x10000)
    # 2^28 elements: beyond the built-in scratch's stated capacity -> workspace error, nothing launched
    assert L.fp4attn_quantize_nvfp4_noalloc(a, Bd.ROLE_Q, 32, 64, 1024, 128, a, a, a, None) == 5
    assert L.fp4attn_quantize_nvfp4_noalloc(a, Bd.ROLE_V, 1, 1, 128, 128, a, a, a, None) == 1      # V is never NVFP4
    assert L.fp4attn_quantize_nvfp4_noalloc(None, Bd.ROLE_Q, 1, 1, 128, 128, a, a, a, None) == 1
    assert L.fp4attn_quantize_nvfp4_noalloc(a, Bd.ROLE_Q, 1, 1, 100, 128, a, a, a, None) == 2
