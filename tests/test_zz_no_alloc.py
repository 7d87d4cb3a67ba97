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
                torch.cuda.synchronize()
                free0, alloc0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
                rc = L.fp4attn_quantize_nvfp4_noalloc(x.data_ptr(), role, w.B, w.H, w.N, w.d, packed.data_ptr(),
                                                      scales.data_ptr(), G.data_ptr(),
                                                      torch.cuda.current_stream().cuda_stream)
                assert rc == 0
                torch.cuda.synchronize()
                if rep:                                            # (the very first call on a device may load the kernels)
                    # what the entry point promises: the driver reports the same free memory, torch the same usage
                    assert torch.cuda.mem_get_info()[0] == free0 and torch.cuda.memory_allocated() == alloc0
                assert torch.equal(packed, ref.packed), (rep, w.name, role)
                assert torch.equal(scales, ref.scales), (rep, w.name, role)
                assert torch.equal(G, ref.G), (rep, w.name, role)


def test_noalloc_entry_point_from_two_host_threads_serialised_by_the_caller():
    """Two host threads call the entry point on tensors of their own.  The built-in scratch is shared, so the
    caller serialises the calls (one lock around call + synchronise, as the header asks); the per-device
    address look-up inside the library must be safe when both threads get there first."""
    import threading
    from paper_2609_04105_b200 import binding as Bd
    L = Bd.lib()
    lock = threading.Lock()
    jobs, errors = [], []
    for t, kw in enumerate((dict(B=1, H=3, N=640), dict(B=2, H=2, N=256, d=128))):
        w = I.shrink(I.WORKLOADS["cfg3"], cfg=30 + t, **kw)
        q, _, _ = I.make_qkv(w)
        x = _dev(q)
        ref = Bd.fp4attn_quantize(x, Bd.FMT_NVFP4, Bd.ROLE_Q)
        jobs.append((w, x, ref, torch.cuda.Stream()))
    torch.cuda.synchronize()

    def work(job):
        w, x, ref, stream = job
        try:
            for _ in range(8):
                packed, scales = torch.zeros_like(ref.packed), torch.zeros_like(ref.scales)
                G = torch.zeros(1, dtype=torch.float32, device="cuda")
                stream.wait_stream(torch.cuda.current_stream())
                with lock:
                    rc = L.fp4attn_quantize_nvfp4_noalloc(x.data_ptr(), Bd.ROLE_Q, w.B, w.H, w.N, w.d, packed.data_ptr(),
                                                          scales.data_ptr(), G.data_ptr(), stream.cuda_stream)
                    stream.synchronize()
                assert rc == 0
                assert torch.equal(packed, ref.packed) and torch.equal(scales, ref.scales) and torch.equal(G, ref.G)
        except Exception as e:                                             # surfaces in the main thread below
            errors.append(e)

    threads = [threading.Thread(target=work, args=(j,)) for j in jobs]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors


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
