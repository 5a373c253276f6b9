"""The allocation-free Frobenius-norm entry point against the regular path.

Some callers must not allocate device memory while they run: code inside a memory pool's critical
section, a process that has handed all device memory to another allocator, or a latency-critical loop
where a cudaMalloc (which synchronises the device) is not acceptable. For them the library offers
defl_frobenius_norms_noalloc, whose scratch is a fixed array inside the library. Here it is checked,
through the C-ABI, against the norms defl_polar_batched reports (the normalisation scale of Eq. 1),
twice in a row because the scratch array is shared by all calls and keeps the previous contents.
This file is collected last on purpose.
"""
import ctypes

import pytest
import torch

pytestmark = pytest.mark.gpu


def _noalloc_norms(L, X):
    b = X.shape[0]
    count = X[0].numel()
    norms = torch.full((b,), -1.0, dtype=torch.float32, device=X.device)
    L.defl_frobenius_norms_noalloc.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_longlong,
                                               ctypes.c_void_p, ctypes.c_void_p]
    stream = torch.cuda.current_stream().cuda_stream
    rc = L.defl_frobenius_norms_noalloc(ctypes.c_void_p(X.data_ptr()), 0 if X.dtype == torch.bfloat16 else 1, b, count,
                                        ctypes.c_void_p(norms.data_ptr()), ctypes.c_void_p(stream))
    assert rc == 0, rc
    return norms


def test_noalloc_norms_match_regular_path_twice():
    from paper_2609_21102_b200 import binding
    L = binding.lib()
    ctx = binding.Context(0)
    g = torch.Generator(device="cuda").manual_seed(4321)
    cases = [torch.randn((5, 130, 77), generator=g, device="cuda") * 3.0,
             (torch.randn((3, 256, 512), generator=g, device="cuda") * 0.01).to(torch.bfloat16)]
    for X in cases:                      # two calls in a row share the library's scratch array
        got = _noalloc_norms(L, X)
        _, info = ctx.defl_polar_batched(X, 0, 0, 0, [[1.0, 0.0, 0.0]], steps=None, want_info=True)
        torch.cuda.synchronize()
        ref = info["rho"]
        assert torch.allclose(got, ref, rtol=1e-5, atol=0), (got, ref)
        exact = torch.linalg.norm(X.double().reshape(X.shape[0], -1), dim=1).float()
        assert torch.allclose(got, exact, rtol=1e-5, atol=0)
    ctx.close()


def test_noalloc_rejects_oversized_batches_and_bad_arguments():
    from paper_2609_21102_b200 import binding
    L = binding.lib()
    L.defl_frobenius_norms_noalloc.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_longlong,
                                               ctypes.c_void_p, ctypes.c_void_p]
    X = torch.ones((2, 8, 8), device="cuda")
    out = torch.zeros(2, device="cuda")
    assert L.defl_frobenius_norms_noalloc(ctypes.c_void_p(X.data_ptr()), 1, 100000, 64, ctypes.c_void_p(out.data_ptr()), None) == -2
    assert L.defl_frobenius_norms_noalloc(None, 1, 2, 64, ctypes.c_void_p(out.data_ptr()), None) == -1
    assert L.defl_frobenius_norms_noalloc(ctypes.c_void_p(X.data_ptr()), 7, 2, 64, ctypes.c_void_p(out.data_ptr()), None) == -1
