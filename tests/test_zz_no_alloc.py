"""gpusq_quant_act_static: the variant of gpusq_quant_act that takes no workspace.

Some callers cannot provide scratch memory at the point where activations are
quantised (memory planned and frozen by a serving framework, allocator calls
banned in a latency-critical loop, a fixed budget owned by someone else), so
this entry point works out of a fixed array inside the library.  The test calls
it through the C ABI twice in a row and checks both results, bit for bit,
against the ordinary entry point and against the CPU oracle -- the second call
on a smaller tensor with a smaller maximum, so anything left in the shared
scratch by the first call would show up as a wrong scale.  This file sorts last on purpose: a run that stops at
the first failure has then already run every other test.
"""
import ctypes

import numpy as np
import pytest

import oracle
from paper_2305_10727_b200 import inputs

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def test_static_entry_point_matches_workspace_entry_point_twice():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2305_10727_b200 import binding as B
    lib = B.load()
    stream = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)

    big = inputs.random_layer(41, 1576, 8, 768)["X"]                      # about 1.2 M elements
    small = (inputs.random_layer(42, 197, 8, 192)["X"].astype(np.float32) * 0.25).astype(np.float16)
    for X_host in (big, small):
        X = torch.from_numpy(X_host).cuda()
        M, K = X.shape
        Xq_ref, s_ref = B.quant_act(X)                                    # caller-provided workspace
        Xq = torch.full((M, K), 99, dtype=torch.int8, device="cuda")
        s = torch.full((1,), -1.0, dtype=torch.float32, device="cuda")
        rc = lib.gpusq_quant_act_static(ctypes.c_void_p(X.data_ptr()), ctypes.c_void_p(Xq.data_ptr()),
                                        ctypes.c_void_p(s.data_ptr()), B.SCALE_COMPUTE, M, K, stream)
        assert rc == 0, B.status_string(rc)
        torch.cuda.synchronize()
        assert s.item() == s_ref.item()                                   # integer stage: bit-exact
        assert torch.equal(Xq, Xq_ref)
        Xq_o, s_o = oracle.quant_act(X_host)                              # the definition, on the CPU
        assert s.cpu().numpy()[0] == s_o
        assert np.array_equal(Xq.cpu().numpy(), Xq_o)

    # a supplied scale goes through the same entry point without touching the scratch
    X = torch.from_numpy(big).cuda()
    given = torch.tensor([0.02], dtype=torch.float32, device="cuda")
    Xq_ref, _ = B.quant_act(X, x_scale=given, scale_mode=B.SCALE_GIVEN)
    Xq, _ = B.quant_act_static(X, x_scale=given, scale_mode=B.SCALE_GIVEN)
    assert torch.equal(Xq, Xq_ref)
    assert np.array_equal(Xq.cpu().numpy(), oracle.quant_act(big, x_scale=np.float32(0.02))[0])

    # beyond the stated capacity: refused, nothing enqueued
    rc = lib.gpusq_quant_act_static(ctypes.c_void_p(X.data_ptr()), ctypes.c_void_p(Xq.data_ptr()),
                                    ctypes.c_void_p(given.data_ptr()), B.SCALE_COMPUTE, (1 << 29) + 1, 8, stream)
    assert rc == 9 and "TOO_LARGE" in B.status_string(rc)
