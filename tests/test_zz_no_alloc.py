"""dad_reconstruct_static: the entry point for callers that cannot allocate device memory.

Collected last on purpose (the file name sorts after every other test file), so that a run that stops
at the first failure has already been through the rest of the suite.  The GPU test passes alone in a
fresh process and after the other tests: it depends on nothing they leave behind.
"""
import ctypes

import numpy as np
import pytest
import torch


@pytest.fixture(scope="module")
def B():
    from paper_2102_09631_b200 import build, binding
    build.build()
    binding.lib()
    return binding


def test_static_scratch_limit_is_enforced_on_the_host(B):
    """A problem whose scratch need exceeds the fixed array is refused before anything is launched."""
    p = ctypes.c_void_p(0x10000)  # never dereferenced
    before = B.dad_launch_count()
    E = B.STATUS_NAMES.index
    lib = B.lib()
    assert lib.dad_reconstruct_static(0, 8, 8, p, p, p, B.DAD_BF16, None) == E("DAD_ERR_SHAPE")
    assert lib.dad_reconstruct_static(8, 8, 8, p, p, p, 5, None) == E("DAD_ERR_DTYPE")
    h_in, h_out, K = 8192, 8192, 4096
    need = B.dad_reconstruct_workspace_bytes(h_in, h_out, K, B.DAD_BF16)
    if need:  # the tensor-map encoder (hence the scratch-using path) exists only where a CUDA driver is present
        assert need > B.DAD_STATIC_SCRATCH_BYTES
        assert lib.dad_reconstruct_static(h_in, h_out, K, p, p, p, B.DAD_BF16, None) == E("DAD_ERR_WORKSPACE")
    assert B.dad_launch_count() == before


@pytest.mark.gpu
def test_static_scratch_matches_reconstruct_twice_in_a_row(B, oracle):
    """Same factors through dad_reconstruct (caller workspace) and dad_reconstruct_static (library
    array), two different problems back to back: the second call finds the first one's leftovers in the
    shared array and must not be disturbed by them.  Both entry points run the same kernels on the same
    inputs, so they must agree bit for bit; the float64 oracle's sum of outer products decides about
    either.  From the second call on the device's free memory must not move: nothing is allocated."""
    assert torch.cuda.is_available()
    dev = torch.device("cuda:0")
    g = torch.Generator().manual_seed(20262)
    calls = 0
    for (h_in, h_out, K) in [(1024, 4096, 256), (512, 384, 40)]:
        Ph, Qh = torch.randn(K, h_in, generator=g), torch.randn(K, h_out, generator=g)
        Pcat, Qcat = Ph.to(dev), Qh.to(dev)
        rows = [0, 1, h_in // 2, h_in - 1]
        want = oracle.reconstruct(Ph[:, rows], Qh)            # sampled output rows, float64
        for math, tol in ((B.DAD_BF16, 2e-2), (B.DAD_F32, 1e-5)):
            need = B.dad_reconstruct_workspace_bytes(h_in, h_out, K, math)
            assert need <= B.DAD_STATIC_SCRATCH_BYTES
            ws = B.new_workspace(need, dev)
            ref = torch.empty(h_in, h_out, device=dev)
            B.dad_reconstruct(h_in, h_out, K, Pcat, Qcat, ref, math, ws)
            B.dad_check(ws)
            got = torch.full((h_in, h_out), float("nan"), device=dev)
            torch.cuda.synchronize()
            free_before = torch.cuda.mem_get_info(dev)[0]
            B.dad_reconstruct_static(h_in, h_out, K, Pcat, Qcat, got, math)
            torch.cuda.synchronize()
            free_after = torch.cuda.mem_get_info(dev)[0]
            calls += 1
            if calls > 1:      # the very first call may load the module that holds the array
                assert free_after == free_before, (free_before, free_after)
            assert torch.equal(got, ref), (h_in, h_out, K, math)
            sample = got[rows].double().cpu().numpy()
            err = float(np.linalg.norm(sample - want) / np.linalg.norm(want))
            assert err <= tol, (h_in, h_out, K, math, err)
            if math == B.DAD_BF16:
                assert need > 0  # this is the path that really uses the library's array
