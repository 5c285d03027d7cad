"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the
header declares, counts bytes exactly, and rejects bad arguments before launching anything."""
import ctypes
import os
import re

import pytest

import oracle_pins as pins

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    from paper_2102_09631_b200 import build, binding
    build.build()
    binding.lib()
    return binding


def declared_functions():
    text = open(os.path.join(ROOT, "include", "dad.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dad_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(B):
    names = declared_functions()
    assert len(names) >= 12
    for n in names:
        assert hasattr(B.lib(), n), n
    assert sorted(B.EXPORTS) == names


def layer(B, S=2, N=16, h_in=64, h_out=32, dtype=0, **kw):
    d = dict(S=S, N=N, h_in=h_in, h_out=h_out, dtype=dtype, ldA=h_in, ldD=h_out, strideA=N * h_in, strideD=N * h_out)
    d.update(kw)
    return B.dad_layer(**d)


def test_byte_counts_are_exact(B, oracle):
    for N, h_in, h_out, e, r, dsgd, dad, rank in pins.read_golden_bytes():
        L = layer(B, S=3, N=N, h_in=h_in, h_out=h_out, dtype=0 if e == 4 else 1)
        assert B.dad_bytes_dsgd(L) == dsgd == oracle.bytes_dsgd(h_in, h_out)
        assert B.dad_bytes_dad(L) == dad == oracle.bytes_dad(N, h_in, h_out, e)
        assert B.dad_bytes_rank(L, r) == rank == oracle.bytes_rank(r, h_in, h_out)
    big = layer(B, S=1, N=1 << 20, h_in=1 << 14, h_out=1 << 14)
    assert B.dad_bytes_dad(big) == (1 << 20) * (1 << 15) * 4  # no 32-bit wrap
    assert B.dad_bytes_dad(layer(B, S=0)) == 0 and B.dad_bytes_rank(layer(B), 0) == 0


def test_gather_charges_each_site_without_a_device(B):
    # the byte accounting is host arithmetic; with stacks aliasing the factors nothing is launched
    L = layer(B, S=5, h_in=40, h_out=24)
    tx = B.bytes_array(5)
    fake = ctypes.c_void_p(0x10000)
    st = B.lib().dad_gather_factors(ctypes.byref(L), 3, fake, fake, fake, fake, tx, None)
    assert st == 0 and list(tx) == [3 * 64 * 4] * 5


def test_workspace_query(B):
    L = layer(B)
    n = B.dad_workspace_bytes(L, 4, 2)
    assert n > 0 and n % 256 == 0
    assert B.dad_workspace_bytes(L, 0, 2) == 0            # r < 1
    assert B.dad_workspace_bytes(L, 33, 2) == 0           # r > h_out
    assert B.dad_workspace_bytes(L, 4, -1) == 0
    assert B.dad_workspace_bytes(layer(B, dtype=7), 4, 2) == 0
    assert B.dad_workspace_bytes(layer(B, N=4096, h_in=1024, h_out=4096, dtype=1, S=16), 64, 3) >= n
    # one site: the site strides are unspecified and must not matter (odd, zero or huge values)
    one = dict(S=1, N=64, h_in=128, h_out=256, dtype=1, ldA=128, ldD=256)
    ref = B.dad_workspace_bytes(layer(B, strideA=64 * 128, strideD=64 * 256, **one), 8, 2)
    assert ref > 0
    for sa, sd in ((0, 0), (3, 5), (1 << 50, 1 << 50)):
        assert B.dad_workspace_bytes(layer(B, strideA=sa, strideD=sd, **one), 8, 2) == ref


def test_bad_arguments_are_rejected_before_any_launch(B):
    lib = B.lib()
    before = B.dad_launch_count()
    p = ctypes.c_void_p(0x10000)   # never dereferenced: every call below fails validation first
    odd = ctypes.c_void_p(0x10004)
    null = ctypes.c_void_p(0)
    L = layer(B)
    ws = B.dad_workspace_bytes(L, 4, 2)
    E = {n: i for i, n in enumerate(B.STATUS_NAMES)}

    def compress(Lx=L, A=p, D=p, r=4, iters=2, Q0=p, P=p, Q=p, sigma=null, w=p, nws=ws):
        return lib.dad_rank_compress(ctypes.byref(Lx), A, D, r, iters, Q0, P, Q, sigma, w, nws, None)

    assert lib.dad_rank_compress(None, p, p, 4, 2, p, p, p, null, p, ws, None) == E["DAD_ERR_NULL"]
    assert compress(A=null) == E["DAD_ERR_NULL"]
    assert compress(w=null) == E["DAD_ERR_NULL"]
    assert compress(Lx=layer(B, dtype=5)) == E["DAD_ERR_DTYPE"]
    assert compress(Lx=layer(B, N=0)) == E["DAD_ERR_SHAPE"]
    assert compress(Lx=layer(B, ldA=63)) == E["DAD_ERR_SHAPE"]
    assert compress(Lx=layer(B, strideD=10)) == E["DAD_ERR_SHAPE"]
    assert compress(iters=-1) == E["DAD_ERR_SHAPE"]
    assert compress(r=0) == E["DAD_ERR_RANK"]
    assert compress(r=33) == E["DAD_ERR_RANK"]      # r > h_out = 32
    assert compress(Lx=layer(B, h_in=128, h_out=128, ldA=128, ldD=128, strideA=16 * 128, strideD=16 * 128), r=65) == E["DAD_ERR_RANK"]
    assert compress(A=odd) == E["DAD_ERR_ALIGN"]
    assert compress(nws=ws - 1) == E["DAD_ERR_WORKSPACE"]
    assert lib.dad_full_grad(ctypes.byref(L), p, p, null, None, null, 0, None) == E["DAD_ERR_NULL"]
    assert lib.dad_full_grad(ctypes.byref(L), p, odd, p, None, null, 0, None) == E["DAD_ERR_ALIGN"]
    assert lib.dad_reconstruct(0, 4, 4, p, p, p, 0, null, 0, None) == E["DAD_ERR_SHAPE"]
    assert lib.dad_reconstruct(4, 4, 4, p, null, p, 0, null, 0, None) == E["DAD_ERR_NULL"]
    assert lib.dad_reconstruct(4, 4, 4, p, p, p, 9, null, 0, None) == E["DAD_ERR_DTYPE"]
    assert lib.dad_reconstruct_batched(4, 4, 4, 0, p, p, p, 0, null, 0, None) == E["DAD_ERR_SHAPE"]
    assert lib.dad_reconstruct_batched(4, 4, 4, 2, p, p, null, 0, null, 0, None) == E["DAD_ERR_NULL"]
    assert lib.dad_reconstruct_batched_workspace_bytes(4, 4, 4, 0, 1) == 0
    assert lib.dad_gather_factors(ctypes.byref(L), 0, p, p, p, p, None, None) == E["DAD_ERR_RANK"]
    assert lib.dad_check(null, None) == E["DAD_ERR_NULL"]
    # host entry point: the caller's own row and site strides are checked before any copy is queued
    def host(Lx, scratch=p, nbytes=1 << 40):
        return lib.dad_rank_dad_host(ctypes.byref(Lx), p, p, p, 4, 2, 0, p, None, scratch, nbytes, None)
    assert host(layer(B, ldA=63)) == E["DAD_ERR_SHAPE"]
    assert host(layer(B, ldD=31)) == E["DAD_ERR_SHAPE"]
    assert host(layer(B, strideA=16 * 64 - 1)) == E["DAD_ERR_SHAPE"]
    assert host(layer(B), scratch=ctypes.c_void_p(0x10100), nbytes=256) == E["DAD_ERR_WORKSPACE"]
    assert B.dad_launch_count() == before
    for code in range(len(B.STATUS_NAMES)):
        assert len(lib.dad_status_string(code)) > 0


def test_pipeline_query_and_diagnostics_validate_their_arguments(B):
    lib = B.lib()
    before = B.dad_launch_count()
    E = {n: i for i, n in enumerate(B.STATUS_NAMES)}
    c = ctypes.c_int(7)
    # invalid layers / ranks give -1 and a cluster size of 0
    assert lib.dad_compress_path(None, 4, 2, ctypes.byref(c)) == -1 and c.value == 0
    assert lib.dad_compress_path(ctypes.byref(layer(B, N=0)), 4, 2, None) == -1
    assert lib.dad_compress_path(ctypes.byref(layer(B)), 33, 2, None) == -1
    assert lib.dad_compress_path(ctypes.byref(layer(B, dtype=2)), 4, 2, None) == -1    # DAD_BF16_1TERM is no storage type
    # a small fp32 layer goes to a one-launch form; switching those off sends it to the general pipeline; the
    # workspace size does not depend on the switch
    L = layer(B)
    n_on = B.dad_workspace_bytes(L, 4, 2)
    path, C = B.dad_compress_path(L, 4, 2)
    assert path in (B.DAD_PATH_FUSED, B.DAD_PATH_FUSED_L2) and 1 <= C <= 8 and L.N >= 4 * C
    B.dad_fused_enable(False)
    try:
        assert B.dad_compress_path(L, 4, 2) == (B.DAD_PATH_GENERAL, 0)
        assert B.dad_workspace_bytes(L, 4, 2) == n_on
    finally:
        B.dad_fused_enable(True)
    # a site far too large for one cluster stays with the streaming pipelines
    big = layer(B, S=16, N=4096, h_in=1024, h_out=4096, dtype=1)
    assert B.dad_compress_path(big, 16, 3)[0] in (B.DAD_PATH_GENERAL, B.DAD_PATH_TENSOR, B.DAD_PATH_TENSOR_PAIRED)
    # the bounded-wait self-test checks its workspace before launching anything
    p = ctypes.c_void_p(0x10000)
    assert lib.dad_selftest_bounded_wait(None, 1 << 20, None) == E["DAD_ERR_NULL"]
    assert lib.dad_selftest_bounded_wait(ctypes.c_void_p(0x10010), 1 << 20, None) == E["DAD_ERR_ALIGN"]
    assert lib.dad_selftest_bounded_wait(p, B.DAD_SELFTEST_BYTES - 1, None) == E["DAD_ERR_WORKSPACE"]
    # the one-term reconstruction is a valid `math`, not a valid input type
    assert lib.dad_reconstruct(8, 8, 8, p, p, None, B.DAD_BF16_1TERM, None, 0, None) == E["DAD_ERR_NULL"]
    assert lib.dad_reconstruct(8, 8, 8, p, p, p, 3, None, 0, None) == E["DAD_ERR_DTYPE"]
    assert B.dad_launch_count() == before


def test_no_cpu_fallback(B):
    """Without a CUDA device a well-formed compute call must fail with DAD_ERR_CUDA, never compute."""
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present; the refusal is only observable on a CPU-only machine")
    p = ctypes.c_void_p(0x10000)
    L = layer(B)
    ws = B.dad_workspace_bytes(L, 4, 2)
    st = B.lib().dad_rank_compress(ctypes.byref(L), p, p, 4, 2, p, p, p, None, p, ws, None)
    assert st == B.STATUS_NAMES.index("DAD_ERR_CUDA")
    with pytest.raises(B.DadError):
        B._check(st, "dad_rank_compress")


def test_missing_library_is_a_loud_error(B, monkeypatch):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", os.path.join(ROOT, "no_such_dir", "libdad.so"))
    with pytest.raises(RuntimeError, match="missing"):
        B.lib()
