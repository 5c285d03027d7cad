"""Thin Python binding of libdad (include/dad.h): same names, argument marshalling only.

Tensors are torch CUDA tensors (torch is used for device memory and streams only); every
step of the path runs in the library's own kernels.  There is no fallback: if libdad.so is
missing or cannot be loaded, or a call returns an error status, a RuntimeError is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# DAD_LIB picks another build of the same library (e.g. the bounds-check build libdad_check.so)
LIB_PATH = os.path.join(_HERE, os.environ.get("DAD_LIB", "libdad.so"))

DAD_OK = 0
DAD_F32, DAD_BF16, DAD_BF16_1TERM = 0, 1, 2
DAD_MAX_RANK = 64
STATUS_NAMES = ["DAD_OK", "DAD_ERR_NULL", "DAD_ERR_SHAPE", "DAD_ERR_DTYPE", "DAD_ERR_RANK", "DAD_ERR_WORKSPACE",
                "DAD_ERR_ALIGN", "DAD_ERR_CUDA", "DAD_ERR_TIMEOUT", "DAD_ERR_NUMERIC"]

# every symbol include/dad.h declares
EXPORTS = ["dad_bytes_dad", "dad_bytes_rank", "dad_bytes_dsgd", "dad_workspace_bytes", "dad_full_grad",
           "dad_full_grad_grouped_workspace_bytes", "dad_full_grad_grouped",
           "dad_rank_compress", "dad_gather_factors", "dad_reconstruct_workspace_bytes", "dad_reconstruct",
           "dad_reconstruct_batched_workspace_bytes", "dad_reconstruct_batched",
           "dad_reconstruct_static", "dad_aggregate_workspace_bytes", "dad_aggregate_compress", "dad_effective_rank",
           "dad_rank_dad_host_scratch_bytes", "dad_rank_dad_host", "dad_rank_compress_gram_workspace_bytes",
           "dad_rank_compress_gram", "dad_rank_compress_sequential_workspace_bytes", "dad_rank_compress_sequential",
           "dad_check", "dad_bounds_check_build", "dad_bounds_report", "dad_selftest_bounded_wait", "dad_compress_path", "dad_fused_enable", "dad_pair_enable", "dad_launch_count", "dad_status_string", "dad_timing_enable", "dad_timing_collect",
           "dad_timing_reset", "dad_timing_name", "dad_timing_ms", "dad_timing_launches"]


class dad_layer(ctypes.Structure):
    _fields_ = [("S", ctypes.c_int32), ("N", ctypes.c_int64), ("h_in", ctypes.c_int64), ("h_out", ctypes.c_int64),
                ("dtype", ctypes.c_int), ("ldA", ctypes.c_int64), ("ldD", ctypes.c_int64),
                ("strideA", ctypes.c_int64), ("strideD", ctypes.c_int64)]


class DadError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        name = STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else str(status)
        super().__init__(f"{where}: {name} ({lib().dad_status_string(status).decode()})")


_lib = None


def lib() -> ctypes.CDLL:
    """Load libdad.so (built in-tree by paper_2102_09631_b200.build); fails loudly if absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2102_09631_b200.build` "
                               "(there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        vp, u64p = ctypes.c_void_p, ctypes.POINTER(ctypes.c_uint64)
        lp = ctypes.POINTER(dad_layer)
        L.dad_bytes_dad.argtypes = [lp]
        L.dad_bytes_dad.restype = ctypes.c_uint64
        L.dad_bytes_rank.argtypes = [lp, ctypes.c_int]
        L.dad_bytes_rank.restype = ctypes.c_uint64
        L.dad_bytes_dsgd.argtypes = [lp]
        L.dad_bytes_dsgd.restype = ctypes.c_uint64
        L.dad_workspace_bytes.argtypes = [lp, ctypes.c_int, ctypes.c_int]
        L.dad_workspace_bytes.restype = ctypes.c_size_t
        L.dad_full_grad.argtypes = [lp, vp, vp, vp, u64p, vp, ctypes.c_size_t, vp]
        L.dad_full_grad.restype = ctypes.c_int
        L.dad_full_grad_grouped_workspace_bytes.argtypes = [lp, ctypes.c_int]
        L.dad_full_grad_grouped_workspace_bytes.restype = ctypes.c_size_t
        L.dad_full_grad_grouped.argtypes = [lp, ctypes.c_int, vp, vp, vp, u64p, vp, ctypes.c_size_t, vp]
        L.dad_full_grad_grouped.restype = ctypes.c_int
        L.dad_rank_compress.argtypes = [lp, vp, vp, ctypes.c_int, ctypes.c_int, vp, vp, vp, vp, vp, ctypes.c_size_t, vp]
        L.dad_rank_compress.restype = ctypes.c_int
        L.dad_gather_factors.argtypes = [lp, ctypes.c_int, vp, vp, vp, vp, u64p, vp]
        L.dad_gather_factors.restype = ctypes.c_int
        L.dad_reconstruct_workspace_bytes.argtypes = [ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, ctypes.c_int]
        L.dad_reconstruct_workspace_bytes.restype = ctypes.c_size_t
        L.dad_reconstruct.argtypes = [ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, vp, vp, vp, ctypes.c_int, vp,
                                      ctypes.c_size_t, vp]
        L.dad_reconstruct.restype = ctypes.c_int
        L.dad_reconstruct_batched_workspace_bytes.argtypes = [ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, ctypes.c_int,
                                                              ctypes.c_int]
        L.dad_reconstruct_batched_workspace_bytes.restype = ctypes.c_size_t
        L.dad_reconstruct_batched.argtypes = [ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, ctypes.c_int, vp, vp, vp,
                                              ctypes.c_int, vp, ctypes.c_size_t, vp]
        L.dad_reconstruct_batched.restype = ctypes.c_int
        L.dad_reconstruct_static.argtypes = [ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, vp, vp, vp, ctypes.c_int, vp]
        L.dad_reconstruct_static.restype = ctypes.c_int
        L.dad_aggregate_workspace_bytes.argtypes = [ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, ctypes.c_int, ctypes.c_int]
        L.dad_aggregate_workspace_bytes.restype = ctypes.c_size_t
        L.dad_aggregate_compress.argtypes = [ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, vp, vp, ctypes.c_int,
                                             ctypes.c_int, vp, vp, vp, vp, vp, ctypes.c_size_t, vp]
        L.dad_aggregate_compress.restype = ctypes.c_int
        L.dad_effective_rank.argtypes = [lp, ctypes.c_int, ctypes.c_float, vp, vp, vp, vp, vp]
        L.dad_effective_rank.restype = ctypes.c_int
        L.dad_rank_dad_host_scratch_bytes.argtypes = [lp, ctypes.c_int, ctypes.c_int, ctypes.c_int]
        L.dad_rank_dad_host_scratch_bytes.restype = ctypes.c_size_t
        L.dad_rank_dad_host.argtypes = [lp, vp, vp, vp, ctypes.c_int, ctypes.c_int, ctypes.c_int, vp, u64p, vp,
                                        ctypes.c_size_t, vp]
        L.dad_rank_dad_host.restype = ctypes.c_int
        L.dad_rank_compress_gram_workspace_bytes.argtypes = [lp, ctypes.c_int, ctypes.c_int]
        L.dad_rank_compress_gram_workspace_bytes.restype = ctypes.c_size_t
        L.dad_rank_compress_gram.argtypes = [lp, vp, vp, ctypes.c_int, ctypes.c_int, vp, vp, vp, vp, vp, ctypes.c_size_t, vp]
        L.dad_rank_compress_gram.restype = ctypes.c_int
        L.dad_rank_compress_sequential_workspace_bytes.argtypes = [lp, ctypes.c_int, ctypes.c_int]
        L.dad_rank_compress_sequential_workspace_bytes.restype = ctypes.c_size_t
        L.dad_rank_compress_sequential.argtypes = [lp, vp, vp, ctypes.c_int, ctypes.c_int, vp, vp, vp, vp, vp,
                                                   ctypes.c_size_t, vp]
        L.dad_rank_compress_sequential.restype = ctypes.c_int
        L.dad_compress_path.argtypes = [lp, ctypes.c_int, ctypes.c_int, ctypes.POINTER(ctypes.c_int)]
        L.dad_compress_path.restype = ctypes.c_int
        L.dad_fused_enable.argtypes = [ctypes.c_int]
        L.dad_fused_enable.restype = None
        L.dad_pair_enable.argtypes = [ctypes.c_int]
        L.dad_pair_enable.restype = None
        L.dad_bounds_check_build.argtypes = []
        L.dad_bounds_check_build.restype = ctypes.c_int
        L.dad_bounds_report.argtypes = [ctypes.POINTER(ctypes.c_uint64), ctypes.c_int, vp]
        L.dad_bounds_report.restype = ctypes.c_int
        L.dad_selftest_bounded_wait.argtypes = [vp, ctypes.c_size_t, vp]
        L.dad_selftest_bounded_wait.restype = ctypes.c_int
        L.dad_check.argtypes = [vp, vp]
        L.dad_check.restype = ctypes.c_int
        L.dad_launch_count.argtypes = []
        L.dad_launch_count.restype = ctypes.c_uint64
        L.dad_status_string.argtypes = [ctypes.c_int]
        L.dad_status_string.restype = ctypes.c_char_p
        L.dad_timing_enable.argtypes = [ctypes.c_int]
        L.dad_timing_enable.restype = None
        L.dad_timing_collect.restype = ctypes.c_int
        L.dad_timing_reset.restype = None
        L.dad_timing_name.argtypes = [ctypes.c_int]
        L.dad_timing_name.restype = ctypes.c_char_p
        L.dad_timing_ms.argtypes = [ctypes.c_int]
        L.dad_timing_ms.restype = ctypes.c_double
        L.dad_timing_launches.argtypes = [ctypes.c_int]
        L.dad_timing_launches.restype = ctypes.c_uint64
        _lib = L
    return _lib


def _dtype_code(t: torch.dtype) -> int:
    if t == torch.float32:
        return DAD_F32
    if t == torch.bfloat16:
        return DAD_BF16
    raise TypeError(f"A and D must be float32 or bfloat16, got {t}")


def make_layer(A: torch.Tensor, D: torch.Tensor) -> dad_layer:
    """Descriptor of a layer whose sites are the leading dimension: A is S x N x h_in, D is S x N x h_out
    (innermost dimension contiguous; row and site strides are taken from the tensors)."""
    if A.dim() != 3 or D.dim() != 3 or A.shape[:2] != D.shape[:2] or A.dtype != D.dtype:
        raise ValueError("A must be S x N x h_in and D S x N x h_out of one dtype")
    if A.stride(2) != 1 or D.stride(2) != 1:
        raise ValueError("innermost dimension must be contiguous")
    S, N, h_in = A.shape
    return dad_layer(S, N, h_in, D.shape[2], _dtype_code(A.dtype), A.stride(1), D.stride(1), A.stride(0), D.stride(0))


def _stream(stream: Optional[torch.cuda.Stream]):
    s = stream if stream is not None else torch.cuda.current_stream()
    return ctypes.c_void_p(s.cuda_stream)


def _ptr(t: Optional[torch.Tensor]):
    return ctypes.c_void_p(t.data_ptr()) if t is not None else ctypes.c_void_p(0)


def _check(status: int, where: str):
    if status != DAD_OK:
        raise DadError(status, where)


def dad_bytes_dad(layer: dad_layer) -> int:
    return int(lib().dad_bytes_dad(ctypes.byref(layer)))


def dad_bytes_rank(layer: dad_layer, r: int) -> int:
    return int(lib().dad_bytes_rank(ctypes.byref(layer), r))


def dad_bytes_dsgd(layer: dad_layer) -> int:
    return int(lib().dad_bytes_dsgd(ctypes.byref(layer)))


def dad_workspace_bytes(layer: dad_layer, r: int, iters: int) -> int:
    return int(lib().dad_workspace_bytes(ctypes.byref(layer), r, iters))


DAD_PATH_GENERAL, DAD_PATH_TENSOR, DAD_PATH_FUSED, DAD_PATH_FUSED_L2, DAD_PATH_TENSOR_PAIRED = 0, 1, 2, 3, 4


def dad_compress_path(layer: dad_layer, r: int, iters: int):
    """(path, cluster size) dad_rank_compress takes for this shape; path is one of DAD_PATH_*."""
    c = ctypes.c_int(0)
    return int(lib().dad_compress_path(ctypes.byref(layer), r, iters, ctypes.byref(c))), c.value


def dad_fused_enable(on: bool):
    lib().dad_fused_enable(1 if on else 0)


def dad_pair_enable(on: bool):
    """Process-wide switch of the paired launches of the tensor-core sequence (for timing one form against the other)."""
    lib().dad_pair_enable(1 if on else 0)


def dad_launch_count() -> int:
    return int(lib().dad_launch_count())


def new_workspace(nbytes: int, device) -> torch.Tensor:
    ws = torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)
    ws[:256].zero_()  # the status words must start out clear
    return ws


def dad_full_grad(layer: dad_layer, A, D, grad, bytes_tx=None, ws=None, stream=None):
    """grad (h_in x h_out fp32) <- sum_s A_s^T D_s; bytes_tx: optional ctypes uint64 array of S entries."""
    st = lib().dad_full_grad(ctypes.byref(layer), _ptr(A), _ptr(D), _ptr(grad), bytes_tx, _ptr(ws),
                             ws.numel() if ws is not None else 0, _stream(stream))
    _check(st, "dad_full_grad")


def dad_full_grad_grouped_workspace_bytes(layer: dad_layer, groups: int) -> int:
    return int(lib().dad_full_grad_grouped_workspace_bytes(ctypes.byref(layer), groups))


def dad_full_grad_grouped(layer: dad_layer, groups: int, A, D, grads, bytes_tx=None, ws=None, stream=None):
    """grads (groups x h_in x h_out fp32) <- the dAD gradients of `groups` layers stacked as slices of A and D."""
    st = lib().dad_full_grad_grouped(ctypes.byref(layer), groups, _ptr(A), _ptr(D), _ptr(grads), bytes_tx, _ptr(ws),
                                     ws.numel() if ws is not None else 0, _stream(stream))
    _check(st, "dad_full_grad_grouped")


def dad_rank_compress(layer: dad_layer, A, D, r: int, iters: int, Q0, P, Q, sigma, ws, stream=None):
    st = lib().dad_rank_compress(ctypes.byref(layer), _ptr(A), _ptr(D), r, iters, _ptr(Q0), _ptr(P), _ptr(Q),
                                 _ptr(sigma), _ptr(ws), ws.numel() if ws is not None else 0, _stream(stream))
    _check(st, "dad_rank_compress")


def dad_gather_factors(layer: dad_layer, r: int, P, Q, Pcat, Qcat, bytes_tx=None, stream=None):
    st = lib().dad_gather_factors(ctypes.byref(layer), r, _ptr(P), _ptr(Q), _ptr(Pcat), _ptr(Qcat), bytes_tx,
                                  _stream(stream))
    _check(st, "dad_gather_factors")


def dad_reconstruct_workspace_bytes(h_in: int, h_out: int, K: int, math: int) -> int:
    return int(lib().dad_reconstruct_workspace_bytes(h_in, h_out, K, math))


def dad_reconstruct(h_in: int, h_out: int, K: int, Pcat, Qcat, grad, math: int = DAD_F32, ws=None, stream=None):
    st = lib().dad_reconstruct(h_in, h_out, K, _ptr(Pcat), _ptr(Qcat), _ptr(grad), math, _ptr(ws),
                               ws.numel() if ws is not None else 0, _stream(stream))
    _check(st, "dad_reconstruct")


def dad_reconstruct_batched_workspace_bytes(h_in: int, h_out: int, K: int, batch: int, math: int) -> int:
    return int(lib().dad_reconstruct_batched_workspace_bytes(h_in, h_out, K, batch, math))


def dad_reconstruct_batched(h_in: int, h_out: int, K: int, batch: int, Pcat, Qcat, grad, math: int = DAD_F32, ws=None,
                            stream=None):
    """`batch` reconstructions of one shape in one go: entry b owns rows b*K .. b*K+K-1 of the stacks and grad[b]."""
    st = lib().dad_reconstruct_batched(h_in, h_out, K, batch, _ptr(Pcat), _ptr(Qcat), _ptr(grad), math, _ptr(ws),
                                       ws.numel() if ws is not None else 0, _stream(stream))
    _check(st, "dad_reconstruct_batched")


DAD_STATIC_SCRATCH_BYTES = 32 << 20


def dad_reconstruct_static(h_in: int, h_out: int, K: int, Pcat, Qcat, grad, math: int = DAD_F32, stream=None):
    """dad_reconstruct for callers that cannot provide scratch: the library's own fixed device array
    (DAD_STATIC_SCRATCH_BYTES, shared by all calls on the device) stands in for `ws`."""
    st = lib().dad_reconstruct_static(h_in, h_out, K, _ptr(Pcat), _ptr(Qcat), _ptr(grad), math, _stream(stream))
    _check(st, "dad_reconstruct_static")


def dad_aggregate_workspace_bytes(h_in: int, h_out: int, K: int, r: int, iters: int) -> int:
    return int(lib().dad_aggregate_workspace_bytes(h_in, h_out, K, r, iters))


def dad_aggregate_compress(h_in: int, h_out: int, K: int, Pcat, Qcat, r: int, iters: int, Q0, Phat, Qhat, sigma, ws,
                           stream=None):
    """Second structured power iteration on the stacked factors (the aggregator's SPI of Algorithm 1)."""
    st = lib().dad_aggregate_compress(h_in, h_out, K, _ptr(Pcat), _ptr(Qcat), r, iters, _ptr(Q0), _ptr(Phat), _ptr(Qhat),
                                      _ptr(sigma), _ptr(ws), ws.numel() if ws is not None else 0, _stream(stream))
    _check(st, "dad_aggregate_compress")


def dad_effective_rank(layer: dad_layer, r: int, theta: float, sigma, r_eff, P=None, Q=None, stream=None):
    """r_eff[s] <- leading components of site s with sigma_j > theta * sigma_1; zeroes the dropped rows of P, Q."""
    st = lib().dad_effective_rank(ctypes.byref(layer), r, ctypes.c_float(theta), _ptr(sigma), _ptr(r_eff), _ptr(P), _ptr(Q),
                                  _stream(stream))
    _check(st, "dad_effective_rank")


def dad_rank_dad_host_scratch_bytes(layer: dad_layer, r: int, iters: int, math: int) -> int:
    return int(lib().dad_rank_dad_host_scratch_bytes(ctypes.byref(layer), r, iters, math))


def dad_rank_dad_host(layer: dad_layer, A_host, D_host, Q0_host, r: int, iters: int, math: int, grad_host, scratch,
                      bytes_tx=None, stream=None):
    """compress -> gather -> reconstruct for HOST tensors (pinned for asynchronous copies); `scratch` is a device
    uint8 tensor of at least dad_rank_dad_host_scratch_bytes.  Queued on the stream; synchronise before reading."""
    for t in (A_host, D_host, Q0_host, grad_host):
        if t.is_cuda:
            raise ValueError("dad_rank_dad_host takes host tensors")
    st = lib().dad_rank_dad_host(ctypes.byref(layer), _ptr(A_host), _ptr(D_host), _ptr(Q0_host), r, iters, math,
                                 _ptr(grad_host), bytes_tx, _ptr(scratch), scratch.numel(), _stream(stream))
    _check(st, "dad_rank_dad_host")


DAD_MAX_GRAM_ROWS = 128


def dad_rank_compress_gram_workspace_bytes(layer: dad_layer, r: int, iters: int) -> int:
    return int(lib().dad_rank_compress_gram_workspace_bytes(ctypes.byref(layer), r, iters))


def dad_rank_compress_gram(layer: dad_layer, A, D, r: int, iters: int, Q0, P, Q, sigma, ws, stream=None):
    """dad_rank_compress through C = A A^T (Algorithm 2 as printed; fp32 inputs, N <= DAD_MAX_GRAM_ROWS)."""
    st = lib().dad_rank_compress_gram(ctypes.byref(layer), _ptr(A), _ptr(D), r, iters, _ptr(Q0), _ptr(P), _ptr(Q),
                                      _ptr(sigma), _ptr(ws), ws.numel() if ws is not None else 0, _stream(stream))
    _check(st, "dad_rank_compress_gram")


def dad_rank_compress_sequential_workspace_bytes(layer: dad_layer, r: int, iters: int) -> int:
    return int(lib().dad_rank_compress_sequential_workspace_bytes(ctypes.byref(layer), r, iters))


def dad_rank_compress_sequential(layer: dad_layer, A, D, r: int, iters: int, Q0, P, Q, sigma, ws, stream=None):
    """dad_rank_compress with the components found one after the other (Algorithm 2 in its printed order)."""
    st = lib().dad_rank_compress_sequential(ctypes.byref(layer), _ptr(A), _ptr(D), r, iters, _ptr(Q0), _ptr(P), _ptr(Q),
                                            _ptr(sigma), _ptr(ws), ws.numel() if ws is not None else 0, _stream(stream))
    _check(st, "dad_rank_compress_sequential")


DAD_SELFTEST_BYTES = 64 << 10


def dad_selftest_bounded_wait(ws, stream=None):
    """Makes one bounded device-side wait run out on purpose (nothing hangs or faults); dad_check(ws) then
    raises DAD_ERR_TIMEOUT."""
    _check(lib().dad_selftest_bounded_wait(_ptr(ws), ws.numel(), _stream(stream)), "dad_selftest_bounded_wait")


def dad_bounds_check_build() -> bool:
    return bool(lib().dad_bounds_check_build())


def dad_bounds_report(reset: bool = False, stream=None):
    """(violations, first address, bytes, source line) recorded by a -DDAD_BOUNDS_CHECK build; zeros otherwise."""
    out = (ctypes.c_uint64 * 4)()
    _check(lib().dad_bounds_report(out, 1 if reset else 0, _stream(stream)), "dad_bounds_report")
    return tuple(int(x) for x in out)


def dad_check(ws, stream=None):
    _check(lib().dad_check(_ptr(ws), _stream(stream)), "dad_check")


def dad_timing_enable(on: bool):
    lib().dad_timing_enable(1 if on else 0)


def dad_timing_reset():
    lib().dad_timing_reset()


def dad_timing_collect() -> dict:
    """{kernel family: (total ms, launches)} of the launches timed since the last reset (synchronises)."""
    n = lib().dad_timing_collect()
    return {lib().dad_timing_name(i).decode(): (float(lib().dad_timing_ms(i)), int(lib().dad_timing_launches(i)))
            for i in range(n)}


def bytes_array(S: int):
    return (ctypes.c_uint64 * S)()


class LayerPlan:
    """Buffers for one layer shape, allocated once: factors, stacks, gradient and workspace.
    `step` runs compress -> gather -> reconstruct on the current stream (marshalling only).

    `groups` > 1 stacks that many layers of the same shape in one plan: A and D then hold
    groups * S slices (layer g owns slices g*S .. g*S+S-1), the power iterations of all of them run
    in the same launches (slices are independent), and each layer is reconstructed from its own rows
    of the stacks (one batched call); `grad` is then groups x h_in x h_out.

    `calls` > 1 keeps the factors and stacks of that many calls of the plan side by side: `step(..., call=c)`
    compresses and gathers into slot c without reconstructing, and `finish()` reconstructs the layers of all
    slots in ONE batched call (`grads_all`: calls * groups x h_in x h_out).  The reconstruction of a handful of
    layers is a few tens of microseconds of work that does not fill the GPU's last round of tiles; a step's worth
    of a shape does."""

    def __init__(self, A: torch.Tensor, D: torch.Tensor, r: int, iters: int, zero_copy_gather: bool = False,
                 groups: int = 1, reconstruct_math: Optional[int] = None, calls: int = 1):
        self.layer = make_layer(A, D)
        L = self.layer
        if groups < 1 or L.S % groups:
            raise ValueError("the slice count must be a multiple of `groups`")
        if calls < 1:
            raise ValueError("`calls` must be at least 1")
        self.groups, self.sites, self.calls = groups, L.S // groups, calls
        dev = A.device
        self.r, self.iters = r, iters
        self.P_all = torch.empty(calls, L.S, r, L.h_in, device=dev, dtype=torch.float32)
        self.Q_all = torch.empty(calls, L.S, r, L.h_out, device=dev, dtype=torch.float32)
        self.sigma_all = torch.empty(calls, L.S, r, device=dev, dtype=torch.float32)
        if zero_copy_gather:
            self.Pcat_all, self.Qcat_all = self.P_all.view(calls, L.S * r, L.h_in), self.Q_all.view(calls, L.S * r, L.h_out)
        else:
            self.Pcat_all = torch.empty(calls, L.S * r, L.h_in, device=dev, dtype=torch.float32)
            self.Qcat_all = torch.empty(calls, L.S * r, L.h_out, device=dev, dtype=torch.float32)
        self.grads_all = torch.empty(calls * groups, L.h_in, L.h_out, device=dev, dtype=torch.float32)
        # slot 0 under the names a plan of one call has always had
        self.P, self.Q, self.sigma = self.P_all[0], self.Q_all[0], self.sigma_all[0]
        self.Pcat, self.Qcat = self.Pcat_all[0], self.Qcat_all[0]
        self.grads = self.grads_all[:groups]
        self.grad = self.grads[0] if groups == 1 else self.grads
        # reconstruction arithmetic: that of the inputs (fp32 FMA / three-term bf16) unless the caller picks one
        self.math = L.dtype if reconstruct_math is None else reconstruct_math
        nws = dad_workspace_bytes(L, r, iters)
        if nws == 0:
            raise ValueError("invalid layer / rank / iteration count")
        self.K = self.sites * r
        self.ws = new_workspace(max(nws, dad_reconstruct_batched_workspace_bytes(L.h_in, L.h_out, self.K, groups,
                                                                                 self.math)), dev)
        self.ws_all = None
        if calls > 1:
            self.ws_all = new_workspace(max(256, dad_reconstruct_batched_workspace_bytes(L.h_in, L.h_out, self.K,
                                                                                          calls * groups, self.math)), dev)
        self.bytes_tx = bytes_array(L.S)

    def step(self, A, D, Q0, stream=None, call: Optional[int] = None):
        L = self.layer
        if call is None:
            dad_rank_compress(L, A, D, self.r, self.iters, Q0, self.P, self.Q, self.sigma, self.ws, stream)
            dad_gather_factors(L, self.r, self.P, self.Q, self.Pcat, self.Qcat, self.bytes_tx, stream)
            dad_reconstruct_batched(L.h_in, L.h_out, self.K, self.groups, self.Pcat, self.Qcat, self.grads, self.math,
                                    self.ws, stream)
            return self.grad
        P, Q = self.P_all[call], self.Q_all[call]
        dad_rank_compress(L, A, D, self.r, self.iters, Q0, P, Q, self.sigma_all[call], self.ws, stream)
        dad_gather_factors(L, self.r, P, Q, self.Pcat_all[call], self.Qcat_all[call], self.bytes_tx, stream)
        return None

    def finish(self, stream=None):
        """Reconstructs the layers of every slot filled by `step(..., call=c)` in one batched call."""
        L = self.layer
        ws = self.ws_all if self.ws_all is not None else self.ws
        dad_reconstruct_batched(L.h_in, L.h_out, self.K, self.calls * self.groups, self.Pcat_all, self.Qcat_all,
                                self.grads_all, self.math, ws, stream)
        return self.grads_all
