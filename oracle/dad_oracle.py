"""ctypes front end of the float64 CPU oracle (``dad_oracle.c``).

TEST INFRASTRUCTURE, not product code: imported only by the tests, by the smoke check
and by the benchmark's CPU-baseline leg.  It shares nothing with the CUDA path; its
inputs are numpy arrays (or anything ``numpy.asarray`` accepts) that are widened
exactly to float64 before the C routines run.

Notation follows the paper: per site, ``A`` is N x h_in (layer inputs), ``D`` is
N x h_out (back-propagated errors, the paper's Delta), the local gradient is
``A.T @ D`` (Eq. "local_grad"), ``Q`` (r x h_out, orthonormal rows) and ``P``
(r x h_in) are the rank-r factors of Algorithm 2 and ``P.T @ Q`` the estimate.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dad_oracle.c")
_SO = os.path.join(_HERE, "libdad_oracle.so")
_lock = threading.Lock()
_lib = None
_SO_OVERRIDE = None

_f64p = ctypes.POINTER(ctypes.c_double)
_u64p = ctypes.POINTER(ctypes.c_uint64)
_i64 = ctypes.c_int64


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (-O2, OpenMP) into ``libdad_oracle.so``."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-Wall", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _SO)
    return _SO


def lib() -> ctypes.CDLL:
    global _lib
    with _lock:
        if _lib is None:
            L = ctypes.CDLL(_SO_OVERRIDE or build())
            L.dad_oracle_max_threads.restype = ctypes.c_int
            L.dad_oracle_full_grad.argtypes = [ctypes.c_int, _i64, _i64, _i64, _f64p, _f64p, _f64p]
            L.dad_oracle_full_grad.restype = None
            L.dad_oracle_reconstruct.argtypes = [_i64, _i64, _i64, _f64p, _f64p, _f64p]
            L.dad_oracle_reconstruct.restype = None
            L.dad_oracle_orth.argtypes = [_i64, _i64, _f64p, _f64p]
            L.dad_oracle_orth.restype = None
            L.dad_oracle_spi_block.argtypes = [ctypes.c_int, _i64, _i64, _i64, _i64, ctypes.c_int,
                                               _f64p, _f64p, _f64p, _f64p, _f64p, _f64p]
            L.dad_oracle_spi_block.restype = ctypes.c_int
            L.dad_oracle_spi_paper_site.argtypes = [_i64, _i64, _i64, _i64, ctypes.c_int,
                                                    _f64p, _f64p, _f64p, _f64p, _f64p, _f64p]
            L.dad_oracle_spi_paper_site.restype = ctypes.c_int
            L.dad_oracle_bytes_dad.argtypes = [_i64, _i64, _i64, ctypes.c_int]
            L.dad_oracle_bytes_dad.restype = ctypes.c_uint64
            L.dad_oracle_bytes_rank.argtypes = [_i64, _i64, _i64]
            L.dad_oracle_bytes_rank.restype = ctypes.c_uint64
            L.dad_oracle_bytes_dsgd.argtypes = [_i64, _i64]
            L.dad_oracle_bytes_dsgd.restype = ctypes.c_uint64
            L.dad_oracle_gather.argtypes = [ctypes.c_int, _i64, _i64, _i64, _f64p, _f64p, _f64p, _f64p, _u64p]
            L.dad_oracle_gather.restype = None
            _lib = L
    return _lib


class use_library:
    """Context manager (tests only): route every call to another build of the C file, e.g. a
    copy with a planted mistake, to show that the pins notice it."""

    def __init__(self, so_path: str):
        self.so_path = so_path

    def __enter__(self):
        global _lib
        lib()
        self._saved = _lib
        _lib = None
        global _SO_OVERRIDE
        _SO_OVERRIDE = self.so_path
        lib()
        return self

    def __exit__(self, *exc):
        global _lib, _SO_OVERRIDE
        _lib = self._saved
        _SO_OVERRIDE = None
        return False


def max_threads() -> int:
    """Threads the OpenMP loops of the oracle may use on this machine."""
    return int(lib().dad_oracle_max_threads())


def widen(x) -> np.ndarray:
    """Exact float64 copy of ``x`` (numpy array, or a torch tensor of any float dtype)."""
    if hasattr(x, "detach"):  # torch tensor; bf16 has no numpy dtype, so go through double
        x = x.detach().to("cpu").double().numpy()
    return np.ascontiguousarray(np.asarray(x, dtype=np.float64))


def _p(a: np.ndarray):
    return a.ctypes.data_as(_f64p)


def _sites(A, D):
    A, D = widen(A), widen(D)
    if A.ndim == 2:
        A, D = A[None], D[None]
    assert A.ndim == 3 and D.ndim == 3 and A.shape[:2] == D.shape[:2], (A.shape, D.shape)
    return A, D


def full_grad(A, D) -> np.ndarray:
    """Uncompressed dAD gradient sum_s A_s^T D_s (Sec. 3.2).  A: S x N x h_in, D: S x N x h_out."""
    A, D = _sites(A, D)
    S, N, h_in = A.shape
    h_out = D.shape[2]
    G = np.empty((h_in, h_out), dtype=np.float64)
    lib().dad_oracle_full_grad(S, N, h_in, h_out, _p(A), _p(D), _p(G))
    return G


def reconstruct(Pcat, Qcat) -> np.ndarray:
    """Gradient estimate Pcat^T Qcat from the stacked factors (Algorithm 1)."""
    Pcat, Qcat = widen(Pcat), widen(Qcat)
    K, h_in = Pcat.shape
    assert Qcat.shape[0] == K
    h_out = Qcat.shape[1]
    G = np.empty((h_in, h_out), dtype=np.float64)
    lib().dad_oracle_reconstruct(K, h_in, h_out, _p(Pcat), _p(Qcat), _p(G))
    return G


def orth(G):
    """Orthonormalise the rows of G (r x h) in order; returns (Q, Rdiag)."""
    Q = widen(G).copy()
    r, h = Q.shape
    R = np.empty(r, dtype=np.float64)
    lib().dad_oracle_orth(r, h, _p(Q), _p(R))
    return Q, R


def spi_block(A, D, Q0, iters: int):
    """Blocked structured power iteration per site (Algorithm 2, all r vectors together).

    A: S x N x h_in, D: S x N x h_out, Q0: S x r x h_out  ->  P (S x r x h_in),
    Q (S x r x h_out), sigma (S x r).  2-D inputs are taken as a single site.
    """
    single = np.asarray(Q0).ndim == 2 if not hasattr(Q0, "detach") else Q0.dim() == 2
    A, D = _sites(A, D)
    Q0 = widen(Q0)
    if Q0.ndim == 2:
        Q0 = Q0[None]
    S, N, h_in = A.shape
    h_out = D.shape[2]
    r = Q0.shape[1]
    assert Q0.shape == (S, r, h_out) and iters >= 0
    P = np.empty((S, r, h_in), dtype=np.float64)
    Q = np.empty((S, r, h_out), dtype=np.float64)
    sig = np.empty((S, r), dtype=np.float64)
    rc = lib().dad_oracle_spi_block(S, N, h_in, h_out, r, int(iters), _p(A), _p(D), _p(Q0), _p(P), _p(Q), _p(sig))
    if rc:
        raise MemoryError("dad_oracle_spi_block")
    if single:
        return P[0], Q[0], sig[0]
    return P, Q, sig


def spi_paper(A, D, Q0, n_iter: int):
    """Algorithm 2 one vector at a time with deflation, for a single site (2-D inputs)."""
    A, D, Q0 = widen(A), widen(D), widen(Q0)
    N, h_in = A.shape
    h_out = D.shape[1]
    r = Q0.shape[0]
    P = np.zeros((r, h_in), dtype=np.float64)
    Q = np.zeros((r, h_out), dtype=np.float64)
    sig = np.zeros(r, dtype=np.float64)
    rc = lib().dad_oracle_spi_paper_site(N, h_in, h_out, r, int(n_iter), _p(A), _p(D), _p(Q0), _p(P), _p(Q), _p(sig))
    if rc:
        raise MemoryError("dad_oracle_spi_paper_site")
    return P, Q, sig


def gather(P, Q):
    """Stack all sites' factors (vertcat, Algorithm 1) and charge each site its bytes."""
    P, Q = widen(P), widen(Q)
    S, r, h_in = P.shape
    h_out = Q.shape[2]
    Pcat = np.empty((S * r, h_in), dtype=np.float64)
    Qcat = np.empty((S * r, h_out), dtype=np.float64)
    tx = np.zeros(S, dtype=np.uint64)
    lib().dad_oracle_gather(S, r, h_in, h_out, _p(P), _p(Q), _p(Pcat), _p(Qcat), tx.ctypes.data_as(_u64p))
    return Pcat, Qcat, tx


def bytes_dad(N: int, h_in: int, h_out: int, elem_bytes: int) -> int:
    return int(lib().dad_oracle_bytes_dad(N, h_in, h_out, elem_bytes))


def bytes_rank(r: int, h_in: int, h_out: int) -> int:
    return int(lib().dad_oracle_bytes_rank(r, h_in, h_out))


def bytes_dsgd(h_in: int, h_out: int) -> int:
    return int(lib().dad_oracle_bytes_dsgd(h_in, h_out))


def rank_dad_layer(A, D, Q0, iters: int):
    """The whole per-layer path: per-site SPI -> gather -> reconstruct.  Returns a dict."""
    P, Q, sig = spi_block(A, D, Q0, iters)
    Pcat, Qcat, tx = gather(P, Q)
    return {"P": P, "Q": Q, "sigma": sig, "Pcat": Pcat, "Qcat": Qcat, "bytes_tx": tx,
            "grad": reconstruct(Pcat, Qcat)}


def aggregate_spi(Pcat, Qcat, Q0, iters: int):
    """Second structured power iteration at the aggregator (Algorithm 1, "SPI(Q_i, G_i)"): the stacks take
    the places of the component matrices (A = Pcat, D = Qcat, one slice of K rows).  Returns Phat, Qhat, sigma."""
    return spi_block(widen(Pcat), widen(Qcat), widen(Q0), iters)


def two_stage_layer(A, D, Q0, iters: int, Q0_agg, iters_agg: int):
    """rank-dAD as Algorithm 1 prints it: per-site SPI, vertcat, SPI of the stacks, Phat^T Qhat."""
    first = rank_dad_layer(A, D, Q0, iters)
    Ph, Qh, sg = aggregate_spi(first["Pcat"], first["Qcat"], Q0_agg, iters_agg)
    r_agg = Ph.shape[0]
    h_in, h_out = Ph.shape[1], Qh.shape[1]
    first.update({"Phat": Ph, "Qhat": Qh, "sigma_hat": sg, "grad_hat": reconstruct(Ph, Qh),
                  "bytes_down": bytes_rank(r_agg, h_in, h_out)})
    return first


def effective_rank(sigma, theta: float) -> np.ndarray:
    """Leading components kept per site: sigma_j > theta * sigma_1, decided in fp32.  sigma: S x r."""
    sg = np.ascontiguousarray(np.asarray(sigma, dtype=np.float32))
    if sg.ndim == 1:
        sg = sg[None]
    S, r = sg.shape
    out = np.zeros(S, dtype=np.int32)
    L = lib()
    L.dad_oracle_effective_rank.argtypes = [ctypes.c_int, _i64, ctypes.POINTER(ctypes.c_float), ctypes.c_float,
                                            ctypes.POINTER(ctypes.c_int32)]
    L.dad_oracle_effective_rank.restype = None
    L.dad_oracle_effective_rank(S, r, sg.ctypes.data_as(ctypes.POINTER(ctypes.c_float)), ctypes.c_float(theta),
                                out.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)))
    return out


def truncate(P, Q, r_eff):
    """Factors with the components j >= r_eff[s] of site s dropped (set to zero)."""
    P, Q = widen(P).copy(), widen(Q).copy()
    for s, k in enumerate(np.asarray(r_eff)):
        P[s, int(k):] = 0.0
        Q[s, int(k):] = 0.0
    return P, Q


def spi_gram(A, D, Q0, iters: int):
    """Algorithm 2 with C = A A^T and B = D^T C formed explicitly (the paper's own N << h form), per site.
    Same arguments and results as spi_block."""
    single = np.asarray(Q0).ndim == 2 if not hasattr(Q0, "detach") else Q0.dim() == 2
    A, D = _sites(A, D)
    Q0 = widen(Q0)
    if Q0.ndim == 2:
        Q0 = Q0[None]
    S, N, h_in = A.shape
    h_out, r = D.shape[2], Q0.shape[1]
    P = np.empty((S, r, h_in))
    Q = np.empty((S, r, h_out))
    sig = np.empty((S, r))
    L = lib()
    L.dad_oracle_spi_gram_site.argtypes = [_i64, _i64, _i64, _i64, ctypes.c_int, _f64p, _f64p, _f64p, _f64p, _f64p, _f64p]
    L.dad_oracle_spi_gram_site.restype = ctypes.c_int
    for s in range(S):
        a, d, q0 = np.ascontiguousarray(A[s]), np.ascontiguousarray(D[s]), np.ascontiguousarray(Q0[s])
        if L.dad_oracle_spi_gram_site(N, h_in, h_out, r, int(iters), _p(a), _p(d), _p(q0), _p(P[s]), _p(Q[s]), _p(sig[s])):
            raise MemoryError("dad_oracle_spi_gram_site")
    if single:
        return P[0], Q[0], sig[0]
    return P, Q, sig
