"""CPU fp64 oracle for cyclic coordinate descent with fixed codebooks (GuidedQuant Section 4.2, Eq. 10;
Appendix B.2, Algorithms 3 and 4).

TEST INFRASTRUCTURE ONLY (see ``gq_oracle.py``): imported by ``tests/`` and by measurement scripts that
time the CPU side; the product package never imports it.

Three statements of the same method:

* :func:`cd` -- ``cd_oracle.c``: Algorithm 4 (precomputation + lazy batch-updates) step by step in fp64
  (``b >= d_in`` gives Algorithm 3);
* :func:`cd_rowwise` -- Algorithm 3 written with numpy fp64 matrix primitives;
* :func:`cd_naive` -- the method's definition with no algebra at all: cyclic CD in which every coordinate
  is set to the codebook value that gives the smallest objective, found by evaluating the objective
  for each of the m candidates (pure Python, tiny inputs only).

Conventions: ``W``, ``W_hat`` fp32 ``[d_out, d_in]`` (row j = output channel j), ``H`` ``[g, d_in, d_in]``
full symmetric, ``codebook`` fp32 ``[d_out, m]``; codes are 0-based indices.  Ties in rounding go to the
smaller index; a coordinate with ``H_ii <= 0`` is rounded to the value nearest to ``W_ij``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "cd_oracle.c")
_LIB = os.path.join(_HERE, "libcd_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _c():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i64, i32, vp = ctypes.c_int64, ctypes.c_int32, ctypes.c_void_p
        lib.gq_oracle_cd.argtypes = [vp, vp, vp, vp, i32, i64, i64, vp, i32, i32, i64]
        lib.gq_oracle_cd.restype = ctypes.c_int
        _lib = lib
    return _lib


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def cd(W, W_hat0, codebook, H, cycles: int = 1, b: int = 128):
    """Algorithm 4.  Returns ``(W_hat fp32 [d_out, d_in], Q int32 [d_out, d_in])``."""
    W, What, cbk, H32 = _f32(W), _f32(W_hat0).copy(), _f32(codebook), _f32(H)
    d_out, d_in = W.shape
    g = H32.shape[0]
    assert H32.shape == (g, d_in, d_in) and cbk.shape[0] == d_out and d_out % g == 0
    Q = np.zeros((d_out, d_in), dtype=np.int32)
    rc = _c().gq_oracle_cd(W.ctypes.data, What.ctypes.data, Q.ctypes.data, cbk.ctypes.data, cbk.shape[1], d_in, d_out,
                           H32.ctypes.data, g, cycles, b)
    if rc != 0:
        raise ValueError("gq_oracle_cd rejected the sizes")
    return What, Q


def round_to_codebook(x: np.ndarray, codebook: np.ndarray):
    """Row j of x ([d_out] or [d_out, r]) to the nearest value of codebook[j]; ties to the smaller index."""
    x = np.asarray(x, dtype=np.float64)
    cbk = np.asarray(codebook, dtype=np.float64)
    dist = np.abs(x[..., None] - (cbk[:, None, :] if x.ndim == 2 else cbk))
    q = np.argmin(dist, axis=-1)                     # argmin returns the first minimiser
    val = np.take_along_axis(cbk[:, None, :] if x.ndim == 2 else cbk, q[..., None], axis=-1)[..., 0]
    return val, q.astype(np.int32)


def cd_rowwise(W, W_hat0, codebook, H, cycles: int = 1):
    """Algorithm 3 with numpy fp64 primitives: B = StrictUpper(Htilde)(What - W), then row by row."""
    W = np.asarray(W, dtype=np.float64)
    What = np.asarray(W_hat0, dtype=np.float64).copy()
    cbk = np.asarray(codebook, dtype=np.float64)
    H = np.asarray(H, dtype=np.float64)
    d_out, d_in = W.shape
    g = H.shape[0]
    mk = d_out // g
    Q = np.zeros((d_out, d_in), dtype=np.int32)
    for k in range(g):
        sl = slice(k * mk, (k + 1) * mk)
        diag = np.diag(H[k]).copy()
        Ht = np.where(diag[:, None] > 0, H[k] / np.where(diag > 0, diag, 1.0)[:, None], 0.0)
        U = np.triu(Ht, 1)
        for _ in range(cycles):
            Bm = U @ (What[sl] - W[sl]).T                                  # [d_in, mk]
            for i in range(d_in):
                val, q = round_to_codebook(W[sl, i] - Bm[i], cbk[sl])
                What[sl, i] = val
                Q[sl, i] = q
                if i + 1 < d_in:
                    Bm[i + 1:] += np.outer(Ht[i + 1:, i], What[sl, i] - W[sl, i])
    return What.astype(np.float32), Q


def coordinate_target(w_j: np.ndarray, what_j: np.ndarray, Hk: np.ndarray, i: int):
    """The argument of Round_j in Eq. 10 for coordinate i of one channel, given the channel's current
    quantised weights: ``W_ij - sum_{c != i} H_ic / H_ii (What_cj - W_cj)``; also returns the magnitude
    ``|W_ij| + sum_{c != i} |H_ic / H_ii (What_cj - W_cj)|`` of what was summed."""
    w = np.asarray(w_j, dtype=np.float64)
    e = np.asarray(what_j, dtype=np.float64) - w
    h = np.asarray(Hk[i], dtype=np.float64)
    if h[i] <= 0:
        return float(w[i]), float(abs(w[i]))
    terms = h / h[i] * e
    terms[i] = 0.0
    return float(w[i] - terms.sum()), float(abs(w[i]) + np.abs(terms).sum())


def channel_objective(delta: np.ndarray, Hk: np.ndarray) -> float:
    """delta^T H_k delta (one term of Eq. 7)."""
    return float(delta @ Hk @ delta)


def cd_naive(W, W_hat0, codebook, H, cycles: int = 1):
    """Cyclic CD by exhaustive evaluation of the objective (tiny inputs only)."""
    W = np.asarray(W, dtype=np.float64)
    What = np.asarray(W_hat0, dtype=np.float64).copy()
    cbk = np.asarray(codebook, dtype=np.float64)
    H = np.asarray(H, dtype=np.float64)
    d_out, d_in = W.shape
    g = H.shape[0]
    mk = d_out // g
    Q = np.zeros((d_out, d_in), dtype=np.int32)
    for _ in range(cycles):
        for j in range(d_out):
            Hk = H[j // mk]
            for i in range(d_in):
                best, best_q = None, 0
                for q in range(cbk.shape[1]):
                    trial = What[j].copy()
                    trial[i] = cbk[j, q]
                    f = channel_objective(trial - W[j], Hk)
                    if best is None or f < best:
                        best, best_q = f, q
                What[j, i] = cbk[j, best_q]
                Q[j, i] = best_q
    return What.astype(np.float32), Q


# --------------------------------------------------------------------------------------------------------
# Codebook step and the LNQ loop (Section 4.2, Eq. 8; Algorithm 2)

def one_hot(q_j: np.ndarray, m: int) -> np.ndarray:
    """Assignment matrix P^(j) in {0,1}^{d_in x m} of one channel from its codes."""
    P = np.zeros((q_j.shape[0], m), dtype=np.float64)
    P[np.arange(q_j.shape[0]), q_j] = 1.0
    return P


def codebook_update(W, Q, H, m: int, lam: float = 1e-7) -> np.ndarray:
    """Eq. 8 for every channel: c^(j) = (P^T H_k P + lam I)^-1 P^T H_k w_j, with the small constant lam on the
    diagonal that the text below Eq. 8 prescribes (1e-7 in the paper).  Returns fp64 [d_out, m]."""
    W = np.asarray(W, dtype=np.float64)
    H = np.asarray(H, dtype=np.float64)
    d_out, d_in = W.shape
    mk = d_out // H.shape[0]
    C = np.zeros((d_out, m), dtype=np.float64)
    for j in range(d_out):
        Hk = H[j // mk]
        P = one_hot(np.asarray(Q[j]), m)
        G = P.T @ Hk @ P + lam * np.eye(m)
        r = P.T @ (Hk @ W[j])
        C[j] = np.linalg.solve(G, r)
    return C


def lnq(W, Q0, H, m: int, T: int, K: int, lam: float = 1e-7, b: int = 128):
    """Algorithm 2: T rounds of (codebook step, K CD cycles), then a final codebook step.
    Returns (W_hat fp32 [d_out, d_in], Q int32, codebook fp32 [d_out, m])."""
    W32 = np.ascontiguousarray(W, dtype=np.float32)
    Q = np.asarray(Q0, dtype=np.int32).copy()
    for _ in range(T):
        cbk = codebook_update(W32, Q, H, m, lam).astype(np.float32)
        What = np.take_along_axis(cbk, Q, axis=1)
        What, Q = cd(W32, What, cbk, H, K, b)
    cbk = codebook_update(W32, Q, H, m, lam).astype(np.float32)
    return np.take_along_axis(cbk, Q, axis=1), Q, cbk
