"""CPU fp64 oracle for the guided layer objective (GuidedQuant, Section 3.2).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by ``__graft_entry__.smoke``
and by the ``cpu_baseline`` / ``--impl reference`` legs of ``bench.py``.  The
product package never imports it and it never imports the product's CUDA path.

Two independent statements of the same definitions live here:

* ``impl="c"`` -- ``gq_oracle.c``: entry-by-entry fp64 loops (the oracle of
  record; fast enough for token prefixes of the large layers);
* ``impl="numpy"`` -- the definitions written with numpy fp64 library
  primitives (``einsum`` / ``@``), used to cross-check the C loops and for
  tiny cases.

Array conventions (identical to the C-ABI library so the same buffers serve
both sides): ``grad`` and ``X`` are ``uint16`` arrays holding bf16 bit patterns,
row = token; ``s`` is ``[g, n]``; ``H`` is ``[g, d_in, d_in]``; ``W``/``W_hat``
are fp32 ``[d_out, d_in]`` with row ``j`` = output channel ``j`` (the paper's
column ``w_j``, Section 2).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gq_oracle.c")
_LIB = os.path.join(_HERE, "libgq_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile ``gq_oracle.c`` with gcc (OpenMP) next to its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def _c():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i64, i32, dbl, vp = ctypes.c_int64, ctypes.c_int32, ctypes.c_double, ctypes.c_void_p
        lib.gq_oracle_saliency.argtypes = [vp, i64, i64, i64, i32, dbl, vp, i64]
        lib.gq_oracle_hessian_accumulate.argtypes = [vp, i64, i64, i64, vp, i64, i32, vp]
        lib.gq_oracle_objective.argtypes = [vp, vp, i64, i64, vp, i32, vp]
        lib.gq_oracle_saliency_strided.argtypes = [vp, i32, i64, i64, i64, i64, i64, i32, dbl, vp, i64]
        lib.gq_oracle_saliency_strided.restype = ctypes.c_int
        lib.gq_oracle_hessian_diag.argtypes = [vp, i64, i64, i64, vp, i64, i32, vp]
        lib.gq_oracle_hessian_apply.argtypes = [vp, i64, i64, i64, vp, i64, i32, vp, i32, vp]
        for f in (lib.gq_oracle_saliency, lib.gq_oracle_hessian_accumulate, lib.gq_oracle_objective,
                  lib.gq_oracle_hessian_diag, lib.gq_oracle_hessian_apply, lib.gq_oracle_threads):
            f.restype = ctypes.c_int
        _lib = lib
    return _lib


def threads() -> int:
    return int(_c().gq_oracle_threads())


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns (uint16) to fp64 exactly."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def f64_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp64/fp32 values to bf16 (nearest, ties to even); for building test inputs."""
    f = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    rounded = (f + 0x7FFF + ((f >> 16) & 1)) >> 16
    return rounded.astype(np.uint16)


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def saliency(grad_bits: np.ndarray, g: int, grad_scale: float = 1.0, impl: str = "c") -> np.ndarray:
    """Algorithm 1, saliency step: ``s[k, i] = mean_{j in J_k} (grad_scale * grad[i, j])**2``."""
    grad_bits = np.ascontiguousarray(grad_bits, dtype=np.uint16)
    n, d_out = grad_bits.shape
    if g < 1 or d_out % g:
        raise ValueError("d_out must be divisible by g")
    if impl == "numpy":
        gr = bf16_bits_to_f64(grad_bits) * float(grad_scale)
        return np.ascontiguousarray((gr * gr).reshape(n, g, d_out // g).mean(axis=2).T)
    s = np.zeros((g, n), dtype=np.float64)
    rc = _c().gq_oracle_saliency(_ptr(grad_bits), n, d_out, d_out, g, float(grad_scale), _ptr(s), n)
    if rc:
        raise RuntimeError("gq_oracle_saliency rc=%d" % rc)
    return s


DTYPE_CODES = {"bf16": 0, "fp16": 1, "fp32": 2}


def saliency_strided(grad: np.ndarray, dtype: str, g: int, grad_scale: float = 1.0, impl: str = "c") -> np.ndarray:
    """Algorithm 1's saliency for a gradient as autograd hands it over: ``grad`` is ``[batch, seq, d_out]`` with a
    contiguous last dimension and arbitrary (non-negative) strides of the first two, holding bf16 bit patterns
    (``uint16``, dtype "bf16"), IEEE half (``float16``, "fp16") or ``float32`` ("fp32").  Token ``i = b * seq + t``.
    Returns fp64 ``[g, batch * seq]``."""
    if grad.ndim != 3 or (grad.shape[2] > 1 and grad.strides[2] != grad.itemsize):
        raise ValueError("grad must be [batch, seq, d_out] with a contiguous last dimension")
    want = {"bf16": np.uint16, "fp16": np.float16, "fp32": np.float32}[dtype]
    if grad.dtype != want:
        raise ValueError("dtype %s needs a %s array" % (dtype, want))
    batch, seq, d_out = grad.shape
    if g < 1 or d_out % g:
        raise ValueError("d_out must be divisible by g")
    n = batch * seq
    if impl == "numpy":
        wide = bf16_bits_to_f64(np.ascontiguousarray(grad)).reshape(grad.shape) if dtype == "bf16" else grad.astype(np.float64)
        gr = wide.reshape(n, g, d_out // g) * float(grad_scale)
        return np.ascontiguousarray((gr * gr).mean(axis=2).T)
    s = np.zeros((g, n), dtype=np.float64)
    sb, st = grad.strides[0] // grad.itemsize, grad.strides[1] // grad.itemsize
    rc = _c().gq_oracle_saliency_strided(ctypes.c_void_p(grad.ctypes.data), DTYPE_CODES[dtype], batch, seq, d_out, sb, st, g,
                                         float(grad_scale), _ptr(s), n)
    if rc:
        raise RuntimeError("gq_oracle_saliency_strided rc=%d" % rc)
    return s


def hessian(x_bits: np.ndarray, s: np.ndarray, H: np.ndarray | None = None, impl: str = "c") -> np.ndarray:
    """Algorithm 1, Hessian step: ``H[k] (+)= X^T Diag(s[k]) X`` (full matrices, no 1/n).

    Passing ``H`` accumulates into it (streaming over token chunks)."""
    x_bits = np.ascontiguousarray(x_bits, dtype=np.uint16)
    s = np.ascontiguousarray(s, dtype=np.float64)
    n, d_in = x_bits.shape
    g = s.shape[0]
    if s.shape[1] != n:
        raise ValueError("s must be [g, n]")
    if H is None:
        H = np.zeros((g, d_in, d_in), dtype=np.float64)
    assert H.shape == (g, d_in, d_in) and H.dtype == np.float64 and H.flags.c_contiguous
    if impl == "numpy":
        x = bf16_bits_to_f64(x_bits)
        for k in range(g):
            H[k] += (x * s[k][:, None]).T @ x
        return H
    rc = _c().gq_oracle_hessian_accumulate(_ptr(x_bits), n, d_in, d_in, _ptr(s), n, g, _ptr(H))
    if rc:
        raise RuntimeError("gq_oracle_hessian_accumulate rc=%d" % rc)
    return H


def _is_widened(x) -> bool:
    """True for activations already widened to fp64 (``bf16_bits_to_f64`` of the bit patterns): the numpy
    statements of the two O(n d_in) forms accept either, so a caller streaming large chunks widens once."""
    return isinstance(x, np.ndarray) and x.dtype == np.float64


def hessian_diag(x_bits: np.ndarray, s: np.ndarray, diag: np.ndarray | None = None, impl: str = "c") -> np.ndarray:
    """The diagonal of Algorithm 1's guided Hessians straight from their definition,
    ``diag[k, a] (+)= sum_i s[k, i] * X[i, a]**2`` -- O(n d_in) per group, so it can be formed for all
    tokens of the large layers.  Passing ``diag`` accumulates into it (streaming over token chunks).
    ``x_bits``: bf16 bit patterns, or (numpy statement only) the same values already widened to fp64."""
    wide = _is_widened(x_bits)
    x_bits = x_bits if wide else np.ascontiguousarray(x_bits, dtype=np.uint16)
    s = np.ascontiguousarray(s, dtype=np.float64)
    n, d_in = x_bits.shape
    g = s.shape[0]
    if s.shape[1] != n:
        raise ValueError("s must be [g, n]")
    if diag is None:
        diag = np.zeros((g, d_in), dtype=np.float64)
    assert diag.shape == (g, d_in) and diag.dtype == np.float64 and diag.flags.c_contiguous
    if impl == "numpy":
        x = x_bits if wide else bf16_bits_to_f64(x_bits)
        diag += s @ (x * x)
        return diag
    if wide:
        raise ValueError("the C loops take bf16 bit patterns")
    rc = _c().gq_oracle_hessian_diag(_ptr(x_bits), n, d_in, d_in, _ptr(s), n, g, _ptr(diag))
    if rc:
        raise RuntimeError("gq_oracle_hessian_diag rc=%d" % rc)
    return diag


def hessian_apply(x_bits: np.ndarray, s: np.ndarray, V: np.ndarray, out: np.ndarray | None = None,
                  impl: str = "c") -> np.ndarray:
    """The guided Hessians applied to probe vectors without forming them,
    ``out[k, v] (+)= X^T (s[k] * (X V[v]))`` ( = H_k V[v] by the definition of H_k) -- O(n d_in) per group
    and probe.  ``V`` is ``[nv, d_in]``; passing ``out`` (``[g, nv, d_in]``) accumulates over token chunks."""
    wide = _is_widened(x_bits)
    x_bits = x_bits if wide else np.ascontiguousarray(x_bits, dtype=np.uint16)
    s = np.ascontiguousarray(s, dtype=np.float64)
    V = np.ascontiguousarray(V, dtype=np.float64)
    n, d_in = x_bits.shape
    g, nv = s.shape[0], V.shape[0]
    if s.shape[1] != n or V.shape[1] != d_in:
        raise ValueError("shape mismatch")
    if out is None:
        out = np.zeros((g, nv, d_in), dtype=np.float64)
    assert out.shape == (g, nv, d_in) and out.dtype == np.float64 and out.flags.c_contiguous
    if impl == "numpy":
        x = x_bits if wide else bf16_bits_to_f64(x_bits)
        y = x @ V.T                                                     # [n, nv]: x_i . V[v]
        z = (s[:, :, None] * y[None, :, :]).transpose(1, 0, 2).reshape(n, g * nv)      # s[k, i] * y[i, v]
        out += (x.T @ z).T.reshape(g, nv, d_in)
        return out
    if wide:
        raise ValueError("the C loops take bf16 bit patterns")
    rc = _c().gq_oracle_hessian_apply(_ptr(x_bits), n, d_in, d_in, _ptr(s), n, g, _ptr(V), nv, _ptr(out))
    if rc:
        raise RuntimeError("gq_oracle_hessian_apply rc=%d" % rc)
    return out


def objective(W: np.ndarray, W_hat: np.ndarray, H: np.ndarray, impl: str = "c") -> np.ndarray:
    """Eq. 7: ``loss[k] = sum_{j in J_k} (w_j - what_j)^T H[k] (w_j - what_j)``; ``loss[g]`` = total."""
    W = np.ascontiguousarray(W, dtype=np.float32)
    W_hat = np.ascontiguousarray(W_hat, dtype=np.float32)
    H = np.ascontiguousarray(H, dtype=np.float64)
    d_out, d_in = W.shape
    g = H.shape[0]
    if W_hat.shape != W.shape or H.shape != (g, d_in, d_in) or d_out % g:
        raise ValueError("shape mismatch")
    loss = np.zeros(g + 1, dtype=np.float64)
    if impl == "numpy":
        m = d_out // g
        delta = W.astype(np.float64) - W_hat.astype(np.float64)
        for k in range(g):
            dk = delta[k * m:(k + 1) * m]
            loss[k] = np.einsum("ja,ab,jb->", dk, H[k], dk, optimize=True)
        loss[g] = loss[:g].sum()
        return loss
    rc = _c().gq_oracle_objective(_ptr(W), _ptr(W_hat), d_in, d_out, _ptr(H), g, _ptr(loss))
    if rc:
        raise RuntimeError("gq_oracle_objective rc=%d" % rc)
    return loss
