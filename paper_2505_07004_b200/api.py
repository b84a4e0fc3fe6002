"""ctypes binding of the C-ABI library ``libgq.so`` (declared in ``include/gq.h``).

Argument marshalling only: every function here checks dtypes/devices, passes raw
device pointers and the current CUDA stream to the entry point of the same name,
and raises :class:`GQError` on a non-zero status.  PyTorch is used for device
memory and streams; no arithmetic of the method runs in Python and there is no
CPU fallback: if ``libgq.so`` is missing or no CUDA device is present the calls fail.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libgq.so")
_lib = None

EXPORTS = (
    "gq_version", "gq_status_string", "gq_last_cuda_error", "gq_saliency", "gq_saliency_prepared", "gq_saliency_strided", "gq_hessian_accumulate",
    "gq_hessian_accumulate_ahead",
    "gq_hessian_workspace_bytes", "gq_hessian_finalize", "gq_objective", "gq_objective_workspace_bytes",
    "gq_layer_objective_host", "gq_layer_host_arena_bytes", "gq_check", "gq_launch_count",
    "gq_kernel_timing_enable", "gq_kernel_timing_read", "gq_objective_noalloc", "gq_cd_cycles", "gq_cd_workspace_bytes",
    "gq_selftest_wait_timeout", "gq_codebook_update", "gq_codebook_workspace_bytes",
    "gq_hessian_reduce_share", "gq_hessian_gather_shares", "gq_lnq", "gq_lnq_workspace_bytes",
)
GQ_HESSIAN_DETERMINISTIC = 1      # flag of gq_hessian_accumulate: single writer per element of H
GQ_HESSIAN_S_PREPARED = 2         # flag of gq_hessian_accumulate: the workspace was filled by gq_saliency_prepared
KERNEL_NAMES = ("saliency", "hessian", "mirror", "split_delta", "gram_dot", "reduce", "split_saliency", "cd_panel",
                "cd_block", "cd_aux", "cb_gemm", "cb_fold", "cb_aux", "exchange")


class GQError(RuntimeError):
    def __init__(self, fn: str, status: int):
        self.status = status
        name = lib().gq_status_string(status).decode()
        extra = ""
        if name == "GQ_ERR_CUDA":
            extra = " (cudaError %d)" % lib().gq_last_cuda_error()
        super().__init__("%s failed: %s%s" % (fn, name, extra))


def lib() -> ctypes.CDLL:
    """Loads the in-tree ``libgq.so``; fails loudly if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                "libgq.so not found at %s: build it with `python -m paper_2505_07004_b200.build` "
                "(there is no CPU fallback)" % LIB_PATH)
        L = ctypes.CDLL(LIB_PATH)
        i64, i32, u32, f32, vp, sz = (ctypes.c_int64, ctypes.c_int32, ctypes.c_uint32, ctypes.c_float,
                                      ctypes.c_void_p, ctypes.c_size_t)
        L.gq_version.restype = ctypes.c_int
        L.gq_status_string.restype = ctypes.c_char_p
        L.gq_status_string.argtypes = [i32]
        L.gq_last_cuda_error.restype = i32
        L.gq_launch_count.restype = ctypes.c_uint64
        L.gq_saliency.restype = i32
        L.gq_saliency.argtypes = [vp, i64, i64, i64, i32, f32, vp, i64, vp]
        L.gq_saliency_prepared.restype = i32
        L.gq_saliency_prepared.argtypes = [vp, i64, i64, i64, i32, f32, vp, i64, vp, sz, vp]
        L.gq_saliency_strided.restype = i32
        L.gq_saliency_strided.argtypes = [vp, i32, i64, i64, i64, i64, i64, i32, f32, vp, i64, vp]
        L.gq_hessian_workspace_bytes.restype = sz
        L.gq_hessian_workspace_bytes.argtypes = [i64, i64, i32, u32]
        L.gq_hessian_accumulate.restype = i32
        L.gq_hessian_accumulate.argtypes = [vp, i64, i64, i64, vp, i64, i32, vp, u32, vp, sz, vp]
        L.gq_hessian_accumulate_ahead.restype = i32
        L.gq_hessian_accumulate_ahead.argtypes = [vp, i64, i64, i64, vp, i64, i32, vp, u32, vp, sz,
                                                  vp, i64, i64, i64, f32, vp, i64, vp, sz, vp]
        L.gq_hessian_finalize.restype = i32
        L.gq_hessian_finalize.argtypes = [vp, i64, i32, vp]
        for f in (L.gq_hessian_reduce_share, L.gq_hessian_gather_shares):
            f.restype = i32
            f.argtypes = [ctypes.POINTER(ctypes.c_void_p), i32, i32, i64, i32, vp]
        L.gq_objective_workspace_bytes.restype = sz
        L.gq_objective_workspace_bytes.argtypes = [i64, i64, i32]
        L.gq_objective.restype = i32
        L.gq_objective.argtypes = [vp, vp, i64, i64, vp, i32, vp, vp, sz, vp]
        L.gq_layer_host_arena_bytes.restype = sz
        L.gq_layer_host_arena_bytes.argtypes = [i64, i64, i64, i32]
        L.gq_layer_objective_host.restype = i32
        L.gq_layer_objective_host.argtypes = [vp, vp, i64, i64, i64, i64, i32, f32, vp, vp, vp, vp, vp, sz, vp]
        L.gq_check.restype = i32
        L.gq_check.argtypes = [vp, vp]
        L.gq_objective_noalloc.restype = i32
        L.gq_objective_noalloc.argtypes = [vp, vp, i64, i64, vp, i32, vp, vp]
        L.gq_cd_workspace_bytes.restype = sz
        L.gq_cd_workspace_bytes.argtypes = [i64, i64, i32]
        L.gq_cd_cycles.restype = i32
        L.gq_cd_cycles.argtypes = [vp, vp, vp, vp, i32, i64, i64, vp, i32, i32, vp, sz, vp]
        L.gq_codebook_workspace_bytes.restype = sz
        L.gq_codebook_workspace_bytes.argtypes = [i64, i64, i32, i32]
        L.gq_codebook_update.restype = i32
        L.gq_codebook_update.argtypes = [vp, vp, i32, i64, i64, vp, i32, ctypes.c_double, vp, vp, vp, sz, vp]
        L.gq_lnq_workspace_bytes.restype = sz
        L.gq_lnq_workspace_bytes.argtypes = [i64, i64, i32, i32]
        L.gq_lnq.restype = i32
        L.gq_lnq.argtypes = [vp, vp, i32, i64, i64, vp, i32, i32, i32, ctypes.c_double, vp, vp, vp, sz, vp]
        L.gq_selftest_wait_timeout.restype = i32
        L.gq_selftest_wait_timeout.argtypes = [i32, vp]
        L.gq_kernel_timing_enable.restype = i32
        L.gq_kernel_timing_enable.argtypes = [i32]
        L.gq_kernel_timing_read.restype = i32
        L.gq_kernel_timing_read.argtypes = [vp, vp]
        _lib = L
    return _lib


def _stream_ptr(stream: Optional[torch.cuda.Stream], device=None) -> int:
    st = stream if stream is not None else torch.cuda.current_stream(device)
    return int(st.cuda_stream)


def _same_device(*named):
    """The one CUDA device all given (name, tensor) pairs live on; ValueError if they differ.  The library
    launches on the CURRENT device, so every wrapper makes this device current around its call: pointers of one
    GPU must never reach kernels of another."""
    dev = None
    for name, t in named:
        if t is None:
            continue
        d = t.device
        if d.type != "cuda":
            raise ValueError("%s must be a CUDA tensor" % name)
        if dev is None:
            dev, first = d, name
        elif d != dev:
            raise ValueError("%s is on %s but %s is on %s: all arguments of a call must live on one device"
                             % (name, d, first, dev))
    if dev is None:
        raise ValueError("no device tensor given")
    return dev


class _on:
    """Context: make `device` current for a library call and resolve the stream on that device."""

    def __init__(self, device, stream):
        if stream is not None and getattr(stream, "device", device) != device:
            raise ValueError("stream belongs to %s, the tensors to %s" % (stream.device, device))
        self.guard = torch.cuda.device(device)
        self.device, self.stream = device, stream

    def __enter__(self) -> int:
        self.guard.__enter__()
        return _stream_ptr(self.stream, self.device)

    def __exit__(self, *exc):
        return self.guard.__exit__(*exc)


def _dev(t: torch.Tensor, dtype, name: str) -> torch.Tensor:
    if not t.is_cuda:
        raise ValueError("%s must be a CUDA tensor" % name)
    if t.dtype != dtype:
        raise ValueError("%s must be %s" % (name, dtype))
    return t


def _rows(t: torch.Tensor, name: str):
    """(n, width, leading dimension) of a 2-D tensor whose last dimension is contiguous."""
    if t.dim() != 2 or (t.shape[1] > 1 and t.stride(1) != 1):
        raise ValueError("%s must be 2-D with a contiguous last dimension" % name)
    return t.shape[0], t.shape[1], (t.stride(0) if t.shape[0] > 1 else max(t.shape[1], t.stride(0)))


def alloc_workspace(nbytes: int, device) -> torch.Tensor:
    """Device scratch of ``nbytes`` bytes whose base is 1024-byte aligned."""
    buf = torch.empty(int(nbytes) + 1024, dtype=torch.uint8, device=device)
    off = (-buf.data_ptr()) % 1024
    return buf[off:off + int(nbytes)]


def gq_version() -> int:
    return int(lib().gq_version())


def gq_launch_count() -> int:
    return int(lib().gq_launch_count())


def gq_saliency(grad: torch.Tensor, g: int, grad_scale: float = 1.0, s: Optional[torch.Tensor] = None,
                stream=None) -> torch.Tensor:
    """``s[k, i] = grad_scale**2 / m * sum_{j in J_k} grad[i, j]**2`` (Algorithm 1, saliency step)."""
    _dev(grad, torch.bfloat16, "grad")
    n, d_out, ld = _rows(grad, "grad")
    if s is None:
        s = torch.empty((g, n), dtype=torch.float32, device=grad.device)
    _dev(s, torch.float32, "s")
    _, s_n, ld_s = _rows(s, "s")
    if s.shape[0] != g or s_n < n:
        raise ValueError("s must be [g, >= n]")
    with _on(_same_device(("grad", grad), ("s", s)), stream) as st:
        rc = lib().gq_saliency(grad.data_ptr(), n, d_out, ld, g, float(grad_scale), s.data_ptr(), ld_s, st)
    if rc:
        raise GQError("gq_saliency", rc)
    return s


def gq_saliency_prepared(grad: torch.Tensor, g: int, hessian_workspace: torch.Tensor, grad_scale: float = 1.0,
                         s: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """:func:`gq_saliency` that also fills ``hessian_workspace`` with ``s`` in the form the Hessian kernel reads;
    the following :func:`gq_hessian_accumulate` for the same tokens is then called with
    ``flags=GQ_HESSIAN_S_PREPARED`` (one launch less per chunk)."""
    _dev(grad, torch.bfloat16, "grad")
    n, d_out, ld = _rows(grad, "grad")
    if s is None:
        s = torch.empty((g, n), dtype=torch.float32, device=grad.device)
    _dev(s, torch.float32, "s")
    _, s_n, ld_s = _rows(s, "s")
    if s.shape[0] != g or s_n < n:
        raise ValueError("s must be [g, >= n]")
    with _on(_same_device(("grad", grad), ("s", s), ("hessian_workspace", hessian_workspace)), stream) as st:
        rc = lib().gq_saliency_prepared(grad.data_ptr(), n, d_out, ld, g, float(grad_scale), s.data_ptr(), ld_s,
                                        hessian_workspace.data_ptr(),
                                        hessian_workspace.numel() * hessian_workspace.element_size(), st)
    if rc:
        raise GQError("gq_saliency_prepared", rc)
    return s


_DTYPE_CODES = {torch.bfloat16: 0, torch.float16: 1, torch.float32: 2}


def gq_saliency_strided(grad: torch.Tensor, g: int, grad_scale: float = 1.0, s: Optional[torch.Tensor] = None,
                        stream=None) -> torch.Tensor:
    """Saliency of a ``[batch, seq, d_out]`` gradient in bf16, fp16 or fp32 with arbitrary batch / sequence strides
    (a contiguous last dimension), e.g. the ``grad_output`` of a backward hook.  Writes ``s[k, b * seq + t]``;
    pass a view ``s_all[:, offset:offset + batch * seq]`` to fill a slice of a calibration-wide buffer in place."""
    if not grad.is_cuda or grad.dtype not in _DTYPE_CODES:
        raise ValueError("grad must be a CUDA tensor of dtype bfloat16, float16 or float32")
    if grad.dim() != 3 or (grad.shape[2] > 1 and grad.stride(2) != 1):
        raise ValueError("grad must be [batch, seq, d_out] with a contiguous last dimension")
    batch, seq, d_out = grad.shape
    n = batch * seq
    if s is None:
        s = torch.empty((g, n), dtype=torch.float32, device=grad.device)
    _dev(s, torch.float32, "s")
    _, s_n, ld_s = _rows(s, "s")
    if s.shape[0] != g or s_n < n:
        raise ValueError("s must be [g, >= batch * seq]")
    stride_b = grad.stride(0) if batch > 1 else max(grad.stride(0), seq * grad.stride(1))
    stride_t = grad.stride(1) if seq > 1 else max(grad.stride(1), d_out)
    with _on(_same_device(("grad", grad), ("s", s)), stream) as st:
        rc = lib().gq_saliency_strided(grad.data_ptr(), _DTYPE_CODES[grad.dtype], batch, seq, d_out, stride_b, stride_t, g,
                                       float(grad_scale), s.data_ptr(), ld_s, st)
    if rc:
        raise GQError("gq_saliency_strided", rc)
    return s


def gq_hessian_workspace_bytes(n_max: int, d_in: int, g: int, flags: int = 0) -> int:
    return int(lib().gq_hessian_workspace_bytes(n_max, d_in, g, flags))


def gq_hessian_accumulate(X: torch.Tensor, s: torch.Tensor, H: torch.Tensor, workspace: torch.Tensor,
                          flags: int = 0, stream=None) -> torch.Tensor:
    """``H[k] += X^T Diag(s[k]) X`` on the upper triangle (Algorithm 1, Hessian step), one token chunk."""
    _dev(X, torch.bfloat16, "X")
    _dev(s, torch.float32, "s")
    _dev(H, torch.float32, "H")
    n, d_in, ld_x = _rows(X, "X")
    g, s_n, ld_s = _rows(s, "s")
    if s_n < n:
        raise ValueError("s must be [g, >= n]")
    s_n = n
    if tuple(H.shape) != (g, d_in, d_in) or not H.is_contiguous():
        raise ValueError("H must be a contiguous [g, d_in, d_in] tensor")
    with _on(_same_device(("X", X), ("s", s), ("H", H), ("workspace", workspace)), stream) as st:
        rc = lib().gq_hessian_accumulate(X.data_ptr(), n, d_in, ld_x, s.data_ptr(), ld_s, g, H.data_ptr(), flags,
                                         workspace.data_ptr(), workspace.numel() * workspace.element_size(), st)
    if rc:
        raise GQError("gq_hessian_accumulate", rc)
    return H


def gq_hessian_accumulate_ahead(X: torch.Tensor, s: torch.Tensor, H: torch.Tensor, workspace: torch.Tensor,
                                next_grad: torch.Tensor, next_workspace: torch.Tensor, grad_scale: float = 1.0,
                                next_s: Optional[torch.Tensor] = None, flags: int = 0, stream=None) -> torch.Tensor:
    """:func:`gq_hessian_accumulate` for this chunk and, in the same launch, :func:`gq_saliency_prepared` for the
    next one (``next_grad`` -> ``next_s`` and ``next_workspace``).  Returns ``next_s``."""
    _dev(X, torch.bfloat16, "X")
    _dev(s, torch.float32, "s")
    _dev(H, torch.float32, "H")
    _dev(next_grad, torch.bfloat16, "next_grad")
    n, d_in, ld_x = _rows(X, "X")
    g, s_n, ld_s = _rows(s, "s")
    if s_n < n:
        raise ValueError("s must be [g, >= n]")
    if tuple(H.shape) != (g, d_in, d_in) or not H.is_contiguous():
        raise ValueError("H must be a contiguous [g, d_in, d_in] tensor")
    next_n, d_out, ld_grad = _rows(next_grad, "next_grad")
    if next_s is None:
        next_s = torch.empty((g, next_n), dtype=torch.float32, device=next_grad.device)
    _dev(next_s, torch.float32, "next_s")
    _, ns_n, next_ld_s = _rows(next_s, "next_s")
    if next_s.shape[0] != g or ns_n < next_n:
        raise ValueError("next_s must be [g, >= next_n]")
    with _on(_same_device(("X", X), ("s", s), ("H", H), ("workspace", workspace), ("next_grad", next_grad),
                          ("next_s", next_s), ("next_workspace", next_workspace)), stream) as st:
        rc = lib().gq_hessian_accumulate_ahead(
            X.data_ptr(), n, d_in, ld_x, s.data_ptr(), ld_s, g, H.data_ptr(), flags, workspace.data_ptr(),
            workspace.numel() * workspace.element_size(), next_grad.data_ptr(), next_n, d_out, ld_grad, float(grad_scale),
            next_s.data_ptr(), next_ld_s, next_workspace.data_ptr(),
            next_workspace.numel() * next_workspace.element_size(), st)
    if rc:
        raise GQError("gq_hessian_accumulate_ahead", rc)
    return next_s


def gq_hessian_finalize(H: torch.Tensor, stream=None) -> torch.Tensor:
    """Mirror the upper triangle of every ``H[k]`` onto the lower one."""
    _dev(H, torch.float32, "H")
    if H.dim() != 3 or H.shape[1] != H.shape[2] or not H.is_contiguous():
        raise ValueError("H must be a contiguous [g, d_in, d_in] tensor")
    with _on(_same_device(("H", H)), stream) as st:
        rc = lib().gq_hessian_finalize(H.data_ptr(), H.shape[1], H.shape[0], st)
    if rc:
        raise GQError("gq_hessian_finalize", rc)
    return H


def _rank_pointers(H_ranks, d_in: int, g: int):
    ptrs = []
    for h in H_ranks:
        if isinstance(h, torch.Tensor):
            _dev(h, torch.float32, "H_ranks[i]")
            if tuple(h.shape) != (g, d_in, d_in) or not h.is_contiguous():
                raise ValueError("every H must be a contiguous [g, d_in, d_in] tensor")
            ptrs.append(h.data_ptr())
        else:
            ptrs.append(int(h))           # a peer's device pointer as mapped into this process
    return (ctypes.c_void_p * len(ptrs))(*ptrs)


def _own_device(H_ranks, rank: int):
    """Device of the calling rank's own matrix (peers may be given as raw pointers)."""
    if 0 <= rank < len(H_ranks):
        own = H_ranks[rank]
        if not isinstance(own, torch.Tensor):
            raise ValueError("H_ranks[rank] must be this process's own tensor")
        return _same_device(("H_ranks[rank]", own))
    # a rank outside the list is the library's to reject; run the call on the device of any tensor given
    tensors = [("H_ranks[%d]" % i, h) for i, h in enumerate(H_ranks) if isinstance(h, torch.Tensor)]
    return _same_device(*tensors[:1])


def gq_hessian_reduce_share(H_ranks, rank: int, d_in: int, g: int, stream=None) -> None:
    """Token-sharded accumulation, step 1: add rank ``rank``'s blocks of the upper triangle over all ranks'
    matrices (tensors of this process, or peers' device pointers as integers) into ``H_ranks[rank]``."""
    arr = _rank_pointers(H_ranks, d_in, g)
    with _on(_own_device(H_ranks, rank), stream) as st:
        rc = lib().gq_hessian_reduce_share(arr, len(arr), rank, d_in, g, st)
    if rc:
        raise GQError("gq_hessian_reduce_share", rc)


def gq_hessian_gather_shares(H_ranks, rank: int, d_in: int, g: int, stream=None) -> None:
    """Token-sharded accumulation, step 2: copy the other ranks' reduced blocks into ``H_ranks[rank]``."""
    arr = _rank_pointers(H_ranks, d_in, g)
    with _on(_own_device(H_ranks, rank), stream) as st:
        rc = lib().gq_hessian_gather_shares(arr, len(arr), rank, d_in, g, st)
    if rc:
        raise GQError("gq_hessian_gather_shares", rc)


def gq_objective_workspace_bytes(d_in: int, d_out: int, g: int) -> int:
    return int(lib().gq_objective_workspace_bytes(d_in, d_out, g))


def gq_objective(W: torch.Tensor, W_hat: torch.Tensor, H: torch.Tensor, workspace: torch.Tensor,
                 loss: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Eq. 7: returns fp64 ``[g + 1]`` = per-group losses followed by their total (device tensor)."""
    _dev(W, torch.float32, "W")
    _dev(W_hat, torch.float32, "W_hat")
    _dev(H, torch.float32, "H")
    if W.dim() != 2 or W.shape != W_hat.shape or not W.is_contiguous() or not W_hat.is_contiguous():
        raise ValueError("W and W_hat must be contiguous [d_out, d_in]")
    d_out, d_in = W.shape
    g = H.shape[0]
    if tuple(H.shape) != (g, d_in, d_in) or not H.is_contiguous():
        raise ValueError("H must be a contiguous [g, d_in, d_in] tensor")
    if loss is None:
        loss = torch.empty(g + 1, dtype=torch.float64, device=W.device)
    _dev(loss, torch.float64, "loss")
    dev = _same_device(("W", W), ("W_hat", W_hat), ("H", H), ("loss", loss), ("workspace", workspace))
    with _on(dev, stream) as st:
        rc = lib().gq_objective(W.data_ptr(), W_hat.data_ptr(), d_in, d_out, H.data_ptr(), g, loss.data_ptr(),
                                workspace.data_ptr(), workspace.numel() * workspace.element_size(), st)
    if rc:
        raise GQError("gq_objective", rc)
    return loss


def gq_layer_host_arena_bytes(chunk: int, d_in: int, d_out: int, g: int) -> int:
    return int(lib().gq_layer_host_arena_bytes(chunk, d_in, d_out, g))


def gq_layer_objective_host(X_host: torch.Tensor, grad_host: torch.Tensor, chunk: int, g: int, grad_scale: float,
                            W_host: torch.Tensor, W_hat_host: torch.Tensor, arena: torch.Tensor,
                            loss_host: Optional[torch.Tensor] = None, H_host: Optional[torch.Tensor] = None,
                            stream=None) -> torch.Tensor:
    """Whole path from HOST tensors (ideally pinned): returns the host fp64 ``[g + 1]`` losses."""
    for t, dt, nm in ((X_host, torch.bfloat16, "X_host"), (grad_host, torch.bfloat16, "grad_host"),
                      (W_host, torch.float32, "W_host"), (W_hat_host, torch.float32, "W_hat_host")):
        if t.is_cuda or t.dtype != dt or not t.is_contiguous():
            raise ValueError("%s must be a contiguous host tensor of dtype %s" % (nm, dt))
    n, d_in = X_host.shape
    d_out = grad_host.shape[1]
    if grad_host.shape[0] != n or tuple(W_host.shape) != (d_out, d_in) or W_hat_host.shape != W_host.shape:
        raise ValueError("shape mismatch")
    if loss_host is None:
        loss_host = torch.empty(g + 1, dtype=torch.float64)
    if H_host is not None and (H_host.is_cuda or H_host.dtype != torch.float32 or not H_host.is_contiguous()
                               or tuple(H_host.shape) != (g, d_in, d_in)):
        raise ValueError("H_host must be a contiguous host fp32 [g, d_in, d_in] tensor")
    if not arena.is_cuda:
        raise ValueError("arena must be device memory")
    with _on(_same_device(("arena", arena)), stream) as st:
        rc = lib().gq_layer_objective_host(X_host.data_ptr(), grad_host.data_ptr(), n, chunk, d_in, d_out, g,
                                           float(grad_scale), W_host.data_ptr(), W_hat_host.data_ptr(),
                                           loss_host.data_ptr(), H_host.data_ptr() if H_host is not None else None,
                                           arena.data_ptr(), arena.numel() * arena.element_size(), st)
    if rc:
        raise GQError("gq_layer_objective_host", rc)
    return loss_host


def gq_check(stream=None, device=None):
    """Synchronises the stream and raises :class:`GQError` if a kernel recorded a device-side error on `device`
    (default: the stream's device, else the current one)."""
    detail = (ctypes.c_uint32 * 4)()
    if device is None:
        device = stream.device if stream is not None else torch.device("cuda", torch.cuda.current_device())
    with _on(torch.device(device), stream) as st:
        rc = lib().gq_check(st, detail)
    if rc:
        err = GQError("gq_check", rc)
        err.detail = tuple(int(v) for v in detail)
        raise err


def gq_kernel_timing_enable(enable: bool) -> None:
    rc = lib().gq_kernel_timing_enable(1 if enable else 0)
    if rc:
        raise GQError("gq_kernel_timing_enable", rc)


def gq_kernel_timing_read() -> dict:
    """``{kernel name: (summed device ms, launches)}`` for the launches recorded since the last read."""
    ms = (ctypes.c_double * len(KERNEL_NAMES))()
    cnt = (ctypes.c_uint64 * len(KERNEL_NAMES))()
    rc = lib().gq_kernel_timing_read(ms, cnt)
    if rc:
        raise GQError("gq_kernel_timing_read", rc)
    return {name: (float(ms[i]), int(cnt[i])) for i, name in enumerate(KERNEL_NAMES)}


def gq_objective_noalloc(W: torch.Tensor, W_hat: torch.Tensor, H: torch.Tensor, loss: torch.Tensor,
                         stream=None) -> torch.Tensor:
    """Eq. 7 for callers that must not allocate: scratch lives in a fixed array inside ``libgq.so``.

    Unlike :func:`gq_objective` this wrapper allocates nothing either, so ``loss`` (fp64 ``[g + 1]`` on the
    device) has to be passed in.  Only small layers fit (``d_in * d_out <= 2**20``); larger ones raise
    ``GQ_ERR_UNSUPPORTED_SHAPE``.  Calls that overlap on the GPU share the scratch and race."""
    _dev(W, torch.float32, "W")
    _dev(W_hat, torch.float32, "W_hat")
    _dev(H, torch.float32, "H")
    _dev(loss, torch.float64, "loss")
    if W.dim() != 2 or W.shape != W_hat.shape or not W.is_contiguous() or not W_hat.is_contiguous():
        raise ValueError("W and W_hat must be contiguous [d_out, d_in]")
    d_out, d_in = W.shape
    g = H.shape[0]
    if tuple(H.shape) != (g, d_in, d_in) or not H.is_contiguous() or loss.numel() != g + 1:
        raise ValueError("H must be contiguous [g, d_in, d_in] and loss must have g + 1 entries")
    with _on(_same_device(("W", W), ("W_hat", W_hat), ("H", H), ("loss", loss)), stream) as st:
        rc = lib().gq_objective_noalloc(W.data_ptr(), W_hat.data_ptr(), d_in, d_out, H.data_ptr(), g, loss.data_ptr(), st)
    if rc:
        raise GQError("gq_objective_noalloc", rc)
    return loss


def gq_cd_workspace_bytes(d_in: int, d_out: int, g: int) -> int:
    return int(lib().gq_cd_workspace_bytes(d_in, d_out, g))


def gq_cd_cycles(W: torch.Tensor, W_hat: torch.Tensor, codebook: torch.Tensor, H: torch.Tensor, cycles: int,
                 workspace: torch.Tensor, Q: Optional[torch.Tensor] = None, stream=None):
    """Cyclic coordinate descent with fixed codebooks (Eq. 10, Algorithm 4): updates ``W_hat`` in place and
    returns ``(W_hat, Q)`` with ``Q`` the uint8 codebook indices."""
    _dev(W, torch.float32, "W")
    _dev(W_hat, torch.float32, "W_hat")
    _dev(codebook, torch.float32, "codebook")
    _dev(H, torch.float32, "H")
    if W.dim() != 2 or W.shape != W_hat.shape or not W.is_contiguous() or not W_hat.is_contiguous():
        raise ValueError("W and W_hat must be contiguous [d_out, d_in]")
    d_out, d_in = W.shape
    g = H.shape[0]
    if tuple(H.shape) != (g, d_in, d_in) or not H.is_contiguous():
        raise ValueError("H must be a contiguous [g, d_in, d_in] tensor")
    if codebook.dim() != 2 or codebook.shape[0] != d_out or not codebook.is_contiguous():
        raise ValueError("codebook must be a contiguous [d_out, m] tensor")
    if Q is None:
        Q = torch.empty((d_out, d_in), dtype=torch.uint8, device=W.device)
    _dev(Q, torch.uint8, "Q")
    dev = _same_device(("W", W), ("W_hat", W_hat), ("Q", Q), ("codebook", codebook), ("H", H), ("workspace", workspace))
    with _on(dev, stream) as st:
        rc = lib().gq_cd_cycles(W.data_ptr(), W_hat.data_ptr(), Q.data_ptr(), codebook.data_ptr(), codebook.shape[1],
                                d_in, d_out, H.data_ptr(), g, int(cycles), workspace.data_ptr(),
                                workspace.numel() * workspace.element_size(), st)
    if rc:
        raise GQError("gq_cd_cycles", rc)
    return W_hat, Q


def gq_selftest_wait_timeout(budget_ms: int = 20, stream=None) -> None:
    """Launches the kernel whose wait runs out after ``budget_ms``; the next :func:`gq_check` raises
    ``GQ_ERR_TIMEOUT`` (site 99)."""
    device = stream.device if stream is not None else torch.device("cuda", torch.cuda.current_device())
    with _on(device, stream) as st:
        rc = lib().gq_selftest_wait_timeout(int(budget_ms), st)
    if rc:
        raise GQError("gq_selftest_wait_timeout", rc)


def gq_codebook_workspace_bytes(d_in: int, d_out: int, g: int, m: int) -> int:
    return int(lib().gq_codebook_workspace_bytes(d_in, d_out, g, m))


def gq_lnq_workspace_bytes(d_in: int, d_out: int, g: int, m: int) -> int:
    return int(lib().gq_lnq_workspace_bytes(d_in, d_out, g, m))


def gq_lnq(W: torch.Tensor, Q: torch.Tensor, m: int, H: torch.Tensor, T: int, K: int, workspace: torch.Tensor,
           lam: float = 1e-7, stream=None):
    """Algorithm 2 in one call: ``T`` rounds of (codebook step, ``K`` CD cycles) and a final codebook step,
    starting from the assignment ``Q`` (uint8, updated in place).  Returns ``(W_hat, Q, codebook)``."""
    _dev(W, torch.float32, "W")
    _dev(Q, torch.uint8, "Q")
    _dev(H, torch.float32, "H")
    if W.dim() != 2 or W.shape != Q.shape or not W.is_contiguous() or not Q.is_contiguous():
        raise ValueError("W and Q must be contiguous [d_out, d_in]")
    d_out, d_in = W.shape
    g = H.shape[0]
    if tuple(H.shape) != (g, d_in, d_in) or not H.is_contiguous():
        raise ValueError("H must be a contiguous [g, d_in, d_in] tensor")
    codebook = torch.empty((d_out, max(int(m), 1)), dtype=torch.float32, device=W.device)
    W_hat = torch.empty_like(W)
    with _on(_same_device(("W", W), ("Q", Q), ("H", H), ("workspace", workspace)), stream) as st:
        rc = lib().gq_lnq(W.data_ptr(), Q.data_ptr(), int(m), d_in, d_out, H.data_ptr(), g, int(T), int(K), float(lam),
                          codebook.data_ptr(), W_hat.data_ptr(), workspace.data_ptr(),
                          workspace.numel() * workspace.element_size(), st)
    if rc:
        raise GQError("gq_lnq", rc)
    return W_hat, Q, codebook


def gq_codebook_update(W: torch.Tensor, Q: torch.Tensor, m: int, H: torch.Tensor, workspace: torch.Tensor,
                       lam: float = 1e-7, codebook: Optional[torch.Tensor] = None,
                       W_hat: Optional[torch.Tensor] = None, stream=None):
    """Eq. 8 for every channel: the optimal codebook for fixed codes ``Q``.  Returns ``(codebook, W_hat)``;
    ``W_hat`` (if a tensor is passed) receives ``codebook[j, Q[j, i]]``."""
    _dev(W, torch.float32, "W")
    _dev(Q, torch.uint8, "Q")
    _dev(H, torch.float32, "H")
    if W.dim() != 2 or W.shape != Q.shape or not W.is_contiguous() or not Q.is_contiguous():
        raise ValueError("W and Q must be contiguous [d_out, d_in]")
    d_out, d_in = W.shape
    g = H.shape[0]
    if tuple(H.shape) != (g, d_in, d_in) or not H.is_contiguous():
        raise ValueError("H must be a contiguous [g, d_in, d_in] tensor")
    if codebook is None:
        codebook = torch.empty((d_out, m), dtype=torch.float32, device=W.device)
    _dev(codebook, torch.float32, "codebook")
    if W_hat is not None:
        _dev(W_hat, torch.float32, "W_hat")
        if W_hat.shape != W.shape or not W_hat.is_contiguous():
            raise ValueError("W_hat must be contiguous [d_out, d_in]")
    dev = _same_device(("W", W), ("Q", Q), ("H", H), ("codebook", codebook), ("W_hat", W_hat), ("workspace", workspace))
    with _on(dev, stream) as st:
        rc = lib().gq_codebook_update(W.data_ptr(), Q.data_ptr(), int(m), d_in, d_out, H.data_ptr(), g, float(lam),
                                      codebook.data_ptr(), W_hat.data_ptr() if W_hat is not None else None,
                                      workspace.data_ptr(), workspace.numel() * workspace.element_size(), st)
    if rc:
        raise GQError("gq_codebook_update", rc)
    return codebook, W_hat
