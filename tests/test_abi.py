"""The C-ABI library loads without a GPU, exports every symbol include/gq.h declares, and its
host-side logic (sizes, validation, status strings) behaves as documented.  No kernel is launched."""
import ctypes
import os
import re

import pytest

from paper_2505_07004_b200 import api as libgq
from paper_2505_07004_b200 import build as gq_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    gq_build.build_libgq()
    return libgq.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "gq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gq_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(L):
    names = declared_functions()
    assert len(names) >= 13
    for name in names:
        assert hasattr(L, name), "libgq.so does not export %s" % name
    assert set(names) == set(libgq.EXPORTS), "binding and header disagree: %s" % (set(names) ^ set(libgq.EXPORTS))


def test_version_and_status_strings(L):
    assert L.gq_version() >= 100
    assert L.gq_status_string(0) == b"GQ_OK"
    for code, name in [(-1, b"GQ_ERR_INVALID_ARG"), (-2, b"GQ_ERR_ALIGNMENT"), (-3, b"GQ_ERR_UNSUPPORTED_SHAPE"),
                       (-4, b"GQ_ERR_WORKSPACE"), (-5, b"GQ_ERR_CUDA"), (-6, b"GQ_ERR_TIMEOUT")]:
        assert L.gq_status_string(code) == name
    assert L.gq_status_string(-99) == b"GQ_ERR_UNKNOWN"


def test_workspace_sizes(L):
    # split saliency words: 8 bytes per (pair of groups, token); no scaled copy of X
    assert L.gq_hessian_workspace_bytes(8192, 4096, 4, 0) == 2 * 8192 * 8
    assert L.gq_hessian_workspace_bytes(8192, 4096, 5, 1) == 3 * 8192 * 8      # GQ_HESSIAN_DETERMINISTIC, odd g
    assert L.gq_hessian_workspace_bytes(1, 8, 1, 0) == 1024                    # rounded up to 1 KiB
    assert L.gq_hessian_workspace_bytes(8192, 4096, 4, 4) == 0                 # unknown flag
    assert L.gq_hessian_workspace_bytes(8192, 4096, 4, 3) == 2 * 8192 * 8      # both known flags
    assert L.gq_hessian_workspace_bytes(8192, 4100, 4, 0) == 0                 # d_in % 8 != 0
    # objective: a 1 KiB header, delta as one fp16 matrix, 16 fp64 partial sums per (upper-triangular 256 x 256 tile, group)
    nj = 4096 // 256
    assert L.gq_objective_workspace_bytes(4096, 4096, 4) == 1024 + 4096 * 4096 * 2 + (nj * (nj + 1) // 2) * 4 * 16 * 8
    assert L.gq_objective_workspace_bytes(4096, 4096, 3) == 0          # d_out % g != 0
    assert L.gq_objective_workspace_bytes(4096, 24, 6) == 0            # (d_out / g) % 8 != 0
    assert L.gq_layer_host_arena_bytes(0, 4096, 4096, 4) == 0
    assert L.gq_layer_host_arena_bytes(8192, 4096, 4096, 4) > 4 * 4096 * 4096 * 4
    # the loss slot holds g + 1 fp64 values rounded up to 1 KiB: 1 KiB for g = 64, 2 KiB for g = 128
    r1k = lambda b: (b + 1023) // 1024 * 1024

    def loss_slot(g, chunk=64, d_in=64, d_out=1024):
        rest = (2 * r1k(chunk * d_in * 2) + 2 * r1k(chunk * d_out * 2) + r1k(g * chunk * 4) + r1k(g * d_in * d_in * 4)
                + 2 * r1k(d_out * d_in * 4) + L.gq_hessian_workspace_bytes(chunk, d_in, g, 0)
                + L.gq_objective_workspace_bytes(d_in, d_out, g))
        return L.gq_layer_host_arena_bytes(chunk, d_in, d_out, g) - rest
    assert loss_slot(64) == 1024 and loss_slot(128) == 2048


def test_host_side_validation_needs_no_gpu(L):
    buf = (ctypes.c_uint8 * 8192)()
    p = ctypes.addressof(buf)
    p16 = (p + 127) // 128 * 128           # 128-byte aligned: what H needs; the other pointers need 16
    INVALID, ALIGN, SHAPE, WS = -1, -2, -3, -4
    # saliency
    assert L.gq_saliency(p16, -1, 64, 64, 2, 1.0, p16, 0, None) == INVALID
    assert L.gq_saliency(p16, 4, 64, 64, 3, 1.0, p16, 4, None) == INVALID      # 64 % 3
    assert L.gq_saliency(p16, 4, 64, 32, 2, 1.0, p16, 4, None) == INVALID      # ld_grad < d_out
    assert L.gq_saliency(p16, 4, 64, 64, 2, 1.0, p16, 3, None) == INVALID      # ld_s < n
    assert L.gq_saliency(p16, 4, 24, 24, 6, 1.0, p16, 4, None) == SHAPE        # m = 4
    assert L.gq_saliency(p16, 4, 64, 68, 2, 1.0, p16, 4, None) == ALIGN        # ld_grad % 8
    assert L.gq_saliency(p16 + 2, 4, 64, 64, 2, 1.0, p16, 4, None) == ALIGN
    assert L.gq_saliency(None, 4, 64, 64, 2, 1.0, p16, 4, None) == INVALID
    assert L.gq_saliency(None, 0, 64, 64, 2, 1.0, None, 0, None) == 0          # empty call: no-op
    # saliency from a [batch, seq, d_out] gradient in another dtype
    assert L.gq_saliency_strided(p16, 3, 2, 4, 64, 256, 64, 2, 1.0, p16 + 4096, 8, None) == INVALID   # unknown dtype
    assert L.gq_saliency_strided(p16, 1, 2, 4, 64, 256, 32, 2, 1.0, p16 + 4096, 8, None) == INVALID   # stride_t < d_out
    assert L.gq_saliency_strided(p16, 1, 2, 4, 64, 128, 64, 2, 1.0, p16 + 4096, 8, None) == INVALID   # sequences overlap
    assert L.gq_saliency_strided(p16, 2, 2, 4, 64, 264, 66, 2, 1.0, p16 + 4096, 8, None) == ALIGN     # 66 floats: not 16 bytes
    assert L.gq_saliency_strided(p16, 1, 2, 4, 64, 256, 64, 2, 1.0, p16 + 4096, 7, None) == INVALID   # ld_s < batch * seq
    assert L.gq_saliency_strided(None, 1, 0, 4, 64, 256, 64, 2, 1.0, None, 0, None) == 0              # empty call
    # hessian
    assert L.gq_hessian_accumulate(p16, 4, 64, 64, p16, 4, 2, p16, 4, p16, 4096, None) == INVALID   # flags
    assert L.gq_hessian_accumulate(p16, 4, 60, 64, p16, 4, 2, p16, 0, p16, 4096, None) == SHAPE     # d_in % 8
    assert L.gq_hessian_accumulate(p16, 4, 64, 64, p16, 4, 2, p16 + 4, 0, p16, 4096, None) == ALIGN
    assert L.gq_hessian_accumulate(p16, 4, 64, 64, p16, 4, 2, p16, 0, None, 0, None) == WS
    assert L.gq_hessian_accumulate(None, 0, 64, 64, None, 0, 2, None, 0, None, 0, None) == 0        # empty chunk
    assert L.gq_hessian_finalize(None, 64, 2, None) == INVALID
    # objective
    assert L.gq_objective(p16, p16, 64, 64, p16, 3, p16, p16, 4096, None) == INVALID                # 64 % 3
    assert L.gq_objective(p16, p16, 64, 64, p16, 2, p16, p16, 16, None) == WS
    assert L.gq_objective(None, p16, 64, 64, p16, 2, p16, p16, 1 << 20, None) == INVALID
    assert L.gq_kernel_timing_read(None, None) == INVALID


def test_aliasing_between_outputs_and_inputs_is_rejected(L):
    """A buffer a call writes may not overlap one it reads (or another one it writes): GQ_ERR_INVALID_ARG on the
    host, before any launch.  Two read-only arguments may alias."""
    buf = (ctypes.c_uint8 * (1 << 20))()
    base = (ctypes.addressof(buf) + 1023) // 1024 * 1024
    INVALID, WS = -1, -4
    # saliency: grad [4, 64] bf16 = 512 bytes, s [2, 4] fp32 = 32 bytes
    assert L.gq_saliency(base, 4, 64, 64, 2, 1.0, base + 496, 4, None) == INVALID       # s inside grad's last row
    assert L.gq_saliency(base + 16, 4, 64, 64, 2, 1.0, base, 4, None) == INVALID        # grad starts inside s
    # hessian: X [4, 64] = 512 B, s [2, 4] = 32 B, H [2, 64, 64] = 32 KiB, workspace 1 KiB
    X, s_, H, ws = base, base + 1024, base + 2048, base + 65536
    assert L.gq_hessian_accumulate(X, 4, 64, 64, s_, 4, 2, X, 0, ws, 1024, None) == INVALID          # H over X
    assert L.gq_hessian_accumulate(X, 4, 64, 64, H + 64, 4, 2, H, 0, ws, 1024, None) == INVALID      # s inside H
    assert L.gq_hessian_accumulate(X, 4, 64, 64, s_, 4, 2, H, 0, H + 1024, 1024, None) == INVALID    # workspace inside H
    assert L.gq_hessian_accumulate(X, 4, 64, 64, s_, 4, 2, H, 0, X, 1024, None) == INVALID           # workspace over X
    # hessian with the next chunk's saliency: next grad [4, 64] = 512 B, next s 32 B, second workspace 1 KiB
    ng, ns, nws = base + 131072, base + 132096, base + 133120
    ahead = lambda ng_, ns_, nws_, nws_bytes=1024: L.gq_hessian_accumulate_ahead(
        X, 4, 64, 64, s_, 4, 2, H, 0, ws, 1024, ng_, 4, 64, 64, 1.0, ns_, 4, nws_, nws_bytes, None)
    assert ahead(ng, ns, ws) == INVALID                       # the second scratch block is the first one
    assert ahead(ng, s_, nws) == INVALID                      # next s over the s being read
    assert ahead(ng, H + 128, nws) == INVALID                 # next s inside H
    assert ahead(ng, ns, X) == INVALID                        # second scratch block over X
    assert ahead(H, ns, nws) == INVALID                       # next grad inside H (written by the same launch)
    assert ahead(ng, ng + 16, nws) == INVALID                 # next s inside next grad
    assert ahead(ng, ns, nws, 16) == WS
    # the next chunk's arguments are checked like gq_saliency_prepared's: (token, group) count below 2^31, d_out % g,
    # 16-byte rows
    big = L.gq_hessian_accumulate_ahead(X, 4, 64, 64, s_, 4, 2, H, 0, ws, 1024, ng, 1 << 30, 64, 64, 1.0, ns, 1 << 30,
                                        nws, 1 << 34, None)
    assert big == -3
    assert L.gq_hessian_accumulate_ahead(X, 4, 64, 64, s_, 4, 2, H, 0, ws, 1024, ng, 4, 63, 64, 1.0, ns, 4, nws, 1024,
                                         None) == INVALID
    assert L.gq_hessian_accumulate_ahead(X, 4, 64, 64, s_, 4, 2, H, 0, ws, 1024, ng, 4, 64, 68, 1.0, ns, 4, nws, 1024,
                                         None) == -2
    # s and next_s as column ranges of one [2, 16] buffer (leading dimension 16): disjoint columns are fine
    # although their spans interleave, shared columns are not
    in_one = lambda col: L.gq_hessian_accumulate_ahead(X, 4, 64, 64, s_, 16, 2, H, 0, ws, 1024, ng, 4, 64, 64, 1.0,
                                                       s_ + 4 * col, 16, nws, 1024, None)
    assert in_one(4) not in (INVALID, WS, -2, -3) and in_one(12) not in (INVALID, WS, -2, -3)
    assert in_one(3) == INVALID and in_one(0) == INVALID and in_one(13) == INVALID      # 13..16 wraps into the next row
    assert ahead(ng, ns, nws) not in (INVALID, WS, -2, -3)    # a valid call gets as far as the device (none here)
    # objective: W, W_hat [64, 64] fp32 = 16 KiB each, H [2, 64, 64] = 32 KiB, loss 24 B
    need = L.gq_objective_workspace_bytes(64, 64, 2)
    W, Wh, Hh, loss, ows = base, base + 16384, base + 32768, base + 65536, base + 131072
    assert need > 0 and need < (1 << 20) - 131072 - 1024
    assert L.gq_objective(W, Wh, 64, 64, Hh, 2, W + 8, ows, need, None) == INVALID                   # loss inside W
    assert L.gq_objective(W, Wh, 64, 64, Hh, 2, loss, Hh, need, None) == INVALID                     # workspace over H
    assert L.gq_objective(W, Wh, 64, 64, Hh, 2, ows + 16, ows, need, None) == INVALID                # loss inside workspace
    assert L.gq_objective(W, Wh, 64, 64, Hh, 2, loss, ows, need - 1, None) == WS                     # size check first
    assert L.gq_objective_noalloc(W, Wh, 64, 64, Hh, 2, Hh + 8, None) == INVALID                     # loss inside H


def test_binding_refuses_tensors_on_different_devices():
    """The library launches on the current device; the binding makes the tensors' device current and refuses
    arguments that live on different GPUs before anything is launched."""
    import types
    import torch
    t0 = types.SimpleNamespace(device=torch.device("cuda", 0))
    t1 = types.SimpleNamespace(device=torch.device("cuda", 1))
    host = types.SimpleNamespace(device=torch.device("cpu"))
    assert libgq._same_device(("X", t0), ("H", t0), ("W_hat", None)) == torch.device("cuda", 0)
    with pytest.raises(ValueError, match="one device"):
        libgq._same_device(("X", t0), ("H", t1))
    with pytest.raises(ValueError, match="CUDA tensor"):
        libgq._same_device(("X", host))
    with pytest.raises(ValueError):
        libgq._same_device(("W_hat", None))
    stream1 = types.SimpleNamespace(device=torch.device("cuda", 1), cuda_stream=0)
    with pytest.raises(ValueError, match="stream belongs"):
        libgq._on(torch.device("cuda", 0), stream1)


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(libgq, "_lib", None)
    monkeypatch.setattr(libgq, "LIB_PATH", str(tmp_path / "libgq.so"))
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        libgq.lib()
