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
    assert L.gq_hessian_workspace_bytes(8192, 4096, 4, 2) == 0                 # unknown flag
    assert L.gq_hessian_workspace_bytes(8192, 4100, 4, 0) == 0                 # d_in % 8 != 0
    # objective: two bf16 copies of delta + room for 16 fp64 partial sums per (upper-triangular 256 x 256 tile, group)
    nj = 4096 // 256
    assert L.gq_objective_workspace_bytes(4096, 4096, 4) == 2 * 4096 * 4096 * 2 + (nj * (nj + 1) // 2) * 4 * 16 * 8
    assert L.gq_objective_workspace_bytes(4096, 4096, 3) == 0          # d_out % g != 0
    assert L.gq_objective_workspace_bytes(4096, 24, 6) == 0            # (d_out / g) % 8 != 0
    assert L.gq_layer_host_arena_bytes(0, 4096, 4096, 4) == 0
    assert L.gq_layer_host_arena_bytes(8192, 4096, 4096, 4) > 4 * 4096 * 4096 * 4


def test_host_side_validation_needs_no_gpu(L):
    buf = (ctypes.c_uint8 * 4096)()
    p = ctypes.addressof(buf)
    p16 = (p + 15) // 16 * 16
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
    # hessian
    assert L.gq_hessian_accumulate(p16, 4, 64, 64, p16, 4, 2, p16, 2, p16, 4096, None) == INVALID   # flags
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


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(libgq, "_lib", None)
    monkeypatch.setattr(libgq, "LIB_PATH", str(tmp_path / "libgq.so"))
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        libgq.lib()
