"""Host-side checks that need no GPU: the library builds for sm_100a, exports every symbol the header
declares, sizes workspaces sanely and rejects bad problems."""
import ctypes
import os
import re

import pytest

import paper_2501_05633_b200 as pkg
from paper_2501_05633_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    pkg.build()
    return pkg.load_library()


def test_header_symbols_exported(lib):
    header = open(os.path.join(ROOT, "include", "regtopk.h")).read()
    declared = set(re.findall(r"\b(regtopk_[a-z_]+)\s*\(", header))
    assert declared, "no declarations found"
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), f"{name} is declared but not exported"


def test_strerror(lib):
    assert lib.regtopk_strerror(0) == b"ok"
    for code in range(-7, 0):
        assert lib.regtopk_strerror(code) not in (b"ok", b"unknown error code")
    assert lib.regtopk_strerror(-99) == b"unknown error code"


def test_workspace_bytes():
    d, N, k = 11_173_962, 8, 11_174
    b = binding.workspace_bytes(d, N, k)
    assert b >= N * d * 4  # the residuals alone
    assert b < 2 * N * d * 4  # no second dense buffer per worker
    assert binding.workspace_bytes(d, N, k, flags=binding.FLAG_HOST_STAGING) >= b + N * d * 4
    assert binding.workspace_bytes(d, N, k, grad_dtype=binding.GRAD_BF16) == b
    # the 1.3e9-coordinate problem fits one 180 GB device with its gradients beside it
    big = binding.workspace_bytes(1_300_000_000, 4, 13_000_000)
    assert 4 * 1_300_000_000 * 4 < big < 40e9


@pytest.mark.parametrize("d,N,k,mu", [(0, 1, 1, 4.0), (10, 0, 1, 4.0), (10, 1, 0, 4.0), (10, 1, 11, 4.0),
                                      (2**31 - 1, 1, 1, 4.0), (10, 1, 1, -1.0), (10, 1, 1, float("nan")),
                                      (10, 70000, 1, 4.0)])
def test_invalid_problems_rejected(d, N, k, mu):
    assert binding.workspace_bytes(d, N, k, mu=mu) == 0


def test_invalid_omega_and_dtype_rejected():
    assert binding.workspace_bytes(10, 2, 1, omega=[0.5, float("inf")]) == 0
    assert binding.workspace_bytes(10, 2, 1, grad_dtype=7) == 0
    assert binding.workspace_bytes(10, 2, 1, omega=[0.5, 0.5]) > 0
    assert binding.workspace_bytes(10, 2, 1, y=0.5) > 0 and binding.workspace_bytes(10, 2, 1, y=0.0) > 0
    assert binding.workspace_bytes(10, 2, 1, y=1.5) == 0 and binding.workspace_bytes(10, 2, 1, y=-0.5) == 0


def test_null_context_calls(lib):
    assert lib.regtopk_worker_step(None, None, 0, None, None) == -1
    assert lib.regtopk_aggregate(None, None) == -1
    assert lib.regtopk_state_reset(None) == -1
    assert lib.regtopk_status(None) == -1
    assert lib.regtopk_destroy(None) == -1
    out = ctypes.c_void_p()
    p, _ = binding._make_params(4.0, None, 0, 0)
    assert lib.regtopk_create(ctypes.byref(out), 10, 1, 1, ctypes.byref(p), None, 0, None) == -1


def test_no_cpu_fallback():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    with pytest.raises(RuntimeError):
        pkg.RegTopK(100, 2, 3)


def test_product_does_not_import_oracle():
    for fn in ("binding.py", "synth.py", "__init__.py"):
        src = open(os.path.join(ROOT, "paper_2501_05633_b200", fn)).read()
        assert "oracle" not in src.replace("the CPU oracle", "").replace("CPU oracle", ""), fn
    cu = open(os.path.join(ROOT, "paper_2501_05633_b200", "csrc", "regtopk.cu")).read()
    assert "oracle" not in cu
