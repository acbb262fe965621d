"""regtopk_aggregate_pairs_static: the aggregation for callers that cannot allocate device memory
(allocator callbacks, processes that gave the whole GPU to a framework's pool, no-cudaMalloc-after-
start-up policies).  It keeps its scratch in an array built into the library, so this test checks that
it gives exactly the aggregate a context computes (bit for bit: same operations in the same order),
twice in a row with different pairs, because the second call meets the first call's bits in the scratch.
Collected last on purpose: a run that stops at the first failure has already run everything else."""
import ctypes

import numpy as np
import pytest
import torch

import paper_2501_05633_b200 as pkg
from paper_2501_05633_b200 import binding

pytestmark = pytest.mark.gpu


def test_static_aggregate_matches_context_twice():
    d, N, k = 200_003, 5, 1500
    omega = [0.3, 0.1, 0.25, 0.15, 0.2]
    lib = pkg.RegTopK(d, N, k, mu=4.0, omega=omega)
    gen = torch.Generator().manual_seed(123)
    out = torch.empty(d, dtype=torch.float32, device="cuda")  # made before the calls under test
    for call in range(2):
        g = torch.randn(N, d, generator=gen).cuda()
        idx, val = lib.worker_step(g)
        want = lib.aggregate().clone()
        out.fill_(float("nan"))  # the entry point must overwrite every element
        got = pkg.aggregate_pairs_static(idx, val, d, omega=omega, out=out)
        assert got is out
        torch.cuda.synchronize()
        assert np.array_equal(got.cpu().numpy().view(np.uint32), want.cpu().numpy().view(np.uint32)), f"call {call}"
    lib.status()


def test_static_aggregate_default_weights_and_limits():
    L = binding.load_library()
    d, N, k = 4096, 8, 41
    lib = pkg.RegTopK(d, N, k)
    idx, val = lib.worker_step(torch.randn(N, d, device="cuda"))
    want = lib.aggregate().clone()
    got = pkg.aggregate_pairs_static(idx, val, d)
    assert torch.equal(got, want)
    out = torch.empty(8, device="cuda")
    big_d = 32 * binding.STATIC_SCRATCH_WORDS  # one worker would already need every scratch word ...
    rc = L.regtopk_aggregate_pairs_static(big_d, 2, 1, idx.data_ptr(), val.data_ptr(), None, out.data_ptr(), None)
    assert rc == -7  # ... so two do not fit: refused with TOO_LARGE, nothing launched
    assert L.regtopk_aggregate_pairs_static(d, binding.STATIC_MAX_WORKERS + 1, k, idx.data_ptr(), val.data_ptr(),
                                            None, out.data_ptr(), None) == -7
    assert L.regtopk_aggregate_pairs_static(d, N, k, None, val.data_ptr(), None, out.data_ptr(), None) == -1
    assert b"static" in L.regtopk_strerror(-7)
