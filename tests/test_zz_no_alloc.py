"""regtopk_aggregate_pairs_static: the aggregation for callers that cannot allocate device memory
(allocator callbacks, processes that gave the whole GPU to a framework's pool, no-cudaMalloc-after-
start-up policies).  It keeps its scratch in an array built into the library, so this test checks that
it gives exactly the aggregate the CPU oracle computes from the same pairs and a context computes on the device
(bit for bit: same operations in the same order), twice in a row with different pairs, because the second call
meets the first call's bits in the scratch; that device memory does not move across a call; and that pairs with
indices outside [0, d) are ignored instead of being trusted.
Collected last on purpose: a run that stops at the first failure has already run everything else."""
import ctypes

import numpy as np
import pytest
import torch

import paper_2501_05633_b200 as pkg
from paper_2501_05633_b200 import binding

pytestmark = pytest.mark.gpu


def _free_bytes():
    """Free device memory as the driver reports it (cudaMemGetInfo): moves whenever anybody calls cudaMalloc/cudaFree."""
    torch.cuda.synchronize()
    return torch.cuda.mem_get_info()[0]


def test_static_aggregate_matches_oracle_and_context_twice():
    from oracle.oracle import default as oracle_default
    d, N, k = 200_003, 5, 1500
    omega = [0.3, 0.1, 0.25, 0.15, 0.2]
    lib = pkg.RegTopK(d, N, k, mu=4.0, omega=omega)
    gen = torch.Generator().manual_seed(123)
    out = torch.empty(d, dtype=torch.float32, device="cuda")  # made before the calls under test
    for call in range(2):
        g = torch.randn(N, d, generator=gen).cuda()
        idx, val = lib.worker_step(g)
        ctx_g = lib.aggregate().clone()
        want = oracle_default().aggregate(d, np.asarray(omega, np.float32), idx.cpu().numpy(), val.cpu().numpy())
        out.fill_(float("nan"))  # the entry point must overwrite every element
        free0 = _free_bytes()
        got = pkg.aggregate_pairs_static(idx, val, d, omega=omega, out=out)
        assert got is out
        assert _free_bytes() == free0, "device memory was allocated or freed around the call"
        assert np.array_equal(got.cpu().numpy().view(np.uint32), want.view(np.uint32)), f"call {call}: oracle"
        assert np.array_equal(got.cpu().numpy().view(np.uint32), ctx_g.cpu().numpy().view(np.uint32)), f"call {call}: context"
    lib.status()


def test_static_aggregate_ignores_out_of_range_pairs():
    """Indices d, -1 and 2^31 - 1 in the caller's arrays: those pairs are skipped, the rest of the call is the
    oracle's aggregate of the remaining pairs, and nothing outside out_g is written (guard elements stay put)."""
    from oracle.oracle import default as oracle_default
    d, N, k = 5000, 3, 40
    gen = torch.Generator().manual_seed(7)
    idx = torch.stack([torch.sort(torch.randperm(d, generator=gen)[:k]).values for _ in range(N)]).to(torch.int32)
    val = torch.randn(N, k, generator=gen)
    bad = idx.clone()
    bad[0, k - 1] = d
    bad[1, 0] = -1
    bad[2, k - 1] = 2**31 - 1
    # the oracle's answer: a skipped pair contributes nothing, which is what a pair (unused index, +0 value) contributes
    # (0 + omega * 0 = +0, the value an untouched entry has anyway)
    used = set(int(i) for i in idx.reshape(-1))
    spare = [j for j in range(d) if j not in used][:3]
    o_idx, o_val = idx.clone(), val.clone()
    for (n, r), j in zip(((0, k - 1), (1, 0), (2, k - 1)), spare):
        o_idx[n, r] = j
        o_val[n, r] = 0.0
    want = oracle_default().aggregate(d, np.full(N, np.float32(1.0) / np.float32(N), np.float32), o_idx.numpy(), o_val.numpy())
    buf = torch.full((d + 64,), 7.0, device="cuda")
    out = buf[32: 32 + d]
    got = pkg.aggregate_pairs_static(bad.cuda(), val.cuda(), d, out=out)
    torch.cuda.synchronize()
    assert np.array_equal(got.cpu().numpy().view(np.uint32), want.view(np.uint32))
    assert torch.all(buf[:32] == 7.0) and torch.all(buf[32 + d:] == 7.0)


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
