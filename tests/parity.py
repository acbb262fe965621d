"""Round-by-round comparison of the CUDA library (through its C ABI) with the CPU oracle on the same
seeded inputs.  Index sets, sent values, residuals and the aggregate must agree bit for bit."""
import numpy as np
import torch

from oracle.oracle import OracleRegTopK, grads_view
from paper_2501_05633_b200 import RegTopK


to_oracle_view = grads_view


def bits(x):
    return np.ascontiguousarray(x).view(np.uint32)


def run_parity(rounds, d, N, k, mu, omega=None, flags=0, check_eps=True, select_mode=0, threads=4,
               reset_after=None, expect_dense=None, y=1.0, inplace=None, layers=None):
    """rounds: iterable of torch tensors [N, ld] (CPU or CUDA, float32 or bfloat16).
    inplace: None, or a function of the round number saying whether that round uses the accumulate-in-place calls.
    layers: None, or (layer_end, layer_k) for one selection per layer (k is then ignored).
    Returns the library's stats after the last round."""
    rounds = iter(rounds)
    first = next(rounds)
    lib = RegTopK(d, N, k, mu=mu, omega=omega, grad_dtype=first.dtype, flags=flags, y=y, layers=layers)
    ora = OracleRegTopK(d, N, k, mu, omega=omega, select_mode=select_mode, threads=threads, y=y, layers=layers)
    t = 0
    g = first
    while g is not None:
        g_dev = g if g.is_cuda else g.cuda()
        g_cpu = g.cpu() if g.is_cuda else g
        if inplace is not None and inplace(t):
            # accumulate-in-place form: the caller adds the gradients into the library's rows itself
            lib.accumulator().add_(g_dev[:, :d].float())
            idx, val = lib.worker_step_inplace()
        else:
            idx, val = lib.worker_step(g_dev)
        o_idx, o_val = ora.worker_step(to_oracle_view(g_cpu, d))
        lib.status()
        idx_h, val_h = idx.cpu().numpy(), val.cpu().numpy()
        assert np.array_equal(idx_h, o_idx), f"round {t}: index sets differ"
        assert np.array_equal(bits(val_h), bits(o_val)), f"round {t}: sent values differ"
        if check_eps:
            eps = lib.residual().cpu().numpy()
            assert np.array_equal(bits(eps), bits(ora.eps)), f"round {t}: residuals differ"
        agg = lib.aggregate().cpu().numpy()
        o_agg = ora.aggregate()
        lib.status()
        assert np.array_equal(bits(agg), bits(o_agg)), f"round {t}: aggregates differ"
        t += 1
        if reset_after is not None and t == reset_after:
            lib.state_reset()
            ora.reset()
        g = next(rounds, None)
    st = lib.stats()
    if expect_dense is True:
        assert st["dense_select_workers"] > 0, st
    if expect_dense is False:
        assert st["dense_select_workers"] == 0, st
    lib.close()
    return st
