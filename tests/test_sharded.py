"""Workers spread over several ranks (paper_2501_05633_b200/sharded.py).

CPU part (gloo, world size 2, no GPU): the host-side logic of the exchange.  Every rank runs the ORACLE for its
block of the workers, the pairs are all-gathered with the module's own gather_pairs, the server sum runs over the
assembled pairs, and the result must equal the oracle's unsharded run of all workers bit for bit, over several
rounds (so that the aggregate that comes back feeds the next round's distortion).

GPU part (one GPU): two library contexts stand in for two ranks one after the other in one process (no kernel of
one waits for the other), their pairs are concatenated as the all-gather would, and regtopk_aggregate_gathered on
both must reproduce the oracle's unsharded run.
"""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _grads(n_total, d, rounds, seed):
    g = torch.Generator().manual_seed(seed)
    base = torch.randn(d, generator=g)
    return [(0.7 * base + torch.randn(n_total, d, generator=g)).numpy().astype(np.float32) for _ in range(rounds)]


def _bits(x):
    return np.ascontiguousarray(x).view(np.uint32)


def _rank_main(rank, world, port, n_total, d, k, rounds, omega, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from oracle.oracle import OracleRegTopK, default
        from paper_2501_05633_b200.sharded import gather_pairs, worker_block
        first, count = worker_block(n_total, rank, world)
        om = (np.full(n_total, np.float32(1.0) / np.float32(n_total), np.float32) if omega is None
              else np.asarray(omega, np.float32))
        data = _grads(n_total, d, rounds, seed=11)
        full = OracleRegTopK(d, n_total, k, 4.0, omega=om)           # the unsharded run, computed by every rank itself
        mine = OracleRegTopK(d, count, k, 4.0, omega=om[first: first + count])  # this rank's block of the workers
        for t in range(rounds):
            f_idx, f_val = full.worker_step(data[t])
            f_g = full.aggregate()
            idx, val = mine.worker_step(data[t][first: first + count])
            all_idx, all_val = gather_pairs(torch.from_numpy(idx), torch.from_numpy(val), n_total)
            all_idx, all_val = all_idx.numpy(), all_val.numpy()
            assert all_idx.shape == (n_total, k)
            assert np.array_equal(all_idx, f_idx), f"rank {rank} round {t}: assembled index sets differ"
            assert np.array_equal(_bits(all_val), _bits(f_val)), f"rank {rank} round {t}: assembled values differ"
            g = default().aggregate(d, om, all_idx, all_val)          # every rank is the server for itself
            assert np.array_equal(_bits(g), _bits(f_g)), f"rank {rank} round {t}: aggregates differ"
            # state roll of the block: its own pairs, the aggregate over ALL workers
            mine.prev_idx, mine.prev_val, mine.g_prev = idx, val, g
            mine.round += 1
        out.put((rank, "ok"))
    except Exception as e:  # reported to the parent instead of a hang
        out.put((rank, f"{type(e).__name__}: {e}"))
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("n_total,omega", [(4, None), (5, [0.1, 0.3, 0.2, 0.25, 0.15])])
def test_sharded_exchange_matches_the_unsharded_oracle(n_total, omega):
    from oracle import oracle
    oracle.build()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    world = 2
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, n_total, 3000, 60, 4, omega, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = [out.get(timeout=240) for _ in range(world)]
    for p in procs:
        p.join(timeout=60)
    assert sorted(results) == [(0, "ok"), (1, "ok")], results


def test_worker_block_covers_all_workers_once():
    from paper_2501_05633_b200.sharded import worker_block
    for n_total in range(1, 20):
        for world in range(1, n_total + 1):
            seen = []
            for r in range(world):
                first, count = worker_block(n_total, r, world)
                assert count in (n_total // world, n_total // world + 1)
                seen += list(range(first, first + count))
            assert seen == list(range(n_total))
    with pytest.raises(ValueError):
        worker_block(2, 0, 3)


@pytest.mark.gpu
@pytest.mark.parametrize("n_total,split,omega", [(4, (2, 2), None), (5, (3, 2), [0.1, 0.3, 0.2, 0.25, 0.15]), (8, (4, 4), None)])
def test_aggregate_gathered_two_contexts_one_gpu(n_total, split, omega):
    from oracle.oracle import OracleRegTopK
    from paper_2501_05633_b200 import RegTopK
    d, k, rounds = 120_001, 1200, 5
    om = (np.full(n_total, np.float32(1.0) / np.float32(n_total), np.float32) if omega is None
          else np.asarray(omega, np.float32))
    data = _grads(n_total, d, rounds, seed=5)
    ora = OracleRegTopK(d, n_total, k, 4.0, omega=om)
    firsts = [0, split[0]]
    libs = [RegTopK(d, split[r], k, mu=4.0, omega=[float(x) for x in om[firsts[r]: firsts[r] + split[r]]]) for r in range(2)]
    for t in range(rounds):
        o_idx, o_val = ora.worker_step(data[t])
        o_g = ora.aggregate()
        parts = [libs[r].worker_step(torch.from_numpy(data[t][firsts[r]: firsts[r] + split[r]]).cuda()) for r in range(2)]
        all_idx = torch.cat([p[0] for p in parts], dim=0).contiguous()  # what the all-gather assembles
        all_val = torch.cat([p[1] for p in parts], dim=0).contiguous()
        assert np.array_equal(all_idx.cpu().numpy(), o_idx), f"round {t}: index sets differ"
        assert np.array_equal(_bits(all_val.cpu().numpy()), _bits(o_val)), f"round {t}: values differ"
        for r in range(2):
            g = libs[r].aggregate_gathered(all_idx, all_val, None if omega is None else [float(x) for x in om])
            libs[r].status()
            assert np.array_equal(_bits(g.cpu().numpy()), _bits(o_g)), f"round {t} rank {r}: aggregates differ"
            eps = libs[r].residual().cpu().numpy()
            assert np.array_equal(_bits(eps), _bits(ora.eps[firsts[r]: firsts[r] + split[r]])), f"round {t}: residuals differ"
    for lib in libs:
        lib.close()


@pytest.mark.gpu
def test_aggregate_gathered_argument_errors():
    from paper_2501_05633_b200 import RegTopK
    from paper_2501_05633_b200.binding import RegTopKError
    lib = RegTopK(1000, 2, 10)
    idx = torch.arange(10, dtype=torch.int32, device="cuda").repeat(4, 1).contiguous()  # distinct within a worker
    val = torch.zeros((4, 10), dtype=torch.float32, device="cuda")
    with pytest.raises(RegTopKError):  # no worker_step yet
        lib.aggregate_gathered(idx, val)
    with pytest.raises(TypeError):
        lib.aggregate_gathered(idx[:, :5].contiguous(), val[:, :5].contiguous())
    lib.worker_step(torch.randn(2, 1000).cuda())
    bad = idx.clone()
    bad[1, 3] = 5000  # an index out of range is ignored, nothing faults
    bad[2, 4] = -7
    val[:] = 1.0
    g = lib.aggregate_gathered(bad, val)
    lib.status()
    assert float(g.sum().item()) == pytest.approx((40 - 2) * 0.25)
    lib.close()
