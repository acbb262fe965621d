"""The checked build of the CUDA library (-DREGTOPK_DEBUG=1: every data-dependent index is range-checked on the
device, a bad one is counted and skipped) run through the parity cases of every code path, in a process of its
own so that no other test sees that library.  Parity must hold and no range check may have fired."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

SCRIPT = r"""
import sys
sys.path.insert(0, %(root)r)
import torch
from paper_2501_05633_b200 import binding
binding._LIB = binding.build_checked()          # before the first load: this process uses the checked library only
from paper_2501_05633_b200 import synth
from tests.parity import run_parity
from tests.test_gpu_parity import gauss_rounds

WIDE, DENSE = binding.FLAG_FORCE_WIDE_LISTS, binding.FLAG_FORCE_DENSE_SELECT
stats = []
for (d, N, k) in [(1, 1, 1), (513, 3, 1), (4096, 8, 41), (65537, 2, 655), (200003, 2, 200003), (3001, 33, 7)]:
    for mu in (4.0, 0.0):
        for flags in (0, WIDE):
            stats.append(run_parity(gauss_rounds(N, d, 3, seed=d + N), d, N, k, mu, flags=flags))
stats.append(run_parity(gauss_rounds(3, 90_001, 4, seed=21), 90_001, 3, 900, 4.0, flags=DENSE, expect_dense=True))
stats.append(run_parity(gauss_rounds(3, 90_001, 4, seed=21), 90_001, 3, 900, 4.0, flags=DENSE | WIDE, expect_dense=True))
stats.append(run_parity(gauss_rounds(3, 150_000, 4, seed=8, quant=2), 150_000, 3, 1500, 4.0))
GRID = binding.FLAG_GRID_DENSE_SELECT
for (d, N, k) in [(1, 1, 1), (513, 3, 1), (16385, 2, 16385), (200003, 4, 2000), (2000, 1100, 20)]:
    stats.append(run_parity(gauss_rounds(N, d, 3, seed=d + N), d, N, k, 4.0, flags=GRID | DENSE, expect_dense=True))
stats.append(run_parity(gauss_rounds(3, 150_000, 4, seed=8, quant=2), 150_000, 3, 1500, 4.0, flags=GRID | DENSE))
stats.append(run_parity([torch.full((2, 70_001), 0.5)] * 3, 70_001, 2, 700, 4.0, flags=GRID, expect_dense=True))
# a threshold bin too crowded for the list space (second digit, then the list), and a block of equal magnitudes at
# the threshold (third digit, ordered ties)
gen = torch.Generator().manual_seed(77)
for ties in (False, True):
    crowded = []
    for t in range(3):
        x = (1.0 + 0.04 * torch.rand(3, 300_000, generator=gen)) * torch.where(torch.rand(3, 300_000, generator=gen) < 0.5, -1.0, 1.0)
        if ties:
            x[:, 1000:60_000] = 1.042
        crowded.append(x)
    stats.append(run_parity(crowded, 300_000, 3, 3000, 4.0, flags=GRID | DENSE, expect_dense=True))
import numpy as np
sizes = [5000, 64, 64, 30_000, 128, 70_003, 3, 16385]
layers = (np.cumsum(sizes).tolist(), [max(1, s // 50) for s in sizes])
for fl in (0, WIDE):
    stats.append(run_parity(gauss_rounds(3, sum(sizes), 4, seed=8, quant=2 if fl else 0), sum(sizes), 3, 0, 4.0, layers=layers, flags=fl))
stats.append(run_parity(gauss_rounds(2, 120_007, 4, seed=12, ld=120_008, dtype=torch.bfloat16), 120_007, 2, 1200, 4.0))
stats.append(run_parity(gauss_rounds(3, 100_001, 4, seed=9, ld=100_004), 100_001, 3, 1000, 4.0,
                        inplace=lambda t: t %% 2 == 1))
for name in ("resnet18", "gpt2"):
    w = synth.workload(name, scale_to=300_000)
    for k in w.k_values():
        s = synth.GradientStream(w, device="cpu", seed=17, pad_to=8)
        stats.append(run_parity((s.next() for _ in range(6)), w.d, w.N, max(k, 1), w.mu))
# non-finite gradients: the checked build says so through status(), and a reset clears it
from paper_2501_05633_b200 import RegTopK
from paper_2501_05633_b200.binding import RegTopKError
lib = RegTopK(50_000, 2, 500)
g = torch.randn(2, 50_000)
lib.worker_step(g.cuda()); lib.aggregate(); lib.status()
g[1, 77] = float("inf")
lib.worker_step(g.cuda()); lib.aggregate()
try:
    lib.status()
    raise SystemExit("non-finite accumulator not reported")
except RegTopKError as e:
    assert e.code == -1, e.code
lib.state_reset()
lib.worker_step(torch.randn(2, 50_000).cuda()); lib.aggregate(); lib.status()
lib.close()
bad = [st for st in stats if st["device_error_bits"]]
assert not bad, bad
assert binding.library_path().endswith("libregtopk_checked.so")
print("checked build: %%d parity runs, no range check fired" %% len(stats))
"""


@pytest.mark.gpu
def test_checked_build_runs_every_path_without_a_range_fault():
    r = subprocess.run([sys.executable, "-c", SCRIPT % {"root": ROOT}], capture_output=True, text=True, timeout=1500)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-4000:]
    assert "no range check fired" in r.stdout
