"""CUDA library against the CPU oracle, element by element, through the C ABI (needs a B200)."""
import numpy as np
import pytest
import torch

from paper_2501_05633_b200 import RegTopK, binding, synth
from paper_2501_05633_b200.binding import RegTopKError
from tests.parity import run_parity

pytestmark = pytest.mark.gpu


def gauss_rounds(N, d, T, seed, ld=None, scale=None, dtype=torch.float32, quant=None):
    g = torch.Generator().manual_seed(seed)
    ld = ld or d
    for t in range(T):
        x = torch.zeros((N, ld), dtype=torch.float32)
        v = torch.randn((N, d), generator=g)
        if scale is not None:
            v = v * scale
        if quant:
            v = torch.round(v * quant) / quant
        x[:, :d] = v
        yield x.to(dtype)


# ---- tiny and ragged sizes, every k regime -----------------------------------------------------------
@pytest.mark.parametrize("d,N,k", [(1, 1, 1), (2, 2, 1), (7, 3, 7), (33, 2, 5), (511, 2, 17), (512, 1, 512),
                                   (513, 3, 1), (4096, 8, 41), (65536, 2, 100), (65537, 2, 655),
                                   (200003, 4, 2000), (200003, 2, 200003), (1_000_003, 2, 1000),
                                   (5000, 20, 50), (3001, 33, 7), (70_000, 150, 70)])
@pytest.mark.parametrize("mu", [4.0, 0.0])
def test_sizes(d, N, k, mu):
    run_parity(gauss_rounds(N, d, 4, seed=d + N), d, N, k, mu)


def test_every_tiny_size():
    """d = 1 .. 64 with k = 1, about d/2 and d (where every entry is sent), ties included."""
    for d in range(1, 65):
        for k in sorted({1, max(1, d // 2), d}):
            run_parity(gauss_rounds(2, d, 3, seed=1000 + d, quant=4 if d % 3 == 0 else 0), d, 2, k, 4.0)


@pytest.mark.parametrize("mu", [1.0, 4.0, 10.0, 1e-30])
def test_mu_sweep(mu):
    run_parity(gauss_rounds(4, 50_001, 5, seed=3), 50_001, 4, 500, mu)


@pytest.mark.parametrize("y", [0.25, 0.5, 0.9])
def test_exponent_variant(y):
    """Remark 3: selection metric |a|^y * regulariser."""
    run_parity(gauss_rounds(4, 60_001, 6, seed=23), 60_001, 4, 600, 2.0, y=y)
    w = synth.workload("resnet18", scale_to=200_000)
    s = synth.GradientStream(w, device="cpu", seed=5, pad_to=8)
    run_parity((s.next() for _ in range(5)), w.d, w.N, w.k_values()[1], w.mu, y=y,
               flags=binding.FLAG_FORCE_DENSE_SELECT if y == 0.5 else 0)


def test_custom_weights():
    run_parity(gauss_rounds(3, 30_000, 4, seed=5), 30_000, 3, 300, 4.0, omega=[0.3, 0.5, 0.2])


@pytest.mark.parametrize("ld_extra", [0, 1, 2, 3, 5])
def test_unaligned_rows(ld_extra):
    d = 100_001
    run_parity(gauss_rounds(3, d, 3, seed=9, ld=d + ld_extra), d, 3, 1000, 4.0)


def test_unaligned_base_pointer():
    d, N, k = 40_000, 2, 400
    rounds = []
    for x in gauss_rounds(N, d, 3, seed=4, ld=d + 4):
        buf = torch.zeros(N * (d + 4) + 1)
        view = buf[1:].view(N, d + 4)  # base pointer 4 bytes off a 16-byte boundary
        view.copy_(x)
        rounds.append(view)

    class DevRounds:
        def __iter__(self):
            for v in rounds:
                dbuf = torch.zeros(N * (d + 4) + 1, device="cuda")
                dv = dbuf[1:].view(N, d + 4)
                dv.copy_(v)
                yield dv

    run_parity(DevRounds(), d, N, k, 4.0)


# ---- degenerate inputs ---------------------------------------------------------------------------------
def test_all_zero_gradients():
    d, N, k = 70_001, 2, 700
    run_parity([torch.zeros(N, d) for _ in range(3)], d, N, k, 4.0, expect_dense=True)


def test_all_equal_gradients():
    d, N, k = 70_001, 2, 700
    run_parity([torch.full((N, d), 0.5), torch.full((N, d), -0.25), torch.full((N, d), 0.5)], d, N, k, 4.0,
               expect_dense=True)


def test_fewer_nonzeros_than_k():
    d, N, k = 100_000, 3, 1000
    rounds = []
    g = torch.Generator().manual_seed(1)
    for t in range(4):
        x = torch.zeros(N, d)
        pos = torch.randint(0, d, (N, 300), generator=g)
        x.scatter_(1, pos, torch.randn(N, 300, generator=g))
        rounds.append(x)
    run_parity(rounds, d, N, k, 4.0)


def test_heavy_ties():
    run_parity(gauss_rounds(3, 150_000, 5, seed=8, quant=2), 150_000, 3, 1500, 4.0)
    run_parity(gauss_rounds(3, 150_000, 4, seed=8, quant=2), 150_000, 3, 1500, 4.0,
               flags=binding.FLAG_FORCE_DENSE_SELECT)


def test_bf16_gradients():
    run_parity(gauss_rounds(4, 120_007, 5, seed=12, ld=120_008, dtype=torch.bfloat16), 120_007, 4, 1200, 4.0)
    run_parity(gauss_rounds(2, 120_007, 3, seed=13, ld=120_007, dtype=torch.bfloat16), 120_007, 2, 120, 4.0)


def test_denormals_and_huge_values():
    d, N = 60_000, 2
    g = torch.Generator().manual_seed(2)
    rounds = []
    for t in range(4):
        x = torch.randn(N, d, generator=g)
        x[:, ::3] *= 1e-42  # subnormal accumulators
        x[:, 1::7] *= 1e30
        rounds.append(x)
    run_parity(rounds, d, N, 600, 4.0)


def test_non_finite_inputs_do_not_break_the_context():
    """Gradients must be finite; if they are not, the result is unspecified but nothing faults, exactly k
    distinct ascending indices still come out, and after a reset the context is exact again."""
    d, N, k = 50_000, 2, 500
    lib = RegTopK(d, N, k)
    g = torch.randn(N, d)
    g[0, 10] = float("nan")
    g[0, 11] = float("inf")
    g[1, 12] = float("-inf")
    for _ in range(3):
        idx, _ = lib.worker_step(g.cuda())
        lib.aggregate()
        torch.cuda.synchronize()
        ih = idx.cpu().numpy()
        assert np.all(np.diff(ih, axis=1) > 0) and ih.min() >= 0 and ih.max() < d
    assert lib.stats()["device_error_bits"] == 0
    lib.close()
    run_parity(gauss_rounds(N, d, 3, seed=77), d, N, k, 4.0)


# ---- the dense exact path --------------------------------------------------------------------------------
@pytest.mark.parametrize("mu", [4.0, 0.0])
def test_forced_dense_select(mu):
    run_parity(gauss_rounds(3, 90_001, 5, seed=21), 90_001, 3, 900, mu, flags=binding.FLAG_FORCE_DENSE_SELECT,
               expect_dense=True)


SAMPLE_SECTORS = 8192  # 32-byte sectors the library's cutoff sample reads per worker


def _sample_positions(d):
    Q = (d + 7) // 8
    s = np.arange(SAMPLE_SECTORS, dtype=np.int64)
    q = s * Q // SAMPLE_SECTORS
    return (q[:, None] * 8 + np.arange(8)[None, :]).reshape(-1)


def test_sample_overestimates_cutoff():
    """Large entries sit exactly where the cutoff sample looks: the guess is too high, too few
    candidates are gathered, and the dense path must still give the exact mask."""
    d, N, k = 1_000_000, 2, 5000
    pos = torch.from_numpy(_sample_positions(d))
    rounds = []
    for x in gauss_rounds(N, d, 3, seed=30):
        x[:, pos] *= 100.0
        rounds.append(x)
    run_parity(rounds, d, N, k, 4.0, expect_dense=True)


def test_sample_underestimates_cutoff():
    """Large entries sit only where the sample does not look: the guess is too low and the candidate
    list overflows."""
    d, N, k = 1_000_000, 2, 200
    keep = torch.ones(d, dtype=torch.bool)
    keep[torch.from_numpy(_sample_positions(d))] = False
    rounds = []
    for x in gauss_rounds(N, d, 3, seed=31):
        x[:, ~keep] *= 1e-3
        rounds.append(x)
    run_parity(rounds, d, N, k, 4.0, expect_dense=True)


# ---- the dense exact path on the whole grid (what large problems and the layer-wise mode use), forced at small sizes ----
GRID = binding.FLAG_GRID_DENSE_SELECT
DENSE = binding.FLAG_FORCE_DENSE_SELECT


@pytest.mark.parametrize("d,N,k", [(1, 1, 1), (7, 3, 7), (33, 2, 5), (513, 3, 1), (4096, 8, 41), (16384, 2, 100),
                                   (16385, 2, 16385), (65537, 2, 655), (200003, 4, 2000), (1_000_003, 2, 10_000),
                                   (3001, 33, 7), (2000, 1100, 20)])
@pytest.mark.parametrize("mu", [4.0, 0.0])
def test_grid_dense_sizes(d, N, k, mu):
    run_parity(gauss_rounds(N, d, 4, seed=d + N + 2), d, N, k, mu, flags=GRID | DENSE, expect_dense=True, threads=8)


def test_grid_dense_ties_zeros_bf16_wide_inplace():
    d, N, k = 70_001, 2, 700
    run_parity([torch.zeros(N, d) for _ in range(3)], d, N, k, 4.0, flags=GRID, expect_dense=True)
    run_parity([torch.full((N, d), 0.5), torch.full((N, d), -0.25), torch.full((N, d), 0.5)], d, N, k, 4.0,
               flags=GRID, expect_dense=True)
    run_parity(gauss_rounds(3, 150_000, 4, seed=8, quant=2), 150_000, 3, 1500, 4.0, flags=GRID | DENSE)
    run_parity(gauss_rounds(3, 150_000, 4, seed=8, quant=2), 150_000, 3, 1500, 4.0, flags=GRID | DENSE | WIDE)
    run_parity(gauss_rounds(2, 100_001, 4, seed=10, ld=100_008, dtype=torch.bfloat16), 100_001, 2, 1000, 4.0,
               flags=GRID | DENSE)
    run_parity(gauss_rounds(3, 80_000, 4, seed=51), 80_000, 3, 800, 2.0, y=0.5, flags=GRID | DENSE,
               inplace=lambda t: t % 2 == 0)


def test_grid_dense_crowded_threshold_bin():
    """Most of a row inside one bin of the first digit (magnitudes within 4 % of each other, all different): the bin
    does not fit the list space, the second digit narrows it until it does.  Then the same with a block of exactly
    equal magnitudes around the threshold, which needs the third digit and the ordered take of ties."""
    d, N, k = 300_000, 3, 3000
    g = torch.Generator().manual_seed(77)

    def rounds(ties):
        out = []
        for t in range(4):
            x = (1.0 + 0.04 * torch.rand(N, d, generator=g)) * torch.where(torch.rand(N, d, generator=g) < 0.5, -1.0, 1.0)
            x[:, ::7] *= 1e-3  # a share of small entries
            if ties:
                x[:, 1000:60_000] = 1.042  # 59,000 equal magnitudes above all others: the threshold falls among them
            out.append(x)
        return out

    for ties in (False, True):
        run_parity(rounds(ties), d, N, k, 4.0, flags=GRID | DENSE, expect_dense=True)
        run_parity(rounds(ties), d, N, 0, 4.0, layers=([100_000, 100_064, 300_000], [1000, 7, 1993]))
        run_parity(rounds(ties), d, N, k, 0.0, flags=GRID | DENSE | WIDE, expect_dense=True)


def test_grid_dense_after_a_missed_cutoff():
    """The sample's guess is too high for both workers (as in test_sample_overestimates_cutoff), with the flag that
    hands such workers to the full-grid kernel; then a run in which only some rounds need it."""
    d, N, k = 1_000_000, 2, 5000
    pos = torch.from_numpy(_sample_positions(d))
    rounds = []
    for t, x in enumerate(gauss_rounds(N, d, 4, seed=30)):
        if t != 2:
            x[:, pos] *= 100.0
        rounds.append(x)
    run_parity(rounds, d, N, k, 4.0, flags=GRID, expect_dense=True)


# ---- numerators of the distortion formed during the aggregation (what large d does), forced at small sizes ----
def _shared_rounds(N, d, T, seed, dtype=torch.float32):
    """Workers share most of their gradient, so that their masks overlap and one g[j] has many contributors."""
    g = torch.Generator().manual_seed(seed)
    for t in range(T):
        base = torch.randn(d, generator=g)
        yield (base[None, :] + 0.3 * torch.randn(N, d, generator=g)).to(dtype)


def test_numerators_at_aggregate():
    NUM = binding.FLAG_NUMERATORS_AT_AGGREGATE
    for (d, N, k) in [(7, 3, 7), (4096, 8, 41), (200_003, 4, 2000), (70_000, 40, 700)]:
        run_parity(_shared_rounds(N, d, 5, seed=d), d, N, k, 4.0, flags=NUM)
    run_parity(_shared_rounds(5, 150_001, 5, seed=3), 150_001, 5, 1500, 2.0, flags=NUM | WIDE, omega=[0.1, 0.3, 0.2, 0.25, 0.15])
    run_parity(_shared_rounds(4, 100_000, 5, seed=4, dtype=torch.bfloat16), 100_000, 4, 1000, 4.0, flags=NUM, y=0.5,
               inplace=lambda t: t % 2 == 1)
    run_parity(_shared_rounds(3, 90_001, 5, seed=5), 90_001, 3, 900, 4.0, flags=NUM | DENSE | GRID)
    # rounds with and without the numerators mixed: a reset and a state import fall back to the gather from g
    d, N, k = 60_000, 3, 600
    rounds = list(_shared_rounds(N, d, 6, seed=6))
    run_parity(rounds, d, N, k, 4.0, flags=NUM, reset_after=3)


# ---- layer-wise selection: one Top-k per contiguous layer --------------------------------------------------
def _layers_of(sizes, frac, kmin=1):
    ends = np.cumsum(sizes).tolist()
    ks = [int(min(s, max(kmin, int(frac * s + 0.5)))) for s in sizes]
    return ends, ks


@pytest.mark.parametrize("mu", [4.0, 0.0])
def test_layerwise_tiny_and_ragged(mu):
    for sizes, frac in [([1], 1.0), ([3, 4], 0.5), ([5, 1, 7, 2, 33], 0.3), ([64, 64, 1728, 64, 36864, 10], 0.05),
                        ([16384, 16385, 3, 16383], 0.01), ([40_001, 7, 99_999], 0.02)]:
        d = int(sum(sizes))
        run_parity(gauss_rounds(3, d, 4, seed=d), d, 3, 0, mu, layers=_layers_of(sizes, frac))


def test_layerwise_one_layer_is_the_global_selection():
    d, N, k = 120_001, 3, 1200
    rounds = list(gauss_rounds(N, d, 4, seed=77))
    lib_l = RegTopK(d, N, k, mu=4.0, layers=([d], [k]))
    lib_g = RegTopK(d, N, k, mu=4.0)
    for g in rounds:
        il, vl = lib_l.worker_step(g.cuda())
        ig, vg = lib_g.worker_step(g.cuda())
        assert torch.equal(il, ig) and torch.equal(vl.view(torch.int32), vg.view(torch.int32))
        assert torch.equal(lib_l.aggregate().view(torch.int32), lib_g.aggregate().view(torch.int32))
    lib_l.status(); lib_g.status()
    run_parity(rounds, d, N, 0, 4.0, layers=([d], [k]))


def test_layerwise_ties_zeros_bf16_wide_exponent():
    sizes = [5000, 64, 64, 30_000, 128, 70_003]
    d = int(sum(sizes))
    L = _layers_of(sizes, 0.02)
    run_parity(gauss_rounds(3, d, 4, seed=8, quant=2), d, 3, 0, 4.0, layers=L)
    run_parity([torch.zeros(2, d) for _ in range(3)], d, 2, 0, 4.0, layers=L)
    run_parity([torch.full((2, d), 0.5), torch.full((2, d), -0.25), torch.full((2, d), 0.5)], d, 2, 0, 4.0, layers=L)
    run_parity(gauss_rounds(2, d, 4, seed=10, ld=d + 5, dtype=torch.bfloat16), d, 2, 0, 4.0, layers=L)
    run_parity(gauss_rounds(3, d, 4, seed=11), d, 3, 0, 4.0, layers=L, flags=WIDE)
    run_parity(gauss_rounds(3, d, 4, seed=12), d, 3, 0, 2.0, y=0.5, layers=L, inplace=lambda t: t % 2 == 1)
    x = [g for g in gauss_rounds(2, d, 3, seed=13)]
    for g in x:
        g[:, 5000:5128] = 0.0  # two layers that are zero throughout: their winners are the lowest indices
    run_parity(x, d, 2, 0, 4.0, layers=L)


@pytest.mark.parametrize("name", ["resnet18", "resnet50", "gpt2"])
def test_layerwise_scaled_workloads(name):
    """The model-shaped tensor tables scaled down, every tensor a layer with the workload's sparsity."""
    w = synth.workload(name, scale_to=300_000)
    L = _layers_of(w.shapes, w.sparsity[-1])
    s = synth.GradientStream(w, device="cpu", seed=19, pad_to=8)
    run_parity((s.next() for _ in range(6)), w.d, w.N, 0, w.mu, layers=L)


def _drift_rounds(N, d, T, seed, scales):
    """A fixed direction plus noise, as error feedback meets it in training: unsent entries pile up under the
    thresholds round after round.  scales[t] multiplies round t (a missing entry is 1)."""
    g = torch.Generator().manual_seed(seed)
    base = torch.randn(d, generator=g)
    for t in range(T):
        v = 0.5 * base + torch.randn((N, d), generator=g)
        yield (v * float(scales.get(t, 1.0))).contiguous()


def test_layerwise_long_in_bin_lists_over_many_rounds():
    """A layer with k_l = 30,000: its in-bin list is ranked from shared memory (more than a block's worth of entries)
    and, when it outgrows that, gathered after a first digit; the bounds for the next round go by rank."""
    sizes = [1_500_000, 300, 64, 200_000, 17]
    d = int(sum(sizes))
    run_parity(_drift_rounds(2, d, 10, seed=31, scales={}), d, 2, 0, 4.0, layers=_layers_of(sizes, 0.02), threads=8)


def test_layerwise_thresholds_that_fall_and_lists_that_overflow():
    """Rounds whose gradients shrink a thousandfold with the sign turned (the accumulators and with them the layers'
    thresholds fall under the bounds left for the streaming pass: those layers are counted again from the rows) and
    rounds that grow a hundredfold (every entry passes the old bounds and the candidate lists overflow)."""
    sizes = [120_000, 64, 64, 260_000, 1000, 30_011]
    d = int(sum(sizes))
    scales = {3: -1e-3, 4: -1e-3, 6: 100.0, 8: 1e-2, 9: -30.0}
    run_parity(_drift_rounds(3, d, 11, seed=5, scales=scales), d, 3, 0, 4.0, layers=_layers_of(sizes, 0.01), threads=8)


@pytest.mark.parametrize("N,n_layers", [(24, 100), (40, 450)])
def test_layerwise_more_segments_than_the_shared_tables_hold(N, n_layers):
    rng = np.random.default_rng(N)
    sizes = [int(x) for x in rng.integers(20, 90, size=n_layers)]
    d = int(sum(sizes))
    run_parity(_drift_rounds(N, d, 5, seed=N, scales={}), d, N, 0, 4.0, layers=_layers_of(sizes, 0.1), threads=8)


def test_layerwise_a_crowded_layer_beside_list_fed_ones():
    """One layer of equal values (its threshold bin never fits the list space: second and third digit on the rows, ties
    in index order) in a worker whose other layers are selected from the candidate list in the same launch."""
    sizes = [30_000, 200_000, 64, 50_000, 20_011]
    d = int(sum(sizes))
    g = torch.Generator().manual_seed(41)
    rounds = []
    for t in range(8):
        x = torch.randn((3, d), generator=g)
        x[:, 30_000:230_000] = 0.25 if t % 2 == 0 else -0.125  # the crowded layer
        rounds.append(x)
    run_parity(rounds, d, 3, 0, 4.0, layers=_layers_of(sizes, 0.005), threads=8)


def test_layerwise_sixty_rounds_on_a_tensor_table():
    """Long enough for the bounds that each layer's selection leaves for the next round to settle and to be missed now
    and then (ResNet-18's tensor table scaled down, error feedback ageing over 60 rounds)."""
    w = synth.workload("resnet18", scale_to=400_000)
    L = _layers_of(w.shapes, 0.01)
    s = synth.GradientStream(w, device="cpu", seed=23, pad_to=8)
    run_parity((s.next() for _ in range(60)), w.d, w.N, 0, w.mu, layers=L, threads=8)


def test_layerwise_argument_errors():
    for layers in [([10, 5], [1, 1]), ([5, 9], [1, 1]), ([5, 10], [0, 1]), ([5, 10], [6, 1]), ([5, 5, 10], [1, 1, 1])]:
        with pytest.raises(RegTopKError):
            RegTopK(10, 2, 2, layers=layers)
    assert binding.workspace_bytes(10, 2, 3, layers=([5, 10], [1, 1])) == 0  # k must be the sum of the per-layer k


# ---- the list handling of large N*k (separate full-grid kernels, pairs unzipped afterwards), forced at small
#      sizes ------------------------------------------------------------------------------------------------
WIDE = binding.FLAG_FORCE_WIDE_LISTS


@pytest.mark.parametrize("d,N,k", [(1, 1, 1), (7, 3, 7), (33, 2, 5), (512, 1, 512), (513, 3, 1), (4096, 8, 41),
                                   (65537, 2, 655), (200003, 4, 2000), (200003, 2, 200003), (1_000_003, 2, 10_000),
                                   (3001, 33, 7), (70_000, 150, 70)])
@pytest.mark.parametrize("mu", [4.0, 0.0])
def test_wide_lists_sizes(d, N, k, mu):
    run_parity(gauss_rounds(N, d, 4, seed=d + N + 1), d, N, k, mu, flags=WIDE)


def test_wide_lists_by_size_alone():
    """N*k large enough for the wide kernels without the flag: one worker with a long list, and a thousand
    workers with short ones (more workers than the grid has blocks)."""
    run_parity(gauss_rounds(1, 1_000_003, 3, seed=3, ld=1_000_008), 1_000_003, 1, 300_000, 4.0, threads=8, select_mode=1)
    run_parity(gauss_rounds(1000, 600_000, 3, seed=0), 600_000, 1000, 300, 4.0, threads=8, select_mode=1)


def test_wide_lists_dense_path_ties_bf16_exponent_inplace():
    run_parity(gauss_rounds(3, 90_001, 4, seed=21), 90_001, 3, 900, 4.0, flags=WIDE | binding.FLAG_FORCE_DENSE_SELECT,
               expect_dense=True)
    run_parity(gauss_rounds(3, 150_000, 4, seed=8, quant=2), 150_000, 3, 1500, 4.0, flags=WIDE)
    run_parity(gauss_rounds(2, 100_001, 4, seed=10, ld=100_008, dtype=torch.bfloat16), 100_001, 2, 1000, 4.0, flags=WIDE)
    run_parity(gauss_rounds(3, 80_000, 4, seed=51), 80_000, 3, 800, 2.0, y=0.5, flags=WIDE, inplace=lambda t: t % 2 == 0)


def test_wide_lists_sample_misses_and_long_run():
    d, N, k = 1_000_000, 2, 5000
    pos = torch.from_numpy(_sample_positions(d))
    rounds = []
    for x in gauss_rounds(N, d, 3, seed=30):
        x[:, pos] *= 100.0
        rounds.append(x)
    run_parity(rounds, d, N, k, 4.0, expect_dense=True, flags=WIDE)
    w = synth.workload("resnet18", scale_to=400_000)
    s = synth.GradientStream(w, device="cpu", seed=31, pad_to=8)
    st = run_parity((s.next() for _ in range(20)), w.d, w.N, w.k_values()[1], w.mu, threads=8, flags=WIDE)
    assert st["dense_select_workers"] == 0, st


# ---- accumulate-in-place calls: the caller adds g into the library's rows, the library only scans them ------
@pytest.mark.parametrize("d,N,k", [(1, 1, 1), (7, 3, 7), (513, 3, 1), (4096, 8, 41), (65537, 2, 655),
                                   (200003, 4, 2000), (200003, 2, 200003), (1_000_003, 2, 1000), (70_000, 150, 70)])
@pytest.mark.parametrize("mu", [4.0, 0.0])
def test_inplace_sizes(d, N, k, mu):
    run_parity(gauss_rounds(N, d, 4, seed=d + N + 2), d, N, k, mu, inplace=lambda t: True)


def test_inplace_mixed_with_plain_rounds_bf16_and_dense_path():
    run_parity(gauss_rounds(3, 150_000, 6, seed=61), 150_000, 3, 1500, 4.0, inplace=lambda t: t % 2 == 1)
    run_parity(gauss_rounds(2, 120_007, 4, seed=62, ld=120_008, dtype=torch.bfloat16), 120_007, 2, 1200, 4.0,
               inplace=lambda t: t >= 2)
    run_parity(gauss_rounds(3, 90_001, 4, seed=63), 90_001, 3, 900, 4.0, flags=binding.FLAG_FORCE_DENSE_SELECT,
               expect_dense=True, inplace=lambda t: True)
    run_parity(gauss_rounds(3, 80_000, 4, seed=64, quant=2), 80_000, 3, 800, 2.0, y=0.5, inplace=lambda t: True)


def test_inplace_scaled_workload_long_run():
    w = synth.workload("resnet18", scale_to=400_000)
    s = synth.GradientStream(w, device="cpu", seed=33, pad_to=8)
    st = run_parity((s.next() for _ in range(20)), w.d, w.N, w.k_values()[0], w.mu, threads=8, inplace=lambda t: True)
    assert st["dense_select_workers"] == 0, st


# ---- model-shaped workloads, scaled down (several tiles, ragged tail) ---------------------------------
@pytest.mark.parametrize("name", ["resnet18", "resnet50", "gpt2", "flat1p3b"])
def test_scaled_workloads(name):
    w = synth.workload(name, scale_to=300_000)
    stream = synth.GradientStream(w, device="cpu", seed=17, pad_to=8)
    for k in w.k_values():
        k = max(k, 1)
        s = synth.GradientStream(w, device="cpu", seed=17, pad_to=8)
        run_parity((s.next() for _ in range(6)), w.d, w.N, k, w.mu)


def test_long_run_stays_exact_and_on_the_fast_path():
    """Forty rounds of error feedback (residuals pile up just below the threshold): still bit-exact, and the
    sampled cutoff never has to fall back to the dense path."""
    w = synth.workload("resnet18", scale_to=400_000)
    s = synth.GradientStream(w, device="cpu", seed=29, pad_to=8)
    st = run_parity((s.next() for _ in range(40)), w.d, w.N, w.k_values()[0], w.mu, threads=8)
    assert st["dense_select_workers"] == 0, st


def test_pile_up_under_the_threshold_does_not_keep_the_dense_path():
    """Thousands of rounds on a short cycle of batches: error feedback packs the unsent entries into a band right
    under the selection threshold that is far narrower than a bin of the cutoff sample.  A cutoff placed by
    interpolation then misses; after the first fallback the library resolves its cutoffs exactly, so the dense
    path stays the exception (the stretches of exact cutoffs double: 1024, 2048, ... rounds)."""
    w = synth.workload("gpt2", scale_to=2_000_000)
    k = w.k_values()[0]
    s = synth.GradientStream(w, device="cuda", seed=8, pad_to=32)
    ring = [s.next() for _ in range(8)]
    lib = RegTopK(w.d, w.N, k, mu=w.mu, grad_dtype=torch.bfloat16)
    rounds = 6000
    for t in range(rounds):
        lib.worker_step(ring[t % 8])
        lib.aggregate()
    lib.status()
    st = lib.stats()
    assert st["dense_select_workers"] <= w.N * 4, st  # stretches of 1024, 2048, 4096 rounds: three fallbacks at most


def test_least_squares_trajectory():
    """N=8, 512x4096 least squares, k=41, 100 rounds with step 0.1: identical masks, residuals and
    aggregates every round, hence the identical loss curve, which must fall."""
    from oracle.oracle import OracleRegTopK
    prob = synth.LeastSquares()
    lib = RegTopK(prob.d, prob.N, 41, mu=4.0)
    ora = OracleRegTopK(prob.d, prob.N, 41, 4.0)
    th_l = np.zeros(prob.d)
    th_o = np.zeros(prob.d)
    losses = [prob.loss(th_l)]
    for t in range(100):
        g_l = prob.gradients(th_l)
        g_o = prob.gradients(th_o)
        idx, val = lib.worker_step(torch.from_numpy(g_l).cuda())
        oi, ov = ora.worker_step(g_o)
        assert np.array_equal(idx.cpu().numpy(), oi) and np.array_equal(val.cpu().numpy().view(np.uint32), ov.view(np.uint32))
        assert np.array_equal(lib.residual().cpu().numpy().view(np.uint32), ora.eps.view(np.uint32))
        agg = lib.aggregate().cpu().numpy()
        assert np.array_equal(agg.view(np.uint32), ora.aggregate().view(np.uint32))
        th_l = th_l - 0.1 * agg.astype(np.float64)
        th_o = th_l.copy()
        losses.append(prob.loss(th_l))
    lib.status()
    assert losses[-1] < 0.9 * losses[0]
    assert losses[50] < losses[0]


def test_toy_logistic_example_on_the_library():
    """The paper's motivational example (Section 1.3: J = 2, two workers with x = [+-100, 1], eta = 0.9,
    theta0 = [0, 1]) run on the library: Top-1 keeps sending the cancelling first coordinate and the loss does
    not move for 90 rounds; RegTop-1 sees Delta = -1 exactly at t = 1, switches to the second coordinate and
    the loss falls.  Same picks as the oracle every round."""
    from oracle.oracle import OracleRegTopK
    from tests.oracle_pins import _toy_gradients, _toy_loss
    for mu in (0.0, 1.0):
        lib = RegTopK(2, 2, 1, mu=mu)
        ora = OracleRegTopK(2, 2, 1, mu)
        theta = np.array([0.0, 1.0])
        losses = [_toy_loss(theta)]
        picks = []
        for t in range(100):
            g = _toy_gradients(theta)
            idx, val = lib.worker_step(torch.from_numpy(g).cuda())
            oi, ov = ora.worker_step(g)
            assert np.array_equal(idx.cpu().numpy(), oi) and np.array_equal(val.cpu().numpy(), ov)
            agg = lib.aggregate().cpu().numpy()
            assert np.array_equal(agg.view(np.uint32), ora.aggregate().view(np.uint32))
            theta = theta - 0.9 * agg.astype(np.float64)
            picks.append(tuple(int(i) for i in idx.cpu().numpy()[:, 0]))
            losses.append(_toy_loss(theta))
        lib.status()
        if mu == 0.0:
            assert all(p == (0, 0) for p in picks[:90]) and all(l == losses[0] for l in losses[:91])
        else:
            assert picks[0] == (0, 0) and picks[1] == (1, 1) and losses[30] < 0.5 * losses[0]


def test_fused_model_update_trajectory():
    """theta <- theta - eta*g fused into the aggregation (Section 1): the fp32 model vector stays bit-identical to
    the oracle's over 40 rounds of the least-squares problem, and the loss falls."""
    from oracle.oracle import OracleRegTopK, default as oracle_default
    prob = synth.LeastSquares(N=4, rows=256, d=2048, seed=3)
    k, eta = 40, 0.1
    lib = RegTopK(prob.d, prob.N, k, mu=4.0)
    ora = OracleRegTopK(prob.d, prob.N, k, 4.0)
    th_dev = torch.zeros(prob.d, device="cuda")
    th_ora = np.zeros(prob.d, np.float32)
    first = prob.loss(th_ora.astype(np.float64))
    for t in range(40):
        g = prob.gradients(th_ora.astype(np.float64))
        idx, val = lib.worker_step(torch.from_numpy(g).cuda())
        oi, ov = ora.worker_step(g)
        assert np.array_equal(idx.cpu().numpy(), oi)
        agg = lib.aggregate_update(th_dev, eta)
        oracle_default().model_update(th_ora, eta, ora.aggregate())
        assert np.array_equal(agg.cpu().numpy().view(np.uint32), ora.g_prev.view(np.uint32))
        assert np.array_equal(th_dev.cpu().numpy().view(np.uint32), th_ora.view(np.uint32)), f"round {t}"
    lib.status()
    assert prob.loss(th_ora.astype(np.float64)) < 0.9 * first


def test_state_export_import_resumes_bit_identically():
    """A context restored from an exported blob continues exactly as the oracle does (which ran all rounds without
    interruption), and so does the context that exported."""
    from oracle.oracle import OracleRegTopK
    d, N, k = 150_001, 3, 1500
    rounds = list(gauss_rounds(N, d, 7, seed=91))
    ora = OracleRegTopK(d, N, k, 4.0)
    want = []
    for g in rounds:
        oi, ov = ora.worker_step(g.numpy())
        want.append((oi, ov.view(np.uint32).copy(), ora.eps.view(np.uint32).copy(), ora.aggregate().view(np.uint32).copy()))

    def check(lib, t):
        idx, val = lib.worker_step(rounds[t].cuda())
        eps = lib.residual().cpu().numpy().view(np.uint32)
        agg = lib.aggregate().cpu().numpy().view(np.uint32)
        oi, ov, oe, og = want[t]
        assert np.array_equal(idx.cpu().numpy(), oi), f"round {t}: index sets"
        assert np.array_equal(val.cpu().numpy().view(np.uint32), ov), f"round {t}: values"
        assert np.array_equal(eps, oe), f"round {t}: residuals"
        assert np.array_equal(agg, og), f"round {t}: aggregate"

    a = RegTopK(d, N, k)
    for t in range(4):
        check(a, t)
    blob = a.state_export()
    a.worker_step(rounds[4].cuda())
    with pytest.raises(RegTopKError) as e:  # mid-round: refused
        a.state_export()
    assert e.value.code == -3
    a.aggregate()
    for t in (5, 6):
        check(a, t)
    b = RegTopK(d, N, k)
    b.state_import(blob)
    for t in (4, 5, 6):
        check(b, t)
    b.status()
    other = RegTopK(d, N, k + 1)
    with pytest.raises(RegTopKError):  # a blob of a different problem
        other.state_import(blob)
    with pytest.raises(RegTopKError):
        b.state_import(blob[:1000].clone())


def test_appendix_a_table1_iteration1_on_the_library():
    """The low-dimensional example of Appendix A (J = 4, two workers, Top-3 / RegTop-3, omega = 1/2): the accumulated
    gradients reconstructed from Table 1's iteration-1 row go through the C ABI; each worker drops the entry the table
    shows as dropped, the sent values are the printed ones, and the aggregate is the printed target without the dropped
    entries' share.  Bit-identical to the oracle as well."""
    import json
    import os
    from oracle.oracle import OracleRegTopK
    fx = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "table1_iteration1.json")))
    acc = np.array(fx["worker_accumulated"], np.float32)
    sent = np.array(fx["worker_sent"], np.float64)
    for mu in (0.0, 4.0):  # iteration 1 has no previous mask: the same for Top-k and RegTop-k
        lib = RegTopK(4, 2, 3, mu=mu, omega=[0.5, 0.5])
        ora = OracleRegTopK(4, 2, 3, mu, omega=[0.5, 0.5])
        idx, val = lib.worker_step(torch.from_numpy(acc).cuda())
        g = lib.aggregate().cpu().numpy()
        lib.status()
        idx_h, val_h = idx.cpu().numpy(), val.cpu().numpy()
        for n in range(2):
            dense = np.zeros(4)
            dense[idx_h[n]] = val_h[n]
            assert np.allclose(dense, sent[n], atol=0.006)
            assert set(range(4)) - set(int(i) for i in idx_h[n]) == {fx["dropped_index_0based"][n]}
        assert np.allclose(g, sent.mean(axis=0), atol=0.006)
        oi, ov = ora.worker_step(acc)
        assert np.array_equal(idx_h, oi) and np.array_equal(val_h.view(np.uint32), ov.view(np.uint32))
        assert np.array_equal(g.view(np.uint32), ora.aggregate().view(np.uint32))


# ---- API behaviour -------------------------------------------------------------------------------------------
def test_state_reset_restarts_at_round_zero():
    run_parity(gauss_rounds(2, 20_000, 6, seed=40), 20_000, 2, 200, 4.0, reset_after=3)


def test_sequence_errors():
    lib = RegTopK(1000, 2, 10)
    g = torch.randn(2, 1000, device="cuda")
    with pytest.raises(RegTopKError) as e:
        lib.aggregate()
    assert e.value.code == -3
    lib.worker_step(g)
    with pytest.raises(RegTopKError) as e:
        lib.worker_step(g)
    assert e.value.code == -3
    lib.aggregate()
    lib.worker_step(g)
    lib.aggregate()
    lib.status()


def test_argument_errors():
    lib = RegTopK(1000, 2, 10)
    L = lib.L
    g = torch.randn(2, 1000, device="cuda")
    oi = torch.empty(2, 10, dtype=torch.int32, device="cuda")
    ov = torch.empty(2, 10, device="cuda")
    assert L.regtopk_worker_step(lib.ctx, g.data_ptr(), 999, oi.data_ptr(), ov.data_ptr()) == -1
    assert L.regtopk_worker_step(lib.ctx, None, 1000, oi.data_ptr(), ov.data_ptr()) == -1
    assert L.regtopk_worker_step(lib.ctx, g.data_ptr(), 1000, None, ov.data_ptr()) == -1
    hi = torch.empty(2, 10, dtype=torch.int32)
    hv = torch.empty(2, 10)
    with pytest.raises(RegTopKError):  # no staging reserved
        lib.round_host(g.cpu(), hi, hv)
    import ctypes
    ws = torch.empty(1024, dtype=torch.uint8, device="cuda")
    p, _ = binding._make_params(4.0, None, 0, 0)
    ctx = ctypes.c_void_p()
    assert L.regtopk_create(ctypes.byref(ctx), 1000, 2, 10, ctypes.byref(p), ws.data_ptr(), 1024, None) == -2
    assert L.regtopk_create(ctypes.byref(ctx), 1000, 2, 10, ctypes.byref(p), ws.data_ptr() + 4, 10**9, None) == -1


def test_determinism_and_output_copy():
    d, N, k = 300_000, 4, 3000
    rounds = [x.cuda() for x in gauss_rounds(N, d, 4, seed=50)]
    outs = []
    for rep in range(2):
        lib = RegTopK(d, N, k)
        rec = []
        for g in rounds:
            idx, val = lib.worker_step(g)
            og = torch.empty(d, device="cuda")
            ret = lib.aggregate(out=og)
            assert ret is og and torch.equal(og, lib.global_gradient())
            rec.append((idx.clone(), val.clone(), og.clone(), lib.residual().clone()))
        lib.status()
        outs.append(rec)
    for a, b in zip(*outs):
        for x, y in zip(a, b):
            assert torch.equal(x, y)


def test_round_host_matches_device_calls():
    d, N, k = 120_000, 3, 1200
    rounds = list(gauss_rounds(N, d, 4, seed=60))
    dev = RegTopK(d, N, k)
    host = RegTopK(d, N, k, flags=binding.FLAG_HOST_STAGING)
    for g in rounds:
        idx, val = dev.worker_step(g.cuda())
        agg = dev.aggregate()
        hi = torch.empty(N, k, dtype=torch.int32).pin_memory()
        hv = torch.empty(N, k).pin_memory()
        hg = torch.empty(d).pin_memory()
        host.round_host(g.pin_memory(), hi, hv, hg)
        assert torch.equal(hi, idx.cpu()) and torch.equal(hv, val.cpu()) and torch.equal(hg, agg.cpu())
    host.status()


def test_fast_path_is_taken_on_ordinary_data():
    w = synth.workload("resnet18", scale_to=2_000_000)
    s = synth.GradientStream(w, device="cuda", seed=3, pad_to=8)
    lib = RegTopK(w.d, w.N, w.k_values()[0])
    for t in range(6):
        lib.worker_step(s.next())
        lib.aggregate()
    lib.status()
    st = lib.stats()
    assert st["dense_select_workers"] == 0, st
    assert st["candidates_last"] <= w.N * st["candidate_capacity"]


# ---- full benchmark sizes, in the layout the benchmark times -------------------------------------------------
@pytest.mark.parametrize("name,ki,rounds", [("resnet18", 0, 3), ("resnet18", 1, 2), ("resnet50", 0, 2)])
def test_full_size_workloads(name, ki, rounds):
    w = synth.workload(name)
    s = synth.GradientStream(w, device="cuda", seed=0, pad_to=32)
    run_parity((s.next() for _ in range(rounds)), w.d, w.N, w.k_values()[ki], w.mu, select_mode=1, threads=8,
               expect_dense=False)


def test_full_size_inplace_calls():
    """The accumulate-in-place calls at the benchmark's size and layout (ResNet-18 shape, k = 0.1 %)."""
    w = synth.workload("resnet18")
    s = synth.GradientStream(w, device="cuda", seed=0, pad_to=32)
    run_parity((s.next() for _ in range(3)), w.d, w.N, w.k_values()[0], w.mu, select_mode=1, threads=8,
               expect_dense=False, inplace=lambda t: True)


# ---- full benchmark sizes too large to sort on the host: certified instead of compared --------------------------
def _certified_round(lib, ora_api, w, k, grads, eps_before, prev, g_prev, omega):
    """One round of the library, checked against the oracle without a sort: the oracle's accumulator and
    scores are computed per worker (O(d)), the library's mask is certified as the selector's answer
    (no record outside it ranks before its last-ranked record), and everything else is element-wise."""
    idx, val = lib.worker_step(grads)
    lib.status()
    idx_h, val_h = idx.cpu().numpy(), val.cpu().numpy()
    eps_after = lib.residual()
    for n in range(w.N):
        g_n = grads[n, : w.d].cpu()
        g_view = g_n.view(torch.int16).numpy().view(np.uint16) if g_n.dtype == torch.bfloat16 else g_n.numpy()
        pi, pv = (None, None) if prev is None else (prev[0][n], prev[1][n])
        a, s = ora_api.scores(g_view, eps_before[n], pi, pv, g_prev, w.mu, float(omega[n]))
        assert ora_api.mask_certificate(s, idx_h[n]) == k, f"worker {n}: not the k largest scores"
        assert np.array_equal(val_h[n].view(np.uint32), a[idx_h[n]].view(np.uint32)), f"worker {n}: sent values"
        a[idx_h[n]] = 0.0
        assert np.array_equal(eps_after[n].cpu().numpy().view(np.uint32), a.view(np.uint32)), f"worker {n}: residual"
        del a, s
    agg = lib.aggregate().cpu().numpy()
    want = ora_api.aggregate(w.d, omega, idx_h, val_h)
    assert np.array_equal(agg.view(np.uint32), want.view(np.uint32)), "aggregate"
    lib.status()
    return (idx_h, val_h), agg


@pytest.mark.parametrize("name,ki,rounds", [("gpt2", 0, 2), ("gpt2", 1, 2), ("flat1p3b", 0, 2), ("flat1p3b", 1, 2),
                                            ("flat1p3b", 2, 2)])
def test_full_size_certified(name, ki, rounds):
    import psutil
    from oracle.oracle import default as oracle_default
    w = synth.workload(name)
    need_host = 5 * w.N * w.d * 4  # residual copies, one worker's gradient, accumulator and scores
    if psutil.virtual_memory().available < need_host:
        pytest.skip("not enough host memory for the element-wise checks")
    k = w.k_values()[ki]
    tdt = torch.bfloat16 if w.grad_dtype == "bf16" else torch.float32
    s = synth.GradientStream(w, device="cuda", seed=0, pad_to=32)
    lib = RegTopK(w.d, w.N, k, mu=w.mu, grad_dtype=tdt)
    omega = np.full(w.N, np.float32(1.0) / np.float32(w.N), np.float32)
    eps_before = np.zeros((w.N, w.d), np.float32)
    prev, g_prev = None, None
    for t in range(rounds):
        grads = s.next()
        prev, g_prev = _certified_round(lib, oracle_default(), w, k, grads, eps_before, prev, g_prev, omega)
        if t + 1 < rounds:
            eps_before = lib.residual().cpu().numpy()
        del grads
    assert lib.stats()["dense_select_workers"] == 0


# ---- layer-wise selection at the benchmark's sizes ----------------------------------------------------------------
def test_full_size_layerwise_resnet18():
    """Every tensor of the ResNet-18 table a layer with 0.1 % of its size, as `bench.py --select layerwise` runs it:
    round 0 from the rows, the later rounds from the candidate lists."""
    w = synth.workload("resnet18")
    L = _layers_of(w.shapes, w.sparsity[0])
    s = synth.GradientStream(w, device="cuda", seed=0, pad_to=32)
    run_parity((s.next() for _ in range(10)), w.d, w.N, 0, w.mu, layers=L, threads=8)


def test_full_size_layerwise_resnet50():
    """The ResNet-50 table at full size: 30 % of its coordinates lie in frozen tensors (no gradient), whose layers select
    their lowest indices; one tensor is frozen in part."""
    w = synth.workload("resnet50")
    L = _layers_of(w.shapes, w.sparsity[0])
    s = synth.GradientStream(w, device="cuda", seed=0, pad_to=32)
    run_parity((s.next() for _ in range(4)), w.d, w.N, 0, w.mu, layers=L, threads=8)


def test_full_size_layerwise_certified_gpt2():
    """The GPT-2 table (bf16 gradients, 148 layers with 0.01 % each) at full size, certified layer by layer without a
    sort: inside every layer no entry outside the library's selection ranks before its last-ranked entry."""
    import psutil
    from oracle.oracle import default as oracle_default
    w = synth.workload("gpt2")
    if psutil.virtual_memory().available < 5 * w.N * w.d * 4:
        pytest.skip("not enough host memory for the element-wise checks")
    ends, ks = _layers_of(w.shapes, w.sparsity[0])
    k = int(sum(ks))
    api = oracle_default()
    s = synth.GradientStream(w, device="cuda", seed=0, pad_to=32)
    lib = RegTopK(w.d, w.N, 0, mu=w.mu, grad_dtype=torch.bfloat16, layers=(ends, ks))
    omega = np.full(w.N, np.float32(1.0) / np.float32(w.N), np.float32)
    eps_before = np.zeros((w.N, w.d), np.float32)
    prev, g_prev = None, None
    for t in range(3):
        grads = s.next()
        idx, val = lib.worker_step(grads)
        lib.status()
        idx_h, val_h = idx.cpu().numpy(), val.cpu().numpy()
        eps_after = lib.residual()
        for n in range(w.N):
            g_view = grads[n, : w.d].cpu().view(torch.int16).numpy().view(np.uint16)
            pi, pv = (None, None) if prev is None else (prev[0][n], prev[1][n])
            a, sc = api.scores(g_view, eps_before[n], pi, pv, g_prev, w.mu, float(omega[n]))
            assert np.all(np.diff(idx_h[n]) > 0), f"worker {n}: indices not ascending"
            cut = np.searchsorted(idx_h[n], np.asarray([0] + ends))
            begin = 0
            for l, end in enumerate(ends):
                sel = idx_h[n][cut[l]: cut[l + 1]] - begin
                assert sel.shape[0] == ks[l], f"worker {n} layer {l}: {sel.shape[0]} selected, {ks[l]} wanted"
                assert api.mask_certificate(sc[begin:end], sel) == ks[l], f"worker {n} layer {l}: not its k largest scores"
                begin = end
            assert np.array_equal(val_h[n].view(np.uint32), a[idx_h[n]].view(np.uint32)), f"worker {n}: sent values"
            a[idx_h[n]] = 0.0
            assert np.array_equal(eps_after[n].cpu().numpy().view(np.uint32), a.view(np.uint32)), f"worker {n}: residual"
            del a, sc
        agg = lib.aggregate().cpu().numpy()
        want = api.aggregate(w.d, omega, idx_h, val_h)
        assert np.array_equal(agg.view(np.uint32), want.view(np.uint32)), "aggregate"
        lib.status()
        prev, g_prev = (idx_h, val_h), agg
        if t < 2:
            eps_before = lib.residual().cpu().numpy()
        del grads
    assert k == lib.k
    lib.close()
