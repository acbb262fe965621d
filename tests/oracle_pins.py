"""Pins of the CPU oracle: checks against what the paper and the mathematics fix, none of which calls
the oracle to produce its own expected value.  Each function takes an OracleAPI so that the mutation
test can run the same pins on deliberately broken builds."""
import itertools
import json
import math
import os

import numpy as np

from oracle.oracle import OracleRegTopK

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
F32_EPS = 2.0 ** -24


# ---- independent Top-k with error feedback (Algorithm 1), numpy only ------------------------------
def topk_error_feedback_numpy(grads_rounds, k, omega):
    """Algorithm 1 for N workers plus the server sum. Ties: lower index (stable sort)."""
    N, d = grads_rounds[0].shape
    eps = np.zeros((N, d), np.float32)
    out = []
    for g in grads_rounds:
        idx = np.empty((N, k), np.int32)
        val = np.empty((N, k), np.float32)
        agg = np.zeros(d, np.float32)
        for n in range(N):
            a = (eps[n] + g[n].astype(np.float32)).astype(np.float32)
            order = np.argsort(-np.abs(a), kind="stable")
            sel = np.sort(order[:k])
            idx[n], val[n] = sel, a[sel]
            sparse = np.zeros(d, np.float32)
            sparse[sel] = a[sel]
            eps[n] = a - sparse
            contrib = np.zeros(d, np.float32)
            contrib[sel] = np.float32(omega[n]) * a[sel]
            agg = (agg + contrib).astype(np.float32)
        out.append((idx, val, eps.copy(), agg))
    return out


# ---- pins ----------------------------------------------------------------------------------------
def pin_tanh(api):
    x = np.concatenate([np.linspace(0, 0.3, 3001), np.linspace(0.2, 9.4, 9201),
                        np.logspace(-30, -1, 300), [0.25, 9.25, 9.2499, 20.0, np.inf]]).astype(np.float32)
    y = api.tanh_spec(x)
    ref = np.tanh(x.astype(np.float64))
    nz = ref > 0
    assert np.max(np.abs(y[nz] - ref[nz]) / ref[nz]) <= 8 * F32_EPS
    assert api.tanh_spec(np.float32(0.0)) == 0.0
    assert np.all(api.tanh_spec(np.array([9.25, 10, 100, np.inf], np.float32)) == 1.0)
    xs = np.sort(x)
    assert np.all(np.diff(api.tanh_spec(xs)) >= 0)
    assert np.all(y <= 1.0)


def pin_bruteforce_selector(api):
    """Definition of Top_k with the lowest-index tie rule, by enumeration of all subsets."""
    rng = np.random.default_rng(7)
    for trial in range(60):
        d = int(rng.integers(1, 8))
        vals = rng.choice(np.array([0.0, 0.0, 0.5, -0.5, 1.0, -1.0, 2.0, 3.5, -3.5], np.float32), size=d)
        g = vals.astype(np.float32)
        eps0 = rng.choice(np.array([0.0, 0.0, 0.25, -1.0], np.float32), size=d).astype(np.float32)
        with_prev = trial % 2 == 1 and d >= 2
        if with_prev:
            kp = int(rng.integers(1, d + 1))
            pidx = np.sort(rng.choice(d, size=kp, replace=False)).astype(np.int32)
            pval = rng.choice(np.array([0.5, -1.0, 2.0, 4.0], np.float32), size=kp).astype(np.float32)
            gprev = rng.choice(np.array([0.0, 0.5, -1.0, 2.0], np.float32), size=d).astype(np.float32)
            eps0[pidx] = 0.0  # the residual is zero where the worker sent last round
        else:
            pidx = pval = gprev = None
        a, s = api.scores(g, eps0, pidx, pval, gprev, 2.0, 0.5)
        assert np.array_equal(a, (eps0 + g).astype(np.float32))
        for k in range(1, d + 1):
            eps = eps0.copy()
            idx, val = api.worker_step(g, eps, k, pidx, pval, gprev, 2.0, 0.5)
            # best subset: maximise the descending score tuple, then minimise the ascending index tuple
            best = None
            for sub in itertools.combinations(range(d), k):
                key = (tuple(sorted((-float(s[j]) for j in sub))), sub)
                if best is None or key < best:
                    best = key
            assert tuple(int(i) for i in idx) == best[1], (d, k, s, idx, best)
            assert np.array_equal(val, a[idx])
            expect_eps = a.copy()
            expect_eps[idx] = 0.0
            assert np.array_equal(eps.view(np.uint32), expect_eps.view(np.uint32))


def pin_dense_passthrough(api):
    """k = d: every entry is sent, nothing is left behind, the server sees the plain weighted sum."""
    rng = np.random.default_rng(3)
    N, d = 3, 17
    omega = np.array([0.5, 0.25, 0.25], np.float32)
    O = OracleRegTopK(d, N, d, 4.0, omega=omega, api=api)
    for t in range(3):
        g = rng.standard_normal((N, d)).astype(np.float32)
        idx, val = O.worker_step(g)
        agg = O.aggregate()
        assert np.array_equal(idx, np.tile(np.arange(d, dtype=np.int32), (N, 1)))
        assert np.array_equal(val, g)  # eps stays 0, so a = g
        assert not O.eps.any()
        hand = np.zeros(d, np.float32)
        for n in range(N):
            hand = (hand + omega[n] * g[n]).astype(np.float32)
        assert np.array_equal(agg, hand)


def pin_reduces_to_topk(api):
    """Round 0 of Algorithm 2, mu = 0 and mu -> 0 are Algorithm 1."""
    rng = np.random.default_rng(11)
    N, d, k, T = 4, 257, 13, 6
    omega = np.full(N, 0.25, np.float32)
    rounds = [rng.standard_normal((N, d)).astype(np.float32) for _ in range(T)]
    ref = topk_error_feedback_numpy(rounds, k, omega)
    for mu in (0.0, 1e-30):
        O = OracleRegTopK(d, N, k, mu, omega=omega, api=api)
        for t in range(T):
            idx, val = O.worker_step(rounds[t])
            agg = O.aggregate()
            assert np.array_equal(idx, ref[t][0]), (mu, t)
            assert np.array_equal(val, ref[t][1])
            assert np.array_equal(O.eps, ref[t][2])
            assert np.array_equal(agg, ref[t][3])
    # mu = 4: round 0 only
    O = OracleRegTopK(d, N, k, 4.0, omega=omega, api=api)
    idx, val = O.worker_step(rounds[0])
    assert np.array_equal(idx, ref[0][0]) and np.array_equal(val, ref[0][1])


def pin_error_feedback_identity(api):
    """ghat + eps' = a exactly, every worker, every round (Algorithm 2 steps 10 and 12)."""
    rng = np.random.default_rng(5)
    N, d, k = 3, 300, 9
    O = OracleRegTopK(d, N, k, 4.0, api=api)
    for t in range(5):
        g = (rng.standard_normal((N, d)) * rng.choice([1e-3, 1.0, 30.0], size=(N, d))).astype(np.float32)
        eps_before = O.eps.copy()
        idx, val = O.worker_step(g)
        a = (eps_before + g).astype(np.float32)
        for n in range(N):
            sent = np.zeros(d, np.float32)
            sent[idx[n]] = val[n]
            assert np.array_equal((sent + O.eps[n]).view(np.uint32), a[n].view(np.uint32))
            assert np.all(O.eps[n][idx[n]] == 0)
        O.aggregate()


def _toy_gradients(theta):
    x = np.array([[100.0, 1.0], [-100.0, 1.0]])
    out = np.empty((2, 2), np.float32)
    for n in range(2):
        z = float(theta @ x[n])
        out[n] = (-(math.exp(-z) / (1.0 + math.exp(-z))) * x[n]).astype(np.float32)
    return out


def _toy_loss(theta):
    x = np.array([[100.0, 1.0], [-100.0, 1.0]])
    return float(np.mean([math.log1p(math.exp(-float(theta @ xn))) for xn in x]))


def pin_toy_example(api):
    """Motivational toy example: J = 2, N = 2, eta = 0.9, theta0 = [0, 1].  Top-1 keeps sending the
    cancelling first coordinate for about a hundred rounds; RegTop-1 sees Delta = -1 at t = 1 and
    switches to the second coordinate."""
    for mu, name in ((0.0, "top1"), (1.0, "regtop1")):
        O = OracleRegTopK(2, 2, 1, mu, api=api)
        theta = np.array([0.0, 1.0])
        losses, picks = [_toy_loss(theta)], []
        for t in range(112):
            idx, _ = O.worker_step(_toy_gradients(theta))
            g = O.aggregate()
            theta = theta - 0.9 * g.astype(np.float64)
            picks.append(tuple(int(i) for i in idx[:, 0]))
            losses.append(_toy_loss(theta))
        if name == "top1":
            assert all(p == (0, 0) for p in picks[:90])
            assert all(l == losses[0] for l in losses[:91])  # aggregate exactly zero: no movement
            assert (1, 1) in picks[90:112]  # the accumulated error finally overtakes
        else:
            assert picks[0] == (0, 0) and losses[1] == losses[0]
            assert picks[1] == (1, 1)  # Delta = -1 exactly -> score 0 on coordinate 0
            assert losses[2] < losses[0]
            assert losses[30] < 0.5 * losses[0]


def pin_table1_iteration1(api):
    fx = json.load(open(os.path.join(GOLDEN, "table1_iteration1.json")))
    acc = np.array(fx["worker_accumulated"], np.float32)
    sent = np.array(fx["worker_sent"], np.float64)
    target = np.array(fx["aggregation_target"], np.float64)
    assert np.allclose(acc.mean(axis=0), target, atol=0.01)  # fixture is self-consistent to the printed 2 decimals
    for mu in (0.0, 4.0):  # iteration 1 is identical for Top-k and RegTop-k
        O = OracleRegTopK(4, 2, 3, mu, omega=[0.5, 0.5], api=api)
        idx, val = O.worker_step(acc)
        for n in range(2):
            dense = np.zeros(4)
            dense[idx[n]] = val[n]
            assert np.allclose(dense, sent[n], atol=0.006)
            assert set(range(4)) - set(int(i) for i in idx[n]) == {fx["dropped_index_0based"][n]}
        g = O.aggregate()
        assert np.allclose(g, sent.mean(axis=0), atol=0.006)


def pin_distortion_cases(api):
    """Eq. (Delta_def) and the tanh regulariser on hand-worked inputs, read back as score / |a|; the
    off-support entry keeps regulariser exactly 1."""
    fx = json.load(open(os.path.join(GOLDEN, "distortion_cases.json")))
    for c in fx["cases"]:
        d = 3
        g = np.array([c["a_now"], 0.375, 0.0], np.float32)  # eps = 0 on the previous support: a = g
        eps = np.array([0.0, 0.125, 0.0], np.float32)
        gprev = np.array([c["g_prev"], 123.0, 0.0], np.float32)
        a, s = api.scores(g, eps, np.array([0], np.int32), np.array([c["a_prev"]], np.float32), gprev,
                          c["mu"], c["omega"])
        assert a[0] == np.float32(c["a_now"]) and a[1] == np.float32(0.5)
        assert s[1] == np.float32(0.5) and s[2] == 0.0
        want = abs(c["a_now"]) * c["regulariser"]
        assert abs(float(s[0]) - want) <= 8 * F32_EPS * max(want, 1e-30) + (0 if want else 0), (c, s)
        if c["regulariser"] == 0.0:
            assert s[0] == 0.0


def pin_regularised_ranking(api):
    """The regulariser changes the mask the way Algorithm 2 says: a previously sent entry whose
    aggregate cancelled drops below smaller fresh entries; one confirmed by the others stays."""
    # worker with omega 1/2; entry 0: sent 2.0, aggregate 0 (cancelled) -> score 0
    # entry 1: sent 1.0, aggregate 1.0 (the other worker sent 1.0 too): Delta = (1 - .5)/(.5*1) = 1,
    #          score = tanh(2/mu) = tanh(0.5) = 0.462 for mu = 4
    # entries 2, 3 fresh with |a| = 0.45 and 0.47
    g = np.array([2.0, 1.0, 0.45, -0.47], np.float32)
    eps = np.zeros(4, np.float32)
    pidx = np.array([0, 1], np.int32)
    pval = np.array([2.0, 1.0], np.float32)
    gprev = np.array([0.0, 1.0, 0.0, 0.0], np.float32)
    e = eps.copy()
    idx, val = api.worker_step(g, e, 1, pidx, pval, gprev, 4.0, 0.5)
    assert list(idx) == [3] and val[0] == np.float32(-0.47)
    e = eps.copy()
    idx, _ = api.worker_step(g, e, 2, pidx, pval, gprev, 4.0, 0.5)
    assert list(idx) == [1, 3]
    e = eps.copy()
    idx, _ = api.worker_step(g, e, 3, pidx, pval, gprev, 4.0, 0.5)
    assert list(idx) == [1, 2, 3]
    assert np.array_equal(e, np.array([2.0, 0, 0, 0], np.float32))
    # mu = 1: tanh(2) = 0.964 puts entry 1 first again
    e = eps.copy()
    idx, _ = api.worker_step(g, e, 1, pidx, pval, gprev, 1.0, 0.5)
    assert list(idx) == [1]
    # zero accumulator on the previous support: score 0, not NaN (0/0 never evaluated)
    a, s = api.scores(np.zeros(2, np.float32), np.zeros(2, np.float32), np.array([0], np.int32),
                      np.array([0.0], np.float32), np.zeros(2, np.float32), 4.0, 0.5)
    assert s[0] == 0.0 and not np.isnan(s).any()


def pin_aggregation(api):
    """Server sum in worker order with each term rounded first; power-of-two weights make the
    products exact, so a hand sum in the same order is the answer; a case where order matters."""
    idx = np.array([[0, 2], [0, 3], [2, 3]], np.int32)
    val = np.array([[1.0, 4.0], [3.0, -8.0], [0.5, 2.0]], np.float32)
    g = api.aggregate(5, np.array([0.5, 0.25, 0.25], np.float32), idx, val)
    assert np.array_equal(g, np.array([0.5 + 0.75, 0.0, 2.0 + 0.125, -2.0 + 0.5, 0.0], np.float32))
    # (1e8 + 1) - 1e8 = 0 in binary32 in worker order 0,1,2; any other order gives 1 or 8
    idx = np.array([[0], [0], [0]], np.int32)
    val = np.array([[1e8], [1.0], [-1e8]], np.float32)
    g = api.aggregate(1, np.ones(3, np.float32), idx, val)
    assert g[0] == 0.0
    # weights that are not powers of two: two roundings per term
    w = np.array([0.3, 0.7], np.float32)
    idx = np.array([[1], [1]], np.int32)
    val = np.array([[1.1], [2.3]], np.float32)
    g = api.aggregate(2, w, idx, val)
    t0 = np.float32(w[0] * val[0, 0])
    t1 = np.float32(w[1] * val[1, 0])
    assert g[1] == np.float32(np.float32(np.float32(0) + t0) + t1)


def pin_pow(api):
    m = np.concatenate([np.linspace(1e-6, 1, 4001), np.logspace(-30, 0, 600)]).astype(np.float32)
    for p in (1.0, 1.25, 2.0, 4.0, 10.0):
        y = api.pow_spec(m, p)
        ref = np.power(m.astype(np.float64), float(np.float32(p)))
        ok = ref > 1e-36
        assert np.max(np.abs(y[ok] - ref[ok]) / ref[ok]) <= 1e-5, p
        assert np.all(np.diff(api.pow_spec(np.sort(m), p)) >= 0)
    assert np.array_equal(api.pow_spec(np.array([0.0, 1.0, 0.5, 0.25], np.float32), 2.0),
                          np.array([0.0, 1.0, 0.25, 0.0625], np.float32))
    assert api.pow_spec(np.float32(1e-30), 10.0) == 0.0  # below 2^-125: flushed to zero by definition


def pin_exponent_variant(api):
    """Remark 3: the selection metric |a|^y * tanh(|1+Delta|/mu).  Its ranking, computed in binary64 from the
    definition, must be the oracle's mask on inputs without near-ties; y = 1 is Algorithm 2 itself."""
    rng = np.random.default_rng(17)
    d, kp, mu, w = 64, 20, 2.0, 0.5
    for y in (0.25, 0.5, 0.8):
        for trial in range(5):
            g = (rng.permutation(d) + 1.0).astype(np.float32) * rng.choice([-1.0, 1.0], size=d).astype(np.float32)
            eps = np.zeros(d, np.float32)
            pidx = np.sort(rng.choice(d, size=kp, replace=False)).astype(np.int32)
            pval = (rng.integers(1, 60, size=kp) * rng.choice([-1.0, 1.0], size=kp)).astype(np.float32)
            gprev = np.zeros(d, np.float32)
            gprev[pidx] = rng.integers(-40, 40, size=kp).astype(np.float32)
            a = g.astype(np.float64)
            metric = np.abs(a) ** y
            delta = (gprev[pidx].astype(np.float64) - w * pval.astype(np.float64)) / (w * a[pidx])
            metric[pidx] *= np.tanh(np.abs(1.0 + delta) / mu)
            order = np.argsort(-metric, kind="stable")
            k = 16
            # only the boundary between the k-th and the (k+1)-th matters for the mask; a near-tie there
            # could fall either way in binary32: skip such a draw
            if metric[order[k - 1]] - metric[order[k]] < 1e-3 * metric[order[k - 1]]:
                continue
            checked = locals().get("checked", 0) + 1
            e = eps.copy()
            idx, val = api.worker_step(g, e, k, pidx, pval, gprev, mu, w, 0, y)
            assert np.array_equal(idx, np.sort(order[:k]).astype(np.int32)), (y, trial)
            assert np.array_equal(val, g[idx])
    assert checked >= 10
    # y = 1 is the unmodified algorithm
    g = rng.standard_normal(200).astype(np.float32)
    pidx = np.arange(0, 200, 7, dtype=np.int32)
    pval = rng.standard_normal(pidx.size).astype(np.float32)
    gprev = rng.standard_normal(200).astype(np.float32)
    a1 = api.scores(g, np.zeros(200, np.float32), pidx, pval, gprev, 4.0, 0.25, 1.0)[1]
    a2 = api.scores(g, np.zeros(200, np.float32), pidx, pval, gprev, 4.0, 0.25)[1]
    assert np.array_equal(a1, a2)
    # off the previous support the score stays |a| for every y
    s = api.scores(g, np.zeros(200, np.float32), pidx, pval, gprev, 4.0, 0.25, 0.5)[1]
    off = np.setdiff1d(np.arange(200), pidx)
    assert np.array_equal(s[off], np.abs(g[off]))
    with np.testing.assert_raises(ValueError):
        api.worker_step(g, np.zeros(200, np.float32), 5, None, None, None, 4.0, 0.25, 0, 1.5)


def pin_model_update(api):
    """theta' = theta - eta*g with the product rounded first; entries with g = 0 keep their bits (also -0)."""
    theta = np.array([1.0, -0.0, 0.5, 2.0, 1.0], np.float32)
    g = np.array([2.0, 0.0, -1.0, 0.0, 3.3], np.float32)
    out = api.model_update(theta.copy(), 0.5, g)
    assert np.array_equal(out[:4], np.array([0.0, -0.0, 1.0, 2.0], np.float32)) and np.signbit(out[1])
    # not a power of two: two roundings, in this order
    out = api.model_update(theta.copy(), 0.1, g)
    want = np.float32(np.float32(1.0) - np.float32(np.float32(0.1) * np.float32(3.3)))
    assert out[4] == want
    # exact cancellation that a fused multiply-subtract would miss: eta*g rounds to 1 exactly
    e = np.float32(1.0) + np.float32(2.0 ** -23)
    gg = np.array([np.float32(1.0) - np.float32(2.0 ** -24)], np.float32)
    out = api.model_update(np.array([1.0], np.float32), float(e), gg)
    assert out[0] == np.float32(np.float32(1.0) - np.float32(e * gg[0]))


def pin_bf16_gradients(api):
    """bfloat16 gradients are widened exactly before the binary32 add."""
    bits = np.array([0x3F80, 0xBF00, 0x0000, 0x4049, 0x8000], np.uint16)  # 1, -0.5, 0, 3.140625, -0
    asf = (bits.astype(np.uint32) << 16).view(np.float32)
    eps = np.array([0.5, 0.25, 0.0, 1e-3, 0.0], np.float32)
    a, s = api.scores(bits, eps, None, None, None, 4.0, 0.5)
    assert np.array_equal(a.view(np.uint32), (eps + asf).astype(np.float32).view(np.uint32))
    assert np.array_equal(s, np.abs(a))


def pin_select_modes_agree(api):
    rng = np.random.default_rng(21)
    N, d, k = 3, 5000, 61
    A = OracleRegTopK(d, N, k, 4.0, select_mode=0, api=api)
    B = OracleRegTopK(d, N, k, 4.0, select_mode=1, api=api)
    for t in range(4):
        g = np.round(rng.standard_normal((N, d)) * 4).astype(np.float32) / 4  # many ties
        ia, va = A.worker_step(g)
        ib, vb = B.worker_step(g)
        assert np.array_equal(ia, ib) and np.array_equal(va, vb) and np.array_equal(A.eps, B.eps)
        assert np.array_equal(A.aggregate(), B.aggregate())


def pin_mask_certificate(api):
    rng = np.random.default_rng(2)
    d, k = 400, 17
    g = np.round(rng.standard_normal(d) * 3).astype(np.float32)
    eps = np.zeros(d, np.float32)
    a, s = api.scores(g, eps, None, None, None, 4.0, 0.5)
    idx, _ = api.worker_step(g, eps.copy(), k, None, None, None, 4.0, 0.5)
    assert api.mask_certificate(s, idx) == k
    order = np.argsort(-s, kind="stable")
    assert np.array_equal(np.sort(order[:k]).astype(np.int32), idx)
    wrong = idx.copy()
    outsider = int(order[-1])
    wrong[0] = outsider if outsider not in idx else int(order[-2])
    wrong = np.sort(wrong)
    assert api.mask_certificate(s, wrong) != k


def _random_layers(rng, d, max_layers):
    n_seg = int(rng.integers(1, min(max_layers, d) + 1))
    cuts = np.sort(rng.choice(np.arange(1, d), size=n_seg - 1, replace=False)) if n_seg > 1 else np.array([], np.int64)
    seg_end = np.concatenate([cuts, [d]]).astype(np.int64)
    sizes = np.diff(np.concatenate([[0], seg_end]))
    seg_k = np.array([int(rng.integers(1, sz + 1)) for sz in sizes], np.int64)
    return seg_end, seg_k


def pin_layered_bruteforce(api):
    """One Top-k per layer, by enumeration: in every layer the chosen set is the best k_l-subset of that layer's
    indices (descending score tuple, then ascending index tuple); all layers' pairs come out in ascending index
    order with the raw accumulator as value; the residual is cleared exactly there."""
    rng = np.random.default_rng(17)
    for trial in range(60):
        d = int(rng.integers(2, 10))
        g = rng.choice(np.array([0.0, 0.0, 0.5, -0.5, 1.0, -1.0, 2.0, 3.5, -3.5], np.float32), size=d).astype(np.float32)
        eps0 = rng.choice(np.array([0.0, 0.0, 0.25, -1.0], np.float32), size=d).astype(np.float32)
        if trial % 2 == 1:
            kp = int(rng.integers(1, d + 1))
            pidx = np.sort(rng.choice(d, size=kp, replace=False)).astype(np.int32)
            pval = rng.choice(np.array([0.5, -1.0, 2.0, 4.0], np.float32), size=kp).astype(np.float32)
            gprev = rng.choice(np.array([0.0, 0.5, -1.0, 2.0], np.float32), size=d).astype(np.float32)
            eps0[pidx] = 0.0
        else:
            pidx = pval = gprev = None
        seg_end, seg_k = _random_layers(rng, d, 4)
        a, s = api.scores(g, eps0, pidx, pval, gprev, 2.0, 0.5)
        eps = eps0.copy()
        idx, val = api.worker_step_layered(g, eps, seg_end, seg_k, pidx, pval, gprev, 2.0, 0.5)
        want = []
        begin = 0
        for end, kl in zip(seg_end, seg_k):
            best = None
            for sub in itertools.combinations(range(begin, int(end)), int(kl)):
                key = (tuple(sorted((-float(s[j]) for j in sub))), sub)
                if best is None or key < best:
                    best = key
            want += list(best[1])
            begin = int(end)
        assert [int(i) for i in idx] == want, (d, seg_end, seg_k, s, idx, want)
        assert np.array_equal(val, a[idx])
        expect_eps = a.copy()
        expect_eps[idx] = 0.0
        assert np.array_equal(eps.view(np.uint32), expect_eps.view(np.uint32))


def pin_layered_special_cases(api):
    """(i) One layer covering everything is the global selector.  (ii) k_l equal to the layer's size sends the whole
    layer.  (iii) A layer's mask depends only on that layer's scores: it equals Algorithm 1 (independent numpy
    Top-k) applied to the layer's slice alone, in round 0, for several rounds of error feedback with mu = 0."""
    rng = np.random.default_rng(23)
    d, N = 300, 2
    rounds = [np.round(rng.standard_normal((N, d)) * 8).astype(np.float32) / 8 for _ in range(5)]  # ties included
    # (i)
    G = OracleRegTopK(d, N, 37, 4.0, api=api)
    L1 = OracleRegTopK(d, N, 0, 4.0, api=api, layers=([d], [37]))
    for g in rounds:
        ig, vg = G.worker_step(g)
        il, vl = L1.worker_step(g)
        assert np.array_equal(ig, il) and np.array_equal(vg, vl) and np.array_equal(G.eps, L1.eps)
        assert np.array_equal(G.aggregate(), L1.aggregate())
    # (ii) and (iii)
    seg_end = np.array([40, 41, 170, 300], np.int64)
    seg_k = np.array([40, 1, 13, 7], np.int64)
    omega = np.full(N, 0.5, np.float32)
    refs = []
    begin = 0
    for end, kl in zip(seg_end, seg_k):
        refs.append(topk_error_feedback_numpy([g[:, begin:end] for g in rounds], int(kl), omega))
        begin = int(end)
    O = OracleRegTopK(d, N, 0, 0.0, omega=omega, api=api, layers=(seg_end, seg_k))
    for t, g in enumerate(rounds):
        idx, val = O.worker_step(g)
        agg = O.aggregate()
        assert np.array_equal(idx[:, :40], np.tile(np.arange(40, dtype=np.int32), (N, 1)))  # (ii)
        begin, col = 0, 0
        for l, (end, kl) in enumerate(zip(seg_end, seg_k)):
            ri, rv, reps, ragg = refs[l][t]
            assert np.array_equal(idx[:, col:col + kl] - begin, ri), (t, l)
            assert np.array_equal(val[:, col:col + kl], rv)
            assert np.array_equal(O.eps[:, begin:end], reps)
            assert np.array_equal(agg[begin:end], ragg)
            begin, col = int(end), col + int(kl)


def pin_layered_rejects_bad_tables(api):
    g = np.ones(10, np.float32)
    for seg_end, seg_k in (([5, 9], [1, 1]), ([5, 5, 10], [1, 1, 1]), ([4, 10], [5, 1]), ([4, 10], [0, 1]), ([10, 4], [1, 1])):
        try:
            api.worker_step_layered(g, np.zeros(10, np.float32), seg_end, seg_k, None, None, None, 4.0, 0.5)
        except ValueError:
            continue
        raise AssertionError(f"layer table {seg_end} / {seg_k} was accepted")


ALL_PINS = [pin_layered_bruteforce, pin_layered_special_cases, pin_layered_rejects_bad_tables, pin_tanh, pin_bruteforce_selector, pin_dense_passthrough, pin_reduces_to_topk,
            pin_error_feedback_identity, pin_toy_example, pin_table1_iteration1, pin_distortion_cases,
            pin_regularised_ranking, pin_aggregation, pin_pow, pin_exponent_variant, pin_model_update, pin_bf16_gradients, pin_select_modes_agree,
            pin_mask_certificate]
