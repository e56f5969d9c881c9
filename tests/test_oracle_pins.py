"""Pins for the CPU oracle: each check ties it to something other than itself - brute force on
tiny inputs, hand-worked traces, closed forms, invariants the paper states, exact rational sums."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from oracle import BLOCKSIGN, TOPK, Oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
PAPER = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8)  # Section 5.1 defaults
# the same hyper-parameters as the fp32 numbers the method actually holds, for closed forms in double
LR, B1, B2, EPS = (float(np.float32(x)) for x in (1e-3, 0.9, 0.999, 1e-8))


def key(x):
    return np.asarray(x, dtype=np.float32).view(np.uint32) & np.uint32(0x7FFFFFFF)


# ---------------------------------------------------------------- Definition 1 (Top-k)

def brute_force_topk(x, k):
    """k times: take the largest remaining magnitude, the lowest index among equals."""
    mags = [abs(float(v)) for v in x]
    left = set(range(len(x)))
    kept = set()
    for _ in range(k):
        best = None
        for j in sorted(left):
            if best is None or mags[j] > mags[best]:
                best = j
        kept.add(best)
        left.remove(best)
    return kept


@pytest.mark.parametrize("seed", range(40))
def test_topk_matches_brute_force_with_many_ties(seed):
    rng = np.random.default_rng(seed)
    d = int(rng.integers(1, 65))
    # a small integer alphabet so that equal magnitudes (and +-0) are everywhere
    x = rng.integers(-3, 4, size=d).astype(np.float32)
    x[rng.random(d) < 0.2] *= np.float32(-1.0)  # turns some 0 into -0
    k = int(rng.integers(1, d + 1))
    mask = oracle.topk_keep_mask(x, k)
    assert set(np.flatnonzero(mask)) == brute_force_topk(x, k)


def test_topk_worked_examples():
    # |3| occurs at 0 and 3: k=1 keeps the lower index, k=2 keeps both.
    x = np.array([3, -1, 2, -3], dtype=np.float32)
    assert list(np.flatnonzero(oracle.topk_keep_mask(x, 1))) == [0]
    assert list(np.flatnonzero(oracle.topk_keep_mask(x, 2))) == [0, 3]
    assert list(np.flatnonzero(oracle.topk_keep_mask(x, 3))) == [0, 2, 3]
    # all equal (including signed zeros): the first k indices
    z = np.array([0.0, -0.0, 0.0, -0.0, 0.0], dtype=np.float32)
    assert list(np.flatnonzero(oracle.topk_keep_mask(z, 2))) == [0, 1]
    # subnormals order below normals and above zero
    s = np.array([1e-45, 0.0, 1e-38, -1e-40], dtype=np.float32)
    assert list(np.flatnonzero(oracle.topk_keep_mask(s, 3))) == [0, 2, 3]


@pytest.mark.parametrize("seed", range(6))
def test_topk_set_properties_random_floats(seed):
    rng = np.random.default_rng(100 + seed)
    d = int(rng.integers(1000, 60000))
    x = rng.standard_normal(d).astype(np.float32)
    x[rng.random(d) < 0.05] = 0.0
    x[: d // 7] = np.round(x[: d // 7], 1)  # duplicated magnitudes
    k = int(rng.integers(1, d))
    mask = oracle.topk_keep_mask(x, k)
    assert mask.sum() == k
    kk = key(x)
    tau = kk[mask].min()
    assert kk[~mask].max() <= tau
    # ties at the threshold: kept ones come first in index order
    tie_kept = np.flatnonzero(mask & (kk == tau))
    tie_left = np.flatnonzero(~mask & (kk == tau))
    if tie_left.size:
        assert tie_kept.max() < tie_left.min()
    # against a stable full sort (numpy): magnitude descending, index ascending
    order = np.lexsort((np.arange(d), -kk.astype(np.int64)))
    assert set(order[:k]) == set(np.flatnonzero(mask))


def test_kept_per_block_counts():
    assert oracle.kept_per_block(0.01, 65536) == 655          # config 1 states k = 655
    assert oracle.kept_per_block(0.01, 64) == 1               # clamp to at least one entry
    assert oracle.kept_per_block(1.0, 12345) == 12345
    assert oracle.kept_per_block(0.001, 11173962) == 11173
    assert oracle.kept_per_block(0.01, 11173962) == 111739
    assert oracle.kept_per_block(0.5, 1) == 1
    from paper_2205_05632_b200 import workloads as W
    sizes = [W.numel(s) for s in W.resnet50_imagenet_shapes()]
    assert sum(max(1, (s * 1) // 100) for s in sizes) == sum(oracle.kept_per_block(0.01, s) for s in sizes)


# ---------------------------------------------------------------- Definition 2 (Block-Sign)

def exact_scale(x):
    """||x||_1 / len in exact rational arithmetic, rounded to the nearest fp32."""
    S = sum(Fraction(abs(float(v))) for v in x)
    q = S / len(x)
    f = np.float32(float(q))
    # float(q) is correctly rounded to binary64; check the fp32 neighbours to exclude double rounding
    cands = [f, np.nextafter(f, np.float32(np.inf)), np.nextafter(f, np.float32(-np.inf))]
    return min(cands, key=lambda c: abs(Fraction(float(c)) - q))


@pytest.mark.parametrize("seed", range(8))
def test_blocksign_scale_is_exactly_rounded_mean_magnitude(seed):
    rng = np.random.default_rng(200 + seed)
    d = int(rng.integers(1, 4000))
    x = rng.standard_normal(d).astype(np.float32)
    if seed % 2:
        # magnitudes spread over 60 binades: a plain fp32 or fp64 running sum would lose the small ones
        x *= np.exp2(rng.integers(-30, 30, size=d)).astype(np.float32)
    assert oracle.blocksign_scale(x) == exact_scale(x)


def test_blocksign_scale_special_values():
    assert oracle.blocksign_scale(np.array([1, -2, 3, -2], dtype=np.float32)) == np.float32(2.0)
    assert oracle.blocksign_scale(np.zeros(7, dtype=np.float32)) == np.float32(0.0)
    tiny = np.full(3, 1e-45, dtype=np.float32)  # subnormal: mean of three equal values is the value
    assert oracle.blocksign_scale(tiny) == tiny[0]
    # 2^24 + 1 is not an fp32 number: the exact mean of {2^24, 1, 0, 0} is 4194304.25
    x = np.array([2.0 ** 24, 1.0, 0.0, 0.0], dtype=np.float32)
    assert oracle.blocksign_scale(x) == np.float32(4194304.25)
    big = np.full(1 << 20, 0.1, dtype=np.float32)  # a running fp32 sum drifts here; the mean must be 0.1f exactly
    assert oracle.blocksign_scale(big) == np.float32(0.1)


def run_one_step(comp, G, offsets, k_ratio=1.0, theta=None, **hp):
    n, d = G.shape
    hp = {**PAPER, **hp}
    o = Oracle(n, d, offsets, comp, k_ratio, **hp)
    theta = np.zeros(d, dtype=np.float32) if theta is None else theta.copy()
    o.step(G, theta)
    return o, theta


def test_blocksign_preserves_block_l1_and_signs():
    rng = np.random.default_rng(7)
    offsets = [0, 1, 11, 75, 1000, 5000]
    d = offsets[-1]
    G = rng.standard_normal((3, d)).astype(np.float32)
    G[0, 20] = 0.0
    G[0, 21] = -0.0
    o, _ = run_one_step(BLOCKSIGN, G, offsets)
    C, S = o.buffer("C"), o.buffer("scales")
    X = G + np.zeros_like(G)  # x = g + e with e = +0: IEEE turns g = -0 into x = +0
    assert np.array_equal(np.signbit(C), np.signbit(X))  # the sign bit of x decides; sign(+0) = +
    assert not np.signbit(C[0, 20]) and not np.signbit(C[0, 21])
    for i in range(3):
        for b in range(len(offsets) - 1):
            lo, hi = offsets[b], offsets[b + 1]
            assert np.all(np.abs(C[i, lo:hi]) == S[i, b])
            l1 = math.fsum(abs(float(v)) for v in G[i, lo:hi])
            assert abs(float(S[i, b]) * (hi - lo) - l1) <= 2.0 ** -23 * l1
    # blocks of one element: q = 0, the compressor is the identity (Remark 1 with d_i = 1)
    assert C[0, 0] == G[0, 0]


def test_blocksign_all_blocks_of_size_one_is_identity():
    rng = np.random.default_rng(8)
    d = 33
    G = rng.standard_normal((2, d)).astype(np.float32)
    o, _ = run_one_step(BLOCKSIGN, G, list(range(d + 1)))
    assert np.array_equal(o.buffer("C"), G)
    assert not o.buffer("E").any()


# ---------------------------------------------------------------- Assumption 1 / Remark 1

@pytest.mark.parametrize("comp", [TOPK, BLOCKSIGN])
def test_q_deviate_bound(comp):
    rng = np.random.default_rng(9)
    offsets = [0, 10, 300, 4096]
    d = offsets[-1]
    G = (rng.standard_t(3, size=(4, d)) * 0.1).astype(np.float32)
    ratio = 0.05
    o, _ = run_one_step(comp, G, offsets, ratio)
    C = o.buffer("C").astype(np.float64)
    X = G.astype(np.float64)
    for i in range(4):
        for b in range(3):
            lo, hi = offsets[b], offsets[b + 1]
            db = hi - lo
            q2 = 1 - oracle.kept_per_block(ratio, db) / db if comp == TOPK else 1 - 1 / db
            err = np.sum((C[i, lo:hi] - X[i, lo:hi]) ** 2)
            assert err <= q2 * np.sum(X[i, lo:hi] ** 2) * (1 + 1e-6)


# ---------------------------------------------------------------- error feedback (Algorithm 2, the corrected-gradient and residual steps)

@pytest.mark.parametrize("comp", [TOPK, BLOCKSIGN])
def test_error_feedback_conservation_over_steps(comp):
    rng = np.random.default_rng(10)
    offsets = [0, 64, 1000, 3000]
    n, d = 3, offsets[-1]
    o = Oracle(n, d, offsets, comp, 0.02, **PAPER)
    theta = np.zeros(d, dtype=np.float32)
    E_prev = np.zeros((n, d), dtype=np.float32)
    for _ in range(5):
        G = rng.standard_normal((n, d)).astype(np.float32)
        o.step(G, theta)
        X = G + E_prev  # one fp32 addition
        C, E = o.buffer("C"), o.buffer("E")
        if comp == TOPK:
            # g~ + e_{t+1} = g + e_t, bit for bit (kept: x + 0, dropped: 0 + x)
            assert np.array_equal((C + E).view(np.uint32) & 0x7FFFFFFF, X.view(np.uint32) & 0x7FFFFFFF)
            assert np.array_equal(C + E, X)
            kept = C != 0
            assert np.array_equal(C[kept], X[kept]) and not E[kept].any()
        else:
            resid = np.abs(C.astype(np.float64) + E.astype(np.float64) - X.astype(np.float64))
            assert np.all(resid <= 2.0 ** -24 * np.abs(X.astype(np.float64) - C.astype(np.float64)))
        E_prev = E.copy()


def test_error_accumulates_until_sent():
    # a coordinate never in the top-1 keeps adding up; once it wins it is sent whole and e resets
    o = Oracle(1, 3, [0, 3], TOPK, 1 / 3, **PAPER)
    theta = np.zeros(3, dtype=np.float32)
    G = np.array([[1.0, 0.75, 0.0]], dtype=np.float32)
    o.step(G, theta)
    assert list(o.buffer("E")[0]) == [0.0, 0.75, 0.0]
    o.step(G, theta)  # x = [1, 1.5, 0] -> coordinate 1 wins with its accumulated value
    assert list(o.buffer("C")[0]) == [0.0, 1.5, 0.0]
    assert list(o.buffer("E")[0]) == [1.0, 0.0, 0.0]


# ---------------------------------------------------------------- Algorithm 1 (AMSGrad)

def test_amsgrad_first_step_closed_form():
    rng = np.random.default_rng(11)
    d = 1000
    g = rng.standard_normal(d).astype(np.float32)
    g[:10] = [0.0, 1e-6, -1e-6, 1e-3, -1e-3, 1.0, -1.0, 100.0, -100.0, 1e-20]
    theta0 = rng.standard_normal(d).astype(np.float32)
    m, v, vh = (np.zeros(d, np.float32) for _ in range(3))
    th = theta0.copy()
    oracle.amsgrad(g, m, v, vh, th, **PAPER)
    g64 = g.astype(np.float64)
    np.testing.assert_allclose(m, (1 - B1) * g64, rtol=1e-6, atol=1e-37)
    np.testing.assert_allclose(v, (1 - B2) * g64 ** 2, rtol=1e-6, atol=1e-37)
    np.testing.assert_array_equal(vh, v)
    # eps sits under the root: for |g| = 1e-6 the step is lr*(1-b1)*g/sqrt(eps) ~ 1e-6, not ~2e-3
    expect = theta0.astype(np.float64) - LR * (1 - B1) * g64 / np.sqrt((1 - B2) * g64 ** 2 + EPS)
    np.testing.assert_allclose(th, expect, rtol=1e-6, atol=1e-7)
    assert th[0] == theta0[0]  # zero gradient at t = 1: no move
    assert abs((theta0[1] - th[1]) - 1e-6) < 2e-7


def test_amsgrad_sign_descent_when_eps_is_zero():
    # eps = 0, t = 1: theta moves by lr (1-b1)/sqrt(1-b2) sign(g) whatever |g| is
    g = np.array([3.0, -0.02, 500.0], dtype=np.float32)
    m, v, vh, th = (np.zeros(3, np.float32) for _ in range(4))
    oracle.amsgrad(g, m, v, vh, th, lr=1e-3, beta1=0.9, beta2=0.999, eps=0.0)
    np.testing.assert_allclose(th, -np.sign(g) * LR * (1 - B1) / math.sqrt(1 - B2), rtol=1e-6)


def test_amsgrad_constant_gradient_geometric_closed_form():
    # constant g: m_T = (1-b1^T) g, v_T = (1-b2^T) g^2 (increasing, so vhat_T = v_T),
    # theta_{T+1} = theta_1 - lr * sum_t (1-b1^t) g / sqrt((1-b2^t) g^2 + eps)
    g = np.array([0.5, -2.0, 1e-3], dtype=np.float32)
    m, v, vh, th = (np.zeros(3, np.float32) for _ in range(4))
    T = 25
    for _ in range(T):
        oracle.amsgrad(g, m, v, vh, th, **PAPER)
    g64 = g.astype(np.float64)
    np.testing.assert_allclose(m, (1 - B1 ** T) * g64, rtol=2e-6)
    np.testing.assert_allclose(v, (1 - B2 ** T) * g64 ** 2, rtol=2e-6)
    np.testing.assert_array_equal(vh, v)
    tot = sum((1 - B1 ** t) * g64 / np.sqrt((1 - B2 ** t) * g64 ** 2 + EPS) for t in range(1, T + 1))
    np.testing.assert_allclose(th, -LR * tot, rtol=2e-6)


def test_amsgrad_vhat_holds_the_running_maximum():
    g1 = np.array([-4.0], dtype=np.float32)
    g2 = np.array([0.0], dtype=np.float32)
    m, v, vh, th = (np.zeros(1, np.float32) for _ in range(4))
    oracle.amsgrad(g1, m, v, vh, th, lr=3.0, beta1=0.5, beta2=0.5, eps=7.0)
    assert (m[0], v[0], vh[0]) == (-2.0, 8.0, 8.0)
    assert abs(th[0] - 6 / math.sqrt(15)) < 1e-6
    oracle.amsgrad(g2, m, v, vh, th, lr=3.0, beta1=0.5, beta2=0.5, eps=7.0)
    assert (m[0], v[0], vh[0]) == (-1.0, 4.0, 8.0)  # v fell, vhat did not
    assert abs(th[0] - 9 / math.sqrt(15)) < 1e-6


# ---------------------------------------------------------------- hand-worked traces of Algorithm 2

def test_learning_rate_schedule_closed_form():
    # Algorithm 2 with eta_t varying: a constant gradient g on one coordinate, k = d, one worker. Then
    # m_t = (1 - b1^t) g, v_t = (1 - b2^t) g^2 (increasing, so vhat_t = v_t) and
    # theta_{T+1} = theta_1 - sum_t eta_t m_t / sqrt(v_t + eps): every eta_t enters exactly one term, with
    # that step's moments. A schedule applied one step late or early, or only the first eta, changes the sum.
    b1, b2, eps, g = B1, B2, EPS, float(np.float32(0.37))  # the fp32 values the oracle computes with
    etas = [float(np.float32(x)) for x in (1e-3, 1e-3, 1e-4, 5e-2, 1e-5, 2e-3)]
    o = Oracle(1, 1, [0, 1], TOPK, 1.0, lr=etas[0], beta1=0.9, beta2=0.999, eps=1e-8)
    theta = np.array([0.25], dtype=np.float32)
    want = 0.25
    for t, eta in enumerate(etas, start=1):
        o.set_lr(eta)
        o.step(np.array([[g]], dtype=np.float32), theta)
        m = (1 - b1 ** t) * g
        v = (1 - b2 ** t) * g * g
        want -= eta * m / math.sqrt(v + eps)
        assert abs(float(theta[0]) - want) <= 2e-6 * 0.25  # fp32 roundings of values up to theta_1 = 0.25
    # the late and the early schedule are far outside that tolerance: the pin discriminates
    late = 0.25 - sum(e * (1 - b1 ** t) * g / math.sqrt((1 - b2 ** t) * g * g + eps)
                      for t, e in enumerate([etas[0]] + etas[:-1], start=1))
    assert abs(late - want) > 1e-3
    o.close()


def read_trace(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, val = line.split(":", 1)
            out[k.strip()] = [[float(t) for t in part.split()] for part in val.split("|")]
    return out


@pytest.mark.parametrize("name,comp", [("alg2_topk_trace.txt", TOPK), ("alg2_blocksign_trace.txt", BLOCKSIGN)])
def test_algorithm2_hand_worked_trace(name, comp):
    t = read_trace(name)
    n, d = int(t["n"][0][0]), int(t["d"][0][0])
    offsets = [int(v) for v in t["block_offsets"][0]]
    o = Oracle(n, d, offsets, comp, t["k_ratio"][0][0], lr=t["lr"][0][0], beta1=t["beta1"][0][0],
               beta2=t["beta2"][0][0], eps=t["eps"][0][0])
    theta = np.array(t["theta0"][0], dtype=np.float32)
    for s in (1, 2):
        G = np.array(t["step%d.g" % s], dtype=np.float32)
        o.step(G, theta)
        np.testing.assert_array_equal(o.buffer("E"), np.array(t["step%d.e" % s], dtype=np.float32))
        np.testing.assert_array_equal(o.buffer("gbar"), np.array(t["step%d.gbar" % s][0], dtype=np.float32))
        np.testing.assert_array_equal(o.buffer("m"), np.array(t["step%d.m" % s][0], dtype=np.float32))
        np.testing.assert_array_equal(o.buffer("v"), np.array(t["step%d.v" % s][0], dtype=np.float32))
        np.testing.assert_array_equal(o.buffer("vhat"), np.array(t["step%d.vhat" % s][0], dtype=np.float32))
        np.testing.assert_allclose(theta, np.array(t["step%d.theta" % s][0]), rtol=1e-6, atol=1e-7)
        if comp == TOPK:
            kept = [[int(v) for v in row] for row in t["step%d.kept" % s]]
            assert o.buffer("kept_idx").tolist() == kept
        else:
            np.testing.assert_array_equal(o.buffer("scales"), np.array(t["step%d.scales" % s], dtype=np.float32))
            signs = np.array(t["step%d.signs" % s]).astype(bool)
            np.testing.assert_array_equal(np.signbit(o.buffer("C")), signs)


# ---------------------------------------------------------------- reductions to simpler algorithms

def test_k_equal_d_is_plain_amsgrad_on_the_mean_gradient():
    # q = 0 (no compression): Algorithm 2 must collapse to Algorithm 1 run on mean_i g_i
    rng = np.random.default_rng(12)
    n, d = 4, 777
    o = Oracle(n, d, [0, 100, d], TOPK, 1.0, **PAPER)
    theta = rng.standard_normal(d).astype(np.float32)
    m, v, vh = (np.zeros(d, np.float32) for _ in range(3))
    th = theta.copy()
    for _ in range(4):
        G = rng.standard_normal((n, d)).astype(np.float32)
        o.step(G, theta)
        assert not o.buffer("E").any()
        gmean = (G.astype(np.float64).sum(axis=0)).astype(np.float32) / np.float32(n)
        oracle.amsgrad(gmean, m, v, vh, th, **PAPER)
        np.testing.assert_array_equal(theta, th)
        np.testing.assert_array_equal(o.buffer("m"), m)


def test_single_worker_average_is_the_compressed_gradient():
    rng = np.random.default_rng(13)
    G = rng.standard_normal((1, 500)).astype(np.float32)
    for comp in (TOPK, BLOCKSIGN):
        o, _ = run_one_step(comp, G, [0, 200, 500], 0.1)
        np.testing.assert_array_equal(o.buffer("gbar"), o.buffer("C")[0])


def test_average_is_invariant_under_worker_permutation_and_replication():
    rng = np.random.default_rng(14)
    n, d = 8, 2000
    G = rng.standard_normal((n, d)).astype(np.float32)
    perm = rng.permutation(n)
    for comp in (TOPK, BLOCKSIGN):
        a, ta = run_one_step(comp, G, [0, 512, d], 0.3)
        b, tb = run_one_step(comp, G[perm].copy(), [0, 512, d], 0.3)
        np.testing.assert_array_equal(a.buffer("gbar"), b.buffer("gbar"))
        np.testing.assert_array_equal(ta, tb)
        # n identical workers: the mean of n copies is the copy (n a power of two: exact)
        same = np.repeat(G[:1], n, axis=0).copy()
        c, _ = run_one_step(comp, same, [0, 512, d], 0.3)
        np.testing.assert_array_equal(c.buffer("gbar"), c.buffer("C")[0])


def test_unsent_coordinates_still_move_with_momentum():
    # Algorithm 2 is dense at the server: gbar_j = 0 decays m and v, holds vhat, and theta still moves
    o = Oracle(1, 2, [0, 2], TOPK, 0.5, **PAPER)
    theta = np.zeros(2, dtype=np.float32)
    o.step(np.array([[1.0, 0.0]], dtype=np.float32), theta)
    t1 = theta.copy()
    o.step(np.array([[0.0, 2.0]], dtype=np.float32), theta)  # now coordinate 1 is sent, 0 is not
    assert o.buffer("gbar")[0] == 0.0
    assert abs(float(o.buffer("m")[0]) - B1 * (1 - B1)) < 1e-8
    assert abs(float(o.buffer("v")[0]) - B2 * (1 - B2)) < 1e-9
    assert abs(float(o.buffer("vhat")[0]) - (1 - B2)) < 1e-10
    assert theta[0] < t1[0] < 0


# ---------------------------------------------------------------- Lemmas 2, 4, 5

@pytest.mark.parametrize("comp", [TOPK, BLOCKSIGN])
def test_lemma_bounds_and_monotone_vhat(comp):
    rng = np.random.default_rng(15)
    n, d, ratio = 4, 1024, 0.25
    offsets = [0, 256, d]
    o = Oracle(n, d, offsets, comp, ratio, **PAPER)
    theta = np.zeros(d, dtype=np.float32)
    q2 = (1 - ratio) if comp == TOPK else (1 - 1 / 256)
    Gmax2 = 0.0
    vh_prev = np.zeros(d, dtype=np.float32)
    for _ in range(10):
        G = rng.standard_normal((n, d)).astype(np.float32)
        Gmax2 = max(Gmax2, float((G.astype(np.float64) ** 2).sum(axis=1).max()))
        o.step(G, theta)
        vh = o.buffer("vhat").copy()
        assert np.all(vh >= vh_prev) and np.all(vh >= o.buffer("v"))            # Lemma 5: vhat non-decreasing
        vh_prev = vh
        e2 = (o.buffer("E").astype(np.float64) ** 2).sum(axis=1).max()
        assert e2 <= 4 * q2 / (1 - q2) ** 2 * Gmax2                              # Lemma 2
        assert vh.max() <= 4 * (1 + q2) ** 3 / (1 - q2) ** 2 * Gmax2             # Lemma 4


# ---------------------------------------------------------------- Random-k (Section 2.1 names it; the index rule is this build's reading)

def test_philox4x64_matches_an_independent_library_implementation():
    # numpy's Philox bit generator is Philox4x64-10; it advances its counter by one before it produces its
    # first block, so its first four raw outputs are the block at counter + 1
    rng = np.random.default_rng(31)
    for _ in range(20):
        ctr = [int(x) for x in rng.integers(0, 2 ** 63, size=4)]
        key = [int(x) for x in rng.integers(0, 2 ** 63, size=2)]
        want = np.random.Philox(counter=ctr, key=key).random_raw(4)
        got = oracle.philox4x64_10([ctr[0] + 1] + ctr[1:], key)
        assert np.array_equal(got, want)
    # counter and key words all play a part: changing any one changes the block
    base = oracle.philox4x64_10([1, 2, 3, 4], [5, 6])
    for pos in range(4):
        c = [1, 2, 3, 4]
        c[pos] += 1
        assert not np.array_equal(oracle.philox4x64_10(c, [5, 6]), base)
    assert not np.array_equal(oracle.philox4x64_10([1, 2, 3, 4], [6, 6]), base)
    assert not np.array_equal(oracle.philox4x64_10([1, 2, 3, 4], [5, 7]), base)


@pytest.mark.parametrize("m", [1, 2, 3, 4, 5, 7, 16, 17, 63, 64, 65, 100, 255, 256, 257, 1000, 4097])
def test_randk_index_map_is_a_bijection(m):
    for seed, step, worker, block in ((0, 1, 0, 0), (7, 3, 2, 5), (2 ** 40 + 1, 1000, 31, 160)):
        image = sorted(oracle.randk_permute(m, r, seed, step, worker, block) for r in range(m))
        assert image == list(range(m))


def test_randk_sets_have_k_distinct_members_and_depend_on_every_identifier():
    m, k = 5000, 50
    base = oracle.randk_keep_mask(m, k, 3, 1, 0, 0)
    assert base.sum() == k
    assert np.array_equal(base, oracle.randk_keep_mask(m, k, 3, 1, 0, 0))  # same identifiers, same set
    for other in ((4, 1, 0, 0), (3, 2, 0, 0), (3, 1, 1, 0), (3, 1, 0, 1)):
        assert not np.array_equal(base, oracle.randk_keep_mask(m, k, *other))
    # nested in k: the first k images of the permutation
    assert np.all(oracle.randk_keep_mask(m, 20, 3, 1, 0, 0) <= base)
    assert oracle.randk_keep_mask(m, m, 3, 1, 0, 0).all()


def test_randk_inclusion_frequencies_are_uniform():
    # over many steps every coordinate is kept about N k / m times: chi-square over the m coordinates against
    # the hypergeometric variance N (k/m)(1 - k/m); 49 degrees of freedom put 99.99 % of the mass below 95.
    # The first image pi(0) alone is uniform too.
    m, k, N = 50, 5, 20000
    counts = np.zeros(m)
    first = np.zeros(m)
    for step in range(1, N + 1):
        counts += oracle.randk_keep_mask(m, k, 12345, step, 0, 0)
        first[oracle.randk_permute(m, 0, 12345, step, 0, 0)] += 1
    p = k / m
    chi2 = float(((counts - N * p) ** 2).sum() / (N * p * (1 - p)))
    assert chi2 < 95.0, chi2
    chi2_first = float(((first - N / m) ** 2).sum() / (N / m))
    assert chi2_first < 95.0, chi2_first
    # pairs: coordinates 0 and 1 are kept together about N k (k-1) / (m (m-1)) times (no pairing by position)
    both = sum(1 for step in range(1, 4001) if oracle.randk_keep_mask(m, k, 99, step, 0, 0)[:2].all())
    expect = 4000 * k * (k - 1) / (m * (m - 1))
    assert abs(both - expect) < 6 * math.sqrt(expect) + 1


def test_randk_step_keeps_the_drawn_coordinates_and_conserves_the_error():
    from oracle import RANDK
    rng = np.random.default_rng(41)
    offsets = [0, 64, 1000, 3000]
    n, d, ratio, seed = 3, offsets[-1], 0.02, 77
    o = Oracle(n, d, offsets, RANDK, ratio, **PAPER)
    o.set_seed(seed)
    theta = np.zeros(d, dtype=np.float32)
    E_prev = np.zeros((n, d), dtype=np.float32)
    for t in range(1, 5):
        G = rng.standard_normal((n, d)).astype(np.float32)
        o.step(G, theta)
        X = G + E_prev
        C, E = o.buffer("C").copy(), o.buffer("E").copy()
        keep = np.zeros((n, d), dtype=bool)
        for i in range(n):
            for b in range(3):
                lo, hi = offsets[b], offsets[b + 1]
                keep[i, lo:hi] = oracle.randk_keep_mask(hi - lo, oracle.kept_per_block(ratio, hi - lo), seed, t, i, b)
        assert np.array_equal(C, np.where(keep, X, np.float32(0)))          # g~ = x on the drawn set, 0 elsewhere
        assert np.array_equal(E, np.where(keep, np.float32(0), X))          # e_{t+1} = x - g~
        assert np.array_equal(o.buffer("kept_idx"), np.stack([np.flatnonzero(keep[i]) for i in range(n)]))
        gbar = (C.astype(np.float64).sum(axis=0)).astype(np.float32) / np.float32(n)
        assert np.array_equal(o.buffer("gbar"), gbar)
        E_prev = E
    o.close()
    # k = d: every coordinate is drawn, the step is Algorithm 1 on the mean gradient
    a = Oracle(2, 100, [0, 100], RANDK, 1.0, **PAPER)
    b = Oracle(2, 100, [0, 100], TOPK, 1.0, **PAPER)
    ta, tb = np.zeros(100, np.float32), np.zeros(100, np.float32)
    G = rng.standard_normal((2, 100)).astype(np.float32)
    a.step(G, ta)
    b.step(G, tb)
    assert np.array_equal(ta, tb) and not a.buffer("E").any()
