"""CPU pins of the oracle: worked values, closed forms, invariants, brute force
and library special cases.  None of these tests touches the CUDA library."""
import itertools
import math

import numpy as np
import pytest
import scipy.spatial.distance
import scipy.stats

import oracle
from conftest import read_golden
from paper_2511_18868_b200 import workloads as wl


# ----------------------------------------------------------------- normalise
def test_normalize_worked_column():
    rows = read_golden("zscore.txt")
    x = np.array([[r[0]] for r in rows], np.float32)[None]          # [1,4,1]
    z, mean, scale = oracle.normalize(x)
    assert mean[0, 0] == pytest.approx(2.5, abs=1e-7)
    assert scale[0, 0] == pytest.approx(1.1180340, abs=1e-6)
    np.testing.assert_allclose(z[0, :, 0], [r[1] for r in rows], atol=1e-6)


def test_normalize_matches_scipy_zscore_and_postconditions():
    rng = np.random.default_rng(1)
    x = (rng.standard_normal((3, 500, 7)) * rng.uniform(0.1, 50, 7) + rng.uniform(-100, 100, 7)).astype(np.float32)
    x[:, :, 3] = 4.25                                               # a constant column
    z, mean, scale = oracle.normalize(x)
    for b in range(3):
        ref = scipy.stats.zscore(x[b].astype(np.float64), axis=0, ddof=0)
        ok = np.arange(7) != 3
        np.testing.assert_allclose(z[b][:, ok], ref[:, ok], rtol=1e-5, atol=1e-6)
        assert np.all(z[b][:, 3] == 0.0) and scale[b, 3] == 1.0
        zz = z[b].astype(np.float64)
        assert np.all(np.abs(zz[:, ok].mean(0)) < 1e-6)
        np.testing.assert_allclose(zz[:, ok].var(0), 1.0, atol=1e-5)
    z2, _, _ = oracle.normalize(z)                                   # idempotent
    np.testing.assert_allclose(z2, z, atol=2e-6)


def test_normalize_then_k1_inertia_is_N_times_D():
    # closed form: after z-scoring, one cluster at the mean has inertia N * D
    rng = np.random.default_rng(2)
    x = rng.standard_normal((1, 300, 5)).astype(np.float32) * 3 + 1
    z, _, _ = oracle.normalize(x)
    c, counts = oracle.cluster_update(z, np.zeros((1, 300), np.int32), np.zeros((1, 1, 5), np.float32))
    a = oracle.cluster_assign(z, c)
    assert counts[0, 0] == 300 and np.all(a["labels"] == 0)
    assert a["inertia"][0] == pytest.approx(300 * 5, rel=1e-5)


# --------------------------------------------------------------------- prune
def test_prune_worked_floor_values():
    for F, Q, P, W, tlb in read_golden("roofline_floor.txt"):
        args = dict(flops=[[F]], bytes_=[[Q]], peak_flops=[P], peak_bw=[W])
        # the floor itself is observable through the threshold: kept iff T_lb < T_inc
        assert oracle.prune(t_inc=[tlb * (1 + 1e-4)], **args)["keep"][0, 0] == 1
        assert oracle.prune(t_inc=[tlb * (1 - 1e-4)], **args)["keep"][0, 0] == 0
        # and through the bound: T_k = 2 * T_lb  ->  B = 0.5 ; T_k < T_lb -> 0
        b = oracle.prune(t_inc=[1.0], t_cur=[[2 * tlb]], want_bound=True, **args)["bound"]
        assert b[0, 0, 0] == pytest.approx(0.5, abs=1e-6)
        b = oracle.prune(t_inc=[1.0], t_cur=[[0.5 * tlb]], want_bound=True, **args)["bound"]
        assert b[0, 0, 0] == 0.0


def test_prune_invariants_and_saturation_mask():
    cfg = wl.scaled(wl.CONFIGS["tiny"], N=400, S=13, K=5)
    inp = wl.make_inputs(cfg, seed=3)
    labels = np.random.default_rng(3).integers(0, cfg.K, (1, cfg.N)).astype(np.int32)
    r = oracle.prune(inp["flops"], inp["bytes"], inp["peak_flops"], inp["peak_bw"], inp["t_inc"], inp["t_cur"],
                     labels, inp["hsig"], inp["target"], 75.0, want_bound=True)
    F, Q = inp["flops"].astype(np.float64), inp["bytes"].astype(np.float64)
    P, W = inp["peak_flops"].astype(np.float64), inp["peak_bw"].astype(np.float64)
    tlb = np.maximum(F[..., None] / P, Q[..., None] / W)
    h = inp["hsig"].astype(np.float64)[0][labels[0]][:, inp["target"]][None]
    bits = (r["keep"][..., None] >> np.arange(cfg.S)) & 1
    # every kept arm: both strict inequalities; every pruned arm: at least one fails
    assert np.all((tlb < inp["t_inc"][0])[bits == 1]) and np.all((h < 75.0)[bits == 1])
    assert np.all(((tlb >= inp["t_inc"][0]) | (h >= 75.0))[bits == 0])
    assert r["kept_count"][0] == bits.sum()
    assert np.all(r["keep"] < (1 << cfg.S))
    assert np.all((r["bound"] >= 0) & (r["bound"] <= 1))
    # the incumbent is the 20th-percentile floor: about a fifth passes the roofline test
    roof = oracle.prune(inp["flops"], inp["bytes"], inp["peak_flops"], inp["peak_bw"], inp["t_inc"])
    frac = roof["kept_count"][0] / (cfg.N * cfg.S)
    assert 0.17 < frac < 0.23
    # monotone: raising the incumbent never clears a set bit
    roof2 = oracle.prune(inp["flops"], inp["bytes"], inp["peak_flops"], inp["peak_bw"], inp["t_inc"] * 3)
    assert np.all((roof["keep"] & ~roof2["keep"]) == 0) and roof2["kept_count"][0] > roof["kept_count"][0]
    # saturation threshold is strict: h == theta is pruned
    hs = np.array([[[75.0, 74.999, 80.0]]], np.float32)
    r = oracle.prune([[1.0]], [[1.0]], [1e12] * 3, [1e12] * 3, [1.0], None, [[0]], hs, [0, 1, 2], 75.0)
    assert r["keep"][0, 0] == 0b010


def test_prune_margin_worked_values():
    """The near-tie margin that arbitrates every keep-bit disagreement in the GPU parity tests, by hand.
    Roofline comparison alone, exactly representable inputs: T_lb = max(3/2, 1/4) = 1.5 against
    T_inc = 1.5 (1 + 2^-18): margin = 2^-18 / (1 + 2^-18)."""
    e = 2.0 ** -18
    r = oracle.prune([[3.0]], [[1.0]], [2.0], [4.0], [1.5 * (1 + e)], want_margin=True)
    assert r["keep"][0, 0] == 1 and r["margin"][0, 0, 0] == pytest.approx(e / (1 + e), rel=1e-12)
    r = oracle.prune([[3.0]], [[1.0]], [2.0], [4.0], [1.5 * (1 - e)], want_margin=True)          # pruned side
    assert r["keep"][0, 0] == 0 and r["margin"][0, 0, 0] == pytest.approx(e / (1 - e), rel=1e-12)
    # the golden floor 5e-5 s against an incumbent 3e-6 above it (fp32 rounding of both: 1.2e-7)
    F, Q, P, W, tlb = read_golden("roofline_floor.txt")[0]
    r = oracle.prune([[F]], [[Q]], [P], [W], [tlb * (1 + 3e-6)], want_margin=True)
    assert r["keep"][0, 0] == 1 and r["margin"][0, 0, 0] == pytest.approx(3e-6, abs=2e-7)
    # saturation comparison: 74.9997 % against theta = 75 %: 0.0003 / 75 = 4e-6 (fp32 rounding of h: 5e-8)
    hs = np.array([[[74.9997, 90.0, 60.0]]], np.float32)
    wide = dict(flops=[[1.0]], bytes_=[[1.0]], peak_flops=[1.0] * 3, peak_bw=[1.0] * 3)
    # roofline decisively kept (floor 1 against incumbent 2: margin 0.5): the saturation comparison decides alone
    r = oracle.prune(t_inc=[2.0], labels=[[0]], hsig=hs, target=[0, 1, 2], theta_sat=75.0, want_margin=True, **wide)
    assert r["keep"][0, 0] == 0b101
    np.testing.assert_allclose(r["margin"][0, 0], [4e-6, 0.2, 0.2], atol=1e-7)     # kept: min(0.5, .); pruned by h: 0.2
    # both comparisons pass, the roofline one nearer its threshold: the smaller margin decides
    r = oracle.prune(t_inc=[1.0 + 2.0 ** -19], labels=[[0]], hsig=hs, target=[2, 2, 2], want_margin=True, **wide)
    assert r["keep"][0, 0] == 0b111 and r["margin"][0, 0, 0] == pytest.approx(2.0 ** -19, rel=1e-5)
    # pruned by the roofline comparison alone, by a hair, while h is far below theta: the hair decides
    r = oracle.prune(t_inc=[1.0 - 2.0 ** -19], labels=[[0]], hsig=hs, target=[2, 2, 2], want_margin=True, **wide)
    assert r["keep"][0, 0] == 0 and r["margin"][0, 0, 0] == pytest.approx(2.0 ** -19, rel=1e-5)
    # pruned by BOTH, one by a hair and one decisively (h = 90): no small change keeps it: the larger margin
    r = oracle.prune(t_inc=[1.0 - 2.0 ** -19], labels=[[0]], hsig=hs, target=[1, 1, 1], want_margin=True, **wide)
    assert r["keep"][0, 0] == 0 and r["margin"][0, 0, 0] == pytest.approx(0.2, rel=1e-6)


def test_prune_margin_says_exactly_which_bits_a_small_change_can_flip():
    """What the margin is for: a bit whose margin exceeds delta must survive every change of the two
    thresholds by less than delta (relative); a bit whose margin is below delta must flip under one.  Inputs are
    built so that thousands of comparisons sit within 1e-7 .. 1e-3 of their thresholds, on both sides."""
    rng = np.random.default_rng(11)
    B, N, S, K = 2, 3000, 6, 4
    delta = 1e-5
    t_inc = np.array([3e-4, 7e-3], np.float32)
    eps = np.exp(rng.uniform(np.log(1e-7), np.log(1e-3), (B, N))) * rng.choice([-1.0, 1.0], (B, N))
    pf, pb = np.full(S, 1e12, np.float32), np.full(S, 1e11, np.float32)
    pf[1::2] *= 4.0                                              # odd strategies: a floor 4x lower (decisively kept)
    flops = (t_inc[:, None].astype(np.float64) * (1 + eps) * 1e12).astype(np.float32)
    byts = np.ones((B, N), np.float32)
    far = rng.uniform(size=(B, N)) < 0.3                         # a third of the candidates far above the incumbent
    flops[far] *= 50.0
    labels = rng.integers(0, K, (B, N)).astype(np.int32)
    theta = 75.0
    hs = (theta * (1 + np.exp(rng.uniform(np.log(1e-7), np.log(1e-1), (B, K, 3))) * rng.choice([-1.0, 1.0], (B, K, 3))))
    hs = hs.astype(np.float32)
    target = (np.arange(S) % 3).astype(np.int32)

    def run(ti, th):
        return oracle.prune(flops, byts, pf, pb, ti, None, labels, hs, target, th, want_margin=True)

    nom = run(t_inc, theta)
    bits = lambda r: ((r["keep"][..., None] >> np.arange(S, dtype=np.uint32)) & 1).astype(bool)
    lo = bits(run((t_inc.astype(np.float64) * (1 - delta)).astype(np.float32), theta * (1 - delta)))
    hi = bits(run((t_inc.astype(np.float64) * (1 + delta)).astype(np.float32), theta * (1 + delta)))
    b0, m = bits(nom), nom["margin"]
    flipped = (lo != b0) | (hi != b0)
    safe, frail = m > 1.05 * delta, m < 0.95 * delta
    assert safe.sum() > 10000 and frail.sum() > 500
    assert not np.any(flipped & safe)
    assert np.all(flipped[frail])
    # without the saturation inputs the margin is the roofline comparison's alone
    r = oracle.prune(flops, byts, pf, pb, t_inc, want_margin=True)
    floor = np.maximum(flops.astype(np.float64)[..., None] / pf, byts.astype(np.float64)[..., None] / pb)
    np.testing.assert_allclose(r["margin"], np.abs(floor / t_inc.astype(np.float64)[:, None, None] - 1), rtol=1e-9, atol=1e-15)


# -------------------------------------------------------------------- assign
def test_assign_against_cdist_and_optimality():
    rng = np.random.default_rng(4)
    B, N, D, K = 2, 700, 9, 11
    z = rng.standard_normal((B, N, D)).astype(np.float32)
    c = rng.standard_normal((B, K, D)).astype(np.float32)
    a = oracle.cluster_assign(z, c, want_margins=True)
    for b in range(B):
        d2 = scipy.spatial.distance.cdist(z[b].astype(np.float64), c[b].astype(np.float64), "sqeuclidean")
        assert np.array_equal(a["labels"][b], d2.argmin(1))
        np.testing.assert_allclose(a["dist2"][b], d2.min(1), rtol=1e-6)
        np.testing.assert_allclose(a["best"][b], d2.min(1), rtol=1e-12)
        np.testing.assert_allclose(a["second"][b], np.sort(d2, 1)[:, 1], rtol=1e-12)
        assert a["inertia"][b] == pytest.approx(d2.min(1).sum(), rel=1e-6)
        # representative: the member nearest its centroid
        for i in range(K):
            members = np.flatnonzero(a["labels"][b] == i)
            if len(members) == 0:
                assert a["rep"][b, i] == -1
            else:
                assert a["rep"][b, i] == members[np.argmin(d2[members, i])]
        np.testing.assert_allclose(oracle.dist2_at(z, c, a["labels"])[b], d2.min(1), rtol=1e-12)


def test_assign_special_cases():
    rng = np.random.default_rng(5)
    z = rng.standard_normal((1, 50, 4)).astype(np.float32)
    # K = 1: everything in cluster 0
    assert np.all(oracle.cluster_assign(z, z[:, :1])["labels"] == 0)
    # centroids that are data rows: those rows are at distance 0 with their own label
    rows = np.array([7, 3, 41, 19])
    a = oracle.cluster_assign(z, z[:, rows])
    assert np.array_equal(a["labels"][0, rows], np.arange(4)) and np.all(a["dist2"][0, rows] == 0)
    assert np.array_equal(a["rep"][0], rows)
    # permuting centroids permutes labels
    perm = np.array([2, 0, 3, 1])
    a2 = oracle.cluster_assign(z, z[:, rows[perm]])
    assert np.array_equal(perm[a2["labels"][0]], a["labels"][0])
    # duplicate centroids: the lowest index wins; an unused one is empty
    a3 = oracle.cluster_assign(z, z[:, [7, 7]])
    assert np.all(a3["labels"] == 0) and a3["rep"][0, 1] == -1


def test_lloyd_textbook_1d():
    rows = read_golden("lloyd_1d.txt")
    z = np.array([0, 1, 9, 10], np.float32).reshape(1, 4, 1)
    c = np.array([rows[0][1], rows[0][2]], np.float32).reshape(1, 2, 1)
    for it, c0, c1, l0, l1, l2, l3, inertia in rows:
        np.testing.assert_allclose(c[0, :, 0], [c0, c1], rtol=1e-6)
        a = oracle.cluster_assign(z, c)
        assert list(a["labels"][0]) == [l0, l1, l2, l3]
        assert a["inertia"][0] == pytest.approx(inertia, rel=1e-6)
        c, counts = oracle.cluster_update(z, a["labels"], c)
        assert counts.sum() == 4


def test_lloyd_matches_sklearn_with_fixed_init():
    from sklearn.cluster import KMeans
    cfg = wl.scaled(wl.CONFIGS["medium"], N=1500, D=6, K=7, components=7)
    inp = wl.make_inputs(cfg, seed=6)
    z, _, _ = oracle.normalize(inp["x"])
    c = oracle.init_centroids(z, inp["init_rows"])
    c0 = c.copy()
    iters = 12
    for _ in range(iters):
        a = oracle.cluster_assign(z, c)
        c, counts = oracle.cluster_update(z, a["labels"], c)
    a = oracle.cluster_assign(z, c)
    km = KMeans(n_clusters=cfg.K, init=c0[0].astype(np.float64), n_init=1, max_iter=iters, tol=0.0,
                algorithm="lloyd").fit(z[0].astype(np.float64))
    np.testing.assert_allclose(c[0], km.cluster_centers_, rtol=1e-4, atol=1e-5)
    assert a["inertia"][0] == pytest.approx(km.inertia_, rel=1e-4)
    assert np.mean(a["labels"][0] == km.labels_) > 0.999


# -------------------------------------------------------------------- update
def test_update_is_group_mean():
    rng = np.random.default_rng(7)
    B, N, D, K = 2, 900, 5, 6
    z = rng.standard_normal((B, N, D)).astype(np.float32)
    labels = rng.integers(0, K - 1, (B, N)).astype(np.int32)      # cluster K-1 stays empty
    prev = rng.standard_normal((B, K, D)).astype(np.float32)
    c, counts = oracle.cluster_update(z, labels, prev)
    for b in range(B):
        sums = np.zeros((K, D))
        np.add.at(sums, labels[b], z[b].astype(np.float64))
        cnt = np.bincount(labels[b], minlength=K)
        assert np.array_equal(counts[b], cnt) and cnt.sum() == N
        np.testing.assert_allclose(c[b, :K - 1], sums[:K - 1] / cnt[:K - 1, None], rtol=1e-6, atol=1e-7)
        assert np.array_equal(c[b, K - 1], prev[b, K - 1])         # empty cluster keeps its centroid
        # count-weighted centroids reproduce the column sums of the members
        np.testing.assert_allclose((counts[b, :K - 1, None] * c[b, :K - 1].astype(np.float64)).sum(0),
                                   z[b].astype(np.float64).sum(0), atol=1e-3)


def test_lloyd_objective_never_increases_and_is_a_local_optimum():
    cfg = wl.scaled(wl.CONFIGS["medium"], N=2000, D=8, K=12, components=10)
    inp = wl.make_inputs(cfg, seed=8)
    out = oracle.bandit_step(inp, iters=15)
    tr = out["inertia_trace"][:, 0].astype(np.float64)
    assert np.all(np.diff(tr) <= 1e-6 * tr[:-1])
    assert tr[-1] < 0.5 * tr[0]


def test_lloyd_vs_exhaustive_labelings():
    rng = np.random.default_rng(9)
    N, D, K = 9, 2, 3
    z = rng.standard_normal((1, N, D)).astype(np.float32)
    c = z[:, :K].copy()
    for _ in range(20):
        a = oracle.cluster_assign(z, c)
        c, _ = oracle.cluster_update(z, a["labels"], c)
    a = oracle.cluster_assign(z, c)
    zz = z[0].astype(np.float64)

    def cost(lab):
        tot = 0.0
        for i in range(K):
            m = zz[np.array(lab) == i]
            if len(m):
                tot += ((m - m.mean(0)) ** 2).sum()
        return tot
    best = min(cost(lab) for lab in itertools.product(range(K), repeat=N))
    mine = cost(tuple(a["labels"][0]))
    assert a["inertia"][0] == pytest.approx(mine, rel=1e-5)        # converged: centroids are the member means
    assert mine >= best - 1e-9
    # no single reassignment against the fixed centroids improves the objective
    d2 = scipy.spatial.distance.cdist(zz, c[0].astype(np.float64), "sqeuclidean")
    assert np.all(d2[np.arange(N), a["labels"][0]] <= d2.min(1) + 1e-12)


# ----------------------------------------------------- statistics and index
def _single_cluster_scores(pulls, rewards, t, **kw):
    pulls = np.asarray(pulls, np.int32)
    N, S = pulls.shape
    return oracle.score_select(np.zeros((1, N), np.int32), np.zeros((1, N), np.float32), pulls[None],
                               np.asarray(rewards, np.float32)[None], [t], K=1, **kw)


def test_index_worked_values():
    for t, n, mu, c, u in read_golden("masked_ucb_index.txt"):
        # one cluster, one strategy: N = 1 + pulls, mu = (0.5 + sum r) / N
        pulls = int(n) - 1
        rsum = mu * n - 0.5
        r = _single_cluster_scores([[pulls]], [[rsum]], int(t), c=c)
        assert r["cl_pulls"][0, 0, 0] == n
        assert r["cl_mean"][0, 0, 0] == pytest.approx(mu, abs=1e-6)
        assert r["cl_index"][0, 0, 0] == pytest.approx(u, abs=2e-6)
        # the same number read backwards: ((U - mu) / c)^2 * N = ln t
        assert math.exp(((r["cl_index"][0, 0, 0] - mu) / c) ** 2 * n) == pytest.approx(t, rel=1e-4)


def test_statistics_equal_algorithm1_running_mean():
    for r1, r2, r3, r4, n_fin, mu_fin in read_golden("running_mean.txt"):
        rewards = [r1, r2, r3, r4]
        # pull-by-pull recursion of Algorithm 1, from its initialisation
        n, mu = 1, 0.5
        for r in rewards:
            n += 1
            mu += (r - mu) / n
        assert (n, mu) == (n_fin, pytest.approx(mu_fin, abs=1e-12))
        # the four pulls spread over two member kernels of the same cluster
        out = _single_cluster_scores([[3], [1]], [[r1 + r2 + r3], [r4]], t=1)
        assert out["cl_pulls"][0, 0, 0] == n_fin
        assert out["cl_mean"][0, 0, 0] == pytest.approx(mu_fin, abs=1e-6)
    # random histories: the batch aggregate equals the online recursion
    rng = np.random.default_rng(10)
    N, S, K = 40, 3, 4
    labels = rng.integers(0, K, (1, N)).astype(np.int32)
    pulls = rng.poisson(2.0, (1, N, S)).astype(np.int32)
    per_pull = [[rng.uniform(0, 1, pulls[0, k, s]) for s in range(S)] for k in range(N)]
    rsum = np.array([[per_pull[k][s].sum() for s in range(S)] for k in range(N)], np.float32)[None]
    out = oracle.score_select(labels, np.zeros((1, N), np.float32), pulls, rsum, [5], K=K)
    for i in range(K):
        for s in range(S):
            n, mu = 1, 0.5
            for k in np.flatnonzero(labels[0] == i):
                for r in per_pull[k][s]:
                    n += 1
                    mu += (r - mu) / n
            assert out["cl_pulls"][0, i, s] == n
            assert out["cl_mean"][0, i, s] == pytest.approx(mu, abs=1e-5)
    assert (out["cl_pulls"].sum() - K * S) == pulls.sum()


def test_unplayed_cluster_arms_outrank_played_ones():
    # 3 clusters x 2 strategies; cluster 2 has never been played on strategy 1
    labels = np.array([[0, 0, 1, 1, 2, 2]], np.int32)
    pulls = np.array([[[4, 3], [2, 5], [6, 1], [3, 3], [2, 0], [5, 0]]], np.int32)
    rsum = (pulls * 0.95).astype(np.float32)                      # played arms have a high mean
    out = oracle.score_select(labels, np.zeros((1, 6), np.float32), pulls, rsum, [int(1 + pulls.sum())], K=3)
    assert out["best_cluster_arm"][0] == 2 * 2 + 1
    assert out["cl_pulls"][0, 2, 1] == 1 and out["cl_mean"][0, 2, 1] == 0.5
    # with L = 0 all members of the winning cluster tie: the lowest k wins
    assert out["best_arm"][0] == 4 * 2 + 1
    # index is decreasing in N at fixed mean and increasing in t
    a = _single_cluster_scores([[3]], [[0.5 * 4 - 0.5]], 50)["cl_index"][0, 0, 0]
    b = _single_cluster_scores([[9]], [[0.5 * 10 - 0.5]], 50)["cl_index"][0, 0, 0]
    c = _single_cluster_scores([[3]], [[0.5 * 4 - 0.5]], 500)["cl_index"][0, 0, 0]
    assert b < a < c


def test_select_k1_is_ucb1_and_masks():
    rng = np.random.default_rng(11)
    N, S = 30, 6
    pulls = rng.poisson(3.0, (N, S)).astype(np.int32)
    rsum = (pulls * rng.uniform(0, 1, (N, S))).astype(np.float32)
    t = int(1 + pulls.sum())
    out = _single_cluster_scores(pulls, rsum, t)
    # K = 1, L = 0: plain UCB1 over the S strategies with pooled statistics
    n = 1 + pulls.sum(0)
    mu = (0.5 + rsum.astype(np.float64).sum(0)) / n
    ucb = mu + 2.0 * np.sqrt(np.log(t) / n)
    assert out["best_cluster_arm"][0] == int(np.argmax(ucb))
    assert out["best_arm"][0] == int(np.argmax(ucb))               # k = 0 wins the tie inside the cluster
    np.testing.assert_allclose(out["cl_index"][0, 0], ucb, rtol=1e-6)
    # mask the winner everywhere: the runner-up strategy is chosen
    s_best = int(np.argmax(ucb))
    keep = np.full((1, N), (1 << S) - 1, np.uint32) & ~np.uint32(1 << s_best)
    out2 = _single_cluster_scores(pulls, rsum, t, keep=keep)
    order = np.argsort(-ucb)
    assert out2["best_cluster_arm"][0] == order[1] and out2["best_arm"][0] == order[1]
    assert np.all(np.isneginf(out2["arm_index"][0, :, s_best]))
    # the winner kept only on candidate 17: that arm is chosen
    keep[0, 17] |= np.uint32(1 << s_best)
    out3 = _single_cluster_scores(pulls, rsum, t, keep=keep)
    assert out3["best_arm"][0] == 17 * S + s_best and out3["best_cluster_arm"][0] == s_best
    # everything masked
    out4 = _single_cluster_scores(pulls, rsum, t, keep=np.zeros((1, N), np.uint32))
    assert out4["best_arm"][0] == -1 and np.isneginf(out4["best_val"][0]) and out4["best_cluster_arm"][0] == -1


def test_lipschitz_term_and_bound_cap():
    labels = np.array([[0, 0, 0]], np.int32)
    dist2 = np.array([[0.0, 4.0, 9.0]], np.float32)
    pulls = np.ones((1, 3, 2), np.int32)
    rsum = np.full((1, 3, 2), 0.25, np.float32)
    out = oracle.score_select(labels, dist2, pulls, rsum, [1], K=1, lipschitz_L=0.5)
    base = out["cl_index"][0, 0]
    # t = 1: no exploration bonus, so U(k,s) = mu + L * sqrt(d2)
    np.testing.assert_allclose(out["arm_index"][0], base[None] + 0.5 * np.array([[0.0], [2.0], [3.0]]), rtol=1e-6)
    assert out["best_arm"][0] == 2 * 2 + 0
    bound = np.full((1, 3, 2), 10.0, np.float32)
    bound[0, 2, :] = 0.1
    out = oracle.score_select(labels, dist2, pulls, rsum, [1], K=1, lipschitz_L=0.5, bound=bound, cap_with_bound=True)
    np.testing.assert_allclose(out["arm_index"][0, 2], 0.1, rtol=1e-6)
    assert out["best_arm"][0] == 1 * 2 + 0


def test_select_brute_force_on_tiny_inputs():
    rng = np.random.default_rng(12)
    for trial in range(20):
        N, S, K = 12, 3, 4
        labels = rng.integers(0, K, (1, N)).astype(np.int32)
        dist2 = rng.uniform(0, 4, (1, N)).astype(np.float32)
        pulls = rng.poisson(1.5, (1, N, S)).astype(np.int32)
        rsum = (pulls * rng.uniform(0, 2, (1, N, S))).astype(np.float32)
        keep = rng.integers(0, 1 << S, (1, N)).astype(np.uint32)
        t = int(1 + pulls.sum())
        out = oracle.score_select(labels, dist2, pulls, rsum, [t], K=K, keep=keep, lipschitz_L=0.1)
        # exhaustive evaluation, arm by arm, from the per-cluster sums
        best, arg = -np.inf, -1
        for k in range(N):
            for s in range(S):
                if not (keep[0, k] >> s) & 1:
                    continue
                m = labels[0] == labels[0, k]
                n = 1 + pulls[0, m, s].sum()
                mu = (0.5 + rsum[0, m, s].astype(np.float64).sum()) / n
                u = mu + 2.0 * math.sqrt(math.log(t) / n) + 0.1 * math.sqrt(dist2[0, k])
                if u > best:
                    best, arg = u, k * S + s
        assert out["best_arm"][0] == arg
        assert out["best_val"][0] == pytest.approx(best, rel=1e-6)


# ------------------------------------------------------- initial centroids
def test_init_centroids_is_a_row_gather():
    """C[b][i] = Z[b][rows[b][i]], written out with numpy indexing: several instances (so that the batch
    strides count), rows unsorted and repeated, first and last row, K > N."""
    rng = np.random.default_rng(21)
    B, N, D, K = 3, 37, 5, 41
    z = rng.standard_normal((B, N, D)).astype(np.float32)
    rows = rng.integers(0, N, (B, K)).astype(np.int32)          # unsorted, with repeats (K > N forces them)
    rows[0, :4] = [N - 1, 0, N - 1, 17]
    rows[2, -1] = 0
    c = oracle.init_centroids(z, rows)
    assert c.shape == (B, K, D)
    for b in range(B):
        for i in range(K):
            assert np.array_equal(c[b, i], z[b, rows[b, i]]), (b, i)
    # every value is distinct, so a wrong stride or a swapped (b, i) cannot pass by accident
    z2 = np.arange(B * N * D, dtype=np.float32).reshape(B, N, D)
    c2 = oracle.init_centroids(z2, rows)
    want = (np.arange(B)[:, None, None] * N + rows[:, :, None]) * D + np.arange(D)[None, None, :]
    assert np.array_equal(c2, want.astype(np.float32))
    # a row id outside [0, N) is rejected
    bad = rows.copy()
    bad[1, 3] = N
    with pytest.raises(ValueError):
        oracle.init_centroids(z, bad)
    bad[1, 3] = -2                                                   # (-1 alone names an unused cluster)
    with pytest.raises(ValueError):
        oracle.init_centroids(z, bad)


# ------------------------------------------------------------ input recipes
def test_workload_shapes_and_determinism():
    cfg = wl.CONFIGS["tiny"]
    a, b = wl.make_inputs(cfg), wl.make_inputs(cfg)
    for k in a:
        assert np.array_equal(a[k], b[k])
    assert a["x"].shape == (1, 256, 16) and a["pulls"].shape == (1, 256, 8)
    assert len(set(a["init_rows"][0])) == cfg.K
    assert a["t"][0] == 1 + a["pulls"].sum()
    assert np.all(a["t_cur"] > 0)
    assert wl.CONFIGS["contraction"].arms == 33554432 and wl.CONFIGS["batched"].arms == 8388608
    m = wl.make_inputs(wl.scaled(wl.CONFIGS["medium"], N=4096))
    assert 0.08 < np.mean(m["pulls"] == 0) < 0.16       # 10 % forced zeros + Poisson(4) zeros (1.8 %)


# ------------------------------------------------- within-cluster draw of k_t
def test_philox_known_answers():
    for row in read_golden("philox4x32_10.txt"):
        w = [int(v) for v in row]
        out = oracle.philox4x32_10(w[0:4], w[4:6])
        assert [int(v) for v in out] == w[6:10]


def _sample_case(M, h_members, theta=75.0, seed=0x1234_5678_9ABC_DEF0):
    """M independent instances with the same candidates: rows 0, 2, 4, ... are the members of cluster 1."""
    n_mem = len(h_members)
    N, K, S, R = 2 * n_mem + 1, 3, 4, 5
    labels = np.zeros((M, N), np.int32)
    labels[:, 1::2] = 2
    labels[:, 0:2 * n_mem:2] = 1
    h = np.full((M, N, R), 1.0e3, np.float32)              # any other column or row would dominate if it were read
    target = np.array([4, 0, 3, 1], np.int32)
    s = 2                                                  # strategy 2 looks at resource 3
    h[:, 0:2 * n_mem:2, 3] = np.asarray(h_members, np.float32)
    h[:, 1::2, 3] = -1.0e3                                 # non-members with a huge potential: never drawn
    cluster_arm = np.full((M,), 1 * S + s, np.int32)
    t = np.arange(1, M + 1, dtype=np.int32)
    return dict(labels=labels, cluster_arm=cluster_arm, h_cand=h, target=target, theta_sat=theta, seed=seed, t=t, K=K)


def test_sample_member_follows_the_softmax():
    """Frequencies over many independent draws match exp(V) / sum exp(V), V = theta_sat - h[Target(s)], computed
    here from the definition: a flipped sign of V or of the perturbation, a wrong column or a biased uniform fails."""
    hm = np.array([70.0, 70.5, 71.0, 72.0, 69.2, 73.5])
    M = 120000
    a = _sample_case(M, hm)
    out = oracle.sample_member(**a, want_prob=True)
    V = 75.0 - hm.astype(np.float32).astype(np.float64)    # the signatures are stored in fp32
    p = np.exp(V - V.max())
    p /= p.sum()
    assert np.all(out["member"] % 2 == 0) and np.all(out["member"] < 2 * len(hm))
    freq = np.bincount(out["member"] // 2, minlength=len(hm)) / M
    sigma = np.sqrt(p * (1 - p) / M)
    assert np.all(np.abs(freq - p) < 4.5 * sigma), (freq, p)
    np.testing.assert_allclose(out["prob"][0, 0:2 * len(hm):2], p, rtol=1e-12)
    assert np.all(out["prob"][:, 1::2] == 0.0)
    # equal potentials: uniform over the members
    out_u = oracle.sample_member(**_sample_case(M, np.full(5, 60.0)))
    fu = np.bincount(out_u["member"] // 2, minlength=5) / M
    assert np.all(np.abs(fu - 0.2) < 4.5 * np.sqrt(0.16 / M))


def test_sample_member_rule_and_counter_layout():
    """The drawn member is the largest of V + G over the cluster's members, G = -ln(-ln u), with u taken from the
    generator at counter (candidate, instance, t, 0) and key = the two halves of the seed."""
    hm = np.array([40.0, 41.5, 39.0, 44.0])
    a = _sample_case(50, hm, seed=(0xCAFEBABE << 32) | 0x0BADF00D)
    out = oracle.sample_member(**a)
    for b in range(50):
        vals = {}
        for j, h in enumerate(hm):
            k = 2 * j
            w = oracle.philox4x32_10([k, b, int(a["t"][b]), 0], [0x0BADF00D, 0xCAFEBABE])
            u = ((int(w[0]) >> 9) + 0.5) / 2.0 ** 23
            vals[k] = (75.0 - h) - math.log(-math.log(u))
        best = max(vals, key=lambda k: (vals[k], -k))
        assert out["member"][b] == best
        assert out["member_val"][b] == pytest.approx(vals[best], rel=1e-12)
        for k, v in vals.items():
            assert out["pert"][b, k] == pytest.approx(v, rel=1e-12)
        assert np.all(np.isneginf(np.delete(out["pert"][b], list(vals))))


def test_sample_member_special_cases():
    hm = np.array([10.0, 20.0, 30.0])
    a = _sample_case(8, hm)
    # theta_sat shifts every potential alike: the draw does not move
    m0 = oracle.sample_member(**a)["member"]
    a2 = dict(a, theta_sat=12.5)
    np.testing.assert_array_equal(oracle.sample_member(**a2)["member"], m0)
    # a potential far above the others always wins; a single member is always drawn
    far = _sample_case(64, np.array([90.0, 5.0, 90.0]))
    assert np.all(oracle.sample_member(**far)["member"] == 2)
    one = _sample_case(64, np.array([33.0]))
    assert np.all(oracle.sample_member(**one)["member"] == 0)
    # no pair chosen, or a cluster without members: no draw
    a["cluster_arm"][0] = -1
    a["cluster_arm"][1] = 0 * 4 + 1                         # cluster 0 holds only the last row
    a["cluster_arm"][2] = 2 * 4 + 2                         # cluster 2: the odd rows, potential 75 + 1000 each
    a["labels"][3, :] = 0                                   # instance 3: cluster 1 is empty
    out = oracle.sample_member(**a)
    assert out["member"][0] == -1 and out["member"][3] == -1
    assert out["member"][1] == a["labels"].shape[1] - 1
    assert out["member"][2] % 2 == 1
    # a NaN signature entry is never drawn
    a["h_cand"][4, 0, 3] = np.nan
    a["h_cand"][4, 2, 3] = np.nan
    assert oracle.sample_member(**a)["member"][4] == 4
    # another seed gives other draws, the same seed the same ones
    b1 = oracle.sample_member(**_sample_case(200, np.array([50.0, 50.3, 50.6, 50.9])))["member"]
    b2 = oracle.sample_member(**_sample_case(200, np.array([50.0, 50.3, 50.6, 50.9])))["member"]
    b3 = oracle.sample_member(**_sample_case(200, np.array([50.0, 50.3, 50.6, 50.9]), seed=7))["member"]
    np.testing.assert_array_equal(b1, b2)
    assert np.any(b1 != b3)


# ------------------------------------------------------ outcome of an iteration
def test_record_outcome_reproduces_algorithm1_statistics():
    """Feeding the golden reward sequences through the update, one iteration at a time and through different member
    kernels of one cluster, leaves statistics whose cluster aggregate is Algorithm 1's (N, mu)."""
    for r1, r2, r3, r4, n_fin, mu_fin in read_golden("running_mean.txt"):
        N, S = 3, 2
        pulls = np.zeros((1, N, S), np.int32)
        rsum = np.zeros((1, N, S), np.float32)
        t = np.array([1], np.int32)
        t_cur = np.array([[2.0, 4.0, 8.0]], np.float32)
        for j, r in enumerate([r1, r2, r3, r4]):
            k = j % 2                                             # members 0 and 1 of cluster 0 take turns
            t_new = np.array([t_cur[0, k] * (1.0 - r)], np.float32)   # a kernel faster by the fraction r
            out = oracle.record_outcome([k], [0 * S + 1], t_cur, t_new, pulls, rsum, t)
            assert out["reward"][0] == pytest.approx(r, abs=1e-7)
            pulls, rsum, t = out["pulls"], out["reward_sum"], out["t"]
        assert t[0] == 5 and pulls[0, :, 1].tolist() == [2, 2, 0] and not pulls[0, :, 0].any()
        sc = oracle.score_select(np.array([[0, 0, 1]], np.int32), np.zeros((1, N), np.float32), pulls, rsum, t, K=2)
        assert sc["cl_pulls"][0, 0, 1] == n_fin
        assert sc["cl_mean"][0, 0, 1] == pytest.approx(mu_fin, abs=1e-6)
        assert sc["cl_pulls"][0, 0, 0] == 1 and sc["cl_mean"][0, 0, 0] == 0.5        # untouched pair: the prior


def test_record_outcome_clip_and_failures():
    N, S = 4, 3
    t_cur = np.array([[10.0, 5.0, 0.0, 2.0]] * 6, np.float32)
    member = np.array([0, 0, 1, 2, -1, 3], np.int32)
    arm = np.array([2, 2, 4, 0, 1, 5], np.int32)                   # strategies 2, 2, 1, 0, 1, 2
    t_new = np.array([12.0, 0.0, np.nan, 1.0, 1.0, 1.5], np.float32)
    pulls = np.ones((6, N, S), np.int32)
    rsum = np.full((6, N, S), 0.25, np.float32)
    t = np.arange(6, dtype=np.int32) + 7
    out = oracle.record_outcome(member, arm, t_cur, t_new, pulls, rsum, t)
    # a regression, a kernel of zero runtime, a NaN measurement, a zero incumbent runtime, nothing drawn, a gain
    np.testing.assert_allclose(out["reward"], [0.0, 1.0, 0.0, 0.0, 0.0, 0.25], atol=1e-7)
    np.testing.assert_array_equal(out["t"], t + 1)
    want_p, want_r = pulls.copy(), rsum.copy()
    for b, upd in enumerate([(0, 2, 0.0), (0, 2, 1.0), (1, 1, 0.0), (2, 0, 0.0), None, (3, 2, 0.25)]):
        if upd is not None:
            k, s, r = upd
            want_p[b, k, s] += 1
            want_r[b, k, s] += r
    np.testing.assert_array_equal(out["pulls"], want_p)
    np.testing.assert_allclose(out["reward_sum"], want_r, atol=1e-7)
    # failed verification: Algorithm 1 leaves the statistics alone; the formal model's reading counts a zero
    ver = np.array([1, 0, 1, 1, 1, 0], np.int32)
    a1 = oracle.record_outcome(member, arm, t_cur, t_new, pulls, rsum, t, verified=ver)
    assert a1["pulls"][1].tolist() == pulls[1].tolist() and a1["pulls"][5].tolist() == pulls[5].tolist()
    assert a1["reward"][1] == 0.0 and a1["reward"][5] == 0.0 and a1["t"][1] == t[1] + 1
    np.testing.assert_array_equal(a1["pulls"][[0, 2, 3]], want_p[[0, 2, 3]])
    fm = oracle.record_outcome(member, arm, t_cur, t_new, pulls, rsum, t, verified=ver, failures_count=True)
    assert fm["pulls"][1, 0, 2] == 2 and fm["reward_sum"][1, 0, 2] == pytest.approx(0.25)
    assert fm["pulls"][5, 3, 2] == 2 and fm["reward_sum"][5, 3, 2] == pytest.approx(0.25) and fm["reward"][5] == 0.0


# --------------------------------------------------------- k-means++ seeding
def test_kmeanspp_rounds_follow_the_d2_weights():
    """Round 0 is uniform; a later round draws row x with probability D(x)^2 / sum D^2, D the distance to the NEAREST
    chosen centre (weights computed here from the definition with scipy's cdist)."""
    pts = np.array([[0, 0], [1, 0], [0, 2], [3, 3], [-2, 1], [0.5, 0.5], [4, 0], [1, 0]], np.float32)   # rows 1, 7 equal
    M, N = 100000, len(pts)
    z = np.broadcast_to(pts, (M, N, 2)).copy()
    r0 = oracle.kmeanspp_round(z, np.zeros((M, 0), np.int32), seed=11)["row"]
    f0 = np.bincount(r0, minlength=N) / M
    assert np.all(np.abs(f0 - 1 / N) < 4.5 * np.sqrt((1 / N) * (1 - 1 / N) / M))
    for chosen in ([1], [3, 0], [6, 4, 1]):
        out = oracle.kmeanspp_round(z, np.tile(np.array(chosen, np.int32), (M, 1)), seed=12, want_weights=True)
        d2 = scipy.spatial.distance.cdist(pts.astype(np.float64), pts[chosen].astype(np.float64), "sqeuclidean").min(axis=1)
        p = d2 / d2.sum()
        np.testing.assert_allclose(out["weights"][0], d2, rtol=1e-12)
        f = np.bincount(out["row"], minlength=N) / M
        assert np.all(np.abs(f - p) < 4.5 * np.sqrt(p * (1 - p) / M) + 1e-12), (chosen, f, p)
        assert f[chosen].max() == 0.0                        # a chosen row (and its duplicate) is never drawn again
        if 1 in chosen:
            assert f[7] == 0.0


def test_kmeanspp_full_seeding():
    rng = np.random.default_rng(3)
    # well separated blobs: D^2 seeding puts one seed in every blob nearly always; uniform seeding would manage
    # that for K = 6 equal blobs only 6!/6^6 = 1.5 % of the time
    K, per, B = 6, 40, 300
    centres = 100.0 * np.stack([np.cos(2 * np.pi * np.arange(K) / K), np.sin(2 * np.pi * np.arange(K) / K)], 1)
    z = (centres[None, :, None, :] + rng.standard_normal((B, K, per, 2))).reshape(B, K * per, 2).astype(np.float32)
    rows = oracle.kmeanspp(z, K, seed=99)
    assert rows.min() >= 0 and rows.max() < K * per
    blobs = rows // per
    hit = np.mean([len(set(b)) == K for b in blobs])
    assert hit > 0.97, hit
    # the whole seeding is its rounds, each fed the rows chosen before
    for j in range(K):
        np.testing.assert_array_equal(oracle.kmeanspp_round(z, rows[:, :j], seed=99)["row"], rows[:, j])
    # fewer distinct rows than K: still K valid rows (the surplus rounds draw uniformly)
    dup = np.zeros((50, 7, 3), np.float32)
    dup[:, 3:, :] = 1.0
    r = oracle.kmeanspp(dup, 4, seed=5)
    assert r.min() >= 0 and r.max() < 7
    assert np.all((r[:, 0] < 3) != (r[:, 1] < 3))            # the second seed is always the other point
    # another seed, other seeds; the same seed, the same ones
    np.testing.assert_array_equal(oracle.kmeanspp(z[:20], K, seed=99), rows[:20])
    assert np.any(oracle.kmeanspp(z[:20], K, seed=100) != rows[:20])


# ------------------------------------------------------------ cluster radius
def test_cluster_radius_bounds_the_diameter():
    rng = np.random.default_rng(21)
    B, N, D, K = 2, 400, 5, 6
    z = rng.standard_normal((B, N, D)).astype(np.float32)
    c = rng.standard_normal((B, K, D)).astype(np.float32)
    a = oracle.cluster_assign(z, c, want_rep=False)
    c2, _ = oracle.cluster_update(z, a["labels"], c)
    d2 = oracle.dist2_at(z, c2, a["labels"]).astype(np.float32)
    rad = oracle.cluster_radius(a["labels"], d2, K)
    for b in range(B):
        for i in range(K):
            m = z[b][a["labels"][b] == i].astype(np.float64)
            if len(m) == 0:
                assert rad[b, i] == 0.0
                continue
            # brute force from the definition, with the distances recomputed by scipy
            want = scipy.spatial.distance.cdist(m, c2[b, i][None].astype(np.float64)).max()
            assert rad[b, i] == pytest.approx(want, rel=1e-5)
            if len(m) > 1:
                diam = scipy.spatial.distance.pdist(m).max()
                assert diam <= 2.0 * rad[b, i] * (1 + 1e-6)          # the term of Theorem 1 is bounded from above
                assert diam >= rad[b, i] * (1 - 1e-6)                # and not by more than a factor 2 (centroid = member mean)
    # members on a circle of radius 3 around their centroid; an empty cluster
    ang = np.linspace(0, 2 * np.pi, 12, endpoint=False)
    pts = 3.0 * np.stack([np.cos(ang), np.sin(ang)], 1)
    d2c = (pts ** 2).sum(1).astype(np.float32)[None]
    r = oracle.cluster_radius(np.zeros((1, 12), np.int32), d2c, 2)
    assert r[0, 0] == pytest.approx(3.0, rel=1e-6) and r[0, 1] == 0.0


# ------------------------------------------------------------------ top-M arms
def test_top_m_is_the_sorted_prefix():
    rng = np.random.default_rng(31)
    B, N, S = 4, 300, 8
    a = rng.integers(0, 40, size=(B, N, S)).astype(np.float32) / 8.0      # many exact ties
    a[rng.uniform(size=a.shape) < 0.3] = -np.inf                         # pruned arms
    a[0, 5, 3] = np.nan
    a[3] = -np.inf                                                       # an instance with nothing valid
    a[3, 7, 1], a[3, 2, 6] = 1.5, 1.5                                    # ... but two equal arms
    for M in (1, 5, 64):
        arm, val = oracle.top_m(a, M)
        for b in range(B):
            flat = a[b].reshape(-1)
            ok = np.flatnonzero(flat > -np.inf)                          # drops NaN as well
            # brute force with numpy: value descending, then index ascending
            order = ok[np.lexsort((ok, -flat[ok]))][:M]
            want = np.full(M, -1)
            want[: len(order)] = order
            np.testing.assert_array_equal(arm[b], want)
            np.testing.assert_array_equal(val[b][: len(order)], flat[order])
            assert np.all(np.isneginf(val[b][len(order):]))
    assert oracle.top_m(a, 3)[0][3].tolist() == [2 * S + 6, 7 * S + 1, -1]
    # M = 1 is the masked argmax of score_select; top-M is a prefix of top-(M+1)
    labels = rng.integers(0, 5, (2, 200)).astype(np.int32)
    pulls = rng.poisson(3.0, (2, 200, 4)).astype(np.int32)
    rs = (pulls * rng.uniform(0, 1, pulls.shape)).astype(np.float32)
    keep = rng.integers(0, 16, (2, 200)).astype(np.uint32)
    sc = oracle.score_select(labels, rng.uniform(0, 2, (2, 200)).astype(np.float32), pulls, rs, [50, 60], K=5, keep=keep,
                             lipschitz_L=0.2)
    a1, v1 = oracle.top_m(sc["arm_index"], 1)
    np.testing.assert_array_equal(a1[:, 0], sc["best_arm"])
    np.testing.assert_array_equal(v1[:, 0], sc["best_val"])
    a7, _ = oracle.top_m(sc["arm_index"], 7)
    a8, _ = oracle.top_m(sc["arm_index"], 8)
    np.testing.assert_array_equal(a8[:, :7], a7)


# -------------------------------------------- the loop on the cluster tables
def test_select_pair_worked_values_and_mask():
    # the golden index values, one pair at a time
    for t, n, mu, c, u in read_golden("masked_ucb_index.txt"):
        out = oracle.select_pair(np.full((1, 1, 1), n, np.float32), np.full((1, 1, 1), mu, np.float32), [int(t)], c=c)
        assert out["cl_index"][0, 0, 0] == pytest.approx(u, abs=2e-6) and out["pair"][0] == 0
    # against the whole-array statistics: same tables in, same cluster-level choice out (no arm masked)
    rng = np.random.default_rng(8)
    B, N, K, S = 5, 300, 6, 4
    labels = rng.integers(0, K, (B, N)).astype(np.int32)
    pulls = rng.poisson(2.0, (B, N, S)).astype(np.int32)
    rs = (pulls * rng.uniform(0, 1, pulls.shape)).astype(np.float32)
    t = (1 + pulls.reshape(B, -1).sum(1)).astype(np.int32)
    sc = oracle.score_select(labels, np.zeros((B, N), np.float32), pulls, rs, t, K=K)
    sp = oracle.select_pair(sc["cl_pulls"], sc["cl_mean"], t)
    np.testing.assert_array_equal(sp["pair"], sc["best_cluster_arm"])
    np.testing.assert_allclose(sp["cl_index"], sc["cl_index"], atol=2e-6)
    # the saturation mask of Algorithm 1: M_{i,s} = [h_c^(i)[Target(s)] < theta]; brute force over the unmasked pairs
    hsig = rng.uniform(0, 100, (B, K, 3)).astype(np.float32)
    target = np.array([2, 0, 1, 0], np.int32)
    spm = oracle.select_pair(sc["cl_pulls"], sc["cl_mean"], t, hsig=hsig, target=target, theta_sat=60.0)
    for b in range(B):
        valid = hsig[b][:, target] < 60.0                                   # [K][S]
        u = np.where(valid, sc["cl_index"][b].astype(np.float64), -np.inf)
        assert spm["pair"][b] == (int(np.argmax(u.reshape(-1))) if valid.any() else -1)
    none = oracle.select_pair(sc["cl_pulls"], sc["cl_mean"], t, hsig=hsig, target=target, theta_sat=-1.0)
    assert np.all(none["pair"] == -1)


def test_update_pair_is_algorithm1_and_matches_the_aggregate():
    for r1, r2, r3, r4, n_fin, mu_fin in read_golden("running_mean.txt"):
        n = np.ones((1, 2, 3), np.float32)
        mu = np.full((1, 2, 3), 0.5, np.float32)
        for r in (r1, r2, r3, r4):
            n, mu = oracle.update_pair([1 * 3 + 2], [r], n, mu)
        assert n[0, 1, 2] == n_fin and mu[0, 1, 2] == pytest.approx(mu_fin, abs=1e-6)
        assert n.sum() == 5 + n_fin and mu[0, 0, 0] == 0.5                   # the other pairs untouched
    n2, mu2 = oracle.update_pair([-1], [0.7], n, mu)                         # nothing chosen: nothing changes
    assert np.array_equal(n2, n) and np.array_equal(mu2, mu)
    # incremental tables track the per-arm bookkeeping of record_outcome + score_select
    rng = np.random.default_rng(2)
    B, N, K, S = 3, 50, 4, 3
    labels = rng.integers(0, K, (B, N)).astype(np.int32)
    pulls = np.zeros((B, N, S), np.int32)
    rs = np.zeros((B, N, S), np.float32)
    t = np.ones(B, np.int32)
    n = np.ones((B, K, S), np.float32)
    mu = np.full((B, K, S), 0.5, np.float32)
    for it in range(40):
        k = rng.integers(0, N, B).astype(np.int32)
        s = rng.integers(0, S, B)
        pair = (labels[np.arange(B), k] * S + s).astype(np.int32)
        t_new = rng.uniform(0.2, 1.4, B).astype(np.float32)
        out = oracle.record_outcome(k, pair, np.ones((B, N), np.float32), t_new, pulls, rs, t)
        pulls, rs, t = out["pulls"], out["reward_sum"], out["t"]
        n, mu = oracle.update_pair(pair, out["reward"], n, mu)
    sc = oracle.score_select(labels, np.zeros((B, N), np.float32), pulls, rs, t, K=K)
    np.testing.assert_array_equal(n, sc["cl_pulls"])
    np.testing.assert_allclose(mu, sc["cl_mean"], atol=2e-6)


# ------------------------------------------------------------- input recipe
def test_candidate_signatures_recipe():
    """Seeded, clipped to the percent range, centred on the cluster's signature (input data only)."""
    rng = np.random.default_rng(0)
    hsig = rng.uniform(0, 100, (2, 5, wl.R_RESOURCES)).astype(np.float32)
    labels = rng.integers(0, 5, (2, 4000)).astype(np.int32)
    h1 = wl.make_candidate_signatures(hsig, labels, seed=3)
    h2 = wl.make_candidate_signatures(hsig, labels, seed=3)
    h3 = wl.make_candidate_signatures(hsig, labels, seed=4)
    assert h1.dtype == np.float32 and h1.shape == (2, 4000, wl.R_RESOURCES)
    np.testing.assert_array_equal(h1, h2)
    assert np.any(h1 != h3)
    assert h1.min() >= 0.0 and h1.max() <= 100.0
    base = hsig[np.arange(2)[:, None], labels]
    inner = (base > 15) & (base < 85)                       # away from the clip
    assert abs(float((h1 - base)[inner].mean())) < 0.1 and 2.7 < float((h1 - base)[inner].std()) < 3.3
    assert wl.make_candidate_signatures(hsig, np.zeros((2, 0), np.int32), seed=1).shape == (2, 0, wl.R_RESOURCES)


# ------------------------------------------------------------------ restarts
def test_best_restart_is_numpy_argmin():
    rng = np.random.default_rng(6)
    x = rng.integers(0, 6, (50, 7)).astype(np.float32)            # many ties: numpy's argmin also takes the first
    np.testing.assert_array_equal(oracle.best_restart(x), np.argmin(x, axis=1))
    x[0, :] = np.nan
    x[1, 0] = np.nan
    x[2, 3] = np.inf
    b = oracle.best_restart(x)
    assert b[0] == -1 and b[1] == 1 + int(np.argmin(x[1, 1:])) and b[2] == int(np.nanargmin(x[2]))
    assert oracle.best_restart(np.array([[3.0]], np.float32))[0] == 0
    # restarts help: the best of several seedings is never worse than the first
    K, per, B, n_init = 5, 30, 6, 4
    cen = rng.standard_normal((K, 3)) * 4
    z = (cen[None, :, None, :] + rng.standard_normal((B, K, per, 3))).reshape(B, K * per, 3).astype(np.float32)
    zz = np.repeat(z, n_init, axis=0)                             # n_init consecutive copies of every instance
    rows = oracle.kmeanspp(zz, K, seed=1)                         # the instance index is in the counter: seeds differ
    c = oracle.init_centroids(zz, rows)
    for _ in range(5):
        a = oracle.cluster_assign(zz, c, want_rep=False)
        c, _ = oracle.cluster_update(zz, a["labels"], c)
    inertia = oracle.cluster_assign(zz, c, want_rep=False)["inertia"].reshape(B, n_init)
    best = oracle.best_restart(inertia)
    assert np.all(inertia[np.arange(B), best] <= inertia[:, 0])
    assert len({tuple(r) for r in rows.reshape(B, n_init, K)[0].tolist()}) > 1


# ------------------------------------------------------- the expanding frontier
def _frontier_state(B, cap, D, S, R, rng):
    """One initial kernel k_0 per search (Algorithm 1: P <- {k_0}, one initial cluster); padding rows carry label -1."""
    st = {"n_active": np.ones(B, np.int32), "x": np.zeros((B, cap, D), np.float32),
          "t_cur": np.zeros((B, cap), np.float32), "labels": np.full((B, cap), -1, np.int32),
          "dist2": np.zeros((B, cap), np.float32), "pulls": np.zeros((B, cap, S), np.int32),
          "reward_sum": np.zeros((B, cap, S), np.float32), "h_cand": np.zeros((B, cap, R), np.float32),
          "flops": np.zeros((B, cap), np.float32), "bytes": np.zeros((B, cap), np.float32),
          "t_inc": np.zeros(B, np.float32)}
    st["x"][:, 0] = rng.standard_normal((B, D)).astype(np.float32)
    st["t_cur"][:, 0] = rng.uniform(1.0, 2.0, B).astype(np.float32)
    st["h_cand"][:, 0] = rng.uniform(0, 100, (B, R)).astype(np.float32)
    st["flops"][:, 0], st["bytes"][:, 0] = 1e9, 1e8
    st["labels"][:, 0] = 0
    st["t_inc"][:] = st["t_cur"][:, 0]
    return st


def test_frontier_growth_and_trigger_against_algorithm1_with_python_lists():
    """Algorithm 1's frontier as plain Python lists (P.append(k') inside `if Verify`, the test
    `t % tau == 0 and len(P) >= 2 * K`), run beside the array form for the paper's own sizes
    (T = 40, tau = 10, K = 3, |S| = 6, phi in R^5, one initial kernel) on three searches."""
    T, tau, K, S, D, R, cap, B = 40, 10, 3, 6, 5, 3, 24, 3
    rng = np.random.default_rng(7)
    st = _frontier_state(B, cap, D, S, R, rng)
    st["pulls"][:, 0] = rng.integers(0, 4, (B, S))                   # history of k_0 must survive every append
    st["reward_sum"][:, 0] = rng.uniform(0, 1, (B, S)).astype(np.float32)
    P = [[dict(phi=st["x"][b, 0].copy(), T=float(st["t_cur"][b, 0]), h=st["h_cand"][b, 0].copy(), cluster=0,
               F=float(st["flops"][b, 0]), Q=float(st["bytes"][b, 0]), pulls=st["pulls"][b, 0].copy(),
               rsum=st["reward_sum"][b, 0].copy(), d2=0.0)] for b in range(B)]
    best = [P[b][0]["T"] for b in range(B)]
    n_due = 0
    for t in range(1, T + 1):
        tt = np.full(B, t, np.int32)
        # ---- the trigger
        lit_due = [int(t % tau == 0 and len(P[b]) >= 2 * K) for b in range(B)]
        assert list(oracle.recluster_due(tt, st["n_active"], tau, K)) == lit_due
        for b in range(B):
            if lit_due[b]:                                           # some re-partition: the growth rule only needs labels to change
                n_due += 1
                for j, k in enumerate(P[b]):
                    k["cluster"] = (j * 7 + t) % K
                    k["d2"] = float(np.float32(0.01 * j))
                    st["labels"][b, j] = k["cluster"]
                    st["dist2"][b, j] = k["d2"]
        # ---- one generation per search: a parent among the active kernels, sometimes nothing drawn, sometimes rejected
        parent = np.array([rng.integers(0, len(P[b])) if rng.uniform() > 0.1 else -1 for b in range(B)], np.int32)
        verified = (rng.uniform(size=B) < 0.8).astype(np.int32)
        x_new = rng.standard_normal((B, D)).astype(np.float32)
        t_new = rng.uniform(0.3, 2.5, B).astype(np.float32)
        f_new, q_new = rng.uniform(1e6, 1e9, B).astype(np.float32), rng.uniform(1e6, 1e9, B).astype(np.float32)
        h_new = rng.uniform(0, 100, (B, R)).astype(np.float32)
        want_row, want_full = [], []
        for b in range(B):
            ok = parent[b] >= 0 and verified[b] != 0
            if ok and len(P[b]) < cap:
                want_row.append(len(P[b]))
                P[b].append(dict(phi=x_new[b].copy(), T=float(t_new[b]), h=h_new[b].copy(), cluster=P[b][parent[b]]["cluster"],
                                 F=float(f_new[b]), Q=float(q_new[b]), pulls=np.zeros(S, np.int32),
                                 rsum=np.zeros(S, np.float32), d2=P[b][parent[b]]["d2"]))
                best[b] = min(best[b], float(t_new[b]))
                want_full.append(0)
            else:
                want_row.append(-1)
                want_full.append(int(ok))
        st, row, full = oracle.append_candidate(st, parent, x_new, t_new, verified, f_new, q_new, h_new)
        assert list(row) == want_row and list(full) == want_full
        # ---- the arrays are the lists, row for row; padding untouched
        for b in range(B):
            n = len(P[b])
            assert st["n_active"][b] == n
            assert np.array_equal(st["x"][b, :n], np.stack([k["phi"] for k in P[b]]))
            assert np.array_equal(st["t_cur"][b, :n], np.array([k["T"] for k in P[b]], np.float32))
            assert np.array_equal(st["h_cand"][b, :n], np.stack([k["h"] for k in P[b]]))
            assert np.array_equal(st["flops"][b, :n], np.array([k["F"] for k in P[b]], np.float32))
            assert np.array_equal(st["bytes"][b, :n], np.array([k["Q"] for k in P[b]], np.float32))
            assert list(st["labels"][b, :n]) == [k["cluster"] for k in P[b]]
            assert np.array_equal(st["dist2"][b, :n], np.array([k["d2"] for k in P[b]], np.float32))
            assert np.array_equal(st["pulls"][b, :n], np.stack([k["pulls"] for k in P[b]]))
            assert np.array_equal(st["reward_sum"][b, :n], np.stack([k["rsum"] for k in P[b]]))
            assert np.all(st["labels"][b, n:] == -1) and np.all(st["x"][b, n:] == 0) and np.all(st["pulls"][b, n:] == 0)
            assert st["t_inc"][b] == np.float32(best[b])             # argmin of T over the frontier (the return line)
    assert n_due >= 4 and max(len(p) for p in P) == cap             # the trigger fired and one frontier filled up
    # an index beyond the frontier is an error, not a silent append
    with pytest.raises(ValueError):
        oracle.append_candidate(st, np.array([cap, 0, 0], np.int32), x_new, t_new)


def test_recluster_trigger_values():
    # t mod tau == 0 and |P| >= 2K, each factor alone is not enough
    t = np.array([10, 10, 20, 15, 0, 30], np.int32)
    n = np.array([6, 5, 100, 100, 6, 6], np.int32)
    assert list(oracle.recluster_due(t, n, 10, 3)) == [1, 0, 1, 0, 1, 1]
    assert list(oracle.recluster_due(t, n, 5, 3)) == [1, 0, 1, 1, 1, 1]
    assert list(oracle.recluster_due(t, n, 10, 4)) == [0, 0, 1, 0, 0, 0]


def test_signatures_from_reps_masks_empty_clusters():
    rng = np.random.default_rng(3)
    B, N, K, R = 2, 9, 4, 3
    h = rng.uniform(0, 100, (B, N, R)).astype(np.float32)
    rep = np.array([[3, -1, 8, 0], [-1, -1, 2, 2]], np.int32)
    hs = oracle.signatures_from_reps(rep, h)
    for b in range(B):
        for i in range(K):
            if rep[b, i] < 0:
                assert np.all(np.isposinf(hs[b, i]))
            else:
                assert np.array_equal(hs[b, i], h[b, rep[b, i]])
    # an empty cluster is never the masked-UCB choice, whatever its statistics say
    cl_pulls, cl_mean = np.ones((B, K, 2), np.float32), np.full((B, K, 2), 0.5, np.float32)
    cl_mean[:, 1] = 10.0                                             # cluster 1 (empty in both) would win otherwise
    pair = oracle.select_pair(cl_pulls, cl_mean, np.array([5, 5], np.int32), hsig=hs, target=np.array([0, 1], np.int32),
                              theta_sat=200.0)["pair"]
    assert pair[0] // 2 in (0, 2, 3) and pair[1] // 2 in (2, 3)
    # instances that are not due keep their signatures
    prev = np.full((B, K, R), 7.0, np.float32)
    hs2 = oracle.signatures_from_reps(rep, h, hsig_prev=prev, run=np.array([0, 1], np.int32))
    assert np.all(hs2[0] == 7.0) and np.array_equal(hs2[1], hs[1])


# ----------------------------------------------------- tolerance stop, unused clusters
def test_lloyd_tol_matches_sklearn_iteration_counts():
    """The tolerance stop against scikit-learn's KMeans (Sec. 3.5) from the same initial centres: the number of
    iterations it reports, its centres and its labels.  scikit-learn scales `tol` by the mean column variance
    (1 for z-scored features without constant columns) and also stops when the labels repeat, which the shift
    rule covers (unchanged labels -> unchanged centres -> shift 0)."""
    sklearn_cluster = pytest.importorskip("sklearn.cluster")
    rng = np.random.default_rng(12)
    for N, D, K, tol in [(400, 5, 3, 1e-4), (900, 8, 6, 1e-2), (600, 4, 5, 0.0), (300, 16, 4, 1e-3), (500, 6, 3, 0.3)]:
        centres = 2.0 * rng.standard_normal((K, D))
        x = (centres[rng.integers(0, K, N)] + rng.standard_normal((N, D))).astype(np.float32)
        z, _, _ = oracle.normalize(x[None])
        init = z[0, rng.choice(N, K, replace=False)]
        scaled_tol = tol * float(np.mean(np.var(z[0].astype(np.float64), axis=0)))
        km = sklearn_cluster.KMeans(n_clusters=K, init=init.astype(np.float64), n_init=1, max_iter=50, tol=tol,
                                    algorithm="lloyd").fit(z[0].astype(np.float64))
        got = oracle.lloyd_tol(z, init[None], 50, scaled_tol)
        assert got["n_iter"][0] == km.n_iter_, (N, D, K, tol, got["n_iter"][0], km.n_iter_)
        np.testing.assert_allclose(got["centroids"][0], km.cluster_centers_, atol=2e-5)
        assert np.array_equal(got["labels"][0], km.labels_)
        assert got["inertia"][0] == pytest.approx(km.inertia_, rel=1e-5)
        assert got["last_shift"][0] <= scaled_tol or got["n_iter"][0] == 50
        assert got["counts"][0].sum() == N                             # (the members of the last update, not of the final labels)


def test_lloyd_tol_is_the_plain_loop_cut_short():
    """tol < 0 never stops early: exactly max_iter plain iterations; with a tolerance the result is the plain loop's
    after n_iter iterations; instances of one batch stop independently."""
    rng = np.random.default_rng(13)
    B, N, D, K = 4, 300, 6, 5
    z = rng.standard_normal((B, N, D)).astype(np.float32)
    z[0] *= 0.01                                                       # instance 0 converges at once on any scale
    init = np.stack([z[b, rng.choice(N, K, replace=False)] for b in range(B)])
    full = oracle.lloyd_tol(z, init, 7, -1.0)
    assert np.all(full["n_iter"] == 7)
    c = init.copy()
    for _ in range(7):
        a = oracle.cluster_assign(z, c, want_rep=False)
        c, n = oracle.cluster_update(z, a["labels"], c)
    assert np.array_equal(full["centroids"], c) and np.array_equal(full["counts"], n)
    tol = oracle.lloyd_tol(z, init, 50, 1e-3)
    assert len(set(tol["n_iter"].tolist())) > 1 and tol["n_iter"].max() < 50
    for b in range(B):
        c = init[b:b + 1].copy()
        for _ in range(int(tol["n_iter"][b])):
            a = oracle.cluster_assign(z[b:b + 1], c, want_rep=False)
            c, _ = oracle.cluster_update(z[b:b + 1], a["labels"], c)
        assert np.array_equal(tol["centroids"][b:b + 1], c)
        a = oracle.cluster_assign(z[b:b + 1], c)
        assert np.array_equal(tol["labels"][b:b + 1], a["labels"]) and np.array_equal(tol["rep"][b:b + 1], a["rep"])
    assert np.all(oracle.lloyd_tol(z, init, 0, 1.0)["n_iter"] == 0)     # no iteration: the labels of the initial centres


def test_unused_clusters_share_a_batch_with_fewer_clusters():
    """rows = -1 marks a cluster as unused (centroid far away): an instance with K_b < K clusters then clusters exactly
    as it would alone with K_b -- the K in {1, 2, 3, 5} sensitivity study as four instances of one call with K = 5."""
    rng = np.random.default_rng(14)
    N, D, K = 200, 5, 5
    x = (3.0 * rng.standard_normal((4, 1, D)) * (rng.integers(0, 3, (4, N, 1)) - 1) + rng.standard_normal((4, N, D))).astype(np.float32)
    z, _, _ = oracle.normalize(x)
    rows = np.full((4, K), -1, np.int32)
    for b, kb in enumerate([1, 2, 3, 5]):
        rows[b, :kb] = rng.choice(N, kb, replace=False)
    c0 = oracle.init_centroids(z, rows)
    assert np.all(c0[0, 1:] == np.float32(1e18)) and np.array_equal(c0[1, :2], z[1, rows[1, :2]])
    got = oracle.lloyd_tol(z, c0, 10, -1.0)
    for b, kb in enumerate([1, 2, 3, 5]):
        alone = oracle.lloyd_tol(z[b:b + 1], oracle.init_centroids(z[b:b + 1], rows[b:b + 1, :kb]), 10, -1.0)
        assert np.array_equal(got["labels"][b], alone["labels"][0]) and got["labels"][b].max() < kb
        assert np.array_equal(got["centroids"][b, :kb], alone["centroids"][0])
        assert np.all(got["centroids"][b, kb:] == np.float32(1e18))       # never moved, never chosen
        assert np.all(got["counts"][b, kb:] == 0) and np.all(got["rep"][b, kb:] == -1)
        assert got["inertia"][b] == alone["inertia"][0]
    with pytest.raises(ValueError):
        oracle.init_centroids(z, np.full((4, K), -2, np.int32))
