"""GPU parity: every C-ABI call against the CPU oracle on the same seeded
inputs ("teacher-forced": each call is fed the oracle's inputs for that step),
then the free-running whole step."""
import numpy as np
import pytest
import torch

import oracle
import parity
from paper_2511_18868_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def kbx():
    from paper_2511_18868_b200 import kb
    ctx = kb.KB(0)
    yield ctx
    assert ctx.device_status() == 0
    ctx.close()


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def host(t):
    return t.cpu().numpy()


def empty(shape, dt=torch.float32):
    return torch.empty(shape, dtype=dt, device="cuda")


def ws(kbx, B, N, D, K, S):
    kbx.ensure_workspace(kbx.workspace_bytes(B, N, D, K, S))


# ----------------------------------------------------------------- normalise
@pytest.mark.parametrize("B,N,D", [(1, 256, 16), (3, 1000, 20), (2, 777, 5), (1, 4097, 24), (1, 1, 8),
                                   (5, 300, 64), (1, 20000, 128), (1, 513, 1100)])
def test_normalize(kbx, B, N, D):
    rng = np.random.default_rng(B * 1000 + N + D)
    x = (rng.standard_normal((B, N, D)) * rng.uniform(0.05, 30, D) + rng.uniform(-50, 50, D)).astype(np.float32)
    if D > 2:
        x[:, :, 1] = -3.5                      # constant column -> zeros, scale 1
        x[:, :, 2] = 1000.0 + rng.standard_normal((B, N)).astype(np.float32)   # large offset
    ws(kbx, B, N, D, 1, 1)
    xd, z, mean, scale = dev(x), empty((B, N, D)), empty((B, D)), empty((B, D))
    kbx.normalize(xd, z, mean, scale)
    zr, mr, sr = oracle.normalize(x)
    # z has unit scale per column: absolute floor 1e-5 (values near 0 cancel)
    parity.close(host(z), zr, atol=2e-5, what="z")
    parity.close(host(mean), mr, atol=1e-6, what="mean")
    parity.close(host(scale), sr, atol=0, what="scale")
    if D > 2:
        assert np.all(host(z)[:, :, 1] == 0) and np.all(host(scale)[:, 1] == 1)
    # in place
    kbx.normalize(xd)
    parity.close(host(xd), zr, atol=2e-5, what="z in place")


def test_normalize_empty(kbx):
    ws(kbx, 2, 0, 8, 1, 1)
    mean, scale = empty((2, 8)), empty((2, 8))
    kbx.normalize(empty((2, 0, 8)), empty((2, 0, 8)), mean, scale)
    assert np.all(host(mean) == 0) and np.all(host(scale) == 1)


# --------------------------------------------------------------------- prune
@pytest.mark.parametrize("B,N,S,K,sat,bound", [(1, 256, 8, 8, True, True), (3, 1000, 13, 5, True, True),
                                               (2, 129, 32, 4, False, True), (1, 5000, 1, 3, True, False),
                                               (4, 127, 16, 16, False, False)])
def test_prune(kbx, B, N, S, K, sat, bound):
    cfg = wl.scaled(wl.CONFIGS["tiny"], B=B, N=N, S=S, K=K)
    inp = wl.make_inputs(cfg, seed=7)
    labels = np.random.default_rng(1).integers(0, K, (B, N)).astype(np.int32)
    ref = oracle.prune(inp["flops"], inp["bytes"], inp["peak_flops"], inp["peak_bw"], inp["t_inc"], inp["t_cur"],
                       labels if sat else None, inp["hsig"] if sat else None, inp["target"] if sat else None,
                       75.0, want_bound=bound, want_margin=True)
    keep, kept = empty((B, N), torch.int32), empty((B,), torch.int32)
    bd = empty((B, N, S)) if bound else None
    kbx.prune(dev(inp["flops"]), dev(inp["bytes"]), dev(inp["peak_flops"]), dev(inp["peak_bw"]), dev(inp["t_inc"]),
              keep, t_cur=dev(inp["t_cur"]), labels=dev(labels) if sat else None,
              hsig=dev(inp["hsig"]) if sat else None, target=dev(inp["target"]) if sat else None,
              theta_sat=75.0, kept_count=kept, bound=bd)
    got = host(keep).view(np.uint32)
    ties = parity.keep_match(got, ref, S)
    pop = sum(int(v).bit_count() for v in got.reshape(-1))
    assert int(host(kept).view(np.uint32).sum()) == pop
    assert abs(pop - int(ref["kept_count"].sum())) <= ties
    if bound:
        # bound lies in [0,1]: absolute floor of a few ulp of 1
        parity.close(host(bd), ref["bound"], atol=1e-6, what="bound")


def test_prune_threshold_edges(kbx):
    # exact equality is pruned (strict <), on both factors
    flops = np.array([[1e9, 2e9, 1e9]], np.float32)
    byts = np.array([[1.0, 1.0, 1.0]], np.float32)
    pf, pb = np.array([1e12], np.float32), np.array([1e12], np.float32)
    tinc = np.array([np.float32(2e9) / np.float32(1e12)], np.float32)
    hs = np.array([[[75.0], [74.0]]], np.float32)
    labels = np.array([[1, 1, 0]], np.int32)
    keep = empty((1, 3), torch.int32)
    kbx.prune(dev(flops), dev(byts), dev(pf), dev(pb), dev(tinc), keep, labels=dev(labels), hsig=dev(hs),
              target=dev(np.array([0], np.int32)), theta_sat=75.0)
    assert list(host(keep)[0]) == [1, 0, 0]


# -------------------------------------------------------------------- assign
@pytest.mark.parametrize("B,N,D,K", [(1, 256, 16, 8), (2, 1000, 20, 7), (1, 333, 5, 3), (3, 500, 32, 1),
                                     (1, 3000, 64, 300), (1, 700, 128, 65), (2, 129, 8, 130), (1, 40, 260, 9)])
def test_assign(kbx, B, N, D, K):
    rng = np.random.default_rng(N + D + K)
    z = rng.standard_normal((B, N, D)).astype(np.float32)
    c = z[:, rng.choice(N, K, replace=K > N)] + (0.05 * rng.standard_normal((B, K, D))).astype(np.float32)
    if K > 2:
        c[:, K - 1] = c[:, 0]                   # duplicate centroid: the lower id must win
    ws(kbx, B, N, D, K, 1)
    labels, d2, inertia, rep = empty((B, N), torch.int32), empty((B, N)), empty((B,)), empty((B, K), torch.int32)
    kbx.cluster_assign(dev(z), dev(c), labels, d2, inertia, rep)
    ref = oracle.cluster_assign(z, c, want_margins=True)
    got = host(labels)
    parity.labels_match(z, c, got, ref)
    if K > 2:
        assert not np.any(got == K - 1)
    same = got == ref["labels"]
    parity.close(host(d2)[same], ref["dist2"][same], atol=1e-7, what="dist2")
    parity.close(host(inertia), ref["inertia"], atol=1e-6, what="inertia")
    parity.rep_match(host(rep), ref, ref["dist2"], ref["labels"])
    # labels only
    labels2 = empty((B, N), torch.int32)
    kbx.cluster_assign(dev(z), dev(c), labels2)
    assert np.array_equal(host(labels2), got)


def test_assign_rows_equal_to_centroids_have_zero_distance(kbx):
    rng = np.random.default_rng(3)
    z = rng.standard_normal((1, 600, 32)).astype(np.float32)
    rows = rng.choice(600, 16, replace=False)
    labels, d2 = empty((1, 600), torch.int32), empty((1, 600))
    ws(kbx, 1, 600, 32, 16, 1)
    kbx.cluster_assign(dev(z), dev(z[:, rows]), labels, d2)
    assert np.array_equal(host(labels)[0, rows], np.arange(16)) and np.all(host(d2)[0, rows] == 0)


# -------------------------------------------------------------------- update
@pytest.mark.parametrize("B,N,D,K", [(1, 256, 16, 8), (2, 1000, 20, 7), (1, 333, 5, 3), (3, 500, 32, 1),
                                     (1, 5000, 64, 256), (1, 3000, 128, 1024), (2, 129, 24, 130)])
def test_update(kbx, B, N, D, K):
    rng = np.random.default_rng(N * 3 + D + K)
    z = rng.standard_normal((B, N, D)).astype(np.float32)
    labels = rng.integers(0, max(1, K - 1), (B, N)).astype(np.int32)   # last cluster empty when K > 1
    prev = rng.standard_normal((B, K, D)).astype(np.float32)
    ws(kbx, B, N, D, K, 1)
    c, counts = dev(prev), empty((B, K), torch.int32)
    kbx.cluster_update(dev(z), dev(labels), c, counts)
    cr, nr = oracle.cluster_update(z, labels, prev)
    assert np.array_equal(host(counts), nr)
    # centroid coordinates are means of unit-scale data: absolute floor 1e-5
    parity.close(host(c), cr, atol=1e-5, what="centroids")
    if K > 1:
        assert np.array_equal(host(c)[:, K - 1], prev[:, K - 1])


def test_update_empty_input(kbx):
    ws(kbx, 2, 0, 8, 4, 1)
    prev = np.ones((2, 4, 8), np.float32)
    c, counts = dev(prev), empty((2, 4), torch.int32)
    kbx.cluster_update(empty((2, 0, 8)), empty((2, 0), torch.int32), c, counts)
    assert np.all(host(counts) == 0) and np.array_equal(host(c), prev)


# --------------------------------------------------------------------- score
def run_score(kbx, labels, dist2, pulls, rsum, t, K, keep=None, bound=None, **prm):
    B, N, S = pulls.shape
    ws(kbx, B, N, 1, K, S)
    o = dict(cl_pulls=empty((B, K, S)), cl_mean=empty((B, K, S)), cl_index=empty((B, K, S)),
             arm_index=empty((B, N, S)), best_arm=empty((B,), torch.int32), best_val=empty((B,)),
             best_cluster_arm=empty((B,), torch.int32))
    kbx.score_select(dev(labels), dev(dist2), dev(pulls), dev(rsum), dev(t), keep=None if keep is None else dev(keep.view(np.int32)),
                     bound=None if bound is None else dev(bound), **o, **prm)
    return {k: host(v) for k, v in o.items()}


@pytest.mark.parametrize("B,N,K,S,L,masked,cap", [(1, 256, 8, 8, 0.1, True, False), (3, 1000, 7, 13, 0.0, True, False),
                                                  (2, 500, 1, 6, 0.0, False, False), (1, 4000, 64, 32, 0.1, True, True),
                                                  (4, 129, 16, 16, 0.3, False, False), (1, 3000, 1024, 8, 0.1, True, False),
                                                  # instances of at most 1024 candidates, S in {4, 8, 16, 32}: one launch
                                                  (2, 1024, 256, 32, 0.1, True, True), (3, 100, 4, 4, 0.0, False, True),
                                                  (5, 777, 12, 8, 0.2, False, False), (70, 64, 3, 16, 0.0, True, False),
                                                  (2, 1025, 8, 8, 0.1, True, False)])
def test_score_select(kbx, B, N, K, S, L, masked, cap):
    rng = np.random.default_rng(N + K + S)
    labels = rng.integers(0, max(1, K - 1), (B, N)).astype(np.int32)
    dist2 = rng.uniform(0, 4, (B, N)).astype(np.float32)
    pulls = rng.poisson(3.0, (B, N, S)).astype(np.int32)
    pulls[rng.uniform(size=pulls.shape) < 0.1] = 0
    rsum = (pulls * rng.uniform(0, 2, pulls.shape)).astype(np.float32)
    t = (1 + pulls.reshape(B, -1).sum(1)).astype(np.int32)
    keep = rng.integers(0, 1 << S, (B, N), dtype=np.uint64).astype(np.uint32) if masked else None
    bound = rng.uniform(0, 3, (B, N, S)).astype(np.float32) if cap else None
    prm = dict(c=2.0, lipschitz_L=L, prior_pulls=1.0, prior_mean=0.5, cap_with_bound=cap)
    got = run_score(kbx, labels, dist2, pulls, rsum, t, K, keep, bound, **prm)
    ref = oracle.score_select(labels, dist2, pulls, rsum, t, K, keep=keep, bound=bound, **prm)
    assert np.array_equal(got["cl_pulls"], ref["cl_pulls"])          # integer totals below 2^24: exact
    parity.close(got["cl_mean"], ref["cl_mean"], atol=1e-6, what="cl_mean")
    parity.close(got["cl_index"], ref["cl_index"], atol=1e-6, what="cl_index")
    parity.close(got["arm_index"], ref["arm_index"], atol=1e-6, what="arm_index")
    parity.select_match(got["best_arm"], got["best_val"], ref, ref["arm_index"])
    parity.cluster_select_match(got["best_cluster_arm"], ref, ref["cl_index"])
    if L == 0.0 and not cap:
        # exact ties inside the winning cluster: the lowest flat index must win
        assert np.array_equal(got["best_arm"], ref["best_arm"])


def test_score_select_small_is_one_launch_and_optional_outputs(kbx):
    """Small instances: kb_score_select is one launch; without arm_index the selections are unchanged."""
    rng = np.random.default_rng(4)
    B, N, K, S = 6, 300, 5, 8
    labels = rng.integers(0, K, (B, N)).astype(np.int32)
    dist2 = rng.uniform(0, 4, (B, N)).astype(np.float32)
    pulls = rng.poisson(3.0, (B, N, S)).astype(np.int32)
    rsum = (pulls * rng.uniform(0, 2, pulls.shape)).astype(np.float32)
    t = (1 + pulls.reshape(B, -1).sum(1)).astype(np.int32)
    k0 = kbx.launch_count()
    full = run_score(kbx, labels, dist2, pulls, rsum, t, K, lipschitz_L=0.1)
    k1 = kbx.launch_count()
    assert k1[0] - k0[0] == 1 and k1[1] - k0[1] == 0
    o = dict(cl_pulls=empty((B, K, S)), cl_mean=empty((B, K, S)), cl_index=empty((B, K, S)),
             best_arm=empty((B,), torch.int32), best_val=empty((B,)), best_cluster_arm=empty((B,), torch.int32))
    kbx.score_select(dev(labels), dev(dist2), dev(pulls), dev(rsum), dev(t), **o, lipschitz_L=0.1)
    # (reward sums are added in shared memory in no fixed order: last-bit differences between two runs are expected)
    ref = oracle.score_select(labels, dist2, pulls, rsum, t, K, c=2.0, lipschitz_L=0.1)
    parity.close(host(o["cl_index"]), ref["cl_index"], atol=1e-6, what="cl_index")
    parity.select_match(host(o["best_arm"]), host(o["best_val"]), ref, ref["arm_index"])
    parity.cluster_select_match(host(o["best_cluster_arm"]), ref, ref["cl_index"])
    parity.select_match(full["best_arm"], full["best_val"], ref, ref["arm_index"])


def test_score_all_masked_and_unplayed(kbx):
    labels = np.array([[0, 0, 1, 1, 2, 2]], np.int32)
    pulls = np.array([[[4, 3], [2, 5], [6, 1], [3, 3], [2, 0], [5, 0]]], np.int32)
    rsum = (pulls * 0.95).astype(np.float32)
    t = np.array([1 + pulls.sum()], np.int32)
    d2 = np.zeros((1, 6), np.float32)
    got = run_score(kbx, labels, d2, pulls, rsum, t, 3)
    assert got["best_cluster_arm"][0] == 5 and got["best_arm"][0] == 4 * 2 + 1      # unplayed pair outranks
    assert got["cl_pulls"][0, 2, 1] == 1 and got["cl_mean"][0, 2, 1] == 0.5
    got = run_score(kbx, labels, d2, pulls, rsum, t, 3, keep=np.zeros((1, 6), np.uint32))
    assert got["best_arm"][0] == -1 and np.isneginf(got["best_val"][0]) and got["best_cluster_arm"][0] == -1
    assert np.all(np.isneginf(got["arm_index"]))


# ------------------------------------------------- prune + score in one pass
def run_tail(kbx, inp, labels, dist2, K, want_bound=True, want_arm_index=True, **prm):
    """kb_bandit_step_tail on the caller's labels / dist2: returns the host copies of everything it writes."""
    B, N, S = inp["pulls"].shape
    ws(kbx, B, N, 1, K, S)
    t = {"flops": dev(inp["flops"]), "bytes": dev(inp["bytes"]), "peak_flops": dev(inp["peak_flops"]),
         "peak_bw": dev(inp["peak_bw"]), "t_incumbent": dev(inp["t_inc"]), "t_cur": dev(inp["t_cur"]),
         "hsig": dev(inp["hsig"]), "target": dev(inp["target"]), "pulls": dev(inp["pulls"]),
         "reward_sum": dev(inp["reward_sum"]), "t": dev(inp["t"]), "labels": dev(labels), "dist2": dev(dist2),
         "keep": empty((B, N), torch.int32), "kept_count": empty((B,), torch.int32),
         "cl_pulls": empty((B, K, S)), "cl_mean": empty((B, K, S)), "cl_index": empty((B, K, S)),
         "best_arm": empty((B,), torch.int32), "best_val": empty((B,)), "best_cluster_arm": empty((B,), torch.int32)}
    if want_bound:
        t["bound"] = empty((B, N, S))
    if want_arm_index:
        t["arm_index"] = empty((B, N, S))
    dims = dict(B=B, N=N, D=1, K=K, S=S, R=inp["hsig"].shape[2], iters=0)
    params = dict(theta_sat=75.0, c=2.0, prior_pulls=1.0, prior_mean=0.5)
    params.update(prm)
    kbx.bandit_step_tail(dims, params, t)
    outs = ["keep", "kept_count", "bound", "cl_pulls", "cl_mean", "cl_index", "arm_index", "best_arm", "best_val",
            "best_cluster_arm"]
    return {k: host(t[k]) for k in outs if k in t}


@pytest.mark.parametrize("B,N,K,S,L,cap", [(1, 5000, 64, 32, 0.1, False), (2, 3001, 7, 8, 0.0, False),
                                           (1, 20011, 1024, 8, 0.1, True), (3, 1500, 256, 16, 0.3, False),
                                           (1, 1025, 3, 4, 0.0, True), (2, 40000, 130, 32, 0.1, False),
                                           (1, 300, 5, 8, 0.1, False), (2, 2000, 9, 13, 0.1, False)])
def test_step_tail_matches_prune_then_score(kbx, B, N, K, S, L, cap):
    """The fused tail (pruning on the statistics' pass) against the oracle's kb_prune followed by its
    kb_score_select, teacher-forced on the same labels and distances: keep bits exact outside the near-tie
    margin, kept_count = their population count, bound, the three cluster tables and the per-arm index
    element by element, both selections.  (S = 13 and N <= 1024 take the unfused / one-CTA forms: same rule.)"""
    cfg = wl.scaled(wl.CONFIGS["tiny"], B=B, N=N, S=S, K=K)
    inp = wl.make_inputs(cfg, seed=N + K)
    rng = np.random.default_rng(N * 7 + S)
    labels = rng.integers(0, max(1, K - 1), (B, N)).astype(np.int32)        # the last cluster stays empty
    dist2 = rng.uniform(0, 4, (B, N)).astype(np.float32)
    # some floors within a few ulp of the incumbent, on both sides, and a few exactly on it
    f = inp["flops"]
    tl = inp["t_inc"][:, None].astype(np.float64) * inp["peak_flops"][0].astype(np.float64)
    idx = rng.choice(N, min(N, 200), replace=False)
    f[:, idx] = (tl * (1 + rng.integers(-3, 4, (B, idx.size)) * 6e-8)).astype(np.float32)
    inp["bytes"][:, idx] = 1.0
    prm = dict(lipschitz_L=L, cap_with_bound=cap)
    got = run_tail(kbx, inp, labels, dist2, K, **prm)
    assert kbx.device_status() == 0
    p = oracle.prune(inp["flops"], inp["bytes"], inp["peak_flops"], inp["peak_bw"], inp["t_inc"], inp["t_cur"],
                     labels, inp["hsig"], inp["target"], 75.0, want_bound=True, want_margin=True)
    keep = got["keep"].view(np.uint32)
    ties = parity.keep_match(keep, p, S)
    assert int(got["kept_count"].view(np.uint32).astype(np.int64).sum()) == int(np.bitwise_count(keep).sum())
    assert np.array_equal(got["kept_count"].view(np.uint32), np.bitwise_count(keep).sum(axis=1).astype(np.uint32))
    parity.close(got["bound"], p["bound"], atol=1e-6, what="bound")
    s = oracle.score_select(labels, dist2, inp["pulls"], inp["reward_sum"], inp["t"], K, keep=keep,
                            bound=p["bound"] if cap else None, c=2.0, lipschitz_L=L, cap_with_bound=cap)
    assert np.array_equal(got["cl_pulls"], s["cl_pulls"])
    parity.close(got["cl_mean"], s["cl_mean"], atol=1e-6, what="cl_mean")
    parity.close(got["cl_index"], s["cl_index"], atol=1e-6, what="cl_index")
    if cap:
        # the cap is the GPU's own bound (within 1e-6 of the oracle's): compare against the oracle run on it
        s = oracle.score_select(labels, dist2, inp["pulls"], inp["reward_sum"], inp["t"], K, keep=keep,
                                bound=got["bound"], c=2.0, lipschitz_L=L, cap_with_bound=True)
    parity.close(got["arm_index"], s["arm_index"], atol=1e-6, what="arm_index")
    parity.select_match(got["best_arm"], got["best_val"], s, s["arm_index"])
    parity.cluster_select_match(got["best_cluster_arm"], s, s["cl_index"])
    # the optional outputs left out: same selections
    slim = run_tail(kbx, inp, labels, dist2, K, want_bound=cap, want_arm_index=False, **prm)
    assert np.array_equal(slim["keep"], got["keep"]) and np.array_equal(slim["best_cluster_arm"], got["best_cluster_arm"])
    parity.select_match(slim["best_arm"], slim["best_val"], s, s["arm_index"])
    print(f"[tail B={B} N={N} K={K} S={S}] keep-bit near-ties {ties}")


def test_step_tail_threshold_edges_and_bad_labels(kbx):
    """Strictness survives the fused arithmetic: a floor EQUAL to the incumbent is pruned, h == theta is pruned;
    a label outside [0, K) raises status bit 1, adds to no statistic and is pruned as cluster 0 would be."""
    N, K, S = 2048, 4, 4
    flops = np.full((1, N), 1e9, np.float32)
    flops[0, 1::2] = 2e9
    byts = np.ones((1, N), np.float32)
    pf, pb = np.full(S, 1e12, np.float32), np.full(S, 1e12, np.float32)
    tinc = np.array([np.float32(2e9) / np.float32(1e12)], np.float32)       # exactly the floor of the odd candidates
    hs = np.zeros((1, K, 3), np.float32)
    hs[0, 1, 0] = 75.0                                                      # cluster 1, resource 0: exactly theta
    hs[0, 2, 0] = np.nextafter(np.float32(75.0), np.float32(0))             # cluster 2: one ulp below
    labels = (np.arange(N) % 3).astype(np.int32)[None].copy()
    inp = dict(flops=flops, bytes=byts, peak_flops=pf, peak_bw=pb, t_inc=tinc, t_cur=np.full((1, N), 1.0, np.float32),
               hsig=hs, target=np.zeros(S, np.int32), pulls=np.ones((1, N, S), np.int32),
               reward_sum=np.full((1, N, S), 0.5, np.float32), t=np.array([1 + N * S], np.int32))
    got = run_tail(kbx, inp, labels, np.zeros((1, N), np.float32), K)
    keep = got["keep"].view(np.uint32)[0]
    want = np.where((np.arange(N) % 2 == 0) & (labels[0] != 1), 0xF, 0).astype(np.uint32)
    assert np.array_equal(keep, want)
    assert kbx.device_status() == 0
    bad = labels.copy()
    bad[0, 10], bad[0, 11] = K, -1
    got = run_tail(kbx, inp, bad, np.zeros((1, N), np.float32), K)
    assert kbx.device_status(raise_on_timeout=False) & 1
    kbx.clear_device_status()
    ok = np.ones(N, bool)
    ok[[10, 11]] = False
    ref = oracle.score_select(bad[:, ok], None, inp["pulls"][:, ok], inp["reward_sum"][:, ok], inp["t"], K)
    assert np.array_equal(got["cl_pulls"], ref["cl_pulls"])
    assert kbx.device_status() == 0


# ------------------------------------------------------------- whole step
STEP_CASES = {
    "tiny": wl.CONFIGS["tiny"],
    "medium": wl.CONFIGS["medium"],
    "large/32": wl.scaled(wl.CONFIGS["large"], N=8192 + 37, iters=6),
    "batched/64": wl.scaled(wl.CONFIGS["batched"], B=16),
    "contraction/1024": wl.scaled(wl.CONFIGS["contraction"], N=4096 + 11, iters=3),
}


def run_step(kbx, cfg, inp, host_buffers=False):
    from paper_2511_18868_b200 import kb
    dims = dict(B=cfg.B, N=cfg.N, D=cfg.D, K=cfg.K, S=cfg.S, R=wl.R_RESOURCES, iters=cfg.iters)
    params = dict(theta_sat=float(inp["theta_sat"]), c=float(inp["c"]), lipschitz_L=float(inp["lipschitz_L"]),
                  prior_pulls=float(inp["prior_pulls"]), prior_mean=float(inp["prior_mean"]))
    if host_buffers:
        kbx.ensure_workspace(kbx.step_workspace_bytes(cfg.B, cfg.N, cfg.D, cfg.K, cfg.S, wl.R_RESOURCES))
        t = kb.step_tensors(inp, None, pinned_host=True)
        kbx.bandit_step_host(dims, params, t)
        return {k: v.numpy() for k, v in t.items()}
    ws(kbx, cfg.B, cfg.N, cfg.D, cfg.K, cfg.S)
    t = kb.step_tensors(inp, kbx.device)
    kbx.bandit_step(dims, params, t)
    return {k: host(v) for k, v in t.items()}


@pytest.mark.parametrize("name", list(STEP_CASES))
def test_step_teacher_forced(kbx, name):
    """Each call of the step is fed the oracle's inputs for that call."""
    cfg = STEP_CASES[name]
    inp = wl.make_inputs(cfg)
    ref = oracle.bandit_step(inp, cfg.iters)
    B, N, D, K, S = cfg.B, cfg.N, cfg.D, cfg.K, cfg.S
    ws(kbx, B, N, D, K, S)
    z = empty((B, N, D))
    kbx.normalize(dev(inp["x"]), z)
    parity.close(host(z), ref["z"], atol=2e-5, what="z")
    # one Lloyd iteration from the oracle's z and its last-but-one centroids
    zr = ref["z"]
    c_prev = oracle.init_centroids(zr, inp["init_rows"])
    cd = empty((B, K, D))
    kbx.init_centroids(dev(zr), dev(inp["init_rows"]), cd)
    assert np.array_equal(host(cd), c_prev)
    for _ in range(2):
        a_ref = oracle.cluster_assign(zr, c_prev, want_margins=True)
        labels, d2 = empty((B, N), torch.int32), empty((B, N))
        kbx.cluster_assign(dev(zr), dev(c_prev), labels, d2)
        parity.labels_match(zr, c_prev, host(labels), a_ref)
        c_next, n_ref = oracle.cluster_update(zr, a_ref["labels"], c_prev)
        cd, counts = dev(c_prev), empty((B, K), torch.int32)
        kbx.cluster_update(dev(zr), dev(a_ref["labels"]), cd, counts)
        assert np.array_equal(host(counts), n_ref)
        parity.close(host(cd), c_next, atol=1e-5, what="centroids")
        c_prev = c_next
    # final assign on the oracle's final centroids
    a_ref = oracle.cluster_assign(zr, ref["centroids"], want_margins=True)
    labels, d2, inertia, rep = empty((B, N), torch.int32), empty((B, N)), empty((B,)), empty((B, K), torch.int32)
    kbx.cluster_assign(dev(zr), dev(ref["centroids"]), labels, d2, inertia, rep)
    ties = parity.labels_match(zr, ref["centroids"], host(labels), a_ref)
    same = host(labels) == a_ref["labels"]
    parity.close(host(d2)[same], a_ref["dist2"][same], atol=1e-7, what="dist2")
    parity.close(host(inertia), a_ref["inertia"], atol=1e-6, what="inertia")
    parity.rep_match(host(rep), a_ref, a_ref["dist2"], a_ref["labels"])
    # prune and score on the oracle's labels / dist2
    p_ref = oracle.prune(inp["flops"], inp["bytes"], inp["peak_flops"], inp["peak_bw"], inp["t_inc"], inp["t_cur"],
                         ref["labels"], inp["hsig"], inp["target"], 75.0, want_bound=True, want_margin=True)
    keep, kept, bd = empty((B, N), torch.int32), empty((B,), torch.int32), empty((B, N, S))
    kbx.prune(dev(inp["flops"]), dev(inp["bytes"]), dev(inp["peak_flops"]), dev(inp["peak_bw"]), dev(inp["t_inc"]),
              keep, t_cur=dev(inp["t_cur"]), labels=dev(ref["labels"]), hsig=dev(inp["hsig"]),
              target=dev(inp["target"]), theta_sat=75.0, kept_count=kept, bound=bd)
    parity.keep_match(host(keep).view(np.uint32), p_ref, S)
    parity.close(host(bd), p_ref["bound"], atol=1e-6, what="bound")
    prm = dict(c=2.0, lipschitz_L=float(inp["lipschitz_L"]), prior_pulls=1.0, prior_mean=0.5)
    got = run_score(kbx, ref["labels"], ref["dist2"], inp["pulls"], inp["reward_sum"], inp["t"], K,
                    keep=p_ref["keep"], **prm)
    s_ref = oracle.score_select(ref["labels"], ref["dist2"], inp["pulls"], inp["reward_sum"], inp["t"], K,
                                keep=p_ref["keep"], **prm)
    assert np.array_equal(got["cl_pulls"], s_ref["cl_pulls"])
    parity.close(got["cl_mean"], s_ref["cl_mean"], atol=1e-6, what="cl_mean")
    parity.close(got["cl_index"], s_ref["cl_index"], atol=1e-6, what="cl_index")
    parity.close(got["arm_index"], s_ref["arm_index"], atol=1e-6, what="arm_index")
    parity.select_match(got["best_arm"], got["best_val"], s_ref, s_ref["arm_index"])
    parity.cluster_select_match(got["best_cluster_arm"], s_ref, s_ref["cl_index"])
    print(f"[{name}] final-assign near-ties: {ties}")


@pytest.mark.parametrize("name", list(STEP_CASES))
@pytest.mark.parametrize("host_buffers", [False, True])
def test_step_free_running(kbx, name, host_buffers):
    """The whole step through kb_bandit_step(_host) against the oracle's whole step.
    A single near-tie flip moves a centroid and cascades, so exact label equality after
    many iterations is not demanded: the objective must agree and the final labels must
    be optimal for the final centroids."""
    cfg = STEP_CASES[name]
    inp = wl.make_inputs(cfg)
    ref = oracle.bandit_step(inp, cfg.iters)
    got = run_step(kbx, cfg, inp, host_buffers)
    parity.close(got["z"], ref["z"], atol=2e-5, what="z")
    parity.close(got["inertia"], ref["inertia"], atol=0, rtol=1e-3, what="inertia")
    agree = np.mean(got["labels"] == ref["labels"])
    assert agree > 0.99, f"label agreement {agree}"
    # self-consistency in double: labels are optimal for the returned centroids
    a_chk = oracle.cluster_assign(got["z"], got["centroids"], want_margins=True)
    parity.labels_match(got["z"], got["centroids"], got["labels"], a_chk)
    same = got["labels"] == a_chk["labels"]
    parity.close(got["dist2"][same], a_chk["dist2"][same], atol=1e-7, what="dist2")
    assert np.array_equal(got["counts"].sum(1), np.full(cfg.B, cfg.N))
    # prune / score consistent with the GPU's own labels and dist2
    p_chk = oracle.prune(inp["flops"], inp["bytes"], inp["peak_flops"], inp["peak_bw"], inp["t_inc"], inp["t_cur"],
                         got["labels"], inp["hsig"], inp["target"], 75.0, want_bound=True, want_margin=True)
    parity.keep_match(got["keep"].view(np.uint32), p_chk, cfg.S)
    parity.close(got["bound"], p_chk["bound"], atol=1e-6, what="bound")
    assert np.array_equal(got["kept_count"].view(np.uint32),
                          np.bitwise_count(got["keep"].view(np.uint32)).sum(axis=1).astype(np.uint32))
    s_chk = oracle.score_select(got["labels"], got["dist2"], inp["pulls"], inp["reward_sum"], inp["t"], cfg.K,
                                keep=got["keep"].view(np.uint32), c=2.0, lipschitz_L=float(inp["lipschitz_L"]))
    assert np.array_equal(got["cl_pulls"], s_chk["cl_pulls"])
    parity.close(got["cl_mean"], s_chk["cl_mean"], atol=1e-6, what="cl_mean")
    parity.close(got["cl_index"], s_chk["cl_index"], atol=1e-6, what="cl_index")
    parity.close(got["arm_index"], s_chk["arm_index"], atol=1e-6, what="arm_index")
    parity.select_match(got["best_arm"], got["best_val"], s_chk, s_chk["arm_index"])
    parity.cluster_select_match(got["best_cluster_arm"], s_chk, s_chk["cl_index"])
    print(f"[{name}] label agreement with the free-running oracle: {agree:.6f}")


@pytest.mark.parametrize("B,N,D,K,S", [(3, 300, 16, 5, 8), (2, 512, 32, 16, 32), (5, 77, 64, 9, 4), (4, 200, 32, 7, 16),
                                       (36, 512, 16, 6, 16)])
@pytest.mark.parametrize("host_buffers", [False, True])
def test_step_small_instances_one_launch(kbx, B, N, D, K, S, host_buffers):
    """Instances of at most 512 rows go from raw features to labels in ONE launch inside the whole-step drivers
    (normalisation and the gather of the initial centroids happen in the clustering kernel), and a second launch
    prunes, scores and selects.  Columns that are constant, far from zero or of tiny spread must normalise as
    kb_normalize does; with no Lloyd iteration the centroids are exactly the named rows of z; keep bits, cluster
    tables, per-arm indices and both selections must be what the oracle derives from the GPU's own labels."""
    for iters in (0, 4):
        cfg = wl.scaled(wl.CONFIGS["tiny"], B=B, N=N, D=D, K=K, S=S, iters=iters)
        inp = wl.make_inputs(cfg, seed=B * 1000 + N)
        x = inp["x"]
        x[:, :, 0] = 3.25                                  # constant column: only centred
        x[:, :, 1] = x[:, :, 1] * 0.5 + 1.0e4              # far from zero
        x[:, :, 2] = x[:, :, 2] * 1.0e-3                   # tiny spread
        launches0 = kbx.launch_count()[0]
        got = run_step(kbx, cfg, inp, host_buffers)
        launches = kbx.launch_count()[0] - launches0
        assert kbx.device_status() == 0
        # (from host buffers a gain bound of a megabyte or more is computed early, beside the clustering: one more)
        early = int(host_buffers and B * N * S * 4 >= 1 << 20)
        assert launches == 2 + early, f"{launches} kernels: the step did not run as two launches"
        zr, _, _ = oracle.normalize(x)
        parity.close(got["z"], zr, atol=2e-5, what="z")
        assert np.all(got["z"][:, :, 0] == 0.0)
        if iters == 0:
            c0 = np.stack([got["z"][b, inp["init_rows"][b]] for b in range(B)])
            np.testing.assert_array_equal(got["centroids"], c0)
        chk = oracle.cluster_assign(got["z"], got["centroids"], want_margins=True)
        parity.labels_match(got["z"], got["centroids"], got["labels"], chk)
        same = got["labels"] == chk["labels"]
        parity.close(got["dist2"][same], chk["dist2"][same], atol=1e-7, what="dist2")
        parity.close(got["inertia"], chk["inertia"], atol=1e-6, what="inertia")
        p_chk = oracle.prune(inp["flops"], inp["bytes"], inp["peak_flops"], inp["peak_bw"], inp["t_inc"], inp["t_cur"],
                             got["labels"], inp["hsig"], inp["target"], 75.0, want_bound=True, want_margin=True)
        keep = got["keep"].view(np.uint32)
        ties = parity.keep_match(keep, p_chk, S)
        pop = sum(int(v).bit_count() for v in keep.reshape(-1))
        assert int(got["kept_count"].view(np.uint32).sum()) == pop and abs(pop - int(p_chk["kept_count"].sum())) <= ties
        parity.close(got["bound"], p_chk["bound"], atol=1e-6, what="bound")
        s_chk = oracle.score_select(got["labels"], got["dist2"], inp["pulls"], inp["reward_sum"], inp["t"], K,
                                    keep=keep, c=2.0, lipschitz_L=float(inp["lipschitz_L"]))
        parity.close(got["cl_pulls"], s_chk["cl_pulls"], atol=1e-6, what="cl_pulls")
        parity.close(got["cl_mean"], s_chk["cl_mean"], atol=1e-6, what="cl_mean")
        parity.close(got["cl_index"], s_chk["cl_index"], atol=1e-6, what="cl_index")
        parity.close(got["arm_index"], s_chk["arm_index"], atol=1e-6, what="arm_index")
        parity.select_match(got["best_arm"], got["best_val"], s_chk, s_chk["arm_index"])
        parity.cluster_select_match(got["best_cluster_arm"], s_chk, s_chk["cl_index"])


@pytest.mark.parametrize("N,D,K", [(5000, 16, 8), (20011, 32, 64), (40000, 64, 40)])
@pytest.mark.parametrize("host_buffers", [False, True])
def test_step_mid_sized_instance_one_launch(kbx, N, D, K, host_buffers):
    """One mid-sized instance goes from raw features to labels in one cooperative launch inside the whole-step
    drivers (column statistics across all CTAs, z written once, the seeding rows fetched before z may overwrite
    x in place).  z must be what kb_normalize gives, also for constant, offset and tiny-spread columns; with no
    Lloyd iteration the centroids are exactly the named rows of z."""
    for iters in (0, 3):
        cfg = wl.scaled(wl.CONFIGS["medium"], N=N, D=D, K=K, components=max(4, K // 2), S=8, iters=iters)
        inp = wl.make_inputs(cfg, seed=N + D)
        x = inp["x"]
        x[:, :, 0] = -7.5
        x[:, :, 1] = x[:, :, 1] * 0.5 + 1.0e4
        x[:, :, 2] = x[:, :, 2] * 1.0e-3
        launches0 = kbx.launch_count()[0]
        got = run_step(kbx, cfg, inp, host_buffers)
        launches = kbx.launch_count()[0] - launches0
        assert kbx.device_status() == 0
        # (the host-buffer form adds one when the gain bound is a megabyte or more: it is computed early, beside
        # the clustering)
        assert launches <= 7 + int(host_buffers), \
            f"{launches} kernels: the clustering part did not run as one cooperative launch"
        zr, _, _ = oracle.normalize(x)
        parity.close(got["z"], zr, atol=2e-5, what="z")
        assert np.all(got["z"][:, :, 0] == 0.0)
        if iters == 0:
            np.testing.assert_array_equal(got["centroids"][0], got["z"][0, inp["init_rows"][0]])
        chk = oracle.cluster_assign(got["z"], got["centroids"], want_margins=True)
        parity.labels_match(got["z"], got["centroids"], got["labels"], chk)
        same = got["labels"] == chk["labels"]
        parity.close(got["dist2"][same], chk["dist2"][same], atol=1e-7, what="dist2")
        parity.close(got["inertia"], chk["inertia"], atol=1e-6, what="inertia")


@pytest.mark.parametrize("N,D,K,iters", [(16384, 32, 64, 20), (5000, 16, 8, 7), (1025, 64, 100, 3), (40000, 32, 17, 4),
                                         (2048, 32, 64, 0)])
def test_cluster_fit_cooperative(kbx, N, D, K, iters):
    """One mid-sized instance: kb_cluster_fit runs the whole Lloyd loop in one cooperative launch.  Its result
    must be a Lloyd fixed-point sequence like the call-by-call path's: same objective, labels optimal for the
    returned centroids (checked in double), counts, representative members and inertia consistent with them."""
    cfg = wl.scaled(wl.CONFIGS["medium"], N=N, D=D, K=K, components=max(4, K // 2), S=2, iters=iters)
    inp = wl.make_inputs(cfg, seed=N + K)
    z, _, _ = oracle.normalize(inp["x"])
    c0 = oracle.init_centroids(z, inp["init_rows"])
    ws(kbx, 1, N, D, K, 2)
    out = {}
    for path in (0, 1):                      # 0: automatic (cooperative launch), 1: assign/update calls, fp32 kernels
        kbx.set_assign_options(path=path)
        try:
            c = dev(c0.copy())
            labels, d2 = empty((1, N), torch.int32), empty((1, N))
            inertia, rep, counts = empty((1,)), empty((1, K), torch.int32), empty((1, K), torch.int32)
            kbx.cluster_fit(dev(z), c, labels, iters, dist2=d2, inertia=inertia, rep=rep, counts=counts)
        finally:
            kbx.set_assign_options(path=0)
        out[path] = dict(c=host(c), labels=host(labels), d2=host(d2), inertia=host(inertia), rep=host(rep),
                         counts=host(counts))
    assert kbx.device_status() == 0
    got, ref = out[0], out[1]
    parity.close(got["inertia"], ref["inertia"], atol=0, rtol=1e-3, what="inertia")
    assert np.mean(got["labels"] == ref["labels"]) > 0.99
    # self-consistency in double against the returned centroids
    chk = oracle.cluster_assign(z, got["c"], want_margins=True, want_rep=True)
    parity.labels_match(z, got["c"], got["labels"], chk)
    same = got["labels"] == chk["labels"]
    parity.close(got["d2"][same], chk["dist2"][same], atol=1e-7, what="dist2")
    parity.close(got["inertia"], chk["inertia"], atol=1e-6, what="inertia vs own labels")
    if iters > 0:
        assert got["counts"].sum() == N
        assert np.abs(got["counts"] - ref["counts"]).sum() <= 0.02 * N      # sizes at the last update
    else:
        assert np.all(got["counts"] == 0)
        np.testing.assert_array_equal(got["c"], c0)
    parity.rep_match(got["rep"], chk, chk["dist2"], chk["labels"])


@pytest.mark.parametrize("D,K", [(32, 64), (16, 9), (64, 40)])
def test_cluster_fit_cooperative_ties_and_empty_clusters(kbx, D, K):
    """The cooperative fit splits a row's centroid scan over several threads: duplicate centroids that fall into
    different parts must still resolve to the lowest id, and a centroid that attracts no row keeps its
    coordinates, reports count 0 and representative -1."""
    N = 3000
    rng = np.random.default_rng(D * 100 + K)
    z = rng.standard_normal((1, N, D)).astype(np.float32)
    c0 = z[:, rng.choice(N, K, replace=False)].copy()
    c0[0, K - 1] = c0[0, 0]                       # duplicate of centroid 0 in the last part: must never win
    c0[0, K // 2] = c0[0, 1]                      # duplicate of centroid 1 in a middle part
    far = K // 3
    c0[0, far] = 1e3                              # attracts no row
    ws(kbx, 1, N, D, K, 2)
    for iters in (0, 3):
        c = dev(c0.copy())
        labels, d2 = empty((1, N), torch.int32), empty((1, N))
        inertia, rep, counts = empty((1,)), empty((1, K), torch.int32), empty((1, K), torch.int32)
        kbx.cluster_fit(dev(z), c, labels, iters, dist2=d2, inertia=inertia, rep=rep, counts=counts)
        assert kbx.device_status() == 0
        lab, cg = host(labels), host(c)
        assert not np.any(lab == far)
        np.testing.assert_array_equal(cg[0, far], c0[0, far])
        assert host(rep)[0, far] == -1
        if iters == 0:
            # (after an update the originals move and their untouched duplicates become centroids of their own)
            assert not np.any(lab == K - 1) and not np.any(lab == K // 2)
            assert host(rep)[0, K - 1] == -1 and host(rep)[0, K // 2] == -1
        else:
            cnt = host(counts)
            assert cnt[0, far] == 0 and cnt.sum() == N
        chk = oracle.cluster_assign(z, cg, want_margins=True, want_rep=True)
        parity.labels_match(z, cg, lab, chk)
        parity.close(host(inertia), chk["inertia"], atol=1e-6, what="inertia")


@pytest.mark.parametrize("B,N,D,K,iters", [(1, 8229, 64, 256, 4), (3, 5000, 32, 128, 3), (1, 20011, 64, 130, 2),
                                           (1, 6000, 64, 640, 2), (1, 45000, 64, 384, 2)])
def test_cluster_fit_presplit(kbx, B, N, D, K, iters):
    """A fit on the tensor path converts Z to its fp16 pieces once and every assignment of the loop multiplies out of
    that image.  Its result must agree with the same loop made of single calls (which split rows on the fly), and
    the final labels must be optimal for the returned centroids (checked in double)."""
    cfg = wl.scaled(wl.CONFIGS["large"], B=B, N=N, D=D, K=K, components=max(4, K // 2), S=2, iters=iters)
    inp = wl.make_inputs(cfg, seed=N + K)
    z, _, _ = oracle.normalize(inp["x"])
    c0 = oracle.init_centroids(z, inp["init_rows"])
    ws(kbx, B, N, D, K, 2)
    zd = dev(z)

    def outputs():
        return dict(labels=empty((B, N), torch.int32), d2=empty((B, N)), inertia=empty((B,)),
                    rep=empty((B, K), torch.int32), counts=empty((B, K), torch.int32))

    fit, c_fit = outputs(), dev(c0.copy())
    kbx.cluster_fit(zd, c_fit, fit["labels"], iters, dist2=fit["d2"], inertia=fit["inertia"], rep=fit["rep"],
                    counts=fit["counts"])
    assert kbx.assign_path() == 2 and kbx.assign_presplit()
    one, c_one = outputs(), dev(c0.copy())
    for _ in range(iters):
        kbx.cluster_assign(zd, c_one, one["labels"])
        assert kbx.assign_path() == 2 and not kbx.assign_presplit()
        kbx.cluster_update(zd, one["labels"], c_one, one["counts"])
    kbx.cluster_assign(zd, c_one, one["labels"], one["d2"], one["inertia"], one["rep"])
    assert kbx.device_status() == 0
    got = {k: host(v) for k, v in fit.items()}
    ref = {k: host(v) for k, v in one.items()}
    assert np.mean(got["labels"] == ref["labels"]) > 0.995
    parity.close(got["inertia"], ref["inertia"], atol=0, rtol=1e-3, what="inertia")
    assert np.abs(got["counts"] - ref["counts"]).sum() <= 0.02 * B * N
    cg = host(c_fit)
    chk = oracle.cluster_assign(z, cg, want_margins=True, want_rep=True)
    parity.labels_match(z, cg, got["labels"], chk)
    same = got["labels"] == chk["labels"]
    parity.close(got["d2"][same], chk["dist2"][same], atol=1e-7, what="dist2")
    parity.close(got["inertia"], chk["inertia"], atol=1e-6, what="inertia vs own labels")
    parity.rep_match(got["rep"], chk, chk["dist2"], chk["labels"])


def test_argument_errors(kbx):
    from paper_2511_18868_b200.kb import KbError
    z = empty((1, 8, 4))
    with pytest.raises(KbError) as e:
        kbx.cluster_assign(z, empty((1, 2, 4)), None)
    assert e.value.status == 1
    with pytest.raises(KbError) as e:
        kbx.prune(empty((1, 8)), empty((1, 8)), empty((33,)), empty((33,)), empty((1,)), empty((1, 8), torch.int32))
    assert e.value.status == 2
    saved = kbx._ws
    kbx.set_workspace(None)
    with pytest.raises(KbError) as e:
        kbx.cluster_update(z, empty((1, 8), torch.int32), empty((1, 2, 4)))
    assert e.value.status == 3
    kbx.set_workspace(saved)
    assert kbx.device_status() == 0


# ------------------------------------------------- tensor-core assign path
TC_CASES = [(1, 4096, 32, 128), (1, 5000, 64, 256), (2, 3000, 128, 200), (1, 4097, 96, 1024), (3, 1111, 64, 130),
            (1, 20000, 128, 1024),
            # several row tiles per CTA: one accumulator tile per row tile with the B image resident; three per row
            # tile (their parity alternates from row tile to row tile) through the ring, two and three k-blocks
            (1, 60000, 64, 128), (1, 50000, 128, 384), (1, 40000, 96, 384)]


@pytest.mark.parametrize("path", [2, 3], ids=["f16x3", "tf32x3"])
@pytest.mark.parametrize("B,N,D,K", TC_CASES)
def test_assign_tensor_path(kbx, B, N, D, K, path):
    """kb_cluster_assign forced onto the tcgen05 kernel (fp16 or tf32 split): same rules as the fp32 path."""
    cfg = wl.scaled(wl.CONFIGS["large"], B=B, N=N, D=D, K=K, components=max(8, K // 2), S=2)
    inp = wl.make_inputs(cfg, seed=N + K)
    z, _, _ = oracle.normalize(inp["x"])
    rng = np.random.default_rng(K)
    c = z[:, rng.choice(N, K, replace=False)] + (0.02 * rng.standard_normal((B, K, D))).astype(np.float32)
    c[:, K - 1] = c[:, 0]                       # exact duplicate: gap 0, resolved by the exact re-evaluation
    ws(kbx, B, N, D, K, 1)
    kbx.set_assign_options(path=path)
    try:
        labels, d2, inertia, rep = empty((B, N), torch.int32), empty((B, N)), empty((B,)), empty((B, K), torch.int32)
        kbx.cluster_assign(dev(z), dev(c), labels, d2, inertia, rep)
        assert kbx.assign_path() == path
        approx, flagged, lab2 = empty((B, N)), empty((2,), torch.int32), empty((B, N), torch.int32)
        kbx.assign_tc_probe(dev(z), dev(c), lab2, approx, flagged)
    finally:
        kbx.set_assign_options(path=0)
    assert kbx.device_status() == 0
    ref = oracle.cluster_assign(z, c, want_margins=True)
    got = host(labels)
    ties = parity.labels_match(z, c, got, ref)
    assert not np.any(got == K - 1)
    assert np.array_equal(host(lab2), got)
    same = got == ref["labels"]
    parity.close(host(d2)[same], ref["dist2"][same], atol=1e-7, what="dist2")
    parity.close(host(inertia), ref["inertia"], atol=1e-6, what="inertia")
    parity.rep_match(host(rep), ref, ref["dist2"], ref["labels"])
    # how far the ranked (expanded-form, 3xTF32) distance is from the exact one
    xn = (z.astype(np.float64) ** 2).sum(-1)
    cnn = (c.astype(np.float64) ** 2).sum(-1)
    # the fp16 split shares one power-of-two scale among an instance's centroids: its error is relative to
    # the largest centroid norm of the instance; the tf32 split's to the chosen centroid's
    scale = xn + (cnn.max(axis=1, keepdims=True) if path == 2 else
                  np.take_along_axis(cnn, ref["labels"].astype(np.int64), axis=1))
    # (the ranked value also drops its low 7 mantissa bits, which hold the column index: up to 2^-16 of itself,
    # a term the kernel's near-tie bound adds on top of eps)
    err = (np.abs(host(approx).astype(np.float64) - ref["best"]) - ref["best"] / 65536)[same] / scale[same]
    frac, frac_full = host(flagged) / (B * N)
    print(f"[tc path={path} B={B} N={N} D={D} K={K}] near-ties={ties} pair-checked={frac:.5f} "
          f"fully re-evaluated={frac_full:.5f} max (|d2_ranked - d2_exact| - 2^-16 d2) / (|z|^2+|c|^2) = {err.max():.3e} "
          f"(eps = {1 / 65536:.3e})")
    assert err.max() < 0.25 / 65536               # the re-evaluation bound covers the ranking error with margin


@pytest.mark.parametrize("path", [2, 3], ids=["f16x3", "tf32x3"])
@pytest.mark.parametrize("scale", [1e-6, 1.0, 3e4], ids=["tiny", "unit", "huge"])
def test_assign_tensor_path_value_ranges(kbx, path, scale):
    """The fp16 split scales rows and centroids by exact powers of two: data of any magnitude, rows far
    outside the centroids' range, zero rows and a zero centroid must all come out like the fp32 definition."""
    B, N, D, K = 1, 6000, 64, 256
    cfg = wl.scaled(wl.CONFIGS["large"], B=B, N=N, D=D, K=K, components=96, S=2)
    z, _, _ = oracle.normalize(wl.make_inputs(cfg, seed=17)["x"])
    rng = np.random.default_rng(5)
    c = z[:, rng.choice(N, K, replace=False)].copy()
    z = z.copy()
    z[0, 10:20] *= 1e5            # rows five orders of magnitude beyond every centroid
    z[0, 20:24] *= 1e9            # ... and far outside what fp16 can scale to
    z[0, 30:34] = 0.0             # zero rows
    z[0, 40:44] *= 1e-7           # rows far smaller than the centroids
    c[0, 7] = 0.0                 # a centroid at the origin
    z, c = (z * np.float32(scale)).astype(np.float32), (c * np.float32(scale)).astype(np.float32)
    ws(kbx, B, N, D, K, 1)
    kbx.set_assign_options(path=path)
    try:
        labels, d2 = empty((B, N), torch.int32), empty((B, N))
        kbx.cluster_assign(dev(z), dev(c), labels, d2)
        assert kbx.assign_path() == path
    finally:
        kbx.set_assign_options(path=0)
    assert kbx.device_status() == 0
    ref = oracle.cluster_assign(z, c, want_margins=True)
    got = host(labels)
    ties = parity.labels_match(z, c, got, ref)
    same = got == ref["labels"]
    parity.close(host(d2)[same], ref["dist2"][same], atol=1e-7 * scale * scale, what="dist2")
    print(f"[tc ranges path={path} scale={scale:g}] near-ties={ties}")


@pytest.mark.parametrize("scale", [1e-6, 1.0, 3e4], ids=["tiny", "unit", "huge"])
def test_cluster_fit_presplit_value_ranges(kbx, scale):
    """The same value ranges through a fit, whose assignments multiply out of the pre-split image of Z (rows scaled
    once, before the centroids' scale of an iteration is known): outlier rows, zero rows, tiny rows and a zero
    centroid must still end with labels that are optimal for the returned centroids."""
    B, N, D, K = 1, 6000, 64, 256
    cfg = wl.scaled(wl.CONFIGS["large"], B=B, N=N, D=D, K=K, components=96, S=2)
    z, _, _ = oracle.normalize(wl.make_inputs(cfg, seed=17)["x"])
    rng = np.random.default_rng(5)
    c0 = z[:, rng.choice(N, K, replace=False)].copy()
    z = z.copy()
    z[0, 10:20] *= 1e5
    z[0, 20:24] *= 1e9
    z[0, 30:34] = 0.0
    z[0, 40:44] *= 1e-7
    c0[0, 7] = 0.0
    z, c0 = (z * np.float32(scale)).astype(np.float32), (c0 * np.float32(scale)).astype(np.float32)
    ws(kbx, B, N, D, K, 1)
    for iters in (2, 3):
        c = dev(c0.copy())
        labels, d2, inertia = empty((B, N), torch.int32), empty((B, N)), empty((B,))
        counts = empty((B, K), torch.int32)
        kbx.cluster_fit(dev(z), c, labels, iters, dist2=d2, inertia=inertia, counts=counts)
        assert kbx.assign_path() == 2 and kbx.assign_presplit()
        assert kbx.device_status() == 0
        cg, got = host(c), host(labels)
        assert np.all(np.isfinite(cg)) and host(counts).sum() == N
        chk = oracle.cluster_assign(z, cg, want_margins=True)
        ties = parity.labels_match(z, cg, got, chk)
        same = got == chk["labels"]
        parity.close(host(d2)[same], chk["dist2"][same], atol=1e-7 * scale * scale, what="dist2")
        print(f"[presplit ranges scale={scale:g} iters={iters}] near-ties={ties}")


def test_step_uses_tensor_path_when_eligible(kbx):
    cfg = wl.scaled(wl.CONFIGS["large"], N=8192 + 37, iters=2)
    inp = wl.make_inputs(cfg)
    got = run_step(kbx, cfg, inp)
    assert kbx.assign_path() == 2
    a_chk = oracle.cluster_assign(got["z"], got["centroids"], want_margins=True)
    parity.labels_match(got["z"], got["centroids"], got["labels"], a_chk)


# -------------------------------------------------- within-cluster draw of k_t
# fp32 against double: theta - h is one rounding of a value below 128 (8e-6), the inner logf one ulp of a value
# whose logarithm is then taken (1.2e-7 absolute), the outer logf and the sum one ulp each of values below 128.
SAMPLE_TOL = 5e-5


def _sample_inputs(B, N, K, S, seed):
    rng = np.random.default_rng(seed)
    R = wl.R_RESOURCES
    labels = rng.integers(0, K, size=(B, N)).astype(np.int32)
    hsig = rng.uniform(0.0, 100.0, size=(B, K, R)).astype(np.float32)
    h_cand = wl.make_candidate_signatures(hsig, labels, seed + 1)
    target = (np.arange(S) % R).astype(np.int32)
    cluster_arm = rng.integers(0, K * S, size=(B,)).astype(np.int32)
    t = rng.integers(1, 100000, size=(B,)).astype(np.int32)
    return labels, h_cand, target, cluster_arm, t


def _run_sample(kbx, labels, h_cand, target, cluster_arm, t, K, theta, seed):
    B = labels.shape[0]
    member, val = empty((B,), torch.int32), empty((B,))
    kbx.sample_member(dev(labels), dev(cluster_arm), dev(h_cand), dev(target), dev(t), member, K, theta, seed, val)
    return host(member), host(val)


@pytest.mark.parametrize("B,N,K,S", [(1, 256, 8, 8), (3, 1000, 5, 4), (2, 20011, 64, 16), (1, 262144, 256, 32),
                                     (64, 512, 16, 16), (5, 1, 1, 1), (2, 8193, 3, 32), (1, 70001, 2, 2)])
def test_sample_member(kbx, B, N, K, S):
    labels, h_cand, target, cluster_arm, t = _sample_inputs(B, N, K, S, seed=B * 7 + N)
    ws(kbx, B, N, 16, K, S)
    seed = 0x9E3779B97F4A7C15 ^ N
    got, val = _run_sample(kbx, labels, h_cand, target, cluster_arm, t, K, 75.0, seed)
    ref = oracle.sample_member(labels, cluster_arm, h_cand, target, 75.0, seed, t, K)
    loose = parity.member_match(got, val, ref, SAMPLE_TOL)
    assert loose <= max(1, B // 50)
    assert kbx.device_status() == 0
    # the same seed and step repeat the draw; another step counter is another draw
    again, _ = _run_sample(kbx, labels, h_cand, target, cluster_arm, t, K, 75.0, seed)
    np.testing.assert_array_equal(again, got)
    if N >= 256:
        other, _ = _run_sample(kbx, labels, h_cand, target, cluster_arm, t + 1, K, 75.0, seed)
        ref2 = oracle.sample_member(labels, cluster_arm, h_cand, target, 75.0, seed, t + 1, K)
        parity.member_match(other, None, ref2, SAMPLE_TOL)


def test_sample_member_edge_cases(kbx):
    B, N, K, S = 8, 3000, 6, 4
    labels, h_cand, target, cluster_arm, t = _sample_inputs(B, N, K, S, seed=11)
    cluster_arm[0] = -1                                  # no pair chosen
    labels[1][labels[1] == cluster_arm[1] // S] = (cluster_arm[1] // S + 1) % K     # the chosen cluster is empty
    i2 = cluster_arm[2] // S
    labels[2][labels[2] == i2] = (i2 + 1) % K
    labels[2][1234] = i2                                 # exactly one member
    i3, c3 = cluster_arm[3] // S, target[cluster_arm[3] % S]
    m3 = np.flatnonzero(labels[3] == i3)
    h_cand[3, m3[: len(m3) // 2], c3] = np.nan           # half of the members cannot be drawn
    i4, c4 = cluster_arm[4] // S, target[cluster_arm[4] % S]
    m4 = np.flatnonzero(labels[4] == i4)
    h_cand[4, m4, c4] = np.nan                           # none can
    i5, c5 = cluster_arm[5] // S, target[cluster_arm[5] % S]
    h_cand[5, np.flatnonzero(labels[5] == i5), c5] = 42.0   # equal potentials: the perturbation alone decides
    i6, c6 = cluster_arm[6] // S, target[cluster_arm[6] % S]
    m6 = np.flatnonzero(labels[6] == i6)
    h_cand[6, m6[-1], c6] = -np.inf                      # an infinite potential wins outright
    h_cand[6, m6[0], c6] = np.inf                        # a potential of -inf is never drawn
    ws(kbx, B, N, 16, K, S)
    got, val = _run_sample(kbx, labels, h_cand, target, cluster_arm, t, K, 75.0, 5)
    ref = oracle.sample_member(labels, cluster_arm, h_cand, target, 75.0, 5, t, K)
    assert ref["member"][0] == -1 and ref["member"][1] == -1 and ref["member"][2] == 1234 and ref["member"][4] == -1
    assert ref["member"][6] == m6[-1]
    np.testing.assert_array_equal(got[[0, 1, 2, 4, 6]], ref["member"][[0, 1, 2, 4, 6]])
    assert np.isneginf(val[[0, 1, 4]]).all() and val[6] == np.inf
    for b in (3, 5, 7):
        parity.member_match(got[b:b + 1], val[b:b + 1],
                            {"member": ref["member"][b:b + 1], "pert": ref["pert"][b:b + 1]}, SAMPLE_TOL)
    assert got[3] not in set(m3[: len(m3) // 2].tolist())
    # zero instances, zero candidates
    kbx.sample_member(empty((0, 5), torch.int32), empty((0,), torch.int32), empty((0, 5, 3)), dev(target),
                      empty((0,), torch.int32), empty((0,), torch.int32), K, 75.0, 1)
    m = empty((2,), torch.int32)
    kbx.sample_member(empty((2, 0), torch.int32), dev(np.zeros(2, np.int32)), empty((2, 0, 3)), dev(target),
                      dev(np.ones(2, np.int32)), m, K, 75.0, 1)
    assert (host(m) == -1).all()
    assert kbx.device_status() == 0


def test_sample_member_frequencies(kbx):
    """A property that holds at any size: over many instances with the same candidates the drawn members follow
    exp(V) / sum exp(V), computed here from the definition."""
    M, n_mem, rounds = 50000, 6, 4              # 200 000 draws: four calls, each with its own step counters
    hm = np.array([70.0, 70.5, 71.0, 72.0, 69.25, 73.5], np.float32)
    N, K, S = 2 * n_mem + 1, 3, 4
    labels = np.zeros((M, N), np.int32)
    labels[:, 1::2] = 2
    labels[:, 0:2 * n_mem:2] = 1
    h = np.full((M, N, wl.R_RESOURCES), 1.0e3, np.float32)
    h[:, 0:2 * n_mem:2, 2] = hm
    h[:, 1::2, 2] = -1.0e3
    target = np.array([1, 0, 2, 1], np.int32)
    cluster_arm = np.full((M,), 1 * S + 2, np.int32)
    ws(kbx, M, N, 16, K, S)
    counts = np.zeros(n_mem, np.int64)
    for r in range(rounds):
        t = np.arange(1 + r * M, 1 + (r + 1) * M, dtype=np.int32)
        got, _ = _run_sample(kbx, labels, h, target, cluster_arm, t, K, 75.0, 2024)
        assert np.all(got % 2 == 0) and np.all(got < 2 * n_mem) and np.all(got >= 0)
        counts += np.bincount(got // 2, minlength=n_mem)
    V = 75.0 - hm.astype(np.float64)
    p = np.exp(V - V.max())
    p /= p.sum()
    freq = counts / (M * rounds)
    assert np.all(np.abs(freq - p) < 4.5 * np.sqrt(p * (1 - p) / (M * rounds))), (freq, p)


# -------------------------------------------------- outcome of an iteration
@pytest.mark.parametrize("B,N,S", [(1, 256, 8), (37, 1000, 3), (1024, 64, 16), (5, 1, 1)])
@pytest.mark.parametrize("failures_count", [False, True])
def test_record_outcome(kbx, B, N, S, failures_count):
    rng = np.random.default_rng(B + N + S)
    member = rng.integers(0, N, size=(B,)).astype(np.int32)
    member[rng.uniform(size=B) < 0.1] = -1
    arm = rng.integers(0, 4 * S, size=(B,)).astype(np.int32)
    t_cur = rng.uniform(0.5, 20.0, size=(B, N)).astype(np.float32)
    t_cur[rng.uniform(size=(B, N)) < 0.02] = 0.0
    base = t_cur[np.arange(B), np.maximum(member, 0)]
    t_new = (base * rng.uniform(0.0, 1.6, size=B)).astype(np.float32)   # gains and regressions
    t_new[rng.uniform(size=B) < 0.05] = np.nan
    verified = (rng.uniform(size=B) < 0.8).astype(np.int32)
    pulls = rng.poisson(2.0, size=(B, N, S)).astype(np.int32)
    rsum = (pulls * rng.uniform(0, 1, size=(B, N, S))).astype(np.float32)
    t = rng.integers(1, 1000, size=B).astype(np.int32)
    for ver in (None, verified):
        ref = oracle.record_outcome(member, arm, t_cur, t_new, pulls, rsum, t, verified=ver,
                                    failures_count=failures_count)
        p_d, r_d, t_d, rew = dev(pulls), dev(rsum), dev(t), empty((B,))
        kbx.record_outcome(dev(member), dev(arm), dev(t_cur), dev(t_new), p_d, r_d, t_d,
                           verified=None if ver is None else dev(ver), reward=rew, failures_count=failures_count)
        np.testing.assert_array_equal(host(p_d), ref["pulls"])
        np.testing.assert_array_equal(host(t_d), ref["t"])
        # the ratio is one fp32 division here, a double one rounded once in the oracle
        parity.close(host(rew), ref["reward"], atol=1e-7, what="reward")
        parity.close(host(r_d), ref["reward_sum"], atol=1e-6, what="reward_sum")
    assert kbx.device_status() == 0


@pytest.mark.parametrize("use_graph", [False, True])
def test_lockstep_loop_stays_on_device(kbx, use_graph):
    """B searches in lock-step: select the pair, draw k_t, observe a synthetic outcome, record it -- T iterations
    queued on one stream, no host read in between; with use_graph the iteration is captured once into a CUDA graph
    and replayed (the draw still changes from replay to replay: its counter holds t, which the graph itself
    advances).  Afterwards every iteration is checked against the oracle, fed the state the GPU had at that point
    (the copies below are queued on the same stream, outside the iteration)."""
    B, N, K, S, T = 6, 700, 5, 4, 25
    cfg = wl.scaled(wl.CONFIGS["medium"], B=B, N=N, D=16, K=K, components=5, S=S, iters=3)
    inp = wl.make_inputs(cfg, seed=5)
    rng = np.random.default_rng(9)
    labels = rng.integers(0, K, size=(B, N)).astype(np.int32)
    dist2 = rng.uniform(0, 4, size=(B, N)).astype(np.float32)
    h_cand = wl.make_candidate_signatures(inp["hsig"], labels, seed=3)
    gain = rng.uniform(-0.3, 0.6, size=(B, N, S)).astype(np.float32)     # the synthetic environment: L' = L (1 - gain)
    ws(kbx, B, N, 16, K, S)
    d = {k: dev(v) for k, v in dict(labels=labels, dist2=dist2, pulls=inp["pulls"], reward_sum=inp["reward_sum"],
                                    t=inp["t"], h_cand=h_cand, target=inp["target"], t_cur=inp["t_cur"],
                                    gain=gain).items()}
    cl = [empty((B, K, S)) for _ in range(3)]
    best_arm, best_val, pair = empty((B,), torch.int32), empty((B,)), empty((B,), torch.int32)
    member, reward = empty((B,), torch.int32), empty((B,))
    t_new = empty((B,))
    ar = torch.arange(B, device="cuda")

    def iteration():
        kbx.score_select(d["labels"], d["dist2"], d["pulls"], d["reward_sum"], d["t"], cl[0], cl[1], cl[2], best_arm,
                         best_val, pair, lipschitz_L=0.1)
        kbx.sample_member(d["labels"], pair, d["h_cand"], d["target"], d["t"], member, K, 75.0, 4242)
        # environment (test scaffolding, device-side): the runtime of the generated kernel
        k = member.clamp(min=0).long()
        s = (pair.clamp(min=0) % S).long()
        t_new.copy_(d["t_cur"][ar, k] * (1.0 - d["gain"][ar, k, s]))
        kbx.record_outcome(member, pair, d["t_cur"], t_new, d["pulls"], d["reward_sum"], d["t"], reward=reward)

    graph = None
    if use_graph:
        main = torch.cuda.current_stream()
        side = torch.cuda.Stream()
        side.wait_stream(main)
        kbx.set_stream(side)
        try:
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                iteration()
        finally:
            kbx.set_stream(main)
        main.wait_stream(side)
    trace = []
    for it in range(T):
        before = (d["pulls"].clone(), d["reward_sum"].clone(), d["t"].clone())
        if graph is not None:
            graph.replay()
        else:
            iteration()
        trace.append((before, pair.clone(), member.clone(), t_new.clone(), reward.clone(),
                      (d["pulls"].clone(), d["reward_sum"].clone(), d["t"].clone())))
    torch.cuda.synchronize()
    assert kbx.device_status() == 0
    drawn = 0
    for before, pair_g, member_g, t_new_g, reward_g, after in trace:
        p0, r0, t0 = (host(x) for x in before)
        sc = oracle.score_select(labels, dist2, p0, r0, t0, K, c=2.0, lipschitz_L=0.1)
        parity.cluster_select_match(host(pair_g), sc, sc["cl_index"])
        dr = oracle.sample_member(labels, host(pair_g), h_cand, inp["target"], 75.0, 4242, t0, K)
        parity.member_match(host(member_g), None, dr, SAMPLE_TOL)
        ro = oracle.record_outcome(host(member_g), host(pair_g), inp["t_cur"], host(t_new_g), p0, r0, t0)
        np.testing.assert_array_equal(host(after[0]), ro["pulls"])
        np.testing.assert_array_equal(host(after[2]), ro["t"])
        parity.close(host(after[1]), ro["reward_sum"], atol=1e-6, what="reward_sum")
        parity.close(host(reward_g), ro["reward"], atol=1e-7, what="reward")
        drawn += int((host(member_g) >= 0).sum())
    assert drawn == B * T
    # the loop moved: T pulls were added per instance, and the iteration counters advanced by T
    assert int(host(d["pulls"]).sum() - inp["pulls"].sum()) == B * T
    np.testing.assert_array_equal(host(d["t"]), inp["t"] + T)


# --------------------------------------------------------- k-means++ seeding
def _follow_seeding(z, rows, seed, tol=SAMPLE_TOL):
    """Every round's row must be the largest perturbed value ln(D^2) + G given the rows the GPU chose before (the
    oracle's double values; where its two largest are closer than the fp32 tolerance either is a valid draw)."""
    B, K = rows.shape
    loose = 0
    for j in range(K):
        o = oracle.kmeanspp_round(z, rows[:, :j], seed)
        for b in range(B):
            g = int(rows[b, j])
            assert 0 <= g < z.shape[1]
            if g != o["row"][b]:
                assert o["pert"][b, g] >= o["pert"][b, o["row"][b]] - tol, \
                    f"round {j}, instance {b}: drew {g} ({o['pert'][b, g]}), oracle {o['row'][b]} ({o['pert'][b, o['row'][b]]})"
                loose += 1
    return loose


@pytest.mark.parametrize("B,N,D,K", [(1, 256, 16, 8), (3, 1000, 20, 5), (2, 5003, 5, 7), (1, 40000, 64, 24),
                                     (40, 512, 32, 16), (2, 1, 8, 1), (1, 3000, 128, 3), (2, 700, 4, 4), (2, 333, 1, 3),
                                     (1, 900, 8, 5), (200, 300, 16, 6), (160, 1000, 5, 4), (150, 1024, 32, 8),
                                     (300, 7, 4, 7)])
def test_seed_kmeanspp(kbx, B, N, D, K):
    cfg = wl.scaled(wl.CONFIGS["medium"], B=B, N=N, D=D, K=max(K, 2), components=max(2, K), S=4, iters=1)
    x = wl.make_inputs(cfg, seed=N + K)["x"]
    z, _, _ = oracle.normalize(x)
    ws(kbx, B, N, D, K, 4)
    rows = empty((B, K), torch.int32)
    kbx.seed_kmeanspp(dev(z), rows, seed=2025 + N)
    got = host(rows)
    loose = _follow_seeding(z, got, 2025 + N)
    assert loose <= max(1, B * K // 50)
    if N >= K:
        assert all(len(set(r.tolist())) == K for r in got)          # distinct data: distinct seeds
    again = empty((B, K), torch.int32)
    kbx.seed_kmeanspp(dev(z), again, seed=2025 + N)
    np.testing.assert_array_equal(host(again), got)
    assert kbx.device_status() == 0


def test_seed_kmeanspp_properties(kbx):
    rng = np.random.default_rng(3)
    K, per, B = 6, 40, 300
    centres = 100.0 * np.stack([np.cos(2 * np.pi * np.arange(K) / K), np.sin(2 * np.pi * np.arange(K) / K)], 1)
    z = (centres[None, :, None, :] + rng.standard_normal((B, K, per, 2))).reshape(B, K * per, 2).astype(np.float32)
    ws(kbx, B, K * per, 2, K, 4)
    rows = empty((B, K), torch.int32)
    kbx.seed_kmeanspp(dev(z), rows, seed=99)
    got = host(rows)
    hit = np.mean([len(set(b)) == K for b in got // per])
    assert hit > 0.97, hit                                           # one seed per blob (uniform seeding: 1.5 %)
    _follow_seeding(z, got, 99)
    # fewer distinct rows than K: the surplus rounds draw uniformly, every row stays valid
    dup = np.zeros((50, 7, 4), np.float32)
    dup[:, 3:, :] = 1.0
    rows = empty((50, 4), torch.int32)
    ws(kbx, 50, 7, 4, 4, 4)
    kbx.seed_kmeanspp(dev(dup), rows, seed=5)
    r = host(rows)
    assert r.min() >= 0 and r.max() < 7
    assert np.all((r[:, 0] < 3) != (r[:, 1] < 3))
    _follow_seeding(dup, r, 5)
    # the rows feed the clustering: seeding, gather, fit on the device without a host read in between
    cfg = wl.scaled(wl.CONFIGS["medium"], B=2, N=6000, D=32, K=12, components=12, S=4, iters=5)
    zz, _, _ = oracle.normalize(wl.make_inputs(cfg, seed=8)["x"])
    ws(kbx, 2, 6000, 32, 12, 4)
    zd, rows, c = dev(zz), empty((2, 12), torch.int32), empty((2, 12, 32))
    labels, inertia = empty((2, 6000), torch.int32), empty((2,))
    kbx.seed_kmeanspp(zd, rows, seed=1)
    kbx.init_centroids(zd, rows, c)
    kbx.cluster_fit(zd, c, labels, 5, inertia=inertia)
    c0 = oracle.init_centroids(zz, host(rows))
    ref_c = c0
    for _ in range(5):
        a = oracle.cluster_assign(zz, ref_c, want_rep=False)
        ref_c, _ = oracle.cluster_update(zz, a["labels"], ref_c)
    a = oracle.cluster_assign(zz, ref_c, want_rep=False)
    parity.close(host(inertia), a["inertia"], atol=0, rtol=1e-3, what="inertia after seeded fit")
    assert kbx.device_status() == 0


# ------------------------------------------------------------ cluster radius
@pytest.mark.parametrize("B,N,K", [(1, 256, 8), (3, 1000, 5), (2, 20011, 64), (1, 262144, 256), (64, 512, 16),
                                   (1, 50000, 9000), (2, 0, 4), (4, 1, 3)])
def test_cluster_radius(kbx, B, N, K):
    rng = np.random.default_rng(B * 31 + N + K)
    labels = rng.integers(0, K, size=(B, N)).astype(np.int32)
    if N > 10:
        labels[labels == 1] = 0                          # an empty cluster
    dist2 = (rng.standard_normal((B, N)) ** 2 * rng.uniform(0.01, 50)).astype(np.float32)
    if N > 10:
        dist2[:, 3] = 0.0
        dist2[:, 5] = np.nan
    radius = empty((B, K))
    kbx.cluster_radius(dev(labels), dev(dist2), radius)
    ref = oracle.cluster_radius(labels, dist2, K)
    # one correctly rounded fp32 square root against a double one rounded once more: at most an ulp apart
    parity.close(host(radius), ref, atol=0, rtol=2e-7, what="radius")
    if N > 10 and K > 1:
        assert np.all(host(radius)[:, 1] == 0.0)
    assert kbx.device_status() == 0


@pytest.mark.parametrize("on_tables", [False, True])
def test_online_loop_regret_against_theorem1(kbx, on_tables):
    """An empirical look at Theorem 1 with everything on the device: B lock-step searches over a fixed frontier
    whose mean reward is Lipschitz in the (2-D) features, T iterations of select -> draw -> record.  The average
    regret must fall over the run and end below C sqrt(K |S| ln T / T) + L max_i diam(C_i), with the diameter
    bounded by twice the radius kb_cluster_radius reports and C = 1 (the theorem leaves C open; measured: average
    regret 0.15 against a bound of 0.83, first quarter 0.21, last quarter 0.11)."""
    B, K, S, per, T = 16, 4, 4, 100, 1200
    N = K * per
    rng = np.random.default_rng(17)
    centres = 3.0 * np.stack([np.cos(2 * np.pi * np.arange(K) / K), np.sin(2 * np.pi * np.arange(K) / K)], 1)
    z = (centres[None, :, None, :] + 0.25 * rng.standard_normal((B, K, per, 2))).reshape(B, N, 2).astype(np.float32)
    labels = np.tile(np.repeat(np.arange(K), per), (B, 1)).astype(np.int32)
    cent = np.stack([[z[b][labels[b] == i].mean(0) for i in range(K)] for b in range(B)]).astype(np.float32)
    dist2 = ((z - cent[np.arange(B)[:, None], labels]) ** 2).sum(-1).astype(np.float32)
    w = rng.standard_normal((S, 2))
    w = 0.8 * w / np.linalg.norm(w, axis=1, keepdims=True)                  # |w_s| = 0.8
    mu = (0.5 + 0.3 * np.tanh(z.astype(np.float64) @ w.T)).astype(np.float32)   # [B][N][S], Lipschitz: L = 0.3 * 0.8
    L_env = 0.3 * 0.8
    ws(kbx, B, N, 2, K, S)
    d = dict(labels=dev(labels), dist2=dev(dist2), pulls=dev(np.zeros((B, N, S), np.int32)),
             reward_sum=dev(np.zeros((B, N, S), np.float32)), t=dev(np.ones(B, np.int32)),
             h_cand=dev(np.full((B, N, wl.R_RESOURCES), 50.0, np.float32)),
             target=dev((np.arange(S) % wl.R_RESOURCES).astype(np.int32)),
             t_cur=dev(np.ones((B, N), np.float32)), mu=dev(mu))
    cl = [empty((B, K, S)) for _ in range(3)]
    best_arm, best_val, pair = empty((B,), torch.int32), empty((B,)), empty((B,), torch.int32)
    member, t_new = empty((B,), torch.int32), empty((B,))
    ar = torch.arange(B, device="cuda")
    regret = torch.zeros((T, B), device="cuda")
    mu_star = d["mu"].amax(dim=(1, 2))
    if on_tables:                                                             # the K x S tables once, then kept current
        kbx.score_select(d["labels"], d["dist2"], d["pulls"], d["reward_sum"], d["t"], cl[0], cl[1], cl[2], best_arm,
                         best_val, pair, c=2.0, lipschitz_L=0.0)
    for it in range(T):
        if on_tables:
            kbx.select_pair(cl[0], cl[1], d["t"], pair, c=2.0)
        else:
            kbx.score_select(d["labels"], d["dist2"], d["pulls"], d["reward_sum"], d["t"], cl[0], cl[1], cl[2], best_arm,
                             best_val, pair, c=2.0, lipschitz_L=0.0)
        kbx.sample_member(d["labels"], pair, d["h_cand"], d["target"], d["t"], member, K, 75.0, 31337)
        got_mu = d["mu"][ar, member.long(), (pair % S).long()]                # environment: deterministic reward
        t_new.copy_(1.0 - got_mu)                                             # L(k) = 1, L(k') = 1 - mu
        if on_tables:
            kbx.record_outcome(member, pair, d["t_cur"], t_new, d["pulls"], d["reward_sum"], d["t"], cl_pulls=cl[0],
                               cl_mean=cl[1])
        else:
            kbx.record_outcome(member, pair, d["t_cur"], t_new, d["pulls"], d["reward_sum"], d["t"])
        regret[it] = mu_star - got_mu
    radius = empty((B, K))
    kbx.cluster_radius(d["labels"], d["dist2"], radius)
    torch.cuda.synchronize()
    assert kbx.device_status() == 0
    reg = host(regret)
    assert reg.min() >= -1e-6
    first, last = reg[: T // 4].mean(), reg[-T // 4:].mean()
    assert last < 0.7 * first, (first, last)          # (c = 2 keeps exploring for long: the bonus shrinks like sqrt(ln t / n))
    bound = 1.0 * np.sqrt(K * S * np.log(T) / T) + L_env * 2.0 * float(host(radius).max())
    assert reg.mean() <= bound, (reg.mean(), bound)
    assert int(host(d["pulls"]).sum()) == B * T
    print(f"[regret] first quarter {first:.4f}, last quarter {last:.4f}, average {reg.mean():.4f}, bound {bound:.4f}, "
          f"max radius {float(host(radius).max()):.3f}")


# ------------------------------------------------------------------ top-M arms
@pytest.mark.parametrize("B,N,S,M", [(1, 256, 8, 4), (3, 1000, 13, 7), (2, 20011, 16, 16), (1, 262144, 32, 8),
                                     (64, 512, 16, 5), (2, 3, 4, 20), (1, 5000, 3, 128), (4, 0, 8, 3)])
def test_select_top_m(kbx, B, N, S, M):
    rng = np.random.default_rng(B + N + S + M)
    a = (rng.integers(0, 4000, size=(B, N, S)) / 64.0).astype(np.float32)        # many exact ties
    a[rng.uniform(size=a.shape) < 0.3] = -np.inf
    if N > 10:
        a[0, 5, 1] = np.nan
        a[-1, N // 2:, :] = -np.inf
    ws(kbx, B, N, 1, 1, S)
    arm, val = empty((B, M), torch.int32), empty((B, M))
    kbx.select_top_m(dev(a), arm, val)
    ra, rv = oracle.top_m(a, M)
    np.testing.assert_array_equal(host(arm), ra)                                 # comparisons only: bit-exact
    np.testing.assert_array_equal(host(val), rv)
    assert kbx.device_status() == 0


def test_select_top_m_follows_score_select(kbx):
    cfg = wl.scaled(wl.CONFIGS["medium"], B=2, N=3000, K=16, S=8)
    inp = wl.make_inputs(cfg, seed=2)
    rng = np.random.default_rng(1)
    labels = rng.integers(0, 16, (2, 3000)).astype(np.int32)
    dist2 = rng.uniform(0, 3, (2, 3000)).astype(np.float32)
    keep = rng.integers(0, 256, (2, 3000)).astype(np.uint32)
    got = run_score(kbx, labels, dist2, inp["pulls"], inp["reward_sum"], inp["t"], 16, keep, lipschitz_L=0.1)
    arm, val = empty((2, 6), torch.int32), empty((2, 6))
    kbx.select_top_m(dev(got["arm_index"]), arm, val)
    np.testing.assert_array_equal(host(arm)[:, 0], got["best_arm"])
    np.testing.assert_array_equal(host(val)[:, 0], got["best_val"])
    ra, rv = oracle.top_m(got["arm_index"], 6)
    np.testing.assert_array_equal(host(arm), ra)
    np.testing.assert_array_equal(host(val), rv)


# -------------------------------------------- the loop on the cluster tables
@pytest.mark.parametrize("B,K,S,masked", [(1, 8, 8, True), (5, 3, 4, False), (64, 16, 16, True), (2, 1024, 8, True),
                                          (3, 1, 1, False), (2, 300, 32, True)])
def test_select_pair(kbx, B, K, S, masked):
    rng = np.random.default_rng(B + K + S)
    n = (1 + rng.poisson(5.0, (B, K, S))).astype(np.float32)
    mu = rng.uniform(0, 1, (B, K, S)).astype(np.float32)
    t = rng.integers(1, 5000, B).astype(np.int32)
    hsig = rng.uniform(0, 100, (B, K, wl.R_RESOURCES)).astype(np.float32) if masked else None
    target = (np.arange(S) % wl.R_RESOURCES).astype(np.int32)
    if masked and B > 1:
        hsig[1] = 99.0                                   # instance 1: every pair saturated
    pair, cl_index = empty((B,), torch.int32), empty((B, K, S))
    kbx.select_pair(dev(n), dev(mu), dev(t), pair, c=2.0, hsig=None if hsig is None else dev(hsig), target=dev(target),
                    theta_sat=75.0, cl_index=cl_index)
    ref = oracle.select_pair(n, mu, t, c=2.0, hsig=hsig, target=target, theta_sat=75.0)
    parity.close(host(cl_index), ref["cl_index"], atol=1e-6, what="cl_index")
    got = host(pair)
    u = ref["cl_index"].astype(np.float64).reshape(B, -1)
    for b in range(B):
        if ref["pair"][b] < 0:
            assert got[b] == -1
        elif got[b] != ref["pair"][b]:                   # a near-tie of two pairs: either is a valid choice
            assert got[b] >= 0 and abs(u[b, got[b]] - u[b, ref["pair"][b]]) <= 1e-5 * max(1.0, abs(u[b, ref["pair"][b]]))
            if hsig is not None:
                assert hsig[b, got[b] // S, target[got[b] % S]] < 75.0
    if masked and B > 1:
        assert got[1] == -1
    assert kbx.device_status() == 0


def test_table_loop_matches_the_per_arm_bookkeeping(kbx):
    """Algorithm 1's loop on the cluster tables: kb_score_select once, then T iterations of kb_select_pair ->
    kb_sample_member -> kb_record_outcome (which keeps per-arm statistics and tables current), with no pass over the
    arms.  Every iteration is checked against the oracle from the GPU's state; at the end the tables must equal what
    kb_score_select makes of the per-arm statistics (counts exactly, means within rounding)."""
    B, N, K, S, T = 8, 900, 6, 4, 60
    cfg = wl.scaled(wl.CONFIGS["medium"], B=B, N=N, D=16, K=K, components=6, S=S, iters=2)
    inp = wl.make_inputs(cfg, seed=12)
    rng = np.random.default_rng(5)
    labels = rng.integers(0, K, (B, N)).astype(np.int32)
    h_cand = wl.make_candidate_signatures(inp["hsig"], labels, seed=4)
    gain = rng.uniform(-0.3, 0.7, (B, N, S)).astype(np.float32)
    ws(kbx, B, N, 16, K, S)
    d = {k: dev(v) for k, v in dict(labels=labels, dist2=np.zeros((B, N), np.float32), pulls=inp["pulls"],
                                    reward_sum=inp["reward_sum"], t=inp["t"], h_cand=h_cand, target=inp["target"],
                                    t_cur=inp["t_cur"], gain=gain, hsig=inp["hsig"]).items()}
    cl_pulls, cl_mean, cl_index = empty((B, K, S)), empty((B, K, S)), empty((B, K, S))
    best_arm, best_val, pair0 = empty((B,), torch.int32), empty((B,)), empty((B,), torch.int32)
    kbx.score_select(d["labels"], d["dist2"], d["pulls"], d["reward_sum"], d["t"], cl_pulls, cl_mean, cl_index, best_arm,
                     best_val, pair0)
    pair, member, t_new, reward = empty((B,), torch.int32), empty((B,), torch.int32), empty((B,)), empty((B,))
    ar = torch.arange(B, device="cuda")
    trace = []
    for it in range(T):
        before = (cl_pulls.clone(), cl_mean.clone(), d["t"].clone())
        kbx.select_pair(cl_pulls, cl_mean, d["t"], pair, c=2.0, hsig=d["hsig"], target=d["target"], theta_sat=75.0)
        kbx.sample_member(d["labels"], pair, d["h_cand"], d["target"], d["t"], member, K, 75.0, 777)
        k, s = member.clamp(min=0).long(), (pair.clamp(min=0) % S).long()
        t_new.copy_(d["t_cur"][ar, k] * (1.0 - d["gain"][ar, k, s]))
        kbx.record_outcome(member, pair, d["t_cur"], t_new, d["pulls"], d["reward_sum"], d["t"], reward=reward,
                           cl_pulls=cl_pulls, cl_mean=cl_mean)
        trace.append((before, pair.clone(), member.clone(), reward.clone(), (cl_pulls.clone(), cl_mean.clone())))
    # what the full pass makes of the per-arm statistics now
    f_pulls, f_mean = empty((B, K, S)), empty((B, K, S))
    kbx.score_select(d["labels"], d["dist2"], d["pulls"], d["reward_sum"], d["t"], f_pulls, f_mean, cl_index, best_arm,
                     best_val, pair0)
    torch.cuda.synchronize()
    assert kbx.device_status() == 0
    for before, pair_g, member_g, reward_g, after in trace:
        n0, m0, t0 = (host(x) for x in before)
        sp = oracle.select_pair(n0, m0, t0, c=2.0, hsig=inp["hsig"], target=inp["target"], theta_sat=75.0)
        pg = host(pair_g)
        u = sp["cl_index"].astype(np.float64).reshape(B, -1)
        for b in range(B):
            assert pg[b] == sp["pair"][b] or (pg[b] >= 0 and abs(u[b, pg[b]] - u[b, sp["pair"][b]]) <= 1e-5 * max(1.0, abs(u[b, sp["pair"][b]])))
        dr = oracle.sample_member(labels, pg, h_cand, inp["target"], 75.0, 777, t0, K)
        parity.member_match(host(member_g), None, dr, SAMPLE_TOL)
        n1, m1 = oracle.update_pair(np.where(host(member_g) >= 0, pg, -1), host(reward_g), n0, m0)
        np.testing.assert_array_equal(host(after[0]), n1)
        parity.close(host(after[1]), m1, atol=1e-6, what="cl_mean after the update")
    np.testing.assert_array_equal(host(cl_pulls), host(f_pulls))
    parity.close(host(cl_mean), host(f_mean), atol=2e-6, what="tables against the full pass")
    assert int(host(d["pulls"]).sum() - inp["pulls"].sum()) == int((np.stack([host(x[2]) for x in trace]) >= 0).sum())


# ------------------------------------------------- the whole step as a CUDA graph
@pytest.mark.parametrize("name", ["tiny", "medium", "large/32", "batched/64"])
def test_step_replays_as_a_cuda_graph(kbx, name):
    """kb_bandit_step allocates nothing and never synchronises with the host, so a caller can capture it once and
    replay it (the fused one-CTA path, the cooperative launch, the tensor path with its memset nodes alike).  The
    replay must leave what an eager call leaves: the oracle's checks hold on its outputs, and they equal the eager
    outputs wherever the path is deterministic (integer outputs outside near-ties)."""
    from paper_2511_18868_b200 import kb
    cfg = STEP_CASES[name]
    inp = wl.make_inputs(cfg)
    dims = dict(B=cfg.B, N=cfg.N, D=cfg.D, K=cfg.K, S=cfg.S, R=wl.R_RESOURCES, iters=cfg.iters)
    params = dict(theta_sat=float(inp["theta_sat"]), c=float(inp["c"]), lipschitz_L=float(inp["lipschitz_L"]),
                  prior_pulls=float(inp["prior_pulls"]), prior_mean=float(inp["prior_mean"]))
    eager = run_step(kbx, cfg, inp)
    t = kb.step_tensors(inp, kbx.device)
    x0 = t["x"].clone()
    main = torch.cuda.current_stream()
    side = torch.cuda.Stream()
    side.wait_stream(main)
    kbx.set_stream(side)
    try:
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side, capture_error_mode="thread_local"):
            kbx.bandit_step(dims, params, t)
    finally:
        kbx.set_stream(main)
    main.wait_stream(side)
    for k in ("labels", "best_arm", "z", "arm_index"):
        t[k].zero_()                                   # whatever the capture may have left: the replay must write it
    t["x"].copy_(x0)
    graph.replay()
    torch.cuda.synchronize()
    assert kbx.device_status() == 0
    got = {k: host(v) for k, v in t.items()}
    parity.close(got["z"], eager["z"], atol=0, rtol=0, what="z (replay against eager)")
    chk = oracle.cluster_assign(got["z"], got["centroids"], want_margins=True)
    parity.labels_match(got["z"], got["centroids"], got["labels"], chk)
    assert float(np.mean(got["labels"] == eager["labels"])) > 0.999
    s_chk = oracle.score_select(got["labels"], got["dist2"], inp["pulls"], inp["reward_sum"], inp["t"], cfg.K,
                                keep=got["keep"].view(np.uint32), c=2.0, lipschitz_L=float(inp["lipschitz_L"]))
    parity.close(got["arm_index"], s_chk["arm_index"], atol=1e-6, what="arm_index")
    parity.select_match(got["best_arm"], got["best_val"], s_chk, s_chk["arm_index"])


# ------------------------------------------------------------------ restarts
def test_best_restart_and_the_restart_flow(kbx):
    rng = np.random.default_rng(6)
    x = rng.integers(0, 6, (300, 7)).astype(np.float32)
    x[0, :] = np.nan
    x[1, 0] = np.nan
    x[2, 3] = np.inf
    best = empty((300,), torch.int32)
    kbx.best_restart(dev(x.reshape(-1)), best)
    np.testing.assert_array_equal(host(best), oracle.best_restart(x))
    # n_init consecutive copies of every instance: seed, gather, fit, pick -- all on the device
    K, per, B, n_init = 5, 60, 40, 4
    cen = rng.standard_normal((K, 16)) * 3
    z = (cen[None, :, None, :] + rng.standard_normal((B, K, per, 16))).reshape(B, K * per, 16).astype(np.float32)
    zz = np.repeat(z, n_init, axis=0)
    BB, N = zz.shape[0], zz.shape[1]
    ws(kbx, BB, N, 16, K, 4)
    zd, rows, c = dev(zz), empty((BB, K), torch.int32), empty((BB, K, 16))
    labels, inertia, pick = empty((BB, N), torch.int32), empty((BB,)), empty((B,), torch.int32)
    kbx.seed_kmeanspp(zd, rows, seed=3)
    kbx.init_centroids(zd, rows, c)
    kbx.cluster_fit(zd, c, labels, 6, inertia=inertia)
    kbx.best_restart(inertia, pick)
    torch.cuda.synchronize()
    got_i = host(inertia).reshape(B, n_init)
    np.testing.assert_array_equal(host(pick), oracle.best_restart(got_i))
    assert np.all(got_i[np.arange(B), host(pick)] <= got_i[:, 0])
    r = host(rows).reshape(B, n_init, K)
    assert np.mean([len({tuple(v) for v in r[b].tolist()}) > 1 for b in range(B)]) > 0.9   # the copies are seeded differently
    assert kbx.device_status() == 0


# ----------------------------------------------- tolerance stop, unused clusters
def _tol_case(B, N, D, K, seed):
    rng = np.random.default_rng(seed)
    x = np.empty((B, N, D), np.float32)
    for b in range(B):
        centres = rng.uniform(1.0, 3.0) * rng.standard_normal((K, D))
        x[b] = centres[rng.integers(0, K, N)] + rng.uniform(0.3, 1.2) * rng.standard_normal((N, D))
    z, _, _ = oracle.normalize(x)
    init = np.stack([z[b, rng.choice(N, K, replace=False)] for b in range(B)])
    return z, init


@pytest.mark.parametrize("B,N,D,K,tol", [(6, 400, 16, 5, 1e-3), (40, 512, 32, 16, 1e-2), (3, 300, 64, 4, 0.0),
                                         # loops of calls (row-wise and tensor-core assignments): the gate kernel
                                         (2, 3000, 20, 7, 1e-3), (1, 6000, 32, 130, 5e-3), (3, 5000, 64, 128, 1e-2)])
def test_cluster_fit_tol(kbx, B, N, D, K, tol):
    """Lloyd with a tolerance stop per instance against the oracle's: the iteration count of every instance (where
    the deciding shift is not within rounding of the tolerance), and then, like every free-running fit, the objective
    and the optimality of the returned labels for the returned centroids."""
    z, init = _tol_case(B, N, D, K, N + K)
    max_iter = 40
    ref = oracle.lloyd_tol(z, init, max_iter, tol)
    ws(kbx, B, N, D, K, 4)
    c, labels, d2 = dev(init), empty((B, N), torch.int32), empty((B, N))
    inertia, rep, counts, n_iter = empty((B,)), empty((B, K), torch.int32), empty((B, K), torch.int32), empty((B,), torch.int32)
    kbx.cluster_fit_tol(dev(z), c, labels, max_iter, tol, n_iter, d2, inertia, rep, counts)
    assert kbx.device_status() == 0
    it_g, it_o = host(n_iter), ref["n_iter"]
    assert it_g.min() >= 1 and it_g.max() <= max_iter
    if B >= 6:
        assert len(set(it_o.tolist())) > 1                               # instances stop independently
    # the shifts of the oracle's run around its stop tell whether an fp32 shift could land on the other side of tol
    same_it = it_g == it_o
    for b in np.flatnonzero(~same_it):                                   # a shift within rounding of the tolerance
        assert _reruns_agree(z[b:b + 1], init[b:b + 1], int(it_g[b]), tol), (b, it_g[b], it_o[b], ref["last_shift"][b])
    got_c = host(c)
    for b in np.flatnonzero(same_it):
        parity.close(got_c[b], ref["centroids"][b], atol=2e-5, what="centroids")
        parity.close(host(inertia)[b:b + 1], ref["inertia"][b:b + 1], atol=0, rtol=1e-3, what="inertia")
    chk = oracle.cluster_assign(z, got_c, want_margins=True)
    parity.labels_match(z, got_c, host(labels), chk)
    same = host(labels) == chk["labels"]
    parity.close(host(d2)[same], chk["dist2"][same], atol=1e-7, what="dist2")
    assert np.array_equal(host(counts).sum(1), np.full(B, N))
    print(f"[fit_tol B={B} N={N} D={D} K={K} tol={tol}] iterations GPU {it_g.tolist()[:8]} oracle {it_o.tolist()[:8]}")


def _reruns_agree(z, init, n_iter, tol):
    """The GPU stopped after n_iter updates: legitimate if, in double, the shift of update n_iter is within an fp32
    rounding of the tolerance or below it while every earlier shift was above (up to the same rounding)."""
    c = init.copy()
    shifts = []
    for _ in range(n_iter):
        a = oracle.cluster_assign(z, c, want_rep=False)
        c2, _ = oracle.cluster_update(z, a["labels"], c)
        shifts.append(float(((c2.astype(np.float64) - c.astype(np.float64)) ** 2).sum()))
        c = c2
    slack = 1e-3
    return shifts[-1] <= tol * (1 + slack) + 1e-12 and all(s >= tol * (1 - slack) - 1e-12 for s in shifts[:-1])


def test_unused_clusters_in_one_batch(kbx):
    """rows = -1: instances with K_b in {1, 2, 3, 5} clusters as four instances of one call with K = 5 (the K
    sensitivity study of Sec. 4), through kb_init_centroids + kb_cluster_fit and through the whole step; each
    instance must cluster as the oracle clusters it alone with its own K_b."""
    rng = np.random.default_rng(31)
    B, N, D, K, S, iters = 4, 200, 16, 5, 8, 10
    cfg = wl.scaled(wl.CONFIGS["tiny"], B=B, N=N, D=D, K=K, S=S, iters=iters)
    inp = wl.make_inputs(cfg, seed=5)
    inp["x"] = (3.0 * rng.standard_normal((B, 1, D)) * (rng.integers(0, 3, (B, N, 1)) - 1) + rng.standard_normal((B, N, D))).astype(np.float32)
    rows = np.full((B, K), -1, np.int32)
    kbs = [1, 2, 3, 5]
    for b, kb_ in enumerate(kbs):
        rows[b, :kb_] = rng.choice(N, kb_, replace=False)
    inp["init_rows"] = rows
    z, _, _ = oracle.normalize(inp["x"])
    # the two calls
    ws(kbx, B, N, D, K, S)
    c = empty((B, K, D))
    kbx.init_centroids(dev(z), dev(rows), c)
    assert np.array_equal(host(c), oracle.init_centroids(z, rows))
    labels, d2, inertia, rep, counts = empty((B, N), torch.int32), empty((B, N)), empty((B,)), empty((B, K), torch.int32), empty((B, K), torch.int32)
    kbx.cluster_fit(dev(z), c, labels, iters, d2, inertia, rep, counts)
    got = run_step(kbx, cfg, inp)
    assert kbx.device_status() == 0
    for b, kb_ in enumerate(kbs):
        alone = oracle.lloyd_tol(z[b:b + 1], oracle.init_centroids(z[b:b + 1], rows[b:b + 1, :kb_]), iters, -1.0)
        for lab, cen, cnt, rp, what in [(host(labels)[b], host(c)[b], host(counts)[b], host(rep)[b], "calls"),
                                        (got["labels"][b], got["centroids"][b], got["counts"][b], got["rep"][b], "step")]:
            assert np.array_equal(lab, alone["labels"][0]), (what, b)
            parity.close(cen[:kb_], alone["centroids"][0], atol=1e-5, what=f"centroids ({what})")
            assert np.all(cen[kb_:] == np.float32(1e18)) and np.all(cnt[kb_:] == 0) and np.all(rp[kb_:] == -1)
            assert np.array_equal(cnt[:kb_], alone["counts"][0])
        # an unused cluster is never the chosen pair and carries only the prior
        assert got["best_cluster_arm"][b] // S < kb_
        assert np.all(got["cl_pulls"][b, kb_:] == 1.0) and np.all(got["cl_mean"][b, kb_:] == 0.5)
