"""The expanding frontier on the device (Sec. 2.2; Algorithm 1's "P <- P U {k'_t}" and its re-cluster test):
kb_append_candidate, kb_recluster_due, kb_signatures_from_reps, the whole step on per-instance candidate
counts, and a 40-iteration search loop (the paper's T = 40, tau = 10, K = 3) that never leaves the device,
checked iteration by iteration against the oracle fed the GPU's own state."""
import numpy as np
import pytest
import torch

import oracle
import parity
from paper_2511_18868_b200 import workloads as wl

pytestmark = pytest.mark.gpu

SAMPLE_TOL = 5e-5


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


def frontier(B, cap, D, S, R, n0, rng, K=1):
    """A frontier of capacity `cap` with n0[b] candidates per search (labels in [0, K)); padding label -1."""
    st = {"n_active": np.asarray(n0, np.int32).copy(), "x": np.zeros((B, cap, D), np.float32),
          "t_cur": np.zeros((B, cap), np.float32), "labels": np.full((B, cap), -1, np.int32),
          "dist2": np.zeros((B, cap), np.float32), "pulls": np.zeros((B, cap, S), np.int32),
          "reward_sum": np.zeros((B, cap, S), np.float32), "h_cand": np.zeros((B, cap, R), np.float32),
          "flops": np.ones((B, cap), np.float32), "bytes": np.ones((B, cap), np.float32),
          "t_inc": np.zeros(B, np.float32)}
    for b in range(B):
        n = int(st["n_active"][b])
        st["x"][b, :n] = rng.standard_normal((n, D))
        st["t_cur"][b, :n] = rng.uniform(1.0, 2.0, n)
        st["labels"][b, :n] = rng.integers(0, K, n)
        st["dist2"][b, :n] = rng.uniform(0, 2, n)
        st["pulls"][b, :n] = rng.poisson(2.0, (n, S))
        st["reward_sum"][b, :n] = st["pulls"][b, :n] * rng.uniform(0, 1, (n, S))
        st["h_cand"][b, :n] = rng.uniform(0, 100, (n, R))
        st["flops"][b, :n] = np.exp(rng.uniform(np.log(1e6), np.log(1e12), n))
        st["bytes"][b, :n] = np.exp(rng.uniform(np.log(1e6), np.log(1e12), n))
        st["t_inc"][b] = st["t_cur"][b, :n].min() if n else 1.0
    return st


def to_dev(st):
    return {k: dev(v) for k, v in st.items()}


def to_host(st):
    return {k: host(v) for k, v in st.items()}


@pytest.mark.parametrize("B,cap,D,S,R", [(1, 8, 5, 6, 3), (37, 48, 16, 8, 3), (300, 20, 64, 32, 4), (5, 3, 1, 1, 1)])
def test_append_candidate(kbx, B, cap, D, S, R):
    rng = np.random.default_rng(B + cap)
    n0 = rng.integers(1, cap + 1, B)                                   # some frontiers are full already
    n0[0] = cap
    st = frontier(B, cap, D, S, R, n0, rng, K=3)
    d = to_dev(st)
    for rnd in range(3):
        parent = np.array([rng.integers(0, st["n_active"][b]) if rng.uniform() > 0.15 else -1 for b in range(B)], np.int32)
        verified = (rng.uniform(size=B) < 0.7).astype(np.int32)
        x_new = rng.standard_normal((B, D)).astype(np.float32)
        t_new = rng.uniform(0.2, 2.5, B).astype(np.float32)
        f_new, q_new = rng.uniform(1e6, 1e9, B).astype(np.float32), rng.uniform(1e6, 1e9, B).astype(np.float32)
        h_new = rng.uniform(0, 100, (B, R)).astype(np.float32)
        appended = torch.full((B,), -7, dtype=torch.int32, device="cuda")
        use_verified = rnd != 1                                        # null = every kernel passed
        kbx.append_candidate(d, dev(parent), dev(x_new), dev(t_new), dev(verified) if use_verified else None,
                             dev(f_new), dev(q_new), dev(h_new), appended)
        st, row, full = oracle.append_candidate(st, parent, x_new, t_new, verified if use_verified else None,
                                                f_new, q_new, h_new)
        got = to_host(d)
        assert np.array_equal(host(appended), row)
        for k in st:                                                   # plain copies and integer updates: bit for bit
            assert np.array_equal(got[k], st[k]), k
        status = kbx.device_status()
        assert status == (8 if full.any() else 0)                      # a full frontier is reported, not an error
        kbx.clear_device_status()
    # a parent beyond the frontier is flagged and nothing is appended
    bad = np.zeros(B, np.int32)
    bad[-1] = st["n_active"][-1]
    before = to_host(d)
    kbx.append_candidate(d, dev(bad), dev(x_new), dev(t_new), None, dev(f_new), dev(q_new), dev(h_new))
    after = to_host(d)
    assert after["n_active"][-1] == before["n_active"][-1] and np.array_equal(after["x"][-1], before["x"][-1])
    assert kbx.device_status() & 4
    kbx.clear_device_status()


def test_recluster_due_and_signatures(kbx):
    rng = np.random.default_rng(5)
    B, K, R, N = 700, 3, 3, 40
    t = rng.integers(0, 61, B).astype(np.int32)
    n = rng.integers(1, 12, B).astype(np.int32)
    due, any_due = torch.empty((B,), dtype=torch.int32, device="cuda"), torch.full((1,), -1, dtype=torch.int32, device="cuda")
    for tau in (10, 5, 1):
        kbx.recluster_due(dev(t), dev(n), tau, K, due, any_due)
        want = oracle.recluster_due(t, n, tau, K)
        assert np.array_equal(host(due), want) and int(any_due[0]) == int(want.any())
    kbx.recluster_due(dev(t), dev(np.ones(B, np.int32)), 10, K, due, any_due)          # nobody has 2K candidates
    assert int(any_due[0]) == 0 and not host(due).any()
    h = rng.uniform(0, 100, (B, N, R)).astype(np.float32)
    rep = rng.integers(-1, N, (B, K)).astype(np.int32)
    run = (rng.uniform(size=B) < 0.5).astype(np.int32)
    prev = rng.uniform(0, 100, (B, K, R)).astype(np.float32)
    hs = dev(prev)
    kbx.signatures_from_reps(dev(rep), dev(h), hs, dev(run))
    assert np.array_equal(host(hs), oracle.signatures_from_reps(rep, h, prev, run))
    kbx.signatures_from_reps(dev(rep), dev(h), hs)
    assert np.array_equal(host(hs), oracle.signatures_from_reps(rep, h))
    assert kbx.device_status() == 0


def _step_tensors(kbx, st, K, S, R, init_rows, peaks, target, t, run=None):
    B, cap, D = st["x"].shape
    T = {"x": dev(st["x"]), "init_rows": dev(init_rows), "flops": dev(st["flops"]), "bytes": dev(st["bytes"]),
         "peak_flops": dev(peaks[0]), "peak_bw": dev(peaks[1]), "t_incumbent": dev(st["t_inc"]), "t_cur": dev(st["t_cur"]),
         "hsig": dev(st["hsig"]), "target": dev(target), "pulls": dev(st["pulls"]), "reward_sum": dev(st["reward_sum"]),
         "t": dev(t), "n_active": dev(st["n_active"])}
    if run is not None:
        T["run_mask"] = dev(run)
    f32, i32 = torch.float32, torch.int32
    sent = dict(z=((B, cap, D), f32), centroids=((B, K, D), f32), counts=((B, K), i32), labels=((B, cap), i32),
                dist2=((B, cap), f32), inertia=((B,), f32), rep=((B, K), i32), keep=((B, cap), i32),
                kept_count=((B,), i32), bound=((B, cap, S), f32), cl_pulls=((B, K, S), f32), cl_mean=((B, K, S), f32),
                cl_index=((B, K, S), f32), arm_index=((B, cap, S), f32), best_arm=((B,), i32), best_val=((B,), f32),
                best_cluster_arm=((B,), i32))
    for k, (shape, dt) in sent.items():                                # a sentinel shows what the step left alone
        T[k] = torch.full(shape, -77, dtype=dt, device="cuda")
    return T


def _check_instance(got, st, b, n, K, S, iters, init_rows, peaks, target, t, L):
    """Instance b of a step on n active rows against the oracle's step on exactly those rows."""
    inp = {"x": st["x"][b:b + 1, :n], "init_rows": init_rows[b:b + 1], "flops": st["flops"][b:b + 1, :n],
           "bytes": st["bytes"][b:b + 1, :n], "peak_flops": peaks[0], "peak_bw": peaks[1], "t_inc": st["t_inc"][b:b + 1],
           "t_cur": st["t_cur"][b:b + 1, :n], "hsig": st["hsig"][b:b + 1], "target": target,
           "pulls": st["pulls"][b:b + 1, :n], "reward_sum": st["reward_sum"][b:b + 1, :n], "t": t[b:b + 1],
           "theta_sat": 75.0, "c": 2.0, "lipschitz_L": L, "prior_pulls": 1.0, "prior_mean": 0.5}
    ref = oracle.bandit_step(inp, iters)
    g = {k: v[b:b + 1] for k, v in got.items()}
    parity.close(g["z"][:, :n], ref["z"], atol=2e-5, what="z")
    parity.close(g["inertia"], ref["inertia"], atol=1e-6, rtol=1e-3, what="inertia")
    chk = oracle.cluster_assign(g["z"][:, :n], g["centroids"], want_margins=True)
    parity.labels_match(g["z"][:, :n], g["centroids"], g["labels"][:, :n], chk)
    same = g["labels"][:, :n] == chk["labels"]
    parity.close(g["dist2"][:, :n][same], chk["dist2"][same], atol=1e-7, what="dist2")
    assert g["counts"].sum() == n
    lab, d2 = g["labels"][:, :n], g["dist2"][:, :n]
    p = oracle.prune(inp["flops"], inp["bytes"], peaks[0], peaks[1], inp["t_inc"], inp["t_cur"], lab, inp["hsig"], target,
                     75.0, want_bound=True, want_margin=True)
    keep = g["keep"][:, :n].view(np.uint32)
    parity.keep_match(keep, p, S)
    assert int(g["kept_count"].view(np.uint32)[0]) == int(np.bitwise_count(keep).sum())
    parity.close(g["bound"][:, :n], p["bound"], atol=1e-6, what="bound")
    s = oracle.score_select(lab, d2, inp["pulls"], inp["reward_sum"], inp["t"], K, keep=keep, c=2.0, lipschitz_L=L)
    assert np.array_equal(g["cl_pulls"], s["cl_pulls"])
    parity.close(g["cl_mean"], s["cl_mean"], atol=1e-6, what="cl_mean")
    parity.close(g["cl_index"], s["cl_index"], atol=1e-6, what="cl_index")
    parity.close(g["arm_index"][:, :n], s["arm_index"], atol=1e-6, what="arm_index")
    parity.select_match(g["best_arm"], g["best_val"], s, s["arm_index"])
    parity.cluster_select_match(g["best_cluster_arm"], s, s["cl_index"])


@pytest.mark.parametrize("B,cap,D,K,S,iters", [(6, 48, 16, 3, 8, 5), (40, 300, 32, 7, 16, 3), (3, 512, 64, 5, 4, 2)])
def test_step_on_per_instance_candidate_counts(kbx, B, cap, D, K, S, iters):
    """kb_bandit_step with n_active and run_mask: every instance that runs equals the oracle's step on its own
    active rows (z-scored over those rows only); padding rows and skipped instances keep whatever they held."""
    rng = np.random.default_rng(cap + K)
    R, L = 3, 0.1
    n0 = rng.integers(2 * K, cap + 1, B)
    n0[0], n0[-1] = cap, 2 * K
    st = frontier(B, cap, D, S, R, n0, rng, K=K)
    st["hsig"] = rng.uniform(0, 100, (B, K, R)).astype(np.float32)
    run = (rng.uniform(size=B) < 0.7).astype(np.int32)
    run[0], run[1] = 1, 0
    init_rows = np.stack([rng.choice(int(n0[b]), K, replace=False) for b in range(B)]).astype(np.int32)
    peaks, target = wl.ceilings(S), (np.arange(S) % R).astype(np.int32)
    for b in range(B):                                                   # an incumbent that keeps about a fifth of the arms
        n = int(n0[b])
        floor = np.maximum(st["flops"][b, :n, None] / peaks[0], st["bytes"][b, :n, None] / peaks[1])
        st["t_inc"][b] = np.percentile(floor, 20.0)
        st["t_cur"][b, :n] = floor.min(axis=1) * rng.uniform(1, 10, n)
    t = (1 + st["pulls"].reshape(B, -1).sum(1)).astype(np.int32)
    kbx.ensure_workspace(kbx.workspace_bytes(B, cap, D, K, S))
    T = _step_tensors(kbx, st, K, S, R, init_rows, peaks, target, t, run)
    dims = dict(B=B, N=cap, D=D, K=K, S=S, R=R, iters=iters)
    params = dict(theta_sat=75.0, c=2.0, lipschitz_L=L, prior_pulls=1.0, prior_mean=0.5)
    k0 = kbx.launch_count()[0]
    kbx.bandit_step(dims, params, T)
    assert kbx.launch_count()[0] - k0 == 2                               # one CTA per instance, two launches
    assert kbx.device_status() == 0
    got = {k: host(v) for k, v in T.items()}
    per_row = ["z", "labels", "dist2", "keep", "bound", "arm_index"]
    per_inst = ["centroids", "counts", "inertia", "rep", "kept_count", "cl_pulls", "cl_mean", "cl_index", "best_arm",
                "best_val", "best_cluster_arm"]
    for b in range(B):
        n = int(n0[b])
        if not run[b]:
            for k in per_row + per_inst:
                assert np.all(got[k][b] == -77), (k, b)
            continue
        for k in per_row:
            assert np.all(got[k][b, n:] == -77), (k, b)                  # padding rows are not written
        _check_instance(got, st, b, n, K, S, iters, init_rows, peaks, target, t, L)
    # the tail alone, on the same frontier, from the step's own labels and distances: the same results
    T2 = {k: v.clone() for k, v in T.items()}
    for k in ["keep", "kept_count", "bound", "cl_pulls", "cl_mean", "cl_index", "arm_index", "best_arm", "best_val",
              "best_cluster_arm"]:
        T2[k].fill_(-77)
    kbx.bandit_step_tail(dims, params, T2)
    for k in ["keep", "kept_count", "best_cluster_arm", "cl_pulls"]:
        assert torch.equal(T2[k], T[k]), k
    # shapes that do not run as one CTA per instance refuse n_active instead of ignoring it
    from paper_2511_18868_b200 import kb
    with pytest.raises(kb.KbError) as e:
        kbx.bandit_step(dict(dims, D=8), params, T)
    assert e.value.status == 2


def test_search_loop_with_an_expanding_frontier_follows_the_oracle(kbx):
    """Algorithm 1 from a single kernel per search with the paper's budget and period (T = 40, tau = 10, K = 3;
    |S| = 8 and phi in R^16: the widths the one-CTA kernels take), everything on the device: trigger, masked
    re-clustering step, signatures of the representatives, pair choice on the tables, draw of k_t, outcome, append.
    The LLM is a seeded stand-in (new features near the parent's, a runtime between 0.7x and 1.2x, 80 % verified).
    Every iteration's results are checked against the oracle run on the GPU's own state before that iteration."""
    rng = np.random.default_rng(2024)
    B, cap, D, K, S, R, T_iters, tau, iters = 4, 48, 16, 3, 8, 3, 40, 10, 5
    L, theta, seed = 0.0, 75.0, 991
    st = frontier(B, cap, D, S, R, np.ones(B, np.int32), rng, K=1)
    st["pulls"][:] = 0
    st["reward_sum"][:] = 0
    st["h_cand"][:, 0] = rng.uniform(0, 60, (B, R))                     # k_0 is not saturated anywhere
    st["hsig"] = np.full((B, K, R), np.inf, np.float32)                  # one initial cluster; the others are empty
    st["hsig"][:, 0] = st["h_cand"][:, 0]
    peaks, target = wl.ceilings(S), (np.arange(S) % R).astype(np.int32)
    st["flops"][:], st["bytes"][:] = 1e6, 1e6                            # floors far below every runtime: the roofline mask keeps all
    d = to_dev(st)
    t = torch.ones((B,), dtype=torch.int32, device="cuda")
    cl_pulls = torch.ones((B, K, S), device="cuda")
    cl_mean = torch.full((B, K, S), 0.5, device="cuda")                  # Algorithm 1: N <- 1, mu <- 0.5
    due, any_due = torch.zeros((B,), dtype=torch.int32, device="cuda"), torch.zeros((1,), dtype=torch.int32, device="cuda")
    pair, member = torch.empty((B,), dtype=torch.int32, device="cuda"), torch.empty((B,), dtype=torch.int32, device="cuda")
    reward = torch.empty((B,), device="cuda")
    init_rows = dev(np.tile(np.arange(K, dtype=np.int32), (B, 1)))       # the K oldest kernels seed the clusters
    kbx.ensure_workspace(kbx.workspace_bytes(B, cap, D, K, S))
    step_out = _step_tensors(kbx, dict(st, hsig=st["hsig"]), K, S, R, host(init_rows), peaks, target, np.ones(B, np.int32))
    dims = dict(B=B, N=cap, D=D, K=K, S=S, R=R, iters=iters)
    params = dict(theta_sat=theta, c=2.0, lipschitz_L=L, prior_pulls=1.0, prior_mean=0.5)
    d_target, d_peaks = dev(target), (dev(peaks[0]), dev(peaks[1]))
    reclusterings, appended_total, ties = 0, 0, 0
    for it in range(1, T_iters + 1):
        before = to_host(d)
        t0, tab0 = host(t), (host(cl_pulls), host(cl_mean))
        # ---- trigger and (masked) re-clustering ---------------------------------------------------
        kbx.recluster_due(t, d["n_active"], tau, K, due, any_due)
        want_due = oracle.recluster_due(t0, before["n_active"], tau, K)
        assert np.array_equal(host(due), want_due) and int(any_due[0]) == int(want_due.any())
        if int(any_due[0]):                                              # the host's one decision, from one word
            reclusterings += int(want_due.sum())
            args = dict(step_out)
            args.update(x=d["x"], flops=d["flops"], bytes=d["bytes"], t_incumbent=d["t_inc"], t_cur=d["t_cur"],
                        hsig=d["hsig"], pulls=d["pulls"], reward_sum=d["reward_sum"], t=t, n_active=d["n_active"],
                        run_mask=due, labels=d["labels"], dist2=d["dist2"], cl_pulls=cl_pulls, cl_mean=cl_mean,
                        z=step_out["z"])
            # the signatures of the new clusters come from their representatives BEFORE the tail masks with them:
            # cluster first (iters Lloyd iterations from raw features), then signatures, then prune + score
            fit_args = dict(args)
            kbx.bandit_step(dims, params, fit_args)
            kbx.signatures_from_reps(args["rep"], d["h_cand"], d["hsig"], due)
            kbx.bandit_step_tail(dims, params, args)
            got = {k: host(v) for k, v in args.items()}
            for b in np.flatnonzero(want_due):
                n = int(before["n_active"][b])
                zr, _, _ = oracle.normalize(before["x"][b:b + 1, :n])
                parity.close(got["z"][b:b + 1, :n], zr, atol=2e-5, what="z")
                chk = oracle.cluster_assign(got["z"][b:b + 1, :n], got["centroids"][b:b + 1], want_margins=True)
                parity.labels_match(got["z"][b:b + 1, :n], got["centroids"][b:b + 1], got["labels"][b:b + 1, :n], chk)
                assert np.all(got["labels"][b, n:] == -1)                # padding keeps its label
                hs = oracle.signatures_from_reps(got["rep"][b:b + 1], before["h_cand"][b:b + 1])
                assert np.array_equal(got["hsig"][b:b + 1], hs)
                # statistics re-aggregated over the new clusters from the per-candidate history
                s = oracle.score_select(got["labels"][b:b + 1, :n], got["dist2"][b:b + 1, :n], before["pulls"][b:b + 1, :n],
                                        before["reward_sum"][b:b + 1, :n], t0[b:b + 1], K,
                                        keep=got["keep"][b:b + 1, :n].view(np.uint32), c=2.0, lipschitz_L=L)
                assert np.array_equal(got["cl_pulls"][b:b + 1], s["cl_pulls"])
                parity.close(got["cl_mean"][b:b + 1], s["cl_mean"], atol=1e-6, what="cl_mean")
            for b in np.flatnonzero(want_due == 0):                      # searches that were not due keep everything
                assert np.array_equal(got["labels"][b], before["labels"][b])
                assert np.array_equal(got["cl_pulls"][b], tab0[0][b]) and np.array_equal(got["hsig"][b], before["hsig"][b])
            before = to_host(d)
            tab0 = (host(cl_pulls), host(cl_mean))
        # ---- choose the pair on the tables, draw k_t ------------------------------------------------
        kbx.select_pair(cl_pulls, cl_mean, t, pair, c=2.0, hsig=d["hsig"], target=d_target, theta_sat=theta)
        sp = oracle.select_pair(tab0[0], tab0[1], t0, c=2.0, hsig=before["hsig"], target=target, theta_sat=theta)
        ties += parity.cluster_select_match(host(pair), {"best_cluster_arm": sp["pair"]}, sp["cl_index"])
        kbx.sample_member(d["labels"], pair, d["h_cand"], d_target, t, member, K, theta, seed)
        dr = oracle.sample_member(before["labels"], host(pair), before["h_cand"], target, theta, seed, t0, K)
        parity.member_match(host(member), None, dr, SAMPLE_TOL)
        m = host(member)
        assert np.all((m >= 0) == (host(pair) >= 0)) and np.all(m < before["n_active"])   # never a padding row, never an empty cluster
        # ---- the stand-in for generation and verification -------------------------------------------
        x_new = (before["x"][np.arange(B), m] + 0.3 * rng.standard_normal((B, D))).astype(np.float32)
        t_new = (before["t_cur"][np.arange(B), m] * rng.uniform(0.7, 1.2, B)).astype(np.float32)
        h_new = np.clip(before["h_cand"][np.arange(B), m] + 5 * rng.standard_normal((B, R)), 0, 100).astype(np.float32)
        verified = (rng.uniform(size=B) < 0.8).astype(np.int32)
        f_new = np.full(B, 1e6, np.float32)
        # ---- outcome and growth -----------------------------------------------------------------------
        kbx.record_outcome(member, pair, d["t_cur"], dev(t_new), d["pulls"], d["reward_sum"], t, verified=dev(verified),
                           reward=reward, cl_pulls=cl_pulls, cl_mean=cl_mean)
        ro = oracle.record_outcome(m, host(pair), before["t_cur"], t_new, before["pulls"], before["reward_sum"], t0,
                                   verified=verified)
        appended = torch.empty((B,), dtype=torch.int32, device="cuda")
        kbx.append_candidate(d, member, dev(x_new), dev(t_new), dev(verified), dev(f_new), dev(f_new), dev(h_new), appended)
        want = dict(before, pulls=ro["pulls"], reward_sum=ro["reward_sum"])
        want, row, full = oracle.append_candidate(want, m, x_new, t_new, verified, f_new, f_new, h_new)
        after = to_host(d)
        assert np.array_equal(host(appended), row) and not full.any()
        for k in want:
            if k == "reward_sum":
                parity.close(after[k], want[k], atol=1e-6, what=k)
            else:
                assert np.array_equal(after[k], want[k]), (k, it)
        assert np.array_equal(host(t), ro["t"])
        parity.close(host(reward), ro["reward"], atol=1e-7, what="reward")
        up = oracle.update_pair(np.where(verified != 0, host(pair), -1), ro["reward"], tab0[0], tab0[1])
        assert np.array_equal(host(cl_pulls), up[0])
        parity.close(host(cl_mean), up[1], atol=1e-6, what="cl_mean")
        appended_total += int((row >= 0).sum())
    assert kbx.device_status() == 0
    n_final = host(d["n_active"])
    assert appended_total == int(n_final.sum()) - B and n_final.min() >= 2 * K
    assert reclusterings >= 2 * B - 2                                    # two or more re-clusterings per search (t = 10 .. 40)
    # Algorithm 1's return line: the best runtime over the frontier
    best = np.array([host(d["t_cur"])[b, :n_final[b]].min() for b in range(B)], np.float32)
    assert np.array_equal(host(d["t_inc"]), best)
    print(f"[expanding frontier] final sizes {n_final.tolist()}, re-clusterings {reclusterings}, pair near-ties {ties}")
