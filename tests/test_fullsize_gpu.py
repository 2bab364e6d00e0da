"""Full-size parity: the workloads the benchmark times (`large`, `contraction`), in the launch
configuration it uses (kb_bandit_step on device buffers), checked against the oracle on what the
oracle can afford: every streaming call in full, the assignment on a seeded row sample, and
properties that hold at any size (counts, centroid = member mean, objective not increasing)."""
import numpy as np
import pytest
import torch

import oracle
import parity
from paper_2511_18868_b200 import workloads as wl

pytestmark = pytest.mark.gpu

SAMPLE = {"large": 32768, "contraction": 65536}


@pytest.mark.parametrize("name", ["large", "contraction"])
def test_fullsize_step(name):
    from paper_2511_18868_b200 import kb
    cfg = wl.CONFIGS[name]
    inp = wl.make_inputs(cfg)
    B, N, D, K, S = cfg.B, cfg.N, cfg.D, cfg.K, cfg.S
    ctx = kb.KB(0)
    try:
        ctx.ensure_workspace(ctx.workspace_bytes(B, N, D, K, S))
        t = kb.step_tensors(inp, ctx.device)
        dims = dict(B=B, N=N, D=D, K=K, S=S, R=wl.R_RESOURCES, iters=cfg.iters)
        params = dict(theta_sat=float(inp["theta_sat"]), c=float(inp["c"]), lipschitz_L=float(inp["lipschitz_L"]),
                      prior_pulls=float(inp["prior_pulls"]), prior_mean=float(inp["prior_mean"]))
        ctx.bandit_step(dims, params, t)
        torch.cuda.synchronize()
        assert ctx.device_status() == 0
        assert ctx.assign_path() == 2                      # the tensor-core kernel is what the benchmark times
        # large: the fit keeps a pre-split image of Z; contraction (D = 128): rows are split inside the kernel
        assert ctx.assign_presplit() == (name == "large")
        got = {k: v.cpu().numpy() for k, v in t.items()}
        # the within-cluster draw of k_t, chained on the step's device results (labels, chosen pair)
        h_cand = wl.make_candidate_signatures(inp["hsig"], got["labels"], seed=77)
        member = torch.empty((B,), dtype=torch.int32, device=ctx.device)
        member_val = torch.empty((B,), dtype=torch.float32, device=ctx.device)
        ctx.sample_member(t["labels"], t["best_cluster_arm"], torch.from_numpy(h_cand).to(ctx.device), t["target"],
                          t["t"], member, K, float(inp["theta_sat"]), 0xC0FFEE, member_val)
        torch.cuda.synchronize()
        assert ctx.device_status() == 0
        got["member"], got["member_val"] = member.cpu().numpy(), member_val.cpu().numpy()
    finally:
        ctx.close()
    del t
    torch.cuda.empty_cache()

    # normalise: the whole array
    zr, _, _ = oracle.normalize(inp["x"])
    parity.close(got["z"], zr, atol=2e-5, what="z")
    del zr
    z, c, labels = got["z"], got["centroids"], got["labels"]

    # assign: a seeded row sample against the GPU's own final centroids (double, all K centroids)
    rows = np.sort(np.random.default_rng(123).choice(N, SAMPLE[name], replace=False))
    zs = np.ascontiguousarray(z[:, rows])
    a = oracle.cluster_assign(zs, c, want_rep=False, want_margins=True)
    ties = parity.labels_match(zs, c, np.ascontiguousarray(labels[:, rows]), a)
    same = labels[:, rows] == a["labels"]
    parity.close(got["dist2"][:, rows][same], a["dist2"][same], atol=1e-7, what="dist2 (sample)")

    # properties at full size: every label in range, counts add up, inertia is the sum of dist2
    assert labels.min() >= 0 and labels.max() < K
    assert got["counts"].sum() == N
    parity.close(got["inertia"], np.array([got["dist2"].astype(np.float64).sum()]), atol=0, rtol=1e-5, what="inertia")
    # one more oracle update from the GPU's labels must not move the objective up (Lloyd's invariant),
    # and the representative of every non-empty cluster is a member at minimal distance
    c_next, n_next = oracle.cluster_update(z, labels, c)
    member = np.bincount(labels[0], minlength=K)
    assert np.array_equal(n_next[0], member)
    d_next = oracle.dist2_at(z, c_next, labels).sum()
    assert d_next <= got["dist2"].astype(np.float64).sum() * (1 + 1e-6)
    rep = got["rep"][0]
    for i in np.flatnonzero(member > 0)[:: max(1, K // 64)]:
        assert labels[0, rep[i]] == i
        assert got["dist2"][0, rep[i]] == got["dist2"][0][labels[0] == i].min()
    assert np.all(rep[member == 0] == -1)

    # prune and score: the whole arrays, from the GPU's own labels / dist2
    p = oracle.prune(inp["flops"], inp["bytes"], inp["peak_flops"], inp["peak_bw"], inp["t_inc"], inp["t_cur"],
                     labels, inp["hsig"], inp["target"], 75.0, want_bound=True, want_margin=True)
    prune_ties = parity.keep_match(got["keep"].view(np.uint32), p, S)
    parity.close(got["bound"], p["bound"], atol=1e-6, what="bound")
    del p
    s = oracle.score_select(labels, got["dist2"], inp["pulls"], inp["reward_sum"], inp["t"], K,
                            keep=got["keep"].view(np.uint32), c=2.0, lipschitz_L=float(inp["lipschitz_L"]))
    assert np.array_equal(got["cl_pulls"], s["cl_pulls"])
    parity.close(got["cl_mean"], s["cl_mean"], atol=1e-6, what="cl_mean")
    parity.close(got["cl_index"], s["cl_index"], atol=1e-6, what="cl_index")
    parity.close(got["arm_index"], s["arm_index"], atol=1e-6, what="arm_index")
    sel_ties = parity.select_match(got["best_arm"], got["best_val"], s, s["arm_index"])
    parity.cluster_select_match(got["best_cluster_arm"], s, s["cl_index"])
    # the draw: every instance in full, from the GPU's own labels and chosen pair
    d = oracle.sample_member(labels, got["best_cluster_arm"], h_cand, inp["target"], float(inp["theta_sat"]), 0xC0FFEE,
                             inp["t"], K)
    assert d["member"][0] >= 0 and labels[0, got["member"][0]] == got["best_cluster_arm"][0] // S
    parity.member_match(got["member"], got["member_val"], d, 5e-5)
    print(f"[{name} full size] near-ties: labels (sample of {len(rows)}) {ties}, keep bits {prune_ties}, "
          f"selection {sel_ties}")
