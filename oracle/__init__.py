"""ctypes front-end of the CPU oracle (oracle/kb_oracle.cpp).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg.  The product package never imports this module.
Arguments and results are numpy arrays; the arithmetic lives in the C++ file.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Dict, Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "kb_oracle.cpp")
_LIB = os.path.join(_HERE, "libkb_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (plain -O2, one translation unit)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["g++", "-std=c++17", "-O2", "-fPIC", "-shared", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def _check(rc: int, name: str):
    if rc != 0:
        raise ValueError(f"oracle {name} rejected its arguments (code {rc})")


def normalize(x):
    x = _f32(x)
    B, N, D = x.shape
    z = np.empty_like(x)
    mean = np.empty((B, D), np.float32)
    scale = np.empty((B, D), np.float32)
    _check(_load().kbo_normalize(B, N, D, _p(x), _p(z), _p(mean), _p(scale)), "normalize")
    return z, mean, scale


def prune(flops, bytes_, peak_flops, peak_bw, t_inc, t_cur=None, labels=None, hsig=None, target=None,
          theta_sat=75.0, K=0, want_bound=False, want_margin=False):
    flops, bytes_ = _f32(flops), _f32(bytes_)
    B, N = flops.shape
    peak_flops, peak_bw, t_inc = _f32(peak_flops), _f32(peak_bw), _f32(t_inc)
    S = peak_flops.shape[0]
    R = 0
    if labels is not None:
        labels, hsig, target = _i32(labels), _f32(hsig), _i32(target)
        K, R = hsig.shape[1], hsig.shape[2]
    if t_cur is not None:
        t_cur = _f32(t_cur)
    keep = np.empty((B, N), np.uint32)
    kept = np.empty((B,), np.uint32)
    bound = np.empty((B, N, S), np.float32) if want_bound else None
    margin = np.empty((B, N, S), np.float64) if want_margin else None
    _check(_load().kbo_prune(B, N, S, K, R, _p(flops), _p(bytes_), _p(peak_flops), _p(peak_bw), _p(t_inc),
                             _p(t_cur), _p(labels), _p(hsig), _p(target), ctypes.c_float(theta_sat),
                             _p(keep), _p(kept), _p(bound), _p(margin)), "prune")
    return {"keep": keep, "kept_count": kept, "bound": bound, "margin": margin}


def cluster_assign(z, centroids, want_rep=True, want_margins=False):
    z, centroids = _f32(z), _f32(centroids)
    B, N, D = z.shape
    K = centroids.shape[1]
    labels = np.empty((B, N), np.int32)
    dist2 = np.empty((B, N), np.float32)
    inertia = np.empty((B,), np.float32)
    rep = np.empty((B, K), np.int32) if want_rep else None
    best = np.empty((B, N), np.float64) if want_margins else None
    second = np.empty((B, N), np.float64) if want_margins else None
    _check(_load().kbo_cluster_assign(B, N, D, K, _p(z), _p(centroids), _p(labels), _p(dist2), _p(inertia),
                                      _p(rep), _p(best), _p(second)), "cluster_assign")
    return {"labels": labels, "dist2": dist2, "inertia": inertia, "rep": rep, "best": best, "second": second}


def dist2_at(z, centroids, labels):
    z, centroids, labels = _f32(z), _f32(centroids), _i32(labels)
    B, N, D = z.shape
    K = centroids.shape[1]
    out = np.empty((B, N), np.float64)
    _check(_load().kbo_dist2_at(B, N, D, K, _p(z), _p(centroids), _p(labels), _p(out)), "dist2_at")
    return out


def cluster_update(z, labels, centroids):
    """Returns (new centroids, counts); `centroids` (previous) is not modified."""
    z, labels = _f32(z), _i32(labels)
    c = np.array(centroids, dtype=np.float32, order="C", copy=True)
    B, N, D = z.shape
    K = c.shape[1]
    counts = np.empty((B, K), np.int32)
    _check(_load().kbo_cluster_update(B, N, D, K, _p(z), _p(labels), _p(c), _p(counts)), "cluster_update")
    return c, counts


def score_select(labels, dist2, pulls, reward_sum, t, K, keep=None, bound=None, c=2.0, lipschitz_L=0.0,
                 prior_pulls=1.0, prior_mean=0.5, cap_with_bound=False, want_arm_index=True):
    labels, pulls, reward_sum, t = _i32(labels), _i32(pulls), _f32(reward_sum), _i32(t)
    B, N, S = pulls.shape
    if dist2 is not None:
        dist2 = _f32(dist2)
    if keep is not None:
        keep = np.ascontiguousarray(keep, dtype=np.uint32)
    if bound is not None:
        bound = _f32(bound)
    cl_pulls = np.empty((B, K, S), np.float32)
    cl_mean = np.empty((B, K, S), np.float32)
    cl_index = np.empty((B, K, S), np.float32)
    arm_index = np.empty((B, N, S), np.float32) if want_arm_index else None
    best_arm = np.empty((B,), np.int32)
    best_val = np.empty((B,), np.float32)
    best_cl = np.empty((B,), np.int32)
    _check(_load().kbo_score_select(B, N, K, S, ctypes.c_float(c), ctypes.c_float(lipschitz_L),
                                    ctypes.c_float(prior_pulls), ctypes.c_float(prior_mean),
                                    int(bool(cap_with_bound)), _p(labels), _p(dist2), _p(pulls), _p(reward_sum),
                                    _p(keep), _p(bound), _p(t), _p(cl_pulls), _p(cl_mean), _p(cl_index),
                                    _p(arm_index), _p(best_arm), _p(best_val), _p(best_cl)),
           "score_select")
    return {"cl_pulls": cl_pulls, "cl_mean": cl_mean, "cl_index": cl_index, "arm_index": arm_index,
            "best_arm": best_arm, "best_val": best_val, "best_cluster_arm": best_cl}


def init_centroids(z, rows):
    z, rows = _f32(z), _i32(rows)
    B, N, D = z.shape
    K = rows.shape[1]
    c = np.empty((B, K, D), np.float32)
    _check(_load().kbo_init_centroids(B, N, D, K, _p(z), _p(rows), _p(c)), "init_centroids")
    return c


def lloyd_tol(z, centroids, max_iter, tol):
    """Lloyd's iteration with a tolerance stop per instance (see kbo_lloyd_tol).  Returns a dict with centroids, labels,
    dist2, inertia, rep, counts, n_iter [B] and last_shift [B]; `centroids` (initial) is not modified."""
    z = _f32(z)
    c = np.array(centroids, dtype=np.float32, order="C", copy=True)
    B, N, D = z.shape
    K = c.shape[1]
    labels = np.empty((B, N), np.int32)
    dist2 = np.empty((B, N), np.float32)
    inertia = np.empty((B,), np.float32)
    rep = np.empty((B, K), np.int32)
    counts = np.empty((B, K), np.int32)
    n_iter = np.empty((B,), np.int32)
    shift = np.empty((B,), np.float64)
    _check(_load().kbo_lloyd_tol(B, N, D, K, int(max_iter), ctypes.c_float(tol), _p(z), _p(c), _p(labels), _p(dist2),
                                 _p(inertia), _p(rep), _p(counts), _p(n_iter), _p(shift)), "lloyd_tol")
    return {"centroids": c, "labels": labels, "dist2": dist2, "inertia": inertia, "rep": rep, "counts": counts,
            "n_iter": n_iter, "last_shift": shift}


def philox4x32_10(counter, key):
    """One block of the counter-based generator: counter = 4 words, key = 2 words -> 4 words (uint32)."""
    c = np.ascontiguousarray(counter, dtype=np.uint32)
    k = np.ascontiguousarray(key, dtype=np.uint32)
    assert c.shape == (4,) and k.shape == (2,)
    out = np.empty((4,), np.uint32)
    _load().kbo_philox4x32_10(_p(c), _p(k), _p(out))
    return out


def sample_member(labels, cluster_arm, h_cand, target, theta_sat, seed, t, K, want_pert=True, want_prob=False):
    """Within-cluster draw of k_t (Algorithm 1, "Sample k_t"): see kbo_sample_member."""
    labels, cluster_arm, h_cand, target, t = _i32(labels), _i32(cluster_arm), _f32(h_cand), _i32(target), _i32(t)
    B, N, R = h_cand.shape
    S = target.shape[0]
    member = np.empty((B,), np.int32)
    val = np.empty((B,), np.float64)
    pert = np.empty((B, N), np.float64) if want_pert else None
    prob = np.empty((B, N), np.float64) if want_prob else None
    _check(_load().kbo_sample_member(B, N, K, S, R, _p(labels), _p(cluster_arm), _p(h_cand), _p(target),
                                     ctypes.c_float(theta_sat), ctypes.c_uint64(int(seed) & (2**64 - 1)), _p(t),
                                     _p(member), _p(val), _p(pert), _p(prob)), "sample_member")
    return {"member": member, "member_val": val, "pert": pert, "prob": prob}


def record_outcome(member, cluster_arm, t_cur, t_new, pulls, reward_sum, t, verified=None, failures_count=False):
    """Reward clip and statistics update of one iteration (see kbo_record_outcome).  Returns new copies."""
    member, cluster_arm, t_cur, t_new = _i32(member), _i32(cluster_arm), _f32(t_cur), _f32(t_new)
    pulls, reward_sum, t = _i32(pulls).copy(), _f32(reward_sum).copy(), _i32(t).copy()
    if verified is not None:
        verified = _i32(verified)
    B, N, S = pulls.shape
    reward = np.empty((B,), np.float32)
    _check(_load().kbo_record_outcome(B, N, S, int(bool(failures_count)), _p(member), _p(cluster_arm), _p(t_cur),
                                      _p(t_new), _p(verified), _p(pulls), _p(reward_sum), _p(t), _p(reward)),
           "record_outcome")
    return {"pulls": pulls, "reward_sum": reward_sum, "t": t, "reward": reward}


def kmeanspp_round(z, chosen, seed, want_pert=True, want_weights=False):
    """One round of k-means++ seeding given the rows chosen so far (chosen [B][round]); see kbo_kmeanspp_round."""
    z = _f32(z)
    chosen = _i32(chosen)
    B, N, D = z.shape
    rnd = chosen.shape[1]
    row = np.empty((B,), np.int32)
    pert = np.empty((B, N), np.float64) if want_pert else None
    w = np.empty((B, N), np.float64) if want_weights else None
    _check(_load().kbo_kmeanspp_round(B, N, D, rnd, _p(z), _p(chosen), max(rnd, 1),
                                      ctypes.c_uint64(int(seed) & (2**64 - 1)), _p(row), _p(pert), _p(w)),
           "kmeanspp_round")
    return {"row": row, "pert": pert, "weights": w}


def kmeanspp(z, K, seed):
    """k-means++ seeding: rows [B][K] (see kbo_kmeanspp)."""
    z = _f32(z)
    B, N, D = z.shape
    rows = np.zeros((B, K), np.int32)
    _check(_load().kbo_kmeanspp(B, N, D, K, _p(z), ctypes.c_uint64(int(seed) & (2**64 - 1)), _p(rows)), "kmeanspp")
    return rows


def cluster_radius(labels, dist2, K):
    """radius [B][K]: the largest member distance to the centroid per cluster (see kbo_cluster_radius)."""
    labels, dist2 = _i32(labels), _f32(dist2)
    B, N = labels.shape
    radius = np.empty((B, K), np.float32)
    _check(_load().kbo_cluster_radius(B, N, K, _p(labels), _p(dist2), _p(radius)), "cluster_radius")
    return radius


def top_m(arm_index, M):
    """The M best arms per instance by arm_index [B][N][S] (see kbo_top_m): (top_arm [B][M], top_val [B][M])."""
    a = _f32(arm_index)
    B = a.shape[0]
    NS = int(np.prod(a.shape[1:])) if a.ndim > 1 else 0
    top_arm = np.empty((B, M), np.int32)
    top_val = np.empty((B, M), np.float32)
    _check(_load().kbo_top_m(B, NS, M, _p(a), _p(top_arm), _p(top_val)), "top_m")
    return top_arm, top_val


def select_pair(cl_pulls, cl_mean, t, c=2.0, hsig=None, target=None, theta_sat=75.0):
    """Masked-UCB choice of (I_t, S_t) from the cluster tables (see kbo_select_pair)."""
    cl_pulls, cl_mean, t = _f32(cl_pulls), _f32(cl_mean), _i32(t)
    B, K, S = cl_pulls.shape
    R = 1
    if hsig is not None:
        hsig, target = _f32(hsig), _i32(target)
        R = hsig.shape[2]
    cl_index = np.empty((B, K, S), np.float32)
    pair = np.empty((B,), np.int32)
    _check(_load().kbo_select_pair(B, K, S, R, ctypes.c_float(c), _p(cl_pulls), _p(cl_mean), _p(t), _p(hsig),
                                   _p(target), ctypes.c_float(theta_sat), _p(cl_index), _p(pair)), "select_pair")
    return {"pair": pair, "cl_index": cl_index}


def update_pair(pair, reward, cl_pulls, cl_mean):
    """Algorithm 1's N <- N + 1, mu <- mu + (r - mu) / N for the chosen pair.  Returns new copies."""
    pair, reward = _i32(pair), _f32(reward)
    cl_pulls, cl_mean = _f32(cl_pulls).copy(), _f32(cl_mean).copy()
    B, K, S = cl_pulls.shape
    _check(_load().kbo_update_pair(B, K, S, _p(pair), _p(reward), _p(cl_pulls), _p(cl_mean)), "update_pair")
    return cl_pulls, cl_mean


def append_candidate(state, parent, x_new, t_new, verified=None, flops_new=None, bytes_new=None, h_new=None):
    """Frontier growth (see kbo_append_candidate).  `state`: dict of the capacity-padded arrays n_active [B], x [B,Ncap,D],
    t_cur [B,Ncap], labels [B,Ncap], pulls / reward_sum [B,Ncap,S] and optionally flops, bytes [B,Ncap], h_cand [B,Ncap,R],
    dist2 [B,Ncap], t_inc [B].  Returns (new state, appended [B], full [B]); the input is not modified."""
    st = {k: np.array(v, copy=True, order="C") for k, v in state.items()}
    B, Ncap, D = st["x"].shape
    S = st["pulls"].shape[2]
    R = st["h_cand"].shape[2] if "h_cand" in st else 1
    f32 = lambda a: None if a is None else _f32(a)
    parent, x_new, t_new = _i32(parent), _f32(x_new), _f32(t_new)
    verified = None if verified is None else _i32(verified)
    flops_new, bytes_new, h_new = f32(flops_new), f32(bytes_new), f32(h_new)
    appended = np.empty((B,), np.int32)
    full = np.empty((B,), np.int32)
    assert st["n_active"].dtype == np.int32 and st["labels"].dtype == np.int32 and st["pulls"].dtype == np.int32
    for k in ("x", "t_cur", "reward_sum", "flops", "bytes", "h_cand", "dist2", "t_inc"):
        assert k not in st or st[k].dtype == np.float32, k
    _check(_load().kbo_append_candidate(B, Ncap, D, S, R, _p(verified), _p(parent), _p(x_new), _p(t_new), _p(flops_new),
                                        _p(bytes_new), _p(h_new), _p(st["n_active"]), _p(st["x"]), _p(st["t_cur"]),
                                        _p(st.get("flops")), _p(st.get("bytes")), _p(st.get("h_cand")), _p(st["labels"]),
                                        _p(st.get("dist2")), _p(st["pulls"]), _p(st["reward_sum"]), _p(st.get("t_inc")),
                                        _p(appended), _p(full)), "append_candidate")
    return st, appended, full


def recluster_due(t, n_active, tau, K):
    """Algorithm 1's test `t mod tau = 0 and |P| >= 2K` per search: due [B] (see kbo_recluster_due)."""
    t, n_active = _i32(t), _i32(n_active)
    due = np.empty(t.shape, np.int32)
    _check(_load().kbo_recluster_due(t.shape[0], int(tau), int(K), _p(t), _p(n_active), _p(due)), "recluster_due")
    return due


def signatures_from_reps(rep, h_cand, hsig_prev=None, run=None):
    """hsig [B,K,R]: the signature of every cluster's representative, +inf for an empty cluster
    (see kbo_signatures_from_reps); instances with run[b] == 0 keep hsig_prev."""
    rep, h_cand = _i32(rep), _f32(h_cand)
    B, K = rep.shape
    N, R = h_cand.shape[1], h_cand.shape[2]
    hsig = np.zeros((B, K, R), np.float32) if hsig_prev is None else np.array(hsig_prev, np.float32, copy=True, order="C")
    run = None if run is None else _i32(run)
    _check(_load().kbo_signatures_from_reps(B, N, K, R, _p(rep), _p(h_cand), _p(run), _p(hsig)), "signatures_from_reps")
    return hsig


def best_restart(inertia):
    """inertia [G][n_init] -> best [G]: the restart with the smallest inertia (see kbo_best_restart)."""
    x = _f32(inertia)
    G, n_init = x.shape
    best = np.empty((G,), np.int32)
    _check(_load().kbo_best_restart(G, n_init, _p(x), _p(best)), "best_restart")
    return best


def bandit_step(inp: Dict[str, np.ndarray], iters: int, want_arm_index: bool = True) -> Dict[str, np.ndarray]:
    """One whole bandit step in the order the library runs it: normalise, seed
    the centroids from data rows, `iters` x (assign, update), a final assign,
    prune (both masks), cluster statistics + index + selection."""
    z, mean, scale = normalize(inp["x"])
    c = init_centroids(z, inp["init_rows"])
    K = c.shape[1]
    inertia_trace = []
    counts = None
    for _ in range(iters):
        a = cluster_assign(z, c, want_rep=False)
        inertia_trace.append(a["inertia"].copy())
        c, counts = cluster_update(z, a["labels"], c)
    a = cluster_assign(z, c, want_rep=True)
    inertia_trace.append(a["inertia"].copy())
    p = prune(inp["flops"], inp["bytes"], inp["peak_flops"], inp["peak_bw"], inp["t_inc"], inp["t_cur"],
              a["labels"], inp["hsig"], inp["target"], float(inp["theta_sat"]), want_bound=True)
    s = score_select(a["labels"], a["dist2"], inp["pulls"], inp["reward_sum"], inp["t"], K, keep=p["keep"],
                     bound=p["bound"], c=float(inp["c"]), lipschitz_L=float(inp["lipschitz_L"]),
                     prior_pulls=float(inp["prior_pulls"]), prior_mean=float(inp["prior_mean"]),
                     cap_with_bound=False, want_arm_index=want_arm_index)
    out = {"z": z, "mean": mean, "scale": scale, "centroids": c, "counts": counts, "labels": a["labels"],
           "dist2": a["dist2"], "inertia": a["inertia"], "rep": a["rep"], "inertia_trace": np.array(inertia_trace),
           "keep": p["keep"], "kept_count": p["kept_count"], "bound": p["bound"]}
    out.update(s)
    return out
