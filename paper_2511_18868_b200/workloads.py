"""Seeded synthetic inputs for the batched bandit step.

This module only *draws inputs*.  It holds none of the step's arithmetic
(no z-scoring, no distances, no index): both the CUDA path and the CPU oracle
are handed the very same numpy arrays it returns.  The one derived quantity is
the incumbent runtime / current runtime of the prune inputs, which the workload
recipe defines as a percentile / multiple of a roofline floor; that is input
synthesis, computed here in float64 numpy and then passed to both sides as
plain fp32 inputs.

Shapes follow the paper's problem statement (Sec. 2.2: action space
A_t = P_t x S; Sec. 3.2: feature vector phi(k), hardware signature h(k) with
three resources SM / DRAM / L2), scaled up to the five synthetic workloads
this repository is measured on.  The public benchmark the paper searches over
is not available; these generators stand in for its search traces.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict

import numpy as np

R_RESOURCES = 3  # SM, DRAM, L2 throughput percentages (App. A.1)


@dataclass(frozen=True)
class Workload:
    name: str
    B: int            # independent bandit instances
    N: int            # candidates (frontier size |P_t|)
    D: int            # trace features per candidate
    K: int            # clusters
    S: int            # strategies
    iters: int        # assign/update iterations (a final assign follows)
    features: str     # "normal" | "mixture"
    components: int   # mixture components (per instance)
    sigma: float      # mixture within-component std
    pull_rate: float  # Poisson rate of per-arm pulls
    zero_frac: float  # fraction of arms forced to zero pulls
    seed: int = 0

    @property
    def arms(self) -> int:
        return self.B * self.N * self.S


CONFIGS: Dict[str, Workload] = {
    # 2 048 arms; launch-latency regime
    "tiny": Workload("tiny", 1, 256, 16, 8, 8, 10, "normal", 0, 0.0, 3.0, 0.0),
    # 262 144 arms; L2-resident
    "medium": Workload("medium", 1, 16384, 32, 64, 16, 20, "mixture", 48, 0.15, 4.0, 0.10),
    # 8.4 M arms
    "large": Workload("large", 1, 262144, 64, 256, 32, 20, "mixture", 200, 0.10, 3.0, 0.0),
    # 1024 independent searches, 8.4 M arms
    "batched": Workload("batched", 1024, 512, 32, 16, 16, 10, "mixture", 48, 0.15, 2.0, 0.20),
    # 33.5 M arms; the distance contraction dominates
    "contraction": Workload("contraction", 1, 4194304, 128, 1024, 8, 5, "mixture", 1500, 0.08, 3.0, 0.0),
}


def scaled(cfg: Workload, **kw) -> Workload:
    """A copy of `cfg` with some sizes replaced (for reduced parity cases)."""
    return replace(cfg, **kw)


def ceilings(S: int):
    """Per-strategy peak-FLOP/s and peak-byte/s table (fixed, not random)."""
    s = np.arange(S)
    peak_flops = (10e12 * (1 + s % 8)).astype(np.float32)
    peak_bw = (1e12 * (1 + s % 4)).astype(np.float32)
    return peak_flops, peak_bw


def _features(cfg: Workload, rng: np.random.Generator) -> np.ndarray:
    B, N, D = cfg.B, cfg.N, cfg.D
    if cfg.features == "normal":
        # log of lognormal(0, 1) counters
        return np.log(rng.lognormal(0.0, 1.0, size=(B, N, D))).astype(np.float32)
    M = cfg.components
    x = np.empty((B, N, D), dtype=np.float32)
    for b in range(B):
        centres = rng.standard_normal((M, D)).astype(np.float32)
        comp = rng.integers(0, M, size=N)
        # draw the noise straight into the output to keep the footprint at one copy
        rng.standard_normal(out=x[b], dtype=np.float32)
        x[b] *= np.float32(cfg.sigma)
        # add centres chunk by chunk (avoids a second N x D temporary)
        step = 1 << 18
        for lo in range(0, N, step):
            hi = min(N, lo + step)
            x[b, lo:hi] += centres[comp[lo:hi]]
    return x


def make_inputs(cfg: Workload, seed: int | None = None) -> Dict[str, np.ndarray]:
    """Draw every input array of one bandit step for workload `cfg`.

    Returns a dict of C-contiguous numpy arrays:
      x [B,N,D] f32          raw trace features (before z-scoring)
      init_rows [B,K] i32    distinct row ids whose z-scored rows seed the centroids
      flops, bytes [B,N] f32 work and traffic of each candidate
      peak_flops, peak_bw [S] f32   per-strategy ceilings
      t_cur [B,N] f32        current runtime of each candidate
      t_inc [B] f32          incumbent runtime
      hsig [B,K,R] f32       per-cluster hardware signature in percent
      target [S] i32         resource each strategy targets
      pulls [B,N,S] i32, reward_sum [B,N,S] f32   per-arm history
      t [B] i32              bandit round (1 + total pulls)
    and scalars theta_sat, c, lipschitz_L, prior_pulls, prior_mean.
    """
    seed = cfg.seed if seed is None else seed
    rng = np.random.default_rng([seed, cfg.B, cfg.N, cfg.D, cfg.K, cfg.S])
    B, N, D, K, S = cfg.B, cfg.N, cfg.D, cfg.K, cfg.S
    out: Dict[str, np.ndarray] = {}
    out["x"] = _features(cfg, rng)

    init_rows = np.empty((B, K), dtype=np.int32)
    for b in range(B):
        init_rows[b] = rng.choice(N, size=K, replace=False) if N >= K else np.arange(K) % max(N, 1)
    out["init_rows"] = init_rows

    # candidate work / traffic: log-uniform on [1e6, 1e12]
    out["flops"] = np.exp(rng.uniform(np.log(1e6), np.log(1e12), size=(B, N))).astype(np.float32)
    out["bytes"] = np.exp(rng.uniform(np.log(1e6), np.log(1e12), size=(B, N))).astype(np.float32)
    peak_flops, peak_bw = ceilings(S)
    out["peak_flops"], out["peak_bw"] = peak_flops, peak_bw

    # recipe-level derived inputs: a runtime floor per (candidate, strategy) taken
    # from the ceilings table, used only to place t_cur above it and t_inc at the
    # 20th percentile.  float64 numpy; both sides receive the rounded fp32 values.
    t_inc = np.empty(B, dtype=np.float32)
    t_cur = np.empty((B, N), dtype=np.float32)
    pf, pb = peak_flops.astype(np.float64), peak_bw.astype(np.float64)
    for b in range(B):
        f = out["flops"][b].astype(np.float64)[:, None]
        q = out["bytes"][b].astype(np.float64)[:, None]
        floor = np.maximum(f / pf[None, :], q / pb[None, :])
        t_inc[b] = np.percentile(floor, 20.0) if N > 0 else 1.0
        u = rng.uniform(0.0, 1.0, size=N)
        t_cur[b] = floor.min(axis=1) * (1.0 + 9.0 * u) if N > 0 else 0.0
    out["t_inc"], out["t_cur"] = t_inc, t_cur

    out["hsig"] = rng.uniform(0.0, 100.0, size=(B, K, R_RESOURCES)).astype(np.float32)
    out["target"] = (np.arange(S) % R_RESOURCES).astype(np.int32)

    pulls = rng.poisson(cfg.pull_rate, size=(B, N, S)).astype(np.int32)
    if cfg.zero_frac > 0.0:
        pulls[rng.uniform(size=(B, N, S)) < cfg.zero_frac] = 0
    out["pulls"] = pulls
    u = rng.uniform(0.0, 2.0, size=(B, N, S)).astype(np.float32)
    out["reward_sum"] = (pulls.astype(np.float32) * u).astype(np.float32)
    out["t"] = (1 + pulls.reshape(B, -1).sum(axis=1)).astype(np.int32)

    out["theta_sat"] = np.float32(75.0)
    out["c"] = np.float32(2.0)
    out["lipschitz_L"] = np.float32(0.1)
    out["prior_pulls"] = np.float32(1.0)
    out["prior_mean"] = np.float32(0.5)
    return out


def make_candidate_signatures(hsig: np.ndarray, labels: np.ndarray, seed: int, spread: float = 3.0) -> np.ndarray:
    """Per-candidate hardware signatures h(k) [B,N,R] f32 for the within-cluster draw of k_t.

    The paper profiles only each cluster's representative (Sec. 3.4); the candidates of a cluster are behaviourally
    similar by construction (Sec. 3.3), so a candidate's signature is drawn here as its cluster's signature plus
    normal noise of `spread` percentage points, clipped to [0, 100].  Input data only: nothing of the draw itself.
    """
    rng = np.random.default_rng(seed)
    B, N = labels.shape
    R = hsig.shape[2]
    base = np.take_along_axis(hsig, np.clip(labels, 0, hsig.shape[1] - 1)[:, :, None].astype(np.int64), axis=1) \
        if N > 0 else np.zeros((B, 0, R), np.float32)
    h = base + spread * rng.standard_normal((B, N, R))
    return np.clip(h, 0.0, 100.0).astype(np.float32)
