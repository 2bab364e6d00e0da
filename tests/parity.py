"""Comparison rules shared by the GPU parity tests.

Integer outputs must equal the oracle's wherever the deciding margin exceeds
1e-5 relative; a disagreement inside that margin is a near-tie and is counted.
Float outputs must agree within 1e-4 relative, plus an absolute floor tied to
the scale of the quantity (stated at each call site) where a value can cancel
to ~0.
"""
import numpy as np

import oracle

NEAR_TIE = 1e-5
RTOL = 1e-4


def close(got, want, atol, rtol=RTOL, what=""):
    got, want = np.asarray(got, np.float64), np.asarray(want, np.float64)
    assert got.shape == want.shape, f"{what}: shape {got.shape} vs {want.shape}"
    both_inf = np.isinf(got) & np.isinf(want) & (np.sign(got) == np.sign(want))
    with np.errstate(invalid="ignore"):
        err = np.where(both_inf, 0.0, np.abs(got - want))
    tol = atol + rtol * np.abs(np.where(both_inf, 0.0, want))
    bad = ~(err <= tol)
    assert not bad.any(), (f"{what}: {bad.sum()} of {bad.size} beyond tolerance; worst "
                           f"|err|={np.nanmax(np.where(bad, err, 0)):.3e} at {np.argwhere(bad)[0]}")


def labels_match(z, c, got, ref, what="labels"):
    """got/ref [B,N] int32; ref from the oracle with `best`.  Returns the near-tie count."""
    diff = got != ref["labels"]
    n = int(diff.sum())
    if n == 0:
        return 0
    assert np.all((got >= 0) & (got < c.shape[1])), f"{what}: label out of range"
    d_at = oracle.dist2_at(z, c, got)
    best = ref["best"]
    rel = (d_at - best) / np.maximum(d_at, 1e-300)
    bad = diff & ~(rel <= NEAR_TIE)
    assert not bad.any(), (f"{what}: {bad.sum()} rows assigned to a centroid that is worse than the optimum by "
                           f"more than {NEAR_TIE} relative (worst {rel[bad].max():.3e})")
    return n


def keep_match(got, ref, S, what="keep"):
    """Bits may differ only where the deciding comparison is within the near-tie margin."""
    got = np.asarray(got).view(np.uint32) if np.asarray(got).dtype != np.uint32 else np.asarray(got)
    x = got ^ ref["keep"]
    n = 0
    if x.any():
        bits = ((x[..., None] >> np.arange(S, dtype=np.uint32)) & 1).astype(bool)
        assert np.all(ref["margin"][bits] <= NEAR_TIE), f"{what}: bit differs outside the near-tie margin"
        n = int(bits.sum())
    assert not np.any(got >> np.uint32(S)) if S < 32 else True, f"{what}: bits set beyond S"
    return n


def select_match(got_arm, got_val, ref, ref_arm_index, what="best_arm"):
    """got_arm [B]; ref from oracle.score_select with arm_index [B,N,S]."""
    n = 0
    for b in range(len(got_arm)):
        want = int(ref["best_arm"][b])
        if want < 0:
            assert got_arm[b] == -1 and np.isneginf(got_val[b]), f"{what}: expected no valid arm"
            continue
        flat = ref_arm_index[b].reshape(-1).astype(np.float64)
        g = int(got_arm[b])
        assert 0 <= g < flat.size and np.isfinite(flat[g]), f"{what}: chose a pruned or invalid arm {g}"
        if g != want:
            rel = (flat[want] - flat[g]) / abs(flat[want])
            assert rel <= NEAR_TIE, f"{what}: arm {g} is worse than {want} by {rel:.3e} relative"
            n += 1
        close(got_val[b], flat[g], atol=1e-6, what=what + " value")
    return n


def cluster_select_match(got, ref, cl_index_ref, what="best_cluster_arm"):
    n = 0
    for b in range(len(got)):
        want = int(ref["best_cluster_arm"][b])
        if want < 0:
            assert got[b] == -1
            continue
        g = int(got[b])
        flat = cl_index_ref[b].reshape(-1).astype(np.float64)
        assert 0 <= g < flat.size
        if g != want:
            rel = (flat[want] - flat[g]) / abs(flat[want])
            assert 0 <= rel <= NEAR_TIE, f"{what}: pair {g} vs {want}: {rel:.3e} relative"
            n += 1
    return n


def rep_match(got, ref, dist2_ref, labels_ref, what="rep"):
    n = 0
    B, K = got.shape
    for b in range(B):
        for i in range(K):
            want, g = int(ref["rep"][b, i]), int(got[b, i])
            if want < 0:
                assert g == -1, f"{what}: empty cluster must report -1"
                continue
            if g != want:
                assert 0 <= g < labels_ref.shape[1] and labels_ref[b, g] == i, f"{what}: {g} is not a member of {i}"
                dw, dg = float(dist2_ref[b, want]), float(dist2_ref[b, g])
                assert dg - dw <= NEAR_TIE * max(dg, 1e-30) + 1e-12, f"{what}: member {g} is not nearest"
                n += 1
    return n


def member_match(got, got_val, ref, tol, what="member"):
    """The drawn member is the largest perturbed value of the chosen cluster.  The library forms that value in fp32
    (two logf), the oracle in double: where the oracle's two largest values are closer than `tol` either candidate
    is a valid draw, everywhere else the index must agree; the returned value must be the chosen candidate's."""
    pert = ref["pert"]
    loose = 0
    for b in range(got.shape[0]):
        want = int(ref["member"][b])
        g = int(got[b])
        if want < 0:
            assert g == -1, f"{what}[{b}]: drew {g} where no member can be drawn"
            assert got_val is None or np.isneginf(got_val[b])
            continue
        assert 0 <= g < pert.shape[1] and np.isfinite(pert[b, g]) or pert[b, g] == np.inf, \
            f"{what}[{b}]: {g} is not a drawable member of the chosen cluster"
        if g != want:
            assert pert[b, g] >= pert[b, want] - tol, \
                f"{what}[{b}]: drew {g} ({pert[b, g]}) but {want} ({pert[b, want]}) is larger by more than {tol}"
            loose += 1
        if got_val is not None:
            assert abs(float(got_val[b]) - pert[b, g]) <= tol, f"{what}_val[{b}]: {got_val[b]} vs {pert[b, g]}"
    return loose
