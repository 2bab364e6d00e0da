"""Bounded device-side waits, seen running out (kb_debug_wait_limit).

The two kernels whose participants wait on one another -- the tensor-core assign kernel (mbarrier waits between its
roles) and the cooperative fit (a grid-wide barrier) -- bound every wait.  Here one participant is kept away and the
limit is cut to a few hundred polls, so the others' waits expire within a millisecond: the kernel must return, the
status word must carry its timeout bit, the synchronising entry points must report KB_ERR_TIMEOUT, and after the word
is cleared the SAME context must produce results that match the oracle.  Nothing here spins without a limit."""
import numpy as np
import pytest
import torch

import oracle
import parity
from paper_2511_18868_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def host(t):
    return t.cpu().numpy()


def _expect_timeout(ctx, kb, bit):
    torch.cuda.synchronize()
    with pytest.raises(kb.KbError) as e:                      # the synchronising read reports it
        ctx.device_status()
    assert e.value.status == 5
    word = ctx.device_status(raise_on_timeout=False)
    assert word & bit, hex(word)
    assert ctx.lib.kb_status_string(ctx.lib.kb_status_of_device_word(word, 0)) == b"KB_ERR_TIMEOUT"
    ctx.clear_device_status()
    ctx.debug_wait_limit(0, False)
    assert ctx.device_status() == 0


def test_cooperative_fit_barrier_times_out_and_the_context_recovers():
    from paper_2511_18868_b200 import kb
    cfg = wl.scaled(wl.CONFIGS["medium"], N=16384, iters=3)
    x = wl.make_inputs(cfg)["x"]
    z, _, _ = oracle.normalize(x)
    init = z[:, np.random.default_rng(0).choice(cfg.N, cfg.K, replace=False)]
    ctx = kb.KB(0)
    try:
        ctx.ensure_workspace(ctx.workspace_bytes(1, cfg.N, cfg.D, cfg.K, 4))
        zd = dev(z)

        def fit():
            c = dev(init)
            labels = torch.zeros((1, cfg.N), dtype=torch.int32, device="cuda")
            inertia = torch.zeros((1,), device="cuda")
            k0 = ctx.launch_count()[0]
            ctx.cluster_fit(zd, c, labels, cfg.iters, inertia=inertia)
            return c, labels, inertia, ctx.launch_count()[0] - k0

        ctx.debug_wait_limit(2000, True)                        # the last CTA never arrives at the grid barrier
        _, _, _, launches = fit()
        assert launches == 2                                    # the clearing kernel and the one cooperative launch
        _expect_timeout(ctx, kb, 0x200)
        c, labels, inertia, _ = fit()                           # the same context, normal limits
        ref = oracle.lloyd_tol(z, init, cfg.iters, -1.0)
        parity.close(host(c), ref["centroids"], atol=1e-5, what="centroids")
        chk = oracle.cluster_assign(z, host(c), want_margins=True)
        parity.labels_match(z, host(c), host(labels), chk)
        parity.close(host(inertia), ref["inertia"], atol=0, rtol=1e-4, what="inertia")
        assert ctx.device_status() == 0
    finally:
        ctx.close()


def test_tensor_assign_wait_times_out_and_the_context_recovers():
    from paper_2511_18868_b200 import kb
    rng = np.random.default_rng(1)
    B, N, D, K = 1, 8192 + 300, 64, 256
    z = rng.standard_normal((B, N, D)).astype(np.float32)
    c = (z[:, rng.choice(N, K, replace=False)] + 0.05 * rng.standard_normal((B, K, D))).astype(np.float32)
    ctx = kb.KB(0)
    try:
        ctx.ensure_workspace(ctx.workspace_bytes(B, N, D, K, 4))
        ctx.set_assign_options(2)                               # the tensor-core kernel, whatever the size
        zd, cd = dev(z), dev(c)
        labels = torch.zeros((B, N), dtype=torch.int32, device="cuda")
        ctx.debug_wait_limit(300, True)                         # CTA 0's B-operand loader stays away
        ctx.cluster_assign(zd, cd, labels)
        assert ctx.assign_path() == 2
        _expect_timeout(ctx, kb, 0x100)
        got = host(labels)
        assert got.min() >= 0 and got.max() < K                 # whatever was written is a centroid id
        # the same context, normal limits: the full result, checked against the oracle
        d2 = torch.empty((B, N), device="cuda")
        ctx.cluster_assign(zd, cd, labels, d2)
        ref = oracle.cluster_assign(z, c, want_margins=True)
        parity.labels_match(z, c, host(labels), ref)
        same = host(labels) == ref["labels"]
        parity.close(host(d2)[same], ref["dist2"][same], atol=1e-7, what="dist2")
        assert ctx.device_status() == 0
    finally:
        ctx.close()


def test_host_step_returns_the_timeout():
    """kb_bandit_step_host synchronises anyway, so it reads the status word and returns KB_ERR_TIMEOUT itself."""
    from paper_2511_18868_b200 import kb
    cfg = wl.scaled(wl.CONFIGS["medium"], N=16384, iters=2)
    inp = wl.make_inputs(cfg)
    ctx = kb.KB(0)
    try:
        ctx.ensure_workspace(ctx.step_workspace_bytes(cfg.B, cfg.N, cfg.D, cfg.K, cfg.S, wl.R_RESOURCES))
        t = kb.step_tensors(inp, None, pinned_host=True)
        dims = dict(B=cfg.B, N=cfg.N, D=cfg.D, K=cfg.K, S=cfg.S, R=wl.R_RESOURCES, iters=cfg.iters)
        params = dict(theta_sat=75.0, c=2.0, lipschitz_L=0.1, prior_pulls=1.0, prior_mean=0.5)
        ctx.debug_wait_limit(2000, True)
        with pytest.raises(kb.KbError) as e:
            ctx.bandit_step_host(dims, params, t)
        assert e.value.status == 5
        ctx.clear_device_status()
        ctx.debug_wait_limit(0, False)
        ctx.bandit_step_host(dims, params, t)                   # and the same call succeeds afterwards
        got = {k: v.numpy() for k, v in t.items()}
        ref = oracle.bandit_step(inp, cfg.iters)
        parity.close(got["inertia"], ref["inertia"], atol=0, rtol=1e-3, what="inertia")
        assert np.mean(got["labels"] == ref["labels"]) > 0.99
        assert ctx.device_status() == 0
    finally:
        ctx.close()


def test_nonfinite_count_matches_numpy():
    """kb_debug_count_nonfinite against its plain definition, on sizes around the grid's stride and with the
    entries that matter: both infinities, quiet and signalling NaN patterns, the largest finite value, denormals."""
    from paper_2511_18868_b200 import kb
    ctx = kb.KB(0)
    rng = np.random.default_rng(11)
    for n in (0, 1, 31, 257, 65536 + 3, 3_000_001):
        x = rng.standard_normal(n).astype(np.float32)
        if n:
            bad = rng.choice(n, size=min(n, 1 + n // 7), replace=False)
            kinds = np.array([np.inf, -np.inf, np.nan], dtype=np.float32)
            x[bad] = kinds[rng.integers(0, 3, size=bad.size)]
            x[rng.integers(0, n)] = np.finfo(np.float32).max          # finite: must not count
            x[rng.integers(0, n)] = np.float32(1e-42)                  # denormal: finite
        if n > 4:
            x.view(np.uint32)[3] = 0x7fa00001                          # a signalling NaN pattern
        want = int((~np.isfinite(x)).sum())
        got = ctx.count_nonfinite(dev(x) if n else torch.empty(0, device="cuda"))
        assert got == want, (n, got, want)
    assert ctx.device_status() == 0
