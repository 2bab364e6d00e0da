"""The centroid update without any allocation (kb_cluster_update_noalloc).

Some hosts of the library may not allocate device memory at all: their memory plan is fixed at
start-up, or an allocation's implicit device-wide synchronisation is unacceptable in their loop.
For them the update's scratch is a fixed array inside the library image.  This test calls that
entry point through the C ABI twice in a row (the array keeps the previous call's contents, so the
second call proves the clearing) and checks it against the CPU oracle's update and against the
regular, workspace-based entry point.

Collected last on purpose: a failure here cannot hide any other test from a run that stops at
the first failure.  It needs no state from other tests and passes in a fresh process.
"""
import numpy as np
import pytest
import torch

import oracle

pytestmark = pytest.mark.gpu


def _case(seed, N, D, K):
    rng = np.random.default_rng(seed)
    z = rng.standard_normal((N, D)).astype(np.float32)
    labels = rng.integers(0, max(1, K - 1), N).astype(np.int32)      # the last cluster stays empty
    prev = rng.standard_normal((K, D)).astype(np.float32)
    return z, labels, prev


def test_noalloc_update_matches_oracle_and_workspace_update_twice():
    from paper_2511_18868_b200 import kb
    ctx = kb.KB(0)
    try:
        # two different problems back to back: the second must not see the first one's sums
        for seed, (N, D, K) in enumerate([(20000, 64, 256), (7001, 32, 100)]):
            z, labels, prev = _case(seed, N, D, K)
            zd, ld = torch.from_numpy(z).cuda(), torch.from_numpy(labels).cuda()
            # the existing entry point (one instance, caller-provided workspace)
            ctx.ensure_workspace(ctx.workspace_bytes(1, N, D, K, 1))
            c_ref = torch.from_numpy(prev[None]).cuda()
            n_ref = torch.empty((1, K), dtype=torch.int32, device="cuda")
            ctx.cluster_update(zd[None], ld[None], c_ref, n_ref)
            # the allocation-free entry point: neither torch's allocator nor the driver's free-memory figure moves
            c_new = torch.from_numpy(prev).cuda()
            n_new = torch.empty((K,), dtype=torch.int32, device="cuda")
            if seed == 0:
                kb.cluster_update_noalloc(zd, ld, c_new.clone(), n_new)          # the first call on a device sets up
            torch.cuda.synchronize()
            before, free_before = torch.cuda.memory_allocated(), torch.cuda.mem_get_info()[0]
            kb.cluster_update_noalloc(zd, ld, c_new, n_new)
            torch.cuda.synchronize()
            assert torch.cuda.memory_allocated() == before
            assert torch.cuda.mem_get_info()[0] == free_before
            # against the oracle (counts exact; centroids 1e-4 relative with the update tests' 1e-5 floor)
            want_c, want_n = oracle.cluster_update(z[None], labels[None], prev[None])
            got = c_new.cpu().numpy()
            assert np.array_equal(n_new.cpu().numpy(), want_n[0])
            assert np.all(np.abs(got - want_c[0]) <= 1e-5 + 1e-4 * np.abs(want_c[0]))
            assert np.array_equal(got[K - 1], prev[K - 1])            # empty cluster keeps its centroid
            # and against the workspace-based entry point
            assert torch.equal(n_new.cpu(), n_ref[0].cpu())
            want = c_ref[0].cpu().numpy()
            assert np.all(np.abs(got - want) <= 1e-5 + 1e-4 * np.abs(want))
        assert kb.cluster_update_noalloc_status() == 0
        assert ctx.device_status() == 0
    finally:
        ctx.close()


def test_noalloc_update_reports_labels_out_of_range():
    """A label outside [0, K) is skipped (nothing is read or written through it) and shows in the entry
    point's own status word, which the reader returns once and clears."""
    from paper_2511_18868_b200 import kb
    N, D, K = 5000, 16, 12
    z, labels, prev = _case(5, N, D, K)
    labels[17], labels[4321] = K, -1
    c = torch.from_numpy(prev).cuda()
    n = torch.empty((K,), dtype=torch.int32, device="cuda")
    kb.cluster_update_noalloc(torch.from_numpy(z).cuda(), torch.from_numpy(labels).cuda(), c, n)
    assert kb.cluster_update_noalloc_status() == 1
    assert kb.cluster_update_noalloc_status() == 0                 # read once, then clear
    assert int(n.sum()) == N - 2
    ok = (labels >= 0) & (labels < K)
    want_c, want_n = oracle.cluster_update(z[ok][None], labels[ok][None], prev[None])
    assert np.array_equal(n.cpu().numpy(), want_n[0])
    got = c.cpu().numpy()
    assert np.all(np.abs(got - want_c[0]) <= 1e-5 + 1e-4 * np.abs(want_c[0]))


def test_noalloc_update_rejects_sizes_beyond_its_scratch():
    from paper_2511_18868_b200 import kb
    z = torch.zeros((16, 128), device="cuda")
    labels = torch.zeros((16,), dtype=torch.int32, device="cuda")
    with pytest.raises(kb.KbError) as e:
        kb.cluster_update_noalloc(z, labels, torch.zeros((1024, 128), device="cuda"))      # K*D = 131072 > 65536
    assert e.value.status == 2
    with pytest.raises(kb.KbError) as e:
        kb.cluster_update_noalloc(z[:, :4].contiguous(), labels, torch.zeros((5000, 4), device="cuda"))   # K > 4096
    assert e.value.status == 2
    with pytest.raises(ValueError):
        kb.cluster_update_noalloc(z, labels, torch.zeros((8, 64), device="cuda"))           # D disagrees
    with pytest.raises(ValueError):
        kb.cluster_update_noalloc(z, labels[:8], torch.zeros((8, 128), device="cuda"))      # N disagrees
