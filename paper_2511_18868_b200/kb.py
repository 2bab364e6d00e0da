"""Thin ctypes binding of libkb.so (include/kb.h).

Argument marshalling only: every method passes `tensor.data_ptr()` and sizes to
the C entry point of the same name.  PyTorch supplies device memory and the
CUDA stream; no torch operator runs on the path.  There is no CPU fallback:
if the library has not been built or no CUDA device is present, loading fails.
"""
from __future__ import annotations

import ctypes
import os
from typing import Dict, Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libkb.so")

KB_OK = 0
STATUS_NAMES = {0: "KB_OK", 1: "KB_ERR_INVALID_ARG", 2: "KB_ERR_UNSUPPORTED", 3: "KB_ERR_WORKSPACE",
                4: "KB_ERR_CUDA", 5: "KB_ERR_TIMEOUT"}

# every symbol include/kb.h declares
EXPORTS = ["kb_create", "kb_destroy", "kb_set_stream", "kb_workspace_bytes", "kb_set_workspace",
           "kb_status_string", "kb_last_error", "kb_get_device_status", "kb_clear_device_status", "kb_debug_wait_limit", "kb_debug_count_nonfinite", "kb_status_of_device_word", "kb_get_launch_count",
           "kb_timing_enable", "kb_timing_read", "kb_probe_peaks", "kb_set_assign_options", "kb_get_assign_path", "kb_get_assign_presplit", "kb_assign_tc_probe",
           "kb_normalize", "kb_prune", "kb_cluster_assign", "kb_cluster_update", "kb_score_select", "kb_sample_member", "kb_record_outcome", "kb_select_pair", "kb_seed_kmeanspp", "kb_cluster_radius", "kb_select_top_m", "kb_best_restart",
           "kb_init_centroids", "kb_cluster_fit", "kb_cluster_fit_tol", "kb_bandit_step", "kb_bandit_step_tail", "kb_step_workspace_bytes",
           "kb_bandit_step_host", "kb_cluster_update_noalloc", "kb_cluster_update_noalloc_status",
           "kb_append_candidate", "kb_recluster_due", "kb_signatures_from_reps"]


TIMING_CLASSES = ["normalize", "assign", "update", "prune", "score", "init", "fit", "assign_kernel", "sample", "prep"]


class PeakProbe(ctypes.Structure):
    _fields_ = [("ffma_tflops", ctypes.c_double), ("mma_f16_tflops", ctypes.c_double), ("mma_tf32_tflops", ctypes.c_double),
                ("ffma_ms", ctypes.c_float), ("mma_f16_ms", ctypes.c_float), ("mma_tf32_ms", ctypes.c_float),
                ("mma_f16_cycles_per_instr", ctypes.c_float), ("mma_tf32_cycles_per_instr", ctypes.c_float),
                ("mma_f16_sm_mhz", ctypes.c_float), ("mma_tf32_sm_mhz", ctypes.c_float)]


class KbError(RuntimeError):
    def __init__(self, status: int, where: str, detail: str = ""):
        self.status = status
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)} {detail}".rstrip())


class ScoreParams(ctypes.Structure):
    _fields_ = [("c", ctypes.c_float), ("lipschitz_L", ctypes.c_float), ("prior_pulls", ctypes.c_float),
                ("prior_mean", ctypes.c_float), ("cap_with_bound", ctypes.c_int)]


_VP = ctypes.c_void_p
_STEP_IN = ["x", "init_rows", "flops", "bytes", "peak_flops", "peak_bw", "t_incumbent", "t_cur", "hsig", "target",
            "pulls", "reward_sum", "t"]
_STEP_OUT = ["z", "centroids", "counts", "labels", "dist2", "inertia", "rep", "keep", "kept_count", "bound",
             "cl_pulls", "cl_mean", "cl_index", "arm_index", "best_arm", "best_val", "best_cluster_arm"]
_STEP_OPT = ["n_active", "run_mask"]          # expanding frontier: candidates per instance, instances to run


class StepArgs(ctypes.Structure):
    _fields_ = ([(n, ctypes.c_int) for n in ["B", "N", "D", "K", "S", "R", "iters"]] +
                [("theta_sat", ctypes.c_float), ("score", ScoreParams)] +
                [(n, _VP) for n in _STEP_IN + _STEP_OUT + _STEP_OPT])


_lib = None


def load_library() -> ctypes.CDLL:
    """dlopen libkb.so and declare the prototypes; raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2511_18868_b200.build` "
            "(there is no CPU fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    i, f, sz = ctypes.c_int, ctypes.c_float, ctypes.c_size_t
    lib.kb_create.argtypes = [ctypes.POINTER(_VP), i, _VP]
    lib.kb_destroy.argtypes = [_VP]
    lib.kb_set_stream.argtypes = [_VP, _VP]
    lib.kb_workspace_bytes.argtypes = [i, i, i, i, i, ctypes.POINTER(sz)]
    lib.kb_set_workspace.argtypes = [_VP, _VP, sz]
    lib.kb_status_string.argtypes = [i]
    lib.kb_status_string.restype = ctypes.c_char_p
    lib.kb_last_error.argtypes = [_VP]
    lib.kb_last_error.restype = ctypes.c_char_p
    lib.kb_get_device_status.argtypes = [_VP, ctypes.POINTER(i)]
    lib.kb_clear_device_status.argtypes = [_VP]
    lib.kb_status_of_device_word.argtypes = [i, i]
    lib.kb_debug_wait_limit.argtypes = [_VP, ctypes.c_uint, i]
    lib.kb_debug_count_nonfinite.argtypes = [_VP, _VP, ctypes.c_size_t, ctypes.POINTER(ctypes.c_uint64)]
    lib.kb_get_launch_count.argtypes = [_VP, ctypes.POINTER(ctypes.c_uint64), ctypes.POINTER(ctypes.c_uint64)]
    lib.kb_timing_enable.argtypes = [_VP, i]
    lib.kb_timing_read.argtypes = [_VP, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_int64)]
    lib.kb_probe_peaks.argtypes = [_VP, ctypes.POINTER(PeakProbe)]
    lib.kb_normalize.argtypes = [_VP, i, i, i, _VP, _VP, _VP, _VP]
    lib.kb_prune.argtypes = [_VP, i, i, i, i, i] + [_VP] * 9 + [f] + [_VP] * 3
    lib.kb_cluster_assign.argtypes = [_VP, i, i, i, i] + [_VP] * 6
    lib.kb_cluster_update.argtypes = [_VP, i, i, i, i] + [_VP] * 4
    lib.kb_score_select.argtypes = [_VP, i, i, i, i, ScoreParams] + [_VP] * 14
    lib.kb_sample_member.argtypes = [_VP, i, i, i, i, i] + [_VP] * 4 + [f, ctypes.c_uint64] + [_VP] * 3
    lib.kb_record_outcome.argtypes = [_VP, i, i, i, i, i] + [_VP] * 11
    lib.kb_select_pair.argtypes = [_VP, i, i, i, i, f] + [_VP] * 5 + [f, _VP, _VP]
    lib.kb_cluster_radius.argtypes = [_VP, i, i, i, _VP, _VP, _VP]
    lib.kb_select_top_m.argtypes = [_VP, i, i, i, i, _VP, _VP, _VP]
    lib.kb_best_restart.argtypes = [_VP, i, i, _VP, _VP]
    lib.kb_seed_kmeanspp.argtypes = [_VP, i, i, i, i, _VP, ctypes.c_uint64, _VP]
    lib.kb_set_assign_options.argtypes = [_VP, i, f]
    lib.kb_get_assign_path.argtypes = [_VP, ctypes.POINTER(i)]
    lib.kb_get_assign_presplit.argtypes = [_VP, ctypes.POINTER(i)]
    lib.kb_assign_tc_probe.argtypes = [_VP, i, i, i, i] + [_VP] * 5
    lib.kb_cluster_update_noalloc.argtypes = [_VP, i, i, i, _VP, _VP, _VP, _VP]
    lib.kb_cluster_update_noalloc_status.argtypes = [_VP, ctypes.POINTER(i)]
    lib.kb_init_centroids.argtypes = [_VP, i, i, i, i, _VP, _VP, _VP]
    lib.kb_cluster_fit.argtypes = [_VP, i, i, i, i, i] + [_VP] * 7
    lib.kb_cluster_fit_tol.argtypes = [_VP, i, i, i, i, i, f] + [_VP] * 8
    lib.kb_append_candidate.argtypes = [_VP, i, i, i, i, i] + [_VP] * 19
    lib.kb_recluster_due.argtypes = [_VP, i, i, i] + [_VP] * 4
    lib.kb_signatures_from_reps.argtypes = [_VP, i, i, i, i] + [_VP] * 4
    lib.kb_bandit_step.argtypes = [_VP, ctypes.POINTER(StepArgs)]
    lib.kb_bandit_step_tail.argtypes = [_VP, ctypes.POINTER(StepArgs)]
    lib.kb_step_workspace_bytes.argtypes = [i, i, i, i, i, i, ctypes.POINTER(sz)]
    lib.kb_bandit_step_host.argtypes = [_VP, ctypes.POINTER(StepArgs)]
    for name in EXPORTS:
        if name not in ("kb_status_string", "kb_last_error"):
            getattr(lib, name).restype = i
    _lib = lib
    return lib


# uint32 arrays (keep, kept_count) travel in int32 tensors: same storage, reinterpreted by the library


def _ptr(t: Optional[torch.Tensor], device: Optional[torch.device] = None) -> Optional[int]:
    if t is None:
        return None
    if not t.is_contiguous():
        raise ValueError("libkb takes dense row-major tensors")
    if device is not None and t.device != device:
        raise ValueError(f"tensor on {t.device}, context on {device}")
    if t.element_size() != 4:
        raise ValueError("libkb arrays are 32-bit")
    return t.data_ptr()


class KB:
    """One library context bound to a device and to the current torch stream."""

    def __init__(self, device: int = 0, stream: Optional[torch.cuda.Stream] = None):
        if not torch.cuda.is_available():
            raise RuntimeError("libkb needs a CUDA device; there is no CPU path")
        self.lib = load_library()
        self.device = torch.device("cuda", device)
        self._stream = stream if stream is not None else torch.cuda.current_stream(self.device)
        h = _VP()
        self._check(self.lib.kb_create(ctypes.byref(h), device, _VP(self._stream.cuda_stream)), "kb_create", ctx=None)
        self.h = h
        self._ws: Optional[torch.Tensor] = None

    # -- plumbing -----------------------------------------------------------
    def _check(self, status: int, where: str, ctx="self"):
        if status != KB_OK:
            detail = ""
            if ctx is not None and getattr(self, "h", None):
                detail = self.lib.kb_last_error(self.h).decode()
            raise KbError(status, where, detail)

    def close(self):
        if getattr(self, "h", None):
            self.lib.kb_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_stream(self, stream: torch.cuda.Stream):
        self._stream = stream
        self._check(self.lib.kb_set_stream(self.h, _VP(stream.cuda_stream)), "kb_set_stream")

    def workspace_bytes(self, B, N, D, K, S) -> int:
        out = ctypes.c_size_t()
        self._check(self.lib.kb_workspace_bytes(B, N, D, K, S, ctypes.byref(out)), "kb_workspace_bytes")
        return out.value

    def step_workspace_bytes(self, B, N, D, K, S, R) -> int:
        out = ctypes.c_size_t()
        self._check(self.lib.kb_step_workspace_bytes(B, N, D, K, S, R, ctypes.byref(out)), "kb_step_workspace_bytes")
        return out.value

    def set_workspace(self, ws: Optional[torch.Tensor]):
        self._ws = ws
        n = 0 if ws is None else ws.numel() * ws.element_size()
        self._check(self.lib.kb_set_workspace(self.h, None if ws is None else ws.data_ptr(), n), "kb_set_workspace")

    def ensure_workspace(self, nbytes: int):
        """Registers a torch-allocated workspace of at least `nbytes` (grows only)."""
        have = 0 if self._ws is None else self._ws.numel()
        if have < nbytes:
            self.set_workspace(torch.empty(max(nbytes, 256), dtype=torch.uint8, device=self.device))

    def device_status(self, raise_on_timeout: bool = True) -> int:
        """The device status word (synchronises).  A timeout bit raises KbError(KB_ERR_TIMEOUT) unless told not to."""
        out = ctypes.c_int()
        rc = self.lib.kb_get_device_status(self.h, ctypes.byref(out))
        if rc != KB_OK and (raise_on_timeout or rc != 5):
            self._check(rc, "kb_get_device_status")
        return out.value

    def debug_wait_limit(self, polls: int = 0, leave_one_out: bool = False):
        """kb_debug_wait_limit: shorten the bounded device-side waits / keep one participant away (tests only)."""
        self._check(self.lib.kb_debug_wait_limit(self.h, int(polls), int(bool(leave_one_out))), "kb_debug_wait_limit")

    def count_nonfinite(self, x) -> int:
        """kb_debug_count_nonfinite: how many entries of a float32 device tensor are NaN or infinite (synchronises)."""
        out = ctypes.c_uint64()
        n = int(x.numel())
        self._check(self.lib.kb_debug_count_nonfinite(self.h, self._p(x) if n else None, n, ctypes.byref(out)),
                    "kb_debug_count_nonfinite")
        return int(out.value)

    def clear_device_status(self):
        self._check(self.lib.kb_clear_device_status(self.h), "kb_clear_device_status")

    def launch_count(self):
        """(kernels, memset nodes) queued by this context so far."""
        k, m = ctypes.c_uint64(), ctypes.c_uint64()
        self._check(self.lib.kb_get_launch_count(self.h, ctypes.byref(k), ctypes.byref(m)), "kb_get_launch_count")
        return k.value, m.value

    def timing_enable(self, on: bool = True):
        self._check(self.lib.kb_timing_enable(self.h, int(on)), "kb_timing_enable")

    def timing_read(self):
        """{class name: (milliseconds, calls)} since the last read; synchronises."""
        ms = (ctypes.c_double * len(TIMING_CLASSES))()
        n = (ctypes.c_int64 * len(TIMING_CLASSES))()
        self._check(self.lib.kb_timing_read(self.h, ms, n), "kb_timing_read")
        return {name: (ms[i], n[i]) for i, name in enumerate(TIMING_CLASSES)}

    def probe_peaks(self) -> Dict[str, float]:
        """kb_probe_peaks: measured fp32 FMA and tcgen05 (kind::f16, kind::tf32) ceilings of this device, TFLOP/s."""
        p = PeakProbe()
        self._check(self.lib.kb_probe_peaks(self.h, ctypes.byref(p)), "kb_probe_peaks")
        return {name: float(getattr(p, name)) for name, _ in PeakProbe._fields_}

    def _p(self, t):
        return _ptr(t, self.device)

    # -- the five calls -----------------------------------------------------
    def normalize(self, x, z=None, mean=None, scale=None):
        B, N, D = x.shape
        z = x if z is None else z
        self._check(self.lib.kb_normalize(self.h, B, N, D, self._p(x), self._p(z), self._p(mean), self._p(scale)),
                    "kb_normalize")
        return z

    def prune(self, flops, bytes_, peak_flops, peak_bw, t_incumbent, keep, t_cur=None, labels=None, hsig=None,
              target=None, theta_sat=75.0, kept_count=None, bound=None):
        B, N = flops.shape
        S = peak_flops.shape[0]
        K, R = (hsig.shape[1], hsig.shape[2]) if hsig is not None else (0, 0)
        self._check(self.lib.kb_prune(self.h, B, N, S, K, R, self._p(flops), self._p(bytes_), self._p(peak_flops),
                                      self._p(peak_bw), self._p(t_incumbent), self._p(t_cur), self._p(labels),
                                      self._p(hsig), self._p(target), float(theta_sat), self._p(keep),
                                      self._p(kept_count), self._p(bound)), "kb_prune")

    def cluster_assign(self, z, centroids, labels, dist2=None, inertia=None, rep=None):
        B, N, D = z.shape
        K = centroids.shape[1]
        self._check(self.lib.kb_cluster_assign(self.h, B, N, D, K, self._p(z), self._p(centroids), self._p(labels),
                                               self._p(dist2), self._p(inertia), self._p(rep)), "kb_cluster_assign")

    def cluster_update(self, z, labels, centroids, counts=None):
        B, N, D = z.shape
        K = centroids.shape[1]
        self._check(self.lib.kb_cluster_update(self.h, B, N, D, K, self._p(z), self._p(labels), self._p(centroids),
                                               self._p(counts)), "kb_cluster_update")

    def score_select(self, labels, dist2, pulls, reward_sum, t, cl_pulls, cl_mean, cl_index, best_arm, best_val,
                     best_cluster_arm, keep=None, bound=None, arm_index=None, c=2.0, lipschitz_L=0.0,
                     prior_pulls=1.0, prior_mean=0.5, cap_with_bound=False):
        B, N, S = pulls.shape
        K = cl_index.shape[1]
        p = ScoreParams(c, lipschitz_L, prior_pulls, prior_mean, int(bool(cap_with_bound)))
        self._check(self.lib.kb_score_select(self.h, B, N, K, S, p, self._p(labels), self._p(dist2), self._p(pulls),
                                             self._p(reward_sum), self._p(keep), self._p(bound), self._p(t),
                                             self._p(cl_pulls), self._p(cl_mean), self._p(cl_index),
                                             self._p(arm_index), self._p(best_arm), self._p(best_val),
                                             self._p(best_cluster_arm)), "kb_score_select")

    def sample_member(self, labels, cluster_arm, h_cand, target, t, member, K, theta_sat, seed, member_val=None):
        """Within-cluster draw of k_t (Algorithm 1, "Sample k_t")."""
        B, N, R = h_cand.shape
        S = target.shape[0]
        self._check(self.lib.kb_sample_member(self.h, B, N, int(K), S, R, self._p(labels), self._p(cluster_arm),
                                              self._p(h_cand), self._p(target), float(theta_sat),
                                              int(seed) & (2 ** 64 - 1), self._p(t), self._p(member),
                                              self._p(member_val)), "kb_sample_member")

    def best_restart(self, inertia, best):
        """inertia [G*n_init] (n_init consecutive instances per search) -> best [G]: the run with the smallest inertia."""
        G = best.shape[0]
        n_init = inertia.numel() // max(G, 1)
        self._check(self.lib.kb_best_restart(self.h, G, n_init, self._p(inertia), self._p(best)), "kb_best_restart")

    def select_top_m(self, arm_index, top_arm, top_val=None):
        """The M best arms per instance by arm_index [B][N][S]: top_arm [B][M] (flat k*S+s), sorted."""
        B, N, S = arm_index.shape
        M = top_arm.shape[1]
        self._check(self.lib.kb_select_top_m(self.h, B, N, S, M, self._p(arm_index), self._p(top_arm),
                                             self._p(top_val)), "kb_select_top_m")

    def cluster_radius(self, labels, dist2, radius):
        """radius [B][K]: largest member distance to the centroid per cluster (bounds Theorem 1's diameter term)."""
        B, N = labels.shape
        K = radius.shape[1]
        self._check(self.lib.kb_cluster_radius(self.h, B, N, K, self._p(labels), self._p(dist2), self._p(radius)),
                    "kb_cluster_radius")

    def seed_kmeanspp(self, z, rows, seed):
        """k-means++ seeding: rows [B][K] of z to start the clustering from."""
        B, N, D = z.shape
        K = rows.shape[1]
        self._check(self.lib.kb_seed_kmeanspp(self.h, B, N, D, K, self._p(z), int(seed) & (2 ** 64 - 1),
                                              self._p(rows)), "kb_seed_kmeanspp")

    def record_outcome(self, member, cluster_arm, t_cur, t_new, pulls, reward_sum, t, verified=None, reward=None,
                       failures_count=False, cl_pulls=None, cl_mean=None):
        """Reward clip and statistics update of one iteration (Algorithm 1, "Generation & update"), in place;
        with cl_pulls / cl_mean [B][K][S] the cluster tables are updated alongside."""
        B, N, S = pulls.shape
        K = cl_pulls.shape[1] if cl_pulls is not None else 1
        self._check(self.lib.kb_record_outcome(self.h, B, N, K, S, int(bool(failures_count)), self._p(member),
                                               self._p(cluster_arm), self._p(t_cur), self._p(t_new),
                                               self._p(verified), self._p(pulls), self._p(reward_sum), self._p(t),
                                               self._p(reward), self._p(cl_pulls), self._p(cl_mean)),
                    "kb_record_outcome")

    def select_pair(self, cl_pulls, cl_mean, t, pair, c=2.0, hsig=None, target=None, theta_sat=75.0, cl_index=None):
        """Masked-UCB choice of (I_t, S_t) from the cluster tables alone (Algorithm 1, "Select (I_t, S_t)")."""
        B, K, S = cl_pulls.shape
        R = hsig.shape[2] if hsig is not None else 1
        self._check(self.lib.kb_select_pair(self.h, B, K, S, R, float(c), self._p(cl_pulls), self._p(cl_mean),
                                            self._p(t), self._p(hsig), self._p(target), float(theta_sat),
                                            self._p(cl_index), self._p(pair)), "kb_select_pair")

    def set_assign_options(self, path: int = 0, tc_eps: float = 0.0):
        """path: 0 automatic, 1 fp32 row-wise kernel, 2 tensor-core kernel."""
        self._check(self.lib.kb_set_assign_options(self.h, int(path), float(tc_eps)), "kb_set_assign_options")

    def assign_path(self) -> int:
        out = ctypes.c_int()
        self._check(self.lib.kb_get_assign_path(self.h, ctypes.byref(out)), "kb_get_assign_path")
        return out.value

    def assign_presplit(self) -> bool:
        out = ctypes.c_int()
        self._check(self.lib.kb_get_assign_presplit(self.h, ctypes.byref(out)), "kb_get_assign_presplit")
        return bool(out.value)

    def assign_tc_probe(self, z, centroids, labels, approx_dist2=None, flagged=None):
        B, N, D = z.shape
        K = centroids.shape[1]
        self._check(self.lib.kb_assign_tc_probe(self.h, B, N, D, K, self._p(z), self._p(centroids), self._p(labels),
                                                self._p(approx_dist2), self._p(flagged)), "kb_assign_tc_probe")

    # -- conveniences -------------------------------------------------------
    def init_centroids(self, z, rows, centroids):
        B, N, D = z.shape
        K = rows.shape[1]
        self._check(self.lib.kb_init_centroids(self.h, B, N, D, K, self._p(z), self._p(rows), self._p(centroids)),
                    "kb_init_centroids")

    def cluster_fit(self, z, centroids, labels, iters, dist2=None, inertia=None, rep=None, counts=None):
        B, N, D = z.shape
        K = centroids.shape[1]
        self._check(self.lib.kb_cluster_fit(self.h, B, N, D, K, int(iters), self._p(z), self._p(centroids),
                                            self._p(labels), self._p(dist2), self._p(inertia), self._p(rep),
                                            self._p(counts)), "kb_cluster_fit")

    def cluster_fit_tol(self, z, centroids, labels, max_iter, tol, n_iter, dist2=None, inertia=None, rep=None, counts=None):
        """kb_cluster_fit_tol: Lloyd with a tolerance stop per instance; n_iter [B] receives the updates done."""
        B, N, D = z.shape
        K = centroids.shape[1]
        self._check(self.lib.kb_cluster_fit_tol(self.h, B, N, D, K, int(max_iter), float(tol), self._p(z),
                                                self._p(centroids), self._p(labels), self._p(dist2), self._p(inertia),
                                                self._p(rep), self._p(counts), self._p(n_iter)), "kb_cluster_fit_tol")

    def _step_args(self, dims: Dict[str, int], params: Dict[str, float], tensors: Dict[str, torch.Tensor], host: bool):
        a = StepArgs()
        for k in ["B", "N", "D", "K", "S", "R", "iters"]:
            setattr(a, k, int(dims[k]))
        a.theta_sat = float(params.get("theta_sat", 75.0))
        a.score = ScoreParams(float(params.get("c", 2.0)), float(params.get("lipschitz_L", 0.0)),
                              float(params.get("prior_pulls", 1.0)), float(params.get("prior_mean", 0.5)),
                              int(bool(params.get("cap_with_bound", False))))
        for name in _STEP_IN + _STEP_OUT + _STEP_OPT:
            t = tensors.get(name)
            setattr(a, name, None if t is None else _ptr(t, None if host else self.device))
        return a

    def bandit_step(self, dims, params, tensors):
        """Whole step on device tensors (dict keyed by the field names of kb_step_args)."""
        a = self._step_args(dims, params, tensors, host=False)
        self._check(self.lib.kb_bandit_step(self.h, ctypes.byref(a)), "kb_bandit_step")

    def append_candidate(self, st, parent, x_new, t_new, verified=None, flops_new=None, bytes_new=None, h_new=None,
                         appended=None):
        """kb_append_candidate on a frontier `st`: dict of device tensors n_active [B], x [B,Ncap,D], t_cur, labels
        [B,Ncap], pulls, reward_sum [B,Ncap,S] and optionally flops, bytes, dist2 [B,Ncap], h_cand [B,Ncap,R], t_inc [B]."""
        B, Ncap, D = st["x"].shape
        S = st["pulls"].shape[2]
        R = st["h_cand"].shape[2] if st.get("h_cand") is not None else 1
        p = self._p
        self._check(self.lib.kb_append_candidate(
            self.h, B, Ncap, D, S, R, p(verified), p(parent), p(x_new), p(t_new), p(flops_new), p(bytes_new), p(h_new),
            p(st["n_active"]), p(st["x"]), p(st["t_cur"]), p(st.get("flops")), p(st.get("bytes")), p(st.get("h_cand")),
            p(st["labels"]), p(st.get("dist2")), p(st["pulls"]), p(st["reward_sum"]), p(st.get("t_inc")), p(appended)),
            "kb_append_candidate")

    def recluster_due(self, t, n_active, tau, K, due, any_due=None):
        self._check(self.lib.kb_recluster_due(self.h, t.shape[0], int(tau), int(K), self._p(t), self._p(n_active),
                                              self._p(due), self._p(any_due)), "kb_recluster_due")

    def signatures_from_reps(self, rep, h_cand, hsig, run_mask=None):
        B, K = rep.shape
        N, R = h_cand.shape[1], h_cand.shape[2]
        self._check(self.lib.kb_signatures_from_reps(self.h, B, N, K, R, self._p(rep), self._p(h_cand), self._p(run_mask),
                                                     self._p(hsig)), "kb_signatures_from_reps")

    def bandit_step_tail(self, dims, params, tensors):
        """kb_bandit_step_tail: prune + score + select from the caller's labels and dist2 (device tensors)."""
        a = self._step_args(dims, params, tensors, host=False)
        self._check(self.lib.kb_bandit_step_tail(self.h, ctypes.byref(a)), "kb_bandit_step_tail")

    def bandit_step_host(self, dims, params, tensors):
        """Whole step on HOST tensors (ideally pinned); returns after the results are in host memory."""
        a = self._step_args(dims, params, tensors, host=True)
        self._check(self.lib.kb_bandit_step_host(self.h, ctypes.byref(a)), "kb_bandit_step_host")


def cluster_update_noalloc(z, labels, centroids, counts=None, stream=None):
    """kb_cluster_update_noalloc: one instance, scratch built into the library, nothing allocated.
    z [N][D], labels [N], centroids [K][D] (updated in place), counts [K] or None; device tensors."""
    lib = load_library()
    # the C entry point takes bare pointers: a wrong shape or dtype here would be an out-of-bounds device access
    if z.dim() != 2 or centroids.dim() != 2 or labels.dim() != 1:
        raise ValueError("cluster_update_noalloc: z [N][D], labels [N], centroids [K][D]")
    N, D = z.shape
    K = centroids.shape[0]
    if centroids.shape[1] != D or labels.numel() != N or (counts is not None and counts.numel() != K):
        raise ValueError("cluster_update_noalloc: shapes disagree")
    if z.dtype != torch.float32 or centroids.dtype != torch.float32 or labels.dtype != torch.int32 or \
            (counts is not None and counts.dtype != torch.int32):
        raise ValueError("cluster_update_noalloc: z, centroids float32; labels, counts int32")
    for a in (z, labels, centroids, counts):
        if a is not None and (not a.is_cuda or not a.is_contiguous() or a.device != z.device):
            raise ValueError("cluster_update_noalloc: contiguous tensors on one CUDA device")
    st = stream if stream is not None else torch.cuda.current_stream(z.device)
    with torch.cuda.device(z.device):
        rc = lib.kb_cluster_update_noalloc(_VP(st.cuda_stream), N, D, K, _ptr(z), _ptr(labels), _ptr(centroids),
                                           _ptr(counts))
    if rc != KB_OK:
        raise KbError(rc, "kb_cluster_update_noalloc")


def cluster_update_noalloc_status(device=None, stream=None) -> int:
    """kb_cluster_update_noalloc_status: reads and clears the status word of the allocation-free update on
    `device` (bit 1: a label outside [0, K) was skipped).  Synchronises the stream."""
    lib = load_library()
    device = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
    st = stream if stream is not None else torch.cuda.current_stream(device)
    out = ctypes.c_int()
    with torch.cuda.device(device):
        rc = lib.kb_cluster_update_noalloc_status(_VP(st.cuda_stream), ctypes.byref(out))
    if rc != KB_OK:
        raise KbError(rc, "kb_cluster_update_noalloc_status")
    return out.value


def step_tensors(inp: Dict, device, want_arm_index=True, want_bound=True, pinned_host=False) -> Dict[str, torch.Tensor]:
    """Moves a workload dict (numpy arrays of `workloads.make_inputs`) into the
    tensors one bandit step takes, plus freshly allocated outputs."""
    import numpy as np
    names = {"x": "x", "init_rows": "init_rows", "flops": "flops", "bytes": "bytes", "peak_flops": "peak_flops",
             "peak_bw": "peak_bw", "t_inc": "t_incumbent", "t_cur": "t_cur", "hsig": "hsig", "target": "target",
             "pulls": "pulls", "reward_sum": "reward_sum", "t": "t"}
    out: Dict[str, torch.Tensor] = {}
    for src, dst in names.items():
        t = torch.from_numpy(np.ascontiguousarray(inp[src]))
        if pinned_host:
            t = t.pin_memory() if torch.cuda.is_available() else t
        else:
            t = t.to(device)
        out[dst] = t
    B, N, D = inp["x"].shape
    K, S = inp["init_rows"].shape[1], inp["pulls"].shape[2]
    kw = dict(device="cpu", pin_memory=torch.cuda.is_available()) if pinned_host else dict(device=device)

    def new(shape, dt):
        return torch.empty(shape, dtype=dt, **kw)
    out.update(
        z=new((B, N, D), torch.float32),
        centroids=new((B, K, D), torch.float32), counts=new((B, K), torch.int32),
        labels=new((B, N), torch.int32), dist2=new((B, N), torch.float32), inertia=new((B,), torch.float32),
        rep=new((B, K), torch.int32), keep=new((B, N), torch.int32), kept_count=new((B,), torch.int32),
        cl_pulls=new((B, K, S), torch.float32), cl_mean=new((B, K, S), torch.float32),
        cl_index=new((B, K, S), torch.float32), best_arm=new((B,), torch.int32),
        best_val=new((B,), torch.float32), best_cluster_arm=new((B,), torch.int32))
    if want_bound:
        out["bound"] = new((B, N, S), torch.float32)
    if want_arm_index:
        out["arm_index"] = new((B, N, S), torch.float32)
    return out
