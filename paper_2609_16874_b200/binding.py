"""Thin ctypes binding of ``libcpe.so`` (the C ABI declared in ``include/cpe.h``).

Argument marshalling only: every step of the decode path runs in the library's CUDA kernels.  The
functions carry the C names; pointers are passed as integers (``tensor.data_ptr()``) and streams as
``torch.cuda.Stream.cuda_stream``.  :class:`Decoder` bundles the bookkeeping (parameter struct,
workspace and output tensors owned by torch) for callers that hold torch tensors.

There is no CPU fallback: if the library cannot be loaded, importing a symbol from it raises.
"""
from __future__ import annotations

import ctypes
import math
import os

from . import build as _build

# ---- constants of include/cpe.h
CPE_F32, CPE_F16 = 0, 1
CPE_OK = 0
CPE_ERR_NULL, CPE_ERR_SIZE, CPE_ERR_DTYPE, CPE_ERR_ALIGN, CPE_ERR_WORKSPACE = -1, -2, -3, -4, -5
CPE_ERR_PARAM, CPE_ERR_CUDA, CPE_ERR_WHICH, CPE_ERR_NOMEM, CPE_ERR_STATIC_LIMIT = -6, -7, -8, -9, -10
CPE_ERR_BUSY = -11
CPE_STATIC_SCRATCH_BYTES = 8 << 20
CPE_STATIC_MAX_BINS = 1024
CPE_FLAG_WRITE_SCORES = 1
CPE_FLAG_EXACT_ASSIGN = 2
CPE_FLAG_KEEP_VOTES = 4
CPE_FLAG_FILTER_ASSIGN = 8
CPE_FLAG_REFINE = 16
CPE_FLAG_NO_PDL = 32
CPE_FLAG_TC_ALL_ROUNDS = 64
CPE_FLAG_TC_ONE_STAGE = 128
CPE_FLAG_MMA_ASSIGN = 256
CPE_FLAG_NO_PRUNE = 512
CPE_FLAG_PRUNE_ALL = 1024
CPE_FLAG_PRUNE_WALK_ONLY = 2048
CPE_FLAG_TEST_STALL = 4096
CPE_FLAG_PRUNE_ANY_SIZE = 8192
CPE_FLAG_SOFT_VOTE = 16384
CPE_FLAG_FUSE_PEAKS = 32768
CPE_STATUS_PEAK_OVERFLOW, CPE_STATUS_NONFINITE, CPE_STATUS_INTERNAL, CPE_STATUS_TIMEOUT = 1, 2, 4, 8
CPE_CNT_VOTING, CPE_CNT_NONFINITE, CPE_CNT_RAW_PEAKS, CPE_CNT_TRUNCATED, CPE_CNT_TAU_REJECTED = 0, 1, 2, 3, 4
CPE_CNT_FILTER_PAIRS, CPE_CNT_RESCORED, CPE_CNT_FULL_SCORED, CPE_CNT_N = 5, 6, 7, 8
(CPE_INT_VOTES, CPE_INT_PEAK_CELLS, CPE_INT_PEAK_VOTES, CPE_INT_PEAK_EMB, CPE_INT_PALETTE_W, CPE_INT_PALETTE_H,
 CPE_INT_BEST_SCORE, CPE_INT_SECOND_SCORE, CPE_INT_STATUS, CPE_INT_COUNTERS, CPE_INT_VOTE_SUMS,
 CPE_INT_PRUNE_STATE) = range(12)
CPE_STAGE_NAMES = ("clear", "decode_vote", "peaks", "lists", "assign")
CPE_STAGE_N = 5

EXPORTS = (
    "cpe_workspace_size", "cpe_init_workspace", "cpe_decode", "cpe_get_intermediate", "cpe_strerror",
    "cpe_last_cuda_error", "cpe_graph_create", "cpe_graph_launch", "cpe_graph_destroy", "cpe_graph_kernel_nodes",
    "cpe_profile_decode", "cpe_host_ctx_create", "cpe_host_decode", "cpe_host_submit", "cpe_host_wait",
    "cpe_host_ctx_traffic", "cpe_host_ctx_destroy",
    "cpe_decode_static", "cpe_soft_votes", "cpe_instance_masks", "cpe_channels_last_to_planar",
    "cpe_selftest_half_division",
)


class cpe_params(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_uint32),
        ("dtype", ctypes.c_int32),
        ("bins_w", ctypes.c_int32),
        ("bins_h", ctypes.c_int32),
        ("levels", ctypes.c_int32),
        ("vote_threshold", ctypes.c_int32),
        ("tau", ctypes.c_float),
        ("max_instances", ctypes.c_int32),
        ("flags", ctypes.c_uint32),
        ("soft_threshold", ctypes.c_float),
        ("workspace", ctypes.c_void_p),
        ("workspace_bytes", ctypes.c_size_t),
    ]


class CpeError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = cpe_strerror(code)
        if code == CPE_ERR_CUDA:
            msg += f" (cudaError {cpe_last_cuda_error()})"
        super().__init__(f"{where}: {msg} [{code}]")


_lib = None


def library_path() -> str:
    return _build.LIB


def load() -> ctypes.CDLL:
    """Load ``libcpe.so`` (building it with nvcc first if it is missing or older than its sources)."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.LIB
    if _build.is_stale():
        try:
            _build.build_library()
        except Exception as exc:  # no nvcc: an existing library is still usable, a missing one is fatal
            if not os.path.exists(path):
                raise RuntimeError(f"libcpe.so is missing and could not be built: {exc}") from exc
    lib = ctypes.CDLL(path)
    vp, ci, cs = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
    pp = ctypes.POINTER(cpe_params)
    lib.cpe_workspace_size.argtypes = [ci, ci, ci, ci, pp]
    lib.cpe_workspace_size.restype = cs
    lib.cpe_init_workspace.argtypes = [vp, ci, ci, ci, ci, pp]
    lib.cpe_init_workspace.restype = ci
    lib.cpe_decode.argtypes = [vp, vp, vp, ci, ci, ci, ci, pp, vp, vp, vp]
    lib.cpe_decode.restype = ci
    lib.cpe_get_intermediate.argtypes = [pp, ci, ci, ci, ci, ci, ctypes.POINTER(vp), ctypes.POINTER(cs)]
    lib.cpe_get_intermediate.restype = ci
    lib.cpe_strerror.argtypes = [ci]
    lib.cpe_strerror.restype = ctypes.c_char_p
    lib.cpe_last_cuda_error.argtypes = []
    lib.cpe_last_cuda_error.restype = ci
    lib.cpe_selftest_half_division.argtypes = [vp, vp]
    lib.cpe_selftest_half_division.restype = ci
    lib.cpe_graph_create.argtypes = [vp, vp, vp, ci, ci, ci, ci, pp, vp, vp, vp, ctypes.POINTER(vp)]
    lib.cpe_graph_create.restype = ci
    lib.cpe_graph_launch.argtypes = [vp, vp]
    lib.cpe_graph_launch.restype = ci
    lib.cpe_graph_destroy.argtypes = [vp]
    lib.cpe_graph_destroy.restype = None
    lib.cpe_graph_kernel_nodes.argtypes = [vp]
    lib.cpe_graph_kernel_nodes.restype = ci
    lib.cpe_profile_decode.argtypes = [vp, vp, vp, ci, ci, ci, ci, pp, vp, vp, vp, ci, ctypes.POINTER(ctypes.c_float)]
    lib.cpe_profile_decode.restype = ci
    lib.cpe_host_ctx_create.argtypes = [ci, ci, ci, ci, pp, ci, ctypes.POINTER(vp)]
    lib.cpe_host_ctx_create.restype = ci
    lib.cpe_host_decode.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.cpe_host_decode.restype = ci
    lib.cpe_host_submit.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.cpe_host_submit.restype = ci
    lib.cpe_host_wait.argtypes = [vp]
    lib.cpe_host_wait.restype = ci
    lib.cpe_host_ctx_traffic.argtypes = [vp, ctypes.POINTER(cs), ctypes.POINTER(cs)]
    lib.cpe_host_ctx_traffic.restype = ci
    lib.cpe_host_ctx_destroy.argtypes = [vp]
    lib.cpe_host_ctx_destroy.restype = None
    lib.cpe_decode_static.argtypes = [vp, vp, vp, ci, ci, ci, ci, pp, vp, vp, vp]
    lib.cpe_decode_static.restype = ci
    lib.cpe_soft_votes.argtypes = [vp, vp, vp, ci, ci, ci, ci, pp, vp]
    lib.cpe_soft_votes.restype = ci
    lib.cpe_instance_masks.argtypes = [vp, vp, ci, ci, ci, ci, vp, vp]
    lib.cpe_instance_masks.restype = ci
    lib.cpe_channels_last_to_planar.argtypes = [vp, vp, vp, ci, ci, ci, ci, ci]
    lib.cpe_channels_last_to_planar.restype = ci
    _lib = lib
    return lib


def make_params(dtype: int, bins_w: int, bins_h: int, levels: int = 0, vote_threshold: int = 8, tau: float = math.inf,
                max_instances: int = 1024, flags: int = 0, workspace: int = 0, workspace_bytes: int = 0,
                soft_threshold: float = 0.0) -> cpe_params:
    return cpe_params(ctypes.sizeof(cpe_params), dtype, bins_w, bins_h, levels, vote_threshold, tau, max_instances,
                      flags, soft_threshold, workspace or None, workspace_bytes)


# ---- the C entry points, same names, integer pointers

def cpe_strerror(code: int) -> str:
    return load().cpe_strerror(code).decode()


def cpe_last_cuda_error() -> int:
    return int(load().cpe_last_cuda_error())


def cpe_selftest_half_division(stream, out_mismatches: int) -> int:
    return int(load().cpe_selftest_half_division(stream, out_mismatches))


def cpe_workspace_size(B, H, W, F, params: cpe_params) -> int:
    return int(load().cpe_workspace_size(B, H, W, F, ctypes.byref(params)))


def cpe_init_workspace(stream, B, H, W, F, params: cpe_params) -> int:
    return int(load().cpe_init_workspace(stream, B, H, W, F, ctypes.byref(params)))


def cpe_decode(stream, emb, fg_mask, B, H, W, F, params: cpe_params, out_labels, out_centroids, out_count) -> int:
    return int(load().cpe_decode(stream, emb, fg_mask or None, B, H, W, F, ctypes.byref(params), out_labels,
                                 out_centroids, out_count))


def cpe_decode_static(stream, emb, fg_mask, B, H, W, F, params: cpe_params, out_labels, out_centroids, out_count) -> int:
    """``cpe_decode`` on the library's built-in scratch array: no workspace, no allocation (see ``cpe.h``)."""
    return int(load().cpe_decode_static(stream, emb, fg_mask or None, B, H, W, F, ctypes.byref(params), out_labels,
                                        out_centroids, out_count))


def cpe_soft_votes(stream, emb, fg_mask, B, H, W, F, params: cpe_params, out_hist) -> int:
    """The soft-vote histogram of Eq. 6, ``float [B, bins_h, bins_w]`` (see ``cpe.h``)."""
    return int(load().cpe_soft_votes(stream, emb, fg_mask or None, B, H, W, F, ctypes.byref(params), out_hist))


def cpe_instance_masks(stream, labels, B, H, W, n_planes, out_planes, out_pixels) -> int:
    """One-hot mask planes and per-instance pixel counters of a label map (see ``cpe.h``)."""
    return int(load().cpe_instance_masks(stream, labels, B, H, W, n_planes, out_planes or None, out_pixels or None))


def cpe_channels_last_to_planar(stream, emb_nhwc, emb_planar, B, H, W, F, dtype) -> int:
    """``[B, H, W, 4F]`` to the planar ``[B, 4F, H, W]`` that ``cpe_decode`` reads (see ``cpe.h``)."""
    return int(load().cpe_channels_last_to_planar(stream, emb_nhwc, emb_planar, B, H, W, F, dtype))


def cpe_get_intermediate(params: cpe_params, which, B, H, W, F):
    ptr, size = ctypes.c_void_p(), ctypes.c_size_t()
    rc = int(load().cpe_get_intermediate(ctypes.byref(params), which, B, H, W, F, ctypes.byref(ptr), ctypes.byref(size)))
    return rc, (ptr.value or 0), int(size.value)


def cpe_graph_create(stream, emb, fg_mask, B, H, W, F, params: cpe_params, out_labels, out_centroids, out_count):
    g = ctypes.c_void_p()
    rc = int(load().cpe_graph_create(stream, emb, fg_mask or None, B, H, W, F, ctypes.byref(params), out_labels,
                                     out_centroids, out_count, ctypes.byref(g)))
    return rc, g.value


def cpe_graph_launch(graph, stream) -> int:
    return int(load().cpe_graph_launch(graph, stream))


def cpe_graph_destroy(graph) -> None:
    load().cpe_graph_destroy(graph)


def cpe_graph_kernel_nodes(graph) -> int:
    return int(load().cpe_graph_kernel_nodes(graph))


def cpe_profile_decode(stream, emb, fg_mask, B, H, W, F, params, out_labels, out_centroids, out_count, iters):
    ms = (ctypes.c_float * CPE_STAGE_N)()
    rc = int(load().cpe_profile_decode(stream, emb, fg_mask or None, B, H, W, F, ctypes.byref(params), out_labels,
                                       out_centroids, out_count, iters, ms))
    return rc, [float(x) for x in ms]


def cpe_host_ctx_create(B, H, W, F, params: cpe_params, has_mask: bool):
    c = ctypes.c_void_p()
    rc = int(load().cpe_host_ctx_create(B, H, W, F, ctypes.byref(params), int(bool(has_mask)), ctypes.byref(c)))
    return rc, c.value


def cpe_host_decode(ctx, emb_host, fg_mask_host, labels_host, centroids_host, count_host) -> int:
    return int(load().cpe_host_decode(ctx, emb_host, fg_mask_host or None, labels_host, centroids_host, count_host))


def cpe_host_submit(ctx, emb_host, fg_mask_host, labels_host, centroids_host, count_host) -> int:
    return int(load().cpe_host_submit(ctx, emb_host, fg_mask_host or None, labels_host, centroids_host, count_host))


def cpe_host_wait(ctx) -> int:
    return int(load().cpe_host_wait(ctx))


def cpe_host_ctx_traffic(ctx):
    a, b = ctypes.c_size_t(), ctypes.c_size_t()
    rc = int(load().cpe_host_ctx_traffic(ctx, ctypes.byref(a), ctypes.byref(b)))
    return rc, int(a.value), int(b.value)


def cpe_host_ctx_destroy(ctx) -> None:
    load().cpe_host_ctx_destroy(ctx)


def _check(rc: int, where: str) -> None:
    if rc != CPE_OK:
        raise CpeError(rc, where)


# ---- bookkeeping for torch callers (device memory and streams come from torch; no arithmetic here)

class Decoder:
    """Holds the parameter struct, the workspace and the output tensors for one problem shape on one device."""

    def __init__(self, B, H, W, F, dtype, bins_w, bins_h, vote_threshold=8, tau=math.inf, max_instances=1024,
                 levels=0, write_scores=False, device="cuda:0", exact_assign=False, keep_votes=False, filter_assign=False,
                 refine=False, flags=0, soft_threshold=None):
        import torch
        self.torch = torch
        self.B, self.H, self.W, self.F = B, H, W, F
        self.device = torch.device(device)
        code = {"f32": CPE_F32, "f16": CPE_F16, torch.float32: CPE_F32, torch.float16: CPE_F16}[dtype]
        self.emb_dtype = torch.float32 if code == CPE_F32 else torch.float16
        flags = ((CPE_FLAG_WRITE_SCORES if write_scores else 0) | (CPE_FLAG_EXACT_ASSIGN if exact_assign else 0) |
                 (CPE_FLAG_KEEP_VOTES if keep_votes else 0) | (CPE_FLAG_FILTER_ASSIGN if filter_assign else 0) |
                 (CPE_FLAG_REFINE if refine else 0) | (CPE_FLAG_SOFT_VOTE if soft_threshold is not None else 0) |
                 int(flags))
        self.params = make_params(code, bins_w, bins_h, levels, vote_threshold, tau, max_instances, flags,
                                  soft_threshold=float(soft_threshold or 0.0))
        n = cpe_workspace_size(B, H, W, F, self.params)
        if n == 0:
            raise CpeError(CPE_ERR_SIZE, "cpe_workspace_size")
        with torch.cuda.device(self.device):
            self.workspace = torch.empty(n, dtype=torch.uint8, device=self.device)
            self.params.workspace = self.workspace.data_ptr()
            self.params.workspace_bytes = n
            self.labels = torch.empty((B, H, W), dtype=torch.int32, device=self.device)
            self.centroids = torch.zeros((B, max_instances, 2), dtype=torch.float32, device=self.device)
            self.count = torch.zeros((B,), dtype=torch.int32, device=self.device)
            stream = torch.cuda.current_stream(self.device)
            _check(cpe_init_workspace(stream.cuda_stream, B, H, W, F, self.params), "cpe_init_workspace")
        self._graphs = []

    def _args(self, emb, fg):
        assert emb.is_cuda and emb.is_contiguous() and emb.dtype == self.emb_dtype
        assert tuple(emb.shape) == (self.B, 4 * self.F, self.H, self.W), tuple(emb.shape)
        if fg is not None:
            assert fg.is_cuda and fg.is_contiguous() and fg.dtype == self.torch.uint8
            assert tuple(fg.shape) == (self.B, self.H, self.W)
        return (emb.data_ptr(), 0 if fg is None else fg.data_ptr(), self.B, self.H, self.W, self.F, self.params,
                self.labels.data_ptr(), self.centroids.data_ptr(), self.count.data_ptr())

    def decode(self, emb, fg=None, stream=None):
        """Enqueue one decode on ``stream`` (default: torch's current stream); results land in ``labels``,
        ``centroids`` and ``count`` once the stream reaches that point."""
        s = stream if stream is not None else self.torch.cuda.current_stream(self.device)
        _check(cpe_decode(s.cuda_stream, *self._args(emb, fg)), "cpe_decode")
        return self.labels, self.centroids, self.count

    def soft_votes(self, emb, fg=None, out=None, stream=None):
        """Enqueue the soft-vote histogram of Eq. 6 of these tensors; returns ``float32 [B, bins_h, bins_w]``."""
        torch = self.torch
        s = stream if stream is not None else torch.cuda.current_stream(self.device)
        if out is None:
            out = torch.empty((self.B, self.params.bins_h, self.params.bins_w), dtype=torch.float32, device=self.device)
        _check(cpe_soft_votes(s.cuda_stream, emb.data_ptr(), 0 if fg is None else fg.data_ptr(), self.B, self.H, self.W,
                              self.F, self.params, out.data_ptr()), "cpe_soft_votes")
        return out

    def instance_masks(self, n_planes, want_planes=True, stream=None):
        """One-hot planes ``uint8 [B, n_planes, H, W]`` (or None) and counters ``int32 [B, n_planes]`` of ``labels``."""
        torch = self.torch
        s = stream if stream is not None else torch.cuda.current_stream(self.device)
        planes = (torch.empty((self.B, n_planes, self.H, self.W), dtype=torch.uint8, device=self.device)
                  if want_planes else None)
        pixels = torch.empty((self.B, n_planes), dtype=torch.int32, device=self.device)
        _check(cpe_instance_masks(s.cuda_stream, self.labels.data_ptr(), self.B, self.H, self.W, n_planes,
                                  0 if planes is None else planes.data_ptr(), pixels.data_ptr()), "cpe_instance_masks")
        return planes, pixels

    def capture(self, emb, fg=None, stream=None):
        """Capture one decode of these tensors into a CUDA graph; returns a handle for :meth:`replay`."""
        s = stream if stream is not None else self.torch.cuda.current_stream(self.device)
        rc, g = cpe_graph_create(s.cuda_stream, *self._args(emb, fg))
        _check(rc, "cpe_graph_create")
        self._graphs.append(g)
        return g

    def replay(self, graph, stream=None):
        s = stream if stream is not None else self.torch.cuda.current_stream(self.device)
        _check(cpe_graph_launch(graph, s.cuda_stream), "cpe_graph_launch")

    def profile(self, emb, fg=None, iters=10, stream=None):
        """Mean device milliseconds of each stage over ``iters`` decodes (synchronises)."""
        s = stream if stream is not None else self.torch.cuda.current_stream(self.device)
        rc, ms = cpe_profile_decode(s.cuda_stream, *self._args(emb, fg), iters)
        _check(rc, "cpe_profile_decode")
        return dict(zip(CPE_STAGE_NAMES, ms))

    def intermediate(self, which):
        """A torch view (no copy) of an intermediate inside the workspace."""
        torch = self.torch
        rc, ptr, size = cpe_get_intermediate(self.params, which, self.B, self.H, self.W, self.F)
        _check(rc, "cpe_get_intermediate")
        off = ptr - self.workspace.data_ptr()
        raw = self.workspace[off:off + size]
        K, D = self.params.max_instances, 4 * self.F
        bw, bh = self.params.bins_w, self.params.bins_h
        shapes = {
            CPE_INT_VOTES: (torch.int32, (self.B, bh, bw)),
            CPE_INT_PEAK_CELLS: (torch.int32, (self.B, K)),
            CPE_INT_PEAK_VOTES: (torch.int32, (self.B, K)),
            CPE_INT_PEAK_EMB: (torch.float32, (self.B, K, D)),
            CPE_INT_PALETTE_W: (torch.float32, (bw, 2 * self.F)),
            CPE_INT_PALETTE_H: (torch.float32, (bh, 2 * self.F)),
            CPE_INT_BEST_SCORE: (torch.float32, (self.B, self.H, self.W)),
            CPE_INT_SECOND_SCORE: (torch.float32, (self.B, self.H, self.W)),
            CPE_INT_STATUS: (torch.int32, (self.B,)),
            CPE_INT_COUNTERS: (torch.int32, (self.B, CPE_CNT_N)),
            CPE_INT_VOTE_SUMS: (torch.int64, (self.B, bh, bw, 2)),
            CPE_INT_PRUNE_STATE: (torch.int32, (self.B, 12)),
        }
        dt, shape = shapes[which]
        return raw.view(dt).view(shape)

    def close(self):
        for g in self._graphs:
            cpe_graph_destroy(g)
        self._graphs = []

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class HostDecoder:
    """End-to-end front end for host buffers (``cpe_host_ctx_*``): numpy in, numpy out, copies included."""

    def __init__(self, B, H, W, F, dtype, bins_w, bins_h, vote_threshold=8, tau=math.inf, max_instances=1024,
                 levels=0, has_mask=True, refine=False, flags=0, soft_threshold=None):
        code = {"f32": CPE_F32, "f16": CPE_F16}[dtype]
        self.params = make_params(code, bins_w, bins_h, levels, vote_threshold, tau, max_instances,
                                  (CPE_FLAG_REFINE if refine else 0) |
                                  (CPE_FLAG_SOFT_VOTE if soft_threshold is not None else 0) | int(flags),
                                  soft_threshold=float(soft_threshold or 0.0))
        self.shape = (B, H, W, F)
        self.max_instances = max_instances
        rc, self.ctx = cpe_host_ctx_create(B, H, W, F, self.params, has_mask)
        _check(rc, "cpe_host_ctx_create")
        rc, self.h2d_bytes, self.d2h_bytes = cpe_host_ctx_traffic(self.ctx)
        _check(rc, "cpe_host_ctx_traffic")

    def decode_ptrs(self, emb_ptr, fg_ptr, labels_ptr, centroids_ptr, count_ptr):
        _check(cpe_host_decode(self.ctx, emb_ptr, fg_ptr, labels_ptr, centroids_ptr, count_ptr), "cpe_host_decode")

    def decode(self, emb, fg, labels, centroids, count):
        """numpy (or pinned torch CPU) arrays, contiguous, of the context's shapes."""
        ptr = lambda a: 0 if a is None else (a.data_ptr() if hasattr(a, "data_ptr") else a.ctypes.data)
        self.decode_ptrs(ptr(emb), ptr(fg), ptr(labels), ptr(centroids), ptr(count))

    def submit(self, emb, fg, labels, centroids, count):
        """Enqueue a decode (at most two in flight); the arrays must stay alive and untouched until `wait`."""
        ptr = lambda a: 0 if a is None else (a.data_ptr() if hasattr(a, "data_ptr") else a.ctypes.data)
        _check(cpe_host_submit(self.ctx, ptr(emb), ptr(fg), ptr(labels), ptr(centroids), ptr(count)), "cpe_host_submit")

    def wait(self):
        """Return when the oldest submission's results have arrived."""
        _check(cpe_host_wait(self.ctx), "cpe_host_wait")

    def close(self):
        if self.ctx:
            cpe_host_ctx_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
