"""ctypes front end of the CPU oracle (``cpe_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the benchmark's
CPU-baseline leg.  The CUDA library and its Python binding never import this package and share
no code with it.  Every function takes and returns host ``numpy`` arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "cpe_oracle.c")
_LIB = os.path.join(_HERE, "libcpe_oracle.so")
_lock = threading.Lock()
_lib = None

CNT_VOTING, CNT_NONFINITE, CNT_RAW_PEAKS, CNT_TRUNCATED, CNT_TAU_REJECTED, CNT_N = 0, 1, 2, 3, 4, 8
F32, F16 = 0, 1


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no contraction, no fast-math) next to its source."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + f".{os.getpid()}.tmp"
            cmd = ["gcc", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-shared", "-fPIC",
                   "-o", tmp, _SRC, "-lm"]
            subprocess.run(cmd, check=True)
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        c_int, c_dbl, vp = ctypes.c_int, ctypes.c_double, ctypes.c_void_p
        lib.cpe_oracle_set_threads.argtypes = [c_int]
        lib.cpe_oracle_max_threads.restype = c_int
        lib.cpe_oracle_get_threads.restype = c_int
        lib.cpe_oracle_bin_position.argtypes = [c_int, c_int]
        lib.cpe_oracle_bin_position.restype = c_dbl
        lib.cpe_oracle_palette.argtypes = [c_int, c_int, vp]
        lib.cpe_oracle_palette.restype = None
        lib.cpe_oracle_atan2_ht.argtypes = [ctypes.c_float, ctypes.c_float]
        lib.cpe_oracle_atan2_ht.restype = ctypes.c_float
        lib.cpe_oracle_atan2_ht_array.argtypes = [vp, vp, ctypes.c_int64, vp]
        lib.cpe_oracle_atan2_ht_array.restype = None
        lib.cpe_oracle_decode_axis_array.argtypes = [vp, ctypes.c_int64, c_int, c_int, vp]
        lib.cpe_oracle_decode_axis_array.restype = None
        lib.cpe_oracle_half_to_float_array.argtypes = [vp, ctypes.c_int64, vp]
        lib.cpe_oracle_half_to_float_array.restype = None
        lib.cpe_oracle_decode_axis.argtypes = [vp, c_int, c_int]
        lib.cpe_oracle_decode_axis.restype = ctypes.c_float
        lib.cpe_oracle_cell_of.argtypes = [ctypes.c_float, c_int]
        lib.cpe_oracle_cell_of.restype = c_int
        lib.cpe_oracle_votes.argtypes = [vp, c_int, vp] + [c_int] * 7 + [vp] * 4
        lib.cpe_oracle_votes.restype = c_int
        lib.cpe_oracle_peaks.argtypes = [vp, c_int, c_int, c_int, c_int, vp, vp, vp]
        lib.cpe_oracle_peaks.restype = c_int
        lib.cpe_oracle_real_peaks.argtypes = [vp, c_int, c_int, c_dbl, c_int, vp, vp]
        lib.cpe_oracle_real_peaks.restype = c_int
        lib.cpe_oracle_centroid_px.argtypes = [c_int] * 6 + [vp]
        lib.cpe_oracle_centroid_px.restype = None
        lib.cpe_oracle_assign_image.argtypes = [vp, c_int, vp, c_int, c_int, c_int, vp, vp, c_int, vp, c_int,
                                                c_dbl, vp, ctypes.c_int64, vp, vp, vp, vp, vp]
        lib.cpe_oracle_assign_image.restype = c_int
        lib.cpe_oracle_vote_sums.argtypes = [vp, vp, c_int, c_int, c_int, c_int, vp]
        lib.cpe_oracle_vote_sums.restype = c_int
        lib.cpe_oracle_refined_peaks.argtypes = [vp, vp, c_int, c_int, vp] + [c_int] * 4 + [vp, vp, vp]
        lib.cpe_oracle_refined_peaks.restype = c_int
        lib.cpe_oracle_decode.argtypes = ([vp, vp] + [c_int] * 9 + [c_dbl, c_int] + [vp] * 9)
        lib.cpe_oracle_decode.restype = c_int
        lib.cpe_oracle_soft_votes.argtypes = [vp, c_int, vp] + [c_int] * 6 + [vp, c_int, vp]
        lib.cpe_oracle_soft_votes.restype = c_int
        lib.cpe_oracle_instance_masks.argtypes = [vp, c_int, c_int, c_int, c_int, vp, vp]
        lib.cpe_oracle_instance_masks.restype = c_int
        _lib = lib
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _dtype_code(emb: np.ndarray) -> int:
    if emb.dtype == np.float32:
        return F32
    if emb.dtype == np.float16:
        return F16
    raise TypeError(f"embedding must be float32 or float16, got {emb.dtype}")


def set_threads(n: int) -> None:
    _load().cpe_oracle_set_threads(int(n))


def max_threads() -> int:
    return int(_load().cpe_oracle_max_threads())


def bin_position(n: int, i: int) -> float:
    """Eq. 9 position of bin ``i`` (1-based) of an ``n``-bin palette."""
    return float(_load().cpe_oracle_bin_position(n, i))


def palette(n: int, F: int) -> np.ndarray:
    """Eq. 9 palette, ``[n, 2F]`` float32, columns (sin, cos) per harmonic."""
    out = np.empty((n, 2 * F), np.float32)
    _load().cpe_oracle_palette(n, F, _ptr(out))
    return out


def atan2_ht(y, x) -> np.ndarray:
    """Element-wise binary32 atan2 in half-turns (the estimate's building block)."""
    y = np.asarray(y, np.float32)
    x = np.asarray(x, np.float32)
    yb, xb = np.broadcast_arrays(y, x)
    yb, xb = np.ascontiguousarray(yb), np.ascontiguousarray(xb)
    out = np.empty(yb.shape, np.float32)
    _load().cpe_oracle_atan2_ht_array(_ptr(yb), _ptr(xb), out.size, _ptr(out))
    return out


def half_to_float(bits: np.ndarray) -> np.ndarray:
    """The oracle's own binary16 -> binary32 widening of raw uint16 bit patterns."""
    bits = np.ascontiguousarray(bits, np.uint16)
    out = np.empty(bits.shape, np.float32)
    _load().cpe_oracle_half_to_float_array(_ptr(bits), bits.size, _ptr(out))
    return out


def decode_axis(sc: np.ndarray, levels: int = 0):
    """Estimate of p from one axis' (sin, cos) channels: ``[2F]`` -> float, ``[n, 2F]`` -> ``[n]`` float32."""
    sc = np.ascontiguousarray(sc, np.float32)
    if sc.ndim == 1:
        return float(_load().cpe_oracle_decode_axis(_ptr(sc), sc.shape[0] // 2, levels))
    out = np.empty(sc.shape[0], np.float32)
    _load().cpe_oracle_decode_axis_array(_ptr(sc), sc.shape[0], sc.shape[1] // 2, levels, _ptr(out))
    return out


def cell_of(p: float, n: int) -> int:
    return int(_load().cpe_oracle_cell_of(float(np.float32(p)), n))


def votes(emb: np.ndarray, fg, bins_w: int, bins_h: int, levels: int = 0, want_est=False, want_cell=False):
    """Hard-vote map ``[B, bins_h, bins_w]`` uint32 (+ optional per-pixel estimate / cell, counters)."""
    emb = np.ascontiguousarray(emb)
    B, D, H, W = emb.shape
    F = D // 4
    fgc = None if fg is None else np.ascontiguousarray(fg, np.uint8)
    V = np.empty((B, bins_h, bins_w), np.uint32)
    est = np.empty((B, H, W, 2), np.float32) if want_est else None
    cell = np.empty((B, H, W), np.int32) if want_cell else None
    counters = np.zeros((B, CNT_N), np.int64)
    rc = _load().cpe_oracle_votes(_ptr(emb), _dtype_code(emb), _ptr(fgc), B, H, W, F, bins_w, bins_h, levels,
                                  _ptr(V), _ptr(est), _ptr(cell), _ptr(counters))
    if rc:
        raise RuntimeError(f"cpe_oracle_votes failed: {rc}")
    return {"votes": V, "est": est, "cell": cell, "counters": counters}


def peaks(V: np.ndarray, T_v: int, K_max: int):
    """Peak list of ONE vote map ``[bins_h, bins_w]``: (cells ascending, their votes, raw count)."""
    V = np.ascontiguousarray(V, np.uint32)
    bh, bw = V.shape
    cells = np.full(K_max, -1, np.int32)
    pv = np.zeros(K_max, np.uint32)
    raw = np.zeros(1, np.int32)
    kept = _load().cpe_oracle_peaks(_ptr(V), bw, bh, T_v, K_max, _ptr(cells), _ptr(pv), _ptr(raw))
    return cells[:kept].copy(), pv[:kept].copy(), int(raw[0])


def real_peaks(Hmap: np.ndarray, threshold: float, K_max: int):
    """The paper's literal local-maxima search on ONE real-valued map ``[bins_h, bins_w]``: (cells ascending, raw count)."""
    Hmap = np.ascontiguousarray(Hmap, np.float64)
    bh, bw = Hmap.shape
    cells = np.full(K_max, -1, np.int32)
    raw = np.zeros(1, np.int32)
    kept = _load().cpe_oracle_real_peaks(_ptr(Hmap), bw, bh, float(threshold), K_max, _ptr(cells), _ptr(raw))
    return cells[:kept].copy(), int(raw[0])


def decode_soft(emb: np.ndarray, fg, bins_w: int, bins_h: int, threshold: float, tau=np.inf, K_max: int = 1024):
    """The paper's own chain: soft-vote histogram (Eq. 6), strict local maxima above ``threshold`` (Sec. 3.2),
    assignment to the peaks' palette rows (Eq. 7-8).  Returns the histogram, the peak lists and the label maps."""
    emb = np.ascontiguousarray(emb)
    B, D, H, W = emb.shape
    Hmap = soft_votes(emb, fg, bins_w, bins_h)
    labels = np.empty((B, H, W), np.int32)
    best = np.empty((B, H, W), np.float64)
    second = np.empty((B, H, W), np.float64)
    pc_all = np.full((B, K_max), -1, np.int32)
    count = np.zeros(B, np.int32)
    centroids = np.full((B, K_max, 2), np.nan, np.float32)
    for b in range(B):
        pc, raw = real_peaks(Hmap[b], threshold, K_max)
        a = assign_image(emb[b], None if fg is None else fg[b], bins_w, bins_h, pc, tau)
        k = pc.shape[0]
        count[b] = k
        pc_all[b, :k] = pc
        for i, lin in enumerate(pc):
            centroids[b, i] = centroid_px(lin % bins_w, lin // bins_w, bins_w, bins_h, H, W)
        labels[b], best[b], second[b] = a["labels"], a["best"], a["second"]
    return {"hist": Hmap, "labels": labels, "best": best, "second": second, "peak_cell": pc_all, "count": count,
            "centroids": centroids}


def centroid_px(cx: int, cy: int, bins_w: int, bins_h: int, H: int, W: int):
    out = np.empty(2, np.float32)
    _load().cpe_oracle_centroid_px(cx, cy, bins_w, bins_h, H, W, _ptr(out))
    return out


def assign_image(emb_img: np.ndarray, fg_img, bins_w: int, bins_h: int, peak_cell: np.ndarray, tau=np.inf,
                 idx=None, peak_emb=None):
    """Eq. 7-8 for one image ``[4F, H, W]``; ``idx`` restricts the work to sampled flat pixel indices.

    ``peak_emb`` ``[count, 4F]`` float32 replaces the palette rows of the peaks' bins as the candidates."""
    emb_img = np.ascontiguousarray(emb_img)
    D, H, W = emb_img.shape
    F = D // 4
    fgc = None if fg_img is None else np.ascontiguousarray(fg_img, np.uint8)
    Pw, Ph = palette(bins_w, F), palette(bins_h, F)
    pc = np.ascontiguousarray(peak_cell, np.int32)
    if idx is not None:
        idx = np.ascontiguousarray(idx, np.int64)
        n = idx.shape[0]
        shape = (n,)
    else:
        n = 0
        shape = (H, W)
    labels = np.empty(shape, np.int32)
    best = np.empty(shape, np.float64)
    second = np.empty(shape, np.float64)
    rej = np.zeros(1, np.int64)
    if peak_emb is not None:
        peak_emb = np.ascontiguousarray(peak_emb, np.float32)
        assert peak_emb.shape == (pc.shape[0], D)
    rc = _load().cpe_oracle_assign_image(_ptr(emb_img), _dtype_code(emb_img), _ptr(fgc), H, W, F, _ptr(Pw), _ptr(Ph),
                                         bins_w, _ptr(pc), pc.shape[0], float(tau), _ptr(idx), n, _ptr(labels),
                                         _ptr(best), _ptr(second), _ptr(rej), _ptr(peak_emb))
    if rc:
        raise RuntimeError(f"cpe_oracle_assign_image failed: {rc}")
    return {"labels": labels, "best": best, "second": second, "tau_rejected": int(rej[0])}


def decode(emb: np.ndarray, fg, bins_w: int, bins_h: int, T_v: int = 8, tau=np.inf, K_max: int = 1024,
           levels: int = 0, want_scores: bool = True):
    """The whole chain on a batch ``[B, 4F, H, W]``; returns every output and intermediate."""
    emb = np.ascontiguousarray(emb)
    B, D, H, W = emb.shape
    F = D // 4
    fgc = None if fg is None else np.ascontiguousarray(fg, np.uint8)
    labels = np.empty((B, H, W), np.int32)
    centroids = np.full((B, K_max, 2), np.nan, np.float32)
    count = np.zeros(B, np.int32)
    V = np.empty((B, bins_h, bins_w), np.uint32)
    pc = np.full((B, K_max), -1, np.int32)
    pv = np.zeros((B, K_max), np.uint32)
    best = np.empty((B, H, W), np.float64) if want_scores else None
    second = np.empty((B, H, W), np.float64) if want_scores else None
    counters = np.zeros((B, CNT_N), np.int64)
    rc = _load().cpe_oracle_decode(_ptr(emb), _ptr(fgc), B, H, W, F, _dtype_code(emb), bins_w, bins_h, levels, T_v,
                                   float(tau), K_max, _ptr(labels), _ptr(centroids), _ptr(count), _ptr(V), _ptr(pc),
                                   _ptr(pv), _ptr(best), _ptr(second), _ptr(counters))
    if rc:
        raise RuntimeError(f"cpe_oracle_decode failed: {rc}")
    return {"labels": labels, "centroids": centroids, "count": count, "votes": V, "peak_cell": pc,
            "peak_votes": pv, "best": best, "second": second, "counters": counters}


def vote_sums(est: np.ndarray, cell: np.ndarray, bins_w: int, bins_h: int) -> np.ndarray:
    """Fixed-point (2^-24) sums of the estimates per cell, ``[B, bins_h, bins_w, 2]`` int64."""
    est = np.ascontiguousarray(est, np.float32)
    cell = np.ascontiguousarray(cell, np.int32)
    B, H, W = cell.shape
    sums = np.empty((B, bins_h, bins_w, 2), np.int64)
    rc = _load().cpe_oracle_vote_sums(_ptr(est), _ptr(cell), B, H, W, bins_w * bins_h, _ptr(sums))
    if rc:
        raise RuntimeError(f"cpe_oracle_vote_sums failed: {rc}")
    return sums


def refined_peaks(V: np.ndarray, sums: np.ndarray, peak_cell: np.ndarray, F: int, H: int, W: int):
    """Refined candidates of ONE image: gamma(mean estimate of the peak's 3x3 window) and the mean in pixels."""
    V = np.ascontiguousarray(V, np.uint32)
    sums = np.ascontiguousarray(sums, np.int64)
    pc = np.ascontiguousarray(peak_cell, np.int32)
    bh, bw = V.shape
    K = pc.shape[0]
    pe = np.empty((K, 4 * F), np.float32)
    cen = np.empty((K, 2), np.float32)
    mean = np.empty((K, 2), np.float64)
    rc = _load().cpe_oracle_refined_peaks(_ptr(V), _ptr(sums), bw, bh, _ptr(pc), K, F, H, W, _ptr(pe), _ptr(cen),
                                          _ptr(mean))
    if rc:
        raise RuntimeError(f"cpe_oracle_refined_peaks failed: {rc}")
    return {"peak_emb": pe, "centroids": cen, "mean": mean}


def decode_refined(emb: np.ndarray, fg, bins_w: int, bins_h: int, T_v: int = 8, tau=np.inf, K_max: int = 1024,
                   levels: int = 0):
    """The chain with sub-cell refined candidates: votes and sums, peaks, gamma(mean), assignment."""
    emb = np.ascontiguousarray(emb)
    B, D, H, W = emb.shape
    F = D // 4
    v = votes(emb, fg, bins_w, bins_h, levels, want_est=True, want_cell=True)
    sums = vote_sums(v["est"], v["cell"], bins_w, bins_h)
    labels = np.empty((B, H, W), np.int32)
    best = np.empty((B, H, W), np.float64)
    second = np.empty((B, H, W), np.float64)
    centroids = np.full((B, K_max, 2), np.nan, np.float32)
    peak_emb = np.zeros((B, K_max, D), np.float32)
    pc_all = np.full((B, K_max), -1, np.int32)
    count = np.zeros(B, np.int32)
    counters = v["counters"].copy()
    for b in range(B):
        pc, _, raw = peaks(v["votes"][b], T_v, K_max)
        r = refined_peaks(v["votes"][b], sums[b], pc, F, H, W)
        a = assign_image(emb[b], None if fg is None else fg[b], bins_w, bins_h, pc, tau, peak_emb=r["peak_emb"])
        k = pc.shape[0]
        count[b] = k
        pc_all[b, :k] = pc
        centroids[b, :k] = r["centroids"]
        peak_emb[b, :k] = r["peak_emb"]
        labels[b], best[b], second[b] = a["labels"], a["best"], a["second"]
        counters[b, CNT_RAW_PEAKS] = raw
        counters[b, CNT_TRUNCATED] = raw - k
        counters[b, CNT_TAU_REJECTED] = a["tau_rejected"]
    return {"labels": labels, "centroids": centroids, "count": count, "votes": v["votes"], "sums": sums,
            "peak_cell": pc_all, "peak_emb": peak_emb, "best": best, "second": second, "counters": counters}


def soft_votes(emb: np.ndarray, fg, bins_w: int, bins_h: int, sample_cells=None) -> np.ndarray:
    """The soft-vote histogram of Eq. 6 in binary64: ``[B, bins_h, bins_w]``, or ``[B, n]`` for the ``n`` linear cells
    ``b * bins_w + a`` listed in ``sample_cells``."""
    emb = np.ascontiguousarray(emb)
    B, D, H, W = emb.shape
    F = D // 4
    fgc = None if fg is None else np.ascontiguousarray(fg, np.uint8)
    if sample_cells is None:
        cells, n = None, 0
        out = np.empty((B, bins_h, bins_w), np.float64)
    else:
        cells = np.ascontiguousarray(sample_cells, np.int32)
        n = int(cells.size)
        out = np.empty((B, n), np.float64)
    rc = _load().cpe_oracle_soft_votes(_ptr(emb), _dtype_code(emb), _ptr(fgc), B, H, W, F, bins_w, bins_h, _ptr(cells), n,
                                       _ptr(out))
    if rc:
        raise RuntimeError(f"cpe_oracle_soft_votes failed: {rc}")
    return out


def instance_masks(labels: np.ndarray, n_planes: int, want_planes: bool = True):
    """One-hot mask planes ``uint8 [B, n_planes, H, W]`` (or None) and pixel counters ``uint32 [B, n_planes]`` of a
    label map (0 = none, m + 1 = mask m)."""
    labels = np.ascontiguousarray(labels, np.int32)
    B, H, W = labels.shape
    planes = np.empty((B, n_planes, H, W), np.uint8) if want_planes else None
    pixels = np.empty((B, n_planes), np.uint32)
    rc = _load().cpe_oracle_instance_masks(_ptr(labels), B, H, W, n_planes, _ptr(planes), _ptr(pixels))
    if rc:
        raise RuntimeError(f"cpe_oracle_instance_masks failed: {rc}")
    return planes, pixels
