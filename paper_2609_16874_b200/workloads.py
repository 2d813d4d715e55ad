"""Seeded synthetic inputs shaped like the five benchmark configurations.

This module only *makes inputs* (instance maps, their sinusoidal centroid encodings plus noise,
foreground masks).  It holds none of the decoder's arithmetic and is the one module that the
tests hand to both the CUDA path and the CPU oracle.  Nothing here touches a GPU.

An instance map is drawn (ellipses or clipped Voronoi cells), the centroid of every instance is
the mean of its pixels' normalised coordinates (pixel centres, x = -1 + (2 col + 1)/W), each
foreground pixel carries the encoding (sin(2^l pi p), cos(2^l pi p)), l < F, of its instance's
centroid for p = x then p = y (Eq. 1-2), background pixels carry zeros, and i.i.d. Gaussian noise is
added to every channel of every pixel before the cast to the storage type.
"""
from __future__ import annotations

import dataclasses
import math

import numpy as np

SEED_BASE = 20260916


@dataclasses.dataclass(frozen=True)
class Config:
    name: str
    B: int
    H: int
    W: int
    F: int
    dtype: str          # "f32" | "f16"
    K: int              # instances per image
    fg: float           # target foreground fraction
    sigma: float        # noise std
    bins_w: int
    bins_h: int
    T_v: int = 8
    K_max: int = 1024
    tau: float = math.inf
    kind: str = "ellipses"
    index: int = 0

    @property
    def D(self) -> int:
        return 4 * self.F

    @property
    def np_dtype(self):
        return np.float32 if self.dtype == "f32" else np.float16

    @property
    def esz(self) -> int:
        return 4 if self.dtype == "f32" else 2

    @property
    def pixels(self) -> int:
        return self.B * self.H * self.W

    @property
    def emb_bytes(self) -> int:
        return self.pixels * self.D * self.esz

    def describe(self) -> str:
        return (f"{self.name}: {self.B}x{self.H}x{self.W} F={self.F} (D={self.D}) {self.dtype}, K={self.K}, "
                f"fg~{self.fg:.2f}, sigma={self.sigma}, bins {self.bins_w}x{self.bins_h}")


CONFIGS = {
    "c1": Config("c1", 1, 128, 128, 4, "f32", 5, 0.70, 0.05, 32, 32, kind="ellipses5", index=1),
    "c2": Config("c2", 1, 512, 512, 8, "f32", 20, 0.60, 0.05, 64, 64, kind="voronoi_blobs", index=2),
    "c3": Config("c3", 1, 1024, 2048, 8, "f16", 60, 0.50, 0.10, 256, 128, kind="loguniform", index=3),
    "c4": Config("c4", 8, 640, 640, 8, "f16", 100, 0.40, 0.10, 80, 80, kind="small_objects", index=4),
    "c5": Config("c5", 1, 2048, 2048, 16, "f16", 300, 0.80, 0.20, 512, 512, kind="dense_voronoi", index=5),
}


def rng_for(cfg: Config, frame: int, image: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64([SEED_BASE, cfg.index, frame, image]))


# ----------------------------------------------------------------------------- shapes

def _ellipse_field(H, W, cx, cy, a, b, theta, cap):
    """Normalised radius of every pixel w.r.t. each ellipse, min over ellipses, inside boxes of `cap` radii."""
    field = np.full((H, W), np.inf, np.float32)
    boxes = []
    for i in range(len(cx)):
        r = cap * max(a[i], b[i])
        x0, x1 = max(0, int(cx[i] - r)), min(W, int(cx[i] + r) + 2)
        y0, y1 = max(0, int(cy[i] - r)), min(H, int(cy[i] + r) + 2)
        boxes.append((x0, x1, y0, y1))
        if x0 >= x1 or y0 >= y1:
            continue
        yy, xx = np.mgrid[y0:y1, x0:x1].astype(np.float32)
        dx, dy = xx - cx[i], yy - cy[i]
        ct, st = math.cos(theta[i]), math.sin(theta[i])
        u = (dx * ct + dy * st) / a[i]
        v = (-dx * st + dy * ct) / b[i]
        f = np.sqrt(u * u + v * v)
        np.minimum(field[y0:y1, x0:x1], f, out=field[y0:y1, x0:x1])
    return field, boxes


def _paint_ellipses(H, W, cx, cy, a, b, theta, scale):
    inst = np.zeros((H, W), np.int32)
    for i in range(len(cx)):
        r = scale * max(a[i], b[i])
        x0, x1 = max(0, int(cx[i] - r)), min(W, int(cx[i] + r) + 2)
        y0, y1 = max(0, int(cy[i] - r)), min(H, int(cy[i] + r) + 2)
        if x0 >= x1 or y0 >= y1:
            continue
        yy, xx = np.mgrid[y0:y1, x0:x1].astype(np.float32)
        dx, dy = xx - cx[i], yy - cy[i]
        ct, st = math.cos(theta[i]), math.sin(theta[i])
        u = (dx * ct + dy * st) / a[i]
        v = (-dx * st + dy * ct) / b[i]
        inside = (u * u + v * v) <= scale * scale
        sub = inst[y0:y1, x0:x1]
        sub[inside] = i + 1
    return inst


def _ellipse_instances(H, W, areas, aspect_max, fg, rng, min_visible=40):
    """Painter's-order ellipses with a common size factor chosen so that coverage hits `fg`."""
    K = len(areas)
    cap = 2.5
    cx = rng.uniform(0.05 * W, 0.95 * W, K)
    cy = rng.uniform(0.05 * H, 0.95 * H, K)
    aspect = rng.uniform(1.0, aspect_max, K)
    theta = rng.uniform(0.0, math.pi, K)
    a = np.sqrt(areas * aspect / math.pi)
    b = np.sqrt(areas / (aspect * math.pi))
    inst = None
    for _ in range(30):
        field, _ = _ellipse_field(H, W, cx, cy, a, b, theta, cap)
        scale = float(np.quantile(field, fg))
        scale = min(scale, cap)
        inst = _paint_ellipses(H, W, cx, cy, a, b, theta, scale)
        vis = np.bincount(inst.ravel(), minlength=K + 1)[1:]
        hidden = np.nonzero(vis < min_visible)[0]
        if hidden.size == 0:
            break
        cx[hidden] = rng.uniform(0.05 * W, 0.95 * W, hidden.size)
        cy[hidden] = rng.uniform(0.05 * H, 0.95 * H, hidden.size)
    return inst


def _blob_mask(H, W, n_discs, fg, rng):
    """Union of random discs, radii scaled so that exactly a fraction `fg` of the pixels is covered."""
    cx = rng.uniform(0.1 * W, 0.9 * W, n_discs)
    cy = rng.uniform(0.1 * H, 0.9 * H, n_discs)
    rad = rng.uniform(0.6, 1.4, n_discs)
    yy, xx = np.mgrid[0:H, 0:W].astype(np.float32)
    field = np.full((H, W), np.inf, np.float32)
    for i in range(n_discs):
        f = np.sqrt((xx - cx[i]) ** 2 + (yy - cy[i]) ** 2) / rad[i]
        np.minimum(field, f, out=field)
    return field <= np.quantile(field, fg)


def _voronoi(H, W, sites_xy):
    from scipy.spatial import cKDTree
    yy, xx = np.mgrid[0:H, 0:W]
    pts = np.stack([xx.ravel(), yy.ravel()], 1).astype(np.float32)
    _, idx = cKDTree(sites_xy).query(pts, k=1, workers=-1)
    return (idx.reshape(H, W) + 1).astype(np.int32)


def _voronoi_instances(H, W, K, fg, n_discs, rng, min_visible=40):
    mask = _blob_mask(H, W, n_discs, fg, rng)
    ys, xs = np.nonzero(mask)
    inst = None
    for _ in range(30):
        pick = rng.choice(ys.size, K, replace=False)
        sites = np.stack([xs[pick], ys[pick]], 1).astype(np.float32)
        inst = _voronoi(H, W, sites) * mask
        vis = np.bincount(inst.ravel(), minlength=K + 1)[1:]
        if (vis >= min_visible).all():
            break
    return inst.astype(np.int32)


def _dense_voronoi_with_pairs(H, W, K, fg, rng):
    """Voronoi cells clipped to a blob mask; one instance in ten is half of a pair of adjacent 8-px-wide strips."""
    n_pairs = max(1, K // 20)
    n_vor = K - 2 * n_pairs
    inst = _voronoi_instances(H, W, n_vor, fg, 24, rng)
    label = n_vor
    for _ in range(n_pairs):
        for _try in range(100):
            h = int(rng.integers(24, 64))
            x0 = int(rng.integers(8, W - 24))
            y0 = int(rng.integers(8, H - h - 8))
            if (inst[y0:y0 + h, x0:x0 + 16] > n_vor).any():
                continue
            # taking the patch must not delete a Voronoi instance
            trial = inst.copy()
            trial[y0:y0 + h, x0:x0 + 8] = label + 1
            trial[y0:y0 + h, x0 + 8:x0 + 16] = label + 2
            if (np.bincount(trial.ravel(), minlength=label + 3)[1:] >= 40).all():
                inst = trial
                label += 2
                break
        else:
            raise RuntimeError("could not place a strip pair")
    return inst


def instance_map(cfg: Config, rng: np.random.Generator) -> np.ndarray:
    """One image's instance map, int32 [H, W], 0 = background, 1..K = instances."""
    H, W, K = cfg.H, cfg.W, cfg.K
    if cfg.kind == "ellipses5":
        areas = rng.uniform(0.10, 0.30, K) * H * W
        return _ellipse_instances(H, W, areas, 2.0, cfg.fg, rng)
    if cfg.kind == "voronoi_blobs":
        return _voronoi_instances(H, W, K, cfg.fg, 12, rng)
    if cfg.kind == "loguniform":
        hi = 0.05 * H * W
        lo = min(200.0, 0.1 * hi)            # 200 px at the full size; scaled-down test images keep the ratio sane
        areas = np.exp(rng.uniform(math.log(lo), math.log(hi), K))
        return _ellipse_instances(H, W, areas, 3.0, cfg.fg, rng)
    if cfg.kind == "small_objects":
        areas = np.clip(900.0 * np.exp(1.15 * rng.standard_normal(K)), 60.0, 0.2 * H * W)
        return _ellipse_instances(H, W, areas, 2.5, cfg.fg, rng)
    if cfg.kind == "dense_voronoi":
        return _dense_voronoi_with_pairs(H, W, K, cfg.fg, rng)
    raise ValueError(cfg.kind)


# ----------------------------------------------------------------------------- encoding

def pixel_centre_coords(H: int, W: int):
    """Normalised coordinates of pixel centres: x[col] = -1 + (2 col + 1)/W, y[row] likewise."""
    x = -1.0 + (2.0 * np.arange(W) + 1.0) / W
    y = -1.0 + (2.0 * np.arange(H) + 1.0) / H
    return x, y


def instance_centroids(inst: np.ndarray) -> np.ndarray:
    """Mean normalised (x, y) of every instance's pixels, float64 [K, 2] (NaN for an empty instance)."""
    H, W = inst.shape
    K = int(inst.max())
    x, y = pixel_centre_coords(H, W)
    flat = inst.ravel()
    cnt = np.bincount(flat, minlength=K + 1).astype(np.float64)
    sx = np.bincount(flat, weights=np.broadcast_to(x[None, :], (H, W)).ravel(), minlength=K + 1)
    sy = np.bincount(flat, weights=np.broadcast_to(y[:, None], (H, W)).ravel(), minlength=K + 1)
    with np.errstate(invalid="ignore", divide="ignore"):
        return np.stack([sx[1:] / cnt[1:], sy[1:] / cnt[1:]], 1)


def encode(inst: np.ndarray, centroids: np.ndarray, F: int, sigma: float, rng, dtype) -> np.ndarray:
    """Planar [4F, H, W] embedding of one image: gamma(centroid of the pixel's instance) + N(0, sigma^2).

    Channel c = axis*2F + 2l + t (axis 0 = x, 1 = y; t = 0 sin, 1 cos).  Background pixels encode zeros.
    """
    H, W = inst.shape
    K = centroids.shape[0]
    table = np.zeros((4 * F, K + 1), np.float64)
    for axis in range(2):
        for l in range(F):
            arg = math.pi * (2.0 ** l) * centroids[:, axis]
            table[axis * 2 * F + 2 * l + 0, 1:] = np.sin(arg)
            table[axis * 2 * F + 2 * l + 1, 1:] = np.cos(arg)
    table = np.nan_to_num(table).astype(np.float32)
    out = np.empty((4 * F, H, W), dtype)
    for c in range(4 * F):
        plane = table[c][inst]
        if sigma > 0:
            plane = plane + np.float32(sigma) * rng.standard_normal((H, W), dtype=np.float32)
        out[c] = plane.astype(dtype)
    return out


def make_frame(cfg: Config, frame: int = 0):
    """One batch of `cfg`: emb [B, 4F, H, W], fg [B, H, W] uint8, inst [B, H, W] int32, centroids (list of [K, 2])."""
    emb = np.empty((cfg.B, cfg.D, cfg.H, cfg.W), cfg.np_dtype)
    fg = np.empty((cfg.B, cfg.H, cfg.W), np.uint8)
    insts = np.empty((cfg.B, cfg.H, cfg.W), np.int32)
    cents = []
    for b in range(cfg.B):
        rng = rng_for(cfg, frame, b)
        inst = instance_map(cfg, rng)
        c = instance_centroids(inst)
        emb[b] = encode(inst, c, cfg.F, cfg.sigma, rng, cfg.np_dtype)
        fg[b] = (inst > 0).astype(np.uint8)
        insts[b] = inst
        cents.append(c)
    return {"emb": emb, "fg": fg, "inst": insts, "centroids": cents, "cfg": cfg, "frame": frame}


def describe_frame(fr) -> dict:
    """Self-check figures of a generated batch: instance count, foreground fraction, closest centroid pair (px)."""
    cfg = fr["cfg"]
    out = []
    for b in range(cfg.B):
        inst, c = fr["inst"][b], fr["centroids"][b]
        px = np.stack([(c[:, 0] + 1) * cfg.W / 2, (c[:, 1] + 1) * cfg.H / 2], 1)
        if len(px) > 1:
            from scipy.spatial import cKDTree
            d, _ = cKDTree(px).query(px, k=2)
            dmin = float(d[:, 1].min())
        else:
            dmin = float("inf")
        areas = np.bincount(inst.ravel(), minlength=len(c) + 1)[1:]
        out.append({"instances": int((areas > 0).sum()), "fg": float((inst > 0).mean()),
                    "min_centroid_dist_px": dmin, "median_area": float(np.median(areas)),
                    "min_area": int(areas.min())})
    return {"images": out}


def scaled(cfg: Config, **kw) -> Config:
    """A copy of a configuration with some fields replaced (tests use smaller images of the same recipe)."""
    return dataclasses.replace(cfg, **kw)
