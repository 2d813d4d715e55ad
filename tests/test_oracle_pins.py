"""Pins of the CPU oracle against what the paper and the mathematics fix.

Nothing here runs the CUDA path.  Each test names the passage or the property that fixes the
expected value; the expected values come from closed forms, library routines on special cases,
brute force on tiny inputs, or invariants - never from the oracle itself.
"""
import math
import os

import numpy as np
import pytest

import oracle
from paper_2609_16874_b200 import workloads as wl


def gamma(p, F):
    """Eq. 2 in double: [..., 2F] with (sin, cos) per harmonic."""
    p = np.asarray(p, np.float64)
    out = np.empty(p.shape + (2 * F,), np.float64)
    for l in range(F):
        out[..., 2 * l] = np.sin(2.0 ** l * np.pi * p)
        out[..., 2 * l + 1] = np.cos(2.0 ** l * np.pi * p)
    return out


def circ_diff(a, b):
    """Difference on the circle of circumference 2 (the encoding identifies -1 and +1)."""
    return (np.asarray(a, np.float64) - np.asarray(b, np.float64) + 1.0) % 2.0 - 1.0


# ---------------------------------------------------------------- Eq. 2 / Eq. 9 palettes

def test_palette_golden_closed_form(golden_dir):
    rows = 0
    for line in open(os.path.join(golden_dir, "palette_closed_form.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        tok = line.split()
        n, F, i = int(tok[0]), int(tok[1]), int(tok[2])
        want = np.array([float(t) for t in tok[3:]], np.float64)
        assert want.size == 2 * F
        got = oracle.palette(n, F)[i - 1].astype(np.float64)
        np.testing.assert_allclose(got, want, rtol=0, atol=2e-7 * 2 ** F)
        rows += 1
    assert rows == 9


@pytest.mark.parametrize("n,F", [(32, 4), (64, 8), (80, 8), (257, 16), (3, 1)])
def test_palette_properties(n, F):
    P = oracle.palette(n, F).astype(np.float64)
    assert P.shape == (n, 2 * F)          # D = 4F channels over two axes; 16 for the paper's L = 4
    pos = np.array([oracle.bin_position(n, i) for i in range(1, n + 1)])
    np.testing.assert_allclose(pos, -pos[::-1], atol=1e-15)           # symmetric about 0
    np.testing.assert_allclose(np.diff(pos), 2.0 / (n + 1), atol=1e-15)  # evenly spaced, step 2/(n+1)
    assert pos[0] == pytest.approx(-1 + 2 / (n + 1)) and pos[-1] == pytest.approx(1 - 2 / (n + 1))
    s, c = P[:, 0::2], P[:, 1::2]
    np.testing.assert_allclose(s * s + c * c, 1.0, atol=3e-7)
    np.testing.assert_allclose(s, -s[::-1], atol=1e-6 * 2 ** F)       # sin odd, cos even in the position
    np.testing.assert_allclose(c, c[::-1], atol=1e-6 * 2 ** F)
    np.testing.assert_allclose(P, gamma(pos, F), atol=1e-7 + 4e-16 * 2 ** F * np.pi)


def test_gamma_is_circular():
    # gamma(-1) = gamma(+1): the reason the estimate is wrapped into [-1, 1)
    np.testing.assert_allclose(gamma(-1.0, 6), gamma(1.0, 6), atol=1e-12)


# ---------------------------------------------------------------- binary16 widening

def test_half_widening_all_bit_patterns():
    bits = np.arange(65536, dtype=np.uint16)
    got = oracle.half_to_float(bits)
    want = bits.view(np.float16).astype(np.float32)     # numpy's conversion is exact
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan].view(np.uint32), want[~nan].view(np.uint32))


# ---------------------------------------------------------------- atan2 in half-turns

def test_atan2_ht_accuracy_dense():
    rng = np.random.default_rng(1)
    ang = np.linspace(-np.pi, np.pi, 400001)
    rad = rng.uniform(0.05, 3.0, ang.size)
    y, x = (rad * np.sin(ang)).astype(np.float32), (rad * np.cos(ang)).astype(np.float32)
    got = oracle.atan2_ht(y, x).astype(np.float64)
    want = np.arctan2(y.astype(np.float64), x.astype(np.float64)) / np.pi
    assert np.abs(got - want).max() <= 1e-6
    assert got.min() >= -1.0 and got.max() <= 1.0


def test_atan2_ht_axes_and_symmetries():
    f = lambda y, x: float(oracle.atan2_ht(np.float32([y]), np.float32([x]))[0])
    assert f(0, 1) == 0.0 and f(1, 0) == 0.5 and f(0, -1) == 1.0 and f(-1, 0) == -0.5
    assert f(0, 0) == 0.0
    assert abs(f(1, 1) - 0.25) <= 1e-6 and abs(f(1, -1) - 0.75) <= 1e-6
    assert abs(f(2.5, 2.5) - 0.25) <= 1e-6               # scale invariant
    rng = np.random.default_rng(2)
    y = np.abs(rng.standard_normal(20000)).astype(np.float32) + np.float32(1e-3)
    x = np.abs(rng.standard_normal(20000)).astype(np.float32) + np.float32(1e-3)
    a = oracle.atan2_ht(y, x)
    assert np.array_equal(oracle.atan2_ht(-y, x), -a)                     # odd in y
    assert np.array_equal(oracle.atan2_ht(y, -x), np.float32(1.0) - a)    # reflection about the y axis
    b = oracle.atan2_ht(x, y)                                             # swapping = reflection about 45 degrees
    np.testing.assert_allclose(a.astype(np.float64) + b.astype(np.float64), 0.5, atol=1.5e-6)


# ---------------------------------------------------------------- the per-pixel estimate

@pytest.mark.parametrize("F", [1, 2, 4, 8, 16])
def test_estimate_round_trip_noise_free(F):
    # decode(gamma(p)) = p: the estimate inverts Eq. 2.  Error budget: polynomial (6e-7 half-turns) and input
    # rounding, divided by 2^(F-1) because the top harmonic decides, plus the binary32 spacing of p itself.
    p = np.concatenate([np.linspace(-1.0, 1.0, 200001)[:-1], [-1.0, -1 + 1e-7, 1 - 1e-7, 0.0, 0.5, -0.5]])
    sc = gamma(p, F).astype(np.float32)
    got = oracle.decode_axis(sc)
    tol = 2e-6 / 2 ** (F - 1) + 2.4e-7
    assert np.abs(circ_diff(got, p)).max() <= tol
    assert got.min() >= -1.0 and got.max() < 1.0


@pytest.mark.parametrize("F,levels", [(8, 1), (8, 3), (8, 8), (4, 2)])
def test_estimate_levels_uses_only_leading_harmonics(F, levels):
    rng = np.random.default_rng(3)
    p = rng.uniform(-1, 1, 5000)
    sc = gamma(p, F).astype(np.float32)
    garbage = sc.copy()
    garbage[:, 2 * levels:] = rng.standard_normal((p.size, 2 * (F - levels))).astype(np.float32)
    a = oracle.decode_axis(sc, levels)
    b = oracle.decode_axis(garbage, levels)
    assert np.array_equal(a, b)                          # harmonics >= levels are never looked at
    assert np.abs(circ_diff(a, p)).max() <= 2e-6 / 2 ** (levels - 1) + 2.4e-7
    assert np.array_equal(oracle.decode_axis(sc, 0), oracle.decode_axis(sc, F))   # 0 means all


def _ml_estimate(sc, F, coarse=1 << 13, fine=401):
    """Brute-force minimiser of the paper's d_x(p) = ||xhat - gamma(p)|| (Eq. 4) over continuous p."""
    grid = -1.0 + 2.0 * np.arange(coarse) / coarse
    G = gamma(grid, F)                                    # [coarse, 2F]
    out = np.empty(sc.shape[0])
    step = 2.0 / coarse
    for i in range(sc.shape[0]):
        d = ((G - sc[i][None, :]) ** 2).sum(1)
        p0 = grid[int(np.argmin(d))]
        loc = p0 + np.linspace(-step, step, fine)
        d2 = ((gamma(loc, F) - sc[i][None, :]) ** 2).sum(1)
        out[i] = loc[int(np.argmin(d2))]
    return out


@pytest.mark.parametrize("F,sigma", [(4, 0.05), (8, 0.1)])
def test_estimate_tracks_maximum_likelihood(F, sigma):
    # For Gaussian noise the ML centroid is argmin_p ||xhat - gamma(p)||; coarse-to-fine unwrapping must land
    # in the same basin and be almost as accurate (it trusts only the top harmonic for the last digits, which
    # carries 3/4 of the Fisher information: rms ratio 1/sqrt(0.75) = 1.155).
    rng = np.random.default_rng(4)
    n = 600
    p = rng.uniform(-1, 1, n)
    sc = (gamma(p, F) + sigma * rng.standard_normal((n, 2 * F))).astype(np.float32)
    got = oracle.decode_axis(sc).astype(np.float64)
    ml = _ml_estimate(sc.astype(np.float64), F)
    basin = 0.5 * 2.0 ** -(F - 1)                         # half a period of the top harmonic, halved
    same = np.abs(circ_diff(got, ml)) < basin
    assert same.mean() >= 0.995
    err_got = np.sqrt((circ_diff(got, p)[same] ** 2).mean())
    err_ml = np.sqrt((circ_diff(ml, p)[same] ** 2).mean())
    assert 0.9 <= err_got / err_ml <= 1.35
    assert err_got <= 1.5 * sigma / (np.pi * 2 ** (F - 1))


@pytest.mark.parametrize("F,sigma,n_bins", [(4, 0.05, 32), (8, 0.1, 256), (16, 0.2, 512)])
def test_estimate_cell_matches_double_precision_libm(F, sigma, n_bins):
    # The same unwrapping evaluated in binary64 with libm's atan2 must give the same bin, except where the
    # estimate sits within 1e-5 of a bin edge.  Catches a wrong coefficient, sign, quadrant or level scale.
    rng = np.random.default_rng(5)
    n = 200000
    p = rng.uniform(-1, 1, n)
    sc = (gamma(p, F) + sigma * rng.standard_normal((n, 2 * F))).astype(np.float32)
    got = oracle.decode_axis(sc)
    s64 = sc.astype(np.float64)
    u = np.arctan2(s64[:, 0::2], s64[:, 1::2]) / np.pi
    q = u[:, 0].copy()
    for l in range(1, F):
        m = np.rint((q * 2.0 ** l - u[:, l]) * 0.5)
        q = (u[:, l] + 2.0 * m) / 2.0 ** l
    q = np.where(q < -1, q + 2, q)
    q = np.where(q >= 1, q - 2, q)
    g = (q + 1.0) * (n_bins + 1) * 0.5
    near_edge = np.abs(g - np.floor(g) - 0.5) < 1e-5 * (n_bins + 1)
    # a branch decision (m) may legitimately flip when t - u sits on a rounding tie; those are gross
    # differences of a whole period and must be vanishingly rare
    gross = np.abs(circ_diff(got, q)) > 1e-4
    assert gross.mean() < 5e-5
    cell64 = np.clip(np.rint(g), 1, n_bins).astype(int) - 1
    cell32 = np.array([oracle.cell_of(v, n_bins) for v in got[:20000]])
    ok = (cell32 == cell64[:20000]) | near_edge[:20000] | gross[:20000]
    assert ok.all()


def test_cell_of_is_nearest_eq9_bin():
    # nearest bin position of Eq. 9 by exhaustive search; the end bins also take what lies beyond them
    for n in (3, 32, 80, 257):
        pos = np.array([oracle.bin_position(n, i) for i in range(1, n + 1)])
        rng = np.random.default_rng(n)
        p = rng.uniform(-1, 1, 4000).astype(np.float32)
        got = np.array([oracle.cell_of(v, n) for v in p])
        dist = np.abs(p.astype(np.float64)[:, None] - pos[None, :])
        want = dist.argmin(1)
        tie = np.abs(np.sort(dist, 1)[:, 0] - np.sort(dist, 1)[:, 1]) < 1e-6
        assert ((got == want) | tie).all()
        assert oracle.cell_of(-1.0, n) == 0 and oracle.cell_of(np.nextafter(np.float32(1), np.float32(0)), n) == n - 1
        for i in (1, n // 2 + 1, n):
            assert oracle.cell_of(pos[i - 1], n) == i - 1


# ---------------------------------------------------------------- votes

def _toy_instances(H, W, boxes):
    inst = np.zeros((H, W), np.int32)
    for k, (y0, y1, x0, x1) in enumerate(boxes):
        inst[y0:y1, x0:x1] = k + 1
    return inst


def test_votes_noise_free_concentrate_on_centroid_bins():
    # V = sum_k area_k * delta(cell_k) for exact encodings (hard-vote reading of Eq. 6 with Eq. 9 bins)
    H, W, F, bw, bh = 48, 64, 4, 32, 24
    inst = _toy_instances(H, W, [(2, 20, 3, 30), (25, 45, 10, 25), (5, 40, 40, 60)])
    cents = np.array([[-0.613, -0.377], [0.05, 0.52], [0.731, -0.11]])
    emb = wl.encode(inst, cents, F, 0.0, None, np.float32)[None]
    fg = (inst > 0).astype(np.uint8)[None]
    res = oracle.votes(emb, fg, bw, bh)
    want = np.zeros((bh, bw), np.uint32)
    for k, (cx, cy) in enumerate(cents):
        ix = int(np.clip(np.rint((cx + 1) * (bw + 1) / 2), 1, bw)) - 1
        iy = int(np.clip(np.rint((cy + 1) * (bh + 1) / 2), 1, bh)) - 1
        want[iy, ix] += (inst == k + 1).sum()
    assert np.array_equal(res["votes"][0], want)
    assert res["counters"][0, oracle.CNT_VOTING] == fg.sum()


def test_votes_sum_mask_and_nonfinite_rules():
    cfg = wl.scaled(wl.CONFIGS["c1"], H=40, W=56)
    fr = wl.make_frame(cfg, 3)
    emb, fg = fr["emb"].copy(), fr["fg"]
    ys, xs = np.nonzero(fg[0])
    emb[0, 5, ys[0], xs[0]] = np.nan
    emb[0, 0, ys[1], xs[1]] = np.inf
    emb[0, 15, ys[2], xs[2]] = -np.inf
    bys, bxs = np.nonzero(fg[0] == 0)
    emb[0, 3, bys[0], bxs[0]] = np.nan                     # background: never looked at
    res = oracle.votes(emb, fg, cfg.bins_w, cfg.bins_h, want_cell=True)
    assert res["votes"].sum() == fg.sum() - 3
    assert res["counters"][0, oracle.CNT_NONFINITE] == 3
    assert (res["cell"][0][fg[0] == 0] == -1).all()
    assert res["cell"][0, ys[0], xs[0]] == -1 and res["cell"][0, ys[3], xs[3]] >= 0
    # every vote sits where the pixel's cell says
    want = np.bincount(res["cell"][0][res["cell"][0] >= 0], minlength=cfg.bins_w * cfg.bins_h)
    assert np.array_equal(want.reshape(cfg.bins_h, cfg.bins_w), res["votes"][0])
    # no mask: every pixel participates (the paper's S is the whole output grid)
    res_all = oracle.votes(fr["emb"], None, cfg.bins_w, cfg.bins_h)
    assert res_all["votes"].sum() == cfg.H * cfg.W


def test_a_finite_pair_whose_magnitudes_overflow_when_added_counts_as_non_finite():
    """The usability rule of a (sin, cos) pair is "fl32(|s| + |c|) is finite": two finite binary32 values whose sum of
    magnitudes overflows make the pixel unusable -- no vote, label 0, counted -- while either value alone (sum still
    finite) is fine.  Pinned here against the rule's own statement: numpy's binary32 addition decides which is which."""
    cfg = wl.scaled(wl.CONFIGS["c1"], H=40, W=56)
    fr = wl.make_frame(cfg, 3)
    emb, fg = fr["emb"].copy(), fr["fg"]
    ys, xs = np.nonzero(fg[0])
    big = np.float32(2.5e38)
    with np.errstate(over="ignore"):
        assert np.isfinite(big) and np.isinf(np.float32(big) + np.float32(big)) and np.isfinite(big + np.float32(1.0))
    emb[0, 4, ys[0], xs[0]], emb[0, 5, ys[0], xs[0]] = big, -big      # harmonic 2 of x: |s| + |c| overflows
    emb[0, 4, ys[1], xs[1]] = big                                     # the same magnitude alone: still usable
    emb[0, 9, ys[2], xs[2]], emb[0, 10, ys[2], xs[2]] = big, big      # cos of one harmonic, sin of the next: different pairs
    res = oracle.votes(emb, fg, cfg.bins_w, cfg.bins_h, want_cell=True)
    assert res["counters"][0, oracle.CNT_NONFINITE] == 1
    assert res["votes"].sum() == fg.sum() - 1
    assert res["cell"][0, ys[0], xs[0]] == -1
    assert res["cell"][0, ys[1], xs[1]] >= 0 and res["cell"][0, ys[2], xs[2]] >= 0
    dec = oracle.decode(emb, fg, cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, cfg.K_max)
    assert dec["labels"][0, ys[0], xs[0]] == 0 and np.isinf(dec["best"][0, ys[0], xs[0]])
    assert dec["labels"][0, ys[1], xs[1]] > 0 and dec["labels"][0, ys[2], xs[2]] > 0


def test_votes_fp16_equals_fp32_of_widened_values():
    cfg = wl.scaled(wl.CONFIGS["c3"], H=32, W=48, K=4, bins_w=32, bins_h=16)
    fr = wl.make_frame(cfg, 0)
    a = oracle.votes(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h, want_est=True)
    b = oracle.votes(fr["emb"].astype(np.float32), fr["fg"], cfg.bins_w, cfg.bins_h, want_est=True)
    assert np.array_equal(a["votes"], b["votes"])
    assert np.array_equal(a["est"], b["est"], equal_nan=True)


# ---------------------------------------------------------------- peaks

def test_peaks_hand_cases():
    V = np.zeros((5, 6), np.uint32)
    V[1, 1] = 20                                          # isolated
    V[3, 3] = 15
    V[3, 4] = 15                                          # horizontal two-cell plateau: lower index wins
    V[0, 5] = 9                                           # corner, just above the threshold
    V[4, 0] = 8                                           # corner, not above (needs V > T_v)
    cells, pv, raw = oracle.peaks(V, 8, 16)
    assert cells.tolist() == [0 * 6 + 5, 1 * 6 + 1, 3 * 6 + 3] and pv.tolist() == [9, 20, 15] and raw == 3
    # diagonal plateau and an 8-neighbour that is larger
    V = np.zeros((4, 4), np.uint32)
    V[0, 0] = V[1, 1] = 12
    V[2, 3] = 30
    V[3, 2] = 29                                          # diagonal neighbour of the 30: suppressed
    cells, _, _ = oracle.peaks(V, 0, 16)
    assert cells.tolist() == [0, 2 * 4 + 3]
    # the literal strict test would delete a plateau entirely; a flat map keeps exactly cell 0
    cells, _, _ = oracle.peaks(np.full((3, 3), 10, np.uint32), 8, 16)
    assert cells.tolist() == [0]
    # truncation keeps the first K_max in ascending linear index and reports how many there were
    V = np.zeros((9, 9), np.uint32)
    V[::2, ::2] = 50
    cells, _, raw = oracle.peaks(V, 8, 7)
    assert raw == 25 and cells.tolist() == [0, 2, 4, 6, 8, 18, 20]


def test_peaks_distinct_values_equal_library_maximum_filter():
    # with pairwise distinct counts the rule is the paper's strict 8-neighbour maximum: a library max filter
    from scipy.ndimage import maximum_filter
    rng = np.random.default_rng(7)
    for shape in [(7, 9), (16, 16), (1, 12), (13, 1), (2, 2)]:
        V = rng.permutation(shape[0] * shape[1]).reshape(shape).astype(np.uint32)
        T = int(V.size // 3)
        want = np.nonzero(((V == maximum_filter(V, size=3, mode="constant", cval=0)) & (V > T)).ravel())[0]
        cells, pv, raw = oracle.peaks(V, T, V.size)
        assert cells.tolist() == want.tolist() and raw == want.size
        assert np.array_equal(pv, V.ravel()[want])


def test_peaks_properties_with_ties_random():
    rng = np.random.default_rng(8)
    for _ in range(50):
        bh, bw = rng.integers(1, 9, 2)
        V = rng.integers(0, 4, (bh, bw)).astype(np.uint32) * 5
        cells, pv, raw = oracle.peaks(V, 4, 64)
        assert (np.diff(cells) > 0).all() and (pv > 4).all() and raw == len(cells)
        ys, xs = cells // bw, cells % bw
        for i in range(len(cells)):                       # no two peaks are 8-adjacent
            for j in range(i + 1, len(cells)):
                assert max(abs(ys[i] - ys[j]), abs(xs[i] - xs[j])) > 1
        # every cell above the threshold is a peak or has a neighbour that beats it (brute force, all cells)
        for y in range(bh):
            for x in range(bw):
                if V[y, x] <= 4:
                    continue
                lin = y * bw + x
                beaten = False
                for ny in range(max(0, y - 1), min(bh, y + 2)):
                    for nx in range(max(0, x - 1), min(bw, x + 2)):
                        nl = ny * bw + nx
                        if nl != lin and (V[ny, nx] > V[y, x] or (V[ny, nx] == V[y, x] and nl < lin)):
                            beaten = True
                assert beaten != (lin in cells)


# ---------------------------------------------------------------- assignment

def _tiny_problem(seed, F=3, H=6, W=7, bw=9, bh=8, K=4, dtype=np.float32):
    rng = np.random.default_rng(seed)
    emb = rng.standard_normal((4 * F, H, W)).astype(dtype)
    fg = (rng.uniform(size=(H, W)) < 0.8).astype(np.uint8)
    cells = np.sort(rng.choice(bw * bh, K, replace=False)).astype(np.int32)
    return emb, fg, cells, bw, bh, F


def _brute_scores(emb, cells, bw, bh, F):
    """d[k, pixel] of Eq. 4 from gamma of the Eq. 9 positions, independent of the oracle's palette code."""
    D, H, W = emb.shape
    e = emb.reshape(D, -1).astype(np.float64)
    d = np.empty((len(cells), H * W))
    for k, lin in enumerate(cells):
        cx, cy = lin % bw, lin // bw
        gx = gamma(-1 + 2 * (cx + 1) / (bw + 1), F).astype(np.float32).astype(np.float64)
        gy = gamma(-1 + 2 * (cy + 1) / (bh + 1), F).astype(np.float32).astype(np.float64)
        d[k] = np.sqrt(((e[:2 * F] - gx[:, None]) ** 2).sum(0)) + np.sqrt(((e[2 * F:] - gy[:, None]) ** 2).sum(0))
    return d


@pytest.mark.parametrize("seed,dtype", [(0, np.float32), (1, np.float16), (2, np.float32)])
def test_assign_brute_force_tiny(seed, dtype):
    emb, fg, cells, bw, bh, F = _tiny_problem(seed, dtype=dtype)
    res = oracle.assign_image(emb, fg, bw, bh, cells)
    d = _brute_scores(emb, cells, bw, bh, F)
    want = np.where(fg.ravel() > 0, d.argmin(0) + 1, 0)
    assert np.array_equal(res["labels"].ravel(), want)
    srt = np.sort(d, 0)
    m = fg.ravel() > 0
    np.testing.assert_allclose(res["best"].ravel()[m], srt[0][m], rtol=1e-12)
    np.testing.assert_allclose(res["second"].ravel()[m], srt[1][m], rtol=1e-12)
    # the paper's formulation of the same choice: largest E_x * E_y, E = exp(-distance) (mask aggregation)
    D, H, W = emb.shape
    e = emb.reshape(D, -1).astype(np.float64)
    aff = np.empty_like(d)
    for k, lin in enumerate(cells):
        ex = np.exp(-np.sqrt(((e[:2 * F] - oracle.palette(bw, F)[lin % bw].astype(np.float64)[:, None]) ** 2).sum(0)))
        ey = np.exp(-np.sqrt(((e[2 * F:] - oracle.palette(bh, F)[lin // bw].astype(np.float64)[:, None]) ** 2).sum(0)))
        aff[k] = ex * ey
    assert np.array_equal(np.where(m, aff.argmax(0) + 1, 0), want)


def test_assign_same_row_peaks_reduce_to_nearest_neighbour_search():
    # if all peaks share the row bin, d_y is common and Eq. 7 is a Euclidean nearest-neighbour query in x-space
    from scipy.spatial import cKDTree
    rng = np.random.default_rng(11)
    F, H, W, bw, bh = 4, 12, 10, 32, 32
    emb = rng.standard_normal((4 * F, H, W)).astype(np.float32)
    cols = np.sort(rng.choice(bw, 9, replace=False))
    cells = (5 * bw + cols).astype(np.int32)
    res = oracle.assign_image(emb, None, bw, bh, cells)
    pts = gamma(np.array([-1 + 2 * (c + 1) / (bw + 1) for c in cols]), F).astype(np.float32).astype(np.float64)
    _, nn = cKDTree(pts).query(emb[:2 * F].reshape(2 * F, -1).T.astype(np.float64), k=1)
    assert np.array_equal(res["labels"].ravel(), nn + 1)


def test_assign_tau_ties_and_degenerate_cases():
    emb, fg, cells, bw, bh, F = _tiny_problem(5)
    d = _brute_scores(emb, cells, bw, bh, F)
    best = d.min(0)
    tau = float(np.median(best[fg.ravel() > 0]))
    res = oracle.assign_image(emb, fg, bw, bh, cells, tau=tau)
    m = fg.ravel() > 0
    want = np.where(m & (best < tau), d.argmin(0) + 1, 0)        # Eq. 8: strictly below tau
    assert np.array_equal(res["labels"].ravel(), want)
    assert res["tau_rejected"] == int((m & ~(best < tau)).sum())
    exact = float(best[m][0])                                     # tau equal to a pixel's own score rejects it
    res2 = oracle.assign_image(emb, fg, bw, bh, cells, tau=exact)
    assert res2["labels"].ravel()[np.nonzero(m)[0][0]] == 0
    # a duplicated peak never wins over its first copy (lowest k on exact ties)
    dup = np.array([cells[0], cells[0]], np.int32)
    assert (oracle.assign_image(emb, None, bw, bh, dup)["labels"] == 1).all()
    # no peaks: every label is 0
    assert (oracle.assign_image(emb, fg, bw, bh, np.zeros(0, np.int32))["labels"] == 0).all()
    # one peak: every participating pixel gets it, runner-up is +inf
    one = oracle.assign_image(emb, fg, bw, bh, cells[:1])
    assert np.array_equal(one["labels"], fg.astype(np.int32)) and np.isinf(one["second"]).all()
    # non-finite pixels get 0
    e2 = emb.copy()
    e2[3, 2, 2] = np.nan
    fg2 = np.ones_like(fg)
    assert oracle.assign_image(e2, fg2, bw, bh, cells)["labels"][2, 2] == 0


def test_assign_is_per_pixel_and_sampling_agrees():
    emb, fg, cells, bw, bh, F = _tiny_problem(9, H=9, W=11)
    full = oracle.assign_image(emb, fg, bw, bh, cells)
    perm = np.random.default_rng(0).permutation(9 * 11)
    embp = emb.reshape(-1, 99)[:, perm].reshape(emb.shape)
    fgp = fg.ravel()[perm].reshape(fg.shape)
    assert np.array_equal(oracle.assign_image(embp, fgp, bw, bh, cells)["labels"].ravel(), full["labels"].ravel()[perm])
    idx = np.array([0, 5, 17, 98, 42], np.int64)
    samp = oracle.assign_image(emb, fg, bw, bh, cells, idx=idx)
    assert np.array_equal(samp["labels"], full["labels"].ravel()[idx])
    assert np.array_equal(samp["best"], full["best"].ravel()[idx])


# ---------------------------------------------------------------- the whole chain

def test_chain_noise_free_on_bin_centroids_recovers_the_instances():
    # exact encodings of centroids sitting on Eq. 9 bin positions, >= 2 cells apart: the decoder must return
    # exactly those instances (count, bins, label map up to the ascending-index numbering)
    H, W, F, bw, bh = 64, 96, 4, 32, 32
    boxes = [(0, 30, 0, 40), (0, 30, 40, 96), (30, 64, 0, 25), (30, 64, 25, 70), (34, 60, 72, 94)]
    bins = [(4, 3), (20, 5), (2, 25), (12, 20), (29, 28)]                  # (cx, cy), 0-based
    inst = _toy_instances(H, W, boxes)
    cents = np.array([[-1 + 2 * (cx + 1) / (bw + 1), -1 + 2 * (cy + 1) / (bh + 1)] for cx, cy in bins])
    for dtype in (np.float32, np.float16):
        emb = wl.encode(inst, cents, F, 0.0, None, dtype)[None]
        fg = (inst > 0).astype(np.uint8)[None]
        res = oracle.decode(emb, fg, bw, bh, T_v=8, K_max=16)
        assert res["count"][0] == 5
        lin = np.array([cy * bw + cx for cx, cy in bins])
        order = np.argsort(lin)
        assert res["peak_cell"][0, :5].tolist() == lin[order].tolist()
        assert res["peak_votes"][0, :5].tolist() == [int((inst == k + 1).sum()) for k in order]
        relabel = np.zeros(6, np.int32)
        relabel[order + 1] = np.arange(1, 6)
        assert np.array_equal(res["labels"][0], relabel[inst])
        if dtype == np.float32:
            assert res["best"][0][inst > 0].max() < 1e-6                    # distance to the own palette row ~ 0
        # centroid in pixel units: inverse of x = -1 + (2 col + 1)/W
        for j, k in enumerate(order):
            want = ((cents[k, 0] + 1) * W - 1) / 2, ((cents[k, 1] + 1) * H - 1) / 2
            np.testing.assert_allclose(res["centroids"][0, j], want, rtol=1e-6)


@pytest.mark.parametrize("name,H,W", [("c1", 128, 128), ("c2", 96, 128), ("c4", 80, 96)])
def test_chain_invariants_on_noisy_workloads(name, H, W):
    base = wl.CONFIGS[name]
    cfg = wl.scaled(base, H=H, W=W, B=min(base.B, 2), K=min(base.K, 6), bins_w=32, bins_h=32)
    fr = wl.make_frame(cfg, 1)
    res = oracle.decode(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h, T_v=cfg.T_v, K_max=cfg.K_max)
    for b in range(cfg.B):
        lab, n = res["labels"][b], int(res["count"][b])
        fg = fr["fg"][b] > 0
        assert n >= 1
        assert ((lab > 0) == fg).all() and lab.max() <= n          # labels partition the foreground (tau = inf)
        assert res["votes"][b].sum() == fg.sum()
        cells = res["peak_cell"][b, :n]
        assert (np.diff(cells) > 0).all()
        assert np.array_equal(res["peak_votes"][b, :n], res["votes"][b].ravel()[cells])
        for k in range(n):                                           # each centroid lies in its vote-peak cell
            x = (2 * res["centroids"][b, k, 0] + 1) / cfg.W - 1
            y = (2 * res["centroids"][b, k, 1] + 1) / cfg.H - 1
            assert oracle.cell_of(x, cfg.bins_w) == cells[k] % cfg.bins_w
            assert oracle.cell_of(y, cfg.bins_h) == cells[k] // cfg.bins_w
        # with this much signal every true instance is found and its pixels mostly carry one label
        assert n == cfg.K or name == "c4"
        for k in range(1, cfg.K + 1):
            m = fr["inst"][b] == k
            if m.sum() > 200:
                assert np.bincount(lab[m]).max() >= 0.9 * m.sum()


def test_hard_vote_peak_equals_soft_vote_argmax_on_alias_free_grid():
    # Eq. 5-6 evaluated directly: H(a,b) = sum_pixels exp(-(d_x + d_y)).  For one isolated instance with an exact
    # encoding on the paper's 32x32, L = 4 grid the soft histogram's arg-max bin is the hard-vote peak.
    H, W, F, bw, bh = 24, 24, 4, 32, 32
    inst = _toy_instances(H, W, [(4, 20, 6, 18)])
    cents = np.array([[0.3217, -0.4581]])
    emb = wl.encode(inst, cents, F, 0.0, None, np.float32)
    res = oracle.decode(emb[None], (inst > 0).astype(np.uint8)[None], bw, bh, T_v=8, K_max=8)
    assert res["count"][0] == 1
    Pw, Ph = oracle.palette(bw, F).astype(np.float64), oracle.palette(bh, F).astype(np.float64)
    e = emb.reshape(4 * F, -1)[:, inst.ravel() > 0].astype(np.float64)
    dx = np.sqrt(((e[None, :2 * F] - Pw[:, :, None]) ** 2).sum(1))       # [bw, P]
    dy = np.sqrt(((e[None, 2 * F:] - Ph[:, :, None]) ** 2).sum(1))       # [bh, P]
    Hsoft = np.exp(-dy) @ np.exp(-dx).T                                   # Eq. 11: the same sum, factorised
    direct = np.exp(-(dy[:, None, :] + dx[None, :, :])).sum(2)           # Eq. 6
    np.testing.assert_allclose(Hsoft, direct, rtol=1e-12)
    assert int(np.argmax(Hsoft)) == int(res["peak_cell"][0, 0])


# ---------------------------------------------------------------- soft-vote histogram (Eq. 4-6)

def _gamma(p, F):
    """Eq. 2 in binary64: (sin, cos) of pi 2^l p, l = 0..F-1, interleaved."""
    out = np.empty(2 * F)
    for l in range(F):
        out[2 * l] = np.sin(np.pi * 2.0 ** l * p)
        out[2 * l + 1] = np.cos(np.pi * 2.0 ** l * p)
    return out


def test_soft_votes_of_one_clean_pixel_follow_the_chord_length_formula():
    """One pixel that encodes (px, py) exactly: ||gamma(p) - gamma(q)||^2 = sum_l (2 - 2 cos(pi 2^l (p - q))), so every
    bin's weight has a closed form that never forms a difference of embeddings (Eq. 2, Eq. 4, Eq. 5)."""
    F, bw, bh = 5, 13, 9
    px, py = 0.3127, -0.6421
    emb = np.zeros((1, 4 * F, 1, 1), np.float64)
    emb[0, :2 * F, 0, 0] = _gamma(px, F)
    emb[0, 2 * F:, 0, 0] = _gamma(py, F)
    H = oracle.soft_votes(emb.astype(np.float32), None, bw, bh)[0]
    def chord(p, q):
        return np.sqrt(sum(2.0 - 2.0 * np.cos(np.pi * 2.0 ** l * (p - q)) for l in range(F)))
    for b in range(bh):
        for a in range(bw):
            qa, qb = -1 + 2 * (a + 1) / (bw + 1), -1 + 2 * (b + 1) / (bh + 1)
            want = np.exp(-(chord(px, qa) + chord(py, qb)))
            assert abs(H[b, a] - want) <= 2e-6 * want + 1e-12, (a, b, H[b, a], want)   # binary32 inputs and palette


def test_soft_votes_match_a_numpy_restatement_and_factorise():
    """Tiny random input: the histogram equals the sum over pixels of the outer product of the two weight vectors
    (Eq. 10-11), computed here with numpy norms and einsum from the oracle-independent Eq. 9 positions."""
    rng = np.random.default_rng(7)
    F, bw, bh, B, Hh, Ww = 3, 6, 5, 2, 4, 7
    emb = rng.standard_normal((B, 4 * F, Hh, Ww)).astype(np.float32)
    fg = (rng.random((B, Hh, Ww)) < 0.7).astype(np.uint8)
    Pw = np.stack([_gamma(-1 + 2 * (i + 1) / (bw + 1), F) for i in range(bw)]).astype(np.float32).astype(np.float64)
    Ph = np.stack([_gamma(-1 + 2 * (i + 1) / (bh + 1), F) for i in range(bh)]).astype(np.float32).astype(np.float64)
    got = oracle.soft_votes(emb, fg, bw, bh)
    for b in range(B):
        x = emb[b, :2 * F].reshape(2 * F, -1).T.astype(np.float64)
        y = emb[b, 2 * F:].reshape(2 * F, -1).T.astype(np.float64)
        keep = fg[b].ravel() != 0
        Ex = np.exp(-np.linalg.norm(x[keep, None, :] - Pw[None], axis=2))
        Ey = np.exp(-np.linalg.norm(y[keep, None, :] - Ph[None], axis=2))
        want = np.einsum("pb,pa->ba", Ey, Ex)
        assert np.allclose(got[b], want, rtol=1e-12, atol=0)
        assert np.isclose(got[b].sum(), (Ex.sum(1) * Ey.sum(1)).sum(), rtol=1e-12)   # separability of the total


def test_soft_votes_skip_masked_and_nonfinite_pixels_and_sampled_cells_agree():
    rng = np.random.default_rng(11)
    F, bw, bh = 2, 5, 4
    emb = rng.standard_normal((1, 4 * F, 3, 8)).astype(np.float32)
    fg = np.ones((1, 3, 8), np.uint8)
    full = oracle.soft_votes(emb, fg, bw, bh)
    # masking a pixel removes exactly its own contribution
    fg2 = fg.copy(); fg2[0, 1, 3] = 0
    one = np.zeros_like(emb[:, :, :1, :1]); one[...] = emb[:, :, 1:2, 3:4]
    assert np.allclose(full - oracle.soft_votes(emb, fg2, bw, bh), oracle.soft_votes(one, None, bw, bh), rtol=1e-9, atol=1e-15)
    # a pixel with a non-finite channel does not take part
    bad = emb.copy(); bad[0, 5, 1, 3] = np.inf
    assert np.allclose(oracle.soft_votes(bad, fg, bw, bh), oracle.soft_votes(emb, fg2, bw, bh), rtol=1e-12, atol=0)
    # fg = None means every pixel
    assert np.array_equal(oracle.soft_votes(emb, None, bw, bh), full)
    cells = np.array([0, 7, bw * bh - 1, 11], np.int32)
    assert np.array_equal(oracle.soft_votes(emb, fg, bw, bh, sample_cells=cells)[0], full[0].ravel()[cells])
    # binary16 inputs are widened exactly
    h = emb.astype(np.float16)
    assert np.array_equal(oracle.soft_votes(h, fg, bw, bh), oracle.soft_votes(h.astype(np.float32), fg, bw, bh))


# ---------------------------------------------------------------- per-instance outputs (Sec. 3.2, Eq. 8)

def test_instance_masks_partition_the_labelled_pixels_and_count_them():
    """Planes are disjoint, their union is the set of labelled pixels, counters equal numpy's bincount, labels beyond
    the planes asked for are left out, and the label map is recovered from the planes."""
    rng = np.random.default_rng(21)
    labels = rng.integers(0, 8, (2, 9, 13)).astype(np.int32)
    planes, pixels = oracle.instance_masks(labels, 5)
    assert planes.dtype == np.uint8 and set(np.unique(planes)) <= {0, 1}
    assert np.array_equal(planes.sum(1), ((labels >= 1) & (labels <= 5)).astype(np.uint64))
    for b in range(2):
        assert np.array_equal(pixels[b], np.bincount(labels[b].ravel(), minlength=9)[1:6])
    back = (planes * np.arange(1, 6, dtype=np.int32)[None, :, None, None]).sum(1)
    assert np.array_equal(back, np.where(labels <= 5, labels, 0))
    assert oracle.instance_masks(labels, 7, want_planes=False)[0] is None
    assert np.array_equal(oracle.instance_masks(labels, 7, want_planes=False)[1][:, :5], pixels)


# ---------------------------------------------------------------- sub-cell refined centroids

def test_vote_sums_equal_a_numpy_scatter_add_of_fixed_point_estimates():
    # definition: sums[cell] = sum of rint(p * 2^24) over the pixels that voted into the cell (integers: any order)
    cfg = wl.scaled(wl.CONFIGS["c2"], H=72, W=88, B=2, K=5, bins_w=24, bins_h=20)
    fr = wl.make_frame(cfg, 3)
    v = oracle.votes(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h, want_est=True, want_cell=True)
    got = oracle.vote_sums(v["est"], v["cell"], cfg.bins_w, cfg.bins_h)
    want = np.zeros((cfg.B, cfg.bins_w * cfg.bins_h, 2), np.int64)
    for b in range(cfg.B):
        c = v["cell"][b].ravel()
        take = c >= 0
        fixed = np.rint(v["est"][b].reshape(-1, 2)[take].astype(np.float64) * 2.0 ** 24).astype(np.int64)
        np.add.at(want[b], c[take], fixed)
    assert np.array_equal(got.reshape(want.shape), want)
    assert (got.reshape(want.shape)[v["votes"].reshape(cfg.B, -1) == 0] == 0).all()
    # |p| <= 1 bounds every cell's sum by its count
    assert (np.abs(got.reshape(want.shape)) <= v["votes"].reshape(cfg.B, -1, 1).astype(np.int64) << 24).all()


def test_refined_peaks_recover_off_bin_centroids_of_clean_encodings():
    # exact encodings of centroids placed anywhere inside a bin: every estimate equals the centroid (to binary32
    # rounding of the estimate), so the mean does too, while the unrefined candidate is off by up to half a bin.
    H, W, F, bw, bh = 64, 96, 4, 32, 32
    boxes = [(0, 30, 0, 40), (0, 30, 40, 96), (30, 64, 0, 25), (30, 64, 25, 70), (34, 60, 72, 94)]
    inst = _toy_instances(H, W, boxes)
    cents = np.array([[-0.713, -0.801], [0.2291, -0.6502], [-0.8333, 0.5477], [-0.2412, 0.2468], [0.8, 0.74]])
    emb = wl.encode(inst, cents, F, 0.0, None, np.float32)[None]
    fg = (inst > 0).astype(np.uint8)[None]
    res = oracle.decode_refined(emb, fg, bw, bh, T_v=8, K_max=16)
    assert res["count"][0] == 5
    lin = np.array([oracle.cell_of(cy, bh) * bw + oracle.cell_of(cx, bw) for cx, cy in cents])
    order = np.argsort(lin)
    assert res["peak_cell"][0, :5].tolist() == lin[order].tolist()
    for j, k in enumerate(order):
        want_px = ((cents[k, 0] + 1) * W - 1) / 2, ((cents[k, 1] + 1) * H - 1) / 2
        np.testing.assert_allclose(res["centroids"][0, j], want_px, atol=2e-4)      # 2e-6 of the unit range
        np.testing.assert_allclose(res["peak_emb"][0, j, :2 * F], gamma(cents[k, 0], F), atol=2e-6 * 2 ** F)
        np.testing.assert_allclose(res["peak_emb"][0, j, 2 * F:], gamma(cents[k, 1], F), atol=2e-6 * 2 ** F)
    relabel = np.zeros(6, np.int32)
    relabel[order + 1] = np.arange(1, 6)
    assert np.array_equal(res["labels"][0], relabel[inst])
    assert res["best"][0][inst > 0].max() < 1e-4          # every pixel sits on its refined candidate
    # the unrefined chain leaves a distance of the order of the bin offset
    plain = oracle.decode(emb, fg, bw, bh, T_v=8, K_max=16)
    assert plain["best"][0][inst > 0].max() > 0.05


def test_refined_mean_pools_the_3x3_window_and_stays_on_the_unit_torus():
    # hand-made maps: a blob straddling a cell border is pooled over the window; window clipped at the map edge
    bw, bh, F, H, W = 6, 5, 3, 40, 60
    V = np.zeros((bh, bw), np.uint32)
    S = np.zeros((bh, bw, 2), np.int64)
    one = 1 << 24
    V[2, 2], S[2, 2] = 10, (int(10 * -0.10 * one), int(10 * 0.05 * one))
    V[2, 3], S[2, 3] = 6, (int(6 * 0.02 * one), int(6 * 0.07 * one))
    V[1, 2], S[1, 2] = 4, (int(4 * -0.12 * one), int(4 * -0.20 * one))
    V[0, 5], S[0, 5] = 9, (int(9 * 0.90 * one), int(9 * -0.95 * one))      # corner cell: 4-cell window
    V[4, 0], S[4, 0] = 1, (123, -456)                                      # outside both windows
    pc = np.array([0 * bw + 5, 2 * bw + 2], np.int32)
    r = oracle.refined_peaks(V, S, pc, F, H, W)
    want1 = np.array([(10 * -0.10 + 6 * 0.02 + 4 * -0.12) / 20, (10 * 0.05 + 6 * 0.07 + 4 * -0.20) / 20])
    np.testing.assert_allclose(r["mean"][0], [0.90, -0.95], atol=1e-7)
    np.testing.assert_allclose(r["mean"][1], want1, atol=1e-7)
    for k in range(2):
        for a in range(2):
            np.testing.assert_allclose(r["peak_emb"][k, a * 2 * F:(a + 1) * 2 * F], gamma(r["mean"][k, a], F),
                                       atol=1.5e-7)
        s, c = r["peak_emb"][k, 0::2].astype(np.float64), r["peak_emb"][k, 1::2].astype(np.float64)
        np.testing.assert_allclose(s * s + c * c, 1.0, atol=3e-7)
        np.testing.assert_allclose(r["centroids"][k], [((r["mean"][k, 0] + 1) * W - 1) / 2,
                                                       ((r["mean"][k, 1] + 1) * H - 1) / 2], rtol=1e-6)


def test_explicit_candidates_reduce_to_the_palette_case_and_to_brute_force():
    # handing the palette rows in explicitly changes nothing; arbitrary rows agree with a direct Eq. 7 in numpy
    emb, fg, cells, bw, bh, F = _tiny_problem(5)
    Pw, Ph = oracle.palette(bw, F), oracle.palette(bh, F)
    rows = np.concatenate([Pw[cells % bw], Ph[cells // bw]], axis=1)
    a0 = oracle.assign_image(emb, fg, bw, bh, cells)
    a1 = oracle.assign_image(emb, fg, bw, bh, cells, peak_emb=rows)
    assert np.array_equal(a0["labels"], a1["labels"]) and np.array_equal(a0["best"], a1["best"])
    rng = np.random.default_rng(11)
    rows2 = rng.standard_normal(rows.shape).astype(np.float32)
    a2 = oracle.assign_image(emb, None, bw, bh, cells, peak_emb=rows2)
    x = emb.astype(np.float64).reshape(4 * F, -1).T                                  # [HW, 4F]
    d = (np.sqrt(((x[:, None, :2 * F] - rows2[None, :, :2 * F].astype(np.float64)) ** 2).sum(-1)) +
         np.sqrt(((x[:, None, 2 * F:] - rows2[None, :, 2 * F:].astype(np.float64)) ** 2).sum(-1)))
    assert np.array_equal(a2["labels"].ravel(), d.argmin(1) + 1)
    np.testing.assert_allclose(a2["best"].ravel(), d.min(1), rtol=1e-12)


# ---------------------------------------------------------------- the paper's literal local-maxima search on a real-valued map

def test_real_peaks_equal_the_library_maximum_filter_and_a_brute_force():
    """Strict 8-neighbour maxima above a threshold (Sec. 3.2): against scipy's maximum filter on maps of distinct values
    (a bin is a strict maximum iff it equals the 3x3 maximum and no neighbour does), and against a differently written
    brute force; border bins have fewer neighbours; equal neighbours are both rejected; truncation keeps the first K."""
    from scipy import ndimage
    rng = np.random.default_rng(21)
    for shape in ((1, 1), (1, 7), (6, 1), (5, 8), (17, 13)):
        Hm = rng.random(shape) * 10.0                           # distinct with probability 1
        thr = 3.0
        cells, raw = oracle.real_peaks(Hm, thr, 10_000)
        mx = ndimage.maximum_filter(Hm, size=3, mode="constant", cval=-np.inf)
        want = np.flatnonzero(((Hm == mx) & (Hm > thr)).ravel())
        assert np.array_equal(cells, want) and raw == want.size, shape
        brute = []
        bh, bw = shape
        for lin in range(bh * bw):
            cy, cx = divmod(lin, bw)
            nb = [Hm[y, x] for y in range(max(0, cy - 1), min(bh, cy + 2)) for x in range(max(0, cx - 1), min(bw, cx + 2))
                  if (y, x) != (cy, cx)]
            if Hm[cy, cx] > thr and all(Hm[cy, cx] > v for v in nb):
                brute.append(lin)
        assert cells.tolist() == brute
        if len(brute) > 2:
            first, raw2 = oracle.real_peaks(Hm, thr, 2)
            assert first.tolist() == brute[:2] and raw2 == len(brute)
    # hand cases: a plateau of two equal bins yields no peak (the literal test; the integer map's tie rule is an extension)
    Hm = np.zeros((4, 5))
    Hm[1, 1] = Hm[1, 2] = 5.0
    Hm[3, 4] = 2.0                                               # a corner bin
    cells, raw = oracle.real_peaks(Hm, 1.0, 16)
    assert cells.tolist() == [3 * 5 + 4] and raw == 1
    cells, _ = oracle.real_peaks(Hm, 2.0, 16)                    # the threshold is strict
    assert cells.tolist() == []


def test_soft_vote_chain_finds_the_instances_of_clean_encodings():
    """Eq. 6 -> local maxima -> Eq. 7 on an alias-free grid (L = 4, 32 bins: the paper's setting) with noise-free
    encodings of centroids on bin positions: the peaks are exactly the centroids' bins and the labels the instances."""
    H, W, F, bw, bh = 48, 64, 4, 32, 32
    inst = np.zeros((H, W), np.int32)
    inst[2:20, 3:30] = 1
    inst[24:46, 5:25] = 2
    inst[10:40, 36:60] = 3
    bins = [(6, 5), (9, 22), (25, 14)]
    cents = np.array([[-1 + 2 * (cx + 1) / (bw + 1), -1 + 2 * (cy + 1) / (bh + 1)] for cx, cy in bins])
    emb = wl.encode(inst, cents, F, 0.0, None, np.float32)[None]
    fg = (inst > 0).astype(np.uint8)[None]
    # side lobes of the sinusoidal kernel reach a quarter of a main lobe here (the largest is 121 against 451..725):
    # the threshold separates them, as the paper's does
    res = oracle.decode_soft(emb, fg, bw, bh, threshold=200.0)
    assert res["count"][0] == 3
    assert res["peak_cell"][0, :3].tolist() == sorted(cy * bw + cx for cx, cy in bins)
    order = np.argsort([cy * bw + cx for cx, cy in bins])
    relabel = np.zeros(4, np.int32)
    relabel[1 + order] = 1 + np.arange(3)
    assert np.array_equal(res["labels"][0], relabel[inst])
    # the histogram's value at an instance's own bin: its pixels contribute exp(-0) = 1 each, the others less
    for (cx, cy), area in zip(bins, [(inst == i).sum() for i in (1, 2, 3)]):
        assert area <= res["hist"][0, cy, cx] < area + (fg.sum() - area) * np.exp(-0.3)
