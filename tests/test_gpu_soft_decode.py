"""The decode with the paper's own vote (Eq. 5-6 -> Sec. 3.2 local maxima -> Eq. 7-8) through the C ABI, against the
binary64 oracle chain.  All tests need a B200.

The histogram is real-valued, so the kernel's H differs from the oracle's within the soft-vote kernel's stated
accuracy, and a bin whose margin to the threshold or to a neighbour is below that accuracy may be decided either way.
The comparison therefore has three parts: (1) H within REL of the oracle's; (2) the kernel's peak list is bit-for-bit
what the printed strict test yields on the kernel's OWN histogram (integer work once H is fixed: exact); (3) every bin
whose decision the oracle takes with a margin above the accuracy is decided the same way.  Labels are then compared
exactly (up to distance near-ties) with the oracle's assignment to the kernel's peaks.
"""
import numpy as np
import pytest

import oracle
from gpu_util import compare_labels
from paper_2609_16874_b200 import binding as cb
from paper_2609_16874_b200 import workloads as wl

pytestmark = pytest.mark.gpu

# accuracy of the soft-vote kernel per bin (see the histogram's own parity test): 1e-4 for F <= 8 (weights as binary16
# high + low parts), 2e-3 for F > 8
def rel_for(F):
    return 1e-4 if F <= 8 else 2e-3


def run_soft_decode(emb, fg, bins_w, bins_h, thr, tau=np.inf, K_max=1024, scores=True, flags=0, twice=False):
    import torch
    B, D, H, W = emb.shape
    F = D // 4
    dtype = "f32" if emb.dtype == np.float32 else "f16"
    dec = cb.Decoder(B, H, W, F, dtype, bins_w, bins_h, 8, float(tau), K_max, 0, write_scores=scores, keep_votes=True,
                     flags=flags, soft_threshold=thr)
    d_emb = torch.from_numpy(emb).cuda()
    d_fg = None if fg is None else torch.from_numpy(np.ascontiguousarray(fg, np.uint8)).cuda()
    dec.decode(d_emb, d_fg)
    if twice:
        dec.decode(d_emb, d_fg)
    torch.cuda.synchronize()
    out = {
        "labels": dec.labels.cpu().numpy(),
        "centroids": dec.centroids.cpu().numpy(),
        "count": dec.count.cpu().numpy(),
        "hist": dec.intermediate(cb.CPE_INT_VOTES).cpu().numpy().view(np.float32),
        "peak_cell": dec.intermediate(cb.CPE_INT_PEAK_CELLS).cpu().numpy(),
        "peak_h": dec.intermediate(cb.CPE_INT_PEAK_VOTES).cpu().numpy().view(np.float32),
        "peak_emb": dec.intermediate(cb.CPE_INT_PEAK_EMB).cpu().numpy(),
        "status": dec.intermediate(cb.CPE_INT_STATUS).cpu().numpy(),
        "counters": dec.intermediate(cb.CPE_INT_COUNTERS).cpu().numpy().astype(np.int64),
    }
    if scores:
        out["best"] = dec.intermediate(cb.CPE_INT_BEST_SCORE).cpu().numpy()
        out["second"] = dec.intermediate(cb.CPE_INT_SECOND_SCORE).cpu().numpy()
    dec.close()
    return out


def robust_decisions(Hm, thr, REL):
    """Per bin of the oracle's map: (is a peak, the decision's margin is above the kernel's accuracy)."""
    bh, bw = Hm.shape
    pad = np.full((bh + 2, bw + 2), -np.inf)
    pad[1:-1, 1:-1] = Hm
    peak = Hm > thr
    robust = np.abs(Hm - thr) > 2 * REL * np.maximum(Hm, thr)
    clear_loss = np.zeros_like(peak)          # some neighbour beats the bin by more than the accuracy
    all_clear_wins = np.ones_like(peak)       # the bin beats every neighbour by more than the accuracy
    for dy in (0, 1, 2):
        for dx in (0, 1, 2):
            if dy == 1 and dx == 1:
                continue
            nb = pad[dy:dy + bh, dx:dx + bw]
            peak &= Hm > nb
            tol = 2 * REL * np.maximum(Hm, np.where(np.isfinite(nb), nb, 0.0))
            clear_loss |= nb - Hm > tol
            all_clear_wins &= Hm - nb > tol
    below = (Hm <= thr) & robust
    decided = below | clear_loss | (robust & all_clear_wins)
    return peak, decided


def check_soft_decode(emb, fg, bins_w, bins_h, thr, tau=np.inf, K_max=1024, min_peaks=1, **kw):
    B, D, H, W = emb.shape
    F = D // 4
    gpu = run_soft_decode(emb, fg, bins_w, bins_h, thr, tau, K_max, **kw)
    assert not (np.bitwise_or.reduce(gpu["status"]) & (cb.CPE_STATUS_INTERNAL | cb.CPE_STATUS_TIMEOUT)), gpu["status"]
    want_h = oracle.soft_votes(emb, fg, bins_w, bins_h)
    err = np.abs(gpu["hist"].astype(np.float64) - want_h)
    REL = rel_for(F)
    assert (err <= REL * want_h + 1e-30).all(), float((err / np.maximum(want_h, 1e-300)).max())
    Pw, Ph = oracle.palette(bins_w, F), oracle.palette(bins_h, F)
    thr32 = float(np.float32(thr))
    n_decided_peaks = 0
    for b in range(B):
        # (2) exact on the kernel's own map
        cells, raw = oracle.real_peaks(gpu["hist"][b].astype(np.float64), thr32, K_max)
        n = int(gpu["count"][b])
        assert n == cells.size and np.array_equal(gpu["peak_cell"][b, :n], cells)
        assert gpu["counters"][b, cb.CPE_CNT_RAW_PEAKS] == raw
        assert gpu["counters"][b, cb.CPE_CNT_TRUNCATED] == raw - n
        assert bool(gpu["status"][b] & cb.CPE_STATUS_PEAK_OVERFLOW) == (raw > K_max)
        assert np.array_equal(gpu["peak_h"][b, :n].view(np.uint32),
                              gpu["hist"][b].ravel()[cells].view(np.uint32))
        want_emb = np.concatenate([Pw[cells % bins_w], Ph[cells // bins_w]], 1)
        assert np.array_equal(gpu["peak_emb"][b, :n].view(np.uint32), want_emb.view(np.uint32))
        for i, lin in enumerate(cells):
            c = oracle.centroid_px(int(lin % bins_w), int(lin // bins_w), bins_w, bins_h, H, W)
            np.testing.assert_allclose(gpu["centroids"][b, i], c, rtol=1e-4, atol=1e-4)
        # (3) the oracle's confident decisions
        o_peak, decided = robust_decisions(want_h[b], thr32, REL)
        if raw <= K_max:
            g_peak = np.zeros(bins_w * bins_h, bool)
            g_peak[cells] = True
            g_peak = g_peak.reshape(bins_h, bins_w)
            assert np.array_equal(g_peak[decided], o_peak[decided])
        n_decided_peaks += int((o_peak & decided).sum())
        # labels: the oracle's assignment to the kernel's peaks
        a = oracle.assign_image(emb[b], None if fg is None else fg[b], bins_w, bins_h, cells.astype(np.int32), tau)
        compare_labels(gpu["labels"][b], gpu["best"][b] if "best" in gpu else None,
                       gpu["second"][b] if "second" in gpu else None, a["labels"], a["best"], a["second"])
    assert n_decided_peaks >= min_peaks            # the confident part of the comparison is not empty
    # participating pixels and the non-finite ones among them
    part = np.ones((B, H, W), bool) if fg is None else fg.astype(bool)
    fin = np.isfinite(emb.astype(np.float32)).all(axis=1)
    assert np.array_equal(gpu["counters"][:, cb.CPE_CNT_VOTING], (part & fin).reshape(B, -1).sum(1))
    assert np.array_equal(gpu["counters"][:, cb.CPE_CNT_NONFINITE], (part & ~fin).reshape(B, -1).sum(1))
    for b in range(B):
        assert bool(gpu["status"][b] & cb.CPE_STATUS_NONFINITE) == bool((part & ~fin)[b].any())
    return gpu


@pytest.mark.parametrize("name,over,thr", [
    ("c1", dict(), 330.0),                                             # 128x128, F=4 fp32, 32x32 bins: the paper's grid
    ("c2", dict(H=192, W=256, K=12), 30.0),                            # F=8 fp32, 64x64 bins
    ("c3", dict(H=96, W=128, K=6, bins_w=72, bins_h=66), 40.0),        # fp16
    ("c5", dict(H=96, W=128, K=12, bins_w=48, bins_h=40), 0.3),        # F=16 fp16
])
def test_soft_vote_decode_matches_the_oracle_chain(name, over, thr):
    cfg = wl.scaled(wl.CONFIGS[name], **over)
    fr = wl.make_frame(cfg, 0)
    gpu = check_soft_decode(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h, thr, min_peaks=2)
    assert gpu["count"][0] >= 2


def test_soft_vote_decode_batch_tau_truncation_and_second_call():
    cfg = wl.scaled(wl.CONFIGS["c1"], B=3, K=9)
    fr = wl.make_frame(cfg, 4)
    emb, fg = fr["emb"].copy(), fr["fg"].copy()
    fg[2] = 0                                                          # an image without participating pixels
    emb[0, 5, 3, 9] = np.nan
    emb[1, 2, 7, 7] = np.inf
    fg[0, 3, 9] = 1
    fg[1, 7, 7] = 1
    gpu = check_soft_decode(emb, fg, cfg.bins_w, cfg.bins_h, 250.0, tau=1.2, twice=True)
    assert gpu["count"][2] == 0 and (gpu["labels"][2] == 0).all()
    assert (gpu["labels"][:2][fg[:2] > 0] == 0).any()                   # tau rejects some pixels
    # a low threshold lets side lobes through: more local maxima than K_max, the first K_max are kept
    gpu = check_soft_decode(emb, fg, cfg.bins_w, cfg.bins_h, 60.0, K_max=4, min_peaks=0)
    assert (gpu["status"][:2] & cb.CPE_STATUS_PEAK_OVERFLOW).all() and (gpu["count"][:2] == 4).all()
    # no mask, no score output, and each assignment kernel family
    for flags in (0, cb.CPE_FLAG_EXACT_ASSIGN, cb.CPE_FLAG_FILTER_ASSIGN):
        check_soft_decode(emb, None, cfg.bins_w, cfg.bins_h, 250.0, scores=False, flags=flags)


def test_soft_vote_decode_many_peaks_takes_the_filtered_assignment():
    cfg = wl.scaled(wl.CONFIGS["c4"], B=1, H=128, W=160, K=40, bins_w=64, bins_h=48)
    fr = wl.make_frame(cfg, 2)
    gpu = check_soft_decode(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h, 5.0, min_peaks=20)
    assert gpu["count"][0] > 32                                         # beyond the all-pairs range


def test_soft_vote_decode_rejects_what_it_cannot_do():
    import torch
    B, H, W, F = 1, 30, 31, 4                                           # H*W not a multiple of 8
    dec = cb.Decoder(B, H, W, F, "f32", 16, 16, soft_threshold=5.0)
    emb = torch.zeros((B, 4 * F, H, W), device="cuda")
    with pytest.raises(cb.CpeError) as e:
        dec.decode(emb, None)
    assert e.value.code == cb.CPE_ERR_ALIGN
    dec.close()
    p = cb.make_params(cb.CPE_F32, 16, 16, flags=cb.CPE_FLAG_SOFT_VOTE | cb.CPE_FLAG_REFINE, soft_threshold=1.0)
    assert cb.cpe_workspace_size(1, 32, 32, 4, p) == 0
    for bad in (-1.0, float("nan"), float("inf")):
        p = cb.make_params(cb.CPE_F32, 16, 16, flags=cb.CPE_FLAG_SOFT_VOTE, soft_threshold=bad)
        assert cb.cpe_workspace_size(1, 32, 32, 4, p) == 0
