"""The pruned assignment (per-peak candidate lists from triangle-inequality bounds, Eq. 7 restricted to the peaks that
can still win) against the CPU oracle and against the all-pairs kernel, through the C ABI.  Needs a B200.

Pruning must not change a single result: labels follow the usual rule (exact except where the oracle's top-2 margin
is a near-tie), and best / second-best distances are the same bits as the all-pairs kernel's, because every kernel
scores a (pixel, peak) pair in the same fixed binary32 order.
"""
import numpy as np
import pytest

import oracle
from paper_2609_16874_b200 import binding as cb
from paper_2609_16874_b200 import workloads as wl

from gpu_util import compare_front, compare_labels, run_gpu

pytestmark = pytest.mark.gpu

PRUNE_ALL = cb.CPE_FLAG_PRUNE_ALL
ANY_SIZE = cb.CPE_FLAG_PRUNE_ANY_SIZE     # the pruned assignment as the library chooses it, also on these small inputs


def check_pruned(emb, fg, bins_w, bins_h, T_v=8, tau=np.inf, K_max=1024, refine=False, flags=PRUNE_ALL, mode="direct",
                 expect_handed_on=None):
    """GPU with the pruned assignment vs the oracle and vs the all-pairs kernel; returns the GPU run with scores."""
    F = emb.shape[1] // 4
    if refine:
        ora = oracle.decode_refined(emb, fg, bins_w, bins_h, T_v, tau, K_max)
    else:
        ora = oracle.decode(emb, fg, bins_w, bins_h, T_v, tau, K_max)
    exact = run_gpu(emb, fg, bins_w, bins_h, T_v, tau, K_max, 0, True, mode, exact_assign=True, refine=refine,
                    keep_votes=False)
    out = None
    # with scores (the one-thread-per-pixel kernel), without (the streaming kernel where the shapes allow it, then the
    # queue walk), and without scores on the one-thread-per-pixel kernel
    for scores, extra in ((True, 0), (False, 0), (False, cb.CPE_FLAG_PRUNE_WALK_ONLY)):
        gpu = run_gpu(emb, fg, bins_w, bins_h, T_v, tau, K_max, 0, scores, mode, keep_votes=False, refine=refine,
                      flags=flags | extra)
        assert not (gpu["status"] & cb.CPE_STATUS_INTERNAL), hex(gpu["status"])
        assert gpu["prune_state"] is not None, "the pruned assignment was not enabled"
        assert np.array_equal(gpu["count"], ora["count"])
        if not refine:
            compare_front(gpu, ora, F, bins_w, bins_h)
        compare_labels(gpu["labels"], gpu.get("best"), gpu.get("second"), ora["labels"], ora["best"], ora["second"])
        assert np.array_equal(gpu["labels"], exact["labels"])
        if scores:
            assert np.array_equal(gpu["best"].view(np.uint32), exact["best"].view(np.uint32))
            assert np.array_equal(gpu["second"].view(np.uint32), exact["second"].view(np.uint32))
            out = gpu
        # the tau-rejected counter is exact whichever kernel finished the image
        assert np.array_equal(gpu["counters"][:, cb.CPE_CNT_TAU_REJECTED], exact["counters"][:, cb.CPE_CNT_TAU_REJECTED])
        # (checked without scores: when the runner-up's distance is wanted as well, a walk can only end at
        # G > second-best + t, which heavy noise puts beyond every candidate)
        handed = gpu["prune_state"][:, 2] != 0
        if expect_handed_on is not None and not scores:
            assert handed.tolist() == list(expect_handed_on), gpu["prune_state"].tolist()
    return out, ora


SMALL = [
    ("c1", dict()),
    ("c1", dict(H=67, W=93)),                                              # odd sizes: scalar-load vote kernel
    ("c2", dict(H=192, W=256, K=12)),
    ("c3", dict(H=256, W=384, K=24, bins_w=96, bins_h=64)),
    ("c3", dict(H=99, W=121, K=8, bins_w=64, bins_h=32)),
    ("c4", dict(B=3, H=160, W=168, K=30, bins_w=40, bins_h=40)),
    ("c5", dict(H=256, W=256, K=40, bins_w=128, bins_h=128)),
]


@pytest.mark.parametrize("name,over", SMALL, ids=[f"{n}-{i}" for i, (n, _) in enumerate(SMALL)])
@pytest.mark.parametrize("refine", [False, True], ids=["bins", "refined"])
@pytest.mark.parametrize("mode", ["direct", "graph"])
def test_pruned_assignment_matches_oracle_and_all_pairs(name, over, refine, mode):
    cfg = wl.scaled(wl.CONFIGS[name], **over)
    fr = wl.make_frame(cfg, 0)
    gpu, ora = check_pruned(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, cfg.K_max, refine, mode=mode)
    voting = gpu["counters"][:, cb.CPE_CNT_VOTING].sum()
    print(name, over, "refined" if refine else "bins", "pairs per voting pixel",
          gpu["counters"][:, cb.CPE_CNT_FILTER_PAIRS].sum() / max(1, voting), "state", gpu["prune_state"].tolist())


def test_refined_candidates_leave_about_one_candidate_per_pixel():
    # what the bounds are for: with candidates on the voted centroids a pixel's own peak is at noise distance and every
    # other peak is excluded without being scored
    cfg = wl.scaled(wl.CONFIGS["c4"], B=2, H=320, W=384, K=100)
    fr = wl.make_frame(cfg, 0)
    gpu, ora = check_pruned(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, cfg.K_max, refine=True, flags=ANY_SIZE,
                            expect_handed_on=[False, False])
    assert ora["count"].min() > 64                                   # more peaks than a list has entries
    # scores wanted: the walk goes on until the runner-up is settled too, i.e. up to G = (second-best distance) + t
    pairs = gpu["counters"][:, cb.CPE_CNT_FILTER_PAIRS].sum()
    voting = gpu["counters"][:, cb.CPE_CNT_VOTING].sum()
    assert pairs <= 12 * voting, (pairs, voting)
    fast = run_gpu(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, cfg.K_max, 0, False, keep_votes=False,
                   refine=True, flags=ANY_SIZE)
    # (every peak is scored for the few pixels whose instance has no peak of its own: they are far from any reference)
    pairs = fast["counters"][:, cb.CPE_CNT_FILTER_PAIRS].sum()
    full = fast["counters"][:, cb.CPE_CNT_FULL_SCORED].sum()
    assert pairs - full * int(ora["count"].max()) <= 2 * voting, (pairs, full, voting)


def test_aliased_grid_is_handed_to_the_filtered_kernel():
    # F = 16 on 128 bins with sigma = 0.2: the palette rows' upper harmonics are unrelated to any pixel's, no bound
    # separates the peaks, most pixels exhaust their lists, and the image must end up with the filtered kernel -- with
    # the same results
    cfg = wl.scaled(wl.CONFIGS["c5"], H=512, W=512, K=200, bins_w=256, bins_h=256)
    fr = wl.make_frame(cfg, 0)
    gpu, ora = check_pruned(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, cfg.K_max, refine=False, flags=ANY_SIZE,
                            expect_handed_on=[True])
    assert ora["count"][0] > 64
    # ... and with refined candidates the same input stays with the pruned kernel
    check_pruned(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, cfg.K_max, refine=True, flags=ANY_SIZE,
                 expect_handed_on=[False])


def _grid_instances(H, W, F, bw, bh, K, run, sigma, dtype, seed):
    rng = np.random.default_rng(seed)
    cells = np.sort(rng.choice(bw // 2 * (bh // 2), K, replace=False))
    cx, cy = 2 * (cells % (bw // 2)), 2 * (cells // (bw // 2))          # no two peaks adjacent
    inst = ((np.arange(H * W) // run) % K + 1).reshape(H, W).astype(np.int32)
    cents = np.stack([-1 + 2 * (cx + 1) / (bw + 1), -1 + 2 * (cy + 1) / (bh + 1)], 1)
    emb = wl.encode(inst, cents, F, sigma, rng, dtype)[None]
    return emb, np.ones((1, H, W), np.uint8)


def test_more_peaks_than_list_entries_and_more_than_the_lists_cover():
    # 600 peaks: lists hold the 64 nearest, alias-free grid (F = 4, 64 x 48 bins), so the bounds close every pixel
    emb, fg = _grid_instances(96, 128, 4, 64, 48, 600, 20, 0.02, np.float32, 5)
    gpu, ora = check_pruned(emb, fg, 64, 48, T_v=8, K_max=1024, flags=ANY_SIZE, expect_handed_on=[False])
    assert ora["count"][0] == 600
    # 1100 peaks: beyond what the list kernel serves, the image goes to the filtered kernel untouched
    emb, fg = _grid_instances(160, 160, 4, 96, 64, 1100, 20, 0.02, np.float16, 6)
    gpu, ora = check_pruned(emb, fg, 96, 64, T_v=8, K_max=2048, flags=ANY_SIZE, expect_handed_on=[True])
    assert ora["count"][0] == 1100


@pytest.mark.parametrize("F,dtype,refine", [(4, np.float32, False), (8, np.float16, False), (8, np.float32, True),
                                            (16, np.float16, True)])
def test_instances_without_a_peak_send_their_pixels_to_the_scan_of_every_peak(F, dtype, refine):
    # 66 instances, room for 63 peaks: the pixels of the three instances whose bins come last find no peak for their bin
    # (4.5 % of the image, far below the eighth at which an image is handed on -- that decision follows the order in
    # which the CTAs report, so the test keeps well away from it).  Thousands of pixels, more than the kernel that
    # scores every peak has CTAs, so it takes them eight lanes per pixel, with the 63 candidate rows in two chunks (32 + 31).
    emb, fg = _grid_instances(256, 384, F, 64, 48, 66, 24, 0.03, dtype, 31)
    gpu, ora = check_pruned(emb, fg, 64, 48, K_max=63, refine=refine, flags=ANY_SIZE, expect_handed_on=[False])
    assert ora["count"][0] == 63
    plain = run_gpu(emb, fg, 64, 48, 8, np.inf, 63, 0, False, "direct", keep_votes=False, refine=refine, flags=ANY_SIZE)
    assert plain["prune_state"][0, 8] > 2000, plain["prune_state"].tolist()       # fill of the second queue
    assert np.array_equal(plain["labels"], gpu["labels"])


def test_pruned_assignment_edge_cases():
    cfg = wl.scaled(wl.CONFIGS["c2"], H=128, W=128, K=6, bins_w=32, bins_h=32, sigma=0.1)
    fr = wl.make_frame(cfg, 0)
    ora = oracle.decode(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h)
    # tau in the middle of the distances: rejected pixels are counted exactly
    tau = float(np.median(ora["best"][np.isfinite(ora["best"])]))
    gpu, _ = check_pruned(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h, tau=tau)
    assert 0 < gpu["counters"][0, cb.CPE_CNT_TAU_REJECTED] < fr["fg"].sum()
    # no mask: background pixels (noise around the zero vector) vote anywhere and belong to no peak's window
    check_pruned(fr["emb"], None, cfg.bins_w, cfg.bins_h)
    check_pruned(fr["emb"], None, cfg.bins_w, cfg.bins_h, refine=True)
    # non-finite pixels neither vote nor get a label
    emb = fr["emb"].copy()
    ys, xs = np.nonzero(fr["fg"][0])
    emb[0, 3, ys[::97], xs[::97]] = np.nan
    emb[0, 17, ys[5::131], xs[5::131]] = np.inf
    gpu, _ = check_pruned(emb, fr["fg"], cfg.bins_w, cfg.bins_h)
    assert (gpu["labels"][0, ys[::97], xs[::97]] == 0).all()
    # no foreground, one peak, a single output slot
    check_pruned(fr["emb"], np.zeros_like(fr["fg"]), cfg.bins_w, cfg.bins_h)
    check_pruned(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h, K_max=1)
    check_pruned(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h, K_max=3, refine=True)
    # a batch with no, few and many peaks per image: the pruned chain serves all three (an image without peaks is
    # zero-filled, not walked)
    H, W, F, bw, bh = 96, 128, 4, 64, 48
    rng = np.random.default_rng(8)
    emb = np.empty((3, 4 * F, H, W), np.float16)
    fg = np.zeros((3, H, W), np.uint8)
    emb[0] = rng.standard_normal((4 * F, H, W)).astype(np.float16)
    for b, K in ((1, 5), (2, 60)):
        e, _ = _grid_instances(H, W, F, bw, bh, K, 40, 0.03, np.float16, 20 + b)
        emb[b] = e[0]
        fg[b] = 1
    gpu, ora = check_pruned(emb, fg, bw, bh, flags=ANY_SIZE, expect_handed_on=[False, False, False])
    assert ora["count"].tolist() == [0, 5, 60]
    assert gpu["prune_state"][2, 0] > 0 and gpu["prune_state"][1, 0] > 0 and gpu["prune_state"][0, 0] == 0
