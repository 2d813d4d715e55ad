"""CUDA path vs CPU oracle, element by element, through the C ABI.  All tests need a B200."""
import numpy as np
import pytest

import oracle
from paper_2609_16874_b200 import binding as cb
from paper_2609_16874_b200 import workloads as wl

from gpu_util import check_case, compare_front, compare_labels, run_gpu

pytestmark = pytest.mark.gpu


# Reduced copies of the five configurations: same recipe, sizes the oracle finishes in seconds, several CTAs
# per kernel, with and without a ragged tail (H*W not a multiple of the vector width -> scalar-load kernels).
SMALL = [
    ("c1", dict()),                                                        # the real c1: 128x128
    ("c1", dict(H=67, W=93)),                                              # odd sizes: scalar path
    ("c2", dict(H=192, W=256, K=12)),
    ("c2", dict(H=131, W=77, K=6, bins_w=48, bins_h=40)),
    ("c3", dict(H=256, W=384, K=24, bins_w=96, bins_h=64)),
    ("c3", dict(H=99, W=121, K=8, bins_w=64, bins_h=32)),
    ("c4", dict(B=3, H=160, W=168, K=30, bins_w=40, bins_h=40)),
    ("c5", dict(H=256, W=256, K=40, bins_w=128, bins_h=128)),
]


@pytest.mark.parametrize("name,over", SMALL, ids=[f"{n}-{i}" for i, (n, _) in enumerate(SMALL)])
@pytest.mark.parametrize("mode", ["direct", "graph"])
def test_small_configs_match_oracle(name, over, mode):
    cfg = wl.scaled(wl.CONFIGS[name], **over)
    fr = wl.make_frame(cfg, 0)
    gpu, ora, rep = check_case(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, cfg.K_max, mode=mode)
    assert ora["count"].min() >= 1
    assert gpu["status"] == 0
    print(name, over, "near ties:", rep)


@pytest.mark.parametrize("F,dtype", [(1, np.float32), (2, np.float16), (3, np.float32), (5, np.float16), (12, np.float32)])
def test_other_harmonic_counts(F, dtype):
    cfg = wl.scaled(wl.CONFIGS["c2"], H=64, W=80, K=5, F=F, bins_w=16, bins_h=16,
                    dtype="f32" if dtype == np.float32 else "f16", sigma=0.02)
    fr = wl.make_frame(cfg, 2)
    check_case(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h)


def test_no_mask_all_pixels_participate():
    cfg = wl.scaled(wl.CONFIGS["c1"], H=64, W=64)
    fr = wl.make_frame(cfg, 1)
    gpu, ora, _ = check_case(fr["emb"], None, cfg.bins_w, cfg.bins_h)
    assert ora["counters"][0, oracle.CNT_VOTING] == 64 * 64


def test_empty_foreground_and_no_peaks():
    cfg = wl.scaled(wl.CONFIGS["c3"], H=64, W=128, K=4, bins_w=32, bins_h=16)
    fr = wl.make_frame(cfg, 0)
    fg = np.zeros_like(fr["fg"])
    gpu, ora, _ = check_case(fr["emb"], fg, cfg.bins_w, cfg.bins_h)
    assert gpu["count"][0] == 0 and (gpu["labels"] == 0).all() and gpu["votes"].sum() == 0
    # foreground too small for any bin to pass the threshold: votes exist, no peak, all labels 0
    fg[0, :2, :3] = 1
    gpu, ora, _ = check_case(fr["emb"], fg, cfg.bins_w, cfg.bins_h)
    assert gpu["count"][0] == 0 and (gpu["labels"] == 0).all() and gpu["votes"].sum() == 6


def test_nonfinite_pixels_are_skipped_and_counted():
    for dtype in ("f32", "f16"):
        cfg = wl.scaled(wl.CONFIGS["c2"], H=96, W=96, K=5, dtype=dtype, bins_w=32, bins_h=32)
        fr = wl.make_frame(cfg, 0)
        emb = fr["emb"].copy()
        ys, xs = np.nonzero(fr["fg"][0])
        rng = np.random.default_rng(0)
        pick = rng.choice(ys.size, 40, replace=False)
        for i, j in enumerate(pick):
            emb[0, rng.integers(0, cfg.D), ys[j], xs[j]] = [np.nan, np.inf, -np.inf][i % 3]
        if dtype == "f32":
            # a FINITE (sin, cos) pair whose |s| + |c| overflows binary32 counts as non-finite too (binary16 cannot hold one)
            j = pick[0]
            emb[0, :, ys[j], xs[j]] = fr["emb"][0, :, ys[j], xs[j]]
            emb[0, 4, ys[j], xs[j]] = 2.5e38
            emb[0, 5, ys[j], xs[j]] = -2.5e38
        gpu, ora, _ = check_case(emb, fr["fg"], cfg.bins_w, cfg.bins_h)
        assert gpu["counters"][0, cb.CPE_CNT_NONFINITE] == 40
        assert gpu["status"] & cb.CPE_STATUS_NONFINITE
        assert (gpu["labels"][0, ys[pick], xs[pick]] == 0).all()


def test_peak_overflow_keeps_first_k_max():
    cfg = wl.scaled(wl.CONFIGS["c4"], B=2, H=160, W=160, K=30, bins_w=40, bins_h=40)
    fr = wl.make_frame(cfg, 0)
    gpu, ora, _ = check_case(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h, K_max=7)
    assert (gpu["count"] == 7).all() and gpu["status"] & cb.CPE_STATUS_PEAK_OVERFLOW
    assert (gpu["counters"][:, cb.CPE_CNT_TRUNCATED] > 0).all()


def test_tau_rejection_and_levels():
    cfg = wl.scaled(wl.CONFIGS["c2"], H=128, W=128, K=6, bins_w=32, bins_h=32, sigma=0.1)
    fr = wl.make_frame(cfg, 0)
    ora = oracle.decode(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h)
    tau = float(np.median(ora["best"][np.isfinite(ora["best"])]))
    gpu, ora2, _ = check_case(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h, tau=tau)
    assert 0 < gpu["counters"][0, cb.CPE_CNT_TAU_REJECTED] < fr["fg"].sum()
    for levels in (1, 3, 6):
        check_case(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h, levels=levels)


def test_threshold_and_tie_rules_on_constructed_votes():
    # Noise-free encodings of centroids on bin positions give an exactly known vote map; equal-area
    # neighbours make a two-bin plateau, which must resolve to the lower linear index on both sides.
    H, W, F, bw, bh = 64, 64, 4, 16, 16
    inst = np.zeros((H, W), np.int32)
    inst[0:16, 0:16] = 1
    inst[0:16, 16:32] = 2          # same area as 1, adjacent bins -> tie
    inst[32:64, 0:32] = 3
    inst[40:43, 40:43] = 4         # 9 pixels: above T_v = 8
    inst[50:52, 50:54] = 5         # 8 pixels: not above
    bins = [(3, 3), (4, 3), (10, 12), (13, 2), (8, 8)]
    cents = np.array([[-1 + 2 * (cx + 1) / (bw + 1), -1 + 2 * (cy + 1) / (bh + 1)] for cx, cy in bins])
    emb = wl.encode(inst, cents, F, 0.0, None, np.float32)[None]
    fg = (inst > 0).astype(np.uint8)[None]
    gpu, ora, _ = check_case(emb, fg, bw, bh, T_v=8)
    assert gpu["count"][0] == 3
    assert gpu["peak_cell"][0, :3].tolist() == sorted([3 * bw + 3, 12 * bw + 10, 2 * bw + 13])


@pytest.mark.parametrize("name,over", [("c2", dict(H=192, W=256, K=12)), ("c5", dict(H=256, W=256, K=40, bins_w=128, bins_h=128)),
                                       ("c3", dict(H=99, W=121, K=8, bins_w=64, bins_h=32))])
def test_exact_all_pairs_assignment_agrees(name, over):
    # the plain-ALU kernel that scores every (pixel, peak) pair and the tensor-core filtered kernel must agree bit for bit
    cfg = wl.scaled(wl.CONFIGS[name], **over)
    fr = wl.make_frame(cfg, 1)
    a = run_gpu(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h, exact_assign=True)
    b = run_gpu(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h, filter_assign=True)
    c = run_gpu(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h, filter_assign=True, scores=False)
    assert np.array_equal(a["labels"], b["labels"]) and np.array_equal(a["labels"], c["labels"])
    assert np.array_equal(a["best"].view(np.uint32), b["best"].view(np.uint32))
    assert np.array_equal(a["second"].view(np.uint32), b["second"].view(np.uint32))
    ora = oracle.decode(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h)
    compare_labels(a["labels"], a["best"], a["second"], ora["labels"], ora["best"], ora["second"])


def test_many_peaks_and_fp32_out_of_half_range():
    # more peaks than fit the resident peak operand (several peak chunks), and binary32 pixels too large for binary16
    rng = np.random.default_rng(5)
    H, W, F, bw, bh = 96, 128, 4, 64, 48
    K = 600
    cells = np.sort(rng.choice(bw // 2 * (bh // 2), K, replace=False))
    cx, cy = 2 * (cells % (bw // 2)), 2 * (cells // (bw // 2))          # no two peaks adjacent
    inst = np.zeros((H, W), np.int32)
    inst.ravel()[:] = (np.arange(H * W) // 20) % K + 1                     # 20 pixels per run: every bin gets > T_v votes
    cents = np.stack([-1 + 2 * (cx + 1) / (bw + 1), -1 + 2 * (cy + 1) / (bh + 1)], 1)
    emb = wl.encode(inst, cents, F, 0.02, rng, np.float32)[None]
    emb[0, 3, 5, 7] = 1e5
    emb[0, 9, 50, 60] = -7e4
    fg = np.ones((1, H, W), np.uint8)
    gpu, ora, rep = check_case(emb, fg, bw, bh, T_v=8, K_max=1024)
    assert ora["count"][0] == K


def test_ragged_batch_scalar_path():
    # H*W odd (no vector loads anywhere), several images
    for dtype in ("f16", "f32"):
        cfg = wl.scaled(wl.CONFIGS["c4"], B=3, H=37, W=53, K=6, bins_w=24, bins_h=20, dtype=dtype, sigma=0.05)
        fr = wl.make_frame(cfg, 0)
        check_case(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h, T_v=4)


def test_degenerate_shapes_and_parameters():
    rng = np.random.default_rng(3)
    # one row of pixels, one bin: every participating pixel votes for it and is assigned to it
    emb = rng.standard_normal((1, 8, 1, 24)).astype(np.float32)
    fg = np.ones((1, 1, 24), np.uint8)
    gpu, ora, _ = check_case(emb, fg, 1, 1, T_v=8)
    assert gpu["count"][0] == 1 and (gpu["labels"] == 1).all()
    # threshold 0, a single output slot, and K_max equal to the number of peaks
    cfg = wl.scaled(wl.CONFIGS["c2"], H=64, W=72, K=5, bins_w=24, bins_h=24)
    fr = wl.make_frame(cfg, 4)
    gpu, ora, _ = check_case(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h, T_v=0)
    n = int(ora["count"][0])
    check_case(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h, T_v=0, K_max=1)
    check_case(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h, T_v=0, K_max=n)
    # long thin vote map (1024 x 2 bins)
    check_case(fr["emb"], fr["fg"], 1024, 2, T_v=2)


def test_batch_with_no_few_and_many_peaks_per_image():
    # one workspace, three images: none / a handful / more than the all-pairs limit of peaks, so that the two
    # assignment kernels each take some of the images and leave the others alone
    H, W, F, bw, bh = 96, 128, 4, 64, 48
    rng = np.random.default_rng(8)
    emb = np.empty((3, 4 * F, H, W), np.float16)
    fg = np.zeros((3, H, W), np.uint8)
    emb[0] = rng.standard_normal((4 * F, H, W)).astype(np.float16)           # image 0: no foreground at all
    for b, K in ((1, 5), (2, 60)):
        cells = np.sort(rng.choice(bw // 2 * (bh // 2), K, replace=False))
        cx, cy = 2 * (cells % (bw // 2)), 2 * (cells // (bw // 2))
        inst = ((np.arange(H * W) // 40) % K + 1).reshape(H, W).astype(np.int32)
        cents = np.stack([-1 + 2 * (cx + 1) / (bw + 1), -1 + 2 * (cy + 1) / (bh + 1)], 1)
        emb[b] = wl.encode(inst, cents, F, 0.03, rng, np.float16)
        fg[b] = 1
    gpu, ora, _ = check_case(emb, fg, bw, bh, T_v=8)
    assert ora["count"].tolist() == [0, 5, 60]


def test_host_front_end_matches_device_path():
    cfg = wl.scaled(wl.CONFIGS["c4"], B=2, H=96, W=104, K=10, bins_w=24, bins_h=24)
    fr = wl.make_frame(cfg, 0)
    ora = oracle.decode(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, cfg.K_max)
    hd = cb.HostDecoder(cfg.B, cfg.H, cfg.W, cfg.F, cfg.dtype, cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, cfg.K_max)
    labels = np.full((cfg.B, cfg.H, cfg.W), -1, np.int32)
    cents = np.zeros((cfg.B, cfg.K_max, 2), np.float32)
    count = np.zeros(cfg.B, np.int32)
    for _ in range(2):
        hd.decode(fr["emb"], fr["fg"], labels, cents, count)
        assert np.array_equal(count, ora["count"])
        rep = compare_labels(labels, None, None, ora["labels"], ora["best"], ora["second"])
    assert hd.h2d_bytes == fr["emb"].nbytes + fr["fg"].nbytes
    assert hd.d2h_bytes == labels.nbytes + cents.nbytes + count.nbytes
    hd.close()


def test_host_front_end_pipelined_submissions_keep_their_order_and_results():
    import torch
    cfg = wl.scaled(wl.CONFIGS["c2"], H=128, W=160, K=7, bins_w=32, bins_h=32)
    frames = [wl.make_frame(cfg, i) for i in range(5)]
    want = [oracle.decode(f["emb"], f["fg"], cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, cfg.K_max) for f in frames]
    hd = cb.HostDecoder(cfg.B, cfg.H, cfg.W, cfg.F, cfg.dtype, cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, cfg.K_max)
    emb = [torch.from_numpy(f["emb"]).pin_memory() for f in frames]
    fg = [torch.from_numpy(f["fg"]).pin_memory() for f in frames]
    out = [(torch.full((cfg.B, cfg.H, cfg.W), -1, dtype=torch.int32).pin_memory(),
            torch.zeros((cfg.B, cfg.K_max, 2), dtype=torch.float32).pin_memory(),
            torch.zeros((cfg.B,), dtype=torch.int32).pin_memory()) for _ in frames]
    assert cb.cpe_host_wait(hd.ctx) == cb.CPE_ERR_PARAM                      # nothing in flight
    hd.submit(emb[0], fg[0], *out[0])
    hd.submit(emb[1], fg[1], *out[1])
    ptr = lambda a: a.data_ptr()
    assert cb.cpe_host_submit(hd.ctx, ptr(emb[2]), ptr(fg[2]), *[ptr(o) for o in out[2]]) == cb.CPE_ERR_BUSY
    assert cb.cpe_host_decode(hd.ctx, ptr(emb[2]), ptr(fg[2]), *[ptr(o) for o in out[2]]) == cb.CPE_ERR_BUSY
    for i in range(2, 5):                                                     # steady state: two in flight
        hd.wait()
        hd.submit(emb[i], fg[i], *out[i])
    hd.wait()
    hd.wait()
    for i in range(5):
        lab, cen, cnt = (o.numpy() for o in out[i])
        assert np.array_equal(cnt, want[i]["count"]), i
        compare_labels(lab, None, None, want[i]["labels"], want[i]["best"], want[i]["second"])
        n = int(cnt[0])
        np.testing.assert_allclose(cen[0, :n], want[i]["centroids"][0, :n], rtol=1e-4, atol=1e-4)
    hd.decode(emb[3], fg[3], *out[0])                                         # the synchronous call still works afterwards
    assert np.array_equal(out[0][0].numpy(), out[3][0].numpy())
    hd.close()


def test_profile_entry_point_reports_all_stages():
    import torch
    cfg = wl.scaled(wl.CONFIGS["c2"], H=128, W=128, K=6, bins_w=32, bins_h=32)
    fr = wl.make_frame(cfg, 0)
    dec = cb.Decoder(cfg.B, cfg.H, cfg.W, cfg.F, cfg.dtype, cfg.bins_w, cfg.bins_h)
    ms = dec.profile(torch.from_numpy(fr["emb"]).cuda(), torch.from_numpy(fr["fg"]).cuda(), iters=3)
    assert set(ms) == set(cb.CPE_STAGE_NAMES) and all(v >= 0 for v in ms.values())
    assert ms["decode_vote"] > 0 and ms["peaks"] > 0 and ms["assign"] > 0
    ora = oracle.decode(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h, want_scores=True)
    compare_labels(dec.labels.cpu().numpy(), None, None, ora["labels"], ora["best"], ora["second"])
    dec.close()


# ---------------------------------------------------------------- the five configurations at full size

@pytest.mark.parametrize("name", ["c1", "c2", "c3", "c4", "c5"])
def test_full_size_configs(name):
    """Full-size inputs in the launch configuration the benchmark times (graph replay): votes, peaks, counts and
    centroids against the full oracle; labels and scores on sampled pixels the oracle scores one by one; label-map
    properties on every pixel."""
    cfg = wl.CONFIGS[name]
    fr = wl.make_frame(cfg, 0)
    emb, fg = fr["emb"], fr["fg"]
    gpu = run_gpu(emb, fg, cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, cfg.K_max, 0, True, "graph")
    ov = oracle.votes(emb, fg, cfg.bins_w, cfg.bins_h)
    ora = {"votes": ov["votes"], "counters": ov["counters"], "count": np.zeros(cfg.B, np.int32),
           "peak_cell": np.full((cfg.B, cfg.K_max), -1, np.int32), "peak_votes": np.zeros((cfg.B, cfg.K_max), np.uint32),
           "centroids": np.zeros((cfg.B, cfg.K_max, 2), np.float32)}
    for b in range(cfg.B):
        cells, pv, raw = oracle.peaks(ov["votes"][b], cfg.T_v, cfg.K_max)
        n = len(cells)
        ora["count"][b] = n
        ora["peak_cell"][b, :n], ora["peak_votes"][b, :n] = cells, pv
        ora["counters"][b, oracle.CNT_RAW_PEAKS], ora["counters"][b, oracle.CNT_TRUNCATED] = raw, raw - n
        for k, lin in enumerate(cells):
            ora["centroids"][b, k] = oracle.centroid_px(lin % cfg.bins_w, lin // cfg.bins_w, cfg.bins_w, cfg.bins_h,
                                                        cfg.H, cfg.W)
    compare_front(gpu, ora, cfg.F, cfg.bins_w, cfg.bins_h)
    rng = np.random.default_rng(99)
    n_sample = {"c1": cfg.H * cfg.W, "c2": 60000, "c3": 40000, "c4": 8000, "c5": 12000}[name]
    near = excused = 0
    for b in range(cfg.B):
        n = int(ora["count"][b])
        idx = np.sort(rng.choice(cfg.H * cfg.W, min(n_sample, cfg.H * cfg.W), replace=False)).astype(np.int64)
        res = oracle.assign_image(emb[b], fg[b], cfg.bins_w, cfg.bins_h, ora["peak_cell"][b, :n], cfg.tau, idx=idx)
        rep = compare_labels(gpu["labels"][b].ravel()[idx], gpu["best"][b].ravel()[idx],
                             gpu["second"][b].ravel()[idx], res["labels"], res["best"], res["second"])
        near += rep["near_tie_pixels"]
        excused += rep["excused_mismatches"]
        lab = gpu["labels"][b]
        assert ((lab > 0) == (fg[b] > 0)).all()          # tau = inf: labels partition the foreground
        assert lab.max() <= n and lab.min() >= 0
    assert gpu["status"] == 0
    print(f"{name}: peaks {ora['count'].tolist()}, sampled near-tie pixels {near}, excused label differences {excused}")
    # the configuration the benchmark times -- no score output, vote map re-zeroed by the last kernel, graph replay --
    # against the oracle's assignment of EVERY pixel (all host threads; a few seconds for c5)
    fast = run_gpu(emb, fg, cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, cfg.K_max, 0, False, "graph", keep_votes=False)
    compare_front(fast, ora, cfg.F, cfg.bins_w, cfg.bins_h)
    assert fast["status"] == 0
    oracle.set_threads(oracle.max_threads())
    near = excused = 0
    for b in range(cfg.B):
        n = int(ora["count"][b])
        res = oracle.assign_image(emb[b], fg[b], cfg.bins_w, cfg.bins_h, ora["peak_cell"][b, :n], cfg.tau)
        rep = compare_labels(fast["labels"][b], None, None, res["labels"], res["best"], res["second"])
        near += rep["near_tie_pixels"]
        excused += rep["excused_mismatches"]
    handed = None if fast["prune_state"] is None else fast["prune_state"][:, 2].tolist()
    pairs = fast["counters"][:, cb.CPE_CNT_FILTER_PAIRS].sum() / max(1, fast["counters"][:, cb.CPE_CNT_VOTING].sum())
    print(f"{name} (no scores, every pixel): near-tie pixels {near}, excused {excused}, handed on {handed}, "
          f"scored pairs per voting pixel {pairs:.2f}")


def test_tensor_memory_path_with_several_rounds_of_peaks():
    """The tcgen05 assignment serves up to 128 peaks by default; with CPE_FLAG_TC_ALL_ROUNDS it takes every image whose
    peaks fit its shared-memory operand, in rounds of 64, and with CPE_FLAG_TC_ONE_STAGE only those with at most 64.
    Labels and scores must be those of the all-pairs kernel, bit for bit.  (CPE_FLAG_NO_PRUNE: these images would
    otherwise go to the pruned assignment first.)"""
    for name, over in (("c4", dict(B=2, H=320, W=384, K=100)), ("c5", dict(H=512, W=512, K=200, bins_w=256, bins_h=256))):
        cfg = wl.scaled(wl.CONFIGS[name], **over)
        fr = wl.make_frame(cfg, 0)
        for scores in (False, True):
            b = run_gpu(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, cfg.K_max, scores=scores,
                        keep_votes=False, exact_assign=True)
            for path in (cb.CPE_FLAG_TC_ALL_ROUNDS, cb.CPE_FLAG_TC_ONE_STAGE, cb.CPE_FLAG_MMA_ASSIGN, 0):
                a = run_gpu(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, cfg.K_max, scores=scores,
                            keep_votes=False, flags=path | cb.CPE_FLAG_NO_PRUNE)
                assert a["count"].min() > 64, a["count"]
                assert a["status"] == 0, hex(a["status"])
                assert a["prune_state"] is None
                assert np.array_equal(a["labels"], b["labels"]), path
                assert a["counters"][:, cb.CPE_CNT_FILTER_PAIRS].min() > 0          # the filter ran (pairs were counted)
                if scores:
                    assert np.array_equal(a["best"].view(np.uint32), b["best"].view(np.uint32))
                    assert np.array_equal(a["second"].view(np.uint32), b["second"].view(np.uint32))


def test_mma_sync_body_as_the_c5_benchmark_instantiates_it():
    """F = 16 binary16, more than 128 peaks, at least 2^20 pixels, no scores: the mma.sync body with 32 k-values per
    axis, 16-byte gathers over the long span and the peak operand re-loaded in chunks (c5's 300 peaks do not fit the
    resident operand) -- against the oracle's assignment of every pixel."""
    cfg = wl.scaled(wl.CONFIGS["c5"], H=1024, W=1024, K=300, bins_w=512, bins_h=512)
    fr = wl.make_frame(cfg, 0)
    emb, fg = fr["emb"], fr["fg"]
    ora = oracle.decode(emb, fg, cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, cfg.K_max)
    assert ora["count"][0] > 246                                   # beyond the resident peak operand
    for mode in ("direct", "graph"):
        gpu = run_gpu(emb, fg, cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, cfg.K_max, 0, False, mode, keep_votes=False,
                      flags=cb.CPE_FLAG_NO_PRUNE)
        compare_front(gpu, ora, cfg.F, cfg.bins_w, cfg.bins_h)
        assert gpu["status"] == 0
        rep = compare_labels(gpu["labels"], None, None, ora["labels"], ora["best"], ora["second"])
        assert gpu["counters"][0, cb.CPE_CNT_FILTER_PAIRS] > 0
    print("c5-like, mma.sync body:", ora["count"].tolist(), rep)


@pytest.mark.parametrize("name,over", [("c2", dict(H=384, W=384, K=90, bins_w=96, bins_h=96)),              # fp32, F = 8
                                       ("c5", dict(H=320, W=352, K=100, bins_w=128, bins_h=128)),           # fp16, F = 16
                                       ("c4", dict(B=2, H=320, W=320, K=70, bins_w=80, bins_h=80))])        # fp16, F = 8
def test_between_65_and_128_peaks_both_tensor_memory_stages_serve_one_tile(name, over):
    cfg = wl.scaled(wl.CONFIGS[name], **over)
    fr = wl.make_frame(cfg, 2)
    gpu, ora, rep = check_case(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, cfg.K_max, mode="graph")
    assert 64 < ora["count"].max() <= 128, ora["count"]
    assert gpu["status"] == 0
    print(name, over, ora["count"].tolist(), rep)


def test_small_max_instances_takes_the_three_kernel_chain():
    """With max_instances inside the all-pairs range no image can need the pruned or the filtered assignment, so neither
    is enqueued: the captured graph has three kernel nodes, results are the oracle's, and replays repeat them
    (the all-pairs kernel then is the one that leaves the vote map zero for the next decode)."""
    import torch
    cfg = wl.scaled(wl.CONFIGS["c2"], H=192, W=256, K=12, bins_w=48, bins_h=32)
    fr = wl.make_frame(cfg, 0)
    check_case(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h, K_max=32, mode="graph")
    ora = oracle.decode(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, 32)
    emb, fg = torch.from_numpy(fr["emb"]).cuda(), torch.from_numpy(fr["fg"]).cuda()
    nodes = {}
    for k_max in (32, 33):
        dec = cb.Decoder(cfg.B, cfg.H, cfg.W, cfg.F, cfg.dtype, cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, k_max)
        stream = torch.cuda.Stream()          # capture needs a stream of its own, not the default one
        torch.cuda.synchronize()
        g = dec.capture(emb, fg, stream=stream)
        nodes[k_max] = cb.cpe_graph_kernel_nodes(g)
        for _ in range(3):
            dec.replay(g, stream=stream)
            torch.cuda.synchronize()
            n = int(ora["count"][0])
            assert int(dec.count.cpu()[0]) == n
            assert np.array_equal(dec.intermediate(cb.CPE_INT_PEAK_CELLS).cpu().numpy()[0, :n], ora["peak_cell"][0, :n])
            lab = dec.labels.cpu().numpy()
            with np.errstate(invalid="ignore"):
                near_tie = (ora["second"] - ora["best"]) < 1e-5
            assert ((lab == ora["labels"]) | near_tie).all()
        dec.close()
    assert nodes[32] == 3 and nodes[33] > nodes[32], nodes


def test_packed_division_of_the_voting_kernel_is_the_ieee_quotient_for_every_binary16_pair():
    """The voting kernel divides binary16-valued operands with a reciprocal estimate and one correction in packed
    binary32; the library's self-test compares it with IEEE division for all 5e8 pairs 0 <= a <= b."""
    import torch
    out = torch.full((1,), 123, dtype=torch.int64, device="cuda")
    rc = cb.cpe_selftest_half_division(torch.cuda.current_stream().cuda_stream, out.data_ptr())
    assert rc == cb.CPE_OK
    torch.cuda.synchronize()
    assert int(out.item()) == 0
