"""Sub-cell refined centroids (CPE_FLAG_REFINE): CUDA path vs CPU oracle through the C ABI.  Needs a B200.

Integer work (votes, per-bin fixed-point sums, peak list, counts) must agree bit for bit; so must the refined
centroids, which both sides derive from the same integers with the same correctly rounded binary64 operations.
The refined candidate embeddings go through sin/cos of different libraries: one unit in the last place of
binary32.  Labels and scores follow the usual rule (exact except where the oracle's top-2 margin is a near-tie).
"""
import numpy as np
import pytest

import oracle
from paper_2609_16874_b200 import binding as cb
from paper_2609_16874_b200 import workloads as wl

from gpu_util import REL, compare_labels, run_gpu

pytestmark = pytest.mark.gpu

EMB_ATOL = 1.5e-7     # |sin|, |cos| <= 1: one binary32 ulp below 1 is 6e-8, two libraries may round apart by one


def run_refined(emb, fg, bins_w, bins_h, T_v=8, tau=np.inf, K_max=1024, scores=True, mode="direct", **flags):
    import torch
    B, D, H, W = emb.shape
    F = D // 4
    dec = cb.Decoder(B, H, W, F, "f32" if emb.dtype == np.float32 else "f16", bins_w, bins_h, T_v, float(tau), K_max,
                     0, write_scores=scores, keep_votes=True, refine=True, **flags)
    d_emb = torch.from_numpy(emb).cuda()
    d_fg = None if fg is None else torch.from_numpy(np.ascontiguousarray(fg, np.uint8)).cuda()
    if mode == "direct":
        dec.decode(d_emb, d_fg)
        dec.decode(d_emb, d_fg)        # the sums are cleared at the start of every decode
    else:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        g = dec.capture(d_emb, d_fg, stream=side)
        dec.labels.fill_(-7)
        dec.replay(g, stream=side)
        dec.replay(g, stream=side)
        side.synchronize()
    torch.cuda.synchronize()
    out = {
        "labels": dec.labels.cpu().numpy(),
        "centroids": dec.centroids.cpu().numpy(),
        "count": dec.count.cpu().numpy(),
        "votes": dec.intermediate(cb.CPE_INT_VOTES).cpu().numpy().view(np.uint32),
        "sums": dec.intermediate(cb.CPE_INT_VOTE_SUMS).cpu().numpy(),
        "peak_cell": dec.intermediate(cb.CPE_INT_PEAK_CELLS).cpu().numpy(),
        "peak_emb": dec.intermediate(cb.CPE_INT_PEAK_EMB).cpu().numpy(),
        "status": int(np.bitwise_or.reduce(dec.intermediate(cb.CPE_INT_STATUS).cpu().numpy())),
        "counters": dec.intermediate(cb.CPE_INT_COUNTERS).cpu().numpy().astype(np.int64),
    }
    if scores:
        out["best"] = dec.intermediate(cb.CPE_INT_BEST_SCORE).cpu().numpy()
        out["second"] = dec.intermediate(cb.CPE_INT_SECOND_SCORE).cpu().numpy()
    dec.close()
    return out


def compare_refined(gpu, ora):
    assert not (gpu["status"] & cb.CPE_STATUS_INTERNAL), hex(gpu["status"])
    assert np.array_equal(gpu["votes"], ora["votes"]), "vote map differs"
    assert np.array_equal(gpu["sums"], ora["sums"]), "per-bin sums differ"
    assert np.array_equal(gpu["count"], ora["count"])
    for b in range(len(ora["count"])):
        n = int(ora["count"][b])
        assert np.array_equal(gpu["peak_cell"][b, :n], ora["peak_cell"][b, :n])
        assert np.array_equal(gpu["centroids"][b, :n].view(np.uint32), ora["centroids"][b, :n].view(np.uint32))
        np.testing.assert_allclose(gpu["peak_emb"][b, :n], ora["peak_emb"][b, :n], rtol=0, atol=EMB_ATOL)
    for c in (cb.CPE_CNT_VOTING, cb.CPE_CNT_NONFINITE, cb.CPE_CNT_RAW_PEAKS, cb.CPE_CNT_TRUNCATED):
        assert np.array_equal(gpu["counters"][:, c], ora["counters"][:, c]), c
    return compare_labels(gpu["labels"], gpu.get("best"), gpu.get("second"), ora["labels"], ora["best"],
                          ora["second"])


CASES = [
    ("c1", dict()),                                                        # vector-load vote kernel, fp32
    ("c1", dict(H=67, W=93)),                                              # scalar-load vote kernel
    ("c2", dict(H=192, W=256, K=12)),
    ("c3", dict(H=256, W=384, K=24, bins_w=96, bins_h=64)),                # fp16
    ("c3", dict(H=99, W=121, K=8, bins_w=64, bins_h=32)),                  # fp16, scalar path
    ("c4", dict(B=3, H=160, W=168, K=30, bins_w=40, bins_h=40)),           # batch, touching instances
    ("c5", dict(H=256, W=256, K=40, bins_w=128, bins_h=128)),              # F = 16
]


@pytest.mark.parametrize("name,over", CASES, ids=[f"{n}-{i}" for i, (n, _) in enumerate(CASES)])
@pytest.mark.parametrize("mode", ["direct", "graph"])
def test_refined_decode_matches_oracle(name, over, mode):
    cfg = wl.scaled(wl.CONFIGS[name], **over)
    fr = wl.make_frame(cfg, 0)
    ora = oracle.decode_refined(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, cfg.K_max)
    assert ora["count"].min() >= 1
    gpu = run_refined(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, cfg.K_max, mode=mode)
    rep = compare_refined(gpu, ora)
    # production configuration (no scores) and the tensor-core filtered kernel forced on
    fast = run_refined(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, cfg.K_max, scores=False, mode=mode)
    compare_refined(fast, ora)
    for sc in (True, False):
        filt = run_refined(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, cfg.K_max, scores=sc,
                           mode=mode, filter_assign=True)
        compare_refined(filt, ora)
    print(name, over, rep)


def test_refined_centroids_are_closer_to_the_truth_than_bin_centres():
    # what the mode is for: on the noisy c2 recipe the refined centroid is well inside a bin width of the instance's
    # true centroid, and the pixels' distances to their candidate drop
    cfg = wl.scaled(wl.CONFIGS["c2"], H=256, W=256, K=10)
    fr = wl.make_frame(cfg, 4)
    gpu = run_refined(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, cfg.K_max)
    plain = oracle.decode(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, cfg.K_max)
    n = int(gpu["count"][0])
    assert n == int(plain["count"][0]) >= 1
    truth = fr["centroids"][0]                                   # [K, 2] in [-1, 1)
    truth_px = np.stack([((truth[:, 0] + 1) * cfg.W - 1) / 2, ((truth[:, 1] + 1) * cfg.H - 1) / 2], 1)

    def err(cent):
        d = np.linalg.norm(cent[:, None, :] - truth_px[None], axis=2)
        return np.nanmin(d, axis=1)
    e_ref, e_bin = err(gpu["centroids"][0, :n]), err(plain["centroids"][0, :n])
    assert np.median(e_ref) < 0.5 * np.median(e_bin)
    fgm = fr["fg"][0] > 0
    assert np.median(gpu["best"][0][fgm]) < np.median(plain["best"][0][fgm])


def test_refine_intermediate_needs_the_flag_and_workspace_grows_by_the_sums():
    # (without the pruned assignment, which keeps the sums for its own use in either mode)
    p0 = cb.make_params(cb.CPE_F32, 64, 48, 0, 8, float("inf"), 128, cb.CPE_FLAG_NO_PRUNE)
    p1 = cb.make_params(cb.CPE_F32, 64, 48, 0, 8, float("inf"), 128, cb.CPE_FLAG_REFINE | cb.CPE_FLAG_NO_PRUNE)
    n0, n1 = cb.cpe_workspace_size(2, 96, 128, 4, p0), cb.cpe_workspace_size(2, 96, 128, 4, p1)
    assert n1 - n0 == 16 * 64 * 48 * 2
    import torch
    ws = torch.empty(n0, dtype=torch.uint8, device="cuda")
    p0.workspace, p0.workspace_bytes = ws.data_ptr(), n0
    rc, _, _ = cb.cpe_get_intermediate(p0, cb.CPE_INT_VOTE_SUMS, 2, 96, 128, 4)
    assert rc == cb.CPE_ERR_WHICH


@pytest.mark.parametrize("name", ["c2", "c3", "c4", "c5"])
def test_refined_full_size_configs(name):
    """Full-size inputs, graph replay as the benchmark runs it: votes, per-bin sums, peak list, refined centroids and
    candidate embeddings against the full oracle; labels and scores on sampled pixels; label-map properties on all."""
    cfg = wl.CONFIGS[name]
    fr = wl.make_frame(cfg, 0)
    emb, fg = fr["emb"], fr["fg"]
    gpu = run_refined(emb, fg, cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, cfg.K_max, mode="graph")
    ov = oracle.votes(emb, fg, cfg.bins_w, cfg.bins_h, want_est=True, want_cell=True)
    sums = oracle.vote_sums(ov["est"], ov["cell"], cfg.bins_w, cfg.bins_h)
    assert np.array_equal(gpu["votes"], ov["votes"])
    assert np.array_equal(gpu["sums"], sums)
    rng = np.random.default_rng(7)
    n_sample = {"c2": 60000, "c3": 40000, "c4": 8000, "c5": 12000}[name]
    for b in range(cfg.B):
        cells, _, raw = oracle.peaks(ov["votes"][b], cfg.T_v, cfg.K_max)
        n = len(cells)
        assert gpu["count"][b] == n and np.array_equal(gpu["peak_cell"][b, :n], cells)
        r = oracle.refined_peaks(ov["votes"][b], sums[b], cells, cfg.F, cfg.H, cfg.W)
        assert np.array_equal(gpu["centroids"][b, :n].view(np.uint32), r["centroids"].view(np.uint32))
        np.testing.assert_allclose(gpu["peak_emb"][b, :n], r["peak_emb"], rtol=0, atol=EMB_ATOL)
        idx = np.sort(rng.choice(cfg.H * cfg.W, n_sample, replace=False)).astype(np.int64)
        res = oracle.assign_image(emb[b], fg[b], cfg.bins_w, cfg.bins_h, cells, cfg.tau, idx=idx, peak_emb=r["peak_emb"])
        rep = compare_labels(gpu["labels"][b].ravel()[idx], gpu["best"][b].ravel()[idx], gpu["second"][b].ravel()[idx],
                             res["labels"], res["best"], res["second"])
        lab = gpu["labels"][b]
        assert ((lab > 0) == (fg[b] > 0)).all() and lab.max() <= n
        print(name, "peaks", n, rep)
    assert gpu["status"] == 0
    # the configuration the benchmark times (no scores, vote map and sums re-zeroed on the device, graph replay) against
    # the oracle's assignment of EVERY pixel
    fast = run_gpu(emb, fg, cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, cfg.K_max, 0, False, "graph", keep_votes=False,
                   refine=True)
    assert fast["status"] == 0 and np.array_equal(fast["count"], gpu["count"])
    oracle.set_threads(oracle.max_threads())
    for b in range(cfg.B):
        cells, _, raw = oracle.peaks(ov["votes"][b], cfg.T_v, cfg.K_max)
        r = oracle.refined_peaks(ov["votes"][b], sums[b], cells, cfg.F, cfg.H, cfg.W)
        res = oracle.assign_image(emb[b], fg[b], cfg.bins_w, cfg.bins_h, cells, cfg.tau, peak_emb=r["peak_emb"])
        rep = compare_labels(fast["labels"][b], None, None, res["labels"], res["best"], res["second"])
    handed = None if fast["prune_state"] is None else fast["prune_state"][:, 2].tolist()
    pairs = fast["counters"][:, cb.CPE_CNT_FILTER_PAIRS].sum() / max(1, fast["counters"][:, cb.CPE_CNT_VOTING].sum())
    print(f"{name} refined (no scores, every pixel): {rep}, handed on {handed}, scored pairs per voting pixel {pairs:.2f}")


def test_refined_edge_cases_empty_truncated_nonfinite_and_border_peaks():
    # no foreground: no votes, zero sums, no peaks, all labels 0
    cfg = wl.scaled(wl.CONFIGS["c3"], H=64, W=128, K=4, bins_w=32, bins_h=16)
    fr = wl.make_frame(cfg, 0)
    fg0 = np.zeros_like(fr["fg"])
    gpu = run_refined(fr["emb"], fg0, cfg.bins_w, cfg.bins_h)
    assert gpu["count"][0] == 0 and (gpu["labels"] == 0).all() and not gpu["sums"].any() and not gpu["votes"].any()

    # more peaks than K_max: the first K_max in bin order are kept and refined; non-finite pixels neither vote nor add
    cfg = wl.scaled(wl.CONFIGS["c4"], B=2, H=96, W=112, K=12, bins_w=28, bins_h=24)
    fr = wl.make_frame(cfg, 1)
    emb = fr["emb"].copy()
    ys, xs = np.nonzero(fr["fg"][1])
    emb[1, 3, ys[::17], xs[::17]] = np.nan
    emb[1, 20, ys[5::29], xs[5::29]] = np.inf
    ora = oracle.decode_refined(emb, fr["fg"], cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, K_max=5)
    assert ora["counters"][:, oracle.CNT_TRUNCATED].min() > 0 and ora["counters"][1, oracle.CNT_NONFINITE] > 0
    gpu = run_refined(emb, fr["fg"], cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, K_max=5)
    compare_refined(gpu, ora)
    assert gpu["status"] & cb.CPE_STATUS_PEAK_OVERFLOW and gpu["status"] & cb.CPE_STATUS_NONFINITE

    # instances whose centroids sit in the border bins (clipped 3x3 windows, estimates near -1 and +1)
    H, W, F, bw, bh = 64, 96, 4, 16, 12
    inst = np.zeros((H, W), np.int32)
    inst[:30, :40], inst[:30, 56:], inst[34:, :40], inst[34:, 56:] = 1, 2, 3, 4
    cents = np.array([[-0.93, -0.90], [0.94, -0.91], [-0.95, 0.92], [0.96, 0.93]])
    emb = wl.encode(inst, cents, F, 0.02, np.random.default_rng(5), np.float32)[None]
    fg = (inst > 0).astype(np.uint8)[None]
    ora = oracle.decode_refined(emb, fg, bw, bh, T_v=8, K_max=8)
    assert ora["count"][0] == 4
    cells = ora["peak_cell"][0, :4]
    assert set((cells % bw).tolist()) <= {0, bw - 1} and set((cells // bw).tolist()) <= {0, bh - 1}
    gpu = run_refined(emb, fg, bw, bh, T_v=8, K_max=8)
    compare_refined(gpu, ora)


FUSE_CASES = [
    ("c1", dict()),                                                        # vector-load vote kernel, fp32
    ("c1", dict(H=67, W=93)),                                              # scalar-load vote kernel
    ("c2", dict(H=192, W=256, K=12)),
    ("c3", dict(H=99, W=121, K=8, bins_w=64, bins_h=32)),                  # fp16, scalar path
    ("c4", dict(B=3, H=160, W=168, K=30, bins_w=40, bins_h=40)),           # batch: one ticket per image
    ("c5", dict(H=256, W=256, K=40, bins_w=96, bins_h=80)),                # F = 16, 7680 bins
]


@pytest.mark.parametrize("name,over", FUSE_CASES, ids=[f"{n}-{i}" for i, (n, _) in enumerate(FUSE_CASES)])
@pytest.mark.parametrize("mode", ["direct", "graph"])
def test_peak_search_inside_the_voting_kernel_gives_the_same_decode(name, over, mode):
    """CPE_FLAG_FUSE_PEAKS: the last voting CTA of an image runs stage 3.  Refined and plain decodes against the oracle,
    twice in a row (the ticket and the accumulators must be left zero), with an image without participating pixels."""
    from gpu_util import compare_front, run_gpu
    cfg = wl.scaled(wl.CONFIGS[name], **over)
    fr = wl.make_frame(cfg, 1)
    emb, fg = fr["emb"], fr["fg"].copy()
    if cfg.B > 1:
        fg[1] = 0
    ora = oracle.decode_refined(emb, fg, cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, cfg.K_max)
    gpu = run_refined(emb, fg, cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, cfg.K_max, mode=mode, flags=cb.CPE_FLAG_FUSE_PEAKS)
    compare_refined(gpu, ora)
    plain = oracle.decode(emb, fg, cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, cfg.K_max)
    for keep in (True, False):
        g = run_gpu(emb, fg, cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, cfg.K_max, 0, True, mode, keep_votes=keep,
                    flags=cb.CPE_FLAG_FUSE_PEAKS)
        compare_front(g, plain, cfg.F, cfg.bins_w, cfg.bins_h)
        compare_labels(g["labels"], g["best"], g["second"], plain["labels"], plain["best"], plain["second"])
