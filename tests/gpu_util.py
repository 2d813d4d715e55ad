"""Helpers of the GPU parity tests: run the CUDA path through the binding, run the oracle, compare."""
import numpy as np

import oracle
from paper_2609_16874_b200 import binding as cb

MARGIN = 1e-5      # label differences are excused where the oracle's top-2 distance margin is below this
REL = 1e-4         # relative tolerance of float scores and centroids


def run_gpu(emb, fg, bins_w, bins_h, T_v=8, tau=np.inf, K_max=1024, levels=0, scores=True, mode="direct",
            exact_assign=False, keep_votes=True, filter_assign=False, refine=False, flags=0):
    import torch
    B, D, H, W = emb.shape
    F = D // 4
    dtype = "f32" if emb.dtype == np.float32 else "f16"
    dec = cb.Decoder(B, H, W, F, dtype, bins_w, bins_h, T_v, float(tau), K_max, levels, write_scores=scores,
                     exact_assign=exact_assign, keep_votes=keep_votes, filter_assign=filter_assign, refine=refine,
                     flags=flags)
    d_emb = torch.from_numpy(emb).cuda()
    d_fg = None if fg is None else torch.from_numpy(np.ascontiguousarray(fg, np.uint8)).cuda()
    if mode == "direct":
        dec.decode(d_emb, d_fg)
    else:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        g = dec.capture(d_emb, d_fg, stream=side)
        dec.labels.fill_(-7)
        dec.replay(g, stream=side)
        dec.replay(g, stream=side)     # a second replay must give the same result (state is re-zeroed)
        side.synchronize()
    torch.cuda.synchronize()
    out = {
        "labels": dec.labels.cpu().numpy(),
        "centroids": dec.centroids.cpu().numpy(),
        "count": dec.count.cpu().numpy(),
        "votes": dec.intermediate(cb.CPE_INT_VOTES).cpu().numpy().view(np.uint32) if keep_votes else None,
        "peak_cell": dec.intermediate(cb.CPE_INT_PEAK_CELLS).cpu().numpy(),
        "peak_votes": dec.intermediate(cb.CPE_INT_PEAK_VOTES).cpu().numpy().view(np.uint32),
        "peak_emb": dec.intermediate(cb.CPE_INT_PEAK_EMB).cpu().numpy(),
        "pal_w": dec.intermediate(cb.CPE_INT_PALETTE_W).cpu().numpy(),
        "pal_h": dec.intermediate(cb.CPE_INT_PALETTE_H).cpu().numpy(),
        "status": int(np.bitwise_or.reduce(dec.intermediate(cb.CPE_INT_STATUS).cpu().numpy())),
        "counters": dec.intermediate(cb.CPE_INT_COUNTERS).cpu().numpy().astype(np.int64),
    }
    rc, _, _ = cb.cpe_get_intermediate(dec.params, cb.CPE_INT_PRUNE_STATE, B, H, W, F)
    out["prune_state"] = (dec.intermediate(cb.CPE_INT_PRUNE_STATE).cpu().numpy().astype(np.int64)
                          if rc == cb.CPE_OK else None)
    if scores:
        out["best"] = dec.intermediate(cb.CPE_INT_BEST_SCORE).cpu().numpy()
        out["second"] = dec.intermediate(cb.CPE_INT_SECOND_SCORE).cpu().numpy()
    dec.close()
    return out


def compare_front(gpu, ora, F, bins_w, bins_h):
    """Palettes, votes, peak list, counts, centroids, counters: bit-exact except the float centroids."""
    assert np.array_equal(gpu["pal_w"].view(np.uint32), oracle.palette(bins_w, F).view(np.uint32))
    assert np.array_equal(gpu["pal_h"].view(np.uint32), oracle.palette(bins_h, F).view(np.uint32))
    assert not (gpu["status"] & cb.CPE_STATUS_INTERNAL), hex(gpu["status"])      # no index self-check fired
    if gpu["votes"] is not None:
        assert np.array_equal(gpu["votes"], ora["votes"]), "vote map differs"
    assert np.array_equal(gpu["count"], ora["count"]), (gpu["count"], ora["count"])
    Pw, Ph = oracle.palette(bins_w, F), oracle.palette(bins_h, F)
    for b in range(len(ora["count"])):
        n = int(ora["count"][b])
        assert np.array_equal(gpu["peak_cell"][b, :n], ora["peak_cell"][b, :n])
        assert np.array_equal(gpu["peak_votes"][b, :n], ora["peak_votes"][b, :n])
        np.testing.assert_allclose(gpu["centroids"][b, :n], ora["centroids"][b, :n], rtol=REL, atol=1e-4)
        cells = ora["peak_cell"][b, :n]
        want = np.concatenate([Pw[cells % bins_w], Ph[cells // bins_w]], 1)
        assert np.array_equal(gpu["peak_emb"][b, :n].view(np.uint32), want.view(np.uint32))
    for c in (cb.CPE_CNT_VOTING, cb.CPE_CNT_NONFINITE, cb.CPE_CNT_RAW_PEAKS, cb.CPE_CNT_TRUNCATED):
        assert np.array_equal(gpu["counters"][:, c], ora["counters"][:, c]), c


def compare_labels(g_lab, g_best, g_second, o_lab, o_best, o_second):
    """Labels bit-exact except near-ties (counted); scores within REL.  Arrays of equal shape."""
    with np.errstate(invalid="ignore"):
        margin = o_second - o_best          # inf - inf (no peak at all) gives nan: never excused, never needed
    diff = g_lab != o_lab
    excused = diff & (margin < MARGIN)
    bad = diff & ~excused
    assert not bad.any(), f"{int(bad.sum())} label mismatches outside near-ties, e.g. index {np.argwhere(bad)[:5].tolist()}"
    if g_best is not None:
        fin = np.isfinite(o_best)
        assert np.array_equal(np.isfinite(g_best), fin)
        np.testing.assert_allclose(g_best[fin], o_best[fin], rtol=REL, atol=1e-6)
        fin2 = np.isfinite(o_second)
        assert np.array_equal(np.isfinite(g_second), fin2)
        np.testing.assert_allclose(g_second[fin2], o_second[fin2], rtol=REL, atol=1e-6)
    return {"near_tie_pixels": int((margin < MARGIN).sum()), "excused_mismatches": int(excused.sum())}


def check_case(emb, fg, bins_w, bins_h, T_v=8, tau=np.inf, K_max=1024, levels=0, mode="direct"):
    F = emb.shape[1] // 4
    gpu = run_gpu(emb, fg, bins_w, bins_h, T_v, tau, K_max, levels, True, mode)
    ora = oracle.decode(emb, fg, bins_w, bins_h, T_v, tau, K_max, levels)
    compare_front(gpu, ora, F, bins_w, bins_h)
    rep = compare_labels(gpu["labels"], gpu["best"], gpu["second"], ora["labels"], ora["best"], ora["second"])
    if rep["excused_mismatches"] == 0:
        assert np.array_equal(gpu["counters"][:, cb.CPE_CNT_TAU_REJECTED], ora["counters"][:, oracle.CNT_TAU_REJECTED])
    # the production configuration: no score output (the filter may then decide a pixel without re-scoring it)
    fast = run_gpu(emb, fg, bins_w, bins_h, T_v, tau, K_max, levels, False, mode, keep_votes=False)
    compare_front(fast, ora, F, bins_w, bins_h)
    rep2 = compare_labels(fast["labels"], None, None, ora["labels"], ora["best"], ora["second"])
    rep["excused_mismatches_no_scores"] = rep2["excused_mismatches"]
    # the tensor-core filtered kernel forced on, with and without scores (images with few peaks would
    # otherwise take the all-pairs kernel)
    for sc in (True, False):
        filt = run_gpu(emb, fg, bins_w, bins_h, T_v, tau, K_max, levels, sc, mode, keep_votes=False, filter_assign=True)
        compare_front(filt, ora, F, bins_w, bins_h)
        compare_labels(filt["labels"], filt.get("best"), filt.get("second"), ora["labels"], ora["best"], ora["second"])
        if sc:   # both kernels compute the same binary32 scores
            assert np.array_equal(filt["best"].view(np.uint32), gpu["best"].view(np.uint32))
            assert np.array_equal(filt["second"].view(np.uint32), gpu["second"].view(np.uint32))
    return gpu, ora, rep
