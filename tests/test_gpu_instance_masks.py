"""Per-instance outputs (Sec. 3.2, Eq. 8): mask planes and pixel counters, CUDA vs oracle, bit-exact.  Needs a B200."""
import numpy as np
import pytest

import oracle
from paper_2609_16874_b200 import binding as cb
from paper_2609_16874_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def run_case(emb, fg, bins_w, bins_h, n_planes, tau=np.inf):
    import torch
    B, D, H, W = emb.shape
    dec = cb.Decoder(B, H, W, D // 4, "f32" if emb.dtype == np.float32 else "f16", bins_w, bins_h, 8, float(tau), 1024)
    d_emb = torch.from_numpy(emb).cuda()
    d_fg = None if fg is None else torch.from_numpy(np.ascontiguousarray(fg, np.uint8)).cuda()
    dec.decode(d_emb, d_fg)
    planes, pixels = dec.instance_masks(n_planes)
    _, pixels_only = dec.instance_masks(n_planes, want_planes=False)
    torch.cuda.synchronize()
    labels = dec.labels.cpu().numpy()
    count = dec.count.cpu().numpy()
    got = planes.cpu().numpy(), pixels.cpu().numpy().view(np.uint32), pixels_only.cpu().numpy().view(np.uint32)
    dec.close()
    want_planes, want_pixels = oracle.instance_masks(labels, n_planes)
    assert np.array_equal(got[0], want_planes)
    assert np.array_equal(got[1], want_pixels)
    assert np.array_equal(got[2], want_pixels)
    return labels, count, want_pixels


@pytest.mark.parametrize("name,over,n_planes", [
    ("c1", dict(), 8),                                          # vector path
    ("c2", dict(H=131, W=77, K=6, bins_w=48, bins_h=40), 7),    # odd sizes: scalar path with a ragged tail
    ("c4", dict(B=3, H=160, W=168, K=30, bins_w=40, bins_h=40), 40),
])
def test_planes_and_counters_match(name, over, n_planes):
    cfg = wl.scaled(wl.CONFIGS[name], **over)
    fr = wl.make_frame(cfg, 0)
    labels, count, pixels = run_case(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h, n_planes)
    assert count.min() >= 1 and pixels.sum() > 0
    # every labelled pixel is in exactly one of the planes asked for (all instances fit here)
    assert int(pixels.sum()) == int((labels > 0).sum())


def test_tau_rejection_without_a_mask_gives_the_implicit_background():
    """fg_mask = NULL and a finite tau (Eq. 8): pixels far from every candidate centroid get no mask; the counters
    shrink accordingly and still match the label map."""
    cfg = wl.scaled(wl.CONFIGS["c1"], H=96, W=128)
    fr = wl.make_frame(cfg, 0)
    lab_inf, cnt, pix_inf = run_case(fr["emb"], None, cfg.bins_w, cfg.bins_h, 256)
    lab_tau, _, pix_tau = run_case(fr["emb"], None, cfg.bins_w, cfg.bins_h, 256, tau=1.5)
    assert cnt.max() <= 256
    assert (lab_inf > 0).all()                    # without tau every pixel of a maskless decode is assigned
    assert 0 < (lab_tau > 0).sum() < lab_tau.size
    assert (pix_tau <= pix_inf).all() and pix_tau.sum() == (lab_tau > 0).sum()
    # background pixels (zero embedding + noise) are the ones that lose their label
    bg = fr["fg"][0] == 0
    assert (lab_tau[0][bg] == 0).mean() > 0.9
