"""cpe_decode_static: the decode for callers that may not allocate device memory (plug-ins inside another
engine's enqueue call, real-time paths, processes with a memory pool fixed at start-up).  It runs on a scratch
array built into the library instead of a caller-provided workspace.  This file is collected last on purpose:
if the entry point misbehaves, every other test has already run.

The check: on the same inputs, through the C ABI, its labels, centroids and counts must equal those of
cpe_decode - bit for bit for the integers, and to the float tolerance the parity tests use for the centroids -
on two calls in a row (the second call finds the scratch as the first left it), and again after a call with
another configuration has used the same scratch in between.  They are also compared with the CPU oracle, and
the device's free memory must be the same before and after the calls (nothing was allocated, nothing freed).
"""
import numpy as np
import pytest

import oracle
from gpu_util import compare_labels
from paper_2609_16874_b200 import binding as cb
from paper_2609_16874_b200 import workloads as wl

pytestmark = pytest.mark.gpu

REL = 1e-4   # the parity tests' tolerance for float outputs


def _decode_both(cfg, frame):
    import torch
    fr = wl.make_frame(cfg, frame)
    emb = torch.from_numpy(fr["emb"]).cuda()
    fg = torch.from_numpy(fr["fg"]).cuda()
    stream = torch.cuda.current_stream()

    ref = cb.Decoder(cfg.B, cfg.H, cfg.W, cfg.F, cfg.dtype, cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, cfg.K_max)
    ref.decode(emb, fg)
    torch.cuda.synchronize()
    want = (ref.labels.cpu().numpy().copy(), ref.centroids.cpu().numpy().copy(), ref.count.cpu().numpy().copy())
    ref.close()

    code = cb.CPE_F32 if cfg.dtype == "f32" else cb.CPE_F16
    params = cb.make_params(code, cfg.bins_w, cfg.bins_h, 0, cfg.T_v, cfg.tau, cfg.K_max, 0)   # no workspace at all
    labels = torch.full((cfg.B, cfg.H, cfg.W), -3, dtype=torch.int32, device="cuda")
    cents = torch.zeros((cfg.B, cfg.K_max, 2), dtype=torch.float32, device="cuda")
    count = torch.full((cfg.B,), -3, dtype=torch.int32, device="cuda")
    outs = []
    torch.cuda.synchronize()
    free_before, reserved_before = torch.cuda.mem_get_info()[0], torch.cuda.memory_reserved()
    for _ in range(2):                                  # two calls in a row on the shared scratch
        labels.fill_(-3)
        count.fill_(-3)
        rc = cb.cpe_decode_static(stream.cuda_stream, emb.data_ptr(), fg.data_ptr(), cfg.B, cfg.H, cfg.W, cfg.F, params,
                                  labels.data_ptr(), cents.data_ptr(), count.data_ptr())
        assert rc == cb.CPE_OK, cb.cpe_strerror(rc)
        torch.cuda.synchronize()
        # no allocation on the device, by the library or through torch, between the calls' start and end
        assert torch.cuda.mem_get_info()[0] == free_before and torch.cuda.memory_reserved() == reserved_before
        outs.append((labels.cpu().numpy().copy(), cents.cpu().numpy().copy(), count.cpu().numpy().copy()))
    ora = oracle.decode(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, cfg.K_max)
    for got in outs:                                    # ... and against the oracle
        assert np.array_equal(got[2], ora["count"])
        compare_labels(got[0], None, None, ora["labels"], ora["best"], ora["second"])
        for b, n in enumerate(ora["count"]):
            np.testing.assert_allclose(got[1][b, :n], ora["centroids"][b, :n], rtol=REL, atol=1e-4)
    return want, outs


def _same(want, got):
    assert np.array_equal(got[2], want[2])                                  # instance counts
    assert np.array_equal(got[0], want[0])                                  # label map, bit for bit
    for b, n in enumerate(want[2]):
        np.testing.assert_allclose(got[1][b, :n], want[1][b, :n], rtol=REL, atol=1e-4)


def test_static_scratch_decode_matches_workspace_decode():
    small = wl.scaled(wl.CONFIGS["c4"], B=2, H=160, W=168, K=30, bins_w=40, bins_h=40)
    other = wl.scaled(wl.CONFIGS["c5"], H=256, W=256, K=40, bins_w=128, bins_h=128)
    for cfg in (small, other, small):          # the third round finds the scratch as another configuration left it
        want, outs = _decode_both(cfg, 0)
        assert want[2].min() >= 1
        _same(want, outs[0])
        _same(want, outs[1])


def test_static_scratch_set_up_is_refused_during_capture_and_a_warm_call_can_be_captured():
    """A call that still has to set the scratch up (first call, or other sizes than the call before) cannot run while
    its stream is being captured: it must return an error and enqueue nothing, leaving the capture valid.  After a
    plain call with the same sizes, the same call inside a capture only enqueues, and replaying the graph decodes."""
    import torch
    cfg = wl.scaled(wl.CONFIGS["c3"], H=128, W=192, K=10, bins_w=48, bins_h=32)
    other = wl.scaled(wl.CONFIGS["c2"], H=96, W=128, K=6, bins_w=24, bins_h=24)
    fr = wl.make_frame(cfg, 0)
    emb, fg = torch.from_numpy(fr["emb"]).cuda(), torch.from_numpy(fr["fg"]).cuda()
    code = cb.CPE_F32 if cfg.dtype == "f32" else cb.CPE_F16
    params = cb.make_params(code, cfg.bins_w, cfg.bins_h, 0, cfg.T_v, cfg.tau, cfg.K_max, 0)
    labels = torch.full((cfg.B, cfg.H, cfg.W), -3, dtype=torch.int32, device="cuda")
    cents = torch.zeros((cfg.B, cfg.K_max, 2), dtype=torch.float32, device="cuda")
    count = torch.full((cfg.B,), -3, dtype=torch.int32, device="cuda")
    args = (emb.data_ptr(), fg.data_ptr(), cfg.B, cfg.H, cfg.W, cfg.F, params, labels.data_ptr(), cents.data_ptr(),
            count.data_ptr())
    # leave the scratch set up for ANOTHER configuration
    fo = wl.make_frame(other, 0)
    eo, go = torch.from_numpy(fo["emb"]).cuda(), torch.from_numpy(fo["fg"]).cuda()
    po = cb.make_params(cb.CPE_F32, other.bins_w, other.bins_h, 0, other.T_v, other.tau, other.K_max, 0)
    lo = torch.empty((other.B, other.H, other.W), dtype=torch.int32, device="cuda")
    co = torch.zeros((other.B, other.K_max, 2), dtype=torch.float32, device="cuda")
    no = torch.zeros((other.B,), dtype=torch.int32, device="cuda")
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        assert cb.cpe_decode_static(s.cuda_stream, eo.data_ptr(), go.data_ptr(), other.B, other.H, other.W, other.F, po,
                                    lo.data_ptr(), co.data_ptr(), no.data_ptr()) == cb.CPE_OK
        s.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            rc_cold = cb.cpe_decode_static(s.cuda_stream, *args)        # needs set-up: refused, capture stays valid
        assert rc_cold == cb.CPE_ERR_PARAM
        assert cb.cpe_decode_static(s.cuda_stream, *args) == cb.CPE_OK  # outside a capture: sets up and decodes
        s.synchronize()
        want = labels.cpu().numpy().copy()
        g2 = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g2, stream=s):
            rc_warm = cb.cpe_decode_static(s.cuda_stream, *args)        # same sizes: only enqueues
        assert rc_warm == cb.CPE_OK
        for _ in range(2):
            labels.fill_(-3)
            g2.replay()
            s.synchronize()
            assert np.array_equal(labels.cpu().numpy(), want)
    ora = oracle.decode(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, cfg.K_max)
    compare_labels(want, None, None, ora["labels"], ora["best"], ora["second"])


def test_static_scratch_limits_are_reported_not_exceeded():
    import torch
    stream = torch.cuda.current_stream().cuda_stream
    fake = 4096
    big = cb.make_params(cb.CPE_F16, 2048, 2048)                         # more bins than the built-in scratch allows
    assert cb.cpe_decode_static(stream, fake, 0, 1, 64, 64, 8, big, fake, fake, fake) == cb.CPE_ERR_STATIC_LIMIT
    huge = cb.make_params(cb.CPE_F16, 1024, 1024, max_instances=1 << 16)  # peak arrays larger than the scratch
    assert cb.cpe_decode_static(stream, fake, 0, 8, 64, 64, 16, huge, fake, fake, fake) == cb.CPE_ERR_STATIC_LIMIT
    scores = cb.make_params(cb.CPE_F16, 32, 32, flags=cb.CPE_FLAG_WRITE_SCORES)
    assert cb.cpe_decode_static(stream, fake, 0, 1, 64, 64, 8, scores, fake, fake, fake) == cb.CPE_ERR_STATIC_LIMIT
    assert "scratch" in cb.cpe_strerror(cb.CPE_ERR_STATIC_LIMIT)
