"""A bounded device-side wait that runs out: the kernel must wind down and return, report CPE_STATUS_TIMEOUT, and
leave the workspace usable.  Needs a B200.

Nothing here hangs or faults a GPU: the test flag makes the producer warps of the tensor-memory assignment withhold
one mbarrier arrival, the consumers' wait gives up after its iteration limit (a fraction of a second), every role
sees the abort flag, tensor memory is returned and the kernel ends normally."""
import numpy as np
import pytest

import oracle
from paper_2609_16874_b200 import binding as cb
from paper_2609_16874_b200 import workloads as wl

from gpu_util import compare_labels

pytestmark = pytest.mark.gpu


def test_a_stalled_pipeline_times_out_returns_and_the_next_decode_is_exact():
    import torch
    cfg = wl.scaled(wl.CONFIGS["c4"], B=2, H=320, W=384, K=100)       # 65..128 peaks: the tensor-memory body
    fr = wl.make_frame(cfg, 0)
    ora = oracle.decode(fr["emb"], fr["fg"], cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, cfg.K_max)
    assert 32 < ora["count"].min() and ora["count"].max() <= 128
    emb, fg = torch.from_numpy(fr["emb"]).cuda(), torch.from_numpy(fr["fg"]).cuda()
    dec = cb.Decoder(cfg.B, cfg.H, cfg.W, cfg.F, cfg.dtype, cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, cfg.K_max,
                     flags=cb.CPE_FLAG_NO_PRUNE | cb.CPE_FLAG_TEST_STALL)
    dec.decode(emb, fg)
    torch.cuda.synchronize()                                          # returns: nothing hangs
    status = dec.intermediate(cb.CPE_INT_STATUS).cpu().numpy()
    assert (status & cb.CPE_STATUS_TIMEOUT).all(), status
    assert not (status & cb.CPE_STATUS_INTERNAL).any(), status
    assert np.array_equal(dec.count.cpu().numpy(), ora["count"])      # the stages before the stalled one are complete
    # the same workspace, without the stall: exact results, status clear
    dec.params.flags &= ~cb.CPE_FLAG_TEST_STALL
    for _ in range(2):
        dec.labels.fill_(-5)
        dec.decode(emb, fg)
        torch.cuda.synchronize()
        assert int(np.bitwise_or.reduce(dec.intermediate(cb.CPE_INT_STATUS).cpu().numpy())) == 0
        assert np.array_equal(dec.count.cpu().numpy(), ora["count"])
        compare_labels(dec.labels.cpu().numpy(), None, None, ora["labels"], ora["best"], ora["second"])
    dec.close()
