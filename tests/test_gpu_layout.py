"""Channels-last input (the paper's H x W x 4L notation): conversion to planes, bit-exact, and the decode of a converted
input equals the decode of the planar one.  Needs a B200."""
import numpy as np
import pytest

from paper_2609_16874_b200 import binding as cb
from paper_2609_16874_b200 import workloads as wl

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("shape,dtype", [((2, 12, 37, 53), np.float32), ((1, 64, 64, 96), np.float16),
                                         ((3, 4, 1, 7), np.float16), ((1, 20, 130, 64), np.float32),
                                         # aligned, whole tiles, power-of-two channel units: the unit-wise kernels
                                         ((2, 32, 64, 64), np.float32), ((1, 32, 32, 64), np.float16),
                                         ((2, 8, 16, 64), np.float16), ((1, 16, 8, 48), np.float32),
                                         ((1, 64, 32, 32), np.float32), ((2, 16, 48, 32), np.float16),
                                         ((1, 4, 16, 16), np.float32)])
def test_conversion_is_a_transpose(shape, dtype):
    import torch
    B, D, H, W = shape
    rng = np.random.default_rng(1)
    planar = rng.standard_normal(shape).astype(dtype)
    planar.reshape(-1)[::97] = np.inf                       # bit patterns are moved, not interpreted
    nhwc = np.ascontiguousarray(planar.transpose(0, 2, 3, 1))
    src = torch.from_numpy(nhwc).cuda()
    dst = torch.empty(shape, dtype=src.dtype, device="cuda")
    rc = cb.cpe_channels_last_to_planar(torch.cuda.current_stream().cuda_stream, src.data_ptr(), dst.data_ptr(), B, H, W,
                                        D // 4, cb.CPE_F32 if dtype == np.float32 else cb.CPE_F16)
    assert rc == 0
    torch.cuda.synchronize()
    u = np.uint32 if dtype == np.float32 else np.uint16
    assert np.array_equal(dst.cpu().numpy().view(u), planar.view(u))


def test_decode_of_a_converted_input_equals_the_planar_decode():
    import torch
    cfg = wl.scaled(wl.CONFIGS["c3"], H=128, W=192, K=10, bins_w=64, bins_h=48)
    fr = wl.make_frame(cfg, 0)
    emb, fg = torch.from_numpy(fr["emb"]).cuda(), torch.from_numpy(fr["fg"]).cuda()
    nhwc = emb.permute(0, 2, 3, 1).contiguous()
    back = torch.empty_like(emb)
    assert cb.cpe_channels_last_to_planar(torch.cuda.current_stream().cuda_stream, nhwc.data_ptr(), back.data_ptr(), cfg.B,
                                          cfg.H, cfg.W, cfg.F, cb.CPE_F16) == 0
    dec = cb.Decoder(cfg.B, cfg.H, cfg.W, cfg.F, cfg.dtype, cfg.bins_w, cfg.bins_h, cfg.T_v, cfg.tau, cfg.K_max)
    dec.decode(emb, fg)
    torch.cuda.synchronize()
    a = dec.labels.cpu().numpy().copy(), dec.count.cpu().numpy().copy()
    dec.decode(back, fg)
    torch.cuda.synchronize()
    assert np.array_equal(a[0], dec.labels.cpu().numpy()) and np.array_equal(a[1], dec.count.cpu().numpy())
    dec.close()


def test_conversion_rejects_bad_arguments():
    assert cb.cpe_channels_last_to_planar(0, 0, 0, 1, 8, 8, 4, cb.CPE_F32) == cb.CPE_ERR_NULL
    assert cb.cpe_channels_last_to_planar(0, 256, 512, 1, 8, 8, 17, cb.CPE_F32) == cb.CPE_ERR_SIZE
    assert cb.cpe_channels_last_to_planar(0, 256, 512, 1, 8, 8, 4, 7) == cb.CPE_ERR_DTYPE
    assert cb.cpe_channels_last_to_planar(0, 258, 512, 1, 8, 8, 4, cb.CPE_F32) == cb.CPE_ERR_ALIGN
