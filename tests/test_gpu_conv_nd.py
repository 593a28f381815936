"""GPU parity of the convolutions with a depth dimension and channel groups (3-D convolution,
Sec. 4.4; depth-wise convolution, Sec. 4.2) against the CPU oracle: accumulators bit-exact,
de-quantized outputs within rel 1e-5 of max|value|; and the 5-D gradient through the gradient
quantizer as (N, C, Do*P, Q)."""
import numpy as np
import pytest
import torch

from oracle import cpu as O
from paper_2102_04782_b200 import api, synth

from helpers import scalar
from test_gpu_gvq import check_grad_quant

pytestmark = pytest.mark.gpu

GEOMS = [
    # N, Cin, Cout, D, H, W, T, R, S, stride, pad, groups
    (2, 16, 24, 6, 9, 10, 3, 3, 3, 1, 1, 1),                  # 3-D convolution, channel words (dp4a)
    (1, 3, 8, 5, 12, 11, 3, 3, 3, (1, 2, 2), (1, 1, 1), 1),   # three input channels, strided in the plane
    (2, 20, 12, 4, 7, 7, 2, 3, 3, (2, 1, 1), (0, 1, 1), 1),   # even depth filter, depth stride 2
    (2, 32, 32, 1, 14, 15, 1, 3, 3, 1, 1, 32),                # depth-wise 2-D
    (2, 24, 24, 1, 16, 16, 1, 3, 3, 2, 1, 24),                # depth-wise, stride 2 (MobileNetV2's down-sampling blocks)
    (1, 16, 32, 3, 8, 8, 3, 3, 3, 1, 1, 4),                   # grouped 3-D convolution
    (2, 8, 8, 4, 6, 6, 3, 3, 3, 1, 1, 8),                     # depth-wise 3-D
]


def rand_codes(rng, shape):
    return rng.integers(-127, 128, size=shape, dtype=np.int64).astype(np.int8)


def act_dev(q):
    """(N,C,D,H,W) codes -> device [N][D][H][W][Cp]."""
    N, C, D, H, W = q.shape
    Cp = (C + 15) // 16 * 16
    out = np.zeros((N, D, H, W, Cp), np.int8)
    out[..., :C] = q.transpose(0, 2, 3, 4, 1)
    return torch.from_numpy(out).cuda()


def w_dev(q):
    """(Cout,Cg,T,R,S) codes -> device [Cout][T][R][S][Cgp]."""
    Co, Cg, T, R, S = q.shape
    Cgp = (Cg + 15) // 16 * 16
    out = np.zeros((Co, T, R, S, Cgp), np.int8)
    out[..., :Cg] = q.transpose(0, 2, 3, 4, 1)
    return torch.from_numpy(out).cuda()


def geom_struct(g):
    N, Cin, Cout, D, H, W, T, R, S, stride, pad, groups = g
    st = (stride,) * 3 if np.isscalar(stride) else stride
    pd = (pad,) * 3 if np.isscalar(pad) else pad
    return api.Conv3dGeom(N, Cin, Cout, D, H, W, T, R, S, *st, *pd, groups)


@pytest.mark.parametrize("g", GEOMS)
def test_accumulators_and_dequantized_outputs(g):
    N, Cin, Cout, D, H, W, T, R, S, stride, pad, groups = g
    rng = np.random.default_rng(91)
    gs = geom_struct(g)
    Do, P, Q = gs.out_dhw()
    qX, qW = rand_codes(rng, (N, Cin, D, H, W)), rand_codes(rng, (Cout, Cin // groups, T, R, S))
    qG = rand_codes(rng, (N, Cout, Do, P, Q))
    y_o, o1 = O.conv3_acc("fwd", qX, qW, g)
    dx_o, o2 = O.conv3_acc("bwd_data", qG, qW, g)
    dw_o, o3 = O.conv3_acc("bwd_filter", qX, qG, g)
    assert o1 == o2 == o3 == 0
    dX_, dW_, dG_ = act_dev(qX), w_dev(qW), act_dev(qG)
    sX, sW, gmax = 2.9, 0.17, 6.1e-4
    s_c = (10.0 ** rng.uniform(-6, -3, Cout)).astype(np.float32)
    for dtype in (torch.int32, torch.float32, torch.bfloat16):
        Y = torch.empty((N, Do, P, Q, Cout), dtype=dtype, device="cuda")
        dX = torch.empty((N, D, H, W, Cin), dtype=dtype, device="cuda")
        api.conv3d_fwd(dX_, dW_, scalar(sX), scalar(sW), gs, Y)
        api.conv3d_bwd_data(dG_, dW_, scalar(gmax), scalar(sW), gs, dX)
        got_y = Y.float().cpu().numpy().transpose(0, 4, 1, 2, 3) if dtype != torch.int32 else Y.cpu().numpy().transpose(0, 4, 1, 2, 3)
        got_dx = dX.float().cpu().numpy().transpose(0, 4, 1, 2, 3) if dtype != torch.int32 else dX.cpu().numpy().transpose(0, 4, 1, 2, 3)
        if dtype == torch.int32:
            np.testing.assert_array_equal(got_y, y_o)
            np.testing.assert_array_equal(got_dx, dx_o)
        else:
            rel = 1e-5 if dtype == torch.float32 else 2.0 ** -8
            want_y, want_dx = O.dequant_acc(y_o, sX, sW), O.dequant_acc(dx_o, gmax, sW)
            assert np.abs(got_y - want_y).max() <= rel * np.abs(want_y).max()
            assert np.abs(got_dx - want_dx).max() <= rel * np.abs(want_dx).max()
    dW = torch.empty((Cout, Cin // groups, T, R, S), dtype=torch.int32, device="cuda")
    api.conv3d_bwd_filter(dX_, dG_, scalar(sX), torch.from_numpy(s_c).cuda(), gs, dW)
    np.testing.assert_array_equal(dW.cpu().numpy(), dw_o)
    dWf = torch.empty((Cout, Cin // groups, T, R, S), dtype=torch.float32, device="cuda")
    api.conv3d_bwd_filter(dX_, dG_, scalar(sX), torch.from_numpy(s_c).cuda(), gs, dWf)
    want = O.dequant_acc(dw_o, sX, s_c)
    got = dWf.cpu().numpy()
    for co in range(Cout):
        assert np.abs(got[co] - want[co]).max() <= 1e-5 * np.abs(want[co]).max() + 1e-45
    assert api.get_device_status() == api.OK


def test_depthwise_agrees_with_the_2d_kernels_on_a_one_group_layer():
    """Depth 1, one group: the same layer through the 2-D entry points and through this family."""
    from helpers import codes_from_nchw, geom, out_to_nchw
    from test_gpu_conv import weights_dev
    rng = np.random.default_rng(92)
    g2 = (2, 32, 48, 12, 12, 3, 3, 2, 1)
    N, Cin, Cout, H, W, R, S, st, pad = g2
    qX, qW = rand_codes(rng, (N, Cin, H, W)), rand_codes(rng, (Cout, Cin, R, S))
    P, Q = O.out_hw(H, W, R, S, st, pad)
    Y2 = torch.empty((N, P, Q, Cout), dtype=torch.int32, device="cuda")
    api.conv_fwd(codes_from_nchw(qX), weights_dev(qW), scalar(1), scalar(1), geom(*g2), Y2, api.NHWC, None)
    gs = api.Conv3dGeom(N, Cin, Cout, 1, H, W, 1, R, S, 1, st, st, 0, pad, pad, 1)
    Y3 = torch.empty((N, 1, P, Q, Cout), dtype=torch.int32, device="cuda")
    api.conv3d_fwd(act_dev(qX[:, :, None]), w_dev(qW[:, :, None]), scalar(1), scalar(1), gs, Y3)
    assert torch.equal(Y2, Y3[:, 0])


def test_five_dimensional_gradient_through_the_quantizer():
    """dY (N, C, Do, P, Q) of a 3-D convolution is quantized as (N, C, Do*P, Q): per-channel statistics
    over everything but the channel, random numbers by the flat index (Sec. 4.4: the depth is treated
    like height and width)."""
    N, C, Do, P, Q = 3, 32, 4, 7, 9
    g, _, _ = synth.channel_mixed_grad(N, C, Do * P, Q, seed=93)
    check_grad_quant(g, False, api.NHWC, iters=2)      # NHWC of the 4-D view = [N][Do][P][Q][C]
    check_grad_quant(synth.round_to_bf16(g), True, api.NCHW, iters=2)


def test_rejections():
    gs = api.Conv3dGeom(1, 6, 6, 1, 4, 4, 1, 3, 3, 1, 1, 1, 0, 1, 1, 3)       # groups of 2 channels
    t = torch.zeros(16 * 16, dtype=torch.int8, device="cuda")
    y = torch.zeros(16 * 6, dtype=torch.int32, device="cuda")
    with pytest.raises(api.Dai8Error) as e:
        api.conv3d_fwd(t, t, scalar(1), scalar(1), gs, y)
    assert e.value.code == api.ERR_UNSUPPORTED
    gs = api.Conv3dGeom(1, 8, 8, 5, 5, 5, 4, 3, 3, 1, 1, 1, 1, 1, 1, 1)       # 36 taps
    with pytest.raises(api.Dai8Error) as e:
        api.conv3d_fwd(t, t, scalar(1), scalar(1), gs, y)
    assert e.value.code == api.ERR_UNSUPPORTED
