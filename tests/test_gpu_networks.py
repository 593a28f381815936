"""Parity on the layer shapes of the three network configurations (all 53 ResNet-50 convolutions,
the 34 MobileNetV2 pointwise convolutions, the 13 VGG-16 convolutions) at a reduced batch.

Every distinct geometry is run once through forward, input-gradient and weight-gradient
convolutions with raw int32 outputs and compared with the CPU oracle on sampled outputs (each output
of a convolution is an independent dot product) and through the exact integer adjoint identity
<Y, G> = <X, dX> = <W, dW> over the whole tensors.  Every distinct gradient shape (C, H, W) goes
through the stage-wise gradient-quantization check on the whole tensor."""
import numpy as np
import pytest
import torch

from oracle import cpu as O
from paper_2102_04782_b200 import api, synth

from helpers import codes_from_nchw, geom, out_to_nchw, scalar, ws_bytes
from test_gpu_conv import rand_codes, weights_dev
from test_gpu_gvq import check_grad_quant

pytestmark = pytest.mark.gpu


def distinct_layers():
    seen, out = set(), []
    for net, layers in (("resnet50", synth.resnet50_convs()), ("mobilenetv2", synth.mobilenetv2_pointwise()),
                        ("vgg16", synth.vgg16_convs())):
        for L in layers:
            key = (L.Cin, L.Cout, L.H, L.W, L.R, L.S, L.stride, L.pad)
            if key not in seen:
                seen.add(key)
                out.append(pytest.param(key, id=f"{net}-{L.name}-{L.Cin}x{L.Cout}-{L.H}-k{L.R}s{L.stride}"))
    return out


def distinct_grad_shapes():
    seen, out = set(), []
    for layers in (synth.resnet50_convs(), synth.mobilenetv2_pointwise(), synth.vgg16_convs()):
        for L in layers:
            key = (L.Cout, L.P, L.Q)
            if key not in seen:
                seen.add(key)
                out.append(pytest.param(key, id=f"C{L.Cout}-{L.P}x{L.Q}"))
    return out


@pytest.mark.parametrize("key", distinct_layers())
def test_network_layer_convolutions(key):
    Cin, Cout, H, W, R, S, st, pad = key
    N = 2
    rng = np.random.default_rng(hash(key) & 0xFFFF)
    P, Q = O.out_hw(H, W, R, S, st, pad)
    qX, qW = rand_codes(rng, (N, Cin, H, W)), rand_codes(rng, (Cout, Cin, R, S))
    qG = rand_codes(rng, (N, Cout, P, Q))
    qG = (qG.astype(np.int16) * (rng.random(qG.shape) < 0.05)).astype(np.int8)   # far from int32 overflow in dW
    gg = geom(N, Cin, Cout, H, W, R, S, st, pad)
    Y = torch.empty((N, P, Q, Cout), dtype=torch.int32, device="cuda")
    dX = torch.empty((N, H, W, Cin), dtype=torch.int32, device="cuda")
    dW = torch.empty((Cout, Cin, R, S), dtype=torch.int32, device="cuda")
    dqX, dqW, dqG = codes_from_nchw(qX), weights_dev(qW), codes_from_nchw(qG)
    one = scalar(1.0)
    api.conv_fwd(dqX, dqW, one, one, gg, Y, api.NHWC, ws_bytes(api.conv_workspace_bytes(api.OP_FWD, gg)))
    api.conv_bwd_data(dqG, dqW, one, one, gg, dX, api.NHWC, ws_bytes(api.conv_workspace_bytes(api.OP_BWD_DATA, gg)))
    api.conv_bwd_filter(dqX, dqG, one, torch.ones(Cout, device="cuda"), gg, dW,
                        ws_bytes(api.conv_workspace_bytes(api.OP_BWD_FILTER, gg)))
    torch.cuda.synchronize()
    assert api.get_device_status() == api.OK
    Y, dX, dW = out_to_nchw(Y, api.NHWC), out_to_nchw(dX, api.NHWC), dW.cpu().numpy()
    for full, fn, args in ((Y, O.conv_fwd_acc, (qX, qW, st, pad)),
                           (dX, O.conv_bwd_data_acc, (qG, qW, (H, W), st, pad)),
                           (dW, O.conv_bwd_filter_acc, (qX, qG, (R, S), st, pad))):
        idx = rng.choice(full.size, min(512, full.size), replace=False)
        want, ov = fn(*args, idx=idx)
        assert ov == 0
        np.testing.assert_array_equal(full.reshape(-1)[idx], want)
    lhs = int((Y.astype(np.int64) * qG).sum())
    assert lhs == int((dX.astype(np.int64) * qX).sum()) == int((dW.astype(np.int64) * qW).sum())


@pytest.mark.parametrize("key", distinct_grad_shapes())
def test_network_gradient_quantization(key):
    C, H, W = key
    g, _, _ = synth.channel_mixed_grad(2, C, H, W, seed=C + H)
    check_grad_quant(synth.round_to_bf16(g), True, api.NHWC, iters=2)
