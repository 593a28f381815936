"""Parity on the layer shapes of the three network configurations (all 53 ResNet-50 convolutions,
the 34 MobileNetV2 pointwise convolutions, the 13 VGG-16 convolutions).

At the networks' own batch (64 / 128), in the launch configuration the benchmark times, every
distinct geometry is run through forward, input-gradient and weight-gradient convolutions with raw
int32 outputs and compared with the CPU oracle on sampled outputs (each output of a convolution is an
independent dot product: 4096 random ones per tensor plus every border row and column of one image)
and through the exact integer adjoint identity <Y, G> = <X, dX> = <W, dW> over the whole tensors.  The
tensor-core kernels are selected explicitly, so a geometry they do not take raises instead of being
served by the direct kernels; the few passes that are expected on the direct kernels are listed.
At batch 2 the same geometries run once more with the kernel family pinned where the tensor-core
kernels apply at that size.  Every distinct gradient shape (C, H, W) goes through the stage-wise
gradient-quantization check on the whole tensor."""
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


def distinct_layers_full_batch():
    seen, out = set(), []
    for net, layers, N in (("resnet50", synth.resnet50_convs(), 64), ("mobilenetv2", synth.mobilenetv2_pointwise(), 128),
                           ("vgg16", synth.vgg16_convs(), 64)):
        for L in layers:
            key = (N, L.Cin, L.Cout, L.H, L.W, L.R, L.S, L.stride, L.pad)
            if key not in seen:
                seen.add(key)
                out.append(pytest.param(key, id=f"{net}-N{N}-{L.name}-{L.Cin}x{L.Cout}-{L.H}-k{L.R}s{L.stride}"))
    return out


# Passes that the tensor-core kernels do not take at full batch (geometry key -> pass names); every
# other pass of every layer must run on them.
EXPECTED_DIRECT_AT_FULL_BATCH = {}


def _border_and_random(rng, shape, nsamp):
    """Flat NCHW indices: nsamp random ones plus every border row and column of image 0 (all channels)."""
    N, C, H, W = shape
    total = N * C * H * W
    idx = [rng.choice(total, min(nsamp, total), replace=False)]
    hh, ww = np.meshgrid(np.arange(H), np.arange(W), indexing="ij")
    border = (hh == 0) | (hh == H - 1) | (ww == 0) | (ww == W - 1)
    pos = (hh * W + ww)[border]
    idx.append((np.arange(C)[:, None] * (H * W) + pos[None, :]).reshape(-1))
    return np.unique(np.concatenate(idx))


def _dot64(a, b):
    """Exact integer inner product of two device tensors of the same shape, image by image."""
    tot = 0
    for i in range(a.shape[0]):
        tot += int((a[i].to(torch.int64) * b[i].to(torch.int64)).sum().item())
    return tot


@pytest.mark.parametrize("key", distinct_layers_full_batch())
def test_network_layer_convolutions_full_batch(key):
    N, Cin, Cout, H, W, R, S, st, pad = key
    P, Q = O.out_hw(H, W, R, S, st, pad)
    gen = torch.Generator(device="cuda").manual_seed(hash(key) & 0xFFFFFF)
    Cip, Cop = api.padded_channels(Cin), api.padded_channels(Cout)

    def codes(shape, C, keep=1.0):
        t = torch.randint(-127, 128, shape, dtype=torch.int8, device="cuda", generator=gen)
        if keep < 1.0:   # sparse gradient codes keep the dW accumulators far from int32 overflow
            t = t * (torch.rand(shape, device="cuda", generator=gen) < keep).to(torch.int8)
        t[..., C:] = 0
        return t

    dqX = codes((N, H, W, Cip), Cin)
    dqW = codes((Cout, R, S, Cip), Cin)
    dqG = codes((N, P, Q, Cop), Cout, keep=0.02)
    gg = geom(N, Cin, Cout, H, W, R, S, st, pad)
    Y = torch.empty((N, P, Q, Cout), dtype=torch.int32, device="cuda")
    dX = torch.empty((N, H, W, Cin), dtype=torch.int32, device="cuda")
    dW = torch.empty((Cout, Cin, R, S), dtype=torch.int32, device="cuda")
    one = scalar(1.0)
    ones = torch.ones(Cout, device="cuda")
    calls = {
        "fwd": lambda: api.conv_fwd(dqX, dqW, one, one, gg, Y, api.NHWC, ws_bytes(api.conv_workspace_bytes(api.OP_FWD, gg))),
        "bwd_data": lambda: api.conv_bwd_data(dqG, dqW, one, one, gg, dX, api.NHWC,
                                              ws_bytes(api.conv_workspace_bytes(api.OP_BWD_DATA, gg))),
        "bwd_filter": lambda: api.conv_bwd_filter(dqX, dqG, one, ones, gg, dW,
                                                  ws_bytes(api.conv_workspace_bytes(api.OP_BWD_FILTER, gg))),
    }
    on_direct = set()
    try:
        for name, call in calls.items():
            api.set_conv_backend(2)
            try:
                call()
            except api.Dai8Error as e:
                assert e.code == api.ERR_UNSUPPORTED
                on_direct.add(name)
                api.set_conv_backend(1)
                call()
        torch.cuda.synchronize()
    finally:
        api.set_conv_backend(0)
    assert api.get_device_status() == api.OK
    assert on_direct == set(EXPECTED_DIRECT_AT_FULL_BATCH.get(key, ())), on_direct
    # exact adjoint identity over the whole tensors (integers)
    lhs = _dot64(Y, dqG[..., :Cout])
    assert lhs == _dot64(dX, dqX[..., :Cin])
    assert lhs == _dot64(dW.permute(0, 2, 3, 1), dqW[..., :Cin])
    # sampled outputs against the oracle
    rng = np.random.default_rng(hash(key) & 0xFFFF)
    qX = np.ascontiguousarray(dqX.cpu().numpy()[..., :Cin].transpose(0, 3, 1, 2))
    qW = np.ascontiguousarray(dqW.cpu().numpy()[..., :Cin].transpose(0, 3, 1, 2))
    qG = np.ascontiguousarray(dqG.cpu().numpy()[..., :Cout].transpose(0, 3, 1, 2))
    for dev_t, shape, to_nchw, fn, args in (
            (Y, (N, Cout, P, Q), True, O.conv_fwd_acc, (qX, qW, st, pad)),
            (dX, (N, Cin, H, W), True, O.conv_bwd_data_acc, (qG, qW, (H, W), st, pad)),
            (dW, (Cout, Cin, R, S), False, O.conv_bwd_filter_acc, (qX, qG, (R, S), st, pad))):
        if to_nchw:
            idx = _border_and_random(rng, shape, 4096)
            n, rem = np.divmod(idx, shape[1] * shape[2] * shape[3])
            c, hw = np.divmod(rem, shape[2] * shape[3])
            flat_nhwc = (n * shape[2] * shape[3] + hw) * shape[1] + c
        else:
            total = int(np.prod(shape))
            idx = rng.choice(total, min(4096, total), replace=False)
            flat_nhwc = idx
        got = dev_t.reshape(-1)[torch.from_numpy(flat_nhwc).cuda()].cpu().numpy()
        want, ov = fn(*args, idx=idx)
        assert ov == 0
        np.testing.assert_array_equal(got, want)


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
    calls = (lambda: api.conv_fwd(dqX, dqW, one, one, gg, Y, api.NHWC, ws_bytes(api.conv_workspace_bytes(api.OP_FWD, gg))),
             lambda: api.conv_bwd_data(dqG, dqW, one, one, gg, dX, api.NHWC, ws_bytes(api.conv_workspace_bytes(api.OP_BWD_DATA, gg))),
             lambda: api.conv_bwd_filter(dqX, dqG, one, torch.ones(Cout, device="cuda"), gg, dW,
                                         ws_bytes(api.conv_workspace_bytes(api.OP_BWD_FILTER, gg))))
    try:
        for call in calls:      # the kernel family is chosen here, never by the library's automatic mode
            api.set_conv_backend(2)
            try:
                call()
            except api.Dai8Error as e:
                assert e.code == api.ERR_UNSUPPORTED
                api.set_conv_backend(1)
                call()
        torch.cuda.synchronize()
    finally:
        api.set_conv_backend(0)
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


@pytest.mark.parametrize("shape", [
    (64, 2048, 7, 7),       # ResNet-50 stage 5: whole vector columns per CTA
    (64, 1024, 14, 14),     # stage 4 outputs
    (64, 512, 28, 28),      # stage 3 outputs / VGG conv8-10
    (128, 96, 56, 56),      # MobileNetV2 expansion: 12 vector columns, rows across warp boundaries
    (128, 24, 56, 56),      # MobileNetV2 projection: padded code channels
    (64, 128, 112, 112),    # VGG conv3-4: 205 MB, mostly streamed through the piece ring
], ids=lambda s: "x".join(map(str, s)))
def test_network_gradient_quantization_full_batch(shape):
    """Gradient shapes of the three networks at their own batch, whole tensor, every stage."""
    N, C, H, W = shape
    g, _, _ = synth.channel_mixed_grad(N, C, H, W, seed=C + H + N)
    check_grad_quant(synth.round_to_bf16(g), True, api.NHWC, iters=2)
