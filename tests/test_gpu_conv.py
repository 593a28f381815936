"""GPU parity of the int8 convolutions against the CPU oracle: int32 accumulators bit-exact given
identical codes, de-quantized outputs within rel 1e-5 of max|value|.  Small shapes are compared
element by element; the benchmark's full-size layers on sampled outputs (each output of a direct
convolution is an independent dot product) plus an exact adjoint identity over the whole tensor."""
import numpy as np
import pytest
import torch

from oracle import cpu as O
from paper_2102_04782_b200 import api, synth

from helpers import codes_from_nchw, geom, out_to_nchw, scalar, ws_bytes

pytestmark = pytest.mark.gpu

REL = 1e-5

GEOMS = [
    # N, Cin, Cout, H, W, R, S, stride, pad
    (8, 64, 64, 14, 14, 3, 3, 1, 1),        # config 1
    (2, 3, 16, 17, 19, 7, 7, 2, 3),         # stem-like: 3 channels, 7x7 stride 2
    (3, 24, 40, 9, 11, 1, 1, 1, 0),         # ragged channels, pointwise
    (2, 32, 48, 12, 12, 3, 3, 2, 1),        # stride-2 3x3
    (2, 48, 32, 10, 10, 1, 1, 2, 0),        # stride-2 projection
    (1, 16, 16, 5, 7, 3, 5, (1, 2), (1, 2)),
    (2, 130, 70, 6, 6, 3, 3, 1, 1),         # channel counts that are not multiples of 16
    (1, 64, 128, 30, 30, 3, 3, 1, 1),       # several 128-pixel tiles with a ragged tail
    (2, 32, 16, 20, 20, 1, 1, 1, 0),        # 16 output channels: input gradient in its packed forward form
    (2, 40, 12, 13, 12, 3, 3, 1, 1),        # the same with a 3x3 filter and ragged channel counts
]


def rand_codes(rng, shape):
    return rng.integers(-127, 128, size=shape, dtype=np.int64).astype(np.int8)


def weights_dev(qW):
    """(Cout,Cin,R,S) codes -> device [Cout][R][S][Cinp]."""
    Cout, Cin, R, S = qW.shape
    Cp = (Cin + 15) // 16 * 16
    out = np.zeros((Cout, R, S, Cp), np.int8)
    out[..., :Cin] = qW.transpose(0, 2, 3, 1)
    return torch.from_numpy(out).cuda()


def run_all(g, qX, qW, qG, sX, sW, gmax, s_c, dtype, layout, backend=0):
    N, Cin, Cout, H, W, R, S, st, pad = g
    gg = geom(*g)
    P, Q = gg.P, gg.Q
    api.set_conv_backend(backend)
    try:
        dX_shape = (N, Cin, H, W) if layout == api.NCHW else (N, H, W, Cin)
        Y_shape = (N, Cout, P, Q) if layout == api.NCHW else (N, P, Q, Cout)
        Y = torch.empty(Y_shape, dtype=dtype, device="cuda")
        dX = torch.empty(dX_shape, dtype=dtype, device="cuda")
        dW = torch.empty((Cout, Cin, R, S), dtype=dtype if dtype != torch.bfloat16 else torch.float32,
                         device="cuda")
        dqX, dqW, dqG = codes_from_nchw(qX), weights_dev(qW), codes_from_nchw(qG)
        api.conv_fwd(dqX, dqW, scalar(sX), scalar(sW), gg, Y, layout,
                     ws_bytes(api.conv_workspace_bytes(api.OP_FWD, gg)))
        api.conv_bwd_data(dqG, dqW, scalar(gmax), scalar(sW), gg, dX, layout,
                          ws_bytes(api.conv_workspace_bytes(api.OP_BWD_DATA, gg)))
        api.conv_bwd_filter(dqX, dqG, scalar(sX), torch.from_numpy(s_c).cuda(), gg, dW,
                            ws_bytes(api.conv_workspace_bytes(api.OP_BWD_FILTER, gg)))
        torch.cuda.synchronize()
        assert api.get_device_status() == api.OK
    finally:
        api.set_conv_backend(0)
    return out_to_nchw(Y, layout), out_to_nchw(dX, layout), dW.cpu().numpy()


@pytest.mark.parametrize("g", GEOMS)
@pytest.mark.parametrize("backend", [0, 1])
def test_accumulators_bit_exact(g, backend):
    N, Cin, Cout, H, W, R, S, st, pad = g
    rng = np.random.default_rng(31)
    P, Q = O.out_hw(H, W, R, S, st, pad)
    qX, qW, qG = rand_codes(rng, (N, Cin, H, W)), rand_codes(rng, (Cout, Cin, R, S)), rand_codes(rng, (N, Cout, P, Q))
    s_c = np.ones(Cout, np.float32)
    for layout in (api.NHWC, api.NCHW):
        Y, dX, dW = run_all(g, qX, qW, qG, 1.0, 1.0, 1.0, s_c, torch.int32, layout, backend)
        y_o, ov1 = O.conv_fwd_acc(qX, qW, st, pad)
        dx_o, ov2 = O.conv_bwd_data_acc(qG, qW, (H, W), st, pad)
        dw_o, ov3 = O.conv_bwd_filter_acc(qX, qG, (R, S), st, pad)
        assert ov1 == ov2 == ov3 == 0
        np.testing.assert_array_equal(Y, y_o)
        np.testing.assert_array_equal(dX, dx_o)
        np.testing.assert_array_equal(dW, dw_o)


# Geometries large enough for the tensor-core kernels (activation tensors of at least 128 KiB),
# chosen to hit every shared-memory swizzle width, ragged channel tails filled by the copy engine,
# 256-wide accumulator tiles, tap groups, strides and a pixel count that is not a tile multiple.
TC_GEOMS = [
    (2, 128, 64, 32, 32, 1, 1, 1, 0),
    (2, 64, 256, 48, 48, 1, 1, 1, 0),
    (2, 64, 64, 34, 34, 3, 3, 1, 1),
    (2, 64, 64, 34, 34, 3, 3, 2, 1),
    (3, 48, 40, 33, 35, 3, 3, 1, 1),
    (2, 256, 512, 24, 24, 1, 1, 1, 0),
    (2, 144, 200, 24, 24, 3, 3, 1, 1),
    (1, 32, 32, 70, 70, 5, 5, 1, 2),
    (2, 384, 130, 16, 16, 1, 1, 1, 0),
    (4, 128, 128, 20, 20, 1, 1, 2, 0),
    # multi-tap filters at stride 1 whose output splits into 16 x 8 patches with little waste: the patch
    # form of the forward / input-gradient kernel (one box per tap column instead of one load per tap)
    (2, 64, 64, 32, 40, 3, 3, 1, 1),        # whole tiles, 64-byte rows, resident weights
    (2, 64, 64, 31, 46, 3, 3, 1, 1),        # ragged tiles: clipped stores, zero-filled loads
    (2, 128, 256, 48, 32, 3, 3, 1, 1),      # 128-byte rows, streamed weights, 256-wide accumulators
    (2, 256, 128, 32, 32, 3, 3, 1, 1),      # two channel chunks per tap
    (2, 96, 80, 32, 32, 3, 3, 1, 1),        # ragged channel chunk, 80 output channels
    (1, 32, 48, 64, 72, 5, 5, 1, 2),        # 5x5 filter, 32-byte rows
    (2, 64, 512, 32, 32, 3, 3, 1, 1),       # two accumulator tiles across the output channels
    (3, 64, 64, 47, 32, 3, 3, 1, 0),        # no padding: output 45 x 30
    (1, 32, 512, 64, 64, 3, 3, 1, 1),       # resident weights with two accumulator tiles per pixel tile
    (4, 64, 64, 28, 28, 3, 3, 1, 1),        # 28 wide: patches of 4 rows x 32 columns
    (8, 64, 128, 24, 16, 3, 3, 1, 1),       # 16 wide: patches of 8 rows x 16 columns
    (2, 64, 48, 30, 60, 3, 3, 1, 1),        # 4 x 32 patches, ragged in both directions, 48 output channels
]


@pytest.mark.parametrize("backend", [2, 3])
@pytest.mark.parametrize("g", TC_GEOMS)
def test_tensor_core_kernels_bit_exact(g, backend):
    """Backend 2 = tensor-core kernels only: a geometry they do not take raises instead of being
    silently served by the direct kernels.  Backend 3 = the same with the im2col form of the forward /
    input-gradient kernel even where the patch form applies."""
    N, Cin, Cout, H, W, R, S, st, pad = g
    rng = np.random.default_rng(33)
    P, Q = O.out_hw(H, W, R, S, st, pad)
    qX, qW, qG = rand_codes(rng, (N, Cin, H, W)), rand_codes(rng, (Cout, Cin, R, S)), rand_codes(rng, (N, Cout, P, Q))
    s_c = np.ones(Cout, np.float32)
    stride1 = st == 1
    gg = geom(*g)
    api.set_conv_backend(backend)
    try:
        for layout in (api.NHWC, api.NCHW):
            Y = torch.empty((N, P, Q, Cout) if layout == api.NHWC else (N, Cout, P, Q), dtype=torch.int32, device="cuda")
            api.conv_fwd(codes_from_nchw(qX), weights_dev(qW), scalar(1), scalar(1), gg, Y, layout, None)
            np.testing.assert_array_equal(out_to_nchw(Y, layout), O.conv_fwd_acc(qX, qW, st, pad)[0])
            if stride1 and N * P * Q * ((Cout + 15) // 16 * 16) >= 131072:
                dX = torch.empty((N, H, W, Cin) if layout == api.NHWC else (N, Cin, H, W), dtype=torch.int32, device="cuda")
                api.conv_bwd_data(codes_from_nchw(qG), weights_dev(qW), scalar(1), scalar(1), gg, dX, layout,
                                  ws_bytes(api.conv_workspace_bytes(api.OP_BWD_DATA, gg)))
                np.testing.assert_array_equal(out_to_nchw(dX, layout), O.conv_bwd_data_acc(qG, qW, (H, W), st, pad)[0])
        dW = torch.empty((Cout, Cin, R, S), dtype=torch.int32, device="cuda")
        api.conv_bwd_filter(codes_from_nchw(qX), codes_from_nchw(qG), scalar(1), torch.from_numpy(s_c).cuda(), gg, dW,
                            ws_bytes(api.conv_workspace_bytes(api.OP_BWD_FILTER, gg)))
        np.testing.assert_array_equal(dW.cpu().numpy(), O.conv_bwd_filter_acc(qX, qG, (R, S), st, pad)[0])
        assert api.get_device_status() == api.OK
    finally:
        api.set_conv_backend(0)


def test_tensor_core_backend_refuses_small_shapes():
    g = GEOMS[0]
    gg = geom(*g)
    api.set_conv_backend(2)
    try:
        with pytest.raises(api.Dai8Error) as e:
            api.conv_fwd(torch.zeros((8, 14, 14, 64), dtype=torch.int8, device="cuda"),
                         torch.zeros((64, 3, 3, 64), dtype=torch.int8, device="cuda"), scalar(1), scalar(1), gg,
                         torch.zeros((8, 14, 14, 64), dtype=torch.int32, device="cuda"), api.NHWC, None)
        assert e.value.code == api.ERR_UNSUPPORTED
    finally:
        api.set_conv_backend(0)


@pytest.mark.parametrize("g", [GEOMS[0], GEOMS[3], GEOMS[6], TC_GEOMS[2], TC_GEOMS[6], TC_GEOMS[11], TC_GEOMS[12]])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_dequantized_outputs(g, dtype):
    N, Cin, Cout, H, W, R, S, st, pad = g
    rng = np.random.default_rng(32)
    P, Q = O.out_hw(H, W, R, S, st, pad)
    qX, qW, qG = rand_codes(rng, (N, Cin, H, W)), rand_codes(rng, (Cout, Cin, R, S)), rand_codes(rng, (N, Cout, P, Q))
    sX, sW, gmax = 3.7, 0.21, 8.3e-4
    s_c = (10.0 ** rng.uniform(-6, -3, Cout)).astype(np.float32)
    Y, dX, dW = run_all(g, qX, qW, qG, sX, sW, gmax, s_c, dtype, api.NHWC)
    y_o = O.dequant_acc(O.conv_fwd_acc(qX, qW, st, pad)[0], sX, sW)
    dx_o = O.dequant_acc(O.conv_bwd_data_acc(qG, qW, (H, W), st, pad)[0], gmax, sW)
    dw_o = O.dequant_acc(O.conv_bwd_filter_acc(qX, qG, (R, S), st, pad)[0], sX, s_c)
    rel = REL if dtype == torch.float32 else 2.0 ** -8   # bf16 output: half an ulp of bf16
    for got, want in ((Y, y_o), (dX, dx_o)):
        assert np.abs(got - want).max() <= rel * np.abs(want).max()
    for co in range(Cout):  # per output channel, since the scales differ by decades
        assert np.abs(dW[co] - dw_o[co]).max() <= REL * np.abs(dw_o[co]).max() + 1e-45


def test_config1_end_to_end_layer_step():
    """One layer step on config 1 through the whole path: forward quantization, forward conv,
    gradient quantization, both backward convolutions -- each stage against the oracle fed with the
    GPU's scales."""
    from helpers import GradQuant, codes_to_nchw, dev_input
    layer = synth.config1_layer()
    N = 8
    x, w, g, _, _ = synth.layer_inputs(layer, N, seed=41, bf16=False)
    gg = geom(N, layer.Cin, layer.Cout, layer.H, layer.W, layer.R, layer.S, layer.stride, layer.pad)
    Cp = api.padded_channels(layer.Cin)
    qX = torch.empty((N, layer.H, layer.W, Cp), dtype=torch.int8, device="cuda")
    qW = torch.empty((layer.Cout, layer.R, layer.S, Cp), dtype=torch.int8, device="cuda")
    sX, sW = scalar(0), scalar(0)
    api.quantize_tensor(dev_input(x, False, api.NHWC), api.NHWC, N, layer.Cin, layer.H, layer.W,
                        api.SCALE_ABSMAX, sX, api.ROUND_NEAREST_EVEN, 0, qX)
    api.quantize_tensor(torch.from_numpy(w).cuda(), api.NCHW, layer.Cout, layer.Cin, layer.R, layer.S,
                        api.SCALE_ABSMAX, sW, api.ROUND_NEAREST_EVEN, 0, qW)
    Y = torch.empty((N, layer.P, layer.Q, layer.Cout), dtype=torch.float32, device="cuda")
    api.conv_fwd(qX, qW, sX, sW, gg, Y, api.NHWC, None)
    gqb = GradQuant(N, layer.Cout, layer.P, layer.Q)
    gqb.run(dev_input(g, False, api.NHWC), api.NHWC, 17, has_prev=False)
    dX = torch.empty((N, layer.H, layer.W, layer.Cin), dtype=torch.float32, device="cuda")
    dW = torch.empty((layer.Cout, layer.Cin, layer.R, layer.S), dtype=torch.float32, device="cuda")
    api.conv_bwd_data(gqb.gq, qW, gqb.gmax, sW, gg, dX, api.NHWC,
                      ws_bytes(api.conv_workspace_bytes(api.OP_BWD_DATA, gg)))
    api.conv_bwd_filter(qX, gqb.vq, sX, gqb.s_state, gg, dW,
                        ws_bytes(api.conv_workspace_bytes(api.OP_BWD_FILTER, gg)))
    torch.cuda.synchronize()
    sx, sw = float(sX.item()), float(sW.item())
    assert sx == float(np.abs(x).max()) and sw == float(np.abs(w).max())
    qx_o, qw_o = O.quantize(x, sx), O.quantize(w, sw)
    np.testing.assert_array_equal(codes_to_nchw(qX, layer.Cin), qx_o)
    s_c = gqb.s_state.cpu().numpy()
    gl = float(gqb.gmax.item())
    vq_o = O.quantize(g, s_c, True, 17, 0)
    gq_o = O.quantize(g, gl, True, 17, 1)
    y_o = O.dequant_acc(O.conv_fwd_acc(qx_o, qw_o, 1, 1)[0], sx, sw)
    dx_o = O.dequant_acc(O.conv_bwd_data_acc(gq_o, qw_o, (layer.H, layer.W), 1, 1)[0], gl, sw)
    dw_o = O.dequant_acc(O.conv_bwd_filter_acc(qx_o, vq_o, (3, 3), 1, 1)[0], sx, s_c)
    assert np.abs(out_to_nchw(Y, api.NHWC) - y_o).max() <= REL * np.abs(y_o).max()
    assert np.abs(out_to_nchw(dX, api.NHWC) - dx_o).max() <= REL * np.abs(dx_o).max()
    got = dW.cpu().numpy()
    for co in range(layer.Cout):
        assert np.abs(got[co] - dw_o[co]).max() <= REL * np.abs(dw_o[co]).max() + 1e-45


def _sample_check(g, rng, backend=0, nsamp=2048):
    """Full-size layer: accumulators at sampled outputs, plus the exact adjoint identity
    <Y, G> = <X, dX> = <W, dW> over whole tensors (integers, so equality is exact)."""
    N, Cin, Cout, H, W, R, S, st, pad = g
    P, Q = O.out_hw(H, W, R, S, st, pad)
    qX, qW, qG = rand_codes(rng, (N, Cin, H, W)), rand_codes(rng, (Cout, Cin, R, S)), rand_codes(rng, (N, Cout, P, Q))
    # keep accumulators far from int32 overflow for the dW contraction over N*P*Q pixels
    qG = (qG.astype(np.int16) * (rng.random(qG.shape) < 0.02)).astype(np.int8)
    s_c = np.ones(Cout, np.float32)
    Y, dX, dW = run_all(g, qX, qW, qG, 1.0, 1.0, 1.0, s_c, torch.int32, api.NHWC, backend)
    for full, fn, args in ((Y, O.conv_fwd_acc, (qX, qW, st, pad)),
                           (dX, O.conv_bwd_data_acc, (qG, qW, (H, W), st, pad)),
                           (dW, O.conv_bwd_filter_acc, (qX, qG, (R, S), st, pad))):
        idx = rng.choice(full.size, min(nsamp, full.size), replace=False)
        want, ov = fn(*args, idx=idx)
        assert ov == 0
        np.testing.assert_array_equal(full.reshape(-1)[idx], want)
    lhs = int((Y.astype(np.int64) * qG).sum())
    assert lhs == int((dX.astype(np.int64) * qX).sum()) == int((dW.astype(np.int64) * qW).sum())


@pytest.mark.parametrize("li", [0, 1, 2])
def test_config2_layers_sampled(li):
    """ResNet-50 conv2_x bottleneck at N=64, 56x56 (the benchmark's configuration)."""
    layer = synth.resnet50_conv2x_block()[li]
    g = (64, layer.Cin, layer.Cout, layer.H, layer.W, layer.R, layer.S, layer.stride, layer.pad)
    _sample_check(g, np.random.default_rng(50 + li))


def test_config2_kernel_families_agree_on_whole_tensors():
    """Full-size 3x3 layer of the benchmark: the tensor-core kernels and the direct kernels are
    independent implementations; every accumulator of Y, dX and dW must be identical."""
    layer = synth.resnet50_conv2x_block()[1]
    g = (64, layer.Cin, layer.Cout, layer.H, layer.W, layer.R, layer.S, layer.stride, layer.pad)
    rng = np.random.default_rng(60)
    qX, qW, qG = rand_codes(rng, (64, 64, 56, 56)), rand_codes(rng, (64, 64, 3, 3)), rand_codes(rng, (64, 64, 56, 56))
    qG = (qG.astype(np.int16) * (rng.random(qG.shape) < 0.02)).astype(np.int8)
    s_c = np.ones(64, np.float32)
    a = run_all(g, qX, qW, qG, 1.0, 1.0, 1.0, s_c, torch.int32, api.NHWC, backend=1)
    b = run_all(g, qX, qW, qG, 1.0, 1.0, 1.0, s_c, torch.int32, api.NHWC, backend=2)
    for x, y in zip(a, b):
        np.testing.assert_array_equal(x, y)


def test_unsupported_and_errors():
    gg = geom(1, 16, 16, 4, 4, 3, 3, 1, 1)
    q = torch.zeros((1, 4, 4, 16), dtype=torch.int8, device="cuda")
    w = torch.zeros((16, 3, 3, 16), dtype=torch.int8, device="cuda")
    out = torch.zeros((1, 4, 4, 16), dtype=torch.float32, device="cuda")
    with pytest.raises(api.Dai8Error) as e:
        api.conv_bwd_data(q, w, scalar(1), scalar(1), gg, out, api.NHWC, ws_bytes(16))
    assert e.value.code == api.ERR_WORKSPACE


@pytest.mark.parametrize("g", [(16, 64, 64, 56, 56, 3, 3, 1, 1), (16, 256, 64, 56, 56, 1, 1, 1, 0),
                               (16, 128, 128, 28, 28, 3, 3, 2, 1)])
def test_back_to_back_calls_match_synchronised_calls(g):
    """The kernels of consecutive calls overlap on the device (a kernel's set-up starts while the
    kernel before it drains).  A whole layer step -- quantize X and W, forward, gradient quantization,
    weight and data gradient -- is run once with a device synchronisation after every call, then six
    times back to back without any, alternating between two input sets that share every intermediate
    buffer: a kernel that started reading before its producer had finished would pick up values of the
    other input set.  The last iteration must reproduce the synchronised run bit for bit."""
    from helpers import ws_bytes as wsb
    N, Cin, Cout, H, W, R, S, st, pad = g
    gg = geom(*g)
    P, Q = gg.P, gg.Q
    Cip, Cop = api.padded_channels(Cin), api.padded_channels(Cout)
    bf = torch.bfloat16
    gen = torch.Generator(device="cuda").manual_seed(5)
    sets = []
    for k in range(2):
        sets.append(((torch.randn((N, H, W, Cin), device="cuda", generator=gen) * (1 + k)).to(bf),
                     (torch.randn((Cout, Cin, R, S), device="cuda", generator=gen) * 0.1 * (1 + k)).to(bf),
                     (torch.randn((N, P, Q, Cout), device="cuda", generator=gen) * 1e-3 * (1 + k)).to(bf)))
    qX = torch.empty((N, H, W, Cip), dtype=torch.int8, device="cuda")
    qW = torch.empty((Cout, R, S, Cip), dtype=torch.int8, device="cuda")
    vq = torch.empty((N, P, Q, Cop), dtype=torch.int8, device="cuda")
    gq = torch.empty_like(vq)
    sX, sW, gmax = scalar(0), scalar(0), scalar(0)
    s_c = torch.zeros(Cout, device="cuda")
    Y = torch.empty((N, P, Q, Cout), dtype=bf, device="cuda")
    dX = torch.empty((N, H, W, Cin), dtype=bf, device="cuda")
    dW = torch.empty((Cout, Cin, R, S), dtype=torch.float32, device="cuda")
    ws_g = wsb(api.quantize_grad_workspace_bytes(Cout))
    ws_f = wsb(max(16, api.conv_workspace_bytes(api.OP_FWD, gg)))
    ws_d = wsb(api.conv_workspace_bytes(api.OP_BWD_DATA, gg))
    ws_w = wsb(api.conv_workspace_bytes(api.OP_BWD_FILTER, gg))

    def step(inputs, sync):
        x, w, dy = inputs
        calls = [
            lambda: api.quantize_tensor(x, api.NHWC, N, Cin, H, W, api.SCALE_ABSMAX, sX, api.ROUND_NEAREST_EVEN, 0, qX),
            lambda: api.quantize_tensor(w, api.NCHW, Cout, Cin, R, S, api.SCALE_ABSMAX, sW, api.ROUND_NEAREST_EVEN, 0, qW),
            lambda: api.conv_fwd(qX, qW, sX, sW, gg, Y, api.NHWC, ws_f),
            lambda: api.quantize_grad(dy, api.NHWC, N, Cout, P, Q, None, s_c, False, gmax, None, None, vq, gq, 9, ws_g),
            lambda: api.conv_bwd_filter(qX, vq, sX, s_c, gg, dW, ws_w),
            lambda: api.conv_bwd_data(gq, qW, gmax, sW, gg, dX, api.NHWC, ws_d),
        ]
        for c in calls:
            c()
            if sync:
                torch.cuda.synchronize()

    step(sets[0], sync=True)
    want = [t.clone() for t in (qX, qW, Y, vq, gq, dW, dX, s_c)]
    for it in range(6):
        step(sets[(it + 1) % 2], sync=False)       # other set first, ends on input set 0
    torch.cuda.synchronize()
    names = ("qX", "qW", "Y", "vq", "gq", "dW", "dX", "s_c")
    bad = [n for n, a, b in zip(names, want, (qX, qW, Y, vq, gq, dW, dX, s_c)) if not torch.equal(a, b)]
    assert not bad, bad
    assert api.get_device_status() == api.OK


def test_bounded_waits_give_up_and_the_library_stays_usable():
    """The give-up path of the device-side waits: barriers nobody completes, a limit of a few thousand
    cycles, nothing in flight.  Each wait must return by itself and leave DAI8_ERR_TIMEOUT in the device
    status word; reading clears it, and a normal call afterwards is bit-exact again."""
    assert api.get_device_status() == api.OK
    flags = api.debug_expire_waits(5000, ws_bytes(64))
    assert flags == [1, 1, 1]
    assert api.get_device_status() == api.ERR_TIMEOUT      # read ...
    assert api.get_device_status() == api.OK               # ... and cleared
    g = TC_GEOMS[2]
    N, Cin, Cout, H, W, R, S, st, pad = g
    rng = np.random.default_rng(77)
    P, Q = O.out_hw(H, W, R, S, st, pad)
    qX, qW = rand_codes(rng, (N, Cin, H, W)), rand_codes(rng, (Cout, Cin, R, S))
    Y = torch.empty((N, P, Q, Cout), dtype=torch.int32, device="cuda")
    api.conv_fwd(codes_from_nchw(qX), weights_dev(qW), scalar(1), scalar(1), geom(*g), Y, api.NHWC, None)
    np.testing.assert_array_equal(out_to_nchw(Y, api.NHWC), O.conv_fwd_acc(qX, qW, st, pad)[0])
    assert api.get_device_status() == api.OK
