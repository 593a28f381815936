"""GPU parity of dai8_quantize_grad / dai8_quantize_tensor against the CPU oracle, stage by stage
so that a discrete decision (class, code) is always compared given identical upstream values:
  (1) |g|max bit-exact, mean / sigma within rel 1e-5;
  (2) density count exact given the GPU's sigma;
  (3) class exact and clip within rel 1e-5 given identical (count, |g|max, s_prev);
  (4) int8 codes bit-exact given identical scales;
then end to end (the oracle running on its own sigma), where only channels whose count lies within
2 of the threshold lambda*M may differ."""
import numpy as np
import pytest
import torch

from oracle import cpu as O
from paper_2102_04782_b200 import api, synth

from helpers import GradQuant, codes_to_nchw, dev_input, padding_is_zero, scalar, ws_bytes

pytestmark = pytest.mark.gpu

REL = 1e-5


def check_grad_quant(g, bf16, layout, seed=5, iters=2, params=None, later=()):
    """`later`: tensors for the iterations after the first (default: the same tensor again)."""
    N, C, H, W = g.shape
    M = N * H * W
    gq = GradQuant(N, C, H, W)
    tensors = [g] + list(later)
    kw = {}
    if params is not None:
        kw = dict(lam=params.lam, k=params.k, A=params.A)
    s_prev_gpu = None
    s_prev_e2e = None
    band_ever = np.zeros(C, bool)
    for t in range(iters):
        g = tensors[min(t, len(tensors) - 1)]
        d = dev_input(g, bf16, layout)
        gq.run(d, layout, seed + t, has_prev=t > 0, params=params)
        stats = gq.stats.cpu().numpy()
        s_gpu = gq.s_state.cpu().numpy()
        cls_gpu = gq.cls.cpu().numpy()
        gmax_gpu = float(gq.gmax.item())
        # (1)
        absmax, mean, sigma, gl = O.channel_stats(g, bool(params.std_unbiased) if params else False,
                                                  bool(params.center_mean) if params else True)
        np.testing.assert_array_equal(stats[:, 0], absmax)
        assert gmax_gpu == gl
        np.testing.assert_allclose(stats[:, 2], sigma, rtol=REL, atol=0)
        assert np.all(np.abs(stats[:, 1] - mean) <= REL * np.maximum(sigma, 1e-30) + 1e-7 * np.abs(mean))
        # (2) count given the GPU's sigma
        cnt = O.density_count(g, stats[:, 2])
        np.testing.assert_array_equal(stats[:, 3], (cnt.astype(np.float64) / M).astype(np.float32))
        # (3) class and clip given identical inputs
        s_or, cls_or = O.classify_clip(cnt, absmax, M, s_prev=s_prev_gpu, **kw)
        np.testing.assert_array_equal(cls_gpu, cls_or)
        np.testing.assert_allclose(s_gpu, s_or, rtol=REL, atol=0)
        # (4) codes given identical scales
        vq = codes_to_nchw(gq.vq, C)
        gqc = codes_to_nchw(gq.gq, C)
        np.testing.assert_array_equal(vq, O.quantize(g, s_gpu, stochastic=True, seed=seed + t, stream=0))
        np.testing.assert_array_equal(gqc, O.quantize(g, gmax_gpu, stochastic=True, seed=seed + t, stream=1))
        assert padding_is_zero(gq.vq, C) and padding_is_zero(gq.gq, C)
        # end to end: the oracle on its own sigma
        cnt_e = O.density_count(g, sigma)
        s_e, cls_e = O.classify_clip(cnt_e, absmax, M, s_prev=s_prev_e2e, **kw)
        lam = np.float32(params.lam if params else 0.3)
        band_ever |= np.abs(cnt_e.astype(np.float64) - float(lam) * M) <= 2
        assert np.array_equal(cls_gpu[~band_ever], cls_e[~band_ever])
        np.testing.assert_allclose(s_gpu[~band_ever], s_e[~band_ever], rtol=REL)
        s_prev_gpu = s_gpu
        s_prev_e2e = s_e
    return gq


@pytest.mark.parametrize("layout", [api.NHWC, api.NCHW])
@pytest.mark.parametrize("bf16", [False, True])
def test_config1_grad_quant(layout, bf16):
    """Config 1: N=8, C=64, 14x14, per-channel bell-shaped / long-tailed mix."""
    g, is_bell, _ = synth.channel_mixed_grad(8, 64, 14, 14, seed=1)
    if bf16:
        g = synth.round_to_bf16(g)
    gq = check_grad_quant(g, bf16, layout, iters=3)
    cls = gq.cls.cpu().numpy()
    # long-tailed channels are never classed bell-shaped; most bell-shaped ones are
    assert not np.any(cls[~is_bell])
    assert cls[is_bell].mean() > 0.8


@pytest.mark.parametrize("shape", [
    (2, 24, 7, 9),      # C multiple of 8 but not 16: padded code channels
    (3, 20, 5, 5),      # bf16: C not a multiple of 8 -> element-wise path; fp32: vector path
    (1, 3, 11, 13),     # tiny C, odd extents, misaligned NCHW rows
    (2, 2048, 2, 2),    # several column blocks
    (5, 96, 9, 9),
    (3, 144, 10, 11),   # 18 bf16 vector columns: rows of the fused kernel run across warp boundaries
    (1, 1, 1, 1),
    (2, 16, 1, 300),
])
@pytest.mark.parametrize("layout", [api.NHWC, api.NCHW])
@pytest.mark.parametrize("bf16", [False, True])
def test_ragged_shapes(shape, layout, bf16):
    g, _, _ = synth.channel_mixed_grad(*shape, seed=2)
    if bf16:
        g = synth.round_to_bf16(g)
    check_grad_quant(g, bf16, layout, iters=2)


@pytest.mark.parametrize("shape", [(8, 64, 14, 14), (4, 256, 40, 40), (64, 64, 56, 56)])
def test_classes_change_between_iterations(shape):
    """The fused kernel writes the codes with the class it predicts (from the previous classes when
    the caller passes them) and redoes mispredicted channels: feed it tensors whose channels swap
    between bell-shaped and long-tailed from one iteration to the next, so that about half of the
    hints are wrong, and check every stage against the oracle as usual."""
    ga, bell_a, _ = synth.channel_mixed_grad(*shape, seed=21)
    gb, bell_b, _ = synth.channel_mixed_grad(*shape, seed=22)
    gc, _, _ = synth.channel_mixed_grad(*shape, seed=23)
    assert np.any(bell_a != bell_b)
    rb = synth.round_to_bf16
    check_grad_quant(rb(ga), True, api.NHWC, iters=3, later=(rb(gb), rb(gc)))
    check_grad_quant(ga, False, api.NHWC, iters=3, later=(gb, gc))


def test_hyper_parameters_and_flags():
    g, _, _ = synth.channel_mixed_grad(4, 32, 12, 12, seed=3)
    g = g + np.float32(2e-5)  # a mean offset so that center_mean matters
    for k, A, unb, cen in [(1.5, 0.5, 0, 1), (1.2, 0.8, 1, 1), (1.0, 0.8, 0, 0)]:
        p = api.mcs_defaults()
        p.k, p.A, p.std_unbiased, p.center_mean = k, A, unb, cen
        check_grad_quant(g, False, api.NHWC, iters=3, params=p)


def test_zero_channel_and_sigma_override():
    g, _, _ = synth.channel_mixed_grad(2, 16, 6, 6, seed=4)
    g[:, 3] = 0.0
    gq = check_grad_quant(g, False, api.NHWC, iters=2)
    assert float(gq.s_state[3].item()) == 0.0
    assert np.all(codes_to_nchw(gq.vq, 16)[:, 3] == 0)
    # a caller-provided sigma replaces the computed one in the density count
    sig = torch.full((16,), 1e-9, dtype=torch.float32, device="cuda")
    d = dev_input(g, False, api.NHWC)
    gq.run(d, api.NHWC, 1, has_prev=False, sigma_override=sig)
    P = gq.stats.cpu().numpy()[:, 3]
    want = O.density_count(g, np.full(16, 1e-9, np.float32)) / (2 * 36)
    np.testing.assert_allclose(P, want, rtol=1e-6)


def test_without_layer_codes():
    g, _, _ = synth.channel_mixed_grad(2, 32, 5, 5, seed=6)
    gq = GradQuant(2, 32, 5, 5)
    gq.run(dev_input(g, False, api.NHWC), api.NHWC, 3, has_prev=False, with_gq=False)
    assert bool((gq.gq == 77).all().item())  # untouched
    s = gq.s_state.cpu().numpy()
    np.testing.assert_array_equal(codes_to_nchw(gq.vq, 32), O.quantize(g, s, True, 3, 0))


@pytest.mark.parametrize("layout", [api.NHWC, api.NCHW])
@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("shape", [(2, 64, 14, 14), (1, 3, 17, 19), (64, 3, 7, 7), (2, 40, 3, 5)])
def test_quantize_tensor(shape, layout, bf16):
    N, C, H, W = shape
    x = synth.activations(N, C, H, W, seed=7) - np.float32(0.3)
    if bf16:
        x = synth.round_to_bf16(x)
    Cp = api.padded_channels(C)
    d = dev_input(x, bf16, layout)
    q = torch.full((N, H, W, Cp), 55, dtype=torch.int8, device="cuda")
    s = scalar(0.0)
    api.quantize_tensor(d, layout, N, C, H, W, api.SCALE_ABSMAX, s, api.ROUND_NEAREST_EVEN, 0, q)
    torch.cuda.synchronize()
    assert float(s.item()) == float(np.abs(x).max())
    np.testing.assert_array_equal(codes_to_nchw(q, C), O.quantize(x, float(s.item())))
    assert padding_is_zero(q, C)
    # given scale (clipping) and stochastic rounding
    s2 = scalar(0.5)
    api.quantize_tensor(d, layout, N, C, H, W, api.SCALE_GIVEN, s2, api.ROUND_STOCHASTIC, 11, q)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(codes_to_nchw(q, C), O.quantize(x, 0.5, stochastic=True, seed=11))


# Tensors above 131072 codes leave the single-launch kernel for small tensors and take the
# large-tensor kernels (layer-scale reduction, then the code kernels), which is what the benchmark
# times.  One case per code path: NHWC with C = Cp (flat walk, nearest), NHWC with padded code channels
# (C a vector multiple or not), NCHW activations, NCHW weights (transposed to [Cout][R][S][Cinp]), and
# a length that is not a multiple of the grid stride.
LARGE_TENSORS = [
    # (N, C, H, W), layout
    ((4, 64, 40, 40), api.NHWC),        # C = Cp: flat path
    ((3, 48, 33, 35), api.NHWC),        # C = Cp, vector count not a multiple of the block size
    ((4, 24, 48, 48), api.NHWC),        # C != Cp, C a multiple of the fp32 and bf16 vector
    ((4, 20, 41, 43), api.NHWC),        # bf16: C not a vector multiple -> element-wise columns
    ((8, 3, 100, 100), api.NHWC),       # stem-like
    ((4, 40, 37, 41), api.NCHW),        # NCHW activation, ragged position tiles
    ((512, 512, 3, 3), api.NCHW),       # VGG weights: rows of 9 elements
    ((256, 130, 3, 3), api.NCHW),       # weights with padded code channels
    ((1024, 256, 1, 1), api.NCHW),      # pointwise weights
    ((2, 130, 31, 33), api.NCHW),       # channel tiles with a ragged tail
    ((5, 13, 61, 67), api.NHWC),        # fewer than 16 channels: one thread per pixel
    ((600, 27, 3, 3), api.NCHW),        # filters whose byte size is not a multiple of 16: ranges of CTAs start unaligned
    ((300, 100, 5, 5), api.NCHW),       # 5x5 filters, several per CTA
]


@pytest.mark.parametrize("with_ws", [False, True])
@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("shape,layout", LARGE_TENSORS)
def test_quantize_tensor_large(shape, layout, bf16, with_ws):
    """with_ws: the caller passes scratch memory, which lets flat tensors take the one-launch kernel
    (scale and codes in one cooperative launch); without it the scale and the codes are two launches."""
    N, C, H, W = shape
    ws = ws_bytes(api.quantize_tensor_workspace_bytes()) if with_ws else None
    Cp = api.padded_channels(C)
    assert N * H * W * Cp > 131072
    x = synth.activations(N, C, H, W, seed=71) - np.float32(0.3)
    if bf16:
        x = synth.round_to_bf16(x)
    d = dev_input(x, bf16, layout)
    for mode, given, rounding in ((api.SCALE_ABSMAX, 0.0, api.ROUND_NEAREST_EVEN),
                                  (api.SCALE_GIVEN, 0.5, api.ROUND_NEAREST_EVEN),
                                  (api.SCALE_GIVEN, 0.75, api.ROUND_STOCHASTIC),
                                  (api.SCALE_ABSMAX, 0.0, api.ROUND_STOCHASTIC)):
        q = torch.full((N, H, W, Cp), 55, dtype=torch.int8, device="cuda")
        s = scalar(given)
        api.quantize_tensor(d, layout, N, C, H, W, mode, s, rounding, 13, q, ws)
        torch.cuda.synchronize()
        sv = float(s.item())
        if mode == api.SCALE_ABSMAX:
            assert sv == float(np.abs(x).max())
        else:
            assert sv == given
        want = O.quantize(x, sv, stochastic=rounding == api.ROUND_STOCHASTIC, seed=13)
        np.testing.assert_array_equal(codes_to_nchw(q, C), want)
        assert padding_is_zero(q, C)


def test_quantize_tensor_benchmark_activation():
    """X of the ResNet-50 conv2_x 1x1 256->64 layer at full size, (64, 256, 56, 56) bf16 NHWC: the
    layer-scale reduction and the flat code kernel in the launch configuration the benchmark times."""
    N, C, H, W = 64, 256, 56, 56
    x = synth.round_to_bf16(synth.activations(N, C, H, W, seed=72) - np.float32(0.1))
    d = dev_input(x, True, api.NHWC)
    want = None
    for ws in (None, ws_bytes(api.quantize_tensor_workspace_bytes())):
        q = torch.full((N, H, W, C), 55, dtype=torch.int8, device="cuda")
        s = scalar(0.0)
        api.quantize_tensor(d, api.NHWC, N, C, H, W, api.SCALE_ABSMAX, s, api.ROUND_NEAREST_EVEN, 0, q, ws)
        torch.cuda.synchronize()
        assert api.get_device_status() == api.OK
        assert float(s.item()) == float(np.abs(x).max())
        if want is None:
            want = O.quantize(x, float(s.item()))
        np.testing.assert_array_equal(codes_to_nchw(q, C), want)


def test_weight_layout_from_quantize_tensor():
    """Weights passed as an NCHW tensor (N=Cout, C=Cin, H=R, W=S) come out as [Cout][R][S][Cinp]."""
    w = synth.weights(8, 5, 3, 3, seed=8)
    q = torch.empty((8, 3, 3, 16), dtype=torch.int8, device="cuda")
    s = scalar(0.0)
    api.quantize_tensor(torch.from_numpy(w).cuda(), api.NCHW, 8, 5, 3, 3, api.SCALE_ABSMAX, s,
                        api.ROUND_NEAREST_EVEN, 0, q)
    torch.cuda.synchronize()
    want = O.quantize(w, float(np.abs(w).max()))           # (Cout,Cin,R,S)
    np.testing.assert_array_equal(q.cpu().numpy()[..., :5], want.transpose(0, 2, 3, 1))


def test_config2_full_size_grad_quant():
    """ResNet-50 conv2_x 3x3 layer: dY (64,64,56,56) bf16 NHWC, the launch configuration the
    benchmark times; full-tensor comparison (the oracle's O(elements) parts run in seconds)."""
    g, _, _ = synth.channel_mixed_grad(64, 64, 56, 56, seed=9)
    g = synth.round_to_bf16(g)
    check_grad_quant(g, True, api.NHWC, iters=2)


def test_benchmark_gradient_full_size():
    """dY of the ResNet-50 conv2_x 1x1 64->256 layer, (64, 256, 56, 56) bf16 NHWC, 102.8 MB: more than a
    CTA keeps resident in shared memory, so part of every CTA's range cycles through the piece ring and
    is fetched again in the second sweep.  Whole tensor, every stage, two iterations."""
    g, _, _ = synth.channel_mixed_grad(64, 256, 56, 56, seed=10)
    g = synth.round_to_bf16(g)
    check_grad_quant(g, True, api.NHWC, iters=2)


def test_more_than_2_32_elements():
    """A gradient with more than 2^32 elements (4097 x 128 x 128 x 64, 8.6 GB in bf16) takes the fused
    kernel's 64-bit index arithmetic, and the generator's key then depends on the high half of the
    element index.  All images but the last are zero, so everything the oracle needs -- |g|max, the
    density count, the codes of the last image, whose element indices lie beyond 2^32 -- follows
    from the last image alone; every other code must be 0."""
    N, C, H, W = 4097, 64, 128, 128
    M = N * H * W
    last, _, _ = synth.channel_mixed_grad(1, C, H, W, seed=31)
    last = synth.round_to_bf16(last)
    dY = torch.zeros((N, H, W, C), dtype=torch.bfloat16, device="cuda")
    dY[N - 1] = torch.from_numpy(last[0].transpose(1, 2, 0).copy()).cuda().to(torch.bfloat16)
    vq = torch.full((N, H, W, C), 77, dtype=torch.int8, device="cuda")
    gq = torch.full((N, H, W, C), 77, dtype=torch.int8, device="cuda")
    s_state = torch.zeros(C, device="cuda"); gmax = torch.zeros(1, device="cuda")
    stats = torch.zeros(C, 4, device="cuda"); cls = torch.zeros(C, dtype=torch.uint8, device="cuda")
    ws = torch.empty(api.quantize_grad_workspace_bytes(C), dtype=torch.uint8, device="cuda")
    seed = 12
    api.quantize_grad(dY, api.NHWC, N, C, H, W, None, s_state, False, gmax, stats, cls, vq, gq, seed, ws)
    torch.cuda.synchronize()
    assert api.get_device_status() == api.OK
    assert int(torch.count_nonzero(vq[: N - 1]).item()) == 0 and int(torch.count_nonzero(gq[: N - 1]).item()) == 0
    st = stats.cpu().numpy()
    absmax, _, _, gl = O.channel_stats(last)
    np.testing.assert_array_equal(st[:, 0], absmax)
    assert float(gmax.item()) == gl
    # moments over all M pixels from the last image's (binary64): the zeros only enter through M
    x = last[0].reshape(C, -1).astype(np.float64)
    mean = x.sum(axis=1) / M
    sigma = np.sqrt(np.maximum((x * x).sum(axis=1) / M - mean * mean, 0.0))
    np.testing.assert_allclose(st[:, 2], sigma, rtol=REL, atol=0)
    cnt = O.density_count(last, st[:, 2])          # zeros never exceed a positive sigma
    np.testing.assert_array_equal(st[:, 3], (cnt.astype(np.float64) / M).astype(np.float32))
    s_or, cls_or = O.classify_clip(cnt, absmax, M, s_prev=None)
    np.testing.assert_array_equal(cls.cpu().numpy(), cls_or)
    s_gpu = s_state.cpu().numpy()
    np.testing.assert_allclose(s_gpu, s_or, rtol=REL, atol=0)
    got_v = vq[N - 1].cpu().numpy().transpose(2, 0, 1)[None]
    got_g = gq[N - 1].cpu().numpy().transpose(2, 0, 1)[None]
    np.testing.assert_array_equal(got_v, O.quantize(last, s_gpu, True, seed, 0, first_image=N - 1))
    np.testing.assert_array_equal(got_g, O.quantize(last, gl, True, seed, 1, first_image=N - 1))


MODES = {"gq": api.GRAD_GQ, "gvq_max": api.GRAD_GVQ_MAX, "layer_mcs": api.GRAD_LAYER_MCS}


@pytest.mark.parametrize("mode", ["gq", "gvq_max", "layer_mcs"])
@pytest.mark.parametrize("layout", [api.NHWC, api.NCHW])
@pytest.mark.parametrize("shape,bf16", [((8, 64, 14, 14), False), ((3, 20, 9, 11), True), ((16, 64, 56, 56), True)])
def test_ablation_modes(mode, layout, shape, bf16):
    """The quantization strategies of the ablation study (Sec. 4.1) as modes of dai8_quantize_grad, three
    iterations each, stage by stage against the oracle's composition of the same steps."""
    N, C, H, W = shape
    M = N * H * W
    g0, _, _ = synth.channel_mixed_grad(N, C, H, W, seed=51)
    if mode == "layer_mcs":
        g0 = g0 / np.float32(g0.std(axis=(0, 2, 3), keepdims=True))     # equal widths: the layer's class can go either way
    p = api.mcs_defaults()
    p.mode = MODES[mode]
    gq = GradQuant(N, C, H, W)
    s_prev = None
    for t in range(3):
        g = g0 * np.float32(1.0 + 0.25 * t)
        if t == 1 and mode == "layer_mcs":
            g = np.random.default_rng(5).laplace(0, 1e-4, g.shape).astype(np.float32)   # a long-tailed layer
        if bf16:
            g = synth.round_to_bf16(g)
        gq.run(dev_input(g, bf16, layout), layout, 40 + t, has_prev=t > 0, params=p)
        stats = gq.stats.cpu().numpy()
        s_gpu, cls_gpu, gl_gpu = gq.s_state.cpu().numpy(), gq.cls.cpu().numpy(), float(gq.gmax.item())
        absmax, mean, sigma, gl = O.channel_stats(g)
        np.testing.assert_array_equal(stats[:, 0], absmax)
        assert gl_gpu == gl
        if mode == "gq":
            assert np.all(s_gpu == gl) and np.all(cls_gpu == 1)
        elif mode == "gvq_max":
            np.testing.assert_array_equal(s_gpu, absmax)
            assert np.all(cls_gpu == 1)
            np.testing.assert_allclose(stats[:, 2], sigma, rtol=REL)
        else:
            one = g.reshape(1, 1, N * C * H, W)
            _, mean_l, sigma_l, _ = O.channel_stats(one)
            np.testing.assert_allclose(stats[:, 2], np.full(C, sigma_l[0]), rtol=REL)
            assert np.all(stats[:, 2] == stats[0, 2])
            cnt = O.density_count(one, stats[:1, 2])                 # given the GPU's sigma of the layer
            np.testing.assert_array_equal(stats[:, 3], np.full(C, np.float32(float(cnt[0]) / (M * C))))
            s_or, cls_or = O.classify_clip(cnt, np.array([gl], np.float32), M * C, s_prev=None if s_prev is None else s_prev[:1])
            assert np.all(cls_gpu == cls_or[0])
            np.testing.assert_allclose(s_gpu, np.full(C, s_or[0]), rtol=REL)
            assert np.all(s_gpu == s_gpu[0])
            # end to end: unless the layer's count sits on the threshold, the oracle's own composition agrees
            if abs(float(cnt[0]) - 0.3 * M * C) > 2:
                s_e, cls_e, _ = O.grad_scales(g, "layer_mcs", s_prev=s_prev)
                assert np.all(cls_gpu == cls_e) and np.allclose(s_gpu, s_e, rtol=REL)
        np.testing.assert_array_equal(codes_to_nchw(gq.vq, C), O.quantize(g, s_gpu, True, 40 + t, 0))
        np.testing.assert_array_equal(codes_to_nchw(gq.gq, C), O.quantize(g, gl_gpu, True, 40 + t, 1))
        assert padding_is_zero(gq.vq, C) and padding_is_zero(gq.gq, C)
        s_prev = s_gpu
