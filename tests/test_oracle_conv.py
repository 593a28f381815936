"""Pins for the oracle's integer convolutions and de-quantization (CPU only)."""
import itertools

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import cpu as O

GEOMS = [
    # N, Cin, Cout, H, W, R, S, stride, pad
    (2, 3, 4, 5, 6, 3, 3, 1, 1),
    (1, 2, 3, 7, 7, 3, 3, 2, 1),
    (2, 4, 2, 6, 5, 1, 1, 1, 0),
    (1, 3, 2, 8, 8, 1, 1, 2, 0),
    (1, 1, 2, 9, 9, 7, 7, 2, 3),
    (2, 2, 2, 4, 4, 3, 3, 1, 0),
    (1, 2, 2, 5, 7, 3, 5, (1, 2), (1, 2)),
]


def rand_codes(rng, shape):
    return rng.integers(-127, 128, size=shape, dtype=np.int64).astype(np.int8)


def make(rng, g):
    N, Cin, Cout, H, W, R, S, st, pad = g
    P, Q = O.out_hw(H, W, R, S, st, pad)
    return (rand_codes(rng, (N, Cin, H, W)), rand_codes(rng, (Cout, Cin, R, S)),
            rand_codes(rng, (N, Cout, P, Q)))


def naive_fwd(X, Wt, st, pad):
    """Seven nested loops straight from the definition."""
    sh, sw = (st, st) if np.isscalar(st) else st
    ph, pw = (pad, pad) if np.isscalar(pad) else pad
    N, Cin, H, W = X.shape
    Cout, _, R, S = Wt.shape
    P, Q = O.out_hw(H, W, R, S, st, pad)
    Y = np.zeros((N, Cout, P, Q), np.int64)
    for n, co, p, q, ci, r, s in itertools.product(range(N), range(Cout), range(P), range(Q),
                                                   range(Cin), range(R), range(S)):
        h, w = p * sh + r - ph, q * sw + s - pw
        if 0 <= h < H and 0 <= w < W:
            Y[n, co, p, q] += int(X[n, ci, h, w]) * int(Wt[co, ci, r, s])
    return Y


@pytest.mark.parametrize("g", GEOMS[:4])
def test_fwd_matches_naive_loops(g):
    rng = np.random.default_rng(10)
    X, Wt, _ = make(rng, g)
    acc, ov = O.conv_fwd_acc(X, Wt, g[7], g[8])
    np.testing.assert_array_equal(acc, naive_fwd(X, Wt, g[7], g[8]))
    assert ov == 0


@pytest.mark.parametrize("g", GEOMS)
def test_all_three_match_torch_float64(g):
    """torch's CPU conv2d and its autograd gradients in float64 are exact on small integers."""
    rng = np.random.default_rng(11)
    X, Wt, G = make(rng, g)
    st, pad = g[7], g[8]
    x = torch.tensor(X.astype(np.float64), requires_grad=True)
    w = torch.tensor(Wt.astype(np.float64), requires_grad=True)
    y = F.conv2d(x, w, stride=st, padding=pad)
    y.backward(torch.tensor(G.astype(np.float64)))
    acc, _ = O.conv_fwd_acc(X, Wt, st, pad)
    np.testing.assert_array_equal(acc, y.detach().numpy().astype(np.int64))
    dx, _ = O.conv_bwd_data_acc(G, Wt, (g[3], g[4]), st, pad)
    np.testing.assert_array_equal(dx, x.grad.numpy().astype(np.int64))
    dw, _ = O.conv_bwd_filter_acc(X, G, (g[5], g[6]), st, pad)
    np.testing.assert_array_equal(dw, w.grad.numpy().astype(np.int64))


@pytest.mark.parametrize("g", GEOMS)
def test_adjoint_identity_is_exact(g):
    """<conv(X,W), G> = <X, G_X> = <W, G_W> holds exactly in integers (Eq. 3, Eq. 4)."""
    rng = np.random.default_rng(12)
    X, Wt, G = make(rng, g)
    st, pad = g[7], g[8]
    y, _ = O.conv_fwd_acc(X, Wt, st, pad)
    dx, _ = O.conv_bwd_data_acc(G, Wt, (g[3], g[4]), st, pad)
    dw, _ = O.conv_bwd_filter_acc(X, G, (g[5], g[6]), st, pad)
    lhs = int((y * G.astype(np.int64)).sum())
    assert lhs == int((dx * X.astype(np.int64)).sum()) == int((dw * Wt.astype(np.int64)).sum())


def test_pointwise_is_integer_matmul():
    rng = np.random.default_rng(13)
    N, Cin, Cout, H, W = 2, 5, 3, 4, 3
    X, Wt, G = make(rng, (N, Cin, Cout, H, W, 1, 1, 1, 0))
    Xm = X.astype(np.int64).transpose(0, 2, 3, 1).reshape(-1, Cin)
    Gm = G.astype(np.int64).transpose(0, 2, 3, 1).reshape(-1, Cout)
    Wm = Wt.astype(np.int64).reshape(Cout, Cin)
    y, _ = O.conv_fwd_acc(X, Wt)
    np.testing.assert_array_equal(y.transpose(0, 2, 3, 1).reshape(-1, Cout), Xm @ Wm.T)
    dx, _ = O.conv_bwd_data_acc(G, Wt, (H, W))
    np.testing.assert_array_equal(dx.transpose(0, 2, 3, 1).reshape(-1, Cin), Gm @ Wm)
    dw, _ = O.conv_bwd_filter_acc(X, G, (1, 1))
    np.testing.assert_array_equal(dw.reshape(Cout, Cin), Gm.T @ Xm)


def test_sampled_outputs_equal_full():
    rng = np.random.default_rng(14)
    g = (2, 3, 4, 6, 6, 3, 3, 2, 1)
    X, Wt, G = make(rng, g)
    full, _ = O.conv_fwd_acc(X, Wt, 2, 1)
    idx = rng.choice(full.size, 17, replace=False)
    samp, _ = O.conv_fwd_acc(X, Wt, 2, 1, idx=idx)
    np.testing.assert_array_equal(samp, full.reshape(-1)[idx])
    full, _ = O.conv_bwd_data_acc(G, Wt, (6, 6), 2, 1)
    idx = rng.choice(full.size, 17, replace=False)
    samp, _ = O.conv_bwd_data_acc(G, Wt, (6, 6), 2, 1, idx=idx)
    np.testing.assert_array_equal(samp, full.reshape(-1)[idx])
    full, _ = O.conv_bwd_filter_acc(X, G, (3, 3), 2, 1)
    idx = rng.choice(full.size, 17, replace=False)
    samp, _ = O.conv_bwd_filter_acc(X, G, (3, 3), 2, 1, idx=idx)
    np.testing.assert_array_equal(samp, full.reshape(-1)[idx])


def test_overflow_is_flagged():
    # K = 140000 products of 127*127 exceeds 2^31 - 1
    K = 140_000
    X = np.full((1, 1, 1, K), 127, np.int8)
    G = np.full((1, 1, 1, K), 127, np.int8)
    acc, ov = O.conv_bwd_filter_acc(X, G, (1, 1))
    assert acc.ravel()[0] == 127 * 127 * K and ov == 1
    acc, ov = O.conv_bwd_filter_acc(X[..., :1000], G[..., :1000], (1, 1))
    assert ov == 0


def test_dequant_acc():
    """Vectorized de-quantization (Eq. 7): acc * (s_x/127) * (s_i/127), one s_i per output channel."""
    acc = np.arange(-6, 6, dtype=np.int64).reshape(3, 2, 2, 1)
    out = O.dequant_acc(acc, 127.0, 127.0)                   # unit steps: identity
    np.testing.assert_array_equal(out, acc.astype(np.float32))
    s = np.array([127.0, 254.0, 12.7], np.float32)
    out = O.dequant_acc(acc, 63.5, s)
    want = acc.astype(np.float64) * 0.5 * (s.astype(np.float64) / 127).reshape(3, 1, 1, 1)
    np.testing.assert_allclose(out, want, rtol=1e-6)
    out = O.dequant_acc(acc, 2.0, 3.0)
    np.testing.assert_allclose(out, acc * (2.0 / 127) * (3.0 / 127), rtol=1e-6)


def test_quantized_conv_approximates_float_conv():
    """End to end on a tiny layer: de-quantized int8 results approach the float convolution
    gradients (coarse bound: this pins scale placement -- s_X with G_W, s_W with G_X)."""
    rng = np.random.default_rng(15)
    N, Cin, Cout, H, W = 2, 8, 4, 6, 6
    x = np.maximum(rng.standard_normal((N, Cin, H, W)), 0).astype(np.float32)
    w = (rng.standard_normal((Cout, Cin, 3, 3)) * 0.1).astype(np.float32)
    g = (rng.standard_normal((N, Cout, H, W)) * np.array([1e-3, 1e-5, 3e-4, 1e-6]).reshape(1, 4, 1, 1)
         ).astype(np.float32)
    sx, sw = float(np.abs(x).max()), float(np.abs(w).max())
    qx, qw = O.quantize(x, sx), O.quantize(w, sw)
    absmax, _, _, gl = O.channel_stats(g)
    vq = O.quantize(g, absmax)
    gq = O.quantize(g, gl)
    tx = torch.tensor(x.astype(np.float64), requires_grad=True)
    tw = torch.tensor(w.astype(np.float64), requires_grad=True)
    F.conv2d(tx, tw, padding=1).backward(torch.tensor(g.astype(np.float64)))
    dw = O.dequant_acc(O.conv_bwd_filter_acc(qx, vq, (3, 3), 1, 1)[0], sx, absmax)
    ref = tw.grad.numpy()
    for co in range(Cout):      # per-channel scales keep every channel accurate
        assert np.abs(dw[co] - ref[co]).max() < 0.03 * np.abs(ref[co]).max()
    dx = O.dequant_acc(O.conv_bwd_data_acc(gq, qw, (H, W), 1, 1)[0], gl, sw)
    assert np.abs(dx - tx.grad.numpy()).max() < 0.03 * np.abs(tx.grad.numpy()).max()
    # the layer-wide scale drowns the small channels (the paper's motivation for GVQ)
    assert np.all(gq[:, 3] == 0) and np.abs(vq[:, 3]).max() == 127


def _codes(rng, shape):
    return rng.integers(-127, 128, size=shape, dtype=np.int64).astype(np.int8)


@pytest.mark.parametrize("geom", [
    # N, Cin, Cout, D, H, W, T, R, S, stride, pad, groups
    (2, 4, 6, 5, 6, 7, 3, 3, 3, 1, 1, 1),                       # 3-D convolution, Sec. 4.4
    (1, 3, 5, 6, 7, 5, 3, 1, 3, (2, 1, 2), (1, 0, 1), 1),        # strides and paddings that differ per axis
    (2, 6, 6, 1, 7, 8, 1, 3, 3, 1, 1, 6),                        # depth-wise 2-D, Sec. 4.2
    (1, 8, 8, 1, 9, 9, 1, 3, 3, 2, 1, 8),                        # depth-wise, stride 2
    (2, 4, 8, 3, 5, 5, 2, 3, 3, 1, (0, 1, 1), 2),                # two groups with a depth tap
])
def test_conv3_against_torch_and_adjoint_identity(geom):
    """The depth / group generalisation against torch's float64 convNd (exact on small integers) and
    its autograd gradients, plus the exact integer adjoint identity <Y,G> = <X,dX> = <W,dW>."""
    import torch
    N, Cin, Cout, D, H, W, T, R, S, stride, pad, groups = geom
    rng = np.random.default_rng(17)
    st = (stride,) * 3 if np.isscalar(stride) else stride
    pd = (pad,) * 3 if np.isscalar(pad) else pad
    Do, P, Q = O.out_dhw(D, H, W, T, R, S, st, pd)
    X, Wt, G = _codes(rng, (N, Cin, D, H, W)), _codes(rng, (Cout, Cin // groups, T, R, S)), _codes(rng, (N, Cout, Do, P, Q))
    y, o1 = O.conv3_acc("fwd", X, Wt, geom)
    dx, o2 = O.conv3_acc("bwd_data", G, Wt, geom)
    dw, o3 = O.conv3_acc("bwd_filter", X, G, geom)
    assert o1 == o2 == o3 == 0
    tx = torch.tensor(X, dtype=torch.float64, requires_grad=True)
    tw = torch.tensor(Wt, dtype=torch.float64, requires_grad=True)
    ty = torch.nn.functional.conv3d(tx, tw, stride=st, padding=pd, groups=groups)
    ty.backward(torch.tensor(G, dtype=torch.float64))
    np.testing.assert_array_equal(y, ty.detach().numpy().astype(np.int64))
    np.testing.assert_array_equal(dx, tx.grad.numpy().astype(np.int64))
    np.testing.assert_array_equal(dw, tw.grad.numpy().astype(np.int64))
    lhs = int((y * G.astype(np.int64)).sum())
    assert lhs == int((dx * X.astype(np.int64)).sum()) == int((dw * Wt.astype(np.int64)).sum())
    # sampled outputs equal the full ones
    idx = rng.choice(y.size, 20, replace=False)
    np.testing.assert_array_equal(O.conv3_acc("fwd", X, Wt, geom, idx=idx)[0], y.reshape(-1)[idx])


def test_conv3_reduces_to_the_2d_functions():
    """Depth 1, one group: the generalised loops are the 2-D ones (which have their own pins)."""
    rng = np.random.default_rng(18)
    X, Wt = _codes(rng, (2, 5, 9, 8)), _codes(rng, (7, 5, 3, 3))
    P, Q = O.out_hw(9, 8, 3, 3, 2, 1)
    G = _codes(rng, (2, 7, P, Q))
    geom = (2, 5, 7, 1, 9, 8, 1, 3, 3, (1, 2, 2), (0, 1, 1), 1)
    np.testing.assert_array_equal(O.conv3_acc("fwd", X[:, :, None], Wt[:, :, None], geom)[0][:, :, 0], O.conv_fwd_acc(X, Wt, 2, 1)[0])
    np.testing.assert_array_equal(O.conv3_acc("bwd_data", G[:, :, None], Wt[:, :, None], geom)[0][:, :, 0],
                                  O.conv_bwd_data_acc(G, Wt, (9, 8), 2, 1)[0])
    np.testing.assert_array_equal(O.conv3_acc("bwd_filter", X[:, :, None], G[:, :, None], geom)[0][:, :, 0],
                                  O.conv_bwd_filter_acc(X, G, (3, 3), 2, 1)[0])
