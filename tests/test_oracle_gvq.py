"""Pins for the oracle's statistics, discriminator, clip update and quantizers (CPU only).

Each test checks the oracle against something other than itself: a library routine, a closed form,
a brute-force loop, an invariant from the paper, or a constant the paper prints.
"""
import math
import os

import numpy as np
import pytest

from oracle import cpu as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_constants.txt")


def paper_constants():
    out = {}
    with open(GOLDEN) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                k, v = line.split()
                out[k] = float(v)
    return out


def test_defaults_are_the_papers():
    c = paper_constants()
    import inspect
    sig = inspect.signature(O.classify_clip)
    assert sig.parameters["lam"].default == c["lambda"]
    assert sig.parameters["k"].default == c["k"]
    assert sig.parameters["A"].default == c["A"]


# ------------------------------------------------------------------ statistics (Algorithm 1)
@pytest.mark.parametrize("shape", [(2, 3, 5, 7), (8, 64, 14, 14), (1, 1, 1, 1), (3, 5, 1, 9)])
def test_stats_match_numpy(shape):
    rng = np.random.default_rng(1)
    g = (rng.standard_normal(shape) * 1e-4 + 3e-5).astype(np.float32)
    absmax, mean, sigma, gl = O.channel_stats(g)
    g64 = g.astype(np.float64).transpose(1, 0, 2, 3).reshape(shape[1], -1)
    np.testing.assert_array_equal(absmax, np.abs(g).transpose(1, 0, 2, 3).reshape(shape[1], -1).max(1))
    np.testing.assert_allclose(mean, g64.mean(1), rtol=1e-6, atol=1e-12)
    np.testing.assert_allclose(sigma, g64.std(1, ddof=0), rtol=1e-6, atol=0)
    assert gl == absmax.max()


def test_stats_flags():
    rng = np.random.default_rng(2)
    g = (rng.standard_normal((4, 3, 6, 6)) + 0.7).astype(np.float32)
    g64 = g.astype(np.float64).transpose(1, 0, 2, 3).reshape(3, -1)
    _, _, s_unb, _ = O.channel_stats(g, std_unbiased=True)
    np.testing.assert_allclose(s_unb, g64.std(1, ddof=1), rtol=1e-6)
    _, _, s_rms, _ = O.channel_stats(g, center_mean=False)
    np.testing.assert_allclose(s_rms, np.sqrt((g64 ** 2).mean(1)), rtol=1e-6)
    # the mean shift matters: centred sigma ~1, rms ~1.22
    _, _, s_c, _ = O.channel_stats(g)
    assert np.all(s_rms > s_c * 1.1)


def test_stats_channel_major_not_sample_major():
    # a transposed-index mistake (reducing over C instead of N,H,W) must fail here
    g = np.zeros((2, 3, 2, 2), np.float32)
    g[:, 1] = 5.0
    g[1, 2, 0, 0] = -9.0
    absmax, mean, sigma, gl = O.channel_stats(g)
    np.testing.assert_array_equal(absmax, [0.0, 5.0, 9.0])
    np.testing.assert_allclose(mean, [0.0, 5.0, -9.0 / 8])
    assert sigma[1] == 0.0 and gl == 9.0


# ------------------------------------------------------------------ density (Algorithm 1)
def test_density_bruteforce_and_strictness():
    g = np.array([0.0, 1.0, -1.0, 2.0, -3.0, 0.5], np.float32).reshape(1, 1, 1, 6)
    assert O.density_count(g, np.array([1.0], np.float32))[0] == 2       # strict '>' on |g|
    assert O.density_count(g, np.array([0.0], np.float32))[0] == 5
    rng = np.random.default_rng(3)
    g = rng.standard_normal((3, 4, 5, 6)).astype(np.float32)
    sig = np.array([0.5, 1.0, 1.5, 0.1], np.float32)
    want = [(np.abs(g[:, c]) > sig[c]).sum() for c in range(4)]
    np.testing.assert_array_equal(O.density_count(g, sig), want)


def test_density_closed_forms():
    """P(|g| > sigma): Gaussian erfc(1/sqrt 2) = 0.3173 ("more than 30%", Sec. 3.4), Laplace
    exp(-sqrt 2) = 0.2431, uniform 1 - 1/sqrt 3 = 0.4226."""
    c = paper_constants()
    rng = np.random.default_rng(4)
    M = 400_000
    g = np.empty((1, 3, 1, M), np.float32)
    g[0, 0, 0] = rng.standard_normal(M) * 3e-5
    g[0, 1, 0] = rng.laplace(0, 3e-5, M)
    g[0, 2, 0] = rng.uniform(-2e-4, 2e-4, M)
    _, _, sigma, _ = O.channel_stats(g)
    P = O.density_count(g, sigma) / M
    se = 3 * math.sqrt(0.25 / M) * 2
    assert abs(P[0] - math.erfc(1 / math.sqrt(2))) < se
    assert abs(P[1] - math.exp(-math.sqrt(2))) < se
    assert abs(P[2] - (1 - 1 / math.sqrt(3))) < se
    assert P[0] > c["gaussian_outside_sigma_min"] > P[1]
    s, cls = O.classify_clip(O.density_count(g, sigma), np.abs(g).max(axis=(0, 2, 3)), M)
    np.testing.assert_array_equal(cls, [1, 0, 1])


# ------------------------------------------------------------------ discriminator + clip
def test_classify_threshold_is_strict_and_on_lambda():
    M = 1000
    absmax = np.ones(4, np.float32)
    cnt = np.array([299, 300, 301, 1000], np.uint32)
    s, cls = O.classify_clip(cnt, absmax, M)
    # lambda = float32(0.3) = 0.300000011920929 -> 300.0000119 ; 300 is not greater
    np.testing.assert_array_equal(cls, [0, 0, 1, 1])
    s, cls = O.classify_clip(cnt, absmax, M, lam=0.5)
    np.testing.assert_array_equal(cls, [0, 0, 0, 1])


def test_clip_rule_values():
    absmax = np.array([2.0, 2.0, 0.5], np.float32)
    cnt = np.array([900, 100, 100], np.uint32)       # channel 0 bell-shaped, others Inverted-T
    prev = np.array([7.0, 1.0, 1.0], np.float32)
    s, cls = O.classify_clip(cnt, absmax, 1000, s_prev=prev)
    np.testing.assert_array_equal(cls, [1, 0, 0])
    # Eq. 11: s = |g|max ; Eq. 14 with k=1, A=0.8: s = 0.2*s_prev + 0.8*gmax
    np.testing.assert_allclose(s, [2.0, 0.2 * 1.0 + 0.8 * 2.0, 0.2 * 1.0 + 0.8 * 0.5], rtol=1e-6)
    # other hyper-parameters of the sensitivity table: k=1.5, A=0.5 -> (1-0.75) s_prev + 0.5 gmax
    s, _ = O.classify_clip(cnt, absmax, 1000, s_prev=prev, k=1.5, A=0.5)
    np.testing.assert_allclose(s[1:], [0.25 + 1.0, 0.25 + 0.25], rtol=1e-6)
    # first iteration: s_prev := gmax, so k = 1 returns gmax itself
    s, _ = O.classify_clip(cnt, absmax, 1000, s_prev=None)
    np.testing.assert_allclose(s, absmax, rtol=1e-6)


def test_clip_recurrence_closed_form():
    """Eq. 14 unrolled: s_t = (1-kA)^t s_0 + A sum_j (1-kA)^(t-1-j) gmax_j; constant gmax -> gmax/k."""
    rng = np.random.default_rng(5)
    for k, A in [(1.0, 0.8), (1.2, 0.5), (1.5, 0.8)]:
        T = 40
        gmax = rng.uniform(0.5, 2.0, T)
        s = np.array([1.3], np.float32)
        for t in range(T):
            s, cls = O.classify_clip(np.array([0], np.uint32), np.array([gmax[t]], np.float32), 10,
                                     s_prev=s, k=k, A=A)
            assert cls[0] == 0
        r = 1.0 - k * A
        want = r ** T * 1.3 + A * sum(r ** (T - 1 - j) * gmax[j] for j in range(T))
        assert abs(float(s[0]) - want) < 1e-5 * abs(want)
        s = np.array([5.0], np.float32)
        for t in range(200):
            s, _ = O.classify_clip(np.array([0], np.uint32), np.array([2.0], np.float32), 10,
                                   s_prev=s, k=k, A=A)
        assert abs(float(s[0]) - 2.0 / k) < 1e-5


def test_state_written_in_both_branches():
    s, cls = O.classify_clip(np.array([10, 0], np.uint32), np.array([3.0, 3.0], np.float32), 10,
                             s_prev=np.array([1.0, 1.0], np.float32))
    assert cls.tolist() == [1, 0] and s[0] == 3.0 and abs(s[1] - 2.6) < 1e-6


# ------------------------------------------------------------------ quantizer (Eq. 1)
def test_nearest_values_and_ties_to_even():
    s = 127.0  # step 1: codes equal rounded values
    x = np.array([0.0, 0.49, 0.5, 1.5, 2.5, -0.5, -1.5, 126.5, 127.0, 300.0, -127.49, -1e9, 3.3],
                 np.float32).reshape(1, 1, 1, -1)
    q = O.quantize(x, s)
    np.testing.assert_array_equal(q.ravel(), [0, 0, 0, 2, 2, 0, -2, 126, 127, 127, -127, -127, 3])
    assert q.min() >= -127


def test_nearest_roundtrip_bound():
    """Assumption 2: in-range error at most half a step, s/254; clipped values map to +-s."""
    rng = np.random.default_rng(6)
    x = (rng.standard_normal((2, 4, 9, 9)) * 1e-4).astype(np.float32)
    s = np.array([1e-4, 2.5e-4, 4e-4, 1e-3], np.float32)
    q = O.quantize(x, s)
    xh = O.dequantize(q, s)
    for c in range(4):
        inr = np.abs(x[:, c]) <= s[c]
        err = np.abs(x[:, c].astype(np.float64) - xh[:, c])
        assert err[inr].max() <= s[c] / 254 * (1 + 1e-5)
        assert np.all(np.abs(xh[:, c][~inr]) == np.float32(127) * (s[c] / np.float32(127)))
        assert np.all(np.sign(xh[:, c][~inr]) == np.sign(x[:, c][~inr]))
    # per-channel scales really are per channel (channel 0 clips, channel 3 does not)
    assert (np.abs(q[:, 0]) == 127).mean() > 0.2 and (np.abs(q[:, 3]) == 127).mean() == 0
    # matches the formula evaluated by numpy in float64 away from ties
    v = 127.0 * np.clip(x[:, 1].astype(np.float64), -s[1], s[1]) / s[1]
    safe = np.abs(v - np.floor(v) - 0.5) > 1e-3
    np.testing.assert_array_equal(q[:, 1][safe], np.rint(v)[safe].astype(np.int8))


def test_zero_scale_gives_zero_codes():
    x = np.zeros((1, 2, 2, 2), np.float32)
    x[0, 1] = 1.0
    q = O.quantize(x, np.array([0.0, 1.0], np.float32))
    assert np.all(q[0, 0] == 0) and np.all(q[0, 1] == 127)
    assert np.all(O.quantize(x, np.array([0.0, 1.0], np.float32), stochastic=True, seed=3)[0, 0] == 0)


def test_uniform_generator():
    u = np.array([O.rand_uniform(11, 0, i) for i in range(20000)])
    v = np.array([O.rand_uniform(11, 1, i) for i in range(20000)])
    for a in (u, v):
        assert a.min() >= 0.0 and a.max() < 1.0
        assert abs(a.mean() - 0.5) < 4 * math.sqrt(1 / 12 / a.size)
        hist = np.histogram(a, bins=16, range=(0, 1))[0]
        chi2 = ((hist - a.size / 16) ** 2 / (a.size / 16)).sum()
        assert chi2 < 45  # 15 dof, p ~ 1e-4
    assert abs(np.corrcoef(u, v)[0, 1]) < 0.03
    assert abs(np.corrcoef(u[:-1], u[1:])[0, 1]) < 0.03
    # depends on seed, stream and on both halves of the 64-bit index
    assert O.rand_bits(1, 0, 5) != O.rand_bits(2, 0, 5)
    assert O.rand_bits(1, 0, 5) != O.rand_bits(1, 1, 5)
    assert O.rand_bits(1, 0, 5) != O.rand_bits(1, 0, 5 + (1 << 32))
    # multiples of 2^-23
    assert all(float(x * 2 ** 23).is_integer() for x in u[:100])


def test_uniform_generator_pairs_and_strides():
    """Joint behaviour, which stochastic rounding of neighbouring elements depends on: pairs at lag 1,
    pairs one channel apart at the same pixel (lag H*W of an NCHW index), the two streams of one
    element, and the sub-sequence a single pixel column sees (stride H*W) -- 16 x 16 chi-square
    (255 degrees of freedom: mean 255, s.d. 22.6) and correlations."""
    n = 1 << 18
    for seed in (11, 12345):
        bits0 = np.array([O.rand_bits(seed, 0, i) for i in range(n)], dtype=np.uint32)
        bits1 = np.array([O.rand_bits(seed, 1, i) for i in range(n)], dtype=np.uint32)
        u, v = (bits0 >> 9) * 2.0 ** -23, (bits1 >> 9) * 2.0 ** -23

        def chi2(a, b):
            h = np.histogram2d(a, b, bins=16, range=((0, 1), (0, 1)))[0]
            e = a.size / 256
            return ((h - e) ** 2 / e).sum()

        for lag in (1, 49, 196, 3136, 12544):
            assert chi2(u[:-lag], u[lag:]) < 255 + 5 * 22.6, lag
            assert abs(np.corrcoef(u[:-lag], u[lag:])[0, 1]) < 4 / math.sqrt(n)
            assert abs(np.corrcoef(u[:-lag], v[lag:])[0, 1]) < 4 / math.sqrt(n)
        assert chi2(u, v) < 255 + 5 * 22.6
        # low-order bits of u (they decide the rounding of values close to an integer)
        w = (u * 4096) % 1
        hist = np.histogram(w, bins=16, range=(0, 1))[0]
        assert ((hist - n / 16) ** 2 / (n / 16)).sum() < 45
        us = np.array([O.rand_uniform(seed, 0, k * 3136) for k in range(1 << 15)])
        assert abs(np.corrcoef(us[:-1], us[1:])[0, 1]) < 4 / math.sqrt(us.size)
        assert abs(us.mean() - 0.5) < 4 * math.sqrt(1 / 12 / us.size)


def test_stochastic_rounding_properties():
    """SR picks floor or ceil, is unbiased, saturates at +-127 and errs by less than one step."""
    rng = np.random.default_rng(7)
    s = 127.0
    x = rng.uniform(-130, 130, size=(4, 2, 50, 50)).astype(np.float32)
    q = O.quantize(x, s, stochastic=True, seed=9).astype(np.int32)
    xc = np.clip(x, -127, 127)
    assert np.all((q == np.floor(xc)) | (q == np.ceil(xc)))
    assert q.max() == 127 and q.min() == -127
    assert np.abs(q - xc).max() < 1.0
    # unbiased: average code over many seeds approaches the value; z-test on a fixed fraction
    x0 = np.full((1, 1, 200, 200), 3.3, np.float32)
    m = O.quantize(x0, s, stochastic=True, seed=1).astype(np.float64).mean()
    assert abs(m - 3.3) < 5 * math.sqrt(0.3 * 0.7 / x0.size)
    # same seed reproduces, other seed / stream differs
    a = O.quantize(x, s, stochastic=True, seed=9)
    b = O.quantize(x, s, stochastic=True, seed=10)
    c = O.quantize(x, s, stochastic=True, seed=9, stream=1)
    assert np.array_equal(a, q.astype(np.int8)) and not np.array_equal(a, b) and not np.array_equal(a, c)
    # exact integers are never moved
    xi = rng.integers(-127, 128, size=(1, 1, 10, 10)).astype(np.float32)
    np.testing.assert_array_equal(O.quantize(xi, s, stochastic=True, seed=4), xi.astype(np.int8))


def test_stochastic_matches_definition_elementwise():
    """q = min(127, floor(clamp(x*inv) + u(index))) recomputed in numpy from rand_uniform."""
    rng = np.random.default_rng(8)
    x = (rng.standard_normal((2, 3, 4, 5)) * 2e-4).astype(np.float32)
    sc = np.array([3e-4, 5e-4, 2e-4], np.float32)
    q = O.quantize(x, sc, stochastic=True, seed=77, stream=1)
    flat = x.reshape(-1)
    want = np.empty(flat.size, np.int8)
    for i in range(flat.size):
        c = (i // 20) % 3
        inv = np.float32(127.0) / sc[c]
        v = np.float32(flat[i] * inv)
        v = min(max(v, np.float32(-127)), np.float32(127))
        u = np.float32(O.rand_uniform(77, 1, i))
        want[i] = min(127, math.floor(np.float32(v + u)))
    np.testing.assert_array_equal(q.reshape(-1), want)


def test_layout_of_global_vs_vector_scale():
    x = np.arange(-8, 8, dtype=np.float32).reshape(1, 4, 2, 2)
    qg = O.quantize(x, 8.0)
    np.testing.assert_array_equal(qg.ravel(), np.rint(np.arange(-8, 8) * 127 / 8.0).clip(-127, 127))
    qv = O.quantize(x, np.abs(x).max(axis=(0, 2, 3)))
    assert np.all(np.abs(qv).max(axis=(0, 2, 3)) == 127)


def test_quantize_slice_of_a_larger_tensor():
    """first_image only moves the generator's counter: the codes of images 2..3 of a tensor equal the
    codes of those two images quantized on their own with first_image = 2, and differ without it."""
    rng = np.random.default_rng(3)
    x = rng.standard_normal((4, 5, 3, 7)).astype(np.float32)
    s = np.abs(x).max(axis=(0, 2, 3))
    whole = O.quantize(x, s, True, 11, 0)
    part = O.quantize(x[2:4], s, True, 11, 0, first_image=2)
    np.testing.assert_array_equal(whole[2:4], part)
    assert np.any(O.quantize(x[2:4], s, True, 11, 0) != part)
    # beyond 2^32 elements the high half of the index enters the key: one element against the scalar generator
    big = O.quantize(x[:1, :1, :1, :1], s[:1], True, 11, 1, first_image=1 << 33)
    u = O.rand_uniform(11, 1, (1 << 33) * 5 * 21)
    v = np.float32(np.float32(x[0, 0, 0, 0]) * np.float32(np.float32(127.0) / s[0]))
    assert int(big[0, 0, 0, 0]) == min(127, int(np.floor(np.float32(v + np.float32(u)))))


def test_ablation_modes_reduce_to_the_definitions():
    """The strategies of the ablation study (Sec. 4.1) as compositions of the pinned steps: checked on
    cases where each reduces to something known."""
    rng = np.random.default_rng(21)
    g = (rng.standard_normal((3, 4, 5, 6)) * np.array([1e-3, 2e-4, 5e-5, 1e-5])[None, :, None, None]).astype(np.float32)
    absmax = np.abs(g).max(axis=(0, 2, 3))
    # GQ: one scale, the layer's |g|max; its codes are the layer-wide quantizer's
    s, cls, gl = O.grad_scales(g, "gq")
    assert gl == absmax.max() and np.all(s == gl) and np.all(cls == 1)
    np.testing.assert_array_equal(O.quantize(g, s), O.quantize(g, float(gl)))
    # per-channel max without the discriminator = the full method when no density can fall below the threshold
    s, cls, _ = O.grad_scales(g, "gvq_max")
    np.testing.assert_array_equal(s, absmax)
    s_full, cls_full, _ = O.grad_scales(g, "full", lam=-1.0)
    np.testing.assert_array_equal(s, s_full)
    assert np.all(cls_full == 1)
    # layer-wise MCS on a one-channel tensor is the full method
    one = g[:, :1]
    for prev in (None, np.array([3e-3], np.float32)):
        a = O.grad_scales(one, "layer_mcs", s_prev=prev)
        b = O.grad_scales(one, "full", s_prev=prev)
        np.testing.assert_array_equal(a[0], b[0]); np.testing.assert_array_equal(a[1], b[1])
    # a long-tailed layer: density against numpy's std of ALL elements, Eq. 14 by hand
    lap = rng.laplace(0.0, 1e-4, size=(4, 3, 20, 20)).astype(np.float32)
    sigma_l = np.float32(np.std(lap.astype(np.float64)))
    P = np.mean(np.abs(lap) > sigma_l)
    assert P < 0.3
    s, cls, gl = O.grad_scales(lap, "layer_mcs", s_prev=np.full(3, 2e-4, np.float32))
    want = np.float32(np.float32(np.float32(1.0) - np.float32(1.0) * np.float32(0.8)) * np.float32(2e-4)) + np.float32(np.float32(0.8) * np.float32(gl))
    assert np.all(cls == 0) and np.all(s == np.float32(want))
    # a bell-shaped layer whose channels differ in width by decades is NOT bell-shaped as a whole: the
    # layer-wise rule clips where the per-channel rule does not (the reason for GVQ + per-channel MCS)
    s_l, cls_l, _ = O.grad_scales(g, "layer_mcs")
    s_c, cls_c, _ = O.grad_scales(g, "full")
    assert np.all(cls_l == 0) and cls_c.sum() >= 3
