"""Pins for the magnitude-weighted error model (Sec. 3.3): closed forms against quadrature and
brute-force minimisation (CPU only)."""
import numpy as np
import pytest

from oracle import emodel as E

CASES = [
    # a/b, eps, gmax, alpha
    (1000.0, 0.01, 1.0, 0.2),
    (200.0, 0.05, 1.0, 1.0),
    (50.0, 0.02, 2.0, 0.5),
]


def density(ratio, eps, gmax):
    # normalise so that 2*(a*eps + b*(gmax-eps)) = 1
    b = 0.5 / (ratio * eps + (gmax - eps))
    return ratio * b, b


@pytest.mark.parametrize("ratio,eps,gmax,alpha", CASES)
def test_printed_derivative_matches_quadrature(ratio, eps, gmax, alpha):
    """The closed-form dE/ds equals the central difference of Eq. 9 integrated numerically."""
    a, b = density(ratio, eps, gmax)
    p = E.inverted_t_density(a, b, eps, gmax)
    for s in np.linspace(eps * 1.5, gmax * 0.999, 7):
        h = 1e-5 * gmax
        num = (E.error_simplified(p, s + h, gmax, alpha, (eps,)) -
               E.error_simplified(p, s - h, gmax, alpha, (eps,))) / (2 * h)
        cf = E.dE_ds_inverted_t(float(s), a, b, eps, gmax, alpha)
        assert abs(num - cf) < 1e-6 * max(1.0, abs(cf)) + 1e-7


@pytest.mark.parametrize("ratio,eps,gmax,alpha", CASES)
def test_root_is_the_bruteforce_minimiser(ratio, eps, gmax, alpha):
    a, b = density(ratio, eps, gmax)
    p = E.inverted_t_density(a, b, eps, gmax)
    root = E.root_inverted_t(a, b, eps, gmax, alpha)
    assert eps < root <= gmax
    assert abs(E.dE_ds_inverted_t(root, a, b, eps, gmax, alpha)) < 1e-9
    s_best, _ = E.argmin_grid(lambda s: E.error_simplified(p, s, gmax, alpha, (eps,)),
                              eps * 1.01, gmax, 1201)
    assert abs(s_best - root) <= 1.5 * (gmax - eps * 1.01) / 1200


def test_alpha_to_zero_limit():
    for ratio, eps, gmax in [(200.0, 0.05, 1.0), (1000.0, 0.01, 1.0)]:
        a, b = density(ratio, eps, gmax)
        lim = E.root_inverted_t_alpha0(a, b, eps, gmax)
        assert abs(E.root_inverted_t(a, b, eps, gmax, 1e-6) - lim) < 1e-5
    # value worked by hand: (254 - 199*0.05)/256
    assert abs(E.root_inverted_t_alpha0(200.0, 1.0, 0.05, 1.0) - 244.05 / 256) < 1e-12


def test_clip_grows_with_alpha_inverted_t():
    """Eq. 12: the optimal s/|g|max does not decrease as alpha grows, and approaches 1."""
    a, b = density(1000.0, 0.01, 1.0)
    roots = [E.root_inverted_t(a, b, 0.01, 1.0, al) for al in (0.01, 0.2, 1.0, 3.0, 10.0)]
    assert all(x < y for x, y in zip(roots, roots[1:]))
    assert roots[0] < 0.96 and roots[-1] > 0.99 and roots[-1] <= 1.0


def test_clip_grows_with_alpha_on_gaussian_sample():
    """On a bell-shaped sample the brute-force minimiser of the true error (Eq. 8) sits below
    |g|max for alpha = 0 and moves to |g|max as alpha grows -- the reason Eq. 11 is reused."""
    rng = np.random.default_rng(20)
    g = rng.standard_normal(1568)
    gmax = np.abs(g).max()
    best = []
    for alpha in (0.0, 0.2, 1.0, 3.0):
        s, _ = E.argmin_grid(lambda s: E.error_sample(g, s, alpha), 0.3 * gmax, gmax, 141)
        best.append(s / gmax)
    assert all(x <= y + 1e-12 for x, y in zip(best, best[1:]))
    assert best[0] < 0.95 and best[-1] > 0.98


def test_error_sample_halves_step_in_range():
    """Assumption 2: for in-range uniform data the mean |g - g_hat| is a quarter step
    (uniform rounding error on [-step/2, step/2]); the bound is half a step."""
    rng = np.random.default_rng(21)
    g = rng.uniform(-1, 1, 200_000)
    e = E.error_sample(g, 1.0, 0.0)
    assert abs(e - 0.25 / 127) < 2e-5
