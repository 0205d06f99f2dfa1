"""Randomised property checks of the CPU oracle (hypothesis): the identities
that follow from Eq. 1-5 must hold for arbitrary small vectors, not only for
the hand-picked cases of the pins."""
import math

import numpy as np
from hypothesis import given, settings, strategies as st

from oracle import gac_oracle as orc

finite = st.floats(min_value=-64.0, max_value=64.0, allow_nan=False, allow_infinity=False, width=32)


def vec_pair(draw, n_min=2, n_max=24):
    n = draw(st.integers(n_min, n_max))
    g = np.array(draw(st.lists(finite, min_size=n, max_size=n)), dtype=np.float32)
    d = np.array(draw(st.lists(finite, min_size=n, max_size=n)), dtype=np.float32)
    return g, d


def fdot(a, b):
    return math.fsum(float(x) * float(y) for x, y in zip(a, b))


@settings(max_examples=150, deadline=None)
@given(st.data())
def test_cosine_is_bounded_symmetric_and_scale_invariant(data):
    g, d = vec_pair(data.draw)
    hp = orc.HParams(eps=0.0)
    c = orc.decide(orc.stats([g], [d]), hp).cos
    assert -1.0 - 1e-12 <= c <= 1.0 + 1e-12                       # Cauchy-Schwarz
    assert orc.decide(orc.stats([d], [g]), hp).cos == c            # Eq. 1 is symmetric
    assert orc.decide(orc.stats([-g], [d]), hp).cos == -c
    s = np.float32(2.0 ** data.draw(st.integers(-8, 8)))
    assert orc.decide(orc.stats([g * s], [d]), hp).cos == c        # power-of-two rescaling is exact


@settings(max_examples=150, deadline=None)
@given(st.data())
def test_projection_identities(data):
    g, d = vec_pair(data.draw)
    dd, gg, dot = fdot(d, d), fdot(g, g), fdot(g, d)
    if dd < 1e-3 or gg < 1e-3:
        return
    c_low = data.draw(st.floats(0.01, 0.4))
    hp = orc.HParams(c_low=c_low, c_high=1.5, eps=0.0)
    g1, d1 = g.copy(), d.copy()
    dec = orc.step([g1], [d1], hp)
    c = dot / math.sqrt(gg * dd)
    assert abs(dec.cos - c) <= 1e-12
    np.testing.assert_array_equal(d1, g)                           # state refresh in every regime
    if abs(c) <= c_low:
        assert dec.regime == orc.SAFE
        np.testing.assert_array_equal(g1, g)
        return
    assert dec.regime == orc.PROJECT
    alpha = c_low / abs(c)
    scale = math.sqrt(gg * dd)
    tol = 4e-7 * scale                                             # binary32 coefficient and outputs
    assert abs(fdot(g1, d) - alpha * dot) <= tol                   # parallel part scaled by alpha (Eq. 5)
    assert abs(fdot(g1, g1) - gg * (1 - c * c + c_low * c_low)) <= 4e-7 * gg + 1e-6
    # g' - g is a multiple of d (rank-one update, App. A.2)
    diff = g1.astype(np.float64) - g
    k = fdot(diff, d) / dd
    assert float(np.abs(diff - k * d).max()) <= 2e-7 * (float(np.abs(g).max()) + abs(k) * float(np.abs(d).max()))
    assert abs(k - dec.coef) <= 2e-7 * abs(dec.coef) + 1e-7


@settings(max_examples=100, deadline=None)
@given(st.data())
def test_full_projection_is_orthogonal_and_idempotent(data):
    g, d = vec_pair(data.draw)
    if fdot(d, d) < 1e-3:
        return
    hp = orc.HParams(mode=orc.MODE_FIXED, alpha_fixed=0.0, eps=0.0, state_mode=orc.STATE_HOLD)
    g1, d1 = g.copy(), d.copy()
    orc.step([g1], [d1], hp)
    scale = math.sqrt(fdot(g, g) * fdot(d, d)) + 1e-30
    assert abs(fdot(g1, d)) <= 4e-7 * scale
    g2 = g1.copy()
    orc.step([g2], [d1], hp)
    assert float(np.abs(g2 - g1).max()) <= 4e-7 * (float(np.abs(g).max()) + 1e-30)
