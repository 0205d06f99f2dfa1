"""Pins the CPU oracle to what the paper and mathematics fix, before it is
trusted as the arbiter of the CUDA library.  Nothing here touches a GPU.

Each test is chosen so that one plausible mistake in the oracle (a dropped
term, a wrong sign, eps in the wrong place, an exclusive threshold, a
transposed operand, double rounding) makes it fail.
"""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import gac_oracle as orc
from paper_2603_01501_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")
REGIME = {"SAFE": orc.SAFE, "PROJECT": orc.PROJECT, "VIOLATION": orc.VIOLATION}


def f32(*xs):
    return np.array(xs, dtype=np.float32)


def dot64(a, b):
    return math.fsum(float(x) * float(y) for x, y in zip(a, b))


# ---------------------------------------------------------------- golden files

def _rows(name):
    with open(os.path.join(GOLD, name)) as fh:
        for line in fh:
            line = line.strip()
            if line and not line.startswith("#"):
                yield [c.strip() for c in line.split("|")]


@pytest.mark.parametrize("row", list(_rows("worked_examples.txt")), ids=lambda r: r[0])
def test_worked_examples(row):
    name, thr, d, g, sums, cos, regime, alpha, coef, g_out, d_out = row
    c_low, c_high = map(float, thr.split())
    d = f32(*map(float, d.split()))
    g = f32(*map(float, g.split()))
    hp = orc.HParams(c_low=c_low, c_high=c_high, eps=0.0)
    s = orc.stats([g], [d])
    assert list(s) == list(map(float, sums.split()))
    dec = orc.decide(s, hp)
    assert dec.cos == pytest.approx(float(cos), rel=1e-15, abs=0)
    assert dec.regime == REGIME[regime]
    assert dec.alpha == pytest.approx(float(alpha), rel=1e-15)
    assert dec.coef64 == pytest.approx(float(coef), rel=1e-15, abs=0)
    # the coefficient is rounded once to binary32 (relative 2^-24) before it multiplies d
    atol = 2.0 ** -24 * abs(dec.coef) * float(np.abs(d).max())
    orc.project([g], [d], hp, dec)
    np.testing.assert_allclose(g, np.array(g_out.split(), dtype=np.float64), rtol=6e-8, atol=atol)
    assert d.tolist() == list(map(float, d_out.split()))


@pytest.mark.parametrize("row", list(_rows("decision_scalars.txt")), ids=lambda r: r[0])
def test_decision_scalars(row):
    ins, cos, regime, alpha = row
    dot, gg, dd, c_low, c_high, eps = map(float, ins.split())
    dec = orc.decide((dot, gg, dd), orc.HParams(c_low=c_low, c_high=c_high, eps=eps))
    assert dec.cos == pytest.approx(float(cos), rel=1e-14, abs=0)
    assert dec.regime == REGIME[regime]
    assert dec.alpha == pytest.approx(float(alpha), rel=1e-9)


# ------------------------------------------------- summation against exact sums

@pytest.mark.parametrize("n", [1, 7, 8, 9, 1000, 65537])
def test_stats_match_exactly_rounded_sums(n):
    rng = np.random.default_rng(n)
    g = (rng.standard_normal(n) * 10.0 ** rng.uniform(-6, 3, n)).astype(np.float32)
    d = (rng.standard_normal(n) * 10.0 ** rng.uniform(-6, 3, n)).astype(np.float32)
    want = (dot64(g, d), dot64(g, g), dot64(d, d))       # math.fsum: exactly rounded
    got = orc.stats([g], [d])
    pw = orc.stats_pairwise([g], [d])
    scale = math.sqrt(want[1] * want[2])
    for k in range(3):
        ref = max(abs(want[k]), 1e-16 * scale)
        assert abs(got[k] - want[k]) <= 4e-16 * ref + 1e-30
        assert abs(pw[k] - want[k]) <= 1e-13 * max(abs(want[k]), scale if k == 0 else 0)


def test_stats_survive_cancellation():
    # sum = 1 exactly, but a plain left-to-right double sum of the products loses it
    g = f32(2.0 ** 40, 1.0, -(2.0 ** 40), 2.0 ** -20) * 1
    d = f32(2.0 ** 40, 1.0, 2.0 ** 40, 0.0)
    dot, gg, dd = orc.stats([g], [d])
    assert dot == 1.0
    assert gg == 2.0 ** 81 + 1.0 + 2.0 ** -40 or gg == pytest.approx(2.0 ** 81, rel=1e-15)
    assert dd == 2.0 ** 81 + 1.0 or dd == pytest.approx(2.0 ** 81, rel=1e-15)


def test_stats_is_not_symmetric_mixup():
    # distinguishes <g,g> from <d,d> and <g,d>: g and d have different norms
    g, d = f32(1, 2, 3), f32(4, 5, 6)
    assert orc.stats([g], [d]) == (32.0, 14.0, 77.0)


def test_stats_agree_with_numpy_dot():
    rng = np.random.default_rng(5)
    g = rng.standard_normal(300_000).astype(np.float32)
    d = rng.standard_normal(300_000).astype(np.float32)
    got = orc.stats([g], [d])
    g64, d64 = g.astype(np.float64), d.astype(np.float64)
    for a, b in zip(got, (np.dot(g64, d64), np.dot(g64, g64), np.dot(d64, d64))):
        assert a == pytest.approx(b, rel=1e-12, abs=1e-9)


def test_list_is_the_flat_concatenation():
    rng = np.random.default_rng(11)
    flat_g = rng.standard_normal(5000).astype(np.float32)
    flat_d = rng.standard_normal(5000).astype(np.float32)
    cuts = [0, 1, 2, 259, 260, 3001, 5000]
    gl = [flat_g[a:b].copy() for a, b in zip(cuts, cuts[1:])]
    dl = [flat_d[a:b].copy() for a, b in zip(cuts, cuts[1:])]
    assert orc.stats(gl, dl) == orc.stats([flat_g], [flat_d])
    thr = orc.stats(gl, dl, threads=3)
    for a, b in zip(thr, orc.stats([flat_g], [flat_d])):
        assert a == pytest.approx(b, rel=1e-15)


# ---------------------------------------------------------- closed forms, Eq. 1

@pytest.mark.parametrize("rho", [0.9, -0.4, 0.0, 0.999])
def test_cosine_by_construction(rho):
    s = 3.0
    g, d = synth.flat_pair_with_cosine(1 << 14, rho, s=s, seed=3)
    dot, gg, dd = orc.stats([g.numpy()], [d.numpy()])
    dec = orc.decide((dot, gg, dd), orc.HParams(eps=0.0))
    assert dec.cos == pytest.approx(rho, abs=2e-7)
    assert gg == pytest.approx(s * s, rel=1e-6)
    assert dot == pytest.approx(rho * s * math.sqrt(dd), rel=1e-6, abs=1e-6)


def test_special_cases():
    rng = np.random.default_rng(2)
    v = rng.standard_normal(1000).astype(np.float32)
    hp = orc.HParams(eps=0.0)
    assert orc.decide(orc.stats([v], [v.copy()]), hp).cos == pytest.approx(1.0, abs=1e-15)
    assert orc.decide(orc.stats([v], [-v]), hp).cos == pytest.approx(-1.0, abs=1e-15)
    z = np.zeros_like(v)
    dec = orc.decide(orc.stats([v], [z]), hp)
    assert (dec.cos, dec.regime, dec.coef) == (0.0, orc.SAFE, 0.0)
    dec = orc.decide(orc.stats([z], [v]), hp)
    assert (dec.cos, dec.regime) == (0.0, orc.SAFE)


def test_power_of_two_rescaling_changes_nothing():
    g, d = synth.flat_pair_with_cosine(4096, 0.2, seed=9)
    g, d = g.numpy(), d.numpy()
    hp = orc.HParams(c_low=0.05, c_high=0.3, eps=0.0)
    base = orc.decide(orc.stats([g], [d]), hp)
    assert base.regime == orc.PROJECT
    g1, d1 = g.copy(), d.copy()
    orc.project([g1], [d1], hp, base)
    for sg, sd in [(2.0 ** 7, 1.0), (1.0, 2.0 ** -9), (2.0 ** -3, 2.0 ** 5)]:
        g2, d2 = (g * np.float32(sg)).copy(), (d * np.float32(sd)).copy()
        dec = orc.decide(orc.stats([g2], [d2]), hp)
        assert (dec.cos, dec.regime, dec.alpha) == (base.cos, base.regime, base.alpha)
        orc.project([g2], [d2], hp, dec)
        np.testing.assert_array_equal(g2, g1 * np.float32(sg))   # exact scaling


# ---------------------------------------- the rule against Eq. 2-3 done exactly

def _decomposition_exact(g, d, alpha: Fraction, beta: Fraction):
    """Eq. 2-3 literally, in exact rational arithmetic: g_par = <g,u>u with
    u = d/|d|  (so g_par = (<g,d>/<d,d>) d),  g_perp = g - g_par,
    g' = alpha g_par + beta g_perp."""
    G = [Fraction(float(x)) for x in g]
    Dv = [Fraction(float(x)) for x in d]
    dot = sum(a * b for a, b in zip(G, Dv))
    dd = sum(b * b for b in Dv)
    par = [dot / dd * b for b in Dv]
    perp = [a - p for a, p in zip(G, par)]
    return [alpha * p + beta * q for p, q in zip(par, perp)]


@pytest.mark.parametrize("alpha,beta", [(0, 1), (Fraction(1, 4), 1), (Fraction(1, 2), Fraction(3, 2)),
                                        (2, 1), (1, 1)])
def test_fixed_gains_match_exact_decomposition(alpha, beta):
    rng = np.random.default_rng(17)
    g = rng.integers(-50, 50, 16).astype(np.float32) / np.float32(8)
    d = rng.integers(-50, 50, 16).astype(np.float32) / np.float32(4)
    want = _decomposition_exact(g, d, Fraction(alpha), Fraction(beta))
    hp = orc.HParams(mode=orc.MODE_FIXED, alpha_fixed=float(alpha), beta=float(beta), eps=0.0)
    dec = orc.step([g], [d], hp)
    assert dec.regime == orc.PROJECT
    tol = 3e-7 * max(abs(float(w)) for w in want) + 1e-7 * float(np.abs(d).max()) * abs(dec.coef)
    for got, w in zip(g, want):
        assert abs(float(got) - float(w)) <= tol


def test_adaptive_rule_matches_exact_decomposition():
    # Eq. 5: alpha = c_low/|c| is irrational in general, so alpha is rebuilt here from
    # exactly rounded sums (math.fsum) and the vector algebra of Eq. 2-3 is then done
    # exactly in rationals with that alpha.
    rng = np.random.default_rng(23)
    d = rng.integers(-9, 10, 12).astype(np.float32)
    g = (0.3 * d + rng.integers(-9, 10, 12)).astype(np.float32)
    g0, d0 = g.copy(), d.copy()
    hp = orc.HParams(c_low=0.05, c_high=0.99, eps=0.0)
    dec = orc.step([g], [d], hp)
    assert dec.regime == orc.PROJECT
    c = dot64(g0, d0) / math.sqrt(dot64(g0, g0) * dot64(d0, d0))
    assert dec.cos == pytest.approx(c, rel=1e-15)
    want = _decomposition_exact(g0, d0, Fraction(hp.c_low / abs(c)), Fraction(1))
    for got, w in zip(g, want):
        assert abs(float(got) - float(w)) <= 2e-7 * float(np.abs(g0).max())
    np.testing.assert_array_equal(d, g0)


def test_adaptive_invariants():
    """Identities that follow from Eq. 2-5 for beta=1, alpha=c_low/|c|:
    <g',d> = alpha <g,d>;  |g'|^2 = |g|^2 (1 - c^2 + c_low^2);
    cos(g',d) = sign(c) c_low / sqrt(1 - c^2 + c_low^2);  <g',w> = <g,w> for w orthogonal to d."""
    for rho in (0.2, -0.6, 0.9):
        g, d = synth.flat_pair_with_cosine(1 << 12, rho, s=2.0, seed=31)
        g, d = g.numpy(), d.numpy()
        w = np.random.default_rng(1).standard_normal(g.size)
        w -= dot64(w, d) / dot64(d, d) * d.astype(np.float64)
        g0, d0 = g.copy(), d.copy()
        hp = orc.HParams(c_low=0.05, c_high=0.95, eps=0.0)
        dec = orc.step([g], [d], hp)
        assert dec.regime == orc.PROJECT
        c, cl = dec.cos, hp.c_low
        assert dec.alpha == pytest.approx(cl / abs(rho), rel=1e-5)
        assert dot64(g, d0) == pytest.approx(dec.alpha * dec.dot, rel=2e-6)
        assert dot64(g, g) == pytest.approx(dec.gg * (1 - c * c + cl * cl), rel=2e-6)
        cos_after = dot64(g, d0) / math.sqrt(dot64(g, g) * dot64(d0, d0))
        assert cos_after == pytest.approx(math.copysign(cl, c) / math.sqrt(1 - c * c + cl * cl),
                                          rel=2e-6)
        assert dot64(g, w) == pytest.approx(dot64(g0, w), abs=1e-6 * math.sqrt(dec.gg * dot64(w, w)))
        # g' - g is parallel to d: one coefficient reproduces every element
        diff = g.astype(np.float64) - g0
        np.testing.assert_allclose(diff, dec.coef * d0.astype(np.float64),
                                   atol=1.2e-7 * float(np.abs(g0).max()) * 2)
        np.testing.assert_array_equal(d, g0)             # state = raw gradient


def test_full_projection_orthogonal_idempotent_pythagoras():
    g, d = synth.flat_pair_with_cosine(1 << 12, 0.7, s=5.0, seed=4)
    g, d = g.numpy(), d.numpy()
    d0 = d.copy()
    hp = orc.HParams(mode=orc.MODE_FIXED, alpha_fixed=0.0, beta=1.0, eps=0.0,
                     state_mode=orc.STATE_HOLD)
    dec = orc.step([g], [d], hp)
    np.testing.assert_array_equal(d, d0)                 # HOLD keeps the reference
    gg1 = dot64(g, g)
    # App. F, proof step 1: |P_perp b|^2 = |b|^2 - <b,d>^2/|d|^2
    assert gg1 == pytest.approx(dec.gg - dec.dot ** 2 / dec.dd, rel=1e-6)
    assert abs(dot64(g, d)) <= 1e-6 * math.sqrt(gg1 * dec.dd)
    g_once = g.copy()
    dec2 = orc.step([g], [d], hp)
    assert abs(dec2.cos) < 1e-6
    np.testing.assert_allclose(g, g_once, atol=2e-7 * float(np.abs(g_once).max()))


def test_transposed_operands_would_fail():
    # g' must move along d, not along g: with d=(0,1) and g=(1,1) full projection gives (1,0)
    g, d = f32(1, 1), f32(0, 1)
    orc.step([g], [d], orc.HParams(mode=orc.MODE_FIXED, alpha_fixed=0.0, eps=0.0))
    assert g.tolist() == [1.0, 0.0] and d.tolist() == [1.0, 1.0]


# ------------------------------------------------------------ state and regimes

def test_state_is_raw_gradient_in_every_regime():
    rng = np.random.default_rng(8)
    hp = orc.HParams(c_low=0.05, c_high=0.3, eps=1e-8)
    d = rng.standard_normal(500).astype(np.float32)
    seen = set()
    prev_gg = None
    for rho in (0.0, 0.15, 0.8, 0.02, 0.2):
        noise = rng.standard_normal(500).astype(np.float32)
        g = (rho * d + math.sqrt(1 - rho * rho) * noise).astype(np.float32)
        raw = g.copy()
        dec = orc.step([g], [d], hp)
        seen.add(dec.regime)
        np.testing.assert_array_equal(d, raw)
        if dec.regime != orc.PROJECT:
            np.testing.assert_array_equal(g, raw)
        if prev_gg is not None:
            assert dec.dd == prev_gg                     # dd(t+1) == gg(t)
        prev_gg = dec.gg
    assert seen == {orc.SAFE, orc.PROJECT, orc.VIOLATION}


def test_first_step_never_reads_d():
    g = f32(1, 2, 3, 4)
    d = np.full(4, np.nan, dtype=np.float32)
    dec = orc.step([g], [d], orc.HParams(), first_step=True)
    assert (dec.dot, dec.dd, dec.cos, dec.regime, dec.nonfinite) == (0.0, 0.0, 0.0, orc.SAFE, 0)
    assert g.tolist() == [1, 2, 3, 4] and d.tolist() == [1, 2, 3, 4]


def test_nonfinite_reading():
    g, d = f32(1, np.inf, 3), f32(1, 1, 1)
    dec = orc.step([g], [d], orc.HParams())
    assert dec.nonfinite == 1 and dec.regime == orc.VIOLATION
    assert d.tolist() == [1, 1, 1]
    g2, d2 = f32(1, 2, 3), f32(1, np.nan, 1)
    dec = orc.step([g2], [d2], orc.HParams())
    assert dec.nonfinite == 1 and g2.tolist() == [1, 2, 3]


def test_zero_on_violation_and_projected_state():
    g, d = f32(1, 2, 3), f32(1, 2, 3)
    dec = orc.step([g], [d], orc.HParams(zero_on_violation=1))
    assert dec.regime == orc.VIOLATION and g.tolist() == [0, 0, 0] and d.tolist() == [1, 2, 3]
    g, d = f32(3, 4, 0, 0), f32(1, 0, 0, 0)
    orc.step([g], [d], orc.HParams(c_low=0.3, c_high=0.9, eps=0, state_mode=orc.STATE_PROJECTED))
    assert g.tolist() == [1.5, 4, 0, 0] and d.tolist() == [1.5, 4, 0, 0]


def test_threads_do_not_change_outputs():
    gl, dl = synth.gradient_list(synth.decoder_tensor_list(synth.DIMS["mini"]), 0.2, 2)
    gl = [t.numpy() for t in gl]
    dl = [t.numpy() for t in dl]
    hp = orc.HParams(c_low=0.05, c_high=0.9)
    g1, d1 = [t.copy() for t in gl], [t.copy() for t in dl]
    a = orc.step(gl, dl, hp, threads=1)
    b = orc.step(g1, d1, hp, threads=4)
    assert a.regime == b.regime == orc.PROJECT
    assert a.cos == pytest.approx(b.cos, rel=1e-14)
    if a.coef == b.coef:
        for x, y in zip(gl + dl, g1 + d1):
            np.testing.assert_array_equal(x, y)


# --------------------------------------------------------------------- bfloat16

def test_bf16_rounding_matches_library_conversion():
    rng = np.random.default_rng(3)
    x = (rng.standard_normal(200_000) * 10.0 ** rng.uniform(-42, 38, 200_000)).astype(np.float32)
    special = f32(0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895314e38, 3.4e38, -3.4e38, 1e-40,
                  9.1835e-41, 4.6e-41, 2.3e-41, np.inf, -np.inf)
    x = np.concatenate([x, special])
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = orc.round_to_bf16(x.astype(np.float64))
    np.testing.assert_array_equal(got, want)


def test_bf16_rounding_is_direct_not_via_float32():
    # 1 + 2^-8 + 2^-30 lies just above a bfloat16 tie: direct rounding goes up to
    # 1 + 2^-7; rounding to float32 first would land on the tie and then go down.
    x = np.array([1.0 + 2.0 ** -8 + 2.0 ** -30, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8])
    assert orc.round_to_bf16(x).tolist() == [0x3F81, 0x3F80, 0x3F82]


def test_bf16_gradient_list_path():
    torch.manual_seed(0)
    g = (torch.randn(3000) * 0.01).to(torch.bfloat16)
    d = torch.randn(3000) * 0.01 + g.float() * 0.5
    want = (dot64(g.float().numpy(), d.numpy()), dot64(g.float().numpy(), g.float().numpy()),
            dot64(d.numpy(), d.numpy()))
    got = orc.stats([g], [d])
    for a, b in zip(got, want):
        assert a == pytest.approx(b, rel=1e-15)
    hp = orc.HParams(c_low=0.05, c_high=0.99, eps=0.0)
    g0, d0 = g.clone(), d.clone()
    dec = orc.step([g], [d], hp)
    assert dec.regime == orc.PROJECT
    assert torch.equal(d, g0.float())
    # every output is a bfloat16 within half a bfloat16 ulp of g + coef*d (nearest rounding)
    x = g0.double().numpy() + dec.coef * d0.double().numpy()
    ulp = 2.0 ** (np.floor(np.log2(np.abs(x))) - 7)
    assert np.all(np.abs(g.double().numpy() - x) <= 0.5 * ulp * (1 + 1e-12))


# ------------------------------------------------- global-norm clipping (Table 2)

def test_clipping_matches_library_clip_after_the_rule():
    """Clipping folded into the update must equal the unclipped rule followed by the
    library's global-norm clip (torch.nn.utils.clip_grad_norm_), up to the extra
    rounding the two-pass form makes."""
    shapes = synth.decoder_tensor_list(synth.DIMS["mini"])
    gl, dl = synth.gradient_list(shapes, 0.2, 2)
    for max_norm in (1e-3, 0.05, 1e6):
        hp0 = orc.HParams(c_low=0.05, c_high=0.9)
        hp1 = orc.HParams(c_low=0.05, c_high=0.9, clip_max_norm=max_norm)
        g0, d0 = [t.clone() for t in gl], [t.clone() for t in dl]
        g1, d1 = [t.clone() for t in gl], [t.clone() for t in dl]
        dec0 = orc.step(g0, d0, hp0)
        dec1 = orc.step(g1, d1, hp1)
        assert dec0.regime == dec1.regime == orc.PROJECT
        params = [torch.nn.Parameter(torch.zeros_like(t)) for t in g0]
        for p_, t in zip(params, g0):
            p_.grad = t.clone()
        total = float(torch.nn.utils.clip_grad_norm_(params, max_norm))
        assert dec1.out_norm == pytest.approx(total, rel=1e-6)
        if max_norm == 1e6:
            assert dec1.clip_scale == 1.0
            for a, b in zip(g1, g0):
                np.testing.assert_array_equal(a.numpy(), b.numpy())
        else:
            assert dec1.clip_scale == pytest.approx(max_norm / (total + 1e-6), rel=1e-6)
            for a, p_ in zip(g1, params):
                # the library rounds g', the factor and the product to binary32: a few ulp apart
                np.testing.assert_allclose(a.numpy(), p_.grad.numpy(), rtol=5e-7, atol=0)
        for a, b in zip(d1, d0):
            np.testing.assert_array_equal(a.numpy(), b.numpy())      # the state is never clipped


def test_clipping_closed_forms_and_regimes():
    g, d = synth.flat_pair_with_cosine(1 << 12, 0.6, s=2.0, seed=12)
    g, d = g.numpy(), d.numpy()
    hp = orc.HParams(c_low=0.05, c_high=0.95, eps=0.0, clip_max_norm=0.5)
    g1, d1 = g.copy(), d.copy()
    dec = orc.step([g1], [d1], hp)
    c, cl = dec.cos, hp.c_low
    assert dec.out_norm ** 2 == pytest.approx(dec.gg * (1 - c * c + cl * cl), rel=1e-6)
    assert dec.clip_scale == pytest.approx(0.5 / (dec.out_norm + 1e-6), rel=1e-12)
    assert math.sqrt(dot64(g1, g1)) == pytest.approx(0.5 * dec.out_norm / (dec.out_norm + 1e-6),
                                                     rel=1e-6)
    # safe step: only the clip acts, g'' = s g
    w = np.random.default_rng(0).standard_normal(g.size).astype(np.float32)
    w -= np.float32(dot64(w, d) / dot64(d, d)) * d
    g2, d2 = w.copy(), d.copy()
    dec = orc.step([g2], [d2], orc.HParams(clip_max_norm=1.0))
    assert dec.regime == orc.SAFE and dec.clip_scale < 1.0
    np.testing.assert_allclose(g2, w.astype(np.float64) * dec.clip_scale, rtol=6e-8)
    np.testing.assert_array_equal(d2, w)
    # skipped step: nothing is sent on, nothing is scaled
    g3, d3 = (d * 3).astype(np.float32), d.copy()
    dec = orc.step([g3], [d3], orc.HParams(clip_max_norm=1e-3))
    assert dec.regime == orc.VIOLATION and dec.clip_scale == 1.0
    np.testing.assert_array_equal(g3, (d * 3).astype(np.float32))


# ---------------------------------------- the update consumed by AdamW (Table 2)

def test_fused_adamw_matches_library_optimizer():
    """Several consecutive steps of the oracle's GAC->AdamW against the unfused
    route: oracle projection (kept in float64 by using float32-exact inputs) followed
    by torch.optim.AdamW in float64."""
    rng = np.random.default_rng(4)
    n = 2000
    opt = orc.AdamW(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=1e-2)
    hp = orc.HParams(c_low=0.05, c_high=0.6)
    p = rng.standard_normal(n).astype(np.float32)
    m = np.zeros(n, np.float32)
    v = np.zeros(n, np.float32)
    d = np.zeros(n, np.float32)
    tp = torch.nn.Parameter(torch.from_numpy(p.astype(np.float64)))
    topt = torch.optim.AdamW([tp], lr=opt.lr, betas=(opt.beta1, opt.beta2), eps=opt.eps,
                             weight_decay=opt.weight_decay)
    t_applied = 0
    prev = rng.standard_normal(n).astype(np.float32)
    regimes = []
    for step, rho in enumerate([None, 0.0, 0.3, 0.9, 0.2, 0.01], start=1):
        noise = rng.standard_normal(n).astype(np.float32)
        g = noise if rho is None else (rho * prev + math.sqrt(1 - rho * rho) * noise).astype(np.float32)
        prev = g.copy()
        first = step == 1
        dec = orc.decide(orc.stats([g], [d], first_step=first), hp, first)
        # unfused reference: g' from the definition in float64 (not rounded), then the library optimizer
        gp = g.astype(np.float64)
        if dec.regime == orc.PROJECT:
            gp = hp.beta * gp + dec.coef * d.astype(np.float64)
        applied = orc.project_adamw([g], [d], [p], [m], [v], hp, dec, opt, t_applied + 1, first)
        regimes.append(dec.regime)
        if applied:
            t_applied += 1
            # the library keeps float64 state, the oracle rounds p, m, v to float32 each step:
            # restart the library from the oracle's rounded state so that one step is compared
            tp.grad = torch.from_numpy(gp)
            topt.step()
            st = topt.state[tp]
            np.testing.assert_allclose(m, st["exp_avg"].numpy(), rtol=1e-6, atol=1e-12)
            np.testing.assert_allclose(v, st["exp_avg_sq"].numpy(), rtol=1e-6, atol=1e-14)
            np.testing.assert_allclose(p, tp.detach().numpy(), rtol=1e-6, atol=1e-9)
            with torch.no_grad():
                tp.copy_(torch.from_numpy(p.astype(np.float64)))
                st["exp_avg"].copy_(torch.from_numpy(m.astype(np.float64)))
                st["exp_avg_sq"].copy_(torch.from_numpy(v.astype(np.float64)))
        np.testing.assert_array_equal(d, g)
    assert set(regimes) == {orc.SAFE, orc.PROJECT, orc.VIOLATION}
    assert t_applied == regimes.count(orc.SAFE) + regimes.count(orc.PROJECT)


def test_fused_adamw_skips_the_update_on_violation():
    g = f32(1, 2, 3, 4)
    d = f32(1, 2, 3, 4)
    p, m, v = f32(5, 6, 7, 8), f32(.1, .2, .3, .4), f32(1, 1, 1, 1)
    dec = orc.decide(orc.stats([g], [d]), orc.HParams())
    assert dec.regime == orc.VIOLATION
    applied = orc.project_adamw([g], [d * 2], [p], [m], [v], orc.HParams(), dec, orc.AdamW(), 1)
    assert not applied
    assert p.tolist() == [5, 6, 7, 8] and v.tolist() == [1, 1, 1, 1]
    np.testing.assert_array_equal(m, f32(.1, .2, .3, .4))


def test_bf16_snapshot_state():
    """A bfloat16 stored direction next to a bfloat16 gradient: the refresh is an exact copy."""
    torch.manual_seed(1)
    d = (torch.randn(4000) * 0.01).to(torch.bfloat16)
    g = (0.5 * d.float() + torch.randn(4000) * 0.01).to(torch.bfloat16)
    g0, d0 = g.clone(), d.clone()
    want = (dot64(g.float().numpy(), d.float().numpy()), dot64(g.float().numpy(), g.float().numpy()),
            dot64(d.float().numpy(), d.float().numpy()))
    got = orc.stats([g], [d])
    for a, b in zip(got, want):
        assert a == pytest.approx(b, rel=1e-15)
    hp = orc.HParams(c_low=0.05, c_high=0.99, eps=0.0)
    dec = orc.step([g], [d], hp)
    assert dec.regime == orc.PROJECT and d.dtype == torch.bfloat16
    assert torch.equal(d.view(torch.int16), g0.view(torch.int16))
    x = g0.double().numpy() + dec.coef * d0.double().numpy()
    ulp = 2.0 ** (np.floor(np.log2(np.abs(x))) - 7)
    assert np.all(np.abs(g.double().numpy() - x) <= 0.5 * ulp * (1 + 1e-12))
    with pytest.raises(TypeError):
        orc.project([g0.float()], [d0], hp, dec)          # a float32 gradient needs a float32 snapshot
