"""Helpers shared by the GPU parity tests: run one step through the C ABI,
run the same step through the CPU oracle, compare with the stated tolerances.

Tolerances (from the problem statement of this library):
  sums and cosine      1e-5 relative; for <g,d> and the cosine, which may be
                       near zero, relative to max(|x|, 1e-6 * natural scale)
  float32 outputs      within 4 units in the last place of the oracle's result
                       given the same binary32 coefficient
  bfloat16 outputs     within 1 bfloat16 unit in the last place
  stored direction     bit-exact (it is a copy / exact widening of g)
  regime               exact
"""
import math

import numpy as np
import torch

from oracle import gac_oracle as orc
from paper_2603_01501_b200 import binding as gb

REL = 1e-5


def to_orc_hp(hp: gb.HParams) -> orc.HParams:
    return orc.HParams(c_low=hp.c_low, c_high=hp.c_high, eps=hp.eps, beta=hp.beta, mode=hp.mode,
                       alpha_fixed=hp.alpha_fixed, state_mode=hp.state_mode,
                       zero_on_violation=hp.zero_on_violation, clip_max_norm=hp.clip_max_norm,
                       clip_eps=hp.clip_eps)


def ordered_int(t: torch.Tensor) -> torch.Tensor:
    """Maps float32/bfloat16 bit patterns to integers whose difference is the
    distance in units in the last place (sign-magnitude to two's complement)."""
    if t.dtype == torch.float32:
        i = t.contiguous().view(torch.int32).to(torch.int64)
        return torch.where(i < 0, -(i & 0x7FFFFFFF), i)
    if t.dtype == torch.bfloat16:
        i = t.contiguous().view(torch.int16).to(torch.int64)
        return torch.where(i < 0, -(i & 0x7FFF), i)
    raise TypeError(t.dtype)


def max_ulp(a: torch.Tensor, b: torch.Tensor) -> int:
    if a.numel() == 0:
        return 0
    return int((ordered_int(a) - ordered_int(b)).abs().max())


def check_sums(res, dec, rel=REL):
    if dec.nonfinite:
        assert res.nonfinite == 1
        return
    scale = math.sqrt(dec.gg * dec.dd)
    assert abs(res.gg - dec.gg) <= rel * dec.gg
    assert abs(res.dd - dec.dd) <= rel * dec.dd
    assert abs(res.dot - dec.dot) <= rel * max(abs(dec.dot), 1e-6 * scale)
    assert abs(res.cos - dec.cos) <= rel * max(abs(dec.cos), 1e-6)


def check_decision(res, dec, rel=REL):
    assert res.regime == dec.regime, (res.regime, dec.regime, res.cos, dec.cos)
    assert res.nonfinite == dec.nonfinite
    assert abs(res.alpha - dec.alpha) <= rel * abs(dec.alpha)
    assert abs(res.coef64 - dec.coef64) <= rel * abs(dec.coef64)
    assert abs(res.coef - dec.coef) <= rel * abs(dec.coef)


def check_outputs(g_gpu, d_gpu, g_ref, d_ref, d_follows_g=False):
    """g_gpu/d_gpu: lists of CUDA tensors after the step; g_ref/d_ref: CPU tensors from the oracle.
    d_follows_g: the stored direction is a copy of g' (PROJECTED state on a step that changed g),
    so it is bit-exact against the library's own g' and only ulp-close to the oracle's."""
    worst = 0
    for i, (a, b, c, e) in enumerate(zip(g_gpu, g_ref, d_gpu, d_ref)):
        a, c = a.cpu(), c.cpu()
        lim = 4 if a.dtype == torch.float32 else 1
        u = max_ulp(a, b)
        assert u <= lim, f"tensor {i}: g' differs by {u} ulp (limit {lim})"
        worst = max(worst, u)
        if d_follows_g:
            assert torch.equal(c.float(), a.float()), f"tensor {i}: d' is not the stored g'"
            assert max_ulp(c.to(a.dtype), e.to(a.dtype)) <= lim
        else:
            bits = torch.int32 if c.dtype == torch.float32 else torch.int16
            assert c.dtype == e.dtype
            assert torch.equal(c.view(bits), e.view(bits)), f"tensor {i}: d' not bit-exact"
    return worst


def step_both(g_cpu, d_cpu, hp: gb.HParams, step=2, device="cuda", launch=None, same_coef=True):
    """Runs one step on copies of the CPU lists through both implementations.
    Returns (gpu result after stats, oracle decision, gpu lists, oracle lists)."""
    g_gpu = [t.to(device) for t in g_cpu]
    d_gpu = [t.to(device) for t in d_cpu]
    g_ref = [t.clone() for t in g_cpu]
    d_ref = [t.clone() for t in d_cpu]
    first = (step == 1)
    ohp = to_orc_hp(hp)
    dec = orc.decide(orc.stats(g_ref, d_ref, first_step=first), ohp, first_step=first)
    orc.project(g_ref, d_ref, ohp, dec, first_step=first)
    ctx = gb.gac_init(g_gpu, d_gpu, hp)
    if launch:
        gb.gac_set_launch(ctx, *launch)
    res = gb.gac_stats(ctx, step)
    after = gb.gac_project(ctx, coef_override=dec.coef if (same_coef and dec.regime == orc.PROJECT) else None,
                           fetch=True)
    torch.cuda.synchronize()
    gb.gac_free(ctx)
    res.after = after            # the record as it stands after the projection pass
    return res, dec, g_gpu, d_gpu, g_ref, d_ref
