"""The (bfloat16 gradient, bfloat16 stored direction) pair: a snapshot of half
the size that is still an exact copy of the gradient (App. A.2, memory
footprint).  Same parity bars as the other pairs."""
import ctypes
import math

import pytest
import torch

from oracle import gac_oracle as orc
from paper_2603_01501_b200 import binding as gb
from paper_2603_01501_b200 import synth

from gpu_util import check_decision, check_outputs, check_sums, max_ulp, step_both, to_orc_hp

pytestmark = pytest.mark.gpu
FORCE = dict(c_low=0.05, c_high=2.0)
BF = torch.bfloat16


def pair(n, rho, seed, scale=0.01):
    gen = torch.Generator().manual_seed(seed)
    d = (torch.randn(n, generator=gen) * scale).to(BF)
    w = torch.randn(n, generator=gen) * scale
    g = (rho * d.float() + math.sqrt(1 - rho * rho) * w).to(BF)
    return g, d


@pytest.mark.parametrize("n", [1, 3, 4, 5, 7, 8, 9, 1023, 1025, 16383, 16384, 16385, 5 * 16384 + 7, 1_000_003])
def test_sizes(n):
    g, d = pair(n, 0.5, n)
    res, dec, gg, dg, gr, dr = step_both([g], [d], gb.HParams(**FORCE))
    check_sums(res, dec)
    check_decision(res, dec)
    check_outputs(gg, dg, gr, dr)
    assert dg[0].dtype == BF


@pytest.mark.parametrize("hp", [gb.HParams(), gb.HParams(**FORCE), gb.HParams(zero_on_violation=1),
                                gb.HParams(**FORCE, state_mode=gb.GAC_STATE_PROJECTED),
                                gb.HParams(**FORCE, state_mode=gb.GAC_STATE_HOLD),
                                gb.HParams(mode=gb.GAC_MODE_FIXED, alpha_fixed=0.25, beta=1.5),
                                gb.HParams(**FORCE, clip_max_norm=0.01)],
                         ids=["defaults", "project", "zero", "projected_state", "hold", "fixed", "clipped"])
def test_decoder_list_and_variants(hp):
    shapes = synth.decoder_tensor_list(synth.DIMS["small"])
    g, d = synth.gradient_list(shapes, 0.7, config_id=3, g_dtype=BF)
    d = [t.to(BF) for t in d]
    res, dec, gg, dg, gr, dr = step_both(g, d, hp)
    check_sums(res, dec)
    check_decision(res, dec)
    follows = hp.state_mode == gb.GAC_STATE_PROJECTED and res.regime == gb.GAC_REGIME_PROJECT
    check_outputs(gg, dg, gr, dr, d_follows_g=follows)


def test_state_carried_over_steps_and_first_step():
    torch.manual_seed(3)
    n = 70_001
    hp = gb.HParams()
    d_gpu = [torch.full((n,), float("nan"), dtype=BF, device="cuda")]
    g_gpu = [torch.empty(n, dtype=BF, device="cuda")]
    d_ref = [torch.full((n,), float("nan"), dtype=BF)]
    ctx = gb.gac_init(g_gpu, d_gpu, hp)
    prev = torch.randn(n)
    seen = set()
    for t, rho in enumerate([None, 0.0, 0.15, 0.8, 0.2], start=1):
        g = (torch.randn(n) if rho is None else rho * prev + math.sqrt(1 - rho * rho) * torch.randn(n)).to(BF)
        prev = g.float()
        g_gpu[0].copy_(g)
        g_ref = [g.clone()]
        dec = orc.step(g_ref, d_ref, to_orc_hp(hp), first_step=(t == 1))
        res = gb.gac_stats(ctx, t)
        gb.gac_project(ctx, coef_override=dec.coef if dec.regime == orc.PROJECT else None)
        check_sums(res, dec)
        check_decision(res, dec)
        check_outputs(g_gpu, d_gpu, g_ref, d_ref)
        assert torch.equal(d_gpu[0].cpu().view(torch.int16), g.view(torch.int16))
        seen.add(res.regime)
    assert seen == {0, 1, 2}
    gb.gac_free(ctx)


def test_misaligned_views():
    sizes, offs = [3, 1000, 40001], [1, 3, 5]
    g_cpu, d_cpu, g_view, d_view = [], [], [], []
    for n, o in zip(sizes, offs):
        g, d = pair(n, 0.4, n + 1)
        g_cpu.append(g)
        d_cpu.append(d)
        gbuf = torch.full((n + 16,), 7.0, dtype=BF, device="cuda")
        dbuf = torch.full((n + 16,), -9.0, dtype=BF, device="cuda")
        gbuf[o:o + n] = g.cuda()
        dbuf[o + 1:o + 1 + n] = d.cuda()
        g_view.append(gbuf[o:o + n])
        d_view.append(dbuf[o + 1:o + 1 + n])
    hp = gb.HParams(**FORCE)
    g_ref, d_ref = [t.clone() for t in g_cpu], [t.clone() for t in d_cpu]
    dec = orc.step(g_ref, d_ref, to_orc_hp(hp))
    ctx = gb.gac_init(g_view, d_view, hp)
    res = gb.gac_stats(ctx, 2)
    gb.gac_project(ctx, coef_override=dec.coef)
    torch.cuda.synchronize()
    check_sums(res, dec)
    check_outputs(g_view, d_view, g_ref, d_ref)
    gb.gac_free(ctx)


def test_fused_adamw_and_static_entry():
    shapes = synth.decoder_tensor_list(synth.DIMS["mini"])
    g, d = synth.gradient_list(shapes, 0.2, config_id=3, g_dtype=BF)
    d = [t.to(BF) for t in d]
    gen = torch.Generator().manual_seed(5)
    p = [torch.randn(t.numel(), generator=gen) * 0.02 for t in g]
    m = [torch.randn(t.numel(), generator=gen) * 1e-3 for t in g]
    v = [torch.rand(t.numel(), generator=gen) * 1e-5 for t in g]
    hp = gb.HParams(c_low=0.05, c_high=0.9)
    gg, dg = [t.cuda() for t in g], [t.cuda() for t in d]
    pg, mg, vg = ([t.cuda() for t in l] for l in (p, m, v))
    out = torch.zeros(ctypes.sizeof(gb.gac_result), dtype=torch.uint8, device="cuda")
    gb.gac_stats_static(gg, dg, hp, 2, out)
    torch.cuda.synchronize()
    st = gb.result_from_tensor(out)
    dec = orc.decide(orc.stats(g, d), to_orc_hp(hp))
    check_sums(st, dec)
    check_decision(st, dec)
    orc.project_adamw(g, d, p, m, v, to_orc_hp(hp), dec, orc.AdamW(lr=1e-3), 4)
    ctx = gb.gac_init(gg, dg, hp)
    gb.gac_attach_adamw(ctx, pg, mg, vg, applied_steps=3)
    gb.gac_stats(ctx, 2)
    after = gb.gac_project_adamw(ctx, gb.AdamW(lr=1e-3), coef_override=dec.coef, fetch=True)
    assert after.applied_steps == 4
    for a, b in zip(pg + mg + vg, p + m + v):
        assert max_ulp(a.cpu(), b) <= 4
    for a, b in zip(dg, d):
        assert torch.equal(a.cpu().view(torch.int16), b.view(torch.int16))
    gb.gac_free(ctx)


def test_float32_gradient_with_bf16_state_is_refused():
    g, d = [torch.ones(8, device="cuda")], [torch.ones(8, dtype=BF, device="cuda")]
    with pytest.raises(gb.GacError) as e:
        gb.gac_init(g, d, gb.HParams())
    assert e.value.status == gb.GAC_ERR_DTYPE
