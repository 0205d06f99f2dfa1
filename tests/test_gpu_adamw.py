"""GPU parity of the fused GAC -> AdamW pass (Algorithm 1's parameter update with
the optimizer of Table 2) against the CPU oracle, over consecutive steps that
visit all three regimes."""
import math

import pytest
import torch

from oracle import gac_oracle as orc
from paper_2603_01501_b200 import binding as gb
from paper_2603_01501_b200 import synth

from gpu_util import check_decision, check_sums, max_ulp, ordered_int, to_orc_hp

pytestmark = pytest.mark.gpu


def run_sequence(g_dtype, hp, opt_kw, shapes_name="mini", rhos=(None, 0.0, 0.3, 0.9, 0.2, 0.01, 0.5)):
    shapes = synth.decoder_tensor_list(synth.DIMS[shapes_name])
    sig = synth.per_tensor_scales(2, len(shapes))
    gen = torch.Generator().manual_seed(7)
    n_t = len(shapes)
    p_cpu = [torch.randn(n, generator=gen) * 0.02 for _, n in shapes]
    m_cpu = [torch.zeros(n) for _, n in shapes]
    v_cpu = [torch.zeros(n) for _, n in shapes]
    d_cpu = [torch.full((n,), float("nan")) for _, n in shapes]
    g_gpu = [torch.empty(n, dtype=g_dtype, device="cuda") for _, n in shapes]
    d_gpu = [t.cuda() for t in d_cpu]
    p_gpu, m_gpu, v_gpu = ([t.cuda() for t in l] for l in (p_cpu, m_cpu, v_cpu))
    ctx = gb.gac_init(g_gpu, d_gpu, hp)
    gb.gac_attach_adamw(ctx, p_gpu, m_gpu, v_gpu, applied_steps=0)
    gopt, oopt = gb.AdamW(**opt_kw), orc.AdamW(**opt_kw)
    ohp = to_orc_hp(hp)
    prev = [torch.randn(n, generator=gen) * s for (_, n), s in zip(shapes, sig)]
    applied, regimes, worst = 0, [], 0
    for t, rho in enumerate(rhos, start=1):
        noise = [torch.randn(n, generator=gen) * s for (_, n), s in zip(shapes, sig)]
        g = noise if rho is None else [rho * a + math.sqrt(1 - rho * rho) * b for a, b in zip(prev, noise)]
        g = [x.to(g_dtype) for x in g]
        prev = [x.float() for x in g]
        for dst, src in zip(g_gpu, g):
            dst.copy_(src)
        first = t == 1
        dec = orc.decide(orc.stats(g, d_cpu, first_step=first), ohp, first)
        m_before = [x.clone() for x in m_cpu]
        d_before = [x.clone().float() for x in d_cpu]
        did = orc.project_adamw(g, d_cpu, p_cpu, m_cpu, v_cpu, ohp, dec, oopt, applied + 1, first)
        applied += int(did)
        res = gb.gac_stats(ctx, t)
        after = gb.gac_project_adamw(ctx, gopt, coef_override=dec.coef if dec.regime == orc.PROJECT else None,
                                     fetch=True)
        check_sums(res, dec)
        check_decision(res, dec)
        assert after.applied_steps == applied
        if hp.clip_max_norm > 0 and dec.regime != orc.VIOLATION:
            assert abs(after.clip_scale - dec.clip_scale) <= 1e-9 * dec.clip_scale
        for i in range(n_t):
            bits = torch.int16 if g_dtype == torch.bfloat16 else torch.int32
            assert torch.equal(g_gpu[i].cpu().view(bits), g[i].view(bits)), "g was written"
            assert torch.equal(d_gpu[i].cpu(), d_cpu[i]), "stored direction is not the raw gradient"
            # v is a sum of non-negative terms: plain ulp distance.  m = b1 m + (1-b1) g' and
            # p = p - delta can cancel (with bfloat16 gradients even exactly), so where they do the
            # bound is the rounding noise of the binary64 terms instead of ulps of the tiny result.
            gmag = g[i].float().abs() + abs(dec.coef) * d_before[i].abs().nan_to_num(0.0)
            checks = (("v", v_gpu[i], v_cpu[i], None),
                      ("m", m_gpu[i], m_cpu[i], 1e-13 * (m_before[i].abs() + gmag)),
                      ("p", p_gpu[i], p_cpu[i], torch.full_like(p_cpu[i], 1e-10 * oopt.lr)))
            for name, a, b, slack in checks:
                a_cpu = a.cpu()
                ulps = (ordered_int(a_cpu) - ordered_int(b)).abs()
                ok = ulps <= 4
                if slack is not None:
                    ok |= (a_cpu.double() - b.double()).abs() <= slack.double()
                assert bool(ok.all()), f"step {t} tensor {i} {name}: {int(ulps[~ok].max())} ulp"
                worst = max(worst, int(ulps[ok & (ulps <= 4)].max()) if bool((ulps <= 4).any()) else 0)
                # each step is compared from identical state: a last-bit difference (a rounding tie
                # taken the other way) would otherwise be carried into later steps
                a.copy_(b)
        regimes.append(dec.regime)
    gb.gac_free(ctx)
    return regimes, applied, worst


@pytest.mark.parametrize("g_dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
def test_fused_adamw_paper_hyperparameters(g_dtype):
    regimes, applied, _ = run_sequence(g_dtype, gb.HParams(), dict())        # Table 2 values
    assert set(regimes) == {0, 1, 2}
    assert applied == sum(r != gb.GAC_REGIME_VIOLATION for r in regimes)


@pytest.mark.parametrize("hp,opt_kw", [
    (gb.HParams(c_low=0.05, c_high=0.6, clip_max_norm=0.05), dict(lr=1e-3)),
    (gb.HParams(c_low=0.05, c_high=0.6, clip_max_norm=1e6), dict(lr=1e-2, weight_decay=0.1)),
    (gb.HParams(mode=gb.GAC_MODE_FIXED, alpha_fixed=0.25, beta=1.5), dict(lr=1e-3, beta1=0.8, beta2=0.95)),
], ids=["clipped", "clip_inactive", "fixed_gains"])
@pytest.mark.parametrize("g_dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
def test_fused_adamw_variants(hp, opt_kw, g_dtype):
    run_sequence(g_dtype, hp, opt_kw)


def test_fused_adamw_larger_list_and_call_rules():
    run_sequence(torch.float32, gb.HParams(c_low=0.05, c_high=0.6), dict(lr=1e-4), shapes_name="small",
                 rhos=(None, 0.3, 0.9))
    g, d = [torch.ones(64, device="cuda")], [torch.ones(64, device="cuda") * 2]
    ctx = gb.gac_init(g, d, gb.HParams())
    gb.gac_stats(ctx, 2)
    with pytest.raises(gb.GacError) as e:
        gb.gac_project_adamw(ctx, gb.AdamW())
    assert e.value.status == gb.GAC_ERR_STATE               # nothing attached
    gb.gac_free(ctx)
    ctx = gb.gac_init(g, d, gb.HParams(state_mode=gb.GAC_STATE_HOLD))
    z = [torch.zeros(64, device="cuda")]
    with pytest.raises(gb.GacError) as e:
        gb.gac_attach_adamw(ctx, z, z, z)
    assert e.value.status == gb.GAC_ERR_INVALID_ARG
    gb.gac_free(ctx)


def ulp32(x: torch.Tensor) -> torch.Tensor:
    """Spacing of binary32 numbers at magnitude x (float64 tensor)."""
    e = torch.floor(torch.log2(x.abs().clamp_min(2.0 ** -126)))
    return torch.pow(torch.tensor(2.0, dtype=torch.float64), e - 23)


@pytest.mark.parametrize("opt_kw", [dict(), dict(lr=1e-3, weight_decay=0.1)], ids=["table2", "large_lr"])
@pytest.mark.parametrize("g_dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
def test_fused_adamw_free_running_trajectory(g_dtype, opt_kw):
    """p, m and v are carried on the GPU for 8 steps and never reset to the oracle's values.  Both sides
    round m, v and p once per step, so per step they can part by one binary32 spacing of the new value;
    an earlier difference is carried on times b1 (m), b2 (v), 1 (p), and reaches p through the update
    lr_t m / (sqrt(v)/sqrt(1-b2^t) + eps) to first order.  The bound below is exactly that recurrence,
    evaluated on the oracle's values (plus the binary64 noise terms the per-step test uses)."""
    shapes = synth.decoder_tensor_list(synth.DIMS["mini"])
    sig = synth.per_tensor_scales(2, len(shapes))
    gen = torch.Generator().manual_seed(21)
    hp = gb.HParams()
    ohp = to_orc_hp(hp)
    gopt, oopt = gb.AdamW(**opt_kw), orc.AdamW(**opt_kw)
    p_cpu = [torch.randn(n, generator=gen) * 0.02 for _, n in shapes]
    m_cpu = [torch.zeros(n) for _, n in shapes]
    v_cpu = [torch.zeros(n) for _, n in shapes]
    d_cpu = [torch.full((n,), float("nan")) for _, n in shapes]
    g_gpu = [torch.empty(n, dtype=g_dtype, device="cuda") for _, n in shapes]
    d_gpu = [t.cuda() for t in d_cpu]
    p_gpu, m_gpu, v_gpu = ([t.cuda() for t in l] for l in (p_cpu, m_cpu, v_cpu))
    ctx = gb.gac_init(g_gpu, d_gpu, hp)
    gb.gac_attach_adamw(ctx, p_gpu, m_gpu, v_gpu, applied_steps=0)
    err_m = [torch.zeros(n, dtype=torch.float64) for _, n in shapes]
    err_v = [torch.zeros(n, dtype=torch.float64) for _, n in shapes]
    err_p = [torch.zeros(n, dtype=torch.float64) for _, n in shapes]
    prev = [torch.randn(n, generator=gen) * s for (_, n), s in zip(shapes, sig)]
    applied, regimes = 0, []
    for t, rho in enumerate((None, 0.0, 0.15, 0.9, 0.2, 0.01, 0.25, 0.1), start=1):
        noise = [torch.randn(n, generator=gen) * s for (_, n), s in zip(shapes, sig)]
        g = noise if rho is None else [rho * a + math.sqrt(1 - rho * rho) * b for a, b in zip(prev, noise)]
        g = [x.to(g_dtype) for x in g]
        prev = [x.float() for x in g]
        for dst, src in zip(g_gpu, g):
            dst.copy_(src)
        first = t == 1
        dec = orc.decide(orc.stats(g, d_cpu, first_step=first), ohp, first)
        m_before = [x.double() for x in m_cpu]
        v_before = [x.double() for x in v_cpu]
        gmag = [x.double().abs() + abs(dec.coef) * y.double().abs().nan_to_num(0.0) for x, y in zip(g, d_cpu)]
        did = orc.project_adamw(g, d_cpu, p_cpu, m_cpu, v_cpu, ohp, dec, oopt, applied + 1, first)
        applied += int(did)
        gb.gac_stats(ctx, t, fetch=False)
        after = gb.gac_project_adamw(ctx, gopt, coef_override=dec.coef if dec.regime == orc.PROJECT else None,
                                     fetch=True)
        assert after.regime == dec.regime and after.applied_steps == applied
        regimes.append(dec.regime)
        if did:
            step_size = oopt.lr / (1.0 - oopt.beta1 ** applied)
            isb2 = 1.0 / math.sqrt(1.0 - oopt.beta2 ** applied)
            for i in range(len(shapes)):
                m_new, v_new = m_cpu[i].double(), v_cpu[i].double()
                err_m[i] = oopt.beta1 * err_m[i] + ulp32(m_new) + 1e-13 * (m_before[i].abs() + gmag[i])
                err_v[i] = oopt.beta2 * err_v[i] + ulp32(v_new) + 1e-13 * (v_before[i] + gmag[i] ** 2)
                root = v_new.sqrt()
                denom = root * isb2 + oopt.eps
                d_denom = isb2 * err_v[i] / (root + 1e-300)
                d_update = step_size * (err_m[i] / denom + m_new.abs() * d_denom / denom ** 2)
                err_p[i] = err_p[i] + ulp32(p_cpu[i].double()) + d_update + 1e-10 * oopt.lr
        for i in range(len(shapes)):
            assert torch.equal(d_gpu[i].cpu(), d_cpu[i]), "stored direction is not the raw gradient"
            for name, a, b, err in (("m", m_gpu[i], m_cpu[i], err_m[i]), ("v", v_gpu[i], v_cpu[i], err_v[i]),
                                    ("p", p_gpu[i], p_cpu[i], err_p[i])):
                diff = (a.cpu().double() - b.double()).abs()
                bad = diff > err
                assert not bool(bad.any()), (f"step {t} tensor {i} {name}: off by {float(diff[bad].max()):.3e}, "
                                             f"bound {float(err[bad].min()):.3e}")
    gb.gac_free(ctx)
    assert set(regimes) == {orc.SAFE, orc.PROJECT, orc.VIOLATION} and applied >= 5
    # the bound stays a rounding-level statement: a few binary32 spacings of p per step, plus a
    # 1e-5-th of one update where p itself is tiny
    for i in range(len(shapes)):
        assert bool((err_p[i] <= 8 * 4 * ulp32(p_cpu[i].double()) + 1e-5 * oopt.lr).all())
