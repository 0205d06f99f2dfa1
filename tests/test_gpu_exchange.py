"""GPU parity of exchange mode (state_mode EXCHANGE) against the CPU oracle.

Exchange mode computes what the paper's rule computes -- g' from Eq. 5 and the
stored direction d' = g of App. A.2 -- without the copy that refreshes the
snapshot: the buffers that held g become the stored direction, g' (when it
differs from g) lands in the buffers that held d, and the two sets swap roles
after every step.  The oracle therefore runs the plain RAW rule; the tests map
its g' and d' onto the buffer sets the record names and check, bit for bit,
that nothing else was written.
"""
import dataclasses
import math

import pytest
import torch

from oracle import gac_oracle as orc
from paper_2603_01501_b200 import binding as gb
from paper_2603_01501_b200 import synth

from gpu_util import check_decision, check_sums, max_ulp, ordered_int, to_orc_hp

pytestmark = pytest.mark.gpu

BITS = {torch.float32: torch.int32, torch.bfloat16: torch.int16}


def raw_hp(hp: gb.HParams) -> orc.HParams:
    """The oracle's rule for an exchange-mode context: the paper's RAW state."""
    return to_orc_hp(dataclasses.replace(hp, state_mode=gb.GAC_STATE_RAW))


def same_bits(a: torch.Tensor, b: torch.Tensor) -> bool:
    return torch.equal(a.cpu().view(BITS[a.dtype]), b.cpu().view(BITS[b.dtype]))


def ar_gradients(shapes, sig, rhos, dtype, seed):
    """One gradient list per entry of rhos: cosine about rho to the previous one (None = fresh noise)."""
    gen = torch.Generator().manual_seed(seed)
    prev = None
    for rho in rhos:
        noise = [torch.randn(n, generator=gen) * s for (_, n), s in zip(shapes, sig)]
        if rho is None or prev is None:
            g = noise
        else:
            g = [rho * a + math.sqrt(1 - rho * rho) * b for a, b in zip(prev, noise)]
        g = [x.to(dtype) for x in g]
        prev = [x.float().clone() for x in g]      # the caller may plant a NaN in what it gets
        yield g


def run_exchange_sequence(dtype, hp, rhos, shapes_name="mini", nan_at=(), views=False):
    """Steps a context in exchange mode and the RAW oracle side by side.  Returns the regimes met."""
    shapes = synth.decoder_tensor_list(synth.DIMS[shapes_name])
    sig = synth.per_tensor_scales(2, len(shapes))
    pad = 3 if views else 0     # odd element offsets: the element-wise path
    bufs = [[torch.full((n + 2 * pad + 1,), 5.0, dtype=dtype, device="cuda") for _, n in shapes] for _ in range(2)]
    sets = [[b[pad:pad + n] if views else b[:n] for b, (_, n) in zip(bs, shapes)] for bs in bufs]
    for t in sets[1]:
        t.fill_(float("nan"))                      # never read on step 1
    ctx = gb.gac_init(sets[0], sets[1], hp)
    if views:
        assert gb.gac_get_info(ctx).misaligned_tensors == len(shapes)
    ohp = raw_hp(hp)
    d_ref = [torch.full((n,), float("nan"), dtype=dtype) for _, n in shapes]
    regimes, lost = [], False
    for t, g in enumerate(ar_gradients(shapes, sig, rhos, dtype, seed=11), start=1):
        if t in nan_at:
            g[len(g) // 2][7] = float("nan")
        gi = gb.gac_next_gradient_set(ctx)
        assert gi == (t - 1) % 2                    # the roles alternate, whatever the steps decide
        di = gi ^ 1
        for dst, src in zip(sets[gi], g):
            dst.copy_(src)
        before_d = [x.clone() for x in sets[di]]
        first = (t == 1) or lost                    # zero reference: Algorithm 1's g_0, or a lost direction
        g_ref = [x.clone() for x in g]
        dec = orc.decide(orc.stats(g_ref, d_ref, first_step=first), ohp, first)
        res = gb.gac_stats(ctx, t)
        after = gb.gac_project(ctx, coef_override=dec.coef if dec.regime == orc.PROJECT else None, fetch=True)
        torch.cuda.synchronize()
        check_sums(res, dec)
        assert res.g_set == gi and after.g_set == gi
        # the buffers that held g are never written: they are the stored direction now
        for a, b in zip(sets[gi], g):
            assert same_bits(a, b), f"step {t}: the gradient buffers were modified"
        if dec.nonfinite:
            assert res.nonfinite == 1 and after.ref_lost == 1 and after.out_set == gi
            for a, b in zip(sets[di], before_d):
                assert same_bits(a, b)
            lost = True
            regimes.append("nonfinite")
            continue
        lost = False
        check_decision(res, dec)
        assert after.ref_lost == 0
        orc.project(g_ref, d_ref, ohp, dec, first_step=first)      # g_ref <- g', d_ref <- raw g
        changed = (dec.regime == orc.PROJECT or (dec.regime == orc.VIOLATION and hp.zero_on_violation)
                   or (dec.regime == orc.SAFE and dec.clip_scale != 1.0))
        assert after.out_set == (di if changed else gi)
        lim = 4 if dtype == torch.float32 else 1
        for i, (a, b) in enumerate(zip(sets[after.out_set], g_ref)):
            assert max_ulp(a.cpu(), b) <= lim, f"step {t} tensor {i}: outgoing gradient off by {max_ulp(a.cpu(), b)} ulp"
        if not changed:
            for a, b in zip(sets[di], before_d):
                assert same_bits(a, b), f"step {t}: a step that leaves g alone must not write anything"
        for a, b in zip(sets[gi], d_ref):
            assert same_bits(a, b)                  # stored direction = raw gradient, bit for bit
        regimes.append(dec.regime)
    if views:                                       # nothing outside the views was touched
        for bs in bufs:
            for b, (_, n) in zip(bs, shapes):
                assert bool((b[:pad] == 5.0).all()) and bool((b[pad + n:] == 5.0).all())
    gb.gac_free(ctx)
    return regimes


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
def test_exchange_mode_over_all_regimes(dtype):
    regimes = run_exchange_sequence(dtype, gb.HParams(state_mode=gb.GAC_STATE_EXCHANGE),
                                    rhos=(None, 0.0, 0.15, 0.8, 0.02, 0.2, 0.25))
    assert set(regimes) == {orc.SAFE, orc.PROJECT, orc.VIOLATION}


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
def test_exchange_mode_restarts_after_a_nonfinite_step(dtype):
    regimes = run_exchange_sequence(dtype, gb.HParams(state_mode=gb.GAC_STATE_EXCHANGE),
                                    rhos=(None, 0.2, 0.2, 0.2, 0.2, 0.9), nan_at=(3,))
    # step 3 is reported and writes nothing; step 4 is taken against the zero reference (safe)
    assert regimes[2] == "nonfinite" and regimes[3] == orc.SAFE and regimes[4] == orc.PROJECT


def test_exchange_mode_statistics_pass_is_idempotent_after_a_nonfinite_step():
    """The reduction may run more than once for a step.  After a non-finite step the stored direction
    is lost; every reduction of the following step must then take the zero reference -- the mark
    stays until the pass that closes that step clears it."""
    n = 50000
    a = torch.randn(n, device="cuda")
    b = torch.randn(n, device="cuda")
    ctx = gb.gac_init([a], [b], gb.HParams(state_mode=gb.GAC_STATE_EXCHANGE))
    gb.gac_stats(ctx, 1)
    gb.gac_project(ctx)                       # a holds the stored direction, b takes the next gradient
    b.copy_(torch.randn(n, device="cuda"))
    b[17] = float("inf")
    r = gb.gac_stats(ctx, 2)
    after = gb.gac_project(ctx, fetch=True)
    assert r.nonfinite == 1 and after.ref_lost == 1
    a.copy_(torch.randn(n, device="cuda"))    # step 3: gradient in a; b still holds the Inf
    gg = float((a.double() ** 2).sum())
    first = gb.gac_stats(ctx, 3)
    second = gb.gac_stats(ctx, 3)
    third = gb.gac_stats(ctx, 3)
    for r in (first, second, third):
        assert (r.nonfinite, r.regime, r.dot, r.dd, r.cos) == (0, gb.GAC_REGIME_SAFE, 0.0, 0.0, 0.0)
        assert r.gg == first.gg and abs(r.gg - gg) <= 1e-9 * gg and r.ref_lost == 1
    after = gb.gac_project(ctx, fetch=True)
    assert after.ref_lost == 0
    # step 4 compares against step 3's gradient again
    b.copy_(0.5 * a + 0.1 * torch.randn(n, device="cuda"))
    r = gb.gac_stats(ctx, 4)
    assert r.nonfinite == 0 and r.dd == first.gg and abs(r.cos) > 0.9
    gb.gac_project(ctx)
    gb.gac_free(ctx)


@pytest.mark.parametrize("hp", [
    gb.HParams(state_mode=gb.GAC_STATE_EXCHANGE, zero_on_violation=1),
    gb.HParams(state_mode=gb.GAC_STATE_EXCHANGE, clip_max_norm=1e-3),
    gb.HParams(state_mode=gb.GAC_STATE_EXCHANGE, clip_max_norm=1e6),
    gb.HParams(state_mode=gb.GAC_STATE_EXCHANGE, mode=gb.GAC_MODE_FIXED, alpha_fixed=0.25, beta=1.5),
    gb.HParams(state_mode=gb.GAC_STATE_EXCHANGE, mode=gb.GAC_MODE_FIXED, alpha_fixed=0.0),
], ids=["zero_on_violation", "clipped", "clip_inactive", "fixed_gains", "full_projection"])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
def test_exchange_mode_variants(hp, dtype):
    run_exchange_sequence(dtype, hp, rhos=(None, 0.0, 0.15, 0.8, 0.02, 0.2))


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
def test_exchange_mode_on_unaligned_views_and_a_larger_list(dtype):
    hp = gb.HParams(state_mode=gb.GAC_STATE_EXCHANGE, c_low=0.05, c_high=0.6)
    run_exchange_sequence(dtype, hp, rhos=(None, 0.3, 0.01, 0.9), views=True)
    run_exchange_sequence(dtype, hp, rhos=(None, 0.3, 0.5), shapes_name="small")


@pytest.mark.parametrize("n", [1, 3, 4, 5, 1023, 4097, 16385, 5 * 16384 + 7])
def test_exchange_mode_sizes_and_tails(n):
    gen = torch.Generator().manual_seed(n)
    d = torch.randn(n, generator=gen)
    g = 0.5 * d + math.sqrt(0.75) * torch.randn(n, generator=gen)
    hp = gb.HParams(state_mode=gb.GAC_STATE_EXCHANGE, c_low=0.05, c_high=2.0)
    a, b = [g.cuda()], [d.cuda()]
    ctx = gb.gac_init(a, b, hp)
    g_ref, d_ref = [g.clone()], [d.clone()]
    dec = orc.step(g_ref, d_ref, raw_hp(hp))
    res = gb.gac_stats(ctx, 2)
    after = gb.gac_project(ctx, coef_override=dec.coef if dec.regime == orc.PROJECT else None, fetch=True)
    check_sums(res, dec)
    check_decision(res, dec)
    if dec.regime == orc.PROJECT:
        assert after.out_set == gb.GAC_SET_D
        assert max_ulp(b[0].cpu(), g_ref[0]) <= 4
    assert same_bits(a[0], g) and gb.gac_next_gradient_set(ctx) == gb.GAC_SET_D
    gb.gac_free(ctx)


def test_exchange_mode_sharded_form_and_rebind():
    """Local sums, the caller's reduction, the decision, the projection: the same roles and
    results as the unsharded calls; gac_rebind starts the alternation over."""
    shapes = synth.decoder_tensor_list(synth.DIMS["mini"])
    g, d = synth.gradient_list(shapes, 0.4, config_id=2, device="cuda")
    g_cpu, d_cpu = [t.cpu() for t in g], [t.cpu() for t in d]
    hp = gb.HParams(state_mode=gb.GAC_STATE_EXCHANGE, c_low=0.05, c_high=0.9)
    ctx = gb.gac_init(g, d, hp)
    sums = torch.zeros(3, dtype=torch.float64, device="cuda")
    gb.gac_stats_partial(ctx, 2, sums)
    res = gb.gac_decide(ctx, sums)
    g_ref, d_ref = [t.clone() for t in g_cpu], [t.clone() for t in d_cpu]
    dec = orc.step(g_ref, d_ref, raw_hp(hp))
    after = gb.gac_project(ctx, coef_override=dec.coef, fetch=True)
    check_sums(res, dec)
    check_decision(res, dec)
    assert dec.regime == orc.PROJECT and after.out_set == gb.GAC_SET_D
    assert all(max_ulp(a.cpu(), b) <= 4 for a, b in zip(d, g_ref))
    assert all(same_bits(a, b) for a, b in zip(g, g_cpu))
    assert gb.gac_next_gradient_set(ctx) == gb.GAC_SET_D
    # second step with swapped roles through the sharded calls: d holds the gradient, g the direction
    g2 = [0.3 * a + math.sqrt(1 - 0.09) * torch.randn_like(a) * a.std() for a in g_cpu]
    for dst, src in zip(d, g2):
        dst.copy_(src)
    gb.gac_stats_partial(ctx, 3, sums)
    res = gb.gac_decide(ctx, sums)
    g_ref2 = [t.clone() for t in g2]
    dec = orc.step(g_ref2, d_ref, raw_hp(hp))
    after = gb.gac_project(ctx, coef_override=dec.coef if dec.regime == orc.PROJECT else None, fetch=True)
    check_sums(res, dec)
    check_decision(res, dec)
    assert res.g_set == gb.GAC_SET_D and dec.regime == orc.PROJECT and after.out_set == gb.GAC_SET_G
    assert all(max_ulp(a.cpu(), b) <= 4 for a, b in zip(g, g_ref2))
    assert gb.gac_next_gradient_set(ctx) == gb.GAC_SET_G
    gb.gac_stats(ctx, 4, fetch=False)
    gb.gac_project(ctx)
    assert gb.gac_next_gradient_set(ctx) == gb.GAC_SET_D
    gb.gac_rebind(ctx, g, d)
    assert gb.gac_next_gradient_set(ctx) == gb.GAC_SET_G
    gb.gac_free(ctx)


def test_exchange_mode_needs_one_element_type_and_a_context():
    g = [torch.ones(64, dtype=torch.bfloat16, device="cuda")]
    d = [torch.ones(64, device="cuda")]
    hp = gb.HParams(state_mode=gb.GAC_STATE_EXCHANGE)
    with pytest.raises(gb.GacError) as e:
        gb.gac_init(g, d, hp)
    assert e.value.status == gb.GAC_ERR_DTYPE
    import ctypes
    out = torch.zeros(ctypes.sizeof(gb.gac_result), dtype=torch.uint8, device="cuda")
    with pytest.raises(gb.GacError) as e:
        gb.gac_stats_static(d, [torch.ones(64, device="cuda")], hp, 2, out)
    assert e.value.status == gb.GAC_ERR_INVALID_ARG


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
def test_exchange_mode_fused_adamw(dtype):
    """The fused optimizer step in exchange mode: same p, m, v as the oracle's AdamW on the RAW
    rule's g', and neither buffer set is written at all."""
    shapes = synth.decoder_tensor_list(synth.DIMS["mini"])
    sig = synth.per_tensor_scales(2, len(shapes))
    gen = torch.Generator().manual_seed(7)
    p_cpu = [torch.randn(n, generator=gen) * 0.02 for _, n in shapes]
    m_cpu = [torch.zeros(n) for _, n in shapes]
    v_cpu = [torch.zeros(n) for _, n in shapes]
    sets = [[torch.full((n,), float("nan"), dtype=dtype, device="cuda") for _, n in shapes] for _ in range(2)]
    p_gpu, m_gpu, v_gpu = ([t.cuda() for t in l] for l in (p_cpu, m_cpu, v_cpu))
    hp = gb.HParams(state_mode=gb.GAC_STATE_EXCHANGE, clip_max_norm=0.5)
    ctx = gb.gac_init(sets[0], sets[1], hp)
    gb.gac_attach_adamw(ctx, p_gpu, m_gpu, v_gpu, applied_steps=0)
    gopt, oopt = gb.AdamW(lr=1e-3), orc.AdamW(lr=1e-3)
    ohp = raw_hp(hp)
    d_ref = [torch.full((n,), float("nan"), dtype=dtype) for _, n in shapes]
    applied, regimes = 0, []
    for t, g in enumerate(ar_gradients(shapes, sig, (None, 0.0, 0.3, 0.9, 0.2, 0.01, 0.5), dtype, seed=3), start=1):
        gi = gb.gac_next_gradient_set(ctx)
        assert gi == (t - 1) % 2
        for dst, src in zip(sets[gi], g):
            dst.copy_(src)
        before_d = [x.clone() for x in sets[gi ^ 1]]
        first = t == 1
        dec = orc.decide(orc.stats(g, d_ref, first_step=first), ohp, first)
        m_before = [x.clone() for x in m_cpu]
        d_before = [x.clone().float() for x in d_ref]
        applied += int(orc.project_adamw(g, d_ref, p_cpu, m_cpu, v_cpu, ohp, dec, oopt, applied + 1, first))
        res = gb.gac_stats(ctx, t)
        after = gb.gac_project_adamw(ctx, gopt, coef_override=dec.coef if dec.regime == orc.PROJECT else None,
                                     fetch=True)
        check_sums(res, dec)
        check_decision(res, dec)
        assert after.applied_steps == applied
        for i in range(len(shapes)):
            assert same_bits(sets[gi][i], g[i]) and same_bits(sets[gi][i], d_ref[i])
            assert same_bits(sets[gi ^ 1][i], before_d[i]), "exchange mode stores no state"
            gmag = g[i].float().abs() + abs(dec.coef) * d_before[i].abs().nan_to_num(0.0)
            for name, a, b, slack in (("v", v_gpu[i], v_cpu[i], None),
                                      ("m", m_gpu[i], m_cpu[i], 1e-13 * (m_before[i].abs() + gmag)),
                                      ("p", p_gpu[i], p_cpu[i], torch.full_like(p_cpu[i], 1e-10 * oopt.lr))):
                a_cpu = a.cpu()
                ok = (ordered_int(a_cpu) - ordered_int(b)).abs() <= 4
                if slack is not None:
                    ok |= (a_cpu.double() - b.double()).abs() <= slack.double()
                assert bool(ok.all()), f"step {t} tensor {i} {name}"
                a.copy_(b)       # every step is compared from identical state
        regimes.append(dec.regime)
    assert set(regimes) == {0, 1, 2}
    gb.gac_free(ctx)


@pytest.mark.parametrize("seed", range(12))
def test_exchange_mode_random_list_structures(seed):
    """Random tensor counts and sizes, odd offsets inside larger buffers, thresholds, chunk sizes and
    element types, over three consecutive steps: the values of the RAW rule in the sets the record
    names, and nothing else written."""
    import random
    rng = random.Random(1000 + seed)
    dtype = rng.choice([torch.float32, torch.bfloat16])
    n_t = rng.randint(1, 30)
    sizes = [rng.choice([1, 2, 3, 5, 17, 255, 1024, 4097, 16384, 16385, 70001, rng.randint(1, 200000)])
             for _ in range(n_t)]
    gen = torch.Generator().manual_seed(seed)
    offs = [(rng.randint(0, 7), rng.randint(0, 7)) if rng.random() < 0.3 else (0, 0) for _ in sizes]
    bufs = [[torch.full((n + 8,), 3.0, dtype=dtype, device="cuda") for n in sizes] for _ in range(2)]
    sets = [[b[o[k]:o[k] + n] for b, o, n in zip(bufs[k], offs, sizes)] for k in range(2)]
    hp = rng.choice([gb.HParams(), gb.HParams(c_low=0.05, c_high=2.0), gb.HParams(c_low=0.3, c_high=0.6),
                     gb.HParams(mode=gb.GAC_MODE_FIXED, alpha_fixed=0.0),
                     gb.HParams(c_low=0.05, c_high=2.0, clip_max_norm=0.5)])
    hp = dataclasses.replace(hp, state_mode=gb.GAC_STATE_EXCHANGE)
    ohp = raw_hp(hp)
    ctx = gb.gac_init(sets[0], sets[1], hp)
    gb.gac_set_launch(ctx, rng.choice([1024, 4096, 16384, 32768]), rng.choice([0, 1, 3]))
    scales = [10.0 ** rng.uniform(-4, 0) for _ in sizes]
    d_ref = [(torch.randn(n, generator=gen) * s).to(dtype) for n, s in zip(sizes, scales)]
    for dst, src in zip(sets[1], d_ref):
        dst.copy_(src)
    for t in (2, 3, 4):
        rho = rng.choice([0.0, 0.1, 0.5, 0.95, -0.7])
        g = [(rho * d.float() + math.sqrt(1 - rho * rho) * torch.randn(n, generator=gen) * s).to(dtype)
             for d, n, s in zip(d_ref, sizes, scales)]
        gi = gb.gac_next_gradient_set(ctx)
        assert gi == t % 2
        for dst, src in zip(sets[gi], g):
            dst.copy_(src)
        before_d = [x.clone() for x in sets[gi ^ 1]]
        g_ref = [x.clone() for x in g]
        dec = orc.step(g_ref, d_ref, ohp)               # g_ref <- g', d_ref <- raw g
        res = gb.gac_stats(ctx, t)
        after = gb.gac_project(ctx, coef_override=dec.coef if dec.regime == orc.PROJECT else None, fetch=True)
        check_sums(res, dec)
        for a, b in zip(sets[gi], g):
            assert same_bits(a, b)
        if abs(abs(dec.cos) - hp.c_low) <= 1e-4 or abs(abs(dec.cos) - hp.c_high) <= 1e-4:
            # too close to a threshold to compare decisions: resynchronise the library's state and go on
            for k in range(2):
                for dst, src in zip(sets[k], (g if k == gi else g_ref)):
                    dst.copy_(src)
            continue
        check_decision(res, dec)
        lim = 4 if dtype == torch.float32 else 1
        for a, b in zip(sets[after.out_set], g_ref):
            assert max_ulp(a.cpu(), b) <= lim
        if after.out_set == gi:
            for a, b in zip(sets[gi ^ 1], before_d):
                assert same_bits(a, b)
    for k in range(2):                                  # guard elements around every view
        for b, o, n in zip(bufs[k], offs, sizes):
            assert bool((b[:o[k]] == 3.0).all()) and bool((b[o[k] + n:] == 3.0).all())
    gb.gac_free(ctx)


def test_exchange_mode_steps_replayed_from_cuda_graphs():
    """The role of each buffer set is a launch argument, so one captured step serves every second
    step: two graphs (gradient in the `g` set, gradient in the `d` set) replayed in turn give what
    direct calls give."""
    n = 1 << 20
    hp = gb.HParams(state_mode=gb.GAC_STATE_EXCHANGE, c_low=0.05, c_high=2.0)
    ohp = raw_hp(hp)
    g0, d0 = synth.flat_pair_with_cosine(n, 0.9, s=1.0, seed=0)
    sets = [[g0.cuda()], [d0.cuda()]]
    ctx = gb.gac_init(sets[0], sets[1], hp)
    gb.gac_stats(ctx, 2, fetch=False)            # two warm-up steps outside capture: roles back where they began
    gb.gac_project(ctx)
    gb.gac_stats(ctx, 3, fetch=False)
    gb.gac_project(ctx)
    torch.cuda.synchronize()
    graphs = []
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        for k in range(2):
            assert gb.gac_next_gradient_set(ctx) == k
            gr = torch.cuda.CUDAGraph()
            gr.capture_begin()
            gb.gac_stats(ctx, 4 + k, fetch=False)
            gb.gac_project(ctx)
            gr.capture_end()
            graphs.append(gr)
    torch.cuda.current_stream().wait_stream(side)
    d_ref = [d0.clone()]
    sets[1][0].copy_(d0)
    for t in range(4):
        gi = t % 2
        gen = torch.Generator().manual_seed(50 + t)
        g_new = (0.6 * d_ref[0] + 0.8 * d_ref[0].std() * torch.randn(n, generator=gen))
        sets[gi][0].copy_(g_new)
        graphs[gi].replay()
        torch.cuda.synchronize()
        g_ref = [g_new.clone()]
        dec = orc.step(g_ref, d_ref, ohp)               # d_ref <- raw gradient
        assert dec.regime == orc.PROJECT
        assert same_bits(sets[gi][0], g_new)            # untouched: it is the stored direction now
        out = sets[gi ^ 1][0].cpu()
        # the coefficient is the library's own here (nothing can be overridden inside a replay)
        assert float((out.double() - g_ref[0].double()).abs().max()) <= 2e-7 * float(g_new.abs().max())
    gb.gac_free(ctx)
