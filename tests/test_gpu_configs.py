"""GPU parity on the benchmark configurations at their full sizes, in the
launch configuration that bench.py times.

The lists do not fit host memory as a whole (the 14 B list is 2 x 55 GiB), so
the oracle is fed tensor by tensor: its three sums run over the whole list in
list order; outputs are compared element by element on whole tensors up to
32 M elements and on slices (head, an odd-offset middle, tail) of larger ones,
after regenerating the pre-step values of that tensor from its seeds.  On top
of that the state refresh d' = g is checked on every element of every tensor.
"""
import math
import os

import pytest
import torch

from oracle import gac_oracle as orc
from paper_2603_01501_b200 import binding as gb
from paper_2603_01501_b200 import synth

from gpu_util import check_decision, check_sums, max_ulp, ordered_int, to_orc_hp

pytestmark = pytest.mark.gpu

THREADS = len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else 4
FORCE = dict(c_low=0.05, c_high=2.0)
FULL_LIMIT = 32 << 20
SLICE = 4 << 20


def oracle_sums_streamed(g_list, d_list, first_step=False):
    big = max(t.numel() for t in g_list)
    stage_g = torch.empty(big, dtype=g_list[0].dtype, pin_memory=True)
    stage_d = torch.empty(big, dtype=d_list[0].dtype, pin_memory=True)
    acc = orc.RunningStats(first_step=first_step, threads=THREADS)
    for g, d in zip(g_list, d_list):
        n = g.numel()
        stage_g[:n].copy_(g)
        stage_d[:n].copy_(d)
        torch.cuda.synchronize()
        acc.add(stage_g[:n], stage_d[:n])
    return acc.value()


def slices_of(n):
    if n <= FULL_LIMIT:
        return [(0, n)]
    mid = (n // 2) | 1          # odd offset: not aligned to any vector or chunk boundary
    return [(0, SLICE), (mid, mid + SLICE + 3), (n - SLICE - 1, n)]


def check_outputs_sampled(shapes, rho, config_id, g_dtype, g_gpu, d_gpu, hp, dec):
    ohp = to_orc_hp(hp)
    lim = 4 if g_dtype == torch.float32 else 1
    d_dtype = d_gpu[0].dtype
    worst = 0
    for i in range(len(shapes)):
        (g0,), (d0,) = synth.gradient_list(shapes, rho, config_id, g_dtype, "cuda", indices=[i])
        d0 = d0.to(d_dtype)
        # state refresh: exact copy (or exact widening) of the raw gradient, every element
        assert torch.equal(d_gpu[i], g0.to(d_dtype)), f"tensor {i}: d' != raw g"
        if dec.regime != orc.PROJECT:
            assert torch.equal(g_gpu[i], g0), f"tensor {i}: g changed outside the projection regime"
            continue
        for lo, hi in slices_of(g0.numel()):
            g_ref = g0[lo:hi].cpu().contiguous()
            d_ref = d0[lo:hi].cpu().contiguous()
            orc.project([g_ref], [d_ref], ohp, dec, threads=THREADS)
            u = max_ulp(g_gpu[i][lo:hi].cpu(), g_ref)
            assert u <= lim, f"tensor {i} [{lo}:{hi}]: g' differs by {u} ulp"
            worst = max(worst, u)
            assert torch.equal(d_gpu[i][lo:hi].cpu(), d_ref)
        del g0, d0
    return worst


def test_config_fused_adamw_full_size():
    """The projection fused with AdamW on the 7 B list (bf16 g, f32 d; 137 GB resident with p, m, v), in the
    configuration bench.py times: one projection step with t = 6.  The oracle's sums run over every element;
    p, m, v are compared on three slices of every tensor (whole tensors up to 32 M elements) with the bars of
    the per-step test; d' = g is checked on every element and g must come out untouched."""
    dims_key, g_dtype, rho, config_id = synth.WORKLOADS["cfg3_7b_bf16"]
    shapes = synth.decoder_tensor_list(synth.DIMS[dims_key])
    torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info()
    if free < (160 << 30):
        pytest.skip(f"needs 160 GiB of device memory, {free >> 30} GiB free")
    hp = gb.HParams(**FORCE)
    ohp = to_orc_hp(hp)
    gopt, oopt = gb.AdamW(lr=1e-4), orc.AdamW(lr=1e-4)

    def state(i, n):
        gen = torch.Generator(device="cuda").manual_seed(77_000 + i)
        p = torch.randn(n, generator=gen, device="cuda") * 0.02
        m = torch.randn(n, generator=gen, device="cuda") * 1e-3
        v = torch.rand(n, generator=gen, device="cuda") * 1e-6
        return p, m, v

    g, d = synth.gradient_list(shapes, rho, config_id, g_dtype, "cuda")
    p, m, v = (list(x) for x in zip(*(state(i, n) for i, (_, n) in enumerate(shapes))))
    dec = orc.decide(oracle_sums_streamed(g, d), ohp)
    assert dec.regime == orc.PROJECT
    ctx = gb.gac_init(g, d, hp)
    gb.gac_attach_adamw(ctx, p, m, v, applied_steps=5)
    res = gb.gac_stats(ctx, 2)
    after = gb.gac_project_adamw(ctx, gopt, coef_override=dec.coef, fetch=True)
    torch.cuda.synchronize()
    check_sums(res, dec)
    check_decision(res, dec)
    assert after.applied_steps == 6
    gb.gac_free(ctx)
    for i, (_, n) in enumerate(shapes):
        (g0,), (d0,) = synth.gradient_list(shapes, rho, config_id, g_dtype, "cuda", indices=[i])
        assert torch.equal(g[i].view(torch.int16), g0.view(torch.int16)), f"tensor {i}: g was written"
        assert torch.equal(d[i], g0.float()), f"tensor {i}: d' != raw g"
        p0, m0, v0 = state(i, n)
        for lo, hi in slices_of(n):
            ref = [x[lo:hi].cpu().contiguous() for x in (g0, d0, p0, m0, v0)]
            m_before = ref[3].clone()
            gmag = ref[0].float().abs() + abs(dec.coef) * ref[1].abs()
            orc.project_adamw([ref[0]], [ref[1]], [ref[2]], [ref[3]], [ref[4]], ohp, dec, oopt, 6)
            for name, got, want, slack in (("v", v[i], ref[4], None),
                                           ("m", m[i], ref[3], 1e-13 * (m_before.abs() + gmag)),
                                           ("p", p[i], ref[2], torch.full_like(ref[2], 1e-10 * oopt.lr))):
                a = got[lo:hi].cpu()
                ulps = (ordered_int(a) - ordered_int(want)).abs()
                ok = ulps <= 4
                if slack is not None:
                    ok |= (a.double() - want.double()).abs() <= slack.double()
                assert bool(ok.all()), f"tensor {i} [{lo}:{hi}] {name}: {int(ulps[~ok].max())} ulp"
        del g0, d0, p0, m0, v0
    del g, d, p, m, v
    torch.cuda.empty_cache()


def run_config(workload, hp):
    dims_key, g_dtype, rho, config_id = synth.WORKLOADS[workload]
    d_dtype = synth.WORKLOAD_D_DTYPE.get(workload, torch.float32)
    shapes = synth.decoder_tensor_list(synth.DIMS[dims_key])
    need = synth.list_numel(shapes) * ((2 if g_dtype == torch.bfloat16 else 4) + 4) + (12 << 30)
    torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info()
    if free < need:
        pytest.skip(f"needs {need >> 30} GiB of device memory, {free >> 30} GiB free")
    g, d = synth.gradient_list(shapes, rho, config_id, g_dtype, "cuda")
    if d_dtype != torch.float32:
        d = [t.to(d_dtype) for t in d]
    dec = orc.decide(oracle_sums_streamed(g, d), to_orc_hp(hp))
    ctx = gb.gac_init(g, d, hp)
    res = gb.gac_stats(ctx, 2, staleness=1)
    again = gb.gac_stats(ctx, 2, staleness=1)
    assert (res.dot, res.gg, res.dd, res.cos) == (again.dot, again.gg, again.dd, again.cos)
    check_sums(res, dec)
    check_decision(res, dec)
    assert abs(res.cos - rho) < 2e-3
    gb.gac_project(ctx, coef_override=dec.coef if dec.regime == orc.PROJECT else None)
    torch.cuda.synchronize()
    worst = check_outputs_sampled(shapes, rho, config_id, g_dtype, g, d, hp, dec)
    gb.gac_free(ctx)
    del g, d
    torch.cuda.empty_cache()
    return res, dec, worst


@pytest.mark.parametrize("workload", ["cfg2_1.5b_f32", "cfg3_7b_bf16", "cfg5_14b_f32", "cfg3_7b_bf16_dbf16"])
def test_config_projection_regime(workload):
    res, dec, worst = run_config(workload, gb.HParams(**FORCE))
    assert res.regime == gb.GAC_REGIME_PROJECT
    assert abs(res.alpha - 0.05 / abs(res.cos)) <= 1e-12


@pytest.mark.parametrize("workload", ["cfg2_1.5b_f32", "cfg3_7b_bf16", "cfg5_14b_f32"])
def test_config_paper_defaults_is_a_violation_step(workload):
    # every configured cosine (0.8 .. 0.95) is above the paper's c_high = 0.3
    res, dec, _ = run_config(workload, gb.HParams())
    assert res.regime == gb.GAC_REGIME_VIOLATION


# ------------------------------------------------------------ staleness runs

def staleness_run(shapes, rho, k, run_id, steps, hp, full_outputs):
    """Feeds the same exogenous gradient sequence to both sides, carrying the
    stored direction across steps on each side independently."""
    proc = synth.StalenessProcess(shapes, rho, k, config_id=4, run_id=run_id, device="cuda")
    g = [torch.empty(n, device="cuda") for _, n in shapes]
    d = [torch.full((n,), float("nan"), device="cuda") for _, n in shapes]
    ctx = gb.gac_init(g, d, hp)
    ohp = to_orc_hp(hp)
    d_ref = [torch.full((n,), float("nan")) for _, n in shapes] if full_outputs else None
    prev_raw = None
    log = []
    for t in range(1, steps + 1):
        raw = proc.next()
        for dst, src in zip(g, raw):
            dst.copy_(src)
        first = (t == 1)
        if full_outputs:
            g_ref = [x.cpu() for x in raw]
            dec = orc.decide(orc.stats(g_ref, d_ref, first_step=first, threads=THREADS), ohp, first)
            orc.project(g_ref, d_ref, ohp, dec, first_step=first, threads=THREADS)
        else:
            # the state is the previous raw gradient (checked bitwise below), so the oracle's
            # sums for this step are those of (raw_t, raw_{t-1})
            sums = oracle_sums_streamed(raw, prev_raw if prev_raw is not None else raw, first)
            dec = orc.decide(sums, ohp, first)
        res = gb.gac_stats(ctx, t, staleness=k)
        gb.gac_project(ctx, coef_override=dec.coef if dec.regime == orc.PROJECT else None)
        torch.cuda.synchronize()
        check_sums(res, dec)
        check_decision(res, dec)
        for i, (a, b) in enumerate(zip(d, raw)):
            assert torch.equal(a, b), f"step {t} tensor {i}: state is not the raw gradient"
        if full_outputs:
            lim = 4
            for a, b in zip(g, g_ref):
                assert max_ulp(a.cpu(), b) <= lim
        elif dec.regime == orc.PROJECT:
            # sampled outputs: one slice per tensor against the oracle
            for i in range(0, len(shapes), 7):
                n = shapes[i][1]
                lo = (n // 3) | 1 if n > SLICE else 0
                hi = min(n, lo + SLICE)
                g_s = raw[i][lo:hi].cpu().contiguous()
                d_s = prev_raw[i][lo:hi].cpu().contiguous()
                orc.project([g_s], [d_s], ohp, dec)
                assert max_ulp(g[i][lo:hi].cpu(), g_s) <= 4
        prev_raw = raw
        log.append((res.cos, res.regime, res.alpha))
    gb.gac_free(ctx)
    return log


@pytest.mark.parametrize("rho", [0.0, 0.5, 0.95])
@pytest.mark.parametrize("k", [1, 4, 8])
def test_staleness_runs_scaled_down_all_steps(rho, k):
    """64 consecutive steps for every (rho, k) on a scaled-down list of the same
    structure, every element of every step compared."""
    shapes = synth.decoder_tensor_list(synth.DIMS["mini"])
    band = gb.HParams(c_low=0.05, c_high=0.99)
    log = staleness_run(shapes, rho, k, run_id=int(rho * 100) * 10 + k, steps=64, hp=band,
                        full_outputs=True)
    assert log[0][1] == gb.GAC_REGIME_SAFE and log[0][0] == 0.0
    cs = [abs(c) for c, _, _ in log[1 + k:]]
    if rho == 0.0:
        assert max(cs) < 0.05
    else:
        assert sum(cs) / len(cs) > 0.1
    log2 = staleness_run(shapes, rho, k, run_id=int(rho * 100) * 10 + k, steps=12, hp=gb.HParams(),
                         full_outputs=True)
    assert [r for _, r, _ in log2][0] == gb.GAC_REGIME_SAFE


def staleness_run_full_size(shapes, rho, k, run_id, steps, hp, host):
    """The same comparison on a list too large to replay element by element on the host every step.
    Both sides get the same exogenous sequence.  Per step: the oracle's three sums over EVERY element
    (host copies of this step's and the previous step's raw gradient -- the state, checked bitwise on
    every element on the device, IS the previous raw gradient), its decision, and its projection on one
    odd-offset slice of every seventh tensor; regime exact, sums and cosine 1e-5, g' within 4 ulp."""
    proc = synth.StalenessProcess(shapes, rho, k, config_id=4, run_id=run_id, device="cuda")
    g = [torch.empty(n, device="cuda") for _, n in shapes]
    d = [torch.full((n,), float("nan"), device="cuda") for _, n in shapes]
    ctx = gb.gac_init(g, d, hp)
    ohp = to_orc_hp(hp)
    h_cur, h_prev = host
    log = []
    for t in range(1, steps + 1):
        raw = proc.next()
        for dst, src, h in zip(g, raw, h_cur):
            dst.copy_(src)
            h.copy_(src, non_blocking=True)
        torch.cuda.synchronize()
        first = (t == 1)
        acc = orc.RunningStats(first_step=first, threads=THREADS)
        for a, b in zip(h_cur, h_prev):
            acc.add(a, b)
        dec = orc.decide(acc.value(), ohp, first)
        res = gb.gac_stats(ctx, t, staleness=k)
        gb.gac_project(ctx, coef_override=dec.coef if dec.regime == orc.PROJECT else None)
        torch.cuda.synchronize()
        check_sums(res, dec)
        check_decision(res, dec)
        for i, (a, b) in enumerate(zip(d, raw)):
            assert torch.equal(a, b), f"step {t} tensor {i}: state is not the raw gradient"
        for i in range(0, len(shapes), 7):
            n = shapes[i][1]
            lo = (n // 3) | 1 if n > SLICE else 0
            hi = min(n, lo + SLICE)
            if dec.regime == orc.PROJECT:
                g_s = h_cur[i][lo:hi].clone()
                d_s = h_prev[i][lo:hi].clone()
                orc.project([g_s], [d_s], ohp, dec)
                assert max_ulp(g[i][lo:hi].cpu(), g_s) <= 4, f"step {t} tensor {i}"
            else:
                assert torch.equal(g[i][lo:hi].cpu(), h_cur[i][lo:hi]), f"step {t} tensor {i}: g changed"
        h_cur, h_prev = h_prev, h_cur
        log.append((res.cos, res.regime, res.alpha))
        del raw
    gb.gac_free(ctx)
    return log


def test_staleness_runs_full_size_every_setting():
    """Every (rho, k) of the staleness configuration on the 1.5 B list at full size, state carried from
    step to step: 16 steps per setting (enough to fill the k = 8 window twice); GAC_FULL_STALENESS=1 runs
    the 64 steps of the configuration.  The band (0.05, 0.9) makes the nine runs meet all three regimes."""
    shapes = synth.decoder_tensor_list(synth.DIMS["1.5b"])
    torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info()
    if free < (110 << 30):
        pytest.skip(f"needs 110 GiB of device memory, {free >> 30} GiB free")
    steps = 64 if os.environ.get("GAC_FULL_STALENESS") == "1" else 16
    band = gb.HParams(c_low=0.05, c_high=0.9)
    host = tuple([torch.empty(n, dtype=torch.float32, pin_memory=True) for _, n in shapes] for _ in range(2))
    seen = set()
    for rho in (0.0, 0.5, 0.95):
        for k in (1, 4, 8):
            log = staleness_run_full_size(shapes, rho, k, run_id=900 + int(rho * 100) * 10 + k, steps=steps,
                                          hp=band, host=host)
            assert log[0][1] == gb.GAC_REGIME_SAFE and log[0][0] == 0.0
            regimes = [r for _, r, _ in log[1:]]
            if rho == 0.0:
                assert all(r == gb.GAC_REGIME_SAFE for r in regimes)
                assert max(abs(c) for c, _, _ in log) < 1e-3
            else:
                assert all(r != gb.GAC_REGIME_SAFE for r in regimes)
            if k == 1 and rho > 0:            # AR(1): the cosine to the previous gradient is rho itself
                assert all(abs(c - rho) < 5e-3 for c, _, _ in log[1:])
            seen |= set(regimes)
            torch.cuda.empty_cache()
    assert seen == {gb.GAC_REGIME_SAFE, gb.GAC_REGIME_PROJECT, gb.GAC_REGIME_VIOLATION}


def test_single_tensor_beyond_32bit_indexing():
    """One tensor of 2^32 + 4099 elements (bfloat16 pair, 8.6 GB per buffer): element offsets do not
    fit 32 bits; sums over all of it, outputs on slices around the 2^32 boundary and at both ends."""
    n = (1 << 32) + 4099
    free, _ = torch.cuda.mem_get_info()
    if free < (40 << 30):
        pytest.skip("needs 40 GiB of device memory")
    gen = torch.Generator(device="cuda").manual_seed(99)
    d = torch.empty(n, dtype=torch.bfloat16, device="cuda")
    g = torch.empty(n, dtype=torch.bfloat16, device="cuda")
    step = 1 << 28
    for lo in range(0, n, step):            # generated piecewise to bound temporaries
        hi = min(n, lo + step)
        z = torch.randn(hi - lo, generator=gen, device="cuda")
        w = torch.randn(hi - lo, generator=gen, device="cuda")
        d[lo:hi] = (0.01 * z).to(torch.bfloat16)
        g[lo:hi] = (0.005 * z + 0.00866 * w).to(torch.bfloat16)
    g0, d0 = g.clone(), d.clone()
    hp = gb.HParams(**FORCE)
    dec = orc.decide(oracle_sums_streamed([g], [d]), to_orc_hp(hp))
    ctx = gb.gac_init([g], [d], hp)
    res = gb.gac_stats(ctx, 2)
    gb.gac_project(ctx, coef_override=dec.coef)
    torch.cuda.synchronize()
    gb.gac_free(ctx)
    check_sums(res, dec)
    check_decision(res, dec)
    assert dec.regime == orc.PROJECT and abs(res.cos - 0.5) < 0.01
    assert torch.equal(d.view(torch.int16), g0.view(torch.int16))       # state = raw gradient, every element
    for lo, hi in [(0, SLICE), ((1 << 32) - SLICE // 2 - 1, (1 << 32) + 4099), ((1 << 31) + 1, (1 << 31) + SLICE)]:
        g_ref, d_ref = g0[lo:hi].cpu().contiguous(), d0[lo:hi].cpu().contiguous()
        orc.project([g_ref], [d_ref], to_orc_hp(hp), dec, threads=THREADS)
        assert max_ulp(g[lo:hi].cpu(), g_ref) <= 1
        assert torch.equal(d[lo:hi].cpu().view(torch.int16), d_ref.view(torch.int16))


# ------------------------------------------------- exchange mode at full size

@pytest.mark.parametrize("workload", ["cfg2_1.5b_f32", "cfg5_14b_f32"])
def test_config_exchange_mode_two_steps(workload):
    """Exchange mode on the full-size float32 lists, in the configuration bench.py times: two
    consecutive projection steps, so that both assignments of the roles run at full size.  The
    oracle computes the plain rule (d' = g by copy); here g' must appear in the buffers that held
    d and the buffers that held g must come out untouched, every element."""
    dims_key, g_dtype, rho, config_id = synth.WORKLOADS[workload]
    shapes = synth.decoder_tensor_list(synth.DIMS[dims_key])
    need = synth.list_numel(shapes) * 8 + (12 << 30)
    free, _ = torch.cuda.mem_get_info()
    if free < need:
        pytest.skip(f"needs {need >> 30} GiB of device memory, {free >> 30} GiB free")
    hp = gb.HParams(state_mode=gb.GAC_STATE_EXCHANGE, **FORCE)
    ohp = to_orc_hp(gb.HParams(**FORCE))
    a, b = synth.gradient_list(shapes, rho, config_id, g_dtype, "cuda")       # a: gradient, b: stored direction
    ctx = gb.gac_init(a, b, hp)

    # step 2: gradient in a, direction in b, g' lands in b
    dec = orc.decide(oracle_sums_streamed(a, b), ohp)
    res = gb.gac_stats(ctx, 2)
    after = gb.gac_project(ctx, coef_override=dec.coef, fetch=True)
    check_sums(res, dec)
    check_decision(res, dec)
    assert dec.regime == orc.PROJECT and (after.g_set, after.out_set) == (gb.GAC_SET_G, gb.GAC_SET_D)
    for i in range(len(shapes)):
        (g0,), (d0,) = synth.gradient_list(shapes, rho, config_id, g_dtype, "cuda", indices=[i])
        assert torch.equal(a[i], g0), f"tensor {i}: the gradient buffers were modified"
        for lo, hi in slices_of(g0.numel()):
            g_ref, d_ref = g0[lo:hi].cpu().contiguous(), d0[lo:hi].cpu().contiguous()
            orc.project([g_ref], [d_ref], ohp, dec, threads=THREADS)
            u = max_ulp(b[i][lo:hi].cpu(), g_ref)
            assert u <= 4, f"step 2 tensor {i} [{lo}:{hi}]: g' differs by {u} ulp"
        del g0, d0

    # step 3: the roles have swapped -- the next gradient goes into b, a is the stored direction
    assert gb.gac_next_gradient_set(ctx) == gb.GAC_SET_D
    sigma = synth.per_tensor_scales(config_id, len(shapes))
    gen = torch.Generator(device="cuda").manual_seed(4242)
    scratch = torch.empty(max(n for _, n in shapes), dtype=torch.float32, device="cuda")
    synth.refresh_gradient_list(b, a, sigma, rho, gen, scratch)
    del scratch
    dec = orc.decide(oracle_sums_streamed(b, a), ohp)
    res = gb.gac_stats(ctx, 3)
    after = gb.gac_project(ctx, coef_override=dec.coef, fetch=True)
    check_sums(res, dec)
    check_decision(res, dec)
    assert dec.regime == orc.PROJECT and (after.g_set, after.out_set) == (gb.GAC_SET_D, gb.GAC_SET_G)
    assert abs(res.cos - rho) < 2e-3
    for i in range(len(shapes)):
        (d0,), _ = synth.gradient_list(shapes, rho, config_id, g_dtype, "cuda", indices=[i])   # a before this step
        for lo, hi in slices_of(d0.numel()):
            g_ref, d_ref = b[i][lo:hi].cpu().contiguous(), d0[lo:hi].cpu().contiguous()
            g_in = g_ref.clone()
            orc.project([g_ref], [d_ref], ohp, dec, threads=THREADS)
            u = max_ulp(a[i][lo:hi].cpu(), g_ref)
            assert u <= 4, f"step 3 tensor {i} [{lo}:{hi}]: g' differs by {u} ulp"
            assert torch.equal(d_ref, g_in)        # the rule's new direction is the raw gradient: b, untouched
        del d0
    gb.gac_free(ctx)
    del a, b
    torch.cuda.empty_cache()
