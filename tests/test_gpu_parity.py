"""GPU parity: the CUDA library, called through its C ABI, against the CPU
oracle on the same seeded inputs, element by element."""
import math

import numpy as np
import pytest
import torch

from oracle import gac_oracle as orc
from paper_2603_01501_b200 import binding as gb
from paper_2603_01501_b200 import synth

from gpu_util import (check_decision, check_outputs, check_sums, max_ulp, step_both, to_orc_hp)

pytestmark = pytest.mark.gpu

FORCE = dict(c_low=0.05, c_high=2.0)      # legal (c_high > 1): every |c| > c_low is projected


def rand_pair(n, rho, seed, g_dtype=torch.float32, scale=1.0):
    gen = torch.Generator().manual_seed(seed)
    d = torch.randn(n, generator=gen) * scale
    w = torch.randn(n, generator=gen) * scale
    g = (rho * d + math.sqrt(max(0.0, 1 - rho * rho)) * w).to(g_dtype)
    return g, d


# ------------------------------------------------------------------ config 1

@pytest.mark.parametrize("hp", [gb.HParams(), gb.HParams(**FORCE),
                                gb.HParams(mode=gb.GAC_MODE_FIXED, alpha_fixed=0.0)],
                         ids=["defaults", "forced_projection", "full_projection"])
def test_flat_pair_2pow20(hp):
    g, d = synth.flat_pair_with_cosine(1 << 20, 0.9, s=1.0, seed=0)
    res, dec, gg, dg, gr, dr = step_both([g], [d], hp)
    check_sums(res, dec)
    check_decision(res, dec)
    assert abs(res.cos - 0.9) < 1e-6
    assert res.regime == (gb.GAC_REGIME_VIOLATION if hp.mode == 0 and hp.c_high < 0.9
                          else gb.GAC_REGIME_PROJECT)
    check_outputs(gg, dg, gr, dr)
    if hp.mode == gb.GAC_MODE_FIXED:      # g' orthogonal to d after a full projection
        d64 = d.double()
        assert abs(float(torch.dot(gg[0].cpu().double(), d64))) <= 1e-6 * math.sqrt(res.gg * res.dd)


# ------------------------------------------------- sizes, tails, several tiles

SIZES = [1, 2, 3, 4, 5, 7, 255, 256, 1023, 1024, 1025, 4095, 4096, 4097, 16383, 16384, 16385,
         5 * 16384 + 7, 1_000_003]


@pytest.mark.parametrize("g_dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("n", SIZES)
def test_single_tensor_sizes(n, g_dtype):
    g, d = rand_pair(n, 0.5, seed=n, g_dtype=g_dtype, scale=0.01)
    res, dec, gg, dg, gr, dr = step_both([g], [d], gb.HParams(**FORCE))
    check_sums(res, dec)
    check_decision(res, dec)
    check_outputs(gg, dg, gr, dr)


@pytest.mark.parametrize("g_dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("name,rho", [("mini", 0.2), ("small", 0.8)])
def test_decoder_shaped_lists(name, rho, g_dtype):
    shapes = synth.decoder_tensor_list(synth.DIMS[name])
    g, d = synth.gradient_list(shapes, rho, config_id=2, g_dtype=g_dtype)
    for hp in (gb.HParams(), gb.HParams(**FORCE)):
        res, dec, gg, dg, gr, dr = step_both(g, d, hp)
        check_sums(res, dec)
        check_decision(res, dec)
        check_outputs(gg, dg, gr, dr)
        assert abs(res.cos - rho) < 0.02


@pytest.mark.parametrize("launch", [(1024, 1), (4096, 2), (65536, 8)])
def test_launch_geometry_does_not_change_results(launch):
    shapes = synth.decoder_tensor_list(synth.DIMS["small"])
    g, d = synth.gradient_list(shapes, 0.6, config_id=2)
    res, dec, gg, dg, gr, dr = step_both(g, d, gb.HParams(**FORCE), launch=launch)
    check_sums(res, dec, rel=1e-12)
    check_decision(res, dec)
    check_outputs(gg, dg, gr, dr)


@pytest.mark.parametrize("g_dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
def test_misaligned_views_and_guard_regions(g_dtype):
    """Tensors that start at odd element offsets inside larger buffers (views):
    the element-wise path must give the same results, and nothing outside the
    views may be touched."""
    torch.manual_seed(5)
    sizes = [1, 3, 1000, 16384, 40001]
    offs = [1, 3, 5, 2, 7]
    hp = gb.HParams(**FORCE)
    g_cpu, d_cpu, g_buf, d_buf, g_view, d_view = [], [], [], [], [], []
    for n, o in zip(sizes, offs):
        g, d = rand_pair(n, 0.4, seed=n + 1, g_dtype=g_dtype)
        g_cpu.append(g)
        d_cpu.append(d)
        gbuf = torch.full((n + 16,), 7.0, dtype=g_dtype, device="cuda")
        dbuf = torch.full((n + 16,), -9.0, dtype=torch.float32, device="cuda")
        gbuf[o:o + n] = g.cuda()
        dbuf[o + 1:o + 1 + n] = d.cuda()
        g_buf.append(gbuf)
        d_buf.append(dbuf)
        g_view.append(gbuf[o:o + n])
        d_view.append(dbuf[o + 1:o + 1 + n])
    ohp = to_orc_hp(hp)
    g_ref, d_ref = [t.clone() for t in g_cpu], [t.clone() for t in d_cpu]
    dec = orc.step(g_ref, d_ref, ohp)
    ctx = gb.gac_init(g_view, d_view, hp)
    assert gb.gac_get_info(ctx).misaligned_tensors == len(sizes)
    res = gb.gac_stats(ctx, 2)
    gb.gac_project(ctx, coef_override=dec.coef)
    torch.cuda.synchronize()
    check_sums(res, dec)
    check_decision(res, dec)
    check_outputs(g_view, d_view, g_ref, d_ref)
    for n, o, gbuf, dbuf in zip(sizes, offs, g_buf, d_buf):
        assert bool((gbuf[:o] == 7.0).all()) and bool((gbuf[o + n:] == 7.0).all())
        assert bool((dbuf[:o + 1] == -9.0).all()) and bool((dbuf[o + 1 + n:] == -9.0).all())


# ------------------------------------------------------- regimes and readings

def test_three_regimes_and_raw_state_over_steps():
    torch.manual_seed(1)
    n = 70_001
    hp = gb.HParams()           # paper defaults 0.05 / 0.3
    d0 = torch.randn(n)
    d_gpu = [torch.full((n,), float("nan"), device="cuda")]      # never read on step 1
    g_gpu = [torch.empty(n, device="cuda")]
    ctx = gb.gac_init(g_gpu, d_gpu, hp)
    d_ref = [torch.full((n,), float("nan"))]
    seen = []
    prev = d0
    for t, rho in enumerate([None, 0.0, 0.15, 0.8, 0.02, 0.2], start=1):
        g = torch.randn(n) if rho is None else rho * prev + math.sqrt(1 - rho * rho) * torch.randn(n)
        prev = g.clone()
        g_gpu[0].copy_(g)
        g_ref = [g.clone()]
        dec = orc.step(g_ref, d_ref, to_orc_hp(hp), first_step=(t == 1))
        res = gb.gac_stats(ctx, t, staleness=t % 3)
        gb.gac_project(ctx, coef_override=dec.coef if dec.regime == orc.PROJECT else None)
        assert res.step == t and res.staleness == t % 3
        if t == 1:
            assert (res.dot, res.dd, res.cos, res.regime) == (0.0, 0.0, 0.0, gb.GAC_REGIME_SAFE)
        check_sums(res, dec)
        check_decision(res, dec)
        check_outputs(g_gpu, d_gpu, g_ref, d_ref)
        assert torch.equal(d_gpu[0].cpu(), g)               # state = raw gradient, every regime
        seen.append(res.regime)
    assert set(seen) == {0, 1, 2}
    gb.gac_free(ctx)


@pytest.mark.parametrize("hp", [
    gb.HParams(zero_on_violation=1),
    gb.HParams(**FORCE, state_mode=gb.GAC_STATE_PROJECTED),
    gb.HParams(**FORCE, state_mode=gb.GAC_STATE_HOLD),
    gb.HParams(mode=gb.GAC_MODE_FIXED, alpha_fixed=0.25, beta=1.5),
    gb.HParams(mode=gb.GAC_MODE_FIXED, alpha_fixed=2.0, beta=0.5, state_mode=gb.GAC_STATE_PROJECTED),
    gb.HParams(zero_on_violation=1, state_mode=gb.GAC_STATE_PROJECTED),
    gb.HParams(zero_on_violation=1, state_mode=gb.GAC_STATE_HOLD),
    gb.HParams(state_mode=gb.GAC_STATE_HOLD),
], ids=["zero_on_violation", "projected_state", "hold_state", "fixed_gains", "fixed_gains_projected",
        "zero_projected", "zero_hold", "violation_hold"])
@pytest.mark.parametrize("g_dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
def test_variants(hp, g_dtype):
    g, d = rand_pair(50_003, 0.7, seed=3, g_dtype=g_dtype)
    res, dec, gg, dg, gr, dr = step_both([g], [d], hp)
    check_sums(res, dec)
    check_decision(res, dec)
    follows = hp.state_mode == gb.GAC_STATE_PROJECTED and res.regime == gb.GAC_REGIME_PROJECT
    check_outputs(gg, dg, gr, dr, d_follows_g=follows)


@pytest.mark.parametrize("g_dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
@pytest.mark.parametrize("max_norm", [1e-3, 0.3, 1e6])
@pytest.mark.parametrize("thr", [FORCE, dict(c_low=0.9, c_high=0.95), dict()], ids=["project", "safe", "violation"])
def test_clipping_folded_into_the_projection_pass(thr, max_norm, g_dtype):
    """Global-norm clipping (Table 2) from the closed-form norm: same factor and
    same outputs as the oracle's brute-force norm over every element."""
    shapes = synth.decoder_tensor_list(synth.DIMS["small"])
    g, d = synth.gradient_list(shapes, 0.6, config_id=2, g_dtype=g_dtype)
    hp = gb.HParams(clip_max_norm=max_norm, **thr)
    res, dec, gg, dg, gr, dr = step_both(g, d, hp)
    check_sums(res, dec)
    check_decision(res, dec)
    after = res.after
    if dec.regime == orc.VIOLATION:
        assert after.clip_scale == 1.0 and dec.clip_scale == 1.0
    else:
        assert abs(after.out_norm - dec.out_norm) <= 1e-9 * dec.out_norm
        assert abs(after.clip_scale - dec.clip_scale) <= 1e-9 * dec.clip_scale
        assert (dec.clip_scale < 1.0) == (max_norm < 1e6)
    check_outputs(gg, dg, gr, dr)


def test_degenerate_vectors():
    n = 5000
    g, d = rand_pair(n, 0.5, seed=9)
    z = torch.zeros(n)
    for gv, dv in [(g, z), (z, d), (z, z), (g, g.clone()), (g, -g)]:
        for hp in (gb.HParams(), gb.HParams(eps=0.0)):
            res, dec, gg, dg, gr, dr = step_both([gv.clone()], [dv.clone()], hp)
            check_sums(res, dec)
            check_decision(res, dec)
            check_outputs(gg, dg, gr, dr)
    res, *_ = step_both([g], [g.clone()], gb.HParams(eps=0.0))
    assert abs(res.cos - 1.0) < 1e-12 and res.regime == gb.GAC_REGIME_VIOLATION


def test_nonfinite_is_reported_and_nothing_is_written():
    g, d = rand_pair(10_000, 0.5, seed=2)
    g[1234] = float("inf")
    g_gpu, d_gpu = [g.cuda()], [d.cuda()]
    ctx = gb.gac_init(g_gpu, d_gpu, gb.HParams())
    res = gb.gac_stats(ctx, 2)
    gb.gac_project(ctx)
    torch.cuda.synchronize()
    assert res.nonfinite == 1 and res.regime == gb.GAC_REGIME_VIOLATION
    assert torch.equal(d_gpu[0].cpu(), d)
    assert torch.equal(g_gpu[0].cpu().view(torch.int32), g.view(torch.int32))
    L = gb.load_library()
    r = gb.gac_result()
    import ctypes
    assert L.gac_stats(ctx.handle, 3, 0, None, ctypes.byref(r)) == gb.GAC_ERR_NONFINITE
    gb.gac_free(ctx)


def test_threshold_equality_is_inclusive_on_device():
    """Exact-equality scalars through gac_decide: |c| == c_low is safe and
    |c| == c_high is a violation (Algorithm 1)."""
    g, d = [torch.ones(8, device="cuda")], [torch.ones(8, device="cuda")]
    sums = torch.tensor([1.0, 4.0, 4.0], dtype=torch.float64, device="cuda")    # c = 0.25 exactly
    scratch = torch.zeros(3, dtype=torch.float64, device="cuda")
    for hp, want in [(gb.HParams(c_low=0.25, c_high=0.5, eps=0.0), gb.GAC_REGIME_SAFE),
                     (gb.HParams(c_low=0.125, c_high=0.25, eps=0.0), gb.GAC_REGIME_VIOLATION),
                     (gb.HParams(c_low=0.125, c_high=0.5, eps=0.0), gb.GAC_REGIME_PROJECT)]:
        ctx = gb.gac_init(g, d, hp)
        gb.gac_stats_partial(ctx, 2, scratch)
        res = gb.gac_decide(ctx, sums)
        assert res.cos == 0.25 and res.regime == want
        dec = orc.decide((1.0, 4.0, 4.0), to_orc_hp(hp))
        assert (res.alpha, res.coef64, res.coef) == (dec.alpha, dec.coef64, dec.coef)
        gb.gac_free(ctx)


# --------------------------------------------------- determinism, sharded form

def test_stats_are_bitwise_reproducible():
    shapes = synth.decoder_tensor_list(synth.DIMS["small"])
    g, d = synth.gradient_list(shapes, 0.3, config_id=2, device="cuda")
    ctx = gb.gac_init(g, d, gb.HParams())
    first = None
    for _ in range(10):
        r = gb.gac_stats(ctx, 2)
        key = (r.dot, r.gg, r.dd, r.cos)
        first = first or key
        assert key == first
    gb.gac_free(ctx)


def test_sharded_partial_sums_add_up_to_the_whole():
    """App. A.1: per-shard inner products, one sum of three numbers, same decision."""
    shapes = synth.decoder_tensor_list(synth.DIMS["small"])
    g, d = synth.gradient_list(shapes, 0.2, config_id=2, device="cuda")
    hp = gb.HParams(**FORCE)
    whole = gb.gac_init(g, d, hp)
    ref = gb.gac_stats(whole, 2)
    cut = len(g) // 2
    parts = [gb.gac_init(g[:cut], d[:cut], hp), gb.gac_init(g[cut:], d[cut:], hp)]
    bufs = [torch.zeros(3, dtype=torch.float64, device="cuda") for _ in parts]
    for c, b in zip(parts, bufs):
        gb.gac_stats_partial(c, 2, b)
    total = bufs[0] + bufs[1]            # stands for the all-reduce
    results = [gb.gac_decide(c, total) for c in parts]
    for r in results:
        assert abs(r.dot - ref.dot) <= 1e-12 * abs(ref.dot)
        assert abs(r.gg - ref.gg) <= 1e-12 * ref.gg and abs(r.dd - ref.dd) <= 1e-12 * ref.dd
        assert r.regime == ref.regime
    assert results[0].coef == results[1].coef and results[0].cos == results[1].cos
    g_ref = [t.cpu() for t in g]
    d_ref = [t.cpu() for t in d]
    dec = orc.decide(orc.stats(g_ref, d_ref), to_orc_hp(hp))
    orc.project(g_ref, d_ref, to_orc_hp(hp), dec)
    for c in parts:
        gb.gac_project(c, coef_override=dec.coef)
    torch.cuda.synchronize()
    check_outputs(g, d, g_ref, d_ref)
    for c in parts + [whole]:
        gb.gac_free(c)


@pytest.mark.parametrize("world", [2, 3, 8])
def test_flat_shard_plan_ranks_emulated_in_turn(world):
    """FSDP-style flat shards (tensors cut at shard boundaries): the ranks' launches run one after
    the other on this GPU, the sum of their three numbers stands for the all-reduce."""
    from paper_2603_01501_b200 import sharding
    shapes = synth.decoder_tensor_list(synth.DIMS["small"])
    g, d = synth.gradient_list(shapes, 0.4, config_id=2, device="cuda")
    hp = gb.HParams(**FORCE)
    g_ref, d_ref = [t.cpu() for t in g], [t.cpu() for t in d]
    dec = orc.decide(orc.stats(g_ref, d_ref), to_orc_hp(hp))
    orc.project(g_ref, d_ref, to_orc_hp(hp), dec)
    plan = sharding.flat_shard_plan([t.numel() for t in g], world)
    ctxs = [gb.gac_init(sharding.shard_views(g, p), sharding.shard_views(d, p), hp) for p in plan]
    bufs = [torch.zeros(3, dtype=torch.float64, device="cuda") for _ in plan]
    for c, b in zip(ctxs, bufs):
        gb.gac_stats_partial(c, 2, b)
    total = torch.stack(bufs).sum(0)
    for c in ctxs:
        res = gb.gac_decide(c, total)
        check_sums(res, dec)
        check_decision(res, dec)
        gb.gac_project(c, coef_override=dec.coef)
    torch.cuda.synchronize()
    check_outputs(g, d, g_ref, d_ref)
    for c in ctxs:
        gb.gac_free(c)


def test_call_order_is_enforced():
    g, d = [torch.ones(100, device="cuda")], [torch.ones(100, device="cuda") * 2]
    ctx = gb.gac_init(g, d, gb.HParams())
    with pytest.raises(gb.GacError) as e:
        gb.gac_project(ctx)
    assert e.value.status == gb.GAC_ERR_STATE
    with pytest.raises(gb.GacError) as e:
        gb.gac_stats(ctx, 0)
    assert e.value.status == gb.GAC_ERR_INVALID_ARG
    gb.gac_stats(ctx, 5)
    gb.gac_project(ctx)
    with pytest.raises(gb.GacError) as e:
        gb.gac_project(ctx)
    assert e.value.status == gb.GAC_ERR_STATE
    with pytest.raises(gb.GacError) as e:
        gb.gac_stats(ctx, 5)
    assert e.value.status == gb.GAC_ERR_STATE
    gb.gac_stats(ctx, 6)
    info = gb.gac_get_info(ctx)
    assert info.launches == 3 and info.total_elems == 100
    # three doubles at a 4-byte aligned address would make the device stores fault: refused on the
    # host, nothing is launched
    import ctypes
    lib = gb.load_library()
    odd = torch.zeros(8, dtype=torch.float32, device="cuda")
    assert (odd.data_ptr() + 4) % 8 == 4
    rc = lib.gac_stats_partial(ctx.handle, 7, 0, None, ctypes.c_void_p(odd.data_ptr() + 4))
    assert rc == gb.GAC_ERR_INVALID_ARG and b"8-byte aligned" in lib.gac_last_error(ctx.handle)
    sums = torch.zeros(3, dtype=torch.float64, device="cuda")
    gb.gac_stats_partial(ctx, 7, sums)
    rc = lib.gac_decide(ctx.handle, None, ctypes.c_void_p(odd.data_ptr() + 4), None)
    assert rc == gb.GAC_ERR_INVALID_ARG and b"8-byte aligned" in lib.gac_last_error(ctx.handle)
    gb.gac_decide(ctx, sums)
    gb.gac_project(ctx)
    assert gb.gac_get_info(ctx).launches == 6
    gb.gac_free(ctx)


def test_step_can_be_captured_in_a_cuda_graph_and_replayed():
    """With no host read-back both calls only enqueue kernels, so a step can be captured once and
    replayed (the launch-bound case of small lists).  Replays must give what direct calls give."""
    g_cpu, d_cpu = synth.flat_pair_with_cosine(1 << 20, 0.9, s=1.0, seed=0)
    hp = gb.HParams(**FORCE)
    g, d = [g_cpu.cuda()], [d_cpu.cuda()]
    ctx = gb.gac_init(g, d, hp)
    gb.gac_stats(ctx, 2, fetch=False)            # warm-up outside capture
    gb.gac_project(ctx)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        graph.capture_begin()
        gb.gac_stats(ctx, 3, fetch=False)
        gb.gac_project(ctx)
        graph.capture_end()
    torch.cuda.current_stream().wait_stream(side)
    for rho_seed in (1, 2):
        g_new, d_new = synth.flat_pair_with_cosine(1 << 20, 0.5 + 0.2 * rho_seed, s=2.0, seed=rho_seed)
        g[0].copy_(g_new)
        d[0].copy_(d_new)
        graph.replay()
        torch.cuda.synchronize()
        g_ref, d_ref = [g_new.clone()], [d_new.clone()]
        dec = orc.step(g_ref, d_ref, to_orc_hp(hp))
        # the coefficient is the library's own here (nothing can be overridden inside a replay)
        assert dec.regime == orc.PROJECT
        assert torch.equal(d[0].cpu(), d_ref[0])
        assert max_ulp(g[0].cpu(), g_ref[0]) <= 64      # own coefficient: may differ in its last bit
        assert float((g[0].cpu().double() - g_ref[0].double()).abs().max()) <= 2e-7 * float(g_new.abs().max())
    gb.gac_free(ctx)


@pytest.mark.parametrize("seed", range(12))
def test_random_list_structures(seed):
    """Random lists: tiny and large tensors mixed, some as odd-offset views, random element types,
    thresholds and chunk sizes -- the chunk table must present them all as one flat vector."""
    import random
    rng = random.Random(seed)
    g_dtype = rng.choice([torch.float32, torch.bfloat16])
    n_t = rng.randint(1, 40)
    sizes = [rng.choice([1, 2, 3, 5, 17, 255, 1024, 4097, 16384, 16385, 70001, rng.randint(1, 300000)])
             for _ in range(n_t)]
    rho = rng.choice([0.0, 0.1, 0.5, 0.95, -0.7])
    gen = torch.Generator().manual_seed(seed)
    g_cpu, d_cpu, g_gpu, d_gpu = [], [], [], []
    for n in sizes:
        scale = 10.0 ** rng.uniform(-4, 0)
        d = torch.randn(n, generator=gen) * scale
        g = (rho * d + math.sqrt(1 - rho * rho) * torch.randn(n, generator=gen) * scale).to(g_dtype)
        g_cpu.append(g)
        d_cpu.append(d)
        og, od = (rng.randint(0, 7), rng.randint(0, 7)) if rng.random() < 0.3 else (0, 0)
        gbuf = torch.zeros(n + 8, dtype=g_dtype, device="cuda")
        dbuf = torch.zeros(n + 8, dtype=torch.float32, device="cuda")
        gbuf[og:og + n] = g.cuda()
        dbuf[od:od + n] = d.cuda()
        g_gpu.append(gbuf[og:og + n])
        d_gpu.append(dbuf[od:od + n])
    hp = rng.choice([gb.HParams(), gb.HParams(**FORCE), gb.HParams(c_low=0.3, c_high=0.6),
                     gb.HParams(mode=gb.GAC_MODE_FIXED, alpha_fixed=0.0),
                     gb.HParams(**FORCE, clip_max_norm=0.5)])
    ohp = to_orc_hp(hp)
    g_ref, d_ref = [t.clone() for t in g_cpu], [t.clone() for t in d_cpu]
    dec = orc.step(g_ref, d_ref, ohp)
    ctx = gb.gac_init(g_gpu, d_gpu, hp)
    gb.gac_set_launch(ctx, rng.choice([1024, 4096, 16384, 32768]), rng.choice([0, 1, 3]))
    res = gb.gac_stats(ctx, 2)
    gb.gac_project(ctx, coef_override=dec.coef if dec.regime == orc.PROJECT else None)
    torch.cuda.synchronize()
    gb.gac_free(ctx)
    check_sums(res, dec)
    if abs(abs(dec.cos) - hp.c_low) > 1e-4 and abs(abs(dec.cos) - hp.c_high) > 1e-4:
        check_decision(res, dec)
        check_outputs(g_gpu, d_gpu, g_ref, d_ref)


def test_state_recurrence_is_bitwise_and_survives_a_new_context():
    """With the raw gradient as state, <d,d> of step t+1 is <g,g> of step t bit for bit (same values
    summed in the same order), also when step t+1 runs in a fresh context on the same buffers."""
    shapes = synth.decoder_tensor_list(synth.DIMS["small"])
    for g_dtype in (torch.float32, torch.bfloat16):
        g, d = synth.gradient_list(shapes, 0.3, config_id=2, g_dtype=g_dtype, device="cuda")
        hp = gb.HParams(**FORCE)
        ctx = gb.gac_init(g, d, hp)
        r1 = gb.gac_stats(ctx, 5)
        gb.gac_project(ctx)
        for t in g:
            t.copy_((torch.randn(t.numel(), device="cuda") * 0.01).to(g_dtype))
        r2 = gb.gac_stats(ctx, 6)
        assert r2.dd == r1.gg
        gb.gac_project(ctx)
        gb.gac_free(ctx)
        ctx = gb.gac_init(g, d, hp)            # resume: same buffers, later step
        for t in g:
            t.copy_((torch.randn(t.numel(), device="cuda") * 0.01).to(g_dtype))
        r3 = gb.gac_stats(ctx, 7)
        assert r3.dd == r2.gg and r3.step == 7
        gb.gac_free(ctx)


def test_rebind_to_moved_buffers_keeps_the_step_sequence():
    shapes = synth.decoder_tensor_list(synth.DIMS["mini"])
    g, d = synth.gradient_list(shapes, 0.4, config_id=2, device="cuda")
    hp = gb.HParams(**FORCE)
    ctx = gb.gac_init(g, d, hp)
    gb.gac_stats(ctx, 2)
    with pytest.raises(gb.GacError) as e:
        gb.gac_rebind(ctx, g, d)                       # a step is open
    assert e.value.status == gb.GAC_ERR_STATE
    gb.gac_project(ctx)
    torch.cuda.synchronize()
    g2 = [torch.randn_like(t) * 0.01 for t in g]        # the framework re-allocated its gradients
    d2 = [t.clone() for t in d]                         # ... and the snapshot moved with them
    gb.gac_rebind(ctx, g2, d2)
    g_ref, d_ref = [t.cpu() for t in g2], [t.cpu() for t in d2]
    dec = orc.step(g_ref, d_ref, to_orc_hp(hp))
    res = gb.gac_stats(ctx, 3)
    gb.gac_project(ctx, coef_override=dec.coef if dec.regime == orc.PROJECT else None)
    torch.cuda.synchronize()
    check_sums(res, dec)
    check_decision(res, dec)
    check_outputs(g2, d2, g_ref, d_ref)
    with pytest.raises(gb.GacError):
        gb.gac_rebind(ctx, g2[:-1], d2[:-1])
    gb.gac_free(ctx)


@pytest.mark.parametrize("g_dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
def test_power_of_two_rescaling_on_device(g_dtype):
    """App. A.1: the cosine does not depend on the gradient's scale.  With eps = 0, rescaling g and d
    by powers of two (exact in binary floating point, far from over- and underflow of the sums in
    binary64) must leave cosine, regime and alpha bit-identical on the device, and scale g' exactly."""
    n = 40_001
    g, d = rand_pair(n, 0.6, seed=21, g_dtype=g_dtype, scale=1.0)
    hp = gb.HParams(c_low=0.05, c_high=2.0, eps=0.0)
    base = None
    # the multiplier of d is one binary32 number that scales as 2^(eg - ed): kept within binary32's range
    for eg, ed in [(0, 0), (-90, 0), (60, 0), (0, -100), (0, 90), (-80, -70), (50, 50)]:
        gs = (g.double() * 2.0 ** eg).to(g_dtype)
        ds = (d.double() * 2.0 ** ed).float()
        assert torch.isfinite(gs.float()).all() and (gs.float().abs() >= 2.0 ** -120)[g.float() != 0].all()
        res, dec, gg, dg, gr, dr = step_both([gs], [ds], hp, same_coef=False)
        check_sums(res, dec, rel=1e-13)
        check_decision(res, dec)
        assert (res.cos, res.regime, res.alpha) == (dec.cos, dec.regime, dec.alpha)
        out = (gg[0].cpu().double() * 2.0 ** -eg)
        if base is None:
            base = (res.cos, res.regime, res.alpha, out)
        else:
            assert (res.cos, res.regime, res.alpha) == base[:3]
            # g' = g + k d with k = (alpha - 1) dot/dd scaling as 2^(eg - ed): every term scales by 2^eg
            assert torch.equal(out, base[3]), (eg, ed)
        assert torch.equal(dg[0].cpu(), gs.float())
