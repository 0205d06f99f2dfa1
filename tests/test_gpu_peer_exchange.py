"""The peer exchange of the three sums (App. A.1's single all-reduce done by the kernels, App. A.2's
"additional synchronization point") on ONE GPU.

Every rank is a context over its shard; the slot arrays are ordinary device memory.  All launches go
onto one stream, posts first, so every wait finds its flags already set: no kernel ever waits for a
kernel that has not run yet.  The timeout case waits for a flag that nothing sets, with a short limit,
and checks the status the host gets and that nothing was written.
"""
import ctypes
import time

import pytest
import torch

from oracle import gac_oracle as orc
from paper_2603_01501_b200 import binding as gb
from paper_2603_01501_b200 import sharding, synth

from gpu_util import check_decision, check_outputs, check_sums, to_orc_hp

pytestmark = pytest.mark.gpu
FORCE = dict(c_low=0.05, c_high=2.0)


def make_ranks(g, d, hp, world, timeout_ms=200):
    plan = sharding.flat_shard_plan([t.numel() for t in g], world)
    ctxs = [gb.gac_init(sharding.shard_views(g, p), sharding.shard_views(d, p), hp) for p in plan]
    slots = [torch.zeros(gb.gac_exchange_bytes(world), dtype=torch.uint8, device="cuda") for _ in range(world)]
    for r, c in enumerate(ctxs):
        gb.gac_exchange_attach(c, r, world, slots, timeout_ms)
    return ctxs, slots


@pytest.mark.parametrize("world", [1, 2, 3, 8])
def test_emulated_ranks_hold_bit_identical_sums_and_match_the_oracle(world):
    shapes = synth.decoder_tensor_list(synth.DIMS["small"])
    g, d = synth.gradient_list(shapes, 0.4, config_id=2, device="cuda")
    hp = gb.HParams(**FORCE)
    g_ref, d_ref = [t.cpu() for t in g], [t.cpu() for t in d]
    dec = orc.decide(orc.stats(g_ref, d_ref), to_orc_hp(hp))
    orc.project(g_ref, d_ref, to_orc_hp(hp), dec)
    ctxs, slots = make_ranks(g, d, hp, world)
    # what the exchange must reproduce: the ranks' partial sums added in rank order
    twins = [gb.gac_init(c._keep[0], c._keep[1], hp) for c in ctxs]
    parts = [torch.zeros(3, dtype=torch.float64, device="cuda") for _ in twins]
    for c, b in zip(twins, parts):
        gb.gac_stats_partial(c, 2, b)
    torch.cuda.synchronize()
    want = [0.0, 0.0, 0.0]
    for b in parts:
        for j, x in enumerate(b.tolist()):
            want[j] += x
    for c in ctxs:                                    # every rank posts ...
        gb.gac_stats_exchange(c, 2, staleness=3)
    results = [gb.gac_decide_exchange(c) for c in ctxs]   # ... then every rank reads: nothing left to wait for
    for r in results:
        assert (r.dot, r.gg, r.dd) == tuple(want)
        assert (r.cos, r.coef, r.regime, r.step, r.staleness, r.timed_out) == \
            (results[0].cos, results[0].coef, results[0].regime, 2, 3, 0)
        check_sums(r, dec)
        check_decision(r, dec)
    for c in ctxs:
        gb.gac_project(c, coef_override=dec.coef)
    torch.cuda.synchronize()
    check_outputs(g, d, g_ref, d_ref)
    for c in ctxs + twins:
        gb.gac_free(c)


def test_steps_alternate_between_the_two_slot_sets_and_first_step_posts_a_zero_reference():
    world = 2
    n = 300000
    gen = torch.Generator(device="cuda").manual_seed(3)
    g = [torch.randn(n, generator=gen, device="cuda")]
    d = [torch.full((n,), float("nan"), device="cuda")]         # never read on step 1
    hp = gb.HParams(c_low=0.05, c_high=0.9)
    ctxs, slots = make_ranks(g, d, hp, world)
    d_ref = [torch.zeros(n)]
    for t in range(1, 6):
        if t > 1:
            g[0].copy_(0.5 * d[0] + 0.5 * torch.randn(n, generator=gen, device="cuda"))
        g_ref = [g[0].cpu()]
        dec = orc.step(g_ref, d_ref, to_orc_hp(hp), first_step=(t == 1))
        for c in ctxs:
            gb.gac_stats_exchange(c, t)
        res = [gb.gac_decide_exchange(c) for c in ctxs]
        assert (res[0].dot, res[0].gg, res[0].dd, res[0].coef) == (res[1].dot, res[1].gg, res[1].dd, res[1].coef)
        check_sums(res[0], dec)
        check_decision(res[0], dec)
        for c in ctxs:
            gb.gac_project(c, coef_override=dec.coef if dec.regime == orc.PROJECT else None)
        torch.cuda.synchronize()
        check_outputs(g, d, g_ref, d_ref)
        # the step number sits in the slot set of its parity, in every rank's array
        for s in slots:
            flags = s.view(torch.int64).view(2, world, 4)[:, :, 3].cpu()
            assert flags[t & 1].tolist() == [t] * world
            assert flags[(t & 1) ^ 1].tolist() == [t - 1] * world
    for c in ctxs:
        gb.gac_free(c)


def test_a_rank_that_never_posts_ends_the_wait_with_a_timeout_and_nothing_is_written():
    world = 2
    shapes = synth.decoder_tensor_list(synth.DIMS["mini"])
    g, d = synth.gradient_list(shapes, 0.5, config_id=2, device="cuda")
    g0, d0 = [t.clone() for t in g], [t.clone() for t in d]
    hp = gb.HParams(**FORCE)
    ctxs, slots = make_ranks(g, d, hp, world, timeout_ms=50)
    gb.gac_stats_exchange(ctxs[0], 2)                 # rank 1 never does
    t0 = time.perf_counter()
    with pytest.raises(gb.GacError) as e:
        gb.gac_decide_exchange(ctxs[0])
    waited = time.perf_counter() - t0
    assert e.value.status == gb.GAC_ERR_TIMEOUT and "did not arrive" in str(e.value)
    assert 0.04 < waited < 5.0
    with pytest.raises(gb.GacError) as e:              # no decision: the update is refused on the host
        gb.gac_project(ctxs[0])
    assert e.value.status == gb.GAC_ERR_STATE
    # the asynchronous form cannot tell the host: the record is marked and the update writes nothing
    gb.gac_decide_exchange(ctxs[0], fetch=False)
    with pytest.raises(gb.GacError) as e:
        gb.gac_project(ctxs[0], fetch=True)
    assert e.value.status == gb.GAC_ERR_TIMEOUT
    torch.cuda.synchronize()
    for a, b in zip(g + d, g0 + d0):
        assert torch.equal(a, b), "a timed-out step wrote to g or d"
    # the late rank arrives: the step is taken again from the posted numbers
    gb.gac_stats_exchange(ctxs[0], 3)
    gb.gac_stats_exchange(ctxs[1], 3)
    r0, r1 = gb.gac_decide_exchange(ctxs[0]), gb.gac_decide_exchange(ctxs[1])
    assert r0.timed_out == 0 and (r0.dot, r0.gg, r0.dd) == (r1.dot, r1.gg, r1.dd)
    g_ref, d_ref = [t.cpu() for t in g0], [t.cpu() for t in d0]
    dec = orc.decide(orc.stats(g_ref, d_ref), to_orc_hp(hp))
    check_sums(r0, dec)
    for c in ctxs:
        gb.gac_project(c, coef_override=dec.coef)
    torch.cuda.synchronize()
    orc.project(g_ref, d_ref, to_orc_hp(hp), dec)
    check_outputs(g, d, g_ref, d_ref)
    for c in ctxs:
        gb.gac_free(c)


def test_retry_after_a_timeout_succeeds_once_the_peer_has_posted():
    world = 2
    n = 100000
    g = [torch.randn(n, device="cuda")]
    d = [torch.randn(n, device="cuda")]
    ctxs, slots = make_ranks(g, d, gb.HParams(**FORCE), world, timeout_ms=20)
    gb.gac_stats_exchange(ctxs[1], 2)
    with pytest.raises(gb.GacError) as e:
        gb.gac_decide_exchange(ctxs[1])
    assert e.value.status == gb.GAC_ERR_TIMEOUT
    gb.gac_stats_exchange(ctxs[0], 2)                 # the straggler
    r1 = gb.gac_decide_exchange(ctxs[1])              # same step, repeated
    r0 = gb.gac_decide_exchange(ctxs[0])
    assert r1.timed_out == 0 and (r1.dot, r1.gg, r1.dd, r1.coef) == (r0.dot, r0.gg, r0.dd, r0.coef)
    gg = float((g[0].double() ** 2).sum())
    assert abs(r0.gg - gg) <= 1e-9 * gg
    for c in ctxs:
        gb.gac_project(c)
        gb.gac_free(c)


def test_call_rules_of_the_peer_exchange():
    g, d = [torch.ones(64, device="cuda")], [torch.ones(64, device="cuda") * 2]
    ctx = gb.gac_init(g, d, gb.HParams())
    with pytest.raises(gb.GacError) as e:
        gb.gac_stats_exchange(ctx, 2)
    assert e.value.status == gb.GAC_ERR_STATE          # not attached
    buf = torch.zeros(gb.gac_exchange_bytes(2) + 32, dtype=torch.uint8, device="cuda")
    lib = gb.load_library()
    arr = (ctypes.c_void_p * 2)(buf.data_ptr(), buf.data_ptr() + 8)
    assert lib.gac_exchange_attach(ctx.handle, 0, 2, arr, 0) == gb.GAC_ERR_INVALID_ARG     # misaligned
    assert lib.gac_exchange_attach(ctx.handle, 2, 2, arr, 0) == gb.GAC_ERR_INVALID_ARG     # rank >= world
    assert lib.gac_exchange_attach(ctx.handle, 0, 0, arr, 0) == gb.GAC_ERR_INVALID_ARG
    assert gb.gac_exchange_bytes(8) == 8 * 2 * 32
    one = torch.zeros(gb.gac_exchange_bytes(1), dtype=torch.uint8, device="cuda")
    gb.gac_exchange_attach(ctx, 0, 1, [one])
    with pytest.raises(gb.GacError) as e:
        gb.gac_decide_exchange(ctx)
    assert e.value.status == gb.GAC_ERR_STATE          # nothing posted
    gb.gac_stats_partial(ctx, 2, torch.zeros(3, dtype=torch.float64, device="cuda"))
    with pytest.raises(gb.GacError) as e:
        gb.gac_decide_exchange(ctx)                    # a partial reduction that was not posted
    assert e.value.status == gb.GAC_ERR_STATE
    gb.gac_stats_exchange(ctx, 2)
    with pytest.raises(gb.GacError) as e:
        gb.gac_decide(ctx, torch.zeros(3, dtype=torch.float64, device="cuda"))
    assert e.value.status == gb.GAC_ERR_STATE
    r = gb.gac_decide_exchange(ctx)
    assert r.gg == 64.0 and r.dd == 256.0 and r.dot == 128.0
    gb.gac_project(ctx)
    gb.gac_free(ctx)
