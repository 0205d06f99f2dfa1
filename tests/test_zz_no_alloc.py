"""The allocation-free entry point against the ordinary one.

`gac_stats_static` serves callers that may not ask the driver for device
memory (a framework pool owns it all, or the implicit device synchronisation of
an allocation is unacceptable on their path); its work memory is an array built
into the library.  It must give what `gac_init` + `gac_stats` give.  The file
name sorts last on purpose: a run that stops at the first failure has then
already run every other test.
"""
import ctypes

import pytest
import torch

from oracle import gac_oracle as orc
from paper_2603_01501_b200 import binding as gb
from paper_2603_01501_b200 import synth

pytestmark = pytest.mark.gpu

REL = 1e-5          # the tolerance the parity tests use for sums and cosine


def _reference(g, d, hp, step):
    ctx = gb.gac_init(g, d, hp)
    res = gb.gac_stats(ctx, step)
    gb.gac_free(ctx)
    return res


def _close(a, b, scale=0.0):
    return abs(a - b) <= REL * max(abs(b), scale)


@pytest.mark.parametrize("g_dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
def test_static_scratch_matches_context_path_twice_in_a_row(g_dtype):
    hp = gb.HParams(c_low=0.05, c_high=2.0)
    out = torch.zeros(ctypes.sizeof(gb.gac_result), dtype=torch.uint8, device="cuda")
    # two calls in a row on different lists: the second must not see what the first left
    for name, rho, cfg in (("small", 0.8, 2), ("mini", 0.3, 3)):
        shapes = synth.decoder_tensor_list(synth.DIMS[name])
        g, d = synth.gradient_list(shapes, rho, config_id=cfg, g_dtype=g_dtype, device="cuda")
        want = _reference(g, d, hp, step=2)
        out.fill_(0xAB)
        gb.gac_stats_static(g, d, hp, 2, out, staleness=7)
        torch.cuda.synchronize()
        got = gb.result_from_tensor(out)
        scale = 1e-6 * (want.gg * want.dd) ** 0.5
        assert _close(got.gg, want.gg) and _close(got.dd, want.dd) and _close(got.dot, want.dot, scale)
        assert _close(got.cos, want.cos, 1e-6)
        assert got.regime == want.regime == gb.GAC_REGIME_PROJECT
        assert _close(got.alpha, want.alpha) and _close(got.coef, want.coef)
        assert (got.step, got.staleness, got.nonfinite) == (2, 7, 0)
        # the inputs are only read
        g2, d2 = synth.gradient_list(shapes, rho, config_id=cfg, g_dtype=g_dtype, device="cuda")
        assert all(torch.equal(a, b) for a, b in zip(g + d, g2 + d2))


def test_static_scratch_first_step_and_limits():
    hp = gb.HParams()
    out = torch.zeros(ctypes.sizeof(gb.gac_result), dtype=torch.uint8, device="cuda")
    g = [torch.randn(5000, device="cuda")]
    d = [torch.full((5000,), float("nan"), device="cuda")]        # never read on step 1
    gb.gac_stats_static(g, d, hp, 1, out)
    torch.cuda.synchronize()
    r = gb.result_from_tensor(out)
    assert (r.dot, r.dd, r.cos, r.regime) == (0.0, 0.0, 0.0, gb.GAC_REGIME_SAFE)
    assert abs(r.gg - float((g[0].double() ** 2).sum())) <= REL * r.gg
    # a list that needs more chunk slots than the built-in scratch has is refused, nothing runs:
    # 65537 one-element tensors (views of one buffer) need 65537 chunks
    buf_g = torch.zeros(65537, device="cuda")
    buf_d = torch.zeros(65537, device="cuda")
    many_g = [buf_g[i:i + 1] for i in range(65537)]
    many_d = [buf_d[i:i + 1] for i in range(65537)]
    with pytest.raises(gb.GacError) as e:
        gb.gac_stats_static(many_g, many_d, hp, 2, out)
    assert e.value.status == gb.GAC_ERR_INVALID_ARG and "scratch" in str(e.value)
    with pytest.raises(gb.GacError):
        gb.gac_stats_static(g, d, hp, 0, out)


def test_static_scratch_against_the_oracle_and_free_memory_unchanged():
    """The property the entry point exists for: ten calls in a row leave the amount of free device
    memory exactly where it was.  The float32 result is checked against the CPU oracle as well, and
    the fields the reduction does not own come back as zero although the record was pre-filled."""
    hp = gb.HParams(c_low=0.05, c_high=2.0)
    shapes = synth.decoder_tensor_list(synth.DIMS["small"])
    g_cpu, d_cpu = synth.gradient_list(shapes, 0.7, config_id=2)
    dec = orc.decide(orc.stats(g_cpu, d_cpu), orc.HParams(c_low=0.05, c_high=2.0))
    g = [t.cuda() for t in g_cpu]
    d = [t.cuda() for t in d_cpu]
    out = torch.zeros(ctypes.sizeof(gb.gac_result), dtype=torch.uint8, device="cuda")
    gb.gac_stats_static(g, d, hp, 2, out)          # the first call on a device looks up the array's address
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    for step in range(2, 12):
        out.fill_(0xAB)
        gb.gac_stats_static(g, d, hp, step, out)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before
    got = gb.result_from_tensor(out)
    scale = 1e-6 * (dec.gg * dec.dd) ** 0.5
    assert _close(got.gg, dec.gg) and _close(got.dd, dec.dd) and _close(got.dot, dec.dot, scale)
    assert _close(got.cos, dec.cos, 1e-6) and got.regime == dec.regime == orc.PROJECT
    assert _close(got.alpha, dec.alpha) and _close(got.coef, dec.coef)
    assert (got.step, got.applied_steps, got.ref_lost, got.g_set, got.out_set) == (11, 0, 0, 0, 0)


def test_static_scratch_is_refused_on_a_capturing_stream():
    """A captured call would replay its table copy from the library's shared host buffer as it stands
    at replay time: the entry point refuses instead, enqueues nothing, and the capture stays valid."""
    hp = gb.HParams()
    g = [torch.randn(70000, device="cuda")]
    d = [torch.randn(70000, device="cuda")]
    out = torch.zeros(ctypes.sizeof(gb.gac_result), dtype=torch.uint8, device="cuda")
    gb.gac_stats_static(g, d, hp, 2, out)          # set-up happens outside the capture
    torch.cuda.synchronize()
    want = gb.result_from_tensor(out)
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    marker = torch.zeros(4, device="cuda")
    with torch.cuda.stream(side):
        graph.capture_begin()
        with pytest.raises(gb.GacError) as e:
            gb.gac_stats_static(g, d, hp, 3, out, stream=side)
        marker.add_(1.0)                            # the capture goes on: the refusal broke nothing
        graph.capture_end()
    assert e.value.status == gb.GAC_ERR_STATE and "captured" in str(e.value)
    graph.replay()
    torch.cuda.synchronize()
    assert marker.tolist() == [1.0] * 4
    again = gb.result_from_tensor(out)
    assert (again.step, again.gg, again.dot) == (want.step, want.gg, want.dot)     # untouched by the refused call
