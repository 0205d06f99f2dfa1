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
