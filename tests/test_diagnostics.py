"""Statistics of an alignment trace (Table 3 definitions) and the regime counts
of the paper's threshold grid."""
import numpy as np
import pytest
import torch

from paper_2603_01501_b200 import diagnostics as dg


def test_summary_matches_numpy_definitions():
    rng = np.random.default_rng(0)
    trace = rng.standard_normal(400) * 0.04
    s = dg.summarize_alignment(trace, c_low=0.05, c_high=0.3, skip=50)
    a = np.abs(trace[50:])
    assert s.updates == 350
    assert s.q90_abs == pytest.approx(np.quantile(a, 0.9), rel=1e-12)
    assert s.max_abs == a.max()
    assert s.frac_within_c_low == pytest.approx((a <= 0.05).mean())
    assert sum(s.regimes.values()) == 350


def test_classification_is_inclusive():
    assert dg.classify(0.05, 0.05, 0.3) == "safe"
    assert dg.classify(-0.3, 0.05, 0.3) == "violation"
    assert dg.classify(0.0500001, 0.05, 0.3) == "project"


def test_threshold_grid_counts_are_monotone():
    rng = np.random.default_rng(1)
    trace = np.clip(np.abs(rng.standard_normal(500)) * 0.15, 0, 1)
    grid = dg.threshold_grid(trace)
    assert len(grid) == 9
    by = {(lo, hi): r for lo, hi, r in grid}
    assert by[(0.03, 0.3)]["safe"] <= by[(0.05, 0.3)]["safe"] <= by[(0.07, 0.3)]["safe"]
    assert by[(0.05, 0.2)]["violation"] >= by[(0.05, 0.3)]["violation"] >= by[(0.05, 0.4)]["violation"]


@pytest.mark.gpu
def test_trace_from_the_library_agrees_with_grid_replay():
    """The library's regimes on a staleness run equal the host classification of its own
    c_t trace under each threshold pair (the trace does not depend on the thresholds)."""
    from paper_2603_01501_b200 import binding as gb, synth
    shapes = synth.decoder_tensor_list(synth.DIMS["mini"])
    traces = {}
    for lo, hi in [(0.03, 0.2), (0.05, 0.3), (0.07, 0.4)]:
        proc = synth.StalenessProcess(shapes, 0.25, 4, config_id=4, run_id=77, device="cuda")
        g = [torch.empty(n, device="cuda") for _, n in shapes]
        d = [torch.zeros(n, device="cuda") for _, n in shapes]
        ctx = gb.gac_init(g, d, gb.HParams(c_low=lo, c_high=hi))
        cs, regs = [], []
        for t in range(1, 41):
            for dst, src in zip(g, proc.next()):
                dst.copy_(src)
            r = gb.gac_stats(ctx, t)
            gb.gac_project(ctx)
            cs.append(r.cos)
            regs.append(gb.REGIME_NAMES[r.regime])
        gb.gac_free(ctx)
        traces[(lo, hi)] = cs
        assert regs == [dg.classify(c, lo, hi) for c in cs]
    keys = list(traces)
    assert traces[keys[0]] == traces[keys[1]] == traces[keys[2]]      # bit-identical traces
    assert dg.summarize_alignment(traces[keys[1]], skip=10).updates == 30
