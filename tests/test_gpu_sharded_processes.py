"""The library's sharded call sequence (App. A.1, "Efficient computation under data parallelism")
across a real process boundary: two processes, each with its own CUDA context on cuda:0 and its own
shard of the flat gradient, joined by a `gloo` group (which accepts CUDA tensors and reduces them
through host memory).  Each runs `sharding.sharded_step` -- local sums, ONE all-reduce of three
doubles, decision, in-place update -- for three steps; rank 0 then checks every rank's sums,
decision and outputs against the CPU oracle run on the unsharded list.  No kernel waits for
another process's kernel: the collective runs on the host between the launches.
"""
import math
import os
import socket

import pytest
import torch

pytestmark = pytest.mark.gpu

RHOS = (0.3, 0.01, 0.9)          # against thresholds (0.05, 0.6): projection, safe, violation
C_LOW, C_HIGH = 0.05, 0.6


def _gradients(shapes, sigma):
    """Step-by-step gradient lists on the CPU (float32), the same in every process."""
    gen = torch.Generator().manual_seed(77)
    prev = [torch.randn(n, generator=gen) * s for (_, n), s in zip(shapes, sigma)]
    out = [prev]
    for rho in RHOS:
        noise = [torch.randn(n, generator=gen) * s for (_, n), s in zip(shapes, sigma)]
        prev = [rho * a + math.sqrt(1 - rho * rho) * b for a, b in zip(prev, noise)]
        out.append(prev)
    return out


def _rank_main(rank, world, port, out, coefs):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    import torch.distributed as dist
    from paper_2603_01501_b200 import binding as gb
    from paper_2603_01501_b200 import sharding, synth
    torch.cuda.set_device(0)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        shapes = synth.decoder_tensor_list(synth.DIMS["small"])
        sigma = synth.per_tensor_scales(2, len(shapes))
        seq = _gradients(shapes, sigma)
        hp = gb.HParams(c_low=C_LOW, c_high=C_HIGH)
        # the whole list lives on the device as a framework would hold it; this rank owns one shard
        g = [torch.empty(n, device="cuda") for _, n in shapes]
        d = [x.cuda() for x in seq[0]]                           # stored direction: the gradient of step 1
        plan = sharding.flat_shard_plan([n for _, n in shapes], world)
        my_g, my_d = sharding.shard_views(g, plan[rank]), sharding.shard_views(d, plan[rank])
        ctx = gb.gac_init(my_g, my_d, hp)
        sums = torch.zeros(3, dtype=torch.float64, device="cuda")
        record = []
        for t, grads in enumerate(seq[1:], start=2):
            for dst, src in zip(g, grads):
                dst.copy_(src)
            res = sharding.sharded_step(gb, ctx, t, sums, fetch=True, coef_override=coefs[t - 2])
            torch.cuda.synchronize()
            record.append(((res.dot, res.gg, res.dd, res.cos, res.alpha, res.coef64, res.coef, res.regime,
                            res.nonfinite, res.step),
                           [x.cpu().numpy().tobytes() for x in my_g], [x.cpu().numpy().tobytes() for x in my_d]))
        gb.gac_free(ctx)
        gathered = [None] * world
        dist.all_gather_object(gathered, (plan[rank], record))
        if rank == 0:
            out.put(gathered)
    finally:
        dist.destroy_process_group()


def test_two_processes_run_the_sharded_step_on_one_gpu():
    import torch.multiprocessing as mp
    from oracle import gac_oracle as orc
    from paper_2603_01501_b200 import synth
    from gpu_util import max_ulp

    shapes = synth.decoder_tensor_list(synth.DIMS["small"])
    sigma = synth.per_tensor_scales(2, len(shapes))
    seq = _gradients(shapes, sigma)
    ohp = orc.HParams(c_low=C_LOW, c_high=C_HIGH)
    # the oracle on the unsharded list, state carried from step to step
    d_ref = [x.clone() for x in seq[0]]
    want = []
    for grads in seq[1:]:
        g_ref = [x.clone() for x in grads]
        dec = orc.step(g_ref, d_ref, ohp)
        want.append((dec, g_ref, [x.clone() for x in d_ref]))
    assert [w[0].regime for w in want] == [orc.PROJECT, orc.SAFE, orc.VIOLATION]
    coefs = [w[0].coef if w[0].regime == orc.PROJECT else None for w in want]

    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out, coefs)) for r in range(2)]
    for p in procs:
        p.start()
    gathered = out.get(timeout=240)
    for p in procs:
        p.join(60)
    assert all(p.exitcode == 0 for p in procs), [p.exitcode for p in procs]

    for step, (dec, g_ref, d_after) in enumerate(want):
        scalars = [rec[step][0] for _, rec in gathered]
        assert scalars[0] == scalars[1]                    # every rank holds the same record, bit for bit
        dot, gg, dd, cos, alpha, coef64, coef, regime, nonfinite, t = scalars[0]
        scale = math.sqrt(dec.gg * dec.dd)
        assert abs(gg - dec.gg) <= 1e-5 * dec.gg and abs(dd - dec.dd) <= 1e-5 * dec.dd
        assert abs(dot - dec.dot) <= 1e-5 * max(abs(dec.dot), 1e-6 * scale)
        assert abs(cos - dec.cos) <= 1e-5 * max(abs(dec.cos), 1e-6)
        assert (regime, nonfinite, t) == (dec.regime, 0, step + 2)
        assert abs(alpha - dec.alpha) <= 1e-5 * abs(dec.alpha) and abs(coef - dec.coef) <= 1e-5 * abs(dec.coef)
        covered = 0
        for pieces, rec in gathered:
            _, g_out, d_out = rec[step]
            for (i, lo, hi), a, b in zip(pieces, g_out, d_out):
                a = torch.frombuffer(bytearray(a), dtype=torch.float32)
                assert max_ulp(a, g_ref[i][lo:hi]) <= 4, f"step {step + 2} tensor {i} [{lo}:{hi}]"
                assert b == d_after[i][lo:hi].contiguous().numpy().tobytes()      # bit for bit
                covered += hi - lo
        assert covered == sum(n for _, n in shapes)
