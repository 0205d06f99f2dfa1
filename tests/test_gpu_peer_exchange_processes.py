"""The library's own exchange of the three sums between two PROCESSES.

Two processes share cuda:0 (two CUDA contexts).  Each allocates its slot array and maps the other's
through CUDA IPC (a CUDA tensor sent over a torch.multiprocessing queue arrives as such a mapping), so a
rank's reduction kernel stores its three sums into memory that belongs to another process.  Per step every rank posts, synchronises its device and
meets the other at a host barrier BEFORE anyone launches the kernel that reads the slots: all flags are
set by then, so no kernel of one process ever waits for a kernel of the other (on one GPU the two could
not run at the same time).  Rank 0 checks sums, decisions and outputs against the CPU oracle on the
unsharded list.
"""
import math
import socket

import pytest
import torch

from test_gpu_sharded_processes import C_HIGH, C_LOW, _gradients

pytestmark = pytest.mark.gpu


def _rank_main(rank, world, port, out, coefs, mail):
    import os
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
        g = [torch.empty(n, device="cuda") for _, n in shapes]
        d = [x.cuda() for x in seq[0]]
        plan = sharding.flat_shard_plan([n for _, n in shapes], world)
        my_g, my_d = sharding.shard_views(g, plan[rank]), sharding.shard_views(d, plan[rank])
        ctx = gb.gac_init(my_g, my_d, gb.HParams(c_low=C_LOW, c_high=C_HIGH))
        mine = torch.zeros(gb.gac_exchange_bytes(world), dtype=torch.uint8, device="cuda")
        torch.cuda.synchronize()
        mail[1 - rank].put(mine)                     # the other process maps it (CUDA IPC)
        theirs = mail[rank].get(timeout=120)
        slots = [mine, theirs] if rank == 0 else [theirs, mine]
        gb.gac_exchange_attach(ctx, rank, world, slots, timeout_ms=200)
        dist.barrier()                               # both arrays are zero and mapped before anybody posts
        record = []
        for t, grads in enumerate(seq[1:], start=2):
            for dst, src in zip(g, grads):
                dst.copy_(src)
            gb.gac_stats_exchange(ctx, t)
            torch.cuda.synchronize()
            dist.barrier()                           # every rank's numbers are in every slot array
            res = gb.gac_decide_exchange(ctx)
            gb.gac_project(ctx, coef_override=coefs[t - 2])
            torch.cuda.synchronize()
            dist.barrier()                           # nobody posts the next step before everybody has read this one
            record.append(((res.dot, res.gg, res.dd, res.cos, res.coef, res.regime, res.timed_out, res.step),
                           [x.cpu().numpy().tobytes() for x in my_g], [x.cpu().numpy().tobytes() for x in my_d]))
        gb.gac_free(ctx)
        del slots, theirs                            # unmap the other's array while its owner is still alive
        dist.barrier()
        gathered = [None] * world
        dist.all_gather_object(gathered, (plan[rank], record))
        if rank == 0:
            out.put(("ok", gathered))
    finally:
        dist.destroy_process_group()


def test_two_processes_exchange_their_sums_through_mapped_slot_arrays():
    import torch.multiprocessing as mp
    from oracle import gac_oracle as orc
    from paper_2603_01501_b200 import synth
    from gpu_util import max_ulp

    shapes = synth.decoder_tensor_list(synth.DIMS["small"])
    sigma = synth.per_tensor_scales(2, len(shapes))
    seq = _gradients(shapes, sigma)
    ohp = orc.HParams(c_low=C_LOW, c_high=C_HIGH)
    d_ref = [x.clone() for x in seq[0]]
    want = []
    for grads in seq[1:]:
        g_ref = [x.clone() for x in grads]
        dec = orc.step(g_ref, d_ref, ohp)
        want.append((dec, g_ref, [x.clone() for x in d_ref]))
    coefs = [w[0].coef if w[0].regime == orc.PROJECT else None for w in want]

    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    mail = [ctx.Queue(), ctx.Queue()]
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out, coefs, mail)) for r in range(2)]
    for p in procs:
        p.start()
    try:
        status, payload = out.get(timeout=240)
    finally:
        for p in procs:
            p.join(60)
    assert all(p.exitcode == 0 for p in procs), [p.exitcode for p in procs]
    assert status == "ok"
    gathered = payload
    for step, (dec, g_ref, d_after) in enumerate(want):
        scalars = [rec[step][0] for _, rec in gathered]
        assert scalars[0] == scalars[1]                    # rank-order sum: bit-identical on both ranks
        dot, gg, dd, cos, coef, regime, timed_out, t = scalars[0]
        scale = math.sqrt(dec.gg * dec.dd)
        assert abs(gg - dec.gg) <= 1e-5 * dec.gg and abs(dd - dec.dd) <= 1e-5 * dec.dd
        assert abs(dot - dec.dot) <= 1e-5 * max(abs(dec.dot), 1e-6 * scale)
        assert abs(cos - dec.cos) <= 1e-5 * max(abs(dec.cos), 1e-6)
        assert (regime, timed_out, t) == (dec.regime, 0, step + 2)
        for pieces, rec in gathered:
            _, g_out, d_out = rec[step]
            for (i, lo, hi), a, b in zip(pieces, g_out, d_out):
                a = torch.frombuffer(bytearray(a), dtype=torch.float32)
                assert max_ulp(a, g_ref[i][lo:hi]) <= 4, f"step {step + 2} tensor {i} [{lo}:{hi}]"
                assert b == d_after[i][lo:hi].contiguous().numpy().tobytes()
