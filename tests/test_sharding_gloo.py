"""The sharded form of the step (App. A.1) on CPU: the shard plan covers the
flat vector exactly once, and two gloo ranks that reduce their shards and
all-reduce three numbers reach the decision of the unsharded step and, put
together, its outputs.  The local arithmetic here is the CPU oracle's; the
point is the host logic around the collective."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import gac_oracle as orc
from paper_2603_01501_b200 import sharding, synth


def test_plan_covers_every_element_once():
    for numels in ([10], [1, 2, 3, 4, 5, 1000, 7], [4096, 1, 4096, 33], [5] * 40):
        for world in (1, 2, 3, 8):
            plan = sharding.flat_shard_plan(numels, world)
            assert len(plan) == world
            seen = [[0] * n for n in numels]
            for pieces in plan:
                for i, lo, hi in pieces:
                    assert 0 <= lo < hi <= numels[i]
                    for e in range(lo, hi):
                        seen[i][e] += 1
            assert all(all(c == 1 for c in s) for s in seen)
            sizes = [sum(hi - lo for _, lo, hi in p) for p in plan]
            nonempty = [z for z in sizes if z]
            assert all(z == nonempty[0] for z in nonempty[:-1]) and nonempty[-1] <= nonempty[0]
            assert sizes == nonempty + [0] * (world - len(nonempty))
            # list order is preserved inside and across shards
            flat = [(i, lo) for p in plan for i, lo, _ in p]
            assert flat == sorted(flat)


def test_plan_balances_a_decoder_list():
    numels = [n for _, n in synth.decoder_tensor_list(synth.DIMS["7b"])]
    plan = sharding.flat_shard_plan(numels, 8)
    sizes = [sum(hi - lo for _, lo, hi in p) for p in plan]
    assert sum(sizes) == sum(numels)
    assert max(sizes) - min(sizes) <= 8 * 8


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _rank_main(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        shapes = synth.decoder_tensor_list(synth.DIMS["mini"])
        g, d = synth.gradient_list(shapes, 0.3, config_id=2)
        hp = orc.HParams(c_low=0.05, c_high=0.9)
        plan = sharding.flat_shard_plan([t.numel() for t in g], world)
        # contiguous copies of this rank's pieces (the oracle wants contiguous memory)
        my_g = [t.clone() for t in sharding.shard_views(g, plan[rank])]
        my_d = [t.clone() for t in sharding.shard_views(d, plan[rank])]
        local = torch.tensor(orc.stats(my_g, my_d), dtype=torch.float64)
        dist.all_reduce(local, op=dist.ReduceOp.SUM)           # the ONE collective of the step
        dec = orc.decide(tuple(local.tolist()), hp)
        orc.project(my_g, my_d, hp, dec)
        gathered = [None] * world
        dist.all_gather_object(gathered, (dec.cos, dec.regime, dec.coef, [t.numpy().tobytes() for t in my_g],
                                          [t.numpy().tobytes() for t in my_d]))
        if rank == 0:
            whole_g, whole_d = [t.clone() for t in g], [t.clone() for t in d]
            ref = orc.step(whole_g, whole_d, hp)
            assert ref.regime == orc.PROJECT
            for cos, regime, coef, _, _ in gathered:           # same decision on every rank
                assert regime == ref.regime
                assert abs(cos - ref.cos) <= 1e-14 * abs(ref.cos)
                assert coef == gathered[0][2]
            assert abs(gathered[0][2] - ref.coef) <= 1.2e-7 * abs(ref.coef)
            # outputs: recompute the unsharded step with the shared coefficient, compare bitwise
            whole_g, whole_d = [t.clone() for t in g], [t.clone() for t in d]
            orc.project(whole_g, whole_d, hp, ref, coef=gathered[0][2])
            for r in range(world):
                for (i, lo, hi), gb_, db_ in zip(plan[r], gathered[r][3], gathered[r][4]):
                    assert whole_g[i][lo:hi].numpy().tobytes() == gb_
                    assert whole_d[i][lo:hi].numpy().tobytes() == db_
            out.put("ok")
    finally:
        dist.destroy_process_group()


@pytest.mark.timeout(300)
def test_two_gloo_ranks_agree_with_the_unsharded_step():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(240)
    assert all(p.exitcode == 0 for p in procs), [p.exitcode for p in procs]
    assert out.get(timeout=5) == "ok"
