"""The controller on real autograd gradients of a small network: the library's
decisions and outputs against the CPU oracle fed with the same gradients, over
steps that reuse a stale batch (aligned consecutive gradients) and fresh ones."""
import pytest
import torch

from oracle import gac_oracle as orc
from paper_2603_01501_b200 import binding as gb
from paper_2603_01501_b200.controller import GradientAlignmentController

from gpu_util import check_decision, check_sums, max_ulp, to_orc_hp

pytestmark = pytest.mark.gpu


def test_controller_follows_algorithm_1_on_autograd_gradients():
    torch.manual_seed(0)
    net = torch.nn.Sequential(torch.nn.Linear(37, 129), torch.nn.Tanh(), torch.nn.Linear(129, 5)).cuda()
    hp = gb.HParams(c_low=0.05, c_high=0.9)
    ctl = GradientAlignmentController(net.parameters(), hp)
    opt = torch.optim.SGD(net.parameters(), lr=1e-3)
    ohp = to_orc_hp(hp)
    d_ref = None
    batches = [torch.randn(64, 37, device="cuda") for _ in range(3)]
    targets = [torch.randn(64, 5, device="cuda") for _ in range(3)]
    order = [0, 0, 1, 1, 1, 2, 0]            # repeated batches give aligned consecutive gradients
    seen = set()
    for t, b in enumerate(order, start=1):
        opt.zero_grad(set_to_none=(t == 4))   # once, force the framework to re-allocate .grad
        loss = torch.nn.functional.mse_loss(net(batches[b]), targets[b])
        loss.backward()
        g_ref = [p.grad.detach().view(-1).cpu().clone() for p in net.parameters()]
        if d_ref is None:
            d_ref = [torch.zeros_like(x) for x in g_ref]
        dec = orc.step(g_ref, d_ref, ohp, first_step=(t == 1))
        take = ctl.step(staleness=1)
        res = ctl.last
        check_sums(res, dec)
        check_decision(res, dec)
        assert take == (dec.regime != orc.VIOLATION)
        for p, want, snap, dwant in zip(net.parameters(), g_ref, ctl.snapshot, d_ref):
            assert torch.equal(snap.cpu(), dwant)
            # the library used its own coefficient here: compare with a bound that covers its last bit
            tol = 2e-7 * float(want.abs().max()) + 1e-12
            assert float((p.grad.view(-1).cpu() - want).abs().max()) <= tol
        seen.add(dec.regime)
        if take:
            opt.step()
    assert orc.PROJECT in seen and orc.SAFE in seen
    state = ctl.state_dict()
    assert state["t"] == len(order)
    ctl.close()


def test_controller_in_exchange_mode_matches_the_raw_rule():
    """Same loop with exchange=True: the snapshot is refreshed by swapping tensors, `.grad`
    follows the outgoing gradient, and the values are those of the paper's rule."""
    torch.manual_seed(0)
    net = torch.nn.Sequential(torch.nn.Linear(37, 129), torch.nn.Tanh(), torch.nn.Linear(129, 5)).cuda()
    hp = gb.HParams(c_low=0.05, c_high=0.9)
    ctl = GradientAlignmentController(net.parameters(), hp, exchange=True)
    opt = torch.optim.SGD(net.parameters(), lr=1e-3)
    ohp = to_orc_hp(hp)                      # the oracle runs the RAW rule
    d_ref = None
    batches = [torch.randn(64, 37, device="cuda") for _ in range(3)]
    targets = [torch.randn(64, 5, device="cuda") for _ in range(3)]
    seen = set()
    for t, b in enumerate([0, 0, 1, 1, 1, 2, 0], start=1):
        if t == 1:
            opt.zero_grad(set_to_none=True)
        else:
            ctl.zero_grad()
        loss = torch.nn.functional.mse_loss(net(batches[b]), targets[b])
        loss.backward()
        raw = [p.grad.detach().view(-1).cpu().clone() for p in net.parameters()]
        g_ref = [x.clone() for x in raw]
        if d_ref is None:
            d_ref = [torch.zeros_like(x) for x in g_ref]
        dec = orc.step(g_ref, d_ref, ohp, first_step=(t == 1))
        take = ctl.step()
        res = ctl.last
        check_sums(res, dec)
        check_decision(res, dec)
        assert take == (dec.regime != orc.VIOLATION)
        for p, want, snap, r in zip(net.parameters(), g_ref, ctl.snapshot, raw):
            assert torch.equal(snap.cpu(), r)                       # stored direction = raw gradient
            tol = 2e-7 * float(want.abs().max()) + 1e-12
            assert float((p.grad.view(-1).cpu() - want).abs().max()) <= tol
            assert (p.grad.data_ptr() == snap.data_ptr()) == (dec.regime != orc.PROJECT)
        seen.add(dec.regime)
        if take:
            opt.step()
    assert orc.PROJECT in seen and orc.SAFE in seen
    # accumulating into a tensor the controller did not hand out is refused
    opt.zero_grad(set_to_none=True)
    torch.nn.functional.mse_loss(net(batches[0]), targets[0]).backward()
    with pytest.raises(RuntimeError):
        ctl.step()
    ctl.close()


@pytest.mark.parametrize("exchange", [False, True], ids=["copy", "exchange"])
def test_controller_resumes_from_its_state_dict(exchange):
    """Save after step 3, build a new controller, load, go on: steps 4 and 5 must equal those of the
    uninterrupted run bit for bit (sums, decision, outgoing gradient, stored direction)."""
    gen = torch.Generator().manual_seed(5)
    sizes = [1000, 33, 70001, 4096]
    seq, prev = [], None
    for rho in (None, 0.2, 0.7, 0.15, 0.3):       # safe first step, then projections and a violation
        noise = [torch.randn(n, generator=gen) for n in sizes]
        g = noise if prev is None else [rho * a + (1 - rho * rho) ** 0.5 * b for a, b in zip(prev, noise)]
        seq.append(g)
        prev = g
    hp = gb.HParams(c_low=0.05, c_high=0.6)

    def feed(ctl, params, g, first):
        if exchange and not first:
            ctl.zero_grad()
            for p, x in zip(params, g):
                p.grad.copy_(x.view_as(p))
        else:
            for p, x in zip(params, g):
                p.grad = x.clone().cuda().view_as(p)

    def snap(ctl, params, take):
        r = ctl.last
        return (take, r.dot, r.gg, r.dd, r.cos, r.coef, r.regime, r.step,
                [p.grad.detach().view(-1).cpu().clone() for p in params],
                [s.cpu().clone() for s in ctl.snapshot])

    def same(a, b):
        assert a[:8] == b[:8]
        for x, y in zip(a[8] + a[9], b[8] + b[9]):
            assert torch.equal(x.view(torch.int32), y.view(torch.int32))

    params = [torch.nn.Parameter(torch.zeros(n, device="cuda")) for n in sizes]
    ctl = GradientAlignmentController(params, hp, exchange=exchange)
    whole = []
    for t, g in enumerate(seq):
        feed(ctl, params, g, t == 0)
        whole.append(snap(ctl, params, ctl.step()))
    ctl.close()
    assert {w[6] for w in whole} == {orc.SAFE, orc.PROJECT, orc.VIOLATION}

    params = [torch.nn.Parameter(torch.zeros(n, device="cuda")) for n in sizes]
    ctl = GradientAlignmentController(params, hp, exchange=exchange)
    for t, g in enumerate(seq[:3]):
        feed(ctl, params, g, t == 0)
        same(snap(ctl, params, ctl.step()), whole[t])
    state = ctl.state_dict()
    ctl.close()
    assert state["t"] == 3

    params = [torch.nn.Parameter(torch.zeros(n, device="cuda")) for n in sizes]
    ctl = GradientAlignmentController(params, hp, exchange=exchange)
    feed(ctl, params, seq[3], True)               # the gradient of step 4 exists before the state is loaded
    ctl.load_state_dict(state)
    same(snap(ctl, params, ctl.step()), whole[3])
    feed(ctl, params, seq[4], False)
    same(snap(ctl, params, ctl.step()), whole[4])
    ctl.close()
