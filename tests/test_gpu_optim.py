"""The torch.optim front end: the same updates as the binding it forwards to, learning-
rate schedulers, checkpoints, and the closure of the true Nesterov variant evaluated by
autograd at the look-ahead point, against the oracle."""
import numpy as np
import pytest
import torch

from harness import assert_close, oracle_config, to_f64
from oracle import novak_oracle as O
from paper_2601_07876_b200 import binding as B
from paper_2601_07876_b200.optim import Novak

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
HYPER = dict(lr=1e-3, betas=(0.9, 0.999), eps=1e-8, weight_decay=1e-2,
             nesterov="approximation", lookahead_k=5, lookahead_alpha=0.5)


def _model(seed=0):
    torch.manual_seed(seed)
    return torch.nn.Sequential(torch.nn.Linear(37, 64), torch.nn.Tanh(),
                               torch.nn.Linear(64, 5)).to(DEV)


def test_same_updates_as_the_binding_with_a_scheduler_and_two_groups():
    a, b = _model(), _model()
    groups = [{"params": [a[0].weight, a[0].bias]},
              {"params": [a[2].weight, a[2].bias], "lr": 5e-4, "weight_decay": 0.0}]
    opt = Novak(groups, **HYPER, clip_threshold=0.5, centralize=True)
    sched = torch.optim.lr_scheduler.StepLR(opt, step_size=2, gamma=0.5)
    ref = [B.NovakOptimizer([b[0].weight, b[0].bias], **HYPER, clip_threshold=0.5, centralize=True),
           B.NovakOptimizer([b[2].weight, b[2].bias], **dict(HYPER, lr=5e-4, weight_decay=0.0),
                            clip_threshold=0.5, centralize=True)]
    x = torch.randn(16, 37, device=DEV)
    for t in range(7):
        for m in (a, b):
            m.zero_grad(set_to_none=True)
            m(x).square().mean().backward()
        opt.step()
        sched.step()
        for r, ps in zip(ref, ([b[0].weight, b[0].bias], [b[2].weight, b[2].bias])):
            r.step([p.grad for p in ps])
        # what StepLR did to the groups, done by hand on the reference handles
        if (t + 1) % 2 == 0:
            for r, base in zip(ref, (1e-3, 5e-4)):
                r.handle.set_option(B.NOVAK_OPT_LR, base * 0.5 ** ((t + 1) // 2))
    for pa, pb in zip(a.parameters(), b.parameters()):
        assert torch.equal(pa, pb)
    assert opt._engines[0].info()["t"] == 7 and opt._engines[1].info()["launches"] > 7


def test_checkpoint_round_trip():
    a = _model()
    opt = Novak(a.parameters(), **HYPER)
    x = torch.randn(8, 37, device=DEV)

    def run(o, m, n):
        for _ in range(n):
            m.zero_grad(set_to_none=True)
            m(x).square().mean().backward()
            o.step()
    run(opt, a, 3)
    sd = opt.state_dict()
    snap = [p.detach().clone() for p in a.parameters()]
    run(opt, a, 4)
    want = [p.detach().clone() for p in a.parameters()]
    b = _model()
    with torch.no_grad():
        for p, s in zip(b.parameters(), snap):
            p.copy_(s)
    opt2 = Novak(b.parameters(), **HYPER)
    opt2.load_state_dict(sd)
    run(opt2, b, 4)
    for p, w in zip(b.parameters(), want):
        assert torch.equal(p, w)


def test_every_parameter_needs_a_gradient_and_cpu_tensors_are_refused():
    a = _model()
    opt = Novak(a.parameters(), **HYPER)
    a[0].weight.grad = torch.zeros_like(a[0].weight)
    with pytest.raises(RuntimeError):
        opt.step()
    cpu = torch.nn.Linear(3, 3)
    bad = Novak(cpu.parameters(), **HYPER)
    for p in cpu.parameters():
        p.grad = torch.zeros_like(p)
    with pytest.raises(ValueError):
        bad.step()


def test_closure_is_evaluated_at_the_look_ahead_point():
    """L(theta) = sum(a theta^2) / 2 + b . theta by autograd: its gradient at theta~ is
    a theta~ + b.  Four true steps, then the approximation; the oracle evaluates the same
    closure in float64 at ITS look-ahead point."""
    n = 5000
    rng = np.random.default_rng(3)
    a64, b64 = rng.uniform(0.5, 2.0, n), rng.normal(0, 1e-2, n)
    a = torch.from_numpy(a64.astype(np.float32)).to(DEV)
    b = torch.from_numpy(b64.astype(np.float32)).to(DEV)
    theta = torch.nn.Parameter(torch.from_numpy(rng.normal(0, 0.05, n).astype(np.float32)).to(DEV))
    hyper = dict(HYPER, nesterov="true", nesterov_beta=0.8, true_nesterov_steps=4)
    opt = Novak([theta], **hyper)
    oracle = O.Oracle(oracle_config(hyper), [to_f64(theta)])
    a_f, b_f = to_f64(a), to_f64(b)                       # the rounded coefficients, widened
    seen = []

    def closure():
        opt.zero_grad(set_to_none=True)
        seen.append(theta.detach().clone())
        loss = (0.5 * a * theta * theta + b * theta).sum()
        loss.backward()
        return loss

    for t in range(1, 8):
        point = oracle.extrapolated()[0] if oracle.wants_extrapolation() else oracle.theta[0]
        loss = opt.step(closure)
        assert_close(seen[-1], point, f"t={t}: where the closure ran")
        oracle.step([a_f * point + b_f])
        assert torch.isfinite(loss)
    torch.cuda.synchronize()
    assert_close(theta, oracle.theta[0], "theta after 7 steps")
    eng = opt._engines[0]
    assert_close(eng.state(0)["m"], oracle.m[0], "m")
    assert eng.info()["t"] == 7 and eng.info()["launches"] == 7 + 4   # look-ahead + step, no restore pass


def test_whole_iteration_captured_into_a_cuda_graph():
    """Forward, backward and the optimizer step captured once (static input buffer) and
    replayed: the same parameters as the eager loop of a twin model."""
    a, b = _model(3), _model(3)
    kw = dict(HYPER, clip_threshold=0.5)
    eager = Novak(a.parameters(), **kw)
    graphed = Novak(b.parameters(), **kw, graph_capturable=True)
    xs = [torch.randn(16, 37, device=DEV) for _ in range(9)]
    static_x = torch.empty(16, 37, device=DEV)

    def iteration(model, opt, x):
        opt.zero_grad(set_to_none=False)         # gradients stay where they are: static buffers
        model(x).square().mean().backward()
        opt.step()

    for x in xs[:2]:                             # warm-up outside the capture, on a side stream
        iteration(a, eager, x)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        for x in xs[:2]:
            static_x.copy_(x)
            iteration(b, graphed, static_x)
    torch.cuda.current_stream().wait_stream(side)
    graph = torch.cuda.CUDAGraph()
    static_x.copy_(xs[2])
    with torch.cuda.graph(graph):
        iteration(b, graphed, static_x)
    for x in xs[2:]:
        iteration(a, eager, x)
        static_x.copy_(x)
        graph.replay()
    torch.cuda.synchronize()
    assert graphed._engines[0].info()["t"] == 9 == eager._engines[0].info()["t"]
    for pa, pb in zip(a.parameters(), b.parameters()):
        torch.testing.assert_close(pb, pa, rtol=1e-5, atol=1e-7)
