"""GPU parity of the 3-layer network workload (Section 5.2) against the CPU oracle: epoch gradient, objective, the
worker's gradient difference, and whole rounds in lockstep (codes bit-exact given the GPU's own gradient)."""
import numpy as np
import pytest

import oracle
from paper_1805_10111_b200 import synth
from test_gpu_round import Lockstep, _close, _dev, dq  # noqa: F401  (fixture and helpers)

pytestmark = pytest.mark.gpu
F32 = np.float32


def _net(n, n_in, hidden, classes, seed):
    h = synth.image_classification(n, n_in, classes, 300 + seed)
    x = synth.mlp_init(n_in, hidden, classes, 310 + seed)
    x = (x + F32(0.05) * np.random.default_rng(seed).standard_normal(x.size).astype(F32)).astype(F32)
    return h, x


@pytest.mark.parametrize("n,n_in,hidden,classes", [(300, 37, 9, 4), (700, 784, 100, 10)])
def test_network_epoch_gradient_objective_and_worker_gradient(dq, n, n_in, hidden, classes):
    import torch
    h, x = _net(n, n_in, hidden, classes, 1)
    od = oracle.Dataset(h.format, h.n, h.d, h.values, h.labels)
    P = x.size
    M, B, bx, seed, rnd = 3, 20, 8, 33, 4
    cfg = dq.make_config(P, M, B=B, bx=bx, seed=seed, lambda2=1e-4, model=dq.DQ_MODEL_MLP, hidden=hidden, classes=classes)
    data = dq.Data(h)
    rc, ctx = dq.dq_create(cfg, data); assert rc == 0
    st = dq.State(x, n=h.n)
    assert dq.dq_epoch_begin(ctx, st) == 0
    g = oracle.mlp_grad(od, hidden, classes, x)
    nbad, worst = _close(st.g_full.cpu().numpy(), g, rel=2e-5)
    assert nbad == 0, (nbad, worst)
    Pobj = torch.zeros(1, dtype=torch.float64, device="cuda")
    assert dq.dq_objective(ctx, st.x, Pobj) == 0
    want = oracle.mlp_objective(od, hidden, classes, x, 0.0, 1e-4)
    assert abs(Pobj.item() - want) < 2e-6 * max(1.0, want)
    # worker gradient difference at a quantised model
    xq = (x + F32(0.01) * np.random.default_rng(2).standard_normal(P).astype(F32)).astype(F32)
    cx, dx, _ = oracle.quantize(xq, bx, seed, rnd, oracle.MASTER, oracle.STREAM_MODEL)
    xhat = cx.astype(F32) * dx
    alpha = torch.full((M, P), 3.0, device="cuda"); ninf = torch.zeros(M, device="cuda")
    assert dq.dq_worker_grad(ctx, _dev(oracle.pack(cx, bx)), _dev(np.array([dx], F32)), 0, st, rnd, None, alpha, ninf) == 0
    for w in range(M):
        rows = oracle.sample_batch(seed, rnd, w, M, h.n, B)
        a, S = oracle.mlp_worker_grad(od, hidden, classes, xhat, x, rows)
        nbad, worst = _close(alpha[w].cpu().numpy(), a, S)
        assert nbad == 0, (w, nbad, worst)
        assert ninf[w].item() == np.abs(alpha[w].cpu().numpy()).max()
    first = alpha.clone()
    assert dq.dq_worker_grad(ctx, _dev(oracle.pack(cx, bx)), _dev(np.array([dx], F32)), 0, st, rnd, None, alpha, ninf) == 0
    assert torch.equal(alpha, first)                                        # no atomics: reproducible
    dq.dq_destroy(ctx)


@pytest.mark.parametrize("extra", [dict(), dict(sparsify=1, phi=0.0, msg_format=1), dict(accelerated=1, box_lo=-2.0, box_hi=2.0)])
def test_network_lockstep_rounds(dq, extra):
    h, x = _net(400, 48, 12, 5, 2)
    kw = dict(M=4, B=20, bx=8, b=4, lambda2=1e-4, seed=40, model=1, hidden=12, classes=5)
    kw.update(extra)
    ls = Lockstep(dq, h, x, **kw)
    acc = bool(extra.get("accelerated", 0))
    rnd = 0
    for s_ in range(1, 3):
        theta = F32(2.0 / (s_ + 2)) if acc else F32(0.0)
        ls.epoch(theta)
        for t in range(8):
            ls.round(rnd, 0.05 if acc else 0.2, theta)
            rnd += 1
    assert ls.far_flips == 0
    ls.close()


@pytest.mark.parametrize("extra", [dict(max_delay=2), dict(max_delay=3, accelerated=1, box_lo=-2.0, box_hi=2.0)])
def test_network_lockstep_delayed_workers(dq, extra):
    """Lagging workers on the network (Algorithm 1 step 11 with x_{D(t)}): each worker's gradient difference is taken at
    the low-precision parameters broadcast `delay` rounds earlier in the epoch (the ring keeps xhat itself here), with
    delays that change every round; B = 20 rows per worker do not fill the kernel's row tiles."""
    h, x = _net(400, 48, 12, 5, 5)
    kw = dict(M=4, B=20, bx=8, b=4, lambda2=1e-4, seed=46, model=1, hidden=12, classes=5)
    kw.update(extra)
    ls = Lockstep(dq, h, x, **kw)
    g = np.random.default_rng(46)
    acc, tau, M = bool(extra.get("accelerated", 0)), extra["max_delay"], kw["M"]
    rnd = 0
    for s_ in range(1, 4):
        theta = F32(2.0 / (s_ + 2)) if acc else F32(0.0)
        ls.epoch(theta)
        for t in range(2 * tau + 3):
            delays = [int(v) for v in g.integers(0, tau + 1, M)] if s_ > 1 else [tau] * M
            tr = ls.round(rnd, 0.05 if acc else 0.2, theta, delays=delays)
            assert tr["delays_used"] == [min(D, t) for D in delays]
            rnd += 1
    assert ls.far_flips == 0
    ls.close()


def test_network_delays_across_epochs(dq):
    """The same for the network: the ring keeps the low-precision parameters themselves, so a worker that lags over
    the epoch boundary evaluates last epoch's parameters against the new snapshot."""
    h, x = _net(400, 48, 12, 5, 6)
    kw = dict(M=4, B=20, bx=8, b=4, lambda2=1e-4, seed=47, model=1, hidden=12, classes=5, max_delay=2, delay_across_epochs=1)
    ls = Lockstep(dq, h, x, **kw)
    g = np.random.default_rng(47)
    rnd = 0
    for s_ in range(3):
        ls.epoch(F32(0.0))
        for t in range(5):
            delays = [2] * 4 if t == 0 else [int(v) for v in g.integers(0, 3, 4)]
            tr = ls.round(rnd, 0.2, F32(0.0), delays=delays)
            assert tr["delays_used"] == [min(D, rnd) for D in delays]
            rnd += 1
    assert ls.far_flips == 0
    ls.close()


def test_network_full_size_rounds(dq):
    """784-100-10 on 2,000 image-shaped rows, M = 8 workers, B = 20, b_x = 8, b = 4 (the paper's setting for this model)."""
    h, x = _net(2000, 784, 100, 10, 3)
    kw = dict(M=8, B=20, bx=8, b=4, lambda2=1e-4, seed=41, model=1, hidden=100, classes=10)
    ls = Lockstep(dq, h, x, **kw)
    ls.epoch()
    for rnd in range(6):
        ls.round(rnd, 0.1)
    print("\n[nn] flips %d of %d, beyond band %d, worst alpha error %.2e" % (ls.flips, ls.coords, ls.far_flips, ls.worst_alpha))
    assert ls.far_flips == 0
    ls.close()


def test_network_free_running_loss(dq):
    """GPU and oracle run on their own for 60 rounds on the network; the objective agrees within 1e-4 relative."""
    import torch
    h, x = _net(500, 48, 12, 5, 4)
    od = oracle.Dataset(h.format, h.n, h.d, h.values, h.labels)
    kw = dict(B=20, bx=8, b=4, lambda2=1e-4, seed=42, model=1, hidden=12, classes=5)
    cfg = dq.make_config(x.size, 4, **kw)
    data = dq.Data(h)
    rc, ctx = dq.dq_create(cfg, data); assert rc == 0
    st = dq.State(x, n=h.n)
    ocfg = oracle.make_config(x.size, 4, 20, 8, 4, l2=1e-4, seed=42, model=1, hidden=12, classes=5)
    run = oracle.Run(ocfg, od, x)
    P = torch.zeros(1, dtype=torch.float64, device="cuda")
    first = last = None
    for rnd in range(60):
        if rnd % 20 == 0:
            assert dq.dq_epoch_begin(ctx, st) == 0; run.epoch_begin()
        assert dq.dq_round(ctx, st, rnd, 0.2) == 0; run.round(rnd, 0.2)
        if rnd % 10 == 9:
            assert dq.dq_objective(ctx, st.x, P) == 0
            Po = oracle.mlp_objective(od, 12, 5, run.x, 0.0, 1e-4)
            assert abs(P.item() - Po) <= 1e-4 * max(abs(Po), 1e-3), (rnd, P.item(), Po)
            first = first if first is not None else Po; last = Po
    assert last < first and dq.dq_poll_status(ctx) == (0, 0)
    dq.dq_destroy(ctx)


def _draw_network_case(g):
    """One random network configuration: any layer sizes up to the paper's 784-100-10 and beyond, any minibatch from one
    row, every model width, every regulariser, with and without sparsification, momentum and the one-by-one master."""
    n_in = int(g.integers(3, 785)); hidden = int(g.integers(1, 301)); classes = int(g.integers(2, 18))
    if g.random() < 0.15:
        n_in, hidden, classes = 784, 100, 10                                   # the shape of Section 5.2
    n = int(g.integers(60, 400))
    h, x = _net(n, n_in, hidden, classes, int(g.integers(1, 1000)))
    M = int(g.choice([1, 2, 4, 8, 17])); B = min(int(g.choice([1, 2, 3, 20, 64, 100, 150])), n)
    kw = dict(M=M, B=B, bx=int(g.integers(2, 12)), b=int(g.choice([2, 4, 8])), seed=int(g.integers(1, 1 << 30)), model=1,
              hidden=hidden, classes=classes)
    r = g.random()
    if r < 0.4:
        kw["lambda2"] = 1e-4
    elif r < 0.6:
        kw["lambda1"] = 1e-5
    else:
        kw.update(box_lo=-2.0, box_hi=2.0)
    if g.random() < 0.3:
        kw.update(sparsify=1, phi=float(g.choice([0.0, 20.0])), msg_format=int(g.integers(0, 2)))
    if g.random() < 0.3:
        kw["accelerated"] = 1
    if g.random() < 0.2:
        kw["sequential"] = 1
    if g.random() < 0.2:
        kw["no_fused"] = 1
    if g.random() < 0.15:
        kw["no_graph"] = 1
    if g.random() < 0.15:
        kw["mu"] = float(g.choice([0.3, 30.0]))
    return h, x, kw


def test_network_random_shapes(dq):
    """200 seeded random network shapes (3..784 inputs, 1..300 hidden units, 2..17 classes, minibatches from one row)
    through two epochs of lockstep rounds: every coordinate of every worker's gradient difference within
    1e-5 max(|oracle|, S_i, 1e-3 ||oracle||_inf), the epoch gradient within 2e-5, codes bit-exact on the GPU's own
    gradient, no flip outside the threshold band.  A failure names its trial, which reproduces alone."""
    worst = 0.0
    for trial in range(200):
        g = np.random.default_rng([1807, trial])
        h, x, kw = _draw_network_case(g)
        acc = bool(kw.get("accelerated", 0))
        try:
            ls = Lockstep(dq, h, x, **kw)
            rnd = 0
            for ep in range(2):
                theta = F32(2.0 / (ep + 3)) if acc else F32(0.0)
                ls.epoch(theta)
                for t in range(4):
                    ls.round(rnd, (0.02 / float(theta)) if acc else 0.1, theta)
                    rnd += 1
            assert ls.far_flips == 0, ("far flips", ls.far_flips)
            worst = max(worst, ls.worst_alpha)
            ls.close()
        except AssertionError as e:
            raise AssertionError("trial %d n=%d n_in=%d %r: %r" % (trial, h.n, h.d, kw, e)) from e
    print("\n[nn random shapes] worst gradient error %.2e of the tolerance scale (bound 1e-5)" % worst)
