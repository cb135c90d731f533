"""Pins for the oracle's 3-layer network (Section 5.2): loss against a plain numpy forward pass, gradients against
finite differences of that loss in double, the worker's gradient difference, and rounds that run on it."""
import numpy as np

import oracle
from paper_1805_10111_b200 import synth

F32 = np.float32


def _net(n=60, n_in=12, hidden=7, classes=4, seed=0):
    h = synth.image_classification(n, n_in, classes, 200 + seed)
    data = oracle.Dataset(h.format, h.n, h.d, h.values, h.labels)
    x = synth.mlp_init(n_in, hidden, classes, 210 + seed)
    x += F32(0.05) * np.random.default_rng(seed).standard_normal(x.size).astype(F32)     # non-zero biases too
    return h, data, x.astype(F32), hidden, classes


def _np_loss(h, x, hidden, classes, rows):
    n_in = h.d
    xd = x.astype(np.float64)
    W1 = xd[:hidden * n_in].reshape(hidden, n_in); b1 = xd[hidden * n_in:hidden * n_in + hidden]
    o = hidden * n_in + hidden
    W2 = xd[o:o + classes * hidden].reshape(classes, hidden); b2 = xd[o + classes * hidden:]
    X = h.values[rows].astype(np.float64); y = h.labels[rows].astype(int)
    H = np.maximum(X @ W1.T + b1, 0.0)
    Z = H @ W2.T + b2
    lse = np.log(np.exp(Z - Z.max(axis=1, keepdims=True)).sum(axis=1)) + Z.max(axis=1)
    return float(np.mean(lse - Z[np.arange(len(rows)), y]))


def test_parameter_count_and_loss():
    h, data, x, hidden, classes = _net()
    assert oracle.mlp_params(784, 100, 10) == 79510 and x.size == oracle.mlp_params(h.d, hidden, classes)
    rows = np.arange(h.n)
    assert abs(oracle.mlp_loss(data, hidden, classes, x) - _np_loss(h, x, hidden, classes, rows)) < 1e-12
    sub = np.array([3, 3, 17, 0, 59])
    assert abs(oracle.mlp_loss(data, hidden, classes, x, sub) - _np_loss(h, x, hidden, classes, sub)) < 1e-12
    zero = np.zeros_like(x)
    assert abs(oracle.mlp_loss(data, hidden, classes, zero) - np.log(classes)) < 1e-12      # uniform softmax
    l1, l2 = 0.01, 0.3
    xd = x.astype(np.float64)
    want = _np_loss(h, x, hidden, classes, rows) + float(F32(l1)) * np.abs(xd).sum() + 0.5 * float(F32(l2)) * (xd ** 2).sum()
    assert abs(oracle.mlp_objective(data, hidden, classes, x, l1, l2) - want) < 1e-10


def test_gradient_against_finite_differences():
    h, data, x, hidden, classes = _net(seed=1)
    rows = np.arange(h.n)
    g = oracle.mlp_grad(data, hidden, classes, x)
    step = F32(2.0 ** -10)
    rng = np.random.default_rng(5)
    for i in list(rng.choice(x.size, 60, replace=False)) + [x.size - 1, hidden * h.d, hidden * h.d + hidden]:
        xp, xm = x.copy(), x.copy()
        xp[i] += step; xm[i] -= step
        fd = (_np_loss(h, xp, hidden, classes, rows) - _np_loss(h, xm, hidden, classes, rows)) / (float(xp[i]) - float(xm[i]))
        assert abs(fd - g[i]) < 2e-5, (i, fd, g[i])                  # ReLU kinks are a set of measure zero
    sub = np.array([1, 1, 8, 40])
    gs = oracle.mlp_grad(data, hidden, classes, x, sub)
    per = np.mean([oracle.mlp_grad(data, hidden, classes, x, np.array([r])) for r in sub], axis=0)
    assert np.allclose(gs, per, rtol=1e-6, atol=1e-9)                   # minibatch gradient = mean of per-sample ones


def test_worker_gradient_difference():
    h, data, x, hidden, classes = _net(seed=2)
    xs = x.copy()
    xh = (x + F32(0.01) * np.random.default_rng(9).standard_normal(x.size).astype(F32)).astype(F32)
    rows = np.array([5, 9, 9, 33, 2, 58])
    a, S = oracle.mlp_worker_grad(data, hidden, classes, xh, xs, rows)
    want = oracle.mlp_grad(data, hidden, classes, xh, rows).astype(np.float64) - oracle.mlp_grad(data, hidden, classes, xs, rows)
    assert np.allclose(a, want, rtol=0, atol=3e-7)
    assert np.all(S >= np.abs(a) * (1 - 1e-6))
    a0, _ = oracle.mlp_worker_grad(data, hidden, classes, xs, xs, rows)
    assert not a0.any()                                                  # flag round: exactly zero


def test_rounds_on_the_network_decrease_the_loss():
    h, data, x, hidden, classes = _net(n=200, n_in=20, hidden=8, classes=5, seed=3)
    P = x.size
    cfg = oracle.make_config(P, 4, 10, 8, 4, l2=1e-4, seed=6, model=oracle.MODEL_MLP, hidden=hidden, classes=classes)
    run = oracle.Run(cfg, data, x)
    first = oracle.mlp_objective(data, hidden, classes, run.x, 0, 1e-4)
    rnd = 0
    for epoch in range(4):
        run.epoch_begin()
        assert np.allclose(run.gfull, oracle.mlp_grad(data, hidden, classes, run.xsnap), rtol=0, atol=0)
        for t in range(25):
            tr = run.round(rnd, 0.2, trace=(t == 3))
            if t == 3:
                a, _ = oracle.mlp_worker_grad(data, hidden, classes, tr["xhat"], run.xsnap, tr["rows"][1])
                assert np.array_equal(a, tr["alpha"][1])
            rnd += 1
    assert oracle.mlp_objective(data, hidden, classes, run.x, 0, 1e-4) < 0.8 * first
