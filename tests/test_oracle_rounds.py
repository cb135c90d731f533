"""Pins for the oracle's round and epoch drivers (Algorithms 1, 2 and 3)."""
import os

import numpy as np
import pytest

import oracle
from paper_1805_10111_b200 import synth

F32 = np.float32
GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _problem(n=300, d=40, seed=21):
    h = synth.dense_logistic(n, d, seed)
    return h, oracle.Dataset(h.format, h.n, h.d, h.values, h.labels)


def _np_slope(X, y, rows, x):
    Xd, yd = X.astype(np.float64), y.astype(np.float64)
    return -yd[rows] / (1.0 + np.exp(yd[rows] * (Xd[rows] @ x.astype(np.float64))))


def _np_soft(v, t):
    return np.sign(v) * np.maximum(np.abs(v) - t, 0.0)


def test_bits_per_round_match_the_papers_message_sizes():
    rows = [l.split() for l in open(os.path.join(GOLD, "bits_per_round.txt")) if not l.startswith("#") and l.strip()]
    small = {r[0]: r for r in rows}
    # the oracle's counters on a scaled-down problem obey the same closed form ...
    h, data = _problem()
    for name, M, b_x, b in (("c1", 4, 8, 8), ("c2", 8, 8, 4)):
        cfg = oracle.make_config(h.d, M, 4, b_x, b, seed=3)
        run = oracle.Run(cfg, data, synth.normal_vector(h.d, 30, 0.1))
        run.epoch_begin()
        t0 = run.round(0, 0.1)
        t1 = run.round(1, 0.1)
        assert t0["flag_round"] and t0["bits_down"] == M                       # one flag bit per worker
        assert t1["bits_down"] == M * (32 + b_x * h.d) and t1["bits_up"] == M * (32 + b * h.d)
    # ... and the closed form reproduces the tabulated values at the full configurations
    for name, r in small.items():
        M, d, b_x, b, total, full = (int(t) for t in r[1:])
        assert M * (32 + b_x * d) + M * (32 + b * d) == total and 2 * M * 32 * d == full


def test_round_wiring_against_textbook_prox_svrg_step():
    """Algorithm 1 with the quantisers' outputs taken as given is ProxSVRG (Theorem 1's setting): every
    round must satisfy  alpha = minibatch grad(xhat) - minibatch grad(xsnap),
    x+ = prox_{eta h}(x - eta (mean_w Q(alpha_w) + grad f(xsnap)))  in independent numpy arithmetic."""
    h, data = _problem()
    X, y = h.values, h.labels
    M, B, eta, l1, l2 = 3, 8, 0.5, 1e-3, 1e-2
    cfg = oracle.make_config(h.d, M, B, 8, 8, l1=l1, l2=l2, seed=77)
    run = oracle.Run(cfg, data, synth.normal_vector(h.d, 31, 0.2))
    rnd = 0
    for epoch in range(2):
        run.epoch_begin()
        xs = run.xsnap.copy()
        gfull_np = (_np_slope(X, y, np.arange(h.n), xs)[:, None] * X.astype(np.float64)).mean(axis=0)
        assert np.allclose(run.gfull, gfull_np, rtol=1e-6, atol=1e-9)
        for t in range(5):
            x_before = run.x.copy()
            tr = run.round(rnd, eta, trace=True)
            assert tr["status"] == 0 and tr["flag_round"] == (t == 0)
            xhat = tr["xhat"]
            if t == 0:
                assert np.array_equal(xhat, xs)
            else:
                assert np.array_equal(xhat, tr["codes_x"].astype(F32) * tr["delta_x"][0])
                assert np.abs(xhat - x_before).max() <= tr["delta_x"][0] * 1.0001         # neighbours on the grid
            for w in range(M):
                rows = tr["rows"][w]
                assert np.array_equal(rows, oracle.sample_batch(77, rnd, w, M, h.n, B))
                a_np = ((_np_slope(X, y, rows, xhat) - _np_slope(X, y, rows, xs))[:, None] * X[rows].astype(np.float64)).mean(axis=0)
                assert np.allclose(tr["alpha"][w], a_np, rtol=1e-6, atol=1e-10)
                cw, dw, rc = oracle.quantize(tr["alpha"][w], 8, 77, rnd, w, oracle.STREAM_GRAD)
                assert np.array_equal(cw, tr["codes"][w]) and dw == tr["delta"][w]
            q_mean = (tr["codes"].astype(np.float64) * tr["delta"].astype(np.float64)[:, None]).mean(axis=0)
            u = q_mean + run.gfull
            v = x_before - eta * u
            x_np = _np_soft(v, eta * l1) / (1 + eta * l2)
            assert np.allclose(run.x, x_np, rtol=2e-6, atol=1e-7)
            assert tr["normx"] == np.abs(run.x).max()
            rnd += 1
        x_end = run.x.copy()
    run.epoch_begin()
    assert np.array_equal(run.xsnap, x_end)                                # xsnap^{s+1} = x_m^{s+1}


def test_quantised_run_tracks_full_precision_prox_svrg():
    """Section 5.1: low-precision runs converge like their full-precision counterparts.  Compared with a
    plain float64 ProxSVRG on the same batches, the oracle's loss stays close and decreases."""
    h, data = _problem(n=400, d=30, seed=22)
    X, y = h.values.astype(np.float64), h.labels.astype(np.float64)
    M, B, eta, l1 = 4, 8, 1.0, 1e-4
    cfg = oracle.make_config(h.d, M, B, 8, 8, l1=l1, seed=5)
    run = oracle.Run(cfg, data, np.zeros(h.d, F32))
    x = np.zeros(h.d); rnd = 0
    P0 = oracle.objective(data, run.x, l1, 0)
    for epoch in range(4):
        run.epoch_begin()
        xs = x.copy()
        gf = (_np_slope(h.values, h.labels, np.arange(h.n), xs)[:, None] * X).mean(axis=0)
        for t in range(25):
            run.round(rnd, eta)
            rows = np.concatenate([oracle.sample_batch(5, rnd, w, M, h.n, B) for w in range(M)])
            a = ((_np_slope(h.values, h.labels, rows, x) - _np_slope(h.values, h.labels, rows, xs))[:, None] * X[rows]).mean(axis=0)
            x = _np_soft(x - eta * (a + gf), eta * l1)
            rnd += 1
    P_or = oracle.objective(data, run.x, l1, 0)
    P_fp = oracle.objective(data, x.astype(F32), l1, 0)
    assert P_or < 0.8 * P0 and abs(P_or - P_fp) < 0.02 * P_fp


def test_sparse_variant_round():
    """Algorithm 2: beta from eq. (4), then Q on beta; message size 32 + nnz (ceil(log2 d) + b) bits."""
    h, data = _problem(n=200, d=100, seed=23)
    M, B, b = 3, 6, 4
    cfg = oracle.make_config(h.d, M, B, 8, b, l1=1e-4, sparsify=1, phi=0.0, msg_format=oracle.MSG_SPARSE, seed=9)
    run = oracle.Run(cfg, data, synth.normal_vector(h.d, 32, 0.2))
    run.epoch_begin()
    run.round(0, 0.3)
    tr = run.round(1, 0.3, trace=True)
    up = 0
    for w in range(M):
        r = oracle.sparsify(tr["alpha"][w], 0.0, 9, 1, w)
        assert np.array_equal(r["Z"], tr["Z"][w]) and np.array_equal(r["beta"], tr["beta"][w])
        cw, dw, _ = oracle.quantize_survivors(r["beta"], r["Z"], b, 9, 1, w)
        assert np.array_equal(cw, tr["codes"][w]) and dw == tr["delta"][w]
        assert tr["nnz"][w] == int(r["Z"].sum()) and 0 < tr["nnz"][w] < h.d
        up += 32 + int(r["Z"].sum()) * (7 + b)                                   # ceil(log2 100) = 7
    assert tr["bits_up"] == up
    cfg2 = oracle.make_config(h.d, M, B, 8, b, l1=1e-4, sparsify=1, phi=0.0, msg_format=oracle.MSG_DENSE, seed=9)
    run2 = oracle.Run(cfg2, data, synth.normal_vector(h.d, 32, 0.2))
    run2.epoch_begin(); run2.round(0, 0.3)
    tr2 = run2.round(1, 0.3, trace=True)
    assert tr2["bits_up"] == M * (32 + b * h.d) and np.array_equal(tr2["codes"], tr["codes"])
    assert np.array_equal(run.x, run2.x)


def test_accelerated_identities_and_snapshot_mean():
    """Algorithm 3: x_{t+1} = xsnap + theta (y_{t+1} - xsnap), hence x_{t+1} - x_t = theta (y_{t+1} - y_t)
    (used in Theorem 4's proof); xsnap^s = mean_t x_{t+1}^s; y carried across epochs; box keeps y in Omega."""
    h, data = _problem(n=200, d=25, seed=24)
    M, B, lr, m = 2, 8, 0.4, 6
    cfg = oracle.make_config(h.d, M, B, 8, 8, box_lo=-0.5, box_hi=0.5, accelerated=1, seed=13)
    run = oracle.Run(cfg, data, synth.normal_vector(h.d, 33, 0.1))
    rnd = 0
    for s in range(1, 4):
        theta = F32(2.0 / (s + 2)); eta = F32(lr) / theta                        # Section 5.1 schedule
        y_prev_epoch = run.y.copy()
        mean_prev = None if s == 1 else np.mean(xs_hist, axis=0)
        run.epoch_begin(theta)
        if s > 1:
            assert np.allclose(run.xsnap, mean_prev, rtol=1e-6, atol=1e-8)       # step 15
        assert np.array_equal(run.y, y_prev_epoch)                               # y_0^s = y_m^{s-1}
        assert np.allclose(run.x, theta * run.y + (1 - theta) * run.xsnap, rtol=1e-6, atol=1e-8)   # step 3
        assert not run.xsum.any()
        xs_hist = []
        for t in range(m):
            x0, y0 = run.x.copy(), run.y.copy()
            tr = run.round(rnd, eta, theta, trace=True)
            assert tr["flag_round"] == (s == 1 and t == 0)
            q_mean = (tr["codes"].astype(np.float64) * tr["delta"].astype(np.float64)[:, None]).mean(axis=0)
            y_np = np.clip(y0 - float(eta) * (q_mean + run.gfull), -0.5, 0.5)    # prox of the box indicator
            assert np.allclose(run.y, y_np, rtol=2e-6, atol=1e-7)
            assert np.abs(run.y).max() <= 0.5
            assert np.allclose(run.x - run.xsnap, theta * (run.y - run.xsnap), rtol=1e-5, atol=1e-7)
            assert np.allclose(run.x - x0, theta * (run.y - y0), rtol=1e-4, atol=2e-7)
            xs_hist.append(run.x.copy()); rnd += 1
        assert np.allclose(run.xsum, np.sum(xs_hist, axis=0), rtol=1e-6, atol=1e-7)


def test_expected_error_closed_form_and_bit_width_search():
    """Condition (3): E_Q||Q(x) - x||^2 <= mu ||x - xsnap||^2.  The closed form sum (x - z)(z + delta - x) is pinned
    by brute force over the grid and by the empirical mean of the oracle's own quantiser; the search returns the
    smallest admissible width among 2..11, is monotone in mu, and the expected error falls with every extra bit."""
    g = np.random.default_rng(31)
    d = 400
    x = g.standard_normal(d).astype(F32)
    for b in (2, 3, 4, 8, 10):
        L = 2 ** (b - 1) - 1
        delta = float(np.abs(x).max() / F32(L))
        grid = np.arange(-L - 1, L + 2) * delta
        want = 0.0
        for xi in x.astype(np.float64):
            z = grid[np.searchsorted(grid, xi, side="right") - 1]           # the grid point at or below x_i
            want += (xi - z) * (z + delta - xi)
        got = oracle.expected_sq_error(x, b)
        assert abs(got - want) <= 1e-9 * want
        assert got <= d * delta ** 2 / 4                                     # the variance bound of the appendix's first lemma
        acc = 0.0; N = 3000
        for rnd in range(N):
            codes, dl, _ = oracle.quantize(x, b, 77, rnd, 0, oracle.STREAM_MODEL)
            acc += float(((codes.astype(np.float64) * float(dl) - x) ** 2).sum())
        assert abs(acc / N - got) < 0.02 * got                               # Monte-Carlo over the oracle's quantiser
    xs = (x + F32(0.05) * g.standard_normal(d).astype(F32)).astype(F32)
    dist = float(((x.astype(np.float64) - xs) ** 2).sum())
    errs = [oracle.expected_sq_error(x, b) for b in range(2, 12)]              # the widths of Table 1
    assert all(errs[k] > errs[k + 1] for k in range(9))
    cases = [(errs[9] / dist * 0.5, 11), (errs[0] / dist * 100, 2)] + [(errs[b - 2] / dist * 1.01, b) for b in range(2, 12)]
    for mu, want_b in cases:
        b, e10, D = oracle.select_bx(x, xs, mu)
        assert b == want_b and np.allclose(e10, errs) and abs(D - dist) < 1e-12 * dist
    assert oracle.select_bx(x, x, 1e9)[0] == 11                              # x = xsnap: nothing admissible (the flag bit handles it)


def test_delayed_rounds_use_the_model_of_t_minus_delay():
    """Algorithm 1 step 11 evaluates the gradient at x_{D(t)} with t - D(t) <= tau (Assumption 3).  With per-worker
    delays the gradient difference of worker w must be the one at the low-precision model broadcast delays[w] rounds
    earlier in the epoch (clamped to the epoch's start), re-derived here in float64 numpy from broadcasts that the
    test rebuilds itself; zero delays must reproduce the ordinary round bit for bit."""
    h, data = _problem()
    M, B, tau = 3, 8, 2
    cfg = oracle.make_config(h.d, M, B, 8, 8, l1=1e-4, seed=9)
    x0 = synth.normal_vector(h.d, 35, 0.2)
    run = oracle.Run(cfg, data, x0); ref = oracle.Run(cfg, data, x0)
    g = np.random.default_rng(5)
    X, y = h.values.astype(np.float64), h.labels
    rnd = 0
    for epoch in range(2):
        run.epoch_begin(); ref.epoch_begin()
        mine = []                                            # this epoch's broadcasts, rebuilt independently
        for t in range(6):
            delays = [int(v) for v in g.integers(0, tau + 1, M)] if epoch == 1 else [0] * M
            x_before = run.x.copy()
            tr = run.round(rnd, 0.4, trace=True, delays=delays)
            if tr["flag_round"]:
                mine.append(run.xsnap.copy())
            else:
                cx, dx, _ = oracle.quantize(x_before, 8, 9, rnd, oracle.MASTER, oracle.STREAM_MODEL)
                mine.append(cx.astype(F32) * dx)
            assert tr["delays_used"] == [min(D, t) for D in delays]
            for w in range(M):
                xw = mine[t - min(delays[w], t)]
                rows = tr["rows"][w]
                want = ((_np_slope(X, y, rows, xw) - _np_slope(X, y, rows, run.xsnap))[:, None] * X[rows]).mean(axis=0)
                assert np.allclose(tr["alpha"][w], want, rtol=1e-5, atol=1e-7), (epoch, t, w)
            if epoch == 0:                                   # zero delays: the ordinary round
                ref.round(rnd, 0.4)
                assert np.array_equal(run.x, ref.x)
            rnd += 1
    # a delay matters: with every worker one round behind, the iterates leave the undelayed run's
    a = oracle.Run(cfg, data, x0); b = oracle.Run(cfg, data, x0)
    a.epoch_begin(); b.epoch_begin()
    for t in range(4):
        a.round(t, 0.4, delays=[1] * M); b.round(t, 0.4)
    assert not np.array_equal(a.x, b.x)


def test_delays_reach_across_the_epoch_boundary():
    """With across_epochs a delay is cut to the rounds of the whole run: in the first rounds of an epoch a lagging
    worker evaluates the PREVIOUS epoch's low-precision model against the NEW snapshot (Algorithm 1 step 11 with
    t - D(t) <= tau across the outer loop).  Re-derived in float64 numpy from broadcasts that the test rebuilds itself;
    a worker with delay 0 in the epoch's first round still sends exactly zero (x = xsnap there)."""
    h, data = _problem()
    M, B, tau = 3, 8, 2
    cfg = oracle.make_config(h.d, M, B, 8, 8, l1=1e-4, seed=11)
    x0 = synth.normal_vector(h.d, 36, 0.2)
    run = oracle.Run(cfg, data, x0)
    X, y = h.values.astype(np.float64), h.labels
    mine = []                                                # every broadcast of the run, rebuilt independently
    rnd = 0
    crossed = 0
    for epoch in range(3):
        run.epoch_begin()
        for t in range(4):
            delays = [tau, 0, 1] if t == 0 else [int(v) for v in np.random.default_rng(100 + rnd).integers(0, tau + 1, M)]
            x_before = run.x.copy()
            tr = run.round(rnd, 0.4, trace=True, delays=delays, across_epochs=True)
            if tr["flag_round"]:
                mine.append(run.xsnap.copy())
            else:
                cx, dx, _ = oracle.quantize(x_before, 8, 11, rnd, oracle.MASTER, oracle.STREAM_MODEL)
                mine.append(cx.astype(F32) * dx)
            assert tr["delays_used"] == [min(D, rnd) for D in delays]
            for w in range(M):
                used = min(delays[w], rnd)
                xw = mine[rnd - used]
                crossed += int(used > t)
                rows = tr["rows"][w]
                want = ((_np_slope(X, y, rows, xw) - _np_slope(X, y, rows, run.xsnap))[:, None] * X[rows]).mean(axis=0)
                assert np.allclose(tr["alpha"][w], want, rtol=1e-5, atol=1e-7), (epoch, t, w)
                if t == 0 and used == 0:
                    assert not np.any(tr["alpha"][w])
                if t == 0 and used > 0 and epoch > 0:
                    assert np.any(tr["alpha"][w])              # the old model is not the new snapshot
            rnd += 1
    assert crossed >= 4


def test_round_with_searched_model_bits():
    """With mu > 0 every non-flag round quantises the model with the searched width and pays for that width."""
    h, data = _problem()
    M, B = 2, 8
    seen = set()
    for mu in (1e-3, 50.0, 1e6):
        cfg = oracle.make_config(h.d, M, B, 8, 8, l1=1e-4, seed=3, mu=mu)
        run = oracle.Run(cfg, data, synth.normal_vector(h.d, 34, 0.2))
        run.epoch_begin()
        for rnd in range(6):
            x_before = run.x.copy()
            tr = run.round(rnd, 0.5, trace=True)
            if tr["flag_round"]:
                assert tr["bx_used"] == 0 and tr["bits_down"] == M
                continue
            want_b = oracle.select_bx(x_before, run.xsnap, mu)[0]
            assert tr["bx_used"] == want_b
            cx, dx, _ = oracle.quantize(x_before, want_b, 3, rnd, oracle.MASTER, oracle.STREAM_MODEL)
            assert np.array_equal(tr["codes_x"], cx) and tr["delta_x"][0] == dx
            assert tr["bits_down"] == M * (32 + want_b * h.d)
            seen.add(want_b)
    assert len(seen) >= 3 and min(seen) == 2 and max(seen) >= 8


def test_sequential_master_is_one_prox_svrg_step_per_message():
    """Algorithm 1 as written applies one message per master tick.  The sequential master must equal M successive
    textbook steps x <- prox(x - eta (Q(alpha_w) + grad f(xsnap))) in independent float64 numpy, reduce to the
    synchronous master for M = 1, and for Algorithm 3 keep x = xsnap + theta (y - xsnap) with the running sum taking
    every tick's x."""
    g = np.random.default_rng(41)
    d, M, eta, l1, l2 = 60, 5, 0.3, 0.02, 0.1
    codes = g.integers(-7, 8, (M, d)).astype(np.int32); delta = (g.random(M) * 0.1).astype(F32)
    gfull = g.standard_normal(d).astype(F32); x0 = g.standard_normal(d).astype(F32)
    x = x0.copy()
    nx = oracle.master_step(codes, delta, gfull, x, eta, l1=l1, l2=l2, sequential=True)
    ref = x0.astype(np.float64)
    for w in range(M):
        u = codes[w].astype(np.float64) * float(delta[w]) + gfull
        ref = _np_soft(ref - eta * u, eta * l1) / (1 + eta * l2)
    assert np.allclose(x, ref, rtol=5e-6, atol=1e-6) and nx == np.abs(x).max()
    # differs from the averaged step, but coincides with it for one worker
    xa = x0.copy(); oracle.master_step(codes, delta, gfull, xa, eta, l1=l1, l2=l2)
    assert np.abs(xa - x).max() > 1e-3
    x1 = x0.copy(); x2 = x0.copy()
    oracle.master_step(codes[:1], delta[:1], gfull, x1, eta, l1=l1, l2=l2, sequential=True)
    oracle.master_step(codes[:1], delta[:1], gfull, x2, eta, l1=l1, l2=l2)
    assert np.array_equal(x1, x2)
    # Algorithm 3
    theta = F32(0.4); xs = g.standard_normal(d).astype(F32); y0 = g.standard_normal(d).astype(F32)
    y = y0.copy(); xx = x0.copy(); xsum = np.zeros(d, F32)
    oracle.master_step(codes, delta, gfull, xx, eta, theta, True, y, xs, xsum, lo=-1.0, hi=1.0, sequential=True)
    yr = y0.astype(np.float64); acc = np.zeros(d)
    for w in range(M):
        yr = np.clip(yr - eta * (codes[w] * float(delta[w]) + gfull), -1.0, 1.0)
        acc += xs + float(theta) * (yr - xs)
    assert np.allclose(y, yr, rtol=5e-6, atol=1e-6)
    assert np.allclose(xx, xs + theta * (y - xs), rtol=1e-6, atol=1e-6) and np.allclose(xsum, acc, rtol=1e-5, atol=1e-5)


def test_sequential_rounds_average_over_ticks():
    h, data = _problem(n=200, d=25, seed=25)
    M, m = 3, 4
    cfg = oracle.make_config(h.d, M, 8, 8, 8, box_lo=-0.5, box_hi=0.5, accelerated=1, seed=15, sequential=1)
    run = oracle.Run(cfg, data, synth.normal_vector(h.d, 35, 0.1))
    theta = F32(0.5)
    run.epoch_begin(theta)
    for rnd in range(m):
        run.round(rnd, 0.2, theta)
    xsum = run.xsum.copy()
    run.epoch_begin(theta)
    assert np.allclose(run.xsnap, xsum / F32(m * M), rtol=1e-6, atol=1e-8)     # mean over the m*M master ticks
