"""Pins for the oracle's logistic gradients, the sparsifier of eq. (4) / Lemma 2 and the prox step."""
import math
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_1805_10111_b200 import synth

F32 = np.float32


def _tiny(n=40, d=12, seed=0, density=0.4):
    g = np.random.default_rng(seed)
    X = g.standard_normal((n, d)).astype(F32)
    X[g.random((n, d)) > density] = 0.0
    X[:, 0] = g.standard_normal(n).astype(F32)           # no empty rows
    y = np.where(g.random(n) < 0.5, 1.0, -1.0).astype(F32)
    dense = oracle.Dataset(oracle.DENSE_F32, n, d, X, y)
    rp = np.zeros(n + 1, np.int64); ci = []; va = []
    for r in range(n):
        nz = np.nonzero(X[r])[0]
        ci += list(nz); va += list(X[r, nz]); rp[r + 1] = len(ci)
    csr = oracle.Dataset(oracle.CSR_F32, n, d, np.array(va, F32), y, np.array(ci, np.int32), rp)
    Xb = synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(X))
    bf = oracle.Dataset(oracle.DENSE_BF16, n, d, synth.f32_to_bf16_bits(X), y)
    bf_as_f32 = oracle.Dataset(oracle.DENSE_F32, n, d, Xb, y)
    return X, y, dense, csr, bf, bf_as_f32


# ---------------------------------------------------------------------------------------------------
# gradients
# ---------------------------------------------------------------------------------------------------
def test_loss_matches_library_logaddexp():
    X, y, dense, csr, _, _ = _tiny()
    x = np.random.default_rng(1).standard_normal(X.shape[1]).astype(F32)
    ref = np.mean(np.logaddexp(0.0, -y.astype(np.float64) * (X.astype(np.float64) @ x.astype(np.float64))))
    assert abs(oracle.smooth_loss(dense, x) - ref) < 1e-13
    assert abs(oracle.smooth_loss(csr, x) - ref) < 1e-13
    l1, l2 = 0.3, 0.7
    P = oracle.objective(dense, x, l1, l2)
    xd = x.astype(np.float64)
    assert abs(P - (ref + float(F32(l1)) * np.abs(xd).sum() + 0.5 * float(F32(l2)) * (xd ** 2).sum())) < 1e-12


def test_full_gradient_against_finite_differences():
    X, y, dense, csr, bf, bf32 = _tiny()
    d = X.shape[1]
    x = (np.random.default_rng(2).standard_normal(d) * 0.5).astype(F32)
    h = F32(2.0 ** -9)
    for data in (dense, csr, bf):
        g, z = oracle.full_grad(data, x)
        Xeff = X if data is not bf else synth.bf16_bits_to_f32(synth.f32_to_bf16_bits(X))
        assert np.allclose(z, Xeff.astype(np.float64) @ x.astype(np.float64), rtol=1e-6, atol=1e-7)
        for i in range(d):
            xp, xm = x.copy(), x.copy()
            xp[i] += h; xm[i] -= h
            fd = (oracle.smooth_loss(data, xp) - oracle.smooth_loss(data, xm)) / (float(xp[i]) - float(xm[i]))
            assert abs(fd - g[i]) < 5e-6                 # O(h^2) truncation, fp32 rounding of g
    g1, _ = oracle.full_grad(bf, x); g2, _ = oracle.full_grad(bf32, x)
    assert np.array_equal(g1, g2)                        # bf16 storage is converted exactly
    g1, _ = oracle.full_grad(dense, x); g2, _ = oracle.full_grad(csr, x)
    assert np.allclose(g1, g2, rtol=1e-6, atol=1e-9)     # same matrix, two layouts (summation order differs)


def test_worker_gradient_is_difference_of_minibatch_gradients():
    """alpha = (1/B) sum_a [grad f_a(xhat) - grad f_a(xsnap)]; with the batch = all rows it must equal
    grad f(xhat) - grad f(xsnap), and with xhat = xsnap it is exactly zero (flag round)."""
    X, y, dense, csr, bf, _ = _tiny()
    n, d = X.shape
    g = np.random.default_rng(3)
    xs = (g.standard_normal(d) * 0.3).astype(F32)
    xh = (xs + g.standard_normal(d).astype(F32) * F32(0.05)).astype(F32)
    for data in (dense, csr, bf):
        a_all, S = oracle.worker_grad(data, xh, xs, np.arange(n))
        gh, _ = oracle.full_grad(data, xh); gs, _ = oracle.full_grad(data, xs)
        assert np.allclose(a_all, gh.astype(np.float64) - gs, rtol=0, atol=2e-7)
        assert np.all(S >= np.abs(a_all) * (1 - 1e-6))
        a0, S0 = oracle.worker_grad(data, xs, xs, np.arange(n))
        assert not a0.any() and not S0.any()
    # a hand-written numpy minibatch gradient with repeated rows
    rows = np.array([3, 3, 7, 0, 39, 7])
    Xd, yd = X.astype(np.float64), y.astype(np.float64)
    slope = lambda xx: -yd[rows] / (1.0 + np.exp(yd[rows] * (Xd[rows] @ xx.astype(np.float64))))
    ref = ((slope(xh) - slope(xs))[:, None] * Xd[rows]).mean(axis=0)
    a, _ = oracle.worker_grad(dense, xh, xs, rows)
    assert np.allclose(a, ref, rtol=1e-6, atol=1e-10)
    a, _ = oracle.worker_grad(csr, xh, xs, rows)
    assert np.allclose(a, ref, rtol=1e-6, atol=1e-10)


def test_batch_sampling_partition_and_words():
    seed, rnd, M, n, B = 99, 12, 5, 1003, 64
    seen = []
    for w in range(M):
        rows = oracle.sample_batch(seed, rnd, w, M, n, B)
        lo, hi = (w * n) // M, ((w + 1) * n) // M
        assert rows.min() >= lo and rows.max() < hi
        for j in (0, 1, 5, 63):
            word = int(oracle.philox4x32_10([j >> 2, rnd, w, oracle.STREAM_BATCH], [seed & 0xFFFFFFFF, seed >> 32])[j & 3])
            assert rows[j] == lo + (word * (hi - lo) >> 32)
        seen.append(rows)
    assert not np.array_equal(seen[0] - 0, seen[1] - (n // M))          # workers draw different slots
    # roughly uniform over the partition
    rows = np.concatenate([oracle.sample_batch(seed, r, 0, 1, 100, 1000) for r in range(20)])
    cnt = np.bincount(rows, minlength=100)
    assert ((cnt - 200) ** 2 / 200).sum() < 99 + 6 * math.sqrt(198)


# ---------------------------------------------------------------------------------------------------
# sparsifier
# ---------------------------------------------------------------------------------------------------
def test_l1_norm_fixed_point_is_exact_and_order_free():
    g = np.random.default_rng(5)
    for trial in range(10):
        d = int(g.integers(1, 5000))
        v = (g.standard_normal(d) * 10.0 ** g.integers(-20, 20)).astype(F32)
        v[g.random(d) < 0.3] = 0.0
        if trial == 4:
            v[:] = 0
        n1 = oracle.norm_l1(v)
        exact = math.fsum(abs(float(t)) for t in v)
        ninf = float(np.abs(v).max())
        assert abs(float(n1) - exact) <= d * ninf * 2.0 ** -34 + exact * 2.0 ** -23
        for _ in range(3):
            assert oracle.norm_l1(g.permutation(v)) == n1                # exactly, any order
    # the definition itself: truncation of |v_i| 2^(35-e) with ||v||_inf in [2^(e-1), 2^e)
    v = np.array([0.75, -0.1, 3e-12, 0.3], F32)
    e = 0                                                                # 0.75 in [2^-1, 2^0)
    tot = sum(int(Fraction(abs(float(t))) * (1 << 35)) for t in v)
    assert oracle.norm_l1(v) == F32(tot / 2.0 ** 35)


def test_sparsifier_probabilities_and_budget():
    g = np.random.default_rng(6)
    d = 4000
    alpha = (g.standard_normal(d) * g.random(d) ** 4).astype(F32)
    alpha[g.random(d) < 0.5] = 0
    ninf, n1 = np.abs(alpha).max(), oracle.norm_l1(alpha)
    cap = float(n1) / float(ninf)
    for phi in (0.0, -1.0, cap * 0.25, cap * 0.999, cap * 3.0, 1e9):
        r = oracle.sparsify(alpha, phi, 3, 1, 2)
        assert r["status"] == 0 and r["ninf"] == ninf and r["n1"] == n1
        phi_eff = float(r["phi_eff"])
        want = cap if phi <= 0 else min(phi, cap)                       # Lemma 2 needs phi <= |a|_1/|a|_inf
        assert abs(phi_eff - want) <= 1e-6 * want
        m = r["m"].astype(np.int64)
        assert m.max() <= 65536 and np.all((m > 0) == (alpha != 0))     # 0 < p_i <= 1 on the support
        p = np.abs(alpha.astype(np.float64)) * phi_eff / float(n1)      # Lemma 2's optimum
        assert np.all(m >= np.minimum(p, 1) * 65536 * (1 - 1e-6)) and np.all(m <= np.minimum(p, 1) * 65536 * (1 + 1e-6) + 1)
        nnz_a = int((alpha != 0).sum())
        assert phi_eff * (1 - 1e-5) <= m.sum() / 65536 <= phi_eff * (1 + 1e-5) + nnz_a / 65536
        Z = r["Z"].astype(bool)
        u = np.array([oracle.u16(3, 1, 2, oracle.STREAM_MASK, i) for i in range(d)])
        assert np.array_equal(Z, u < m)                                 # Z_i ~ Bernoulli(m_i / 2^16)
        beta = r["beta"]
        assert not beta[~Z].any()
        assert np.array_equal(beta[Z], (alpha[Z] * F32(65536.0)) / m[Z].astype(F32))   # alpha_i / p_i
        if phi <= 0 or phi >= cap:
            i = int(np.argmax(np.abs(alpha)))
            assert m[i] == 65536 and Z[i] and beta[i] == alpha[i]        # equality budget keeps the max coordinate


def test_sparsifier_subnormal_vectors_exact():
    """eq. (4) on vectors whose l1 norm is a subnormal number, against exact rationals.  (a) phi/|alpha|_1 still a finite
    fp32 number: every p_i 2^16 equals Lemma 2's value computed with fractions.  (b) phi/|alpha|_1 beyond the fp32
    range: a zero coordinate has p_i = 0 and never survives, a nonzero one has p_i = 1 (eq. (4) allows any
    0 < p_i <= 1), so beta = alpha; no NaN reaches a code, a mask bit or a norm."""
    sub = lambda k, e: F32(math.ldexp(float(k), e))
    # (a) |alpha|_1 = 2^-127 (subnormal), budget 1: s = 2^127 is finite
    alpha = np.array([sub(1, -128), 0.0, sub(-1, -129), sub(1, -129), 0.0], F32)
    r = oracle.sparsify(alpha, 1.0, 4, 2, 1)
    n1 = sum(Fraction(abs(float(t))) for t in alpha)
    assert r["status"] == 0 and Fraction(float(r["n1"])) == n1 == Fraction(1, 2 ** 127) and r["phi_eff"] == 1.0
    want_m = [math.ceil(Fraction(abs(float(t))) * 1 / n1 * 65536) for t in alpha]          # p_i = |alpha_i| phi / |alpha|_1
    assert list(r["m"]) == want_m == [32768, 0, 16384, 16384, 0]
    u = [oracle.u16(4, 2, 1, oracle.STREAM_MASK, i) for i in range(alpha.size)]
    assert list(r["Z"]) == [int(ui < mi) for ui, mi in zip(u, want_m)]
    for i in range(alpha.size):
        want = Fraction(float(alpha[i])) * 65536 / want_m[i] if r["Z"][i] else 0           # alpha_i / p_i
        assert Fraction(float(r["beta"][i])) == want
    # (b) |alpha|_1 = 6 * 2^-149: phi_eff / |alpha|_1 = 2^149 / 3 overflows
    alpha = np.array([sub(3, -149), 0.0, sub(-1, -149), 0.0, sub(2, -149), 0.0, 0.0], F32)
    for phi in (0.0, 1.5, 100.0):
        r = oracle.sparsify(alpha, phi, 4, 3, 0)
        assert r["status"] == 0 and Fraction(float(r["n1"])) == Fraction(6, 2 ** 149)
        assert r["phi_eff"] == (2.0 if phi != 1.5 else 1.5)                                 # clamp of Lemma 2: 6/3
        assert list(r["m"]) == [65536, 0, 65536, 0, 65536, 0, 0]
        assert list(r["Z"]) == [1, 0, 1, 0, 1, 0, 0]
        assert np.array_equal(r["beta"], alpha) and not np.isnan(r["beta"]).any()
        codes, delta, rc = oracle.quantize_survivors(r["beta"], r["Z"], 4, 4, 3, 0)
        assert rc == 0 and np.isfinite(delta) and not codes[[1, 3, 5, 6]].any() and np.abs(codes).max() <= 7


def test_sparsifier_moments():
    """E[beta] = alpha, E||beta||^2 = sum alpha_i^2/p_i (= |alpha|_1^2/phi at Lemma 2's p), E[nnz] = sum p_i."""
    g = np.random.default_rng(7)
    d, N = 300, 6000
    alpha = (g.standard_normal(d) * g.random(d)).astype(F32)
    alpha[::7] = 0
    n1, ninf = float(oracle.norm_l1(alpha)), float(np.abs(alpha).max())
    phi = 0.5 * n1 / ninf
    acc = np.zeros(d); sq = 0.0; nnz = 0
    for rnd in range(N):
        r = oracle.sparsify(alpha, phi, 11, rnd, 0)
        acc += r["beta"]; sq += float((r["beta"].astype(np.float64) ** 2).sum()); nnz += int(r["Z"].sum())
    p = r["m"] / 65536.0
    supp = p > 0
    var = np.zeros(d); var[supp] = alpha[supp].astype(np.float64) ** 2 * (1 / p[supp] - 1)
    assert np.all(np.abs(acc / N - alpha) <= 5.5 * np.sqrt(var / N) + 1e-7 * np.abs(alpha))
    second = float((alpha[supp].astype(np.float64) ** 2 / p[supp]).sum())
    assert abs(sq / N - second) < 0.05 * second
    assert second <= n1 ** 2 / phi * (1 + 1e-5)                          # rounding p up can only lower it
    assert second >= n1 ** 2 / phi * 0.97
    assert abs(nnz / N - p.sum()) < 5 * math.sqrt(p.sum() / N) + 1e-9
    assert abs(p.sum() - phi) < 0.02 * phi + d / 65536


def test_sparse_quantise_keys_rounding_by_coordinate():
    g = np.random.default_rng(8)
    d, b = 2000, 4
    L = 7
    alpha = g.standard_normal(d).astype(F32)
    r = oracle.sparsify(alpha, 0.1 * d, 5, 9, 3)
    codes, delta, rc = oracle.quantize_survivors(r["beta"], r["Z"], b, 5, 9, 3)
    Z = r["Z"].astype(bool)
    assert rc == 0 and not codes[~Z].any() and np.abs(codes).max() <= L
    nrm = np.abs(r["beta"][Z]).max()
    assert delta == nrm / F32(L)
    inv = oracle.scale_inv(nrm, b)
    for i in np.nonzero(Z)[0][:50]:
        assert codes[i] == oracle.q_code(r["beta"][i], inv, b, oracle.u15(5, 9, 3, oracle.STREAM_GRAD, int(i)))
    empty = oracle.sparsify(np.zeros(10, F32), 3.0, 1, 1, 1)
    assert not empty["Z"].any() and empty["phi_eff"] == 0


# ---------------------------------------------------------------------------------------------------
# prox
# ---------------------------------------------------------------------------------------------------
def _prox_brute(v, eta, l1, l2, lo, hi):
    """argmin_y h(y) + (y-v)^2/(2 eta) over [lo,hi] by grid + golden section (the definition itself)."""
    a = max(lo, -50.0); b = min(hi, 50.0)
    obj = lambda y: l1 * abs(y) + 0.5 * l2 * y * y + (y - v) ** 2 / (2 * eta)
    ys = np.linspace(a, b, 200001)
    j = int(np.argmin(l1 * np.abs(ys) + 0.5 * l2 * ys * ys + (ys - v) ** 2 / (2 * eta)))
    cands = [ys[j], 0.0 if a <= 0.0 <= b else ys[j]]
    l, r = ys[max(j - 1, 0)], ys[min(j + 1, ys.size - 1)]
    phi = (math.sqrt(5) - 1) / 2
    for _ in range(100):
        m1, m2 = r - phi * (r - l), l + phi * (r - l)
        if obj(m1) < obj(m2): r = m2
        else: l = m1
    cands.append(0.5 * (l + r))
    return min(cands, key=obj)


def test_prox_against_brute_force_minimisation():
    g = np.random.default_rng(9)
    for _ in range(60):
        v = float(g.standard_normal() * 3); eta = float(10 ** g.uniform(-2, 0.5))
        l1 = float(g.choice([0.0, 10 ** g.uniform(-3, 0.3)])); l2 = float(g.choice([0.0, 10 ** g.uniform(-3, 0.5)]))
        lo, hi = (-np.inf, np.inf) if g.random() < 0.4 else (-float(g.random() * 2), float(g.random() * 2))
        got = float(oracle.prox(v, eta, l1, l2, lo, hi))
        assert abs(got - _prox_brute(v, eta, l1, l2, lo, hi)) < 2e-6 * max(1.0, abs(v))


def test_prox_special_cases():
    inf = np.inf
    for v in (-2.5, -0.01, 0.0, 0.3, 7.0):
        assert oracle.prox(v, 0.1, 0, 0, -inf, inf) == F32(v)                                   # h = 0: identity
        st = np.sign(F32(v)) * max(F32(abs(F32(v))) - F32(0.1) * F32(0.5), F32(0))
        assert oracle.prox(v, 0.1, 0.5, 0, -inf, inf) == F32(st)                                 # soft-threshold
        assert oracle.prox(v, 0.1, 0, 2.0, -inf, inf) == F32(v) / (F32(1) + F32(0.1) * F32(2.0))  # ridge shrink
        assert oracle.prox(v, 0.1, 0, 0, -1.0, 0.25) == F32(min(max(v, -1.0), 0.25))             # projection on the box
