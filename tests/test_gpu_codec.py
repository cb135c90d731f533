"""GPU parity of the codec stages (quantise+pack, sparsify, master step, model quantise) against the
CPU oracle: bit-exact codes, masks, scales and iterates on the same seeded inputs, through the C ABI."""
import numpy as np
import pytest

import oracle
from paper_1805_10111_b200 import synth

pytestmark = pytest.mark.gpu
F32 = np.float32


@pytest.fixture(scope="module")
def dq():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    import paper_1805_10111_b200 as dq
    dq.lib()
    return dq


def _dev(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _vectors(M, d, seed, outliers=True):
    g = np.random.default_rng(seed)
    v = g.standard_normal((M, d)).astype(F32)
    if outliers and d > 10:
        for w in range(M):
            v[w, g.integers(0, d, max(1, d // 1000))] *= F32(100)
    return v


def _oracle_dense_msgs(v, b, seed, rnd, stride):
    M, d = v.shape
    codes = np.zeros((M, stride), np.uint8); delta = np.zeros(M, F32); raw = np.zeros((M, d), np.int32)
    for w in range(M):
        c, dl, rc = oracle.quantize(v[w], b, seed, rnd, w, oracle.STREAM_GRAD)
        assert rc == 0
        raw[w] = c; delta[w] = dl
        codes[w] = oracle.pack(c, b, stride)
    return codes, delta, raw


@pytest.mark.parametrize("b", [2, 4, 8])
@pytest.mark.parametrize("d", [1, 7, 8, 130, 1000, 4099, 20958, (1 << 16) + 24])
def test_quantize_pack_bit_exact(dq, b, d):
    M, seed, rnd = 3, 0xABCDEF0123, 17
    v = _vectors(M, d, d + b)
    cfg = dq.make_config(d, M, b=b, seed=seed)
    rc, ctx = dq.dq_create(cfg); assert rc == 0
    msgs = dq.Msgs(cfg)
    msgs.codes.fill_(0xEE)                                  # padding must be overwritten with zeros
    dv = _dev(v)
    assert dq.dq_quantize_sparsify_pack(ctx, dv, None, rnd, msgs) == 0
    assert dq.dq_poll_status(ctx) == (0, 0)
    want_codes, want_delta, _ = _oracle_dense_msgs(v, b, seed, rnd, msgs.stride)
    assert np.array_equal(msgs.scale.cpu().numpy(), want_delta)
    assert np.array_equal(msgs.codes.cpu().numpy(), want_codes)
    # the caller may supply the norms
    import torch
    ninf = _dev(np.abs(v).max(axis=1).astype(F32))
    msgs.codes.zero_()
    assert dq.dq_quantize_sparsify_pack(ctx, dv, ninf, rnd, msgs) == 0
    assert np.array_equal(msgs.codes.cpu().numpy(), want_codes)
    # another round draws other bits
    assert dq.dq_quantize_sparsify_pack(ctx, dv, None, rnd + 1, msgs) == 0
    if d >= 130:
        assert not np.array_equal(msgs.codes.cpu().numpy(), want_codes)
    dq.dq_destroy(ctx)


def test_quantize_misaligned_rows_and_large(dq):
    """Row length not a multiple of 8 (rows start off the 32-byte grid) and a multi-tile size with a tail."""
    for d, M, b in ((1000003, 2, 4), ((1 << 20) + 8 * 37, 8, 8)):
        v = _vectors(M, d, d)
        cfg = dq.make_config(d, M, b=b, seed=5)
        rc, ctx = dq.dq_create(cfg); assert rc == 0
        msgs = dq.Msgs(cfg)
        assert dq.dq_quantize_sparsify_pack(ctx, _dev(v), None, 3, msgs) == 0
        want_codes, want_delta, _ = _oracle_dense_msgs(v, b, 5, 3, msgs.stride)
        assert np.array_equal(msgs.scale.cpu().numpy(), want_delta)
        assert np.array_equal(msgs.codes.cpu().numpy(), want_codes)
        dq.dq_destroy(ctx)


@pytest.mark.parametrize("bx", [2, 3, 4, 5, 6, 7, 8, 9, 10, 11])
@pytest.mark.parametrize("d", [50021, 113, 8, 1])
def test_quantize_model_bit_exact(dq, bx, d):
    """Every model width of Table 1 (2..11 bits), including sizes whose last group of eight runs past the padded message."""
    import torch
    seed, rnd = 99, 1234567
    x = synth.normal_vector(d, 40, 0.3)
    cfg = dq.make_config(d, 2, bx=bx, seed=seed)
    rc, ctx = dq.dq_create(cfg); assert rc == 0
    nb = dq.dq_packed_bytes(d, bx)
    codes = torch.full((nb,), 0x55, dtype=torch.uint8, device="cuda"); delta = torch.zeros(1, device="cuda")
    assert dq.dq_quantize_model(ctx, _dev(x), None, rnd, codes, delta) == 0
    c, dl, _ = oracle.quantize(x, bx, seed, rnd, oracle.MASTER, oracle.STREAM_MODEL)
    assert delta.item() == dl
    assert np.array_equal(codes.cpu().numpy(), oracle.pack(c, bx, nb))
    dq.dq_destroy(ctx)


def test_zero_and_nonfinite_vectors(dq):
    d, M = 3000, 3
    v = _vectors(M, d, 1)
    v[1] = 0
    v[2, 77] = np.nan
    cfg = dq.make_config(d, M, b=4, seed=1)
    rc, ctx = dq.dq_create(cfg); assert rc == 0
    msgs = dq.Msgs(cfg)
    assert dq.dq_quantize_sparsify_pack(ctx, _dev(v), None, 0, msgs) == 0
    assert dq.dq_poll_status(ctx) == (0, dq.DQ_ERR_NONFINITE)
    assert dq.dq_poll_status(ctx) == (0, 0)                  # cleared after being read
    assert msgs.scale[1].item() == 0 and not msgs.codes[1].any().item()
    assert msgs.scale[2].item() == 0 and not msgs.codes[2].any().item()      # the NaN coordinate's own code is 0 too
    c, dl, _ = oracle.quantize(v[0], 4, 1, 0, 0, oracle.STREAM_GRAD)
    assert np.array_equal(msgs.codes[0].cpu().numpy(), oracle.pack(c, 4, msgs.stride))
    assert oracle.quantize(v[2], 4, 1, 0, 2, oracle.STREAM_GRAD)[2] == oracle.ERR_NONFINITE   # the oracle refuses the vector
    dq.dq_destroy(ctx)
    # the model quantiser for every width, NaN and Inf, and the merged quantiser + master kernel of a whole round
    import torch
    for bx, bad in ((8, np.inf), (2, np.nan), (5, -np.inf), (11, np.nan)):
        x = synth.normal_vector(d, 41, 0.3); x[d - 1] = bad
        cfg = dq.make_config(d, 2, bx=bx, seed=2)
        rc, ctx = dq.dq_create(cfg); assert rc == 0
        nb = dq.dq_packed_bytes(d, bx)
        codes = torch.full((nb,), 0x55, dtype=torch.uint8, device="cuda"); delta = torch.full((1,), 3.0, device="cuda")
        assert dq.dq_quantize_model(ctx, _dev(x), None, 5, codes, delta) == 0
        assert dq.dq_poll_status(ctx) == (0, dq.DQ_ERR_NONFINITE)
        assert delta.item() == 0 and not codes.any().item()
        dq.dq_destroy(ctx)


def test_argument_errors(dq):
    import torch
    assert dq.dq_create(dq.make_config(100, 2, b=3))[0] == dq.DQ_ERR_BITS
    assert dq.dq_create(dq.make_config(100, 2, bx=1))[0] == dq.DQ_ERR_BITS
    assert dq.dq_create(dq.make_config(0, 2))[0] == dq.DQ_ERR_ARG
    assert dq.dq_create(dq.make_config(100, 2, msg_format=dq.DQ_MSG_SPARSE))[0] == dq.DQ_ERR_ARG
    cfg = dq.make_config(1000, 2, b=8)
    rc, ctx = dq.dq_create(cfg); assert rc == 0
    msgs = dq.Msgs(cfg)
    v = torch.zeros((2, 1000), device="cuda")
    assert dq.dq_quantize_sparsify_pack(ctx, None, None, 0, msgs) == dq.DQ_ERR_ARG
    small = dq.Msgs(dq.make_config(500, 2, b=8))
    assert dq.dq_quantize_sparsify_pack(ctx, v, None, 0, small) == dq.DQ_ERR_SHAPE
    st = dq.State(np.zeros(1000, F32))
    assert dq.dq_master_unpack_aggregate_prox(ctx, msgs, st, -1.0) == dq.DQ_ERR_ARG
    assert dq.dq_round(ctx, st, 0, 0.1) == dq.DQ_ERR_ARG    # no training data in this context
    dq.dq_destroy(ctx)


def _run_master(dq, cfg, raw_codes, delta, gfull, x0, eta, theta=0.0, y0=None, xsnap=None, xsum0=None, msgs=None, ctx=None):
    st = dq.State(x0, accelerated=bool(cfg.accelerated))
    st.g_full.copy_(_dev(gfull))
    if cfg.accelerated:
        st.y.copy_(_dev(y0)); st.x_snap.copy_(_dev(xsnap)); st.x_sum.copy_(_dev(xsum0))
    assert dq.dq_master_unpack_aggregate_prox(ctx, msgs, st, eta, theta) == 0
    x = x0.copy(); y = None if y0 is None else y0.copy(); xs = None if xsum0 is None else xsum0.copy()
    nx = oracle.master_step(raw_codes, delta, gfull, x, eta, theta, bool(cfg.accelerated), y, xsnap, xs,
                            cfg.lambda1, cfg.lambda2, cfg.box_lo, cfg.box_hi)
    assert np.array_equal(st.x.cpu().numpy(), x)
    assert st.norm_x.item() == nx
    if cfg.accelerated:
        assert np.array_equal(st.y.cpu().numpy(), y) and np.array_equal(st.x_sum.cpu().numpy(), xs)
    return st


@pytest.mark.parametrize("b", [2, 4, 8])
@pytest.mark.parametrize("reg", ["l1", "l2", "box", "all", "none"])
def test_master_dense_bit_exact(dq, b, reg):
    d, M, seed = 10007, 5, 3
    kw = dict(l1=dict(lambda1=3e-2), l2=dict(lambda2=0.5), box=dict(box_lo=-0.4, box_hi=0.6),
              all=dict(lambda1=1e-2, lambda2=0.1, box_lo=-1.0, box_hi=1.0), none={})[reg]
    v = _vectors(M, d, 9, outliers=False)
    for acc in (0, 1):
        cfg = dq.make_config(d, M, b=b, seed=seed, accelerated=acc, **kw)
        rc, ctx = dq.dq_create(cfg); assert rc == 0
        msgs = dq.Msgs(cfg)
        assert dq.dq_quantize_sparsify_pack(ctx, _dev(v), None, 5, msgs) == 0
        _, delta, raw = _oracle_dense_msgs(v, b, seed, 5, msgs.stride)
        gfull = synth.normal_vector(d, 41); x0 = synth.normal_vector(d, 42)
        if acc:
            _run_master(dq, cfg, raw, delta, gfull, x0, 0.37, 0.25, y0=synth.normal_vector(d, 43),
                        xsnap=synth.normal_vector(d, 44), xsum0=synth.normal_vector(d, 45), msgs=msgs, ctx=ctx)
        else:
            _run_master(dq, cfg, raw, delta, gfull, x0, 0.37, msgs=msgs, ctx=ctx)
        dq.dq_destroy(ctx)


@pytest.mark.parametrize("b", [2, 4, 8])
@pytest.mark.parametrize("M", [1, 8, 19, 33])
def test_master_dense_worker_counts(dq, b, M):
    """Worker counts around the batches of eight that the master kernel keeps in flight (none, exact, remainder)."""
    d, seed = 4104, 17
    v = _vectors(M, d, 100 + M, outliers=False)
    cfg = dq.make_config(d, M, b=b, seed=seed, lambda1=1e-3, lambda2=0.01)
    rc, ctx = dq.dq_create(cfg); assert rc == 0
    msgs = dq.Msgs(cfg)
    assert dq.dq_quantize_sparsify_pack(ctx, _dev(v), None, 2, msgs) == 0
    _, delta, raw = _oracle_dense_msgs(v, b, seed, 2, msgs.stride)
    _run_master(dq, cfg, raw, delta, synth.normal_vector(d, 50), synth.normal_vector(d, 51), 0.21, msgs=msgs, ctx=ctx)
    dq.dq_destroy(ctx)


def _oracle_sparse(v, b, phi, seed, rnd):
    M, d = v.shape
    out = []
    for w in range(M):
        r = oracle.sparsify(v[w], phi, seed, rnd, w)
        codes, delta, rc = oracle.quantize_survivors(r["beta"], r["Z"], b, seed, rnd, w)
        assert rc == 0 and r["status"] == 0
        out.append(dict(Z=r["Z"].astype(bool), codes=codes, delta=delta))
    return out


def _check_sparsify(dq, v, b, phi, seed, rnd):
    """Both message formats of the sparsifier against the oracle, bit for bit, then the master step on the list."""
    import torch
    M, d = v.shape
    want = _oracle_sparse(v, b, phi, seed, rnd)
    # dense container
    cfg = dq.make_config(d, M, b=b, seed=seed, sparsify=1, phi=phi)
    rc, ctx = dq.dq_create(cfg); assert rc == 0
    msgs = dq.Msgs(cfg); msgs.codes.fill_(0x77)
    for _ in range(2):                                       # the second call meets the first call's scratch contents
        assert dq.dq_quantize_sparsify_pack(ctx, _dev(v), None, rnd, msgs) == 0
        assert dq.dq_poll_status(ctx) == (0, 0)
        for w in range(M):
            assert msgs.scale[w].item() == want[w]["delta"]
            assert np.array_equal(msgs.codes[w].cpu().numpy(), oracle.pack(want[w]["codes"], b, msgs.stride))
    dq.dq_destroy(ctx)
    # (position, value) list
    cfg = dq.make_config(d, M, b=b, seed=seed, sparsify=1, phi=phi, msg_format=dq.DQ_MSG_SPARSE)
    rc, ctx = dq.dq_create(cfg); assert rc == 0
    msgs = dq.Msgs(cfg); msgs.codes.fill_(0x77)
    for _ in range(2):
        assert dq.dq_quantize_sparsify_pack(ctx, _dev(v), None, rnd, msgs) == 0
        assert dq.dq_poll_status(ctx) == (0, 0)
        for w in range(M):
            pos = np.nonzero(want[w]["Z"])[0]
            assert msgs.nnz[w].item() == pos.size
            assert np.array_equal(msgs.idx[w, :pos.size].cpu().numpy().astype(np.int64), pos)     # mask, ascending
            assert msgs.scale[w].item() == want[w]["delta"]
            assert np.array_equal(msgs.codes[w].cpu().numpy(), oracle.pack(want[w]["codes"][pos], b, msgs.stride))
            out = torch.full((d,), 7.0, device="cuda")
            assert dq.dq_unpack(ctx, msgs, w, out) == 0
            assert np.array_equal(out.cpu().numpy(), want[w]["codes"].astype(F32) * want[w]["delta"])
    # master step on the sparse messages
    raw = np.stack([t["codes"] for t in want]); delta = np.array([t["delta"] for t in want], F32)
    _run_master(dq, cfg, raw, delta, synth.normal_vector(d, 46), synth.normal_vector(d, 47), 0.2, msgs=msgs, ctx=ctx)
    dq.dq_destroy(ctx)
    return want


@pytest.mark.parametrize("b", [2, 4, 8])
@pytest.mark.parametrize("d,phi_frac", [(5, 0.0), (2048, 0.01), (4099, 0.0), (70001, 0.01), ((1 << 17) + 8, 0.001)])
def test_sparsify_bit_exact_both_formats(dq, b, d, phi_frac):
    M, seed, rnd = 3, 777, 21
    v = _vectors(M, d, 5 * d + b)
    v[:, ::3] = 0                                            # exact zeros never survive
    _check_sparsify(dq, v, b, phi_frac * d, seed, rnd)


@pytest.mark.parametrize("b", [2, 4, 8])
@pytest.mark.parametrize("kind", ["dense", "near_limit", "half_empty"])
def test_sparsify_beyond_the_staging_limits(dq, b, kind):
    """Densities at which the survivors of a chunk (or of a whole vector) no longer fit the staging area, so that
    the chunk or the worker is redone from the vector: every chunk ("dense", about 20 % survive), a mixture of
    chunks on both sides of the limit ("near_limit", 6 % of +-1 entries), and the same behind an all-zero half."""
    M, seed, rnd = 3, 4242, 5
    d = (1 << 16) + 2048 + 8
    g = np.random.default_rng(600 + b)
    if kind == "dense":
        v = _vectors(M, d, 31 + b, outliers=False); phi = 0.0
    else:
        v = np.where(g.random((M, d)) < 0.5, F32(-1), F32(1)).astype(F32)
        phi = 0.06 * d
        if kind == "half_empty":
            v[:, : d // 2] = 0; phi = 0.03 * d
    want = _check_sparsify(dq, v, b, phi, seed, rnd)
    per_chunk = [np.add.reduceat(t["Z"].astype(np.int64), np.arange(0, d, 2048)) for t in want]
    if kind == "dense":
        assert min(c[:-1].min() for c in per_chunk) > 128
    else:
        assert any((c > 128).any() for c in per_chunk) and any(((c > 0) & (c <= 128)).any() for c in per_chunk)


@pytest.mark.parametrize("b", [2, 8])
@pytest.mark.parametrize("d", [1, 9, 4099])
def test_sparsify_subnormal_vectors(dq, b, d):
    """||alpha||_1 so small that phi / ||alpha||_1 overflows: every nonzero coordinate survives with p = 1, and a zero
    coordinate (0 * inf) must not turn into a survivor, in either message format."""
    g = np.random.default_rng(300 + d)
    v = (g.integers(-3, 4, (3, d)) * np.float64(1.4e-45)).astype(F32)          # a few units of the smallest subnormal, and zeros
    v[:, 0] = F32(4e-45)
    want = _check_sparsify(dq, v, b, 0.0, 4242, 6)
    for w in range(3):
        assert np.array_equal(want[w]["Z"], v[w] != 0)


def test_sparsify_survivor_overflow_is_reported(dq):
    """A survivor alpha_i / p_i beyond the fp32 range: the oracle reports a non-finite vector, and so must the library."""
    g = np.random.default_rng(301)
    d, M, b, seed, rnd = 2049, 2, 4, 77, 9
    v = (g.standard_normal((M, d)) * 1e-6).astype(F32)
    v[0, 5] = F32(3e38); v[1, 2000] = F32(-3e38)
    r = oracle.sparsify(v[0], 0.0, seed, rnd, 0)
    assert oracle.quantize_survivors(r["beta"], r["Z"], b, seed, rnd, 0)[2] == dq.DQ_ERR_NONFINITE
    for fmt in (dq.DQ_MSG_DENSE, dq.DQ_MSG_SPARSE):
        cfg = dq.make_config(d, M, b=b, seed=seed, sparsify=1, phi=0.0, msg_format=fmt)
        rc, ctx = dq.dq_create(cfg); assert rc == 0
        msgs = dq.Msgs(cfg)
        assert dq.dq_quantize_sparsify_pack(ctx, _dev(v), None, rnd, msgs) == 0
        assert dq.dq_poll_status(ctx) == (0, dq.DQ_ERR_NONFINITE)
        dq.dq_destroy(ctx)


def test_sparse_capacity_overflow_is_reported(dq):
    d, M = 30000, 2
    v = _vectors(M, d, 3, outliers=False)
    cfg = dq.make_config(d, M, b=4, seed=1, sparsify=1, phi=0.0, msg_format=dq.DQ_MSG_SPARSE)
    rc, ctx = dq.dq_create(cfg); assert rc == 0
    msgs = dq.Msgs(cfg, cap=64)
    assert dq.dq_quantize_sparsify_pack(ctx, _dev(v), None, 0, msgs) == 0
    assert dq.dq_poll_status(ctx) == (0, dq.DQ_ERR_CAPACITY)
    assert int(msgs.nnz.max().item()) == 64
    dq.dq_destroy(ctx)


def test_unpack_dense(dq):
    import torch
    d, M, b = 3001, 2, 4
    v = _vectors(M, d, 8)
    cfg = dq.make_config(d, M, b=b, seed=2)
    rc, ctx = dq.dq_create(cfg); assert rc == 0
    msgs = dq.Msgs(cfg)
    assert dq.dq_quantize_sparsify_pack(ctx, _dev(v), None, 9, msgs) == 0
    _, delta, raw = _oracle_dense_msgs(v, b, 2, 9, msgs.stride)
    out = torch.zeros(d, device="cuda")
    assert dq.dq_unpack(ctx, msgs, 1, out) == 0
    assert np.array_equal(out.cpu().numpy(), raw[1].astype(F32) * delta[1])
    dq.dq_destroy(ctx)


@pytest.mark.parametrize("sparsify", [0, 1])
def test_codec_round_chain(dq, sparsify):
    """quantise(+sparsify)+pack -> master step -> model quantisation, three rounds in a row, device and host entry."""
    import torch
    d, M, b, bx, seed, eta = 9001, 4, 4, 8, 31, 0.1
    v = _vectors(M, d, 12)
    gfull = synth.normal_vector(d, 48); x0 = synth.normal_vector(d, 49)
    cfg = dq.make_config(d, M, b=b, bx=bx, seed=seed, lambda1=1e-3, sparsify=sparsify, phi=0.05 * d)
    rc, ctx = dq.dq_create(cfg); assert rc == 0
    st = dq.State(x0); st.g_full.copy_(_dev(gfull))
    nb = dq.dq_packed_bytes(d, bx)
    codes_x = torch.zeros(nb, dtype=torch.uint8, device="cuda"); delta_x = torch.zeros(1, device="cuda")
    hv = torch.from_numpy(v).pin_memory()
    hcodes = torch.zeros(nb, dtype=torch.uint8).pin_memory(); hdelta = torch.zeros(1).pin_memory()
    assert dq.dq_codec_host_setup(ctx, x0, gfull) == 0
    x = x0.copy()
    for rnd in range(3):
        assert dq.dq_codec_round(ctx, _dev(v), st, rnd, eta, 0.0, codes_x, delta_x) == 0
        assert dq.dq_codec_round_host(ctx, hv, rnd, eta, hcodes, hdelta) == 0
        if sparsify:
            want = _oracle_sparse(v, b, cfg.phi, seed, rnd)
            raw = np.stack([t["codes"] for t in want]); delta = np.array([t["delta"] for t in want], F32)
        else:
            _, delta, raw = _oracle_dense_msgs(v, b, seed, rnd, dq.dq_packed_bytes(d, b))
        oracle.master_step(raw, delta, gfull, x, eta, l1=1e-3)
        assert np.array_equal(st.x.cpu().numpy(), x)
        c, dl, _ = oracle.quantize(x, bx, seed, rnd, oracle.MASTER, oracle.STREAM_MODEL)
        assert delta_x.item() == dl and np.array_equal(codes_x.cpu().numpy(), oracle.pack(c, bx, nb))
        assert hdelta.item() == dl and np.array_equal(hcodes.numpy(), oracle.pack(c, bx, nb))
    assert dq.dq_launch_count(ctx) > 0
    dq.dq_destroy(ctx)
