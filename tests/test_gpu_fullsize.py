"""Parity at the benchmark's full size (d = 2^27, M = 8, b = 4, b_x = 8) in the launch sequence bench.py times.

The oracle cannot redo 2^30 coordinates in seconds, so outputs are checked on samples it can compute one by
one (random coordinates, the first and last groups of every message) plus properties that hold at any size
(scales equal the exact maxima, padding is zero, ||x||_inf equals the maximum of the new model)."""
import numpy as np
import pytest

import oracle
from paper_1805_10111_b200 import synth

pytestmark = pytest.mark.gpu
F32 = np.float32


def _codes_at(packed_row, idx, b):
    per = 8 // b
    field = (packed_row[idx // per].astype(np.int32) >> ((idx % per) * b)) & ((1 << b) - 1)
    return np.where(field >= (1 << (b - 1)), field - (1 << b), field).astype(np.int32)


@pytest.mark.parametrize("log2d,b", [(27, 4), (24, 2), (24, 8)])
def test_codec_round_at_bench_size_on_samples(log2d, b):
    import torch
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    import paper_1805_10111_b200 as dq
    d, M, bx, seed, rnd, eta, l1 = 1 << log2d, 8, 8, 1805, 1003, 0.1, 1e-6
    g = synth.rng(500 + log2d)
    hv = torch.empty((M, d), dtype=torch.float32).pin_memory()
    v = hv.numpy()
    for w in range(M):
        g.standard_normal(d, dtype=np.float32, out=v[w])
        v[w][g.integers(0, d, d // 1000)] *= F32(100.0)
    x0 = synth.normal_vector(d, 6); gf = synth.normal_vector(d, 7)
    cfg = dq.make_config(d, M, b=b, bx=bx, seed=seed, lambda1=l1)
    rc, ctx = dq.dq_create(cfg); assert rc == 0
    dv = hv.cuda()
    st = dq.State(x0); st.g_full.copy_(torch.from_numpy(gf).cuda())
    msgs = dq.Msgs(cfg); ninf = torch.zeros(M, device="cuda")
    nbx = dq.dq_packed_bytes(d, bx)
    codes_x = torch.zeros(nbx, dtype=torch.uint8, device="cuda"); delta_x = torch.zeros(1, device="cuda")
    # the same four calls as one bench step
    assert dq.dq_norm_inf(ctx, dv, M, ninf) == 0
    assert dq.dq_quantize_sparsify_pack(ctx, dv, ninf, rnd, msgs) == 0
    assert dq.dq_master_unpack_aggregate_prox(ctx, msgs, st, eta) == 0
    assert dq.dq_quantize_model(ctx, st.x, st.norm_x, rnd, codes_x, delta_x) == 0
    assert dq.dq_poll_status(ctx) == (0, 0)

    L = 2 ** (b - 1) - 1
    nrm = np.abs(v).max(axis=1)
    assert np.array_equal(ninf.cpu().numpy(), nrm)                                   # exact maxima
    delta = msgs.scale.cpu().numpy()
    assert np.array_equal(delta, nrm / F32(L))                                       # delta = ||v||_inf / (2^(b-1)-1)
    packed = msgs.codes.cpu().numpy()
    assert packed.shape[1] == d * b // 8
    sample = np.unique(np.concatenate([g.integers(0, d, 1500), np.arange(0, 64), np.arange(d - 64, d),
                                       np.argmax(np.abs(v), axis=1)]))
    raw = np.zeros((M, sample.size), np.int32)
    for w in range(M):
        inv = oracle.scale_inv(nrm[w], b)
        raw[w] = _codes_at(packed[w], sample, b)
        want = [oracle.q_code(v[w, i], inv, b, oracle.u15(seed, rnd, w, oracle.STREAM_GRAD, int(i))) for i in sample]
        assert np.array_equal(raw[w], np.array(want, np.int32)), w
        # any-size property: every code within the grid, the maximum coordinate at its end
        assert np.abs(raw[w]).max() <= L
    # master step on the sampled coordinates, from the GPU's own codes: bit-exact
    x_gpu = st.x.cpu().numpy()
    xs = x0[sample].copy()
    oracle.master_step(raw, delta, gf[sample], xs, eta, l1=l1)
    assert np.array_equal(x_gpu[sample], xs)
    assert st.norm_x.item() == np.abs(x_gpu).max()
    # model quantisation of the new x
    nx = np.abs(x_gpu).max()
    assert delta_x.item() == nx / F32(127)
    invx = oracle.scale_inv(nx, bx)
    cx = _codes_at(codes_x.cpu().numpy(), sample, bx)
    want = [oracle.q_code(x_gpu[i], invx, bx, oracle.u15(seed, rnd, oracle.MASTER, oracle.STREAM_MODEL, int(i))) for i in sample]
    assert np.array_equal(cx, np.array(want, np.int32))
    dq.dq_destroy(ctx)


@pytest.mark.parametrize("log2d,workers", [(24, range(8)), (27, (5,))])
def test_sparsified_messages_at_bench_size(log2d, workers):
    """The sparsified stage as bench.py --sparsify 1 launches it (M = 8, b = 4, phi = 0.01 d): the norm pass, the mask
    pass that stages the survivors, and their placement, for both containers.  The oracle redoes whole vectors: all
    eight at d = 2^24, one at d = 2^27 (about ten seconds each); the other messages are checked through properties
    that hold at any size."""
    import torch
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    import paper_1805_10111_b200 as dq
    d, M, b, seed, rnd = 1 << log2d, 8, 4, 1805, 1004
    phi = 0.01 * d
    g = synth.rng(700 + log2d)
    hv = torch.empty((M, d), dtype=torch.float32).pin_memory()
    v = hv.numpy()
    for w in range(M):
        g.standard_normal(d, dtype=np.float32, out=v[w])
        v[w][g.integers(0, d, d // 1000)] *= F32(100.0)
    dv = hv.cuda()
    want = {}
    for w in workers:
        r = oracle.sparsify(v[w], phi, seed, rnd, w)
        codes, delta, rc = oracle.quantize_survivors(r["beta"], r["Z"], b, seed, rnd, w)
        assert rc == 0 and r["status"] == 0
        want[w] = (np.nonzero(r["Z"])[0], codes, delta)
    L = 2 ** (b - 1) - 1
    for fmt in (dq.DQ_MSG_DENSE, dq.DQ_MSG_SPARSE):
        cfg = dq.make_config(d, M, b=b, bx=8, seed=seed, sparsify=1, phi=phi, msg_format=fmt, sparse_cap=d // 64)
        rc, ctx = dq.dq_create(cfg); assert rc == 0
        msgs = dq.Msgs(cfg, cap=d // 64); ninf = torch.zeros(M, device="cuda")
        assert dq.dq_norm_inf(ctx, dv, M, ninf) == 0
        assert dq.dq_quantize_sparsify_pack(ctx, dv, ninf, rnd, msgs) == 0
        assert dq.dq_poll_status(ctx) == (0, 0)
        scale = msgs.scale.cpu().numpy()
        for w in range(M):
            row = msgs.codes[w].cpu().numpy()
            if fmt == dq.DQ_MSG_DENSE:
                lo, hi = row & 0x0F, row >> 4                                        # two codes per byte at b = 4
                nz = int(np.count_nonzero(lo) + np.count_nonzero(hi))
                assert 0 < nz <= 0.004 * d                                           # realised density about 0.2 %
                assert max(int(np.abs(_codes_at(row, np.flatnonzero(lo) * 2, b)).max()), 1) <= L
            else:
                n = int(msgs.nnz[w].item())
                idx = msgs.idx[w, :n].cpu().numpy().astype(np.int64)
                assert np.all(np.diff(idx) > 0) and idx[-1] < d                      # ascending, in range
                assert not row[(n * b + 7) // 8:].any()                              # nothing behind the list
            if w in want:
                pos, codes, delta = want[w]
                assert scale[w] == delta
                if fmt == dq.DQ_MSG_DENSE:
                    assert np.array_equal(row, oracle.pack(codes, b, msgs.stride))
                else:
                    assert n == pos.size and np.array_equal(idx, pos)
                    assert np.array_equal(row, oracle.pack(codes[pos], b, msgs.stride))
        dq.dq_destroy(ctx)
        del msgs
