"""Randomly drawn configurations of the round, GPU against oracle in lockstep.

The hand-picked cases of test_gpu_round.py fix one shape per feature; here the features are combined at random:
data format and shape (models below one group of eight coordinates up to beyond what the one-cluster kernel takes),
worker count (up to 20, beyond a cluster's 16 blocks), minibatch size from one row up, every model width of
Table 1, every gradient width, regulariser, sparsification with both message formats, momentum, the one-by-one
master, the searched model width, delayed workers, and the switches that pick between the kernel chains.  Each draw
runs two epochs of five rounds through the same checks as the hand-picked cases.  The draws are seeded: a failure
names its trial, which reproduces alone."""
import numpy as np
import pytest

import test_gpu_round as T
from paper_1805_10111_b200 import synth

pytestmark = pytest.mark.gpu
F32 = np.float32
dq = T.dq                      # the module-scoped fixture of the round tests


def draw_case(g):
    kind = str(g.choice(["dense", "csr", "bf16"]))
    if kind == "dense":
        d = int(g.choice([1, 5, 8, 37, 256, 300, 1000, 2049, 4096, 8191, 8192, 8193, 12000]))
        h = synth.dense_logistic(int(g.integers(40, 400)), d, int(g.integers(1, 1 << 20)))
    elif kind == "bf16":
        d = int(g.choice([8, 24, 301, 512, 1000, 4096, 8200]))
        h = synth.dense_bf16_logistic(int(g.integers(40, 400)), d, int(g.integers(1, 1 << 20)))
    else:
        d = int(g.choice([50, 777, 3001, 8192, 20011, 70001]))
        h = synth.sparse_logistic(int(g.integers(200, 3000)), d, float(g.choice([3.0, 20.0, 60.0])), 1.1, int(g.integers(1, 1 << 20)))
    M = int(g.choice([1, 2, 3, 4, 7, 8, 16, 17, 20]))
    B = min(int(g.choice([1, 3, 8, 16, 64, 70, 130])), h.n)
    kw = dict(M=M, B=B, bx=int(g.integers(2, 12)), b=int(g.choice([2, 4, 8])), seed=int(g.integers(1, 1 << 30)))
    r = g.random()
    if r < 0.3:
        kw["lambda1"] = float(g.choice([1e-6, 1e-4, 1e-2]))
    elif r < 0.5:
        kw["lambda2"] = float(g.choice([1e-5, 1e-3]))
    elif r < 0.8:
        kw.update(box_lo=-float(g.choice([0.5, 2.0])), box_hi=float(g.choice([0.5, 2.0])))
    else:
        kw.update(lambda1=1e-4, lambda2=1e-3, box_lo=-1.0, box_hi=1.0)
    if g.random() < 0.4:
        kw.update(sparsify=1, phi=float(g.choice([0.0, 0.0, 5.0, 50.0])), msg_format=int(g.integers(0, 2)))
    if g.random() < 0.3:
        kw["accelerated"] = 1
    if g.random() < 0.2:
        kw["sequential"] = 1
    if g.random() < 0.2:
        kw["no_fused"] = 1
    if g.random() < 0.15:
        kw["no_graph"] = 1
    if g.random() < 0.2:
        kw["mu"] = float(g.choice([1e-3, 0.3, 30.0, 1e4]))
    tau = int(g.choice([0, 0, 0, 1, 3]))
    if tau:
        kw["max_delay"] = tau
    return kind, h, kw, tau


@pytest.mark.parametrize("block", range(4))
def test_random_configurations(dq, block):
    per_block = 40
    for trial in range(block * per_block, (block + 1) * per_block):
        g = np.random.default_rng([1805, trial])
        kind, h, kw, tau = draw_case(g)
        acc = bool(kw.get("accelerated", 0))
        eta = 0.01 if kind == "bf16" else (0.05 if acc else 0.3)       # bf16 rows are not normalised
        try:
            ls = T.Lockstep(dq, h, synth.normal_vector(h.d, int(g.integers(1, 1000)), 0.05), **kw)
            rnd = 0
            for ep in range(2):
                theta = F32(2.0 / (ep + 3)) if acc else F32(0.0)
                ls.epoch(theta)
                for t in range(5):
                    delays = [int(v) for v in g.integers(0, tau + 1, kw["M"])] if tau else None
                    ls.round(rnd, eta / float(theta) if acc else eta, theta, delays=delays)
                    rnd += 1
            assert ls.far_flips == 0, ("far flips", ls.far_flips)
            ls.close()
        except AssertionError as e:
            raise AssertionError("trial %d %s n=%d d=%d %r: %r" % (trial, kind, h.n, h.d, kw, e)) from e


def test_random_configurations_every_chain_leaves_the_same_iterates(dq):
    """The same rounds by single calls (graph replay), by dq_rounds in random chunks, without graphs, and as separate
    kernels must leave the same bits in x (and y), the same ||x||_inf and the same bit counts.  Every gradient kernel
    sums in a fixed order (dense rows) or on an exact integer grid (CSR rows); where the one-cluster kernel or the
    one-pass dense gradient applies, the separate-kernel chain sums in another order and is left out."""
    import torch
    done = 0
    for trial in range(200):
        g = np.random.default_rng([1806, trial])
        kind, h, kw, tau = draw_case(g)
        for k in ("no_fused", "no_graph", "max_delay"):
            kw.pop(k, None)
        cluster = (not kw.get("sparsify") and not kw.get("sequential") and kw.get("mu", 0.0) == 0.0 and kw["bx"] in (2, 4, 8)
                   and h.d <= 8192 and kw["M"] <= 16)
        row_bytes = h.d * (2 if kind == "bf16" else 4)
        if kind != "csr" and kw["B"] >= 64 and row_bytes % 16 == 0 and row_bytes <= 8192:
            cluster = True          # the one-pass dense gradient sums a worker's rows per block, the two-kernel plan per warp: left out likewise
        acc = bool(kw.get("accelerated", 0))
        theta, eta = (0.5, 0.02 if kind == "bf16" else 0.05) if acc else (0.0, 0.01 if kind == "bf16" else 0.3)
        x0 = synth.normal_vector(h.d, int(g.integers(1, 1000)), 0.05)
        data = dq.Data(h)
        nr = int(g.integers(3, 25))
        chunks, left = [], nr
        while left > 0:
            chunks.append(int(g.integers(1, left + 1))); left -= chunks[-1]
        outs = {}
        for variant in ("single", "batched", "no_graph") + (() if cluster else ("no_fused",)):
            extra = {"no_graph": 1} if variant == "no_graph" else ({"no_fused": 1} if variant == "no_fused" else {})
            cfg = dq.make_config(h.d, kw["M"], **{k: v for k, v in kw.items() if k != "M"}, **extra)
            rc, ctx = dq.dq_create(cfg, data); assert rc == 0
            st = dq.State(x0, n=h.n, accelerated=acc)
            bits = torch.zeros(2, dtype=torch.int64, device="cuda")
            rnd = 0
            for epoch in range(2):
                assert dq.dq_epoch_begin(ctx, st, theta) == 0
                if variant == "batched":
                    for c in chunks:
                        assert dq.dq_rounds(ctx, st, rnd, c, eta, theta, bits[0:1], bits[1:2]) == 0
                        rnd += c
                else:
                    for t in range(nr):
                        assert dq.dq_round(ctx, st, rnd, eta, theta, bits[0:1], bits[1:2]) == 0
                        rnd += 1
            assert dq.dq_poll_status(ctx) == (0, 0), (trial, variant)
            outs[variant] = (st.x.cpu().numpy().copy(), st.norm_x.item(), bits.cpu().numpy().copy(),
                             st.y.cpu().numpy().copy() if acc else None)
            dq.dq_destroy(ctx)
        ref = outs["single"]
        for variant, o in outs.items():
            where = (trial, variant, kind, h.d, kw, chunks)
            assert np.array_equal(ref[0], o[0]) and ref[1] == o[1], where
            assert np.array_equal(ref[2], o[2]), where
            if acc:
                assert np.array_equal(ref[3], o[3]), where
        done += 1
    assert done >= 100
