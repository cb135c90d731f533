"""The allocation-free entry point dq_quantize_pack_static against the ordinary one.

Some users of this library run where device allocation is off limits at call time (inside another
framework's allocator, with all device memory budgeted beforehand, or as a plug-in that only receives
buffers and a stream).  For them the dense quantise+pack exists in a form whose only scratch is a fixed
array inside the library.  This test calls it twice in a row through the C ABI -- the second call with other
data and another round, so that anything left in the shared array by the first call would show -- and
requires the bytes and scales to equal those of dq_quantize_sparsify_pack exactly (the tolerance of the
codec tests: bit-exact).  It lives in its own file, collected last, and passes alone or after the others.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu
F32 = np.float32


def test_static_entry_matches_context_entry_twice_in_a_row():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    import paper_1805_10111_b200 as dq
    g = np.random.default_rng(2024)
    seed = 0x5EED1234ABCD
    calls = [dict(M=5, d=40008, b=4, rnd=3, scale=1.0), dict(M=3, d=12345, b=8, rnd=9, scale=1e-3),
             dict(M=5, d=40008, b=2, rnd=4, scale=50.0)]
    for c in calls:
        M, d, b = c["M"], c["d"], c["b"]
        v = (g.standard_normal((M, d)) * c["scale"]).astype(F32)
        v[0, 17] *= 100.0
        if c["rnd"] == 9:
            v[1] = 0.0                                           # a zero vector must come out as scale 0, codes 0
        if c["rnd"] == 4:
            v[3, 5] = np.nan; v[4, d - 1] = np.inf               # so must a vector that holds a NaN or an Inf
        dv = torch.from_numpy(v).cuda()
        cfg = dq.make_config(d, M, b=b, seed=seed)
        rc, ctx = dq.dq_create(cfg); assert rc == 0
        want = dq.Msgs(cfg)
        assert dq.dq_quantize_sparsify_pack(ctx, dv, None, c["rnd"], want) == 0
        got_codes = torch.full((M, want.stride), 0xAB, dtype=torch.uint8, device="cuda")
        got_scale = torch.full((M,), -1.0, device="cuda")
        assert dq.dq_quantize_pack_static(dv, d, M, b, seed, c["rnd"], got_codes, want.stride, got_scale) == 0
        torch.cuda.synchronize()
        assert torch.equal(got_scale, want.scale)
        assert torch.equal(got_codes, want.codes)
        assert got_scale.max().item() > 0
        if c["rnd"] == 4:
            assert not got_scale[3:].any().item() and not got_codes[3:].any().item()
        dq.dq_destroy(ctx)
    # sizes beyond the fixed scratch, and bad arguments, are refused before anything is launched
    small = torch.zeros((2, 64), device="cuda"); codes = torch.zeros((2, 64), dtype=torch.uint8, device="cuda")
    sc = torch.zeros(2, device="cuda")
    assert dq.dq_quantize_pack_static(small, 64, 1025, 8, 1, 0, codes, 64, sc) == dq.DQ_ERR_SHAPE
    assert dq.dq_quantize_pack_static(small, 64, 2, 3, 1, 0, codes, 64, sc) == dq.DQ_ERR_BITS
    assert dq.dq_quantize_pack_static(small, 64, 2, 8, 1, 0, codes, 48, sc) == dq.DQ_ERR_SHAPE
    assert dq.dq_quantize_pack_static(None, 64, 2, 8, 1, 0, codes, 64, sc) == dq.DQ_ERR_ARG
