"""Byte offsets beyond 2^31 and 2^32: a cache of 40 heads x 2^21 token slots holds 2.7 GB of key codes (and as
many of value codes), so the slabs of the last heads, and the end of every slab's token range, lie past what 32-bit
offset arithmetic reaches.  One chunk is appended at the very end of the capacity and attended there; the last
head's bytes and output must match the oracle's (which keeps the same tokens in a small cache of its own)."""
import numpy as np
import pytest
import torch

from oracle import kvq_oracle as O
from paper_2605_26266_b200 import inputs
from tests import kvq_testlib as T

pytestmark = pytest.mark.gpu


def test_append_and_attention_at_the_end_of_a_multi_gigabyte_cache():
    from paper_2605_26266_b200 import binding as B
    heads, cap, n_tok, m = 40, 1 << 21, 384, 200
    w = inputs.Workload("far", 901, 1, heads, 128, n_tok, 0, 2, 128, 1, k_outliers=2, k_outlier_scale=6.0)
    free, _ = torch.cuda.mem_get_info()
    if free < 12 << 30:
        pytest.skip("needs 12 GB of free device memory")
    g = B.Cache(1, heads, 128, 2, 128, cap)
    assert g.buffers[0].numel() > (1 << 31) and heads * cap * 32 > (1 << 31)
    _, k, v = inputs.make_chunk(w, 0)
    begin = cap - n_tok
    assert B.kvq_quantize_append(g, T.to_dev(k), T.to_dev(v), cache_len=begin) == cap

    units = [(0, 0), (0, 26), (0, heads - 1)]           # byte offsets 0, 1.7 GB (past 2^30), 2.6 GB (past 2^31)
    sel = lambda a: np.stack([a[b, h] for (b, h) in units])[None]
    o = O.Cache(1, len(units), 128, 2, 128, n_tok)
    O.quantize_append(o, 0, sel(k), sel(v))

    # bytes of the appended tokens, read back from the far end of each slab
    views = g.views()
    far = lambda name, b, h: views[name][b, h, begin:].cpu().numpy()
    for i, (b, h) in enumerate(units):
        assert np.array_equal(far("k_codes", b, h), o.k_codes[0, i])
        assert np.array_equal(far("v_codes", b, h), o.v_codes[0, i])
        assert np.array_equal(far("k_scale", b, h), o.k_scale[0, i])
        assert np.array_equal(far("v_scale", b, h), o.v_scale[0, i])
        assert np.array_equal(far("k_zero", b, h).view(np.uint16), o.k_zero[0, i])
        assert np.array_equal(far("v_zero", b, h).view(np.uint16), o.v_zero[0, i])
    got_codes = B.kvq_unpack_codes(g, 0, begin, n_tok).cpu().numpy()
    assert np.array_equal(sel(got_codes)[0], O.unpack_codes(o.k_codes[0], 2))

    q, kr, vr = inputs.make_chunk(w, 1, tokens=m)
    want = O.attn_corrected(o, 0, n_tok, sel(q), sel(kr), sel(vr), T.sigma_of(128))
    for kname, kflag in (("tcgen05", B.KVQ_KERNEL_TCGEN05), ("tcgen05_pair", B.KVQ_KERNEL_TCGEN05_PAIR), ("mma_sync", B.KVQ_KERNEL_MMA_SYNC)):
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        out = B.kvq_attn_corrected(g, T.to_dev(q), T.to_dev(kr), T.to_dev(vr), T.sigma_of(128),
                                   B.KVQ_CORRECTION_ON | kflag, cache_begin=begin, cache_len=n_tok, status_word=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        T.assert_attn_close(sel(T.from_dev_bf16(out))[0], want["out"], kname)
