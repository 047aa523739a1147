"""Ring cache (sliding window of the last cached chunks): the GPU path against the oracle's ring cache.

Appends that wrap around the end of the buffer (also inside one 32-token tile of the append kernel) must leave
bit-identical bytes in every slot, and attention over a window that wraps must match the oracle with both kernels.
"""
import numpy as np
import pytest
import torch

from oracle import kvq_oracle as O
from paper_2605_26266_b200 import inputs
from tests import kvq_testlib as T

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2605_26266_b200 import binding
    return binding


def _fill(B, w, cap, chunk_tokens):
    g = B.Cache(w.batch, w.heads, w.head_dim, w.bits, w.group, cap, ring=True)
    o = O.Cache(w.batch, w.heads, w.head_dim, w.bits, w.group, cap, ring=True)
    n = 0
    for c, nt in enumerate(chunk_tokens):
        _, k, v = inputs.make_chunk(w, c, tokens=nt)
        assert B.kvq_quantize_append(g, T.to_dev(k), T.to_dev(v), cache_len=n) == n + nt
        n = O.quantize_append(o, n, k, v)
    return g, o, n


@pytest.mark.parametrize("d,bits,group", [(128, 2, 32), (128, 4, 128), (64, 2, 64)])
def test_wrapping_appends_are_bit_exact(B, d, bits, group):
    w = inputs.Workload("ring", 500 + d + bits, 2, 3, d, 100, 0, bits, group, 1, k_outliers=1, k_outlier_scale=4.0)
    # 256 slots; chunk sizes chosen so that the wrap falls between tiles, inside a tile, and on a full-capacity append
    g, o, n = _fill(B, w, 256, [100, 100, 77, 256, 19, 130])
    assert n == 682
    T.assert_cache_equal(T.gpu_cache_arrays(g, 256), o, 256)
    # the canonical code order seen through kvq_unpack_codes, over a range that wraps
    got = B.kvq_unpack_codes(g, 0, 200, 120).cpu().numpy()
    want = O.unpack_codes(o.k_codes[:, :, o.slots(200, 120)], bits)
    assert np.array_equal(got, want)


@pytest.mark.parametrize("d", [128, 64])
def test_attention_over_a_wrapping_window(B, d):
    w = inputs.Workload("ringattn", 520 + d, 1, 3, d, 160, 0, 2, 32, 2, k_outliers=2, k_outlier_scale=5.0)
    g, o, n = _fill(B, w, 512, [160, 160, 160, 160, 90])        # 730 tokens through 512 slots
    q, kc, vc = inputs.make_chunk(w, 11)
    qd, kd, vd = T.to_dev(q), T.to_dev(kc), T.to_dev(vc)
    for begin, length in ((n - 512 + 6, 506), (400, 330), (512, 128), (n - 16, 16)):
        begin -= begin % 16                                         # window starts are multiples of 16 tokens
        length = min(length, n - begin)
        want = O.attn_corrected(o, begin, length, q, kc, vc, T.sigma_of(d))
        for kname, kflag in ([("mma_sync", B.KVQ_KERNEL_MMA_SYNC)] + ([("tcgen05", B.KVQ_KERNEL_TCGEN05), ("tcgen05_pair", B.KVQ_KERNEL_TCGEN05_PAIR)] if d == 128 else [])):
            status = torch.zeros(1, dtype=torch.int32, device="cuda")
            mass = torch.zeros(q.shape[:3], dtype=torch.float32, device="cuda")
            out = B.kvq_attn_corrected(g, qd, kd, vd, T.sigma_of(d), B.KVQ_CORRECTION_ON | kflag, cache_begin=begin,
                                       cache_len=length, cached_mass=mass, status_word=status)
            torch.cuda.synchronize()
            assert int(status.item()) == 0
            T.assert_attn_close(T.from_dev_bf16(out).reshape(want["out"].shape), want["out"], f"{kname} window {begin}+{length}")
            assert np.abs(mass.cpu().numpy().reshape(want["cached_mass"].shape) - want["cached_mass"]).max() < 1e-2
