"""Per-channel keys (App. E): the append must leave bit-identical bytes in the per-channel layout, and attention
(warp-level kernel, one bias scalar per query row and token block) must match the oracle."""
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


@pytest.mark.parametrize("d,bits,group,ring", [(128, 2, 32, False), (128, 4, 64, True), (128, 2, 128, False), (64, 2, 32, True)])
def test_per_channel_keys(B, d, bits, group, ring):
    w = inputs.Workload("pc", 950 + d + bits + group, 2, 3, d, 2 * group, 0, bits, group, 9, k_outliers=2, k_outlier_scale=6.0)
    cap = 1024
    g = B.Cache(2, 3, d, bits, group, cap, k_per_channel=True, ring=ring)
    o = O.Cache(2, 3, d, bits, group, cap, k_per_channel=True, ring=ring)
    pos = cap - 128 if ring else 0                                  # a ring cache: the appended blocks wrap around the end
    first = pos
    for c in range(3):
        nt = (c + 1) * group                                   # whole blocks: g, 2g, 3g tokens
        if nt > 256:
            nt = 256
        _, k, v = inputs.make_chunk(w, c, tokens=nt)
        B.kvq_quantize_append(g, T.to_dev(k), T.to_dev(v), cache_len=pos)
        O.quantize_append(o, pos, k, v)
        pos += nt
    T.assert_cache_equal(T.gpu_cache_arrays(g, cap), o, cap)
    n = pos - first
    q, _, _ = inputs.make_chunk(w, 7, tokens=100)
    _, kc, vc = inputs.make_chunk(w, 8, tokens=70)
    qd, kd, vd = T.to_dev(q), T.to_dev(kc), T.to_dev(vc)
    sigma = T.sigma_of(d)
    for begin, length in ((first, n), (first + group, n - group - 5)):
        for corr in (True, False):
            want = O.attn_corrected(o, begin, length, q, kc, vc, sigma, correction=corr)
            mass = torch.zeros(q.shape[:3], dtype=torch.float32, device="cuda")
            out = B.kvq_attn_corrected(g, qd, kd, vd, sigma, B.KVQ_CORRECTION_ON if corr else B.KVQ_CORRECTION_OFF,
                                       cache_begin=begin, cache_len=length, cached_mass=mass)
            torch.cuda.synchronize()
            T.assert_attn_close(T.from_dev_bf16(out).reshape(want["out"].shape), want["out"], f"window {begin}+{length} corr={corr}")
            assert np.abs(mass.cpu().numpy().reshape(want["cached_mass"].shape) - want["cached_mass"]).max() < 1e-2
    on = O.attn_corrected(o, first, n, q, kc, vc, sigma, correction=True)["cached_mass"]
    off = O.attn_corrected(o, first, n, q, kc, vc, sigma, correction=False)["cached_mass"]
    assert np.abs(on - off).max() > 1e-3                       # the correction is visible on this input
    # rules of the layout
    with pytest.raises(B.KvqError) as e:
        B.kvq_quantize_append(g, qd[:, :, :group - 1], qd[:, :, :group - 1], cache_len=0)
    assert e.value.status == B.KVQ_ERR_ALIGNMENT
    with pytest.raises(B.KvqError) as e:
        B.kvq_attn_corrected(g, qd, kd, vd, sigma, B.KVQ_CORRECTION_ON, cache_begin=first + 16, cache_len=16)   # inside a block
    assert e.value.status == B.KVQ_ERR_ALIGNMENT
    if d == 128:
        with pytest.raises(B.KvqError) as e:
            B.kvq_attn_corrected(g, qd, kd, vd, sigma, B.KVQ_CORRECTION_ON | B.KVQ_KERNEL_TCGEN05, cache_begin=first, cache_len=n)
        assert e.value.status == B.KVQ_ERR_UNSUPPORTED
