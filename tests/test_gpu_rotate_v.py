"""KVQ_ROTATE_V: values stored rotated.  The append must leave bit-identical bytes (the oracle's FP32-step
rotation applied to V too), and attention — value pre-pass, kernel, output post-pass — must match the oracle,
which rotates the cached part of the output back in FP64."""
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


@pytest.mark.parametrize("d,bits,group,with_signs", [(128, 2, 32, True), (128, 4, 128, False), (64, 2, 64, True)])
def test_rotated_values_append_and_attention(B, d, bits, group, with_signs):
    w = inputs.Workload("rotv", 800 + d + bits, 2, 3, d, 150, 0, bits, group, 6, k_outliers=2, k_outlier_scale=5.0)
    signs = np.random.default_rng(d).choice([-1, 1], size=d).astype(np.int8) if with_signs else None
    g = B.Cache(2, 3, d, bits, group, 512, signs=signs, rotate_v=True)
    o = O.Cache(2, 3, d, bits, group, 512, signs=signs, rotate_v=True)
    n = 0
    for c in range(3):
        _, k, v = inputs.make_chunk(w, c, tokens=111)
        B.kvq_quantize_append(g, T.to_dev(k), T.to_dev(v))
        n = O.quantize_append(o, n, k, v)
    T.assert_cache_equal(T.gpu_cache_arrays(g, n), o, n)
    q, _, _ = inputs.make_chunk(w, 7, tokens=140)
    _, kc, vc = inputs.make_chunk(w, 8, tokens=77)
    qd, kd, vd = T.to_dev(q), T.to_dev(kc), T.to_dev(vc)
    sigma = T.sigma_of(d)
    want = O.attn_corrected(o, 0, n, q, kc, vc, sigma)
    plain = O.Cache(2, 3, d, bits, group, 512, signs=signs)          # same bytes read as if V were not rotated
    for name in ("k_codes", "v_codes", "k_scale", "v_scale", "k_zero", "v_zero"):
        getattr(plain, name)[:] = getattr(o, name)
    assert np.abs(O.attn_corrected(plain, 0, n, q, kc, vc, sigma)["out"] - want["out"]).max() > 0.1   # the flag matters
    kernels = [("mma_sync", B.KVQ_KERNEL_MMA_SYNC)] + ([("tcgen05", B.KVQ_KERNEL_TCGEN05), ("tcgen05_pair", B.KVQ_KERNEL_TCGEN05_PAIR)] if d == 128 else [])
    for kname, kflag in kernels:
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        mass = torch.zeros(q.shape[:3], dtype=torch.float32, device="cuda")
        flags = B.KVQ_CORRECTION_ON | kflag
        assert B.kvq_attn_workspace_bytes(g, n, 140, 77, flags) >= 2 * 3 * 77 * d * 2
        out = B.kvq_attn_corrected(g, qd, kd, vd, sigma, flags, cached_mass=mass, status_word=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        T.assert_attn_close(T.from_dev_bf16(out).reshape(want["out"].shape), want["out"], kname)
        assert np.abs(mass.cpu().numpy().reshape(want["cached_mass"].shape) - want["cached_mass"]).max() < 1e-2
        # an empty window needs no rotation and no workspace for it
        out0 = B.kvq_attn_corrected(g, qd, kd, vd, sigma, flags, cache_len=0)
        want0 = O.attn_corrected(o, 0, 0, q, kc, vc, sigma)
        T.assert_attn_close(T.from_dev_bf16(out0).reshape(want0["out"].shape), want0["out"], kname + " empty window")
    if d == 128:
        with pytest.raises(B.KvqError) as e:
            B.kvq_attn_corrected_static_scratch(g, qd, kd, vd, sigma, B.KVQ_CORRECTION_ON, out=torch.empty_like(qd))
        assert e.value.status == B.KVQ_ERR_UNSUPPORTED
