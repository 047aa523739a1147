"""GPU parity: kvq_quantize_append against the oracle, bit for bit (codes, scale bytes,
zero-point bits), through the C ABI."""
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


def _append_both(B, w, chunks, rotate=True, signs=None, tokens=None, units=None):
    """Appends `chunks` chunks on the GPU (all heads) and in the oracle (all heads, or `units`)."""
    cap = w.capacity
    g = B.Cache(w.batch, w.heads, w.head_dim, w.bits, w.group, cap, rotate_k=rotate, signs=signs)
    if units is None:
        o = O.Cache(w.batch, w.heads, w.head_dim, w.bits, w.group, cap, rotate_k=rotate, signs=signs)
    else:
        o = O.Cache(1, len(units), w.head_dim, w.bits, w.group, cap, rotate_k=rotate, signs=signs)
    n = 0
    for c in range(chunks):
        _, k, v = inputs.make_chunk(w, c, tokens=tokens)
        B.kvq_quantize_append(g, T.to_dev(k), T.to_dev(v))
        if units is not None:
            k = np.stack([k[b, h] for (b, h) in units])[None]
            v = np.stack([v[b, h] for (b, h) in units])[None]
        n = O.quantize_append(o, n, k, v)
    torch.cuda.synchronize()
    assert g.length == n
    return g, o, n


@pytest.mark.parametrize("name", ["tiny", "sweep_int4", "sweep_int2"])
def test_full_config_bit_exact(B, name):
    w = inputs.WORKLOADS[name]
    g, o, n = _append_both(B, w, w.cached_chunks)
    T.assert_cache_equal(T.gpu_cache_arrays(g, n), o, n)
    # nothing past the appended tokens was written
    v = g.views()
    assert not v["k_codes"][:, :, n:].any() and not v["v_zero"][:, :, n:].any()


@pytest.mark.parametrize("name,chunks,units", [
    ("dit", 2, [(0, 0), (0, 11), (0, 23)]),
    ("long", 2, [(0, 5), (0, 23)]),
    ("pipeline", 3, [(0, 0), (1, 17), (1, 31)]),
])
def test_large_config_head_subset_bit_exact(B, name, chunks, units):
    w = inputs.WORKLOADS[name]
    g, o, n = _append_both(B, w, chunks, units=units)
    T.assert_cache_equal(T.gpu_cache_arrays(g, n), o, n, units=units)


@pytest.mark.parametrize("d,bits,group", [(64, 2, 32), (64, 2, 64), (64, 4, 32), (64, 4, 64),
                                          (128, 2, 32), (128, 2, 64), (128, 2, 128),
                                          (128, 4, 32), (128, 4, 64), (128, 4, 128)])
@pytest.mark.parametrize("rotate", [True, False])
def test_all_formats_ragged_chunks(B, d, bits, group, rotate):
    # chunks of 1, 37 and 200 tokens: ragged tiles, unaligned append offsets
    w = inputs.Workload("fmt", 90 + d + bits + group, 2, 3, d, 64, 0, bits, group, 7,
                        k_dist="student_t3", k_outliers=3, k_outlier_scale=10.0)
    cap = 256
    signs = np.random.default_rng(d + bits).choice([-1, 1], size=d).astype(np.int8) if rotate else None
    g = B.Cache(w.batch, w.heads, d, bits, group, cap, rotate_k=rotate, signs=signs)
    o = O.Cache(w.batch, w.heads, d, bits, group, cap, rotate_k=rotate, signs=signs)
    n = 0
    for c, tok in enumerate((1, 37, 200)):
        _, k, v = inputs.make_chunk(w, c, tokens=tok)
        B.kvq_quantize_append(g, T.to_dev(k), T.to_dev(v))
        n = O.quantize_append(o, n, k, v)
    T.assert_cache_equal(T.gpu_cache_arrays(g, n), o, n)
    # the test aid expands codes in canonical channel order
    for which, name in ((0, "k_codes"), (1, "v_codes")):
        got = B.kvq_unpack_codes(g, which, 0, n).cpu().numpy()
        assert np.array_equal(got, O.unpack_codes(getattr(o, name)[:, :, :n], bits))


def test_degenerate_groups_and_strided_input(B):
    d, bits, group = 128, 2, 32
    r = np.random.default_rng(0)
    x = r.standard_normal((1, 2, 40, d)).astype(np.float32)
    x[0, 0, 0] = 0.0                    # all-zero vector
    x[0, 0, 1] = 1.0                    # constant vector
    x[0, 0, 2, :32] = -2.5              # one constant group
    x[0, 1, 3] *= 1e4                   # step saturates E4M3 (448)
    x[0, 1, 4] *= 1e-6                  # step in the subnormal range / floored
    x[0, 1, 5] += 100.0                 # large zero-point
    x[0, 1, 6] *= 1e25                  # magnitudes beyond 2^60: the kernel's IEEE-division path
    x[0, 1, 7] *= 1e-25                 # magnitudes far below the step floor
    x[0, 1, 8, ::3] *= 1e-30            # tiny elements inside a normal range
    x[0, 1, 9] = 1e6 + 1e-3 * x[0, 1, 9]   # quotients x/step beyond 2^21 (zero-point far outside BF16's integers)
    x[0, 1, 10, :32] = 3e4              # a constant group whose quotient is large
    kb = inputs.f32_to_bf16_bits(x)
    vb = inputs.f32_to_bf16_bits(x[..., ::-1].copy())
    for rotate in (False, True):
        g = B.Cache(1, 2, d, bits, group, 128, rotate_k=rotate)
        o = O.Cache(1, 2, d, bits, group, 128, rotate_k=rotate)
        # strided inputs: tokens interleaved in a [B, n, H, d] buffer
        kd = T.to_dev(kb).permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
        vd = T.to_dev(vb).permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
        assert not kd.is_contiguous()
        B.kvq_quantize_append(g, kd, vd)
        O.quantize_append(o, 0, kb, vb)
        T.assert_cache_equal(T.gpu_cache_arrays(g, 40), o, 40)


def test_append_errors(B):
    g = B.Cache(1, 1, 128, 2, 128, 128)
    k = torch.zeros(1, 1, 100, 128, dtype=torch.bfloat16, device="cuda")
    B.kvq_quantize_append(g, k, k)
    with pytest.raises(B.KvqError) as e:
        B.kvq_quantize_append(g, k, k)
    assert e.value.status == B.KVQ_ERR_CAPACITY
    assert g.length == 100
