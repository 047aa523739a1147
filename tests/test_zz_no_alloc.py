"""kvq_attn_corrected_static_scratch: the entry point for callers that may not allocate device memory.

It must give what kvq_attn_corrected gives (same kernel; the partial results of split units sit in the
library's built-in scratch buffer instead of a caller workspace), on consecutive calls that reuse that one
buffer, and it must refuse split problems larger than the buffer was sized for.  This file sorts last so that
a run that stops at the first failure has already run every other test.
"""
import numpy as np
import pytest
import torch

from paper_2605_26266_b200 import inputs
from tests import kvq_testlib as T

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2605_26266_b200 import binding
    return binding


def _problem(B, heads, m, chunks, chunk_tokens, n_cur, seed):
    w = inputs.Workload("noalloc", 400 + seed, 1, heads, 128, m, 0, 2, 64, seed, k_outliers=2, k_outlier_scale=4.0)
    cap = (chunks * chunk_tokens + 127) // 128 * 128
    g = B.Cache(1, heads, 128, 2, 64, cap)
    for c in range(chunks):
        _, k, v = inputs.make_chunk(w, c, tokens=chunk_tokens)
        B.kvq_quantize_append(g, T.to_dev(k), T.to_dev(v))
    q, _, _ = inputs.make_chunk(w, 90, tokens=m)
    _, kc, vc = inputs.make_chunk(w, 91, tokens=n_cur)
    return g, T.to_dev(q), T.to_dev(kc), T.to_dev(vc)


def _both(B, g, q, kc, vc, flags):
    """Runs the workspace entry point and the static-scratch one; returns (out, lse, mass) of each."""
    res = []
    for fn in (B.kvq_attn_corrected, B.kvq_attn_corrected_static_scratch):
        lse = torch.zeros(q.shape[:3], dtype=torch.float32, device="cuda")
        mass = torch.zeros_like(lse)
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        out = torch.empty_like(q)                      # outputs are the caller's: nothing is allocated by the call
        fn(g, q, kc, vc, T.sigma_of(128), flags, out=out, lse=lse, cached_mass=mass, status_word=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        res.append((T.from_dev_bf16(out), lse.cpu().numpy(), mass.cpu().numpy()))
    return res


def test_matches_workspace_entry_point_on_two_calls_in_a_row(B):
    # two different split problems back to back: the second call finds the first call's partials in the buffer
    p1 = _problem(B, heads=2, m=200, chunks=6, chunk_tokens=1000, n_cur=200, seed=1)    # 2 units, 49 tiles each
    p2 = _problem(B, heads=3, m=300, chunks=3, chunk_tokens=777, n_cur=150, seed=2)     # 6 units, ragged tiles
    assert B.kvq_attn_workspace_bytes(p1[0], p1[0].length, 200, 200, B.KVQ_CORRECTION_ON) > 0   # really the split path
    for g, q, kc, vc in (p1, p2, p1):
        for flags in (B.KVQ_CORRECTION_ON, B.KVQ_CORRECTION_OFF):
            (o_ws, lse_ws, mass_ws), (o_st, lse_st, mass_st) = _both(B, g, q, kc, vc, flags)
            T.assert_attn_close(o_st, o_ws, "static scratch vs workspace")
            assert np.abs(lse_st - lse_ws).max() < 2e-2
            assert np.abs(mass_st - mass_ws).max() < 1e-2


def test_against_the_oracle_with_the_cta_count_capped(B):
    """2 units of about 158 key tiles: the planner wants about 79 CTAs, the built-in buffer holds the partial
    results of 32, so this entry point runs a different split (longer ranges per CTA, both slots of a CTA in
    use) from kvq_attn_corrected.  Checked against the workspace entry point and, independently, the oracle."""
    from oracle import kvq_oracle as O
    w = inputs.Workload("noalloc_cap", 470, 1, 2, 128, 200, 0, 2, 64, 7, k_outliers=2, k_outlier_scale=4.0)
    chunks, tokens = 5, 4000
    g = B.Cache(1, 2, 128, 2, 64, 20096)
    o = O.Cache(1, 2, 128, 2, 64, 20096)
    n = 0
    for c in range(chunks):
        _, k, v = inputs.make_chunk(w, c, tokens=tokens)
        B.kvq_quantize_append(g, T.to_dev(k), T.to_dev(v))
        n = O.quantize_append(o, n, k, v)
    q, kc, vc = inputs.make_chunk(w, 90)
    qd, kd, vd = T.to_dev(q), T.to_dev(kc), T.to_dev(vc)
    # the workspace entry would use far more CTAs than the static buffer has slots for
    assert B.kvq_attn_workspace_bytes(g, n, 200, 200, B.KVQ_CORRECTION_ON) > 2 * 200 * 272 + 2 * 32 * 68608
    for corr, flags in ((True, B.KVQ_CORRECTION_ON), (False, B.KVQ_CORRECTION_OFF)):
        (o_ws, lse_ws, mass_ws), (o_st, lse_st, mass_st) = _both(B, g, qd, kd, vd, flags)
        T.assert_attn_close(o_st, o_ws, "static scratch vs workspace")
        want = O.attn_corrected(o, 0, n, q, kc, vc, T.sigma_of(128), correction=corr)
        T.assert_attn_close(o_st, want["out"], "static scratch vs oracle")
        assert np.abs(lse_st - want["lse"]).max() < 2e-2
        assert np.abs(mass_st - want["cached_mass"]).max() < 1e-2


def test_unsplit_problem_uses_only_the_query_area_and_is_identical(B):
    g, q, kc, vc = _problem(B, heads=80, m=100, chunks=2, chunk_tokens=300, n_cur=256, seed=3)   # 80 units: one CTA each
    # no partial-result slots: the workspace is just the rotated queries (256 + 16 bytes per query row)
    assert B.kvq_attn_workspace_bytes(g, g.length, 100, 256, B.KVQ_CORRECTION_ON) == 80 * 100 * 272
    (o_ws, _, _), (o_st, _, _) = _both(B, g, q, kc, vc, B.KVQ_CORRECTION_ON)
    assert np.array_equal(o_ws, o_st)


def test_sizes_beyond_the_buffer_are_refused(B):
    g, q, kc, vc = _problem(B, heads=40, m=100, chunks=2, chunk_tokens=2000, n_cur=100, seed=4)   # 40 units of 33 tiles: split
    out = torch.empty_like(q)
    with pytest.raises(B.KvqError) as e:
        B.kvq_attn_corrected_static_scratch(g, q, kc, vc, T.sigma_of(128), B.KVQ_CORRECTION_ON, out=out)
    assert e.value.status == B.KVQ_ERR_WORKSPACE
    # more than 8192 query rows over a non-empty cache: the rotated queries do not fit
    g2, q2, k2, v2 = _problem(B, heads=40, m=512, chunks=2, chunk_tokens=300, n_cur=256, seed=5)
    with pytest.raises(B.KvqError) as e:
        B.kvq_attn_corrected_static_scratch(g2, q2, k2, v2, T.sigma_of(128), B.KVQ_CORRECTION_ON, out=torch.empty_like(q2))
    assert e.value.status == B.KVQ_ERR_WORKSPACE
    # head_dim 64 has no tcgen05 kernel, kernel-selection flags are not accepted
    w = inputs.Workload("noalloc64", 499, 1, 2, 64, 100, 0, 2, 64, 0)
    g64 = B.Cache(1, 2, 64, 2, 64, 128)
    q64, k64, v64 = (T.to_dev(a) for a in inputs.make_chunk(w, 0))
    with pytest.raises(B.KvqError) as e:
        B.kvq_attn_corrected_static_scratch(g64, q64, k64, v64, 0.125, B.KVQ_CORRECTION_ON, cache_len=0)
    assert e.value.status == B.KVQ_ERR_UNSUPPORTED
    with pytest.raises(B.KvqError) as e:
        B.kvq_attn_corrected_static_scratch(g, q, kc, vc, T.sigma_of(128), B.KVQ_CORRECTION_ON | B.KVQ_KERNEL_TCGEN05, out=out)
    assert e.value.status == B.KVQ_ERR_INVALID_ARG
