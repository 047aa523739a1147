"""Repeated launches on the same inputs give the same bytes: nothing on the path depends on the order in which
CTAs, warps or copies happen to run (split units are merged in a fixed order, no atomics touch the data).  A missing
fence or a reused buffer released too early would show up here as a rare difference."""
import math

import numpy as np
import pytest
import torch

from paper_2605_26266_b200 import inputs
from tests import kvq_testlib as T

pytestmark = pytest.mark.gpu

CASES = [
    # workload, heads, tokens per chunk, cached chunks, launches
    ("sweep_int2", 16, 1560, 4, 60),     # every unit split over the SMs, ragged last query block
    ("dit", 24, 1560, 3, 40),            # a round of 148 whole units, then 20 units split; two groups per key
    ("pipeline", 6, 300, 5, 60),         # four groups per key, heavy-tailed keys, 12 units split
    ("sweep_int4", 3, 129, 2, 60),       # INT4, three whole units, one row past a tile in both directions
]


@pytest.mark.parametrize("kernel", ["KVQ_KERNEL_TCGEN05", "KVQ_KERNEL_TCGEN05_PAIR"])
@pytest.mark.parametrize("name,heads,tokens,chunks,launches", CASES, ids=[c[0] for c in CASES])
def test_repeated_launches_give_identical_bytes(name, heads, tokens, chunks, launches, kernel):
    from paper_2605_26266_b200 import binding as B
    w = inputs.WORKLOADS[name]
    sigma = 1.0 / math.sqrt(w.head_dim)
    cut = lambda a: T.to_dev(np.ascontiguousarray(a[:1, :heads]))
    cache = B.Cache(1, heads, w.head_dim, w.bits, w.group, 128 * (-(-tokens * (chunks + 1) // 128)))
    first_bytes = None
    for c in range(chunks):
        _, k, v = (cut(a) for a in inputs.make_chunk(w, c, tokens=tokens))
        B.kvq_quantize_append(cache, k, v)
    q, k, v = (cut(a) for a in inputs.make_chunk(w, chunks, tokens=tokens))
    n = cache.length
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ref_out = ref_lse = None
    for i in range(launches):
        out = torch.empty_like(q)
        lse = torch.empty(q.shape[:3], dtype=torch.float32, device="cuda")
        B.kvq_attn_corrected(cache, q, k, v, sigma, B.KVQ_CORRECTION_ON | getattr(B, kernel), cache_len=n,
                             out=out, lse=lse, status_word=status)
        B.kvq_quantize_append(cache, k, v, cache_len=n)          # the append of the step, every time at the same place
        if ref_out is None:
            ref_out, ref_lse = out, lse
            first_bytes = [b.clone() for b in cache.buffers]
        else:
            assert torch.equal(out.view(torch.int16), ref_out.view(torch.int16)), f"launch {i}"
            assert torch.equal(lse.view(torch.int32), ref_lse.view(torch.int32)), f"launch {i}"
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for a, b in zip(cache.buffers, first_bytes):
        assert torch.equal(a, b)
