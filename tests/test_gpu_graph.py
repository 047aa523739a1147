"""The calls only enqueue work on the caller's stream (no allocation, no synchronisation), so a step
(attention over the cache, then quantize-append of the chunk) can be captured in a CUDA graph and replayed.
The replayed step must give the bytes of the eager one."""
import math

import numpy as np
import pytest
import torch

from paper_2605_26266_b200 import inputs
from tests import kvq_testlib as T

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("kernel", ["KVQ_KERNEL_TCGEN05", "KVQ_KERNEL_TCGEN05_PAIR"])
@pytest.mark.parametrize("heads,tokens", [(4, 600), (40, 1560)])   # units split over the SMs + merge / persistent rounds of whole units
def test_step_replayed_from_a_graph_equals_the_eager_step(heads, tokens, kernel):
    from paper_2605_26266_b200 import binding as B
    w = inputs.WORKLOADS["sweep_int2"]
    sigma = 1.0 / math.sqrt(w.head_dim)
    reps = -(-heads // w.heads)                  # more heads than the workload has: its heads again
    chunks = [[T.to_dev(np.ascontiguousarray(np.tile(a, (1, reps, 1, 1))[:, :heads]))
               for a in inputs.make_chunk(w, c, tokens=tokens)] for c in range(3)]

    def fresh():
        cache = B.Cache(1, heads, w.head_dim, w.bits, w.group, 5120)
        for q, k, v in chunks[:2]:
            B.kvq_quantize_append(cache, k, v)
        return cache

    q, k, v = chunks[2]
    flags = B.KVQ_CORRECTION_ON | getattr(B, kernel)

    eager = fresh()
    n = eager.length
    out_e = B.kvq_attn_corrected(eager, q, k, v, sigma, flags)
    B.kvq_quantize_append(eager, k, v)
    torch.cuda.synchronize()

    cache = fresh()
    out_g = torch.zeros_like(out_e)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    # the workspace is sized before the capture: nothing may allocate inside it
    need = B.kvq_attn_workspace_bytes(cache, n, tokens, tokens, flags)
    cache.workspace = torch.empty(max(need, 16), dtype=torch.uint8, device="cuda")
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            B.kvq_attn_corrected(cache, q, k, v, sigma, flags, cache_len=n, out=out_g, status_word=status)
            B.kvq_quantize_append(cache, k, v, cache_len=n)
    torch.cuda.synchronize()
    for _ in range(2):                       # a replay writes the same slots again
        out_g.zero_()
        graph.replay()
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.equal(out_g.view(torch.int16), out_e.view(torch.int16))
    for a, b in zip(cache.buffers, eager.buffers):
        assert torch.equal(a.view(torch.uint8), b.view(torch.uint8))
