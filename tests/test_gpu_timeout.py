"""The bounded-wait path of the tcgen05 kernel, exercised in the one permitted way: the wait budget is cut to a
few cycles, so that a wait which is merely not complete at its first poll gives up.  Nothing is left waiting:
every role of the CTA leaves at its next wait, the kernel returns by itself and reports a site code in the
caller's status word; the context stays usable, and the same call with the default budget is right again."""
import numpy as np
import pytest
import torch

from oracle import kvq_oracle as O
from paper_2605_26266_b200 import inputs
from tests import kvq_testlib as T

pytestmark = pytest.mark.gpu

SITE_CODES = {100, 101, 102, 103, 104, 201, 203, 204, 205, 207, 209, 301, 302, 303, 401, 402, 404, 406}


@pytest.mark.parametrize("kernel", ["KVQ_KERNEL_TCGEN05", "KVQ_KERNEL_TCGEN05_PAIR"])
def test_expired_wait_sets_the_status_word_and_the_kernel_returns(kernel):
    from paper_2605_26266_b200 import binding as B
    w = inputs.Workload("timeout", 91, 1, 1, 128, 256, 2, 2, 128, 3)     # one unit of 256 rows: one CTA, 6 key tiles
    g = B.Cache(w.batch, w.heads, w.head_dim, w.bits, w.group, w.capacity)
    o = O.Cache(w.batch, w.heads, w.head_dim, w.bits, w.group, w.capacity)
    n = 0
    for c in range(w.cached_chunks):
        _, k, v = inputs.make_chunk(w, c)
        B.kvq_quantize_append(g, T.to_dev(k), T.to_dev(v))
        n = O.quantize_append(o, n, k, v)
    q, k, v = inputs.make_chunk(w, w.cached_chunks)
    qd, kd, vd = T.to_dev(q), T.to_dev(k), T.to_dev(v)
    sigma = T.sigma_of(w.head_dim)
    flags = B.KVQ_CORRECTION_ON | getattr(B, kernel)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    try:
        B.kvq_set_wait_budget_cycles(2)
        B.kvq_attn_corrected(g, qd, kd, vd, sigma, flags, cache_len=n, status_word=status)
        torch.cuda.synchronize()                       # the kernel came back by itself
    finally:
        B.kvq_set_wait_budget_cycles(0)
    word = int(status.item())
    assert word in SITE_CODES, word
    assert B.kvq_status_word_result(word) == B.KVQ_ERR_TIMEOUT
    assert B.kvq_status_word_result(0) == B.KVQ_OK
    # default budget again: the same call on the same context gives the right answer
    status.zero_()
    out = B.kvq_attn_corrected(g, qd, kd, vd, sigma, flags, cache_len=n, status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    want = O.attn_corrected(o, 0, n, q, k, v, sigma, correction=True)
    T.assert_attn_close(T.from_dev_bf16(out), want["out"], "after a timed-out call")

