"""Attention-level diagnostics of Section 6 ("attention stealing"), on the GPU path.

The cached-mass shift of Eq. (9), dP_S = P^_S - P_S, the Jensen-Shannon divergence of the attention weights
and the error of the attention output against the unquantized cache, with the correction off and on.  Everything heavy is a call of the C ABI (through the
binding): the quantized numbers are kvq_attn_corrected's `cached_mass_out` and output; the unquantized
reference is the same kernel run with an empty cache window and the BF16 cached keys/values passed as part of
the "current chunk", where P_S follows from two log-sum-exps (all keys, current keys only).  What is left
here is elementwise arithmetic on [batch, heads, rows] tensors.

This is an analysis aid (it needs the BF16 copy of the cached chunks, which a deployment does not keep), not
part of the hot path.
"""
from __future__ import annotations

import torch

from . import binding as B


def attention_stealing(cache: "B.Cache", k_cached, v_cached, q, k_cur, v_cur, softmax_scale,
                       cache_begin: int = 0, cache_len: int | None = None, kernel_flag: int = B.KVQ_KERNEL_AUTO,
                       exact: bool = True):
    """k_cached, v_cached: the BF16 tensors [batch, heads, n, head_dim] whose quantized form is the window
    [cache_begin, cache_begin + n) of `cache`.  Returns a dict of per-row tensors [batch, heads, rows]:
    `p_s_ref`, `p_s_uncorrected`, `p_s_corrected`, `p_s_exact` (Taylor correction of Eq. (15), exact one of
    Eq. (12)), their differences to the reference `dps_*` (Eq. (9)), `mse_*` (mean squared error of the
    output rows against the unquantized cache) and `jsd_uncorrected`, `jsd_corrected` (divergence of the attention
    weights over all keys from those of the unquantized cache, kvq_attn_weight_jsd)."""
    n = k_cached.shape[2]
    n_cache = n if cache_len is None else cache_len
    assert n_cache == n, "the BF16 copy must cover exactly the attended window"
    shape = q.shape[:3]
    f32 = dict(dtype=torch.float32, device=q.device)

    # unquantized reference: one softmax over [cached ; current] keys, all of them BF16
    lse_all, lse_cur = torch.empty(shape, **f32), torch.empty(shape, **f32)
    k_all = torch.cat([k_cached, k_cur], dim=2)
    v_all = torch.cat([v_cached, v_cur], dim=2)
    out_ref = B.kvq_attn_corrected(cache, q, k_all, v_all, softmax_scale, B.KVQ_CORRECTION_OFF | kernel_flag,
                                   cache_len=0, lse=lse_all)
    B.kvq_attn_corrected(cache, q, k_cur, v_cur, softmax_scale, B.KVQ_CORRECTION_OFF | kernel_flag,
                         cache_len=0, lse=lse_cur)
    p_s_ref = 1.0 - torch.exp(lse_cur - lse_all)             # P_S = Z_S / (Z_S + Z_R) = 1 - Z_R / Z

    res = {"p_s_ref": p_s_ref}
    for name, flag in (("uncorrected", B.KVQ_CORRECTION_OFF), ("corrected", B.KVQ_CORRECTION_ON),
                       ("exact", B.KVQ_CORRECTION_EXACT)):
        if flag == B.KVQ_CORRECTION_EXACT and not exact:
            continue
        mass = torch.empty(shape, **f32)
        # the exact form of Eq. (12) exists in the warp-level kernel only
        out = B.kvq_attn_corrected(cache, q, k_cur, v_cur, softmax_scale,
                                   flag | (B.KVQ_KERNEL_AUTO if flag == B.KVQ_CORRECTION_EXACT else kernel_flag),
                                   cache_begin=cache_begin, cache_len=n_cache, cached_mass=mass)
        res["p_s_" + name] = mass
        res["dps_" + name] = mass - p_s_ref
        res["mse_" + name] = (out.float() - out_ref.float()).pow(2).mean(dim=-1)
        if flag != B.KVQ_CORRECTION_EXACT and not (cache.desc.flags & B.KVQ_K_PER_CHANNEL):
            res["jsd_" + name] = B.kvq_attn_weight_jsd(cache, q, k_cur, k_cached, softmax_scale, flag,
                                                       cache_begin=cache_begin, cache_len=n_cache)
    return res


def summarize(res) -> dict:
    """Means over all rows, as plain floats."""
    return {k: float(v.double().mean().item()) for k, v in res.items()}


def _main():
    """python -m paper_2605_26266_b200.diagnostics [workload]: the diagnostics on one synthetic workload."""
    import json
    import math
    import sys

    import numpy as np

    from . import inputs
    w = inputs.WORKLOADS[sys.argv[1] if len(sys.argv) > 1 else "sweep_int2"]
    dev = lambda a: torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
    cache = B.Cache(w.batch, w.heads, w.head_dim, w.bits, w.group, w.capacity)
    ks, vs = [], []
    for c in range(w.cached_chunks):
        _, k, v = inputs.make_chunk(w, c)
        ks.append(dev(k)); vs.append(dev(v))
        B.kvq_quantize_append(cache, ks[-1], vs[-1])
    q, k, v = (dev(a) for a in inputs.make_chunk(w, w.cached_chunks))
    res = attention_stealing(cache, torch.cat(ks, dim=2), torch.cat(vs, dim=2), q, k, v, 1.0 / math.sqrt(w.head_dim))
    torch.cuda.synchronize()
    print(json.dumps({"workload": w.name, **summarize(res)}))


if __name__ == "__main__":
    _main()
