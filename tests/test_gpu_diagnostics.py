"""The attention-stealing diagnostics (Eq. (9), Section 6) computed through the C ABI against the oracle:
the quantized cached mass from the oracle's Algorithm 1, the unquantized one from a textbook FP64 softmax."""
import numpy as np
import pytest
import torch

from oracle import kvq_oracle as O
from paper_2605_26266_b200 import inputs
from tests import kvq_testlib as T

pytestmark = pytest.mark.gpu


def test_cached_mass_shift_and_output_error_match_the_oracle():
    from paper_2605_26266_b200 import binding as B, diagnostics as D
    d, sigma = 128, T.sigma_of(128)
    w = inputs.Workload("diag", 700, 1, 2, d, 150, 0, 2, 32, 3, k_outliers=4, k_outlier_scale=8.0)
    g = B.Cache(1, 2, d, 2, 32, 384)
    o = O.Cache(1, 2, d, 2, 32, 384)
    ks, vs, n = [], [], 0
    for c in range(2):
        _, k, v = inputs.make_chunk(w, c)
        ks.append(k); vs.append(v)
        B.kvq_quantize_append(g, T.to_dev(k), T.to_dev(v))
        n = O.quantize_append(o, n, k, v)
    kb, vb = np.concatenate(ks, axis=2), np.concatenate(vs, axis=2)
    q, kc, vc = inputs.make_chunk(w, 5)
    res = D.attention_stealing(g, T.to_dev(kb), T.to_dev(vb), T.to_dev(q), T.to_dev(kc), T.to_dev(vc), sigma)
    torch.cuda.synchronize()
    # unquantized cached mass and output: plain FP64 softmax over [cached ; current] BF16 keys
    f = O.bf16_bits_to_f64
    s = sigma * np.einsum("bhmd,bhnd->bhmn", f(q), np.concatenate([f(kb), f(kc)], axis=2))
    p = np.exp(s - s.max(-1, keepdims=True)); p /= p.sum(-1, keepdims=True)
    p_s_ref = p[..., :n].sum(-1)
    out_ref = np.einsum("bhmn,bhnd->bhmd", p, np.concatenate([f(vb), f(vc)], axis=2))
    assert np.abs(res["p_s_ref"].cpu().numpy() - p_s_ref).max() < 1e-2
    for name, corr in (("uncorrected", False), ("corrected", True)):
        want = O.attn_corrected(o, 0, n, q, kc, vc, sigma, correction=corr)
        dps = want["cached_mass"].reshape(p_s_ref.shape) - p_s_ref
        assert np.abs(res["dps_" + name].cpu().numpy() - dps).max() < 2e-2, name
        mse = ((want["out"].reshape(out_ref.shape) - out_ref) ** 2).mean(-1)
        got = res["mse_" + name].cpu().numpy()            # BF16 outputs on both sides: compare the means
        assert abs(got.mean() - mse.mean()) < 1e-4 + 0.1 * mse.mean(), (name, got.mean(), mse.mean())
    # the paper's observation on its models holds on this synthetic heavy-tailed chunk too: quantization moves mass
    # onto the cached keys, the correction moves most of it back
    s_ = D.summarize(res)
    assert s_["dps_uncorrected"] > 0 and abs(s_["dps_corrected"]) < s_["dps_uncorrected"]
