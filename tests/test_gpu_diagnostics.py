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


@pytest.mark.parametrize("d,bits,group,rotate,m,chunk_tokens,n_cur", [
    (128, 2, 32, True, 150, 97, 150), (128, 2, 128, True, 33, 200, 77), (128, 4, 64, True, 70, 130, 70),
    (64, 2, 64, True, 61, 100, 40), (128, 2, 64, False, 45, 111, 45)])
def test_weight_jsd_matches_the_oracle(d, bits, group, rotate, m, chunk_tokens, n_cur):
    """kvq_attn_weight_jsd against the oracle's row-by-row definition: ragged row and key counts, every format,
    rotation with random signs and without, a window that does not start at the cache's first token."""
    from paper_2605_26266_b200 import binding as B
    sigma = T.sigma_of(d)
    w = inputs.Workload("jsd", 710 + d + bits + group, 2, 2, d, m, 0, bits, group, 5, k_outliers=3, k_outlier_scale=6.0)
    signs = np.random.default_rng(group).choice([-1, 1], size=d).astype(np.int8) if rotate else None
    g = B.Cache(2, 2, d, bits, group, 768, rotate_k=rotate, signs=signs)
    o = O.Cache(2, 2, d, bits, group, 768, rotate_k=rotate, signs=signs)
    ks, n = [], 0
    for c in range(3):
        _, k, v = inputs.make_chunk(w, c, tokens=chunk_tokens)
        ks.append(k)
        B.kvq_quantize_append(g, T.to_dev(k), T.to_dev(v))
        n = O.quantize_append(o, n, k, v)
    kb = np.concatenate(ks, axis=2)
    q, _, _ = inputs.make_chunk(w, 7)
    _, kc, _ = inputs.make_chunk(w, 8, tokens=n_cur)
    begin = 16
    for corr, flags in ((True, B.KVQ_CORRECTION_ON), (False, B.KVQ_CORRECTION_OFF)):
        got = B.kvq_attn_weight_jsd(g, T.to_dev(q), T.to_dev(kc), T.to_dev(np.ascontiguousarray(kb[:, :, begin:n])), sigma,
                                    flags, cache_begin=begin, cache_len=n - begin)
        torch.cuda.synchronize()
        want = O.attn_weight_jsd(o, begin, n - begin, q, kc, kb[:, :, begin:n], sigma, correction=corr)
        got = got.cpu().numpy().astype(np.float64).reshape(want.shape)
        assert (want > 0).all() and (want < np.log(2)).all()
        assert np.abs(got - want).max() <= 2e-5 + 2e-3 * want.max(), (corr, np.abs(got - want).max(), want.max())
    # an empty cache: both weight vectors are the same softmax over the current keys
    z = B.kvq_attn_weight_jsd(g, T.to_dev(q), T.to_dev(kc), None, sigma, B.KVQ_CORRECTION_ON, cache_len=0)
    assert float(z.abs().max().item()) < 1e-6


def test_jsd_in_the_diagnostics_summary():
    """On a heavy-tailed synthetic chunk the corrected weights are closer to the unquantized ones than the
    uncorrected (the trend the paper reports for INT2), as seen through the diagnostics helper."""
    from paper_2605_26266_b200 import binding as B, diagnostics as D
    w = inputs.Workload("jsd_sum", 720, 1, 2, 128, 300, 0, 2, 128, 0, k_outliers=4, k_outlier_scale=8.0)
    g = B.Cache(1, 2, 128, 2, 128, 1280)
    ks, vs = [], []
    for c in range(4):
        _, k, v = inputs.make_chunk(w, c)
        ks.append(T.to_dev(k)); vs.append(T.to_dev(v))
        B.kvq_quantize_append(g, ks[-1], vs[-1])
    q, kc, vc = (T.to_dev(a) for a in inputs.make_chunk(w, 9))
    res = D.summarize(D.attention_stealing(g, torch.cat(ks, 2), torch.cat(vs, 2), q, kc, vc, T.sigma_of(128), exact=False))
    assert 0 < res["jsd_corrected"] < res["jsd_uncorrected"] < np.log(2)
