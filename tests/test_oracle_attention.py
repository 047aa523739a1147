"""Pins for the oracle's correction and attention: closed forms, Monte-Carlo,
library softmax attention, invariants and a pure-Python brute force of
Algorithm 1 on tiny inputs."""
import math
import os

import numpy as np
import scipy.integrate
import scipy.linalg
import torch

from oracle import kvq_oracle as O
from paper_2605_26266_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _golden_mgf():
    rows = []
    for line in open(os.path.join(GOLDEN, "uniform_mgf.txt")):
        if line.startswith("#") or not line.strip():
            continue
        rows.append(tuple(float(t) for t in line.split()))
    return rows


def test_uniform_mgf_closed_form():
    # E[e^{s+delta}] = e^s * sinh(D/2)/(D/2) for delta ~ U(-D/2, D/2): quadrature vs exact bias
    for step, mgf, _ in _golden_mgf():
        num, _ = scipy.integrate.quad(lambda u: math.exp(u) / step, -step / 2, step / 2, epsabs=1e-13)
        got = math.exp(float(O.log_sinhc(np.array([step / 2]))[0]))
        assert abs(num - mgf) < 1e-9
        assert abs(got - mgf) < 1e-9
    # one channel, one key: exact_bias is log of that MGF with step = sigma*q*Delta
    q = np.zeros((1, 64)); q[0, 5] = 3.0
    ds = np.array([[0.75]])
    b = O.exact_bias(q, ds, 64, sigma=0.125)
    a = 0.125 * 3.0 * 0.75 / 2
    assert abs(b[0, 0] - math.log(math.sinh(a) / a)) < 1e-12


def test_log_sinhc_branches():
    a = np.array([1e-6, 5e-4, 1e-3, 0.01, 0.049, 0.051, 0.3, 2.0, 20.0])
    import mpmath
    mpmath.mp.dps = 40
    ref = np.array([float(mpmath.log(mpmath.sinh(mpmath.mpf(float(t))) / mpmath.mpf(float(t)))) for t in a])
    assert np.allclose(O.log_sinhc(a), ref, rtol=2e-12, atol=0)
    assert np.isfinite(O.log_sinhc(np.array([1000.0]))[0])          # no sinh overflow
    assert abs(O.log_sinhc(np.array([1000.0]))[0] - (1000 - math.log(2000))) < 1e-9
    assert np.array_equal(O.log_sinhc(-a), O.log_sinhc(a))


def test_taylor_vs_exact_residual():
    # log(sinh a / a) = a^2/6 - a^4/180 + ...; Taylor over-estimates
    for step, _, resid in _golden_mgf():
        a = step / 2
        exact = float(O.log_sinhc(np.array([a]))[0])
        taylor = a * a / 6
        assert taylor >= exact
        assert abs((exact - taylor) - resid) < abs(resid) * 0.25 + 1e-7
        assert abs(math.exp(exact - taylor) - 1 - resid) < abs(resid) * 0.25 + 1e-7


def test_taylor_bias_is_per_channel_formula():
    # Eq. (13) channel by channel equals Eq. (15) when channels of a group share the step
    r = np.random.default_rng(0)
    d, g = 128, 32
    q = r.standard_normal((3, d))
    ds = np.abs(r.standard_normal((5, d // g))) + 0.1
    nu = (q.reshape(3, d // g, g) ** 2).sum(-1)
    got = O.taylor_bias(nu, ds, sigma=1 / math.sqrt(d))
    for m in range(3):
        for i in range(5):
            want = sum(q[m, c] ** 2 * ds[i, c // g] ** 2 for c in range(d)) / (24 * d)
            assert abs(got[m, i] - want) < 1e-12
    assert np.all(got >= 0)
    # grows with the step; scales with sigma^2
    assert np.all(O.taylor_bias(nu, 2 * ds, 0.1) > O.taylor_bias(nu, ds, 0.1))
    assert np.allclose(O.taylor_bias(nu, ds, 0.2), 4 * O.taylor_bias(nu, ds, 0.1))
    # exact <= Taylor, and close for small steps
    ex = O.exact_bias(q, 0.05 * ds, g, 1 / math.sqrt(d))
    ta = O.taylor_bias(nu, 0.05 * ds, 1 / math.sqrt(d))
    assert np.all(ex <= ta) and np.allclose(ex, ta, rtol=1e-3)


def test_monte_carlo_unbiasedness():
    # uniform noise on keys: Var(delta) = (1/(12 d)) sum q_c^2 D_c^2 = 2 b_taylor (Eq. (7), (14));
    # E[e^{delta - b_exact}] = 1; E[e^{delta - b_taylor}] - 1 ~ -sum alpha^4/180
    r = np.random.default_rng(1)
    d, g = 64, 32
    sigma = 1 / math.sqrt(d)
    q = r.standard_normal((1, d)) * 2.0
    ds = np.array([[1.5, 0.7]])
    n = 400000
    eps = (r.random((n, d)) - 0.5) * np.repeat(ds, g, axis=-1)
    delta = sigma * (eps @ q[0])
    nu = (q.reshape(1, d // g, g) ** 2).sum(-1)
    bt = float(O.taylor_bias(nu, ds, sigma)[0, 0])
    be = float(O.exact_bias(q, ds, g, sigma)[0, 0])
    se = 3.5 * delta.std() / math.sqrt(n)
    assert abs(delta.mean()) < se
    assert abs(delta.var() - 2 * bt) < 0.01 * 2 * bt
    assert abs(np.exp(delta - be).mean() - 1) < 1.2 * se
    alpha = 0.5 * sigma * q[0] * np.repeat(ds, g, axis=-1)[0]
    resid = -(alpha ** 4).sum() / 180
    assert abs((np.exp(delta - bt).mean() - 1) - resid) < 1.2 * se + 0.3 * abs(resid)
    assert np.exp(delta).mean() > 1 + 0.5 * bt                       # Jensen bias without correction


def _sdpa(q, k, v, sigma, bias=None):
    t = lambda a: torch.tensor(a, dtype=torch.float64)[None, None]
    mask = None if bias is None else t(bias)
    return torch.nn.functional.scaled_dot_product_attention(t(q), t(k), t(v), attn_mask=mask, scale=sigma)[0, 0].numpy()


def _tiny_problem(seed, d, group, bits, n_s, n_r, m, rotate=True, lossless=False):
    r = np.random.default_rng(seed)
    bf = lambda a: inputs.f32_to_bf16_bits(a.astype(np.float32))
    q = bf(r.standard_normal((1, 1, m, d)))
    kc = bf(r.standard_normal((1, 1, n_r, d)))
    vc = bf(r.standard_normal((1, 1, n_r, d)))
    if lossless:
        L = 2 ** bits
        ks = bf(r.integers(0, L, (1, 1, n_s, d)) * 0.5 - 1.0)
        vs = bf(r.integers(0, L, (1, 1, n_s, d)) * 0.25 - 0.5)
        # make every group span the full range so the step is exactly 0.5 / 0.25
        ks[..., 0::group] = bf(np.array(-1.0)); ks[..., 1::group] = bf(np.array((L - 1) * 0.5 - 1.0))
        vs[..., 0::group] = bf(np.array(-0.5)); vs[..., 1::group] = bf(np.array((L - 1) * 0.25 - 0.5))
    else:
        ks = bf(r.standard_normal((1, 1, n_s, d)))
        vs = bf(r.standard_normal((1, 1, n_s, d)))
    cache = O.Cache(1, 1, d, bits, group, max(n_s, 1), rotate_k=rotate)
    if n_s:
        O.quantize_append(cache, 0, ks, vs)
    return q, kc, vc, ks, vs, cache


def test_empty_cache_is_textbook_attention():
    q, kc, vc, _, _, cache = _tiny_problem(0, 64, 64, 2, 0, 37, 11)
    for corr in (True, False):
        r = O.attn_corrected(cache, 0, 0, q, kc, vc, 0.125, correction=corr)
        want = _sdpa(O.bf16_bits_to_f64(q[0, 0]), O.bf16_bits_to_f64(kc[0, 0]), O.bf16_bits_to_f64(vc[0, 0]), 0.125)
        assert np.allclose(r["out"][0], want, atol=1e-12)
        assert np.allclose(r["cached_mass"], 0) and np.allclose(r["current_mass"], 1)
        s = 0.125 * O.bf16_bits_to_f64(q[0, 0]) @ O.bf16_bits_to_f64(kc[0, 0]).T
        assert np.allclose(r["lse"][0], torch.logsumexp(torch.tensor(s), dim=1).numpy(), atol=1e-12)


def test_lossless_cache_reduces_to_textbook_attention():
    # keys/values on the quantization grid and no rotation: the cache is exact, so
    # uncorrected attention equals softmax attention over concat(cache, current);
    # corrected attention equals the same with an additive mask -b on the cached block.
    for bits, group in ((2, 32), (4, 64), (2, 128)):
        d, n_s, n_r, m = 128, 19, 7, 5
        q, kc, vc, ks, vs, cache = _tiny_problem(1, d, group, bits, n_s, n_r, m, rotate=False, lossless=True)
        f = O.bf16_bits_to_f64
        kall = np.concatenate([f(ks[0, 0]), f(kc[0, 0])])
        vall = np.concatenate([f(vs[0, 0]), f(vc[0, 0])])
        sigma = 1 / math.sqrt(d)
        off = O.attn_corrected(cache, 0, n_s, q, kc, vc, sigma, correction=False)
        assert np.allclose(off["out"][0], _sdpa(f(q[0, 0]), kall, vall, sigma), atol=1e-12)
        on = O.attn_corrected(cache, 0, n_s, q, kc, vc, sigma, correction=True)
        kstep = 0.5
        qq = f(q[0, 0])
        b = np.array([[sum(qq[mm, c] ** 2 for c in range(d)) * kstep ** 2 / (24 * d)] * n_s for mm in range(m)])
        bias = np.concatenate([-b, np.zeros((m, n_r))], axis=1)
        assert np.allclose(on["out"][0], _sdpa(qq, kall, vall, sigma, bias), atol=1e-12)
        assert np.all(on["cached_mass"] < off["cached_mass"])


def test_mass_sums_to_one_and_correction_lowers_cached_mass():
    q, kc, vc, _, _, cache = _tiny_problem(2, 128, 32, 2, 50, 20, 9)
    on = O.attn_corrected(cache, 0, 50, q, kc, vc, 1 / math.sqrt(128), correction=True)
    off = O.attn_corrected(cache, 0, 50, q, kc, vc, 1 / math.sqrt(128), correction=False)
    for r in (on, off):
        assert np.allclose(r["cached_mass"] + r["current_mass"], 1.0, atol=1e-14)
        assert np.all(r["cached_mass"] > 0) and np.all(r["current_mass"] > 0)
    assert np.all(on["cached_mass"] < off["cached_mass"])                 # b >= 0
    assert not np.allclose(on["out"], off["out"], atol=1e-4)


def test_zero_step_sizes_make_correction_a_noop():
    q, kc, vc, _, _, cache = _tiny_problem(3, 64, 64, 2, 30, 10, 6)
    cache.k_scale[:] = 0                                                # hand-made step 0
    on = O.attn_corrected(cache, 0, 30, q, kc, vc, 0.125, correction=True)
    off = O.attn_corrected(cache, 0, 30, q, kc, vc, 0.125, correction=False)
    assert np.array_equal(on["out"], off["out"])
    assert np.all(np.isfinite(on["out"]))


def test_window_and_row_subset():
    q, kc, vc, _, _, cache = _tiny_problem(4, 64, 64, 2, 40, 10, 8)
    full = O.attn_corrected(cache, 0, 40, q, kc, vc, 0.125)
    rows = np.array([1, 6])
    sub = O.attn_corrected(cache, 0, 40, q, kc, vc, 0.125, rows=rows)
    assert np.array_equal(sub["out"][0], full["out"][0][rows])
    win = O.attn_corrected(cache, 8, 16, q, kc, vc, 0.125)
    c2 = O.Cache(1, 1, 64, 2, 64, 16)
    for name in ("k_codes", "v_codes", "k_scale", "v_scale", "k_zero", "v_zero"):
        getattr(c2, name)[:] = getattr(cache, name)[:, :, 8:24]
    assert np.array_equal(win["out"], O.attn_corrected(c2, 0, 16, q, kc, vc, 0.125)["out"])


def test_ring_cache_is_the_sliding_window():
    """A ring cache of C slots after appending T > C tokens, attended over its last W tokens, must give exactly
    what a linear cache holding all T tokens gives over the same window [T - W, T): the ring only changes where
    a token is stored (slot t mod C), and the newest tokens overwrite the oldest."""
    d, bits, group, C = 64, 2, 32, 48
    w = inputs.Workload("ring", 77, 1, 2, d, 20, 0, bits, group, 5)
    ring = O.Cache(1, 2, d, bits, group, C, ring=True)
    lin = O.Cache(1, 2, d, bits, group, 200)
    n = 0
    for c in range(7):                                   # 140 tokens through 48 slots: wraps twice, chunks straddle the end
        _, k, v = inputs.make_chunk(w, c)
        assert O.quantize_append(ring, n, k, v) == O.quantize_append(lin, n, k, v)
        n += 20
    q, kc, vc = inputs.make_chunk(w, 9)
    for W in (48, 40, 13, 0):
        a = O.attn_corrected(ring, n - W, W, q, kc, vc, 0.125)
        b = O.attn_corrected(lin, n - W, W, q, kc, vc, 0.125)
        for key in ("out", "lse", "cached_mass"):
            assert np.array_equal(a[key], b[key]), (W, key)
    # slot s holds the newest token t with t = s (mod C), by brute force over the stored bytes
    for s_ in range(C):
        t = max(t for t in range(n) if t % C == s_)
        assert np.array_equal(ring.k_codes[:, :, s_], lin.k_codes[:, :, t])
        assert np.array_equal(ring.v_zero[:, :, s_], lin.v_zero[:, :, t])
    # a window longer than the ring, or a linear cache run past its end, is refused
    for bad in (lambda: O.attn_corrected(ring, n - 49, 49, q, kc, vc, 0.125),
                lambda: O.quantize_append(lin, 190, *inputs.make_chunk(w, 0)[1:])):
        try:
            bad()
            raise AssertionError("accepted")
        except ValueError:
            pass


def test_rotated_values_equal_the_unrotated_path_on_prerotated_inputs():
    """rotate_v: quantizing R v and rotating the cached part of the output back must equal what the plain path
    gives when it is handed values rotated beforehand with a library Hadamard matrix (exact in FP64 here: the
    entries are small integers / 4, so R v needs no rounding) and its cached output is rotated back by hand."""
    d, bits, group = 64, 4, 32
    r = np.random.default_rng(5)
    signs = r.choice([-1, 1], size=d).astype(np.int8)
    Hn = scipy.linalg.hadamard(d) / math.sqrt(d)
    R = Hn * signs[None, :]                                   # R v = H (s * v)
    ints = lambda shape: r.integers(-8, 9, size=shape).astype(np.float32) * 0.25
    k, v, q, kc, vc = ints((1, 2, 40, d)), ints((1, 2, 40, d)), ints((1, 2, 9, d)), ints((1, 2, 12, d)), ints((1, 2, 12, d))
    b = inputs.f32_to_bf16_bits
    v_rot = np.einsum("ij,bhnj->bhni", R, v.astype(np.float64))
    assert np.array_equal(O.bf16_bits_to_f64(b(v_rot.astype(np.float32))), v_rot)       # representable: no rounding hidden here
    a = O.Cache(1, 2, d, bits, group, 128, signs=signs, rotate_v=True)
    p = O.Cache(1, 2, d, bits, group, 128, signs=signs)
    O.quantize_append(a, 0, b(k), b(v))
    O.quantize_append(p, 0, b(k), b(v_rot.astype(np.float32)))
    for name in ("v_codes", "v_scale", "v_zero", "k_codes"):
        assert np.array_equal(getattr(a, name), getattr(p, name)), name
    got = O.attn_corrected(a, 0, 40, b(q), b(kc), b(vc), 0.125)
    # plain path twice: cached part alone (current values zero) and current part alone, then R^-1 on the cached part
    zeros = np.zeros_like(vc)
    cached = O.attn_corrected(p, 0, 40, b(q), b(kc), b(zeros), 0.125)["out"]
    allv = O.attn_corrected(p, 0, 40, b(q), b(kc), b(vc), 0.125)["out"]
    want = (cached @ Hn) * signs[None, None, :] + (allv - cached)
    assert np.abs(got["out"] - want).max() < 1e-12
    assert np.array_equal(got["cached_mass"], O.attn_corrected(p, 0, 40, b(q), b(kc), b(vc), 0.125)["cached_mass"])


def _brute_force(q_bits, kc_bits, vc_bits, cache, n_s, sigma, correction):
    """Algorithm 1 with Python loops, its own dequantization from the stored bytes and
    an explicit Hadamard matrix.  Written separately from the oracle."""
    d, g, bits = cache.head_dim, cache.group, cache.bits
    G = d // g
    H = scipy.linalg.hadamard(d) / math.sqrt(d)
    tof = lambda u: float(np.array([int(u) << 16], dtype=np.uint32).view(np.float32)[0])

    def fp8(b):
        e, mnt = (b >> 3) & 15, b & 7
        return mnt / 8 * 2.0 ** -6 if e == 0 else (1 + mnt / 8) * 2.0 ** (e - 7)

    def deq(codes, scale, zero, i):
        out = []
        for c in range(d):
            byte = int(codes[i, c * bits // 8])
            code = (byte >> ((c * bits) % 8)) & (2 ** bits - 1)
            out.append((code - tof(zero[i, c // g])) * fp8(int(scale[i, c // g])))
        return out

    M, n_r = q_bits.shape[0], kc_bits.shape[0]
    outs = []
    for m in range(M):
        qv = [tof(u) for u in q_bits[m]]
        qr = [sum(H[a, c] * qv[c] for c in range(d)) for a in range(d)] if cache.rotate_k else qv
        nu = [sum(qr[c] ** 2 for c in range(j * g, (j + 1) * g)) for j in range(G)]
        scores, vals = [], []
        for i in range(n_s):
            kh = deq(cache.k_codes[0, 0], cache.k_scale[0, 0], cache.k_zero[0, 0], i)
            s = sum(a * b for a, b in zip(qr, kh)) / (1 / sigma)
            if correction:
                s -= sigma * sigma / 24 * sum(fp8(int(cache.k_scale[0, 0, i, j])) ** 2 * nu[j] for j in range(G))
            scores.append(s)
            vals.append(deq(cache.v_codes[0, 0], cache.v_scale[0, 0], cache.v_zero[0, 0], i))
        for r_ in range(n_r):
            scores.append(sigma * sum(a * tof(b) for a, b in zip(qv, kc_bits[r_])))
            vals.append([tof(u) for u in vc_bits[r_]])
        mx = max(scores)
        w = [math.exp(s - mx) for s in scores]
        z = sum(w)
        outs.append([sum(w[i] * vals[i][c] for i in range(len(w))) / z for c in range(d)])
    return np.array(outs)


def test_brute_force_tiny():
    for bits, group, d in ((2, 64, 64), (4, 32, 64), (2, 32, 128), (4, 128, 128), (2, 64, 128)):
        for rotate in (True, False):
            q, kc, vc, _, _, cache = _tiny_problem(10 + bits + group, d, group, bits, 5, 2, 3, rotate=rotate)
            sigma = 1 / math.sqrt(d)
            for corr in (True, False):
                got = O.attn_corrected(cache, 0, 5, q, kc, vc, sigma, correction=corr)["out"][0]
                want = _brute_force(q[0, 0], kc[0, 0], vc[0, 0], cache, 5, sigma, corr)
                assert np.allclose(got, want, atol=1e-12), (bits, group, d, rotate, corr)


def test_workload_recipes_are_deterministic_and_shaped():
    w = inputs.WORKLOADS["tiny"]
    a = inputs.make_chunk(w, 2)
    b = inputs.make_chunk(w, 2)
    assert all(np.array_equal(x, y) for x, y in zip(a, b))
    assert a[0].shape == (1, 2, 256, 64) and a[0].dtype == np.uint16
    assert not np.array_equal(inputs.make_chunk(w, 3)[1], a[1])
    w5 = inputs.WORKLOADS["pipeline"]
    _, k, _ = inputs.make_chunk(w5, 0, tokens=64)
    kf = np.abs(O.bf16_bits_to_f64(k)).mean(axis=(0, 2))            # [heads, d]
    assert ((kf > 4 * np.median(kf, axis=1, keepdims=True)).sum(axis=1) == 8).all()   # 8 outlier channels
    rows = inputs.sample_rows(1560, 128, 16)
    assert rows[0] == 0 and rows[-1] == 1559 and len(set(rows // 128)) == 13


def test_per_channel_keys_bias_is_one_scalar_per_block_and_matches_app_e():
    """App. E: with per-channel keys the Taylor bias is (sigma^2 / 24) sum_c q_c^2 step_c^2, the same for every
    token of a block.  Brute force over the stored bytes, with an explicit softmax."""
    d, bits, g, sigma = 64, 2, 32, 0.125
    w = inputs.Workload("pc", 88, 1, 1, d, 64, 0, bits, g, 2, k_outliers=2, k_outlier_scale=5.0)
    c = O.Cache(1, 1, d, bits, g, 128, k_per_channel=True)
    _, k, v = inputs.make_chunk(w, 0)
    O.quantize_append(c, 0, k, v)
    q, kc, vc = inputs.make_chunk(w, 3, tokens=10)
    got = O.attn_corrected(c, 0, 64, q, kc, vc, sigma)
    H = scipy.linalg.hadamard(d) / math.sqrt(d)
    f = O.bf16_bits_to_f64
    q_rot = f(q)[0, 0] @ H.T
    codes = O.unpack_codes(c.k_codes[0, 0, :64], bits).astype(np.float64)
    s = np.zeros((10, 64 + 10))
    for i in range(64):
        ds = O.e4m3_decode(c.k_scale[0, 0, i // g])              # [d] steps of the token's block
        zs = f(c.k_zero[0, 0, i // g])
        k_hat = (codes[i] - zs) * ds
        for m in range(10):
            b = sigma ** 2 / 24.0 * float(np.sum(q_rot[m] ** 2 * ds ** 2))
            s[m, i] = sigma * float(q_rot[m] @ k_hat) - b
    s[:, 64:] = sigma * f(q)[0, 0] @ f(kc)[0, 0].T
    p = np.exp(s - s.max(1, keepdims=True)); p /= p.sum(1, keepdims=True)
    v_hat = O.dequant(c.v_codes[0, 0, :64], c.v_scale[0, 0, :64], c.v_zero[0, 0, :64], bits, g)
    want = p[:, :64] @ v_hat + p[:, 64:] @ f(vc)[0, 0]
    assert np.abs(got["out"][0] - want).max() < 1e-12
    assert np.abs(got["cached_mass"][0] - p[:, :64].sum(1)).max() < 1e-12


# ---- attention-weight diagnostics: the Jensen-Shannon divergence of the appendix on attention JSD ----

def test_jsd_closed_forms_and_library_routine():
    import scipy.spatial.distance
    ln2 = math.log(2.0)
    p = np.array([[1.0, 0.0, 0.0], [0.5, 0.5, 0.0], [0.2, 0.3, 0.5]])
    assert np.abs(O.jsd_rows(p, p)).max() == 0.0                         # a distribution against itself
    assert abs(O.jsd_rows([[1.0, 0.0]], [[0.0, 1.0]])[0] - ln2) < 1e-15  # disjoint supports: the upper bound log 2
    # (1/2, 1/2) against (1, 0): KL(p||m) = log 2 - (1/2) log 3 ... worked by hand: (3/4) log(4/3) - ... = below
    want = 0.5 * (0.5 * math.log(0.5 / 0.75) + 0.5 * math.log(0.5 / 0.25)) + 0.5 * math.log(1.0 / 0.75)
    assert abs(O.jsd_rows([[0.5, 0.5]], [[1.0, 0.0]])[0] - want) < 1e-15 and abs(want - 0.21576155433883565) < 1e-12
    r = np.random.default_rng(5)
    a = r.random((40, 17)); a /= a.sum(1, keepdims=True)
    b = r.random((40, 17)); b[:, :3] = 0.0; b /= b.sum(1, keepdims=True)  # zeros: 0 log 0 = 0
    got = O.jsd_rows(a, b)
    lib = np.array([scipy.spatial.distance.jensenshannon(a[i], b[i]) ** 2 for i in range(40)])   # a distance: the square root
    assert np.abs(got - lib).max() < 1e-14
    assert np.abs(got - O.jsd_rows(b, a)).max() < 1e-15                  # symmetric
    assert (got > 0).all() and (got < ln2).all()


def test_bf16_reference_weights_are_the_library_softmax():
    r = np.random.default_rng(6)
    bf = lambda x: inputs.f32_to_bf16_bits(x.astype(np.float32))
    q, k = bf(r.standard_normal((9, 64))), bf(r.standard_normal((21, 64)))
    got = O.attention_weights_bf16(q, k, 0.2, rows=np.array([0, 4, 8]))
    qt = torch.from_numpy(O.bf16_bits_to_f64(q))[[0, 4, 8]]
    kt = torch.from_numpy(O.bf16_bits_to_f64(k))
    want = torch.softmax(0.2 * qt @ kt.T, dim=-1).numpy()
    assert np.abs(got - want).max() < 1e-15


def test_returned_weights_are_the_rows_behind_output_and_mass():
    q, kc, vc, ks, vs, cache = _tiny_problem(31, 64, 32, 2, 7, 4, 5)
    sl = cache.slots(0, 7)
    res = O.attn_corrected_head(q[0, 0], kc[0, 0], vc[0, 0], cache.k_codes[0, 0, sl], cache.k_scale[0, 0, sl],
                                cache.k_zero[0, 0, sl], cache.v_codes[0, 0, sl], cache.v_scale[0, 0, sl],
                                cache.v_zero[0, 0, sl], 2, 32, 0.125, return_weights=True)
    w = res["weights"]
    assert w.shape == (5, 11) and np.abs(w.sum(1) - 1).max() < 1e-14
    assert np.abs(w[:, :7].sum(1) - res["cached_mass"]).max() < 1e-15
    v_all = np.concatenate([O.dequant(cache.v_codes[0, 0, sl], cache.v_scale[0, 0, sl], cache.v_zero[0, 0, sl], 2, 32),
                            O.bf16_bits_to_f64(vc[0, 0])])
    assert np.abs(w @ v_all - res["out"]).max() < 1e-13


def test_weight_jsd_vanishes_for_a_lossless_cache_and_not_otherwise():
    # codes that reproduce the keys exactly, no rotation, no correction: the two weight vectors coincide
    q, kc, vc, ks, vs, cache = _tiny_problem(32, 64, 32, 2, 9, 3, 4, rotate=False, lossless=True)
    j = O.attn_weight_jsd(cache, 0, 9, q, kc, ks, 0.125, correction=False)
    assert j.shape == (1, 4) and np.abs(j).max() < 1e-25
    # the correction alone moves the weights (the steps are 0.5, not 0)
    assert O.attn_weight_jsd(cache, 0, 9, q, kc, ks, 0.125, correction=True).min() > 1e-9
    # a lossy cache: positive, below log 2, and equal to the definition written out for one row
    q, kc, vc, ks, vs, cache = _tiny_problem(33, 64, 32, 2, 9, 3, 4)
    j = O.attn_weight_jsd(cache, 0, 9, q, kc, ks, 0.125, correction=True, rows=np.array([2]))
    assert 0 < j[0, 0] < math.log(2.0)
    p = O.attn_corrected_head(q[0, 0], kc[0, 0], vc[0, 0], cache.k_codes[0, 0, :9], cache.k_scale[0, 0, :9],
                              cache.k_zero[0, 0, :9], cache.v_codes[0, 0, :9], cache.v_scale[0, 0, :9],
                              cache.v_zero[0, 0, :9], 2, 32, 0.125, rows=np.array([2]), return_weights=True)["weights"][0]
    f = O.bf16_bits_to_f64
    s = [0.125 * float(f(q)[0, 0, 2] @ kk) for kk in np.concatenate([f(ks)[0, 0], f(kc)[0, 0]])]
    z = sum(math.exp(x) for x in s)
    total = 0.0
    for pi, si in zip(p, s):
        ri = math.exp(si) / z
        mi = 0.5 * (pi + ri)
        total += 0.5 * pi * math.log(pi / mi) + 0.5 * ri * math.log(ri / mi)
    assert abs(total - j[0, 0]) < 1e-15
