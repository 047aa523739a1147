"""FP64 CPU oracle for the corrected low-bit KV-cache chunk attention path.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain statement of what the
CUDA library must compute.  It shares no code with the CUDA path and is only
to be imported by tests, by the smoke check and by the benchmark's CPU-baseline
leg.  The product never routes through it.

What it follows (paper sections / equations):

* Quantizer: Eq. (1) (asymmetric integer round-to-nearest with scale and
  zero-point covering [min, max]), "Quantization granularity" (group-wise
  per-token), "Hadamard rotation" (orthogonal H applied to keys and queries),
  and the storage formats of Sec. 5.1 / App. B (FP8-E4M3 scale and BF16
  zero-point per group, 24 metadata bits per group, Eq. (21)).
* Attention: Algorithm 1 (Taylor-corrected attention, group-wise), Eqs. (2)-(4)
  (scores, partition sums, cached mass), Eq. (15) / Eq. (25) (grouped Taylor
  correction, with the rotated query under QuaRot), Eq. (12) (exact sinh form).
* Diagnostics: the Jensen-Shannon divergence between the attention weights over
  all keys with the quantized (or corrected) cache and with the BF16 cache
  (App. "Attention JSD Distributions").

Readings of points the paper leaves open (each one is a reading, "parity
unpinned" by the paper itself; the quantizer as a whole is pinned by the error
bound, the worked example and brute force in the tests):

* rounding is ties-to-even;
* scale  = E4M3((max-min)/(2^B-1)) round-to-nearest-even, saturating at 448 and
  floored at the smallest subnormal 2^-9;
* zero-point z = -round(min/scale), an integer, stored as BF16;
* codes use the *stored* scale and zero-point, so dequantization is
  self-consistent;
* Hadamard matrix in Sylvester (natural) order times an optional diagonal of
  +-1 signs, normalised by 1/sqrt(d);
* values are not rotated; current-chunk scores use the unrotated q and k;
* packing is little-endian, element 0 in the least significant bits.

Part Q (quantizer) is the bit-exact contract: FP64 arithmetic with an explicit
rounding to binary32 after every add, subtract, multiply and divide.  Because
binary64 carries more than 2*24+2 significand bits, that equals the correctly
rounded binary32 operation, i.e. what an IEEE FP32 kernel without contraction
produces.  Part A (attention) is pure FP64.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import numpy as np

# --------------------------------------------------------------------------
# number formats
# --------------------------------------------------------------------------


def f32(x):
    """Round a float64 array to binary32 and return it as float64."""
    return np.asarray(x, dtype=np.float64).astype(np.float32).astype(np.float64)


def bf16_bits_to_f64(bits):
    """BF16 bit patterns (uint16) -> float64, exact."""
    b = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return b.view(np.float32).astype(np.float64)


def f64_to_bf16_bits(x):
    """Round-to-nearest-even of finite binary32-representable values to BF16 bits."""
    u = np.asarray(x, dtype=np.float64).astype(np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = (u + np.uint32(0x7FFF) + lsb) >> np.uint32(16)
    return r.astype(np.uint16)


def e4m3_decode(byte):
    """OCP FP8 E4M3 byte -> float64.  1 sign, 4 exponent (bias 7), 3 mantissa bits;
    exponent field 0 is subnormal (m/8 * 2^-6); S.1111.111 is NaN; no infinities."""
    b = np.asarray(byte, dtype=np.uint8).astype(np.int64)
    s = np.where(b & 0x80, -1.0, 1.0)
    e = (b >> 3) & 0xF
    m = b & 0x7
    sub = (m / 8.0) * 2.0 ** -6
    nor = (1.0 + m / 8.0) * np.exp2((e - 7).astype(np.float64))
    v = np.where(e == 0, sub, nor)
    v = np.where((e == 15) & (m == 7), np.nan, v)
    return s * v


def e4m3_encode_scale(x):
    """Non-negative step size -> E4M3 byte: round-to-nearest-even on the E4M3 grid,
    saturate at 448 (0x7E), floor at the smallest subnormal 2^-9 (0x01)."""
    v = np.asarray(x, dtype=np.float64)
    if not np.all(v >= 0.0):
        raise ValueError("scale must be a non-negative number")
    v = np.minimum(v, 448.0)
    # grid spacing around v: 2^(e-3), e = floor(log2 v), clipped below at the subnormal binade
    _, ex = np.frexp(v)                       # v = m * 2^ex, m in [0.5, 1)
    e = np.maximum(ex - 1, -6)
    ulp = np.exp2((e - 3).astype(np.float64))
    q = np.rint(v / ulp) * ulp                # ties-to-even; may roll over into the next binade
    q = np.clip(q, 2.0 ** -9, 448.0)
    # q is on the grid: encode it
    _, exq = np.frexp(q)
    eq = exq - 1
    sub = q < 2.0 ** -6
    byte_sub = np.rint(q / 2.0 ** -9).astype(np.int64)
    mant = np.rint((q / np.exp2(eq.astype(np.float64)) - 1.0) * 8.0).astype(np.int64)
    byte_nor = ((eq.astype(np.int64) + 7) << 3) | mant
    return np.where(sub, byte_sub, byte_nor).astype(np.uint8)


# --------------------------------------------------------------------------
# Hadamard rotation ("Hadamard rotation" paragraph; App. F)
# --------------------------------------------------------------------------

C_D = {64: 0.125, 128: float(np.float32(2.0 ** -3.5))}


def _butterflies(y, d, rounder):
    shape = y.shape
    h = 1
    while h < d:
        y = y.reshape(shape[:-1] + (d // (2 * h), 2, h))
        a = y[..., 0, :]
        b = y[..., 1, :]
        y = np.stack([rounder(a + b), rounder(a - b)], axis=-2).reshape(shape)
        h *= 2
    return y


def rotate_f32_steps(x, signs=None):
    """y = (1/sqrt d) H_d (s * x) with binary32 rounding after every butterfly add/sub
    (stages h = 1, 2, 4, ... in that order) and after the final scaling by the
    binary32 constant c_d."""
    x = np.asarray(x, dtype=np.float64)
    d = x.shape[-1]
    if signs is not None:
        x = x * np.asarray(signs, dtype=np.float64)
    y = _butterflies(x, d, f32)
    return f32(y * C_D[d])


def rotate_f64(x, signs=None):
    """y = (1/sqrt d) H_d (s * x) in plain float64."""
    x = np.asarray(x, dtype=np.float64)
    d = x.shape[-1]
    if signs is not None:
        x = x * np.asarray(signs, dtype=np.float64)
    y = _butterflies(x, d, lambda t: t)
    return y / math.sqrt(d)


# --------------------------------------------------------------------------
# Part Q: quantizer, bit-exact contract (Eq. (1), group-wise per-token)
# --------------------------------------------------------------------------


def quantize_vectors(y, bits, group, fp32_steps=True):
    """Quantize vectors y[..., d] (binary32-representable float64) group-wise.

    Returns (codes int64 [..., d], scale_byte uint8 [..., G], zero_bits uint16 [..., G]).
    With fp32_steps=False the same steps run without intermediate binary32
    rounding (informational variant)."""
    rnd = f32 if fp32_steps else (lambda t: np.asarray(t, dtype=np.float64))
    y = np.asarray(y, dtype=np.float64)
    d = y.shape[-1]
    G = d // group
    L = float(2 ** bits - 1)
    yg = y.reshape(y.shape[:-1] + (G, group))
    mn = yg.min(axis=-1)
    mx = yg.max(axis=-1)
    step = rnd(rnd(mx - mn) / L)
    scale_byte = e4m3_encode_scale(step)
    ds = e4m3_decode(scale_byte)
    z = -np.rint(rnd(mn / ds))
    z = z + 0.0                                   # -0.0 -> +0.0
    zero_bits = f64_to_bf16_bits(z)
    zs = bf16_bits_to_f64(zero_bits)
    c = np.rint(rnd(yg / ds[..., None])) + zs[..., None]
    c = np.clip(c, 0.0, L)
    return c.reshape(y.shape).astype(np.int64), scale_byte, zero_bits


def pack_codes(codes, bits):
    """codes int [..., d] -> uint8 [..., d*bits/8]; element 0 in the least significant bits."""
    codes = np.asarray(codes, dtype=np.uint8)
    per = 8 // bits
    c = codes.reshape(codes.shape[:-1] + (codes.shape[-1] // per, per))
    out = np.zeros(c.shape[:-1], dtype=np.uint8)
    for i in range(per):
        out |= (c[..., i] << np.uint8(i * bits)).astype(np.uint8)
    return out


def unpack_codes(packed, bits):
    """Inverse of pack_codes."""
    packed = np.asarray(packed, dtype=np.uint8)
    per = 8 // bits
    mask = np.uint8(2 ** bits - 1)
    parts = [(packed >> np.uint8(i * bits)) & mask for i in range(per)]
    return np.stack(parts, axis=-1).reshape(packed.shape[:-1] + (packed.shape[-1] * per,))


@dataclass
class Cache:
    """Quantized KV cache: what Sec. 5.1 stores per (batch, head, token): packed
    codes for K and V, and per group one E4M3 scale byte and one BF16 zero-point."""
    batch: int
    heads: int
    head_dim: int
    bits: int
    group: int
    capacity: int
    rotate_k: bool = True
    signs: np.ndarray | None = None
    rotate_v: bool = False  # values rotated too before quantization (the value path of the rotation scheme the
                            # paper extends in App. F); the attention output is rotated back
    k_per_channel: bool = False  # App. E: key steps and zero-points per channel, shared by the `group` tokens of a
                            # block (k_scale, k_zero are then [B, H, capacity // group, d]); values stay per token
    ring: bool = False      # sliding-window use (Sec. 2: attend to the last n cached chunks): token t lives in slot t mod capacity

    def slots(self, begin, n):
        """Slots of the tokens [begin, begin + n): themselves, or taken modulo the capacity for a ring cache."""
        idx = np.arange(begin, begin + n, dtype=np.int64)
        if self.ring:
            if n > self.capacity:
                raise ValueError("more tokens than slots")
            return idx % self.capacity
        if begin + n > self.capacity:
            raise ValueError("capacity exceeded")
        return idx

    def __post_init__(self):
        B, H, C, d = self.batch, self.heads, self.capacity, self.head_dim
        G = d // self.group
        nb = d * self.bits // 8
        self.k_codes = np.zeros((B, H, C, nb), np.uint8)
        self.v_codes = np.zeros((B, H, C, nb), np.uint8)
        self.k_scale = np.zeros((B, H, C // self.group, d) if self.k_per_channel else (B, H, C, G), np.uint8)
        self.v_scale = np.zeros((B, H, C, G), np.uint8)
        self.k_zero = np.zeros((B, H, C // self.group, d) if self.k_per_channel else (B, H, C, G), np.uint16)
        self.v_zero = np.zeros((B, H, C, G), np.uint16)

    @property
    def G(self):
        return self.head_dim // self.group


def quantize_append(cache: Cache, cache_len: int, k_bits, v_bits):
    """Rotate (keys only), quantize, pack and store a finished chunk at tokens
    [cache_len, cache_len + n) (slots taken modulo the capacity for a ring cache, where the
    new tokens overwrite the oldest ones).  k_bits, v_bits: BF16 bit patterns [B, H, n, d]."""
    n = k_bits.shape[2]
    sl = cache.slots(cache_len, n)
    k = bf16_bits_to_f64(k_bits)
    v = bf16_bits_to_f64(v_bits)
    if cache.rotate_k:
        k = rotate_f32_steps(k, cache.signs)
    if cache.k_per_channel:
        # App. E: for every block of `group` consecutive tokens and every channel, one step and one zero-point over
        # the block's tokens: Eq. (1) with the roles of tokens and channels exchanged inside a block
        g = cache.group
        if cache_len % g or n % g:
            raise ValueError("per-channel keys are appended in whole blocks of `group` tokens")
        kb = np.swapaxes(k.reshape(k.shape[:2] + (n // g, g, k.shape[-1])), -1, -2)      # [B, H, blocks, d, g]
        kc, ks, kz = quantize_vectors(kb, cache.bits, g)
        kc = np.swapaxes(kc, -1, -2).reshape(k.shape)
        blocks = sl[::g] // g
        cache.k_codes[:, :, sl] = pack_codes(kc, cache.bits)
        cache.k_scale[:, :, blocks] = ks[..., 0]
        cache.k_zero[:, :, blocks] = kz[..., 0]
    else:
        kc, ks, kz = quantize_vectors(k, cache.bits, cache.group)
        cache.k_codes[:, :, sl] = pack_codes(kc, cache.bits)
        cache.k_scale[:, :, sl] = ks
        cache.k_zero[:, :, sl] = kz
    if cache.rotate_v:
        v = rotate_f32_steps(v, cache.signs)
    vc, vs, vz = quantize_vectors(v, cache.bits, cache.group)
    cache.v_codes[:, :, sl] = pack_codes(vc, cache.bits)
    cache.v_scale[:, :, sl] = vs
    cache.v_zero[:, :, sl] = vz
    return cache_len + n


def dequant(codes_packed, scale_byte, zero_bits, bits, group):
    """x_hat = (x_q - z) * scale from the stored bytes (reconstruction of Eq. (1))."""
    c = unpack_codes(codes_packed, bits).astype(np.float64)
    ds = e4m3_decode(scale_byte)
    zs = bf16_bits_to_f64(zero_bits)
    G = ds.shape[-1]
    cg = c.reshape(c.shape[:-1] + (G, group))
    return ((cg - zs[..., None]) * ds[..., None]).reshape(c.shape)


# --------------------------------------------------------------------------
# Part A: corrected attention (Algorithm 1), pure FP64
# --------------------------------------------------------------------------


def log_sinhc(alpha):
    """log(sinh(a)/a), stable: Maclaurin series for |a| < 0.05, the definition up to |a| = 20, the overflow-free form |a| - log(2|a|) + log1p(-e^{-2|a|}) beyond (Eq. (12))."""
    a = np.abs(np.asarray(alpha, dtype=np.float64))
    out = np.empty_like(a)
    small = a < 0.05
    a2 = a[small] ** 2
    out[small] = a2 / 6.0 - a2 ** 2 / 180.0 + a2 ** 3 / 2835.0 - a2 ** 4 / 37800.0
    mid = (~small) & (a < 20.0)
    out[mid] = np.log(np.sinh(a[mid]) / a[mid])
    big = a >= 20.0
    out[big] = a[big] - np.log(2.0 * a[big]) + np.log1p(-np.exp(-2.0 * a[big]))
    return out


def taylor_bias(nu, key_scale, sigma):
    """b[m, i] = (sigma^2 / 24) * sum_j scale[i, j]^2 * nu[m, j]   (Eq. (15); with
    sigma = 1/sqrt(d) this is the 1/(24 d) prefactor)."""
    return (sigma * sigma / 24.0) * (nu @ (key_scale ** 2).T)


def exact_bias(q_rot, key_scale, group, sigma):
    """b[m, i] = sum_c log(sinh(a)/a), a = sigma * q_c * scale[i, group(c)] / 2  (Eq. (12))."""
    sc = np.repeat(key_scale, group, axis=-1)          # [N, d]
    a = 0.5 * sigma * q_rot[:, None, :] * sc[None, :, :]
    return log_sinhc(a).sum(axis=-1)


def attn_corrected_head(q_bits, kcur_bits, vcur_bits, k_codes, k_scale, k_zero,
                        v_codes, v_scale, v_zero, bits, group, sigma, correction=True,
                        rotate=True, signs=None, rows=None, exact=False, rotate_v=False, k_group=None,
                        return_weights=False):
    """One (batch, head) unit of Algorithm 1.

    q_bits [M, d], kcur_bits/vcur_bits [N_R, d] BF16 bit patterns; cache slices for
    the attended window, [N_S, ...].  rows: optional index array of query rows.
    Returns dict(out [m, d], lse [m], cached_mass [m], current_mass [m]); the two masses are
    P_S and P_R of Eq. (4), summed separately.  k_group: channels per key group if it differs from the values'
    (1 for per-channel keys, whose k_scale / k_zero arrive expanded to one row per token, [N_S, d]).
    return_weights: also return "weights" [m, N_S + N_R], the softmax rows themselves (cached keys first)."""
    k_group = group if k_group is None else k_group
    q = bf16_bits_to_f64(q_bits)
    if rows is not None:
        q = q[rows]
    d = q.shape[-1]
    G = d // k_group
    kr = bf16_bits_to_f64(kcur_bits)
    vr = bf16_bits_to_f64(vcur_bits)
    n_s = k_codes.shape[0]
    q_rot = rotate_f64(q, signs) if rotate else q
    nu = (q_rot.reshape(q.shape[0], G, k_group) ** 2).sum(axis=-1)        # Alg. 1: nu[m, j]
    s_r = sigma * (q @ kr.T)                                                # S_R
    if n_s > 0:
        k_hat = dequant(k_codes, k_scale, k_zero, bits, k_group)            # dequant(K^q)
        v_hat = dequant(v_codes, v_scale, v_zero, bits, group)
        s_s = sigma * (q_rot @ k_hat.T)                                     # S_S
        if correction:
            ds = e4m3_decode(k_scale)
            b = exact_bias(q_rot, ds, k_group, sigma) if exact else taylor_bias(nu, ds, sigma)
            s_s = s_s - b                                                   # cached scores only
    else:
        s_s = np.zeros((q.shape[0], 0))
        v_hat = np.zeros((0, d))
    s = np.concatenate([s_s, s_r], axis=1)
    mx = s.max(axis=1, keepdims=True)
    e = np.exp(s - mx)
    z = e.sum(axis=1, keepdims=True)
    p = e / z
    o_s = p[:, :n_s] @ v_hat
    if rotate_v:
        # the cached values are stored rotated: R v with R = (1/sqrt d) H diag(s), R^-1 y = s * ((1/sqrt d) H y)
        o_s = rotate_f64(o_s, None)
        if signs is not None:
            o_s = o_s * np.asarray(signs, dtype=np.float64)
    out = o_s + p[:, n_s:] @ vr
    res = {"out": out, "lse": (mx + np.log(z))[:, 0],
           "cached_mass": p[:, :n_s].sum(axis=1), "current_mass": p[:, n_s:].sum(axis=1)}
    if return_weights:
        res["weights"] = p
    return res


def attn_corrected(cache: Cache, cache_begin, cache_len, q_bits, kcur_bits, vcur_bits,
                   sigma, correction=True, rows=None, heads=None, exact=False):
    """All (batch, head) units.  q_bits [B, H, M, d]; kcur/vcur [B, H, N_R, d].
    heads: optional list of (b, h) pairs to evaluate (others are skipped).
    Returns dict of arrays indexed [unit, row, ...] in the order of `heads`."""
    B, H = q_bits.shape[:2]
    units = heads if heads is not None else [(b, h) for b in range(B) for h in range(H)]
    sl = cache.slots(cache_begin, cache_len)
    outs, lses, masses, cmasses = [], [], [], []
    # per-channel keys (App. E): every token takes the steps and zero-points of its block, one per channel; the bias
    # of Eq. (15) with groups of one channel is then the App. E form (1/24d) sum_c q_c^2 step_c^2, equal for all
    # tokens of a block
    ksl = sl // cache.group if cache.k_per_channel else sl
    for (b, h) in units:
        r = attn_corrected_head(
            q_bits[b, h], kcur_bits[b, h], vcur_bits[b, h],
            cache.k_codes[b, h, sl], cache.k_scale[b, h, ksl], cache.k_zero[b, h, ksl],
            cache.v_codes[b, h, sl], cache.v_scale[b, h, sl], cache.v_zero[b, h, sl],
            cache.bits, cache.group, sigma, correction, cache.rotate_k, cache.signs,
            rows, exact, cache.rotate_v, 1 if cache.k_per_channel else None)
        outs.append(r["out"])
        lses.append(r["lse"])
        masses.append(r["cached_mass"])
        cmasses.append(r["current_mass"])
    return {"out": np.stack(outs), "lse": np.stack(lses), "cached_mass": np.stack(masses),
            "current_mass": np.stack(cmasses)}


def attention_weights_bf16(q_bits, k_bits, sigma, rows=None):
    """softmax(sigma q k^T) row by row for BF16 q [M, d] and k [N, d]: the attention weights of the unquantized
    (BF16) cache that the quantized ones are compared with."""
    q = bf16_bits_to_f64(q_bits)
    if rows is not None:
        q = q[rows]
    s = sigma * (q @ bf16_bits_to_f64(k_bits).T)
    e = np.exp(s - s.max(axis=1, keepdims=True))
    return e / e.sum(axis=1, keepdims=True)


def jsd_rows(p, r):
    """Jensen-Shannon divergence of each row of p from the same row of r (natural logarithm, 0 log 0 = 0):
    JSD = KL(p || m) / 2 + KL(r || m) / 2 with the mixture m = (p + r) / 2; between 0 and log 2."""
    p = np.asarray(p, dtype=np.float64)
    r = np.asarray(r, dtype=np.float64)
    m = 0.5 * (p + r)

    def kl(a):
        t = np.zeros_like(a)
        nz = a > 0
        t[nz] = a[nz] * np.log(a[nz] / m[nz])
        return t.sum(axis=-1)

    return 0.5 * kl(p) + 0.5 * kl(r)


def attn_weight_jsd(cache: Cache, cache_begin, cache_len, q_bits, kcur_bits, kcached_bits, sigma,
                    correction=True, rows=None, heads=None):
    """Per query row, the JSD between the attention weights over all keys [cached ; current] computed with the
    quantized cache (Algorithm 1, with or without the correction) and with the BF16 keys `kcached_bits`
    [B, H, cache_len, d] those cache entries were quantized from.  Returns [unit, row]."""
    B, H = q_bits.shape[:2]
    units = heads if heads is not None else [(b, h) for b in range(B) for h in range(H)]
    sl = cache.slots(cache_begin, cache_len)
    out = []
    for (b, h) in units:
        vz = np.zeros_like(kcur_bits[b, h])                # the weights do not depend on the values
        wq = attn_corrected_head(
            q_bits[b, h], kcur_bits[b, h], vz,
            cache.k_codes[b, h, sl], cache.k_scale[b, h, sl], cache.k_zero[b, h, sl],
            cache.v_codes[b, h, sl], cache.v_scale[b, h, sl], cache.v_zero[b, h, sl],
            cache.bits, cache.group, sigma, correction, cache.rotate_k, cache.signs, rows,
            return_weights=True)["weights"]
        k_all = np.concatenate([kcached_bits[b, h], kcur_bits[b, h]], axis=0)
        out.append(jsd_rows(wq, attention_weights_bf16(q_bits[b, h], k_all, sigma, rows)))
    return np.stack(out)


def effective_bits(bits, group):
    """B_eff = B + 24/g: 8-bit scale + 16-bit zero-point per group (Eq. (21))."""
    return bits + 24.0 / group
