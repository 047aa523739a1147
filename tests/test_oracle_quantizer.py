"""Pins for the oracle's quantizer (Eq. (1), group-wise per-token, E4M3 scale,
BF16 zero-point): worked example, error bound, brute force with a second
implementation, packing order, storage accounting."""
import os

import numpy as np

from oracle import kvq_oracle as O
from paper_2605_26266_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def test_worked_example_int2():
    # x = [-1, -0.25, 0.5, 2], B = 2, one group: step = (2 - -1)/3 = 1, z = -round(-1/1) = 1,
    # codes = clamp(round(x) + 1, 0, 3) with ties to even (round(0.5) = 0, round(-0.25) = -0).
    x = np.array([[-1.0, -0.25, 0.5, 2.0]])
    codes, sb, zb = O.quantize_vectors(x, bits=2, group=4)
    assert codes.tolist() == [[0, 1, 1, 3]]
    assert O.e4m3_decode(sb).tolist() == [[1.0]]
    assert O.bf16_bits_to_f64(zb).tolist() == [[1.0]]
    xh = O.dequant(O.pack_codes(codes, 2), sb, zb, 2, 4)
    assert xh.tolist() == [[-1.0, 0.0, 0.0, 2.0]]
    assert np.all(np.abs(xh - x) <= 0.5)


def test_worked_example_int4():
    # 16 levels over [0, 15] * 0.25: step 0.25 exactly, z = 0, codes = index.
    x = (np.arange(16) * 0.25)[None, :]
    codes, sb, zb = O.quantize_vectors(x, bits=4, group=16)
    assert codes.tolist() == [list(range(16))]
    assert float(O.e4m3_decode(sb)[0, 0]) == 0.25 and float(O.bf16_bits_to_f64(zb)[0, 0]) == 0.0
    # shifted range: [10, 13.75] -> z = -40
    codes, sb, zb = O.quantize_vectors(x + 10.0, bits=4, group=16)
    assert codes.tolist() == [list(range(16))]
    assert float(O.bf16_bits_to_f64(zb)[0, 0]) == -40.0
    assert np.array_equal(O.dequant(O.pack_codes(codes, 4), sb, zb, 4, 16), x + 10.0)


def test_error_bound_and_clamping():
    r = np.random.default_rng(0)
    for bits in (2, 4):
        for group in (32, 64, 128):
            y = O.f32(r.standard_normal((2000, 128)) * np.exp(r.uniform(-3, 3, (2000, 1))))
            codes, sb, zb = O.quantize_vectors(y, bits, group)
            ds = np.repeat(O.e4m3_decode(sb), group, axis=-1)
            zs = np.repeat(O.bf16_bits_to_f64(zb), group, axis=-1)
            L = 2 ** bits - 1
            assert codes.min() >= 0 and codes.max() <= L
            xh = (codes - zs) * ds
            unclamped = np.rint(y / ds) + zs
            inside = (unclamped >= 0) & (unclamped <= L)
            # |eps| <= step/2 wherever the clamp did not act (Eq. (1) and the bound below it)
            assert np.all(np.abs(xh - y)[inside] <= ds[inside] / 2 * (1 + 1e-6))
            # the clamp acts only on a small fraction (stored step rounded below the exact one)
            assert inside.mean() > 0.97
            # the stored step is the exact one within E4M3 rounding (relative 2^-4; absolute 2^-10 in the subnormal range)
            yg = y.reshape(2000, 128 // group, group)
            exact = (yg.max(-1) - yg.min(-1)) / L
            assert np.all(np.abs(O.e4m3_decode(sb) - exact) <= np.maximum(exact / 16, 2.0 ** -10) * (1 + 1e-6))
            # the step and the zero-point cover [min, max] (the sentence below Eq. (1)): with the zero-point taken
            # from the stored step, the minimum of a group gets code 0 exactly, and the maximum, whose distance
            # from it is at least L / (1 + 2^-4) stored steps, code L - 1 or L
            cg = codes.reshape(2000, 128 // group, group)
            at_min = np.take_along_axis(cg, yg.argmin(-1)[..., None], -1)[..., 0]
            at_max = np.take_along_axis(cg, yg.argmax(-1)[..., None], -1)[..., 0]
            normal = O.e4m3_decode(sb) >= 2.0 ** -6
            assert np.all(at_min[normal] == 0)
            assert np.all(at_max[normal] >= L - 1)


def _scalar_quantize_f32(vec, bits, group):
    """Second implementation: per-element Python loop in native numpy float32 scalars."""
    d = len(vec)
    L = np.float32(2 ** bits - 1)
    grid = [float(O.e4m3_decode(np.uint8(b))) for b in range(0x7F)]
    codes, sbytes, zbits = [], [], []
    for j in range(d // group):
        seg = [np.float32(t) for t in vec[j * group:(j + 1) * group]]
        mn, mx = min(seg), max(seg)
        step = np.float32(np.float32(mx - mn) / L)
        # nearest E4M3 value, ties to even byte, floor at byte 1, saturate
        best = min(range(1, 0x7F), key=lambda b: (abs(grid[b] - float(step)), b % 2))
        if float(step) >= 448:
            best = 0x7E
        ds = np.float32(grid[best])
        z = np.float32(0) - np.float32(np.rint(np.float32(mn / ds)))
        zb = int(O.f64_to_bf16_bits(np.array(float(z))))
        zs = np.float32(O.bf16_bits_to_f64(np.uint16(zb)))
        for t in seg:
            c = np.float32(np.rint(np.float32(t / ds))) + zs
            codes.append(int(min(max(c, np.float32(0)), L)))
        sbytes.append(best)
        zbits.append(zb)
    return codes, sbytes, zbits


def test_brute_force_second_implementation():
    r = np.random.default_rng(1)
    for bits, group, d in ((2, 64, 64), (2, 32, 128), (4, 128, 128), (4, 64, 128), (2, 128, 128)):
        y = (r.standard_normal((12, d)) * np.exp(r.uniform(-2, 4, (12, 1))) + r.uniform(-3, 3, (12, 1)))
        y = O.f32(y)
        codes, sb, zb = O.quantize_vectors(y, bits, group)
        for n in range(12):
            c2, s2, z2 = _scalar_quantize_f32(y[n], bits, group)
            assert codes[n].tolist() == c2
            assert sb[n].tolist() == s2
            assert zb[n].tolist() == z2


def test_constant_and_zero_groups():
    for v in (0.0, 1.0, -2.5):
        y = np.full((1, 64), v)
        codes, sb, zb = O.quantize_vectors(y, 2, 64)
        assert int(sb[0, 0]) == 0x01                      # floored at 2^-9, no division by zero
        xh = O.dequant(O.pack_codes(codes, 2), sb, zb, 2, 64)
        assert np.all(np.abs(xh - v) <= max(abs(v) * 2.0 ** -8, 2.0 ** -10))
    codes, sb, zb = O.quantize_vectors(np.zeros((1, 64)), 2, 64)
    assert codes.sum() == 0 and int(zb[0, 0]) == 0        # +0.0, not -0.0


def test_pack_order_little_endian():
    assert O.pack_codes(np.array([[1, 2, 3, 0]]), 2).tolist() == [[0b00111001]]
    assert O.pack_codes(np.array([[0xA, 0x3]]), 4).tolist() == [[0x3A]]
    r = np.random.default_rng(2)
    for bits in (2, 4):
        c = r.integers(0, 2 ** bits, size=(5, 128))
        p = O.pack_codes(c, bits)
        assert p.shape == (5, 128 * bits // 8)
        assert np.array_equal(O.unpack_codes(p, bits), c)
        # 32-bit word view: element e sits at bit (e mod 32/b)*b of word e // (32/b)
        w = p.view("<u4")
        per = 32 // bits
        for e in (0, 1, per - 1, per, 127):
            assert np.array_equal((w[:, e // per] >> ((e % per) * bits)) & (2 ** bits - 1), c[:, e])


def test_effective_bits_golden():
    for line in open(os.path.join(GOLDEN, "effective_bits.txt")):
        if line.startswith("#") or not line.strip():
            continue
        bits, group, printed, dec = line.split()
        assert round(O.effective_bits(int(bits), int(group)) + 1e-9, int(dec)) == float(printed)
    # byte accounting of a stored cache matches the formula
    c = O.Cache(1, 2, 128, 2, 32, 128)
    total_bits = 8 * (c.k_codes.nbytes + c.k_scale.nbytes + c.k_zero.nbytes)
    assert total_bits / (1 * 2 * 128 * 128) == O.effective_bits(2, 32) == 2.75


def test_quantize_append_places_chunks_and_rotates_keys_only():
    w = inputs.WORKLOADS["tiny"]
    _, k0, v0 = inputs.make_chunk(w, 0, tokens=40)
    _, k1, v1 = inputs.make_chunk(w, 1, tokens=24)
    c = O.Cache(w.batch, w.heads, w.head_dim, w.bits, w.group, 128)
    n = O.quantize_append(c, 0, k0, v0)
    n = O.quantize_append(c, n, k1, v1)
    assert n == 64
    assert not c.k_codes[:, :, 64:].any() and not c.k_scale[:, :, 64:].any()
    # keys: dequantized cache approximates the ROTATED key within step/2 (+ clamp cases)
    kall = O.bf16_bits_to_f64(np.concatenate([k0, k1], axis=2))
    vall = O.bf16_bits_to_f64(np.concatenate([v0, v1], axis=2))
    kh = O.dequant(c.k_codes[:, :, :64], c.k_scale[:, :, :64], c.k_zero[:, :, :64], w.bits, w.group)
    vh = O.dequant(c.v_codes[:, :, :64], c.v_scale[:, :, :64], c.v_zero[:, :, :64], w.bits, w.group)
    dk = O.e4m3_decode(c.k_scale[:, :, :64])
    dv = O.e4m3_decode(c.v_scale[:, :, :64])
    err_rot = np.abs(kh - O.rotate_f64(kall))
    err_unrot = np.abs(kh - kall)
    assert np.mean(err_rot <= dk / 2 + 1e-6) > 0.97
    assert np.mean(err_unrot <= dk / 2 + 1e-6) < 0.6
    assert np.mean(np.abs(vh - vall) <= dv / 2 + 1e-6) > 0.97      # values are not rotated
    # appending beyond capacity is an error
    try:
        O.quantize_append(c, 120, k0, v0)
        assert False
    except ValueError:
        pass


def test_fp32_steps_vs_unrounded_informational():
    """The binary32 rounding points move only a tiny fraction of codes (ties)."""
    r = np.random.default_rng(3)
    y = O.f32(r.standard_normal((4000, 128)))
    a, _, _ = O.quantize_vectors(y, 2, 64, fp32_steps=True)
    b, _, _ = O.quantize_vectors(y, 2, 64, fp32_steps=False)
    assert np.mean(a != b) < 1e-4 and np.abs(a - b).max() <= 1


def test_per_channel_keys_against_the_scalar_implementation():
    """App. E layout: one step / zero-point per (block of `group` tokens, channel).  The stored bytes must equal the
    scalar second implementation run over the `group` tokens of each channel of each block, and the dequantized
    keys must be (code - zero_c) * step_c."""
    from paper_2605_26266_b200 import inputs
    r = np.random.default_rng(3)
    for bits, g, d in ((2, 32, 64), (4, 64, 128)):
        n = 2 * g
        x = (r.standard_normal((1, 2, n, d)) * np.exp(r.uniform(-1, 2, (1, 2, 1, d)))).astype(np.float32)
        kb = inputs.f32_to_bf16_bits(x)
        vb = inputs.f32_to_bf16_bits(x[..., ::-1].copy())
        c = O.Cache(1, 2, d, bits, g, 4 * g, rotate_k=False, k_per_channel=True)
        assert c.k_scale.shape == (1, 2, 4, d) and c.v_scale.shape == (1, 2, 4 * g, d // g)
        O.quantize_append(c, g, kb, vb)                         # blocks 1 and 2
        k = O.bf16_bits_to_f64(kb)
        codes = O.unpack_codes(c.k_codes[:, :, g:3 * g], bits)
        for h in range(2):
            for blk in range(2):
                for ch in range(0, d, 7):
                    col = k[0, h, blk * g:(blk + 1) * g, ch]
                    c2, s2, z2 = _scalar_quantize_f32(col, bits, g)
                    assert codes[0, h, blk * g:(blk + 1) * g, ch].tolist() == c2
                    assert int(c.k_scale[0, h, 1 + blk, ch]) == s2[0] and int(c.k_zero[0, h, 1 + blk, ch]) == z2[0]
        # values keep the per-token layout of the plain cache
        p = O.Cache(1, 2, d, bits, g, 4 * g, rotate_k=False)
        O.quantize_append(p, g, kb, vb)
        assert np.array_equal(p.v_codes, c.v_codes) and np.array_equal(p.v_scale, c.v_scale)
        # whole blocks only
        try:
            O.quantize_append(c, 0, kb[:, :, :g - 1], vb[:, :, :g - 1])
            raise AssertionError("accepted a partial block")
        except ValueError:
            pass
