"""Pins for the oracle's number formats and rotation, against library routines,
textbook definitions and brute force (none of them the oracle's own code)."""
import math

import numpy as np
import scipy.linalg
import torch

from oracle import kvq_oracle as O


def test_e4m3_decode_all_bytes_against_torch():
    b = np.arange(256, dtype=np.uint8)
    want = torch.tensor(b).view(torch.float8_e4m3fn).double().numpy()
    assert np.array_equal(O.e4m3_decode(b), want, equal_nan=True)
    # landmarks of the format: 1.0, max 448, smallest subnormal 2^-9, smallest normal 2^-6
    assert O.e4m3_decode(np.uint8(0x38)) == 1.0
    assert O.e4m3_decode(np.uint8(0x7E)) == 448.0
    assert O.e4m3_decode(np.uint8(0x01)) == 2.0 ** -9
    assert O.e4m3_decode(np.uint8(0x08)) == 2.0 ** -6


def test_e4m3_encode_against_torch_in_range():
    r = np.random.default_rng(0)
    x = np.abs(r.standard_normal(100000)) * np.exp(r.uniform(-8, 6, 100000))
    x = x[(x < 440) & (x > 2.0 ** -9)].astype(np.float32).astype(np.float64)
    want = torch.tensor(x, dtype=torch.float32).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    got = O.e4m3_encode_scale(x)
    ok = want != 0            # torch may round to zero below 2^-9 * 1.5; the scale floor forbids that
    assert np.array_equal(got[ok], want[ok])
    assert np.all(got[~ok] == 1)


def test_e4m3_encode_brute_force_nearest_even():
    grid = O.e4m3_decode(np.arange(0, 0x7F, dtype=np.uint8))       # 0 .. 448, ascending
    r = np.random.default_rng(1)
    xs = list(np.exp(r.uniform(math.log(2.0 ** -9), math.log(448), 3000)))
    xs += [float(0.5 * (grid[i] + grid[i + 1])) for i in range(1, 0x7E - 1)]   # exact ties
    for x in xs:
        dist = np.abs(grid - x)
        best = np.flatnonzero(dist == dist.min())
        if len(best) == 2:                                          # tie: even mantissa wins
            pick = best[0] if best[0] % 2 == 0 else best[1]
        else:
            pick = best[0]
        pick = max(int(pick), 1)
        assert int(O.e4m3_encode_scale(np.array(x))) == pick, x


def test_e4m3_scale_saturates_and_floors():
    assert int(O.e4m3_encode_scale(np.array(1000.0))) == 0x7E
    assert int(O.e4m3_encode_scale(np.array(448.0))) == 0x7E
    assert int(O.e4m3_encode_scale(np.array(0.0))) == 0x01
    assert int(O.e4m3_encode_scale(np.array(1e-6))) == 0x01


def test_bf16_round_against_torch():
    r = np.random.default_rng(2)
    x = (r.standard_normal(100000) * np.exp(r.uniform(-20, 20, 100000))).astype(np.float32)
    want = torch.tensor(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = O.f64_to_bf16_bits(x.astype(np.float64))
    assert np.array_equal(got, want)
    back = torch.tensor(want.view(np.int16)).view(torch.bfloat16).double().numpy()
    assert np.array_equal(O.bf16_bits_to_f64(want), back)
    # a tie: 1 + 2^-8 lies halfway between 1 and 1 + 2^-7 -> even (1.0)
    assert int(O.f64_to_bf16_bits(np.array(1.0 + 2.0 ** -8))) == 0x3F80
    assert int(O.f64_to_bf16_bits(np.array(1.0 + 3 * 2.0 ** -8))) == 0x3F82


def test_rotation_is_sylvester_hadamard():
    r = np.random.default_rng(3)
    for d in (64, 128):
        x = r.standard_normal((5, d))
        H = scipy.linalg.hadamard(d).astype(np.float64)
        want = x @ H.T / math.sqrt(d)
        assert np.allclose(O.rotate_f64(x), want, rtol=0, atol=1e-12)
        # entry (a, b) of the Sylvester matrix is (-1)^popcount(a & b)
        a, b = 37 % d, 21
        assert H[a, b] == (-1) ** bin(a & b).count("1")
        s = r.choice([-1.0, 1.0], size=d)
        assert np.allclose(O.rotate_f64(x, s), (x * s) @ H.T / math.sqrt(d), atol=1e-12)
        # the binary32-stepped variant is the same map up to binary32 rounding
        x32 = x.astype(np.float32).astype(np.float64)
        y32 = O.rotate_f32_steps(x32)
        assert np.array_equal(y32, y32.astype(np.float32).astype(np.float64))
        assert np.allclose(y32, x32 @ H.T / math.sqrt(d), rtol=0, atol=2e-6)


def test_rotation_invariants():
    r = np.random.default_rng(4)
    d = 128
    q = r.standard_normal((7, d))
    k = r.standard_normal((9, d))
    qr, kr = O.rotate_f64(q), O.rotate_f64(k)
    assert np.allclose(qr @ kr.T, q @ k.T, atol=1e-10)              # (Hq)^T(Hk) = q^T k
    assert np.allclose((qr ** 2).sum(-1), (q ** 2).sum(-1))          # ||Hq|| = ||q||
    g = 32                                                           # per-group norms differ
    assert not np.allclose((qr.reshape(7, d // g, g) ** 2).sum(-1), (q.reshape(7, d // g, g) ** 2).sum(-1))
    assert np.allclose(O.rotate_f64(O.rotate_f64(q)), q, atol=1e-12)  # H symmetric and orthogonal


def test_scaling_constants():
    assert O.C_D[64] == 0.125
    assert np.float32(O.C_D[128]).view(np.uint32) == 0x3DB504F3
    assert abs(O.C_D[128] - 2.0 ** -3.5) < 2.0 ** -3.5 * 2.0 ** -24


def test_rotate_f32_steps_matches_native_float32_butterfly():
    """Second implementation: the same butterfly in native numpy float32 arithmetic."""
    r = np.random.default_rng(5)
    for d in (64, 128):
        x = r.standard_normal((4, d)).astype(np.float32)
        y = x.copy()
        h = 1
        while h < d:
            for i in range(d):
                if (i & h) == 0:
                    a, b = y[:, i].copy(), y[:, i + h].copy()
                    y[:, i], y[:, i + h] = a + b, a - b
            h *= 2
        y = y * np.float32(O.C_D[d])
        assert np.array_equal(O.rotate_f32_steps(x.astype(np.float64)).astype(np.float32), y)
