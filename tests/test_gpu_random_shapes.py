"""Seeded random shapes: small problems with lengths that hit every tile boundary case (1 row, 1 key, exact
multiples, one past a multiple), random formats, windows, rotation flags and ring wrap, both kernels against
the oracle.  Sizes stay small so that the oracle runs all rows."""
import numpy as np
import pytest
import torch

from oracle import kvq_oracle as O
from paper_2605_26266_b200 import inputs
from tests import kvq_testlib as T

pytestmark = pytest.mark.gpu

LENGTHS = [1, 2, 15, 16, 17, 63, 64, 65, 127, 128, 129, 255, 256, 257, 300, 511, 513]


def _cases():
    r = np.random.default_rng(20260527)
    out = []
    for i in range(24):
        d = int(r.choice([64, 128, 128]))
        bits = int(r.choice([2, 4]))
        group = int(r.choice([g for g in (32, 64, 128) if g <= d]))
        out.append(dict(i=i, d=d, bits=bits, group=group, batch=int(r.integers(1, 3)), heads=int(r.integers(1, 4)),
                        m=int(r.choice(LENGTHS)), n_cur=int(r.choice(LENGTHS)), n_cached=int(r.choice([0] + LENGTHS)),
                        begin=16 * int(r.integers(0, 5)), rotate=bool(r.integers(0, 2)), rotate_v=bool(r.integers(0, 2)),
                        ring=bool(r.integers(0, 2)), signs=bool(r.integers(0, 2)), corr=bool(r.integers(0, 2))))
    return out


@pytest.mark.parametrize("c", _cases(), ids=lambda c: f"{c['i']}-d{c['d']}b{c['bits']}g{c['group']}-m{c['m']}n{c['n_cur']}c{c['n_cached']}")
def test_random_shape(c):
    from paper_2605_26266_b200 import binding as B
    d, cap = c["d"], 640
    w = inputs.Workload("rand", 900 + c["i"], c["batch"], c["heads"], d, 32, 0, c["bits"], c["group"], c["i"],
                        k_outliers=2, k_outlier_scale=4.0, head_scale=True)
    signs = np.random.default_rng(c["i"]).choice([-1, 1], size=d).astype(np.int8) if c["signs"] else None
    kw = dict(rotate_k=c["rotate"], signs=signs, ring=c["ring"], rotate_v=c["rotate_v"])
    g = B.Cache(c["batch"], c["heads"], d, c["bits"], c["group"], cap, **kw)
    o = O.Cache(c["batch"], c["heads"], d, c["bits"], c["group"], cap, **kw)
    # fill up to begin + n_cached tokens; a ring cache starts far enough along that the window wraps
    start = 512 if c["ring"] else 0
    total = c["begin"] + c["n_cached"]
    pos, chunk_id = start, 0
    while pos < start + total:
        nt = min(150, start + total - pos)
        _, k, v = inputs.make_chunk(w, chunk_id, tokens=nt)
        B.kvq_quantize_append(g, T.to_dev(k), T.to_dev(v), cache_len=pos)
        O.quantize_append(o, pos, k, v)
        pos += nt; chunk_id += 1
    q, _, _ = inputs.make_chunk(w, 40, tokens=c["m"])
    _, kc, vc = inputs.make_chunk(w, 41, tokens=c["n_cur"])
    sigma = T.sigma_of(d) * (1.0 + 0.25 * (c["i"] % 3))
    begin = start + c["begin"]
    want = O.attn_corrected(o, begin, c["n_cached"], q, kc, vc, sigma, correction=c["corr"])
    flag = B.KVQ_CORRECTION_ON if c["corr"] else B.KVQ_CORRECTION_OFF
    for kname, kflag in [("mma_sync", B.KVQ_KERNEL_MMA_SYNC)] + ([("tcgen05", B.KVQ_KERNEL_TCGEN05), ("tcgen05_pair", B.KVQ_KERNEL_TCGEN05_PAIR)] if d == 128 else []):
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        lse = torch.zeros(q.shape[:3], dtype=torch.float32, device="cuda")
        mass = torch.zeros_like(lse)
        out = B.kvq_attn_corrected(g, T.to_dev(q), T.to_dev(kc), T.to_dev(vc), sigma, flag | kflag, cache_begin=begin,
                                   cache_len=c["n_cached"], lse=lse, cached_mass=mass, status_word=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        T.assert_attn_close(T.from_dev_bf16(out).reshape(want["out"].shape), want["out"], kname)
        assert np.abs(lse.cpu().numpy().reshape(want["lse"].shape) - want["lse"]).max() < 2e-2, kname
        assert np.abs(mass.cpu().numpy().reshape(want["cached_mass"].shape) - want["cached_mass"]).max() < 1e-2, kname


def _append_cases():
    r = np.random.default_rng(7)
    out = []
    for i in range(16):
        d = int(r.choice([64, 128]))
        out.append(dict(i=i, d=d, bits=int(r.choice([2, 4])), group=int(r.choice([g for g in (32, 64, 128) if g <= d])),
                        batch=int(r.integers(1, 3)), heads=int(r.integers(1, 5)), n=int(r.choice(LENGTHS[:15])),
                        pos=int(r.integers(0, 200)), rotate=bool(r.integers(0, 2)), rotate_v=bool(r.integers(0, 2)),
                        ring=bool(r.integers(0, 2)), scale=float(r.choice([1e-3, 1.0, 37.0, 1e4]))))
    return out


@pytest.mark.parametrize("c", _append_cases(), ids=lambda c: f"{c['i']}-d{c['d']}b{c['bits']}g{c['group']}-n{c['n']}p{c['pos']}")
def test_random_append_bit_exact(c):
    """Appends of random length at random positions (unaligned destinations, ring wrap) with random magnitudes."""
    from paper_2605_26266_b200 import binding as B
    d, cap = c["d"], 384
    r = np.random.default_rng(100 + c["i"])
    x = (r.standard_normal((2, c["batch"], c["heads"], c["n"], d)) * c["scale"]).astype(np.float32)
    x[0, ..., : d // 4] += 3.0 * c["scale"]                      # a shifted block: non-trivial zero-points
    kb, vb = inputs.f32_to_bf16_bits(x[0]), inputs.f32_to_bf16_bits(x[1])
    kw = dict(rotate_k=c["rotate"], ring=c["ring"], rotate_v=c["rotate_v"])
    g = B.Cache(c["batch"], c["heads"], d, c["bits"], c["group"], cap, **kw)
    o = O.Cache(c["batch"], c["heads"], d, c["bits"], c["group"], cap, **kw)
    pos = c["pos"] + (cap - 100 if c["ring"] else 0)              # a ring append straddles the end of the buffer
    if not c["ring"] and pos + c["n"] > cap:
        pos = cap - c["n"]
    B.kvq_quantize_append(g, T.to_dev(kb), T.to_dev(vb), cache_len=pos)
    O.quantize_append(o, pos, kb, vb)
    T.assert_cache_equal(T.gpu_cache_arrays(g, cap), o, cap)
