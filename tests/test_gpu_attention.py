"""GPU parity: kvq_attn_corrected against the oracle (Algorithm 1 in FP64), through the C ABI.
Tolerances: relative L2 <= 1e-2 and max-abs <= 2e-2 on the BF16 output."""
import math

import numpy as np
import pytest
import torch

from oracle import kvq_oracle as O
from paper_2605_26266_b200 import inputs
from tests import kvq_testlib as T

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2605_26266_b200 import binding
    return binding


def kernels(B, head_dim=128):
    """Every kernel that covers the shape: the warp-level one always, the tcgen05 ones (one CTA per 256 query
    rows; a pair of CTAs per 512) for head_dim 128."""
    ks = [("mma_sync", B.KVQ_KERNEL_MMA_SYNC)]
    if head_dim == 128:
        ks.append(("tcgen05", B.KVQ_KERNEL_TCGEN05))
        ks.append(("tcgen05_pair", B.KVQ_KERNEL_TCGEN05_PAIR))
    return ks


def _build(B, w, chunks, tokens=None, rotate=True, signs=None, units=None, cap=None):
    """GPU cache of all heads; oracle cache of `units` (or all heads); returns also the current chunk."""
    cap = cap or w.capacity
    g = B.Cache(w.batch, w.heads, w.head_dim, w.bits, w.group, cap, rotate_k=rotate, signs=signs)
    if units is None:
        units = [(b, h) for b in range(w.batch) for h in range(w.heads)]
    o = O.Cache(1, len(units), w.head_dim, w.bits, w.group, cap, rotate_k=rotate, signs=signs)
    sel = lambda a: np.stack([a[b, h] for (b, h) in units])[None]
    n = 0
    for c in range(chunks):
        _, k, v = inputs.make_chunk(w, c, tokens=tokens)
        B.kvq_quantize_append(g, T.to_dev(k), T.to_dev(v))
        n = O.quantize_append(o, n, sel(k), sel(v))
    return g, o, n, sel


def _compare(B, g, o, n_cache, q, kc, vc, sigma, sel, rows=None, flags_list=None, begin=0, check_aux=True):
    qd, kd, vd = T.to_dev(q), T.to_dev(kc), T.to_dev(vc)
    res = {}
    for corr in (True, False):
        want = O.attn_corrected(o, begin, n_cache, sel(q), sel(kc), sel(vc), sigma, correction=corr, rows=rows)
        for kname, kflag in (flags_list or kernels(B, q.shape[-1])):
            flags = (B.KVQ_CORRECTION_ON if corr else B.KVQ_CORRECTION_OFF) | kflag
            lse = torch.zeros(q.shape[:3], dtype=torch.float32, device="cuda")
            mass = torch.zeros_like(lse)
            status = torch.zeros(1, dtype=torch.int32, device="cuda")
            out = B.kvq_attn_corrected(g, qd, kd, vd, sigma, flags, cache_begin=begin, cache_len=n_cache,
                                       lse=lse, cached_mass=mass, status_word=status)
            torch.cuda.synchronize()
            assert int(status.item()) == 0
            got = sel(T.from_dev_bf16(out))[0]
            lse_g = sel(lse.cpu().numpy().astype(np.float64))[0]
            mass_g = sel(mass.cpu().numpy().astype(np.float64))[0]
            if rows is not None:
                got, lse_g, mass_g = got[:, rows], lse_g[:, rows], mass_g[:, rows]
            res[(corr, kname)] = T.assert_attn_close(got, want["out"], f"corr={corr} kernel={kname}")
            if check_aux:
                assert np.abs(lse_g - want["lse"]).max() < 2e-2, kname
                assert np.abs(mass_g - want["cached_mass"]).max() < 1e-2, kname
    return res


def test_tiny_config_full_parity(B):
    w = inputs.WORKLOADS["tiny"]
    g, o, n, sel = _build(B, w, w.cached_chunks)
    q, kc, vc = inputs.make_chunk(w, w.cached_chunks)
    _compare(B, g, o, n, q, kc, vc, T.sigma_of(w.head_dim), sel)


@pytest.mark.parametrize("d,bits,group", [(64, 2, 32), (64, 4, 64), (128, 2, 32), (128, 2, 64),
                                          (128, 2, 128), (128, 4, 32), (128, 4, 128)])
def test_ragged_shapes_all_formats(B, d, bits, group):
    # m, cache and current lengths that are no multiple of any tile size
    w = inputs.Workload("rag", 200 + d + bits + group, 2, 3, d, 173, 0, bits, group, 3,
                        k_outliers=2, k_outlier_scale=6.0, head_scale=True)
    signs = np.random.default_rng(group).choice([-1, 1], size=d).astype(np.int8)
    g, o, n, sel = _build(B, w, 3, tokens=111, signs=signs, cap=512)
    assert n == 333
    q, _, _ = inputs.make_chunk(w, 5, tokens=173)
    _, kc, vc = inputs.make_chunk(w, 6, tokens=77)
    _compare(B, g, o, n, q, kc, vc, T.sigma_of(d), sel)


def test_short_chunk_long_cache_is_split_over_ctas(B):
    """Few (batch, head, query block) units and a long cache: the tcgen05 kernel cuts the key tiles of a unit
    over several CTAs and merges their partial results (needs the workspace)."""
    w = inputs.Workload("split", 320, 1, 2, 128, 200, 0, 2, 64, 0, k_outliers=2, k_outlier_scale=4.0)
    g, o, n, sel = _build(B, w, 9, tokens=1111, cap=10112)
    assert n == 9999
    q, kc, vc = inputs.make_chunk(w, 20)
    assert B.kvq_attn_workspace_bytes(g, n, 200, 200, B.KVQ_CORRECTION_ON | B.KVQ_KERNEL_TCGEN05) > 0
    _compare(B, g, o, n, q, kc, vc, T.sigma_of(128), sel)
    # a missing workspace is refused on the host
    import ctypes as C
    d = g.desc
    s = B.kvq_strides(q.shape[1] * 200 * 128, 200 * 128, 128)
    qd = T.to_dev(q)
    out = torch.empty_like(qd)
    rc = B.lib.kvq_attn_corrected(C.byref(d), 0, n, qd.data_ptr(), s, qd.data_ptr(), qd.data_ptr(), s, 200, 200,
                                  out.data_ptr(), s, 0.088, B.KVQ_CORRECTION_ON | B.KVQ_KERNEL_TCGEN05,
                                  None, None, None, 0, None, None)
    assert rc == B.KVQ_ERR_WORKSPACE


@pytest.mark.parametrize("heads,picked", [(152, [0, 77, 147, 148, 150, 151]), (230, [0, 147, 148, 229])])
def test_more_units_than_sms(B, heads, picked):
    """More (head, query block) units than SMs: persistent CTAs take whole units in rounds; a short last round
    (152 units on 148 SMs) is split over all CTAs and merged, a long one (230 units) is dealt out whole."""
    w = inputs.Workload("many", 330 + heads, 1, heads, 128, 200, 0, 2, 32, 0, k_outliers=1, k_outlier_scale=5.0)
    units = [(0, h) for h in picked]
    g, o, n, sel = _build(B, w, 3, tokens=150, units=units, cap=512)
    assert n == 450
    q, _, _ = inputs.make_chunk(w, 7)
    _, kc, vc = inputs.make_chunk(w, 8, tokens=130)
    _compare(B, g, o, n, q, kc, vc, T.sigma_of(128), sel, flags_list=[("tcgen05", B.KVQ_KERNEL_TCGEN05)])


def test_empty_cache_is_plain_attention(B):
    w = inputs.Workload("empty", 300, 1, 2, 128, 150, 0, 2, 64, 0)
    g = B.Cache(1, 2, 128, 2, 64, 128)
    o = O.Cache(1, 2, 128, 2, 64, 128)
    q, kc, vc = inputs.make_chunk(w, 0)
    _compare(B, g, o, 0, q, kc, vc, T.sigma_of(128), lambda a: a)
    # library attention in BF16 on the same device agrees too
    qd, kd, vd = T.to_dev(q), T.to_dev(kc), T.to_dev(vc)
    ref = torch.nn.functional.scaled_dot_product_attention(qd.float(), kd.float(), vd.float())
    out = B.kvq_attn_corrected(g, qd, kd, vd, T.sigma_of(128), B.KVQ_CORRECTION_ON, cache_len=0)
    assert (out.float() - ref).abs().max().item() < 2e-2


def test_zero_steps_make_correction_a_noop(B):
    w = inputs.Workload("zstep", 301, 1, 2, 128, 96, 0, 2, 32, 0)
    g, o, n, sel = _build(B, w, 2, tokens=100, cap=256)
    g.views()["k_scale"].zero_()
    o.k_scale[:] = 0
    q, kc, vc = inputs.make_chunk(w, 3)
    qd, kd, vd = T.to_dev(q), T.to_dev(kc), T.to_dev(vc)
    for _, kflag in kernels(B, 128):
        on = B.kvq_attn_corrected(g, qd, kd, vd, T.sigma_of(128), B.KVQ_CORRECTION_ON | kflag)
        off = B.kvq_attn_corrected(g, qd, kd, vd, T.sigma_of(128), B.KVQ_CORRECTION_OFF | kflag)
        assert torch.equal(on, off) and torch.isfinite(on.float()).all()
    _compare(B, g, o, n, q, kc, vc, T.sigma_of(128), sel)


def test_rotation_off_window_scale_and_strides(B):
    # no rotation (Eq. (15) with the unrotated query), a window inside the cache, a softmax
    # scale other than 1/sqrt(d), and non-contiguous q/k/v/out
    w = inputs.Workload("norot", 302, 1, 4, 128, 130, 0, 2, 64, 0, k_outliers=2, k_outlier_scale=4.0)
    g, o, n, sel = _build(B, w, 2, tokens=120, rotate=False, cap=256)
    q, kc, vc = inputs.make_chunk(w, 4)
    sigma = 0.05
    _compare(B, g, o, 150, q, kc, vc, sigma, sel, begin=48)
    # strided tensors: [B, n, H, d] storage viewed as [B, H, n, d]
    qd, kd, vd = [T.to_dev(a).permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3) for a in (q, kc, vc)]
    out = torch.empty_like(qd)
    assert not out.is_contiguous()
    B.kvq_attn_corrected(g, qd, kd, vd, sigma, B.KVQ_CORRECTION_ON, cache_begin=48, cache_len=150, out=out)
    want = O.attn_corrected(o, 48, 150, q, kc, vc, sigma, correction=True)["out"]
    T.assert_attn_close(T.from_dev_bf16(out), want, "strided")


def test_auto_dispatch_and_forced_kernel_errors(B):
    # head_dim 128 -> tcgen05 kernel, head_dim 64 -> warp-level kernel; forcing tcgen05 on 64 is refused
    for d in (64, 128):
        w = inputs.Workload("auto", 310 + d, 1, 2, d, 140, 0, 2, 64, 0)
        g, o, n, sel = _build(B, w, 2, tokens=90, cap=256)
        q, kc, vc = inputs.make_chunk(w, 3)
        _compare(B, g, o, n, q, kc, vc, T.sigma_of(d), sel, flags_list=[("auto", B.KVQ_KERNEL_AUTO)])
        if d == 64:
            with pytest.raises(B.KvqError) as e:
                B.kvq_attn_corrected(g, T.to_dev(q), T.to_dev(kc), T.to_dev(vc), 0.125,
                                     B.KVQ_CORRECTION_ON | B.KVQ_KERNEL_TCGEN05)
            assert e.value.status == B.KVQ_ERR_UNSUPPORTED


@pytest.mark.parametrize("m,bits,expect", [(140, 2, "KVQ_KERNEL_TCGEN05"), (256, 2, "KVQ_KERNEL_TCGEN05"),
                                           (300, 2, "KVQ_KERNEL_TCGEN05_PAIR"), (1560, 2, "KVQ_KERNEL_TCGEN05"),
                                           (1560, 4, "KVQ_KERNEL_TCGEN05_PAIR"), (2048, 2, "KVQ_KERNEL_TCGEN05_PAIR")])
def test_auto_picks_the_pair_kernel_by_padded_rows(B, m, bits, expect):
    """KVQ_KERNEL_AUTO on head_dim 128: the pair kernel unless its 512-row units pad the chunk too far beyond a
    multiple of 256 (a little further at 4 bits).  The two tcgen05 kernels differ in a quarter of their exponentials, so the bytes of the output
    tell which one ran (and both are checked against the oracle elsewhere)."""
    w = inputs.Workload("autopair", 77, 1, 2, 128, m, 1, bits, 64, 0)
    g, o, n, sel = _build(B, w, 1, tokens=700, cap=768)
    q, kc, vc = inputs.make_chunk(w, 2)
    qd, kd, vd = T.to_dev(q), T.to_dev(kc), T.to_dev(vc)
    outs = {k: B.kvq_attn_corrected(g, qd, kd, vd, T.sigma_of(128), B.KVQ_CORRECTION_ON | getattr(B, k), cache_len=n)
            for k in ("KVQ_KERNEL_AUTO", "KVQ_KERNEL_TCGEN05", "KVQ_KERNEL_TCGEN05_PAIR")}
    torch.cuda.synchronize()
    assert not torch.equal(outs["KVQ_KERNEL_TCGEN05"].view(torch.int16), outs["KVQ_KERNEL_TCGEN05_PAIR"].view(torch.int16))
    assert torch.equal(outs["KVQ_KERNEL_AUTO"].view(torch.int16), outs[expect].view(torch.int16))


def test_correction_lowers_cached_mass_and_mass_is_consistent(B):
    w = inputs.WORKLOADS["tiny"]
    g, o, n, sel = _build(B, w, 4)
    q, kc, vc = inputs.make_chunk(w, 4)
    qd, kd, vd = T.to_dev(q), T.to_dev(kc), T.to_dev(vc)
    masses = {}
    for corr in (B.KVQ_CORRECTION_ON, B.KVQ_CORRECTION_OFF):
        mass = torch.zeros(q.shape[:3], dtype=torch.float32, device="cuda")
        B.kvq_attn_corrected(g, qd, kd, vd, 0.125, corr, cached_mass=mass)
        masses[corr] = mass
    assert (masses[B.KVQ_CORRECTION_ON] < masses[B.KVQ_CORRECTION_OFF]).all()
    assert (masses[B.KVQ_CORRECTION_OFF] <= 1).all() and (masses[B.KVQ_CORRECTION_ON] > 0).all()


@pytest.mark.parametrize("name", ["sweep_int4", "sweep_int2"])
@pytest.mark.parametrize("seed", [0, 1, 2])
def test_sweep_config_full_rows(B, name, seed):
    w = inputs.with_seed(inputs.WORKLOADS[name], seed)
    units = [(0, 0), (0, 7), (0, 15)] if seed == 0 else [(0, 3)]
    g, o, n, sel = _build(B, w, w.cached_chunks, units=units)
    q, kc, vc = inputs.make_chunk(w, w.cached_chunks)
    _compare(B, g, o, n, q, kc, vc, T.sigma_of(w.head_dim), sel)


@pytest.mark.parametrize("name", ["dit", "long", "prefix"])
def test_large_configs_every_head(B, name):
    """Full-size launch, in the configuration bench.py times; the oracle on EVERY head, on rows that touch every
    128-row tile (first, middle, last row of each, the ragged tail included) plus a few random ones.  The
    oracle works head by head on host threads (one oracle cache per head), so its time stays in seconds."""
    import concurrent.futures as cf
    w = inputs.WORKLOADS[name]
    heads = [(b, h) for b in range(w.batch) for h in range(w.heads)]
    g = B.Cache(w.batch, w.heads, w.head_dim, w.bits, w.group, w.capacity)
    caches = [O.Cache(1, 1, w.head_dim, w.bits, w.group, w.capacity) for _ in heads]
    one = lambda a, u: a[u[0]:u[0] + 1, u[1]:u[1] + 1]
    n = 0
    with cf.ThreadPoolExecutor(max_workers=16) as pool:
        for c in range(w.cached_chunks):
            _, k, v = inputs.make_chunk(w, c, need_q=False)
            B.kvq_quantize_append(g, T.to_dev(k), T.to_dev(v))
            lens = list(pool.map(lambda i: O.quantize_append(caches[i], n, one(k, heads[i]), one(v, heads[i])), range(len(heads))))
            n = lens[0]
        q, kc, vc = inputs.make_chunk(w, w.cached_chunks)
        rows = inputs.sample_rows(w.chunk, 128, 8, seed=w.cfg_id)
        sigma = T.sigma_of(w.head_dim)
        qd, kd, vd = T.to_dev(q), T.to_dev(kc), T.to_dev(vc)
        got_by_kernel = {}
        for kname, kflag in (("tcgen05", B.KVQ_KERNEL_TCGEN05), ("tcgen05_pair", B.KVQ_KERNEL_TCGEN05_PAIR)):
            lse = torch.zeros(q.shape[:3], dtype=torch.float32, device="cuda")
            mass = torch.zeros_like(lse)
            status = torch.zeros(1, dtype=torch.int32, device="cuda")
            out = B.kvq_attn_corrected(g, qd, kd, vd, sigma, B.KVQ_CORRECTION_ON | kflag, cache_len=n,
                                       lse=lse, cached_mass=mass, status_word=status)
            torch.cuda.synchronize()
            assert int(status.item()) == 0, kname
            got_by_kernel[kname] = (T.from_dev_bf16(out), lse.cpu().numpy().astype(np.float64),
                                    mass.cpu().numpy().astype(np.float64))
        want = list(pool.map(lambda i: O.attn_corrected(caches[i], 0, n, one(q, heads[i]), one(kc, heads[i]),
                                                         one(vc, heads[i]), sigma, correction=True, rows=rows),
                             range(len(heads))))
    for kname, (got, lse_h, mass_h) in got_by_kernel.items():
        worst = (0.0, 0.0)
        for (b, h), wnt in zip(heads, want):
            rel, mx = T.assert_attn_close(got[b, h][rows], wnt["out"][0], f"{name} {kname} head ({b},{h})")
            worst = (max(worst[0], rel), max(worst[1], mx))
            assert np.abs(lse_h[b, h][rows] - wnt["lse"][0]).max() < 2e-2, (kname, b, h)
            assert np.abs(mass_h[b, h][rows] - wnt["cached_mass"][0]).max() < 1e-2, (kname, b, h)
        print(f"{name} {kname}: worst rel-L2 {worst[0]:.2e}, worst max-abs {worst[1]:.2e} over {len(heads)} heads x {len(rows)} rows")
    # the correction-off kernels on two heads
    for i in (0, len(heads) - 1):
        b, h = heads[i]
        wnt = O.attn_corrected(caches[i], 0, n, one(q, heads[i]), one(kc, heads[i]), one(vc, heads[i]), sigma,
                               correction=False, rows=rows)
        for kname, kflag in (("tcgen05", B.KVQ_KERNEL_TCGEN05), ("tcgen05_pair", B.KVQ_KERNEL_TCGEN05_PAIR)):
            out_off = B.kvq_attn_corrected(g, qd, kd, vd, sigma, B.KVQ_CORRECTION_OFF | kflag, cache_len=n)
            T.assert_attn_close(T.from_dev_bf16(out_off)[b, h][rows], wnt["out"][0], f"{name} {kname} head ({b},{h}) uncorrected")


def test_pipeline_config_steps(B):
    """Attend-then-append over the 16 successive chunks; the attention is checked at steps 0, 1, 2, 5 and 15
    (step 0 has an empty cache, step 15 is the shape bench.py times: 30 720 cached tokens)."""
    w = inputs.WORKLOADS["pipeline"]
    units = [(0, 0), (1, 20)]
    sel = lambda a: np.stack([a[b, h] for (b, h) in units])[None]
    g = B.Cache(w.batch, w.heads, w.head_dim, w.bits, w.group, w.capacity)
    o = O.Cache(1, len(units), w.head_dim, w.bits, w.group, w.capacity)
    rows = inputs.sample_rows(w.chunk, 128, 16, seed=5)
    n = 0
    for step in range(16):
        check = step in (0, 1, 2, 5, 15)
        q, k, v = inputs.make_chunk(w, step, need_q=check)
        if check:
            _compare(B, g, o, n, q, k, v, T.sigma_of(w.head_dim), sel, rows=rows,
                     flags_list=None if step < 15 else [("tcgen05", B.KVQ_KERNEL_TCGEN05), ("tcgen05_pair", B.KVQ_KERNEL_TCGEN05_PAIR)])
        if step < 15:
            B.kvq_quantize_append(g, T.to_dev(k), T.to_dev(v))
            n = O.quantize_append(o, n, sel(k), sel(v))
    assert n == 15 * w.chunk
    T.assert_cache_equal(T.gpu_cache_arrays(g, n), o, n, units=units)


def test_chunk_shared_by_all_heads_goes_to_the_warp_level_kernel(B):
    """K_cur / V_cur with a head stride of 0 (one chunk expanded over the heads): TMA cannot address that, so the
    automatic choice is the warp-level kernel, and forcing the tcgen05 kernel is refused before any launch."""
    w = inputs.Workload("shared", 340, 1, 3, 128, 150, 0, 2, 64, 0, k_outliers=2, k_outlier_scale=4.0)
    g, o, n, sel = _build(B, w, 2, tokens=140, cap=384)
    q, kc, vc = inputs.make_chunk(w, 5)
    kc[:] = kc[:, :1]; vc[:] = vc[:, :1]                     # every head sees head 0's chunk
    qd = T.to_dev(q)
    kd = T.to_dev(kc[:, :1]).expand(1, 3, 150, 128)
    vd = T.to_dev(vc[:, :1]).expand(1, 3, 150, 128)
    assert kd.stride(1) == 0
    sigma = T.sigma_of(128)
    out = B.kvq_attn_corrected(g, qd, kd, vd, sigma, B.KVQ_CORRECTION_ON, cache_len=n)
    want = O.attn_corrected(o, 0, n, q, kc, vc, sigma, correction=True)["out"]
    T.assert_attn_close(T.from_dev_bf16(out), want, "expanded chunk")
    with pytest.raises(B.KvqError) as e:
        B.kvq_attn_corrected(g, qd, kd, vd, sigma, B.KVQ_CORRECTION_ON | B.KVQ_KERNEL_TCGEN05, cache_len=n)
    assert e.value.status == B.KVQ_ERR_UNSUPPORTED


@pytest.mark.parametrize("d,bits,group,dist", [(128, 2, 32, "student_t3"), (128, 2, 128, "normal"), (64, 4, 64, "normal")])
def test_exact_correction_matches_the_oracle(B, d, bits, group, dist):
    """KVQ_CORRECTION_EXACT: the bias of Eq. (12) (warp-level kernel, a table over the 127 E4M3 step values) against
    the oracle's exact form, on inputs where it differs visibly from the Taylor form."""
    w = inputs.Workload("exact", 610 + d + group, 1, 2, d, 140, 0, bits, group, 4, k_dist=dist, k_outliers=8, k_outlier_scale=10.0)
    g, o, n, sel = _build(B, w, 3, tokens=100, cap=384)
    q, kc, vc = inputs.make_chunk(w, 6)
    qd, kd, vd = T.to_dev(q), T.to_dev(kc), T.to_dev(vc)
    sigma = T.sigma_of(d)
    want = O.attn_corrected(o, 0, n, q, kc, vc, sigma, correction=True, exact=True)
    taylor = O.attn_corrected(o, 0, n, q, kc, vc, sigma, correction=True)
    mass = torch.zeros(q.shape[:3], dtype=torch.float32, device="cuda")
    out = B.kvq_attn_corrected(g, qd, kd, vd, sigma, B.KVQ_CORRECTION_EXACT, cached_mass=mass)
    torch.cuda.synchronize()
    got = T.from_dev_bf16(out).reshape(want["out"].shape)
    T.assert_attn_close(got, want["out"], "exact correction")
    assert np.abs(mass.cpu().numpy().reshape(want["cached_mass"].shape) - want["cached_mass"]).max() < 1e-2
    if dist == "student_t3":      # here the two forms are far apart, so the test cannot pass by computing the Taylor one
        assert np.abs(taylor["cached_mass"] - want["cached_mass"]).max() > 0.05
    # the tcgen05 kernel does not have it
    with pytest.raises(B.KvqError) as e:
        B.kvq_attn_corrected(g, qd, kd, vd, sigma, B.KVQ_CORRECTION_EXACT | B.KVQ_KERNEL_TCGEN05)
    assert e.value.status == B.KVQ_ERR_UNSUPPORTED
    with pytest.raises(B.KvqError) as e:
        B.kvq_attn_corrected(g, qd, kd, vd, sigma, B.KVQ_CORRECTION_EXACT | B.KVQ_CORRECTION_ON)
    assert e.value.status == B.KVQ_ERR_INVALID_ARG
