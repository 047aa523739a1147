"""ctypes binding of libkvq.so: argument marshalling only.

Every function here has the name of the C entry point it calls (include/kvq.h)
and does nothing but turn torch tensors into device pointers, strides and a
stream handle.  All of the method's arithmetic runs in the CUDA kernels behind
the C ABI; there is no CPU or PyTorch fallback: if the library cannot be loaded,
importing this module raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libkvq.so")

KVQ_OK = 0
KVQ_ERR_INVALID_ARG, KVQ_ERR_UNSUPPORTED, KVQ_ERR_ALIGNMENT = -1, -2, -3
KVQ_ERR_CAPACITY, KVQ_ERR_CUDA, KVQ_ERR_TIMEOUT, KVQ_ERR_WORKSPACE = -4, -5, -6, -7
KVQ_ROTATE_K = 1
KVQ_RING = 2
KVQ_ROTATE_V = 4
KVQ_K_PER_CHANNEL = 8
KVQ_CORRECTION_OFF, KVQ_CORRECTION_ON, KVQ_CORRECTION_EXACT = 0, 1, 2
KVQ_KERNEL_AUTO, KVQ_KERNEL_MMA_SYNC, KVQ_KERNEL_TCGEN05, KVQ_KERNEL_TCGEN05_PAIR = 0, 1 << 8, 2 << 8, 3 << 8


class kvq_cache_desc(C.Structure):
    _fields_ = [
        ("batch", C.c_int32), ("heads", C.c_int32), ("head_dim", C.c_int32),
        ("bits", C.c_int32), ("group", C.c_int32), ("flags", C.c_uint32),
        ("capacity", C.c_int64),
        ("k_codes", C.c_void_p), ("v_codes", C.c_void_p),
        ("k_scale", C.c_void_p), ("v_scale", C.c_void_p),
        ("k_zero", C.c_void_p), ("v_zero", C.c_void_p),
        ("signs", C.c_void_p),
    ]


class kvq_strides(C.Structure):
    _fields_ = [("b", C.c_int64), ("h", C.c_int64), ("t", C.c_int64)]


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2605_26266_b200.build` "
            "(there is no fallback path)")
    lib = C.CDLL(LIB_PATH)
    lib.kvq_version.restype = C.c_int
    lib.kvq_last_cuda_error.restype = C.c_int
    lib.kvq_status_string.restype = C.c_char_p
    lib.kvq_status_string.argtypes = [C.c_int]
    lib.kvq_cache_bytes.restype = C.c_int
    lib.kvq_cache_bytes.argtypes = [C.POINTER(kvq_cache_desc), C.POINTER(C.c_size_t)]
    lib.kvq_quantize_append.restype = C.c_int
    lib.kvq_quantize_append.argtypes = [C.POINTER(kvq_cache_desc), C.c_int64, C.c_void_p, C.c_void_p,
                                        kvq_strides, C.c_int64, C.c_void_p]
    lib.kvq_attn_workspace_bytes.restype = C.c_int
    lib.kvq_attn_workspace_bytes.argtypes = [C.POINTER(kvq_cache_desc), C.c_int64, C.c_int64, C.c_int64,
                                             C.c_uint32, C.POINTER(C.c_size_t)]
    lib.kvq_attn_kernel_launches.restype = C.c_int
    lib.kvq_attn_kernel_launches.argtypes = [C.POINTER(kvq_cache_desc), C.c_int64, C.c_int64, C.c_int64,
                                             C.c_uint32, C.POINTER(C.c_int)]
    lib.kvq_attn_corrected.restype = C.c_int
    lib.kvq_attn_corrected.argtypes = [
        C.POINTER(kvq_cache_desc), C.c_int64, C.c_int64,
        C.c_void_p, kvq_strides, C.c_void_p, C.c_void_p, kvq_strides,
        C.c_int64, C.c_int64, C.c_void_p, kvq_strides,
        C.c_float, C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]
    lib.kvq_attn_corrected_static_scratch.restype = C.c_int
    lib.kvq_attn_corrected_static_scratch.argtypes = [
        C.POINTER(kvq_cache_desc), C.c_int64, C.c_int64,
        C.c_void_p, kvq_strides, C.c_void_p, C.c_void_p, kvq_strides,
        C.c_int64, C.c_int64, C.c_void_p, kvq_strides,
        C.c_float, C.c_uint32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    lib.kvq_status_word_result.restype = C.c_int
    lib.kvq_status_word_result.argtypes = [C.c_int32]
    lib.kvq_set_wait_budget_cycles.restype = C.c_int
    lib.kvq_set_wait_budget_cycles.argtypes = [C.c_uint64]
    lib.kvq_attn_weight_jsd.restype = C.c_int
    lib.kvq_attn_weight_jsd.argtypes = [
        C.POINTER(kvq_cache_desc), C.c_int64, C.c_int64, C.c_void_p, kvq_strides, C.c_void_p, kvq_strides,
        C.c_void_p, kvq_strides, C.c_int64, C.c_int64, C.c_float, C.c_uint32, C.c_void_p, C.c_void_p]
    lib.kvq_unpack_codes.restype = C.c_int
    lib.kvq_unpack_codes.argtypes = [C.POINTER(kvq_cache_desc), C.c_int, C.c_int64, C.c_int64,
                                     C.c_void_p, C.c_void_p]
    return lib


lib = _load()


class KvqError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib.kvq_status_string(status).decode()
        if status == KVQ_ERR_CUDA:
            msg += f" (cudaError {lib.kvq_last_cuda_error()})"
        super().__init__(f"{where}: {msg} [{status}]")


def _check(status: int, where: str):
    if status != KVQ_OK:
        raise KvqError(status, where)


def _strides(t: torch.Tensor) -> kvq_strides:
    assert t.dim() == 4 and t.stride(3) == 1, "tensor must be [batch, heads, tokens, head_dim] with unit inner stride"
    return kvq_strides(t.stride(0), t.stride(1), t.stride(2))


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t):
    return None if t is None else t.data_ptr()


class Cache:
    """Caller-side owner of the six device buffers of one quantized cache plus its descriptor."""

    def __init__(self, batch, heads, head_dim, bits, group, capacity, rotate_k=True, signs=None, device="cuda",
                 ring=False, rotate_v=False, k_per_channel=False):
        self.desc = kvq_cache_desc(batch, heads, head_dim, bits, group,
                                   (KVQ_ROTATE_K if rotate_k else 0) | (KVQ_RING if ring else 0)
                                   | (KVQ_ROTATE_V if rotate_v else 0) | (KVQ_K_PER_CHANNEL if k_per_channel else 0),
                                   capacity)
        sizes = kvq_cache_bytes(self.desc)
        self.buffers = [torch.zeros(n, dtype=torch.uint8, device=device) for n in sizes]
        (self.desc.k_codes, self.desc.v_codes, self.desc.k_scale, self.desc.v_scale,
         self.desc.k_zero, self.desc.v_zero) = [b.data_ptr() for b in self.buffers]
        self.signs = None
        if signs is not None:
            self.signs = torch.as_tensor(signs, dtype=torch.int8).to(device).contiguous()
            self.desc.signs = self.signs.data_ptr()
        self.length = 0
        self.workspace = None

    @property
    def groups(self):
        return self.desc.head_dim // self.desc.group

    def views(self):
        """The six buffers shaped [batch, heads, capacity, ...] (codes u8, scale u8, zero as int16 bits)."""
        d = self.desc
        B, H, Cp, G = d.batch, d.heads, d.capacity, self.groups
        kc, vc, ks, vs, kz, vz = self.buffers
        # per-channel keys: one row of head_dim steps / zero-points per block of `group` tokens
        kshape = (B, H, Cp // d.group, d.head_dim) if d.flags & KVQ_K_PER_CHANNEL else (B, H, Cp, G)
        return {
            "k_codes": kc.view(B, H, Cp, -1), "v_codes": vc.view(B, H, Cp, -1),
            "k_scale": ks.view(*kshape), "v_scale": vs.view(B, H, Cp, G),
            "k_zero": kz.view(torch.int16).view(*kshape), "v_zero": vz.view(torch.int16).view(B, H, Cp, G),
        }


def kvq_version() -> int:
    return lib.kvq_version()


def kvq_cache_bytes(desc: kvq_cache_desc):
    out = (C.c_size_t * 6)()
    _check(lib.kvq_cache_bytes(C.byref(desc), out), "kvq_cache_bytes")
    return list(out)


def kvq_quantize_append(cache: Cache, k: torch.Tensor, v: torch.Tensor, cache_len: int | None = None) -> int:
    """Appends the chunk k, v ([batch, heads, n, head_dim] BF16, CUDA) at token `cache_len`
    (default: the cache's running length) and returns the new length."""
    assert k.dtype == torch.bfloat16 and v.dtype == torch.bfloat16 and k.is_cuda and v.is_cuda
    assert k.shape == v.shape and k.stride() == v.stride()
    pos = cache.length if cache_len is None else cache_len
    n = k.shape[2]
    _check(lib.kvq_quantize_append(C.byref(cache.desc), pos, k.data_ptr(), v.data_ptr(), _strides(k), n, _stream()),
           "kvq_quantize_append")
    cache.length = pos + n
    return cache.length


def kvq_attn_workspace_bytes(cache: Cache, cache_len: int, m_tokens: int, n_cur: int, flags: int) -> int:
    out = C.c_size_t(0)
    _check(lib.kvq_attn_workspace_bytes(C.byref(cache.desc), cache_len, m_tokens, n_cur, flags, C.byref(out)),
           "kvq_attn_workspace_bytes")
    return out.value


def kvq_attn_kernel_launches(cache: Cache, cache_len: int, m_tokens: int, n_cur: int, flags: int) -> int:
    out = C.c_int(0)
    _check(lib.kvq_attn_kernel_launches(C.byref(cache.desc), cache_len, m_tokens, n_cur, flags, C.byref(out)),
           "kvq_attn_kernel_launches")
    return out.value


def kvq_attn_corrected(cache: Cache, q, k_cur, v_cur, softmax_scale, flags=KVQ_CORRECTION_ON,
                       cache_begin=0, cache_len=None, out=None, lse=None, cached_mass=None,
                       status_word=None):
    """out = corrected attention of q over [cache window ; current chunk].  Tensors are
    [batch, heads, tokens, head_dim] BF16 CUDA; returns `out` (allocated if not given)."""
    for t in (q, k_cur, v_cur):
        assert t.dtype == torch.bfloat16 and t.is_cuda
    assert k_cur.shape == v_cur.shape and k_cur.stride() == v_cur.stride()
    n_cache = cache.length - cache_begin if cache_len is None else cache_len
    if out is None:
        out = torch.empty_like(q, memory_format=torch.contiguous_format)
    m, n_cur = q.shape[2], k_cur.shape[2]
    need = kvq_attn_workspace_bytes(cache, n_cache, m, n_cur, flags)
    if need and (cache.workspace is None or cache.workspace.numel() < need):
        cache.workspace = torch.empty(need, dtype=torch.uint8, device=q.device)
    ws = cache.workspace if need else None
    _check(lib.kvq_attn_corrected(
        C.byref(cache.desc), cache_begin, n_cache, q.data_ptr(), _strides(q), k_cur.data_ptr(), v_cur.data_ptr(),
        _strides(k_cur), m, n_cur, out.data_ptr(), _strides(out), float(softmax_scale), flags,
        _ptr(lse), _ptr(cached_mass), _ptr(ws), ws.numel() if ws is not None else 0, _ptr(status_word), _stream()),
        "kvq_attn_corrected")
    return out


def kvq_attn_corrected_static_scratch(cache: Cache, q, k_cur, v_cur, softmax_scale, flags=KVQ_CORRECTION_ON,
                                      cache_begin=0, cache_len=None, out=None, lse=None, cached_mass=None,
                                      status_word=None):
    """kvq_attn_corrected without a workspace: split units keep their partial results in the scratch buffer
    built into the library.  `out` must be given by callers that may not allocate; it is allocated here only
    as a convenience when omitted."""
    for t in (q, k_cur, v_cur):
        assert t.dtype == torch.bfloat16 and t.is_cuda
    assert k_cur.shape == v_cur.shape and k_cur.stride() == v_cur.stride()
    n_cache = cache.length - cache_begin if cache_len is None else cache_len
    if out is None:
        out = torch.empty_like(q, memory_format=torch.contiguous_format)
    _check(lib.kvq_attn_corrected_static_scratch(
        C.byref(cache.desc), cache_begin, n_cache, q.data_ptr(), _strides(q), k_cur.data_ptr(), v_cur.data_ptr(),
        _strides(k_cur), q.shape[2], k_cur.shape[2], out.data_ptr(), _strides(out), float(softmax_scale), flags,
        _ptr(lse), _ptr(cached_mass), _ptr(status_word), _stream()), "kvq_attn_corrected_static_scratch")
    return out


def kvq_attn_weight_jsd(cache: Cache, q, k_cur, k_cached, softmax_scale, flags=KVQ_CORRECTION_ON, cache_begin=0,
                        cache_len=None, out=None):
    """Per-row JSD of the attention weights against those of the BF16 keys k_cached ([batch, heads, cache_len,
    head_dim], the keys the attended cache window was quantized from); returns float32 [batch, heads, rows]."""
    for t in (q, k_cur) + ((k_cached,) if k_cached is not None else ()):
        assert t.dtype == torch.bfloat16 and t.is_cuda
    n_cache = cache.length - cache_begin if cache_len is None else cache_len
    assert n_cache == 0 or k_cached.shape[2] == n_cache
    if out is None:
        out = torch.empty(q.shape[:3], dtype=torch.float32, device=q.device)
    kc_ptr, kc_str = (k_cached.data_ptr(), _strides(k_cached)) if n_cache else (None, kvq_strides(0, 0, 0))
    _check(lib.kvq_attn_weight_jsd(
        C.byref(cache.desc), cache_begin, n_cache, q.data_ptr(), _strides(q), k_cur.data_ptr(), _strides(k_cur),
        kc_ptr, kc_str, q.shape[2], k_cur.shape[2], float(softmax_scale), flags, out.data_ptr(), _stream()),
        "kvq_attn_weight_jsd")
    return out


def kvq_status_word_result(word: int) -> int:
    return lib.kvq_status_word_result(int(word))


def kvq_set_wait_budget_cycles(cycles: int) -> None:
    _check(lib.kvq_set_wait_budget_cycles(int(cycles)), "kvq_set_wait_budget_cycles")


def kvq_unpack_codes(cache: Cache, which: int, begin: int, n: int) -> torch.Tensor:
    d = cache.desc
    out = torch.empty((d.batch, d.heads, n, d.head_dim), dtype=torch.uint8, device=cache.buffers[0].device)
    _check(lib.kvq_unpack_codes(C.byref(d), which, begin, n, out.data_ptr(), _stream()), "kvq_unpack_codes")
    return out
