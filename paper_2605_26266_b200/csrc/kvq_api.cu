// C-ABI entry points of libkvq: argument validation and dispatch to the kernels.
#include "kvq_common.cuh"

namespace kvq {

static thread_local int g_last_cuda_error = 0;

int record_cuda_error(cudaError_t e) {
  g_last_cuda_error = (int)e;
  return KVQ_ERR_CUDA;
}

int current_device(int* dev) {
  KVQ_CUDA_TRY(cudaGetDevice(dev));
  if (*dev < 0 || *dev >= kMaxDevices) return KVQ_ERR_UNSUPPORTED;
  return KVQ_OK;
}

int device_sm_count(int* sms) {
  static std::atomic<int> cache[kMaxDevices] = {};
  int dev = 0;
  const int r = current_device(&dev);
  if (r != KVQ_OK) return r;
  int n = cache[dev].load(std::memory_order_relaxed);
  if (n == 0) {
    KVQ_CUDA_TRY(cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev));
    if (n <= 0) return record_cuda_error(cudaErrorInvalidDevice);
    cache[dev].store(n, std::memory_order_relaxed);
  }
  *sms = n;
  return KVQ_OK;
}

int check_shape(const kvq_cache_desc* d) {
  if (!d) return KVQ_ERR_INVALID_ARG;
  if (d->batch <= 0 || d->heads <= 0 || d->head_dim <= 0 || d->group <= 0 || d->capacity <= 0)
    return KVQ_ERR_INVALID_ARG;
  if (d->head_dim % d->group != 0) return KVQ_ERR_INVALID_ARG;
  if (d->head_dim != 64 && d->head_dim != 128) return KVQ_ERR_UNSUPPORTED;
  if ((int64_t)d->batch * d->heads > 65535) return KVQ_ERR_UNSUPPORTED;     // (batch, head) is a grid dimension
  if (d->bits != 2 && d->bits != 4) return KVQ_ERR_UNSUPPORTED;
  if (d->group != 32 && d->group != 64 && d->group != 128) return KVQ_ERR_UNSUPPORTED;
  if (d->capacity % 128 != 0) return KVQ_ERR_INVALID_ARG;
  if (d->flags & ~(KVQ_ROTATE_K | KVQ_ROTATE_V | KVQ_RING | KVQ_K_PER_CHANNEL)) return KVQ_ERR_INVALID_ARG;
  return KVQ_OK;
}

int check_desc(const kvq_cache_desc* d) {
  int r = check_shape(d);
  if (r != KVQ_OK) return r;
  const void* ptrs[6] = {d->k_codes, d->v_codes, d->k_scale, d->v_scale, d->k_zero, d->v_zero};
  for (const void* p : ptrs) {
    if (!p) return KVQ_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(p) % 16 != 0) return KVQ_ERR_ALIGNMENT;
  }
  return KVQ_OK;
}

int check_tensor(const void* p, kvq_strides s) {
  if (!p) return KVQ_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(p) % 16 != 0) return KVQ_ERR_ALIGNMENT;
  if (s.b < 0 || s.h < 0 || s.t <= 0) return KVQ_ERR_INVALID_ARG;
  if (s.b % 8 != 0 || s.h % 8 != 0 || s.t % 8 != 0) return KVQ_ERR_ALIGNMENT;
  return KVQ_OK;
}

static int check_attn_args(const kvq_cache_desc* d, int64_t cache_begin, int64_t cache_len,
                           int64_t m_tokens, int64_t n_cur, uint32_t flags) {
  int r = check_shape(d);
  if (r != KVQ_OK) return r;
  if (cache_begin < 0 || cache_len < 0 || m_tokens < 0 || n_cur < 1) return KVQ_ERR_INVALID_ARG;
  if (cache_begin % 16 != 0) return KVQ_ERR_ALIGNMENT;
  if ((d->flags & KVQ_K_PER_CHANNEL) && cache_begin % d->group != 0) return KVQ_ERR_ALIGNMENT;   // windows start on a block
  if ((d->flags & KVQ_K_PER_CHANNEL) && (flags & KVQ_CORRECTION_EXACT)) return KVQ_ERR_UNSUPPORTED;
  // linear cache: the window ends inside the capacity; ring cache: it has at most `capacity` tokens
  if (((d->flags & KVQ_RING) ? cache_len : cache_begin + cache_len) > d->capacity) return KVQ_ERR_CAPACITY;
  if (m_tokens > 0x7FFFFFFFLL || n_cur > 0x7FFFFFFFLL || cache_len > 0x7FFFFFFFLL) return KVQ_ERR_UNSUPPORTED;
  const uint32_t kern = flags & KVQ_KERNEL_MASK;
  if (kern != KVQ_KERNEL_AUTO && kern != KVQ_KERNEL_MMA_SYNC && kern != KVQ_KERNEL_TCGEN05 && kern != KVQ_KERNEL_TCGEN05_PAIR)
    return KVQ_ERR_INVALID_ARG;
  if (flags & ~(KVQ_CORRECTION_ON | KVQ_CORRECTION_EXACT | KVQ_KERNEL_MASK)) return KVQ_ERR_INVALID_ARG;
  if ((flags & KVQ_CORRECTION_ON) && (flags & KVQ_CORRECTION_EXACT)) return KVQ_ERR_INVALID_ARG;   // one form or the other
  return KVQ_OK;
}

// KVQ_ROTATE_V: bytes at the front of the workspace for the rotated copy of the current chunk's values
// (dense [batch, heads, n_cur, head_dim] BF16, rounded up to 256).  Nothing without cached keys: the output
// then never leaves the unrotated space.
static size_t rotv_bytes(const kvq_cache_desc* d, int64_t cache_len, int64_t m_tokens, int64_t n_cur) {
  if (!(d->flags & KVQ_ROTATE_V) || cache_len <= 0 || m_tokens <= 0) return 0;
  return ((size_t)d->batch * d->heads * (size_t)n_cur * d->head_dim * 2 + 255) / 256 * 256;
}

static bool use_tcgen05(const kvq_cache_desc* d, int64_t m_tokens, int64_t n_cur, uint32_t flags, int* err) {
  const uint32_t kern = flags & KVQ_KERNEL_MASK;
  *err = KVQ_OK;
  if (kern == KVQ_KERNEL_MMA_SYNC) return false;
  // the exact correction (a table look-up per score and group) exists in the warp-level kernel only
  const bool ok = attn_tcgen05_supports(d, m_tokens, n_cur) && !(flags & KVQ_CORRECTION_EXACT) && !(d->flags & KVQ_K_PER_CHANNEL);
  if ((kern == KVQ_KERNEL_TCGEN05 || kern == KVQ_KERNEL_TCGEN05_PAIR) && !ok) *err = KVQ_ERR_UNSUPPORTED;
  return ok;
}
// Which tcgen05 kernel: the one asked for, else (KVQ_KERNEL_AUTO) the pair kernel unless its units of 512 query
// rows pad the chunk so much more than units of 256 that its measured advantage per row is lost (12 % or more at
// 2 bits; more at 4 bits, where there is more dequantization work to halve: M = 1560 pads to 2048 against 1792,
// and the pair kernel measures 1 % slower at 2 bits, 3 % faster at 4).
static bool is_pair(const kvq_cache_desc* d, uint32_t flags, int64_t m_tokens) {
  const uint32_t kern = flags & KVQ_KERNEL_MASK;
  if (kern != KVQ_KERNEL_AUTO) return kern == KVQ_KERNEL_TCGEN05_PAIR;
  const int64_t rows_pair = (m_tokens + 511) / 512 * 512, rows_single = (m_tokens + 255) / 256 * 256;
  return rows_pair * (d->bits == 4 ? 86 : 88) <= rows_single * 100;
}

// Checks shared by the two attention entry points, then the argument block the launchers take.
static int check_attn_call(const kvq_cache_desc* d, int64_t cache_begin, int64_t cache_len, const void* q,
                           kvq_strides qs, const void* k_cur, const void* v_cur, kvq_strides kvs, int64_t m_tokens,
                           int64_t n_cur, const void* out, kvq_strides os, float softmax_scale, uint32_t flags) {
  int r = check_attn_args(d, cache_begin, cache_len, m_tokens, n_cur, flags);
  if (r != KVQ_OK) return r;
  if ((r = check_desc(d)) != KVQ_OK) return r;
  if ((r = check_tensor(q, qs)) != KVQ_OK) return r;
  if ((r = check_tensor(k_cur, kvs)) != KVQ_OK) return r;
  if ((r = check_tensor(v_cur, kvs)) != KVQ_OK) return r;
  if ((r = check_tensor(out, os)) != KVQ_OK) return r;
  if (!(softmax_scale > 0.0f) || !(softmax_scale < 1e30f)) return KVQ_ERR_INVALID_ARG;
  return KVQ_OK;
}

static AttnArgs make_attn_args(const kvq_cache_desc* d, int64_t cache_begin, int64_t cache_len, const void* q,
                               kvq_strides qs, const void* k_cur, const void* v_cur, kvq_strides kvs,
                               int64_t m_tokens, int64_t n_cur, void* out, kvq_strides os, float softmax_scale,
                               uint32_t flags, float* lse, float* cached_mass, void* workspace,
                               size_t workspace_bytes, int32_t* status_word, kvq_stream_t stream) {
  AttnArgs a;
  a.desc = d; a.cache_begin = cache_begin; a.cache_len = cache_len;
  a.q = q; a.qs = qs; a.k_cur = k_cur; a.v_cur = v_cur; a.kvs = kvs; a.vs = kvs;
  a.m_tokens = m_tokens; a.n_cur = n_cur; a.out = out; a.os = os;
  a.softmax_scale = softmax_scale; a.flags = flags; a.lse = lse; a.cached_mass = cached_mass;
  a.workspace = workspace; a.workspace_bytes = workspace_bytes; a.status_word = status_word;
  a.stream = (cudaStream_t)stream;
  return a;
}

}  // namespace kvq

using namespace kvq;

extern "C" {

int kvq_version(void) { return KVQ_VERSION; }

int kvq_last_cuda_error(void) { return g_last_cuda_error; }

const char* kvq_status_string(int status) {
  switch (status) {
    case KVQ_OK: return "ok";
    case KVQ_ERR_INVALID_ARG: return "invalid argument";
    case KVQ_ERR_UNSUPPORTED: return "unsupported shape or option";
    case KVQ_ERR_ALIGNMENT: return "pointer or stride alignment";
    case KVQ_ERR_CAPACITY: return "cache capacity exceeded";
    case KVQ_ERR_CUDA: return "CUDA error";
    case KVQ_ERR_TIMEOUT: return "device-side wait timed out";
    case KVQ_ERR_WORKSPACE: return "workspace missing or too small";
    default: return "unknown status";
  }
}

int kvq_status_word_result(int32_t word) { return word == 0 ? KVQ_OK : KVQ_ERR_TIMEOUT; }

int kvq_set_wait_budget_cycles(uint64_t cycles) {
  if (cycles > 0xFFFF0000ull) return KVQ_ERR_INVALID_ARG;     // waits compare 32-bit clock differences
  set_attn_wait_budget((uint32_t)cycles);
  return KVQ_OK;
}

int kvq_cache_bytes(const kvq_cache_desc* desc, size_t out_bytes[6]) {
  int r = check_shape(desc);
  if (r != KVQ_OK) return r;
  if (!out_bytes) return KVQ_ERR_INVALID_ARG;
  const size_t tok = (size_t)desc->batch * desc->heads * (size_t)desc->capacity;
  const size_t G = (size_t)groups_of(desc);
  out_bytes[0] = out_bytes[1] = tok * (size_t)code_bytes_of(desc);
  out_bytes[2] = out_bytes[3] = tok * G;
  out_bytes[4] = out_bytes[5] = tok * G * 2;
  return KVQ_OK;
}

int kvq_quantize_append(const kvq_cache_desc* desc, int64_t cache_len, const void* k_bf16,
                        const void* v_bf16, kvq_strides kv, int64_t n_tokens, kvq_stream_t stream) {
  int r = check_desc(desc);
  if (r != KVQ_OK) return r;
  if (cache_len < 0 || n_tokens < 0) return KVQ_ERR_INVALID_ARG;
  if (((desc->flags & KVQ_RING) ? n_tokens : cache_len + n_tokens) > desc->capacity) return KVQ_ERR_CAPACITY;
  if ((desc->flags & KVQ_K_PER_CHANNEL) && (cache_len % desc->group != 0 || n_tokens % desc->group != 0))
    return KVQ_ERR_ALIGNMENT;                          // per-channel keys come in whole blocks of `group` tokens
  if ((r = check_tensor(k_bf16, kv)) != KVQ_OK) return r;
  if ((r = check_tensor(v_bf16, kv)) != KVQ_OK) return r;
  if (n_tokens == 0) return KVQ_OK;
  return launch_quantize_append(desc, cache_len, k_bf16, v_bf16, kv, n_tokens, (cudaStream_t)stream);
}

int kvq_attn_workspace_bytes(const kvq_cache_desc* desc, int64_t cache_len, int64_t m_tokens,
                             int64_t n_cur, uint32_t flags, size_t* out_bytes) {
  if (!out_bytes) return KVQ_ERR_INVALID_ARG;
  int r = check_attn_args(desc, 0, cache_len, m_tokens, n_cur, flags);
  if (r != KVQ_OK) return r;
  int err;
  const bool tc = use_tcgen05(desc, m_tokens, n_cur, flags, &err);
  if (err != KVQ_OK) return err;
  *out_bytes = rotv_bytes(desc, cache_len, m_tokens, n_cur) + (tc ? attn_tcgen05_workspace_bytes(desc, cache_len, m_tokens, n_cur, is_pair(desc, flags, m_tokens)) : 0);
  return KVQ_OK;
}

int kvq_attn_kernel_launches(const kvq_cache_desc* desc, int64_t cache_len, int64_t m_tokens,
                             int64_t n_cur, uint32_t flags, int* out_count) {
  if (!out_count) return KVQ_ERR_INVALID_ARG;
  int r = check_attn_args(desc, 0, cache_len, m_tokens, n_cur, flags);
  if (r != KVQ_OK) return r;
  int err;
  const bool tc = use_tcgen05(desc, m_tokens, n_cur, flags, &err);
  if (err != KVQ_OK) return err;
  *out_count = (tc ? attn_tcgen05_kernel_launches(desc, cache_len, m_tokens, n_cur, is_pair(desc, flags, m_tokens)) : (m_tokens > 0 ? 1 : 0)) +
               (rotv_bytes(desc, cache_len, m_tokens, n_cur) ? 2 : 0);      // value pre-pass and output post-pass
  return KVQ_OK;
}

int kvq_attn_corrected(const kvq_cache_desc* desc, int64_t cache_begin, int64_t cache_len,
                       const void* q, kvq_strides q_strides, const void* k_cur, const void* v_cur,
                       kvq_strides kv_strides, int64_t m_tokens, int64_t n_cur, void* out_bf16,
                       kvq_strides o_strides, float softmax_scale, uint32_t flags, float* lse_out,
                       float* cached_mass_out, void* workspace, size_t workspace_bytes,
                       int32_t* status_word, kvq_stream_t stream) {
  int r = check_attn_call(desc, cache_begin, cache_len, q, q_strides, k_cur, v_cur, kv_strides, m_tokens, n_cur,
                          out_bf16, o_strides, softmax_scale, flags);
  if (r != KVQ_OK) return r;
  int err;
  bool tc = use_tcgen05(desc, m_tokens, n_cur, flags, &err);
  if (err != KVQ_OK) return err;
  AttnArgs a = make_attn_args(desc, cache_begin, cache_len, q, q_strides, k_cur, v_cur, kv_strides, m_tokens, n_cur,
                              out_bf16, o_strides, softmax_scale, flags, lse_out, cached_mass_out, workspace,
                              workspace_bytes, status_word, stream);
  // Tensors TMA cannot address (a stride of 0, as in a chunk expanded over heads) go to the warp-level kernel,
  // which takes any stride; a forced tcgen05 kernel fails here, before anything is launched.
  if (tc && m_tokens > 0 && !attn_tcgen05_addressable(a)) {
    if ((flags & KVQ_KERNEL_MASK) != KVQ_KERNEL_AUTO) return KVQ_ERR_UNSUPPORTED;
    tc = false;
  }
  const size_t rotv = rotv_bytes(desc, cache_len, m_tokens, n_cur);
  {
    const size_t need = rotv + (tc ? attn_tcgen05_workspace_bytes(desc, cache_len, m_tokens, n_cur, is_pair(desc, flags, m_tokens)) : 0);
    if (need > 0) {
      if (!workspace || workspace_bytes < need) return KVQ_ERR_WORKSPACE;
      if (reinterpret_cast<uintptr_t>(workspace) % 256 != 0) return KVQ_ERR_ALIGNMENT;
    }
  }
  if (m_tokens == 0) return KVQ_OK;
  if (tc)     // the launcher takes the choice between the two tcgen05 kernels from the flags
    a.flags = (a.flags & ~KVQ_KERNEL_MASK) | (is_pair(desc, flags, m_tokens) ? KVQ_KERNEL_TCGEN05_PAIR : KVQ_KERNEL_TCGEN05);
  if (rotv) {
    // values are cached rotated: bring the current chunk's values into the same space, attend, rotate the output back
    const kvq_strides dense{(int64_t)desc->heads * n_cur * desc->head_dim, n_cur * (int64_t)desc->head_dim, (int64_t)desc->head_dim};
    if ((r = launch_rotate_rows(desc, v_cur, kv_strides, workspace, dense, n_cur, false, a.stream)) != KVQ_OK) return r;
    a.v_cur = workspace; a.vs = dense;
    a.workspace = static_cast<uint8_t*>(workspace) + rotv; a.workspace_bytes = workspace_bytes - rotv;
  }
  r = tc ? launch_attn_tcgen05(a) : launch_attn_mma_sync(a);
  if (r == KVQ_OK && rotv) r = launch_rotate_rows(desc, out_bf16, o_strides, out_bf16, o_strides, m_tokens, true, a.stream);
  return r;
}

int kvq_attn_corrected_static_scratch(const kvq_cache_desc* desc, int64_t cache_begin, int64_t cache_len,
                                      const void* q, kvq_strides q_strides, const void* k_cur, const void* v_cur,
                                      kvq_strides kv_strides, int64_t m_tokens, int64_t n_cur, void* out_bf16,
                                      kvq_strides o_strides, float softmax_scale, uint32_t flags, float* lse_out,
                                      float* cached_mass_out, int32_t* status_word, kvq_stream_t stream) {
  if (flags & KVQ_KERNEL_MASK) return KVQ_ERR_INVALID_ARG;      // this entry point has one kernel only
  int r = check_attn_call(desc, cache_begin, cache_len, q, q_strides, k_cur, v_cur, kv_strides, m_tokens, n_cur,
                          out_bf16, o_strides, softmax_scale, flags);
  if (r != KVQ_OK) return r;
  if (!attn_tcgen05_supports(desc, m_tokens, n_cur) || (flags & KVQ_CORRECTION_EXACT) ||
      (desc->flags & (KVQ_ROTATE_V | KVQ_K_PER_CHANNEL)))
    return KVQ_ERR_UNSUPPORTED;
  if (m_tokens == 0) return KVQ_OK;
  const AttnArgs a = make_attn_args(desc, cache_begin, cache_len, q, q_strides, k_cur, v_cur, kv_strides, m_tokens,
                                    n_cur, out_bf16, o_strides, softmax_scale, flags, lse_out, cached_mass_out,
                                    nullptr, 0, status_word, stream);
  if (!attn_tcgen05_addressable(a)) return KVQ_ERR_UNSUPPORTED;
  return launch_attn_tcgen05_static(a);
}

int kvq_attn_weight_jsd(const kvq_cache_desc* desc, int64_t cache_begin, int64_t cache_len,
                        const void* q, kvq_strides q_strides, const void* k_cur, kvq_strides kcur_strides,
                        const void* k_cached_bf16, kvq_strides kcached_strides, int64_t m_tokens, int64_t n_cur,
                        float softmax_scale, uint32_t flags, float* jsd_out, kvq_stream_t stream) {
  int r = check_attn_args(desc, cache_begin, cache_len, m_tokens, n_cur, flags);
  if (r != KVQ_OK) return r;
  if ((r = check_desc(desc)) != KVQ_OK) return r;
  if (flags & (KVQ_CORRECTION_EXACT | KVQ_KERNEL_MASK)) return KVQ_ERR_UNSUPPORTED;      // Taylor form or none; one kernel
  if (desc->flags & KVQ_K_PER_CHANNEL) return KVQ_ERR_UNSUPPORTED;
  if (!jsd_out) return KVQ_ERR_INVALID_ARG;
  if (!(softmax_scale > 0.0f) || !(softmax_scale < 1e30f)) return KVQ_ERR_INVALID_ARG;
  if ((r = check_tensor(q, q_strides)) != KVQ_OK) return r;
  if ((r = check_tensor(k_cur, kcur_strides)) != KVQ_OK) return r;
  if (cache_len > 0 && (r = check_tensor(k_cached_bf16, kcached_strides)) != KVQ_OK) return r;
  if (m_tokens == 0) return KVQ_OK;
  const AttnArgs a = make_attn_args(desc, cache_begin, cache_len, q, q_strides, k_cur, k_cur, kcur_strides, m_tokens,
                                    n_cur, nullptr, q_strides, softmax_scale, flags, nullptr, nullptr, nullptr, 0,
                                    nullptr, stream);
  return launch_attn_jsd(a, k_cached_bf16, kcached_strides, jsd_out);
}

int kvq_unpack_codes(const kvq_cache_desc* desc, int which, int64_t begin, int64_t n,
                     uint8_t* out_codes, kvq_stream_t stream) {
  int r = check_desc(desc);
  if (r != KVQ_OK) return r;
  if ((which != 0 && which != 1) || begin < 0 || n < 0 || !out_codes) return KVQ_ERR_INVALID_ARG;
  if (((desc->flags & KVQ_RING) ? n : begin + n) > desc->capacity) return KVQ_ERR_CAPACITY;
  return launch_unpack_codes(desc, which, begin, n, out_codes, (cudaStream_t)stream);
}

}  // extern "C"
