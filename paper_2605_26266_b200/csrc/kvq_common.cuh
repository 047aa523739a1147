// Shared host/device helpers of libkvq (internal; not part of the C ABI).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "kvq.h"

namespace kvq {

// Records a failing CUDA runtime call for kvq_last_cuda_error() and maps it to KVQ_ERR_CUDA.
int record_cuda_error(cudaError_t e);

#define KVQ_CUDA_TRY(expr)                                   \
  do {                                                       \
    cudaError_t kvq_e_ = (expr);                             \
    if (kvq_e_ != cudaSuccess) return ::kvq::record_cuda_error(kvq_e_); \
  } while (0)

// Per-device host state.  One process may drive several GPUs, and several threads may call into the library:
// whatever is looked up or configured once is kept per device ordinal, in atomics (a race only repeats an
// idempotent CUDA call).
constexpr int kMaxDevices = 64;
// Ordinal of the calling thread's current device; KVQ_ERR_UNSUPPORTED beyond kMaxDevices.
int current_device(int* dev);
// Multiprocessor count of the current device (looked up once per device).
int device_sm_count(int* sms);
// "Has this been set up on the current device?" for one kernel instantiation: declare one static PerDevice per
// instantiation; first() is true until done() has been called on that device.
struct PerDevice {
  std::atomic<unsigned char> flag[kMaxDevices] = {};
  bool first(int dev) const { return flag[dev].load(std::memory_order_acquire) == 0; }
  void done(int dev) { flag[dev].store(1, std::memory_order_release); }
};

// Shape part of the descriptor check (no pointers).
int check_shape(const kvq_cache_desc* d);
// Shape + the six buffer pointers.
int check_desc(const kvq_cache_desc* d);
int check_tensor(const void* p, kvq_strides s);

inline int groups_of(const kvq_cache_desc* d) { return d->head_dim / d->group; }
inline int code_bytes_of(const kvq_cache_desc* d) { return d->head_dim * d->bits / 8; }

// launchers implemented in the kernel translation units
int launch_quantize_append(const kvq_cache_desc* d, int64_t cache_len, const void* k, const void* v,
                           kvq_strides kv, int64_t n_tokens, cudaStream_t st);
int launch_unpack_codes(const kvq_cache_desc* d, int which, int64_t begin, int64_t n, uint8_t* out,
                        cudaStream_t st);

struct AttnArgs {
  const kvq_cache_desc* desc;
  int64_t cache_begin, cache_len;
  const void* q; kvq_strides qs;
  const void* k_cur; const void* v_cur; kvq_strides kvs;   // strides of k_cur
  kvq_strides vs;                                            // strides of v_cur
  int64_t m_tokens, n_cur;
  void* out; kvq_strides os;
  float softmax_scale;
  uint32_t flags;
  float* lse; float* cached_mass;
  void* workspace; size_t workspace_bytes;
  int32_t* status_word;
  cudaStream_t stream;
};
int launch_attn_mma_sync(const AttnArgs& a);
// Per-row Jensen-Shannon divergence of the attention weights against those of the BF16 keys k_ref (analysis kernel).
int launch_attn_jsd(const AttnArgs& a, const void* k_ref, kvq_strides ref_strides, float* jsd_out);
// y = (1/sqrt d) H (signs . x) per row (inverse: x = signs . ((1/sqrt d) H y)), BF16 [batch, heads, tokens, head_dim]
int launch_rotate_rows(const kvq_cache_desc* d, const void* src, kvq_strides ss, void* dst, kvq_strides ds,
                       int64_t tokens, bool inverse, cudaStream_t st);
// tcgen05 kernel: returns KVQ_ERR_UNSUPPORTED for shapes it does not cover.
bool attn_tcgen05_supports(const kvq_cache_desc* d, int64_t m_tokens, int64_t n_cur);
// Can TMA address the call's Q, K_cur, V_cur (no zero stride in a real dimension, byte strides below 2^40)?
bool attn_tcgen05_addressable(const AttnArgs& a);
// pair: the CTA-pair form of the kernel (KVQ_KERNEL_TCGEN05_PAIR), which plans 512-row units over SM pairs
size_t attn_tcgen05_workspace_bytes(const kvq_cache_desc* d, int64_t cache_len, int64_t m_tokens, int64_t n_cur, bool pair);
int attn_tcgen05_kernel_launches(const kvq_cache_desc* d, int64_t cache_len, int64_t m_tokens, int64_t n_cur, bool pair);
int launch_attn_tcgen05(const AttnArgs& a);
// Cycle budget of the tcgen05 kernel's device-side waits for later launches (0 = the default of about a second).
void set_attn_wait_budget(uint32_t cycles);
// Same kernel, partial results of split units in the library's built-in scratch buffer (no caller workspace).
int launch_attn_tcgen05_static(const AttnArgs& a);

#ifdef __CUDACC__
// ---- device-side number-format helpers -------------------------------------------------

// FP32 -> E4M3 byte, round-to-nearest-even, saturating to +-448 (hardware conversion).
__device__ __forceinline__ uint32_t f32_to_e4m3_byte(float x) {
  uint16_t r;
  asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(0.0f), "f"(x));
  return r & 0xFFu;
}

// E4M3 byte -> FP32 (exact).
__device__ __forceinline__ float e4m3_byte_to_f32(uint32_t b) {
  uint32_t h2;
  uint16_t in = (uint16_t)(b & 0xFFu);
  asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"(in));
  __half lo = __ushort_as_half((unsigned short)(h2 & 0xFFFFu));
  return __half2float(lo);
}

__device__ __forceinline__ float bf16_bits_to_f32(uint32_t bits16) { return __uint_as_float(bits16 << 16); }

__device__ __forceinline__ uint32_t f32_to_bf16_bits(float x) {
  return (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(x));
}
#endif

}  // namespace kvq
