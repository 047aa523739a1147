// Row-wise Hadamard rotation of a [batch, heads, tokens, head_dim] BF16 tensor, for caches whose values are
// stored rotated (KVQ_ROTATE_V).  Forward: y = (1/sqrt d) H (s . x), applied to the current chunk's values before
// the attention kernel so that they live in the same space as the cached ones.  Inverse: x = s . ((1/sqrt d) H y),
// applied in place to the attention output (H is symmetric and orthogonal after scaling, s is +-1).
// FP32 butterflies, stages h = 1, 2, 4, ... like every other rotation of this library; BF16 in, BF16 out.
// Eight channels per lane, head_dim / 8 lanes per row, 256-thread blocks.
#include <cuda_runtime.h>

#include "kvq_common.cuh"

namespace kvq {
namespace {

struct RowsParams {
  const uint16_t* src; int64_t s_sb, s_sh, s_st;
  uint16_t* dst; int64_t d_sb, d_sh, d_st;
  const int8_t* signs;
  int heads, tokens, inverse;
};

template <int D>
__global__ void __launch_bounds__(256) rotate_rows_kernel(const RowsParams p) {
  constexpr int kLanes = D / 8;                       // lanes per row: 8 or 16
  constexpr int kRowsPerBlock = 256 / kLanes;
  const int lane = threadIdx.x & 31;
  const int l = lane % kLanes;
  const int row = blockIdx.x * kRowsPerBlock + threadIdx.x / kLanes;
  const int bh = blockIdx.y, b = bh / p.heads, h = bh - b * p.heads;
  const bool valid = row < p.tokens;                  // no early exit: the shuffles need every lane
  float sgn[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) sgn[e] = p.signs ? (float)p.signs[l * 8 + e] : 1.0f;
  uint4 raw = make_uint4(0, 0, 0, 0);
  if (valid) raw = __ldg(reinterpret_cast<const uint4*>(p.src + (int64_t)b * p.s_sb + (int64_t)h * p.s_sh + (int64_t)row * p.s_st) + l);
  float x[8];
  x[0] = bf16_bits_to_f32(raw.x & 0xFFFFu); x[1] = bf16_bits_to_f32(raw.x >> 16);
  x[2] = bf16_bits_to_f32(raw.y & 0xFFFFu); x[3] = bf16_bits_to_f32(raw.y >> 16);
  x[4] = bf16_bits_to_f32(raw.z & 0xFFFFu); x[5] = bf16_bits_to_f32(raw.z >> 16);
  x[6] = bf16_bits_to_f32(raw.w & 0xFFFFu); x[7] = bf16_bits_to_f32(raw.w >> 16);
  if (!p.inverse) {
#pragma unroll
    for (int e = 0; e < 8; ++e) x[e] *= sgn[e];
  }
#pragma unroll
  for (int hh = 1; hh < 8; hh *= 2)
#pragma unroll
    for (int i = 0; i < 8; ++i)
      if ((i & hh) == 0) { const float a = x[i], c = x[i + hh]; x[i] = a + c; x[i + hh] = a - c; }
#pragma unroll
  for (int lm = 1; lm < kLanes; lm *= 2)
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const float o = __shfl_xor_sync(0xFFFFFFFFu, x[e], lm);
      x[e] = (l & lm) ? (o - x[e]) : (x[e] + o);
    }
  const float c_d = (D == 64) ? 0.125f : 0.08838834764831845f;
#pragma unroll
  for (int e = 0; e < 8; ++e) x[e] *= p.inverse ? c_d * sgn[e] : c_d;
  if (valid) {
    uint4 o;
    o.x = f32_to_bf16_bits(x[0]) | (f32_to_bf16_bits(x[1]) << 16);
    o.y = f32_to_bf16_bits(x[2]) | (f32_to_bf16_bits(x[3]) << 16);
    o.z = f32_to_bf16_bits(x[4]) | (f32_to_bf16_bits(x[5]) << 16);
    o.w = f32_to_bf16_bits(x[6]) | (f32_to_bf16_bits(x[7]) << 16);
    *(reinterpret_cast<uint4*>(p.dst + (int64_t)b * p.d_sb + (int64_t)h * p.d_sh + (int64_t)row * p.d_st) + l) = o;
  }
}

}  // namespace

int launch_rotate_rows(const kvq_cache_desc* d, const void* src, kvq_strides ss, void* dst, kvq_strides ds,
                       int64_t tokens, bool inverse, cudaStream_t st) {
  if (tokens <= 0) return KVQ_OK;
  const int64_t bh = (int64_t)d->batch * d->heads;
  if (bh > 65535 || tokens > 0x7FFFFFFFLL) return KVQ_ERR_UNSUPPORTED;
  RowsParams p;
  p.src = static_cast<const uint16_t*>(src); p.s_sb = ss.b; p.s_sh = ss.h; p.s_st = ss.t;
  p.dst = static_cast<uint16_t*>(dst); p.d_sb = ds.b; p.d_sh = ds.h; p.d_st = ds.t;
  p.signs = d->signs; p.heads = d->heads; p.tokens = (int)tokens; p.inverse = inverse ? 1 : 0;
  if (d->head_dim == 128) {
    rotate_rows_kernel<128><<<dim3((unsigned)((tokens + 15) / 16), (unsigned)bh), 256, 0, st>>>(p);
  } else if (d->head_dim == 64) {
    rotate_rows_kernel<64><<<dim3((unsigned)((tokens + 31) / 32), (unsigned)bh), 256, 0, st>>>(p);
  } else {
    return KVQ_ERR_UNSUPPORTED;
  }
  KVQ_CUDA_TRY(cudaGetLastError());
  return KVQ_OK;
}

}  // namespace kvq
