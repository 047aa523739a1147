// Jensen-Shannon divergence between the attention weights computed with the quantized cache (Algorithm 1, with
// or without the Taylor correction of Eq. (15) / Eq. (25)) and with the BF16 keys the cache was quantized from,
// per query row, over all keys [cached ; current] (the paper's appendix on attention JSD distributions).
//
// An analysis kernel, not part of the hot path: plain FP32 on the CUDA cores, nothing of size M x N is ever
// written.  A warp owns four query rows; its lanes walk the keys (key = lane, lane + 32, ...), each lane forming
// the four rows' scores against its key from the packed codes (dequantized in registers: (code - zero) * step)
// and from the BF16 key.  Two passes over the keys: the first takes both log-sum-exps (online maximum and sum per
// lane, combined by shuffles), the second accumulates
//   JSD = 1/2 sum_i p_i ln(p_i / m_i) + 1/2 sum_i r_i ln(r_i / m_i),   m_i = (p_i + r_i) / 2,
// with p the quantized-cache weights and r the BF16 ones.  Current-chunk keys have the same score in both
// (they are never quantized); their weights still differ through the two normalisers.
#include "kvq_common.cuh"

namespace kvq {
namespace {

constexpr int kWarps = 8;          // per block
constexpr int kRowsPerWarp = 4;
constexpr int kRowsPerBlock = kWarps * kRowsPerWarp;
constexpr float kLog2e = 1.4426950408889634f;

struct JParams {
  const uint16_t* q; int64_t q_sb, q_sh, q_st;
  const uint16_t* kcur; int64_t c_sb, c_sh, c_st;
  const uint16_t* kref; int64_t r_sb, r_sh, r_st;      // BF16 keys of the attended window
  const uint8_t* k_codes; const uint8_t* k_scale; const uint16_t* k_zero;
  const int8_t* signs;
  int64_t capacity, cache_begin;
  int heads, rotate, correction;
  int m_tokens, n_cached, n_cur;
  float sigma;
  float* jsd;
};

template <int D, int BITS, int GROUP>
__global__ void __launch_bounds__(kWarps * 32) attn_jsd_kernel(const JParams p) {
  constexpr int G = D / GROUP;
  constexpr int kCodesPerWord = 32 / BITS;
  // per warp: the four rows' rotated and plain queries, one float4 (row 0..3) per channel
  __shared__ float4 s_qrot[kWarps][D];
  __shared__ float4 s_q[kWarps][D];
  __shared__ float s_rot[kWarps][D];                    // butterfly scratch, one row at a time
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int bh = blockIdx.y, b = bh / p.heads, h = bh - b * p.heads;
  const int row0 = blockIdx.x * kRowsPerBlock + warp * kRowsPerWarp;
  if (row0 >= p.m_tokens) return;                       // whole warp; no block-wide barrier below

  // ---- set-up: load the four rows, rotate them in FP32 (Sylvester butterflies, then 1/sqrt d) ----
  float nu[kRowsPerWarp][G];
  for (int r = 0; r < kRowsPerWarp; ++r) {
    const int row = row0 + r;
    const bool valid = row < p.m_tokens;
    const uint16_t* qp = p.q + (int64_t)b * p.q_sb + (int64_t)h * p.q_sh + (int64_t)row * p.q_st;
    for (int c = lane; c < D; c += 32) {
      const float x = valid ? bf16_bits_to_f32(qp[c]) : 0.f;
      reinterpret_cast<float*>(&s_q[warp][c])[r] = x;
      s_rot[warp][c] = (p.rotate && p.signs) ? x * (float)p.signs[c] : x;
    }
    __syncwarp();
    if (p.rotate) {
      for (int hh = 1; hh < D; hh *= 2) {
        for (int i = lane; i < D / 2; i += 32) {
          const int lo = ((i / hh) * 2 * hh) + (i % hh);
          const float a = s_rot[warp][lo], c = s_rot[warp][lo + hh];
          s_rot[warp][lo] = a + c; s_rot[warp][lo + hh] = a - c;
        }
        __syncwarp();
      }
    }
    const float norm = p.rotate ? rsqrtf((float)D) : 1.f;
    for (int c = lane; c < D; c += 32) reinterpret_cast<float*>(&s_qrot[warp][c])[r] = s_rot[warp][c] * norm;
    __syncwarp();
    // per-group squared norms of the rotated row (Algorithm 1): every lane ends up with all of them
#pragma unroll
    for (int g = 0; g < G; ++g) {
      float acc = 0.f;
      for (int c = g * GROUP + lane; c < (g + 1) * GROUP; c += 32) {
        const float x = reinterpret_cast<const float*>(&s_qrot[warp][c])[r];
        acc += x * x;
      }
      for (int off = 16; off; off >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, off);
      nu[r][g] = acc;
    }
    __syncwarp();
  }

  const int64_t slab0 = (int64_t)bh * p.capacity;
  const float c_sc = p.sigma * kLog2e;                          // scores are kept in log2 units
  const float c_bias = p.sigma * p.sigma / 24.0f * kLog2e;
  const int n_all = p.n_cached + p.n_cur;

  // the four rows' scores against key i: xq with the quantized key (or the current one), xr with the BF16 one
  auto scores = [&](int i, float* xq, float* xr) {
    float aq[4] = {0.f, 0.f, 0.f, 0.f}, ar[4] = {0.f, 0.f, 0.f, 0.f};
    if (i < p.n_cached) {
      int64_t slot = p.cache_begin + i;
      if (slot >= p.capacity) slot -= p.capacity;
      const int64_t tok = slab0 + slot;
      const uint32_t* cw = reinterpret_cast<const uint32_t*>(p.k_codes + tok * (D * BITS / 8));
      const uint16_t* kr = p.kref + (int64_t)b * p.r_sb + (int64_t)h * p.r_sh + (int64_t)i * p.r_st;
      float bias_rows[4] = {0.f, 0.f, 0.f, 0.f};          // sum_g step_g^2 nu_g, the bias of Eq. (15) up to its constant
#pragma unroll
      for (int g = 0; g < G; ++g) {
        const float step = e4m3_byte_to_f32(p.k_scale[tok * G + g]);
        const float zs = bf16_bits_to_f32(p.k_zero[tok * G + g]) * step;
#pragma unroll
        for (int r = 0; r < 4; ++r) bias_rows[r] += step * step * nu[r][g];
        for (int wi = g * (GROUP / kCodesPerWord); wi < (g + 1) * (GROUP / kCodesPerWord); ++wi) {
          const uint32_t w = __ldg(cw + wi);
#pragma unroll
          for (int e = 0; e < kCodesPerWord; e += 2) {
            const int c = wi * kCodesPerWord + e;
            const uint32_t two = __ldg(reinterpret_cast<const uint32_t*>(kr + c));      // channels c, c + 1 of the BF16 key
            const float k0 = fmaf((float)((w >> (BITS * e)) & ((1u << BITS) - 1u)), step, -zs);
            const float k1 = fmaf((float)((w >> (BITS * (e + 1))) & ((1u << BITS) - 1u)), step, -zs);
            const float4 qa = s_qrot[warp][c], qb = s_qrot[warp][c + 1];
            aq[0] = fmaf(qa.x, k0, aq[0]); aq[1] = fmaf(qa.y, k0, aq[1]); aq[2] = fmaf(qa.z, k0, aq[2]); aq[3] = fmaf(qa.w, k0, aq[3]);
            aq[0] = fmaf(qb.x, k1, aq[0]); aq[1] = fmaf(qb.y, k1, aq[1]); aq[2] = fmaf(qb.z, k1, aq[2]); aq[3] = fmaf(qb.w, k1, aq[3]);
            const float r0 = bf16_bits_to_f32(two & 0xFFFFu), r1 = bf16_bits_to_f32(two >> 16);
            const float4 pa = s_q[warp][c], pb = s_q[warp][c + 1];
            ar[0] = fmaf(pa.x, r0, ar[0]); ar[1] = fmaf(pa.y, r0, ar[1]); ar[2] = fmaf(pa.z, r0, ar[2]); ar[3] = fmaf(pa.w, r0, ar[3]);
            ar[0] = fmaf(pb.x, r1, ar[0]); ar[1] = fmaf(pb.y, r1, ar[1]); ar[2] = fmaf(pb.z, r1, ar[2]); ar[3] = fmaf(pb.w, r1, ar[3]);
          }
        }
      }
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        xq[r] = c_sc * aq[r] - (p.correction ? c_bias * bias_rows[r] : 0.f);
        xr[r] = c_sc * ar[r];
      }
    } else {
      const uint16_t* kc = p.kcur + (int64_t)b * p.c_sb + (int64_t)h * p.c_sh + (int64_t)(i - p.n_cached) * p.c_st;
      for (int c = 0; c < D; c += 2) {
        const uint32_t two = __ldg(reinterpret_cast<const uint32_t*>(kc + c));
        const float r0 = bf16_bits_to_f32(two & 0xFFFFu), r1 = bf16_bits_to_f32(two >> 16);
        const float4 pa = s_q[warp][c], pb = s_q[warp][c + 1];
        ar[0] = fmaf(pa.x, r0, ar[0]); ar[1] = fmaf(pa.y, r0, ar[1]); ar[2] = fmaf(pa.z, r0, ar[2]); ar[3] = fmaf(pa.w, r0, ar[3]);
        ar[0] = fmaf(pb.x, r1, ar[0]); ar[1] = fmaf(pb.y, r1, ar[1]); ar[2] = fmaf(pb.z, r1, ar[2]); ar[3] = fmaf(pb.w, r1, ar[3]);
      }
#pragma unroll
      for (int r = 0; r < 4; ++r) xq[r] = xr[r] = c_sc * ar[r];
    }
  };

  // ---- pass 1: log-sum-exp (log2 units) of both score sets ----
  float mq[4], lq[4], mr[4], lr[4];
#pragma unroll
  for (int r = 0; r < 4; ++r) { mq[r] = mr[r] = -INFINITY; lq[r] = lr[r] = 0.f; }
  for (int i = lane; i < n_all; i += 32) {
    float xq[4], xr[4];
    scores(i, xq, xr);
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      float m2 = fmaxf(mq[r], xq[r]);
      lq[r] = lq[r] * exp2f(mq[r] - m2) + exp2f(xq[r] - m2); mq[r] = m2;
      m2 = fmaxf(mr[r], xr[r]);
      lr[r] = lr[r] * exp2f(mr[r] - m2) + exp2f(xr[r] - m2); mr[r] = m2;
    }
  }
  float lse_q[4], lse_r[4];
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    float m = mq[r], l = lq[r];
    for (int off = 16; off; off >>= 1) {
      const float om = __shfl_xor_sync(0xFFFFFFFFu, m, off), ol = __shfl_xor_sync(0xFFFFFFFFu, l, off);
      const float m2 = fmaxf(m, om);
      l = (m == -INFINITY ? 0.f : l * exp2f(m - m2)) + (om == -INFINITY ? 0.f : ol * exp2f(om - m2));
      m = m2;
    }
    lse_q[r] = m + log2f(l);
    m = mr[r]; l = lr[r];
    for (int off = 16; off; off >>= 1) {
      const float om = __shfl_xor_sync(0xFFFFFFFFu, m, off), ol = __shfl_xor_sync(0xFFFFFFFFu, l, off);
      const float m2 = fmaxf(m, om);
      l = (m == -INFINITY ? 0.f : l * exp2f(m - m2)) + (om == -INFINITY ? 0.f : ol * exp2f(om - m2));
      m = m2;
    }
    lse_r[r] = m + log2f(l);
  }

  // ---- pass 2: the divergence ----
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  for (int i = lane; i < n_all; i += 32) {
    float xq[4], xr[4];
    scores(i, xq, xr);
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const float pw = exp2f(xq[r] - lse_q[r]), rw = exp2f(xr[r] - lse_r[r]);
      const float mw = 0.5f * (pw + rw);
      float t = 0.f;
      if (pw > 0.f) t += pw * logf(pw / mw);
      if (rw > 0.f) t += rw * logf(rw / mw);
      acc[r] += t;
    }
  }
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    float a = acc[r];
    for (int off = 16; off; off >>= 1) a += __shfl_xor_sync(0xFFFFFFFFu, a, off);
    if (lane == 0 && row0 + r < p.m_tokens) p.jsd[(int64_t)bh * p.m_tokens + row0 + r] = 0.5f * a;
  }
}

}  // namespace

int launch_attn_jsd(const AttnArgs& a, const void* k_ref, kvq_strides rs, float* jsd_out) {
  const kvq_cache_desc* d = a.desc;
  JParams p;
  p.q = static_cast<const uint16_t*>(a.q); p.q_sb = a.qs.b; p.q_sh = a.qs.h; p.q_st = a.qs.t;
  p.kcur = static_cast<const uint16_t*>(a.k_cur); p.c_sb = a.kvs.b; p.c_sh = a.kvs.h; p.c_st = a.kvs.t;
  p.kref = static_cast<const uint16_t*>(k_ref); p.r_sb = rs.b; p.r_sh = rs.h; p.r_st = rs.t;
  p.k_codes = static_cast<const uint8_t*>(d->k_codes); p.k_scale = static_cast<const uint8_t*>(d->k_scale);
  p.k_zero = static_cast<const uint16_t*>(d->k_zero);
  p.signs = d->signs;
  p.capacity = d->capacity; p.cache_begin = a.cache_begin % d->capacity;
  p.heads = d->heads; p.rotate = (d->flags & KVQ_ROTATE_K) ? 1 : 0;
  p.correction = (a.flags & KVQ_CORRECTION_ON) ? 1 : 0;
  p.m_tokens = (int)a.m_tokens; p.n_cached = (int)a.cache_len; p.n_cur = (int)a.n_cur;
  p.sigma = a.softmax_scale;
  p.jsd = jsd_out;
  const int64_t bh = (int64_t)d->batch * d->heads;
  if (bh > 65535) return KVQ_ERR_UNSUPPORTED;
  const dim3 grid((unsigned)((a.m_tokens + kRowsPerBlock - 1) / kRowsPerBlock), (unsigned)bh), block(kWarps * 32);
  bool launched = false;
#define KVQ_J(D_, B_, G_) if (d->head_dim == D_ && d->bits == B_ && d->group == G_) { attn_jsd_kernel<D_, B_, G_><<<grid, block, 0, a.stream>>>(p); launched = true; }
  KVQ_J(128, 2, 32) KVQ_J(128, 2, 64) KVQ_J(128, 2, 128) KVQ_J(128, 4, 32) KVQ_J(128, 4, 64) KVQ_J(128, 4, 128)
  KVQ_J(64, 2, 32) KVQ_J(64, 2, 64) KVQ_J(64, 4, 32) KVQ_J(64, 4, 64)
#undef KVQ_J
  if (!launched) return KVQ_ERR_UNSUPPORTED;
  KVQ_CUDA_TRY(cudaGetLastError());
  return KVQ_OK;
}

}  // namespace kvq
