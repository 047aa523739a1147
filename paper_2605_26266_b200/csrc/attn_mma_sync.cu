// Corrected chunk attention, warp-level tensor-core kernel (mma.sync m16n8k16, BF16 -> FP32).
//
// This is the general-shape kernel: any m_tokens / cache_len / n_cur, head_dim 64 or 128,
// 2- or 4-bit codes, any supported group size.  It follows Algorithm 1 tile by tile with an
// online softmax: a CTA owns 64 query rows (4 warps x 16 rows), walks the cached keys in
// tiles of 64 (dequantized on the fly into shared memory, never to HBM), subtracts the
// Taylor bias from those scores, then walks the current chunk's BF16 keys with the
// unrotated query and no bias, and normalises once at the end.  The rotated query and the
// dequantized keys are held in FP16 (11-bit significands; the rotated query is not exactly
// representable in BF16 and its rounding would dominate the error budget on heavy-tailed
// keys), so the cached-score contraction is FP16 x FP16 -> FP32; everything else is BF16.
// Rotated queries and dequantized keys must stay below the FP16 maximum (65504); queries
// are clamped there.  The tcgen05 kernel is the fast path for the large shapes; this one is
// the cross-check and covers everything else.
#include "kvq_common.cuh"

namespace kvq {
namespace {

constexpr int kBM = 64;      // query rows per CTA
constexpr int kBN = 64;      // keys per tile
constexpr int kThreads = 128;
constexpr float kLog2e = 1.4426950408889634f;

struct AParams {
  const uint16_t* q; const uint16_t* kc; const uint16_t* vc; uint16_t* out;
  int64_t q_sb, q_sh, q_st, kv_sb, kv_sh, kv_st, v_sb, v_sh, v_st, o_sb, o_sh, o_st;
  const uint8_t* k_codes; const uint8_t* v_codes; const uint8_t* k_scale; const uint8_t* v_scale;
  const uint16_t* k_zero; const uint16_t* v_zero;
  const int8_t* signs;
  int64_t capacity, cache_begin;
  int heads, group, rotate, correction;   // correction: 0 off, 1 Taylor (Eq. 15), 2 exact (Eq. 12)
  int k_per_channel;                      // App. E: key steps / zero-points per (block of `group` tokens, channel)
  int m_tokens, n_cached, n_cur;
  float scale_log2, bias_coef_log2;   // sigma*log2(e), (sigma^2/24)*log2(e)
  float softmax_scale;
  float* lse; float* cached_mass;
};

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], const void* p) {
  uint32_t a = (uint32_t)__cvta_generic_to_shared(p);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], const void* p) {
  uint32_t a = (uint32_t)__cvta_generic_to_shared(p);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_f16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  return f32_to_bf16_bits(lo) | (f32_to_bf16_bits(hi) << 16);
}
__device__ __forceinline__ uint32_t pack_f16(float lo, float hi) {
  lo = fminf(fmaxf(lo, -65504.f), 65504.f);
  hi = fminf(fmaxf(hi, -65504.f), 65504.f);
  return (uint32_t)__half_as_ushort(__float2half_rn(lo)) | ((uint32_t)__half_as_ushort(__float2half_rn(hi)) << 16);
}

template <int D, int BITS>
struct Packed {   // raw packed data of one key-half held by one thread
  static constexpr int kWords = (D / 2) * BITS / 32;
  uint32_t w[kWords];
  uint32_t sbytes;   // up to 4 scale bytes of the token
  uint32_t z[2];     // up to 4 zero-points (BF16 bits)
};

template <int D, int BITS>
__device__ __forceinline__ void load_packed(Packed<D, BITS>& r, const uint8_t* codes, const uint8_t* scale,
                                            const uint16_t* zero, int64_t tok, int half, int G) {
  constexpr int CB = D * BITS / 8;
  const uint32_t* cw = reinterpret_cast<const uint32_t*>(codes + tok * CB) + half * Packed<D, BITS>::kWords;
#pragma unroll
  for (int i = 0; i < Packed<D, BITS>::kWords; ++i) r.w[i] = __ldg(cw + i);
  r.sbytes = 0; r.z[0] = r.z[1] = 0;
  for (int j = 0; j < G; ++j) {
    r.sbytes |= (uint32_t)__ldg(scale + tok * G + j) << (8 * j);
    r.z[j >> 1] |= (uint32_t)__ldg(zero + tok * G + j) << (16 * (j & 1));
  }
}

// x_hat = (code - zero) * step, rounded once to FP16 (keys) or BF16 (values), written to row
// `key` of a [kBN][D+8] tile.
template <int D, int BITS, bool kHalf>
__device__ __forceinline__ void dequant_store(const Packed<D, BITS>& r, uint16_t* tile, int key, int half, int group) {
  constexpr int LD = D + 8;
  constexpr int per = 32 / BITS;
  constexpr uint32_t mask = (1u << BITS) - 1;
  uint16_t* row = tile + key * LD + half * (D / 2);
#pragma unroll
  for (int c8 = 0; c8 < D / 2; c8 += 8) {
    const int ch = half * (D / 2) + c8;
    const int j = ch / group;
    const float ds = e4m3_byte_to_f32((r.sbytes >> (8 * j)) & 0xFFu);
    const float zs = bf16_bits_to_f32((r.z[j >> 1] >> (16 * (j & 1))) & 0xFFFFu);
    uint32_t o[4];
#pragma unroll
    for (int e = 0; e < 8; e += 2) {
      const int c0 = c8 + e, c1 = c8 + e + 1;
      const float x0 = ((float)((r.w[c0 / per] >> ((c0 % per) * BITS)) & mask) - zs) * ds;
      const float x1 = ((float)((r.w[c1 / per] >> ((c1 % per) * BITS)) & mask) - zs) * ds;
      o[e / 2] = kHalf ? pack_f16(x0, x1) : pack_bf16(x0, x1);
    }
    *reinterpret_cast<uint4*>(row + c8) = make_uint4(o[0], o[1], o[2], o[3]);
  }
}

// Per-channel keys (App. E): x_hat = (code - zero_c) * step_c with the steps and zero-points of the key's token block,
// staged in shared memory as floats ([D] each), rounded once to FP16.
template <int D, int BITS>
__device__ __forceinline__ void dequant_store_per_channel(const Packed<D, BITS>& r, uint16_t* tile, int key, int half,
                                                          const float* step, const float* zero) {
  constexpr int LD = D + 8;
  constexpr int per = 32 / BITS;
  constexpr uint32_t mask = (1u << BITS) - 1;
  uint16_t* row = tile + key * LD + half * (D / 2);
#pragma unroll
  for (int c8 = 0; c8 < D / 2; c8 += 8) {
    const int ch = half * (D / 2) + c8;
    uint32_t o[4];
#pragma unroll
    for (int e = 0; e < 8; e += 2) {
      const int c0 = c8 + e, c1 = c8 + e + 1;
      const float x0 = ((float)((r.w[c0 / per] >> ((c0 % per) * BITS)) & mask) - zero[ch + e]) * step[ch + e];
      const float x1 = ((float)((r.w[c1 / per] >> ((c1 % per) * BITS)) & mask) - zero[ch + e + 1]) * step[ch + e + 1];
      o[e / 2] = pack_f16(x0, x1);
    }
    *reinterpret_cast<uint4*>(row + c8) = make_uint4(o[0], o[1], o[2], o[3]);
  }
}

// log(sinh(a)/a) for a >= 0 (Eq. (12)): series below 0.5, a - log(2a) + log1p(-exp(-2a)) above.
__device__ __forceinline__ float log_sinhc(float a) {
  if (a < 0.5f) {
    const float a2 = a * a;
    return a2 * (1.0f / 6.0f + a2 * (-1.0f / 180.0f + a2 * (1.0f / 2835.0f - a2 * (1.0f / 37800.0f))));
  }
  return a - __logf(2.0f * a) + log1pf(-__expf(-2.0f * a));
}

template <int D, int BITS>
__global__ void __launch_bounds__(kThreads) attn_mma_sync_kernel(AParams p) {
  constexpr int LD = D + 8;
  constexpr int EPL = D / 32;
  constexpr int KS = D / 16;       // k-steps of QK^T
  constexpr int NBO = D / 8;       // n-blocks of the output
  extern __shared__ __align__(16) uint8_t smem_raw[];
  uint16_t* sQ = reinterpret_cast<uint16_t*>(smem_raw);       // unrotated query  [kBM][LD]
  uint16_t* sQr = sQ + kBM * LD;                               // rotated query    [kBM][LD], FP16
  uint16_t* sK = sQr + kBM * LD;                               // key tile         [kBN][LD]
  uint16_t* sV = sK + kBN * LD;                                // value tile       [kBN][LD]
  float* sNu = reinterpret_cast<float*>(sV + kBN * LD);        // [kBM][4]
  float* sW = sNu + kBM * 4;                                   // [kBN][4]
  // exact correction only: E4M3 step bytes of the tile's keys, and per (row, group, step byte) the bias
  // log2(e) * sum over the group's channels of log(sinh(a)/a), a = sigma |q~_c| step / 2 (Eq. (12)): a step
  // takes one of 127 values, so the exact bias of a score is one table look-up per group
  uint32_t* sWb = reinterpret_cast<uint32_t*>(sW + kBN * 4);   // [kBN]
  // per-channel keys only: steps and zero-points of the (at most two) token blocks a 64-key tile touches, and the
  // bias of every (query row, block): (sigma^2/24) log2(e) sum_c q~_c^2 step_c^2, one scalar for all keys of a block
  float* sPcStep = reinterpret_cast<float*>(sWb + kBN);        // [2][D]
  float* sPcZero = sPcStep + 2 * D;                            // [2][D]
  float* sPcBias = sPcZero + 2 * D;                            // [kBM][2]
  float* sT = sPcBias + kBM * 2;                               // [kBM][G][128]

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int bh = blockIdx.y, b = bh / p.heads, h = bh - b * p.heads;
  const int row0 = blockIdx.x * kBM;
  const int G = D / p.group;

  // ---- prologue: stage q, rotate it, per-group squared norms ---------------------------
  {
    const float c_d = (D == 64) ? 0.125f : __uint_as_float(0x3DB504F3u);
    const int lanes_per_group = p.group / EPL;
    for (int r = warp; r < kBM; r += kThreads / 32) {
      const int row = row0 + r;
      float x[EPL];
      uint32_t raw[EPL / 2];
      if (row < p.m_tokens) {
        const uint16_t* src = p.q + (int64_t)b * p.q_sb + (int64_t)h * p.q_sh + (int64_t)row * p.q_st + lane * EPL;
#pragma unroll
        for (int e = 0; e < EPL / 2; ++e) raw[e] = __ldg(reinterpret_cast<const uint32_t*>(src) + e);
      } else {
#pragma unroll
        for (int e = 0; e < EPL / 2; ++e) raw[e] = 0;
      }
#pragma unroll
      for (int e = 0; e < EPL / 2; ++e) {
        reinterpret_cast<uint32_t*>(sQ + r * LD + lane * EPL)[e] = raw[e];
        x[2 * e] = bf16_bits_to_f32(raw[e] & 0xFFFFu);
        x[2 * e + 1] = bf16_bits_to_f32(raw[e] >> 16);
      }
      if (p.rotate) {
#pragma unroll
        for (int e = 0; e < EPL; ++e)
          if (p.signs) x[e] *= (float)p.signs[lane * EPL + e];
#pragma unroll
        for (int hh = 1; hh < EPL; hh *= 2)
#pragma unroll
          for (int i = 0; i < EPL; ++i)
            if ((i & hh) == 0) { float a = x[i], c = x[i + hh]; x[i] = a + c; x[i + hh] = a - c; }
#pragma unroll
        for (int lm = 1; lm < 32; lm *= 2)
#pragma unroll
          for (int e = 0; e < EPL; ++e) {
            float o = __shfl_xor_sync(0xFFFFFFFFu, x[e], lm);
            x[e] = (lane & lm) ? (o - x[e]) : (x[e] + o);
          }
#pragma unroll
        for (int e = 0; e < EPL; ++e) x[e] *= c_d;
      }
      float nu = 0.f;
#pragma unroll
      for (int e = 0; e < EPL; ++e) nu += x[e] * x[e];
      for (int off = 1; off < lanes_per_group; off *= 2) nu += __shfl_xor_sync(0xFFFFFFFFu, nu, off);
      if ((lane % lanes_per_group) == 0) sNu[r * 4 + lane / lanes_per_group] = nu;
      if (p.correction == 2) {
        const int j = lane / lanes_per_group;
        for (int e = 0; e < 128; ++e) {
          const float half_step = 0.5f * p.softmax_scale * e4m3_byte_to_f32((uint32_t)e);
          float t = 0.f;
#pragma unroll
          for (int c = 0; c < EPL; ++c) t += log_sinhc(fabsf(x[c]) * half_step);
          for (int off = 1; off < lanes_per_group; off *= 2) t += __shfl_xor_sync(0xFFFFFFFFu, t, off);
          if ((lane % lanes_per_group) == 0) sT[(r * G + j) * 128 + e] = (e == 127) ? 0.f : t * kLog2e;
        }
      }
#pragma unroll
      for (int e = 0; e < EPL / 2; ++e)
        reinterpret_cast<uint32_t*>(sQr + r * LD + lane * EPL)[e] = pack_f16(x[2 * e], x[2 * e + 1]);
    }
  }
  __syncthreads();

  // per-thread softmax state for rows (lane/4) and (lane/4 + 8) of this warp's 16 rows
  const int rA = warp * 16 + (lane >> 2), rB = rA + 8;
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
  float acc[NBO][4];
#pragma unroll
  for (int n = 0; n < NBO; ++n) acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.f;
  float nuA[4], nuB[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) { nuA[j] = (j < G) ? sNu[rA * 4 + j] : 0.f; nuB[j] = (j < G) ? sNu[rB * 4 + j] : 0.f; }

  uint32_t qf[KS][4];
  auto load_q_frags = [&](const uint16_t* src) {
#pragma unroll
    for (int ks = 0; ks < KS; ++ks)
      ldmatrix_x4(qf[ks], src + (warp * 16 + (lane & 15)) * LD + ks * 16 + (lane >> 4) * 8);
  };

  // One tile of scores + softmax update + PV.  `biased` selects the cached-segment treatment.
  auto process_tile = [&](int n_valid, bool biased) {
    float s[kBN / 8][4];
#pragma unroll
    for (int nb = 0; nb < kBN / 8; ++nb) s[nb][0] = s[nb][1] = s[nb][2] = s[nb][3] = 0.f;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
#pragma unroll
      for (int nb2 = 0; nb2 < kBN / 16; ++nb2) {
        uint32_t kb[4];
        ldmatrix_x4(kb, sK + (nb2 * 16 + (lane >> 4) * 8 + (lane & 7)) * LD + ks * 16 + ((lane >> 3) & 1) * 8);
        if (biased) {      // cached segment: FP16 operands
          mma_f16(s[2 * nb2], qf[ks], kb[0], kb[1]);
          mma_f16(s[2 * nb2 + 1], qf[ks], kb[2], kb[3]);
        } else {
          mma_bf16(s[2 * nb2], qf[ks], kb[0], kb[1]);
          mma_bf16(s[2 * nb2 + 1], qf[ks], kb[2], kb[3]);
        }
      }
    }
    float mx[2] = {m_run[0], m_run[1]};
#pragma unroll
    for (int nb = 0; nb < kBN / 8; ++nb) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int col = nb * 8 + (lane & 3) * 2 + (e & 1);
        float v = s[nb][e] * p.scale_log2;
        if (biased) {
          float bsum = 0.f;
          if (p.correction == 2) {
            const float* trow = sT + (size_t)((e < 2) ? rA : rB) * G * 128;
            const uint32_t sb = sWb[col];
#pragma unroll
            for (int j = 0; j < 4; ++j) bsum += (j < G) ? trow[j * 128 + ((sb >> (8 * j)) & 0x7Fu)] : 0.f;
          } else {
            const float* nu = (e < 2) ? nuA : nuB;
#pragma unroll
            for (int j = 0; j < 4; ++j) bsum += (j < G) ? nu[j] * sW[col * 4 + j] : 0.f;
          }
          if (p.k_per_channel) bsum = sPcBias[((e < 2) ? rA : rB) * 2 + ((p.group == 32) ? (col >> 5) : 0)];
          v -= bsum;
        }
        if (col >= n_valid) v = -INFINITY;
        s[nb][e] = v;
        mx[e >> 1] = fmaxf(mx[e >> 1], v);
      }
    }
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xFFFFFFFFu, mx[r], 1));
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xFFFFFFFFu, mx[r], 2));
    }
    float corr[2], rs[2] = {0.f, 0.f};
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      corr[r] = exp2f(m_run[r] - mx[r]);       // m_run = -inf on the first tile -> 0
      m_run[r] = mx[r];
    }
    uint32_t pf[kBN / 16][4];
#pragma unroll
    for (int nb = 0; nb < kBN / 8; ++nb) {
      const float p0 = exp2f(s[nb][0] - mx[0]), p1 = exp2f(s[nb][1] - mx[0]);
      const float p2 = exp2f(s[nb][2] - mx[1]), p3 = exp2f(s[nb][3] - mx[1]);
      rs[0] += p0 + p1; rs[1] += p2 + p3;
      pf[nb >> 1][(nb & 1) * 2 + 0] = pack_bf16(p0, p1);
      pf[nb >> 1][(nb & 1) * 2 + 1] = pack_bf16(p2, p3);
    }
#pragma unroll
    for (int r = 0; r < 2; ++r) l_run[r] = l_run[r] * corr[r] + rs[r];
#pragma unroll
    for (int n = 0; n < NBO; ++n) {
      acc[n][0] *= corr[0]; acc[n][1] *= corr[0]; acc[n][2] *= corr[1]; acc[n][3] *= corr[1];
    }
#pragma unroll
    for (int kk = 0; kk < kBN / 16; ++kk) {
#pragma unroll
      for (int n2 = 0; n2 < NBO / 2; ++n2) {
        uint32_t vb[4];
        ldmatrix_x4_trans(vb, sV + (kk * 16 + ((lane >> 3) & 1) * 8 + (lane & 7)) * LD + n2 * 16 + (lane >> 4) * 8);
        mma_bf16(acc[2 * n2], pf[kk], vb[0], vb[1]);
        mma_bf16(acc[2 * n2 + 1], pf[kk], vb[2], vb[3]);
      }
    }
  };

  // ---- cached segment ----------------------------------------------------------------
  const int key = tid >> 1, half = tid & 1;
  const int n_ctiles = (p.n_cached + kBN - 1) / kBN;
  const int64_t tok_base = (int64_t)bh * p.capacity;
  if (n_ctiles > 0) {
    load_q_frags(sQr);
    Packed<D, BITS> pk, pv;
    // reading past n_cached stays inside `capacity` only up to the last token; clamp the index
    // window key -> slot, modulo the capacity (ring caches wrap)
    auto tok_of = [&](int t) {
      const int64_t slot = p.cache_begin + min((int64_t)t * kBN + key, (int64_t)p.n_cached - 1);
      return tok_base + (slot >= p.capacity ? slot - p.capacity : slot);
    };
    const int Gk = p.k_per_channel ? 0 : G;                      // per-channel keys have no per-token metadata
    load_packed<D, BITS>(pk, p.k_codes, p.k_scale, p.k_zero, tok_of(0), half, Gk);
    load_packed<D, BITS>(pv, p.v_codes, p.v_scale, p.v_zero, tok_of(0), half, G);
    for (int t = 0; t < n_ctiles; ++t) {
      __syncthreads();
      if (p.k_per_channel) {
        // the tile's keys lie in one token block (group 64, 128: windows start on a block) or two (group 32)
        const int nblk = (p.group == 32) ? 2 : 1;
        for (int i = tid; i < nblk * D; i += kThreads) {
          const int bi = i / D, c = i - bi * D;
          int64_t slot = p.cache_begin + min((int64_t)t * kBN + bi * 32, (int64_t)p.n_cached - 1);
          if (slot >= p.capacity) slot -= p.capacity;
          const int64_t blk = (int64_t)bh * (p.capacity / p.group) + slot / p.group;
          sPcStep[bi * D + c] = e4m3_byte_to_f32(__ldg(p.k_scale + blk * D + c));
          sPcZero[bi * D + c] = bf16_bits_to_f32(__ldg(p.k_zero + blk * D + c));
        }
        __syncthreads();
        {
          const int r = tid >> 1, bi = tid & 1;                  // kThreads = 2 * kBM: one (row, block) per thread
          float acc = 0.f;
          if (p.correction && bi < nblk) {
            for (int c = 0; c < D; ++c) {
              const float qv = __half2float(__ushort_as_half(sQr[r * LD + c])), ds = sPcStep[bi * D + c];
              acc += qv * qv * ds * ds;
            }
          }
          sPcBias[r * 2 + bi] = p.bias_coef_log2 * acc;
        }
        dequant_store_per_channel<D, BITS>(pk, sK, key, half, sPcStep + ((p.group == 32) ? (key >> 5) : 0) * D,
                                           sPcZero + ((p.group == 32) ? (key >> 5) : 0) * D);
      } else
      dequant_store<D, BITS, true>(pk, sK, key, half, p.group);
      dequant_store<D, BITS, false>(pv, sV, key, half, p.group);
      if (half == 0) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float ds = e4m3_byte_to_f32((pk.sbytes >> (8 * j)) & 0xFFu);
          sW[key * 4 + j] = (p.correction && j < G) ? p.bias_coef_log2 * ds * ds : 0.f;
        }
        sWb[key] = pk.sbytes;
      }
      __syncthreads();
      if (t + 1 < n_ctiles) {
        load_packed<D, BITS>(pk, p.k_codes, p.k_scale, p.k_zero, tok_of(t + 1), half, Gk);
        load_packed<D, BITS>(pv, p.v_codes, p.v_scale, p.v_zero, tok_of(t + 1), half, G);
      }
      process_tile(min(kBN, p.n_cached - t * kBN), true);
    }
  }
  const float m_s[2] = {m_run[0], m_run[1]}, l_s[2] = {l_run[0], l_run[1]};

  // ---- current segment: unrotated query, BF16 keys and values, no bias -----------------
  load_q_frags(sQ);
  const int n_rtiles = (p.n_cur + kBN - 1) / kBN;
  for (int t = 0; t < n_rtiles; ++t) {
    __syncthreads();
    {
      const int kidx = t * kBN + key;
      uint4* dk = reinterpret_cast<uint4*>(sK + key * LD + half * (D / 2));
      uint4* dv = reinterpret_cast<uint4*>(sV + key * LD + half * (D / 2));
      if (kidx < p.n_cur) {
        const int64_t off = (int64_t)b * p.kv_sb + (int64_t)h * p.kv_sh + (int64_t)kidx * p.kv_st + half * (D / 2);
        const uint4* gk = reinterpret_cast<const uint4*>(p.kc + off);
        const uint4* gv = reinterpret_cast<const uint4*>(p.vc + (int64_t)b * p.v_sb + (int64_t)h * p.v_sh + (int64_t)kidx * p.v_st + half * (D / 2));
#pragma unroll
        for (int i = 0; i < D / 16; ++i) { dk[i] = __ldg(gk + i); dv[i] = __ldg(gv + i); }
      } else {
#pragma unroll
        for (int i = 0; i < D / 16; ++i) { dk[i] = make_uint4(0, 0, 0, 0); dv[i] = make_uint4(0, 0, 0, 0); }
      }
    }
    __syncthreads();
    process_tile(min(kBN, p.n_cur - t * kBN), false);
  }

  // ---- epilogue ----------------------------------------------------------------------
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    l_run[r] += __shfl_xor_sync(0xFFFFFFFFu, l_run[r], 1);
    l_run[r] += __shfl_xor_sync(0xFFFFFFFFu, l_run[r], 2);
  }
  float l_s_tot[2] = {l_s[0], l_s[1]};
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    l_s_tot[r] += __shfl_xor_sync(0xFFFFFFFFu, l_s_tot[r], 1);
    l_s_tot[r] += __shfl_xor_sync(0xFFFFFFFFu, l_s_tot[r], 2);
  }
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const int row = row0 + (r == 0 ? rA : rB);
    if (row >= p.m_tokens) continue;
    const float inv = 1.0f / l_run[r];
    uint16_t* dst = p.out + (int64_t)b * p.o_sb + (int64_t)h * p.o_sh + (int64_t)row * p.o_st;
#pragma unroll
    for (int n = 0; n < NBO; ++n)
      *reinterpret_cast<uint32_t*>(dst + n * 8 + (lane & 3) * 2) = pack_bf16(acc[n][2 * r] * inv, acc[n][2 * r + 1] * inv);
    if ((lane & 3) == 0) {
      const int64_t idx = (int64_t)bh * p.m_tokens + row;
      if (p.lse) p.lse[idx] = (m_run[r] + log2f(l_run[r])) * 0.6931471805599453f;
      if (p.cached_mass)
        p.cached_mass[idx] = (n_ctiles > 0) ? l_s_tot[r] * exp2f(m_s[r] - m_run[r]) * inv : 0.f;
    }
  }
}

template <int D, int BITS>
int launch(const AParams& p, dim3 grid, cudaStream_t st) {
  constexpr int LD = D + 8;
  constexpr size_t base = (size_t)(2 * kBM + 2 * kBN) * LD * 2 + (kBM + kBN) * 4 * sizeof(float) + kBN * sizeof(uint32_t) +
                          (size_t)(4 * D + 2 * kBM) * sizeof(float);
  // the exact correction adds its table: 64 rows x groups x 128 step values
  const size_t smem = base + (p.correction == 2 ? (size_t)kBM * (D / p.group) * 128 * sizeof(float) : 0);
  static PerDevice configured;                       // the attribute is per device
  int dev = 0;
  { const int r = current_device(&dev); if (r != KVQ_OK) return r; }
  if (configured.first(dev)) {
    KVQ_CUDA_TRY(cudaFuncSetAttribute(attn_mma_sync_kernel<D, BITS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)(base + (size_t)kBM * 4 * 128 * sizeof(float))));
    configured.done(dev);
  }
  attn_mma_sync_kernel<D, BITS><<<grid, kThreads, smem, st>>>(p);
  KVQ_CUDA_TRY(cudaGetLastError());
  return KVQ_OK;
}

}  // namespace

int launch_attn_mma_sync(const AttnArgs& a) {
  const kvq_cache_desc* d = a.desc;
  AParams p;
  p.q = static_cast<const uint16_t*>(a.q); p.kc = static_cast<const uint16_t*>(a.k_cur);
  p.vc = static_cast<const uint16_t*>(a.v_cur); p.out = static_cast<uint16_t*>(a.out);
  p.q_sb = a.qs.b; p.q_sh = a.qs.h; p.q_st = a.qs.t;
  p.kv_sb = a.kvs.b; p.kv_sh = a.kvs.h; p.kv_st = a.kvs.t;
  p.v_sb = a.vs.b; p.v_sh = a.vs.h; p.v_st = a.vs.t;
  p.o_sb = a.os.b; p.o_sh = a.os.h; p.o_st = a.os.t;
  p.k_codes = static_cast<const uint8_t*>(d->k_codes); p.v_codes = static_cast<const uint8_t*>(d->v_codes);
  p.k_scale = static_cast<const uint8_t*>(d->k_scale); p.v_scale = static_cast<const uint8_t*>(d->v_scale);
  p.k_zero = static_cast<const uint16_t*>(d->k_zero); p.v_zero = static_cast<const uint16_t*>(d->v_zero);
  p.signs = d->signs;
  p.capacity = d->capacity; p.cache_begin = a.cache_begin % d->capacity;
  p.heads = d->heads; p.group = d->group; p.rotate = (d->flags & KVQ_ROTATE_K) ? 1 : 0;
  p.correction = (a.flags & KVQ_CORRECTION_EXACT) ? 2 : ((a.flags & KVQ_CORRECTION_ON) ? 1 : 0);
  p.softmax_scale = a.softmax_scale;
  p.k_per_channel = (d->flags & KVQ_K_PER_CHANNEL) ? 1 : 0;
  p.m_tokens = (int)a.m_tokens; p.n_cached = (int)a.cache_len; p.n_cur = (int)a.n_cur;
  p.scale_log2 = a.softmax_scale * kLog2e;
  p.bias_coef_log2 = a.softmax_scale * a.softmax_scale / 24.0f * kLog2e;
  p.lse = a.lse; p.cached_mass = a.cached_mass;
  const int64_t bh = (int64_t)d->batch * d->heads;
  if (bh > 65535) return KVQ_ERR_UNSUPPORTED;
  dim3 grid((unsigned)((a.m_tokens + kBM - 1) / kBM), (unsigned)bh);
  if (d->head_dim == 128 && d->bits == 2) return launch<128, 2>(p, grid, a.stream);
  if (d->head_dim == 128 && d->bits == 4) return launch<128, 4>(p, grid, a.stream);
  if (d->head_dim == 64 && d->bits == 2) return launch<64, 2>(p, grid, a.stream);
  if (d->head_dim == 64 && d->bits == 4) return launch<64, 4>(p, grid, a.stream);
  return KVQ_ERR_UNSUPPORTED;
}

}  // namespace kvq
