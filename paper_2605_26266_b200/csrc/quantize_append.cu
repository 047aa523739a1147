// Quantize-append kernel: Hadamard rotation (keys), group-wise asymmetric round-to-nearest
// quantization (Eq. (1)), bit packing and coalesced append of one finished chunk's K and V.
//
// Eight lanes own one token-head vector (lane l8 holds channels [l8*EPL, (l8+1)*EPL), EPL = head_dim/8), so a
// warp works on four vectors at a time.  The Walsh-Hadamard butterfly runs its first log2(EPL) stages inside a
// lane and the remaining three across lanes with shuffles; group minimum/maximum are shuffle reductions over
// the lanes of a group, and a lane's codes fill whole 32-bit words.  Every add, subtract, multiply and divide
// is a single IEEE binary32 operation (no contraction), so the stored codes, steps and zero-points are
// reproducible bit for bit.  A CTA stages the packed bytes of 32 consecutive tokens in shared memory and
// writes them out with 128-bit stores (tokens of one (batch, head) are contiguous in the cache).  CTAs are
// persistent (a few per SM) and keep the next tile's loads in flight while they work on the current one.
// By its bytes the kernel would be HBM-bound on its BF16 input; in fact it is bound by instruction issue: the
// bit-exact contract fixes one IEEE operation per butterfly, division, rounding and clamp, about 230 warp
// instructions per token-head, against 576 bytes.
#include "kvq_common.cuh"

namespace kvq {
namespace {

constexpr int kTileTokens = 32;
constexpr int kWarps = 8;
constexpr int kTokPerWarp = kTileTokens / kWarps;
constexpr int kCtasPerSm = 4;      // persistent grid: SMs x this (a multiple of the SM count)

struct QParams {
  const uint16_t* k; const uint16_t* v;
  int64_t sb, sh, st;          // element strides of k and v
  int64_t n_tokens, cache_len, capacity;
  int heads, group, rotate, rotate_v;
  int skip_k;                  // per-channel keys: the keys are written by quantize_k_per_channel_kernel instead
  const int8_t* signs;
  uint8_t* codes[2]; uint8_t* scale[2]; uint16_t* zero[2];
  int tiles_per_bh;
  int64_t total_tiles;
};

// y = c_d * H_d * x for a vector spread over 8 lanes (lane l8 holds channels [l8*EPL, (l8+1)*EPL)):
// stages h = 1, 2, 4, ... in that order, one rounding per operation.  The first log2(EPL) stages stay in
// registers, the last three exchange with lanes l8^1, l8^2, l8^4.
template <int EPL>
__device__ __forceinline__ void hadamard(float (&x)[EPL], int l8, float c_d) {
#pragma unroll
  for (int h = 1; h < EPL; h *= 2) {
#pragma unroll
    for (int i = 0; i < EPL; ++i) {
      if ((i & h) == 0) {
        const float a = x[i], b = x[i + h];
        x[i] = __fadd_rn(a, b);
        x[i + h] = __fsub_rn(a, b);
      }
    }
  }
#pragma unroll
  for (int lm = 1; lm < 8; lm *= 2) {
    const float sg = (l8 & lm) ? -1.0f : 1.0f;       // upper partner: other - own; fma(+-1, own, other) rounds once
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
      const float o = __shfl_xor_sync(0xFFFFFFFFu, x[e], lm);
      x[e] = __fmaf_rn(sg, x[e], o);
    }
  }
#pragma unroll
  for (int e = 0; e < EPL; ++e) x[e] = __fmul_rn(x[e], c_d);
}

// Quantizes the vector held by 8 lanes and stages codes / step / zero-point of token slot `tok` in shared
// memory.  The per-group work (range, step, zero-point) is shared by the GROUP/EPL lanes of a group.
template <int EPL, int BITS, int GROUP>
__device__ __forceinline__ void quantize_stage(const float (&x)[EPL], int l8, int tok,
                                               uint32_t* s_codes, uint8_t* s_scale, uint16_t* s_zero) {
  constexpr float L = (float)((1 << BITS) - 1);
  constexpr int kBitsPerLane = EPL * BITS;             // 16, 32 or 64
  constexpr int kWordsPerTok = 8 * kBitsPerLane / 32;
  constexpr int lanes_per_group = GROUP / EPL;
  constexpr int G = (8 * EPL) / GROUP;

  float mn = fminf(x[0], x[1]), mx = fmaxf(x[0], x[1]);
#pragma unroll
  for (int e = 2; e < EPL; e += 2) {                  // three-input minimum and maximum: one instruction per two elements
    asm("min.f32 %0, %1, %2, %3;" : "=f"(mn) : "f"(mn), "f"(x[e]), "f"(x[e + 1]));
    asm("max.f32 %0, %1, %2, %3;" : "=f"(mx) : "f"(mx), "f"(x[e]), "f"(x[e + 1]));
  }
#pragma unroll
  for (int off = 1; off < lanes_per_group; off *= 2) {
    mn = fminf(mn, __shfl_xor_sync(0xFFFFFFFFu, mn, off));
    mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, off));
  }
  // Divisions.  x / b as q0 = x*r, rem = fma(-q0, b, x), q = fma(rem, r, q0) with r = RN(1/b) is the correctly
  // rounded quotient for every divisor used here (3, 15 and the 126 positive E4M3 values: checked against
  // IEEE division for all 2^23 significands of x) as long as nothing overflows.  A quotient too small to be
  // computed exactly needs no care: it is below 2^-40 and rounds to the integer 0, or to the step floor 2^-9,
  // either way.  Rounding to an integer is q + 1.5*2^23 - 1.5*2^23 (the FMA pipe instead of the quarter-rate
  // conversion unit), which is rint(q) while |q| < 2^22.  Vectors with magnitudes or quotients beyond those
  // bounds take IEEE division and rintf instead, the whole warp together.
  const float range = __fsub_rn(mx, mn);
  const float amax = fmaxf(fabsf(range), fmaxf(fabsf(mn), fabsf(mx)));
  auto fast_div = [](float a, float b, float r) {
    const float q0 = __fmul_rn(a, r);
    return __fmaf_rn(__fmaf_rn(-q0, b, a), r, q0);
  };
  const bool big = !(amax < 0x1p60f);
  float step = fast_div(range, L, (BITS == 2) ? __uint_as_float(0x3EAAAAABu) : __uint_as_float(0x3D888889u));
  if (big) step = __fdiv_rn(range, L);
  uint32_t sbyte = f32_to_e4m3_byte(step);
  if (sbyte == 0) sbyte = 1;                       // floor at the smallest subnormal 2^-9
  const float ds = e4m3_byte_to_f32(sbyte);
  const float rds = __frcp_rn(ds);
  const bool slow = __any_sync(0xFFFFFFFFu, big || !(__fmul_rn(amax, rds) < 0x1p21f));
  constexpr float kRound = 12582912.f;             // 1.5 * 2^23
  const float z = __fsub_rn(0.0f, slow ? rintf(__fdiv_rn(mn, ds)) : __fsub_rn(__fadd_rn(fast_div(mn, ds, rds), kRound), kRound));
  const uint32_t zbits = f32_to_bf16_bits(z);
  const float zs = bf16_bits_to_f32(zbits);

  // Codes are packed 16 bits at a time as exact float sums c_e * 2^(bit position), then read out of the low
  // mantissa bits of sum + 2^23.
  constexpr int kChunks = kBitsPerLane / 16;
  float acc[kChunks];
#pragma unroll
  for (int k = 0; k < kChunks; ++k) acc[k] = 8388608.f;
  if (!slow) {
    // q + 1.5*2^23 is 1.5*2^23 + rint(q); taking off 1.5*2^23 - zero (an integer below 2^24, so exact) leaves
    // rint(q) + zero, the sum Eq. (1) clamps.  While the zero-point is exact in BF16 (|zero| <= 256) the sum cannot
    // be negative (x >= min and both roundings are monotonic), so the lower clamp is only taken when some group of
    // the warp has a rounded zero-point.
    const float kz = __fsub_rn(kRound, zs);
    if (__any_sync(0xFFFFFFFFu, zs != z)) {
#pragma unroll
      for (int e = 0; e < EPL; ++e) {
        const float c = fminf(fmaxf(__fsub_rn(__fadd_rn(fast_div(x[e], ds, rds), kRound), kz), 0.0f), L);
        acc[(e * BITS) / 16] = __fmaf_rn(c, (float)(1u << ((e * BITS) % 16)), acc[(e * BITS) / 16]);
      }
    } else {
#pragma unroll
      for (int e = 0; e < EPL; ++e) {
        const float c = fminf(__fsub_rn(__fadd_rn(fast_div(x[e], ds, rds), kRound), kz), L);
        acc[(e * BITS) / 16] = __fmaf_rn(c, (float)(1u << ((e * BITS) % 16)), acc[(e * BITS) / 16]);
      }
    }
  } else {
#pragma unroll
    for (int e = 0; e < EPL; ++e) {
      const float c = fminf(fmaxf(__fadd_rn(rintf(__fdiv_rn(x[e], ds)), zs), 0.0f), L);
      acc[(e * BITS) / 16] = __fmaf_rn(c, (float)(1u << ((e * BITS) % 16)), acc[(e * BITS) / 16]);
    }
  }
  uint32_t piece[(kBitsPerLane + 31) / 32];
  if constexpr (kChunks == 1) {
    piece[0] = __float_as_uint(acc[0]) & 0xFFFFu;
  } else {
#pragma unroll
    for (int k = 0; k < kChunks; k += 2)
      piece[k / 2] = __byte_perm(__float_as_uint(acc[k]), __float_as_uint(acc[k + 1]), 0x5410);
  }
  if constexpr (kBitsPerLane == 16) {                  // two lanes share a word
    const uint32_t other = __shfl_xor_sync(0xFFFFFFFFu, piece[0], 1);
    if ((l8 & 1) == 0) s_codes[tok * kWordsPerTok + (l8 >> 1)] = piece[0] | (other << 16);
  } else if constexpr (kBitsPerLane == 32) {
    s_codes[tok * kWordsPerTok + l8] = piece[0];
  } else {
    *reinterpret_cast<uint2*>(&s_codes[tok * kWordsPerTok + 2 * l8]) = make_uint2(piece[0], piece[1]);
  }
  if ((l8 % lanes_per_group) == 0) {
    s_scale[tok * G + l8 / lanes_per_group] = (uint8_t)sbyte;
    s_zero[tok * G + l8 / lanes_per_group] = (uint16_t)zbits;
  }
}

// Cooperative shared->global copy with the widest store both sides allow.
__device__ __forceinline__ void copy_out(uint8_t* dst, const uint8_t* src, int nbytes, int tid, int nthreads) {
  const uintptr_t a = reinterpret_cast<uintptr_t>(dst) | reinterpret_cast<uintptr_t>(src) | (uintptr_t)nbytes;
  if ((a & 15) == 0) {
    for (int i = tid; i < nbytes / 16; i += nthreads)
      reinterpret_cast<uint4*>(dst)[i] = reinterpret_cast<const uint4*>(src)[i];
  } else if ((a & 3) == 0) {
    for (int i = tid; i < nbytes / 4; i += nthreads)
      reinterpret_cast<uint32_t*>(dst)[i] = reinterpret_cast<const uint32_t*>(src)[i];
  } else if ((a & 1) == 0) {
    for (int i = tid; i < nbytes / 2; i += nthreads)
      reinterpret_cast<uint16_t*>(dst)[i] = reinterpret_cast<const uint16_t*>(src)[i];
  } else {
    for (int i = tid; i < nbytes; i += nthreads) dst[i] = src[i];
  }
}

template <int EPL>
struct RawVec { uint4 r[EPL / 8]; };      // EPL BF16 values of one lane

template <int EPL>
__device__ __forceinline__ void load_raw_vec(RawVec<EPL>& v, const uint16_t* p, int l8) {
#pragma unroll
  for (int i = 0; i < EPL / 8; ++i) v.r[i] = __ldg(reinterpret_cast<const uint4*>(p) + l8 * (EPL / 8) + i);
}
template <int EPL>
__device__ __forceinline__ void decode_vec(const RawVec<EPL>& v, float (&x)[EPL]) {
#pragma unroll
  for (int i = 0; i < EPL / 8; ++i) {
    const uint32_t w[4] = {v.r[i].x, v.r[i].y, v.r[i].z, v.r[i].w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      x[8 * i + 2 * e] = bf16_bits_to_f32(w[e] & 0xFFFFu);
      x[8 * i + 2 * e + 1] = bf16_bits_to_f32(w[e] >> 16);
    }
  }
}

// Persistent CTAs: each walks tiles of 32 consecutive tokens of one (batch, head) with a stride of gridDim.x
// and has the next tile's loads in flight while it rotates, quantizes and packs the current one.  A warp
// works on four token-head vectors at a time, eight lanes per vector.
template <int D, int BITS, int GROUP>
__global__ void __launch_bounds__(kWarps * 32) quantize_append_kernel(QParams p) {
  constexpr int EPL = D / 8;
  constexpr int CB = D * BITS / 8;
  __shared__ __align__(16) uint32_t s_codes[2][kTileTokens * CB / 4];
  __shared__ __align__(16) uint8_t s_scale[2][kTileTokens * 4];
  __shared__ __align__(16) uint16_t s_zero[2][kTileTokens * 4];

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int l8 = lane & 7;
  const int tok = warp * kTokPerWarp + (lane >> 3);          // token slot inside the tile
  constexpr int G = D / GROUP;
  const float c_d = (D == 64) ? 0.125f : __uint_as_float(0x3DB504F3u);

  RawVec<EPL> rk, rv;
  auto fetch = [&](int tile_g) {
    const int bh = tile_g / p.tiles_per_bh;
    const int tile = tile_g - bh * p.tiles_per_bh;
    const int b = bh / p.heads, h = bh - b * p.heads;
    const int64_t t = (int64_t)tile * kTileTokens + tok;
    if (t < p.n_tokens) {
      const int64_t off = (int64_t)b * p.sb + (int64_t)h * p.sh + t * p.st;
      load_raw_vec<EPL>(rk, p.k + off, l8);
      load_raw_vec<EPL>(rv, p.v + off, l8);
    } else {                                                  // slots past the end quantize zeros, never stored
#pragma unroll
      for (int i = 0; i < EPL / 8; ++i) { rk.r[i] = make_uint4(0, 0, 0, 0); rv.r[i] = make_uint4(0, 0, 0, 0); }
    }
  };

  int tile_g = blockIdx.x;
  const int total_tiles = (int)p.total_tiles;
  if (tile_g < total_tiles) fetch(tile_g);
  for (; tile_g < total_tiles; tile_g += gridDim.x) {
    const int bh = tile_g / p.tiles_per_bh;
    const int tile = tile_g - bh * p.tiles_per_bh;
    const int64_t t0 = (int64_t)tile * kTileTokens;
    const int nt = (int)min((int64_t)kTileTokens, p.n_tokens - t0);
    float x[EPL];
    decode_vec<EPL>(rk, x);
    const RawVec<EPL> rv_cur = rv;
    if (tile_g + (int)gridDim.x < total_tiles) fetch(tile_g + (int)gridDim.x);
    if (!p.skip_k) {
      if (p.rotate) {
        if (p.signs) {
#pragma unroll
          for (int e = 0; e < EPL; ++e) x[e] = __fmul_rn(x[e], (float)p.signs[l8 * EPL + e]);
        }
        hadamard<EPL>(x, l8, c_d);
      }
      quantize_stage<EPL, BITS, GROUP>(x, l8, tok, s_codes[0], s_scale[0], s_zero[0]);
    }
    decode_vec<EPL>(rv_cur, x);
    if (p.rotate_v) {                                       // values stored rotated too (KVQ_ROTATE_V)
      if (p.signs) {
#pragma unroll
        for (int e = 0; e < EPL; ++e) x[e] = __fmul_rn(x[e], (float)p.signs[l8 * EPL + e]);
      }
      hadamard<EPL>(x, l8, c_d);
    }
    quantize_stage<EPL, BITS, GROUP>(x, l8, tok, s_codes[1], s_scale[1], s_zero[1]);
    __syncthreads();
    // The tile goes to slots slot0 .. slot0 + nt - 1, modulo the capacity: one piece, or two when a ring
    // cache wraps inside the tile (p.cache_len is already reduced modulo the capacity, so one subtraction does).
    int64_t slot0 = p.cache_len + t0;
    if (slot0 >= p.capacity) slot0 -= p.capacity;
    const int n_first = (int)min((int64_t)nt, p.capacity - slot0);
#pragma unroll 1
    for (int piece = 0; piece < 2; ++piece) {
      const int ntok = piece ? nt - n_first : n_first;
      if (ntok <= 0) break;
      const int skip = piece ? n_first : 0;                    // tokens of the tile stored by the first piece
      const int64_t tok_index = (int64_t)bh * p.capacity + (piece ? 0 : slot0);
#pragma unroll
      for (int w = 0; w < 2; ++w) {
        if (w == 0 && p.skip_k) continue;
        copy_out(p.codes[w] + tok_index * CB, reinterpret_cast<const uint8_t*>(s_codes[w]) + skip * CB, ntok * CB, threadIdx.x, kWarps * 32);
        copy_out(p.scale[w] + tok_index * G, s_scale[w] + skip * G, ntok * G, threadIdx.x, kWarps * 32);
        copy_out(reinterpret_cast<uint8_t*>(p.zero[w] + tok_index * G), reinterpret_cast<const uint8_t*>(s_zero[w] + skip * G),
                 ntok * G * 2, threadIdx.x, kWarps * 32);
      }
    }
    __syncthreads();
  }
}

// ---- per-channel keys (App. E) -----------------------------------------------------------------------
// One CTA per (batch*head, block of g = p.group tokens): the g x D block is rotated into shared memory (FP32), then
// thread c owns channel c: minimum and maximum over the block's tokens, step and zero-point with the arithmetic of
// Eq. (1) in plain IEEE operations (range / L, E4M3 rounding, -rint(min / step), rint(y / step) + zero, clamp),
// codes as bytes in shared memory; finally the codes of a token are packed 32 / BITS per word along the channels,
// the layout every other kernel reads.  An analysis option: nothing here is tuned.
template <int D, int BITS>
__global__ void __launch_bounds__(256) quantize_k_per_channel_kernel(QParams p) {
  constexpr int EPL = D / 8;
  constexpr int CB = D * BITS / 8;
  constexpr int LDY = D + 1;
  extern __shared__ __align__(16) uint8_t pc_smem[];
  const int g = p.group;
  float* y = reinterpret_cast<float*>(pc_smem);                       // [g][D + 1]
  uint8_t* codes = pc_smem + (size_t)g * LDY * sizeof(float);          // [g][D]
  const int bh = blockIdx.y, b = bh / p.heads, h = bh - b * p.heads;
  const int64_t t0 = (int64_t)blockIdx.x * g;                          // first token of the block within the chunk
  const int lane = threadIdx.x & 31, l8 = lane & 7;
  const float c_d = (D == 64) ? 0.125f : __uint_as_float(0x3DB504F3u);
  for (int r = threadIdx.x >> 3; r < g; r += 32) {                     // 8 lanes per token, 32 tokens per pass
    RawVec<EPL> raw;
    load_raw_vec<EPL>(raw, p.k + (int64_t)b * p.sb + (int64_t)h * p.sh + (t0 + r) * p.st, l8);
    float x[EPL];
    decode_vec<EPL>(raw, x);
    if (p.rotate) {
      if (p.signs) {
#pragma unroll
        for (int e = 0; e < EPL; ++e) x[e] = __fmul_rn(x[e], (float)p.signs[l8 * EPL + e]);
      }
      hadamard<EPL>(x, l8, c_d);
    }
#pragma unroll
    for (int e = 0; e < EPL; ++e) y[r * LDY + l8 * EPL + e] = x[e];
  }
  __syncthreads();
  int64_t slot0 = p.cache_len + t0;                                    // whole blocks never straddle the end of a ring
  slot0 %= p.capacity;
  if (threadIdx.x < D) {
    const int c = threadIdx.x;
    constexpr float L = (float)((1 << BITS) - 1);
    float mn = y[c], mx = y[c];
    for (int t = 1; t < g; ++t) { mn = fminf(mn, y[t * LDY + c]); mx = fmaxf(mx, y[t * LDY + c]); }
    const float step = __fdiv_rn(__fsub_rn(mx, mn), L);
    uint32_t sbyte = f32_to_e4m3_byte(step);
    if (sbyte == 0) sbyte = 1;                                         // floor at the smallest subnormal 2^-9
    const float ds = e4m3_byte_to_f32(sbyte);
    const float z = __fsub_rn(0.0f, rintf(__fdiv_rn(mn, ds)));
    const uint32_t zbits = f32_to_bf16_bits(z);
    const float zs = bf16_bits_to_f32(zbits);
    for (int t = 0; t < g; ++t) {
      const float cc = fminf(fmaxf(__fadd_rn(rintf(__fdiv_rn(y[t * LDY + c], ds)), zs), 0.0f), L);
      codes[t * D + c] = (uint8_t)cc;
    }
    const int64_t blk = (int64_t)bh * (p.capacity / g) + slot0 / g;
    p.scale[0][blk * D + c] = (uint8_t)sbyte;
    p.zero[0][blk * D + c] = (uint16_t)zbits;
  }
  __syncthreads();
  constexpr int kPer = 32 / BITS;                                      // codes per 32-bit word
  uint32_t* out = reinterpret_cast<uint32_t*>(p.codes[0] + ((int64_t)bh * p.capacity + slot0) * CB);
  for (int i = threadIdx.x; i < g * (CB / 4); i += 256) {
    const int t = i / (CB / 4), w = i - t * (CB / 4);
    uint32_t word = 0;
#pragma unroll
    for (int j = 0; j < kPer; ++j) word |= (uint32_t)codes[t * D + w * kPer + j] << (j * BITS);
    out[i] = word;                                                     // tokens of a block are contiguous: out[t * CB/4 + w]
  }
}

template <int BITS>
__global__ void unpack_codes_kernel(const uint8_t* codes, uint8_t* out, int64_t capacity, int64_t begin,
                                    int64_t n, int D, int64_t total) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total) return;
  const int c = (int)(i % D);
  const int64_t t = (i / D) % n;
  const int64_t bh = i / ((int64_t)D * n);
  const int CB = D * BITS / 8;
  int64_t slot = begin + t;                                   // begin is already reduced modulo the capacity
  if (slot >= capacity) slot -= capacity;
  const uint8_t byte = codes[(bh * capacity + slot) * CB + (c * BITS) / 8];
  out[i] = (byte >> ((c * BITS) % 8)) & ((1 << BITS) - 1);
}

}  // namespace

int launch_quantize_append(const kvq_cache_desc* d, int64_t cache_len, const void* k, const void* v,
                           kvq_strides kv, int64_t n_tokens, cudaStream_t st) {
  QParams p;
  p.k = static_cast<const uint16_t*>(k);
  p.v = static_cast<const uint16_t*>(v);
  p.sb = kv.b; p.sh = kv.h; p.st = kv.t;
  p.n_tokens = n_tokens; p.cache_len = cache_len % d->capacity; p.capacity = d->capacity;
  p.heads = d->heads; p.group = d->group; p.rotate = (d->flags & KVQ_ROTATE_K) ? 1 : 0;
  p.rotate_v = (d->flags & KVQ_ROTATE_V) ? 1 : 0;
  p.skip_k = (d->flags & KVQ_K_PER_CHANNEL) ? 1 : 0;
  p.signs = d->signs;
  p.codes[0] = static_cast<uint8_t*>(d->k_codes); p.codes[1] = static_cast<uint8_t*>(d->v_codes);
  p.scale[0] = static_cast<uint8_t*>(d->k_scale); p.scale[1] = static_cast<uint8_t*>(d->v_scale);
  p.zero[0] = static_cast<uint16_t*>(d->k_zero); p.zero[1] = static_cast<uint16_t*>(d->v_zero);
  p.tiles_per_bh = (int)((n_tokens + kTileTokens - 1) / kTileTokens);
  p.total_tiles = (int64_t)d->batch * d->heads * p.tiles_per_bh;
  int sms = 0;
  { const int r = device_sm_count(&sms); if (r != KVQ_OK) return r; }
  const int64_t blocks = p.total_tiles < (int64_t)sms * kCtasPerSm ? p.total_tiles : (int64_t)sms * kCtasPerSm;
  dim3 grid((unsigned)blocks), block(kWarps * 32);
  if (p.total_tiles > 0x7FFFFFFFLL - 65536) return KVQ_ERR_UNSUPPORTED;
#define KVQ_QA(D_, B_, G_) if (d->head_dim == D_ && d->bits == B_ && d->group == G_) { quantize_append_kernel<D_, B_, G_><<<grid, block, 0, st>>>(p); launched = true; }
  bool launched = false;
  KVQ_QA(128, 2, 32) KVQ_QA(128, 2, 64) KVQ_QA(128, 2, 128) KVQ_QA(128, 4, 32) KVQ_QA(128, 4, 64) KVQ_QA(128, 4, 128)
  KVQ_QA(64, 2, 32) KVQ_QA(64, 2, 64) KVQ_QA(64, 4, 32) KVQ_QA(64, 4, 64)
#undef KVQ_QA
  if (!launched) return KVQ_ERR_UNSUPPORTED;
  KVQ_CUDA_TRY(cudaGetLastError());
  if (p.skip_k) {                                     // per-channel keys: one CTA per block of `group` tokens
    const int64_t bh = (int64_t)d->batch * d->heads;
    if (bh > 65535) return KVQ_ERR_UNSUPPORTED;
    const dim3 pgrid((unsigned)(n_tokens / d->group), (unsigned)bh);
    const size_t smem = (size_t)d->group * (d->head_dim + 1) * sizeof(float) + (size_t)d->group * d->head_dim;
#define KVQ_PC(D_, B_) if (d->head_dim == D_ && d->bits == B_) { \
      KVQ_CUDA_TRY(cudaFuncSetAttribute(quantize_k_per_channel_kernel<D_, B_>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)); \
      quantize_k_per_channel_kernel<D_, B_><<<pgrid, 256, smem, st>>>(p); }
    KVQ_PC(128, 2) KVQ_PC(128, 4) KVQ_PC(64, 2) KVQ_PC(64, 4)
#undef KVQ_PC
    KVQ_CUDA_TRY(cudaGetLastError());
  }
  return KVQ_OK;
}

int launch_unpack_codes(const kvq_cache_desc* d, int which, int64_t begin, int64_t n, uint8_t* out,
                        cudaStream_t st) {
  const int64_t total = (int64_t)d->batch * d->heads * n * d->head_dim;
  if (total == 0) return KVQ_OK;
  const uint8_t* codes = static_cast<const uint8_t*>(which == 0 ? d->k_codes : d->v_codes);
  const int threads = 256;
  const int64_t blocks = (total + threads - 1) / threads;
  if (blocks > 0x7FFFFFFFLL) return KVQ_ERR_UNSUPPORTED;
  if (d->bits == 2)
    unpack_codes_kernel<2><<<(unsigned)blocks, threads, 0, st>>>(codes, out, d->capacity, begin % d->capacity, n, d->head_dim, total);
  else
    unpack_codes_kernel<4><<<(unsigned)blocks, threads, 0, st>>>(codes, out, d->capacity, begin % d->capacity, n, d->head_dim, total);
  KVQ_CUDA_TRY(cudaGetLastError());
  return KVQ_OK;
}

}  // namespace kvq
