// Corrected chunk attention for sm_100a: TMA + tcgen05.mma with TMEM accumulators.
//
// One CTA owns 256 query rows of one (batch, head) — two 128-row tiles that ping-pong on the
// tensor pipe — and walks all keys in tiles of 128: first the current chunk's BF16 keys and
// values (TMA straight into the 128-byte-swizzled operand layout, unrotated query, no bias),
// then the cached keys and values, which four "dequant" warps expand from the packed
// 2-/4-bit codes into the same operand layout in shared memory (never to HBM).  Between the
// two segments the same warps rotate the query tile in place (Hadamard, FP32 butterflies),
// and compute the per-group squared norms nu of Algorithm 1.
//
// Score of a cached key (Eq. (15) / Eq. (25)):  s = sigma*q~.k^ - (sigma^2/24) sum_j step_j^2 nu_j.
// The bias is folded into the score contraction as one extra K=16 MMA step per tile:
// A_extra[m, j] = -(sigma/24) nu_{m,j} (split into a BF16 high and low part, two columns) and
// B_extra[i, j] = step_{i,j}^2 (exact in BF16), so the softmax warps spend no instruction on
// it; correction off simply skips that step.
//
// Numerics: the rotated query and the dequantized keys are FP16 (the rotated query is not
// representable in BF16; FP16's 11-bit significand keeps its rounding well inside the error
// budget), so cached scores are an FP16 x FP16 -> FP32 contraction; current-chunk scores and
// both PV products are BF16 x BF16 -> FP32.  P is written back to TMEM as BF16 over the score
// columns and consumed from there by the PV MMA.  Rotated queries are clamped to the FP16
// range; dequantized keys must lie inside it.
//
// Roles (512 threads): warp 0 lane 0 issues TMA, warp 1 lane 0 issues all MMAs, warps 4-7 and
// 8-11 are the softmax groups of query tile 0 and 1 (one thread per row = one TMEM lane),
// warps 12-15 dequantize and rotate.  Every wait on an mbarrier is bounded: on expiry the CTA
// records a diagnostic in the caller's status word, all roles leave their loops, in-flight
// work is drained with a bounded wait, TMEM is freed and the kernel returns.
#include <cuda_fp16.h>

#include "kvq_common.cuh"
#include "sm100_ptx.cuh"

namespace kvq {
namespace {
using namespace ptx;

constexpr int kD = 128;
constexpr int kBlockM = 128;
constexpr int kBlockN = 128;
constexpr int kThreads = 512;
constexpr int kTileBytes = kBlockN * kD * 2;       // 32 KiB: one 128 x 128 16-bit operand tile
constexpr int kHalfTile = kTileBytes / 2;          // one 64-column block of it
constexpr int kXBytes = 128 * 16 * 2;              // 4 KiB: one 128 x 16 bias operand tile

constexpr int kOffQ = 0;                           // 2 query tiles
constexpr int kOffK = kOffQ + 2 * kTileBytes;      // 2 stages
constexpr int kOffV = kOffK + 2 * kTileBytes;      // 2 stages
constexpr int kOffAx = kOffV + 2 * kTileBytes;     // 2 query tiles
constexpr int kOffBx = kOffAx + 2 * kXBytes;       // 2 stages
constexpr int kOffBar = kOffBx + 2 * kXBytes;
constexpr int kNumBars = 20;
constexpr int kOffMisc = kOffBar + kNumBars * 8;
constexpr int kSmemBytes = kOffMisc + 64 + 1024;   // + slack to align the base to 1024

enum Bar { kQFull = 0, kKFull = 1, kVFull = 3, kKEmpty = 5, kVEmpty = 7, kSFull = 9, kPFull = 11,
           kODone = 13, kQCurDone = 15, kQRotFull = 16, kDrain = 17 };

constexpr long long kTimeoutCycles = 2000000000LL;   // about a second
constexpr long long kDrainCycles = 20000000LL;
constexpr float kLog2e = 1.4426950408889634f;
// registers per thread after reallocation: 128 * 72 + 256 * 168 + 128 * 96 = 64512 <= 65536
constexpr int kRegsIssue = 72, kRegsSoftmax = 168, kRegsDequant = 96;
constexpr float kRescaleThreshold = 8.0f;          // lazy rescale of O: only when the max grows by > 2^8

struct TParams {
  uint16_t* out; int64_t o_sb, o_sh, o_st;
  const uint8_t* k_codes; const uint8_t* v_codes; const uint8_t* k_scale; const uint8_t* v_scale;
  const uint16_t* k_zero; const uint16_t* v_zero;
  const int8_t* signs;
  int64_t capacity, cache_begin;
  int heads, group, rotate, correction;
  int m_tokens, n_cached, n_cur;
  float scale_log2;        // sigma * log2(e)
  float ax_coef;           // -sigma / 24
  float* lse; float* cached_mass;
  int32_t* status;
};

struct Ctx {
  uint32_t bar0;
  volatile int* abort;
  int32_t* status;
  __device__ __forceinline__ uint32_t bar(int i) const { return bar0 + 8u * i; }
  // Bounded wait; false once the CTA is aborting.
  __device__ __forceinline__ bool wait(int i, uint32_t parity, int code) const {
    const uint32_t b = bar(i);
    if (mbar_try_wait(b, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
      if (mbar_try_wait(b, parity)) return true;
      if (*abort) return false;
      if (clock64() - t0 > kTimeoutCycles) {
        *abort = 1;
        if (status) atomicCAS(status, 0, code);
        return false;
      }
    }
  }
  // Used only on the way out: lets work already in flight finish, ignoring the abort flag.
  __device__ __forceinline__ void drain(int i, uint32_t parity) const {
    const uint32_t b = bar(i);
    const long long t0 = clock64();
    while (!mbar_try_wait(b, parity) && clock64() - t0 < kDrainCycles) {}
  }
};

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  return f32_to_bf16_bits(lo) | (f32_to_bf16_bits(hi) << 16);
}
__device__ __forceinline__ uint32_t pack_f16x2_sat(float lo, float hi) {
  lo = fminf(fmaxf(lo, -65504.f), 65504.f);
  hi = fminf(fmaxf(hi, -65504.f), 65504.f);
  return (uint32_t)__half_as_ushort(__float2half_rn(lo)) | ((uint32_t)__half_as_ushort(__float2half_rn(hi)) << 16);
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t hfma2_f16(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t d;
  asm("fma.rn.f16x2 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}
__device__ __forceinline__ uint32_t hfma2_bf16(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t d;
  asm("fma.rn.bf16x2 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}
__device__ __forceinline__ uint32_t hsub2_bf16(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("sub.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}
__device__ __forceinline__ uint32_t hmul2_bf16(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}
__device__ __forceinline__ uint32_t and_or(uint32_t a, uint32_t mask, uint32_t orv) { return (a & mask) | orv; }

// Byte offset of 16-byte chunk `chunk` (0..15) of row `row` inside a 128-row, 128-column 16-bit tile
// stored as two 64-column blocks in the 128-byte-swizzled layout the tensor core reads.
__device__ __forceinline__ uint32_t sw128_offset(int row, int chunk) {
  return (uint32_t)((chunk >> 3) * kHalfTile + row * 128 + (((chunk & 7) ^ (row & 7)) << 4));
}
// Byte offset of row `row`, 16-byte k-chunk `kc` (0..1) inside a 128 x 16 unswizzled bias operand tile:
// 8-row x 16-byte core matrices, the two k-chunks 128 bytes apart, 8-row groups 256 bytes apart.
__device__ __forceinline__ uint32_t xtile_offset(int row, int kc) {
  return (uint32_t)((row >> 3) * 256 + kc * 128 + (row & 7) * 16);
}

template <int BITS>
struct Raw {   // packed codes and metadata of one cached token (keys or values)
  static constexpr int kWords = kD * BITS / 32;
  uint32_t w[kWords];
  uint32_t sbytes;       // scale bytes of up to 4 groups
  uint32_t z01, z23;     // zero-points (BF16 bits) of up to 4 groups
};

template <int BITS, int G>
__device__ __forceinline__ void load_raw(Raw<BITS>& r, const uint8_t* codes, const uint8_t* scale, const uint16_t* zero,
                                         int64_t tok, bool valid) {
  if (!valid) {   // rows past the end of the cache dequantize to exact zeros
#pragma unroll
    for (int i = 0; i < Raw<BITS>::kWords; ++i) r.w[i] = 0;
    r.sbytes = 0; r.z01 = 0; r.z23 = 0;
    return;
  }
  const uint4* cw = reinterpret_cast<const uint4*>(codes + tok * (kD * BITS / 8));
#pragma unroll
  for (int i = 0; i < Raw<BITS>::kWords / 4; ++i) {
    const uint4 v = __ldg(cw + i);
    r.w[4 * i] = v.x; r.w[4 * i + 1] = v.y; r.w[4 * i + 2] = v.z; r.w[4 * i + 3] = v.w;
  }
  if constexpr (G == 1) {
    r.sbytes = __ldg(scale + tok); r.z01 = __ldg(zero + tok); r.z23 = 0;
  } else if constexpr (G == 2) {
    r.sbytes = __ldg(reinterpret_cast<const uint16_t*>(scale + tok * 2));
    r.z01 = __ldg(reinterpret_cast<const uint32_t*>(zero + tok * 2)); r.z23 = 0;
  } else {
    r.sbytes = __ldg(reinterpret_cast<const uint32_t*>(scale + tok * 4));
    const uint2 z = __ldg(reinterpret_cast<const uint2*>(zero + tok * 4));
    r.z01 = z.x; r.z23 = z.y;
  }
}

template <int BITS>
__device__ __forceinline__ float raw_step(const Raw<BITS>& r, int j) { return e4m3_byte_to_f32((r.sbytes >> (8 * j)) & 0xFFu); }
template <int BITS>
__device__ __forceinline__ float raw_zero(const Raw<BITS>& r, int j) {
  const uint32_t z = (j < 2) ? r.z01 : r.z23;
  return bf16_bits_to_f32((z >> (16 * (j & 1))) & 0xFFFFu);
}

// Keys: x^ = (code - zero) * step as FP16, one FMA per pair: (OFF + code) * step - (OFF + zero) * step
// with OFF = 4 (2-bit) or 16 (4-bit) coming for free from the exponent bits OR-ed over the code.
// Pairs are (i, i + 8) of each 16-code word (2-bit) or (i, i + 4) of each 8-code word (4-bit): the
// contraction dimension is stored permuted, and the rotated query is stored with the same permutation.
template <int BITS, int GROUP>
__device__ __forceinline__ void dequant_keys(const Raw<BITS>& r, uint8_t* tile, int key) {
  constexpr int group = GROUP;
  constexpr float kOff = (BITS == 2) ? 4.f : 16.f;
  uint32_t step2[4], c2[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const float ds = raw_step<BITS>(r, j), zs = raw_zero<BITS>(r, j);
    step2[j] = pack_f16x2_sat(ds, ds);
    const float c = -(kOff + zs) * ds;
    c2[j] = pack_f16x2_sat(c, c);
  }
  if constexpr (BITS == 2) {
#pragma unroll
    for (int wi = 0; wi < 8; ++wi) {
      const int j = (wi * 16) / group;
      const uint32_t w = r.w[wi];
      uint32_t o[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const uint32_t sh = (i <= 4) ? (w << (8 - 2 * i)) : (w >> (2 * i - 8));
        o[i] = hfma2_f16(and_or(sh, 0x03000300u, 0x44004400u), step2[j], c2[j]);
      }
      *reinterpret_cast<uint4*>(tile + sw128_offset(key, 2 * wi)) = make_uint4(o[0], o[1], o[2], o[3]);
      *reinterpret_cast<uint4*>(tile + sw128_offset(key, 2 * wi + 1)) = make_uint4(o[4], o[5], o[6], o[7]);
    }
  } else {
#pragma unroll
    for (int wi = 0; wi < 16; ++wi) {
      const int j = (wi * 8) / group;
      const uint32_t w = r.w[wi];
      uint32_t o[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint32_t sh = (i <= 1) ? (w << (6 - 4 * i)) : (w >> (4 * i - 6));
        o[i] = hfma2_f16(and_or(sh, 0x03C003C0u, 0x4C004C00u), step2[j], c2[j]);
      }
      *reinterpret_cast<uint4*>(tile + sw128_offset(key, wi)) = make_uint4(o[0], o[1], o[2], o[3]);
    }
  }
}

// Values: same reconstruction as BF16, channels in natural order (the output dimension cannot be permuted
// because current-chunk values arrive unpermuted).  2-bit: one FMA per pair; 4-bit: exact subtract then
// multiply (the 16 + zero offset times the step is not always representable in BF16).
template <int BITS, int GROUP>
__device__ __forceinline__ void dequant_values(const Raw<BITS>& r, uint8_t* tile, int key) {
  constexpr int group = GROUP;
  uint32_t step2[4], c2[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const float ds = raw_step<BITS>(r, j), zs = raw_zero<BITS>(r, j);
    step2[j] = pack_bf16x2(ds, ds);
    const float c = (BITS == 2) ? -(4.f + zs) * ds : (16.f + zs);
    c2[j] = pack_bf16x2(c, c);
  }
  if constexpr (BITS == 2) {
#pragma unroll
    for (int wi = 0; wi < 8; ++wi) {
      const int j = (wi * 16) / group;
      const uint32_t w = r.w[wi];
      const uint32_t lo = w & 0x33333333u, hi = (w >> 2) & 0x33333333u;
      const uint32_t z1 = (lo & 0xFFFFu) | (hi << 16), z2 = (lo >> 16) | (hi & 0xFFFF0000u);
      uint32_t o[8];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint32_t s1 = (i <= 1) ? (z1 << (5 - 4 * i)) : (z1 >> (4 * i - 5));
        const uint32_t s2 = (i <= 1) ? (z2 << (5 - 4 * i)) : (z2 >> (4 * i - 5));
        o[i] = hfma2_bf16(and_or(s1, 0x00600060u, 0x40804080u), step2[j], c2[j]);
        o[4 + i] = hfma2_bf16(and_or(s2, 0x00600060u, 0x40804080u), step2[j], c2[j]);
      }
      *reinterpret_cast<uint4*>(tile + sw128_offset(key, 2 * wi)) = make_uint4(o[0], o[1], o[2], o[3]);
      *reinterpret_cast<uint4*>(tile + sw128_offset(key, 2 * wi + 1)) = make_uint4(o[4], o[5], o[6], o[7]);
    }
  } else {
#pragma unroll
    for (int wi = 0; wi < 16; ++wi) {
      const int j = (wi * 8) / group;
      const uint32_t w = r.w[wi];
      const uint32_t lo = w & 0x0F0F0F0Fu, hi = (w >> 4) & 0x0F0F0F0Fu;
      const uint32_t z1 = (lo & 0xFFFFu) | (hi << 16), z2 = (lo >> 16) | (hi & 0xFFFF0000u);
      uint32_t o[4];
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const uint32_t s1 = (i == 0) ? (z1 << 3) : (z1 >> 5);
        const uint32_t s2 = (i == 0) ? (z2 << 3) : (z2 >> 5);
        o[i] = hmul2_bf16(hsub2_bf16(and_or(s1, 0x00780078u, 0x41804180u), c2[j]), step2[j]);
        o[2 + i] = hmul2_bf16(hsub2_bf16(and_or(s2, 0x00780078u, 0x41804180u), c2[j]), step2[j]);
      }
      *reinterpret_cast<uint4*>(tile + sw128_offset(key, wi)) = make_uint4(o[0], o[1], o[2], o[3]);
    }
  }
}

template <int BITS, int GROUP>
__global__ void __launch_bounds__(kThreads, 1)
attn_tcgen05_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                    const __grid_constant__ CUtensorMap tm_v, const TParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t sbase = smem_u32(smem);
  volatile int* misc = reinterpret_cast<volatile int*>(smem + kOffMisc);   // [0] tmem base, [1] abort flag
  Ctx cx{sbase + kOffBar, misc + 1, p.status};

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int bh = blockIdx.y, b = bh / p.heads, h = bh - b * p.heads;
  const int row0 = blockIdx.x * (2 * kBlockM);
  const int n_rt = (p.n_cur + kBlockN - 1) / kBlockN;
  const int n_ct = (p.n_cached + kBlockN - 1) / kBlockN;
  const int T = n_rt + n_ct;
  constexpr int G = kD / GROUP;

  if (tid == 0) {
    misc[1] = 0;
    mbar_init(cx.bar(kQFull), 1);
    for (int s = 0; s < 2; ++s) {
      mbar_init(cx.bar(kKFull + s), 129);   // 128 dequant threads + the TMA thread, every tile
      mbar_init(cx.bar(kVFull + s), 129);
      mbar_init(cx.bar(kKEmpty + s), 1);
      mbar_init(cx.bar(kVEmpty + s), 1);
      mbar_init(cx.bar(kSFull + s), 1);
      mbar_init(cx.bar(kPFull + s), 128);
      mbar_init(cx.bar(kODone + s), 1);
    }
    mbar_init(cx.bar(kQCurDone), 1);
    mbar_init(cx.bar(kQRotFull), 128);
    mbar_init(cx.bar(kDrain), 1);
    fence_barrier_init();
    prefetch_tensormap(&tm_q); prefetch_tensormap(&tm_k); prefetch_tensormap(&tm_v);
  }
  // bias operand tiles start as zeros (columns beyond the group count stay zero for good)
  for (int i = tid; i < 4 * kXBytes / 16; i += kThreads)
    reinterpret_cast<uint4*>(smem + kOffAx)[i] = make_uint4(0, 0, 0, 0);
  if (warp == 0) {
    tmem_alloc(sbase + kOffMisc, 512);
    tmem_relinquish();
  }
  fence_proxy_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(smem + kOffMisc);
  // TMEM columns: S0 [0,128) S1 [128,256) O0 [256,384) O1 [384,512); P_q aliases the first 64 columns of S_q.

  if (warp < 4) {
    setmaxnreg_dec<kRegsIssue>();
  if (warp == 0) {
    // ================= TMA producer =================
    if (lane == 0) {
      mbar_arrive_expect_tx(cx.bar(kQFull), 2 * kTileBytes);
      for (int qt = 0; qt < 2; ++qt)
        for (int kb = 0; kb < 2; ++kb)
          tma_load_4d(sbase + kOffQ + qt * kTileBytes + kb * kHalfTile, &tm_q, cx.bar(kQFull), kb * 64, row0 + qt * kBlockM, h, b);
      int issued = 0;
      for (int t = 0; t < T; ++t) {
        const int s = t & 1;
        const uint32_t ph = (t >> 1) & 1;
        if (!cx.wait(kKEmpty + s, ph ^ 1, 101)) break;
        if (t < n_rt) {
          mbar_arrive_expect_tx(cx.bar(kKFull + s), kTileBytes);
          for (int kb = 0; kb < 2; ++kb)
            tma_load_4d(sbase + kOffK + s * kTileBytes + kb * kHalfTile, &tm_k, cx.bar(kKFull + s), kb * 64, t * kBlockN, h, b);
        } else {
          mbar_arrive(cx.bar(kKFull + s));
        }
        if (!cx.wait(kVEmpty + s, ph ^ 1, 102)) break;
        if (t < n_rt) {
          mbar_arrive_expect_tx(cx.bar(kVFull + s), kTileBytes);
          for (int kb = 0; kb < 2; ++kb)
            tma_load_4d(sbase + kOffV + s * kTileBytes + kb * kHalfTile, &tm_v, cx.bar(kVFull + s), kb * 64, t * kBlockN, h, b);
          issued = t + 1;
        } else {
          mbar_arrive(cx.bar(kVFull + s));
        }
      }
      if (*cx.abort) {   // drain: give loads already in flight a bounded time to land before the CTA exits
        cx.drain(kQFull, 0);
        for (int t = max(0, issued - 2); t < issued; ++t) {
          cx.drain(kKFull + (t & 1), (t >> 1) & 1);
          cx.drain(kVFull + (t & 1), (t >> 1) & 1);
        }
      }
    }
  } else if (warp == 1) {
    // ================= MMA issuer =================
    if (lane == 0) {
      const uint32_t idesc_bf16 = make_idesc_bf16(128, 128, 0, 0);
      const uint32_t idesc_f16 = idesc_bf16 & ~((7u << 7) | (7u << 10));     // A, B format 0 = FP16
      const uint32_t idesc_pv = make_idesc_bf16(128, 128, 0, 1);              // B (values) is MN-major
      auto issue_qk = [&](int qt, int t) {
        const int s = t & 1;
        const bool cached = t >= n_rt;
        const uint32_t idesc = cached ? idesc_f16 : idesc_bf16;
        const uint32_t qa = sbase + kOffQ + qt * kTileBytes, ka = sbase + kOffK + s * kTileBytes;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          const uint32_t off = (ks >> 2) * kHalfTile + (ks & 3) * 32;
          mma_ss(tmem + qt * 128, make_smem_desc(qa + off, 16, 1024, kLayoutSw128),
                 make_smem_desc(ka + off, 16, 1024, kLayoutSw128), idesc, ks > 0);
        }
        if (cached && p.correction)
          mma_ss(tmem + qt * 128, make_smem_desc(sbase + kOffAx + qt * kXBytes, 128, 256, kLayoutNone),
                 make_smem_desc(sbase + kOffBx + s * kXBytes, 128, 256, kLayoutNone), idesc_bf16, 1);
        tc_commit(cx.bar(kSFull + qt));
      };
      auto issue_pv = [&](int qt, int t) {
        const int s = t & 1;
        const uint32_t va = sbase + kOffV + s * kTileBytes;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks)
          mma_ts(tmem + 256 + qt * 128, tmem + qt * 128 + ks * 8,
                 make_smem_desc(va + ks * 2048, kHalfTile, 1024, kLayoutSw128), idesc_pv, (t > 0 || ks > 0));
        tc_commit(cx.bar(kODone + qt));
      };
      bool ok = cx.wait(kQFull, 0, 201) && cx.wait(kKFull + 0, 0, 202);
      if (ok) {
        tc_fence_after();
        issue_qk(0, 0);
        issue_qk(1, 0);
        tc_commit(cx.bar(kKEmpty + 0));
        if (n_rt == 1) tc_commit(cx.bar(kQCurDone));
      }
      for (int t = 0; ok && t < T; ++t) {
        const int s = t & 1;
        const uint32_t ph = (t >> 1) & 1;
        const bool next = t + 1 < T;
        const bool switch_next = next && (t + 1 == n_rt);
        const int s1 = (t + 1) & 1;
        const uint32_t ph1 = ((t + 1) >> 1) & 1;
        if (!(ok = cx.wait(kVFull + s, ph, 203))) break;
        if (!(ok = cx.wait(kPFull + 0, t & 1, 204))) break;
        tc_fence_after();
        issue_pv(0, t);
        if (next && !switch_next) {
          if (!(ok = cx.wait(kKFull + s1, ph1, 205))) break;
          tc_fence_after();
          issue_qk(0, t + 1);
        }
        if (!(ok = cx.wait(kPFull + 1, t & 1, 206))) break;
        tc_fence_after();
        issue_pv(1, t);
        tc_commit(cx.bar(kVEmpty + s));
        if (next) {
          if (switch_next) {
            if (!(ok = cx.wait(kQRotFull, 0, 207))) break;
            if (!(ok = cx.wait(kKFull + s1, ph1, 208))) break;
            tc_fence_after();
            issue_qk(0, t + 1);
          }
          issue_qk(1, t + 1);
          tc_commit(cx.bar(kKEmpty + s1));
          if (t + 1 == n_rt - 1) tc_commit(cx.bar(kQCurDone));
        }
      }
      // everything issued so far must have retired before TMEM is freed
      tc_commit(cx.bar(kDrain));
      cx.drain(kDrain, 0);
    }
  }
  } else if (warp < 12) {
    // ================= softmax groups =================
    setmaxnreg_inc<kRegsSoftmax>();
    const int qt = (warp - 4) >> 2;
    const int wq = warp & 3;
    const int r_in_tile = wq * 32 + lane;
    const int row = row0 + qt * kBlockM + r_in_tile;
    const uint32_t lane_addr = (uint32_t)(wq * 32) << 16;
    const uint32_t s_addr = tmem + lane_addr + qt * 128;
    const uint32_t o_addr = tmem + lane_addr + 256 + qt * 128;
    const float c_row = p.scale_log2;
    float m = -INFINITY, l_cur = 0.f, l_cac = 0.f;
    bool ok = true;
    for (int t = 0; t < T; ++t) {
      const bool cached = t >= n_rt;
      const int n_valid = cached ? min(kBlockN, p.n_cached - (t - n_rt) * kBlockN) : min(kBlockN, p.n_cur - t * kBlockN);
      ok = __all_sync(0xFFFFFFFFu, cx.wait(kSFull + qt, t & 1, 301));
      if (!ok) break;
      tc_fence_after();
      uint32_t sr[128];                          // this row's 128 scores, then its 64 packed probabilities
#pragma unroll
      for (int c = 0; c < 4; ++c) tmem_ld32(s_addr + 32 * c, sr + 32 * c);
      tmem_wait_ld();
      if (n_valid < kBlockN) {                   // ragged last tile of a segment
#pragma unroll
        for (int i = 0; i < 128; ++i)
          if (i >= n_valid) sr[i] = 0xFF800000u;  // -inf
      }
      float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
      for (int i = 0; i < 128; i += 4) {
        mx0 = max3(mx0, __uint_as_float(sr[i]), __uint_as_float(sr[i + 1]));
        mx1 = max3(mx1, __uint_as_float(sr[i + 2]), __uint_as_float(sr[i + 3]));
      }
      const float m_new = fmaxf(m, fmaxf(mx0, mx1) * c_row);
      if (__any_sync(0xFFFFFFFFu, m_new - m > kRescaleThreshold)) {
        if (t > 0) {
          ok = __all_sync(0xFFFFFFFFu, cx.wait(kODone + qt, (t - 1) & 1, 302));
          if (!ok) break;
          tc_fence_after();
          const float f = ex2(m - m_new);
#pragma unroll 1
          for (int c = 0; c < 8; ++c) {
            uint32_t r[16];
            tmem_ld16(o_addr + 16 * c, r);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 16; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * f);
            tmem_st16(o_addr + 16 * c, r);
          }
          l_cur *= f; l_cac *= f;
        }
        m = m_new;
      }
      const float2 c2 = make_float2(c_row, c_row), nm2 = make_float2(-m, -m);
      float2 sum2 = make_float2(0.f, 0.f);
#pragma unroll
      for (int i = 0; i < 128; i += 2) {
        const float2 x = __ffma2_rn(make_float2(__uint_as_float(sr[i]), __uint_as_float(sr[i + 1])), c2, nm2);
        const float p0 = ex2(x.x), p1 = ex2(x.y);
        sum2 = __fadd2_rn(sum2, make_float2(p0, p1));
        sr[i >> 1] = cvt_bf16x2(p0, p1);
      }
      tmem_st32(s_addr, sr);
      tmem_st32(s_addr + 32, sr + 32);
      if (cached) l_cac += sum2.x + sum2.y; else l_cur += sum2.x + sum2.y;
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(cx.bar(kPFull + qt));
    }
    if (ok) ok = __all_sync(0xFFFFFFFFu, cx.wait(kODone + qt, (T - 1) & 1, 303));
    if (ok) {
      tc_fence_after();
      const float l = l_cur + l_cac;
      const float inv = 1.0f / l;
      uint16_t* dst = p.out + (int64_t)b * p.o_sb + (int64_t)h * p.o_sh + (int64_t)row * p.o_st;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t r[32];
        tmem_ld32(o_addr + 32 * c, r);
        tmem_wait_ld();
        if (row < p.m_tokens) {
#pragma unroll
          for (int i = 0; i < 32; i += 8) {
            uint4 v;
            v.x = pack_bf16x2(__uint_as_float(r[i]) * inv, __uint_as_float(r[i + 1]) * inv);
            v.y = pack_bf16x2(__uint_as_float(r[i + 2]) * inv, __uint_as_float(r[i + 3]) * inv);
            v.z = pack_bf16x2(__uint_as_float(r[i + 4]) * inv, __uint_as_float(r[i + 5]) * inv);
            v.w = pack_bf16x2(__uint_as_float(r[i + 6]) * inv, __uint_as_float(r[i + 7]) * inv);
            *reinterpret_cast<uint4*>(dst + 32 * c + i) = v;
          }
        }
      }
      if (row < p.m_tokens) {
        const int64_t idx = (int64_t)bh * p.m_tokens + row;
        if (p.lse) p.lse[idx] = (m + log2f(l)) * 0.6931471805599453f;
        if (p.cached_mass) p.cached_mass[idx] = l_cac * inv;
      }
    }
    tc_fence_before();
  } else {
    // ================= dequant + query rotation =================
    setmaxnreg_dec<kRegsDequant>();
    const int dt = tid - 12 * 32;          // 0..127: the key of the tile this thread expands
    const int64_t tok0 = (int64_t)bh * p.capacity + p.cache_begin;
    Raw<BITS> rk, rv;
    if (n_ct > 0) {
      const bool valid = dt < p.n_cached;
      load_raw<BITS, G>(rk, p.k_codes, p.k_scale, p.k_zero, tok0 + dt, valid);
      load_raw<BITS, G>(rv, p.v_codes, p.v_scale, p.v_zero, tok0 + dt, valid);
    }
    bool ok = true;
    for (int t = 0; t < T; ++t) {
      const int s = t & 1;
      const uint32_t ph = (t >> 1) & 1;
      const int ct = t - n_rt;
      ok = __all_sync(0xFFFFFFFFu, cx.wait(kKEmpty + s, ph ^ 1, 401));
      if (!ok) break;
      if (ct >= 0) {
        dequant_keys<BITS, GROUP>(rk, smem + kOffK + s * kTileBytes, dt);
        if (p.correction) {   // B_extra row: step_j^2, exact in BF16
          const float d0 = raw_step<BITS>(rk, 0), d1 = raw_step<BITS>(rk, 1), d2 = raw_step<BITS>(rk, 2), d3 = raw_step<BITS>(rk, 3);
          const uint32_t b01 = pack_bf16x2(d0 * d0, G > 1 ? d1 * d1 : 0.f), b23 = pack_bf16x2(G > 2 ? d2 * d2 : 0.f, G > 3 ? d3 * d3 : 0.f);
          // columns 0..3 meet the high parts of A_extra, columns 4..7 the low parts
          *reinterpret_cast<uint4*>(smem + kOffBx + s * kXBytes + xtile_offset(dt, 0)) = make_uint4(b01, b23, b01, b23);
        }
        fence_proxy_async_smem();
        if (ct + 1 < n_ct) {
          const int k1 = (ct + 1) * kBlockN + dt;
          load_raw<BITS, G>(rk, p.k_codes, p.k_scale, p.k_zero, tok0 + k1, k1 < p.n_cached);
        }
      }
      mbar_arrive(cx.bar(kKFull + s));
      if (ct == 0) {
        // ---- rotate the query tile in place; per-group squared norms -> A_extra ----
        ok = __all_sync(0xFFFFFFFFu, cx.wait(kQFull, 0, 402) && cx.wait(kQCurDone, 0, 403));
        if (!ok) break;
        const int l16 = lane & 15, rsub = lane >> 4;
        constexpr int lanes_per_group = GROUP / 8;
        float sgn[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) sgn[e] = (p.rotate && p.signs) ? (float)p.signs[l16 * 8 + e] : 1.0f;
        for (int pass = 0; pass < 32; ++pass) {
          const int qrow = pass * 8 + (warp - 12) * 2 + rsub;     // 0..255
          const int qt = qrow >> 7, rr = qrow & 127;
          uint8_t* qtile = smem + kOffQ + qt * kTileBytes;
          const uint4 raw = *reinterpret_cast<const uint4*>(qtile + sw128_offset(rr, l16));
          float x[8];
          x[0] = bf16_bits_to_f32(raw.x & 0xFFFFu); x[1] = bf16_bits_to_f32(raw.x >> 16);
          x[2] = bf16_bits_to_f32(raw.y & 0xFFFFu); x[3] = bf16_bits_to_f32(raw.y >> 16);
          x[4] = bf16_bits_to_f32(raw.z & 0xFFFFu); x[5] = bf16_bits_to_f32(raw.z >> 16);
          x[6] = bf16_bits_to_f32(raw.w & 0xFFFFu); x[7] = bf16_bits_to_f32(raw.w >> 16);
          if (p.rotate) {
#pragma unroll
            for (int e = 0; e < 8; ++e) x[e] *= sgn[e];
#pragma unroll
            for (int hh = 1; hh < 8; hh *= 2)
#pragma unroll
              for (int i = 0; i < 8; ++i)
                if ((i & hh) == 0) { const float a = x[i], c = x[i + hh]; x[i] = a + c; x[i + hh] = a - c; }
#pragma unroll
            for (int lm = 1; lm < 16; lm *= 2)
#pragma unroll
              for (int e = 0; e < 8; ++e) {
                const float o = __shfl_xor_sync(0xFFFFFFFFu, x[e], lm);
                x[e] = (l16 & lm) ? (o - x[e]) : (x[e] + o);
              }
#pragma unroll
            for (int e = 0; e < 8; ++e) x[e] *= 0.08838834764831845f;
          }
          float nu = 0.f;
#pragma unroll
          for (int e = 0; e < 8; ++e) nu += x[e] * x[e];
          for (int off = 1; off < lanes_per_group; off *= 2) nu += __shfl_xor_sync(0xFFFFFFFFu, nu, off);
          if ((l16 % lanes_per_group) == 0) {
            const int j = l16 / lanes_per_group;
            // -(sigma/24) nu as a BF16 high part plus a BF16 low part (columns j and 4 + j)
            const float a = p.ax_coef * nu;
            const uint32_t hi = f32_to_bf16_bits(a);
            uint8_t* ax = smem + kOffAx + qt * kXBytes + xtile_offset(rr, 0);
            *reinterpret_cast<uint16_t*>(ax + 2 * j) = (uint16_t)hi;
            *reinterpret_cast<uint16_t*>(ax + 8 + 2 * j) = (uint16_t)f32_to_bf16_bits(a - bf16_bits_to_f32(hi));
          }
          float y[8];
          if constexpr (BITS == 2) {
            // physical column 16w + 2i + hsel <- channel 16w + i + 8*hsel: even lanes own the low half
            // of a 16-channel word, odd lanes the high half; swap four values with the neighbour
            const bool odd = l16 & 1;
            float rcv[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) rcv[i] = __shfl_xor_sync(0xFFFFFFFFu, odd ? x[i] : x[4 + i], 1);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              y[2 * i] = odd ? rcv[i] : x[i];
              y[2 * i + 1] = odd ? x[4 + i] : rcv[i];
            }
          } else {
            // physical column 8w + 2i + hsel <- channel 8w + i + 4*hsel
#pragma unroll
            for (int i = 0; i < 4; ++i) { y[2 * i] = x[i]; y[2 * i + 1] = x[4 + i]; }
          }
          *reinterpret_cast<uint4*>(qtile + sw128_offset(rr, l16)) =
              make_uint4(pack_f16x2_sat(y[0], y[1]), pack_f16x2_sat(y[2], y[3]), pack_f16x2_sat(y[4], y[5]), pack_f16x2_sat(y[6], y[7]));
        }
        fence_proxy_async_smem();
        mbar_arrive(cx.bar(kQRotFull));
      }
      ok = __all_sync(0xFFFFFFFFu, cx.wait(kVEmpty + s, ph ^ 1, 404));
      if (!ok) break;
      if (ct >= 0) {
        dequant_values<BITS, GROUP>(rv, smem + kOffV + s * kTileBytes, dt);
        fence_proxy_async_smem();
        if (ct + 1 < n_ct) {
          const int k1 = (ct + 1) * kBlockN + dt;
          load_raw<BITS, G>(rv, p.v_codes, p.v_scale, p.v_zero, tok0 + k1, k1 < p.n_cached);
        }
      }
      mbar_arrive(cx.bar(kVFull + s));
    }
  }

  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

// ---- host side -----------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

int get_encode_fn(EncodeTiledFn* fn) {
  static EncodeTiledFn cached = nullptr;
  if (!cached) {
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult qres;
    KVQ_CUDA_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres));
    if (qres != cudaDriverEntryPointSuccess || !sym) return record_cuda_error(cudaErrorSymbolNotFound);
    cached = reinterpret_cast<EncodeTiledFn>(sym);
  }
  *fn = cached;
  return KVQ_OK;
}

// [batch, heads, tokens, 128] BF16 tensor -> 4-D map with a 64-column x 128-row box, 128-byte swizzle.
int make_map(EncodeTiledFn enc, CUtensorMap* map, const void* ptr, kvq_strides s, int64_t tokens, int heads, int batch) {
  cuuint64_t dims[4] = {(cuuint64_t)kD, (cuuint64_t)tokens, (cuuint64_t)heads, (cuuint64_t)batch};
  // a size-1 dimension may come with any stride; give it a harmless valid one
  const cuuint64_t st = (cuuint64_t)s.t * 2;
  const cuuint64_t sh = heads > 1 ? (cuuint64_t)s.h * 2 : st * (cuuint64_t)tokens;
  const cuuint64_t sb = batch > 1 ? (cuuint64_t)s.b * 2 : sh * (cuuint64_t)heads;
  cuuint64_t strides[3] = {st, sh, sb};
  for (cuuint64_t v : strides)
    if (v == 0 || v % 16 != 0 || v >= (1ull << 40)) return KVQ_ERR_UNSUPPORTED;
  cuuint32_t box[4] = {64, (cuuint32_t)kBlockN, 1, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(ptr), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return record_cuda_error(cudaErrorInvalidValue);
  return KVQ_OK;
}

template <int BITS, int GROUP>
int launch(const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv, const TParams& p, dim3 grid, cudaStream_t st) {
  static bool configured = false;
  if (!configured) {
    KVQ_CUDA_TRY(cudaFuncSetAttribute(attn_tcgen05_kernel<BITS, GROUP>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
    configured = true;
  }
  attn_tcgen05_kernel<BITS, GROUP><<<grid, kThreads, kSmemBytes, st>>>(mq, mk, mv, p);
  KVQ_CUDA_TRY(cudaGetLastError());
  return KVQ_OK;
}

}  // namespace

bool attn_tcgen05_supports(const kvq_cache_desc* d, int64_t m_tokens, int64_t n_cur) {
  return d->head_dim == kD && m_tokens >= 1 && n_cur >= 1 && (int64_t)d->batch * d->heads <= 65535;
}

size_t attn_tcgen05_workspace_bytes(const kvq_cache_desc*, int64_t, int64_t, int64_t) { return 0; }

int launch_attn_tcgen05(const AttnArgs& a) {
  const kvq_cache_desc* d = a.desc;
  EncodeTiledFn enc;
  int r = get_encode_fn(&enc);
  if (r != KVQ_OK) return r;
  CUtensorMap mq, mk, mv;
  if ((r = make_map(enc, &mq, a.q, a.qs, a.m_tokens, d->heads, d->batch)) != KVQ_OK) return r;
  if ((r = make_map(enc, &mk, a.k_cur, a.kvs, a.n_cur, d->heads, d->batch)) != KVQ_OK) return r;
  if ((r = make_map(enc, &mv, a.v_cur, a.kvs, a.n_cur, d->heads, d->batch)) != KVQ_OK) return r;
  TParams p;
  p.out = static_cast<uint16_t*>(a.out); p.o_sb = a.os.b; p.o_sh = a.os.h; p.o_st = a.os.t;
  p.k_codes = static_cast<const uint8_t*>(d->k_codes); p.v_codes = static_cast<const uint8_t*>(d->v_codes);
  p.k_scale = static_cast<const uint8_t*>(d->k_scale); p.v_scale = static_cast<const uint8_t*>(d->v_scale);
  p.k_zero = static_cast<const uint16_t*>(d->k_zero); p.v_zero = static_cast<const uint16_t*>(d->v_zero);
  p.signs = d->signs;
  p.capacity = d->capacity; p.cache_begin = a.cache_begin;
  p.heads = d->heads; p.group = d->group; p.rotate = (d->flags & KVQ_ROTATE_K) ? 1 : 0;
  p.correction = (a.flags & KVQ_CORRECTION_ON) ? 1 : 0;
  p.m_tokens = (int)a.m_tokens; p.n_cached = (int)a.cache_len; p.n_cur = (int)a.n_cur;
  p.scale_log2 = a.softmax_scale * kLog2e;
  p.ax_coef = -a.softmax_scale / 24.0f;
  p.lse = a.lse; p.cached_mass = a.cached_mass; p.status = a.status_word;
  dim3 grid((unsigned)((a.m_tokens + 2 * kBlockM - 1) / (2 * kBlockM)), (unsigned)((int64_t)d->batch * d->heads));
  if (d->bits == 2) {
    if (d->group == 32) return launch<2, 32>(mq, mk, mv, p, grid, a.stream);
    if (d->group == 64) return launch<2, 64>(mq, mk, mv, p, grid, a.stream);
    return launch<2, 128>(mq, mk, mv, p, grid, a.stream);
  }
  if (d->group == 32) return launch<4, 32>(mq, mk, mv, p, grid, a.stream);
  if (d->group == 64) return launch<4, 64>(mq, mk, mv, p, grid, a.stream);
  return launch<4, 128>(mq, mk, mv, p, grid, a.stream);
}

}  // namespace kvq
