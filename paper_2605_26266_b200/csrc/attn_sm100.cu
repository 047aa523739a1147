// Corrected chunk attention for sm_100a: TMA + tcgen05.mma with TMEM accumulators.
//
// A CTA works on 256 query rows of one (batch, head) at a time — two 128-row tiles that share the key and value
// tiles — and walks keys in tiles of 128: first the current chunk's BF16 keys and
// values (TMA straight into the 128-byte-swizzled operand layout, unrotated query, no bias),
// then the cached keys and values, which four "dequant" warps expand from the packed
// 2-/4-bit codes into the same operand layout in shared memory (never to HBM).  Between the
// two segments the rotated query tile (Hadamard, FP32 butterflies) and the per-group squared norms nu
// of Algorithm 1, both written by a small pre-pass kernel of the same call, replace the unrotated tile.
//
// Score of a cached key (Eq. (15) / Eq. (25)):  s = sigma*q~.k^ - (sigma^2/24) sum_j step_j^2 nu_j.
// The bias is folded into the score contraction as one extra K=16 MMA step per half tile:
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
// Roles (512 threads): warp 0 lane 0 issues TMA; warps 1 and 2 issue the tcgen05.mma of query tile 0 and 1 (each
// warp runs its schedule converged, one lane elected once issues); warps 4-7 are the softmax warps of query tile
// 0, warps 8-11 those of query tile 1: warp w reads TMEM lanes 32 (w % 4) .. + 31, one query row per lane, so
// row maxima and row sums need no exchange; warps 12-15 dequantize.  Registers are re-split between the roles
// with setmaxnreg.
//
// A key tile of 128 keys is processed in two halves of 64 keys, each with its own 64 score columns in TMEM:
// as soon as the softmax warps hand over P of one half (BF16 pairs written over the first 32 of that half's
// columns), the issuer adds P V of those 64 keys to O and computes the same half's scores of the NEXT key tile
// into the columns just freed, while the softmax warps work on the other half.  The scores a group needs next
// are therefore usually ready when it asks for them.
//
// The roles' loops are written to stay small (rolled over halves, query tiles and MMA groups): the SM's
// instruction cache, and the GPC-level one behind it, bounded this kernel before any pipe did; what bounds it
// now is the chain through a softmax group (score load, maximum, exponentials, store, hand-over).
//
// Work is cut into units (batch*head, 256-row query block) of `tiles` key tiles each.  Persistent CTAs take
// whole units in rounds; where that would leave SMs idle (a short last round, or fewer units than SMs) the
// unit x tile steps are divided evenly over one CTA per SM instead, a CTA walks its range segment by
// segment, split units leave partial results (their own normalised rows, running max, row sums) in the
// caller's workspace and a small kernel merges them.
//
// The same source also gives the pair kernel (template parameter PAIR): a cluster of two CTAs on 512 query rows
// whose tensor cores work as one (tcgen05 cta_group::2), described at the kernel.
//
// Every wait on an mbarrier is bounded: on expiry the CTA records a diagnostic in the caller's status
// word, all roles leave their loops, in-flight work is drained with a bounded wait, TMEM is freed and the
// kernel returns.
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
constexpr int kNumBars = 32;                       // mbarriers, 8 bytes each (enum Bar below)
static_assert(kNumBars * 8 <= 256, "barrier area");
constexpr int kOffMisc = kOffBar + 256;
constexpr int kSmemBytes = kOffMisc + 64 + 1024;   // + slack to align the base to 1024

// kSFull, kPFull and kODone have four barriers each: index 2 * (half of the key tile) + (query tile); each of
// them completes once per key tile, so that a waiter is never more than one phase behind
enum Bar { kQFull = 0, kKFull = 1, kVFull = 3, kKEmpty = 5, kVEmpty = 7, kSFull = 9, kPFull = 13,
           kODone = 17, kQCurDone = 21, kQRotFull = 22, kDrain = 23, kQEmpty = 25, kOFree = 26,
           kRawFull = 28, kRawEmpty = 30 };

// Pair kernel only: a CTA of a pair fills half of every operand stage (64 of the 128 key rows of each 64-column
// block, one of the two 64-channel value blocks), and the other half holds the staging ring for the PACKED tiles:
// codes and metadata of the 128 cached tokens of a tile, brought in by bulk copies one tile ahead, two stages.
// Codes of stage r sit in the unused value block of operand stage r (keys' codes, then values' codes, 8 KiB
// each), metadata in the unused rows of its first key block (key scales, key zero-points, value scales, value
// zero-points).
constexpr int kRawCodesOff = kHalfTile;            // from the start of the value stage
constexpr int kRawVCodes = 8192;                   // values' codes after the keys' codes
constexpr int kRawMetaOff = 64 * 128;              // from the start of the key stage: behind its 64 rows in use
constexpr int kRawKZero = 512, kRawVScale = 1536, kRawVZero = 2048;
static_assert(128 * (kD * 4 / 8) <= kRawVCodes && 2 * kRawVCodes <= kHalfTile, "packed codes fit the unused value block");
static_assert(kRawVZero + 128 * 4 * 2 <= kHalfTile - kRawMetaOff, "metadata fits the unused key rows");

constexpr uint32_t kTimeoutCycles = 2000000000u;   // about a second; 32-bit clock differences stay exact below 2^32
constexpr uint32_t kDrainCycles = 20000000u;
constexpr float kLog2e = 1.4426950408889634f;
// registers per thread after reallocation: 128 * 96 + 256 * 144 + 128 * 112 = 63488 <= 65536
constexpr int kRegsIssue = 96, kRegsSoftmax = 144, kRegsDequant = 112;
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
  uint32_t wait_budget;    // cycles a device-side wait may take (kTimeoutCycles unless a test has shortened it)
  // schedule: units = (batch*head, 256-row query block); every unit has `tiles` key tiles (see Schedule)
  int q_blocks, n_units, tiles;
  int n_whole;             // units [0, n_whole) are computed whole; the rest are split over all CTAs
  uint8_t* partial;        // workspace: 2 slots per CTA, see kSlotBytes
  const uint16_t* ax_rows; // workspace: bias operand rows written by rotate_query_kernel, [batch*heads][m_tokens][8]
};

// One partial result: the segment's own normalised output O / l as BF16, then FP32 m[256], l_cur[256],
// l_cached[256] (running maximum in log2 units and the row sums over current and cached keys).  The output is
// stored by 16-byte pieces of 8 columns, piece (column group g, row r) at (g * 256 + r) * 16: the softmax
// threads hold one row each, so the 32 lanes of a store instruction write 512 contiguous bytes (row-major, they
// would write 32 pieces 256 bytes apart, and the load/store unit takes them one line at a time).
constexpr int kSlotStats = 256 * kD * 2;
constexpr int kSlotBytes = kSlotStats + 3 * 256 * 4;
static_assert(kSlotBytes % 256 == 0, "slots stay 256-byte aligned");

// A contiguous run of key tiles [tb, te) of one unit; `slot` is the CTA's partial-result slot if the run is
// not the whole unit.
struct Segment { int unit, tb, te, slot; };
// Work of one CTA.  Units [0, n_whole) are computed whole, CTA c taking units c, c + n_ctas, ... so that
// neighbouring CTAs walk the key tiles of neighbouring units (mostly the same head) at the same time and
// share them in L2.  The key-tile steps of the remaining units are cut into n_ctas equal contiguous
// ranges, one per CTA.  n_units * tiles < 2^31 (checked on the host).
struct Schedule {
  int tiles, n_ctas, n_whole;
  int u;                   // next whole unit of this CTA
  int g, g_end, first;     // range in the split part (tile steps counted from unit n_whole); its first unit
  __device__ __forceinline__ Schedule(int cta, int n_ctas_, const TParams& p)
      : tiles(p.tiles), n_ctas(n_ctas_), n_whole(p.n_whole), u(cta) {
    const long long Wr = (long long)(p.n_units - p.n_whole) * p.tiles;
    g = (int)(Wr * cta / n_ctas_);
    g_end = (int)(Wr * (cta + 1) / n_ctas_);
    first = n_whole + g / max(tiles, 1);
  }
  __device__ __forceinline__ bool next(Segment& sg) {
    if (u < n_whole) {
      sg.unit = u; sg.tb = 0; sg.te = tiles; sg.slot = 0;
      u += n_ctas;
      return true;
    }
    if (g >= g_end) return false;
    const int ru = g / tiles;
    sg.unit = n_whole + ru;
    sg.tb = g - ru * tiles;
    const int n = min(tiles - sg.tb, g_end - g);
    sg.te = sg.tb + n;
    sg.slot = sg.unit == first ? 0 : 1;
    g += n;
    return true;
  }
};

struct Ctx {
  uint32_t bar0;
  volatile int* abort;     // shared-memory word: 0, or the diagnostic code of the wait that gave up
  uint32_t budget;         // cycles a wait may take before it gives up
  __device__ __forceinline__ uint32_t bar(int i) const { return bar0 + 8u * i; }
  // Bounded wait; false once the CTA is aborting.  Written to be small: it is inlined at some forty
  // sites, and the roles' loops have to stay resident in the SM's instruction cache.
  __device__ __forceinline__ bool wait(int i, uint32_t parity, int code) const {
    const uint32_t b = bar(i);
    if (mbar_try_wait(b, parity)) return true;
    const uint32_t t0 = (uint32_t)clock();
    while (!mbar_try_wait(b, parity)) {
      if (*abort) return false;
      if ((uint32_t)clock() - t0 > budget) { *abort = code; return false; }
    }
    return true;
  }
  // Used only on the way out: lets work already in flight finish, ignoring the abort flag.
  __device__ __forceinline__ void drain(int i, uint32_t parity) const {
    const uint32_t b = bar(i);
    const uint32_t t0 = (uint32_t)clock();
    while (!mbar_try_wait(b, parity) && (uint32_t)clock() - t0 < kDrainCycles) {}
  }
};

// Development aid, compiled in only with -DKVQ_TRACE: lane 0 of every warp of CTA 0 records (event id, clock)
// pairs in a device array that kvq_debug_trace_read() copies to the host.  The library proper has none of it.
#ifdef KVQ_TRACE
constexpr int kTraceLen = 4096;
__device__ uint32_t g_trace[16][kTraceLen];
#define KVQ_TRACE_DECL int trace_n = 0
#define KVQ_STAMP(id)                                                                            \
  do {                                                                                           \
    if (blockIdx.x == 0 && (threadIdx.x & 31) == 0 && trace_n < kTraceLen)                       \
      g_trace[threadIdx.x >> 5][trace_n++] = ((uint32_t)(id) << 26) | ((uint32_t)clock() & 0x3FFFFFFu); \
  } while (0)
#else
#define KVQ_TRACE_DECL
#define KVQ_STAMP(id)
#endif

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
// Of every four pairs of scores, how many take their exponentials on the FMA pipe instead of the MUFU (16 lanes
// per SM: the two softmax warps of a scheduler share 4).  Measured: one of four is worth 2 to 5 % in the pair
// kernel, where the MUFU is what the softmax groups wait for; in the one-CTA kernel the extra instructions cost as
// much as they save, so it keeps the MUFU for all.
constexpr int kPolyPairs = 1;
// 2^x for a pair of arguments without the MUFU: x = n + r with n the nearest integer (taken from the low mantissa
// bits of x + 1.5 * 2^23) and r in [-0.5, 0.5]; 2^r by a cubic (relative error 7.5e-5, far below the BF16
// rounding that follows); n goes into the exponent field by an integer add.  Arguments are clamped at -125, so
// the result is at least 2^-126 where the MUFU would flush to zero; x may be -inf.
__device__ __forceinline__ float2 ex2_poly2(float2 x) {
  const float kMagic = 12582912.f;
  x.x = fmaxf(x.x, -125.f); x.y = fmaxf(x.y, -125.f);
  const float2 fl = __fadd2_rn(x, make_float2(kMagic, kMagic));
  const float2 n = __fadd2_rn(fl, make_float2(-kMagic, -kMagic));
  const float2 r = __fadd2_rn(x, make_float2(-n.x, -n.y));
  float2 q = __ffma2_rn(r, make_float2(0.05517164617776871f, 0.05517164617776871f), make_float2(0.2426111251115799f, 0.2426111251115799f));
  q = __ffma2_rn(q, r, make_float2(0.6932609677314758f, 0.6932609677314758f));
  q = __ffma2_rn(q, r, make_float2(0.9999280571937561f, 0.9999280571937561f));
  return make_float2(__uint_as_float(__float_as_uint(q.x) + (__float_as_uint(fl.x) << 23)),
                     __uint_as_float(__float_as_uint(q.y) + (__float_as_uint(fl.y) << 23)));
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

// Loads NW code words of the token, starting at word `word0` (a multiple of 4), into r.w[0 .. NW), and the token's
// metadata.  NW is the whole row, or half of it for a CTA of a pair.
template <int BITS, int G, int NW = Raw<BITS>::kWords>
__device__ __forceinline__ void load_raw(Raw<BITS>& r, const uint8_t* codes, const uint8_t* scale, const uint16_t* zero,
                                         int64_t tok, bool valid, int word0 = 0) {
  if (!valid) {   // rows past the end of the cache dequantize to exact zeros
#pragma unroll
    for (int i = 0; i < NW; ++i) r.w[i] = 0;
    r.sbytes = 0; r.z01 = 0; r.z23 = 0;
    return;
  }
  const uint4* cw = reinterpret_cast<const uint4*>(codes + tok * (kD * BITS / 8)) + (word0 >> 2);
#pragma unroll
  for (int i = 0; i < NW / 4; ++i) {
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

// The same from the staging ring in shared memory (pair kernel): `key` is the token's place in its tile.
template <int BITS, int G, int NW>
__device__ __forceinline__ void load_raw_staged(Raw<BITS>& r, const uint8_t* codes, const uint8_t* scale, const uint8_t* zero,
                                                int key, bool valid, int word0) {
  if (!valid) {
#pragma unroll
    for (int i = 0; i < NW; ++i) r.w[i] = 0;
    r.sbytes = 0; r.z01 = 0; r.z23 = 0;
    return;
  }
  const uint4* cw = reinterpret_cast<const uint4*>(codes + key * (kD * BITS / 8)) + (word0 >> 2);
#pragma unroll
  for (int i = 0; i < NW / 4; ++i) {
    const uint4 v = cw[i];
    r.w[4 * i] = v.x; r.w[4 * i + 1] = v.y; r.w[4 * i + 2] = v.z; r.w[4 * i + 3] = v.w;
  }
  if constexpr (G == 1) {
    r.sbytes = scale[key]; r.z01 = *reinterpret_cast<const uint16_t*>(zero + key * 2); r.z23 = 0;
  } else if constexpr (G == 2) {
    r.sbytes = *reinterpret_cast<const uint16_t*>(scale + key * 2);
    r.z01 = *reinterpret_cast<const uint32_t*>(zero + key * 4); r.z23 = 0;
  } else {
    r.sbytes = *reinterpret_cast<const uint32_t*>(scale + key * 4);
    const uint2 z = *reinterpret_cast<const uint2*>(zero + key * 8);
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

// One of up to four per-group constants, picked by a group index that may only be known at run time (a CTA of a
// pair works on the half of the row its rank selects); with a compile-time index this folds to a[j].
template <int G>
__device__ __forceinline__ uint32_t pick_group(const uint32_t* a, int j) {
  if constexpr (G == 1) return a[0];
  else if constexpr (G == 2) return j ? a[1] : a[0];
  else return (j & 2) ? ((j & 1) ? a[3] : a[2]) : ((j & 1) ? a[1] : a[0]);
}

// Keys: x^ = (code - zero) * step as FP16, one FMA per pair: (OFF + code) * step - (OFF + zero) * step
// with OFF = 4 (2-bit) or 16 (4-bit) coming for free from the exponent bits OR-ed over the code.
// Pairs are (i, i + 8) of each 16-code word (2-bit) or (i, i + 4) of each 8-code word (4-bit): the
// contraction dimension is stored permuted, and the rotated query is stored with the same permutation.
// Expands the NW words r.w[0 .. NW), which are words word0 .. word0 + NW - 1 of the token, into row `row` of the tile.
template <int BITS, int GROUP, int NW = Raw<BITS>::kWords>
__device__ __forceinline__ void dequant_keys(const Raw<BITS>& r, uint8_t* tile, int row, int word0 = 0) {
  constexpr int G = kD / GROUP;
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
    for (int wi = 0; wi < NW; ++wi) {
      const int gw = word0 + wi;
      const int j = (gw * 16) / GROUP;
      const uint32_t st = pick_group<G>(step2, j), cc = pick_group<G>(c2, j);
      const uint32_t w = r.w[wi];
      uint32_t o[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const uint32_t sh = (i <= 4) ? (w << (8 - 2 * i)) : (w >> (2 * i - 8));
        o[i] = hfma2_f16(and_or(sh, 0x03000300u, 0x44004400u), st, cc);
      }
      *reinterpret_cast<uint4*>(tile + sw128_offset(row, 2 * gw)) = make_uint4(o[0], o[1], o[2], o[3]);
      *reinterpret_cast<uint4*>(tile + sw128_offset(row, 2 * gw + 1)) = make_uint4(o[4], o[5], o[6], o[7]);
    }
  } else {
#pragma unroll
    for (int wi = 0; wi < NW; ++wi) {
      const int gw = word0 + wi;
      const int j = (gw * 8) / GROUP;
      const uint32_t st = pick_group<G>(step2, j), cc = pick_group<G>(c2, j);
      const uint32_t w = r.w[wi];
      uint32_t o[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint32_t sh = (i <= 1) ? (w << (6 - 4 * i)) : (w >> (4 * i - 6));
        o[i] = hfma2_f16(and_or(sh, 0x03C003C0u, 0x4C004C00u), st, cc);
      }
      *reinterpret_cast<uint4*>(tile + sw128_offset(row, gw)) = make_uint4(o[0], o[1], o[2], o[3]);
    }
  }
}

// Values: same reconstruction as BF16, channels in natural order (the output dimension cannot be permuted
// because current-chunk values arrive unpermuted).  2-bit: one FMA per pair; 4-bit: exact subtract then
// multiply (the 16 + zero offset times the step is not always representable in BF16).  Words as for the keys;
// the 16-byte pieces land at piece index (token's piece index - piece0), so that a CTA of a pair keeps its 64
// channels in one 64-column block.
template <int BITS, int GROUP, int NW = Raw<BITS>::kWords>
__device__ __forceinline__ void dequant_values(const Raw<BITS>& r, uint8_t* tile, int row, int word0 = 0, int piece0 = 0) {
  constexpr int G = kD / GROUP;
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
    for (int wi = 0; wi < NW; ++wi) {
      const int gw = word0 + wi;
      const int j = (gw * 16) / GROUP;
      const uint32_t st = pick_group<G>(step2, j), cc = pick_group<G>(c2, j);
      const uint32_t w = r.w[wi];
      const uint32_t lo = w & 0x33333333u, hi = (w >> 2) & 0x33333333u;
      const uint32_t z1 = (lo & 0xFFFFu) | (hi << 16), z2 = (lo >> 16) | (hi & 0xFFFF0000u);
      uint32_t o[8];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint32_t s1 = (i <= 1) ? (z1 << (5 - 4 * i)) : (z1 >> (4 * i - 5));
        const uint32_t s2 = (i <= 1) ? (z2 << (5 - 4 * i)) : (z2 >> (4 * i - 5));
        o[i] = hfma2_bf16(and_or(s1, 0x00600060u, 0x40804080u), st, cc);
        o[4 + i] = hfma2_bf16(and_or(s2, 0x00600060u, 0x40804080u), st, cc);
      }
      *reinterpret_cast<uint4*>(tile + sw128_offset(row, 2 * gw - piece0)) = make_uint4(o[0], o[1], o[2], o[3]);
      *reinterpret_cast<uint4*>(tile + sw128_offset(row, 2 * gw + 1 - piece0)) = make_uint4(o[4], o[5], o[6], o[7]);
    }
  } else {
#pragma unroll
    for (int wi = 0; wi < NW; ++wi) {
      const int gw = word0 + wi;
      const int j = (gw * 8) / GROUP;
      const uint32_t st = pick_group<G>(step2, j), cc = pick_group<G>(c2, j);
      const uint32_t w = r.w[wi];
      const uint32_t lo = w & 0x0F0F0F0Fu, hi = (w >> 4) & 0x0F0F0F0Fu;
      const uint32_t z1 = (lo & 0xFFFFu) | (hi << 16), z2 = (lo >> 16) | (hi & 0xFFFF0000u);
      uint32_t o[4];
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const uint32_t s1 = (i == 0) ? (z1 << 3) : (z1 >> 5);
        const uint32_t s2 = (i == 0) ? (z2 << 3) : (z2 >> 5);
        o[i] = hmul2_bf16(hsub2_bf16(and_or(s1, 0x00780078u, 0x41804180u), cc), st);
        o[2 + i] = hmul2_bf16(hsub2_bf16(and_or(s2, 0x00780078u, 0x41804180u), cc), st);
      }
      *reinterpret_cast<uint4*>(tile + sw128_offset(row, gw - piece0)) = make_uint4(o[0], o[1], o[2], o[3]);
    }
  }
}

// Pre-pass over the query chunk (one launch before the attention kernel): q~ = (1/sqrt d) H (signs . q) in
// FP32, stored as FP16 with the contraction dimension permuted the way the dequantized keys are laid out,
// and -(sigma/24) nu_{m,j} (per-group squared norms of q~) as a BF16 high part plus a BF16 low part.  The
// attention kernel swaps the rotated tile in by TMA once the current chunk's score MMAs are done, so units
// split over several CTAs rotate their rows once instead of once per CTA.
// 16 lanes per row, 8 channels per lane; a warp handles two rows, a block of 8 warps 16 rows (many small
// blocks: the kernel is a chain of dependent shuffles per row, so it wants every row in flight at once).
struct RotParams {
  const uint16_t* q; int64_t q_sb, q_sh, q_st;
  uint16_t* qr;            // [batch * heads][m_tokens][128] FP16
  uint16_t* ax;            // [batch * heads][m_tokens][8] BF16: high parts of groups 0..3, then low parts
  const int8_t* signs;
  int heads, m_tokens, rotate;
  float ax_coef;           // -sigma / 24
};

template <int BITS, int GROUP>
__global__ void __launch_bounds__(256) rotate_query_kernel(const RotParams p) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int l16 = lane & 15, rsub = lane >> 4;
  constexpr int lanes_per_group = GROUP / 8;
  const int bh = blockIdx.y, b = bh / p.heads, h = bh - b * p.heads;
  float sgn[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) sgn[e] = (p.rotate && p.signs) ? (float)p.signs[l16 * 8 + e] : 1.0f;
  {
    const int row = blockIdx.x * 16 + warp * 2 + rsub;
    const bool valid = row < p.m_tokens;             // no early exit: the shuffles below need every lane
    uint4 raw = make_uint4(0, 0, 0, 0);
    if (valid) raw = __ldg(reinterpret_cast<const uint4*>(p.q + (int64_t)b * p.q_sb + (int64_t)h * p.q_sh + (int64_t)row * p.q_st) + l16);
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
    {
      // -(sigma/24) nu_j as a BF16 high part plus a BF16 low part: columns j and 4 + j of the row's 16 bytes,
      // zeros for groups the format does not have; gathered from the group leaders and written by lane 0 of the row
      const float a = p.ax_coef * nu;
      const uint32_t hi = f32_to_bf16_bits(a);
      const uint32_t lo = f32_to_bf16_bits(a - bf16_bits_to_f32(hi));
      uint32_t h4[4], l4[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int src = (lane & 16) + ((j * lanes_per_group) & 15);
        const uint32_t hj = __shfl_sync(0xFFFFFFFFu, hi, src), lj = __shfl_sync(0xFFFFFFFFu, lo, src);
        const bool have = j * GROUP < kD;
        h4[j] = have ? hj : 0u; l4[j] = have ? lj : 0u;
      }
      if (valid && l16 == 0)
        *reinterpret_cast<uint4*>(p.ax + ((int64_t)bh * p.m_tokens + row) * 8) =
            make_uint4(h4[0] | (h4[1] << 16), h4[2] | (h4[3] << 16), l4[0] | (l4[1] << 16), l4[2] | (l4[3] << 16));
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
    if (valid)
      *(reinterpret_cast<uint4*>(p.qr + ((int64_t)bh * p.m_tokens + row) * kD) + l16) =
        make_uint4(pack_f16x2_sat(y[0], y[1]), pack_f16x2_sat(y[2], y[3]), pack_f16x2_sat(y[4], y[5]), pack_f16x2_sat(y[6], y[7]));
  }
}


// PAIR: two CTAs of a cluster work as one (tcgen05 cta_group::2).  The pair shares the key and value tiles of one
// (batch, head): CTA r owns query rows [256 r, 256 r + 256) of a 512-row unit and dequantizes (or loads) HALF of
// every operand tile - 32 of the 64 keys of each score product's B operand, 64 of the 128 value channels - so the
// dequantization work, the stores and the B-operand reads per SM halve.  The leader CTA (rank 0) issues every
// MMA, with M = 256: 128 rows in each CTA's own TMEM.  Barriers the issuer waits on live in the leader and take
// arrivals from both CTAs; barriers the issuer signals are committed to both CTAs at once.  No load is multicast:
// each CTA fetches its own half.  The halves of the operand stages a CTA of a pair does not use hold a two-stage
// ring for the PACKED tiles: the TMA thread brings the codes and metadata of the next cached tile in with bulk
// copies, and the dequant warps expand them from shared memory (the one-CTA kernel has no room for that and
// reads them from global memory into registers a tile ahead).
template <int BITS, int GROUP, bool PAIR>
__global__ void __launch_bounds__(kThreads, 1)
attn_tcgen05_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_qr,
                    const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v, const TParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t sbase = smem_u32(smem);
  volatile int* misc = reinterpret_cast<volatile int*>(smem + kOffMisc);   // [0] tmem base, [1] abort flag
  Ctx cx{sbase + kOffBar, misc + 1, p.wait_budget};

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  KVQ_TRACE_DECL;
  const uint32_t rank = PAIR ? cluster_ctarank() : 0u;            // 0: the CTA that issues the MMAs
  const int sched_id = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;   // which range of the schedule (one per pair)
  const int n_sched = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;
  constexpr int kC = PAIR ? 2 : 1;                                // CTAs that arrive on the issuer's barriers
  // barrier i of the issuing CTA, as an address an arrival (or a TMA completion) from either CTA can use
  auto lead = [&](int i) -> uint32_t { return PAIR ? map_to_cta(cx.bar(i), 0) : cx.bar(i); };
  auto arrive_lead = [&](int i) { if constexpr (PAIR) mbar_arrive_cluster(lead(i)); else mbar_arrive(cx.bar(i)); };
  auto expect_tx_lead = [&](int i, uint32_t bytes) {
    if constexpr (PAIR) mbar_arrive_expect_tx_cluster(lead(i), bytes); else mbar_arrive_expect_tx(cx.bar(i), bytes);
  };
  // first query row of this CTA in schedule unit `unit` (a unit is 256 rows, 512 for a pair)
  auto unit_row0 = [&](int unit, int bh) { return (unit - bh * p.q_blocks) * (2 * kC * kBlockM) + (int)rank * 2 * kBlockM; };
  const int n_rt = (p.n_cur + kBlockN - 1) / kBlockN;
  const int n_ct = (p.n_cached + kBlockN - 1) / kBlockN;
  const int T = n_rt + n_ct;
  constexpr int G = kD / GROUP;

  if (tid == 0) {
    misc[1] = 0;
    mbar_init(cx.bar(kQFull), kC);
    for (int s = 0; s < 2; ++s) {
      mbar_init(cx.bar(kKFull + s), 129 * kC);   // 128 dequant threads + the TMA thread (of each CTA), every tile
      mbar_init(cx.bar(kVFull + s), 129 * kC);
      mbar_init(cx.bar(kKEmpty + s), 2);    // both MMA issuers commit
      mbar_init(cx.bar(kVEmpty + s), 2);
      mbar_init(cx.bar(kSFull + s), 1);
      mbar_init(cx.bar(kSFull + 2 + s), 1);
      mbar_init(cx.bar(kPFull + s), 128 * kC);   // the four softmax warps of a query tile (of each CTA)
      mbar_init(cx.bar(kPFull + 2 + s), 128 * kC);
      mbar_init(cx.bar(kODone + s), 1);
      mbar_init(cx.bar(kODone + 2 + s), 1);
    }
    mbar_init(cx.bar(kQCurDone), 2);
    mbar_init(cx.bar(kQRotFull), 129 * kC);   // 128 dequant threads (bias rows) + the TMA thread (rotated query tile)
    mbar_init(cx.bar(kDrain + 0), 1);
    mbar_init(cx.bar(kDrain + 1), 1);
    mbar_init(cx.bar(kQEmpty), 2);
    for (int s = 0; s < 2; ++s) {
      mbar_init(cx.bar(kRawFull + s), 1);     // the TMA thread's expect-tx; the copies complete the bytes
      mbar_init(cx.bar(kRawEmpty + s), 128);  // the dequant threads have the stage's contents in registers
    }
    mbar_init(cx.bar(kOFree + 0), 128 * kC);
    mbar_init(cx.bar(kOFree + 1), 128 * kC);
    fence_barrier_init();
    prefetch_tensormap(&tm_q); prefetch_tensormap(&tm_qr); prefetch_tensormap(&tm_k); prefetch_tensormap(&tm_v);
  }
  // bias operand tiles start as zeros (columns beyond the group count stay zero for good)
  for (int i = tid; i < 4 * kXBytes / 16; i += kThreads)
    reinterpret_cast<uint4*>(smem + kOffAx)[i] = make_uint4(0, 0, 0, 0);
  if (warp == 0) {
    if constexpr (PAIR) { tmem_alloc_pair(sbase + kOffMisc, 512); tmem_relinquish_pair(); }
    else { tmem_alloc(sbase + kOffMisc, 512); tmem_relinquish(); }
  }
  fence_proxy_async_smem();
  tc_fence_before();
  __syncthreads();
  if constexpr (PAIR) cluster_sync_all();        // the peer's barriers exist before anything arrives on them
  tc_fence_after();
  const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(smem + kOffMisc);
  // TMEM columns: S0 [0,128) S1 [128,256) O0 [256,384) O1 [384,512); P_q aliases the first 64 columns of S_q.

  if (warp < 4) {
    setmaxnreg_dec<kRegsIssue>();
  if (warp == 0) {
    // ================= TMA producer =================
    if (lane == 0) {
      auto load_q = [&](uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2, int c3) {
        if constexpr (PAIR) tma_load_4d_pair(dst, map, bar, c0, c1, c2, c3);
        else tma_load_4d(dst, map, bar, c0, c1, c2, c3);
      };
      // Pair kernel: the packed codes and metadata of cached tile ct of (batch, head) bh into the next stage of
      // the staging ring.  A tile is 128 consecutive slots of the head's slab, taken modulo the capacity: one run,
      // or two where the window wraps.  Slot numbers are multiples of 16 (cache_begin is, the capacity is a
      // multiple of 128), so every source address and size below is a multiple of 16 bytes.
      int n_raw = 0;
      auto stage_packed = [&](int ct, int bh) -> bool {
        constexpr int kCB = kD * BITS / 8;
        const int rs = n_raw & 1;
        if (!cx.wait(kRawEmpty + rs, ((n_raw >> 1) & 1) ^ 1, 104)) return false;
        const uint32_t bar = cx.bar(kRawFull + rs);
        mbar_arrive_expect_tx(bar, 128u * (2 * kCB + 6 * G));
        const uint32_t codes = sbase + kOffV + rs * kTileBytes + kRawCodesOff;
        const uint32_t meta = sbase + kOffK + rs * kTileBytes + kRawMetaOff;
        int64_t slot = p.cache_begin + (int64_t)ct * kBlockN;
        if (slot >= p.capacity) slot -= p.capacity;
        const int n1 = (int)min((int64_t)kBlockN, p.capacity - slot);
        for (int part = 0; part < 2; ++part) {
          const int n = part == 0 ? n1 : kBlockN - n1, at = part == 0 ? 0 : n1;
          if (n == 0) break;
          const int64_t tok = (int64_t)bh * p.capacity + (part == 0 ? slot : 0);
          bulk_load(codes + at * kCB, p.k_codes + tok * kCB, n * kCB, bar);
          bulk_load(codes + kRawVCodes + at * kCB, p.v_codes + tok * kCB, n * kCB, bar);
          bulk_load(meta + at * G, p.k_scale + tok * G, n * G, bar);
          bulk_load(meta + kRawKZero + at * 2 * G, p.k_zero + tok * G, n * 2 * G, bar);
          bulk_load(meta + kRawVScale + at * G, p.v_scale + tok * G, n * G, bar);
          bulk_load(meta + kRawVZero + at * 2 * G, p.v_zero + tok * G, n * 2 * G, bar);
        }
        ++n_raw;
        return true;
      };
      Schedule sch(sched_id, n_sched, p);
      Segment sg;
      int it = 0, nseg = 0, issued_it = -1, rot_seg = -1;
      bool ok = true;
      while (ok && sch.next(sg)) {
        const int bh = sg.unit / p.q_blocks, b = bh / p.heads, h = bh - b * p.heads;
        const int row0 = unit_row0(sg.unit, bh);
        const int t_first_cached = max(sg.tb, n_rt);
        if constexpr (PAIR) {       // the segment's first cached tile; every later one is staged a tile ahead
          if (t_first_cached < sg.te && !(ok = stage_packed(t_first_cached - n_rt, bh))) break;
        }
        // the query buffer is free once every score MMA of the previous segment has retired (the MMA warp says so
        // in its last iteration, before the last P V products)
        if (!(ok = cx.wait(kQEmpty, (nseg & 1) ^ 1, 100))) break;
        // a segment that starts in the cache never needs the unrotated query: load the rotated one right away
        const bool cached0 = sg.tb >= n_rt;
        expect_tx_lead(kQFull, 2 * kTileBytes);
        for (int qt = 0; qt < 2; ++qt)
          for (int kb = 0; kb < 2; ++kb)
            load_q(sbase + kOffQ + qt * kTileBytes + kb * kHalfTile, cached0 ? &tm_qr : &tm_q, lead(kQFull), kb * 64, row0 + qt * kBlockM, h, b);
        if (cached0 || sg.te <= n_rt) arrive_lead(kQRotFull);   // this thread's share of the phase
        for (int t = sg.tb; t < sg.te; ++t, ++it) {
          const int s = it & 1;
          const uint32_t ph = (it >> 1) & 1;
          if (t == n_rt && !cached0) {
            // first cached tile: once no MMA reads the unrotated query any more, the rotated tile replaces it
            if (!(ok = cx.wait(kQCurDone, nseg & 1, 103))) break;
            expect_tx_lead(kQRotFull, 2 * kTileBytes);
            for (int qt = 0; qt < 2; ++qt)
              for (int kb = 0; kb < 2; ++kb)
                load_q(sbase + kOffQ + qt * kTileBytes + kb * kHalfTile, &tm_qr, lead(kQRotFull), kb * 64, row0 + qt * kBlockM, h, b);
            rot_seg = nseg;
          }
          if (!(ok = cx.wait(kKEmpty + s, ph ^ 1, 101))) break;
          if (t < n_rt) {
            expect_tx_lead(kKFull + s, kTileBytes / kC);
            if constexpr (PAIR) {
              // this CTA's 32 keys of each half of the tile (local rows 32 hf .. 32 hf + 31): boxes of 32 rows
              for (int hf = 0; hf < 2; ++hf)
                for (int kb = 0; kb < 2; ++kb)
                  tma_load_4d_pair(sbase + kOffK + s * kTileBytes + kb * kHalfTile + hf * 32 * 128, &tm_k, lead(kKFull + s), kb * 64,
                              t * kBlockN + 64 * hf + 32 * (int)rank, h, b);
            } else {
              for (int kb = 0; kb < 2; ++kb)
                tma_load_4d(sbase + kOffK + s * kTileBytes + kb * kHalfTile, &tm_k, cx.bar(kKFull + s), kb * 64, t * kBlockN, h, b);
            }
          } else {
            arrive_lead(kKFull + s);
          }
          if (!(ok = cx.wait(kVEmpty + s, ph ^ 1, 102))) break;
          if (t < n_rt) {
            expect_tx_lead(kVFull + s, kTileBytes / kC);
            if constexpr (PAIR) {   // this CTA's 64 value channels of all 128 keys: one 64-column block
              tma_load_4d_pair(sbase + kOffV + s * kTileBytes, &tm_v, lead(kVFull + s), 64 * (int)rank, t * kBlockN, h, b);
            } else {
              for (int kb = 0; kb < 2; ++kb)
                tma_load_4d(sbase + kOffV + s * kTileBytes + kb * kHalfTile, &tm_v, cx.bar(kVFull + s), kb * 64, t * kBlockN, h, b);
            }
            issued_it = it;
          } else {
            arrive_lead(kVFull + s);
          }
          if constexpr (PAIR) {
            if (t + 1 < sg.te && t + 1 > t_first_cached && !(ok = stage_packed(t + 1 - n_rt, bh))) break;
          }
        }
        ++nseg;
      }
      // drain: give loads already in flight a bounded time to land before the CTA exits (of a pair, the barriers
      // are the leader's and count both CTAs' bytes; the peer stays until the leader has come through, below)
      if (*cx.abort && n_raw > 0) cx.drain(kRawFull + ((n_raw - 1) & 1), ((n_raw - 1) >> 1) & 1);   // this CTA's own copies
      if (*cx.abort && rank == 0) {
        if (nseg > 0) cx.drain(kQFull, (nseg - 1) & 1);
        if (rot_seg >= 0) cx.drain(kQRotFull, rot_seg & 1);
        if (issued_it >= 0) {
          cx.drain(kKFull + (issued_it & 1), (issued_it >> 1) & 1);
          cx.drain(kVFull + (issued_it & 1), (issued_it >> 1) & 1);
        }
      }
    }
  } else if (warp <= 2) {
    // ================= MMA issuers =================
    // Warp 1 issues for query tile 0, warp 2 for query tile 1.  Each runs this code converged; one lane, elected
    // once, issues every tcgen05.mma and commit of its query tile.
    //
    // A key tile is worked on in two halves of 64 keys, each with its own 64 score columns in TMEM, so that the
    // scores of the next tile's half can be computed while the softmax warps are still busy with the other half
    // of this tile: per (half, query tile) the issuer waits for that half of P, issues O += P V over its 64 keys
    // and then at once S = Q K^T of the same half of the NEXT tile into the columns P has just left.  The tensor
    // pipe executes this thread's MMAs in order, so the new scores cannot overtake the product that reads P.
    // Of a pair only the leader CTA issues (M = 256: its own 128 rows and the peer's); the peer's two warps idle.
    if (rank == 0) {
      const bool leader = elect_one();
      const int qt = warp - 1;
      constexpr int kM = PAIR ? 256 : 128;
      const uint32_t idesc_bf16 = make_idesc_bf16(kM, 64, 0, 0);
      const uint32_t idesc_f16 = idesc_bf16 & ~((7u << 7) | (7u << 10));     // A, B format 0 = FP16
      const uint32_t idesc_pv = make_idesc_bf16(kM, 128, 0, 1);               // B (values) is MN-major
      // commit: one arrival when every MMA issued so far has completed; of a pair, on the barrier of both CTAs
      auto commit = [&](int i) { if constexpr (PAIR) tc_commit_pair(cx.bar(i), (uint16_t)3); else tc_commit(cx.bar(i)); };
      // Descriptors are built once; stepping along K only adds a constant to the 14-bit address field
      // (all operand tiles live below 256 KiB of shared memory, so the field cannot overflow).
      const uint64_t dq0 = make_smem_desc(sbase + kOffQ, 16, 1024, kLayoutSw128);
      const uint64_t dk0 = make_smem_desc(sbase + kOffK, 16, 1024, kLayoutSw128);
      const uint64_t dv0 = make_smem_desc(sbase + kOffV, kHalfTile, 1024, kLayoutSw128);
      const uint64_t dax0 = make_smem_desc(sbase + kOffAx, 128, 256, kLayoutNone);
      const uint64_t dbx0 = make_smem_desc(sbase + kOffBx, 128, 256, kLayoutNone);
      // S[:, 64 hf .. 64 hf + 63] = Q_qt K^T over keys 64 hf .. 64 hf + 63 of stage s (+ the bias step)
      auto issue_qk = [&](int s, int hf, bool cached) {
        if (!leader) return;
        const uint32_t idesc = cached ? idesc_f16 : idesc_bf16;
        const uint64_t qd = dq0 + (uint64_t)(qt * (kTileBytes >> 4));
        // key rows are 128 bytes; a half is 64 rows of the stage, or each CTA's 32 of them for a pair
        const uint64_t kd = dk0 + (uint64_t)(s * (kTileBytes >> 4) + hf * ((64 / kC) * 128 >> 4));
        const uint32_t d_tmem = tmem + qt * 128 + hf * 64;
        constexpr int kBlk = kHalfTile >> 4;
        // rows 64 hf .. (32 hf .. for a pair) of the bias tile: 8-row groups are 256 bytes apart
        const uint64_t axd = dax0 + (uint64_t)(qt * (kXBytes >> 4));
        const uint64_t bxd = dbx0 + (uint64_t)(s * (kXBytes >> 4) + hf * ((8 / kC) * 256 >> 4));
        if constexpr (PAIR) {
          mma_ss_off_pair<0>(d_tmem, qd, kd, idesc, 0);
          mma_ss_off_pair<2>(d_tmem, qd, kd, idesc, 1);
          mma_ss_off_pair<4>(d_tmem, qd, kd, idesc, 1);
          mma_ss_off_pair<6>(d_tmem, qd, kd, idesc, 1);
          mma_ss_off_pair<kBlk>(d_tmem, qd, kd, idesc, 1);
          mma_ss_off_pair<kBlk + 2>(d_tmem, qd, kd, idesc, 1);
          mma_ss_off_pair<kBlk + 4>(d_tmem, qd, kd, idesc, 1);
          mma_ss_off_pair<kBlk + 6>(d_tmem, qd, kd, idesc, 1);
          if (cached && p.correction) mma_ss_pair(d_tmem, axd, bxd, idesc_bf16, 1);
        } else {
          mma_ss_off<0>(d_tmem, qd, kd, idesc, 0);
          mma_ss_off<2>(d_tmem, qd, kd, idesc, 1);
          mma_ss_off<4>(d_tmem, qd, kd, idesc, 1);
          mma_ss_off<6>(d_tmem, qd, kd, idesc, 1);
          mma_ss_off<kBlk>(d_tmem, qd, kd, idesc, 1);
          mma_ss_off<kBlk + 2>(d_tmem, qd, kd, idesc, 1);
          mma_ss_off<kBlk + 4>(d_tmem, qd, kd, idesc, 1);
          mma_ss_off<kBlk + 6>(d_tmem, qd, kd, idesc, 1);
          if (cached && p.correction) mma_ss(d_tmem, axd, bxd, idesc_bf16, 1);
        }
        commit(kSFull + 2 * hf + qt);
      };
      // O_qt += P V over keys 64 hf .. 64 hf + 63 of stage s; P (BF16 pairs) sits in the first 32 of that half's
      // score columns
      auto issue_pv = [&](int s, int hf, bool accumulate) {
        if (!leader) return;
        const uint64_t vd = dv0 + (uint64_t)(s * (kTileBytes >> 4) + hf * (4 * 128));
        const uint32_t d_tmem = tmem + 256 + qt * 128, a_tmem = tmem + qt * 128 + hf * 64;
        if constexpr (PAIR) {
          mma_ts_off_pair<0 * 128>(d_tmem, a_tmem + 0, vd, idesc_pv, accumulate ? 1u : 0u);
          mma_ts_off_pair<1 * 128>(d_tmem, a_tmem + 8, vd, idesc_pv, 1);
          mma_ts_off_pair<2 * 128>(d_tmem, a_tmem + 16, vd, idesc_pv, 1);
          mma_ts_off_pair<3 * 128>(d_tmem, a_tmem + 24, vd, idesc_pv, 1);
        } else {
          mma_ts_off<0 * 128>(d_tmem, a_tmem + 0, vd, idesc_pv, accumulate ? 1u : 0u);
          mma_ts_off<1 * 128>(d_tmem, a_tmem + 8, vd, idesc_pv, 1);
          mma_ts_off<2 * 128>(d_tmem, a_tmem + 16, vd, idesc_pv, 1);
          mma_ts_off<3 * 128>(d_tmem, a_tmem + 24, vd, idesc_pv, 1);
        }
        commit(kODone + 2 * hf + qt);
      };
      Schedule sch(sched_id, n_sched, p);
      Segment sg;
      int it = 0, nseg = 0;
      bool ok = true;
      while (ok && sch.next(sg)) {
        const uint32_t sp = nseg & 1;
        // last current-chunk tile of this segment (-1 if the segment starts in the cache): after its
        // score MMAs nothing reads the unrotated query any more
        const int t_lastcur = (sg.tb < n_rt) ? min(sg.te, n_rt) - 1 : -1;
        const int t_rot = max(sg.tb, n_rt);          // first cached tile: its scores need the rotated query
        if (!(ok = cx.wait(kQFull, sp, 201))) break;
        // Iteration t issues the products of tile t and the scores of tile t + 1 (t = tb - 1: only the scores of
        // the first tile), in the order (half 0, tile 0) (half 0, tile 1) (half 1, tile 0) (half 1, tile 1), each
        // as "P V, then Q K^T".  If tile t + 1 is the first cached one, all four products come first: its scores
        // wait for the rotated query, which itself waits for every earlier score MMA.
        --it;
        for (int t = sg.tb - 1; ok && t < sg.te; ++t, ++it) {
          const int s = it & 1, s1 = (it + 1) & 1;
          const uint32_t ph = (it >> 1) & 1, ph1 = ((it + 1) >> 1) & 1;
          const bool has_pv = t >= sg.tb, has_qk = t + 1 < sg.te, first = t == sg.tb;
          const bool rot = has_qk && t + 1 == t_rot;
          KVQ_STAMP(32);
          if (rot && !has_pv && leader) commit(kQCurDone);      // the segment starts in the cache
          // last iteration: every score MMA of the segment is issued, so the query buffer (and the bias rows) can
          // be handed to the next segment while the last P V products still run
          if (!has_qk && leader) commit(kQEmpty);
          const int n_ops = rot ? 4 : 2;
#pragma unroll 1
          for (int op = 0; op < n_ops; ++op) {
            const int hf = op & 1;
            if (has_pv && op < 2) {
              if (op == 0 && !(ok = cx.wait(kVFull + s, ph, 203))) break;
              if (!(ok = cx.wait(kPFull + 2 * hf + qt, it & 1, 204))) break;
              // first product of a segment: the previous segment's O must have been read out
              if (first && hf == 0 && !(ok = cx.wait(kOFree + qt, sp ^ 1, 209))) break;
              KVQ_STAMP(34);
              tc_fence_after();
              issue_pv(s, hf, !(first && hf == 0));
              if (op == 1 && leader) commit(kVEmpty + s);
              KVQ_STAMP(10 + qt);
            }
            if (has_qk && (!rot || op >= 2)) {
              if (hf == 0) {
                if (rot && !(ok = cx.wait(kQRotFull, sp, 207))) break;
                if (!(ok = cx.wait(kKFull + s1, ph1, 205))) break;
                tc_fence_after();
              }
              KVQ_STAMP(36);
              issue_qk(s1, hf, t + 1 >= n_rt);
              if (hf == 1 && leader) {
                commit(kKEmpty + s1);
                if (t + 1 == t_lastcur) commit(kQCurDone);
              }
              KVQ_STAMP(14 + qt);
            }
          }
        }
        if (!ok) break;
        ++nseg;
      }
      // everything issued so far must have retired before TMEM is freed
      if (leader) commit(kDrain + qt);
      cx.drain(kDrain + qt, 0);
    }
  }
  } else if (warp < 12) {
    // ================= softmax groups =================
    // Warps 4-7 own query tile 0, warps 8-11 query tile 1; warp w reads TMEM lanes 32 (w % 4) .. + 31, one query
    // row per lane, so the row maximum and the row sums need no exchange between threads.  A key tile is taken
    // in two halves of 64 keys, each one step of the online softmax: 64 scores into registers, maximum,
    // exponentials, 32 columns of BF16 pairs back over the scores.  While a group works on one half the tensor
    // pipe computes the other half's next scores, so a group seldom waits.
    setmaxnreg_inc<kRegsSoftmax>();
    const int qt = (warp - 4) >> 2;                           // which query tile
    const int wq = warp & 3;                                  // which 32 rows (TMEM lane quarter)
    const int r256 = qt * kBlockM + wq * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(wq * 32) << 16;
    const uint32_t s_addr = tmem + lane_addr + qt * 128;      // scores of half hf at columns 64 hf; P over their first 32
    const uint32_t o_addr = tmem + lane_addr + 256 + qt * 128;
    const float c_row = p.scale_log2;
    Schedule sch(sched_id, n_sched, p);
    Segment sg;
    int it = 0, nseg = 0;
    bool ok = true;
    while (ok && sch.next(sg)) {
      float m_run = -INFINITY, lcur = 0.f, lcac = 0.f;   // running max (log2 units), row sums over current / cached keys
      bool fresh = true;                                 // no product has been added to O in this segment yet
      for (int t = sg.tb; ok && t < sg.te; ++t, ++it) {
        const bool cached = t >= n_rt;
        const int n_valid = cached ? min(kBlockN, p.n_cached - (t - n_rt) * kBlockN) : min(kBlockN, p.n_cur - t * kBlockN);
#pragma unroll 1
        for (int hf = 0; hf < 2; ++hf) {
          uint32_t sr[64];                         // this thread's 64 scores, then its 32 packed probabilities
          KVQ_STAMP(0);
          ok = __all_sync(0xFFFFFFFFu, cx.wait(kSFull + 2 * hf + qt, it & 1, 301));
          if (!ok) break;
          KVQ_STAMP(1);
          tc_fence_after();
          tmem_ld32(s_addr + 64 * hf, sr);
          tmem_ld32(s_addr + 64 * hf + 32, sr + 32);
          tmem_wait_ld();
          KVQ_STAMP(2);
          const int nv = n_valid - 64 * hf;
          if (nv < 64) {                           // ragged last tile of the current chunk or of the cache
#pragma unroll
            for (int i = 0; i < 64; ++i)
              if (i >= nv) sr[i] = 0xFF800000u;    // -inf
          }
          float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
          for (int i = 0; i < 64; i += 8) {
#pragma unroll
            for (int c = 0; c < 4; ++c) mx[c] = max3(mx[c], __uint_as_float(sr[i + 2 * c]), __uint_as_float(sr[i + 2 * c + 1]));
          }
          const float m_new = fmaxf(m_run, fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * c_row);
          if (__any_sync(0xFFFFFFFFu, m_new - m_run > kRescaleThreshold)) {
            if (!fresh) {
              // the product of the previous half (the last one issued on this O) must have retired
              ok = __all_sync(0xFFFFFFFFu, cx.wait(kODone + 2 * (hf ^ 1) + qt, (it - (hf ^ 1)) & 1, 302));
              if (!ok) break;
              tc_fence_after();
              const float f = ex2(m_run - m_new);
#pragma unroll 1
              for (int c = 0; c < 8; ++c) {
                uint32_t r[16];
                tmem_ld16(o_addr + 16 * c, r);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 16; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * f);
                tmem_st16(o_addr + 16 * c, r);
              }
              lcur *= f; lcac *= f;
            }
            m_run = m_new;
          }
          const float2 c2 = make_float2(c_row, c_row), nm2 = make_float2(-m_run, -m_run);
          float2 sum2 = make_float2(0.f, 0.f);
          KVQ_STAMP(3);
#pragma unroll
          for (int i = 0; i < 64; i += 2) {
            const float2 x = __ffma2_rn(make_float2(__uint_as_float(sr[i]), __uint_as_float(sr[i + 1])), c2, nm2);
            const float2 pr = ((i >> 1) & 3) < (PAIR ? kPolyPairs : 0) ? ex2_poly2(x) : make_float2(ex2(x.x), ex2(x.y));
            sum2 = __fadd2_rn(sum2, pr);
            sr[i >> 1] = cvt_bf16x2(pr.x, pr.y);
          }
          tmem_st32(s_addr + 64 * hf, sr);
          if (cached) lcac += sum2.x + sum2.y; else lcur += sum2.x + sum2.y;
          tmem_wait_st();
          tc_fence_before();
          arrive_lead(kPFull + 2 * hf + qt);
          KVQ_STAMP(4 + hf);
          fresh = false;
        }
      }
      if (!ok) break;
      // ---- segment epilogue: read this row of O out of TMEM, release it, write the normalised row ----
      const int bh = sg.unit / p.q_blocks, b = bh / p.heads, h = bh - b * p.heads;
      const bool whole = sg.tb == 0 && sg.te == T;
      uint8_t* slot = p.partial + (size_t)(2 * blockIdx.x + sg.slot) * kSlotBytes;   // partial segments only
      ok = __all_sync(0xFFFFFFFFu, cx.wait(kODone + 2 + qt, (it - 1) & 1, 303));            // the last product of the segment is a second half
      if (!ok) break;
      tc_fence_after();
      const int row = unit_row0(sg.unit, bh) + r256;
      // a whole unit writes its rows of the output; a partial segment writes the same normalised rows into its
      // slot, with the statistics the merge kernel weighs them by
      const float l = lcur + lcac;
      const float inv = 1.0f / l;
      const bool store = !whole || row < p.m_tokens;
      // consecutive 8-column pieces: 16 bytes apart in a row of the output, 4096 bytes apart in a slot
      uint8_t* dst = whole ? reinterpret_cast<uint8_t*>(p.out + (int64_t)b * p.o_sb + (int64_t)h * p.o_sh + (int64_t)row * p.o_st)
                           : slot + r256 * 16;
      const int piece = whole ? 16 : 4096;
#pragma unroll 1
      for (int hf = 0; hf < 2; ++hf) {               // 64 columns at a time
        uint32_t sr[64];
        tmem_ld32(o_addr + 64 * hf, sr);
        tmem_ld32(o_addr + 64 * hf + 32, sr + 32);
        tmem_wait_ld();
        if (hf == 1) {                               // the whole row is in registers: O can be overwritten
          tc_fence_before();
          arrive_lead(kOFree + qt);
        }
        if (store) {
#pragma unroll
          for (int i = 0; i < 64; i += 8) {
            uint4 v;
            v.x = cvt_bf16x2(__uint_as_float(sr[i]) * inv, __uint_as_float(sr[i + 1]) * inv);
            v.y = cvt_bf16x2(__uint_as_float(sr[i + 2]) * inv, __uint_as_float(sr[i + 3]) * inv);
            v.z = cvt_bf16x2(__uint_as_float(sr[i + 4]) * inv, __uint_as_float(sr[i + 5]) * inv);
            v.w = cvt_bf16x2(__uint_as_float(sr[i + 6]) * inv, __uint_as_float(sr[i + 7]) * inv);
            *reinterpret_cast<uint4*>(dst + (8 * hf + (i >> 3)) * piece) = v;
          }
        }
      }
      if (store) {
        if (whole) {
          const int64_t idx = (int64_t)bh * p.m_tokens + row;
          if (p.lse) p.lse[idx] = (m_run + log2f(l)) * 0.6931471805599453f;
          if (p.cached_mass) p.cached_mass[idx] = lcac * inv;
        } else {
          float* st = reinterpret_cast<float*>(slot + kSlotStats);
          st[r256] = m_run; st[256 + r256] = lcur; st[512 + r256] = lcac;
        }
      }
      ++nseg;
    }
    tc_fence_before();
  } else {
    // ================= dequant warps =================
    setmaxnreg_dec<kRegsDequant>();
    const int dt = tid - 12 * 32;          // 0..127: the key of the tile this thread expands
    // One CTA: thread dt expands key dt of the tile, keys and values.  A CTA of a pair expands half of each
    // tile: of the keys, its 32 keys of either half tile (local row dt / 2 = 32 hf + j is key 64 hf + 32 rank + j),
    // two threads per key with 64 channels each; of the values, channels [64 rank, 64 rank + 64) of key dt.
    constexpr int kNW = Raw<BITS>::kWords / kC;                    // code words per thread and tile (keys or values)
    const int k_row = PAIR ? (dt >> 1) : dt;                       // row of the key stage this thread writes
    const int k_key = PAIR ? 64 * (k_row >> 5) + 32 * (int)rank + (k_row & 31) : dt;   // its key within the tile
    const int k_word0 = PAIR ? (dt & 1) * kNW : 0;                 // first code word of the key it expands
    const int v_word0 = PAIR ? (int)rank * kNW : 0;                // first code word of value row dt it expands
    const int v_piece0 = PAIR ? (int)rank * 8 : 0;                 // its 16-byte pieces start at piece 0 of the block
    Schedule sch(sched_id, n_sched, p);
    Segment sg;
    int it = 0, nseg = 0;
    int n_raw = 0;                         // cached tiles taken from the staging ring so far (pair kernel)
    bool ok = true;
    Raw<BITS> rk, rv;
    while (ok && sch.next(sg)) {
      const int bh = sg.unit / p.q_blocks;
      // key k of the window lives in slot cache_begin + k, taken modulo the capacity (ring caches wrap; for
      // linear ones the host has checked that the window ends inside the capacity)
      const int64_t slab0 = (int64_t)bh * p.capacity;
      auto tok_of = [&](int k) {
        const int64_t slot = p.cache_begin + k;
        return slab0 + (slot >= p.capacity ? slot - p.capacity : slot);
      };
      const int t_rot = max(sg.tb, n_rt);          // first cached tile of the segment: the query is rotated there
      if (!PAIR && sg.te > n_rt) {                 // one CTA: packed data comes one tile ahead into registers
        const int k0 = (t_rot - n_rt) * kBlockN + k_key, v0 = (t_rot - n_rt) * kBlockN + dt;
        load_raw<BITS, G, kNW>(rk, p.k_codes, p.k_scale, p.k_zero, tok_of(k0), k0 < p.n_cached, k_word0);
        load_raw<BITS, G, kNW>(rv, p.v_codes, p.v_scale, p.v_zero, tok_of(v0), v0 < p.n_cached, v_word0);
      }
      for (int t = sg.tb; t < sg.te; ++t, ++it) {
        const int s = it & 1;
        const uint32_t ph = (it >> 1) & 1;
        const int ct = t - n_rt;
        const int k1 = (ct + 1) * kBlockN + k_key, v1 = (ct + 1) * kBlockN + dt;   // this thread's keys in the next tile
        ok = __all_sync(0xFFFFFFFFu, cx.wait(kKEmpty + s, ph ^ 1, 401));
        if (!ok) break;
        KVQ_STAMP(22);
        // pair: the tile's packed codes and metadata are in the staging ring (the TMA thread keeps it a tile ahead)
        const uint8_t* raw_codes = smem + kOffV + (n_raw & 1) * kTileBytes + kRawCodesOff;
        const uint8_t* raw_meta = smem + kOffK + (n_raw & 1) * kTileBytes + kRawMetaOff;
        if (PAIR && ct >= 0) {
          ok = __all_sync(0xFFFFFFFFu, cx.wait(kRawFull + (n_raw & 1), (n_raw >> 1) & 1, 406));
          if (!ok) break;
          load_raw_staged<BITS, G, kNW>(rk, raw_codes, raw_meta, raw_meta + kRawKZero, k_key,
                                        ct * kBlockN + k_key < p.n_cached, k_word0);
        }
        if (ct >= 0) {
          dequant_keys<BITS, GROUP, kNW>(rk, smem + kOffK + s * kTileBytes, k_row, k_word0);
          if (p.correction && k_word0 == 0) {   // B_extra row: step_j^2, exact in BF16
            const float d0 = raw_step<BITS>(rk, 0), d1 = raw_step<BITS>(rk, 1), d2 = raw_step<BITS>(rk, 2), d3 = raw_step<BITS>(rk, 3);
            const uint32_t b01 = pack_bf16x2(d0 * d0, G > 1 ? d1 * d1 : 0.f), b23 = pack_bf16x2(G > 2 ? d2 * d2 : 0.f, G > 3 ? d3 * d3 : 0.f);
            // columns 0..3 meet the high parts of A_extra, columns 4..7 the low parts
            *reinterpret_cast<uint4*>(smem + kOffBx + s * kXBytes + xtile_offset(k_row, 0)) = make_uint4(b01, b23, b01, b23);
          }
          fence_proxy_async_smem();
          if (!PAIR && t + 1 < sg.te) load_raw<BITS, G, kNW>(rk, p.k_codes, p.k_scale, p.k_zero, tok_of(k1), k1 < p.n_cached, k_word0);
        }
        arrive_lead(kKFull + s);
        KVQ_STAMP(20);
        if (t == t_rot) {
          // ---- A_extra: -(sigma/24) nu rows of this unit's 256 queries, written by the pre-pass ----
          // (the new query tile being in means every MMA of the previous segment, which read the old rows, retired)
          // (of a pair that barrier is the leader's alone; both CTAs see "query buffer free", which the issuer commits
          // once the previous segment's score MMAs, the readers of the old rows, are all issued and retired)
          if constexpr (PAIR) ok = __all_sync(0xFFFFFFFFu, cx.wait(kQEmpty, (nseg & 1) ^ 1, 402));
          else ok = __all_sync(0xFFFFFFFFu, cx.wait(kQFull, nseg & 1, 402));
          if (!ok) break;
          const int row0 = unit_row0(sg.unit, bh);
#pragma unroll
          for (int qt = 0; qt < 2; ++qt) {
            const int row = row0 + qt * kBlockM + dt;
            uint4 a = make_uint4(0, 0, 0, 0);
            if (row < p.m_tokens) a = __ldg(reinterpret_cast<const uint4*>(p.ax_rows + ((int64_t)bh * p.m_tokens + row) * 8));
            *reinterpret_cast<uint4*>(smem + kOffAx + qt * kXBytes + xtile_offset(dt, 0)) = a;
          }
          fence_proxy_async_smem();
          arrive_lead(kQRotFull);
        }
        ok = __all_sync(0xFFFFFFFFu, cx.wait(kVEmpty + s, ph ^ 1, 404));
        if (!ok) break;
        KVQ_STAMP(23);
        if (PAIR && ct >= 0) {
          load_raw_staged<BITS, G, kNW>(rv, raw_codes + kRawVCodes, raw_meta + kRawVScale, raw_meta + kRawVZero, dt,
                                        ct * kBlockN + dt < p.n_cached, v_word0);
          mbar_arrive(cx.bar(kRawEmpty + (n_raw & 1)));      // the stage's contents are in registers
          ++n_raw;
        }
        if (ct >= 0) {
          dequant_values<BITS, GROUP, kNW>(rv, smem + kOffV + s * kTileBytes, dt, v_word0, v_piece0);
          fence_proxy_async_smem();
          if (!PAIR && t + 1 < sg.te) load_raw<BITS, G, kNW>(rv, p.v_codes, p.v_scale, p.v_zero, tok_of(v1), v1 < p.n_cached, v_word0);
        }
        arrive_lead(kVFull + s);
        KVQ_STAMP(21);
      }
      if (!ok) break;
      if (sg.te <= n_rt) arrive_lead(kQRotFull);   // no rotation in this segment: keep the phase count in step
      ++nseg;
    }
  }

  __syncthreads();
  // A pair leaves together: neither CTA's shared memory or TMEM may go while the other still arrives on its
  // barriers or the leader's MMAs still read its operands (every role above has come out through bounded waits).
  if constexpr (PAIR) cluster_sync_all();
  if (warp == 0) {
    tc_fence_after();
    if constexpr (PAIR) tmem_dealloc_pair(tmem, 512); else tmem_dealloc(tmem, 512);
    // a wait that gave up left its diagnostic code in the abort word: report the first one
    if (lane == 0 && misc[1] != 0 && p.status) atomicCAS(p.status, 0, misc[1]);
  }
}

// Combines the partial results of every unit whose key tiles were split over several CTAs.
// grid (n_units - n_whole, 16): a block handles 16 rows x 128 columns; thread = (8-column piece, row).
// pair = 1: the schedule's units are 512 rows worked on by CTA pairs (n_ctas counts pairs); the grid has two blocks
// per unit in x, one for each 256-row half, whose partial results are those of the CTAs of that rank.
__global__ void __launch_bounds__(256) attn_merge_kernel(const TParams p, int n_ctas, int pair) {
  const int su = pair ? blockIdx.x >> 1 : blockIdx.x, rank = pair ? blockIdx.x & 1 : 0, kc = pair ? 2 : 1;
  const int unit = p.n_whole + su;
  const int T = p.tiles;
  // Which CTAs worked on this unit, found once per block (64-bit divisions): CTA c owns the tile steps
  // [W c / n_ctas, W (c + 1) / n_ctas) of the split part.  A CTA's slot 0 belongs to the unit its range starts
  // in, slot 1 to the next one, so only the first CTA of a unit can have used slot 1 for it.
  __shared__ int s_first, s_last, s_first_slot;
  if (threadIdx.x == 0) {
    const long long W = (long long)(p.n_units - p.n_whole) * T;     // tile steps of the split part
    const long long g_lo = (long long)su * T, g_hi = g_lo + T;
    // floor(W c / n) <= g  <=>  W c < (g + 1) n: the exact tests need no division, a double gives the first guess
    auto starts_by = [&](long long c, long long g) { return W * c < (g + 1) * n_ctas; };
    auto owner = [&](long long g) {
      long long c = (long long)((double)g * n_ctas / (double)W);
      c = c < 0 ? 0 : (c > n_ctas - 1 ? n_ctas - 1 : c);
      while (c + 1 < n_ctas && starts_by(c + 1, g)) ++c;
      while (c > 0 && !starts_by(c, g)) --c;
      return (int)c;
    };
    s_first = owner(g_lo);
    s_last = owner(g_hi - 1);
    s_first_slot = W * s_first >= g_lo * n_ctas ? 0 : 1;       // its range starts in this unit
  }
  __syncthreads();
  const int c_first = s_first, c_last = s_last, first_slot = s_first_slot;
  if (c_first == c_last) return;                       // the unit was computed whole by one CTA
  // A thread combines the 8-column piece (cg, row): consecutive lanes take consecutive rows, which are 16 bytes
  // apart in a slot.  The finished pieces change places through shared memory so that the output rows are
  // written 256 contiguous bytes at a time.
  __shared__ uint4 s_tile[16 * 16];
  const int cg = threadIdx.x >> 4, rr = threadIdx.x & 15;
  const int bh = unit / p.q_blocks, b = bh / p.heads, h = bh - b * p.heads;
  const int r256 = blockIdx.y * 16 + rr;
  const int row = (unit - bh * p.q_blocks) * (256 * kc) + rank * 256 + r256;
  if (row - rr >= p.m_tokens) return;                  // the same for the whole block: no rows left in this block
  // Partials are taken four at a time with all of their loads issued before any is used: a thread moves only
  // 16 bytes per partial, so the kernel lives on loads in flight.
  // CTA c of the schedule is CTA kc * c + rank of the grid; every CTA of the grid has two slots
  auto slot_of = [&](int c) { return p.partial + (size_t)(2 * (kc * c + rank) + (c == c_first ? first_slot : 0)) * kSlotBytes; };
  float m = -INFINITY;
  for (int c0 = c_first; c0 <= c_last; c0 += 4) {
    float mm[4];
#pragma unroll
    for (int j = 0; j < 4; ++j)
      mm[j] = (c0 + j <= c_last) ? reinterpret_cast<const float*>(slot_of(c0 + j) + kSlotStats)[r256] : -INFINITY;
    m = fmaxf(fmaxf(m, fmaxf(mm[0], mm[1])), fmaxf(mm[2], mm[3]));
  }
  // out = sum_i w_i O_i / sum_i w_i with w_i = l_i 2^(m_i - m): every partial row is already normalised by its l_i
  float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  float l_cur = 0.f, l_cac = 0.f;
  for (int c0 = c_first; c0 <= c_last; c0 += 4) {
    float sm[4], sc[4], sa[4];
    uint4 a[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const bool have = c0 + j <= c_last;
      const uint8_t* sl = slot_of(have ? c0 + j : c_last);
      const float* st = reinterpret_cast<const float*>(sl + kSlotStats);
      sm[j] = have ? st[r256] : -INFINITY;                  // weight 2^(-inf) = 0 for the slots that are not there
      sc[j] = st[256 + r256]; sa[j] = st[512 + r256];
      a[j] = *reinterpret_cast<const uint4*>(sl + ((size_t)cg * 256 + r256) * 16);
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float f = exp2f(sm[j] - m);
      const float lc = f * sc[j], la = f * sa[j];
      l_cur += lc; l_cac += la;
      const float w = lc + la;
      acc[0] += w * bf16_bits_to_f32(a[j].x & 0xFFFFu); acc[1] += w * bf16_bits_to_f32(a[j].x >> 16);
      acc[2] += w * bf16_bits_to_f32(a[j].y & 0xFFFFu); acc[3] += w * bf16_bits_to_f32(a[j].y >> 16);
      acc[4] += w * bf16_bits_to_f32(a[j].z & 0xFFFFu); acc[5] += w * bf16_bits_to_f32(a[j].z >> 16);
      acc[6] += w * bf16_bits_to_f32(a[j].w & 0xFFFFu); acc[7] += w * bf16_bits_to_f32(a[j].w >> 16);
    }
  }
  const float l = l_cur + l_cac, inv = 1.0f / l;
  uint4 v;
  v.x = cvt_bf16x2(acc[0] * inv, acc[1] * inv); v.y = cvt_bf16x2(acc[2] * inv, acc[3] * inv);
  v.z = cvt_bf16x2(acc[4] * inv, acc[5] * inv); v.w = cvt_bf16x2(acc[6] * inv, acc[7] * inv);
  s_tile[rr * 16 + (cg ^ rr)] = v;
  __syncthreads();
  {
    const int orr = threadIdx.x >> 4, ocg = threadIdx.x & 15;          // output side: a row per 16 lanes
    const int orow = row - rr + orr;
    if (orow < p.m_tokens)
      *reinterpret_cast<uint4*>(p.out + (int64_t)b * p.o_sb + (int64_t)h * p.o_sh + (int64_t)orow * p.o_st + ocg * 8) = s_tile[orr * 16 + (ocg ^ orr)];
  }
  if (cg == 0 && row < p.m_tokens) {
    const int64_t idx = (int64_t)bh * p.m_tokens + row;
    if (p.lse) p.lse[idx] = (m + log2f(l)) * 0.6931471805599453f;
    if (p.cached_mass) p.cached_mass[idx] = l_cac * inv;
  }
}

// ---- host side -----------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

int get_encode_fn(EncodeTiledFn* fn) {
  static std::atomic<EncodeTiledFn> cached{nullptr};     // a driver entry point: the same for every device
  EncodeTiledFn f = cached.load(std::memory_order_acquire);
  if (!f) {
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult qres;
    KVQ_CUDA_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres));
    if (qres != cudaDriverEntryPointSuccess || !sym) return record_cuda_error(cudaErrorSymbolNotFound);
    f = reinterpret_cast<EncodeTiledFn>(sym);
    cached.store(f, std::memory_order_release);
  }
  *fn = f;
  return KVQ_OK;
}

// Byte strides of a [batch, heads, tokens, 128] BF16 tensor as a tensor map wants them: non-zero multiples of 16
// below 2^40.  A size-1 dimension may come with any stride and gets a harmless valid one.  False if a real
// dimension's stride cannot be encoded (0, as in a tensor expanded over heads, or too large).
bool map_strides(kvq_strides s, int64_t tokens, int heads, int batch, cuuint64_t out[3]) {
  const cuuint64_t st = tokens > 1 ? (cuuint64_t)s.t * 2 : (cuuint64_t)kD * 2;
  const cuuint64_t sh = heads > 1 ? (cuuint64_t)s.h * 2 : st * (cuuint64_t)tokens;
  const cuuint64_t sb = batch > 1 ? (cuuint64_t)s.b * 2 : sh * (cuuint64_t)heads;
  out[0] = st; out[1] = sh; out[2] = sb;
  if (s.t < 0 || s.h < 0 || s.b < 0) return false;
  for (int i = 0; i < 3; ++i)
    if (out[i] == 0 || out[i] % 16 != 0 || out[i] >= (1ull << 40)) return false;
  return true;
}

// [batch, heads, tokens, 128] BF16 tensor -> 4-D map with a 64-column x 128-row box, 128-byte swizzle.
int make_map(EncodeTiledFn enc, CUtensorMap* map, const void* ptr, kvq_strides s, int64_t tokens, int heads, int batch,
             int box_rows = kBlockN) {
  cuuint64_t dims[4] = {(cuuint64_t)kD, (cuuint64_t)tokens, (cuuint64_t)heads, (cuuint64_t)batch};
  cuuint64_t strides[3];
  if (!map_strides(s, tokens, heads, batch, strides)) return KVQ_ERR_UNSUPPORTED;
  cuuint32_t box[4] = {64, (cuuint32_t)box_rows, 1, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(ptr), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return record_cuda_error(cudaErrorInvalidValue);
  return KVQ_OK;
}

// SM count of the current device; 148 (a B200) if the device cannot be asked: only sizes and launch counts
// reported before a launch depend on it, and the launch itself fails loudly on such a device.
int num_sms() {
  int n = 0;
  return device_sm_count(&n) == KVQ_OK ? n : 148;
}

// Grid policy: how many CTAs, and how many leading units are computed whole (the rest are split).
//  * At least as many units as SMs: one persistent CTA per SM.  Whole units are dealt out in rounds of
//    one per CTA; the last, incomplete round of R units would leave sms - R SMs idle for a whole unit's
//    time, so its key-tile steps are split evenly over all CTAs instead, when that is worth its cost (below).
//  * Fewer units than SMs: one CTA per unit leaves sms - n_units SMs idle for `tiles` tile steps each.
//    Cutting all tile steps into equal ranges, one per SM, uses them, at a measured cost of about ten
//    tile steps per CTA (a second prologue and epilogue, FP32 partial results, the merge kernel): split
//    when the idle time is worth more than that.
// CTA pairs that can be resident at once on the current device: a cluster of two needs two free SMs of one GPC,
// so a device whose GPCs hold odd numbers of usable SMs fits fewer pairs than SMs / 2, and a persistent grid
// larger than that would run its last clusters after all the others.  Asked once per device; SMs / 2 if the
// device cannot be asked (the launch then fails loudly by itself).
int max_resident_pairs() {
  static std::atomic<int> cache[kMaxDevices] = {};
  int dev = 0;
  if (current_device(&dev) != KVQ_OK) return num_sms() / 2;
  int n = cache[dev].load(std::memory_order_relaxed);
  if (n == 0) {
    auto kern = attn_tcgen05_kernel<2, 128, true>;     // every instantiation has the same footprint
    n = num_sms() / 2;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * (unsigned)n); cfg.blockDim = dim3(kThreads); cfg.dynamicSmemBytes = kSmemBytes;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    int clusters = 0;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) == cudaSuccess &&
        cudaOccupancyMaxActiveClusters(&clusters, kern, &cfg) == cudaSuccess && clusters > 0 && clusters < n)
      n = clusters;
    (void)cudaGetLastError();
    cache[dev].store(n, std::memory_order_relaxed);
  }
  return n;
}

struct Plan { int ctas; int n_whole; };
Plan plan_grid(int64_t n_units, int64_t tiles, bool pair = false) {
  const int sms = pair ? max_resident_pairs() : num_sms();      // CTAs, or CTA pairs, that run at once
  if (n_units >= sms) {
    const int64_t r = n_units % sms;
    return {sms, (int)((r == 0 || tiles * (sms - r) <= 10 * (int64_t)sms) ? n_units : n_units - r)};
  }
  if (tiles * (sms - n_units) <= 10 * (int64_t)sms) return {(int)n_units, (int)n_units};
  const int64_t W = n_units * tiles;
  int64_t c = W / 4;
  if (c < n_units) c = n_units;
  if (c > sms) c = sms;
  if (c > W) c = W;
  return {(int)(c < 1 ? 1 : c), 0};
}

template <int BITS, int GROUP, bool PAIR>
int launch(const CUtensorMap& mq, const CUtensorMap& mqr, const CUtensorMap& mk, const CUtensorMap& mv, const TParams& p,
           const RotParams& rp, dim3 grid, cudaStream_t st) {
  static PerDevice configured;                       // the attribute is per device
  int dev = 0;
  { const int r = current_device(&dev); if (r != KVQ_OK) return r; }
  if (configured.first(dev)) {
    KVQ_CUDA_TRY(cudaFuncSetAttribute(attn_tcgen05_kernel<BITS, GROUP, PAIR>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
    configured.done(dev);
  }
  if (rp.qr) {                      // there are cached keys: rotate the query chunk first
    rotate_query_kernel<BITS, GROUP><<<dim3((unsigned)((rp.m_tokens + 15) / 16), (unsigned)(p.n_units / p.q_blocks)), 256, 0, st>>>(rp);
    KVQ_CUDA_TRY(cudaGetLastError());
  }
  if constexpr (PAIR) {             // grid.x counts pairs: two CTAs each, launched as clusters of two
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * grid.x); cfg.blockDim = dim3(kThreads); cfg.dynamicSmemBytes = kSmemBytes; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    KVQ_CUDA_TRY(cudaLaunchKernelEx(&cfg, attn_tcgen05_kernel<BITS, GROUP, true>, mq, mqr, mk, mv, p));
  } else {
    attn_tcgen05_kernel<BITS, GROUP, false><<<grid, kThreads, kSmemBytes, st>>>(mq, mqr, mk, mv, p);
  }
  KVQ_CUDA_TRY(cudaGetLastError());
  if (p.n_whole != p.n_units) {   // units were split over CTAs: combine their partial results
    attn_merge_kernel<<<dim3((unsigned)((p.n_units - p.n_whole) * (PAIR ? 2 : 1)), 16), 256, 0, st>>>(p, (int)grid.x, PAIR ? 1 : 0);
    KVQ_CUDA_TRY(cudaGetLastError());
  }
  return KVQ_OK;
}

}  // namespace

bool attn_tcgen05_supports(const kvq_cache_desc* d, int64_t m_tokens, int64_t n_cur) {
  return d->head_dim == kD && m_tokens >= 1 && n_cur >= 1;
}

bool attn_tcgen05_addressable(const AttnArgs& a) {
  cuuint64_t st[3];
  return map_strides(a.qs, a.m_tokens, a.desc->heads, a.desc->batch, st) &&
         map_strides(a.kvs, a.n_cur, a.desc->heads, a.desc->batch, st) &&
         map_strides(a.vs, a.n_cur, a.desc->heads, a.desc->batch, st);
}

static void schedule_shape(const kvq_cache_desc* d, int64_t cache_len, int64_t m_tokens, int64_t n_cur,
                           int64_t* q_blocks, int64_t* n_units, int64_t* tiles, bool pair = false) {
  const int64_t rows = (pair ? 4 : 2) * kBlockM;           // query rows of a unit: two tiles per CTA
  *q_blocks = (m_tokens + rows - 1) / rows;
  *n_units = (int64_t)d->batch * d->heads * *q_blocks;
  *tiles = (n_cur + kBlockN - 1) / kBlockN + (cache_len + kBlockN - 1) / kBlockN;
}

// Bytes of the rotated-query area of the workspace: q~ rows (256 bytes each), then bias rows (16 bytes each),
// rounded up to a multiple of 256.  Nothing when there are no cached keys.
static size_t rot_area_bytes(const kvq_cache_desc* d, int64_t cache_len, int64_t m_tokens) {
  if (cache_len <= 0) return 0;
  const size_t rows = (size_t)d->batch * d->heads * (size_t)m_tokens;
  return (rows * (2 * kD + 16) + 255) / 256 * 256;
}

size_t attn_tcgen05_workspace_bytes(const kvq_cache_desc* d, int64_t cache_len, int64_t m_tokens, int64_t n_cur, bool pair) {
  if (m_tokens <= 0) return 0;
  int64_t qb, nu, tiles;
  schedule_shape(d, cache_len, m_tokens, n_cur, &qb, &nu, &tiles, pair);
  const Plan pl = plan_grid(nu, tiles, pair);
  const size_t slots = pl.n_whole != nu ? (size_t)pl.ctas * (pair ? 2 : 1) * 2 * kSlotBytes : 0;
  return rot_area_bytes(d, cache_len, m_tokens) + slots;
}

int attn_tcgen05_kernel_launches(const kvq_cache_desc* d, int64_t cache_len, int64_t m_tokens, int64_t n_cur, bool pair) {
  if (m_tokens <= 0) return 0;
  int64_t qb, nu, tiles;
  schedule_shape(d, cache_len, m_tokens, n_cur, &qb, &nu, &tiles, pair);
  const Plan pl = plan_grid(nu, tiles, pair);
  return 1 + (cache_len > 0 ? 1 : 0) + (pl.n_whole != nu ? 1 : 0);   // attention, query pre-pass, merge
}

static std::atomic<uint32_t> g_wait_budget{0};           // 0: the default, kTimeoutCycles
void set_attn_wait_budget(uint32_t cycles) { g_wait_budget.store(cycles, std::memory_order_relaxed); }

// Common tail of both entry points.  `rot_area` (rot_area_bytes() bytes, 256-byte aligned; null only when
// there are no cached keys) receives the rotated queries; `slots` holds the partial results of split units.
static int launch_planned(const AttnArgs& a, const Plan& pl, int64_t qb, int64_t nu, int64_t tiles, uint8_t* rot_area, uint8_t* slots,
                          bool pair = false) {
  const kvq_cache_desc* d = a.desc;
  EncodeTiledFn enc;
  int r = get_encode_fn(&enc);
  if (r != KVQ_OK) return r;
  CUtensorMap mq, mqr, mk, mv;
  if ((r = make_map(enc, &mq, a.q, a.qs, a.m_tokens, d->heads, d->batch)) != KVQ_OK) return r;
  // a CTA of a pair loads its 32 keys of each half tile: boxes of 32 rows
  if ((r = make_map(enc, &mk, a.k_cur, a.kvs, a.n_cur, d->heads, d->batch, pair ? 32 : kBlockN)) != KVQ_OK) return r;
  if ((r = make_map(enc, &mv, a.v_cur, a.vs, a.n_cur, d->heads, d->batch)) != KVQ_OK) return r;
  if ((int64_t)d->batch * d->heads > 65535) return KVQ_ERR_UNSUPPORTED;   // second grid dimension of the pre-pass
  RotParams rp{};
  mqr = mq;                                                  // never read when there are no cached keys
  if (rot_area) {
    const int64_t rows = (int64_t)d->batch * d->heads * a.m_tokens;
    rp.q = static_cast<const uint16_t*>(a.q); rp.q_sb = a.qs.b; rp.q_sh = a.qs.h; rp.q_st = a.qs.t;
    rp.qr = reinterpret_cast<uint16_t*>(rot_area);
    rp.ax = reinterpret_cast<uint16_t*>(rot_area + (size_t)rows * 2 * kD);
    rp.signs = d->signs;
    rp.heads = d->heads; rp.m_tokens = (int)a.m_tokens; rp.rotate = (d->flags & KVQ_ROTATE_K) ? 1 : 0;
    rp.ax_coef = -a.softmax_scale / 24.0f;
    const kvq_strides dense{(int64_t)d->heads * a.m_tokens * kD, a.m_tokens * (int64_t)kD, (int64_t)kD};
    if ((r = make_map(enc, &mqr, rp.qr, dense, a.m_tokens, d->heads, d->batch)) != KVQ_OK) return r;
  }
  TParams p;
  p.out = static_cast<uint16_t*>(a.out); p.o_sb = a.os.b; p.o_sh = a.os.h; p.o_st = a.os.t;
  p.k_codes = static_cast<const uint8_t*>(d->k_codes); p.v_codes = static_cast<const uint8_t*>(d->v_codes);
  p.k_scale = static_cast<const uint8_t*>(d->k_scale); p.v_scale = static_cast<const uint8_t*>(d->v_scale);
  p.k_zero = static_cast<const uint16_t*>(d->k_zero); p.v_zero = static_cast<const uint16_t*>(d->v_zero);
  p.signs = d->signs;
  p.capacity = d->capacity; p.cache_begin = a.cache_begin % d->capacity;
  p.heads = d->heads; p.group = d->group; p.rotate = (d->flags & KVQ_ROTATE_K) ? 1 : 0;
  p.correction = (a.flags & KVQ_CORRECTION_ON) ? 1 : 0;
  p.m_tokens = (int)a.m_tokens; p.n_cached = (int)a.cache_len; p.n_cur = (int)a.n_cur;
  p.scale_log2 = a.softmax_scale * kLog2e;
  p.ax_coef = -a.softmax_scale / 24.0f;
  p.lse = a.lse; p.cached_mass = a.cached_mass; p.status = a.status_word;
  { const uint32_t b = g_wait_budget.load(std::memory_order_relaxed); p.wait_budget = b ? b : kTimeoutCycles; }
  p.q_blocks = (int)qb; p.n_units = (int)nu; p.tiles = (int)tiles;
  p.partial = slots;
  p.ax_rows = rp.ax;
  p.n_whole = pl.n_whole;
  dim3 grid((unsigned)pl.ctas);
#define KVQ_LAUNCH(B_, G_) (pair ? launch<B_, G_, true>(mq, mqr, mk, mv, p, rp, grid, a.stream) \
                                 : launch<B_, G_, false>(mq, mqr, mk, mv, p, rp, grid, a.stream))
  if (d->bits == 2) {
    if (d->group == 32) return KVQ_LAUNCH(2, 32);
    if (d->group == 64) return KVQ_LAUNCH(2, 64);
    return KVQ_LAUNCH(2, 128);
  }
  if (d->group == 32) return KVQ_LAUNCH(4, 32);
  if (d->group == 64) return KVQ_LAUNCH(4, 64);
  return KVQ_LAUNCH(4, 128);
#undef KVQ_LAUNCH
}

int launch_attn_tcgen05(const AttnArgs& a) {
  const bool pair = (a.flags & KVQ_KERNEL_MASK) == KVQ_KERNEL_TCGEN05_PAIR;
  int64_t qb, nu, tiles;
  schedule_shape(a.desc, a.cache_len, a.m_tokens, a.n_cur, &qb, &nu, &tiles, pair);
  if (nu * tiles > 0x7FFFFFFFLL) return KVQ_ERR_UNSUPPORTED;
  const Plan pl = plan_grid(nu, tiles, pair);
  // workspace: [rotated-query area][partial-result slots]; its size was checked by the caller
  const size_t rot = rot_area_bytes(a.desc, a.cache_len, a.m_tokens);
  uint8_t* ws = static_cast<uint8_t*>(a.workspace);
  return launch_planned(a, pl, qb, nu, tiles, rot ? ws : nullptr, ws + rot, pair);
}


// ---- variant with built-in scratch ---------------------------------------------------------------
//
// Some callers may not allocate device memory at all (an inference server that hands its whole memory pool
// to a framework allocator up front, a plug-in that is only given input and output pointers).  For them the split-unit path can run on a scratch buffer that is
// part of the library image: every GPU that loads libkvq.so carries these 6.3 MiB until the process exits.
// Layout: the rotated-query area for up to kStaticMaxRows query rows (batch * heads * m_tokens), then two
// partial results for each of up to kStaticMaxCtas CTAs.
constexpr int kStaticMaxRows = 8192;
constexpr int kStaticMaxCtas = 32;                         // split problems run on at most this many CTAs
constexpr int kStaticSlots = 2 * kStaticMaxCtas;           // two partial results per CTA
constexpr size_t kStaticRotBytes = (size_t)kStaticMaxRows * (2 * kD + 16);
static_assert(kStaticRotBytes % 256 == 0, "slots must start 256-byte aligned");
static __device__ __align__(256) uint8_t g_static_scratch[kStaticRotBytes + (size_t)kStaticSlots * kSlotBytes];

// The array's name is only a host-side handle; the device address has to be asked for, once per device,
// with that device current.
static int static_scratch_ptr(uint8_t** out) {
  static std::atomic<uint8_t*> ptrs[kMaxDevices] = {};
  int dev = 0;
  { const int r = current_device(&dev); if (r != KVQ_OK) return r; }
  uint8_t* ptr = ptrs[dev].load(std::memory_order_acquire);
  if (!ptr) {
    void* p = nullptr;
    KVQ_CUDA_TRY(cudaGetSymbolAddress(&p, g_static_scratch));
    if (!p) return record_cuda_error(cudaErrorInvalidSymbol);
    ptr = static_cast<uint8_t*>(p);
    ptrs[dev].store(ptr, std::memory_order_release);
  }
  *out = ptr;
  return KVQ_OK;
}

int launch_attn_tcgen05_static(const AttnArgs& a) {
  const kvq_cache_desc* d = a.desc;
  int64_t qb, nu, tiles;
  schedule_shape(d, a.cache_len, a.m_tokens, a.n_cur, &qb, &nu, &tiles);
  if (nu * tiles > 0x7FFFFFFFLL) return KVQ_ERR_UNSUPPORTED;
  Plan pl = plan_grid(nu, tiles);
  bool need_slots = false;
  if (pl.n_whole != nu) {
    if (pl.n_whole > 0) {
      pl.n_whole = (int)nu;                                // many units: deal all of them out whole, no slots
    } else {                                               // few units, all split: partial results need the slots
      if (nu > kStaticMaxCtas) return KVQ_ERR_WORKSPACE;   // stated maximum: 32 units when splitting
      if (pl.ctas > kStaticMaxCtas) pl.ctas = kStaticMaxCtas;
      if (pl.ctas < nu) pl.ctas = (int)nu;
      need_slots = true;
    }
  }
  const size_t rot = rot_area_bytes(d, a.cache_len, a.m_tokens);
  if (rot > kStaticRotBytes) return KVQ_ERR_WORKSPACE;  // stated maximum: 8192 query rows over a non-empty cache
  uint8_t* scratch = nullptr;
  if (rot || need_slots) {
    const int r = static_scratch_ptr(&scratch);
    if (r != KVQ_OK) return r;
  }
  return launch_planned(a, pl, qb, nu, tiles, rot ? scratch : nullptr, need_slots ? scratch + kStaticRotBytes : nullptr);
}

}  // namespace kvq

#ifdef KVQ_TRACE
extern "C" int kvq_debug_trace_read(uint32_t* host_out) {
  return (int)cudaMemcpyFromSymbol(host_out, kvq::g_trace, sizeof(kvq::g_trace));
}
extern "C" int kvq_debug_trace_clear() {
  static uint32_t zeros[16 * kvq::kTraceLen];
  return (int)cudaMemcpyToSymbol(kvq::g_trace, zeros, sizeof(zeros));
}
#endif
