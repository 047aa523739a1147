/*
 * kvq — corrected low-bit KV-cache chunk attention for NVIDIA B200 (sm_100a).
 *
 * C ABI of libkvq.so.  Two operations of the method are exported:
 *
 *   kvq_quantize_append   Hadamard-rotate (keys), quantize, pack and append a
 *                         finished chunk's K/V to the low-bit cache.
 *   kvq_attn_corrected    attention of a BF16 current chunk over [packed cache +
 *                         BF16 current chunk] with the per-score Jensen-bias
 *                         correction subtracted from cached-key scores only.
 *
 * Conventions
 *   - Every call returns an int: KVQ_OK (0) or a negative KVQ_ERR_* code.
 *   - All data pointers are DEVICE pointers unless a parameter says "host".
 *     The descriptor structs themselves are host memory, read during the call.
 *   - The caller owns every buffer.  The library allocates no device memory,
 *     never synchronises and only enqueues work on the given stream.  Calls that
 *     touch one cache must be ordered by the caller (same stream or events).
 *   - Argument errors are detected on the host before anything is launched and
 *     leave all buffers untouched.  A CUDA launch error is returned as
 *     KVQ_ERR_CUDA; kvq_last_cuda_error() gives the cudaError_t value.
 *   - Tensors are [batch, heads, tokens, head_dim] with element strides given by
 *     kvq_strides; the innermost (head_dim) stride is 1.
 *
 * Cache format (paper Sec. 5.1 "Quantization configuration", App. B storage
 * paragraph and Eq. (21)): per (batch, head, token) head_dim*bits/8 bytes of
 * packed codes for K and for V, and per group of `group` consecutive channels
 * one FP8-E4M3 scale (the step size) and one BF16 zero-point: 24 metadata bits
 * per group, effective width bits + 24/group.
 *   codes  u8  [batch, heads, capacity, head_dim*bits/8]   little-endian, element 0 in
 *                                                          the least significant bits
 *   scale  u8  [batch, heads, capacity, head_dim/group]    raw E4M3 byte
 *   zero   u16 [batch, heads, capacity, head_dim/group]    raw BF16 bits, integer-valued
 */
#ifndef KVQ_H_
#define KVQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define KVQ_VERSION 1

/* status codes */
#define KVQ_OK                 0
#define KVQ_ERR_INVALID_ARG   -1   /* null pointer, non-positive size, group does not divide head_dim */
#define KVQ_ERR_UNSUPPORTED   -2   /* head_dim / bits / group combination not built, or batch * heads > 65535 */
#define KVQ_ERR_ALIGNMENT     -3   /* pointer not 16-byte aligned, stride not a multiple of 8 elements */
#define KVQ_ERR_CAPACITY      -4   /* the append or the window would run past `capacity` */
#define KVQ_ERR_CUDA          -5   /* a CUDA runtime/driver call failed; see kvq_last_cuda_error() */
#define KVQ_ERR_TIMEOUT       -6   /* a bounded device-side wait expired: what kvq_status_word_result() returns for a
                                      non-zero status_word */
#define KVQ_ERR_WORKSPACE     -7   /* workspace missing or smaller than kvq_attn_workspace_bytes() */

/* kvq_cache_desc.flags */
#define KVQ_ROTATE_K          1u   /* keys (and queries) are Hadamard-rotated before quantization */
#define KVQ_ROTATE_V          4u   /* values are rotated too before quantization (y = (1/sqrt d) H (signs . v), the value
                                      path of the rotation scheme App. F extends); kvq_attn_corrected then rotates the
                                      current chunk's values the same way (a pre-pass into the workspace) and rotates
                                      the output back (a post-pass over out).  Not with the static-scratch entry. */
#define KVQ_K_PER_CHANNEL     8u   /* App. E: key steps and zero-points per channel, shared by the `group` tokens of a
                                      block: k_scale and k_zero are then [batch,heads,capacity/group,head_dim] (the same
                                      bytes in all), values keep the per-token layout.  Appends and windows must start
                                      on multiples of `group` tokens and appends bring whole blocks
                                      (KVQ_ERR_ALIGNMENT).  Attention: warp-level kernel only, Taylor form only. */
#define KVQ_RING              2u   /* ring cache for sliding-window attention (Section 2; the windows of Section 5.1):
                                      token t lives in slot t mod capacity, new tokens overwrite the oldest.  Token
                                      positions (cache_len of kvq_quantize_append, cache_begin of the attention calls)
                                      are then unbounded; one append may bring at most `capacity` tokens and a window
                                      may hold at most `capacity` tokens.  Which tokens are still stored is the
                                      caller's bookkeeping: the last `capacity` appended ones. */

/* kvq_attn_corrected flags */
#define KVQ_CORRECTION_OFF    0u
#define KVQ_CORRECTION_ON     1u   /* subtract the Taylor bias (Eq. 15 / Eq. 25) from cached scores */
#define KVQ_CORRECTION_EXACT  2u   /* subtract the exact bias of Eq. (12) instead: sum over channels of
                                      log(sinh(a)/a), a = softmax_scale * |q~_c| * step / 2.  Not together with
                                      KVQ_CORRECTION_ON.  Warp-level kernel only (KVQ_KERNEL_AUTO picks it;
                                      KVQ_KERNEL_TCGEN05 and the static-scratch entry return
                                      KVQ_ERR_UNSUPPORTED): an analysis option, several times slower. */
#define KVQ_KERNEL_AUTO       0u         /* head_dim 128 with TMA-addressable strides: the pair kernel unless its units of 512
                                            query rows pad m_tokens too far beyond a multiple of 256 (by more than 1/0.88
                                            at 2 bits, 1/0.86 at 4), then the one-CTA tcgen05 kernel; everything else: the
                                            warp-level kernel */
#define KVQ_KERNEL_MMA_SYNC   (1u << 8)  /* force the warp-level mma.sync kernel (cross-check / fallback shapes) */
#define KVQ_KERNEL_TCGEN05    (2u << 8)  /* force the tcgen05/TMEM kernel; KVQ_ERR_UNSUPPORTED if the shape is not covered */
#define KVQ_KERNEL_TCGEN05_PAIR (3u << 8) /* the tcgen05 kernel on pairs of SMs (thread-block clusters of two CTAs that share
                                            one tcgen05.mma of 256 rows): each CTA of a pair expands only half of every
                                            cached key and value tile.  Same shapes as KVQ_KERNEL_TCGEN05; results equal to
                                            its within rounding (a quarter of the exponentials are a cubic on the FMA
                                            pipe, relative error 7.5e-5, before the BF16 rounding of the weights) */
#define KVQ_KERNEL_MASK       (3u << 8)

typedef void* kvq_stream_t;          /* a cudaStream_t */

/* Describes one caller-owned cache.  Plain data, host memory. */
typedef struct kvq_cache_desc {
  int32_t  batch, heads, head_dim;   /* head_dim: 64 or 128; batch * heads <= 65535 (a grid dimension) */
  int32_t  bits;                     /* 2 or 4 */
  int32_t  group;                    /* 32, 64 or 128; divides head_dim */
  uint32_t flags;                    /* KVQ_ROTATE_K | KVQ_ROTATE_V | KVQ_RING | KVQ_K_PER_CHANNEL */
  int64_t  capacity;                 /* tokens per (batch, head); a multiple of 128 */
  void*    k_codes;  void* v_codes;  /* device, u8  [batch,heads,capacity, head_dim*bits/8] */
  void*    k_scale;  void* v_scale;  /* device, u8  [batch,heads,capacity, head_dim/group] (E4M3) */
  void*    k_zero;   void* v_zero;   /* device, u16 [batch,heads,capacity, head_dim/group] (BF16) */
  const int8_t* signs;               /* device, +1/-1 [head_dim] of the randomised Hadamard, or NULL = all +1 */
} kvq_cache_desc;

/* Element strides of a [batch, heads, tokens, head_dim] BF16 tensor. */
typedef struct kvq_strides { int64_t b, h, t; } kvq_strides;

/*
 * Sizes in bytes of the six cache buffers, in the order k_codes, v_codes, k_scale,
 * v_scale, k_zero, v_zero (App. B storage paragraph, Eq. (21)).  Only the shape
 * fields of the descriptor are read; out_bytes is host memory.
 * Errors: KVQ_ERR_INVALID_ARG, KVQ_ERR_UNSUPPORTED.
 */
int kvq_cache_bytes(const kvq_cache_desc* desc, size_t out_bytes[6]);

/*
 * Quantize-append (paper Sec. 3: Eq. (1) asymmetric round-to-nearest; "Quantization
 * granularity": group-wise per-token; "Hadamard rotation": keys rotated by the normalised
 * Hadamard matrix; Sec. 5.1: E4M3 scales, BF16 zero-points).
 *
 * For every (batch, head) and every token t in [0, n_tokens) of the BF16 inputs k, v:
 *   y  = (1/sqrt(head_dim)) * H * (signs . k_t)   if KVQ_ROTATE_K, else k_t; values are not rotated
 *   per group: step = E4M3((max - min) / (2^bits - 1)), floored at 2^-9, saturated at 448
 *              zero = BF16(-round(min / step))
 *              code = clamp(round(y / step) + zero, 0, 2^bits - 1)          (ties to even)
 * and stores codes, step and zero at cache token cache_len + t.  All arithmetic is IEEE
 * binary32 with one rounding per operation (butterfly stages h = 1, 2, 4, ... in that order,
 * then one multiply by the binary32 value of 1/sqrt(head_dim)), so results are reproducible
 * bit for bit.
 *
 * k, v: device BF16, strides `kv`, 16-byte aligned, strides multiples of 8 elements.
 * The cache tokens [cache_len, cache_len + n_tokens) are overwritten; nothing else is.
 * n_tokens == 0 is a no-op.  Errors: KVQ_ERR_INVALID_ARG, KVQ_ERR_UNSUPPORTED,
 * KVQ_ERR_ALIGNMENT, KVQ_ERR_CAPACITY (cache_len + n_tokens > capacity), KVQ_ERR_CUDA.
 */
int kvq_quantize_append(const kvq_cache_desc* desc, int64_t cache_len,
                        const void* k_bf16, const void* v_bf16, kvq_strides kv,
                        int64_t n_tokens, kvq_stream_t stream);

/*
 * Bytes of device workspace kvq_attn_corrected needs for this problem (may be 0).  With the tcgen05 kernel
 * and a non-empty cache window it holds the rotated query chunk (Section 3.1: q~ = H q in FP16, plus the
 * per-group squared norms nu of Eq. 15, 272 bytes per query row, written by a pre-pass kernel of the same
 * call) and, when the key tiles of a unit are split over several CTAs, their partial results.
 * out_bytes is host memory.  Same errors as kvq_attn_corrected's argument checks.
 */
int kvq_attn_workspace_bytes(const kvq_cache_desc* desc, int64_t cache_len,
                             int64_t m_tokens, int64_t n_cur, uint32_t flags, size_t* out_bytes);

/*
 * How many kernels one kvq_attn_corrected call launches for this problem (host-side bookkeeping for
 * benchmarks and launch-bound callers): the attention kernel, the query pre-pass when the cache window
 * is not empty, the merge kernel when units are split over CTAs.  out_count is host memory.  Same
 * argument checks and errors as kvq_attn_workspace_bytes.
 */
int kvq_attn_kernel_launches(const kvq_cache_desc* desc, int64_t cache_len,
                             int64_t m_tokens, int64_t n_cur, uint32_t flags, int* out_count);

/*
 * Corrected chunk attention (paper Algorithm 1; Eqs. (2)-(4) for scores, partition sums and
 * cached mass; Eq. (15) and its rotated form Eq. (25) for the bias; Sec. 4.2: the bias is
 * subtracted from cached scores only).
 *
 * For every (batch, head) and query row m in [0, m_tokens):
 *   q~      = (1/sqrt(head_dim)) * H * (signs . q_m)  if KVQ_ROTATE_K, else q_m
 *   nu_j    = sum over channels c of group j of q~_c^2
 *   k^_i    = (code_i - zero_i) * step_i,  v^_i likewise        (cache tokens cache_begin + i, i < cache_len)
 *   s_i     = softmax_scale * q~ . k^_i  -  [flags & KVQ_CORRECTION_ON] (softmax_scale^2 / 24) * sum_j step_{i,j}^2 * nu_j
 *   s_r     = softmax_scale * q_m . k_cur_r                      (r < n_cur; never corrected)
 *   out_m   = softmax over all s_i and s_r, applied to [v^_i ; v_cur_r]            (no mask)
 * Accumulation is FP32, operands of the two contractions are BF16, the output is BF16.
 *
 * q: [batch,heads,m_tokens,head_dim] strides q_strides; k_cur, v_cur: [batch,heads,n_cur,head_dim]
 * strides kv_strides; out: strides o_strides.  All device BF16, 16-byte aligned, strides
 * multiples of 8 elements.  A batch or head stride of 0 (a chunk shared by all heads) is accepted: the tcgen05
 * kernel cannot address such a tensor, so KVQ_KERNEL_AUTO runs the warp-level kernel for it and a forced
 * KVQ_KERNEL_TCGEN05 returns KVQ_ERR_UNSUPPORTED.  cache_begin must be a multiple of 16 and
 * cache_begin + cache_len <= capacity.  cache_len == 0 is legal (plain attention over the
 * current chunk); n_cur must be >= 1; m_tokens == 0 is a no-op.
 *
 * lse_out          optional device float [batch,heads,m_tokens]: log of the softmax denominator
 *                  (natural log, scores as defined above); NULL to skip.
 * cached_mass_out  optional device float [batch,heads,m_tokens]: P_S of Eq. (4), the softmax mass on
 *                  cached keys; NULL to skip.
 * workspace        device scratch of at least kvq_attn_workspace_bytes() bytes, 256-byte aligned;
 *                  may be NULL when that size is 0.  Contents need not be initialised.
 * status_word      optional device int32, must be zero on entry: set to a non-zero diagnostic if a
 *                  bounded device-side wait expires (the output is then undefined); NULL to skip.
 * Errors: KVQ_ERR_INVALID_ARG, KVQ_ERR_UNSUPPORTED, KVQ_ERR_ALIGNMENT, KVQ_ERR_CAPACITY,
 * KVQ_ERR_WORKSPACE, KVQ_ERR_CUDA.
 */
int kvq_attn_corrected(const kvq_cache_desc* desc, int64_t cache_begin, int64_t cache_len,
                       const void* q, kvq_strides q_strides,
                       const void* k_cur, const void* v_cur, kvq_strides kv_strides,
                       int64_t m_tokens, int64_t n_cur,
                       void* out_bf16, kvq_strides o_strides,
                       float softmax_scale, uint32_t flags,
                       float* lse_out, float* cached_mass_out,
                       void* workspace, size_t workspace_bytes,
                       int32_t* status_word, kvq_stream_t stream);

/*
 * kvq_attn_corrected for callers that cannot allocate device memory.  (The paper has no counterpart: this
 * is a deployment variant of the call above, same arithmetic, same outputs.)
 *
 * Who needs it: code that must not call cudaMalloc — a serving process that has handed all device memory
 * to its framework's pool, a plug-in that only ever receives input and output pointers, anything that runs
 * where an allocation would synchronise the device or is forbidden.  kvq_attn_corrected needs a caller
 * workspace for the rotated query chunk and, when it splits the key tiles of a unit over several CTAs (few
 * query rows, long cache), for their partial results; this entry point keeps both in a scratch buffer that
 * is part of the library image instead: 8192 query rows of 272 bytes plus 64 slots of 68 608 bytes =
 * 6 619 136 bytes of device memory on every GPU that loads libkvq.so, held until the process exits.  It
 * calls no allocating routine of CUDA or of any other library.
 *
 * Limits: head_dim 128 only (the tcgen05 kernel; no kernel-selection flags).  Over a non-empty cache window
 * batch * heads * m_tokens may be at most 8192 query rows.  A problem with fewer units (batch * heads *
 * ceil(m_tokens / 256)) than SMs whose idle SMs are worth splitting for is split, on at most 32 CTAs, and
 * may then have at most 32 units.  Beyond either limit the call returns KVQ_ERR_WORKSPACE and launches
 * nothing.
 *
 * The first call on a device looks up the buffer's device address (cudaGetSymbolAddress, with that device
 * current) and remembers it; make that first call outside any stream capture.
 * All calls on a device share the one buffer and it keeps the previous call's contents.  Nothing in it has
 * to start at zero (every row and slot is written in full before it is read), so no clearing is done; but two calls
 * whose kernels overlap on the GPU (different streams, no ordering between them) race on it: order them.
 *
 * Arguments, outputs and the other error codes are those of kvq_attn_corrected, without the workspace.
 */
int kvq_attn_corrected_static_scratch(const kvq_cache_desc* desc, int64_t cache_begin, int64_t cache_len,
                                      const void* q, kvq_strides q_strides,
                                      const void* k_cur, const void* v_cur, kvq_strides kv_strides,
                                      int64_t m_tokens, int64_t n_cur,
                                      void* out_bf16, kvq_strides o_strides,
                                      float softmax_scale, uint32_t flags,
                                      float* lse_out, float* cached_mass_out,
                                      int32_t* status_word, kvq_stream_t stream);

/*
 * Attention-weight diagnostic (the paper's appendix "Attention JSD Distributions"): for every (batch, head) and
 * query row, the Jensen-Shannon divergence (natural logarithm, between 0 and log 2) between
 *   p = softmax over the scores s_i, s_r of kvq_attn_corrected (quantized cache, correction on or off), and
 *   r = softmax over softmax_scale * q . k for the BF16 keys [k_cached_bf16 ; k_cur],
 * both over all cache_len + n_cur keys.  k_cached_bf16 [batch, heads, cache_len, head_dim] (device BF16, strides
 * kcached_strides) are the keys the cache window [cache_begin, cache_begin + cache_len) was quantized from: an
 * analysis input that a deployment does not keep; may be NULL when cache_len is 0.
 * jsd_out: device float [batch, heads, m_tokens].  Nothing of size m_tokens x keys is written: scores are
 * recomputed in FP32 on the CUDA cores in two passes (log-sum-exps, then the divergence), so this is an
 * analysis call, not a fast one.  flags: KVQ_CORRECTION_ON or KVQ_CORRECTION_OFF only; not for
 * KVQ_K_PER_CHANNEL caches.  Errors: as kvq_attn_corrected's argument checks, KVQ_ERR_UNSUPPORTED for the
 * options above, KVQ_ERR_CUDA.
 */
int kvq_attn_weight_jsd(const kvq_cache_desc* desc, int64_t cache_begin, int64_t cache_len,
                        const void* q, kvq_strides q_strides,
                        const void* k_cur, kvq_strides kcur_strides,
                        const void* k_cached_bf16, kvq_strides kcached_strides,
                        int64_t m_tokens, int64_t n_cur, float softmax_scale, uint32_t flags,
                        float* jsd_out, kvq_stream_t stream);

/*
 * Test aid: expand the packed codes of cache tokens [begin, begin + n) to one byte per element,
 * out_codes device u8 [batch, heads, n, head_dim], in canonical channel order (the order of
 * Eq. (1)'s vector x).  which: 0 = keys, 1 = values.
 * Errors: KVQ_ERR_INVALID_ARG, KVQ_ERR_UNSUPPORTED, KVQ_ERR_CAPACITY, KVQ_ERR_CUDA.
 */
int kvq_unpack_codes(const kvq_cache_desc* desc, int which, int64_t begin, int64_t n,
                     uint8_t* out_codes, kvq_stream_t stream);

/*
 * Bounded device-side waits.  (The paper has no counterpart: this is how the tcgen05 kernel fails.)
 *
 * Inside the tcgen05 kernel the roles of a CTA (TMA producer, MMA issuer, softmax warps, dequantization warps)
 * hand tiles to one another through shared-memory barriers.  No wait on such a barrier is unbounded: a wait
 * that does not complete within its cycle budget (about one second by default) records a site code in the
 * CTA, every role of that CTA leaves its loop at its next wait, work in flight is drained, and the kernel
 * returns.  The first site code reaches the caller's status_word; the outputs are then undefined.
 * Site codes: TMA producer 100 (query buffer free), 101 (key stage free), 102 (value stage free), 103 (last
 * unrotated score product done), 104 (stage of the packed-tile ring free); MMA issuer 201 (query tile), 203 (value tile), 204 (probabilities), 205 (key
 * tile), 207 (rotated query), 209 (output accumulator read out); softmax warps 301 (scores), 302 (product
 * retired before a rescale), 303 (last product before the epilogue); dequantization warps 401 (key stage free),
 * 402 (query tile, for the bias rows), 404 (value stage free), 406 (packed tile in the ring).
 *
 * kvq_status_word_result maps a status word read back by the caller (host value) to KVQ_OK (0) or
 * KVQ_ERR_TIMEOUT (anything else).
 * kvq_set_wait_budget_cycles sets the budget, in SM clock cycles, for kernels launched afterwards by this
 * process (0 restores the default; values above 0xFFFF0000 are KVQ_ERR_INVALID_ARG).  It exists so that the
 * time-out path can be exercised on purpose: with a budget of a few cycles the first wait that is not complete
 * at its first poll gives up, and the call returns with a status word set, on a healthy GPU and without any
 * wait left hanging.  Not meant for production use.
 */
int kvq_status_word_result(int32_t status_word_value);
int kvq_set_wait_budget_cycles(uint64_t cycles);

/* Host-side helpers. */
const char* kvq_status_string(int status);   /* static string, never NULL */
int kvq_last_cuda_error(void);               /* cudaError_t of the last KVQ_ERR_CUDA on this thread, else 0 */
int kvq_version(void);                       /* KVQ_VERSION the library was built with */

#ifdef __cplusplus
}
#endif
#endif /* KVQ_H_ */
