/* gear.h -- C ABI of the B200-native GEAR hot path (arXiv 2403.05527).
 *
 * GEAR keeps a KV cache as  X ~= D^ + L + S :  a b-bit uniformly quantized
 * backbone D^ (Eq. 2, Eq. 5), a head-wise rank-r matrix L_h = A_h B_h^T fitted
 * to the quantization residual by power iteration (Eq. 6, Algorithm 2) and a
 * sparse matrix S of filtered outliers (Eq. 4).  New tokens wait in a small
 * fp16 streaming buffer and are compressed every n_b steps (Algorithm 1).
 * Decode attention (Eq. 1) reads the compressed cache directly.
 *
 * Conventions
 *  - Every pointer argument says "device" or "host".  Device buffers are
 *    borrowed for the duration of the work enqueued on `stream`; the library
 *    never frees or keeps them.  All tensors are contiguous, row-major.
 *  - The library owns a gear_cache (one per layer): all of its device memory
 *    is allocated when the cache is created and released by gear_free.
 *  - Calls enqueue work on `stream` (a cudaStream_t passed as void*) and return
 *    without synchronising, except where stated (the *_host variants,
 *    gear_export, gear_last_device_status).
 *  - Errors are return codes only; arguments are validated on the host before
 *    anything is launched; no entry point aborts, throws or traps the device.
 *  - Not thread-safe per cache: calls on one cache must be issued from one
 *    thread at a time and on one stream (or streams ordered by the caller).
 *  - Inputs are assumed finite; NaN / Inf give unspecified results, no error.
 *  - Range of the decode kernel's fixed-point operands: per block it scales q * scale_K (per
 *    channel) and p * scale_V (per token and group) by a power of two taken from their largest
 *    magnitude, clamped to 2^+-60.  Every finite fp16 input stays inside that range.
 */
#ifndef GEAR_H_
#define GEAR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t gear_status;
enum {
  GEAR_OK = 0,
  GEAR_FLUSHED = 1,        /* gear_append_buffer: this push filled the buffer and compressed it */
  GEAR_ERR_ARG = -1,       /* NULL / out-of-range argument */
  GEAR_ERR_SHAPE = -2,     /* sizes violate the grouping rules */
  GEAR_ERR_ALIGN = -3,     /* pointer not 16-byte aligned */
  GEAR_ERR_CAPACITY = -4,  /* max_tokens / arena exhausted */
  GEAR_ERR_ALLOC = -5,     /* device allocation failed */
  GEAR_ERR_CUDA = -6,      /* a CUDA runtime call failed */
  GEAR_ERR_TIMEOUT = -7,   /* a bounded device-side wait gave up (see gear_last_device_status) */
  GEAR_ERR_STATE = -8      /* call not valid in the cache's current state */
};

enum {
  GEAR_FLAG_KEEP_FP32_FACTORS = 1u  /* also keep A, B in fp32 (before the fp16 rounding) for gear_export */
};

/* Device memory of the caches.  By default gear_create uses cudaMalloc / cudaFree.  A caller that owns the
 * device heap installs its own pair here (process-wide; NULL, NULL restores the default): alloc returns a
 * device pointer aligned to 256 bytes or NULL, which gear_create reports as GEAR_ERR_ALLOC after handing back
 * what it had taken.  A cache frees through the pair it was created with. */
typedef void* (*gear_alloc_fn)(size_t bytes, void* ctx);
typedef void (*gear_free_fn)(void* ptr, void* ctx);

/* Hyper-parameters in the paper's notation (Section 2 and 3; Algorithm 1, 2). */
#define GEAR_GROUP_PER_VECTOR 0

typedef struct gear_config {
  int32_t batch;        /* sequences in the batch                                              */
  int32_t n_q_heads;    /* H_q query heads; n_q_heads % n_kv_heads == 0                        */
  int32_t n_kv_heads;   /* H   key/value heads                                                  */
  int32_t head_dim;     /* d_H; this build supports 128                                         */
  int32_t bits;         /* b in {2, 4}                                                           */
  int32_t group;        /* g in {16, 32, 64, 128}: keys are grouped per channel over
                           min(g, n_c) consecutive tokens of a segment, values per token over
                           min(g, d_H) consecutive channels (KIVI grouping, Section 2).
                           GEAR_GROUP_PER_VECTOR: the per-vector grouping of the same section (KCVT):
                           one key group per channel over all tokens of a segment, one value group
                           per token; Filter_s then acts on those whole vectors, so a channel of an
                           n-token segment gives up ceil(s n / 200) entries per side (any count
                           below n / 2).  Needs buffer_cap <= 128; segments longer than 128 tokens
                           must be multiples of 64 and at most 8192 tokens long.                  */
  float   outlier_pct;  /* s in percent, 0 <= s <= 10.  Filter_s (Eq. 4) takes
                           k = ceil(s * len / 200) largest and k smallest entries of every
                           group of length len; need k <= 8 and 2k < len                        */
  int32_t buffer_cap;   /* n_b: streaming-buffer capacity in tokens, 16..1024.  A multiple of 16, and of
                           `group` when larger than it; or a multiple of 4 that is smaller than `group`
                           (at most 128 with per-vector grouping), e.g. the paper's n_b = 20: the
                           flushed buffer is then one block whose last 16-token slab is partly empty   */
  int32_t rank_flush;   /* r_g: rank used when a full buffer is compressed, 0..16               */
  int32_t rank_max;     /* largest rank any gear_compress call will use (sizes the arena), 0..16 */
  int32_t power_iters;  /* L >= 1 loops of Algorithm 2                                           */
  int64_t max_tokens;   /* capacity in compressed tokens per sequence (arena is sized from it)   */
  uint64_t seed;        /* start vectors when the caller passes no B0                           */
  uint32_t flags;       /* GEAR_FLAG_*                                                           */
  uint32_t max_queries; /* most query rows per head a gear_decode_attn_multi call will bring (0 or 1: one) */
} gear_config;

typedef struct gear_cache gear_cache;   /* opaque */

gear_status gear_set_allocator(gear_alloc_fn alloc_fn, gear_free_fn free_fn, void* ctx);

/* Create an empty cache (no segment, empty buffer) on the current device.
 * Allocates everything the cache will ever use.  *cache must be NULL. */
gear_status gear_create(gear_cache** cache, const gear_config* cfg);

/* Algorithm 1, prefill body, applied to a block of n tokens: for X in {K, V}
 *   S = Filter_s(X) (Eq. 4);  D^ = Quant_b(X - S) (Eq. 5);  R = X - D^ - S;
 *   per head  A_h B_h^T = SVDSolver_rank(R_h) (Eq. 6, Algorithm 2),
 * and append the result as one compressed segment.
 *   cache  in/out: *cache == NULL creates the cache from cfg first (cfg may be NULL otherwise).
 *   K, V   device fp16 [batch, n_kv_heads, n, head_dim], 16-byte aligned.
 *   n      segment length; multiple of 16, and of `group` when n >= group.
 *   rank   r for this segment, 0 <= rank <= min(rank_max, n).
 *   B0     device fp32 [batch, n_kv_heads, 2 (0 = K, 1 = V), head_dim, rank]: the
 *          power-iteration start (Algorithm 2's random B), or NULL to draw it
 *          from cfg.seed.
 * Must not be called while the streaming buffer holds tokens (GEAR_ERR_STATE). */
gear_status gear_compress(gear_cache** cache, const gear_config* cfg,
                          const void* K, const void* V, int64_t n, int32_t rank,
                          const float* B0, void* stream);

/* Algorithm 1, decoding phase: push (k_t, v_t) into the fp16 buffer; when the
 * push fills it (n_b tokens) compress the buffer with rank r_g as one more
 * segment and clear it (returns GEAR_FLUSHED).
 *   k_new, v_new  device fp16 [batch, n_kv_heads, head_dim].
 *   B0_flush      device fp32 [batch, n_kv_heads, 2, head_dim, rank_flush] or NULL; only
 *                 read by the call that flushes. */
gear_status gear_append_buffer(gear_cache* cache, const void* k_new, const void* v_new,
                               const float* B0_flush, void* stream);

/* Eq. 1 for one query per sequence over the compressed cache, evaluated as
 *   scores = q . dequant(codes_K)^T + (q B_K) A_K^T + q . S_K^T   (+ q . K_buffer^T)
 *   out    = softmax(scores * scale) applied to dequant(codes_V) + A_V B_V^T + S_V (+ V_buffer)
 * with the low-rank terms taken as down- then up-projection (Section 4,
 * "Implementation optimization"); fp16 K/V are never materialised.
 *   q     device fp16 [batch, n_q_heads, head_dim];  query head h reads kv head h / (H_q / H).
 *   out   device fp32 [batch, n_q_heads, head_dim].
 *   softmax_scale  <= 0 selects 1 / sqrt(head_dim).
 * The cache must hold at least one token (GEAR_ERR_STATE otherwise). */
gear_status gear_decode_attn(gear_cache* cache, const void* q, float* out,
                             float softmax_scale, void* stream);

/* Eq. 1 for n_queries query rows per sequence and head at once (several positions scored against the same
 * cache, as in speculative or chunked decoding): every row attends to every cached token, no mask among the rows.
 *   q     device fp16 [batch, n_q_heads, n_queries, head_dim];  out device fp32, same shape.
 *   n_queries  1 .. cfg.max_queries.
 * The rows of a kv head share each read of its compressed blocks four at a time: G * n_queries rows take
 * ceil(G * n_queries / 4) passes over the cache. */
gear_status gear_decode_attn_multi(gear_cache* cache, const void* q, float* out, int32_t n_queries,
                                   float softmax_scale, void* stream);

/* Release the cache and everything it owns.  NULL is allowed. */
void gear_free(gear_cache* cache);

/* gear_compress takes its transient workspace (the residual of the block being compressed, up to 3 GB)
 * from a stream-ordered pool that the library keeps per device, so that repeated calls do not go back
 * to the driver.  This call synchronises the current device and returns that memory to the driver. */
gear_status gear_release_workspace(void);

/* ---- host-buffer variants (copies inside the call) ---- */

/* gear_append_buffer with k_new, v_new (and B0_flush) in HOST memory (pinned or pageable).  The rows are copied
 * to pinned memory of the library before the call returns, so the caller may reuse its buffers at once; the call
 * does not wait for the device, except when it passes B0_flush on to a flush (that array is read in place, and
 * the call then synchronises `stream`).  Calls on one cache must use one stream. */
gear_status gear_append_buffer_host(gear_cache* cache, const void* k_new_host, const void* v_new_host,
                                    const float* B0_flush_host, void* stream);
/* gear_decode_attn with q and out in HOST memory; waits for the result (out_host is valid on return). */
gear_status gear_decode_attn_host(gear_cache* cache, const void* q_host, float* out_host,
                                  float softmax_scale, void* stream);
/* The same without the wait: the copies and the kernel are queued and the call returns.  q_host must stay
 * unchanged, and out_host is not valid, until gear_cache_wait(cache) has returned.  A model step queues all its
 * layers this way and then waits for each cache once.  Errors as gear_decode_attn. */
gear_status gear_decode_attn_host_async(gear_cache* cache, const void* q_host, float* out_host,
                                        float softmax_scale, void* stream);
/* One decoding step of one layer through HOST buffers, queued like gear_decode_attn_host_async: the new key / value
 * rows and the query go up in one copy (through pinned memory of the library: k_new_host, v_new_host and q_host may
 * be reused on return), the rows are pushed (gear_append_buffer with library-drawn start vectors if the push
 * flushes), the query attends to the cache including the new token, and the result comes down into out_host, valid
 * after gear_cache_wait(cache).  Returns GEAR_OK, GEAR_FLUSHED or an error of the two calls it combines. */
gear_status gear_step_host(gear_cache* cache, const void* k_new_host, const void* v_new_host, const void* q_host,
                           float* out_host, float softmax_scale, void* stream);
/* Blocks the calling host thread until the host-buffer calls queued on `cache` so far have finished: their copies
 * run on a stream of the cache's own (ordered against the caller's stream by events, so that one cache's copies run
 * beside another cache's kernels), which this call waits for.  GEAR_ERR_CUDA if that stream reports an error. */
gear_status gear_cache_wait(gear_cache* cache);

/* ---- FP16-cache reference point for the same decode step (Eq. 1 on uncompressed K, V) ---- */

/* out = softmax(q K^T * scale) V over an fp16 cache.
 *   K, V  device fp16 [batch, n_kv_heads, n_alloc, head_dim] of which the first n tokens are used;
 *   q     device fp16 [batch, n_q_heads, head_dim];  out device fp32 [batch, n_q_heads, head_dim];
 *   scratch  device, at least gear_fp16_attn_scratch_bytes(...) bytes, 16-byte aligned. */
gear_status gear_fp16_decode_attn(const void* K, const void* V, const void* q, float* out,
                                  int32_t batch, int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim,
                                  int64_t n, int64_t n_alloc, float softmax_scale,
                                  void* scratch, size_t scratch_bytes, void* stream);
size_t gear_fp16_attn_scratch_bytes(int32_t batch, int32_t n_q_heads, int32_t head_dim);

/* gear_fp16_decode_attn for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a packaging variant of the call above, not a step of the method.)
 *
 * Some hosts of this library are not allowed to call cudaMalloc at the point where they need
 * attention: code running inside a framework that owns the whole device heap, a plug-in that is
 * handed buffers but no allocator, or a latency-critical loop in which an allocation (which may
 * synchronise the device) is not acceptable.  For them the scratch memory that
 * gear_fp16_decode_attn takes from the caller lives in a fixed array of
 * GEAR_STATIC_SCRATCH_BYTES inside the library's device image: every GPU that loads the
 * library holds that much memory until the process exits.  The call allocates and frees
 * nothing, on the device or through any library.
 *
 * Arguments and result are those of gear_fp16_decode_attn (K, V, q, out are device pointers,
 * 16-byte aligned, borrowed for the duration of the enqueued work) without the scratch pair.
 *   - batch * n_q_heads must not exceed GEAR_STATIC_MAX_QUERY_HEADS; larger problems, or any
 *     problem whose bookkeeping does not fit the array, return GEAR_ERR_CAPACITY and launch
 *     nothing.  Within the limit the launch may use fewer CTAs than gear_fp16_decode_attn
 *     would, so that its partial results fit; the output is the same up to rounding order.
 *   - The first call on a device looks up the array's device address (once per device, with
 *     that device current).  Make that first call outside any stream capture.
 *   - All calls on a device share the one array, and the array keeps what the last call left
 *     in it; each call clears the part that must start at zero on `stream` before its kernel.
 *     Two calls whose GPU work can overlap (different streams without an ordering between
 *     them, or several host threads) race on the array: order them. */
#define GEAR_STATIC_SCRATCH_BYTES (4u << 20)
#define GEAR_STATIC_MAX_QUERY_HEADS 256
gear_status gear_fp16_decode_attn_static(const void* K, const void* V, const void* q, float* out,
                                         int32_t batch, int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim,
                                         int64_t n, int64_t n_alloc, float softmax_scale, void* stream);

/* ---- test / accounting helpers (not on the timed path; gear_export synchronises) ---- */

enum {                       /* `what` of gear_export; K_ / V_ select the side                      */
  GEAR_EXP_K_CODES = 0,      /* u8  [B, H, n_c, d_H]            one code per byte                    */
  GEAR_EXP_V_CODES = 1,
  GEAR_EXP_K_SCALE = 2,      /* f16 [B, H, n_c / g_K, d_H]      scale (Delta) of every key group     */
  GEAR_EXP_V_SCALE = 3,      /* f16 [B, H, n_c, d_H / g_V]                                            */
  GEAR_EXP_K_ZERO = 4,       /* f16, same shape as the scale: zero-point (group minimum)             */
  GEAR_EXP_V_ZERO = 5,
  GEAR_EXP_K_OUT_IDX = 6,    /* u8  [B, H, n_c / g_K, d_H, 2k]  in-group token index, ascending      */
  GEAR_EXP_V_OUT_IDX = 7,    /* u8  [B, H, n_c, d_H / g_V, 2k]  in-group channel index, ascending    */
  GEAR_EXP_K_OUT_VAL = 8,    /* f16, same shape as the index: the outlier values, same order         */
  GEAR_EXP_V_OUT_VAL = 9,
  GEAR_EXP_K_A = 10,         /* f32 [B, H, n_c, r]   as stored (fp16 rounded)                        */
  GEAR_EXP_V_A = 11,
  GEAR_EXP_K_B = 12,         /* f32 [B, H, d_H, r]   as stored (fp16 rounded)                        */
  GEAR_EXP_V_B = 13,
  GEAR_EXP_K_A_FP32 = 14,    /* f32, before the fp16 rounding (needs GEAR_FLAG_KEEP_FP32_FACTORS)    */
  GEAR_EXP_V_A_FP32 = 15,
  GEAR_EXP_K_B_FP32 = 16,
  GEAR_EXP_V_B_FP32 = 17,
  GEAR_EXP_K_BUFFER = 18,    /* f16 [B, H, buffer_len, d_H]  (segment argument ignored)              */
  GEAR_EXP_V_BUFFER = 19
};

/* Copy one piece of segment `segment` to HOST memory in the canonical
 * (unpacked) layout above.  `bytes` must equal the piece's size exactly. */
gear_status gear_export(gear_cache* cache, int32_t segment, int32_t what,
                        void* host_dst, size_t bytes);

typedef struct gear_info {
  int32_t n_segments;
  int32_t buffer_len;        /* tokens waiting in the fp16 buffer */
  int64_t n_compressed;      /* tokens in compressed segments     */
} gear_info;
gear_status gear_cache_info(const gear_cache* cache, gear_info* info);

typedef struct gear_segment_info {
  int64_t n_c;               /* tokens in the segment                          */
  int32_t rank;
  int32_t g_k, g_v;          /* effective group lengths                        */
  int32_t k_k, k_v;          /* outliers per side per key / value group        */
} gear_segment_info;
gear_status gear_segment_info_get(const gear_cache* cache, int32_t segment, gear_segment_info* info);

/* Bytes the decode kernel reads per call, by component (whole batch, all kv
 * heads): the denominator of the bandwidth figures.  `stored_*` include the
 * layout's padding; `alloc_total` is what gear_create allocated. */
typedef struct gear_bytes {
  int64_t codes, scale_zero, outliers, lowrank_a, lowrank_b, buffer;
  int64_t stored_total;      /* bytes of records + B factors + buffer actually read */
  int64_t alloc_total;
} gear_bytes;
gear_status gear_cache_bytes(const gear_cache* cache, gear_bytes* out);

/* Read (and clear) the device status word: 0, or the GEAR_ERR_* a kernel recorded (GEAR_ERR_TIMEOUT: a bounded
 * wait on a copy gave up; the outputs of the calls since the last read are then undefined).  Synchronises the
 * device.  When the word was set, the call also resets the cache's merge counters, so that the next
 * gear_decode_attn on the cache starts clean. */
gear_status gear_last_device_status(gear_cache* cache, int32_t* code);
/* The same word for gear_fp16_decode_attn (it lives at the start of the caller's scratch buffer) and for
 * gear_fp16_decode_attn_static (it lives in the library's array on the current device). */
gear_status gear_fp16_attn_status(void* scratch, int32_t* code);
gear_status gear_fp16_attn_static_status(int32_t* code);
/* Test only: while `on`, every decode call on the cache first waits, with a limit of a few dozen polls, on a
 * barrier that nothing completes, so that the give-up path runs: the kernel drains its copies, records
 * GEAR_ERR_TIMEOUT and returns.  Nothing faults, traps or hangs. */
gear_status gear_test_dead_wait(gear_cache* cache, int32_t on);

const char* gear_strerror(gear_status s);

/* Number of kernels this library has launched in this process so far (all caches). */
uint64_t gear_kernel_launches(void);

#ifdef __cplusplus
}
#endif
#endif /* GEAR_H_ */
