// C ABI of the library: cache object, argument checks, launch sequences.
#include <cuda_runtime.h>
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <atomic>
#include <mutex>
#include <new>
#include <unordered_map>
#include <vector>

#include "../../include/gear.h"
#include "gear_internal.cuh"

using namespace gear;

static std::atomic<unsigned long long> g_launches{0};
// Calls of the library that launch kernels, numbered per stream: a decode call may request its first copies before
// it waits for the kernel in front of it only if that kernel cannot be the one that last wrote the cache.
static std::mutex g_seq_mutex;
static std::unordered_map<cudaStream_t, unsigned long long> g_stream_seq;
static unsigned long long next_call_number(cudaStream_t st) {
  std::lock_guard<std::mutex> lock(g_seq_mutex);
  return ++g_stream_seq[st];
}

void gear::count_launches(int n) { g_launches.fetch_add((unsigned long long)n, std::memory_order_relaxed); }
extern "C" uint64_t gear_kernel_launches(void) { return g_launches.load(std::memory_order_relaxed); }

// Transient workspace of gear_compress comes from one stream-ordered pool per device that keeps its memory between
// calls (the default pool hands it back to the driver at every synchronisation, which costs milliseconds per call).
static std::mutex g_pool_mutex;
static cudaMemPool_t g_pool[64];
static bool g_pool_ready[64];
static cudaMemPool_t workspace_pool(int dev) {
  if (dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> lock(g_pool_mutex);
  if (!g_pool_ready[dev]) {
    cudaMemPoolProps props;
    memset(&props, 0, sizeof(props));
    props.allocType = cudaMemAllocationTypePinned;
    props.handleTypes = cudaMemHandleTypeNone;
    props.location.type = cudaMemLocationTypeDevice;
    props.location.id = dev;
    cudaMemPool_t pool = nullptr;
    if (cudaMemPoolCreate(&pool, &props) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    unsigned long long keep = ~0ull;
    cudaMemPoolSetAttribute(pool, cudaMemPoolAttrReleaseThreshold, &keep);
    g_pool[dev] = pool;
    g_pool_ready[dev] = true;
  }
  return g_pool[dev];
}

extern "C" gear_status gear_release_workspace(void) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceSynchronize() != cudaSuccess) { cudaGetLastError(); return GEAR_ERR_CUDA; }
  std::lock_guard<std::mutex> lock(g_pool_mutex);
  if (dev >= 0 && dev < 64 && g_pool_ready[dev] && cudaMemPoolTrimTo(g_pool[dev], 0) != cudaSuccess) {
    cudaGetLastError();
    return GEAR_ERR_CUDA;
  }
  return GEAR_OK;
}

// Device memory of the caches comes from cudaMalloc unless the caller installed a pair of its own (gear_set_allocator).
static std::mutex g_alloc_mutex;
static gear_alloc_fn g_alloc = nullptr;
static gear_free_fn g_free = nullptr;
static void* g_alloc_ctx = nullptr;

extern "C" gear_status gear_set_allocator(gear_alloc_fn alloc_fn, gear_free_fn free_fn, void* ctx) {
  if ((alloc_fn == nullptr) != (free_fn == nullptr)) return GEAR_ERR_ARG;
  std::lock_guard<std::mutex> lock(g_alloc_mutex);
  g_alloc = alloc_fn; g_free = free_fn; g_alloc_ctx = ctx;
  return GEAR_OK;
}

struct DeviceAllocator {       // the pair a cache was created with (it frees through the same pair)
  gear_alloc_fn alloc; gear_free_fn free; void* ctx;
  void* get(size_t bytes) const {
    if (alloc) return alloc(bytes, ctx);
    void* p = nullptr;
    if (cudaMalloc(&p, bytes) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    return p;
  }
  void put(void* p) const {
    if (!p) return;
    if (free) free(p, ctx); else cudaFree(p);
  }
};

struct gear_cache {
  DeviceAllocator mem;
  gear_config cfg;
  CacheConst cc;
  int device;
  int sm_count;
  int G;                         // query heads per kv head
  int k_k_full;                  // outliers per side for a key group of length g
  // device memory
  unsigned char* arena; size_t arena_bytes; size_t arena_used;
  float* dbg; size_t dbg_bytes; size_t dbg_used;        // fp32 factor copies (GEAR_FLAG_KEEP_FP32_FACTORS)
  SegDesc* table_dev; int table_cap;
  int* blk2seg; int blk_cap;                             // segment index of every compressed block
  void* buf_k; void* buf_v;                              // [BH][n_b][128] fp16
  unsigned char* flush_ws; size_t flush_ws_bytes;
  float* partial; size_t partial_bytes; int max_parts;
  int* tickets; int* status;
  void* stage_k; void* stage_v; void* stage_q; float* stage_out; float* stage_b0;   // for the *_host calls
  // gear_append_buffer_host: pinned copies of the caller's rows, so that the call neither waits for the device nor
  // holds on to the caller's memory.  A slot is reused once the copy that read it has finished (its event).
  static constexpr int kHostSlots = 4;
  unsigned char* host_ring[kHostSlots]; cudaEvent_t host_ev[kHostSlots]; bool host_used[kHostSlots]; int host_next;
  // The host-buffer entry points copy on a stream of the cache's own, tied to the caller's stream by events, so that
  // the copies of one cache run beside the kernels of another that shares the caller's stream.
  cudaStream_t copy_st;
  cudaEvent_t ev_rows_up, ev_rows_used, ev_q_up, ev_attn_done, ev_out_down;
  // host state
  std::vector<SegDesc> segs;
  std::vector<long long> dbgA_off, dbgB_off;             // float offsets into dbg (or -1)
  int buf_len;
  long long n_compressed;
  int n_blocks_c;
  // cached launch plan of the decode kernel (depends on the segments' shapes)
  int plan_key, plan_occ;
  DecodeArgs plan;
  int test_dead_wait;            // gear_test_dead_wait: the next decode calls wait on a barrier nothing completes
  int max_queries, units_alloc;  // query rows per head the scratch was sized for; units of that size
  // the last call that wrote the cache (records, descriptors, buffer rows): its stream and its number on that stream
  cudaStream_t write_stream; unsigned long long write_call; bool written;
};

static int outlier_count(float s_pct, int len) {
  const long long s_units = llroundf(s_pct * 10000.0f);
  return (int)((s_units * len + 1999999LL) / 2000000LL);
}

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

static gear_status check_config(const gear_config* c) {
  if (!c) return GEAR_ERR_ARG;
  if (c->batch < 1 || c->n_kv_heads < 1 || c->n_q_heads < 1 || c->max_tokens < 16) return GEAR_ERR_ARG;
  if (c->n_q_heads % c->n_kv_heads) return GEAR_ERR_SHAPE;
  if (c->head_dim != kHeadDim) return GEAR_ERR_SHAPE;
  if (c->bits != 2 && c->bits != 4) return GEAR_ERR_ARG;
  const bool per_vector = c->group == GEAR_GROUP_PER_VECTOR;
  if (!per_vector && c->group != 16 && c->group != 32 && c->group != 64 && c->group != 128) return GEAR_ERR_ARG;
  if (!(c->outlier_pct >= 0.f) || c->outlier_pct > 10.f) return GEAR_ERR_ARG;
  if (c->buffer_cap < 16 || c->buffer_cap % 4 || c->buffer_cap > 1024) return GEAR_ERR_ARG;
  if (per_vector ? c->buffer_cap > 128 : (c->buffer_cap > c->group && c->buffer_cap % c->group)) return GEAR_ERR_SHAPE;
  // a capacity that is not a multiple of 16 (the paper's n_b = 20): the flushed buffer must be a single block
  if (c->buffer_cap % 16 && !per_vector && c->buffer_cap > c->group) return GEAR_ERR_SHAPE;
  if (c->rank_flush < 0 || c->rank_flush > kMaxRank || c->rank_max < 0 || c->rank_max > kMaxRank) return GEAR_ERR_ARG;
  if (c->rank_flush > c->rank_max) return GEAR_ERR_ARG;
  if (c->rank_flush > c->buffer_cap) return GEAR_ERR_SHAPE;
  if (c->max_queries > 64) return GEAR_ERR_ARG;
  if (c->power_iters < 1 || c->power_iters > 64) return GEAR_ERR_ARG;
  const int gv = per_vector || c->group > kHeadDim ? kHeadDim : c->group;
  const int kv = outlier_count(c->outlier_pct, gv);
  if (kv > kMaxOutliers || (kv > 0 && 2 * kv >= gv)) return GEAR_ERR_SHAPE;
  const int tf = per_vector || c->buffer_cap < c->group ? c->buffer_cap : c->group;
  const int kf = outlier_count(c->outlier_pct, tf);
  if (kf > kMaxOutliers || (kf > 0 && 2 * kf >= tf)) return GEAR_ERR_SHAPE;
  return GEAR_OK;
}

static SegDesc shape_segment(const gear_cache* c, int n_c, int rank) {
  SegDesc s;
  memset(&s, 0, sizeof(s));
  s.n_c = n_c;
  s.rank = rank;
  if (c->cfg.group == GEAR_GROUP_PER_VECTOR && n_c > 128) {
    // one key group per channel over the whole segment: 64-token record blocks without outlier slots, the
    // outliers in a list behind the records (csr_base16 is set when the segment is placed)
    s.T = 64;
    s.k_k = 0;
    s.csr_k = 2 * outlier_count(c->cfg.outlier_pct, n_c);
    s.csr_base16 = 1;
  } else {
    s.T = c->cfg.group == GEAR_GROUP_PER_VECTOR || n_c < c->cfg.group ? n_c : c->cfg.group;
    s.k_k = outlier_count(c->cfg.outlier_pct, s.T);
  }
  layout_segment(s, c->cc);
  return s;
}

extern "C" void gear_free(gear_cache* c) {
  if (!c) return;
  if (c->copy_st) cudaStreamSynchronize(c->copy_st);      // copies queued by the host-buffer calls still use the staging rows
  const DeviceAllocator& m = c->mem;
  m.put(c->arena); m.put(c->dbg); m.put(c->table_dev); m.put(c->blk2seg); m.put(c->buf_k); m.put(c->buf_v);
  m.put(c->flush_ws); m.put(c->partial); m.put(c->tickets); m.put(c->status);
  m.put(c->stage_k); m.put(c->stage_out); m.put(c->stage_b0);
  for (int i = 0; i < gear_cache::kHostSlots; ++i) {
    if (c->host_ring[i]) cudaFreeHost(c->host_ring[i]);
    if (c->host_ev[i]) cudaEventDestroy(c->host_ev[i]);
  }
  cudaEvent_t* evs[5] = {&c->ev_rows_up, &c->ev_rows_used, &c->ev_q_up, &c->ev_attn_done, &c->ev_out_down};
  for (cudaEvent_t* e : evs)
    if (*e) cudaEventDestroy(*e);
  if (c->copy_st) cudaStreamDestroy(c->copy_st);
  delete c;
}

#define GEAR_TRY_ALLOC(ptr, bytes)                                                   \
  do {                                                                               \
    *reinterpret_cast<void**>(&(ptr)) = c->mem.get(bytes);                           \
    if ((ptr) == nullptr) {                                                          \
      gear_free(c);                                                                  \
      return GEAR_ERR_ALLOC;                                                         \
    }                                                                                \
  } while (0)

extern "C" gear_status gear_create(gear_cache** out, const gear_config* cfg) {
  if (!out || *out) return GEAR_ERR_ARG;
  gear_status st = check_config(cfg);
  if (st != GEAR_OK) return st;
  gear_cache* c = new (std::nothrow) gear_cache();
  if (!c) return GEAR_ERR_ALLOC;
  c->cfg = *cfg;
  {
    std::lock_guard<std::mutex> lock(g_alloc_mutex);
    c->mem.alloc = g_alloc; c->mem.free = g_free; c->mem.ctx = g_alloc_ctx;
  }
  c->test_dead_wait = 0;
  c->write_stream = nullptr; c->write_call = 0; c->written = false;
  c->arena = nullptr; c->dbg = nullptr; c->table_dev = nullptr; c->blk2seg = nullptr; c->buf_k = c->buf_v = nullptr; c->flush_ws = nullptr;
  c->partial = nullptr; c->tickets = nullptr; c->status = nullptr;
  c->stage_k = c->stage_v = c->stage_q = nullptr; c->stage_out = nullptr; c->stage_b0 = nullptr;
  for (int i = 0; i < gear_cache::kHostSlots; ++i) { c->host_ring[i] = nullptr; c->host_ev[i] = nullptr; c->host_used[i] = false; }
  c->host_next = 0;
  c->copy_st = nullptr;
  c->ev_rows_up = c->ev_rows_used = c->ev_q_up = c->ev_attn_done = c->ev_out_down = nullptr;
  c->cc.bits = cfg->bits;
  c->cc.g_v = cfg->group == GEAR_GROUP_PER_VECTOR || cfg->group > kHeadDim ? kHeadDim : cfg->group;
  c->cc.ngv = kHeadDim / c->cc.g_v;
  c->cc.k_v = outlier_count(cfg->outlier_pct, c->cc.g_v);
  c->cc.BH = cfg->batch * cfg->n_kv_heads;
  c->cc.n_b = cfg->buffer_cap;
  c->G = cfg->n_q_heads / cfg->n_kv_heads;
  c->buf_len = 0; c->n_compressed = 0; c->n_blocks_c = 0; c->plan_key = -1;
  if (cudaGetDevice(&c->device) != cudaSuccess ||
      cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, c->device) != cudaSuccess) {
    delete c;
    return GEAR_ERR_CUDA;
  }
  const size_t BH = c->cc.BH;
  // arena: worst bytes per token over the two segment shapes the cache can see (full groups at rank_max,
  // flushed buffers at rank_flush), plus the per-segment B factors
  const int n_b = cfg->buffer_cap;
  const bool per_vector = cfg->group == GEAR_GROUP_PER_VECTOR;
  SegDesc sp = shape_segment(c, per_vector ? 192 : cfg->group, cfg->rank_max);
  SegDesc sf = shape_segment(c, n_b, cfg->rank_flush);
  const double dens_p = (double)sp.rec_bytes / sp.T, dens_f = (double)sf.rec_bytes / sf.T;
  const double dens = dens_p > dens_f ? dens_p : dens_f;
  const size_t n_flush_max = (size_t)(cfg->max_tokens / n_b) + 1;
  size_t per_bh = (size_t)(dens * (double)cfg->max_tokens) + n_flush_max * sf.bfac_bytes + 8 * (size_t)sp.bfac_bytes +
                  16 * (size_t)(sp.rec_bytes > sf.rec_bytes ? sp.rec_bytes : sf.rec_bytes);
  if (per_vector)      // outlier lists of per-vector key segments: offsets per block, entries per channel (rounded up per segment)
    per_bh += (size_t)(cfg->max_tokens / 64 + 8) * 4 + 64 * 16 +
              (size_t)kHeadDim * 4 * (2 * (size_t)outlier_count(cfg->outlier_pct, (int)cfg->max_tokens) + 2 * 8);
  c->arena_bytes = align_up(per_bh, 256) * BH + 4096;
  c->arena_used = 0;
  GEAR_TRY_ALLOC(c->arena, c->arena_bytes);
  c->table_cap = (int)(cfg->max_tokens / 16 + 8);
  GEAR_TRY_ALLOC(c->table_dev, sizeof(SegDesc) * (size_t)c->table_cap);
  c->blk_cap = (int)(cfg->max_tokens / 16 + 8);
  GEAR_TRY_ALLOC(c->blk2seg, sizeof(int) * (size_t)c->blk_cap);
  GEAR_TRY_ALLOC(c->buf_k, BH * n_b * kHeadDim * 2);
  GEAR_TRY_ALLOC(c->buf_v, BH * n_b * kHeadDim * 2);
  c->flush_ws_bytes = compress_workspace_bytes((int)BH, n_b, cfg->rank_flush);
  GEAR_TRY_ALLOC(c->flush_ws, c->flush_ws_bytes);
  if (cfg->flags & GEAR_FLAG_KEEP_FP32_FACTORS) {
    const size_t rm = cfg->rank_max > 0 ? cfg->rank_max : 1;
    c->dbg_bytes = (BH * 2 * (size_t)cfg->max_tokens * rm + BH * 2 * kHeadDim * rm * (size_t)c->table_cap) * 4;
    c->dbg_used = 0;
    GEAR_TRY_ALLOC(c->dbg, c->dbg_bytes);
  }
  // decode scratch: one partial per (unit, warp touching it); upper bound of warps in a launch
  // scratch for the largest group of query rows a call may bring: G query heads x max_queries rows per kv head
  c->max_queries = cfg->max_queries > 1 ? (int)cfg->max_queries : 1;
  const int hp = decode_heads_per_pass(c->G * c->max_queries);
  const int passes = decode_passes(c->G * c->max_queries);
  c->units_alloc = (int)(BH * passes);
  const size_t units = BH * passes;
  const size_t nw_max = (size_t)c->sm_count * 32;        // one warp per CTA, at most 32 CTAs per SM
  c->max_parts = (int)(nw_max / units + 3);
  c->partial_bytes = units * c->max_parts * (size_t)hp * kPartRow * 4;
  GEAR_TRY_ALLOC(c->partial, c->partial_bytes);
  GEAR_TRY_ALLOC(c->tickets, units * 4);
  GEAR_TRY_ALLOC(c->status, 4);
  cudaMemset(c->tickets, 0, units * 4);
  cudaMemset(c->status, 0, 4);
  const size_t tok_bytes = BH * kHeadDim * 2;
  // key row, value row, query: one copy can bring all three (gear_step_host)
  const size_t q_bytes = (size_t)cfg->batch * cfg->n_q_heads * kHeadDim * 2;
  GEAR_TRY_ALLOC(c->stage_k, 2 * tok_bytes + q_bytes);
  c->stage_v = reinterpret_cast<unsigned char*>(c->stage_k) + tok_bytes;
  c->stage_q = reinterpret_cast<unsigned char*>(c->stage_k) + 2 * tok_bytes;
  for (int i = 0; i < gear_cache::kHostSlots; ++i) {
    if (cudaHostAlloc((void**)&c->host_ring[i], 2 * tok_bytes + q_bytes, cudaHostAllocDefault) != cudaSuccess ||
        cudaEventCreateWithFlags(&c->host_ev[i], cudaEventDisableTiming) != cudaSuccess) {
      cudaGetLastError();
      gear_free(c);
      return GEAR_ERR_ALLOC;
    }
  }
  {
    cudaEvent_t* evs[5] = {&c->ev_rows_up, &c->ev_rows_used, &c->ev_q_up, &c->ev_attn_done, &c->ev_out_down};
    bool ok = cudaStreamCreateWithFlags(&c->copy_st, cudaStreamNonBlocking) == cudaSuccess;
    for (cudaEvent_t* e : evs) ok = ok && cudaEventCreateWithFlags(e, cudaEventDisableTiming) == cudaSuccess;
    if (!ok) {
      cudaGetLastError();
      gear_free(c);
      return GEAR_ERR_ALLOC;
    }
  }
  GEAR_TRY_ALLOC(c->stage_out, (size_t)cfg->batch * cfg->n_q_heads * kHeadDim * 4);
  GEAR_TRY_ALLOC(c->stage_b0, BH * 2 * kHeadDim * (size_t)(cfg->rank_flush > 0 ? cfg->rank_flush : 1) * 4);
  if (cudaDeviceSynchronize() != cudaSuccess) { gear_free(c); return GEAR_ERR_CUDA; }
  *out = c;
  return GEAR_OK;
}

// Append one compressed segment built from K, V [BH][n][128] on the device.
static gear_status compress_segment(gear_cache* c, const void* K, const void* V, int n, int rank, const float* B0,
                                    bool is_flush, cudaStream_t st) {
  if ((int)c->segs.size() >= c->table_cap) return GEAR_ERR_CAPACITY;
  if (c->n_compressed + n > c->cfg.max_tokens) return GEAR_ERR_CAPACITY;
  SegDesc sd = shape_segment(c, n, rank);
  if (c->n_blocks_c + sd.nblk > c->blk_cap) return GEAR_ERR_CAPACITY;
  if (sd.k_k > kMaxOutliers || (sd.k_k > 0 && 2 * sd.k_k >= sd.T)) return GEAR_ERR_SHAPE;
  size_t need = align_up((size_t)sd.bh_stride, 16) * c->cc.BH;
  sd.bh_stride = (long long)align_up((size_t)sd.bh_stride, 16);
  const bool per_vector = sd.csr_base16 != 0;
  if (per_vector) {
    if (!kcvt_fits(n) || sd.csr_k >= n || (need >> 4) > 0xFFFFFFFFull) return GEAR_ERR_SHAPE;
    sd.csr_base16 = (unsigned int)(need >> 4);
    need += align_up((size_t)csr_stride_bytes(sd.nblk, sd.csr_k) * c->cc.BH, 16);
  }
  if (c->arena_used + need > c->arena_bytes) return GEAR_ERR_CAPACITY;
  sd.seg_base = (long long)c->arena_used;
  sd.tok_start = (int)c->n_compressed;
  sd.blk_start = c->n_blocks_c;
  sd.dbg_base = -1;
  sd.shape_id = static_shape_id(sd, c->cc);
  float* dbgA = nullptr; float* dbgB = nullptr;
  long long offA = -1, offB = -1;
  if (c->dbg && rank > 0) {
    const size_t nA = (size_t)c->cc.BH * 2 * n * rank, nB = (size_t)c->cc.BH * 2 * kHeadDim * rank;
    if ((c->dbg_used + nA + nB) * 4 > c->dbg_bytes) return GEAR_ERR_CAPACITY;
    offA = (long long)c->dbg_used; offB = offA + (long long)nA;
    dbgA = c->dbg + offA; dbgB = c->dbg + offB;
  }
  CompressJob job;
  job.seg = sd; job.cc = c->cc; job.arena = c->arena;
  job.K = (const __half*)K; job.V = (const __half*)V; job.B0 = B0;
  job.dbgA = dbgA; job.dbgB = dbgB;
  job.seed = c->cfg.seed; job.segment_index = (int)c->segs.size(); job.iters = c->cfg.power_iters;

  cudaError_t e = cudaSuccess;
  if (sd.T % 16) {     // the last slab of every block is partly empty: its codes, factor rows and scales read as zero
    if (cudaMemsetAsync(c->arena + sd.seg_base, 0, need, st) != cudaSuccess) { cudaGetLastError(); return GEAR_ERR_CUDA; }
    if (!compress_tile_fits(sd.T, sd.n_c, sd.rank)) return GEAR_ERR_SHAPE;
  }
  if (!per_vector && compress_tile_fits(sd.T, sd.n_c, sd.rank)) {
    e = compress_tile(job, c->cc.BH, st);              // short segment: one launch, residual in shared memory
  } else if (is_flush) {
    e = compress_range(job, 0, c->cc.BH, c->flush_ws, st);
  } else {
    // bounded transient workspace, (batch, head) pairs processed in ranges
    const int csr_k = per_vector ? sd.csr_k : -1;
    const size_t per_bh = compress_workspace_bytes(1, n, rank, csr_k);
    const size_t budget = (size_t)3 << 30;
    int chunk = (int)(budget / per_bh);
    if (chunk < 1) chunk = 1;
    if (chunk > c->cc.BH) chunk = c->cc.BH;
    unsigned char* ws = nullptr;
    const size_t ws_bytes = compress_workspace_bytes(chunk, n, rank, csr_k);
    cudaMemPool_t pool = workspace_pool(c->device);
    if (pool == nullptr || cudaMallocFromPoolAsync((void**)&ws, ws_bytes, pool, st) != cudaSuccess) {
      cudaGetLastError();
      return GEAR_ERR_ALLOC;
    }
    for (int bh0 = 0; bh0 < c->cc.BH && e == cudaSuccess; bh0 += chunk) {
      const int nbh = bh0 + chunk <= c->cc.BH ? chunk : c->cc.BH - bh0;
      e = compress_range(job, bh0, nbh, ws, st);
    }
    cudaFreeAsync(ws, st);
  }
  if (e != cudaSuccess) { cudaGetLastError(); return GEAR_ERR_CUDA; }
  e = launch_write_desc(c->table_dev, c->blk2seg, (int)c->segs.size(), sd, st);
  if (e != cudaSuccess) { cudaGetLastError(); return GEAR_ERR_CUDA; }
  c->segs.push_back(sd);
  c->dbgA_off.push_back(offA); c->dbgB_off.push_back(offB);
  if (offA >= 0) c->dbg_used += (size_t)c->cc.BH * 2 * n * rank + (size_t)c->cc.BH * 2 * kHeadDim * rank;
  c->arena_used += need;
  c->n_compressed += n;
  c->n_blocks_c += sd.nblk;
  c->plan_key = -1;
  c->write_stream = st; c->write_call = next_call_number(st); c->written = true;
  return GEAR_OK;
}

extern "C" gear_status gear_compress(gear_cache** cache, const gear_config* cfg, const void* K, const void* V,
                                     int64_t n, int32_t rank, const float* B0, void* stream) {
  if (!cache || !K || !V) return GEAR_ERR_ARG;
  if (((uintptr_t)K | (uintptr_t)V) & 15) return GEAR_ERR_ALIGN;
  const gear_config* use = *cache ? &(*cache)->cfg : cfg;
  if (!use) return GEAR_ERR_ARG;
  gear_status st = check_config(use);
  if (st != GEAR_OK) return st;
  if (n < 16 || n % 16 || n > (1 << 30)) return GEAR_ERR_SHAPE;
  if (use->group == GEAR_GROUP_PER_VECTOR ? (n > 128 && n % 64) : (n >= use->group && n % use->group)) return GEAR_ERR_SHAPE;
  if (rank < 0 || rank > use->rank_max || rank > n) return GEAR_ERR_ARG;
  bool created = false;
  if (!*cache) {
    st = gear_create(cache, cfg);
    if (st != GEAR_OK) return st;
    created = true;
  }
  gear_cache* c = *cache;
  if (c->buf_len != 0) return GEAR_ERR_STATE;
  st = compress_segment(c, K, V, (int)n, rank, B0, false, (cudaStream_t)stream);
  if (st != GEAR_OK && created) { gear_free(c); *cache = nullptr; }
  return st;
}

extern "C" gear_status gear_append_buffer(gear_cache* c, const void* k_new, const void* v_new, const float* B0_flush,
                                          void* stream) {
  if (!c || !k_new || !v_new) return GEAR_ERR_ARG;
  if (((uintptr_t)k_new | (uintptr_t)v_new) & 15) return GEAR_ERR_ALIGN;
  cudaStream_t st = (cudaStream_t)stream;
  const int n_b = c->cfg.buffer_cap;
  if (c->buf_len + 1 == n_b) {     // this push will flush: make sure the segment fits before touching anything
    if (c->n_compressed + n_b > c->cfg.max_tokens || (int)c->segs.size() >= c->table_cap) return GEAR_ERR_CAPACITY;
  }
  if (launch_append(c->buf_k, c->buf_v, k_new, v_new, c->cc.BH, n_b, c->buf_len, st) != cudaSuccess) {
    cudaGetLastError();
    return GEAR_ERR_CUDA;
  }
  c->buf_len += 1;
  c->plan_key = -1;
  c->write_stream = st; c->write_call = next_call_number(st); c->written = true;
  if (c->buf_len < n_b) return GEAR_OK;
  gear_status s = compress_segment(c, c->buf_k, c->buf_v, n_b, c->cfg.rank_flush, B0_flush, true, st);
  if (s != GEAR_OK) { c->buf_len -= 1; return s; }
  c->buf_len = 0;
  return GEAR_FLUSHED;
}

static gear_status plan_decode(gear_cache* c, int Gq) {
  const int key = (int)c->segs.size() * 4096 + Gq;
  if (c->plan_key == key) return GEAR_OK;
  // One-head passes: with four warps per scheduler the warps of a scheduler slow one another down by more than
  // the fourth warp adds (measured: 3 warps finish 0.85 blocks per microsecond and scheduler, 4 warps 0.79), so
  // long streams run with twelve resident warps.  Short streams (few blocks per warp) keep sixteen: there the
  // fixed cost per warp and the granularity of the split weigh more.
  int warps_cap = 0;
  if (Gq == 1) {
    const long long blocks = (long long)c->cc.BH * (c->n_blocks_c + (c->buf_len + 15) / 16);
    if (blocks >= 24LL * 16 * c->sm_count) warps_cap = 12;
  }
  int max_k = 0, max_v = 0, max_bfac = 0, max_T = 16;
  for (const SegDesc& s : c->segs) {
    if (s.off_vpart > max_k) max_k = s.off_vpart;
    if (s.rec_bytes - s.off_vpart > max_v) max_v = s.rec_bytes - s.off_vpart;
    if (s.bfac_bytes > max_bfac) max_bfac = s.bfac_bytes;
    if ((s.T + 31) / 32 * 32 > max_T) max_T = (s.T + 31) / 32 * 32;
  }
  if (!decode_plan(c->cc.bits, Gq, c->cc.ngv, max_k, max_v, max_bfac, max_T, 227 * 1024, warps_cap, &c->plan))
    return GEAR_ERR_SHAPE;
  const int occ = decode_occupancy(c->cc.bits, Gq, c->cc.ngv, c->plan.wide, (size_t)c->plan.ws.total);
  if (occ < 1) return GEAR_ERR_CUDA;
  c->plan_occ = occ;
  c->plan_key = key;
  return GEAR_OK;
}

// Decode attention for Gq query rows per kv head: q, out [B][H][Gq][128] (Gq = G for one query per head).
static gear_status decode_rows(gear_cache* c, const void* q, float* out, int Gq, float softmax_scale, void* stream) {
  if (!c || !q || !out) return GEAR_ERR_ARG;
  if (((uintptr_t)q | (uintptr_t)out) & 15) return GEAR_ERR_ALIGN;
  if (c->n_compressed == 0 && c->buf_len == 0) return GEAR_ERR_STATE;
  gear_status s = plan_decode(c, Gq);
  if (s != GEAR_OK) return s;
  DecodeArgs a = c->plan;
  a.arena = c->arena; a.table = c->table_dev; a.blk2seg = c->blk2seg;
  a.buf_k = (const __half*)c->buf_k; a.buf_v = (const __half*)c->buf_v;
  a.q = (const __half*)q; a.out = out; a.partial = c->partial; a.tickets = c->tickets; a.status = c->status;
  a.cc = c->cc; a.n_blocks_c = c->n_blocks_c; a.buf_len = c->buf_len;
  a.n_kv_heads = c->cfg.n_kv_heads; a.group_heads = Gq;
  const float sc = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)kHeadDim);
  a.scale_log2 = sc * 1.4426950408889634f;
  a.test_dead_wait = c->test_dead_wait;
  {
    const unsigned long long call = next_call_number((cudaStream_t)stream);
    a.early_reads = c->written && c->write_stream == (cudaStream_t)stream && call >= c->write_call + 2 ? 1 : 0;
  }
  // one warp per CTA; never more warps than blocks of work
  const int passes = decode_passes(Gq);
  if ((long long)c->cc.BH * passes > c->units_alloc) return GEAR_ERR_CAPACITY;
  // partial slots per unit for this call's unit count (the scratch was sized for the most units: fewer units get more
  // slots each out of the same memory)
  a.max_parts = (int)((size_t)c->sm_count * 32 / ((size_t)c->cc.BH * passes) + 3);
  if ((size_t)c->cc.BH * passes * a.max_parts * decode_heads_per_pass(Gq) * kPartRow * 4 > c->partial_bytes)
    return GEAR_ERR_CAPACITY;
  const long long work = (long long)c->cc.BH * passes * (c->n_blocks_c + (c->buf_len + 15) / 16);
  long long grid = (long long)c->sm_count * c->plan_occ;
  if (grid > work) grid = work;
  // With few blocks per warp, a warp that runs from one unit into the next pays a second prologue and epilogue and
  // finishes last.  When every unit gets at least six warps, cut each unit into ranges of its own instead: the first
  // units into one range more than the others so that every resident warp has work, and order the CTAs by the length
  // of their range, longest first (the hardware dispatches them in index order, and the oldest warps of an SM
  // finish first).  Otherwise (many blocks per warp) cut the flat space evenly.
  {
    const long long units = (long long)c->cc.BH * passes, nb = work / units;
    const long long pb = grid / units, ua = grid - pb * units;         // ua units get pb + 1 ranges
    if (pb >= 6 && pb + 1 <= nb && pb + 1 < a.max_parts) {
      a.aligned = 1;
      a.units_a = (int)ua; a.parts_a = (int)pb + 1; a.parts_b = (int)pb;
      struct Cls { int len, u0, nu, p0, n; } cls[4];
      const int base_a = (int)(nb / (pb + 1)), rem_a = (int)(nb % (pb + 1));
      const int base_b = (int)(nb / pb), rem_b = (int)(nb % pb);
      cls[0] = {base_b + 1, (int)ua, (int)(units - ua), 0, rem_b};
      cls[1] = {base_b, (int)ua, (int)(units - ua), rem_b, (int)pb - rem_b};
      cls[2] = {base_a + 1, 0, (int)ua, 0, rem_a};
      cls[3] = {base_a, 0, (int)ua, rem_a, (int)pb + 1 - rem_a};
      for (int i = 1; i < 4; ++i)                                       // insertion sort, longest first, stable
        for (int j = i; j > 0 && cls[j].len > cls[j - 1].len; --j) { const Cls t = cls[j]; cls[j] = cls[j - 1]; cls[j - 1] = t; }
      int start = 0;
      for (int k = 0; k < 4; ++k) {
        a.cls_start[k] = start; a.cls_u0[k] = cls[k].u0; a.cls_n[k] = cls[k].n > 0 ? cls[k].n : 1; a.cls_p0[k] = cls[k].p0;
        start += cls[k].nu * cls[k].n;
      }
      a.cls_start[4] = start;
      grid = start;                                                     // = units * pb + ua
    }
  }
  if (launch_decode(a, (int)grid, (cudaStream_t)stream) != cudaSuccess) {
    cudaGetLastError();
    return GEAR_ERR_CUDA;
  }
  return GEAR_OK;
}

extern "C" gear_status gear_decode_attn(gear_cache* c, const void* q, float* out, float softmax_scale, void* stream) {
  if (!c) return GEAR_ERR_ARG;
  return decode_rows(c, q, out, c->G, softmax_scale, stream);
}

extern "C" gear_status gear_decode_attn_multi(gear_cache* c, const void* q, float* out, int32_t n_queries,
                                              float softmax_scale, void* stream) {
  if (!c) return GEAR_ERR_ARG;
  if (n_queries < 1 || n_queries > c->max_queries) return GEAR_ERR_ARG;
  // The rows of one kv head -- its G query heads times n_queries positions -- are consecutive in q and out, and every
  // row attends to the whole cache: to the kernel they are G * n_queries query heads of that kv head.
  return decode_rows(c, q, out, c->G * n_queries, softmax_scale, stream);
}

extern "C" gear_status gear_append_buffer_host(gear_cache* c, const void* k_host, const void* v_host,
                                               const float* B0_host, void* stream) {
  if (!c || !k_host || !v_host) return GEAR_ERR_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  const size_t tok_bytes = (size_t)c->cc.BH * kHeadDim * 2;
  // the rows go through a pinned slot of the library's own, so the caller's memory is free again on return and
  // nothing waits for the device (a slot is waited for only if its copy of four calls ago is still running)
  const int slot = c->host_next;
  c->host_next = (slot + 1) % gear_cache::kHostSlots;
  if (c->host_used[slot] && cudaEventSynchronize(c->host_ev[slot]) != cudaSuccess) { cudaGetLastError(); return GEAR_ERR_CUDA; }
  memcpy(c->host_ring[slot], k_host, tok_bytes);
  memcpy(c->host_ring[slot] + tok_bytes, v_host, tok_bytes);
  // copy stream: after the previous push has read the staging rows; caller's stream: after the copy
  if (cudaStreamWaitEvent(c->copy_st, c->ev_rows_used, 0) != cudaSuccess ||
      cudaMemcpyAsync(c->stage_k, c->host_ring[slot], 2 * tok_bytes, cudaMemcpyHostToDevice, c->copy_st) != cudaSuccess ||
      cudaEventRecord(c->host_ev[slot], c->copy_st) != cudaSuccess ||
      cudaEventRecord(c->ev_rows_up, c->copy_st) != cudaSuccess ||
      cudaStreamWaitEvent(st, c->ev_rows_up, 0) != cudaSuccess) {
    cudaGetLastError();
    return GEAR_ERR_CUDA;
  }
  c->host_used[slot] = true;
  const float* b0 = nullptr;
  const bool with_b0 = B0_host && c->cfg.rank_flush > 0 && c->buf_len + 1 == c->cfg.buffer_cap;
  if (with_b0) {
    if (cudaMemcpyAsync(c->stage_b0, B0_host, (size_t)c->cc.BH * 2 * kHeadDim * c->cfg.rank_flush * 4,
                        cudaMemcpyHostToDevice, st) != cudaSuccess) {
      cudaGetLastError();
      return GEAR_ERR_CUDA;
    }
    b0 = c->stage_b0;
  }
  gear_status s = gear_append_buffer(c, c->stage_k, c->stage_v, b0, stream);
  if (s < 0) return s;
  if (cudaEventRecord(c->ev_rows_used, st) != cudaSuccess) { cudaGetLastError(); return GEAR_ERR_CUDA; }
  // the start vectors are read straight from the caller's memory: only then wait for the copy
  if (with_b0 && cudaStreamSynchronize(st) != cudaSuccess) { cudaGetLastError(); return GEAR_ERR_CUDA; }
  return s;
}

static gear_status decode_host(gear_cache* c, const void* q_host, float* out_host, float softmax_scale, void* stream,
                               bool wait) {
  if (!c || !q_host || !out_host) return GEAR_ERR_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  const size_t nq = (size_t)c->cfg.batch * c->cfg.n_q_heads * kHeadDim;
  // query up on the copy stream once the previous call's kernel has read the staging query; the kernel after that
  // copy and after the previous call's result has left the staging output
  if (cudaStreamWaitEvent(c->copy_st, c->ev_attn_done, 0) != cudaSuccess ||
      cudaMemcpyAsync(c->stage_q, q_host, nq * 2, cudaMemcpyHostToDevice, c->copy_st) != cudaSuccess ||
      cudaEventRecord(c->ev_q_up, c->copy_st) != cudaSuccess ||
      cudaStreamWaitEvent(st, c->ev_q_up, 0) != cudaSuccess ||
      cudaStreamWaitEvent(st, c->ev_out_down, 0) != cudaSuccess) {
    cudaGetLastError();
    return GEAR_ERR_CUDA;
  }
  gear_status s = gear_decode_attn(c, c->stage_q, c->stage_out, softmax_scale, stream);
  if (s != GEAR_OK) return s;
  if (cudaEventRecord(c->ev_attn_done, st) != cudaSuccess ||
      cudaStreamWaitEvent(c->copy_st, c->ev_attn_done, 0) != cudaSuccess ||
      cudaMemcpyAsync(out_host, c->stage_out, nq * 4, cudaMemcpyDeviceToHost, c->copy_st) != cudaSuccess ||
      cudaEventRecord(c->ev_out_down, c->copy_st) != cudaSuccess ||
      (wait && cudaStreamSynchronize(c->copy_st) != cudaSuccess)) {
    cudaGetLastError();
    return GEAR_ERR_CUDA;
  }
  return GEAR_OK;
}

extern "C" gear_status gear_decode_attn_host(gear_cache* c, const void* q_host, float* out_host, float softmax_scale,
                                             void* stream) {
  return decode_host(c, q_host, out_host, softmax_scale, stream, true);
}

extern "C" gear_status gear_decode_attn_host_async(gear_cache* c, const void* q_host, float* out_host,
                                                   float softmax_scale, void* stream) {
  return decode_host(c, q_host, out_host, softmax_scale, stream, false);
}

// One token of one layer through host buffers: push the rows, attend, all queued.  One copy up (rows and query
// through one pinned slot), one copy down.
extern "C" gear_status gear_step_host(gear_cache* c, const void* k_host, const void* v_host, const void* q_host,
                                      float* out_host, float softmax_scale, void* stream) {
  if (!c || !k_host || !v_host || !q_host || !out_host) return GEAR_ERR_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  const size_t tok_bytes = (size_t)c->cc.BH * kHeadDim * 2;
  const size_t nq = (size_t)c->cfg.batch * c->cfg.n_q_heads * kHeadDim;
  const int slot = c->host_next;
  c->host_next = (slot + 1) % gear_cache::kHostSlots;
  if (c->host_used[slot] && cudaEventSynchronize(c->host_ev[slot]) != cudaSuccess) { cudaGetLastError(); return GEAR_ERR_CUDA; }
  memcpy(c->host_ring[slot], k_host, tok_bytes);
  memcpy(c->host_ring[slot] + tok_bytes, v_host, tok_bytes);
  memcpy(c->host_ring[slot] + 2 * tok_bytes, q_host, nq * 2);
  // copy stream: after the previous push and the previous kernel have read the staging area; caller's stream: after the
  // copy, and after the previous result has left the staging output
  if (cudaStreamWaitEvent(c->copy_st, c->ev_rows_used, 0) != cudaSuccess ||
      cudaStreamWaitEvent(c->copy_st, c->ev_attn_done, 0) != cudaSuccess ||
      cudaMemcpyAsync(c->stage_k, c->host_ring[slot], 2 * tok_bytes + nq * 2, cudaMemcpyHostToDevice, c->copy_st) != cudaSuccess ||
      cudaEventRecord(c->host_ev[slot], c->copy_st) != cudaSuccess ||
      cudaStreamWaitEvent(st, c->host_ev[slot], 0) != cudaSuccess ||
      cudaStreamWaitEvent(st, c->ev_out_down, 0) != cudaSuccess) {
    cudaGetLastError();
    return GEAR_ERR_CUDA;
  }
  c->host_used[slot] = true;
  gear_status pushed = gear_append_buffer(c, c->stage_k, c->stage_v, nullptr, stream);
  if (pushed < 0) return pushed;
  gear_status s = gear_decode_attn(c, c->stage_q, c->stage_out, softmax_scale, stream);
  if (s != GEAR_OK) return s;
  if (cudaEventRecord(c->ev_attn_done, st) != cudaSuccess ||
      cudaEventRecord(c->ev_rows_used, st) != cudaSuccess ||
      cudaStreamWaitEvent(c->copy_st, c->ev_attn_done, 0) != cudaSuccess ||
      cudaMemcpyAsync(out_host, c->stage_out, nq * 4, cudaMemcpyDeviceToHost, c->copy_st) != cudaSuccess ||
      cudaEventRecord(c->ev_out_down, c->copy_st) != cudaSuccess) {
    cudaGetLastError();
    return GEAR_ERR_CUDA;
  }
  return pushed;
}

extern "C" gear_status gear_cache_wait(gear_cache* c) {
  if (!c) return GEAR_ERR_ARG;
  if (cudaStreamSynchronize(c->copy_st) != cudaSuccess) {
    cudaGetLastError();
    return GEAR_ERR_CUDA;
  }
  return GEAR_OK;
}

extern "C" gear_status gear_fp16_decode_attn(const void* K, const void* V, const void* q, float* out, int32_t batch,
                                             int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim, int64_t n,
                                             int64_t n_alloc, float softmax_scale, void* scratch, size_t scratch_bytes,
                                             void* stream) {
  if (!K || !V || !q || !out || !scratch) return GEAR_ERR_ARG;
  if (batch < 1 || n_kv_heads < 1 || n_q_heads < 1 || n < 1 || n_alloc < n) return GEAR_ERR_ARG;
  if (n_alloc > 0x7fffffffLL) return GEAR_ERR_ARG;                  // token counts travel as 32-bit integers
  if (head_dim != kHeadDim || n_q_heads % n_kv_heads) return GEAR_ERR_SHAPE;
  if (((uintptr_t)K | (uintptr_t)V | (uintptr_t)q | (uintptr_t)out | (uintptr_t)scratch) & 15) return GEAR_ERR_ALIGN;
  if (scratch_bytes < gear_fp16_attn_scratch_bytes(batch, n_q_heads, head_dim)) return GEAR_ERR_CAPACITY;
  const float sc = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)kHeadDim);
  if (launch_fp16_attn(K, V, q, out, batch, n_q_heads, n_kv_heads, n, n_alloc, sc, scratch, scratch_bytes,
                       (cudaStream_t)stream) != cudaSuccess) {
    cudaGetLastError();
    return GEAR_ERR_CUDA;
  }
  return GEAR_OK;
}

extern "C" size_t gear_fp16_attn_scratch_bytes(int32_t batch, int32_t n_q_heads, int32_t head_dim) {
  (void)head_dim;
  return fp16_attn_scratch(batch, n_q_heads);
}

// ------------------------------------------------------------------ helpers
static size_t export_elems(const gear_cache* c, const SegDesc& s, int what, size_t* elem_bytes) {
  const size_t BH = c->cc.BH, d = kHeadDim;
  switch (what) {
    case GEAR_EXP_K_CODES: case GEAR_EXP_V_CODES: *elem_bytes = 1; return BH * s.n_c * d;
    case GEAR_EXP_K_SCALE: case GEAR_EXP_K_ZERO: *elem_bytes = 2; return BH * (s.csr_base16 ? 1 : s.nblk) * d;
    case GEAR_EXP_V_SCALE: case GEAR_EXP_V_ZERO: *elem_bytes = 2; return BH * s.n_c * c->cc.ngv;
    case GEAR_EXP_K_OUT_IDX:
      if (s.csr_base16) { *elem_bytes = 4; return BH * d * s.csr_k; }      // token in the segment, 32-bit
      *elem_bytes = 1; return BH * s.nblk * d * 2 * s.k_k;
    case GEAR_EXP_K_OUT_VAL: *elem_bytes = 2; return s.csr_base16 ? BH * d * s.csr_k : BH * s.nblk * d * 2 * s.k_k;
    case GEAR_EXP_V_OUT_IDX: *elem_bytes = 1; return BH * s.n_c * c->cc.ngv * 2 * c->cc.k_v;
    case GEAR_EXP_V_OUT_VAL: *elem_bytes = 2; return BH * s.n_c * c->cc.ngv * 2 * c->cc.k_v;
    case GEAR_EXP_K_A: case GEAR_EXP_V_A: case GEAR_EXP_K_A_FP32: case GEAR_EXP_V_A_FP32:
      *elem_bytes = 4; return BH * s.n_c * s.rank;
    case GEAR_EXP_K_B: case GEAR_EXP_V_B: case GEAR_EXP_K_B_FP32: case GEAR_EXP_V_B_FP32:
      *elem_bytes = 4; return BH * d * s.rank;
    default: *elem_bytes = 0; return 0;
  }
}

extern "C" gear_status gear_export(gear_cache* c, int32_t segment, int32_t what, void* host_dst, size_t bytes) {
  if (!c || (!host_dst && bytes)) return GEAR_ERR_ARG;
  if (what == GEAR_EXP_K_BUFFER || what == GEAR_EXP_V_BUFFER) {
    const size_t row = (size_t)c->buf_len * kHeadDim * 2;
    if (bytes != row * c->cc.BH) return GEAR_ERR_ARG;
    if (row == 0) return GEAR_OK;
    const void* src = what == GEAR_EXP_K_BUFFER ? c->buf_k : c->buf_v;
    if (cudaDeviceSynchronize() != cudaSuccess ||
        cudaMemcpy2D(host_dst, row, src, (size_t)c->cfg.buffer_cap * kHeadDim * 2, row, c->cc.BH,
                     cudaMemcpyDeviceToHost) != cudaSuccess) {
      cudaGetLastError();
      return GEAR_ERR_CUDA;
    }
    return GEAR_OK;
  }
  if (segment < 0 || segment >= (int)c->segs.size()) return GEAR_ERR_ARG;
  const SegDesc& s = c->segs[segment];
  size_t eb = 0;
  const size_t n = export_elems(c, s, what, &eb);
  if (eb == 0) return GEAR_ERR_ARG;
  if (bytes != n * eb) return GEAR_ERR_ARG;
  if (n == 0) return GEAR_OK;
  if (cudaDeviceSynchronize() != cudaSuccess) { cudaGetLastError(); return GEAR_ERR_CUDA; }
  if (what >= GEAR_EXP_K_A_FP32 && what <= GEAR_EXP_V_B_FP32) {
    if (!c->dbg || c->dbgA_off[segment] < 0) return GEAR_ERR_STATE;
    // stored as [BH][2][rows][rank]; gather the side
    const int side = what & 1;
    const bool isA = what == GEAR_EXP_K_A_FP32 || what == GEAR_EXP_V_A_FP32;
    const size_t rows = isA ? (size_t)s.n_c : (size_t)kHeadDim;
    const float* base = c->dbg + (isA ? c->dbgA_off[segment] : c->dbgB_off[segment]);
    const size_t tile = rows * s.rank * 4;
    if (cudaMemcpy2D(host_dst, tile, base + (size_t)side * rows * s.rank, 2 * tile, tile, c->cc.BH,
                     cudaMemcpyDeviceToHost) != cudaSuccess) {
      cudaGetLastError();
      return GEAR_ERR_CUDA;
    }
    return GEAR_OK;
  }
  void* tmp = nullptr;
  if (cudaMalloc(&tmp, bytes) != cudaSuccess) { cudaGetLastError(); return GEAR_ERR_ALLOC; }
  gear_status r = GEAR_OK;
  if (launch_export(c->arena, s, c->cc, what, tmp, n, 0) != cudaSuccess ||
      cudaMemcpy(host_dst, tmp, bytes, cudaMemcpyDeviceToHost) != cudaSuccess) {
    cudaGetLastError();
    r = GEAR_ERR_CUDA;
  }
  cudaFree(tmp);
  return r;
}

extern "C" gear_status gear_cache_info(const gear_cache* c, gear_info* info) {
  if (!c || !info) return GEAR_ERR_ARG;
  info->n_segments = (int)c->segs.size();
  info->buffer_len = c->buf_len;
  info->n_compressed = c->n_compressed;
  return GEAR_OK;
}

extern "C" gear_status gear_segment_info_get(const gear_cache* c, int32_t segment, gear_segment_info* info) {
  if (!c || !info || segment < 0 || segment >= (int)c->segs.size()) return GEAR_ERR_ARG;
  const SegDesc& s = c->segs[segment];
  info->n_c = s.n_c; info->rank = s.rank; info->g_k = s.T; info->g_v = c->cc.g_v; info->k_k = s.k_k; info->k_v = c->cc.k_v;
  if (s.csr_base16 != 0) { info->g_k = s.n_c; info->k_k = s.csr_k / 2; }      // per-vector keys: the whole segment
  return GEAR_OK;
}

extern "C" gear_status gear_cache_bytes(const gear_cache* c, gear_bytes* out) {
  if (!c || !out) return GEAR_ERR_ARG;
  memset(out, 0, sizeof(*out));
  const long long BH = c->cc.BH, d = kHeadDim;
  for (const SegDesc& s : c->segs) {
    out->codes += BH * 2 * (long long)s.n_c * d * c->cc.bits / 8;
    out->scale_zero += BH * ((long long)s.nblk * d * 4 + (long long)s.n_c * c->cc.ngv * 4);
    out->outliers += BH * ((long long)s.nblk * d * 2 * s.k_k * 3 + (long long)s.n_c * c->cc.ngv * 2 * c->cc.k_v * 3);
    out->lowrank_a += BH * 2 * (long long)s.n_c * s.rank * 2;
    out->lowrank_b += BH * 2 * d * s.rank * 2;
    out->stored_total += BH * s.bh_stride;
    if (s.csr_base16 != 0) {     // per-vector keys: the list of the segment's key outliers (the records repeat the scales)
      const long long list = BH * (long long)csr_stride_bytes(s.nblk, s.csr_k);
      out->outliers += list;
      out->stored_total += list;
    }
  }
  out->buffer = BH * 2 * (long long)c->buf_len * d * 2;
  out->stored_total += out->buffer;
  out->alloc_total = (long long)(c->arena_bytes + c->dbg_bytes + c->flush_ws_bytes + c->partial_bytes +
                                 2 * (size_t)BH * c->cfg.buffer_cap * d * 2 + sizeof(SegDesc) * (size_t)c->table_cap);
  return GEAR_OK;
}

extern "C" gear_status gear_last_device_status(gear_cache* c, int32_t* code) {
  if (!c || !code) return GEAR_ERR_ARG;
  int v = 0;
  if (cudaDeviceSynchronize() != cudaSuccess || cudaMemcpy(&v, c->status, 4, cudaMemcpyDeviceToHost) != cudaSuccess ||
      cudaMemset(c->status, 0, 4) != cudaSuccess) {
    cudaGetLastError();
    return GEAR_ERR_CUDA;
  }
  if (v != 0) {
    // a warp that gave up left without taking its tickets: start the next call from a clean count
    const size_t units = (size_t)c->units_alloc;
    if (cudaMemset(c->tickets, 0, units * 4) != cudaSuccess) { cudaGetLastError(); return GEAR_ERR_CUDA; }
  }
  *code = v;
  return GEAR_OK;
}

extern "C" gear_status gear_test_dead_wait(gear_cache* c, int32_t on) {
  if (!c) return GEAR_ERR_ARG;
  c->test_dead_wait = on ? 1 : 0;
  return GEAR_OK;
}

extern "C" gear_status gear_fp16_attn_status(void* scratch, int32_t* code) {
  if (!scratch || !code) return GEAR_ERR_ARG;
  int v = 0;
  if (cudaDeviceSynchronize() != cudaSuccess || cudaMemcpy(&v, scratch, 4, cudaMemcpyDeviceToHost) != cudaSuccess ||
      cudaMemset(scratch, 0, 4) != cudaSuccess) {
    cudaGetLastError();
    return GEAR_ERR_CUDA;
  }
  *code = v;
  return GEAR_OK;
}

extern "C" const char* gear_strerror(gear_status s) {
  switch (s) {
    case GEAR_OK: return "ok";
    case GEAR_FLUSHED: return "buffer flushed";
    case GEAR_ERR_ARG: return "invalid argument";
    case GEAR_ERR_SHAPE: return "sizes violate the grouping rules";
    case GEAR_ERR_ALIGN: return "pointer not 16-byte aligned";
    case GEAR_ERR_CAPACITY: return "capacity exhausted";
    case GEAR_ERR_ALLOC: return "device allocation failed";
    case GEAR_ERR_CUDA: return "CUDA runtime error";
    case GEAR_ERR_TIMEOUT: return "bounded device-side wait gave up";
    case GEAR_ERR_STATE: return "call not valid in the cache's current state";
    default: return "unknown status";
  }
}
