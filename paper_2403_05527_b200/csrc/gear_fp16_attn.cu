// Decode attention (Eq. 1) over an uncompressed fp16 cache: the reference point
// the compressed path is compared with.  It runs the same streaming kernel with
// every block taken as fp16 rows (the path the streaming buffer uses), so both
// formats share the softmax, split and merge code.
#include <cuda_runtime.h>
#include <math.h>

#include <mutex>

#include "../../include/gear.h"
#include "gear_internal.cuh"

namespace gear {

static const int kFp16MaxWarps = 148 * 32 * 2;

size_t fp16_attn_scratch(int batch, int n_q_heads) {
  // tickets + status, then partials: one per (unit, warp touching it); units <= batch * n_q_heads
  const size_t units = (size_t)batch * n_q_heads;
  const size_t parts = (size_t)kFp16MaxWarps + 3 * units;
  return 256 + units * 4 + 256 + parts * 8 * kPartRow * 4;
}

cudaError_t launch_fp16_attn(const void* K, const void* V, const void* q, float* out, int batch, int n_q_heads,
                             int n_kv_heads, long long n, long long n_alloc, float scale, void* scratch,
                             size_t scratch_bytes, cudaStream_t st) {
  (void)scratch_bytes;
  const int G = n_q_heads / n_kv_heads, passes = decode_passes(G);
  const size_t units = (size_t)batch * n_kv_heads * passes;
  int dev = 0, sms = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  DecodeArgs a;
  if (!decode_plan(2, G, 1, 0, 0, 0, 16, 227 * 1024, 0, &a)) return cudaErrorInvalidConfiguration;
  const int occ = decode_occupancy(2, G, 1, a.wide, (size_t)a.ws.total);
  if (occ < 1) return cudaErrorInvalidConfiguration;
  long long grid = (long long)sms * occ;
  const long long work = (long long)units * ((n + 15) / 16);
  if (grid > work) grid = work;
  if (grid > kFp16MaxWarps) grid = kFp16MaxWarps;
  unsigned char* s = reinterpret_cast<unsigned char*>(scratch);
  a.arena = nullptr; a.table = nullptr; a.blk2seg = nullptr;
  a.buf_k = (const __half*)K; a.buf_v = (const __half*)V; a.q = (const __half*)q; a.out = out;
  a.status = reinterpret_cast<int*>(s);
  a.tickets = reinterpret_cast<int*>(s + 256);
  a.partial = reinterpret_cast<float*>(s + 256 + ((units * 4 + 255) / 256) * 256);
  a.cc.bits = 2; a.cc.g_v = kHeadDim; a.cc.ngv = 1; a.cc.k_v = 0; a.cc.BH = batch * n_kv_heads; a.cc.n_b = (int)n_alloc;
  a.n_blocks_c = 0; a.buf_len = (int)n;
  a.n_kv_heads = n_kv_heads; a.group_heads = G;
  a.max_parts = (int)((size_t)grid / units + 3);
  a.scale_log2 = scale * 1.4426950408889634f;
  cudaError_t e = cudaMemsetAsync(s, 0, 256 + units * 4, st);
  if (e != cudaSuccess) return e;
  return launch_decode(a, (int)grid, st);
}

}  // namespace gear

// ---------------------------------------------------------------------------
// gear_fp16_decode_attn_static: the same launch with its scratch (status word,
// tickets, per-CTA partial results) in a fixed device array that is part of the
// library image, for callers that must not allocate device memory.
// ---------------------------------------------------------------------------
namespace {

constexpr size_t kStaticScratchBytes = (size_t)GEAR_STATIC_SCRATCH_BYTES;
constexpr int kStaticMaxQueryHeads = GEAR_STATIC_MAX_QUERY_HEADS;
constexpr int kMaxDevices = 64;

// One copy per GPU that loads the library, held until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

std::mutex g_static_mutex;
void* g_static_ptr[kMaxDevices];          // device address of g_static_scratch, per device ordinal
bool g_static_ready[kMaxDevices];

// Device address of the array on the current device.  In host code the symbol itself is only a
// handle, so the address is asked for once per device (with that device current) and kept.
cudaError_t static_scratch_address(void** ptr) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_static_mutex);
  if (!g_static_ready[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess) return e;
    g_static_ptr[dev] = p;
    g_static_ready[dev] = true;
  }
  *ptr = g_static_ptr[dev];
  return cudaSuccess;
}

}  // namespace

extern "C" gear_status gear_fp16_decode_attn_static(const void* K, const void* V, const void* q, float* out,
                                                    int32_t batch, int32_t n_q_heads, int32_t n_kv_heads,
                                                    int32_t head_dim, int64_t n, int64_t n_alloc, float softmax_scale,
                                                    void* stream) {
  using namespace gear;
  if (!K || !V || !q || !out) return GEAR_ERR_ARG;
  if (batch < 1 || n_kv_heads < 1 || n_q_heads < 1 || n < 1 || n_alloc < n) return GEAR_ERR_ARG;
  if (n_alloc > 0x7fffffffLL) return GEAR_ERR_ARG;                  // token counts travel as 32-bit integers
  if (head_dim != kHeadDim || n_q_heads % n_kv_heads) return GEAR_ERR_SHAPE;
  if (((uintptr_t)K | (uintptr_t)V | (uintptr_t)q | (uintptr_t)out) & 15) return GEAR_ERR_ALIGN;
  if ((long long)batch * n_q_heads > kStaticMaxQueryHeads) return GEAR_ERR_CAPACITY;
  cudaStream_t st = (cudaStream_t)stream;
  const int G = n_q_heads / n_kv_heads;
  const int hp = decode_heads_per_pass(G);                // query heads per pass of the kernel that will run
  const int passes = decode_passes(G);
  const size_t units = (size_t)batch * n_kv_heads * passes;
  // layout of the array: status word, tickets, then one partial slot per (unit, CTA touching it)
  const size_t header = 256 + ((units * 4 + 255) / 256) * 256;
  const size_t slot = (size_t)hp * kPartRow * 4;
  const size_t slots = (kStaticScratchBytes - header) / slot;
  const long long parts_cap = (long long)(slots / units);   // partial slots per unit that fit
  if (parts_cap < 4) return GEAR_ERR_CAPACITY;

  void* scratch = nullptr;
  if (static_scratch_address(&scratch) != cudaSuccess) { cudaGetLastError(); return GEAR_ERR_CUDA; }

  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
    cudaGetLastError();
    return GEAR_ERR_CUDA;
  }
  DecodeArgs a;
  if (!decode_plan(2, G, 1, 0, 0, 0, 16, 227 * 1024, 0, &a)) return GEAR_ERR_SHAPE;
  const int occ = decode_occupancy(2, G, 1, a.wide, (size_t)a.ws.total);
  if (occ < 1) return GEAR_ERR_CUDA;
  long long grid = (long long)sms * occ;
  const long long work = (long long)units * ((n + 15) / 16);
  if (grid > work) grid = work;
  const long long grid_cap = (parts_cap - 3) * (long long)units;    // keeps grid / units + 3 slots per unit inside the array
  if (grid > grid_cap) grid = grid_cap;
  unsigned char* s = reinterpret_cast<unsigned char*>(scratch);
  a.arena = nullptr; a.table = nullptr; a.blk2seg = nullptr;
  a.buf_k = (const __half*)K; a.buf_v = (const __half*)V; a.q = (const __half*)q; a.out = out;
  a.status = reinterpret_cast<int*>(s);
  a.tickets = reinterpret_cast<int*>(s + 256);
  a.partial = reinterpret_cast<float*>(s + header);
  a.cc.bits = 2; a.cc.g_v = kHeadDim; a.cc.ngv = 1; a.cc.k_v = 0; a.cc.BH = batch * n_kv_heads; a.cc.n_b = (int)n_alloc;
  a.n_blocks_c = 0; a.buf_len = (int)n;
  a.n_kv_heads = n_kv_heads; a.group_heads = G;
  a.max_parts = (int)((size_t)grid / units + 3);
  const float sc = softmax_scale > 0.f ? softmax_scale : 1.0f / sqrtf((float)kHeadDim);
  a.scale_log2 = sc * 1.4426950408889634f;
  // the array keeps what the previous call left: the status word and the tickets must start at zero
  if (cudaMemsetAsync(s, 0, header, st) != cudaSuccess || launch_decode(a, (int)grid, st) != cudaSuccess) {
    cudaGetLastError();
    return GEAR_ERR_CUDA;
  }
  return GEAR_OK;
}

extern "C" gear_status gear_fp16_attn_static_status(int32_t* code) {
  if (!code) return GEAR_ERR_ARG;
  void* scratch = nullptr;
  if (static_scratch_address(&scratch) != cudaSuccess) { cudaGetLastError(); return GEAR_ERR_CUDA; }
  return gear_fp16_attn_status(scratch, code);
}
