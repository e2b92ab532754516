// Decode attention (Eq. 1) over an uncompressed fp16 cache: the reference point
// the compressed path is compared with.  It runs the same streaming kernel with
// every block taken as fp16 rows (the path the streaming buffer uses), so both
// formats share the softmax, split and merge code.
#include <cuda_runtime.h>

#include "gear_internal.cuh"

namespace gear {

static const int kFp16MaxWarps = 148 * 32 * 2;

size_t fp16_attn_scratch(int batch, int n_q_heads) {
  // tickets + status, then partials: one per (unit, warp touching it); units <= batch * n_q_heads
  const size_t units = (size_t)batch * n_q_heads;
  const size_t parts = (size_t)kFp16MaxWarps + 3 * units;
  return 256 + units * 4 + 256 + parts * 8 * 130 * 4;
}

cudaError_t launch_fp16_attn(const void* K, const void* V, const void* q, float* out, int batch, int n_q_heads,
                             int n_kv_heads, long long n, long long n_alloc, float scale, void* scratch,
                             size_t scratch_bytes, cudaStream_t st) {
  (void)scratch_bytes;
  const int G = n_q_heads / n_kv_heads, hp = G <= 4 ? 4 : 8, passes = (G + hp - 1) / hp;
  const size_t units = (size_t)batch * n_kv_heads * passes;
  int dev = 0, sms = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  DecodeArgs a;
  if (!decode_plan(2, G, 1, 0, 0, 0, 16, 227 * 1024, &a)) return cudaErrorInvalidConfiguration;
  const int occ = decode_occupancy(2, G, 1, (size_t)a.ws.total);
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
