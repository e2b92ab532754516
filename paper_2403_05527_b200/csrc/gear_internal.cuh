// Internal declarations shared by the library's translation units.
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "gear_layout.cuh"

namespace gear {

// process-wide count of kernels this library launched (read through gear_kernel_launches)
void count_launches(int n);

struct CompressArgs {
  SegDesc seg;
  CacheConst cc;
  unsigned char* arena;
  const __half* K;      // [nbh][n_c][128], already offset to the first (batch, head) of the range
  const __half* V;
  float* R;             // residual workspace [nbh][2][n_c][128] or nullptr (rank 0)
  int bh0;              // first (batch, head) of the range, for addressing the records
};

struct PiArgs {
  SegDesc seg;
  unsigned char* arena;
  float* R;             // [ntiles][n_c][128]
  float* Bcur;          // [ntiles][128][16]
  float* Bp;            // [ntiles][nchunk][128][16]
  float* A0;            // [ntiles][n_c][16]
  float* Gp;            // [ntiles][nchunk][256]
  float* W;             // [ntiles][256]
  float* dbgA;          // fp32 copies for export, whole segment: [BH][2][n_c][rank] / [BH][2][128][rank]
  float* dbgB;
  int bh0, ntiles, n_c, rank, nchunk;
};

struct CompressJob {
  SegDesc seg;
  CacheConst cc;
  unsigned char* arena;
  const __half* K;      // [BH][n_c][128]
  const __half* V;
  const float* B0;      // [BH][2][128][rank] or nullptr
  float* dbgA;
  float* dbgB;
  unsigned long long seed;
  int segment_index;
  int iters;
};

size_t compress_workspace_bytes(int nbh, int n_c, int rank);
cudaError_t compress_range(const CompressJob& job, int bh0, int nbh, unsigned char* ws, cudaStream_t st);
cudaError_t launch_write_desc(SegDesc* table, int index, const SegDesc& d, cudaStream_t st);
cudaError_t launch_append(void* buf_k, void* buf_v, const void* k_new, const void* v_new, int BH, int n_b, int slot,
                          cudaStream_t st);

// decode attention over the compressed cache
struct DecodeArgs {
  const unsigned char* arena;
  const SegDesc* table;
  const __half* buf_k;        // [BH][n_b][128]
  const __half* buf_v;
  const __half* q;            // [B][Hq][128]
  float* out;                 // [B][Hq][128]
  float* partial;             // [BH][max_parts][G][130]
  int* tickets;               // [BH * head passes]
  int* status;
  CacheConst cc;
  int nseg;
  int n_blocks_c;             // compressed blocks per (batch, head)
  int buf_len;                // tokens in the fp16 buffer
  int n_kv_heads, group_heads;   // H, G = Hq / H
  int max_parts;
  int stage_bytes;            // bytes of one ring stage
  int warp_smem;              // bytes of shared memory per warp
  int max_T;                  // largest block length over the segments
  int max_rpad;
  float scale_log2;           // softmax scale * log2(e)
};
cudaError_t launch_decode(const DecodeArgs& a, int warps_per_cta, int grid, size_t smem, cudaStream_t st);
void decode_smem_plan(int bits, int max_rec, int max_bfac, int max_T, int max_rpad, int heads_per_pass,
                      int* stage_bytes, int* warp_smem);

// fp16-cache attention
cudaError_t launch_fp16_attn(const void* K, const void* V, const void* q, float* out, int batch, int n_q_heads,
                             int n_kv_heads, long long n, long long n_alloc, float scale, void* scratch,
                             size_t scratch_bytes, cudaStream_t st);
size_t fp16_attn_scratch(int batch, int n_q_heads);

// canonical export
cudaError_t launch_export(const unsigned char* arena, const SegDesc& sd, const CacheConst& cc, int what, void* dst,
                          size_t n_elems, cudaStream_t st);

}  // namespace gear
