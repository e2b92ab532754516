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
  unsigned int* Rmax;   // [nbh][2] bit patterns of max |R| per tile (zeroed before the launch), with R
  int bh0;              // first (batch, head) of the range, for addressing the records
  int side0;            // first side the launch covers (blockIdx.z + side0: 0 keys, 1 values)
};

// Key side of a segment with per-vector grouping (gear_kcvt.cu)
struct KcvtArgs {
  SegDesc seg;
  unsigned char* arena;
  const __half* K;      // [nbh][n_c][128], already offset to the first (batch, head) of the range
  float* R;             // residual workspace [nbh][2][n_c][128] or nullptr (rank 0)
  unsigned int* Rmax;   // [nbh][2] (see CompressArgs) or nullptr
  int bh0;
  unsigned char* codes8;   // workspace: [nbh][n_c][128] one code per byte
  unsigned int* olist;     // workspace: [nbh][128][csr_k] token | fp16 value << 16, token ascending
  __half2* sz;             // workspace: [nbh][128] (scale, zero)
};
bool kcvt_fits(int n_c);
size_t kcvt_workspace_bytes(int nbh, int n_c, int csr_k);
cudaError_t launch_kcvt_keys(KcvtArgs a, int nbh, int bits, unsigned char* ws, cudaStream_t st);

struct PiArgs {
  SegDesc seg;
  unsigned char* arena;
  float* R;             // [ntiles][n_c][128]
  unsigned int* Rmax;   // [ntiles] bit pattern of the tile's largest |R|
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

size_t compress_workspace_bytes(int nbh, int n_c, int rank, int csr_k = -1);
// whole-tile path for short segments (one launch): usable when compress_tile_fits()
bool compress_tile_fits(int T, int n_c, int rank);
cudaError_t compress_tile(const CompressJob& job, int BH, cudaStream_t st);
cudaError_t compress_range(const CompressJob& job, int bh0, int nbh, unsigned char* ws, cudaStream_t st);
cudaError_t launch_write_desc(SegDesc* table, int* blk2seg, int index, const SegDesc& d, cudaStream_t st);
cudaError_t launch_append(void* buf_k, void* buf_v, const void* k_new, const void* v_new, int BH, int n_b, int slot,
                          cudaStream_t st);

// decode attention over the compressed cache
constexpr int kMaxStages = 4;
constexpr int kPartRow = 132;     // floats per head of a partial result: 128 outputs, running max, denominator, padding to 16 bytes
struct WarpSmem {      // byte offsets of a warp's (= a CTA's) shared-memory regions
  int ring, sdc, qs, xr, ps, corr_k, corr_v, ocorr, wl, misc, total;
  int fragv_stride;    // words per row of the value B-operand staging area
  int fragp;           // byte offset of the fp16 probability fragments inside the xr region
};
struct DecodeArgs {
  const unsigned char* arena;
  const SegDesc* table;
  const int* blk2seg;         // [n_blocks_c] segment index of every compressed block
  const __half* buf_k;        // [BH][n_b][128]
  const __half* buf_v;
  const __half* q;            // [B][Hq][128]
  float* out;                 // [B][Hq][128]
  float* partial;             // [units][max_parts][HP][kPartRow]
  int* tickets;               // [units]
  int* status;
  CacheConst cc;
  int n_blocks_c;             // compressed blocks per (batch, head)
  int buf_len;                // tokens in the fp16 buffer
  int n_kv_heads, group_heads;   // H, G = Hq / H
  int max_parts;
  // Unit-aligned split (aligned != 0): no warp crosses from one unit into the next.  Units [0, units_a) are cut into
  // parts_a ranges, the others into parts_b = parts_a - 1; the CTAs are ordered by the length of their range,
  // longest first, in up to four classes (unit type x one-block-longer or not): class k holds the CTAs
  // [cls_start[k], cls_start[k + 1]), cls_n[k] consecutive parts from cls_p0[k] on per unit, units from cls_u0[k] on.
  // aligned == 0: the flat (unit, block) space is cut into gridDim.x equal ranges.
  int aligned, units_a, parts_a, parts_b;
  int cls_start[5], cls_u0[4], cls_n[4], cls_p0[4];
  int nstage;                 // ring stages (<= kMaxStages)
  int stage_bytes;            // bytes of one ring stage
  int bregion;                // bytes at the front of a stage reserved for one B factor
  int max_T;                  // largest block length over the segments
  int hpa;                    // query heads per pass (1 or 4)
  int spin_limit;             // polls a consumer spends on one ring stage before it gives up
  int test_dead_wait;         // test only: wait once on a barrier that nothing completes, with a short limit
  int wide;                   // one head per pass: use the kernel built for twelve resident warps (more registers)
  int early_reads;            // the cache's data was last written at least two launches back on this stream (see the kernel)
  WarpSmem ws;
  float scale_log2;           // softmax scale * log2(e)
};
cudaError_t launch_decode(const DecodeArgs& a, int grid, cudaStream_t st);
// Shared-memory plan of one warp; returns false if no stage count fits.  heads = G (query heads per kv head).
// warps_cap > 0 limits the resident warps per SM below what registers and shared memory allow.
bool decode_plan(int bits, int heads, int ngv, int max_kpart, int max_vpart, int max_bfac, int max_T, size_t smem_budget,
                 int warps_cap, DecodeArgs* a);
int decode_occupancy(int bits, int heads, int ngv, int wide, size_t smem);
int static_shape_id(const SegDesc& s, const CacheConst& c);
// query heads one pass of the kernel takes for G query heads per kv head, and the number of passes
inline int decode_heads_per_pass(int G) { return G == 1 ? 1 : 4; }
inline int decode_passes(int G) { return (G + decode_heads_per_pass(G) - 1) / decode_heads_per_pass(G); }
constexpr int kDecodeSpinLimit = 4000000;

// fp16-cache attention
cudaError_t launch_fp16_attn(const void* K, const void* V, const void* q, float* out, int batch, int n_q_heads,
                             int n_kv_heads, long long n, long long n_alloc, float scale, void* scratch,
                             size_t scratch_bytes, cudaStream_t st);
size_t fp16_attn_scratch(int batch, int n_q_heads);

// canonical export
cudaError_t launch_export(const unsigned char* arena, const SegDesc& sd, const CacheConst& cc, int what, void* dst,
                          size_t n_elems, cudaStream_t st);

}  // namespace gear
