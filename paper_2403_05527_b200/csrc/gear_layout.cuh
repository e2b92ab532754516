// Packed layout of a compressed GEAR segment in HBM, shared by the compress,
// decode and export kernels.
//
// A segment (the prefill block or one flushed buffer, Algorithm 1) of n_c
// tokens is cut into blocks of T = g_K = min(g, n_c) tokens: one key
// quantization group per channel spans exactly one block.  For every
// (batch, kv head) the segment stores, contiguously,
//     [ B factors ][ record of block 0 ][ record of block 1 ] ...
// so that the decode kernel fetches a block (and, for block 0, the factors in
// front of it) with one bulk copy.  A record holds, section by section:
// key part (everything the score pass needs), then value part:
//     header     16 B : fp32 max |x - zero| over the block's key / value outliers, then the
//                       largest key scale and the largest value scale of the block
//     kscale     128 x (scale fp16, zero fp16)                 one pair per channel
//     koval      128 x 2k_K fp16   outlier values, per channel, in-group index ascending
//     koidx      128 x 2k_K u8     their token index inside the block
//     kcodes     ceil(T/16) slabs x 16*128*b/8 bytes, in mma-fragment order (see code_coord_k; tokens past T: code 0)
//     ak         ceil(T/16) slabs x [16 tokens][r_pad] fp16    rows of A_K (zero past T)
//   -- off_vpart --
//     vcodes     ceil(T/32) chunks x 32*128*b/8 bytes (see code_coord_v; tokens past T hold code 0)
//     av         ceil(T/16) slabs x [r_pad][16 tokens] fp16    rows of A_V, transposed per slab (zero past T)
//     vscale     T x (d_H/g_V) x (scale fp16, zero fp16)
//     voval      T x (d_H/g_V) x 2k_V fp16
//     voidx      T x (d_H/g_V) x 2k_V u8   channel index inside the group
// Every section starts on a 16-byte boundary, so the decode kernel can fetch the
// key part and the value part of a block with one bulk copy each.  The B factors
// are  [r_pad][128] fp16 (B_K transposed)  then  [128][r_pad] fp16 (B_V).
#pragma once
#include <stdint.h>

namespace gear {

constexpr int kHeadDim = 128;
constexpr int kSlab = 16;          // tokens per mma slab
constexpr int kMaxRank = 16;
constexpr int kMaxOutliers = 8;    // per side per group
constexpr int kRecHeader = 16;

struct SegDesc {
  long long seg_base;    // byte offset in the arena of (bh = 0)'s data
  long long bh_stride;   // bytes per (batch, kv head): bfac_bytes + nblk * rec_bytes
  long long dbg_base;    // byte offset in the debug arena of the fp32 factor copies (or -1)
  int tok_start;         // first token of the segment in the sequence
  int n_c;               // tokens
  int T;                 // tokens per block (= g_K)
  int nblk;              // blocks
  int blk_start;         // blocks before this segment
  int rank;              // r
  int r_pad;             // r rounded up to 2, 4, 8 or 16 (0 when r = 0)
  int k_k;               // outliers per side per key group
  int bfac_bytes;        // 2 * 128 * r_pad * 2
  int rec_bytes;
  int off_kscale, off_koval, off_koidx, off_kcodes, off_vcodes, off_ak, off_av,
      off_vscale, off_voval, off_voidx;
  int slab_codes;        // bytes of codes per slab and side
  int slab_a;            // bytes of A rows per slab and side
  int off_vpart;         // start of the value part inside a record (= bytes of the key part)
  int shape_id;          // compile-time block shape of the decode kernel that fits this segment, 0 = none
  // Per-vector key grouping over a whole segment (one key group per channel over all n_c tokens): the records keep
  // their 64-token blocks, every block repeats the channel's (scale, zero), k_k is 0 and the outliers of the
  // segment live in a list per (batch, kv head) behind the records (see csr_stride_bytes).
  int csr_k;             // outliers per channel, both sides together (0: the segment has per-block key groups)
  unsigned int csr_base16;   // the list of (batch, kv head) 0: offset from seg_base in units of 16 bytes
};
static_assert(sizeof(SegDesc) == 128, "a warp copies a descriptor with one 32-bit load per lane");

// Outlier list of one (batch, kv head) of such a segment: offsets u32 [nblk + 1] (padded to 16 bytes), then
// 128 * csr_k entries sorted by block, then channel, then token: token in block | channel << 8 | fp16 value << 16.
__host__ __device__ inline int csr_offsets_bytes(int nblk) { return ((nblk + 1) * 4 + 15) / 16 * 16; }
__host__ __device__ inline int csr_stride_bytes(int nblk, int csr_k) { return csr_offsets_bytes(nblk) + 128 * csr_k * 4; }

// Cache-wide constants the kernels need.
struct CacheConst {
  int bits;      // b
  int g_v;       // value group length
  int ngv;       // value groups per token = 128 / g_v
  int k_v;       // outliers per side per value group
  int BH;        // batch * kv heads
  int n_b;       // buffer capacity
};

__host__ __device__ inline int round_up(int x, int m) { return (x + m - 1) / m * m; }

__host__ __device__ inline int rank_pad(int r) {
  return r == 0 ? 0 : (r <= 2 ? 2 : (r <= 4 ? 4 : (r <= 8 ? 8 : 16)));
}

// Fill the size / offset fields of a descriptor from (T, n_c, rank, k_k) and the cache constants.
__host__ __device__ inline void layout_segment(SegDesc& s, const CacheConst& c) {
  const int nslab = (s.T + kSlab - 1) / kSlab;     // a flushed buffer may end inside a slab: its tail rows hold zeros
  const int nchunk_v = (s.T + 31) / 32;
  s.r_pad = rank_pad(s.rank);
  s.nblk = s.n_c / s.T;
  s.slab_codes = kSlab * kHeadDim * c.bits / 8;
  s.slab_a = kSlab * s.r_pad * 2;
  s.bfac_bytes = 2 * kHeadDim * s.r_pad * 2;
  int o = kRecHeader;
  s.off_kscale = o;  o += kHeadDim * 4;
  s.off_koval = o;   o += kHeadDim * 2 * s.k_k * 2;
  s.off_koidx = o;   o += round_up(kHeadDim * 2 * s.k_k, 16);
  s.off_kcodes = o;  o += nslab * s.slab_codes;
  s.off_ak = o;      o += round_up(nslab * s.slab_a, 16);
  s.off_vpart = o;
  s.off_vcodes = o;  o += nchunk_v * 2 * s.slab_codes;
  s.off_av = o;      o += round_up(nslab * s.slab_a, 16);
  s.off_vscale = o;  o += s.T * c.ngv * 4;
  s.off_voval = o;   o += round_up(s.T * c.ngv * 2 * c.k_v * 2, 16);
  s.off_voidx = o;   o += round_up(s.T * c.ngv * 2 * c.k_v, 16);
  s.rec_bytes = o;
  s.bh_stride = (long long)s.bfac_bytes + (long long)s.nblk * s.rec_bytes;
}

// ---------------------------------------------------------------------------
// Where a code lives.  The decode kernel multiplies codes on the integer tensor
// cores (mma.m16n8k32, u8 x s8): a byte of the A operand is one code, and a
// b-bit field left where it sits in its byte is the code times 2^(b * field),
// so a 32-bit word of packed codes becomes F = 8 / b fragment registers with one
// AND each.  The power of two is absorbed where it is free: by the fixed-point
// scale of the B operand (keys) or by the output row (values).
//
// A "tuple" is four 32-bit words per lane -- the registers a0..a3 of one A
// fragment (16 rows x 32 k) -- whose F fields are the same fragment of F
// different tiles.  Lane (gid = lane / 4, t = lane % 4), word w = r + 2 * kh,
// byte i, field j:
//   keys   (rows = tokens of a 16-token slab, k = channels): tuple tau of the slab
//          token   = gid + 8 r
//          channel = 32 (F tau + j) + 16 kh + 4 t + i        field <-> 32-channel chunk
//   values (rows = channels, k = tokens of a 32-token chunk): tuple tau of the chunk
//          channel = 16 (F tau + j) + gid + 8 r              field <-> 16-channel tile
//          token   = 16 kh + 4 t + i
// The four words of a lane are one uint4: tuple number * 32 + lane in uint4 units
// from the start of the slab (keys: 4 / F tuples per slab) or chunk (values:
// 8 / F tuples per chunk).
// ---------------------------------------------------------------------------
__host__ __device__ inline int fields_per_byte(int bits) { return 8 / bits; }
__host__ __device__ inline int key_tuples_per_slab(int bits) { return 4 / fields_per_byte(bits); }
__host__ __device__ inline int value_tuples_per_chunk(int bits) { return 8 / fields_per_byte(bits); }

// key code of (lane, tuple, word, byte, field) -> token in slab, channel
__host__ __device__ inline void code_coord_k(int bits, int lane, int tau, int w, int i, int j, int& tok, int& ch) {
  tok = (lane >> 2) + 8 * (w & 1);
  ch = 32 * (fields_per_byte(bits) * tau + j) + 16 * (w >> 1) + 4 * (lane & 3) + i;
}
// value code of (lane, tuple, word, byte, field) -> token in chunk, channel
__host__ __device__ inline void code_coord_v(int bits, int lane, int tau, int w, int i, int j, int& tok, int& ch) {
  ch = 16 * (fields_per_byte(bits) * tau + j) + (lane >> 2) + 8 * (w & 1);
  tok = 16 * (w >> 1) + 4 * (lane & 3) + i;
}
// inverse maps: 32-bit word index inside the slab / chunk and bit position of the code
__host__ __device__ inline void code_slot_k(int bits, int tok, int ch, int& word, int& shift) {
  const int F = fields_per_byte(bits);
  const int c32 = ch >> 5, c = ch & 31;
  const int tau = c32 / F, j = c32 % F, kh = c >> 4, t = (c & 15) >> 2, i = c & 3;
  const int gid = tok & 7, r = tok >> 3;
  word = (tau * 32 + gid * 4 + t) * 4 + r + 2 * kh;
  shift = 8 * i + bits * j;
}
__host__ __device__ inline void code_slot_v(int bits, int tok, int ch, int& word, int& shift) {
  const int F = fields_per_byte(bits);
  const int tile = ch >> 4, c = ch & 15;
  const int tau = tile / F, j = tile % F, gid = c & 7, r = c >> 3;
  const int kh = tok >> 4, t = (tok & 15) >> 2, i = tok & 3;
  word = (tau * 32 + gid * 4 + t) * 4 + r + 2 * kh;
  shift = 8 * i + bits * j;
}

}  // namespace gear
