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
//     header     16 B : fp32 max |x - zero| over the block's key / value outliers
//     kscale     128 x (scale fp16, zero fp16)                 one pair per channel
//     koval      128 x 2k_K fp16   outlier values, per channel, in-group index ascending
//     koidx      128 x 2k_K u8     their token index inside the block
//     kcodes     T/16 slabs x 16*128*b/8 bytes, in mma-fragment order (see code_coord_k)
//     ak         T/16 slabs x [16 tokens][r_pad] fp16          rows of A_K
//   -- off_vpart --
//     vcodes     same size as kcodes (see code_coord_v)
//     av         T/16 slabs x [r_pad][16 tokens] fp16          rows of A_V, transposed per slab
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
};

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
  const int nslab = s.T / kSlab;
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
  s.off_vcodes = o;  o += nslab * s.slab_codes;
  s.off_av = o;      o += round_up(nslab * s.slab_a, 16);
  s.off_vscale = o;  o += s.T * c.ngv * 4;
  s.off_voval = o;   o += round_up(s.T * c.ngv * 2 * c.k_v * 2, 16);
  s.off_voidx = o;   o += round_up(s.T * c.ngv * 2 * c.k_v, 16);
  s.rec_bytes = o;
  s.bh_stride = (long long)s.bfac_bytes + (long long)s.nblk * s.rec_bytes;
}

// ---------------------------------------------------------------------------
// Where a code lives.  Per slab and side the codes are 32-bit words; lane `lane`
// of a warp owns words q = 0 .. nq-1 (nq = 4 for 2-bit, 8 for 4-bit).  Word q of
// lane `lane` sits at 32-bit index (q / 4) * 128 + lane * 4 + (q % 4) of the
// slab, so one 128-bit shared-memory load per lane fetches four of them.
// Inside a word, 16-bit half e (0 = low) holds, at bits [b*u, b*u + b), the code
// that becomes half e of fragment register u of that word.
//
// Keys are the A operand (tokens x channels) of mma.m16n8k16: for channel
// chunk kc (16 channels) lane (gid = lane/4, t = lane%4) needs
//   a0 = {tok gid,   ch 2t, 2t+1}   a1 = {tok gid+8, ch 2t, 2t+1}
//   a2 = {tok gid,   ch 2t+8, +9}   a3 = {tok gid+8, ch 2t+8, +9}
// Values are the A operand (channels x tokens): for channel tile mt
//   a0 = {ch gid,   tok 2t, 2t+1}   a1 = {ch gid+8, tok 2t, 2t+1}
//   a2 = {ch gid,   tok 2t+8, +9}   a3 = {ch gid+8, tok 2t+8, +9}
//
// The decode kernel turns a word into fragment registers with one AND per
// register: the masked field, left where it is, read as fp16 is the subnormal
// code * 2^(b*u' - 24) (u' = u for the fields the 10-bit mantissa holds, after
// one shift of the word for the others).  A power of two per register is
// harmless only where the product can absorb it, which fixes who shares a field
// position: for keys a0 and a1 (they meet the same B register: its q * scale is
// pre-divided), for values a0 and a2 (they feed the same output row, which
// carries the factor until the end).  Hence keys take (a0, a2) of a tile from
// fields 2j, 2j+1 of one word and (a1, a3) from the same fields of a second
// word; values take (a0, a1) from fields 2j, 2j+1 of one word and (a2, a3) from
// a second word.
// ---------------------------------------------------------------------------
__host__ __device__ inline int words_per_lane(int bits) { return bits == 2 ? 4 : 8; }
__host__ __device__ inline int regs_per_word(int bits) { return bits == 2 ? 8 : 4; }   // half2 per word

// key code at (lane, q, u, e) -> token in slab, channel
__host__ __device__ inline void code_coord_k(int bits, int lane, int q, int u, int e, int& tok, int& ch) {
  const int hpw = regs_per_word(bits);
  const int wpt = 16 / hpw;                 // words per token half (2 or 4)
  const int th = q / wpt, w = q % wpt;
  const int kc = (hpw / 2) * w + (u >> 1);
  const int hi = u & 1;                     // 0: a0/a1 columns, 1: a2/a3 columns (+8)
  tok = 8 * th + (lane >> 2);
  ch = 16 * kc + 8 * hi + 2 * (lane & 3) + e;
}

// value code at (lane, q, u, e) -> token in slab, channel
__host__ __device__ inline void code_coord_v(int bits, int lane, int q, int u, int e, int& tok, int& ch) {
  const int tpp = regs_per_word(bits) / 2;  // channel tiles per pair of words (4 or 2)
  const int mt = tpp * (q >> 1) + (u >> 1);
  const int a = (u & 1) + 2 * (q & 1);      // fragment register a0..a3
  ch = 16 * mt + 8 * (a & 1) + (lane >> 2);
  tok = 2 * (lane & 3) + 8 * (a >> 1) + e;
}

__host__ __device__ inline int word_index(int lane, int q) { return (q >> 2) * 128 + lane * 4 + (q & 3); }

}  // namespace gear
