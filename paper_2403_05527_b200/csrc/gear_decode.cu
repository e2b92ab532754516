// Decode attention (Eq. 1, one query per sequence) over the compressed cache:
//   scores = q . dequant(codes_K)^T + (q B_K) A_K^T + q . S_K^T      (+ q . K_buffer^T)
//   out    = softmax(scores) . [dequant(codes_V) + A_V B_V^T + S_V]  (+ . V_buffer)
// fp16 K / V are never materialised.
//
// Every warp is its own CTA and an independent stream processor.  The
// (batch, kv head, head pass, block) space is cut into equal contiguous ranges,
// one per warp.  A block travels as two items -- its key part and its value
// part -- through a private shared-memory ring filled by bulk asynchronous
// copies (cp.async.bulk + mbarrier), so that the copies of the next items run
// while the warp works on the current one.
//
// Codes are unpacked in registers straight into the A operand of
// mma.sync.m16n8k16 (tokens x channels for keys, channels x tokens for values).
// The B operand holds the query heads of the GQA group, each split into an fp16
// high and low part (two columns), so that every product is exact and every sum
// is fp32.  Per-group scales are folded into the B operand (q * scale per channel
// for keys, p * scale per token for values), zero-points into one constant per
// block (keys) or an fp32 side sum (values).  Outlier corrections are scattered
// with 32-bit fixed-point shared-memory adds, which keeps the result independent
// of the order of the adds.  A warp writes one partial (m, l, o) per (batch,
// head) it touched; the last warp to arrive for a (batch, head) merges them.
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <math.h>

#include <type_traits>

#include "gear_internal.cuh"

namespace gear {

constexpr int kBufPitch = 272;                  // bytes per fp16 row of a buffer slab in shared memory
constexpr int kBufItem = kSlab * kBufPitch;     // one slab of key rows or of value rows
constexpr int kSpinLimit = 4000000;
// 32-bit words per B-fragment row set.  A row set holds, for every column that carries a query head (hi, lo) and
// every lane column t, two registers; with one head only two of the eight columns exist and the lanes of the other
// columns read those (their results are never used).  Padded against bank conflicts.
__host__ __device__ constexpr int frag_row_words(int hp) { return hp == 1 ? 24 : 72; }

static_assert(sizeof(SegDesc) <= 128 && sizeof(SegDesc) % 4 == 0, "descriptor copy assumes <= 32 words");

// ------------------------------------------------------------------ PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* b, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(b)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* b, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(b)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* b) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(dst)),
               "l"(src), "r"(bytes), "r"(smem_u32(b))
               : "memory");
}
__device__ __forceinline__ bool mbar_try(uint64_t* b, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(smem_u32(b)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: gives up after kSpinLimit polls and reports through `status`.
__device__ __forceinline__ bool mbar_wait(uint64_t* b, uint32_t parity, int* status) {
#pragma unroll 1
  for (int i = 0; i < kSpinLimit; ++i)
    if (mbar_try(b, parity)) return true;
  atomicExch(status, -7 /* GEAR_ERR_TIMEOUT */);
  return false;
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void mma16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// d = a * b (no accumulator input)
__device__ __forceinline__ void mma16816_z(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  const float z = 0.f;
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
      : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "f"(z));
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], const void* p) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(smem_u32(p)));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], const void* p) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(smem_u32(p)));
}
__device__ __forceinline__ uint32_t h2_as_u32(__half2 h) { return *reinterpret_cast<uint32_t*>(&h); }
__device__ __forceinline__ __half2 u32_as_h2(uint32_t u) { return *reinterpret_cast<__half2*>(&u); }

// Codes become fragment registers with one AND each.  A masked field left in place, read as fp16, is the
// subnormal  code * 2^(field_shift - 24)  (the tensor cores take subnormal inputs exactly); fields above the
// 10-bit mantissa are reached through one shifted copy of the word.  The power of two is undone where it is free:
// in the B operand for keys, in the output row for values.
template <int BITS>
__host__ __device__ constexpr int field_shift(int u) {     // bit position of field u once it sits in the mantissa
  return BITS == 2 ? 2 * (u < 5 ? u : u - 5) : 4 * (u & 1);
}
// One 32-bit word of codes -> its fragment registers r[0 .. 16/BITS).
template <int BITS>
__device__ __forceinline__ void unpack_word(uint32_t x, uint32_t* r) {
  if (BITS == 2) {
    const uint32_t y = x >> 10;
    r[0] = x & 0x00030003u;
    r[1] = x & 0x000C000Cu;
    r[2] = x & 0x00300030u;
    r[3] = x & 0x00C000C0u;
    r[4] = x & 0x03000300u;
    r[5] = y & 0x00030003u;
    r[6] = y & 0x000C000Cu;
    r[7] = y & 0x00300030u;
  } else {
    const uint32_t y = x >> 8;
    r[0] = x & 0x000F000Fu;
    r[1] = x & 0x00F000F0u;
    r[2] = y & 0x000F000Fu;
    r[3] = y & 0x00F000F0u;
  }
}
// Keys: the B register that meets fields 2j (b0) / 2j+1 (b1) holds q * scale * 2^(kKeyExp - field_shift), so every
// product carries 2^(kKeyExp - 24); the exponent keeps the scaled operand inside the fp16 range both ways.
template <int BITS> constexpr int kKeyExp = BITS == 2 ? 4 : 2;

// fp32 pair -> half2 of the high parts and half2 of the rounding remainders
__device__ __forceinline__ void split_hi_lo(float x0, float x1, uint32_t& hi, uint32_t& lo) {
  const __half2 h = __floats2half2_rn(x0, x1);
  hi = h2_as_u32(h);
  lo = h2_as_u32(__floats2half2_rn(x0 - __low2float(h), x1 - __high2float(h)));
}

// maximum over the warp in one instruction
__device__ __forceinline__ float warp_max(float x) {
  float r;
  asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(r) : "f"(x));
  return r;
}
__device__ __forceinline__ int float_exponent(float x) { return (int)((__float_as_uint(x) >> 23) & 0xFFu) - 127; }
// 2^e for |e| <= 60
__device__ __forceinline__ float pow2i(int e) { return __uint_as_float((uint32_t)(127 + e) << 23); }
__device__ __forceinline__ int clamp60(int e) { return max(-60, min(60, e)); }

// ------------------------------------------------------------------ shared memory plan (per warp)
bool decode_plan(int bits, int heads, int ngv, int max_kpart, int max_vpart, int max_bfac, int max_T, size_t smem_budget,
                 DecodeArgs* a) {
  (void)bits;
  const int HP = heads == 1 ? 1 : (heads <= 4 ? 4 : 8), NT = HP > 4 ? 2 : 1;
  const int frs = frag_row_words(HP);
  const int bregion = round_up(max_bfac / 2, 16);
  int part = max_kpart > max_vpart ? max_kpart : max_vpart;
  int stage = bregion + part;
  if (stage < kBufItem) stage = kBufItem;
  stage = round_up(stage, 16);
  if (max_T < kSlab) max_T = kSlab;
  const int nslab = max_T / kSlab;
  const int frag_rows = 8 > nslab * (ngv + 1) ? 8 : nslab * (ngv + 1);
  WarpSmem w;
  int o = 0;
  w.sdp = 0;
  w.sdc = o;     o += 128;
  w.qf = o;      o += HP == 1 ? kHeadDim * 4 : 0;   // grouped queries rebuild it from qs: their warps are short of shared memory
  w.qs = o;      o += HP * kHeadDim * 2;
  w.frag = o;    o += round_up(NT * frag_rows * frs * 4, 16);
  w.corr_k = o;  o += HP * max_T * 4;
  w.ps = o;      o += HP * max_T * 4;
  w.corr_v = o;  o += HP * kHeadDim * 4;
  w.ocorr = o;   o += HP * kHeadDim * 4;
  w.wl = o;      o += kMaxRank * (HP == 1 ? 1 : 8) * 4 + 16;
  w.misc = o;    o += 32 + kMaxStages * 8;   // exponents of max |q| per head, then the ring's mbarriers
  w.ring = round_up(o, 16);
  // most resident warps (in steps of four: one per scheduler) whose ring still holds two stages; then as many
  // stages as fit
  const int reg_limit = HP == 1 ? 16 : (HP == 4 ? 8 : 6);
  for (int warps = reg_limit; warps >= 1; warps -= (warps > 8 ? 4 : 1)) {
    const long long per = (long long)smem_budget / warps - 1024;     // the system reserves 1 KB per CTA
    long long ns = (per - w.ring) / stage;
    if (ns < 2) continue;
    if (ns > kMaxStages) ns = kMaxStages;
    w.total = w.ring + (int)ns * stage;
    a->aligned = 0;
    a->nstage = (int)ns; a->stage_bytes = stage; a->bregion = bregion; a->max_T = max_T; a->hpa = HP; a->ws = w;
    return true;
  }
  return false;
}

// ------------------------------------------------------------------ block shapes
// The work on a block depends on its shape: tokens T, outliers per key group, padded rank, outliers per value
// group.  The shapes of the usual configurations are compile-time constants (every offset inside the record becomes
// an immediate and the slab loops unroll); any other segment runs through the same code with run-time values.
struct DynShape {                      // values read from the segment descriptor
  static constexpr bool kDyn = true, kBuf = false;
  static constexpr int T = 0, k2k = 0, r_pad = 0, k2v = 0, unroll = 1, tok_unroll = 1;
  static constexpr int off_kscale = 0, off_koval = 0, off_koidx = 0, off_kcodes = 0, off_ak = 0, off_av = 0, off_vscale = 0,
                       off_voval = 0, off_voidx = 0;
};
struct BufShape {                      // one slab of fp16 rows of the streaming buffer
  static constexpr bool kDyn = false, kBuf = true;
  static constexpr int T = kSlab, k2k = 0, r_pad = 0, k2v = 0, unroll = 1, tok_unroll = 1;
  static constexpr int off_kscale = 0, off_koval = 0, off_koidx = 0, off_kcodes = 0, off_ak = 0, off_av = 0, off_vscale = 0,
                       off_voval = 0, off_voidx = 0;
};
template <int BITS, int NGV, int T_, int KK, int RP, int KV>
struct StaticShape {                   // mirrors layout_segment(); checked against it on the host (static_shape_id)
  static constexpr bool kDyn = false, kBuf = false;
  static constexpr int T = T_, k2k = 2 * KK, r_pad = RP, k2v = 2 * KV, unroll = 2, tok_unroll = T_ / 32;
  static constexpr int nslab = T_ / kSlab, slab_codes = kSlab * kHeadDim * BITS / 8;
  static constexpr int off_kscale = kRecHeader;
  static constexpr int off_koval = off_kscale + kHeadDim * 4;
  static constexpr int off_koidx = off_koval + kHeadDim * 2 * KK * 2;
  static constexpr int off_kcodes = off_koidx + (kHeadDim * 2 * KK + 15) / 16 * 16;
  static constexpr int off_ak = off_kcodes + nslab * slab_codes;
  static constexpr int off_vpart = off_ak + (nslab * kSlab * RP * 2 + 15) / 16 * 16;
  // value part, relative to its start
  static constexpr int off_av = nslab * slab_codes;
  static constexpr int off_vscale = off_av + (nslab * kSlab * RP * 2 + 15) / 16 * 16;
  static constexpr int off_voval = off_vscale + T_ * NGV * 4;
  static constexpr int off_voidx = off_voval + (T_ * NGV * 2 * KV * 2 + 15) / 16 * 16;
  static constexpr int rec_bytes = off_vpart + off_voidx + (T_ * NGV * 2 * KV + 15) / 16 * 16;
  static bool matches(const SegDesc& s, const CacheConst& c) {
    return c.bits == BITS && c.ngv == NGV && c.k_v == KV && s.T == T_ && s.k_k == KK && s.r_pad == RP &&
           s.off_kscale == off_kscale && s.off_koval == off_koval && s.off_koidx == off_koidx &&
           s.off_kcodes == off_kcodes && s.off_ak == off_ak && s.off_vpart == off_vpart &&
           s.off_vcodes == off_vpart && s.off_av == off_vpart + off_av && s.off_vscale == off_vpart + off_vscale &&
           s.off_voval == off_vpart + off_voval && s.off_voidx == off_vpart + off_voidx && s.rec_bytes == rec_bytes;
  }
};
// static shapes by id (0 = none).  Two value groups per token (g = 64): ids 1, 2; one group (g = 128): ids 3, 4.
template <int BITS> using ShapeA1 = StaticShape<BITS, 2, 64, 1, 4, 1>;     // g 64, s <= 3 %, rank 3..4
template <int BITS> using ShapeA2 = StaticShape<BITS, 2, 64, 1, 8, 1>;     // g 64, rank 5..8
template <int BITS> using ShapeB1 = StaticShape<BITS, 1, 128, 2, 4, 2>;    // g 128 prefill blocks
template <int BITS> using ShapeB2 = StaticShape<BITS, 1, 64, 1, 4, 2>;     // g 128, flushed 64-token buffers

int static_shape_id(const SegDesc& s, const CacheConst& c) {
  if (ShapeA1<2>::matches(s, c) || ShapeA1<4>::matches(s, c)) return 1;
  if (ShapeA2<2>::matches(s, c) || ShapeA2<4>::matches(s, c)) return 2;
  if (ShapeB1<2>::matches(s, c) || ShapeB1<4>::matches(s, c)) return 3;
  if (ShapeB2<2>::matches(s, c) || ShapeB2<4>::matches(s, c)) return 4;
  return 0;
}

// ------------------------------------------------------------------ the kernel
// HEADS = query heads handled per pass: 1 (multi-head attention), 4 or 8 (grouped queries; a pass may hold fewer).
template <int BITS, int HEADS, int NGV>
__global__ void __launch_bounds__(32, HEADS == 1 ? 16 : (HEADS == 4 ? 8 : 6)) gear_decode_kernel(const __grid_constant__ DecodeArgs a) {
  constexpr int HP = HEADS;
  constexpr int NT = HEADS > 4 ? 2 : 1;           // 8-column tiles of the B operand
  constexpr int GV = kHeadDim / NGV;              // channels per value group
  constexpr int SLABW = kSlab * kHeadDim * BITS / 8 / 16;   // uint4 per slab of codes
  constexpr int kFragStride = frag_row_words(HP);
  constexpr int CMASK = HP == 1 ? 1 : 7;          // fragment columns that exist, as a mask on the lane's column
  constexpr int WLS = HP == 1 ? 1 : 8;            // row stride of the small factor exchange buffer wl[16][heads]
  constexpr int HMASK = HP == 1 ? 0 : 7;          // heads that exist in wl, as a mask on the lane's head
  extern __shared__ __align__(128) unsigned char smem[];

  const int lane = threadIdx.x, gid = lane >> 2, t = lane & 3;
  const int G = a.group_heads;
  const int passes = (G + HP - 1) / HP;
  const int maxT = a.max_T;
  const int NS = a.nstage;
  unsigned char* ring = smem + a.ws.ring;
  SegDesc* sdc = reinterpret_cast<SegDesc*>(smem + a.ws.sdc);
  float* qf = reinterpret_cast<float*>(smem + a.ws.qf);          // [128] q * scale * log2(e) (one query head per pass only)
  __half* qs = reinterpret_cast<__half*>(smem + a.ws.qs);        // [HP][128] q
  uint32_t* frag = reinterpret_cast<uint32_t*>(smem + a.ws.frag);
  int* corr_k = reinterpret_cast<int*>(smem + a.ws.corr_k);      // [HP][maxT]
  float* ps = reinterpret_cast<float*>(smem + a.ws.ps);          // [HP][maxT] scores, then probabilities
  int* corr_v = reinterpret_cast<int*>(smem + a.ws.corr_v);      // [HP][128]
  float* ocorr = reinterpret_cast<float*>(smem + a.ws.ocorr);    // [HP][128]
  float* wl = reinterpret_cast<float*>(smem + a.ws.wl);          // [16][heads]
  int* qexp_s = reinterpret_cast<int*>(smem + a.ws.misc);        // [HP]
  uint64_t* bar = reinterpret_cast<uint64_t*>(smem + a.ws.misc + 32);   // [kMaxStages]; no static shared memory, so
                                                                         // that sixteen warps fit one SM

  // this lane's four channels in the key set-up sit in B register (lane / 2) % 2 of channel chunk lane / 4, which
  // meets field 2 * (chunk % 4) + register of the 2-bit words (any field of that parity of the 4-bit words)
  const float kfac = pow2i(kKeyExp<BITS> - (BITS == 2 ? 2 * ((2 * ((lane >> 2) & 3) + ((lane >> 1) & 1)) % 5)
                                                      : 4 * ((lane >> 1) & 1)));
  constexpr float kKeyBack = (float)(1 << (24 - kKeyExp<BITS>));       // undoes 2^(kKeyExp - 24)
  const bool o_plain = a.n_blocks_c == 0;       // no compressed block: the output rows carry no factor

  if (lane == 0)
    for (int s = 0; s < NS; ++s) mbar_init(&bar[s], 1);
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  for (int i = lane; i < (a.ws.corr_k - a.ws.frag) / 4; i += 32) frag[i] = 0u;
  for (int i = lane; i < HP * maxT; i += 32) corr_k[i] = 0;
  for (int i = lane; i < HP * kHeadDim; i += 32) corr_v[i] = 0;
  __syncwarp();

  // ---- this warp's range of the flat (unit, block) space; unit = (batch, kv head, head pass)
  const int nbuf_blocks = (a.buf_len + kSlab - 1) / kSlab;
  const int NB = a.n_blocks_c + nbuf_blocks;
  int n_left, u, blk_lo;                        // blocks left for this warp, current unit, first block in it
  int part = 0, parts_u = 0;                    // unit-aligned split: this warp's range inside its unit, ranges of the unit
  if (a.aligned) {
    int k = 0;
    while (k < 3 && (int)blockIdx.x >= a.cls_start[k + 1]) ++k;
    const int idx = blockIdx.x - a.cls_start[k];
    u = a.cls_u0[k] + idx / a.cls_n[k];
    part = a.cls_p0[k] + idx % a.cls_n[k];
    parts_u = u < a.units_a ? a.parts_a : a.parts_b;
    const int base = NB / parts_u, rem = NB - base * parts_u;       // base > 0: the host keeps parts <= NB
    blk_lo = part * base + min(part, rem);                          // the first `rem` ranges are one block longer
    n_left = base + (part < rem ? 1 : 0);
  } else {
    const long long F = (long long)a.cc.BH * passes * NB;
    const long long NW = gridDim.x, gw = blockIdx.x;
    const long long f0 = gw * F / NW, f1 = (gw + 1) * F / NW;
    if (f0 >= f1) return;                       // the host launches no more warps than blocks
    n_left = (int)(f1 - f0);
    u = (int)(f0 / NB);
    blk_lo = (int)(f0 - (long long)u * NB);
  }

  auto load_desc = [&](SegDesc* dst, int blk) {
    const int* src = reinterpret_cast<const int*>(a.table + a.blk2seg[blk]);
    __syncwarp();
    if (lane < (int)(sizeof(SegDesc) / 4)) reinterpret_cast<int*>(dst)[lane] = src[lane];
    __syncwarp();
  };

  // ---- producer: two items per block (key part, value part), issued in order into the ring
  int p_left = n_left, p_blk = blk_lo, p_share_lo = blk_lo, p_half = 0, p_stage = 0;
  int p_bh = u / passes, p_pass = u - p_bh * passes;
  int p_seg_lo = 0, p_seg_hi = 0, p_kbytes = 0, p_vbytes = 0, p_hb = 0;
  const unsigned char* p_segb = nullptr;        // B factors of the producer's (segment, batch, head)
  const unsigned char* p_rec = nullptr;         // record of block p_blk
  int n_inflight = 0;
  auto issue = [&]() {
    if (p_left == 0) return;
    unsigned char* dst = ring + p_stage * a.stage_bytes;
    uint64_t* b = &bar[p_stage];
    if (p_blk < a.n_blocks_c) {
      if (p_blk >= p_seg_hi) {                  // new segment (or new unit): read its descriptor
        const SegDesc* sd = a.table + a.blk2seg[p_blk];
        p_seg_lo = sd->blk_start;
        p_seg_hi = p_seg_lo + sd->nblk;
        p_kbytes = sd->off_vpart;
        p_vbytes = sd->rec_bytes - p_kbytes;
        p_hb = sd->bfac_bytes >> 1;
        p_segb = a.arena + sd->seg_base + (size_t)p_bh * sd->bh_stride;
        p_rec = p_segb + 2 * p_hb + (size_t)(p_blk - p_seg_lo) * (p_kbytes + p_vbytes);
      }
      if (lane == 0) {
        if (p_half == 0) {
          const bool wb = p_hb > 0 && (p_blk == p_seg_lo || p_blk == p_share_lo);
          mbar_expect_tx(b, p_kbytes + (wb ? p_hb : 0));
          if (wb) bulk_g2s(dst, p_segb, p_hb, b);
          bulk_g2s(dst + a.bregion, p_rec, p_kbytes, b);
        } else {
          const bool wb = p_hb > 0 && (p_blk == p_seg_hi - 1 || p_left == 1);
          mbar_expect_tx(b, p_vbytes + (wb ? p_hb : 0));
          if (wb) bulk_g2s(dst, p_segb + p_hb, p_hb, b);
          bulk_g2s(dst + a.bregion, p_rec + p_kbytes, p_vbytes, b);
        }
      }
    } else if (lane == 0) {
      const int j = p_blk - a.n_blocks_c;
      const int rows = min(kSlab, a.buf_len - j * kSlab);
      const __half* src = (p_half == 0 ? a.buf_k : a.buf_v) + ((size_t)p_bh * a.cc.n_b + (size_t)j * kSlab) * kHeadDim;
      mbar_expect_tx(b, rows * 256);
      for (int r = 0; r < rows; ++r) bulk_g2s(dst + r * kBufPitch, src + r * kHeadDim, 256, b);
    }
    ++n_inflight;
    if (++p_stage == NS) p_stage = 0;
    if (p_half == 0) {
      p_half = 1;
    } else {
      p_half = 0; --p_left; ++p_blk;
      p_rec += p_kbytes + p_vbytes;
      if (p_blk == NB) {
        p_blk = 0; p_share_lo = 0; p_seg_hi = 0;
        if (++p_pass == passes) { p_pass = 0; ++p_bh; }
      }
    }
  };
  for (int s = 0; s < NS; ++s) issue();

  int c_stage = 0, c_par = 0, c_seg_lo = 0, c_seg_hi = 0, c_shape = 0;
  bool alive = true;
  // wait for the next item (items are consumed in order); returns its stage
  auto acquire = [&]() -> unsigned char* {
    unsigned char* st = ring + c_stage * a.stage_bytes;
    if (!mbar_wait(&bar[c_stage], (uint32_t)c_par, a.status)) alive = false;
    if (++c_stage == NS) { c_stage = 0; c_par ^= 1; }
    --n_inflight;
    return st;
  };
  auto release = [&]() {       // the oldest item is consumed: refill its stage
    __syncwarp();
    issue();
  };

  // Output rows fed by the codes carry the factor of the field their codes came from: row half hf (channel gid + 8 hf)
  // of channel tile mt holds  value * 2^(row_shift - 24).  A product of full-range operands (buffer rows, B_V U) joins
  // such a row through a zero-based product and one multiply-add per element.
  auto row_shift = [](int mt, int hf) { return field_shift<BITS>(2 * (mt % (8 / BITS)) + hf); };
  auto add_scaled = [&](float (&o)[4], int mt, const uint32_t (&av)[4], uint32_t b0, uint32_t b1) {
    float d[4];
    mma16816_z(d, av, b0, b1);
    const float f0 = 1.f / (float)(1 << (24 - row_shift(mt, 0))), f1 = 1.f / (float)(1 << (24 - row_shift(mt, 1)));
    o[0] = fmaf(d[0], f0, o[0]); o[1] = fmaf(d[1], f0, o[1]);
    o[2] = fmaf(d[2], f1, o[2]); o[3] = fmaf(d[3], f1, o[3]);
  };

  // ---- loop over the units this warp touches
  while (n_left > 0 && alive) {
    const int blk_hi = min(NB, blk_lo + n_left);
    const int bh = u / passes, pass = u - bh * passes;
    const int HPu = HEADS == 1 ? 1 : min(HP, G - pass * HP);
    const int hq0 = bh * G + pass * HP;                 // first query head of this pass

    // unit state
    float O[8][NT][4], U[NT][4], m_run[HP], l_run[HP], cm[HP][NGV];
    uint32_t bw[NT][2];                                  // low-rank key term: B operand (q B_K) of the current segment
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      bw[nt][0] = bw[nt][1] = 0u;
#pragma unroll
      for (int i = 0; i < 4; ++i) U[nt][i] = 0.f;
#pragma unroll
      for (int mt = 0; mt < 8; ++mt)
#pragma unroll
        for (int i = 0; i < 4; ++i) O[mt][nt][i] = 0.f;
    }
#pragma unroll
    for (int h = 0; h < HP; ++h) {
      m_run[h] = -INFINITY; l_run[h] = 0.f;
#pragma unroll
      for (int g = 0; g < NGV; ++g) cm[h][g] = 0.f;
    }
    bool u_pending = false;

    // query rows of this pass -> shared (fp16 as given, and fp32 times scale * log2 e); exponent of max |q|
    __syncwarp();
#pragma unroll
    for (int h = 0; h < HP; ++h) {
      if (h < HPu) {
        const uint2 v = *reinterpret_cast<const uint2*>(a.q + (size_t)(hq0 + h) * kHeadDim + lane * 4);
        *reinterpret_cast<uint2*>(qs + h * kHeadDim + lane * 4) = v;
        const __half2 q01 = u32_as_h2(v.x), q23 = u32_as_h2(v.y);
        const float4 qv = make_float4(__low2float(q01) * a.scale_log2, __high2float(q01) * a.scale_log2,
                                      __low2float(q23) * a.scale_log2, __high2float(q23) * a.scale_log2);
        if (HP == 1) *reinterpret_cast<float4*>(qf + h * kHeadDim + lane * 4) = qv;
        *reinterpret_cast<float4*>(ocorr + h * kHeadDim + lane * 4) = make_float4(0.f, 0.f, 0.f, 0.f);
        float mx = fmaxf(fmaxf(fabsf(qv.x), fabsf(qv.y)), fmaxf(fabsf(qv.z), fabsf(qv.w)));
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        if (lane == 0) qexp_s[h] = float_exponent(mx);
      }
    }
    __syncwarp();

#pragma unroll 1
    for (int blk = blk_lo; blk < blk_hi; ++blk) {
      const bool buf_blk = blk >= a.n_blocks_c;
      if (!buf_blk && (blk >= c_seg_hi || blk < c_seg_lo)) {
        load_desc(sdc, blk);
        c_seg_lo = sdc->blk_start;
        c_seg_hi = c_seg_lo + sdc->nblk;
        c_shape = sdc->shape_id;
      }
      auto body = [&](auto shape_tag) {
      using S = decltype(shape_tag);
      constexpr bool is_buf = S::kBuf;
      constexpr int TU = HP == 1 ? S::tok_unroll : 1;     // unrolling of the per-token loops (latency, one head only)
      // ---------------- block geometry
      const int T = S::kDyn ? sdc->T : S::T;
      const int r_pad = S::kDyn ? sdc->r_pad : S::r_pad;
      const int k2k = S::kDyn ? 2 * sdc->k_k : S::k2k;
      const int k2v = S::kDyn ? 2 * a.cc.k_v : S::k2v;
      const int off_kscale = S::kDyn ? sdc->off_kscale : S::off_kscale;
      const int off_koval = S::kDyn ? sdc->off_koval : S::off_koval;
      const int off_koidx = S::kDyn ? sdc->off_koidx : S::off_koidx;
      const int off_kcodes = S::kDyn ? sdc->off_kcodes : S::off_kcodes;
      const int off_ak = S::kDyn ? sdc->off_ak : S::off_ak;
      const int o_av = S::kDyn ? sdc->off_av - sdc->off_vpart : S::off_av;
      const int o_vsz = S::kDyn ? sdc->off_vscale - sdc->off_vpart : S::off_vscale;
      const int o_voval = S::kDyn ? sdc->off_voval - sdc->off_vpart : S::off_voval;
      const int o_voidx = S::kDyn ? sdc->off_voidx - sdc->off_vpart : S::off_voidx;
      int valid_tokens = T;
      bool with_bk = false, with_bv = false;
      if (!is_buf) {
        with_bk = r_pad > 0 && (blk == c_seg_lo || blk == blk_lo);
        with_bv = r_pad > 0 && (blk == c_seg_hi - 1 || blk == blk_hi - 1);
      } else {
        valid_tokens = min(kSlab, a.buf_len - (blk - a.n_blocks_c) * kSlab);
      }
      const int nslab = T / kSlab;

      // ================================================================ key item
      unsigned char* stK = acquire();
      if (!alive) return;
      const unsigned char* kp = stK + a.bregion;
      float dmax_v = 0.f;
      int sexp_k[HP];                                 // per head: exponent of the sparse key term's fixed-point scale
      float c_zero[HP];                               // per head: sum over channels of q * zero-point
#pragma unroll
      for (int h = 0; h < HP; ++h) { sexp_k[h] = 0; c_zero[h] = 0.f; }

      if (with_bk) {
        // w = q B_K through the tensor cores, kept as the B operand of the low-rank key term
        const __half* bk = reinterpret_cast<const __half*>(stK);     // [r_pad][128]
        float wacc[NT][4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
          for (int i = 0; i < 4; ++i) wacc[nt][i] = 0.f;
#pragma unroll 2
        for (int kc = 0; kc < 8; ++kc) {
          uint32_t af[4] = {0u, 0u, 0u, 0u};
          if (gid < r_pad) {
            af[0] = *reinterpret_cast<const uint32_t*>(bk + gid * kHeadDim + 16 * kc + 2 * t);
            af[2] = *reinterpret_cast<const uint32_t*>(bk + gid * kHeadDim + 16 * kc + 2 * t + 8);
          }
          if (gid + 8 < r_pad) {
            af[1] = *reinterpret_cast<const uint32_t*>(bk + (gid + 8) * kHeadDim + 16 * kc + 2 * t);
            af[3] = *reinterpret_cast<const uint32_t*>(bk + (gid + 8) * kHeadDim + 16 * kc + 2 * t + 8);
          }
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) {
            uint32_t b0 = 0u, b1 = 0u;
            const int h = (gid >> 1) + 4 * nt;
            if ((gid & 1) == 0 && h < HPu) {
              const __half* qrow = qs + h * kHeadDim + 16 * kc + 2 * t;
              b0 = *reinterpret_cast<const uint32_t*>(qrow);
              b1 = *reinterpret_cast<const uint32_t*>(qrow + 8);
            }
            mma16816(wacc[nt], af, b0, b1);
          }
        }
        __syncwarp();
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {       // D[rho][col 2t] = w[rho][head t + 4nt]
          if (t + 4 * nt < HP) {
            wl[gid * WLS + t + 4 * nt] = wacc[nt][0] * a.scale_log2;
            wl[(gid + 8) * WLS + t + 4 * nt] = wacc[nt][2] * a.scale_log2;
          }
        }
        __syncwarp();
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          const int h = (gid >> 1) + 4 * nt;
          uint32_t hi0, lo0, hi1, lo1;
          split_hi_lo(wl[(2 * t) * WLS + (h & HMASK)], wl[(2 * t + 1) * WLS + (h & HMASK)], hi0, lo0);
          split_hi_lo(wl[(2 * t + 8) * WLS + (h & HMASK)], wl[(2 * t + 9) * WLS + (h & HMASK)], hi1, lo1);
          bw[nt][0] = (gid & 1) ? lo0 : hi0;
          bw[nt][1] = (gid & 1) ? lo1 : hi1;
        }
        __syncwarp();
      }

      // ---------------- B operand of the key scores: q * scale per channel, split hi / lo;
      //                  c_h = sum q * zero;  sparse key term scattered to its token
      {
        float sc4[4] = {1.f, 1.f, 1.f, 1.f}, zr4[4] = {0.f, 0.f, 0.f, 0.f};
        int ed = 0;
        if (!is_buf) {
          const float dmax_k = reinterpret_cast<const float*>(kp)[0];
          dmax_v = reinterpret_cast<const float*>(kp)[1];
          ed = float_exponent(dmax_k);
          const uint4 kz = reinterpret_cast<const uint4*>(kp + off_kscale)[lane];
          const uint32_t w4[4] = {kz.x, kz.y, kz.z, kz.w};
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            sc4[j] = __low2float(u32_as_h2(w4[j])) * kfac;
            zr4[j] = __high2float(u32_as_h2(w4[j]));
          }
        }
        float qS[HP][4];
        const int kc = lane >> 2, reg = (lane >> 1) & 1, tA = 2 * (lane & 1);
#pragma unroll
        for (int h = 0; h < HP; ++h) {
          if (h < HPu) {
            float4 qv;
            if (HP == 1) {
              qv = *reinterpret_cast<const float4*>(qf + h * kHeadDim + lane * 4);
            } else {
              const uint2 qh = *reinterpret_cast<const uint2*>(qs + h * kHeadDim + lane * 4);
              const __half2 q01 = u32_as_h2(qh.x), q23 = u32_as_h2(qh.y);
              qv = make_float4(__low2float(q01) * a.scale_log2, __high2float(q01) * a.scale_log2,
                               __low2float(q23) * a.scale_log2, __high2float(q23) * a.scale_log2);
            }
            uint32_t hiA, loA, hiB, loB;
            split_hi_lo(qv.x * sc4[0], qv.y * sc4[1], hiA, loA);
            split_hi_lo(qv.z * sc4[2], qv.w * sc4[3], hiB, loB);
            uint32_t* base = frag + ((h >> 2) * 8 + kc) * kFragStride + reg;
            const int cl = 2 * (h & 3);
            base[(4 * cl + tA) * 2] = hiA;
            base[(4 * (cl + 1) + tA) * 2] = loA;
            base[(4 * cl + tA + 1) * 2] = hiB;
            base[(4 * (cl + 1) + tA + 1) * 2] = loB;
            if (!is_buf) {
              float c = fmaf(qv.x, zr4[0], fmaf(qv.y, zr4[1], fmaf(qv.z, zr4[2], qv.w * zr4[3])));   // this lane's part
              if (HP != 4) {
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
              }
              const int sexp = clamp60(21 - qexp_s[h] - ed);
              const float S = pow2i(sexp);
              qS[h][0] = qv.x * S; qS[h][1] = qv.y * S; qS[h][2] = qv.z * S; qS[h][3] = qv.w * S;
              c_zero[h] = c; sexp_k[h] = sexp;
            }
          }
        }
        if (!is_buf && HP == 4) {            // c_zero of four heads: sums over the warp
          {
            // four sums at once: two exchange steps halve what a lane carries, a butterfly finishes the one value left
            // (head 2 * bit4 + bit3 of the lane), four broadcasts hand the sums back: 10 shuffles instead of 20
            float s0 = c_zero[0], s1 = c_zero[1];
            {
              const bool up = (lane & 16) != 0;
              const float send0 = up ? c_zero[0] : c_zero[2], keep0 = up ? c_zero[2] : c_zero[0];
              const float send1 = up ? c_zero[1] : c_zero[3], keep1 = up ? c_zero[3] : c_zero[1];
              s0 = keep0 + __shfl_xor_sync(0xffffffffu, send0, 16);
              s1 = keep1 + __shfl_xor_sync(0xffffffffu, send1, 16);
            }
            {
              const bool up = (lane & 8) != 0;
              const float send = up ? s0 : s1, keep = up ? s1 : s0;
              s0 = keep + __shfl_xor_sync(0xffffffffu, send, 8);
            }
#pragma unroll
            for (int o = 4; o > 0; o >>= 1) s0 += __shfl_xor_sync(0xffffffffu, s0, o);
#pragma unroll
            for (int h = 0; h < HP; ++h) c_zero[h] = __shfl_sync(0xffffffffu, s0, 8 * h);
          }
        }
        if (!is_buf && k2k > 0) {
          auto k_entry = [&](int j, float val, int idx) {
            const float d = val - zr4[j];
#pragma unroll
            for (int h = 0; h < HP; ++h)
              if (h < HPu) atomicAdd(&corr_k[h * maxT + idx], __float2int_rn(qS[h][j] * d));
          };
          if (k2k == 2) {
            const uint4 ov = reinterpret_cast<const uint4*>(kp + off_koval)[lane];
            const uint2 oi = reinterpret_cast<const uint2*>(kp + off_koidx)[lane];
            const uint32_t o4[4] = {ov.x, ov.y, ov.z, ov.w};
            const uint32_t i2[2] = {oi.x, oi.y};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              k_entry(j, __low2float(u32_as_h2(o4[j])), (i2[j >> 1] >> (16 * (j & 1))) & 0xFFu);
              k_entry(j, __high2float(u32_as_h2(o4[j])), (i2[j >> 1] >> (16 * (j & 1) + 8)) & 0xFFu);
            }
          } else if (k2k == 4) {
            // this lane's 4 channels x 4 entries: 32 bytes of values, 16 bytes of token indices
            const uint4 ova = reinterpret_cast<const uint4*>(kp + off_koval)[2 * lane];
            const uint4 ovb = reinterpret_cast<const uint4*>(kp + off_koval)[2 * lane + 1];
            const uint4 oi = reinterpret_cast<const uint4*>(kp + off_koidx)[lane];
            const uint32_t o8[8] = {ova.x, ova.y, ova.z, ova.w, ovb.x, ovb.y, ovb.z, ovb.w};
            const uint32_t i4[4] = {oi.x, oi.y, oi.z, oi.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              k_entry(j, __low2float(u32_as_h2(o8[2 * j])), i4[j] & 0xFFu);
              k_entry(j, __high2float(u32_as_h2(o8[2 * j])), (i4[j] >> 8) & 0xFFu);
              k_entry(j, __low2float(u32_as_h2(o8[2 * j + 1])), (i4[j] >> 16) & 0xFFu);
              k_entry(j, __high2float(u32_as_h2(o8[2 * j + 1])), i4[j] >> 24);
            }
          } else {
            const __half* ov = reinterpret_cast<const __half*>(kp + off_koval) + lane * 4 * k2k;
            const unsigned char* oi = kp + off_koidx + lane * 4 * k2k;
#pragma unroll
            for (int j = 0; j < 4; ++j)
#pragma unroll 1
              for (int e = 0; e < k2k; ++e) k_entry(j, __half2float(ov[j * k2k + e]), oi[j * k2k + e]);
          }
        }
      }
      __syncwarp();
      uint32_t bq[NT][8][2];
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int kc = 0; kc < 8; ++kc) {
          const uint2 v = *reinterpret_cast<const uint2*>(frag + (nt * 8 + kc) * kFragStride + ((gid & CMASK) * 4 + t) * 2);
          bq[nt][kc][0] = v.x; bq[nt][kc][1] = v.y;
        }

      // ---------------- key scores, slab by slab; scores go to shared memory
      {
        int psoff[NT];                                  // this lane's first score slot (head t + 4 nt, token gid)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) psoff[nt] = (t + 4 * nt) * maxT + gid;
        const bool pa0 = 2 * t < r_pad, pa1 = 2 * t + 8 < r_pad;
        auto k_slabs = [&](auto buf_tag) {
          constexpr bool kBuf = decltype(buf_tag)::value;
          const uint4* cwp = reinterpret_cast<const uint4*>(kp + off_kcodes) + lane;
          const __half* akp = reinterpret_cast<const __half*>(kp + off_ak) + gid * r_pad + 2 * t;
          const int ak8 = 8 * r_pad, ak_step = kSlab * r_pad;
          int tok0 = 0;
#pragma unroll (S::unroll)
          for (int slab = 0; slab < nslab; ++slab) {
            float acc[2][NT][4];
#pragma unroll
            for (int hf = 0; hf < 2; ++hf)
#pragma unroll
              for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int i = 0; i < 4; ++i) acc[hf][nt][i] = 0.f;
            uint4 w0 = make_uint4(0u, 0u, 0u, 0u), w1 = w0;
            if (!kBuf) {
              w0 = cwp[0];
              if (BITS == 4) w1 = cwp[32];
              cwp += SLABW;
            }
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {            // channel chunks 4 hf .. 4 hf + 3
              uint32_t af[4][4];
              if (!kBuf) {
                if (BITS == 2) {
                  uint32_t r[8];
                  unpack_word<2>(hf == 0 ? w0.x : w0.y, r);
#pragma unroll
                  for (int u2 = 0; u2 < 8; ++u2) af[u2 >> 1][(u2 & 1) * 2] = r[u2];
                  unpack_word<2>(hf == 0 ? w0.z : w0.w, r);
#pragma unroll
                  for (int u2 = 0; u2 < 8; ++u2) af[u2 >> 1][(u2 & 1) * 2 + 1] = r[u2];
                } else {
#pragma unroll
                  for (int th = 0; th < 2; ++th) {
                    const uint4 w = th == 0 ? w0 : w1;
                    uint32_t r[4];
                    unpack_word<4>(hf == 0 ? w.x : w.z, r);
#pragma unroll
                    for (int u2 = 0; u2 < 4; ++u2) af[u2 >> 1][(u2 & 1) * 2 + th] = r[u2];
                    unpack_word<4>(hf == 0 ? w.y : w.w, r);
#pragma unroll
                    for (int u2 = 0; u2 < 4; ++u2) af[2 + (u2 >> 1)][(u2 & 1) * 2 + th] = r[u2];
                  }
                }
              } else {
#pragma unroll
                for (int k4 = 0; k4 < 4; ++k4)
                  ldmatrix_x4(af[k4], stK + ((lane & 7) + 8 * ((lane >> 3) & 1)) * kBufPitch +
                                          (16 * (4 * hf + k4) + 8 * (lane >> 4)) * 2);
              }
#pragma unroll
              for (int k4 = 0; k4 < 4; ++k4)
#pragma unroll
                for (int nt = 0; nt < NT; ++nt)
                  mma16816(acc[hf][nt], af[k4], bq[nt][4 * hf + k4][0], bq[nt][4 * hf + k4][1]);
            }
            if (!kBuf) {                                // low-rank key term: A_K rows times w (zero rows when r = 0)
#pragma unroll
              for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int i = 0; i < 4; ++i) acc[1][nt][i] *= kKeyBack;
              uint32_t aa[4] = {0u, 0u, 0u, 0u};
              if (pa0) {
                aa[0] = *reinterpret_cast<const uint32_t*>(akp);
                aa[1] = *reinterpret_cast<const uint32_t*>(akp + ak8);
              }
              if (pa1) {
                aa[2] = *reinterpret_cast<const uint32_t*>(akp + 8);
                aa[3] = *reinterpret_cast<const uint32_t*>(akp + ak8 + 8);
              }
              akp += ak_step;
#pragma unroll
              for (int nt = 0; nt < NT; ++nt) mma16816(acc[1][nt], aa, bw[nt][0], bw[nt][1]);
            }
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
              if (t + 4 * nt < HPu) {
                // raw sums only: the zero-point constant and the sparse term are added in the softmax pass
                const float back = kBuf ? 1.f : kKeyBack;
                const float v0 = fmaf(acc[0][nt][0] + acc[0][nt][1], back, acc[1][nt][0] + acc[1][nt][1]);
                const float v1 = fmaf(acc[0][nt][2] + acc[0][nt][3], back, acc[1][nt][2] + acc[1][nt][3]);
                float* pr = ps + psoff[nt] + tok0;
                pr[0] = v0; pr[8] = v1;
              }
            }
            tok0 += kSlab;
          }
        };
        k_slabs(std::integral_constant<bool, is_buf>{});
      }
      release();                                      // the key item is consumed

      // after the running maximum grew: everything accumulated so far is scaled by alpha (per head)
      auto apply_alpha = [&](const float (&alpha)[HP]) {                                      // warp-uniform: m_run is the same in every lane
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) {
            float al = alpha[4 * nt];
#pragma unroll
            for (int hh = 1; hh < 4; ++hh)
              if (4 * nt + hh < HP && t == hh) al = alpha[4 * nt + hh];
#pragma unroll
            for (int i = 0; i < 4; ++i) U[nt][i] *= al;
#pragma unroll
            for (int mt = 0; mt < 8; ++mt)
#pragma unroll
              for (int i = 0; i < 4; ++i) O[mt][nt][i] *= al;
          }
#pragma unroll
          for (int h = 0; h < HP; ++h) {
            if (h < HPu) {
#pragma unroll
              for (int g = 0; g < NGV; ++g) cm[h][g] *= alpha[h];
              float4* oc = reinterpret_cast<float4*>(ocorr + h * kHeadDim + lane * 4);
              float4 v = *oc;
              v.x *= alpha[h]; v.y *= alpha[h]; v.z *= alpha[h]; v.w *= alpha[h];
              *oc = v;
            }
          }
              };
      // Up to four query heads and a compile-time block shape: the softmax, the value operands and the value outliers
      // run as one pass over this lane's token pairs with the probabilities in registers (the value item is waited
      // for first, since its scales are needed).  Every other case takes the separate passes below.
      constexpr bool kFuse = HP <= 4 && !S::kDyn && !is_buf;
      unsigned char* stV = nullptr;
      if (!kFuse) {
      // ---------------- online softmax over the block: one rescale at most
      {
        float alpha[HP];
        bool grew = false;
#pragma unroll
        for (int h = 0; h < HP; ++h) {
          alpha[h] = 1.f;
          if (h < HPu) {
            float* row = ps + h * maxT;
            int* crow = corr_k + h * maxT;
            const float Sik = pow2i(-sexp_k[h]);
            float mx = -INFINITY;
#pragma unroll (TU)
            for (int tk = lane; tk < valid_tokens; tk += 32) {
              float v = row[tk] + c_zero[h];
              if (!is_buf && k2k > 0) {
                v = fmaf((float)crow[tk], Sik, v);
                crow[tk] = 0;
              }
              row[tk] = v;
              mx = fmaxf(mx, v);
            }
            mx = warp_max(mx);
            const float m_new = fmaxf(m_run[h], mx);       // finite: every block holds a valid token
            if (m_new > m_run[h]) {
              alpha[h] = exp2f(m_run[h] - m_new);
              grew = true;
              m_run[h] = m_new;
            }
            float l = 0.f;
#pragma unroll (TU)
            for (int tk = lane; tk < T; tk += 32) {
              const float p = tk < valid_tokens ? exp2f(row[tk] - m_new) : 0.f;   // tokens past the end of the buffer
              l += p;
              row[tk] = p;
            }
            l_run[h] = fmaf(l_run[h], alpha[h], l);
          }
        }
        if (grew) apply_alpha(alpha);
      }
      __syncwarp();
      }

      // ================================================================ value item
      stV = acquire();
      if (!alive) return;
      const unsigned char* vp = stV + a.bregion;          // value part of the record
      uint32_t* fragV = frag;                                         // [NT][NGV][nslab] rows of kFragStride words
      uint32_t* fragP = frag + NT * NGV * nslab * kFragStride;        // [NT][nslab]
      if (is_buf && valid_tokens < kSlab) {
        // rows past the end of the buffer hold stale bytes: clear them (0 * garbage must stay 0)
        for (int i = lane; i < (kSlab - valid_tokens) * (kBufPitch / 16); i += 32) {
          const int r = valid_tokens + i / (kBufPitch / 16), cc = i % (kBufPitch / 16);
          reinterpret_cast<uint4*>(stV + r * kBufPitch)[cc] = make_uint4(0u, 0u, 0u, 0u);
        }
        fence_async_smem();
      }

      if (kFuse) {
        constexpr int NPR = S::T >= 64 ? S::T / 64 : 1;   // token pairs per lane
        float2 sc[HP][NPR];
        float alpha[HP], m_new[HP];
        bool grew = false;
#pragma unroll
        for (int h = 0; h < HP; ++h) {
          alpha[h] = 1.f; m_new[h] = 0.f;
          if (h < HPu) {
            const float Sik = pow2i(-sexp_k[h]);
            float mx = -INFINITY;
#pragma unroll
            for (int i = 0; i < NPR; ++i) {
              const int tp = 2 * (lane + 32 * i);
              float2 v = *reinterpret_cast<const float2*>(ps + h * maxT + tp);
              v.x += c_zero[h]; v.y += c_zero[h];
              if (k2k > 0) {
                const int2 c = *reinterpret_cast<const int2*>(corr_k + h * maxT + tp);
                v.x = fmaf((float)c.x, Sik, v.x);
                v.y = fmaf((float)c.y, Sik, v.y);
                *reinterpret_cast<int2*>(corr_k + h * maxT + tp) = make_int2(0, 0);
              }
              sc[h][i] = v;
              mx = fmaxf(mx, fmaxf(v.x, v.y));
            }
            mx = warp_max(mx);
            m_new[h] = fmaxf(m_run[h], mx);
            if (m_new[h] > m_run[h]) {                    // warp-uniform
              alpha[h] = exp2f(m_run[h] - m_new[h]);
              m_run[h] = m_new[h];
              grew = true;
            }
          }
        }
        if (grew) apply_alpha(alpha);
        const float Sv = pow2i(clamp60(21 - float_exponent(dmax_v)));
        const __half2* vsz = reinterpret_cast<const __half2*>(vp + o_vsz);
        float l[HP];
#pragma unroll
        for (int h = 0; h < HP; ++h) l[h] = 0.f;
#pragma unroll
        for (int i = 0; i < NPR; ++i) {
          const int pr = lane + 32 * i, tp = 2 * pr;
          const int s = pr >> 3, pi = pr & 7, tw = pi & 3, rg = pi >> 2;
          float p[HP][2];
          __half2 z[2][NGV];
#pragma unroll
          for (int g = 0; g < NGV; ++g) { z[0][g] = vsz[tp * NGV + g]; z[1][g] = vsz[(tp + 1) * NGV + g]; }
#pragma unroll
          for (int h = 0; h < HP; ++h) {
            p[h][0] = p[h][1] = 0.f;
            if (h < HPu) {
              const float p0 = exp2f(sc[h][i].x - m_new[h]), p1 = exp2f(sc[h][i].y - m_new[h]);
              p[h][0] = p0; p[h][1] = p1;
              l[h] += p0 + p1;
              const int col = 2 * (h & 3);
              uint32_t hi, lo;
              split_hi_lo(p0, p1, hi, lo);
              uint32_t* bp = fragP + ((h >> 2) * nslab + s) * kFragStride + rg;
              bp[(col * 4 + tw) * 2] = hi;
              bp[((col + 1) * 4 + tw) * 2] = lo;
#pragma unroll
              for (int g = 0; g < NGV; ++g) {
                split_hi_lo(p0 * __low2float(z[0][g]), p1 * __low2float(z[1][g]), hi, lo);
                uint32_t* bv = fragV + (((h >> 2) * NGV + g) * nslab + s) * kFragStride + rg;
                bv[(col * 4 + tw) * 2] = hi;
                bv[((col + 1) * 4 + tw) * 2] = lo;
                cm[h][g] = fmaf(p0, __high2float(z[0][g]), fmaf(p1, __high2float(z[1][g]), cm[h][g]));
              }
            }
          }
          if (k2v > 0) {                                  // sparse value term of the two tokens, scattered in fixed point
#pragma unroll
            for (int e2 = 0; e2 < 2; ++e2) {
              const int tk = tp + e2;
              auto v_entry = [&](int g, float val, int idx) {
                const float d = (val - __high2float(z[e2][g])) * Sv;
#pragma unroll
                for (int h = 0; h < HP; ++h)
                  if (h < HPu) atomicAdd(&corr_v[h * kHeadDim + g * GV + idx], __float2int_rn(p[h][e2] * d));
              };
              if (NGV * k2v == 4) {
                const uint2 ov = reinterpret_cast<const uint2*>(vp + o_voval)[tk];
                const uint32_t oi = reinterpret_cast<const uint32_t*>(vp + o_voidx)[tk];
                v_entry(0, __low2float(u32_as_h2(ov.x)), oi & 0xFFu);
                v_entry(0, __high2float(u32_as_h2(ov.x)), (oi >> 8) & 0xFFu);
                v_entry(NGV == 2 ? 1 : 0, __low2float(u32_as_h2(ov.y)), (oi >> 16) & 0xFFu);
                v_entry(NGV == 2 ? 1 : 0, __high2float(u32_as_h2(ov.y)), oi >> 24);
              } else {
                const __half* ov = reinterpret_cast<const __half*>(vp + o_voval) + (size_t)tk * NGV * k2v;
                const unsigned char* oi = vp + o_voidx + (size_t)tk * NGV * k2v;
#pragma unroll
                for (int g = 0; g < NGV; ++g)
#pragma unroll 1
                  for (int e = 0; e < k2v; ++e) v_entry(g, __half2float(ov[g * k2v + e]), oi[g * k2v + e]);
              }
            }
          }
        }
#pragma unroll
        for (int h = 0; h < HP; ++h)
          if (h < HPu) l_run[h] = fmaf(l_run[h], alpha[h], l[h]);
      } else {
      // ---------------- B operands of the value products: p * scale (per token and group) and p, split hi / lo;
      //                  the zero-point term goes to the fp32 side sums cm
#pragma unroll (TU)
      for (int pr = lane; pr < T / 2; pr += 32) {      // this lane's token pairs
        const int s = pr >> 3, pi = pr & 7, tw = pi & 3, rg = pi >> 2;
        const int tp = 2 * pr;
#pragma unroll
        for (int h = 0; h < HP; ++h) {
          if (h < HPu) {
            const float2 pp = *reinterpret_cast<const float2*>(ps + h * maxT + tp);
            const int col = 2 * (h & 3);
            uint32_t hi, lo;
            {
              split_hi_lo(pp.x, pp.y, hi, lo);
              uint32_t* bp = fragP + ((h >> 2) * nslab + s) * kFragStride + rg;
              bp[(col * 4 + tw) * 2] = hi;
              bp[((col + 1) * 4 + tw) * 2] = lo;
            }
            if (!is_buf) {
              const __half2* vsz = reinterpret_cast<const __half2*>(vp + o_vsz) + tp * NGV;
#pragma unroll
              for (int g = 0; g < NGV; ++g) {
                const __half2 z0 = vsz[g], z1 = vsz[NGV + g];
                split_hi_lo(pp.x * __low2float(z0), pp.y * __low2float(z1), hi, lo);
                uint32_t* bv = fragV + (((h >> 2) * NGV + g) * nslab + s) * kFragStride + rg;
                bv[(col * 4 + tw) * 2] = hi;
                bv[((col + 1) * 4 + tw) * 2] = lo;
                cm[h][g] = fmaf(pp.x, __high2float(z0), fmaf(pp.y, __high2float(z1), cm[h][g]));
              }
            }
          }
        }
      }
      }
      __syncwarp();

      // ---------------- values: out += sum_tok (p * scale) * code on the tensor cores, low rank on the side
      {
        const bool pv0 = gid < r_pad, pv1 = gid + 8 < r_pad;
        auto v_slabs = [&](auto buf_tag) {
          constexpr bool kBuf = decltype(buf_tag)::value;
          const uint4* cwp = reinterpret_cast<const uint4*>(vp) + lane;
          const __half* avp = reinterpret_cast<const __half*>(vp + o_av) + gid * kSlab + 2 * t;
          const uint32_t* fvp = fragV + ((gid & CMASK) * 4 + t) * 2;
          const uint32_t* fpp = fragP + ((gid & CMASK) * 4 + t) * 2;
          const int fstep = nslab * kFragStride, av_step = kSlab * r_pad;
#pragma unroll (S::unroll)
          for (int slab = 0; slab < nslab; ++slab) {
            uint32_t bp[NT][2];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
              const uint2 v = *reinterpret_cast<const uint2*>(fpp + nt * fstep);
              bp[nt][0] = v.x; bp[nt][1] = v.y;
            }
            fpp += kFragStride;
            if (!kBuf) {
              uint32_t bv[NT][NGV][2];
#pragma unroll
              for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int g = 0; g < NGV; ++g) {
                  const uint2 v = *reinterpret_cast<const uint2*>(fvp + (nt * NGV + g) * fstep);
                  bv[nt][g][0] = v.x; bv[nt][g][1] = v.y;
                }
              fvp += kFragStride;
              constexpr int TPP = 8 / BITS;               // channel tiles per pair of words
#pragma unroll
              for (int pl = 0; pl < BITS / 2; ++pl) {
                const uint4 w = cwp[pl * 32];
                const uint32_t wv[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                for (int wp = 0; wp < 2; ++wp) {
                  uint32_t rA[16 / BITS], rB[16 / BITS];
                  unpack_word<BITS>(wv[2 * wp], rA);
                  unpack_word<BITS>(wv[2 * wp + 1], rB);
#pragma unroll
                  for (int j = 0; j < TPP; ++j) {
                    const int mt = TPP * (2 * pl + wp) + j, g = (mt * 16) / GV;
                    const uint32_t av[4] = {rA[2 * j], rA[2 * j + 1], rB[2 * j], rB[2 * j + 1]};
#pragma unroll
                    for (int nt = 0; nt < NT; ++nt) mma16816(O[mt][nt], av, bv[nt][g][0], bv[nt][g][1]);
                  }
                }
              }
              cwp += SLABW;
              // low-rank value term, first product: U = A_V^T p (zero rows when r = 0)
              uint32_t aa[4] = {0u, 0u, 0u, 0u};
              if (pv0) {
                aa[0] = *reinterpret_cast<const uint32_t*>(avp);
                aa[2] = *reinterpret_cast<const uint32_t*>(avp + 8);
              }
              if (pv1) {
                aa[1] = *reinterpret_cast<const uint32_t*>(avp + 8 * kSlab);
                aa[3] = *reinterpret_cast<const uint32_t*>(avp + 8 * kSlab + 8);
              }
              avp += av_step;
#pragma unroll
              for (int nt = 0; nt < NT; ++nt) mma16816(U[nt], aa, bp[nt][0], bp[nt][1]);
            } else {
#pragma unroll
              for (int mt = 0; mt < 8; ++mt) {
                uint32_t av[4];
                ldmatrix_x4_trans(av, stV + ((lane & 7) + 8 * (lane >> 4)) * kBufPitch + (16 * mt + 8 * ((lane >> 3) & 1)) * 2);
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                  if (o_plain) mma16816(O[mt][nt], av, bp[nt][0], bp[nt][1]);
                  else add_scaled(O[mt][nt], mt, av, bp[nt][0], bp[nt][1]);
                }
              }
            }
          }
        };
        v_slabs(std::integral_constant<bool, is_buf>{});
        if (!is_buf && r_pad > 0) u_pending = true;
      }

      // ---------------- sparse value term: p[tok] * (x - zero[tok, g]) scattered to the outlier's channel
      if (!is_buf && k2v > 0) {
        const int sexp = clamp60(21 - float_exponent(dmax_v));
        const float S = pow2i(sexp), Si = pow2i(-sexp);
        const __half2* vsz = reinterpret_cast<const __half2*>(vp + o_vsz);
        const unsigned char* voval = vp + o_voval;
        const unsigned char* voidx = vp + o_voidx;
#pragma unroll (TU)
        for (int tk = lane; tk < (kFuse ? 0 : T); tk += 32) {      // the fused pass above has scattered them already
          float pS[HP];
#pragma unroll
          for (int h = 0; h < HP; ++h) pS[h] = h < HPu ? ps[h * maxT + tk] * S : 0.f;
          auto v_entry = [&](int g, float val, int idx) {
            const float d = val - __high2float(vsz[tk * NGV + g]);
            const int ch = g * GV + idx;
#pragma unroll
            for (int h = 0; h < HP; ++h)
              if (h < HPu) atomicAdd(&corr_v[h * kHeadDim + ch], __float2int_rn(pS[h] * d));
          };
          if (NGV * k2v == 4) {
            const uint2 ov = reinterpret_cast<const uint2*>(voval)[tk];
            const uint32_t oi = reinterpret_cast<const uint32_t*>(voidx)[tk];
            v_entry(0, __low2float(u32_as_h2(ov.x)), oi & 0xFFu);
            v_entry(0, __high2float(u32_as_h2(ov.x)), (oi >> 8) & 0xFFu);
            v_entry(NGV == 2 ? 1 : 0, __low2float(u32_as_h2(ov.y)), (oi >> 16) & 0xFFu);
            v_entry(NGV == 2 ? 1 : 0, __high2float(u32_as_h2(ov.y)), oi >> 24);
          } else {
            const __half* ov = reinterpret_cast<const __half*>(voval) + (size_t)tk * NGV * k2v;
            const unsigned char* oi = voidx + (size_t)tk * NGV * k2v;
#pragma unroll
            for (int g = 0; g < NGV; ++g)
#pragma unroll 1
              for (int e = 0; e < k2v; ++e) v_entry(g, __half2float(ov[g * k2v + e]), oi[g * k2v + e]);
          }
        }
        __syncwarp();
#pragma unroll
        for (int h = 0; h < HP; ++h) {
          if (h < HPu) {
            int4* cv = reinterpret_cast<int4*>(corr_v + h * kHeadDim) + lane;
            float4* oc = reinterpret_cast<float4*>(ocorr + h * kHeadDim) + lane;
            const int4 v = *cv;
            *cv = make_int4(0, 0, 0, 0);
            float4 o = *oc;
            o.x = fmaf((float)v.x, Si, o.x);
            o.y = fmaf((float)v.y, Si, o.y);
            o.z = fmaf((float)v.z, Si, o.z);
            o.w = fmaf((float)v.w, Si, o.w);
            *oc = o;
          }
        }
      }

      // ---------------- end of a segment (or of this warp's share of it): out += B_V U
      if (with_bv && u_pending) {
        __syncwarp();
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          if (t + 4 * nt < HP) {
            wl[gid * WLS + t + 4 * nt] = U[nt][0] + U[nt][1];
            wl[(gid + 8) * WLS + t + 4 * nt] = U[nt][2] + U[nt][3];
          }
#pragma unroll
          for (int i = 0; i < 4; ++i) U[nt][i] = 0.f;
        }
        __syncwarp();
        uint32_t bu[NT][2];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          const int h = (gid >> 1) + 4 * nt;
          uint32_t hi0, lo0, hi1, lo1;
          split_hi_lo(wl[(2 * t) * WLS + (h & HMASK)], wl[(2 * t + 1) * WLS + (h & HMASK)], hi0, lo0);
          split_hi_lo(wl[(2 * t + 8) * WLS + (h & HMASK)], wl[(2 * t + 9) * WLS + (h & HMASK)], hi1, lo1);
          bu[nt][0] = (gid & 1) ? lo0 : hi0;
          bu[nt][1] = (gid & 1) ? lo1 : hi1;
        }
        const __half* bvf = reinterpret_cast<const __half*>(stV);      // B_V [128][r_pad]
#pragma unroll
        for (int mt = 0; mt < 8; ++mt) {
          uint32_t aa[4] = {0u, 0u, 0u, 0u};
          const __half* r0 = bvf + (16 * mt + gid) * r_pad, *r1 = bvf + (16 * mt + gid + 8) * r_pad;
          if (2 * t < r_pad) {
            aa[0] = *reinterpret_cast<const uint32_t*>(r0 + 2 * t);
            aa[1] = *reinterpret_cast<const uint32_t*>(r1 + 2 * t);
          }
          if (2 * t + 8 < r_pad) {
            aa[2] = *reinterpret_cast<const uint32_t*>(r0 + 2 * t + 8);
            aa[3] = *reinterpret_cast<const uint32_t*>(r1 + 2 * t + 8);
          }
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) add_scaled(O[mt][nt], mt, aa, bu[nt][0], bu[nt][1]);
        }
        u_pending = false;
      }
      release();                                      // the value item is consumed
      };
      if (buf_blk) body(BufShape{});
      else if (NGV == 2 && c_shape == 1) body(ShapeA1<BITS>{});
      else if (NGV == 2 && c_shape == 2) body(ShapeA2<BITS>{});
      else if (NGV == 1 && c_shape == 3) body(ShapeB1<BITS>{});
      else if (NGV == 1 && c_shape == 4) body(ShapeB2<BITS>{});
      else body(DynShape{});
      if (!alive) break;
    }
    if (!alive) break;

    // ---------------- partial result of this unit: (m, l, o) per head
    int n_parts, slot;
    if (a.aligned) {
      n_parts = parts_u;
      slot = part;
    } else {
      const long long F = (long long)a.cc.BH * passes * NB, NW = gridDim.x;
      const long long bflat = (long long)u * NB, eflat = bflat + NB;
      const long long w_first = ((bflat + 1) * NW + F - 1) / F - 1;
      const long long w_last = (eflat * NW + F - 1) / F - 1;
      n_parts = (int)(w_last - w_first + 1);
      slot = (int)(blockIdx.x - w_first);
    }
    float* part_base = a.partial + ((size_t)u * a.max_parts + slot) * (HP * kPartRow);
    float cm_own[NT][NGV], m_own[NT], l_own[NT];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      m_own[nt] = 0.f; l_own[nt] = 0.f;
#pragma unroll
      for (int g = 0; g < NGV; ++g) cm_own[nt][g] = 0.f;
    }
#pragma unroll
    for (int h = 0; h < HP; ++h) {
      float l = l_run[h];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
      if ((h & 3) == t) { m_own[h >> 2] = m_run[h]; l_own[h >> 2] = l; }
#pragma unroll
      for (int g = 0; g < NGV; ++g) {
        float c = cm[h][g];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
        if ((h & 3) == t) cm_own[h >> 2][g] = c;
      }
    }
    __syncwarp();
    // the tensor-core part of the output joins the sparse part in shared memory, so that the partial goes out as
    // one 16-byte store per lane and head
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      const int h = t + 4 * nt;
      if (h < HPu) {
#pragma unroll
        for (int mt = 0; mt < 8; ++mt)
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            const int ch = 16 * mt + gid + 8 * half;
            const float back = o_plain ? 1.f : (float)(1 << (24 - row_shift(mt, half)));
            ocorr[h * kHeadDim + ch] += fmaf(O[mt][nt][2 * half] + O[mt][nt][2 * half + 1], back, cm_own[nt][(mt * 16) / GV]);
          }
        if (gid == 0) { part_base[h * kPartRow + 128] = m_own[nt]; part_base[h * kPartRow + 129] = l_own[nt]; }
      }
    }
    __syncwarp();
#pragma unroll
    for (int h = 0; h < HP; ++h)
      if (h < HPu)
        reinterpret_cast<float4*>(part_base + h * kPartRow)[lane] = reinterpret_cast<const float4*>(ocorr + h * kHeadDim)[lane];
    // The ticket is one acquire-release atomic at device scope: it publishes this warp's partial (the warp barrier
    // before it orders the other lanes' stores) and, for the warp that takes the last ticket, makes the others' visible.
    __syncwarp();
    int last = 0;
    if (lane == 0) {
      int old;
      asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], 1;" : "=r"(old) : "l"(a.tickets + u) : "memory");
      last = old == n_parts - 1;
    }
    last = __shfl_sync(0xffffffffu, last, 0);
    if (last) {
      const float* pb = a.partial + (size_t)u * a.max_parts * (HP * kPartRow);
      const size_t pstride = (size_t)HP * kPartRow;
      for (int h = 0; h < HPu; ++h) {
        // Chunks of up to 16 partials: every load of a chunk (lane i: max and denominator of partial i; all lanes: their
        // four channels of every partial) is issued before anything is used, so a chunk costs one round trip to L2.
        float M = -INFINITY, den = 0.f, n0 = 0.f, n1 = 0.f, n2 = 0.f, n3 = 0.f;
        for (int base = 0; base < n_parts; base += 16) {
          const int cnt = min(16, n_parts - base);
          const float* ph = pb + (size_t)base * pstride + h * kPartRow;
          float mi = -INFINITY, li = 0.f;
          if (lane < cnt) { mi = __ldcg(ph + lane * pstride + 128); li = __ldcg(ph + lane * pstride + 129); }
          float4 v[16];
#pragma unroll
          for (int j = 0; j < 16; ++j)
            v[j] = j < cnt ? __ldcg(reinterpret_cast<const float4*>(ph + j * pstride) + lane) : make_float4(0.f, 0.f, 0.f, 0.f);
          float cm_ = mi;
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) cm_ = fmaxf(cm_, __shfl_xor_sync(0xffffffffu, cm_, o));
          const float Mn = fmaxf(M, cm_);
          const float resc = M == -INFINITY ? 0.f : exp2f(M - Mn);
          const float wgt = mi == -INFINITY ? 0.f : exp2f(mi - Mn);
          float dsum = wgt * li;
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) dsum += __shfl_xor_sync(0xffffffffu, dsum, o);
          den = fmaf(den, resc, dsum);
          n0 *= resc; n1 *= resc; n2 *= resc; n3 *= resc;
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const float wj = __shfl_sync(0xffffffffu, wgt, j);
            n0 = fmaf(wj, v[j].x, n0); n1 = fmaf(wj, v[j].y, n1); n2 = fmaf(wj, v[j].z, n2); n3 = fmaf(wj, v[j].w, n3);
          }
          M = Mn;
        }
        const float inv = 1.0f / den;
        *reinterpret_cast<float4*>(a.out + (size_t)(hq0 + h) * kHeadDim + lane * 4) =
            make_float4(n0 * inv, n1 * inv, n2 * inv, n3 * inv);
      }
      if (lane == 0) a.tickets[u] = 0;
    }
    n_left -= blk_hi - blk_lo;
    blk_lo = 0;
    ++u;
  }
  // a warp that gave up still has copies in flight: let them land (bounded) before leaving
  if (!alive) {
    for (int i = 0; i < n_inflight; ++i) {
      for (int k = 0; k < kSpinLimit && !mbar_try(&bar[c_stage], (uint32_t)c_par); ++k) {}
      if (++c_stage == NS) { c_stage = 0; c_par ^= 1; }
    }
  }
}

// ------------------------------------------------------------------ host side
template <class Fn>
static bool with_decode_kernel(int bits, int heads, int ngv, Fn fn) {
  const int hp = heads == 1 ? 1 : (heads <= 4 ? 4 : 8);
#define GEAR_DEC_CASE(B, N, V) \
  if (bits == B && hp == N && ngv == V) { fn(gear_decode_kernel<B, N, V>); return true; }
#define GEAR_DEC_HEADS(B, V) GEAR_DEC_CASE(B, 1, V) GEAR_DEC_CASE(B, 4, V) GEAR_DEC_CASE(B, 8, V)
  GEAR_DEC_HEADS(2, 1) GEAR_DEC_HEADS(2, 2) GEAR_DEC_HEADS(2, 4) GEAR_DEC_HEADS(2, 8)
  GEAR_DEC_HEADS(4, 1) GEAR_DEC_HEADS(4, 2) GEAR_DEC_HEADS(4, 4) GEAR_DEC_HEADS(4, 8)
#undef GEAR_DEC_HEADS
#undef GEAR_DEC_CASE
  return false;
}

cudaError_t launch_decode(const DecodeArgs& a, int grid, cudaStream_t st) {
  cudaError_t e = cudaSuccess;
  const size_t smem = (size_t)a.ws.total;
  const bool ok = with_decode_kernel(a.cc.bits, a.group_heads, a.cc.ngv, [&](auto kern) {
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return;
    kern<<<grid, 32, smem, st>>>(a);
    e = cudaGetLastError();
  });
  if (!ok) return cudaErrorInvalidValue;
  if (e == cudaSuccess) count_launches(1);
  return e;
}

int decode_occupancy(int bits, int heads, int ngv, size_t smem) {
  int occ = 0;
  cudaError_t e = cudaErrorInvalidValue;
  with_decode_kernel(bits, heads, ngv, [&](auto kern) {
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e == cudaSuccess) e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kern, 32, smem);
  });
  if (e != cudaSuccess) { cudaGetLastError(); return 0; }
  return occ;
}

}  // namespace gear
