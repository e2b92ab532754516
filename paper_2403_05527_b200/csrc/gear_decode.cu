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

#include "gear_internal.cuh"

namespace gear {

constexpr int kBufPitch = 272;                  // bytes per fp16 row of a buffer slab in shared memory
constexpr int kBufItem = kSlab * kBufPitch;     // one slab of key rows or of value rows
constexpr int kSpinLimit = 4000000;
constexpr int kChunkSlabs = 4;                  // slabs whose scores are held in registers at once
constexpr int kChunkTok = kChunkSlabs * kSlab;
constexpr int kFragStride = 72;                 // 32-bit words per fragment row set (64 + padding against bank conflicts)

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
__device__ __forceinline__ uint32_t lop3_and_or(uint32_t x, uint32_t mask, uint32_t orv) {
  uint32_t r;
  asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(r) : "r"(x), "r"(mask), "r"(orv));
  return r;
}
__device__ __forceinline__ uint32_t h2_as_u32(__half2 h) { return *reinterpret_cast<uint32_t*>(&h); }
__device__ __forceinline__ __half2 u32_as_h2(uint32_t u) { return *reinterpret_cast<__half2*>(&u); }

// (x & mask) | 0x6400 puts each masked field into the mantissa of 1024.0; one
// half2 fma with exact constants brings it back to the integer code.
__device__ __forceinline__ uint32_t field_to_h2(uint32_t x, uint32_t mask, float inv_step, float offs) {
  const __half2 h = u32_as_h2(lop3_and_or(x, mask, 0x64006400u));
  return h2_as_u32(__hfma2(h, __float2half2_rn(inv_step), __float2half2_rn(offs)));
}
// One 32-bit word of codes -> its fragment registers r[0 .. 16/BITS).
template <int BITS>
__device__ __forceinline__ void unpack_word(uint32_t x, uint32_t* r) {
  if (BITS == 2) {
    const uint32_t y = x >> 10;
    r[0] = field_to_h2(x, 0x00030003u, 1.0f, -1024.0f);
    r[1] = field_to_h2(x, 0x000C000Cu, 0.25f, -256.0f);
    r[2] = field_to_h2(x, 0x00300030u, 0.0625f, -64.0f);
    r[3] = field_to_h2(x, 0x00C000C0u, 0.015625f, -16.0f);
    r[4] = field_to_h2(x, 0x03000300u, 0.00390625f, -4.0f);
    r[5] = field_to_h2(y, 0x00030003u, 1.0f, -1024.0f);
    r[6] = field_to_h2(y, 0x000C000Cu, 0.25f, -256.0f);
    r[7] = field_to_h2(y, 0x00300030u, 0.0625f, -64.0f);
  } else {
    const uint32_t y = x >> 8;
    r[0] = field_to_h2(x, 0x000F000Fu, 1.0f, -1024.0f);
    r[1] = field_to_h2(x, 0x00F000F0u, 0.0625f, -64.0f);
    r[2] = field_to_h2(y, 0x000F000Fu, 1.0f, -1024.0f);
    r[3] = field_to_h2(y, 0x00F000F0u, 0.0625f, -64.0f);
  }
}

// fp32 pair -> half2 of the high parts and half2 of the rounding remainders
__device__ __forceinline__ void split_hi_lo(float x0, float x1, uint32_t& hi, uint32_t& lo) {
  const __half2 h = __floats2half2_rn(x0, x1);
  hi = h2_as_u32(h);
  lo = h2_as_u32(__floats2half2_rn(x0 - __low2float(h), x1 - __high2float(h)));
}

__device__ __forceinline__ int float_exponent(float x) { return (int)((__float_as_uint(x) >> 23) & 0xFFu) - 127; }
// 2^e for |e| <= 60
__device__ __forceinline__ float pow2i(int e) { return __uint_as_float((uint32_t)(127 + e) << 23); }
__device__ __forceinline__ int clamp60(int e) { return max(-60, min(60, e)); }

// ------------------------------------------------------------------ shared memory plan (per warp)
bool decode_plan(int bits, int heads, int ngv, int max_kpart, int max_vpart, int max_bfac, int max_T, size_t smem_budget,
                 DecodeArgs* a) {
  (void)bits;
  const int NT = heads <= 4 ? 1 : 2, HP = 4 * NT;
  const int hpa = heads < HP ? heads : HP;
  const int bregion = round_up(max_bfac / 2, 128);
  int part = max_kpart > max_vpart ? max_kpart : max_vpart;
  int stage = bregion + part;
  if (stage < kBufItem) stage = kBufItem;
  stage = round_up(stage, 128);
  if (max_T < kSlab) max_T = kSlab;
  const int frag_rows = 8 > kChunkSlabs * (ngv + 1) ? 8 : kChunkSlabs * (ngv + 1);
  for (int ns = kMaxStages; ns >= 2; --ns) {
    WarpSmem w;
    int o = 0;
    w.ring = o;    o += ns * stage;
    w.sdp = o;     o += 128;
    w.sdc = o;     o += 128;
    w.qf = o;      o += hpa * kHeadDim * 4;
    w.qs = o;      o += hpa * kHeadDim * 2;
    w.frag = o;    o += NT * frag_rows * kFragStride * 4;
    w.corr_k = o;  o += hpa * max_T * 4;
    w.ps = o;      o += hpa * kChunkTok * 4;
    w.corr_v = o;  o += hpa * kHeadDim * 4;
    w.ocorr = o;   o += hpa * kHeadDim * 4;
    w.wl = o;      o += kMaxRank * HP * 4;
    w.misc = o;    o += 4 * HP * 4;
    w.total = round_up(o, 128);
    // prefer three stages with more resident warps over four stages with fewer
    if (ns == kMaxStages && (size_t)w.total * 10 > smem_budget) continue;
    if ((size_t)w.total > smem_budget) continue;
    a->nstage = ns; a->stage_bytes = stage; a->bregion = bregion; a->max_T = max_T; a->hpa = hpa; a->ws = w;
    return true;
  }
  return false;
}

// ------------------------------------------------------------------ the kernel
template <int BITS, int NT, int NGV>
__global__ void __launch_bounds__(32, NT == 1 ? 10 : 5) gear_decode_kernel(const __grid_constant__ DecodeArgs a) {
  constexpr int HP = 4 * NT;                      // query heads per pass
  constexpr int GV = kHeadDim / NGV;              // channels per value group
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ __align__(8) uint64_t bar[kMaxStages];

  const int lane = threadIdx.x, gid = lane >> 2, t = lane & 3;
  const int G = a.group_heads;
  const int passes = (G + HP - 1) / HP;
  const int maxT = a.max_T;
  const int NS = a.nstage;
  unsigned char* ring = smem + a.ws.ring;
  SegDesc* sdp = reinterpret_cast<SegDesc*>(smem + a.ws.sdp);
  SegDesc* sdc = reinterpret_cast<SegDesc*>(smem + a.ws.sdc);
  float* qf = reinterpret_cast<float*>(smem + a.ws.qf);          // [hpa][128] q * scale * log2(e)
  __half* qs = reinterpret_cast<__half*>(smem + a.ws.qs);        // [hpa][128] q
  uint32_t* frag = reinterpret_cast<uint32_t*>(smem + a.ws.frag);
  int* corr_k = reinterpret_cast<int*>(smem + a.ws.corr_k);      // [hpa][maxT]
  float* ps = reinterpret_cast<float*>(smem + a.ws.ps);          // [hpa][64]
  int* corr_v = reinterpret_cast<int*>(smem + a.ws.corr_v);      // [hpa][128]
  float* ocorr = reinterpret_cast<float*>(smem + a.ws.ocorr);    // [hpa][128]
  float* wl = reinterpret_cast<float*>(smem + a.ws.wl);          // [16][HP]
  int* qexp_s = reinterpret_cast<int*>(smem + a.ws.misc);        // [HP]
  float* alpha_s = reinterpret_cast<float*>(smem + a.ws.misc) + HP;

  // value-phase fragments share the region of the key-phase ones
  uint32_t* fragV = frag;                                        // [NT][NGV][4 slabs] rows of kFragStride words
  uint32_t* fragP = frag + NT * NGV * kChunkSlabs * kFragStride; // [NT][4 slabs]

  if (lane == 0)
    for (int s = 0; s < NS; ++s) mbar_init(&bar[s], 1);
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  for (int i = lane; i < (a.ws.corr_k - a.ws.frag) / 4; i += 32) frag[i] = 0u;
  for (int i = lane; i < a.hpa * maxT; i += 32) corr_k[i] = 0;
  for (int i = lane; i < a.hpa * kHeadDim; i += 32) corr_v[i] = 0;
  __syncwarp();

  // ---- this warp's range of the flat (unit, block) space; unit = (batch, kv head, head pass)
  const int nbuf_blocks = (a.buf_len + kSlab - 1) / kSlab;
  const int NB = a.n_blocks_c + nbuf_blocks;
  const long long F = (long long)a.cc.BH * passes * NB;
  const long long NW = gridDim.x, gw = blockIdx.x;
  const long long f0 = gw * F / NW, f1 = (gw + 1) * F / NW;
  if (f0 >= f1) return;                      // the host launches no more warps than blocks

  // ---- producer: two items per block (key part, value part), issued in order into ring stage n_issued % NS
  long long p_f = f0;
  int p_unit = (int)(f0 / NB);
  int p_blk = (int)(f0 - (long long)p_unit * NB);
  int p_share_lo = p_blk, p_half = 0, n_issued = 0, p_seg_lo = 0, p_seg_hi = 0;
  auto load_desc = [&](SegDesc* dst, int blk) {
    const int* src = reinterpret_cast<const int*>(a.table + a.blk2seg[blk]);
    __syncwarp();
    if (lane < (int)(sizeof(SegDesc) / 4)) reinterpret_cast<int*>(dst)[lane] = src[lane];
    __syncwarp();
  };
  auto issue = [&]() {
    if (p_f >= f1) return;
    const int s = n_issued % NS;
    unsigned char* dst = ring + (size_t)s * a.stage_bytes;
    if (p_blk < a.n_blocks_c) {
      if (p_blk < p_seg_lo || p_blk >= p_seg_hi) {
        load_desc(sdp, p_blk);
        p_seg_lo = sdp->blk_start;
        p_seg_hi = p_seg_lo + sdp->nblk;
      }
      if (lane == 0) {
        const int bl = p_blk - p_seg_lo;
        const int bh = p_unit / passes;
        const int hb = sdp->bfac_bytes >> 1;
        const unsigned char* src_b = a.arena + sdp->seg_base + (size_t)bh * sdp->bh_stride;
        const unsigned char* src_r = src_b + sdp->bfac_bytes + (size_t)bl * sdp->rec_bytes;
        if (p_half == 0) {
          const bool wb = hb > 0 && (bl == 0 || p_blk == p_share_lo);
          mbar_expect_tx(&bar[s], sdp->off_vpart + (wb ? hb : 0));
          if (wb) bulk_g2s(dst, src_b, hb, &bar[s]);
          bulk_g2s(dst + a.bregion, src_r, sdp->off_vpart, &bar[s]);
        } else {
          const bool wb = hb > 0 && (bl == p_seg_hi - p_seg_lo - 1 || p_f == f1 - 1);
          const int vbytes = sdp->rec_bytes - sdp->off_vpart;
          mbar_expect_tx(&bar[s], vbytes + (wb ? hb : 0));
          if (wb) bulk_g2s(dst, src_b + hb, hb, &bar[s]);
          bulk_g2s(dst + a.bregion, src_r + sdp->off_vpart, vbytes, &bar[s]);
        }
      }
    } else if (lane == 0) {
      const int j = p_blk - a.n_blocks_c;
      const int rows = min(kSlab, a.buf_len - j * kSlab);
      const int bh = p_unit / passes;
      const __half* src = (p_half == 0 ? a.buf_k : a.buf_v) + ((size_t)bh * a.cc.n_b + (size_t)j * kSlab) * kHeadDim;
      mbar_expect_tx(&bar[s], rows * 256);
      for (int r = 0; r < rows; ++r) bulk_g2s(dst + r * kBufPitch, src + r * kHeadDim, 256, &bar[s]);
    }
    ++n_issued;
    if (p_half == 0) {
      p_half = 1;
    } else {
      p_half = 0; ++p_f; ++p_blk;
      if (p_blk == NB) { p_blk = 0; ++p_unit; p_share_lo = 0; }
    }
  };
  for (int s = 0; s < NS; ++s) issue();

  int n_released = 0, item_k = 0, c_seg_lo = 0, c_seg_hi = 0;     // item_k: index of the current block's key item
  bool alive = true;
  // wait for item `idx`; returns its stage
  auto acquire = [&](int idx) -> unsigned char* {
    const int s = idx % NS;
    if (!mbar_wait(&bar[s], (uint32_t)((idx / NS) & 1), a.status)) { alive = false; return nullptr; }
    return ring + (size_t)s * a.stage_bytes;
  };
  auto release = [&]() {       // the oldest item is consumed (items are released in order): refill its stage
    __syncwarp();
    ++n_released;
    issue();
  };

  // ---- loop over the units this warp touches
  long long f = f0;
  while (f < f1 && alive) {
    const int u = (int)(f / NB);
    const int blk_lo = (int)(f - (long long)u * NB);
    const int blk_hi = (int)min((long long)NB, blk_lo + (f1 - f));
    const int bh = u / passes, pass = u - bh * passes;
    const int HPu = min(HP, G - pass * HP);
    const int hq0 = bh * G + pass * HP;                 // first query head of this pass

    // unit state
    float O[8][NT][4], U[NT][4], m_run[NT], l_run[NT], cm[HP][NGV];
    uint32_t bw[NT][2];                                  // low-rank key term: B operand (q B_K) of the current segment
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      m_run[nt] = -INFINITY; l_run[nt] = 0.f; bw[nt][0] = bw[nt][1] = 0u;
#pragma unroll
      for (int i = 0; i < 4; ++i) U[nt][i] = 0.f;
#pragma unroll
      for (int mt = 0; mt < 8; ++mt)
#pragma unroll
        for (int i = 0; i < 4; ++i) O[mt][nt][i] = 0.f;
    }
#pragma unroll
    for (int h = 0; h < HP; ++h)
#pragma unroll
      for (int g = 0; g < NGV; ++g) cm[h][g] = 0.f;
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
        *reinterpret_cast<float4*>(qf + h * kHeadDim + lane * 4) = qv;
        *reinterpret_cast<float4*>(ocorr + h * kHeadDim + lane * 4) = make_float4(0.f, 0.f, 0.f, 0.f);
        float mx = fmaxf(fmaxf(fabsf(qv.x), fabsf(qv.y)), fmaxf(fabsf(qv.z), fabsf(qv.w)));
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        if (lane == 0) qexp_s[h] = float_exponent(mx);
      }
    }
    __syncwarp();

    for (int blk = blk_lo; blk < blk_hi && alive; ++blk) {
      const bool is_buf = blk >= a.n_blocks_c;
      // ---------------- block geometry
      int nslab = 1, r_pad = 0, k2k = 0, valid_tokens = kSlab, slab_a = 0;
      bool with_bk = false, with_bv = false;
      if (!is_buf) {
        if (blk < c_seg_lo || blk >= c_seg_hi) {
          load_desc(sdc, blk);
          c_seg_lo = sdc->blk_start;
          c_seg_hi = c_seg_lo + sdc->nblk;
        }
        const int bl = blk - c_seg_lo;
        nslab = sdc->T / kSlab; r_pad = sdc->r_pad; k2k = 2 * sdc->k_k; slab_a = sdc->slab_a;
        valid_tokens = sdc->T;
        with_bk = r_pad > 0 && (bl == 0 || blk == blk_lo);
        with_bv = r_pad > 0 && (bl == c_seg_hi - c_seg_lo - 1 || blk == blk_hi - 1);
      } else {
        valid_tokens = min(kSlab, a.buf_len - (blk - a.n_blocks_c) * kSlab);
      }

      // ================================================================ key item
      unsigned char* stK = acquire(item_k);
      if (!alive) break;
      const unsigned char* kp = stK + a.bregion;
      float dmax_v = 0.f;
      int own_sexp[NT];
      float ch_own[NT];
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) { own_sexp[nt] = 0; ch_own[nt] = 0.f; }

      if (with_bk) {
        // w = q B_K through the tensor cores, kept as the B operand of the low-rank key term
        const __half* bk = reinterpret_cast<const __half*>(stK);     // [r_pad][128]
        float wacc[NT][4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
          for (int i = 0; i < 4; ++i) wacc[nt][i] = 0.f;
#pragma unroll
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
          wl[gid * HP + t + 4 * nt] = wacc[nt][0] * a.scale_log2;
          wl[(gid + 8) * HP + t + 4 * nt] = wacc[nt][2] * a.scale_log2;
        }
        __syncwarp();
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          const int h = (gid >> 1) + 4 * nt;
          uint32_t hi0, lo0, hi1, lo1;
          split_hi_lo(wl[(2 * t) * HP + h], wl[(2 * t + 1) * HP + h], hi0, lo0);
          split_hi_lo(wl[(2 * t + 8) * HP + h], wl[(2 * t + 9) * HP + h], hi1, lo1);
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
          const uint4 kz = reinterpret_cast<const uint4*>(kp + sdc->off_kscale)[lane];
          const uint32_t w4[4] = {kz.x, kz.y, kz.z, kz.w};
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            sc4[j] = __low2float(u32_as_h2(w4[j]));
            zr4[j] = __high2float(u32_as_h2(w4[j]));
          }
        }
        float qS[HP][4];
        const int kc = lane >> 2, reg = (lane >> 1) & 1, tA = 2 * (lane & 1);
#pragma unroll
        for (int h = 0; h < HP; ++h) {
          if (h < HPu) {
            const float4 qv = *reinterpret_cast<const float4*>(qf + h * kHeadDim + lane * 4);
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
              float c = fmaf(qv.x, zr4[0], fmaf(qv.y, zr4[1], fmaf(qv.z, zr4[2], qv.w * zr4[3])));
#pragma unroll
              for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
              const int sexp = clamp60(21 - qexp_s[h] - ed);
              const float S = pow2i(sexp);
              qS[h][0] = qv.x * S; qS[h][1] = qv.y * S; qS[h][2] = qv.z * S; qS[h][3] = qv.w * S;
              if ((h & 3) == t) { ch_own[h >> 2] = c; own_sexp[h >> 2] = sexp; }
            }
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
            const uint4 ov = reinterpret_cast<const uint4*>(kp + sdc->off_koval)[lane];
            const uint2 oi = reinterpret_cast<const uint2*>(kp + sdc->off_koidx)[lane];
            const uint32_t o4[4] = {ov.x, ov.y, ov.z, ov.w};
            const uint32_t i2[2] = {oi.x, oi.y};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              k_entry(j, __low2float(u32_as_h2(o4[j])), (i2[j >> 1] >> (16 * (j & 1))) & 0xFFu);
              k_entry(j, __high2float(u32_as_h2(o4[j])), (i2[j >> 1] >> (16 * (j & 1) + 8)) & 0xFFu);
            }
          } else {
            const __half* ov = reinterpret_cast<const __half*>(kp + sdc->off_koval) + lane * 4 * k2k;
            const unsigned char* oi = kp + sdc->off_koidx + lane * 4 * k2k;
#pragma unroll
            for (int j = 0; j < 4; ++j)
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
          const uint2 v = *reinterpret_cast<const uint2*>(frag + (nt * 8 + kc) * kFragStride + lane * 2);
          bq[nt][kc][0] = v.x; bq[nt][kc][1] = v.y;
        }
      __syncwarp();                                  // the fragment region is rewritten in the value phase

      unsigned char* stV = nullptr;
      const int nchunk = (nslab + kChunkSlabs - 1) / kChunkSlabs;
      for (int c = 0; c < nchunk && alive; ++c) {
        const int ns = min(kChunkSlabs, nslab - c * kChunkSlabs);
        // ---------------- key scores of up to four slabs, kept in registers
        float sc[NT][kChunkSlabs][2];
#pragma unroll
        for (int s = 0; s < kChunkSlabs; ++s) {
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) sc[nt][s][0] = sc[nt][s][1] = -INFINITY;
          if (s < ns) {
            const int slab = c * kChunkSlabs + s;
            float acc[NT][4];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
              for (int i = 0; i < 4; ++i) acc[nt][i] = 0.f;
            uint4 w0 = make_uint4(0u, 0u, 0u, 0u), w1 = w0;
            if (!is_buf) {
              const uint4* cw = reinterpret_cast<const uint4*>(kp + sdc->off_kcodes + slab * sdc->slab_codes);
              w0 = cw[lane];
              if (BITS == 4) w1 = cw[32 + lane];
            }
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {            // channel chunks 4 hf .. 4 hf + 3
              uint32_t af[4][4];
              if (!is_buf) {
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
                for (int nt = 0; nt < NT; ++nt) mma16816(acc[nt], af[k4], bq[nt][4 * hf + k4][0], bq[nt][4 * hf + k4][1]);
            }
            if (r_pad > 0) {                          // low-rank key term: A_K rows times w
              const __half* ak = reinterpret_cast<const __half*>(kp + sdc->off_ak + slab * slab_a);
              uint32_t aa[4] = {0u, 0u, 0u, 0u};
              if (2 * t < r_pad) {
                aa[0] = *reinterpret_cast<const uint32_t*>(ak + gid * r_pad + 2 * t);
                aa[1] = *reinterpret_cast<const uint32_t*>(ak + (gid + 8) * r_pad + 2 * t);
              }
              if (2 * t + 8 < r_pad) {
                aa[2] = *reinterpret_cast<const uint32_t*>(ak + gid * r_pad + 2 * t + 8);
                aa[3] = *reinterpret_cast<const uint32_t*>(ak + (gid + 8) * r_pad + 2 * t + 8);
              }
#pragma unroll
              for (int nt = 0; nt < NT; ++nt) mma16816(acc[nt], aa, bw[nt][0], bw[nt][1]);
            }
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
              const int h = t + 4 * nt;
              const float Si = pow2i(-own_sexp[nt]);
#pragma unroll
              for (int half = 0; half < 2; ++half) {
                const int tok = slab * kSlab + gid + 8 * half;          // token inside the block
                float v = acc[nt][2 * half] + acc[nt][2 * half + 1] + ch_own[nt];
                if (k2k > 0 && h < HPu) {
                  v = fmaf((float)corr_k[h * maxT + tok], Si, v);
                  corr_k[h * maxT + tok] = 0;
                }
                sc[nt][s][half] = (tok < valid_tokens && h < HPu) ? v : -INFINITY;
              }
            }
          }
        }
        if (c == nchunk - 1) release();               // the key item is consumed

        // ---------------- online softmax over the chunk: one rescale at most
        bool grew = false;
        float m_new[NT];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          float mx = -INFINITY;
#pragma unroll
          for (int s = 0; s < kChunkSlabs; ++s) mx = fmaxf(mx, fmaxf(sc[nt][s][0], sc[nt][s][1]));
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
          m_new[nt] = fmaxf(m_run[nt], mx);
          grew |= m_new[nt] > m_run[nt];
        }
        if (__any_sync(0xffffffffu, grew)) {
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) {
            const float al = (m_new[nt] == -INFINITY) ? 1.f : exp2f(m_run[nt] - m_new[nt]);
            if (gid == 0) alpha_s[t + 4 * nt] = al;
            l_run[nt] *= al;
#pragma unroll
            for (int i = 0; i < 4; ++i) U[nt][i] *= al;
#pragma unroll
            for (int mt = 0; mt < 8; ++mt)
#pragma unroll
              for (int i = 0; i < 4; ++i) O[mt][nt][i] *= al;
          }
          __syncwarp();
#pragma unroll
          for (int h = 0; h < HP; ++h) {
            if (h < HPu) {
              const float al = alpha_s[h];
#pragma unroll
              for (int g = 0; g < NGV; ++g) cm[h][g] *= al;
              float4* oc = reinterpret_cast<float4*>(ocorr + h * kHeadDim + lane * 4);
              float4 v = *oc;
              v.x *= al; v.y *= al; v.z *= al; v.w *= al;
              *oc = v;
            }
          }
          __syncwarp();
        }
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          m_run[nt] = m_new[nt];
          const int h = t + 4 * nt;
#pragma unroll
          for (int s = 0; s < kChunkSlabs; ++s) {
            if (s < ns) {
#pragma unroll
              for (int half = 0; half < 2; ++half) {
                const float p = exp2f(sc[nt][s][half] - m_new[nt]);     // exp2(-inf) = 0 for masked tokens
                l_run[nt] += p;
                if (h < HPu) ps[h * kChunkTok + s * kSlab + gid + 8 * half] = p;
              }
            }
          }
        }
        __syncwarp();

        // ================================================================ value item
        if (stV == nullptr) {
          stV = acquire(item_k + 1);
          if (!alive) break;
          if (is_buf && valid_tokens < kSlab) {
            // rows past the end of the buffer hold stale bytes: clear them (0 * garbage must stay 0)
            for (int i = lane; i < (kSlab - valid_tokens) * (kBufPitch / 16); i += 32) {
              const int r = valid_tokens + i / (kBufPitch / 16), cc = i % (kBufPitch / 16);
              reinterpret_cast<uint4*>(stV + r * kBufPitch)[cc] = make_uint4(0u, 0u, 0u, 0u);
            }
            fence_async_smem();
            __syncwarp();
          }
        }
        const unsigned char* vp = stV + a.bregion - (is_buf ? 0 : sdc->off_vpart);   // record base seen from the value part
        const int tok0c = c * kChunkTok;                                               // first token of the chunk

        // ---------------- B operands of the value products: p * scale (per token and group) and p, split hi / lo;
        //                  the zero-point term goes to the fp32 side sums cm
        {
          const int s = lane >> 3, pi = lane & 7;        // this lane's token pair of the chunk
          const int tp = s * kSlab + 2 * pi;
          const int tw = (pi & 3), rg = pi >> 2;
          if (s < ns) {
#pragma unroll
            for (int h = 0; h < HP; ++h) {
              if (h < HPu) {
                const float2 pp = *reinterpret_cast<const float2*>(ps + h * kChunkTok + tp);
                const int col = 2 * (h & 3);
                uint32_t hi, lo;
                if (r_pad > 0 || is_buf) {
                  split_hi_lo(pp.x, pp.y, hi, lo);
                  uint32_t* bp = fragP + ((h >> 2) * kChunkSlabs + s) * kFragStride + rg;
                  bp[(col * 4 + tw) * 2] = hi;
                  bp[((col + 1) * 4 + tw) * 2] = lo;
                }
                if (!is_buf) {
                  const __half2* vsz = reinterpret_cast<const __half2*>(vp + sdc->off_vscale) + (size_t)(tok0c + tp) * NGV;
#pragma unroll
                  for (int g = 0; g < NGV; ++g) {
                    const __half2 z0 = vsz[g], z1 = vsz[NGV + g];
                    split_hi_lo(pp.x * __low2float(z0), pp.y * __low2float(z1), hi, lo);
                    uint32_t* bv = fragV + (((h >> 2) * NGV + g) * kChunkSlabs + s) * kFragStride + rg;
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
#pragma unroll 1
        for (int s = 0; s < ns; ++s) {
          const int slab = c * kChunkSlabs + s;
          uint32_t bp[NT][2];
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) {
            const uint2 v = *reinterpret_cast<const uint2*>(fragP + (nt * kChunkSlabs + s) * kFragStride + lane * 2);
            bp[nt][0] = v.x; bp[nt][1] = v.y;
          }
          if (!is_buf) {
            const uint4* cw = reinterpret_cast<const uint4*>(vp + sdc->off_vcodes + slab * sdc->slab_codes);
            uint32_t bv[NT][NGV][2];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
              for (int g = 0; g < NGV; ++g) {
                const uint2 v = *reinterpret_cast<const uint2*>(fragV + ((nt * NGV + g) * kChunkSlabs + s) * kFragStride + lane * 2);
                bv[nt][g][0] = v.x; bv[nt][g][1] = v.y;
              }
            if (BITS == 2) {
              const uint4 w = cw[lane];
              const uint32_t wv[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
              for (int q4 = 0; q4 < 4; ++q4) {
                uint32_t r[8];
                unpack_word<2>(wv[q4], r);
#pragma unroll
                for (int m2 = 0; m2 < 2; ++m2) {
                  const int mt = 2 * q4 + m2, g = (mt * 16) / GV;
                  const uint32_t av[4] = {r[4 * m2], r[4 * m2 + 1], r[4 * m2 + 2], r[4 * m2 + 3]};
#pragma unroll
                  for (int nt = 0; nt < NT; ++nt) mma16816(O[mt][nt], av, bv[nt][g][0], bv[nt][g][1]);
                }
              }
            } else {
#pragma unroll
              for (int pl = 0; pl < 2; ++pl) {
                const uint4 w = cw[pl * 32 + lane];
                const uint32_t wv[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4) {
                  const int mt = 4 * pl + q4, g = (mt * 16) / GV;
                  uint32_t av[4];
                  unpack_word<4>(wv[q4], av);
#pragma unroll
                  for (int nt = 0; nt < NT; ++nt) mma16816(O[mt][nt], av, bv[nt][g][0], bv[nt][g][1]);
                }
              }
            }
            if (r_pad > 0) {                          // low-rank value term, first product: U = A_V^T p
              const __half* avs = reinterpret_cast<const __half*>(vp + sdc->off_av + slab * slab_a);
              uint32_t aa[4] = {0u, 0u, 0u, 0u};
              if (gid < r_pad) {
                aa[0] = *reinterpret_cast<const uint32_t*>(avs + gid * kSlab + 2 * t);
                aa[2] = *reinterpret_cast<const uint32_t*>(avs + gid * kSlab + 2 * t + 8);
              }
              if (gid + 8 < r_pad) {
                aa[1] = *reinterpret_cast<const uint32_t*>(avs + (gid + 8) * kSlab + 2 * t);
                aa[3] = *reinterpret_cast<const uint32_t*>(avs + (gid + 8) * kSlab + 2 * t + 8);
              }
#pragma unroll
              for (int nt = 0; nt < NT; ++nt) mma16816(U[nt], aa, bp[nt][0], bp[nt][1]);
              u_pending = true;
            }
          } else {
#pragma unroll
            for (int mt = 0; mt < 8; ++mt) {
              uint32_t av[4];
              ldmatrix_x4_trans(av, stV + ((lane & 7) + 8 * (lane >> 4)) * kBufPitch + (16 * mt + 8 * ((lane >> 3) & 1)) * 2);
#pragma unroll
              for (int nt = 0; nt < NT; ++nt) mma16816(O[mt][nt], av, bp[nt][0], bp[nt][1]);
            }
          }
        }

        // ---------------- sparse value term: p[tok] * (x - zero[tok, g]) scattered to the outlier's channel
        if (!is_buf && a.cc.k_v > 0) {
          const int k2v = 2 * a.cc.k_v;
          const int sexp = clamp60(21 - float_exponent(dmax_v));
          const float S = pow2i(sexp), Si = pow2i(-sexp);
          const __half2* vsz = reinterpret_cast<const __half2*>(vp + sdc->off_vscale);
          for (int tk = lane; tk < ns * kSlab; tk += 32) {
            const int tb = tok0c + tk;
            float pS[HP];
#pragma unroll
            for (int h = 0; h < HP; ++h) pS[h] = h < HPu ? ps[h * kChunkTok + tk] * S : 0.f;
            auto v_entry = [&](int g, float val, int idx) {
              const float d = val - __high2float(vsz[tb * NGV + g]);
              const int ch = g * GV + idx;
#pragma unroll
              for (int h = 0; h < HP; ++h)
                if (h < HPu) atomicAdd(&corr_v[h * kHeadDim + ch], __float2int_rn(pS[h] * d));
            };
            if (NGV * k2v == 4) {
              const uint2 ov = reinterpret_cast<const uint2*>(vp + sdc->off_voval)[tb];
              const uint32_t oi = reinterpret_cast<const uint32_t*>(vp + sdc->off_voidx)[tb];
              v_entry(0, __low2float(u32_as_h2(ov.x)), oi & 0xFFu);
              v_entry(NGV == 2 ? 0 : (NGV == 4 ? 1 : 0), __high2float(u32_as_h2(ov.x)), (oi >> 8) & 0xFFu);
              v_entry(NGV == 2 ? 1 : (NGV == 4 ? 2 : 0), __low2float(u32_as_h2(ov.y)), (oi >> 16) & 0xFFu);
              v_entry(NGV == 2 ? 1 : (NGV == 4 ? 3 : 0), __high2float(u32_as_h2(ov.y)), oi >> 24);
            } else {
              const __half* ov = reinterpret_cast<const __half*>(vp + sdc->off_voval) + (size_t)tb * NGV * k2v;
              const unsigned char* oi = vp + sdc->off_voidx + (size_t)tb * NGV * k2v;
#pragma unroll
              for (int g = 0; g < NGV; ++g)
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
        __syncwarp();                                 // ps and the fragments are rewritten by the next chunk
      }
      if (!alive) break;

      // ---------------- end of a segment (or of this warp's share of it): out += B_V U
      if (with_bv && u_pending) {
        __syncwarp();
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          wl[gid * HP + t + 4 * nt] = U[nt][0] + U[nt][1];
          wl[(gid + 8) * HP + t + 4 * nt] = U[nt][2] + U[nt][3];
#pragma unroll
          for (int i = 0; i < 4; ++i) U[nt][i] = 0.f;
        }
        __syncwarp();
        uint32_t bu[NT][2];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          const int h = (gid >> 1) + 4 * nt;
          uint32_t hi0, lo0, hi1, lo1;
          split_hi_lo(wl[(2 * t) * HP + h], wl[(2 * t + 1) * HP + h], hi0, lo0);
          split_hi_lo(wl[(2 * t + 8) * HP + h], wl[(2 * t + 9) * HP + h], hi1, lo1);
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
          for (int nt = 0; nt < NT; ++nt) mma16816(O[mt][nt], aa, bu[nt][0], bu[nt][1]);
        }
        u_pending = false;
      }
      release();                                      // the value item is consumed
      item_k += 2;
    }
    if (!alive) break;

    // ---------------- partial result of this unit: (m, l, o) per head
    const long long bflat = (long long)u * NB, eflat = bflat + NB;
    const long long w_first = ((bflat + 1) * NW + F - 1) / F - 1;
    const long long w_last = (eflat * NW + F - 1) / F - 1;
    const int n_parts = (int)(w_last - w_first + 1);
    const int slot = (int)(gw - w_first);
    float* part_base = a.partial + ((size_t)u * a.max_parts + slot) * (HP * 130);
    float cm_own[NT][NGV];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      float l = l_run[nt];
      l += __shfl_xor_sync(0xffffffffu, l, 4);
      l += __shfl_xor_sync(0xffffffffu, l, 8);
      l += __shfl_xor_sync(0xffffffffu, l, 16);
      l_run[nt] = l;
#pragma unroll
      for (int g = 0; g < NGV; ++g) cm_own[nt][g] = 0.f;
    }
#pragma unroll
    for (int h = 0; h < HP; ++h)
#pragma unroll
      for (int g = 0; g < NGV; ++g) {
        float c = cm[h][g];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
        if ((h & 3) == t) cm_own[h >> 2][g] = c;
      }
    __syncwarp();
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      const int h = t + 4 * nt;
      if (h < HPu) {
        float* dst = part_base + h * 130;
#pragma unroll
        for (int mt = 0; mt < 8; ++mt)
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            const int ch = 16 * mt + gid + 8 * half;
            dst[ch] = O[mt][nt][2 * half] + O[mt][nt][2 * half + 1] + ocorr[h * kHeadDim + ch] + cm_own[nt][(mt * 16) / GV];
          }
        if (gid == 0) { dst[128] = m_run[nt]; dst[129] = l_run[nt]; }
      }
    }
    __threadfence();
    __syncwarp();
    int last = 0;
    if (lane == 0) last = (atomicAdd(&a.tickets[u], 1) == n_parts - 1);
    last = __shfl_sync(0xffffffffu, last, 0);
    if (last) {
      __threadfence();
      const float* pb = a.partial + (size_t)u * a.max_parts * (HP * 130);
      for (int h = 0; h < HPu; ++h) {
        float M = -INFINITY;
        for (int i = 0; i < n_parts; ++i) M = fmaxf(M, __ldcg(pb + (size_t)i * HP * 130 + h * 130 + 128));
        float den = 0.f, n0 = 0.f, n1 = 0.f, n2 = 0.f, n3 = 0.f;
        for (int i = 0; i < n_parts; ++i) {
          const float* pp = pb + (size_t)i * HP * 130 + h * 130;
          const float mi = __ldcg(pp + 128);
          if (mi == -INFINITY) continue;
          const float wgt = exp2f(mi - M);
          den = fmaf(wgt, __ldcg(pp + 129), den);
          n0 = fmaf(wgt, __ldcg(pp + lane * 4 + 0), n0);
          n1 = fmaf(wgt, __ldcg(pp + lane * 4 + 1), n1);
          n2 = fmaf(wgt, __ldcg(pp + lane * 4 + 2), n2);
          n3 = fmaf(wgt, __ldcg(pp + lane * 4 + 3), n3);
        }
        const float inv = 1.0f / den;
        *reinterpret_cast<float4*>(a.out + (size_t)(hq0 + h) * kHeadDim + lane * 4) =
            make_float4(n0 * inv, n1 * inv, n2 * inv, n3 * inv);
      }
      if (lane == 0) a.tickets[u] = 0;
    }
    f += blk_hi - blk_lo;
  }
  // a warp that gave up still has copies in flight: let them land (bounded) before leaving
  if (!alive) {
    for (int i = n_released; i < n_issued; ++i) {
      const int s = i % NS;
      for (int k = 0; k < kSpinLimit && !mbar_try(&bar[s], (uint32_t)((i / NS) & 1)); ++k) {}
    }
  }
}

// ------------------------------------------------------------------ host side
template <class Fn>
static bool with_decode_kernel(int bits, int heads, int ngv, Fn fn) {
  const int nt = heads <= 4 ? 1 : 2;
#define GEAR_DEC_CASE(B, N, V) \
  if (bits == B && nt == N && ngv == V) { fn(gear_decode_kernel<B, N, V>); return true; }
  GEAR_DEC_CASE(2, 1, 1) GEAR_DEC_CASE(2, 1, 2) GEAR_DEC_CASE(2, 1, 4) GEAR_DEC_CASE(2, 1, 8)
  GEAR_DEC_CASE(2, 2, 1) GEAR_DEC_CASE(2, 2, 2) GEAR_DEC_CASE(2, 2, 4) GEAR_DEC_CASE(2, 2, 8)
  GEAR_DEC_CASE(4, 1, 1) GEAR_DEC_CASE(4, 1, 2) GEAR_DEC_CASE(4, 1, 4) GEAR_DEC_CASE(4, 1, 8)
  GEAR_DEC_CASE(4, 2, 1) GEAR_DEC_CASE(4, 2, 2) GEAR_DEC_CASE(4, 2, 4) GEAR_DEC_CASE(4, 2, 8)
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
