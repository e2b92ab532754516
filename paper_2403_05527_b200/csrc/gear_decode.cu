// Decode attention (Eq. 1, one query per sequence) over the compressed cache:
//   scores = q . dequant(codes_K)^T + (q B_K) A_K^T + q . S_K^T      (+ q . K_buffer^T)
//   out    = softmax(scores) . [dequant(codes_V) + A_V B_V^T + S_V]  (+ . V_buffer)
// fp16 K / V are never materialised.
//
// Every warp is an independent stream processor.  The (batch, kv head, block)
// space is cut into equal contiguous ranges, one per warp; lane 0 of a warp
// streams its blocks' records from HBM into a private shared-memory ring with
// bulk asynchronous copies (cp.async.bulk + mbarrier) while the warp consumes
// the previous one.  Codes are unpacked in registers straight into the A
// operand of mma.sync.m16n8k16 (tokens x channels for keys, channels x tokens
// for values); the B operand holds the query heads of the GQA group, each split
// into an fp16 high and low part (two columns) so that products are exact and
// sums are fp32.  Per-group scales are folded into the B operand (q * scale per
// channel for keys, p * scale per token for values), zero-points into a constant
// per block (keys) or an fp32 side sum (values).  Outlier corrections are
// scattered through 32-bit fixed-point shared-memory adds (deterministic).
// A warp writes one partial (m, l, o) per (batch, head) it touched; the last
// warp to arrive for a (batch, head) merges the partials.
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <math.h>

#include "gear_internal.cuh"

namespace gear {

constexpr int kStages = 2;
constexpr int kBufPitch = 272;                      // bytes per fp16 row of a buffer slab in shared memory
constexpr int kBufStage = 2 * kSlab * kBufPitch;    // K rows then V rows
constexpr int kSpinLimit = 4000000;

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

// fp32 pair -> half2 of the high parts (part 0) or of the rounding remainders (part 1)
__device__ __forceinline__ uint32_t split_h2(float x0, float x1, int part) {
  const __half2 h = __floats2half2_rn(x0, x1);
  if (part == 0) return h2_as_u32(h);
  return h2_as_u32(__floats2half2_rn(x0 - __low2float(h), x1 - __high2float(h)));
}

// power-of-two scale S with bound * S < 2^23, and 1 / S
__device__ __forceinline__ void fixed_scale(float bound, float& s, float& inv) {
  int e = (int)((__float_as_uint(bound) >> 23) & 0xFFu) - 127;   // floor(log2(bound)) for normal bound
  e = max(-100, min(100, e));
  s = __uint_as_float((uint32_t)(127 + 22 - e) << 23);
  inv = __uint_as_float((uint32_t)(127 - 22 + e) << 23);
}

// ------------------------------------------------------------------ shared memory plan (per warp)
struct WarpSmem {
  int stage, keep_bv, qs, bfrag, wl, corr_k, ps, corr_v, misc, total;
};
__host__ __device__ inline WarpSmem warp_smem_plan(int stage_bytes, int max_T, int max_rpad, int HP) {
  WarpSmem w;
  int o = 0;
  w.stage = o;   o += kStages * stage_bytes;
  w.keep_bv = o; o += round_up(kHeadDim * max_rpad * 2, 16);
  w.qs = o;      o += HP * kHeadDim * 2;
  w.bfrag = o;   o += (HP / 4) * 8 * 32 * 8;
  w.wl = o;      o += kMaxRank * HP * 4;
  w.corr_k = o;  o += HP * max_T * 4;
  w.ps = o;      o += HP * max_T * 4;
  w.corr_v = o;  o += HP * kHeadDim * 4;
  w.misc = o;    o += 4 * HP * 4 + HP * 8 * 4;       // c_h, alpha, pmax, spare ; cm[HP][8]
  w.total = round_up(o, 128);
  return w;
}

void decode_smem_plan(int bits, int max_rec, int max_bfac, int max_T, int max_rpad, int heads_per_pass,
                      int* stage_bytes, int* warp_smem) {
  (void)bits;
  int st = max_rec + max_bfac;
  if (st < kBufStage) st = kBufStage;
  st = round_up(st, 128);
  *stage_bytes = st;
  *warp_smem = warp_smem_plan(st, max_T < kSlab ? kSlab : max_T, max_rpad, heads_per_pass).total;
}

constexpr int kMaxDecWarps = 8;

// ------------------------------------------------------------------ the kernel
template <int BITS, int NT>
__global__ void __launch_bounds__(kMaxDecWarps * 32) gear_decode_kernel(DecodeArgs a) {
  constexpr int HP = 4 * NT;                      // query heads per pass
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ __align__(8) uint64_t bars[kMaxDecWarps][kStages];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, gid = lane >> 2, t = lane & 3;
  const int nwarps = blockDim.x >> 5;
  const int G = a.group_heads;
  const int passes = (G + HP - 1) / HP;
  const int max_T = a.max_T < kSlab ? kSlab : a.max_T;
  const WarpSmem ws = warp_smem_plan(a.stage_bytes, max_T, a.max_rpad, HP);
  unsigned char* wbase = smem + (size_t)warp * a.warp_smem;
  unsigned char* stage_base = wbase + ws.stage;
  __half* keep_bv = reinterpret_cast<__half*>(wbase + ws.keep_bv);
  __half* qs = reinterpret_cast<__half*>(wbase + ws.qs);
  uint32_t* bfrag = reinterpret_cast<uint32_t*>(wbase + ws.bfrag);
  float* wl = reinterpret_cast<float*>(wbase + ws.wl);
  int* corr_k = reinterpret_cast<int*>(wbase + ws.corr_k);
  float* ps = reinterpret_cast<float*>(wbase + ws.ps);
  int* corr_v = reinterpret_cast<int*>(wbase + ws.corr_v);
  float* ch_s = reinterpret_cast<float*>(wbase + ws.misc);
  float* alpha_s = ch_s + HP;
  float* pmax_s = alpha_s + HP;
  float* sik_s = pmax_s + HP;                     // 1 / fixed-point scale of the sparse key term, per head
  float* cm_s = pmax_s + 2 * HP;                  // [HP][8]
  uint64_t* bar = bars[warp];

  if (lane == 0)
    for (int s = 0; s < kStages; ++s) mbar_init(&bar[s], 1);
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  // zero what is only ever partly written
  for (int i = lane; i < (ws.corr_k - ws.bfrag) / 4; i += 32) bfrag[i] = 0u;          // bfrag, wl
  for (int i = lane; i < HP * max_T; i += 32) { corr_k[i] = 0; ps[i] = 0.f; }
  for (int i = lane; i < HP * kHeadDim; i += 32) corr_v[i] = 0;
  __syncwarp();

  // ---- this warp's range of the flat (unit, block) space; unit = (batch, kv head, head pass)
  const int nbuf_blocks = (a.buf_len + kSlab - 1) / kSlab;
  const int NB = a.n_blocks_c + nbuf_blocks;
  const long long units = (long long)a.cc.BH * passes;
  const long long F = units * NB;
  const long long NW = (long long)gridDim.x * nwarps;
  const long long gw = (long long)blockIdx.x * nwarps + warp;
  const long long f0 = gw * F / NW, f1 = (gw + 1) * F / NW;

  // ---- producer (lane 0): issue the copies of flat block pf into ring stage (n_issued % kStages)
  long long pf = f0;
  int n_issued = 0, pseg = 0;
  auto issue = [&]() {
    if (lane != 0 || pf >= f1) { if (pf < f1) { ++pf; ++n_issued; } return; }
    const long long u = pf / NB;
    const int blk = (int)(pf % NB);
    const int bh = (int)(u / passes);
    const int s = n_issued % kStages;
    unsigned char* dst = stage_base + (size_t)s * a.stage_bytes;
    if (blk < a.n_blocks_c) {
      if (blk < a.table[pseg].blk_start) pseg = 0;
      while (blk >= a.table[pseg].blk_start + a.table[pseg].nblk) ++pseg;
      const SegDesc& sd = a.table[pseg];
      const int bl = blk - sd.blk_start;
      const bool with_b = sd.bfac_bytes > 0 && (bl == 0 || pf == f0);
      const unsigned char* src_b = a.arena + sd.seg_base + (size_t)bh * sd.bh_stride;
      const unsigned char* src_r = src_b + sd.bfac_bytes + (size_t)bl * sd.rec_bytes;
      if (with_b && bl == 0) {
        mbar_expect_tx(&bar[s], sd.bfac_bytes + sd.rec_bytes);
        bulk_g2s(dst, src_b, sd.bfac_bytes + sd.rec_bytes, &bar[s]);
      } else if (with_b) {
        mbar_expect_tx(&bar[s], sd.bfac_bytes + sd.rec_bytes);
        bulk_g2s(dst, src_b, sd.bfac_bytes, &bar[s]);
        bulk_g2s(dst + sd.bfac_bytes, src_r, sd.rec_bytes, &bar[s]);
      } else {
        mbar_expect_tx(&bar[s], sd.rec_bytes);
        bulk_g2s(dst, src_r, sd.rec_bytes, &bar[s]);
      }
    } else {
      const int j = blk - a.n_blocks_c;
      const int rows = min(kSlab, a.buf_len - j * kSlab);
      mbar_expect_tx(&bar[s], rows * 512);
      const __half* kb = a.buf_k + ((size_t)bh * a.cc.n_b + (size_t)j * kSlab) * kHeadDim;
      const __half* vb = a.buf_v + ((size_t)bh * a.cc.n_b + (size_t)j * kSlab) * kHeadDim;
      for (int r = 0; r < rows; ++r) {
        bulk_g2s(dst + r * kBufPitch, kb + r * kHeadDim, 256, &bar[s]);
        bulk_g2s(dst + (kSlab + r) * kBufPitch, vb + r * kHeadDim, 256, &bar[s]);
      }
    }
    ++pf; ++n_issued;
  };
  for (int s = 0; s < kStages; ++s) issue();

  int n_consumed = 0, cseg = 0;
  bool alive = true;

  // ---- loop over the units this warp touches
  long long f = f0;
  while (alive) {
    const bool empty_range = (f0 == f1);
    if (empty_range && !(f0 % NB != 0 && f0 < F)) break;
    if (!empty_range && f >= f1) break;
    const long long u = f / NB;
    const int blk_lo = (int)(f % NB);
    const int blk_hi = empty_range ? blk_lo : (int)min((long long)NB, blk_lo + (f1 - f));
    const int bh = (int)(u / passes), pass = (int)(u % passes);
    const int b_idx = bh / a.n_kv_heads, hkv = bh % a.n_kv_heads;
    const int HPu = min(HP, G - pass * HP);
    const int hq0 = (b_idx * a.n_kv_heads + hkv) * G + pass * HP;    // first query head of this pass

    // unit state
    float O[8][NT][4], U[NT][4], m_run[NT], l_run[NT], cm[NT][8], ocorr[HP][4], qmax[HP];
#pragma unroll
    for (int mt = 0; mt < 8; ++mt)
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int i = 0; i < 4; ++i) O[mt][nt][i] = 0.f;
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      m_run[nt] = -INFINITY; l_run[nt] = 0.f;
#pragma unroll
      for (int i = 0; i < 4; ++i) U[nt][i] = 0.f;
#pragma unroll
      for (int g = 0; g < 8; ++g) cm[nt][g] = 0.f;
    }
#pragma unroll
    for (int h = 0; h < HP; ++h)
#pragma unroll
      for (int j = 0; j < 4; ++j) ocorr[h][j] = 0.f;
    bool u_pending = false;

    // query rows of this pass -> shared (zero rows for absent heads), max |q| per head
    __syncwarp();
#pragma unroll
    for (int h = 0; h < HP; ++h) {
      uint2 v = make_uint2(0u, 0u);
      if (h < HPu) v = *reinterpret_cast<const uint2*>(a.q + (size_t)(hq0 + h) * kHeadDim + lane * 4);
      *reinterpret_cast<uint2*>(qs + h * kHeadDim + lane * 4) = v;
      const __half2 q01 = u32_as_h2(v.x), q23 = u32_as_h2(v.y);
      float mx = fmaxf(fmaxf(fabsf(__low2float(q01)), fabsf(__high2float(q01))),
                       fmaxf(fabsf(__low2float(q23)), fabsf(__high2float(q23))));
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      qmax[h] = mx;
    }
    __syncwarp();

    uint32_t bw[NT][2];          // low-rank key term: B operand (q B_K), valid for the current segment
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) bw[nt][0] = bw[nt][1] = 0u;

    for (int blk = blk_lo; blk < blk_hi && alive; ++blk) {
      const int s = n_consumed % kStages;
      const uint32_t parity = (uint32_t)((n_consumed / kStages) & 1);
      if (!mbar_wait(&bar[s], parity, a.status)) { alive = false; break; }
      unsigned char* st = stage_base + (size_t)s * a.stage_bytes;
      const bool is_buf = blk >= a.n_blocks_c;

      // ---------------- block geometry
      int T, nslab, r_pad = 0, k_k = 0, valid_tokens;
      const unsigned char* rec = st;
      SegDesc sd;
      bool seg_last_block = true;
      if (!is_buf) {
        if (blk < a.table[cseg].blk_start) cseg = 0;
        while (blk >= a.table[cseg].blk_start + a.table[cseg].nblk) ++cseg;
        sd = a.table[cseg];
        const int bl = blk - sd.blk_start;
        const bool with_b = sd.bfac_bytes > 0 && (bl == 0 || (f == f0 && blk == blk_lo));
        T = sd.T; nslab = T / kSlab; r_pad = sd.r_pad; k_k = sd.k_k; valid_tokens = T;
        seg_last_block = (bl == sd.nblk - 1) || (blk == blk_hi - 1);
        if (with_b) {
          rec = st + sd.bfac_bytes;
          // keep B_V for the flush at the end of the segment; w = q B_K through the tensor cores
          const uint4* src = reinterpret_cast<const uint4*>(st + kHeadDim * r_pad * 2);
          for (int i = lane; i < kHeadDim * r_pad * 2 / 16; i += 32) reinterpret_cast<uint4*>(keep_bv)[i] = src[i];
          const __half* bk = reinterpret_cast<const __half*>(st);     // [r_pad][128]
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
              if ((gid & 1) == 0) {
                const __half* qrow = qs + ((gid >> 1) + 4 * nt) * kHeadDim + 16 * kc + 2 * t;
                b0 = *reinterpret_cast<const uint32_t*>(qrow);
                b1 = *reinterpret_cast<const uint32_t*>(qrow + 8);
              }
              mma16816(wacc[nt], af, b0, b1);
            }
          }
          __syncwarp();
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) {       // D[rho][col 2t] = w[rho][head t + 4nt]
            wl[gid * HP + t + 4 * nt] = wacc[nt][0];
            wl[(gid + 8) * HP + t + 4 * nt] = wacc[nt][2];
          }
          __syncwarp();
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) {
            const int h = (gid >> 1) + 4 * nt, part = gid & 1;
            bw[nt][0] = split_h2(wl[(2 * t) * HP + h], wl[(2 * t + 1) * HP + h], part);
            bw[nt][1] = split_h2(wl[(2 * t + 8) * HP + h], wl[(2 * t + 9) * HP + h], part);
          }
          __syncwarp();
        }
      } else {
        const int j = blk - a.n_blocks_c;
        T = kSlab; nslab = 1;
        valid_tokens = min(kSlab, a.buf_len - j * kSlab);
        // rows past the end of the buffer hold stale bytes: clear them
        for (int i = lane; i < (kSlab - valid_tokens) * (kBufPitch / 16); i += 32) {
          const int r = valid_tokens + i / (kBufPitch / 16), c = i % (kBufPitch / 16);
          reinterpret_cast<uint4*>(st + r * kBufPitch)[c] = make_uint4(0u, 0u, 0u, 0u);
          reinterpret_cast<uint4*>(st + (kSlab + r) * kBufPitch)[c] = make_uint4(0u, 0u, 0u, 0u);
        }
        __syncwarp();
      }

      // ---------------- B operand for the key scores: q * scale per channel, split hi / lo; c_h = sum q * zero
      float dmax_k = 0.f, dmax_v = 0.f;
      {
        float sc4[4] = {1.f, 1.f, 1.f, 1.f}, zr4[4] = {0.f, 0.f, 0.f, 0.f};
        if (!is_buf) {
          dmax_k = reinterpret_cast<const float*>(rec)[0];
          dmax_v = reinterpret_cast<const float*>(rec)[1];
          const uint4 kz = reinterpret_cast<const uint4*>(rec + sd.off_kscale)[lane];
          const uint32_t w4[4] = {kz.x, kz.y, kz.z, kz.w};
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            sc4[j] = __low2float(u32_as_h2(w4[j]));
            zr4[j] = __high2float(u32_as_h2(w4[j]));
          }
        }
        const int kc = lane >> 2, bsel = (lane & 3) >> 1, tA = 2 * (lane & 1);
#pragma unroll
        for (int h = 0; h < HP; ++h) {
          if (h < HPu) {
            const uint2 qv = *reinterpret_cast<const uint2*>(qs + h * kHeadDim + lane * 4);
            const float q0 = __low2float(u32_as_h2(qv.x)), q1 = __high2float(u32_as_h2(qv.x));
            const float q2 = __low2float(u32_as_h2(qv.y)), q3 = __high2float(u32_as_h2(qv.y));
            const float p0 = q0 * sc4[0], p1 = q1 * sc4[1], p2 = q2 * sc4[2], p3 = q3 * sc4[3];
            const int nt = h >> 2, cl = 2 * (h & 3);
            uint32_t* base = bfrag + ((nt * 8 + kc) * 32) * 2 + bsel;
            base[(4 * cl + tA) * 2] = split_h2(p0, p1, 0);
            base[(4 * (cl + 1) + tA) * 2] = split_h2(p0, p1, 1);
            base[(4 * cl + tA + 1) * 2] = split_h2(p2, p3, 0);
            base[(4 * (cl + 1) + tA + 1) * 2] = split_h2(p2, p3, 1);
            float c = fmaf(q0, zr4[0], fmaf(q1, zr4[1], fmaf(q2, zr4[2], q3 * zr4[3])));
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
            if (lane == 0) ch_s[h] = c;
            // ---- sparse key term: q_h[ch] * (x - zero[ch]) scattered to the outlier's token (fixed point)
            if (!is_buf && k_k > 0) {
              float S, Si;
              fixed_scale(qmax[h] * dmax_k, S, Si);
              if (lane == 0) sik_s[h] = Si;
              const float qj[4] = {q0, q1, q2, q3};
              const __half* ov = reinterpret_cast<const __half*>(rec + sd.off_koval) + lane * 4 * 2 * k_k;
              const unsigned char* oi = rec + sd.off_koidx + lane * 4 * 2 * k_k;
#pragma unroll
              for (int j = 0; j < 4; ++j)
                for (int e = 0; e < 2 * k_k; ++e) {
                  const float d = __half2float(ov[j * 2 * k_k + e]) - zr4[j];
                  atomicAdd(&corr_k[h * max_T + oi[j * 2 * k_k + e]], __float2int_rn(qj[j] * d * S));
                }
            }
          }
        }
      }
      __syncwarp();
      uint32_t bq[NT][8][2];
#pragma unroll
      for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int kc = 0; kc < 8; ++kc) {
          const uint2 v = *reinterpret_cast<const uint2*>(bfrag + ((nt * 8 + kc) * 32 + lane) * 2);
          bq[nt][kc][0] = v.x; bq[nt][kc][1] = v.y;
        }

      // ---------------- key scores, slab by slab; scaled scores go to shared memory
      float blk_max[NT];
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) blk_max[nt] = -INFINITY;
      for (int slab = 0; slab < nslab; ++slab) {
        uint32_t af[8][4];
        if (!is_buf) {
          const uint4* cw = reinterpret_cast<const uint4*>(rec + sd.off_kcodes + slab * sd.slab_codes);
          if (BITS == 2) {
            const uint4 w = cw[lane];
            uint32_t r[8];
            unpack_word<2>(w.x, r);
#pragma unroll
            for (int u2 = 0; u2 < 8; ++u2) af[u2 >> 1][(u2 & 1) * 2] = r[u2];
            unpack_word<2>(w.y, r);
#pragma unroll
            for (int u2 = 0; u2 < 8; ++u2) af[4 + (u2 >> 1)][(u2 & 1) * 2] = r[u2];
            unpack_word<2>(w.z, r);
#pragma unroll
            for (int u2 = 0; u2 < 8; ++u2) af[u2 >> 1][(u2 & 1) * 2 + 1] = r[u2];
            unpack_word<2>(w.w, r);
#pragma unroll
            for (int u2 = 0; u2 < 8; ++u2) af[4 + (u2 >> 1)][(u2 & 1) * 2 + 1] = r[u2];
          } else {
#pragma unroll
            for (int th = 0; th < 2; ++th) {
              const uint4 w = cw[th * 32 + lane];
              const uint32_t wv[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
              for (int q4 = 0; q4 < 4; ++q4) {
                uint32_t r[4];
                unpack_word<4>(wv[q4], r);
#pragma unroll
                for (int u2 = 0; u2 < 4; ++u2) af[2 * q4 + (u2 >> 1)][(u2 & 1) * 2 + th] = r[u2];
              }
            }
          }
        } else {
#pragma unroll
          for (int kc = 0; kc < 8; ++kc)
            ldmatrix_x4(af[kc], st + ((lane & 7) + 8 * ((lane >> 3) & 1)) * kBufPitch + (16 * kc + 8 * (lane >> 4)) * 2);
        }
        float acc[NT][4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
          for (int i = 0; i < 4; ++i) acc[nt][i] = 0.f;
#pragma unroll
        for (int kc = 0; kc < 8; ++kc)
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) mma16816(acc[nt], af[kc], bq[nt][kc][0], bq[nt][kc][1]);
        if (r_pad > 0) {                          // low-rank key term: A_K rows times w
          const __half* ak = reinterpret_cast<const __half*>(rec + sd.off_ak + slab * sd.slab_a);
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
          const float Si = sik_s[h];
          const float ch = ch_s[h];
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            const int tok = slab * kSlab + gid + 8 * half;
            float sc = acc[nt][2 * half] + acc[nt][2 * half + 1] + ch;
            if (!is_buf && k_k > 0) {
              sc = fmaf((float)corr_k[h * max_T + tok], Si, sc);
              corr_k[h * max_T + tok] = 0;
            }
            sc = (tok < valid_tokens) ? sc * a.scale_log2 : -INFINITY;
            ps[h * max_T + tok] = sc;
            blk_max[nt] = fmaxf(blk_max[nt], sc);
          }
        }
      }
      // ---------------- online softmax: one rescale per block at most
      bool grew = false;
      float m_new[NT];
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        float mx = blk_max[nt];
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
        blk_max[nt] = mx;
        m_new[nt] = fmaxf(m_run[nt], mx);
        grew |= m_new[nt] > m_run[nt];
      }
      const bool any_grew = __any_sync(0xffffffffu, grew);
      if (gid == 0) {
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          alpha_s[t + 4 * nt] = (m_new[nt] == -INFINITY) ? 1.f : exp2f(m_run[nt] - m_new[nt]);
          pmax_s[t + 4 * nt] = (m_new[nt] == -INFINITY) ? 0.f : exp2f(blk_max[nt] - m_new[nt]);
        }
      }
      __syncwarp();
      if (any_grew) {
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          const float al = alpha_s[t + 4 * nt];
          l_run[nt] *= al;
#pragma unroll
          for (int i = 0; i < 4; ++i) U[nt][i] *= al;
#pragma unroll
          for (int mt = 0; mt < 8; ++mt)
#pragma unroll
            for (int i = 0; i < 4; ++i) O[mt][nt][i] *= al;
          const float alv = alpha_s[(gid >> 1) + 4 * nt];
#pragma unroll
          for (int g = 0; g < 8; ++g) cm[nt][g] *= alv;
        }
#pragma unroll
        for (int h = 0; h < HP; ++h) {
          const float al = alpha_s[h];
#pragma unroll
          for (int j = 0; j < 4; ++j) ocorr[h][j] *= al;
        }
      }
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        m_run[nt] = m_new[nt];
        const int h = t + 4 * nt;
        for (int slab = 0; slab < nslab; ++slab)
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            const int tok = slab * kSlab + gid + 8 * half;
            const float sc = ps[h * max_T + tok];
            const float p = (sc == -INFINITY) ? 0.f : exp2f(sc - m_new[nt]);
            ps[h * max_T + tok] = p;
            l_run[nt] += p;
          }
      }
      __syncwarp();

      // ---------------- values: out += sum_tok p' * code (tensor cores), constants and low rank on the side
      const int ngv = is_buf ? 1 : a.cc.ngv, gv = is_buf ? kHeadDim : a.cc.g_v;
      for (int slab = 0; slab < nslab; ++slab) {
        uint32_t av[8][4];
        if (!is_buf) {
          const uint4* cw = reinterpret_cast<const uint4*>(rec + sd.off_vcodes + slab * sd.slab_codes);
          if (BITS == 2) {
            const uint4 w = cw[lane];
            const uint32_t wv[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) {
              uint32_t r[8];
              unpack_word<2>(wv[q4], r);
#pragma unroll
              for (int u2 = 0; u2 < 8; ++u2) av[2 * q4 + (u2 >> 2)][u2 & 3] = r[u2];
            }
          } else {
#pragma unroll
            for (int pl = 0; pl < 2; ++pl) {
              const uint4 w = cw[pl * 32 + lane];
              const uint32_t wv[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
              for (int q4 = 0; q4 < 4; ++q4) unpack_word<4>(wv[q4], av[4 * pl + q4]);
            }
          }
        } else {
#pragma unroll
          for (int mt = 0; mt < 8; ++mt)
            ldmatrix_x4_trans(av[mt], st + (kSlab + (lane & 7) + 8 * (lane >> 4)) * kBufPitch +
                                          (16 * mt + 8 * ((lane >> 3) & 1)) * 2);
        }
        const int part = gid & 1;
        float p4[NT][4];
        uint32_t bp[NT][2];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          const float* pr = ps + ((gid >> 1) + 4 * nt) * max_T + slab * kSlab + 2 * t;
          const float2 pa = *reinterpret_cast<const float2*>(pr), pb = *reinterpret_cast<const float2*>(pr + 8);
          p4[nt][0] = pa.x; p4[nt][1] = pa.y; p4[nt][2] = pb.x; p4[nt][3] = pb.y;
          bp[nt][0] = split_h2(pa.x, pa.y, part);
          bp[nt][1] = split_h2(pb.x, pb.y, part);
        }
        for (int g = 0; g < ngv; ++g) {
          float vs[4] = {1.f, 1.f, 1.f, 1.f}, vz[4] = {0.f, 0.f, 0.f, 0.f};
          if (!is_buf) {
            const __half2* vsz = reinterpret_cast<const __half2*>(rec + sd.off_vscale);
            const int tk[4] = {2 * t, 2 * t + 1, 2 * t + 8, 2 * t + 9};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const __half2 z = vsz[(slab * kSlab + tk[i]) * ngv + g];
              vs[i] = __low2float(z); vz[i] = __high2float(z);
            }
          }
          uint32_t bv[NT][2];
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) {
            bv[nt][0] = split_h2(p4[nt][0] * vs[0], p4[nt][1] * vs[1], part);
            bv[nt][1] = split_h2(p4[nt][2] * vs[2], p4[nt][3] * vs[3], part);
            if (part == 0) {
              const float c = fmaf(p4[nt][0], vz[0], fmaf(p4[nt][1], vz[1], fmaf(p4[nt][2], vz[2], p4[nt][3] * vz[3])));
#pragma unroll
              for (int gg = 0; gg < 8; ++gg) if (gg == g) cm[nt][gg] += c;
            }
          }
#pragma unroll
          for (int mt = 0; mt < 8; ++mt) {
            if ((mt * 16) / gv == g) {
#pragma unroll
              for (int nt = 0; nt < NT; ++nt) mma16816(O[mt][nt], av[mt], bv[nt][0], bv[nt][1]);
            }
          }
        }
        if (r_pad > 0) {                          // low-rank value term, first product: U = A_V^T p
          const __half* avs = reinterpret_cast<const __half*>(rec + sd.off_av + slab * sd.slab_a);
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
      }
      // ---------------- sparse value term: p[tok] * (x - zero[tok, g]) scattered to the outlier's channel
      if (!is_buf && a.cc.k_v > 0) {
        const int per_tok = ngv * 2 * a.cc.k_v, n_ent = T * per_tok;
        const __half* ov = reinterpret_cast<const __half*>(rec + sd.off_voval);
        const unsigned char* oi = rec + sd.off_voidx;
        const __half2* vsz = reinterpret_cast<const __half2*>(rec + sd.off_vscale);
        float S[HP], Si[HP];
#pragma unroll
        for (int h = 0; h < HP; ++h) fixed_scale(pmax_s[h] * dmax_v, S[h], Si[h]);
        for (int e = lane; e < n_ent; e += 32) {
          const int tok = e / per_tok, g = (e % per_tok) / (2 * a.cc.k_v);
          const float d = __half2float(ov[e]) - __high2float(vsz[tok * ngv + g]);
          const int ch = g * gv + oi[e];
#pragma unroll
          for (int h = 0; h < HP; ++h)
            if (h < HPu) atomicAdd(&corr_v[h * kHeadDim + ch], __float2int_rn(ps[h * max_T + tok] * d * S[h]));
        }
        __syncwarp();
#pragma unroll
        for (int h = 0; h < HP; ++h) {
          if (h < HPu) {
            int4* cv = reinterpret_cast<int4*>(corr_v + h * kHeadDim) + lane;
            const int4 v = *cv;
            *cv = make_int4(0, 0, 0, 0);
            ocorr[h][0] = fmaf((float)v.x, Si[h], ocorr[h][0]);
            ocorr[h][1] = fmaf((float)v.y, Si[h], ocorr[h][1]);
            ocorr[h][2] = fmaf((float)v.z, Si[h], ocorr[h][2]);
            ocorr[h][3] = fmaf((float)v.w, Si[h], ocorr[h][3]);
          }
        }
      }
      // ---------------- end of a segment (or of this warp's share of it): out += B_V U
      if (!is_buf && u_pending && seg_last_block) {
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
          const int h = (gid >> 1) + 4 * nt, part = gid & 1;
          bu[nt][0] = split_h2(wl[(2 * t) * HP + h], wl[(2 * t + 1) * HP + h], part);
          bu[nt][1] = split_h2(wl[(2 * t + 8) * HP + h], wl[(2 * t + 9) * HP + h], part);
        }
#pragma unroll
        for (int mt = 0; mt < 8; ++mt) {
          uint32_t aa[4] = {0u, 0u, 0u, 0u};
          const __half* r0 = keep_bv + (16 * mt + gid) * r_pad, *r1 = keep_bv + (16 * mt + gid + 8) * r_pad;
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
        __syncwarp();
      }
      // ---------------- this stage is free again: fetch the block kStages ahead
      __syncwarp();
      ++n_consumed;
      issue();
    }
    if (!alive) break;

    // ---------------- partial result of this unit: (m, l, o) per head
    const long long bflat = u * NB, eflat = bflat + NB;
    const long long w_first = ((bflat + 1) * NW + F - 1) / F - 1;
    const long long w_last = (eflat * NW + F - 1) / F - 1;
    const int n_parts = (int)(w_last - w_first + 1);
    const int slot = (int)(gw - w_first);
    float* part_base = a.partial + ((size_t)u * a.max_parts + slot) * (HP * 130);
    __syncwarp();
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      float l = l_run[nt];
      l += __shfl_xor_sync(0xffffffffu, l, 4);
      l += __shfl_xor_sync(0xffffffffu, l, 8);
      l += __shfl_xor_sync(0xffffffffu, l, 16);
      l_run[nt] = l;
#pragma unroll
      for (int g = 0; g < 8; ++g) {
        float c = cm[nt][g];
        c += __shfl_xor_sync(0xffffffffu, c, 1);
        c += __shfl_xor_sync(0xffffffffu, c, 2);
        if (t == 0 && (gid & 1) == 0) cm_s[((gid >> 1) + 4 * nt) * 8 + g] = c;
      }
    }
    float* oc = reinterpret_cast<float*>(corr_v);          // borrow as fp32 [HP][128]
#pragma unroll
    for (int h = 0; h < HP; ++h)
      *reinterpret_cast<float4*>(oc + h * kHeadDim + lane * 4) =
          make_float4(ocorr[h][0], ocorr[h][1], ocorr[h][2], ocorr[h][3]);
    __syncwarp();
    const int gvc = a.cc.g_v;
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
            dst[ch] = O[mt][nt][2 * half] + O[mt][nt][2 * half + 1] + oc[h * kHeadDim + ch] + cm_s[h * 8 + ch / gvc];
          }
        if (gid == 0) { dst[128] = m_run[nt]; dst[129] = l_run[nt]; }
      }
    }
    __syncwarp();
    for (int i = lane; i < HP * kHeadDim; i += 32) corr_v[i] = 0;
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
    if (empty_range) break;
    f += blk_hi - blk_lo;
  }
  // a warp that gave up still has copies in flight: let them land (bounded) before leaving
  if (!alive) {
    for (int i = n_consumed; i < n_issued; ++i) {
      const int s = i % kStages;
      for (int k = 0; k < kSpinLimit && !mbar_try(&bar[s], (uint32_t)((i / kStages) & 1)); ++k) {}
    }
  }
}

cudaError_t launch_decode(const DecodeArgs& a, int warps_per_cta, int grid, size_t smem, cudaStream_t st) {
  const int G = a.group_heads;
#define GEAR_DEC(B, N)                                                                                         \
  {                                                                                                            \
    cudaError_t e = cudaFuncSetAttribute(gear_decode_kernel<B, N>, cudaFuncAttributeMaxDynamicSharedMemorySize, \
                                         (int)smem);                                                          \
    if (e != cudaSuccess) return e;                                                                            \
    gear_decode_kernel<B, N><<<grid, warps_per_cta * 32, smem, st>>>(a);                                       \
  }
  if (a.cc.bits == 2) { if (G <= 4) GEAR_DEC(2, 1) else GEAR_DEC(2, 2) }
  else { if (G <= 4) GEAR_DEC(4, 1) else GEAR_DEC(4, 2) }
#undef GEAR_DEC
  count_launches(1);
  return cudaGetLastError();
}

int decode_occupancy(int bits, int G, int warps_per_cta, size_t smem) {
  int occ = 0;
  cudaError_t e;
  if (bits == 2) {
    if (G <= 4) {
      cudaFuncSetAttribute(gear_decode_kernel<2, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, gear_decode_kernel<2, 1>, warps_per_cta * 32, smem);
    } else {
      cudaFuncSetAttribute(gear_decode_kernel<2, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, gear_decode_kernel<2, 2>, warps_per_cta * 32, smem);
    }
  } else {
    if (G <= 4) {
      cudaFuncSetAttribute(gear_decode_kernel<4, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, gear_decode_kernel<4, 1>, warps_per_cta * 32, smem);
    } else {
      cudaFuncSetAttribute(gear_decode_kernel<4, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, gear_decode_kernel<4, 2>, warps_per_cta * 32, smem);
    }
  }
  if (e != cudaSuccess) { cudaGetLastError(); return 0; }
  return occ;
}

}  // namespace gear
