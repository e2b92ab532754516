// GEAR compression of one segment (Algorithm 1, prefill body / buffer flush):
//   quant_pack_kernel : Filter_s (Eq. 4), Quant_b(X - S) (Eq. 2, Eq. 5), packing, residual R = X - D^ - S
//   pi_* kernels      : SVDSolver (Algorithm 2) on every head's residual R_h, batch-wise and head-wise
// All arithmetic that decides a code is a fixed sequence of binary32 operations
// (round-to-nearest-even, no fused multiply-add, no fast-math).
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <math.h>

#include "gear_internal.cuh"

namespace gear {

// ---------------------------------------------------------------------------
// Filter + Quant + pack for one block (T tokens x 128 channels) of K or V.
// ---------------------------------------------------------------------------
constexpr int kXPitch = 130;   // halves per row of the fp16 tile in shared memory
constexpr int kRPitch = 129;   // floats per row of the residual tile

struct TopList {
  float v[kMaxOutliers];
  int i[kMaxOutliers];
};

// (value, index) order used by Filter_s: larger value first (smaller for the
// bottom list), then lower index.
template <bool TOP>
__device__ __forceinline__ bool goes_before(float va, int ia, float vb, int ib) {
  if (ib < 0) return ia >= 0;
  if (ia < 0) return false;
  if (TOP ? (va > vb) : (va < vb)) return true;
  return va == vb && ia < ib;
}

template <int KMAX, bool TOP>
__device__ __forceinline__ void list_insert(TopList& l, int k, float v, int idx) {
#pragma unroll
  for (int s = 0; s < KMAX; ++s) {
    if (s < k && goes_before<TOP>(v, idx, l.v[s], l.i[s])) {
      float tv = l.v[s]; int ti = l.i[s];
      l.v[s] = v; l.i[s] = idx;
      v = tv; idx = ti;
    }
  }
}

template <int KMAX>
__device__ __forceinline__ bool list_has(const TopList& l, int k, int idx) {
  bool h = false;
#pragma unroll
  for (int s = 0; s < KMAX; ++s) h |= (s < k && l.i[s] == idx);
  return h;
}

struct GroupResult {
  __half scale, zero;
  float dmax;   // max |x - zero| over the group's outliers
};

// One quantization group of `len` entries reached through x_at(e); writes the
// code and residual of every entry through put(e, code, resid) and the sorted
// outlier list (in-group index ascending) through put_out(slot, idx, value).
template <int BITS, int KMAX, class XAt, class Put, class PutOut>
__device__ __forceinline__ GroupResult process_group(int len, int k, XAt x_at, Put put, PutOut put_out) {
  TopList top, bot;
#pragma unroll
  for (int s = 0; s < KMAX; ++s) { top.v[s] = 0.f; top.i[s] = -1; bot.v[s] = 0.f; bot.i[s] = -1; }
  float mn = INFINITY, mx = -INFINITY;
  if (KMAX == 1 && k == 1) {
    // One outlier per side: a single pass finds the first maximum, the first minimum and the second largest /
    // second smallest instances, which bound the kept entries.  (The first maximum is also the first minimum
    // only when all entries are equal; the bottom entry is then the next index.)
    float max1 = -INFINITY, max2 = -INFINITY, min1 = INFINITY, min2 = INFINITY;
    int imax = 0, imin = 0;
    for (int e = 0; e < len; ++e) {
      const float x = x_at(e);
      if (x > max1) { max2 = max1; max1 = x; imax = e; } else if (x > max2) { max2 = x; }
      if (x < min1) { min2 = min1; min1 = x; imin = e; } else if (x < min2) { min2 = x; }
    }
    if (imin == imax) imin = 1;
    top.v[0] = max1; top.i[0] = imax;
    bot.v[0] = min1; bot.i[0] = imin;
    mn = min2; mx = max2;
  } else {
    if (k > 0) {
      for (int e = 0; e < len; ++e) list_insert<KMAX, true>(top, k, x_at(e), e);
      for (int e = 0; e < len; ++e)
        if (!list_has<KMAX>(top, k, e)) list_insert<KMAX, false>(bot, k, x_at(e), e);
    }
    for (int e = 0; e < len; ++e) {
      if (k > 0 && (list_has<KMAX>(top, k, e) || list_has<KMAX>(bot, k, e))) continue;
      const float x = x_at(e);
      mn = fminf(mn, x);
      mx = fmaxf(mx, x);
    }
  }
  // Eq. 2 on the kept entries: binary32, one rounding per operation.
  const float levels = (float)((1 << BITS) - 1);
  const float range = __fsub_rn(mx, mn);
  const float d32 = __fdiv_rn(range, levels);
  const __half d16 = __float2half_rn(d32);
  const float d = __half2float(d16);
  const float inv = d != 0.f ? __fdiv_rn(1.0f, d) : 0.f;
  for (int e = 0; e < len; ++e) {
    const float x = x_at(e);
    const bool out = k > 0 && (list_has<KMAX>(top, k, e) || list_has<KMAX>(bot, k, e));
    int code = 0;
    float resid = 0.f;
    if (!out) {
      if (d != 0.f) {
        const float t = __fmul_rn(__fsub_rn(x, mn), inv);
        code = (int)fminf(fmaxf(rintf(t), 0.f), levels);
      }
      resid = x - fmaf((float)code, d, mn);
    }
    put(e, code, resid);
  }
  GroupResult r;
  r.scale = d16;
  r.zero = __float2half_rn(mn);
  r.dmax = 0.f;
  if (k > 0) {
    // merge the two lists by index: rank of each entry among the 2k
#pragma unroll
    for (int a = 0; a < 2 * KMAX; ++a) {
      const bool from_top = a < KMAX;
      const int s = from_top ? a : a - KMAX;
      if (s >= k) continue;
      const int ia = from_top ? top.i[s] : bot.i[s];
      const float va = from_top ? top.v[s] : bot.v[s];
      int rank = 0;
#pragma unroll
      for (int b = 0; b < KMAX; ++b) {
        rank += (b < k && top.i[b] < ia);
        rank += (b < k && bot.i[b] < ia);
      }
      put_out(rank, ia, va);
      r.dmax = fmaxf(r.dmax, fabsf(va - mn));
    }
  }
  return r;
}

// Pack the codes of one block (T tokens x 128 channels, xs[token * kXPitch + channel]) into the fragment order of
// the integer tensor-core product (gear_layout.cuh); one 32-bit word per thread and step, stores coalesced.
template <int BITS>
__device__ __forceinline__ void pack_block_codes(const unsigned short* xs, int T, int side, unsigned int* dst, int tid,
                                                 int nthreads) {
  constexpr int F = 8 / BITS;
  if (side == 0) {
    constexpr int kWords = kSlab * kHeadDim * BITS / 32;            // words per slab
    for (int li = tid; li < ((T + kSlab - 1) / kSlab) * kWords; li += nthreads) {
      const int slab = li / kWords, wl = li % kWords;
      const int w = wl & 3, lane = (wl >> 2) & 31, tau = wl >> 7;
      unsigned int word = 0;
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < F; ++j) {
          int tok, ch;
          code_coord_k(BITS, lane, tau, w, i, j, tok, ch);
          tok += slab * kSlab;
          if (tok < T) word |= (unsigned int)xs[tok * kXPitch + ch] << (8 * i + BITS * j);
        }
      dst[li] = word;
    }
  } else {
    constexpr int kWords = 32 * kHeadDim * BITS / 32;               // words per 32-token chunk
    const int nchunk = (T + 31) / 32;
    for (int li = tid; li < nchunk * kWords; li += nthreads) {
      const int chunk = li / kWords, wl = li % kWords;
      const int w = wl & 3, lane = (wl >> 2) & 31, tau = wl >> 7;
      unsigned int word = 0;
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < F; ++j) {
          int tok, ch;
          code_coord_v(BITS, lane, tau, w, i, j, tok, ch);
          tok += chunk * 32;
          if (tok < T) word |= (unsigned int)xs[tok * kXPitch + ch] << (8 * i + BITS * j);
        }
      dst[li] = word;
    }
  }
}

template <int BITS, int KMAX>
__global__ void __launch_bounds__(128) quant_pack_kernel(CompressArgs p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const SegDesc& sd = p.seg;
  const int T = sd.T;
  const int side = blockIdx.z + p.side0, bhl = blockIdx.y, blk = blockIdx.x, tid = threadIdx.x;
  unsigned short* xs = reinterpret_cast<unsigned short*>(smem_raw);   // fp16 bits of the block; each entry is replaced by its code
  float* rs = reinterpret_cast<float*>(smem_raw + round_up(T * kXPitch * 2, 16));
  auto x_of = [&](int idx) { return __half2float(__ushort_as_half(xs[idx])); };
  __shared__ unsigned int dmax_bits, smax_bits;
  if (tid == 0) { dmax_bits = 0u; smax_bits = 0u; }

  const __half* X = (side == 0 ? p.K : p.V) + ((size_t)bhl * sd.n_c + (size_t)blk * T) * kHeadDim;
  for (int i = tid; i < T * 16; i += 128) {
    const int row = i >> 4, c = i & 15;
    const uint4 v = *reinterpret_cast<const uint4*>(X + row * kHeadDim + c * 8);
    unsigned int* dst = reinterpret_cast<unsigned int*>(xs + row * kXPitch + c * 8);
    dst[0] = v.x; dst[1] = v.y; dst[2] = v.z; dst[3] = v.w;
  }
  __syncthreads();

  unsigned char* rec = p.arena + sd.seg_base + (size_t)(p.bh0 + bhl) * sd.bh_stride + sd.bfac_bytes +
                       (size_t)blk * sd.rec_bytes;
  float my_dmax = 0.f, my_smax = 0.f;
  if (side == 0) {
    // keys: one group per channel over the T tokens of the block (per-channel grouping)
    const int j = tid;
    const int k = sd.k_k;
    __half* oval = reinterpret_cast<__half*>(rec + sd.off_koval) + j * 2 * k;
    unsigned char* oidx = rec + sd.off_koidx + j * 2 * k;
    GroupResult g = process_group<BITS, KMAX>(
        T, k, [&](int e) { return x_of(e * kXPitch + j); },
        [&](int e, int code, float r) { xs[e * kXPitch + j] = (unsigned short)code; rs[e * kRPitch + j] = r; },
        [&](int slot, int idx, float v) { oval[slot] = __float2half_rn(v); oidx[slot] = (unsigned char)idx; });
    reinterpret_cast<__half2*>(rec + sd.off_kscale)[j] = __halves2half2(g.scale, g.zero);
    my_dmax = g.dmax;
    my_smax = __half2float(g.scale);
  } else {
    // values: one group per token over g_V consecutive channels (per-token grouping)
    const int k = p.cc.k_v, gv = p.cc.g_v, ngv = p.cc.ngv;
    for (int gi = tid; gi < T * ngv; gi += 128) {
      const int tok = gi / ngv, c = gi % ngv;
      __half* oval = reinterpret_cast<__half*>(rec + sd.off_voval) + gi * 2 * k;
      unsigned char* oidx = rec + sd.off_voidx + gi * 2 * k;
      GroupResult g = process_group<BITS, KMAX>(
          gv, k, [&](int e) { return x_of(tok * kXPitch + c * gv + e); },
          [&](int e, int code, float r) {
            xs[tok * kXPitch + c * gv + e] = (unsigned short)code;
            rs[tok * kRPitch + c * gv + e] = r;
          },
          [&](int slot, int idx, float v) { oval[slot] = __float2half_rn(v); oidx[slot] = (unsigned char)idx; });
      reinterpret_cast<__half2*>(rec + sd.off_vscale)[gi] = __halves2half2(g.scale, g.zero);
      my_dmax = fmaxf(my_dmax, g.dmax);
      my_smax = fmaxf(my_smax, __half2float(g.scale));
    }
  }
  atomicMax(&dmax_bits, __float_as_uint(my_dmax));   // non-negative floats order like their bit patterns
  atomicMax(&smax_bits, __float_as_uint(my_smax));
  __syncthreads();
  if (tid == 0) {
    reinterpret_cast<float*>(rec)[side] = __uint_as_float(dmax_bits);
    reinterpret_cast<float*>(rec)[2 + side] = __uint_as_float(smax_bits);
  }

  // pack the codes into mma-fragment order
  pack_block_codes<BITS>(xs, T, side, reinterpret_cast<unsigned int*>(rec + (side == 0 ? sd.off_kcodes : sd.off_vcodes)),
                         tid, 128);
  // residual tile -> workspace (only needed when a low-rank part is fitted)
  if (p.R != nullptr) {
    float* R = p.R + (((size_t)bhl * 2 + side) * sd.n_c + (size_t)blk * T) * kHeadDim;
    float rmax = 0.f;
    for (int i = tid; i < T * kHeadDim; i += 128) {
      const float v = rs[(i >> 7) * kRPitch + (i & 127)];
      R[i] = v;
      rmax = fmaxf(rmax, fabsf(v));
    }
    // the largest residual magnitude of the (batch, head, side) tile: the power iteration scales by it
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) rmax = fmaxf(rmax, __shfl_xor_sync(0xffffffffu, rmax, o));
    if ((tid & 31) == 0) atomicMax(p.Rmax + bhl * 2 + side, __float_as_uint(rmax));
  }
}

// ---------------------------------------------------------------------------
// The same step for the common shape -- blocks of 64 tokens, value groups of 64 channels, one outlier per side and
// group (s <= 3.1 %) -- with the group in registers: a thread owns one group (keys: a channel's 64 tokens, read as a
// column; values: 64 consecutive channels of a token), walks it in fully unrolled loops, stores the residual itself and
// leaves only the codes in shared memory, one byte each, transposed so that the packing step fetches the four codes
// of an output byte row with one 32-bit load.  Every code, scale, outlier and residual is bit-identical to
// quant_pack_kernel: the operations on a group are the same binary32 sequence.
// ---------------------------------------------------------------------------
constexpr int kFastLen = 64;
constexpr int kCodePitchK = kHeadDim + 4;   // bytes per token row of the key codes  [token][channel]
constexpr int kCodePitchV = kFastLen + 4;   // bytes per channel row of the value codes [channel][token]

// Value side, shared-memory staging (a thread's 64 channels are contiguous in memory, so direct accesses of a warp
// would touch 32 lines each): the fp16 tile comes in with coalesced loads, the fp32 residual tile leaves the same way.
// Row (c, token) of the fp16 tile holds the 64 channels of group c; rows are 36 words apart and the second group
// starts 16 words late, rows of the residual tile are 164 words with group 1 at word 80: both make the 128-bit
// accesses of a quarter warp (four tokens x two groups) hit 32 different banks.
constexpr int kStageRowWords = 36, kStageGroupSkew = 16;
constexpr int kResPitch = 164, kResGroup = 80;
constexpr int kFastSmemV = kFastLen * kResPitch * 4;     // the residual tile; the fp16 tile lives in it first

template <int BITS, int SIDE>
__global__ void __launch_bounds__(128) quant_fast_kernel(CompressArgs p) {
  constexpr int L = kFastLen, F = 8 / BITS;
  constexpr int side = SIDE;
  extern __shared__ __align__(16) unsigned char stage_raw[];    // value side only
  __shared__ __align__(16) unsigned char codes[SIDE == 0 ? L * kCodePitchK : kHeadDim * kCodePitchV];
  __shared__ unsigned int dmax_bits, smax_bits, rmax_bits;
  const SegDesc& sd = p.seg;
  const int bhl = blockIdx.y, blk = blockIdx.x, tid = threadIdx.x;
  if (tid == 0) { dmax_bits = 0u; smax_bits = 0u; rmax_bits = 0u; }
  const __half* X = (side == 0 ? p.K : p.V) + ((size_t)bhl * sd.n_c + (size_t)blk * L) * kHeadDim;
  float* R = p.R ? p.R + (((size_t)bhl * 2 + side) * sd.n_c + (size_t)blk * L) * kHeadDim : nullptr;
  unsigned char* rec = p.arena + sd.seg_base + (size_t)(p.bh0 + bhl) * sd.bh_stride + sd.bfac_bytes +
                       (size_t)blk * sd.rec_bytes;
  // element e of this thread's group sits at X[first + e * step]
  const int first = side == 0 ? tid : (tid >> 1) * kHeadDim + (tid & 1) * L;
  const int step = side == 0 ? kHeadDim : 1;
  float* rs = reinterpret_cast<float*>(stage_raw);

  // the group as 32 packed pairs (entries 2q, 2q + 1)
  __half2 xp[L / 2];
  if (side == 0) {
#pragma unroll
    for (int q = 0; q < L / 2; ++q) xp[q] = __halves2half2(X[first + (2 * q) * kHeadDim], X[first + (2 * q + 1) * kHeadDim]);
  } else {
    uint4* xs = reinterpret_cast<uint4*>(stage_raw);
    for (int i = tid; i < L * 16; i += 128) {           // 16-byte pieces of the tile, in memory order
      const int tok = i >> 4, c = (i >> 3) & 1, q = i & 7;
      xs[(((c * L + tok) * kStageRowWords + c * kStageGroupSkew) >> 2) + q] = reinterpret_cast<const uint4*>(X)[i];
    }
    __syncthreads();
    const int tok = tid >> 1, c = tid & 1;
    const uint4* src = xs + (((c * L + tok) * kStageRowWords + c * kStageGroupSkew) >> 2);
#pragma unroll
    for (int q = 0; q < L / 8; ++q) {
      const uint4 v = src[q];
      xp[4 * q] = *reinterpret_cast<const __half2*>(&v.x);
      xp[4 * q + 1] = *reinterpret_cast<const __half2*>(&v.y);
      xp[4 * q + 2] = *reinterpret_cast<const __half2*>(&v.z);
      xp[4 * q + 3] = *reinterpret_cast<const __half2*>(&v.w);
    }
    __syncthreads();                                     // the residual tile takes the place of the fp16 tile
  }
  // Filter_s (Eq. 4), one entry per side: the largest and the smallest entry leave the group, the second largest and
  // second smallest instances bound what is kept.  Comparisons of fp16 values are exact in fp16, so the search runs on
  // the packed pairs: even and odd entries keep their own two largest / smallest and are merged at the end.
  float max1, max2, min1, min2;
  {
    const __half2 ninf = __float2half2_rn(-INFINITY), pinf = __float2half2_rn(INFINITY);
    __half2 M1 = ninf, M2 = ninf, m1 = pinf, m2 = pinf;
#pragma unroll
    for (int q = 0; q < L / 2; ++q) {
      M2 = __hmax2(M2, __hmin2(xp[q], M1));
      M1 = __hmax2(M1, xp[q]);
      m2 = __hmin2(m2, __hmax2(xp[q], m1));
      m1 = __hmin2(m1, xp[q]);
    }
    const float2 fM1 = __half22float2(M1), fM2 = __half22float2(M2), fm1 = __half22float2(m1), fm2 = __half22float2(m2);
    max1 = fmaxf(fM1.x, fM1.y);
    max2 = fmaxf(fminf(fM1.x, fM1.y), fmaxf(fM2.x, fM2.y));
    min1 = fminf(fm1.x, fm1.y);
    min2 = fminf(fmaxf(fm1.x, fm1.y), fminf(fm2.x, fm2.y));
  }
  // first index of the maximum and of the minimum (ties go to the lower index): one mask bit per entry
  int imax, imin;
  {
    const __half2 vM = __float2half2_rn(max1), vm = __float2half2_rn(min1);
    unsigned int a0 = 0u, a1 = 0u, b0 = 0u, b1 = 0u;   // bit q of a half word: pair q (a0, b0) or pair 16 + q (a1, b1)
#pragma unroll
    for (int q = 0; q < L / 2; ++q) {
      const unsigned int bit = 0x00010001u << (q & 15);
      const unsigned int eM = __heq2_mask(xp[q], vM) & bit, em = __heq2_mask(xp[q], vm) & bit;
      if (q < 16) { a0 |= eM; b0 |= em; } else { a1 |= eM; b1 |= em; }
    }
    auto first_set = [](unsigned int lo16, unsigned int hi16) {
      const unsigned int even = __byte_perm(lo16, hi16, 0x5410);   // bit q: entry 2 q
      const unsigned int odd = __byte_perm(lo16, hi16, 0x7632);    // bit q: entry 2 q + 1
      const int fe = even ? 2 * (__ffs((int)even) - 1) : L;
      const int fo = odd ? 2 * (__ffs((int)odd) - 1) + 1 : L;
      return min(fe, fo);
    };
    imax = first_set(a0, a1);
    imin = first_set(b0, b1);
  }
  if (imin == imax) imin = 1;               // all entries equal: the bottom entry is the next index
  const float mn = min2, mx = max2;
  // Eq. 2 on the kept entries: binary32, one rounding per operation
  const float levels = (float)((1 << BITS) - 1);
  const float range = __fsub_rn(mx, mn);
  const float d32 = __fdiv_rn(range, levels);
  const __half d16 = __float2half_rn(d32);
  const float d = __half2float(d16);
  const float inv = d != 0.f ? __fdiv_rn(1.0f, d) : 0.f;
  // Codes and residuals are computed for every entry as if it were kept; the two filtered entries are cleared
  // afterwards.  round-to-nearest-even of the clamped quotient by adding 1.5 * 2^23: the code is the low byte of the sum.
  constexpr float kRound = 12582912.0f;
  auto quantize = [&](float x, unsigned int& code) {
    const float t = __fmul_rn(__fsub_rn(x, mn), inv);
    const float y = __fadd_rn(fminf(fmaxf(t, 0.f), levels), kRound);
    code = __float_as_uint(y) & 0xFFu;
    return x - fmaf(__fsub_rn(y, kRound), d, mn);
  };
  if (side == 0) {
#pragma unroll
    for (int q = 0; q < L / 2; ++q) {
      const float2 f = __half22float2(xp[q]);
      unsigned int c0, c1;
      const float r0 = quantize(f.x, c0), r1 = quantize(f.y, c1);
      codes[(2 * q) * kCodePitchK + tid] = (unsigned char)c0;
      codes[(2 * q + 1) * kCodePitchK + tid] = (unsigned char)c1;
      if (R != nullptr) {
        R[(2 * q) * kHeadDim + tid] = r0;
        R[(2 * q + 1) * kHeadDim + tid] = r1;
      }
    }
    codes[imax * kCodePitchK + tid] = 0;
    codes[imin * kCodePitchK + tid] = 0;
    if (R != nullptr) {
      R[imax * kHeadDim + tid] = 0.f;
      R[imin * kHeadDim + tid] = 0.f;
    }
  } else {
    const int tok = tid >> 1, c0 = (tid & 1) * L;
    float* rrow = rs + tok * kResPitch + (tid & 1) * kResGroup;
#pragma unroll
    for (int q = 0; q < L / 4; ++q) {
      const float2 f0 = __half22float2(xp[2 * q]), f1 = __half22float2(xp[2 * q + 1]);
      unsigned int k0, k1, k2, k3;
      const float4 rr = make_float4(quantize(f0.x, k0), quantize(f0.y, k1), quantize(f1.x, k2), quantize(f1.y, k3));
      codes[(c0 + 4 * q) * kCodePitchV + tok] = (unsigned char)k0;
      codes[(c0 + 4 * q + 1) * kCodePitchV + tok] = (unsigned char)k1;
      codes[(c0 + 4 * q + 2) * kCodePitchV + tok] = (unsigned char)k2;
      codes[(c0 + 4 * q + 3) * kCodePitchV + tok] = (unsigned char)k3;
      *reinterpret_cast<float4*>(rrow + 4 * q) = rr;
    }
    codes[(c0 + imax) * kCodePitchV + tok] = 0;
    codes[(c0 + imin) * kCodePitchV + tok] = 0;
    rrow[imax] = 0.f;
    rrow[imin] = 0.f;
  }
  // A bound on the group's residuals instead of their maximum (it only picks the power of two the power iteration
  // scales by): half a step for a kept entry, the whole range if the step rounded to zero, plus the rounding of the
  // dequantised value
  float rmax = (d != 0.f ? 0.50390625f * d : range) + 2.4e-7f * (fabsf(mn) + fabsf(mx));
  // the group's scale, zero point and its two outliers (in-group index ascending)
  {
    const __half vmax = X[first + imax * step], vmin = X[first + imin * step];
    const bool max_first = imax < imin;
    const __half2 ov = max_first ? __halves2half2(vmax, vmin) : __halves2half2(vmin, vmax);
    const uchar2 oi = max_first ? make_uchar2((unsigned char)imax, (unsigned char)imin)
                                : make_uchar2((unsigned char)imin, (unsigned char)imax);
    reinterpret_cast<__half2*>(rec + (side == 0 ? sd.off_koval : sd.off_voval))[tid] = ov;
    reinterpret_cast<uchar2*>(rec + (side == 0 ? sd.off_koidx : sd.off_voidx))[tid] = oi;
    reinterpret_cast<__half2*>(rec + (side == 0 ? sd.off_kscale : sd.off_vscale))[tid] =
        __halves2half2(d16, __float2half_rn(mn));
    float dm = fmaxf(fabsf(__half2float(vmax) - mn), fabsf(__half2float(vmin) - mn));
    float sm = d;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      dm = fmaxf(dm, __shfl_xor_sync(0xffffffffu, dm, o));
      sm = fmaxf(sm, __shfl_xor_sync(0xffffffffu, sm, o));
      rmax = fmaxf(rmax, __shfl_xor_sync(0xffffffffu, rmax, o));
    }
    if ((tid & 31) == 0) {                   // non-negative floats order like their bit patterns
      atomicMax(&dmax_bits, __float_as_uint(dm));
      atomicMax(&smax_bits, __float_as_uint(sm));
      atomicMax(&rmax_bits, __float_as_uint(rmax));
    }
  }
  __syncthreads();
  if (tid == 0) {
    reinterpret_cast<float*>(rec)[side] = __uint_as_float(dmax_bits);
    reinterpret_cast<float*>(rec)[2 + side] = __uint_as_float(smax_bits);
    if (R != nullptr) atomicMax(p.Rmax + bhl * 2 + side, rmax_bits);
  }
  if (side == 1 && R != nullptr) {
    for (int i = tid; i < L * 32; i += 128) {            // 16-byte pieces of the residual tile, in memory order
      const int tok = i >> 5, c = (i >> 4) & 1, q = i & 15;
      reinterpret_cast<float4*>(R)[i] = *reinterpret_cast<const float4*>(rs + tok * kResPitch + c * kResGroup + 4 * q);
    }
  }
  // pack the codes into mma-fragment order (code_coord_k / code_coord_v): the four codes of a byte row are neighbours
  // in shared memory, a field of the word is one 32-bit load shifted into place
  unsigned int* dst = reinterpret_cast<unsigned int*>(rec + (side == 0 ? sd.off_kcodes : sd.off_vcodes));
  if (side == 0) {
    constexpr int kWords = kSlab * kHeadDim * BITS / 32;            // words per slab
    for (int li = tid; li < (L / kSlab) * kWords; li += 128) {
      const int slab = li / kWords, wl = li % kWords;
      const int w = wl & 3, lane = (wl >> 2) & 31, tau = wl >> 7;
      const int tok = slab * kSlab + (lane >> 2) + 8 * (w & 1);
      const int ch = 32 * F * tau + 16 * (w >> 1) + 4 * (lane & 3);
      unsigned int word = 0;
#pragma unroll
      for (int j = 0; j < F; ++j)
        word |= *reinterpret_cast<const unsigned int*>(&codes[tok * kCodePitchK + ch + 32 * j]) << (BITS * j);
      dst[li] = word;
    }
  } else {
    constexpr int kWords = 32 * kHeadDim * BITS / 32;               // words per 32-token chunk
    for (int li = tid; li < (L / 32) * kWords; li += 128) {
      const int chunk = li / kWords, wl = li % kWords;
      const int w = wl & 3, lane = (wl >> 2) & 31, tau = wl >> 7;
      const int ch = 16 * F * tau + (lane >> 2) + 8 * (w & 1);
      const int tok = chunk * 32 + 16 * (w >> 1) + 4 * (lane & 3);
      unsigned int word = 0;
#pragma unroll
      for (int j = 0; j < F; ++j)
        word |= *reinterpret_cast<const unsigned int*>(&codes[(ch + 16 * j) * kCodePitchV + tok]) << (BITS * j);
      dst[li] = word;
    }
  }
}

// ---------------------------------------------------------------------------
// Groups of 128 entries with two outliers per side (g = 128 at s = 2 %: keys in blocks of 128 tokens, values one
// group per token), again with the group in registers.  Per half of the packed pairs a chain keeps the three largest
// and three smallest instances; the halves are merged; the entries above / equal to the second largest instance (and
// below / equal to the second smallest) are found as bit masks, which give the two filtered entries per side in
// (value, index) order.  A group in which the two sides would share an entry (nearly constant groups) takes the
// general routine instead.  Same binary32 sequence per entry as everywhere else.
// ---------------------------------------------------------------------------
constexpr int kFast2Len = 128;
constexpr int kCodePitch2 = kFast2Len + 4;

// first set entry of the pair of 64-bit masks (even entries, odd entries), removed from them; 2 * 64 if none
__device__ __forceinline__ int take_first(unsigned long long& even, unsigned long long& odd) {
  const int fe = even ? 2 * (__ffsll((long long)even) - 1) : 2 * 64;
  const int fo = odd ? 2 * (__ffsll((long long)odd) - 1) + 1 : 2 * 64;
  if (fe < fo) { even &= even - 1; return fe; }
  if (fo < 2 * 64) odd &= odd - 1;
  return fo;
}
// four accumulators (bit q of the low / high half word: even / odd entry of pair 16 w + q) -> the two 64-bit masks
__device__ __forceinline__ void masks_of(const unsigned int (&a)[4], unsigned long long& even, unsigned long long& odd) {
  const unsigned int e0 = __byte_perm(a[0], a[1], 0x5410), e1 = __byte_perm(a[2], a[3], 0x5410);
  const unsigned int o0 = __byte_perm(a[0], a[1], 0x7632), o1 = __byte_perm(a[2], a[3], 0x7632);
  even = ((unsigned long long)e1 << 32) | e0;
  odd = ((unsigned long long)o1 << 32) | o0;
}
// the three largest of six values (with multiplicity), in order
__device__ __forceinline__ void top3_of6(float (&v)[6], float (&out)[3]) {
#pragma unroll
  for (int r = 0; r < 3; ++r) {
    float m = v[0];
#pragma unroll
    for (int i = 1; i < 6; ++i) m = fmaxf(m, v[i]);
    out[r] = m;
    bool gone = false;
#pragma unroll
    for (int i = 0; i < 6; ++i) {
      const bool hit = !gone && v[i] == m;
      v[i] = hit ? -INFINITY : v[i];
      gone = gone || hit;
    }
  }
}

template <int BITS, int SIDE>
__global__ void __launch_bounds__(128) quant_fast2_kernel(CompressArgs p) {
  constexpr int L = kFast2Len, F = 8 / BITS;
  __shared__ __align__(16) unsigned char codes[L * kCodePitch2];    // keys [token][channel], values [channel][token]
  __shared__ unsigned int dmax_bits, smax_bits, rmax_bits;
  const SegDesc& sd = p.seg;
  const int T = sd.T;                               // keys: 128; values: tokens (= groups) of the block
  const int bhl = blockIdx.y, blk = blockIdx.x, tid = threadIdx.x;
  if (tid == 0) { dmax_bits = 0u; smax_bits = 0u; rmax_bits = 0u; }
  __syncthreads();
  const __half* X = (SIDE == 0 ? p.K : p.V) + ((size_t)bhl * sd.n_c + (size_t)blk * T) * kHeadDim;
  float* R = p.R ? p.R + (((size_t)bhl * 2 + SIDE) * sd.n_c + (size_t)blk * T) * kHeadDim : nullptr;
  unsigned char* rec = p.arena + sd.seg_base + (size_t)(p.bh0 + bhl) * sd.bh_stride + sd.bfac_bytes +
                       (size_t)blk * sd.rec_bytes;
  const int first = SIDE == 0 ? tid : tid * kHeadDim;      // element e of the group: X[first + e * step]
  const int step = SIDE == 0 ? kHeadDim : 1;
  // where code / residual of element e go
  auto code_at = [&](int e) -> unsigned char& { return codes[e * kCodePitch2 + tid]; };   // row: token (keys) / channel (values)
  const bool active = SIDE == 0 || tid < T;

  if (active) {
    __half2 xp[L / 2];
    if (SIDE == 0) {
#pragma unroll
      for (int q = 0; q < L / 2; ++q) xp[q] = __halves2half2(X[first + (2 * q) * kHeadDim], X[first + (2 * q + 1) * kHeadDim]);
    } else {
      const uint4* src = reinterpret_cast<const uint4*>(X + first);
#pragma unroll
      for (int q = 0; q < L / 8; ++q) {
        const uint4 v = src[q];
        xp[4 * q] = *reinterpret_cast<const __half2*>(&v.x);
        xp[4 * q + 1] = *reinterpret_cast<const __half2*>(&v.y);
        xp[4 * q + 2] = *reinterpret_cast<const __half2*>(&v.z);
        xp[4 * q + 3] = *reinterpret_cast<const __half2*>(&v.w);
      }
    }
    // the three largest / smallest instances of the even and of the odd entries, then of all
    float top[3], bot[3];
    {
      const __half2 ninf = __float2half2_rn(-INFINITY), pinf = __float2half2_rn(INFINITY);
      __half2 M1 = ninf, M2 = ninf, M3 = ninf, m1 = pinf, m2 = pinf, m3 = pinf;
#pragma unroll
      for (int q = 0; q < L / 2; ++q) {
        const __half2 t = __hmin2(xp[q], M1);
        M1 = __hmax2(M1, xp[q]);
        const __half2 u = __hmin2(t, M2);
        M2 = __hmax2(M2, t);
        M3 = __hmax2(M3, u);
        const __half2 tb = __hmax2(xp[q], m1);
        m1 = __hmin2(m1, xp[q]);
        const __half2 ub = __hmax2(tb, m2);
        m2 = __hmin2(m2, tb);
        m3 = __hmin2(m3, ub);
      }
      float v[6] = {__low2float(M1), __low2float(M2), __low2float(M3), __high2float(M1), __high2float(M2), __high2float(M3)};
      top3_of6(v, top);
      float w[6] = {-__low2float(m1), -__low2float(m2), -__low2float(m3), -__high2float(m1), -__high2float(m2), -__high2float(m3)};
      top3_of6(w, bot);
      bot[0] = -bot[0]; bot[1] = -bot[1]; bot[2] = -bot[2];
    }
    // entries above / equal to the second largest instance, below / equal to the second smallest
    int it[2], ib[2];
    {
      const __half2 vT = __float2half2_rn(top[1]), vB = __float2half2_rn(bot[1]);
      unsigned int gt[4] = {0u, 0u, 0u, 0u}, et[4] = {0u, 0u, 0u, 0u}, lt[4] = {0u, 0u, 0u, 0u}, eb[4] = {0u, 0u, 0u, 0u};
#pragma unroll
      for (int q = 0; q < L / 2; ++q) {
        const unsigned int bit = 0x00010001u << (q & 15);
        gt[q >> 4] |= __hgt2_mask(xp[q], vT) & bit;
        et[q >> 4] |= __heq2_mask(xp[q], vT) & bit;
        lt[q >> 4] |= __hlt2_mask(xp[q], vB) & bit;
        eb[q >> 4] |= __heq2_mask(xp[q], vB) & bit;
      }
      unsigned long long ge, go, ee, eo;
      masks_of(gt, ge, go); masks_of(et, ee, eo);
      it[0] = take_first(ge, go);                      // the one entry above the second largest instance, if any
      if (it[0] >= L) it[0] = take_first(ee, eo);
      it[1] = take_first(ee, eo);
      masks_of(lt, ge, go); masks_of(eb, ee, eo);
      ib[0] = take_first(ge, go);
      if (ib[0] >= L) ib[0] = take_first(ee, eo);
      ib[1] = take_first(ee, eo);
    }
    const bool shared_entry = it[0] == ib[0] || it[0] == ib[1] || it[1] == ib[0] || it[1] == ib[1];
    const float levels = (float)((1 << BITS) - 1);
    float d, mn, dm, rmax;
    __half d16;
    unsigned char* orec_v = rec + (SIDE == 0 ? sd.off_koval : sd.off_voval) + tid * 8;
    unsigned char* orec_i = rec + (SIDE == 0 ? sd.off_koidx : sd.off_voidx) + tid * 4;
    if (!shared_entry) {
      mn = bot[2];
      const float mx = top[2];
      // Eq. 2 on the kept entries: binary32, one rounding per operation
      const float range = __fsub_rn(mx, mn);
      const float d32 = __fdiv_rn(range, levels);
      d16 = __float2half_rn(d32);
      d = __half2float(d16);
      const float inv = d != 0.f ? __fdiv_rn(1.0f, d) : 0.f;
      constexpr float kRound = 12582912.0f;
      auto quantize = [&](float x, unsigned int& code) {
        const float t = __fmul_rn(__fsub_rn(x, mn), inv);
        const float y = __fadd_rn(fminf(fmaxf(t, 0.f), levels), kRound);
        code = __float_as_uint(y) & 0xFFu;
        return x - fmaf(__fsub_rn(y, kRound), d, mn);
      };
      if (SIDE == 0) {
#pragma unroll
        for (int q = 0; q < L / 2; ++q) {
          const float2 f = __half22float2(xp[q]);
          unsigned int c0, c1;
          const float r0 = quantize(f.x, c0), r1 = quantize(f.y, c1);
          code_at(2 * q) = (unsigned char)c0;
          code_at(2 * q + 1) = (unsigned char)c1;
          if (R != nullptr) {
            R[(2 * q) * kHeadDim + tid] = r0;
            R[(2 * q + 1) * kHeadDim + tid] = r1;
          }
        }
      } else {
#pragma unroll
        for (int q = 0; q < L / 4; ++q) {
          const float2 f0 = __half22float2(xp[2 * q]), f1 = __half22float2(xp[2 * q + 1]);
          unsigned int k0, k1, k2, k3;
          const float4 rr = make_float4(quantize(f0.x, k0), quantize(f0.y, k1), quantize(f1.x, k2), quantize(f1.y, k3));
          code_at(4 * q) = (unsigned char)k0;
          code_at(4 * q + 1) = (unsigned char)k1;
          code_at(4 * q + 2) = (unsigned char)k2;
          code_at(4 * q + 3) = (unsigned char)k3;
          if (R != nullptr) *reinterpret_cast<float4*>(R + first + 4 * q) = rr;
        }
      }
      // the four filtered entries: cleared, and stored in-group index ascending
      int oi[4] = {it[0], it[1], ib[0], ib[1]};
#pragma unroll
      for (int a = 0; a < 4; ++a) {
        code_at(oi[a]) = 0;
        if (R != nullptr) R[SIDE == 0 ? oi[a] * kHeadDim + tid : first + oi[a]] = 0.f;
      }
      auto order = [&](int a, int b) { if (oi[a] > oi[b]) { const int t = oi[a]; oi[a] = oi[b]; oi[b] = t; } };
      order(0, 1); order(2, 3); order(0, 2); order(1, 3); order(1, 2);
      unsigned short ov[4];
      dm = 0.f;
#pragma unroll
      for (int a = 0; a < 4; ++a) {
        const __half h = X[first + oi[a] * step];
        ov[a] = __half_as_ushort(h);
        dm = fmaxf(dm, fabsf(__half2float(h) - mn));
      }
      *reinterpret_cast<uint2*>(orec_v) = make_uint2(ov[0] | ((unsigned int)ov[1] << 16), ov[2] | ((unsigned int)ov[3] << 16));
      *reinterpret_cast<unsigned int*>(orec_i) = (unsigned int)oi[0] | ((unsigned int)oi[1] << 8) |
                                                 ((unsigned int)oi[2] << 16) | ((unsigned int)oi[3] << 24);
      rmax = (d != 0.f ? 0.50390625f * d : range) + 2.4e-7f * (fabsf(mn) + fabsf(mx));
    } else {
      rmax = 0.f;
      GroupResult g = process_group<BITS, 2>(
          L, 2, [&](int e) { return __half2float(X[first + e * step]); },
          [&](int e, int code, float r) {
            code_at(e) = (unsigned char)code;
            if (R != nullptr) R[SIDE == 0 ? e * kHeadDim + tid : first + e] = r;
            rmax = fmaxf(rmax, fabsf(r));
          },
          [&](int slot, int idx, float v) {
            reinterpret_cast<__half*>(orec_v)[slot] = __float2half_rn(v);
            orec_i[slot] = (unsigned char)idx;
          });
      d16 = g.scale;
      d = __half2float(d16);
      mn = __half2float(g.zero);
      dm = g.dmax;
    }
    reinterpret_cast<__half2*>(rec + (SIDE == 0 ? sd.off_kscale : sd.off_vscale))[tid] = __halves2half2(d16, __float2half_rn(mn));
    atomicMax(&dmax_bits, __float_as_uint(dm));       // non-negative floats order like their bit patterns
    atomicMax(&smax_bits, __float_as_uint(d));
    atomicMax(&rmax_bits, __float_as_uint(rmax));
  }
  __syncthreads();
  if (tid == 0) {
    reinterpret_cast<float*>(rec)[SIDE] = __uint_as_float(dmax_bits);
    reinterpret_cast<float*>(rec)[2 + SIDE] = __uint_as_float(smax_bits);
    if (R != nullptr) atomicMax(p.Rmax + bhl * 2 + SIDE, rmax_bits);
  }
  // pack the codes into mma-fragment order (code_coord_k / code_coord_v), one 32-bit load per field
  unsigned int* dst = reinterpret_cast<unsigned int*>(rec + (SIDE == 0 ? sd.off_kcodes : sd.off_vcodes));
  if (SIDE == 0) {
    constexpr int kWords = kSlab * kHeadDim * BITS / 32;            // words per slab
    for (int li = tid; li < (L / kSlab) * kWords; li += 128) {
      const int slab = li / kWords, wl = li % kWords;
      const int w = wl & 3, lane = (wl >> 2) & 31, tau = wl >> 7;
      const int tok = slab * kSlab + (lane >> 2) + 8 * (w & 1);
      const int ch = 32 * F * tau + 16 * (w >> 1) + 4 * (lane & 3);
      unsigned int word = 0;
#pragma unroll
      for (int j = 0; j < F; ++j)
        word |= *reinterpret_cast<const unsigned int*>(&codes[tok * kCodePitch2 + ch + 32 * j]) << (BITS * j);
      dst[li] = word;
    }
  } else {
    constexpr int kWords = 32 * kHeadDim * BITS / 32;               // words per 32-token chunk
    for (int li = tid; li < (T / 32) * kWords; li += 128) {
      const int chunk = li / kWords, wl = li % kWords;
      const int w = wl & 3, lane = (wl >> 2) & 31, tau = wl >> 7;
      const int ch = 16 * F * tau + (lane >> 2) + 8 * (w & 1);
      const int tok = chunk * 32 + 16 * (w >> 1) + 4 * (lane & 3);
      unsigned int word = 0;
#pragma unroll
      for (int j = 0; j < F; ++j)
        word |= *reinterpret_cast<const unsigned int*>(&codes[(ch + 16 * j) * kCodePitch2 + tok]) << (BITS * j);
      dst[li] = word;
    }
  }
}

// ---------------------------------------------------------------------------
// Power iteration (Algorithm 2).  A "tile" is one (batch, head, K|V) residual
// R_h [n_c, 128] in the workspace.  Factor buffers are [128][16] fp32, zero
// beyond the rank.
// ---------------------------------------------------------------------------
// ---- helpers of the tensor-core pass
__device__ __forceinline__ void mma16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// transpose of an 8 x 8 tile of 16-bit elements held one row pair per lane (the ldmatrix distribution)
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
  uint32_t d;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
  return d;
}
// floor(log2 |x|) for a finite x > 0 (0 for x == 0): the power of two that brings x into [1, 2)
__device__ __forceinline__ int pow2_exponent(float x) { return x > 0.f ? ilogbf(x) : 0; }
__device__ __forceinline__ float exp2_int(int e) { return scalbnf(1.0f, e); }
// (x0, x1) -> packed fp16 heads and packed fp16 remainders (x - head, exact in fp32 before its own rounding)
__device__ __forceinline__ void split_pair(float x0, float x1, uint32_t& hi, uint32_t& lo) {
  const __half2 h = __floats2half2_rn(x0, x1);
  const float2 hf = __half22float2(h);
  const __half2 l = __floats2half2_rn(x0 - hf.x, x1 - hf.y);
  hi = *reinterpret_cast<const uint32_t*>(&h);
  lo = *reinterpret_cast<const uint32_t*>(&l);
}
// x -> (head, remainder) packed in one register, head in the low half
__device__ __forceinline__ void split_pair_hl(float x, uint32_t& hl) {
  const __half h = __float2half_rn(x);
  const __half l = __float2half_rn(x - __half2float(h));
  const __half2 v = __halves2half2(h, l);
  hl = *reinterpret_cast<const uint32_t*>(&v);
}

constexpr int kChunkRows = 512;
constexpr int kPassWarps = 4;

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Counter-based Gaussian for library-drawn start vectors (splitmix64 + Box-Muller).
__device__ __forceinline__ unsigned long long mix64(unsigned long long z) {
  z += 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

__global__ void pi_init_kernel(PiArgs p, const float* B0, int bh0, int BH_total_rank_stride,
                               unsigned long long seed, int segment) {
  // one thread per (tile, channel, rho); B0 layout [bh][2][128][rank]
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  const int total = p.ntiles * kHeadDim * kMaxRank;
  if (idx >= total) return;
  const int rho = idx % kMaxRank, ch = (idx / kMaxRank) % kHeadDim, tile = idx / (kMaxRank * kHeadDim);
  float v = 0.f;
  if (rho < p.rank) {
    const size_t gtile = (size_t)bh0 * 2 + tile;
    if (B0 != nullptr) {
      v = B0[(gtile * kHeadDim + ch) * p.rank + rho];
    } else {
      const unsigned long long h = mix64(seed ^ mix64(((unsigned long long)segment << 40) ^ (gtile * 4096ull + ch * 16 + rho)));
      const float u1 = ((float)(unsigned int)(h >> 40) + 1.0f) * (1.0f / 16777217.0f);
      const float u2 = (float)(unsigned int)((h >> 8) & 0xFFFFFFu) * (1.0f / 16777216.0f);
      v = sqrtf(-2.0f * logf(u1)) * cospif(2.0f * u2);
    }
  }
  p.Bcur[idx] = v;
  (void)BH_total_rank_stride;
}

// One pass over the residual: a = R b for every row, and this chunk's partial of R^T a.
// mode 0: loops before the last.
// mode 1: last loop: the rows a are also stored (A0).  Its Gram matrix and the orthonormalising factor W come from
//         the small kernels below, and since R^T (A0 W) = (R^T A0) W, with W only 16 x 16, R is not read again.
//
// Both products run on the tensor cores (mma.sync.m16n8k16, fp16 operands, fp32 accumulation) with every fp32
// operand cut into an fp16 head and an fp16 remainder, the four cross products summed in fp32: 22 bits of each
// operand survive.  Powers of two bring the operands into fp16's range first (R by the tile's largest magnitude, each
// column of b by its own, a by the bound that follows) and are divided out of the results, so the scaling itself is
// exact.  A warp owns 16 rows at a time.  A lane loads, for rows gid and gid + 8, the four channels 16c + 4t .. + 3 of
// each 16-channel step c as one 128-bit load; since a contraction does not care about the order of its index, these
// four channels serve as the step's k indices 2t, 2t+1, 2t+8, 2t+9 of the A fragment.  For R^T a the same registers,
// transposed 8 x 8 by movmatrix, are the A fragment of R^T (rows: channels 4j, 4j+1 | 4j+2, 4j+3 of the step).
// NT = 8-column tiles of n per CTA: one (four rank columns; three CTAs per SM) or two (eight columns, the residual is
// converted once for both; two CTAs per SM).
template <int MODE, int NT>
__global__ void __launch_bounds__(kPassWarps * 32, NT == 1 ? 3 : 2) pi_pass_kernel(PiArgs p) {
  constexpr int RP = 4 * NT;                       // rank columns per CTA: each gives a (head, remainder) column pair of n
  __shared__ float red[kHeadDim * RP];             // cross-warp sum, accumulated warp by warp
  __shared__ __align__(16) __half bsplit[2 * RP][kHeadDim];   // [2 rho + (0: head, 1: remainder)][channel]
  __shared__ float colmax[kPassWarps][RP];
  __shared__ float gred[MODE == 1 ? kPassWarps : 1][RP][RP];   // Gram partials of the rows a (last loop, all columns here)
  // grid (rank column groups, chunks, tiles): the CTAs that read the same chunk of R are neighbours in launch order,
  // so all but the first find it in L2
  const int tile = blockIdx.z, chunk = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, gid = lane >> 2, t = lane & 3;
  const int row0 = chunk * kChunkRows;
  const int row1 = min(p.n_c, row0 + kChunkRows);
  const int rho0 = blockIdx.x * RP;                // this CTA's rank columns [rho0, rho0 + RP)
  const float* R = p.R + (size_t)tile * p.n_c * kHeadDim;
  float* A0 = p.A0 + (size_t)tile * p.n_c * kMaxRank + rho0;

  // ---- the scaled, split factor columns
  const int er = pow2_exponent(__uint_as_float(p.Rmax[tile]));
  const float sr = exp2_int(-er);
  int eb[RP];
  {
    const int j = threadIdx.x;                     // one channel per thread (kPassWarps * 32 == kHeadDim)
    float bj[RP];
#pragma unroll
    for (int r = 0; r < RP; ++r) {
      bj[r] = p.Bcur[((size_t)tile * kHeadDim + j) * kMaxRank + rho0 + r];
      float m = fabsf(bj[r]);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
      if (lane == 0) colmax[warp][r] = m;
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < RP; ++r) {
      float m = 0.f;
#pragma unroll
      for (int w = 0; w < kPassWarps; ++w) m = fmaxf(m, colmax[w][r]);
      eb[r] = pow2_exponent(m);
      const float v = bj[r] * exp2_int(-eb[r]);
      const __half h = __float2half_rn(v);
      bsplit[2 * r][j] = h;
      bsplit[2 * r + 1][j] = __float2half_rn(v - __half2float(h));
    }
    for (int i = threadIdx.x; i < kHeadDim * RP; i += blockDim.x) red[i] = 0.f;
    __syncthreads();
  }
  // B fragments of a = R b: column n = gid of tile nt is (rho = 4 nt + gid / 2, head | remainder), k as described above
  uint32_t bf[8][NT][2];
#pragma unroll
  for (int c = 0; c < 8; ++c)
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      const uint2 v = *reinterpret_cast<const uint2*>(&bsplit[8 * nt + gid][16 * c + 4 * t]);
      bf[c][nt][0] = v.x; bf[c][nt][1] = v.y;
    }
  // |R sr| < 2 and |b 2^-eb| < 2, so |a| < 512 in these units: a 2^-10 stays below one half
  constexpr float kScaleA = 1.0f / 1024.0f;
  float inv_a[NT], inv_acc[NT];                    // back to a = R b and to R^T a for column rho = 4 nt + t
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
    int ebt = eb[4 * nt];
#pragma unroll
    for (int q = 1; q < 4; ++q) ebt = t == q ? eb[4 * nt + q] : ebt;
    inv_a[nt] = exp2_int(er + ebt);
    inv_acc[nt] = exp2_int(2 * er + ebt + 10);
  }

  // Last loop, and this CTA holds every rank column: the Gram matrix of the rows a (first round of CholeskyQR) is
  // summed here, so that A0 is not read again for it.  gram[nt][v]: row rho = 4 nt + t of the matrix, column v.
  const bool with_gram = MODE == 1 && gridDim.x == 1;
  float gram[NT][RP];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt)
#pragma unroll
    for (int v = 0; v < RP; ++v) gram[nt][v] = 0.f;

  float acc[8][NT][4];    // R^T a: [step c][tile][(channel 4 gid/2 + gid%2 of the step | the same + 2) x (head, remainder)]
#pragma unroll
  for (int c = 0; c < 8; ++c)
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int i = 0; i < 4; ++i) acc[c][nt][i] = 0.f;

  for (int rb = row0 + warp * 16; rb < row1; rb += kPassWarps * 16) {
    const int ra = rb + gid, rc = rb + gid + 8;
    const bool va = ra < row1, vc = rc < row1;
    float4 xa[8], xc[8];
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      xa[c] = va ? *reinterpret_cast<const float4*>(R + (size_t)ra * kHeadDim + 16 * c + 4 * t) : make_float4(0.f, 0.f, 0.f, 0.f);
      xc[c] = vc ? *reinterpret_cast<const float4*>(R + (size_t)rc * kHeadDim + 16 * c + 4 * t) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    uint32_t fh[8][4], fl[8][4];
    float d[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) d[nt][0] = d[nt][1] = d[nt][2] = d[nt][3] = 0.f;
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      split_pair(xa[c].x * sr, xa[c].y * sr, fh[c][0], fl[c][0]);
      split_pair(xc[c].x * sr, xc[c].y * sr, fh[c][1], fl[c][1]);
      split_pair(xa[c].z * sr, xa[c].w * sr, fh[c][2], fl[c][2]);
      split_pair(xc[c].z * sr, xc[c].w * sr, fh[c][3], fl[c][3]);
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        mma16816(d[nt], fh[c], bf[c][nt][0], bf[c][nt][1]);
        mma16816(d[nt], fl[c], bf[c][nt][0], bf[c][nt][1]);
      }
    }
    // B fragment of R^T a: k = row, n = (rho, head | remainder): the 8 x 8 tiles [row][2 rho + part], transposed
    uint32_t ab[NT][2];
    if (MODE == 1 && with_gram) {
      float mine[2][NT];                            // a[row gid | gid + 8][rho 4 nt + t]; rows past the chunk are zero
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        mine[0][nt] = (d[nt][0] + d[nt][1]) * inv_a[nt];
        mine[1][nt] = (d[nt][2] + d[nt][3]) * inv_a[nt];
      }
#pragma unroll
      for (int half = 0; half < 2; ++half)
#pragma unroll
        for (int nv = 0; nv < NT; ++nv)
#pragma unroll
          for (int tv = 0; tv < 4; ++tv) {
            const float other = __shfl_sync(0xffffffffu, mine[half][nv], (lane & ~3) | tv);   // a[row][4 nv + tv]
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) gram[nt][4 * nv + tv] = fmaf(mine[half][nt], other, gram[nt][4 * nv + tv]);
          }
    }
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      const float a_lo_rows = d[nt][0] + d[nt][1], a_hi_rows = d[nt][2] + d[nt][3];   // a[row gid | gid + 8][rho 4 nt + t], scaled
      if (MODE == 1) {
        if (va) A0[(size_t)ra * kMaxRank + 4 * nt + t] = a_lo_rows * inv_a[nt];
        if (vc) A0[(size_t)rc * kMaxRank + 4 * nt + t] = a_hi_rows * inv_a[nt];
      }
      uint32_t m0, m1;
      split_pair_hl(a_lo_rows * kScaleA, m0);
      split_pair_hl(a_hi_rows * kScaleA, m1);
      ab[nt][0] = movmatrix_trans(m0);
      ab[nt][1] = movmatrix_trans(m1);
    }
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      uint32_t th[4], tl[4];
      th[0] = movmatrix_trans(fh[c][0]); th[1] = movmatrix_trans(fh[c][2]);
      th[2] = movmatrix_trans(fh[c][1]); th[3] = movmatrix_trans(fh[c][3]);
      tl[0] = movmatrix_trans(fl[c][0]); tl[1] = movmatrix_trans(fl[c][2]);
      tl[2] = movmatrix_trans(fl[c][1]); tl[3] = movmatrix_trans(fl[c][3]);
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        mma16816(acc[c][nt], th, ab[nt][0], ab[nt][1]);
        mma16816(acc[c][nt], tl, ab[nt][0], ab[nt][1]);
      }
    }
  }
  if (MODE == 1 && with_gram) {      // rows of the warp (over gid), then the warps, in a fixed order
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
      for (int v = 0; v < RP; ++v) {
        float g = gram[nt][v];
#pragma unroll
        for (int o = 4; o < 32; o <<= 1) g += __shfl_xor_sync(0xffffffffu, g, o);
        if (gid == 0) gred[MODE == 1 ? warp : 0][4 * nt + t][v] = g;
      }
    __syncthreads();
    for (int i = threadIdx.x; i < 256; i += blockDim.x) {
      const int u = i / kMaxRank, v = i % kMaxRank;
      float g = 0.f;
      if (u < RP && v < RP)
        for (int w = 0; w < kPassWarps; ++w) g += gred[MODE == 1 ? w : 0][u][v];
      p.Gp[((size_t)tile * p.nchunk + chunk) * 256 + i] = g;
    }
  }
  // combine the warps of this block in a fixed order, write the chunk's partial
  for (int w = 0; w < kPassWarps; ++w) {
    if (warp == w) {
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        const int ch = 16 * c + 4 * (gid >> 1) + (gid & 1);
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          red[ch * RP + 4 * nt + t] += (acc[c][nt][0] + acc[c][nt][1]) * inv_acc[nt];
          red[(ch + 2) * RP + 4 * nt + t] += (acc[c][nt][2] + acc[c][nt][3]) * inv_acc[nt];
        }
      }
    }
    __syncthreads();
  }
  for (int i = threadIdx.x; i < kHeadDim * RP; i += blockDim.x)
    p.Bp[(((size_t)tile * p.nchunk + chunk) * kHeadDim + i / RP) * kMaxRank + rho0 + i % RP] = red[i];
}

// The stored A = A0 W (W = R1^-1 R2^-1 of the two CholeskyQR rounds): one thread per row.  Keys: a row is r_pad
// consecutive fp16 of its slab; values: the slab is transposed ([r_pad][16 tokens]), so the threads of a slab fill
// 32 contiguous bytes per rank index.  fp32 copy on request.
__global__ void __launch_bounds__(256) pi_store_a_kernel(PiArgs p) {
  __shared__ float Wm[kMaxRank * kMaxRank];
  const int tile = blockIdx.y;
  for (int i = threadIdx.x; i < kMaxRank * kMaxRank; i += blockDim.x) Wm[i] = p.W[(size_t)tile * 256 + i];
  __syncthreads();
  const int row = blockIdx.x * blockDim.x + threadIdx.x;
  if (row >= p.n_c) return;
  const SegDesc& sd = p.seg;
  const int r = sd.rank;
  const float* a0p = p.A0 + ((size_t)tile * p.n_c + row) * kMaxRank;
  float a0[kMaxRank], a[kMaxRank];
#pragma unroll
  for (int q = 0; q < kMaxRank; ++q) a0[q] = q < r ? a0p[q] : 0.f;
#pragma unroll
  for (int c = 0; c < kMaxRank; ++c) {
    float v = 0.f;
#pragma unroll
    for (int q = 0; q < kMaxRank; ++q)
      if (q < r && c < r) v = fmaf(a0[q], Wm[q * kMaxRank + c], v);
    a[c] = v;
  }
  const int bhl = tile >> 1, side = tile & 1;
  const int blk = row / sd.T, tib = row % sd.T, slab = tib / kSlab, ts = tib % kSlab;
  unsigned char* rec = p.arena + sd.seg_base + (size_t)(p.bh0 + bhl) * sd.bh_stride + sd.bfac_bytes +
                       (size_t)blk * sd.rec_bytes;
  if (side == 0) {
    __half2* dst = reinterpret_cast<__half2*>(rec + sd.off_ak + slab * sd.slab_a) + ts * (sd.r_pad / 2);
#pragma unroll
    for (int c = 0; c < kMaxRank; c += 2)
      if (c < sd.r_pad) dst[c / 2] = __floats2half2_rn(a[c], a[c + 1]);
  } else {
    __half* dst = reinterpret_cast<__half*>(rec + sd.off_av + slab * sd.slab_a) + ts;
#pragma unroll
    for (int c = 0; c < kMaxRank; ++c)
      if (c < sd.r_pad) dst[c * kSlab] = __float2half_rn(a[c]);
  }
  if (p.dbgA != nullptr) {
    float* dd = p.dbgA + (((size_t)(p.bh0 + bhl) * 2 + side) * sd.n_c + row) * r;
#pragma unroll
    for (int c = 0; c < kMaxRank; ++c)
      if (c < r) dd[c] = a[c];
  }
}

// Sum the chunk partials of R^T a into the factor buffer (fixed order).  With
// `orth`, orthonormalise its columns (modified Gram-Schmidt, two sweeps per
// column) -- the QR of B at the top of Algorithm 2's last loop.  With `store`,
// write the final B as fp16 ([r_pad][128] for keys, [128][r_pad] for values).
__global__ void __launch_bounds__(kHeadDim) pi_reduce_b_kernel(PiArgs p, int orth, int store, int apply_w) {
  __shared__ float wsum[4];
  const int tile = blockIdx.x, j = threadIdx.x, lane = j & 31, warp = j >> 5;
  float b[kMaxRank];
#pragma unroll
  for (int r = 0; r < kMaxRank; ++r) {
    float s = 0.f;
    if (r < p.rank)
      for (int c = 0; c < p.nchunk; ++c) s += p.Bp[(((size_t)tile * p.nchunk + c) * kHeadDim + j) * kMaxRank + r];
    b[r] = s;
  }
  if (apply_w) {                 // the sums are R^T A0: the factor of the orthonormalised A = A0 W is (R^T A0) W
    float bw[kMaxRank];
#pragma unroll
    for (int r = 0; r < kMaxRank; ++r) {
      float v = 0.f;
#pragma unroll
      for (int q = 0; q < kMaxRank; ++q)
        if (q < p.rank && r < p.rank) v = fmaf(b[q], p.W[(size_t)tile * 256 + q * kMaxRank + r], v);
      bw[r] = v;
    }
#pragma unroll
    for (int r = 0; r < kMaxRank; ++r) b[r] = bw[r];
  }
  auto block_sum = [&](float v) {
    v = warp_sum(v);
    __syncthreads();
    if (lane == 0) wsum[warp] = v;
    __syncthreads();
    return (wsum[0] + wsum[1]) + (wsum[2] + wsum[3]);
  };
  if (orth) {
#pragma unroll
    for (int c = 0; c < kMaxRank; ++c) {
      if (c < p.rank) {                      // uniform over the block
#pragma unroll
        for (int sweep = 0; sweep < 2; ++sweep) {
#pragma unroll
          for (int q = 0; q < kMaxRank; ++q) {
            if (q < c) {
              const float d = block_sum(b[q] * b[c]);
              b[c] = fmaf(-d, b[q], b[c]);
            }
          }
        }
        const float nrm2 = block_sum(b[c] * b[c]);
        b[c] = nrm2 > 0.f ? b[c] * rsqrtf(nrm2) : 0.f;
        // one Newton step on the normalisation keeps the column norm at 1 to rounding
        const float n2 = block_sum(b[c] * b[c]);
        if (n2 > 0.f) b[c] *= (1.5f - 0.5f * n2);
      }
    }
  }
#pragma unroll
  for (int r = 0; r < kMaxRank; ++r) p.Bcur[((size_t)tile * kHeadDim + j) * kMaxRank + r] = b[r];
  if (store) {
    const SegDesc& sd = p.seg;
    const int bhl = tile >> 1, side = tile & 1;
    __half* bf = reinterpret_cast<__half*>(p.arena + sd.seg_base + (size_t)(p.bh0 + bhl) * sd.bh_stride);
#pragma unroll
    for (int r = 0; r < kMaxRank; ++r) {
      if (r < sd.r_pad) {
        const __half v = __float2half_rn(r < sd.rank ? b[r] : 0.f);
        if (side == 0) bf[r * kHeadDim + j] = v;
        else bf[sd.r_pad * kHeadDim + j * sd.r_pad + r] = v;
        if (p.dbgB != nullptr && r < sd.rank)
          p.dbgB[(((size_t)(p.bh0 + bhl) * 2 + side) * kHeadDim + j) * sd.rank + r] = b[r];
      }
    }
  }
}

// Gram matrix of the current A (sum of chunk partials), its Cholesky factor
// U (G = U^T U) and U^-1.  first = 1: W <- U^-1.  first = 0: W <- W U^-1.
// A column whose pivot vanishes (rank-deficient residual) is zeroed.
__global__ void __launch_bounds__(32) pi_chol_kernel(PiArgs p, int first) {
  __shared__ float G[kMaxRank][kMaxRank + 1], U[kMaxRank][kMaxRank + 1], Ui[kMaxRank][kMaxRank + 1],
      Wo[kMaxRank][kMaxRank + 1];
  const int tile = blockIdx.x, lane = threadIdx.x, r = p.rank;
  for (int i = lane; i < 256; i += 32) {
    float s = 0.f;
    for (int c = 0; c < p.nchunk; ++c) s += p.Gp[((size_t)tile * p.nchunk + c) * 256 + i];
    G[i / kMaxRank][i % kMaxRank] = s;
    U[i / kMaxRank][i % kMaxRank] = 0.f;
    Ui[i / kMaxRank][i % kMaxRank] = 0.f;
    Wo[i / kMaxRank][i % kMaxRank] = first ? 0.f : p.W[(size_t)tile * 256 + i];
  }
  __syncwarp();
  if (lane == 0) {
    float tr = 0.f;
    for (int i = 0; i < r; ++i) tr += G[i][i];
    const float tiny = tr * 1e-12f;
    for (int j = 0; j < r; ++j) {          // upper-triangular U, row by row
      float d = G[j][j];
      for (int k = 0; k < j; ++k) d -= U[k][j] * U[k][j];
      const bool ok = d > tiny && d > 0.f;
      const float ujj = ok ? sqrtf(d) : 0.f;
      U[j][j] = ujj;
      for (int i = j + 1; i < r; ++i) {
        float s = G[j][i];
        for (int k = 0; k < j; ++k) s -= U[k][j] * U[k][i];
        U[j][i] = ok ? s / ujj : 0.f;
      }
    }
    for (int c = 0; c < r; ++c) {          // U^-1 by back substitution, column by column
      for (int i = c; i >= 0; --i) {
        if (U[i][i] == 0.f) { Ui[i][c] = 0.f; continue; }
        float s = (i == c) ? 1.f : 0.f;
        for (int k = i + 1; k <= c; ++k) s -= U[i][k] * Ui[k][c];
        Ui[i][c] = s / U[i][i];
      }
      if (U[c][c] == 0.f) for (int i = 0; i <= c; ++i) Ui[i][c] = 0.f;
    }
  }
  __syncwarp();
  for (int i = lane; i < 256; i += 32) {
    const int a = i / kMaxRank, b = i % kMaxRank;
    float v = 0.f;
    if (a < r && b < r) {
      if (first) v = Ui[a][b];
      else for (int k = 0; k < r; ++k) v = fmaf(Wo[a][k], Ui[k][b], v);
    }
    p.W[(size_t)tile * 256 + i] = v;
  }
}

// Gram partials of A0 W (W = identity in the first round of CholeskyQR): one thread per row.
__global__ void __launch_bounds__(256) pi_gram2_kernel(PiArgs p, int identity) {
  __shared__ float Wm[kMaxRank * kMaxRank];
  __shared__ float rows[8][32][kMaxRank + 1];
  __shared__ float red[8][256];
  const int tile = blockIdx.y, chunk = blockIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int i = threadIdx.x; i < 256; i += blockDim.x)
    Wm[i] = identity ? (i / kMaxRank == i % kMaxRank ? 1.f : 0.f) : p.W[(size_t)tile * 256 + i];
  __syncthreads();
  const int r = p.rank;
  const int row0 = chunk * kChunkRows, row1 = min(p.n_c, row0 + kChunkRows);
  const float* A0 = p.A0 + (size_t)tile * p.n_c * kMaxRank;
  float g[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) g[i] = 0.f;
  for (int base = row0 + warp * 32; base < row1; base += 8 * 32) {
    const int row = base + lane;
    float a0[kMaxRank];
#pragma unroll
    for (int q = 0; q < kMaxRank; ++q) a0[q] = (row < row1 && q < r) ? A0[(size_t)row * kMaxRank + q] : 0.f;
#pragma unroll
    for (int c = 0; c < kMaxRank; ++c) {
      if (c < r) {                               // uniform over the block: only the rank's columns exist
        float s = 0.f;
#pragma unroll
        for (int q = 0; q < kMaxRank; ++q) s = fmaf(a0[q], Wm[q * kMaxRank + c], s);
        rows[warp][lane][c] = s;
      }
    }
    __syncwarp();
    // entry (u, v) of the Gram matrix, u, v < r: pair number i * 32 + lane, so that a small rank takes one round
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      if (i * 32 < r * r) {
        const int pr = i * 32 + lane, u = min(pr / r, kMaxRank - 1), v = pr % r;
        float s = g[i];
        for (int t = 0; t < 32; ++t) s = fmaf(rows[warp][t][u], rows[warp][t][v], s);
        g[i] = s;
      }
    }
    __syncwarp();
  }
  for (int i = threadIdx.x; i < 8 * 256; i += blockDim.x) (&red[0][0])[i] = 0.f;
  __syncthreads();
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int pr = i * 32 + lane;
    if (pr < r * r) red[warp][(pr / r) * kMaxRank + pr % r] = g[i];
  }
  __syncthreads();
  for (int i = threadIdx.x; i < 256; i += blockDim.x) {
    float s = 0.f;
    for (int w = 0; w < 8; ++w) s += red[w][i];
    p.Gp[((size_t)tile * p.nchunk + chunk) * 256 + i] = s;
  }
}

// ---------------------------------------------------------------------------
// Whole-tile compression for short segments (a flushed buffer, Algorithm 1's
// decoding phase): one CTA takes one (batch, head, K|V) tile of n_c <= 128
// tokens through Filter, Quant, residual and all of Algorithm 2 with the
// residual held in shared memory, so that a flush is one launch instead of a
// chain of a dozen latency-bound ones.
// ---------------------------------------------------------------------------
constexpr int kTileMaxTokens = 128;
constexpr int kFPitch = kMaxRank + 1;      // floats per row of the factor matrices in shared memory

struct TileArgs {
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

__device__ __forceinline__ float block_sum128(float v, float* wsum, int lane, int warp) {
  v = warp_sum(v);
  __syncthreads();
  if (lane == 0) wsum[warp] = v;
  __syncthreads();
  return (wsum[0] + wsum[1]) + (wsum[2] + wsum[3]);
}

// G = U^T U (upper Cholesky factor) and U^-1 for the r x r Gram matrix G; first: W <- U^-1, else W <- W U^-1.
// A column whose pivot vanishes is zeroed.  Run by one warp; matrices have pitch kFPitch.
__device__ void chol_update(const float* G, float* U, float* Ui, float* W, int r, int first, int lane) {
  for (int i = lane; i < kMaxRank * kFPitch; i += 32) { U[i] = 0.f; Ui[i] = 0.f; }
  __syncwarp();
  if (lane == 0) {
    float tr = 0.f;
    for (int i = 0; i < r; ++i) tr += G[i * kFPitch + i];
    const float tiny = tr * 1e-12f;
    for (int j = 0; j < r; ++j) {
      float d = G[j * kFPitch + j];
      for (int k = 0; k < j; ++k) d -= U[k * kFPitch + j] * U[k * kFPitch + j];
      const bool ok = d > tiny && d > 0.f;
      const float ujj = ok ? sqrtf(d) : 0.f;
      U[j * kFPitch + j] = ujj;
      for (int i = j + 1; i < r; ++i) {
        float sacc = G[j * kFPitch + i];
        for (int k = 0; k < j; ++k) sacc -= U[k * kFPitch + j] * U[k * kFPitch + i];
        U[j * kFPitch + i] = ok ? sacc / ujj : 0.f;
      }
    }
    for (int c = 0; c < r; ++c) {
      for (int i = c; i >= 0; --i) {
        if (U[i * kFPitch + i] == 0.f) { Ui[i * kFPitch + c] = 0.f; continue; }
        float sacc = (i == c) ? 1.f : 0.f;
        for (int k = i + 1; k <= c; ++k) sacc -= U[i * kFPitch + k] * Ui[k * kFPitch + c];
        Ui[i * kFPitch + c] = sacc / U[i * kFPitch + i];
      }
      if (U[c * kFPitch + c] == 0.f) for (int i = 0; i <= c; ++i) Ui[i * kFPitch + c] = 0.f;
    }
  }
  __syncwarp();
  // W (r x r): each lane owns entries lane, lane + 32, ...; the product needs the old W, so read it all first
  float wn[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    const int i = lane + 32 * e, a = i / kMaxRank, b = i % kMaxRank;
    float v = 0.f;
    if (a < r && b < r) {
      if (first) v = Ui[a * kFPitch + b];
      else for (int k = 0; k < r; ++k) v = fmaf(W[a * kFPitch + k], Ui[k * kFPitch + b], v);
    }
    wn[e] = v;
  }
  __syncwarp();
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    const int i = lane + 32 * e;
    W[(i / kMaxRank) * kFPitch + i % kMaxRank] = wn[e];
  }
  __syncwarp();
}

// Shared memory: [ region 0 | residual rs[n_c][kRPitch] ].  Region 0 first holds the fp16 tile of the block being
// quantized (each entry is replaced by its code once it is known), later the factor matrices of Algorithm 2.
template <int RP>
__host__ __device__ constexpr int tile_factor_bytes(int n_c) {
  return ((kHeadDim + n_c) * (RP + 1) + 4 * kMaxRank * kFPitch + 8) * 4;
}

template <int BITS, int KMAX, int RP>
__global__ void __launch_bounds__(128) compress_tile_kernel(TileArgs p) {
  constexpr int FP = RP + 1;                 // floats per row of B and A in shared memory
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const SegDesc& sd = p.seg;
  const int T = sd.T, n_c = sd.n_c, r = sd.rank;
  const int side = blockIdx.y, bh = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int reg0 = max(round_up(T * kXPitch * 2, 16), tile_factor_bytes<RP>(n_c));
  unsigned short* xs = reinterpret_cast<unsigned short*>(smem_raw);      // [T][kXPitch] fp16 bits, then codes
  float* rs = reinterpret_cast<float*>(smem_raw + reg0);                 // [n_c][kRPitch] residual of the whole tile
  float* Bm = reinterpret_cast<float*>(smem_raw);                        // [128][FP]
  float* Am = Bm + kHeadDim * FP;                                        // [n_c][FP]
  float* Gm = Am + n_c * FP;                                             // [16][kFPitch]
  float* Um = Gm + kMaxRank * kFPitch;
  float* Uim = Um + kMaxRank * kFPitch;
  float* Wm = Uim + kMaxRank * kFPitch;
  float* wsum = Wm + kMaxRank * kFPitch;                                 // [4]
  __shared__ unsigned int dmax_bits, smax_bits;

  const __half* Xt = (side == 0 ? p.K : p.V) + (size_t)bh * n_c * kHeadDim;
  unsigned char* seg_bh = p.arena + sd.seg_base + (size_t)bh * sd.bh_stride;
  auto x_of = [&](int idx) { return __half2float(__ushort_as_half(xs[idx])); };

  // ---- Filter, Quant, pack, residual: block by block (one key group per channel spans one block)
  for (int blk = 0; blk < sd.nblk; ++blk) {
    if (tid == 0) { dmax_bits = 0u; smax_bits = 0u; }
    const __half* X = Xt + (size_t)blk * T * kHeadDim;
    for (int i = tid; i < T * 16; i += 128) {
      const int row = i >> 4, c = i & 15;
      const uint4 v = *reinterpret_cast<const uint4*>(X + row * kHeadDim + c * 8);
      unsigned int* dst = reinterpret_cast<unsigned int*>(xs + row * kXPitch + c * 8);
      dst[0] = v.x; dst[1] = v.y; dst[2] = v.z; dst[3] = v.w;
    }
    __syncthreads();
    unsigned char* rec = seg_bh + sd.bfac_bytes + (size_t)blk * sd.rec_bytes;
    float* rb = rs + (size_t)blk * T * kRPitch;
    float my_dmax = 0.f, my_smax = 0.f;
    if (side == 0) {
      const int j = tid, k = sd.k_k;
      __half* oval = reinterpret_cast<__half*>(rec + sd.off_koval) + j * 2 * k;
      unsigned char* oidx = rec + sd.off_koidx + j * 2 * k;
      GroupResult g = process_group<BITS, KMAX>(
          T, k, [&](int e) { return x_of(e * kXPitch + j); },
          [&](int e, int code, float res) { xs[e * kXPitch + j] = (unsigned short)code; rb[e * kRPitch + j] = res; },
          [&](int slot, int idx, float v) { oval[slot] = __float2half_rn(v); oidx[slot] = (unsigned char)idx; });
      reinterpret_cast<__half2*>(rec + sd.off_kscale)[j] = __halves2half2(g.scale, g.zero);
      my_dmax = g.dmax;
      my_smax = __half2float(g.scale);
    } else {
      const int k = p.cc.k_v, gv = p.cc.g_v, ngv = p.cc.ngv;
      for (int gi = tid; gi < T * ngv; gi += 128) {
        const int tok = gi / ngv, c = gi % ngv;
        __half* oval = reinterpret_cast<__half*>(rec + sd.off_voval) + gi * 2 * k;
        unsigned char* oidx = rec + sd.off_voidx + gi * 2 * k;
        GroupResult g = process_group<BITS, KMAX>(
            gv, k, [&](int e) { return x_of(tok * kXPitch + c * gv + e); },
            [&](int e, int code, float res) {
              xs[tok * kXPitch + c * gv + e] = (unsigned short)code;
              rb[tok * kRPitch + c * gv + e] = res;
            },
            [&](int slot, int idx, float v) { oval[slot] = __float2half_rn(v); oidx[slot] = (unsigned char)idx; });
        reinterpret_cast<__half2*>(rec + sd.off_vscale)[gi] = __halves2half2(g.scale, g.zero);
        my_dmax = fmaxf(my_dmax, g.dmax);
        my_smax = fmaxf(my_smax, __half2float(g.scale));
      }
    }
    atomicMax(&dmax_bits, __float_as_uint(my_dmax));
    atomicMax(&smax_bits, __float_as_uint(my_smax));
    __syncthreads();
    if (tid == 0) {
      reinterpret_cast<float*>(rec)[side] = __uint_as_float(dmax_bits);
      reinterpret_cast<float*>(rec)[2 + side] = __uint_as_float(smax_bits);
    }
    pack_block_codes<BITS>(xs, T, side, reinterpret_cast<unsigned int*>(rec + (side == 0 ? sd.off_kcodes : sd.off_vcodes)),
                           tid, 128);
    __syncthreads();
  }
  if (r == 0) return;

  // ---- Algorithm 2 on the residual in shared memory.  Thread `tid` owns channel tid of B.
  const size_t gtile = (size_t)bh * 2 + side;
  float b[RP];
#pragma unroll
  for (int rho = 0; rho < RP; ++rho) {
    float v = 0.f;
    if (rho < r) {
      if (p.B0 != nullptr) {
        v = p.B0[(gtile * kHeadDim + tid) * r + rho];
      } else {
        const unsigned long long h =
            mix64(p.seed ^ mix64(((unsigned long long)p.segment_index << 40) ^ (gtile * 4096ull + tid * 16 + rho)));
        const float u1 = ((float)(unsigned int)(h >> 40) + 1.0f) * (1.0f / 16777217.0f);
        const float u2 = (float)(unsigned int)((h >> 8) & 0xFFFFFFu) * (1.0f / 16777216.0f);
        v = sqrtf(-2.0f * logf(u1)) * cospif(2.0f * u2);
      }
    }
    b[rho] = v;
  }
  for (int l = 0; l < p.iters; ++l) {
    const bool last = l == p.iters - 1;
    if (last) {
      // B <- Q(B): modified Gram-Schmidt, two sweeps per column, then a Newton step on the norm
#pragma unroll
      for (int c = 0; c < RP; ++c) {
        if (c < r) {
#pragma unroll
          for (int sweep = 0; sweep < 2; ++sweep) {
#pragma unroll
            for (int q = 0; q < RP; ++q) {
              if (q < c) {
                const float d = block_sum128(b[q] * b[c], wsum, lane, warp);
                b[c] = fmaf(-d, b[q], b[c]);
              }
            }
          }
          const float nrm2 = block_sum128(b[c] * b[c], wsum, lane, warp);
          b[c] = nrm2 > 0.f ? b[c] * rsqrtf(nrm2) : 0.f;
          const float n2 = block_sum128(b[c] * b[c], wsum, lane, warp);
          if (n2 > 0.f) b[c] *= (1.5f - 0.5f * n2);
        }
      }
    }
    __syncthreads();
#pragma unroll
    for (int rho = 0; rho < RP; ++rho) Bm[tid * FP + rho] = b[rho];
    __syncthreads();
    // A = R B: one row of A per thread and round (all columns at once)
    for (int i = tid; i < n_c; i += 128) {
      const float* rr = rs + i * kRPitch;
      float acc[RP];
#pragma unroll
      for (int rho = 0; rho < RP; ++rho) acc[rho] = 0.f;
#pragma unroll 4
      for (int c = 0; c < kHeadDim; ++c) {
        const float x = rr[c];
#pragma unroll
        for (int rho = 0; rho < RP; ++rho) acc[rho] = fmaf(x, Bm[c * FP + rho], acc[rho]);
      }
#pragma unroll
      for (int rho = 0; rho < RP; ++rho) Am[i * FP + rho] = acc[rho];
    }
    __syncthreads();
    if (last) {
      // A <- Q(A) by Cholesky QR, twice: Gram matrix, U^-1 of its Cholesky factor, A <- A U^-1
      for (int round = 0; round < 2; ++round) {
        for (int o = tid; o < r * r; o += 128) {
          const int u = o / r, v = o % r;
          float acc = 0.f;
          for (int i = 0; i < n_c; ++i) acc = fmaf(Am[i * FP + u], Am[i * FP + v], acc);
          Gm[u * kFPitch + v] = acc;
        }
        __syncthreads();
        if (warp == 0) chol_update(Gm, Um, Uim, Wm, r, 1, lane);
        __syncthreads();
        for (int i = tid; i < n_c; i += 128) {           // one row per thread
          float a0[RP], an[RP];
#pragma unroll
          for (int k = 0; k < RP; ++k) a0[k] = Am[i * FP + k];
#pragma unroll
          for (int c = 0; c < RP; ++c) {
            float acc = 0.f;
#pragma unroll
            for (int k = 0; k < RP; ++k) acc = fmaf(a0[k], Wm[k * kFPitch + c], acc);
            an[c] = acc;
          }
#pragma unroll
          for (int c = 0; c < RP; ++c) Am[i * FP + c] = an[c];
          if (round == 1) {
            // the final A: fp16 in the records (fragment order), fp32 copy on request
            const int blk = i / T, tib = i % T, slab = tib / kSlab, ts = tib % kSlab;
            unsigned char* rec = seg_bh + sd.bfac_bytes + (size_t)blk * sd.rec_bytes;
#pragma unroll
            for (int c = 0; c < RP; ++c) {
              if (c < sd.r_pad) {
                const float val = c < r ? an[c] : 0.f;
                if (side == 0)
                  reinterpret_cast<__half*>(rec + sd.off_ak + slab * sd.slab_a)[ts * sd.r_pad + c] = __float2half_rn(val);
                else
                  reinterpret_cast<__half*>(rec + sd.off_av + slab * sd.slab_a)[c * kSlab + ts] = __float2half_rn(val);
                if (p.dbgA != nullptr && c < r) p.dbgA[(gtile * n_c + i) * r + c] = val;
              }
            }
          }
        }
        __syncthreads();
      }
    }
    // B = R^T A: channel tid
#pragma unroll
    for (int rho = 0; rho < RP; ++rho) b[rho] = 0.f;
#pragma unroll 4
    for (int i = 0; i < n_c; ++i) {
      const float x = rs[i * kRPitch + tid];
#pragma unroll
      for (int rho = 0; rho < RP; ++rho) b[rho] = fmaf(x, Am[i * FP + rho], b[rho]);
    }
  }
  // ---- store B: fp16 [r_pad][128] for keys, [128][r_pad] for values
  __half* bf = reinterpret_cast<__half*>(seg_bh);
#pragma unroll
  for (int rho = 0; rho < RP; ++rho) {
    if (rho < sd.r_pad) {
      const __half v = __float2half_rn(rho < r ? b[rho] : 0.f);
      if (side == 0) bf[rho * kHeadDim + tid] = v;
      else bf[sd.r_pad * kHeadDim + tid * sd.r_pad + rho] = v;
      if (p.dbgB != nullptr && rho < r) p.dbgB[(gtile * kHeadDim + tid) * r + rho] = b[rho];
    }
  }
}

static int tile_rp(int rank) { return rank <= 4 ? 4 : (rank <= 8 ? 8 : 16); }

static size_t tile_smem_bytes(int T, int n_c, int rank) {
  const int rp = tile_rp(rank);
  const int fb = rp == 4 ? tile_factor_bytes<4>(n_c) : (rp == 8 ? tile_factor_bytes<8>(n_c) : tile_factor_bytes<16>(n_c));
  const int x = round_up(T * kXPitch * 2, 16);
  return (size_t)(x > fb ? x : fb) + (size_t)n_c * kRPitch * 4;
}

bool compress_tile_fits(int T, int n_c, int rank) {
  return n_c <= kTileMaxTokens && tile_smem_bytes(T, n_c, rank) <= 200 * 1024;
}

cudaError_t compress_tile(const CompressJob& job, int BH, cudaStream_t st) {
  TileArgs a;
  a.seg = job.seg; a.cc = job.cc; a.arena = job.arena; a.K = job.K; a.V = job.V; a.B0 = job.B0;
  a.dbgA = job.dbgA; a.dbgB = job.dbgB; a.seed = job.seed; a.segment_index = job.segment_index; a.iters = job.iters;
  const size_t smem = tile_smem_bytes(job.seg.T, job.seg.n_c, job.seg.rank);
  const int kneed = job.seg.k_k > job.cc.k_v ? job.seg.k_k : job.cc.k_v;
  const int rp = tile_rp(job.seg.rank);
  dim3 grid(BH, 2);
  cudaError_t e = cudaSuccess;
#define GEAR_TILE(B, KM, R)                                                                                          \
  {                                                                                                                  \
    e = cudaFuncSetAttribute(compress_tile_kernel<B, KM, R>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem); \
    if (e != cudaSuccess) return e;                                                                                  \
    compress_tile_kernel<B, KM, R><<<grid, 128, smem, st>>>(a);                                                      \
  }
#define GEAR_TILE_R(B, KM) \
  { if (rp == 4) GEAR_TILE(B, KM, 4) else if (rp == 8) GEAR_TILE(B, KM, 8) else GEAR_TILE(B, KM, 16) }
  if (job.cc.bits == 2) {
    if (kneed <= 1) GEAR_TILE_R(2, 1) else if (kneed <= 2) GEAR_TILE_R(2, 2) else GEAR_TILE_R(2, 8)
  } else {
    if (kneed <= 1) GEAR_TILE_R(4, 1) else if (kneed <= 2) GEAR_TILE_R(4, 2) else GEAR_TILE_R(4, 8)
  }
#undef GEAR_TILE_R
#undef GEAR_TILE
  count_launches(1);
  return cudaGetLastError();
}

// Segment with rank 0: nothing to fit, but the A sections of the records do not exist either.
// Segment descriptor table entry, written by the device so that no host copy is needed.
__global__ void write_desc_kernel(SegDesc* table, int* blk2seg, int index, SegDesc d) {
  if (threadIdx.x == 0) table[index] = d;
  for (int b = threadIdx.x; b < d.nblk; b += blockDim.x) blk2seg[d.blk_start + b] = index;
}

__global__ void append_kernel(__half* buf_k, __half* buf_v, const __half* k_new, const __half* v_new,
                              int BH, int n_b, int slot) {
  // one 16-byte chunk per thread: BH * 16 chunks per side
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= BH * 16 * 2) return;
  const int side = i / (BH * 16), r = i % (BH * 16), bh = r >> 4, c = r & 15;
  const uint4 v = reinterpret_cast<const uint4*>(side == 0 ? k_new : v_new)[bh * 16 + c];
  reinterpret_cast<uint4*>(side == 0 ? buf_k : buf_v)[((size_t)bh * n_b + slot) * 16 + c] = v;
}

// ---------------------------------------------------------------------------
// host side: launch sequence for a range of (batch, head) pairs
// ---------------------------------------------------------------------------
// Filter / Quant / pack / residual of a long segment: per side, the register-resident kernel that fits the group
// shape, else the general one.  side0 = 1: the value side only.  Returns the number of launches through *launches.
template <int BITS>
static cudaError_t launch_quant(CompressArgs a, int nbh, int kmax_needed, cudaStream_t st, int* launches) {
  const int T = a.seg.T;
  const size_t smem = round_up(T * kXPitch * 2, 16) + (size_t)T * kRPitch * 4;
  const dim3 grid(a.seg.nblk, nbh, 1);
  const int first_side = a.side0;
  *launches = 0;
  for (int side = first_side; side < 2; ++side) {
    const int len = side == 0 ? T : a.cc.g_v, k = side == 0 ? a.seg.k_k : a.cc.k_v;
    cudaError_t e = cudaSuccess;
    if (T == kFastLen && len == kFastLen && k == 1) {
      if (side == 0) {
        quant_fast_kernel<BITS, 0><<<grid, 128, 0, st>>>(a);
      } else {
        e = cudaFuncSetAttribute(quant_fast_kernel<BITS, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kFastSmemV);
        if (e != cudaSuccess) return e;
        quant_fast_kernel<BITS, 1><<<grid, 128, kFastSmemV, st>>>(a);
      }
    } else if (len == kFast2Len && k == 2 && T % 32 == 0 && T <= kFast2Len) {
      if (side == 0) quant_fast2_kernel<BITS, 0><<<grid, 128, 0, st>>>(a);
      else quant_fast2_kernel<BITS, 1><<<grid, 128, 0, st>>>(a);
    } else {
      a.side0 = side;
#define GEAR_LAUNCH_Q(KM)                                                                                   \
  {                                                                                                         \
    e = cudaFuncSetAttribute(quant_pack_kernel<BITS, KM>, cudaFuncAttributeMaxDynamicSharedMemorySize,      \
                             (int)smem);                                                                   \
    if (e != cudaSuccess) return e;                                                                         \
    quant_pack_kernel<BITS, KM><<<grid, 128, smem, st>>>(a);                                                \
  }
      if (kmax_needed <= 1) GEAR_LAUNCH_Q(1)
      else if (kmax_needed <= 2) GEAR_LAUNCH_Q(2)
      else if (kmax_needed <= 4) GEAR_LAUNCH_Q(4)
      else GEAR_LAUNCH_Q(8)
#undef GEAR_LAUNCH_Q
    }
    *launches += 1;
  }
  return cudaGetLastError();
}

template <int MODE>
static void launch_pass(const PiArgs& p, cudaStream_t st) {
  // Four or eight rank columns per CTA; rank 16 is spread over two CTAs that read the same chunk of R one after the
  // other (the second finds it in L2).
  if (p.rank <= 4) pi_pass_kernel<MODE, 1><<<dim3(1, p.nchunk, p.ntiles), kPassWarps * 32, 0, st>>>(p);
  else pi_pass_kernel<MODE, 2><<<dim3(p.rank <= 8 ? 1 : 2, p.nchunk, p.ntiles), kPassWarps * 32, 0, st>>>(p);
}

// bytes of the power iteration's part of the workspace (a multiple of 256)
static size_t pi_workspace_bytes(int nbh, int n_c, int rank) {
  if (rank == 0) return 256;
  const size_t ntiles = (size_t)nbh * 2;
  const size_t nchunk = (n_c + kChunkRows - 1) / kChunkRows;
  size_t b = 0;
  b += ntiles * n_c * kHeadDim * 4;               // R
  b += ntiles * kHeadDim * kMaxRank * 4;          // Bcur
  b += ntiles * nchunk * kHeadDim * kMaxRank * 4; // Bp
  b += ntiles * n_c * kMaxRank * 4;               // A0
  b += ntiles * nchunk * 256 * 4;                 // Gp
  b += ntiles * 256 * 4;                          // W
  b += ntiles * 4;                                // Rmax
  return (b + 1024 + 255) / 256 * 256;
}

// csr_k < 0: a segment with per-block key groups; otherwise one with per-vector keys and csr_k outliers per channel
size_t compress_workspace_bytes(int nbh, int n_c, int rank, int csr_k) {
  return pi_workspace_bytes(nbh, n_c, rank) + (csr_k >= 0 ? kcvt_workspace_bytes(nbh, n_c, csr_k) : 0);
}

cudaError_t compress_range(const CompressJob& job, int bh0, int nbh, unsigned char* ws, cudaStream_t st) {
  const SegDesc& sd = job.seg;
  const size_t ntiles = (size_t)nbh * 2;
  const int nchunk = (sd.n_c + kChunkRows - 1) / kChunkRows;
  float* wsf = reinterpret_cast<float*>(ws);
  PiArgs pa;
  pa.seg = sd; pa.arena = job.arena; pa.bh0 = bh0; pa.ntiles = (int)ntiles; pa.n_c = sd.n_c; pa.rank = sd.rank;
  pa.nchunk = nchunk;
  pa.R = nullptr; pa.Rmax = nullptr; pa.Bcur = nullptr; pa.Bp = nullptr; pa.A0 = nullptr; pa.Gp = nullptr; pa.W = nullptr;
  pa.dbgA = job.dbgA; pa.dbgB = job.dbgB;
  if (sd.rank > 0) {
    pa.R = wsf;       wsf += ntiles * sd.n_c * kHeadDim;
    pa.Bcur = wsf;    wsf += ntiles * kHeadDim * kMaxRank;
    pa.Bp = wsf;      wsf += ntiles * nchunk * kHeadDim * kMaxRank;
    pa.A0 = wsf;      wsf += ntiles * sd.n_c * kMaxRank;
    pa.Gp = wsf;      wsf += ntiles * nchunk * 256;
    pa.W = wsf;       wsf += ntiles * 256;
    pa.Rmax = reinterpret_cast<unsigned int*>(wsf);
    if (cudaMemsetAsync(pa.Rmax, 0, ntiles * 4, st) != cudaSuccess) return cudaGetLastError();
  }
  CompressArgs ca;
  ca.seg = sd; ca.cc = job.cc; ca.arena = job.arena; ca.bh0 = bh0;
  ca.K = job.K + (size_t)bh0 * sd.n_c * kHeadDim;
  ca.V = job.V + (size_t)bh0 * sd.n_c * kHeadDim;
  ca.R = pa.R; ca.Rmax = pa.Rmax;
  const int kneed = sd.k_k > job.cc.k_v ? sd.k_k : job.cc.k_v;
  const bool per_vector = sd.csr_base16 != 0;          // keys: one group per channel over the whole segment
  ca.side0 = per_vector ? 1 : 0;
  int n_quant = 0;
  cudaError_t e = job.cc.bits == 2 ? launch_quant<2>(ca, nbh, kneed, st, &n_quant) : launch_quant<4>(ca, nbh, kneed, st, &n_quant);
  if (e != cudaSuccess) return e;
  count_launches(n_quant);
  if (per_vector) {
    KcvtArgs ka;
    ka.seg = sd; ka.arena = job.arena; ka.K = ca.K; ka.R = pa.R; ka.Rmax = pa.Rmax; ka.bh0 = bh0;
    e = launch_kcvt_keys(ka, nbh, job.cc.bits, ws + pi_workspace_bytes(nbh, sd.n_c, sd.rank), st);
    if (e != cudaSuccess) return e;
  }
  if (sd.rank == 0) return cudaSuccess;
  // init + per early loop (pass, reduce) + last loop (pass, gram, chol, gram, chol, store, reduce)
  count_launches(1 + 2 * (job.iters - 1) + (sd.rank > 8 ? 7 : 6) + (job.iters == 1 ? 1 : 0));

  const int tot = (int)ntiles * kHeadDim * kMaxRank;
  const float* b0 = job.B0 ? job.B0 : nullptr;
  pi_init_kernel<<<(tot + 255) / 256, 256, 0, st>>>(pa, b0, bh0, 0, job.seed, job.segment_index);
  for (int l = 0; l < job.iters; ++l) {
    const bool last = l == job.iters - 1;
    if (!last) {
      launch_pass<0>(pa, st);                                   // A = R B ; B = R^T A
      // the loop after this one is the last: its QR of B is folded into the reduction
      pi_reduce_b_kernel<<<(int)ntiles, kHeadDim, 0, st>>>(pa, (l + 1 == job.iters - 1) ? 1 : 0, 0, 0);
    } else {
      if (job.iters == 1) {                                     // single loop: orthonormalise the start itself
        PiArgs q = pa; q.nchunk = 0;
        // Bp unused with zero chunks: re-use the reduce kernel on Bcur through a one-chunk view
        cudaMemcpyAsync(pa.Bp, pa.Bcur, ntiles * kHeadDim * kMaxRank * 4, cudaMemcpyDeviceToDevice, st);
        q.nchunk = 1;
        pi_reduce_b_kernel<<<(int)ntiles, kHeadDim, 0, st>>>(q, 1, 0, 0);
      }
      launch_pass<1>(pa, st);                                   // A0 = R B, R^T A0; for ranks up to 8 also A0^T A0
      if (sd.rank > 8) pi_gram2_kernel<<<dim3(nchunk, (int)ntiles), 256, 0, st>>>(pa, 1);
      pi_chol_kernel<<<(int)ntiles, 32, 0, st>>>(pa, 1);        // A <- Q(A) by CholeskyQR, twice
      pi_gram2_kernel<<<dim3(nchunk, (int)ntiles), 256, 0, st>>>(pa, 0);
      pi_chol_kernel<<<(int)ntiles, 32, 0, st>>>(pa, 0);
      pi_store_a_kernel<<<dim3((sd.n_c + 255) / 256, (int)ntiles), 256, 0, st>>>(pa);   // A = A0 W
      pi_reduce_b_kernel<<<(int)ntiles, kHeadDim, 0, st>>>(pa, 0, 1, 1);
    }
  }
  return cudaGetLastError();
}

cudaError_t launch_write_desc(SegDesc* table, int* blk2seg, int index, const SegDesc& d, cudaStream_t st) {
  write_desc_kernel<<<1, 256, 0, st>>>(table, blk2seg, index, d);
  count_launches(1);
  return cudaGetLastError();
}

cudaError_t launch_append(void* buf_k, void* buf_v, const void* k_new, const void* v_new, int BH, int n_b, int slot,
                          cudaStream_t st) {
  const int n = BH * 16 * 2;
  append_kernel<<<(n + 255) / 256, 256, 0, st>>>((__half*)buf_k, (__half*)buf_v, (const __half*)k_new,
                                                 (const __half*)v_new, BH, n_b, slot);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace gear
