// Keys of a segment under per-vector grouping (Section 2, "Group-wise Quantization": per-channel key vectors; the
// KCVT backbone of Section 4): one quantization group per channel over all n_c tokens of the segment, Filter_s
// (Eq. 4) on that whole vector.
//   kcvt_select_kernel : per channel, the k largest and k smallest entries by a two-level radix select on the fp16
//                        order (ties to the lower token), Eq. 2 on the rest, codes (one byte each, token-major) and
//                        the fp32 residual
//   kcvt_list_kernel   : the outliers of a (batch, head), sorted into per-block lists; block headers, scales
//   kcvt_pack_kernel   : codes of a 64-token block into the fragment order of the decode kernel
// The arithmetic that decides a code is the same binary32 sequence as in the per-group kernels.
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <math.h>

#include "gear_internal.cuh"

namespace gear {

constexpr int kSelChannels = 8;     // channels per CTA of the select kernel, one per warp
constexpr int kSelChunk = 256;      // tokens whose codes and residuals are staged before they are written out
constexpr int kBlockTok = 64;       // tokens per record block of such a segment

// fp16 bits -> 16-bit key with the order of the values; -0 and +0 share a key
__device__ __forceinline__ unsigned int order_key(unsigned int h) {
  if ((h & 0x7FFFu) == 0u) h = 0u;
  return (h & 0x8000u) ? (~h & 0xFFFFu) : (h | 0x8000u);
}
__device__ __forceinline__ float key_value(unsigned int key) {
  const unsigned int h = (key & 0x8000u) ? (key & 0x7FFFu) : (~key & 0xFFFFu);
  return __half2float(__ushort_as_half((unsigned short)h));
}

// Of a 256-bin histogram, the highest bin b with (count of the bins above b) < want <= (count of the bins >= b);
// over = the count of the bins above it.  One warp; lane l owns bins 8 l .. 8 l + 7.
__device__ __forceinline__ int pick_bin(const unsigned int* hist, int want, int lane, int& over) {
  unsigned int mine = 0u;
#pragma unroll
  for (int b = 0; b < 8; ++b) mine += hist[8 * lane + b];
  unsigned int incl = mine;                      // sum over lanes >= this one
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned int v = __shfl_down_sync(0xffffffffu, incl, o);
    if (lane + o < 32) incl += v;
  }
  const unsigned int above = incl - mine;
  const bool here = above < (unsigned int)want && (unsigned int)want <= incl;
  const int src = __ffs((int)__ballot_sync(0xffffffffu, here)) - 1;
  int bin = 0, ov = 0;
  if (here) {
    unsigned int acc = above;
    for (int b = 7; b >= 0; --b) {
      const unsigned int c = hist[8 * lane + b];
      if (acc + c >= (unsigned int)want) { bin = 8 * lane + b; ov = (int)acc; break; }
      acc += c;
    }
  }
  over = __shfl_sync(0xffffffffu, ov, src);
  return __shfl_sync(0xffffffffu, bin, src);
}

// The k-th largest key of keys[0 .. n) and the k-th smallest, by two 8-bit histogram levels; beyond_t / beyond_b: how
// many keys lie strictly beyond them.  The smallest is the largest of the complemented keys: its first-level histogram
// is the mirror image of the other one, its second level is counted in the same pass.  One warp, hist = 512 words.
__device__ __forceinline__ void warp_select(const unsigned short* keys, int n, int k, unsigned int* hist, int lane,
                                            unsigned int& key_t, int& beyond_t, unsigned int& key_b, int& beyond_b) {
  unsigned int* hist_b = hist + 256;
  for (int i = lane; i < 256; i += 32) hist[i] = 0u;
  __syncwarp();
  for (int i = lane; i < n; i += 32) atomicAdd(&hist[keys[i] >> 8], 1u);
  __syncwarp();
  for (int i = lane; i < 256; i += 32) hist_b[i] = hist[255 - i];
  __syncwarp();
  int over_t, over_b;
  const unsigned int pre_t = (unsigned int)pick_bin(hist, k, lane, over_t);
  const unsigned int pre_b = (unsigned int)pick_bin(hist_b, k, lane, over_b);
  __syncwarp();
  for (int i = lane; i < 512; i += 32) hist[i] = 0u;
  __syncwarp();
  for (int i = lane; i < n; i += 32) {
    const unsigned int key = keys[i], kf = key ^ 0xFFFFu;
    if ((key >> 8) == pre_t) atomicAdd(&hist[key & 0xFFu], 1u);
    if ((kf >> 8) == pre_b) atomicAdd(&hist_b[kf & 0xFFu], 1u);
  }
  __syncwarp();
  int over2_t, over2_b;
  const unsigned int lo_t = (unsigned int)pick_bin(hist, k - over_t, lane, over2_t);
  const unsigned int lo_b = (unsigned int)pick_bin(hist_b, k - over_b, lane, over2_b);
  __syncwarp();
  key_t = (pre_t << 8) | lo_t;
  key_b = ((pre_b << 8) | lo_b) ^ 0xFFFFu;
  beyond_t = over_t + over2_t;
  beyond_b = over_b + over2_b;
}

template <int BITS>
__global__ void __launch_bounds__(kSelChannels * 32) kcvt_select_kernel(KcvtArgs p) {
  extern __shared__ __align__(16) unsigned char sm_raw[];
  const SegDesc& sd = p.seg;
  const int n_c = sd.n_c, k = sd.csr_k / 2;
  const int cg = blockIdx.x, bhl = blockIdx.y, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int ch = cg * kSelChannels + warp;
  // shared memory: keys [8][n_c] u16 | outlier bitmask [8][n_c / 32] | histograms [8][512] | stage of a chunk
  unsigned short* keys_all = reinterpret_cast<unsigned short*>(sm_raw);
  unsigned int* mask_all = reinterpret_cast<unsigned int*>(sm_raw + (size_t)kSelChannels * n_c * 2);
  unsigned int* hist_all = mask_all + kSelChannels * (n_c / 32);
  float* stage_r = reinterpret_cast<float*>(hist_all + kSelChannels * 512);       // [kSelChunk][8]
  unsigned char* stage_c = reinterpret_cast<unsigned char*>(stage_r + kSelChunk * kSelChannels);   // [kSelChunk][8]
  unsigned short* keys = keys_all + (size_t)warp * n_c;
  unsigned int* omask = mask_all + warp * (n_c / 32);
  unsigned int* hist = hist_all + warp * 512;

  const __half* X = p.K + (size_t)bhl * n_c * kHeadDim;
  for (int tok = tid; tok < n_c; tok += blockDim.x) {          // 16 bytes (this CTA's 8 channels) of every token row
    const uint4 v = *reinterpret_cast<const uint4*>(X + (size_t)tok * kHeadDim + cg * kSelChannels);
    const unsigned int w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      keys_all[(size_t)(2 * i) * n_c + tok] = (unsigned short)order_key(w[i] & 0xFFFFu);
      keys_all[(size_t)(2 * i + 1) * n_c + tok] = (unsigned short)order_key(w[i] >> 16);
    }
  }
  __syncthreads();

  // ---- Filter_s (Eq. 4) on the channel's whole vector
  unsigned int key_t = 0xFFFFu, key_b = 0u;
  int need_t = 0, need_b = 0;                   // entries equal to the threshold key that still leave, lowest tokens first
  if (k > 0) {
    int beyond_t, beyond_b;
    warp_select(keys, n_c, k, hist, lane, key_t, beyond_t, key_b, beyond_b);
    need_t = k - beyond_t;
    need_b = k - beyond_b;
  }
  const bool same = key_t == key_b;             // the thresholds meet only when all kept entries would be equal
  unsigned int kmin = 0xFFFFu, kmax = 0u;
  int eq_t = 0, eq_b = 0, n_out = 0;
  unsigned int* olist = p.olist + ((size_t)bhl * kHeadDim + ch) * sd.csr_k;
  for (int base = 0; base < n_c; base += 32) {
    const unsigned int key = keys[base + lane];
    bool out = false;
    if (k > 0) {
      const bool is_t = key == key_t, is_b = key == key_b;
      out = key > key_t || key < key_b;
      if (__any_sync(0xffffffffu, is_t || is_b)) {        // an entry on a threshold: ties go to the lower token
        const unsigned int bt = __ballot_sync(0xffffffffu, is_t), bb = __ballot_sync(0xffffffffu, is_b);
        const unsigned int below = (1u << lane) - 1u;
        const int rt = eq_t + __popc(bt & below), rb = eq_b + __popc(bb & below);
        out = out || (is_t && rt < need_t) ||
              (is_b && (same ? (rt >= need_t && rt < need_t + need_b) : rb < need_b));
        eq_t += __popc(bt); eq_b += __popc(bb);
      }
    }
    const unsigned int bo = __ballot_sync(0xffffffffu, out);
    if (lane == 0) omask[base >> 5] = bo;
    if (out) {
      const int pos = n_out + __popc(bo & ((1u << lane) - 1u));
      const unsigned int bits = __half_as_ushort(X[(size_t)(base + lane) * kHeadDim + ch]);
      olist[pos] = (unsigned int)(base + lane) | (bits << 16);
    } else {
      kmin = min(kmin, key); kmax = max(kmax, key);
    }
    n_out += __popc(bo);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    kmin = min(kmin, __shfl_xor_sync(0xffffffffu, kmin, o));
    kmax = max(kmax, __shfl_xor_sync(0xffffffffu, kmax, o));
  }
  // ---- Eq. 2 on the kept entries: binary32, one rounding per operation
  const float mn = key_value(kmin), mx = key_value(kmax);
  const float levels = (float)((1 << BITS) - 1);
  const float range = __fsub_rn(mx, mn);
  const float d32 = __fdiv_rn(range, levels);
  const __half d16 = __float2half_rn(d32);
  const float d = __half2float(d16);
  const float inv = d != 0.f ? __fdiv_rn(1.0f, d) : 0.f;
  if (lane == 0) {
    p.sz[(size_t)bhl * kHeadDim + ch] = __halves2half2(d16, __float2half_rn(mn));
    if (p.Rmax != nullptr) {        // a bound on the residuals of the channel (see quant_fast_kernel)
      const float rb = (d != 0.f ? 0.50390625f * d : range) + 2.4e-7f * (fabsf(mn) + fabsf(mx));
      atomicMax(p.Rmax + bhl * 2, __float_as_uint(rb));
    }
  }
  // ---- codes and residuals, a chunk of tokens at a time through shared memory so that rows leave whole
  constexpr float kRound = 12582912.0f;
  float* R = p.R ? p.R + ((size_t)bhl * 2) * n_c * kHeadDim : nullptr;
  unsigned char* C8 = p.codes8 + (size_t)bhl * n_c * kHeadDim;
  for (int c0 = 0; c0 < n_c; c0 += kSelChunk) {
    const int nt = min(kSelChunk, n_c - c0);
    for (int i = lane; i < nt; i += 32) {
      const int tok = c0 + i;
      const bool out = (omask[tok >> 5] >> (tok & 31)) & 1u;
      const float x = key_value(keys[tok]);
      const float t = __fmul_rn(__fsub_rn(x, mn), inv);
      const float y = __fadd_rn(fminf(fmaxf(t, 0.f), levels), kRound);
      const float resid = x - fmaf(__fsub_rn(y, kRound), d, mn);
      stage_c[i * kSelChannels + warp] = out ? 0 : (unsigned char)(__float_as_uint(y) & 0xFFu);
      stage_r[i * kSelChannels + warp] = out ? 0.f : resid;
    }
    __syncthreads();
    for (int i = tid; i < nt; i += blockDim.x) {
      const size_t row = (size_t)(c0 + i) * kHeadDim + cg * kSelChannels;
      *reinterpret_cast<uint2*>(C8 + row) = *reinterpret_cast<const uint2*>(stage_c + i * kSelChannels);
      if (R != nullptr) {
        const float4* src = reinterpret_cast<const float4*>(stage_r + i * kSelChannels);
        reinterpret_cast<float4*>(R + row)[0] = src[0];
        reinterpret_cast<float4*>(R + row)[1] = src[1];
      }
    }
    __syncthreads();
  }
}

// One CTA per (batch, head): the per-channel outlier lists (token ascending) become per-block lists, and every
// block record gets its header fields of the key side and the channels' (scale, zero).
__global__ void __launch_bounds__(256) kcvt_list_kernel(KcvtArgs p) {
  extern __shared__ __align__(16) unsigned char sm_raw[];
  const SegDesc& sd = p.seg;
  const int nblk = sd.nblk, k2 = sd.csr_k, bhl = blockIdx.x, tid = threadIdx.x;
  unsigned int* cnt = reinterpret_cast<unsigned int*>(sm_raw);          // [nblk][128], then exclusive offsets
  unsigned int* off = cnt + (size_t)nblk * kHeadDim;                   // [nblk + 1]
  unsigned int* dmax = off + nblk + 1;                                  // [nblk] bit patterns
  __shared__ unsigned int smax_bits;
  for (int i = tid; i < nblk * kHeadDim; i += blockDim.x) cnt[i] = 0u;
  for (int i = tid; i < nblk; i += blockDim.x) dmax[i] = 0u;
  if (tid == 0) smax_bits = 0u;
  __syncthreads();
  const unsigned int* olist = p.olist + (size_t)bhl * kHeadDim * k2;
  const __half2* sz = p.sz + (size_t)bhl * kHeadDim;
  if (tid < kHeadDim) {
    for (int e = 0; e < k2; ++e) cnt[((olist[tid * k2 + e] & 0xFFFFu) / kBlockTok) * kHeadDim + tid] += 1u;
    atomicMax(&smax_bits, __float_as_uint(__low2float(sz[tid])));      // scales are non-negative
  }
  __syncthreads();
  for (int b = tid; b < nblk; b += blockDim.x) {          // exclusive scan over the channels of a block
    unsigned int acc = 0u;
    for (int c = 0; c < kHeadDim; ++c) { const unsigned int v = cnt[b * kHeadDim + c]; cnt[b * kHeadDim + c] = acc; acc += v; }
    off[b + 1] = acc;
  }
  __syncthreads();
  if (tid == 0) {
    off[0] = 0u;
    for (int b = 0; b < nblk; ++b) off[b + 1] += off[b];
  }
  __syncthreads();
  unsigned char* seg0 = p.arena + sd.seg_base;
  unsigned char* csr = seg0 + (size_t)sd.csr_base16 * 16 + (size_t)(p.bh0 + bhl) * csr_stride_bytes(nblk, k2);
  unsigned int* g_off = reinterpret_cast<unsigned int*>(csr);
  unsigned int* g_ent = reinterpret_cast<unsigned int*>(csr + csr_offsets_bytes(nblk));
  for (int i = tid; i <= nblk; i += blockDim.x) g_off[i] = off[i];
  if (tid < kHeadDim) {
    const float zero = __high2float(sz[tid]);
    int prev_blk = -1, run = 0;
    for (int e = 0; e < k2; ++e) {
      const unsigned int w = olist[tid * k2 + e];
      const int tok = (int)(w & 0xFFFFu), blk = tok / kBlockTok;
      run = blk == prev_blk ? run + 1 : 0;
      prev_blk = blk;
      g_ent[off[blk] + cnt[blk * kHeadDim + tid] + run] =
          (unsigned int)(tok - blk * kBlockTok) | ((unsigned int)tid << 8) | (w & 0xFFFF0000u);
      const float v = __half2float(__ushort_as_half((unsigned short)(w >> 16)));
      atomicMax(&dmax[blk], __float_as_uint(fabsf(v - zero)));
    }
  }
  __syncthreads();
  unsigned char* recs = seg0 + (size_t)(p.bh0 + bhl) * sd.bh_stride + sd.bfac_bytes;
  for (int i = tid; i < nblk * kHeadDim; i += blockDim.x) {
    const int b = i / kHeadDim, c = i % kHeadDim;
    reinterpret_cast<__half2*>(recs + (size_t)b * sd.rec_bytes + sd.off_kscale)[c] = sz[c];
  }
  for (int b = tid; b < nblk; b += blockDim.x) {
    float* hdr = reinterpret_cast<float*>(recs + (size_t)b * sd.rec_bytes);
    hdr[0] = __uint_as_float(dmax[b]);
    hdr[2] = __uint_as_float(smax_bits);
  }
}

template <int BITS>
__global__ void __launch_bounds__(128) kcvt_pack_kernel(KcvtArgs p) {
  constexpr int F = 8 / BITS, kPitch = kHeadDim + 4;
  __shared__ __align__(16) unsigned char codes[kBlockTok * kPitch];
  const SegDesc& sd = p.seg;
  const int blk = blockIdx.x, bhl = blockIdx.y, tid = threadIdx.x;
  const unsigned char* C8 = p.codes8 + ((size_t)bhl * sd.n_c + (size_t)blk * kBlockTok) * kHeadDim;
  for (int i = tid; i < kBlockTok * 8; i += 128) {          // 16-byte pieces
    const int tok = i >> 3, q = i & 7;
    const uint4 v = reinterpret_cast<const uint4*>(C8)[i];
    unsigned int* dst = reinterpret_cast<unsigned int*>(codes + tok * kPitch + 16 * q);
    dst[0] = v.x; dst[1] = v.y; dst[2] = v.z; dst[3] = v.w;
  }
  __syncthreads();
  unsigned char* rec = p.arena + sd.seg_base + (size_t)(p.bh0 + bhl) * sd.bh_stride + sd.bfac_bytes +
                       (size_t)blk * sd.rec_bytes;
  unsigned int* dst = reinterpret_cast<unsigned int*>(rec + sd.off_kcodes);
  constexpr int kWords = kSlab * kHeadDim * BITS / 32;            // words per slab
  for (int li = tid; li < (kBlockTok / kSlab) * kWords; li += 128) {
    const int slab = li / kWords, wl = li % kWords;
    const int w = wl & 3, lane = (wl >> 2) & 31, tau = wl >> 7;
    const int tok = slab * kSlab + (lane >> 2) + 8 * (w & 1);
    const int ch = 32 * F * tau + 16 * (w >> 1) + 4 * (lane & 3);
    unsigned int word = 0;
#pragma unroll
    for (int j = 0; j < F; ++j)
      word |= *reinterpret_cast<const unsigned int*>(&codes[tok * kPitch + ch + 32 * j]) << (BITS * j);
    dst[li] = word;
  }
}

size_t kcvt_select_smem(int n_c) {
  return (size_t)kSelChannels * n_c * 2 + (size_t)kSelChannels * (n_c / 32) * 4 + kSelChannels * 512 * 4 +
         (size_t)kSelChunk * kSelChannels * 5;
}
size_t kcvt_list_smem(int nblk) { return ((size_t)nblk * kHeadDim + 2 * (size_t)nblk + 1) * 4; }

bool kcvt_fits(int n_c) {
  return n_c % kBlockTok == 0 && n_c <= 65535 && kcvt_select_smem(n_c) <= 200 * 1024 &&
         kcvt_list_smem(n_c / kBlockTok) <= 200 * 1024;
}

size_t kcvt_workspace_bytes(int nbh, int n_c, int csr_k) {
  return (size_t)nbh * n_c * kHeadDim + (size_t)nbh * kHeadDim * csr_k * 4 + (size_t)nbh * kHeadDim * 4 + 256;
}

// Key side of a per-vector segment for the (batch, head) range of `a`; three launches.
cudaError_t launch_kcvt_keys(KcvtArgs a, int nbh, int bits, unsigned char* ws, cudaStream_t st) {
  const SegDesc& sd = a.seg;
  a.codes8 = ws;
  a.olist = reinterpret_cast<unsigned int*>(ws + (size_t)nbh * sd.n_c * kHeadDim);
  a.sz = reinterpret_cast<__half2*>(a.olist + (size_t)nbh * kHeadDim * sd.csr_k);
  const size_t sm_sel = kcvt_select_smem(sd.n_c), sm_list = kcvt_list_smem(sd.nblk);
  cudaError_t e;
  if (bits == 2) {
    e = cudaFuncSetAttribute(kcvt_select_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm_sel);
    if (e != cudaSuccess) return e;
    kcvt_select_kernel<2><<<dim3(kHeadDim / kSelChannels, nbh), kSelChannels * 32, sm_sel, st>>>(a);
  } else {
    e = cudaFuncSetAttribute(kcvt_select_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm_sel);
    if (e != cudaSuccess) return e;
    kcvt_select_kernel<4><<<dim3(kHeadDim / kSelChannels, nbh), kSelChannels * 32, sm_sel, st>>>(a);
  }
  e = cudaFuncSetAttribute(kcvt_list_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm_list);
  if (e != cudaSuccess) return e;
  kcvt_list_kernel<<<nbh, 256, sm_list, st>>>(a);
  if (bits == 2) kcvt_pack_kernel<2><<<dim3(sd.nblk, nbh), 128, 0, st>>>(a);
  else kcvt_pack_kernel<4><<<dim3(sd.nblk, nbh), 128, 0, st>>>(a);
  count_launches(3);
  return cudaGetLastError();
}

}  // namespace gear
