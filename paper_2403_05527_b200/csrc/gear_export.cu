// Canonical (unpacked) dump of one compressed segment: the parity surface of
// the tests.  One thread per output element; not on any timed path.
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "../../include/gear.h"
#include "gear_internal.cuh"

namespace gear {

__device__ __forceinline__ const unsigned char* record_of(const unsigned char* arena, const SegDesc& sd, int bh, int blk) {
  return arena + sd.seg_base + (size_t)bh * sd.bh_stride + sd.bfac_bytes + (size_t)blk * sd.rec_bytes;
}

// inverse of code_coord_k / code_coord_v: where does the code of (token in slab, channel) sit?
__device__ __forceinline__ unsigned int load_code(const unsigned char* rec, const SegDesc& sd, int bits, int side,
                                                  int slab, int ts, int ch) {
  const int hpw = regs_per_word(bits);
  int lane, q, u, e;
  if (side == 0) {
    const int th = ts >> 3, gid = ts & 7, kc = ch >> 4, c16 = ch & 15;
    const int hi = c16 >> 3, t = (c16 & 7) >> 1;
    e = c16 & 1;
    lane = gid * 4 + t;
    const int kpw = hpw / 2, wpt = 16 / hpw;
    q = th * wpt + kc / kpw;
    u = 2 * (kc % kpw) + hi;
  } else {
    const int mt = ch >> 4, c16 = ch & 15, gid = c16 & 7;
    const int a = (c16 >> 3) | ((ts >> 3) << 1), t = (ts & 7) >> 1;
    e = ts & 1;
    lane = gid * 4 + t;
    const int tpp = hpw / 2;
    q = 2 * (mt / tpp) + (a >> 1);
    u = 2 * (mt % tpp) + (a & 1);
  }
  const unsigned int* words =
      reinterpret_cast<const unsigned int*>(rec + (side == 0 ? sd.off_kcodes : sd.off_vcodes) + slab * sd.slab_codes);
  return (words[word_index(lane, q)] >> (16 * e + bits * u)) & ((1u << bits) - 1u);
}

__global__ void export_kernel(const unsigned char* arena, SegDesc sd, CacheConst cc, int what, void* dst, size_t n) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const int side = what & 1;
  const int d = kHeadDim, T = sd.T, ngv = cc.ngv;
  switch (what) {
    case GEAR_EXP_K_CODES: case GEAR_EXP_V_CODES: {
      const int ch = i % d; const size_t r = i / d; const int tok = r % sd.n_c, bh = r / sd.n_c;
      const unsigned char* rec = record_of(arena, sd, bh, tok / T);
      const int tib = tok % T;
      reinterpret_cast<unsigned char*>(dst)[i] = (unsigned char)load_code(rec, sd, cc.bits, side, tib / kSlab, tib % kSlab, ch);
      break;
    }
    case GEAR_EXP_K_SCALE: case GEAR_EXP_K_ZERO: {
      const int ch = i % d; const size_t r = i / d; const int blk = r % sd.nblk, bh = r / sd.nblk;
      const __half2 z = reinterpret_cast<const __half2*>(record_of(arena, sd, bh, blk) + sd.off_kscale)[ch];
      reinterpret_cast<__half*>(dst)[i] = what == GEAR_EXP_K_SCALE ? __low2half(z) : __high2half(z);
      break;
    }
    case GEAR_EXP_V_SCALE: case GEAR_EXP_V_ZERO: {
      const int g = i % ngv; const size_t r = i / ngv; const int tok = r % sd.n_c, bh = r / sd.n_c;
      const __half2 z = reinterpret_cast<const __half2*>(record_of(arena, sd, bh, tok / T) + sd.off_vscale)[(tok % T) * ngv + g];
      reinterpret_cast<__half*>(dst)[i] = what == GEAR_EXP_V_SCALE ? __low2half(z) : __high2half(z);
      break;
    }
    case GEAR_EXP_K_OUT_IDX: case GEAR_EXP_K_OUT_VAL: {
      const int k2 = 2 * sd.k_k;
      const int e = i % k2; size_t r = i / k2; const int ch = r % d; r /= d; const int blk = r % sd.nblk, bh = r / sd.nblk;
      const unsigned char* rec = record_of(arena, sd, bh, blk);
      if (what == GEAR_EXP_K_OUT_IDX) reinterpret_cast<unsigned char*>(dst)[i] = rec[sd.off_koidx + ch * k2 + e];
      else reinterpret_cast<__half*>(dst)[i] = reinterpret_cast<const __half*>(rec + sd.off_koval)[ch * k2 + e];
      break;
    }
    case GEAR_EXP_V_OUT_IDX: case GEAR_EXP_V_OUT_VAL: {
      const int k2 = 2 * cc.k_v;
      const int e = i % k2; size_t r = i / k2; const int g = r % ngv; r /= ngv; const int tok = r % sd.n_c, bh = r / sd.n_c;
      const unsigned char* rec = record_of(arena, sd, bh, tok / T);
      const int li = ((tok % T) * ngv + g) * k2 + e;
      if (what == GEAR_EXP_V_OUT_IDX) reinterpret_cast<unsigned char*>(dst)[i] = rec[sd.off_voidx + li];
      else reinterpret_cast<__half*>(dst)[i] = reinterpret_cast<const __half*>(rec + sd.off_voval)[li];
      break;
    }
    case GEAR_EXP_K_A: case GEAR_EXP_V_A: {
      const int rho = i % sd.rank; const size_t r = i / sd.rank; const int tok = r % sd.n_c, bh = r / sd.n_c;
      const unsigned char* rec = record_of(arena, sd, bh, tok / T);
      const int tib = tok % T, slab = tib / kSlab, ts = tib % kSlab;
      const __half v = side == 0 ? reinterpret_cast<const __half*>(rec + sd.off_ak + slab * sd.slab_a)[ts * sd.r_pad + rho]
                                 : reinterpret_cast<const __half*>(rec + sd.off_av + slab * sd.slab_a)[rho * kSlab + ts];
      reinterpret_cast<float*>(dst)[i] = __half2float(v);
      break;
    }
    case GEAR_EXP_K_B: case GEAR_EXP_V_B: {
      const int rho = i % sd.rank; const size_t r = i / sd.rank; const int ch = r % d, bh = r / d;
      const __half* bf = reinterpret_cast<const __half*>(arena + sd.seg_base + (size_t)bh * sd.bh_stride);
      const __half v = side == 0 ? bf[rho * d + ch] : bf[sd.r_pad * d + ch * sd.r_pad + rho];
      reinterpret_cast<float*>(dst)[i] = __half2float(v);
      break;
    }
    default: break;
  }
}

cudaError_t launch_export(const unsigned char* arena, const SegDesc& sd, const CacheConst& cc, int what, void* dst,
                          size_t n_elems, cudaStream_t st) {
  if (n_elems == 0) return cudaSuccess;
  export_kernel<<<(unsigned int)((n_elems + 255) / 256), 256, 0, st>>>(arena, sd, cc, what, dst, n_elems);
  return cudaGetLastError();
}

}  // namespace gear
