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

// the code of (token in block, channel): inverse of code_coord_k / code_coord_v
__device__ __forceinline__ unsigned int load_code(const unsigned char* rec, const SegDesc& sd, int bits, int side,
                                                  int tib, int ch) {
  int word, shift;
  const unsigned int* words;
  if (side == 0) {
    code_slot_k(bits, tib % kSlab, ch, word, shift);
    words = reinterpret_cast<const unsigned int*>(rec + sd.off_kcodes + (tib / kSlab) * sd.slab_codes);
  } else {
    code_slot_v(bits, tib % 32, ch, word, shift);
    words = reinterpret_cast<const unsigned int*>(rec + sd.off_vcodes + (tib / 32) * 2 * sd.slab_codes);
  }
  return (words[word] >> shift) & ((1u << bits) - 1u);
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
      reinterpret_cast<unsigned char*>(dst)[i] = (unsigned char)load_code(rec, sd, cc.bits, side, tib, ch);
      break;
    }
    case GEAR_EXP_K_SCALE: case GEAR_EXP_K_ZERO: {
      const int rows = sd.csr_base16 ? 1 : sd.nblk;       // per-vector keys: every block repeats the segment's pair
      const int ch = i % d; const size_t r = i / d; const int blk = r % rows, bh = r / rows;
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

// Key outliers of a segment with per-vector keys: one thread per (batch, head, channel) walks the list of its
// (batch, head) -- sorted by block, channel, token -- and writes the channel's entries, token ascending.
__global__ void export_list_kernel(const unsigned char* arena, SegDesc sd, int what, void* dst, int BH) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= BH * kHeadDim) return;
  const int bh = i / kHeadDim, ch = i % kHeadDim;
  const unsigned char* csr = arena + sd.seg_base + (size_t)sd.csr_base16 * 16 + (size_t)bh * csr_stride_bytes(sd.nblk, sd.csr_k);
  const unsigned int* offs = reinterpret_cast<const unsigned int*>(csr);
  const unsigned int* ent = reinterpret_cast<const unsigned int*>(csr + csr_offsets_bytes(sd.nblk));
  int n = 0;
  for (int b = 0; b < sd.nblk; ++b)
    for (unsigned int e = offs[b]; e < offs[b + 1]; ++e) {
      const unsigned int w = ent[e];
      if ((int)((w >> 8) & 0xFFu) != ch || n >= sd.csr_k) continue;
      if (what == GEAR_EXP_K_OUT_IDX) reinterpret_cast<int*>(dst)[(size_t)i * sd.csr_k + n] = b * sd.T + (int)(w & 0xFFu);
      else reinterpret_cast<unsigned short*>(dst)[(size_t)i * sd.csr_k + n] = (unsigned short)(w >> 16);
      ++n;
    }
}

cudaError_t launch_export(const unsigned char* arena, const SegDesc& sd, const CacheConst& cc, int what, void* dst,
                          size_t n_elems, cudaStream_t st) {
  if (n_elems == 0) return cudaSuccess;
  if (sd.csr_base16 != 0 && (what == GEAR_EXP_K_OUT_IDX || what == GEAR_EXP_K_OUT_VAL)) {
    export_list_kernel<<<(cc.BH * kHeadDim + 127) / 128, 128, 0, st>>>(arena, sd, what, dst, cc.BH);
    return cudaGetLastError();
  }
  export_kernel<<<(unsigned int)((n_elems + 255) / 256), 256, 0, st>>>(arena, sd, cc, what, dst, n_elems);
  return cudaGetLastError();
}

}  // namespace gear
