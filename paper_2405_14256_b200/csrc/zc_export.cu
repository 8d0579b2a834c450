// Export of cache contents in canonical layouts, for parity checks and inspection.
#include "zc_internal.h"
#include "zc_layout.cuh"

namespace {

__global__ void k_export_scores(const char* cache, ZcLayout lay, int n, float* __restrict__ out) {
  const int unit = blockIdx.y;
  const float* s = reinterpret_cast<const float*>(cache + unit * lay.unit_stride + lay.off_scores);
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j < n) out[(long long)unit * n + j] = s[j];
}

// grid.x: tile of the subset, grid.y: unit; 256 threads
__global__ void k_export_segment(const char* cache, ZcLayout lay, ZcSeg seg, int tensor, int subset,
                                 int32_t* __restrict__ idx_out, uint8_t* __restrict__ codes_out,
                                 float* __restrict__ sz_out, float* __restrict__ cf_out) {
  const int unit = blockIdx.y, tile = blockIdx.x;
  const int n = seg.n_tok[subset], bits = lay.bits[subset];
  const char* ub = cache + unit * lay.unit_stride;
  const int row_bytes = 16 * bits;
  const char* tp = ub + lay.off_tiles[subset] + (long long)(seg.tile0[subset] + tile) * lay.tile_bytes[subset];
  const int t0 = tile * ZC_TILE;
  const int n_here = min(ZC_TILE, n - t0);
  if (idx_out) {
    const int32_t* idx = reinterpret_cast<const int32_t*>(ub + lay.off_idx) + seg.idx_off +
                         (subset == 0 ? 0 : seg.n_tok[0]);
    for (int i = threadIdx.x; i < n_here; i += blockDim.x)
      idx_out[(long long)unit * n + t0 + i] = idx[t0 + i];
  }
  const int kch = lay.kch;
  if (bits == 16) {
    // rows kept at full precision: "codes" are the rows' bytes, there are no parameters
    if (codes_out) {
      for (int i = threadIdx.x; i < n_here * 64; i += blockDim.x) {
        const int tl = i >> 6, wd = i & 63;
        const char* sb = tp + (tl / ZC_SUB) * zc_sub_bytes(16, 0) + (tensor ? ZC_SUB * ZC_D * 2 : 0);
        reinterpret_cast<unsigned*>(codes_out + ((long long)unit * n + t0 + tl) * row_bytes)[wd] =
            reinterpret_cast<const unsigned*>(sb + (tl % ZC_SUB) * ZC_D * 2)[wd];
      }
    }
    return;
  }
  if (sz_out && kch && tensor == 0) {
    // channelwise keys: (scale, zero point) of every channel, from the run's factor block
    if (tile == 0) {
      const float* fac = reinterpret_cast<const float*>(ub + lay.off_fac) + (seg.run0 + subset) * ZC_FAC_FLOATS;
      for (int i = threadIdx.x; i < 2 * ZC_D; i += blockDim.x)
        sz_out[(long long)unit * 2 * ZC_D + i] = (i & 1) ? fac[ZC_FAC_ZK + (i >> 1)] : fac[i >> 1];
    }
  } else if (sz_out) {
    const int poff = zc_sub_off_par(bits);
    for (int i = threadIdx.x; i < 2 * n_here; i += blockDim.x) {
      const int tl = i >> 1;
      const char* blk = tp + (tl / ZC_SUB) * zc_sub_bytes(bits, kch, lay.p16) + poff;
      float val;
      if (lay.p16) {   // (fp16 scale, int16 zero point) per tensor
        const unsigned short raw = reinterpret_cast<const unsigned short*>(blk)[4 * (tl % ZC_SUB) + 2 * tensor + (i & 1)];
        val = (i & 1) ? (float)(short)raw : __half2float(__ushort_as_half(raw));
      } else {
        const float* par = reinterpret_cast<const float*>(blk);
        val = kch ? par[2 * (tl % ZC_SUB) + (i & 1)] : par[4 * (tl % ZC_SUB) + 2 * tensor + (i & 1)];
      }
      sz_out[((long long)unit * n + t0) * 2 + i] = val;
    }
  }
  if (cf_out && tile == 0 && !(kch && tensor == 0)) {
    const float* fac = reinterpret_cast<const float*>(ub + lay.off_fac) +
                       (seg.run0 + subset) * ZC_FAC_FLOATS + (tensor == 0 ? 0 : ZC_D);
    for (int i = threadIdx.x; i < ZC_D; i += blockDim.x) cf_out[(long long)unit * ZC_D + i] = fac[i];
  }
  if (codes_out) {
    const int per = 8 / bits;
    for (int i = threadIdx.x; i < n_here * row_bytes; i += blockDim.x) {
      const int tl = i / row_bytes, m = i % row_bytes;
      unsigned byte = 0;
      const char* sb = tp + (tl / ZC_SUB) * zc_sub_bytes(bits, kch, lay.p16);
      if (tensor == 0) {
        byte = reinterpret_cast<const unsigned char*>(sb)[(tl % ZC_SUB) * row_bytes + m];
      } else {
        const unsigned* vblk = reinterpret_cast<const unsigned*>(sb + zc_sub_off_vcodes(bits));
        for (int e = 0; e < per; ++e) {
          int word, shift;
          zc_vcode_pos(bits, tl % ZC_SUB, m * per + e, &word, &shift);
          byte |= ((vblk[word] >> shift) & ((1u << bits) - 1u)) << (bits * e);
        }
      }
      codes_out[((long long)unit * n + t0 + tl) * row_bytes + m] = (uint8_t)byte;
    }
  }
}

}  // namespace

int zc_launch_export_scores(zc_cache* c, float* out, int n, cudaStream_t st) {
  dim3 grid(zc_ceil_div(n, 256), c->lay.units);
  k_export_scores<<<grid, 256, 0, st>>>(c->base, c->lay, n, out);
  c->launches += 1;
  return cudaGetLastError();
}

int zc_launch_export_segment(zc_cache* c, const ZcSeg& seg, int tensor, int subset, int32_t* idx,
                             uint8_t* codes, float* sz, float* cf, cudaStream_t st) {
  const int n = seg.n_tok[subset];
  if (n <= 0) return cudaSuccess;
  dim3 grid(zc_ceil_div(n, ZC_TILE), c->lay.units);
  k_export_segment<<<grid, 256, 0, st>>>(c->base, c->lay, seg, tensor, subset, idx, codes, sz, cf);
  c->launches += 1;
  return cudaGetLastError();
}
