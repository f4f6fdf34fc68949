// Re-tiling kernels: interchange layout (see include/eora_linear.h) -> WMat tiles
// (see eora_common.cuh).  Run once per layer inside eora_linear_create; not on the hot path.
#include "eora_common.cuh"

namespace eora {
namespace {

// b-bit code k of column n from an LSB-first stream along the rows of `words` (leading dim ld)
__device__ inline uint32_t src_code(const uint32_t* words, int bits, int k, int n, int ld) {
  int p = bits * k, i = p >> 5, off = p & 31;
  uint32_t v = words[(int64_t)i * ld + n] >> off;
  if (off + bits > 32) v |= words[(int64_t)(i + 1) * ld + n] << (32 - off);
  return v & ((1u << bits) - 1u);
}
// zero-point of (group row g, column n): the stream runs along n inside row g (ldz words per row)
__device__ inline uint32_t src_zero(const uint32_t* zeros, int bits, int g, int n, int ldz) {
  int p = bits * n, i = p >> 5, off = p & 31;
  const uint32_t* row = zeros + (int64_t)g * ldz;
  uint32_t v = row[i] >> off;
  if (off + bits > 32) v |= row[i + 1] << (32 - off);
  return v & ((1u << bits) - 1u);
}

struct Pos { int tile, c, lane, g, t; };
__device__ inline Pos pos_of(int64_t idx, int kc) {
  Pos p;
  p.lane = (int)(idx & 31);
  int64_t ti = idx >> 5;
  p.c = (int)(ti % kc);
  p.tile = (int)(ti / kc);
  p.g = p.lane >> 2;
  p.t = p.lane & 3;
  return p;
}

// code of (k, n) with padding: outside the source the code equals the zero-point (k) or 0 (n)
__device__ inline uint32_t padded_code(const uint32_t* codes, const uint32_t* zeros, int bits, int k, int n,
                                       int rows_src, int k_src, int group, int ldz) {
  if (n >= rows_src) return 0;
  if (k >= k_src) return src_zero(zeros, bits, (k_src - 1) / group, n, ldz);
  return src_code(codes, bits, k, n, rows_src);
}

__global__ void k_repack_q4(WMat d, int nt_sub, const uint32_t* codes, const uint32_t* zeros, int rows_src, int k_src, int ldz) {
  int64_t total = (int64_t)nt_sub * d.kc * 32;
  for (int64_t idx = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * blockDim.x) {
    Pos p = pos_of(idx, d.kc);
    uint32_t out[4];
    for (int part = 0; part < 4; ++part) {
      int n = p.tile * 16 + p.g + 8 * (part & 1);
      int k0 = p.c * 64 + (part >> 1) * 32 + 8 * p.t;
      uint32_t w = 0;
      for (int e = 0; e < 8; ++e)
        w |= padded_code(codes, zeros, 4, k0 + e, n, rows_src, k_src, d.group, ldz) << (4 * q4_nibble(e));
      out[part] = w;
    }
    reinterpret_cast<uint4*>(const_cast<uint8_t*>(wmat_tile(d, p.tile, p.c)))[p.lane] = make_uint4(out[0], out[1], out[2], out[3]);
  }
}

__global__ void k_repack_q3(WMat d, int nt_sub, const uint32_t* codes, const uint32_t* zeros, int rows_src, int k_src, int ldz) {
  int64_t total = (int64_t)nt_sub * d.kc * 32;
  for (int64_t idx = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * blockDim.x) {
    Pos p = pos_of(idx, d.kc);
    uint32_t wd[3] = {0, 0, 0};
    for (int part = 0; part < 4; ++part) {
      int n = p.tile * 16 + p.g + 8 * (part & 1);
      int k0 = p.c * 64 + (part >> 1) * 32 + 8 * p.t;
      for (int e = 0; e < 8; ++e) {
        uint32_t q = padded_code(codes, zeros, 3, k0 + e, n, rows_src, k_src, d.group, ldz);
        q3_put(wd, part, e, q);
      }
    }
    uint32_t* blob = reinterpret_cast<uint32_t*>(const_cast<uint8_t*>(wmat_tile(d, p.tile, p.c)));
    blob[p.lane * 2] = wd[0];
    blob[p.lane * 2 + 1] = wd[1];
    blob[64 + p.lane] = wd[2];
  }
}

__global__ void k_repack_q8(WMat d, int nt_sub, const uint8_t* codes, const uint8_t* zeros, int rows_src, int k_src) {
  int64_t total = (int64_t)nt_sub * d.kc * 32;
  for (int64_t idx = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * blockDim.x) {
    Pos p = pos_of(idx, d.kc);
    uint8_t* tb = const_cast<uint8_t*>(wmat_tile(d, p.tile, p.c));
    for (int part = 0; part < 4; ++part) {
      int n = p.tile * 16 + p.g + 8 * (part & 1);
      int k0 = p.c * 64 + (part >> 1) * 32 + 8 * p.t;
      uint32_t w2[2] = {0, 0};
      for (int e = 0; e < 8; ++e) {
        uint32_t q = 0;
        if (n < rows_src) q = (k0 + e < k_src) ? codes[(int64_t)(k0 + e) * rows_src + n] : zeros[n];
        w2[e >> 2] |= q << (8 * q8_byte(e & 3));
      }
      uint32_t* dst = reinterpret_cast<uint32_t*>(tb) + ((part >> 1) * 32 + p.lane) * 4;
      dst[2 * (part & 1)] = w2[0];
      dst[2 * (part & 1) + 1] = w2[1];
    }
  }
}

// src element (k, n) at src[k * rows_src + n]  ([reduction][rows] row-major, as A [K][r] and B [r][N])
__global__ void k_repack_f16(WMat d, int nt_sub, const __half* src, int rows_src, int k_src) {
  int64_t total = (int64_t)nt_sub * d.kc * 32;
  for (int64_t idx = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * blockDim.x) {
    Pos p = pos_of(idx, d.kc);
    uint8_t* tb = const_cast<uint8_t*>(wmat_tile(d, p.tile, p.c));
    for (int part = 0; part < 4; ++part) {
      int n = p.tile * 16 + p.g + 8 * (part & 1);
      int k0 = p.c * 64 + (part >> 1) * 32 + 8 * p.t;
      __half* dst = reinterpret_cast<__half*>(tb) + (part * 32 + p.lane) * 8;
      for (int e = 0; e < 8; ++e) {
        int k = k0 + e;
        dst[e] = (n < rows_src && k < k_src) ? src[(int64_t)k * rows_src + n] : __float2half(0.f);
      }
    }
  }
}

__global__ void k_repack_sp24(WMat d, int nt_sub, const __half* values, const uint32_t* meta, int rows_src, int k_src) {
  int64_t total = (int64_t)nt_sub * d.kc * 32;
  for (int64_t idx = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * blockDim.x) {
    Pos p = pos_of(idx, d.kc);
    uint8_t* tb = const_cast<uint8_t*>(wmat_tile(d, p.tile, p.c));
    uint32_t m = 0;
    for (int part = 0; part < 4; ++part) {
      int n = p.tile * 16 + p.g + 8 * (part & 1);
      int k0 = p.c * 64 + (part >> 1) * 32 + 8 * p.t;
      int j0 = k0 >> 2;   // first of the part's two quads
      __half* dst = reinterpret_cast<__half*>(tb) + ((part >> 1) * 32 + p.lane) * 8 + 4 * (part & 1);
      uint32_t mb = 0x44;  // positions (0,1) with zero values outside the source
      if (n < rows_src && k0 < k_src) {
        for (int i = 0; i < 4; ++i) dst[i] = values[(int64_t)n * (k_src / 2) + 2 * j0 + i];
        mb = (meta[(int64_t)n * (k_src / 32) + (j0 >> 3)] >> (4 * (j0 & 7))) & 255u;
      } else {
        for (int i = 0; i < 4; ++i) dst[i] = __float2half(0.f);
      }
      m |= mb << (8 * part);
    }
    reinterpret_cast<uint32_t*>(tb + 1024)[p.lane] = m;
  }
}

// 2:4 pattern with 4-bit kept values: `codes` is the 4-bit stream of the [k_src/2][rows_src] matrix of kept values.
__global__ void k_repack_sq4(WMat d, int nt_sub, const uint32_t* codes, const uint32_t* meta, int rows_src, int k_src) {
  int64_t total = (int64_t)nt_sub * d.kc * 32;
  for (int64_t idx = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * blockDim.x) {
    Pos p = pos_of(idx, d.kc);
    uint32_t* tb = reinterpret_cast<uint32_t*>(const_cast<uint8_t*>(wmat_tile(d, p.tile, p.c)));
    uint32_t m = 0, wd[2] = {0, 0};
    for (int part = 0; part < 4; ++part) {
      int n = p.tile * 16 + p.g + 8 * (part & 1);
      int k0 = p.c * 64 + (part >> 1) * 32 + 8 * p.t;
      int j0 = k0 >> 2;   // first of the part's two quads
      uint32_t mb = 0x44;  // rows past the source: positions (0,1); their scale entry is zero
      if (n < rows_src && k0 < k_src) {
        for (int i = 0; i < 4; ++i)
          wd[part >> 1] |= src_code(codes, 4, 2 * j0 + i, n, rows_src) << (4 * q4_nibble(4 * (part & 1) + i));
        mb = (meta[(int64_t)n * (k_src / 32) + (j0 >> 3)] >> (4 * (j0 & 7))) & 255u;
      }
      m |= mb << (8 * part);
    }
    tb[p.lane * 2] = wd[0];
    tb[p.lane * 2 + 1] = wd[1];
    tb[64 + p.lane] = m;
  }
}

// Scale entries.  scales fp16 [G][rows_src]; zeros packed stream.  One thread per (k-tile c, row tile, g);
// the entry of k-tile c is written once per blob (by the even tile when the pair shares one entry).
__global__ void k_repack_sz(WMat d, int nt_sub, const __half* scales, const uint32_t* zeros, int bits, int rows_src, int ldz,
                            int ng_src) {
  int total = nt_sub * d.kc * 8;
  for (int idx = blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += gridDim.x * blockDim.x) {
    int g = idx & 7, c = (idx >> 3) % d.kc, tile = (idx >> 3) / d.kc;
    if (!d.sz2 && (c & 1)) continue;
    int grp = (c * 64) / d.group;
    uint32_t s2 = 0, z2 = 0;
    for (int half = 0; half < 2; ++half) {
      int n = tile * 16 + g + 8 * half;
      uint32_t sb = 0, zb = 0;
      if (n < rows_src) {
        int gs = grp < ng_src ? grp : ng_src - 1;
        sb = __half_as_ushort(scales[(int64_t)gs * rows_src + n]);
        zb = src_zero(zeros, bits, gs, n, ldz);
      }
      s2 |= sb << (16 * half);
      z2 |= zb << (8 * half);
    }
    uint8_t* sz = const_cast<uint8_t*>(wmat_sz(d, tile, c));
    reinterpret_cast<uint32_t*>(sz)[g] = s2;
    reinterpret_cast<uint16_t*>(sz + 32)[g] = (uint16_t)z2;
  }
}

__global__ void k_repack_sz_q8(WMat d, int nt_sub, const __half* scales, const uint8_t* zeros, int rows_src) {
  int total = nt_sub * d.kc * 8;   // one group: every pair carries a copy
  for (int idx = blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += gridDim.x * blockDim.x) {
    int g = idx & 7, c = (idx >> 3) % d.kc, tile = (idx >> 3) / d.kc;
    if (!d.sz2 && (c & 1)) continue;
    uint32_t s2 = 0, z2 = 0;
    for (int half = 0; half < 2; ++half) {
      int n = tile * 16 + g + 8 * half;
      if (n < rows_src) {
        s2 |= (uint32_t)__half_as_ushort(scales[n]) << (16 * half);
        z2 |= (uint32_t)zeros[n] << (8 * half);
      }
    }
    uint8_t* sz = const_cast<uint8_t*>(wmat_sz(d, tile, c));
    reinterpret_cast<uint32_t*>(sz)[g] = s2;
    reinterpret_cast<uint16_t*>(sz + 32)[g] = (uint16_t)z2;
  }
}

inline int grid_for(int64_t total, int block) {
  int64_t g = (total + block - 1) / block;
  if (g > 148 * 16) g = 148 * 16;
  if (g < 1) g = 1;
  return (int)g;
}

}  // namespace

// All launchers fill the first nt_sub row tiles of `d` (nt_sub < 0: all of them).  To fill row tiles
// [t0, t0 + n) of a larger matrix pass a copy of its WMat whose q points at row tile t0 and nt_sub = n.
cudaError_t launch_repack_quant(const WMat& d, const void* codes, const void* scales, const void* zeros, int bits,
                                int rows_src, int k_src, cudaStream_t st, int nt_sub) {
  if (nt_sub < 0) nt_sub = d.nt;
  int64_t total = (int64_t)nt_sub * d.kc * 32;
  int ldz = bits * rows_src / 32;
  int ng_src = k_src / d.group;
  if (ng_src < 1) ng_src = 1;
  if (bits == 4)
    k_repack_q4<<<grid_for(total, 256), 256, 0, st>>>(d, nt_sub, (const uint32_t*)codes, (const uint32_t*)zeros, rows_src, k_src, ldz);
  else
    k_repack_q3<<<grid_for(total, 256), 256, 0, st>>>(d, nt_sub, (const uint32_t*)codes, (const uint32_t*)zeros, rows_src, k_src, ldz);
  k_repack_sz<<<grid_for((int64_t)nt_sub * d.kc * 8, 256), 256, 0, st>>>(d, nt_sub, (const __half*)scales, (const uint32_t*)zeros, bits,
                                                                        rows_src, ldz, ng_src);
  return cudaGetLastError();
}

cudaError_t launch_repack_q8(const WMat& d, const void* codes, const void* scales, const void* zeros, int rows_src,
                             int k_src, cudaStream_t st, int nt_sub) {
  if (nt_sub < 0) nt_sub = d.nt;
  int64_t total = (int64_t)nt_sub * d.kc * 32;
  k_repack_q8<<<grid_for(total, 256), 256, 0, st>>>(d, nt_sub, (const uint8_t*)codes, (const uint8_t*)zeros, rows_src, k_src);
  k_repack_sz_q8<<<grid_for((int64_t)nt_sub * d.kc * 8, 256), 256, 0, st>>>(d, nt_sub, (const __half*)scales, (const uint8_t*)zeros, rows_src);
  return cudaGetLastError();
}

cudaError_t launch_repack_f16(const WMat& d, const void* src, int rows_src, int k_src, cudaStream_t st, int nt_sub) {
  if (nt_sub < 0) nt_sub = d.nt;
  int64_t total = (int64_t)nt_sub * d.kc * 32;
  k_repack_f16<<<grid_for(total, 256), 256, 0, st>>>(d, nt_sub, (const __half*)src, rows_src, k_src);
  return cudaGetLastError();
}

cudaError_t launch_repack_sp24(const WMat& d, const void* values, const void* meta, int rows_src, int k_src,
                               cudaStream_t st, int nt_sub) {
  if (nt_sub < 0) nt_sub = d.nt;
  int64_t total = (int64_t)nt_sub * d.kc * 32;
  k_repack_sp24<<<grid_for(total, 256), 256, 0, st>>>(d, nt_sub, (const __half*)values, (const uint32_t*)meta, rows_src, k_src);
  return cudaGetLastError();
}

cudaError_t launch_repack_sq4(const WMat& d, const void* codes, const void* scales, const void* zeros, const void* meta,
                              int rows_src, int k_src, cudaStream_t st, int nt_sub) {
  if (nt_sub < 0) nt_sub = d.nt;
  int64_t total = (int64_t)nt_sub * d.kc * 32;
  int ldz = 4 * rows_src / 32;
  int ng_src = k_src / d.group;
  if (ng_src < 1) ng_src = 1;
  k_repack_sq4<<<grid_for(total, 256), 256, 0, st>>>(d, nt_sub, (const uint32_t*)codes, (const uint32_t*)meta, rows_src, k_src);
  k_repack_sz<<<grid_for((int64_t)nt_sub * d.kc * 8, 256), 256, 0, st>>>(d, nt_sub, (const __half*)scales, (const uint32_t*)zeros, 4,
                                                                        rows_src, ldz, ng_src);
  return cudaGetLastError();
}

}  // namespace eora
