// Builds the TMat copy (tmat.cuh) of a matrix from its WMat (eora_common.cuh).  Runs once per layer inside
// eora_linear_create; not on the hot path.
#include "tmat.cuh"

namespace eora {
namespace {

// One thread per (unit, row).
__global__ void k_tmat_from_wmat(TMat d, WMat s) {
  const int64_t total = (int64_t)d.nt * d.nkb * 128;
  for (int64_t idx = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * blockDim.x) {
    const int row = (int)(idx & 127);
    const int64_t u = idx >> 7;
    const int j = (int)(u % d.nkb), T = (int)(u / d.nkb);
    const int n = T * 128 + row, k0 = j * d.ku;
    const bool live = n < s.n_rows;
    uint8_t* unit = d.q + u * d.unit;
    uint32_t w[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) w[i] = 0u;
    if (d.fmt == FMT_Q4) {
      for (int e = 0; e < 128 && live; ++e)
        w[e >> 3] |= (uint32_t)wmat_code(s, k0 + e, n) << (8 * (e & 3) + 4 * ((e >> 2) & 1));
    } else if (d.fmt == FMT_Q3) {
      for (int e = 0; e < 128 && live; ++e) {
        const uint32_t q = (uint32_t)wmat_code(s, k0 + e, n);
        const int b = e >> 5, c = e & 31;
        if (c < 24) {
          w[3 * b + (c >> 3)] |= q << (8 * (c & 3) + 3 * ((c >> 2) & 1));
        } else {
          const int by = c & 3, hi = (c >> 2) & 1;                 // hi = 0: codes 24..27, 1: codes 28..31
          w[3 * b + hi] |= (q & 3u) << (8 * by + 6);
          w[3 * b + 2] |= (q >> 2) << (8 * by + 6 + hi);
        }
      }
    } else if (d.fmt == FMT_Q8) {
      for (int e = 0; e < 64 && live; ++e) w[e >> 2] |= (uint32_t)wmat_code(s, k0 + e, n) << (8 * (e & 3));
    } else {   // FMT_F16
      for (int e = 0; e < 32 && live; ++e)
        w[e >> 1] |= (uint32_t)__half_as_ushort(__float2half_rn(wmat_elem(s, k0 + e, n))) << (16 * (e & 1));
    }
    const int pieces = tmat_pieces(d.fmt);
    for (int p = 0; p < pieces; ++p)
      reinterpret_cast<uint4*>(unit)[p * 128 + row] = make_uint4(w[4 * p], w[4 * p + 1], w[4 * p + 2], w[4 * p + 3]);
    if (tmat_quant(d.fmt)) {
      uint16_t sb = 0;
      uint8_t zb = 0;
      if (live) {
        const uint8_t* sz = wmat_sz(s, n >> 4, k0 >> 6);
        const int g = n & 7, half = (n >> 3) & 1;
        const uint32_t s2 = reinterpret_cast<const uint32_t*>(sz)[g];
        const uint32_t z2 = reinterpret_cast<const uint16_t*>(sz + 32)[g];
        sb = (uint16_t)(half ? (s2 >> 16) : (s2 & 0xffffu));
        zb = (uint8_t)(half ? (z2 >> 8) : (z2 & 255u));
      }
      reinterpret_cast<uint16_t*>(unit + pieces * 2048)[row] = sb;
      (unit + pieces * 2048 + 256)[row] = zb;
    }
  }
}

}  // namespace

cudaError_t launch_tmat_from_wmat(const TMat& dst, const WMat& src, cudaStream_t st) {
  const int64_t total = (int64_t)dst.nt * dst.nkb * 128;
  int64_t g = (total + 127) / 128;
  if (g > 148 * 32) g = 148 * 32;
  if (g < 1) g = 1;
  k_tmat_from_wmat<<<(int)g, 128, 0, st>>>(dst, src);
  return cudaGetLastError();
}

}  // namespace eora
