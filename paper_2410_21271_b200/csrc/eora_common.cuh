// Internal definitions shared by the kernels of libeora_linear: the re-tiled weight layout
// ("WMat"), its element accessors, and the handle.  Nothing here is visible through the C ABI.
#pragma once
#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include "../../include/eora_linear.h"

namespace eora {

// ---------------------------------------------------------------------------------------------
// WMat: a "weight-like" matrix with n_rows output rows and a reduction axis of length k_red,
// used for all three operands of Eq. 4:  the backbone (rows = d_out, reduction = d_in), A
// (rows = rank, reduction = d_in) and B (rows = d_out, reduction = rank).
//
// Tiling.  The matrix is cut into tiles of 16 rows x 64 reduction elements.  One tile is what a
// warp consumes per step with four mma.m16n8k16 (weights are the 16-row operand).  Inside a tile
// lane L = 4*g + t (g = L/4, t = L%4) owns rows n_a = 16*tile + g and n_b = n_a + 8 and the
// reduction elements ka = 64*c + 8*t + [0,8) and kb = ka + 32, i.e. four "parts"
//     part 0 = (n_a, ka)   part 1 = (n_b, ka)   part 2 = (n_a, kb)   part 3 = (n_b, kb)
// of 8 consecutive reduction elements each.  Eight consecutive elements of one row are also one
// 16-byte chunk of a K-major tensor-core operand, so the same layout feeds the prefill kernel.
// Tiles of one row-tile are contiguous along the reduction axis: index = tile * kc + c.
//
// Every tile is one contiguous blob of tile_bytes(fmt) bytes, so the tiles a CTA needs are one
// contiguous byte range that a single bulk copy can bring into shared memory.
// Per format, the payload of lane L inside the blob of tile (tile, c):
//   Q4  : 512 B: one uint4 per lane; word `part` holds the 8 codes of that part, element e in nibble
//         (e & 1) * 4 + (e >> 1)   (so that (w & 0x000f000f) is the pair (e0, e1), ...).
//   Q3  : 384 B: three words; w0, w1 as a uint2 per lane in bytes [0, 256), w2 as one word per lane
//         in bytes [256, 384).  The 32 codes form 16 pairs,
//         pair p = part*4 + e/2; for p < 15 the pair lives in word p/5, field f = p%5: the even
//         element in bits [3f, 3f+3), the odd one in bits [16+3f, 16+3f+3).  Pair 15 is spread
//         over the spare bits: bit i of the even element is bit 15 of word i, bit i of the odd
//         element is bit 31 of word i.
//   Q8  : 1024 B: two planes of one uint4 per lane (plane = part/2); words 2*(part%2) and 2*(part%2)+1
//         hold elements 0..3 and 4..7; inside a word element i sits in byte {0, 2, 1, 3}[i].
//   F16 : 2048 B: four planes of one uint4 per lane (plane = part), 8 fp16 in natural order.
//   SP24: 1152 B: values in two planes of one uint4 per lane (plane = part/2), the half (part%2) holds
//         the 4 kept fp16 values of the part's two quads; then one word per lane in bytes [1024, 1152),
//         byte `part` = nibble(quad0) | nibble(quad1)<<4.
// Scales / zero-points (Q4, Q3, Q8): sc[(tile*G + grp)*8 + g] = half2(s[n_a], s[n_b]),
//   zz[(tile*G + grp)*8 + g] = z[n_a] | z[n_b] << 8, with grp = k / group.
// ---------------------------------------------------------------------------------------------
enum Fmt : int { FMT_NONE = 0, FMT_Q4 = 1, FMT_Q3 = 2, FMT_Q8 = 3, FMT_F16 = 4, FMT_SP24 = 5 };

struct WMat {
  int fmt;
  int n_rows;      // padded to a multiple of 16
  int k_red;       // padded to a multiple of 64
  int group;       // quantisation group along the reduction axis (multiple of 64)
  int nt;          // n_rows / 16
  int kc;          // k_red / 64
  int ng;          // k_red / group
  const uint8_t* q;      // tile blobs
  const uint32_t* sc;    // half2 scales
  const uint16_t* zz;    // u8x2 zero-points
};

__host__ __device__ inline int tile_bytes(int fmt) {
  switch (fmt) {
    case FMT_Q4: return 512;
    case FMT_Q3: return 384;
    case FMT_Q8: return 1024;
    case FMT_F16: return 2048;
    case FMT_SP24: return 1152;
    default: return 0;
  }
}
__host__ __device__ inline int64_t wmat_q_bytes(int fmt, int nt, int kc) { return (int64_t)nt * kc * tile_bytes(fmt); }

// nibble / byte positions (shared by the repack kernels and the accessors below)
__host__ __device__ inline int q4_nibble(int e) { return (e & 1) * 4 + (e >> 1); }
__host__ __device__ inline int q8_byte(int i) { return (i == 1) ? 2 : (i == 2) ? 1 : i; }

// Integer code of element (k, n) of a quantised WMat.
__device__ inline int wmat_code(const WMat& w, int k, int n) {
  int tile = n >> 4, g = n & 7, half = (n >> 3) & 1;
  int c = k >> 6, blk = (k >> 5) & 1, t = (k >> 3) & 3, e = k & 7;
  int lane = g * 4 + t, part = blk * 2 + half;
  const uint32_t* blob = reinterpret_cast<const uint32_t*>(w.q + ((int64_t)tile * w.kc + c) * tile_bytes(w.fmt));
  if (w.fmt == FMT_Q4) {
    return (blob[lane * 4 + part] >> (4 * q4_nibble(e))) & 15;
  } else if (w.fmt == FMT_Q3) {
    uint32_t wd[3] = {blob[lane * 2], blob[lane * 2 + 1], blob[64 + lane]};
    int pr = part * 4 + (e >> 1), hi = (e & 1) * 16;
    if (pr < 15) return (wd[pr / 5] >> (3 * (pr % 5) + hi)) & 7;
    int b = 15 + hi;
    return ((wd[0] >> b) & 1) | (((wd[1] >> b) & 1) << 1) | (((wd[2] >> b) & 1) << 2);
  } else {  // FMT_Q8
    uint32_t wd = blob[(part >> 1) * 128 + lane * 4 + 2 * (part & 1) + (e >> 2)];
    return (wd >> (8 * q8_byte(e & 3))) & 255;
  }
}

// Dequantised element (k, n) as fp32: exactly (float)(q - z) * (float)s for the quantised formats.
__device__ inline float wmat_elem(const WMat& w, int k, int n) {
  int tile = n >> 4, g = n & 7, half = (n >> 3) & 1;
  if (w.fmt == FMT_Q4 || w.fmt == FMT_Q3 || w.fmt == FMT_Q8) {
    int q = wmat_code(w, k, n);
    int64_t si = ((int64_t)tile * w.ng + k / w.group) * 8 + g;
    uint32_t s2 = w.sc[si];
    uint32_t z2 = w.zz[si];
    float s = __half2float(__ushort_as_half((unsigned short)(half ? (s2 >> 16) : (s2 & 0xffff))));
    int z = half ? (int)(z2 >> 8) : (int)(z2 & 255);
    return (float)(q - z) * s;
  }
  int c = k >> 6, blk = (k >> 5) & 1, t = (k >> 3) & 3, e = k & 7;
  int lane = g * 4 + t, part = blk * 2 + half;
  const uint8_t* blob = w.q + ((int64_t)tile * w.kc + c) * tile_bytes(w.fmt);
  if (w.fmt == FMT_F16) {
    const __half* p = reinterpret_cast<const __half*>(blob) + (part * 32 + lane) * 8;
    return __half2float(p[e]);
  }
  // FMT_SP24
  const __half* v = reinterpret_cast<const __half*>(blob) + ((part >> 1) * 32 + lane) * 8 + 4 * (part & 1);
  uint32_t meta = (reinterpret_cast<const uint32_t*>(blob + 1024)[lane] >> (8 * part)) & 255;
  int quad = e >> 2, pos = e & 3;
  uint32_t nib = (meta >> (4 * quad)) & 15;
  int p0 = nib & 3, p1 = nib >> 2;
  if (pos == p0) return __half2float(v[2 * quad]);
  if (pos == p1) return __half2float(v[2 * quad + 1]);
  return 0.f;
}

// ---------------------------------------------------------------------------------------------
// Handle
// ---------------------------------------------------------------------------------------------
struct DecodePlan {      // launch shape of the decode kernel for this layer
  int a_split;           // A units: a.nt row-tiles x a_split reduction slices
  int w_split;           // backbone units: w.nt row-tiles x w_split reduction slices
  int a_units, w_units;
};

struct Handle {
  eora_linear_config cfg;
  int device;
  int r_pad;             // rank padded to a multiple of 64
  WMat w, a, b;          // b: rows = d_out, reduction = r_pad
  void* weight_mem;      // one allocation holding all re-tiled payloads
  int64_t weight_bytes;
  void* scratch_mem;     // one allocation: t, split-K sums, counters, staging
  int64_t scratch_bytes;
  float* t_ws;           // [max_m][r_pad] fp32 sums of the fast kernels; zero between calls
  float* t_gen;          // [max_m][r_pad] fp32, simple kernels only
  float* y_ws;           // [min(max_m,64)][d_out] fp32 split-K sums (decode)
  __half* t16;           // [max_m][r_pad] fp16 (prefill)
  uint32_t* counters;    // see decode.cu
  int* dev_status;       // latched device status
  void* x_stage;         // [max_m][d_in] staging for forward_host
  void* y_stage;         // [max_m][d_out]
  DecodePlan plan;
  int sm_count;
  void* prefill_state;   // owned by prefill.cu (tensor maps), may be NULL
  void* trace;           // optional caller-owned timestamp buffer (decode kernel), may be NULL
};

// kernels / launchers implemented in the other translation units ------------------------------
cudaError_t launch_repack_quant(const WMat& dst, const void* codes, const void* scales, const void* zeros,
                                int bits, int rows_src, int k_src, cudaStream_t st);
cudaError_t launch_repack_q8(const WMat& dst, const void* codes, const void* scales, const void* zeros,
                             int rows_src, int k_src, cudaStream_t st);
cudaError_t launch_repack_f16(const WMat& dst, const void* src, int rows_src, int k_src, cudaStream_t st);
cudaError_t launch_repack_sp24(const WMat& dst, const void* values, const void* meta, int rows_src, int k_src,
                               cudaStream_t st);
cudaError_t launch_dump(const Handle* h, int what, void* out, cudaStream_t st);
cudaError_t launch_generic_forward(const Handle* h, const void* x, int m, void* y, cudaStream_t st);
int generic_launch_count(const Handle* h);

bool decode_supported(const Handle* h, int m);
void decode_make_plan(Handle* h);
cudaError_t launch_decode_forward(const Handle* h, const void* x, int m, void* y, cudaStream_t st);
int decode_launch_count(const Handle* h, int m);
int decode_grid(const Handle* h, int m);
bool decode_stream_supported(const Handle* h, int m);
int decode_stream_grid(const Handle* h, int m);
cudaError_t launch_decode_stream(const Handle* h, const void* x, int m, void* y, cudaStream_t st);

bool prefill_supported(const Handle* h, int m);
cudaError_t prefill_init(Handle* h);
void prefill_free(Handle* h);
cudaError_t launch_prefill_forward(const Handle* h, const void* x, int m, void* y, cudaStream_t st);
int prefill_launch_count(const Handle* h, int m);

}  // namespace eora
