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
//
// Blobs.  Two tiles that are neighbours along the reduction axis (k-tiles 2p and 2p+1, "pair" p: 128
// reduction elements) plus the scales and zero-points they need form one contiguous blob, and the
// blobs are ordered pair-major:  blob (p, tile) sits at  q + (p * nt + tile) * blob.  A run of consecutive
// blobs is therefore a set of row tiles that all multiply the same 128 activations, and it is one
// contiguous byte range that a single bulk copy brings into shared memory, scales included.
//   blob = [tile 2p][tile 2p+1][sz entry 0][sz entry 1 (only if sz2)]
//   sz entry (48 B) = 8 x half2 scales (s[n_a], s[n_b]) indexed by g, then 8 x u8x2 zero-points (z[n_a] | z[n_b] << 8).
//   If the group size is a multiple of 128 the pair has one entry (its group), otherwise (64, 192, ...)
//   one per tile (sz2).  Unquantised formats have no entries.
// Per format, the payload of lane L inside the tile:
//   Q4  : 512 B: one uint4 per lane; word `part` holds the 8 codes of that part, element e in nibble
//         (e & 1) * 4 + (e >> 1)   (so that (w & 0x000f000f) is the pair (e0, e1), ...).
//   Q3  : 384 B: three words; w0, w1 as a uint2 per lane in bytes [0, 256), w2 as one word per lane
//         in bytes [256, 384).  Byte-planar: for part p < 3, byte b of word p holds element b in bits
//         [0, 3) and element 4 + b in bits [3, 6), so that (w & 0x07070707) and ((w >> 3) & 0x07070707)
//         are the part's two quads of codes, one code per byte.  Part 3 lives in the spare bits: element
//         4*quad + b has its low two bits in bits [6, 8) of byte b of word `quad`, its high bit in bit
//         6 + quad of byte b of w2.
//   Q8  : 1024 B: two planes of one uint4 per lane (plane = part/2); words 2*(part%2) and 2*(part%2)+1
//         hold elements 0..3 and 4..7; inside a word element i sits in byte {0, 2, 1, 3}[i].
//   F16 : 2048 B: four planes of one uint4 per lane (plane = part), 8 fp16 in natural order.
//   SP24: 1152 B: values in two planes of one uint4 per lane (plane = part/2), the half (part%2) holds
//         the 4 kept fp16 values of the part's two quads; then one word per lane in bytes [1024, 1152),
//         byte `part` = nibble(quad0) | nibble(quad1)<<4.
//   SQ4 : 384 B (2:4 pattern, kept values as 4-bit codes): one uint2 per lane in bytes [0, 256): word blk
//         (= part/2) holds the 8 kept codes of parts 2*blk and 2*blk+1; kept value i (0..3: two per quad) of
//         the part with half = part%2 sits in nibble q4_nibble(4*half + i), so that (w >> 8*half) & 0x000f000f
//         is the pair kept by the part's first quad and the same with >> 4 more its second quad's.  Then the
//         position word of SP24 in bytes [256, 384).  Scale entries as for the quantised formats; a group
//         is counted along the original reduction axis.
// ---------------------------------------------------------------------------------------------
enum Fmt : int { FMT_NONE = 0, FMT_Q4 = 1, FMT_Q3 = 2, FMT_Q8 = 3, FMT_F16 = 4, FMT_SP24 = 5, FMT_SQ4 = 6 };

struct WMat {
  int fmt;
  int n_rows;      // padded to a multiple of 16
  int k_red;       // padded to a multiple of 128
  int group;       // quantisation group along the reduction axis (multiple of 64)
  int nt;          // n_rows / 16
  int kc;          // k_red / 64
  int np;          // k_red / 128: pairs of k-tiles
  int sz2;         // 1: one scale entry per tile, 0: one per pair
  int blob;        // bytes of one blob
  const uint8_t* q;      // blobs
};

constexpr int kSzEntryBytes = 48;

__host__ __device__ constexpr int tile_bytes(int fmt) {
  return fmt == FMT_Q4 ? 512 : fmt == FMT_Q3 ? 384 : fmt == FMT_Q8 ? 1024 : fmt == FMT_F16 ? 2048 : fmt == FMT_SP24 ? 1152
       : fmt == FMT_SQ4 ? 384 : 0;
}
// formats whose blobs carry scale / zero-point entries
__host__ __device__ constexpr bool fmt_quantised(int fmt) { return fmt == FMT_Q4 || fmt == FMT_Q3 || fmt == FMT_Q8 || fmt == FMT_SQ4; }
__host__ __device__ constexpr int blob_bytes(int fmt, int sz2) {
  return 2 * tile_bytes(fmt) + (fmt_quantised(fmt) ? (sz2 ? 2 : 1) * kSzEntryBytes : 0);
}
__host__ __device__ inline int64_t wmat_q_bytes(const WMat& w) { return (int64_t)w.np * w.nt * w.blob; }

// tile (row tile `tile`, k-tile c) and the scale entry that covers it
__host__ __device__ inline const uint8_t* wmat_blob(const WMat& w, int tile, int pair) {
  return w.q + ((int64_t)pair * w.nt + tile) * w.blob;
}
__host__ __device__ inline const uint8_t* wmat_tile(const WMat& w, int tile, int c) {
  return wmat_blob(w, tile, c >> 1) + (c & 1) * tile_bytes(w.fmt);
}
__host__ __device__ inline const uint8_t* wmat_sz(const WMat& w, int tile, int c) {
  return wmat_blob(w, tile, c >> 1) + 2 * tile_bytes(w.fmt) + (w.sz2 ? (c & 1) * kSzEntryBytes : 0);
}

// nibble / byte positions (shared by the repack kernels and the accessors below)
__host__ __device__ inline int q4_nibble(int e) { return (e & 1) * 4 + (e >> 1); }
__host__ __device__ inline int q8_byte(int i) { return (i == 1) ? 2 : (i == 2) ? 1 : i; }

// 3-bit code of element e of part `part` from the three words of a lane (see the Q3 layout above)
__host__ __device__ inline int q3_code(const uint32_t (&wd)[3], int part, int e) {
  const int quad = e >> 2, b = e & 3;
  if (part < 3) return (wd[part] >> (8 * b + 3 * quad)) & 7;
  return ((wd[quad] >> (8 * b + 6)) & 3) | (((wd[2] >> (8 * b + 6 + quad)) & 1) << 2);
}
// and the inverse: put code q there
__host__ __device__ inline void q3_put(uint32_t (&wd)[3], int part, int e, uint32_t q) {
  const int quad = e >> 2, b = e & 3;
  if (part < 3) {
    wd[part] |= q << (8 * b + 3 * quad);
  } else {
    wd[quad] |= (q & 3u) << (8 * b + 6);
    wd[2] |= ((q >> 2) & 1u) << (8 * b + 6 + quad);
  }
}

// Integer code of element (k, n) of a quantised WMat.
__device__ inline int wmat_code(const WMat& w, int k, int n) {
  int tile = n >> 4, g = n & 7, half = (n >> 3) & 1;
  int c = k >> 6, blk = (k >> 5) & 1, t = (k >> 3) & 3, e = k & 7;
  int lane = g * 4 + t, part = blk * 2 + half;
  const uint32_t* blob = reinterpret_cast<const uint32_t*>(wmat_tile(w, tile, c));
  if (w.fmt == FMT_Q4) {
    return (blob[lane * 4 + part] >> (4 * q4_nibble(e))) & 15;
  } else if (w.fmt == FMT_Q3) {
    uint32_t wd[3] = {blob[lane * 2], blob[lane * 2 + 1], blob[64 + lane]};
    return q3_code(wd, part, e);
  } else {  // FMT_Q8
    uint32_t wd = blob[(part >> 1) * 128 + lane * 4 + 2 * (part & 1) + (e >> 2)];
    return (wd >> (8 * q8_byte(e & 3))) & 255;
  }
}

// Kept value of a 2:4 quad that element e (0..7) of a part refers to: 2*quad + {0, 1}, or -1 if the position is pruned.
__host__ __device__ inline int sp24_kept(uint32_t meta_byte, int e) {
  const int quad = e >> 2, pos = e & 3;
  const uint32_t nib = (meta_byte >> (4 * quad)) & 15u;
  if (pos == (int)(nib & 3u)) return 2 * quad;
  if (pos == (int)(nib >> 2)) return 2 * quad + 1;
  return -1;
}

// Dequantised element (k, n) as fp32: exactly (float)(q - z) * (float)s for the quantised formats.
__device__ inline float wmat_elem(const WMat& w, int k, int n) {
  int tile = n >> 4, g = n & 7, half = (n >> 3) & 1;
  if (w.fmt == FMT_Q4 || w.fmt == FMT_Q3 || w.fmt == FMT_Q8 || w.fmt == FMT_SQ4) {
    int q;
    if (w.fmt == FMT_SQ4) {
      const int c = k >> 6, blk = (k >> 5) & 1, t = (k >> 3) & 3, lane = g * 4 + t, part = blk * 2 + half;
      const uint32_t* tb = reinterpret_cast<const uint32_t*>(wmat_tile(w, tile, c));
      const int i = sp24_kept((tb[64 + lane] >> (8 * part)) & 255u, k & 7);
      if (i < 0) return 0.f;
      q = (tb[lane * 2 + blk] >> (4 * q4_nibble(4 * half + i))) & 15;
    } else {
      q = wmat_code(w, k, n);
    }
    const uint8_t* sz = wmat_sz(w, tile, k >> 6);
    uint32_t s2 = reinterpret_cast<const uint32_t*>(sz)[g];
    uint32_t z2 = reinterpret_cast<const uint16_t*>(sz + 32)[g];
    float s = __half2float(__ushort_as_half((unsigned short)(half ? (s2 >> 16) : (s2 & 0xffff))));
    int z = half ? (int)(z2 >> 8) : (int)(z2 & 255);
    return (float)(q - z) * s;
  }
  int c = k >> 6, blk = (k >> 5) & 1, t = (k >> 3) & 3, e = k & 7;
  int lane = g * 4 + t, part = blk * 2 + half;
  const uint8_t* blob = wmat_tile(w, tile, c);
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
struct Handle {
  eora_linear_config cfg;
  int device;
  int r_pad;             // rank padded to a multiple of 128 (reduction length of B, row stride of t)
  WMat w, a, b;          // a: rows = rank (padded to 16); b: rows = d_out, reduction = r_pad
  void* weight_mem;      // one allocation holding all re-tiled payloads
  int64_t weight_bytes;
  void* scratch_mem;     // one allocation: t, partial sums, counters, staging
  int64_t scratch_bytes;
  float* t_gen;          // [max_m][r_pad] fp32, simple kernels only
  __half* t16;           // [max_m][r_pad] fp16 (prefill)
  float* d_t;            // [8][t_cols] fp32 sums of t (decode); zero between calls
  float* y_ws;           // [8][d_out] fp32 sums of y (decode); zero between calls
  uint32_t* counters;    // decode: [0] blobs of A done, [1] row tiles finished, [2 + tile] blobs of that row tile done
  int* dev_status;       // latched device status
  void* stage_mem;       // staging for the *_host entry points, allocated by the first such call (NULL until then)
  int64_t stage_bytes;
  void* x_stage;         // [max_m][d_in]
  void* y_stage;         // [max_m][d_out]
  unsigned long long wait_limit_ns;   // how long the kernels wait for t = X.A to be complete before they give up
  int sm_count;
  // Fused layers (several layers that read the same X, e.g. q/k/v): their backbones and B's are stacked
  // along the output axis (sub i owns row tiles [sub_tile0[i], sub_tile0[i+1])), their A's along the rank
  // axis (sub i owns columns [i * r_pad, (i+1) * r_pad) of t).  n_sub == 1 for a plain layer.
  int n_sub;
  int sub_tile0[5];
  int sub_dout[4];
  int t_cols;            // columns of t: n_sub * r_pad (or n_adapters * r_pad)
  // Several adapters for one backbone: their A's are stacked along the rank axis like those of fused layers,
  // their B's along the reduction axis (adapter j owns pairs [j * r_pad / 128, (j + 1) * r_pad / 128) of B).
  int n_adapters;        // 1 for a plain layer
  int multi;             // 1: created with per-token adapter selection (eora_linear_create_multi)
  void* prefill_state;   // owned by prefill.cu (tensor maps), may be NULL
  void* tc_state;        // owned by decode_tc.cu (its copy of the weights, scratch, work split), NULL if that family does not serve the handle
  void* trace;           // optional caller-owned timestamp buffer, may be NULL
};

// kernels / launchers implemented in the other translation units ------------------------------
cudaError_t launch_repack_quant(const WMat& dst, const void* codes, const void* scales, const void* zeros,
                                int bits, int rows_src, int k_src, cudaStream_t st, int nt_sub = -1);
cudaError_t launch_repack_q8(const WMat& dst, const void* codes, const void* scales, const void* zeros,
                             int rows_src, int k_src, cudaStream_t st, int nt_sub = -1);
cudaError_t launch_repack_f16(const WMat& dst, const void* src, int rows_src, int k_src, cudaStream_t st, int nt_sub = -1);
cudaError_t launch_repack_sp24(const WMat& dst, const void* values, const void* meta, int rows_src, int k_src,
                               cudaStream_t st, int nt_sub = -1);
cudaError_t launch_repack_sq4(const WMat& dst, const void* codes, const void* scales, const void* zeros, const void* meta,
                              int rows_src, int k_src, cudaStream_t st, int nt_sub = -1);
cudaError_t launch_dump(const Handle* h, int what, void* out, cudaStream_t st);
cudaError_t launch_generic_forward(const Handle* h, const void* x, int m, void* y, cudaStream_t st);
int generic_launch_count(const Handle* h);

bool decode_supported(const Handle* h, int m);
cudaError_t launch_decode_forward(const Handle* h, const void* x, int m, void* const* ys, cudaStream_t st,
                                  const int32_t* adapter_ids = nullptr);
int decode_launch_count(const Handle* h, int m);
int decode_grid(const Handle* h, int m);
cudaError_t launch_wait_selftest(const Handle* h, cudaStream_t st);

// tensor-memory decode family (decode_tc.cu)
cudaError_t decode_tc_init(Handle* h, cudaStream_t st);
void decode_tc_free(Handle* h);
bool decode_tc_supported(const Handle* h, int m);
cudaError_t launch_decode_tc_forward(const Handle* h, const void* x, int m, void* const* ys, cudaStream_t st);
int decode_tc_launch_count(const Handle* h, int m);
int decode_tc_grid(const Handle* h);
int64_t decode_tc_weight_bytes(const Handle* h);
int64_t decode_tc_scratch_bytes(const Handle* h);
cudaError_t decode_tc_reset(const Handle* h, cudaStream_t st);

bool prefill_supported(const Handle* h, int m);
cudaError_t prefill_init(Handle* h);
void prefill_free(Handle* h);
cudaError_t prefill_reset(Handle* h, cudaStream_t st);   // after a launch that gave up: split-K sums and tickets back to zero
cudaError_t launch_prefill_forward(const Handle* h, const void* x, int m, void* const* ys, cudaStream_t st);
int prefill_launch_count(const Handle* h, int m);

}  // namespace eora
