// TMat: the weight layout of the tensor-memory decode kernel (decode_tc.cu).
//
// Like a WMat (eora_common.cuh) a TMat is a "weight-like" matrix with n_rows output rows and a reduction axis
// k_red, used for all three operands of Eq. 4 (backbone: rows = d_out, reduction = d_in; A: rows = rank,
// reduction = d_in; B: rows = d_out, reduction = rank).  It is cut into UNITS of 128 rows x KU reduction
// elements; a unit is what one tcgen05.mma sequence consumes with the 128 rows as the lanes of tensor memory.
// Units of a row tile are consecutive along the reduction axis:  unit (T, j) sits at  q + (T * nkb + j) * unit.
// A contiguous run of units is therefore one row tile walked along K (then the next row tile), and it is one
// contiguous byte range, fetched with one bulk copy per unit.
//
// Inside a unit thread `row` (0..127) of the CTA owns row 128 * T + row: its packed reduction elements are
// `pieces` 16-byte pieces, piece p of row r at byte (p * 128 + r) * 16 (piece-major, so that the 32 lanes of a
// warp read 512 consecutive bytes per piece: no bank conflicts).  Quantised formats append the unit's scales
// (fp16 [128]) and zero-points (u8 [128]).
//
//   Q4  (KU = 128, 4 pieces): word i (0..15) of a row holds codes k = 8 i + b in the low nibble and k = 8 i + 4 + b
//        in the high nibble of byte b, so that  w & 0x0f0f0f0f  and  (w >> 4) & 0x0f0f0f0f  are two registers of
//        four consecutive codes, one per byte: the 8-bit tensor-core operand as it is stored to tensor memory.
//   Q3  (KU = 128, 3 pieces): four blocks of 32 codes in three words (w0, w1, w2) each; for i < 3 byte b of word i
//        holds code 8 i + b in bits [0, 3) and code 8 i + 4 + b in bits [3, 6); code 24 + b has its low two bits
//        in bits [6, 8) of byte b of w0 and its high bit in bit 6 of byte b of w2; code 28 + b has its low two
//        bits in bits [6, 8) of byte b of w1 and its high bit in bit 7 of byte b of w2.
//   Q8  (KU = 64, 4 pieces): the codes as bytes in natural order.
//   F16 (KU = 32, 4 pieces): the values in natural order.
#pragma once
#include "eora_common.cuh"

namespace eora {

struct TMat {
  int fmt;
  int n_rows;      // padded to a multiple of 128
  int k_red;       // padded to a multiple of ku
  int ku;          // reduction elements per unit
  int nt;          // n_rows / 128
  int nkb;         // k_red / ku
  int unit;        // bytes per unit
  uint8_t* q;
};

__host__ __device__ constexpr int tmat_ku(int fmt) { return fmt == FMT_Q8 ? 64 : fmt == FMT_F16 ? 32 : 128; }
__host__ __device__ constexpr int tmat_pieces(int fmt) { return fmt == FMT_Q3 ? 3 : 4; }
__host__ __device__ constexpr bool tmat_quant(int fmt) { return fmt == FMT_Q4 || fmt == FMT_Q3 || fmt == FMT_Q8; }
__host__ __device__ constexpr int tmat_unit_bytes(int fmt) { return tmat_pieces(fmt) * 2048 + (tmat_quant(fmt) ? 384 : 0); }
// 32-bit columns of tensor memory a unit's operand takes (8-bit: four elements per column, fp16: two)
__host__ __device__ constexpr int tmat_cols(int fmt) { return fmt == FMT_F16 ? 16 : fmt == FMT_Q8 ? 16 : 32; }
__host__ __device__ constexpr bool tmat_supported(int fmt) { return fmt == FMT_Q4 || fmt == FMT_Q3 || fmt == FMT_Q8 || fmt == FMT_F16; }

inline int64_t tmat_bytes(const TMat& t) { return (int64_t)t.nt * t.nkb * t.unit; }

// Fill `dst` (shape already set, q allocated) from the WMat `src` holding the same matrix.
cudaError_t launch_tmat_from_wmat(const TMat& dst, const WMat& src, cudaStream_t st);

}  // namespace eora
