// Decode path on the fifth-generation tensor core (m <= 16 tokens per launch): one kernel computes Eq. 4 for a layer,
//     Y = X . deq(Wq) + (X . A) . B,
// streaming every weight byte exactly once.
//
// Why the tensor core for a matrix-vector product.  Three-bit weights arrive from HBM at ~58 weights per cycle and
// SM; that leaves ~2 thread-instructions per weight, and any inner product on the ALUs (or on the legacy mma.sync)
// spends more than that.  Here the ALUs only unpack: a thread owns one output row of a 128-row tile, turns its
// packed codes into bytes (one and-or per four codes) and stores them to TENSOR MEMORY as the 128-row operand of
// tcgen05.mma (kind::i8), which reads that operand at full rate from there (from shared memory a 128-row operand
// is fetched at ~32 bytes per cycle, below the HBM rate).  The activations are the narrow operand in shared
// memory: per token two signed byte planes of a 16-bit block-fixed-point number (one power-of-two scale per token
// and 128 reduction elements, so the integer products are exact and one-hot inputs reproduce the weights bit for
// bit).  The accumulator (int32, exact) is read back once per 128 reduction elements and row, where zero-point and
// scale are applied in fp32:   y += s * sx * (sum q x - z * sum x).   fp16 adapters take the same route with
// kind::f16 (operand copied to tensor memory as it is; t = X.A enters the product with B as an fp16 high + low
// pair of columns, so it keeps fp32-like accuracy).
//
// Work decomposition.  The three matrices are stored as units of 128 rows x KU reduction elements (tmat.cuh).
// One CTA per SM; CTA c owns a contiguous run of units of A (first), of W and of B (last), dealt on the host so
// that all CTAs finish together.  Inside a run the units of one row tile are consecutive along K: the partial
// sums stay in registers and are added to the fp32 sums in global memory (red.add) once per row tile and CTA.
// A ticket per row tile tells the last contributor, which converts the sums, writes Y and restores the scratch.
// B needs all of t = X.A: the warps that prepare B's activations wait (bounded) on a counter the A owners raise;
// A owners never wait and have the lowest CTA indices.
//
// Warp roles (12 warps): 0..7 unpack + read back (two sets of four, alternating units; warp w serves the
// tensor-memory lanes 32 (w % 4) ..), 8 bulk copies (cp.async.bulk, one per unit, ring of slots), 9 issues the
// MMAs, 10..11 prepare the activation operand.  Everything is handed over through mbarriers; every wait is bounded.
//
// Programmatic dependent launch: the weight copies start before griddepcontrol.wait, i.e. while the previous
// kernel of the stream is still running (a CTA takes half an SM's shared memory and tensor memory, so the next
// launch's CTAs are resident beside the running ones); activations and scratch are touched only after it.
#include <cstring>
#include <new>
#include <type_traits>
#include <vector>
#include "decode_common.cuh"
#include "tmat.cuh"

namespace eora {
using namespace dec;
namespace {

constexpr int kSlotBytes = 8704;          // one ring slot = one unit (largest: Q4 / Q8, 8576 bytes)
constexpr int kConvWarps = 2;
constexpr int kMaxCtas = 148;
constexpr int kTmemCols = 256;
constexpr int kACols = 32;                // tensor-memory columns of one operand stage

enum { SEG_A = 0, SEG_W = 1, SEG_B = 2 };
enum { CNT_A_FLUSHED = 0, CNT_TILES_DONE = 1, CNT_TICKET0 = 2 };

struct CtaPlan { uint32_t a0, w0, b0, an_bn, wn; };   // first unit and number of units of the CTA's three runs

struct TcArgs {
  const uint8_t* q[3];                    // units of A, W, B
  uint32_t nkb[3];                        // units per row tile
  uint32_t nt_w;                          // row tiles (128 rows) of W and B
  const void* x;
  void* ys[4];
  uint32_t sub_tile0[5];                  // fused layers: layer i owns row tiles [sub_tile0[i], sub_tile0[i+1])
  int sub_dout[4];
  int n_sub;
  float* d_t;                             // [m][t_cols] sums of t, zero between launches
  float* y_ws;                            // [m][n_pad] sums of y, zero between launches
  uint32_t* counters;                     // [0] flushes of A done, [1] row tiles finished, [2 + T] tickets
  const uint32_t* targets;                // [T] tickets that complete row tile T
  int* dev_status;
  uint32_t a_flush_total;
  int m, d_in, t_cols, r_pad, n_pad, x_dtype, y_dtype;
  unsigned long long wait_ns;             // limit of the wait for t
  CtaPlan plan[kMaxCtas];
};

// ---------------------------------------------------------------------------------------------- PTX
// The MMAs of one unit of format FMT.  The issuing thread is what bounds a unit (a lone thread retires an instruction
// every ~9 cycles), so the sequence is a straight line whose operands are a register plus an immediate: d, a: tensor-
// memory addresses of the accumulator and of the weight operand; blo / bhi: the activation stage's descriptor.
template <bool I8, int K>
__device__ __forceinline__ void issue_one(uint32_t d, uint32_t a, uint32_t blo, uint32_t bhi, uint32_t idesc) {
  if constexpr (I8)
    asm volatile("{\n\t.reg .b64 bd;\n\t.reg .pred p;\n\tmov.b64 bd, {%2, %3};\n\tsetp.ne.b32 p, %5, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::i8 [%0], [%1], bd, %4, p;\n\t}"
                 ::"r"(d), "r"(a + 8 * K), "r"(blo + 2 * K), "r"(bhi), "r"(idesc), "n"(K > 0 ? 1 : 0) : "memory");
  else
    asm volatile("{\n\t.reg .b64 bd;\n\t.reg .pred p;\n\tmov.b64 bd, {%2, %3};\n\tsetp.ne.b32 p, %5, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], bd, %4, p;\n\t}"
                 ::"r"(d), "r"(a + 8 * K), "r"(blo + 2 * K), "r"(bhi), "r"(idesc), "n"(K > 0 ? 1 : 0) : "memory");
}
template <int FMT, int NCOL>
__device__ __forceinline__ void issue_unit(uint32_t d, uint32_t a, uint32_t blo, uint32_t bhi) {
  constexpr bool I8 = tmat_quant(FMT);
  constexpr uint32_t idesc = I8 ? ((2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(NCOL >> 3) << 17) | ((128u >> 4) << 24))
                                : ((1u << 4) | ((uint32_t)(NCOL >> 3) << 17) | ((128u >> 4) << 24));
  constexpr int N = tmat_cols(FMT) / 8;
  issue_one<I8, 0>(d, a, blo, bhi, idesc);
  issue_one<I8, 1>(d, a, blo, bhi, idesc);
  if constexpr (N > 2) { issue_one<I8, 2>(d, a, blo, bhi, idesc); issue_one<I8, 3>(d, a, blo, bhi, idesc); }
}
__device__ __forceinline__ void umma_commit_tc(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t* r) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
               ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]) : "memory");
}
__device__ __forceinline__ void tmem_ld2(uint32_t taddr, uint32_t* v) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x2.b32 {%0, %1}, [%2];" : "=r"(v[0]), "=r"(v[1]) : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* v) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
               : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
                 "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
               : "r"(taddr) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ uint32_t atom_add_acq_rel_tc(uint32_t* p, uint32_t v) {
  uint32_t old;
  asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(v) : "memory");
  return old;
}
__device__ __forceinline__ void st_shared_u32(uint32_t addr, uint32_t v) { asm volatile("st.shared.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory"); }
__device__ __forceinline__ void st_shared_u16(uint32_t addr, uint32_t v) { asm volatile("st.shared.u16 [%0], %1;" ::"r"(addr), "r"(v) : "memory"); }
__device__ __forceinline__ void st_shared_v4u(uint32_t addr, uint4 v) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

// K-major, 128-byte swizzle operand descriptor: rows of 128 B, 8-row groups 1024 B apart (the activation operand).
__device__ __forceinline__ uint64_t make_desc_tc(uint32_t addr) {
  const uint32_t lo = ((addr & 0x3FFFFu) >> 4) | (1u << 16);
  const uint32_t hi = (1024u >> 4) | (1u << 14) | (2u << 29);
  return ((uint64_t)hi << 32) | lo;
}
// byte offset of byte kb (0..127) of row n inside an activation stage (128-byte swizzle)
__device__ __forceinline__ uint32_t x_off(uint32_t n, uint32_t kb) {
  return (n >> 3) * 1024u + (n & 7u) * 128u + ((((kb >> 4) ^ (n & 7u)) << 4) | (kb & 15u));
}

// ---------------------------------------------------------------------------------------------- the run of a CTA
struct Run { uint32_t u0[3], n[3]; };

__device__ __forceinline__ uint32_t sel3(uint32_t s, uint32_t a, uint32_t b, uint32_t c) { return s == 0 ? a : s == 1 ? b : c; }

// The CTA's run as a table in shared memory, one word per unit: segment | k-block j << 2 | row tile T << 16, closed by
// an all-ones entry.  Every role walks the table; the serial roles (one warp or one thread each) cannot afford index
// arithmetic per unit.
constexpr int kMaxUnits = 511;
__device__ __forceinline__ uint32_t ent_seg(uint32_t e) { return e & 3u; }
__device__ __forceinline__ uint32_t ent_j(uint32_t e) { return (e >> 2) & 0x3fffu; }
__device__ __forceinline__ uint32_t ent_T(uint32_t e) { return e >> 16; }

constexpr int kRawSlots = 8;              // units whose raw activations are in flight (bulk copies)
constexpr int kRawBytes = 256;            // bytes per token and unit of the raw activations (128 fp16 / 32 fp32 of t / ...)
// stages of the activation operand (shared memory) and of the accumulator (tensor memory: 128 + XS * NCOL <= 256 columns)
__host__ __device__ constexpr int tc_ncol(int mt) { return mt <= 8 ? 16 : 32; }
__host__ __device__ constexpr int tc_xstages(int) { return 8; }
__host__ __device__ constexpr int tc_ring_slots(int mt) { return mt == 1 ? 9 : mt <= 8 ? 16 : 14; }   // one token: two CTAs per SM

struct Shared {
  uint64_t w_full[16], w_empty[16];       // weight ring: copy landed / unit consumed
  uint64_t x_full[8], x_empty[8];         // activation stage written / its unit's accumulator (and scales) read back by the four warps
  uint64_t mma_done[8];                   // per set: the MMAs of its unit are complete
  uint64_t a_full[8];                     // per set: its four warps have stored their quarters of the weight operand
  float2 xaux[8][16];                     // per stage and token: (scale of the fixed-point activations, their integer sum)
  uint32_t tab[kMaxUnits + 9];            // the run (see above)
  uint32_t tmem_base;
};

// ---------------------------------------------------------------------------------------------- unpack -> tensor memory
// Thread `rr` (its row of the unit) turns its packed pieces into operand registers and stores them to the stage.
template <int FMT>
__device__ __forceinline__ void unpack_store(const uint8_t* unit, int rr, uint32_t taddr) {
  const uint4* pc = reinterpret_cast<const uint4*>(unit) + rr;
  if constexpr (FMT == FMT_Q3) {
    const uint4 p0 = pc[0], p1 = pc[128], p2 = pc[256];
    const uint32_t w[12] = {p0.x, p0.y, p0.z, p0.w, p1.x, p1.y, p1.z, p1.w, p2.x, p2.y, p2.z, p2.w};
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      const uint32_t w0 = w[3 * b], w1 = w[3 * b + 1], w2 = w[3 * b + 2];
      uint32_t r[8];
      r[0] = w0 & 0x07070707u; r[1] = (w0 >> 3) & 0x07070707u;
      r[2] = w1 & 0x07070707u; r[3] = (w1 >> 3) & 0x07070707u;
      r[4] = w2 & 0x07070707u; r[5] = (w2 >> 3) & 0x07070707u;
      r[6] = and_or(w2 >> 4, 0x04040404u, (w0 >> 6) & 0x03030303u);
      r[7] = and_or(w2 >> 5, 0x04040404u, (w1 >> 6) & 0x03030303u);
      tmem_st8(taddr + 8 * b, r);
    }
  } else if constexpr (FMT == FMT_Q4) {
#pragma unroll
    for (int pz = 0; pz < 4; ++pz) {
      const uint4 v = pc[128 * pz];
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
      uint32_t r[8];
#pragma unroll
      for (int i = 0; i < 4; ++i) { r[2 * i] = w[i] & 0x0f0f0f0fu; r[2 * i + 1] = (w[i] >> 4) & 0x0f0f0f0fu; }
      tmem_st8(taddr + 8 * pz, r);
    }
  } else if constexpr (FMT == FMT_Q8) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const uint4 v0 = pc[256 * h], v1 = pc[256 * h + 128];
      const uint32_t r[8] = {v0.x ^ 0x80808080u, v0.y ^ 0x80808080u, v0.z ^ 0x80808080u, v0.w ^ 0x80808080u,
                             v1.x ^ 0x80808080u, v1.y ^ 0x80808080u, v1.z ^ 0x80808080u, v1.w ^ 0x80808080u};
      tmem_st8(taddr + 8 * h, r);
    }
  } else {   // FMT_F16
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const uint4 v0 = pc[256 * h], v1 = pc[256 * h + 128];
      const uint32_t r[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
      tmem_st8(taddr + 8 * h, r);
    }
  }
}

// (scale as fp32, zero-point) of row rr of a quantised unit; Q8 codes are stored minus 128, so is its zero-point
template <int FMT>
__device__ __forceinline__ void unit_sz(const uint8_t* unit, int rr, float& s, int& z) {
  if constexpr (tmat_quant(FMT)) {
    const uint8_t* sz = unit + tmat_pieces(FMT) * 2048;
    s = __half2float(__ushort_as_half(reinterpret_cast<const uint16_t*>(sz)[rr]));
    z = (int)sz[256 + rr] - (FMT == FMT_Q8 ? 128 : 0);
  } else {
    s = 1.f; z = 0;
  }
}

// ---------------------------------------------------------------------------------------------- activations
// Token m's values f[0..EL) of this lane (reduction elements EL * lane + e of the unit) -> two signed byte planes of
// v = round(f / 2^e) (rows 2m: low plane, 2m + 1: high plane; v = 256 * high + low), with 2^e the smallest power of
// two that keeps the largest magnitude of the unit's 128 (or 64) values at or below 32639 = 127 * 256 + 127.
// The low plane is the low byte of v as it is (a signed byte), the high plane is byte 1 of v + 128.
template <int EL>
__device__ __forceinline__ void fixed_point_rows(const float (&f)[EL], uint32_t stage, float2* aux, int m, int lane, uint32_t mask = 0xffffffffu) {
  float am = 0.f;
#pragma unroll
  for (int e = 0; e < EL; ++e) am = fmaxf(am, fabsf(f[e]));
  am = __uint_as_float(__reduce_max_sync(mask, __float_as_uint(am)));     // non-negative floats order like integers
  const uint32_t eb = __float_as_uint(am * 1.00396f) >> 23;          // biased exponent of a value just above the maximum
  const bool live = eb >= 15u && eb < 255u;
  const float inv = live ? __uint_as_float((268u - eb) << 23) : 0.f;  // 2^(14 - exponent)
  const float sx = live ? __uint_as_float((eb - 14u) << 23) : 0.f;    // 2^(exponent - 14)
  int v[EL];
  int sum = 0;
#pragma unroll
  for (int e = 0; e < EL; ++e) { v[e] = __float2int_rn(f[e] * inv); sum += v[e]; }
  uint32_t lo[(EL + 3) / 4], hi[(EL + 3) / 4];
  if constexpr (EL >= 4) {
#pragma unroll
    for (int w = 0; w < EL / 4; ++w) {
      lo[w] = prmt(prmt(v[4 * w], v[4 * w + 1], 0x0040u), prmt(v[4 * w + 2], v[4 * w + 3], 0x0040u), 0x5410u);
      hi[w] = prmt(prmt(v[4 * w] + 128, v[4 * w + 1] + 128, 0x0051u), prmt(v[4 * w + 2] + 128, v[4 * w + 3] + 128, 0x0051u), 0x5410u);
    }
  } else {
    lo[0] = prmt(v[0], v[1], 0x0040u);
    hi[0] = prmt(v[0] + 128, v[1] + 128, 0x0051u);
  }
  sum = __reduce_add_sync(mask, sum);
  // rows n = 2m and n + 1 share their 8-row group; byte kb = EL * lane of the row
  const uint32_t n = 2u * (uint32_t)m, kb = EL * lane, r7 = n & 7u;
  const uint32_t base = stage + (n >> 3) * 1024u + r7 * 128u + (kb & 15u);
  const uint32_t c = kb >> 4;
  if constexpr (EL == 8) {
    asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(base + ((c ^ r7) << 4)), "r"(lo[0]), "r"(lo[1]) : "memory");
    asm volatile("st.shared.v2.b32 [%0], {%1, %2};" ::"r"(base + 128u + ((c ^ (r7 + 1u)) << 4)), "r"(hi[0]), "r"(hi[1]) : "memory");
  } else if constexpr (EL == 4) {
    st_shared_u32(base + ((c ^ r7) << 4), lo[0]);
    st_shared_u32(base + 128u + ((c ^ (r7 + 1u)) << 4), hi[0]);
  } else {
    st_shared_u16(base + ((c ^ r7) << 4), lo[0]);
    st_shared_u16(base + 128u + ((c ^ (r7 + 1u)) << 4), hi[0]);
  }
  if (lane == 0) aux[m] = make_float2(sx, __int_as_float(sum));
}

__device__ __forceinline__ float2 h2_to_f2(uint32_t v, bool bf16) {
  if (bf16) return make_float2(__uint_as_float(v << 16), __uint_as_float(v & 0xffff0000u));
  return __half22float2(*reinterpret_cast<const __half2*>(&v));
}
__device__ __forceinline__ uint32_t bf2_to_h2_tc(uint32_t v) {
  const __half2 h = __floats2half2_rn(__uint_as_float(v << 16), __uint_as_float(v & 0xffff0000u));
  return *reinterpret_cast<const uint32_t*>(&h);
}

// Where the raw activations of unit (T, j) of a segment with format FMT come from (FROM_T: from t, else from X):
// bytes per token, and the address of token m's piece.
template <int FMT, bool FROM_T>
__device__ __forceinline__ uint32_t raw_bytes() { return FROM_T ? tmat_ku(FMT) * 4u : tmat_ku(FMT) * 2u; }
template <int FMT, bool FROM_T>
__device__ __forceinline__ const uint8_t* raw_src(const TcArgs& p, uint32_t T, uint32_t j, int m) {
  constexpr int KU = tmat_ku(FMT);
  if constexpr (FROM_T) {
    uint32_t sub = 0;
#pragma unroll
    for (int i = 1; i < 4; ++i)
      if (i < p.n_sub && T >= p.sub_tile0[i]) sub = i;
    return reinterpret_cast<const uint8_t*>(p.d_t + (size_t)m * p.t_cols + sub * (uint32_t)p.r_pad + j * KU);
  } else {
    return reinterpret_cast<const uint8_t*>(p.x) + ((size_t)m * p.d_in + j * KU) * 2;
  }
}

// Activation operand of one unit from the raw copy in this warp's ring.  The unit's tokens are dealt to the two converter
// warps by the parity of (unit index + token), `par` = this warp's parity; the warp's q-th token (m = 2q + par) sits at
// q * (bytes per token).  The rows of an fp16 A (64 bytes per token) are all written by the warp with par == 0: token m at m * 64.
template <int FMT, bool FROM_T>
__device__ __forceinline__ void convert_unit(const TcArgs& p, uint32_t stage, float2* aux, const uint8_t* raw, int par, int lane) {
  constexpr int KU = tmat_ku(FMT);
  const bool bf16 = p.x_dtype == EORA_X_BF16;
  if constexpr (tmat_quant(FMT)) {
    constexpr int EL = KU / 32;
    for (int m = par; m < p.m; m += 2) {
      float f[EL];
      const uint8_t* src = raw + (m >> 1) * raw_bytes<FMT, FROM_T>();
      if constexpr (FROM_T) {
        if constexpr (EL == 4) {
          const float4 u = reinterpret_cast<const float4*>(src)[lane];
          f[0] = u.x; f[1] = u.y; f[2] = u.z; f[3] = u.w;
        } else {
          const float2 u = reinterpret_cast<const float2*>(src)[lane];
          f[0] = u.x; f[1] = u.y;
        }
      } else {
        if constexpr (EL == 4) {
          const uint2 u = reinterpret_cast<const uint2*>(src)[lane];
          const float2 a = h2_to_f2(u.x, bf16), b = h2_to_f2(u.y, bf16);
          f[0] = a.x; f[1] = a.y; f[2] = b.x; f[3] = b.y;
        } else {
          const float2 a = h2_to_f2(reinterpret_cast<const uint32_t*>(src)[lane], bf16);
          f[0] = a.x; f[1] = a.y;
        }
      }
      fixed_point_rows<EL>(f, stage, aux, m, lane);
    }
  } else if constexpr (FROM_T) {
    // fp16 B: token m's 32 values of t as an fp16 high part (row 2m) and low part (row 2m + 1)
    for (int m = par; m < p.m; m += 2) {
      const float v = reinterpret_cast<const float*>(raw + (m >> 1) * raw_bytes<FMT, FROM_T>())[lane];
      const __half h = __float2half_rn(v);
      const __half l = __float2half_rn(v - __half2float(h));
      st_shared_u16(stage + x_off(2 * m, 2 * lane), __half_as_ushort(h));
      st_shared_u16(stage + x_off(2 * m + 1, 2 * lane), __half_as_ushort(l));
    }
  } else {
    // fp16 A: token m's 32 values of X (64 bytes) as row 2m (row 2m + 1 is not used); four lanes per token
    if (par == 0) {
      for (int m = lane >> 2; m < p.m; m += 8) {
        uint4 u = reinterpret_cast<const uint4*>(raw + m * raw_bytes<FMT, FROM_T>())[lane & 3];
        if (bf16) { u.x = bf2_to_h2_tc(u.x); u.y = bf2_to_h2_tc(u.y); u.z = bf2_to_h2_tc(u.z); u.w = bf2_to_h2_tc(u.w); }
        st_shared_v4u(stage + x_off(2 * m, 16 * (lane & 3)), u);
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------- read back
// Add the unit's contribution to the thread's sums.  v: accumulator columns of this row for the NT tokens from m0 on.
template <int FMT, bool FROM_T, int MT, int NT>
__device__ __forceinline__ void accumulate_unit(float (&acc)[MT], int m0, const uint32_t* v, const float2* aux, float s, int z, int m_live) {
#pragma unroll
  for (int i = 0; i < NT; ++i) {
    const int m = m0 + i;
    if (m < m_live) {
      if constexpr (tmat_quant(FMT)) {
        const float2 ax = aux[m];
        const int V = (int)v[2 * i + 1] * 256 + (int)v[2 * i];
        const float f = (float)(V - z * __float_as_int(ax.y));
        acc[m] = fmaf(f, s * ax.x, acc[m]);
      } else if constexpr (FROM_T) {
        acc[m] += __uint_as_float(v[2 * i]) + __uint_as_float(v[2 * i + 1]);
      } else {
        acc[m] += __uint_as_float(v[2 * i]);
      }
    }
  }
}

template <int NCOL>
__device__ __forceinline__ void tmem_ld_cols(uint32_t taddr, uint32_t* v) {
  if constexpr (NCOL == 2) tmem_ld2(taddr, v);
  else tmem_ld16(taddr, v);
}

// ---------------------------------------------------------------------------------------------- the kernel
// WF / ABF: formats of the backbone and of the adapter (FMT_NONE: no adapter).  MT: tokens the launch is compiled
// for (1, 8 or 16); the accumulator has NCOL = 16 columns (two per token) up to eight tokens, 32 above.
//
// Sets.  The worker warps form NS sets of four (one warp per quarter of the 128 tensor-memory lanes).  Set k takes
// units k, k + NS, ... of the CTA's run and does everything for a unit by itself, one step after the other: wait for the
// unit's bytes, unpack them into the set's own 32 columns of tensor memory, one thread (once all four have stored) issues the
// unit's MMAs into the set's own accumulator columns, all four warps wait for them, read their rows back and add them to
// their sums.  A unit therefore takes a set a long time (~1500 cycles, most of it latency), but the sets, and the sets of
// the next launch's CTA on the same SM, run side by side: throughput comes from the number of units in flight, not
// from a deep pipeline inside one unit, and there is no stage that every unit has to pass one at a time.
template <int MT> struct TcShape {
  static constexpr int NS = MT <= 8 ? 5 : 4;            // sets: NS * (32 + NCOL) columns of tensor memory <= 256
  static constexpr int kWorkers = 4 * NS;
  static constexpr int kThreads = (kWorkers + 1 + kConvWarps) * 32;
  static constexpr int kCtasPerSm = MT == 1 ? 2 : 1;    // one token: 40 registers per thread are enough, two CTAs fit
};

template <int WF, int ABF, int MT>
__global__ void __launch_bounds__(TcShape<MT>::kThreads, TcShape<MT>::kCtasPerSm) k_decode_tc(const __grid_constant__ TcArgs p) {
  constexpr int NS = TcShape<MT>::NS;
  constexpr int kThreads = TcShape<MT>::kThreads;
  constexpr int kWarpProd = 4 * NS, kWarpConv = 4 * NS + 1;
  constexpr int NCOL = tc_ncol(MT);
  constexpr int XS = 8;                                  // activation stages
  constexpr int kXStage = NCOL * 128;
  constexpr int RS = tc_ring_slots(MT);
  constexpr int kSetCols = kACols + NCOL;                // a set's columns: weight operand, then accumulator
  constexpr int kWarpRaw = MT == 1 ? 512 : ((MT + 1) / 2) * kRawBytes;   // one slot of a converter warp's ring of raw activations
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* xst = smem;                                  // XS activation stages (1024-byte aligned: swizzle anchor)
  uint8_t* ring = xst + XS * kXStage;                   // RS slots of packed weights
  uint8_t* rawr = ring + RS * kSlotBytes;               // per converter warp: kRawSlots slots of raw activations
  Shared& sh = *reinterpret_cast<Shared*>(rawr + kConvWarps * kRawSlots * kWarpRaw);

  asm volatile("griddepcontrol.launch_dependents;");
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  Run run;
  {
    const CtaPlan& pl = p.plan[blockIdx.x];
    run.u0[0] = pl.a0; run.u0[1] = pl.w0; run.u0[2] = pl.b0;
    run.n[0] = pl.an_bn & 0xffffu; run.n[1] = pl.wn; run.n[2] = pl.an_bn >> 16;
  }
  const uint32_t n_units = run.n[0] + run.n[1] + run.n[2];
  for (uint32_t i = threadIdx.x; i < n_units + NS + 1; i += kThreads) {
    uint32_t e = 0xffffffffu;                            // the table ends in NS + 1 all-ones entries
    if (i < n_units) {
      const uint32_t seg = i < run.n[0] ? 0u : i < run.n[0] + run.n[1] ? 1u : 2u;
      const uint32_t u = sel3(seg, run.u0[0] + i, run.u0[1] + (i - run.n[0]), run.u0[2] + (i - run.n[0] - run.n[1]));
      const uint32_t nkb = sel3(seg, p.nkb[0], p.nkb[1], p.nkb[2]);
      const uint32_t T = u / nkb;
      e = seg | ((u - T * nkb) << 2) | (T << 16);
    }
    sh.tab[i] = e;
  }
  if (threadIdx.x == 0) {
    for (int i = 0; i < RS; ++i) { mbar_init(sh.w_full + i, 1); mbar_init(sh.w_empty + i, 4); }
    for (int i = 0; i < XS; ++i) { mbar_init(sh.x_full + i, MT == 1 ? 1 : kConvWarps); mbar_init(sh.x_empty + i, 4); }
    for (int i = 0; i < NS; ++i) { mbar_init(sh.mma_done + i, 1); mbar_init(sh.a_full + i, 4); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == kWarpProd) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh.tmem_base)), "r"((uint32_t)kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = sh.tmem_base;
  const uint32_t* tab = sh.tab;

  if (warp == kWarpProd) {
    // ------------------------------------------------------------------ bulk copies of the weights: one unit per slot
    if (lane == 0) {
      uint32_t slot = 0, sph = 0;
      bool ok = true;
      for (uint32_t i = 0; i < n_units; ++i) {
        if (i >= (uint32_t)RS && !mbar_wait(sh.w_empty + slot, sph ^ 1u, p.dev_status)) { ok = false; break; }
        const uint32_t e = tab[i], seg = ent_seg(e);
        const uint32_t bytes = seg == SEG_W ? tmat_unit_bytes(WF) : tmat_unit_bytes(ABF);
        const uint8_t* src = seg == 0 ? p.q[0] : seg == 1 ? p.q[1] : p.q[2];
        src += ((size_t)ent_T(e) * sel3(seg, p.nkb[0], p.nkb[1], p.nkb[2]) + ent_j(e)) * bytes;
        mbar_expect_tx(sh.w_full + slot, bytes);
        bulk_g2s(ring + slot * kSlotBytes, src, bytes, sh.w_full + slot);
        if (++slot == (uint32_t)RS) { slot = 0; sph ^= 1u; }
      }
      if (!ok) {
        // a consumer gave up: wait (bounded) for the copies still in flight before the CTA may exit
        for (uint32_t s2 = 0; s2 < (uint32_t)RS; ++s2) mbar_wait(sh.w_full + s2, slot > s2 ? sph : sph ^ 1u, p.dev_status);
      }
    }
  } else if (warp >= kWarpConv) {
    // ------------------------------------------------------------------ activation operand
    const int cw = warp - kWarpConv;
    uint8_t* myraw = rawr + cw * (kRawSlots * kWarpRaw);
    asm volatile("griddepcontrol.wait;" ::: "memory");
    bool t_ready = false, ok = true;
    // t must be complete before B's activations are read.  ahead: only look (never wait for t ahead of time: the flushes
    // of A it waits for may be this CTA's own, behind units that still need this warp).  1: go on, 0: not yet, -1: gave up.
    auto t_check = [&](bool ahead) -> int {
      int rdy = 0;
      if (lane == 0) {
        if (ahead) rdy = ld_acquire(p.counters + CNT_A_FLUSHED) >= p.a_flush_total ? 1 : 0;
        else rdy = counter_wait(p.counters + CNT_A_FLUSHED, p.a_flush_total, p.dev_status, p.wait_ns) ? 1 : -1;
      }
      return __shfl_sync(0xffffffffu, rdy, 0);
    };
    auto wait_groups = [&](uint32_t pending) {               // all but the newest `pending` commit groups have landed
      switch (pending) {
        case 0: asm volatile("cp.async.wait_group 0;" ::: "memory"); break;
        case 1: asm volatile("cp.async.wait_group 1;" ::: "memory"); break;
        case 2: asm volatile("cp.async.wait_group 2;" ::: "memory"); break;
        case 3: asm volatile("cp.async.wait_group 3;" ::: "memory"); break;
        case 4: asm volatile("cp.async.wait_group 4;" ::: "memory"); break;
        case 5: asm volatile("cp.async.wait_group 5;" ::: "memory"); break;
        case 6: asm volatile("cp.async.wait_group 6;" ::: "memory"); break;
        default: asm volatile("cp.async.wait_group 7;" ::: "memory"); break;
      }
    };
    // stage i % XS may be rewritten once the set that used it for unit i - XS has read its accumulator (and scales) back
    auto stage_free = [&](uint32_t i) -> bool {
      return i < (uint32_t)XS || mbar_wait_warp(sh.x_empty + i % XS, ((i / XS) & 1u) ^ 1u, p.dev_status, lane);
    };
    if constexpr (MT == 1) {
      // One token.  The units are taken in PASSES: two consecutive units of the backbone (half a warp each, eight values
      // per lane) or one unit of another kind; the two warps alternate passes.  A warp fetches the raw activations of its
      // own passes kRawSlots of them ahead with one 16-byte cp.async per lane, which the same lane reads back later.
      const int half = lane >> 4, l16 = lane & 15;
      const uint32_t hmask = half ? 0xffff0000u : 0x0000ffffu;
      uint32_t ci = 0, cpn = 0;                              // conversion side: next unit, pass number
      uint32_t fi = 0, fpn = 0, fown = 0;                    // fetch side: next unit, pass number, own passes requested so far
      uint32_t cown = 0;                                     // own passes converted so far
      auto pass_len = [&](uint32_t i) -> uint32_t {
        return (ent_seg(tab[i]) == SEG_W && ent_seg(tab[i + 1]) == SEG_W) ? 2u : 1u;     // the table ends in all-ones entries
      };
      auto fetch_pass = [&](uint32_t i, uint32_t len, uint32_t slot) {
        const uint32_t dst = smem_u32(myraw + slot * kWarpRaw);
        if (len == 2) {
          const uint32_t e = tab[i + half];
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + lane * 16),
                       "l"(reinterpret_cast<const uint8_t*>(p.x) + ent_j(e) * (tmat_ku(WF) * 2) + l16 * 16) : "memory");
        } else {
          const uint32_t e = tab[i], seg = ent_seg(e);
          if (seg == SEG_W) {
            if (lane < 16) asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + lane * 16),
                                        "l"(raw_src<WF, false>(p, ent_T(e), ent_j(e), 0) + lane * 16) : "memory");
          } else if constexpr (ABF != FMT_NONE) {
            if (seg == SEG_A) {
              if (lane < (int)(raw_bytes<ABF, false>() / 16)) asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + lane * 16),
                                        "l"(raw_src<ABF, false>(p, ent_T(e), ent_j(e), 0) + lane * 16) : "memory");
            } else {
              if (lane < (int)(raw_bytes<ABF, true>() / 16)) asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + lane * 16),
                                        "l"(raw_src<ABF, true>(p, ent_T(e), ent_j(e), 0) + lane * 16) : "memory");
            }
          }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
      };
      while (ci < n_units && ok) {
        const uint32_t len = pass_len(ci);
        if ((int)(cpn & 1u) == cw) {
          // ---- fetch ahead: own passes up to kRawSlots beyond the one converted now
          while (fi < n_units && fown < cown + kRawSlots) {
            const uint32_t flen = pass_len(fi);
            if ((int)(fpn & 1u) == cw) {
              if constexpr (ABF != FMT_NONE) {
                if (ent_seg(tab[fi]) == SEG_B && !t_ready) {
                  const int rdy = t_check(fi > ci);
                  if (rdy < 0) { ok = false; break; }
                  if (rdy == 0) break;
                  t_ready = true;
                }
              }
              fetch_pass(fi, flen, fown % kRawSlots);
              ++fown;
            }
            fi += flen; ++fpn;
          }
          if (!ok) break;
          wait_groups(fown - 1 - cown);
          __syncwarp();
          // ---- convert this pass
          const uint8_t* raw = myraw + (cown % kRawSlots) * kWarpRaw;
          const uint32_t i0 = ci + (len == 2 ? (uint32_t)half : 0u);
          const uint32_t sx = i0 % XS;
          if (len == 2) {
            if (!stage_free(ci) || !stage_free(ci + 1)) break;
            const uint4 u = reinterpret_cast<const uint4*>(raw)[lane];
            const bool bf16 = p.x_dtype == EORA_X_BF16;
            const float2 a = h2_to_f2(u.x, bf16), b = h2_to_f2(u.y, bf16), c2 = h2_to_f2(u.z, bf16), d2 = h2_to_f2(u.w, bf16);
            const float f[8] = {a.x, a.y, b.x, b.y, c2.x, c2.y, d2.x, d2.y};
            fixed_point_rows<8>(f, smem_u32(xst + sx * kXStage), sh.xaux[sx], 0, l16, hmask);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (l16 == 0) mbar_arrive(sh.x_full + sx);
          } else {
            if (!stage_free(ci)) break;
            const uint32_t stage = smem_u32(xst + sx * kXStage);
            const uint32_t seg = ent_seg(tab[ci]);
            if (seg == SEG_W) convert_unit<WF, false>(p, stage, sh.xaux[sx], raw, 0, lane);
            else if constexpr (ABF != FMT_NONE) {
              if (seg == SEG_A) convert_unit<ABF, false>(p, stage, sh.xaux[sx], raw, 0, lane);
              else convert_unit<ABF, true>(p, stage, sh.xaux[sx], raw, 0, lane);
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(sh.x_full + sx);
          }
          ++cown;
        }
        ci += len; ++cpn;
      }
    } else {
      // Several tokens.  Tokens of unit i are dealt to the two warps by the parity of (i + token).  A warp fetches the raw
      // activations of ITS tokens for the next kRawSlots units with 16-byte cp.async into a ring of its own (the latency of
      // global memory would otherwise be paid once per unit), one commit group per unit.
      uint32_t pf = 0;
      auto request = [&](uint32_t u) {
        const uint32_t e = tab[u], seg = ent_seg(e), T = ent_T(e), j = ent_j(e);
        const int par = (cw + (int)u) & 1;
        const uint32_t dst0 = smem_u32(myraw + (u % kRawSlots) * kWarpRaw);
        auto fetch = [&](auto fmt_tag, auto from_t_tag, bool all_tokens) {
          constexpr int FMT = decltype(fmt_tag)::value;
          constexpr bool FROM_T = decltype(from_t_tag)::value;
          constexpr int pieces = (FROM_T ? tmat_ku(FMT) * 4 : tmat_ku(FMT) * 2) / 16;     // 16-byte pieces per token
          constexpr int tpi = 32 / pieces;                                                  // tokens per instruction
          const int piece = lane % pieces, sub = lane / pieces;
          if (all_tokens) {
            if (par == 0)
              for (int m = sub; m < p.m; m += tpi)
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst0 + m * (pieces * 16) + piece * 16),
                             "l"(raw_src<FMT, FROM_T>(p, T, j, m) + piece * 16) : "memory");
          } else {
            for (int q = sub; 2 * q + par < p.m; q += tpi)
              asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst0 + q * (pieces * 16) + piece * 16),
                           "l"(raw_src<FMT, FROM_T>(p, T, j, 2 * q + par) + piece * 16) : "memory");
          }
        };
        if (seg == SEG_W) fetch(std::integral_constant<int, WF>{}, std::false_type{}, false);
        else if constexpr (ABF != FMT_NONE) {
          if (seg == SEG_A) fetch(std::integral_constant<int, ABF>{}, std::false_type{}, !tmat_quant(ABF));
          else fetch(std::integral_constant<int, ABF>{}, std::true_type{}, false);
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
      };
      for (uint32_t i = 0; i < n_units && ok; ++i) {
        while (pf < n_units && pf < i + kRawSlots) {
          if constexpr (ABF != FMT_NONE) {
            if (ent_seg(tab[pf]) == SEG_B && !t_ready) {
              const int rdy = t_check(pf > i);
              if (rdy < 0) { ok = false; break; }
              if (rdy == 0) break;
              t_ready = true;
            }
          }
          request(pf);
          ++pf;
        }
        if (!ok) break;
        const uint32_t sx = i % XS;
        wait_groups(pf - 1 - i);
        __syncwarp();
        if (!stage_free(i)) break;
        const uint32_t stage = smem_u32(xst + sx * kXStage);
        const uint8_t* raw = myraw + (i % kRawSlots) * kWarpRaw;
        const int par = (cw + (int)i) & 1;
        const uint32_t seg = ent_seg(tab[i]);
        if (seg == SEG_W) {
          convert_unit<WF, false>(p, stage, sh.xaux[sx], raw, par, lane);
        } else if constexpr (ABF != FMT_NONE) {
          if (seg == SEG_A) convert_unit<ABF, false>(p, stage, sh.xaux[sx], raw, par, lane);
          else convert_unit<ABF, true>(p, stage, sh.xaux[sx], raw, par, lane);
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(sh.x_full + sx);
      }
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");   // nothing of this warp is in flight when the CTA exits
  } else {
    // ------------------------------------------------------------------ workers
    // A warp never meets a warp of another set: it adds its 32 rows' sums to global memory when its set's units leave a
    // (segment, row tile), takes its own ticket for that row tile one unit later (the release in front of the ticket then
    // finds the adds already performed) and looks at the ticket's answer another unit later.
    const int set = warp >> 2, quad = warp & 3;
    const int rr = quad * 32 + lane;                      // this thread's row of every unit
    const uint32_t lane_base = tmem + ((uint32_t)(quad * 32) << 16) + set * kSetCols;
    const uint64_t bdesc0 = make_desc_tc(smem_u32(xst));
    const uint32_t blo0 = (uint32_t)bdesc0, bhi = (uint32_t)(bdesc0 >> 32);
    float acc[MT];
#pragma unroll
    for (int m = 0; m < MT; ++m) acc[m] = 0.f;
    bool ok = true, dep_waited = false;
    // ticket state: 0 nothing pending, 1 sums of (tk_seg, tk_T) are out and its ticket is still to be taken, 2 ticket taken, answer in tk_old
    uint32_t tk_state = 0, tk_seg = 0, tk_T = 0, tk_old = 0, tk_target = 0;

    // Row tile T is complete (this warp's ticket was the last): convert its sums, write Y, put the scratch back.
    auto finish_tile = [&](uint32_t T) {
      void* y = p.ys[0];
      uint32_t tile0 = 0;
      int dout = p.sub_dout[0];
#pragma unroll
      for (int i = 1; i < 4; ++i)
        if (i < p.n_sub && T >= p.sub_tile0[i]) { y = p.ys[i]; tile0 = p.sub_tile0[i]; dout = p.sub_dout[i]; }
      for (int m = 0; m < p.m; ++m) {
        float* sp = p.y_ws + (size_t)m * p.n_pad + T * 128 + lane;
        float v[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) v[q] = ld_cg(sp + 32 * q);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          sp[32 * q] = 0.f;
          const int n = (int)(T - tile0) * 128 + 32 * q + lane;
          if (n < dout) {
            const int64_t o = (int64_t)m * dout + n;
            if (p.y_dtype == EORA_Y_F32) reinterpret_cast<float*>(y)[o] = v[q];
            else if (p.y_dtype == EORA_Y_F16) reinterpret_cast<__half*>(y)[o] = __float2half_rn(v[q]);
            else reinterpret_cast<__nv_bfloat16*>(y)[o] = __float2bfloat16_rn(v[q]);
          }
        }
      }
      if (lane == 0) p.counters[CNT_TICKET0 + T] = 0u;
      if constexpr (ABF != FMT_NONE) {
        // count the finished row tiles: the last one restores t and the counters (nobody reads t any more)
        uint32_t last = 0;
        if (lane == 0) last = atom_add_acq_rel_tc(p.counters + CNT_TILES_DONE, 1u) + 1u == p.nt_w ? 1u : 0u;
        last = __shfl_sync(0xffffffffu, last, 0);
        if (last) {
          for (int i = lane; i < p.m * p.t_cols; i += 32) p.d_t[i] = 0.f;
          if (lane == 0) { p.counters[CNT_A_FLUSHED] = 0u; p.counters[CNT_TILES_DONE] = 0u; }
        }
      }
    };
    auto take_ticket = [&]() {                               // state 1 -> 2 (or 0 for a flush of A, which only counts)
      __syncwarp();                                          // the lanes' adds are ordered before lane 0's release
      if (lane == 0 && ok) {
        if (tk_seg == SEG_A) {
          asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p.counters + CNT_A_FLUSHED), "r"(1u) : "memory");
        } else {
          tk_target = p.targets[tk_T];
          tk_old = atom_add_acq_rel_tc(p.counters + CNT_TICKET0 + tk_T, 1u);
        }
      }
      tk_state = tk_seg == SEG_A ? 0u : 2u;
    };
    auto resolve_ticket = [&]() {                            // state 2 -> 0
      uint32_t fin = 0;
      if (lane == 0 && ok) fin = tk_old + 1u == tk_target ? 1u : 0u;
      fin = __shfl_sync(0xffffffffu, fin, 0);
      if (fin) finish_tile(tk_T);
      tk_state = 0;
    };

    uint32_t own = 0;                                        // units this set has done: parity of its MMA barrier
    for (uint32_t i = set; i < n_units; i += NS, ++own) {
      const uint32_t e = tab[i], seg = ent_seg(e);
      const uint32_t slot = i % RS, sph = (i / RS) & 1u, sx = i % XS, px = (i / XS) & 1u;
      // tickets move one step per unit of this warp
      if (tk_state == 2) resolve_ticket();
      else if (tk_state == 1) take_ticket();
      // ---- the unit's bytes -> the set's weight operand in tensor memory
      float sc = 0.f;
      int zz = 0;
      if (ok) ok = mbar_wait_warp_fast(sh.w_full + slot, sph, p.dev_status, lane);
      if (ok) {
        const uint8_t* unit = ring + slot * kSlotBytes;
        if (seg == SEG_W) { unpack_store<WF>(unit, rr, lane_base); unit_sz<WF>(unit, rr, sc, zz); }
        else if constexpr (ABF != FMT_NONE) { unpack_store<ABF>(unit, rr, lane_base); unit_sz<ABF>(unit, rr, sc, zz); }
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
        if (lane == 0) { mbar_arrive(sh.a_full + set); mbar_arrive(sh.w_empty + slot); }
      }
      // ---- one thread of the set issues the unit's MMAs once the four quarters are stored and the activations are there
      if (quad == 0 && lane == 0 && ok) {
        if (mbar_wait(sh.a_full + set, own & 1u, p.dev_status) && mbar_wait(sh.x_full + sx, px, p.dev_status)) {
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t a = tmem + set * kSetCols, d = a + kACols, blo = blo0 + sx * (kXStage >> 4);
          if (seg == SEG_W) issue_unit<WF, NCOL>(d, a, blo, bhi);
          else if constexpr (ABF != FMT_NONE) issue_unit<ABF, NCOL>(d, a, blo, bhi);
          umma_commit_tc(sh.mma_done + set);
        }
      }
      // ---- read the rows back
      __syncwarp();                                          // the issuing lane is back
      if (ok) ok = mbar_wait_warp_fast(sh.mma_done + set, own & 1u, p.dev_status, lane);
      if (ok) ok = mbar_wait(sh.x_full + sx, px, p.dev_status);     // complete: this thread's acquire of the stage's scales
      if (ok) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const float2* aux = sh.xaux[sx];
#pragma unroll
        for (int m0 = 0; m0 < MT; m0 += 8) {                   // eight tokens (sixteen columns) at a time
          constexpr int NT = MT < 8 ? MT : 8;
          uint32_t v[2 * NT];
          tmem_ld_cols<2 * NT>(lane_base + kACols + 2 * m0, v);
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
          if (seg == SEG_W) accumulate_unit<WF, false, MT, NT>(acc, m0, v, aux, sc, zz, p.m);
          else if constexpr (ABF != FMT_NONE) {
            if (seg == SEG_A) accumulate_unit<ABF, false, MT, NT>(acc, m0, v, aux, sc, zz, p.m);
            else accumulate_unit<ABF, true, MT, NT>(acc, m0, v, aux, sc, zz, p.m);
          }
        }
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        __syncwarp();
        if (lane == 0) mbar_arrive(sh.x_empty + sx);
      }
      // ---- the set's next unit belongs to another (segment, row tile), or there is none: the sums go out
      if ((e ^ tab[i + NS]) & 0xffff0003u) {
        if (!dep_waited) { asm volatile("griddepcontrol.wait;" ::: "memory"); dep_waited = true; }
        if (tk_state == 1) take_ticket();
        if (tk_state == 2) resolve_ticket();
        if (ok) {
          const uint32_t T = ent_T(e);
          float* dst = seg == SEG_A ? p.d_t + T * 128 + rr : p.y_ws + T * 128 + rr;
          const size_t ld = seg == SEG_A ? (size_t)p.t_cols : (size_t)p.n_pad;
#pragma unroll
          for (int m = 0; m < MT; ++m)
            if (m < p.m) red_add(dst + m * ld, acc[m]);
        }
#pragma unroll
        for (int m = 0; m < MT; ++m) acc[m] = 0.f;
        tk_state = 1; tk_seg = seg; tk_T = ent_T(e);
      }
    }
    // the last tickets
    if (tk_state == 1) take_ticket();
    if (tk_state == 2) resolve_ticket();
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == kWarpProd) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)kTmemCols) : "memory");
}

template <int WF, int ABF, int MT>
cudaError_t launch_tc_kernel(const cudaLaunchConfig_t& cfg, const TcArgs& args, int device) {
  static bool attr_set[64] = {};          // the attribute belongs to the device that is current at the call
  if (device < 0 || device >= 64) return cudaErrorInvalidDevice;
  if (!attr_set[device]) {
    cudaError_t e = cudaFuncSetAttribute(k_decode_tc<WF, ABF, MT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)cfg.dynamicSmemBytes);
    if (e != cudaSuccess) return e;
    attr_set[device] = true;
  }
  return cudaLaunchKernelEx(&cfg, k_decode_tc<WF, ABF, MT>, args);
}

template <int WF, int ABF>
cudaError_t launch_tc_mt(const cudaLaunchConfig_t& cfg, const TcArgs& args, int device, int mt) {
  if (mt == 1) return launch_tc_kernel<WF, ABF, 1>(cfg, args, device);
  if (mt == 8) return launch_tc_kernel<WF, ABF, 8>(cfg, args, device);
  return launch_tc_kernel<WF, ABF, 16>(cfg, args, device);
}
template <int WF>
cudaError_t launch_tc_ab(const cudaLaunchConfig_t& cfg, const TcArgs& args, int device, int mt, int abf) {
  switch (abf) {
    case FMT_F16: return launch_tc_mt<WF, FMT_F16>(cfg, args, device, mt);
    default: return launch_tc_mt<WF, FMT_NONE>(cfg, args, device, mt);
  }
}

int tc_smem_bytes(int mt) {
  return 1024 + tc_xstages(mt) * tc_ncol(mt) * 128 + tc_ring_slots(mt) * kSlotBytes + kConvWarps * kRawSlots * (mt == 1 ? 512 : ((mt + 1) / 2) * kRawBytes) + (int)sizeof(Shared);
}

void tmat_shape(TMat& t, int fmt, const WMat& src) {
  t.fmt = fmt;
  t.ku = tmat_ku(fmt);
  t.n_rows = (src.n_rows + 127) / 128 * 128;
  t.k_red = src.k_red;
  t.nt = t.n_rows / 128;
  t.nkb = t.k_red / t.ku;
  t.unit = tmat_unit_bytes(fmt);
  t.q = nullptr;
}

}  // namespace

// Per-handle state of this kernel family (owned through Handle::tc_state).
struct TcState {
  TMat w, a, b;
  void* weight_mem;
  int64_t weight_bytes;
  void* scratch_mem;           // d_t, y_ws, counters (zero between launches), targets (constant)
  int64_t scratch_bytes, zero_bytes;
  float* d_t; float* y_ws; uint32_t* counters;
  uint32_t* targets[2];        // tickets per row tile, for CTAs of five and of four sets
  int grid;
  uint32_t a_flush_total[2];
  CtaPlan plan[kMaxCtas];
};

constexpr int kTcMaxTokens = 16;

static bool tc_formats_ok(const Handle* h) {
  if (h->w.fmt != FMT_Q4 && h->w.fmt != FMT_Q3) return false;
  if (h->w.group % 128) return false;
  if (h->cfg.rank > 0 && h->a.fmt != FMT_F16) return false;
  if (h->multi) return false;
  for (int i = 0; i < h->n_sub; ++i)
    if (h->n_sub > 1 && h->sub_dout[i] % 128) return false;
  return true;
}

bool decode_tc_supported(const Handle* h, int m) { return h->tc_state != nullptr && m >= 1 && m <= 64; }
int decode_tc_launch_count(const Handle*, int m) { return (m + kTcMaxTokens - 1) / kTcMaxTokens; }
int decode_tc_grid(const Handle* h) { return h->tc_state ? reinterpret_cast<const TcState*>(h->tc_state)->grid : 0; }
int64_t decode_tc_weight_bytes(const Handle* h) { return h->tc_state ? reinterpret_cast<const TcState*>(h->tc_state)->weight_bytes : 0; }
int64_t decode_tc_scratch_bytes(const Handle* h) { return h->tc_state ? reinterpret_cast<const TcState*>(h->tc_state)->scratch_bytes : 0; }

void decode_tc_free(Handle* h) {
  TcState* t = reinterpret_cast<TcState*>(h->tc_state);
  if (!t) return;
  if (t->weight_mem) cudaFree(t->weight_mem);
  if (t->scratch_mem) cudaFree(t->scratch_mem);
  delete t;
  h->tc_state = nullptr;
}

// Put the scratch back to its between-launches state (after a device-side wait ran out).
cudaError_t decode_tc_reset(const Handle* h, cudaStream_t st) {
  const TcState* t = reinterpret_cast<const TcState*>(h->tc_state);
  if (!t) return cudaSuccess;
  return cudaMemsetAsync(t->scratch_mem, 0, (size_t)t->zero_bytes, st);
}

// Deal the units to the CTAs.  Cost of a unit = its bytes plus a fixed part; every CTA gets the same total.
// A's units go to the first CTAs (at the start of their runs), B's to the last ones (at the end of theirs), so
// that t is complete long before the first unit of B is reached; the backbone fills every CTA up to the mean.
static void tc_plan(TcState* t, bool ab) {
  const int G = t->grid;
  const uint32_t nA = ab ? (uint32_t)t->a.nt * t->a.nkb : 0u, nB = ab ? (uint32_t)t->b.nt * t->b.nkb : 0u;
  const uint32_t nW = (uint32_t)t->w.nt * t->w.nkb;
  const double fixed = 1500.0;
  const double cW = t->w.unit + fixed, cA = ab ? t->a.unit + fixed : 0.0, cB = ab ? t->b.unit + fixed : 0.0;
  const int gA = nA ? (int)(nA < (uint32_t)G ? nA : G) : 0, gB = nB ? (int)(nB < (uint32_t)G ? nB : G) : 0;
  const double mean = (nA * cA + nB * cB + nW * cW) / G;
  std::vector<uint32_t> an(G, 0), bn(G, 0);
  std::vector<double> want(G, 0.0);
  for (int c = 0; c < gA; ++c) an[c] = nA / gA + ((uint32_t)c < nA % gA ? 1u : 0u);
  for (int c = 0; c < gB; ++c) bn[G - gB + c] = nB / gB + ((uint32_t)c < nB % gB ? 1u : 0u);
  double want_total = 0.0;
  for (int c = 0; c < G; ++c) {
    const double rest = mean - an[c] * cA - bn[c] * cB;
    want[c] = rest > 0.0 ? rest : 0.0;
    want_total += want[c];
  }
  uint32_t a0 = 0, b0 = 0, w0 = 0;
  double cum = 0.0;
  for (int c = 0; c < G; ++c) {
    cum += want[c];
    uint32_t w_end = want_total > 0.0 ? (uint32_t)((double)nW * cum / want_total + 0.5) : (uint32_t)((uint64_t)nW * (c + 1) / G);
    if (c == G - 1 || w_end > nW) w_end = nW;
    if (w_end < w0) w_end = w0;
    CtaPlan& p = t->plan[c];
    p.a0 = a0; p.w0 = w0; p.b0 = b0;
    p.an_bn = an[c] | (bn[c] << 16);
    p.wn = w_end - w0;
    a0 += an[c]; b0 += bn[c]; w0 = w_end;
  }
}

cudaError_t decode_tc_init(Handle* h, cudaStream_t st) {
  h->tc_state = nullptr;
  if (h->cfg.kernel_policy != EORA_POLICY_TMEM_DECODE || !tc_formats_ok(h)) return cudaSuccess;
  const bool ab = h->cfg.rank > 0;
  TcState* t = new (std::nothrow) TcState();
  if (!t) return cudaErrorMemoryAllocation;
  *t = TcState();
  tmat_shape(t->w, h->w.fmt, h->w);
  if (ab) { tmat_shape(t->a, h->a.fmt, h->a); tmat_shape(t->b, h->b.fmt, h->b); }
  t->grid = h->sm_count < kMaxCtas ? h->sm_count : kMaxCtas;
  // units per run are 16-bit in the plan
  if ((ab && ((int64_t)t->a.nt * t->a.nkb / t->grid + 1 > 65535 || (int64_t)t->b.nt * t->b.nkb / t->grid + 1 > 65535))) { delete t; return cudaSuccess; }
  auto up = [](int64_t v) { return (v + 255) / 256 * 256; };
  const int64_t wb = up(tmat_bytes(t->w)), abytes = ab ? up(tmat_bytes(t->a)) : 0, bb = ab ? up(tmat_bytes(t->b)) : 0;
  t->weight_bytes = wb + abytes + bb;
  cudaError_t e = cudaMalloc(&t->weight_mem, (size_t)t->weight_bytes);
  if (e != cudaSuccess) { delete t; return e; }
  t->w.q = reinterpret_cast<uint8_t*>(t->weight_mem);
  t->a.q = t->w.q + wb;
  t->b.q = t->a.q + abytes;
  const int64_t tcols = h->t_cols;
  const int64_t dt_b = up((int64_t)kTcMaxTokens * tcols * 4), yws_b = up((int64_t)kTcMaxTokens * t->w.n_rows * 4);
  const int64_t cnt_b = up((int64_t)(t->w.nt + 2) * 4), tgt_b = up((int64_t)t->w.nt * 4);   // one array of targets; there are two
  t->zero_bytes = dt_b + yws_b + cnt_b;
  t->scratch_bytes = t->zero_bytes + 2 * tgt_b;
  e = cudaMalloc(&t->scratch_mem, (size_t)t->scratch_bytes);
  if (e != cudaSuccess) { cudaFree(t->weight_mem); delete t; return e; }
  char* sp = reinterpret_cast<char*>(t->scratch_mem);
  t->d_t = reinterpret_cast<float*>(sp);
  t->y_ws = reinterpret_cast<float*>(sp + dt_b);
  t->counters = reinterpret_cast<uint32_t*>(sp + dt_b + yws_b);
  t->targets[0] = reinterpret_cast<uint32_t*>(sp + t->zero_bytes);
  t->targets[1] = reinterpret_cast<uint32_t*>(sp + t->zero_bytes + tgt_b);
  h->tc_state = t;
  auto fail = [&](cudaError_t err) { decode_tc_free(h); return err; };
  if ((e = cudaMemsetAsync(t->scratch_mem, 0, (size_t)t->scratch_bytes, st)) != cudaSuccess) return fail(e);
  if ((e = launch_tmat_from_wmat(t->w, h->w, st)) != cudaSuccess) return fail(e);
  if (ab) {
    if ((e = launch_tmat_from_wmat(t->a, h->a, st)) != cudaSuccess) return fail(e);
    if ((e = launch_tmat_from_wmat(t->b, h->b, st)) != cudaSuccess) return fail(e);
  }
  tc_plan(t, ab);
  for (int c = 0; c < t->grid; ++c) {        // the kernel keeps a CTA's run as a table of at most kMaxUnits entries
    const CtaPlan& pl = t->plan[c];
    if ((pl.an_bn & 0xffffu) + (pl.an_bn >> 16) + pl.wn > (uint32_t)kMaxUnits) { decode_tc_free(h); return cudaSuccess; }
  }
  // Tickets per row tile and flushes of A: set k of a CTA takes units k, k + NS, ... of the CTA's run (A, then W, then B);
  // each of its four warps adds its sums and takes a ticket whenever the set's next unit belongs to another (segment, row
  // tile) or there is none.  The kernel's walk, repeated here for both numbers of sets.
  std::vector<uint32_t> targets[2];
  for (int v = 0; v < 2; ++v) {
    const uint32_t NS = v == 0 ? (uint32_t)TcShape<1>::NS : (uint32_t)TcShape<16>::NS;
    targets[v].assign(t->w.nt, 0u);
    t->a_flush_total[v] = 0;
    for (int c = 0; c < t->grid; ++c) {
      const CtaPlan& pl = t->plan[c];
      const uint32_t an = pl.an_bn & 0xffffu, bn = pl.an_bn >> 16, n = an + pl.wn + bn;
      auto key = [&](uint32_t i) -> uint64_t {          // (segment, row tile) of unit i of the run
        if (i < an) return ((uint64_t)0 << 32) | ((pl.a0 + i) / t->a.nkb);
        if (i < an + pl.wn) return ((uint64_t)1 << 32) | ((pl.w0 + (i - an)) / t->w.nkb);
        return ((uint64_t)2 << 32) | ((pl.b0 + (i - an - pl.wn)) / t->b.nkb);
      };
      for (uint32_t k = 0; k < NS; ++k)
        for (uint32_t i = k; i < n; i += NS)
          if (i + NS >= n || key(i) != key(i + NS)) {
            const uint64_t kk = key(i);
            if ((kk >> 32) == 0) t->a_flush_total[v] += 4;
            else targets[v][(uint32_t)kk] += 4;
          }
    }
    if ((e = cudaMemcpyAsync(t->targets[v], targets[v].data(), targets[v].size() * 4, cudaMemcpyHostToDevice, st)) != cudaSuccess) return fail(e);
  }
  if ((e = cudaStreamSynchronize(st)) != cudaSuccess) return fail(e);   // `targets` are locals
  return cudaSuccess;
}

cudaError_t launch_decode_tc_forward(const Handle* h, const void* x, int m, void* const* ys, cudaStream_t st) {
  const TcState* t = reinterpret_cast<const TcState*>(h->tc_state);
  if (!t) return cudaErrorInvalidValue;
  const bool ab = h->cfg.rank > 0;
  TcArgs a = {};
  a.q[0] = t->a.q; a.q[1] = t->w.q; a.q[2] = t->b.q;
  a.nkb[0] = ab ? (uint32_t)t->a.nkb : 1u; a.nkb[1] = (uint32_t)t->w.nkb; a.nkb[2] = ab ? (uint32_t)t->b.nkb : 1u;
  a.nt_w = (uint32_t)t->w.nt;
  a.n_sub = h->n_sub;
  for (int i = 0; i <= h->n_sub; ++i) a.sub_tile0[i] = (uint32_t)h->sub_tile0[i] / 8u;     // the handle counts tiles of 16 rows
  for (int i = h->n_sub + 1; i < 5; ++i) a.sub_tile0[i] = (uint32_t)t->w.nt;
  for (int i = 0; i < 4; ++i) a.sub_dout[i] = i < h->n_sub ? h->sub_dout[i] : 0;
  a.d_t = t->d_t; a.y_ws = t->y_ws; a.counters = t->counters; a.dev_status = h->dev_status;
  a.d_in = h->cfg.d_in; a.t_cols = h->t_cols; a.r_pad = h->r_pad; a.n_pad = t->w.n_rows;
  a.x_dtype = h->cfg.x_dtype; a.y_dtype = h->cfg.y_dtype;
  a.wait_ns = h->wait_limit_ns;
  memcpy(a.plan, t->plan, sizeof(CtaPlan) * (size_t)t->grid);

  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(t->grid);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const int abf = ab ? h->a.fmt : FMT_NONE;
  const size_t ybytes = h->cfg.y_dtype == EORA_Y_F32 ? 4 : 2;
  for (int m0 = 0; m0 < m; m0 += kTcMaxTokens) {
    a.m = m - m0 < kTcMaxTokens ? m - m0 : kTcMaxTokens;
    const int mt = a.m == 1 ? 1 : a.m <= 8 ? 8 : 16;
    cfg.dynamicSmemBytes = (size_t)tc_smem_bytes(mt);
    cfg.blockDim = dim3(mt == 1 ? TcShape<1>::kThreads : mt == 8 ? TcShape<8>::kThreads : TcShape<16>::kThreads);
    const int v = mt <= 8 ? 0 : 1;                      // sets per CTA: five up to eight tokens, four above
    a.targets = t->targets[v]; a.a_flush_total = t->a_flush_total[v];
    a.x = reinterpret_cast<const uint8_t*>(x) + (size_t)m0 * h->cfg.d_in * 2;
    for (int i = 0; i < h->n_sub; ++i) a.ys[i] = reinterpret_cast<uint8_t*>(ys[i]) + (size_t)m0 * h->sub_dout[i] * ybytes;
    cudaError_t e = h->w.fmt == FMT_Q4 ? launch_tc_ab<FMT_Q4>(cfg, a, h->device, mt, abf) : launch_tc_ab<FMT_Q3>(cfg, a, h->device, mt, abf);
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

}  // namespace eora
