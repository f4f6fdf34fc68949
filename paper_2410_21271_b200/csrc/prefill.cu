// Prefill kernel family (M > 64, and 16 < M <= 64 where it beats the decode passes): Y = X.deq(Wq) + (X.A).B
// (paper Eq. 4) as a tcgen05 GEMM.
//
// The paper measures only batch-1 decoding (Section 4.5); for many tokens the layer is a dense
// contraction, so it runs on the 5th-generation tensor cores.  The product is computed transposed,
// Yt[n][m] = sum_k w[n][k] X[m][k], so that the operand that has to be produced on chip is the small one:
//   * MMA "A" operand (128 rows): a tile of 128 output columns n of the weights.  Sixteen dequant warps
//     read the packed tiles of the shared layout straight from global memory (512 contiguous bytes per
//     warp), turn them into fp16 RN((q - z) * s) in registers and store them as a K-major,
//     128-byte-swizzled operand tile (bank-conflict-free stores);
//   * MMA "B" operand (up to 256 rows): a tile of tokens of X, K-major, brought in by TMA
//     (cp.async.bulk.tensor, 128-byte swizzle, no multicast) into the same ring of k-block stages as
//     the dequantised weight tile;
//   * one thread issues tcgen05.mma (M = 128, N = tokens, K = 16) with the fp32 accumulator in tensor
//     memory; tcgen05.commit releases the ring slots when the MMAs have drained;
//   * the low-rank term is a K-extension: after the d_in/64 backbone k-blocks come r/64 k-blocks whose
//     token operand is t = X.A (fp16, from a first launch of the same kernel with A as the weight) and
//     whose weight operand is B, so (X.A).B lands in the same accumulator.  The two launches overlap:
//     the main one is a programmatic dependent launch that waits for t only in front of the K-extension;
//   * epilogue (all sixteen dequant warps): tcgen05.ld -> fp16/bf16/fp32 -> transpose through shared
//     memory -> 16-byte row stores, so Y is written once.
// Launches per forward: 1 (rank 0) or 2 (t = X.A, then the main product), plus a conversion launch
// when X is bf16 (the f16 MMA kind needs both operands in fp16; weights are kept fp16 because
// bf16 weights alone cost 1.7e-3 of the 2e-3 error budget).
#include <cuda.h>
#include "decode_common.cuh"

namespace eora {
using namespace dec;
namespace {

constexpr int BN_W = 128, BK = 64;               // weight rows per MMA (its M), k-block; a CTA owns up to two such halves
constexpr int kDqWarps = 16;                    // dequant warps (warps 4..19): one 16-row tile of the 256 weight rows each
constexpr int kThreadsP = (4 + kDqWarps) * 32;  // warp 0: TMA, warp 1: MMA, warp 2: TMEM alloc, warp 3: idle
constexpr int kMaxWStages = 4;                  // ring of k-block stages (token tile + dequantised weight tile)
constexpr int kSmallTile = 128;                // rows and tokens of the small tiles that fill a launch's last wave
constexpr int kPrefetch = 4;                    // k-blocks of packed weights held in registers ahead of use (2 for fp16)

struct PrefillArgs {
  WMat w;            // weight operand of the first nkb_w k-blocks (rows = output columns)
  WMat b;            // weight operand of the K-extension (FMT_NONE if none)
  void* out;         // [m][ld_out]
  int out_dtype;     // EORA_Y_*
  int ld_out;        // leading dimension of out (elements)
  int n_valid;       // columns of out to write
  int m;
  int bt;            // token tile (the MMA N): multiple of 16, at most 256
  int rows;          // weight rows per CTA: 256 (two MMA halves) or 128 (small matrices: more CTAs, half the dequant work each)
  // The grid is one-dimensional.  CTAs [0, n_small) take tiles of 128 rows x 128 tokens of the weight rows
  // [n_split, n_valid) (small_x row tiles per token tile); the others take tiles of rows x bt of the weight rows
  // [0, n_split) (big_x row tiles per token tile).  Without small tiles n_small = 0 and n_split = n_valid.
  int n_small, small_x, n_split, big_x;
  int nkb_w, nkb_b;  // k-blocks of each part
  int sx, sw;        // stages of the ring (sx == sw: token tiles first, weight tiles from w_off on)
  int w_off;         // byte offset of the weight ring (after sx token tiles of bt*128 bytes)
  // Few tokens (one token tile): the reduction axis is split over ksplit CTAs per tile (kchunk k-blocks each; the
  // first one also takes the K-extension).  Each adds its accumulator to ws (fp32, [tokens][ld_ws], zero between
  // launches) and takes a ticket of its tile; the CTA that takes the last one converts the sums to `out` and puts
  // ws and the ticket back to zero.  ksplit == 1: the accumulator goes straight to `out`.
  // Fused layers (stacked along the weight rows): layer i owns rows [sub_row0[i], sub_row0[i + 1]),
  // writes to outs[i] (leading dimension sub_ld[i]) and takes columns [i * t_sub, (i + 1) * t_sub) of t in the
  // K-extension.  A plain layer: n_sub = 1, sub_row0 = {0, n_valid}, outs[0] = out.
  int n_sub;
  int sub_row0[5];
  void* outs[4];
  int sub_ld[4];
  int t_sub;
  int ksplit, kchunk;
  float* ws;
  int ld_ws;
  uint32_t* tickets;
  int* dev_status;
  long long* trace;  // optional: for CTA (0,0), 4 clock64() stamps per k-block (token copy requested, W ready, X ready, MMA issued),
                     // then one more row: kernel entry, set-up done, accumulators complete, epilogue done
};

#define CTRACE(slot) do { if (p.trace) p.trace[1024 + 4 * blockIdx.x + (slot)] = (long long)globaltimer_ns(); } while (0)
#define PTRACE(it, slot) do { if (p.trace && blockIdx.x == 0 && blockIdx.y == 0) p.trace[(it) * 4 + (slot)] = clock64(); } while (0)

struct PrefillState {
  __half* x16;       // fp16 copy of a bf16 X, [max_m][d_in] (bf16 handles only)
  // split-K workspace of launches with few tokens (see PrefillArgs::ksplit): sums and tickets of the main product
  // and of t = X.A; one allocation, zero between launches
  void* split_mem;
  size_t split_bytes;
  float* ws_y; float* ws_t;
  uint32_t* tk_y; uint32_t* tk_t;
};

constexpr int kThinTokens = 64;        // launches of up to this many tokens may split the reduction axis

// ---------------------------------------------------------------------------------------------- PTX
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* tm, int c0, int c1, uint64_t* bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
               ::"r"(smem_u32(dst)), "l"(tm), "r"(c0), "r"(c1), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void umma_f16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
               ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
               "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
               : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
                 "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
                 "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
                 "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
               : "r"(taddr) : "memory");
}

// K-major, 128-byte swizzle operand descriptor: rows of 128 B, 8-row groups 1024 B apart.
__device__ __forceinline__ uint64_t make_desc(const void* smem_ptr) {
  const uint32_t addr = smem_u32(smem_ptr);
  const uint32_t lo = ((addr & 0x3FFFFu) >> 4) | (1u << 16);            // start address, leading byte offset (unused) = 1
  const uint32_t hi = (1024u >> 4) | (1u << 14) | (2u << 29);           // stride byte offset, descriptor version 1, SWIZZLE_128B
  return ((uint64_t)hi << 32) | lo;
}

// packed tile payload of one lane, by format
template <int FMT> struct Packed;
template <> struct Packed<FMT_Q4> { uint4 v; };
template <> struct Packed<FMT_Q3> { uint2 v; uint32_t w2; };
template <> struct Packed<FMT_Q8> { uint4 v[2]; };
template <> struct Packed<FMT_F16> { uint4 v[4]; };
template <> struct Packed<FMT_SP24> { uint4 v[2]; uint32_t meta; };
template <> struct Packed<FMT_SQ4> { uint2 v; uint32_t meta; };

// Lanes with an odd row index g store the two 32-element halves of their rows in the opposite order
// (see dequant_store), so they take them in the opposite order too: where a half is a separate piece of
// the tile the swap is done here, by address (sw = 1 for such lanes); otherwise swap_halves does it on
// the loaded words, at the time they are used.
template <int FMT>
__device__ __forceinline__ void load_packed(Packed<FMT>& r, const uint8_t* blob, int lane, int sw) {
  if constexpr (FMT == FMT_Q4) r.v = __ldg(reinterpret_cast<const uint4*>(blob) + lane);
  else if constexpr (FMT == FMT_Q3) {
    r.v = __ldg(reinterpret_cast<const uint2*>(blob) + lane);
    r.w2 = __ldg(reinterpret_cast<const uint32_t*>(blob + 256) + lane);
  } else if constexpr (FMT == FMT_Q8) {
    r.v[0] = __ldg(reinterpret_cast<const uint4*>(blob + 512 * sw) + lane);
    r.v[1] = __ldg(reinterpret_cast<const uint4*>(blob + 512 * (sw ^ 1)) + lane);
  } else if constexpr (FMT == FMT_F16) {
#pragma unroll
    for (int p = 0; p < 4; ++p) r.v[p] = __ldg(reinterpret_cast<const uint4*>(blob + 512 * (p ^ (2 * sw))) + lane);
  } else if constexpr (FMT == FMT_SQ4) {
    r.v = __ldg(reinterpret_cast<const uint2*>(blob) + lane);
    r.meta = __ldg(reinterpret_cast<const uint32_t*>(blob + 256) + lane);
  } else {
    r.v[0] = __ldg(reinterpret_cast<const uint4*>(blob + 512 * sw) + lane);
    r.v[1] = __ldg(reinterpret_cast<const uint4*>(blob + 512 * (sw ^ 1)) + lane);
    r.meta = __ldg(reinterpret_cast<const uint32_t*>(blob + 1024) + lane);
  }
}
__device__ __forceinline__ void cswap(uint32_t& a, uint32_t& b, bool sw) {
  const uint32_t x = sw ? b : a, y = sw ? a : b;
  a = x; b = y;
}
// The value-level part of the swap (formats whose halves share a load; the position bytes of the 2:4 formats).
template <int FMT>
__device__ __forceinline__ void swap_halves(Packed<FMT>& r, bool sw) {
  if constexpr (FMT == FMT_Q4) { cswap(r.v.x, r.v.z, sw); cswap(r.v.y, r.v.w, sw); }
  else if constexpr (FMT == FMT_SQ4) { cswap(r.v.x, r.v.y, sw); r.meta = __funnelshift_l(r.meta, r.meta, sw ? 16 : 0); }
  else if constexpr (FMT == FMT_SP24) r.meta = __funnelshift_l(r.meta, r.meta, sw ? 16 : 0);
}

__device__ __forceinline__ uint32_t h2mul(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("mul.rn.f16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}

__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

// Byte offsets, inside one stage of the weight ring, of the four 16-byte chunks (8 consecutive reduction
// elements of one row each) that a lane stores per tile.  Store k holds row g + 8 * (k & 1) and the half
// (k >> 1) ^ (g & 1) of the 64 reduction elements: in step k lanes with even g write one half and lanes
// with odd g the other, so that the 8 lanes of a quarter warp (two rows) hit 8 different 16-byte columns
// of the 128-byte swizzle.
__device__ __forceinline__ void store_offsets(uint32_t (&off)[4], int tile, int lane) {
  const int g = lane >> 2, t = lane & 3;
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const int row = tile * 16 + g + 8 * (k & 1);
    const int chunk = (((k >> 1) ^ (g & 1)) << 2) + t;          // 16-byte chunk index along K inside the 128-byte row
    off[k] = (uint32_t)(row * 128 + ((chunk ^ (row & 7)) << 4));
  }
}

// Per-tile constants (1024 + z), -(64 + z) as fp16x2 for the two rows of a lane, one byte permute each.
template <int FMT>
__device__ __forceinline__ void make_zc_p(ZC& zc, uint32_t zz) {
  zc.c[0][0] = prmt(zz, 0x64646464u, 0x4040u);
  zc.c[1][0] = prmt(zz, 0x64646464u, 0x4141u);
  if constexpr (FMT == FMT_Q4) {
    const uint32_t z4 = zz << 4;                                  // bytes: z_a << 4, z_b << 4 (zero-points < 16)
    zc.c[0][1] = prmt(z4, 0xD4D4D4D4u, 0x4040u);
    zc.c[1][1] = prmt(z4, 0xD4D4D4D4u, 0x4141u);
  }
}

// Dequantise one 16 x 64 tile to fp16 RN((q - z) * s) and store this lane's four chunks into the swizzled
// operand of the stage at shared address `stage`.  The lane's words arrive with their halves in storage
// order; `odd` (= g & 1) says that this lane stores them in the opposite order (store_offsets).
template <int FMT>
__device__ __forceinline__ void dequant_store(Packed<FMT> r, uint32_t sc2, uint32_t zz2, uint32_t stage, const uint32_t (&off)[4], bool odd,
                                              uint32_t lut) {
  swap_halves<FMT>(r, odd);
  uint32_t out[4][4];     // [part][pair]; part = 2 * (half as stored by this lane) + (row g or g + 8)
  if constexpr (FMT == FMT_F16) {
#pragma unroll
    for (int p = 0; p < 4; ++p) { out[p][0] = r.v[p].x; out[p][1] = r.v[p].y; out[p][2] = r.v[p].z; out[p][3] = r.v[p].w; }
  } else if constexpr (FMT == FMT_SP24 || FMT == FMT_SQ4) {
    // A quad's two kept values (one register) are spread over its four positions (two registers) with two
    // byte permutes whose selectors come from a 16-entry table in shared memory indexed by the quad's
    // position nibble (sp24_selectors).
    [[maybe_unused]] ZC zc;
    if constexpr (FMT == FMT_SQ4) make_zc_p<FMT>(zc, zz2);
#pragma unroll
    for (int p = 0; p < 4; ++p) {
      uint32_t vq[2];                                                         // (val0,val1) of quad 0, of quad 1
      if constexpr (FMT == FMT_SP24) {
        const uint4 u = r.v[p >> 1];
        vq[0] = (p & 1) ? u.z : u.x; vq[1] = (p & 1) ? u.w : u.y;
      } else {                                                                // kept codes -> RN((q - z) * s)
        const int hf = p & 1;
        const uint32_t w = (p >> 1) ? r.v.y : r.v.x;
        const uint32_t s2 = prmt(sc2, 0u, hf ? 0x3232u : 0x1010u);
        vq[0] = h2mul(h2sub(and_or(w >> (8 * hf), 0x000f000fu, kMagic), zc.c[hf][0]), s2);
        vq[1] = h2mul(h2sub(and_or(w >> (8 * hf + 4), 0x000f000fu, kMagic), zc.c[hf][0]), s2);
      }
#pragma unroll
      for (int quad = 0; quad < 2; ++quad) {
        const int sh = 8 * p + 4 * quad - 2;                                  // nibble * 4 = byte offset into the table
        const uint32_t offb = (sh < 0 ? (r.meta << 2) : (r.meta >> (sh < 0 ? 0 : sh))) & 0x3Cu;
        uint32_t sel;
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(sel) : "r"(lut + offb));
        out[p][2 * quad] = prmt(vq[quad], 0u, sel);
        out[p][2 * quad + 1] = prmt(vq[quad], 0u, sel >> 16);
      }
    }
  } else {
    ZC zc;
    make_zc_p<FMT>(zc, zz2);
    uint32_t a[4][4];
    if constexpr (FMT == FMT_Q4) {
      const uint32_t w[4] = {r.v.x, r.v.y, r.v.z, r.v.w};
#pragma unroll
      for (int part = 0; part < 4; ++part) {
        const int hf = part & 1;
        uint32_t lo = w[part], hi = w[part] >> 8;
        a[part][0] = h2sub(and_or(lo, 0x000f000fu, kMagic), zc.c[hf][0]);
        a[part][1] = h2fma(and_or(lo, 0x00f000f0u, kMagic), 0x2C002C00u, zc.c[hf][1]);
        a[part][2] = h2sub(and_or(hi, 0x000f000fu, kMagic), zc.c[hf][0]);
        a[part][3] = h2fma(and_or(hi, 0x00f000f0u, kMagic), 0x2C002C00u, zc.c[hf][1]);
      }
    } else if constexpr (FMT == FMT_Q3) {
      uint32_t q[4][2];
      q3_quads(r.v.x, r.v.y, r.w2, q);
#pragma unroll
      for (int j = 0; j < 2; ++j) { cswap(q[0][j], q[2][j], odd); cswap(q[1][j], q[3][j], odd); }
#pragma unroll
      for (int part = 0; part < 4; ++part) {
        const int hf = part & 1;
#pragma unroll
        for (int j = 0; j < 4; ++j) a[part][j] = h2sub(quad_pair(q[part][j >> 1], j & 1), zc.c[hf][0]);
      }
    } else {   // FMT_Q8
#pragma unroll
      for (int part = 0; part < 4; ++part) {
        const int hf = part & 1;
        const uint4 u = r.v[part >> 1];
        const uint32_t w0 = hf ? u.z : u.x, w1 = hf ? u.w : u.y;
        a[part][0] = h2sub(and_or(w0, 0x00ff00ffu, kMagic), zc.c[hf][0]);
        a[part][1] = h2sub(and_or(w0 >> 8, 0x00ff00ffu, kMagic), zc.c[hf][0]);
        a[part][2] = h2sub(and_or(w1, 0x00ff00ffu, kMagic), zc.c[hf][0]);
        a[part][3] = h2sub(and_or(w1 >> 8, 0x00ff00ffu, kMagic), zc.c[hf][0]);
      }
    }
    const uint32_t s_a = prmt(sc2, 0u, 0x1010u), s_b = prmt(sc2, 0u, 0x3232u);
#pragma unroll
    for (int part = 0; part < 4; ++part)
#pragma unroll
      for (int j = 0; j < 4; ++j) out[part][j] = h2mul(a[part][j], (part & 1) ? s_b : s_a);
  }
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const int part = (k >> 1) * 2 + (k & 1);
    st_shared_v4(stage + off[k], out[part][0], out[part][1], out[part][2], out[part][3]);
  }
}

__device__ __forceinline__ bool mbar_try_wait_a(uint32_t bar_addr, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
               : "=r"(ok) : "r"(bar_addr), "r"(parity) : "memory");
  return ok != 0;
}

// One part (W or the K-extension B) of a dequant warp's work.  The warp owns row tile `tile` (0..15) of
// the CTA's 256 weight rows; k-blocks [kb_lo, kb_hi) of `mat` land in pipeline iterations it0, it0 + 1, ...,
// and the warp takes those with index kb_lo + kphase + i * kstep (kstep = 2 when two warps share a row
// tile, which is how a CTA with 128 rows keeps all sixteen warps and twice the loads in flight).
// Packed weights, scales and zero-points are loaded PF of the warp's k-blocks ahead.  The loop is what bounds the
// kernel (four of these warps share a scheduler), so everything that does not change per k-block is
// computed once: the store offsets, the ring position as a running (slot, wrap) pair, shared addresses.
template <int FMT>
__device__ __forceinline__ bool dequant_part(const WMat& mat, int n0, int kb_lo, int kb_hi, int it0, int tile, int kphase,
                                             int kstep, int lane, uint8_t* smem, const PrefillArgs& p, uint64_t* full_w,
                                             uint64_t* empty_w, uint32_t lut) {
  if constexpr (FMT == FMT_NONE) {
    return true;
  } else {
    constexpr int PF = FMT == FMT_F16 ? 3 : kPrefetch;
    constexpr bool quant = fmt_quantised(FMT);
    constexpr int tb = tile_bytes(FMT);
    const int rt = (n0 >> 4) + tile;                     // this warp's row tile of the matrix
    const bool active = rt < mat.nt;
    const int g = lane >> 2;
    const int odd = g & 1;
    uint32_t off[4];
    store_offsets(off, tile, lane);
    const uint8_t* base = mat.q + (int64_t)rt * mat.blob;                 // this row tile's blob of pair 0
    const int64_t pair_stride = (int64_t)mat.nt * mat.blob;
    const int sz_step = mat.sz2 ? kSzEntryBytes : 0;
    const uint32_t ring = smem_u32(smem + p.w_off), full0 = smem_u32(full_w), empty0 = smem_u32(empty_w);
    Packed<FMT> pk[PF];
    uint32_t scq[PF], zzq[PF];
    auto issue = [&](int kb, int slot) {
      if (!active || kb >= kb_hi) return;
      const uint8_t* blob = base + (kb >> 1) * pair_stride;
      load_packed<FMT>(pk[slot], blob + (kb & 1) * tb, lane, odd);
      if constexpr (quant) {
        const uint8_t* sz = blob + 2 * tb + (kb & 1) * sz_step;
        scq[slot] = __ldg(reinterpret_cast<const uint32_t*>(sz) + g);
        zzq[slot] = __ldg(reinterpret_cast<const uint16_t*>(sz + 32) + g);
      }
    };
#pragma unroll
    for (int j = 0; j < PF; ++j) { scq[j] = 0; zzq[j] = 0; issue(kb_lo + kphase + j * kstep, j); }
    int it = it0 + kphase;
    int s = it % p.sw, wrap = it / p.sw;                 // ring slot of iteration `it`, and how often it has been used before
    for (int kbb = kb_lo + kphase; kbb < kb_hi; kbb += PF * kstep) {
#pragma unroll
      for (int j = 0; j < PF; ++j) {
        const int kb = kbb + j * kstep;
        if (kb < kb_hi) {
          if (wrap > 0 && !mbar_try_wait_a(empty0 + 8 * s, (wrap - 1) & 1) &&
              !mbar_wait_warp(empty_w + s, (wrap - 1) & 1, p.dev_status, lane)) return false;
          const uint32_t stage = ring + (uint32_t)s * (2 * BN_W * 128);
          if (active) {
            dequant_store<FMT>(pk[j], scq[j], zzq[j], stage, off, odd != 0, lut);
          } else {                                        // rows past the matrix: keep the operand finite
#pragma unroll
            for (int k = 0; k < 4; ++k) st_shared_v4(stage + off[k], 0u, 0u, 0u, 0u);
          }
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy stores -> visible to the MMA
          __syncwarp();
          if (lane == 0) {
            asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(full0 + 8 * s) : "memory");
            if (tile == 0) PTRACE(it, 1);
          }
          issue(kb + PF * kstep, j);
          it += kstep;
          s += kstep;
          if (s >= p.sw) { s -= p.sw; ++wrap; }             // kstep <= 2 <= stages
        }
      }
    }
    return true;
  }
}

template <int WF, int BF>
__global__ void __launch_bounds__(kThreadsP, 1) k_prefill(const __grid_constant__ CUtensorMap tm_x,
                                                          const __grid_constant__ CUtensorMap tm_t,
                                                          const __grid_constant__ CUtensorMap tm_x_small,
                                                          const __grid_constant__ CUtensorMap tm_t_small, const PrefillArgs p) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  // One ring for both operands: stage s holds the token tile and the dequantised weight tile of a k-block, full_w[s]
  // collects the copy's bytes and the dequant warps' arrivals, empty_w[s] one commit.  The thread that issues the MMAs
  // is what bounds a k-block (every MMA blocks it for the ~130 cycles its 128-row operand takes to load), so it gets
  // one wait and one commit per k-block instead of two of each.
  __shared__ __align__(8) uint64_t full_w[kMaxWStages], empty_w[kMaxWStages], acc_full;
  __shared__ uint32_t tmem_base_s;
  __shared__ uint32_t sp_lut[16];        // 2:4 expansion selectors (2:4 backbones only)
  __shared__ int fail_s;                 // set by an epilogue warp whose bounded wait ran out
  __shared__ int last_s;                 // split-K: this CTA took its tile's last ticket
  // 1024-byte alignment of the operand tiles (the swizzle pattern is anchored at 1 KB)
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));

  // Programmatic dependent launch: a kernel launched behind this one with the serialisation attribute may
  // start at once (the main product behind the launch that computes t; see launch_prefill_forward).
  asm volatile("griddepcontrol.launch_dependents;");
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const bool small = (int)blockIdx.x < p.n_small;
  const int big_id = (int)blockIdx.x - p.n_small;
  const int bt = small ? kSmallTile : p.bt;                 // tokens of this CTA's tile (the MMA N)
  const int rows = small ? kSmallTile : p.rows;
  // big tiles: row tile fastest, then the split of the reduction axis, then the token tile
  const int tile_x = big_id % p.big_x, split = small ? 0 : (big_id / p.big_x) % p.ksplit, tile_y = big_id / (p.big_x * p.ksplit);
  const int n0 = small ? p.n_split + ((int)blockIdx.x % p.small_x) * kSmallTile : tile_x * rows;
  const int m0 = small ? ((int)blockIdx.x / p.small_x) * kSmallTile : tile_y * bt;
  int sub = 0;                                              // fused layers: whose rows these are (tiles never straddle)
#pragma unroll
  for (int i = 1; i < 4; ++i)
    if (i < p.n_sub && n0 >= p.sub_row0[i]) sub = i;
  const int n_end = min(small ? p.n_valid : p.n_split, p.sub_row0[sub + 1]);   // this CTA writes columns n0 .. n_end - 1 at most
  void* const out_p = p.outs[sub];
  const int ld_o = p.sub_ld[sub], col0 = p.sub_row0[sub];   // output column of weight row n: n - col0
  const int nh = (rows > BN_W && n_end - n0 > BN_W) ? 2 : 1;   // 128-row halves of this CTA that hold real rows
  const CUtensorMap* map_x = small ? &tm_x_small : &tm_x;
  const CUtensorMap* map_t = small ? &tm_t_small : &tm_t;
  const int kw_lo = split * p.kchunk, kw_hi = min(p.nkb_w, kw_lo + p.kchunk);
  const int nkw = kw_hi - kw_lo;
  const int nkb_ext = split == 0 ? p.nkb_b : 0;             // the K-extension goes with the first split
  const int nkb = nkw + nkb_ext;
  const uint32_t xbytes = (uint32_t)bt * 128;               // bytes of a token tile; the ring's slots are p.bt * 128 apart
  const uint32_t xslot = (uint32_t)p.bt * 128;

  if constexpr (WF == FMT_SP24 || WF == FMT_SQ4) {
    if (threadIdx.x >= 32 && threadIdx.x < 48) sp_lut[threadIdx.x - 32] = sp24_selectors(threadIdx.x - 32);
  }
  const uint32_t lut = smem_u32(sp_lut);
  if (threadIdx.x == 0) {
    PTRACE(nkb, 0);
    CTRACE(0);
    fail_s = 0;
    for (int i = 0; i < p.sw; ++i) { mbar_init(full_w + i, 8 * nh + 1); mbar_init(empty_w + i, 1); }
    mbar_init(&acc_full, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 2) {   // tensor memory: two accumulators of 128 lanes x 256 fp32 columns
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_d = tmem_base_s;
  if (threadIdx.x == 0) PTRACE(nkb, 1);

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (token tiles)
    if (lane == 0) {
      int s = 0, wrap = 0;                          // ring slot of iteration `it`, and how often it has been used before
      for (int it = 0; it < nkb; ++it) {
        if (wrap > 0 && !mbar_wait(empty_w + s, (wrap - 1) & 1, p.dev_status)) break;
        PTRACE(it, 0);
        mbar_expect_tx(full_w + s, xbytes);
        uint8_t* xt = smem + (size_t)s * xslot;
        if (it < nkw) {
          tma_load_2d(xt, map_x, (kw_lo + it) * BK, m0, full_w + s);
        } else {
          // t comes from the previous launch, which may still be running: everything up to here overlapped with it
          if (it == nkw) asm volatile("griddepcontrol.wait;" ::: "memory");
          tma_load_2d(xt, map_t, (it - nkw) * BK + sub * p.t_sub, m0, full_w + s);
        }
        if (++s == p.sw) { s = 0; ++wrap; }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      // instruction descriptor: fp32 accumulate, fp16 x fp16, both operands K-major, M = 128 weight rows, N = bt tokens
      const uint32_t idesc = (1u << 4) | ((uint32_t)(bt >> 3) << 17) | ((uint32_t)(BN_W >> 4) << 24);
      bool ok = true;
      int sw = 0;                                   // ring slot of iteration `it` and its phase
      uint32_t pw = 0;
      for (int it = 0; it < nkb && ok; ++it) {
        ok = mbar_wait(full_w + sw, pw, p.dev_status);   // token tile copied and weight tile dequantised
        if (!ok) break;
        PTRACE(it, 2);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint64_t bdesc = make_desc(smem + (size_t)sw * xslot);
        const uint64_t adesc = make_desc(smem + p.w_off + (size_t)sw * (2 * BN_W * 128));
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          // half j / 4 of the weight rows is 128 rows = 16 KB further (+1024 in the address field), each K step of
          // 16 fp16 is 32 bytes further (+2)
          if (j < 4 * nh)
            umma_f16(tmem_d + (j >> 2) * 256, adesc + (uint64_t)((j >> 2) * ((BN_W * 128) >> 4) + 2 * (j & 3)), bdesc + 2 * (j & 3),
                     idesc, (it > 0 || (j & 3) > 0) ? 1u : 0u);
        }
        umma_commit(empty_w + sw);                  // arrives when these MMAs have finished reading their operands
        PTRACE(it, 3);
        if (++sw == p.sw) { sw = 0; pw ^= 1u; }
      }
      umma_commit(&acc_full);                       // arrives when every MMA above has completed
    }
  } else if (warp >= 4) {
    // ------------------------------------------------------------------ dequant warps, then epilogue
    const int dw = warp - 4;
    bool ok = true;
    {
      // two halves: one row tile per warp; one half: two warps per row tile, alternating k-blocks
      const int kstep = 3 - nh, tile = nh == 2 ? dw : (dw & 7), kphase = nh == 2 ? 0 : (dw >> 3);
      ok = dequant_part<WF>(p.w, n0, kw_lo, kw_hi, 0, tile, kphase, kstep, lane, smem, p, full_w, empty_w, lut);
      if (ok && nkb_ext > 0) ok = dequant_part<BF>(p.b, n0, 0, nkb_ext, nkw, tile, kphase, kstep, lane, smem, p, full_w, empty_w, lut);
    }
    {
      // Epilogue: all sixteen warps, as four groups of four.  A warp can read the quarter of the TMEM lanes
      // that its index selects (warp % 4 == dw % 4), i.e. accumulator rows (= weight rows n) 32 * (dw % 4) ...
      // of each half; columns are tokens.  The chunks of 32 tokens are dealt to the groups round-robin.
      if (ok) ok = mbar_wait_warp(&acc_full, 0, p.dev_status, lane);
      // the warps meet at barriers below: they must all take the same way
      if (!ok) *reinterpret_cast<volatile int*>(&fail_s) = 1;
      asm volatile("bar.sync 1, 512;" ::: "memory");
      ok = *reinterpret_cast<volatile int*>(&fail_s) == 0;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      if (dw == 0 && lane == 0) { PTRACE(nkb, 2); CTRACE(1); }
      const int grp = dw >> 2, lq = dw & 3;
      const int nl = lq * 32 + lane;                     // local weight row inside the half = thread index inside the group
      const int nchunk = (bt + 31) >> 5;
      const uint32_t lane_base = tmem_d + ((uint32_t)(lq * 32) << 16);
      if (p.ksplit > 1) {
        // Split reduction axis: add this CTA's share to the fp32 sums (a thread holds one column n for the 32 tokens of a
        // chunk; a warp's 32 lanes add 128 contiguous bytes per token), then one ticket per CTA.
        const int tok_valid = min(bt, p.m - m0);
        if (ok) {
          float* wsb = p.ws + (int64_t)m0 * p.ld_ws;
          for (int hh = 0; hh < nh; ++hh) {
            const int col = n0 + hh * BN_W + nl;
            for (int cc = 0; cc < nchunk; ++cc) {
              if (((hh * nchunk + cc) & 3) != grp) continue;
              const int c0 = cc * 32;
              uint32_t v[32];
              tmem_ld32(lane_base + hh * 256 + (uint32_t)c0, v);
              asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
              if (col < n_end) {
#pragma unroll
                for (int j = 0; j < 32; ++j)
                  if (c0 + j < tok_valid)
                    asm volatile("red.global.add.f32 [%0], %1;" ::"l"(wsb + (int64_t)(c0 + j) * p.ld_ws + col), "f"(__uint_as_float(v[j])) : "memory");
              }
            }
          }
          __threadfence();
        }
        asm volatile("bar.sync 1, 512;" ::: "memory");
        if (dw == 0 && lane == 0) {
          uint32_t old = 0;
          uint32_t* tk = p.tickets + tile_y * p.big_x + tile_x;
          if (ok) asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], %2;" : "=r"(old) : "l"(tk), "r"(1u) : "memory");
          last_s = (ok && old + 1u == (uint32_t)p.ksplit) ? 1 : 0;
          if (last_s) *tk = 0u;                          // nobody else touches the ticket any more
        }
        asm volatile("bar.sync 1, 512;" ::: "memory");
        if (*reinterpret_cast<volatile int*>(&last_s)) {
          __threadfence();
          // every share is in: sums -> output type, one token row per warp and step, 32 columns per instruction
          // (all loads of a warp's share first: one round trip to L2, not one per row)
          const int ncols = min(rows, n_end - n0);
          const int esz = p.out_dtype == EORA_Y_F32 ? 4 : 2;
          constexpr int kTok = (kThinTokens + kDqWarps - 1) / kDqWarps, kCol = 2 * BN_W / 32;
          float f[kTok][kCol];
#pragma unroll
          for (int i = 0; i < kTok; ++i) {
            const int tok = dw + i * kDqWarps;
#pragma unroll
            for (int k = 0; k < kCol; ++k) {
              const int c = lane + 32 * k;
              f[i][k] = (tok < tok_valid && c < ncols) ? __ldcg(p.ws + (int64_t)(m0 + tok) * p.ld_ws + n0 + c) : 0.f;
            }
          }
#pragma unroll
          for (int i = 0; i < kTok; ++i) {
            const int tok = dw + i * kDqWarps;
            if (tok >= tok_valid) continue;
            float* src = p.ws + (int64_t)(m0 + tok) * p.ld_ws + n0;
            uint8_t* dst = reinterpret_cast<uint8_t*>(out_p) + ((int64_t)(m0 + tok) * ld_o + n0 - col0) * esz;
#pragma unroll
            for (int k = 0; k < kCol; ++k) {
              const int c = lane + 32 * k;
              if (c >= ncols) continue;
              src[c] = 0.f;
              if (p.out_dtype == EORA_Y_F32) reinterpret_cast<float*>(dst)[c] = f[i][k];
              else if (p.out_dtype == EORA_Y_F16) reinterpret_cast<__half*>(dst)[c] = __float2half_rn(f[i][k]);
              else reinterpret_cast<__nv_bfloat16*>(dst)[c] = __float2bfloat16_rn(f[i][k]);
            }
          }
        }
      } else {
        // A chunk goes through shared memory as [32 tokens][128 n] so that the global stores are 16-byte
        // pieces of rows of Y.  The rings are free by now (every MMA has completed).  Each group has two
        // buffers and alternates: a buffer is rewritten two chunks later, after a barrier that every thread of
        // the group passes only when it has read the buffer out, so one barrier per chunk is enough.
        const int esz = p.out_dtype == EORA_Y_F32 ? 4 : 2;
        const int row_sh = esz == 4 ? 5 : 4;             // log2 of the 16-byte pieces per token row (128 n)
        uint8_t* gbuf = smem + grp * 32768;              // 2 x (32 tokens x 128 n x esz bytes <= 16 KB)
        int flip = 0;
        for (int hh = 0; hh < nh && ok; ++hh) {
          for (int cc = 0; cc < nchunk; ++cc) {
            if (((hh * nchunk + cc) & 3) != grp) continue;
            const int c0 = cc * 32;
            uint8_t* tbuf = gbuf + flip * 16384;
            flip ^= 1;
            uint32_t v[32];
            tmem_ld32(lane_base + hh * 256 + (uint32_t)c0, v);
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              const float f = __uint_as_float(v[j]);
              if (p.out_dtype == EORA_Y_F32) reinterpret_cast<float*>(tbuf)[j * BN_W + nl] = f;
              else if (p.out_dtype == EORA_Y_F16) reinterpret_cast<__half*>(tbuf)[j * BN_W + nl] = __float2half_rn(f);
              else reinterpret_cast<__nv_bfloat16*>(tbuf)[j * BN_W + nl] = __float2bfloat16_rn(f);
            }
            asm volatile("bar.sync %0, 128;" ::"r"(2 + grp) : "memory");
            const int pieces = 32 << row_sh;
            for (int i = nl; i < pieces; i += 128) {
              const int tok = i >> row_sh, piece = i & ((1 << row_sh) - 1);
              const int row = m0 + c0 + tok, col = n0 + hh * BN_W + piece * (16 / esz);
              if (c0 + tok < bt && row < p.m && col < n_end) {     // a chunk may reach past the tile's tokens
                const uint4 val = *reinterpret_cast<const uint4*>(tbuf + (size_t)tok * BN_W * esz + piece * 16);
                *reinterpret_cast<uint4*>(reinterpret_cast<uint8_t*>(out_p) + ((int64_t)row * ld_o + col - col0) * esz) = val;
              }
            }
          }
        }
      }
      if (dw == 0 && lane == 0) { PTRACE(nkb, 3); CTRACE(2); }
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 2) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_d), "r"(512u) : "memory");
}

// n is a multiple of 8 (d_in is a multiple of 128): 16 bytes in, 16 bytes out per step
__global__ void k_bf16_to_f16(const __nv_bfloat16* in, __half* out, int64_t n) {
  for (int64_t i = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x) * 8; i < n; i += (int64_t)gridDim.x * blockDim.x * 8) {
    const uint4 v = __ldg(reinterpret_cast<const uint4*>(in + i));
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    uint32_t o[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const __half2 h = __floats2half2_rn(__uint_as_float(w[j] << 16), __uint_as_float(w[j] & 0xffff0000u));
      o[j] = *reinterpret_cast<const uint32_t*>(&h);
    }
    *reinterpret_cast<uint4*>(out + i) = make_uint4(o[0], o[1], o[2], o[3]);
  }
}

// ---------------------------------------------------------------------------------------------- host
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess || !p) return nullptr;
    fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// fp16 [rows][cols] row-major, box = 64 columns x box_rows rows, 128-byte swizzle, zero fill out of bounds
bool make_map(CUtensorMap* tm, const void* base, int rows, int cols, int ld, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

constexpr int kSmemP = 225 * 1024;

// pdl: the launch may begin while the previous kernel of the stream is still running (it waits, on the
// device, before it touches what that kernel writes).
template <auto KERNEL>
cudaError_t launch_p(dim3 grid, int smem, cudaStream_t st, const CUtensorMap& tx, const CUtensorMap& tt, const CUtensorMap& txs,
                     const CUtensorMap& tts, const PrefillArgs& a, bool pdl) {
  static bool attr_set[64] = {};   // per kernel and device: the attribute belongs to the device that is current at the call
  int device = 0;
  if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= 64) return cudaErrorInvalidDevice;
  if (!attr_set[device]) {
    cudaError_t e = cudaFuncSetAttribute(KERNEL, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemP);
    if (e != cudaSuccess) return e;
    attr_set[device] = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(kThreadsP);
  cfg.dynamicSmemBytes = (size_t)smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, KERNEL, tx, tt, txs, tts, a);
}

template <int WF>
cudaError_t launch_bf(int bf, dim3 grid, int smem, cudaStream_t st, const CUtensorMap& tx, const CUtensorMap& tt,
                      const CUtensorMap& txs, const CUtensorMap& tts, const PrefillArgs& a, bool pdl) {
  switch (bf) {
    case FMT_F16: return launch_p<k_prefill<WF, FMT_F16>>(grid, smem, st, tx, tt, txs, tts, a, pdl);
    case FMT_Q4: return launch_p<k_prefill<WF, FMT_Q4>>(grid, smem, st, tx, tt, txs, tts, a, pdl);
    case FMT_Q8: return launch_p<k_prefill<WF, FMT_Q8>>(grid, smem, st, tx, tt, txs, tts, a, pdl);
    case FMT_Q3: return launch_p<k_prefill<WF, FMT_Q3>>(grid, smem, st, tx, tt, txs, tts, a, pdl);
    default: return launch_p<k_prefill<WF, FMT_NONE>>(grid, smem, st, tx, tt, txs, tts, a, pdl);
  }
}

cudaError_t launch_any(int wf, int bf, dim3 grid, int smem, cudaStream_t st, const CUtensorMap& tx, const CUtensorMap& tt,
                       const CUtensorMap& txs, const CUtensorMap& tts, const PrefillArgs& a, bool pdl) {
  switch (wf) {
    case FMT_Q4: return launch_bf<FMT_Q4>(bf, grid, smem, st, tx, tt, txs, tts, a, pdl);
    case FMT_Q3: return launch_bf<FMT_Q3>(bf, grid, smem, st, tx, tt, txs, tts, a, pdl);
    case FMT_SP24: return launch_bf<FMT_SP24>(bf, grid, smem, st, tx, tt, txs, tts, a, pdl);
    case FMT_SQ4: return launch_bf<FMT_SQ4>(bf, grid, smem, st, tx, tt, txs, tts, a, pdl);
    // A as the weight of the first launch (t = X.A): no K-extension there
    case FMT_F16: return launch_p<k_prefill<FMT_F16, FMT_NONE>>(grid, smem, st, tx, tt, txs, tts, a, pdl);
    case FMT_Q8: return launch_p<k_prefill<FMT_Q8, FMT_NONE>>(grid, smem, st, tx, tt, txs, tts, a, pdl);
    default: return cudaErrorInvalidValue;
  }
}

int fill_stages(PrefillArgs& a) {      // returns the dynamic shared memory to request
  const int stage = a.bt * 128 + 2 * BN_W * 128;       // token tile + weight tile of one k-block
  a.sw = (kSmemP - 1024) / stage;
  if (a.sw > kMaxWStages) a.sw = kMaxWStages;
  a.sx = a.sw;
  a.w_off = a.sx * a.bt * 128;
  return a.w_off + a.sw * 2 * BN_W * 128 + 1024;
}

// Weight rows per CTA: 256 or 128, whichever tiling needs less time counted in waves of sm_count CTAs (a CTA needs an SM
// of its own).  The dequantisation of a CTA's rows is what bounds its k-block period (1200 cycles for 256 rows, 763 for
// 128), so a 128-row tile costs 0.64 of a 256-row one.  A last partial wave of 256-row tiles that is at most a quarter
// of the SMs is covered by small tiles inside the first wave (launch_prefill_forward), counted as half a wave.
int cta_rows(int n_rows, int m, int bt, int sm_count) {
  if (n_rows <= BN_W) return 2 * BN_W;
  const int ty = (m + bt - 1) / bt;
  const int t256 = ((n_rows + 2 * BN_W - 1) / (2 * BN_W)) * ty, t128 = ((n_rows + BN_W - 1) / BN_W) * ty;
  const int over = t256 % sm_count;
  float w256 = (float)(t256 / sm_count);
  if (over > 0) w256 += (bt == 256 && t256 > sm_count && 4 * over <= sm_count) ? 0.5f : 1.0f;
  const float w128 = 0.64f * (float)((t128 + sm_count - 1) / sm_count);
  return w128 < w256 ? BN_W : 2 * BN_W;
}

int token_tile(int m) {                // the MMA N: a multiple of 16 up to 256
  if (m >= 256) return 256;
  return (m + 15) / 16 * 16;
}

}  // namespace

bool prefill_supported(const Handle* h, int m) {
  if (m <= 8) return false;              // one decode pass is always cheaper
  if (h->multi) return false;            // per-token adapters: decode family only
  if (h->n_sub > 1) {                    // fused layers: tiles of 128 rows must not straddle two layers
    for (int i = 0; i < h->n_sub; ++i)
      if (h->sub_dout[i] % BN_W) return false;
  }
  if (h->w.group % 64) return false;
  return encode_fn() != nullptr;
}

int prefill_launch_count(const Handle* h, int) {
  return (h->cfg.rank > 0 ? 2 : 1) + (h->cfg.x_dtype == EORA_X_BF16 ? 1 : 0);
}

cudaError_t prefill_init(Handle* h) {
  h->prefill_state = nullptr;
  if (h->cfg.max_m <= 8) return cudaSuccess;
  PrefillState* ps = new PrefillState();
  *ps = PrefillState();
  cudaError_t e = cudaSuccess;
  if (h->cfg.x_dtype == EORA_X_BF16) e = cudaMalloc(&ps->x16, (size_t)h->cfg.max_m * h->cfg.d_in * 2);
  if (e == cudaSuccess) {
    // split-K sums and tickets for launches of up to kThinTokens tokens
    const size_t tok = (size_t)(h->cfg.max_m < kThinTokens ? h->cfg.max_m : kThinTokens);
    const size_t rp = (size_t)(h->cfg.rank > 0 ? h->t_cols : 0);
    const size_t n_all = (size_t)(h->n_sub > 1 ? 16 * h->sub_tile0[h->n_sub] : h->cfg.d_out);
    const size_t y_b = tok * n_all * 4, t_b = tok * rp * 4;
    const size_t tky_b = ((n_all + BN_W - 1) / BN_W) * 4, tkt_b = ((rp + BN_W - 1) / BN_W) * 4;
    auto up = [](size_t v) { return (v + 255) & ~size_t(255); };
    ps->split_bytes = up(y_b) + up(t_b) + up(tky_b) + up(tkt_b) + 256;
    e = cudaMalloc(&ps->split_mem, ps->split_bytes);
    if (e == cudaSuccess) e = cudaMemset(ps->split_mem, 0, ps->split_bytes);
    char* q = reinterpret_cast<char*>(ps->split_mem);
    ps->ws_y = reinterpret_cast<float*>(q); q += up(y_b);
    ps->ws_t = reinterpret_cast<float*>(q); q += up(t_b);
    ps->tk_y = reinterpret_cast<uint32_t*>(q); q += up(tky_b);
    ps->tk_t = reinterpret_cast<uint32_t*>(q);
  }
  if (e != cudaSuccess) { cudaFree(ps->x16); cudaFree(ps->split_mem); delete ps; return e; }
  h->prefill_state = ps;
  h->scratch_bytes += (int64_t)ps->split_bytes;
  return cudaSuccess;
}

void prefill_free(Handle* h) {
  PrefillState* ps = reinterpret_cast<PrefillState*>(h->prefill_state);
  if (!ps) return;
  cudaFree(ps->x16);
  cudaFree(ps->split_mem);
  delete ps;
  h->prefill_state = nullptr;
}

// After a launch that gave up: sums and tickets back to zero.
cudaError_t prefill_reset(Handle* h, cudaStream_t st) {
  PrefillState* ps = reinterpret_cast<PrefillState*>(h->prefill_state);
  if (!ps || !ps->split_mem) return cudaSuccess;
  return cudaMemsetAsync(ps->split_mem, 0, ps->split_bytes, st);
}

// How many CTAs share a tile's reduction axis in a launch of few tokens: as many as there are SMs for, each with at
// least min_kb k-blocks (a CTA's set-up and epilogue are worth about eight of them).
int pick_ksplit(int tiles, int nkb, int sm_count, int min_kb, int cap) {
  int s = sm_count / (tiles > 0 ? tiles : 1);
  if (s > nkb / min_kb) s = nkb / min_kb;
  if (s > cap) s = cap;
  return s < 1 ? 1 : s;
}

cudaError_t launch_prefill_forward(const Handle* h, const void* x, int m, void* const* ys, cudaStream_t st) {
  const eora_linear_config& c = h->cfg;
  const void* x16 = x;
  if (c.x_dtype == EORA_X_BF16) {
    PrefillState* ps = reinterpret_cast<PrefillState*>(h->prefill_state);
    if (!ps || !ps->x16) return cudaErrorInvalidValue;
    int64_t n = (int64_t)m * c.d_in;
    int64_t blocks = (n / 8 + 255) / 256;
    if (blocks > h->sm_count * 8) blocks = h->sm_count * 8;
    k_bf16_to_f16<<<(int)blocks, 256, 0, st>>>(reinterpret_cast<const __nv_bfloat16*>(x), ps->x16, n);
    x16 = ps->x16;
  }
  const int bt = token_tile(m);
  PrefillState* pst = reinterpret_cast<PrefillState*>(h->prefill_state);
  const bool thin = m <= kThinTokens && pst && pst->split_mem;      // one token tile: split the reduction axis instead
  CUtensorMap tm_x, tm_t;
  if (!make_map(&tm_x, x16, m, c.d_in, c.d_in, bt)) return cudaErrorInvalidValue;
  const bool ab = c.rank > 0;
  if (ab) {
    if (!make_map(&tm_t, h->t16, m, h->t_cols, h->t_cols, bt)) return cudaErrorInvalidValue;
    // launch 1: t = X.A with A as the weight (rows = r_pad), written as fp16.  It is a small product (a few
    // CTAs with token tiles of 128), and the main launch behind it starts at once (programmatic dependent
    // launch) on the other SMs: the main product needs t only for its last k-blocks and waits for this
    // launch there, so the two overlap.
    // Its tile: 128 rows and 128 tokens per CTA give the shortest chain of k-blocks, but a CTA of either
    // launch needs an SM of its own, so when the main launch fits into one wave the first shape whose CTAs
    // fit beside it is taken (more rows, then more tokens per CTA: fewer CTAs, longer chain).
    const int n_rows_all = h->n_sub > 1 ? 16 * h->sub_tile0[h->n_sub] : c.d_out;
    const int rows_m = thin ? BN_W : cta_rows(n_rows_all, m, bt, h->sm_count);
    const int main_tiles = ((n_rows_all + rows_m - 1) / rows_m) * ((m + bt - 1) / bt);
    const int room = main_tiles <= h->sm_count ? h->sm_count - main_tiles : h->sm_count;
    int rows_t = 2 * BN_W, bt_t = bt;
    {
      const int cand[4][2] = {{BN_W, 128}, {2 * BN_W, 128}, {BN_W, 256}, {2 * BN_W, 256}};
      for (int i = 0; i < 4; ++i) {
        const int rr = h->t_cols > BN_W ? cand[i][0] : 2 * BN_W;    // one half of rows at most: the tile height does not matter
        const int tt = cand[i][1] < bt ? cand[i][1] : bt;
        rows_t = rr; bt_t = tt;
        if (((h->t_cols + rr - 1) / rr) * ((m + tt - 1) / tt) <= room) break;
      }
    }
    CUtensorMap tm_xt;
    if (!make_map(&tm_xt, x16, m, c.d_in, c.d_in, bt_t)) return cudaErrorInvalidValue;
    PrefillArgs a = {};
    a.w = h->a; a.b = WMat(); a.b.fmt = FMT_NONE;
    a.out = h->t16; a.out_dtype = EORA_Y_F16; a.ld_out = h->t_cols; a.n_valid = h->t_cols; a.m = m; a.bt = bt_t;
    a.nkb_w = c.d_in / BK; a.nkb_b = 0; a.dev_status = h->dev_status; a.trace = nullptr;
    a.rows = rows_t;
    a.n_small = 0; a.small_x = 1; a.n_split = a.n_valid; a.big_x = (h->t_cols + a.rows - 1) / a.rows;
    a.n_sub = 1; a.sub_row0[0] = 0; a.outs[0] = a.out; a.sub_ld[0] = a.ld_out; a.t_sub = 0;
    for (int i = 1; i < 5; ++i) a.sub_row0[i] = a.n_valid;
    a.ksplit = 1; a.kchunk = a.nkb_w; a.ws = nullptr; a.ld_ws = 0; a.tickets = nullptr;
    if (thin) {
      // t is the head of the chain (the main product waits for it in front of its K-extension): as short as possible
      a.rows = h->t_cols > BN_W ? BN_W : a.rows;
      a.big_x = (h->t_cols + a.rows - 1) / a.rows;
      a.ksplit = pick_ksplit(a.big_x, a.nkb_w, h->sm_count / 4, 4, 16);
      a.kchunk = (a.nkb_w + a.ksplit - 1) / a.ksplit;
      a.ksplit = (a.nkb_w + a.kchunk - 1) / a.kchunk;
      a.ws = pst->ws_t; a.ld_ws = h->t_cols; a.tickets = pst->tk_t;
    }
    const int smem_t = fill_stages(a);
    dim3 grid(a.big_x * a.ksplit * ((m + bt_t - 1) / bt_t), 1, 1);
    cudaError_t e = launch_any(h->a.fmt, FMT_NONE, grid, smem_t, st, tm_xt, tm_xt, tm_xt, tm_xt, a, false);
    if (e != cudaSuccess) return e;
  } else {
    tm_t = tm_x;
  }
  PrefillArgs a = {};
  a.w = h->w; a.b = h->b;
  if (!ab) a.b.fmt = FMT_NONE;
  // fused layers: the stacked rows; a plain layer has one part
  const int n_all = h->w.n_rows < 16 * h->sub_tile0[h->n_sub] ? h->w.n_rows : 16 * h->sub_tile0[h->n_sub];
  const int n_valid = h->n_sub > 1 ? n_all : c.d_out;
  a.out = ys[0]; a.out_dtype = c.y_dtype; a.ld_out = c.d_out; a.n_valid = n_valid; a.m = m; a.bt = bt;
  a.n_sub = h->n_sub; a.t_sub = h->n_sub > 1 ? h->r_pad : 0;
  for (int i = 0; i < 5; ++i) a.sub_row0[i] = n_valid;
  for (int i = 0; i < h->n_sub; ++i) {
    a.sub_row0[i] = h->n_sub > 1 ? 16 * h->sub_tile0[i] : 0;
    a.outs[i] = ys[i];
    a.sub_ld[i] = h->n_sub > 1 ? h->sub_dout[i] : c.d_out;
  }
  a.nkb_w = c.d_in / BK; a.nkb_b = ab ? h->r_pad / BK : 0; a.dev_status = h->dev_status;
  a.trace = reinterpret_cast<long long*>(h->trace);
  a.rows = cta_rows(n_valid, m, bt, h->sm_count);
  for (int i = 0; i < h->n_sub && h->n_sub > 1; ++i)          // fused layers: every layer a whole number of tiles
    if (h->sub_dout[i] % (2 * BN_W)) a.rows = BN_W;
  a.n_small = 0; a.small_x = 1; a.n_split = n_valid; a.big_x = (n_valid + a.rows - 1) / a.rows;
  a.ksplit = 1; a.kchunk = a.nkb_w; a.ws = nullptr; a.ld_ws = 0; a.tickets = nullptr;
  if (thin) {
    // tiles of 128 rows, unless those need a second wave and tiles of 256 rows do not (fused layers: every layer a whole
    // number of tiles)
    bool r256 = (n_valid + BN_W - 1) / BN_W > h->sm_count && (n_valid + 2 * BN_W - 1) / (2 * BN_W) <= h->sm_count;
    for (int i = 0; i < h->n_sub && h->n_sub > 1; ++i) r256 = r256 && h->sub_dout[i] % (2 * BN_W) == 0;
    a.rows = n_valid > BN_W && !r256 ? BN_W : 2 * BN_W;
    a.big_x = (n_valid + a.rows - 1) / a.rows;
    const int t_ctas = ab ? 16 : 0;                         // leave room for the CTAs of the t launch
    a.ksplit = pick_ksplit(a.big_x, a.nkb_w, h->sm_count - t_ctas, 8, 16);
    a.kchunk = (a.nkb_w + a.ksplit - 1) / a.ksplit;
    a.ksplit = (a.nkb_w + a.kchunk - 1) / a.kchunk;
    a.ws = pst->ws_y; a.ld_ws = n_valid; a.tickets = pst->tk_y;
  }
  const int big_y = (m + bt - 1) / bt;
  // Wave quantisation: a CTA needs an SM of its own, so a few tiles more than a whole number of waves cost a whole
  // wave (gate / up at M = 2048: 448 tiles on 148 SMs).  Then the last row tiles are taken out of the big grid until
  // it fits, and their rows are covered by small tiles (128 x 128, about half the time of a big one each) that are
  // dispatched first and share the launch's first wave with the big tiles.
  CUtensorMap tm_xs = tm_x, tm_ts = tm_t;
  const int tiles = a.big_x * big_y, over = tiles % h->sm_count;
  if (a.rows == 2 * BN_W && bt == 256 && tiles > h->sm_count && over > 0 && 4 * over <= h->sm_count) {
    const int peel = (over + big_y - 1) / big_y;                 // row tiles to take out
    if (peel < a.big_x) {
      a.big_x -= peel;
      a.n_split = a.big_x * a.rows;
      a.small_x = (n_valid - a.n_split + kSmallTile - 1) / kSmallTile;
      a.n_small = a.small_x * ((m + kSmallTile - 1) / kSmallTile);
      if (!make_map(&tm_xs, x16, m, c.d_in, c.d_in, kSmallTile)) return cudaErrorInvalidValue;
      if (ab && !make_map(&tm_ts, h->t16, m, h->t_cols, h->t_cols, kSmallTile)) return cudaErrorInvalidValue;
      if (!ab) tm_ts = tm_xs;
    }
  }
  const int smem_y = fill_stages(a);
  dim3 grid(a.n_small + a.big_x * a.ksplit * big_y, 1, 1);
  return launch_any(h->w.fmt, ab ? h->b.fmt : FMT_NONE, grid, smem_y, st, tm_x, tm_t, tm_xs, tm_ts, a, ab);
}

}  // namespace eora
