// Decode path (m <= 8 tokens per launch): one kernel computes Eq. 4 for a whole layer,
//     Y = X . deq(Wq) + (X . A) . B,
// streaming every weight byte exactly once.
//
// Work decomposition.  All three matrices are stored as blobs of 16 rows x 128 reduction elements,
// ordered pair-major (see eora_common.cuh), and every blob is an independent piece of work: a warp
// multiplies it with the 128 activations it needs (kept in registers as tensor-core operand
// fragments, tokens as the n8 side of the MMA) and adds the 16 x m partial sums to an fp32
// accumulator array in global memory with red.add.  Blobs of a 3/4-bit backbone go through an integer
// product (mma.m16n8k32 on the byte codes against two byte planes of 16-bit block fixed point activations,
// see decode_common.cuh), all other blobs (adapters, 2:4 backbones) are dequantised to exact fp16 integers
// and go through mma.m16n8k16.  Warps are fully independent: each owns a
// contiguous run of blobs of up to three matrices, fetches it with its own bulk copies into its own
// shared-memory ring and never synchronises with another warp of its CTA.
//
//   * the first warps ("A owners") take the blobs of A first (t += X . A, sums in d_t) and then a share of W,
//   * the last warps ("B owners") take one copy of W, then their blobs of B, for which the activations are t
//     (read back as fp32 and split into an fp16 high and low part, so that t keeps fp32-like accuracy),
//     then the rest of their share of W,
//   * the warps in between take backbone blobs only.
// The only wait in the kernel is the one before the B share: all of A must have been added to t.  A
// owners never wait, and they sit in the first half of the CTAs, which are dispatched first and hold no B
// owner, so a waiting warp never holds the place of a CTA it is waiting for.  The wait is bounded like every other.
//
// Completion.  Every blob of W or B that has been added to y_ws bumps the ticket of its row tile; the
// warp that brings a ticket to its final count converts the 16 x m sums to the output type, writes Y and
// puts the sums and the ticket back to zero.  The warp that finishes the last row tile also clears t
// and the counters, so all scratch is back to zero when the kernel ends.
//
// Programmatic dependent launch: the first bulk copies (weights never change) are issued before
// griddepcontrol.wait, i.e. while the previous kernel in the stream is still draining; activations
// and scratch are only touched after it.
#include "decode_common.cuh"

namespace eora {
namespace {
using namespace dec;

// One CTA of sixteen warps per SM.  The warps of a CTA start together; with several smaller CTAs per SM the ones that
// are placed last ran a fifth slower than the first (the scheduler prefers the older warps) and ended the kernel late.
constexpr int kWarps = 16;
constexpr int kThreads = kWarps * 32;
constexpr int kCtasPerSm = 1;
constexpr int kRing = 2;                  // bulk copies in flight per warp
constexpr int kSlotBytes = 6528;          // one ring slot = one bulk copy (a run of whole blobs: eight 3-bit, six 4-bit ones)
constexpr int kBarBytes = 512;            // kWarps * kRing mbarriers
constexpr int kSmemBytes = kWarps * kRing * kSlotBytes + kBarBytes + kSp24LutBytes;

enum { CNT_A_DONE = 0, CNT_TILES_DONE = 1, CNT_TICKET0 = 2 };

struct Share { uint32_t per, rem; };      // blobs of a matrix dealt to n warps: warp i gets per + (i < rem)

struct DecodeArgs {
  const uint8_t* a_q; const uint8_t* w_q; const uint8_t* b_q;
  uint32_t a_nt, w_nt;                    // row tiles of A and of W (= of B)
  uint32_t a_blobs;                       // all of A
  uint32_t a_per_copy, w_per_copy, b_per_copy;   // blobs per bulk copy
  uint32_t a_sz2, w_sz2, b_sz2;
  // Three groups of warps: [0, n1) hold the blobs of A ("A owners"), [n1, n12) only backbone blobs,
  // [n12, all) the blobs of B.  Every group has its own share of the backbone, starting at w_base[group].
  uint32_t n1, n12;
  Share sh_a, sh_b, sh_w[3];
  uint32_t w_base[3];
  uint32_t tile_target;                   // blobs per output row tile: pairs of W + pairs of B
  const void* x;
  void* ys[4];                            // outputs of the fused layers (one for a plain layer)
  uint32_t sub_tile0[5];                  // layer i owns row tiles [sub_tile0[i], sub_tile0[i+1])
  int sub_dout[4];
  int n_sub;
  uint32_t b_np;                          // pairs of B per layer: the activations of B's blob (pair, tile) are
                                          // pair (layer(tile) * b_np + pair) of t
  // Several adapters on one backbone: pair p of B belongs to adapter p / adp_pairs, and token i uses adapter
  // adp[i] (-1: none).  adp_pairs == 0: one adapter for all tokens.
  uint32_t adp_pairs;
  int adp[8];
  float* d_t; float* y_ws; uint32_t* counters; int* dev_status;
  int m, d_in, r_pad, n_pad, x_dtype, y_dtype;   // r_pad: columns of t (all fused layers / adapters)
  unsigned long long wait_ns;             // limit of the wait for t
  unsigned long long* trace;
};

__device__ __forceinline__ uint32_t share_lo(const Share& s, uint32_t i) { return i * s.per + (i < s.rem ? i : s.rem); }
__device__ __forceinline__ uint32_t share_n(const Share& s, uint32_t i) { return s.per + (i < s.rem ? 1u : 0u); }

__device__ __forceinline__ uint4 ld_cg_u4(const void* p) {
  uint4 v;
  asm volatile("ld.global.cg.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ uint32_t pack_h2(float a, float b) {
  __half2 h = __floats2half2_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ uint32_t bf2_to_h2(uint32_t v) {
  return pack_h2(__uint_as_float(v << 16), __uint_as_float(v & 0xffff0000u));
}

// Activation fragments of one pair (128 reduction elements) for lane (g, t): token g, elements
// 64*c + 32*blk + 8*t + [0, 8) in xr[8*c + 4*blk + 0..3].
__device__ __forceinline__ void load_x_pair(uint32_t (&xr)[16], const DecodeArgs& p, uint32_t pair, int lane) {
  const int g = lane >> 2, t = lane & 3;
  if (g < p.m) {
    const uint16_t* src = reinterpret_cast<const uint16_t*>(p.x) + (size_t)g * p.d_in + pair * 128 + 8 * t;
    uint4 u[4];                            // all loads first: a use in between would serialise the round trips
#pragma unroll
    for (int i = 0; i < 4; ++i) u[i] = ld_cg_u4(src + 32 * i);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      uint4 v = u[i];
      if (p.x_dtype == EORA_X_BF16) { v.x = bf2_to_h2(v.x); v.y = bf2_to_h2(v.y); v.z = bf2_to_h2(v.z); v.w = bf2_to_h2(v.w); }
      xr[4 * i] = v.x; xr[4 * i + 1] = v.y; xr[4 * i + 2] = v.z; xr[4 * i + 3] = v.w;
    }
  } else {
#pragma unroll
    for (int i = 0; i < 16; ++i) xr[i] = 0u;
  }
}

// The same for t (fp32 sums in d_t [8][r_pad]), split into high and low fp16 parts.
__device__ __forceinline__ void load_t_pair(uint32_t (&xh)[16], uint32_t (&xl)[16], const DecodeArgs& p, uint32_t pair, int lane) {
  const int g = lane >> 2, t = lane & 3;
  if (p.adp_pairs) {                      // the token takes part only in its own adapter's pairs
    int mine = p.adp[0];
#pragma unroll
    for (int i = 1; i < 8; ++i) if (g == i) mine = p.adp[i];
    if (mine < 0 || (uint32_t)mine != pair / p.adp_pairs) {
#pragma unroll
      for (int i = 0; i < 16; ++i) { xh[i] = 0u; xl[i] = 0u; }
      return;
    }
  }
  const float* src = p.d_t + (size_t)g * p.r_pad + pair * 128 + 8 * t;
  uint4 ua[8];                             // all loads first: a use in between would serialise the round trips
#pragma unroll
  for (int i = 0; i < 8; ++i) ua[i] = ld_cg_u4(src + 32 * (i >> 1) + 4 * (i & 1));
#pragma unroll
  for (int i = 0; i < 4; ++i) {
#pragma unroll
    for (int hq = 0; hq < 2; ++hq) {
      const uint4 u = ua[2 * i + hq];
      const float f[4] = {__uint_as_float(u.x), __uint_as_float(u.y), __uint_as_float(u.z), __uint_as_float(u.w)};
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        const __half h0 = __float2half_rn(f[2 * j]), h1 = __float2half_rn(f[2 * j + 1]);
        const __half2 hi = __halves2half2(h0, h1);
        xh[4 * i + 2 * hq + j] = *reinterpret_cast<const uint32_t*>(&hi);
        xl[4 * i + 2 * hq + j] = pack_h2(f[2 * j] - __half2float(h0), f[2 * j + 1] - __half2float(h1));
      }
    }
  }
}

// red.add under a predicate (no branch: with one token only a quarter of the lanes has something to add,
// and a divergent branch per blob costs more than the adds).
__device__ __forceinline__ void red_add_if(float* p, float v, uint32_t pred) {
  asm volatile("{\n\t.reg .pred q;\n\tsetp.ne.u32 q, %2, 0;\n\t@q red.global.add.f32 [%0], %1;\n\t}" ::"l"(p), "f"(v), "r"(pred) : "memory");
}

// Where a lane's partial sums go: sums[token][ld] for rows 16 * tile + {g, g + 8} and tokens {2t, 2t + 1}.
struct Flush {
  float* base;              // sums + 2t * ld + g
  uint32_t ld;
  uint32_t has0, has1;      // token 2t / 2t + 1 exists
};
__device__ __forceinline__ Flush make_flush(float* sums, int ld, int m, int lane) {
  const int g = lane >> 2, t = lane & 3;
  Flush f;
  f.base = sums + (size_t)(2 * t) * ld + g;
  f.ld = (uint32_t)ld;
  f.has0 = 2 * t < m ? 1u : 0u;
  f.has1 = 2 * t + 1 < m ? 1u : 0u;
  return f;
}
__device__ __forceinline__ void flush_sums(const Flush& f, uint32_t tile, const float (&tot)[4]) {
  float* b = f.base + tile * 16;
  red_add_if(b, tot[0], f.has0); red_add_if(b + 8, tot[2], f.has0);
  red_add_if(b + f.ld, tot[1], f.has1); red_add_if(b + f.ld + 8, tot[3], f.has1);
}

__device__ __forceinline__ uint32_t atom_add_acq_rel(uint32_t* p, uint32_t v) {
  uint32_t old;
  asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(v) : "memory");
  return old;
}
__device__ __forceinline__ void red_add_release(uint32_t* p, uint32_t v) {
  asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// Per-warp state of the copy ring.  All lanes keep the same copy of it; lane 0 issues.
struct Ring {
  uint8_t* slots;
  uint64_t* bars;
  // producer side: the run of blobs still to be requested, over up to three segments
  const uint8_t* ptr[3];
  uint32_t rem[3], blob[3], per[3];
  int pseg;
  // consumer side
  int slot;
  uint32_t phase;           // bit i: parity of the phase that the next copy into slot i completes
  int deferred;             // slots [kRing - deferred, kRing) have not had their first copy requested yet
  uint32_t aux;             // shared-memory address of the 2:4 expansion table (2:4 backbone only)
};

constexpr uint32_t kNone = 0xffffffffu;
__device__ __forceinline__ uint32_t slot_parity(const Ring& r) { return (r.phase >> r.slot) & 1u; }
__device__ __forceinline__ void slot_consumed(Ring& r) {
  r.phase ^= 1u << r.slot;
  if (++r.slot == kRing) r.slot = 0;
}

__device__ __forceinline__ void ring_issue(Ring& r, int slot, int lane) {
  if (r.pseg == 0 && r.rem[0] == 0) r.pseg = 1;
  if (r.pseg == 1 && r.rem[1] == 0) r.pseg = 2;
  if (r.pseg == 2 && r.rem[2] == 0) r.pseg = 3;
  if (r.pseg >= 3) return;
  // runtime-indexed reads of three-element arrays would go to local memory: select instead
  const int s = r.pseg;
  const uint8_t* src = s == 0 ? r.ptr[0] : s == 1 ? r.ptr[1] : r.ptr[2];
  const uint32_t rem = s == 0 ? r.rem[0] : s == 1 ? r.rem[1] : r.rem[2];
  const uint32_t blob = s == 0 ? r.blob[0] : s == 1 ? r.blob[1] : r.blob[2];
  const uint32_t per = s == 0 ? r.per[0] : s == 1 ? r.per[1] : r.per[2];
  const uint32_t n = rem < per ? rem : per;
  const uint32_t bytes = n * blob;
  if (lane == 0) {
    mbar_expect_tx(r.bars + slot, bytes);
    bulk_g2s(r.slots + slot * kSlotBytes, src, bytes, r.bars + slot);
  }
  if (s == 0) { r.ptr[0] = src + bytes; r.rem[0] = rem - n; }
  else if (s == 1) { r.ptr[1] = src + bytes; r.rem[1] = rem - n; }
  else { r.ptr[2] = src + bytes; r.rem[2] = rem - n; }
}

enum { OUT_T = 0, OUT_Y = 1 };

__device__ __forceinline__ void st_zero4(float* p) {
  *reinterpret_cast<float4*>(p) = make_float4(0.f, 0.f, 0.f, 0.f);
}

// Row tile `tile` of the output is complete.  Called by ONE lane (the one whose ticket was the last);
// it converts the tile's 16 x m sums, stores them and puts the scratch back to zero.  Several lanes of a
// warp may each be finishing a tile of their own at the same time.
__device__ __forceinline__ void finish_row_tile(const DecodeArgs& p, uint32_t tile) {
  void* y = p.ys[0];
  uint32_t tile0 = 0;
  int dout = p.sub_dout[0];
#pragma unroll
  for (int i = 1; i < 4; ++i)
    if (i < p.n_sub && tile >= p.sub_tile0[i]) { y = p.ys[i]; tile0 = p.sub_tile0[i]; dout = p.sub_dout[i]; }
  for (int token = 0; token < p.m; ++token) {
    float* s = p.y_ws + (size_t)token * p.n_pad + tile * 16;
    uint4 u[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) u[i] = ld_cg_u4(s + 4 * i);
#pragma unroll
    for (int i = 0; i < 4; ++i) st_zero4(s + 4 * i);
    const float v[16] = {__uint_as_float(u[0].x), __uint_as_float(u[0].y), __uint_as_float(u[0].z), __uint_as_float(u[0].w),
                         __uint_as_float(u[1].x), __uint_as_float(u[1].y), __uint_as_float(u[1].z), __uint_as_float(u[1].w),
                         __uint_as_float(u[2].x), __uint_as_float(u[2].y), __uint_as_float(u[2].z), __uint_as_float(u[2].w),
                         __uint_as_float(u[3].x), __uint_as_float(u[3].y), __uint_as_float(u[3].z), __uint_as_float(u[3].w)};
    const int64_t o = (int64_t)token * dout + (tile - tile0) * 16;   // d_out is a multiple of 32: the 16 outputs exist
    if (p.y_dtype == EORA_Y_F32) {
      float4* dst = reinterpret_cast<float4*>(reinterpret_cast<float*>(y) + o);
#pragma unroll
      for (int i = 0; i < 4; ++i) dst[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
    } else {
      uint32_t h[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        if (p.y_dtype == EORA_Y_F16) {
          h[i] = pack_h2(v[2 * i], v[2 * i + 1]);
        } else {
          const __nv_bfloat162 b = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
          h[i] = *reinterpret_cast<const uint32_t*>(&b);
        }
      }
      uint4* dst = reinterpret_cast<uint4*>(reinterpret_cast<uint16_t*>(y) + o);
      dst[0] = make_uint4(h[0], h[1], h[2], h[3]);
      dst[1] = make_uint4(h[4], h[5], h[6], h[7]);
    }
  }
  p.counters[CNT_TICKET0 + tile] = 0u;
}

// One segment: `n` consecutive blobs of one matrix starting at blob index b0.
// I8M: backbone blobs of a launch with two to eight tokens go through the integer product (blob_product_i8m).
template <int FMT, bool HILO, int OUT, bool I8M = false>
__device__ __forceinline__ bool run_segment(const DecodeArgs& p, Ring& r, uint32_t b0, uint32_t n, uint32_t nt, uint32_t blob_b,
                                            uint32_t per_copy, uint32_t sz2, int lane) {
  if constexpr (FMT == FMT_NONE) {
    return true;
  } else {
    if (n == 0) return true;
    uint32_t pair = b0 / nt, tile = b0 - pair * nt;
    uint32_t xr[16], xl[16];
    XI8M xm;
    const bool x_bf16 = p.x_dtype == EORA_X_BF16;
    uint32_t sub = 0, sub_end = nt;
    Flush fl = OUT == OUT_T ? make_flush(p.d_t, p.r_pad, p.m, lane) : make_flush(p.y_ws, p.n_pad, p.m, lane);
    if constexpr (HILO) {
      // all of A must be in t
      int ok = 1;
      if (lane == 0) ok = counter_wait(p.counters + CNT_A_DONE, p.a_blobs, p.dev_status, p.wait_ns) ? 1 : 0;
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) return false;
      __syncwarp();
      // the activations of B's blob (pair, tile) belong to the layer that owns the row tile
      sub = 0;
#pragma unroll
      for (int i = 1; i < 4; ++i)
        if (i < p.n_sub && tile >= p.sub_tile0[i]) sub = i;
      sub_end = p.sub_tile0[sub + 1];
      load_t_pair(xr, xl, p, sub * p.b_np + pair, lane);
    } else if constexpr (I8M) {
      load_x_i8m<FMT>(xm, p.x, x_bf16, p.m, p.d_in, pair, lane);
    } else {
      load_x_pair(xr, p, pair, lane);
    }
    // The first copies that were held back (see the kernel) go out behind the loads of the activations,
    // not in front of them.
    for (; r.deferred > 0; --r.deferred) ring_issue(r, kRing - r.deferred, lane);
    // Tickets of the blobs flushed so far are taken in batches of up to 32 (one atomic per lane, one
    // round trip per batch): batch_tile is the row tile of the batch's first blob, batch_n its size.
    uint32_t batch_tile = tile, batch_n = 0, flushed = 0;
    auto commit_batch = [&]() {
      __syncwarp();
      uint32_t done = 0, my_tile = 0;
      if ((uint32_t)lane < batch_n) {
        my_tile = (batch_tile + lane) % nt;
        done = atom_add_acq_rel(p.counters + CNT_TICKET0 + my_tile, 1u) + 1u == p.tile_target ? 1u : 0u;
      }
      const uint32_t mask = __ballot_sync(0xffffffffu, done != 0);
      if (mask) {
        // With an adapter the finished row tiles are counted (the count is taken before the tiles are
        // written out, so that the two round trips overlap): the last one restores t and the counters.
        uint32_t last = 0;
        if (p.a_blobs && lane == 0)
          last = atom_add_acq_rel(p.counters + CNT_TILES_DONE, (uint32_t)__popc(mask)) + __popc(mask) == p.w_nt ? 1u : 0u;
        if (done) finish_row_tile(p, my_tile);
        last = __shfl_sync(0xffffffffu, last, 0);
        if (last) {                               // the whole layer is done: nobody reads t any more
          for (int i = lane; i < 8 * p.r_pad / 4; i += 32) st_zero4(p.d_t + 4 * i);
          if (lane == 0) { p.counters[CNT_A_DONE] = 0u; p.counters[CNT_TILES_DONE] = 0u; }
        }
      }
      batch_n = 0;
    };
    while (n > 0) {
      const uint32_t cn = n < per_copy ? n : per_copy;
      if (!mbar_wait_warp(r.bars + r.slot, slot_parity(r), p.dev_status, lane)) return false;
      const uint8_t* src = r.slots + r.slot * kSlotBytes;
#pragma unroll 2
      for (uint32_t j = 0; j < cn; ++j) {
        float tot[4];
        if constexpr (I8M) blob_product_i8m<FMT>(src + j * blob_b, lane, sz2, xm, tot);
        else blob_product<FMT, HILO>(src + j * blob_b, lane, sz2, xr, xl, tot, r.aux);
        if constexpr (OUT == OUT_T) {
          flush_sums(fl, tile, tot);
          ++flushed;
        } else {
          if (batch_n == 0) batch_tile = tile;
          flush_sums(fl, tile, tot);
          if (++batch_n == 32) commit_batch();
        }
        if (++tile == nt) {
          tile = 0;
          ++pair;
          if (j + 1 < cn || n > cn) {
            if constexpr (HILO) {
              sub = 0; sub_end = p.sub_tile0[1];
              load_t_pair(xr, xl, p, pair, lane);
            } else if constexpr (I8M) {
              load_x_i8m<FMT>(xm, p.x, x_bf16, p.m, p.d_in, pair, lane);
            } else {
              load_x_pair(xr, p, pair, lane);
            }
          }
        } else if constexpr (HILO) {
          if (tile == sub_end && (j + 1 < cn || n > cn)) {      // the next row tile belongs to the next fused layer
            ++sub;
            sub_end = p.sub_tile0[sub + 1];
            load_t_pair(xr, xl, p, sub * p.b_np + pair, lane);
          }
        }
      }
      __syncwarp();                               // every lane is done with the slot
      ring_issue(r, r.slot, lane);
      slot_consumed(r);
      n -= cn;
    }
    if constexpr (OUT == OUT_T) {
      __syncwarp();
      if (lane == 0) red_add_release(p.counters + CNT_A_DONE, flushed);
    } else {
      if (batch_n) commit_batch();
    }
    return true;
  }
}

// The backbone share of a single-token launch (integer inner product): the same walk as run_segment, written for
// instruction count -- this loop is what bounds the kernel (a warp retires an instruction every ~10 cycles, and every
// instruction around the product of a blob costs as much as one inside it): running addresses instead of index
// arithmetic, the group layout as a compile-time constant, runs of blobs without a branch in between.
struct WalkI8 {
  XI8 xi;
  uint32_t pair, tile;          // the next blob; pair == kNone: no activations loaded yet
  uint32_t next_b;              // its index (to tell whether the next run continues this one)
  float* yb;
  uint32_t batch_n, my_tile;    // blobs added but without a ticket yet; lane i < batch_n: the row tile of the i-th
  uint32_t tk_old, tk_tile, tk_n;   // tickets asked for (lane i: the one of the batch's blob i), not looked at yet
};

// The tickets asked for last time: whoever holds a row tile's last one finishes the tile.
__device__ __forceinline__ void tickets_resolve(const DecodeArgs& p, WalkI8& w, int lane) {
  if (w.tk_n == 0) return;
  const uint32_t done = ((uint32_t)lane < w.tk_n && w.tk_old + 1u == p.tile_target) ? 1u : 0u;
  const uint32_t mask = __ballot_sync(0xffffffffu, done != 0);
  if (mask) {
    // With an adapter the finished row tiles are counted (before they are written out, so that the two round
    // trips overlap): the last one restores t and the counters.
    uint32_t last = 0;
    if (p.a_blobs && lane == 0)
      last = atom_add_acq_rel(p.counters + CNT_TILES_DONE, (uint32_t)__popc(mask)) + __popc(mask) == p.w_nt ? 1u : 0u;
    if (done) finish_row_tile(p, w.tk_tile);
    last = __shfl_sync(0xffffffffu, last, 0);
    if (last) {
      for (int i = lane; i < 8 * p.r_pad / 4; i += 32) st_zero4(p.d_t + 4 * i);
      if (lane == 0) { p.counters[CNT_A_DONE] = 0u; p.counters[CNT_TILES_DONE] = 0u; }
    }
  }
  w.tk_n = 0;
}
// Tickets for the blobs added since the last batch (the release in front of them waits for the warp's additions
// to arrive, which is why they are not taken more often than every 32 blobs).  The answers are looked at one batch later: nothing waits for
// the round trip.
__device__ __forceinline__ void tickets_take(const DecodeArgs& p, WalkI8& w, int lane) {
  tickets_resolve(p, w, lane);
  if (w.batch_n == 0) return;
  __syncwarp();
  if ((uint32_t)lane < w.batch_n) {
    w.tk_tile = w.my_tile;
    w.tk_old = atom_add_acq_rel(p.counters + CNT_TICKET0 + w.my_tile, 1u);
  }
  w.tk_n = w.batch_n;
  w.batch_n = 0;
}

// The next blobs are b0, b0 + 1, ...
template <int FMT>
__device__ __forceinline__ void walk_seek(const DecodeArgs& p, WalkI8& w, uint32_t b0, int lane) {
  if (b0 == w.next_b && w.pair != kNone) return;
  const uint32_t pair = b0 / p.w_nt;
  w.tile = b0 - pair * p.w_nt;
  w.next_b = b0;
  w.yb = p.y_ws + (lane >> 2) + w.tile * 16;
  if (pair != w.pair) load_x_i8<FMT>(w.xi, p.x, p.x_dtype == EORA_X_BF16, pair, lane);
  w.pair = pair;
}

// cn blobs in shared memory at bp; more: blobs follow after these (then the activations of the next pair are
// fetched when these end a pair).
template <int FMT, bool SZ2>
__device__ __forceinline__ void walk_blobs(const DecodeArgs& p, WalkI8& w, const uint8_t* bp, uint32_t cn, bool more, int lane) {
  constexpr uint32_t blob_b = blob_bytes(FMT, SZ2 ? 1 : 0);
  const uint32_t nt = p.w_nt;
  const uint32_t owner = (lane & 3) == 0 ? 1u : 0u;
  const uint8_t* bl = bp + (FMT == FMT_Q4 ? 16 : 8) * lane;
  const uint8_t* bg = bp + 4 * (lane >> 2);
  w.next_b += cn;
  for (uint32_t left = cn; left > 0;) {
    // a run of blobs without a change of pair and without a ticket batch filling up: nothing but products and adds
    uint32_t run = min(left, min(nt - w.tile, 32u - w.batch_n));
    if ((uint32_t)lane - w.batch_n < run) w.my_tile = w.tile + ((uint32_t)lane - w.batch_n);
    left -= run; w.tile += run; w.batch_n += run;
#pragma unroll 2
    for (; run > 0; --run, bl += blob_b, bg += blob_b, w.yb += 16) {
      float t2[2];
      blob_product_i8<FMT, SZ2>(bl, bg, lane, w.xi, t2);
      red_add_if(w.yb, t2[0], owner);
      red_add_if(w.yb + 8, t2[1], owner);
    }
    if (w.tile == nt) {                                 // next pair of reduction elements: other activations
      w.tile = 0; ++w.pair; w.yb = p.y_ws + (lane >> 2);
      if (left > 0 || more) load_x_i8<FMT>(w.xi, p.x, p.x_dtype == EORA_X_BF16, w.pair, lane);
      else w.pair = kNone;
    }
    if (w.batch_n == 32) tickets_take(p, w, lane);
  }
}

// n blobs from b0 on, dealt to this warp ahead of time.
template <int FMT, bool SZ2>
__device__ __forceinline__ bool run_backbone_i8(const DecodeArgs& p, Ring& r, WalkI8& w, uint32_t b0, uint32_t n, int lane) {
  if (n == 0) return true;
  walk_seek<FMT>(p, w, b0, lane);
  for (; r.deferred > 0; --r.deferred) ring_issue(r, kRing - r.deferred, lane);
  while (n > 0) {
    const uint32_t cn = n < p.w_per_copy ? n : p.w_per_copy;
    if (!mbar_wait_warp(r.bars + r.slot, slot_parity(r), p.dev_status, lane)) return false;
    walk_blobs<FMT, SZ2>(p, w, r.slots + r.slot * kSlotBytes, cn, n > cn, lane);
    __syncwarp();                                       // every lane is done with the slot
    ring_issue(r, r.slot, lane);
    slot_consumed(r);
    n -= cn;
  }
  return true;
}

template <int WF, int I8>
__device__ __forceinline__ bool run_backbone(const DecodeArgs& p, Ring& r, WalkI8& w, uint32_t first, uint32_t count, uint32_t blob_w, int lane) {
  if constexpr (I8 == 2) {
    return run_segment<WF, false, OUT_Y, true>(p, r, first, count, p.w_nt, blob_w, p.w_per_copy, p.w_sz2, lane);
  } else if constexpr (I8 == 1) {
    return p.w_sz2 ? run_backbone_i8<WF, true>(p, r, w, first, count, lane) : run_backbone_i8<WF, false>(p, r, w, first, count, lane);
  } else {
    return run_segment<WF, false, OUT_Y>(p, r, first, count, p.w_nt, blob_w, p.w_per_copy, p.w_sz2, lane);
  }
}

// I8: the backbone goes through the integer inner product -- 1: one token (the walk above), 2: two to eight tokens
// (tokens as the columns of the narrow operand, two byte planes = two MMAs per weight fragment), 0: fp16 product.
template <int WF, int ABF, int I8>
__global__ void __launch_bounds__(kThreads, kCtasPerSm) k_decode(const __grid_constant__ DecodeArgs p) {
  extern __shared__ __align__(128) uint8_t smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // Position in the deal.  Neighbours in the deal sit on different SMs, so that the few warps that hold A (whose sums
  // everybody's B share waits for) work in parallel on many SMs: the A owners are dealt warp by warp over the first
  // half of the CTAs, the B owners over the second half, and the warps left over are numbered after them.  No CTA
  // holds both kinds: the CTAs with A owners are dispatched first and never wait, so a waiting warp never holds the
  // place of a CTA that it is waiting for.
  uint32_t gw;
  {
    const uint32_t ca = gridDim.x / 2, cb = gridDim.x - ca, n3 = gridDim.x * kWarps - p.n12;
    if (blockIdx.x < ca) {
      gw = warp * ca + blockIdx.x;                                    // < n1: an A owner
    } else {
      const uint32_t rid = warp * cb + (blockIdx.x - ca);
      gw = rid < n3 ? p.n12 + rid : p.n1 + (kWarps * ca - p.n1) + (rid - n3);
    }
  }
  asm volatile("griddepcontrol.launch_dependents;");
  unsigned long long* tr = p.trace ? p.trace + (size_t)(blockIdx.x * kWarps + warp) * 4 : nullptr;
  if (tr && lane == 0) tr[0] = globaltimer_ns();

  Ring r;
  r.slots = smem + warp * (kRing * kSlotBytes);
  r.bars = reinterpret_cast<uint64_t*>(smem + kWarps * kRing * kSlotBytes) + warp * kRing;
  r.slot = 0; r.phase = 0; r.pseg = 0;
  r.aux = 0;
  if constexpr (WF == FMT_SP24 || WF == FMT_SQ4) {
    // every warp writes the same 16 values, so no CTA-wide barrier is needed before a warp reads them
    uint32_t* lut = reinterpret_cast<uint32_t*>(smem + kWarps * kRing * kSlotBytes + kBarBytes);
    if (lane < 16) lut[lane] = sp24_selectors((uint32_t)lane);
    r.aux = smem_u32(lut);
  }
  if (lane == 0) {
#pragma unroll
    for (int i = 0; i < kRing; ++i) mbar_init(r.bars + i, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncwarp();

  // this warp's three runs: A, W, B (one of A / B is empty)
  const bool a_owner = gw < p.n1, b_owner = gw >= p.n12;
  uint32_t a0 = 0, an = 0, w0, wn, bb0 = 0, bn = 0;
  if (a_owner) {
    a0 = share_lo(p.sh_a, gw); an = share_n(p.sh_a, gw);
    w0 = p.w_base[0] + share_lo(p.sh_w[0], gw); wn = share_n(p.sh_w[0], gw);
  } else if (!b_owner) {
    const uint32_t i = gw - p.n1;
    w0 = p.w_base[1] + share_lo(p.sh_w[1], i); wn = share_n(p.sh_w[1], i);
  } else {
    const uint32_t i = gw - p.n12;
    w0 = p.w_base[2] + share_lo(p.sh_w[2], i); wn = share_n(p.sh_w[2], i);
    bb0 = share_lo(p.sh_b, i); bn = share_n(p.sh_b, i);
  }
  const uint32_t blob_a = blob_bytes(ABF, p.a_sz2), blob_w = blob_bytes(WF, p.w_sz2), blob_b = blob_bytes(ABF, p.b_sz2);
  // Order of the runs.  A owners: A, then W.  The others: the first copy's worth of W, then B, then the
  // rest of W: by then t is complete, and the round trips of the B share (reading t back, its tickets)
  // are hidden behind the other warps' W work instead of sitting at the end of the kernel.
  const uint32_t wf = !b_owner ? wn : (wn < p.w_per_copy ? wn : p.w_per_copy);
  if (!b_owner) {
    r.ptr[0] = p.a_q + (size_t)a0 * blob_a; r.rem[0] = an; r.blob[0] = blob_a; r.per[0] = p.a_per_copy;
    r.ptr[1] = p.w_q + (size_t)w0 * blob_w; r.rem[1] = wn; r.blob[1] = blob_w; r.per[1] = p.w_per_copy;
    r.ptr[2] = p.w_q; r.rem[2] = 0; r.blob[2] = blob_w; r.per[2] = p.w_per_copy;
  } else {
    r.ptr[0] = p.w_q + (size_t)w0 * blob_w; r.rem[0] = wf; r.blob[0] = blob_w; r.per[0] = p.w_per_copy;
    r.ptr[1] = p.b_q + (size_t)bb0 * blob_b; r.rem[1] = bn; r.blob[1] = blob_b; r.per[1] = p.b_per_copy;
    r.ptr[2] = p.w_q + (size_t)(w0 + wf) * blob_w; r.rem[2] = wn - wf; r.blob[2] = blob_w; r.per[2] = p.w_per_copy;
  }

  // Before the dependency resolves at most two first copies per warp are requested (with a deeper ring the others
  // follow the loads of the activations, which are read right after the wait and would otherwise queue behind the
  // weight requests).
  ring_issue(r, 0, lane);
  ring_issue(r, 1, lane);
  r.deferred = kRing - 2;

  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (tr && lane == 0) tr[1] = globaltimer_ns();

  WalkI8 wk;
  if constexpr (I8 == 1) {
    wk.pair = kNone; wk.next_b = kNone; wk.tile = 0; wk.yb = p.y_ws; wk.my_tile = 0; wk.batch_n = 0; wk.tk_n = 0; wk.tk_old = 0; wk.tk_tile = 0;
  }
  bool ok = true;
  if (a_owner) ok = run_segment<ABF, false, OUT_T>(p, r, a0, an, p.a_nt, blob_a, p.a_per_copy, p.a_sz2, lane);
  if (ok) ok = run_backbone<WF, I8>(p, r, wk, w0, wf, blob_w, lane);
  if (tr && lane == 0) tr[2] = globaltimer_ns();
  if (b_owner) {
    if (ok) ok = run_segment<ABF, true, OUT_Y>(p, r, bb0, bn, p.w_nt, blob_b, p.b_per_copy, p.b_sz2, lane);
    if (ok) ok = run_backbone<WF, I8>(p, r, wk, w0 + wf, wn - wf, blob_w, lane);
  }
  if constexpr (I8 == 1) {
    if (ok) { tickets_take(p, wk, lane); tickets_resolve(p, wk, lane); }
  }
  if (!ok) {
    // This warp gave up: its bulk copies still in flight must land before the CTA's shared memory may be reused.  A slot
    // of the ring is in flight exactly if a copy was requested for it and not consumed: slots from the consumer position on
    // waits for the phase its next copy completes; a slot without a copy in flight runs into the drain's short limit.
    for (int i = 0; i < kRing - r.deferred; ++i) mbar_drain_warp(r.bars + i, (r.phase >> i) & 1u, lane);
  }
  if (tr && lane == 0) tr[3] = globaltimer_ns();
}

template <auto KERNEL>
cudaError_t launch_kernel(const cudaLaunchConfig_t& cfg, const DecodeArgs& args, int device) {
  static bool attr_set[64] = {};  // per kernel (KERNEL is a template argument) and device: the attribute belongs to the current device
  if (device < 0 || device >= 64) return cudaErrorInvalidDevice;
  if (!attr_set[device]) {
    cudaError_t e = cudaFuncSetAttribute(KERNEL, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    attr_set[device] = true;
  }
  return cudaLaunchKernelEx(&cfg, KERNEL, args);
}

// Formats whose backbone blobs have an integer inner product.
constexpr bool has_i8(int fmt) { return fmt == FMT_Q4 || fmt == FMT_Q3; }

template <int WF, int I8>
cudaError_t launch_ab2(const cudaLaunchConfig_t& cfg, const DecodeArgs& args, int abf, int device) {
  switch (abf) {
    case FMT_F16: return launch_kernel<k_decode<WF, FMT_F16, I8>>(cfg, args, device);
    case FMT_Q4: return launch_kernel<k_decode<WF, FMT_Q4, I8>>(cfg, args, device);
    case FMT_Q8: return launch_kernel<k_decode<WF, FMT_Q8, I8>>(cfg, args, device);
    case FMT_Q3: return launch_kernel<k_decode<WF, FMT_Q3, I8>>(cfg, args, device);
    default: return launch_kernel<k_decode<WF, FMT_NONE, I8>>(cfg, args, device);
  }
}
template <int WF>
cudaError_t launch_ab(const cudaLaunchConfig_t& cfg, const DecodeArgs& args, int abf, int device) {
  if constexpr (has_i8(WF)) {
    if (args.m == 1) return launch_ab2<WF, 1>(cfg, args, abf, device);
    return launch_ab2<WF, 2>(cfg, args, abf, device);
  }
  return launch_ab2<WF, 0>(cfg, args, abf, device);
}

// Relative cost of one blob (time a warp spends on it); only the ratios matter.
double blob_cost(int fmt, bool hilo) {
  switch (fmt) {
    case FMT_Q3: return 1.00;
    case FMT_Q4: return 1.05;
    case FMT_Q8: return 1.40;
    case FMT_F16: return hilo ? 1.30 : 1.10;
    case FMT_SP24: return 1.60;
    case FMT_SQ4: return 1.10;
    default: return 0.0;
  }
}

Share make_share(uint32_t total, uint32_t n) {
  Share s;
  s.per = n ? total / n : 0;
  s.rem = n ? total % n : 0;
  return s;
}

uint32_t blobs_per_copy(const WMat& m) {
  int n = kSlotBytes / m.blob;
  return (uint32_t)(n < 1 ? 1 : n);
}

}  // namespace

// One thread waits, bounded by the handle's limit, for a count that nobody raises, after leaving the kind of debris a
// kernel that gives up leaves behind (a partial sum, a partial t, a ticket).  See eora_linear_selftest_wait_timeout.
__global__ void k_wait_selftest(uint32_t* counters, float* y_ws, float* d_t, int* dev_status, unsigned long long limit_ns) {
  if (threadIdx.x == 0) {
    y_ws[0] += 1.f;
    d_t[0] += 1.f;
    counters[CNT_TICKET0] += 1u;
    dec::counter_wait(counters + CNT_A_DONE, 0xffffffffu, dev_status, limit_ns);
  }
}

cudaError_t launch_wait_selftest(const Handle* h, cudaStream_t st) {
  k_wait_selftest<<<1, 32, 0, st>>>(h->counters, h->y_ws, h->d_t, h->dev_status, h->wait_limit_ns);
  return cudaGetLastError();
}

bool decode_supported(const Handle* h, int m) {
  if (m < 1 || m > 64) return false;
  if (h->sm_count < 2) return false;
  if (h->w.fmt != FMT_Q4 && h->w.fmt != FMT_Q3 && h->w.fmt != FMT_SP24 && h->w.fmt != FMT_SQ4) return false;
  if (h->w.blob > kSlotBytes) return false;
  if (h->cfg.rank > 0 && (h->a.blob > kSlotBytes || h->b.blob > kSlotBytes)) return false;
  return true;
}

int decode_launch_count(const Handle*, int m) { return (m + 7) / 8; }

int decode_grid(const Handle* h, int m) {
  const bool i8 = m == 1 && (h->w.fmt == FMT_Q4 || h->w.fmt == FMT_Q3);
  (void)i8;
  return h->sm_count * kCtasPerSm;
}

cudaError_t launch_decode_forward(const Handle* h, const void* x, int m, void* const* ys, cudaStream_t st,
                                  const int32_t* adapter_ids) {
  const bool ab = h->cfg.rank > 0;
  DecodeArgs a = {};
  a.w_q = h->w.q; a.w_nt = h->w.nt; a.w_sz2 = h->w.sz2; a.w_per_copy = blobs_per_copy(h->w);
  const uint32_t w_blobs = (uint32_t)h->w.np * h->w.nt;
  uint32_t b_blobs = 0;
  if (ab) {
    a.a_q = h->a.q; a.a_nt = h->a.nt; a.a_sz2 = h->a.sz2; a.a_per_copy = blobs_per_copy(h->a);
    a.b_q = h->b.q; a.b_sz2 = h->b.sz2; a.b_per_copy = blobs_per_copy(h->b);
    a.a_blobs = (uint32_t)h->a.np * h->a.nt;
    b_blobs = (uint32_t)h->b.np * h->b.nt;
  } else {
    a.a_nt = 1; a.a_per_copy = 1; a.b_per_copy = 1;
  }
  const int grid = decode_grid(h, m);
  const uint32_t nw = (uint32_t)grid * kWarps;
  if (ab) {
    // with one token the backbone blobs go through the integer inner product, which is cheaper
    const bool i8 = h->w.fmt == FMT_Q4 || h->w.fmt == FMT_Q3;       // (one to eight tokens: this function's passes)
    // at most a sixth of the warps hold A, a sixth B (measured on the whole block: a third of each 1.4 % slower, an
    // eighth 2 % slower)
    uint32_t n1 = a.a_blobs < nw / 6 ? a.a_blobs : nw / 6;
    uint32_t n3 = b_blobs < nw / 6 ? b_blobs : nw / 6;
    if (n1 < 1) n1 = 1;
    if (n3 < 1) n3 = 1;
    // the A owners sit in the first half of the CTAs, the B owners in the second (see the kernel)
    if (n1 > (uint32_t)(grid / 2) * kWarps) n1 = (uint32_t)(grid / 2) * kWarps;
    if (n3 > (uint32_t)(grid - grid / 2) * kWarps) n3 = (uint32_t)(grid - grid / 2) * kWarps;
    const uint32_t n2 = nw - n1 - n3;
    // Deal the blobs so that every warp gets the same estimated time.  Costs are in units of one backbone
    // blob on the tensor-core path.  Besides its blobs of A or B a warp of the first or third group has a
    // fixed extra cost: the A owners fetch a second set of activations, the B owners read t back and end
    // with their own round of tickets, which is latency that a warp cannot hide from itself.
    const double cw1 = blob_cost(h->w.fmt, false) * (i8 ? 0.75 : 1.0);
    const double fixed_a = i8 ? 4.0 : 2.0, fixed_b = 9.0;
    const double e1 = fixed_a + (double)a.a_blobs / n1 * blob_cost(h->a.fmt, false);
    const double e3 = fixed_b + (double)b_blobs / n3 * blob_cost(h->b.fmt, true);
    const double T = (w_blobs * cw1 + n1 * e1 + n3 * e3) / nw;      // finishing time of every warp
    double W1 = T > e1 ? n1 * (T - e1) / cw1 : 0.0, W3 = T > e3 ? n3 * (T - e3) / cw1 : 0.0;
    if (W1 + W3 > w_blobs) { const double f = w_blobs / (W1 + W3); W1 *= f; W3 *= f; }
    const uint32_t w1 = (uint32_t)W1, w3 = (uint32_t)W3, w2 = w_blobs - w1 - w3;
    a.n1 = n1; a.n12 = n1 + n2;
    a.sh_a = make_share(a.a_blobs, n1);
    a.sh_b = make_share(b_blobs, n3);
    a.sh_w[0] = make_share(w1, n1); a.sh_w[1] = make_share(w2, n2); a.sh_w[2] = make_share(w3, n3);
    a.w_base[0] = 0; a.w_base[1] = w1; a.w_base[2] = w1 + w2;
  } else {
    a.n1 = 0; a.n12 = nw;
    a.sh_a = make_share(0, 0);
    a.sh_b = make_share(0, 0);
    a.sh_w[0] = make_share(0, 0); a.sh_w[1] = make_share(w_blobs, nw); a.sh_w[2] = make_share(0, 0);
    a.w_base[0] = 0; a.w_base[1] = 0; a.w_base[2] = w_blobs;
  }
  a.tile_target = (uint32_t)h->w.np + (ab ? (uint32_t)h->b.np : 0u);
  a.d_t = h->d_t; a.y_ws = h->y_ws; a.counters = h->counters; a.dev_status = h->dev_status;
  a.d_in = h->cfg.d_in; a.r_pad = h->t_cols; a.n_pad = h->w.n_rows;
  a.n_sub = h->n_sub;
  a.b_np = ab ? (uint32_t)h->b.np : 0u;
  for (int i = 0; i <= h->n_sub; ++i) a.sub_tile0[i] = (uint32_t)h->sub_tile0[i];
  for (int i = h->n_sub + 1; i < 5; ++i) a.sub_tile0[i] = (uint32_t)h->w.nt;
  for (int i = 0; i < 4; ++i) a.sub_dout[i] = i < h->n_sub ? h->sub_dout[i] : 0;
  a.x_dtype = h->cfg.x_dtype; a.y_dtype = h->cfg.y_dtype;
  a.trace = reinterpret_cast<unsigned long long*>(h->trace);
  a.wait_ns = h->wait_limit_ns;

  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = kSmemBytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const int abf = ab ? h->a.fmt : FMT_NONE;
  const size_t ybytes = h->cfg.y_dtype == EORA_Y_F32 ? 4 : 2;
  for (int m0 = 0; m0 < m; m0 += 8) {             // eight tokens per pass (the n8 side of the mma)
    a.m = m - m0 < 8 ? m - m0 : 8;
    a.x = reinterpret_cast<const uint8_t*>(x) + (size_t)m0 * h->cfg.d_in * 2;
    for (int i = 0; i < h->n_sub; ++i) a.ys[i] = reinterpret_cast<uint8_t*>(ys[i]) + (size_t)m0 * h->sub_dout[i] * ybytes;
    a.adp_pairs = 0;
    if (h->multi) {
      a.adp_pairs = (uint32_t)h->r_pad / 128;
      for (int i = 0; i < 8; ++i) {
        const int id = (adapter_ids && m0 + i < m) ? adapter_ids[m0 + i] : -1;
        a.adp[i] = (id >= 0 && id < h->n_adapters) ? id : -1;
      }
    }
    cudaError_t e = h->w.fmt == FMT_Q4 ? launch_ab<FMT_Q4>(cfg, a, abf, h->device)
                  : h->w.fmt == FMT_Q3 ? launch_ab<FMT_Q3>(cfg, a, abf, h->device)
                  : h->w.fmt == FMT_SQ4 ? launch_ab<FMT_SQ4>(cfg, a, abf, h->device) : launch_ab<FMT_SP24>(cfg, a, abf, h->device);
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

}  // namespace eora
