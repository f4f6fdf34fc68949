// Decode kernel family (M <= 64): one launch computes  Y = X.deq(Wq) + (X.A).B  (paper Eq. 4).
//
// Section 4.5 of the paper fuses only the product with B into the quantised mat-vec kernel and
// leaves t = A.x to a separate op.  Here the whole layer is one pass: A is treated as `rank`
// more output rows of the same streaming product over X, and B as `rank` more reduction
// elements of the backbone product with t in the place of X, so Y is written exactly once.
//
// Work decomposition.  A CTA (8 warps) owns one unit = (matrix, 16-row tile, reduction slice).
// Units of A come first in blockIdx order, backbone units after them.  Inside a unit each warp
// streams whole quantisation quanta (<= 128 reduction elements sharing one scale / zero-point)
// of packed weights with 128-bit loads, turns the codes into exact fp16 integers (q - z) in
// registers, multiplies them with the activations on the tensor cores (mma.m16n8k16, weights as
// the 16-row operand, fp32 accumulate) and applies the scale once per quantum in fp32.
// The 8 warps are then summed through shared memory.
//   A unit       : adds its partial t to the fp32 buffer t_ws (red.add), then bumps T_DONE.
//   backbone unit: the last reduction slice of each row tile also owns the B extension: it waits
//                  (bounded) for T_DONE, reads t, splits it into fp16 hi + lo parts and runs the
//                  B tiles against them.  With one slice per row tile the result goes straight
//                  to Y; otherwise slices add into y_ws and the last one to arrive converts.
// All scratch words are returned to zero before the kernel ends, so calls need no memset.
//
// Programmatic dependent launch: the first batch of weight loads is issued before
// griddepcontrol.wait, i.e. while the previous kernel in the stream is still draining;
// activations and scratch are touched only after it.
#include "eora_common.cuh"

namespace eora {
namespace {

constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;
constexpr int kXPad = 32;                // halves of padding per activation row in shared memory
constexpr int kXSmemBudget = 64 * 1024;  // bytes of staged activations per CTA
constexpr uint32_t kSpinLimit = 1u << 21;

enum { CNT_T_DONE = 0, CNT_T_CONSUMED = 1, CNT_TILE0 = 2 };

// ------------------------------------------------------------------------------------------ loads
__device__ __forceinline__ uint4 ldg_stream(const uint4* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ uint2 ldg_stream(const uint2* p) {
  uint2 v;
  asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
  return v;
}
__device__ __forceinline__ uint32_t ldg_stream(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.global.nc.L1::no_allocate.u32 %0, [%1];" : "=r"(v) : "l"(p));
  return v;
}
__device__ __forceinline__ uint32_t ld_acquire(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ float ld_cg(const float* p) {
  float v;
  asm volatile("ld.global.cg.f32 %0, [%1];" : "=f"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void red_add(float* p, float v) {
  asm volatile("red.global.add.f32 [%0], %1;" ::"l"(p), "f"(v) : "memory");
}

template <int FMT> struct TileRegs;
template <> struct TileRegs<FMT_Q4> { uint4 v; };
template <> struct TileRegs<FMT_Q3> { uint2 v; uint32_t w2; };
template <> struct TileRegs<FMT_Q8> { uint4 v[2]; };
template <> struct TileRegs<FMT_F16> { uint4 v[4]; };
template <> struct TileRegs<FMT_NONE> { int unused; };

template <int FMT>
__device__ __forceinline__ void tile_load(TileRegs<FMT>& r, const WMat& m, int64_t ti, int lane) {
  if constexpr (FMT == FMT_Q4) {
    r.v = ldg_stream(reinterpret_cast<const uint4*>(m.q) + ti * 32 + lane);
  } else if constexpr (FMT == FMT_Q3) {
    r.v = ldg_stream(reinterpret_cast<const uint2*>(m.q) + ti * 32 + lane);
    r.w2 = ldg_stream(m.q2 + ti * 32 + lane);
  } else if constexpr (FMT == FMT_Q8) {
    r.v[0] = ldg_stream(reinterpret_cast<const uint4*>(m.q) + (ti * 2 + 0) * 32 + lane);
    r.v[1] = ldg_stream(reinterpret_cast<const uint4*>(m.q) + (ti * 2 + 1) * 32 + lane);
  } else if constexpr (FMT == FMT_F16) {
#pragma unroll
    for (int p = 0; p < 4; ++p) r.v[p] = ldg_stream(reinterpret_cast<const uint4*>(m.q) + (ti * 4 + p) * 32 + lane);
  }
}

// ------------------------------------------------------------------------------------------ dequant
__device__ __forceinline__ uint32_t h2sub(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("sub.f16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}
__device__ __forceinline__ uint32_t h2fma(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t d;
  asm("fma.rn.f16x2 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}

// Per-quantum constants of the two rows a lane owns: fp16x2 values that turn the magic-number
// form of a code into the exact integer q - z.
struct ZC { uint32_t c[2][3]; };

template <int FMT>
__device__ __forceinline__ void make_zc(ZC& zc, uint32_t zz) {
#pragma unroll
  for (int hf = 0; hf < 2; ++hf) {
    uint32_t z = (zz >> (8 * hf)) & 255u;
    zc.c[hf][0] = (0x6400u | z) * 0x00010001u;                                      //  1024 + z
    if constexpr (FMT == FMT_Q4) zc.c[hf][1] = (0xD400u | (z << 4)) * 0x00010001u;   // -(64 + z)
    if constexpr (FMT == FMT_Q3) {
      zc.c[hf][1] = (0xD800u | (z << 3)) * 0x00010001u;                              // -(128 + z)
      zc.c[hf][2] = (0xCC00u | (z << 6)) * 0x00010001u;                              // -(16 + z)
    }
  }
}

constexpr uint32_t kMagic = 0x64006400u;   // fp16x2 (1024, 1024)

// a[i][*]: the A-operand registers of mma i (i = 2*blk + sub) for this lane; entries are fp16x2.
template <int FMT>
__device__ __forceinline__ void tile_frags(const TileRegs<FMT>& r, const ZC& zc, uint32_t (&a)[4][4]) {
  if constexpr (FMT == FMT_Q4) {
    const uint32_t w[4] = {r.v.x, r.v.y, r.v.z, r.v.w};
#pragma unroll
    for (int part = 0; part < 4; ++part) {
      const int hf = part & 1, blk = part >> 1;
      uint32_t lo = w[part], hi = w[part] >> 8;
      uint32_t h0 = (lo & 0x000f000fu) | kMagic, h1 = (lo & 0x00f000f0u) | kMagic;
      uint32_t h2 = (hi & 0x000f000fu) | kMagic, h3 = (hi & 0x00f000f0u) | kMagic;
      a[blk * 2 + 0][hf] = h2sub(h0, zc.c[hf][0]);
      a[blk * 2 + 0][hf + 2] = h2fma(h1, 0x2C002C00u, zc.c[hf][1]);   // * 1/16
      a[blk * 2 + 1][hf] = h2sub(h2, zc.c[hf][0]);
      a[blk * 2 + 1][hf + 2] = h2fma(h3, 0x2C002C00u, zc.c[hf][1]);
    }
  } else if constexpr (FMT == FMT_Q3) {
    const uint32_t w[3] = {r.v.x, r.v.y, r.w2};
    const uint32_t ws[3] = {r.v.x >> 9, r.v.y >> 9, r.w2 >> 9};
#pragma unroll
    for (int p = 0; p < 16; ++p) {
      const int part = p >> 2, j = p & 3, hf = part & 1, blk = part >> 1;
      uint32_t v;
      if (p < 15) {
        const int wi = p / 5, f = p % 5, ff = f >= 3 ? f - 3 : f;
        const uint32_t src = f >= 3 ? ws[wi] : w[wi];
        const uint32_t h = (src & (0x00070007u << (3 * ff))) | kMagic;
        if (ff == 0) v = h2sub(h, zc.c[hf][0]);
        else if (ff == 1) v = h2fma(h, 0x30003000u, zc.c[hf][1]);   // * 1/8
        else v = h2fma(h, 0x24002400u, zc.c[hf][2]);                // * 1/64
      } else {
        uint32_t h = ((w[0] >> 15) & 0x00010001u) | kMagic;
        h |= (w[1] >> 14) & 0x00020002u;
        h |= (w[2] >> 13) & 0x00040004u;
        v = h2sub(h, zc.c[hf][0]);
      }
      a[blk * 2 + (j >> 1)][hf + 2 * (j & 1)] = v;
    }
  } else if constexpr (FMT == FMT_Q8) {
#pragma unroll
    for (int part = 0; part < 4; ++part) {
      const int hf = part & 1, blk = part >> 1;
      const uint4 u = r.v[part >> 1];
      const uint32_t w0 = (part & 1) ? u.z : u.x, w1 = (part & 1) ? u.w : u.y;
      a[blk * 2 + 0][hf] = h2sub((w0 & 0x00ff00ffu) | kMagic, zc.c[hf][0]);
      a[blk * 2 + 0][hf + 2] = h2sub(((w0 >> 8) & 0x00ff00ffu) | kMagic, zc.c[hf][0]);
      a[blk * 2 + 1][hf] = h2sub((w1 & 0x00ff00ffu) | kMagic, zc.c[hf][0]);
      a[blk * 2 + 1][hf + 2] = h2sub(((w1 >> 8) & 0x00ff00ffu) | kMagic, zc.c[hf][0]);
    }
  } else if constexpr (FMT == FMT_F16) {
#pragma unroll
    for (int part = 0; part < 4; ++part) {
      const int hf = part & 1, blk = part >> 1;
      a[blk * 2 + 0][hf] = r.v[part].x;
      a[blk * 2 + 0][hf + 2] = r.v[part].y;
      a[blk * 2 + 1][hf] = r.v[part].z;
      a[blk * 2 + 1][hf + 2] = r.v[part].w;
    }
  }
}

__device__ __forceinline__ void mma16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

template <int FMT> constexpr bool is_quant() { return FMT == FMT_Q4 || FMT == FMT_Q3 || FMT == FMT_Q8; }
template <int FMT> constexpr int prefetch_quanta() { return FMT == FMT_F16 ? 2 : 4; }

// Stream the quanta [q0, q1) of row tile `tile` of matrix `m` against NX activation sources held in
// shared memory (source s at xs + s * xsrc_stride; row `token` at + token * xrow; the element for
// reduction index k at + (k - k_base)).  QT = tiles per quantum.  Quanta are dealt round-robin to
// the warps.  `pre` / `have_pre`: the first batch, already loaded by the caller.
template <int FMT, int MT, int QT, int NX>
struct Streamer {
  static constexpr int PF = prefetch_quanta<FMT>();
  TileRegs<FMT> regs[PF][QT];
  uint32_t sc[PF];
  uint32_t zz[PF];

  __device__ __forceinline__ void issue(const WMat& m, int tile, int qfirst, int q1, int warp, int lane) {
#pragma unroll
    for (int j = 0; j < PF; ++j) {
      int qi = qfirst + warp + kWarps * j;
      if (qi < q1) {
#pragma unroll
        for (int tt = 0; tt < QT; ++tt) tile_load<FMT>(regs[j][tt], m, (int64_t)tile * m.kc + (int64_t)qi * QT + tt, lane);
        if constexpr (is_quant<FMT>()) {
          int grp = (qi * QT * 64) / m.group;
          int64_t si = ((int64_t)tile * m.ng + grp) * 8 + (lane >> 2);
          sc[j] = __ldg(m.sc + si);
          zz[j] = __ldg(m.zz + si);
        }
      }
    }
  }

  __device__ __forceinline__ void compute(int qfirst, int q1, int warp, int lane, const __half* xs, int xrow,
                                          int xsrc_stride, int k_base, int m_rows, float (&acc)[MT][4]) {
    const int g = lane >> 2, t = lane & 3;
#pragma unroll
    for (int j = 0; j < PF; ++j) {
      int qi = qfirst + warp + kWarps * j;
      if (qi < q1) {
        float gacc[MT][4];
        if constexpr (is_quant<FMT>()) {
#pragma unroll
          for (int mt = 0; mt < MT; ++mt) { gacc[mt][0] = gacc[mt][1] = gacc[mt][2] = gacc[mt][3] = 0.f; }
        }
        ZC zc;
        if constexpr (is_quant<FMT>()) make_zc<FMT>(zc, zz[j]);
#pragma unroll
        for (int tt = 0; tt < QT; ++tt) {
          uint32_t a[4][4];
          tile_frags<FMT>(regs[j][tt], zc, a);
          const int koff = (qi * QT + tt) * 64 - k_base + 8 * t;
#pragma unroll
          for (int s = 0; s < NX; ++s) {
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
              const int token = mt * 8 + g;
              uint4 x0 = make_uint4(0, 0, 0, 0), x1 = make_uint4(0, 0, 0, 0);
              if (token < m_rows) {
                const __half* p = xs + s * xsrc_stride + token * xrow + koff;
                x0 = *reinterpret_cast<const uint4*>(p);
                x1 = *reinterpret_cast<const uint4*>(p + 32);
              }
              float(&d)[4] = is_quant<FMT>() ? gacc[mt] : acc[mt];
              mma16816(d, a[0], x0.x, x0.y);
              mma16816(d, a[1], x0.z, x0.w);
              mma16816(d, a[2], x1.x, x1.y);
              mma16816(d, a[3], x1.z, x1.w);
            }
          }
        }
        if constexpr (is_quant<FMT>()) {
          const float sa = __half2float(__ushort_as_half((unsigned short)(sc[j] & 0xffffu)));
          const float sb = __half2float(__ushort_as_half((unsigned short)(sc[j] >> 16)));
#pragma unroll
          for (int mt = 0; mt < MT; ++mt) {
            acc[mt][0] = fmaf(sa, gacc[mt][0], acc[mt][0]);
            acc[mt][1] = fmaf(sa, gacc[mt][1], acc[mt][1]);
            acc[mt][2] = fmaf(sb, gacc[mt][2], acc[mt][2]);
            acc[mt][3] = fmaf(sb, gacc[mt][3], acc[mt][3]);
          }
        }
      }
    }
  }
};

struct DecodeArgs {
  WMat w, a, b;
  const void* x;
  void* y;
  float* t_ws;
  float* y_ws;
  uint32_t* counters;
  int* dev_status;
  int m, d_in, d_out, r_pad;
  int x_dtype, y_dtype;
  int a_units, a_split, w_split;
  int qt_w, qt_a, qt_b;     // tiles per quantum of each matrix
};

__device__ __forceinline__ void store_y(void* y, int dtype, int64_t i, float v) {
  if (dtype == EORA_Y_F16) reinterpret_cast<__half*>(y)[i] = __float2half_rn(v);
  else if (dtype == EORA_Y_BF16) reinterpret_cast<__nv_bfloat16*>(y)[i] = __float2bfloat16_rn(v);
  else reinterpret_cast<float*>(y)[i] = v;
}

// Stage activation rows [0, m) x reduction range [k0, k0 + len) into shared memory as fp16.
__device__ __forceinline__ void stage_x(__half* xs, int xrow, const void* x, int x_dtype, int m, int d_in, int k0, int len) {
  const int chunks = len >> 3;   // 16-byte chunks per row
  for (int i = threadIdx.x; i < m * chunks; i += kThreads) {
    int row = i / chunks, c = i - row * chunks;
    uint4 v = *reinterpret_cast<const uint4*>(reinterpret_cast<const uint16_t*>(x) + (int64_t)row * d_in + k0 + c * 8);
    if (x_dtype == EORA_X_BF16) {
      uint32_t* pv = reinterpret_cast<uint32_t*>(&v);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        __nv_bfloat162 b2 = *reinterpret_cast<__nv_bfloat162*>(&pv[j]);
        float2 f = __bfloat1622float2(b2);
        __half2 h2 = __floats2half2_rn(f.x, f.y);
        pv[j] = *reinterpret_cast<uint32_t*>(&h2);
      }
    }
    *reinterpret_cast<uint4*>(xs + row * xrow + c * 8) = v;
  }
}

template <int FMT, int MT, int NX>
__device__ __forceinline__ void stream_range(const WMat& m, int qt, int tile, int q0, int q1, int warp, int lane,
                                             const __half* xs, int xrow, int xsrc_stride, int k_base, int m_rows,
                                             float (&acc)[MT][4]) {
  if (qt == 2) {
    Streamer<FMT, MT, 2, NX> s;
    for (int qf = q0; qf < q1; qf += kWarps * s.PF) {
      s.issue(m, tile, qf, q1, warp, lane);
      s.compute(qf, q1, warp, lane, xs, xrow, xsrc_stride, k_base, m_rows, acc);
    }
  } else {
    Streamer<FMT, MT, 1, NX> s;
    for (int qf = q0; qf < q1; qf += kWarps * s.PF) {
      s.issue(m, tile, qf, q1, warp, lane);
      s.compute(qf, q1, warp, lane, xs, xrow, xsrc_stride, k_base, m_rows, acc);
    }
  }
}

// Same, but the first batch is loaded before `sync_point()` (the dependent-launch wait and the
// activation staging) runs, so that weight traffic overlaps the previous kernel.
template <int FMT, int MT, int QT, typename F>
__device__ __forceinline__ void stream_first(const WMat& m, int tile, int q0, int q1, int warp, int lane, F&& sync_point,
                                             const __half* xs, int xrow, int k_base, int m_rows, float (&acc)[MT][4]) {
  Streamer<FMT, MT, QT, 1> s;
  s.issue(m, tile, q0, q1, warp, lane);
  sync_point();
  s.compute(q0, q1, warp, lane, xs, xrow, 0, k_base, m_rows, acc);
  for (int qf = q0 + kWarps * s.PF; qf < q1; qf += kWarps * s.PF) {
    s.issue(m, tile, qf, q1, warp, lane);
    s.compute(qf, q1, warp, lane, xs, xrow, 0, k_base, m_rows, acc);
  }
}

template <int WF, int ABF, int MT>
__global__ void __launch_bounds__(kThreads, MT <= 2 ? 2 : 1) k_decode(const DecodeArgs p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __shared__ float red[kWarps][MT * 4 * 32];
  __shared__ uint32_t s_flag;

  asm volatile("griddepcontrol.launch_dependents;");

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int unit = blockIdx.x;
  const bool is_a = unit < p.a_units;
  int tile, slice, split;
  if (is_a) { tile = unit / p.a_split; slice = unit % p.a_split; split = p.a_split; }
  else { int u = unit - p.a_units; tile = u / p.w_split; slice = u % p.w_split; split = p.w_split; }
  const WMat& mat = is_a ? p.a : p.w;
  const int qt = is_a ? p.qt_a : p.qt_w;
  const int nq = mat.kc / qt;                       // quanta per row tile
  const int q0 = (int)((int64_t)nq * slice / split), q1 = (int)((int64_t)nq * (slice + 1) / split);
  const int k_base = q0 * qt * 64, k_len = (q1 - q0) * qt * 64;
  const int xrow = k_len + kXPad;
  __half* xs = reinterpret_cast<__half*>(smem_raw);

  float acc[MT][4];
#pragma unroll
  for (int mt = 0; mt < MT; ++mt) acc[mt][0] = acc[mt][1] = acc[mt][2] = acc[mt][3] = 0.f;

  auto sync_point = [&]() {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    stage_x(xs, xrow, p.x, p.x_dtype, p.m, p.d_in, k_base, k_len);
    __syncthreads();
  };

  if (is_a) {
    if constexpr (ABF != FMT_NONE) {
      if (qt == 2) stream_first<ABF, MT, 2>(mat, tile, q0, q1, warp, lane, sync_point, xs, xrow, k_base, p.m, acc);
      else stream_first<ABF, MT, 1>(mat, tile, q0, q1, warp, lane, sync_point, xs, xrow, k_base, p.m, acc);
    }
  } else {
    if (qt == 2) stream_first<WF, MT, 2>(mat, tile, q0, q1, warp, lane, sync_point, xs, xrow, k_base, p.m, acc);
    else stream_first<WF, MT, 1>(mat, tile, q0, q1, warp, lane, sync_point, xs, xrow, k_base, p.m, acc);
  }

  // ---- B extension: the last slice of a backbone row tile adds (X.A).B for its 16 output columns
  const bool owns_b = !is_a && slice == split - 1 && p.a_units > 0;
  if constexpr (ABF != FMT_NONE) {
    if (owns_b) {
      __syncthreads();                                   // everyone is done reading the staged X
      if (threadIdx.x == 0) {
        uint32_t it = 0;
        while (ld_acquire(p.counters + CNT_T_DONE) < (uint32_t)p.a_units) {
          if (++it > kSpinLimit) { atomicExch(p.dev_status, EORA_ERR_DEVICE_TIMEOUT); break; }
          __nanosleep(64);
        }
      }
      __syncthreads();
      // t -> fp16 hi + lo in shared memory (two sources), rows padded like X
      const int trow = p.r_pad + kXPad;
      __half* ts = xs;
      for (int i = threadIdx.x; i < p.m * p.r_pad; i += kThreads) {
        int row = i / p.r_pad, j = i - row * p.r_pad;
        float v = ld_cg(p.t_ws + (int64_t)row * p.r_pad + j);
        __half hi = __float2half_rn(v);
        __half lo = __float2half_rn(v - __half2float(hi));
        ts[row * trow + j] = hi;
        ts[p.m * trow + row * trow + j] = lo;
      }
      __syncthreads();
      // all reads of t by this CTA are done: the last consumer returns t_ws and the counters to zero
      if (threadIdx.x == 0) {
        __threadfence();
        uint32_t c = atomicAdd(p.counters + CNT_T_CONSUMED, 1u);
        s_flag = (c == (uint32_t)p.w.nt - 1) ? 1u : 0u;
      }
      __syncthreads();
      if (s_flag) {
        for (int i = threadIdx.x; i < p.m * p.r_pad; i += kThreads) p.t_ws[i] = 0.f;
        if (threadIdx.x == 0) { p.counters[CNT_T_DONE] = 0; p.counters[CNT_T_CONSUMED] = 0; }
      }
      const int nqb = p.b.kc / p.qt_b;
      stream_range<ABF, MT, 2>(p.b, p.qt_b, tile, 0, nqb, warp, lane, ts, trow, p.m * trow, 0, p.m, acc);
    }
  }

  // ---- sum the 8 warps
#pragma unroll
  for (int mt = 0; mt < MT; ++mt)
#pragma unroll
    for (int c = 0; c < 4; ++c) red[warp][(mt * 4 + c) * 32 + lane] = acc[mt][c];
  __syncthreads();

  // outputs of this unit: 16 rows x 8*MT tokens; element idx of the warp sums is
  // (mt, c, lane) = (idx >> 7, (idx >> 5) & 3, idx & 31)
  auto out_pos = [&](int idx, int& token, int& row) {
    const int l = idx & 31, c = (idx >> 5) & 3, mt = idx >> 7;
    token = mt * 8 + 2 * (l & 3) + (c & 1);
    row = tile * 16 + (l >> 2) + 8 * (c >> 1);
  };
  auto warp_sum = [&](int idx) {
    float v = 0.f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) v += red[w][idx];
    return v;
  };

  if (is_a) {
    for (int idx = threadIdx.x; idx < MT * 128; idx += kThreads) {
      int token, row;
      out_pos(idx, token, row);
      if (token < p.m) red_add(p.t_ws + (int64_t)token * p.r_pad + row, warp_sum(idx));
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) atomicAdd(p.counters + CNT_T_DONE, 1u);
    return;
  }
  if (split == 1) {
    for (int idx = threadIdx.x; idx < MT * 128; idx += kThreads) {
      int token, row;
      out_pos(idx, token, row);
      if (token < p.m) store_y(p.y, p.y_dtype, (int64_t)token * p.d_out + row, warp_sum(idx));
    }
    return;
  }
  for (int idx = threadIdx.x; idx < MT * 128; idx += kThreads) {
    int token, row;
    out_pos(idx, token, row);
    if (token < p.m) red_add(p.y_ws + (int64_t)token * p.d_out + row, warp_sum(idx));
  }
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    uint32_t c = atomicAdd(p.counters + CNT_TILE0 + tile, 1u);
    s_flag = (c == (uint32_t)split - 1) ? 1u : 0u;
  }
  __syncthreads();
  if (s_flag) {
    __threadfence();
    for (int idx = threadIdx.x; idx < MT * 128; idx += kThreads) {
      int token, row;
      out_pos(idx, token, row);
      if (token < p.m) {
        float* src = p.y_ws + (int64_t)token * p.d_out + row;
        store_y(p.y, p.y_dtype, (int64_t)token * p.d_out + row, ld_cg(src));
        *src = 0.f;
      }
    }
    if (threadIdx.x == 0) p.counters[CNT_TILE0 + tile] = 0;
  }
}

int quantum_tiles(const WMat& m) {
  if (m.fmt == FMT_F16) return 1;
  return (m.group % 128 == 0) ? 2 : 1;
}

struct Plan { int a_units, a_split, w_split, smem; };

Plan make_plan(const Handle* h, int m) {
  Plan pl;
  const int slots = 2 * h->sm_count;
  const int max_slice_k = (kXSmemBudget / (2 * m)) & ~127;          // activations staged per CTA
  auto split_for = [&](const WMat& mat, int want) {
    int qt = quantum_tiles(mat), nq = mat.kc / qt;
    int min_split = (mat.k_red + max_slice_k - 1) / max_slice_k;
    int s = want > min_split ? want : min_split;
    if (s > nq) s = nq;
    if (s < 1) s = 1;
    return s;
  };
  int want_w = (h->w.nt * 4 >= slots * 3) ? 1 : (slots + h->w.nt - 1) / h->w.nt;
  pl.w_split = split_for(h->w, want_w);
  pl.a_units = 0; pl.a_split = 1;
  if (h->cfg.rank > 0) {
    // size A units like backbone units (in bytes streamed)
    int64_t w_unit_bytes = wmat_q_bytes(h->w.fmt, 1, h->w.kc) / pl.w_split;
    if (w_unit_bytes < 8192) w_unit_bytes = 8192;
    int64_t a_tile_bytes = wmat_q_bytes(h->a.fmt, 1, h->a.kc);
    int want_a = (int)((a_tile_bytes + w_unit_bytes - 1) / w_unit_bytes);
    pl.a_split = split_for(h->a, want_a);
    pl.a_units = h->a.nt * pl.a_split;
  }
  // shared memory: the staged X slice, or the hi/lo copies of t
  int64_t max_k = 0;
  auto slice_len = [&](const WMat& mat, int split) {
    int qt = quantum_tiles(mat), nq = mat.kc / qt;
    int best = 0;
    for (int s = 0; s < split; ++s) {
      int l = (int)(((int64_t)nq * (s + 1) / split) - ((int64_t)nq * s / split)) * qt * 64;
      if (l > best) best = l;
    }
    return best;
  };
  max_k = slice_len(h->w, pl.w_split);
  if (h->cfg.rank > 0) {
    int la = slice_len(h->a, pl.a_split);
    if (la > max_k) max_k = la;
  }
  int64_t xb = (int64_t)m * (max_k + kXPad) * 2;
  int64_t tb = h->cfg.rank > 0 ? (int64_t)2 * m * (h->r_pad + kXPad) * 2 : 0;
  pl.smem = (int)(xb > tb ? xb : tb);
  return pl;
}

template <auto KERNEL>
cudaError_t launch_kernel(const cudaLaunchConfig_t& cfg, const DecodeArgs& args) {
  static bool attr_set = false;   // one per kernel (KERNEL is a template argument)
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(KERNEL, cudaFuncAttributeMaxDynamicSharedMemorySize, 160 * 1024);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  return cudaLaunchKernelEx(&cfg, KERNEL, args);
}

template <int WF, int ABF>
cudaError_t launch_mt(const DecodeArgs& args, int mt, int grid, int smem, cudaStream_t st) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  switch (mt) {
    case 1: return launch_kernel<k_decode<WF, ABF, 1>>(cfg, args);
    case 2: return launch_kernel<k_decode<WF, ABF, 2>>(cfg, args);
    case 4: return launch_kernel<k_decode<WF, ABF, 4>>(cfg, args);
    default: return launch_kernel<k_decode<WF, ABF, 8>>(cfg, args);
  }
}

template <int WF>
cudaError_t launch_ab(const DecodeArgs& args, int abf, int mt, int grid, int smem, cudaStream_t st) {
  switch (abf) {
    case FMT_F16: return launch_mt<WF, FMT_F16>(args, mt, grid, smem, st);
    case FMT_Q4: return launch_mt<WF, FMT_Q4>(args, mt, grid, smem, st);
    case FMT_Q8: return launch_mt<WF, FMT_Q8>(args, mt, grid, smem, st);
    default: return launch_mt<WF, FMT_NONE>(args, mt, grid, smem, st);
  }
}

}  // namespace

bool decode_supported(const Handle* h, int m) {
  if (m < 1 || m > 64) return false;
  if (h->w.fmt != FMT_Q4 && h->w.fmt != FMT_Q3) return false;
  if (h->w.group % 64) return false;
  Plan pl = make_plan(h, m);
  return pl.smem <= 160 * 1024;
}

void decode_make_plan(Handle* h) { h->plan = DecodePlan(); }

int decode_launch_count(const Handle*, int) { return 1; }

cudaError_t launch_decode_forward(const Handle* h, const void* x, int m, void* y, cudaStream_t st) {
  Plan pl = make_plan(h, m);
  DecodeArgs a;
  a.w = h->w; a.a = h->a; a.b = h->b;
  a.x = x; a.y = y;
  a.t_ws = h->t_ws; a.y_ws = h->y_ws; a.counters = h->counters; a.dev_status = h->dev_status;
  a.m = m; a.d_in = h->cfg.d_in; a.d_out = h->cfg.d_out; a.r_pad = h->r_pad;
  a.x_dtype = h->cfg.x_dtype; a.y_dtype = h->cfg.y_dtype;
  a.a_units = pl.a_units; a.a_split = pl.a_split; a.w_split = pl.w_split;
  a.qt_w = quantum_tiles(h->w);
  a.qt_a = h->cfg.rank > 0 ? quantum_tiles(h->a) : 1;
  a.qt_b = h->cfg.rank > 0 ? quantum_tiles(h->b) : 1;
  int grid = pl.a_units + h->w.nt * pl.w_split;
  int mt = m <= 8 ? 1 : m <= 16 ? 2 : m <= 32 ? 4 : 8;
  int abf = h->cfg.rank > 0 ? h->a.fmt : FMT_NONE;
  if (h->w.fmt == FMT_Q4) return launch_ab<FMT_Q4>(a, abf, mt, grid, pl.smem, st);
  return launch_ab<FMT_Q3>(a, abf, mt, grid, pl.smem, st);
}

}  // namespace eora
