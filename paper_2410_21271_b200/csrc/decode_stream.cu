// Streaming decode kernel for M <= 8: the same fused layer as decode.cu
//     Y = X.deq(Wq) + (X.A).B   (paper Eq. 4; Section 4.5 fuses only the product with B),
// organised as a persistent, warp-specialised pipeline so that the per-unit fixed costs
// (index math, copy latency, cross-warp sum, split-K combine, the wait for t) stay off the
// path that streams weights.
//
// A CTA has 10 warps and owns the units  blockIdx.x, blockIdx.x + gridDim.x, ...  (a unit is a
// 16-row tile x reduction slice of A or of the backbone; A units come first).
//   producer warp (1 lane): walks the CTA's units chunk by chunk (a chunk = up to two quanta per compute
//       warp, at most 16 KB) and bulk-copies the packed tiles into a ring of shared-memory slots
//       (cp.async.bulk + mbarrier, no multicast).  Weights never change, so it starts before the
//       dependency wait of programmatic dependent launch and keeps the whole ring in flight.
//   8 compute warps: per chunk, wait for the slot, dequantise their quantum in registers to the
//       exact fp16 integers (q - z), multiply with the staged activations on the tensor cores
//       (mma.m16n8k16, fp32 accumulate), apply the scale per quantum, and drop their partial
//       16 x 8 result into a ring of reduction slots.
//   epilogue warp: sums the 8 partials; for an A unit adds them into t_ws and bumps T_DONE; for
//       a backbone unit that owns the B extension waits (bounded, once per CTA) for t, runs the
//       prefetched B tiles against fp16 hi + lo copies of t, then writes Y or joins the split-K
//       combine through y_ws.  Compute warps never wait for any of this.
// All scratch words are returned to zero before the kernel ends.
#include "decode_common.cuh"

namespace eora {
using namespace dec;
namespace {

constexpr int kCW = 8;                         // compute warps
constexpr int kEpiWarp = kCW, kProdWarp = kCW + 1;
constexpr int kThreadsS = (kCW + 2) * 32;
constexpr int kXPad = 32;
constexpr int kMaxStages = 12;
constexpr int kSlotBytes = 16 * 1024;          // one ring slot = one chunk (up to two quanta per compute warp)
constexpr int kRed = 4;                        // reduction-slot ring depth
constexpr int kBRing = 2;
constexpr int kSmemPerCta = 110 * 1024;        // two CTAs per SM

struct StreamArgs {
  WMat w, a, b;
  const void* x;
  void* y;
  float* t_ws;
  float* y_ws;
  uint32_t* counters;
  int* dev_status;
  unsigned long long* trace;
  int m, d_in, d_out, r_pad;
  int x_dtype, y_dtype;
  int a_units, a_split, w_split, n_units;
  int qt_w, qt_a, qt_b;
  int stages;                 // ring slots of kSlotBytes
  int cq_w, cq_a;             // quanta per chunk of the backbone / of A
  int nqu_w, nqu_a;           // quanta per unit (the split divides the quanta of a row tile evenly)
  int dt_w, ds_w, dt_a, ds_a; // gridDim.x / split and gridDim.x % split: unit index stepping without division
  int qpg_shift_w, qpg_shift_a;   // log2(quanta per group), or -1 if not a power of two
  int off_x, off_red, off_b, b_bytes, b_sc_off, b_zz_off, off_t;
};

struct Unit {
  bool is_a, owns_b;
  int tile, split, q0, nq;      // quanta [q0, q0 + nq) of row tile `tile`
};

// Walks the units  u0, u0 + G, u0 + 2G, ...  of one CTA.  Only the first unit and the first backbone
// unit after the A units cost an integer division.
struct UnitIter {
  int u, tile, slice;
  bool is_a;
  __device__ __forceinline__ void locate(const StreamArgs& p) {
    is_a = u < p.a_units;
    if (is_a) { tile = u / p.a_split; slice = u - tile * p.a_split; }
    else { int v = u - p.a_units; tile = v / p.w_split; slice = v - tile * p.w_split; }
  }
  __device__ __forceinline__ void init(const StreamArgs& p, int u0) { u = u0; locate(p); }
  __device__ __forceinline__ void next(const StreamArgs& p, int G) {
    u += G;
    if (is_a) {
      if (u >= p.a_units) { locate(p); return; }
      tile += p.dt_a; slice += p.ds_a;
      if (slice >= p.a_split) { slice -= p.a_split; ++tile; }
    } else {
      tile += p.dt_w; slice += p.ds_w;
      if (slice >= p.w_split) { slice -= p.w_split; ++tile; }
    }
  }
  __device__ __forceinline__ Unit get(const StreamArgs& p) const {
    Unit r;
    r.is_a = is_a; r.tile = tile;
    r.split = is_a ? p.a_split : p.w_split;
    r.nq = is_a ? p.nqu_a : p.nqu_w;
    r.q0 = slice * r.nq;
    r.owns_b = !is_a && slice == r.split - 1 && p.a_units > 0;
    return r;
  }
};

__device__ __forceinline__ int group_of(int quantum, int shift, int qpg) {
  return shift >= 0 ? (quantum >> shift) : quantum / qpg;
}

#define STRACE(slot) do { if (p.trace) p.trace[(size_t)blockIdx.x * 16 + (slot)] = globaltimer_ns(); } while (0)

// NQ quanta (QT tiles each, sharing one scale / zero-point per quantum) for one compute warp, in one
// straight-line block so that the independent dequant / MMA chains of the quanta interleave.
// Quantum j: tiles at blob + j * blob_stride, activations at xl + j * x_stride (halves).
template <int FMT, int QT, int NQ>
__device__ __forceinline__ void run_quanta(const uint8_t* blob, int blob_stride, const uint32_t (&sc2)[2], const uint32_t (&zz2)[2],
                                           int lane, const __half* xl, int x_stride, bool have_x, float (&acc)[4]) {
  constexpr int TB = FMT == FMT_Q4 ? 512 : FMT == FMT_Q3 ? 384 : FMT == FMT_Q8 ? 1024 : 2048;
  float gacc[NQ][QT][4];
#pragma unroll
  for (int j = 0; j < NQ; ++j) {
    ZC zc;
    if constexpr (is_quant<FMT>()) make_zc<FMT>(zc, zz2[j]);
#pragma unroll
    for (int tt = 0; tt < QT; ++tt) {
      gacc[j][tt][0] = gacc[j][tt][1] = gacc[j][tt][2] = gacc[j][tt][3] = 0.f;
      uint32_t a[4][4];
      tile_frags<FMT>(blob + j * blob_stride + tt * TB, lane, zc, a);
      uint4 x0 = make_uint4(0, 0, 0, 0), x1 = make_uint4(0, 0, 0, 0);
      if (have_x) {
        x0 = *reinterpret_cast<const uint4*>(xl + j * x_stride + tt * 64);
        x1 = *reinterpret_cast<const uint4*>(xl + j * x_stride + tt * 64 + 32);
      }
      mma16816(gacc[j][tt], a[0], x0.x, x0.y);
      mma16816(gacc[j][tt], a[1], x0.z, x0.w);
      mma16816(gacc[j][tt], a[2], x1.x, x1.y);
      mma16816(gacc[j][tt], a[3], x1.z, x1.w);
    }
  }
#pragma unroll
  for (int j = 0; j < NQ; ++j) {
    float sa = 1.f, sb = 1.f;
    if constexpr (is_quant<FMT>()) {
      sa = __half2float(__ushort_as_half((unsigned short)(sc2[j] & 0xffffu)));
      sb = __half2float(__ushort_as_half((unsigned short)(sc2[j] >> 16)));
    }
#pragma unroll
    for (int tt = 0; tt < QT; ++tt) {
      acc[0] = fmaf(sa, gacc[j][tt][0], acc[0]);
      acc[1] = fmaf(sa, gacc[j][tt][1], acc[1]);
      acc[2] = fmaf(sb, gacc[j][tt][2], acc[2]);
      acc[3] = fmaf(sb, gacc[j][tt][3], acc[3]);
    }
  }
}

template <int FMT>
__device__ __forceinline__ void run_chunk(int qt, int nq_here, const uint8_t* blob, int blob_stride, const uint32_t (&sc2)[2],
                                          const uint32_t (&zz2)[2], int lane, const __half* xl, int x_stride, bool have_x,
                                          float (&acc)[4]) {
  if constexpr (FMT != FMT_NONE) {
    if (qt == 2) {
      if (nq_here == 2) run_quanta<FMT, 2, 2>(blob, blob_stride, sc2, zz2, lane, xl, x_stride, have_x, acc);
      else run_quanta<FMT, 2, 1>(blob, blob_stride, sc2, zz2, lane, xl, x_stride, have_x, acc);
    } else {
      if (nq_here == 2) run_quanta<FMT, 1, 2>(blob, blob_stride, sc2, zz2, lane, xl, x_stride, have_x, acc);
      else run_quanta<FMT, 1, 1>(blob, blob_stride, sc2, zz2, lane, xl, x_stride, have_x, acc);
    }
  }
}

// What a compute warp needs to know about the matrix of a unit.  The two possible matrices (A and the
// backbone) are turned into registers once per kernel: picking between two kernel-parameter structs at run
// time costs a chain of dependent constant-bank loads at every unit boundary.
struct MatInfo {
  const uint32_t* scp;      // scales of the unit's row tile (+ g), set per unit
  const uint16_t* zzp;
  const uint32_t* sc_base;  // matrix base (+ g)
  const uint16_t* zz_base;
  int ng8;                  // words per row tile in sc / zz
  int qt, cq, tb, qsh, qpg;
  bool quant;
};
__device__ __forceinline__ MatInfo mat_base(const WMat& mat, int qt, int cq, int qsh, int g) {
  MatInfo m;
  m.qt = qt; m.cq = cq; m.qsh = qsh;
  m.tb = tile_bytes(mat.fmt);
  m.qpg = mat.fmt == FMT_NONE ? 1 : mat.group / (64 * qt);
  m.quant = mat.fmt != FMT_F16;
  m.sc_base = mat.sc + g; m.zz_base = mat.zz + g;
  m.ng8 = mat.ng * 8;
  m.scp = m.sc_base; m.zzp = m.zz_base;
  return m;
}
__device__ __forceinline__ MatInfo mat_info(const MatInfo& ma, const MatInfo& mw, const Unit& u) {
  MatInfo m = u.is_a ? ma : mw;
  m.scp = m.sc_base + (int64_t)u.tile * m.ng8;
  m.zzp = m.zz_base + (int64_t)u.tile * m.ng8;
  return m;
}
// scales / zero-points of this warp's (up to two) quanta of the chunk that starts at quantum q of unit u
__device__ __forceinline__ void load_sz(const MatInfo& m, const Unit& u, int q, int warp, uint32_t (&sc)[2], uint32_t (&zz)[2]) {
#pragma unroll
  for (int j = 0; j < 2; ++j) {
    const int lq = j * kCW + warp, qq = q + lq;
    sc[j] = 0; zz[j] = 0;
    if (m.quant && lq < m.cq && qq < u.nq) {
      const int gi = group_of(u.q0 + qq, m.qsh, m.qpg);
      sc[j] = __ldg(m.scp + gi * 8);
      zz[j] = __ldg(m.zzp + gi * 8);
    }
  }
}

// B extension by the epilogue warp alone: all tiles of B's row tile against t (hi + lo copies).
template <int FMT>
__device__ __forceinline__ void run_b(const uint8_t* bbuf, const uint32_t* sc, const uint16_t* zz, int ntiles, int qt,
                                      int group_tiles, int lane, const __half* ts, int trow, int m_rows, float (&acc)[4]) {
  constexpr int TB = FMT == FMT_Q4 ? 512 : FMT == FMT_Q3 ? 384 : FMT == FMT_Q8 ? 1024 : 2048;
  const int g = lane >> 2, t = lane & 3;
  const bool have_x = g < m_rows;
#pragma unroll 1
  for (int q = 0; q < ntiles / qt; ++q) {
    float gacc[4] = {0.f, 0.f, 0.f, 0.f};
    ZC zc;
    uint32_t sc2 = 0;
    if constexpr (is_quant<FMT>()) {
      const int gi = (q * qt) / group_tiles;
      sc2 = sc[gi * 8 + g];
      make_zc<FMT>(zc, zz[gi * 8 + g]);
    }
#pragma unroll 1
    for (int tt = 0; tt < qt; ++tt) {
      const int tile = q * qt + tt;
      uint32_t a[4][4];
      tile_frags<FMT>(bbuf + tile * TB, lane, zc, a);
#pragma unroll
      for (int s = 0; s < 2; ++s) {
        uint4 x0 = make_uint4(0, 0, 0, 0), x1 = make_uint4(0, 0, 0, 0);
        if (have_x) {
          const __half* xl = ts + (s * m_rows + g) * trow + 8 * t + tile * 64;
          x0 = *reinterpret_cast<const uint4*>(xl);
          x1 = *reinterpret_cast<const uint4*>(xl + 32);
        }
        float(&d)[4] = is_quant<FMT>() ? gacc : acc;
        mma16816(d, a[0], x0.x, x0.y);
        mma16816(d, a[1], x0.z, x0.w);
        mma16816(d, a[2], x1.x, x1.y);
        mma16816(d, a[3], x1.z, x1.w);
      }
    }
    if constexpr (is_quant<FMT>()) {
      const float sa = __half2float(__ushort_as_half((unsigned short)(sc2 & 0xffffu)));
      const float sb = __half2float(__ushort_as_half((unsigned short)(sc2 >> 16)));
      acc[0] = fmaf(sa, gacc[0], acc[0]);
      acc[1] = fmaf(sa, gacc[1], acc[1]);
      acc[2] = fmaf(sb, gacc[2], acc[2]);
      acc[3] = fmaf(sb, gacc[3], acc[3]);
    }
  }
}

template <int WF, int ABF>
__global__ void __launch_bounds__(kThreadsS, 2) k_decode_stream(const StreamArgs p) {
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ __align__(8) uint64_t full[kMaxStages], empty[kMaxStages], red_full[kRed], red_free[kRed], b_full[kBRing];

  asm volatile("griddepcontrol.launch_dependents;");
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int G = gridDim.x;
  const int n_mine = (p.n_units - (int)blockIdx.x + G - 1) / G;      // units of this CTA
  __half* xs = reinterpret_cast<__half*>(smem + p.off_x);
  float* red = reinterpret_cast<float*>(smem + p.off_red);
  const int xrow = p.d_in + kXPad;

  if (threadIdx.x == 0) {
    STRACE(0);
    for (int i = 0; i < p.stages; ++i) { mbar_init(full + i, 1); mbar_init(empty + i, kCW); }
    for (int i = 0; i < kRed; ++i) { mbar_init(red_full + i, kCW); mbar_init(red_free + i, 1); }
    for (int i = 0; i < kBRing; ++i) mbar_init(b_full + i, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();

  if (warp == kProdWarp) {
    // ------------------------------------------------------------------ producer
    if (lane == 0) {
      int s = 0, ph = 0, c = 0;                     // ring slot, its phase, chunk counter of this CTA
      bool alive = true;
      UnitIter it;
      it.init(p, (int)blockIdx.x);
      for (int i = 0; i < n_mine && alive; ++i, it.next(p, G)) {
        const Unit u = it.get(p);
        const WMat& mat = u.is_a ? p.a : p.w;
        const int qt = u.is_a ? p.qt_a : p.qt_w, cq = u.is_a ? p.cq_a : p.cq_w;
        const int tb = tile_bytes(mat.fmt);
        const uint8_t* src = mat.q + ((int64_t)u.tile * mat.kc + (int64_t)u.q0 * qt) * tb;
        for (int q = 0; q < u.nq; q += cq, ++c) {
          if (c >= p.stages && !mbar_wait(empty + s, ph ^ 1, p.dev_status)) { alive = false; break; }
          const int n = u.nq - q < cq ? u.nq - q : cq;
          const uint32_t bytes = (uint32_t)n * qt * tb;
          mbar_expect_tx(full + s, bytes);
          bulk_g2s(smem + (size_t)s * kSlotBytes, src + (size_t)q * qt * tb, bytes, full + s);
          if (c == 0) STRACE(1);
          if (++s == p.stages) { s = 0; ph ^= 1; }
        }
      }
    }
    return;
  }

  asm volatile("griddepcontrol.wait;" ::: "memory");

  if (warp < kCW) {
    // ------------------------------------------------------------------ compute warps
    if (threadIdx.x == 0) STRACE(2);
    // stage all of X (M rows x d_in) as fp16
    {
      const int chunks = p.d_in >> 3;
      for (int row = 0; row < p.m; ++row) {
        for (int c = threadIdx.x; c < chunks; c += kCW * 32) {
          uint4 v = *reinterpret_cast<const uint4*>(reinterpret_cast<const uint16_t*>(p.x) + (int64_t)row * p.d_in + c * 8);
          if (p.x_dtype == EORA_X_BF16) {
            uint32_t* pv = reinterpret_cast<uint32_t*>(&v);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              float2 f = __bfloat1622float2(*reinterpret_cast<__nv_bfloat162*>(&pv[j]));
              __half2 h2 = __floats2half2_rn(f.x, f.y);
              pv[j] = *reinterpret_cast<uint32_t*>(&h2);
            }
          }
          *reinterpret_cast<uint4*>(xs + row * xrow + c * 8) = v;
        }
      }
      asm volatile("bar.sync 1, %0;" ::"n"(kCW * 32) : "memory");
    }
    if (threadIdx.x == 0) STRACE(3);
    const int g = lane >> 2;
    const bool have_x = g < p.m;
    const __half* xlane = xs + g * xrow + 8 * (lane & 3);
    int cstamp = 0;                                 // per-chunk trace stamps of CTA 0 (see eora_linear_set_trace)
    int s = 0, ph = 0;                              // ring slot and phase, in step with the producer
    int rb = 0, rph = 0;                            // reduction slot and phase
    bool alive = true;
    UnitIter it;
    it.init(p, (int)blockIdx.x);
    const MatInfo base_a = mat_base(p.a, p.qt_a, p.cq_a, p.qpg_shift_a, g);
    const MatInfo base_w = mat_base(p.w, p.qt_w, p.cq_w, p.qpg_shift_w, g);
    Unit u = it.get(p);
    MatInfo mi = mat_info(base_a, base_w, u);
    uint32_t sc2[2], zz2[2];
    load_sz(mi, u, 0, warp, sc2, zz2);            // weights are immutable: plain cached loads, always one chunk ahead
    for (int i = 0; i < n_mine && alive; ++i) {
      UnitIter itn = it;
      itn.next(p, G);
      const bool have_next = i + 1 < n_mine;
      Unit un = u;
      MatInfo mn = mi;
      if (have_next) { un = itn.get(p); mn = mat_info(base_a, base_w, un); }
      float acc[4] = {0.f, 0.f, 0.f, 0.f};
      for (int q = 0; q < u.nq; q += mi.cq) {
        if (threadIdx.x == 0 && p.trace && blockIdx.x == 0 && cstamp < 500) p.trace[(size_t)gridDim.x * 16 + cstamp * 4 + 0] = clock64();
        if (!mbar_wait_warp(full + s, ph, p.dev_status, lane)) { alive = false; break; }
        if (threadIdx.x == 0 && p.trace && blockIdx.x == 0 && cstamp < 500) p.trace[(size_t)gridDim.x * 16 + cstamp * 4 + 1] = clock64();
        uint32_t sc_n[2] = {0, 0}, zz_n[2] = {0, 0};
        if (q + mi.cq < u.nq) load_sz(mi, u, q + mi.cq, warp, sc_n, zz_n);
        else if (have_next) load_sz(mn, un, 0, warp, sc_n, zz_n);
        // this warp's quanta of the chunk: local indices warp and warp + 8
        int nq_here = 0;
        if (warp < mi.cq && q + warp < u.nq) nq_here = (warp + kCW < mi.cq && q + warp + kCW < u.nq) ? 2 : 1;
        if (nq_here) {
          const int qbytes = mi.qt * mi.tb;
          const uint8_t* blob = smem + (size_t)s * kSlotBytes + warp * qbytes;
          const __half* xl = xlane + (u.q0 + q + warp) * mi.qt * 64;
          if (u.is_a) run_chunk<ABF>(mi.qt, nq_here, blob, kCW * qbytes, sc2, zz2, lane, xl, kCW * mi.qt * 64, have_x, acc);
          else run_chunk<WF>(mi.qt, nq_here, blob, kCW * qbytes, sc2, zz2, lane, xl, kCW * mi.qt * 64, have_x, acc);
        }
        sc2[0] = sc_n[0]; sc2[1] = sc_n[1]; zz2[0] = zz_n[0]; zz2[1] = zz_n[1];
        if (threadIdx.x == 0 && p.trace && blockIdx.x == 0 && cstamp < 500) { p.trace[(size_t)gridDim.x * 16 + cstamp * 4 + 2] = clock64(); ++cstamp; }
        __syncwarp();
        if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(empty + s)) : "memory");
        if (++s == p.stages) { s = 0; ph ^= 1; }
      }
      if (!alive) break;
      if (threadIdx.x == 0 && p.trace && blockIdx.x == 0 && cstamp > 0 && cstamp <= 500) p.trace[(size_t)gridDim.x * 16 + (cstamp - 1) * 4 + 3] = clock64();
      if (i >= kRed && !mbar_wait_warp(red_free + rb, rph ^ 1, p.dev_status, lane)) break;
      float* r = red + (rb * kCW + warp) * 128;
#pragma unroll
      for (int cc = 0; cc < 4; ++cc) r[cc * 32 + lane] = acc[cc];
      __syncwarp();
      if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(red_full + rb)) : "memory");
      if (++rb == kRed) { rb = 0; rph ^= 1; }
      it = itn; u = un; mi = mn;
    }
    if (threadIdx.x == 0) STRACE(4);
    return;
  }

  // -------------------------------------------------------------------- epilogue warp
  const bool have_ab = p.a_units > 0;
  __half* ts = reinterpret_cast<__half*>(smem + p.off_t);
  const int trow = p.r_pad + kXPad;
  bool t_staged = false;
  int b_issued = 0, b_used = 0, b_scan = 0;       // ring bookkeeping over this CTA's owns_b units
  UnitIter bit;
  bit.init(p, (int)blockIdx.x);
  auto issue_b = [&]() {                           // lane 0: copy the B tiles of the next owns_b unit
    while (b_scan < n_mine && b_issued - b_used < kBRing) {
      const Unit u = bit.get(p);
      ++b_scan;
      bit.next(p, G);
      if (!u.owns_b) continue;
      const int slot = b_issued % kBRing;
      uint8_t* bb = smem + p.off_b + (size_t)slot * p.b_bytes;
      const uint32_t bytes = (uint32_t)p.b.kc * tile_bytes(p.b.fmt);
      const bool quant = p.b.fmt != FMT_F16;
      const uint32_t scb = quant ? (uint32_t)p.b.ng * 32u : 0u, zzb = quant ? (uint32_t)p.b.ng * 16u : 0u;
      mbar_expect_tx(b_full + slot, bytes + scb + zzb);
      bulk_g2s(bb, p.b.q + (int64_t)u.tile * p.b.kc * tile_bytes(p.b.fmt), bytes, b_full + slot);
      if (quant) {
        bulk_g2s(bb + p.b_sc_off, p.b.sc + (int64_t)u.tile * p.b.ng * 8, scb, b_full + slot);
        bulk_g2s(bb + p.b_zz_off, p.b.zz + (int64_t)u.tile * p.b.ng * 8, zzb, b_full + slot);
      }
      ++b_issued;
    }
  };
  auto stage_t = [&]() {      // wait (bounded) for t, copy it to shared memory as fp16 hi + lo
    if (lane == 0) {
      counter_wait(p.counters + CNT_T_DONE, (uint32_t)p.a_units, p.dev_status);
      STRACE(5);
    }
    __syncwarp();
    for (int row = 0; row < p.m; ++row) {
      for (int j = lane; j < p.r_pad; j += 32) {
        float v = ld_cg(p.t_ws + (int64_t)row * p.r_pad + j);
        __half hi = __float2half_rn(v);
        ts[row * trow + j] = hi;
        ts[(p.m + row) * trow + j] = __float2half_rn(v - __half2float(hi));
      }
    }
    __threadfence();
    __syncwarp();
    // every CTA reads t exactly once; the last reader returns t_ws and the counters to zero
    uint32_t last = 0;
    if (lane == 0) last = (atomicAdd(p.counters + CNT_T_CONSUMED, 1u) == (uint32_t)G - 1) ? 1u : 0u;
    last = __shfl_sync(0xffffffffu, last, 0);
    if (last) {
      for (int i = lane; i < p.m * p.r_pad; i += 32) p.t_ws[i] = 0.f;
      if (lane == 0) { p.counters[CNT_T_DONE] = 0; p.counters[CNT_T_CONSUMED] = 0; }
    }
    t_staged = true;
  };

  if constexpr (ABF != FMT_NONE) {
    if (have_ab && lane == 0) issue_b();
  }
  const int g = lane >> 2, t4 = lane & 3;
  bool pend = false;            // a split-K ticket whose count has not been looked at yet
  uint32_t pend_cnt = 0;
  int pend_tile = 0, pend_split = 0;
  auto settle = [&]() {         // the last slice to arrive converts the sums of its row tile and clears them
    if (!pend) return;
    pend = false;
    const uint32_t last = __shfl_sync(0xffffffffu, (pend_cnt == (uint32_t)pend_split - 1) ? 1u : 0u, 0);
    if (!last) return;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const int tok = 2 * t4 + (c & 1), row = pend_tile * 16 + g + 8 * (c >> 1);
      if (tok < p.m) {
        float* src = p.y_ws + (int64_t)tok * p.d_out + row;
        store_y(p.y, p.y_dtype, (int64_t)tok * p.d_out + row, ld_cg(src));
        *src = 0.f;
      }
    }
    if (lane == 0) p.counters[CNT_TILE0 + pend_tile] = 0;
  };
  UnitIter eit;
  eit.init(p, (int)blockIdx.x);
  for (int i = 0; i < n_mine; ++i, eit.next(p, G)) {
    const int rb = i & (kRed - 1);
    const Unit u = eit.get(p);
    if (!mbar_wait_warp(red_full + rb, (i / kRed) & 1, p.dev_status, lane)) break;
    float acc[4];
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      float v = 0.f;
#pragma unroll
      for (int w = 0; w < kCW; ++w) v += red[(rb * kCW + w) * 128 + c * 32 + lane];
      acc[c] = v;
    }
    __syncwarp();
    if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(red_free + rb)) : "memory");
    // this lane holds rows (g, g + 8) of the tile and tokens (2*t4, 2*t4 + 1)
    const int row0 = u.tile * 16 + g;
    const int tok0 = 2 * t4;
    if (u.is_a) {
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const int tok = tok0 + (c & 1), row = row0 + 8 * (c >> 1);
        if (tok < p.m) red_add(p.t_ws + (int64_t)tok * p.r_pad + row, acc[c]);
      }
      __syncwarp();      // every lane's adds happen-before lane 0's release
      if (lane == 0) asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(p.counters + CNT_T_DONE) : "memory");
      continue;
    }
    if constexpr (ABF != FMT_NONE) {
      if (u.owns_b) {
        if (!t_staged) stage_t();
        const int slot = b_used % kBRing;
        const uint8_t* bb = smem + p.off_b + (size_t)slot * p.b_bytes;
        if (!mbar_wait_warp(b_full + slot, (b_used / kBRing) & 1, p.dev_status, lane)) break;
        run_b<ABF>(bb, reinterpret_cast<const uint32_t*>(bb + p.b_sc_off), reinterpret_cast<const uint16_t*>(bb + p.b_zz_off),
                   p.b.kc, p.qt_b, p.b.group / 64, lane, ts, trow, p.m, acc);
        __syncwarp();
        ++b_used;
        if (lane == 0) issue_b();
      }
    }
    if (u.split == 1) {
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const int tok = tok0 + (c & 1), row = row0 + 8 * (c >> 1);
        if (tok < p.m) store_y(p.y, p.y_dtype, (int64_t)tok * p.d_out + row, acc[c]);
      }
      continue;
    }
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const int tok = tok0 + (c & 1), row = row0 + 8 * (c >> 1);
      if (tok < p.m) red_add(p.y_ws + (int64_t)tok * p.d_out + row, acc[c]);
    }
    // Split-K ticket.  The counter round trip is long, so its result is only looked at after the next
    // unit has been summed: first settle the previous ticket, then take this one.
    settle();
    __syncwarp();        // every lane's adds happen-before lane 0's release
    if (lane == 0)
      asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;" : "=r"(pend_cnt) : "l"(p.counters + CNT_TILE0 + u.tile) : "memory");
    pend = true; pend_tile = u.tile; pend_split = u.split;
  }
  settle();
  // a CTA without a B-owning unit still takes part in the hand-back of t_ws
  if constexpr (ABF != FMT_NONE) {
    if (have_ab && !t_staged) stage_t();
  }
  if (lane == 0) STRACE(9);
}

// ------------------------------------------------------------------------------------------ host
inline int align_up_i(int v, int a) { return (v + a - 1) / a * a; }

struct SPlan {
  bool ok;
  int grid, smem;
  StreamArgs a;
};

SPlan make_splan(const Handle* h, int m) {
  SPlan pl = {};
  StreamArgs& a = pl.a;
  pl.ok = false;
  if (m < 1 || m > 8) return pl;
  const bool ab = h->cfg.rank > 0;
  const int xbytes = m * (h->cfg.d_in + kXPad) * 2;
  a.qt_w = quantum_tiles(h->w);
  a.qt_a = ab ? quantum_tiles(h->a) : 1;
  a.qt_b = ab ? quantum_tiles(h->b) : 1;
  auto chunk_quanta = [](const WMat& mat, int qt) {
    int cq = kSlotBytes / (qt * tile_bytes(mat.fmt));
    return cq > 2 * kCW ? 2 * kCW : cq;
  };
  a.cq_w = chunk_quanta(h->w, a.qt_w);
  a.cq_a = ab ? chunk_quanta(h->a, a.qt_a) : 1;
  if (a.cq_w < 1 || a.cq_a < 1) return pl;
  const int G_max = 2 * h->sm_count;
  const int tbw = tile_bytes(h->w.fmt);
  const int nq_w = h->w.kc / a.qt_w;

  // shared memory: [ring of slots][X][reduction slots][B ring][t]
  int off = 0;
  const int x_rel = off; off += align_up_i(xbytes, 128);
  const int red_rel = off; off += kRed * kCW * 128 * 4;
  const int b_rel = off;
  a.b_bytes = 0; a.b_sc_off = 0; a.b_zz_off = 0;
  if (ab) {
    int bb = align_up_i(h->b.kc * tile_bytes(h->b.fmt), 128);
    a.b_sc_off = bb; bb += align_up_i(h->b.ng * 32, 128);
    a.b_zz_off = bb; bb += align_up_i(h->b.ng * 16, 128);
    a.b_bytes = bb;
    off += kBRing * bb;
  }
  const int t_rel = off;
  if (ab) off += align_up_i(2 * m * (h->r_pad + kXPad) * 2, 128);
  const int fixed = off;
  a.stages = (kSmemPerCta - fixed) / kSlotBytes;
  if (a.stages > kMaxStages) a.stages = kMaxStages;
  if (a.stages < 3) return pl;
  const int ring = a.stages * kSlotBytes;
  a.off_x = ring + x_rel; a.off_red = ring + red_rel; a.off_b = ring + b_rel; a.off_t = ring + t_rel;
  pl.smem = ring + fixed;

  // backbone split: best balance of units over the grid, units of at least ~8 KB
  int best_split = 1;
  double best_eff = -1.0;
  for (int s = 1; s <= 8 && s <= nq_w; ++s) {
    if (nq_w % s) continue;
    int ubytes = (nq_w / s) * a.qt_w * tbw;
    if (s > 1 && ubytes < 8192) break;
    int units = h->w.nt * s;
    // two CTAs share an SM and its issue slots, so what has to balance is units per SM
    int sms = h->sm_count;
    double per_sm = (double)units / sms;
    double eff = per_sm >= 1.0 ? per_sm / (double)((units + sms - 1) / sms) : per_sm;
    if (s > 1) eff -= 0.02 * (s - 1);                          // split-K has a price
    if (eff > best_eff) { best_eff = eff; best_split = s; }
  }
  a.w_split = best_split;
  a.a_split = 1; a.a_units = 0;
  if (ab) {
    // small A units (>= 4 KB), about one per CTA, so that t is complete early
    const int nq_a = h->a.kc / a.qt_a, tba = tile_bytes(h->a.fmt);
    int want = (G_max + h->a.nt - 1) / h->a.nt;
    int max_by_size = nq_a * a.qt_a * tba / 4096;
    if (want > max_by_size) want = max_by_size;
    if (want > nq_a) want = nq_a;
    if (want < 1) want = 1;
    while (nq_a % want) --want;                               // the split must divide the quanta evenly
    a.a_split = want;
    a.a_units = h->a.nt * a.a_split;
  }
  a.n_units = a.a_units + h->w.nt * a.w_split;
  pl.grid = a.n_units < G_max ? a.n_units : G_max;
  auto shift_of = [](int v) { int sh = 0; while ((1 << sh) < v) ++sh; return (1 << sh) == v ? sh : -1; };
  a.nqu_w = nq_w / a.w_split;
  a.dt_w = pl.grid / a.w_split; a.ds_w = pl.grid % a.w_split;
  a.qpg_shift_w = shift_of(h->w.group / (64 * a.qt_w));
  a.nqu_a = 0; a.dt_a = 0; a.ds_a = 0; a.qpg_shift_a = 0;
  if (ab) {
    a.nqu_a = (h->a.kc / a.qt_a) / a.a_split;
    a.dt_a = pl.grid / a.a_split; a.ds_a = pl.grid % a.a_split;
    a.qpg_shift_a = shift_of(h->a.group / (64 * a.qt_a));
  }
  pl.ok = true;
  return pl;
}

template <auto KERNEL>
cudaError_t launch_stream_kernel(const cudaLaunchConfig_t& cfg, const StreamArgs& args) {
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(KERNEL, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemPerCta);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  return cudaLaunchKernelEx(&cfg, KERNEL, args);
}

template <int WF>
cudaError_t launch_stream_ab(const cudaLaunchConfig_t& cfg, const StreamArgs& args, int abf) {
  switch (abf) {
    case FMT_F16: return launch_stream_kernel<k_decode_stream<WF, FMT_F16>>(cfg, args);
    case FMT_Q4: return launch_stream_kernel<k_decode_stream<WF, FMT_Q4>>(cfg, args);
    case FMT_Q8: return launch_stream_kernel<k_decode_stream<WF, FMT_Q8>>(cfg, args);
    default: return launch_stream_kernel<k_decode_stream<WF, FMT_NONE>>(cfg, args);
  }
}

}  // namespace

bool decode_stream_supported(const Handle* h, int m) {
  if (h->w.fmt != FMT_Q4 && h->w.fmt != FMT_Q3) return false;
  return make_splan(h, m).ok;
}

int decode_stream_grid(const Handle* h, int m) { return make_splan(h, m).grid; }

cudaError_t launch_decode_stream(const Handle* h, const void* x, int m, void* y, cudaStream_t st) {
  SPlan pl = make_splan(h, m);
  if (!pl.ok) return cudaErrorInvalidValue;
  StreamArgs& a = pl.a;
  a.w = h->w; a.a = h->a; a.b = h->b;
  a.x = x; a.y = y;
  a.t_ws = h->t_ws; a.y_ws = h->y_ws; a.counters = h->counters; a.dev_status = h->dev_status;
  a.trace = reinterpret_cast<unsigned long long*>(h->trace);
  a.m = m; a.d_in = h->cfg.d_in; a.d_out = h->cfg.d_out; a.r_pad = h->r_pad;
  a.x_dtype = h->cfg.x_dtype; a.y_dtype = h->cfg.y_dtype;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(pl.grid);
  cfg.blockDim = dim3(kThreadsS);
  cfg.dynamicSmemBytes = pl.smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int abf = h->cfg.rank > 0 ? h->a.fmt : FMT_NONE;
  if (h->w.fmt == FMT_Q4) return launch_stream_ab<FMT_Q4>(cfg, a, abf);
  return launch_stream_ab<FMT_Q3>(cfg, a, abf);
}

}  // namespace eora
