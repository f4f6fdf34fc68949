// Decode kernel family (M <= 64): one launch computes  Y = X.deq(Wq) + (X.A).B  (paper Eq. 4).
//
// Section 4.5 of the paper fuses only the product with B into the quantised mat-vec kernel and
// leaves t = A.x to a separate op.  Here the whole layer is one pass: A is treated as `rank`
// more output rows of the same streaming product over X, and B as `rank` more reduction
// elements of the backbone product with t in the place of X, so Y is written exactly once.
//
// Work decomposition.  A CTA (8 warps) owns one unit = (matrix, 16-row tile, reduction slice).
// Units of A come first in blockIdx order, backbone units after them.  The packed weights of a
// unit are one contiguous byte range; one thread brings them into shared memory with a few bulk
// async copies (cp.async.bulk + mbarrier, no multicast) issued at the very start of the CTA, so
// a whole layer is in flight at once and no registers are spent on prefetch.  Each warp then
// walks its quanta (<= 128 reduction elements sharing one scale / zero-point): codes become the
// exact fp16 integers (q - z) in registers, are multiplied with the activations on the tensor
// cores (mma.m16n8k16, weights as the 16-row operand, fp32 accumulate) and the scale is applied
// once per quantum in fp32.  The 8 warps are then summed through shared memory.
//   A unit       : adds its partial t to the fp32 buffer t_ws (red.add), then bumps T_DONE.
//   backbone unit: the last reduction slice of each row tile also owns the B extension: it waits
//                  (bounded) for T_DONE, reads t, splits it into fp16 hi + lo parts and runs the
//                  B tiles (prefetched with the weights) against them.  With one slice per row
//                  tile the result goes straight to Y; otherwise slices add into y_ws and the
//                  last one to arrive converts.
// All scratch words are returned to zero before the kernel ends, so calls need no memset.
//
// Programmatic dependent launch: the bulk copies of the weights are issued before
// griddepcontrol.wait, i.e. while the previous kernel in the stream is still draining;
// activations and scratch are touched only after it.
#include "decode_common.cuh"

namespace eora {
using namespace dec;
namespace {

constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;
constexpr int kXPad = 32;                 // halves of padding per activation row in shared memory
constexpr int kChunks = 4;                // bulk-copy chunks (one mbarrier each) per unit
constexpr int kUnitBytes = 32 * 1024;     // largest packed-weight slice of one unit
constexpr int kXSmemBudget = 64 * 1024;   // bytes of staged activations per CTA
constexpr int kMaxSmem = 200 * 1024;


// What one CTA streams: a slice of nq quanta of one row tile, (being) copied to shared memory.
struct SliceView {
  const uint8_t* wbuf;      // tile blobs of the slice, first tile of the slice at offset 0
  const uint32_t* sc;       // scales from the first group the slice touches (8 words per group)
  const uint16_t* zz;
  uint64_t* bars;           // kChunks barriers, chunk c covers quanta [c*cq, (c+1)*cq) of the slice
  int nq;                   // quanta in the slice
  int qt;                   // tiles per quantum
  int cq;                   // quanta per chunk
  int group_tiles;          // tiles per quantisation group
  int gofs;                 // tiles between the start of that first group and the slice start
};

// Accumulate the slice against NX activation sources in shared memory (source s at
// xs + s * xsrc_stride halves; row `token` at + token * xrow; reduction index 0 = slice start).
template <int FMT, int MT, int NX>
__device__ __forceinline__ void run_slice(const SliceView& sv, int warp, int lane, const __half* xs, int xrow,
                                          int xsrc_stride, int m_rows, int* dev_status, float (&acc)[MT][4]) {
  constexpr int TB = FMT == FMT_Q4 ? 512 : FMT == FMT_Q3 ? 384 : FMT == FMT_Q8 ? 1024 : 2048;
  const int g = lane >> 2, t = lane & 3;
  int chunk_ready = -1;
#pragma unroll 1
  for (int q = warp; q < sv.nq; q += kWarps) {
    const int chunk = q / sv.cq;
    if (chunk > chunk_ready) {
      mbar_wait_warp(sv.bars + chunk, 0, dev_status, lane);
      chunk_ready = chunk;
    }
    float gacc[MT][4];
    ZC zc;
    uint32_t sc2 = 0;
    if constexpr (is_quant<FMT>()) {
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) gacc[mt][0] = gacc[mt][1] = gacc[mt][2] = gacc[mt][3] = 0.f;
      const int gi = (sv.gofs + q * sv.qt) / sv.group_tiles;
      sc2 = sv.sc[gi * 8 + g];
      make_zc<FMT>(zc, sv.zz[gi * 8 + g]);
    }
#pragma unroll 1
    for (int tt = 0; tt < sv.qt; ++tt) {
      const int tile = q * sv.qt + tt;
      uint32_t a[4][4];
      tile_frags<FMT>(sv.wbuf + tile * TB, lane, zc, a);
      const int koff = tile * 64 + 8 * t;
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
      const float sa = __half2float(__ushort_as_half((unsigned short)(sc2 & 0xffffu)));
      const float sb = __half2float(__ushort_as_half((unsigned short)(sc2 >> 16)));
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
  // shared-memory carve-up (byte offsets from the dynamic shared memory base)
  int off_sc, off_zz, off_b, off_bsc, off_bzz, off_x, off_red;
  unsigned long long* trace;   // optional: 16 timestamps (ns) per CTA, see eora_linear_set_trace
};

#define EORA_TRACE(slot) do { if (p.trace && threadIdx.x == 0) p.trace[(size_t)blockIdx.x * 16 + (slot)] = globaltimer_ns(); } while (0)

// Stage activation rows [0, m) x reduction range [k0, k0 + len) into shared memory as fp16.
__device__ __forceinline__ void stage_x(__half* xs, int xrow, const void* x, int x_dtype, int m, int d_in, int k0, int len) {
  const int chunks = len >> 3;   // 16-byte chunks per row
  for (int row = 0; row < m; ++row) {
    for (int c = threadIdx.x; c < chunks; c += kThreads) {
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
}

// Issue the bulk copies of one slice (quanta [q0, q0 + nq) of row tile `tile`) in kChunks pieces,
// plus (with the first piece) the scales and zero-points of the groups the slice touches.
// Returns the tile offset of the slice start inside its first group.
__device__ __forceinline__ int issue_slice(const WMat& m, int tile, int q0, int nq, int qt, int cq, uint8_t* wbuf,
                                           uint32_t* sc_s, uint16_t* zz_s, uint64_t* bars) {
  const int tb = tile_bytes(m.fmt);
  const uint8_t* src = m.q + ((int64_t)tile * m.kc + (int64_t)q0 * qt) * tb;
  const bool quant = m.fmt == FMT_Q4 || m.fmt == FMT_Q3 || m.fmt == FMT_Q8;
  const int gt = m.group / 64;
  const int g0 = (q0 * qt) / gt;
  for (int c = 0; c < kChunks; ++c) {
    int qa = c * cq, qb = (c + 1) * cq < nq ? (c + 1) * cq : nq;
    uint32_t bytes = qb > qa ? (uint32_t)(qb - qa) * qt * tb : 0u;
    uint32_t extra_sc = 0, extra_zz = 0;
    if (c == 0 && quant) {
      const int g1 = ((q0 + nq) * qt + gt - 1) / gt;
      extra_sc = (uint32_t)(g1 - g0) * 32u;
      extra_zz = (uint32_t)(g1 - g0) * 16u;
    }
    mbar_expect_tx(bars + c, bytes + extra_sc + extra_zz);
    if (bytes) bulk_g2s(wbuf + (size_t)qa * qt * tb, src + (size_t)qa * qt * tb, bytes, bars + c);
    if (extra_sc) {
      bulk_g2s(sc_s, m.sc + ((int64_t)tile * m.ng + g0) * 8, extra_sc, bars + c);
      bulk_g2s(zz_s, m.zz + ((int64_t)tile * m.ng + g0) * 8, extra_zz, bars + c);
    }
  }
  return q0 * qt - g0 * gt;
}

template <int WF, int ABF, int MT>
__global__ void __launch_bounds__(kThreads, MT == 1 ? 3 : (MT == 2 ? 2 : 1)) k_decode(const DecodeArgs p) {
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ __align__(8) uint64_t bars[2 * kChunks];
  __shared__ uint32_t s_flag;

  asm volatile("griddepcontrol.launch_dependents;");
  EORA_TRACE(0);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int unit = blockIdx.x;
  const bool is_a = unit < p.a_units;
  int tile, slice, split;
  if (is_a) { tile = unit / p.a_split; slice = unit % p.a_split; split = p.a_split; }
  else { int u = unit - p.a_units; tile = u / p.w_split; slice = u % p.w_split; split = p.w_split; }
  const WMat& mat = is_a ? p.a : p.w;
  const int qt = is_a ? p.qt_a : p.qt_w;
  const int nq_all = mat.kc / qt;                   // quanta per row tile
  const int q0 = (int)((int64_t)nq_all * slice / split), q1 = (int)((int64_t)nq_all * (slice + 1) / split);
  const int nq = q1 - q0;
  const int cq = (nq + kChunks - 1) / kChunks;
  const int k_base = q0 * qt * 64, k_len = nq * qt * 64;
  const int xrow = k_len + kXPad;
  const bool owns_b = !is_a && slice == split - 1 && p.a_units > 0;
  const int nqb = owns_b ? p.b.kc / p.qt_b : 0;
  const int cqb = owns_b ? (nqb + kChunks - 1) / kChunks : 1;

  uint8_t* wbuf = smem;
  uint32_t* sc_s = reinterpret_cast<uint32_t*>(smem + p.off_sc);
  uint16_t* zz_s = reinterpret_cast<uint16_t*>(smem + p.off_zz);
  uint8_t* bbuf = smem + p.off_b;
  uint32_t* bsc_s = reinterpret_cast<uint32_t*>(smem + p.off_bsc);
  uint16_t* bzz_s = reinterpret_cast<uint16_t*>(smem + p.off_bzz);
  __half* xs = reinterpret_cast<__half*>(smem + p.off_x);
  float* red = reinterpret_cast<float*>(smem + p.off_red);

  // the slice start inside its first quantisation group, in tiles (same formula as issue_slice)
  const int gofs = q0 * qt - ((q0 * qt) / (mat.group / 64)) * (mat.group / 64);

  if (threadIdx.x == 0) {
    for (int i = 0; i < 2 * kChunks; ++i) mbar_init(bars + i, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    // weights are immutable: their copies may start before the previous kernel has finished
    issue_slice(mat, tile, q0, nq, qt, cq, wbuf, sc_s, zz_s, bars);
    if (owns_b) issue_slice(p.b, tile, 0, nqb, p.qt_b, cqb, bbuf, bsc_s, bzz_s, bars + kChunks);
  }
  EORA_TRACE(1);
  asm volatile("griddepcontrol.wait;" ::: "memory");
  EORA_TRACE(2);
  stage_x(xs, xrow, p.x, p.x_dtype, p.m, p.d_in, k_base, k_len);
  __syncthreads();      // barriers initialised, X staged
  EORA_TRACE(3);

  float acc[MT][4];
#pragma unroll
  for (int mt = 0; mt < MT; ++mt) acc[mt][0] = acc[mt][1] = acc[mt][2] = acc[mt][3] = 0.f;

  SliceView sv;
  sv.wbuf = wbuf; sv.sc = sc_s; sv.zz = zz_s; sv.bars = bars; sv.nq = nq; sv.qt = qt; sv.cq = cq;
  sv.group_tiles = mat.group / 64; sv.gofs = gofs;
  if (is_a) {
    if constexpr (ABF != FMT_NONE) run_slice<ABF, MT, 1>(sv, warp, lane, xs, xrow, 0, p.m, p.dev_status, acc);
  } else {
    run_slice<WF, MT, 1>(sv, warp, lane, xs, xrow, 0, p.m, p.dev_status, acc);
  }

  EORA_TRACE(4);
  // ---- B extension: the last slice of a backbone row tile adds (X.A).B for its 16 output columns
  if constexpr (ABF != FMT_NONE) {
    if (owns_b) {
      __syncthreads();                                   // everyone is done reading the staged X
      if (threadIdx.x == 0) {
        counter_wait(p.counters + CNT_T_DONE, (uint32_t)p.a_units, p.dev_status);
      }
      __syncthreads();
      EORA_TRACE(5);
      // t -> fp16 hi + lo in shared memory (two sources), rows padded like X
      const int trow = p.r_pad + kXPad;
      __half* ts = xs;
      for (int row = 0; row < p.m; ++row) {
        for (int j = threadIdx.x; j < p.r_pad; j += kThreads) {
          float v = ld_cg(p.t_ws + (int64_t)row * p.r_pad + j);
          __half hi = __float2half_rn(v);
          __half lo = __float2half_rn(v - __half2float(hi));
          ts[row * trow + j] = hi;
          ts[(p.m + row) * trow + j] = lo;
        }
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
      EORA_TRACE(6);
      SliceView sb;
      sb.wbuf = bbuf; sb.sc = bsc_s; sb.zz = bzz_s; sb.bars = bars + kChunks; sb.nq = nqb; sb.qt = p.qt_b; sb.cq = cqb;
      sb.group_tiles = p.b.group / 64; sb.gofs = 0;
      run_slice<ABF, MT, 2>(sb, warp, lane, ts, trow, p.m * trow, p.m, p.dev_status, acc);
    }
  }

  EORA_TRACE(7);
  // ---- sum the 8 warps
#pragma unroll
  for (int mt = 0; mt < MT; ++mt)
#pragma unroll
    for (int c = 0; c < 4; ++c) red[warp * (MT * 128) + (mt * 4 + c) * 32 + lane] = acc[mt][c];
  __syncthreads();
  EORA_TRACE(8);

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
    for (int w = 0; w < kWarps; ++w) v += red[w * (MT * 128) + idx];
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
    EORA_TRACE(9);
    return;
  }
  if (split == 1) {
    for (int idx = threadIdx.x; idx < MT * 128; idx += kThreads) {
      int token, row;
      out_pos(idx, token, row);
      if (token < p.m) store_y(p.y, p.y_dtype, (int64_t)token * p.d_out + row, warp_sum(idx));
    }
    EORA_TRACE(9);
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
  EORA_TRACE(9);
}

// ------------------------------------------------------------------------------------------ host
struct Plan {
  int a_units, a_split, w_split, smem;
  int off_sc, off_zz, off_b, off_bsc, off_bzz, off_x, off_red;
};

inline int align_up_i(int v, int a) { return (v + a - 1) / a * a; }

Plan make_plan(const Handle* h, int m) {
  Plan pl = {};
  const int slots = 3 * h->sm_count;
  const int mt = m <= 8 ? 1 : m <= 16 ? 2 : m <= 32 ? 4 : 8;
  const int max_slice_k_x = (kXSmemBudget / (2 * m)) & ~127;          // activations staged per CTA
  auto max_slice_k = [&](const WMat& mat) {
    int by_bytes = ((kUnitBytes / tile_bytes(mat.fmt)) * 64) & ~127;
    return by_bytes < max_slice_k_x ? by_bytes : max_slice_k_x;
  };
  auto split_for = [&](const WMat& mat, int want) {
    int qt = quantum_tiles(mat), nq = mat.kc / qt;
    int msk = max_slice_k(mat);
    int min_split = (mat.k_red + msk - 1) / msk;
    int s = want > min_split ? want : min_split;
    if (s > nq) s = nq;
    if (s < 1) s = 1;
    return s;
  };
  auto slice_len = [&](const WMat& mat, int split) {      // longest slice in reduction elements
    int qt = quantum_tiles(mat), nq = mat.kc / qt, best = 0;
    for (int s = 0; s < split; ++s) {
      int l = (int)(((int64_t)nq * (s + 1) / split) - ((int64_t)nq * s / split)) * qt * 64;
      if (l > best) best = l;
    }
    return best;
  };
  int want_w = (h->w.nt * 4 >= slots * 3) ? 1 : (slots + h->w.nt - 1) / h->w.nt;
  pl.w_split = split_for(h->w, want_w);
  const bool ab = h->cfg.rank > 0;
  if (ab) {
    // size A units like backbone units (in bytes streamed)
    int64_t w_unit_bytes = wmat_q_bytes(h->w.fmt, 1, h->w.kc) / pl.w_split;
    if (w_unit_bytes < 8192) w_unit_bytes = 8192;
    int64_t a_tile_bytes = wmat_q_bytes(h->a.fmt, 1, h->a.kc);
    pl.a_split = split_for(h->a, (int)((a_tile_bytes + w_unit_bytes - 1) / w_unit_bytes));
    pl.a_units = h->a.nt * pl.a_split;
  } else {
    pl.a_split = 1;
  }
  int lw = slice_len(h->w, pl.w_split), la = ab ? slice_len(h->a, pl.a_split) : 0;
  int wbytes = lw / 64 * tile_bytes(h->w.fmt);
  if (ab && la / 64 * tile_bytes(h->a.fmt) > wbytes) wbytes = la / 64 * tile_bytes(h->a.fmt);
  int max_k = lw > la ? lw : la;
  int groups_w = lw / h->w.group + 2;
  int groups_a = ab ? la / h->a.group + 2 : 0;
  int groups = groups_w > groups_a ? groups_w : groups_a;
  int off = align_up_i(wbytes, 128);
  pl.off_sc = off; off += align_up_i(groups * 32, 128);
  pl.off_zz = off; off += align_up_i(groups * 16, 128);
  pl.off_b = off; off += ab ? align_up_i(h->b.kc * tile_bytes(h->b.fmt), 128) : 0;
  pl.off_bsc = off; off += ab ? align_up_i((h->b.ng + 1) * 32, 128) : 0;
  pl.off_bzz = off; off += ab ? align_up_i((h->b.ng + 1) * 16, 128) : 0;
  pl.off_x = off;
  int xb = m * (max_k + kXPad) * 2;
  int tb = ab ? 2 * m * (h->r_pad + kXPad) * 2 : 0;
  off += align_up_i(xb > tb ? xb : tb, 128);
  pl.off_red = off; off += kWarps * mt * 128 * 4;
  pl.smem = off;
  return pl;
}

template <auto KERNEL>
cudaError_t launch_kernel(const cudaLaunchConfig_t& cfg, const DecodeArgs& args) {
  static bool attr_set = false;   // one per kernel (KERNEL is a template argument)
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(KERNEL, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmem);
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
  return pl.smem <= kMaxSmem;
}

void decode_make_plan(Handle* h) { h->plan = DecodePlan(); }

int decode_launch_count(const Handle*, int) { return 1; }

int decode_grid(const Handle* h, int m) {
  if (decode_stream_supported(h, m)) return decode_stream_grid(h, m);
  Plan pl = make_plan(h, m);
  return pl.a_units + h->w.nt * pl.w_split;
}

cudaError_t launch_decode_forward(const Handle* h, const void* x, int m, void* y, cudaStream_t st) {
  if (decode_stream_supported(h, m)) return launch_decode_stream(h, x, m, y, st);
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
  a.off_sc = pl.off_sc; a.off_zz = pl.off_zz; a.off_b = pl.off_b; a.off_bsc = pl.off_bsc; a.off_bzz = pl.off_bzz;
  a.off_x = pl.off_x; a.off_red = pl.off_red;
  a.trace = reinterpret_cast<unsigned long long*>(h->trace);
  int grid = pl.a_units + h->w.nt * pl.w_split;
  int mt = m <= 8 ? 1 : m <= 16 ? 2 : m <= 32 ? 4 : 8;
  int abf = h->cfg.rank > 0 ? h->a.fmt : FMT_NONE;
  if (h->w.fmt == FMT_Q4) return launch_ab<FMT_Q4>(a, abf, mt, grid, pl.smem, st);
  return launch_ab<FMT_Q3>(a, abf, mt, grid, pl.smem, st);
}

}  // namespace eora
