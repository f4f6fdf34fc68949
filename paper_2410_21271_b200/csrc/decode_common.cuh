// Device helpers shared by the decode kernels: PTX wrappers (mbarrier, bulk copy, mma) and the
// in-register dequantisation of one 16 x 64 tile into tensor-core operand registers.
#pragma once
#include "eora_common.cuh"

namespace eora {
namespace dec {

// ------------------------------------------------------------------------------------------ PTX
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
               : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long globaltimer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
constexpr unsigned long long kWaitLimitNs = 1000000000ull;   // every device-side wait gives up after 1 s
// Bounded wait: returns false (and latches the status word) if the phase does not complete in time.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, int* dev_status) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = globaltimer_ns();
  for (;;) {
#pragma unroll 1
    for (int it = 0; it < 64; ++it)
      if (mbar_try_wait(bar, parity)) return true;
    if (globaltimer_ns() - t0 > kWaitLimitNs) break;
  }
  atomicExch(dev_status, EORA_ERR_DEVICE_TIMEOUT);
  return false;
}
// The same wait for a whole warp.  Only lane 0 polls, and it backs off between polls: a warp-wide
// spin costs a shared-memory access per poll, and a dozen spinning warps are enough to starve the
// bulk-copy engine and the tensor core of shared-memory bandwidth.  Once lane 0 has seen the phase
// complete, every lane tests it once itself (which succeeds at once) so that each thread has its own
// acquire of the data behind the barrier.
__device__ __forceinline__ bool mbar_wait_warp(uint64_t* bar, uint32_t parity, int* dev_status, int lane) {
  if (mbar_try_wait(bar, parity)) return true;
  int ok = 1;
  if (lane == 0) {
    const unsigned long long t0 = globaltimer_ns();
    ok = 0;
    for (;;) {
#pragma unroll 1
      for (int it = 0; it < 64 && !ok; ++it) {
        __nanosleep(40);
        ok = mbar_try_wait(bar, parity) ? 1 : 0;
      }
      if (ok || globaltimer_ns() - t0 > kWaitLimitNs) break;
    }
    if (!ok) atomicExch(dev_status, EORA_ERR_DEVICE_TIMEOUT);
  }
  ok = __shfl_sync(0xffffffffu, ok, 0);
  if (ok) { while (!mbar_try_wait(bar, parity)) {} }
  return ok != 0;
}

// Bounded spin on a global counter reaching `target`.
__device__ __forceinline__ uint32_t ld_acquire(const uint32_t* p);
__device__ __forceinline__ bool counter_wait(const uint32_t* cnt, uint32_t target, int* dev_status) {
  const unsigned long long t0 = globaltimer_ns();
  for (;;) {
#pragma unroll 1
    for (int it = 0; it < 64; ++it) {
      if (ld_acquire(cnt) >= target) return true;
      __nanosleep(32);
    }
    if (globaltimer_ns() - t0 > kWaitLimitNs) break;
  }
  atomicExch(dev_status, EORA_ERR_DEVICE_TIMEOUT);
  return false;
}
// global -> shared bulk copy of `bytes` (multiple of 16; both addresses 16-byte aligned)
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
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
__device__ __forceinline__ void mma16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// ------------------------------------------------------------------------------------------ dequant
// Per-quantum constants of the two rows a lane owns: fp16x2 values that turn the magic-number
// form of a code (1024 + q * 2^s as fp16) into the exact integer q - z.
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

// (a & mask) | c in ONE instruction.  Written as `(a & mask) | kMagic` with two immediates the compiler
// emits two logic instructions (an instruction holds only one 32-bit immediate), and those run on the
// half-rate integer pipe that bounds the decode kernel; with the constant in a register it is one LOP3.
__device__ __forceinline__ uint32_t and_or(uint32_t a, uint32_t mask, uint32_t c) {
  uint32_t d;
  asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(a), "r"(mask), "r"(c));
  return d;
}

template <int FMT> constexpr bool is_quant() { return FMT == FMT_Q4 || FMT == FMT_Q3 || FMT == FMT_Q8; }

// Build the A-operand registers of the four mma of one tile from its blob in shared memory.
// a[i][*]: mma i = 2*blk + sub; entries are fp16x2.
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t d;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
  return d;
}

// 2:4 expansion table: for the position nibble p0 | p1 << 2 of a quad, the two byte-permute selectors that
// spread the quad's two kept fp16 values (one register) over its four positions (two registers), zero
// elsewhere.  Low half: selector of positions (0, 1), high half: of positions (2, 3).  Selector bytes: 0x10 =
// first value, 0x32 = second value, 0x44 = zero (the permute's other operand).
__host__ __device__ constexpr uint32_t sp24_selectors(uint32_t nib) {
  const uint32_t p0 = nib & 3u, p1 = nib >> 2;
  uint32_t r = 0;
  for (uint32_t e = 0; e < 4; ++e) {
    const uint32_t sel = e == p0 ? 0x10u : e == p1 ? 0x32u : 0x44u;
    r |= sel << (8 * e);
  }
  return r;
}
constexpr int kSp24LutBytes = 64;       // 16 entries; every entry in its own shared-memory bank

// `aux`: shared-memory address (32-bit, shared window) of the 2:4 expansion table; unused by other formats.
template <int FMT>
__device__ __forceinline__ void tile_frags(const uint8_t* blob, int lane, const ZC& zc, uint32_t (&a)[4][4], uint32_t aux = 0) {
  if constexpr (FMT == FMT_Q4) {
    const uint4 v = *reinterpret_cast<const uint4*>(blob + lane * 16);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int part = 0; part < 4; ++part) {
      const int hf = part & 1, blk = part >> 1;
      uint32_t lo = w[part], hi = w[part] >> 8;
      uint32_t h0 = and_or(lo, 0x000f000fu, kMagic), h1 = and_or(lo, 0x00f000f0u, kMagic);
      uint32_t h2 = and_or(hi, 0x000f000fu, kMagic), h3 = and_or(hi, 0x00f000f0u, kMagic);
      a[blk * 2 + 0][hf] = h2sub(h0, zc.c[hf][0]);
      a[blk * 2 + 0][hf + 2] = h2fma(h1, 0x2C002C00u, zc.c[hf][1]);   // * 1/16
      a[blk * 2 + 1][hf] = h2sub(h2, zc.c[hf][0]);
      a[blk * 2 + 1][hf + 2] = h2fma(h3, 0x2C002C00u, zc.c[hf][1]);
    }
  } else if constexpr (FMT == FMT_Q3) {
    const uint2 v01 = *reinterpret_cast<const uint2*>(blob + lane * 8);
    const uint32_t v2 = *reinterpret_cast<const uint32_t*>(blob + 256 + lane * 4);
    const uint32_t w[3] = {v01.x, v01.y, v2};
    const uint32_t ws[3] = {v01.x >> 9, v01.y >> 9, v2 >> 9};
#pragma unroll
    for (int p = 0; p < 16; ++p) {
      const int part = p >> 2, j = p & 3, hf = part & 1, blk = part >> 1;
      uint32_t v;
      if (p < 15) {
        const int wi = p / 5, f = p % 5, ff = f >= 3 ? f - 3 : f;
        const uint32_t src = f >= 3 ? ws[wi] : w[wi];
        const uint32_t h = and_or(src, 0x00070007u << (3 * ff), kMagic);
        if (ff == 0) v = h2sub(h, zc.c[hf][0]);
        else if (ff == 1) v = h2fma(h, 0x30003000u, zc.c[hf][1]);   // * 1/8
        else v = h2fma(h, 0x24002400u, zc.c[hf][2]);                // * 1/64
      } else {
        uint32_t h = and_or(w[0] >> 15, 0x00010001u, kMagic);
        h = and_or(w[1] >> 14, 0x00020002u, h);
        h = and_or(w[2] >> 13, 0x00040004u, h);
        v = h2sub(h, zc.c[hf][0]);
      }
      a[blk * 2 + (j >> 1)][hf + 2 * (j & 1)] = v;
    }
  } else if constexpr (FMT == FMT_Q8) {
#pragma unroll
    for (int pl = 0; pl < 2; ++pl) {
      const uint4 u = *reinterpret_cast<const uint4*>(blob + pl * 512 + lane * 16);
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
        const uint32_t w0 = hf ? u.z : u.x, w1 = hf ? u.w : u.y;
        a[pl * 2 + 0][hf] = h2sub(and_or(w0, 0x00ff00ffu, kMagic), zc.c[hf][0]);
        a[pl * 2 + 0][hf + 2] = h2sub(and_or(w0 >> 8, 0x00ff00ffu, kMagic), zc.c[hf][0]);
        a[pl * 2 + 1][hf] = h2sub(and_or(w1, 0x00ff00ffu, kMagic), zc.c[hf][0]);
        a[pl * 2 + 1][hf + 2] = h2sub(and_or(w1 >> 8, 0x00ff00ffu, kMagic), zc.c[hf][0]);
      }
    }
  } else if constexpr (FMT == FMT_F16) {
#pragma unroll
    for (int part = 0; part < 4; ++part) {
      const int hf = part & 1, blk = part >> 1;
      const uint4 u = *reinterpret_cast<const uint4*>(blob + part * 512 + lane * 16);
      a[blk * 2 + 0][hf] = u.x;
      a[blk * 2 + 0][hf + 2] = u.y;
      a[blk * 2 + 1][hf] = u.z;
      a[blk * 2 + 1][hf + 2] = u.w;
    }
  } else if constexpr (FMT == FMT_SP24) {
    const uint32_t meta = *reinterpret_cast<const uint32_t*>(blob + 1024 + lane * 4);
#pragma unroll
    for (int blk = 0; blk < 2; ++blk) {
      const uint4 u = *reinterpret_cast<const uint4*>(blob + blk * 512 + lane * 16);
      const uint32_t vv[2][2] = {{u.x, u.y}, {u.z, u.w}};       // [hf][quad]: the quad's two kept values
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
#pragma unroll
        for (int quad = 0; quad < 2; ++quad) {
          const uint32_t nib = (meta >> (8 * (blk * 2 + hf) + 4 * quad)) & 15u;
          uint32_t sel;
          asm volatile("ld.shared.u32 %0, [%1];" : "=r"(sel) : "r"(aux + nib * 4));
          a[blk * 2 + quad][hf] = prmt(vv[hf][quad], 0u, sel);
          a[blk * 2 + quad][hf + 2] = prmt(vv[hf][quad], 0u, sel >> 16);
        }
      }
    }
  }
}


// One blob: 16 rows x 128 reduction elements times the activation fragments -> tot (this lane's four
// entries of the 16 x 8 result: rows g / g + 8, tokens 2t / 2t + 1).
template <int FMT, bool HILO>
__device__ __forceinline__ void blob_product(const uint8_t* blob, int lane, uint32_t sz2, const uint32_t (&xr)[16],
                                             const uint32_t (&xl)[16], float (&tot)[4], uint32_t aux = 0) {
  constexpr int tb = tile_bytes(FMT);
  constexpr bool quant = fmt_quantised(FMT);
  const int g = lane >> 2;
  // Two independent accumulator chains per tile: the four mma of a tile would otherwise wait for one
  // another (an mma takes ~30 cycles to deliver its accumulator), and with four warps per scheduler that
  // latency is not hidden.
  float acc[2][4];
#pragma unroll
  for (int k = 0; k < 4; ++k) { acc[0][k] = 0.f; acc[1][k] = 0.f; tot[k] = 0.f; }
  ZC zc;
  float s_a = 0.f, s_b = 0.f;
#pragma unroll
  for (int c = 0; c < 2; ++c) {
    if constexpr (quant) {
      if (c == 0 || sz2) {
        const uint8_t* sz = blob + 2 * tb + c * kSzEntryBytes;      // c != 0 only with two entries
        const uint32_t s2 = reinterpret_cast<const uint32_t*>(sz)[g];
        const uint32_t z2 = reinterpret_cast<const uint16_t*>(sz + 32)[g];
        make_zc<FMT>(zc, z2);
        s_a = __half2float(__ushort_as_half((unsigned short)(s2 & 0xffffu)));
        s_b = __half2float(__ushort_as_half((unsigned short)(s2 >> 16)));
      }
    }
    uint32_t a[4][4];
    tile_frags<FMT>(blob + c * tb, lane, zc, a, aux);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      mma16816(acc[i & 1], a[i], xr[8 * c + 2 * i], xr[8 * c + 2 * i + 1]);
      if constexpr (HILO) mma16816(acc[i & 1], a[i], xl[8 * c + 2 * i], xl[8 * c + 2 * i + 1]);
    }
    if constexpr (quant) {
      if (c == 1 || sz2) {
        tot[0] = fmaf(acc[0][0] + acc[1][0], s_a, tot[0]); tot[1] = fmaf(acc[0][1] + acc[1][1], s_a, tot[1]);
        tot[2] = fmaf(acc[0][2] + acc[1][2], s_b, tot[2]); tot[3] = fmaf(acc[0][3] + acc[1][3], s_b, tot[3]);
#pragma unroll
        for (int k = 0; k < 4; ++k) { acc[0][k] = 0.f; acc[1][k] = 0.f; }
      }
    }
  }
  if constexpr (!quant) {
#pragma unroll
    for (int k = 0; k < 4; ++k) tot[k] = acc[0][k] + acc[1][k];
  }
}


__device__ __forceinline__ void store_y(void* y, int dtype, int64_t i, float v) {
  if (dtype == EORA_Y_F16) reinterpret_cast<__half*>(y)[i] = __float2half_rn(v);
  else if (dtype == EORA_Y_BF16) reinterpret_cast<__nv_bfloat16*>(y)[i] = __float2bfloat16_rn(v);
  else reinterpret_cast<float*>(y)[i] = v;
}

}  // namespace dec
}  // namespace eora
