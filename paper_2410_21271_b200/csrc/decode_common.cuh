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
// The same test, but the thread may stay suspended (taking no issue slots) until the phase completes or `ns` nanoseconds
// have passed: what a waiting loop polls with, so that many waiting warps do not crowd out the working ones.
__device__ __forceinline__ bool mbar_try_wait_susp(uint64_t* bar, uint32_t parity, uint32_t ns) {
  uint32_t ok;
  asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
               : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity), "r"(ns) : "memory");
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
      if (mbar_try_wait_susp(bar, parity, 20000u)) return true;
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
// The same without the back-off, for hand-overs that are short and sit on the critical path of a pipeline (a sleeping
// poll adds up to its period to every hand-over).  The polling try_wait suspends the thread until the phase completes.
__device__ __forceinline__ bool mbar_wait_warp_fast(uint64_t* bar, uint32_t parity, int* dev_status, int lane) {
  // The vote makes the lanes take the same way even if they arrive one after the other (a lane that saw the phase
  // complete and left would leave the others waiting for it in the shuffle below).
  if (__all_sync(0xffffffffu, mbar_try_wait(bar, parity) ? 1 : 0)) return true;
  int ok = 1;
  if (lane == 0) {
    const unsigned long long t0 = globaltimer_ns();
    ok = 0;
    for (;;) {
#pragma unroll 1
      for (int it = 0; it < 256 && !ok; ++it) ok = mbar_try_wait_susp(bar, parity, 20000u) ? 1 : 0;
      if (ok || globaltimer_ns() - t0 > kWaitLimitNs) break;
    }
    if (!ok) atomicExch(dev_status, EORA_ERR_DEVICE_TIMEOUT);
  }
  ok = __shfl_sync(0xffffffffu, ok, 0);
  if (ok) { while (!mbar_try_wait(bar, parity)) {} }
  return ok != 0;
}

// Wait, for at most two milliseconds and without touching the status word, for a bulk copy that may still be in flight:
// used by a warp that has already given up and only has to let its copies land before it leaves.
__device__ __forceinline__ void mbar_drain_warp(uint64_t* bar, uint32_t parity, int lane) {
  if (lane == 0) {
    const unsigned long long t0 = globaltimer_ns();
    while (!mbar_try_wait(bar, parity) && globaltimer_ns() - t0 < 2000000ull) __nanosleep(200);
  }
  __syncwarp();
}

// Bounded spin on a global counter reaching `target`.
__device__ __forceinline__ uint32_t ld_acquire(const uint32_t* p);
__device__ __forceinline__ bool counter_wait(const uint32_t* cnt, uint32_t target, int* dev_status,
                                             unsigned long long limit_ns = kWaitLimitNs) {
  const unsigned long long t0 = globaltimer_ns();
  for (;;) {
#pragma unroll 1
    for (int it = 0; it < 64; ++it) {
      if (ld_acquire(cnt) >= target) return true;
      __nanosleep(32);
    }
    if (globaltimer_ns() - t0 > limit_ns) break;
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

template <int FMT> constexpr bool is_quant() { return fmt_quantised(FMT); }

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

// The eight byte quads (one code per byte) of a lane's 32 codes of a 3-bit tile: q[part][quad].
__device__ __forceinline__ void q3_quads(uint32_t w0, uint32_t w1, uint32_t w2, uint32_t (&q)[4][2]) {
  const uint32_t w[3] = {w0, w1, w2};
#pragma unroll
  for (int p = 0; p < 3; ++p) {
    q[p][0] = w[p] & 0x07070707u;
    q[p][1] = (w[p] >> 3) & 0x07070707u;
  }
  q[3][0] = and_or(w2 >> 4, 0x04040404u, (w0 >> 6) & 0x03030303u);
  q[3][1] = and_or(w2 >> 5, 0x04040404u, (w1 >> 6) & 0x03030303u);
}
// Two neighbouring codes of a byte quad as fp16x2 (1024 + c0, 1024 + c1): which = 0: bytes 0, 1; 1: bytes 2, 3.
__device__ __forceinline__ uint32_t quad_pair(uint32_t quad, int which) {
  return prmt(quad, 0x64646464u, which ? 0x4342u : 0x4140u);
}

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
    uint32_t q[4][2];
    q3_quads(v01.x, v01.y, v2, q);
#pragma unroll
    for (int part = 0; part < 4; ++part) {
      const int hf = part & 1, blk = part >> 1;
#pragma unroll
      for (int quad = 0; quad < 2; ++quad) {          // quad = which of the part's two mma
        a[blk * 2 + quad][hf] = h2sub(quad_pair(q[part][quad], 0), zc.c[hf][0]);
        a[blk * 2 + quad][hf + 2] = h2sub(quad_pair(q[part][quad], 1), zc.c[hf][0]);
      }
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
  } else if constexpr (FMT == FMT_SQ4) {
    // 2:4 pattern with 4-bit kept values: the quad's two codes -> exact fp16 (q - z), then spread like SP24
    const uint2 v = *reinterpret_cast<const uint2*>(blob + lane * 8);
    const uint32_t meta = *reinterpret_cast<const uint32_t*>(blob + 256 + lane * 4);
#pragma unroll
    for (int blk = 0; blk < 2; ++blk) {
      const uint32_t w = blk ? v.y : v.x;
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
#pragma unroll
        for (int quad = 0; quad < 2; ++quad) {
          const uint32_t kept = h2sub(and_or(w >> (8 * hf + 4 * quad), 0x000f000fu, kMagic), zc.c[hf][0]);
          const uint32_t nib = (meta >> (8 * (blk * 2 + hf) + 4 * quad)) & 15u;
          uint32_t sel;
          asm volatile("ld.shared.u32 %0, [%1];" : "=r"(sel) : "r"(aux + nib * 4));
          a[blk * 2 + quad][hf] = prmt(kept, 0u, sel);
          a[blk * 2 + quad][hf + 2] = prmt(kept, 0u, sel >> 16);
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


// ------------------------------------------------------------------------------------------ integer path (M = 1)
// With a single token the fp16 tensor-core product wastes seven of its eight columns and needs the codes as fp16 pairs
// (one conversion per two codes).  The integer product keeps the codes as bytes (one and-or extracts four of them) and
// multiplies them with mma.m16n8k32 (s8 x s8 -> s32): a 16 x 128 blob is four instructions.  The 128 activations of a
// pair are turned once into a 16-bit block fixed-point number, x = v * 2^e with |v| <= 32639 and one power-of-two scale
// per pair (so the products are exact and one-hot inputs reproduce the weights bit for bit), split into two signed byte
// planes (v = 256 * high + low) that are columns 0 and 1 of the MMA's narrow operand.  Zero-point and scales follow per
// group, in fp32:   y += s * 2^e * (sum q v - z * sum v).
struct XI8 {
  uint32_t b[4][2];         // this lane's registers of the narrow operand for the four MMAs of a pair (zero for columns >= 2)
  int sum[2];               // sum of v over tile c of the pair (all lanes hold it)
  float scale;              // 2^e
};

__device__ __forceinline__ void mma16832_s8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// x: token 0's activations (fp16 or bf16 bits), pair: which 128 of them.  Lane l converts elements 4l .. 4l + 3; the
// byte planes are then handed to the lanes that own them in the MMA's operand layout: lane (g, t) holds column g (0: low
// plane, 1: high plane, others: zero) and, for MMA j (tile j / 2, half j % 2 of the tile), the eight reduction elements
// 32 j + 8 t .. + 7 -- the ones lane t's weight registers of that MMA hold (in the order the and-or delivers the codes).
template <int FMT>
__device__ __forceinline__ void load_x_i8(XI8& xi, const void* x, bool bf16, uint32_t pair, int lane) {
  const uint16_t* src = reinterpret_cast<const uint16_t*>(x) + pair * 128 + 4 * lane;
  uint2 u;
  asm volatile("ld.global.cg.v2.u32 {%0,%1}, [%2];" : "=r"(u.x), "=r"(u.y) : "l"(src) : "memory");
  float f[4];
  if (bf16) {
    f[0] = __uint_as_float(u.x << 16); f[1] = __uint_as_float(u.x & 0xffff0000u);
    f[2] = __uint_as_float(u.y << 16); f[3] = __uint_as_float(u.y & 0xffff0000u);
  } else {
    const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&u.x)), b = __half22float2(*reinterpret_cast<const __half2*>(&u.y));
    f[0] = a.x; f[1] = a.y; f[2] = b.x; f[3] = b.y;
  }
  float am = fmaxf(fmaxf(fabsf(f[0]), fabsf(f[1])), fmaxf(fabsf(f[2]), fabsf(f[3])));
  am = __uint_as_float(__reduce_max_sync(0xffffffffu, __float_as_uint(am)));      // non-negative floats order like integers
  const uint32_t eb = __float_as_uint(am * 1.00396f) >> 23;           // biased exponent of a value just above the maximum
  const bool live = eb >= 15u && eb < 255u;
  const float inv = live ? __uint_as_float((268u - eb) << 23) : 0.f;   // 2^(14 - exponent): |v| <= 32639 = 127 * 256 + 127
  xi.scale = live ? __uint_as_float((eb - 14u) << 23) : 0.f;           // 2^(exponent - 14)
  int v[4], s = 0;
#pragma unroll
  for (int e = 0; e < 4; ++e) { v[e] = __float2int_rn(f[e] * inv); s += v[e]; }
  // the low plane is the low byte of v as it is (a signed byte), the high plane byte 1 of v + 128
  const uint32_t lo = prmt(prmt(v[0], v[1], 0x0040u), prmt(v[2], v[3], 0x0040u), 0x5410u);
  const uint32_t hi = prmt(prmt(v[0] + 128, v[1] + 128, 0x0051u), prmt(v[2] + 128, v[3] + 128, 0x0051u), 0x5410u);
  // sums per tile (64 elements: lanes 0..15 / 16..31)
  const int s_half = __reduce_add_sync(0xffffffffu, lane < 16 ? s : 0);
  const int s_all = __reduce_add_sync(0xffffffffu, s);
  xi.sum[0] = s_half; xi.sum[1] = s_all - s_half;
  const int g = lane >> 2, t = lane & 3;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int src_lane = 8 * j + 2 * t;
    const uint32_t l0 = __shfl_sync(0xffffffffu, lo, src_lane), l1 = __shfl_sync(0xffffffffu, lo, src_lane + 1);
    const uint32_t h0 = __shfl_sync(0xffffffffu, hi, src_lane), h1 = __shfl_sync(0xffffffffu, hi, src_lane + 1);
    uint32_t w0 = g == 0 ? l0 : g == 1 ? h0 : 0u, w1 = g == 0 ? l1 : g == 1 ? h1 : 0u;
    if constexpr (FMT == FMT_Q4) {                 // the and-or delivers the codes as (0, 4, 1, 5) and (2, 6, 3, 7)
      const uint32_t p0 = prmt(w0, w1, 0x5140u), p1 = prmt(w0, w1, 0x7362u);
      w0 = p0; w1 = p1;
    }
    xi.b[j][0] = w0; xi.b[j][1] = w1;
  }
}

// Byte quads of one part (8 codes of one row): q[part][0] the codes an and-or delivers first, q[part][1] the others.
// tile: the tile plus the lane's offset into it (16 lane bytes for 4-bit codes, 8 lane for 3-bit ones).
template <int FMT>
__device__ __forceinline__ void tile_quads(const uint8_t* tile, int lane, uint32_t (&q)[4][2]) {
  if constexpr (FMT == FMT_Q4) {
    const uint4 v = *reinterpret_cast<const uint4*>(tile);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int part = 0; part < 4; ++part) {
      q[part][0] = w[part] & 0x0f0f0f0fu;
      q[part][1] = (w[part] >> 4) & 0x0f0f0f0fu;
    }
  } else if constexpr (FMT == FMT_Q3) {
    const uint2 v01 = *reinterpret_cast<const uint2*>(tile);
    const uint32_t v2 = *reinterpret_cast<const uint32_t*>(tile + 256 - 4 * lane);
    q3_quads(v01.x, v01.y, v2, q);
  }
}

// One blob times the byte planes; blob_l: the blob plus the lane's offset into a tile (see tile_quads), blob_g: the blob
// plus 4 (lane / 4), the offset into a scale entry.  tot[0] / tot[1]: the blob's contribution to rows g /
// g + 8 (token 0), held by the lanes with t == 0 (the owners of columns 0 and 1 of the accumulator); the other lanes
// return zeros.  SZ2: one scale entry per tile (groups of 64) instead of one per pair.
template <int FMT, bool SZ2>
__device__ __forceinline__ void blob_product_i8(const uint8_t* blob_l, const uint8_t* blob_g, int lane, const XI8& xi, float (&tot)[2]) {
  constexpr int tb = tile_bytes(FMT);
  const int g = lane >> 2;
  const bool owner = (lane & 3) == 0;
  tot[0] = tot[1] = 0.f;
  int z_a = 0, z_b = 0;
  float s_a = 0.f, s_b = 0.f;
  int zsum_a = 0, zsum_b = 0;          // z * sum v over the tiles of the current scale entry
  int d[4] = {0, 0, 0, 0};             // rows g / g + 8 x columns (low, high) for the owners
#pragma unroll
  for (int c = 0; c < 2; ++c) {
    if (c == 0 || SZ2) {
      const uint8_t* sz = blob_g + 2 * tb + c * kSzEntryBytes;
      const uint32_t s2 = *reinterpret_cast<const uint32_t*>(sz);
      const uint32_t z2 = *reinterpret_cast<const uint16_t*>(sz + 32 - 2 * g);
      z_a = (int)(z2 & 255u); z_b = (int)(z2 >> 8);
      const float2 sf = __half22float2(*reinterpret_cast<const __half2*>(&s2));
      s_a = owner ? sf.x * xi.scale : 0.f;
      s_b = owner ? sf.y * xi.scale : 0.f;
      zsum_a = 0; zsum_b = 0;
    }
    zsum_a += z_a * xi.sum[c];
    zsum_b += z_b * xi.sum[c];
    uint32_t q[4][2];
    tile_quads<FMT>(blob_l + c * tb, lane, q);
#pragma unroll
    for (int blk = 0; blk < 2; ++blk)          // parts 2 blk (row g) and 2 blk + 1 (row g + 8): one MMA
      mma16832_s8(d, q[2 * blk][0], q[2 * blk + 1][0], q[2 * blk][1], q[2 * blk + 1][1], xi.b[2 * c + blk][0], xi.b[2 * c + blk][1]);
    if (c == 1 || SZ2) {
      tot[0] = fmaf((float)(d[1] * 256 + d[0] - zsum_a), s_a, tot[0]);
      tot[1] = fmaf((float)(d[3] * 256 + d[2] - zsum_b), s_b, tot[1]);
      d[0] = d[1] = d[2] = d[3] = 0;
    }
  }
}

// ---- the same integer product for two to eight tokens -------------------------------------------------------------
// Tokens are the columns of the MMA's narrow operand: lane (g, t) holds, for token g, the eight reduction elements
// 32 j + 8 t .. + 7 of MMA j -- exactly the sixteen bytes per MMA that it loads from its token's row -- as a low and a
// high byte plane (two MMAs per weight fragment instead of one).  Every token has its own block scale and sums; the
// accumulator of lane (g, t) belongs to tokens 2t and 2t + 1, whose scale and sums it fetches once per pair.
struct XI8M {
  uint32_t lo[4][2], hi[4][2];   // narrow-operand registers of the four MMAs of a pair, low and high plane (token g)
  float scale[2];                // 2^e of tokens 2t, 2t + 1
  int sum[2][2];                 // [token 2t + i][tile c]: sum of v over the tile
};

template <int FMT>
__device__ __forceinline__ void load_x_i8m(XI8M& xm, const void* x, bool bf16, int m, int d_in, uint32_t pair, int lane) {
  const int g = lane >> 2, t = lane & 3;
  float f[4][8];
  if (g < m) {
    const uint16_t* src = reinterpret_cast<const uint16_t*>(x) + (size_t)g * d_in + pair * 128 + 8 * t;
    uint4 u[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) asm volatile("ld.global.cg.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(u[j].x), "=r"(u[j].y), "=r"(u[j].z), "=r"(u[j].w) : "l"(src + 32 * j) : "memory");
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const uint32_t w[4] = {u[j].x, u[j].y, u[j].z, u[j].w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        if (bf16) { f[j][2 * e] = __uint_as_float(w[e] << 16); f[j][2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u); }
        else { const float2 v = __half22float2(*reinterpret_cast<const __half2*>(&w[e])); f[j][2 * e] = v.x; f[j][2 * e + 1] = v.y; }
      }
    }
  } else {
#pragma unroll
    for (int j = 0; j < 4; ++j)
#pragma unroll
      for (int e = 0; e < 8; ++e) f[j][e] = 0.f;
  }
  float am = 0.f;
#pragma unroll
  for (int j = 0; j < 4; ++j)
#pragma unroll
    for (int e = 0; e < 8; ++e) am = fmaxf(am, fabsf(f[j][e]));
  am = fmaxf(am, __shfl_xor_sync(0xffffffffu, am, 1));
  am = fmaxf(am, __shfl_xor_sync(0xffffffffu, am, 2));               // the token's 128 elements sit in its four lanes
  const uint32_t eb = __float_as_uint(am * 1.00396f) >> 23;
  const bool live = eb >= 15u && eb < 255u;
  const float inv = live ? __uint_as_float((268u - eb) << 23) : 0.f;
  const float my_scale = live ? __uint_as_float((eb - 14u) << 23) : 0.f;
  int my_sum[2] = {0, 0};
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    int v[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) { v[e] = __float2int_rn(f[j][e] * inv); my_sum[j >> 1] += v[e]; }
    uint32_t l0 = prmt(prmt(v[0], v[1], 0x0040u), prmt(v[2], v[3], 0x0040u), 0x5410u);
    uint32_t l1 = prmt(prmt(v[4], v[5], 0x0040u), prmt(v[6], v[7], 0x0040u), 0x5410u);
    uint32_t h0 = prmt(prmt(v[0] + 128, v[1] + 128, 0x0051u), prmt(v[2] + 128, v[3] + 128, 0x0051u), 0x5410u);
    uint32_t h1 = prmt(prmt(v[4] + 128, v[5] + 128, 0x0051u), prmt(v[6] + 128, v[7] + 128, 0x0051u), 0x5410u);
    if constexpr (FMT == FMT_Q4) {                 // the and-or delivers the codes as (0, 4, 1, 5) and (2, 6, 3, 7)
      const uint32_t a = prmt(l0, l1, 0x5140u), b = prmt(l0, l1, 0x7362u), c = prmt(h0, h1, 0x5140u), d = prmt(h0, h1, 0x7362u);
      l0 = a; l1 = b; h0 = c; h1 = d;
    }
    xm.lo[j][0] = l0; xm.lo[j][1] = l1; xm.hi[j][0] = h0; xm.hi[j][1] = h1;
  }
#pragma unroll
  for (int c = 0; c < 2; ++c) {
    my_sum[c] += __shfl_xor_sync(0xffffffffu, my_sum[c], 1);
    my_sum[c] += __shfl_xor_sync(0xffffffffu, my_sum[c], 2);
  }
#pragma unroll
  for (int i = 0; i < 2; ++i) {                    // what belongs to the accumulator's columns: tokens 2t and 2t + 1
    const int from = (2 * t + i) * 4;
    xm.scale[i] = __shfl_sync(0xffffffffu, my_scale, from);
    xm.sum[i][0] = __shfl_sync(0xffffffffu, my_sum[0], from);
    xm.sum[i][1] = __shfl_sync(0xffffffffu, my_sum[1], from);
  }
}

// tot[i] as the accumulator of mma.m16n8k16: (row g, token 2t), (row g, token 2t + 1), (row g + 8, token 2t), (row g + 8, 2t + 1).
template <int FMT>
__device__ __forceinline__ void blob_product_i8m(const uint8_t* blob, int lane, uint32_t sz2, const XI8M& xm, float (&tot)[4]) {
  constexpr int tb = tile_bytes(FMT);
  const int g = lane >> 2;
  const uint8_t* blob_l = blob + (FMT == FMT_Q4 ? 16 : 8) * lane;
  const uint8_t* blob_g = blob + 4 * g;
  tot[0] = tot[1] = tot[2] = tot[3] = 0.f;
  int z_a = 0, z_b = 0;
  float s_a = 0.f, s_b = 0.f;
  int zs[2] = {0, 0};                    // sum of v over the tiles of the current scale entry, tokens 2t and 2t + 1
  int dl[4] = {0, 0, 0, 0}, dh[4] = {0, 0, 0, 0};
#pragma unroll
  for (int c = 0; c < 2; ++c) {
    if (c == 0 || sz2) {
      const uint8_t* sz = blob_g + 2 * tb + c * kSzEntryBytes;
      const uint32_t s2 = *reinterpret_cast<const uint32_t*>(sz);
      const uint32_t z2 = *reinterpret_cast<const uint16_t*>(sz + 32 - 2 * g);
      z_a = (int)(z2 & 255u); z_b = (int)(z2 >> 8);
      const float2 sf = __half22float2(*reinterpret_cast<const __half2*>(&s2));
      s_a = sf.x; s_b = sf.y;
      zs[0] = zs[1] = 0;
    }
    zs[0] += xm.sum[0][c];
    zs[1] += xm.sum[1][c];
    uint32_t q[4][2];
    tile_quads<FMT>(blob_l + c * tb, lane, q);
#pragma unroll
    for (int blk = 0; blk < 2; ++blk) {
      mma16832_s8(dl, q[2 * blk][0], q[2 * blk + 1][0], q[2 * blk][1], q[2 * blk + 1][1], xm.lo[2 * c + blk][0], xm.lo[2 * c + blk][1]);
      mma16832_s8(dh, q[2 * blk][0], q[2 * blk + 1][0], q[2 * blk][1], q[2 * blk + 1][1], xm.hi[2 * c + blk][0], xm.hi[2 * c + blk][1]);
    }
    if (c == 1 || sz2) {
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int tok = i & 1, z = i < 2 ? z_a : z_b;
        const float s = (i < 2 ? s_a : s_b) * xm.scale[tok];
        tot[i] = fmaf((float)(dh[i] * 256 + dl[i] - z * zs[tok]), s, tot[i]);
        dl[i] = 0; dh[i] = 0;
      }
    }
  }
}

__device__ __forceinline__ void store_y(void* y, int dtype, int64_t i, float v) {
  if (dtype == EORA_Y_F16) reinterpret_cast<__half*>(y)[i] = __float2half_rn(v);
  else if (dtype == EORA_Y_BF16) reinterpret_cast<__nv_bfloat16*>(y)[i] = __float2bfloat16_rn(v);
  else reinterpret_cast<float*>(y)[i] = v;
}

}  // namespace dec
}  // namespace eora
