// eora_linear_forward_noalloc: the compensated layer for callers that must not allocate.
//
// Every other path of this library needs a handle, and building a handle calls cudaMalloc (for
// the re-tiled weights and for scratch).  Some callers cannot do that: code that runs after a
// framework has claimed all device memory for its own pool, code inside a latency-critical loop
// where an allocation (and the implicit synchronisation that may come with it) is forbidden, or
// a plug-in that is only handed buffers and a stream.  This entry point takes the weights in the
// interchange layout straight from the caller's buffers and keeps its only scratch -- the thin
// product t = X.A -- in a fixed array that lives in the library image on every GPU that loads it.
//
// It is a variant of the simple two-kernel path (t first, then Y), slow but self-contained.
#include "eora_common.cuh"

namespace {

// Scratch for t [m][rank] as fp32.  256 KB per GPU, held from library load until process exit.
constexpr int kNoAllocScratchFloats = EORA_NOALLOC_MAX_T_ELEMS;
static __device__ __align__(256) float g_noalloc_t[kNoAllocScratchFloats];

constexpr int kMaxDevices = 64;
float* g_scratch_addr[kMaxDevices];     // device address of g_noalloc_t, per device (0 = not looked up yet)

__device__ inline uint32_t na_code(const uint32_t* words, int bits, int k, int n, int ld) {
  int p = bits * k, i = p >> 5, off = p & 31;
  uint32_t v = words[(int64_t)i * ld + n] >> off;
  if (off + bits > 32) v |= words[(int64_t)(i + 1) * ld + n] << (32 - off);
  return v & ((1u << bits) - 1u);
}
__device__ inline uint32_t na_zero(const uint32_t* zeros, int bits, int g, int n, int ldz) {
  int p = bits * n, i = p >> 5, off = p & 31;
  const uint32_t* row = zeros + (int64_t)g * ldz;
  uint32_t v = row[i] >> off;
  if (off + bits > 32) v |= row[i + 1] << (32 - off);
  return v & ((1u << bits) - 1u);
}
__device__ inline float na_x(const void* x, int dtype, int64_t i) {
  if (dtype == EORA_X_F16) return __half2float(reinterpret_cast<const __half*>(x)[i]);
  return __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(x)[i]);
}
__device__ inline void na_store(void* y, int dtype, int64_t i, float v) {
  if (dtype == EORA_Y_F16) reinterpret_cast<__half*>(y)[i] = __float2half_rn(v);
  else if (dtype == EORA_Y_BF16) reinterpret_cast<__nv_bfloat16*>(y)[i] = __float2bfloat16_rn(v);
  else reinterpret_cast<float*>(y)[i] = v;
}

// t[m][j] = sum_k X[m][k] * A[k][j]; every used element of t is overwritten, nothing is accumulated,
// so the previous call's contents of the shared array do not matter.
__global__ void k_noalloc_t(const void* x, int x_dtype, const __half* a, int m, int d_in, int rank, float* t) {
  int64_t total = (int64_t)m * rank;
  for (int64_t idx = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * blockDim.x) {
    int j = (int)(idx % rank), mm = (int)(idx / rank);
    float acc = 0.f;
    for (int k = 0; k < d_in; ++k) acc = fmaf(na_x(x, x_dtype, (int64_t)mm * d_in + k), __half2float(a[(int64_t)k * rank + j]), acc);
    t[idx] = acc;
  }
}

// y[m][n] = sum_k X[m][k] * (q - z) * s + sum_j t[m][j] * B[j][n], weights read in the interchange layout
__global__ void k_noalloc_y(const void* x, int x_dtype, const uint32_t* codes, const __half* scales, const uint32_t* zeros,
                            int bits, int group, const __half* b, const float* t, int m, int d_in, int d_out, int rank,
                            void* y, int y_dtype) {
  const int ldz = bits * d_out / 32;
  int64_t total = (int64_t)m * d_out;
  for (int64_t idx = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * blockDim.x) {
    int n = (int)(idx % d_out), mm = (int)(idx / d_out);
    float acc = 0.f;
    for (int g = 0; g < d_in / group; ++g) {
      const float s = __half2float(scales[(int64_t)g * d_out + n]);
      const int z = (int)na_zero(zeros, bits, g, n, ldz);
      float part = 0.f;
      for (int k = g * group; k < (g + 1) * group; ++k)
        part = fmaf(na_x(x, x_dtype, (int64_t)mm * d_in + k), (float)((int)na_code(codes, bits, k, n, d_out) - z), part);
      acc = fmaf(part, s, acc);
    }
    float lr = 0.f;
    for (int j = 0; j < rank; ++j) lr = fmaf(t[(int64_t)mm * rank + j], __half2float(b[(int64_t)j * d_out + n]), lr);
    na_store(y, y_dtype, idx, acc + lr);
  }
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

extern "C" int eora_linear_forward_noalloc(const eora_linear_config* cfg, const eora_linear_weights* w, const void* x,
                                           int32_t m, void* y, void* stream) {
  if (!cfg || !w) return EORA_ERR_NULL_ARG;
  const eora_linear_config& c = *cfg;
  if (c.d_in <= 0 || c.d_out <= 0 || c.rank < 0 || c.d_in % 128 || c.d_out % 32 || c.rank % 8) return EORA_ERR_BAD_SHAPE;
  if (c.w_format != EORA_W_QUANT || (c.w_bits != 3 && c.w_bits != 4)) return EORA_ERR_UNSUPPORTED;
  if (c.w_group <= 0 || c.w_group % 64 || c.d_in % c.w_group) return EORA_ERR_BAD_SHAPE;
  if (c.rank > 0 && c.ab_format != EORA_AB_F16) return EORA_ERR_UNSUPPORTED;
  if (c.x_dtype != EORA_X_F16 && c.x_dtype != EORA_X_BF16) return EORA_ERR_UNSUPPORTED;
  if (c.y_dtype != EORA_Y_F16 && c.y_dtype != EORA_Y_BF16 && c.y_dtype != EORA_Y_F32) return EORA_ERR_UNSUPPORTED;
  if (m == 0) return EORA_OK;
  if (m < 0) return EORA_ERR_BAD_SHAPE;
  // the fixed scratch bounds the size of t: m * rank fp32 values
  if ((int64_t)m * c.rank > kNoAllocScratchFloats) return EORA_ERR_M_TOO_LARGE;
  if (!x || !y || !w->w_codes || !w->w_scales || !w->w_zeros) return EORA_ERR_NULL_ARG;
  if (c.rank > 0 && (!w->a || !w->b)) return EORA_ERR_NULL_ARG;
  if (!aligned16(x) || !aligned16(y) || !aligned16(w->w_codes) || !aligned16(w->w_scales) || !aligned16(w->w_zeros) ||
      !aligned16(w->a) || !aligned16(w->b))
    return EORA_ERR_MISALIGNED;

  // Set-up, once per device, with that device current: the array's name is only a host-side stand-in,
  // the kernels need its device address.
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return EORA_ERR_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return EORA_ERR_UNSUPPORTED;
  if (!g_scratch_addr[dev]) {
    float* p = nullptr;
    if (cudaGetSymbolAddress((void**)&p, g_noalloc_t) != cudaSuccess || !p) return EORA_ERR_CUDA;
    g_scratch_addr[dev] = p;
  }
  float* t = g_scratch_addr[dev];

  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  auto grid_for = [](int64_t total, int block) {
    int64_t g = (total + block - 1) / block;
    return (int)(g > 148 * 32 ? 148 * 32 : (g < 1 ? 1 : g));
  };
  if (c.rank > 0)
    k_noalloc_t<<<grid_for((int64_t)m * c.rank, 128), 128, 0, s>>>(x, c.x_dtype, (const __half*)w->a, m, c.d_in, c.rank, t);
  k_noalloc_y<<<grid_for((int64_t)m * c.d_out, 128), 128, 0, s>>>(x, c.x_dtype, (const uint32_t*)w->w_codes,
                                                                 (const __half*)w->w_scales, (const uint32_t*)w->w_zeros,
                                                                 c.w_bits, c.w_group, (const __half*)w->b, t, m, c.d_in,
                                                                 c.d_out, c.rank, y, c.y_dtype);
  return cudaGetLastError() == cudaSuccess ? EORA_OK : EORA_ERR_CUDA;
}
