// Simple kernels: any format, any M.  They read the same re-tiled weights as the fast kernels
// through the element accessors, one thread per output element.  They serve shapes and M the
// fast families do not cover, the read-back used by the bit-exact unpack / dequant checks, and
// EORA_POLICY_GENERIC.
#include "eora_common.cuh"

namespace eora {
namespace {

__device__ inline float load_x(const void* x, int dtype, int64_t i) {
  if (dtype == EORA_X_F16) return __half2float(reinterpret_cast<const __half*>(x)[i]);
  return __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(x)[i]);
}
__device__ inline void store_y(void* y, int dtype, int64_t i, float v) {
  if (dtype == EORA_Y_F16) reinterpret_cast<__half*>(y)[i] = __float2half_rn(v);
  else if (dtype == EORA_Y_BF16) reinterpret_cast<__nv_bfloat16*>(y)[i] = __float2bfloat16_rn(v);
  else reinterpret_cast<float*>(y)[i] = v;
}

// step a4: t[m][j] = sum_k X[m][k] * A[k][j]
__global__ void k_generic_t(WMat a, const void* x, int x_dtype, int m, int d_in, float* t, int r_pad) {
  int64_t total = (int64_t)m * r_pad;
  for (int64_t idx = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * blockDim.x) {
    int j = (int)(idx % r_pad), mm = (int)(idx / r_pad);
    float acc = 0.f;
    if (j < a.n_rows)
      for (int k = 0; k < d_in; ++k) acc = fmaf(load_x(x, x_dtype, (int64_t)mm * d_in + k), wmat_elem(a, k, j), acc);
    t[idx] = acc;
  }
}

// steps a1-a3, a5, a6: y[m][n] = sum_k X[m][k] * w[k][n] + sum_j t[m][j] * B[j][n]
__global__ void k_generic_y(WMat w, WMat b, bool has_ab, const void* x, int x_dtype, int m, int d_in, int d_out,
                            const float* t, int r_pad, void* y, int y_dtype) {
  int64_t total = (int64_t)m * d_out;
  for (int64_t idx = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * blockDim.x) {
    int n = (int)(idx % d_out), mm = (int)(idx / d_out);
    float acc = 0.f;
    for (int k = 0; k < d_in; ++k) acc = fmaf(load_x(x, x_dtype, (int64_t)mm * d_in + k), wmat_elem(w, k, n), acc);
    if (has_ab) {
      float lr = 0.f;
      for (int j = 0; j < r_pad; ++j) lr = fmaf(t[(int64_t)mm * r_pad + j], wmat_elem(b, j, n), lr);
      acc += lr;
    }
    store_y(y, y_dtype, idx, acc);
  }
}

__global__ void k_dump_codes(WMat w, int rows, int cols, int32_t* out) {   // out [rows = k][cols = n]
  int64_t total = (int64_t)rows * cols;
  for (int64_t idx = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * blockDim.x)
    out[idx] = wmat_code(w, (int)(idx / cols), (int)(idx % cols));
}
__global__ void k_dump_elems(WMat w, int rows, int cols, float* out) {
  int64_t total = (int64_t)rows * cols;
  for (int64_t idx = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * blockDim.x)
    out[idx] = wmat_elem(w, (int)(idx / cols), (int)(idx % cols));
}

inline int grid_for(int64_t total, int block) {
  int64_t g = (total + block - 1) / block;
  if (g > 148 * 32) g = 148 * 32;
  if (g < 1) g = 1;
  return (int)g;
}

}  // namespace

int generic_launch_count(const Handle* h) { return h->cfg.rank > 0 ? 2 : 1; }

cudaError_t launch_generic_forward(const Handle* h, const void* x, int m, void* y, cudaStream_t st) {
  const eora_linear_config& c = h->cfg;
  bool has_ab = c.rank > 0;
  if (has_ab)
    k_generic_t<<<grid_for((int64_t)m * h->r_pad, 128), 128, 0, st>>>(h->a, x, c.x_dtype, m, c.d_in, h->t_gen, h->r_pad);
  k_generic_y<<<grid_for((int64_t)m * c.d_out, 128), 128, 0, st>>>(h->w, h->b, has_ab, x, c.x_dtype, m, c.d_in, c.d_out,
                                                                  h->t_gen, h->r_pad, y, c.y_dtype);
  return cudaGetLastError();
}

cudaError_t launch_dump(const Handle* h, int what, void* out, cudaStream_t st) {
  const eora_linear_config& c = h->cfg;
  if (what == 0)
    k_dump_codes<<<grid_for((int64_t)c.d_in * c.d_out, 256), 256, 0, st>>>(h->w, c.d_in, c.d_out, (int32_t*)out);
  else if (what == 1)
    k_dump_elems<<<grid_for((int64_t)c.d_in * c.d_out, 256), 256, 0, st>>>(h->w, c.d_in, c.d_out, (float*)out);
  else if (what == 2)   // A [d_in][rank]: element (k, j) of the WMat whose rows are j
    k_dump_elems<<<grid_for((int64_t)c.d_in * c.rank, 256), 256, 0, st>>>(h->a, c.d_in, c.rank, (float*)out);
  else                  // B [rank][d_out]: element (j, n) of the WMat whose reduction axis is j
    k_dump_elems<<<grid_for((int64_t)c.rank * c.d_out, 256), 256, 0, st>>>(h->b, c.rank, c.d_out, (float*)out);
  return cudaGetLastError();
}

}  // namespace eora
