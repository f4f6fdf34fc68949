// Offline EoRA solve (Algorithm 1, steps 1-6) on the GPU; the interface and the mathematics are in eora_solve.h.
//
//   1.  dW = W - W^                                                    (k_sub)
//   2-4 the paper projects dW into the eigenspace of X~ X~^T, dW' = dW Q sqrt(L).  Only dW' dW'^T is needed here:
//       G = X~ X~^T  (k x k),  T = dW G,  Mm = T dW^T = dW' dW'^T  (d x d)   (three fp32 contractions)
//   5.  top-r eigenpairs (U', S'^2) of Mm by subspace iteration on m = r + oversample vectors:
//         Y = Mm Q;  Q = orth(Y)  by Cholesky-QR (Gram matrix and factor in fp64);  repeated `iters` times, then a
//         Rayleigh-Ritz step:  H = Q^T Mm Q  (m x m, fp64),  H = V diag(lam) V^T  by one-sided Jacobi in one CTA,
//         U' = Q V[:, top r],  S' = sqrt(lam)
//   6.  B' = U' S',  A = S'^{-1} U'^T dW
//
// Every kernel here is plain fp32 / fp64 CUDA-core arithmetic: the large contractions are tiled SGEMMs
// (128 x 128 x 16 tiles through shared memory, 8 x 8 outputs per thread; for the skinny products of the iteration
// 32 x 160 tiles at the default width of 160 vectors, else 64 x 128); fp32 because the quality of the eigenvectors near the cut depends on the small differences
// between neighbouring eigenvalues of Mm.  The (r + oversample)^2 problems run in fp64 in one CTA each.
#include <cuda_runtime.h>
#include <stdint.h>
#include "../../include/eora_linear.h"
#include "../../include/eora_solve.h"

namespace {

// ------------------------------------------------------------------------------------------------ SGEMM
constexpr int BM = 128, BN = 128, BKS = 16, PAD = 4;

// C[M][N] (ldc) = sum_p opA[m][p] opB[p][n];  opA[m][p] = ta ? A[p * lda + m] : A[m * lda + p];
// opB[p][n] = tb ? B[n * ldb + p] : B[p * ldb + n].  Out-of-range elements read as zero.
__global__ void __launch_bounds__(256) k_sgemm(int M, int N, int P, const float* __restrict__ A, int lda, int ta,
                                               const float* __restrict__ B, int ldb, int tb, float* __restrict__ C, int ldc) {
  __shared__ float As[BKS][BM + PAD];
  __shared__ float Bs[BKS][BN + PAD];
  const int t = threadIdx.x, tx = t & 15, ty = t >> 4;
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  float acc[8][8];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;
  for (int p0 = 0; p0 < P; p0 += BKS) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int e = t + 256 * i;
      {
        const int m = ta ? (e & (BM - 1)) : (e >> 4), p = ta ? (e >> 7) : (e & 15);
        const int gm = m0 + m, gp = p0 + p;
        float v = 0.f;
        if (gm < M && gp < P) v = ta ? A[(int64_t)gp * lda + gm] : A[(int64_t)gm * lda + gp];
        As[p][m] = v;
      }
      {
        const int n = tb ? (e >> 4) : (e & (BN - 1)), p = tb ? (e & 15) : (e >> 7);
        const int gn = n0 + n, gp = p0 + p;
        float v = 0.f;
        if (gn < N && gp < P) v = tb ? B[(int64_t)gn * ldb + gp] : B[(int64_t)gp * ldb + gn];
        Bs[p][n] = v;
      }
    }
    __syncthreads();
#pragma unroll
    for (int p = 0; p < BKS; ++p) {
      float a[8], b[8];
      const float4 a0 = *reinterpret_cast<const float4*>(&As[p][ty * 4]), a1 = *reinterpret_cast<const float4*>(&As[p][64 + ty * 4]);
      const float4 b0 = *reinterpret_cast<const float4*>(&Bs[p][tx * 4]), b1 = *reinterpret_cast<const float4*>(&Bs[p][64 + tx * 4]);
      a[0] = a0.x; a[1] = a0.y; a[2] = a0.z; a[3] = a0.w; a[4] = a1.x; a[5] = a1.y; a[6] = a1.z; a[7] = a1.w;
      b[0] = b0.x; b[1] = b0.y; b[2] = b0.z; b[3] = b0.w; b[4] = b1.x; b[5] = b1.y; b[6] = b1.z; b[7] = b1.w;
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int gm = m0 + (i < 4 ? ty * 4 + i : 64 + ty * 4 + i - 4);
    if (gm >= M) continue;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int gn = n0 + (j < 4 ? tx * 4 + j : 64 + tx * 4 + j - 4);
      if (gn < N) C[(int64_t)gm * ldc + gn] = acc[i][j];
    }
  }
}

// The same product for whole tiles (M, N multiples of 128, P of 16, rows 16-byte aligned): 16-byte global loads, the
// next k-slice fetched into registers while the current one is multiplied.
// TM: output rows per thread (8: tiles of 128 rows; 4: tiles of 64 rows, for products with few tiles).
template <bool TA, bool TB, int TM>
__global__ void __launch_bounds__(256) k_sgemm_full(int P, const float* __restrict__ A, int lda, const float* __restrict__ B, int ldb,
                                                    float* __restrict__ C, int ldc) {
  constexpr int BMT = 16 * TM, NA = TM / 4;          // tile rows; 16-byte pieces of the A tile per thread
  __shared__ __align__(16) float As[2][BKS][BMT + PAD];
  __shared__ __align__(16) float Bs[2][BKS][BN + PAD];
  const int t = threadIdx.x, tx = t & 15, ty = t >> 4;
  const int m0 = blockIdx.y * BMT, n0 = blockIdx.x * BN;
  // this thread's two 16-byte pieces of each operand tile
  // A not transposed: tile rows m (128) x 16 p: piece = (row, p4), 4 pieces per row;  transposed: A[p][m]: (p, m4), 32 per p
  int a_r[NA], a_c[NA], b_r[2], b_c[2];
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    const int e = t + 256 * i;
    if (i < NA) {
      if (TA) { a_r[i] = e / (BMT / 4); a_c[i] = (e % (BMT / 4)) * 4; } else { a_r[i] = e >> 2; a_c[i] = (e & 3) * 4; }
    }
    if (TB) { b_r[i] = e >> 2; b_c[i] = (e & 3) * 4; } else { b_r[i] = e >> 5; b_c[i] = (e & 31) * 4; }
  }
  auto load_a = [&](int p0, int i) -> float4 {
    return TA ? *reinterpret_cast<const float4*>(A + (int64_t)(p0 + a_r[i]) * lda + m0 + a_c[i])
              : *reinterpret_cast<const float4*>(A + (int64_t)(m0 + a_r[i]) * lda + p0 + a_c[i]);
  };
  auto load_b = [&](int p0, int i) -> float4 {
    return TB ? *reinterpret_cast<const float4*>(B + (int64_t)(n0 + b_r[i]) * ldb + p0 + b_c[i])
              : *reinterpret_cast<const float4*>(B + (int64_t)(p0 + b_r[i]) * ldb + n0 + b_c[i]);
  };
  auto store_a = [&](int buf, int i, const float4& v) {
    if (TA) *reinterpret_cast<float4*>(&As[buf][a_r[i]][a_c[i]]) = v;
    else { As[buf][a_c[i]][a_r[i]] = v.x; As[buf][a_c[i] + 1][a_r[i]] = v.y; As[buf][a_c[i] + 2][a_r[i]] = v.z; As[buf][a_c[i] + 3][a_r[i]] = v.w; }
  };
  auto store_b = [&](int buf, int i, const float4& v) {
    if (TB) { Bs[buf][b_c[i]][b_r[i]] = v.x; Bs[buf][b_c[i] + 1][b_r[i]] = v.y; Bs[buf][b_c[i] + 2][b_r[i]] = v.z; Bs[buf][b_c[i] + 3][b_r[i]] = v.w; }
    else *reinterpret_cast<float4*>(&Bs[buf][b_r[i]][b_c[i]]) = v;
  };
  float acc[TM][8];
#pragma unroll
  for (int i = 0; i < TM; ++i)
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;
  float4 ra[NA], rb[2];
#pragma unroll
  for (int i = 0; i < 2; ++i) { if (i < NA) ra[i] = load_a(0, i); rb[i] = load_b(0, i); }
#pragma unroll
  for (int i = 0; i < 2; ++i) { if (i < NA) store_a(0, i, ra[i]); store_b(0, i, rb[i]); }
  __syncthreads();
  int buf = 0;
  for (int p0 = 0; p0 < P; p0 += BKS) {
    const bool more = p0 + BKS < P;
    if (more) {
#pragma unroll
      for (int i = 0; i < 2; ++i) { if (i < NA) ra[i] = load_a(p0 + BKS, i); rb[i] = load_b(p0 + BKS, i); }
    }
#pragma unroll
    for (int p = 0; p < BKS; ++p) {
      float a[8], b[8];
      const float4 a0 = *reinterpret_cast<const float4*>(&As[buf][p][ty * 4]);
      const float4 a1 = TM == 8 ? *reinterpret_cast<const float4*>(&As[buf][p][(BMT / 2) + ty * 4]) : a0;
      const float4 b0 = *reinterpret_cast<const float4*>(&Bs[buf][p][tx * 4]), b1 = *reinterpret_cast<const float4*>(&Bs[buf][p][64 + tx * 4]);
      a[0] = a0.x; a[1] = a0.y; a[2] = a0.z; a[3] = a0.w; a[4] = a1.x; a[5] = a1.y; a[6] = a1.z; a[7] = a1.w;
      b[0] = b0.x; b[1] = b0.y; b[2] = b0.z; b[3] = b0.w; b[4] = b1.x; b[5] = b1.y; b[6] = b1.z; b[7] = b1.w;
#pragma unroll
      for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    if (more) {
#pragma unroll
      for (int i = 0; i < 2; ++i) { if (i < NA) store_a(buf ^ 1, i, ra[i]); store_b(buf ^ 1, i, rb[i]); }
    }
    __syncthreads();
    buf ^= 1;
  }
#pragma unroll
  for (int i = 0; i < TM; ++i) {
    const int gm = m0 + (i < 4 ? ty * 4 + i : (BMT / 2) + ty * 4 + i - 4);
    float* row = C + (int64_t)gm * ldc + n0;
    *reinterpret_cast<float4*>(row + tx * 4) = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
    *reinterpret_cast<float4*>(row + 64 + tx * 4) = make_float4(acc[i][4], acc[i][5], acc[i][6], acc[i][7]);
  }
}

// C[M][160] = A[M][P] B[P][160] (nothing transposed; M a multiple of 32, P of 16, rows 16-byte aligned): the products of the
// subspace iteration with its default width of 160 vectors.  Tiles of 32 rows x all 160 columns, so that a product
// with 4096 rows is 128 CTAs and no flop goes into padding columns; 2 x 10 outputs per thread.
constexpr int NQ = 160, BMQ = 32;
__global__ void __launch_bounds__(256) k_sgemm_n160(int P, const float* __restrict__ A, int lda, const float* __restrict__ B, int ldb,
                                                    float* __restrict__ C, int ldc) {
  __shared__ __align__(16) float As[2][BKS][BMQ + PAD];
  __shared__ __align__(16) float Bs[2][BKS][NQ + PAD];
  const int t = threadIdx.x, tx = t & 15, ty = t >> 4;
  const int m0 = blockIdx.x * BMQ;
  // 16-byte pieces: A tile 32 rows x 16 p = 128 pieces (threads 0..127), B tile 16 p x 160 = 640 pieces (2.5 per thread)
  const int a_r = (t & 127) >> 2, a_c = (t & 3) * 4;
  int b_r[3], b_c[3];
#pragma unroll
  for (int i = 0; i < 3; ++i) { const int e = t + 256 * i; b_r[i] = e / (NQ / 4); b_c[i] = (e % (NQ / 4)) * 4; }
  const bool has_a = t < 128, has_b2 = t + 512 < BKS * NQ / 4;
  auto load_a = [&](int p0) -> float4 { return *reinterpret_cast<const float4*>(A + (int64_t)(m0 + a_r) * lda + p0 + a_c); };
  auto load_b = [&](int p0, int i) -> float4 { return *reinterpret_cast<const float4*>(B + (int64_t)(p0 + b_r[i]) * ldb + b_c[i]); };
  auto store_a = [&](int buf, const float4& v) {
    As[buf][a_c][a_r] = v.x; As[buf][a_c + 1][a_r] = v.y; As[buf][a_c + 2][a_r] = v.z; As[buf][a_c + 3][a_r] = v.w;
  };
  auto store_b = [&](int buf, int i, const float4& v) { *reinterpret_cast<float4*>(&Bs[buf][b_r[i]][b_c[i]]) = v; };
  float acc[2][10];
#pragma unroll
  for (int i = 0; i < 2; ++i)
#pragma unroll
    for (int j = 0; j < 10; ++j) acc[i][j] = 0.f;
  float4 ra = make_float4(0.f, 0.f, 0.f, 0.f), rb[3];
  if (has_a) ra = load_a(0);
#pragma unroll
  for (int i = 0; i < 3; ++i) if (i < 2 || has_b2) rb[i] = load_b(0, i);
  if (has_a) store_a(0, ra);
#pragma unroll
  for (int i = 0; i < 3; ++i) if (i < 2 || has_b2) store_b(0, i, rb[i]);
  __syncthreads();
  int buf = 0;
  for (int p0 = 0; p0 < P; p0 += BKS) {
    const bool more = p0 + BKS < P;
    if (more) {
      if (has_a) ra = load_a(p0 + BKS);
#pragma unroll
      for (int i = 0; i < 3; ++i) if (i < 2 || has_b2) rb[i] = load_b(p0 + BKS, i);
    }
#pragma unroll
    for (int p = 0; p < BKS; ++p) {
      const float2 a = *reinterpret_cast<const float2*>(&As[buf][p][ty * 2]);
      const float4 b0 = *reinterpret_cast<const float4*>(&Bs[buf][p][tx * 4]), b1 = *reinterpret_cast<const float4*>(&Bs[buf][p][64 + tx * 4]);
      const float2 b2 = *reinterpret_cast<const float2*>(&Bs[buf][p][128 + tx * 2]);
      const float b[10] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w, b2.x, b2.y};
#pragma unroll
      for (int j = 0; j < 10; ++j) { acc[0][j] = fmaf(a.x, b[j], acc[0][j]); acc[1][j] = fmaf(a.y, b[j], acc[1][j]); }
    }
    if (more) {
      if (has_a) store_a(buf ^ 1, ra);
#pragma unroll
      for (int i = 0; i < 3; ++i) if (i < 2 || has_b2) store_b(buf ^ 1, i, rb[i]);
    }
    __syncthreads();
    buf ^= 1;
  }
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    float* row = C + (int64_t)(m0 + ty * 2 + i) * ldc;
    *reinterpret_cast<float4*>(row + tx * 4) = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
    *reinterpret_cast<float4*>(row + 64 + tx * 4) = make_float4(acc[i][4], acc[i][5], acc[i][6], acc[i][7]);
    *reinterpret_cast<float2*>(row + 128 + tx * 2) = make_float2(acc[i][8], acc[i][9]);
  }
}

cudaError_t sgemm(cudaStream_t st, int M, int N, int P, const float* A, int lda, bool ta, const float* B, int ldb, bool tb, float* C, int ldc) {
  dim3 grid((N + BN - 1) / BN, (M + BM - 1) / BM);
  const bool full = M % BM == 0 && N % BN == 0 && P % BKS == 0 && lda % 4 == 0 && ldb % 4 == 0 && ldc % 4 == 0 &&
                    ((reinterpret_cast<uintptr_t>(A) | reinterpret_cast<uintptr_t>(B) | reinterpret_cast<uintptr_t>(C)) & 15) == 0;
  const bool al = lda % 4 == 0 && ldb % 4 == 0 && ldc % 4 == 0 &&
                  ((reinterpret_cast<uintptr_t>(A) | reinterpret_cast<uintptr_t>(B) | reinterpret_cast<uintptr_t>(C)) & 15) == 0;
  if (N == NQ && !ta && !tb && M % BMQ == 0 && P % BKS == 0 && al) {
    k_sgemm_n160<<<M / BMQ, 256, 0, st>>>(P, A, lda, B, ldb, C, ldc);
    return cudaGetLastError();
  }
  if (full) {
    // products with few tiles (the 4096 x 256 iterates: 64 tiles of 128 rows on 148 SMs) take tiles of 64 rows
    const bool half = (int)(grid.x * grid.y) < 120;
    if (half) {
      dim3 g2(grid.x, M / 64);
      if (ta && tb) k_sgemm_full<true, true, 4><<<g2, 256, 0, st>>>(P, A, lda, B, ldb, C, ldc);
      else if (ta) k_sgemm_full<true, false, 4><<<g2, 256, 0, st>>>(P, A, lda, B, ldb, C, ldc);
      else if (tb) k_sgemm_full<false, true, 4><<<g2, 256, 0, st>>>(P, A, lda, B, ldb, C, ldc);
      else k_sgemm_full<false, false, 4><<<g2, 256, 0, st>>>(P, A, lda, B, ldb, C, ldc);
    } else if (ta && tb) k_sgemm_full<true, true, 8><<<grid, 256, 0, st>>>(P, A, lda, B, ldb, C, ldc);
    else if (ta) k_sgemm_full<true, false, 8><<<grid, 256, 0, st>>>(P, A, lda, B, ldb, C, ldc);
    else if (tb) k_sgemm_full<false, true, 8><<<grid, 256, 0, st>>>(P, A, lda, B, ldb, C, ldc);
    else k_sgemm_full<false, false, 8><<<grid, 256, 0, st>>>(P, A, lda, B, ldb, C, ldc);
  } else {
    k_sgemm<<<grid, 256, 0, st>>>(M, N, P, A, lda, ta ? 1 : 0, B, ldb, tb ? 1 : 0, C, ldc);
  }
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------ small pieces
__global__ void k_sub(const float* __restrict__ a, const float* __restrict__ b, float* __restrict__ c, int64_t n) {
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) c[i] = a[i] - b[i];
}

// A fixed start for the iteration: values in (-1, 1) from a counter hash (any full-rank start converges).  The iterate
// is stored with a leading dimension ld >= m (a multiple of the SGEMM tile); the columns past m are zero and stay zero.
__global__ void k_init(float* y, int rows, int m, int ld) {
  const int64_t n = (int64_t)rows * ld;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
    uint64_t z = (uint64_t)i * 0x9E3779B97F4A7C15ull + 0xD1B54A32D192ED03ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    z ^= z >> 31;
    y[i] = (int)(i % ld) < m ? (float)((double)(z >> 11) * (2.0 / 9007199254740992.0) - 1.0) : 0.f;
  }
}

// S[i][j] = sum_row A[row][i] B[row][j]  for two [rows][m] fp32 matrices, products and sums in fp64.
// One CTA per 16 x 16 block of S and per part of the rows (blockIdx.z; `chunk` rows each, a multiple of the slice), one
// thread per element; slices of 64 rows go through shared memory.  Part z writes its sums to parts[z][m][m];
// k_sum_parts adds the parts in a fixed order, so the result does not depend on the order the CTAs ran in.
constexpr int kGramParts = 4;
__global__ void __launch_bounds__(256) k_gram64(const float* __restrict__ A, const float* __restrict__ B, int rows, int chunk, int m, int ld,
                                                double* __restrict__ parts) {
  constexpr int RS = 64;                               // rows per slice
  __shared__ float sa[RS][17], sb[RS][17];
  const int i0 = blockIdx.y * 16, j0 = blockIdx.x * 16, t = threadIdx.x, ti = t >> 4, tj = t & 15;
  const int r_lo = blockIdx.z * chunk, r_hi = min(rows, r_lo + chunk);
  double acc = 0.0;
  for (int r0 = r_lo; r0 < r_hi; r0 += RS) {
#pragma unroll
    for (int k = 0; k < RS / 16; ++k) {
      const int rr = r0 + ti + 16 * k;
      sa[ti + 16 * k][tj] = (rr < r_hi && i0 + tj < m) ? A[(int64_t)rr * ld + i0 + tj] : 0.f;
      sb[ti + 16 * k][tj] = (rr < r_hi && j0 + tj < m) ? B[(int64_t)rr * ld + j0 + tj] : 0.f;
    }
    __syncthreads();
#pragma unroll 16
    for (int r = 0; r < RS; ++r) acc += (double)sa[r][ti] * (double)sb[r][tj];
    __syncthreads();
  }
  if (i0 + ti < m && j0 + tj < m) parts[((int64_t)blockIdx.z * m + i0 + ti) * m + j0 + tj] = acc;
}
__global__ void k_sum_parts(const double* __restrict__ parts, int n_parts, int n, double* __restrict__ S) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  double v = parts[i];
  for (int z = 1; z < n_parts; ++z) v += parts[(int64_t)z * n + i];
  S[i] = v;
}
// S = A^T B over all rows: the parts, then their sum.
cudaError_t gram64(cudaStream_t st, const float* A, const float* B, int rows, int m, int ld, double* parts, double* S) {
  const int chunk = ((rows + kGramParts - 1) / kGramParts + 63) / 64 * 64;
  dim3 g((m + 15) / 16, (m + 15) / 16, kGramParts);
  k_gram64<<<g, 256, 0, st>>>(A, B, rows, chunk, m, ld, parts);
  k_sum_parts<<<(m * m + 255) / 256, 256, 0, st>>>(parts, kGramParts, m * m, S);
  return cudaGetLastError();
}

// Largest m for which the one-CTA kernels below keep their fp64 matrix in shared memory.
constexpr int kCholSmem = 160;
// The factorisation proper on an m x m matrix S with row stride ls (shared or global memory, the code is the same).
// In shared memory ls is odd: threads that walk down a column (one row each) would otherwise all hit one bank when m
// is a multiple of 16.
__device__ __forceinline__ void chol_inverse_in_place(double* S, const int m, const int ls, double* shift_slot, double* scratch) {
  const int t = threadIdx.x, warp = t >> 5, lane = t & 31;
  if (warp == 0) {
    double tr = 0.0;
    for (int i = lane; i < m; i += 32) tr += S[i * ls + i];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) tr += __shfl_xor_sync(0xffffffffu, tr, o);
    if (lane == 0) *shift_slot = 1e-13 * tr + 1e-300;
  }
  __syncthreads();
  const double shift = *shift_slot;
  for (int i = t; i < m; i += 1024) S[i * ls + i] += shift;
  __syncthreads();
  // Blocked right-looking factorisation, panels of 16 columns: (A) the 16 x 16 diagonal block by one warp, (B) the rows
  // below it by one thread per row (forward substitution against the block), (C) the rank-16 update of the trailing
  // lower triangle by everybody -- three barriers per panel instead of three per column.
  constexpr int NB = 16;
  for (int j0 = 0; j0 < m; j0 += NB) {
    const int jb = m - j0 < NB ? m - j0 : NB;
    if (warp == 0) {
      for (int j = 0; j < jb; ++j) {
        double* dj = S + (j0 + j) * ls + j0;                 // row j0 + j of the block
        const double v = dj[j];
        const double ljj = sqrt(v > shift * 1e-3 ? v : shift * 1e-3);
        __syncwarp();
        if (lane == 0) dj[j] = ljj;
        if (lane > j && lane < jb) S[(j0 + lane) * ls + j0 + j] /= ljj;
        __syncwarp();
        if (lane > j && lane < jb) {
          double* dr = S + (j0 + lane) * ls + j0;
          const double lrj = dr[j];
          for (int c = j + 1; c <= lane; ++c) dr[c] -= lrj * S[(j0 + c) * ls + j0 + j];
        }
        __syncwarp();
      }
    }
    __syncthreads();
    for (int i = j0 + jb + t; i < m; i += 1024) {           // (B)
      double* ri = S + i * ls + j0;
      for (int j = 0; j < jb; ++j) {
        const double* dj = S + (j0 + j) * ls + j0;
        double v = ri[j];
        for (int q = 0; q < j; ++q) v -= ri[q] * dj[q];
        ri[j] = v / dj[j];
      }
    }
    __syncthreads();
    for (int i = j0 + jb + warp; i < m; i += 32) {          // (C)
      const double* li = S + i * ls + j0;
      double lr[NB];
#pragma unroll
      for (int q = 0; q < NB; ++q) lr[q] = q < jb ? li[q] : 0.0;
      for (int c = j0 + jb + lane; c <= i; c += 32) {
        const double* lc = S + c * ls + j0;
        double acc = 0.0;
#pragma unroll
        for (int q = 0; q < NB; ++q) acc += q < jb ? lr[q] * lc[q] : 0.0;
        S[i * ls + c] -= acc;
      }
    }
    __syncthreads();
  }
  // X = L^{-1} by blocks of 16, kept transposed in the strict upper triangle of S (free after the factorisation):
  // S[j][i] = X[i][j] for i > j; the diagonal of X is 1 / L[j][j].
  //   diagonal blocks: X_bb = L_bb^{-1}, one thread per column (16 steps of forward substitution);
  //   then block diagonal by block diagonal (distance dd = 1, 2, ...: the blocks of one diagonal are independent):
  //     P = sum_{kb = jb}^{ib - 1} L_{ib,kb} X_{kb,jb}   (into the scratch, one thread per element),
  //     X_{ib,jb} = - X_{ib,ib} P.
  const int nblk = (m + NB - 1) / NB;
  auto X_at = [&](int i, int j) -> double {               // X[i][j], i >= j
    return i == j ? 1.0 / S[j * ls + j] : S[j * ls + i];
  };
  for (int j = t; j < m; j += 1024) {
    const int b0 = (j / NB) * NB, b1 = b0 + NB < m ? b0 + NB : m;
    const double xjj = 1.0 / S[j * ls + j];
    for (int i = j + 1; i < b1; ++i) {
      double acc = S[i * ls + j] * xjj;
      for (int q = j + 1; q < i; ++q) acc += S[i * ls + q] * S[j * ls + q];
      S[j * ls + i] = -acc / S[i * ls + i];
    }
  }
  __syncthreads();
  for (int dd = 1; dd < nblk; ++dd) {
    const int nb_d = nblk - dd;                            // blocks on this diagonal: (ib, jb) = (jb + dd, jb)
    for (int e = t; e < nb_d * NB * NB; e += 1024) {
      const int jb = e / (NB * NB), r = (e / NB) % NB, c = e % NB, ib = jb + dd;
      const int i = ib * NB + r, j = jb * NB + c;
      double acc = 0.0;
      if (i < m && j < m) {
        const double* li = S + i * ls;
        for (int q = j; q < ib * NB; ++q) acc += li[q] * X_at(q, j);      // X[q][j] = 0 for q < j
      }
      scratch[e] = acc;
    }
    __syncthreads();
    for (int e = t; e < nb_d * NB * NB; e += 1024) {
      const int jb = e / (NB * NB), r = (e / NB) % NB, c = e % NB, ib = jb + dd;
      const int i = ib * NB + r, j = jb * NB + c;
      if (i < m && j < m) {
        double acc = 0.0;
        for (int q = 0; q <= r; ++q) acc += X_at(i, ib * NB + q) * scratch[(jb * NB + q) * NB + c];
        S[j * ls + i] = -acc;
      }
    }
    __syncthreads();
  }
}

// Cholesky S = L L^T (fp64) of an m x m Gram matrix and the inverse of the factor, by one CTA: writes W = L^{-T} as fp32
// into an [ld][ld] matrix (zero outside its upper triangle), so that Q = Y W is orth(Y).  The matrix is worked on in
// shared memory when it fits (m <= kCholSmem), else in place in global memory.  A small multiple of the trace is added
// to the diagonal first, so that a rank-deficient iterate still factors.
__global__ void __launch_bounds__(1024) k_chol_inv64(double* Sg, int m, float* W, int ld) {
  extern __shared__ double sm[];
  __shared__ double shift_s;
  const int t = threadIdx.x;
  const bool in_smem = m <= kCholSmem;
  const int ls = in_smem ? (m | 1) : m;
  if (in_smem) {
    for (int e = t; e < m * m; e += 1024) sm[(e / m) * ls + e % m] = Sg[e];
    __syncthreads();
    chol_inverse_in_place(sm, m, ls, &shift_s, sm + m * ls);
  } else {
    chol_inverse_in_place(Sg, m, ls, &shift_s, sm);
  }
  const double* S = in_smem ? sm : Sg;
  // W[j][i] = X[i][j] (upper triangle of W = L^{-T}); everything else zero
  for (int j = t >> 5; j < ld; j += 32) {
    for (int i = t & 31; i < ld; i += 32) {
      float v = 0.f;
      if (j < m && i < m) {
        if (i == j) v = (float)(1.0 / S[j * ls + j]);
        else if (i > j) v = (float)S[j * ls + i];
      }
      W[j * ld + i] = v;
    }
  }
}

// Symmetric positive semi-definite eigenproblem H = V diag(lam) V^T, m x m, fp64, by one-sided (Hestenes) Jacobi in one
// CTA: pairs of rows of H (= columns, H is symmetric) are rotated until they are orthogonal.  With J the product of the
// rotations the result is J^T H = diag(lam) J^T: row i has norm lam_i and direction v_i, so the eigenvectors are the
// normalised rows and no separate accumulation of the rotations is needed (a row whose norm is zero up to rounding has
// no direction; its eigenvalue is far below the ones that are kept).
// Pairs follow the round-robin tournament (m' / 2 disjoint pairs per step, m' - 1 steps per sweep); a warp takes a pair.
// Output: eigenvalues in descending order (lam) and the matching eigenvectors as fp32 columns of Vf ([m][m] row-major).
__global__ void __launch_bounds__(1024) k_jacobi64(double* Hg, double* V, int m, double* lam, float* Vf, int max_sweeps) {
  extern __shared__ double smj[];
  __shared__ int moved_s;
  __shared__ int rank_s[512];
  const int t = threadIdx.x, nt = blockDim.x, warp = t >> 5, lane = t & 31, nwarp = nt >> 5;
  // the matrix whose columns are rotated is read three times per pair: in shared memory when it fits
  double* H = m <= kCholSmem ? smj : Hg;
  (void)V;
  if (m <= kCholSmem) for (int e = t; e < m * m; e += nt) smj[e] = Hg[e];
  __syncthreads();
  const int mp = (m + 1) & ~1;                       // players of the tournament (one bye if m is odd)
  for (int sweep = 0; sweep < max_sweeps; ++sweep) {
    if (t == 0) moved_s = 0;
    __syncthreads();
    for (int step = 0; step < mp - 1; ++step) {
      for (int pr = warp; pr < mp / 2; pr += nwarp) {
        // circle method: player mp - 1 is fixed, the others rotate
        int p = pr == 0 ? mp - 1 : (step + pr) % (mp - 1);
        int q = (step + mp - 1 - pr) % (mp - 1);
        if (p > q) { const int x = p; p = q; q = x; }
        if (q >= m) continue;                        // the bye
        // columns p and q of H (column c of the symmetric start is stored as row c: H[c * m + i])
        double* hp = H + (int64_t)p * m; double* hq = H + (int64_t)q * m;
        double al = 0.0, be = 0.0, ga = 0.0;
        // up to 160 columns a lane keeps its five elements of both rows in registers between the products and the
        // rotation: the kernel is bound by shared-memory traffic, and this takes a third of it away
        constexpr int KE = 5;
        const bool keep = m <= 32 * KE;
        double av[KE], bv[KE];
        if (keep) {
#pragma unroll
          for (int e = 0; e < KE; ++e) {
            const int i = lane + 32 * e;
            const double a = i < m ? hp[i] : 0.0, b = i < m ? hq[i] : 0.0;
            av[e] = a; bv[e] = b;
            al += a * a; be += b * b; ga += a * b;
          }
        } else {
          for (int i = lane; i < m; i += 32) { const double a = hp[i], b = hq[i]; al += a * a; be += b * b; ga += a * b; }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          al += __shfl_xor_sync(0xffffffffu, al, o); be += __shfl_xor_sync(0xffffffffu, be, o); ga += __shfl_xor_sync(0xffffffffu, ga, o);
        }
        if (fabs(ga) <= 1e-11 * sqrt(al * be) || ga == 0.0) continue;      // orthogonal far beyond what the fp32 operands carry
        const double zeta = (be - al) / (2.0 * ga);
        const double tt = (zeta >= 0.0 ? 1.0 : -1.0) / (fabs(zeta) + sqrt(1.0 + zeta * zeta));
        const double c = 1.0 / sqrt(1.0 + tt * tt), s = c * tt;
        if (keep) {
#pragma unroll
          for (int e = 0; e < KE; ++e) {
            const int i = lane + 32 * e;
            if (i < m) { hp[i] = c * av[e] - s * bv[e]; hq[i] = s * av[e] + c * bv[e]; }
          }
        } else {
          for (int i = lane; i < m; i += 32) {
            const double a = hp[i], b = hq[i];
            hp[i] = c * a - s * b; hq[i] = s * a + c * b;
          }
        }
        if (lane == 0) moved_s = 1;
      }
      __syncthreads();
    }
    const int moved = moved_s;
    __syncthreads();
    if (!moved) break;
  }
  // eigenvalues = column norms; order them (descending; ties by index)
  for (int c = warp; c < m; c += nwarp) {
    double al = 0.0;
    for (int i = lane; i < m; i += 32) { const double a = H[(int64_t)c * m + i]; al += a * a; }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) al += __shfl_xor_sync(0xffffffffu, al, o);
    if (lane == 0) lam[m + c] = sqrt(al);            // unsorted, behind the sorted ones
  }
  __syncthreads();
  for (int c = t; c < m; c += nt) {
    int rk = 0;
    const double mine = lam[m + c];
    for (int o = 0; o < m; ++o) { const double v = lam[m + o]; rk += (v > mine || (v == mine && o < c)) ? 1 : 0; }
    rank_s[c] = rk;
  }
  __syncthreads();
  for (int c = t; c < m; c += nt) lam[rank_s[c]] = lam[m + c];
  __syncthreads();
  for (int e = t; e < m * m; e += nt) {
    const int c = e / m, i = e % m;                  // eigenvector c, component i  ->  Vf[i][rank of c]
    const double nrm = lam[rank_s[c]];
    Vf[(int64_t)i * m + rank_s[c]] = nrm > 0.0 ? (float)(H[e] / nrm) : 0.f;
  }
}

// sigma_i = sqrt(lam_i);  B'[row][i] = U[row][i] sigma_i  (U: [d][r])
__global__ void k_finish_b(const float* __restrict__ U, const double* __restrict__ lam, int d, int r, float* __restrict__ Bp, float* __restrict__ sigma) {
  const int64_t n = (int64_t)d * r;
  for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < n; e += (int64_t)gridDim.x * blockDim.x) {
    const int i = (int)(e % r);
    const float s = (float)sqrt(fmax(lam[i], 0.0));
    Bp[e] = U[e] * s;
    if (e < r) sigma[e] = (float)sqrt(fmax(lam[e], 0.0));
  }
}
// A[i][:] /= sigma_i  (A: [r][k] holding U^T dW)
__global__ void k_finish_a(float* __restrict__ A, const double* __restrict__ lam, int r, int k) {
  const int64_t n = (int64_t)r * k;
  for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < n; e += (int64_t)gridDim.x * blockDim.x) {
    const double s = sqrt(fmax(lam[e / k], 0.0));
    A[e] = s > 0.0 ? (float)((double)A[e] / s) : 0.f;
  }
}
// sum of squares of a matrix, fp64, into *out (zeroed by the caller)
__global__ void k_sumsq(const float* __restrict__ a, int64_t n, double* out) {
  double acc = 0.0;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) acc += (double)a[i] * (double)a[i];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if ((threadIdx.x & 31) == 0) atomicAdd(out, acc);
}
__global__ void k_axpy_neg(float* __restrict__ c, const float* __restrict__ a, int64_t n) {      // c = a - c
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) c[i] = a[i] - c[i];
}

// ------------------------------------------------------------------------------------------------ workspace
struct Plan {
  int d, k, n, r, m, ldm, iters;       // ldm: leading dimension of the iterates (m rounded up to the SGEMM tile, or 160)
  size_t off_w, off_dw, off_g, off_t, off_m, off_y, off_q, off_z, off_u, off_s, off_sp, off_h, off_v, off_lam, off_vf, total;
};
size_t up256(size_t v) { return (v + 255) & ~size_t(255); }
bool make_plan(const eora_solve_config* c, Plan& p) {
  if (!c || c->d < 1 || c->k < 1 || c->n < 1 || c->rank < 1) return false;
  p.d = c->d; p.k = c->k; p.n = c->n; p.r = c->rank;
  int over = c->oversample > 0 ? c->oversample : 32;
  p.m = p.r + over;
  if (p.m > p.d) p.m = p.d;
  if (p.r > p.m || p.m > 512) return false;
  p.iters = c->iters > 0 ? c->iters : 24;
  p.ldm = (p.m + BN - 1) / BN * BN;
  if (p.m > BN && p.m <= NQ && p.d % BMQ == 0) p.ldm = NQ;          // the default width: its own kernel, no padding columns
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o += up256(bytes); return at; };
  p.off_dw = take((size_t)p.d * p.k * 4);
  p.off_g = take((size_t)p.k * p.k * 4);
  p.off_t = take((size_t)p.d * (p.k > p.n ? p.k : p.n) * 4);      // T = dW G; the loss check keeps dW X~ here
  p.off_m = take((size_t)p.d * p.d * 4);
  p.off_y = take((size_t)p.d * p.ldm * 4);
  p.off_q = take((size_t)p.d * p.ldm * 4);
  p.off_z = take((size_t)p.d * p.ldm * 4);
  p.off_w = take((size_t)p.ldm * p.ldm * 4);
  p.off_u = take((size_t)p.d * p.r * 4);
  p.off_s = take((size_t)p.m * p.m * 8);
  p.off_sp = take((size_t)kGramParts * p.m * p.m * 8);
  p.off_h = take((size_t)p.m * p.m * 8);
  p.off_v = take((size_t)p.m * p.m * 8);
  p.off_lam = take((size_t)2 * p.m * 8);
  p.off_vf = take((size_t)p.m * p.m * 4);
  p.total = o;
  return true;
}
inline bool aligned16(const void* q) { return (reinterpret_cast<uintptr_t>(q) & 15) == 0; }

#define CK(x) do { cudaError_t e__ = (x); if (e__ != cudaSuccess) return EORA_ERR_CUDA; } while (0)

// Q = orth(Y) by Cholesky-QR: Gram matrix, factor and its inverse in fp64, then Q = Y L^{-T} as a contraction.
int orthonormalise(cudaStream_t st, const Plan& p, const float* Y, float* Q, double* S, double* parts, float* W) {
  CK(gram64(st, Y, Y, p.d, p.m, p.ldm, parts, S));
  static bool attr_set[64] = {};
  int device = 0;
  if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= 64) return EORA_ERR_CUDA;
  const int smem = (p.m <= kCholSmem ? p.m * (p.m | 1) * 8 : 0) + ((p.m + 15) / 16) * 16 * 16 * 8;     // the matrix (if it fits) and the scratch of the block inverse
  if (!attr_set[device]) {
    CK(cudaFuncSetAttribute(k_chol_inv64, cudaFuncAttributeMaxDynamicSharedMemorySize, kCholSmem * (kCholSmem | 1) * 8 + ((kCholSmem + 15) / 16) * 16 * 16 * 8));
    attr_set[device] = true;
  }
  k_chol_inv64<<<1, 1024, smem, st>>>(S, p.m, W, p.ldm);
  CK(cudaGetLastError());
  CK(sgemm(st, p.d, p.ldm, p.ldm, Y, p.ldm, false, W, p.ldm, false, Q, p.ldm));
  return EORA_OK;
}

}  // namespace

extern "C" {

size_t eora_solve_workspace_bytes(const eora_solve_config* cfg) {
  Plan p;
  return make_plan(cfg, p) ? p.total : 0;
}

int eora_solve(const eora_solve_config* cfg, const float* w, const float* w_hat, const float* x_tilde, float* b_prime, float* a,
               float* sigma, void* workspace, size_t workspace_bytes, void* stream) {
  if (!cfg || !w || !w_hat || !x_tilde || !b_prime || !a || !sigma || !workspace) return EORA_ERR_NULL_ARG;
  Plan p;
  if (!make_plan(cfg, p) || workspace_bytes < p.total) return EORA_ERR_BAD_SHAPE;
  if (!aligned16(w) || !aligned16(w_hat) || !aligned16(x_tilde) || !aligned16(b_prime) || !aligned16(a) || !aligned16(workspace)) return EORA_ERR_MISALIGNED;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  char* ws = reinterpret_cast<char*>(workspace);
  float* dW = reinterpret_cast<float*>(ws + p.off_dw);
  float* G = reinterpret_cast<float*>(ws + p.off_g);
  float* T = reinterpret_cast<float*>(ws + p.off_t);
  float* Mm = reinterpret_cast<float*>(ws + p.off_m);
  float* Y = reinterpret_cast<float*>(ws + p.off_y);
  float* Q = reinterpret_cast<float*>(ws + p.off_q);
  float* Z = reinterpret_cast<float*>(ws + p.off_z);
  float* Wm = reinterpret_cast<float*>(ws + p.off_w);
  float* U = reinterpret_cast<float*>(ws + p.off_u);
  double* S = reinterpret_cast<double*>(ws + p.off_s);
  double* Sp = reinterpret_cast<double*>(ws + p.off_sp);
  double* H = reinterpret_cast<double*>(ws + p.off_h);
  double* V = reinterpret_cast<double*>(ws + p.off_v);
  double* lam = reinterpret_cast<double*>(ws + p.off_lam);
  float* Vf = reinterpret_cast<float*>(ws + p.off_vf);
  const int d = p.d, k = p.k, n = p.n, r = p.r, m = p.m, ldm = p.ldm;

  // step 1
  k_sub<<<592, 256, 0, st>>>(w, w_hat, dW, (int64_t)d * k);
  // steps 2-4, as the d x d matrix dW' dW'^T = dW (X~ X~^T) dW^T
  CK(sgemm(st, k, k, n, x_tilde, n, false, x_tilde, n, true, G, k));          // G = X~ X~^T
  CK(sgemm(st, d, k, k, dW, k, false, G, k, true, T, k));                     // T = dW G = dW G^T (G is symmetric; the row-by-row form of the product is the faster one)
  CK(sgemm(st, d, d, k, T, k, false, dW, k, true, Mm, d));                    // Mm = T dW^T
  // step 5: subspace iteration
  k_init<<<592, 256, 0, st>>>(Y, d, m, ldm);
  if (int rc = orthonormalise(st, p, Y, Q, S, Sp, Wm)) return rc;
  for (int it = 0; it < p.iters; ++it) {
    CK(sgemm(st, d, ldm, d, Mm, d, false, Q, ldm, false, Y, ldm));            // Y = Mm Q
    if (int rc = orthonormalise(st, p, Y, Q, S, Sp, Wm)) return rc;
  }
  if (int rc = orthonormalise(st, p, Q, Y, S, Sp, Wm)) return rc;                 // second pass: orthogonal to fp32 rounding
  // Rayleigh-Ritz on span(Y)
  CK(sgemm(st, d, ldm, d, Mm, d, false, Y, ldm, false, Z, ldm));              // Z = Mm Y
  CK(gram64(st, Y, Z, d, m, ldm, Sp, H));                                     // H = Y^T Mm Y
  {
    static bool jattr[64] = {};
    int device = 0;
    if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= 64) return EORA_ERR_CUDA;
    if (!jattr[device]) { CK(cudaFuncSetAttribute(k_jacobi64, cudaFuncAttributeMaxDynamicSharedMemorySize, kCholSmem * kCholSmem * 8)); jattr[device] = true; }
    k_jacobi64<<<1, 1024, m <= kCholSmem ? m * m * 8 : 0, st>>>(H, V, m, lam, Vf, 40);
  }
  CK(cudaGetLastError());
  CK(sgemm(st, d, r, m, Y, ldm, false, Vf, m, false, U, r));                  // U' = Y V[:, :r]
  // step 6
  k_finish_b<<<296, 256, 0, st>>>(U, lam, d, r, b_prime, sigma);
  CK(sgemm(st, r, k, d, U, r, true, dW, k, false, a, k));                     // U'^T dW
  k_finish_a<<<296, 256, 0, st>>>(a, lam, r, k);
  CK(cudaGetLastError());
  return EORA_OK;
}

int eora_solve_loss(const eora_solve_config* cfg, const float* w, const float* w_hat, const float* x_tilde, const float* b_prime,
                    const float* a, double* loss_sq, void* workspace, size_t workspace_bytes, void* stream) {
  if (!cfg || !w || !w_hat || !x_tilde || !b_prime || !a || !loss_sq || !workspace) return EORA_ERR_NULL_ARG;
  Plan p;
  if (!make_plan(cfg, p) || workspace_bytes < p.total) return EORA_ERR_BAD_SHAPE;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  char* ws = reinterpret_cast<char*>(workspace);
  float* dW = reinterpret_cast<float*>(ws + p.off_dw);
  float* R = reinterpret_cast<float*>(ws + p.off_g);       // B'A, then the residual (d x k fits: the slot holds k x k ... see below)
  float* E = reinterpret_cast<float*>(ws + p.off_t);       // (dW - B'A) X~  (d x n)
  if ((size_t)p.d * p.k > (size_t)p.k * p.k) R = reinterpret_cast<float*>(ws + p.off_m);   // d > k: use the d x d slot
  k_sub<<<592, 256, 0, st>>>(w, w_hat, dW, (int64_t)p.d * p.k);
  CK(sgemm(st, p.d, p.k, p.r, b_prime, p.r, false, a, p.k, false, R, p.k));    // B' A
  k_axpy_neg<<<592, 256, 0, st>>>(R, dW, (int64_t)p.d * p.k);                  // dW - B'A
  CK(sgemm(st, p.d, p.n, p.k, R, p.k, false, x_tilde, p.n, false, E, p.n));
  CK(cudaMemsetAsync(loss_sq, 0, sizeof(double), st));
  k_sumsq<<<592, 256, 0, st>>>(E, (int64_t)p.d * p.n, loss_sq);
  CK(cudaGetLastError());
  return EORA_OK;
}

}  // extern "C"
