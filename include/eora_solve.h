/*
 * Offline EoRA solve on the GPU: Algorithm 1, steps 1-6 (Section 3 of the paper) for one layer.
 *
 *   input   W, W^  [d][k]   full-precision and compressed weight (d outputs, k inputs; the paper's orientation)
 *           X~     [k][n]   calibration activations of the layer (n columns)
 *           r               compensation rank
 *   output  B'     [d][r],  A [r][k]    with   W^ X + B' A X   the compensated layer (step 7 / Eq. 4),
 *           sigma  [r]      the top-r singular values of the projected error dW' = dW Q sqrt(L)
 *
 * What is computed.  Steps 2-6 define B' = U' S' and A = S'^{-1} U'^T dW, where U' (d x r) and S'^2 are the top-r
 * eigenpairs of  dW (X~ X~^T) dW^T = dW' dW'^T  (the left singular vectors and squared singular values of dW'):
 * with dW' = U' S' V'^T,  A = V'^T Q'^{-1} = S'^{-1} U'^T dW' Q'^{-1} = S'^{-1} U'^T dW.  The library forms that
 * d x d matrix and takes its top-r eigenpairs by subspace iteration with a Rayleigh-Ritz step, so it needs neither
 * the k x k eigendecomposition nor the inverse square roots of its (possibly zero) eigenvalues.  B' and A are
 * determined up to one common sign per rank-one pair (as with any SVD); B' A, sigma and the remaining loss are unique
 * where sigma_r > sigma_{r+1}.  Subspace iteration converges like (sigma_{m+1} / sigma_r)^(2 iters), m = r + oversample:
 * the remaining layer-wise loss || (dW - B'A) X~ ||_F is within a factor 1 + O(that) of the optimum of Theorem 1.
 *
 * All pointers are DEVICE pointers to row-major fp32, 16-byte aligned, caller-owned; nothing is allocated, all work is
 * enqueued on `stream` and nothing synchronises.  `workspace` must hold eora_solve_workspace_bytes(cfg) bytes.
 * Arithmetic: fp32 products with fp32 accumulation for the large contractions, fp64 for the small (r + oversample)^2
 * problems (Gram matrices of the iterate, Cholesky factor, Jacobi eigenproblem).
 *
 * Returns EORA_OK, or EORA_ERR_NULL_ARG / _BAD_SHAPE (d, k, n, rank < 1, rank + oversample > min(d, 512), workspace too
 * small) / _MISALIGNED / _CUDA (codes of eora_linear.h).
 */
#ifndef EORA_SOLVE_H
#define EORA_SOLVE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct {
  int32_t d, k, n;        /* W, W^: [d][k];  X~: [k][n] */
  int32_t rank;           /* r */
  int32_t oversample;     /* extra vectors carried by the subspace iteration (0: library default, 32) */
  int32_t iters;          /* subspace iterations (0: library default, 24) */
} eora_solve_config;

size_t eora_solve_workspace_bytes(const eora_solve_config* cfg);

int eora_solve(const eora_solve_config* cfg, const float* w, const float* w_hat, const float* x_tilde,
               float* b_prime, float* a, float* sigma, void* workspace, size_t workspace_bytes, void* stream);

/* || (dW - B' A) X~ ||_F^2 on the device (fp32 products, fp64 sum), written to *loss_sq (device, one double):
 * the quantity Theorem 1 is about, for checking a solution without leaving the GPU.  Same conventions as eora_solve;
 * workspace of eora_solve_workspace_bytes(cfg) bytes. */
int eora_solve_loss(const eora_solve_config* cfg, const float* w, const float* w_hat, const float* x_tilde,
                    const float* b_prime, const float* a, double* loss_sq, void* workspace, size_t workspace_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif
