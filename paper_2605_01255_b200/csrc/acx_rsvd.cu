// Second factor of the randomized-SVD compressor (Section 5, set-up; Halko, Martinsson, Tropp 2011, Algorithms 4.1
// and 5.1): with the sketch U = X S that the forward stores, the compressed activation of that method is the
// orthogonal projection of X on the range of U, X^ = U (U^T U)^-1 U^T X.  Its factor pair in the sense of Section 4
// is (U, V) with V^T = (U^T U)^-1 U^T X (r x d_in): the same X^ as Q Q^T X with Q from a QR of U, without forming Q,
// so the stored first factor stays the one the forward already wrote.
//
//   C  = X^T U   (d_in x r, fp32)   gradient-factor kernel with X in the place of G_out   (tcgen05, HBM-bound)
//   Gm = U^T U   (r x r, fp32)      the same kernel with U in both places
//   Gi = (Gm + ridge I)^-1          block Gauss-Jordan in double precision, r / 32 launches of (r / 32)^2 CTAs
//   V^T = Gi C^T (r x d_in, bf16)   small FMA kernel, also in double precision: when U is nearly rank deficient the
//                                   entries of Gi are huge and cancel in this product (binary32 lost two digits there)
#include <algorithm>

#include <cuda_bf16.h>

#include "acx_internal.h"

namespace acx {
namespace {

// The sketch is rank deficient when X has rank below r; the ridge (relative to the largest diagonal entry) keeps the
// solve defined and is far below the bfloat16 rounding of U.
constexpr double kRidgeRel = 1.0 / (1 << 20);

// The inverse of Gs = G + ridge I (symmetric positive definite, r <= 256) in double precision by block Gauss-Jordan
// elimination with 32 x 32 blocks: r / 32 launches, each one block pivot of the in-place inversion, spread over
// (r / 32)^2 CTAs.  With pivot block P and Pinv = Gs[P,P]^-1 a launch maps the matrix X to
//     [P,P] -> Pinv      [P,j] -> Pinv X[P,j]      [i,P] -> -X[i,P] Pinv      [i,j] -> X[i,j] - X[i,P] Pinv X[P,j],
// and after the last pivot the matrix is the inverse.  Every CTA inverts the small pivot block itself (unblocked
// Gauss-Jordan in shared memory, one element per thread), so a launch needs nothing from its own grid.
// (An unblocked sweep of the whole matrix in one CTA took 0.35 ms at r = 128: 128 pivots of 2.7 us, the latency of
// barrier -> pivot -> quotient -> update; registers instead of shared memory, a Cholesky factorisation with
// per-column solves, a binary32 sweep with Newton refinement and the symmetric sweep operator did not help.)
constexpr int kBlk = 32;

// Gs (rp x rp, rp = r rounded up to a multiple of 32): symmetrised G plus the ridge, identity in the padding.
// One CTA of 256 threads per row; every CTA finds the largest diagonal entry itself.
__global__ void __launch_bounds__(256) prepare_gram_kernel(const float* __restrict__ G, double* __restrict__ Gs, int r, int rp) {
  __shared__ float red[256];
  const int i = blockIdx.x, j = threadIdx.x;
  red[j] = j < r ? G[j * r + j] : 0.f;
  __syncthreads();
  for (int s = 128; s > 0; s >>= 1) {
    if (j < s) red[j] = fmaxf(red[j], red[j + s]);
    __syncthreads();
  }
  const double mx = red[0] > 0.f ? double(red[0]) : 1.0;
  if (j >= rp) return;
  double v = i == j ? 1.0 : 0.0;
  // symmetrise: the two halves come from different summation orders
  if (i < r && j < r) v = 0.5 * (double(G[i * r + j]) + double(G[j * r + i])) + (i == j ? kRidgeRel * mx : 0.0);
  Gs[i * rp + j] = v;
}

__global__ void __launch_bounds__(kBlk * kBlk) block_gauss_jordan_kernel(const double* __restrict__ in, double* __restrict__ out,
                                                                         int rp, int pb) {
  __shared__ double sP[kBlk][kBlk + 1], sL[kBlk][kBlk + 1], sR[kBlk][kBlk + 1], sT[kBlk][kBlk + 1];
  const int i = threadIdx.x / kBlk, j = threadIdx.x % kBlk;
  const int ib = blockIdx.y, jb = blockIdx.x;
  const int p0 = pb * kBlk, i0 = ib * kBlk, j0 = jb * kBlk;
  sP[i][j] = in[(p0 + i) * rp + p0 + j];
  sL[i][j] = in[(i0 + i) * rp + p0 + j];  // X[i-block, P]
  sR[i][j] = in[(p0 + i) * rp + j0 + j];  // X[P, j-block]
  const double own = in[(i0 + i) * rp + j0 + j];
  __syncthreads();
  // Pinv: unblocked in-place Gauss-Jordan without pivoting (the pivot block is a Schur complement of a positive
  // definite matrix, so its pivots are positive)
  for (int k = 0; k < kBlk; ++k) {
    const double p = sP[k][k], rk = sP[k][j], ci = sP[i][k], a = sP[i][j];
    __syncthreads();
    const double ip = 1.0 / fmax(p, 1e-290);
    sP[i][j] = (i == k) ? ((j == k) ? ip : rk * ip) : ((j == k) ? -ci * ip : fma(-ci * ip, rk, a));
    __syncthreads();
  }
  double v;
  if (ib == pb && jb == pb) {
    v = sP[i][j];
  } else if (ib == pb) {  // Pinv X[P,j]
    v = 0.0;
#pragma unroll 8
    for (int k = 0; k < kBlk; ++k) v = fma(sP[i][k], sR[k][j], v);
  } else if (jb == pb) {  // -X[i,P] Pinv
    v = 0.0;
#pragma unroll 8
    for (int k = 0; k < kBlk; ++k) v = fma(sL[i][k], sP[k][j], v);
    v = -v;
  } else {  // X[i,j] - X[i,P] (Pinv X[P,j])
    double t = 0.0;
#pragma unroll 8
    for (int k = 0; k < kBlk; ++k) t = fma(sP[i][k], sR[k][j], t);
    sT[i][j] = t;
    __syncthreads();
    v = own;
#pragma unroll 8
    for (int k = 0; k < kBlk; ++k) v = fma(-sL[i][k], sT[k][j], v);
  }
  out[(i0 + i) * rp + j0 + j] = v;
}

// Vt[j][i] = sum_k Gi[j][k] C[i][k] in bfloat16 (Gi with leading dimension ld); blockDim = r rounded up to 128.  A block (thread = row j of V^T) takes 8 columns i.
__global__ void __launch_bounds__(256) apply_inverse_kernel(const double* __restrict__ Gi, int ld, const float* __restrict__ C,
                                                            __nv_bfloat16* __restrict__ Vt, int r, int64_t d_in) {
  __shared__ float c_rows[8][256];
  const int64_t i0 = int64_t(blockIdx.x) * 8;
  for (int idx = threadIdx.x; idx < 8 * r; idx += blockDim.x) {
    const int c = idx / r, k = idx - c * r;
    c_rows[c][k] = (i0 + c < d_in) ? C[(i0 + c) * r + k] : 0.f;
  }
  __syncthreads();
  const int j = threadIdx.x;
  if (j >= r) return;
  double acc[8] = {0.0, 0.0, 0.0, 0.0, 0.0, 0.0, 0.0, 0.0};
  for (int k = 0; k < r; ++k) {
    const double g = Gi[k * ld + j];  // Gi is symmetric: row k read along j is contiguous over the threads
#pragma unroll
    for (int c = 0; c < 8; ++c) acc[c] = fma(g, double(c_rows[c][k]), acc[c]);
  }
  uint32_t w[4];
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    __nv_bfloat162 h = __floats2bfloat162_rn(float(acc[2 * c]), float(acc[2 * c + 1]));
    w[c] = *reinterpret_cast<uint32_t*>(&h);
  }
  // d_in is a multiple of 8, so the 8 columns are all inside the matrix and the 16-byte store is aligned
  *reinterpret_cast<uint4*>(Vt + int64_t(j) * d_in + i0) = make_uint4(w[0], w[1], w[2], w[3]);
}

size_t align256(size_t n) { return (n + 255) & ~size_t(255); }

Problem with_rows(const Problem& q, int64_t d_out) {
  Problem p = q;
  p.d_out = d_out;
  return p;
}

}  // namespace

size_t sm100_rsvd_workspace_bytes(const Problem& q) {
  const size_t scratch = std::max(sm100_bwd_workspace_bytes(with_rows(q, q.d_in)), sm100_bwd_workspace_bytes(with_rows(q, q.r)));
  const size_t rp = (size_t(q.r) + kBlk - 1) / kBlk * kBlk;
  return align256(size_t(q.d_in) * q.r * 4) + align256(size_t(q.r) * q.r * 4) + 2 * align256(rp * rp * 8) + align256(scratch);
}

cudaError_t sm100_rsvd_factor(const Problem& q, const void* X, const void* U, void* Vt, void* ws, int* status, cudaStream_t st) {
  uint8_t* base = static_cast<uint8_t*>(ws);
  float* C = reinterpret_cast<float*>(base);
  float* Gm = reinterpret_cast<float*>(base + align256(size_t(q.d_in) * q.r * 4));
  const int rp = (q.r + kBlk - 1) / kBlk * kBlk, nb = rp / kBlk;
  const size_t rr8 = align256(size_t(rp) * rp * 8);
  double* Xa = reinterpret_cast<double*>(reinterpret_cast<uint8_t*>(Gm) + align256(size_t(q.r) * q.r * 4));
  double* Xb = reinterpret_cast<double*>(reinterpret_cast<uint8_t*>(Xa) + rr8);
  void* scratch = reinterpret_cast<uint8_t*>(Xb) + rr8;
  // C = X^T U and Gm = U^T U: contractions over the tokens, exactly the gradient factor's shape
  cudaError_t e = sm100_factor(with_rows(q, q.d_in), X, U, C, scratch, status, st, /*allow_cluster=*/true);
  if (e != cudaSuccess) return e;
  e = sm100_factor(with_rows(q, q.r), U, U, Gm, scratch, status, st, /*allow_cluster=*/true);
  if (e != cudaSuccess) return e;
  prepare_gram_kernel<<<unsigned(rp), 256, 0, st>>>(Gm, Xa, q.r, rp);
  e = launched();
  if (e != cudaSuccess) return e;
  double* cur = Xa;
  double* nxt = Xb;
  for (int pb = 0; pb < nb; ++pb) {
    block_gauss_jordan_kernel<<<dim3(unsigned(nb), unsigned(nb)), kBlk * kBlk, 0, st>>>(cur, nxt, rp, pb);
    e = launched();
    if (e != cudaSuccess) return e;
    std::swap(cur, nxt);
  }
  apply_inverse_kernel<<<unsigned((q.d_in + 7) / 8), q.r > 128 ? 256 : 128, 0, st>>>(cur, rp, C, static_cast<__nv_bfloat16*>(Vt), q.r, q.d_in);
  return launched();
}

}  // namespace acx
