// Second factor of the randomized-SVD compressor (Section 5, set-up; Halko, Martinsson, Tropp 2011, Algorithms 4.1
// and 5.1): with the sketch U = X S that the forward stores, the compressed activation of that method is the
// orthogonal projection of X on the range of U, X^ = U (U^T U)^-1 U^T X.  Its factor pair in the sense of Section 4
// is (U, V) with V^T = (U^T U)^-1 U^T X (r x d_in): the same X^ as Q Q^T X with Q from a QR of U, without forming Q,
// so the stored first factor stays the one the forward already wrote.
//
//   C  = X^T U   (d_in x r, fp32)   gradient-factor kernel with X in the place of G_out   (tcgen05, HBM-bound)
//   Gm = U^T U   (r x r, fp32)      the same kernel with U in both places
//   Gi = (Gm + ridge I)^-1          one CTA, Gauss-Jordan in double precision in shared memory
//   V^T = Gi C^T (r x d_in, bf16)   small FMA kernel, also in double precision: when U is nearly rank deficient the
//                                   entries of Gi are huge and cancel in this product (binary32 lost two digits there)
#include <algorithm>

#include <cuda_bf16.h>

#include "acx_internal.h"

namespace acx {
namespace {

constexpr int kInvThreads = 1024;
// The sketch is rank deficient when X has rank below r; the ridge (relative to the largest diagonal entry) keeps the
// solve defined and is far below the bfloat16 rounding of U.
constexpr double kRidgeRel = 1.0 / (1 << 20);

// Gi = (G + ridge I)^-1 for a symmetric positive semi-definite r x r matrix, r <= 128: the in-place Gauss-Jordan sweep
// without pivoting (pivot k: a_kk <- 1/p, row k <- row k / p, column k <- -column k / p, a_ij <- a_ij - a_ik a_kj / p)
// in double precision in shared memory, one CTA: r^3 element updates on one SM (0.35 ms at r = 128, 10 us at r = 32).
// Keeping the matrix in registers, and a binary32 sweep, were both slower: the instructions per update, not the
// double-precision rate, are what a single SM cannot hide.
__global__ void __launch_bounds__(kInvThreads) spd_inverse_kernel(const float* __restrict__ G, double* __restrict__ Gi, int r) {
  extern __shared__ double sm[];
  double* a = sm;             // r x r
  double* colk = sm + r * r;  // r
  double* rowk = colk + r;    // r
  __shared__ double s_max;
  if (threadIdx.x == 0) {
    double mx = 0.0;
    for (int i = 0; i < r; ++i) mx = fmax(mx, double(G[i * r + i]));
    s_max = mx > 0.0 ? mx : 1.0;
  }
  __syncthreads();
  const double ridge = kRidgeRel * s_max;
  for (int idx = threadIdx.x; idx < r * r; idx += kInvThreads) {
    const int i = idx / r, j = idx - i * r;
    // symmetrise: the two halves come from different summation orders
    a[idx] = 0.5 * (double(G[idx]) + double(G[j * r + i])) + (i == j ? ridge : 0.0);
  }
  // thread -> one column j and every groups-th row from its group on: no index arithmetic inside the sweep, and a
  // warp's accesses to a row are contiguous
  const int groups = kInvThreads / r;  // >= 8
  const int j = int(threadIdx.x) % r, g = int(threadIdx.x) / r;
  const bool active = g < groups;
  for (int k = 0; k < r; ++k) {
    __syncthreads();
    if (threadIdx.x < r) {
      colk[threadIdx.x] = a[threadIdx.x * r + k];
      rowk[threadIdx.x] = a[k * r + threadIdx.x];
    }
    __syncthreads();
    const double p = fmax(rowk[k], ridge * 1e-3);  // positive by construction; the floor only guards rounding
    const double ip = 1.0 / p;
    if (active) {
      const double rj = rowk[j] * ip;  // the new row k, except its diagonal entry
      for (int i = g; i < r; i += groups) {
        double v;
        if (i == k) v = (j == k) ? ip : rj;
        else v = (j == k) ? -colk[i] * ip : fma(-colk[i], rj, a[i * r + j]);
        a[i * r + j] = v;
      }
    }
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < r * r; idx += kInvThreads) Gi[idx] = a[idx];
}

// Vt[j][i] = sum_k Gi[j][k] C[i][k] in bfloat16.  A block of 128 threads (thread = row j of V^T) takes 8 columns i.
__global__ void __launch_bounds__(128) apply_inverse_kernel(const double* __restrict__ Gi, const float* __restrict__ C,
                                                            __nv_bfloat16* __restrict__ Vt, int r, int64_t d_in) {
  __shared__ float c_rows[8][128];
  const int64_t i0 = int64_t(blockIdx.x) * 8;
  for (int idx = threadIdx.x; idx < 8 * r; idx += 128) {
    const int c = idx / r, k = idx - c * r;
    c_rows[c][k] = (i0 + c < d_in) ? C[(i0 + c) * r + k] : 0.f;
  }
  __syncthreads();
  const int j = threadIdx.x;
  if (j >= r) return;
  double acc[8] = {0.0, 0.0, 0.0, 0.0, 0.0, 0.0, 0.0, 0.0};
  for (int k = 0; k < r; ++k) {
    const double g = Gi[k * r + j];  // Gi is symmetric: row k read along j is contiguous over the threads
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
  return align256(size_t(q.d_in) * q.r * 4) + align256(size_t(q.r) * q.r * 4) + align256(size_t(q.r) * q.r * 8) + align256(scratch);
}

cudaError_t sm100_rsvd_factor(const Problem& q, const void* X, const void* U, void* Vt, void* ws, int* status, cudaStream_t st) {
  uint8_t* base = static_cast<uint8_t*>(ws);
  float* C = reinterpret_cast<float*>(base);
  float* Gm = reinterpret_cast<float*>(base + align256(size_t(q.d_in) * q.r * 4));
  double* Gi = reinterpret_cast<double*>(reinterpret_cast<uint8_t*>(Gm) + align256(size_t(q.r) * q.r * 4));
  void* scratch = reinterpret_cast<uint8_t*>(Gi) + align256(size_t(q.r) * q.r * 8);
  // C = X^T U and Gm = U^T U: contractions over the tokens, exactly the gradient factor's shape
  cudaError_t e = sm100_factor(with_rows(q, q.d_in), X, U, C, scratch, status, st, /*allow_cluster=*/true);
  if (e != cudaSuccess) return e;
  e = sm100_factor(with_rows(q, q.r), U, U, Gm, scratch, status, st, /*allow_cluster=*/true);
  if (e != cudaSuccess) return e;
  const int smem = int(sizeof(double)) * (q.r * q.r + 2 * q.r);
  static DeviceOnce once;
  if (once.needed()) {
    e = cudaFuncSetAttribute(spd_inverse_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(sizeof(double)) * (128 * 128 + 256));
    if (e != cudaSuccess) return e;
    once.done();
  }
  spd_inverse_kernel<<<1, kInvThreads, smem, st>>>(Gm, Gi, q.r);
  e = launched();
  if (e != cudaSuccess) return e;
  apply_inverse_kernel<<<unsigned((q.d_in + 7) / 8), 128, 0, st>>>(Gi, C, static_cast<__nv_bfloat16*>(Vt), q.r, q.d_in);
  return launched();
}

}  // namespace acx
