// Bias gradient of the affine operator Z = X W^T + 1 b^T (appendix, "Bias term": the bias gradient does not depend
// on X, so activation compression leaves it exact): db[c] = sum over the tokens of G[t][c].
// Two deterministic stages: partial sums over token ranges (fixed order inside a block), then the ranges in order.
#include <algorithm>

#include <cuda_bf16.h>

#include "acx_internal.h"
#include "acx_tmap.h"

namespace acx {
namespace {

constexpr int kColsPerBlock = 256;  // a warp = 32 threads x 8 columns (16 bytes): 512 contiguous bytes of a row
constexpr int kRowLanes = 8;

int bias_grad_splits(const Problem& q) {
  const int col_blocks = int((q.d_out + kColsPerBlock - 1) / kColsPerBlock);
  const int want = (4 * sm_count() + col_blocks - 1) / col_blocks;
  const int by_rows = int(std::max<int64_t>(1, q.m / (4 * kRowLanes)));
  return std::max(1, std::min(std::min(want, by_rows), 64));
}

__global__ void __launch_bounds__(256) column_partial_sums_kernel(const __nv_bfloat16* __restrict__ G, float* __restrict__ part,
                                                                  int64_t m, int64_t d_out, int64_t rows_per_split) {
  __shared__ float red[kRowLanes][kColsPerBlock + 1];
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const int64_t col = int64_t(blockIdx.x) * kColsPerBlock + tx * 8;
  const int64_t r0 = int64_t(blockIdx.y) * rows_per_split, r1 = min(m, r0 + rows_per_split);
  float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  if (col < d_out) {  // d_out is a multiple of 8: a group of 8 columns is inside or outside as a whole
    // four rows in flight per thread: the pass is bound by HBM latency times the bytes outstanding
    for (int64_t t = r0 + ty; t < r1; t += 4 * kRowLanes) {
      uint4 v[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int64_t tu = t + u * kRowLanes;
        v[u] = tu < r1 ? __ldg(reinterpret_cast<const uint4*>(G + tu * d_out + col)) : make_uint4(0u, 0u, 0u, 0u);
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {  // rows are added in token order, whatever the unrolling
        const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          acc[2 * i] += __uint_as_float(w[i] << 16);
          acc[2 * i + 1] += __uint_as_float(w[i] & 0xFFFF0000u);
        }
      }
    }
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) red[ty][tx * 8 + i] = acc[i];
  __syncthreads();
  if (threadIdx.x < kColsPerBlock) {
    const int64_t c = int64_t(blockIdx.x) * kColsPerBlock + threadIdx.x;
    if (c < d_out) {
      float s = 0.f;
      for (int y = 0; y < kRowLanes; ++y) s += red[y][threadIdx.x];
      part[int64_t(blockIdx.y) * d_out + c] = s;
    }
  }
}

__global__ void __launch_bounds__(256) sum_partials_kernel(const float* __restrict__ part, float* __restrict__ db, int64_t d_out,
                                                           int splits) {
  const int64_t c = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
  if (c >= d_out) return;
  float s = 0.f;
  for (int z = 0; z < splits; ++z) s += part[int64_t(z) * d_out + c];
  db[c] = s;
}

}  // namespace

cudaError_t sum_column_partials(const float* part, float* db, int64_t d_out, int splits, cudaStream_t st) {
  sum_partials_kernel<<<unsigned((d_out + 255) / 256), 256, 0, st>>>(part, db, d_out, splits);
  return launched();
}

size_t bias_grad_workspace_bytes(const Problem& q) { return size_t(bias_grad_splits(q)) * size_t(q.d_out) * 4; }

cudaError_t bias_grad(const Problem& q, const void* G, float* db, void* ws, cudaStream_t st) {
  const int splits = bias_grad_splits(q);
  const int64_t rows_per_split = (q.m + splits - 1) / splits;
  const dim3 grid(unsigned((q.d_out + kColsPerBlock - 1) / kColsPerBlock), unsigned(splits));
  column_partial_sums_kernel<<<grid, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(G), static_cast<float*>(ws), q.m, q.d_out,
                                                   rows_per_split);
  cudaError_t e = launched();
  if (e != cudaSuccess) return e;
  sum_partials_kernel<<<unsigned((q.d_out + 255) / 256), 256, 0, st>>>(static_cast<const float*>(ws), db, q.d_out, splits);
  return launched();
}

}  // namespace acx
