// SIMT (CUDA-core) kernels: the fp32 data path of every op, for any valid shape.
//
// fp32 inputs must meet a 1e-5 relative error, which tensor-core tf32 (10-bit significand) cannot,
// so this path multiplies and accumulates in binary32 on the FMA pipes.  One tiled kernel serves all
// five products of the compressed linear operator (Definition 3.1, Section 4):
//   Y = X W^T,  XS = X S,  dX = G W,  A = G^T XS (split over tokens),  dW = beta dW + A S^T,
// with the sketch operand generated in place of a global-memory load.
#include "acx_internal.h"
#include "acx_tmap.h"

namespace acx {
namespace {

constexpr int BM = 64, BN = 64, BK = 32, NT = 256, PAD = 1;

enum BMode { B_STRIDED = 0, B_SKETCH_KN = 1 /* B(k,n) = S[k][n] */, B_SKETCH_NK = 2 /* B(k,n) = S[n][k] */ };

struct GemmArgs {
  const void* A; int64_t a_sm, a_sk;   // A(m,k) = A[m*a_sm + k*a_sk]
  const void* B; int64_t b_sk, b_sn;   // B(k,n) = B[k*b_sk + n*b_sn]   (B_STRIDED only)
  void* C; int64_t ldc;                // C(m,n) = C[m*ldc + n]  (+ blockIdx.z * c_split_stride)
  int64_t M, N, K;
  int64_t k_per_split, c_split_stride; // split over K by blockIdx.z
  float beta;
  SketchParams sp;
  int sketch_bf16;                     // round generated S through bf16
};

template <typename T> __device__ __forceinline__ float load_f(const T* p);
template <> __device__ __forceinline__ float load_f<float>(const float* p) { return __ldg(p); }
template <> __device__ __forceinline__ float load_f<__nv_bfloat16>(const __nv_bfloat16* p) { return __bfloat162float(*p); }
template <typename T> __device__ __forceinline__ void store_f(T* p, float v);
template <> __device__ __forceinline__ void store_f<float>(float* p, float v) { *p = v; }
template <> __device__ __forceinline__ void store_f<__nv_bfloat16>(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

template <typename TA, typename TB, typename TC, bool A_KCONTIG, bool B_KCONTIG, int BMODE>
__global__ void __launch_bounds__(NT) simt_gemm_kernel(const GemmArgs g) {
  __shared__ float As[BK][BM + PAD];
  __shared__ float Bs[BK][BN + PAD];
  const int tid = threadIdx.x;
  // tiles are numbered along grid.x, N fastest (grid.y would cap the row tiles at 65535)
  const int64_t n_tiles = (g.N + BN - 1) / BN;
  const int64_t m0 = (int64_t(blockIdx.x) / n_tiles) * BM, n0 = (int64_t(blockIdx.x) % n_tiles) * BN;
  const int64_t k_begin = int64_t(blockIdx.z) * g.k_per_split;
  const int64_t k_end = min(g.K, k_begin + g.k_per_split);
  const TA* __restrict__ A = static_cast<const TA*>(g.A);
  const TB* __restrict__ B = static_cast<const TB*>(g.B);
  const int tx = tid % 16, ty = tid / 16;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

  for (int64_t k0 = k_begin; k0 < k_end; k0 += BK) {
    // ---- stage A
    if (A_KCONTIG) {
      const int kk = tid % BK;
#pragma unroll
      for (int i = 0; i < BM * BK / NT; ++i) {
        const int mm = tid / BK + (NT / BK) * i;
        const int64_t m = m0 + mm, k = k0 + kk;
        As[kk][mm] = (m < g.M && k < k_end) ? load_f(A + m * g.a_sm + k * g.a_sk) : 0.f;
      }
    } else {
      const int mm = tid % BM;
#pragma unroll
      for (int i = 0; i < BM * BK / NT; ++i) {
        const int kk = tid / BM + (NT / BM) * i;
        const int64_t m = m0 + mm, k = k0 + kk;
        As[kk][mm] = (m < g.M && k < k_end) ? load_f(A + m * g.a_sm + k * g.a_sk) : 0.f;
      }
    }
    // ---- stage B
    if (BMODE == B_STRIDED) {
      if (B_KCONTIG) {
        const int kk = tid % BK;
#pragma unroll
        for (int i = 0; i < BN * BK / NT; ++i) {
          const int nn = tid / BK + (NT / BK) * i;
          const int64_t n = n0 + nn, k = k0 + kk;
          Bs[kk][nn] = (n < g.N && k < k_end) ? load_f(B + k * g.b_sk + n * g.b_sn) : 0.f;
        }
      } else {
        const int nn = tid % BN;
#pragma unroll
        for (int i = 0; i < BN * BK / NT; ++i) {
          const int kk = tid / BN + (NT / BN) * i;
          const int64_t n = n0 + nn, k = k0 + kk;
          Bs[kk][nn] = (n < g.N && k < k_end) ? load_f(B + k * g.b_sk + n * g.b_sn) : 0.f;
        }
      }
    } else if (BMODE == B_SKETCH_KN) {
      // rows of S along k, column quads along n: (BN/4) quads per k row
#pragma unroll
      for (int i = 0; i < (BK * BN / 4) / NT; ++i) {
        const int q = tid % (BN / 4), kk = tid / (BN / 4) + (NT / (BN / 4)) * i;
        const int64_t k = k0 + kk, n = n0 + 4 * q;
        float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
        if (k < k_end && n < g.N) z = sketch_quad(g.sp, uint32_t(k), uint32_t(n >> 2));
        if (g.sketch_bf16) { z.x = round_through_bf16(z.x); z.y = round_through_bf16(z.y); z.z = round_through_bf16(z.z); z.w = round_through_bf16(z.w); }
        Bs[kk][4 * q + 0] = z.x; Bs[kk][4 * q + 1] = z.y; Bs[kk][4 * q + 2] = z.z; Bs[kk][4 * q + 3] = z.w;
      }
    } else {
      // rows of S along n, column quads along k: (BK/4) quads per n row
#pragma unroll
      for (int i = 0; i < (BK * BN / 4) / NT; ++i) {
        const int q = tid % (BK / 4), nn = tid / (BK / 4) + (NT / (BK / 4)) * i;
        const int64_t n = n0 + nn, k = k0 + 4 * q;
        float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
        if (n < g.N && k < k_end) z = sketch_quad(g.sp, uint32_t(n), uint32_t(k >> 2));
        if (g.sketch_bf16) { z.x = round_through_bf16(z.x); z.y = round_through_bf16(z.y); z.z = round_through_bf16(z.z); z.w = round_through_bf16(z.w); }
        Bs[4 * q + 0][nn] = z.x; Bs[4 * q + 1][nn] = z.y; Bs[4 * q + 2][nn] = z.z; Bs[4 * q + 3][nn] = z.w;
      }
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = Bs[kk][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }

  TC* __restrict__ C = static_cast<TC*>(g.C) + int64_t(blockIdx.z) * g.c_split_stride;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int64_t m = m0 + ty * 4 + i;
    if (m >= g.M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int64_t n = n0 + tx * 4 + j;
      if (n >= g.N) continue;
      float v = acc[i][j];
      if (g.beta != 0.f) v = fmaf(g.beta, load_f(C + m * g.ldc + n), v);
      store_f(C + m * g.ldc + n, v);
    }
  }
}

// Sum the split-K partials in a fixed order (bitwise reproducible), 4 outputs per thread.
__global__ void __launch_bounds__(256) reduce_partials_kernel(const float4* __restrict__ part, float4* __restrict__ out,
                                                              int64_t n4, int splits) {
  const int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i >= n4) return;
  float4 s = part[i];
  for (int z = 1; z < splits; ++z) {
    const float4 v = part[int64_t(z) * n4 + i];
    s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
  }
  out[i] = s;
}

__global__ void __launch_bounds__(256) sketch_materialize_kernel(void* out, int64_t d_in, int r, SketchParams sp, int bf16) {
  const int quads_per_row = r / 4;
  const int64_t idx = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
  if (idx >= d_in * quads_per_row) return;
  const int64_t i = idx / quads_per_row;
  const int q = int(idx % quads_per_row);
  const float4 z = sketch_quad(sp, uint32_t(i), uint32_t(q));
  if (bf16) {
    __nv_bfloat162 lo = __floats2bfloat162_rn(z.x, z.y), hi = __floats2bfloat162_rn(z.z, z.w);
    uint2 v;
    v.x = *reinterpret_cast<uint32_t*>(&lo);
    v.y = *reinterpret_cast<uint32_t*>(&hi);
    reinterpret_cast<uint2*>(out)[idx] = v;
  } else {
    reinterpret_cast<float4*>(out)[idx] = z;
  }
}

template <typename TA, typename TB, typename TC, bool AK, bool BK_, int BMODE>
cudaError_t launch(const GemmArgs& g, int splits, cudaStream_t st) {
  if (g.M == 0 || g.N == 0) return cudaSuccess;
  const int64_t tiles = ((g.N + BN - 1) / BN) * ((g.M + BM - 1) / BM);
  if (tiles > 0x7FFFFFFFll) return cudaErrorInvalidConfiguration;   // validate() rejects such shapes before any launch
  dim3 grid((unsigned)tiles, 1u, (unsigned)splits);
  simt_gemm_kernel<TA, TB, TC, AK, BK_, BMODE><<<grid, NT, 0, st>>>(g);
  return launched();
}

int bwd_splits(const Problem& p) {
  // enough CTAs to fill the machine, at least 256 tokens per split
  const int64_t tiles = ((p.d_out + BM - 1) / BM) * ((p.r + BN - 1) / BN);
  int64_t s = (4 * int64_t(sm_count()) + tiles - 1) / tiles;
  const int64_t max_s = (p.m + 255) / 256;
  if (s > max_s) s = max_s;
  if (s < 1) s = 1;
  if (s > 64) s = 64;
  return int(s);
}

template <typename T>
cudaError_t fwd_t(const Problem& p, const void* X, const void* W, void* Y, void* XS, cudaStream_t st, const void* Vt) {
  GemmArgs g{};
  g.A = X; g.a_sm = p.d_in; g.a_sk = 1;
  g.M = p.m; g.K = p.d_in; g.k_per_split = p.d_in; g.c_split_stride = 0; g.beta = 0.f;
  g.sp = p.sp; g.sketch_bf16 = p.bf16;
  g.B = W; g.b_sk = 1; g.b_sn = p.d_in; g.C = Y; g.ldc = p.d_out; g.N = p.d_out;
  cudaError_t e = launch<T, T, T, true, true, B_STRIDED>(g, 1, st);
  if (e != cudaSuccess || !XS) return e;
  g.C = XS; g.ldc = p.r; g.N = p.r;
  if (Vt) {  // XS = X V with V^T (r x d_in) in memory: B(k, n) = Vt[n * d_in + k]
    g.B = Vt; g.b_sk = 1; g.b_sn = p.d_in;
    return launch<T, T, T, true, true, B_STRIDED>(g, 1, st);
  }
  g.B = nullptr;
  return launch<T, T, T, true, true, B_SKETCH_KN>(g, 1, st);
}

template <typename T>
cudaError_t bwd_t(const Problem& p, const void* G, const void* W, const void* XS, void* dX, float* A, void* ws,
                  cudaStream_t st) {
  if (dX) {
    GemmArgs g{};
    g.A = G; g.a_sm = p.d_out; g.a_sk = 1;
    g.B = W; g.b_sk = p.d_in; g.b_sn = 1;
    g.C = dX; g.ldc = p.d_in; g.M = p.m; g.N = p.d_in; g.K = p.d_out; g.k_per_split = p.d_out;
    cudaError_t e = launch<T, T, T, true, false, B_STRIDED>(g, 1, st);
    if (e != cudaSuccess) return e;
  }
  if (A) {
    const int splits = bwd_splits(p);
    GemmArgs g{};
    g.A = G; g.a_sm = 1; g.a_sk = p.d_out;     // A(m = o, k = t) = G[t][o]
    g.B = XS; g.b_sk = p.r; g.b_sn = 1;        // B(k = t, n = j) = XS[t][j]
    g.M = p.d_out; g.N = p.r; g.K = p.m; g.ldc = p.r;
    g.k_per_split = ((p.m + splits - 1) / splits + BK - 1) / BK * BK;
    if (p.m == 0) return cudaMemsetAsync(A, 0, sizeof(float) * p.d_out * p.r, st);
    if (splits == 1) {
      g.C = A; g.c_split_stride = 0;
      return launch<T, T, float, false, false, B_STRIDED>(g, 1, st);
    }
    g.C = ws; g.c_split_stride = p.d_out * int64_t(p.r);
    cudaError_t e = launch<T, T, float, false, false, B_STRIDED>(g, splits, st);
    if (e != cudaSuccess) return e;
    const int64_t n4 = p.d_out * int64_t(p.r) / 4;
    reduce_partials_kernel<<<(unsigned)((n4 + 255) / 256), 256, 0, st>>>(static_cast<const float4*>(ws),
                                                                        reinterpret_cast<float4*>(A), n4, splits);
    return launched();
  }
  return cudaSuccess;
}

}  // namespace

size_t simt_bwd_workspace_bytes(const Problem& p) {
  const int splits = bwd_splits(p);
  return splits > 1 ? size_t(splits) * size_t(p.d_out) * size_t(p.r) * sizeof(float) : 0;
}

cudaError_t simt_fwd(const Problem& p, const void* X, const void* W, void* Y, void* XS, cudaStream_t st, const void* Vt) {
  return p.bf16 ? fwd_t<__nv_bfloat16>(p, X, W, Y, XS, st, Vt) : fwd_t<float>(p, X, W, Y, XS, st, Vt);
}

cudaError_t simt_bwd(const Problem& p, const void* G, const void* W, const void* XS, void* dX, float* A, void* ws,
                     cudaStream_t st) {
  return p.bf16 ? bwd_t<__nv_bfloat16>(p, G, W, XS, dX, A, ws, st) : bwd_t<float>(p, G, W, XS, dX, A, ws, st);
}

cudaError_t simt_reconstruct(const Problem& p, const float* A, float* dW, float beta, cudaStream_t st, const void* Vt) {
  GemmArgs g{};
  g.A = A; g.a_sm = p.r; g.a_sk = 1;
  g.C = dW; g.ldc = p.d_in; g.M = p.d_out; g.N = p.d_in; g.K = p.r; g.k_per_split = p.r;
  g.beta = beta; g.sp = p.sp; g.sketch_bf16 = p.bf16;
  if (Vt) {  // dW = A V^T with V^T (r x d_in, fp32) in memory: B(k, n) = Vt[k * d_in + n]
    g.B = Vt; g.b_sk = p.d_in; g.b_sn = 1;
    return launch<float, float, float, true, false, B_STRIDED>(g, 1, st);
  }
  return launch<float, float, float, true, true, B_SKETCH_NK>(g, 1, st);
}

cudaError_t sketch_materialize(const Problem& p, void* S_out, cudaStream_t st) {
  const int64_t quads = p.d_in * (p.r / 4);
  if (quads == 0) return cudaSuccess;
  sketch_materialize_kernel<<<(unsigned)((quads + 255) / 256), 256, 0, st>>>(S_out, p.d_in, p.r, p.sp, p.bf16);
  return launched();
}

}  // namespace acx
