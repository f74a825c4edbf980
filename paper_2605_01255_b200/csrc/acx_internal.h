// Internal declarations shared by the translation units of libacx (not part of the C ABI).
#pragma once
#include <cuda_runtime.h>
#include <atomic>
#include <cstddef>
#include <cstdint>

#include "../../include/acx.h"
#include "acx_sketch.cuh"

namespace acx {

// Everything a launcher needs, derived from a validated acx_desc.
struct Problem {
  int64_t m, d_in, d_out;
  int r;
  bool bf16;
  SketchParams sp;
};

// Device-side status word values (written by kernels whose bounded waits expire).
constexpr int kDevOk = 0;
constexpr int kDevTimeout = 1;

// Counts every kernel launch the library makes (reported by acx_kernel_launches()).
inline std::atomic<unsigned long long>& kernel_launch_counter() {
  static std::atomic<unsigned long long> counter{0};
  return counter;
}
inline cudaError_t launched() {
  kernel_launch_counter().fetch_add(1, std::memory_order_relaxed);
  return cudaGetLastError();
}

// One-time set-up that holds per device (a kernel's function attributes are set for the device that is current):
// `static DeviceOnce once; if (once.needed()) { ...; once.done(); }`.  Safe to race: the set-up is idempotent.
class DeviceOnce {
  std::atomic<unsigned long long> mask_{0};
  static unsigned long long bit() {
    int dev = 0;
    cudaGetDevice(&dev);
    return 1ull << (unsigned(dev) & 63u);
  }

 public:
  bool needed() const { return (mask_.load(std::memory_order_acquire) & bit()) == 0; }
  void done() { mask_.fetch_or(bit(), std::memory_order_release); }
};

// Checks a caller's descriptor and derives the launch problem from it (defined with the C ABI).
acx_status validate(const acx_desc* d, Problem* out);
// Device address of the status word on the current device (nullptr on a CUDA error).
int* device_status_ptr();

// ---- SIMT path (fp32 I/O; any valid shape) -------------------------------------------------------
size_t simt_bwd_workspace_bytes(const Problem& p);
// Vt != nullptr in the calls below: the second factor V^T (r x d_in) is read from memory instead of generated.
cudaError_t simt_fwd(const Problem& p, const void* X, const void* W, void* Y, void* XS, cudaStream_t st, const void* Vt = nullptr);
cudaError_t simt_bwd(const Problem& p, const void* G, const void* W, const void* XS, void* dX, float* A,
                     void* ws, cudaStream_t st);
cudaError_t simt_reconstruct(const Problem& p, const float* A, float* dW, float beta, cudaStream_t st, const void* Vt = nullptr);
cudaError_t sketch_materialize(const Problem& p, void* S_out, cudaStream_t st);

// ---- tcgen05 path (bf16 I/O; any valid shape) ----------------------------------------------------
size_t sm100_bwd_workspace_bytes(const Problem& p);
// Vt != nullptr: the second factor V^T (r x d_in, bf16) is read from memory instead of generated from the seed.
// Vt == nullptr and ws != nullptr: S^T is written once into ws (sm100_fwd_workspace_bytes) by a small grid and the
// GEMM reads it from there; with neither, each CTA generates its slices of S in shared memory.
size_t sm100_fwd_workspace_bytes(const Problem& p);
cudaError_t sm100_fwd(const Problem& p, const void* X, const void* W, void* Y, void* XS, int* status, cudaStream_t st,
                      const void* Vt = nullptr, void* ws = nullptr, const void* bias = nullptr);
// db[c] = sum over the tokens of G[t][c] (bf16 in, fp32 out), two deterministic stages through ws.
size_t bias_grad_workspace_bytes(const Problem& p);
cudaError_t bias_grad(const Problem& p, const void* G, float* db, void* ws, cudaStream_t st);
// db[c] = sum over z < splits of part[z][c], in order.
cudaError_t sum_column_partials(const float* part, float* db, int64_t d_out, int splits, cudaStream_t st);
constexpr int kMaxFactorSplits = 128;  // upper bound of the token ranges of the gradient factor (sizes the partial column sums)
cudaError_t sm100_dx(const Problem& p, const void* G, const void* W, void* dX, int* status, cudaStream_t st);
size_t sm100_reconstruct_workspace_bytes(const Problem& p);
cudaError_t sm100_reconstruct(const Problem& p, const float* A, float* dW, float beta, void* ws, int* status, cudaStream_t st,
                              const void* Vt = nullptr);
cudaError_t sm100_reconstruct_adamw(const Problem& p, const float* A, float* W, float* m, float* v, void* W_lp, float lr, float beta1,
                                    float beta2, float eps, float weight_decay, int step, void* ws, int* status, cudaStream_t st);
cudaError_t sm100_lowrank_adamw(const Problem& p, const float* A, float* mA, float* vA, const void* Vt, float* W, float lr,
                                float beta1, float beta2, float eps, float weight_decay, int step, void* ws, int* status,
                                cudaStream_t st);
// Second factor of the randomized-SVD compressor: Vt = (U^T U)^-1 U^T X (r x d_in, bf16).
size_t sm100_rsvd_workspace_bytes(const Problem& p);
cudaError_t sm100_rsvd_factor(const Problem& p, const void* X, const void* U, void* Vt, void* ws, int* status, cudaStream_t st);
size_t sm100_factor_scratch_bytes(const Problem& p);  // split-K partials through global memory (no cluster)
// db_part != nullptr: the kernel also adds up G's columns over each token range into db_part[range][d_out] (room for
// kMaxFactorSplits ranges) and *db_splits receives the number of ranges.
cudaError_t sm100_factor(const Problem& p, const void* G, const void* XS, float* A, void* ws, int* status, cudaStream_t st,
                         bool allow_cluster, float* db_part = nullptr, int* db_splits = nullptr, bool after_dx = false);

// Test/debug: overrides the tile-shape cost models of the forward and dX (0 = off, 1..4 = a GEMM mode).
void sm100_force_gemm_mode(int mode);

}  // namespace acx
