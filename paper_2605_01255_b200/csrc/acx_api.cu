// The C ABI of libacx (declared in include/acx.h): argument validation and dispatch to the kernels.
#include <cmath>
#include <cstring>

#include "acx_internal.h"
#include "acx_umma.cuh"

namespace acx {
namespace {

// Status word written by kernels whose bounded waits give up.  Lives in the library image.
__device__ int g_device_status = 0;

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

acx_status from_cuda(cudaError_t e) { return e == cudaSuccess ? ACX_OK : ACX_ERR_CUDA; }

}  // namespace

acx_status validate(const acx_desc* d, Problem* out) {
  if (!d) return ACX_ERR_INVALID_ARG;
  if (d->struct_size != sizeof(acx_desc)) return ACX_ERR_INVALID_ARG;
  if (d->sketch_kind != 0) return ACX_ERR_INVALID_ARG;
  if (d->io_dtype != ACX_F32 && d->io_dtype != ACX_BF16) return ACX_ERR_INVALID_ARG;
  if (d->tokens < 0 || d->tokens > (int64_t(1) << 31) - 1) return ACX_ERR_UNSUPPORTED_SHAPE;
  if (d->d_in < 8 || d->d_out < 8 || (d->d_in % 8) || (d->d_out % 8)) return ACX_ERR_UNSUPPORTED_SHAPE;
  if (d->d_in > (int64_t(1) << 24) || d->d_out > (int64_t(1) << 24)) return ACX_ERR_UNSUPPORTED_SHAPE;
  if (d->r < 16 || d->r > 256 || (d->r % 16) || d->r > d->d_in) return ACX_ERR_UNSUPPORTED_SHAPE;
  if (d->io_dtype == ACX_F32) {  // the fp32 kernels number their 64 x 64 output tiles along one grid dimension
    const int64_t widest = d->d_in > d->d_out ? d->d_in : d->d_out;
    if (((d->tokens + 63) / 64) * ((widest + 63) / 64) > 0x7FFFFFFFll) return ACX_ERR_UNSUPPORTED_SHAPE;
  }
  out->m = d->tokens;
  out->d_in = d->d_in;
  out->d_out = d->d_out;
  out->r = d->r;
  out->bf16 = d->io_dtype == ACX_BF16;
  out->sp.key0 = uint32_t(d->seed & 0xFFFFFFFFull);
  out->sp.key1 = uint32_t(d->seed >> 32);
  out->sp.kind = d->sketch_kind;
  out->sp.scale = float(1.0 / std::sqrt(double(d->r)));
  fill_round_keys(out->sp);
  return ACX_OK;
}

// Device address of the status word on the current device (looked up once per device).
int* device_status_ptr() {
  static int* cache[64] = {nullptr};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  if (!cache[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_device_status) != cudaSuccess) return nullptr;
    cache[dev] = static_cast<int*>(ptr);
  }
  return cache[dev];
}

namespace {

// One warp waits, with the library's bounded wait, on a barrier that nobody arrives at; when the limit runs
// out it reports through the status word like the production kernels do, and returns.
__global__ void expired_wait_kernel(int* status, unsigned long long limit_ns) {
  __shared__ __align__(8) unsigned long long bar;
  __shared__ int abort_flag;
  const uint32_t bar_addr = ptx::smem_u32(&bar);
  if (threadIdx.x == 0) {
    abort_flag = 0;
    ptx::mbar_init(bar_addr, 1);
    ptx::fence_barrier_init();
  }
  __syncwarp();
  if (!__all_sync(0xFFFFFFFFu, ptx::mbar_wait(bar_addr, 0u, &abort_flag, limit_ns)) && threadIdx.x == 0)
    atomicExch(status, kDevTimeout);
}

size_t bwd_workspace_bytes(const Problem& p) { return p.bf16 ? sm100_bwd_workspace_bytes(p) : simt_bwd_workspace_bytes(p); }
// acx_linear_bwd_bias: the backward's own scratch, then the partial column sums (256-byte aligned)
size_t bwd_bias_partials_offset(const Problem& p) { return (bwd_workspace_bytes(p) + 255) & ~size_t(255); }

}  // namespace
}  // namespace acx

using namespace acx;

extern "C" {

size_t acx_workspace_bytes(const acx_desc* desc, int op) {
  Problem p;
  if (validate(desc, &p) != ACX_OK) return 0;
  switch (op) {
    case ACX_OP_FWD: return p.bf16 ? sm100_fwd_workspace_bytes(p) : 0;
    case ACX_OP_BWD: return bwd_workspace_bytes(p);
    case ACX_OP_RECONSTRUCT: return p.bf16 ? sm100_reconstruct_workspace_bytes(p) : 0;
    case ACX_OP_BWD_BUILTIN_SCRATCH: return p.bf16 ? sm100_factor_scratch_bytes(p) : 0;
    case ACX_OP_RSVD: return p.bf16 ? sm100_rsvd_workspace_bytes(p) : 0;
    case ACX_OP_BIAS_GRAD: return (p.bf16 && p.m > 0) ? bias_grad_workspace_bytes(p) : 0;
    case ACX_OP_BWD_BIAS: return p.bf16 ? bwd_bias_partials_offset(p) + size_t(kMaxFactorSplits) * size_t(p.d_out) * 4 : 0;
    default: return 0;
  }
}

namespace {
acx_status linear_fwd_impl(const acx_desc* desc, const void* X, const void* W, const void* Vt, bool v_given, void* Y, void* XS,
                           void* cuda_stream, void* ws = nullptr, size_t ws_bytes = 0, const void* bias = nullptr);
}

acx_status acx_linear_fwd_bias(const acx_desc* desc, const void* X, const void* W, const void* bias, void* Y, void* XS, void* ws,
                               size_t ws_bytes, void* cuda_stream) {
  if (!bias) return ACX_ERR_INVALID_ARG;
  if (desc && desc->io_dtype != ACX_BF16) return ACX_ERR_INVALID_ARG;
  return linear_fwd_impl(desc, X, W, nullptr, false, Y, XS, cuda_stream, ws, ws_bytes, bias);
}

acx_status acx_linear_bwd_bias(const acx_desc* desc, const void* G_out, const void* W, const void* XS, void* dX, float* dW_A,
                               float* db, void* ws, size_t ws_bytes, void* cuda_stream) {
  Problem p;
  acx_status s = validate(desc, &p);
  if (s != ACX_OK) return s;
  if (!p.bf16 || !dW_A || !db) return ACX_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (p.m == 0) {
    cudaError_t e = cudaMemsetAsync(dW_A, 0, size_t(p.d_out) * size_t(p.r) * sizeof(float), st);
    if (e == cudaSuccess) e = cudaMemsetAsync(db, 0, size_t(p.d_out) * sizeof(float), st);
    return from_cuda(e);
  }
  if (!G_out || !XS || (dX && !W)) return ACX_ERR_INVALID_ARG;
  if (!aligned16(G_out) || !aligned16(W) || !aligned16(XS) || !aligned16(dX) || !aligned16(dW_A) || !aligned16(db) || !aligned16(ws))
    return ACX_ERR_ALIGNMENT;
  const size_t off = bwd_bias_partials_offset(p);
  if (!ws || ws_bytes < off + size_t(kMaxFactorSplits) * size_t(p.d_out) * 4) return ACX_ERR_WORKSPACE;
  int* status = device_status_ptr();
  if (!status) return ACX_ERR_CUDA;
  if (dX) {
    cudaError_t e = sm100_dx(p, G_out, W, dX, status, st);
    if (e != cudaSuccess) return ACX_ERR_CUDA;
  }
  float* part = reinterpret_cast<float*>(static_cast<uint8_t*>(ws) + off);
  int splits = 1;
  cudaError_t e = sm100_factor(p, G_out, XS, dW_A, ws, status, st, /*allow_cluster=*/true, part, &splits, /*after_dx=*/dX != nullptr);
  if (e != cudaSuccess) return ACX_ERR_CUDA;
  return from_cuda(sum_column_partials(part, db, p.d_out, splits, st));
}

acx_status acx_bias_grad(const acx_desc* desc, const void* G_out, float* db, void* ws, size_t ws_bytes, void* cuda_stream) {
  Problem p;
  acx_status s = validate(desc, &p);
  if (s != ACX_OK) return s;
  if (!p.bf16 || !db) return ACX_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (p.m == 0) return from_cuda(cudaMemsetAsync(db, 0, size_t(p.d_out) * sizeof(float), st));
  if (!G_out) return ACX_ERR_INVALID_ARG;
  if (!aligned16(G_out) || !aligned16(db) || !aligned16(ws)) return ACX_ERR_ALIGNMENT;
  if (!ws || ws_bytes < bias_grad_workspace_bytes(p)) return ACX_ERR_WORKSPACE;
  return from_cuda(bias_grad(p, G_out, db, ws, st));
}

acx_status acx_linear_fwd(const acx_desc* desc, const void* X, const void* W, void* Y, void* XS, void* ws,
                          size_t ws_bytes, void* cuda_stream) {
  return linear_fwd_impl(desc, X, W, nullptr, false, Y, XS, cuda_stream, ws, ws_bytes);
}

acx_status acx_linear_fwd_v(const acx_desc* desc, const void* X, const void* W, const void* Vt, void* Y, void* XV, void* ws,
                            size_t ws_bytes, void* cuda_stream) {
  (void)ws; (void)ws_bytes;
  if (!Vt || !XV) return ACX_ERR_INVALID_ARG;
  return linear_fwd_impl(desc, X, W, Vt, true, Y, XV, cuda_stream);
}

namespace {
acx_status linear_fwd_impl(const acx_desc* desc, const void* X, const void* W, const void* Vt, bool v_given, void* Y, void* XS,
                           void* cuda_stream, void* ws, size_t ws_bytes, const void* bias) {
  Problem p;
  acx_status s = validate(desc, &p);
  if (s != ACX_OK) return s;
  if (p.m == 0) return ACX_OK;  // nothing to compute; token-sized buffers may be empty
  if (!X || !W || !Y) return ACX_ERR_INVALID_ARG;  // XS may be NULL: another linear on the same input stores the factor
  if (!aligned16(X) || !aligned16(W) || !aligned16(Y) || !aligned16(XS) || !aligned16(Vt) || !aligned16(bias)) return ACX_ERR_ALIGNMENT;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (!p.bf16) return from_cuda(simt_fwd(p, X, W, Y, XS, st, v_given ? Vt : nullptr));
  if (ws && XS && (ws_bytes < sm100_fwd_workspace_bytes(p))) return ACX_ERR_WORKSPACE;
  if (!aligned16(ws)) return ACX_ERR_ALIGNMENT;
  int* status = device_status_ptr();
  if (!status) return ACX_ERR_CUDA;
  return from_cuda(sm100_fwd(p, X, W, Y, XS, status, st, v_given ? Vt : nullptr, v_given ? nullptr : ws, bias));
}
}  // namespace

acx_status acx_linear_bwd(const acx_desc* desc, const void* G_out, const void* W, const void* XS, void* dX,
                          float* dW_A, void* ws, size_t ws_bytes, void* cuda_stream) {
  Problem p;
  acx_status s = validate(desc, &p);
  if (s != ACX_OK) return s;
  if (p.m == 0) {  // an empty batch contributes a zero gradient factor
    if (!dW_A) return ACX_OK;
    if (!aligned16(dW_A)) return ACX_ERR_ALIGNMENT;
    return from_cuda(cudaMemsetAsync(dW_A, 0, sizeof(float) * size_t(p.d_out) * size_t(p.r),
                                     static_cast<cudaStream_t>(cuda_stream)));
  }
  if (!G_out || !W) return ACX_ERR_INVALID_ARG;
  if (dW_A && !XS) return ACX_ERR_INVALID_ARG;
  if (!aligned16(G_out) || !aligned16(W) || !aligned16(XS) || !aligned16(dX) || !aligned16(dW_A) || !aligned16(ws))
    return ACX_ERR_ALIGNMENT;
  if (dW_A) {
    const size_t need = bwd_workspace_bytes(p);
    if (need > 0 && (!ws || ws_bytes < need)) return ACX_ERR_WORKSPACE;
  }
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (!p.bf16) return from_cuda(simt_bwd(p, G_out, W, XS, dX, dW_A, ws, st));
  int* status = device_status_ptr();
  if (!status) return ACX_ERR_CUDA;
  if (dX) {
    cudaError_t e = sm100_dx(p, G_out, W, dX, status, st);
    if (e != cudaSuccess) return ACX_ERR_CUDA;
  }
  if (dW_A) return from_cuda(sm100_factor(p, G_out, XS, dW_A, ws, status, st, /*allow_cluster=*/true, nullptr, nullptr, /*after_dx=*/dX != nullptr));
  return ACX_OK;
}

namespace {
acx_status reconstruct_impl(const acx_desc* desc, const float* dW_A, const void* Vt, bool v_given, float* dW, float beta, void* ws,
                            size_t ws_bytes, void* cuda_stream);
}

acx_status acx_reconstruct(const acx_desc* desc, const float* dW_A, float* dW, float beta, void* ws, size_t ws_bytes,
                           void* cuda_stream) {
  return reconstruct_impl(desc, dW_A, nullptr, false, dW, beta, ws, ws_bytes, cuda_stream);
}

acx_status acx_reconstruct_v(const acx_desc* desc, const float* dW_A, const void* Vt, float* dW, float beta, void* ws,
                             size_t ws_bytes, void* cuda_stream) {
  if (!Vt) return ACX_ERR_INVALID_ARG;
  return reconstruct_impl(desc, dW_A, Vt, true, dW, beta, ws, ws_bytes, cuda_stream);
}

namespace {
acx_status reconstruct_impl(const acx_desc* desc, const float* dW_A, const void* Vt, bool v_given, float* dW, float beta, void* ws,
                            size_t ws_bytes, void* cuda_stream) {
  Problem p;
  acx_status s = validate(desc, &p);
  if (s != ACX_OK) return s;
  if (!dW_A || !dW) return ACX_ERR_INVALID_ARG;
  if (!aligned16(dW_A) || !aligned16(dW) || !aligned16(ws) || !aligned16(Vt)) return ACX_ERR_ALIGNMENT;
  if (!(beta == beta)) return ACX_ERR_INVALID_ARG;
  const size_t need = p.bf16 ? sm100_reconstruct_workspace_bytes(p) : 0;
  if (need > 0 && (!ws || ws_bytes < need)) return ACX_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (!p.bf16) return from_cuda(simt_reconstruct(p, dW_A, dW, beta, st, v_given ? Vt : nullptr));
  int* status = device_status_ptr();
  if (!status) return ACX_ERR_CUDA;
  return from_cuda(sm100_reconstruct(p, dW_A, dW, beta, ws, status, st, v_given ? Vt : nullptr));
}
}  // namespace

acx_status acx_reconstruct_adamw(const acx_desc* desc, const float* dW_A, float* W, float* m, float* v, void* W_lp,
                                 const acx_adamw_params* hp, void* ws, size_t ws_bytes, void* cuda_stream) {
  Problem p;
  acx_status s = validate(desc, &p);
  if (s != ACX_OK) return s;
  if (!p.bf16 || !dW_A || !W || !m || !v || !hp) return ACX_ERR_INVALID_ARG;
  if (hp->struct_size != sizeof(acx_adamw_params) || hp->step < 1) return ACX_ERR_INVALID_ARG;
  const float hv[5] = {hp->lr, hp->beta1, hp->beta2, hp->eps, hp->weight_decay};
  for (float x : hv)
    if (!(x == x)) return ACX_ERR_INVALID_ARG;
  if (hp->beta1 < 0.f || hp->beta1 >= 1.f || hp->beta2 < 0.f || hp->beta2 >= 1.f || hp->eps < 0.f) return ACX_ERR_INVALID_ARG;
  if (!aligned16(dW_A) || !aligned16(W) || !aligned16(m) || !aligned16(v) || !aligned16(W_lp) || !aligned16(ws))
    return ACX_ERR_ALIGNMENT;
  const size_t need = sm100_reconstruct_workspace_bytes(p);
  if (!ws || ws_bytes < need) return ACX_ERR_WORKSPACE;
  int* status = device_status_ptr();
  if (!status) return ACX_ERR_CUDA;
  return from_cuda(sm100_reconstruct_adamw(p, dW_A, W, m, v, W_lp, hp->lr, hp->beta1, hp->beta2, hp->eps, hp->weight_decay,
                                           hp->step, ws, status, static_cast<cudaStream_t>(cuda_stream)));
}

acx_status acx_lowrank_adamw(const acx_desc* desc, const float* dW_A, float* m_A, float* v_A, const void* Vt, float* W,
                             const acx_adamw_params* hp, void* ws, size_t ws_bytes, void* cuda_stream) {
  Problem p;
  acx_status s = validate(desc, &p);
  if (s != ACX_OK) return s;
  if (!p.bf16 || !dW_A || !W || !m_A || !v_A || !hp) return ACX_ERR_INVALID_ARG;
  if (hp->struct_size != sizeof(acx_adamw_params) || hp->step < 1) return ACX_ERR_INVALID_ARG;
  const float hv[5] = {hp->lr, hp->beta1, hp->beta2, hp->eps, hp->weight_decay};
  for (float x : hv)
    if (!(x == x)) return ACX_ERR_INVALID_ARG;
  if (hp->beta1 < 0.f || hp->beta1 >= 1.f || hp->beta2 < 0.f || hp->beta2 >= 1.f || hp->eps < 0.f) return ACX_ERR_INVALID_ARG;
  if (!aligned16(dW_A) || !aligned16(W) || !aligned16(m_A) || !aligned16(v_A) || !aligned16(Vt) || !aligned16(ws))
    return ACX_ERR_ALIGNMENT;
  if (!ws || ws_bytes < sm100_reconstruct_workspace_bytes(p)) return ACX_ERR_WORKSPACE;
  int* status = device_status_ptr();
  if (!status) return ACX_ERR_CUDA;
  return from_cuda(sm100_lowrank_adamw(p, dW_A, m_A, v_A, Vt, W, hp->lr, hp->beta1, hp->beta2, hp->eps, hp->weight_decay,
                                       hp->step, ws, status, static_cast<cudaStream_t>(cuda_stream)));
}

acx_status acx_rsvd_factor(const acx_desc* desc, const void* X, const void* U, void* Vt, void* ws, size_t ws_bytes,
                           void* cuda_stream) {
  Problem p;
  acx_status s = validate(desc, &p);
  if (s != ACX_OK) return s;
  if (!p.bf16 || !X || !U || !Vt) return ACX_ERR_INVALID_ARG;
  if (!aligned16(X) || !aligned16(U) || !aligned16(Vt) || !aligned16(ws)) return ACX_ERR_ALIGNMENT;
  if (p.m == 0) return ACX_ERR_INVALID_ARG;  // no tokens, no range to project on
  if (!ws || ws_bytes < sm100_rsvd_workspace_bytes(p)) return ACX_ERR_WORKSPACE;
  int* status = device_status_ptr();
  if (!status) return ACX_ERR_CUDA;
  return from_cuda(sm100_rsvd_factor(p, X, U, Vt, ws, status, static_cast<cudaStream_t>(cuda_stream)));
}

acx_status acx_sketch_materialize(const acx_desc* desc, void* S_out, void* cuda_stream) {
  Problem p;
  acx_status s = validate(desc, &p);
  if (s != ACX_OK) return s;
  if (!S_out) return ACX_ERR_INVALID_ARG;
  if (!aligned16(S_out)) return ACX_ERR_ALIGNMENT;
  return from_cuda(sketch_materialize(p, S_out, static_cast<cudaStream_t>(cuda_stream)));
}

acx_status acx_debug_expired_wait(uint64_t limit_ns, void* cuda_stream) {
  if (limit_ns == 0 || limit_ns > 1000000000ull) return ACX_ERR_INVALID_ARG;  // at most one second
  int* status = device_status_ptr();
  if (!status) return ACX_ERR_CUDA;
  expired_wait_kernel<<<1, 32, 0, static_cast<cudaStream_t>(cuda_stream)>>>(status, limit_ns);
  return from_cuda(launched());
}

acx_status acx_debug_force_gemm_mode(int mode) {
  if (mode < 0 || mode > 4) return ACX_ERR_INVALID_ARG;
  sm100_force_gemm_mode(mode);
  return ACX_OK;
}

acx_status acx_last_device_status(void* cuda_stream) {
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (cudaStreamSynchronize(st) != cudaSuccess) return ACX_ERR_CUDA;
  int v = 0;
  if (cudaMemcpyFromSymbol(&v, g_device_status, sizeof(int)) != cudaSuccess) return ACX_ERR_CUDA;
  if (v != kDevOk) {
    const int zero = 0;
    if (cudaMemcpyToSymbol(g_device_status, &zero, sizeof(int)) != cudaSuccess) return ACX_ERR_CUDA;
    return ACX_ERR_TIMEOUT;
  }
  return ACX_OK;
}

const char* acx_status_string(int status) {
  switch (status) {
    case ACX_OK: return "ACX_OK";
    case ACX_ERR_INVALID_ARG: return "ACX_ERR_INVALID_ARG: null pointer, wrong struct_size or unknown enum value";
    case ACX_ERR_UNSUPPORTED_SHAPE:
      return "ACX_ERR_UNSUPPORTED_SHAPE: need d_in, d_out multiples of 8 (>= 8), r a multiple of 16 in [16, 256], r <= d_in";
    case ACX_ERR_ALIGNMENT: return "ACX_ERR_ALIGNMENT: every device pointer must be 16-byte aligned";
    case ACX_ERR_WORKSPACE: return "ACX_ERR_WORKSPACE: workspace missing or smaller than acx_workspace_bytes()";
    case ACX_ERR_CUDA: return "ACX_ERR_CUDA: a CUDA runtime call or kernel launch failed";
    case ACX_ERR_TIMEOUT: return "ACX_ERR_TIMEOUT: a bounded device-side wait expired; outputs are undefined";
    case ACX_ERR_SCRATCH_LIMIT:
      return "ACX_ERR_SCRATCH_LIMIT: this shape needs more split-K scratch than the 16 MiB built into the library; "
             "use acx_linear_bwd with a workspace of acx_workspace_bytes()";
    default: return "unknown acx_status";
  }
}

int acx_version(void) { return ACX_VERSION; }

unsigned long long acx_kernel_launches(void) { return acx::kernel_launch_counter().load(); }

}  // extern "C"
