// Reconstruct dW = beta * dW + A V^T (Section 4, optimizer strategy (i)) on the tcgen05 tensor cores, with
// V = S(seed) or a second factor given in memory.
//
// The contraction length is only r, so the call is bound by the write of dW (d_out x d_in fp32).  Two kernels:
//   1. reconstruct_prepass_kernel writes A (fp32) once as two bf16 terms, A = hi + lo + O(2^-17 |A|), into the
//      caller's workspace (2 x d_out x r bf16) and, for the seeded sketch, S^T (r x d_in bf16) behind them, each
//      element of S generated exactly once.
//   2. reconstruct_umma_kernel: a CTA owns `nw` consecutive columns of dW and a group of 128-row tiles of A.
//      It fetches its slice of V^T ONCE by TMA (64-column chunks, consumed as an N-major B operand), then
//      streams the hi/lo tiles of its group in by TMA; D = hi V^T + lo V^T accumulates in fp32 in tensor
//      memory; the epilogue adds beta * dW and writes 32 x 32 boxes through shared memory with bulk tensor
//      (TMA) stores, so that HBM sees whole lines.
// The second kernel is launched with programmatic stream serialization: its prologue overlaps the first and
// it only waits for it (griddepcontrol.wait) before its first read of the workspace.
// The slice width and the number of row groups are chosen on the host so that the CTAs fill the machine once.
// Roles: warps 0-7 epilogue (TMEM lane quarter = warp % 4, the two halves interleave 32-column chunks),
// warp 8 TMA producer, warp 9 MMA issuer.  Two accumulators and four A stages (64 contraction elements of both
// terms each) overlap loads, MMAs and stores.  Every wait is bounded.
#include <algorithm>
#include <cmath>

#include "acx_internal.h"
#include "acx_tmap.h"
#include "acx_umma.cuh"

namespace acx {
namespace {

constexpr int kRM = 128;              // rows of A (and dW) per tile = TMEM lanes
constexpr int kKStep = 64;            // contraction elements staged per step: one 64-wide swizzle chunk of each term
constexpr int kMaxSliceElems = 16384; // nw * r <= this (32 KiB of bf16)
constexpr int kSBytes = kMaxSliceElems * 2;
constexpr int kChunkBytes = kRM * 64 * 2;             // one 64-wide K chunk of one term: 16 KiB
constexpr int kAHalfBytes = kRM * kKStep * 2;         // one bf16 term of an A step: 16 KiB
constexpr int kEpiWarps = 8, kTmaWarp = 8, kMmaWarp = 9, kRecThreads = 512;
constexpr int kOutBoxBytes = 32 * 32 * 4;             // one TMA box: 32 rows x 32 fp32 columns

// Shared-memory plan.  Plain reconstruct: four A stages of 32 KiB (64 contraction elements of both terms: a stage is
// refilled as soon as its eight MMAs are done, so the loads run up to two 128-row tiles ahead at r = 128), two store
// boxes per epilogue warp.  With the fused AdamW update an epilogue warp stages the m, v and W boxes of its chunk
// (loaded by TMA, updated in place, stored by TMA) and a bf16 box for the low-precision copy of W: 16 KiB per warp,
// paid for with two A stages.
template <bool ADAMW>
struct RecCfg {
  static constexpr int kAStages = ADAMW ? 2 : 4;
  static constexpr int kWarpOutBytes = ADAMW ? 4 * kOutBoxBytes : 2 * kOutBoxBytes;
  static constexpr int kOutOffset = kSBytes + kAStages * 2 * kAHalfBytes;
  static constexpr int kBarOffset = kOutOffset + kEpiWarps * kWarpOutBytes;
  static constexpr int kSmemBytes = kBarOffset + 256 + 1024;
};

// AdamW constants derived on the host (double precision, rounded once).
struct AdamConsts {
  float beta1, one_minus_beta1, beta2, one_minus_beta2;
  float inv_bias1, inv_bias2;  // 1 / (1 - beta^t)
  float eps, lr, weight_decay;
  int has_wlp;                 // also write W rounded to bf16
};

struct RecParams {
  float* dW;        // d_out x d_in
  int d_out, d_in, r;
  int nw;                // columns of dW per CTA slice (multiple of 32, nw * r <= kMaxSliceElems)
  int n_slices;          // ceil(d_in / nw)
  int tiles_per_group;   // 128-row tiles of A handled by one CTA
  int m_tiles;           // ceil(d_out / 128)
  float beta;
  SketchParams sp;
  int* status;
  AdamConsts adam;       // fused-update kernel only
  int v_from_prepass;    // V^T is the S^T that the grid launched just before this one writes
};

__device__ __forceinline__ uint2 pack_bf16x4(float a, float b, float c, float d) {
  __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
  uint2 v;
  v.x = *reinterpret_cast<uint32_t*>(&lo);
  v.y = *reinterpret_cast<uint32_t*>(&hi);
  return v;
}

// One component of the factor-space Adam step (Section 4, optimizer strategy (ii)): updates the moments of the
// gradient factor and returns -lr times the normalised step, the factor that is then projected back through V^T.
__device__ __forceinline__ float lowrank_adam(float a, float& m, float& v, const AdamConsts& c) {
  m = fmaf(c.beta1, m, c.one_minus_beta1 * a);
  v = fmaf(c.beta2, v, c.one_minus_beta2 * a * a);
  return -c.lr * ((m * c.inv_bias1) / (sqrtf(v * c.inv_bias2) + c.eps));
}

// Blocks [0, split_blocks): A (fp32, n4 float4) -> hi = bf16(A), lo = bf16(A - hi), both row-major like A; with
// factor-space moments (mA != nullptr) A is first replaced by the Adam step formed from it and the moments.
// Blocks from split_blocks on (seeded sketch only): S^T in bf16, r x d_in.
__global__ void __launch_bounds__(256) reconstruct_prepass_kernel(const float4* __restrict__ A, uint2* __restrict__ hi,
                                                                  uint2* __restrict__ lo, int64_t n4, unsigned split_blocks,
                                                                  __nv_bfloat16* __restrict__ St, int64_t d_in, int r,
                                                                  SketchParams sp, float4* __restrict__ mA,
                                                                  float4* __restrict__ vA, AdamConsts adam) {
  // let the dependent grid start right away: it only needs this grid's output after its own prologue
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (blockIdx.x >= split_blocks) {
    const uint32_t half = uint32_t(d_in >> 1);
    const int64_t idx = int64_t(blockIdx.x - split_blocks) * blockDim.x + threadIdx.x;
    if (idx < int64_t(half) * (r >> 2)) sketch_transposed_store(sp, St, d_in, uint32_t(idx % half), uint32_t(idx / half));
    return;
  }
  const int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i >= n4) return;
  float4 a = __ldg(A + i);
  if (mA) {
    float4 m = mA[i], v = vA[i];
    a.x = lowrank_adam(a.x, m.x, v.x, adam);
    a.y = lowrank_adam(a.y, m.y, v.y, adam);
    a.z = lowrank_adam(a.z, m.z, v.z, adam);
    a.w = lowrank_adam(a.w, m.w, v.w, adam);
    mA[i] = m;
    vA[i] = v;
  }
  const uint2 h = pack_bf16x4(a.x, a.y, a.z, a.w);
  const float hx = __uint_as_float(h.x << 16), hy = __uint_as_float(h.x & 0xFFFF0000u), hz = __uint_as_float(h.y << 16),
              hw = __uint_as_float(h.y & 0xFFFF0000u);
  hi[i] = h;
  lo[i] = pack_bf16x4(a.x - hx, a.y - hy, a.z - hz, a.w - hw);
}

// ADAMW = false: tmap_dw is the store map of dW, the other three output maps are unused.
// ADAMW = true: tmap_dw is the load/store map of the fp32 master weights W, tmap_m / tmap_v those of the moments,
// tmap_wlp the store map of the bf16 copy of W; dW itself is never written.
template <bool ADAMW>
__global__ void __launch_bounds__(kRecThreads, 1)
    reconstruct_umma_kernel(const __grid_constant__ CUtensorMap tmap_hi, const __grid_constant__ CUtensorMap tmap_lo,
                            const __grid_constant__ CUtensorMap tmap_dw, const __grid_constant__ CUtensorMap tmap_m,
                            const __grid_constant__ CUtensorMap tmap_v, const __grid_constant__ CUtensorMap tmap_wlp,
                            const __grid_constant__ CUtensorMap tmap_vt, const RecParams p) {
  using RC = RecCfg<ADAMW>;
  constexpr int kAStages = RC::kAStages, kOutOffset = RC::kOutOffset, kBarOffset = RC::kBarOffset;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - ptx::smem_u32(smem_raw));
  const uint32_t s_addr = smem_base, a_addr = smem_base + kSBytes;  // A stages: each the hi term, then the lo term
  const uint32_t bar_base = smem_base + kBarOffset;
  // barriers: tfull[2], tempty[2], afree[kAStages], afull[kAStages], one load barrier per epilogue warp; then the
  // TMEM pointer and the abort flag
  auto tfull_bar = [&](int a) { return bar_base + 8u * a; };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 + a); };
  auto afree_bar = [&](int s) { return bar_base + 8u * (4 + s); };
  auto afull_bar = [&](int s) { return bar_base + 8u * (4 + kAStages + s); };
  auto load_bar = [&](int w) { return bar_base + 8u * (4 + 2 * kAStages + w); };
  const uint32_t slice_bar = bar_base + 8u * (4 + 2 * kAStages + kEpiWarps);  // the slice of a given V^T has landed
  constexpr int kSlot = 8 * (4 + 2 * kAStages + kEpiWarps + 1);
  const uint32_t tmem_slot = bar_base + kSlot;
  volatile uint32_t* tmem_slot_gen = reinterpret_cast<volatile uint32_t*>(smem_gen + kBarOffset + kSlot);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_gen + kBarOffset + kSlot + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int slice = blockIdx.x % p.n_slices, group = blockIdx.x / p.n_slices;
  const int n0 = slice * p.nw;
  const int nw = min(p.nw, ((p.d_in - n0) + 15) & ~15);  // UMMA N of this slice (multiple of 16)
  const int tile0 = group * p.tiles_per_group;
  const int tile1 = min(p.m_tiles, tile0 + p.tiles_per_group);
  const int k_steps = (p.r + kKStep - 1) / kKStep;

  if (threadIdx.x == 0) {
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(tfull_bar(a), 1);
      ptx::mbar_init(tempty_bar(a), kEpiWarps);
    }
    for (int st = 0; st < kAStages; ++st) {
      ptx::mbar_init(afree_bar(st), 1);
      ptx::mbar_init(afull_bar(st), 1);
    }
    for (int w = 0; w < kEpiWarps; ++w) ptx::mbar_init(load_bar(w), 1);
    ptx::mbar_init(slice_bar, 1);
    *abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::prefetch_tensormap(&tmap_hi);
    ptx::prefetch_tensormap(&tmap_lo);
    ptx::prefetch_tensormap(&tmap_dw);
    if (ADAMW) {
      ptx::prefetch_tensormap(&tmap_m);
      ptx::prefetch_tensormap(&tmap_v);
      ptx::prefetch_tensormap(&tmap_wlp);
    }
  }
  if (warp == kMmaWarp) {
    ptx::tmem_alloc(tmem_slot, 512);
    ptx::tmem_relinquish_alloc_permit();
  }

  // ---- the slice of the second factor: columns n0 .. n0+nw of V^T (r x d_in), i.e. B(n, k) = V^T[k][n0 + n],
  // N-major in 64-column chunks of r rows of 128 bytes; boxes of 64 columns x 16 rows (columns past d_in read zero)
  if (threadIdx.x == 0) {
    const int n_chunks = (nw + 63) >> 6;
    if (p.v_from_prepass) asm volatile("griddepcontrol.wait;" ::: "memory");
    ptx::mbar_arrive_expect_tx(slice_bar, uint32_t(n_chunks * p.r * 128));
    for (int c = 0; c < n_chunks; ++c)
      for (int j = 0; j < p.r; j += 16)
        ptx::tma_load_2d(s_addr + uint32_t(c * p.r + j) * 128u, &tmap_vt, slice_bar, n0 + 64 * c, j);
  }
  __syncthreads();  // the barrier was initialised and armed before anybody polls it
  const bool slice_ok = ptx::mbar_wait(slice_bar, 0u, abort_flag);
  ptx::tcgen05_fence_before_sync();
  __syncthreads();
  ptx::tcgen05_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot_gen;

  auto give_up = [&]() {
    *abort_flag = 1;
    atomicExch(p.status, kDevTimeout);
  };
  if (!slice_ok) give_up();  // every role below sees the abort flag at its first wait

  if (warp == kTmaWarp) {
    // ------------------------------------------------------------------ TMA producer (one thread)
    if (lane == 0) {
      // the hi/lo terms are written by the grid launched just before this one
      asm volatile("griddepcontrol.wait;" ::: "memory");
      uint32_t step = 0;
      bool ok = true;
      for (int tile = tile0; ok && tile < tile1; ++tile) {
        for (int ks = 0; ks < k_steps; ++ks, ++step) {
          const int k0 = ks * kKStep, kw = min(kKStep, p.r - k0);
          const int stage = step % kAStages;
          const uint32_t round = step / kAStages;
          if (!ptx::mbar_wait(afree_bar(stage), (round & 1u) ^ 1u, abort_flag)) { give_up(); ok = false; break; }
          const int chunks = (kw + 63) >> 6;
          ptx::mbar_arrive_expect_tx(afull_bar(stage), uint32_t(2 * chunks * kChunkBytes));
          const uint32_t dst = a_addr + stage * (2 * kAHalfBytes);
          for (int c = 0; c < chunks; ++c) {
            ptx::tma_load_2d(dst + c * kChunkBytes, &tmap_hi, afull_bar(stage), k0 + 64 * c, tile * kRM);
            ptx::tma_load_2d(dst + kAHalfBytes + c * kChunkBytes, &tmap_lo, afull_bar(stage), k0 + 64 * c, tile * kRM);
          }
        }
      }
      if (!ok) {
        // wait (bounded) for the copies still in flight before the CTA leaves: the last armed round of each stage
        for (int s = 0; s < kAStages && uint32_t(s) < step; ++s) {
          const uint32_t last = step - 1 - ((step - 1 - s) % kAStages);  // last step issued on stage s
          const uint64_t t0 = ptx::globaltimer_ns();
          while (!ptx::mbar_try_wait(afull_bar(s), (last / kAStages) & 1u) && ptx::globaltimer_ns() - t0 < ptx::kWaitLimitNs) {}
        }
      }
    }
  } else if (warp == kMmaWarp) {
    // ------------------------------------------------------------------ MMA issue (one thread)
    if (lane == 0) {
      const uint32_t idesc = ptx::make_idesc_bf16(kRM, nw, false, true);
      uint32_t step = 0;
      bool ok = true;
      for (int tile = tile0, it = 0; ok && tile < tile1; ++tile, ++it) {
        const int acc = it & 1;
        const uint32_t acc_phase = (it >> 1) & 1;
        if (!ptx::mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag)) { give_up(); break; }
        ptx::tcgen05_fence_after_sync();
        const uint32_t d_tmem = tmem_base + acc * 256;
        for (int ks = 0; ks < k_steps; ++ks, ++step) {
          const int k0 = ks * kKStep, kw = min(kKStep, p.r - k0);
          const int stage = step % kAStages;
          if (!ptx::mbar_wait(afull_bar(stage), (step / kAStages) & 1u, abort_flag)) { give_up(); ok = false; break; }
          ptx::tcgen05_fence_after_sync();
          const uint32_t a_stage_addr = a_addr + stage * (2 * kAHalfBytes);
          // Descriptors advance by constants (16 contraction elements: 32 bytes of a K-major A row, 16 rows of 128 bytes
          // of the N-major slice), so the issuing thread adds instead of re-encoding: one thread issues every MMA, and
          // its dependent integer chain, not the tensor core, set the pace before.
          // V^T slice: N-major, one 128-byte row per k, the 64-column chunks r rows apart
          const uint64_t db0 = ptx::make_smem_desc(s_addr + uint32_t(k0) * 128u, uint32_t(p.r) * 128u, 1024);
#pragma unroll
          for (int term = 0; term < 2; ++term) {
            const uint64_t da0 = ptx::make_smem_desc(a_stage_addr + term * kAHalfBytes, 16, 1024);
#pragma unroll
            for (int k16 = 0; k16 < kKStep / 16; ++k16) {
              if (16 * k16 < kw)
                ptx::umma_bf16(d_tmem, da0 + uint64_t(2 * k16), db0 + uint64_t(128 * k16), idesc, ks > 0 || term > 0 || k16 > 0);
            }
          }
          ptx::umma_commit(afree_bar(stage));
          if (ks == k_steps - 1) ptx::umma_commit(tfull_bar(acc));
        }
      }
    }
  } else if (warp < kEpiWarps) {
    // ------------------------------------------------------------------ epilogue: TMEM -> (+ beta dW) -> smem -> TMA store
    // A warp owns 32 rows (its TMEM lane quarter) and every second 32-column chunk.  Each chunk goes
    // through a swizzled 32 x 128-byte staging box and leaves as one bulk tensor store; the tensor map
    // clips rows past d_out and columns past d_in.
    const int quarter = warp & 3;  // TMEM lanes [32*quarter, +32)
    const int half = warp >> 2;
    uint8_t* out_gen = smem_gen + kOutOffset + warp * RC::kWarpOutBytes;
    const uint32_t out_addr = smem_base + kOutOffset + warp * RC::kWarpOutBytes;
    uint32_t n_stores = 0;
    bool ok = true;
    // beta != 0: the old values of a chunk (this thread's row, 32 columns) are fetched one chunk ahead, so that their
    // latency overlaps the staging and store of the chunk before
    float4 old[8];
    int pre_row0 = -1, pre_c0 = -1;  // the chunk `old` was fetched for
    auto fetch_old = [&](int r0, int c, int ncols) {
      if (r0 + lane < p.d_out) {
        const float4* src = reinterpret_cast<const float4*>(p.dW + int64_t(r0 + lane) * p.d_in + n0 + c);
#pragma unroll
        for (int j = 0; j < 8; ++j)
          if (c + 4 * j < ncols) old[j] = src[j];
      }
      pre_row0 = r0;
      pre_c0 = c;
    };
    // ... and the lines of the chunks after that are asked into L2 a few chunks ahead (one 128-byte line per thread
    // and chunk), so that the register fetch meets L2 instead of HBM latency.  The cursor walks this warp's chunk
    // sequence (alternate 32-column chunks, the starting chunk alternating with the tile) kPrefetchAhead chunks ahead.
    constexpr int kPrefetchAhead = 4;
    const int pf_cols = min(nw, p.d_in - n0);
    int pf_tile = tile0, pf_it = 0, pf_c = 32 * (half & 1) - 64;
    auto prefetch_next = [&]() {
      pf_c += 64;
      while (pf_tile < tile1 && pf_c >= pf_cols) {
        ++pf_tile; ++pf_it;
        pf_c = 32 * ((half + pf_it) & 1);
      }
      if (pf_tile >= tile1) return;
      const int r = pf_tile * kRM + quarter * 32 + lane;
      if (r < p.d_out) asm volatile("prefetch.global.L2 [%0];" ::"l"(p.dW + int64_t(r) * p.d_in + n0 + pf_c));
    };
    if (!ADAMW && p.beta != 0.f)
      for (int a = 0; a < kPrefetchAhead; ++a) prefetch_next();
    for (int tile = tile0, it = 0; ok && tile < tile1; ++tile, ++it) {
      const int acc = it & 1;
      const uint32_t acc_phase = (it >> 1) & 1;
      if (!__all_sync(0xFFFFFFFFu, ptx::mbar_wait(tfull_bar(acc), acc_phase, abort_flag))) { give_up(); ok = false; break; }
      ptx::tcgen05_fence_after_sync();
      const int row0 = tile * kRM + quarter * 32;
      const uint32_t taddr = tmem_base + (uint32_t(quarter * 32) << 16) + acc * 256;
      const int cols = min(nw, p.d_in - n0);  // multiple of 8
      uint32_t v[32];
      // the two warps of a lane quarter take alternate 32-column chunks; which of them starts alternates with the
      // tile, so that an odd number of chunks does not always burden the same warp
      for (int c0 = 32 * ((half + it) & 1); c0 < cols; c0 += 64) {
        __syncwarp();
        ptx::tmem_ld_x32(taddr + c0, v);
        ptx::tmem_ld_wait();
        if (row0 >= p.d_out) continue;  // whole box below the matrix (warp-uniform)
        if (ADAMW) {
          // W, m, v of this 32 x 32 box come in by TMA (zeros outside the matrix), are updated in place with the
          // gradient held in registers, and leave by TMA (clipped to the matrix); dW is never written.
          const uint32_t ld_phase = n_stores & 1u;
          if (lane == 0) {
            ptx::tma_store_wait_read<0>();  // the stores of the previous box have read the staging boxes
            ptx::mbar_arrive_expect_tx(load_bar(warp), 3 * kOutBoxBytes);
            ptx::tma_load_2d(out_addr, &tmap_dw, load_bar(warp), n0 + c0, row0);
            ptx::tma_load_2d(out_addr + kOutBoxBytes, &tmap_m, load_bar(warp), n0 + c0, row0);
            ptx::tma_load_2d(out_addr + 2 * kOutBoxBytes, &tmap_v, load_bar(warp), n0 + c0, row0);
          }
          if (!__all_sync(0xFFFFFFFFu, ptx::mbar_wait(load_bar(warp), ld_phase, abort_flag))) { give_up(); ok = false; break; }
          const AdamConsts& h = p.adam;
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const uint32_t off = lane * 128 + ((j ^ (lane & 7)) << 4);
            float4 w4 = *reinterpret_cast<float4*>(out_gen + off);
            float4 m4 = *reinterpret_cast<float4*>(out_gen + kOutBoxBytes + off);
            float4 v4 = *reinterpret_cast<float4*>(out_gen + 2 * kOutBoxBytes + off);
            float* wp = &w4.x; float* mp = &m4.x; float* vp = &v4.x;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float g = __uint_as_float(v[4 * j + e]);
              const float mn = h.beta1 * mp[e] + h.one_minus_beta1 * g;
              const float vn = h.beta2 * vp[e] + h.one_minus_beta2 * g * g;
              // square root and quotient with the approximate hardware units (about 1 ulp and 2 ulp): the correctly
              // rounded sequences cost several times the rest of the update, and the error is far below the 2^-17
              // that the gradient already carries
              float root;
              asm("sqrt.approx.f32 %0, %1;" : "=f"(root) : "f"(vn * h.inv_bias2));
              wp[e] = wp[e] - h.lr * (__fdividef(mn * h.inv_bias1, root + h.eps) + h.weight_decay * wp[e]);
              mp[e] = mn;
              vp[e] = vn;
            }
            *reinterpret_cast<float4*>(out_gen + off) = w4;
            *reinterpret_cast<float4*>(out_gen + kOutBoxBytes + off) = m4;
            *reinterpret_cast<float4*>(out_gen + 2 * kOutBoxBytes + off) = v4;
            if (h.has_wlp) *reinterpret_cast<uint2*>(out_gen + 3 * kOutBoxBytes + lane * 64 + j * 8) = pack_bf16x4(w4.x, w4.y, w4.z, w4.w);
          }
          ptx::fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) {
            ptx::tma_store_2d(&tmap_dw, out_addr, n0 + c0, row0);
            ptx::tma_store_2d(&tmap_m, out_addr + kOutBoxBytes, n0 + c0, row0);
            ptx::tma_store_2d(&tmap_v, out_addr + 2 * kOutBoxBytes, n0 + c0, row0);
            if (h.has_wlp) ptx::tma_store_2d(&tmap_wlp, out_addr + 3 * kOutBoxBytes, n0 + c0, row0);
            ptx::tma_store_commit();
          }
          ++n_stores;
          continue;
        }
        if (!ADAMW && p.beta != 0.f) {
          prefetch_next();
          if (pre_row0 != row0 || pre_c0 != c0) fetch_old(row0, c0, cols);  // the first chunk of this warp
          if (row0 + lane < p.d_out) {
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              if (c0 + 4 * j < cols) {
                const float4 o = old[j];
                v[4 * j + 0] = __float_as_uint(fmaf(p.beta, o.x, __uint_as_float(v[4 * j + 0])));
                v[4 * j + 1] = __float_as_uint(fmaf(p.beta, o.y, __uint_as_float(v[4 * j + 1])));
                v[4 * j + 2] = __float_as_uint(fmaf(p.beta, o.z, __uint_as_float(v[4 * j + 2])));
                v[4 * j + 3] = __float_as_uint(fmaf(p.beta, o.w, __uint_as_float(v[4 * j + 3])));
              }
            }
          }
          // the next chunk of this warp: further along this tile, else the first one of the next tile
          if (c0 + 64 < cols) {
            fetch_old(row0, c0 + 64, cols);
          } else if (tile + 1 < tile1) {
            const int nc = 32 * ((half + it + 1) & 1), nr = row0 + kRM;
            if (nc < cols && nr < p.d_out) fetch_old(nr, nc, cols);
          }
        }
        const uint32_t box = (n_stores & 1u) * kOutBoxBytes;
        if (lane == 0) ptx::tma_store_wait_read<1>();  // the store that last used this box has read it
        __syncwarp();
#pragma unroll
        for (int j = 0; j < 8; ++j)
          *reinterpret_cast<uint4*>(out_gen + box + lane * 128 + ((j ^ (lane & 7)) << 4)) =
              make_uint4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
        ptx::fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          ptx::tma_store_2d(&tmap_dw, out_addr + box, n0 + c0, row0);
          ptx::tma_store_commit();
        }
        ++n_stores;
      }
      ptx::tcgen05_fence_before_sync();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(tempty_bar(acc));
    }
    if (lane == 0) ptx::tma_store_wait_read<0>();  // shared memory must outlive the stores' reads
  }

  ptx::tcgen05_fence_before_sync();
  __syncthreads();
  if (warp == kMmaWarp) {
    __syncwarp();
    ptx::tcgen05_fence_after_sync();
    ptx::tmem_dealloc(tmem_base, 512);
  }
}

// Pick the slice width and the row groups.  Time model of one CTA in microseconds, fitted to measurements on a B200 (calls
// back to back, 16384-token LLaMA shapes and the Qwen MLP shapes): about 3.5 us before the first tile leaves (launch, the
// wait for the pre-pass, the slice of V^T, the first A stages), then 0.3 + 0.0095 * nw per 128-row tile (MMA issue and the
// shared-memory traffic of operands and store staging both grow with the slice width).  The cheapest plan wins: in
// practice slices of 128 columns and row groups that put a CTA on every SM.
#ifndef ACX_REC_FORCE_NW
#define ACX_REC_FORCE_NW 0   // experiments only: a slice width to use wherever it fits
#endif
void plan(const Problem& q, RecParams* p) {
  const int sms = sm_count();
  const int m_tiles = int((q.d_out + kRM - 1) / kRM);
  double best = 1e300;
  for (int nw = 64; nw <= 256; nw += 32) {
    if (ACX_REC_FORCE_NW && nw != ACX_REC_FORCE_NW && ACX_REC_FORCE_NW * q.r <= kMaxSliceElems) continue;
    if ((nw + 63) / 64 * 64 * q.r > kMaxSliceElems) continue;  // the slice of V^T is staged in whole 64-column chunks
    const int n_slices = int((q.d_in + nw - 1) / nw);
    int groups = std::max(1, std::min(m_tiles, sms / std::max(1, n_slices)));
    const int tpg = (m_tiles + groups - 1) / groups;
    groups = (m_tiles + tpg - 1) / tpg;
    const double ctas = double(n_slices) * groups;
    const double waves = std::ceil(ctas / sms);
    const double cost = waves * (3.5 + tpg * (0.3 + 0.0095 * nw));
    if (cost < best - 1e-9) {
      best = cost;
      p->nw = nw; p->n_slices = n_slices; p->tiles_per_group = tpg;
    }
  }
  p->m_tiles = m_tiles;
}

}  // namespace

// hi and lo terms of A, then S^T of the seeded sketch (256-byte aligned)
static size_t split_bytes(const Problem& q) { return (size_t(q.d_out) * size_t(q.r) * 4 + 255) & ~size_t(255); }
size_t sm100_reconstruct_workspace_bytes(const Problem& q) { return split_bytes(q) + size_t(q.r) * size_t(q.d_in) * 2; }

namespace {

// Both variants: split A into the workspace, then the tensor-core kernel with programmatic stream serialization.
// `out` is dW (plain) or the fp32 master weights W (fused AdamW).
template <bool ADAMW>
cudaError_t launch_reconstruct(const Problem& q, const float* A, float* out, float* m, float* v, void* wlp, RecParams p, void* ws,
                               cudaStream_t st, const void* Vt = nullptr, float* mA = nullptr, float* vA = nullptr) {
  using RC = RecCfg<ADAMW>;
  auto kernel = reconstruct_umma_kernel<ADAMW>;
  static DeviceOnce once;  // per instantiation
  if (once.needed()) {
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, RC::kSmemBytes);
    if (e != cudaSuccess) return e;
    once.done();
  }
  p.v_from_prepass = Vt ? 0 : 1;
  __nv_bfloat16* St = Vt ? nullptr : reinterpret_cast<__nv_bfloat16*>(static_cast<uint8_t*>(ws) + split_bytes(q));
  if (!Vt) Vt = St;
  plan(q, &p);
  uint8_t* hi = static_cast<uint8_t*>(ws);
  uint8_t* lo = hi + size_t(q.d_out) * size_t(q.r) * 2;
  CUtensorMap tmap_hi, tmap_lo, tmap_out, tmap_m, tmap_v, tmap_wlp;
  if (!make_tmap_bf16(&tmap_hi, hi, q.d_out, q.r, 64, kRM)) return cudaErrorInvalidValue;
  if (!make_tmap_bf16(&tmap_lo, lo, q.d_out, q.r, 64, kRM)) return cudaErrorInvalidValue;
  if (!make_tmap_f32(&tmap_out, out, q.d_out, q.d_in, 32, 32)) return cudaErrorInvalidValue;
  CUtensorMap tmap_vt;
  if (!make_tmap_bf16(&tmap_vt, Vt, q.r, q.d_in, 64, 16)) return cudaErrorInvalidValue;
  tmap_m = tmap_out; tmap_v = tmap_out; tmap_wlp = tmap_out;  // placeholders where unused
  if (ADAMW) {
    if (!make_tmap_f32(&tmap_m, m, q.d_out, q.d_in, 32, 32)) return cudaErrorInvalidValue;
    if (!make_tmap_f32(&tmap_v, v, q.d_out, q.d_in, 32, 32)) return cudaErrorInvalidValue;
    if (wlp && !make_tmap_bf16_store(&tmap_wlp, wlp, q.d_out, q.d_in)) return cudaErrorInvalidValue;
  }

  const int64_t n4 = q.d_out * int64_t(q.r) / 4;
  const unsigned split_blocks = unsigned((n4 + 255) / 256);
  const unsigned sketch_blocks = St ? unsigned(((q.d_in / 2) * int64_t(q.r / 4) + 255) / 256) : 0u;
  reconstruct_prepass_kernel<<<split_blocks + sketch_blocks, 256, 0, st>>>(reinterpret_cast<const float4*>(A),
                                                                          reinterpret_cast<uint2*>(hi), reinterpret_cast<uint2*>(lo),
                                                                          n4, split_blocks, St, q.d_in, q.r, q.sp,
                                                                          reinterpret_cast<float4*>(mA), reinterpret_cast<float4*>(vA),
                                                                          p.adam);
  cudaError_t e = launched();
  if (e != cudaSuccess) return e;

  const int groups = (p.m_tiles + p.tiles_per_group - 1) / p.tiles_per_group;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(unsigned(p.n_slices * groups));
  cfg.blockDim = dim3(kRecThreads);
  cfg.dynamicSmemBytes = RC::kSmemBytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  e = cudaLaunchKernelEx(&cfg, kernel, tmap_hi, tmap_lo, tmap_out, tmap_m, tmap_v, tmap_wlp, tmap_vt, p);
  kernel_launch_counter().fetch_add(1, std::memory_order_relaxed);
  return e;
}

}  // namespace

cudaError_t sm100_reconstruct(const Problem& q, const float* A, float* dW, float beta, void* ws, int* status, cudaStream_t st,
                              const void* Vt) {
  RecParams p{};
  p.dW = dW; p.d_out = int(q.d_out); p.d_in = int(q.d_in); p.r = q.r; p.beta = beta; p.sp = q.sp; p.status = status;
  return launch_reconstruct<false>(q, A, dW, nullptr, nullptr, nullptr, p, ws, st, Vt);
}

cudaError_t sm100_reconstruct_adamw(const Problem& q, const float* A, float* W, float* m, float* v, void* W_lp, float lr, float beta1,
                                    float beta2, float eps, float weight_decay, int step, void* ws, int* status, cudaStream_t st) {
  RecParams p{};
  p.dW = W; p.d_out = int(q.d_out); p.d_in = int(q.d_in); p.r = q.r; p.beta = 0.f; p.sp = q.sp; p.status = status;
  p.adam.beta1 = beta1; p.adam.one_minus_beta1 = float(1.0 - double(beta1));
  p.adam.beta2 = beta2; p.adam.one_minus_beta2 = float(1.0 - double(beta2));
  p.adam.inv_bias1 = float(1.0 / (1.0 - std::pow(double(beta1), double(step))));
  p.adam.inv_bias2 = float(1.0 / (1.0 - std::pow(double(beta2), double(step))));
  p.adam.eps = eps; p.adam.lr = lr; p.adam.weight_decay = weight_decay; p.adam.has_wlp = W_lp ? 1 : 0;
  return launch_reconstruct<true>(q, A, W, m, v, W_lp, p, ws, st);
}

// W <- (1 - lr * weight_decay) W + A' V^T with A' = -lr * (Adam step of the factor): the plain kernel, accumulating into W.
cudaError_t sm100_lowrank_adamw(const Problem& q, const float* A, float* mA, float* vA, const void* Vt, float* W, float lr,
                                float beta1, float beta2, float eps, float weight_decay, int step, void* ws, int* status,
                                cudaStream_t st) {
  RecParams p{};
  p.dW = W; p.d_out = int(q.d_out); p.d_in = int(q.d_in); p.r = q.r; p.sp = q.sp; p.status = status;
  p.beta = float(1.0 - double(lr) * double(weight_decay));
  p.adam.beta1 = beta1; p.adam.one_minus_beta1 = float(1.0 - double(beta1));
  p.adam.beta2 = beta2; p.adam.one_minus_beta2 = float(1.0 - double(beta2));
  p.adam.inv_bias1 = float(1.0 / (1.0 - std::pow(double(beta1), double(step))));
  p.adam.inv_bias2 = float(1.0 / (1.0 - std::pow(double(beta2), double(step))));
  p.adam.eps = eps; p.adam.lr = lr; p.adam.weight_decay = weight_decay; p.adam.has_wlp = 0;
  return launch_reconstruct<false>(q, A, W, nullptr, nullptr, nullptr, p, ws, st, Vt, mA, vA);
}

}  // namespace acx
