// Persistent, warp-specialised tcgen05 GEMM for sm_100a: D[M x N] = A[M x K] * B[N x K]^T in bf16
// with fp32 accumulation in tensor memory.  One kernel template serves the dense contractions of the
// compressed linear operator (Definition 3.1, Section 4):
//
//   forward   Y = X W^T and XS = X S from the same staged X tile: the B tile of one UMMA is
//             [bn_w rows of W (TMA) | a slice of S^T (generated in place from the seed)], so one
//             instruction feeds both products and S never exists in global memory;
//   dX        G W          (B is read MN-major straight from row-major W);
//   factor    G^T XS       (A and B MN-major, the token dimension split across CTAs).
//
// Roles per CTA (one CTA per SM, tiles handed out round-robin; MT = row blocks of 128 per tile, see Cfg):
//   warp 0            TMA producer             warp 1      UMMA issuer, owns the TMEM allocation
//   warps 2..2+4*MT   epilogue (TMEM -> regs -> global), four warps per row block
//   then 4 warps per pipeline stage of sketch generators (forward only): Philox + Box-Muller straight into the B stage
// Pipeline: shared-memory stages guarded by full/empty mbarriers; all waits are bounded.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "acx_internal.h"
#include "acx_umma.cuh"

namespace acx {
namespace gemm {

constexpr int kBM = 128;            // UMMA M (rows of D per MMA) = TMEM lanes
constexpr int kBK = 64;             // bf16 elements per stage along K = one 128-byte swizzle row
constexpr int kUmmaK = 16;          // K of one tcgen05.mma for 16-bit operands
constexpr int kMaxBN = 256;         // UMMA N limit
constexpr int kASubBytes = kBM * kBK * 2;   // 16 KiB: the A operand of one 128-row MMA
constexpr int kChunkBytes = 64 * kBK * 2;   // one 64-wide MN-major chunk: 64 k-rows of 128 B
constexpr int kAccCols = 256;               // TMEM columns per accumulator
constexpr int kTmemCols = 512;
constexpr int kBarBytes = 256;
constexpr int kEpiWarp0 = 2;
constexpr int kOutBoxBytes = 32 * 32 * 2;   // one bulk tensor store of a bf16 output: 32 rows x 32 columns
constexpr int kGenWarpsPerGroup = 4;        // one generator group per pipeline stage
// The producer asks the A boxes this many k-blocks ahead of its loads into L2 (A streams from HBM once; with two or
// three 64 KiB stages the loads themselves run only ~1 us ahead of the tensor core, less than a loaded HBM round trip).
#ifndef ACX_L2_PREFETCH_DIST
#define ACX_L2_PREFETCH_DIST 0
#endif
#ifndef ACX_L2_PREFETCH_B
#define ACX_L2_PREFETCH_B 0
#endif
constexpr int kPrefetchDist = ACX_L2_PREFETCH_DIST;

// A CTA tile is MT row blocks of 128 (MT = 1 or 2) that share one staged B tile.
//   MT = 1: 4 stages of 48 KiB, two accumulators (the epilogue of tile i overlaps the mainloop of tile i+1).
//   MT = 2: 3 stages of 64 KiB, B is read from L2 and shared memory once for 256 rows and, in the forward,
//           a generated slice of S serves twice the MMA work; the two row blocks fill the 512 TMEM columns,
//           so the next tile's MMAs of a row block start when that block's accumulator has been drained.
// BROWS = rows reserved for the B operand per stage (256 in general; 128 for the gradient factor at r <= 128, whose
// HBM-bound mainloop then has six 32 KiB stages in flight instead of four).
template <int MT, int BROWS = kMaxBN>
struct Cfg {
  static constexpr int kStages = MT == 2 ? 3 : (BROWS == kMaxBN ? 4 : 6);
  static constexpr int kABytes = MT * kASubBytes;
  static constexpr int kBBytes = BROWS * kBK * 2;
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kNumAcc = MT == 1 ? 2 : 1;   // accumulator sets (each MT x 256 columns)
  static constexpr int kEpiWarps = 4 * MT;          // four warps (the four TMEM lane quarters) per row block
  static constexpr int kOutOffset = kStages * kStageBytes + kBarBytes;  // store staging: two boxes per epilogue warp
  static constexpr int kSmemBytes = kOutOffset + kEpiWarps * 2 * kOutBoxBytes + 1024;  // + slack to align to 1024
  static constexpr int kGenWarp0 = kEpiWarp0 + kEpiWarps;
  static constexpr int kGenWarps = kGenWarpsPerGroup * kStages;
  static constexpr int kTileM = kBM * MT;
  static constexpr int threads(bool sketch) { return 32 * (kGenWarp0 + (sketch ? kGenWarps : 0)); }
};

// EPI_F32_CLUSTER: the splits of one output tile form a thread-block cluster; every CTA leaves its fp32 partial
// in its own shared memory and the cluster sums the partials over distributed shared memory in rank order.
// How the second factor V (d_in x r) of the stored activation reaches the forward's B tile.
enum SketchMode { SKETCH_NONE = 0, SKETCH_GENERATED = 1 /* V = S(seed), made in place */, SKETCH_LOADED = 2 /* V^T from memory */ };

enum Epilogue { EPI_BF16 = 0, EPI_F32_SPLIT = 1, EPI_F32_CLUSTER = 2 };
constexpr int kPartialPad = 4;  // floats of padding per row of the shared-memory partial (keeps 16-byte accesses conflict-free)

struct Params {
  int M, N, K;            // D is M x N; for the forward N = d_out (the sketch columns come on top)
  int bn;                 // B rows per tile of the kernels without sketch (<= 256; multiple of 64 when B is MN-major)
  int m_tiles, n_tiles;   // tiles per problem; forward: n_tiles counts tiles that carry W rows or a slice
  int splits, kb_per_split;  // K split (factor kernel); 1 / all otherwise
  // Forward only.  N-tile nt holds [bn rows of W | sw columns of S^T] in its B stage:
  //   nt <  n_class1            : bn1 rows, sw1 columns  (W rows from nt*bn1, S columns from nt*sw1)
  //   the other tiles           : bn0 rows, sw0 columns
  // with n_class1 * sw1 + (n_tiles - n_class1) * sw0 = r and bn + sw = 256 in both classes.
  int r, n_class1, bn1, sw1, bn0, sw0;
  // Work units, kernels without cluster only:
  //   [0, full_units)                whole tiles of the first n_main N-tiles (index = nt + n_main * (mt + m_tiles * split));
  //   then extra_units               whole tiles of the other n_tiles - n_main N-tiles (index = nt' + n_extra * mt), which
  //                                  carry sketch columns only and cost less than a whole tile;
  //   then the rest of the main tiles, each cut into tail_parts row blocks of 128 (1, or 2 with 256-row tiles):
  //                                  the last round of a launch then ends sooner.
  // CTA c takes the main units (whole, then cut) c, c + grid, ... in order; extra unit e belongs to CTA
  // (e + extra_shift) mod grid, which runs it right after its main unit of the round in which the W tiles of the
  // same rows run (those rows of A are then still in L2), and before a cut unit in any case: a CTA never gets a
  // whole tile after a cut one.  extra_shift keeps the extras off the CTAs that get a cut unit.
  int n_main, full_units, extra_units, tail_parts, total_units, extra_shift;
  SketchParams sp;
  void* C;   int64_t ldc;       // D (bf16 or fp32 partials)
  void* C2;  int64_t ldc2;      // XS (bf16), forward only
  const void* bias;             // forward only, may be null: bf16 [N], added to every row of D before rounding
  float* colsum_part;           // gradient factor only, may be null: [splits][M] sums over the k range of A's columns
                                // (the bias gradient: A is G_out read MN-major, so a column of A^T is a row of D)
  int64_t c_split_stride;       // elements between split partials
  int* status;                  // device status word (kDevTimeout on give-up)
};

struct Tile {
  int m0, n0, nt, split;
  int nh;         // row blocks of 128 in this unit (the tile's MT, or 1 for a cut tile)
  int bn;         // B rows that come from global memory (W rows; 0 on a slice-only tile)
  int s0, width;  // forward: columns [s0, s0 + width) of S ride on this tile, as B rows [bn, bn + width)
};

template <int SKETCH, bool CLUSTER = false, int MT = 1>
__device__ __forceinline__ Tile decode_tile(const Params& p, int tile) {
  Tile t;
  t.nh = MT;
  if (CLUSTER) {  // consecutive CTAs (one cluster) are the splits of one M-tile; one N-tile
    t.nt = 0; t.split = tile % p.splits; t.m0 = (tile / p.splits) * kBM;
    t.n0 = 0; t.bn = p.bn; t.s0 = 0; t.width = 0;
    return t;
  }
  int mt, part = 0;
  if (tile >= p.full_units && tile < p.full_units + p.extra_units) {
    const int e = tile - p.full_units, n_extra = p.n_tiles - p.n_main;
    t.nt = p.n_main + e % n_extra;
    mt = e / n_extra;
    t.split = 0;
  } else {
    int idx = tile;
    if (tile >= p.full_units) {
      const int v = tile - p.full_units - p.extra_units;
      idx = p.full_units + v / p.tail_parts;
      if (MT == 2 && p.tail_parts == 2) { part = v & 1; t.nh = 1; }
    }
    t.nt = idx % p.n_main;
    const int rest = idx / p.n_main;
    mt = rest % p.m_tiles;
    t.split = rest / p.m_tiles;
  }
  t.m0 = mt * (kBM * MT) + part * kBM;
  if (!SKETCH) {
    t.n0 = t.nt * p.bn; t.bn = p.bn; t.s0 = 0; t.width = 0;
    return t;
  }
  int sw;
  if (t.nt < p.n_class1) {
    t.n0 = t.nt * p.bn1; t.bn = p.bn1; t.s0 = t.nt * p.sw1; sw = p.sw1;
  } else {
    t.n0 = p.n_class1 * p.bn1 + (t.nt - p.n_class1) * p.bn0; t.bn = p.bn0;
    t.s0 = p.n_class1 * p.sw1 + (t.nt - p.n_class1) * p.sw0; sw = p.sw0;
  }
  t.width = max(0, min(sw, p.r - t.s0));
  return t;
}

// The sequence of work units of one CTA (see Params); next() returns the unit's index or -1 at the end.  Every role
// of the CTA runs its own copy and sees the same sequence.
struct UnitIter {
  int main_units, extra_units, full_units, n_extra, n_main, grid, c, k, e;
  __device__ UnitIter(const Params& p, bool cluster) {
    grid = int(gridDim.x);
    c = int(blockIdx.x);
    k = 0;
    if (cluster) {
      main_units = full_units = p.m_tiles * p.n_tiles * p.splits;
      extra_units = 0; n_extra = 1; n_main = 1; e = 0;
    } else {
      extra_units = p.extra_units;
      full_units = p.full_units;
      main_units = p.total_units - p.extra_units;
      n_main = p.n_main;
      n_extra = max(1, p.n_tiles - p.n_main);
      e = (c - p.extra_shift % grid + grid) % grid;  // the first extra unit of this CTA
    }
  }
  __device__ int next() {
    const int m = c + grid * k;
    const bool has_m = m < main_units;
    if (e < extra_units && (!has_m || m >= full_units || ((e / n_extra) * n_main) / grid < k)) {
      const int unit = full_units + e;
      e += grid;
      return unit;
    }
    if (!has_m) return -1;
    ++k;
    return m < full_units ? m : m + extra_units;
  }
};

// v[0..7] += bias[0..7] (bf16, 16-byte aligned), in binary32.
__device__ __forceinline__ void add_bias8(uint32_t* v, const __nv_bfloat16* bias) {
  const uint4 b = __ldg(reinterpret_cast<const uint4*>(bias));
  const uint32_t w[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    v[2 * i] = __float_as_uint(__uint_as_float(v[2 * i]) + __uint_as_float(w[i] << 16));
    v[2 * i + 1] = __float_as_uint(__uint_as_float(v[2 * i + 1]) + __uint_as_float(w[i] & 0xFFFF0000u));
  }
}

__device__ __forceinline__ void store_bf16x16(__nv_bfloat16* dst, const uint32_t (&v)[16], int valid) {
  // valid: number of leading columns to write (multiple of 8; 8 or 16)
  uint32_t w[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(v[2 * i]), __uint_as_float(v[2 * i + 1]));
    w[i] = *reinterpret_cast<uint32_t*>(&h);
  }
  uint4* d = reinterpret_cast<uint4*>(dst);
  d[0] = make_uint4(w[0], w[1], w[2], w[3]);
  if (valid > 8) d[1] = make_uint4(w[4], w[5], w[6], w[7]);
}

__device__ __forceinline__ void store_f32x16(float* dst, const uint32_t (&v)[16], int valid) {
  uint4* d = reinterpret_cast<uint4*>(dst);
#pragma unroll
  for (int i = 0; i < 4; ++i)
    if (4 * i < valid) d[i] = make_uint4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
}

__device__ __forceinline__ void store_bf16x8(__nv_bfloat16* dst, const uint32_t (&v)[8]) {
  uint32_t w[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(v[2 * i]), __uint_as_float(v[2 * i + 1]));
    w[i] = *reinterpret_cast<uint32_t*>(&h);
  }
  *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
}

// tmap_b2 is only used by the forward: the box of the W tiles of the second class (bn0 rows).
// tmap_v / tmap_v2 (SKETCH_LOADED only): V^T (r x d_in, K-major) with boxes of sw1 / sw0 rows, the slices of the
// two tile classes.
// tmap_c is the store map of a bf16 output (32 x 32 boxes, see the epilogue); unused by the fp32 epilogues.
template <bool A_MN, bool B_MN, int SKETCH, int EPI, int MT = 1, int BROWS = kMaxBN>
__global__ void __launch_bounds__(Cfg<MT, BROWS>::threads(SKETCH == SKETCH_GENERATED), 1)
    umma_gemm_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                     const __grid_constant__ CUtensorMap tmap_b2, const __grid_constant__ CUtensorMap tmap_c,
                     const __grid_constant__ CUtensorMap tmap_v, const __grid_constant__ CUtensorMap tmap_v2, const Params p) {
  using C = Cfg<MT, BROWS>;
  static_assert(BROWS == kMaxBN || (MT == 1 && A_MN && B_MN), "narrow B stages serve the gradient factor only");
  static_assert(MT == 1 || (!A_MN && EPI == EPI_BF16), "256-row tiles serve the K-major-A kernels with bf16 output");
  constexpr int kStages = C::kStages, kStageBytes = C::kStageBytes, kABytes = C::kABytes;
  constexpr int kEpiWarps = C::kEpiWarps, kGenWarp0 = C::kGenWarp0, kNumAcc = C::kNumAcc;
  constexpr bool kFastDrain = MT == 2 && EPI == EPI_BF16 && SKETCH != SKETCH_GENERATED;  // see the epilogue
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (ptx::smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - ptx::smem_u32(smem_raw));  // generic pointer to the aligned base
  const uint32_t bar_base = smem_base + kStages * kStageBytes;
  // barrier layout (8 bytes each): full[kStages], empty[kStages], tmem_full[2], tmem_empty[2 sets][2 row blocks];
  // then the TMEM pointer and the abort flag
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (kStages + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * kStages + a); };
  auto tempty_bar = [&](int a, int h) { return bar_base + 8u * (2 * kStages + 2 + 2 * a + h); };
  constexpr int kSlot = 8 * (2 * kStages + 6);
  const uint32_t tmem_slot = bar_base + kSlot;
  volatile uint32_t* tmem_slot_gen = reinterpret_cast<volatile uint32_t*>(smem_gen + kStages * kStageBytes + kSlot);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_gen + kStages * kStageBytes + kSlot + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_kb_total = (p.K + kBK - 1) / kBK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      ptx::mbar_init(full_bar(s), SKETCH == SKETCH_GENERATED ? 1 + kGenWarpsPerGroup : 1);
      // a stage is free when its MMAs have been committed and, if they sum the staged A tile, the epilogue warps are done
      ptx::mbar_init(empty_bar(s), (A_MN && p.colsum_part != nullptr) ? 1 + kEpiWarps : 1);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(tfull_bar(a), 1);
      for (int h = 0; h < 2; ++h) ptx::mbar_init(tempty_bar(a, h), 4);
    }
    *abort_flag = 0;
    ptx::fence_barrier_init();
    ptx::prefetch_tensormap(&tmap_a);
    ptx::prefetch_tensormap(&tmap_b);
    if (SKETCH) ptx::prefetch_tensormap(&tmap_b2);
    if (SKETCH == SKETCH_LOADED) {
      ptx::prefetch_tensormap(&tmap_v);
      ptx::prefetch_tensormap(&tmap_v2);
    }
    if (EPI == EPI_BF16) ptx::prefetch_tensormap(&tmap_c);
  }
  if (warp == 1) {
    ptx::tmem_alloc(tmem_slot, kTmemCols);
    ptx::tmem_relinquish_alloc_permit();
  }
  ptx::tcgen05_fence_before_sync();
  __syncthreads();
  ptx::tcgen05_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot_gen;

  auto give_up = [&]() {
    *abort_flag = 1;
    atomicExch(p.status, kDevTimeout);
  };

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      uint32_t armed = 0;  // bit s: full[s] was armed at least once
      bool ok = true;
      UnitIter units(p, EPI == EPI_F32_CLUSTER);
      bool first_tile = true;
      for (int tile = units.next(); ok && tile >= 0; tile = units.next(), first_tile = false) {
        const Tile t = decode_tile<SKETCH, EPI == EPI_F32_CLUSTER, MT>(p, tile);
        const int kb0 = t.split * p.kb_per_split, kb1 = min(num_kb_total, kb0 + p.kb_per_split);
        const bool has_w = t.bn > 0;
        const int b_chunks = B_MN ? (min(t.bn, p.N - t.n0) + 63) / 64 : 0;
        const uint32_t bytes = (A_MN ? kABytes : t.nh * kASubBytes) + (B_MN ? b_chunks * kChunkBytes : t.bn * kBK * 2) +
                               (SKETCH == SKETCH_LOADED ? t.width * kBK * 2 : 0);
        const CUtensorMap* map_b = (SKETCH && t.nt >= p.n_class1) ? &tmap_b2 : &tmap_b;
        const CUtensorMap* map_v = t.nt >= p.n_class1 ? &tmap_v2 : &tmap_v;
        // L2 prefetch of the operand boxes of k-block kb of tile u (same coordinates as the loads below)
        auto prefetch_kb = [&](const Tile& u, int kb) {
          if (A_MN) {
            ptx::tma_prefetch_2d(&tmap_a, u.m0, kb * kBK);
            ptx::tma_prefetch_2d(&tmap_a, u.m0 + 64, kb * kBK);
          } else {
            for (int h = 0; h < u.nh; ++h) ptx::tma_prefetch_2d(&tmap_a, kb * kBK, u.m0 + h * kBM);
          }
          if (ACX_L2_PREFETCH_B) {
            if (B_MN) {
              const int chunks = (min(u.bn, p.N - u.n0) + 63) / 64;
              for (int c = 0; c < chunks; ++c) ptx::tma_prefetch_2d(&tmap_b, u.n0 + c * 64, kb * kBK);
            } else if (u.bn > 0) {
              ptx::tma_prefetch_2d((SKETCH && u.nt >= p.n_class1) ? &tmap_b2 : &tmap_b, kb * kBK, u.n0);
            }
          }
        };
        Tile t_next = t;
        int next_kb0 = 0, next_kb1 = 0;
        if (kPrefetchDist > 0) {
          UnitIter peek = units;   // the unit after this one, for the prefetches that run past this tile's last k-block
          const int nxt = peek.next();
          if (nxt >= 0) {
            t_next = decode_tile<SKETCH, EPI == EPI_F32_CLUSTER, MT>(p, nxt);
            next_kb0 = t_next.split * p.kb_per_split;
            next_kb1 = min(num_kb_total, next_kb0 + p.kb_per_split);
          }
          if (first_tile)
            for (int d = 0; d < kPrefetchDist && kb0 + d < kb1; ++d) prefetch_kb(t, kb0 + d);
        }
        for (int kb = kb0; kb < kb1; ++kb) {
          if (kPrefetchDist > 0) {
            const int pk = kb + kPrefetchDist;
            if (pk < kb1) prefetch_kb(t, pk);
            else if (next_kb0 + (pk - kb1) < next_kb1) prefetch_kb(t_next, next_kb0 + (pk - kb1));
          }
          if (!ptx::mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) { give_up(); ok = false; break; }
          const uint32_t a_dst = smem_base + stage * kStageBytes, b_dst = a_dst + kABytes;
          ptx::mbar_arrive_expect_tx(full_bar(stage), bytes);
          armed |= 1u << stage;
          if (A_MN) {
            ptx::tma_load_2d(a_dst, &tmap_a, full_bar(stage), t.m0, kb * kBK);
            ptx::tma_load_2d(a_dst + kChunkBytes, &tmap_a, full_bar(stage), t.m0 + 64, kb * kBK);
          } else {
            for (int h = 0; h < t.nh; ++h)  // one 128-row box per row block
              ptx::tma_load_2d(a_dst + h * kASubBytes, &tmap_a, full_bar(stage), kb * kBK, t.m0 + h * kBM);
          }
          if (B_MN) {
            for (int c = 0; c < b_chunks; ++c)
              ptx::tma_load_2d(b_dst + c * kChunkBytes, &tmap_b, full_bar(stage), t.n0 + c * 64, kb * kBK);
          } else if (has_w) {
            ptx::tma_load_2d(b_dst, map_b, full_bar(stage), kb * kBK, t.n0);
          }
          if (SKETCH == SKETCH_LOADED) {
            // V^T may be the output of the grid launched just before this one (the written-out seeded sketch):
            // everything above was issued without waiting for it
            if (first_tile && kb == kb0) asm volatile("griddepcontrol.wait;" ::: "memory");
            if (t.width > 0)  // rows [bn, bn + width) of the B stage: rows s0.. of V^T
              ptx::tma_load_2d(b_dst + t.bn * (kBK * 2), map_v, full_bar(stage), kb * kBK, t.s0);
          }
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        // wait (bounded) for the copies still in flight before the CTA leaves
        for (int s = 0; s < kStages; ++s) {
          if (!(armed & (1u << s))) continue;
          const uint32_t ph = (s < stage) ? phase : (phase ^ 1u);
          const uint64_t t0 = ptx::globaltimer_ns();
          while (!ptx::mbar_try_wait(full_bar(s), ph) && ptx::globaltimer_ns() - t0 < ptx::kWaitLimitNs) {}
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ UMMA issuer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int it = 0;
      bool ok = true;
      UnitIter units(p, EPI == EPI_F32_CLUSTER);
      for (int tile = units.next(); ok && tile >= 0; tile = units.next(), ++it) {
        const Tile t = decode_tile<SKETCH, EPI == EPI_F32_CLUSTER, MT>(p, tile);
        const int kb0 = t.split * p.kb_per_split, kb1 = min(num_kb_total, kb0 + p.kb_per_split);
        // with a slice the MMA spans the W rows and the slice; bn + width is a multiple of 16 by construction
        const int n_mma = (SKETCH && t.width > 0) ? t.bn + t.width : ((min(t.bn, p.N - t.n0) + 15) & ~15);
        const uint32_t idesc = ptx::make_idesc_bf16(kBM, n_mma, A_MN, B_MN);
        const int acc = it % kNumAcc;
        const uint32_t acc_phase = (it / kNumAcc) & 1;
        const uint32_t d_tmem = tmem_base + acc * MT * kAccCols;  // row block h accumulates at + h * kAccCols
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!ptx::mbar_wait(full_bar(stage), phase, abort_flag)) { give_up(); ok = false; break; }
          ptx::tcgen05_fence_after_sync();
          const uint32_t a_addr = smem_base + stage * kStageBytes, b_addr = a_addr + kABytes;
          const uint64_t da = A_MN ? ptx::make_smem_desc(a_addr, kChunkBytes, 1024) : ptx::make_smem_desc(a_addr, 16, 1024);
          const uint64_t db = B_MN ? ptx::make_smem_desc(b_addr, kChunkBytes, 1024) : ptx::make_smem_desc(b_addr, 16, 1024);
          constexpr uint32_t a_step = (A_MN ? kUmmaK * 128 : kUmmaK * 2) >> 4;
          constexpr uint32_t b_step = (B_MN ? kUmmaK * 128 : kUmmaK * 2) >> 4;
          constexpr uint32_t a_block = kASubBytes >> 4;  // next 128 rows of a K-major A stage
#pragma unroll
          for (int k = 0; k < kBK / kUmmaK; ++k) {
#pragma unroll
            for (int h = 0; h < MT; ++h) {
              if (h >= t.nh) break;
              if (kb == kb0 && k == 0) {
                // the accumulator of this row block must have been drained by the epilogue of its last use
                if (!ptx::mbar_wait(tempty_bar(acc, h), acc_phase ^ 1u, abort_flag)) { give_up(); ok = false; break; }
                ptx::tcgen05_fence_after_sync();
              }
              ptx::umma_bf16(d_tmem + h * kAccCols, da + uint64_t(k * a_step + h * a_block), db + uint64_t(k * b_step), idesc,
                             kb > kb0 || k > 0);
            }
            if (!ok) break;
          }
          if (!ok) break;
          ptx::umma_commit(empty_bar(stage));
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (ok) ptx::umma_commit(tfull_bar(acc));
      }
    }
  } else if (warp < kGenWarp0) {
    // ------------------------------------------------------------------ epilogue
    const int quarter = warp & 3;  // TMEM lanes [32*quarter, +32) are the ones this warp may read
    const int hblock = (warp - kEpiWarp0) >> 2;  // which 128-row block of the tile this warp drains
    uint8_t* out_gen = smem_gen + C::kOutOffset + (warp - kEpiWarp0) * 2 * kOutBoxBytes;
    const uint32_t out_addr = smem_base + C::kOutOffset + (warp - kEpiWarp0) * 2 * kOutBoxBytes;
    uint32_t n_stores = 0;
    int it = 0;
    bool ok = true;
    UnitIter units(p, EPI == EPI_F32_CLUSTER);
    int cs_stage = 0;        // column sums: this warp's own walk through the pipeline stages
    uint32_t cs_phase = 0;
    for (int tile = units.next(); ok && tile >= 0; tile = units.next(), ++it) {
      const Tile t = decode_tile<SKETCH, EPI == EPI_F32_CLUSTER, MT>(p, tile);
      if (hblock >= t.nh) continue;  // a cut tile: the second row block's warps have nothing to drain (and no whole tile follows)
      if (A_MN && p.colsum_part != nullptr) {
        // While the tensor core multiplies, the (otherwise idle) epilogue warps add up the staged A tile along k:
        // thread c of the 128 owns row m0 + c of D = column c of the MN-major A stage (two chunks of 64 columns,
        // 64 k-rows of 128 bytes each, 16-byte units XOR-swizzled with the row).
        const int c = (warp - kEpiWarp0) * 32 + lane, chunk = c >> 6, cc = c & 63;
        const int kb0 = t.split * p.kb_per_split, kb1 = min(num_kb_total, kb0 + p.kb_per_split);
        float s0 = 0.f, s1 = 0.f;
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!__all_sync(0xFFFFFFFFu, ptx::mbar_wait(full_bar(cs_stage), cs_phase, abort_flag))) { give_up(); ok = false; break; }
          const uint8_t* a_chunk = smem_gen + cs_stage * kStageBytes + chunk * kChunkBytes;
#pragma unroll 8
          for (int k = 0; k < kBK; k += 2) {
            const uint16_t e0 = *reinterpret_cast<const uint16_t*>(a_chunk + k * 128 + ((((cc >> 3) ^ (k & 7))) << 4) + (cc & 7) * 2);
            const uint16_t e1 = *reinterpret_cast<const uint16_t*>(a_chunk + (k + 1) * 128 + ((((cc >> 3) ^ ((k + 1) & 7))) << 4) + (cc & 7) * 2);
            s0 += __uint_as_float(uint32_t(e0) << 16);
            s1 += __uint_as_float(uint32_t(e1) << 16);
          }
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(empty_bar(cs_stage));
          if (++cs_stage == kStages) { cs_stage = 0; cs_phase ^= 1u; }
        }
        if (t.m0 + c < p.M && ok) p.colsum_part[int64_t(t.split) * p.M + t.m0 + c] = s0 + s1;
        // The epilogue below may reuse the pipeline stages (the cluster variant parks its partial tile there) as soon as
        // the MMAs are done: no epilogue warp may get there while another still reads a staged tile.  Reached by all
        // four warps also after a give-up (the abort flag ends everybody's waits).
        asm volatile("bar.sync 1, %0;" ::"n"(kEpiWarps * 32) : "memory");
        if (!ok) break;
      }
      const int acc = it % kNumAcc;
      const uint32_t acc_phase = (it / kNumAcc) & 1;
      if (!__all_sync(0xFFFFFFFFu, ptx::mbar_wait(tfull_bar(acc), acc_phase, abort_flag))) { give_up(); ok = false; break; }
      ptx::tcgen05_fence_after_sync();
      const int row = t.m0 + hblock * kBM + quarter * 32 + lane;
      const uint32_t taddr = tmem_base + (uint32_t(quarter * 32) << 16) + (acc * MT + hblock) * kAccCols;
      const int w_cols = max(0, min(t.bn, p.N - t.n0));  // multiple of 8
      int c_direct = 0;  // columns from here on are stored straight from registers
      // 256-row tiles have one accumulator set, so the next tile's MMAs of a row block wait until that block has been
      // drained.  With kFastDrain the 32-column chunks are first only read out of tensor memory and kept, rounded to
      // bf16, in registers (up to 8 chunks x 16 registers); the accumulator is released after that, and the staging
      // and bulk stores follow while the next tile's MMAs already run.
      uint32_t packed[kFastDrain ? 8 : 1][16];
      int n_box = 0;
      if (kFastDrain) {
        const int row0 = t.m0 + hblock * kBM + quarter * 32;
        n_box = (row0 < p.M) ? (w_cols >> 5) : 0;
        c_direct = (row0 < p.M) ? (w_cols & ~31) : w_cols;  // a warp whose rows are all past M stores nothing
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          if (c < n_box) {
            uint32_t v32[32];
            __syncwarp();
            ptx::tmem_ld_x32(taddr + 32 * c, v32);
            ptx::tmem_ld_wait();
            if (p.bias != nullptr) {
#pragma unroll
              for (int j = 0; j < 4; ++j) add_bias8(v32 + 8 * j, static_cast<const __nv_bfloat16*>(p.bias) + t.n0 + 32 * c + 8 * j);
            }
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              __nv_bfloat162 h2 = __floats2bfloat162_rn(__uint_as_float(v32[2 * i]), __uint_as_float(v32[2 * i + 1]));
              packed[kFastDrain ? c : 0][i] = *reinterpret_cast<uint32_t*>(&h2);
            }
          }
        }
      } else if (EPI == EPI_BF16) {
        // Chunks of 32 columns go through a 32 x 64-byte box in shared memory and leave as one bulk tensor
        // store each: a thread holds one row, so direct stores would touch 32 lines per instruction.
        const int row0 = t.m0 + hblock * kBM + quarter * 32;
        c_direct = (row0 < p.M) ? (w_cols & ~31) : w_cols;  // a warp whose rows are all past M stores nothing
        uint32_t v32[32];
        for (int c0 = 0; c0 < (w_cols & ~31) && row0 < p.M; c0 += 32) {
          __syncwarp();
          ptx::tmem_ld_x32(taddr + c0, v32);
          ptx::tmem_ld_wait();
          if (p.bias != nullptr) {
#pragma unroll
            for (int j = 0; j < 4; ++j) add_bias8(v32 + 8 * j, static_cast<const __nv_bfloat16*>(p.bias) + t.n0 + c0 + 8 * j);
          }
          const uint32_t box = (n_stores & 1u) * kOutBoxBytes;
          if (lane == 0) ptx::tma_store_wait_read<1>();  // the store that last used this box has read it
          __syncwarp();
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            uint32_t w[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              __nv_bfloat162 h2 = __floats2bfloat162_rn(__uint_as_float(v32[8 * j + 2 * i]), __uint_as_float(v32[8 * j + 2 * i + 1]));
              w[i] = *reinterpret_cast<uint32_t*>(&h2);
            }
            *reinterpret_cast<uint4*>(out_gen + box + lane * 64 + j * 16) = make_uint4(w[0], w[1], w[2], w[3]);
          }
          ptx::fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) {
            ptx::tma_store_2d(&tmap_c, out_addr + box, t.n0 + c0, row0);
            ptx::tma_store_commit();
          }
          ++n_stores;
        }
      }
      uint32_t v[16];
      for (int c0 = c_direct; c0 < w_cols; c0 += 16) {
        __syncwarp();
        ptx::tmem_ld_x16(taddr + c0, v);
        ptx::tmem_ld_wait();
        if (row < p.M) {
          const int valid = min(16, w_cols - c0);
          if (EPI == EPI_BF16 && p.bias != nullptr) {
            add_bias8(v, static_cast<const __nv_bfloat16*>(p.bias) + t.n0 + c0);
            if (valid > 8) add_bias8(v + 8, static_cast<const __nv_bfloat16*>(p.bias) + t.n0 + c0 + 8);
          }
          if (EPI == EPI_BF16)
            store_bf16x16(static_cast<__nv_bfloat16*>(p.C) + int64_t(row) * p.ldc + t.n0 + c0, v, valid);
          else if (EPI == EPI_F32_SPLIT)
            store_f32x16(static_cast<float*>(p.C) + int64_t(t.split) * p.c_split_stride + int64_t(row) * p.ldc + t.n0 + c0, v, valid);
        }
        if (EPI == EPI_F32_CLUSTER) {
          // the pipeline stages are idle once the accumulator is full: the partial tile lives there
          // (every row is written, also those past M, so that the reduction reads defined values)
          float* part = reinterpret_cast<float*>(smem_gen) + (quarter * 32 + lane) * (p.N + kPartialPad) + c0;
#pragma unroll
          for (int i = 0; i < 4; ++i)
            reinterpret_cast<uint4*>(part)[i] = make_uint4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
        }
      }
      if (SKETCH) {
        uint32_t u[8];
        for (int c0 = 0; c0 < t.width; c0 += 8) {  // slices are multiples of 8 columns
          __syncwarp();
          ptx::tmem_ld_x8(taddr + t.bn + c0, u);
          ptx::tmem_ld_wait();
          if (row < p.M) store_bf16x8(static_cast<__nv_bfloat16*>(p.C2) + int64_t(row) * p.ldc2 + t.s0 + c0, u);
        }
      }
      ptx::tcgen05_fence_before_sync();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(tempty_bar(acc, hblock));
      if (kFastDrain) {
        // the accumulator is free; now the kept chunks leave through the staging boxes as bulk tensor stores
        const int row0 = t.m0 + hblock * kBM + quarter * 32;
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          if (c < n_box) {
            const uint32_t box = (n_stores & 1u) * kOutBoxBytes;
            if (lane == 0) ptx::tma_store_wait_read<1>();  // the store that last used this box has read it
            __syncwarp();
#pragma unroll
            for (int j = 0; j < 4; ++j)
              *reinterpret_cast<uint4*>(out_gen + box + lane * 64 + j * 16) =
                  make_uint4(packed[kFastDrain ? c : 0][4 * j], packed[kFastDrain ? c : 0][4 * j + 1],
                             packed[kFastDrain ? c : 0][4 * j + 2], packed[kFastDrain ? c : 0][4 * j + 3]);
            ptx::fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) {
              ptx::tma_store_2d(&tmap_c, out_addr + box, t.n0 + 32 * c, row0);
              ptx::tma_store_commit();
            }
            ++n_stores;
          }
        }
      }
    }
    if (EPI == EPI_BF16 && lane == 0) ptx::tma_store_wait_read<0>();  // shared memory must outlive the stores' reads
  } else if (SKETCH == SKETCH_GENERATED) {
    // ------------------------------------------------------------------ sketch generators
    // Rows [bn, bn + width) of the K-major B stage hold S^T: B(n = bn + j - s0, k) = S[k0 + k][j].
    // Generator group g (four warps) owns pipeline stage g, so each group has the time of kStages - 1
    // k-blocks of MMA work to produce its slice.  A work item is one quad of columns for TWO adjacent rows
    // of S (k, k+1): two independent Philox + Box-Muller chains per thread, and the two values of a column
    // leave as one packed bf16x2 store.  Which of a group's warps take the first items rotates with the
    // group, so that the busy warps spread over the SM's four schedulers.
    const int gwarp = warp - kGenWarp0;
    const int group = gwarp / kGenWarpsPerGroup;
    const int gt = (((gwarp % kGenWarpsPerGroup) - group) & (kGenWarpsPerGroup - 1)) * 32 + lane;
    constexpr int kGroupThreads = 32 * kGenWarpsPerGroup;
    static_assert(C::kGenWarps == kGenWarpsPerGroup * kStages, "one generator group per stage");
    uint32_t counter = 0;  // k-blocks issued so far over all tiles of this CTA
    bool ok = true;
    UnitIter units(p, EPI == EPI_F32_CLUSTER);
    for (int tile = units.next(); ok && tile >= 0; tile = units.next()) {
      const Tile t = decode_tile<SKETCH, EPI == EPI_F32_CLUSTER, MT>(p, tile);
      const int s0 = t.s0, width = t.width;
      const int quads = width >> 2;
      for (int kb = 0; kb < num_kb_total; ++kb, ++counter) {
        const int stage = counter % kStages;
        if (stage != group) continue;
        const uint32_t phase = (counter / kStages) & 1u;
        if (!__all_sync(0xFFFFFFFFu, ptx::mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag))) { give_up(); ok = false; break; }
        if (width > 0) {
          uint8_t* b_stage = smem_gen + stage * kStageBytes + kABytes;
          for (int idx = gt; idx < (kBK / 2) * quads; idx += kGroupThreads) {
            const int kp = idx % (kBK / 2), q = idx / (kBK / 2);  // a warp covers all 64 k of one quad of columns
            const int kk = 2 * kp, i = kb * kBK + kk;
            float4 za = make_float4(0.f, 0.f, 0.f, 0.f), zb = za;
            if (i < p.K) {  // rows past d_in multiply zero-filled X: keep them zero (K is even)
              za = sketch_quad(p.sp, uint32_t(i), uint32_t((s0 >> 2) + q));
              zb = sketch_quad(p.sp, uint32_t(i + 1), uint32_t((s0 >> 2) + q));
            }
            const float a4[4] = {za.x, za.y, za.z, za.w}, b4[4] = {zb.x, zb.y, zb.z, zb.w};
            const uint32_t unit = uint32_t(kk >> 3), within = uint32_t(kk & 7) * 2u;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const int n = t.bn + 4 * q + e;  // row of the B tile
              const __nv_bfloat162 h2 = __floats2bfloat162_rn(a4[e], b4[e]);
              *reinterpret_cast<__nv_bfloat162*>(b_stage + uint32_t(n) * 128u + ((unit ^ uint32_t(n & 7)) << 4) + within) = h2;
            }
          }
          ptx::fence_proxy_async_smem();
        }
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(full_bar(stage));
      }
    }
  }

  if (EPI == EPI_F32_CLUSTER) {
    // ------------------------------------------------------------------ cluster reduction over DSMEM
    // Every thread of every CTA of the cluster arrives (also after a give-up, so nobody waits for ever).
    // CTA `rank` then owns the rank-th contiguous share of the 128 x N tile (in float4s) and adds the partials
    // of ranks 0, 1, ... in that fixed order, which makes the result bitwise reproducible; 128-bit stores.
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
    const int rank = blockIdx.x % p.splits, m0 = (blockIdx.x / p.splits) * kBM;
    const int f4_per_row = p.N >> 2, total = kBM * f4_per_row;
    const uint32_t part_addr = ptx::smem_u32(smem_gen);
    float* out = static_cast<float*>(p.C);
    const int share = (total + p.splits - 1) / p.splits, i_end = min(total, (rank + 1) * share);
    for (int i = rank * share + int(threadIdx.x); i < i_end; i += int(blockDim.x)) {
      const int row = i / f4_per_row, c4 = i - row * f4_per_row;
      const uint32_t local = part_addr + uint32_t(row * (p.N + kPartialPad) + 4 * c4) * 4u;
      float4 acc4 = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int s = 0; s < p.splits; ++s) {
        uint32_t remote;
        float4 v4;
        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"(s));
        asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];"
                     : "=f"(v4.x), "=f"(v4.y), "=f"(v4.z), "=f"(v4.w)
                     : "r"(remote)
                     : "memory");
        acc4.x += v4.x; acc4.y += v4.y; acc4.z += v4.z; acc4.w += v4.w;
      }
      if (m0 + row < p.M) *reinterpret_cast<float4*>(out + int64_t(m0 + row) * p.ldc + 4 * c4) = acc4;
    }
    // nobody may leave (and free its shared memory) while a peer can still read it
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
  }

  // ------------------------------------------------------------------ teardown
  ptx::tcgen05_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    ptx::tcgen05_fence_after_sync();
    ptx::tmem_dealloc(tmem_base, kTmemCols);
  }
}

}  // namespace gemm
}  // namespace acx
