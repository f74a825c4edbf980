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
//
// PAIR = true: two CTAs (a cluster of two, one SM each) share one tile of 256 * MT rows.  Each CTA stages its own
// 128 * MT rows of A and HALF of the B rows; the leader CTA (cluster rank 0) issues tcgen05.mma.cta_group::2 instructions
// of 256 x N that read A from each CTA's own shared memory and B from both, and accumulate each CTA's 128 rows in its own
// tensor memory.  With MT = 1 a CTA has two accumulator sets and six 32 KiB stages: the epilogue of a tile overlaps the
// whole mainloop of the next one (that, not the bytes moved, is what made it faster than the 256-row tile of one CTA: a
// build without any epilogue ran 8-10 % faster, one with 25 % fewer bytes from L2 no faster).  With MT = 2 the pair's
// tile has 512 rows and moves 3/4 of the bytes per flop of a 256 x 256 tile.  Every CTA loads its own boxes with plain
// (non-multicast) bulk tensor copies whose completion is counted on the leader's barrier; stage and accumulator
// hand-over between the two CTAs goes through tcgen05.commit to both CTAs' barriers and through remote mbarrier
// arrivals.  In the forward each CTA's half of B is [its half of the tile's W rows | its half of the tile's slice of
// S^T], so each CTA generates (or loads) half of the slice.
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
constexpr int kBarBytes = 1024;           // barriers, TMEM pointer, abort flag; keeps the store staging behind them 1024-byte aligned
constexpr int kEpiWarp0 = 2;
constexpr int kOutBoxBytes = 32 * 32 * 2;   // one bulk tensor store of a bf16 output: 32 rows x 32 columns, 64-byte swizzle
constexpr int kGenWarpsPerGroup = 4;        // one generator group per pipeline stage

// A CTA tile is MT row blocks of 128 (MT = 1 or 2) that share one staged B tile.
//   MT = 1: 4 stages of 48 KiB, two accumulators (the epilogue of tile i overlaps the mainloop of tile i+1).
//   MT = 2: 3 stages of 64 KiB, B is read from L2 and shared memory once for 256 rows and, in the forward,
//           a generated slice of S serves twice the MMA work; the two row blocks fill the 512 TMEM columns,
//           so the next tile's MMAs of a row block start when that block's accumulator has been drained.
// BROWS = rows reserved for the B operand per stage (256 in general; 128 for the gradient factor at r <= 128, whose
// HBM-bound mainloop then has six 32 KiB stages in flight instead of four).
template <int MT, int BROWS = kMaxBN, bool PAIR = false>
struct Cfg {
  static_assert(!PAIR || BROWS == kMaxBN, "a CTA pair stages 128 B rows per CTA");
  // stages: alone 4 x 48 KiB (MT = 1), 3 x 64 KiB (MT = 2) or 6 x 32 KiB (narrow B); a pair 6 x 32 KiB or 4 x 48 KiB
  static constexpr int kStages = PAIR ? (MT == 2 ? 4 : 6) : (MT == 2 ? 3 : (BROWS == kMaxBN ? 4 : 6));
  static constexpr int kABytes = MT * kASubBytes;
  static constexpr int kBBytes = (PAIR ? BROWS / 2 : BROWS) * kBK * 2;   // a CTA of a pair stages half of the B rows
  static constexpr int kGenWarpsPerStage = PAIR ? 2 : kGenWarpsPerGroup;  // ... and generates half of the slice
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kNumAcc = MT == 1 ? 2 : 1;   // accumulator sets (each MT x 256 columns)
  static constexpr int kEpiWarps = 4 * MT;          // four warps (the four TMEM lane quarters) per row block
  static constexpr int kOutOffset = kStages * kStageBytes + kBarBytes;  // store staging: two boxes per epilogue warp
  static constexpr int kSmemBytes = kOutOffset + kEpiWarps * 2 * kOutBoxBytes + 1024;  // + slack to align to 1024
  static constexpr int kGenWarp0 = kEpiWarp0 + kEpiWarps;
  static constexpr int kGenWarps = kGenWarpsPerStage * kStages;
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
  // Sketch generated in place, one CTA per tile: the last N-tile, when only part of its W columns exist, takes bn_last
  // W rows instead of its class's (bn_last + its slice width is a multiple of 16, so the MMA is that much narrower and
  // nothing is multiplied for columns past N); its W boxes come through tmap_v.  0: the tile is like its class.
  int bn_last;
  // Work units, kernels without cluster only:
  //   [0, full_units)                whole tiles of the first n_main N-tiles (index = nt + n_main * (mt + m_tiles * split));
  //   then extra_units               whole tiles of the other n_tiles - n_main N-tiles (index = nt' + n_extra * mt), which
  //                                  carry sketch columns only and cost less than a whole tile;
  //   then the rest of the main tiles, each cut into tail_parts units (1 or 2): the two row blocks of a tile that has
  //                                  two (MT = 2), or the two column halves of a pair's tile with one row block per
  //                                  CTA (PAIR, MT = 1; only tiles without slice whose columns all exist): the last
  //                                  round of a launch then ends sooner.
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
  int ncut;       // 1: a column half of a pair's tile (the W boxes then have half the height: tmap_b2)
  int m0, n0, nt, split;
  int nh;         // row blocks of 128 in this unit (the tile's MT, or 1 for a cut tile)
  int bn;         // B rows that come from global memory (W rows; 0 on a slice-only tile)
  int s0, width;  // forward: columns [s0, s0 + width) of S ride on this tile, as B rows [bn, bn + width)
};

// PAIR: the unit's rows are those of both CTAs (2 * nh row blocks from m0 on; CTA `rank` takes the second half), bn and
// width are those of the whole B tile (each CTA stages half of each, so both are multiples of 16), and a last,
// partly filled N-tile without slice shrinks to the multiple of 64 columns it needs.
template <int SKETCH, bool CLUSTER = false, int MT = 1, bool PAIR = false>
__device__ __forceinline__ Tile decode_tile(const Params& p, int tile) {
  Tile t;
  t.nh = MT;
  t.ncut = 0;
  if (CLUSTER) {  // consecutive CTAs (one cluster) are the splits of one M-tile; one N-tile
    t.nt = 0; t.split = tile % p.splits; t.m0 = (tile / p.splits) * kBM;
    t.n0 = 0; t.bn = p.bn; t.s0 = 0; t.width = 0;
    return t;
  }
  int mt, part = 0, npart = 0;
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
      if (PAIR && MT == 1 && p.tail_parts == 2) { npart = v & 1; t.ncut = 1; }
    }
    t.nt = idx % p.n_main;
    const int rest = idx / p.n_main;
    mt = rest % p.m_tiles;
    t.split = rest / p.m_tiles;
  }
  t.m0 = (mt * (kBM * MT) + part * kBM) * (PAIR ? 2 : 1);
  if (!SKETCH) {
    t.n0 = t.nt * p.bn; t.bn = p.bn; t.s0 = 0; t.width = 0;
    if (t.ncut) { t.bn = p.bn >> 1; t.n0 += npart * t.bn; }
    if (PAIR) t.bn = min(t.bn, (p.N - t.n0 + 63) & ~63);
    return t;
  }
  int sw;
  if (t.nt < p.n_class1) {
    t.n0 = t.nt * p.bn1; t.bn = p.bn1; t.s0 = t.nt * p.sw1; sw = p.sw1;
    if (t.ncut) { t.bn = p.bn1 >> 1; t.n0 += npart * t.bn; }   // planned only where sw1 = 0
  } else {
    t.n0 = p.n_class1 * p.bn1 + (t.nt - p.n_class1) * p.bn0; t.bn = p.bn0;
    t.s0 = p.n_class1 * p.sw1 + (t.nt - p.n_class1) * p.sw0; sw = p.sw0;
  }
  t.width = max(0, min(sw, p.r - t.s0));
  if (PAIR && t.bn > 0 && t.width == 0) t.bn = min(t.bn, (p.N - t.n0 + 63) & ~63);
  if (SKETCH == SKETCH_GENERATED && !PAIR && p.bn_last > 0 && t.nt == p.n_tiles - 1) t.bn = p.bn_last;
  return t;
}

// The sequence of work units of one CTA (see Params); next() returns the unit's index or -1 at the end.  Every role
// of the CTA runs its own copy and sees the same sequence.
struct UnitIter {
  int main_units, extra_units, full_units, n_extra, n_main, grid, c, k, e;
  __device__ UnitIter(const Params& p, bool cluster, bool pair = false) {
    grid = int(gridDim.x) >> (pair ? 1 : 0);   // the two CTAs of a pair walk the same sequence
    c = int(blockIdx.x) >> (pair ? 1 : 0);
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
// tmap_v / tmap_v2 (SKETCH_LOADED): V^T (r x d_in, K-major) with boxes of sw1 / sw0 rows, the slices of the
// two tile classes.  SKETCH_GENERATED on one CTA per tile with Params::bn_last > 0: tmap_v is the map of W with boxes of
// bn_last rows (the narrower last N-tile).
// tmap_c is the store map of a bf16 output (32 x 32 boxes, see the epilogue); unused by the fp32 epilogues.
template <bool A_MN, bool B_MN, int SKETCH, int EPI, int MT = 1, int BROWS = kMaxBN, bool PAIR = false>
__global__ void __launch_bounds__(Cfg<MT, BROWS, PAIR>::threads(SKETCH == SKETCH_GENERATED), 1)
    umma_gemm_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                     const __grid_constant__ CUtensorMap tmap_b2, const __grid_constant__ CUtensorMap tmap_c,
                     const __grid_constant__ CUtensorMap tmap_v, const __grid_constant__ CUtensorMap tmap_v2, const Params p) {
  using C = Cfg<MT, BROWS, PAIR>;
  static_assert(BROWS == kMaxBN || (MT == 1 && A_MN && B_MN), "narrow B stages serve the gradient factor only");
  static_assert(MT == 1 || (!A_MN && EPI == EPI_BF16), "256-row tiles serve the K-major-A kernels with bf16 output");
  constexpr int kStages = C::kStages, kStageBytes = C::kStageBytes, kABytes = C::kABytes;
  constexpr int kEpiWarps = C::kEpiWarps, kGenWarp0 = C::kGenWarp0, kNumAcc = C::kNumAcc;
  constexpr int kGenPerStage = C::kGenWarpsPerStage;
  constexpr bool kFastDrain = MT == 2 && EPI == EPI_BF16 && SKETCH != SKETCH_GENERATED;  // see the epilogue
  constexpr bool kCluster = EPI == EPI_F32_CLUSTER;
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
  // A pair: rank 0 leads (issues the MMAs, owns the full and accumulator-empty barriers both CTAs signal).
  const uint32_t rank = PAIR ? ptx::cluster_ctarank() : 0u;
  // The leader's copy of a barrier of this CTA, as a shared::cluster address (this CTA's own when it leads)
  auto on_leader = [&](uint32_t bar) { return PAIR ? ptx::map_to_rank(bar, 0u) : bar; };

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      // producer's arm + the generator warps that write into the stage (of both CTAs of a pair)
      ptx::mbar_init(full_bar(s), SKETCH == SKETCH_GENERATED ? 1 + kGenPerStage * (PAIR ? 2 : 1) : 1);
      // a stage is free when its MMAs have been committed and, if they sum the staged A tile, the epilogue warps are done
      ptx::mbar_init(empty_bar(s), (A_MN && p.colsum_part != nullptr) ? 1 + kEpiWarps : 1);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(tfull_bar(a), 1);
      for (int h = 0; h < 2; ++h) ptx::mbar_init(tempty_bar(a, h), PAIR ? 8 : 4);   // the four warps per row block, of both CTAs
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
    if (SKETCH == SKETCH_GENERATED && !PAIR && p.bn_last > 0) ptx::prefetch_tensormap(&tmap_v);
    if (EPI == EPI_BF16) ptx::prefetch_tensormap(&tmap_c);
  }
  if (warp == 1) {
    if (PAIR) {
      ptx::tmem_alloc_pair(tmem_slot, kTmemCols);
      ptx::tmem_relinquish_alloc_permit_pair();
    } else {
      ptx::tmem_alloc(tmem_slot, kTmemCols);
      ptx::tmem_relinquish_alloc_permit();
    }
  }
  ptx::tcgen05_fence_before_sync();
  if (PAIR) ptx::cluster_sync_all();   // the peer's barriers are initialised before anything is signalled there
  else __syncthreads();
  ptx::tcgen05_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot_gen;
  // A grid launched behind this one with programmatic stream serialization may take the SMs that this grid's CTAs
  // leave as they finish (the gradient factor of the same call behind dX: it needs nothing that dX writes).
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

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
      UnitIter units(p, kCluster, PAIR);
      bool first_tile = true;
      for (int tile = units.next(); ok && tile >= 0; tile = units.next(), first_tile = false) {
        const Tile t = decode_tile<SKETCH, kCluster, MT, PAIR>(p, tile);
        const int kb0 = t.split * p.kb_per_split, kb1 = min(num_kb_total, kb0 + p.kb_per_split);
        const bool has_w = t.bn > 0;
        const bool class1 = !SKETCH || t.nt < p.n_class1;
        const bool narrow_last = SKETCH == SKETCH_GENERATED && !PAIR && p.bn_last > 0 && t.nt == p.n_tiles - 1;
        const CUtensorMap* map_b = narrow_last ? &tmap_v : ((class1 && !t.ncut) ? &tmap_b : &tmap_b2);
        const CUtensorMap* map_v = class1 ? &tmap_v : &tmap_v2;
        // what this CTA stages of B: the W rows first, the slice below them.  Alone: all of both.  In a pair: its half
        // of the W rows (the box has the height of the class, bn_class / 2; of a shrunk last N-tile, which carries no
        // slice, only the first t.bn / 2 rows are multiplied), then its half of the slice; MN-major B: its half of the
        // 64-column chunks.
        const int hs = PAIR ? t.width >> 1 : t.width;
        const int hw = PAIR ? t.bn >> 1 : t.bn;
        const int w_box_rows = !PAIR ? t.bn : ((SKETCH ? (class1 ? p.bn1 : p.bn0) : p.bn) >> (t.ncut ? 2 : 1));
        const int v_box_rows = !PAIR ? t.width : ((class1 ? p.sw1 : p.sw0) >> 1);
        const int b_chunks = B_MN ? (PAIR ? (hw + 63) / 64 : (min(t.bn, p.N - t.n0) + 63) / 64) : 0;
        const uint32_t bytes = (A_MN ? kABytes : t.nh * kASubBytes) + (B_MN ? b_chunks * kChunkBytes : (has_w ? w_box_rows * kBK * 2 : 0)) +
                               (SKETCH == SKETCH_LOADED && t.width > 0 ? v_box_rows * kBK * 2 : 0);
        const int a_row0 = t.m0 + int(rank) * t.nh * kBM;   // a pair: this CTA's rows of the unit
        const int w_row0 = t.n0 + int(rank) * hw, v_row0 = t.s0 + int(rank) * hs;
        const uint32_t v_off = uint32_t(hw) * (kBK * 2);
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!ptx::mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) { give_up(); ok = false; break; }
          const uint32_t a_dst = smem_base + stage * kStageBytes, b_dst = a_dst + kABytes;
          // completions are counted on the leader's barrier, which the leader arms for the bytes of both CTAs
          const uint32_t bar = PAIR ? on_leader(full_bar(stage)) : full_bar(stage);
          if (!PAIR) ptx::mbar_arrive_expect_tx(full_bar(stage), bytes);
          else if (rank == 0) ptx::mbar_arrive_expect_tx(full_bar(stage), 2 * bytes);
          armed |= 1u << stage;
          auto load = [&](uint32_t dst, const CUtensorMap* map, int x, int y) {
            if (PAIR) ptx::tma_load_2d_pair(dst, map, bar, x, y);
            else ptx::tma_load_2d(dst, map, bar, x, y);
          };
          if (A_MN) {
            load(a_dst, &tmap_a, t.m0, kb * kBK);
            load(a_dst + kChunkBytes, &tmap_a, t.m0 + 64, kb * kBK);
          } else {
            for (int h = 0; h < t.nh; ++h)  // one 128-row box per row block
              load(a_dst + h * kASubBytes, &tmap_a, kb * kBK, a_row0 + h * kBM);
          }
          if (B_MN) {
            for (int c = 0; c < b_chunks; ++c) load(b_dst + c * kChunkBytes, &tmap_b, w_row0 + c * 64, kb * kBK);
          } else if (has_w) {
            load(b_dst, map_b, kb * kBK, w_row0);
          }
          if (SKETCH == SKETCH_LOADED) {
            // V^T may be the output of the grid launched just before this one (the written-out seeded sketch):
            // everything above was issued without waiting for it
            if (first_tile && kb == kb0) asm volatile("griddepcontrol.wait;" ::: "memory");
            if (t.width > 0)  // the tile's rows of V^T (a pair: this CTA's half of them)
              load(b_dst + v_off, map_v, kb * kBK, v_row0);
          }
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        // wait (bounded, one limit for all stages) for the copies still in flight before the CTA leaves; the peer of a
        // pair cannot see its copies complete (they are counted on the leader's barrier) and waits out the limit
        const uint64_t t0 = ptx::globaltimer_ns();
        for (int s = 0; s < kStages; ++s) {
          if (!(armed & (1u << s))) continue;
          const uint32_t ph = (s < stage) ? phase : (phase ^ 1u);
          while (!ptx::mbar_try_wait(full_bar(s), ph) && ptx::globaltimer_ns() - t0 < ptx::kWaitLimitNs) {}
        }
      } else if (PAIR) {
        // The leader's tensor core signals this CTA's empty barriers too: stay until the last of those arrivals has
        // landed (every stage this CTA filled has been released), so that none can reach the memory of a CTA that left.
        for (int s = 0; s < kStages && ok; ++s) {
          if (!(armed & (1u << s))) continue;
          const uint32_t ph = (s < stage) ? phase : (phase ^ 1u);   // parity of the last phase filled on stage s
          if (!ptx::mbar_wait(empty_bar(s), ph, abort_flag)) { give_up(); ok = false; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ UMMA issuer (of a pair: the leader's only)
    if (lane == 0 && rank == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int it = 0;
      bool ok = true;
      UnitIter units(p, kCluster, PAIR);
      for (int tile = units.next(); ok && tile >= 0; tile = units.next(), ++it) {
        const Tile t = decode_tile<SKETCH, kCluster, MT, PAIR>(p, tile);
        const int kb0 = t.split * p.kb_per_split, kb1 = min(num_kb_total, kb0 + p.kb_per_split);
        // with a slice the MMA spans the W rows and the slice; bn + width is a multiple of 16 by construction
        const int n_mma = PAIR ? t.bn + t.width : ((SKETCH && t.width > 0) ? t.bn + t.width : ((min(t.bn, p.N - t.n0) + 15) & ~15));
        const uint32_t idesc = ptx::make_idesc_bf16(PAIR ? 2 * kBM : kBM, n_mma, A_MN, B_MN);
        const int acc = it % kNumAcc;
        const uint32_t acc_phase = (it / kNumAcc) & 1;
        const uint32_t d_tmem = tmem_base + acc * MT * kAccCols;  // row block h accumulates at + h * kAccCols
        for (int kb = kb0; kb < kb1; ++kb) {
          const bool full_ok = PAIR ? ptx::mbar_wait_cluster(full_bar(stage), phase, abort_flag) : ptx::mbar_wait(full_bar(stage), phase, abort_flag);
          if (!full_ok) { give_up(); ok = false; break; }
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
                // the accumulator of this row block must have been drained by the epilogue of its last use (in both CTAs)
                const bool acc_ok = PAIR ? ptx::mbar_wait_cluster(tempty_bar(acc, h), acc_phase ^ 1u, abort_flag)
                                         : ptx::mbar_wait(tempty_bar(acc, h), acc_phase ^ 1u, abort_flag);
                if (!acc_ok) { give_up(); ok = false; break; }
                ptx::tcgen05_fence_after_sync();
              }
              if (PAIR)
                ptx::umma_bf16_pair(d_tmem + h * kAccCols, da + uint64_t(k * a_step + h * a_block), db + uint64_t(k * b_step), idesc,
                                    kb > kb0 || k > 0);
              else
                ptx::umma_bf16(d_tmem + h * kAccCols, da + uint64_t(k * a_step + h * a_block), db + uint64_t(k * b_step), idesc,
                               kb > kb0 || k > 0);
            }
            if (!ok) break;
          }
          if (!ok) break;
          if (PAIR) ptx::umma_commit_pair(empty_bar(stage), 3);   // frees the stage in both CTAs
          else ptx::umma_commit(empty_bar(stage));
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (ok) {
          if (PAIR) ptx::umma_commit_pair(tfull_bar(acc), 3);     // both CTAs' epilogues
          else ptx::umma_commit(tfull_bar(acc));
        }
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
    UnitIter units(p, kCluster, PAIR);
    int cs_stage = 0;        // column sums: this warp's own walk through the pipeline stages
    uint32_t cs_phase = 0;
    for (int tile = units.next(); ok && tile >= 0; tile = units.next(), ++it) {
      const Tile t = decode_tile<SKETCH, kCluster, MT, PAIR>(p, tile);
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
      const bool tfull_ok = PAIR ? ptx::mbar_wait_cluster(tfull_bar(acc), acc_phase, abort_flag) : ptx::mbar_wait(tfull_bar(acc), acc_phase, abort_flag);
      if (!__all_sync(0xFFFFFFFFu, tfull_ok)) { give_up(); ok = false; break; }
      ptx::tcgen05_fence_after_sync();
      const int row0 = t.m0 + (int(rank) * t.nh + hblock) * kBM + quarter * 32;   // first row of this warp
      const int row = row0 + lane;
      const uint32_t taddr = tmem_base + (uint32_t(quarter * 32) << 16) + (acc * MT + hblock) * kAccCols;
      // Where the output columns sit in the accumulator.  One CTA: the W columns from column 0, the slice behind them.
      // A pair: two such segments, one per CTA's half of B, each [hw W columns | hs slice columns]; segment g starts at
      // accumulator column g * (hw + hs) and holds output columns n0 + g * hw .. and slice columns s0 + g * hs ..
      const int n_seg = PAIR ? 2 : 1;
      const int hs = PAIR ? t.width >> 1 : t.width, hw = PAIR ? t.bn >> 1 : t.bn;
      const int seg_stride = hs + hw, w_acc0 = 0, s_acc0 = hw;
      auto seg_cols = [&](int g) { return max(0, min(hw, p.N - (t.n0 + g * hw))); };   // valid W columns of segment g (multiple of 8)
      const bool rows_live = row0 < p.M;   // a warp whose rows are all past M stores nothing
      const int nb0 = rows_live ? seg_cols(0) >> 5 : 0, nb1 = (rows_live && n_seg > 1) ? seg_cols(1) >> 5 : 0;   // whole 32-column boxes
      // chunk c of the boxed part: (accumulator column, output column)
      auto box_acc = [&](int c) { return c < nb0 ? w_acc0 + 32 * c : seg_stride + w_acc0 + 32 * (c - nb0); };
      auto box_col = [&](int c) { return c < nb0 ? t.n0 + 32 * c : t.n0 + hw + 32 * (c - nb0); };
      const int n_box = EPI == EPI_BF16 ? nb0 + nb1 : 0;
      // 256-row tiles have one accumulator set, so the next tile's MMAs of a row block wait until that block has been
      // drained.  With kFastDrain the 32-column chunks are first only read out of tensor memory and kept, rounded to
      // bf16, in registers (up to 8 chunks x 16 registers); the accumulator is released after that, and the staging
      // and bulk stores follow while the next tile's MMAs already run.
      uint32_t packed[kFastDrain ? 8 : 1][16];
      if (kFastDrain) {
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          if (c < n_box) {
            uint32_t v32[32];
            __syncwarp();
            ptx::tmem_ld_x32(taddr + box_acc(c), v32);
            ptx::tmem_ld_wait();
            if (p.bias != nullptr) {
#pragma unroll
              for (int j = 0; j < 4; ++j) add_bias8(v32 + 8 * j, static_cast<const __nv_bfloat16*>(p.bias) + box_col(c) + 8 * j);
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
        uint32_t v32[32];
        for (int c = 0; c < n_box; ++c) {
          __syncwarp();
          ptx::tmem_ld_x32(taddr + box_acc(c), v32);
          ptx::tmem_ld_wait();
          if (p.bias != nullptr) {
#pragma unroll
            for (int j = 0; j < 4; ++j) add_bias8(v32 + 8 * j, static_cast<const __nv_bfloat16*>(p.bias) + box_col(c) + 8 * j);
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
            *reinterpret_cast<uint4*>(out_gen + box + lane * 64 + ((j ^ ((lane >> 1) & 3)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
          }
          ptx::fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) {
            ptx::tma_store_2d(&tmap_c, out_addr + box, box_col(c), row0);
            ptx::tma_store_commit();
          }
          ++n_stores;
        }
      }
      // what the boxes do not cover (the last columns of a segment; everything with an fp32 epilogue): straight from registers
      uint32_t v[16];
      for (int g = 0; g < n_seg; ++g) {
        const int cols = seg_cols(g), done = EPI == EPI_BF16 && rows_live ? (cols & ~31) : (EPI == EPI_BF16 ? cols : 0);
        const int acc0 = g * seg_stride + w_acc0, col0 = t.n0 + g * hw;
        for (int c0 = done; c0 < cols; c0 += 16) {
          __syncwarp();
          ptx::tmem_ld_x16(taddr + acc0 + c0, v);
          ptx::tmem_ld_wait();
          if (row < p.M) {
            const int valid = min(16, cols - c0);
            if (EPI == EPI_BF16 && p.bias != nullptr) {
              add_bias8(v, static_cast<const __nv_bfloat16*>(p.bias) + col0 + c0);
              if (valid > 8) add_bias8(v + 8, static_cast<const __nv_bfloat16*>(p.bias) + col0 + c0 + 8);
            }
            if (EPI == EPI_BF16)
              store_bf16x16(static_cast<__nv_bfloat16*>(p.C) + int64_t(row) * p.ldc + col0 + c0, v, valid);
            else if (EPI == EPI_F32_SPLIT)
              store_f32x16(static_cast<float*>(p.C) + int64_t(t.split) * p.c_split_stride + int64_t(row) * p.ldc + col0 + c0, v, valid);
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
      }
      if (SKETCH) {
        uint32_t u[8];
        for (int g = 0; g < n_seg; ++g) {
          for (int c0 = 0; c0 < hs; c0 += 8) {  // slices are multiples of 8 columns
            __syncwarp();
            ptx::tmem_ld_x8(taddr + g * seg_stride + s_acc0 + c0, u);
            ptx::tmem_ld_wait();
            if (row < p.M) store_bf16x8(static_cast<__nv_bfloat16*>(p.C2) + int64_t(row) * p.ldc2 + t.s0 + g * hs + c0, u);
          }
        }
      }
      ptx::tcgen05_fence_before_sync();
      __syncwarp();
      if (lane == 0) {
        if (PAIR) ptx::mbar_arrive_cluster(on_leader(tempty_bar(acc, hblock)));   // the leader's MMA thread waits for both CTAs
        else ptx::mbar_arrive(tempty_bar(acc, hblock));
      }
      if (kFastDrain) {
        // the accumulator is free; now the kept chunks leave through the staging boxes as bulk tensor stores
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          if (c < n_box) {
            const uint32_t box = (n_stores & 1u) * kOutBoxBytes;
            if (lane == 0) ptx::tma_store_wait_read<1>();  // the store that last used this box has read it
            __syncwarp();
#pragma unroll
            for (int j = 0; j < 4; ++j)
              *reinterpret_cast<uint4*>(out_gen + box + lane * 64 + ((j ^ ((lane >> 1) & 3)) << 4)) =
                  make_uint4(packed[kFastDrain ? c : 0][4 * j], packed[kFastDrain ? c : 0][4 * j + 1],
                             packed[kFastDrain ? c : 0][4 * j + 2], packed[kFastDrain ? c : 0][4 * j + 3]);
            ptx::fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) {
              ptx::tma_store_2d(&tmap_c, out_addr + box, box_col(c), row0);
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
    // Rows [hw, hw + hs) of this CTA's K-major B stage hold its part of S^T (alone: the whole slice, hw = bn, hs = width;
    // in a pair: half of the W rows and half of the slice each): B(n = hw + j, k) = S[k0 + k][s0 + rank * hs + j].
    // Generator group g owns pipeline stage g, so each group has the time of kStages - 1
    // k-blocks of MMA work to produce its slice.  A work item is one quad of columns for TWO adjacent rows
    // of S (k, k+1): two independent Philox + Box-Muller chains per thread, and the two values of a column
    // leave as one packed bf16x2 store.  Which of a group's warps take the first items rotates with the
    // group, so that the busy warps spread over the SM's four schedulers.
    const int gwarp = warp - kGenWarp0;
    const int group = gwarp / kGenPerStage;
    const int gt = (((gwarp % kGenPerStage) - group) & (kGenPerStage - 1)) * 32 + lane;
    constexpr int kGroupThreads = 32 * kGenPerStage;
    static_assert(C::kGenWarps == kGenPerStage * kStages && (kGenPerStage & (kGenPerStage - 1)) == 0, "one generator group per stage");
    uint32_t counter = 0;  // k-blocks issued so far over all tiles of this CTA
    bool ok = true;
    UnitIter units(p, kCluster, PAIR);
    for (int tile = units.next(); ok && tile >= 0; tile = units.next()) {
      const Tile t = decode_tile<SKETCH, kCluster, MT, PAIR>(p, tile);
      const int hs = PAIR ? t.width >> 1 : t.width, hw = PAIR ? t.bn >> 1 : t.bn;
      const int s0 = t.s0 + int(rank) * hs;
      const int quads = hs >> 2;
      for (int kb = 0; kb < num_kb_total; ++kb, ++counter) {
        const int stage = counter % kStages;
        if (stage != group) continue;
        const uint32_t phase = (counter / kStages) & 1u;
        // The values do not depend on the stage being free: in a pair a thread computes its first kPre items before it
        // waits for the MMAs that last read the stage, so that the latency of the arithmetic (two dependent chains of a
        // few hundred instructions per item) lies beside the wait and not between the release of a stage and its refill
        // (a pair finishes a k-block in half the time of one CTA on the same tile; measured: 4-15 % faster on pairs,
        // 3 % slower on one CTA per tile, which keeps the plain order).
        constexpr int kPre = PAIR ? 2 : 0;
        uint32_t pre[kPre > 0 ? kPre : 1][4];
        const int n_items = (kBK / 2) * quads;
        auto make_item = [&](int idx, uint32_t (&w)[4]) {
          const int kp = idx % (kBK / 2), q = idx / (kBK / 2);  // a warp covers all 64 k of one quad of columns
          const int i = kb * kBK + 2 * kp;
          float4 za = make_float4(0.f, 0.f, 0.f, 0.f), zb = za;
          if (i < p.K) {  // rows past d_in multiply zero-filled X: keep them zero (K is even)
            za = sketch_quad(p.sp, uint32_t(i), uint32_t((s0 >> 2) + q));
            zb = sketch_quad(p.sp, uint32_t(i + 1), uint32_t((s0 >> 2) + q));
          }
          const float a4[4] = {za.x, za.y, za.z, za.w}, b4[4] = {zb.x, zb.y, zb.z, zb.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const __nv_bfloat162 h2 = __floats2bfloat162_rn(a4[e], b4[e]);
            w[e] = *reinterpret_cast<const uint32_t*>(&h2);
          }
        };
        uint8_t* b_stage = smem_gen + stage * kStageBytes + kABytes;
        auto store_item = [&](int idx, const uint32_t (&w)[4]) {
          const int kp = idx % (kBK / 2), q = idx / (kBK / 2);
          const int kk = 2 * kp;
          const uint32_t unit = uint32_t(kk >> 3), within = uint32_t(kk & 7) * 2u;
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int n = hw + 4 * q + e;  // row of the B stage
            *reinterpret_cast<uint32_t*>(b_stage + uint32_t(n) * 128u + ((unit ^ uint32_t(n & 7)) << 4) + within) = w[e];
          }
        };
#pragma unroll
        for (int j = 0; j < kPre; ++j)
          if (gt + j * kGroupThreads < n_items) make_item(gt + j * kGroupThreads, pre[j]);
        if (!__all_sync(0xFFFFFFFFu, ptx::mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag))) { give_up(); ok = false; break; }
        if (hs > 0) {
#pragma unroll
          for (int j = 0; j < kPre; ++j)
            if (gt + j * kGroupThreads < n_items) store_item(gt + j * kGroupThreads, pre[j]);
          for (int idx = gt + kPre * kGroupThreads; idx < n_items; idx += kGroupThreads) {
            uint32_t w[4];
            make_item(idx, w);
            store_item(idx, w);
          }
          ptx::fence_proxy_async_smem();
        }
        __syncwarp();
        if (lane == 0) {
          if (PAIR) ptx::mbar_arrive_cluster(on_leader(full_bar(stage)));   // the leader's MMA thread waits for both CTAs' parts
          else ptx::mbar_arrive(full_bar(stage));
        }
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
  if (PAIR) ptx::cluster_sync_all();   // neither CTA frees tensor memory or leaves while the other may still signal or read it
  else __syncthreads();
  if (warp == 1) {
    __syncwarp();
    ptx::tcgen05_fence_after_sync();
    if (PAIR) ptx::tmem_dealloc_pair(tmem_base, kTmemCols);
    else ptx::tmem_dealloc(tmem_base, kTmemCols);
  }
}

}  // namespace gemm
}  // namespace acx
