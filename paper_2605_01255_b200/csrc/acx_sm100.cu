// Host side of the tcgen05 path: tensor-map encoding, tile-shape selection and launches.
#include <algorithm>
#include <mutex>
#include <vector>

#include "acx_gemm_sm100.cuh"
#include "acx_tmap.h"

namespace acx {
namespace {

using gemm::Params;

// Time per flop of the forward's 256-row mainloop relative to its 128-row one (measured at the LLaMA-3B shapes):
// it generates each slice of S once for 256 rows.
constexpr double kFwdRowBlocks2Speed = 0.90;

// S^T (r x d_in, bf16) written out once, for the GEMM that reads the sketch from memory.
__global__ void __launch_bounds__(256) sketch_transposed_kernel(__nv_bfloat16* __restrict__ St, int64_t d_in, int r, SketchParams sp) {
  // the dependent GEMM may start now: it waits for this grid only before its first read of S^T
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const uint32_t half = uint32_t(d_in >> 1);
  const int64_t idx = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
  if (idx >= int64_t(half) * (r >> 2)) return;
  sketch_transposed_store(sp, St, d_in, uint32_t(idx % half), uint32_t(idx / half));
}

// Relative cost of half a 256-row tile, measured: it has half the MMA work, but each pipeline stage then holds half
// as much work while a load takes as long, and three stages no longer cover the latency.
constexpr double kCutTileCost = 0.8;
// Relative cost of a column half (128 columns) of a pair's 256 x 256 tile: half the MMA work with the same A traffic.
constexpr double kColumnHalfCost = 0.62;

// Orders the work units of a launch (see Params).  The last, partly filled round of a persistent launch costs a
// whole tile time however few tiles it holds; cutting its 256-row tiles into two row blocks (when those still
// fit one round) and putting the cheaper sketch-only tiles there shortens it.  Returns the launch time in whole
// tile times: CTA c runs units c, c + grid, ...
// n_main of the n_tiles N-tiles are whole-cost tiles; the other n_tiles - n_main cost extra_cost each.
double plan_units(Params* p, int n_main, double extra_cost, bool may_cut, int grid, double cut_cost = kCutTileCost) {
  const int main_tiles = n_main * p->m_tiles * p->splits;
  const int extras = (p->n_tiles - n_main) * p->m_tiles;
  p->n_main = n_main;
  p->extra_units = extras;
  double best = 1e300;
  std::vector<double> load(size_t(grid), 0.0);
  for (int parts = 1; parts <= (may_cut ? 2 : 1); ++parts) {
    for (int drop = 0; drop <= 1; ++drop) {  // drop = 1: one more round of whole tiles joins the tail
      const int rounds = main_tiles / grid - drop;
      if (rounds < 0 || (drop && extras == 0 && parts == 1)) continue;
      const int full = rounds * grid;
      std::fill(load.begin(), load.end(), 0.0);
      const int tail = (main_tiles - full) * parts;
      for (int t = 0; t < tail; ++t) load[size_t(t % grid)] += parts == 2 ? cut_cost : 1.0;
      for (int e = 0; e < extras; ++e) load[size_t((e + tail) % grid)] += extra_cost;  // extra_shift = tail: next to the tail units
      const double time = rounds + *std::max_element(load.begin(), load.end());
      if (time < best - 1e-9) {
        best = time;
        p->full_units = full;
        p->tail_parts = parts;
        p->total_units = full + extras + tail;
        p->extra_shift = tail % grid;
      }
    }
  }
  return best;
}

// CTA pairs (clusters of two) of the 512-row kernels that the device holds at once: 74 on a B200.  Asked of the
// driver once (one representative instantiation: all of them take a whole SM per CTA).
int pair_slots();

// pdl: the kernel is launched with programmatic stream serialization on the grid launched just before it.
// PAIR: 512-row tiles on clusters of two CTAs (MT must be 2); the units of p were planned for pair_slots() pairs.
template <bool A_MN, bool B_MN, int SKETCH, int EPI, int MT = 1, int BROWS = gemm::kMaxBN, bool PAIR = false>
cudaError_t launch_gemm(const CUtensorMap& ta, const CUtensorMap& tb, const CUtensorMap& tb2, const CUtensorMap& tc,
                        const Params& p_in, cudaStream_t st, const CUtensorMap* tv = nullptr, const CUtensorMap* tv2 = nullptr,
                        bool pdl = false) {
  Params p = p_in;
  const int slots = PAIR ? pair_slots() : sm_count();
  if (EPI != gemm::EPI_F32_CLUSTER && p.total_units == 0) {  // the caller planned no order: every N-tile whole-cost
    const bool column_halves = PAIR && MT == 1 && SKETCH == gemm::SKETCH_NONE && p.bn == gemm::kMaxBN && p.N % p.bn == 0;
    plan_units(&p, p.n_tiles, 1.0, (MT == 2 && p.splits == 1) || column_halves, slots, column_halves ? kColumnHalfCost : kCutTileCost);
  }
  using C = gemm::Cfg<MT, BROWS, PAIR>;
  auto kernel = gemm::umma_gemm_kernel<A_MN, B_MN, SKETCH, EPI, MT, BROWS, PAIR>;
  static DeviceOnce once;  // per instantiation
  if (once.needed()) {
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes);
    if (e != cudaSuccess) return e;
    once.done();
  }
  const int tiles = p.total_units;
  if (tiles == 0) return cudaSuccess;
  const int grid = std::min(tiles, slots) * (PAIR ? 2 : 1);
  if (pdl || PAIR) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(unsigned(grid));
    cfg.blockDim = dim3(unsigned(C::threads(SKETCH == gemm::SKETCH_GENERATED)));
    cfg.dynamicSmemBytes = C::kSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    int n_attr = 0;
    if (pdl) {
      attr[n_attr].id = cudaLaunchAttributeProgrammaticStreamSerialization;
      attr[n_attr].val.programmaticStreamSerializationAllowed = 1;
      ++n_attr;
    }
    if (PAIR) {
      attr[n_attr].id = cudaLaunchAttributeClusterDimension;
      attr[n_attr].val.clusterDim.x = 2;
      attr[n_attr].val.clusterDim.y = 1;
      attr[n_attr].val.clusterDim.z = 1;
      ++n_attr;
    }
    cfg.attrs = attr;
    cfg.numAttrs = unsigned(n_attr);
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, ta, tb, tb2, tc, tv ? *tv : ta, tv2 ? *tv2 : ta, p);
    kernel_launch_counter().fetch_add(1, std::memory_order_relaxed);
    return e;
  }
  kernel<<<grid, C::threads(SKETCH == gemm::SKETCH_GENERATED), C::kSmemBytes, st>>>(ta, tb, tb2, tc, tv ? *tv : ta, tv2 ? *tv2 : ta, p);
  return launched();
}

int pair_slots() {
  static int cache[64] = {0};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return std::max(1, sm_count() / 2);
  if (cache[dev] == 0) {
    using C = gemm::Cfg<2, gemm::kMaxBN, true>;
    auto kernel = gemm::umma_gemm_kernel<false, false, gemm::SKETCH_NONE, gemm::EPI_BF16, 2, gemm::kMaxBN, true>;
    int n = 0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2);
    cfg.blockDim = dim3(unsigned(C::threads(false)));
    cfg.dynamicSmemBytes = C::kSmemBytes;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes) != cudaSuccess ||
        cudaOccupancyMaxActiveClusters(&n, kernel, &cfg) != cudaSuccess || n <= 0) {
      (void)cudaGetLastError();
      n = std::max(1, sm_count() / 2);
    }
    cache[dev] = n;
  }
  return cache[dev];
}

// Row blocks per CTA tile for the forward and dX: 256-row tiles halve the L2 and shared-memory traffic of B (and
// the sketch generation of the forward) per flop; 128-row tiles give twice as many tiles to spread over the SMs.
// Cost = rounds of tiles x tile time, with the measured relative speed of the two mainloops.
// Returns 1 or 2 (row blocks of one CTA's tile), or 3 / 4: a CTA pair on a 256- / 512-row tile (when pair_tiles > 0
// N-tiles of the pair layout are given).
// Test/debug override of the cost models (acx_debug_force_gemm_mode): 0 = none, 1 / 2 = row blocks of one CTA's tile,
// 3 / 4 = a CTA pair on 256- / 512-row tiles.  A mode that a kernel variant does not exist for is ignored.
std::atomic<int>& forced_gemm_mode() {
  static std::atomic<int> mode{0};
  return mode;
}
#define ACX_FORCE_GEMM_MODE (forced_gemm_mode().load(std::memory_order_relaxed))
// speed3 / speed4: time per flop of the two pair modes relative to the 128-row tile of one CTA (0 = mode not offered).
int pick_row_blocks(int64_t m, int n_tiles, double kRowBlocks2Speed, int pair_tiles = 0, double speed3 = 0.0, double speed4 = 0.0) {
  const int sms = sm_count();
  Params p1{}, p2{}, p4{};
  p1.n_tiles = p2.n_tiles = n_tiles;
  p1.splits = p2.splits = p4.splits = 1;
  p1.m_tiles = int((m + 127) / 128);
  p2.m_tiles = int((m + 255) / 256);
  const double c1 = plan_units(&p1, n_tiles, 1.0, false, sms) * 1.0;
  const double c2 = plan_units(&p2, n_tiles, 1.0, true, sms) * 2.0 * kRowBlocks2Speed;
  int best = c2 < c1 ? 2 : 1;
  if (pair_tiles > 0) {
    Params p3{};
    p3.splits = 1;
    p3.n_tiles = p4.n_tiles = pair_tiles;
    p3.m_tiles = int((m + 255) / 256);
    p4.m_tiles = int((m + 511) / 512);
    // a CTA's share of a pair tile: 128 or 256 rows
    const double c3 = speed3 > 0 ? plan_units(&p3, pair_tiles, 1.0, false, pair_slots()) * 1.0 * speed3 : 1e300;
    const double c4 = speed4 > 0 ? plan_units(&p4, pair_tiles, 1.0, true, pair_slots()) * 2.0 * speed4 : 1e300;
    double cb = std::min(c1, c2);
    if (c3 < cb) { best = 3; cb = c3; }
    if (c4 < cb) best = 4;
    if (ACX_FORCE_GEMM_MODE == 3 || ACX_FORCE_GEMM_MODE == 4) best = ACX_FORCE_GEMM_MODE;
  }
  if (ACX_FORCE_GEMM_MODE == 1 || ACX_FORCE_GEMM_MODE == 2) best = ACX_FORCE_GEMM_MODE;
  return best;
}

// Time per flop of the pair kernels relative to the 128-row tile of one CTA, measured at the LLaMA-3B shapes
// (16384 tokens; the 256-row tile of one CTA is 0.905).  A pair on 256-row tiles (two accumulator sets per CTA: the
// epilogue never holds up the tensor core) is the fastest for the plain product and for a sketch read from memory.
// With the sketch generated in place it is the slowest (a CTA then has half the time per slice element), and a pair
// on 512-row tiles, which generates each slice once per 512 rows, pays off from about 192 sketch columns on.
constexpr double kPair256Speed = 0.85, kPair512Speed = 0.905, kPair512SpeedGenWide = 0.87;
// (With the 512-row pair at every rank the step under sustained load measured the same as with one CTA per tile,
// 6.20-6.21 against 6.21-6.24 ms at r = 128; alone it was 7 % faster at d_in = 8192, equal at 3072 -> 3072, 2 % slower at
// 3072 -> 8192.)
constexpr int kGenPair512MinRank = 192;


// Forward tile shapes.  The r columns of S are spread over the N-tiles as evenly as multiples of 8 allow,
// so that every tile brings about the same amount of generation work for its MMA time: with T tiles,
// (r/8) mod T of them carry 8*(r/8/T + 1) columns and 256 minus that many rows of W, the others one
// multiple of 8 less.  T is the smallest count whose W rows cover d_out with at most 128 columns of S per tile;
// T = ceil(d_out / 128) + 1 always qualifies (r <= 256 gives at most 128 columns per tile from two tiles on, and
// every tile then still has 128 rows for W), so the search cannot fail for a valid descriptor.
// gran = 8, or 16 for a CTA pair (each CTA stages half of the slice and half of the W rows, both multiples of 8).
bool fwd_shape(const Problem& q, Params* p, int gran = 8) {
  const int units = q.r / gran;
  const int t_min = int((q.d_out + 255) / 256), t_max = int((q.d_out + 127) / 128) + 1;
  for (int T = t_min; T <= t_max; ++T) {
    const int base = units / T, extra = units % T;
    const int sw1 = gran * (base + 1), sw0 = gran * base;
    if ((extra ? sw1 : sw0) > 128) continue;
    const int64_t covered = int64_t(extra) * (256 - sw1) + int64_t(T - extra) * (256 - sw0);
    if (covered < q.d_out) continue;
    p->n_class1 = extra; p->bn1 = 256 - sw1; p->sw1 = sw1; p->bn0 = 256 - sw0; p->sw0 = sw0;
    p->n_tiles = T;
    return true;
  }
  return false;
}

struct FactorPlan { int splits, kb_per_split; bool cluster; double cost; };

// Split of the token range whose partial sums go through global memory (workspace + reduce kernel).
// A token range is added up in one fp32 tensor-core accumulator, whose rounding error grows with the length of that
// chain (1.4e-4 relative at 125 000 tokens per range, 1e-6 at 3 000): ranges are kept to at most this many k-blocks
// (65 536 tokens) where the split count allows it.
constexpr int kMaxChainKb = 1024;

FactorPlan factor_plan(const Problem& q) {
  const int m_tiles = int((q.d_out + gemm::kBM - 1) / gemm::kBM);
  const int num_kb = int((q.m + gemm::kBK - 1) / gemm::kBK);
  const int sms = sm_count();
  int best_s = 1;
  double best_cost = 1e30;
  const int max_s = std::max(1, std::min(std::max(32, std::min(128, (num_kb + kMaxChainKb - 1) / kMaxChainKb)), num_kb / 4));
  for (int s = 1; s <= max_s; ++s) {
    const int kbs = (num_kb + s - 1) / s;
    if (kbs > kMaxChainKb && s < max_s) continue;
    const int real_s = (num_kb + kbs - 1) / kbs;
    const int waves = (m_tiles * real_s + sms - 1) / sms;
    // 6 k-block times per tile for pipeline ramp-up and the epilogue
    const double cost = double(waves) * (kbs + 6.0) + 0.5 * real_s + (real_s > 1 ? 2.0 : 0.0);
    if (cost < best_cost) { best_cost = cost; best_s = real_s; }
  }
  FactorPlan f;
  f.kb_per_split = (num_kb + best_s - 1) / best_s;
  f.splits = std::max(1, (num_kb + f.kb_per_split - 1) / f.kb_per_split);
  f.cluster = false;
  f.cost = best_cost + (f.splits > 1 ? 8.0 : 0.0);  // the reduce kernel and the gap before it, in k-block times
  return f;
}

// The cluster kernel comes with wide (r > 128) and narrow B stages.
template <int BROWS>
cudaError_t configure_cluster_kernel() {
  static DeviceOnce once;
  if (!once.needed()) return cudaSuccess;
  cudaError_t e = cudaFuncSetAttribute(gemm::umma_gemm_kernel<true, true, false, gemm::EPI_F32_CLUSTER, 1, BROWS>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, gemm::Cfg<1, BROWS>::kSmemBytes);
  if (e == cudaSuccess) once.done();
  return e;
}

cudaLaunchConfig_t cluster_config(int ctas, int cluster, cudaStream_t st, cudaLaunchAttribute* attr) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(unsigned(ctas));
  cfg.blockDim = dim3(gemm::Cfg<1>::threads(false));
  cfg.dynamicSmemBytes = gemm::Cfg<1>::kSmemBytes;  // both variants: 4 x 48 KiB = 6 x 32 KiB of stages
  cfg.stream = st;
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = unsigned(cluster);
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cfg;
}

// Clusters of `size` CTAs of the factor kernel that the device can hold at once (cached; an estimate
// from the SM count where the device cannot be asked).
int max_resident_clusters(int size) {
  static int cache[9] = {0};
  if (cache[size] == 0) {
    int n = 0;
    cudaLaunchAttribute attr[1];
    cudaLaunchConfig_t cfg = cluster_config(size, size, nullptr, attr);
    if (configure_cluster_kernel<gemm::kMaxBN>() != cudaSuccess ||
        cudaOccupancyMaxActiveClusters(&n, gemm::umma_gemm_kernel<true, true, false, gemm::EPI_F32_CLUSTER, 1, gemm::kMaxBN>, &cfg) != cudaSuccess ||
        n <= 0) {
      (void)cudaGetLastError();
      n = std::max(1, sm_count() / size);
    }
    cache[size] = n;
  }
  return cache[size];
}

// The plan acx_linear_bwd uses: the splits of one output tile either form a thread-block cluster of 2 to 8
// CTAs that adds its partial sums over distributed shared memory, or go through the workspace.  How many
// clusters of a size the GPU holds at once is asked of the driver (e.g. 26 of 5 but only 22 of 6 on a B200).
FactorPlan factor_plan_public(const Problem& q) {
  FactorPlan best = factor_plan(q);
  const int m_tiles = int((q.d_out + gemm::kBM - 1) / gemm::kBM);
  const int num_kb = int((q.m + gemm::kBK - 1) / gemm::kBK);
  for (int s = 2; s <= 8; ++s) {
    if (s > num_kb / 4) break;
    const int kbs = (num_kb + s - 1) / s;
    if ((num_kb + kbs - 1) / kbs != s) continue;  // no empty split inside a cluster
    if (kbs > kMaxChainKb) continue;               // the workspace path can split further
    const int resident = max_resident_clusters(s);
    const int waves = (m_tiles + resident - 1) / resident;
    const double cost = double(waves) * (kbs + 6.0) + 0.25 * s + 1.0;
    if (cost < best.cost) best = FactorPlan{s, kbs, true, cost};
  }
  return best;
}

__global__ void __launch_bounds__(256) reduce_splits_kernel(const float4* __restrict__ part, float4* __restrict__ out, int64_t n4,
                                                            int splits) {
  const int64_t i = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i >= n4) return;
  float4 s = part[i];
  for (int z = 1; z < splits; ++z) {
    const float4 v = part[int64_t(z) * n4 + i];
    s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
  }
  out[i] = s;
}

}  // namespace

// Bytes of split-K partials the factor needs when they go through global memory.
size_t sm100_factor_scratch_bytes(const Problem& q) {
  if (q.m == 0) return 0;
  const FactorPlan f = factor_plan(q);
  return f.splits > 1 ? size_t(f.splits) * size_t(q.d_out) * size_t(q.r) * sizeof(float) : 0;
}

// Workspace of acx_linear_bwd: none when the splits are reduced inside a cluster.
size_t sm100_bwd_workspace_bytes(const Problem& q) {
  if (q.m == 0) return 0;
  return factor_plan_public(q).cluster ? 0 : sm100_factor_scratch_bytes(q);
}

// Tile shape of a plain GEMM (dX = G W, or Y = X W^T without sketch): (row blocks, N-tile width) among 128 x 256, 256 x 256 and 256 x 192.  Cost in k-block
// units of a 128 x 256 tile = rounds of tiles x (mainloop + what does not overlap), with relative mainloop speeds
// and the per-tile overhead of the 256-row tile (its epilogue only partly overlaps the next tile) measured at the
// LLaMA-3B shapes; 128-row tiles re-read a W that does not fit L2 comfortably (> 32 MB) more often.
struct DxPlan { int row_blocks, bn; };   // row_blocks 3 / 4: a CTA pair on 256- / 512-row tiles

// n = output columns, k = contraction length of the plain GEMM (dX: n = d_in, k = d_out; forward without
// sketch: n = d_out, k = d_in).
DxPlan gemm_plan(int64_t m, int64_t n, int64_t k) {
  const int sms = sm_count();
  const double num_kb = double((k + gemm::kBK - 1) / gemm::kBK);
  const bool big_w = double(n) * double(k) * 2.0 > 32e6;
  // (192-column tiles of a pair would fill the last round of tiles better at 3072 columns, but ran 12-37 % slower.)
  const struct { int mt, bn; double speed, overhead; } cand[5] = {
      {1, 256, big_w ? 1.08 : 1.0, 0.0}, {2, 256, 0.905, 5.0}, {2, 192, 1.0, 1.0}, {3, 256, kPair256Speed, 0.0}, {4, 256, kPair512Speed, 5.0}};
  DxPlan best{1, 256};
  double best_cost = 1e300;
  for (const auto& c : cand) {
    Params t{};
    const int cta_blocks = c.mt >= 3 ? c.mt - 2 : c.mt;                  // row blocks one CTA multiplies per tile
    const int tile_rows = 128 * cta_blocks * (c.mt >= 3 ? 2 : 1);
    t.m_tiles = int((m + tile_rows - 1) / tile_rows);
    t.n_tiles = int((n + c.bn - 1) / c.bn);
    t.splits = 1;
    const double rounds = plan_units(&t, t.n_tiles, 1.0, cta_blocks == 2, c.mt >= 3 ? pair_slots() : sms);
    const double cost = rounds * (cta_blocks * (c.bn / 256.0) * num_kb * c.speed + c.overhead);
    if (cost < best_cost) { best_cost = cost; best = DxPlan{c.mt, c.bn}; }
    if (ACX_FORCE_GEMM_MODE == c.mt && (c.bn == 256)) return DxPlan{c.mt, c.bn};
  }
  return best;
}

// Row tiles of a GEMM mode: 1, 2 = row blocks of one CTA's tile; 3, 4 = a CTA pair on 256- or 512-row tiles.
int tiles_along_m(int64_t m, int mode) {
  const int rows = mode >= 3 ? 256 * (mode - 2) : 128 * mode;
  return int((m + rows - 1) / rows);
}

// Y = X W^T alone (the factor of this input is stored by another linear): the plain mainloop, B K-major.
cudaError_t sm100_fwd_plain(const Problem& q, const void* X, const void* W, void* Y, int* status, cudaStream_t st,
                            const void* bias) {
  Params p{};
  p.bias = bias;
  const DxPlan plan = gemm_plan(q.m, q.d_out, q.d_in);
  const int mt = plan.row_blocks;
  p.M = int(q.m); p.N = int(q.d_out); p.K = int(q.d_in);
  p.bn = plan.bn;
  p.n_tiles = (p.N + p.bn - 1) / p.bn;
  p.m_tiles = tiles_along_m(q.m, mt);
  p.splits = 1; p.kb_per_split = (p.K + gemm::kBK - 1) / gemm::kBK;
  p.C = Y; p.ldc = q.d_out; p.status = status;
  CUtensorMap ta, tb, tc;
  if (!make_tmap_bf16(&ta, X, q.m, q.d_in, gemm::kBK, gemm::kBM)) return cudaErrorInvalidValue;  // one box per row block
  if (!make_tmap_bf16(&tb, W, q.d_out, q.d_in, gemm::kBK, mt >= 3 ? p.bn / 2 : p.bn)) return cudaErrorInvalidValue;  // a pair: half the rows per CTA
  if (!make_tmap_bf16_store_sw64(&tc, Y, q.m, q.d_out)) return cudaErrorInvalidValue;
  if (mt == 4) return launch_gemm<false, false, false, gemm::EPI_BF16, 2, gemm::kMaxBN, true>(ta, tb, tb, tc, p, st);
  if (mt == 3) {  // the boxes of a column half of a tile (the last round's tiles may be cut in two): a quarter of the rows per CTA
    CUtensorMap tb2;
    if (!make_tmap_bf16(&tb2, W, q.d_out, q.d_in, gemm::kBK, p.bn / 4)) return cudaErrorInvalidValue;
    return launch_gemm<false, false, false, gemm::EPI_BF16, 1, gemm::kMaxBN, true>(ta, tb, tb2, tc, p, st);
  }
  if (mt == 2) return launch_gemm<false, false, false, gemm::EPI_BF16, 2>(ta, tb, tb, tc, p, st);
  return launch_gemm<false, false, false, gemm::EPI_BF16>(ta, tb, tb, tc, p, st);
}

size_t sm100_fwd_workspace_bytes(const Problem& q) { return size_t(q.r) * size_t(q.d_in) * 2; }

cudaError_t sm100_fwd(const Problem& q, const void* X, const void* W, void* Y, void* XS, int* status, cudaStream_t st,
                      const void* Vt, void* ws, const void* bias) {
  if (!XS) return sm100_fwd_plain(q, X, W, Y, status, st, bias);
  bool pdl = false;
  if (!Vt && ws) {  // the seeded sketch, written out once instead of once per row-tile
    const int64_t threads = (q.d_in / 2) * int64_t(q.r / 4);
    sketch_transposed_kernel<<<unsigned((threads + 255) / 256), 256, 0, st>>>(static_cast<__nv_bfloat16*>(ws), q.d_in, q.r, q.sp);
    const cudaError_t e = launched();
    if (e != cudaSuccess) return e;
    Vt = ws;
    pdl = true;
  }
  Params p{};
  if (!fwd_shape(q, &p)) return cudaErrorInvalidValue;
  Params pp{};   // the layout for a CTA pair: slices in multiples of 16 columns
  const bool pair_ok = fwd_shape(q, &pp, 16);
  p.M = int(q.m); p.N = int(q.d_out); p.K = int(q.d_in);
  const bool generated = !Vt;   // (a written-out seeded sketch has become Vt above)
  const int mt = pick_row_blocks(q.m, p.n_tiles, kFwdRowBlocks2Speed, pair_ok ? pp.n_tiles : 0, generated ? 0.0 : kPair256Speed,
                                 generated ? (q.r >= kGenPair512MinRank ? kPair512SpeedGenWide : 0.0) : 0.0);
  const bool pair = mt >= 3;
  if (pair) { pp.M = p.M; pp.N = p.N; pp.K = p.K; p = pp; }
  const int slots = pair ? pair_slots() : sm_count();
  p.m_tiles = tiles_along_m(q.m, mt);
  p.splits = 1; p.kb_per_split = (p.K + gemm::kBK - 1) / gemm::kBK;
  if (Vt) {
    // A sketch that is read from memory need not be spread over the W tiles (nothing is generated per tile):
    // the alternative is whole 256-column W tiles plus one cheap tile per row-tile that carries all r sketch
    // columns and goes to the last round.  Take whichever order ends sooner.
    const bool may_cut = mt == 2 || mt == 4;
    const bool column_halves = mt == 3 && q.d_out % 256 == 0;   // a pair on 256-row tiles: whole W tiles may be cut in column halves
    const double mixed = plan_units(&p, p.n_tiles, 1.0, may_cut, slots);
    const double sketch_tile_cost = kCutTileCost + 0.2 * (std::max(q.r, 128) - 128) / 128.0;  // like a cut tile up to r = 128
    Params s = p;
    const int n_w = int((q.d_out + 255) / 256);
    s.n_class1 = n_w; s.bn1 = 256; s.sw1 = 0; s.bn0 = 0; s.sw0 = q.r;
    s.n_tiles = n_w + 1;
    const double apart = plan_units(&s, n_w, sketch_tile_cost, may_cut || column_halves, slots, column_halves ? kColumnHalfCost : kCutTileCost);
    if (apart < mixed) p = s;
  } else if (pair) {
    plan_units(&p, p.n_tiles, 1.0, mt == 4, slots);
  }
  p.r = q.r; p.sp = q.sp;
  p.C = Y; p.ldc = q.d_out; p.C2 = XS; p.ldc2 = q.r; p.status = status;
  p.bias = bias;
  const int div = pair ? 2 : 1;   // a CTA of a pair stages half of the W rows and half of the slice
  CUtensorMap ta, tb, tb2, tc;
  if (!make_tmap_bf16(&ta, X, q.m, q.d_in, gemm::kBK, gemm::kBM)) return cudaErrorInvalidValue;  // one box per row block
  if (!make_tmap_bf16(&tb, W, q.d_out, q.d_in, gemm::kBK, std::max(p.bn1 / div, 8))) return cudaErrorInvalidValue;
  // second W map: the boxes of the other tile class, or (that class has no W rows) of a column half of the first one
  const int tb2_rows = p.bn0 > 0 ? p.bn0 / div : (mt == 3 ? p.bn1 / 4 : 8);
  if (!make_tmap_bf16(&tb2, W, q.d_out, q.d_in, gemm::kBK, std::max(tb2_rows, 8))) return cudaErrorInvalidValue;
  if (!make_tmap_bf16_store_sw64(&tc, Y, q.m, q.d_out)) return cudaErrorInvalidValue;
  if (Vt) {  // the second factor comes from memory: V^T is r x d_in, its slices go below the W rows of each B tile
    CUtensorMap tv, tv2;
    if (!make_tmap_bf16(&tv, Vt, q.r, q.d_in, gemm::kBK, std::max(p.sw1 / div, 8))) return cudaErrorInvalidValue;
    if (!make_tmap_bf16(&tv2, Vt, q.r, q.d_in, gemm::kBK, std::max(p.sw0 / div, 8))) return cudaErrorInvalidValue;
    if (mt == 4) return launch_gemm<false, false, gemm::SKETCH_LOADED, gemm::EPI_BF16, 2, gemm::kMaxBN, true>(ta, tb, tb2, tc, p, st, &tv, &tv2, pdl);
    if (mt == 3) return launch_gemm<false, false, gemm::SKETCH_LOADED, gemm::EPI_BF16, 1, gemm::kMaxBN, true>(ta, tb, tb2, tc, p, st, &tv, &tv2, pdl);
    if (mt == 2) return launch_gemm<false, false, gemm::SKETCH_LOADED, gemm::EPI_BF16, 2>(ta, tb, tb2, tc, p, st, &tv, &tv2, pdl);
    return launch_gemm<false, false, gemm::SKETCH_LOADED, gemm::EPI_BF16>(ta, tb, tb2, tc, p, st, &tv, &tv2, pdl);
  }
  if (!pair) {
    // The last N-tile with only part of its W columns inside d_out: as many W rows as exist (rounded so that rows + slice
    // are a multiple of 16), a narrower MMA, and its own box height.
    const int last = p.n_tiles - 1;
    const bool last_class1 = last < p.n_class1;
    const int n0_last = last_class1 ? last * p.bn1 : p.n_class1 * p.bn1 + (last - p.n_class1) * p.bn0;
    const int bn_class = last_class1 ? p.bn1 : p.bn0, sw_class = last_class1 ? p.sw1 : p.sw0;
    const int s0_last = last_class1 ? last * p.sw1 : p.n_class1 * p.sw1 + (last - p.n_class1) * p.sw0;
    const int width_last = std::max(0, std::min(sw_class, q.r - s0_last));
    const int real = int(q.d_out) - n0_last;
    if (real > 0 && width_last > 0) {
      int rows = (real + 7) & ~7;
      if ((rows + width_last) % 16) rows += 8;
      if (rows < bn_class) {
        CUtensorMap tbl;
        if (!make_tmap_bf16(&tbl, W, q.d_out, q.d_in, gemm::kBK, rows)) return cudaErrorInvalidValue;
        p.bn_last = rows;
        if (mt == 2) return launch_gemm<false, false, gemm::SKETCH_GENERATED, gemm::EPI_BF16, 2>(ta, tb, tb2, tc, p, st, &tbl);
        return launch_gemm<false, false, gemm::SKETCH_GENERATED, gemm::EPI_BF16>(ta, tb, tb2, tc, p, st, &tbl);
      }
    }
  }
  if (mt == 4) return launch_gemm<false, false, gemm::SKETCH_GENERATED, gemm::EPI_BF16, 2, gemm::kMaxBN, true>(ta, tb, tb2, tc, p, st);
  if (mt == 3) return launch_gemm<false, false, gemm::SKETCH_GENERATED, gemm::EPI_BF16, 1, gemm::kMaxBN, true>(ta, tb, tb2, tc, p, st);
  if (mt == 2) return launch_gemm<false, false, gemm::SKETCH_GENERATED, gemm::EPI_BF16, 2>(ta, tb, tb2, tc, p, st);
  return launch_gemm<false, false, gemm::SKETCH_GENERATED, gemm::EPI_BF16>(ta, tb, tb2, tc, p, st);
}

cudaError_t sm100_dx(const Problem& q, const void* G, const void* W, void* dX, int* status, cudaStream_t st) {
  Params p{};
  p.M = int(q.m); p.N = int(q.d_in); p.K = int(q.d_out);
  const DxPlan plan = gemm_plan(q.m, q.d_in, q.d_out);
  const int mt = plan.row_blocks;
  p.bn = plan.bn;
  p.n_tiles = (p.N + p.bn - 1) / p.bn;
  p.m_tiles = tiles_along_m(q.m, mt);
  p.splits = 1; p.kb_per_split = (p.K + gemm::kBK - 1) / gemm::kBK;
  p.C = dX; p.ldc = q.d_in; p.status = status;
  CUtensorMap ta, tb, tc;
  if (!make_tmap_bf16(&ta, G, q.m, q.d_out, gemm::kBK, gemm::kBM)) return cudaErrorInvalidValue;  // one box per row block
  if (!make_tmap_bf16(&tb, W, q.d_out, q.d_in, 64, gemm::kBK)) return cudaErrorInvalidValue;  // MN-major chunks: 64 d_in x 64 d_out
  if (!make_tmap_bf16_store_sw64(&tc, dX, q.m, q.d_in)) return cudaErrorInvalidValue;
  if (mt == 4) return launch_gemm<false, true, false, gemm::EPI_BF16, 2, gemm::kMaxBN, true>(ta, tb, tb, tc, p, st);
  if (mt == 3) return launch_gemm<false, true, false, gemm::EPI_BF16, 1, gemm::kMaxBN, true>(ta, tb, tb, tc, p, st);
  if (mt == 2) return launch_gemm<false, true, false, gemm::EPI_BF16, 2>(ta, tb, tb, tc, p, st);
  return launch_gemm<false, true, false, gemm::EPI_BF16>(ta, tb, tb, tc, p, st);
}

// after_dx: the grid launched just before on this stream is the dX kernel of the same call.  The factor reads nothing
// that dX writes, so it is launched with programmatic stream serialization and never waits for it: its thread blocks
// take over the SMs as the dX kernel's last round of tiles leaves them idle.
cudaError_t sm100_factor(const Problem& q, const void* G, const void* XS, float* A, void* ws, int* status, cudaStream_t st,
                         bool allow_cluster, float* db_part, int* db_splits, bool after_dx) {
  const FactorPlan f = allow_cluster ? factor_plan_public(q) : factor_plan(q);
  Params p{};
  p.colsum_part = db_part;
  if (db_splits) *db_splits = f.splits;
  p.M = int(q.d_out); p.N = q.r; p.K = int(q.m);
  p.bn = 256;
  p.m_tiles = int((q.d_out + gemm::kBM - 1) / gemm::kBM);
  p.n_tiles = 1;
  p.splits = f.splits; p.kb_per_split = f.kb_per_split;
  p.ldc = q.r; p.status = status;
  p.c_split_stride = q.d_out * int64_t(q.r);
  p.C = (f.splits > 1 && !f.cluster) ? ws : static_cast<void*>(A);
  CUtensorMap ta, tb;
  if (!make_tmap_bf16(&ta, G, q.m, q.d_out, 64, gemm::kBK)) return cudaErrorInvalidValue;   // A(m = o, k = t): 64 d_out x 64 tokens
  if (!make_tmap_bf16(&tb, XS, q.m, q.r, 64, gemm::kBK)) return cudaErrorInvalidValue;      // B(n = j, k = t): 64 r x 64 tokens
  const bool narrow = q.r <= 128;  // B stage of 128 rows: six stages instead of four
  if (f.cluster) {
    cudaError_t ec = narrow ? configure_cluster_kernel<128>() : configure_cluster_kernel<gemm::kMaxBN>();
    if (ec != cudaSuccess) return ec;
    cudaLaunchAttribute attr[2];
    cudaLaunchConfig_t cfg = cluster_config(p.m_tiles * p.splits, p.splits, st, attr);
    if (after_dx) {
      attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
      attr[1].val.programmaticStreamSerializationAllowed = 1;
      cfg.numAttrs = 2;
    }
    ec = narrow ? cudaLaunchKernelEx(&cfg, gemm::umma_gemm_kernel<true, true, false, gemm::EPI_F32_CLUSTER, 1, 128>, ta, tb, tb, tb, tb, tb, p)
                : cudaLaunchKernelEx(&cfg, gemm::umma_gemm_kernel<true, true, false, gemm::EPI_F32_CLUSTER, 1, gemm::kMaxBN>, ta, tb, tb, tb, tb, tb, p);
    kernel_launch_counter().fetch_add(1, std::memory_order_relaxed);
    return ec;
  }
  cudaError_t e = narrow ? launch_gemm<true, true, false, gemm::EPI_F32_SPLIT, 1, 128>(ta, tb, tb, tb, p, st, nullptr, nullptr, after_dx)
                         : launch_gemm<true, true, false, gemm::EPI_F32_SPLIT>(ta, tb, tb, tb, p, st, nullptr, nullptr, after_dx);
  if (e != cudaSuccess || f.splits == 1) return e;
  const int64_t n4 = q.d_out * int64_t(q.r) / 4;
  reduce_splits_kernel<<<unsigned((n4 + 255) / 256), 256, 0, st>>>(static_cast<const float4*>(ws), reinterpret_cast<float4*>(A), n4,
                                                                  f.splits);
  return launched();
}

void sm100_force_gemm_mode(int mode) { forced_gemm_mode().store(mode, std::memory_order_relaxed); }

}  // namespace acx

// ---- gradient factor with scratch that is part of the library image ---------------------------------
// For callers that cannot allocate device memory where the backward pass runs: the split-K partial
// sums of the factor kernel go to this fixed array instead of a caller's workspace.  The name below is
// only a host-side handle; the kernels need the device address, which cudaGetSymbolAddress gives for
// the device that is current, so it is looked up once per device and cached.
static __device__ __align__(256) unsigned char g_builtin_scratch[ACX_BUILTIN_SCRATCH_BYTES];

namespace acx {
namespace {

// Device address of g_builtin_scratch on the current device, or nullptr on a CUDA error.
void* builtin_scratch_ptr() {
  static std::mutex mu;
  static void* cache[64] = {nullptr};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> lock(mu);
  if (!cache[dev]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_builtin_scratch) != cudaSuccess || !ptr) return nullptr;
    cache[dev] = ptr;
  }
  return cache[dev];
}

}  // namespace
}  // namespace acx

extern "C" acx_status acx_linear_bwd_factor_builtin_scratch(const acx_desc* desc, const void* G_out, const void* XS,
                                                            float* dW_A, void* cuda_stream) {
  using namespace acx;
  Problem p;
  acx_status s = validate(desc, &p);
  if (s != ACX_OK) return s;
  if (!p.bf16) return ACX_ERR_INVALID_ARG;
  if (!dW_A) return ACX_ERR_INVALID_ARG;
  auto misaligned = [](const void* q) { return (reinterpret_cast<uintptr_t>(q) & 15u) != 0; };
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (p.m == 0) {
    if (misaligned(dW_A)) return ACX_ERR_ALIGNMENT;
    return cudaMemsetAsync(dW_A, 0, sizeof(float) * size_t(p.d_out) * size_t(p.r), st) == cudaSuccess ? ACX_OK : ACX_ERR_CUDA;
  }
  if (!G_out || !XS) return ACX_ERR_INVALID_ARG;
  if (misaligned(G_out) || misaligned(XS) || misaligned(dW_A)) return ACX_ERR_ALIGNMENT;
  if (sm100_factor_scratch_bytes(p) > size_t(ACX_BUILTIN_SCRATCH_BYTES)) return ACX_ERR_SCRATCH_LIMIT;
  void* scratch = builtin_scratch_ptr();
  int* status = device_status_ptr();
  if (!scratch || !status) return ACX_ERR_CUDA;
  return sm100_factor(p, G_out, XS, dW_A, scratch, status, st, /*allow_cluster=*/false) == cudaSuccess ? ACX_OK : ACX_ERR_CUDA;
}
