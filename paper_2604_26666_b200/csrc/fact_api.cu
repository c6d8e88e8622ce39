// Host side of libfact: argument validation, configuration choice, tensor-map
// encoding, kernel launch, the tile-configuration tuner and its table.
// Declarations and per-call contracts are in include/fact.h.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <array>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <bitset>
#include <map>
#include <memory>
#include <queue>
#include <string>
#include <tuple>
#include <utility>
#include <vector>

#include "fact.h"
#include "gemm_kernel.cuh"
#include "kcluster_kernel.cuh"
#include "attention_kernel.cuh"
#include "norm_kernel.cuh"
#include "tune_kernels.cuh"

// Storage of fact_gemm_splitk_static: split-K scratch and a status word that live in the library's own
// device image, so that entry point never has to allocate.  Every GPU that loads the library holds these
// 16 MiB until the process exits.  In host code these names are only stand-ins for the device symbols; the
// device addresses the kernels get come from cudaGetSymbolAddress (see static_setup below).
constexpr size_t kStaticScratchBytes = (size_t)16 << 20;
constexpr int kStaticStatusInts = 64;  // the words a split-K launch touches: error word, clock stamps, grid-barrier counters
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];
static __device__ __align__(256) int g_static_status[kStaticStatusInts];

namespace {

using namespace fact;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

constexpr int kSmemBudget = 227 * 1024;  // dynamic shared memory per CTA: the whole 227 KB opt-in limit (no static
                                         // shared memory is used; the kernel checks the 1024-byte alignment of its base)
constexpr int kMinSmemRequest = 120 * 1024;  // > half an SM: one CTA per SM, so TMEM allocation never blocks
constexpr int kStatusInts = 64;  // status word, clock / profile counters, grid-barrier counters; stream-K flags follow
constexpr int kDiagnosticFlags = 256 | 2048 | 4096 | 8192;  // FACT_DEBUG_FLAGS bits that leave results intact: cycle
                                                             // counters, no K serpentine, no programmatic dependent
                                                             // launch, no L2 eviction priority on operand loads
constexpr int kMaxGroups = 4096;  // row groups of a grouped GEMM (the handle's device table holds 2 x (kMaxGroups + 1) ints)

// Key of the tuner's table: everything that changes which configuration is best.
typedef std::tuple<int, int, int, int, long long, long long, long long, long long> TuneKey;

struct Problem {
  fact_op_t op;
  long long batch, M, N_out, K;
  const void* A;
  long long lda, strideA;
  const void* B;
  long long ldb, strideB;
  fact_blayout_t layout;
  const void* bias;
  const void* R;
  long long ldr, strideR;
  void* C;
  long long ldc, strideC;
  fact_out_t out;
  fact_epilogue_t epi;
  int groups = 0;                        // > 0: grouped GEMM, A and C rows in consecutive groups, B = W[group]
  const int64_t* group_rows = nullptr;   // host: rows of each group
  bool fp8 = false;    // operands are FP8 E4M3 (one byte per element) instead of BF16
  float alpha = 1.f;   // FP8: the accumulator is multiplied by this before the epilogue
  float* stats_out = nullptr;       // partial row sums of the stored output, for a normalisation folded into the next call
  const float* stats_in = nullptr;  // partial row sums of A from the call that produced it
  int norm = 0;                     // 0: none; 1: A's rows are layer-normalised over K; 2: RMS-normalised
  const float* colsum = nullptr;    // norm == 1: sum over k of the folded W[n][k]
  float norm_eps = 0.f;
  long long Nw() const { return epi == FACT_EPI_SILU_GATE ? 2 * N_out : N_out; }
  int k_elems() const { return fp8 ? 2 * kTileK : kTileK; }  // elements of K in a 128-byte row of a stage
  int op_align() const { return fp8 ? 16 : 8; }              // elements in 16 bytes of an operand
};

struct Plan {
  fact_config_t cfg;
  bool from_table = false;  // cfg came from the tuner's table: its store mode and K slices are hints, not demands
  bool dynamic = false;     // tiles are handed out through cluster launch control (one cluster of the grid per tile)
  bool kcluster = false;    // the K slices of a tile run as one cluster and are added up through shared memory
  int smem_bytes;
  int grid;
  size_t ws_bytes;
  GemmParams p;
};

}  // namespace

struct fact_handle_s {
  int device = 0;
  int sm_count = 0;
  int max_smem = 0;
  int cc_major = 0, cc_minor = 0;
  int* d_status = nullptr;
  EncodeTiledFn encode = nullptr;
  long long launches = 0;
  std::map<TuneKey, fact_config_t> table;
  std::bitset<192> configured_mask;  // kernels whose dynamic shared-memory limit was raised
  std::unique_ptr<AttnDeal> attn_deal;         // the host's deal of the last causal attention shape (see fact_attention)
  std::array<long long, 6> attn_deal_key{};
  int kc_clusters[6] = {0, 0, 0, 0, 0, 0};  // clusters of 2 / 4 / 8 CTAs of the K-slice kernel (single CTAs, pairs) the
                                            // device holds at once
  std::string last_error;        // text of the most recent CUDA failure
  int debug_flags = 0;           // FACT_DEBUG_FLAGS: diagnostics (256 cycle counters, 2048 no K serpentine); the
                                 // work-skipping experiment switches only in a -DFACT_EXPERIMENTS build
  int* d_groups = nullptr;       // grouped GEMM: m-tile prefix and row offsets of the call in flight
  // fact_gemm_host: copy-in, compute and copy-out streams and a ring of events, created by its first call
  cudaStream_t host_streams[3] = {nullptr, nullptr, nullptr};
  static constexpr int kHostEvents = 16;
  cudaEvent_t host_events[kHostEvents] = {};
  int host_event_next = 0;
  std::map<const void*, cudaEvent_t> scratch_busy;  // device scratch -> "the call that last used it has copied out"
  // Encoded tensor maps, direct-mapped on a hash of everything an encoding depends on: a caller that repeats a
  // call (same pointers, same shapes) pays for the driver's encoder once.
  struct MapKey {
    const void* base;
    uint64_t d0, d1, d2, s1, s2;
    uint32_t box0, box1, kind;
    bool operator==(const MapKey& o) const {
      return base == o.base && d0 == o.d0 && d1 == o.d1 && d2 == o.d2 && s1 == o.s1 && s2 == o.s2 && box0 == o.box0 &&
             box1 == o.box1 && kind == o.kind;
    }
  };
  struct MapEntry {
    bool used = false;
    MapKey key;
    CUtensorMap map;
  };
  static constexpr int kMapCacheSize = 256;
  std::vector<MapEntry> map_cache = std::vector<MapEntry>(kMapCacheSize);
  int* sk_flags() const { return d_status + kStatusInts; }  // stream-K flags: [SM][epilogue warp], 0 between launches
  size_t status_ints() const { return (size_t)kStatusInts + (size_t)sm_count * kEpiWarps; }
};

namespace {

TuneKey make_key(const Problem& q) {
  return TuneKey((int)q.op, (int)q.epi, (int)q.layout, (int)q.out, q.batch, q.M, q.N_out, q.K);
}

fact_status_t cuda_fail(fact_handle_t h, const char* where, cudaError_t e) {
  h->last_error = std::string(where) + ": " + cudaGetErrorName(e) + " (" + cudaGetErrorString(e) + ")";
  cudaGetLastError();
  return FACT_ERR_CUDA;
}

// Launch with programmatic stream serialization: the kernel may be scheduled while its predecessor in the stream
// is still running (its own griddepcontrol.wait holds it before its first global-memory access), so its set-up --
// barrier initialisation, tensor-memory allocation, descriptor prefetch -- overlaps the predecessor's tail.
// Every kernel launched this way executes griddepcontrol.wait before it touches global memory.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(fact_handle_t h, void (*kern)(KArgs...), unsigned grid, unsigned block, size_t smem,
                       cudaStream_t stream, int cluster, Args&&... args) {
  cudaLaunchConfig_t lc;
  memset(&lc, 0, sizeof lc);
  lc.gridDim = dim3(grid, 1, 1);
  lc.blockDim = dim3(block, 1, 1);
  lc.dynamicSmemBytes = smem;
  lc.stream = stream;
  cudaLaunchAttribute attr[2];
  unsigned n = 0;
  if (cluster > 1) {
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = (unsigned)cluster;
    attr[n].val.clusterDim.y = 1;
    attr[n].val.clusterDim.z = 1;
    ++n;
  }
  if (!(h->debug_flags & 4096)) {
    attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
  }
  lc.attrs = attr;
  lc.numAttrs = n;
  return cudaLaunchKernelEx(&lc, kern, std::forward<Args>(args)...);
}

int round_up(int x, int m) { return (x + m - 1) / m * m; }
uint32_t pow2_at_least(uint32_t x) {
  uint32_t r = 32;
  while (r < x) r <<= 1;
  return r;
}

// Per-CTA bytes of one pipeline stage.
int stage_bytes_for(int tile_n, int cta_group) { return (int)kStageBytesA + (tile_n / cta_group) * kTileK * 2; }

// Staging buffers per epilogue warp: a residual tile that arrives by TMA wants a second buffer to prefetch
// into, but only short main loops (small K) have no slack to hide that load behind.
int epi_bufs_for(const Problem& q) { return (q.epi == FACT_EPI_BIAS_RESIDUAL && q.K <= 2048) ? 2 : 1; }

// (the dynamic scheduler's ring is counted for every configuration: 192 bytes never cost a stage)
int smem_bytes_for(const Problem& q, int tile_n, int cta_group, int stages) {
  return stages * stage_bytes_for(tile_n, cta_group) + (int)epi_smem_bytes(epi_bufs_for(q)) + (int)kCtrlSmemBytes +
         (q.norm == 1 ? (int)kNormCsBytes : (int)kSchedSmemBytes);
}

int max_stages_for(const Problem& q, int tile_n, int cta_group) {
  int s = kMaxStages;
  while (s > 0 && smem_bytes_for(q, tile_n, cta_group, s) > kSmemBudget) --s;
  return s;
}

long long ws_ld_for(const Problem& q) { return round_up((int)q.N_out, 4); }
int ws_planes_for(const Problem& q) { return q.epi == FACT_EPI_SILU_GATE ? 2 : 1; }

// Is (tile_n, cta_group) runnable for this problem's layout / epilogue?
bool tile_ok(const Problem& q, int tile_n, int cg) {
  if (cg != 1 && cg != 2) return false;
  if (tile_n < 32 || tile_n > 256 || tile_n % 32) return false;
  const bool gate = q.epi == FACT_EPI_SILU_GATE;
  const int per_cta = tile_n / cg;
  if (cg == 2 && tile_n % 64) return false;
  if (gate && tile_n % 64) return false;
  if (q.layout == FACT_B_KN) {
    if (per_cta % 64) return false;
    if (gate && (tile_n / 2) % 64) return false;
  }
  return true;
}

// Raster model: which tiles run at the same time decides the DRAM traffic, and on a power-limited part every extra
// gigabyte costs SM clock.  All CTA groups walk K in step, so what one wave of `slots` concurrent tiles fetches is
// the union of its operand slabs: with groups of G tiles of one dimension (the raster walks those fastest) a wave
// covers G slabs of that operand and ceil(slots / G) slabs of the other.  Between waves the G slabs of the grouped
// operand are wanted again and the others are new; what survives in L2 is what the streamed slabs of two waves
// leave of an effective capacity of 55 MB -- the figure that reproduces the measured DRAM reads (8192^3, 256 x 256
// tiles: 1.04 GB with groups of 8 m-tiles, 1.00 GB with 12, 0.96 GB with 16; the Llama down projection: 1.43 GB with
// groups of 4 n-tiles, 1.01 GB with 8; nominal L2 126 MB on two dies).  Returns G > 0 for groups of m-tiles, G < 0
// for groups of n-tiles.
// How many clusters of `slices` CTAs of the K-slice kernel are resident at once (a cluster needs its SMs inside one
// GPC, so this is less than SMs / slices); asked of the runtime once per cluster size.
int kc_max_clusters(fact_handle_t h, int slices, int cg = 1) {
  const int ctas = slices * cg;  // CTAs per cluster: 2, 4 or 8
  const int idx = (ctas == 2 ? 0 : (ctas == 4 ? 1 : 2)) + 3 * (cg - 1);
  if (h->kc_clusters[idx] == 0) {
    int n = 0, dev = -1;
    const bool switched = cudaGetDevice(&dev) == cudaSuccess && dev != h->device && cudaSetDevice(h->device) == cudaSuccess;
    auto kern = cg == 2 ? fact_gemm_kcluster_kernel<kEpiNone, 2> : fact_gemm_kcluster_kernel<kEpiNone, 1>;
    cudaLaunchConfig_t lc;
    memset(&lc, 0, sizeof lc);
    lc.gridDim = dim3((unsigned)(ctas * h->sm_count), 1, 1);
    lc.blockDim = dim3((unsigned)kKcThreads, 1, 1);
    lc.dynamicSmemBytes = (size_t)kSmemBudget;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)ctas;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    lc.attrs = attr;
    lc.numAttrs = 1;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget) != cudaSuccess ||
        cudaOccupancyMaxActiveClusters(&n, kern, &lc) != cudaSuccess || n <= 0) {
      cudaGetLastError();
      n = std::max(1, (h->sm_count / ctas) * 3 / 4);  // (what GPCs of 16 usable SMs out of 18 or 20 would hold)
    }
    if (switched) cudaSetDevice(dev);
    h->kc_clusters[idx] = n;
  }
  return h->kc_clusters[idx];
}

int raster_model(fact_handle_t h, const Problem& q, const fact_config_t& c) {
  const double l2_eff = 55.0 * 1024 * 1024;
  const int out_cols = q.epi == FACT_EPI_SILU_GATE ? c.tile_n / 2 : c.tile_n;
  const long long tiles_m = std::max<long long>(1, (q.M + c.tile_m - 1) / c.tile_m);
  const long long tiles_n = std::max<long long>(1, (q.N_out + out_cols - 1) / out_cols);
  const double esz = q.fp8 ? 1.0 : 2.0;
  const double slab_m = esz * c.tile_m * (double)std::max<long long>(q.K, 1);  // rows of X of one m-tile
  const double slab_n = esz * c.tile_n * (double)std::max<long long>(q.K, 1);  // columns of W of one n-tile
  const double slots = std::max(1, h->sm_count / std::max(1, c.cta_group));
  double best = 1e300;
  int best_g = (int)tiles_m;
  for (int dir = 0; dir < 2; ++dir) {
    const long long n_grouped = dir == 0 ? tiles_m : tiles_n, n_other = dir == 0 ? tiles_n : tiles_m;
    const double slab_g = dir == 0 ? slab_m : slab_n, slab_o = dir == 0 ? slab_n : slab_m;
    // DRAM bytes of the waves that work through one group of `gs` tiles of the grouped dimension
    auto group_bytes = [&](double gs) {
      // (a wave that straddles two groups touches the slabs of both: on average slots / (2 x tiles per group) more;
      // a group smaller than a wave: the wave spans several groups and every slab of the other operand)
      const double straddle = 1.0 + std::min(1.0, slots / (2.0 * gs * (double)n_other));
      const double kept = std::max(gs, slots / (double)n_other) * slab_g * straddle;                     // wanted again
      const double streamed = std::min<double>((double)n_other, std::ceil(slots / gs)) * slab_o;        // new per wave
      const double survive = std::max(0.0, std::min(1.0, (l2_eff - 2.0 * streamed) / kept));
      const double group_waves = gs * (double)n_other / slots;
      // what survives is fetched once per group, the rest once per wave
      return group_waves * (streamed + (1.0 - survive) * kept) + survive * gs * slab_g;
    };
    for (long long g = 1; g <= n_grouped; ++g) {
      const long long full = n_grouped / g, rem = n_grouped % g;
      const double total = (double)full * group_bytes((double)g) + (rem ? group_bytes((double)rem) : 0.0);
      if (total < best * 0.999) {
        best = total;
        best_g = dir == 0 ? (int)g : -(int)g;
      }
    }
  }
  return best_g;
}

// Fill every zero field of `cfg`.  Returns FACT_ERR_UNSUPPORTED for a combination the kernels cannot run.
fact_status_t resolve_config(fact_handle_t h, const Problem& q, const fact_config_t* user, int splits_override,
                             fact_config_t* out, bool* from_table_out = nullptr) {
  fact_config_t c;
  memset(&c, 0, sizeof c);
  bool from_table = false;
  if (user) c = *user;
  else {
    auto it = h->table.find(make_key(q));
    if (it != h->table.end()) {
      c = it->second;
      from_table = true;
    }
  }
  if (splits_override > 0) c.split_k = splits_override;
  if (c.tile_k != 0 && c.tile_k != q.k_elems()) return FACT_ERR_UNSUPPORTED;
  c.tile_k = q.k_elems();
  const long long Nw = q.Nw();
  if (q.epi == FACT_EPI_BIAS_SOFTMAX) {
    // the softmax of a row is taken inside one tile: the tile is as wide as the row, tiles are data-parallel and
    // stored by the direct path
    if (q.N_out > 256) return FACT_ERR_UNSUPPORTED;
    const int want = std::max(32, round_up((int)q.N_out, 32));
    if (c.tile_n != 0 && c.tile_n < want) return FACT_ERR_UNSUPPORTED;
    if (c.tile_n == 0) {  // the narrowest width the layout and the pair size allow
      const int cg_try = c.cta_group ? c.cta_group : ((c.tile_m == 256) ? 2 : 1);
      for (int tn = want; tn <= 256 && c.tile_n == 0; tn += 32)
        if (tile_ok(q, tn, cg_try)) c.tile_n = tn;
      if (c.tile_n == 0) return FACT_ERR_UNSUPPORTED;
      if (c.cta_group == 0) c.cta_group = cg_try;
    }
    if (c.split_k > 1 || c.split_k < 0 || c.store_mode == 2) return FACT_ERR_UNSUPPORTED;
    c.split_k = 1;
    c.store_mode = 1;
  }
  if (c.cta_group == 0 && c.tile_m != 0) c.cta_group = (c.tile_m == 256) ? 2 : 1;
  // The cost model of an untuned problem, in SM cycles: waves over the SMs times the cycles of one tile (k-blocks at
  // the tensor-pipe rate of that width, plus a fixed hand-over cost).  A 2-CTA pair halves each CTA's B traffic and
  // wins ties; narrow tiles only pay when wide ones leave SMs idle.  Where the tiles are few and K is long, K slices
  // that fill the SMs in one wave are weighed against the reduction they need (a barrier, and the partial planes
  // through L2): a 256 x 4096 x 14336 product is 16 wide tiles of 224 k-blocks, or four times as many of 56.
  const int k_blocks_all = std::max(1, (int)((q.K + q.k_elems() - 1) / q.k_elems()));
  const bool gate_epi = q.epi == FACT_EPI_SILU_GATE;
  const bool may_slice = c.split_k == 0 &&
                         (q.op == FACT_OP_GEMM || q.op == FACT_OP_LINEAR || q.op == FACT_OP_GEMM_SPLITK) && q.batch == 1 &&
                         q.groups == 0 && !q.fp8 && !q.stats_out && !q.norm && q.epi != FACT_EPI_BIAS_SOFTMAX;
  auto model = [&](int cg, int tn, int* slices_out, bool calibrated = false) -> double {
    const int out_cols = q.epi == FACT_EPI_SILU_GATE ? tn / 2 : tn;
    // (a grouped problem's m-tiles are counted group by group: every group ends in a ragged tile of its own, and
    // 64 groups of 222-291 rows are 1.5 pair tiles of 256 rows each but 2.5 single tiles of 128)
    long long m_tiles = (q.M + 128 * cg - 1) / (128 * cg);
    if (q.groups > 0 && q.group_rows != nullptr) {
      m_tiles = 0;
      for (int g = 0; g < q.groups; ++g) m_tiles += (q.group_rows[g] + 128 * cg - 1) / (128 * cg);
    }
    const long long tiles = std::max<long long>(1, q.batch) * m_tiles * ((q.N_out + out_cols - 1) / out_cols);
    const long long slots = std::max(1, h->sm_count / cg);
    // (narrower tiles re-read the A operand from shared memory for less work: 0.65 of the full rate at 128 columns,
    // taken as 0.85 at 192, rank the widths against each other; timed on untuned shapes a k-block costs 450 cycles
    // at 128 columns and 420 at 64 -- 0.57 and 0.45 -- which is what the comparison with the cluster schedule uses)
    const double eff = tn >= 256 ? 1.0 : (tn >= 192 ? 0.85 : (!calibrated ? 0.65 : (tn >= 128 ? 0.57 : 0.45)));
    auto per_tile = [&](double kb) {
      return kb * 512.0 * std::max(tn, 96) / 256.0 / eff + 1500.0 + (cg == 1 ? 60.0 * kb : 0.0);
    };
    double best_cost = (double)((tiles + slots - 1) / slots) * per_tile(k_blocks_all);
    int best_s = 1;
    if (may_slice) {
      const double plane_bytes = (double)q.M * (double)round_up((int)q.N_out, 4) * 4.0 * ws_planes_for(q);
      for (int s2 = 2; tiles * s2 <= slots && k_blocks_all / s2 >= 4; ++s2) {
        if (plane_bytes * s2 > 64.0 * 1024 * 1024) break;  // scratch a caller would not expect to be asked for
        const double kb = std::ceil((double)k_blocks_all / s2);
        // measured on the part: the partial stores, the grid barrier and the reduction cost 8-12 us even for a
        // 256 x 256 output (256 x 256 x 32768: 108 us in one slice, 65 / 43 / 31 in 2 / 4 / 8), and the planes
        // travel at about 900 bytes a cycle (two 1536 x 1536 planes: 21k cycles)
        const double cost = per_tile(kb) + 18000.0 + plane_bytes * s2 / 900.0;
        if (cost < best_cost * 0.8) {  // (slices must win clearly: they cost scratch and a second rounding order)
          best_cost = cost;
          best_s = s2;
        }
      }
    }
    if (slices_out) *slices_out = best_s;
    return best_cost;
  };
  int model_slices = 1;
  if (c.cta_group == 0 || c.tile_n == 0) {
    double best = 1e300;
    int best_cg = 0, best_tn = 0;
    for (int cg = 2; cg >= 1; --cg) {
      if (c.cta_group != 0 && c.cta_group != cg) continue;
      for (int tn = 256; tn >= 64; tn -= 64) {
        if (c.tile_n != 0 && c.tile_n != tn) continue;
        if (!tile_ok(q, tn, cg) || max_stages_for(q, tn, cg) < 2) continue;
        int sl = 1;
        const double cost = model(cg, tn, &sl);
        if (cost < best * 0.999) {
          best = cost;
          best_cg = cg;
          best_tn = tn;
          model_slices = sl;
        }
      }
    }
    if (best_cg == 0) {  // nothing in the 64-column grid fits (a user-chosen odd width): keep what was asked
      best_cg = c.cta_group ? c.cta_group : 1;
      best_tn = c.tile_n ? c.tile_n : 64;
      model_slices = 1;
    }
    c.cta_group = best_cg;
    c.tile_n = best_tn;
    // K slices as a cluster (schedule 3: no workspace, no grid barrier): one wave of clusters of at most 8 CTAs, the
    // slices single CTAs on 128-row tiles or pairs on 256-row tiles.  Per k-block 400 / 450 / 1000 cycles at 64 / 128 /
    // 256 columns (pairs: 400 / 400 / 880), never faster than the operands stream from DRAM, plus 10k cycles (13k at
    // 256 columns) for the exchange, the epilogue and a cold start -- fitted to 66 timed (shape, slices, width)
    // combinations of single CTAs, within a few percent where the cluster schedule wins; pairs timed on 19 shapes.
    if (may_slice && c.schedule == 0 && !gate_epi && (user == nullptr || user->tile_n == 0)) {
      const double hbm = ((double)q.M + (double)Nw) * (double)q.K * 2.0 / 3686.0 * 1.15;
      double best_kc = 1e300;
      int kc_s = 0, kc_tn = 0, kc_cg = 0;
      for (int cg = 1; cg <= 2; ++cg) {
        if (user != nullptr && user->cta_group != 0 && user->cta_group != cg) continue;
        if (user != nullptr && user->tile_m != 0 && user->tile_m != 128 * cg) continue;
        for (int sl = 2; sl * cg <= 8; sl *= 2)
          for (int tn = 64; tn <= 256; tn *= 2) {
            if (tn % (32 * sl) || !tile_ok(q, tn, cg) || max_stages_for(q, tn, cg) < 2 || k_blocks_all < 4 * sl) continue;
            const long long tiles = ((q.M + 128 * cg - 1) / (128 * cg)) * ((q.N_out + tn - 1) / tn);
            if (tiles > kc_max_clusters(h, sl, cg)) continue;
            const double per_kb = cg == 1 ? (tn == 64 ? 400.0 : (tn == 128 ? 450.0 : 1000.0)) : (tn == 256 ? 880.0 : 400.0);
            const double cost =
                std::max(std::ceil((double)k_blocks_all / sl) * per_kb, hbm) + (tn == 256 ? 13000.0 : 10000.0);
            if (cost < best_kc * 0.999) {
              best_kc = cost;
              kc_s = sl;
              kc_tn = tn;
              kc_cg = cg;
            }
          }
      }
      int unused = 1;
      const double best_timed = best_cg != 0 ? model(best_cg, best_tn, &unused, true) : best;
      if (kc_s != 0 && best_kc < 0.92 * best_timed) {
        c.cta_group = kc_cg;
        c.tile_n = kc_tn;
        c.split_k = kc_s;
        c.schedule = 3;
      }
    }
  } else if (may_slice && !from_table && tile_ok(q, c.tile_n, c.cta_group)) {
    (void)model(c.cta_group, c.tile_n, &model_slices);
  }
  if (c.tile_m == 0) c.tile_m = 128 * c.cta_group;
  if (c.tile_m != 128 * c.cta_group) return FACT_ERR_UNSUPPORTED;
  (void)Nw;
  if (!tile_ok(q, c.tile_n, c.cta_group)) return FACT_ERR_UNSUPPORTED;
  const int smax = max_stages_for(q, c.tile_n, c.cta_group);
  if (c.stages == 0) c.stages = smax;
  if (from_table && c.stages > smax) c.stages = smax;  // a table written when the other buffers were smaller
  if (c.stages < 2 || c.stages > smax) return FACT_ERR_UNSUPPORTED;
  if (c.raster_group == 0) c.raster_group = raster_model(h, q, c);
  const int k_blocks = (int)((q.K + q.k_elems() - 1) / q.k_elems());
  if (c.split_k == 0) {
    c.split_k = may_slice ? model_slices : 1;
    if (q.op == FACT_OP_GEMM_SPLITK) {
      const int out_cols = q.epi == FACT_EPI_SILU_GATE ? c.tile_n / 2 : c.tile_n;
      const long long tiles = q.batch * ((q.M + c.tile_m - 1) / c.tile_m) * ((q.N_out + out_cols - 1) / out_cols);
      const long long slots = h->sm_count / c.cta_group;
      long long s = tiles > 0 ? slots / tiles : 1;
      s = std::min<long long>(s, k_blocks / 4);  // at least four k-blocks per slice
      c.split_k = (int)std::max<long long>(1, s);
    }
  }
  if (c.split_k < -2) return FACT_ERR_INVALID_ARG;
  if (c.split_k > 0) c.split_k = std::max(1, std::min(c.split_k, std::max(1, k_blocks)));
  if (c.store_mode < 0 || c.store_mode > 3) return FACT_ERR_INVALID_ARG;
  if (c.schedule < 0 || c.schedule > 3) return FACT_ERR_INVALID_ARG;
  if (c.schedule == 0) c.schedule = 1;
  *out = c;
  if (from_table_out) *from_table_out = from_table;
  return FACT_OK;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

fact_status_t validate(const Problem& q) {
  if (q.batch < 0 || q.M < 0 || q.N_out < 0 || q.K < 0) return FACT_ERR_INVALID_ARG;
  if (q.epi < FACT_EPI_NONE || q.epi > FACT_EPI_BIAS_SOFTMAX) return FACT_ERR_INVALID_ARG;
  if (q.layout != FACT_B_KN && q.layout != FACT_B_NK) return FACT_ERR_INVALID_ARG;
  if (q.out != FACT_OUT_BF16 && q.out != FACT_OUT_F32) return FACT_ERR_INVALID_ARG;
  if (q.batch == 0 || q.M == 0 || q.N_out == 0) return FACT_OK;
  if (q.M > 0x7fffffffLL - 512 || q.Nw() > 0x7fffffffLL - 512 || q.K > 0x7fffffffLL - 512 || q.batch > 65535 * 16)
    return FACT_ERR_INVALID_ARG;
  if (!q.C) return FACT_ERR_INVALID_ARG;
  const bool needs_bias = q.epi == FACT_EPI_BIAS || q.epi == FACT_EPI_BIAS_RELU || q.epi == FACT_EPI_BIAS_GELU_TANH;
  if (needs_bias && !q.bias) return FACT_ERR_INVALID_ARG;
  if ((q.epi == FACT_EPI_NONE || q.epi == FACT_EPI_SILU_GATE) && q.bias) return FACT_ERR_INVALID_ARG;
  if (q.epi == FACT_EPI_BIAS_RESIDUAL) {
    if (!q.R || q.ldr < q.N_out) return FACT_ERR_INVALID_ARG;
    if (q.R == q.C && q.ldr != q.ldc) return FACT_ERR_INVALID_ARG;
    if (q.R == q.C && q.out != FACT_OUT_BF16) return FACT_ERR_INVALID_ARG;
  } else if (q.R) {
    return FACT_ERR_INVALID_ARG;
  }
  if (q.ldc < q.N_out) return FACT_ERR_INVALID_ARG;
  if (q.stats_out || q.norm) {
    if (q.norm < 0 || q.norm > 2) return FACT_ERR_INVALID_ARG;
    if (q.op != FACT_OP_LINEAR || q.batch != 1 || q.groups > 0 || q.fp8 || q.epi == FACT_EPI_BIAS_SOFTMAX || q.K == 0)
      return FACT_ERR_UNSUPPORTED;
    if (q.stats_out && q.out != FACT_OUT_BF16) return FACT_ERR_UNSUPPORTED;  // the sums are over stored BF16 values
    if (q.norm) {
      if (!q.stats_in || !(q.norm_eps >= 0.f)) return FACT_ERR_INVALID_ARG;
      if (q.norm == 1) {
        if (!q.colsum) return FACT_ERR_INVALID_ARG;
        if (q.epi == FACT_EPI_SILU_GATE || q.N_out % 64) return FACT_ERR_UNSUPPORTED;
        if (!aligned16(q.colsum)) return FACT_ERR_BAD_ALIGNMENT;
      }
    }
  }
  if (q.K > 0) {
    if (!q.A || !q.B) return FACT_ERR_INVALID_ARG;
    if (q.lda < q.K) return FACT_ERR_INVALID_ARG;
    if (q.ldb < (q.layout == FACT_B_KN ? q.Nw() : q.K)) return FACT_ERR_INVALID_ARG;
    if (!aligned16(q.A) || !aligned16(q.B)) return FACT_ERR_BAD_ALIGNMENT;
    if (q.lda % q.op_align() || q.ldb % q.op_align()) return FACT_ERR_BAD_ALIGNMENT;
    if (q.fp8 && q.layout != FACT_B_NK) return FACT_ERR_UNSUPPORTED;  // 8-bit operands are read K-major only
    if (q.batch > 1) {
      if (q.strideA % q.op_align() || q.strideB % q.op_align()) return FACT_ERR_BAD_ALIGNMENT;
      if (q.strideA < 0 || q.strideB < 0 || q.strideC < 0) return FACT_ERR_INVALID_ARG;
    }
  }
  return FACT_OK;
}

// Stream-K (split_k < 0): how many tiles at the end of the tile list are cut along K and shared out evenly over all
// CTA groups.  -1: the tiles of the last, partial wave; -2: those plus one full wave (shorter runs of partial
// pieces per tile when the partial wave is small).  0 when there is nothing to share (the tiles fill whole waves,
// K is empty, or the run of a group would be shorter than one k-block): the call is then data-parallel.
int sk_tiles_for(fact_handle_t h, const Problem& q, const fact_config_t& c) {
  if (c.split_k >= 0 || q.K <= 0) return 0;
  const int out_cols = q.epi == FACT_EPI_SILU_GATE ? c.tile_n / 2 : c.tile_n;
  // the pieces are parked and finished by the staged epilogue, which stores whole 128-byte chunks per tile
  const bool f32 = q.out == FACT_OUT_F32;
  if (out_cols % (f32 ? 32 : 64) != 0 || (f32 && q.epi == FACT_EPI_BIAS_RESIDUAL) || c.store_mode == 1 || c.store_mode == 3) return 0;
  const long long tiles = q.batch * ((q.M + c.tile_m - 1) / c.tile_m) * ((q.N_out + out_cols - 1) / out_cols);
  const long long groups = std::max(1, h->sm_count / c.cta_group);
  const long long k_blocks = (q.K + q.k_elems() - 1) / q.k_elems();
  long long sk = tiles % groups;
  if (sk == 0) return 0;
  if (c.split_k == -2 && tiles >= sk + groups) sk += groups;
  if (sk * k_blocks < groups || sk * k_blocks > 0x3fffffffLL) return 0;
  return (int)sk;
}

size_t workspace_for(fact_handle_t h, const Problem& q, const fact_config_t& c) {
  if (c.schedule == 3) return 0;  // K slices as a cluster: the partial sums never leave the SMs
  if (c.split_k < 0) {  // stream-K: one FP32 accumulator tile per CTA
    if (sk_tiles_for(h, q, c) == 0) return 0;
    const size_t ctas = (size_t)std::max(1, h->sm_count / c.cta_group) * (size_t)c.cta_group;
    return ctas * (size_t)kTileM * (size_t)c.tile_n * sizeof(float);
  }
  if (c.split_k <= 1) return 0;
  return (size_t)c.split_k * (size_t)q.batch * (size_t)ws_planes_for(q) * (size_t)q.M * (size_t)ws_ld_for(q) *
         sizeof(float);
}

uint64_t smem_desc_template(uint32_t lbo_bytes, uint32_t sbo_bytes) {
  // 64-bit shared-memory matrix descriptor without the start address:
  // [16,30) leading byte offset >> 4, [32,46) stride byte offset >> 4, [46,48) version 1 (sm_100),
  // [61,64) layout type 2 = 128-byte swizzle
  return ((uint64_t)((lbo_bytes >> 4) & 0x3fffu) << 16) | ((uint64_t)((sbo_bytes >> 4) & 0x3fffu) << 32) |
         (1ull << 46) | (2ull << 61);
}

fact_status_t make_plan(fact_handle_t h, const Problem& q, const fact_config_t* user, int splits_override,
                        Plan* plan) {
  fact_status_t st = resolve_config(h, q, user, splits_override, &plan->cfg, &plan->from_table);
  if (st != FACT_OK) return st;
  const fact_config_t& c = plan->cfg;
  GemmParams& p = plan->p;
  memset(&p, 0, sizeof p);
  const int cg = c.cta_group;
  const bool gate = q.epi == FACT_EPI_SILU_GATE;
  p.M = (int)q.M;
  p.N_out = (int)q.N_out;
  p.Nw = (int)q.Nw();
  p.K = (int)q.K;
  p.batch = (int)q.batch;
  p.tile_n = c.tile_n;
  p.out_cols = gate ? c.tile_n / 2 : c.tile_n;
  p.tiles_m = (int)((q.M + c.tile_m - 1) / c.tile_m);
  p.tiles_n = (int)((q.N_out + p.out_cols - 1) / p.out_cols);
  p.k_blocks = (int)((q.K + q.k_elems() - 1) / q.k_elems());
  const int slices = std::max(1, c.split_k);  // (stream-K, split_k < 0, cuts no tile into equal slices)
  p.split_k = slices;
  p.k_serpentine = (h->debug_flags & 2048) ? 0 : 1;
  // L2 eviction priority of the operand loads: last where tiles share operand slabs (whole tiles, K slices as a
  // cluster), first where K slices through the workspace stream every operand byte past once or twice and what must
  // stay in L2 are the partial planes the tail of the launch reads back
  p.l2_keep_operands = (h->debug_flags & 8192) ? 0 : (slices > 1 && c.schedule != 3 ? 1 : 2);
  p.k_base = p.k_blocks / slices;
  p.k_rem = p.k_blocks % slices;
  p.raster_along_n = c.raster_group < 0;
  p.raster_group = p.raster_along_n ? std::min(-c.raster_group, std::max(1, p.tiles_n))
                                    : std::min(c.raster_group, std::max(1, p.tiles_m));
  p.stages = c.stages;
  const long long units = (long long)p.batch * p.tiles_m * p.tiles_n * p.split_k;
  if (units > 0x7fffffffLL) return FACT_ERR_UNSUPPORTED;
  p.total_units = (int)units;
  const int per_cta = c.tile_n / cg;
  p.b_kn = q.layout == FACT_B_KN;
  p.gate = gate;
  if (p.b_kn) {
    p.b_box_n = 64;
    p.b_loads = per_cta / 64;
  } else if (gate && cg == 1) {
    p.b_box_n = c.tile_n / 2;
    p.b_loads = 2;
  } else {
    p.b_box_n = per_cta;
    p.b_loads = 1;
  }
  p.b_box_bytes = (uint32_t)p.b_box_n * kTileK * 2;
  p.stage_bytes = (uint32_t)stage_bytes_for(c.tile_n, cg);
  p.tx_bytes = p.stage_bytes * (uint32_t)cg;
  // A and W[N x K]: K-major, rows of 128 bytes, 8-row swizzle atoms 1024 bytes apart; 16 K-elements = 32 bytes.
  p.a_desc = smem_desc_template(16, 1024);
  p.a_k_step = 32 >> 4;
  if (p.b_kn) {
    // B[K x N]: N-major.  One TMA box = 64 k-rows of 64 n (128 bytes): 8-k groups are 1024 bytes apart
    // (stride offset), successive 64-n chunks one box (8192 bytes) apart (leading offset); 16 k = 2048 bytes.
    p.b_desc = smem_desc_template(kTileK * 128, 1024);
    p.b_k_step = (kUmmaK * 128) >> 4;
  } else {
    p.b_desc = p.a_desc;
    p.b_k_step = p.a_k_step;
  }
  // instruction descriptor: D = F32 (1 @ bit 4), A = B = BF16 (1 @ bits 7, 10), A K-major, B major-ness @ bit 16,
  // N >> 3 @ bit 17, M >> 4 @ bit 24
  p.idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)p.b_kn << 16) | ((uint32_t)(c.tile_n >> 3) << 17) |
            ((uint32_t)((kTileM * cg) >> 4) << 24);
  // kind::f8f6f4: format 0 = E4M3 for A and B (bits 7 and 10 clear), K-major both, one instruction per 32 bytes of K
  if (q.fp8) p.idesc &= ~((1u << 7) | (1u << 10));
  p.k_elems = q.k_elems();
  p.fp8 = q.fp8 ? 1 : 0;
  p.use_alpha = (q.fp8 && q.alpha != 1.f) ? 1 : 0;
  p.alpha = q.alpha;
  p.tmem_cols = pow2_at_least((uint32_t)(2 * c.tile_n));
  p.C = q.C;
  p.ldc = q.ldc;
  p.strideC = q.strideC;
  p.out_f32 = q.out == FACT_OUT_F32;
  const int c_elems16 = p.out_f32 ? 4 : 8;
  p.c_vec = aligned16(q.C) && (q.ldc % c_elems16 == 0) && (q.batch <= 1 || q.strideC % c_elems16 == 0);
  p.bias = reinterpret_cast<const __nv_bfloat16*>(q.bias);
  p.bias_vec = q.bias && aligned16(q.bias);
  p.R = reinterpret_cast<const __nv_bfloat16*>(q.R);
  p.ldr = q.ldr;
  p.strideR = q.strideR;
  p.r_vec = q.R && aligned16(q.R) && (q.ldr % 8 == 0) && (q.batch <= 1 || q.strideR % 8 == 0);
  p.ws_ld = ws_ld_for(q);
  p.ws_planes = ws_planes_for(q);
  // Staged TMA stores need a 16-byte aligned output whose rows are 16-byte multiples, whole 128-byte chunks per
  // tile, and (for a residual) a BF16 output; anything else is stored directly from registers.
  const int chunk_cols = p.out_f32 ? 32 : 64;
  const bool can_stage = p.c_vec && (p.out_cols % chunk_cols == 0) &&
                         !(p.out_f32 && q.epi == FACT_EPI_BIAS_RESIDUAL);
  // The table is keyed on the shape alone, so what it says about the store path is a hint: this call's output may
  // be less aligned than the one the entry was tuned on.  Only a caller's own configuration is refused.
  const long long esz_c = p.out_f32 ? 4 : 2;
  const bool rows32 = (reinterpret_cast<uintptr_t>(q.C) & 31u) == 0 && (q.ldc * esz_c) % 32 == 0 &&
                      (q.N_out * esz_c) % 32 == 0 && (q.batch <= 1 || (q.strideC * esz_c) % 32 == 0);
  const bool can_rows32 = can_stage && rows32 && c.split_k == 1 && q.groups == 0 && !q.stats_out && !q.norm &&
                          q.epi != FACT_EPI_BIAS_SOFTMAX;
  if (plan->from_table && ((c.store_mode == 2 && !can_stage) || (c.store_mode == 3 && !can_rows32)))
    plan->cfg.store_mode = 0;
  if (c.store_mode == 2 && !can_stage) return FACT_ERR_UNSUPPORTED;
  const int asked_store = c.store_mode;  // (c aliases plan->cfg, which is rewritten below)
  p.store_tma = (c.store_mode == 1) ? 0 : (can_stage ? 1 : 0);
  p.r_tma = p.store_tma && q.epi == FACT_EPI_BIAS_RESIDUAL && p.r_vec;
  plan->cfg.store_mode = p.store_tma ? 2 : 1;
  if (asked_store == 3) {
    // the staged epilogue's arithmetic with each row stored from registers in 32-byte pieces: whole, unsliced,
    // ungrouped tiles whose output rows are 32-byte aligned multiples of 32 bytes
    if (!can_rows32) return FACT_ERR_UNSUPPORTED;
    p.row_stores = 1;
    plan->cfg.store_mode = 3;
  }
  // row sums out and the folded normalisation live in the staged epilogue of an unsliced product
  if ((q.stats_out || q.norm) && (!p.store_tma || c.split_k > 1)) return FACT_ERR_UNSUPPORTED;
  p.stats_out = reinterpret_cast<float2*>(q.stats_out);
  p.stats_in = reinterpret_cast<const float2*>(q.stats_in);
  p.colsum = q.colsum;
  p.norm_mode = q.norm;
  p.norm_eps = q.norm_eps;
  p.status = h->d_status;
  p.debug = h->debug_flags;
  plan->ws_bytes = workspace_for(h, q, c);
  p.epi_bufs = epi_bufs_for(q);
  plan->smem_bytes = std::max(smem_bytes_for(q, c.tile_n, cg, c.stages), kMinSmemRequest);
  if (plan->smem_bytes > kSmemBudget || kSmemBudget > h->max_smem) return FACT_ERR_UNSUPPORTED;
  const int slots = std::max(1, h->sm_count / cg);
  plan->grid = (int)std::min<long long>(slots, units) * cg;
  plan->dynamic = false;
  if (c.schedule == 2) {
    // whole data-parallel tiles through the ordinary epilogues only; a table entry tuned on another call's
    // circumstances falls back to the static schedule, a caller's own request is refused
    const bool can = c.split_k == 1 && !p.row_stores && !q.stats_out && !q.norm && q.epi != FACT_EPI_BIAS_SOFTMAX &&
                     units * cg <= 0x7fffffffLL;
    if (!can && !plan->from_table) return FACT_ERR_UNSUPPORTED;
    if (can && units > slots) {  // (one wave or less: every cluster has an SM at once, nothing to hand out)
      plan->dynamic = true;
      plan->grid = (int)(units * cg);
    } else if (!can) {
      plan->cfg.schedule = 1;
    }
  }
  if (c.schedule == 3) {
    // K slices as a cluster: 2 / 4 / 8 slices of single CTAs (128-row tiles) or 2 / 4 of pairs (256-row tiles), at
    // most 8 CTAs; every CTA finishes tile_n / slices columns (whole 32-column pieces); column-wise epilogues on
    // BF16 operands; every slice has at least one k-block
    const bool can = (c.split_k == 2 || c.split_k == 4 || c.split_k == 8) && c.split_k * cg <= 8 &&
                     c.tile_n % (32 * c.split_k) == 0 &&
                     !gate && q.epi != FACT_EPI_BIAS_SOFTMAX && !q.fp8 && q.groups == 0 && !q.stats_out && !q.norm &&
                     p.k_blocks >= c.split_k && units <= 0x7fffffffLL;
    if (!can) return FACT_ERR_UNSUPPORTED;
    plan->kcluster = true;
    plan->ws_bytes = 0;
    plan->smem_bytes = std::max((int)kc_smem_bytes(c.tile_n, c.split_k, c.stages, p.stage_bytes), kMinSmemRequest);
    if (plan->smem_bytes > kSmemBudget) return FACT_ERR_UNSUPPORTED;
    const long long tiles = units / c.split_k;
    plan->grid = (int)std::min<long long>(tiles, kc_max_clusters(h, c.split_k, cg)) * c.split_k * cg;
  }
  if (c.split_k < 0) {
    // Stream-K: the staged epilogue parks and finishes the pieces, so an output it cannot store is data-parallel.
    const int sk = p.store_tma ? sk_tiles_for(h, q, c) : 0;
    if (sk == 0) {
      plan->cfg.split_k = 1;
      plan->ws_bytes = 0;
    } else {
      const long long iters = (long long)sk * p.k_blocks;
      p.sk_tiles = sk;
      p.sk_first = p.total_units - sk;
      p.total_units = p.sk_first;  // what is left for the data-parallel walk
      p.sk_len = (int)(iters / slots);
      p.sk_rem = (int)(iters % slots);
      plan->grid = slots * cg;     // every group takes a run, whatever the number of tiles
    }
  }
  return FACT_OK;
}

// A rank-3 tensor map (inner, rows, batch) with a (box0 x box1 x 1) box and 128-byte swizzle.
fact_status_t encode_map(fact_handle_t h, CUtensorMap* map, const void* base, uint64_t d0, uint64_t d1, uint64_t d2,
                         uint64_t stride1_elems, uint64_t stride2_elems, uint32_t box0, uint32_t box1,
                         bool f32 = false, bool u8 = false) {
  const uint64_t esz = f32 ? 4 : (u8 ? 1 : 2);
  fact_handle_s::MapKey key = {base, d0, d1, d2, stride1_elems, stride2_elems, box0, box1, (uint32_t)(f32 ? 1 : (u8 ? 2 : 0))};
  uint64_t hsh = reinterpret_cast<uintptr_t>(base) * 0x9E3779B97F4A7C15ull;
  for (uint64_t v : {d0, d1, d2, stride1_elems, stride2_elems, (uint64_t)box0 << 32 | box1, (uint64_t)key.kind})
    hsh = (hsh ^ v) * 0x9E3779B97F4A7C15ull;
  fact_handle_s::MapEntry& slot = h->map_cache[(size_t)(hsh >> 40) % fact_handle_s::kMapCacheSize];
  if (slot.used && slot.key == key) {
    *map = slot.map;
    return FACT_OK;
  }
  cuuint64_t dims[3] = {d0, d1, d2};
  cuuint64_t strides[2] = {stride1_elems * esz, stride2_elems * esz};
  cuuint32_t box[3] = {box0, box1, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = h->encode(map, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : (u8 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16), 3,
                         const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                         CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r == CUDA_SUCCESS) {
    slot.used = true;
    slot.key = key;
    slot.map = *map;
  }
  if (r != CUDA_SUCCESS) {
    h->last_error = "cuTensorMapEncodeTiled failed with CUresult " + std::to_string((int)r);
    return FACT_ERR_CUDA;
  }
  return FACT_OK;
}

template <int CG, int EPI, bool SK = false, bool GROUPED = false, int EXT = 0, bool DYN = false>
fact_status_t launch_instance(fact_handle_t h, int slot, const Plan& plan, const CUtensorMap* tm,
                              cudaStream_t stream) {
  auto kern = fact_gemm_kernel<CG, EPI, SK, GROUPED, EXT, DYN>;
  if (slot < 0) {  // (no bit left in the handle's mask for these instantiations: set the attribute on every launch)
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget);
    if (e != cudaSuccess) return cuda_fail(h, "cudaFuncSetAttribute(MaxDynamicSharedMemorySize)", e);
  } else if (!h->configured_mask.test((size_t)slot)) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget);
    if (e != cudaSuccess) return cuda_fail(h, "cudaFuncSetAttribute(MaxDynamicSharedMemorySize)", e);
    h->configured_mask.set((size_t)slot);
  }
  cudaError_t e = launch_pdl(h, kern, (unsigned)plan.grid, (unsigned)(kThreads + (DYN ? 32 : 0)),
                             (size_t)plan.smem_bytes, stream, CG, tm[0], tm[1], tm[2], tm[3], plan.p);
  if (e != cudaSuccess) return cuda_fail(h, "cudaLaunchKernelEx", e);
  h->launches++;
  return FACT_OK;
}

template <int EPI, int CG>
fact_status_t launch_kcluster_instance(fact_handle_t h, int slot, const Plan& plan, const CUtensorMap* tm,
                                       cudaStream_t stream) {
  auto kern = fact_gemm_kcluster_kernel<EPI, CG>;
  if (!h->configured_mask.test((size_t)slot)) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget);
    if (e != cudaSuccess) return cuda_fail(h, "cudaFuncSetAttribute(MaxDynamicSharedMemorySize)", e);
    h->configured_mask.set((size_t)slot);
  }
  cudaError_t e = launch_pdl(h, kern, (unsigned)plan.grid, (unsigned)kKcThreads, (size_t)plan.smem_bytes, stream,
                             plan.cfg.split_k * CG, tm[0], tm[1], plan.p);
  if (e != cudaSuccess) return cuda_fail(h, "cudaLaunchKernelEx (K slices as a cluster)", e);
  h->launches++;
  return FACT_OK;
}

fact_status_t launch_kcluster(fact_handle_t h, int epi, const Plan& plan, const CUtensorMap* tm, cudaStream_t stream) {
  if (plan.cfg.cta_group == 2) {
    switch (epi) {
      case kEpiNone: return launch_kcluster_instance<kEpiNone, 2>(h, 160, plan, tm, stream);
      case kEpiBias: return launch_kcluster_instance<kEpiBias, 2>(h, 161, plan, tm, stream);
      case kEpiBiasRelu: return launch_kcluster_instance<kEpiBiasRelu, 2>(h, 162, plan, tm, stream);
      case kEpiBiasGeluTanh: return launch_kcluster_instance<kEpiBiasGeluTanh, 2>(h, 163, plan, tm, stream);
      case kEpiBiasResidual: return launch_kcluster_instance<kEpiBiasResidual, 2>(h, 164, plan, tm, stream);
      default: return FACT_ERR_UNSUPPORTED;
    }
  }
  switch (epi) {
    case kEpiNone: return launch_kcluster_instance<kEpiNone, 1>(h, 150, plan, tm, stream);
    case kEpiBias: return launch_kcluster_instance<kEpiBias, 1>(h, 151, plan, tm, stream);
    case kEpiBiasRelu: return launch_kcluster_instance<kEpiBiasRelu, 1>(h, 152, plan, tm, stream);
    case kEpiBiasGeluTanh: return launch_kcluster_instance<kEpiBiasGeluTanh, 1>(h, 153, plan, tm, stream);
    case kEpiBiasResidual: return launch_kcluster_instance<kEpiBiasResidual, 1>(h, 154, plan, tm, stream);
    default: return FACT_ERR_UNSUPPORTED;
  }
}

template <int CG>
fact_status_t launch_epi(fact_handle_t h, int epi, const Plan& plan, const CUtensorMap* tm, cudaStream_t stream) {
  const int base = (CG - 1) * 8;
  switch (epi) {
    case kEpiNone: return launch_instance<CG, kEpiNone>(h, base + 0, plan, tm, stream);
    case kEpiBias: return launch_instance<CG, kEpiBias>(h, base + 1, plan, tm, stream);
    case kEpiBiasRelu: return launch_instance<CG, kEpiBiasRelu>(h, base + 2, plan, tm, stream);
    case kEpiBiasGeluTanh: return launch_instance<CG, kEpiBiasGeluTanh>(h, base + 3, plan, tm, stream);
    case kEpiSiluGate: return launch_instance<CG, kEpiSiluGate>(h, base + 4, plan, tm, stream);
    case kEpiBiasResidual: return launch_instance<CG, kEpiBiasResidual>(h, base + 5, plan, tm, stream);
    case kEpiPartial: return launch_instance<CG, kEpiPartial>(h, base + 6, plan, tm, stream);
    case kEpiBiasSoftmax: return launch_instance<CG, kEpiBiasSoftmax>(h, base + 7, plan, tm, stream);
    default: return FACT_ERR_INVALID_ARG;
  }
}

// The instantiations with row sums out (EXT 1), a folded row normalisation in, with or without row sums out
// (EXT 2), or rows stored from registers in 32-byte pieces (EXT 3): staged epilogue, data-parallel tiles.  Two sets, because the consumer's code slows the producer's
// epilogue down even when it does not run.
template <int CG, int EXT>
fact_status_t launch_epi_ext(fact_handle_t h, int epi, const Plan& plan, const CUtensorMap* tm, cudaStream_t stream) {
  const int base = 32 + (EXT - 1) * 16 + (CG - 1) * 8;
  switch (epi) {
    case kEpiNone: return launch_instance<CG, kEpiNone, false, false, EXT>(h, base + 0, plan, tm, stream);
    case kEpiBias: return launch_instance<CG, kEpiBias, false, false, EXT>(h, base + 1, plan, tm, stream);
    case kEpiBiasRelu: return launch_instance<CG, kEpiBiasRelu, false, false, EXT>(h, base + 2, plan, tm, stream);
    case kEpiBiasGeluTanh: return launch_instance<CG, kEpiBiasGeluTanh, false, false, EXT>(h, base + 3, plan, tm, stream);
    case kEpiSiluGate: return launch_instance<CG, kEpiSiluGate, false, false, EXT>(h, base + 4, plan, tm, stream);
    case kEpiBiasResidual: return launch_instance<CG, kEpiBiasResidual, false, false, EXT>(h, base + 5, plan, tm, stream);
    default: return FACT_ERR_UNSUPPORTED;
  }
}

// The stream-K instantiations (every epilogue but the split-K partial store).
template <int CG>
fact_status_t launch_epi_sk(fact_handle_t h, int epi, const Plan& plan, const CUtensorMap* tm, cudaStream_t stream) {
  const int base = 16 + (CG - 1) * 8;
  switch (epi) {
    case kEpiNone: return launch_instance<CG, kEpiNone, true>(h, base + 0, plan, tm, stream);
    case kEpiBias: return launch_instance<CG, kEpiBias, true>(h, base + 1, plan, tm, stream);
    case kEpiBiasRelu: return launch_instance<CG, kEpiBiasRelu, true>(h, base + 2, plan, tm, stream);
    case kEpiBiasGeluTanh: return launch_instance<CG, kEpiBiasGeluTanh, true>(h, base + 3, plan, tm, stream);
    case kEpiSiluGate: return launch_instance<CG, kEpiSiluGate, true>(h, base + 4, plan, tm, stream);
    case kEpiBiasResidual: return launch_instance<CG, kEpiBiasResidual, true>(h, base + 5, plan, tm, stream);
    default: return FACT_ERR_INVALID_ARG;
  }
}

// The grouped instantiations (data-parallel tiles), and the dynamically scheduled ones, grouped or not.
template <int CG, bool GROUPED, bool DYN>
fact_status_t launch_epi_dp(fact_handle_t h, int epi, const Plan& plan, const CUtensorMap* tm, cudaStream_t stream) {
  const int base = 80 + (GROUPED ? 32 : 0) + (DYN ? 16 : 0) + (CG - 1) * 8;
  switch (epi) {
    case kEpiNone: return launch_instance<CG, kEpiNone, false, GROUPED, 0, DYN>(h, base + 0, plan, tm, stream);
    case kEpiBias: return launch_instance<CG, kEpiBias, false, GROUPED, 0, DYN>(h, base + 1, plan, tm, stream);
    case kEpiBiasRelu: return launch_instance<CG, kEpiBiasRelu, false, GROUPED, 0, DYN>(h, base + 2, plan, tm, stream);
    case kEpiBiasGeluTanh: return launch_instance<CG, kEpiBiasGeluTanh, false, GROUPED, 0, DYN>(h, base + 3, plan, tm, stream);
    case kEpiSiluGate: return launch_instance<CG, kEpiSiluGate, false, GROUPED, 0, DYN>(h, base + 4, plan, tm, stream);
    case kEpiBiasResidual: return launch_instance<CG, kEpiBiasResidual, false, GROUPED, 0, DYN>(h, base + 5, plan, tm, stream);
    default: return FACT_ERR_INVALID_ARG;
  }
}

fact_status_t launch_reduce(fact_handle_t h, const Problem& q, const Plan& plan, int splits, const float* ws,
                            cudaStream_t stream) {
  ReduceParams r;
  memset(&r, 0, sizeof r);
  r.ws = ws;
  r.ws_ld = plan.p.ws_ld;
  r.planes = plan.p.ws_planes;
  r.splits = splits;
  r.M = plan.p.M;
  r.N_out = plan.p.N_out;
  r.batch = plan.p.batch;
  r.epi = (int)q.epi;
  r.C = q.C;
  r.ldc = q.ldc;
  r.strideC = q.strideC;
  r.out_f32 = q.out == FACT_OUT_F32;
  r.bias = reinterpret_cast<const __nv_bfloat16*>(q.bias);
  r.R = reinterpret_cast<const __nv_bfloat16*>(q.R);
  r.ldr = q.ldr;
  r.strideR = q.strideR;
  r.alpha = q.fp8 ? q.alpha : 1.f;
  const long long total = 4LL * r.batch * r.M * ((r.N_out + 3) / 4);  // four threads per group of 4 columns
  const int blocks = (int)std::min<long long>((total + 127) / 128, (long long)h->sm_count * 16);
  cudaError_t e = launch_pdl(h, fact_splitk_reduce_kernel, (unsigned)std::max(1, blocks), 128u, 0, stream, 1, r);
  if (e != cudaSuccess) return cuda_fail(h, "split-K reduce launch", e);
  h->launches++;
  return FACT_OK;
}

fact_status_t run(fact_handle_t h, const Problem& q, const fact_config_t* user, int splits_override, void* ws,
                  size_t ws_bytes, void* stream_v) {
  if (!h) return FACT_ERR_INVALID_ARG;
  fact_status_t st = validate(q);
  if (st != FACT_OK) return st;
  if (q.batch == 0 || q.M == 0 || q.N_out == 0) return FACT_OK;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_v);
  Plan plan;
  st = make_plan(h, q, user, splits_override, &plan);
  if (st == FACT_ERR_UNSUPPORTED && plan.from_table && plan.cfg.schedule == 3) {
    // a table entry with K slices as a cluster, tuned on a plain call of this shape: this call (row sums, a folded
    // normalisation) takes the library's own choice instead
    fact_config_t none;
    memset(&none, 0, sizeof none);
    none.split_k = 1;
    st = make_plan(h, q, &none, 0, &plan);
  }
  if (st != FACT_OK) return st;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return FACT_ERR_CUDA;
  if (dev != h->device && cudaSetDevice(h->device) != cudaSuccess) return FACT_ERR_CUDA;

  std::vector<int> group_table;
  if (q.groups > 0) {
    // Grouped: tiles never cross a group boundary (a group's last m-tile is ragged), every tile is data-parallel and
    // stored by the row-predicated direct path.  The table -- m-tiles before each group, first row of each group --
    // goes to the handle's device buffer in stream order.
    fact_config_t gc = plan.cfg;
    gc.split_k = 1;
    // staged through shared memory (then the warp's own row-predicated 16-byte stores) when the output's rows are
    // whole 16-byte pieces; otherwise straight from registers
    const bool whole16 = q.N_out % (q.out == FACT_OUT_F32 ? 4 : 8) == 0;
    if (!whole16 || !plan.p.store_tma) {
      if (user && user->store_mode == 2) return FACT_ERR_UNSUPPORTED;
      gc.store_mode = 1;
    }
    st = make_plan(h, q, &gc, 0, &plan);
    if (st != FACT_OK) return st;
    const int G = q.groups;
    group_table.resize(2 * (size_t)(G + 1));
    long long tiles = 0, rows = 0;
    for (int g = 0; g < G; ++g) {
      group_table[g] = (int)tiles;
      group_table[G + 1 + g] = (int)rows;
      tiles += (q.group_rows[g] + plan.cfg.tile_m - 1) / plan.cfg.tile_m;
      rows += q.group_rows[g];
    }
    group_table[G] = (int)tiles;
    group_table[2 * G + 1] = (int)rows;
    const long long units = tiles * plan.p.tiles_n;
    if (units > 0x7fffffffLL) return FACT_ERR_UNSUPPORTED;
    // slabs of m-tiles whose rows of A fit a 32 MB share of L2
    plan.p.raster_group = (int)std::max<long long>(
        1, (32LL << 20) / ((long long)plan.cfg.tile_m * std::max<long long>(q.K, 1) * (q.fp8 ? 1 : 2)));
    plan.p.groups = G;
    plan.p.grp_tiles = h->d_groups;
    plan.p.grp_rows = h->d_groups + (G + 1);
    plan.p.total_units = (int)units;
    plan.p.strideC = 0;
    plan.p.strideR = 0;
    const long long g_slots = std::max(1, h->sm_count / plan.cfg.cta_group);
    plan.grid = (int)std::min<long long>(g_slots, std::max<long long>(units, 1)) * plan.cfg.cta_group;
    plan.dynamic = plan.cfg.schedule == 2 && units > g_slots && units * plan.cfg.cta_group <= 0x7fffffffLL;
    if (plan.dynamic) plan.grid = (int)(units * plan.cfg.cta_group);
  }
  if (plan.cfg.split_k < 0 && (q.stats_out || q.norm)) {
    // the extras live in the data-parallel instantiations: a stream-K choice (the caller's or the table's) is dropped
    fact_config_t dp = plan.cfg;
    dp.split_k = 1;
    st = make_plan(h, q, &dp, 0, &plan);
    if (st != FACT_OK) return st;
  }
  if (plan.cfg.split_k < 0 && (!ws || ws_bytes < plan.ws_bytes) && !user) {
    // a tuned stream-K entry, but this caller brought no scratch: run the tiles data-parallel
    fact_config_t dp = plan.cfg;
    dp.split_k = 1;
    st = make_plan(h, q, &dp, 0, &plan);
    if (st != FACT_OK) return st;
  }
  if (plan.cfg.split_k > 1 && !plan.kcluster && (plan.from_table || !user || user->split_k == 0) && splits_override == 0 &&
      q.op != FACT_OP_GEMM_SPLITK && (!ws || ws_bytes < plan.ws_bytes || !aligned16(ws))) {
    // K slices from the tuner's table or the library's own model, but this caller brought no (or too little)
    // scratch: one slice
    fact_config_t dp = plan.cfg;
    if (!plan.from_table) {  // the model's choice: choose the tiles again, for one slice
      memset(&dp, 0, sizeof dp);
      if (user) dp = *user;
    }
    dp.split_k = 1;
    dp.store_mode = plan.from_table ? 0 : dp.store_mode;
    st = make_plan(h, q, &dp, 0, &plan);
    if (st != FACT_OK) return st;
  }
  if (q.K == 0 && q.epi == FACT_EPI_BIAS_SOFTMAX) return FACT_ERR_UNSUPPORTED;  // (the stand-alone epilogue has no softmax)
  if (q.K == 0) {  // empty sum: the epilogue of a zero accumulator
    st = launch_reduce(h, q, plan, 0, reinterpret_cast<const float*>(q.C), stream);
  } else {
    const bool split = plan.cfg.split_k > 1 && !plan.kcluster;
    const bool stream_k = plan.cfg.split_k < 0;
    if (stream_k) {
      if (!ws || ws_bytes < plan.ws_bytes) return FACT_ERR_WORKSPACE_TOO_SMALL;
      if (!aligned16(ws)) return FACT_ERR_BAD_ALIGNMENT;
      plan.p.sk_ws = reinterpret_cast<float*>(ws);
      plan.p.sk_flags = h->sk_flags();
    }
    if (split) {
      if (!ws || ws_bytes < plan.ws_bytes) return FACT_ERR_WORKSPACE_TOO_SMALL;
      if (!aligned16(ws)) return FACT_ERR_BAD_ALIGNMENT;
      plan.p.store_tma = 1;  // partials always go through the staged path: the workspace layout is the library's
      plan.p.r_tma = 0;
      plan.p.ws = reinterpret_cast<const float*>(ws);
      // the reduction runs in the kernel's tail (the grid never exceeds the SM count, so the barrier there is safe)
      // unless the slices are few enough for the wide walk of the stand-alone reduction kernel
      plan.p.fused_reduce = !(plan.cfg.split_k <= kReduceWideSlices && q.epi != FACT_EPI_SILU_GATE &&
                              (plan.p.ws_ld & 7) == 0);
      plan.p.reduce_epi = (int)q.epi;
    }
    if (h->debug_flags & 256) {  // the all-CTA span stamps start from "no start yet" / "no end yet"
      cudaMemsetAsync(h->d_status + 40, 0xff, 2 * sizeof(int), stream);
      cudaMemsetAsync(h->d_status + 42, 0, 2 * sizeof(int), stream);
    }
    CUtensorMap tm[4];  // A, B, output (or split-K workspace), residual
    CUtensorMap& tmA = tm[0];
    CUtensorMap& tmB = tm[1];
    memset(tm, 0, sizeof tm);
    const uint64_t batch_dim = (uint64_t)q.batch;
    const uint64_t b_batch_dim = q.groups > 0 ? (uint64_t)q.groups : batch_dim;  // grouped: B is W[group]
    const bool b_strided = q.batch > 1 || q.groups > 0;
    if (q.groups > 0) {
      cudaError_t e = cudaMemcpyAsync(h->d_groups, group_table.data(), group_table.size() * sizeof(int),
                                      cudaMemcpyHostToDevice, stream);  // pageable source: staged before it returns
      if (e != cudaSuccess) return cuda_fail(h, "cudaMemcpyAsync(group table)", e);
    }
    const uint64_t sA = q.batch > 1 ? (uint64_t)q.strideA : (uint64_t)q.lda * (uint64_t)q.M;
    const uint32_t kbox = (uint32_t)q.k_elems();  // 128 bytes of K
    st = encode_map(h, &tmA, q.A, (uint64_t)q.K, (uint64_t)q.M, batch_dim, (uint64_t)q.lda, std::max<uint64_t>(sA, 16),
                    kbox, kTileM, false, q.fp8);
    if (st != FACT_OK) return st;
    if (q.layout == FACT_B_KN) {
      const uint64_t sB = b_strided ? (uint64_t)q.strideB : (uint64_t)q.ldb * (uint64_t)q.K;
      st = encode_map(h, &tmB, q.B, (uint64_t)q.Nw(), (uint64_t)q.K, b_batch_dim, (uint64_t)q.ldb,
                      std::max<uint64_t>(sB, 8), 64, kTileK);
    } else {
      const uint64_t sB = b_strided ? (uint64_t)q.strideB : (uint64_t)q.ldb * (uint64_t)q.Nw();
      st = encode_map(h, &tmB, q.B, (uint64_t)q.K, (uint64_t)q.Nw(), b_batch_dim, (uint64_t)q.ldb,
                      std::max<uint64_t>(sB, 16), kbox, (uint32_t)plan.p.b_box_n, false, q.fp8);
    }
    if (st != FACT_OK) return st;
    if (split) {
      // FP32 partial planes: (ws_ld, M, splits * batch * planes), stored 32 columns x 32 rows at a time
      const uint64_t planes = (uint64_t)plan.cfg.split_k * q.batch * plan.p.ws_planes;
      st = encode_map(h, &tm[2], ws, (uint64_t)plan.p.ws_ld, (uint64_t)q.M, planes, (uint64_t)plan.p.ws_ld,
                      (uint64_t)plan.p.ws_ld * (uint64_t)q.M, 32, 32, true);
      if (st != FACT_OK) return st;
    } else if (plan.p.store_tma && !plan.kcluster) {
      const bool f32 = q.out == FACT_OUT_F32;
      const uint64_t sC = q.batch > 1 ? (uint64_t)q.strideC : (uint64_t)q.ldc * (uint64_t)q.M;
      st = encode_map(h, &tm[2], q.C, (uint64_t)q.N_out, (uint64_t)q.M, batch_dim, (uint64_t)q.ldc,
                      std::max<uint64_t>(sC, 8), f32 ? 32 : 64, 32, f32);
      if (st != FACT_OK) return st;
      if (plan.p.r_tma) {
        const uint64_t sR = q.batch > 1 ? (uint64_t)q.strideR : (uint64_t)q.ldr * (uint64_t)q.M;
        st = encode_map(h, &tm[3], q.R, (uint64_t)q.N_out, (uint64_t)q.M, batch_dim, (uint64_t)q.ldr,
                        std::max<uint64_t>(sR, 8), 64, 32, false);
        if (st != FACT_OK) return st;
      }
    }
    const int epi = split ? (int)kEpiPartial : (int)q.epi;
    const bool two = plan.cfg.cta_group == 2;
    if (plan.kcluster) st = launch_kcluster(h, epi, plan, tm, stream);
    else if (q.groups > 0 && plan.dynamic) st = two ? launch_epi_dp<2, true, true>(h, epi, plan, tm, stream)
                                               : launch_epi_dp<1, true, true>(h, epi, plan, tm, stream);
    else if (q.groups > 0) st = two ? launch_epi_dp<2, true, false>(h, epi, plan, tm, stream)
                                    : launch_epi_dp<1, true, false>(h, epi, plan, tm, stream);
    else if (plan.dynamic) st = two ? launch_epi_dp<2, false, true>(h, epi, plan, tm, stream)
                                    : launch_epi_dp<1, false, true>(h, epi, plan, tm, stream);
    else if (plan.p.row_stores && !split) st = plan.cfg.cta_group == 2 ? launch_epi_ext<2, 3>(h, epi, plan, tm, stream)
                                                                       : launch_epi_ext<1, 3>(h, epi, plan, tm, stream);
    else if (q.norm) st = plan.cfg.cta_group == 2 ? launch_epi_ext<2, 2>(h, epi, plan, tm, stream)
                                                  : launch_epi_ext<1, 2>(h, epi, plan, tm, stream);
    else if (q.stats_out) st = plan.cfg.cta_group == 2 ? launch_epi_ext<2, 1>(h, epi, plan, tm, stream)
                                                       : launch_epi_ext<1, 1>(h, epi, plan, tm, stream);
    else if (stream_k) st = plan.cfg.cta_group == 2 ? launch_epi_sk<2>(h, epi, plan, tm, stream)
                                                    : launch_epi_sk<1>(h, epi, plan, tm, stream);
    else if (plan.cfg.cta_group == 2) st = launch_epi<2>(h, epi, plan, tm, stream);
    else st = launch_epi<1>(h, epi, plan, tm, stream);
    if (st == FACT_OK && split && !plan.p.fused_reduce)
      st = launch_reduce(h, q, plan, plan.cfg.split_k, reinterpret_cast<const float*>(ws), stream);
  }
  if (dev != h->device) cudaSetDevice(dev);
  return st;
}

// Which items of a causal attention problem every CTA takes: the items in order of weight (the key blocks an item's
// later tile sees, plus about one block of fixed cost), each given to the CTA that has the least so far (the lower
// CTA on a tie, so the first round is CTA c <- item c).  Item idx is (query pair qr = idx / bh counted from the
// end of the sequence, head idx % bh), the kernel's own numbering.
void build_attention_deal(int G, long long bh, int q_pairs, int bk, long long seq_kv, AttnDeal& d) {
  const int items = (int)(bh * q_pairs);
  const int kv_blocks = (int)((seq_kv + bk - 1) / bk);
  std::vector<std::vector<uint16_t>> mine((size_t)G);
  using Slot = std::pair<double, int>;  // (load, CTA)
  std::priority_queue<Slot, std::vector<Slot>, std::greater<Slot>> heap;
  for (int c = 0; c < G; ++c) heap.push({0.0, c});
  for (int idx = 0; idx < items; ++idx) {
    const int qp = q_pairs - 1 - (int)(idx / bh);
    const int nb1 = std::min(kv_blocks, (qp * 2 * kAttnBlockQ + 2 * kAttnBlockQ - 1) / bk + 1);
    const double w = nb1 + (bk == 128 ? 1.0 : 2.0);
    const Slot s = heap.top();
    heap.pop();
    mine[(size_t)s.second].push_back((uint16_t)idx);
    heap.push({s.first + w, s.second});
  }
  int pos = 0;
  for (int c = 0; c < G; ++c) {
    d.off[c] = (uint16_t)pos;
    for (uint16_t v : mine[(size_t)c]) d.list[pos++] = v;
  }
  d.off[G] = (uint16_t)pos;
}

Problem make_problem(fact_op_t op, long long batch, long long M, long long N, long long K, const void* A,
                     long long lda, long long sA, const void* B, long long ldb, long long sB, fact_blayout_t layout,
                     const void* bias, const void* R, long long ldr, long long sR, void* C, long long ldc,
                     long long sC, fact_out_t out, fact_epilogue_t epi) {
  Problem q;
  q.op = op;
  q.batch = batch;
  q.M = M;
  q.N_out = N;
  q.K = K;
  q.A = A;
  q.lda = lda;
  q.strideA = sA;
  q.B = B;
  q.ldb = ldb;
  q.strideB = sB;
  q.layout = layout;
  q.bias = bias;
  q.R = R;
  q.ldr = ldr;
  q.strideR = sR;
  q.C = C;
  q.ldc = ldc;
  q.strideC = sC;
  q.out = out;
  q.epi = epi;
  q.fp8 = op == FACT_OP_LINEAR_FP8;
  q.alpha = 1.f;
  return q;
}

}  // namespace

extern "C" {

const char* fact_status_string(fact_status_t s) {
  switch (s) {
    case FACT_OK: return "FACT_OK";
    case FACT_ERR_INVALID_ARG: return "FACT_ERR_INVALID_ARG";
    case FACT_ERR_BAD_ALIGNMENT: return "FACT_ERR_BAD_ALIGNMENT";
    case FACT_ERR_UNSUPPORTED: return "FACT_ERR_UNSUPPORTED";
    case FACT_ERR_ARCH: return "FACT_ERR_ARCH";
    case FACT_ERR_WORKSPACE_TOO_SMALL: return "FACT_ERR_WORKSPACE_TOO_SMALL";
    case FACT_ERR_CUDA: return "FACT_ERR_CUDA";
    case FACT_ERR_DEVICE_TIMEOUT: return "FACT_ERR_DEVICE_TIMEOUT";
    default: return "FACT_ERR_UNKNOWN";
  }
}

fact_status_t fact_create(fact_handle_t* handle, int device) {
  if (!handle) return FACT_ERR_INVALID_ARG;
  *handle = nullptr;
  int n = 0;
  if (cudaGetDeviceCount(&n) != cudaSuccess || device < 0 || device >= n) {
    cudaGetLastError();
    return FACT_ERR_CUDA;
  }
  if (cudaSetDevice(device) != cudaSuccess) return FACT_ERR_CUDA;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return FACT_ERR_CUDA;
  if (prop.major != 10) return FACT_ERR_ARCH;
  fact_handle_s* h = new fact_handle_s();
  h->device = device;
  h->sm_count = prop.multiProcessorCount;
  h->max_smem = (int)prop.sharedMemPerBlockOptin;
  h->cc_major = prop.major;
  h->cc_minor = prop.minor;
  if (const char* dbg = getenv("FACT_DEBUG_FLAGS")) h->debug_flags = atoi(dbg);
#ifndef FACT_EXPERIMENTS
  h->debug_flags &= kDiagnosticFlags;  // the work-skipping switches do not exist in this build
#endif
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
      qres != cudaDriverEntryPointSuccess) {
    delete h;
    return FACT_ERR_CUDA;
  }
  h->encode = reinterpret_cast<EncodeTiledFn>(fn);
  if (cudaMalloc(&h->d_status, h->status_ints() * sizeof(int)) != cudaSuccess ||
      cudaMemset(h->d_status, 0, h->status_ints() * sizeof(int)) != cudaSuccess) {
    delete h;
    return FACT_ERR_CUDA;
  }
  if (cudaMalloc(&h->d_groups, 2 * (kMaxGroups + 1) * sizeof(int)) != cudaSuccess) {
    cudaFree(h->d_status);
    delete h;
    return FACT_ERR_CUDA;
  }
  *handle = h;
  return FACT_OK;
}

fact_status_t fact_destroy(fact_handle_t h) {
  if (!h) return FACT_OK;
  for (cudaStream_t st : h->host_streams)
    if (st) {
      cudaStreamSynchronize(st);
      cudaStreamDestroy(st);
    }
  for (cudaEvent_t e : h->host_events)
    if (e) cudaEventDestroy(e);
  for (auto& kv : h->scratch_busy) cudaEventDestroy(kv.second);
  if (h->d_groups) cudaFree(h->d_groups);
  if (h->d_status) cudaFree(h->d_status);
  delete h;
  return FACT_OK;
}

fact_status_t fact_device_info(fact_handle_t h, int* sm_count, int* max_smem, int* cc_major, int* cc_minor) {
  if (!h) return FACT_ERR_INVALID_ARG;
  if (sm_count) *sm_count = h->sm_count;
  if (max_smem) *max_smem = h->max_smem;
  if (cc_major) *cc_major = h->cc_major;
  if (cc_minor) *cc_minor = h->cc_minor;
  return FACT_OK;
}

fact_status_t fact_attention_deal(int ctas, int64_t batch_heads, int64_t seq, int head_dim, int cta, int max_items,
                                  int32_t* items, int* n_items) {
  if (ctas < 1 || ctas > kAttnDealCtas || batch_heads < 1 || seq < 1 || (head_dim != 64 && head_dim != 128) || cta < 0 ||
      cta >= ctas || max_items < 0 || !n_items || (max_items > 0 && !items))
    return FACT_ERR_INVALID_ARG;
  const long long q_pairs = (seq + 2 * kAttnBlockQ - 1) / (2 * kAttnBlockQ);
  if (batch_heads * q_pairs > kAttnDealItems) return FACT_ERR_UNSUPPORTED;
  std::unique_ptr<AttnDeal> d(new AttnDeal());
  build_attention_deal(ctas, batch_heads, (int)q_pairs, head_dim == 64 ? 128 : 64, seq, *d);
  const int n = (int)d->off[cta + 1] - (int)d->off[cta];
  *n_items = n;
  for (int i = 0; i < n && i < max_items; ++i) items[i] = d->list[d->off[cta] + i];
  return FACT_OK;
}

fact_status_t fact_stream_k_pieces(int groups, int64_t sk_tiles, int64_t k_blocks, int group, int max_pieces,
                                   int32_t* pieces, int* n_pieces) {
  if (groups < 1 || sk_tiles < 0 || k_blocks < 1 || group < 0 || group >= groups || max_pieces < 0 || !n_pieces ||
      (max_pieces > 0 && !pieces) || sk_tiles * k_blocks > 0x3fffffffLL)
    return FACT_ERR_INVALID_ARG;
  const long long iters = sk_tiles * k_blocks;
  const int len = (int)(iters / groups), rem = (int)(iters % groups);
  int pos = sk_group_begin(len, rem, group);
  const int end = sk_group_begin(len, rem, group + 1);
  int n = 0;
  while (pos < end) {
    const SkPiece pc = sk_next_piece((int)k_blocks, len, rem, groups, group, pos, end);
    if (n < max_pieces) {
      int32_t* row = pieces + 5 * n;
      row[0] = pc.tile;
      row[1] = pc.k0;
      row[2] = pc.k1;
      row[3] = pc.role;
      row[4] = pc.peers;
    }
    ++n;
  }
  *n_pieces = n;
  return FACT_OK;
}

int64_t fact_launch_count(fact_handle_t h) { return h ? h->launches : 0; }

fact_status_t fact_last_kernel_clock(fact_handle_t h, void* stream, int64_t* sm_cycles, int64_t* nanoseconds) {
  if (!h || !sm_cycles || !nanoseconds) return FACT_ERR_INVALID_ARG;
  if (cudaStreamSynchronize(reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess) return FACT_ERR_CUDA;
  long long v[2] = {0, 0};
  if (cudaMemcpy(v, h->d_status + 2, sizeof v, cudaMemcpyDeviceToHost) != cudaSuccess) return FACT_ERR_CUDA;
  *sm_cycles = v[0];
  *nanoseconds = v[1];
  return FACT_OK;
}

fact_status_t fact_last_kernel_profile(fact_handle_t h, void* stream, int64_t counters[8]) {
  if (!h || !counters) return FACT_ERR_INVALID_ARG;
  if (cudaStreamSynchronize(reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess) return FACT_ERR_CUDA;
  long long v[8];
  if (cudaMemcpy(v, h->d_status + 2, sizeof v, cudaMemcpyDeviceToHost) != cudaSuccess) return FACT_ERR_CUDA;
  for (int i = 0; i < 8; ++i) counters[i] = v[i];
  return FACT_OK;
}

fact_status_t fact_last_kernel_span(fact_handle_t h, void* stream, int64_t* nanoseconds) {
  if (!h || !nanoseconds) return FACT_ERR_INVALID_ARG;
  if (cudaStreamSynchronize(reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess) return FACT_ERR_CUDA;
  unsigned long long v[2] = {0, 0};
  if (cudaMemcpy(v, h->d_status + 40, sizeof v, cudaMemcpyDeviceToHost) != cudaSuccess) return FACT_ERR_CUDA;
  *nanoseconds = (v[1] > v[0] && v[0] != ~0ull) ? (int64_t)(v[1] - v[0]) : 0;
  return FACT_OK;
}

fact_status_t fact_selftest_wait_timeout(fact_handle_t h, void* stream, double limit_ms) {
  if (!h || !(limit_ms > 0.0) || limit_ms > 1000.0) return FACT_ERR_INVALID_ARG;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  // d_status[30] receives "the wait gave up" (1) or "the wait returned" (0)
  if (cudaMemsetAsync(h->d_status + 30, 0xff, sizeof(int), s) != cudaSuccess) return FACT_ERR_CUDA;
  fact_wait_timeout_selftest_kernel<<<1, 32, 0, s>>>(h->d_status, (unsigned long long)(limit_ms * 1e6), h->d_status + 30);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(h, "wait-timeout self-test launch", e);
  if (cudaStreamSynchronize(s) != cudaSuccess) return FACT_ERR_CUDA;
  int gave_up = -1;
  if (cudaMemcpy(&gave_up, h->d_status + 30, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return FACT_ERR_CUDA;
  return gave_up == 1 ? FACT_OK : FACT_ERR_CUDA;
}

const char* fact_last_error(fact_handle_t h) { return h ? h->last_error.c_str() : ""; }

fact_status_t fact_device_status(fact_handle_t h, void* stream, int* status) {
  if (!h || !status) return FACT_ERR_INVALID_ARG;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  if (cudaStreamSynchronize(s) != cudaSuccess) return FACT_ERR_CUDA;
  int v = 0;
  if (cudaMemcpy(&v, h->d_status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return FACT_ERR_CUDA;
  // (a launch that gave up may have left stream-K flags and grid-barrier counters set: clear them with the word)
  if (v != 0 && (cudaMemset(h->d_status, 0, sizeof(int)) != cudaSuccess ||
                 cudaMemset(h->d_status + 24, 0, 2 * sizeof(int)) != cudaSuccess ||
                 cudaMemset(h->sk_flags(), 0, (size_t)h->sm_count * kEpiWarps * sizeof(int)) != cudaSuccess))
    return FACT_ERR_CUDA;
  *status = v;
  return FACT_OK;
}

static Problem shape_only(fact_op_t op, int64_t batch, int64_t M, int64_t N, int64_t K, fact_epilogue_t epi,
                          fact_blayout_t layout, fact_out_t out) {
  return make_problem(op, batch, M, N, K, nullptr, K, 0, nullptr, 0, 0, layout, nullptr, nullptr, 0, 0, nullptr, N, 0,
                      out, epi);
}

fact_status_t fact_get_config(fact_handle_t h, fact_op_t op, int64_t batch, int64_t M, int64_t N, int64_t K,
                              fact_epilogue_t epi, fact_blayout_t layout, fact_out_t out, fact_config_t* cfg_out) {
  if (!h || !cfg_out || batch < 0 || M < 0 || N < 0 || K < 0) return FACT_ERR_INVALID_ARG;
  Problem q = shape_only(op, batch, M, N, K, epi, layout, out);
  return resolve_config(h, q, nullptr, 0, cfg_out);
}

fact_status_t fact_workspace_bytes(fact_handle_t h, fact_op_t op, int64_t batch, int64_t M, int64_t N, int64_t K,
                                   fact_epilogue_t epi, fact_blayout_t layout, fact_out_t out,
                                   const fact_config_t* cfg, size_t* bytes) {
  if (!h || !bytes || batch < 0 || M < 0 || N < 0 || K < 0) return FACT_ERR_INVALID_ARG;
  Problem q = shape_only(op, batch, M, N, K, epi, layout, out);
  fact_config_t c;
  fact_status_t st = resolve_config(h, q, cfg, 0, &c);
  if (st != FACT_OK) return st;
  *bytes = workspace_for(h, q, c);
  return FACT_OK;
}

fact_status_t fact_gemm(fact_handle_t h, int64_t M, int64_t N, int64_t K, const void* A, int64_t lda, const void* B,
                        int64_t ldb, fact_blayout_t layout, void* C, int64_t ldc, fact_out_t out,
                        const fact_config_t* cfg, void* ws, size_t ws_bytes, void* stream) {
  Problem q = make_problem(FACT_OP_GEMM, 1, M, N, K, A, lda, 0, B, ldb, 0, layout, nullptr, nullptr, 0, 0, C, ldc, 0,
                           out, FACT_EPI_NONE);
  return run(h, q, cfg, 0, ws, ws_bytes, stream);
}

namespace {
// Device copies of A, B and C of a host-buffer product (operand rows padded to whole 16-byte pieces), each on a
// 256-byte boundary; the product's own workspace, if its configuration wants one, follows.
size_t host_gemm_operand_bytes(int64_t M, int64_t N, int64_t K, fact_out_t out) {
  auto up = [](size_t v) { return (v + 255) & ~(size_t)255; };
  auto up8 = [](int64_t v) { return (size_t)((v + 7) / 8 * 8); };
  return up((size_t)M * up8(K) * 2) + up(std::max(up8(K) * (size_t)N, up8(N) * (size_t)K) * 2) +
         up((size_t)M * N * (out == FACT_OUT_F32 ? 4 : 2));
}
}  // namespace

fact_status_t fact_gemm_host_scratch_bytes(fact_handle_t h, int64_t M, int64_t N, int64_t K, fact_blayout_t layout,
                                           fact_out_t out, const fact_config_t* cfg, size_t* bytes) {
  if (!h || !bytes || M < 0 || N < 0 || K < 0) return FACT_ERR_INVALID_ARG;
  Problem q = shape_only(FACT_OP_GEMM, 1, M, N, K, FACT_EPI_NONE, layout, out);
  fact_config_t c;
  const fact_status_t st = resolve_config(h, q, cfg, 0, &c);
  if (st != FACT_OK) return st;
  *bytes = host_gemm_operand_bytes(M, N, K, out) + workspace_for(h, q, c);
  return FACT_OK;
}

fact_status_t fact_gemm_host(fact_handle_t h, int64_t M, int64_t N, int64_t K, const void* A_host, int64_t lda,
                             const void* B_host, int64_t ldb, fact_blayout_t layout, void* C_host, int64_t ldc,
                             fact_out_t out, const fact_config_t* cfg, void* scratch, size_t scratch_bytes,
                             void* stream_v) {
  if (!h || M < 0 || N < 0 || K < 0) return FACT_ERR_INVALID_ARG;
  if (layout != FACT_B_KN && layout != FACT_B_NK) return FACT_ERR_INVALID_ARG;
  if (out != FACT_OUT_BF16 && out != FACT_OUT_F32) return FACT_ERR_INVALID_ARG;
  if (M == 0 || N == 0) return FACT_OK;
  const int64_t b_rows = layout == FACT_B_KN ? K : N, b_cols = layout == FACT_B_KN ? N : K;
  if (!C_host || ldc < N || (K > 0 && (!A_host || !B_host || lda < K || ldb < b_cols))) return FACT_ERR_INVALID_ARG;
  const size_t operand_bytes = host_gemm_operand_bytes(M, N, K, out);
  if (!scratch || scratch_bytes < operand_bytes) return FACT_ERR_WORKSPACE_TOO_SMALL;
  if (reinterpret_cast<uintptr_t>(scratch) & 255u) return FACT_ERR_BAD_ALIGNMENT;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return FACT_ERR_CUDA;
  if (dev != h->device && cudaSetDevice(h->device) != cudaSuccess) return FACT_ERR_CUDA;
  auto fail = [&](const char* where, cudaError_t e) {
    const fact_status_t r = cuda_fail(h, where, e);
    if (dev != h->device) cudaSetDevice(dev);
    return r;
  };
  if (!h->host_streams[0]) {  // first call: the three streams and the event ring (no device memory)
    for (int i = 0; i < 3; ++i) {
      cudaError_t e = cudaStreamCreateWithFlags(&h->host_streams[i], cudaStreamNonBlocking);
      if (e != cudaSuccess) return fail("cudaStreamCreate (fact_gemm_host)", e);
    }
    for (int i = 0; i < fact_handle_s::kHostEvents; ++i) {
      cudaError_t e = cudaEventCreateWithFlags(&h->host_events[i], cudaEventDisableTiming);
      if (e != cudaSuccess) return fail("cudaEventCreate (fact_gemm_host)", e);
    }
  }
  auto next_event = [&]() {
    cudaEvent_t e = h->host_events[h->host_event_next];
    h->host_event_next = (h->host_event_next + 1) % fact_handle_s::kHostEvents;
    return e;
  };
  cudaStream_t caller = reinterpret_cast<cudaStream_t>(stream_v);
  cudaStream_t s_in = h->host_streams[0], s_mm = h->host_streams[1], s_out = h->host_streams[2];
  auto up = [](size_t v) { return (v + 255) & ~(size_t)255; };
  auto up8 = [](int64_t v) { return (size_t)((v + 7) / 8 * 8); };
  const size_t esz_c = out == FACT_OUT_F32 ? 4 : 2;
  const size_t lda_dev = up8(K), ldb_dev = up8(b_cols);  // operand rows padded to whole 16-byte pieces (TMA)
  uint8_t* dA = reinterpret_cast<uint8_t*>(scratch);
  uint8_t* dB = dA + up((size_t)M * lda_dev * 2);
  uint8_t* dC = dB + up(std::max(up8(K) * (size_t)N, up8(N) * (size_t)K) * 2);
  cudaError_t e;
  // what the caller's stream has enqueued so far comes first; so does the copy-out of the call that last used this
  // scratch (a wait captures the event's most recent record, so the ring may wrap)
  cudaEvent_t ev_entry = next_event();
  if ((e = cudaEventRecord(ev_entry, caller)) != cudaSuccess) return fail("cudaEventRecord", e);
  if ((e = cudaStreamWaitEvent(s_in, ev_entry, 0)) != cudaSuccess) return fail("cudaStreamWaitEvent", e);
  auto busy = h->scratch_busy.find(scratch);
  if (busy == h->scratch_busy.end()) {  // first use of this scratch: an event of its own
    cudaEvent_t ne;
    if ((e = cudaEventCreateWithFlags(&ne, cudaEventDisableTiming)) != cudaSuccess) return fail("cudaEventCreate", e);
    busy = h->scratch_busy.emplace(scratch, ne).first;
  } else if ((e = cudaStreamWaitEvent(s_in, busy->second, 0)) != cudaSuccess) {
    return fail("cudaStreamWaitEvent", e);
  }
  // one flat copy where source and destination rows are back to back, a pitched copy otherwise
  auto copy_rows = [](void* dst, size_t dpitch, const void* src, size_t spitch, size_t width, size_t rows,
                      cudaMemcpyKind kind, cudaStream_t st) {
    if (dpitch == width && spitch == width) return cudaMemcpyAsync(dst, src, width * rows, kind, st);
    return cudaMemcpy2DAsync(dst, dpitch, src, spitch, width, rows, kind, st);
  };
  if (K > 0) {
    if ((e = copy_rows(dA, lda_dev * 2, A_host, (size_t)lda * 2, (size_t)K * 2, (size_t)M, cudaMemcpyHostToDevice,
                       s_in)) != cudaSuccess)
      return fail("copy of A to the device", e);
    if ((e = copy_rows(dB, ldb_dev * 2, B_host, (size_t)ldb * 2, (size_t)b_cols * 2, (size_t)b_rows,
                       cudaMemcpyHostToDevice, s_in)) != cudaSuccess)
      return fail("copy of B to the device", e);
  }
  cudaEvent_t ev_loaded = next_event();
  if ((e = cudaEventRecord(ev_loaded, s_in)) != cudaSuccess) return fail("cudaEventRecord", e);
  if ((e = cudaStreamWaitEvent(s_mm, ev_loaded, 0)) != cudaSuccess) return fail("cudaStreamWaitEvent", e);
  Problem q = make_problem(FACT_OP_GEMM, 1, M, N, K, dA, (long long)lda_dev, 0, dB, (long long)ldb_dev, 0, layout, nullptr,
                           nullptr, 0, 0, dC, N, 0, out, FACT_EPI_NONE);
  // what is left of the scratch behind the operands is the product's workspace (K slices, stream-K); a tuned entry
  // that wants more than there is runs without
  const fact_status_t st = run(h, q, cfg, 0, scratch_bytes > operand_bytes ? dA + operand_bytes : nullptr,
                               scratch_bytes - operand_bytes, s_mm);
  if (st != FACT_OK) {
    if (dev != h->device) cudaSetDevice(dev);
    return st;
  }
  cudaEvent_t ev_done = next_event();
  if ((e = cudaEventRecord(ev_done, s_mm)) != cudaSuccess) return fail("cudaEventRecord", e);
  if ((e = cudaStreamWaitEvent(s_out, ev_done, 0)) != cudaSuccess) return fail("cudaStreamWaitEvent", e);
  if ((e = copy_rows(C_host, (size_t)ldc * esz_c, dC, (size_t)N * esz_c, (size_t)N * esz_c, (size_t)M,
                     cudaMemcpyDeviceToHost, s_out)) != cudaSuccess)
    return fail("copy of C to the host", e);
  cudaEvent_t ev_out = busy->second;
  if ((e = cudaEventRecord(ev_out, s_out)) != cudaSuccess) return fail("cudaEventRecord", e);
  if (dev != h->device) cudaSetDevice(dev);
  return FACT_OK;
}

fact_status_t fact_gemm_host_wait(fact_handle_t h, void* stream_v) {
  if (!h) return FACT_ERR_INVALID_ARG;
  if (!h->host_streams[2]) return FACT_OK;  // no host-buffer call has run
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return FACT_ERR_CUDA;
  if (dev != h->device && cudaSetDevice(h->device) != cudaSuccess) return FACT_ERR_CUDA;
  cudaEvent_t ev = h->host_events[h->host_event_next];
  h->host_event_next = (h->host_event_next + 1) % fact_handle_s::kHostEvents;
  fact_status_t st = FACT_OK;
  cudaError_t e = cudaEventRecord(ev, h->host_streams[2]);  // copy-outs complete in the order they were enqueued
  if (e == cudaSuccess) e = cudaStreamWaitEvent(reinterpret_cast<cudaStream_t>(stream_v), ev, 0);
  if (e != cudaSuccess) st = cuda_fail(h, "fact_gemm_host_wait", e);
  if (dev != h->device) cudaSetDevice(dev);
  return st;
}

fact_status_t fact_gemm_batched(fact_handle_t h, int64_t batch, int64_t M, int64_t N, int64_t K, const void* A,
                                int64_t lda, int64_t strideA, const void* B, int64_t ldb, int64_t strideB,
                                fact_blayout_t layout, void* C, int64_t ldc, int64_t strideC, fact_out_t out,
                                const fact_config_t* cfg, void* ws, size_t ws_bytes, void* stream) {
  Problem q = make_problem(FACT_OP_GEMM_BATCHED, batch, M, N, K, A, lda, strideA, B, ldb, strideB, layout, nullptr,
                           nullptr, 0, 0, C, ldc, strideC, out, FACT_EPI_NONE);
  return run(h, q, cfg, 0, ws, ws_bytes, stream);
}

fact_status_t fact_gemm_splitk(fact_handle_t h, int64_t M, int64_t N, int64_t K, const void* A, int64_t lda,
                               const void* B, int64_t ldb, fact_blayout_t layout, void* C, int64_t ldc,
                               fact_out_t out, int splits, const fact_config_t* cfg, void* ws, size_t ws_bytes,
                               void* stream) {
  if (splits < 0) return FACT_ERR_INVALID_ARG;
  Problem q = make_problem(FACT_OP_GEMM_SPLITK, 1, M, N, K, A, lda, 0, B, ldb, 0, layout, nullptr, nullptr, 0, 0, C,
                           ldc, 0, out, FACT_EPI_NONE);
  return run(h, q, cfg, splits, ws, ws_bytes, stream);
}

fact_status_t fact_linear(fact_handle_t h, int64_t M, int64_t N_out, int64_t K, const void* X, int64_t ldx,
                          const void* W, int64_t ldw, fact_blayout_t layout, const void* bias, const void* residual,
                          int64_t ldr, void* Y, int64_t ldy, fact_out_t out, fact_epilogue_t epi,
                          const fact_config_t* cfg, void* ws, size_t ws_bytes, void* stream) {
  Problem q = make_problem(FACT_OP_LINEAR, 1, M, N_out, K, X, ldx, 0, W, ldw, 0, layout, bias, residual, ldr, 0, Y,
                           ldy, 0, out, epi);
  return run(h, q, cfg, 0, ws, ws_bytes, stream);
}

fact_status_t fact_linear_ex(fact_handle_t h, int64_t M, int64_t N_out, int64_t K, const void* X, int64_t ldx,
                             const void* W, int64_t ldw, fact_blayout_t layout, const void* bias, const void* residual,
                             int64_t ldr, void* Y, int64_t ldy, fact_out_t out, fact_epilogue_t epi,
                             const fact_linear_ext_t* ext, const fact_config_t* cfg, void* ws, size_t ws_bytes,
                             void* stream) {
  Problem q = make_problem(FACT_OP_LINEAR, 1, M, N_out, K, X, ldx, 0, W, ldw, 0, layout, bias, residual, ldr, 0, Y,
                           ldy, 0, out, epi);
  if (ext) {
    if (ext->x_norm != FACT_XNORM_NONE && ext->x_norm != FACT_XNORM_LAYER && ext->x_norm != FACT_XNORM_RMS)
      return FACT_ERR_INVALID_ARG;
    q.stats_out = ext->row_stats_out;
    q.norm = (int)ext->x_norm;
    q.stats_in = ext->x_row_stats;
    q.colsum = ext->w_colsum;
    q.norm_eps = ext->eps;
    if (q.norm == 0 && (q.stats_in || q.colsum)) return FACT_ERR_INVALID_ARG;
  }
  return run(h, q, cfg, 0, ws, ws_bytes, stream);
}

static fact_status_t linear_grouped_impl(fact_handle_t h, bool fp8, float scale, int groups, const int64_t* group_rows,
                                         int64_t N_out, int64_t K, const void* X, int64_t ldx, const void* W,
                                         int64_t ldw, int64_t strideW, fact_blayout_t layout, const void* bias,
                                         const void* residual, int64_t ldr, void* Y, int64_t ldy, fact_out_t out,
                                         fact_epilogue_t epi, const fact_config_t* cfg, void* stream) {
  if (!h || groups < 0 || groups > kMaxGroups || (groups > 0 && !group_rows) || strideW < 0) return FACT_ERR_INVALID_ARG;
  if (!(scale == scale) || std::isinf(scale)) return FACT_ERR_INVALID_ARG;
  long long M = 0;
  for (int g = 0; g < groups; ++g) {
    if (group_rows[g] < 0) return FACT_ERR_INVALID_ARG;
    M += group_rows[g];
    if (M > 0x7fffffffLL - 512) return FACT_ERR_INVALID_ARG;
  }
  if (groups == 0 || M == 0) return FACT_OK;
  if (cfg && (cfg->split_k > 1 || cfg->split_k < 0)) return FACT_ERR_UNSUPPORTED;
  if (epi == FACT_EPI_BIAS_SOFTMAX) return FACT_ERR_UNSUPPORTED;
  Problem q = make_problem(fp8 ? FACT_OP_LINEAR_FP8 : FACT_OP_LINEAR, 1, M, N_out, K, X, ldx, 0, W, ldw, strideW, layout,
                           bias, residual, ldr, 0, Y, ldy, 0, out, epi);
  q.groups = groups;
  q.group_rows = group_rows;
  q.alpha = scale;
  if (strideW % q.op_align()) return FACT_ERR_BAD_ALIGNMENT;
  const long long w_rows = layout == FACT_B_KN ? K : q.Nw();
  if (groups > 1 && K > 0 && strideW < w_rows * ldw) return FACT_ERR_INVALID_ARG;  // the groups' weights overlap
  return run(h, q, cfg, 0, nullptr, 0, stream);
}

fact_status_t fact_linear_grouped(fact_handle_t h, int groups, const int64_t* group_rows, int64_t N_out, int64_t K,
                                  const void* X, int64_t ldx, const void* W, int64_t ldw, int64_t strideW,
                                  fact_blayout_t layout, const void* bias, const void* residual, int64_t ldr, void* Y,
                                  int64_t ldy, fact_out_t out, fact_epilogue_t epi, const fact_config_t* cfg,
                                  void* stream) {
  return linear_grouped_impl(h, false, 1.f, groups, group_rows, N_out, K, X, ldx, W, ldw, strideW, layout, bias, residual,
                             ldr, Y, ldy, out, epi, cfg, stream);
}

fact_status_t fact_linear_grouped_fp8(fact_handle_t h, int groups, const int64_t* group_rows, int64_t N_out, int64_t K,
                                      const void* X, int64_t ldx, const void* W, int64_t ldw, int64_t strideW,
                                      float scale, const void* bias, const void* residual, int64_t ldr, void* Y,
                                      int64_t ldy, fact_out_t out, fact_epilogue_t epi, const fact_config_t* cfg,
                                      void* stream) {
  return linear_grouped_impl(h, true, scale, groups, group_rows, N_out, K, X, ldx, W, ldw, strideW, FACT_B_NK, bias,
                             residual, ldr, Y, ldy, out, epi, cfg, stream);
}

fact_status_t fact_linear_fp8(fact_handle_t h, int64_t M, int64_t N_out, int64_t K, const void* X, int64_t ldx,
                              const void* W, int64_t ldw, float scale, const void* bias, const void* residual,
                              int64_t ldr, void* Y, int64_t ldy, fact_out_t out, fact_epilogue_t epi,
                              const fact_config_t* cfg, void* ws, size_t ws_bytes, void* stream) {
  if (!(scale == scale) || std::isinf(scale)) return FACT_ERR_INVALID_ARG;
  Problem q = make_problem(FACT_OP_LINEAR_FP8, 1, M, N_out, K, X, ldx, 0, W, ldw, 0, FACT_B_NK, bias, residual, ldr, 0,
                           Y, ldy, 0, out, epi);
  q.alpha = scale;
  return run(h, q, cfg, 0, ws, ws_bytes, stream);
}

fact_status_t fact_tune_ex(fact_handle_t h, fact_op_t op, int64_t batch, int64_t M, int64_t N, int64_t K,
                           const void* A, int64_t lda, int64_t strideA, const void* B, int64_t ldb, int64_t strideB,
                           fact_blayout_t layout, const void* bias, const void* residual, int64_t ldr,
                           int64_t strideR, void* C, int64_t ldc, int64_t strideC, fact_out_t out, fact_epilogue_t epi,
                           void* ws, size_t ws_bytes, int warmup, int iters, void* stream_v,
                           const fact_tune_opts_t* opts, fact_config_t* best, double* best_ms, int* n_tried) {
  if (!h || !best) return FACT_ERR_INVALID_ARG;
  Problem q = make_problem(op, batch, M, N, K, A, lda, strideA, B, ldb, strideB, layout, bias, residual, ldr, strideR,
                           C, ldc, strideC, out, epi);
  fact_status_t st = validate(q);
  if (st != FACT_OK) return st;
  if (q.batch == 0 || q.M == 0 || q.N_out == 0 || q.K == 0) return resolve_config(h, q, nullptr, 0, best);
  if (q.R && q.R == q.C) return FACT_ERR_UNSUPPORTED;  // every candidate would read the previous one's output
  if (warmup <= 0) warmup = 5;
  if (iters <= 0) iters = 20;
  const bool verify = !opts || opts->verify != 0;
  const bool cold = opts && opts->cold_l2 != 0;
  const int inject = opts ? opts->inject_fault : -1;
  fact_tune_record_t* recs = opts ? opts->records : nullptr;
  const int max_recs = (opts && recs) ? opts->max_records : 0;
  int n_recs = 0;
  auto record = [&](const fact_config_t& c, int status, double ms, double rel, double verr) -> int {
    const int at = n_recs++;
    if (at < max_recs) {
      recs[at].cfg = c;
      recs[at].status = status;
      recs[at].ms = (float)ms;
      recs[at].rel = (float)rel;
      recs[at].verify_err = (float)verr;
    }
    return at;
  };
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_v);
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return FACT_ERR_CUDA;
  if (dev != h->device && cudaSetDevice(h->device) != cudaSuccess) return FACT_ERR_CUDA;

  // The tuner is off the per-call path and owns what it needs for the length of this call: event pairs, a dense FP32
  // copy of the reference output for the verify gate, a buffer larger than L2 for the cold-L2 mode.
  const int n_ev = cold ? iters : 1;
  std::vector<cudaEvent_t> ev0((size_t)n_ev), ev1((size_t)n_ev);
  float* d_ref = nullptr;
  double* d_sum = nullptr;       // [0] sum |ref|, then two 32-bit result words behind it
  unsigned char* d_flush = nullptr;
  size_t flush_bytes = 0;
  bool setup_ok = true;
  for (int i = 0; i < n_ev; ++i)
    setup_ok = setup_ok && cudaEventCreate(&ev0[(size_t)i]) == cudaSuccess && cudaEventCreate(&ev1[(size_t)i]) == cudaSuccess;
  const long long out_elems = (long long)q.batch * q.M * q.N_out;
  if (verify)
    setup_ok = setup_ok && cudaMalloc(&d_ref, (size_t)out_elems * sizeof(float)) == cudaSuccess &&
               cudaMalloc(&d_sum, 2 * sizeof(double)) == cudaSuccess;
  if (cold) {
    int l2 = 0;
    cudaDeviceGetAttribute(&l2, cudaDevAttrL2CacheSize, h->device);
    flush_bytes = std::max<size_t>((size_t)256 << 20, 2 * (size_t)std::max(l2, 0));
    setup_ok = setup_ok && cudaMalloc(&d_flush, flush_bytes) == cudaSuccess;
  }
  auto cleanup = [&]() {
    for (int i = 0; i < n_ev; ++i) {
      cudaEventDestroy(ev0[(size_t)i]);
      cudaEventDestroy(ev1[(size_t)i]);
    }
    if (d_ref) cudaFree(d_ref);
    if (d_sum) cudaFree(d_sum);
    if (d_flush) cudaFree(d_flush);
    if (dev != h->device) cudaSetDevice(dev);
  };
  if (!setup_ok) {
    cudaGetLastError();
    cleanup();
    return FACT_ERR_CUDA;
  }

  // Candidate axes: pair size, tile width, ring depth, K slices / stream-K, store path.
  std::vector<fact_config_t> cands;
  const int k_blocks = (int)((K + q.k_elems() - 1) / q.k_elems());
  for (int cg = 1; cg <= 2; ++cg) {
    for (int tn = 32; tn <= 256; tn += 32) {
      if (!tile_ok(q, tn, cg)) continue;
      const int out_cols = epi == FACT_EPI_SILU_GATE ? tn / 2 : tn;
      if (out_cols >= 2 * N && tn > 64) continue;  // more than half the tile would be padding
      const int smax = max_stages_for(q, tn, cg);
      if (smax < 2) continue;
      const long long tiles = batch * ((M + 128 * cg - 1) / (128 * cg)) * ((N + out_cols - 1) / out_cols);
      const long long slots = h->sm_count / cg;
      // K slices: none, and -- when the tiles alone leave SMs idle, or the caller asked for a split --
      // enough to fill the machine once, half of that and twice that
      std::vector<int> splits = {1};
      if (op == FACT_OP_GEMM_SPLITK || tiles * 2 <= slots) {
        const long long fill = std::max<long long>(1, slots / std::max<long long>(tiles, 1));
        for (long long sp : {fill, fill / 2, fill * 2, fill / 4}) {
          sp = std::min<long long>(sp, k_blocks / 2);
          if (sp > 1 && std::find(splits.begin(), splits.end(), (int)sp) == splits.end()) splits.push_back((int)sp);
        }
      }
      // stream-K, when the last wave is partial and short enough in waves for that to matter
      if (tiles % slots != 0 && tiles <= 12 * slots) {
        splits.push_back(-1);
        if (tiles > slots) splits.push_back(-2);
      }
      std::vector<int> stage_opts = {smax};
      if (smax > 3) stage_opts.push_back(smax - 1);
      // (the raster group is not swept: its effect is on DRAM traffic and, through power, on the clock, which a
      // short timing run cannot resolve; the model in resolve_config chooses it)
      for (int stg : stage_opts)
        for (int sp : splits) {
          fact_config_t c = {128 * cg, tn, q.k_elems(), stg, cg, 0, sp, 0, 0};
          cands.push_back(c);
          // whole tiles with a long main loop: also with the rows stored from registers (infeasible ones drop out)
          if (sp == 1 && k_blocks >= 32) {
            c.store_mode = 3;
            cands.push_back(c);
            c.store_mode = 0;
          }
          // more than one wave of whole tiles: also handed out dynamically
          if (sp == 1 && tiles > slots && stg == smax) {
            c.schedule = 2;
            cands.push_back(c);
          }
        }
    }
  }
  // K slices as a cluster (schedule 3): up to two waves of clusters of at most 8 CTAs, the slices single CTAs or pairs
  // (make_plan refuses what the kernel cannot run: gated or row-softmax epilogues, 8-bit operands, groups)
  for (int cg = 1; cg <= 2; ++cg)
    for (int sl = 2; sl * cg <= 8; sl *= 2)
      for (int tn = 64; tn <= 256; tn *= 2) {
        if (tn % (32 * sl) || !tile_ok(q, tn, cg) || k_blocks < 2 * sl) continue;
        const int smax = max_stages_for(q, tn, cg);
        if (smax < 2) continue;
        const long long tiles = batch * ((M + 128 * cg - 1) / (128 * cg)) * ((N + tn - 1) / tn);
        if (tiles > 2LL * kc_max_clusters(h, sl, cg)) continue;
        fact_config_t c = {128 * cg, tn, q.k_elems(), smax, cg, 0, sl, 0, 3};
        cands.push_back(c);
      }
  // Time `c` over `n` launches (per launch, ms); a negative result means the candidate failed.  Warm L2: the launches
  // run back to back between one event pair.  Cold L2: a buffer twice the size of L2 is overwritten before each
  // launch and every launch has an event pair of its own (what a benchmark that flushes L2 between launches sees).
  double last_mhz = 0.0;  // SM clock inside the last launch of the most recent time_cfg (from the kernel's own stamps)
  auto time_cfg = [&](const fact_config_t& c, int n_warm, int n) -> double {
    bool ok = true;
    last_mhz = 0.0;
    for (int i = 0; i < n_warm && ok; ++i) ok = run(h, q, &c, 0, ws, ws_bytes, stream_v) == FACT_OK;
    if (!ok) return -1.0;
    n = cold ? std::min(n, n_ev) : n;
    if (cold) {
      for (int i = 0; i < n && ok; ++i) {
        ok = cudaMemsetAsync(d_flush, i & 0xff, flush_bytes, stream) == cudaSuccess;
        cudaEventRecord(ev0[(size_t)i], stream);
        ok = ok && run(h, q, &c, 0, ws, ws_bytes, stream_v) == FACT_OK;
        cudaEventRecord(ev1[(size_t)i], stream);
      }
    } else {
      cudaEventRecord(ev0[0], stream);
      for (int i = 0; i < n && ok; ++i) ok = run(h, q, &c, 0, ws, ws_bytes, stream_v) == FACT_OK;
      cudaEventRecord(ev1[0], stream);
    }
    int dev_status = 0;
    if (fact_device_status(h, stream_v, &dev_status) != FACT_OK || dev_status != 0 || !ok) return -1.0;
    double total = 0.0;
    for (int i = 0; i < (cold ? n : 1); ++i) {
      float ms = 0.f;
      if (cudaEventElapsedTime(&ms, ev0[(size_t)i], ev1[(size_t)i]) != cudaSuccess) return -1.0;
      total += ms;
    }
    long long stamp[2] = {0, 0};  // SM cycles and nanoseconds of the first CTA of the last launch
    if (cudaMemcpy(stamp, h->d_status + 2, sizeof stamp, cudaMemcpyDeviceToHost) == cudaSuccess && stamp[1] > 0)
      last_mhz = 1e3 * (double)stamp[0] / (double)stamp[1];
    return total / n;
  };
  // A time in SM cycles rather than seconds: on a power-limited part the clock of one candidate's run differs from
  // the next one's by more than the candidates do.  (Without a clock reading: the time itself.)
  auto cyc = [&](double ms) { return last_mhz > 0.0 ? ms * last_mhz : ms * 1500.0; };
  // The reference: the library's default configuration, never a previously tuned entry.
  fact_config_t ref_c;
  {
    auto saved = h->table;
    h->table.erase(make_key(q));
    const fact_status_t rs = resolve_config(h, q, nullptr, 0, &ref_c);
    h->table = saved;
    if (rs != FACT_OK || workspace_for(h, q, ref_c) > ws_bytes) {
      cleanup();
      return rs != FACT_OK ? rs : FACT_ERR_WORKSPACE_TOO_SMALL;
    }
  }
  // Verify gate.  The reference configuration's output is kept as a dense FP32 copy; a candidate's output must agree
  // with it element by element to within what two correct results can differ by: both are FP32 sums of the same
  // products in different orders (accumulation noise ~ sqrt(K) 2^-24 of the output scale), each rounded once to the
  // output type (one BF16 ulp = 2^-8 relative when they straddle a rounding boundary).
  TuneViewParams view;
  view.C = C;
  view.ldc = ldc;
  view.strideC = strideC;
  view.batch = (int)q.batch;
  view.M = (int)q.M;
  view.N = (int)q.N_out;
  view.f32 = out == FACT_OUT_F32;
  const int vgrid = (int)std::min<long long>((out_elems + 255) / 256, (long long)h->sm_count * 8);
  float floor_abs = 0.f;
  const float rel_tol = view.f32 ? 1e-3f : 0.0078125f;  // 2^-7 for BF16 outputs; half the stated FP32 tolerance
  unsigned int* d_result = verify ? reinterpret_cast<unsigned int*>(d_sum + 1) : nullptr;
  if (verify) {
    bool ok = cudaMemsetAsync(d_sum, 0, 2 * sizeof(double), stream) == cudaSuccess;
    fact_tune_poison_kernel<<<vgrid, 256, 0, stream>>>(view);
    ok = ok && run(h, q, &ref_c, 0, ws, ws_bytes, stream_v) == FACT_OK;
    fact_tune_snapshot_kernel<<<vgrid, 256, 0, stream>>>(view, d_ref, d_sum);
    double abs_sum = 0.0;
    int dev_status = 0;
    ok = ok && cudaGetLastError() == cudaSuccess && fact_device_status(h, stream_v, &dev_status) == FACT_OK &&
         dev_status == 0 && cudaMemcpy(&abs_sum, d_sum, sizeof(double), cudaMemcpyDeviceToHost) == cudaSuccess;
    if (!ok || !(abs_sum == abs_sum)) {  // the reference itself failed to run, or produced NaNs
      cudaGetLastError();
      cleanup();
      return FACT_ERR_CUDA;
    }
    const double mean_abs = abs_sum / (double)out_elems;
    floor_abs = (float)(1e-3 * mean_abs + 1e-30);
  }
  // worst |candidate - reference| / tolerance over the whole output; negative if the check itself failed
  auto verify_cfg = [&](const fact_config_t& c, bool perturb) -> double {
    fact_tune_poison_kernel<<<vgrid, 256, 0, stream>>>(view);
    if (run(h, q, &c, 0, ws, ws_bytes, stream_v) != FACT_OK) return -1.0;
    if (cudaMemsetAsync(d_result, 0, 2 * sizeof(unsigned int), stream) != cudaSuccess) return -1.0;
    fact_tune_compare_kernel<<<vgrid, 256, 0, stream>>>(view, d_ref, rel_tol, floor_abs, perturb ? 1 : 0, d_result);
    unsigned int res[2] = {0u, 0u};
    int dev_status = 0;
    if (cudaGetLastError() != cudaSuccess || fact_device_status(h, stream_v, &dev_status) != FACT_OK ||
        dev_status != 0 || cudaMemcpy(res, d_result, sizeof res, cudaMemcpyDeviceToHost) != cudaSuccess)
      return -1.0;
    float worst;
    memcpy(&worst, &res[1], sizeof worst);
    return res[0] != 0 ? std::max(1.0000001, (double)worst) : (double)worst;
  };

  // Sweep: every feasible candidate once.  A sweep lasts seconds on a power-limited part whose clock drifts, so
  // a candidate is ranked by its time RELATIVE to the reference configuration timed right before and after.
  const int ref_iters = std::max(3, iters / 4);
  struct Timed {
    double rel;
    fact_config_t cfg;
    int rec;
  };
  std::vector<Timed> timed;
  double t_ref = time_cfg(ref_c, warmup, ref_iters);
  double c_ref = cyc(t_ref);
  int cand_index = 0;
  for (const fact_config_t& c : cands) {
    const int my_index = cand_index++;
    Plan plan;
    if (make_plan(h, q, &c, 0, &plan) != FACT_OK) {  // over a budget, or a combination the kernels cannot run
      record(c, FACT_TUNE_INFEASIBLE, -1.0, -1.0, -1.0);
      continue;
    }
    if (plan.ws_bytes > ws_bytes) {
      record(plan.cfg, FACT_TUNE_NO_WORKSPACE, -1.0, -1.0, -1.0);
      continue;
    }
    double verr = 0.0;
    if (verify) {
      verr = verify_cfg(c, my_index == inject);
      if (verr < 0.0) {
        record(plan.cfg, FACT_TUNE_LAUNCH_FAILED, -1.0, -1.0, -1.0);
        continue;
      }
      if (verr > 1.0) {  // wrong numbers: recorded, never timed, never eligible
        record(plan.cfg, FACT_TUNE_VERIFY_FAILED, -1.0, -1.0, verr);
        continue;
      }
    }
    const double t = time_cfg(c, warmup, iters);
    const double c_cand = cyc(t);
    const double t_ref_after = time_cfg(ref_c, 1, ref_iters);
    const double c_ref_after = cyc(t_ref_after);
    if (t >= 0 && t_ref > 0 && t_ref_after > 0) {
      const double rel = 2.0 * c_cand / (c_ref + c_ref_after);
      timed.push_back({rel, plan.cfg, record(plan.cfg, FACT_TUNE_TIMED, t, rel, verr)});
    } else {
      record(plan.cfg, FACT_TUNE_LAUNCH_FAILED, -1.0, -1.0, verr);
    }
    if (t_ref_after > 0) {
      t_ref = t_ref_after;
      c_ref = c_ref_after;
    }
  }
  const int tried = (int)timed.size();
  std::sort(timed.begin(), timed.end(), [](const Timed& x, const Timed& y) { return x.rel < y.rel; });
  // Play-off: the few fastest candidates are timed again, five rounds in alternation, and ranked by the median of
  // their cycle-normalised times; the time reported is the winner's best round.
  double best_t = 1e30, best_score = 1e300;
  fact_config_t best_c;
  memset(&best_c, 0, sizeof best_c);
  const int finalists = std::min(tried, 5);
  const int rounds = 5;
  std::vector<std::vector<double>> scores((size_t)finalists);
  std::vector<double> best_round((size_t)finalists, 1e30);
  for (int round = 0; round < rounds; ++round)
    for (int i = 0; i < finalists; ++i) {
      const double t = time_cfg(timed[(size_t)i].cfg, 2, iters);
      if (t >= 0) {
        best_round[(size_t)i] = std::min(best_round[(size_t)i], t);
        scores[(size_t)i].push_back(cyc(t));
      }
    }
  for (int i = 0; i < finalists; ++i) {
    std::vector<double>& v = scores[(size_t)i];
    if (v.empty()) continue;
    std::sort(v.begin(), v.end());
    const double med = v[v.size() / 2];
    if (med < best_score) {
      best_score = med;
      best_t = best_round[(size_t)i];
      best_c = timed[(size_t)i].cfg;
    }
  }
  // the caller's output ends as the winner's (or, with nothing timed, the reference's) result
  if (tried > 0) run(h, q, &best_c, 0, ws, ws_bytes, stream_v);
  cudaStreamSynchronize(stream);
  cleanup();
  if (opts && opts->n_records) *opts->n_records = n_recs;
  if (n_tried) *n_tried = tried;
  if (tried == 0) return FACT_ERR_UNSUPPORTED;
  h->table[make_key(q)] = best_c;
  *best = best_c;
  if (best_ms) *best_ms = best_t;
  return FACT_OK;
}

fact_status_t fact_tune(fact_handle_t h, fact_op_t op, int64_t batch, int64_t M, int64_t N, int64_t K, const void* A,
                        int64_t lda, int64_t strideA, const void* B, int64_t ldb, int64_t strideB,
                        fact_blayout_t layout, const void* bias, const void* residual, int64_t ldr, int64_t strideR,
                        void* C, int64_t ldc, int64_t strideC, fact_out_t out, fact_epilogue_t epi, void* ws,
                        size_t ws_bytes, int warmup, int iters, void* stream_v, fact_config_t* best, double* best_ms,
                        int* n_tried) {
  return fact_tune_ex(h, op, batch, M, N, K, A, lda, strideA, B, ldb, strideB, layout, bias, residual, ldr, strideR, C,
                      ldc, strideC, out, epi, ws, ws_bytes, warmup, iters, stream_v, nullptr, best, best_ms, n_tried);
}

fact_status_t fact_tune_cache_save(fact_handle_t h, const char* path) {
  if (!h || !path) return FACT_ERR_INVALID_ARG;
  FILE* f = fopen(path, "w");
  if (!f) return FACT_ERR_INVALID_ARG;
  fprintf(f, "# libfact tuner table v2: op epilogue layout out batch M N K | tile_m tile_n tile_k stages cta_group raster_group split_k store_mode schedule\n");
  for (const auto& kv : h->table) {
    const TuneKey& k = kv.first;
    const fact_config_t& c = kv.second;
    fprintf(f, "%d %d %d %d %lld %lld %lld %lld | %d %d %d %d %d %d %d %d %d\n", std::get<0>(k), std::get<1>(k),
            std::get<2>(k), std::get<3>(k), std::get<4>(k), std::get<5>(k), std::get<6>(k), std::get<7>(k), c.tile_m,
            c.tile_n, c.tile_k, c.stages, c.cta_group, c.raster_group, c.split_k, c.store_mode, c.schedule);
  }
  fclose(f);
  return FACT_OK;
}

fact_status_t fact_tune_cache_load(fact_handle_t h, const char* path) {
  if (!h || !path) return FACT_ERR_INVALID_ARG;
  FILE* f = fopen(path, "r");
  if (!f) return FACT_ERR_INVALID_ARG;
  char line[512];
  while (fgets(line, sizeof line, f)) {
    if (line[0] == '#' || line[0] == '\n') continue;
    int op, epi, lay, out;
    long long b, M, N, K;
    fact_config_t c;
    memset(&c, 0, sizeof c);
    // (the ninth configuration field is absent from tables written before the schedule field existed)
    if (sscanf(line, "%d %d %d %d %lld %lld %lld %lld | %d %d %d %d %d %d %d %d %d", &op, &epi, &lay, &out, &b, &M, &N,
               &K, &c.tile_m, &c.tile_n, &c.tile_k, &c.stages, &c.cta_group, &c.raster_group, &c.split_k,
               &c.store_mode, &c.schedule) < 16)
      continue;
    h->table[TuneKey(op, epi, lay, out, b, M, N, K)] = c;
  }
  fclose(f);
  return FACT_OK;
}

// ---------------------------------------------------------------------------------------------
// Fused multi-head attention
namespace {
// Rank-4 BF16 tensor map over [B][T][H][D]-like storage, dims ordered (D, H, T, B), box 64 x 1 x box_rows x 1.
fact_status_t encode_map_bthd(fact_handle_t h, CUtensorMap* map, const void* base, long long D, long long H, long long T,
                              long long B, long long stride_h, long long stride_t, long long stride_b,
                              int box_rows = kAttnBlockQ) {
  cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)H, (cuuint64_t)T, (cuuint64_t)B};
  cuuint64_t strides[3] = {(cuuint64_t)stride_h * 2, (cuuint64_t)stride_t * 2, (cuuint64_t)stride_b * 2};
  cuuint32_t box[4] = {64, 1, (cuuint32_t)box_rows, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = h->encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    h->last_error = "cuTensorMapEncodeTiled (attention operand) failed with CUresult " + std::to_string((int)r);
    return FACT_ERR_CUDA;
  }
  return FACT_OK;
}
}  // namespace

fact_status_t fact_attention(fact_handle_t h, int64_t batch, int64_t seq_q, int64_t seq_kv, int64_t heads_q,
                             int64_t heads_kv, int64_t head_dim, const void* Q, int64_t q_sb, int64_t q_st,
                             int64_t q_sh, const void* K, int64_t k_sb, int64_t k_st, int64_t k_sh, const void* V,
                             int64_t v_sb, int64_t v_st, int64_t v_sh, void* O, int64_t o_sb, int64_t o_st,
                             int64_t o_sh, int causal, float scale, void* stream_v) {
  if (!h) return FACT_ERR_INVALID_ARG;
  if (batch < 0 || seq_q < 0 || seq_kv < 0 || heads_q <= 0 || heads_kv <= 0 || heads_q % heads_kv) return FACT_ERR_INVALID_ARG;
  if (head_dim != 64 && head_dim != 128) return FACT_ERR_UNSUPPORTED;
  if (batch == 0 || seq_q == 0) return FACT_OK;
  if (seq_kv == 0 || !Q || !K || !V || !O) return FACT_ERR_INVALID_ARG;
  if (causal && seq_q != seq_kv) return FACT_ERR_UNSUPPORTED;
  if (seq_q > 0x7fffff00LL || seq_kv > 0x7fffff00LL || batch * heads_q > 0x7fffffLL) return FACT_ERR_INVALID_ARG;
  const int64_t strides[12] = {q_sb, q_st, q_sh, k_sb, k_st, k_sh, v_sb, v_st, v_sh, o_sb, o_st, o_sh};
  for (int i = 0; i < 12; ++i)
    if (strides[i] < 0) return FACT_ERR_INVALID_ARG;
  // head_dim must be contiguous; every other stride a multiple of 8 elements (16 bytes), pointers 16-byte aligned
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O)) return FACT_ERR_BAD_ALIGNMENT;
  for (int i = 0; i < 12; ++i) {
    const bool batch_stride = (i % 3) == 0;
    if (strides[i] % 8) return FACT_ERR_BAD_ALIGNMENT;
    if (!batch_stride && strides[i] < head_dim) return FACT_ERR_INVALID_ARG;
  }
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_v);
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return FACT_ERR_CUDA;
  if (dev != h->device && cudaSetDevice(h->device) != cudaSuccess) return FACT_ERR_CUDA;
  CUtensorMap tq, tk, tv, to;
  auto bs = [&](int64_t s, int64_t fallback) { return (batch > 1 && s > 0) ? s : std::max<int64_t>(fallback, 8); };
  // keys go in blocks of 128 at head_dim 64 and of 64 at head_dim 128 (the kernel's tensor-memory budget)
  const int block_k = attn_block_k((int)head_dim);
  fact_status_t st = encode_map_bthd(h, &tq, Q, head_dim, heads_q, seq_q, batch, q_sh, q_st, bs(q_sb, q_st * seq_q));
  if (st == FACT_OK)
    st = encode_map_bthd(h, &tk, K, head_dim, heads_kv, seq_kv, batch, k_sh, k_st, bs(k_sb, k_st * seq_kv), block_k);
  if (st == FACT_OK)
    st = encode_map_bthd(h, &tv, V, head_dim, heads_kv, seq_kv, batch, v_sh, v_st, bs(v_sb, v_st * seq_kv), block_k);
  if (st == FACT_OK) st = encode_map_bthd(h, &to, O, head_dim, heads_q, seq_q, batch, o_sh, o_st, bs(o_sb, o_st * seq_q));
  if (st == FACT_OK) {
    AttnParams p;
    memset(&p, 0, sizeof p);
    p.B = (int)batch;
    p.Tq = (int)seq_q;
    p.Tk = (int)seq_kv;
    p.Hq = (int)heads_q;
    p.Hkv = (int)heads_kv;
    p.D = (int)head_dim;
    p.causal = causal != 0;
    const double sc = scale > 0.f ? (double)scale : 1.0 / std::sqrt((double)head_dim);
    p.scale_log2 = (float)(sc * 1.4426950408889634);
    p.kmajor_desc = smem_desc_template(16, 1024);
    p.v_desc = smem_desc_template(block_k * 128, 1024);  // 64-column chunks of V are one block of keys apart
    p.idesc_s = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(block_k >> 3) << 17) | ((uint32_t)(kAttnBlockQ >> 4) << 24);
    p.idesc_pv = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(head_dim >> 3) << 17) |
                 ((uint32_t)(kAttnBlockQ >> 4) << 24);
    p.status = h->d_status;
    p.debug = h->debug_flags;
    p.q_pairs = (int)((seq_q + 2 * kAttnBlockQ - 1) / (2 * kAttnBlockQ));  // an item is two tiles of 128 query rows
    const long long items = (long long)p.q_pairs * heads_q * batch;
    if (items > 0x7fffffffLL) {
      if (dev != h->device) cudaSetDevice(dev);
      return FACT_ERR_UNSUPPORTED;
    }
    p.items = (int)items;
    const long long ctas = std::min<long long>(p.items, h->sm_count);  // persistent: one CTA per SM
    const int smem = std::max((int)attn_smem_bytes(p.D), kMinSmemRequest);
    if (!h->configured_mask.test(30)) {
      cudaError_t e = cudaFuncSetAttribute(fact_attention_kernel<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget);
      if (e == cudaSuccess)
        e = cudaFuncSetAttribute(fact_attention_kernel<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget);
      if (e == cudaSuccess)
        e = cudaFuncSetAttribute(fact_attention_kernel<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget);
      if (e == cudaSuccess)
        e = cudaFuncSetAttribute(fact_attention_kernel<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget);
      cudaFuncAttributes fa, fb;
      if (e == cudaSuccess) e = cudaFuncGetAttributes(&fa, fact_attention_kernel<64, false>);
      if (e == cudaSuccess) e = cudaFuncGetAttributes(&fb, fact_attention_kernel<128, false>);
      if (e == cudaSuccess) fa.numRegs = std::min(fa.numRegs, fb.numRegs);
      if (e == cudaSuccess) e = cudaFuncGetAttributes(&fb, fact_attention_kernel<64, true>);
      if (e == cudaSuccess) fa.numRegs = std::min(fa.numRegs, fb.numRegs);
      if (e == cudaSuccess) e = cudaFuncGetAttributes(&fb, fact_attention_kernel<128, true>);
      if (e == cudaSuccess) fa.numRegs = std::min(fa.numRegs, fb.numRegs);
      if (e != cudaSuccess) {
        st = cuda_fail(h, "cudaFuncSetAttribute(attention)", e);
      } else if (fa.numRegs < kAttnRegsAtLaunch) {
        // the kernel's register rebalancing would wait forever for registers the CTA does not own
        h->last_error = "attention kernel compiled with " + std::to_string(fa.numRegs) + " registers per thread, needs " +
                        std::to_string(kAttnRegsAtLaunch);
        st = FACT_ERR_UNSUPPORTED;
      } else {
        h->configured_mask.set(30);
      }
    }
    if (st == FACT_OK) {
      // Causal problems of few rounds: the closed-form deal (round by round, every second round reversed) leaves some
      // CTAs up to 10 % more key blocks than the mean (16 x 12 heads x 1024 tokens: 28 block-times against 25.9), so
      // the host deals the items out itself -- heaviest first, each to the CTA with the least so far -- and hands the
      // list to the kernel as a parameter.  The list is kept for the next call of the same shape.
      const int bk = head_dim == 64 ? 128 : 64;
      const bool deal = causal != 0 && p.items > ctas && p.items <= kAttnDealItems && ctas <= kAttnDealCtas &&
                        p.items < 16 * ctas;
      if (deal) {
        const std::array<long long, 6> key = {(long long)batch * heads_q, (long long)p.q_pairs, (long long)bk, (long long)seq_kv, (long long)ctas, (long long)seq_q};
        if (!h->attn_deal || h->attn_deal_key != key) {
          if (!h->attn_deal) h->attn_deal.reset(new AttnDeal());
          build_attention_deal((int)ctas, batch * heads_q, p.q_pairs, bk, seq_kv, *h->attn_deal);
          h->attn_deal_key = key;
        }
      }
      const AttnNoDeal none = {0};
      cudaError_t e;
      if (deal)
        e = head_dim == 64 ? launch_pdl(h, fact_attention_kernel<64, true>, (unsigned)ctas, (unsigned)kAttnThreads,
                                        (size_t)smem, stream, 1, tq, tk, tv, to, p, *h->attn_deal)
                           : launch_pdl(h, fact_attention_kernel<128, true>, (unsigned)ctas, (unsigned)kAttnThreads,
                                        (size_t)smem, stream, 1, tq, tk, tv, to, p, *h->attn_deal);
      else
        e = head_dim == 64 ? launch_pdl(h, fact_attention_kernel<64, false>, (unsigned)ctas, (unsigned)kAttnThreads,
                                        (size_t)smem, stream, 1, tq, tk, tv, to, p, none)
                           : launch_pdl(h, fact_attention_kernel<128, false>, (unsigned)ctas, (unsigned)kAttnThreads,
                                        (size_t)smem, stream, 1, tq, tk, tv, to, p, none);
      if (e != cudaSuccess) st = cuda_fail(h, "attention launch", e);
      else h->launches++;
    }
  }
  if (dev != h->device) cudaSetDevice(dev);
  return st;
}

// ---------------------------------------------------------------------------------------------
// Row normalisation and the whole-block chain
fact_status_t fact_norm(fact_handle_t h, fact_norm_t kind, int64_t M, int64_t C, const void* X, int64_t ldx,
                        const void* gamma, const void* beta, float eps, void* Y, int64_t ldy, void* stream_v) {
  if (!h || M < 0 || (kind != FACT_NORM_LAYER && kind != FACT_NORM_RMS)) return FACT_ERR_INVALID_ARG;
  if (C < 8 || C > 8192 || C % 8) return FACT_ERR_UNSUPPORTED;
  if (M == 0) return FACT_OK;
  if (!X || !Y || !gamma || (kind == FACT_NORM_RMS && beta) || !(eps >= 0.f)) return FACT_ERR_INVALID_ARG;
  if (ldx < C || ldy < C || M > 0x7fffffffLL * kNormWarps) return FACT_ERR_INVALID_ARG;
  if (!aligned16(X) || !aligned16(Y) || !aligned16(gamma) || (beta && !aligned16(beta)) || ldx % 8 || ldy % 8)
    return FACT_ERR_BAD_ALIGNMENT;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_v);
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return FACT_ERR_CUDA;
  if (dev != h->device && cudaSetDevice(h->device) != cudaSuccess) return FACT_ERR_CUDA;
  NormParams p;
  p.X = reinterpret_cast<const __nv_bfloat16*>(X);
  p.Y = reinterpret_cast<__nv_bfloat16*>(Y);
  p.gamma = reinterpret_cast<const __nv_bfloat16*>(gamma);
  p.beta = reinterpret_cast<const __nv_bfloat16*>(beta);
  p.M = M;
  p.C = (int)C;
  p.ldx = ldx;
  p.ldy = ldy;
  p.eps = eps;
  const unsigned grid = (unsigned)((M + kNormWarps - 1) / kNormWarps);
  const int threads = kNormWarps * 32;
  const bool rms = kind == FACT_NORM_RMS;
  // a lane keeps ceil(C / 256) 16-byte chunks of its row in registers
  cudaError_t e;
  if (C <= 1024) {
    e = rms ? launch_pdl(h, fact_norm_kernel<4, true>, grid, (unsigned)threads, 0, stream, 1, p)
            : launch_pdl(h, fact_norm_kernel<4, false>, grid, (unsigned)threads, 0, stream, 1, p);
  } else if (C <= 4096) {
    e = rms ? launch_pdl(h, fact_norm_kernel<16, true>, grid, (unsigned)threads, 0, stream, 1, p)
            : launch_pdl(h, fact_norm_kernel<16, false>, grid, (unsigned)threads, 0, stream, 1, p);
  } else {
    e = rms ? launch_pdl(h, fact_norm_kernel<32, true>, grid, (unsigned)threads, 0, stream, 1, p)
            : launch_pdl(h, fact_norm_kernel<32, false>, grid, (unsigned)threads, 0, stream, 1, p);
  }
  fact_status_t st = FACT_OK;
  if (e != cudaSuccess) st = cuda_fail(h, "norm launch", e);
  else h->launches++;
  if (dev != h->device) cudaSetDevice(dev);
  return st;
}

fact_status_t fact_row_stats(fact_handle_t h, int64_t M, int64_t C, const void* X, int64_t ldx, float* stats,
                             void* stream_v) {
  if (!h || M < 0) return FACT_ERR_INVALID_ARG;
  if (C < 8 || C % 8) return FACT_ERR_UNSUPPORTED;
  if (M == 0) return FACT_OK;
  if (!X || !stats || ldx < C || M > 0x7fffffffLL) return FACT_ERR_INVALID_ARG;
  if (!aligned16(X) || ldx % 8 || ((uintptr_t)stats & 7u)) return FACT_ERR_BAD_ALIGNMENT;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return FACT_ERR_CUDA;
  if (dev != h->device && cudaSetDevice(h->device) != cudaSuccess) return FACT_ERR_CUDA;
  const unsigned grid = (unsigned)((M + kNormWarps - 1) / kNormWarps);
  fact_row_stats_kernel<<<grid, kNormWarps * 32, 0, reinterpret_cast<cudaStream_t>(stream_v)>>>(
      reinterpret_cast<const __nv_bfloat16*>(X), (long long)M, (int)C, (long long)ldx, reinterpret_cast<float2*>(stats));
  fact_status_t st = FACT_OK;
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) st = cuda_fail(h, "row stats launch", e);
  else h->launches++;
  if (dev != h->device) cudaSetDevice(dev);
  return st;
}

fact_status_t fact_fold_norm(fact_handle_t h, int64_t N_w, int64_t K, const void* W, int64_t ldw, const void* gamma,
                             const void* beta, const void* bias, void* W_folded, int64_t ldwf, float* colsum,
                             void* bias_folded, void* stream_v) {
  if (!h || N_w < 0 || K < 0) return FACT_ERR_INVALID_ARG;
  if (K % 8) return FACT_ERR_UNSUPPORTED;
  if (N_w == 0) return FACT_OK;
  if (!W || !gamma || !W_folded || ldw < K || ldwf < K || N_w > 0x7fffffffLL || K > 0x7fffffffLL)
    return FACT_ERR_INVALID_ARG;
  if ((beta != nullptr) != (bias_folded != nullptr)) return FACT_ERR_INVALID_ARG;  // the shift moves into the bias
  if (!beta && bias) return FACT_ERR_INVALID_ARG;                                   // (without a shift the bias stays as it is)
  if (!aligned16(W) || !aligned16(W_folded) || !aligned16(gamma) || (beta && !aligned16(beta)) || ldw % 8 || ldwf % 8)
    return FACT_ERR_BAD_ALIGNMENT;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return FACT_ERR_CUDA;
  if (dev != h->device && cudaSetDevice(h->device) != cudaSuccess) return FACT_ERR_CUDA;
  FoldParams p;
  p.W = reinterpret_cast<const __nv_bfloat16*>(W);
  p.Wf = reinterpret_cast<__nv_bfloat16*>(W_folded);
  p.gamma = reinterpret_cast<const __nv_bfloat16*>(gamma);
  p.beta = reinterpret_cast<const __nv_bfloat16*>(beta);
  p.bias = reinterpret_cast<const __nv_bfloat16*>(bias);
  p.bias_out = reinterpret_cast<__nv_bfloat16*>(bias_folded);
  p.colsum = colsum;
  p.N = (int)N_w;
  p.K = (int)K;
  p.ldw = ldw;
  p.ldwf = ldwf;
  const unsigned grid = (unsigned)((N_w + kNormWarps - 1) / kNormWarps);
  fact_fold_norm_kernel<<<grid, kNormWarps * 32, 0, reinterpret_cast<cudaStream_t>(stream_v)>>>(p);
  fact_status_t st = FACT_OK;
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) st = cuda_fail(h, "fold launch", e);
  else h->launches++;
  if (dev != h->device) cudaSetDevice(dev);
  return st;
}

namespace {
// Workspace carve-up of one block (element counts; every buffer starts on a 256-byte boundary).
struct BlockLayout {
  int64_t tokens, qkv_cols, h_cols;
  size_t off_n, off_qkv, off_a, off_x1, off_h, total;
};
bool block_layout(const fact_block_t* b, BlockLayout* L) {
  if (!b || (b->kind != FACT_BLOCK_GPT && b->kind != FACT_BLOCK_LLAMA)) return false;
  if (b->batch < 0 || b->seq < 0 || b->hidden <= 0 || b->heads_q <= 0 || b->heads_kv <= 0 || b->ffn <= 0) return false;
  if (b->heads_q % b->heads_kv || b->hidden != b->heads_q * b->head_dim || b->hidden % 8 || b->ffn % 8) return false;
  if (b->batch > 0 && b->seq > 0x7fffffffLL / std::max<int64_t>(b->batch, 1)) return false;
  L->tokens = b->batch * b->seq;
  L->qkv_cols = (b->heads_q + 2 * b->heads_kv) * b->head_dim;
  L->h_cols = b->ffn;
  auto up = [](size_t v) { return (v + 255) & ~(size_t)255; };
  const size_t t = (size_t)L->tokens;
  L->off_n = 0;
  L->off_qkv = up(L->off_n + t * (size_t)b->hidden * 2);
  L->off_a = up(L->off_qkv + t * (size_t)L->qkv_cols * 2);
  L->off_x1 = up(L->off_a + t * (size_t)b->hidden * 2);
  L->off_h = up(L->off_x1 + t * (size_t)b->hidden * 2);
  L->total = up(L->off_h + t * (size_t)L->h_cols * 2);
  return true;
}
}  // namespace

size_t fact_block_workspace_bytes(const fact_block_t* b) {
  BlockLayout L;
  return block_layout(b, &L) ? L.total : 0;
}

fact_status_t fact_block_workspace_offsets(const fact_block_t* b, size_t offsets[5]) {
  BlockLayout L;
  if (!offsets || !block_layout(b, &L)) return FACT_ERR_INVALID_ARG;
  offsets[0] = L.off_n;
  offsets[1] = L.off_qkv;
  offsets[2] = L.off_a;
  offsets[3] = L.off_x1;
  offsets[4] = L.off_h;
  return FACT_OK;
}

fact_status_t fact_block_forward(fact_handle_t h, const fact_block_t* b, const void* x, void* y, void* ws,
                                 size_t ws_bytes, void* stream) {
  BlockLayout L;
  if (!h || !block_layout(b, &L)) return FACT_ERR_INVALID_ARG;
  if (b->head_dim != 64 && b->head_dim != 128) return FACT_ERR_UNSUPPORTED;
  if (L.tokens == 0) return FACT_OK;
  const bool llama = b->kind == FACT_BLOCK_LLAMA;
  if (!x || !y || !b->norm1_gamma || !b->norm2_gamma || !b->wqkv || !b->wo || !b->w1 || !b->w2) return FACT_ERR_INVALID_ARG;
  if (llama && (b->norm1_beta || b->norm2_beta || b->bqkv || b->bo || b->b1 || b->b2)) return FACT_ERR_INVALID_ARG;
  if (!llama && !b->b1) return FACT_ERR_INVALID_ARG;  // the GELU epilogue carries the bias
  if (!ws || ws_bytes < L.total) return FACT_ERR_WORKSPACE_TOO_SMALL;
  if (!aligned16(ws)) return FACT_ERR_BAD_ALIGNMENT;
  uint8_t* w8 = reinterpret_cast<uint8_t*>(ws);
  void* n = w8 + L.off_n;
  __nv_bfloat16* qkv = reinterpret_cast<__nv_bfloat16*>(w8 + L.off_qkv);
  void* a = w8 + L.off_a;
  void* x1 = w8 + L.off_x1;
  void* hbuf = w8 + L.off_h;
  const int64_t T = L.tokens, C = b->hidden, D = b->head_dim, QC = L.qkv_cols;
  const fact_norm_t nk = llama ? FACT_NORM_RMS : FACT_NORM_LAYER;
  fact_status_t st = fact_norm(h, nk, T, C, x, C, b->norm1_gamma, b->norm1_beta, b->eps, n, C, stream);
  if (st != FACT_OK) return st;
  st = fact_linear(h, T, QC, C, n, C, b->wqkv, C, FACT_B_NK, b->bqkv, nullptr, 0, qkv, QC, FACT_OUT_BF16,
                   b->bqkv ? FACT_EPI_BIAS : FACT_EPI_NONE, nullptr, nullptr, 0, stream);
  if (st != FACT_OK) return st;
  // Q, K, V are column ranges of qkv: token stride QC, head stride D, batch stride seq * QC
  const __nv_bfloat16* qp = qkv;
  const __nv_bfloat16* kp = qkv + b->heads_q * D;
  const __nv_bfloat16* vp = kp + b->heads_kv * D;
  st = fact_attention(h, b->batch, b->seq, b->seq, b->heads_q, b->heads_kv, D, qp, b->seq * QC, QC, D, kp, b->seq * QC,
                      QC, D, vp, b->seq * QC, QC, D, a, b->seq * C, C, D, 1, 0.f, stream);
  if (st != FACT_OK) return st;
  st = fact_linear(h, T, C, C, a, C, b->wo, C, FACT_B_NK, b->bo, x, C, x1, C, FACT_OUT_BF16, FACT_EPI_BIAS_RESIDUAL,
                   nullptr, nullptr, 0, stream);
  if (st != FACT_OK) return st;
  st = fact_norm(h, nk, T, C, x1, C, b->norm2_gamma, b->norm2_beta, b->eps, n, C, stream);
  if (st != FACT_OK) return st;
  st = fact_linear(h, T, b->ffn, C, n, C, b->w1, C, FACT_B_NK, b->b1, nullptr, 0, hbuf, b->ffn, FACT_OUT_BF16,
                   llama ? FACT_EPI_SILU_GATE : FACT_EPI_BIAS_GELU_TANH, nullptr, nullptr, 0, stream);
  if (st != FACT_OK) return st;
  return fact_linear(h, T, C, b->ffn, hbuf, b->ffn, b->w2, b->ffn, FACT_B_NK, b->b2, x1, C, y, C, FACT_OUT_BF16,
                     FACT_EPI_BIAS_RESIDUAL, nullptr, nullptr, 0, stream);
}

// ---------------------------------------------------------------------------------------------
// Allocation-free split-K GEMM.  One host-side state per device, filled on the first call for that device.
namespace {
constexpr int kMaxStaticDevices = 64;
struct StaticDeviceState {
  bool ready = false;
  void* scratch = nullptr;  // device address of g_static_scratch on this device
  fact_handle_s handle;     // host-side bookkeeping only; its status word is g_static_status on this device
};
StaticDeviceState g_static_state[kMaxStaticDevices];

// Resolve, with `device` current, the device addresses of the static arrays and the few device facts the
// planner needs.  Nothing here allocates device memory.
fact_status_t static_setup(int device, StaticDeviceState* st) {
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return FACT_ERR_CUDA;
  if (prop.major != 10) return FACT_ERR_ARCH;
  void* scratch = nullptr;
  void* status = nullptr;
  if (cudaGetSymbolAddress(&scratch, g_static_scratch) != cudaSuccess || !scratch) {
    cudaGetLastError();
    return FACT_ERR_CUDA;
  }
  if (cudaGetSymbolAddress(&status, g_static_status) != cudaSuccess || !status) {
    cudaGetLastError();
    return FACT_ERR_CUDA;
  }
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
      qres != cudaDriverEntryPointSuccess) {
    cudaGetLastError();
    return FACT_ERR_CUDA;
  }
  fact_handle_s& h = st->handle;
  h.device = device;
  h.sm_count = prop.multiProcessorCount;
  h.max_smem = (int)prop.sharedMemPerBlockOptin;
  h.cc_major = prop.major;
  h.cc_minor = prop.minor;
  h.encode = reinterpret_cast<EncodeTiledFn>(fn);
  h.d_status = reinterpret_cast<int*>(status);
  st->scratch = scratch;
  st->ready = true;
  return FACT_OK;
}
}  // namespace

fact_status_t fact_gemm_splitk_static(int device, int64_t M, int64_t N, int64_t K, const void* A, int64_t lda,
                                      const void* B, int64_t ldb, fact_blayout_t layout, void* C, int64_t ldc,
                                      fact_out_t out, int splits, void* stream) {
  if (device < 0 || device >= kMaxStaticDevices || splits < 0) return FACT_ERR_INVALID_ARG;
  int n_dev = 0;
  if (cudaGetDeviceCount(&n_dev) != cudaSuccess || device >= n_dev) {
    cudaGetLastError();
    return FACT_ERR_CUDA;
  }
  int prev = -1;
  if (cudaGetDevice(&prev) != cudaSuccess) return FACT_ERR_CUDA;
  if (prev != device && cudaSetDevice(device) != cudaSuccess) return FACT_ERR_CUDA;
  StaticDeviceState* st = &g_static_state[device];
  fact_status_t rc = FACT_OK;
  if (!st->ready) rc = static_setup(device, st);  // first call on this device, with this device current
  if (rc == FACT_OK) {
    Problem q = make_problem(FACT_OP_GEMM_SPLITK, 1, M, N, K, A, lda, 0, B, ldb, 0, layout, nullptr, nullptr, 0, 0, C,
                             ldc, 0, out, FACT_EPI_NONE);
    rc = validate(q);
    if (rc == FACT_OK && M > 0 && N > 0) {
      Plan plan;
      rc = make_plan(&st->handle, q, nullptr, splits, &plan);
      // the partial planes of this problem must fit the fixed scratch: refuse, never spill elsewhere
      if (rc == FACT_OK && plan.ws_bytes > kStaticScratchBytes) rc = FACT_ERR_WORKSPACE_TOO_SMALL;
      if (rc == FACT_OK) rc = run(&st->handle, q, nullptr, splits, st->scratch, kStaticScratchBytes, stream);
    }
  }
  if (prev != device) cudaSetDevice(prev);
  return rc;
}

fact_status_t fact_gemm_splitk_static_status(int device, void* stream, int* status) {
  if (device < 0 || device >= kMaxStaticDevices || !status) return FACT_ERR_INVALID_ARG;
  StaticDeviceState* st = &g_static_state[device];
  *status = 0;
  if (!st->ready) return FACT_OK;  // no call has run on this device yet
  int prev = -1;
  if (cudaGetDevice(&prev) != cudaSuccess) return FACT_ERR_CUDA;
  if (prev != device && cudaSetDevice(device) != cudaSuccess) return FACT_ERR_CUDA;
  // read (and, after a give-up, clear) the static status word and the grid-barrier counters: a stream
  // synchronisation, one 4-byte copy and memsets -- nothing allocates
  fact_status_t rc = FACT_OK;
  int v = 0;
  int* word = st->handle.d_status;
  if (cudaStreamSynchronize(reinterpret_cast<cudaStream_t>(stream)) != cudaSuccess ||
      cudaMemcpy(&v, word, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess ||
      (v != 0 && (cudaMemset(word, 0, sizeof(int)) != cudaSuccess ||
                  cudaMemset(word + 24, 0, 2 * sizeof(int)) != cudaSuccess))) {
    cudaGetLastError();
    rc = FACT_ERR_CUDA;
  }
  *status = v;
  if (prev != device) cudaSetDevice(prev);
  return rc;
}

int fact_debug_flags(fact_handle_t h) { return h ? h->debug_flags : 0; }

}  // extern "C"
