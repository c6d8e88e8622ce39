// The persistent, warp-specialised BF16 GEMM kernel for sm_100a and the
// split-K reduction kernel.
//
// One CTA (or a 2-CTA cluster when CG == 2) walks a static list of work units
// (batch, m-tile, n-tile, k-slice).  Roles run concurrently:
//   warps 0, 6 TMA producers (A tiles / B tiles): fill a ring of shared-memory stages with
//              128B-swizzled A (128 x 64) and B (tile_n x 64) tiles, signalling `full` mbarriers
//   warp 1     MMA issuer: issues tcgen05.mma (UMMA K = 16, four per stage) into one of two
//              FP32 accumulators in tensor memory, releasing stages through
//              tcgen05.commit -> `empty`, and publishing a finished accumulator through
//              tcgen05.commit -> `acc_full`
//   warps 2-5  epilogue: tcgen05.ld the accumulator (one output row per thread), apply the
//              fused element-wise operation in FP32, round once, and store -- either through
//              128-byte-swizzled shared-memory staging and TMA tensor stores (residual tiles
//              arrive the same way, by TMA loads), or directly from registers when the output
//              is not 16-byte aligned; then hand the accumulator back (`acc_empty`) so the
//              next tile's main loop overlaps
// Every mbarrier wait is bounded in time; an expired wait records
// FACT_ERR_DEVICE_TIMEOUT in the status word, all roles leave their loops, tensor
// memory is released and the kernel returns.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "ptx.cuh"

// Work-skipping experiment switches (loads, products or stores left out to isolate one ceiling; the results are
// garbage) exist only in a -DFACT_EXPERIMENTS build.  In the ordinary build the tests are the constant 0 and the
// compiler drops the code behind them.
#ifdef FACT_EXPERIMENTS
#define FACT_SKIP(p, bit) (((p).debug & (bit)) != 0)
#else
#define FACT_SKIP(p, bit) false
#endif

namespace fact {

constexpr int kMaxStages = 8;
constexpr int kTileM = 128;       // rows per CTA (= TMEM lanes)
constexpr int kTileK = 64;        // BF16 elements per 128-byte swizzle row
constexpr int kUmmaK = 16;        // K of one tcgen05.mma.kind::f16
constexpr int kThreads = 352;     // 11 warps: A producer, MMA, 4 x epilogue, B producer, 4 x epilogue
constexpr int kProducerBWarp = 6;
constexpr int kEpiSetBWarp0 = 7;  // warps 7..10 share the TMEM lane quarters of warps 2..5 (quarter = warp % 4)
constexpr uint32_t kStageBytesA = kTileM * kTileK * 2;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;  // 2 s per wait

// Epilogue staging in shared memory, per epilogue warp: one or two 32-row x 128-byte buffers
// (residual tile in, result tile out) and the BF16 bias values of the 128 columns the warp owns.
constexpr int kEpiWarps = 8;
constexpr int kEpiMaxBufs = 2;
constexpr uint32_t kEpiBufBytes = 32 * 128;
constexpr uint32_t kEpiBiasBytes = 128 * 2;
constexpr uint32_t epi_smem_bytes(int bufs) { return kEpiWarps * ((uint32_t)bufs * kEpiBufBytes + kEpiBiasBytes); }
// Shared-memory layout (dynamic, 1024-byte aligned): [stage ring][epilogue staging][bias][mbarriers, flags]
constexpr int kNumBarriers = 2 * kMaxStages + 4 + kEpiWarps * kEpiMaxBufs;
constexpr uint32_t kCtrlSmemBytes = kNumBarriers * 8 + 16;
// folded LayerNorm only: the FP32 column sums of each epilogue warp's 128 columns, behind the control words
constexpr uint32_t kNormCsBytes = kEpiWarps * 128 * 4;
// Dynamic tile scheduling (the DYN instantiations only), behind the control words of the leader CTA: a ring of
// kSchedDepth unit numbers that a twelfth warp obtains by cancelling the launch of clusters that have not started
// (clusterlaunchcontrol) and every other warp of the CTA group consumes.  Per slot: the 16-byte answer, the unit
// number, and three mbarriers (answer arrived / unit published / unit consumed by everyone).
constexpr int kSchedDepth = 4;
constexpr int kSchedConsumers = 11;  // warps per CTA that walk the tile list: 2 producers, MMA, 8 epilogue
constexpr uint32_t kSchedRespOff = 0, kSchedUnitOff = 16 * kSchedDepth, kSchedBarOff = kSchedUnitOff + 4 * kSchedDepth;
constexpr uint32_t kSchedSmemBytes = kSchedBarOff + 3 * 8 * kSchedDepth;
static_assert(kSchedBarOff % 8 == 0, "mbarriers are 8-byte aligned");

// Epilogue selector of the kernel: the public enum plus the split-K partial store.
enum : int {
  kEpiNone = 0,
  kEpiBias = 1,
  kEpiBiasRelu = 2,
  kEpiBiasGeluTanh = 3,
  kEpiSiluGate = 4,
  kEpiBiasResidual = 5,
  kEpiBiasSoftmax = 6,  // softmax over the whole output row (one n-tile per row), direct stores only
  kEpiPartial = 7       // raw FP32 accumulator to the split-K workspace
};
constexpr int kDeviceTimeoutCode = 7;  // FACT_ERR_DEVICE_TIMEOUT
struct FactTrue { static constexpr bool value = true; };    // compile-time tags for code written once and
struct FactFalse { static constexpr bool value = false; };  // instantiated for both operand formats

struct GemmParams {
  // problem
  int M, N_out, Nw, K, batch;
  // tiling and schedule
  int tile_n;        // accumulator columns per tile (UMMA N)
  int out_cols;      // output columns per tile: tile_n, or tile_n / 2 for SILU_GATE
  int tiles_m, tiles_n, k_blocks, split_k, raster_group, stages;
  int raster_along_n; // 1: the raster groups n-tiles (a slab of W stays in L2), 0: m-tiles (a slab of X)
  int k_serpentine;   // 1: every second tile of a CTA walks K downwards (L2 reuse between waves)
  int l2_keep_operands;  // L2 eviction priority of the operand loads (ptx::l2_policy)
  int k_base, k_rem;  // k_blocks = split_k * k_base + k_rem: slice s covers k_base (+1 if s < k_rem) k-blocks
  int total_units;   // batch * tiles_m * tiles_n * split_k
  // B operand loads issued by ONE CTA per stage
  int b_loads;       // number of TMA boxes
  int b_box_n;       // accumulator columns covered by one box
  int b_kn;          // 1: B is [K x N] (N contiguous), 0: W is [N x K]
  int gate;          // 1: SILU_GATE column pairing
  uint32_t b_box_bytes;
  uint32_t stage_bytes;  // A + B bytes of one CTA's stage
  uint32_t tx_bytes;     // bytes the `full` barrier expects (both CTAs' stages when CG == 2)
  // UMMA descriptors: everything but the start address; K advance in 16-byte units
  uint64_t a_desc, b_desc;
  uint32_t a_k_step, b_k_step;
  uint32_t idesc;
  uint32_t tmem_cols;
  // epilogue operands
  void* C;
  long long ldc, strideC;
  int out_f32, c_vec;
  int store_tma;  // 1: staged shared memory + TMA tensor stores (tmC); 0: direct register stores
  int epi_bufs;   // staging buffers per epilogue warp (1 or 2)
  int r_tma;      // 1: residual tiles come in by TMA (tmR); 0: direct loads
  const __nv_bfloat16* bias;
  int bias_vec;
  const __nv_bfloat16* R;
  long long ldr, strideR;
  int r_vec;
  // split-K partials, FP32: ws[(split * batch + b) * ws_planes + plane][M][ws_ld];
  // plane 1 holds the "up" columns of a gated accumulator
  int ws_planes;
  long long ws_ld;
  const float* ws;    // the partial planes, for the reduction in the kernel's tail
  int fused_reduce;   // 1: after a grid-wide barrier every CTA reduces its share of the output (split-K only)
  int reduce_epi;     // the epilogue the reduction applies
  int* status;        // [0] error word, [2..17] clock / profile counters, [24], [25] grid-barrier counters
  // grouped GEMM (the GROUPED instantiations only): the rows of A and C are cut into `groups` consecutive row
  // groups, group g multiplies W[g]; see decode_grouped
  int groups;
  const int* grp_tiles;   // [groups + 1] m-tiles (of tile_m rows) before each group
  const int* grp_rows;    // [groups + 1] first row of each group; grp_rows[groups] = M
  // 8-bit operands (FP8 E4M3, one byte per element): a k-block is 128 elements, still 128 bytes per row
  int k_elems;        // elements of K per k-block: 64 (BF16) or 128 (FP8)
  int fp8;            // 1: tcgen05.mma.kind::f8f6f4, else kind::f16
  int use_alpha;      // 1: the accumulator is multiplied by alpha before the epilogue (FP8: the operands' scales)
  float alpha;
  // stream-K (the SK instantiations only): the last `sk_tiles` tiles of the tile list are cut along K into one
  // contiguous run of k-blocks per CTA group; see UnitWalk
  int sk_tiles;       // 0: every tile is data-parallel
  int sk_first;       // index of the first stream-K tile (= number of data-parallel tiles = total_units)
  int sk_len, sk_rem; // group c owns k-block iterations [c * sk_len + min(c, sk_rem), + sk_len + (c < sk_rem))
  float* sk_ws;       // one FP32 accumulator tile per CTA: [gridDim.x][tile_n / 32][8][128] float4
  int* sk_flags;      // [gridDim.x][kEpiWarps]: 1 while that warp's share of the CTA's partial tile is ready
  // GEMM -> row normalisation -> GEMM without a pass over the activations (the EXT instantiations only: staged
  // BF16 epilogue of data-parallel tiles).
  // Producer: stats_out[chunk][row] = (sum, sum of squares) of the row's 64 stored BF16 values of column chunk
  // `chunk`.  Consumer: the rows of A are to be normalised over K (norm_mode 1: LayerNorm, 2: RMSNorm); the scale
  // vector is folded into W beforehand, so acc' = rstd[r] * acc - rstd[r] * mean[r] * colsum[n], with mean and
  // rstd from the K / 64 partial sums of stats_in.
  float2* stats_out;       // [ceil(N_out / 64)][M] or null
  const float2* stats_in;  // [ceil(K / 64)][M] or null
  const float* colsum;     // [N_out]: sum over k of the folded W[n][k] (LayerNorm only)
  int norm_mode;
  float norm_eps;
  // EXT = 3 instantiations: the staged epilogue's arithmetic, but every thread stores its own row's 128 bytes of a
  // chunk straight from registers as four 32-byte stores (no staging traffic through shared memory)
  int row_stores;
  // bit 256: the first CTA counts where its cycles go (fact_last_kernel_profile).  In a -DFACT_EXPERIMENTS build
  // also the work-skipping switches: 1 = no loads, MMA on stale shared memory; 2 = loads only, no MMA; 4 = the
  // epilogue skips its global stores (they isolate the feed, issue and store ceilings; results are garbage).
  int debug;
};

struct WorkUnit {
  int b, tm, tn, kb_begin, kb_end, split;
  int m_base;    // grouped: first row of the unit's group (0 otherwise; rows are m_base + tm * tile_m + ...)
  int m_end;     // grouped: one past the last row of the group (M otherwise)
  int wave;      // ordinal of this data-parallel unit within its CTA (0 for stream-K pieces)
  int sk_role;   // 0: a whole tile; 1: the piece with the tile's first k-block (it finishes the tile); 2: a later piece
  int sk_peers;  // role 1: how many following CTA groups hold the tile's other pieces
};

__device__ __forceinline__ WorkUnit decode_unit(const GemmParams& p, int u) {
  // 32-bit unsigned arithmetic only, and no division at all on the common paths (one slice, one batch):
  // this runs once per tile in every role, on the critical path of short-K tiles.
  WorkUnit w;
  unsigned t = (unsigned)u;
  if (p.split_k > 1) {
    w.split = (int)(t % (unsigned)p.split_k);
    t /= (unsigned)p.split_k;
    // slices differ by at most one k-block: the first `k_rem` slices take `k_base + 1`
    const int lead = min(w.split, p.k_rem);
    w.kb_begin = w.split * p.k_base + lead;
    w.kb_end = w.kb_begin + p.k_base + (w.split < p.k_rem ? 1 : 0);
  } else {
    w.split = 0;
    w.kb_begin = 0;
    w.kb_end = p.k_blocks;
  }
  unsigned r = t;
  w.b = 0;
  if (p.batch > 1) {
    const unsigned per_batch = (unsigned)(p.tiles_m * p.tiles_n);
    w.b = (int)(t / per_batch);
    r = t - (unsigned)w.b * per_batch;
  }
  // grouped raster: within a group of `raster_group` tiles of the grouped dimension, walk those tiles
  // fastest and the other dimension slowest; then the next group
  const int grouped = p.raster_along_n ? p.tiles_n : p.tiles_m;
  const int other = p.raster_along_n ? p.tiles_m : p.tiles_n;
  const unsigned group_sz = (unsigned)(p.raster_group * other);
  const unsigned g = r / group_sz;
  const int first = (int)g * p.raster_group;
  const unsigned gsz = (unsigned)min(p.raster_group, grouped - first);
  const unsigned in = r - g * group_sz;
  const int o = (int)(in / gsz);
  const int gi = first + (int)(in - (unsigned)o * gsz);
  w.tm = p.raster_along_n ? o : gi;
  w.tn = p.raster_along_n ? gi : o;
  return w;
}

// Grouped GEMM: units are numbered group by group, tiles_n per m-tile.  The group of a unit is found by bisection in
// the prefix table of m-tiles.  Inside a group the walk takes slabs of `raster_group` m-tiles (their rows of A stay
// in L2) and, within a slab, the m-tiles fastest: CTAs that run at the same time then share the group's weight
// columns, which are streamed once per slab.
__device__ __forceinline__ WorkUnit decode_grouped(const GemmParams& p, int u) {
  WorkUnit w;
  const int mt = u / p.tiles_n;
  int lo = 0, hi = p.groups;  // invariant: grp_tiles[lo] <= mt < grp_tiles[hi]
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (__ldg(p.grp_tiles + mid) <= mt) lo = mid;
    else hi = mid;
  }
  const int first = __ldg(p.grp_tiles + lo);
  const int mtiles = __ldg(p.grp_tiles + lo + 1) - first;  // m-tiles of this group (> 0: empty groups own no unit)
  const int local = u - first * p.tiles_n;
  const int per_slab = p.raster_group * p.tiles_n;
  const int slab = local / per_slab;
  const int rem = local - slab * per_slab;
  const int height = min(p.raster_group, mtiles - slab * p.raster_group);
  w.tn = rem / height;
  w.tm = slab * p.raster_group + (rem - w.tn * height);
  w.b = lo;
  w.m_base = __ldg(p.grp_rows + lo);
  w.m_end = __ldg(p.grp_rows + lo + 1);
  w.split = 0;
  w.kb_begin = 0;
  w.kb_end = p.k_blocks;
  return w;
}

// ---------------------------------------------------------------------------------------------
// Stream-K partition (host and device share this arithmetic).  The k-block iterations of the stream-K tiles are
// numbered tile by tile, `k_blocks` per tile, and dealt out in contiguous runs: group c owns
// [sk_group_begin(c), sk_group_begin(c + 1)), runs differing by at most one iteration.
__host__ __device__ inline int sk_group_begin(int len, int rem, int c) { return c * len + (c < rem ? c : rem); }

struct SkPiece {
  int tile;        // index among the stream-K tiles
  int k0, k1;      // k-blocks [k0, k1) of that tile
  int role;        // 0: the whole tile; 1: the piece with the tile's first k-block (it finishes the tile); 2: a later piece
  int peers;       // role 1: how many following groups hold the tile's other pieces
};

// The next piece of `group`'s run, which currently stands at iteration `pos` and ends at `end`.
__host__ __device__ inline SkPiece sk_next_piece(int k_blocks, int len, int rem, int groups, int group, int& pos,
                                                 int end) {
  SkPiece pc;
  pc.tile = pos / k_blocks;
  pc.k0 = pos - pc.tile * k_blocks;
  const int left = end - pos;
  pc.k1 = (k_blocks - pc.k0 < left) ? k_blocks : pc.k0 + left;
  pc.role = pc.k0 > 0 ? 2 : (pc.k1 < k_blocks ? 1 : 0);
  pc.peers = 0;
  if (pc.role == 1) {
    const int tile_end = (pc.tile + 1) * k_blocks;
    int c2 = group + 1;
    while (c2 < groups && sk_group_begin(len, rem, c2) < tile_end) ++c2;
    pc.peers = c2 - group - 1;
  }
  pos += pc.k1 - pc.k0;
  return pc;
}

// The sequence of work units of one CTA group.  Data-parallel kernels: units unit0, unit0 + stride, ...
// Stream-K kernels: first the group's run of k-block iterations in the stream-K region -- a run covers the tail
// of one tile, whole tiles, and the head of another, each a unit of its own -- then its data-parallel tiles.
// A tile's pieces belong to consecutive groups; the group with the first k-block adds the others' FP32
// partials (in group order) to its own accumulator and applies the epilogue.  Those others meet that piece first
// of all their work and depend on nobody, so the wait for them cannot be circular.
// What a warp needs to take unit numbers from the dynamic scheduler's ring (DYN instantiations).
struct SchedCtx {
  uint32_t unit_full0;    // this CTA's "unit published" barriers (the scheduler of the leader CTA arrives on both CTAs')
  uint32_t unit_empty0;   // the leader CTA's "unit consumed" barriers, as a shared::cluster address
  uint32_t unit_ring0;    // the leader CTA's unit numbers, as a shared::cluster address
  volatile int* abort_flag;
  int* status;
};

__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status,
                                         unsigned long long limit_ns);
__device__ __forceinline__ bool wait_bar_cluster(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status);

template <bool SK, bool GROUPED = false, bool DYN = false, int CG = 1>
struct UnitWalk {
  int u, stride, wave;
  int sk_pos, sk_end, group;
  int slot;
  uint32_t phase;
  const SchedCtx* sc;
  __device__ __forceinline__ UnitWalk(const GemmParams& p, int unit0, int unit_stride, const SchedCtx* sched = nullptr)
      : u(unit0), stride(unit_stride), wave(0), sk_pos(0), sk_end(0), group(unit0), slot(0), phase(0), sc(sched) {
    if constexpr (SK) {
      sk_pos = sk_group_begin(p.sk_len, p.sk_rem, unit0);
      sk_end = sk_group_begin(p.sk_len, p.sk_rem, unit0 + 1);
    }
  }
  // DYN: the number of the next unit from the scheduler's ring (warp-uniform; -1: no more, or the wait was given up).
  // The first unit of a CTA group is its own cluster's; the others come in the order the scheduler obtained them.
  __device__ __forceinline__ int next_dynamic() {
    if (wave == 0) return u;
    const uint32_t fb = sc->unit_full0 + 8u * (uint32_t)slot;
    bool ok;
    if constexpr (CG == 2) ok = wait_bar_cluster(fb, phase, sc->abort_flag, sc->status);
    else ok = wait_bar(fb, phase, sc->abort_flag, sc->status, kWaitLimitNs);
    int v = -1;
    if ((threadIdx.x & 31) == 0 && ok) {
      if constexpr (CG == 2) v = ptx::ld_shared_cluster_s32(sc->unit_ring0 + 4u * (uint32_t)slot);
      else asm volatile("ld.shared.s32 %0, [%1];" : "=r"(v) : "r"(sc->unit_ring0 + 4u * (uint32_t)slot) : "memory");
    }
    // (the shuffle cannot issue before the load has returned, and the arrival below is issued after the shuffle: the
    // slot is not handed back to the scheduler before its value has been read)
    v = __shfl_sync(0xffffffffu, v, 0);
    ok = __all_sync(0xffffffffu, ok) != 0;
    if (!ok) return -1;
    if ((threadIdx.x & 31) == 0) {
      const uint32_t eb = sc->unit_empty0 + 8u * (uint32_t)slot;
      if constexpr (CG == 2) ptx::mbar_arrive_cluster_relaxed(eb);
      else ptx::mbar_arrive(eb);
    }
    if (++slot == kSchedDepth) {
      slot = 0;
      phase ^= 1u;
    }
    return v;
  }
  __device__ __forceinline__ bool next(const GemmParams& p, WorkUnit& w) {
    if constexpr (SK) {
      if (sk_pos < sk_end) {
        const SkPiece pc = sk_next_piece(p.k_blocks, p.sk_len, p.sk_rem, stride, group, sk_pos, sk_end);
        w = decode_unit(p, p.sk_first + pc.tile);
        w.m_base = 0;
        w.m_end = p.M;
        w.kb_begin = pc.k0;
        w.kb_end = pc.k1;
        w.wave = 0;
        w.sk_role = pc.role;
        w.sk_peers = pc.peers;
        return true;
      }
    }
    if constexpr (DYN) {
      u = next_dynamic();
      if (u < 0 || u >= p.total_units) return false;
    } else {
      if (u >= p.total_units) return false;
    }
    if constexpr (GROUPED) {
      w = decode_grouped(p, u);
    } else {
      w = decode_unit(p, u);
      w.m_base = 0;
      w.m_end = p.M;
    }
    w.wave = wave++;
    w.sk_role = 0;
    w.sk_peers = 0;
    if constexpr (!DYN) u += stride;
    return true;
  }
};

// Bounded wait for a flag in global memory to become `want`.  Returns false if the wait was abandoned.
__device__ __forceinline__ bool wait_flag(const int* flag, int want, volatile int* abort_flag, int* status) {
  unsigned long long t0 = 0;
  for (uint32_t it = 1;; ++it) {
    if (ptx::ld_acquire_gpu(flag) == want) return true;
    if ((it & 255u) == 0) {
      if (*abort_flag) return false;
      const unsigned long long now = ptx::globaltimer_ns();
      if (t0 == 0) {
        t0 = now;
      } else if (now - t0 > kWaitLimitNs) {
        *abort_flag = 1;
        atomicExch(status, kDeviceTimeoutCode);
        return false;
      }
    }
  }
}

// Bounded mbarrier wait.  Returns false if the wait was abandoned.
__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status,
                                         unsigned long long limit_ns) {
  if (ptx::mbar_try_wait(bar, parity)) return true;
  unsigned long long t0 = 0;
  for (uint32_t it = 1;; ++it) {
    if (ptx::mbar_try_wait(bar, parity)) return true;
    if ((it & 1023u) == 0) {
      if (*abort_flag) return false;
      const unsigned long long now = ptx::globaltimer_ns();
      if (t0 == 0) {
        t0 = now;
      } else if (now - t0 > limit_ns) {
        *abort_flag = 1;
        atomicExch(status, kDeviceTimeoutCode);
        return false;
      }
    }
  }
}

__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status) {
  return wait_bar(bar, parity, abort_flag, status, kWaitLimitNs);
}

// The same wait with cluster-scope acquire: for a barrier the peer CTA arrives on after writing data this CTA reads.
__device__ __forceinline__ bool wait_bar_cluster(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status) {
  if (ptx::mbar_try_wait_cluster(bar, parity)) return true;
  unsigned long long t0 = 0;
  for (uint32_t it = 1;; ++it) {
    if (ptx::mbar_try_wait_cluster(bar, parity)) return true;
    if ((it & 1023u) == 0) {
      if (*abort_flag) return false;
      const unsigned long long now = ptx::globaltimer_ns();
      if (t0 == 0) {
        t0 = now;
      } else if (now - t0 > kWaitLimitNs) {
        *abort_flag = 1;
        atomicExch(status, kDeviceTimeoutCode);
        return false;
      }
    }
  }
}

__device__ __forceinline__ void unpack_bf16x8(const uint4& q, float (&f)[8]) {
  f[0] = __uint_as_float(q.x << 16);
  f[1] = __uint_as_float(q.x & 0xffff0000u);
  f[2] = __uint_as_float(q.y << 16);
  f[3] = __uint_as_float(q.y & 0xffff0000u);
  f[4] = __uint_as_float(q.z << 16);
  f[5] = __uint_as_float(q.z & 0xffff0000u);
  f[6] = __uint_as_float(q.w << 16);
  f[7] = __uint_as_float(q.w & 0xffff0000u);
}

// 8 consecutive BF16 values starting at ptr[0]; entries >= nvalid read as 0.
__device__ __forceinline__ void load_bf16x8(const __nv_bfloat16* ptr, int nvalid, bool vec, float (&f)[8]) {
  if (vec && nvalid >= 8) {
    const uint4 q = __ldg(reinterpret_cast<const uint4*>(ptr));
    unpack_bf16x8(q, f);
  } else {
#pragma unroll
    for (int j = 0; j < 8; ++j) f[j] = (j < nvalid) ? __bfloat162float(ptr[j]) : 0.f;
  }
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}

__device__ __forceinline__ void store_bf16x8(__nv_bfloat16* dst, const float (&y)[8], int nvalid, bool vec) {
  if (vec && nvalid >= 8) {
    uint4 q;
    q.x = pack_bf16x2(y[0], y[1]);
    q.y = pack_bf16x2(y[2], y[3]);
    q.z = pack_bf16x2(y[4], y[5]);
    q.w = pack_bf16x2(y[6], y[7]);
    *reinterpret_cast<uint4*>(dst) = q;
  } else {
#pragma unroll
    for (int j = 0; j < 8; ++j)
      if (j < nvalid) dst[j] = __float2bfloat16_rn(y[j]);
  }
}

__device__ __forceinline__ void store_f32x8(float* dst, const float (&y)[8], int nvalid, bool vec) {
  if (vec && nvalid >= 8) {
    *reinterpret_cast<float4*>(dst) = make_float4(y[0], y[1], y[2], y[3]);
    *reinterpret_cast<float4*>(dst + 4) = make_float4(y[4], y[5], y[6], y[7]);
  } else {
#pragma unroll
    for (int j = 0; j < 8; ++j)
      if (j < nvalid) dst[j] = y[j];
  }
}

__device__ __forceinline__ float gelu_tanh_f32(float z) {
  // 0.5 z (1 + tanh(sqrt(2/pi) (z + 0.044715 z^3)))
  const float u = 0.7978845608028654f * fmaf(0.044715f * z * z, z, z);
  return 0.5f * z * (1.f + ptx::tanh_approx(u));
}
__device__ __forceinline__ float silu_f32(float g) { return __fdividef(g, 1.f + __expf(-g)); }

template <int EPI>
constexpr bool epi_has_bias() {
  return EPI == kEpiBias || EPI == kEpiBiasRelu || EPI == kEpiBiasGeluTanh || EPI == kEpiBiasResidual ||
         EPI == kEpiBiasSoftmax;
}

// The fused element-wise operation on 8 consecutive output columns.
template <int EPI>
__device__ __forceinline__ void apply_epilogue8(const uint32_t* acc, const uint32_t* acc_up, const float (&bias)[8],
                                                const float (&res)[8], float (&y)[8]) {
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const float a = __uint_as_float(acc[j]);
    if constexpr (EPI == kEpiNone || EPI == kEpiPartial) {
      y[j] = a;
    } else if constexpr (EPI == kEpiBias) {
      y[j] = a + bias[j];
    } else if constexpr (EPI == kEpiBiasRelu) {
      y[j] = fmaxf(a + bias[j], 0.f);
    } else if constexpr (EPI == kEpiBiasGeluTanh) {
      y[j] = gelu_tanh_f32(a + bias[j]);
    } else if constexpr (EPI == kEpiSiluGate) {
      y[j] = silu_f32(a) * __uint_as_float(acc_up[j]);
    } else {  // kEpiBiasResidual
      y[j] = a + bias[j] + res[j];
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Split-K reduction: adds the S partials of every output element in ascending slice order,
// applies the epilogue and stores.  One thread per 4 consecutive output columns.  The same routine
// serves the tail of the GEMM kernel (all CTAs, after a grid-wide barrier) and a stand-alone kernel.
struct ReduceParams {
  const float* ws;  // ws[(split * batch + b) * planes + plane][M][ws_ld]
  long long ws_ld;
  int planes;
  int splits;
  int M, N_out, batch;
  int epi;
  void* C;
  long long ldc, strideC;
  int out_f32;
  const __nv_bfloat16* bias;
  const __nv_bfloat16* R;
  long long ldr, strideR;
  float alpha;  // the summed accumulator is multiplied by this first (1 unless the operands carry scales)
};

__device__ __forceinline__ float reduce_epilogue(int epi, float a, float up, float bias, float res) {
  switch (epi) {
    case kEpiBias: return a + bias;
    case kEpiBiasRelu: return fmaxf(a + bias, 0.f);
    case kEpiBiasGeluTanh: return gelu_tanh_f32(a + bias);
    case kEpiSiluGate: return silu_f32(a) * up;
    case kEpiBiasResidual: return a + bias + res;
    default: return a;
  }
}

constexpr int kReduceBatch = 10;  // loads in flight per thread and round trip: 40 slices (the 37 of a 148-SM part in one trip)

// Four adjacent lanes share one group of 4 output columns: lane q of the quad adds slices q, q+4, q+8, ...
// in ascending order, then the four sums are combined as (s0 + s1) + (s2 + s3).  The order of every
// addition depends only on the number of slices, so the result is reproducible bit for bit.
// `first` and `stride` count threads and must be multiples of 32 (whole warps walk the loop together).
__device__ __forceinline__ void reduce_groups(const ReduceParams& p, long long first, long long stride) {
  const long long groups_per_row = (p.N_out + 3) / 4;
  const long long total = (long long)p.batch * p.M * groups_per_row;
  const long long plane_stride = (long long)p.M * p.ws_ld;
  const long long slice_stride = (long long)p.batch * p.planes * plane_stride;
  const bool gate = p.epi == kEpiSiluGate;
  const long long warp_first = first & ~31LL;
  const int lane = (int)(first & 31);
  const int sub = lane & 3;
  for (long long t0 = warp_first; t0 < total * 4; t0 += stride) {  // uniform trip count within a warp
    const long long i = (t0 + lane) >> 2;                           // the quad's group
    const bool valid = i < total;
    const long long ii = valid ? i : 0;
    int gcol, m, b;
    if (total < 0x7fffffffLL) {  // 32-bit index arithmetic: 64-bit division costs hundreds of cycles
      const unsigned iu = (unsigned)ii, gpr = (unsigned)groups_per_row;
      const unsigned rmu = iu / gpr;
      gcol = (int)(iu - rmu * gpr);
      b = (int)(rmu / (unsigned)p.M);
      m = (int)(rmu - (unsigned)b * (unsigned)p.M);
    } else {
      gcol = (int)(ii % groups_per_row);
      const long long rm = ii / groups_per_row;
      m = (int)(rm % p.M);
      b = (int)(rm / p.M);
    }
    const int n = gcol * 4;
    const int nvalid = min(4, p.N_out - n);
    float a[4] = {0.f, 0.f, 0.f, 0.f}, up[4] = {0.f, 0.f, 0.f, 0.f};
    const float* base = p.ws + ((long long)b * p.planes) * plane_stride + (long long)m * p.ws_ld + n;
    if (valid) {
      for (int s0 = sub; s0 < p.splits; s0 += 4 * kReduceBatch) {  // this lane's slices, a batch of loads at a time
        float4 v[kReduceBatch], t[kReduceBatch];
#pragma unroll
        for (int i8 = 0; i8 < kReduceBatch; ++i8) {
          const int sl = s0 + 4 * i8;
          if (sl < p.splits) {
            const float* ps = base + (long long)sl * slice_stride;
            v[i8] = __ldcg(reinterpret_cast<const float4*>(ps));  // ws_ld is a multiple of 4: padding is in bounds
            if (gate) t[i8] = __ldcg(reinterpret_cast<const float4*>(ps + plane_stride));
          }
        }
#pragma unroll
        for (int i8 = 0; i8 < kReduceBatch; ++i8) {
          if (s0 + 4 * i8 < p.splits) {
            a[0] += v[i8].x; a[1] += v[i8].y; a[2] += v[i8].z; a[3] += v[i8].w;
            if (gate) {
              up[0] += t[i8].x; up[1] += t[i8].y; up[2] += t[i8].z; up[3] += t[i8].w;
            }
          }
        }
      }
    }
    // (s0 + s1) + (s2 + s3): every lane of the quad ends with the same total
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      a[j] += __shfl_xor_sync(0xffffffffu, a[j], 1);
      a[j] += __shfl_xor_sync(0xffffffffu, a[j], 2);
      if (gate) {
        up[j] += __shfl_xor_sync(0xffffffffu, up[j], 1);
        up[j] += __shfl_xor_sync(0xffffffffu, up[j], 2);
      }
    }
    // lane `sub` of the quad finishes column n + sub
    if (valid && sub < nvalid) {
      const int j = sub;
      const float av = sub == 0 ? a[0] : sub == 1 ? a[1] : sub == 2 ? a[2] : a[3];
      const float uv = sub == 0 ? up[0] : sub == 1 ? up[1] : sub == 2 ? up[2] : up[3];
      const float bias = p.bias ? __bfloat162float(p.bias[n + j]) : 0.f;
      const float res =
          (p.epi == kEpiBiasResidual) ? __bfloat162float(p.R[(long long)b * p.strideR + (long long)m * p.ldr + n + j]) : 0.f;
      const float y = reduce_epilogue(p.epi, av * p.alpha, uv * p.alpha, bias, res);
      const long long off = (long long)b * p.strideC + (long long)m * p.ldc + n + j;
      if (p.out_f32) reinterpret_cast<float*>(p.C)[off] = y;
      else reinterpret_cast<__nv_bfloat16*>(p.C)[off] = __float2bfloat16_rn(y);
    }
  }
}

// The same sums for a few slices of a large output: one thread adds every slice of 8 adjacent columns of a row,
// with all its loads in flight at once, and stores 16 (BF16) or 32 (FP32) bytes.  (The quads above keep one round
// trip to L2 per 32 outputs of a warp, which a 16384 x 768 output with two slices pays 400 000 times over: 445 us.)
// Same association as the quads -- s_q = slices q, q + 4 in ascending order, then (s0 + s1) + (s2 + s3) -- so the
// two walks agree bit for bit and either may serve a call.
constexpr int kReduceWideSlices = 8;
__device__ __forceinline__ bool reduce_wide_applies(const ReduceParams& p) {
  return p.splits <= kReduceWideSlices && p.epi != kEpiSiluGate && (p.ws_ld & 7) == 0;
}
// G groups per trip, each with up to S slices: G * S * 2 16-byte loads in flight per thread.
template <int G, int S>
__device__ __forceinline__ void reduce_wide_gs(const ReduceParams& p, long long first, long long stride) {
  const long long groups_per_row = (p.N_out + 7) / 8;
  const long long total = (long long)p.batch * p.M * groups_per_row;
  const long long plane_stride = (long long)p.M * p.ws_ld;
  const long long slice_stride = (long long)p.batch * p.planes * plane_stride;
  const size_t esz = p.out_f32 ? 4 : 2;
  const bool c_vec = (reinterpret_cast<uintptr_t>(p.C) & 15) == 0 && ((p.ldc * esz) & 15) == 0 && ((p.strideC * esz) & 15) == 0;
  const bool r_vec = p.R != nullptr && (reinterpret_cast<uintptr_t>(p.R) & 15) == 0 && (p.ldr & 7) == 0 && (p.strideR & 7) == 0;
  const bool b_vec = p.bias != nullptr && (reinterpret_cast<uintptr_t>(p.bias) & 15) == 0;
  for (long long i0 = first; i0 < total; i0 += stride * G) {
    int n[G], m[G], b[G];
    bool valid[G];
    float4 v[G][S][2];
#pragma unroll
    for (int g = 0; g < G; ++g) {
      const long long i = i0 + (long long)g * stride;
      valid[g] = i < total;
      const long long ii = valid[g] ? i : 0;
      int gcol;
      if (total < 0x7fffffffLL) {
        const unsigned iu = (unsigned)ii, gpr = (unsigned)groups_per_row;
        const unsigned rmu = iu / gpr;
        gcol = (int)(iu - rmu * gpr);
        b[g] = (int)(rmu / (unsigned)p.M);
        m[g] = (int)(rmu - (unsigned)b[g] * (unsigned)p.M);
      } else {
        gcol = (int)(ii % groups_per_row);
        const long long rm = ii / groups_per_row;
        m[g] = (int)(rm % p.M);
        b[g] = (int)(rm / p.M);
      }
      n[g] = gcol * 8;
      const float* base = p.ws + ((long long)b[g] * p.planes) * plane_stride + (long long)m[g] * p.ws_ld + n[g];
#pragma unroll
      for (int sl = 0; sl < S; ++sl)
        if (valid[g] && sl < p.splits) {  // (ws_ld is a multiple of 8 here: both loads stay inside the row's padding)
          const float4* ps = reinterpret_cast<const float4*>(base + (long long)sl * slice_stride);
          v[g][sl][0] = __ldcg(ps);
          v[g][sl][1] = __ldcg(ps + 1);
        }
    }
#pragma unroll
    for (int g = 0; g < G; ++g) {
      if (!valid[g]) continue;
      const int nvalid = min(8, p.N_out - n[g]);
      float acc[4][8];
#pragma unroll
      for (int q = 0; q < 4; ++q)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[q][j] = 0.f;
#pragma unroll
      for (int sl = 0; sl < S; ++sl)
        if (sl < p.splits) {
          const int q = sl & 3;
          acc[q][0] += v[g][sl][0].x; acc[q][1] += v[g][sl][0].y; acc[q][2] += v[g][sl][0].z; acc[q][3] += v[g][sl][0].w;
          acc[q][4] += v[g][sl][1].x; acc[q][5] += v[g][sl][1].y; acc[q][6] += v[g][sl][1].z; acc[q][7] += v[g][sl][1].w;
        }
      float bias[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f}, res[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
      if (p.bias != nullptr) load_bf16x8(p.bias + n[g], nvalid, b_vec, bias);
      if (p.epi == kEpiBiasResidual)
        load_bf16x8(p.R + (long long)b[g] * p.strideR + (long long)m[g] * p.ldr + n[g], nvalid, r_vec, res);
      float y[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const float tot = (acc[0][j] + acc[1][j]) + (acc[2][j] + acc[3][j]);
        y[j] = reduce_epilogue(p.epi, tot * p.alpha, 0.f, bias[j], res[j]);
      }
      const long long off = (long long)b[g] * p.strideC + (long long)m[g] * p.ldc + n[g];
      if (p.out_f32) {
        float* dst = reinterpret_cast<float*>(p.C) + off;
        if (c_vec && nvalid == 8) {
          reinterpret_cast<float4*>(dst)[0] = make_float4(y[0], y[1], y[2], y[3]);
          reinterpret_cast<float4*>(dst)[1] = make_float4(y[4], y[5], y[6], y[7]);
        } else {
#pragma unroll
          for (int j = 0; j < 8; ++j)
            if (j < nvalid) dst[j] = y[j];
        }
      } else {
        store_bf16x8(reinterpret_cast<__nv_bfloat16*>(p.C) + off, y, nvalid, c_vec);
      }
    }
  }
}
__device__ __forceinline__ void reduce_wide(const ReduceParams& p, long long first, long long stride) {
  if (p.splits <= 2) reduce_wide_gs<4, 2>(p, first, stride);
  else if (p.splits <= 4) reduce_wide_gs<2, 4>(p, first, stride);
  else reduce_wide_gs<1, kReduceWideSlices>(p, first, stride);
}

__device__ __forceinline__ void reduce_slices(const ReduceParams& p, long long first, long long stride) {
  if (reduce_wide_applies(p)) reduce_wide(p, first, stride);
  else reduce_groups(p, first, stride);
}

__global__ void __launch_bounds__(128) fact_splitk_reduce_kernel(const ReduceParams p) {
  ptx::grid_dependency_wait();  // (the successor is released when this grid's CTAs exit)
  reduce_slices(p, blockIdx.x * (long long)blockDim.x + threadIdx.x, (long long)gridDim.x * blockDim.x);
}

// The fused element-wise operation on two adjacent output columns, as packed FP32 pairs
// (add/mul/fma.f32x2 halve the instruction count of the epilogue, which is issue-bound).
template <int EPI>
__device__ __forceinline__ uint64_t epilogue_pair(uint64_t acc, uint64_t up, uint64_t bias, uint64_t res) {
  if constexpr (EPI == kEpiNone || EPI == kEpiPartial) {
    return acc;
  } else if constexpr (EPI == kEpiBias) {
    return ptx::add_f32x2(acc, bias);
  } else if constexpr (EPI == kEpiBiasRelu) {
    uint32_t lo, hi;
    ptx::unpack_f32x2(ptx::add_f32x2(acc, bias), lo, hi);
    return ptx::pack_f32x2(__float_as_uint(fmaxf(__uint_as_float(lo), 0.f)),
                           __float_as_uint(fmaxf(__uint_as_float(hi), 0.f)));
  } else if constexpr (EPI == kEpiBiasGeluTanh) {
    // z (k0 + k1 z^2) = sqrt(2/pi) (z + 0.044715 z^3);  0.5 z (1 + tanh u) = h + h tanh u with h = 0.5 z
    const uint64_t k0 = ptx::pack_f32x2(__float_as_uint(0.7978845608028654f), __float_as_uint(0.7978845608028654f));
    const uint64_t k1 = ptx::pack_f32x2(__float_as_uint(0.7978845608028654f * 0.044715f),
                                        __float_as_uint(0.7978845608028654f * 0.044715f));
    const uint64_t half2 = ptx::pack_f32x2(__float_as_uint(0.5f), __float_as_uint(0.5f));
    const uint64_t z = ptx::add_f32x2(acc, bias);
    const uint64_t u = ptx::mul_f32x2(ptx::fma_f32x2(ptx::mul_f32x2(z, z), k1, k0), z);
    uint32_t ulo, uhi;
    ptx::unpack_f32x2(u, ulo, uhi);
    const uint64_t t = ptx::pack_f32x2(__float_as_uint(ptx::tanh_approx(__uint_as_float(ulo))),
                                       __float_as_uint(ptx::tanh_approx(__uint_as_float(uhi))));
    const uint64_t h = ptx::mul_f32x2(z, half2);
    return ptx::fma_f32x2(h, t, h);
  } else if constexpr (EPI == kEpiSiluGate) {
    uint32_t glo, ghi;
    ptx::unpack_f32x2(acc, glo, ghi);
    const uint64_t s = ptx::pack_f32x2(__float_as_uint(silu_f32(__uint_as_float(glo))),
                                       __float_as_uint(silu_f32(__uint_as_float(ghi))));
    return ptx::mul_f32x2(s, up);
  } else {  // kEpiBiasResidual
    return ptx::add_f32x2(ptx::add_f32x2(acc, bias), res);
  }
}

template <int CG, int EPI, bool SK = false, bool GROUPED = false, int EXT = 0, bool DYN = false>
__global__ void __launch_bounds__(kThreads + (DYN ? 32 : 0), 1)
    fact_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                     const __grid_constant__ CUtensorMap tmC, const __grid_constant__ CUtensorMap tmR,
                     const GemmParams p) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];

  // The warp index is made provably warp-uniform (a shuffle result), and the producer / MMA roles
  // run their loops with all 32 lanes converged, electing one lane only for the instruction that
  // must be issued once.  Loop state then lives in uniform registers; running the whole loop in a
  // single divergent lane instead costs ~80 cycles per tcgen05/TMA instruction and starves the
  // tensor pipe.
  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);
  const int lane = threadIdx.x & 31;
  const uint32_t cta_rank = (CG == 2) ? ptx::cluster_ctarank() : 0u;
  const uint32_t smem_base = ptx::smem_u32(smem_raw);
  if (smem_base & 1023u) {  // the swizzled tiles need a 1024-byte aligned ring: refuse to run otherwise
    if (threadIdx.x == 0) atomicExch(p.status, kDeviceTimeoutCode);
    return;
  }
  if constexpr (GROUPED) {  // (group boundaries are kept by row-predicated stores, staged or direct)
    static_assert(!SK && EPI != kEpiPartial, "grouped tiles are data-parallel");
    if (p.grp_tiles == nullptr || p.grp_rows == nullptr) {
      if (threadIdx.x == 0) atomicExch(p.status, kDeviceTimeoutCode);
      return;
    }
  }
  if constexpr (EXT != 0) {  // 1: row sums out; 2: a folded normalisation in (and row sums out); 3: rows stored
                             // from registers -- all in the staged epilogue of a whole, ungrouped tile
    static_assert(!SK && !GROUPED && EPI != kEpiPartial && EPI != kEpiBiasSoftmax, "extras: plain data-parallel tiles");
    if (!p.store_tma || (EXT != 2 && p.norm_mode != 0) || (p.norm_mode != 0 && p.stats_in == nullptr) ||
        (p.norm_mode == 1 && p.colsum == nullptr) || (EXT == 3) != (p.row_stores != 0) ||
        (EXT == 3 && p.stats_out != nullptr)) {
      if (threadIdx.x == 0) atomicExch(p.status, kDeviceTimeoutCode);
      return;
    }
  } else if (p.norm_mode != 0 || p.stats_out != nullptr || p.row_stores != 0) {  // asked of an instantiation that has no code for it
    if (threadIdx.x == 0) atomicExch(p.status, kDeviceTimeoutCode);
    return;
  }
  if constexpr (DYN) {  // dynamic scheduling hands out whole data-parallel tiles, one cluster of the grid per tile
    static_assert(!SK && EXT == 0 && EPI != kEpiPartial, "dynamic scheduling: plain data-parallel tiles");
    if ((int)(gridDim.x / CG) != p.total_units || p.split_k != 1) {
      if (threadIdx.x == 0) atomicExch(p.status, kDeviceTimeoutCode);
      return;
    }
  }
  if constexpr (EPI == kEpiBiasSoftmax) {  // a row's softmax needs the whole row in one tile and the direct stores
    if (p.store_tma || p.tiles_n != 1) {
      if (threadIdx.x == 0) atomicExch(p.status, kDeviceTimeoutCode);
      return;
    }
  }
  if constexpr (SK) {  // stream-K pieces are parked and finished by the staged epilogue only: refuse anything else
    if (!p.store_tma || p.sk_ws == nullptr || p.sk_flags == nullptr) {
      if (threadIdx.x == 0) atomicExch(p.status, kDeviceTimeoutCode);
      return;
    }
  }
  const uint32_t epi_base = smem_base + (uint32_t)p.stages * p.stage_bytes;
  const uint32_t bias_base = epi_base + (uint32_t)(kEpiWarps * p.epi_bufs) * kEpiBufBytes;
  const uint32_t bar_base = bias_base + kEpiWarps * kEpiBiasBytes;
  const uint32_t ctrl_off = bar_base - smem_base + kNumBarriers * 8;
  const uint32_t norm_cs_base = bar_base + kCtrlSmemBytes;  // (present only when the host asked for it: norm_mode 1)
  volatile uint32_t* tmem_holder_p = reinterpret_cast<volatile uint32_t*>(smem_raw + ctrl_off);
  volatile int* abort_p = reinterpret_cast<volatile int*>(smem_raw + ctrl_off + 4);
  auto full_bar = [&](int s) { return bar_base + 8u * (uint32_t)s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (uint32_t)(kMaxStages + s); };
  auto accf_bar = [&](int b) { return bar_base + 8u * (uint32_t)(2 * kMaxStages + b); };
  auto acce_bar = [&](int b) { return bar_base + 8u * (uint32_t)(2 * kMaxStages + 2 + b); };
  auto res_bar = [&](int e, int b) {
    return bar_base + 8u * (uint32_t)(2 * kMaxStages + 4 + e * kEpiMaxBufs + b);
  };

  // dynamic scheduler's ring (DYN only; the host reserved the bytes): answers, unit numbers, barriers
  const uint32_t sched_base = bar_base + kCtrlSmemBytes;
  auto clc_bar = [&](int s) { return sched_base + kSchedBarOff + 8u * (uint32_t)s; };
  auto unit_full_bar = [&](int s) { return sched_base + kSchedBarOff + 8u * (uint32_t)(kSchedDepth + s); };
  auto unit_empty_bar = [&](int s) { return sched_base + kSchedBarOff + 8u * (uint32_t)(2 * kSchedDepth + s); };
  SchedCtx sched_ctx;
  if constexpr (DYN) {
    sched_ctx.unit_full0 = unit_full_bar(0);
    sched_ctx.unit_empty0 = (CG == 2) ? ptx::mapa(unit_empty_bar(0), 0) : unit_empty_bar(0);
    sched_ctx.unit_ring0 = (CG == 2) ? ptx::mapa(sched_base + kSchedUnitOff, 0) : sched_base + kSchedUnitOff;
    sched_ctx.abort_flag = abort_p;
    sched_ctx.status = p.status;
    if (threadIdx.x >= 64 && threadIdx.x < 64 + 3 * kSchedDepth) {
      const int i = (int)threadIdx.x - 64;
      // answer arrived: the requesting thread; unit published: the scheduler; unit consumed: every walking warp of
      // the CTA group
      ptx::mbar_init(sched_base + kSchedBarOff + 8u * (uint32_t)i, i >= 2 * kSchedDepth ? kSchedConsumers * CG : 1);
      ptx::fence_mbar_init();
    }
  }
  const SchedCtx* const sched = DYN ? &sched_ctx : nullptr;

  // One thread per mbarrier: serial initialisation by a single thread costs about a thousand cycles of prologue.
  if (threadIdx.x < kNumBarriers) {
    const int i = (int)threadIdx.x;
    uint32_t count = 1;                                                                  // full / empty / acc_full / residual
    if (i >= 2 * kMaxStages + 2 && i < 2 * kMaxStages + 4) count = kEpiWarps * CG;       // acc_empty: one arrival per
    ptx::mbar_init(bar_base + 8u * (uint32_t)i, count);                                  // epilogue warp of the group
    if (i == 0) *abort_p = 0;
    ptx::fence_mbar_init();
  }
  if (warp == 0 && lane == 0) {
    ptx::prefetch_tensormap(&tmA);
    ptx::prefetch_tensormap(&tmB);
  }
  if (warp == 1) {
    __syncwarp();  // lanes 0..3 of this warp initialised barriers above: reconverge for the warp-wide allocation
    ptx::tmem_alloc<CG>(smem_base + ctrl_off, p.tmem_cols);
    ptx::tmem_relinquish<CG>();
  }
  ptx::tc_fence_before();
  __syncthreads();
  if constexpr (CG == 2) {  // the peer's barriers must exist before anything arrives on them
    ptx::cluster_arrive();
    ptx::cluster_wait();
  }
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_holder_p;
  // Everything above touched shared and tensor memory only and may overlap the tail of the kernel before this one
  // in the stream; from here on global memory is read and written.
  ptx::grid_dependency_wait();
  const long long t_go = clock64();

  // CTA 0 stamps the SM cycle counter and the nanosecond timer around its work (status[2..5]):
  // their ratio is the SM clock this launch really ran at.
  long long t_clk0 = 0;
  unsigned long long t_ns0 = 0;
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    t_clk0 = clock64();
    t_ns0 = ptx::globaltimer_ns();
  }
  // With debug bit 256 the first CTA also counts where its cycles go (status[2..]: see fact_last_kernel_profile), and
  // every CTA stamps the nanosecond timer on its way in and out (status[40..43]: earliest start, latest end).
  const bool prof = (p.debug & 256) && blockIdx.x == 0;
  if ((p.debug & 256) && threadIdx.x == 0)
    atomicMin(reinterpret_cast<unsigned long long*>(p.status + 40), (unsigned long long)ptx::globaltimer_ns());
  const int unit0 = (int)(blockIdx.x / CG);
  const int unit_stride = (int)(gridDim.x / CG);
  // a bounded wait whose verdict is warp-uniform
  auto wait_all = [&](uint32_t bar, uint32_t parity) -> bool {
    return __all_sync(0xffffffffu, wait_bar(bar, parity, abort_p, p.status)) != 0;
  };

  if (warp == 0 || warp == kProducerBWarp) {
    // ------------------------------------------------------------ TMA producers
    // Warp 0 loads the A tiles (and posts the expected byte count), warp 6 the B boxes.
    const bool do_a = warp == 0;
    if (!FACT_SKIP(p, 1)) {
      const uint64_t pol = ptx::l2_policy(p.l2_keep_operands);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      UnitWalk<SK, GROUPED, DYN, CG> walk(p, unit0, unit_stride, sched);
      WorkUnit w;
      while (ok && walk.next(p, w)) {
        // Odd waves walk K downwards: the wave before ended at the top of K, so the operand slabs both waves
        // share (same m-tiles of A, or same n-tiles of B) are met while they are still in L2.  The sum of an
        // output element is then taken in descending k in those tiles, still fixed by (shape, config).
        // (not with dynamic scheduling: which tiles a CTA gets, and so the parity of their count, is not fixed there,
        // and the order of a sum must not depend on it)
        const bool k_down = !DYN && (w.wave & 1) && p.k_serpentine;
        const int m0 = (GROUPED ? w.m_base : 0) + (w.tm * CG + (int)cta_rank) * kTileM;
        const int a_batch = GROUPED ? 0 : w.b;  // grouped: A is one matrix, the group selects the weights only
        // first accumulator column this CTA's B boxes feed, and the W column of every box
        const int col0 = (CG == 2) ? (int)cta_rank * (p.tile_n / 2) : 0;
        int n_box[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int col = col0 + i * p.b_box_n;
          if (p.gate) {
            const int half = p.tile_n >> 1;
            n_box[i] = (col < half) ? (w.tn * half + col) : (p.N_out + w.tn * half + (col - half));
          } else {
            n_box[i] = w.tn * p.tile_n + col;
          }
        }
        for (int kbi = w.kb_begin; kbi < w.kb_end; ++kbi) {
          const int kb = k_down ? (w.kb_end - 1 - (kbi - w.kb_begin)) : kbi;
          if (!wait_all(empty_bar(stage), phase ^ 1u)) {
            ok = false;
            break;
          }
          const uint32_t sa = smem_base + (uint32_t)stage * p.stage_bytes;
          const uint32_t sb = sa + kStageBytesA;
          uint32_t fb = full_bar(stage);
          if (ptx::elect_one()) {
            if (do_a) {
              if constexpr (CG == 2) {
                if (cta_rank == 0) ptx::mbar_arrive_expect_tx(fb, p.tx_bytes);
                fb = ptx::mapa(fb, 0);  // both CTAs' loads complete on the leader's barrier
                ptx::tma_load_3d_cg2_hint(sa, &tmA, fb, kb * p.k_elems, m0, a_batch, pol);
              } else {
                ptx::mbar_arrive_expect_tx(fb, p.tx_bytes);
                ptx::tma_load_3d_hint(sa, &tmA, fb, kb * p.k_elems, m0, a_batch, pol);
              }
            } else {
              if constexpr (CG == 2) fb = ptx::mapa(fb, 0);
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                if (i < p.b_loads) {
                  const uint32_t dst = sb + (uint32_t)i * p.b_box_bytes;
                  if constexpr (CG == 2) {
                    if (p.b_kn) ptx::tma_load_3d_cg2_hint(dst, &tmB, fb, n_box[i], kb * p.k_elems, w.b, pol);
                    else ptx::tma_load_3d_cg2_hint(dst, &tmB, fb, kb * p.k_elems, n_box[i], w.b, pol);
                  } else {
                    if (p.b_kn) ptx::tma_load_3d_hint(dst, &tmB, fb, n_box[i], kb * p.k_elems, w.b, pol);
                    else ptx::tma_load_3d_hint(dst, &tmB, fb, kb * p.k_elems, n_box[i], w.b, pol);
                  }
                }
              }
            }
          }
          if (++stage == p.stages) {
            stage = 0;
            phase ^= 1u;
          }
        }
      }
      // Drain: wait until every stage this CTA filled has been released, so that no
      // commit arrival is still on its way to this CTA's barriers when it exits.
      for (int s = 0; ok && do_a && s < p.stages; ++s) {
        if (!wait_all(empty_bar(stage), phase ^ 1u)) ok = false;
        if (++stage == p.stages) {
          stage = 0;
          phase ^= 1u;
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    // The operand format is chosen once, outside every loop: whatever the issuing thread does between two
    // instructions is idle time on the tensor pipe (a warp-uniform `if (p.fp8)` in front of every instruction cost
    // 16 % of the 8192^3 product: 1.086 M instead of 0.933 M cycles).
    auto issue_all = [&](auto fp8_tag) {
      constexpr bool kFp8 = decltype(fp8_tag)::value;
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      long long prof_acc_wait = 0, prof_full_wait = 0, prof_first_full = 0;
      UnitWalk<SK, GROUPED, DYN, CG> walk(p, unit0, unit_stride, sched);
      WorkUnit w;
      while (ok && walk.next(p, w)) {
        long long t0 = prof ? clock64() : 0;
        if (!wait_all(acce_bar(acc), acc_phase ^ 1u)) {
          ok = false;
          break;
        }
        if (prof) prof_acc_wait += clock64() - t0;
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * p.tile_n);
        for (int kb = w.kb_begin; kb < w.kb_end; ++kb) {
          if (prof) t0 = clock64();
          if (!FACT_SKIP(p, 1) && !wait_all(full_bar(stage), phase)) {
            ok = false;
            break;
          }
          if (prof) {
            const long long now = clock64();
            prof_full_wait += now - t0;
            if (prof_first_full == 0) prof_first_full = now - t_go;
          }
          ptx::tc_fence_after();
          const uint32_t sa = smem_base + (uint32_t)stage * p.stage_bytes;
          const uint32_t sb = sa + kStageBytesA;
          const uint64_t adesc = p.a_desc | (uint64_t)((sa >> 4) & 0x3fffu);
          const uint64_t bdesc = p.b_desc | (uint64_t)((sb >> 4) & 0x3fffu);
          if (ptx::elect_one()) {
            if (!FACT_SKIP(p, 2)) {
#pragma unroll
              for (int k = 0; k < kTileK / kUmmaK; ++k) {
                if constexpr (kFp8)
                  ptx::umma_f8<CG>(d_tmem, adesc + (uint64_t)(k * p.a_k_step), bdesc + (uint64_t)(k * p.b_k_step),
                                   p.idesc, (kb > w.kb_begin || k > 0) ? 1u : 0u);
                else
                  ptx::umma_bf16<CG>(d_tmem, adesc + (uint64_t)(k * p.a_k_step), bdesc + (uint64_t)(k * p.b_k_step),
                                     p.idesc, (kb > w.kb_begin || k > 0) ? 1u : 0u);
              }
            }
            // release the stage (in both CTAs of a pair) once these MMAs have read it
            if constexpr (CG == 2) ptx::umma_commit_pair(empty_bar(stage));
            else ptx::umma_commit<CG>(empty_bar(stage));
          }
          if (++stage == p.stages) {
            stage = 0;
            phase ^= 1u;
          }
        }
        if (!ok) break;
        if (ptx::elect_one()) {
          if constexpr (CG == 2) ptx::umma_commit_pair(accf_bar(acc));
          else ptx::umma_commit<CG>(accf_bar(acc));
        }
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1u;
      }
      if (prof && lane == 0) {
        long long* c = reinterpret_cast<long long*>(p.status + 2);
        c[2] = prof_acc_wait;
        c[3] = prof_full_wait;
        c[7] = prof_first_full;  // cycles from "may touch global memory" to the first operand stage being ready
      }
    };
    if (cta_rank == 0) {
      if (p.fp8) issue_all(FactTrue{});
      else issue_all(FactFalse{});
    } else if constexpr (DYN) {
      // the peer's MMA warp issues nothing, but it is one of the warps the scheduler counts: it walks the list
      UnitWalk<SK, GROUPED, DYN, CG> walk(p, unit0, unit_stride, sched);
      WorkUnit w;
      while (walk.next(p, w)) {
      }
    }
    __syncwarp();
  } else if (DYN && warp == kThreads / 32) {
    // ------------------------------------------------------------ dynamic tile scheduler (twelfth warp, DYN only)
    // Obtains the CTA group's further units by cancelling the launch of clusters of this grid that have not started:
    // the group then owes that cluster's tile.  One request is always in flight ahead of the consumers, so the next
    // unit is known before the current tile ends.  The first answer that says "nothing left" is published as -1 and
    // ends every walk; no request follows it.
    if (cta_rank == 0) {
      int slot = 0;
      uint32_t phase = 0;
      for (bool more = true; more;) {
        if (!wait_all(unit_empty_bar(slot), phase ^ 1u)) break;  // every walking warp has read the slot's last value
        const uint32_t resp = sched_base + kSchedRespOff + 16u * (uint32_t)slot;
        if (ptx::elect_one()) {
          ptx::mbar_arrive_expect_tx(clc_bar(slot), 16);
          ptx::clc_try_cancel(resp, clc_bar(slot));
        }
        if (!wait_all(clc_bar(slot), phase)) break;
        int unit = -1;
        if (lane == 0) {
          const int x = ptx::clc_query_ctaid_x(resp);
          unit = x < 0 ? -1 : x / CG;
          ptx::fence_proxy_async_smem();  // the answer was written through the async proxy and will be again
          asm volatile("st.shared.s32 [%0], %1;" ::"r"(sched_base + kSchedUnitOff + 4u * (uint32_t)slot), "r"(unit)
                       : "memory");
        }
        unit = __shfl_sync(0xffffffffu, unit, 0);
        __syncwarp();
        if (lane == 0) {
          ptx::mbar_arrive(unit_full_bar(slot));
          if constexpr (CG == 2) ptx::mbar_arrive_cluster(ptx::mapa(unit_full_bar(slot), 1));  // (release, cluster scope)
        }
        more = unit >= 0;
        if (++slot == kSchedDepth) {
          slot = 0;
          phase ^= 1u;
        }
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------ epilogue warps (2..5 and 7..10)
    // Two warps share each TMEM lane quarter; they take alternate 128-byte column chunks of the tile.
    const int q = warp & 3;                            // the TMEM lane quarter this warp may read
    const int half = warp >= kEpiSetBWarp0 ? 1 : 0;    // which of the two warps of the quarter
    const int e = half * 4 + q;                        // this warp's staging slot
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    // FP8 operands: the accumulator times alpha (the product of the operands' scales), before anything else.  Not for
    // the split-K partial store: there the reduction applies it to the sum.
    const bool scale_acc = p.use_alpha != 0 && EPI != kEpiPartial;
    const float alpha = p.alpha;
    auto scale32 = [&](uint32_t (&v)[32]) {
#pragma unroll
      for (int i = 0; i < 32; ++i) v[i] = __float_as_uint(__uint_as_float(v[i]) * alpha);
    };
    if (p.store_tma) {
      // ---- staged: registers -> swizzled shared memory -> TMA tensor store, 32 rows x 128 bytes at a time
      const int bufs = p.epi_bufs;
      const uint32_t stg0 = epi_base + (uint32_t)(e * bufs) * kEpiBufBytes;
      const uint32_t bias_s = bias_base + (uint32_t)e * kEpiBiasBytes;
      const bool f32 = (EPI == kEpiPartial) || (p.out_f32 != 0);
      const int chunk_cols = f32 ? 32 : 64;               // 128 bytes of output per row
      const bool use_r = (EPI == kEpiBiasResidual) && p.r_tma;
      const uint32_t my_row = (uint32_t)lane * 128u;      // this thread's row inside a staging buffer
      const uint32_t swz = (uint32_t)(lane & 7);          // 128-byte swizzle: 16-byte chunk j lives at j ^ (row & 7)
      long long prof_epi_busy = 0, prof_epi_wait = 0, prof_tiles = 0;
      uint32_t gc = 0;      // chunks this warp has stored so far: buffer = gc % bufs
      uint32_t r_next = 0;  // residual loads have been issued for every chunk counter below this
      UnitWalk<SK, GROUPED, DYN, CG> walk(p, unit0, unit_stride, sched);
      WorkUnit w;
      // hand the accumulator back to the MMA issuer (of the leader CTA) and move on to the other one
      // (a relaxed arrival: the barrier orders tensor-memory reads only, which the tcgen05 fences take care of; a
      // cluster-scope release here waited for the TMA stores in flight, 2500-3600 cycles per tile)
      auto release_acc = [&]() {
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          if constexpr (CG == 2) ptx::mbar_arrive_cluster_relaxed(ptx::mapa(acce_bar(acc), 0));
          else ptx::mbar_arrive(acce_bar(acc));
        }
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1u;
      };
      // stream-K scratch: this CTA's partial tile and the flags of its epilogue warps
      constexpr int kSkPieceF4 = 8 * kTileM;  // float4 words of one 32-column piece of a CTA's 128 accumulator rows
      const int sk_pieces = p.tile_n >> 5;
      float4* const sk_ws4 = reinterpret_cast<float4*>(p.sk_ws);
      while (ok && walk.next(p, w)) {
        if constexpr (SK) {
          if (w.sk_role == 2) {
            // ---- a later piece of a tile another group finishes: park the raw FP32 accumulator in this CTA's
            // scratch tile.  Layout [piece][16-byte word j of the thread's 32 columns][row]: consecutive lanes
            // write consecutive 16-byte words, and the finishing warp reads them back the same way.
            if (!wait_all(accf_bar(acc), acc_phase)) {  // (a warp-uniform verdict: what follows is warp-wide)
              ok = false;
              break;
            }
            ptx::tc_fence_after();
            const uint32_t t_acc = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * p.tile_n);
            float4* const mine = sk_ws4 + (size_t)blockIdx.x * (size_t)(sk_pieces * kSkPieceF4) + (q * 32 + lane);
            for (int pc = half; pc < sk_pieces; pc += 2) {
              uint32_t v[32];
              ptx::tmem_ld_32x32b_x32(t_acc + (uint32_t)(pc * 32), v);
              ptx::tmem_wait_ld();
              float4* dst = mine + (size_t)pc * kSkPieceF4;
#pragma unroll
              for (int j = 0; j < 8; ++j)
                __stcg(dst + j * kTileM, make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]),
                                                     __uint_as_float(v[4 * j + 2]), __uint_as_float(v[4 * j + 3])));
            }
            release_acc();  // (contains the __syncwarp that orders every lane's stores before lane 0's fence)
            if (lane == 0) {
              __threadfence();
              ptx::st_release_gpu(p.sk_flags + (size_t)blockIdx.x * kEpiWarps + e, 1);
            }
            continue;
          }
        }
        const int row0 = (GROUPED ? w.m_base : 0) + (w.tm * CG + (int)cta_rank) * kTileM + q * 32;
        const int n_tile0 = w.tn * p.out_cols;
        const int acc_cols = (EPI == kEpiPartial) ? p.tile_n : p.out_cols;
        const int n_chunks = acc_cols / chunk_cols;
        // The coordinates of chunk `ci`: first column, plane / batch coordinate, whether it exists.
        auto chunk_coord = [&](int ci, int& n, int& z) -> bool {
          const int c = ci * chunk_cols;
          if (EPI == kEpiPartial) {
            int plane = 0;
            if (p.gate) {
              const int hw = p.tile_n >> 1;
              plane = c >= hw;
              n = w.tn * hw + (c - plane * hw);
            } else {
              n = w.tn * p.tile_n + c;
            }
            z = (w.split * p.batch + w.b) * p.ws_planes + plane;
          } else {
            n = n_tile0 + c;
            z = GROUPED ? 0 : w.b;  // (grouped: w.b selects the weights; the rows of C and R are one matrix)
          }
          return ci < n_chunks && n < p.N_out;
        };
        // Start the TMA load of the residual tile of chunk `ci` into the buffer of chunk counter `g`.
        auto issue_residual = [&](int ci, uint32_t g, bool newest_store_too = false) -> bool {
          int n, z;
          if (!chunk_coord(ci, n, z)) return false;
          if (lane == 0) {
            // the store that last read this buffer must be done with it (with two buffers that is the store before
            // the newest one, unless the caller is about to fill the newest store's buffer)
            if (bufs == 1 || newest_store_too) ptx::bulk_wait_group_read<0>();
            else ptx::bulk_wait_group_read<1>();
            const uint32_t rb = res_bar(e, (int)(g % bufs));
            ptx::mbar_arrive_expect_tx(rb, kEpiBufBytes);
            ptx::tma_load_3d(stg0 + (g % bufs) * kEpiBufBytes, &tmR, rb, n, row0, z);
          }
          return true;
        };
        // rows of A normalised over K: this thread's row scale (and scale times mean) come from the partial sums the
        // producing call left, and the column sums of the folded weights for the warp's own 128 columns go to the
        // warp's slice of shared memory (lane l fetches local columns 4l .. 4l+3).  Every load is issued here, ahead
        // of the bias loads below, so that one trip to L2 serves them all; their values are used further down.
        float nrm_rs = 1.f, nrm_rm = 0.f;
        const uint32_t nrm_cs_s = norm_cs_base + (uint32_t)e * 512u;  // this warp's slice of the column sums
        constexpr int kHeldSlots = 16;  // K <= 1024: the partial sums wait in registers until the accumulator is there
        float2 nrm_held[kHeldSlots];
        float nrm_s1 = 0.f, nrm_s2 = 0.f;
        float4 nrm_cs4 = make_float4(0.f, 0.f, 0.f, 0.f);
        if (EXT == 2 && p.norm_mode != 0) {
          const int row = row0 + lane;
          const int slots = (p.K + 63) >> 6;
          const float2* src = p.stats_in + min(row, p.M - 1);  // (rows past M compute a scale nobody stores)
          if (p.norm_mode == 1) {
            const int local = lane * 4;
            const int ci = 2 * (local / chunk_cols) + half;
            const int nc = n_tile0 + ci * chunk_cols + (local % chunk_cols);
            if (ci < n_chunks && nc < p.N_out) nrm_cs4 = __ldg(reinterpret_cast<const float4*>(p.colsum + nc));
          }
          if (slots <= kHeldSlots) {
            // a short main loop leaves these warps no idle time: the sums are added up only after the wait for the
            // accumulator
#pragma unroll
            for (int u = 0; u < kHeldSlots; ++u)
              nrm_held[u] = u < slots ? __ldg(src + (size_t)u * (size_t)p.M) : make_float2(0.f, 0.f);
          } else {
            for (int s = 0; s < slots; ++s) {
              const float2 t = __ldg(src + (size_t)s * (size_t)p.M);
              nrm_s1 += t.x;
              nrm_s2 += t.y;
            }
          }
        }
        // the bias values of this warp's own chunks, as BF16, into the warp's shared-memory slice
        if constexpr (epi_has_bias<EPI>()) {
          __syncwarp();
          if (lane < 16) {
            const int local = lane * 8;                      // index among the warp's 128 columns
            const int ci = 2 * (local / chunk_cols) + half;  // the chunk that column belongs to
            const int nb = n_tile0 + ci * chunk_cols + (local % chunk_cols);
            float bv[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
            if (p.bias != nullptr && ci < n_chunks && nb < p.N_out)
              load_bf16x8(p.bias + nb, min(8, p.N_out - nb), p.bias_vec != 0, bv);
            ptx::st_shared_v4(bias_s + (uint32_t)lane * 16u, pack_bf16x2(bv[0], bv[1]), pack_bf16x2(bv[2], bv[3]),
                              pack_bf16x2(bv[4], bv[5]), pack_bf16x2(bv[6], bv[7]));
          }
          __syncwarp();
        }
        if (EXT == 2 && p.norm_mode == 1) {
          __syncwarp();  // the previous tile's reads of the slice are done
          ptx::st_shared_v4(nrm_cs_s + (uint32_t)lane * 16u, __float_as_uint(nrm_cs4.x), __float_as_uint(nrm_cs4.y),
                            __float_as_uint(nrm_cs4.z), __float_as_uint(nrm_cs4.w));
          __syncwarp();
        }
        if (use_r && r_next <= gc && issue_residual(half, gc)) r_next = gc + 1;
        // with two buffers the residual tile of this warp's second chunk starts now as well (the stores that last read
        // the buffers are a whole main loop old): a load issued only after the first chunk's store leaves most of its
        // latency exposed, 3000 cycles per tile on the 768 -> 768 projection
        if (use_r && bufs == 2 && r_next == gc + 1 && issue_residual(half + 2, gc + 1, true)) r_next = gc + 2;
        auto norm_finish = [&]() {
          if (((p.K + 63) >> 6) <= kHeldSlots) {
#pragma unroll
            for (int u = 0; u < kHeldSlots; ++u) {
              nrm_s1 += nrm_held[u].x;
              nrm_s2 += nrm_held[u].y;
            }
          }
          const float inv_k = 1.f / (float)p.K;
          const float mean = p.norm_mode == 1 ? nrm_s1 * inv_k : 0.f;
          nrm_rs = rsqrtf(fmaxf(nrm_s2 * inv_k - mean * mean, 0.f) + p.norm_eps);
          nrm_rm = nrm_rs * mean;
        };
        // v <- rstd * v - rstd * mean * colsum  (LayerNorm) or rstd * v (RMSNorm), for the 32 accumulator columns
        // whose index among the warp's 128 columns starts at local0 (a multiple of 32)
        auto norm32 = [&](uint32_t (&v)[32], int local0) {
          const uint64_t rs2 = ptx::pack_f32x2(__float_as_uint(nrm_rs), __float_as_uint(nrm_rs));
          if (p.norm_mode == 1) {
            const uint64_t rm2 = ptx::pack_f32x2(__float_as_uint(-nrm_rm), __float_as_uint(-nrm_rm));
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const uint4 c = ptx::ld_shared_v4(nrm_cs_s + (uint32_t)(local0 + 4 * j) * 4u);  // a broadcast read
              const uint64_t t0 = ptx::mul_f32x2(rm2, ptx::pack_f32x2(c.x, c.y));
              const uint64_t t1 = ptx::mul_f32x2(rm2, ptx::pack_f32x2(c.z, c.w));
              ptx::unpack_f32x2(ptx::fma_f32x2(rs2, ptx::pack_f32x2(v[4 * j], v[4 * j + 1]), t0), v[4 * j], v[4 * j + 1]);
              ptx::unpack_f32x2(ptx::fma_f32x2(rs2, ptx::pack_f32x2(v[4 * j + 2], v[4 * j + 3]), t1), v[4 * j + 2],
                                v[4 * j + 3]);
            }
          } else {
#pragma unroll
            for (int i = 0; i < 32; i += 2)
              ptx::unpack_f32x2(ptx::mul_f32x2(rs2, ptx::pack_f32x2(v[i], v[i + 1])), v[i], v[i + 1]);
          }
        };
        long long tw = prof ? clock64() : 0;
        if (!wait_all(accf_bar(acc), acc_phase)) {  // (a warp-uniform verdict: what follows is warp-wide)
          ok = false;
          break;
        }
        const long long tb = prof ? clock64() : 0;
        if (prof) prof_epi_wait += tb - tw;
        ptx::tc_fence_after();
        const uint32_t t_acc = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * p.tile_n);
        if (EXT == 2 && p.norm_mode != 0) norm_finish();
        if constexpr (SK) {
          // the first piece of a tile: the same warp of the same CTA rank in each of the following groups parks
          // the rest of the sum; wait until those are complete (they precede everything else those groups do)
          if (w.sk_role == 1) {
            int good = 1;
            if (lane == 0) {
              for (int pe = 1; pe <= w.sk_peers && good; ++pe)
                good = wait_flag(p.sk_flags + (size_t)(blockIdx.x + CG * pe) * kEpiWarps + e, 1, abort_p, p.status);
            }
            if (!__shfl_sync(0xffffffffu, good, 0)) {
              ok = false;
              break;
            }
          }
        }
        // add the parked partials of accumulator columns [col, col + 32) to v, in group order
        auto add_peers = [&](uint32_t (&v)[32], int col) {
          if constexpr (SK) {
            if (w.sk_role != 1) return;
            for (int pe = 1; pe <= w.sk_peers; ++pe) {
              const float4* src = sk_ws4 + (size_t)(blockIdx.x + CG * pe) * (size_t)(sk_pieces * kSkPieceF4) +
                                  (size_t)(col >> 5) * kSkPieceF4 + (q * 32 + lane);
#pragma unroll
              for (int j0 = 0; j0 < 8; j0 += 4) {  // four 16-byte loads in flight per thread
                float4 t[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) t[j] = __ldcg(src + (j0 + j) * kTileM);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                  const int o = 4 * (j0 + j);
                  v[o] = __float_as_uint(__uint_as_float(v[o]) + t[j].x);
                  v[o + 1] = __float_as_uint(__uint_as_float(v[o + 1]) + t[j].y);
                  v[o + 2] = __float_as_uint(__uint_as_float(v[o + 2]) + t[j].z);
                  v[o + 3] = __float_as_uint(__uint_as_float(v[o + 3]) + t[j].w);
                }
              }
            }
          }
        };
        for (int ci = half; ci < n_chunks; ci += 2) {
          int n_chunk, z;
          if (!chunk_coord(ci, n_chunk, z)) continue;  // uniform across the warp
          const uint32_t buf = stg0 + (gc % bufs) * kEpiBufBytes;
          const int c0 = ci * chunk_cols;  // first accumulator column of the chunk
          const int pieces = chunk_cols / 32;
          // Start the TMEM loads; compute the whole chunk into packed registers; only then claim the staging
          // buffer (the TMA store that last read it has had the time of the math to finish) and write it.
          uint32_t v0[32];
          uint32_t v1[32];
          uint32_t outw[32];  // the chunk's 128 bytes per row: 64 BF16 or 32 FP32 values
          ptx::tmem_ld_32x32b_x32(t_acc + (uint32_t)c0, v0);
          if constexpr (EPI == kEpiSiluGate) {
            ptx::tmem_ld_32x32b_x32(t_acc + (uint32_t)(p.out_cols + c0), v1);
          } else {
            if (pieces == 2) ptx::tmem_ld_32x32b_x32(t_acc + (uint32_t)(c0 + 32), v1);
          }
          if (use_r) {
            if (r_next <= gc && issue_residual(ci, gc)) r_next = gc + 1;
            if (!wait_all(res_bar(e, (int)(gc % bufs)), (gc / bufs) & 1u)) {
              ok = false;
              break;
            }
          }
          ptx::tmem_wait_ld();
          add_peers(v0, c0);
          if constexpr (EPI == kEpiSiluGate) add_peers(v1, p.out_cols + c0);
          else if (pieces == 2) add_peers(v1, c0 + 32);
          if (scale_acc) {
            scale32(v0);
            if (EPI == kEpiSiluGate || pieces == 2) scale32(v1);
          }
          if (EXT == 2 && p.norm_mode != 0) {  // (gated: RMSNorm only, the column index is not used)
            norm32(v0, (ci >> 1) * chunk_cols);
            if (EPI == kEpiSiluGate || pieces == 2) norm32(v1, (ci >> 1) * chunk_cols + 32);
          }
          // one 32-column piece: fused operation on packed FP32 pairs, rounding, into outw
          auto do_piece = [&](int piece, const uint32_t (&a)[32], const uint32_t (&up)[32]) {
            const int local0 = (ci >> 1) * chunk_cols + piece * 32;  // index among the warp's 128 columns
#pragma unroll
            for (int g = 0; g < 4; ++g) {
              uint32_t bw[4] = {0u, 0u, 0u, 0u};  // 8 BF16 bias values
              uint32_t rw[4] = {0u, 0u, 0u, 0u};  // 8 BF16 residual values
              if constexpr (epi_has_bias<EPI>()) {
                const uint4 bq = ptx::ld_shared_v4(bias_s + (uint32_t)(local0 + g * 8) * 2u);
                bw[0] = bq.x; bw[1] = bq.y; bw[2] = bq.z; bw[3] = bq.w;
              }
              if constexpr (EPI == kEpiBiasResidual) {
                if (use_r) {
                  const uint32_t j = (uint32_t)(piece * 4 + g);
                  const uint4 rq = ptx::ld_shared_v4(buf + my_row + ((j ^ swz) << 4));
                  rw[0] = rq.x; rw[1] = rq.y; rw[2] = rq.z; rw[3] = rq.w;
                } else {
                  const int row = row0 + lane;
                  const int n = n_chunk + piece * 32 + g * 8;
                  if (row < p.M && n < p.N_out) {
                    float rf[8];
                    load_bf16x8(p.R + (long long)z * p.strideR + (long long)row * p.ldr + n, min(8, p.N_out - n),
                                p.r_vec != 0, rf);
#pragma unroll
                    for (int t = 0; t < 4; ++t) rw[t] = pack_bf16x2(rf[2 * t], rf[2 * t + 1]);  // exact: BF16 values
                  }
                }
              }
#pragma unroll
              for (int t = 0; t < 4; ++t) {
                const uint64_t y2 = epilogue_pair<EPI>(ptx::pack_f32x2(a[g * 8 + 2 * t], a[g * 8 + 2 * t + 1]),
                                                       ptx::pack_f32x2(up[g * 8 + 2 * t], up[g * 8 + 2 * t + 1]),
                                                       ptx::bf16x2_to_f32x2(bw[t]), ptx::bf16x2_to_f32x2(rw[t]));
                uint32_t lo, hi;
                ptx::unpack_f32x2(y2, lo, hi);
                if (f32) {
                  outw[g * 8 + 2 * t] = lo;
                  outw[g * 8 + 2 * t + 1] = hi;
                } else {
                  outw[piece * 16 + g * 4 + t] = pack_bf16x2(__uint_as_float(lo), __uint_as_float(hi));
                }
              }
            }
          };
          if constexpr (EPI == kEpiSiluGate) {
            do_piece(0, v0, v1);
            if (pieces == 2) {
              ptx::tmem_ld_32x32b_x32(t_acc + (uint32_t)(c0 + 32), v0);
              ptx::tmem_ld_32x32b_x32(t_acc + (uint32_t)(p.out_cols + c0 + 32), v1);
              ptx::tmem_wait_ld();
              add_peers(v0, c0 + 32);
              add_peers(v1, p.out_cols + c0 + 32);
              if (scale_acc) {
                scale32(v0);
                scale32(v1);
              }
              if (EXT == 2 && p.norm_mode != 0) {
                norm32(v0, 0);
                norm32(v1, 0);
              }
              do_piece(1, v0, v1);
            }
          } else {
            do_piece(0, v0, v0);
            if (pieces == 2) do_piece(1, v1, v1);
          }
          if ((EXT == 1 || EXT == 2) && p.stats_out != nullptr && !f32) {
            // partial sums of this row's 64 stored values (as rounded), for a normalisation folded into the next product
            uint64_t sum2 = 0ull, sq2 = 0ull;  // (even columns, odd columns)
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              const uint64_t y2 = ptx::bf16x2_to_f32x2(outw[i]);
              sum2 = ptx::add_f32x2(sum2, y2);
              sq2 = ptx::fma_f32x2(y2, y2, sq2);
            }
            uint32_t a0, a1, b0, b1;
            ptx::unpack_f32x2(sum2, a0, a1);
            ptx::unpack_f32x2(sq2, b0, b1);
            const int row = row0 + lane;
            if (row < p.M)
              p.stats_out[(size_t)(n_chunk >> 6) * (size_t)p.M + row] =
                  make_float2(__uint_as_float(a0) + __uint_as_float(a1), __uint_as_float(b0) + __uint_as_float(b1));
          }
          if constexpr (EXT == 3) {
            // The row leaves straight from registers: four 32-byte stores, each a whole sector of its own.  A long
            // main loop hides their scatter (32 rows per instruction), and the 128 KB per tile that staging writes to
            // and reads from shared memory no longer compete with the operand reads of the tensor pipe.
            const int row = row0 + lane;
            if (row < p.M && !FACT_SKIP(p, 4)) {
              uint8_t* dst = reinterpret_cast<uint8_t*>(p.C) +
                             ((long long)z * p.strideC + (long long)row * p.ldc + n_chunk) * (long long)(f32 ? 4 : 2);
              const int e32 = f32 ? 8 : 16;  // elements in 32 bytes (N_out is a multiple of it on this path)
#pragma unroll
              for (int j = 0; j < 4; ++j)
                if (n_chunk + (j + 1) * e32 <= p.N_out) ptx::st_global_v8(dst + 32 * j, &outw[8 * j]);
            }
            if (use_r && bufs == 2 && r_next <= gc + 1 && issue_residual(ci + 2, gc + 1)) r_next = gc + 2;
            ++gc;
            continue;
          }
          if (!use_r) {
            if (lane == 0) {
              if (bufs == 1) ptx::bulk_wait_group_read<0>();
              else ptx::bulk_wait_group_read<1>();
            }
            __syncwarp();
          }
#pragma unroll
          for (int j = 0; j < 8; ++j)
            ptx::st_shared_v4(buf + my_row + (((uint32_t)j ^ swz) << 4), outw[4 * j], outw[4 * j + 1],
                              outw[4 * j + 2], outw[4 * j + 3]);
          ptx::fence_proxy_async_smem();
          __syncwarp();
          if constexpr (GROUPED) {
            // A tensor store would run over the end of the group into the next group's rows: the warp writes the
            // chunk itself, four whole 128-byte rows per instruction (eight lanes a row), rows past the end left out.
            const int rows_left = w.m_end - row0;  // (<= 0: this warp's rows all lie past the group)
            const int piece = lane & 7, rsub = lane >> 3;
            const int elems16 = f32 ? 4 : 8;
            const int col = n_chunk + piece * elems16;
            const bool col_ok = col + elems16 <= p.N_out;  // (N_out is a multiple of 16 bytes on this path)
            uint8_t* const out_b = reinterpret_cast<uint8_t*>(p.C) +
                                   ((long long)row0 * p.ldc + col) * (long long)(f32 ? 4 : 2);
            const long long row_bytes = p.ldc * (long long)(f32 ? 4 : 2);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const int r = 4 * j + rsub;
              const uint4 v = ptx::ld_shared_v4(buf + (uint32_t)r * 128u + ((uint32_t)(piece ^ (r & 7)) << 4));
              if (r < rows_left && col_ok && !FACT_SKIP(p, 4)) *reinterpret_cast<uint4*>(out_b + r * row_bytes) = v;
            }
            ptx::fence_proxy_async_smem();  // (a residual tile may be loaded into this buffer next, by TMA)
            __syncwarp();
          } else {
            if (lane == 0) {
              if (row0 < p.M && !FACT_SKIP(p, 4)) ptx::tma_store_3d(&tmC, buf, n_chunk, row0, z);
              ptx::bulk_commit_group();
            }
          }
          // with two buffers the next residual tile can start now: its buffer's last store is one chunk old
          if (use_r && bufs == 2 && r_next <= gc + 1 && issue_residual(ci + 2, gc + 1)) r_next = gc + 2;
          ++gc;
        }
        if (!ok) break;
        release_acc();
        if constexpr (SK) {
          // the parked partials have been consumed: clear their flags for the next launch (this warp is their
          // only reader; release_acc's __syncwarp put every lane's reads before this)
          if (w.sk_role == 1 && lane == 0)
            for (int pe = 1; pe <= w.sk_peers; ++pe) p.sk_flags[(size_t)(blockIdx.x + CG * pe) * kEpiWarps + e] = 0;
        }
        if (prof) {
          prof_epi_busy += clock64() - tb;
          ++prof_tiles;
        }
      }
      if (prof && e == 0 && lane == 0) {
        long long* c = reinterpret_cast<long long*>(p.status + 2);
        c[4] = prof_epi_busy;
        c[5] = prof_epi_wait;
        c[6] = prof_tiles;
      }
      if (lane == 0) {
        if (EPI == kEpiPartial) {
          ptx::bulk_wait_group<0>();  // the reduction in the tail reads these partials: wait until they are in global
          asm volatile("fence.proxy.async;" ::: "memory");  // memory, and order them before generic-proxy traffic
        } else {
          ptx::bulk_wait_group_read<0>();  // shared memory may go once every store has read it; the writes complete
        }                                  // with the grid
      }
      __syncwarp();
    } else {
      // ---- direct: each thread stores its own row from registers (any alignment, any leading dimension)
      const bool c_vec = p.c_vec != 0;
      uint32_t xch_count = 0;  // exchanges with the other warp of the lane quarter so far (row softmax only)
      UnitWalk<false, GROUPED, DYN, CG> walk(p, unit0, unit_stride, sched);  // (stream-K always stores through the staged path)
      WorkUnit w;
      while (ok && walk.next(p, w)) {
        if (!wait_all(accf_bar(acc), acc_phase)) {  // (a warp-uniform verdict: what follows is warp-wide)
          ok = false;
          break;
        }
        ptx::tc_fence_after();
        const int row = (GROUPED ? w.m_base : 0) + (w.tm * CG + (int)cta_rank) * kTileM + q * 32 + lane;
        const bool row_ok = row < (GROUPED ? w.m_end : p.M);
        const uint32_t t_acc = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * p.tile_n);
        const int n_tile0 = w.tn * p.out_cols;
        const long long off = (GROUPED ? 0LL : (long long)w.b * p.strideC) + (long long)row * p.ldc;
        char* c_row = reinterpret_cast<char*>(p.C) + off * (p.out_f32 ? 4 : 2);
        const __nv_bfloat16* r_row = nullptr;
        if constexpr (EPI == kEpiBiasResidual)
          r_row = p.R + (GROUPED ? 0LL : (long long)w.b * p.strideR) + (long long)row * p.ldr;
        if constexpr (EPI == kEpiBiasSoftmax) {
          // ---- y = softmax(acc + bias) over the whole row (the host made the tile as wide as the row).  The two warps
          // of a lane quarter hold alternate 32-column pieces of every row, so the row maximum and the row sum are
          // each exchanged once through shared memory, with an mbarrier handshake whose wait is bounded like every
          // other.  Three passes over tensor memory (maximum, sum, normalise) instead of 128 live registers.
          const int e_peer = (half ^ 1) * 4 + q;
          const uint32_t my_slots = epi_base + (uint32_t)(e * p.epi_bufs) * kEpiBufBytes;       // 2 x 32 floats
          const uint32_t peer_slots = epi_base + (uint32_t)(e_peer * p.epi_bufs) * kEpiBufBytes;
          auto exchange = [&](float mine, float& theirs) -> bool {
            const uint32_t slot = (xch_count & 1u) * 128u + (uint32_t)lane * 4u;
            asm volatile("st.shared.f32 [%0], %1;" ::"r"(my_slots + slot), "f"(mine) : "memory");
            __syncwarp();
            // (two barriers in turn: the peer may arrive for the next exchange before this warp has seen this one
            // complete, which a single one-bit phase could not tell from "not yet")
            if (lane == 0) ptx::mbar_arrive(res_bar(e_peer, (int)(xch_count & 1u)));
            if (!wait_all(res_bar(e, (int)(xch_count & 1u)), (xch_count >> 1) & 1u)) return false;
            asm volatile("ld.shared.f32 %0, [%1];" : "=f"(theirs) : "r"(peer_slots + slot) : "memory");
            ++xch_count;
            return true;
          };
          // z = alpha * acc + bias of one 32-column piece, columns past the row's end at -inf
          auto load_piece = [&](int c, float (&z)[32]) {
            uint32_t v[32];
            ptx::tmem_ld_32x32b_x32(t_acc + (uint32_t)c, v);
            ptx::tmem_wait_ld();
            if (scale_acc) scale32(v);
#pragma unroll
            for (int g = 0; g < 4; ++g) {
              const int n = c + g * 8;
              float b8[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
              if (p.bias != nullptr && n < p.N_out) load_bf16x8(p.bias + n, min(8, p.N_out - n), p.bias_vec != 0, b8);
#pragma unroll
              for (int j = 0; j < 8; ++j)
                z[g * 8 + j] = (n + j < p.N_out) ? __uint_as_float(v[g * 8 + j]) + b8[j] : -INFINITY;
            }
          };
          float mloc = -INFINITY;
          for (int c = half * 32; c < p.N_out; c += 64) {
            float z[32];
            load_piece(c, z);
#pragma unroll
            for (int i = 0; i < 32; ++i) mloc = fmaxf(mloc, z[i]);
          }
          float mpeer;
          if (!exchange(mloc, mpeer)) {
            ok = false;
            break;
          }
          const float m = fmaxf(mloc, mpeer);  // finite: the row has at least one column and column 0 is in a piece
          float lloc = 0.f;
          for (int c = half * 32; c < p.N_out; c += 64) {
            float z[32];
            load_piece(c, z);
#pragma unroll
            for (int i = 0; i < 32; ++i) lloc += __expf(z[i] - m);
          }
          float lpeer;
          if (!exchange(lloc, lpeer)) {
            ok = false;
            break;
          }
          const float inv = 1.f / (lloc + lpeer);
          for (int c = half * 32; c < p.N_out; c += 64) {
            float z[32];
            load_piece(c, z);
#pragma unroll
            for (int g = 0; g < 4; ++g) {
              const int n = c + g * 8;
              const int nvalid = min(8, p.N_out - n);
              if (nvalid > 0 && row_ok && !FACT_SKIP(p, 4)) {
                float y[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) y[j] = __expf(z[g * 8 + j] - m) * inv;
                if (p.out_f32) store_f32x8(reinterpret_cast<float*>(c_row) + n, y, nvalid, c_vec);
                else store_bf16x8(reinterpret_cast<__nv_bfloat16*>(c_row) + n, y, nvalid, c_vec);
              }
            }
          }
        } else
        for (int c = half * 32; c < p.out_cols; c += 64) {  // the two warps of a quarter alternate 32-column pieces
          const int n0 = n_tile0 + c;
          if (n0 >= p.N_out) break;  // uniform across the warp
          uint32_t v[32];
          uint32_t vu[32];
          ptx::tmem_ld_32x32b_x32(t_acc + (uint32_t)c, v);
          if constexpr (EPI == kEpiSiluGate) ptx::tmem_ld_32x32b_x32(t_acc + (uint32_t)(p.out_cols + c), vu);
          ptx::tmem_wait_ld();
          if (scale_acc) {
            scale32(v);
            if (EPI == kEpiSiluGate) scale32(vu);
          }
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            const int n = n0 + g * 8;
            const int nvalid = min(8, p.N_out - n);
            float bias[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
            float res[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
            float y[8];
            if (nvalid > 0) {
              if constexpr (epi_has_bias<EPI>()) {
                if (p.bias != nullptr) load_bf16x8(p.bias + n, nvalid, p.bias_vec != 0, bias);
              }
              if constexpr (EPI == kEpiBiasResidual) {
                if (row_ok) load_bf16x8(r_row + n, nvalid, p.r_vec != 0, res);
              }
              apply_epilogue8<EPI>(&v[g * 8], &vu[g * 8], bias, res, y);
              if (row_ok && !FACT_SKIP(p, 4)) {
                if (p.out_f32) store_f32x8(reinterpret_cast<float*>(c_row) + n, y, nvalid, c_vec);
                else store_bf16x8(reinterpret_cast<__nv_bfloat16*>(c_row) + n, y, nvalid, c_vec);
              }
            }
          }
        }
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          if constexpr (CG == 2) ptx::mbar_arrive_cluster_relaxed(ptx::mapa(acce_bar(acc), 0));
          else ptx::mbar_arrive(acce_bar(acc));
        }
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1u;
      }
    }
  }

  // ------------------------------------------------------------ split-K: reduce in the tail
  if constexpr (EPI == kEpiPartial) {
    if (p.fused_reduce) {
      // Every CTA's partial stores are complete (the epilogue warps waited for their bulk groups).  A
      // grid-wide barrier -- all CTAs are resident: at most one per SM and never more CTAs than SMs --
      // then every thread of the grid reduces its share of the output in ascending slice order.
      __syncthreads();
      volatile int* arrived = p.status + 24;
      int* leaving = p.status + 25;
      if (threadIdx.x == 0) {
        __threadfence();
        atomicAdd(p.status + 24, 1);
        const unsigned long long t0 = ptx::globaltimer_ns();
        while (*arrived < (int)gridDim.x) {
          if (ptx::globaltimer_ns() - t0 > kWaitLimitNs) {  // bounded: give up, flag, skip the reduction
            *abort_p = 1;
            atomicExch(p.status, kDeviceTimeoutCode);
            break;
          }
        }
        __threadfence();
      }
      __syncthreads();
      if (prof && threadIdx.x == 0) reinterpret_cast<long long*>(p.status + 2)[7] = clock64() - t_clk0;
      if (!*abort_p) {
        ReduceParams r;
        r.ws = p.ws;
        r.ws_ld = p.ws_ld;
        r.planes = p.ws_planes;
        r.splits = p.split_k;
        r.M = p.M;
        r.N_out = p.N_out;
        r.batch = p.batch;
        r.epi = p.reduce_epi;
        r.C = p.C;
        r.ldc = p.ldc;
        r.strideC = p.strideC;
        r.out_f32 = p.out_f32;
        r.bias = p.bias;
        r.R = p.R;
        r.ldr = p.ldr;
        r.strideR = p.strideR;
        r.alpha = p.use_alpha ? p.alpha : 1.f;
        // (the quads only: the host sends a product of few slices, which the wide walk serves better, to the
        // stand-alone reduction kernel, and this kernel's tail stays short -- cold, every extra line of code on the
        // way to the reduction is a trip to DRAM: 41 against 37 us for the 256 x 256 x 131072 product)
        reduce_groups(r, (long long)blockIdx.x * blockDim.x + threadIdx.x, (long long)gridDim.x * blockDim.x);
      }
      __syncthreads();
      // the last CTA to leave resets both counters for the next launch
      if (threadIdx.x == 0 && atomicAdd(leaving, 1) == (int)gridDim.x - 1) {
        *arrived = 0;
        *leaving = 0;
        __threadfence();
      }
    }
  }

  // ------------------------------------------------------------ teardown
  // This CTA's work is done: the next kernel of the stream may be scheduled onto the SMs as they are vacated and set
  // itself up while the rest of this grid finishes (it still waits for the whole grid before it touches memory).
  // Said at the start of the kernel instead, the same permission cost the long-K split-K launches 4-12 %
  // (256 x 256 x 524288: 100.7 instead of 89.7 us per launch in a train) and gained nothing elsewhere.
  ptx::grid_launch_dependents();
  if (*abort_p) {
    // a wait expired somewhere: give copies that may still be in flight time to land
    const unsigned long long t0 = ptx::globaltimer_ns();
    while (ptx::globaltimer_ns() - t0 < 200000ull) {
    }
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    long long* stamp = reinterpret_cast<long long*>(p.status + 2);
    stamp[0] = clock64() - t_clk0;
    stamp[1] = (long long)(ptx::globaltimer_ns() - t_ns0);
  }
  if ((p.debug & 256) && threadIdx.x == 0)
    atomicMax(reinterpret_cast<unsigned long long*>(p.status + 42), (unsigned long long)ptx::globaltimer_ns());
  if constexpr (CG == 2) {  // neither CTA may free tensor memory or exit while its peer still uses it
    ptx::cluster_arrive();
    ptx::cluster_wait();
  }
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc<CG>(tmem_base, p.tmem_cols);
  }
}

// Self-test of the give-up path: one warp waits on an mbarrier that nothing will ever complete, with a short
// limit.  The wait expires, the status word receives the timeout code, the kernel returns normally.
__global__ void fact_wait_timeout_selftest_kernel(int* status, unsigned long long limit_ns, int* gave_up) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    ptx::mbar_init(ptx::smem_u32(&bar), 1);
    abort_flag = 0;
    ptx::fence_mbar_init();
  }
  __syncthreads();
  const bool ok = wait_bar(ptx::smem_u32(&bar), 0, &abort_flag, status, limit_ns);
  if (threadIdx.x == 0) *gave_up = ok ? 0 : 1;
}

}  // namespace fact
