// K slices of a tile as one thread-block cluster: the slices are added up through distributed shared memory.
//
// For products of few tiles and long K (Section 5.2, Problem 6: the K-sliced / stream-K regime).  A cluster of S CTAs
// (S = 2, 4 or 8) owns one 128 x tile_n output tile at a time; CTA r of the cluster multiplies the r-th slice of K
// with its own TMA ring and its own FP32 accumulator in tensor memory -- the slices share no operand, so nothing is
// loaded twice and every CTA issues only its own plain loads.  When the S accumulators are complete, CTA r sends the
// j-th block of tile_n / S columns of its accumulator to CTA j (vector stores to the peer's shared memory), CTA j adds the
// S blocks it received in a fixed order, applies the epilogue and stores its columns of the tile.  No partial planes
// in global memory, no workspace, no grid-wide barrier: the clusters of a launch do not depend on one another, so
// the grid may be larger than what is resident.
//
// The order of the additions is that of the workspace reduction with the same number of slices (s_q = slices q and
// q + 4, then (s0 + s1) + (s2 + s3)), so the two paths give the same bits.
//
// Warps: 0 TMA producer, 1 MMA issuer, 2-5 exchange and epilogue (one accumulator row per thread).  Every wait is
// bounded; a CTA that gives up still takes part in the cluster barrier at the end, so that no CTA of the cluster
// leaves while a peer may still write to its shared memory.
#pragma once
#include "gemm_kernel.cuh"

namespace fact {

constexpr int kKcThreads = 192;

// What a CTA receives: from each of the S senders its block of tile_n / S columns of 128 rows, kept as
// [sender][group of 4 columns][row] 16-byte pieces -- the 32 lanes of a warp (32 rows) write, and later read, 512
// contiguous bytes per instruction.  (Row-major blocks made every lane's 16 bytes a transaction of its own: 1000-1300
// cycles per 32-column piece sent instead of 300.)
__host__ __device__ constexpr uint32_t kc_exchange_bytes(int tile_n, int slices) {
  return (uint32_t)tile_n * kTileM * 4u + 0u * (uint32_t)slices;
}
__host__ __device__ constexpr uint32_t kc_smem_bytes(int tile_n, int slices, int stages, uint32_t stage_bytes) {
  const uint32_t ring = (uint32_t)stages * stage_bytes, xch = kc_exchange_bytes(tile_n, slices);
  return (ring > xch ? ring : xch) + (2 * kMaxStages + 5) * 8 + 16;
}

__device__ __forceinline__ void st_shared_cluster_v4(uint32_t cluster_addr, uint32_t x, uint32_t y, uint32_t z, uint32_t w) {
  asm volatile("st.shared::cluster.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(cluster_addr), "r"(x), "r"(y), "r"(z), "r"(w)
               : "memory");
}

template <int EPI, int CG>
__global__ void __launch_bounds__(kKcThreads, 1)
    fact_gemm_kcluster_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                              const GemmParams p) {
  static_assert(EPI != kEpiSiluGate && EPI != kEpiBiasSoftmax && EPI != kEpiPartial, "plain column-wise epilogues");
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);
  const int lane = threadIdx.x & 31;
  const uint32_t smem_base = ptx::smem_u32(smem_raw);
  const int S = p.split_k;                      // K slices per tile; the cluster has S CTAs (CG == 1) or S pairs
  const uint32_t rank = ptx::cluster_ctarank();
  const uint32_t half = rank % (uint32_t)CG;     // which CTA of its pair: the first (the leader) issues the pair's products
  const uint32_t kr = rank / (uint32_t)CG;       // the slice of K this CTA (pair) multiplies
  const uint32_t leader = rank - half;
  const int cb = p.tile_n / S;                  // accumulator columns each CTA finishes (a multiple of 32)
  const uint32_t ring_bytes = (uint32_t)p.stages * p.stage_bytes;
  const uint32_t xch_bytes = kc_exchange_bytes(p.tile_n, S);
  const uint32_t bar_base = smem_base + (ring_bytes > xch_bytes ? ring_bytes : xch_bytes);
  const uint32_t ctrl_off = bar_base - smem_base + (2 * kMaxStages + 5) * 8;
  volatile uint32_t* tmem_holder_p = reinterpret_cast<volatile uint32_t*>(smem_raw + ctrl_off);
  volatile int* abort_p = reinterpret_cast<volatile int*>(smem_raw + ctrl_off + 4);
  auto full_bar = [&](int s) { return bar_base + 8u * (uint32_t)s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (uint32_t)(kMaxStages + s); };
  const uint32_t accf_bar = bar_base + 8u * (uint32_t)(2 * kMaxStages);       // this CTA's accumulator is complete
  const uint32_t peers_bar = bar_base + 8u * (uint32_t)(2 * kMaxStages + 1);  // ... and so is every peer's: S arrivals
  const uint32_t xfull_bar = bar_base + 8u * (uint32_t)(2 * kMaxStages + 2);  // all S blocks have arrived: 4 S arrivals
  const uint32_t xdone_bar = bar_base + 8u * (uint32_t)(2 * kMaxStages + 3);  // ... and have been added up: 4 arrivals
  const uint32_t mdone_bar = bar_base + 8u * (uint32_t)(2 * kMaxStages + 4);  // the same for every CTA of the pair (the
                                                                              // leader's products write both): 4 CG
  // A launch this kernel cannot serve is refused by every CTA alike, before any barrier exists.
  const bool refuse = (smem_base & 1023u) || S < 2 || S * CG > 8 || (int)ptx::cluster_nctarank() != S * CG || cb * S != p.tile_n ||
                      (cb & 31) || p.k_base < 1 || p.gate;
  if (refuse) {
    if (threadIdx.x == 0) atomicExch(p.status, kDeviceTimeoutCode);
    return;
  }
  if (threadIdx.x < 2 * kMaxStages + 5) {
    const int i = (int)threadIdx.x;
    uint32_t count = 1;
    if (i == 2 * kMaxStages + 1) count = (uint32_t)S;
    if (i == 2 * kMaxStages + 2) count = 4u * (uint32_t)S;
    if (i == 2 * kMaxStages + 3) count = 4u;
    if (i == 2 * kMaxStages + 4) count = 4u * (uint32_t)CG;
    ptx::mbar_init(bar_base + 8u * (uint32_t)i, count);
    if (i == 0) *abort_p = 0;
    ptx::fence_mbar_init();
  }
  if (warp == 0 && lane == 0) {
    ptx::prefetch_tensormap(&tmA);
    ptx::prefetch_tensormap(&tmB);
  }
  if (warp == 1) {
    __syncwarp();
    ptx::tmem_alloc<CG>(smem_base + ctrl_off, p.tmem_cols);
    ptx::tmem_relinquish<CG>();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::cluster_arrive();  // the peers' barriers must exist before anything arrives on them
  ptx::cluster_wait();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_holder_p;
  ptx::grid_dependency_wait();  // set-up above overlaps the tail of the kernel before; global memory from here on
  // With debug bit 256 the first CTA stamps its first tile's milestones, in SM cycles from here (status[2..17], read by
  // fact_last_kernel_profile): [0] whole kernel, [1] the same in nanoseconds, [2] first operand stage ready,
  // [3] accumulator complete, [4] every peer's complete, [5] blocks sent, [6] blocks received, [7] tile stored.
  const bool prof = (p.debug & 256) && blockIdx.x == 0;
  const long long t_go = clock64();
  const unsigned long long ns_go = prof ? ptx::globaltimer_ns() : 0ull;
  long long* const prof_c = reinterpret_cast<long long*>(p.status + 2);

  const int cluster_id = (int)(blockIdx.x / (unsigned)(S * CG));
  const int n_clusters = (int)(gridDim.x / (unsigned)(S * CG));
  const int tiles = p.total_units / S;  // (units are numbered tile-major, slice-minor)
  auto wait_all = [&](uint32_t bar, uint32_t parity) -> bool {
    return __all_sync(0xffffffffu, wait_bar(bar, parity, abort_p, p.status)) != 0;
  };
  auto wait_all_cluster = [&](uint32_t bar, uint32_t parity) -> bool {  // ... for barriers the peers arrive on
    return __all_sync(0xffffffffu, wait_bar_cluster(bar, parity, abort_p, p.status)) != 0;
  };

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true;
    int it = 0;
    const uint64_t pol = ptx::l2_policy(p.l2_keep_operands);
    for (int tile = cluster_id; ok && tile < tiles; tile += n_clusters, ++it) {
      const WorkUnit w = decode_unit(p, tile * S + (int)kr);
      // the ring doubles as the exchange buffer: the blocks of the tile before must have been added up
      if (it > 0) ok = wait_all(xdone_bar, (uint32_t)(it - 1) & 1u);
      if (!ok) break;
      const int m0 = (w.tm * CG + (int)half) * kTileM;
      const int col0 = (int)half * (p.tile_n / CG);  // a pair's CTAs load one half of the B tile each
      for (int kb = w.kb_begin; kb < w.kb_end; ++kb) {
        if (!wait_all(empty_bar(stage), phase ^ 1u)) {
          ok = false;
          break;
        }
        const uint32_t sa = smem_base + (uint32_t)stage * p.stage_bytes;
        const uint32_t sb = sa + kStageBytesA;
        uint32_t fb = full_bar(stage);
        if (ptx::elect_one()) {
          if (half == 0) ptx::mbar_arrive_expect_tx(fb, p.tx_bytes);  // (the bytes of both CTAs of a pair)
          if constexpr (CG == 2) {
            fb = ptx::mapa(fb, leader);  // both CTAs' loads complete on the leader's barrier
            ptx::tma_load_3d_cg2_hint(sa, &tmA, fb, kb * kTileK, m0, w.b, pol);
          } else {
            ptx::tma_load_3d_hint(sa, &tmA, fb, kb * kTileK, m0, w.b, pol);
          }
#pragma unroll
          for (int i = 0; i < 4; ++i)
            if (i < p.b_loads) {
              const int n = w.tn * p.tile_n + col0 + i * p.b_box_n;
              const uint32_t dst = sb + (uint32_t)i * p.b_box_bytes;
              if constexpr (CG == 2) {
                if (p.b_kn) ptx::tma_load_3d_cg2_hint(dst, &tmB, fb, n, kb * kTileK, w.b, pol);
                else ptx::tma_load_3d_cg2_hint(dst, &tmB, fb, kb * kTileK, n, w.b, pol);
              } else {
                if (p.b_kn) ptx::tma_load_3d_hint(dst, &tmB, fb, n, kb * kTileK, w.b, pol);
                else ptx::tma_load_3d_hint(dst, &tmB, fb, kb * kTileK, n, w.b, pol);
              }
            }
        }
        if (++stage == p.stages) {
          stage = 0;
          phase ^= 1u;
        }
      }
    }
    __syncwarp();
  } else if (warp == 1 && half == 0) {
    // ------------------------------------------------------------ MMA issuer (of the pair's leader)
    auto commit = [&](uint32_t b) {  // to this CTA's barrier and, for a pair, to the peer's at the same offset
      ptx::umma_commit<CG>(b);
      if constexpr (CG == 2) ptx::umma_commit<2>(ptx::mapa(b, rank + 1));
    };
    int stage = 0;
    uint32_t phase = 0;
    bool ok = true;
    int it = 0;
    for (int tile = cluster_id; ok && tile < tiles; tile += n_clusters, ++it) {
      const WorkUnit w = decode_unit(p, tile * S + (int)kr);
      // the accumulators of the tile before must have been read (their blocks are added up only after that)
      if (it > 0) ok = wait_all_cluster(mdone_bar, (uint32_t)(it - 1) & 1u);
      if (!ok) break;
      ptx::tc_fence_after();
      for (int kb = w.kb_begin; kb < w.kb_end; ++kb) {
        if (!wait_all(full_bar(stage), phase)) {
          ok = false;
          break;
        }
        if (prof && it == 0 && kb == w.kb_begin && lane == 0) prof_c[2] = clock64() - t_go;
        ptx::tc_fence_after();
        const uint32_t sa = smem_base + (uint32_t)stage * p.stage_bytes;
        const uint32_t sb = sa + kStageBytesA;
        const uint64_t adesc = p.a_desc | (uint64_t)((sa >> 4) & 0x3fffu);
        const uint64_t bdesc = p.b_desc | (uint64_t)((sb >> 4) & 0x3fffu);
        if (ptx::elect_one()) {
#pragma unroll
          for (int k = 0; k < kTileK / kUmmaK; ++k)
            ptx::umma_bf16<CG>(tmem_base, adesc + (uint64_t)(k * p.a_k_step), bdesc + (uint64_t)(k * p.b_k_step), p.idesc,
                               (kb > w.kb_begin || k > 0) ? 1u : 0u);
          commit(empty_bar(stage));
        }
        if (++stage == p.stages) {
          stage = 0;
          phase ^= 1u;
        }
      }
      if (!ok) break;
      if (ptx::elect_one()) commit(accf_bar);
    }
    __syncwarp();
  } else if (warp >= 2) {
    // ------------------------------------------------------------ exchange and epilogue: one accumulator row per thread
    const int q = warp & 3;  // the TMEM lane quarter this warp may read
    const int row_in_tile = q * 32 + lane;
    const uint32_t chunk_stride = (uint32_t)kTileM * 16u;                   // bytes between two 4-column groups
    const uint32_t block_stride = (uint32_t)(cb >> 2) * chunk_stride;       // ... between the blocks of two senders
    const uint32_t my_slot = smem_base + kr * block_stride + (uint32_t)row_in_tile * 16u;  // where a peer keeps MY block
    const bool c_vec = p.c_vec != 0;
    bool ok = true;
    int it = 0;
    for (int tile = cluster_id; ok && tile < tiles; tile += n_clusters, ++it) {
      const WorkUnit w = decode_unit(p, tile * S + (int)kr);
      const uint32_t par = (uint32_t)it & 1u;
      // ---- this CTA's slice is complete: tell every CTA of the cluster, then wait until all of them are (their
      // rings are then idle and may receive blocks)
      if (!wait_all(accf_bar, par)) {  // (every verdict is warp-uniform: what follows is warp-wide)
        ok = false;
        break;
      }
      ptx::tc_fence_after();
      const bool stamp = prof && it == 0 && warp == 2 && lane == 0;
      if (stamp) prof_c[3] = clock64() - t_go;
      if (warp == 2) {
        // (a relaxed arrival: it publishes no data, it says that this CTA's products have stopped reading its ring,
        // which this thread has just observed through the accumulator's barrier)
        if (lane < S) ptx::mbar_arrive_cluster_relaxed(ptx::mapa(peers_bar, (uint32_t)lane * CG + half));
        __syncwarp();
      }
      if (!wait_all_cluster(peers_bar, par)) {
        ok = false;
        break;
      }
      if (stamp) prof_c[4] = clock64() - t_go;
      // ---- send: 32 accumulator columns at a time, starting with the block of the next CTA round the cluster so
      // that the S senders do not all write to the same receiver at once
      const int pieces = p.tile_n >> 5;
      const int per_owner = cb >> 5;
      auto piece_of = [&](int i) {
        int pc = i + ((int)kr + 1) * per_owner;
        if (pc >= pieces) pc -= pieces;
        if (pc >= pieces) pc -= pieces;  // ((kr + 1) * per_owner may equal pieces)
        return pc;
      };
      const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16);
      auto send = [&](int pc, const uint32_t (&v)[32]) {
        const int owner = pc / per_owner;
        const int col = (pc - owner * per_owner) << 5;  // first column inside the owner's block
        const uint32_t dst = ptx::mapa(my_slot + (uint32_t)(col >> 2) * chunk_stride, (uint32_t)owner * CG + half);
#pragma unroll
        for (int j = 0; j < 8; ++j)
          st_shared_cluster_v4(dst + chunk_stride * (uint32_t)j, v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
      };
      // two pieces per trip: the second piece's tensor-memory load is in flight while the first is sent
      for (int i = 0; i < pieces; i += 2) {
        uint32_t v0[32], v1[32];
        const int pc0 = piece_of(i), pc1 = i + 1 < pieces ? piece_of(i + 1) : 0;
        ptx::tmem_ld_32x32b_x32(t_row + (uint32_t)(pc0 << 5), v0);
        ptx::tmem_wait_ld();
        if (i + 1 < pieces) ptx::tmem_ld_32x32b_x32(t_row + (uint32_t)(pc1 << 5), v1);
        send(pc0, v0);
        if (i + 1 < pieces) {
          ptx::tmem_wait_ld();
          send(pc1, v1);
        }
      }
      ptx::tc_fence_before();
      __syncwarp();  // every lane's stores are ordered before lane 0's releasing arrivals
      if (lane < S) ptx::mbar_arrive_cluster(ptx::mapa(xfull_bar, (uint32_t)lane * CG + half));
      if (stamp) prof_c[5] = clock64() - t_go;
      // ---- receive: add the S blocks of this CTA's columns in the order of the workspace reduction, apply the
      // epilogue, store
      if (!wait_all_cluster(xfull_bar, par)) {
        ok = false;
        break;
      }
      if (stamp) prof_c[6] = clock64() - t_go;
      const int row = (w.tm * CG + (int)half) * kTileM + row_in_tile;
      const bool row_ok = row < p.M;
      const int n_block0 = w.tn * p.tile_n + (int)kr * cb;
      const long long off = (long long)w.b * p.strideC + (long long)row * p.ldc;
      char* c_row = reinterpret_cast<char*>(p.C) + off * (p.out_f32 ? 4 : 2);
      const __nv_bfloat16* r_row = nullptr;
      if constexpr (EPI == kEpiBiasResidual) r_row = p.R + (long long)w.b * p.strideR + (long long)row * p.ldr;
      const uint32_t mine = smem_base + (uint32_t)row_in_tile * 16u;
      for (int c = 0; c < cb; c += 8) {
        const int n = n_block0 + c;
        const int nvalid = min(8, p.N_out - n);
        if (nvalid <= 0) break;  // (columns only grow: nothing further to the right either)
        float acc[4][8];
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
          for (int j = 0; j < 8; ++j) acc[a][j] = 0.f;
#pragma unroll
        for (int s = 0; s < 8; ++s)
          if (s < S) {
            const uint4 lo = ptx::ld_shared_v4(mine + (uint32_t)s * block_stride + (uint32_t)(c >> 2) * chunk_stride);
            const uint4 hi = ptx::ld_shared_v4(mine + (uint32_t)s * block_stride + (uint32_t)((c >> 2) + 1) * chunk_stride);
            const int a = s & 3;
            acc[a][0] += __uint_as_float(lo.x); acc[a][1] += __uint_as_float(lo.y);
            acc[a][2] += __uint_as_float(lo.z); acc[a][3] += __uint_as_float(lo.w);
            acc[a][4] += __uint_as_float(hi.x); acc[a][5] += __uint_as_float(hi.y);
            acc[a][6] += __uint_as_float(hi.z); acc[a][7] += __uint_as_float(hi.w);
          }
        uint32_t tot[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) tot[j] = __float_as_uint((acc[0][j] + acc[1][j]) + (acc[2][j] + acc[3][j]));
        float bias[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        float res[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        float y[8];
        if constexpr (epi_has_bias<EPI>()) {
          if (p.bias != nullptr) load_bf16x8(p.bias + n, nvalid, p.bias_vec != 0, bias);
        }
        if constexpr (EPI == kEpiBiasResidual) {
          if (row_ok) load_bf16x8(r_row + n, nvalid, p.r_vec != 0, res);
        }
        apply_epilogue8<EPI>(tot, tot, bias, res, y);
        if (row_ok) {
          if (p.out_f32) store_f32x8(reinterpret_cast<float*>(c_row) + n, y, nvalid, c_vec);
          else store_bf16x8(reinterpret_cast<__nv_bfloat16*>(c_row) + n, y, nvalid, c_vec);
        }
      }
      // the next tile's operands arrive in this memory through the asynchronous proxy
      ptx::fence_proxy_async_smem();
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        ptx::mbar_arrive(xdone_bar);
        ptx::mbar_arrive_cluster_relaxed(ptx::mapa(mdone_bar, leader));  // (orders tensor-memory reads: the fences do)
      }
      if (stamp) prof_c[7] = clock64() - t_go;
    }
    __syncwarp();
  }

  // ------------------------------------------------------------ teardown
  ptx::grid_launch_dependents();
  if (*abort_p) {  // a wait expired somewhere: give copies that may still be in flight time to land
    const unsigned long long t0 = ptx::globaltimer_ns();
    while (ptx::globaltimer_ns() - t0 < 200000ull) {
    }
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::cluster_arrive();  // no CTA leaves while a peer may still write to its shared memory or arrive on its barriers
  ptx::cluster_wait();
  if (prof && threadIdx.x == 0) {
    prof_c[0] = clock64() - t_go;
    prof_c[1] = (long long)(ptx::globaltimer_ns() - ns_go);
  }
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc<CG>(tmem_base, p.tmem_cols);
  }
}

}  // namespace fact
