// Fused multi-head attention forward for sm_100a: O = softmax(scale * Q K^T + causal mask) V, BF16 in and out,
// FP32 scores / probabilities / accumulation, grouped queries (several query heads share one key/value head).
//
// Persistent kernel: one CTA per SM walks a static list of work items (a tile of 128 query positions of one
// (batch, query head)), heaviest first, and streams each tile's key/value sequence in blocks of 128 keys with the
// online-softmax recurrence (a reference maximum m and row sum l per row; the output accumulator is rescaled by
// 2^(m_old - m_new) only when the block maximum exceeds m by more than 8, so probabilities stay below 2^8 and the
// final division by l removes the stale reference exactly).  All roles run ahead across tile boundaries, so the
// loads, the first product and the Q copy of the next tile overlap the last blocks and the epilogue of this one.
//   warp 8      TMA producer: K and V blocks into two three-stage rings; the next tile's Q into a staging buffer
//   warp 9      issuer of the first products, up to two blocks ahead of the softmax:
//                 Q                    tcgen05.cp from the staging buffer into tensor memory, once per tile
//                 S(g)  = Q K^T        tcgen05.mma, M = 128, N = 128, K = head_dim, A = Q read from tensor memory
//                                      (so the product reads only K from shared memory), into score buffer g & 1,
//                                      once O += P(g-2) V has completed (P(g-2) lived in that buffer)
//   warp 11     issuer of the second products:
//                 O    += P(g) V       tcgen05.mma, M = 128, N = head_dim, K = 128, A = P(g) read from tensor memory
//   warp 10     store warp: a finished tile's O / l from its staging buffer to global memory by TMA
//   warps 0-7   softmax: two threads per query row (warps w and w + 4 share a lane quarter and split the block's
//               keys in halves): tcgen05.ld the scores, mask, maximum (exchanged between the two halves through
//               shared memory), exponentials, row sum; rescale O in tensor memory when needed; tcgen05.st the BF16
//               probabilities over the first 64 columns of the score buffer they came from.  A finished tile's
//               O is read, released and written (O / l, BF16) to the staging buffer inside the first block of the
//               next tile, between storing that block's probabilities and announcing them, so the last product's
//               latency is never waited for.
// Tensor memory (512 columns): S/P buffer 0 at 0, buffer 1 at 128, O at 256, Q at 384 (two BF16 values per
// column; one buffer is enough because the copy of the next tile's Q follows this tile's last first-product on
// the in-order tensor pipe).  P(g) may overwrite S(g) because both threads of a row have read their scores
// before either stores (the exchange of the maxima orders them), and S(g+2) is issued once O += P(g) V has
// completed.  Every mbarrier wait is bounded, as in the GEMM kernel; the named barriers between the two warps
// of a row are reached unconditionally, also by a warp whose wait gave up.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "gemm_kernel.cuh"
#include "ptx.cuh"

namespace fact {

constexpr int kAttnThreads = 384;   // 12 warps: 0-7 softmax, 8 TMA producer, 9 and 11 MMA issuers, 10 store
constexpr int kAttnBlockQ = 128;    // query rows per tile (= TMEM lanes)
constexpr int kAttnBlockK = 128;    // keys per block
constexpr int kAttnStagesK = 3;     // K ring depth: a K block is wanted one block before its V block
constexpr int kAttnStagesV = 2;     // V ring depth (two: block g's V slot, g & 1, is released when O += P(g) V has completed,
                                    // which is also the event the softmax warps wait for before rescaling O)
constexpr uint32_t kAttnChunkBytes = 128 * 128;  // one 64-column chunk of a 128-row tile, 128-byte rows
constexpr float kAttnRescaleThreshold = 8.f;     // log2 units
// Registers per thread after the warpgroups rebalance (setmaxnreg): the eight softmax warps take what the other four
// give back.  A request for more than the CTA's pool holds would block forever, so the host checks before the
// first launch that the kernel was compiled with at least kAttnRegsAtLaunch registers per thread.
constexpr int kAttnRegsSoftmax = 208;
constexpr int kAttnRegsOther = 80;
constexpr int kAttnRegsAtLaunch = 168;
static_assert(kAttnStagesV == 2, "the softmax warps use V_EMPTY[g & 1] as \"O += P(g) V has completed\"");
static_assert(4 * kAttnRegsOther + 8 * kAttnRegsSoftmax <= 12 * kAttnRegsAtLaunch, "setmaxnreg requests exceed the pool");

struct AttnParams {
  int B, Tq, Tk, Hq, Hkv, D;  // D = 64 or 128
  int causal;
  float scale_log2;           // softmax scale * log2(e)
  int q_tiles;                // ceil(Tq / 128)
  int q_pairs;                // ceil(Tq / 256): the two-tile kernel's unit
  int items;                  // B * Hq * q_tiles (q_pairs) work items, ordered heaviest query tile first
  uint64_t kmajor_desc;       // UMMA descriptor template, K-major 128B-swizzled tiles (K)
  uint64_t v_desc;            // UMMA descriptor template, V as an N-major operand
  uint32_t idesc_s, idesc_pv;
  int* status;                // (debug bits 8 / 16 / 64 / 128 switch off the softmax arithmetic / the K, V loads /
                              // the first / the second product: experiments on where the time goes, results wrong)
                              // [0] error word; with debug bit 256 eight 64-bit counters of the first CTA from [2]:
                              // cycles, nanoseconds, first wait that gave up, cycles warp 0 waited for scores, its
                              // blocks, -, cycles it spent finishing tiles, its tiles
  int debug;
};

// Shared-memory carve-up (dynamic, 1024-byte aligned): K ring | V ring | Q staging | O staging | exchange (2 x 2 x
// 128 floats) | barriers and control words
__host__ __device__ constexpr uint32_t attn_tile_bytes(int D) { return (uint32_t)(D / 64) * kAttnChunkBytes; }
__host__ __device__ constexpr uint32_t attn_smem_bytes(int D) {
  return attn_tile_bytes(D) * (uint32_t)(kAttnStagesK + kAttnStagesV + 2) + 2048u + 24u * 8u + 16u;
}

struct AttnTile {
  int b, h, kvh, t0, nb;
};

template <int HD>  // head_dim: 64 or 128
__global__ void __launch_bounds__(kAttnThreads, 1)
    fact_attention_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                          const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmO,
                          const AttnParams p) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);
  const int lane = threadIdx.x & 31;
  const uint32_t smem_base = ptx::smem_u32(smem_raw);
  if (smem_base & 1023u) {
    if (threadIdx.x == 0) atomicExch(p.status, kDeviceTimeoutCode);
    return;
  }
  const bool prof = (p.debug & 256) && blockIdx.x == 0;
  const long long t_entry = prof ? clock64() : 0;
  const unsigned long long ns_entry = prof ? ptx::globaltimer_ns() : 0ull;
  constexpr uint32_t tile_bytes = attn_tile_bytes(HD);
  const uint32_t k_s0 = smem_base;
  const uint32_t v_s0 = k_s0 + (uint32_t)kAttnStagesK * tile_bytes;
  const uint32_t q_stage = v_s0 + (uint32_t)kAttnStagesV * tile_bytes;
  const uint32_t o_stage = q_stage + tile_bytes;
  const uint32_t xch_off = (uint32_t)(kAttnStagesK + kAttnStagesV + 2) * tile_bytes;  // [parity][half][row] floats
  const uint32_t bar_base = smem_base + xch_off + 2048u;
  const uint32_t ctrl_off = xch_off + 2048u + 24u * 8u;
  float* xch = reinterpret_cast<float*>(smem_raw + xch_off);
  volatile uint32_t* tmem_holder_p = reinterpret_cast<volatile uint32_t*>(smem_raw + ctrl_off);
  volatile int* abort_p = reinterpret_cast<volatile int*>(smem_raw + ctrl_off + 4);
  enum {
    QS_FULL = 0,                      // the staging buffer holds a tile's Q (TMA bytes)
    QS_EMPTY = 1,                     // its copy into tensor memory has completed
    K_FULL = 2,
    V_FULL = K_FULL + kAttnStagesK,
    K_EMPTY = V_FULL + kAttnStagesV,
    V_EMPTY = K_EMPTY + kAttnStagesK,
    S_FULL = V_EMPTY + kAttnStagesV,  // two: one per score buffer
    P_FULL = S_FULL + 2,              // two: a warp may finish block g + 1 before another has finished block g
    O_DONE = P_FULL + 2,              // a tile's last product has completed (the one-bit phase of V_EMPTY cannot tell
                                      // "two products behind" from "done", so the epilogue has its own barrier)
    O_FREE = O_DONE + 1,              // the softmax warps have read a finished tile's O
    O_STAGED = O_FREE + 1,            // ... and written O / l into the staging buffer
    OS_DONE = O_STAGED + 1,           // the store warp's TMA store has read the staging buffer
    N_BARS = OS_DONE + 1
  };
  static_assert(N_BARS <= 24, "barrier area");
  auto bar = [&](int i) { return bar_base + 8u * (uint32_t)i; };

  if (threadIdx.x < N_BARS) {
    const int i = (int)threadIdx.x;
    const bool by_softmax = i == P_FULL || i == P_FULL + 1 || i == O_FREE || i == O_STAGED;
    ptx::mbar_init(bar(i), by_softmax ? 8u : 1u);  // one arrival per softmax warp
    if (i == 0) *abort_p = 0;
    ptx::fence_mbar_init();
  }
  if (warp == 8 && lane == 0) {
    ptx::prefetch_tensormap(&tmQ);
    ptx::prefetch_tensormap(&tmK);
    ptx::prefetch_tensormap(&tmV);
    ptx::prefetch_tensormap(&tmO);
  }
  if (warp == 9) {
    __syncwarp();
    ptx::tmem_alloc<1>(smem_base + ctrl_off, 512);
    ptx::tmem_relinquish<1>();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_holder_p;
  const uint32_t tmem_o = tmem_base + 256u;
  const uint32_t tmem_q = tmem_base + 384u;

  // This CTA's work items: blockIdx.x, blockIdx.x + gridDim.x, ...  Items are numbered with the query tile as
  // the slow index, heaviest first (the late tiles of a causal problem), so every CTA gets a similar mix and
  // neighbouring CTAs work on query heads that share K and V.
  const int n_items = ((int)blockIdx.x < p.items) ? (p.items - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
  const int kv_blocks_all = (p.Tk + kAttnBlockK - 1) / kAttnBlockK;
  const int bh_count = p.B * p.Hq;
  auto tile_of = [&](int n) -> AttnTile {
    const int idx = (int)blockIdx.x + n * (int)gridDim.x;
    const int qr = idx / bh_count;
    const int bh = idx - qr * bh_count;
    const int qt = p.causal ? (p.q_tiles - 1 - qr) : qr;
    AttnTile t;
    t.h = bh % p.Hq;
    t.b = bh / p.Hq;
    t.kvh = t.h / (p.Hq / p.Hkv);
    t.t0 = qt * kAttnBlockQ;
    t.nb = p.causal ? min(kv_blocks_all, qt + 1) : kv_blocks_all;
    return t;
  };
  constexpr int chunks = HD / 64;
  // A wait that is already satisfied costs one try_wait and a vote.  (The abort flag is read only on the slow
  // path: a volatile generic load of shared memory costs about 170 cycles here, which on every wait of the MMA
  // warp was most of its time.)
  auto wait_all = [&](uint32_t br, uint32_t parity) -> bool {
    if (__all_sync(0xffffffffu, ptx::mbar_try_wait(br, parity))) return true;
    const bool okw = __all_sync(0xffffffffu, wait_bar(br, parity, abort_p, p.status)) != 0;
    if (!okw && lane == 0 && (p.debug & 256))  // which wait gave up first: barrier index, warp, CTA
      atomicCAS(reinterpret_cast<unsigned long long*>(p.status + 6), 0ull,
                (unsigned long long)((br - bar_base) / 8u) | ((unsigned long long)warp << 8) |
                    ((unsigned long long)blockIdx.x << 16) | (1ull << 40));
    return okw;
  };

  // The softmax warpgroups take the registers the third warpgroup gives back (see kAttnRegsSoftmax).
  if (warp >= 8) {
    ptx::setmaxnreg_dec<kAttnRegsOther>();
  if (warp == 8) {
    // ------------------------------------------------------------ TMA producer
    auto load_q = [&](int n) {  // tile n's Q into the staging buffer
      const AttnTile t = tile_of(n);
      if (ptx::elect_one()) {
        ptx::mbar_arrive_expect_tx(bar(QS_FULL), tile_bytes);
        for (int c = 0; c < chunks; ++c)
          ptx::tma_load_4d(q_stage + c * kAttnChunkBytes, &tmQ, bar(QS_FULL), c * 64, t.h, t.t0, t.b);
      }
    };
    if (n_items > 0) load_q(0);
    int ks = 0, vs = 0;
    uint32_t kpar = 1, vpar = 1;  // an empty slot's first wait passes
    const bool skip_loads = (p.debug & 16) != 0;  // experiment switch: K and V are loaded once only
    bool ok = true;
    for (int n = 0; ok && n < n_items; ++n) {
      const AttnTile t = tile_of(n);
      for (int j = 0; ok && j < t.nb; ++j) {
        ok = wait_all(bar(K_EMPTY + ks), kpar);
        if (!ok) break;
        if (skip_loads && n + j > 0) {
          if (ptx::elect_one()) ptx::mbar_arrive(bar(K_FULL + ks));
        } else if (ptx::elect_one()) {
          ptx::mbar_arrive_expect_tx(bar(K_FULL + ks), tile_bytes);
          for (int c = 0; c < chunks; ++c)
            ptx::tma_load_4d(k_s0 + ks * tile_bytes + c * kAttnChunkBytes, &tmK, bar(K_FULL + ks), c * 64, t.kvh,
                             j * kAttnBlockK, t.b);
        }
        if (++ks == kAttnStagesK) {
          ks = 0;
          kpar ^= 1u;
        }
        ok = wait_all(bar(V_EMPTY + vs), vpar);
        if (!ok) break;
        if (skip_loads && n + j > 0) {
          if (ptx::elect_one()) ptx::mbar_arrive(bar(V_FULL + vs));
        } else if (ptx::elect_one()) {
          ptx::mbar_arrive_expect_tx(bar(V_FULL + vs), tile_bytes);
          for (int c = 0; c < chunks; ++c)
            ptx::tma_load_4d(v_s0 + vs * tile_bytes + c * kAttnChunkBytes, &tmV, bar(V_FULL + vs), c * 64, t.kvh,
                             j * kAttnBlockK, t.b);
        }
        if (++vs == kAttnStagesV) {
          vs = 0;
          vpar ^= 1u;
        }
        // the next tile's Q follows this tile's first block, once this tile's Q has left the staging buffer
        if (j == 0 && n + 1 < n_items) {
          ok = wait_all(bar(QS_EMPTY), (uint32_t)n & 1u);
          if (ok) load_q(n + 1);
        }
      }
    }
    __syncwarp();
  } else if (warp == 9) {
    // ------------------------------------------------------------ issuer of the first products, S(g) = Q K^T
    // Two warps issue tensor-core work, one per kind of product: the queue behind the issuing thread is shallow,
    // so a single issuer's waits and commits between two batches leave the pipe idle; with two, each one's
    // bookkeeping hides behind the other's batch.  What in-order issue from one thread gave for free is now an
    // explicit wait: S(g) overwrites the buffer that held P(g-2), so it follows the completion of O += P(g-2) V.
    const bool skip_s = (p.debug & 64) != 0;  // experiment switch, 0 in normal use
    int ks = 0;
    uint32_t kpar = 0;
    int g = 0;
    bool ok = true;
    for (int n = 0; ok && n < n_items; ++n) {
      const int nb = tile_of(n).nb;
      // a new tile: its Q from the staging buffer into tensor memory, 16 elements of every row a copy (the copy
      // follows this thread's earlier products, the last readers of the previous tile's Q, on the in-order pipe)
      ok = wait_all(bar(QS_FULL), (uint32_t)n & 1u);
      if (!ok) break;
      ptx::tc_fence_after();
      if (ptx::elect_one()) {
#pragma unroll
        for (int kk = 0; kk < HD / kUmmaK; ++kk) {
          const uint32_t off = (uint32_t)(kk >> 2) * kAttnChunkBytes + (uint32_t)(kk & 3) * 32u;
          ptx::tmem_cp_128x256b(tmem_q + (uint32_t)kk * 8u, p.kmajor_desc | (uint64_t)(((q_stage + off) >> 4) & 0x3fffu));
        }
        ptx::umma_commit<1>(bar(QS_EMPTY));
      }
      for (int j = 0; ok && j < nb; ++j, ++g) {
        ok = wait_all(bar(K_FULL + ks), kpar);
        if (ok && g >= 2) ok = wait_all(bar(V_EMPTY + (g & 1)), (((uint32_t)g >> 1) - 1u) & 1u);  // O += P(g-2) V done
        if (!ok) break;
        ptx::tc_fence_after();
        if (ptx::elect_one()) {
          const uint32_t kaddr = k_s0 + (uint32_t)ks * tile_bytes;
          const uint32_t d = tmem_base + (uint32_t)(g & 1) * 128u;
          // (shared-memory addresses stay below 2^18, so adding an offset never carries out of the 14-bit field)
          const uint64_t kdesc0 = p.kmajor_desc | (uint64_t)((kaddr >> 4) & 0x3fffu);
#pragma unroll
          for (int kk = 0; kk < HD / kUmmaK; ++kk) {  // 16 elements of head_dim: 8 columns of Q, 32 bytes of a K row
            const uint32_t off = (uint32_t)(kk >> 2) * kAttnChunkBytes + (uint32_t)(kk & 3) * 32u;
            if (!skip_s) ptx::umma_bf16_ts(d, tmem_q + (uint32_t)kk * 8u, kdesc0 + (uint64_t)(off >> 4), p.idesc_s, kk > 0 ? 1u : 0u);
          }
          ptx::umma_commit<1>(bar(S_FULL + (g & 1)));
          ptx::umma_commit<1>(bar(K_EMPTY + ks));
        }
        if (++ks == kAttnStagesK) {
          ks = 0;
          kpar ^= 1u;
        }
      }
    }
    __syncwarp();
  } else if (warp == 11) {
    // ------------------------------------------------------------ issuer of the second products, O += P(g) V
    const bool skip_pv = (p.debug & 128) != 0;  // experiment switch, 0 in normal use
    int g = 0;
    bool ok = true;
    for (int n = 0; ok && n < n_items; ++n) {
      const int nb = tile_of(n).nb;
      for (int j = 0; ok && j < nb; ++j, ++g) {
        const int vs = g & 1;
        ok = wait_all(bar(P_FULL + vs), ((uint32_t)g >> 1) & 1u);
        // the first block of a tile overwrites O: the previous tile's epilogue must have read it
        if (ok && j == 0 && n > 0) ok = wait_all(bar(O_FREE), (uint32_t)(n - 1) & 1u);
        if (ok) ok = wait_all(bar(V_FULL + vs), ((uint32_t)g >> 1) & 1u);
        if (!ok) break;
        ptx::tc_fence_after();
        if (ptx::elect_one()) {
          const uint32_t vaddr = v_s0 + (uint32_t)vs * tile_bytes;
          const uint32_t p_t = tmem_base + (uint32_t)vs * 128u;  // BF16 pairs: 8 columns per 16 keys
          const uint64_t vdesc0 = p.v_desc | (uint64_t)((vaddr >> 4) & 0x3fffu);
#pragma unroll
          for (int kk = 0; kk < kAttnBlockK / kUmmaK; ++kk)  // 16 keys = 2048 bytes further on in V, 8 columns in P
            if (!skip_pv)
              ptx::umma_bf16_ts(tmem_o, p_t + (uint32_t)kk * 8u, vdesc0 + (uint64_t)(kk * 128), p.idesc_pv,
                                (j > 0 || kk > 0) ? 1u : 0u);
          ptx::umma_commit<1>(bar(V_EMPTY + vs));
          if (j == nb - 1) ptx::umma_commit<1>(bar(O_DONE));
        }
      }
    }
    __syncwarp();
  } else if (warp == 10) {
    // ------------------------------------------------------------ store warp: staged O tiles -> global by TMA
    bool ok = true;
    for (int n = 0; ok && n < n_items; ++n) {
      ok = wait_all(bar(O_STAGED), (uint32_t)n & 1u);
      if (!ok) break;
      const AttnTile t = tile_of(n);
      if (lane == 0) {  // bulk groups belong to the issuing thread
        for (int c = 0; c < chunks; ++c) ptx::tma_store_4d(&tmO, o_stage + c * kAttnChunkBytes, c * 64, t.h, t.t0, t.b);
        ptx::bulk_commit_group();
        ptx::bulk_wait_group_read<0>();  // the staging buffer may be rewritten
        ptx::mbar_arrive(bar(OS_DONE));
      }
      __syncwarp();
    }
    if (lane == 0) ptx::bulk_wait_group<0>();  // every store has reached global memory before the CTA exits
    __syncwarp();
  }
  } else {
    ptx::setmaxnreg_inc<kAttnRegsSoftmax>();
    // ------------------------------------------------------------ softmax warps: two threads per query row
    const int half = warp >> 2;        // which 64 keys of every block this thread owns
    const int q4 = warp & 3;           // the TMEM lane quarter this warp may access
    const int row = q4 * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(q4 * 32) << 16;
    const uint32_t pair_bar = 1u + (uint32_t)q4;  // named barrier of this warp and its partner (warp +- 4)
    constexpr int o_cols = HD / 2;                // output columns this thread rescales and stores
    const uint32_t o_addr = tmem_o + lane_addr + (uint32_t)(half * o_cols);
    bool ok = true;  // warp-uniform; a warp whose wait gave up keeps meeting its partner at the named barriers
    long long prof_s_wait = 0, prof_epi = 0, prof_blocks = 0;
    // A finished tile whose output has not been stored yet: this thread's part of the row sums and the tile's ordinal.
    bool pend = false;
    float pend_l = 0.f;
    int pend_n = 0;
    // O / l of the pending tile -> staging buffer -> (store warp) global.  The row sum is the sum of the two
    // halves', exchanged through the buffer `xbuf` that the latest exchange of maxima did not use; the second
    // barrier keeps the next block's maxima from overwriting a sum not yet read.  O is read into registers and
    // released first, so the next tile's products may overwrite it.
    auto finish_tile = [&](int xbuf) {
      const long long te0 = prof ? clock64() : 0;
      pend = false;
      float* xl = xch + xbuf * 256;
      xl[half * 128 + row] = pend_l;
      ptx::named_bar_sync(pair_bar, 64);
      const float lsum = pend_l + xl[(half ^ 1) * 128 + row];
      ptx::named_bar_sync(pair_bar, 64);
      if (ok) ok = wait_all(bar(O_DONE), (uint32_t)pend_n & 1u);
      if (!ok) return;
      ptx::tc_fence_after();
      uint32_t o[2][32];
      ptx::tmem_ld_32x32b_x32(o_addr, o[0]);
      if (o_cols > 32) ptx::tmem_ld_32x32b_x32(o_addr + 32u, o[1]);
      ptx::tmem_wait_ld();
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(bar(O_FREE));
      // O / l as BF16 into the staging tile (128-byte rows of 64 columns, 16-byte pieces swizzled by the row like
      // every other tile here), once the store of the tile before has read it
      if (pend_n > 0) ok = wait_all(bar(OS_DONE), (uint32_t)(pend_n - 1) & 1u);
      if (!ok) return;
      {
        const float inv = (lsum > 0.f) ? __fdividef(1.f, lsum) : 0.f;
        const int col0 = half * o_cols;  // this thread's first output column
        const uint32_t dst = o_stage + (uint32_t)(col0 >> 6) * kAttnChunkBytes + (uint32_t)row * 128u;
        const uint32_t piece0 = (uint32_t)(col0 & 63) >> 3;
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          if (c * 32 < o_cols) {
#pragma unroll
            for (int gq = 0; gq < 4; ++gq) {
              const uint32_t piece = piece0 + (uint32_t)(c * 4 + gq);
              ptx::st_shared_v4(
                  dst + ((piece ^ (uint32_t)(row & 7)) << 4),
                  pack_bf16x2(__uint_as_float(o[c][gq * 8 + 0]) * inv, __uint_as_float(o[c][gq * 8 + 1]) * inv),
                  pack_bf16x2(__uint_as_float(o[c][gq * 8 + 2]) * inv, __uint_as_float(o[c][gq * 8 + 3]) * inv),
                  pack_bf16x2(__uint_as_float(o[c][gq * 8 + 4]) * inv, __uint_as_float(o[c][gq * 8 + 5]) * inv),
                  pack_bf16x2(__uint_as_float(o[c][gq * 8 + 6]) * inv, __uint_as_float(o[c][gq * 8 + 7]) * inv));
            }
          }
        }
      }
      ptx::fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(bar(O_STAGED));
      if (prof) prof_epi += clock64() - te0;
    };
    int g = 0;  // global block counter
    for (int n = 0; n < n_items; ++n) {
      const AttnTile tile = tile_of(n);
      const int nb = tile.nb;
      const int t_row = tile.t0 + row;
      float m = -INFINITY;  // reference maximum of scale_log2 * score the exponentials are taken against
      float l = 0.f;        // this thread's part of the running sum of 2^(scale_log2 * score - m)
      for (int j = 0; j < nb; ++j, ++g) {
        const long long tc1 = prof ? clock64() : 0;
        if (ok) ok = wait_all(bar(S_FULL + (g & 1)), ((uint32_t)g >> 1) & 1u);
        if (prof) {
          prof_s_wait += clock64() - tc1;
          ++prof_blocks;
        }
        if (p.debug & 8) {  // experiment switch: no softmax arithmetic, the barrier protocol only
          ptx::named_bar_sync(pair_bar, 64);
          if (j == 0 && pend) finish_tile((g + 1) & 1);
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(bar(P_FULL + (g & 1)));
          continue;
        }
        const uint32_t buf = tmem_base + lane_addr + (uint32_t)(g & 1) * 128u;
        uint32_t sraw[2][32];
        float hm = -INFINITY;
        if (ok) {
          ptx::tc_fence_after();
          ptx::tmem_ld_32x32b_x32(buf + (uint32_t)half * 64u, sraw[0]);
          ptx::tmem_ld_32x32b_x32(buf + (uint32_t)half * 64u + 32u, sraw[1]);
          ptx::tmem_wait_ld();
          // Only the block on the diagonal (or the ragged last one) needs the per-key mask.
          const int key_limit = min(p.Tk, p.causal ? t_row + 1 : p.Tk) - (j * kAttnBlockK + half * 64);
          if (__any_sync(0xffffffffu, key_limit < 64)) {
#pragma unroll
            for (int c = 0; c < 2; ++c)
#pragma unroll
              for (int i = 0; i < 32; ++i)
                if (c * 32 + i >= key_limit) sraw[c][i] = 0xff800000u;  // -inf
          }
          // four independent chains of three-input maxima
          float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
          for (int c = 0; c < 2; ++c)
#pragma unroll
            for (int i = 0; i < 32; i += 2)
              mx4[(i >> 1) & 3] = ptx::max3(mx4[(i >> 1) & 3], __uint_as_float(sraw[c][i]), __uint_as_float(sraw[c][i + 1]));
          hm = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
        }
        // the row maximum is the larger of the two halves'; passing the barrier also tells each thread that its
        // partner has read its scores, so the probabilities may now overwrite them
        float* xj = xch + (g & 1) * 256;
        xj[half * 128 + row] = hm;
        ptx::named_bar_sync(pair_bar, 64);
        if (!ok) {
          if (j == 0 && pend) finish_tile((g + 1) & 1);  // keeps the pair's barrier sequence identical
          continue;
        }
        const float mx = fmaxf(hm, xj[(half ^ 1) * 128 + row]) * p.scale_log2;  // scale > 0
        // Move the reference maximum only when this block exceeds it by more than the threshold (always from
        // -inf); both threads of a row take the same decision from the same numbers.
        if (__any_sync(0xffffffffu, mx > m + kAttnRescaleThreshold)) {
          const float m_new = fmaxf(m, mx);
          const float alpha = ptx::ex2_approx(m - ((m_new == -INFINITY) ? 0.f : m_new));
          l *= alpha;
          m = m_new;
          if (j > 0) {
            // O is rescaled between O += P(g-1) V, which must have completed, and O += P(g) V, which waits for P(g)
            ok = wait_all(bar(V_EMPTY + ((g - 1) & 1)), ((uint32_t)(g - 1) >> 1) & 1u);
            if (!ok) continue;  // j > 0: no finished tile is pending here
            ptx::tc_fence_after();
            for (int c = 0; c < o_cols; c += 32) {
              uint32_t o[32];
              ptx::tmem_ld_32x32b_x32(o_addr + (uint32_t)c, o);
              ptx::tmem_wait_ld();
#pragma unroll
              for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
              ptx::tmem_st_32x32b_x32(o_addr + (uint32_t)c, o);
            }
          }
        }
        const float m_use = (m == -INFINITY) ? 0.f : m;  // a row with nothing visible yet
        float sum4[4] = {0.f, 0.f, 0.f, 0.f};
        uint32_t pw[32];  // this thread's 64 probabilities as BF16 pairs
#pragma unroll
        for (int c = 0; c < 2; ++c)
#pragma unroll
          for (int i = 0; i < 32; i += 2) {
            // 2^(scale_log2 * s - m): one fused multiply-add and one ex2 per probability
            const float p0 = ptx::ex2_approx(fmaf(__uint_as_float(sraw[c][i]), p.scale_log2, -m_use));
            const float p1 = ptx::ex2_approx(fmaf(__uint_as_float(sraw[c][i + 1]), p.scale_log2, -m_use));
            sum4[(i >> 1) & 3] += p0 + p1;
            pw[c * 16 + (i >> 1)] = pack_bf16x2(p0, p1);
          }
        l += (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
        // P(g) over the first 64 columns of S(g): lane = row, column c holds keys 2c and 2c + 1
        ptx::tmem_st_32x32b_x32(buf + (uint32_t)half * 32u, pw);
        ptx::tmem_wait_st();
        // The previous tile's O: its last product was issued a whole block ago, and the first product that
        // overwrites O waits for the probabilities announced below.
        if (j == 0 && pend) finish_tile((g + 1) & 1);
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(bar(P_FULL + (g & 1)));
      }
      // this tile's output is finished inside the next tile's first block (or after the loop)
      pend = true;
      pend_l = l;
      pend_n = n;
    }
    if (pend) finish_tile(g & 1);
    if (prof && warp == 0 && lane == 0) {
      long long* prof_c = reinterpret_cast<long long*>(p.status + 2);
      prof_c[3] = prof_s_wait;
      prof_c[4] = prof_blocks;
      prof_c[6] = prof_epi;
      prof_c[7] = n_items;
    }
  }

  // ------------------------------------------------------------ teardown
  if (*abort_p) {
    const unsigned long long tw = ptx::globaltimer_ns();
    while (ptx::globaltimer_ns() - tw < 200000ull) {
    }
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (warp == 9) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc<1>(tmem_base, 512);
  }
  if (prof && threadIdx.x == 0) {
    long long* prof_c = reinterpret_cast<long long*>(p.status + 2);
    prof_c[0] = clock64() - t_entry;
    prof_c[1] = (long long)(ptx::globaltimer_ns() - ns_entry);
  }
}

}  // namespace fact
