// Fused multi-head attention forward for sm_100a, two query tiles per CTA: O = softmax(scale * Q K^T + causal mask) V,
// BF16 in and out, FP32 scores / probabilities / accumulation, grouped queries.
//
// Persistent kernel: one CTA per SM walks a static list of work items, heaviest first.  An item is 256 query
// positions of one (batch, query head), handled as two tiles of 128 rows (0 and 1) that share every key/value
// block the CTA loads.  Each tile is a pipeline of its own -- an MMA-issuing warp and a warpgroup of softmax
// threads, one thread per query row -- so that one tile's loads, maxima and stores fill the gaps the other leaves
// on the special-function units, and both tiles' products share the tensor pipe.  Per block j of BK keys of tile t
// (online softmax: a reference maximum m and row sum l per row; the output accumulator is rescaled by
// 2^(m_old - m_new) only when a block maximum exceeds m by more than 8, so probabilities stay below 2^8 and the
// final division by l removes the stale reference exactly):
//   issuer t     S_t(j) = Q_t K_j^T       tcgen05.mma, M = 128, N = BK, K = head_dim, Q_t and K_j from shared memory
//                O_t   += P_t(j) V_j      tcgen05.mma, M = 128, N = head_dim, K = BK, A = P_t(j) read from tensor memory
//   softmax t    tcgen05.ld the BK scores of its row and say so (S_READ), mask, maximum, exponentials, row sum;
//                rescale O_t in tensor memory when the reference maximum moves; tcgen05.st the BF16 probabilities;
//                after the tile's last block O_t / l -> staging buffer
//   warp 8       TMA producer: Q_0, Q_1 of the next item as soon as their buffers are free; K and V blocks into
//                two four-stage rings (a slot is released by both issuers)
//   warp 10      store warp: staged output tiles to global memory by TMA, tile 0 and tile 1 of an item in turn
// Scores and probabilities have tensor-memory columns of their own, so S_t(j+1) is issued as soon as the softmax
// threads have read S_t(j) -- before they have computed anything -- and the scores of the next block are always
// waiting when a block's probabilities have been stored: the softmax threads never wait for the tensor pipe, and
// the products never wait for anything but the probabilities.  That takes BK/2 + BK + head_dim columns per tile:
// 128 keys per block at head_dim 64, 64 keys at head_dim 128.  (With probabilities written over the scores they
// came from, as tensor memory forces at BK = 128 and head_dim 128, every block is a serial chain softmax ->
// O += P V -> next S -> softmax, and a tile-block takes 1900 cycles instead of the 1100 the exponentials need.)
// In a causal problem tile 0 may see one key block fewer than tile 1; its issuer releases that block's slots unused.
// Every mbarrier wait is bounded, as in the GEMM kernel.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "gemm_kernel.cuh"
#include "ptx.cuh"

namespace fact {

constexpr int kAttnThreads = 384;   // 12 warps: 0-3 softmax of tile 0, 4-7 of tile 1, 8 TMA producer, 9 and 11 MMA issuers, 10 store
constexpr int kAttnBlockQ = 128;    // query rows per tile (= TMEM lanes); a work item is two tiles
constexpr uint32_t kAttnChunkBytes = 128 * 128;  // one 64-column chunk of a 128-row tile, 128-byte rows
constexpr float kAttnRescaleThreshold = 8.f;     // log2 units
// Registers per thread after the warpgroups rebalance (setmaxnreg): the eight softmax warps take what the other four
// give back.  A request for more than the CTA's pool holds would block forever, so the host checks before the
// first launch that the kernel was compiled with at least kAttnRegsAtLaunch registers per thread.
constexpr int kAttnRegsSoftmax = 208;
constexpr int kAttnRegsOther = 80;
constexpr int kAttnRegsAtLaunch = 168;
static_assert(4 * kAttnRegsOther + 8 * kAttnRegsSoftmax <= 12 * kAttnRegsAtLaunch, "setmaxnreg requests exceed the pool");

struct AttnParams {
  int B, Tq, Tk, Hq, Hkv, D;  // D = 64 or 128
  int causal;
  float scale_log2;           // softmax scale * log2(e)
  int q_pairs;                // ceil(Tq / 256)
  int items;                  // B * Hq * q_pairs work items, ordered heaviest first
  uint64_t kmajor_desc;       // UMMA descriptor template, K-major 128B-swizzled tiles (Q, K)
  uint64_t v_desc;            // UMMA descriptor template, V as an N-major operand
  uint32_t idesc_s, idesc_pv;
  int* status;                // [0] error word; with debug bit 256 eight 64-bit counters of the first CTA from [2]:
                              // cycles, nanoseconds, first wait that gave up, cycles the first softmax warp waited for
                              // scores, its blocks, -, cycles it spent writing tiles out, its items
  int debug;                  // experiment switches, 0 in normal use: 8 no softmax arithmetic, 64 / 128 no first /
                              // second products (timing experiments; the output is then meaningless), 256 counters
};

__host__ __device__ constexpr uint32_t attn_tile_bytes(int D) { return (uint32_t)(D / 64) * kAttnChunkBytes; }

constexpr int kAttnStages = 4;  // K ring and V ring depth (a block of either is 16 KB in both configurations)
__host__ __device__ constexpr int attn_block_k(int D) { return D == 64 ? 128 : 64; }

// Shared-memory carve-up (dynamic, 1024-byte aligned): K ring | V ring | Q_0 | Q_1 | O staging | barriers, control
__host__ __device__ constexpr uint32_t attn_kv_bytes(int D) { return (uint32_t)attn_block_k(D) * (uint32_t)D * 2u; }
__host__ __device__ constexpr uint32_t attn_smem_bytes(int D) {
  return attn_kv_bytes(D) * (uint32_t)(2 * kAttnStages) + attn_tile_bytes(D) * 3u + 40u * 8u + 16u;
}

// How many of every eight key pairs take their exponential on the FMA pipe (0 = all on the special-function unit).
constexpr int kAttnPolyOf8 = 1;

// 2^x for a pair of FP32 values, x <= 8 or so, without the special-function unit: x = n + f with n = rint(x)
// (adding 1.5 * 2^23 leaves n in the low mantissa bits), 2^f on [-0.5, 0.5] by a cubic with relative error
// 7.5e-5 (the probabilities are rounded to BF16, 2e-3, right after), and n added to the exponent field.
// Inputs below -126 (masked keys arrive as -inf) give 2^-126.
__device__ __forceinline__ uint64_t attn_exp2_poly(uint64_t x2) {
  uint32_t a, b;
  ptx::unpack_f32x2(x2, a, b);
  x2 = ptx::pack_f32x2(__float_as_uint(fmaxf(__uint_as_float(a), -126.f)), __float_as_uint(fmaxf(__uint_as_float(b), -126.f)));
  const uint64_t magic = ptx::pack_f32x2(0x4B400000u, 0x4B400000u);      // 12582912.0f
  const uint64_t neg_magic = ptx::pack_f32x2(0xCB400000u, 0xCB400000u);
  const uint64_t neg_one = ptx::pack_f32x2(0xBF800000u, 0xBF800000u);
  const uint64_t c0 = ptx::pack_f32x2(__float_as_uint(0.9999280572f), __float_as_uint(0.9999280572f));
  const uint64_t c1 = ptx::pack_f32x2(__float_as_uint(0.6932609677f), __float_as_uint(0.6932609677f));
  const uint64_t c2 = ptx::pack_f32x2(__float_as_uint(0.2426111251f), __float_as_uint(0.2426111251f));
  const uint64_t c3 = ptx::pack_f32x2(__float_as_uint(0.0551716648f), __float_as_uint(0.0551716648f));
  const uint64_t t2 = ptx::add_f32x2(x2, magic);
  const uint64_t n2 = ptx::add_f32x2(t2, neg_magic);
  const uint64_t f2 = ptx::fma_f32x2(n2, neg_one, x2);
  uint64_t q2 = ptx::fma_f32x2(c3, f2, c2);
  q2 = ptx::fma_f32x2(q2, f2, c1);
  q2 = ptx::fma_f32x2(q2, f2, c0);
  uint32_t ta, tb, qa, qb;
  ptx::unpack_f32x2(t2, ta, tb);
  ptx::unpack_f32x2(q2, qa, qb);
  return ptx::pack_f32x2(qa + (ta << 23), qb + (tb << 23));
}

struct AttnItem {
  int b, h, kvh, t0;
  int nb0, nb1;  // key blocks tile 0 / tile 1 see
  int nbi;       // key blocks the item loads
};

// Which items a CTA works through, decided on the host for causal problems of few rounds: the items in order of
// weight (key blocks they see), each given to the CTA that has the least so far.  list[off[c] .. off[c + 1]) are CTA
// c's items.  Travels as a kernel parameter, so no call shares it with another.
constexpr int kAttnDealItems = 8192;
constexpr int kAttnDealCtas = 256;
struct AttnDeal {
  uint16_t off[kAttnDealCtas + 1];
  uint16_t list[kAttnDealItems];
};
struct AttnNoDeal {
  int unused;
};
template <bool DEAL>
struct AttnDealArg {
  using type = AttnNoDeal;
};
template <>
struct AttnDealArg<true> {
  using type = AttnDeal;
};

template <int HD, bool DEAL = false>  // head_dim: 64 or 128; DEAL: the items come from the host's list
__global__ void __launch_bounds__(kAttnThreads, 1)
    fact_attention_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                               const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmO,
                               const AttnParams p, const __grid_constant__ typename AttnDealArg<DEAL>::type deal) {
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
  constexpr int BK = attn_block_k(HD);              // keys per block
  constexpr uint32_t tile_bytes = attn_tile_bytes(HD);   // a 128-row tile (Q, O)
  constexpr uint32_t kv_bytes = attn_kv_bytes(HD);  // a BK-row tile (K, V)
  constexpr uint32_t kv_chunk = (uint32_t)BK * 128u;     // one 64-column chunk of it
  constexpr int chunks = HD / 64;
  constexpr int NS = kAttnStages;
  // tensor-memory columns of tile t, from t * 256: probabilities (two BF16 per column), scores, output
  constexpr uint32_t kColP = 0, kColS = BK / 2, kColO = BK / 2 + BK;
  static_assert(kColO + HD <= 256, "tensor memory: two tiles of P + S + O");
  const uint32_t k_s0 = smem_base;
  const uint32_t v_s0 = k_s0 + (uint32_t)NS * kv_bytes;
  const uint32_t q_s0 = v_s0 + (uint32_t)NS * kv_bytes;  // Q_0, Q_1
  const uint32_t o_stage = q_s0 + 2u * tile_bytes;
  const uint32_t bar_off = 2u * (uint32_t)NS * kv_bytes + 3u * tile_bytes;
  const uint32_t bar_base = smem_base + bar_off;
  const uint32_t ctrl_off = bar_off + 40u * 8u;
  volatile uint32_t* tmem_holder_p = reinterpret_cast<volatile uint32_t*>(smem_raw + ctrl_off);
  volatile int* abort_p = reinterpret_cast<volatile int*>(smem_raw + ctrl_off + 4);
  enum {
    Q_FULL = 0,      // + tile: the tile's Q has landed
    Q_EMPTY = 2,     // + tile: the tile's last first-product has read it
    S_FULL = 4,      // + tile: a block's scores are complete
    S_READ = 6,      // + tile: the four softmax warps hold the block's scores in registers
    P_FULL = 8,      // + tile: the four softmax warps have stored the block's probabilities
    PV_DONE = 10,    // + tile: a block's second product has completed (P may be rewritten; O may be rescaled or read)
    O_FREE = 12,     // + tile: the softmax warps have read the finished O
    O_STAGED = 14,   // + tile: ... and written O / l into the staging buffer
    OS_DONE = 16,    // + tile: the store warp's TMA store of the tile's output has read the staging buffer
    K_FULL = 18,
    V_FULL = K_FULL + NS,
    K_EMPTY = V_FULL + NS,  // both issuers arrive
    V_EMPTY = K_EMPTY + NS,
    N_BARS = V_EMPTY + NS
  };
  static_assert(N_BARS <= 40, "barrier area");
  auto bar = [&](int i) { return bar_base + 8u * (uint32_t)i; };

  if (threadIdx.x < N_BARS) {
    const int i = (int)threadIdx.x;
    uint32_t count = 1;
    if ((i >= S_READ && i < P_FULL + 2) || (i >= O_FREE && i < O_STAGED + 2)) count = 4;  // one arrival per softmax warp
    if (i >= K_EMPTY) count = 2;                                                          // one per issuer
    ptx::mbar_init(bar(i), count);
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
  // the set-up above may overlap the tail of the previous kernel in the stream; global memory only from here on
  ptx::grid_dependency_wait();

  // Items are numbered with the query position as the slow index, heaviest first (the late rows of a causal
  // problem), so neighbouring CTAs work on query heads that share K and V.
  // Items are dealt out round by round, every second round in the opposite direction: with the heaviest items
  // first, a CTA that got a heavy item in one round gets a light one in the next, and the last, partial round goes
  // to the CTAs that have had the least (plain round-robin left the first CTAs of a causal LLaMA 4 x 2048 problem
  // with 133 key blocks against 102 for the last).
  const int G = (int)gridDim.x;
  const int full_rounds = p.items / G, tail = p.items - full_rounds * G;
  auto pos_in_round = [&](int n) { return (n & 1) ? (G - 1 - (int)blockIdx.x) : (int)blockIdx.x; };
  int n_items = full_rounds + (pos_in_round(full_rounds) < tail ? 1 : 0);
  int deal_first = 0;
  if constexpr (DEAL) {
    deal_first = deal.off[blockIdx.x];
    n_items = (int)deal.off[blockIdx.x + 1] - deal_first;
  }
  const int kv_blocks_all = (p.Tk + BK - 1) / BK;
  const int bh_count = p.B * p.Hq;
  auto item_of = [&](int n) -> AttnItem {
    int idx = n * G + pos_in_round(n);
    if constexpr (DEAL) idx = deal.list[deal_first + n];
    const int qr = idx / bh_count;
    const int bh = idx - qr * bh_count;
    const int qp = p.causal ? (p.q_pairs - 1 - qr) : qr;
    AttnItem it;
    it.h = bh % p.Hq;
    it.b = bh / p.Hq;
    it.kvh = it.h / (p.Hq / p.Hkv);
    it.t0 = qp * 2 * kAttnBlockQ;
    // causal: a tile whose last row is r sees keys 0 .. r
    it.nb0 = p.causal ? min(kv_blocks_all, (it.t0 + kAttnBlockQ - 1) / BK + 1) : kv_blocks_all;
    it.nb1 = p.causal ? min(kv_blocks_all, (it.t0 + 2 * kAttnBlockQ - 1) / BK + 1) : kv_blocks_all;
    it.nbi = it.nb1;
    return it;
  };
  auto wait_all = [&](uint32_t br, uint32_t parity) -> bool {
    if (__all_sync(0xffffffffu, ptx::mbar_try_wait(br, parity))) return true;
    const bool okw = __all_sync(0xffffffffu, wait_bar(br, parity, abort_p, p.status)) != 0;
    if (!okw && lane == 0 && (p.debug & 256))  // which wait gave up first: barrier index, warp, CTA
      atomicCAS(reinterpret_cast<unsigned long long*>(p.status + 6), 0ull,
                (unsigned long long)((br - bar_base) / 8u) | ((unsigned long long)warp << 8) |
                    ((unsigned long long)blockIdx.x << 16) | (1ull << 40));
    return okw;
  };
  // ring slot and pass parity of the g-th key block this CTA loads
  auto slot_of = [](int g) { return g % NS; };
  auto pass_of = [](int g) { return (uint32_t)(g / NS) & 1u; };

  // The softmax warpgroups take the registers the third warpgroup gives back (see kAttnRegsSoftmax).
  if (warp >= 8) {
    ptx::setmaxnreg_dec<kAttnRegsOther>();
    if (warp == 8) {
      // ------------------------------------------------------------ TMA producer
      int g = 0;  // key blocks loaded so far
      bool ok = true;
      // keys and values are read again by every query tile of their head (and of the heads that share them)
      const uint64_t keep = ptx::l2_policy((p.debug & 8192) ? 0 : 2);
      for (int n = 0; ok && n < n_items; ++n) {
        const AttnItem it = item_of(n);
        for (int t = 0; ok && t < 2; ++t) {
          if (n > 0) ok = wait_all(bar(Q_EMPTY + t), (uint32_t)(n - 1) & 1u);
          if (ok && ptx::elect_one()) {
            ptx::mbar_arrive_expect_tx(bar(Q_FULL + t), tile_bytes);
            for (int c = 0; c < chunks; ++c)
              ptx::tma_load_4d(q_s0 + (uint32_t)t * tile_bytes + c * kAttnChunkBytes, &tmQ, bar(Q_FULL + t), c * 64, it.h,
                               it.t0 + t * kAttnBlockQ, it.b);
          }
        }
        for (int j = 0; ok && j < it.nbi; ++j, ++g) {
          const int s = slot_of(g);
          const uint32_t par = pass_of(g) ^ 1u;  // an empty slot's first wait passes
          ok = wait_all(bar(K_EMPTY + s), par);
          if (!ok) break;
          if (ptx::elect_one()) {
            ptx::mbar_arrive_expect_tx(bar(K_FULL + s), kv_bytes);
            for (int c = 0; c < chunks; ++c)
              ptx::tma_load_4d_hint(k_s0 + s * kv_bytes + c * kv_chunk, &tmK, bar(K_FULL + s), c * 64, it.kvh, j * BK, it.b,
                                    keep);
          }
          ok = wait_all(bar(V_EMPTY + s), par);
          if (!ok) break;
          if (ptx::elect_one()) {
            ptx::mbar_arrive_expect_tx(bar(V_FULL + s), kv_bytes);
            for (int c = 0; c < chunks; ++c)
              ptx::tma_load_4d_hint(v_s0 + s * kv_bytes + c * kv_chunk, &tmV, bar(V_FULL + s), c * 64, it.kvh, j * BK, it.b,
                                    keep);
          }
        }
      }
      __syncwarp();
    } else if (warp == 9 || warp == 11) {
      // ------------------------------------------------------------ issuer of tile t's products
      const int t = warp == 9 ? 0 : 1;
      const uint32_t tmem_p = tmem_base + (uint32_t)t * 256u + kColP;
      const uint32_t tmem_s = tmem_base + (uint32_t)t * 256u + kColS;
      const uint32_t tmem_o = tmem_base + (uint32_t)t * 256u + kColO;
      const uint32_t q_addr = q_s0 + (uint32_t)t * tile_bytes;
      const uint64_t qdesc0 = p.kmajor_desc | (uint64_t)((q_addr >> 4) & 0x3fffu);
      const bool skip_s = FACT_SKIP(p, 64), skip_pv = FACT_SKIP(p, 128);  // experiment switches, 0 in normal use
      int g = 0;   // key blocks of the items so far (the producer's numbering)
      int gt = 0;  // blocks this tile has processed
      bool ok = true;
      // S_t of the block in slot s: 16 elements of head_dim = 32 bytes of a Q row and of a K row per instruction
      auto issue_s = [&](int s, bool last_of_tile) {
        ptx::tc_fence_after();
        if (ptx::elect_one()) {
          const uint32_t kaddr = k_s0 + (uint32_t)s * kv_bytes;
          const uint64_t kdesc0 = p.kmajor_desc | (uint64_t)((kaddr >> 4) & 0x3fffu);
#pragma unroll
          for (int kk = 0; kk < HD / kUmmaK; ++kk) {
            const uint32_t qoff = (uint32_t)(kk >> 2) * kAttnChunkBytes + (uint32_t)(kk & 3) * 32u;
            const uint32_t koff = (uint32_t)(kk >> 2) * kv_chunk + (uint32_t)(kk & 3) * 32u;
            if (!skip_s)
              ptx::umma_bf16<1>(tmem_s, qdesc0 + (uint64_t)(qoff >> 4), kdesc0 + (uint64_t)(koff >> 4), p.idesc_s,
                                kk > 0 ? 1u : 0u);
          }
          ptx::umma_commit<1>(bar(S_FULL + t));
          ptx::umma_commit<1>(bar(K_EMPTY + s));
          if (last_of_tile) ptx::umma_commit<1>(bar(Q_EMPTY + t));
        }
      };
      for (int n = 0; ok && n < n_items; ++n) {
        const AttnItem it = item_of(n);
        const int nbt = (t ? it.nb1 : it.nb0);
        ok = wait_all(bar(Q_FULL + t), (uint32_t)n & 1u);
        // the scores of the previous item's last block have been read (every other block's S_READ is waited for below)
        if (ok && gt > 0) ok = wait_all(bar(S_READ + t), (uint32_t)(gt - 1) & 1u);
        if (ok) ok = wait_all(bar(K_FULL + slot_of(g)), pass_of(g));
        if (!ok) break;
        issue_s(slot_of(g), nbt == 1);
        for (int j = 0; ok && j < it.nbi; ++j) {
          // ---- the next block's scores, as soon as this block's have been read
          if (j + 1 < it.nbi) {
            const int s1 = slot_of(g + j + 1);
            if (j + 1 < nbt) {
              ok = wait_all(bar(S_READ + t), (uint32_t)gt & 1u);
              if (ok) ok = wait_all(bar(K_FULL + s1), pass_of(g + j + 1));
              if (!ok) break;
              issue_s(s1, j + 1 == nbt - 1);
            } else {
              // a block this tile does not see (causal, tile 0): release its K slot unused, once it has been filled
              ok = wait_all(bar(K_FULL + s1), pass_of(g + j + 1));
              if (!ok) break;
              if (ptx::elect_one()) ptx::mbar_arrive(bar(K_EMPTY + s1));
            }
          }
          // ---- this block's second product
          const int s = slot_of(g + j);
          if (j < nbt) {
            ok = wait_all(bar(P_FULL + t), (uint32_t)gt & 1u);
            // the first block of an item overwrites O_t: the previous item's epilogue must have read it
            if (ok && j == 0 && n > 0) ok = wait_all(bar(O_FREE + t), (uint32_t)(n - 1) & 1u);
            if (ok) ok = wait_all(bar(V_FULL + s), pass_of(g + j));
            if (!ok) break;
            ptx::tc_fence_after();
            if (ptx::elect_one()) {
              const uint32_t vaddr = v_s0 + (uint32_t)s * kv_bytes;
              const uint64_t vdesc0 = p.v_desc | (uint64_t)((vaddr >> 4) & 0x3fffu);
#pragma unroll
              for (int kk = 0; kk < BK / kUmmaK; ++kk)  // 16 keys = 2048 bytes further on in V, 8 columns in P
                if (!skip_pv)
                  ptx::umma_bf16_ts(tmem_o, tmem_p + (uint32_t)kk * 8u, vdesc0 + (uint64_t)(kk * 128), p.idesc_pv,
                                    (j > 0 || kk > 0) ? 1u : 0u);
              ptx::umma_commit<1>(bar(V_EMPTY + s));
              ptx::umma_commit<1>(bar(PV_DONE + t));
            }
            ++gt;
          } else {
            ok = wait_all(bar(V_FULL + s), pass_of(g + j));
            if (!ok) break;
            if (ptx::elect_one()) ptx::mbar_arrive(bar(V_EMPTY + s));
          }
        }
        g += it.nbi;
      }
      __syncwarp();
    } else {
      // ------------------------------------------------------------ store warp: staged O tiles -> global by TMA
      bool ok = true;
      for (int n = 0; ok && n < n_items; ++n) {
        const AttnItem it = item_of(n);
        for (int t = 0; ok && t < 2; ++t) {
          ok = wait_all(bar(O_STAGED + t), (uint32_t)n & 1u);
          if (!ok) break;
          if (lane == 0) {  // bulk groups belong to the issuing thread
            const int t0 = it.t0 + t * kAttnBlockQ;
            if (t0 < p.Tq) {  // (a second tile wholly past the end of the sequence computed on zero-filled Q)
              for (int c = 0; c < chunks; ++c) ptx::tma_store_4d(&tmO, o_stage + c * kAttnChunkBytes, c * 64, it.h, t0, it.b);
              ptx::bulk_commit_group();
              ptx::bulk_wait_group_read<0>();  // the staging buffer may be rewritten
            }
            ptx::mbar_arrive(bar(OS_DONE + t));
          }
          __syncwarp();
        }
      }
      if (lane == 0) ptx::bulk_wait_group<0>();  // every store has reached global memory before the CTA exits
      __syncwarp();
    }
  } else {
    ptx::setmaxnreg_inc<kAttnRegsSoftmax>();
    // ------------------------------------------------------------ softmax warps: one thread per query row
    const int t = warp >> 2;   // the tile this warpgroup serves
    const int q4 = warp & 3;   // the TMEM lane quarter this warp may access
    const int row = q4 * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(q4 * 32) << 16;
    const uint32_t p_addr = tmem_base + lane_addr + (uint32_t)t * 256u + kColP;
    const uint32_t s_addr = tmem_base + lane_addr + (uint32_t)t * 256u + kColS;
    const uint32_t o_addr = tmem_base + lane_addr + (uint32_t)t * 256u + kColO;
    bool ok = true;  // warp-uniform
    long long prof_s_wait = 0, prof_epi = 0, prof_blocks = 0;
    int gt = 0;
    for (int n = 0; ok && n < n_items; ++n) {
      const AttnItem it = item_of(n);
      const int nbt = (t ? it.nb1 : it.nb0);
      const int t_row = it.t0 + t * kAttnBlockQ + row;
      float m = -INFINITY;  // reference maximum of scale_log2 * score the exponentials are taken against
      float l = 0.f;        // running sum of 2^(scale_log2 * score - m)
      for (int j = 0; ok && j < nbt; ++j, ++gt) {
        const long long tc1 = prof ? clock64() : 0;
        ok = wait_all(bar(S_FULL + t), (uint32_t)gt & 1u);
        if (!ok) break;
        if (prof) {
          prof_s_wait += clock64() - tc1;
          ++prof_blocks;
        }
        ptx::tc_fence_after();
        uint32_t s64[BK / 64][64];
#pragma unroll
        for (int c = 0; c < BK / 64; ++c) ptx::tmem_ld_32x32b_x64(s_addr + (uint32_t)c * 64u, s64[c]);
        uint32_t (&s)[BK / 32][32] = *reinterpret_cast<uint32_t (*)[BK / 32][32]>(&s64[0][0]);
        ptx::tmem_wait_ld();
        // the scores are in registers: the next block's may overwrite them
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(bar(S_READ + t));
        if (FACT_SKIP(p, 8)) {  // experiment switch: no softmax arithmetic, the barrier protocol only
          if (gt > 0) ok = wait_all(bar(PV_DONE + t), (uint32_t)(gt - 1) & 1u);
          if (!ok) break;
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(bar(P_FULL + t));
          continue;
        }
        // Only the block on the diagonal (or the ragged last one) needs the per-key mask.
        const int key_limit = min(p.Tk, p.causal ? t_row + 1 : p.Tk) - j * BK;
        if (__any_sync(0xffffffffu, key_limit < BK)) {
#pragma unroll
          for (int c = 0; c < BK / 32; ++c)
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (c * 32 + i >= key_limit) s[c][i] = 0xff800000u;  // -inf
        }
        // four independent chains of three-input maxima
        float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
        for (int c = 0; c < BK / 32; ++c)
#pragma unroll
          for (int i = 0; i < 32; i += 2)
            mx4[(i >> 1) & 3] = ptx::max3(mx4[(i >> 1) & 3], __uint_as_float(s[c][i]), __uint_as_float(s[c][i + 1]));
        const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * p.scale_log2;  // scale > 0
        bool pv_waited = false;  // whether this block has already made sure that O_t += P_t(j-1) V has completed
        // Move the reference maximum only when this block exceeds it by more than the threshold (always from -inf).
        if (__any_sync(0xffffffffu, mx > m + kAttnRescaleThreshold)) {
          const float m_new = fmaxf(m, mx);
          const float alpha = ptx::ex2_approx(m - ((m_new == -INFINITY) ? 0.f : m_new));
          l *= alpha;
          m = m_new;
          if (j > 0) {
            // O_t is rescaled between O_t += P_t(j-1) V, which must have completed, and O_t += P_t(j) V, which waits
            // for the probabilities announced below
            ok = wait_all(bar(PV_DONE + t), (uint32_t)(gt - 1) & 1u);
            if (!ok) break;
            pv_waited = true;
            ptx::tc_fence_after();
#pragma unroll 1
            for (int c = 0; c < HD; c += 32) {
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
        // 2^(scale_log2 * s - m) on pairs of keys with packed FP32 arithmetic; kAttnPolyOf8 of every eight pairs take
        // the exponential on the FMA pipe (attn_exp2_poly), the others on the special-function unit, whose four
        // results a cycle and partition are what bounds this kernel.
        const uint64_t scale2 = ptx::pack_f32x2(__float_as_uint(p.scale_log2), __float_as_uint(p.scale_log2));
        const uint64_t negm2 = ptx::pack_f32x2(__float_as_uint(-m_use), __float_as_uint(-m_use));
        uint64_t sum2[4] = {0ull, 0ull, 0ull, 0ull};
        uint32_t pw[BK / 64][32];
#pragma unroll
        for (int hh = 0; hh < BK / 64; ++hh) {  // 64 keys = 32 columns of BF16 pairs at a time
#pragma unroll
          for (int c = 0; c < 2; ++c)
#pragma unroll
            for (int i = 0; i < 32; i += 2) {
              const int pr = c * 16 + (i >> 1);
              const uint64_t x2 = ptx::fma_f32x2(ptx::pack_f32x2(s[hh * 2 + c][i], s[hh * 2 + c][i + 1]), scale2, negm2);
              uint64_t p2;
              if ((pr & 7) < kAttnPolyOf8) {
                p2 = attn_exp2_poly(x2);
              } else {
                uint32_t x0, x1;
                ptx::unpack_f32x2(x2, x0, x1);
                p2 = ptx::pack_f32x2(__float_as_uint(ptx::ex2_approx(__uint_as_float(x0))),
                                     __float_as_uint(ptx::ex2_approx(__uint_as_float(x1))));
              }
              sum2[pr & 3] = ptx::add_f32x2(sum2[pr & 3], p2);
              uint32_t p0, p1;
              ptx::unpack_f32x2(p2, p0, p1);
              pw[hh][pr] = pack_bf16x2(__uint_as_float(p0), __uint_as_float(p1));
            }
        }
        // the probabilities of the block before must have been consumed before these overwrite them
        if (gt > 0 && !pv_waited) {
          ok = wait_all(bar(PV_DONE + t), (uint32_t)(gt - 1) & 1u);
          if (!ok) break;
        }
        // lane = row, column c holds keys 2c and 2c + 1
        if constexpr (BK == 128) {
          ptx::tmem_st_32x32b_x64(p_addr, *reinterpret_cast<uint32_t (*)[64]>(&pw[0][0]));
        } else {
          ptx::tmem_st_32x32b_x32(p_addr, pw[0]);
        }
        {
          const uint64_t st = ptx::add_f32x2(ptx::add_f32x2(sum2[0], sum2[1]), ptx::add_f32x2(sum2[2], sum2[3]));
          uint32_t lo, hi;
          ptx::unpack_f32x2(st, lo, hi);
          l += __uint_as_float(lo) + __uint_as_float(hi);
        }
        ptx::tmem_wait_st();
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(bar(P_FULL + t));
      }
      if (!ok) break;
      // ---- the tile's output: O_t / l as BF16 into the staging tile (128-byte rows of 64 columns, 16-byte pieces
      // swizzled by the row like every other tile here), which tiles 0 and 1 of every item use in turn
      const long long te0 = prof ? clock64() : 0;
      ok = wait_all(bar(PV_DONE + t), (uint32_t)(gt - 1) & 1u);  // the tile's last product
      // The staging buffer is used in the order tile 0, tile 1 of item 0, tile 0, tile 1 of item 1, ...: wait until
      // the store of the use before this one has read it.  (One barrier per tile: each warpgroup then waits for
      // every completion of the other tile's barrier in turn, which a one-bit phase can express.)
      if (ok && t == 1) ok = wait_all(bar(OS_DONE + 0), (uint32_t)n & 1u);
      if (ok && t == 0 && n > 0) ok = wait_all(bar(OS_DONE + 1), (uint32_t)(n - 1) & 1u);
      if (!ok) break;
      ptx::tc_fence_after();
      const float inv = (l > 0.f) ? __fdividef(1.f, l) : 0.f;
#pragma unroll
      for (int c = 0; c < HD / 32; ++c) {
        uint32_t o[32];
        ptx::tmem_ld_32x32b_x32(o_addr + (uint32_t)(c * 32), o);
        ptx::tmem_wait_ld();
        const uint32_t dst = o_stage + (uint32_t)(c >> 1) * kAttnChunkBytes + (uint32_t)row * 128u;
#pragma unroll
        for (int gq = 0; gq < 4; ++gq) {
          const uint32_t piece = (uint32_t)((c & 1) * 4 + gq);
          ptx::st_shared_v4(dst + ((piece ^ (uint32_t)(row & 7)) << 4),
                            pack_bf16x2(__uint_as_float(o[gq * 8 + 0]) * inv, __uint_as_float(o[gq * 8 + 1]) * inv),
                            pack_bf16x2(__uint_as_float(o[gq * 8 + 2]) * inv, __uint_as_float(o[gq * 8 + 3]) * inv),
                            pack_bf16x2(__uint_as_float(o[gq * 8 + 4]) * inv, __uint_as_float(o[gq * 8 + 5]) * inv),
                            pack_bf16x2(__uint_as_float(o[gq * 8 + 6]) * inv, __uint_as_float(o[gq * 8 + 7]) * inv));
        }
      }
      ptx::tc_fence_before();
      ptx::fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) {
        ptx::mbar_arrive(bar(O_FREE + t));
        ptx::mbar_arrive(bar(O_STAGED + t));
      }
      if (prof) prof_epi += clock64() - te0;
    }
    if (prof && warp == 0 && lane == 0) {
      long long* prof_c = reinterpret_cast<long long*>(p.status + 2);
      prof_c[3] = prof_s_wait;
      prof_c[4] = prof_blocks;
      prof_c[6] = prof_epi;
      prof_c[7] = n_items;
    }
  }

  // ------------------------------------------------------------ teardown
  ptx::grid_launch_dependents();  // this CTA's items are done: the next kernel of the stream may move in behind it
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
