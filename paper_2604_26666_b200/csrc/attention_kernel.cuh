// Fused multi-head attention forward for sm_100a: O = softmax(scale * Q K^T + causal mask) V, BF16 in and out,
// FP32 scores / probabilities / accumulation, grouped queries (several query heads share one key/value head).
//
// One CTA owns 256 query positions of one (batch, query head) as two tiles of 128 rows (A and B) that share every
// key/value block it loads, and walks the key/value sequence in blocks of 128 keys with the online-softmax
// recurrence (a reference maximum m and row sum l per row; the output accumulator is rescaled by
// 2^(m_old - m_new) only when the block maximum exceeds m by more than 8, so probabilities stay below 2^8 and the
// final division by l removes the stale reference exactly).  Roles:
//   warp 0      TMA producer: both Q tiles once, then K and V blocks into two two-stage rings
//   warp 1      MMA issuer, in the order  S_A(j), PV_B(j-1), S_B(j), PV_A(j):
//                 S_t(j) = Q_t K_j^T     tcgen05.mma, M = 128, N = 128, K = head_dim, both operands from shared memory
//                 O_t   += P_t(j) V_j    tcgen05.mma, M = 128, N = head_dim, K = 128, A = P_t read from tensor memory
//   warps 2-5   softmax of tile A, warps 6-9 of tile B: one query row per thread: tcgen05.ld the scores, mask,
//               maximum, exponentials, row sum; rescale O_t in tensor memory when needed; tcgen05.st the BF16
//               probabilities over the first 64 columns of the scores they replace; at the end O_t / l -> global
// While one tile's softmax runs, the tensor pipe works on the other tile's products.  Tensor memory (512 columns):
// S_A/P_A at 0, S_B/P_B at 128, O_A at 256, O_B at 384.  P_t(j) may overwrite S_t(j) because every thread has read
// its own row (lane) before it writes it, and S_t(j+1) is issued after PV_t(j) on the same in-order pipe.
// Every mbarrier wait is bounded, as in the GEMM kernel.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "gemm_kernel.cuh"
#include "ptx.cuh"

namespace fact {

constexpr int kAttnThreads = 320;   // 10 warps
constexpr int kAttnBlockQ = 128;    // query rows per tile (= TMEM lanes); a CTA owns two tiles
constexpr int kAttnBlockK = 128;    // keys per block
constexpr uint32_t kAttnChunkBytes = 128 * 128;  // one 64-column chunk of a 128-row tile, 128-byte rows
constexpr float kAttnRescaleThreshold = 8.f;     // log2 units

struct AttnParams {
  int B, Tq, Tk, Hq, Hkv, D;  // D = 64 or 128
  int causal;
  float scale_log2;           // softmax scale * log2(e)
  int q_pairs;                // ceil(Tq / 256)
  __nv_bfloat16* O;
  long long o_stride_b, o_stride_t, o_stride_h;  // in elements; head_dim is contiguous
  uint64_t kmajor_desc;       // UMMA descriptor template, K-major 128B-swizzled tiles (Q, K)
  uint64_t v_desc;            // UMMA descriptor template, V as an N-major operand
  uint32_t idesc_s, idesc_pv;
  int* status;
};

// Shared-memory carve-up (dynamic, 1024-byte aligned): Q[2] | K[2] | V[2] | barriers
__host__ __device__ constexpr uint32_t attn_tile_bytes(int D) { return (uint32_t)(D / 64) * kAttnChunkBytes; }
__host__ __device__ constexpr uint32_t attn_smem_bytes(int D) { return attn_tile_bytes(D) * 6u + 16u * 8u + 16u; }

__global__ void __launch_bounds__(kAttnThreads, 1)
    fact_attention_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                          const __grid_constant__ CUtensorMap tmV, const AttnParams p) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);
  const int lane = threadIdx.x & 31;
  const uint32_t smem_base = ptx::smem_u32(smem_raw);
  if (smem_base & 1023u) {
    if (threadIdx.x == 0) atomicExch(p.status, kDeviceTimeoutCode);
    return;
  }
  const uint32_t tile_bytes = attn_tile_bytes(p.D);
  const uint32_t q_s = smem_base;
  const uint32_t k_s0 = q_s + 2u * tile_bytes;
  const uint32_t v_s0 = k_s0 + 2u * tile_bytes;
  const uint32_t bar_base = v_s0 + 2u * tile_bytes;
  const uint32_t ctrl_off = bar_base - smem_base + 16u * 8u;
  volatile uint32_t* tmem_holder_p = reinterpret_cast<volatile uint32_t*>(smem_raw + ctrl_off);
  volatile int* abort_p = reinterpret_cast<volatile int*>(smem_raw + ctrl_off + 4);
  enum { Q_FULL = 0, K_FULL = 1, V_FULL = 3, K_EMPTY = 5, V_EMPTY = 7, S_FULL = 9, P_FULL = 11, O_DONE = 13, N_BARS = 15 };
  auto bar = [&](int i) { return bar_base + 8u * (uint32_t)i; };

  if (threadIdx.x < N_BARS) {
    const int i = (int)threadIdx.x;
    const uint32_t count = (i == P_FULL || i == P_FULL + 1) ? 4u : 1u;  // one arrival per softmax warp of the tile
    ptx::mbar_init(bar(i), count);
    if (i == 0) *abort_p = 0;
    ptx::fence_mbar_init();
  }
  if (warp == 0 && lane == 0) {
    ptx::prefetch_tensormap(&tmQ);
    ptx::prefetch_tensormap(&tmK);
    ptx::prefetch_tensormap(&tmV);
  }
  if (warp == 1) {
    __syncwarp();
    ptx::tmem_alloc<1>(smem_base + ctrl_off, 512);
    ptx::tmem_relinquish<1>();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_holder_p;

  // this CTA's pair of tiles: heavy (late) query tiles of a causal problem are launched first
  int t = (int)blockIdx.x;
  const int qp_raw = t % p.q_pairs;
  t /= p.q_pairs;
  const int h = t % p.Hq;
  const int b = t / p.Hq;
  const int qp = p.causal ? (p.q_pairs - 1 - qp_raw) : qp_raw;
  const int t0 = qp * 2 * kAttnBlockQ;
  const int kvh = h / (p.Hq / p.Hkv);
  const int kv_blocks_all = (p.Tk + kAttnBlockK - 1) / kAttnBlockK;
  // key blocks each tile visits: a causal tile stops at its diagonal block; tile B does not exist past the last row
  const int nb_a = p.causal ? min(kv_blocks_all, 2 * qp + 1) : kv_blocks_all;
  const int nb_b = (t0 + kAttnBlockQ < p.Tq) ? (p.causal ? min(kv_blocks_all, 2 * qp + 2) : kv_blocks_all) : 0;
  const int nb = max(nb_a, nb_b);
  const int chunks = p.D / 64;
  auto wait_all = [&](uint32_t br, uint32_t parity) -> bool {
    return __all_sync(0xffffffffu, wait_bar(br, parity, abort_p, p.status)) != 0;
  };

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (ptx::elect_one()) {
      ptx::mbar_arrive_expect_tx(bar(Q_FULL), 2u * tile_bytes);
      for (int tl = 0; tl < 2; ++tl)
        for (int c = 0; c < chunks; ++c)
          ptx::tma_load_4d(q_s + tl * tile_bytes + c * kAttnChunkBytes, &tmQ, bar(Q_FULL), c * 64, h,
                           t0 + tl * kAttnBlockQ, b);
    }
    for (int j = 0; j < nb; ++j) {
      const int s = j & 1;
      const uint32_t par = (((uint32_t)j >> 1) & 1u) ^ 1u;
      if (!wait_all(bar(K_EMPTY + s), par)) break;
      if (ptx::elect_one()) {
        ptx::mbar_arrive_expect_tx(bar(K_FULL + s), tile_bytes);
        for (int c = 0; c < chunks; ++c)
          ptx::tma_load_4d(k_s0 + s * tile_bytes + c * kAttnChunkBytes, &tmK, bar(K_FULL + s), c * 64, kvh,
                           j * kAttnBlockK, b);
      }
      if (!wait_all(bar(V_EMPTY + s), par)) break;
      if (ptx::elect_one()) {
        ptx::mbar_arrive_expect_tx(bar(V_FULL + s), tile_bytes);
        for (int c = 0; c < chunks; ++c)
          ptx::tma_load_4d(v_s0 + s * tile_bytes + c * kAttnChunkBytes, &tmV, bar(V_FULL + s), c * 64, kvh,
                           j * kAttnBlockK, b);
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    bool ok = wait_all(bar(Q_FULL), 0);
    ptx::tc_fence_after();
    auto issue_s = [&](int tl, int j) {  // S_tl(j) = Q_tl K_j^T
      const uint32_t qs = q_s + (uint32_t)tl * tile_bytes;
      const uint32_t ks = k_s0 + (uint32_t)(j & 1) * tile_bytes;
      const uint32_t d = tmem_base + (uint32_t)tl * 128u;
      if (ptx::elect_one()) {
        for (int kk = 0; kk < p.D / kUmmaK; ++kk) {
          const uint32_t off = (uint32_t)(kk >> 2) * kAttnChunkBytes + (uint32_t)(kk & 3) * 32u;
          const uint64_t adesc = p.kmajor_desc | (uint64_t)(((qs + off) >> 4) & 0x3fffu);
          const uint64_t bdesc = p.kmajor_desc | (uint64_t)(((ks + off) >> 4) & 0x3fffu);
          ptx::umma_bf16<1>(d, adesc, bdesc, p.idesc_s, kk > 0 ? 1u : 0u);
        }
        ptx::umma_commit<1>(bar(S_FULL + tl));
      }
    };
    // O_tl += P_tl(j) V_j once the tile's softmax has stored P_tl(j); releases V_j after its last reader
    auto issue_pv = [&](int tl, int j, bool last_reader_of_v, bool last_block) -> bool {
      if (!wait_all(bar(P_FULL + tl), (uint32_t)j & 1u)) return false;
      if (!wait_all(bar(V_FULL + (j & 1)), ((uint32_t)j >> 1) & 1u)) return false;
      ptx::tc_fence_after();
      if (ptx::elect_one()) {
        const uint32_t vs = v_s0 + (uint32_t)(j & 1) * tile_bytes;
        const uint32_t p_t = tmem_base + (uint32_t)tl * 128u;          // BF16 pairs: 8 columns per 16 keys
        const uint32_t o_t = tmem_base + 256u + (uint32_t)tl * 128u;
        for (int kk = 0; kk < kAttnBlockK / kUmmaK; ++kk) {
          const uint64_t bdesc = p.v_desc | (uint64_t)(((vs + (uint32_t)kk * 2048u) >> 4) & 0x3fffu);
          ptx::umma_bf16_ts(o_t, p_t + (uint32_t)kk * 8u, bdesc, p.idesc_pv, (j > 0 || kk > 0) ? 1u : 0u);
        }
        if (last_reader_of_v) ptx::umma_commit<1>(bar(V_EMPTY + (j & 1)));
        if (last_block) ptx::umma_commit<1>(bar(O_DONE + tl));
      }
      return true;
    };
    for (int j = 0; ok && j < nb; ++j) {
      if (!wait_all(bar(K_FULL + (j & 1)), ((uint32_t)j >> 1) & 1u)) break;
      ptx::tc_fence_after();
      if (j < nb_a) issue_s(0, j);
      if (j >= 1 && j - 1 < nb_b) ok = issue_pv(1, j - 1, true, j == nb_b);
      if (!ok) break;
      if (j < nb_b) issue_s(1, j);
      if (ptx::elect_one()) ptx::umma_commit<1>(bar(K_EMPTY + (j & 1)));
      if (j < nb_a) ok = issue_pv(0, j, j >= nb_b, j == nb_a - 1);
    }
    if (ok && nb_b == nb && nb_b > 0) issue_pv(1, nb_b - 1, true, true);
    __syncwarp();
  } else {
    // ------------------------------------------------------------ softmax warps: one query row per thread
    const int tl = (warp - 2) >> 2;  // 0: tile A, 1: tile B
    const int q4 = warp & 3;         // the TMEM lane quarter this warp may access
    const int row = q4 * 32 + lane;
    const int t_row = t0 + tl * kAttnBlockQ + row;
    const int nb_t = tl ? nb_b : nb_a;
    const uint32_t lane_addr = (uint32_t)(q4 * 32) << 16;
    const uint32_t s_addr = tmem_base + lane_addr + (uint32_t)tl * 128u;
    const uint32_t o_addr = tmem_base + lane_addr + 256u + (uint32_t)tl * 128u;
    float m = -INFINITY;  // reference maximum of scale_log2 * score the exponentials are taken against
    float l = 0.f;        // running sum of 2^(scale_log2 * score - m)
    bool ok = true;
    for (int j = 0; ok && j < nb_t; ++j) {
      if (!wait_bar(bar(S_FULL + tl), (uint32_t)j & 1u, abort_p, p.status)) {
        ok = false;
        break;
      }
      ptx::tc_fence_after();
      uint32_t sraw[4][32];
#pragma unroll
      for (int c = 0; c < 4; ++c) ptx::tmem_ld_32x32b_x32(s_addr + (uint32_t)c * 32u, sraw[c]);
      ptx::tmem_wait_ld();
      // Mask and maximum.  Only the block on the diagonal (or the ragged last one) needs the per-key mask; four
      // independent chains keep the maximum and the sum from serialising on the instruction latency.
      const int key0 = j * kAttnBlockK;
      const int key_limit = min(p.Tk, p.causal ? t_row + 1 : p.Tk) - key0;  // keys [0, key_limit) of this block count
      if (__any_sync(0xffffffffu, key_limit < kAttnBlockK)) {
#pragma unroll
        for (int c = 0; c < 4; ++c)
#pragma unroll
          for (int i = 0; i < 32; ++i)
            if (c * 32 + i >= key_limit) sraw[c][i] = 0xff800000u;  // -inf
      }
      float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
      for (int c = 0; c < 4; ++c)
#pragma unroll
        for (int i = 0; i < 32; ++i) mx4[i & 3] = fmaxf(mx4[i & 3], __uint_as_float(sraw[c][i]));
      const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * p.scale_log2;  // scale > 0
      // Move the reference maximum only when this block exceeds it by more than the threshold (always from -inf).
      // PV_t(j-1) has completed (S_t(j) was issued after it on the same pipe), so O_t may be rescaled here.
      if (__any_sync(0xffffffffu, mx > m + kAttnRescaleThreshold)) {
        const float m_new = fmaxf(m, mx);
        const float alpha = ptx::ex2_approx(m - ((m_new == -INFINITY) ? 0.f : m_new));
        l *= alpha;
        m = m_new;
        if (j > 0) {
          for (int c = 0; c < p.D; c += 32) {
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
      uint32_t pw[2][32];  // the row's 128 probabilities as BF16 pairs
#pragma unroll
      for (int c = 0; c < 4; ++c)
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
          // 2^(scale_log2 * s - m): one fused multiply-add and one ex2 per probability
          const float p0 = ptx::ex2_approx(fmaf(__uint_as_float(sraw[c][i]), p.scale_log2, -m_use));
          const float p1 = ptx::ex2_approx(fmaf(__uint_as_float(sraw[c][i + 1]), p.scale_log2, -m_use));
          sum4[(i >> 1) & 3] += p0 + p1;
          pw[c >> 1][(c & 1) * 16 + (i >> 1)] = pack_bf16x2(p0, p1);
        }
      l += (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
      // P_t(j) over the first 64 columns of S_t(j): lane = row, column c holds keys 2c and 2c + 1
      ptx::tmem_st_32x32b_x32(s_addr, pw[0]);
      ptx::tmem_st_32x32b_x32(s_addr + 32u, pw[1]);
      ptx::tmem_wait_st();
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(bar(P_FULL + tl));
    }
    // O / l -> global (one row of head_dim BF16 values per thread)
    if (ok && nb_t > 0) {
      if (wait_bar(bar(O_DONE + tl), 0u, abort_p, p.status)) {
        ptx::tc_fence_after();
        const float inv = (l > 0.f) ? __fdividef(1.f, l) : 0.f;
        __nv_bfloat16* dst = p.O + (long long)b * p.o_stride_b + (long long)t_row * p.o_stride_t + (long long)h * p.o_stride_h;
        for (int c = 0; c < p.D; c += 32) {
          uint32_t o[32];
          ptx::tmem_ld_32x32b_x32(o_addr + (uint32_t)c, o);
          ptx::tmem_wait_ld();
          if (t_row < p.Tq) {
#pragma unroll
            for (int g = 0; g < 4; ++g) {
              uint4 qv;
              qv.x = pack_bf16x2(__uint_as_float(o[g * 8 + 0]) * inv, __uint_as_float(o[g * 8 + 1]) * inv);
              qv.y = pack_bf16x2(__uint_as_float(o[g * 8 + 2]) * inv, __uint_as_float(o[g * 8 + 3]) * inv);
              qv.z = pack_bf16x2(__uint_as_float(o[g * 8 + 4]) * inv, __uint_as_float(o[g * 8 + 5]) * inv);
              qv.w = pack_bf16x2(__uint_as_float(o[g * 8 + 6]) * inv, __uint_as_float(o[g * 8 + 7]) * inv);
              *reinterpret_cast<uint4*>(dst + c + g * 8) = qv;
            }
          }
        }
      }
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
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc<1>(tmem_base, 512);
  }
}

}  // namespace fact
