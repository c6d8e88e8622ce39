// Fused multi-head attention forward for sm_100a: O = softmax(scale * Q K^T + causal mask) V, BF16 in and out,
// FP32 scores / probabilities / accumulation, grouped queries (several query heads share one key/value head).
//
// One CTA owns 128 query positions of one (batch, query head) and walks the key/value sequence in blocks of
// 128 keys with the online-softmax recurrence (running row maximum m and row sum l; the output accumulator is
// rescaled by 2^(m_old - m_new) whenever the maximum grows).  Roles:
//   warp 0     TMA producer: the Q tile once, then K and V blocks into a two-stage ring
//   warp 1     MMA issuer:   S_j = Q K_j^T   (tcgen05.mma, M = 128, N = 128, K = head_dim) into one of two S
//                            accumulators in tensor memory, and O += P_j V_j (M = 128, N = head_dim, K = 128)
//   warps 2-5  softmax:      one query row per thread: tcgen05.ld the scores, mask, maximum, exponentials,
//                            row sum; rescale O in tensor memory when needed; write P_j (BF16) into shared
//                            memory in the swizzled K-major layout the second MMA reads; at the end O / l
// S_{j+1} is issued before the softmax of block j finishes (two S buffers), so the first product of the next
// block overlaps the exponentials of this one.  Every mbarrier wait is bounded, as in the GEMM kernel.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "gemm_kernel.cuh"
#include "ptx.cuh"

namespace fact {

constexpr int kAttnThreads = 192;   // 6 warps
constexpr int kAttnBlockQ = 128;    // query rows per CTA (= TMEM lanes)
constexpr int kAttnBlockK = 128;    // keys per block
constexpr uint32_t kAttnChunkBytes = 128 * 128;  // one 64-column chunk of a 128-row tile, 128-byte rows

struct AttnParams {
  int B, Tq, Tk, Hq, Hkv, D;  // D = 64 or 128
  int causal;
  float scale_log2;           // softmax scale * log2(e)
  int q_tiles;                // ceil(Tq / 128)
  __nv_bfloat16* O;
  long long o_stride_b, o_stride_t, o_stride_h;  // in elements; head_dim is contiguous
  uint64_t kmajor_desc;       // UMMA descriptor template, K-major 128B-swizzled tiles (Q, K, P)
  uint64_t v_desc;            // UMMA descriptor template, V as an N-major operand
  uint32_t idesc_s, idesc_pv;
  int* status;
};

// Shared-memory carve-up (dynamic, 1024-byte aligned): Q | K[2] | V[2] | P | barriers
__host__ __device__ constexpr uint32_t attn_tile_bytes(int D) { return (uint32_t)(D / 64) * kAttnChunkBytes; }
__host__ __device__ constexpr uint32_t attn_smem_bytes(int D) {
  return attn_tile_bytes(D) * 5u + 2u * kAttnChunkBytes + 16u * 8u + 16u;
}

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
  const uint32_t k_s0 = q_s + tile_bytes;
  const uint32_t v_s0 = k_s0 + 2u * tile_bytes;
  const uint32_t p_s = v_s0 + 2u * tile_bytes;
  const uint32_t bar_base = p_s + 2u * kAttnChunkBytes;
  const uint32_t ctrl_off = bar_base - smem_base + 16u * 8u;
  volatile uint32_t* tmem_holder_p = reinterpret_cast<volatile uint32_t*>(smem_raw + ctrl_off);
  volatile int* abort_p = reinterpret_cast<volatile int*>(smem_raw + ctrl_off + 4);
  enum { Q_FULL = 0, K_FULL = 1, V_FULL = 3, KV_EMPTY = 5, S_FULL = 7, S_FREE = 9, P_FULL = 11, PV_DONE = 12, N_BARS = 13 };
  auto bar = [&](int i) { return bar_base + 8u * (uint32_t)i; };

  if (threadIdx.x < N_BARS) {
    const int i = (int)threadIdx.x;
    const uint32_t count = (i == S_FREE || i == S_FREE + 1 || i == P_FULL) ? 4u : 1u;  // one arrival per softmax warp
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
  const uint32_t tmem_o = tmem_base + 256u;  // columns [0,128) and [128,256) hold S_0 / S_1, [256, 256+D) holds O

  // this CTA's tile: heavy (late) query tiles of a causal problem are launched first
  int t = (int)blockIdx.x;
  const int qt_raw = t % p.q_tiles;
  t /= p.q_tiles;
  const int h = t % p.Hq;
  const int b = t / p.Hq;
  const int qt = p.causal ? (p.q_tiles - 1 - qt_raw) : qt_raw;
  const int t0 = qt * kAttnBlockQ;
  const int kvh = h / (p.Hq / p.Hkv);
  const int kv_blocks_all = (p.Tk + kAttnBlockK - 1) / kAttnBlockK;
  const int nb = p.causal ? min(kv_blocks_all, qt + 1) : kv_blocks_all;
  const int chunks = p.D / 64;
  auto wait_all = [&](uint32_t br, uint32_t parity) -> bool {
    return __all_sync(0xffffffffu, wait_bar(br, parity, abort_p, p.status)) != 0;
  };

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    bool ok = true;
    if (ptx::elect_one()) {
      ptx::mbar_arrive_expect_tx(bar(Q_FULL), tile_bytes);
      for (int c = 0; c < chunks; ++c) ptx::tma_load_4d(q_s + c * kAttnChunkBytes, &tmQ, bar(Q_FULL), c * 64, h, t0, b);
    }
    for (int j = 0; ok && j < nb; ++j) {
      const int s = j & 1;
      if (!wait_all(bar(KV_EMPTY + s), (((uint32_t)j >> 1) & 1u) ^ 1u)) {
        ok = false;
        break;
      }
      if (ptx::elect_one()) {
        ptx::mbar_arrive_expect_tx(bar(K_FULL + s), tile_bytes);
        for (int c = 0; c < chunks; ++c)
          ptx::tma_load_4d(k_s0 + s * tile_bytes + c * kAttnChunkBytes, &tmK, bar(K_FULL + s), c * 64, kvh,
                           j * kAttnBlockK, b);
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
    auto issue_s = [&](int j) {  // S_j = Q K_j^T into S buffer j & 1
      const uint32_t ks = k_s0 + (uint32_t)(j & 1) * tile_bytes;
      const uint32_t d = tmem_base + (uint32_t)(j & 1) * 128u;
      if (ptx::elect_one()) {
        for (int kk = 0; kk < p.D / kUmmaK; ++kk) {
          const uint32_t off = (uint32_t)(kk >> 2) * kAttnChunkBytes + (uint32_t)(kk & 3) * 32u;
          const uint64_t adesc = p.kmajor_desc | (uint64_t)(((q_s + off) >> 4) & 0x3fffu);
          const uint64_t bdesc = p.kmajor_desc | (uint64_t)(((ks + off) >> 4) & 0x3fffu);
          ptx::umma_bf16<1>(d, adesc, bdesc, p.idesc_s, kk > 0 ? 1u : 0u);
        }
        ptx::umma_commit<1>(bar(S_FULL + (j & 1)));
      }
    };
    if (ok && nb > 0) {
      ok = wait_all(bar(K_FULL), 0);
      ptx::tc_fence_after();
      if (ok) issue_s(0);
    }
    for (int j = 0; ok && j < nb; ++j) {
      if (j + 1 < nb) {
        const int jn = j + 1;
        // the S buffer of block j+1 was last read by the softmax of block j-1
        if (jn >= 2 && !wait_all(bar(S_FREE + (jn & 1)), (((uint32_t)jn >> 1) - 1u) & 1u)) {
          ok = false;
          break;
        }
        if (!wait_all(bar(K_FULL + (jn & 1)), ((uint32_t)jn >> 1) & 1u)) {
          ok = false;
          break;
        }
        ptx::tc_fence_after();
        issue_s(jn);
      }
      if (!wait_all(bar(P_FULL), (uint32_t)j & 1u) || !wait_all(bar(V_FULL + (j & 1)), ((uint32_t)j >> 1) & 1u)) {
        ok = false;
        break;
      }
      ptx::tc_fence_after();
      if (ptx::elect_one()) {  // O += P_j V_j
        const uint32_t vs = v_s0 + (uint32_t)(j & 1) * tile_bytes;
        for (int kk = 0; kk < kAttnBlockK / kUmmaK; ++kk) {
          const uint32_t poff = (uint32_t)(kk >> 2) * kAttnChunkBytes + (uint32_t)(kk & 3) * 32u;
          const uint64_t adesc = p.kmajor_desc | (uint64_t)(((p_s + poff) >> 4) & 0x3fffu);
          const uint64_t bdesc = p.v_desc | (uint64_t)(((vs + (uint32_t)kk * 2048u) >> 4) & 0x3fffu);
          ptx::umma_bf16<1>(tmem_o, adesc, bdesc, p.idesc_pv, (j > 0 || kk > 0) ? 1u : 0u);
        }
        ptx::umma_commit<1>(bar(PV_DONE));
        ptx::umma_commit<1>(bar(KV_EMPTY + (j & 1)));
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------ softmax warps: one query row per thread
    const int q4 = warp & 3;
    const int row = q4 * 32 + lane;
    const int t_row = t0 + row;
    const uint32_t lane_addr = (uint32_t)(q4 * 32) << 16;
    const uint32_t my_row = (uint32_t)row * 128u;
    const uint32_t swz = (uint32_t)(row & 7);
    float m = -INFINITY;  // running maximum of scale_log2 * score
    float l = 0.f;        // running sum of 2^(scale_log2 * score - m)
    bool ok = true;
    for (int j = 0; ok && j < nb; ++j) {
      if (!wait_bar(bar(S_FULL + (j & 1)), ((uint32_t)j >> 1) & 1u, abort_p, p.status)) {
        ok = false;
        break;
      }
      ptx::tc_fence_after();
      const uint32_t s_addr = tmem_base + lane_addr + (uint32_t)(j & 1) * 128u;
      uint32_t sraw[4][32];
#pragma unroll
      for (int c = 0; c < 4; ++c) ptx::tmem_ld_32x32b_x32(s_addr + (uint32_t)c * 32u, sraw[c]);
      ptx::tmem_wait_ld();
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(bar(S_FREE + (j & 1)));
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
      const float m_new = fmaxf(m, mx);
      const float m_use = (m_new == -INFINITY) ? 0.f : m_new;  // a row with nothing visible yet
      const float alpha = ptx::ex2_approx(m - m_use);
      float sum4[4] = {0.f, 0.f, 0.f, 0.f};
      uint32_t pw[64];  // the row's 128 probabilities as BF16 pairs
#pragma unroll
      for (int c = 0; c < 4; ++c)
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
          // 2^(scale_log2 * s - m): one fused multiply-add and one ex2 per probability
          const float p0 = ptx::ex2_approx(fmaf(__uint_as_float(sraw[c][i]), p.scale_log2, -m_use));
          const float p1 = ptx::ex2_approx(fmaf(__uint_as_float(sraw[c][i + 1]), p.scale_log2, -m_use));
          sum4[(i >> 1) & 3] += p0 + p1;
          pw[c * 16 + (i >> 1)] = pack_bf16x2(p0, p1);
        }
      l = l * alpha + ((sum4[0] + sum4[1]) + (sum4[2] + sum4[3]));
      m = m_new;
      // P's buffer and O are free once the previous block's second product has completed
      if (j > 0) {
        if (!wait_bar(bar(PV_DONE), (uint32_t)(j - 1) & 1u, abort_p, p.status)) {
          ok = false;
          break;
        }
        ptx::tc_fence_after();
        if (__any_sync(0xffffffffu, alpha != 1.f)) {  // rescale O by 2^(m_old - m_new)
          for (int c = 0; c < p.D; c += 32) {
            uint32_t o[32];
            ptx::tmem_ld_32x32b_x32(tmem_o + lane_addr + (uint32_t)c, o);
            ptx::tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
            ptx::tmem_st_32x32b_x32(tmem_o + lane_addr + (uint32_t)c, o);
          }
          ptx::tmem_wait_st();
        }
      }
      // P_j into shared memory: K-major, two 64-key chunks of 128-byte rows, 128-byte swizzle
#pragma unroll
      for (int jj = 0; jj < 16; ++jj) {
        const uint32_t chunk = (uint32_t)(jj >> 3), c16 = (uint32_t)(jj & 7);
        ptx::st_shared_v4(p_s + chunk * kAttnChunkBytes + my_row + ((c16 ^ swz) << 4), pw[4 * jj], pw[4 * jj + 1],
                          pw[4 * jj + 2], pw[4 * jj + 3]);
      }
      ptx::fence_proxy_async_smem();
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(bar(P_FULL));
    }
    // O / l -> global (one row of head_dim BF16 values per thread)
    if (ok && nb > 0) {
      if (wait_bar(bar(PV_DONE), (uint32_t)(nb - 1) & 1u, abort_p, p.status)) {
        ptx::tc_fence_after();
        const float inv = (l > 0.f) ? __fdividef(1.f, l) : 0.f;
        __nv_bfloat16* dst = p.O + (long long)b * p.o_stride_b + (long long)t_row * p.o_stride_t + (long long)h * p.o_stride_h;
        for (int c = 0; c < p.D; c += 32) {
          uint32_t o[32];
          ptx::tmem_ld_32x32b_x32(tmem_o + lane_addr + (uint32_t)c, o);
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
