// Fused multi-head attention forward for sm_100a: O = softmax(scale * Q K^T + causal mask) V, BF16 in and out,
// FP32 scores / probabilities / accumulation, grouped queries (several query heads share one key/value head).
//
// One CTA owns 128 query positions of one (batch, query head) and walks the key/value sequence in blocks of 128
// keys with the online-softmax recurrence (a reference maximum m and row sum l per row; the output accumulator is
// rescaled by 2^(m_old - m_new) only when the block maximum exceeds m by more than 8, so probabilities stay below
// 2^8 and the final division by l removes the stale reference exactly).  Roles:
//   warp 0      TMA producer: the Q tile once, then K and V blocks into two three-stage rings
//   warp 1      MMA issuer:
//                 S(j)  = Q K_j^T      tcgen05.mma, M = 128, N = 128, K = head_dim, both operands from shared memory,
//                                      into one of two score buffers in tensor memory
//                 O    += P(j) V_j     tcgen05.mma, M = 128, N = head_dim, K = 128, A = P(j) read from tensor memory
//   warps 2-9   softmax: two threads per query row (warps w and w + 4 share a lane quarter and split the block's
//               keys in halves): tcgen05.ld the scores, mask, maximum (exchanged between the two halves through
//               shared memory), exponentials, row sum; rescale O in tensor memory when needed; tcgen05.st the BF16
//               probabilities over the first 64 columns of the score buffer they came from; at the end O / l -> global
// S(j+1) is issued before the softmax of block j starts, so the softmax warps never wait for the tensor pipe in
// steady state and the pipe works on S(j+1) and O += P(j-1) V while they compute.  Tensor memory (512 columns):
// S/P buffer 0 at 0, buffer 1 at 128, O at 256.  P(j) may overwrite S(j) because both threads of a row have read
// their scores before either stores (the exchange of the maxima orders them), and S(j+2) is issued after
// O += P(j) V on the same in-order pipe.  Every mbarrier wait is bounded, as in the GEMM kernel.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "gemm_kernel.cuh"
#include "ptx.cuh"

namespace fact {

constexpr int kAttnThreads = 320;   // 10 warps
constexpr int kAttnBlockQ = 128;    // query rows per CTA (= TMEM lanes)
constexpr int kAttnBlockK = 128;    // keys per block
constexpr int kAttnStages = 3;      // K and V ring depth
constexpr uint32_t kAttnChunkBytes = 128 * 128;  // one 64-column chunk of a 128-row tile, 128-byte rows
constexpr float kAttnRescaleThreshold = 8.f;     // log2 units

struct AttnParams {
  int B, Tq, Tk, Hq, Hkv, D;  // D = 64 or 128
  int causal;
  float scale_log2;           // softmax scale * log2(e)
  int q_tiles;                // ceil(Tq / 128)
  __nv_bfloat16* O;
  long long o_stride_b, o_stride_t, o_stride_h;  // in elements; head_dim is contiguous
  uint64_t kmajor_desc;       // UMMA descriptor template, K-major 128B-swizzled tiles (Q, K)
  uint64_t v_desc;            // UMMA descriptor template, V as an N-major operand
  uint32_t idesc_s, idesc_pv;
  int* status;                // [0] error word, [2..17] eight 64-bit profile counters (debug bit 256)
  int debug;
};

// Shared-memory carve-up (dynamic, 1024-byte aligned): Q | K[stages] | V[stages] | exchange (2 x 2 x 128 floats) |
// barriers and control words
__host__ __device__ constexpr uint32_t attn_tile_bytes(int D) { return (uint32_t)(D / 64) * kAttnChunkBytes; }
__host__ __device__ constexpr uint32_t attn_smem_bytes(int D) {
  return attn_tile_bytes(D) * (1u + 2u * kAttnStages) + 2048u + 24u * 8u + 16u;
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
  // With debug bit 256 the first CTA counts where its cycles go: [0] CTA cycles, [1] CTA nanoseconds, [2] / [3]
  // cycles warp 2 waited for scores / spent on them, [4] its blocks, [5] its rescales, [6] cycles the MMA warp
  // waited for probabilities, [7] cycles from entry to the first scores.
  const bool prof = (p.debug & 256) && blockIdx.x == 0;
  const bool trace = (p.debug & 512) && blockIdx.x == 0;
  long long* prof_c = reinterpret_cast<long long*>(p.status + 2);
  const long long t_entry = prof ? clock64() : 0;
  const unsigned long long ns_entry = prof ? ptx::globaltimer_ns() : 0ull;
  const uint32_t tile_bytes = attn_tile_bytes(p.D);
  const uint32_t q_s = smem_base;
  const uint32_t k_s0 = q_s + tile_bytes;
  const uint32_t v_s0 = k_s0 + (uint32_t)kAttnStages * tile_bytes;
  const uint32_t xch_off = (1u + 2u * kAttnStages) * tile_bytes;  // [parity][half][row] floats
  const uint32_t bar_base = smem_base + xch_off + 2048u;
  const uint32_t ctrl_off = xch_off + 2048u + 24u * 8u;
  float* xch = reinterpret_cast<float*>(smem_raw + xch_off);
  volatile uint32_t* tmem_holder_p = reinterpret_cast<volatile uint32_t*>(smem_raw + ctrl_off);
  volatile int* abort_p = reinterpret_cast<volatile int*>(smem_raw + ctrl_off + 4);
  enum {
    Q_FULL = 0,
    K_FULL = 1,
    V_FULL = K_FULL + kAttnStages,
    K_EMPTY = V_FULL + kAttnStages,
    V_EMPTY = K_EMPTY + kAttnStages,
    S_FULL = V_EMPTY + kAttnStages,  // two: one per score buffer
    P_FULL = S_FULL + 2,
    PV_DONE = P_FULL + 1,
    N_BARS = PV_DONE + 1
  };
  static_assert(N_BARS <= 24, "barrier area");
  auto bar = [&](int i) { return bar_base + 8u * (uint32_t)i; };

  if (threadIdx.x < N_BARS) {
    const int i = (int)threadIdx.x;
    ptx::mbar_init(bar(i), i == P_FULL ? 8u : 1u);  // one arrival per softmax warp
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
  const uint32_t tmem_o = tmem_base + 256u;

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
    if (ptx::elect_one()) {
      ptx::mbar_arrive_expect_tx(bar(Q_FULL), tile_bytes);
      for (int c = 0; c < chunks; ++c) ptx::tma_load_4d(q_s + c * kAttnChunkBytes, &tmQ, bar(Q_FULL), c * 64, h, t0, b);
    }
    int s = 0;
    uint32_t par = 1;  // an empty slot's first wait passes
    for (int j = 0; j < nb; ++j) {
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
      if (++s == kAttnStages) {
        s = 0;
        par ^= 1u;
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    bool ok = wait_all(bar(Q_FULL), 0);
    ptx::tc_fence_after();
    int ks = 0, vs = 0;          // ring slots of the next K block to multiply and the next V block
    uint32_t kpar = 0, vpar = 0;
    long long prof_p_wait = 0, prof_kv_wait = 0;
    auto issue_s = [&](int j) -> bool {  // S(j) = Q K_j^T into score buffer j & 1; releases K_j when done
      const long long tk = prof ? clock64() : 0;
      if (!wait_all(bar(K_FULL + ks), kpar)) return false;
      if (prof) prof_kv_wait += clock64() - tk;
      ptx::tc_fence_after();
      if (ptx::elect_one()) {
        const uint32_t kaddr = k_s0 + (uint32_t)ks * tile_bytes;
        const uint32_t d = tmem_base + (uint32_t)(j & 1) * 128u;
        for (int kk = 0; kk < ((p.debug & 1) ? 0 : p.D / kUmmaK); ++kk) {
          const uint32_t off = (uint32_t)(kk >> 2) * kAttnChunkBytes + (uint32_t)(kk & 3) * 32u;
          const uint64_t adesc = p.kmajor_desc | (uint64_t)(((q_s + off) >> 4) & 0x3fffu);
          const uint64_t bdesc = p.kmajor_desc | (uint64_t)(((kaddr + off) >> 4) & 0x3fffu);
          ptx::umma_bf16<1>(d, adesc, bdesc, p.idesc_s, kk > 0 ? 1u : 0u);
        }
        ptx::umma_commit<1>(bar(S_FULL + (j & 1)));
        ptx::umma_commit<1>(bar(K_EMPTY + ks));
      }
      if (++ks == kAttnStages) {
        ks = 0;
        kpar ^= 1u;
      }
      return true;
    };
    if (ok && nb > 0) ok = issue_s(0);
    for (int j = 0; ok && j < nb; ++j) {
      // score buffer (j + 1) & 1 held P(j-1), which O += P(j-1) V (issued in the previous iteration) reads first
      if (j + 1 < nb && !issue_s(j + 1)) break;
      if (trace && lane == 0 && (j == 6 || j == 7)) prof_c[j == 6 ? 0 : 3] = clock64() - t_entry;
      const long long tw = prof ? clock64() : 0;
      if (!wait_all(bar(P_FULL), (uint32_t)j & 1u)) break;
      const long long tv = prof ? clock64() : 0;
      if (prof) prof_p_wait += tv - tw;
      if (trace && lane == 0 && j == 6) prof_c[1] = clock64() - t_entry;
      if (!wait_all(bar(V_FULL + vs), vpar)) break;
      if (prof) prof_kv_wait += clock64() - tv;
      ptx::tc_fence_after();
      if (ptx::elect_one()) {  // O += P(j) V_j
        const uint32_t vaddr = v_s0 + (uint32_t)vs * tile_bytes;
        const uint32_t p_t = tmem_base + (uint32_t)(j & 1) * 128u;  // BF16 pairs: 8 columns per 16 keys
        for (int kk = 0; kk < ((p.debug & 2) ? 0 : kAttnBlockK / kUmmaK); ++kk) {
          const uint64_t bdesc = p.v_desc | (uint64_t)(((vaddr + (uint32_t)kk * 2048u) >> 4) & 0x3fffu);
          ptx::umma_bf16_ts(tmem_o, p_t + (uint32_t)kk * 8u, bdesc, p.idesc_pv, (j > 0 || kk > 0) ? 1u : 0u);
        }
        ptx::umma_commit<1>(bar(V_EMPTY + vs));
        ptx::umma_commit<1>(bar(PV_DONE));
      }
      if (trace && lane == 0 && j == 6) prof_c[2] = clock64() - t_entry;
      if (++vs == kAttnStages) {
        vs = 0;
        vpar ^= 1u;
      }
    }
    if (prof && !trace && lane == 0) {
      prof_c[6] = prof_p_wait;
      prof_c[7] = prof_kv_wait;
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------ softmax warps: two threads per query row
    const int half = (warp - 2) >> 2;  // which 64 keys of every block this thread owns
    const int q4 = warp & 3;           // the TMEM lane quarter this warp may access
    const int row = q4 * 32 + lane;
    const int t_row = t0 + row;
    const uint32_t lane_addr = (uint32_t)(q4 * 32) << 16;
    const uint32_t pair_bar = 1u + (uint32_t)q4;  // named barrier of this warp and its partner (warp +- 4)
    const int o_cols = p.D / 2;                   // output columns this thread rescales and stores
    const uint32_t o_addr = tmem_o + lane_addr + (uint32_t)(half * o_cols);
    float m = -INFINITY;  // reference maximum of scale_log2 * score the exponentials are taken against
    float l = 0.f;        // this thread's part of the running sum of 2^(scale_log2 * score - m)
    bool ok = true;       // warp-uniform; a warp whose wait gave up keeps meeting its partner at the named barrier
    long long prof_wait = 0, prof_busy = 0, prof_first = 0, prof_rescales = 0;
    for (int j = 0; j < nb; ++j) {
      const long long tw = prof ? clock64() : 0;
      if (ok) ok = wait_all(bar(S_FULL + (j & 1)), ((uint32_t)j >> 1) & 1u);
      const long long tb = prof ? clock64() : 0;
      if (prof) {
        prof_wait += tb - tw;
        if (j == 0) prof_first = tb - t_entry;
      }
      if (trace && warp == 2 && lane == 0 && (j == 6 || j == 7)) prof_c[j == 6 ? 4 : 6] = clock64() - t_entry;
      const uint32_t buf = tmem_base + lane_addr + (uint32_t)(j & 1) * 128u;
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
      float* xj = xch + (j & 1) * 256;
      xj[half * 128 + row] = hm;
      ptx::named_bar_sync(pair_bar, 64);
      if (!ok) continue;
      const float mx = fmaxf(hm, xj[(half ^ 1) * 128 + row]) * p.scale_log2;  // scale > 0
      // Move the reference maximum only when this block exceeds it by more than the threshold (always from -inf);
      // both threads of a row take the same decision from the same numbers.
      if (__any_sync(0xffffffffu, mx > m + kAttnRescaleThreshold)) {
        const float m_new = fmaxf(m, mx);
        const float alpha = ptx::ex2_approx(m - ((m_new == -INFINITY) ? 0.f : m_new));
        l *= alpha;
        m = m_new;
        if (prof) ++prof_rescales;
        if (j > 0) {
          // O is rescaled between O += P(j-1) V, which must have completed, and O += P(j) V, which waits for P(j)
          ok = wait_all(bar(PV_DONE), (uint32_t)(j - 1) & 1u);
          if (!ok) continue;
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
          float p0 = fmaf(__uint_as_float(sraw[c][i]), p.scale_log2, -m_use);
          float p1 = fmaf(__uint_as_float(sraw[c][i + 1]), p.scale_log2, -m_use);
          if (!(p.debug & 4)) {
            p0 = ptx::ex2_approx(p0);
            p1 = ptx::ex2_approx(p1);
          }
          sum4[(i >> 1) & 3] += p0 + p1;
          pw[c * 16 + (i >> 1)] = pack_bf16x2(p0, p1);
        }
      l += (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
      // P(j) over the first 64 columns of S(j): lane = row, column c holds keys 2c and 2c + 1
      ptx::tmem_st_32x32b_x32(buf + (uint32_t)half * 32u, pw);
      ptx::tmem_wait_st();
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(bar(P_FULL));
      if (prof) prof_busy += clock64() - tb;
      if (trace && warp == 2 && lane == 0 && (j == 6 || j == 7)) prof_c[j == 6 ? 5 : 7] = clock64() - t_entry;
    }
    if (prof && !trace && warp == 2 && lane == 0) {
      prof_c[2] = prof_wait;
      prof_c[3] = prof_busy;
      prof_c[4] = nb;
      prof_c[5] = prof_rescales;
    }
    // the row sum is the sum of the two halves' (the exchange buffer of the parity the last block did not use)
    float* xl = xch + (nb & 1) * 256;
    xl[half * 128 + row] = l;
    ptx::named_bar_sync(pair_bar, 64);
    l += xl[(half ^ 1) * 128 + row];
    // O / l -> global: each thread stores its half of the row's head_dim BF16 values
    if (ok && nb > 0 && wait_all(bar(PV_DONE), (uint32_t)(nb - 1) & 1u)) {
      ptx::tc_fence_after();
      const float inv = (l > 0.f) ? __fdividef(1.f, l) : 0.f;
      __nv_bfloat16* dst = p.O + (long long)b * p.o_stride_b + (long long)t_row * p.o_stride_t +
                           (long long)h * p.o_stride_h + half * o_cols;
      for (int c = 0; c < o_cols; c += 32) {
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
  if (prof && !trace && threadIdx.x == 0) {
    prof_c[0] = clock64() - t_entry;
    prof_c[1] = (long long)(ptx::globaltimer_ns() - ns_entry);
  }
}

}  // namespace fact
