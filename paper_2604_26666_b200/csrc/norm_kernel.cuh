// Row normalisations of the transformer blocks (Section 5.2: the MiniGPT block's layer norms, the Llama block's
// RMS norms): Y[m, :] = (X[m, :] - mean) / sqrt(var + eps) * gamma + beta   (LayerNorm, biased variance), or
//           Y[m, :] =  X[m, :] / sqrt(mean(x^2) + eps) * gamma               (RMSNorm),
// BF16 in and out, all arithmetic in FP32, one rounding at the store.
//
// HBM-bound: a row is read once and written once.  One warp owns one row and keeps it in registers as the BF16
// words it loaded (16-byte loads, CH chunks of 8 values per lane, widened on use), so mean and variance are
// taken in two exact passes over registers without reading anything twice; lanes are reduced with shuffles.
// Grid = rows / 8 warps per CTA.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "ptx.cuh"

namespace fact {

constexpr int kNormWarps = 8;

struct NormParams {
  const __nv_bfloat16* X;
  __nv_bfloat16* Y;
  const __nv_bfloat16* gamma;  // [C]
  const __nv_bfloat16* beta;   // [C] or null
  long long M;
  int C;                       // a multiple of 8, at most 256 * CH
  long long ldx, ldy;          // in elements, multiples of 8
  float eps;
};

__device__ __forceinline__ void norm_unpack8(const uint4& q, float (&f)[8]) {
  f[0] = __uint_as_float(q.x << 16);
  f[1] = __uint_as_float(q.x & 0xffff0000u);
  f[2] = __uint_as_float(q.y << 16);
  f[3] = __uint_as_float(q.y & 0xffff0000u);
  f[4] = __uint_as_float(q.z << 16);
  f[5] = __uint_as_float(q.z & 0xffff0000u);
  f[6] = __uint_as_float(q.w << 16);
  f[7] = __uint_as_float(q.w & 0xffff0000u);
}
__device__ __forceinline__ uint32_t norm_pack2(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ float norm_warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

template <int CH, bool RMS>
__global__ void __launch_bounds__(kNormWarps * 32, (CH <= 16) ? 2 : 1) fact_norm_kernel(const NormParams p) {
  ptx::grid_dependency_wait();  // (launched with programmatic stream serialization: see ptx.cuh; the successor is
                                // released when this grid's CTAs exit)
  const int lane = threadIdx.x & 31;
  const long long row = (long long)blockIdx.x * kNormWarps + (threadIdx.x >> 5);
  if (row >= p.M) return;
  const int chunks = p.C >> 3;  // 16-byte chunks in a row
  const uint4* src = reinterpret_cast<const uint4*>(p.X + row * p.ldx);
  uint4 raw[CH];
  float sum = 0.f;
#pragma unroll
  for (int c = 0; c < CH; ++c) {
    const int idx = c * 32 + lane;
    raw[c] = (idx < chunks) ? __ldg(src + idx) : make_uint4(0u, 0u, 0u, 0u);
    float x[8];
    norm_unpack8(raw[c], x);
#pragma unroll
    for (int i = 0; i < 8; ++i) sum += x[i];  // absent chunks add zeros
  }
  const float inv_c = 1.f / (float)p.C;
  const float mean = RMS ? 0.f : norm_warp_sum(sum) * inv_c;
  float sq = 0.f;
#pragma unroll
  for (int c = 0; c < CH; ++c) {
    if (c * 32 + lane < chunks) {
      float x[8];
      norm_unpack8(raw[c], x);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float d = x[i] - mean;
        sq = fmaf(d, d, sq);
      }
    }
  }
  const float rstd = rsqrtf(norm_warp_sum(sq) * inv_c + p.eps);
  uint4* dst = reinterpret_cast<uint4*>(p.Y + row * p.ldy);
  const uint4* gsrc = reinterpret_cast<const uint4*>(p.gamma);
  const uint4* bsrc = reinterpret_cast<const uint4*>(p.beta);
#pragma unroll
  for (int c = 0; c < CH; ++c) {
    const int idx = c * 32 + lane;
    if (idx < chunks) {
      float x[8], g[8], b[8], y[8];
      norm_unpack8(raw[c], x);
      norm_unpack8(__ldg(gsrc + idx), g);
      if (bsrc != nullptr) {
        norm_unpack8(__ldg(bsrc + idx), b);
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) b[i] = 0.f;
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) y[i] = fmaf((x[i] - mean) * rstd, g[i], b[i]);
      uint4 q;
      q.x = norm_pack2(y[0], y[1]);
      q.y = norm_pack2(y[2], y[3]);
      q.z = norm_pack2(y[4], y[5]);
      q.w = norm_pack2(y[6], y[7]);
      dst[idx] = q;
    }
  }
}

// Partial row sums for a normalisation that is folded into the next product instead of being applied here:
// stats[chunk][row] = (sum, sum of squares) of X[row][64 * chunk .. 64 * chunk + 64), the layout the GEMM
// epilogue writes for its own output.  One warp per row, 16 bytes per lane and step; the eight lanes of a
// 64-column chunk are reduced with shuffles.  Reads X once, writes 8 bytes per 128 read.
__global__ void __launch_bounds__(kNormWarps * 32) fact_row_stats_kernel(const __nv_bfloat16* __restrict__ X, long long M,
                                                                        int C, long long ldx, float2* __restrict__ stats) {
  const int lane = threadIdx.x & 31;
  const long long row = (long long)blockIdx.x * kNormWarps + (threadIdx.x >> 5);
  if (row >= M) return;
  const int chunks = C >> 3;
  const uint4* src = reinterpret_cast<const uint4*>(X + row * ldx);
  for (int base = 0; base < chunks; base += 32) {  // uniform trip count: the shuffles below are warp-wide
    const int idx = base + lane;
    float s1 = 0.f, s2 = 0.f;
    if (idx < chunks) {
      float x[8];
      norm_unpack8(__ldg(src + idx), x);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        s1 += x[i];
        s2 = fmaf(x[i], x[i], s2);
      }
    }
#pragma unroll
    for (int o = 1; o < 8; o <<= 1) {
      s1 += __shfl_xor_sync(0xffffffffu, s1, o);
      s2 += __shfl_xor_sync(0xffffffffu, s2, o);
    }
    if ((lane & 7) == 0 && idx < chunks) stats[(size_t)(idx >> 3) * (size_t)M + row] = make_float2(s1, s2);
  }
}

// Folding a row normalisation's scale and shift into the weights of the linear layer that follows it:
//   norm(x) . W^T + b = rstd * (x . Wf^T) - rstd * mean * colsum + bf,
//   Wf[n][k] = bf16(gamma[k] * W[n][k]),  colsum[n] = sum_k Wf[n][k],  bf[n] = bf16(b[n] + sum_k beta[k] * W[n][k]).
// (colsum is taken over the rounded Wf, the values the product will use.)  One warp per weight row, run once per model.
struct FoldParams {
  const __nv_bfloat16* W;      // [N x K], K contiguous
  __nv_bfloat16* Wf;           // [N x K]
  const __nv_bfloat16* gamma;  // [K]
  const __nv_bfloat16* beta;   // [K] or null
  const __nv_bfloat16* bias;   // [N] or null
  __nv_bfloat16* bias_out;     // [N], written iff beta is given
  float* colsum;               // [N] or null
  int N, K;
  long long ldw, ldwf;
};

__global__ void __launch_bounds__(kNormWarps * 32) fact_fold_norm_kernel(const FoldParams p) {
  const int lane = threadIdx.x & 31;
  const long long n = (long long)blockIdx.x * kNormWarps + (threadIdx.x >> 5);
  if (n >= p.N) return;
  const int chunks = p.K >> 3;
  const uint4* src = reinterpret_cast<const uint4*>(p.W + n * p.ldw);
  uint4* dst = reinterpret_cast<uint4*>(p.Wf + n * p.ldwf);
  const uint4* gsrc = reinterpret_cast<const uint4*>(p.gamma);
  const uint4* bsrc = reinterpret_cast<const uint4*>(p.beta);
  float cs = 0.f, shift = 0.f;
  for (int idx = lane; idx < chunks; idx += 32) {
    float w[8], g[8];
    norm_unpack8(__ldg(src + idx), w);
    norm_unpack8(__ldg(gsrc + idx), g);
    if (bsrc != nullptr) {
      float b[8];
      norm_unpack8(__ldg(bsrc + idx), b);
#pragma unroll
      for (int i = 0; i < 8; ++i) shift = fmaf(b[i], w[i], shift);
    }
    uint4 q;
    q.x = norm_pack2(g[0] * w[0], g[1] * w[1]);  // (a product of two BF16 values is exact in FP32: one rounding)
    q.y = norm_pack2(g[2] * w[2], g[3] * w[3]);
    q.z = norm_pack2(g[4] * w[4], g[5] * w[5]);
    q.w = norm_pack2(g[6] * w[6], g[7] * w[7]);
    dst[idx] = q;
    float f[8];
    norm_unpack8(q, f);
#pragma unroll
    for (int i = 0; i < 8; ++i) cs += f[i];
  }
  cs = norm_warp_sum(cs);
  shift = norm_warp_sum(shift);
  if (lane == 0) {
    if (p.colsum != nullptr) p.colsum[n] = cs;
    if (p.bias_out != nullptr)
      p.bias_out[n] = __float2bfloat16_rn(shift + (p.bias != nullptr ? __bfloat162float(p.bias[n]) : 0.f));
  }
}

}  // namespace fact
