// Device-side helpers of the tuner's verify gate (Section 4.2: a candidate is verified before it is benchmarked).
// The tuner runs the library's default configuration once, keeps a copy of its output, and compares every
// candidate's output with that copy on the device, element by element, before the candidate is timed.  A candidate
// that differs by more than two correct FP32-accumulated results can differ is recorded and never timed.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace fact {

struct TuneViewParams {
  const void* C;      // the output as the GEMM call addressed it
  long long ldc, strideC;
  int batch, M, N;
  int f32;            // 1: FP32 elements, 0: BF16
};

// A view's element at flat index i over (batch, M, N), widened to FP32.
__device__ __forceinline__ float tune_load(const TuneViewParams& v, long long i, long long* off_out = nullptr) {
  const int n = (int)(i % v.N);
  const long long r = i / v.N;
  const int m = (int)(r % v.M);
  const int b = (int)(r / v.M);
  const long long off = (long long)b * v.strideC + (long long)m * v.ldc + n;
  if (off_out) *off_out = off;
  return v.f32 ? reinterpret_cast<const float*>(v.C)[off]
               : __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(v.C)[off]);
}

// Overwrites the valid (batch, M, N) region of the output with NaNs: what a candidate fails to write then fails the
// comparison instead of passing on the previous candidate's values.
__global__ void fact_tune_poison_kernel(TuneViewParams v) {
  const long long total = (long long)v.batch * v.M * v.N;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    long long off;
    (void)tune_load(v, i, &off);
    if (v.f32) reinterpret_cast<uint32_t*>(const_cast<void*>(v.C))[off] = 0x7fc00000u;
    else reinterpret_cast<uint16_t*>(const_cast<void*>(v.C))[off] = 0x7fc0u;
  }
}

// Copies the valid (batch, M, N) region of the output into a dense FP32 array and adds up sum |x| (double, atomics;
// the value only sets the scale of the tolerance, so the order of the additions does not matter).
__global__ void fact_tune_snapshot_kernel(TuneViewParams v, float* dense, double* abs_sum) {
  const long long total = (long long)v.batch * v.M * v.N;
  double local = 0.0;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const float x = tune_load(v, i);
    dense[i] = x;
    local += fabs((double)x);
  }
  for (int o = 16; o > 0; o >>= 1) local += __shfl_xor_sync(0xffffffffu, local, o);
  if ((threadIdx.x & 31) == 0 && local != 0.0) atomicAdd(abs_sum, local);
}

// result[0] = number of elements outside the tolerance (or not finite), result[1] = worst |c - r| / tolerance as
// float bits (non-negative floats order like their bit patterns, so atomicMax on the bits is a float maximum).
// Tolerance per element: rel * |r| + floor_abs.  `perturb` != 0 is the gate's own test: the reference is read with
// a deliberate error in its first 64 columns of its first 128 rows, so that a correct candidate must be rejected.
__global__ void fact_tune_compare_kernel(TuneViewParams v, const float* dense_ref, float rel, float floor_abs,
                                         int perturb, unsigned int* result) {
  const long long total = (long long)v.batch * v.M * v.N;
  unsigned int bad = 0;
  float worst = 0.f;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const float c = tune_load(v, i);
    float r = dense_ref[i];
    if (perturb) {
      const int n = (int)(i % v.N);
      const int m = (int)((i / v.N) % v.M);
      if (m < 128 && n < 64) r = 1.25f * r + 64.f * floor_abs;
    }
    const float tol = rel * fabsf(r) + floor_abs;
    const float ratio = fabsf(c - r) / tol;
    if (!(ratio <= 1.f)) ++bad;  // (a NaN compares false)
    worst = fmaxf(worst, isfinite(ratio) ? ratio : 3.0e38f);
  }
  for (int o = 16; o > 0; o >>= 1) {
    bad += __shfl_xor_sync(0xffffffffu, bad, o);
    worst = fmaxf(worst, __shfl_xor_sync(0xffffffffu, worst, o));
  }
  if ((threadIdx.x & 31) == 0) {
    if (bad) atomicAdd(result, bad);
    atomicMax(result + 1, __float_as_uint(worst));
  }
}

}  // namespace fact
