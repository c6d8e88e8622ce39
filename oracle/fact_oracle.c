/*
 * fact_oracle.c -- TEST INFRASTRUCTURE, not product code.
 *
 * A plain FP64 CPU statement of what the fused-epilogue GEMM family computes:
 * the matrix products of the paper's Section 5.1 "Benchmark problems"
 * (Problem 1: C = A x B; Problem 3: C[b] = A[b] x B[b]; Problem 6: C = A x B
 * with a very long K) and the linear layers of its Section 5.2 transformer
 * blocks (MiniGPT pattern p2: Linear + GELU, Linear with a standard epilogue;
 * Llama pattern p2: SiLU(gate) x up, down projection), each followed by the
 * epilogue the block applies to it.
 *
 * Only the tests, the smoke check and the CPU-baseline / reference legs of the
 * benchmark may call this file.  It shares nothing with the CUDA library: its
 * own BF16 widening, its own epilogue formulas, no common headers.
 *
 * Inputs are BF16 bit patterns (uint16_t), exactly the bits the GPU receives.
 * Every value is widened to double without rounding, every product of two
 * widened BF16 values is exact in double (8 x 8 significant bits), and every
 * output element is the sum of its K products taken in ascending k, in
 * double, with no intermediate rounding to a narrower type.  The output is
 * double.
 *
 * Two loop orders are provided.  `fact_oracle_linear` with variant 0 is the
 * definition written out as a triple loop.  Variant 1 interchanges loops over
 * small row/column blocks so that it runs at tens of GFLOP/s, but still adds
 * the products of each output element one by one in ascending k, so both
 * variants return bit-identical results (a CPU test asserts this on shapes
 * that span several blocks and ragged tails).  Variant 1 is the one timed as
 * the CPU baseline.
 *
 * Parity pins (tests/test_oracle_pins.py): library dgemm on the widened
 * inputs, identity / all-ones / one-hot closed forms, exact integer inputs,
 * exact rational brute force on tiny shapes, library GELU(tanh) / SiLU,
 * GELU's odd-part identity and asymptotes.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* Epilogue selector.  The numbering is this file's own; the test harness maps
 * names to these numbers. */
enum {
  ORACLE_EPI_NONE = 0,           /* y = acc                                   (Section 5.1, Problems 1/3/6) */
  ORACLE_EPI_BIAS = 1,           /* y = acc + bias[n]                         (a Linear layer)              */
  ORACLE_EPI_BIAS_RELU = 2,      /* y = max(acc + bias[n], 0)                                               */
  ORACLE_EPI_BIAS_GELU_TANH = 3, /* y = gelu_tanh(acc + bias[n])              (Section 5.2, MiniGPT p2 GEMM 1) */
  ORACLE_EPI_SILU_GATE = 4,      /* y = silu(acc[m,n]) * acc[m,N_out+n]       (Section 5.2, Llama p2 GEMM 1)   */
  ORACLE_EPI_BIAS_RESIDUAL = 5   /* y = acc + bias[n] + R[m,n], bias optional (GEMM 2 feeding the residual add) */
};

/* Layout of the second operand. */
enum {
  ORACLE_B_KN = 0, /* B[K x N], n contiguous: torch.matmul(A, B)      */
  ORACLE_B_NK = 1  /* W[N x K], k contiguous: torch.nn.Linear.weight  */
};

/* BF16 is the upper half of an IEEE binary32; widening is exact. */
static inline double bf16_bits_to_f64(uint16_t bits) {
  uint32_t u = ((uint32_t)bits) << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return (double)f;
}

double fact_oracle_bf16_to_f64(uint16_t bits) { return bf16_bits_to_f64(bits); }

/* Round a double to the nearest BF16 (ties to even) in ONE rounding, straight
 * from the double.  Going through float first could round twice. */
uint16_t fact_oracle_round_bf16(double x) {
  if (x != x) return 0x7fc0;
  uint16_t sign = signbit(x) ? 0x8000 : 0;
  double a = fabs(x);
  if (a == 0.0) return sign;
  if (isinf(a)) return (uint16_t)(sign | 0x7f80);
  int e;
  double frac = frexp(a, &e); /* a = frac * 2^e, frac in [0.5, 1) */
  int exp_unb = e - 1;        /* a = (2 frac) * 2^exp_unb, 2 frac in [1, 2) */
  if (exp_unb < -126) exp_unb = -126; /* subnormal range: fixed quantum 2^-133 */
  /* quantum = 2^(exp_unb - 7): BF16 keeps 7 fraction bits */
  double q = ldexp(a, -(exp_unb - 7)); /* a / quantum, in [128, 256) for normals */
  double fl = floor(q);
  double rem = q - fl;
  uint64_t n = (uint64_t)fl;
  if (rem > 0.5 || (rem == 0.5 && (n & 1))) n += 1;
  /* n is now an integer count of quanta; rebuild the value and re-split it */
  double r = ldexp((double)n, exp_unb - 7);
  float rf = (float)r; /* exact: r has at most 8 significant bits */
  if (isinf(rf)) return (uint16_t)(sign | 0x7f80);
  uint32_t u;
  memcpy(&u, &rf, sizeof u);
  return (uint16_t)(sign | (uint16_t)(u >> 16));
}

/* GELU, tanh form: 0.5 z (1 + tanh( sqrt(2/pi) (z + 0.044715 z^3) )). */
static inline double gelu_tanh_f64(double z) {
  const double c = 0.79788456080286535588; /* sqrt(2/pi) */
  return 0.5 * z * (1.0 + tanh(c * (z + 0.044715 * z * z * z)));
}

/* SiLU: g * sigmoid(g) = g / (1 + exp(-g)). */
static inline double silu_f64(double g) { return g / (1.0 + exp(-g)); }

double fact_oracle_gelu_tanh(double z) { return gelu_tanh_f64(z); }
double fact_oracle_silu(double g) { return silu_f64(g); }

/* The epilogue applied to one output element.
 * acc  : the K-term sum for column n (for SILU_GATE: the gate column n)
 * acc2 : for SILU_GATE the K-term sum for column N_out + n (the "up" column) */
static inline double apply_epilogue(int epi, double acc, double acc2, int has_bias, double bias, double resid) {
  switch (epi) {
    case ORACLE_EPI_NONE: return acc;
    case ORACLE_EPI_BIAS: return acc + bias;
    case ORACLE_EPI_BIAS_RELU: {
      double z = acc + bias;
      return z > 0.0 ? z : 0.0;
    }
    case ORACLE_EPI_BIAS_GELU_TANH: return gelu_tanh_f64(acc + bias);
    case ORACLE_EPI_SILU_GATE: return silu_f64(acc) * acc2;
    case ORACLE_EPI_BIAS_RESIDUAL: return (has_bias ? acc + bias : acc) + resid;
    default: return NAN;
  }
}

static inline double b_elem(const uint16_t* W, int64_t ldw, int layout, int64_t k, int64_t n) {
  return bf16_bits_to_f64(layout == ORACLE_B_KN ? W[k * ldw + n] : W[n * ldw + k]);
}

/*
 * fact_oracle_linear
 *
 *   for b in [0, batch), for each selected row m, for n in [0, N_out):
 *     acc  = sum_{k=0..K-1} X[b][m,k] * W[b][k, n]
 *     acc2 = sum_{k=0..K-1} X[b][m,k] * W[b][k, N_out + n]     (SILU_GATE only)
 *     Y[b][i, n] = epilogue(acc, acc2, bias[n], R[b][m, n])
 *
 * Arguments (all host pointers, leading dimensions and strides in ELEMENTS):
 *   X      BF16 bits, row-major [M x K], row stride ldx, batch stride strideX
 *   W      BF16 bits; layout ORACLE_B_KN: [K x Nw] row stride ldw;
 *          ORACLE_B_NK: [Nw x K] row stride ldw.  Nw = N_out, or 2*N_out for
 *          SILU_GATE (gate columns first, then up columns).
 *   bias   BF16 bits [N_out] or NULL (shared by all batches)
 *   R      BF16 bits [M x N_out], row stride ldr, batch stride strideR, or NULL
 *   rows   NULL -> all M rows, n_rows ignored; else n_rows row indices in
 *          [0, M): output row i holds row rows[i]
 *   Y      double, [n_out_rows x N_out] per batch, row stride ldy, batch
 *          stride strideY
 *   variant 0 = triple loop, 1 = interchanged loops (same per-element order)
 *   nthreads <= 0 -> OpenMP default
 * Returns 0, or a negative number for an invalid argument.
 */
int fact_oracle_linear(int64_t batch, int64_t M, int64_t N_out, int64_t K,
                       const uint16_t* X, int64_t ldx, int64_t strideX,
                       const uint16_t* W, int64_t ldw, int64_t strideW, int w_layout,
                       const uint16_t* bias,
                       const uint16_t* R, int64_t ldr, int64_t strideR,
                       int epi,
                       const int64_t* rows, int64_t n_rows,
                       double* Y, int64_t ldy, int64_t strideY,
                       int variant, int nthreads) {
  if (batch < 0 || M < 0 || N_out < 0 || K < 0) return -1;
  if (epi < ORACLE_EPI_NONE || epi > ORACLE_EPI_BIAS_RESIDUAL) return -2;
  if (w_layout != ORACLE_B_KN && w_layout != ORACLE_B_NK) return -3;
  const int needs_bias = (epi == ORACLE_EPI_BIAS || epi == ORACLE_EPI_BIAS_RELU || epi == ORACLE_EPI_BIAS_GELU_TANH);
  if (needs_bias && !bias) return -4;
  if (epi == ORACLE_EPI_BIAS_RESIDUAL && !R) return -5;
  if (epi == ORACLE_EPI_SILU_GATE && bias) return -6;
  const int64_t n_out_rows = rows ? n_rows : M;
  if (rows) {
    for (int64_t i = 0; i < n_rows; ++i)
      if (rows[i] < 0 || rows[i] >= M) return -7;
  }
  if (batch == 0 || n_out_rows == 0 || N_out == 0) return 0;
#ifdef _OPENMP
  if (nthreads <= 0) nthreads = omp_get_max_threads();
#else
  nthreads = 1;
#endif
  const int gate = (epi == ORACLE_EPI_SILU_GATE);
  const int has_bias = bias != NULL;

  if (variant == 0) {
    /* The definition, written out. */
#pragma omp parallel for collapse(2) num_threads(nthreads) schedule(static)
    for (int64_t b = 0; b < batch; ++b) {
      for (int64_t i = 0; i < n_out_rows; ++i) {
        const int64_t m = rows ? rows[i] : i;
        const uint16_t* Xb = X + b * strideX;
        const uint16_t* Wb = W + b * strideW;
        for (int64_t n = 0; n < N_out; ++n) {
          double acc = 0.0, acc2 = 0.0;
          for (int64_t k = 0; k < K; ++k) {
            const double x = bf16_bits_to_f64(Xb[m * ldx + k]);
            acc += x * b_elem(Wb, ldw, w_layout, k, n);
            if (gate) acc2 += x * b_elem(Wb, ldw, w_layout, k, N_out + n);
          }
          const double bv = has_bias ? bf16_bits_to_f64(bias[n]) : 0.0;
          const double rv = (epi == ORACLE_EPI_BIAS_RESIDUAL) ? bf16_bits_to_f64(R[b * strideR + m * ldr + n]) : 0.0;
          Y[b * strideY + i * ldy + n] = apply_epilogue(epi, acc, acc2, has_bias, bv, rv);
        }
      }
    }
    return 0;
  }
  if (variant != 1) return -8;

  /* Same sums, loops interchanged.  A task owns RB output rows x CB output
   * columns.  It walks k upward in chunks of KC; inside a chunk it widens the
   * needed X and W entries to double once, then for every k (ascending) adds
   * x[r][k] * w[k][n] to acc[r][n].  Each acc[r][n] therefore receives its K
   * products in ascending k, exactly as in the triple loop. */
  enum { RB = 8, CB = 256, KC = 256 };
  const int64_t n_rb = (n_out_rows + RB - 1) / RB;
  const int64_t n_cb = (N_out + CB - 1) / CB;
  const int n_acc = gate ? 2 : 1;
  int failed = 0;
#pragma omp parallel num_threads(nthreads)
  {
    double* wbuf = (double*)malloc(sizeof(double) * (size_t)KC * CB * n_acc);
    double* xbuf = (double*)malloc(sizeof(double) * (size_t)RB * KC);
    double* acc = (double*)malloc(sizeof(double) * (size_t)RB * CB * n_acc);
    if (!wbuf || !xbuf || !acc) {
#pragma omp atomic write
      failed = 1;
    } else {
#pragma omp for collapse(3) schedule(dynamic, 1)
      for (int64_t b = 0; b < batch; ++b) {
        for (int64_t rb = 0; rb < n_rb; ++rb) {
          for (int64_t cb = 0; cb < n_cb; ++cb) {
            const uint16_t* Xb = X + b * strideX;
            const uint16_t* Wb = W + b * strideW;
            const int64_t i0 = rb * RB, n0 = cb * CB;
            const int nr = (int)((n_out_rows - i0) < RB ? (n_out_rows - i0) : RB);
            const int nc = (int)((N_out - n0) < CB ? (N_out - n0) : CB);
            for (int t = 0; t < RB * CB * n_acc; ++t) acc[t] = 0.0;
            for (int64_t k0 = 0; k0 < K; k0 += KC) {
              const int kc = (int)((K - k0) < KC ? (K - k0) : KC);
              for (int r = 0; r < nr; ++r) {
                const int64_t m = rows ? rows[i0 + r] : (i0 + r);
                for (int k = 0; k < kc; ++k) xbuf[r * KC + k] = bf16_bits_to_f64(Xb[m * ldx + k0 + k]);
              }
              for (int h = 0; h < n_acc; ++h) {
                const int64_t ncol0 = n0 + (int64_t)h * N_out;
                if (w_layout == ORACLE_B_KN) {
                  for (int k = 0; k < kc; ++k)
                    for (int c = 0; c < nc; ++c)
                      wbuf[((size_t)h * KC + k) * CB + c] = bf16_bits_to_f64(Wb[(k0 + k) * ldw + ncol0 + c]);
                } else {
                  for (int c = 0; c < nc; ++c)
                    for (int k = 0; k < kc; ++k)
                      wbuf[((size_t)h * KC + k) * CB + c] = bf16_bits_to_f64(Wb[(ncol0 + c) * ldw + k0 + k]);
                }
              }
              for (int h = 0; h < n_acc; ++h) {
                for (int k = 0; k < kc; ++k) {
                  const double* wrow = wbuf + ((size_t)h * KC + k) * CB;
                  for (int r = 0; r < nr; ++r) {
                    const double x = xbuf[r * KC + k];
                    double* arow = acc + ((size_t)h * RB + r) * CB;
#pragma omp simd
                    for (int c = 0; c < nc; ++c) arow[c] += x * wrow[c];
                  }
                }
              }
            }
            for (int r = 0; r < nr; ++r) {
              const int64_t m = rows ? rows[i0 + r] : (i0 + r);
              for (int c = 0; c < nc; ++c) {
                const int64_t n = n0 + c;
                const double a1 = acc[(size_t)r * CB + c];
                const double a2 = gate ? acc[((size_t)RB + r) * CB + c] : 0.0;
                const double bv = has_bias ? bf16_bits_to_f64(bias[n]) : 0.0;
                const double rv =
                    (epi == ORACLE_EPI_BIAS_RESIDUAL) ? bf16_bits_to_f64(R[b * strideR + m * ldr + n]) : 0.0;
                Y[b * strideY + (i0 + r) * ldy + n] = apply_epilogue(epi, a1, a2, has_bias, bv, rv);
              }
            }
          }
        }
      }
    }
    free(wbuf);
    free(xbuf);
    free(acc);
  }
  return failed ? -9 : 0;
}

int fact_oracle_max_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}
