/*
 * libfact -- fused-epilogue BF16 GEMMs for NVIDIA B200 (sm_100a).  C ABI.
 *
 * The library computes the GEMM family of the paper's evaluation: the three
 * matrix-product problems of Section 5.1 "Benchmark problems" (Problem 1: one
 * square product, data-parallel tiles; Problem 3: a batch of independent
 * products; Problem 6: a product with a very long K, cut along K) and the
 * linear layers that Section 5.2 fuses with their element-wise successors
 * (MiniGPT pattern p2: Linear + GELU, Linear + standard epilogue; Llama
 * pattern p2: SiLU(gate) x up, down projection).
 *
 * Conventions shared by every entry point
 *   - All matrix pointers are DEVICE pointers on the handle's device.  Only
 *     the handle, the status/size out-parameters, config structs and file
 *     paths are host memory.
 *   - Matrices are row-major.  Leading dimensions (ld*) and batch strides are
 *     in ELEMENTS.  Inputs are BF16; products are accumulated in FP32; the
 *     output is BF16 (round to nearest even, once, after the epilogue) or
 *     FP32.
 *   - Operand loads go through TMA, hence: every operand base pointer (A/X,
 *     B/W) must be 16-byte aligned and its leading dimension and batch stride
 *     a multiple of 8 elements.  Output and residual rows are written/read in
 *     16-byte vectors when the pointer is 16-byte aligned and the leading
 *     dimension a multiple of 8 (BF16) / 4 (FP32) elements; otherwise element
 *     by element (slower, still correct).  M, N, K themselves are arbitrary.
 *   - Ownership: the caller owns every buffer and the stream.  The library
 *     never allocates or frees device memory on a call path; split-K scratch
 *     is a caller-provided workspace sized by fact_workspace_bytes.  The handle
 *     owns a small device status area (status word, counters, stream-K flags),
 *     a 32 KB device table for grouped calls and the tuner's table.
 *   - Calls only enqueue work on `cuda_stream` (a cudaStream_t passed as
 *     void*; NULL = the legacy default stream) and return; results are valid
 *     in stream order.
 *   - Errors: a status code is returned; argument errors are detected before
 *     anything is launched and leave the outputs untouched.  There is no CPU
 *     fallback and no library GEMM fallback: on a device that is not sm_100
 *     fact_create fails with FACT_ERR_ARCH.
 *   - A handle must not be used from two host threads at once.
 *   - M == 0 or N == 0 (or batch == 0) is a successful no-op.  K == 0 applies
 *     the epilogue to a zero accumulator.
 */
#ifndef FACT_H_
#define FACT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct fact_handle_s* fact_handle_t;

typedef enum {
  FACT_OK = 0,
  FACT_ERR_INVALID_ARG = 1,         /* null pointer, negative size, bad enum, inconsistent arguments */
  FACT_ERR_BAD_ALIGNMENT = 2,       /* operand pointer / leading dimension breaks the 16-byte TMA rule */
  FACT_ERR_UNSUPPORTED = 3,         /* a config the kernels cannot run (tile shape, smem/TMEM budget) */
  FACT_ERR_ARCH = 4,                /* device is not sm_100 */
  FACT_ERR_WORKSPACE_TOO_SMALL = 5, /* split-K needs more scratch than was passed */
  FACT_ERR_CUDA = 6,                /* a CUDA runtime/driver call failed */
  FACT_ERR_DEVICE_TIMEOUT = 7       /* a bounded device-side wait expired (reported by fact_device_status) */
} fact_status_t;

/* Element-wise work fused into the GEMM epilogue (computed in FP32 on the
 * accumulator, before the single rounding to the output type):
 *   NONE            y = acc                                   (Section 5.1 problems)
 *   BIAS            y = acc + bias[n]
 *   BIAS_RELU       y = max(acc + bias[n], 0)
 *   BIAS_GELU_TANH  z = acc + bias[n];  y = 0.5 z (1 + tanh(sqrt(2/pi) (z + 0.044715 z^3)))
 *                                                             (Section 5.2, MiniGPT p2 GEMM 1)
 *   SILU_GATE       y = silu(acc[m, n]) * acc[m, N_out + n],  silu(g) = g / (1 + exp(-g))
 *                   W carries 2*N_out columns: gate columns first, then up columns
 *                                                             (Section 5.2, Llama p2 GEMM 1)
 *   BIAS_RESIDUAL   y = acc + bias[n] + R[m, n]   (bias may be NULL)
 *                                                             (GEMM 2 of both blocks + the residual add)
 *   BIAS_SOFTMAX    z = acc[m, :] + bias;  y[m, n] = exp(z[n] - max z) / sum_j exp(z[j] - max z)   (bias may be NULL)
 *                   the softmax of every output row, inside the tile that holds the row: N_out <= 256, no K split,
 *                   no stream-K, register stores (FACT_ERR_UNSUPPORTED otherwise)
 *                                                             (Table 1: the "GEMM-Softmax" fusion) */
typedef enum {
  FACT_EPI_NONE = 0,
  FACT_EPI_BIAS = 1,
  FACT_EPI_BIAS_RELU = 2,
  FACT_EPI_BIAS_GELU_TANH = 3,
  FACT_EPI_SILU_GATE = 4,
  FACT_EPI_BIAS_RESIDUAL = 5,
  FACT_EPI_BIAS_SOFTMAX = 6
} fact_epilogue_t;

typedef enum { FACT_OUT_BF16 = 0, FACT_OUT_F32 = 1 } fact_out_t;

/* Storage of the second operand. */
typedef enum {
  FACT_B_KN = 0, /* B[K x N], N contiguous  (torch.matmul(A, B))      */
  FACT_B_NK = 1  /* W[N x K], K contiguous  (torch.nn.Linear.weight)  */
} fact_blayout_t;

/* Which entry point a workspace / tuning query is about. */
typedef enum {
  FACT_OP_GEMM = 0,
  FACT_OP_GEMM_BATCHED = 1,
  FACT_OP_GEMM_SPLITK = 2,
  FACT_OP_LINEAR = 3,
  FACT_OP_LINEAR_FP8 = 4
} fact_op_t;

/* One kernel configuration.  A zero field means "let the library choose".
 *   tile_m       128 (one CTA per tile) or 256 (a 2-CTA cluster per tile; then cta_group must be 2)
 *   tile_n       accumulator columns per tile, a multiple of 16 in [32, 256] (FACT_B_KN: multiple of 64;
 *                SILU_GATE: multiple of 32, half gate + half up)
 *   tile_k       elements of K per pipeline stage: 64 for BF16 operands, 128 for FP8 (one 128-byte swizzle row)
 *   stages       depth of the shared-memory ring, 2..8, limited by 227 KB
 *   cta_group    1 or 2
 *   raster_group G > 0: the scheduler walks groups of G m-tiles (their slab of A/X stays in L2 while the
 *                n-tiles stream by); G < 0: groups of |G| n-tiles (a slab of B/W stays); 0: the library's
 *                traffic model chooses
 *   split_k      number of K slices, >= 1 (> 1 needs a workspace); or a stream-K schedule (Section 4.2, Action 2:
 *                the third grid-level policy): -1 cuts the tiles of the last, partial wave along K and deals their
 *                k-blocks out evenly over all CTAs, so that every SM ends at the same time; -2 does so with the
 *                partial wave plus one full wave (fewer pieces per tile when the partial wave is small).  The
 *                tiles of the full waves before stay data-parallel with the fused epilogue.  A tile cut this way
 *                is finished by the CTA that holds its first k-block: the CTAs with the other pieces park their
 *                FP32 accumulators in the workspace (one tile per CTA, fact_workspace_bytes), the finishing CTA
 *                adds them to its own in CTA order and applies the epilogue -- a fixed order, so results are
 *                reproducible bit for bit, and bounded waits like everywhere else.  Where there is nothing to cut
 *                (whole waves, K == 0, an output the staged store cannot write) the call is data-parallel.
 *                Stream-K calls through one handle must be stream-ordered with respect to each other (they share
 *                the handle's flags) and must not share a workspace while they overlap.
 *                0 (the library's choice) is one slice, except for an untuned fact_gemm / fact_linear (and for
 *                fact_gemm_splitk called with splits = 0, whose choice is always the library's) whose tiles
 *                are few and whose K is long (say 256 x 4096 x 14336): there the library's cost model may take
 *                the K slices that fill the SMs in one wave, if the call brings the workspace that
 *                fact_workspace_bytes reports for it -- without it the same call runs in one slice, like a table
 *                entry -- or 2 / 4 / 8 slices as a cluster (schedule 3), which needs no workspace.  The choices
 *                differ in the order of the FP32 additions, not in anything else.
 *   store_mode   0 = library default, 1 = direct register stores (any alignment), 2 = shared-memory staged
 *                tensor stores, 3 = the staged epilogue's arithmetic with every row stored from registers in
 *                32-byte pieces (Y 32-byte aligned, ldy and N_out multiples of 32 bytes, whole data-parallel
 *                tiles: no K slices, stream-K, groups or row sums; pays when K is long, FACT_ERR_UNSUPPORTED
 *                where it cannot run)
 *   schedule     how data-parallel tiles reach the CTAs (the grid-level policy of Section 4.2, Action 2): 0 = the
 *                library's choice, 1 = static: a persistent grid of one CTA group per SM (pair of SMs), group g
 *                takes tiles g, g + G, g + 2G, ...; 2 = dynamic: the grid has one cluster per tile, the clusters
 *                that get an SM keep it and obtain further tiles by cancelling the launch of clusters that have
 *                not started (clusterlaunchcontrol; a twelfth warp per CTA keeps one request in flight ahead of
 *                the tile in progress), so a CTA group that falls behind simply takes fewer tiles.  Which group
 *                computes a tile never changes a value: every tile is summed by one group in the same order.
 *                Dynamic scheduling serves whole tiles only (no K slices, stream-K, row sums, folded
 *                normalisation, register row stores or row softmax: FACT_ERR_UNSUPPORTED with those), and is
 *                the static schedule when all tiles fit one wave.
 *                3 = the K slices of a tile as one thread-block cluster (the K-sliced regime of Section 5.2,
 *                Problem 6, for products of few tiles and long K): split_k = 2, 4 or 8 CTAs share a 128-row tile
 *                (tile_m 128, cta_group 1), or split_k = 2 or 4 CTA pairs share a 256-row tile (tile_m 256,
 *                cta_group 2; a cluster holds at most 8 CTAs); tile_n is a multiple of 32 * split_k.  Each slice
 *                multiplies its part of K with its own plain loads and its own accumulator -- no operand is
 *                loaded twice -- and the slices are added up through distributed shared memory: slice r sends
 *                block j of its accumulator's columns to slice j, which adds the blocks in the order of the workspace reduction
 *                (same bits as the same split_k through a workspace), applies the epilogue and stores.  No
 *                workspace, no partial planes in global memory, no grid-wide barrier.  Column-wise epilogues on
 *                BF16 operands (not SILU_GATE, row softmax, 8-bit operands, groups, row sums or a folded
 *                normalisation: FACT_ERR_UNSUPPORTED).  An untuned fact_gemm / fact_linear may take this schedule
 *                on its own (see split_k). */
typedef struct {
  int tile_m, tile_n, tile_k, stages, cta_group, raster_group, split_k, store_mode, schedule;
} fact_config_t;

/* Create / destroy a handle bound to CUDA device `device`.  fact_create makes
 * that device current, checks for sm_100, allocates the handle's two small device
 * buffers and resolves the driver's tensor-map encoder.  These two calls and the tuner
 * (fact_tune, which is off the per-call path) are the only ones that allocate or free
 * device memory. */
fact_status_t fact_create(fact_handle_t* handle, int device);
fact_status_t fact_destroy(fact_handle_t handle);

/* Static, never NULL. */
const char* fact_status_string(fact_status_t status);

/* Scratch bytes the given problem needs with `cfg` (NULL = the library's own
 * choice, the same one the compute call will make with cfg == NULL).  0 when
 * no K split is used.  N is the number of OUTPUT columns; `epilogue` matters
 * because SILU_GATE partials are twice as wide. */
fact_status_t fact_workspace_bytes(fact_handle_t handle, fact_op_t op, int64_t batch, int64_t M, int64_t N, int64_t K,
                                   fact_epilogue_t epilogue, fact_blayout_t b_layout, fact_out_t out_type,
                                   const fact_config_t* cfg, size_t* bytes);

/* C[M x N] = A[M x K] . B          (Section 5.1, Problem 1: data-parallel tiles)
 * A: BF16 [M x K], lda.  B: BF16, [K x N] (FACT_B_KN, ldb >= N) or [N x K]
 * (FACT_B_NK, ldb >= K).  C: BF16 or FP32 [M x N], ldc.  The library may
 * still split K when cfg (or its own choice) says so; then `workspace` must
 * hold fact_workspace_bytes(...) bytes, else it may be NULL/0. */
fact_status_t fact_gemm(fact_handle_t handle, int64_t M, int64_t N, int64_t K, const void* A, int64_t lda,
                        const void* B, int64_t ldb, fact_blayout_t b_layout, void* C, int64_t ldc,
                        fact_out_t out_type, const fact_config_t* cfg, void* workspace, size_t workspace_bytes,
                        void* cuda_stream);

/* C = A . B for operands and a result that live in HOST memory -- the call a caller without device-resident data
 * makes (the drop-in replacement of the paper's problem statement, Section 3, for tensors that have not been
 * moved yet).  A, B, C are host pointers (row-major, leading dimensions in elements, same layouts and output
 * types as fact_gemm); `device_scratch` is device memory of at least fact_gemm_host_scratch_bytes(...) bytes
 * (the dense device copies of A, B and C, plus the workspace the product's configuration wants), 256-byte
 * aligned, owned by the caller.  The call enqueues and returns: a copy of A and B to the
 * scratch on the handle's copy-in stream, the product on its compute stream, the copy of C back on its copy-out
 * stream, chained by events.  It is ordered after everything enqueued on `cuda_stream` before the call.
 * fact_gemm_host_wait(handle, stream) makes `stream` wait for the copy-out of every host-buffer call made so far:
 * C_host is valid once that stream reaches that point (synchronise it before reading C on the host; the wait is
 * a call of its own so that a train of products does not serialise on the caller's stream).  Consecutive calls
 * overlap -- the copy-in of one runs during the product of the one before and the copy-out of the one before that
 * -- provided they are given different scratch buffers; a call waits for the copy-out of the last call that used
 * the same scratch.  The copies are
 * asynchronous only for page-locked host memory.  The first call through a handle creates the three streams
 * and the events (no device memory).  Product configuration as in fact_gemm with cfg (NULL = the library's choice);
 * a scratch that holds the operands but not the configuration's workspace makes a tuned entry run without K slices
 * or stream-K, and a caller's own such configuration fail with FACT_ERR_WORKSPACE_TOO_SMALL. */
fact_status_t fact_gemm_host_scratch_bytes(fact_handle_t handle, int64_t M, int64_t N, int64_t K,
                                           fact_blayout_t b_layout, fact_out_t out_type, const fact_config_t* cfg,
                                           size_t* bytes);
fact_status_t fact_gemm_host(fact_handle_t handle, int64_t M, int64_t N, int64_t K, const void* A_host, int64_t lda,
                             const void* B_host, int64_t ldb, fact_blayout_t b_layout, void* C_host, int64_t ldc,
                             fact_out_t out_type, const fact_config_t* cfg, void* device_scratch,
                             size_t device_scratch_bytes, void* cuda_stream);
fact_status_t fact_gemm_host_wait(fact_handle_t handle, void* cuda_stream);

/* C[b] = A[b] . B[b] for b in [0, batch)      (Section 5.1, Problem 3: batched)
 * Batch b of an operand starts stride* elements after batch b-1. */
fact_status_t fact_gemm_batched(fact_handle_t handle, int64_t batch, int64_t M, int64_t N, int64_t K, const void* A,
                                int64_t lda, int64_t strideA, const void* B, int64_t ldb, int64_t strideB,
                                fact_blayout_t b_layout, void* C, int64_t ldc, int64_t strideC, fact_out_t out_type,
                                const fact_config_t* cfg, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* C = A . B with K cut into `splits` contiguous slices (0 = library's choice)
 *                                              (Section 5.1, Problem 6: long K)
 * Each (tile, slice) CTA writes an FP32 partial to the workspace.  After a grid-wide barrier in the
 * tail of the same kernel (the grid never exceeds the SM count, so all CTAs are resident; the wait is
 * bounded like every other device wait) all threads share out the output and add the partials of
 * each element in a fixed order: four sums over slices q, q+4, q+8, ... (ascending, q = 0..3), combined
 * as (s0 + s1) + (s2 + s3); then the epilogue and the store.  Slice boundaries and the order of every
 * addition depend only on (M, N, K, config), so repeated calls return bit-identical results.  Split-K
 * calls through one handle must be stream-ordered with respect to each other (they share the handle's
 * barrier counters), and must not share a workspace while they overlap. */
fact_status_t fact_gemm_splitk(fact_handle_t handle, int64_t M, int64_t N, int64_t K, const void* A, int64_t lda,
                               const void* B, int64_t ldb, fact_blayout_t b_layout, void* C, int64_t ldc,
                               fact_out_t out_type, int splits, const fact_config_t* cfg, void* workspace,
                               size_t workspace_bytes, void* cuda_stream);

/* fact_gemm_splitk for callers that must not allocate device memory.  (The paper has no counterpart
 * of this entry point; it exists for integration, not for the method.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a region whose device memory
 * is owned by a pool or arena that forbids side allocations, in a latency-critical loop that may not
 * take the allocator's locks or implicit synchronisation, or in a process that has handed all of its
 * memory budget to someone else.  Such a caller can create neither a handle (fact_create allocates
 * the status word) nor a split-K workspace.  This call needs neither: it takes no handle, and its
 * scratch is a fixed 16 MiB array that is part of the library's device image (so every GPU that loads
 * the library carries those 16 MiB until the process exits).
 *
 * Computes C[M x N] = A[M x K] . B exactly like fact_gemm_splitk (same kernels, same fixed-order
 * reduction, same argument rules for A, B, C, leading dimensions, b_layout, out_type; `splits` = 0
 * lets the library choose), on CUDA device `device`, enqueued on `cuda_stream`.  The caller still
 * owns and passes the inputs and the output.  It calls no cudaMalloc / cudaFree and no allocating
 * library routine.
 *
 * Limits and rules:
 *   - the FP32 partial planes, splits * M * round_up(N, 4) * 4 bytes, must fit in 16 MiB; a larger
 *     problem (or split count) is refused with FACT_ERR_WORKSPACE_TOO_SMALL and nothing is launched
 *     -- pass fewer splits, or use fact_gemm_splitk with your own workspace;
 *   - the first call on a device resolves the device addresses of the static arrays and a few device
 *     properties (it makes `device` current for the duration of the call); make that first call
 *     outside any stream capture;
 *   - all calls on a device share the one scratch array and it keeps whatever the last call left in
 *     it.  Nothing in it has to start at zero (every partial that is read is written first by the
 *     same call), but two calls that overlap on the GPU -- different streams, or different host
 *     threads -- race on it and both results are garbage: keep calls on one device in one stream
 *     order;
 *   - a device-side wait that expires (every wait in the kernels is bounded) is recorded in a status
 *     word that is likewise static and per device; the output of that call is then undefined.  The
 *     call itself is asynchronous and cannot report it: ask fact_gemm_splitk_static_status. */
fact_status_t fact_gemm_splitk_static(int device, int64_t M, int64_t N, int64_t K, const void* A, int64_t lda,
                                      const void* B, int64_t ldb, fact_blayout_t b_layout, void* C, int64_t ldc,
                                      fact_out_t out_type, int splits, void* cuda_stream);

/* The fact_device_status of fact_gemm_splitk_static (no counterpart in the paper either): synchronise
 * `cuda_stream`, write the static status word of `device` to *status (FACT_OK or
 * FACT_ERR_DEVICE_TIMEOUT) and clear it.  0 if no static call has run on that device yet.  Like the
 * call it serves it allocates nothing: one 4-byte copy, and memsets after a give-up. */
fact_status_t fact_gemm_splitk_static_status(int device, void* cuda_stream, int* status);

/* Y[M x N_out] = epilogue(X[M x K] . W)        (Section 5.2: fused linear layers)
 * W: FACT_B_NK [Nw x K] (nn.Linear weight) or FACT_B_KN [K x Nw]; Nw = N_out,
 * or 2*N_out for SILU_GATE.  bias: BF16 [N_out]; required by BIAS, BIAS_RELU,
 * BIAS_GELU_TANH, optional for BIAS_RESIDUAL, must be NULL otherwise.
 * residual: BF16 [M x N_out] with ldr; required by BIAS_RESIDUAL, must be NULL
 * otherwise.  Y may alias residual only if pointer and leading dimension are
 * identical. */
fact_status_t fact_linear(fact_handle_t handle, int64_t M, int64_t N_out, int64_t K, const void* X, int64_t ldx,
                          const void* W, int64_t ldw, fact_blayout_t w_layout, const void* bias,
                          const void* residual, int64_t ldr, void* Y, int64_t ldy, fact_out_t out_type,
                          fact_epilogue_t epilogue, const fact_config_t* cfg, void* workspace,
                          size_t workspace_bytes, void* cuda_stream);

/* Grouped linear layer: the rows of X and Y are cut into `groups` consecutive row groups and group g is multiplied
 * by its own weight matrix,      Y[rows of g, :] = epilogue(X[rows of g, :] . W[g])
 * (Table 1 lists "Grouped GEMM" among the Level-3 kernels of the registry for both architectures: a list of
 * products of different sizes in one launch, as a mixture-of-experts layer needs after its tokens have been sorted
 * by expert).  group_rows: HOST array of `groups` row counts (>= 0, at most 4096 groups); M is their sum.
 * X: BF16 [M x K], ldx.  W[g]: BF16 at W + g * strideW elements, [Nw x K] (FACT_B_NK) or [K x Nw] (FACT_B_KN), ldw;
 * strideW a multiple of 8.  bias [N_out] (shared by the groups), residual [M x N_out], Y, out_type, epilogue as in
 * fact_linear.  One launch: tiles never cross a group boundary (the last tile of a group is ragged), all tiles are
 * data-parallel, the output is stored by row-predicated 16-byte stores -- staged through shared memory so that
 * they are whole 128-byte rows when Y is 16-byte aligned with ldy and N_out multiples of 16 bytes, straight from
 * registers otherwise or with cfg->store_mode == 1 (the group table travels to a buffer of
 * the handle in stream order, so grouped calls through one handle must be stream-ordered with respect to each
 * other, and not inside a stream capture: the table is copied from pageable host memory).  cfg: tile shape, pair
 * size, stages and store mode only (K slices, stream-K and the row softmax are refused with
 * FACT_ERR_UNSUPPORTED).  groups == 0 or M == 0 is a successful no-op. */
fact_status_t fact_linear_grouped(fact_handle_t handle, int groups, const int64_t* group_rows, int64_t N_out, int64_t K,
                                  const void* X, int64_t ldx, const void* W, int64_t ldw, int64_t strideW,
                                  fact_blayout_t w_layout, const void* bias, const void* residual, int64_t ldr, void* Y,
                                  int64_t ldy, fact_out_t out_type, fact_epilogue_t epilogue, const fact_config_t* cfg,
                                  void* cuda_stream);

/* The grouped linear layer on FP8 E4M3 operands (Table 1: "FP8 Grouped GEMM"): fact_linear_grouped with the
 * operand rules of fact_linear_fp8 -- X [M x K] and W[g] [Nw x K] one byte per element, K-major, ldx, ldw and
 * strideW multiples of 16, one FP32 `scale` for all groups applied to the accumulator before the epilogue. */
fact_status_t fact_linear_grouped_fp8(fact_handle_t handle, int groups, const int64_t* group_rows, int64_t N_out,
                                      int64_t K, const void* X, int64_t ldx, const void* W, int64_t ldw,
                                      int64_t strideW, float scale, const void* bias, const void* residual, int64_t ldr,
                                      void* Y, int64_t ldy, fact_out_t out_type, fact_epilogue_t epilogue,
                                      const fact_config_t* cfg, void* cuda_stream);

/* Y[M x N_out] = epilogue(scale * X[M x K] . W^T)  with FP8 operands      (Section 3, the pattern table indexed by
 * rule, data type and architecture; Table 1 lists an FP8 GEMM among the Level-1 kernels the registry holds)
 * X: FP8 E4M3 [M x K], one byte per element (the OCP "e4m3fn" format: no infinities, S.1111.111 is NaN, largest
 * magnitude 448); W: FP8 E4M3 [Nw x K] as torch.nn.Linear stores it (Nw = N_out, or 2 * N_out for SILU_GATE).
 * Products are exact and accumulated in FP32 on the tensor cores (tcgen05.mma.kind::f8f6f4).  `scale` (host
 * value, finite) multiplies the accumulator before anything else -- the product of the operands' per-tensor
 * scales; the paper fixes no scaling convention.  bias, residual, Y, out_type, epilogue, cfg and the workspace
 * are those of fact_linear (bias and residual stay BF16).  ldx and ldw are in elements and must be multiples of
 * 16 (rows of 16-byte multiples for TMA); X and W 16-byte aligned.  The tuner's key for this entry point is
 * FACT_OP_LINEAR_FP8 (fact_get_config, fact_workspace_bytes, fact_tune with X, W as A, B and FACT_B_NK). */
fact_status_t fact_linear_fp8(fact_handle_t handle, int64_t M, int64_t N_out, int64_t K, const void* X, int64_t ldx,
                              const void* W, int64_t ldw, float scale, const void* bias, const void* residual,
                              int64_t ldr, void* Y, int64_t ldy, fact_out_t out_type, fact_epilogue_t epilogue,
                              const fact_config_t* cfg, void* workspace, size_t workspace_bytes, void* cuda_stream);

/* O = softmax(scale * Q K^T + causal mask) V, fused           (Section 5.2, pattern p1: fused multi-head
 * attention -- causal for the MiniGPT block; grouped queries, 32 query heads over 8 key/value heads of
 * dimension 128, for the Llama block, where the paper first expands K/V with repeat_interleave: here the
 * shared key/value heads are read in place)
 * Q: BF16 [batch][seq_q][heads_q][head_dim], K and V: BF16 [batch][seq_kv][heads_kv][head_dim], O: BF16 like Q,
 * each addressed by three strides in elements (batch, token, head; head_dim itself is contiguous), so the
 * operands may be views into a fused QKV projection or stored heads-first.  Query head h uses key/value
 * head h / (heads_q / heads_kv).  Scores and probabilities are FP32, P is rounded to BF16 for the second
 * product, O is accumulated in FP32 and rounded once.  causal != 0 masks keys j > i and requires
 * seq_q == seq_kv; scale <= 0 means 1 / sqrt(head_dim).
 * Requirements: head_dim 64 or 128; heads_q a multiple of heads_kv; all four pointers 16-byte aligned and
 * every stride a multiple of 8 elements (operands are read and O is written through TMA).  Errors: FACT_ERR_UNSUPPORTED for another head_dim or causal with seq_q != seq_kv,
 * FACT_ERR_BAD_ALIGNMENT, FACT_ERR_INVALID_ARG; nothing is launched on an error.  batch == 0 or
 * seq_q == 0 is a successful no-op. */
fact_status_t fact_attention(fact_handle_t handle, int64_t batch, int64_t seq_q, int64_t seq_kv, int64_t heads_q,
                             int64_t heads_kv, int64_t head_dim, const void* Q, int64_t q_stride_batch,
                             int64_t q_stride_token, int64_t q_stride_head, const void* K, int64_t k_stride_batch,
                             int64_t k_stride_token, int64_t k_stride_head, const void* V, int64_t v_stride_batch,
                             int64_t v_stride_token, int64_t v_stride_head, void* O, int64_t o_stride_batch,
                             int64_t o_stride_token, int64_t o_stride_head, int causal, float scale,
                             void* cuda_stream);

/* Row normalisation of the transformer blocks (Section 5.2: the MiniGPT block is a pre-norm GPT block with
 * layer norms, the Llama block uses RMS norms; the paper leaves them in the surrounding graph, they are here so
 * that a whole block runs through this library):
 *   FACT_NORM_LAYER:  Y[m,:] = (X[m,:] - mean) / sqrt(var + eps) * gamma + beta    (biased variance)
 *   FACT_NORM_RMS:    Y[m,:] =  X[m,:] / sqrt(mean(X[m,:]^2) + eps) * gamma
 * X, Y: BF16 [M x C] with leading dimensions ldx, ldy (elements); gamma: BF16 [C]; beta: BF16 [C] or NULL
 * (must be NULL for FACT_NORM_RMS).  FP32 arithmetic, one rounding at the store.  C a multiple of 8 in
 * [8, 8192]; pointers 16-byte aligned, ldx and ldy multiples of 8.  Y may alias X. */
typedef enum { FACT_NORM_LAYER = 0, FACT_NORM_RMS = 1 } fact_norm_t;
fact_status_t fact_norm(fact_handle_t handle, fact_norm_t kind, int64_t M, int64_t C, const void* X, int64_t ldx,
                        const void* gamma, const void* beta, float eps, void* Y, int64_t ldy, void* cuda_stream);

/* A row normalisation between two linear layers without its own pass over the activations (Table 1 lists
 * "GEMM-LayerNorm-GEMM fusion" among the registry's Level-2 kernels; Section 5.2's blocks have a norm between
 * the attention output projection and the MLP).  Three pieces:
 *
 *  1. the call that PRODUCES the activations also leaves partial sums of every output row:
 *     row_stats_out[c][m] = (sum, sum of squares) of the stored BF16 values Y[m][64c .. 64c+64), as FP32 pairs,
 *     [ceil(N_out / 64)][M][2] floats (fact_row_stats computes the same array for a tensor that no call of this
 *     library produced);
 *  2. the scale and shift of the normalisation are folded into the next layer's weights once (fact_fold_norm):
 *     Wf[n][k] = bf16(gamma[k] W[n][k]), colsum[n] = sum_k Wf[n][k], bf[n] = bf16(b[n] + sum_k beta[k] W[n][k]);
 *  3. the call that CONSUMES them multiplies the raw activations by Wf and corrects the accumulator per row,
 *         norm(x) . W^T + b  =  rstd[m] * (x . Wf^T)[m][n] - rstd[m] * mean[m] * colsum[n] + bf[n],
 *     with mean = S1 / K, rstd = 1 / sqrt(S2 / K - mean^2 + eps) (FACT_XNORM_LAYER), or mean = 0 (FACT_XNORM_RMS,
 *     no colsum), S1, S2 the sums of x_row_stats over the K / 64 chunks; then the epilogue as usual.
 *
 * Numerics: x is not centred before the product, so the two terms cancel when |mean| is large against the
 * standard deviation: the absolute error grows like (|mean| / std) * 2^-8 * |output|.  Residual streams of
 * pre-norm transformers have |mean| well below std; for data that does not, use fact_norm.
 *
 * Limits: fact_linear_ex only (one BF16 product, batch 1); the staged (TMA) store path must be in use (Y 16-byte
 * aligned, ldy a multiple of 8) and K not sliced (cfg->split_k 0, 1 or negative); row_stats_out needs a BF16
 * output; FACT_XNORM_LAYER needs N_out a multiple of 64, w_colsum 16-byte aligned, and is not combined with
 * SILU_GATE (FACT_XNORM_RMS is); BIAS_SOFTMAX takes neither; a stream-K choice (cfg->split_k < 0) is ignored, the tiles run
 * data-parallel.  FACT_ERR_UNSUPPORTED otherwise. */
typedef enum { FACT_XNORM_NONE = 0, FACT_XNORM_LAYER = 1, FACT_XNORM_RMS = 2 } fact_xnorm_t;
typedef struct fact_linear_ext {
  float* row_stats_out;      /* device, [ceil(N_out / 64)][M][2], or NULL: partial row sums of Y */
  fact_xnorm_t x_norm;       /* normalisation of X's rows folded into this product */
  const float* x_row_stats;  /* device, [ceil(K / 64)][M][2]: partial row sums of X (x_norm != NONE) */
  const float* w_colsum;     /* device, [N_out]: column sums of the folded weights (FACT_XNORM_LAYER) */
  float eps;                 /* the normalisation's epsilon, >= 0 */
} fact_linear_ext_t;

/* fact_linear with the extras of fact_linear_ext_t (ext == NULL: exactly fact_linear). */
fact_status_t fact_linear_ex(fact_handle_t handle, int64_t M, int64_t N_out, int64_t K, const void* X, int64_t ldx,
                             const void* W, int64_t ldw, fact_blayout_t w_layout, const void* bias,
                             const void* residual, int64_t ldr, void* Y, int64_t ldy, fact_out_t out_type,
                             fact_epilogue_t epilogue, const fact_linear_ext_t* ext, const fact_config_t* cfg,
                             void* workspace, size_t workspace_bytes, void* cuda_stream);

/* stats[c][m] = (sum, sum of squares) over X[m][64c .. 64c+64) in FP32, [ceil(C / 64)][M][2] floats: the row sums
 * fact_linear_ex consumes, for an X that came from elsewhere.  X: BF16 [M x C], 16-byte aligned, ldx and C
 * multiples of 8; stats 8-byte aligned. */
fact_status_t fact_row_stats(fact_handle_t handle, int64_t M, int64_t C, const void* X, int64_t ldx, float* stats,
                             void* cuda_stream);

/* Fold a normalisation's gamma [K] (and beta [K], or NULL for an RMS norm) into the weights W [N_w x K] (BF16,
 * FACT_B_NK layout, ldw) of the linear layer that follows it: writes W_folded [N_w x K] (ldwf; may alias W when
 * ldwf == ldw), colsum [N_w] FP32 (or NULL), and -- iff beta is given -- bias_folded [N_w] BF16 from bias [N_w]
 * (or NULL for no bias).  For SILU_GATE pass the stacked gate and up rows, N_w = 2 N_out.  Run once per model;
 * K a multiple of 8, pointers 16-byte aligned, ldw and ldwf multiples of 8. */
fact_status_t fact_fold_norm(fact_handle_t handle, int64_t N_w, int64_t K, const void* W, int64_t ldw,
                             const void* gamma, const void* beta, const void* bias, void* W_folded, int64_t ldwf,
                             float* colsum, void* bias_folded, void* cuda_stream);

/* One pre-norm transformer block, forward, as a chain of this library's kernels on one stream (Section 5.2:
 * the two Level-3 blocks the paper composes from its attention and MLP patterns):
 *     n1  = norm1(x)
 *     qkv = n1 . Wqkv^T (+ bqkv)                       [tokens x (heads_q + 2 heads_kv) head_dim], Q | K | V
 *     a   = causal attention over the Q, K, V slices of qkv, read in place (grouped queries if heads_kv < heads_q)
 *     x1  = a . Wo^T (+ bo) + x                        fused residual
 *     n2  = norm2(x1)
 *     h   = gelu_tanh(n2 . W1^T + b1)                  FACT_BLOCK_GPT:   W1 [ffn x hidden]
 *         = silu(n2 . Wg^T) * (n2 . Wu^T)              FACT_BLOCK_LLAMA: W1 [2 ffn x hidden], gate rows first
 *     y   = h . W2^T (+ b2) + x1                       fused residual
 * FACT_BLOCK_GPT uses layer norms (gamma, beta) and biases; FACT_BLOCK_LLAMA uses RMS norms and no biases (the
 * bias and beta pointers must be NULL).  The paper's block descriptions name no positional rotation of Q and K;
 * none is applied.  All tensors BF16, row-major, dense: x, y [batch * seq x hidden]; weights [out x in] as
 * torch.nn.Linear stores them; every intermediate is rounded to BF16 once, where it is stored.
 * hidden must equal heads_q * head_dim; head_dim 64 or 128; hidden and ffn multiples of 8.
 * `workspace` (device) holds the intermediates; fact_block_workspace_bytes gives its size.  y may alias x. */
typedef enum { FACT_BLOCK_GPT = 0, FACT_BLOCK_LLAMA = 1 } fact_block_kind_t;
typedef struct {
  fact_block_kind_t kind;
  int64_t batch, seq, hidden, heads_q, heads_kv, head_dim, ffn;
  float eps;
  const void *norm1_gamma, *norm1_beta; /* [hidden] */
  const void *wqkv, *bqkv;              /* [(heads_q + 2 heads_kv) head_dim x hidden], [(heads_q + 2 heads_kv) head_dim] */
  const void *wo, *bo;                  /* [hidden x hidden], [hidden] */
  const void *norm2_gamma, *norm2_beta; /* [hidden] */
  const void *w1, *b1;                  /* GPT [ffn x hidden], [ffn]; LLAMA [2 ffn x hidden] (gate | up), NULL */
  const void *w2, *b2;                  /* [hidden x ffn], [hidden] */
} fact_block_t;
size_t fact_block_workspace_bytes(const fact_block_t* block);
/* Where fact_block_forward keeps its intermediates, as byte offsets into the workspace (each dense, BF16,
 * row-major [tokens x columns]): offsets[0] the norm output (n1, later overwritten by n2; hidden columns),
 * [1] qkv ((heads_q + 2 heads_kv) head_dim columns), [2] a (hidden), [3] x1 (hidden), [4] h (ffn).  After a
 * call they still hold that call's values, which lets a caller inspect or check every stage.  Returns
 * FACT_ERR_INVALID_ARG for an inconsistent descriptor. */
fact_status_t fact_block_workspace_offsets(const fact_block_t* block, size_t offsets[5]);
fact_status_t fact_block_forward(fact_handle_t handle, const fact_block_t* block, const void* x, void* y,
                                 void* workspace, size_t workspace_bytes, void* cuda_stream);

/* The configuration the library would run for this problem when cfg == NULL
 * (its tuned entry if fact_tune / fact_tune_cache_load provided one, else a
 * heuristic).  The paper's counterpart is the lookup in its pattern table
 * (Section 3; Section 4.2, Action 6). */
fact_status_t fact_get_config(fact_handle_t handle, fact_op_t op, int64_t batch, int64_t M, int64_t N, int64_t K,
                              fact_epilogue_t epilogue, fact_blayout_t b_layout, fact_out_t out_type,
                              fact_config_t* cfg_out);

/* On-device tile-configuration search for one problem (Section 4.2, Actions 4 and 5: every candidate is
 * verified, then benchmarked; the sweep covers tile shapes, pipeline depth, cluster size, grid schedule and
 * store path, and the best verified candidate is kept).  Runs on the given device buffers (the output is
 * overwritten; it ends holding the winner's result), synchronises the stream, stores the winner in the
 * handle's table and returns it.
 *   - Feasibility: candidates over the shared-memory or TMEM budget, or that the kernels cannot run on this
 *     problem, are rejected on the host and never launched; candidates that need more than `workspace_bytes`
 *     of scratch are skipped.  (The paper's sweep launches them and records the failures, Section 5.1.)
 *   - Verify gate: the library's default configuration is run once and a dense FP32 copy of its output kept;
 *     before a candidate is timed, its output (written over NaNs) is compared with that copy element by
 *     element on the device, tolerance 2^-7 |ref| + 1e-3 mean|ref| for BF16 outputs and 1e-3 (|ref| +
 *     mean|ref|) for FP32 outputs -- above what two correct FP32-accumulated results in different summation
 *     orders differ by (one BF16 ulp; for FP32 outputs half the stated tolerance: a single 131072-term
 *     accumulator and a sliced sum of the same products differ by 3.4e-4), far below what a dropped k-block or
 *     a misplaced tile changes.  A candidate outside it is recorded as FACT_TUNE_VERIFY_FAILED, is never
 *     timed and can never win.
 *   - Timing: `warmup` + `iters` launches per candidate (0 = 5 and 20, the paper's protocol in Section 5.1),
 *     CUDA events, each time multiplied by the SM clock the kernel itself measured (a time in cycles: the
 *     clock of a power-limited part drifts by more than candidates differ) and ranked relative to the default
 *     configuration timed right before and after; the five fastest are timed five more times in alternation
 *     and the best median wins.  Warm L2 by default: launches back to back.
 * fact_tune_ex takes options (NULL = the defaults of fact_tune):
 *   cold_l2       1: a buffer twice the size of L2 is overwritten before every timed launch and every launch
 *                 is timed by an event pair of its own -- the protocol of a benchmark that flushes L2
 *   verify        0 switches the verify gate off (default 1)
 *   inject_fault  index (in sweep order) of a candidate whose verification is run against a deliberately
 *                 wrong reference, -1 for none: the gate's own test -- that candidate must come back
 *                 FACT_TUNE_VERIFY_FAILED although its output is right
 *   records       caller's array of max_records entries (may be NULL): one per candidate in sweep order --
 *                 the configuration as resolved, what happened to it, its time per launch (ms), that time
 *                 relative to the default configuration's, and worst |cand - ref| / tolerance; *n_records
 *                 receives the number of candidates (which may exceed max_records)
 * This is the one compute-path call that allocates: for its own duration it holds the FP32 reference copy
 * (4 bytes per output element), its events and, in cold mode, the L2-sized buffer.  It returns
 * FACT_ERR_UNSUPPORTED when the residual aliases the output (every candidate would read its predecessor's
 * result) and when no candidate could be timed. */
typedef enum {
  FACT_TUNE_TIMED = 0,         /* verified and timed */
  FACT_TUNE_INFEASIBLE = 1,    /* rejected on the host (budget / unsupported combination): never launched */
  FACT_TUNE_NO_WORKSPACE = 2,  /* needs more scratch than the caller passed: never launched */
  FACT_TUNE_LAUNCH_FAILED = 3, /* a launch returned an error or a device-side wait gave up */
  FACT_TUNE_VERIFY_FAILED = 4  /* output differs from the reference configuration's: never timed */
} fact_tune_outcome_t;
typedef struct {
  fact_config_t cfg;
  int status;        /* fact_tune_outcome_t */
  float ms;          /* per launch in the sweep; < 0 if not timed */
  float rel;         /* ms relative to the default configuration's; < 0 if not timed */
  float verify_err;  /* worst |candidate - reference| / tolerance; < 0 if not verified */
} fact_tune_record_t;
typedef struct {
  int cold_l2;
  int verify;
  int inject_fault;
  fact_tune_record_t* records;
  int max_records;
  int* n_records;
} fact_tune_opts_t;
fact_status_t fact_tune(fact_handle_t handle, fact_op_t op, int64_t batch, int64_t M, int64_t N, int64_t K,
                        const void* A, int64_t lda, int64_t strideA, const void* B, int64_t ldb, int64_t strideB,
                        fact_blayout_t b_layout, const void* bias, const void* residual, int64_t ldr,
                        int64_t strideR, void* C, int64_t ldc, int64_t strideC, fact_out_t out_type,
                        fact_epilogue_t epilogue, void* workspace, size_t workspace_bytes, int warmup, int iters,
                        void* cuda_stream, fact_config_t* best, double* best_ms, int* n_tried);
fact_status_t fact_tune_ex(fact_handle_t handle, fact_op_t op, int64_t batch, int64_t M, int64_t N, int64_t K,
                           const void* A, int64_t lda, int64_t strideA, const void* B, int64_t ldb, int64_t strideB,
                           fact_blayout_t b_layout, const void* bias, const void* residual, int64_t ldr,
                           int64_t strideR, void* C, int64_t ldc, int64_t strideC, fact_out_t out_type,
                           fact_epilogue_t epilogue, void* workspace, size_t workspace_bytes, int warmup, int iters,
                           void* cuda_stream, const fact_tune_opts_t* opts, fact_config_t* best, double* best_ms,
                           int* n_tried);

/* Persist / restore the tuner's table as a text file (one line per problem
 * key; host path).  Loading merges into the handle's table. */
fact_status_t fact_tune_cache_save(fact_handle_t handle, const char* path);
fact_status_t fact_tune_cache_load(fact_handle_t handle, const char* path);

/* Synchronise `cuda_stream`, read the device status word into *status
 * (FACT_OK or FACT_ERR_DEVICE_TIMEOUT) and clear it.  Every device-side wait
 * in the kernels is bounded; a wait that expires records the timeout, the
 * kernel releases its tensor memory and returns, and the output of that call
 * is undefined. */
fact_status_t fact_device_status(fact_handle_t handle, void* cuda_stream, int* status);

/* Self-test of the bounded-wait path, without faulting or hanging anything: launches one warp that waits on
 * an mbarrier nothing will ever complete, with a limit of `limit_ms` milliseconds (0 < limit_ms <= 1000).
 * The wait expires, the kernel records FACT_ERR_DEVICE_TIMEOUT in the handle's status word and returns
 * normally; the call synchronises the stream and returns FACT_OK if that is what happened.  A following
 * fact_device_status reports (and clears) the timeout; the context stays usable. */
fact_status_t fact_selftest_wait_timeout(fact_handle_t handle, void* cuda_stream, double limit_ms);

/* Diagnostic, host arithmetic only (no device is touched): the items CTA `cta` of `ctas` works through in a causal
 * fact_attention call of few rounds (more items than CTAs, fewer than 16 per CTA, at most 8192 items; other calls
 * deal the items out in closed form inside the kernel).  An item is 256 query rows of one (batch, head); item idx
 * is head idx % batch_heads and the (idx / batch_heads)-th pair of tiles counted from the END of the sequence, so
 * items come heaviest first.  The host gives each item, in that order, to the CTA whose items so far see the fewest
 * key blocks (plus a fixed cost per item; the lower CTA on a tie) and hands the list to the kernel as a parameter.
 * Writes at most max_items item numbers and their count to *n_items.  FACT_ERR_UNSUPPORTED above 8192 items. */
fact_status_t fact_attention_deal(int ctas, int64_t batch_heads, int64_t seq, int head_dim, int cta, int max_items,
                                  int32_t* items, int* n_items);

/* Diagnostic, host arithmetic only (no device is touched): the stream-K schedule of one CTA group.  With
 * `sk_tiles` tiles of `k_blocks` k-blocks each shared out over `groups` CTA groups, writes the pieces group
 * `group` processes, in its order, as rows of five ints -- tile (index among the stream-K tiles), first k-block,
 * one past the last k-block, role (0 whole tile; 1 the piece with the tile's first k-block, which finishes the
 * tile; 2 a later piece, parked in the workspace), and for role 1 the number of following groups that hold the
 * tile's other pieces -- and their number in *n_pieces (at most max_pieces rows are written).  The kernels walk
 * exactly this schedule. */
fact_status_t fact_stream_k_pieces(int groups, int64_t sk_tiles, int64_t k_blocks, int group, int max_pieces,
                                   int32_t* pieces, int* n_pieces);

/* Number of kernels this handle has launched so far (for benchmark reports). */
int64_t fact_launch_count(fact_handle_t handle);

/* Diagnostic: synchronise `cuda_stream` and return how many SM clock cycles and
 * how many nanoseconds the first CTA of the most recent GEMM kernel launch spent
 * between its start and its end.  cycles / nanoseconds is the SM clock (GHz)
 * that launch really ran at, which a power-limited part does not keep constant. */
fact_status_t fact_last_kernel_clock(fact_handle_t handle, void* cuda_stream, int64_t* sm_cycles,
                                     int64_t* nanoseconds);

/* Diagnostic: where the first CTA of the most recent GEMM launch spent its SM cycles.  Only filled when
 * the process was started with FACT_DEBUG_FLAGS=256 (the counters cost a few clock reads per tile);
 * otherwise counters[2..7] keep older values.  counters[0] cycles from start to end, [1] the same span
 * in nanoseconds, [2] MMA issuer waiting for a free accumulator (epilogue too slow), [3] MMA issuer waiting
 * for operand stages (loads too slow), [4] one epilogue warp busy from "accumulator ready" to "accumulator
 * released", [5] that warp waiting for an accumulator, [6] tiles that CTA processed, [7] cycles from kernel
 * entry until the first operand stage was ready (the prologue).
 * After a fact_attention launch (same environment variable) the counters are that kernel's: [0] cycles and [1]
 * nanoseconds of the first CTA, [2] a tag of the first device-side wait that gave up (0 if none: barrier index,
 * warp << 8, CTA << 16), [3] cycles the first softmax warp of tile 0 waited for scores, [4] key blocks it
 * processed, [6] cycles it spent writing finished tiles out, [7] work items of that CTA.
 * After a launch with K slices as a cluster (schedule 3) they are the milestones of the first CTA's first tile, in
 * cycles from the moment the kernel may touch global memory: [0] end of the kernel and [1] the same in nanoseconds,
 * [2] first operand stage ready, [3] accumulator complete, [4] every peer's accumulator complete, [5] column blocks
 * sent, [6] column blocks received, [7] tile stored.
 * FACT_DEBUG_FLAGS is read once, by fact_create.  The library as built by default honours four bits, none of
 * which changes a result: 256 (these counters), 2048 (no downward K walk on every second tile), 4096 (no
 * programmatic dependent launch) and 8192 (operand loads without the evict-last L2 policy).  The
 * work-skipping experiment switches (1, 2, 4: the GEMM kernel's loads, products, stores; 8, 64, 128: the attention
 * kernel's softmax arithmetic and its two products), whose output is meaningless, exist only in a library
 * compiled with -DFACT_EXPERIMENTS; the default build ignores those bits. */
fact_status_t fact_last_kernel_profile(fact_handle_t handle, void* cuda_stream, int64_t counters[8]);

/* Diagnostic (FACT_DEBUG_FLAGS=256 only, else 0): nanoseconds from the moment the first CTA of the most recent
 * GEMM launch was allowed to touch global memory to the moment its last CTA left -- the kernel's span over all CTAs,
 * without the launch and completion latencies an event pair around one launch also contains. */
fact_status_t fact_last_kernel_span(fact_handle_t handle, void* cuda_stream, int64_t* nanoseconds);

/* The FACT_DEBUG_FLAGS bits in effect for this handle (0 in normal use; see fact_last_kernel_profile). */
int fact_debug_flags(fact_handle_t handle);

/* Text of the most recent CUDA runtime/driver failure seen through this handle
 * (the call that returned FACT_ERR_CUDA), "" if none.  Owned by the handle;
 * valid until the next failing call or fact_destroy. */
const char* fact_last_error(fact_handle_t handle);

/* Device properties the handle saw (any pointer may be NULL). */
fact_status_t fact_device_info(fact_handle_t handle, int* sm_count, int* max_smem_per_block, int* cc_major,
                               int* cc_minor);

#ifdef __cplusplus
}
#endif
#endif /* FACT_H_ */
