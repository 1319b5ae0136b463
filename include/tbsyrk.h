/*
 * tbsyrk - symmetric rank-k update on the lower triangle, scheduled by triangle
 * blocks, for NVIDIA B200 (sm_100a).
 *
 * C ABI of libtbsyrk.so.  Plain pointers and sizes only.  Unless a function says
 * otherwise, matrix pointers are DEVICE pointers and the call only enqueues work
 * on the given CUDA stream: it never synchronises the device, never aborts and
 * never throws.  Every function returns 0 (SYRK_OK) or a negative SYRK_ERR_*.
 *
 * The operation (Algorithm 1 of "I/O-Optimal Algorithms for Symmetric Linear
 * Algebra Kernels": for i, for j <= i, for k: C[i][j] += A[i][k] * A[j][k]),
 * extended with the usual scalars:
 *
 *     C[i*ldc + j] <- alpha * sum_{k<M} A[i*lda + k] * A[j*lda + k] + beta * C[i*ldc + j]
 *
 * for all 0 <= j <= i < N.  Entries with i < j are never read or written.  The
 * work is partitioned as in Algorithm 4 (TBS) in its tiled form (Section 5.1.4):
 * a thread block owns the accumulators of every pair among k row-segments of A
 * (a triangle block, Section 3.2) and streams only those k segments along M;
 * what triangle blocks cannot cover is done with square and diagonal blocks.
 */
#ifndef TBSYRK_H
#define TBSYRK_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* dtype argument */
#define SYRK_DTYPE_F64      0  /* A and C binary64; binary64 accumulation (DMMA)          */
#define SYRK_DTYPE_BF16_F32 1  /* A bfloat16, C binary32; binary32 accumulation (tcgen05) */
#define SYRK_DTYPE_TF32_F32 2  /* A binary32 read as TF32 (sign, exponent and the 10 leading
                                  fraction bits: the 13 low-order bits of every element are
                                  ignored), C binary32; binary32 accumulation (tcgen05
                                  kind::tf32).  The paper fixes no input precision; this is
                                  the same update on FP32 data.                           */
#define SYRK_DTYPE_E4M3_F32 3  /* A bytes in the OCP FP8 format E4M3 (1 sign, 4 exponent bits
                                  with bias 7, 3 fraction bits; no infinities; 0x7F and 0xFF
                                  are NaN; largest value 448), C binary32; binary32
                                  accumulation (tcgen05 kind::f8f6f4).                    */
#define SYRK_DTYPE_F16_F32  4  /* A IEEE 754 binary16 (1 sign, 5 exponent bits with bias 15,
                                  10 fraction bits; subnormals, infinities and NaN as in
                                  the standard), C binary32; binary32 accumulation (tcgen05
                                  kind::f16).  Both storage orders run on the tensor cores. */

/* return codes */
#define SYRK_OK                 0
#define SYRK_ERR_NULL          -1  /* a required pointer is null                          */
#define SYRK_ERR_SIZE          -2  /* N < 0 or M < 0, or a size beyond a stated maximum   */
#define SYRK_ERR_LD            -3  /* lda < max(1, M) or ldc < max(1, N)                  */
#define SYRK_ERR_DTYPE         -4  /* unknown dtype                                       */
#define SYRK_ERR_ALLOC         -5  /* a device or host allocation of the library failed   */
#define SYRK_ERR_CUDA          -6  /* a CUDA runtime/driver call failed                   */
#define SYRK_ERR_PLAN          -7  /* invalid schedule parameters                         */
#define SYRK_ERR_DEVICE_WAIT   -8  /* a bounded wait inside a kernel ran out (see syrk_last_status) */
#define SYRK_ERR_NO_DEVICE     -9  /* no CUDA device / not an sm_100 device               */
#define SYRK_ERR_NOT_SPD      -11  /* cholesky_lower met a non-positive pivot (see cholesky_last_info) */
#define SYRK_ERR_STATIC_LIMIT -10  /* syrk_lower_bf16_static: problem exceeds its fixed arrays */

/* schedules (syrk_set_schedule) */
#define SYRK_SCHEDULE_TBS     0    /* triangle blocks + square/diagonal leftovers, whatever the size */
#define SYRK_SCHEDULE_SQUARE  1    /* square and diagonal blocks only (comparison schedule) */
#define SYRK_SCHEDULE_PAIR_SQUARE 2 /* square blocks of 256 x 256 on pairs of thread blocks (tcgen05
                                      cta_group::2: the pair shares the N-operand, which halves its
                                      shared-memory traffic) for the tcgen05 types (every dtype but
                                      binary64), operands stored N x M, lower triangle, when the
                                      problem (cut along the inner dimension if need be) gives every
                                      pair a block; every other call runs
                                      SYRK_SCHEDULE_SQUARE.  A second comparison schedule: the pair
                                      form does not fit triangle blocks.                          */
#define SYRK_SCHEDULE_AUTO 3        /* THE DEFAULT.  Triangle blocks, except that a tcgen05-type call
                                      (operand N x M, lower triangle) whose triangle-block list is
                                      shorter than four times the SM count (N below about 7500) runs
                                      SYRK_SCHEDULE_PAIR_SQUARE: such a list fills the GPU unevenly
                                      or only as many short K-slices, and the pair form is measured
                                      1.0-1.5x faster there (2048 x 262144: 0.78 against 0.99 ms).
                                      The paper's tiled scheme needs N large against the block side
                                      (Section 5.1.4) and leaves smaller N to square blocks; this is
                                      that rule with the threshold measured on this GPU.
                                      syrk_effective_schedule() tells which one a call takes.       */

/*
 * The update itself (see the formula above).
 *
 *   N, M     rows and columns of A; N == 0 returns at once.
 *   A        device pointer, row-major N x M, row pitch lda >= max(1, M) elements;
 *            read only.  Element type as `dtype` says (binary64, bfloat16, binary32, FP8 bytes, binary16).
 *   C        device pointer, row-major N x N, row pitch ldc >= max(1, N) elements;
 *            binary64 for SYRK_DTYPE_F64, binary32 for every other dtype.  Only j <= i is touched.  With
 *            beta == 0 the old C is not read (NaN or Inf there do not propagate).
 *   alpha, beta   scalars, passed through as given (non-finite values included).
 *            alpha == 0 or M == 0: the lower triangle becomes beta * C (zero when
 *            beta == 0, untouched when beta == 1).
 *   stream   a cudaStream_t (0 = the legacy default stream).
 *
 * Layout and alignment: the fast kernels fetch A with TMA and need A 16-byte
 * aligned and lda * sizeof(element) a multiple of 16; any other A takes a slower
 * plain-load kernel with the same result.  C may have any alignment.
 *
 * Ownership: the caller owns A and C, keeps them alive until the stream has run
 * the enqueued work, and must not let them overlap.  The library owns a cache of
 * device-resident work lists (one per N, dtype and schedule) and, for the
 * K-split path, a device workspace PER STREAM; both are created on first use (that
 * first call allocates device memory; a workspace that must grow is freed and
 * allocated anew, which synchronises the device) and released by syrk_shutdown().
 * syrk_plan_prepare_stream() does all of that ahead of time.  Calls are
 * stream-ordered, and calls on different streams may overlap on the GPU: each of
 * the first 256 streams the library sees on a device has its own workspace,
 * status word and work-item counter.  A K-split call on a further stream, or one
 * whose workspace would have to grow while the stream is being captured into a
 * graph, returns SYRK_ERR_ALLOC and enqueues nothing.  The K-split path is taken when the
 * work list is too short to fill the GPU and the inner dimension is long (FP64:
 * fewer items than SMs and M >= 1024; the other types: a cost
 * model over the work list, slices of at least 8 K-steps): the inner dimension is cut
 * into slices, the slices' partial results go to the workspace and are summed in
 * slice order (deterministic) before alpha and beta are applied.
 */
int syrk_lower(int64_t N, int64_t M,
               const void* A, int64_t lda,
               void* C, int64_t ldc,
               double alpha, double beta,
               int dtype, void* stream);

/*
 * The same update for the other storage order of the operand (the Gram-matrix form):
 *
 *     C[i][j] = alpha * sum_k A[k][i] * A[k][j] + beta * C[i][j]      for 0 <= j <= i < N,
 *
 * i.e. Algorithm 1 of the paper applied to the N x M matrix A^T, where A is a DEVICE
 * pointer to an M x N row-major array with row pitch lda >= max(1, N) elements.  The
 * paper states the operation for an N x M operand only; the work list (Algorithm 4,
 * Section 5.1.4), C, alpha, beta, dtype, stream, alignment rule (A 16-byte aligned and
 * lda * sizeof(element) a multiple of 16, else a slower plain-load kernel), ownership
 * and error codes are those of syrk_lower (SYRK_ERR_LD refers to lda < N here).
 * Every dtype runs on the tensor-core kernels (FP64: both launch forms; the others:
 * tcgen05 with MN-major operands, K-split included).
 */
int syrk_lower_tn(int64_t N, int64_t M,
                  const void* A, int64_t lda,
                  void* C, int64_t ldc,
                  double alpha, double beta,
                  int dtype, void* stream);

/*
 * The general form: which triangle of C is stored and how the operand is stored.
 *
 *     uplo = SYRK_UPLO_LOWER: the entries C[i][j] with j <= i are updated (as syrk_lower);
 *     uplo = SYRK_UPLO_UPPER: the entries C[i][j] with j >= i are updated, the strict lower
 *                             triangle is never read or written;
 *     trans = SYRK_OP_N: A is N x M row-major, C <- alpha * A A^T + beta * C  (as syrk_lower);
 *     trans = SYRK_OP_T: A is M x N row-major, C <- alpha * A^T A + beta * C  (as syrk_lower_tn).
 *
 * The result is that of Algorithm 1 of the paper: C is symmetric, so the upper form holds the
 * same numbers mirrored.  The paper works on the lower triangle only; the upper form runs the
 * mirror image of the same work list (every tile (x, y) of Algorithm 4 / Section 5.1.4 becomes
 * the tile (y, x), i.e. the roles of the two MMA operands are exchanged and the triangle mask
 * is flipped), so the I/O count is unchanged.
 * For callers holding COLUMN-major data (BLAS convention): a column-major N x K matrix with
 * leading dimension lda is a row-major K x N array with pitch lda, and a column-major triangle
 * 'L' is the row-major upper triangle.  Hence  xSYRK('L', 'N', n, k, alpha, A, lda, beta, C, ldc)
 * == syrk_ex(SYRK_UPLO_UPPER, SYRK_OP_T, n, k, A, lda, C, ldc, alpha, beta, ...), 'U' maps to
 * SYRK_UPLO_LOWER, and trans 'T' to SYRK_OP_N.
 * Everything else (alignment rule and plain-load fallback, K-split, ownership, stream semantics,
 * quick returns, error codes) is as for syrk_lower; an unknown uplo or trans gives SYRK_ERR_SIZE.
 */
#define SYRK_UPLO_LOWER 0
#define SYRK_UPLO_UPPER 1
#define SYRK_OP_N 0
#define SYRK_OP_T 1
int syrk_ex(int uplo, int trans, int64_t N, int64_t M,
            const void* A, int64_t lda,
            void* C, int64_t ldc,
            double alpha, double beta,
            int dtype, void* stream);

/*
 * Symmetric rank-2k update on the lower triangle, binary64:
 *
 *     C[i][j] = alpha * sum_k (A[i][k] * B[j][k] + B[i][k] * A[j][k]) + beta * C[i][j]     0 <= j <= i < N,
 *
 * A and B DEVICE pointers to N x M row-major arrays (pitches lda, ldb >= max(1, M)), C as for
 * syrk_lower.  The paper treats the rank-k update and names, in its conclusion, kernels that use
 * the same input several times as the place its ideas extend to; this is that extension for the
 * nearest such kernel.  The schedule is Algorithm 4 / Section 5.1.4 unchanged: a thread block owns
 * the accumulators of every pair among k = 4 row segments and streams those rows of A and of B
 * (8 segments per step, where a square block of the same 6 tiles would need more), every tile
 * receiving both products.  FP64 tensor cores (DMMA); A and B 16-byte aligned with even pitches,
 * else a plain-load kernel.  Quick returns, ownership, stream semantics and error codes as for
 * syrk_lower (SYRK_ERR_LD also for ldb < max(1, M), SYRK_ERR_NULL for a null B with M > 0).
 */
int syr2k_lower(int64_t N, int64_t M,
                const void* A, int64_t lda,
                const void* B, int64_t ldb,
                void* C, int64_t ldc,
                double alpha, double beta, void* stream);

/*
 * The rank-2k update for every dtype of the library:
 *
 *     C[i][j] = alpha * sum_k (A[i][k] * B[j][k] + B[i][k] * A[j][k]) + beta * C[i][j]     0 <= j <= i < N,
 *
 * A and B of the element type `dtype` names, C binary64 (SYRK_DTYPE_F64, which is syr2k_lower) or binary32.
 * For the tcgen05 types the work list is the rank-k update's (Algorithm 4 / Section 5.1.4: triangle blocks of
 * k = 3 segments, or the square list when that schedule is set); a pipeline stage carries the block's rows of
 * both operands and every accumulator takes both products, A_x B_y^T and B_x A_y^T, in binary32 (each
 * product exact).  K-splits as for syrk_lower; operands that break the TMA rules (16-byte aligned, pitch a
 * multiple of 16 bytes) take a plain-load kernel.  The CTA-pair schedule has no rank-2k form: the default rule
 * runs triangle blocks here at every size.  Arguments, quick returns, ownership and errors as for syr2k_lower.
 */
int syr2k_lower_ex(int64_t N, int64_t M,
                   const void* A, int64_t lda,
                   const void* B, int64_t ldb,
                   void* C, int64_t ldc,
                   double alpha, double beta, int dtype, void* stream);

/*
 * Hermitian rank-k update on the lower triangle, complex128:
 *
 *     C[i][j] = alpha * sum_k A[i][k] * conj(A[j][k]) + beta * C[i][j]     0 <= j <= i < N,
 *
 * alpha and beta real.  A is a DEVICE pointer to an N x M row-major array of complex numbers stored as
 * (real, imaginary) pairs of binary64, pitch lda >= max(1, M) complex entries; C likewise N x N, pitch
 * ldc >= max(1, N) complex entries.  Entries with j > i are never read or written.  The imaginary part
 * of a diagonal entry is not read and is written as zero.  beta == 0: C is not read.
 * This is Algorithm 1 of the paper over the complex numbers (second factor conjugated), one more of
 * the kernels "which use the same input several times" of the paper's conclusion.  Schedule: Algorithm 4 /
 * Section 5.1.4 unchanged - a thread block owns the accumulators of every pair among k = 4 row segments
 * and streams those rows of A once; what changes is the arithmetic per pair: on the real view of A
 * (2M reals per row) the real part is the symmetric update, and the imaginary part is the product of
 * the same rows with those of i * A, which a warp forms from the neighbouring shared-memory word of
 * the same stage (no second operand is loaded).  FP64 tensor cores (DMMA).
 * A and C 16-byte aligned, else (and for the scale-only cases) a plain-load kernel (8-byte alignment,
 * that of binary64, is the caller's to keep).  Quick returns: N == 0; (alpha == 0 or M == 0) and
 * beta == 1: nothing is touched; alpha == 0 or M == 0: the lower triangle is scaled by beta (zeroed
 * for beta == 0) and the diagonal's imaginary part is zeroed.  Ownership, stream semantics, status
 * word and the other error codes as for syrk_lower.
 */
int herk_lower(int64_t N, int64_t M,
               const void* A, int64_t lda,
               void* C, int64_t ldc,
               double alpha, double beta, void* stream);

/*
 * A strided batch of independent updates of the same shape:
 *
 *     C_b[i][j] = alpha * sum_k A_b[i][k] * A_b[j][k] + beta * C_b[i][j]    0 <= j <= i < N, 0 <= b < batch,
 *
 * i.e. Algorithm 1 of the paper applied to each of `batch` problems, with A_b = A + b * stride_a
 * (N x M row-major, pitch lda) and C_b = C + b * stride_c (N x N row-major, pitch ldc), all DEVICE
 * memory, strides in elements.  The paper states the update for one matrix; the batch exists because a
 * small problem (tens of work items) cannot fill the GPU on its own: every matrix uses the work list
 * of Algorithm 4 / Section 5.1.4 for its N, and one launch runs the (matrix, item) pairs of the whole
 * batch (FP64: one thread block per pair, or persistent blocks drawing the pairs from a counter,
 * by the rule of syrk_set_f64_launch; tcgen05 types: pairs dealt to the persistent blocks; the
 * inner dimension is never split here).  Requirements for that single launch: A 16-byte aligned and
 * lda * sizeof(element) and stride_a * sizeof(element) multiples of 16; otherwise, and for alpha == 0
 * or M == 0, the matrices are enqueued one after the other exactly as `batch` syrk_lower calls.
 * Matrices must not overlap: for batch > 1, stride_a >= (N-1) * lda + M and stride_c >= (N-1) * ldc + N
 * (else SYRK_ERR_LD); batch < 0 or batch * items >= 2^31 gives SYRK_ERR_SIZE; batch == 0 returns at
 * once.  Everything else (upper triangles untouched, beta == 0 not reading C, ownership, stream
 * semantics, error codes) is as for syrk_lower.
 */
int syrk_lower_batched(int64_t batch, int64_t N, int64_t M,
                       const void* A, int64_t lda, int64_t stride_a,
                       void* C, int64_t ldc, int64_t stride_c,
                       double alpha, double beta,
                       int dtype, void* stream);

/*
 * Same operation with HOST buffers: copies A (and C when beta != 0) to the
 * device, runs syrk_lower on a stream of the library, copies the lower triangle
 * back into C, and waits for completion.  A and C are host pointers (pageable or
 * pinned; pinned memory copies faster).  The strict upper triangle of the host C is
 * left as it was.  The device and pinned staging buffers are kept by the library
 * (they only grow) and are released by syrk_shutdown().
 * Large inputs are pipelined.  With a page-locked C and N >= 4096 the call works band of
 * rows by band of rows (up to 16): rows [r0, r1) of C need rows [0, r1) of A only, so A
 * is uploaded band by band, a band's work items (square blocks in row order; this path
 * does not use triangle blocks) run as soon as its rows have landed, and the band of C
 * is downloaded while later bands are still uploaded and computed - the rectangle left
 * of the band's diagonal block straight into the caller's C, the diagonal block's lower
 * triangle packed and put in place by the host.  Otherwise A is uploaded in blocks of
 * columns (multiples of 256, at least 32 MB each, at most 8) and each block's update
 * C <- alpha * A_c A_c^T + (beta for the first block, 1 after) * C runs while the next
 * block is in flight (the sum over k is then taken block by block, within the stated
 * tolerance of the one-call result), and C comes back after the last block: in bands as
 * above when it is page-locked, else packed in four groups of rows that host threads
 * unpack while the next group is copied.
 */
int syrk_lower_host(int64_t N, int64_t M,
                    const void* A, int64_t lda,
                    void* C, int64_t ldc,
                    double alpha, double beta, int dtype);

/*
 * Which of the two pipelines above syrk_lower_host uses (process-wide; no counterpart in the paper).
 * SYRK_HOST_AUTO (default): bands of rows where they apply, blocks of columns otherwise.
 * SYRK_HOST_COLUMN_BLOCKS: always blocks of columns.  The difference matters for the schedule: a triangle
 * block of Algorithm 4 owns tiles in k - 1 different zone rows (its rows are R = {u c + f(u)}), so a band of
 * rows of C is complete only after blocks that also need later rows of A; the row-band pipeline therefore
 * runs the square-block list, and only the column-block pipeline runs the schedule syrk_lower would run
 * (syrk_effective_schedule) on each block of columns.
 * syrk_host_pipeline_for tells which one a call with these sizes takes for alpha != 0 (host only):
 * SYRK_HOST_ROW_BANDS or SYRK_HOST_COLUMN_BLOCKS.
 */
#define SYRK_HOST_AUTO          0
#define SYRK_HOST_ROW_BANDS     1
#define SYRK_HOST_COLUMN_BLOCKS 2
int syrk_set_host_pipeline(int mode);
int syrk_host_pipeline_for(int64_t N, int64_t M, int c_is_page_locked);

/*
 * Allocation-free variant of the K-split BF16 path (no counterpart in the paper; it
 * exists for callers that cannot let a library call cudaMalloc: code that runs while
 * another allocator owns the device heap, services whose device memory budget is fixed
 * at start-up, loops where the implicit synchronisation of an allocation is not
 * acceptable).
 *
 * Same operation, arguments and result as syrk_lower with dtype SYRK_DTYPE_BF16_F32,
 * computed as `slices` >= 2 partial products over M that are summed in slice order.
 * The work list, the partial tiles and the status word live in fixed device arrays
 * inside the library image (about 34 MiB on every GPU that loads the library, held
 * until the process exits) instead of cudaMalloc'ed memory; the call itself makes no
 * cudaMalloc / cudaFree and uses no allocating library routine.
 *
 * Limits: at most 1024 work items and
 *     slices * (number of 128 x 128 output tiles) <= SYRK_STATIC_MAX_SLICE_TILES
 * (e.g. N = 2048: 136 tiles, up to 3 slices; N = 1024: 36 tiles, up to 14 slices).
 * Larger problems are refused with SYRK_ERR_STATIC_LIMIT and nothing is enqueued.
 * A must meet the TMA rules (16-byte aligned, lda * 2 a multiple of 16), else
 * SYRK_ERR_LD; alpha == 0 or M == 0 have nothing to split and return SYRK_ERR_SIZE.
 *
 * The first call on a device also resolves the device addresses of those arrays
 * (cudaGetSymbolAddress); make that first call before any stream capture begins.  A call
 * on a stream that is being captured is refused with SYRK_ERR_CUDA: the work list is
 * copied from host memory on the caller's stream when its size differs from the previous
 * call's on that device (a pageable copy, staged before the call returns), and the arrays
 * are shared.  Every call rewrites the shared arrays, so calls whose GPU work may overlap
 * (other streams, other host threads) race: serialise them.  A bounded-wait failure inside
 * this variant's kernels is recorded in its own status word, not the one syrk_last_status
 * reads: after synchronising, syrk_lower_bf16_static_status() returns SYRK_OK, or
 * SYRK_ERR_DEVICE_WAIT once (the result of that call is then undefined) and clears the
 * word; it allocates nothing either.
 */
#define SYRK_STATIC_MAX_SLICE_TILES 512
int syrk_lower_bf16_static(int64_t N, int64_t M,
                           const void* A, int64_t lda,
                           void* C, int64_t ldc,
                           double alpha, double beta,
                           int slices, void* stream);
int syrk_lower_bf16_static_status(void);

/*
 * The lower triangle in packed form, for exchanging it between GPUs (no counterpart in the paper, which
 * names parallel algorithms as future work).  Packed order: row i holds its i + 1 entries at
 * [i (i + 1) / 2, (i + 1) (i + 2) / 2), N (N + 1) / 2 elements of C's type in all (binary64 for
 * SYRK_DTYPE_F64, binary32 otherwise).  All pointers are DEVICE pointers; both calls only enqueue.
 *   syrk_pack_lower:          packed[i (i + 1) / 2 + j] <- C[i][j] for every j <= i.
 *   syrk_unpack_lower_axpby:  for the packed entries first .. first + count - 1, whose values are in
 *                             packed[0 .. count): C[i][j] <- value + beta * C[i][j]  (beta == 0: C not read).
 * Used by the K-sharded multi-GPU update: every GPU holds a block of columns of A, computes alpha times
 * its own A_r A_r^T with syrk_lower (the sum over k of Algorithm 1 splits over the blocks), the packed
 * triangles are summed across GPUs by one reduce-scatter, and each GPU adds beta times its share of C.
 * SYRK_ERR_SIZE for a range outside the triangle, SYRK_ERR_LD for ldc < N.
 */
int syrk_pack_lower(int64_t N, const void* C, int64_t ldc, int dtype, void* packed, void* stream);
int syrk_unpack_lower_axpby(int64_t N, int64_t first, int64_t count, const void* packed, double beta,
                            void* C, int64_t ldc, int dtype, void* stream);

/*
 * Cholesky factorisation by Large Block Cholesky (Algorithm 5 of the paper, LBC): replaces the
 * lower triangle of the symmetric positive definite FP64 matrix A (device pointer, row-major
 * N x N, row pitch lda >= N) by L with A = L * L^T.  Entries above the diagonal are never read
 * or written.  Right-looking with panels of `block` columns (0 = 512, or 1024 from N = 16384 on; a
 * multiple of 128 up to 4096; the paper suggests about sqrt(N)): each panel is factored and the rows below it solved
 * in 128-column steps, then the trailing matrix gets A[I1,I1] -= A[I1,I0] * A[I1,I0]^T through
 * syrk_lower's triangle-block kernel, which is where almost all the arithmetic is.
 *
 * A must be 16-byte aligned and lda even (SYRK_ERR_LD otherwise).  The call enqueues all work on
 * `stream` and returns (part of it runs on a second stream of the library that is ordered after the
 * work already in `stream` and joined back into it before the call returns); workspaces (N x 128 doubles and a few 128 x 128 blocks) are created on
 * first use and kept until syrk_shutdown().  A non-positive pivot does not stop the enqueued
 * work: after synchronising the stream, cholesky_last_info() returns 0, or k + 1 for the first
 * pivot k that was not positive (the contents of A are then undefined from column k on).
 * The workspaces, the second stream and the pivot word are one per device: factorisations whose GPU
 * work could overlap (different streams or host threads) must be serialised by the caller.
 */
int     cholesky_lower(int64_t N, double* A, int64_t lda, int64_t block, void* stream);
int64_t cholesky_last_info(void* stream);

/* Take, ahead of time, every decision a later syrk_lower(N, M, ..., dtype, stream) takes under the
 * current settings (schedule, number of K-slices) and create what that call would allocate: the
 * device-resident work list (or the block list of the CTA-pair schedule) and `stream`'s K-split
 * workspace, for every dtype.  After it, such a call allocates nothing, does not synchronise and
 * may be captured into a graph.  syrk_plan_prepare is the same for the legacy default stream (0).
 * Launches nothing.  (No counterpart in the paper.) */
int syrk_plan_prepare_stream(int64_t N, int64_t M, int dtype, void* stream);
int syrk_plan_prepare(int64_t N, int64_t M, int dtype);

/* Free every cached work list and workspace of the calling process. */
void syrk_shutdown(void);

/* After the caller has synchronised `stream`: 0, or SYRK_ERR_DEVICE_WAIT when a
 * kernel enqueued on that stream gave up on a bounded wait since the last query (the
 * result of that call is then undefined; the context stays usable).  Clears the flag.
 * Every stream has its own flag; stream == 0 asks for all streams of the current device
 * at once (after a device-wide synchronisation) - the form to use after cholesky_lower
 * and syrk_lower_host, which run part of their work on streams of the library. */
int syrk_last_status(void* stream);

/* Human-readable text for a return code (static storage). */
const char* syrk_strerror(int code);

/* Select the schedule used by later calls (process-wide; SYRK_SCHEDULE_AUTO at start). */
int syrk_set_schedule(int schedule);

/* Which schedule syrk_lower(N, M, ..., dtype) runs under the current setting on a 148-SM device, for
 * an aligned operand: SYRK_SCHEDULE_TBS, SYRK_SCHEDULE_SQUARE or SYRK_SCHEDULE_PAIR_SQUARE (host only;
 * a negative SYRK_ERR_* for bad arguments).  Under SYRK_SCHEDULE_AUTO this is where the rule of
 * Section 5.1.4 - triangle blocks once N is large against the block side, squares below - shows. */
int syrk_effective_schedule(int64_t N, int64_t M, int dtype);

/*
 * Diagnostic, no counterpart in the paper: measures this GPU's FP64 tensor-core
 * (DMMA) throughput with a register-only mma.sync loop of `iters` iterations per
 * warp (about 20000 gives ~20 ms) on the current device and default stream, waits
 * for it, and returns TFLOP/s in *tflops.  Allocates and frees a small device buffer.
 */
int syrk_probe_f64_mma_peak(int iters, double* tflops);

/*
 * Diagnostic, no counterpart in the paper: enqueues on `stream` a one-warp kernel that waits on a
 * barrier nothing arrives on.  Every wait inside the library's kernels has a time limit (about two
 * seconds); this call makes one run out on purpose, so that a caller (or a test) can see the whole
 * path work: the kernel returns normally, and after the stream is synchronised syrk_last_status()
 * reports SYRK_ERR_DEVICE_WAIT once, then SYRK_OK again; the context stays usable.
 */
int syrk_selftest_bounded_wait(void* stream);

/* Force the number of K-slices (0 = automatic) used by later calls of every dtype. */
int syrk_set_split_k(int slices);

/*
 * Tail K-split of binary64 calls (no counterpart in the paper; results within the stated tolerance, and
 * the same bits from run to run).  In the one-block-per-item launch form the thread blocks of Algorithm 4's
 * block loop reach the SMs in list order, and with a list of only a few rounds of long items the last round
 * leaves SMs idle.  The library then runs the last items of the list as `slices` blocks each, one per slice
 * of the inner dimension, and a second kernel adds the slices' partial tiles in slice order.
 *   slices == 0 (default): automatic - a replay of the dispatch with a cost model decides whether, how many
 *                          items and how many slices (used when modelled at least 1.5 % faster);
 *   slices == 1: never;
 *   slices >= 2: always, for the last `tail_items` items of the list (tests and measurements).
 * Both launch forms take it (in the persistent form the slices are further tickets).  Not used by the
 * upper triangle, batches, or calls that cut every item (fewer items than SMs).  Process-wide.  SYRK_ERR_PLAN for slices outside 0..64 or tail_items < 0.
 */
int syrk_set_f64_tail_split(int slices, int64_t tail_items);

/*
 * How later FP64 calls (syrk_lower and its variants, syr2k_lower, herk_lower) hand the work items
 * of the schedule (Algorithm 4, tiled as in Section 5.1.4) to thread blocks; the paper has no counterpart, results are the same
 * entry for entry.  PER_ITEM: one thread block per item.  PERSISTENT: one block per SM
 * that draws items from a device-side counter; its MMA warps leave each item's
 * accumulators in shared memory and separate warps write them out during the next item's
 * M loop (beta == 0: stores; beta == 1: one floating-point add per entry done by the memory
 * system, the correctly rounded sum; another beta: a multiply-add in those warps, which is slow
 * because the tensor-core work holds the FP64 pipes).  Used only outside stream capture and for
 * at most 256 distinct streams per device, else the call falls back to PER_ITEM.  AUTO (default):
 * PERSISTENT for beta == 0 or 1 when the list has at least one item per SM; PER_ITEM otherwise.
 * Both forms cut the last items of a list of a few rounds of long items into K-slices
 * (syrk_set_f64_tail_split).
 * Returns SYRK_ERR_PLAN for another value.  Process-wide.
 */
#define SYRK_F64_LAUNCH_AUTO 0
#define SYRK_F64_LAUNCH_PER_ITEM 1
#define SYRK_F64_LAUNCH_PERSISTENT 2
int syrk_set_f64_launch(int mode);

/*
 * What a call with these sizes would run (host only, no device needed).
 * All counts refer to one call.  "a_loads" is the number of elements of A the
 * work list moves from slow to fast memory in the paper's two-level model
 * (Section 3): for every work item, rows held x M.  The work-list fields (items ..
 * a_loads, tile, k, c, s_acc, s_total) describe the single-block list of the current
 * setting (triangle blocks unless SYRK_SCHEDULE_SQUARE / _PAIR_SQUARE is set);
 * effective_schedule, split_k and launches describe what the call really runs, which
 * under SYRK_SCHEDULE_AUTO may be square blocks on CTA pairs.
 */
typedef struct {
    int32_t tile;            /* b: rows per segment                                  */
    int32_t k;               /* segments per triangle block                          */
    int32_t c;               /* zone side of the top level (in tiles)                */
    int32_t split_k;         /* K-slices the call would use on a 148-SM device (1: none) */
    int64_t n_tiles;         /* ceil(N / b)                                          */
    int64_t items;           /* work items                                           */
    int64_t tri_items;       /* of which triangle blocks                             */
    int64_t rect_items;      /* of which square / rectangular blocks                 */
    int64_t diag_items;      /* of which blocks on the diagonal                      */
    int64_t tri_tiles;       /* b x b output tiles owned by triangle blocks          */
    int64_t all_tiles;       /* b x b output tiles in total: n_tiles(n_tiles+1)/2    */
    int64_t a_loads;         /* elements of A loaded (two-level model)               */
    int64_t c_elems;         /* elements of C owned: N(N+1)/2                        */
    int64_t s_acc;           /* accumulator elements a thread block may hold         */
    int64_t s_total;         /* s_acc + staging elements (all pipeline stages; for the
                                persistent FP64 form also the accumulators' image)   */
    int32_t effective_schedule; /* what the call runs: syrk_effective_schedule()      */
    int32_t launches;        /* kernels the call enqueues: 1, or 2 with a K-split of the whole
                                list or of its tail (the slices' partial results are summed
                                by a second kernel); under the automatic FP64 settings     */
} syrk_schedule_stats;

int syrk_get_schedule_stats(int64_t N, int64_t M, int dtype, syrk_schedule_stats* out);

/*
 * Work-list inspection (host only).  A plan is the tiled Algorithm 4 over
 * n_tiles tile rows: triangle blocks of k tile rows chosen by the cyclic indexing
 * family, square blocks (rect_rows x rect_cols tiles) for the last l tile rows and
 * for zones too small to recurse into, and diagonal blocks (diag_side adjacent
 * tile rows, including their diagonal tiles).  schedule == SYRK_SCHEDULE_SQUARE
 * drops the triangle blocks.  Returns NULL on invalid parameters.
 *
 * An item holds n_seg tile rows ("segments") and n_tile output tiles; tile t is
 * C[seg[tile_x[t]] , seg[tile_y[t]]] (tile row, tile column), seg[x] >= seg[y].
 */
#define TBS_ITEM_TRI  0
#define TBS_ITEM_RECT 1
#define TBS_ITEM_DIAG 2
#define TBS_MAX_SEG   8
#define TBS_MAX_TILE 16

void*   tbs_plan_build(int64_t n_tiles, int k, int rect_rows, int rect_cols,
                       int diag_side, int schedule);
/* Reorder a plan for a machine that runs `slots` items at a time (heaviest items first, some
 * full rectangles at the end cut into quarters so that the last wave fills evenly); the set of
 * tiles covered does not change.  The library's own FP64 path only sorts heaviest first (slots = 0):
 * the quartered rectangles measured slower than the uneven last wave they avoid. */
int     tbs_plan_balance(void* plan, int slots);
int64_t tbs_plan_num_items(const void* plan);
int     tbs_plan_item(const void* plan, int64_t index, int32_t* kind,
                      int32_t* n_seg, int32_t seg[TBS_MAX_SEG],
                      int32_t* n_tile, int32_t tile_x[TBS_MAX_TILE],
                      int32_t tile_y[TBS_MAX_TILE]);
void    tbs_plan_free(void* plan);

/* Replay a plan in the two-level model for an N x M matrix cut into tiles of b
 * rows (the last tile may be ragged): elements of A and of C moved, and the
 * smallest / largest number of items that own a lower-triangle tile (both 1 for a
 * correct plan; tiles above the diagonal must stay at 0 and are reported through
 * *upper_cover). */
int tbs_plan_simulate(const void* plan, int64_t N, int64_t M, int b,
                      int64_t* a_loads, int64_t* c_loads,
                      int32_t* min_cover, int32_t* max_cover, int32_t* upper_cover);

#ifdef __cplusplus
}
#endif
#endif /* TBSYRK_H */
