// Launchers of the CUDA kernels (internal to the library).
#pragma once
#include <cstdint>
#include <cuda.h>
#include <cuda_runtime.h>

#include "tbs_plan.h"

namespace tbsyrk {

// FP64 triangle-block kernel.  `tmC` (may be null): tensor map over C with 32 x 32 FP64 boxes, no
// swizzle, through which the old C tiles are fetched when beta != 0 (one block per item).  With
// `d_tickets` null there is one thread block per work item; otherwise `n_blocks` persistent blocks
// draw the items from d_tickets[0] (d_tickets[0..1] must be zero and must not be shared with a launch
// that can run at the same time; the kernel leaves them zero); that form writes C from three extra
// warps per block and reads old C from memory.  `a_is_m_by_n`: A is stored M x N row-major (the
// Gram form C = A^T A); `tmA` then has boxes of 16 rows x 16 columns over that array.
// `batch` > 0: strided batch of `batch` problems; `tmA` and `tmC` are then 3-D maps whose last
// coordinate is the matrix number, matrix b of C starts at C + b * c_batch_stride, and the launch
// has one block per (matrix, item).  `split_k` > 1 with `d_partial` (split_k x N x N doubles): the
// inner dimension is cut into that many slices, one block per (slice, item) writes partial
// matrices and a second kernel sums them in slice order and applies alpha and beta.  `upper`: the
// work list holds the tiles on and above the diagonal and entries with col >= row are written (one
// block per item; not with `batch`).  `tail_slices` > 1 (one block per item, lower triangle, split_k == 1):
// the items from `tail_first` on run as tail_slices blocks each, one per slice of the inner dimension,
// whose raw partial tiles (in `d_partial`) a second kernel sums in slice order: smaller units for the
// last round of blocks, same bits whatever the order the blocks ran in.
cudaError_t launch_syrk_f64(const CUtensorMap& tmA, const CUtensorMap* tmC, const WorkItem* d_items,
                            int64_t n_items, int64_t N, int64_t M, double* C, int64_t ldc, double alpha,
                            double beta, int a_is_m_by_n, int* d_tickets, int n_blocks, int* d_status,
                            cudaStream_t stream, int64_t batch = 0, int64_t c_batch_stride = 0, int split_k = 1,
                            double* d_partial = nullptr, int upper = 0, int64_t tail_first = 0, int tail_slices = 1);
// Elements of `d_partial` a tail K-split needs: (n_items - tail_first) * tail_slices units of 16 tiles.
int64_t f64_tail_partial_elems(int64_t n_tail_items, int tail_slices);
// Rank-2k update C = alpha (A B^T + B A^T) + beta C on the lower triangle with the same kernel: the work
// items name at most 4 segments and 8 tiles; every stage holds the segments' rows of A (tmA) and of
// B (tmB); a tile is shared by two warps (16 rows each) that add both products.  One block per item, or, with
// `d_tickets` (as for launch_syrk_f64), `n_blocks` persistent blocks whose write-out warps store C.
cudaError_t launch_syr2k_f64(const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap* tmC,
                             const WorkItem* d_items, int64_t n_items, int64_t N, int64_t M, double* C, int64_t ldc,
                             double alpha, double beta, int* d_status, cudaStream_t stream, int* d_tickets = nullptr,
                             int n_blocks = 0);
// Hermitian rank-k update C = alpha A A^H + beta C on the lower triangle with the same kernel: `tmA` covers
// the real view of the complex operand (N rows of 2M binary64 values, re and im interleaved), C and ldc
// address complex entries (C 16-byte aligned); work items as for the rank-2k update (at most 8 tiles, a
// tile shared by two warps, each with a real and an imaginary accumulator).  One block per item, or persistent
// blocks when `d_tickets` is given.
cudaError_t launch_herk_f64(const CUtensorMap& tmA, const WorkItem* d_items, int64_t n_items, int64_t N, int64_t M,
                            double* C, int64_t ldc, double alpha, double beta, int* d_status, cudaStream_t stream,
                            int* d_tickets = nullptr, int n_blocks = 0);
// The same kernel in two-operand mode: D (nrows x ncols, pitch ldd) = alpha * P * Q^T + beta * D with
// P nrows x K and Q ncols x K, both row-major through their tensor maps (boxes of 32 rows x 16
// columns, 128-byte swizzle); `tmD` (may be null) as `tmC` above.  Requires K > 0.
cudaError_t launch_gemm_nt_f64(const CUtensorMap& tmP, const CUtensorMap& tmQ, const CUtensorMap* tmD,
                               int64_t nrows, int64_t ncols, int64_t K, double* D, int64_t ldd, double alpha,
                               double beta, int* d_status, cudaStream_t stream);
int f64_tile();
int f64_bk();
int f64_stages();
int f64_persistent_stages();    // ring depth of the persistent launch form

// BF16 -> FP32 triangle-block kernel (tcgen05 / TMEM): persistent, one thread block per SM.
// `split_k` > 1 makes every item run once per K-slice, partial tiles going to `d_partial`
// (split_k x tiles x 128 x 128 floats) to be summed by the reduce kernel.  `tmC` is a tensor
// map over C for the asynchronous store path (32 x 32 FP32 boxes, 128-byte swizzle), or null
// when C does not meet the TMA alignment rules.  With split_k == 1 and `d_cta_begin` given, block b
// runs items [d_cta_begin[b], d_cta_begin[b+1]) of the list (n_ctas blocks).  `a_is_m_by_n`: A is
// stored M x N row-major and `tmA` has square boxes of one stage's k-rows x 128 bytes of columns
// over that array (64 x 64 for the 16-bit kinds, 32 x 32 for TF32, 128 x 128 for FP8).  `a_kind`:
// 0 bfloat16; 1 binary32 read as TF32 (N x M order: boxes of 128 rows x 32 columns); 2 FP8 E4M3 bytes
// (boxes of 128 rows x 128 columns); 3 IEEE binary16 (boxes as for bfloat16).
// `tmB` (N x M operands, lower triangle, no batch): the rank-2k update alpha (A B^T + B A^T) + beta C; `tmB`
// is the map of B with the boxes of `tmA`; a stage then holds the segments of both operands (two stages).
// `batch` > 0: strided batch (3-D maps as for the FP64 kernel); the units are then (matrix, item)
// pairs dealt round-robin, split_k must be 1.  `upper`: the work list holds the tiles on and above
// the diagonal and the entries with col >= row are written (not with `batch`).
cudaError_t launch_syrk_bf16(const CUtensorMap& tmA, const CUtensorMap* tmC, const WorkItem* d_items,
                             int64_t n_items, int64_t N, int64_t M, float* C, int64_t ldc, float alpha,
                             float beta, int split_k, float* d_partial, const int64_t* d_tile_base,
                             int64_t total_tiles, const int64_t* d_cta_begin, int n_ctas, int a_is_m_by_n,
                             int a_kind, int* d_status, int sm_count, cudaStream_t stream,
                             int64_t batch = 0, int64_t c_batch_stride = 0, int upper = 0, const CUtensorMap* tmB = nullptr);
// Square-block comparison kernel on CTA pairs (tcgen05 cta_group::2) for operands of input kind `a_kind`
// (as launch_syrk_bf16) stored N x M: block i of `d_blocks` = {X0, X1, Y0, Y1}, tile rows (128 rows each) of a 256 x 256 block
// strictly below the diagonal; pair p of the grid runs blocks p, p + pairs, ...  `tmA` and `tmC` as for
// launch_syrk_bf16 (boxes of 128 rows x 64 columns; 32 x 32 binary32 boxes).  Lower triangle only.
// Blocks with X = Y lie on the diagonal.  `split_k` > 1 with `d_partial` (split_k x n_blocks x 4 tiles of
// 128 x 128 floats): units are (block, K-slice) pairs, partial tiles summed in slice order by a second kernel.
cudaError_t launch_syrk_pair_square(const CUtensorMap& tmA, const CUtensorMap* tmC, const int4* d_blocks, int32_t n_blocks,
                                    int64_t N, int64_t M, float* C, int64_t ldc, float alpha, float beta, int a_kind,
                                    int* d_status, int sm_count, cudaStream_t stream, int split_k = 1,
                                    float* d_partial = nullptr);
int bf16_tile();
int bf16_bk();
int bf16_stages();
int bf16_seg_slots();
int bf16_store_box();

// Plain-load kernels: one thread per lower-triangle entry.  Used when A does not meet
// the TMA alignment rules; same result, much slower.
cudaError_t launch_syrk_plain(int dtype, int64_t N, int64_t M, const void* A, int64_t lda, void* C,
                              int64_t ldc, double alpha, double beta, int a_is_m_by_n, cudaStream_t stream,
                              int upper = 0);

// Lower triangle <- beta * lower triangle (zero when beta == 0, without reading C).
// Plain-load rank-2k update (binary64): one thread per lower-triangle entry; for unaligned operands.
cudaError_t launch_syr2k_plain(int64_t N, int64_t M, const double* A, int64_t lda, const double* B, int64_t ldb,
                               double* C, int64_t ldc, double alpha, double beta, cudaStream_t stream);

// Plain-load Hermitian rank-k update (complex128 as pairs of binary64; pitches in complex entries): one thread
// per lower-triangle entry; for unaligned operands, and (M == 0 or alpha == 0) for the scale-only case.  The
// diagonal's imaginary part is written as zero and not read; beta == 0: C is not read.
cudaError_t launch_herk_plain(int64_t N, int64_t M, const double* A, int64_t lda, double* C, int64_t ldc,
                              double alpha, double beta, cudaStream_t stream);

// The same for the tcgen05 storage types (dtype 1..4; binary32 accumulation and C).
cudaError_t launch_syr2k_plain_f32(int dtype, int64_t N, int64_t M, const void* A, int64_t lda, const void* B, int64_t ldb,
                                   float* C, int64_t ldc, float alpha, float beta, cudaStream_t stream);

cudaError_t launch_scale_lower(int dtype, int64_t N, void* C, int64_t ldc, double beta,
                               cudaStream_t stream, int upper = 0);

}  // namespace tbsyrk
