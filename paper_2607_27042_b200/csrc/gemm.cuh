// Host-side interface of the library's own fp64 GEMM (DMMA tiles, see dmma_gemm.cuh).
// Used by the set-up (Gram, blocked Cholesky, triangular inverse) and by the objective.
#pragma once
#include <cuda_runtime.h>

namespace gptq2d {

enum GemmOp { OP_N = 0, OP_T = 1 };

struct GemmArgs {
    // C[b] = alpha * op(A[b]) * op(B[b]) + beta * C[b]   for b in [0, batch)
    // op(A) is M x K, op(B) is K x N, all row-major with leading dimensions in elements.
    GemmOp opA, opB;
    int M, N, K;
    double alpha, beta;
    const double *A; long lda; long strideA;
    const double *B; long ldb; long strideB;
    double *C; long ldc; long strideC;
    int batch;
    int lower_tiles_only;   // skip 128 x 128 output tiles strictly above the block diagonal
    // Triangular operands: the part of the contraction that only meets structural zeros is skipped.
    int a_lower;            // op(A) is lower triangular (M x K, zero for k > m): tile row tm stops at k = 128 (tm + 1)
    int b_lower;            // op(B) is lower triangular (K x N, zero for k < n): tile column tn starts at k = 128 tn
    double *sumsq_partials; // if non-null: do not store C; write sum(C^2) of each CTA tile
                            // to sumsq_partials[tile index] (tiles_m * tiles_n * batch entries)
    unsigned *abort;        // optional device word: raised if a bounded wait of the TMA-fed kernel runs out
                            // (the tile is then not written); NULL: nobody is told
};

// Enqueues the GEMM on `stream`.  Returns cudaSuccess or the launch error.
cudaError_t launch_gemm(const GemmArgs &g, cudaStream_t stream);
// 1 (default): products with a ragged tile edge whose operands are 16-byte aligned with even leading dimensions
// go through the TMA-fed kernel, full tiles through the cp.async kernel; 3: TMA-fed kernel whenever the operands
// allow it; 2: the same with a CTA barrier per slab; 0: everything through the cp.async kernel.
void gemm_set_tma_mode(int mode);

}  // namespace gptq2d
