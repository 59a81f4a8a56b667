// Internal interface of the set-up (not part of the C ABI).
#pragma once
#include <cuda_runtime.h>

namespace gptq2d {

// Optional second stream and five events of the caller's.  With it the serial spine of the blocked
// Cholesky (diagonal block, panel, and the update of the next block row) runs on `spine`, one block ahead
// of the large trailing updates on the main stream.
struct FactorLookahead {
    cudaStream_t spine;
    cudaEvent_t fork, join, panel, t2[2];
};

size_t factor_workspace_bytes(int m, int n);
size_t factor_side_workspace_bytes(int k);
// side 0: S = M^T M -> out = F (unit lower).  side 1: S = M M^T -> out = F^T (unit upper).
int factor_one_side(int k, const double *M, long ldm, int side, double *out, long ldo, double *dinv, void *ws,
                    int *info, cudaStream_t stream, const FactorLookahead *look);

// One side of a small problem for factor_small_kernel (order k <= FACTOR_SMALL_MAX).
constexpr int FACTOR_SMALL_MAX = 128;
struct FactorSmallSide {
    int k, side, index;        // order; 0: out = F(M^T M) unit lower, 1: out = F(M M^T)^T unit upper; problem index
    const double *M; long ldm; // NULL: identity
    double *out; long ldo;
    double *dinv;              // optional
};
// dev_sides: device array of nsides descriptors
int launch_factor_small(int nsides, const FactorSmallSide *dev_sides, int *info, cudaStream_t stream);

}  // namespace gptq2d
