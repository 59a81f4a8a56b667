// Thin compositions around the forward kernels: reverse-order rounding and fp32-stored inputs.
//
// Reverse-order rounding (paper Section 2, "Two-sided and Kronecker-factored rounding": the same
// greedy rounding taken from the last row and column towards the first).
//
// With P the index reversal, the reverse-order problem on (X; A, B) is the forward problem on
// (P X P; A P, P B): its Gram matrices are P G P and P H P, its trajectory visits the entries in
// exactly the reversed order, and
//     Z = P Z' P,   E = P E' P,   L~ = P L' P (unit upper),   U~ = P U' P (unit lower).
// So both entry points here reverse their operands into the workspace, run the forward kernels,
// and reverse the results back.  The reversals move O(m n + m^2 + n^2) words, against the
// O(m n (m + n)) flops of the sweep.
#include <cuda_runtime.h>
#include "../../include/gptq2d.h"

namespace gptq2d {

// dst[i][j] = src[fr ? rows-1-i : i][fc ? cols-1-j : j]
template <typename T>
__global__ void flip_kernel(T *dst, long ldd, const T *src, long lds, int rows, int cols, int fr, int fc) {
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    const int i = blockIdx.y;
    if (j >= cols) return;
    const int si = fr ? rows - 1 - i : i, sj = fc ? cols - 1 - j : j;
    dst[(long)i * ldd + j] = src[(long)si * lds + sj];
}

template <typename T>
static bool flip(T *dst, long ldd, const T *src, long lds, int rows, int cols, int fr, int fc, cudaStream_t stream) {
    if (rows <= 0 || cols <= 0) return true;
    for (int r0 = 0; r0 < rows; r0 += 65535) {           // grid.y limit
        const int nr = rows - r0 < 65535 ? rows - r0 : 65535;
        // rows [r0, r0 + nr) of dst come from rows [rows-1-r0-(nr-1), rows-1-r0] of src when fr is set
        const T *s = fr ? src + (long)(rows - r0 - nr) * lds : src + (long)r0 * lds;
        dim3 grid((cols + 255) / 256, nr);
        flip_kernel<T><<<grid, 256, 0, stream>>>(dst + (long)r0 * ldd, ldd, s, lds, nr, cols, fr, fc);
        if (cudaGetLastError() != cudaSuccess) return false;
    }
    return true;
}

// dst (double, leading dimension ldd) = src (float, leading dimension lds)
__global__ void widen_kernel(double *dst, long ldd, const float *src, long lds, int rows, int cols) {
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= cols) return;
    for (int i = blockIdx.y; i < rows; i += gridDim.y) dst[(long)i * ldd + j] = (double)src[(long)i * lds + j];
}
static bool widen(double *dst, long ldd, const float *src, long lds, int rows, int cols, cudaStream_t stream) {
    dim3 grid((cols + 255) / 256, rows < 65535 ? rows : 65535);
    widen_kernel<<<grid, 256, 0, stream>>>(dst, ldd, src, lds, rows, cols);
    return cudaGetLastError() == cudaSuccess;
}

static size_t pad256(size_t x) { return (x + 255) / 256 * 256; }
static bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

}  // namespace gptq2d

using namespace gptq2d;

extern "C" {

size_t gptq2d_factor_reverse_workspace_bytes(int m, int n) {
    if (m < 1 || n < 1) return 0;
    const size_t mm = pad256((size_t)m * m * 8), nn = pad256((size_t)n * n * 8);
    return 2 * mm + 2 * nn + pad256((size_t)m * 8) + pad256((size_t)n * 8) + gptq2d_factor_workspace_bytes(m, n);
}

int gptq2d_factor_reverse(int m, int n, const double *A, long lda, const double *B, long ldb, double *Lr, long ldl,
                          double *Ur, long ldu, double *dL, double *dU, void *workspace, size_t workspace_bytes,
                          int *info, void *stream_) {
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (m < 1 || n < 1 || !Lr || !Ur || ldl < m || ldu < n) return GPTQ2D_ERR_INVALID_ARG;
    if ((A && lda < m) || (B && ldb < n)) return GPTQ2D_ERR_INVALID_ARG;
    if (!aligned(A, 8) || !aligned(B, 8) || !aligned(Lr, 8) || !aligned(Ur, 8) || !aligned(dL, 8) || !aligned(dU, 8))
        return GPTQ2D_ERR_INVALID_ARG;
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < gptq2d_factor_reverse_workspace_bytes(m, n))
        return GPTQ2D_ERR_WORKSPACE;
    const size_t mm = pad256((size_t)m * m * 8), nn = pad256((size_t)n * n * 8);
    char *w = static_cast<char *>(workspace);
    double *Ap = reinterpret_cast<double *>(w); w += mm;
    double *Lp = reinterpret_cast<double *>(w); w += mm;
    double *Bp = reinterpret_cast<double *>(w); w += nn;
    double *Up = reinterpret_cast<double *>(w); w += nn;
    double *dLp = reinterpret_cast<double *>(w); w += pad256((size_t)m * 8);
    double *dUp = reinterpret_cast<double *>(w); w += pad256((size_t)n * 8);
    // A P reverses the columns of A, P B the rows of B (an absent basis is the identity either way)
    if (A && !flip(Ap, (long)m, A, lda, m, m, 0, 1, stream)) return GPTQ2D_ERR_CUDA;
    if (B && !flip(Bp, (long)n, B, ldb, n, n, 1, 0, stream)) return GPTQ2D_ERR_CUDA;
    int st = gptq2d_factor(m, n, A ? Ap : nullptr, m, B ? Bp : nullptr, n, Lp, m, Up, n, dLp, dUp, w,
                           gptq2d_factor_workspace_bytes(m, n), info, stream_);
    if (st != GPTQ2D_OK) return st;
    if (!flip(Lr, ldl, Lp, (long)m, m, m, 1, 1, stream) || !flip(Ur, ldu, Up, (long)n, n, n, 1, 1, stream))
        return GPTQ2D_ERR_CUDA;
    if (dL && !flip(dL, (long)m, dLp, (long)m, 1, m, 0, 1, stream)) return GPTQ2D_ERR_CUDA;
    if (dU && !flip(dU, (long)n, dUp, (long)n, 1, n, 0, 1, stream)) return GPTQ2D_ERR_CUDA;
    return GPTQ2D_OK;
}

size_t gptq2d_round_reverse_workspace_bytes(int m, int n) {
    if (m < 1 || n < 1) return 0;
    return pad256((size_t)m * n * 8) * 2 + pad256((size_t)m * m * 8) + pad256((size_t)n * n * 8) +
           pad256((size_t)m * n * 4) + gptq2d_round_workspace_bytes(m, n, GPTQ2D_FP64);
}

int gptq2d_round_reverse(int m, int n, const double *X, long ldx, const double *Lr, long ldl, const double *Ur, long ldu,
                         int32_t *Z, long ldz, double *E, long lde, double *min_margin, void *workspace,
                         size_t workspace_bytes, int *info, void *stream_) {
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (m < 1 || n < 1 || !X || !Lr || !Ur || !Z) return GPTQ2D_ERR_INVALID_ARG;
    if (ldx < n || ldl < m || ldu < n || ldz < n || (E && lde < n)) return GPTQ2D_ERR_INVALID_ARG;
    if (!aligned(X, 8) || !aligned(Lr, 8) || !aligned(Ur, 8) || !aligned(Z, 4) || !aligned(E, 8) ||
        !aligned(min_margin, 8))
        return GPTQ2D_ERR_INVALID_ARG;
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < gptq2d_round_reverse_workspace_bytes(m, n))
        return GPTQ2D_ERR_WORKSPACE;
    char *w = static_cast<char *>(workspace);
    double *Xp = reinterpret_cast<double *>(w); w += pad256((size_t)m * n * 8);
    double *Ep = reinterpret_cast<double *>(w); w += pad256((size_t)m * n * 8);
    double *Lp = reinterpret_cast<double *>(w); w += pad256((size_t)m * m * 8);
    double *Up = reinterpret_cast<double *>(w); w += pad256((size_t)n * n * 8);
    int32_t *Zp = reinterpret_cast<int32_t *>(w); w += pad256((size_t)m * n * 4);
    if (!flip(Xp, (long)n, X, ldx, m, n, 1, 1, stream) || !flip(Lp, (long)m, Lr, ldl, m, m, 1, 1, stream) ||
        !flip(Up, (long)n, Ur, ldu, n, n, 1, 1, stream))
        return GPTQ2D_ERR_CUDA;
    int st = gptq2d_round(m, n, Xp, n, Lp, m, Up, n, Zp, n, E ? Ep : nullptr, n, min_margin, GPTQ2D_FP64, w,
                          gptq2d_round_workspace_bytes(m, n, GPTQ2D_FP64), info, stream_);
    if (st != GPTQ2D_OK) return st;
    if (!flip(Z, ldz, Zp, (long)n, m, n, 1, 1, stream)) return GPTQ2D_ERR_CUDA;
    if (E && !flip(E, lde, Ep, (long)n, m, n, 1, 1, stream)) return GPTQ2D_ERR_CUDA;
    return GPTQ2D_OK;
}

size_t gptq2d_round_f32in_workspace_bytes(int m, int n) {
    if (m < 1 || n < 1) return 0;
    return pad256((size_t)m * n * 8) + pad256((size_t)m * m * 8) + pad256((size_t)n * n * 8) +
           gptq2d_round_workspace_bytes(m, n, GPTQ2D_FP64);
}

int gptq2d_round_f32in(int m, int n, const float *X, long ldx, const float *L, long ldl, const float *U, long ldu,
                       int32_t *Z, long ldz, double *E, long lde, double *min_margin, void *workspace,
                       size_t workspace_bytes, int *info, void *stream_) {
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (m < 1 || n < 1 || !X || !L || !U || !Z) return GPTQ2D_ERR_INVALID_ARG;
    if (ldx < n || ldl < m || ldu < n || ldz < n || (E && lde < n)) return GPTQ2D_ERR_INVALID_ARG;
    if (!aligned(X, 4) || !aligned(L, 4) || !aligned(U, 4) || !aligned(Z, 4) || !aligned(E, 8) ||
        !aligned(min_margin, 8))
        return GPTQ2D_ERR_INVALID_ARG;
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < gptq2d_round_f32in_workspace_bytes(m, n))
        return GPTQ2D_ERR_WORKSPACE;
    char *w = static_cast<char *>(workspace);
    double *Xd = reinterpret_cast<double *>(w); w += pad256((size_t)m * n * 8);
    double *Ld = reinterpret_cast<double *>(w); w += pad256((size_t)m * m * 8);
    double *Ud = reinterpret_cast<double *>(w); w += pad256((size_t)n * n * 8);
    if (!widen(Xd, (long)n, X, ldx, m, n, stream) || !widen(Ld, (long)m, L, ldl, m, m, stream) ||
        !widen(Ud, (long)n, U, ldu, n, n, stream))
        return GPTQ2D_ERR_CUDA;
    return gptq2d_round(m, n, Xd, n, Ld, m, Ud, n, Z, ldz, E, lde, min_margin, GPTQ2D_FP64, w,
                        gptq2d_round_workspace_bytes(m, n, GPTQ2D_FP64), info, stream_);
}

}  // extern "C"
