// Set-up of the feedback factors (Section 3.1 and Section 4.1; Algorithm 3 lines 1-2).
//
// For a Gram S (= A^T A, or B B^T) the paper wants the unit lower factor F of the LDL
// decomposition of S^{-1}.  Writing S = P^T P with P LOWER triangular (a Cholesky
// factorisation that eliminates from the last index to the first) gives
//     S^{-1} = P^{-1} P^{-T} = F Lambda F^T,   F = P^{-1} diag(P),   Lambda^{-1} = diag(P)^2,
// so no Gram inverse is ever formed.  L = F(A^T A); U = F(B B^T)^T.
//
// Blocked, right-looking, block size 128, from the last diagonal block to the first:
//   diag kernel  : P_KK from the 128 x 128 Schur complement, and W_KK = P_KK^{-1}
//   panel GEMM   : P_K,0:K = W_KK^T G_K,0:K
//   trailing GEMM: G_0:K,0:K -= P_K,0:K^T P_K,0:K           (lower tiles only)
// then the triangular inverse X = P^{-1} by recursive doubling over diagonal blocks
//   X21 = -X22 (P21 X11)      (strided-batched GEMMs, one batch entry per block pair)
// and a final column scaling (transposed on the way out for U).
#include "common.cuh"
#include "dmma_gemm.cuh"
#include "gemm.cuh"
#include "factor.cuh"

namespace gptq2d {

constexpr int FB = 128;

// One CTA.  S: bs x bs Schur complement (lower triangle read).  Writes P (lower, in place),
// W = P^{-1} (full block, zeros above the diagonal) and diag(P).
// The block is padded to 128 x 128 with the identity in shared memory.  Cholesky runs from the last
// index to the first, blocked sixteen rows at a time (row scaling + rank-one update of the block's own rows
// per step, one rank-16 DMMA update of the rows above per block); the inverse is built from 32 x 32 diagonal blocks by doubling,
// W21 = -W22 (P21 W11), both products as m8n8k4 DMMA fragments, with the temporary product kept in
// the unused upper triangle of the P array.
__device__ __forceinline__ int tri(int i, int j) { return i * (i + 1) / 2 + j; }   // packed lower triangle

// In place, in shared memory, by one CTA of 256 threads: a [128][129] holds the lower triangle of a Schur
// complement padded to 128 x 128 with the identity (bs rows are real); on return its lower triangle is P
// (S = P^T P, Cholesky from the last index to the first) and w is the packed lower triangle of W = P^{-1}.
// Ends with a barrier.  err_c: what a non-positive pivot reports in info[3], beside its index and the side.
__device__ __forceinline__ void chol_inverse_128(double *a, double *w, int bs, int *info, int side, int k0, int err_c) {
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    // Blocked, sixteen rows R = [r_lo, r_hi) at a time from the last block to the first, three barriers a block:
    //  (1) warp 0 factors the block's own 16 x 16 part in place (the unblocked steps -- scale row k, rank-one update of
    //      the rows of R above k -- between warp barriers only) and leaves 1 / P[k][k] in s_rk;
    //  (2) every column j < r_lo of the block's rows is a triangular solve of its own, one thread per column, sixteen
    //      values in registers:  P[k][j] = (A[k][j] - sum_{k' in R, k' > k} P[k'][k] P[k'][j]) / P[k][k],  k descending;
    //  (3) the rows above the block receive the block's sixteen rank-one updates at once, as 8 x 8 fragments of the
    //      lower triangle on the fp64 tensor path (four m8n8k4 products each).
    // (The unblocked loop rewrote up to 128 x 128 entries of shared memory per step behind two CTA barriers: 57 of the
    // kernel's 102 us.)  Rows from bs on are identity padding: they factor to the identity and contribute nothing.
    __shared__ double s_rk[16];
    // warp 0's share of the 16 x 16 lower triangle in (1): entries e = lane + 32 u -> (ii, jj), jj <= ii, row by row
    int tri_i[4], tri_j[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        int ii = 0, r = (tid & 31) + 32 * u;
        while (r > ii) { r -= ii + 1; ++ii; }
        tri_i[u] = ii; tri_j[u] = r;
    }
    for (int kb = (bs - 1) >> 4; kb >= 0; --kb) {
        const int r_lo = 16 * kb;
        if (tid < 32) {
            for (int kk = 15; kk >= 0; --kk) {
                const int k = r_lo + kk;
                double d = a[k * 129 + k];
                if (!(d > 0.0) || !isfinite(d)) {
                    if (tid == 0) report(info, GPTQ2D_ERR_NOT_SPD, k0 + k, side, err_c);
                    d = 1.0;
                }
                double rk = rsqrt(d);
                rk = rk * fma(-0.5 * d, rk * rk, 1.5);         // one Newton step: 1 / sqrt(d) to the last bit or two
                // entries (i, j) of the rows of R above k, r_lo <= j <= i < k: at most 120, four per lane
                double v[4], pi[4], pj[4];
                int at[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const bool on = tri_i[u] < kk;
                    at[u] = on ? (r_lo + tri_i[u]) * 129 + r_lo + tri_j[u] : -1;
                    v[u] = on ? a[at[u]] : 0.0;
                    pi[u] = on ? a[k * 129 + r_lo + tri_i[u]] * rk : 0.0;
                    pj[u] = on ? a[k * 129 + r_lo + tri_j[u]] * rk : 0.0;
                }
                __syncwarp();
                if (tid < kk) a[k * 129 + r_lo + tid] *= rk;   // P[k][r_lo + tid]
                if (tid == 0) { a[k * 129 + k] = d * rk; s_rk[kk] = rk; }
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    if (at[u] >= 0) a[at[u]] = fma(-pi[u], pj[u], v[u]);
                __syncwarp();
            }
        }
        __syncthreads();
        if (kb > 0 && tid < r_lo) {
            double x[16];
#pragma unroll
            for (int kk = 0; kk < 16; ++kk) x[kk] = a[(r_lo + kk) * 129 + tid];
#pragma unroll
            for (int kk = 15; kk >= 0; --kk) {
                double sum = x[kk];
#pragma unroll
                for (int k2 = 15; k2 > kk; --k2) sum = fma(-a[(r_lo + k2) * 129 + r_lo + kk], x[k2], sum);
                x[kk] = sum * s_rk[kk];
            }
#pragma unroll
            for (int kk = 0; kk < 16; ++kk) a[(r_lo + kk) * 129 + tid] = x[kk];
        }
        __syncthreads();
        if (kb > 0) {
            // leading (16 kb) x (16 kb) lower triangle -= P[R, :]^T P[R, :]
            const int warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
            const int nb = 2 * kb, nfrag = nb * (nb + 1) / 2;
            for (int f = warp; f < nfrag; f += 8) {
                int bi = 0, r = f;
                while (r > bi) { r -= bi + 1; ++bi; }
                const int bj = r;
                double c0 = 0.0, c1 = 0.0;
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) {
                    const double *row = a + (r_lo + 4 * kk + t) * 129;
                    dmma_m8n8k4(c0, c1, row[8 * bi + g], row[8 * bj + g]);
                }
                const int ri = 8 * bi + g, cj = 8 * bj + 2 * t;
                if (cj <= ri) a[ri * 129 + cj] -= c0;
                if (cj + 1 <= ri) a[ri * 129 + cj + 1] -= c1;
            }
            __syncthreads();
        }
    }
    // ---- W = P^{-1}.  Level 0: the four 32 x 32 diagonal blocks, one column per thread.
    if (tid < 128) {
        const int r0 = tid & ~31, j = tid & 31;
        w[tri(r0 + j, r0 + j)] = 1.0 / a[(r0 + j) * 129 + r0 + j];
        for (int i = j + 1; i < 32; ++i) {
            double s0 = 0.0, s1 = 0.0;
            int k = j;
            for (; k + 1 < i; k += 2) {
                s0 = fma(a[(r0 + i) * 129 + r0 + k], w[tri(r0 + k, r0 + j)], s0);
                s1 = fma(a[(r0 + i) * 129 + r0 + k + 1], w[tri(r0 + k + 1, r0 + j)], s1);
            }
            if (k < i) s0 = fma(a[(r0 + i) * 129 + r0 + k], w[tri(r0 + k, r0 + j)], s0);
            w[tri(r0 + i, r0 + j)] = -(s0 + s1) / a[(r0 + i) * 129 + r0 + i];
        }
    }
    __syncthreads();
    // ---- doubling: blocks of b = 32, then 64, on the fp64 tensor path.  The 128 / (2 b) pairs have b / 8
    // rows of 8 x 8 fragments each, eight rows in all: one per warp, which takes every fragment of its row.
    // The triangular operands come from the packed array, zeros where the packed array has no entry.
    {
        const int warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
        for (int b = 32; b < 128; b *= 2) {
            const int nf = b >> 3, pr = warp / nf, fr = warp - pr * nf, s0 = pr * 2 * b;
            // T = P21 W11, stored above the diagonal at rows s0 .., columns s0 + b ..
            for (int fc = 0; fc < nf; ++fc) {
                double c0 = 0.0, c1 = 0.0;
                const int cc = 8 * fc + g;
                for (int kk = 8 * fc; kk < b; kk += 4) {       // W11[k][c] = 0 for k < c
                    const int k = kk + t;
                    const double af = a[(s0 + b + 8 * fr + g) * 129 + s0 + k];
                    const double bf = k >= cc ? w[tri(s0 + k, s0 + min(cc, k))] : 0.0;     // index clamped: stays inside the array
                    dmma_m8n8k4(c0, c1, af, bf);
                }
                double *dst = a + (s0 + 8 * fr + g) * 129 + s0 + b + 8 * fc + 2 * t;
                dst[0] = c0;
                dst[1] = c1;
            }
            __syncthreads();
            // W21 = -W22 T
            for (int fc = 0; fc < nf; ++fc) {
                double c0 = 0.0, c1 = 0.0;
                const int rr = 8 * fr + g;
                for (int kk = 0; kk < 8 * fr + 8; kk += 4) {   // W22[r][k] = 0 for k > r
                    const int k = kk + t;
                    const double af = k <= rr ? w[tri(s0 + b + rr, s0 + b + min(k, rr))] : 0.0;
                    const double bf = a[(s0 + k) * 129 + s0 + b + 8 * fc + g];
                    dmma_m8n8k4(c0, c1, af, bf);
                }
                double *dst = w + tri(s0 + b + rr, s0 + 8 * fc + 2 * t);
                dst[0] = -c0;
                dst[1] = -c1;
            }
            __syncthreads();
        }
    }
}

__global__ void __launch_bounds__(256) factor_diag_kernel(double *S, long lds, int bs, double *W, long ldw,
                                                          double *pdiag, int *info, int side, int k0) {
    extern __shared__ double sm[];
    double *a = sm;               // [128][129]: P in the lower triangle, scratch above it
    double *w = sm + 128 * 129;   // packed lower triangle of W
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    // the block, padded with the identity: the kernel sits on the serial spine of the set-up, so a thread's 64 loads
    // are issued in two batches of 32 (entry idx = 256 u + tid: a warp reads 32 consecutive columns of one row)
    for (int base = 0; base < 128 * 128; base += 32 * 256) {
        double v[32];
#pragma unroll
        for (int u = 0; u < 32; ++u) {
            const int idx = base + u * 256 + tid, i = idx >> 7, j = idx & 127;
            v[u] = (j <= i && i < bs) ? S[(long)i * lds + j] : (i == j ? 1.0 : 0.0);
        }
#pragma unroll
        for (int u = 0; u < 32; ++u) {
            const int idx = base + u * 256 + tid, i = idx >> 7, j = idx & 127;
            if (j <= i) a[i * 129 + j] = v[u];
        }
    }
    __syncthreads();
    chol_inverse_128(a, w, bs, info, side, k0, 0);
    for (int idx = tid; idx < 128 * 128; idx += 256) {
        const int i = idx >> 7, j = idx & 127;
        if (i < bs && j < bs) {
            if (j <= i) S[(long)i * lds + j] = a[i * 129 + j];
            W[(long)i * ldw + j] = (j <= i) ? w[tri(i, j)] : 0.0;
        }
    }
    for (int i = tid; i < bs; i += blockDim.x) pdiag[i] = a[i * 129 + i];
}

// out[i][j] (transpose == 0) or out[j][i] (transpose == 1) = X[i][j] * p[j] below the
// diagonal, 1 on it, 0 above; dinv[j] = p[j]^2.
__global__ void __launch_bounds__(256) factor_finish_kernel(const double *X, long ldx, const double *p, int k,
                                                            double *out, long ldo, int transpose, double *dinv) {
    __shared__ double tile[32][33];
    const int bi = blockIdx.y * 32, bj = blockIdx.x * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;   // 32 x 8
    for (int r = ty; r < 32; r += 8) {
        int i = bi + r, j = bj + tx;
        double v = 0.0;
        if (i < k && j < k) v = (i > j) ? X[(long)i * ldx + j] * p[j] : (i == j ? 1.0 : 0.0);
        tile[r][tx] = v;
    }
    __syncthreads();
    if (!transpose) {
        for (int r = ty; r < 32; r += 8) {
            int i = bi + r, j = bj + tx;
            if (i < k && j < k) out[(long)i * ldo + j] = tile[r][tx];
        }
    } else {
        for (int r = ty; r < 32; r += 8) {
            int j = bj + r, i = bi + tx;      // out row = j, out col = i
            if (i < k && j < k) out[(long)j * ldo + i] = tile[tx][r];
        }
    }
    if (dinv && blockIdx.y == 0 && ty == 0) {
        int j = bj + tx;
        if (j < k) dinv[j] = p[j] * p[j];
    }
}

__global__ void identity_kernel(double *out, long ldo, int k, double *dinv) {
    long idx = (long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx < (long)k * k) {
        int i = (int)(idx / k), j = (int)(idx % k);
        out[(long)i * ldo + j] = (i == j) ? 1.0 : 0.0;
    }
    if (dinv && idx < k) dinv[idx] = 1.0;
}

// One side of one small problem (order k <= 128) per CTA, everything in shared memory: the Gram of the
// basis, its Cholesky factorisation and inverse (chol_inverse_128), the unit triangular factor and 1/Lambda.
// For the set-up of many small matrices at once, where one launch sequence per matrix would cost far more
// than the arithmetic.
__global__ void __launch_bounds__(256) factor_small_kernel(const FactorSmallSide *sides, int *info) {
    extern __shared__ double sm[];
    double *a = sm;               // [128][129]
    double *w = sm + 128 * 129;   // packed lower triangle of W
    const FactorSmallSide q = sides[blockIdx.x];
    const int k = q.k, tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    if (!q.M) {                                           // identity basis
        for (int idx = tid; idx < k * k; idx += blockDim.x) {
            const int i = idx / k, j = idx - i * k;
            q.out[(long)i * q.ldo + j] = i == j ? 1.0 : 0.0;
        }
        if (q.dinv)
            for (int j = tid; j < k; j += blockDim.x) q.dinv[j] = 1.0;
        return;
    }
    // a[r][i] = M[r][i] (side 0, S = M^T M) or M[i][r] (side 1, S = M M^T), zero outside k x k
    for (int base = 0; base < 128 * 128; base += 8 * 256) {
        double v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int idx = base + u * 256 + tid, r = idx >> 7, i = idx & 127;
            v[u] = (r < k && i < k) ? (q.side == 0 ? q.M[(long)r * q.ldm + i] : q.M[(long)i * q.ldm + r]) : 0.0;
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int idx = base + u * 256 + tid;
            a[(idx >> 7) * 129 + (idx & 127)] = v[u];
        }
    }
    __syncthreads();
    // S[i][j] = sum_r a[r][i] a[r][j]; thread (tx, ty) owns i = ty + 16 ii, j = tx + 16 jj
    double acc[8][8];
#pragma unroll
    for (int ii = 0; ii < 8; ++ii)
#pragma unroll
        for (int jj = 0; jj < 8; ++jj) acc[ii][jj] = 0.0;
    for (int r = 0; r < k; ++r) {
        double ai[8], aj[8];
#pragma unroll
        for (int x = 0; x < 8; ++x) {
            ai[x] = a[r * 129 + ty + 16 * x];
            aj[x] = a[r * 129 + tx + 16 * x];
        }
#pragma unroll
        for (int ii = 0; ii < 8; ++ii)
#pragma unroll
            for (int jj = 0; jj < 8; ++jj) acc[ii][jj] = fma(ai[ii], aj[jj], acc[ii][jj]);
    }
    __syncthreads();
    // the Gram, padded with the identity, replaces the basis
#pragma unroll
    for (int ii = 0; ii < 8; ++ii)
#pragma unroll
        for (int jj = 0; jj < 8; ++jj) {
            const int i = ty + 16 * ii, j = tx + 16 * jj;
            if (j <= i) a[i * 129 + j] = i < k ? acc[ii][jj] : (i == j ? 1.0 : 0.0);
        }
    __syncthreads();
    chol_inverse_128(a, w, k, info, q.side, 0, q.index);
    // F = W diag(P): unit lower (side 0) or, transposed on the way out, unit upper (side 1)
    for (int idx = tid; idx < k * k; idx += blockDim.x) {
        const int i = idx / k, j = idx - i * k;
        const double v = i > j ? w[tri(i, j)] * a[j * 129 + j] : (i == j ? 1.0 : 0.0);
        if (q.side == 0) q.out[(long)i * q.ldo + j] = v;
        else q.out[(long)j * q.ldo + i] = v;
    }
    if (q.dinv)
        for (int j = tid; j < k; j += blockDim.x) q.dinv[j] = a[j * 129 + j] * a[j * 129 + j];
}

int launch_factor_small(int nsides, const FactorSmallSide *dev_sides, int *info, cudaStream_t stream) {
    if (nsides <= 0) return GPTQ2D_OK;
    const size_t smem = (128 * 129 + 128 * 129 / 2) * sizeof(double);
    if (cudaFuncSetAttribute(factor_small_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return GPTQ2D_ERR_CUDA;
    factor_small_kernel<<<nsides, 256, smem, stream>>>(dev_sides, info);
    return cudaGetLastError() == cudaSuccess ? GPTQ2D_OK : GPTQ2D_ERR_CUDA;
}

static inline long round_up(long x, long a) { return (x + a - 1) / a * a; }

// one side: three k x k matrices (Gram / Cholesky factor, its inverse, a product buffer) and the pivots
size_t factor_side_workspace_bytes(int k) {
    long ld = round_up(k, 16);
    size_t mat = (size_t)ld * (size_t)round_up(k, 16) * sizeof(double);
    size_t b = 3 * mat + (size_t)round_up(k, 32) * sizeof(double) + 256;
    return (b + 255) / 256 * 256;
}
// the two sides are factorised at the same time (two streams), each in its own part of the workspace
size_t factor_workspace_bytes(int m, int n) { return factor_side_workspace_bytes(m) + factor_side_workspace_bytes(n); }

#define CK(x)                                          \
    do {                                               \
        if ((x) != cudaSuccess) return GPTQ2D_ERR_CUDA; \
    } while (0)

// side 0: S = M^T M -> out = F (unit lower).  side 1: S = M M^T -> out = F^T (unit upper).
int factor_one_side(int k, const double *M, long ldm, int side, double *out, long ldo, double *dinv, void *ws,
                    int *info, cudaStream_t stream, const FactorLookahead *look) {
    if (!M) {
        long tot = (long)k * k;
        identity_kernel<<<(unsigned)((tot + 255) / 256), 256, 0, stream>>>(out, ldo, k, dinv);
        CK(cudaGetLastError());
        return GPTQ2D_OK;
    }
    const long ld = round_up(k, 16);
    const size_t mat = (size_t)ld * (size_t)round_up(k, 16);
    double *G = static_cast<double *>(ws);
    double *X = G + mat;
    double *T = X + mat;
    double *p = T + mat;
    const int nblk = (k + FB - 1) / FB;

    CK(cudaMemsetAsync(X, 0, mat * sizeof(double), stream));
    {   // Gram, lower tiles: S = M^T M or M M^T
        GemmArgs g{};
        g.opA = side == 0 ? OP_T : OP_N;
        g.opB = side == 0 ? OP_N : OP_T;
        g.M = g.N = g.K = k;
        g.alpha = 1.0; g.beta = 0.0;
        g.A = M; g.lda = ldm; g.B = M; g.ldb = ldm;
        g.C = G; g.ldc = ld; g.batch = 1; g.lower_tiles_only = 1;
        CK(launch_gemm(g, stream));
    }
    const size_t diag_smem = (128 * 129 + 128 * 129 / 2) * sizeof(double);
    CK(cudaFuncSetAttribute(factor_diag_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)diag_smem));
    CK(cudaFuncSetAttribute(factor_diag_kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                            cudaSharedmemCarveoutMaxShared));
    auto diag = [&](int K, cudaStream_t s) -> int {
        const long k0 = (long)K * FB;
        const int bs = (int)((k - k0) < FB ? (k - k0) : FB);
        factor_diag_kernel<<<1, 256, diag_smem, s>>>(G + k0 * ld + k0, ld, bs, X + k0 * ld + k0, ld, p + k0, info, side,
                                                     (int)k0);
        CK(cudaGetLastError());
        return GPTQ2D_OK;
    };
    auto panel = [&](int K, cudaStream_t s) -> int {       // in place: P_K,0:k0 = W^T G_K,0:k0
        const long k0 = (long)K * FB;
        const int bs = (int)((k - k0) < FB ? (k - k0) : FB);
        GemmArgs g{};
        g.opA = OP_T; g.opB = OP_N;
        g.M = bs; g.N = (int)k0; g.K = bs;
        g.alpha = 1.0; g.beta = 0.0;
        g.A = X + k0 * ld + k0; g.lda = ld; g.B = G + k0 * ld; g.ldb = ld;
        g.C = G + k0 * ld; g.ldc = ld; g.batch = 1;
        CK(launch_gemm(g, s));
        return GPTQ2D_OK;
    };
    // trailing update with the panel of block row K: rows [r0, r1) of the leading part,
    // G[r0:r1, 0:r1] -= P_K,r0:r1^T P_K,0:r1 (lower tiles only when the rows start at 0)
    auto trailing = [&](int K, long r0, long r1, cudaStream_t s) -> int {
        const long k0 = (long)K * FB;
        const int bs = (int)((k - k0) < FB ? (k - k0) : FB);
        if (r1 <= r0) return GPTQ2D_OK;
        GemmArgs t{};
        t.opA = OP_T; t.opB = OP_N;
        t.M = (int)(r1 - r0); t.N = (int)r1; t.K = bs;
        t.alpha = -1.0; t.beta = 1.0;
        t.A = G + k0 * ld + r0; t.lda = ld; t.B = G + k0 * ld; t.ldb = ld;
        t.C = G + r0 * ld; t.ldc = ld; t.batch = 1; t.lower_tiles_only = r0 == 0 ? 1 : 0;
        CK(launch_gemm(t, s));
        return GPTQ2D_OK;
    };
    // the same update with the panels of block rows [K0, K1) at once (contraction over all their rows): a rank-128
    // update runs at 23.5 TFLOP/s, rank 256 at 28, rank 512 at 31.5 (measured, 8192^2 target, C read and rewritten)
    auto trailing_multi = [&](int K0, int K1, long r0, long r1, cudaStream_t s) -> int {
        const long k0 = (long)K0 * FB;
        const long k1 = (long)K1 * FB < k ? (long)K1 * FB : k;
        if (r1 <= r0 || k1 <= k0) return GPTQ2D_OK;
        GemmArgs t{};
        t.opA = OP_T; t.opB = OP_N;
        t.M = (int)(r1 - r0); t.N = (int)r1; t.K = (int)(k1 - k0);
        t.alpha = -1.0; t.beta = 1.0;
        t.A = G + k0 * ld + r0; t.lda = ld; t.B = G + k0 * ld; t.ldb = ld;
        t.C = G + r0 * ld; t.ldc = ld; t.batch = 1; t.lower_tiles_only = r0 == 0 ? 1 : 0;
        CK(launch_gemm(t, s));
        return GPTQ2D_OK;
    };
    constexpr int OUTER = 4;                 // block rows per outer block (512 rows; 2, 6 and 8 measured slower at order 8192)
    // (orders below about 5 500 are faster with the one-level loop further down: 11.9 against 12.2 ms at 4096, 28.9
    // against 29.2 at 6144, but 62.0 against 60.2 at 8192)
    if (look && nblk >= 44) {
        // Two-level right-looking factorisation.  The block rows are grouped four by four into outer blocks of 512
        // rows.  Inside an outer block S the 128-row steps run as before (diag, panel, update of the outer block's
        // own rows above the step), all on look->spine; the rows ABOVE the outer block receive the four panels in
        // one update of rank 512: its first 512 rows (the next outer block, which the spine needs next) on the
        // spine, the rest on `stream`, one outer block behind.  Event logic as in the one-level loop below, with
        // outer blocks in place of block rows: the large update of S+2 is the last one that touched the rows of S
        // before its own steps; the spine's update of the rows of S-1 and the large update of S+1 both write them.
        const int nS = (nblk + OUTER - 1) / OUTER;
        cudaStream_t sp = look->spine;
        const int st_spine = [&]() -> int {
            CK(cudaEventRecord(look->fork, stream));
            CK(cudaStreamWaitEvent(sp, look->fork, 0));
            for (int S = nS - 1; S >= 0; --S) {
                const int Kb = S * OUTER, Ke = (S + 1) * OUTER < nblk ? (S + 1) * OUTER : nblk;     // block rows [Kb, Ke)
                if (S + 2 <= nS - 1) CK(cudaStreamWaitEvent(sp, look->t2[(S + 2) & 1], 0));
                for (int K = Ke - 1; K >= Kb; --K) {
                    int st = diag(K, sp);
                    if (st != GPTQ2D_OK) return st;
                    if (K == 0) break;
                    if ((st = panel(K, sp)) != GPTQ2D_OK) return st;
                    // rows of this outer block above block row K
                    if ((st = trailing(K, (long)Kb * FB, (long)K * FB, sp)) != GPTQ2D_OK) return st;
                }
                if (S == 0) break;
                CK(cudaEventRecord(look->panel, sp));
                if (S + 1 <= nS - 1 && S + 1 >= 2) CK(cudaStreamWaitEvent(sp, look->t2[(S + 1) & 1], 0));
                int st = trailing_multi(Kb, Ke, (long)(S - 1) * OUTER * FB, (long)Kb * FB, sp);
                if (st != GPTQ2D_OK) return st;
                if (S >= 2) {
                    CK(cudaStreamWaitEvent(stream, look->panel, 0));
                    if ((st = trailing_multi(Kb, Ke, 0, (long)(S - 1) * OUTER * FB, stream)) != GPTQ2D_OK) return st;
                    CK(cudaEventRecord(look->t2[S & 1], stream));
                }
            }
            return GPTQ2D_OK;
        }();
        const bool joined = cudaEventRecord(look->join, sp) == cudaSuccess &&
                            cudaStreamWaitEvent(stream, look->join, 0) == cudaSuccess;
        if (st_spine != GPTQ2D_OK) return st_spine;
        if (!joined) return GPTQ2D_ERR_CUDA;
    } else if (!look || nblk < 4) {
        for (int K = nblk - 1; K >= 0; --K) {
            int st = diag(K, stream);
            if (st != GPTQ2D_OK) return st;
            if (K == 0) break;
            if ((st = panel(K, stream)) != GPTQ2D_OK || (st = trailing(K, 0, (long)K * FB, stream)) != GPTQ2D_OK) return st;
        }
    } else {
        // Spine (diag K, panel K, then the update of block row K-1, which the next diagonal block needs) on
        // look->spine; the update of rows 0 .. K-2 with panel K on `stream`.  What diag K reads has been
        // updated by the row update of K+1 (same stream, before it) and by the large updates of K+2 and
        // earlier; the row update of K and the large update of K+1 both write block row K-1, so the former
        // waits for the latter.  An event waited on takes its latest record at the time of the call, so two
        // alternating events tell the large updates of K+2 and K+1 apart.
        cudaStream_t sp = look->spine;
        const int st_spine = [&]() -> int {
            CK(cudaEventRecord(look->fork, stream));
            CK(cudaStreamWaitEvent(sp, look->fork, 0));
            for (int K = nblk - 1; K >= 0; --K) {
                if (K + 2 <= nblk - 1) CK(cudaStreamWaitEvent(sp, look->t2[(K + 2) & 1], 0));
                int st = diag(K, sp);
                if (st != GPTQ2D_OK) return st;
                if (K == 0) break;
                if ((st = panel(K, sp)) != GPTQ2D_OK) return st;
                CK(cudaEventRecord(look->panel, sp));
                if (K + 1 <= nblk - 1 && K + 1 >= 2) CK(cudaStreamWaitEvent(sp, look->t2[(K + 1) & 1], 0));
                if ((st = trailing(K, (long)(K - 1) * FB, (long)K * FB, sp)) != GPTQ2D_OK) return st;
                if (K >= 2) {
                    CK(cudaStreamWaitEvent(stream, look->panel, 0));
                    if ((st = trailing(K, 0, (long)(K - 1) * FB, stream)) != GPTQ2D_OK) return st;
                    CK(cudaEventRecord(look->t2[K & 1], stream));
                }
            }
            return GPTQ2D_OK;
        }();
        // join whatever happened above, so that nothing of this call runs on behind the caller's stream
        const bool joined = cudaEventRecord(look->join, sp) == cudaSuccess &&
                            cudaStreamWaitEvent(stream, look->join, 0) == cudaSuccess;
        if (st_spine != GPTQ2D_OK) return st_spine;
        if (!joined) return GPTQ2D_ERR_CUDA;
    }
    // X = P^{-1}: diagonal blocks are in place; double the block size level by level
    for (long b = FB; b < k; b *= 2) {
        const long npair_full = k / (2 * b);            // pairs with two full halves
        const long rem = k - npair_full * 2 * b;        // what is left after them
        for (int pass = 0; pass < 2; ++pass) {
            long s0, b2, cnt;
            if (pass == 0) { s0 = 0; b2 = b; cnt = npair_full; }
            else { s0 = npair_full * 2 * b; b2 = rem - b; cnt = 1; }
            if (cnt <= 0 || b2 <= 0) continue;
            const long off11 = s0 * ld + s0, off21 = (s0 + b) * ld + s0, off22 = (s0 + b) * ld + (s0 + b);
            const long stride = 2 * b * (ld + 1);
            GemmArgs g1{};   // T21 = P21 X11
            g1.opA = OP_N; g1.opB = OP_N;
            g1.M = (int)b2; g1.N = (int)b; g1.K = (int)b;
            g1.alpha = 1.0; g1.beta = 0.0;
            g1.A = G + off21; g1.lda = ld; g1.strideA = stride;
            g1.B = X + off11; g1.ldb = ld; g1.strideB = stride;
            g1.C = T + off21; g1.ldc = ld; g1.strideC = stride;
            g1.batch = (int)cnt;
            g1.b_lower = 1;  // X11 is lower triangular
            CK(launch_gemm(g1, stream));
            GemmArgs g2{};   // X21 = -X22 T21
            g2.opA = OP_N; g2.opB = OP_N;
            g2.M = (int)b2; g2.N = (int)b; g2.K = (int)b2;
            g2.alpha = -1.0; g2.beta = 0.0;
            g2.A = X + off22; g2.lda = ld; g2.strideA = stride;
            g2.B = T + off21; g2.ldb = ld; g2.strideB = stride;
            g2.C = X + off21; g2.ldc = ld; g2.strideC = stride;
            g2.batch = (int)cnt;
            g2.a_lower = 1;  // X22 is lower triangular
            CK(launch_gemm(g2, stream));
        }
    }
    dim3 grid((k + 31) / 32, (k + 31) / 32);
    factor_finish_kernel<<<grid, 256, 0, stream>>>(X, ld, p, k, out, ldo, side, dinv);
    CK(cudaGetLastError());
    return GPTQ2D_OK;
}

}  // namespace gptq2d
