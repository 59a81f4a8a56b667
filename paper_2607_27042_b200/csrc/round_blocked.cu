// Blocked GPTQ-2D (Algorithm 4, Section 4 "Blocked GPTQ-2D") as an alternative to the tiled sweep.
//
// The sweep runs in blocks of w consecutive anti-diagonals with ONE buffer C = L E kept across
// blocks.  Per block [s0, s1] two kernels run back to back on the stream:
//
//   blocked_inblock_kernel   Algorithm 3 cut off at the block boundary.  The clipped pushes are taken
//       in pull form: an entry (i, j) of anti-diagonal s0 + t reads, at rounding time, its t
//       in-block predecessors above it (through L) and its t in-block predecessors to its left
//       (their C through U), every contribution exactly once, so the sums equal those of the
//       clipped fold and pushes.  Four lanes per matrix row; a CTA owns 64 rows of the band and
//       recomputes the cone of at most w - 1 rows above them that its own rows depend on (an entry
//       of in-block depth t depends only on rows i - t .. i), so the CTAs of a block need no
//       synchronisation among themselves.  Outputs: Z, E, and the block's band of C in skewed
//       form Cband[i][t] = C[i, s0 + t - i].
//
//   blocked_flush_kernel     Both flushes for every later entry (i + j > s1) of a 64 x 64 tile:
//       M = L[i, s0-j : s1-j] E[s0-j : s1-j, j]   (down flush; added to Y and, as the outer fold, to C)
//       R = C[i, s0-i : s1-i] U[s0-i : s1-i, j]   (right flush; added to Y)
//       The windows shift with the column (row), so each is a band-like product.  It runs on the
//       fp64 tensor path as a dense product with the band operand masked to the block: warp v owns
//       columns 8v .. 8v+7 of the tile, whose windows span w + 7 values of k, and skips the rest.
//
// Y (the corrected matrix), C and E live in the workspace.  Every block re-reads and re-writes all
// later entries of Y and C and re-reads the rows of L and columns of U that reach them: that
// traffic, 32 B per later entry per block, is what the square-tile restatement avoids.
#include "common.cuh"
#include "dmma_gemm.cuh"

namespace gptq2d {

constexpr int BLK_WMAX = 64;                    // largest block width
constexpr int BLK_R = 64;                       // band rows owned by one CTA of the in-block kernel
constexpr int BLK_LDB = BLK_WMAX + 4;           // row stride of the in-block arrays: 68 = 4 (mod 16), no bank conflicts
constexpr int BLK_ROWS = 128;                   // >= BLK_R + BLK_WMAX - 1 rows of the band per CTA
constexpr int BLK_IN_THREADS = 4 * BLK_ROWS;    // four lanes per row
constexpr int BLK_RING = 128;                   // slots of the ring of U bands (one more than columns in use)
constexpr int FT = 64;                          // flush tile
constexpr int FKC = 32;                         // k-chunk staged per step
constexpr int FLDA = FKC + 4;                   // A stage [64][FKC], row stride 36 = 4 (mod 16): conflict-free
constexpr int FLDB = FT + 4;                    // B stage [FKC][64], row stride 68 = 4 (mod 16)
constexpr int FSTAGE = FT * FLDA + FKC * FLDB;  // doubles per stage
constexpr int FNSTAGE = 3;                      // stages of the copy pipeline (two chunks in flight)
constexpr int FLUSH_THREADS = 256;

struct BlockedParams {
    int m, n, w;
    const double *X; long ldx;
    const double *L; long ldl;
    const double *U; long ldu;
    int *Z; long ldz;
    double *E; long lde;          // optional user copy
    double *max_abs_e;
    int *info;
    double *Y, *C, *Eb;           // m x n, dense
    double *Cband;                // m x w: C of the current block, Cband[i*w + t] = C[i, s0 + t - i]
    double *Lband;                // m x w: Lband[i*w + k] = L[i, i-k]
    double *Uband;                // n x w: Uband[j*w + k] = U[j-k, j]
};

__global__ void blocked_init_kernel(BlockedParams p) {
    CHECKED_SET_INFO(p.info);
    const long nthreads = (long)gridDim.x * blockDim.x, tid0 = (long)blockIdx.x * blockDim.x + threadIdx.x;
    const int m = p.m, n = p.n, w = p.w;
    for (long idx = tid0; idx < (long)m * n; idx += nthreads) {
        const int i = (int)(idx / n), j = (int)(idx % n);
        p.Y[idx] = p.X[CI((long)i * p.ldx + j, (long)(m - 1) * p.ldx + n, 301)];
        p.C[idx] = 0.0;
    }
    for (long idx = tid0; idx < (long)m * w; idx += nthreads) {
        const int i = (int)(idx / w), k = (int)(idx % w);
        p.Lband[idx] = (k >= 1 && i - k >= 0) ? p.L[CI((long)i * p.ldl + (i - k), (long)(m - 1) * p.ldl + m, 302)] : 0.0;
    }
    for (long idx = tid0; idx < (long)n * w; idx += nthreads) {
        const int j = (int)(idx / w), k = (int)(idx % w);
        p.Uband[idx] = (k >= 1 && j - k >= 0) ? p.U[CI((long)(j - k) * p.ldu + j, (long)(n - 1) * p.ldu + n, 303)] : 0.0;
    }
}

// One block of w anti-diagonals, rows [rlo + 64 b, rlo + 64 b + 64) of its band per CTA.
// Four lanes share matrix row i = r0 - (w - 1) + q for the whole block and walk along it, one column
// per anti-diagonal; lane `sub` takes the predecessors k = 1 + sub, 5 + sub, ... of both sums and the
// four partial sums meet in two shuffles.  The lane's part of the row's band of L, L[i, i-k], stays in
// registers.  The columns in use at a step form a window of consecutive columns that slides by one
// per step; their bands of U live in a ring of BLK_RING slots in shared memory (slot = column mod
// BLK_RING), and the column that enters at the next step is fetched ahead of time.
__global__ void __launch_bounds__(BLK_IN_THREADS) blocked_inblock_kernel(BlockedParams p, int s0, int s1, int rlo) {
    CHECKED_SET_INFO(p.info);
    extern __shared__ double sm[];
    double *Es = sm, *Cs = sm + BLK_ROWS * BLK_LDB, *Us = Cs + BLK_ROWS * BLK_LDB;
    __shared__ double red[BLK_IN_THREADS / 32];
    const int tid = threadIdx.x, q = tid >> 2, sub = tid & 3;
    const int w = p.w, wb = s1 - s0 + 1, m = p.m, n = p.n;
    const int r0 = rlo + (int)blockIdx.x * BLK_R;
    const int rend = min(r0 + BLK_R, min(m, s1 + 1));          // rows below s1 hold no entry of the block
    const int ibase = r0 - (w - 1);
    const int i = ibase + q;
    const bool row_ok = q < BLK_R + w - 1 && i >= 0 && i < rend;
    const bool owned = i >= r0;
    // a row `a` above the owned rows matters up to in-block depth wb - 1 - a only
    const int tmax = wb - 1 - (owned ? 0 : r0 - i);
    double *Eq = Es + q * BLK_LDB, *Cq = Cs + q * BLK_LDB;
    double max_abs_e = 0.0;

    double Lr[BLK_WMAX / 4];                                    // Lr[x] = L[i, i-k], k = 1 + sub + 4x; 0 where absent
#pragma unroll
    for (int x = 0; x < BLK_WMAX / 4; ++x) {
        const int k = 1 + sub + 4 * x;
        Lr[x] = (row_ok && k < w) ? p.Lband[CI((long)i * w + k, (long)p.m * w, 304)] : 0.0;
    }

    // columns of step 0: s0 - ibase - (BLK_ROWS - 1) .. s0 - ibase
    const int jtop = s0 - ibase;
    for (int idx = tid; idx < BLK_ROWS * w; idx += BLK_IN_THREADS) {
        const int j = jtop - (BLK_ROWS - 1) + idx / w, k = idx % w;
        Us[CI((j & (BLK_RING - 1)) * BLK_LDB + k, BLK_RING * BLK_LDB, 305)] = (j >= 0 && j < n) ? p.Uband[CI((long)j * w + k, (long)n * w, 306)] : 0.0;
    }
    __syncthreads();

    // Fetched two steps ahead, so that a step never waits for global memory: Y and C of the row's
    // entries as the earlier blocks' flushes left them, and the band of U of the column that enters
    // the window (stored into the ring one step before it is used).
    auto fetch_yc = [&](int tt, double &c, double &y) {
        const int jj = s0 + tt - i;
        c = y = 0.0;
        if (row_ok && tt <= tmax && jj >= 0 && jj < n) {
            c = p.C[CI((long)i * n + jj, (long)p.m * n, 307)];
            y = p.Y[(long)i * n + jj];
        }
    };
    auto fetch_u = [&](int jj) { return (tid < w && jj >= 0 && jj < n) ? p.Uband[(long)jj * w + tid] : 0.0; };
    double c0, y0, c1, y1;
    fetch_yc(0, c0, y0);
    fetch_yc(1, c1, y1);
    double u1 = fetch_u(jtop + 1);
    for (int t = 0; t < wb; ++t) {
        const double cfl = c0, yfl = y0, unew = u1;
        const int jnew = jtop + t + 1;               // enters the window at step t + 1
        c0 = c1;
        y0 = y1;
        fetch_yc(t + 2, c1, y1);
        u1 = fetch_u(jnew + 1);
        const int j = s0 + t - i;
        const bool act = row_ok && t <= tmax && j >= 0 && j < n;
        double up = 0.0, lf = 0.0;
        if (act) {
            const int ku = min(t, i), kl = min(t, j);
            // in-block predecessors above: (i-k, j) has depth t-k and lives in row q-k of the arrays
#pragma unroll
            for (int x = 0; x < BLK_WMAX / 4; ++x) {
                const int k = 1 + sub + 4 * x;
                if (k <= ku) up = fma(Lr[x], Eq[-k * BLK_LDB + t - k], up);
            }
            // in-block predecessors to the left: (i, j-k) has depth t-k in this row
            const double *Ub = Us + (j & (BLK_RING - 1)) * BLK_LDB;
#pragma unroll 4
            for (int k = 1 + sub; k <= kl; k += 4) lf = fma(Cq[t - k], Ub[k], lf);
        }
        up += __shfl_xor_sync(0xffffffffu, up, 1);
        lf += __shfl_xor_sync(0xffffffffu, lf, 1);
        up += __shfl_xor_sync(0xffffffffu, up, 2);
        lf += __shfl_xor_sync(0xffffffffu, lf, 2);
        if (act && sub == 0) {
            const double y = yfl + up + lf;
            double z = rint(y);
            const double e = z - y;
            const double c = cfl + up + e;
            Eq[t] = e;
            Cq[t] = c;
            if (owned) {
                if (!(fabs(y) < 2147483648.0)) {
                    report(p.info, isfinite(y) ? GPTQ2D_ERR_INT_OVERFLOW : GPTQ2D_ERR_NONFINITE, i, j, 0);
                    z = 0.0;
                }
                p.Z[CI((long)i * p.ldz + j, (long)(p.m - 1) * p.ldz + n, 308)] = (int)z;
                p.Eb[CI((long)i * n + j, (long)p.m * n, 309)] = e;
                if (p.E) p.E[(long)i * p.lde + j] = e;
                p.Cband[CI((long)i * w + t, (long)p.m * w, 310)] = c;
                max_abs_e = fmax(max_abs_e, fabs(e));
            }
        }
        if (tid < w) Us[(jnew & (BLK_RING - 1)) * BLK_LDB + tid] = unew;
        __syncthreads();
    }

    max_abs_e = fmax(max_abs_e, 0.0);     // drops a NaN
    for (int o = 16; o > 0; o >>= 1) max_abs_e = fmax(max_abs_e, __shfl_xor_sync(0xffffffffu, max_abs_e, o));
    if ((tid & 31) == 0) red[tid >> 5] = max_abs_e;
    __syncthreads();
    if (tid == 0) {
        double v = 0.0;
        for (int x = 0; x < BLK_IN_THREADS / 32; ++x) v = fmax(v, red[x]);
        atomic_max_nonneg_double(p.max_abs_e, v);
    }
}

// Eight 8-byte copies dst[it * dst_step] <- src[it * src_step]; those outside [lo, hi] are zero-filled.
__device__ __forceinline__ void copy_rows8(double *dst, int dst_step, const double *src, long src_step, int lo, int hi,
                                           const double *safe) {
#pragma unroll
    for (int it = 0; it < 8; ++it) {
        const bool ok = it >= lo && it <= hi;
        cp_async8(dst + it * dst_step, ok ? src + it * src_step : safe, ok ? 8 : 0);
    }
}

// acc[a][0..1] += A(64 rows x FKC, rows a*8+g) * B(FKC x 8 columns of this warp) for the k-steps of the
// chunk [kc0, kc0 + FKC) that meet [wlo, whi].  With ROWWIN, row fragment a is skipped at a k-step that
// misses its own window [alo - 8a - 7, ahi - 8a] (the rows' bands of the masked A operand).
template <bool ROWWIN>
__device__ __forceinline__ void flush_mma(double (&acc)[8][2], const double *As, const double *Bs, int kc0, int wlo,
                                          int whi, int alo, int ahi, int cg, int g, int t) {
    const int lo = max(wlo, kc0), hi = min(whi, kc0 + FKC - 1);
    if (lo > hi) return;
    for (int kk = (lo - kc0) & ~3; kc0 + kk <= hi; kk += 4) {
        const double bf = Bs[(kk + t) * FLDB + cg * 8 + g];
        // fragment a is needed iff alo - 8a - 7 <= k0 + 3 and k0 <= ahi - 8a
        const int k0 = kc0 + kk;
        const int amin = ROWWIN ? max(0, (alo - k0 - 3) >> 3) : 0, amax = ROWWIN ? min(7, (ahi - k0) >> 3) : 7;
#pragma unroll
        for (int a = 0; a < 8; ++a) {
            if (ROWWIN && (a < amin || a > amax)) continue;
            dmma_m8n8k4(acc[a][0], acc[a][1], As[(a * 8 + g) * FLDA + kk + t], bf);
        }
    }
}

// Both flushes of block [s0, s1] for the tile rows ti0 + blockIdx.y, tile column blockIdx.x.
// The k-ranges of the two products are cut into chunks of FKC; chunks c + 1 and c + 2 are on their way
// (8-byte cp.async, zero-filled where the mask says so) into the other stages while chunk c is multiplied.
__global__ void __launch_bounds__(FLUSH_THREADS, 2) blocked_flush_kernel(BlockedParams p, int s0, int s1, int ti0) {
    CHECKED_SET_INFO(p.info);
    extern __shared__ double sm[];
    const int m = p.m, n = p.n, w = p.w;
    const int i0 = (ti0 + (int)blockIdx.y) * FT, j0 = (int)blockIdx.x * FT;
    const int ihi = min(i0 + FT, m) - 1, jhi = min(j0 + FT, n) - 1;
    if (ihi + jhi <= s1) return;                     // no later entry here
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
    const int jg0 = j0 + warp * 8;
    double accD[8][2], accR[8][2];
#pragma unroll
    for (int a = 0; a < 8; ++a) accD[a][0] = accD[a][1] = accR[a][0] = accR[a][1] = 0.0;

    // down flush: k runs over the rows of E that the block holds in this tile's columns
    const int dlo = max(s0 - jhi, 0), dhi = min(s1 - j0, m - 1);
    // right flush: k runs over the columns of C that the block holds in this tile's rows
    const int rlo = max(s0 - ihi, 0), rhi = min(s1 - i0, n - 1);
    const int nd = dhi >= dlo ? (dhi - dlo) / FKC + 1 : 0, nr = rhi >= rlo ? (rhi - rlo) / FKC + 1 : 0;
    const double *safe = p.Y;                        // any mapped address, for copies of zero bytes

    // Each thread copies one column of a stage, eight rows apart; which of its eight rows pass the mask
    // is a range [lo, hi] that a few integer operations give per chunk.
    const int ac = tid & (FKC - 1), ar = tid / FKC;                // A: k index ac, rows ar, ar + 8, ...
    const int bc = tid & (FT - 1), br = tid / FT;                  // B: column bc, k rows br, br + 4, ...
    const int ia = i0 + ar, jb = j0 + bc;
    auto issue = [&](int ch) {
        double *As = sm + (ch % FNSTAGE) * FSTAGE, *Bs = As + FT * FLDA;
        if (ch < nd) {
            const int kc0 = dlo + ch * FKC, k = kc0 + ac, kb0 = kc0 + br;
            // L[i, k], strictly lower part only: k < i < m
            const int alo = max(0, (k - ia + 8) >> 3), ahi = k <= dhi ? min(7, (m - 1 - ia) >> 3) : -1;
            copy_rows8(As + ar * FLDA + ac, 8 * FLDA, p.L + (long)ia * p.ldl + k, 8 * p.ldl, alo, ahi, safe);
            // E[kb, j] where (kb, j) is in the block: s0 - j <= kb <= min(s1 - j, dhi)
            const int blo = max(0, (s0 - jb - kb0 + 3) >> 2), bhi = jb < n ? min(7, (min(dhi, s1 - jb) - kb0) >> 2) : -1;
            copy_rows8(Bs + br * FLDB + bc, 4 * FLDB, p.Eb + (long)kb0 * n + jb, 4 * (long)n, blo, bhi, safe);
        } else {
            const int kc0 = rlo + (ch - nd) * FKC, k = kc0 + ac, kb0 = kc0 + br;
            // C[i, k] where (i, k) is in the block: s0 - k <= i <= min(s1 - k, m - 1)
            const int alo = max(0, (s0 - k - ia + 7) >> 3), ahi = k <= rhi ? min(7, (min(m - 1, s1 - k) - ia) >> 3) : -1;
            copy_rows8(As + ar * FLDA + ac, 8 * FLDA, p.Cband + (long)ia * w + (ia + k - s0), 8 * (long)(w + 1), alo, ahi,
                       safe);
            // U[kb, j], strictly upper part only: kb < j
            const int bhi = jb < n ? min(7, (min(rhi, jb - 1) - kb0) >> 2) : -1;
            copy_rows8(Bs + br * FLDB + bc, 4 * FLDB, p.U + (long)kb0 * p.ldu + jb, 4 * p.ldu, 0, bhi, safe);
        }
    };

    const int total = nd + nr;
#pragma unroll
    for (int c = 0; c < FNSTAGE - 1; ++c) {
        if (c < total) issue(c);
        cp_async_commit();
    }
    for (int ch = 0; ch < total; ++ch) {
        if (ch + FNSTAGE - 1 < total) issue(ch + FNSTAGE - 1);
        cp_async_commit();
        cp_async_wait<FNSTAGE - 1>();
        __syncthreads();
        const double *As = sm + (ch % FNSTAGE) * FSTAGE, *Bs = As + FT * FLDA;
        if (ch < nd)
            flush_mma<false>(accD, As, Bs, dlo + ch * FKC, s0 - (jg0 + 7), s1 - jg0, 0, 0, warp, g, t);
        else
            flush_mma<true>(accR, As, Bs, rlo + (ch - nd) * FKC, rlo, min(rhi, jg0 + 6), s0 - i0, s1 - i0, warp, g, t);
        __syncthreads();
    }
    cp_async_wait<0>();
    // Y += M + R, C += M for the later entries.  All loads of a half tile are issued before the first
    // store (Y and C are distinct buffers, which the compiler cannot know), 16 bytes each where n is even.
    const bool vec = (n & 1) == 0;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        double yv[4][2], cv[4][2];
#pragma unroll
        for (int a4 = 0; a4 < 4; ++a4) {
            const int i = i0 + (h * 4 + a4) * 8 + g, j = jg0 + 2 * t;
            const long idx = (long)i * n + j;
            yv[a4][0] = yv[a4][1] = cv[a4][0] = cv[a4][1] = 0.0;
            if (i < m && j < n) {
                if (vec) {
                    const double2 y2 = *reinterpret_cast<const double2 *>(p.Y + idx);
                    const double2 c2 = *reinterpret_cast<const double2 *>(p.C + idx);
                    yv[a4][0] = y2.x; yv[a4][1] = y2.y; cv[a4][0] = c2.x; cv[a4][1] = c2.y;
                } else {
                    yv[a4][0] = p.Y[idx]; cv[a4][0] = p.C[idx];
                    if (j + 1 < n) { yv[a4][1] = p.Y[idx + 1]; cv[a4][1] = p.C[idx + 1]; }
                }
            }
        }
#pragma unroll
        for (int a4 = 0; a4 < 4; ++a4) {
            const int a = h * 4 + a4, i = i0 + a * 8 + g;
#pragma unroll
            for (int x = 0; x < 2; ++x) {
                const int j = jg0 + 2 * t + x;
                if (i < m && j < n && i + j > s1) {
                    const long idx = CI((long)i * n + j, (long)m * n, 311);
                    p.Y[idx] = yv[a4][x] + (accD[a][x] + accR[a][x]);
                    p.C[idx] = cv[a4][x] + accD[a][x];
                }
            }
        }
    }
}

__global__ void blocked_margin_kernel(const double *max_abs_e, double *min_margin) { *min_margin = 0.5 - *max_abs_e; }

static size_t pad256(size_t x) { return (x + 255) / 256 * 256; }
static bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

}  // namespace gptq2d

using namespace gptq2d;

extern "C" {

size_t gptq2d_round_blocked_workspace_bytes(int m, int n, int w) {
    if (m < 1 || n < 1 || w < 1 || w > BLK_WMAX) return 0;
    return 256 + 3 * pad256((size_t)m * n * 8) + 2 * pad256((size_t)m * w * 8) + pad256((size_t)n * w * 8);
}

int gptq2d_round_blocked(int m, int n, const double *X, long ldx, const double *L, long ldl, const double *U, long ldu,
                         int w, int32_t *Z, long ldz, double *E, long lde, double *min_margin, void *workspace,
                         size_t workspace_bytes, int *info, void *stream_) {
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (m < 1 || n < 1 || !X || !L || !U || !Z || w < 1 || w > BLK_WMAX) return GPTQ2D_ERR_INVALID_ARG;
    if (ldx < n || ldl < m || ldu < n || ldz < n || (E && lde < n)) return GPTQ2D_ERR_INVALID_ARG;
    if (!aligned(X, 8) || !aligned(L, 8) || !aligned(U, 8) || !aligned(Z, 4) || !aligned(E, 8) ||
        !aligned(min_margin, 8))
        return GPTQ2D_ERR_INVALID_ARG;
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < gptq2d_round_blocked_workspace_bytes(m, n, w))
        return GPTQ2D_ERR_WORKSPACE;
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return GPTQ2D_ERR_CUDA;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return GPTQ2D_ERR_CUDA;
    if (major != 10) return GPTQ2D_ERR_UNSUPPORTED_DEVICE;

    BlockedParams p{};
    p.m = m; p.n = n; p.w = w;
    p.X = X; p.ldx = ldx; p.L = L; p.ldl = ldl; p.U = U; p.ldu = ldu;
    p.Z = Z; p.ldz = ldz; p.E = E; p.lde = lde; p.info = info;
    char *ws = static_cast<char *>(workspace);
    p.max_abs_e = reinterpret_cast<double *>(ws + 64);
    char *q = ws + 256;
    const size_t mn = pad256((size_t)m * n * 8);
    p.Y = reinterpret_cast<double *>(q); q += mn;
    p.C = reinterpret_cast<double *>(q); q += mn;
    p.Eb = reinterpret_cast<double *>(q); q += mn;
    p.Cband = reinterpret_cast<double *>(q); q += pad256((size_t)m * w * 8);
    p.Lband = reinterpret_cast<double *>(q); q += pad256((size_t)m * w * 8);
    p.Uband = reinterpret_cast<double *>(q);

    const int in_smem = (2 * BLK_ROWS + BLK_RING) * BLK_LDB * (int)sizeof(double);
    const int fl_smem = FNSTAGE * FSTAGE * (int)sizeof(double);
    if (cudaFuncSetAttribute(blocked_inblock_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, in_smem) != cudaSuccess ||
        cudaFuncSetAttribute(blocked_flush_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, fl_smem) != cudaSuccess ||
        // two CTAs of the flush kernel per SM need the largest shared-memory carve-out
        cudaFuncSetAttribute(blocked_flush_kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                             cudaSharedmemCarveoutMaxShared) != cudaSuccess)
        return GPTQ2D_ERR_CUDA;
    if (info && cudaMemsetAsync(info, 0, 4 * sizeof(int), stream) != cudaSuccess) return GPTQ2D_ERR_CUDA;
    if (cudaMemsetAsync(ws, 0, 256, stream) != cudaSuccess) return GPTQ2D_ERR_CUDA;
    blocked_init_kernel<<<1184, 256, 0, stream>>>(p);
    if (cudaGetLastError() != cudaSuccess) return GPTQ2D_ERR_CUDA;

    const int last = m + n - 2, ntm = (m + FT - 1) / FT, ntn = (n + FT - 1) / FT;
    for (int s0 = 0; s0 <= last; s0 += w) {
        const int s1 = s0 + w - 1 < last ? s0 + w - 1 : last;
        const int rlo = s0 - (n - 1) > 0 ? s0 - (n - 1) : 0, rhi = s1 < m - 1 ? s1 : m - 1;
        const int chunks = (rhi - rlo + 1 + BLK_R - 1) / BLK_R;
        blocked_inblock_kernel<<<chunks, BLK_IN_THREADS, in_smem, stream>>>(p, s0, s1, rlo);
        if (cudaGetLastError() != cudaSuccess) return GPTQ2D_ERR_CUDA;
        if (s1 == last) break;
        const int first_row = s1 - n + 2 > 0 ? s1 - n + 2 : 0;          // first row with an entry behind s1
        const int ti0 = first_row / FT;
        dim3 grid(ntn, ntm - ti0);
        blocked_flush_kernel<<<grid, FLUSH_THREADS, fl_smem, stream>>>(p, s0, s1, ti0);
        if (cudaGetLastError() != cudaSuccess) return GPTQ2D_ERR_CUDA;
    }
    if (min_margin) {
        blocked_margin_kernel<<<1, 1, 0, stream>>>(p.max_abs_e, min_margin);
        if (cudaGetLastError() != cudaSuccess) return GPTQ2D_ERR_CUDA;
    }
    return GPTQ2D_OK;
}

}  // extern "C"
