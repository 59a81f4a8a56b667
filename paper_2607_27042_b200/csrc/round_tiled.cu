// GPTQ-2D sweep as a persistent tiled wavefront (fp64), one launch for the whole matrix.
//
// Restatement of Algorithm 3 on 128 x 128 tiles (follows from Eq. 11 and Eq. 15-17): for
// tile (I, J) with rows r and columns c,
//     Cd = sum_{I' < I} L[r, I'] E[I', c]          (feedback folded from the tiles above)
//     Rt = sum_{J' < J} C[r, J'] U[J', c]          (rightward pushes from the tiles to the left)
// and Algorithm 3 run on the tile alone with Y initialised to X[r,c] + Rt + Cd, C initialised
// to Cd, factors L[r,r], U[c,c] produces exactly the Z, E and C = L E entries of the full
// sweep.  Cd and Rt are dense contractions and carry all but a T/(m+n) share of the flops,
// so they run on the fp64 tensor path (dmma_gemm.cuh); tiles with equal I + J are independent.
//
// Scheduling.  Every tile has two bulk tasks (Cd and Rt).  Tasks are listed wave by wave
// (I + J ascending) and claimed in that order from one atomic counter by persistent CTAs
// (one per SM, cooperatively launched so that all are resident).  A bulk task consumes its
// source tiles in the order they become available, waiting (bounded) on per-tile ready
// flags; whichever CTA finishes the second bulk task of a tile runs that tile's in-tile
// sweep right away and then raises the tile's flag.  A task only ever waits on tiles of
// earlier waves, whose tasks were claimed earlier, so the earliest unfinished task can
// always progress.
//
// In-tile sweep.  The tile is processed as four 64 x 64 quadrants (the same restatement one
// level down, cross terms as 64^3 DMMA products).  Inside a quadrant the anti-diagonal
// sweep runs on 8 x 8 leaves: the leaves of one leaf-wave are swept by groups of 8 lanes
// (lane = row; each row is kept in registers rotated by its row index, so that at step s
// every lane touches register slot s mod 8; downward pushes travel by warp shuffle, with the
// lane's L coefficients held in registers), then all warps apply the leaves' feedback to
// the remaining 8 x 8 blocks of the quadrant with m8n8k4 DMMA.
#include "common.cuh"
#include "dmma_gemm.cuh"
#include "round_internal.cuh"

namespace gptq2d {

constexpr int T = 128;           // tile edge
constexpr int Q = 64;            // quadrant edge
constexpr int QLD = 68;          // shared-memory row stride of quadrant matrices (68 mod 16 == 4)
constexpr int QMAT = Q * QLD;    // doubles per quadrant matrix
constexpr int BULK_NSTAGE = 4;
constexpr int TILED_THREADS = 256;

struct TiledKernelParams {
    int m, n, ntm, ntn, ntasks;
    long np;                     // leading dimension of Ebuf / Cbuf (= ntn * 128)
    const double *X; long ldx;
    const double *L; long ldl;
    const double *U; long ldu;
    int *Z; long ldz;
    double *Euser; long lde;
    double *Ebuf, *Cbuf;
    unsigned *counter, *abort;
    unsigned *flagS;             // [ntm*ntn] tile swept
    unsigned *bulk_done;         // [ntm*ntn] number of finished bulk tasks
    double *max_abs_e;
    int *info;
    int l_al16, u_al16;
};

constexpr size_t SWEEP_SMEM = (size_t)5 * QMAT * sizeof(double) + (size_t)Q * Q * sizeof(int);
constexpr size_t BULK_SMEM = (size_t)BULK_NSTAGE * SlabLayout<true, false>::STAGE_DOUBLES * sizeof(double);
constexpr size_t TILED_SMEM = SWEEP_SMEM > BULK_SMEM ? SWEEP_SMEM : BULK_SMEM;

// ---------------------------------------------------------------------------------------------
// bounded wait until flags[first] is set; returns the index of the first flag in
// [first, count) that is not set yet (> first), or -1 on abort / timeout.
__device__ __forceinline__ int wait_ready_prefix(const unsigned *flags, long stride, int first, int count,
                                                 const TiledKernelParams &p, int where) {
    __shared__ int s_first;
    const int tid = threadIdx.x;
    unsigned long long spins = 0;
    for (;;) {
        __syncthreads();
        if (tid == 0) s_first = count;
        __syncthreads();
        for (int idx = first + tid; idx < count; idx += blockDim.x)
            if (ld_acquire_u32(flags + (long)idx * stride) == 0u) atomicMin(&s_first, idx);
        __syncthreads();
        int f = s_first;
        if (f > first) return f;
        // nothing ready: thread 0 spins on the first flag
        __shared__ int s_ok;
        if (tid == 0) {
            int ok = 1;
            while (ld_acquire_u32(flags + (long)first * stride) == 0u) {
                if (ld_relaxed_u32(p.abort) != 0u) { ok = 0; break; }
                if (++spins > SPIN_LIMIT) {
                    report(p.info, GPTQ2D_ERR_DEVICE_TIMEOUT, where, first, (int)blockIdx.x);
                    atomicExch(p.abort, 1u);
                    ok = 0;
                    break;
                }
                __nanosleep(100);
            }
            s_ok = ok;
        }
        __syncthreads();
        if (!s_ok) return -1;
    }
}

// ---------------------------------------------------------------------------------------------
// quadrant <-> shared memory
__device__ __forceinline__ void load_quadrant_cg(double *dst, const double *src, long ld) {
    // dense 64 x 64 from a padded workspace buffer (always in range, 16-byte aligned)
    for (int c = threadIdx.x; c < Q * Q / 2; c += blockDim.x) {
        int r = c >> 5, cc = (c & 31) * 2;
        double2 v = __ldcg(reinterpret_cast<const double2 *>(src + (long)r * ld + cc));
        *reinterpret_cast<double2 *>(dst + r * QLD + cc) = v;
    }
}
__device__ __forceinline__ void store_quadrant(double *dst, long ld, const double *src) {
    for (int c = threadIdx.x; c < Q * Q / 2; c += blockDim.x) {
        int r = c >> 5, cc = (c & 31) * 2;
        *reinterpret_cast<double2 *>(dst + (long)r * ld + cc) = *reinterpret_cast<const double2 *>(src + r * QLD + cc);
    }
}
// 64 x 64 block of a user matrix (k x k, leading dimension ld) whose top-left element is
// (r0, c0); mode 0: everything in range, 1: strictly lower part only, 2: strictly upper only
// (relative to the matrix diagonal).  Out-of-range and masked elements become zero.
__device__ __forceinline__ void load_factor_block(double *dst, const double *M, long ld, int k, int r0, int c0,
                                                  int mode) {
    for (int c = threadIdx.x; c < Q * Q; c += blockDim.x) {
        int r = c >> 6, cc = c & 63;
        int gr = r0 + r, gc = c0 + cc;
        double v = 0.0;
        bool take = gr < k && gc < k;
        if (mode == 1) take = take && gc < gr;
        if (mode == 2) take = take && gc > gr;
        if (take) v = __ldg(M + (long)gr * ld + gc);
        dst[r * QLD + cc] = v;
    }
}

// G (global 64 x 64, row stride ld) += As (64 x 64, [m][k]) * Bs (64 x 64, [k][n])
__device__ __forceinline__ void cross_gemm(double *G, long ld, const double *As, const double *Bs) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    const int wr = warp >> 1, wc = warp & 1;
    double acc[2][4][2];
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b][0] = acc[a][b][1] = 0.0;
#pragma unroll 4
    for (int kk = 0; kk < Q; kk += 4) {
        double af[2], bf[4];
#pragma unroll
        for (int a = 0; a < 2; ++a) af[a] = As[(wr * 16 + a * 8 + g) * QLD + kk + t];
#pragma unroll
        for (int b = 0; b < 4; ++b) bf[b] = Bs[(kk + t) * QLD + wc * 32 + b * 8 + g];
#pragma unroll
        for (int a = 0; a < 2; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) dmma_m8n8k4(acc[a][b][0], acc[a][b][1], af[a], bf[b]);
    }
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            double2 *ptr = reinterpret_cast<double2 *>(G + (long)(wr * 16 + a * 8 + g) * ld + wc * 32 + b * 8 + t * 2);
            double2 v = __ldcg(ptr);
            v.x += acc[a][b][0];
            v.y += acc[a][b][1];
            *ptr = v;
        }
}

// ---------------------------------------------------------------------------------------------
// Algorithm 3 on one 64 x 64 quadrant held in shared memory.
//   Ys: in  Y (corrected values, already including the C the quadrant starts with)
//       out E (local errors)
//   Cs: in  C at entry; out final C = L E rows of the quadrant
//   Ls / Us: strictly lower / strictly upper 64 x 64 diagonal blocks of the factors
//   Zs: out rounded integers
// row0/col0: global coordinates of the quadrant (for masking the status checks).
__device__ __forceinline__ void quadrant_sweep(double *Ys, double *Cs, const double *Ls, const double *Us, int *Zs,
                                               int row0, int col0, const TiledKernelParams &p, double &max_abs_e) {
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, t = lane & 3;
    for (int lw = 0; lw < 15; ++lw) {
        __syncthreads();
        // ---------------- phase A: sweep the leaves (a, lw - a) of this leaf-wave
        if (warp < 2) {
            const int a_lo = max(0, lw - 7), a_hi = min(7, lw);
            const int grp = tid >> 3, i = tid & 7;          // 8 groups of 8 lanes in warps 0-1
            const int a = a_lo + grp, b = lw - a;
            const bool live = a <= a_hi;
            double y[8], c[8], lrow[8];
            int z[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                int j = (k - i) & 7;                         // slot k holds column j of the leaf row
                y[k] = live ? Ys[(a * 8 + i) * QLD + b * 8 + j] : 0.0;
                c[k] = live ? Cs[(a * 8 + i) * QLD + b * 8 + j] : 0.0;
                z[k] = 0;
            }
#pragma unroll
            for (int d = 1; d < 8; ++d) lrow[d] = (live && i - d >= 0) ? Ls[(a * 8 + i) * QLD + a * 8 + i - d] : 0.0;
#pragma unroll
            for (int s = 0; s < 15; ++s) {
                const int k = s & 7;
                const int j = s - i;
                const bool act = live && j >= 0 && j < 8;
                double e = 0.0;
                if (act) {
                    const double yv = y[k];
                    double zv = rint(yv);
                    if (!(fabs(yv) < 2147483648.0)) {
                        int gr = row0 + a * 8 + i, gc = col0 + b * 8 + j;
                        if (gr < p.m && gc < p.n)
                            report(p.info, isfinite(yv) ? GPTQ2D_ERR_INT_OVERFLOW : GPTQ2D_ERR_NONFINITE, gr, gc, 0);
                        zv = 0.0;
                    }
                    e = zv - yv;                                           // line 5: E = Z - Y
                    z[k] = (int)zv;
                    y[k] = e;                                              // the slot now carries E
                    c[k] += e;                                             // fold, L_ii = 1
                    const double cf = c[k];
                    const double *urow = Us + (b * 8 + j) * QLD + b * 8 + j;
#pragma unroll
                    for (int d = 1; d < 8; ++d)                            // push right inside the leaf
                        if (j + d < 8) y[(k + d) & 7] = fma(cf, urow[d], y[(k + d) & 7]);
                }
#pragma unroll
                for (int d = 1; d < 8; ++d) {                              // fold + push down inside the leaf
                    const double ed = __shfl_up_sync(0xffffffffu, e, d, 8);
                    const double mm = lrow[d] * ed;
                    c[(k + d) & 7] += mm;
                    y[(k + d) & 7] += mm;
                }
            }
            if (live) {
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    int j = (k - i) & 7;
                    Ys[(a * 8 + i) * QLD + b * 8 + j] = y[k];
                    Cs[(a * 8 + i) * QLD + b * 8 + j] = c[k];
                    Zs[(a * 8 + i) * Q + b * 8 + j] = z[k];
                    int gr = row0 + a * 8 + i, gc = col0 + b * 8 + j;
                    if (gr < p.m && gc < p.n) max_abs_e = fmax(max_abs_e, fabs(y[k]));
                }
            }
        }
        __syncthreads();
        if (lw == 14) break;
        // ---------------- phase B: feedback of this leaf-wave to the blocks still to come
        {
            const int pb = warp;                                   // warp owns block row pb
            const int bsrc = lw - pb;                              // leaf (pb, bsrc) pushes right
            const bool has_right = bsrc >= 0 && bsrc <= 7;
            double ar0 = 0.0, ar1 = 0.0;
            if (has_right) {
                ar0 = Cs[(pb * 8 + g) * QLD + bsrc * 8 + t];
                ar1 = Cs[(pb * 8 + g) * QLD + bsrc * 8 + 4 + t];
            }
            for (int qb = max(0, lw - pb + 1); qb < 8; ++qb) {
                double *yp = Ys + (pb * 8 + g) * QLD + qb * 8 + t * 2;
                double2 yv = *reinterpret_cast<double2 *>(yp);
                const int asrc = lw - qb;                          // leaf (asrc, qb) pushes down
                if (asrc >= 0 && asrc <= 7) {
                    double p0 = 0.0, p1 = 0.0;
#pragma unroll
                    for (int kk = 0; kk < 8; kk += 4) {
                        double af = Ls[(pb * 8 + g) * QLD + asrc * 8 + kk + t];
                        double bf = Ys[(asrc * 8 + kk + t) * QLD + qb * 8 + g];
                        dmma_m8n8k4(p0, p1, af, bf);
                    }
                    double *cp = Cs + (pb * 8 + g) * QLD + qb * 8 + t * 2;
                    double2 cv = *reinterpret_cast<double2 *>(cp);
                    cv.x += p0;
                    cv.y += p1;
                    *reinterpret_cast<double2 *>(cp) = cv;
                    yv.x += p0;
                    yv.y += p1;
                }
                if (has_right) {
                    double b0 = Us[(bsrc * 8 + t) * QLD + qb * 8 + g];
                    double b1 = Us[(bsrc * 8 + 4 + t) * QLD + qb * 8 + g];
                    dmma_m8n8k4(yv.x, yv.y, ar0, b0);
                    dmma_m8n8k4(yv.x, yv.y, ar1, b1);
                }
                *reinterpret_cast<double2 *>(yp) = yv;
            }
        }
    }
}

// ---------------------------------------------------------------------------------------------
// in-tile sweep of tile (I, J): Ebuf tile holds X + Rt, Cbuf tile holds Cd on entry;
// E and C = L E on exit.
__device__ __forceinline__ void sweep_tile(int I, int J, double *smem, const TiledKernelParams &p, double &max_abs_e) {
    double *Ys = smem, *Cs = smem + QMAT, *Ls = smem + 2 * QMAT, *Us = smem + 3 * QMAT, *Xop = smem + 4 * QMAT;
    int *Zs = reinterpret_cast<int *>(smem + 5 * QMAT);
    double *eT = p.Ebuf + (long)I * T * p.np + (long)J * T;
    double *cT = p.Cbuf + (long)I * T * p.np + (long)J * T;
    const int tid = threadIdx.x;
#pragma unroll 1
    for (int q = 0; q < 4; ++q) {
        const int qi = q >> 1, qj = q & 1;
        const int row0 = I * T + qi * Q, col0 = J * T + qj * Q;
        double *eQ = eT + (long)qi * Q * p.np + qj * Q;
        double *cQ = cT + (long)qi * Q * p.np + qj * Q;
        __syncthreads();
        load_factor_block(Ls, p.L, p.ldl, p.m, row0, row0, 1);
        load_factor_block(Us, p.U, p.ldu, p.n, col0, col0, 2);
        load_quadrant_cg(Cs, cQ, p.np);
        load_quadrant_cg(Ys, eQ, p.np);
        __syncthreads();
        for (int c = tid; c < Q * Q; c += blockDim.x) {       // Y = X + Rt + Cd
            int r = c >> 6, cc = c & 63;
            Ys[r * QLD + cc] += Cs[r * QLD + cc];
        }
        quadrant_sweep(Ys, Cs, Ls, Us, Zs, row0, col0, p, max_abs_e);
        // results of the quadrant
        store_quadrant(eQ, p.np, Ys);
        store_quadrant(cQ, p.np, Cs);
        for (int c = tid; c < Q * Q; c += blockDim.x) {
            int r = c >> 6, cc = c & 63;
            int gr = row0 + r, gc = col0 + cc;
            if (gr < p.m && gc < p.n) {
                p.Z[(long)gr * p.ldz + gc] = Zs[r * Q + cc];
                if (p.Euser) p.Euser[(long)gr * p.lde + gc] = Ys[r * QLD + cc];
            }
        }
        // cross terms to the quadrants of this tile that follow
        if (q == 0 || q == 2) {   // C of the left quadrant pushes right through U[left cols, right cols]
            load_factor_block(Xop, p.U, p.ldu, p.n, J * T, J * T + Q, 0);
            __syncthreads();
            cross_gemm(eT + (long)qi * Q * p.np + Q, p.np, Cs, Xop);
            __syncthreads();
        }
        if (q == 0 || q == 1) {   // E of the upper quadrant folds down through L[lower rows, upper rows]
            load_factor_block(Xop, p.L, p.ldl, p.m, I * T + Q, I * T, 0);
            __syncthreads();
            cross_gemm(cT + (long)Q * p.np + qj * Q, p.np, Xop, Ys);
            __syncthreads();
        }
    }
}

// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void decode_task(int task, int ntm, int ntn, int &type, int &I, int &J) {
    type = task & 1;
    int tt = task >> 1;
    for (int w = 0; w < ntm + ntn - 1; ++w) {
        int lo = max(0, w - ntn + 1), hi = min(ntm - 1, w);
        int cnt = hi - lo + 1;
        if (tt < cnt) {
            I = lo + tt;
            J = w - I;
            return;
        }
        tt -= cnt;
    }
    I = J = 0;
}

__global__ void __launch_bounds__(TILED_THREADS, 1) round_tiled_kernel(TiledKernelParams p) {
    extern __shared__ __align__(16) double smem[];
    __shared__ int s_task[4];
    __shared__ double s_red[TILED_THREADS / 32];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int wm = warp >> 2, wn = warp & 3, g = lane >> 2, t = lane & 3;
    double max_abs_e = 0.0;

    for (;;) {
        __syncthreads();
        if (tid == 0) {
            int task = (int)atomicAdd(p.counter, 1u);
            int type = 0, I = 0, J = 0;
            if (task < p.ntasks) decode_task(task, p.ntm, p.ntn, type, I, J);
            if (ld_relaxed_u32(p.abort) != 0u) task = p.ntasks;
            s_task[0] = task; s_task[1] = type; s_task[2] = I; s_task[3] = J;
        }
        __syncthreads();
        const int task = s_task[0], type = s_task[1], I = s_task[2], J = s_task[3];
        if (task >= p.ntasks) break;

        // ---------------- bulk contraction: type 0 = Cd (sources above), 1 = Rt (sources left)
        Acc acc;
        acc.zero();
        const int nsrc = type == 0 ? I : J;
        const unsigned *flags = type == 0 ? p.flagS + J : p.flagS + (long)I * p.ntn;
        const long fstride = type == 0 ? p.ntn : 1;
        Operand A, B;
        if (type == 0) {
            A.ptr = p.L + (long)I * T * p.ldl; A.ld = p.ldl; A.mn_valid = min(T, p.m - I * T); A.aligned16 = p.l_al16;
            B.ptr = p.Ebuf + (long)J * T; B.ld = p.np; B.mn_valid = T; B.aligned16 = true;
        } else {
            A.ptr = p.Cbuf + (long)I * T * p.np; A.ld = p.np; A.mn_valid = T; A.aligned16 = true;
            B.ptr = p.U + (long)J * T; B.ld = p.ldu; B.mn_valid = min(T, p.n - J * T); B.aligned16 = p.u_al16;
        }
        bool dead = false;
        for (int pos = 0; pos < nsrc;) {
            int upto = wait_ready_prefix(flags, fstride, pos, nsrc, p, task);
            if (upto < 0) { dead = true; break; }
            Operand a = A, b = B;
            a.ptr = A.ptr + (long)pos * T;                 // k offset along the contiguous index
            b.ptr = B.ptr + (long)pos * T * B.ld;          // k offset along rows
            gemm_mainloop<true, false, BULK_NSTAGE>(acc, smem, a, b, (upto - pos) * T);
            pos = upto;
        }
        if (dead) break;

        // ---------------- bulk epilogue
        {
            double *dstT = (type == 0 ? p.Cbuf : p.Ebuf) + (long)I * T * p.np + (long)J * T;
#pragma unroll
            for (int a = 0; a < 8; ++a) {
                const int r = wm * 64 + a * 8 + g;
                const int gr = I * T + r;
#pragma unroll
                for (int b = 0; b < 4; ++b) {
                    const int c = wn * 32 + b * 8 + t * 2;
                    const int gc = J * T + c;
                    double2 v;
                    v.x = acc.v[a][b][0];
                    v.y = acc.v[a][b][1];
                    if (type == 1) {                       // Y0 = X + Rt, zero outside the matrix
                        double x0 = 0.0, x1 = 0.0;
                        if (gr < p.m) {
                            if (gc < p.n) x0 = __ldg(p.X + (long)gr * p.ldx + gc);
                            if (gc + 1 < p.n) x1 = __ldg(p.X + (long)gr * p.ldx + gc + 1);
                        }
                        v.x += x0;
                        v.y += x1;
                    }
                    *reinterpret_cast<double2 *>(dstT + (long)r * p.np + c) = v;
                }
            }
        }
        __syncthreads();
        if (tid == 0) {
            __threadfence();
            unsigned old = atomicAdd(p.bulk_done + (long)I * p.ntn + J, 1u);
            __threadfence();
            s_task[1] = (old == 1u) ? 1 : 0;
        }
        __syncthreads();
        if (s_task[1]) {
            sweep_tile(I, J, smem, p, max_abs_e);
            __syncthreads();
            if (tid == 0) {
                __threadfence();
                st_release_u32(p.flagS + (long)I * p.ntn + J, 1u);
            }
        }
    }

    for (int o = 16; o > 0; o >>= 1) max_abs_e = fmax(max_abs_e, __shfl_xor_sync(0xffffffffu, max_abs_e, o));
    if (lane == 0) s_red[warp] = max_abs_e;
    __syncthreads();
    if (tid == 0) {
        double v = 0.0;
        for (int w = 0; w < TILED_THREADS / 32; ++w) v = fmax(v, s_red[w]);
        if (v > 0.0) atomic_max_nonneg_double(p.max_abs_e, v);
    }
}

// ---------------------------------------------------------------------------------------------
static size_t pad256(size_t x) { return (x + 255) / 256 * 256; }

struct TiledLayout {
    int ntm, ntn;
    size_t flags_off, done_off, e_off, c_off, total;
};
static TiledLayout tiled_layout(int m, int n) {
    TiledLayout l;
    l.ntm = (m + T - 1) / T;
    l.ntn = (n + T - 1) / T;
    size_t tiles = (size_t)l.ntm * l.ntn;
    size_t mat = (size_t)l.ntm * T * (size_t)l.ntn * T * sizeof(double);
    l.flags_off = 256;
    l.done_off = l.flags_off + pad256(tiles * sizeof(unsigned));
    l.e_off = l.done_off + pad256(tiles * sizeof(unsigned));
    l.c_off = l.e_off + pad256(mat);
    l.total = l.c_off + pad256(mat);
    return l;
}

size_t round_tiled_workspace_bytes(int m, int n) { return tiled_layout(m, n).total; }

int launch_round_tiled(const TiledParams &in, void *ws, size_t ws_bytes, cudaStream_t stream) {
    TiledLayout l = tiled_layout(in.m, in.n);
    if (ws_bytes < l.total) return GPTQ2D_ERR_WORKSPACE;
    char *w = static_cast<char *>(ws);
    TiledKernelParams p{};
    p.m = in.m; p.n = in.n; p.ntm = l.ntm; p.ntn = l.ntn;
    p.ntasks = 2 * l.ntm * l.ntn;
    p.np = (long)l.ntn * T;
    p.X = in.X; p.ldx = in.ldx; p.L = in.L; p.ldl = in.ldl; p.U = in.U; p.ldu = in.ldu;
    p.Z = in.Z; p.ldz = in.ldz; p.Euser = in.E; p.lde = in.lde;
    p.counter = reinterpret_cast<unsigned *>(w);
    p.abort = reinterpret_cast<unsigned *>(w) + 1;
    p.max_abs_e = workspace_max_abs_e(ws);
    p.flagS = reinterpret_cast<unsigned *>(w + l.flags_off);
    p.bulk_done = reinterpret_cast<unsigned *>(w + l.done_off);
    p.Ebuf = reinterpret_cast<double *>(w + l.e_off);
    p.Cbuf = reinterpret_cast<double *>(w + l.c_off);
    p.info = in.info;
    p.l_al16 = ((reinterpret_cast<uintptr_t>(in.L) & 15) == 0) && ((in.ldl & 1) == 0);
    p.u_al16 = ((reinterpret_cast<uintptr_t>(in.U) & 15) == 0) && ((in.ldu & 1) == 0);

    if (cudaMemsetAsync(w, 0, l.e_off, stream) != cudaSuccess) return GPTQ2D_ERR_CUDA;   // header, flags, counters
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return GPTQ2D_ERR_CUDA;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return GPTQ2D_ERR_CUDA;
    if (cudaFuncSetAttribute(round_tiled_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)TILED_SMEM) !=
        cudaSuccess)
        return GPTQ2D_ERR_CUDA;
    int grid = sms < p.ntasks ? sms : p.ntasks;
    void *args[] = {&p};
    if (cudaLaunchCooperativeKernel((const void *)round_tiled_kernel, dim3(grid), dim3(TILED_THREADS), args,
                                    TILED_SMEM, stream) != cudaSuccess)
        return GPTQ2D_ERR_CUDA;
    return GPTQ2D_OK;
}

}  // namespace gptq2d
