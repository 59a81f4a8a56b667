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
// sweep runs on 8 x 8 leaves: each leaf of a leaf-wave is swept by one warp (two entries per
// lane, errors exchanged through a 16-double shared-memory buffer, branch-free pushes), then
// all warps apply the leaves' feedback to the remaining 8 x 8 blocks of the quadrant with
// m8n8k4 DMMA.
#include "common.cuh"
#include "dmma_gemm.cuh"
#include "round_internal.cuh"

namespace gptq2d {

constexpr int T = 128;           // tile edge
constexpr int Q = 64;            // quadrant edge
constexpr int QLD = 68;          // shared-memory row stride of quadrant matrices (68 mod 16 == 4)
constexpr int QMAT = Q * QLD;    // doubles per quadrant matrix
constexpr int TAB_LD = 24;       // row stride of the leaf coefficient tables (22 used)
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

constexpr size_t SWEEP_SMEM = (size_t)(5 * QMAT + 2 * Q * TAB_LD) * sizeof(double) + (size_t)Q * Q * sizeof(int);
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
// quadrant <-> shared memory.  The *_async loaders only issue cp.async copies; the caller
// commits, waits and barriers once for all operands of a quadrant.
__device__ __forceinline__ void load_quadrant_async(double *dst, const double *src, long ld) {
    // dense 64 x 64 from a padded workspace buffer (always in range, 16-byte aligned); L2 only
#pragma unroll
    for (int it = 0; it < 8; ++it) {
        int c = threadIdx.x + it * TILED_THREADS;
        cp_async16(dst + (c >> 5) * QLD + (c & 31) * 2, src + (long)(c >> 5) * ld + (c & 31) * 2, 16);
    }
}
__device__ __forceinline__ void store_quadrant(double *dst, long ld, const double *src) {
#pragma unroll
    for (int it = 0; it < 8; ++it) {
        int c = threadIdx.x + it * TILED_THREADS;
        int r = c >> 5, cc = (c & 31) * 2;
        *reinterpret_cast<double2 *>(dst + (long)r * ld + cc) = *reinterpret_cast<const double2 *>(src + r * QLD + cc);
    }
}
// 64 x 64 block of a user matrix (k x k, leading dimension ld) whose top-left element is
// (r0, c0); mode 0: everything in range, 1: strictly lower part only, 2: strictly upper only
// (relative to the matrix diagonal).  Out-of-range and masked elements become zero.
__device__ __forceinline__ void load_factor_block_async(double *dst, const double *M, long ld, int k, int r0, int c0,
                                                        int mode) {
#pragma unroll
    for (int it = 0; it < 16; ++it) {
        int c = threadIdx.x + it * TILED_THREADS;
        int r = c >> 6, cc = c & 63;
        int gr = r0 + r, gc = c0 + cc;
        bool take = gr < k && gc < k;
        if (mode == 1) take = take && gc < gr;
        if (mode == 2) take = take && gc > gr;
        cp_async8(dst + r * QLD + cc, take ? M + (long)gr * ld + gc : M, take ? 8 : 0);
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

// One 8 x 8 target block (pb, qb) of the quadrant receives the feedback of leaf-wave `lw`:
// the downward push of leaf (lw - qb, qb) through L and the rightward push of leaf
// (pb, lw - pb) through U, as m8n8k4 products on the warp's fragments.  Warp-uniform.
__device__ __forceinline__ void block_feedback(double *Ys, double *Cs, const double *Ls, const double *Us, int lw,
                                               int pb, int qb, int g, int t) {
    const int asrc = lw - qb, bsrc = lw - pb;
    const bool down = asrc >= 0 && asrc < pb, right = bsrc >= 0 && bsrc < qb;
    if (!down && !right) return;
    double *yp = Ys + (pb * 8 + g) * QLD + qb * 8 + t * 2;
    double2 yv = *reinterpret_cast<double2 *>(yp);
    if (down) {
        double p0 = 0.0, p1 = 0.0;
        dmma_m8n8k4(p0, p1, Ls[(pb * 8 + g) * QLD + asrc * 8 + t], Ys[(asrc * 8 + t) * QLD + qb * 8 + g]);
        dmma_m8n8k4(p0, p1, Ls[(pb * 8 + g) * QLD + asrc * 8 + 4 + t], Ys[(asrc * 8 + 4 + t) * QLD + qb * 8 + g]);
        double *cp = Cs + (pb * 8 + g) * QLD + qb * 8 + t * 2;
        double2 cv = *reinterpret_cast<double2 *>(cp);
        cv.x += p0;
        cv.y += p1;
        *reinterpret_cast<double2 *>(cp) = cv;
        yv.x += p0;
        yv.y += p1;
    }
    if (right) {
        dmma_m8n8k4(yv.x, yv.y, Cs[(pb * 8 + g) * QLD + bsrc * 8 + t], Us[(bsrc * 8 + t) * QLD + qb * 8 + g]);
        dmma_m8n8k4(yv.x, yv.y, Cs[(pb * 8 + g) * QLD + bsrc * 8 + 4 + t], Us[(bsrc * 8 + 4 + t) * QLD + qb * 8 + g]);
    }
    *reinterpret_cast<double2 *>(yp) = yv;
}

// ---------------------------------------------------------------------------------------------
// Algorithm 3 on one 64 x 64 quadrant held in shared memory.
//   Ys: in  Y (corrected values, already including the C the quadrant starts with)
//       out E (local errors)
//   Cs: in  C at entry; out final C = L E rows of the quadrant
//   Ls / Us: strictly lower / strictly upper 64 x 64 diagonal blocks of the factors
//   Zs: out rounded integers
// row0/col0: global coordinates of the quadrant (for masking the status checks).
//
// Leaf-wave lw (leaves (a, lw - a)) runs in two barrier-separated parts:
//   part 1: each leaf is swept by one warp (phase A); meanwhile every warp applies the feedback
//           of the PREVIOUS leaf-wave to the blocks of its block row that lie two or more
//           leaf-waves ahead (interleaved with the sweep steps, which are latency bound);
//   part 2: every warp applies the feedback of THIS leaf-wave to the one block of its block
//           row that belongs to the next leaf-wave.
__device__ __forceinline__ void quadrant_sweep(double *Ys, double *Cs, const double *Ls, const double *Us, int *Zs,
                                               double *tabL, double *tabU, int row0, int col0,
                                               const TiledKernelParams &p, double &max_abs_e) {
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, t = lane & 3;
    __shared__ double xch[8 * 2 * 16];
    __shared__ unsigned long long s_badkey;
    // coefficient tables of the 8 diagonal leaves (see phase A); also clears the exchange buffers
    for (int c = tid; c < Q * TAB_LD; c += blockDim.x) {
        const int r = c / TAB_LD, k = c - r * TAB_LD;       // r: row (L) or column (U) inside the quadrant
        const int src = k - 7, blk = r & ~7, in = r & 7;    // source index inside the leaf
        const bool ok = src >= 0 && src < in;
        tabL[c] = ok ? Ls[r * QLD + blk + src] : 0.0;
        tabU[c] = ok ? Us[(blk + src) * QLD + r] : 0.0;
    }
    if (tid < 8 * 2 * 16) xch[tid] = 0.0;
    if (tid == 0) s_badkey = ~0ull;
    unsigned long long badkey = ~0ull;

    for (int lw = 0; lw < 15; ++lw) {
        __syncthreads();
        // ---------------- part 1
        const int a_lo = max(0, lw - 7), a_hi = min(7, lw);
        const int a = a_lo + warp, b = lw - a;
        if (a <= a_hi) {
            // Phase A.  Lane l owns entries (i0, j) and (i0 + 4, j) of the 8 x 8 leaf, i0 = l & 3,
            // j = l >> 2.  At step s the lane whose entry lies on anti-diagonal s rounds it and posts
            // the error (by column) and the final C value (by row) to a 16-double per-warp exchange
            // buffer; after a warp barrier EVERY lane applies one downward and one rightward push
            // to both of its entries (Algorithm 3 lines 8-16 restricted to the leaf).  The pushes
            // are branch-free: the coefficients come from tables that hold zeros wherever no push
            // is due (source not on this anti-diagonal, or entry already rounded), so stale
            // exchange slots are multiplied by zero.
            const int i0 = lane & 3, j = lane >> 2;
            double *yp = Ys + (a * 8 + i0) * QLD + b * 8 + j;
            double *cp = Cs + (a * 8 + i0) * QLD + b * 8 + j;
            double y0 = yp[0], y1 = yp[4 * QLD], c0 = cp[0], c1 = cp[4 * QLD];
            // tabL[row][7 + is] = L(row, is) for 0 <= is < row else 0; at step s, is = s - j
            const double *tl0 = tabL + (a * 8 + i0) * TAB_LD + 7 - j;
            const double *tl1 = tl0 + 4 * TAB_LD;
            // tabU[col][7 + js] = U(js, col) for 0 <= js < col else 0; at step s, js = s - i
            const double *tu0 = tabU + (b * 8 + j) * TAB_LD + 7 - i0;
            const double *tu1 = tu0 - 4;
            double *exw = xch + warp * 32;
            int z0 = 0, z1 = 0;
            const int t0 = i0 + j, t1 = t0 + 4;
#pragma unroll
            for (int s = 0; s < 15; ++s) {
                double *ex = exw + (s & 1) * 16;                        // [0..7] e by column, [8..15] C by row
                const bool r0 = (t0 == s), r1 = (t1 == s);
                if (r0 || r1) {
                    const double yv = r0 ? y0 : y1;
                    const double zv = rint(yv);
                    const double e = zv - yv;                           // line 5: E = Z - Y
                    const double cf = (r0 ? c0 : c1) + e;               // fold, L_ii = 1
                    ex[j] = e;
                    ex[8 + i0 + (r0 ? 0 : 4)] = cf;
                    if (r0) { y0 = e; c0 = cf; z0 = (int)zv; }
                    else { y1 = e; c1 = cf; z1 = (int)zv; }
                    if (!(fabs(yv) < 2147483648.0)) {                   // not representable: remember the first
                        const unsigned long long gr = row0 + a * 8 + i0 + (r0 ? 0 : 4), gc = col0 + b * 8 + j;
                        const unsigned long long key = ((gr + gc) << 42) | ((isfinite(yv) ? 1ull : 0ull) << 41) |
                                                       (gr << 20) | gc;
                        if (gr < (unsigned long long)p.m && gc < (unsigned long long)p.n && key < badkey) badkey = key;
                    }
                }
                __syncwarp();
                if (s < 8 && warp + s > lw) block_feedback(Ys, Cs, Ls, Us, lw - 1, warp, s, g, t);   // far feedback
                const double ed = ex[j], cr0 = ex[8 + i0], cr1 = ex[12 + i0];
                const double l0 = tl0[s], l1 = tl1[s], u0 = tu0[s], u1 = tu1[s];
                y0 = fma(l0, ed, y0); c0 = fma(l0, ed, c0); y0 = fma(cr0, u0, y0);   // fold, push down, push right
                y1 = fma(l1, ed, y1); c1 = fma(l1, ed, c1); y1 = fma(cr1, u1, y1);
            }
            yp[0] = y0; yp[4 * QLD] = y1; cp[0] = c0; cp[4 * QLD] = c1;
            Zs[(a * 8 + i0) * Q + b * 8 + j] = z0;
            Zs[(a * 8 + i0 + 4) * Q + b * 8 + j] = z1;
            if (col0 + b * 8 + j < p.n) {
                if (row0 + a * 8 + i0 < p.m) max_abs_e = fmax(max_abs_e, fabs(y0));
                if (row0 + a * 8 + i0 + 4 < p.m) max_abs_e = fmax(max_abs_e, fabs(y1));
            }
        } else if (lw > 0) {
            // no leaf for this warp in this leaf-wave: only the far feedback of the previous one
#pragma unroll
            for (int qb = 0; qb < 8; ++qb)
                if (warp + qb > lw) block_feedback(Ys, Cs, Ls, Us, lw - 1, warp, qb, g, t);
        }
        __syncthreads();
        if (lw == 14) break;
        // ---------------- part 2: feedback of this leaf-wave to the next one
        {
            const int qb = lw + 1 - warp;
            if (qb >= 0 && qb < 8) block_feedback(Ys, Cs, Ls, Us, lw, warp, qb, g, t);
        }
    }
    // status: the earliest (in sweep order) unrepresentable value of the quadrant, if any
    if (badkey != ~0ull) atomicMin(&s_badkey, badkey);
    __syncthreads();
    if (tid == 0 && s_badkey != ~0ull) {
        const unsigned long long k = s_badkey;
        report(p.info, ((k >> 41) & 1ull) ? GPTQ2D_ERR_INT_OVERFLOW : GPTQ2D_ERR_NONFINITE,
               (int)((k >> 20) & 0x1fffffull), (int)(k & 0xfffffull), 0);
    }
}

// ---------------------------------------------------------------------------------------------
// in-tile sweep of tile (I, J): Ebuf tile holds X + Rt, Cbuf tile holds Cd on entry;
// E and C = L E on exit.
__device__ __forceinline__ void sweep_tile(int I, int J, double *smem, const TiledKernelParams &p, double &max_abs_e) {
    double *Ys = smem, *Cs = smem + QMAT, *Ls = smem + 2 * QMAT, *Us = smem + 3 * QMAT, *Xop = smem + 4 * QMAT;
    double *tabL = smem + 5 * QMAT, *tabU = tabL + Q * TAB_LD;
    int *Zs = reinterpret_cast<int *>(tabU + Q * TAB_LD);
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
        load_factor_block_async(Ls, p.L, p.ldl, p.m, row0, row0, 1);
        load_factor_block_async(Us, p.U, p.ldu, p.n, col0, col0, 2);
        load_quadrant_async(Cs, cQ, p.np);
        load_quadrant_async(Ys, eQ, p.np);
        // the operand of the first cross term that follows this quadrant
        if (q == 0 || q == 2) load_factor_block_async(Xop, p.U, p.ldu, p.n, J * T, J * T + Q, 0);
        if (q == 1) load_factor_block_async(Xop, p.L, p.ldl, p.m, I * T + Q, I * T, 0);
        cp_async_commit();
        cp_async_wait<0>();
        __syncthreads();
#pragma unroll
        for (int it = 0; it < 16; ++it) {                     // Y = X + Rt + Cd
            int c = tid + it * TILED_THREADS;
            int r = c >> 6, cc = c & 63;
            Ys[r * QLD + cc] += Cs[r * QLD + cc];
        }
        quadrant_sweep(Ys, Cs, Ls, Us, Zs, tabL, tabU, row0, col0, p, max_abs_e);
        // results of the quadrant
        store_quadrant(eQ, p.np, Ys);
        store_quadrant(cQ, p.np, Cs);
#pragma unroll
        for (int it = 0; it < 16; ++it) {
            int c = tid + it * TILED_THREADS;
            int r = c >> 6, cc = c & 63;
            int gr = row0 + r, gc = col0 + cc;
            if (gr < p.m && gc < p.n) {
                p.Z[(long)gr * p.ldz + gc] = Zs[r * Q + cc];
                if (p.Euser) p.Euser[(long)gr * p.lde + gc] = Ys[r * QLD + cc];
            }
        }
        // cross terms to the quadrants of this tile that follow
        if (q == 0 || q == 2)     // C of the left quadrant pushes right through U[left cols, right cols]
            cross_gemm(eT + (long)qi * Q * p.np + Q, p.np, Cs, Xop);
        if (q == 0) {
            __syncthreads();
            load_factor_block_async(Xop, p.L, p.ldl, p.m, I * T + Q, I * T, 0);
            cp_async_commit();
            cp_async_wait<0>();
            __syncthreads();
        }
        if (q == 0 || q == 1)     // E of the upper quadrant folds down through L[lower rows, upper rows]
            cross_gemm(cT + (long)Q * p.np + qj * Q, p.np, Xop, Ys);
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
