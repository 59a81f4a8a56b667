// GPTQ-2D sweep (fp64) with the dense feedback and the dependent chain running SIDE BY SIDE on every SM.
//
// Same restatement of Algorithm 3 on 128 x 128 tiles as round_tiled.cu (Eq. 11, Eq. 15-17): for tile
// (I, J), Cd = sum_{I' < I} L[r, I'] E[I', c] and Rt = sum_{J' < J} C[r, J'] U[J', c] are dense
// contractions, and Algorithm 3 on the tile alone, started from Y = X + Rt + Cd, C = Cd, gives the
// tile's Z, E and C = L E.  There, one CTA of eight warps does either a far contraction or a 64 x 64
// quadrant task at a time, so the fp64 tensor pipe of an SM idles for most of every quadrant task
// (leaf sweeps are chains of dependent rint / add / fma steps).  Here a CTA has sixteen warps with two
// fixed roles that share nothing but the device-wide scheduler words:
//   * warps 0-7, the FAR group: claim far parts wave by wave from one atomic counter and run them as a
//     DMMA contraction on a 128 x 64 register accumulator, operand slabs brought in by TMA
//     (cp.async.bulk.tensor, 128-byte swizzle; every CTA fetches its own copy) through a three-stage mbarrier
//     ring.  The group synchronises only with itself (mbarriers, one named barrier per far part).
//   * warps 8-15, the QUADRANT group: serve the ready ring; a quadrant task is the one of round_tiled.cu
//     (pulls from the two nearest tiles, then 15 leaf-waves streamed from its two neighbours) on the
//     group's own 150 KB of shared memory, synchronising on its own named barrier.
// The warp schedulers interleave the two: while a leaf sweep waits on its dependent arithmetic the far
// group's DMMAs keep the tensor pipe busy, and the quadrant task's own products share the pipe.
//
// Far parts are half tiles (128 rows x 64 columns): that halves the accumulator (64 registers a thread),
// which is what lets sixteen warps fit the register file at 128 registers each, at the price of reading
// the row operand twice (from L2: the two halves of a tile are claimed back to back).  Each half
// announces itself to the two quadrants below it.
//
// Requirements beyond round_tiled.cu: L and U 16-byte aligned with even leading dimensions (TMA row
// pitch).  launch_round_fused returns -1 when it cannot take the problem; the caller then uses the
// eight-warp kernel.  Every wait (flags, ring, mbarriers) is bounded and raises the abort word.
#include <cstdio>
#include "common.cuh"
#include "dmma_gemm.cuh"
#include "dmma_tma.cuh"
#include "tma_host.cuh"
#include "round_internal.cuh"

namespace gptq2d {
namespace fused {

constexpr int T = 128;            // tile edge
constexpr int Q = 64;             // quadrant edge
constexpr int QLD = 68;           // shared-memory row stride of quadrant matrices (68 mod 16 == 4)
constexpr int QMAT = Q * QLD;
constexpr int TAB_LD = 24;        // row stride of the leaf coefficient tables (22 used)
// far warps pause between slabs while the SM's quadrant group sweeps leaves: measured 42.6 ms at 8192^2 against
// 40.5 without (the far group loses more than the chain gains), 7.9 against 10.2 ms at 4096^2; off
constexpr bool FUSED_THROTTLE = false;
constexpr int F_WARPS = 8;        // far warps: 2 x 2 (64 x 32 each) or 4 x 2 (32 x 32 each)
constexpr int F_THREADS = 32 * F_WARPS;
constexpr int F_FRAGS_M = 32 / F_WARPS;   // row fragments of a far warp
constexpr int GROUP = 256;        // threads of the quadrant group
constexpr int THREADS = F_THREADS + GROUP;
constexpr int FN = 64;            // columns of a far part
constexpr int F_NSTAGE = 3;
constexpr int F_A_DOUBLES = 128 * TMA_BK;                 // row operand slab: 128 rows x 16 k (K-contiguous)
constexpr int F_B_DOUBLES = TMA_BK * FN;                  // column operand slab: 4 boxes of 16 k x 16 columns
constexpr int F_STAGE_DOUBLES = F_A_DOUBLES + F_B_DOUBLES;
constexpr unsigned F_STAGE_BYTES = F_STAGE_DOUBLES * 8;   // 24 KB
constexpr int STG_E_LD = 12;                 // staged 64 x 8 column block of E, [k][n], 12 = 8 + 4 pad
constexpr int STG_E = Q * STG_E_LD;
constexpr int STG_C = 8 * QLD;               // staged 8 x 64 row block of C, [m][k]
constexpr int Q_AUX_DOUBLES = 2 * Q * TAB_LD + 2 * STG_E + 2 * STG_C;      // tables + streaming stages (45.5 KB)
static_assert(Q_AUX_DOUBLES >= QMAT, "the auxiliary region doubles as a staging matrix during start-up");
constexpr int Q_DOUBLES = 3 * QMAT + Q_AUX_DOUBLES;
constexpr size_t FUSED_SMEM = (size_t)(F_NSTAGE * F_STAGE_DOUBLES + Q_DOUBLES) * sizeof(double) + 1024;

struct FusedParams {
    int m, n, ntm, ntn, ntasks, ntiles_total;
    long np;                     // leading dimension of Ebuf / Cbuf (= ntn * 128)
    const double *X; long ldx;
    const double *L; long ldl;
    const double *U; long ldu;
    int *Z; long ldz;
    double *Euser; long lde;
    double *Ebuf, *Cbuf;
    unsigned *counter, *abort, *q_head, *q_tail, *tiles_done;
    unsigned *q_slots; unsigned qmask;
    unsigned *flagS, *quad_done, *qdep, *qprog, *rowdone;
    double *max_abs_e;
    int *info;
    int l_al16, u_al16;
    unsigned long long spin_limit;
};

template <int COUNT>
__device__ __forceinline__ void group_sync(int id) { asm volatile("bar.sync %0, %1;\n" ::"r"(id), "n"(COUNT) : "memory"); }
#define FSYNC() group_sync<F_THREADS>(1)
#define QSYNC() group_sync<GROUP>(2)

// optional in-kernel timing (scratch builds only: -DFUSED_STATS), cycles summed by one thread per group
#ifdef FUSED_STATS
#define STAT_DECL(x) long long x = 0
#define STAT_T0(t) const long long t = clock64()
#define STAT_ADD(x, t) x += clock64() - t
#else
#define STAT_DECL(x)
#define STAT_T0(t)
#define STAT_ADD(x, t)
#endif

// ---------------------------------------------------------------------------------------------
// quadrant group: loaders (index by the thread's position in the group)
__device__ __forceinline__ void load_quadrant_async(double *dst, const double *src, long ld, int qtid) {
#pragma unroll
    for (int it = 0; it < 8; ++it) {
        int c = qtid + it * GROUP;
        cp_async16(dst + (c >> 5) * QLD + (c & 31) * 2, src + (long)(c >> 5) * ld + (c & 31) * 2, 16);
    }
}
__device__ __forceinline__ void load_block_async8(double *dst, const double *M, long ld, int rows, int cols, int r0, int c0,
                                                  int qtid) {
#pragma unroll
    for (int it = 0; it < 16; ++it) {
        int c = qtid + it * GROUP;
        int r = c >> 6, cc = c & 63;
        int gr = r0 + r, gc = c0 + cc;
        bool take = gr < rows && gc < cols;
        cp_async8(dst + r * QLD + cc, take ? M + (long)gr * ld + gc : M, take ? 8 : 0);
    }
}
__device__ __forceinline__ void load_block_async16(double *dst, const double *M, long ld, int rows, int cols, int r0, int c0,
                                                   int qtid) {
#pragma unroll
    for (int it = 0; it < 8; ++it) {
        int c = qtid + it * GROUP;
        int r = c >> 5, cc = (c & 31) * 2;
        int gr = r0 + r, gc = c0 + cc;
        int nv = (gr < rows) ? min(2, max(0, cols - gc)) : 0;
        cp_async16(dst + r * QLD + cc, nv ? M + (long)gr * ld + gc : M, nv * 8);
    }
}
// 64 x 64 diagonal blocks of both factors in one matrix: below the diagonal L, above it U, zeros elsewhere
__device__ __forceinline__ void load_lu_diag_async(double *dst, const FusedParams &p, int r0, int c0, int qtid) {
#pragma unroll
    for (int it = 0; it < 16; ++it) {
        const int c = qtid + it * GROUP;
        const int i = c >> 6, j = c & 63;
        const bool lower = j < i, upper = j > i;
        const bool take = lower ? (r0 + i < p.m) : (upper && c0 + j < p.n);
        const double *src = lower ? p.L + (long)(r0 + i) * p.ldl + r0 + j : p.U + (long)(c0 + i) * p.ldu + c0 + j;
        cp_async8(dst + i * QLD + j, take ? src : p.L, take ? 8 : 0);
    }
}

struct QAcc {
    double v[2][4][2];
    __device__ __forceinline__ void zero() {
#pragma unroll
        for (int a = 0; a < 2; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) v[a][b][0] = v[a][b][1] = 0.0;
    }
};
// acc += As (64 x 64, [m][k]) * Bs (64 x 64, [k][n]); warp w of the group owns a 16 x 32 piece
__device__ __forceinline__ void quad_mma(QAcc &acc, const double *As, const double *Bs, int warp, int lane) {
    const int g = lane >> 2, t = lane & 3;
    const int wr = warp >> 1, wc = warp & 1;
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
            for (int b = 0; b < 4; ++b) dmma_m8n8k4(acc.v[a][b][0], acc.v[a][b][1], af[a], bf[b]);
    }
}
// the warp's piece of a 64 x 64 matrix (row stride ld; shared or global memory) <-> accumulator
__device__ __forceinline__ void quad_store_to(double *D, long ld, const QAcc &acc, int warp, int lane) {
    const int g = lane >> 2, t = lane & 3;
    const int wr = warp >> 1, wc = warp & 1;
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            double2 v;
            v.x = acc.v[a][b][0];
            v.y = acc.v[a][b][1];
            *reinterpret_cast<double2 *>(D + (long)(wr * 16 + a * 8 + g) * ld + wc * 32 + b * 8 + t * 2) = v;
        }
}
__device__ __forceinline__ void quad_load_from(QAcc &acc, const double *D, long ld, int warp, int lane) {
    const int g = lane >> 2, t = lane & 3;
    const int wr = warp >> 1, wc = warp & 1;
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            const double2 v = __ldcg(reinterpret_cast<const double2 *>(D + (long)(wr * 16 + a * 8 + g) * ld + wc * 32 + b * 8 + t * 2));
            acc.v[a][b][0] = v.x;
            acc.v[a][b][1] = v.y;
        }
}
// left-looking feedback of the leaves already swept into leaf (a, b); see round_tiled.cu
__device__ __forceinline__ void leaf_pull(double *Ys, double *Cs, const double *Ls, const double *Us, int a, int b,
                                          int g, int t) {
    double p0 = 0.0, p1 = 0.0, p2 = 0.0, p3 = 0.0, r0 = 0.0, r1 = 0.0, r2 = 0.0, r3 = 0.0;
    const double *La = Ls + (a * 8 + g) * QLD + t;
    const double *Eb = Ys + t * QLD + b * 8 + g;
#pragma unroll 2
    for (int ap = 0; ap < a; ++ap) {
        dmma_m8n8k4(p0, p1, La[ap * 8], Eb[(ap * 8) * QLD]);
        dmma_m8n8k4(p2, p3, La[ap * 8 + 4], Eb[(ap * 8 + 4) * QLD]);
    }
    const double *Ca = Cs + (a * 8 + g) * QLD + t;
    const double *Ub = Us + t * QLD + b * 8 + g;
#pragma unroll 2
    for (int bp = 0; bp < b; ++bp) {
        dmma_m8n8k4(r0, r1, Ca[bp * 8], Ub[(bp * 8) * QLD]);
        dmma_m8n8k4(r2, r3, Ca[bp * 8 + 4], Ub[(bp * 8 + 4) * QLD]);
    }
    p0 += p2; p1 += p3;
    double *yp = Ys + (a * 8 + g) * QLD + b * 8 + t * 2;
    double *cp = Cs + (a * 8 + g) * QLD + b * 8 + t * 2;
    double2 yv = *reinterpret_cast<double2 *>(yp), cv = *reinterpret_cast<double2 *>(cp);
    cv.x += p0; cv.y += p1;
    yv.x += p0 + (r0 + r2); yv.y += p1 + (r1 + r3);
    *reinterpret_cast<double2 *>(yp) = yv;
    *reinterpret_cast<double2 *>(cp) = cv;
}

struct Stream {
    const unsigned *prog_above, *prog_left;
    unsigned *prog_self;
    const double *e_above, *c_left;
    int I, J, q;
};

// one warp: lane 0 polls until both progress words have reached `need` (bounded)
__device__ __forceinline__ void await_progress(const FusedParams &p, const unsigned *wa, const unsigned *wl, unsigned need,
                                               int lane) {
    if (lane == 0) {
        unsigned long long it = 0;
        for (;;) {
            const unsigned va = wa ? ld_acquire_u32(wa) : need, vl = wl ? ld_acquire_u32(wl) : need;
            if (va >= need && vl >= need) break;
            if (++it > p.spin_limit || ld_relaxed_u32(p.abort) != 0u) {
                report(p.info, GPTQ2D_ERR_DEVICE_TIMEOUT, -8, (int)need, (int)blockIdx.x);
                atomicExch(p.abort, 1u);
                break;
            }
            __nanosleep(40);
        }
    }
    __syncwarp();
}

// ---- ready ring and arrivals (same protocol as round_tiled.cu) --------------------------------
__device__ __forceinline__ void ready_push(const FusedParams &p, unsigned entry) {
    unsigned t = atomicAdd(p.q_tail, 1u);
    st_release_u32(p.q_slots + (t & p.qmask), entry | 0x80000000u);
}
__device__ __forceinline__ unsigned ready_pop(const FusedParams &p) {
    for (;;) {
        unsigned h = ld_relaxed_u32(p.q_head), t = ld_relaxed_u32(p.q_tail);
        if ((int)(t - h) <= 0) return 0u;
        if (atomicCAS(p.q_head, h, h + 1u) != h) continue;
        unsigned *slot = p.q_slots + (h & p.qmask);
        unsigned long long spins = 0;
        unsigned e;
        while ((e = ld_acquire_u32(slot)) == 0u) {
            if (++spins > p.spin_limit || ld_relaxed_u32(p.abort) != 0u) {
                report(p.info, GPTQ2D_ERR_DEVICE_TIMEOUT, -3, (int)h, (int)blockIdx.x);
                atomicExch(p.abort, 1u);
                return 0u;
            }
        }
        *slot = 0u;
        return e;
    }
}
__device__ __forceinline__ unsigned quadrant_needed(int I, int J, int q) {
    const int r = 2 * I + (q >> 1), c = 2 * J + (q & 1);
    return 2u + (r >= 1 ? 1u : 0u) + (c >= 1 ? 1u : 0u);
}
__device__ __forceinline__ bool quadrant_exists(const FusedParams &p, int I, int J, int q) {
    return I * T + (q >> 1) * Q < p.m && J * T + (q & 1) * Q < p.n;
}
__device__ __forceinline__ void quadrant_arrive(const FusedParams &p, int I, int J, int q) {
    if (!quadrant_exists(p, I, J, q)) return;
    unsigned old = atomicAdd(p.qdep + ((long)I * p.ntn + J) * 4 + q, 1u);
    if (old + 1u == quadrant_needed(I, J, q)) {
        const unsigned entry = ((unsigned)q << 29) | ((unsigned)I << 15) | (unsigned)J | 0x80000000u;
        __threadfence();
        ready_push(p, entry);
    }
}

// Algorithm 3 on one 64 x 64 quadrant in shared memory, streamed from its two neighbours; identical in
// arithmetic and order to quadrant_sweep of round_tiled.cu.  The off-diagonal factor blocks that feed
// the streamed pulls (L[rows, rows above], U[columns left, columns]) come as register fragments:
// lfa[i] = L[row block `warp`, k = t + 4 i], ufl[i] = U[k = t + 4 i, column block `warp`].
__device__ __forceinline__ void quadrant_sweep(double *Ys, double *Cs, const double *LU, const double (&lfa)[16],
                                               const double (&ufl)[16], double *stg, double *tabL, double *tabU,
                                               double *xch, unsigned long long *s_badkey, int row0, int col0,
                                               const Stream &sm, const FusedParams &p, double &max_abs_e, int qtid) {
    const int warp = qtid >> 5, lane = qtid & 31;
    const int g = lane >> 2, t = lane & 3;
    const double *Ls = LU, *Us = LU;
    for (int c = qtid; c < Q * TAB_LD; c += GROUP) {
        const int r = c / TAB_LD, k = c - r * TAB_LD;
        const int src = k - 7, blk = r & ~7, in = r & 7;
        const bool ok = src >= 0 && src < in;
        tabL[c] = ok ? Ls[r * QLD + blk + src] : 0.0;
        tabU[c] = ok ? Us[(blk + src) * QLD + r] : 0.0;
    }
    if (qtid < 8 * 2 * 16) xch[qtid] = 0.0;
    if (qtid == 0) *s_badkey = ~0ull;
    unsigned long long badkey = ~0ull;
    const bool fresh = sm.prog_above != nullptr || sm.prog_left != nullptr;
    double *stgE = stg, *stgC = stg + 2 * STG_E;
    auto fetch_block = [&](int blk) {
        await_progress(p, sm.prog_above, sm.prog_left, (unsigned)(blk + 8), lane);
        if (sm.prog_above) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int piece = lane + 32 * i, r = piece >> 2, c2 = (piece & 3) * 2;
                cp_async16(stgE + (blk & 1) * STG_E + r * STG_E_LD + c2, sm.e_above + (long)r * p.np + blk * 8 + c2, 16);
            }
        }
        if (sm.prog_left) {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int piece = lane + 32 * i, r = piece >> 5, c2 = (piece & 31) * 2;
                cp_async16(stgC + (blk & 1) * STG_C + r * QLD + c2, sm.c_left + (long)(blk * 8 + r) * p.np + c2, 16);
            }
        }
        cp_async_commit();
        cp_async_wait<0>();
    };
    if (qtid == 7 * 32) {
        const int qi = sm.q >> 1, qj = sm.q & 1;
        if (qi == 0) quadrant_arrive(p, sm.I, sm.J, sm.q + 2);
        else if (sm.I + 1 < p.ntm) quadrant_arrive(p, sm.I + 1, sm.J, sm.q - 2);
        if (qj == 0) quadrant_arrive(p, sm.I, sm.J, sm.q + 1);
        else if (sm.J + 1 < p.ntn) quadrant_arrive(p, sm.I, sm.J + 1, sm.q - 1);
    }
    __syncwarp();
    if (fresh && warp == 7) fetch_block(0);

    for (int lw = 0; lw < 15; ++lw) {
        QSYNC();
        if (fresh && lw <= 7) {
            if (sm.prog_above) {
                double p0 = 0.0, p1 = 0.0, p2 = 0.0, p3 = 0.0;
                const double *B = stgE + (lw & 1) * STG_E + t * STG_E_LD + g;
#pragma unroll
                for (int i = 0; i < 16; i += 2) {
                    dmma_m8n8k4(p0, p1, lfa[i], B[(4 * i) * STG_E_LD]);
                    dmma_m8n8k4(p2, p3, lfa[i + 1], B[(4 * i + 4) * STG_E_LD]);
                }
                p0 += p2; p1 += p3;
                double2 *yq = reinterpret_cast<double2 *>(Ys + (warp * 8 + g) * QLD + lw * 8 + t * 2);
                double2 *cq = reinterpret_cast<double2 *>(Cs + (warp * 8 + g) * QLD + lw * 8 + t * 2);
                double2 yv = *yq, cv = *cq;
                yv.x += p0; yv.y += p1; cv.x += p0; cv.y += p1;
                *yq = yv; *cq = cv;
            }
            __syncwarp();
            if (sm.prog_left) {
                double r0 = 0.0, r1 = 0.0, r2 = 0.0, r3 = 0.0;
                const double *A = stgC + (lw & 1) * STG_C + g * QLD + t;
#pragma unroll
                for (int i = 0; i < 16; i += 2) {
                    dmma_m8n8k4(r0, r1, A[4 * i], ufl[i]);
                    dmma_m8n8k4(r2, r3, A[4 * i + 4], ufl[i + 1]);
                }
                r0 += r2; r1 += r3;
                double2 *yq = reinterpret_cast<double2 *>(Ys + (lw * 8 + g) * QLD + warp * 8 + t * 2);
                double2 yv = *yq;
                yv.x += r0; yv.y += r1;
                *yq = yv;
            }
            QSYNC();
        }
        if (warp == 7 && fresh && lw < 7) fetch_block(lw + 1);
        if (qtid == 6 * 32 && lw > 0) {
            __threadfence();
            fence_proxy_async();              // the far groups read E and C through the copy engine
            st_release_u32(sm.prog_self, (unsigned)lw);
        }
        const int a_lo = max(0, lw - 7), a_hi = min(7, lw);
        const int a = a_lo + warp, b = lw - a;
        if (a <= a_hi) {
            leaf_pull(Ys, Cs, Ls, Us, a, b, g, t);
            __syncwarp();
            const int i0 = lane & 3, j = lane >> 2;
            double *yp = Ys + (a * 8 + i0) * QLD + b * 8 + j;
            double *cp = Cs + (a * 8 + i0) * QLD + b * 8 + j;
            double y0 = yp[0], y1 = yp[4 * QLD], c0 = cp[0], c1 = cp[4 * QLD];
            const double *tl0 = tabL + (a * 8 + i0) * TAB_LD + 7 - j;
            const double *tl1 = tl0 + 4 * TAB_LD;
            const double *tu0 = tabU + (b * 8 + j) * TAB_LD + 7 - i0;
            const double *tu1 = tu0 - 4;
            double *exw = xch + warp * 32;
            int z0 = 0, z1 = 0;
            const int t0 = i0 + j, t1 = t0 + 4;
#pragma unroll
            for (int s = 0; s < 15; ++s) {
                double *ex = exw + (s & 1) * 16;
                const bool r0 = (t0 == s), r1 = (t1 == s);
                if (r0 || r1) {
                    const double yv = r0 ? y0 : y1;
                    const double zv = rint(yv);
                    const double e = zv - yv;                           // E = Z - Y
                    const double cf = (r0 ? c0 : c1) + e;               // fold, L_ii = 1
                    ex[j] = e;
                    ex[8 + i0 + (r0 ? 0 : 4)] = cf;
                    if (r0) { y0 = e; c0 = cf; z0 = (int)zv; }
                    else { y1 = e; c1 = cf; z1 = (int)zv; }
                    if (!(fabs(yv) < 2147483648.0)) {
                        const unsigned long long gr = row0 + a * 8 + i0 + (r0 ? 0 : 4), gc = col0 + b * 8 + j;
                        const unsigned long long key = ((gr + gc) << 42) | ((isfinite(yv) ? 1ull : 0ull) << 41) |
                                                       (gr << 20) | gc;
                        if (gr < (unsigned long long)p.m && gc < (unsigned long long)p.n && key < badkey) badkey = key;
                    }
                }
                __syncwarp();
                const double ed = ex[j], cr0 = ex[8 + i0], cr1 = ex[12 + i0];
                const double l0 = tl0[s], l1 = tl1[s], u0 = tu0[s], u1 = tu1[s];
                y0 = fma(l0, ed, y0); c0 = fma(l0, ed, c0); y0 = fma(cr0, u0, y0);
                y1 = fma(l1, ed, y1); c1 = fma(l1, ed, c1); y1 = fma(cr1, u1, y1);
            }
            yp[0] = y0; yp[4 * QLD] = y1; cp[0] = c0; cp[4 * QLD] = c1;
            {
                const int gr = row0 + a * 8 + i0, gc = col0 + b * 8 + j;
                const long at = (long)gr * p.np + gc;
                p.Ebuf[at] = y0; p.Ebuf[at + 4 * p.np] = y1;
                p.Cbuf[at] = c0; p.Cbuf[at + 4 * p.np] = c1;
                if (gc < p.n) {
                    if (gr < p.m) {
                        p.Z[(long)gr * p.ldz + gc] = z0;
                        if (p.Euser) p.Euser[(long)gr * p.lde + gc] = y0;
                        max_abs_e = fmax(max_abs_e, fabs(y0));
                    }
                    if (gr + 4 < p.m) {
                        p.Z[(long)(gr + 4) * p.ldz + gc] = z1;
                        if (p.Euser) p.Euser[(long)(gr + 4) * p.lde + gc] = y1;
                        max_abs_e = fmax(max_abs_e, fabs(y1));
                    }
                }
            }
        }
    }
    QSYNC();
    if (qtid == 0) {
        __threadfence();
        fence_proxy_async();
        st_release_u32(sm.prog_self, 15u);
    }
    if (badkey != ~0ull) atomicMin(s_badkey, badkey);
    QSYNC();
    if (qtid == 0 && *s_badkey != ~0ull) {
        const unsigned long long k = *s_badkey;
        report(p.info, ((k >> 41) & 1ull) ? GPTQ2D_ERR_INT_OVERFLOW : GPTQ2D_ERR_NONFINITE,
               (int)((k >> 20) & 0x1fffffull), (int)(k & 0xfffffull), 0);
    }
}

// One quadrant task (see round_tiled.cu, sweep_quadrant).  qs: the group's shared memory.
__device__ __forceinline__ void sweep_quadrant(int I, int J, int q, double *qs, double *xch, unsigned long long *s_badkey,
                                               const FusedParams &p, double &max_abs_e, int qtid, volatile int *qsweeping) {
    double *Ys = qs, *Cs = qs + QMAT, *LU = qs + 2 * QMAT, *AUX = qs + 3 * QMAT;
    double *tabL = AUX, *tabU = tabL + Q * TAB_LD, *stg = tabU + Q * TAB_LD;
    const int warp = qtid >> 5, lane = qtid & 31, g = lane >> 2, t = lane & 3;
    const int qi = q >> 1, qj = q & 1;
    const int row0 = I * T + qi * Q, col0 = J * T + qj * Q;
    double *eQ = p.Ebuf + (long)row0 * p.np + col0;
    double *cQ = p.Cbuf + (long)row0 * p.np + col0;

    // ---- 1. pulls from complete quadrants of the two nearest tiles (two staging pairs: one multiplied, one filled)
    // The accumulators start from what the far parts parked for this quadrant (the far part of Cd in the
    // tile's Cbuf region, of Rt in its Ebuf region); the pulls add the two nearest tiles' share on top.
    QAcc accC, accR;
    quad_load_from(accC, cQ, p.np, warp, lane);
    quad_load_from(accR, eQ, p.np, warp, lane);
    {
        const int r = 2 * I + qi, c = 2 * J + qj;
        const int fa = max(0, 2 * I - 4), fl = max(0, 2 * J - 4);
        const int nsa = max(0, r - 1 - fa), nsl = max(0, c - 1 - fl), ns = nsa + nsl;
        auto prog_of = [&](int rr, int cc) {
            return p.qprog + ((long)(rr >> 1) * p.ntn + (cc >> 1)) * 4 + (rr & 1) * 2 + (cc & 1);
        };
        const int olda = max(0, nsa - 1), oldl = max(0, nsl - 1);
        auto step_dir = [&](int i) {
            return i < olda ? 0 : (i < olda + oldl ? 1 : ((i == olda + oldl && nsa > 0) ? 0 : 1));
        };
        auto step_blk = [&](int i) {
            return i < olda ? fa + i : (i < olda + oldl ? fl + (i - olda) : (step_dir(i) == 0 ? r - 2 : c - 2));
        };
        auto bufA = [&](int j) { return j == 0 ? LU : Ys; };
        auto bufB = [&](int j) { return j == 0 ? Cs : AUX; };
        auto issue = [&](int i) {
            double *Ab = bufA(i & 1), *Bb = bufB(i & 1);
            const int dir = step_dir(i), blk = step_blk(i), k0 = blk * Q;
            if (i >= olda + oldl) await_progress(p, dir == 0 ? prog_of(blk, c) : prog_of(r, blk), nullptr, 15u, lane);
            if (dir == 0) {
                if (p.l_al16) load_block_async16(Ab, p.L, p.ldl, p.m, p.m, row0, k0, qtid);
                else load_block_async8(Ab, p.L, p.ldl, p.m, p.m, row0, k0, qtid);
                load_quadrant_async(Bb, p.Ebuf + (long)k0 * p.np + col0, p.np, qtid);
            } else {
                load_quadrant_async(Ab, p.Cbuf + (long)row0 * p.np + k0, p.np, qtid);
                if (p.u_al16) load_block_async16(Bb, p.U, p.ldu, p.n, p.n, k0, col0, qtid);
                else load_block_async8(Bb, p.U, p.ldu, p.n, p.n, k0, col0, qtid);
            }
            cp_async_commit();
        };
        if (warp < olda) await_progress(p, prog_of(fa + warp, c), nullptr, 15u, lane);
        else if (warp < olda + oldl) await_progress(p, prog_of(r, fl + (warp - olda)), nullptr, 15u, lane);
        QSYNC();
        if (ns > 0) issue(0);
        for (int i = 0; i < ns; ++i) {
            cp_async_wait<0>();
            QSYNC();                 // step i has landed; every warp is past product i - 1, so its pair is free
            if (i + 1 < ns) issue(i + 1);
            if (step_dir(i) == 0) quad_mma(accC, bufA(i & 1), bufB(i & 1), warp, lane);
            else quad_mma(accR, bufA(i & 1), bufB(i & 1), warp, lane);
        }
        QSYNC();
    }

    // ---- 2. operands of the sweep.  Cd and Rt leave the registers (the staging matrices are free now) ...
    quad_store_to(Cs, QLD, accC, warp, lane);
    quad_store_to(Ys, QLD, accR, warp, lane);
    Stream sm;
    sm.I = I; sm.J = J; sm.q = q;
    const long tq = ((long)I * p.ntn + J) * 4;
    sm.prog_self = p.qprog + tq + q;
    sm.prog_above = nullptr; sm.prog_left = nullptr; sm.e_above = nullptr; sm.c_left = nullptr;
    load_lu_diag_async(LU, p, row0, col0, qtid);
    // X of the quadrant into the auxiliary region (dense 64 x 64, zero outside the matrix)
    double *Xs = AUX;
#pragma unroll
    for (int it = 0; it < 16; ++it) {
        const int c = qtid + it * GROUP;
        const int rr = c >> 6, cc = c & 63;
        const int gr = row0 + rr, gc = col0 + cc;
        const bool take = gr < p.m && gc < p.n;
        cp_async8(Xs + rr * 64 + cc, take ? p.X + (long)gr * p.ldx + gc : p.X, take ? 8 : 0);
    }
    cp_async_commit();
    // ... and make room for the fragments of the two off-diagonal factor blocks, straight from global memory (L2)
    double lfa[16], ufl[16];
    if (row0 > 0) {
        sm.prog_above = qi ? p.qprog + tq + (q - 2) : p.qprog + ((long)(I - 1) * p.ntn + J) * 4 + (q + 2);
        sm.e_above = p.Ebuf + (long)(row0 - Q) * p.np + col0;
        const int gr = row0 + warp * 8 + g;
        const double *src = p.L + (long)gr * p.ldl + (row0 - Q) + t;
#pragma unroll
        for (int i = 0; i < 16; ++i) lfa[i] = gr < p.m ? __ldg(src + 4 * i) : 0.0;
    } else {
#pragma unroll
        for (int i = 0; i < 16; ++i) lfa[i] = 0.0;
    }
    if (col0 > 0) {
        sm.prog_left = qj ? p.qprog + tq + (q - 1) : p.qprog + ((long)I * p.ntn + (J - 1)) * 4 + (q + 1);
        sm.c_left = p.Cbuf + (long)row0 * p.np + (col0 - Q);
        const int gc = col0 + warp * 8 + g;
        const double *src = p.U + (long)(col0 - Q + t) * p.ldu + gc;
#pragma unroll
        for (int i = 0; i < 16; ++i) ufl[i] = gc < p.n ? __ldg(src + (long)(4 * i) * p.ldu) : 0.0;
    } else {
#pragma unroll
        for (int i = 0; i < 16; ++i) ufl[i] = 0.0;
    }
    cp_async_wait<0>();
    QSYNC();
#pragma unroll
    for (int it = 0; it < 16; ++it) {                     // Y = X + Rt + Cd
        const int c = qtid + it * GROUP;
        const int rr = c >> 6, cc = c & 63;
        Ys[rr * QLD + cc] += Xs[rr * 64 + cc] + Cs[rr * QLD + cc];
    }
    QSYNC();                                              // Xs is dead: the tables are built over it
    if (FUSED_THROTTLE && qtid == 0) *qsweeping = 1;
    quadrant_sweep(Ys, Cs, LU, lfa, ufl, stg, tabL, tabU, xch, s_badkey, row0, col0, sm, p, max_abs_e, qtid);
    if (FUSED_THROTTLE && qtid == 0) *qsweeping = 0;
    QSYNC();
}

// ---------------------------------------------------------------------------------------------
// far parts: task index -> (type, I, J, half).  Wave by wave (I + J ascending); inside a wave the longest
// contractions first, the two halves of a tile back to back (they share the row operand in L2).
__device__ __forceinline__ void decode_task(int task, int ntm, int ntn, int &type, int &I, int &J, int &h) {
    int tt = task;
    for (int w = 0; w < ntm + ntn - 1; ++w) {
        int lo = max(0, w - ntn + 1), hi = min(ntm - 1, w);
        int cnt = 4 * (hi - lo + 1);
        if (tt < cnt) {
            const int k = tt >> 2;
            type = (tt >> 1) & 1;
            h = tt & 1;
            I = type == 0 ? hi - k : lo + k;
            J = w - I;
            return;
        }
        tt -= cnt;
    }
    type = 0; I = J = h = 0;
}

struct FAcc {
    double v[F_FRAGS_M][4][2];       // fragment (a, b) of the warp's (8 F_FRAGS_M) x 32 piece
    __device__ __forceinline__ void zero() {
#pragma unroll
        for (int a = 0; a < F_FRAGS_M; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) v[a][b][0] = v[a][b][1] = 0.0;
    }
};

struct FarRing {
    unsigned long long *full, *empty;
    double *stages;
    unsigned slabs;          // slabs issued = consumed so far (uniform over the group between calls)
};

// acc += rowop[128 rows at y = row_y, k from k0] * colop[k from k0, 64 columns at x = col_x], nk slabs of 16.
// Called by the eight far warps with uniform arguments.  Returns false if a wait ran out.
__device__ __forceinline__ bool far_mainloop(FAcc &acc, FarRing &ring, const CUtensorMap *mapA, const CUtensorMap *mapB,
                                             int row_y, int col_x, int k0, int nk, int warp, int lane, unsigned *abort,
                                             const volatile int *stand_back) {
    constexpr int PREF = F_NSTAGE - 1;
    const int wm = warp >> 1, wn = warp & 1, g = lane >> 2, t = lane & 3;
    bool ok = true;
    unsigned issued_upto = 0;
    // per-lane fragment offsets inside a stage: [fragment parity][k4-step]; fragment f adds (f >> 1) * 256 doubles
    int offA[2][4], offB[2][4];
#pragma unroll
    for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            offA[h][q] = slab_offset<true>(wm * (8 * F_FRAGS_M) + frag_index<true>(h, g), 4 * q + t);
            offB[h][q] = slab_offset<false>(wn * 32 + frag_index<false>(h, g), 4 * q + t) + F_A_DOUBLES;
        }
    auto issue = [&](unsigned s) {        // one lane: slab s of this call
        const unsigned pidx = ring.slabs + s;
        const unsigned st = pidx % F_NSTAGE, use = pidx / F_NSTAGE;
        if (use > 0 && !mbar_wait(ring.empty + st, (use - 1) & 1u, abort)) { ok = false; return; }
        issued_upto = s + 1;
        double *dst = ring.stages + (size_t)st * F_STAGE_DOUBLES;
        const int k = k0 + (int)s * TMA_BK;
        fence_proxy_async();
        mbar_arrive_expect_tx(ring.full + st, F_STAGE_BYTES);
        tma_load_3d(dst, mapA, k, row_y, 0, ring.full + st);
#pragma unroll
        for (int i = 0; i < FN / 16; ++i) tma_load_3d(dst + F_A_DOUBLES + i * 256, mapB, col_x + 16 * i, k, 0, ring.full + st);
    };
    if (warp == 0 && lane == 0)
        for (int s = 0; s < PREF && s < nk; ++s) issue((unsigned)s);
    int kt_stop = nk;
    for (int kt = 0; kt < nk; ++kt) {
        const unsigned c = ring.slabs + (unsigned)kt;
        const unsigned st = c % F_NSTAGE, use = c / F_NSTAGE;
        if (FUSED_THROTTLE) {
            // The scalar fp64 steps of a leaf sweep queue behind DMMAs on the sub-partition's one fp64 pipe, so while
            // this SM's quadrant group is inside its leaf-waves the far warps pause between slabs (bounded: the flag
            // is cleared at the end of every quadrant task).
            unsigned pause = 0;
            while (*stand_back != 0 && ++pause < 200000u) __nanosleep(200);
        }
        if (!__all_sync(0xffffffffu, mbar_wait(ring.full + st, use & 1u, abort))) { ok = false; kt_stop = kt; break; }
        const double *S = ring.stages + (size_t)st * F_STAGE_DOUBLES;
        const bool my_turn = (kt + PREF < nk) && ((kt & (F_WARPS - 1)) == warp);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            double af[F_FRAGS_M], bf[4];
#pragma unroll
            for (int a = 0; a < F_FRAGS_M; ++a) af[a] = S[offA[a & 1][q] + (a >> 1) * 256];
#pragma unroll
            for (int b = 0; b < 4; ++b) bf[b] = S[offB[b & 1][q] + (b >> 1) * 256];
#pragma unroll
            for (int a = 0; a < F_FRAGS_M; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) dmma_m8n8k4(acc.v[a][b][0], acc.v[a][b][1], af[a], bf[b]);
            if (q == 1 && my_turn) {
                if (lane == 0) issue((unsigned)(kt + PREF));
                __syncwarp();
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(ring.empty + st);
    }
    ok = __all_sync(0xffffffffu, ok);
    if (!ok) {
        if (abort && lane == 0) atomicExch(abort, 1u);
        for (unsigned s = (unsigned)kt_stop; s < issued_upto; ++s) {
            const unsigned c = ring.slabs + s;
            (void)mbar_wait(ring.full + c % F_NSTAGE, (c / F_NSTAGE) & 1u, nullptr, 1000000ull);
        }
    }
    ring.slabs += (unsigned)nk;
    return ok;
}

// accumulator <-> its 128 x 64 region of a padded workspace buffer (row stride np)
__device__ __forceinline__ void store_facc(const FAcc &acc, double *dst, long np, int warp, int lane) {
    const int wm = warp >> 1, wn = warp & 1, g = lane >> 2, t = lane & 3;
#pragma unroll
    for (int a = 0; a < F_FRAGS_M; ++a) {
        const int r = wm * (8 * F_FRAGS_M) + frag_index<true>(a, g);
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            const int c = wn * 32 + frag_index<false>(b, 2 * t);
            double2 v;
            v.x = acc.v[a][b][0];
            v.y = acc.v[a][b][1];
            *reinterpret_cast<double2 *>(dst + (long)r * np + c) = v;
        }
    }
}

__global__ void __launch_bounds__(THREADS, 1)
round_fused_kernel(FusedParams p, const __grid_constant__ CUtensorMap mapL, const __grid_constant__ CUtensorMap mapE,
                   const __grid_constant__ CUtensorMap mapC, const __grid_constant__ CUtensorMap mapU) {
    extern __shared__ __align__(16) double smem_raw[];
    __shared__ __align__(8) unsigned long long bars[2 * F_NSTAGE];
    __shared__ double xch[8 * 2 * 16];
    __shared__ unsigned long long s_badkey;
    __shared__ int s_ftask, s_fupto, s_fok;
    __shared__ volatile int s_qsweeping;       // the quadrant group is inside its leaf-waves: the far group stands back
    __shared__ unsigned s_qpop;
    __shared__ int s_qstate;
    __shared__ double s_red[GROUP / 32];
    // aligned to 1024 bytes by an offset into the shared array (pointer arithmetic keeps the shared address space)
    if (threadIdx.x == 0) s_qsweeping = 0;
    __syncthreads();
    double *ring_mem = smem_raw + (((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u) >> 3);
    double *qs = ring_mem + F_NSTAGE * F_STAGE_DOUBLES;
    const int tid = threadIdx.x;

    if (tid < F_THREADS) {
        // =============================== FAR group ===============================
        const int warp = tid >> 5, lane = tid & 31;
        FarRing ring;
        ring.full = bars; ring.empty = bars + F_NSTAGE; ring.stages = ring_mem; ring.slabs = 0;
        if (tid == 0) {
            for (int s = 0; s < F_NSTAGE; ++s) { mbar_init(ring.full + s, 1); mbar_init(ring.empty + s, F_WARPS); }
            mbar_init_fence();
        }
        FSYNC();
        STAT_DECL(st_main); STAT_DECL(st_wait); STAT_DECL(st_park); STAT_DECL(st_nparts);
        STAT_T0(st_begin);
        for (;;) {
            if (tid == 0) {
                int task = -1;
                if (ld_relaxed_u32(p.abort) == 0u && ld_relaxed_u32(p.counter) < (unsigned)p.ntasks) {
                    task = (int)atomicAdd(p.counter, 1u);
                    if (task >= p.ntasks) task = -1;
                }
                s_ftask = task;
            }
            FSYNC();
            const int task = s_ftask;
            if (task < 0) break;
            int type, I, J, h;
            decode_task(task, p.ntm, p.ntn, type, I, J, h);
            const int nfar = max(0, (type == 0 ? I : J) - 2);
            const unsigned *flags = type == 0 ? p.flagS + J : p.flagS + (long)I * p.ntn;
            const long fstride = type == 0 ? p.ntn : 1;
            FAcc acc;
            acc.zero();
            bool ok = true;
            int pos = 0;
            while (pos < nfar) {
                // source tiles pos .. upto-1 are swept (thread 0 waits, bounded, for the first of them)
                FSYNC();
                STAT_T0(tw);
                if (tid == 0) {
                    unsigned long long it = 0;
                    int upto = pos;
                    for (;;) {
                        while (upto < nfar && ld_acquire_u32(flags + (long)upto * fstride) != 0u) ++upto;
                        if (upto > pos) break;
                        if (++it > p.spin_limit || ld_relaxed_u32(p.abort) != 0u) {
                            report(p.info, GPTQ2D_ERR_DEVICE_TIMEOUT, -5, task, (int)blockIdx.x);
                            atomicExch(p.abort, 1u);
                            upto = -1;
                            break;
                        }
                        __nanosleep(100);
                    }
                    s_fupto = upto;
                    s_fok = 1;
                }
                FSYNC();
                const int upto = s_fupto;
                STAT_ADD(st_wait, tw);
                if (upto < 0) { ok = false; break; }
                STAT_T0(tm);
                const int nk = (upto - pos) * (T / TMA_BK);
                if (type == 0) ok = far_mainloop(acc, ring, &mapL, &mapE, I * T, J * T + h * FN, pos * T, nk, warp, lane, p.abort, &s_qsweeping);
                else ok = far_mainloop(acc, ring, &mapC, &mapU, I * T, J * T + h * FN, pos * T, nk, warp, lane, p.abort, &s_qsweeping);
                // a wait that ran out in one warp ends the far part for the whole group
                if (!ok && lane == 0) {
                    report(p.info, GPTQ2D_ERR_DEVICE_TIMEOUT, -7, task, (int)blockIdx.x);
                    s_fok = 0;
                }
                FSYNC();
                STAT_ADD(st_main, tm);
                ok = s_fok != 0;
                if (!ok) break;
                pos = upto;
            }
            if (!ok) break;
            // park the sum (zeros included: the quadrant tasks start from it) and announce it to the two
            // quadrants of this half
            STAT_T0(tp);
            double *region = (type == 0 ? p.Cbuf : p.Ebuf) + (long)I * T * p.np + (long)J * T + h * FN;
            store_facc(acc, region, p.np, warp, lane);
            FSYNC();
            if (tid < 2) {
                __threadfence();
                quadrant_arrive(p, I, J, h + 2 * tid);
            }
            STAT_ADD(st_park, tp);
#ifdef FUSED_STATS
            st_nparts += 1;
#endif
        }
#ifdef FUSED_STATS
        if (tid == 0 && (blockIdx.x % 37) == 0)
            printf("cta %3d F: total %lld main %lld flagwait %lld park %lld parts %lld\n", (int)blockIdx.x,
                   clock64() - st_begin, st_main, st_wait, st_park, st_nparts);
#endif
        return;
    }

    // =============================== QUADRANT group ===============================
    const int qtid = tid - F_THREADS, qwarp = qtid >> 5, lane = qtid & 31;
    double max_abs_e = 0.0;
    STAT_DECL(sq_task); STAT_DECL(sq_idle); STAT_DECL(sq_n);
    STAT_T0(sq_begin);
    for (;;) {
        STAT_T0(ti);
        if (qtid == 0) {
            int state = 0;
            unsigned e = 0u;
            unsigned long long spins = 0;
            for (;;) {
                if (ld_relaxed_u32(p.abort) != 0u) { state = 4; break; }
                e = ready_pop(p);
                if (e != 0u) { state = 1; break; }
                if (ld_relaxed_u32(p.tiles_done) >= (unsigned)p.ntiles_total) { state = 3; break; }
                if (++spins > p.spin_limit) {
                    report(p.info, GPTQ2D_ERR_DEVICE_TIMEOUT, -4, (int)blockIdx.x, 0);
                    atomicExch(p.abort, 1u);
                    state = 4;
                    break;
                }
                __nanosleep(300);
            }
            s_qstate = state; s_qpop = e;
        }
        QSYNC();
        const int state = s_qstate;
        const unsigned e = s_qpop;
        STAT_ADD(sq_idle, ti);
        if (state != 1) break;
        const int q = (int)((e >> 29) & 3u), I = (int)((e >> 15) & 0x3fffu), J = (int)(e & 0x7fffu);
        STAT_T0(tt);
        sweep_quadrant(I, J, q, qs, xch, &s_badkey, p, max_abs_e, qtid, &s_qsweeping);
        STAT_ADD(sq_task, tt);
#ifdef FUSED_STATS
        sq_n += 1;
#endif
        if (qtid == 6) {
            __threadfence();
            fence_proxy_async();
            unsigned done = atomicAdd(p.quad_done + (long)I * p.ntn + J, 1u);
            const unsigned nquad = (p.m - I * T > Q ? 2u : 1u) * (p.n - J * T > Q ? 2u : 1u);
            if (done + 1u == nquad) {
                __threadfence();
                st_release_u32(p.flagS + (long)I * p.ntn + J, 1u);
                atomicAdd(p.rowdone + I, 1u);
                atomicAdd(p.tiles_done, 1u);
            }
        }
        // (the QSYNC at the top of the next round orders s_qstate / s_qpop: thread 0 rewrites them only after
        // every thread has read them, because sweep_quadrant contains group barriers)
    }
#ifdef FUSED_STATS
    if (qtid == 0 && (blockIdx.x % 37) == 0)
        printf("cta %3d Q: total %lld tasks %lld idle %lld n %lld (per task %lld)\n", (int)blockIdx.x, clock64() - sq_begin,
               sq_task, sq_idle, sq_n, sq_n ? sq_task / sq_n : 0);
#endif
    for (int o = 16; o > 0; o >>= 1) max_abs_e = fmax(max_abs_e, __shfl_xor_sync(0xffffffffu, max_abs_e, o));
    if (lane == 0) s_red[qwarp] = max_abs_e;
    QSYNC();
    if (qtid == 0) {
        double v = 0.0;
        for (int w = 0; w < GROUP / 32; ++w) v = fmax(v, s_red[w]);
        if (v > 0.0) atomic_max_nonneg_double(p.max_abs_e, v);
    }
}

}  // namespace fused

// Workspace: the layout of round_tiled.cu (same size query), so the two kernels are interchangeable.
struct TiledLayoutView {
    int ntm, ntn;
    size_t q_off, flags_off, quad_off, qdep_off, qprog_off, rowdone_off, e_off, c_off, total;
};
TiledLayoutView round_tiled_layout_view(int m, int n);     // round_tiled.cu

// 0 (default): never -- on B200 the side-by-side kernel measures slower than the eight-warp kernel at every
// size (the scalar fp64 steps of the leaf sweeps queue behind the far group's DMMAs on the one fp64 pipe);
// 1: problems of at least 8 x 8 tiles; 2: whenever the operands allow it (tests, comparison runs).
static int g_fused_mode = 0;
void round_fused_set_mode(int mode) { g_fused_mode = mode; }

// Returns -1 if this problem does not go through the fused kernel (switched off, too small to gain, operands
// not TMA-aligned, no tensor-map encoder), else a gptq2d status.
int launch_round_fused(const TiledParams &in, void *ws, size_t ws_bytes, cudaStream_t stream, bool force) {
    using namespace fused;
    if (g_fused_mode == 0 && !force) return -1;
    if (in.panels_ready) return -1;
    const TiledLayoutView l = round_tiled_layout_view(in.m, in.n);
    if (!force && g_fused_mode != 2 && (l.ntm < 8 || l.ntn < 8)) return -1;   // far parts only exist from the third tile on
    if (!tma_operand_ok(in.L, in.ldl, 2) || !tma_operand_ok(in.U, in.ldu, 2)) return -1;
    if (ws_bytes < l.total) return GPTQ2D_ERR_WORKSPACE;
    char *w = static_cast<char *>(ws);
    FusedParams p{};
    p.m = in.m; p.n = in.n; p.ntm = l.ntm; p.ntn = l.ntn;
    p.ntasks = 4 * l.ntm * l.ntn;
    p.ntiles_total = l.ntm * l.ntn;
    p.np = (long)l.ntn * T;
    p.X = in.X; p.ldx = in.ldx; p.L = in.L; p.ldl = in.ldl; p.U = in.U; p.ldu = in.ldu;
    p.Z = in.Z; p.ldz = in.ldz; p.Euser = in.E; p.lde = in.lde;
    p.counter = reinterpret_cast<unsigned *>(w);
    p.abort = reinterpret_cast<unsigned *>(w) + 1;
    p.q_head = reinterpret_cast<unsigned *>(w) + 2;
    p.q_tail = reinterpret_cast<unsigned *>(w) + 3;
    p.tiles_done = reinterpret_cast<unsigned *>(w) + 4;
    p.q_slots = reinterpret_cast<unsigned *>(w + l.q_off);
    p.qmask = 4096 - 1;
    p.max_abs_e = workspace_max_abs_e(ws);
    p.flagS = reinterpret_cast<unsigned *>(w + l.flags_off);
    p.quad_done = reinterpret_cast<unsigned *>(w + l.quad_off);
    p.qdep = reinterpret_cast<unsigned *>(w + l.qdep_off);
    p.qprog = reinterpret_cast<unsigned *>(w + l.qprog_off);
    p.rowdone = reinterpret_cast<unsigned *>(w + l.rowdone_off);
    p.Ebuf = reinterpret_cast<double *>(w + l.e_off);
    p.Cbuf = reinterpret_cast<double *>(w + l.c_off);
    p.info = in.info;
    p.l_al16 = 1; p.u_al16 = 1;
    p.spin_limit = SPIN_LIMIT;

    CUtensorMap mapL, mapE, mapC, mapU;
    const long mp = (long)l.ntm * T;
    // row operands (K-contiguous): boxes of 16 k x 128 rows; column operands: boxes of 16 columns x 16 k
    if (!encode_f64_matrix_map(&mapL, in.L, in.m, in.m, in.ldl, 1, 0, 16, 128)) return -1;
    if (!encode_f64_matrix_map(&mapC, p.Cbuf, mp, p.np, p.np, 1, 0, 16, 128)) return -1;
    if (!encode_f64_matrix_map(&mapE, p.Ebuf, mp, p.np, p.np, 1, 0, 16, 16)) return -1;
    if (!encode_f64_matrix_map(&mapU, in.U, in.n, in.n, in.ldu, 1, 0, 16, 16)) return -1;

    if (cudaMemsetAsync(w, 0, l.e_off, stream) != cudaSuccess) return GPTQ2D_ERR_CUDA;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return GPTQ2D_ERR_CUDA;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return GPTQ2D_ERR_CUDA;
    if (cudaFuncSetAttribute(round_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)FUSED_SMEM) != cudaSuccess)
        return GPTQ2D_ERR_CUDA;
    int grid = sms < p.ntiles_total ? sms : p.ntiles_total;
    void *args[] = {&p, &mapL, &mapE, &mapC, &mapU};
    if (cudaLaunchCooperativeKernel((const void *)round_fused_kernel, dim3(grid), dim3(THREADS), args, FUSED_SMEM, stream) !=
        cudaSuccess)
        return GPTQ2D_ERR_CUDA;
    return GPTQ2D_OK;
}

}  // namespace gptq2d
