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
// Scheduling.  Two kinds of work, one persistent cooperatively launched grid (one CTA per SM):
//  * FAR parts.  Each tile's Cd and Rt contractions over every source tile EXCEPT the two nearest
//    ones.  Listed wave by wave (I + J ascending) and claimed in that order from one atomic
//    counter.  A far part waits (bounded) only on tiles three or more waves back, parks its
//    partial sum in the tile's own workspace region and then announces it to the tile's four
//    quadrant tasks; it is done long before they need it.  This is >90 % of the flops and runs on
//    the fp64 tensor path.
//  * QUADRANT tasks (64 x 64), the critical path.  In the grid of quadrants, (r, c) needs all
//    quadrants above it in its column and to its left in its row.  What the quadrants of the two
//    nearest tiles contribute (rows 2 I - 4 .. r - 2 of the grid, columns likewise) it pulls itself
//    when it starts: up to eight 64^3 DMMA products.  The quadrant right above and the one right to
//    the left are NOT waited for: every quadrant publishes its 8 x 8 leaves leaf-wave by leaf-wave
//    (results to the workspace, a progress word per quadrant), and its two neighbours take them in
//    as they come, running nine leaf-waves behind (block b of a neighbour is final after its
//    leaf-wave 7 + b).  A task counts arrivals from the two far parts of its tile and from
//    (r-1, c) and (r, c-1) beginning to sweep; the last arrival puts it on a global ready ring.  A
//    running quadrant task waits -- bounded -- only on quadrants above it / to its left, which are
//    running by then (or done).
// Every CTA serves the ready ring first: at the top of its loop, while a far part waits, and
// every 64 chunks of a far part (its accumulator stays in registers meanwhile).
// A far part only ever waits on tiles of earlier waves, whose far parts were claimed earlier and
// whose quadrant tasks wait on running tasks only, so the earliest unfinished work can always
// progress.
//
// In-tile sweep.  Inside a quadrant the anti-diagonal sweep runs on 8 x 8 leaves: each leaf of a
// leaf-wave is swept by one warp (two entries per lane, errors exchanged through a 16-double
// shared-memory buffer, branch-free pushes against zero-padded coefficient tables), and the
// leaves' feedback to the remaining 8 x 8 blocks of the quadrant is m8n8k4 DMMA.
#include <cstdio>
#include "common.cuh"
#include "dmma_gemm.cuh"
#include "round_internal.cuh"
#include <vector>

namespace gptq2d {

// optional in-kernel timing of the quadrant task (scratch builds only: -DTILED_STATS): cycles seen by lane 0 of
// warp 0, which has a leaf in every leaf-wave, summed per phase over a CTA's tasks
#ifdef TILED_STATS
#define TS_MARK(slot)                                            \
    do {                                                         \
        if (threadIdx.x == 0) {                                  \
            const long long now_ = clock64();                    \
            g_ts[slot] += now_ - g_tlast;                        \
            g_tlast = now_;                                      \
        }                                                        \
    } while (0)
#define TS_RESET()                                               \
    do {                                                         \
        if (threadIdx.x == 0) g_tlast = clock64();               \
    } while (0)
__shared__ long long g_ts[16];
__shared__ long long g_tlast;
__shared__ long long g_sched[8];     // 0 quadrant tasks, 1 far main loop, 2 far park/unpark + flag scan, 3 idle, 4 looking for work, 5 far parts
#else
#define TS_MARK(slot)
#define TS_RESET()
#endif

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
    unsigned *counter, *abort, *q_head, *q_tail, *tiles_done;
    unsigned *q_slots;           // [qmask + 1] ready quadrant tasks
    unsigned qmask;              // ring size - 1 (power of two)
    unsigned *flagS;             // [ntm*ntn] tile swept
    unsigned *quad_done;         // [ntm*ntn] swept quadrants of the tile (4 -> tile flag)
    unsigned *qdep;              // [ntm*ntn][4] arrivals each quadrant task has received
    unsigned *qprog;             // [ntm*ntn][4] leaf-waves each quadrant has published (15: complete)
    unsigned *rowdone;           // [ntm] tiles of each tile row that are swept (the host entry copies Z back row by row)
    double *max_abs_e;
    int *info;
    int l_al16, u_al16;
    // batched launches only (one descriptor per matrix in device memory; the kernel argument then
    // carries the shared scheduler words, the totals in ntasks / ntiles_total, and these tables)
    int batch_index;             // -1: single-matrix launch
    int ntiles_total;
    const TiledKernelParams *probs;
    const unsigned *far_tasks;   // far parts of all matrices in claim order: b << 17 | type << 16 | I << 8 | J
    // pipelined host entry only: number of 128-row panels of X, L and U that have reached the device
    const unsigned *panels_ready;
    // polls after which a device-side wait gives up (host-set; SPIN_LIMIT unless a test shortens it):
    // every wait of the kernel, and the wait for an announced copy step of the host entry on its own
    unsigned long long spin_limit, panel_spin_limit;
};
static_assert(sizeof(TiledKernelParams) % 8 == 0, "descriptors are copied as 8-byte words");

constexpr size_t SWEEP_SMEM = (size_t)(5 * QMAT + 2 * Q * TAB_LD + 2 * (64 * 12) + 2 * (8 * QLD)) * sizeof(double);
constexpr size_t BULK_SMEM = (size_t)BULK_NSTAGE * SlabLayout<true, false>::STAGE_DOUBLES * sizeof(double);
constexpr size_t TILED_SMEM = SWEEP_SMEM > BULK_SMEM ? SWEEP_SMEM : BULK_SMEM;

// ---------------------------------------------------------------------------------------------
// workspace / factors -> shared memory.  The *_async loaders only issue cp.async copies; the caller
// commits, waits and barriers once for all operands of a quadrant.
__device__ __forceinline__ void load_quadrant_async(double *dst, const double *src, long ld) {
    // dense 64 x 64 from a padded workspace buffer (always in range, 16-byte aligned); L2 only
#pragma unroll
    for (int it = 0; it < 8; ++it) {
        int c = threadIdx.x + it * TILED_THREADS;
        cp_async16(dst + CI((c >> 5) * QLD + (c & 31) * 2, QMAT - 1, 101), src + (long)(c >> 5) * ld + (c & 31) * 2, 16);
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
        cp_async8(dst + CI(r * QLD + cc, QMAT, 102), take ? M + CI((long)gr * ld + gc, (long)(k - 1) * ld + k, 103) : M, take ? 8 : 0);
    }
}

// Whole 64 x 64 block (no triangle mask) with 16-byte copies; needs M 16-byte aligned, ld and c0 even.
__device__ __forceinline__ void load_full_block_async16(double *dst, const double *M, long ld, int k, int r0, int c0) {
#pragma unroll
    for (int it = 0; it < 8; ++it) {
        int c = threadIdx.x + it * TILED_THREADS;
        int r = c >> 5, cc = (c & 31) * 2;
        int gr = r0 + r, gc = c0 + cc;
        int nv = (gr < k) ? min(2, max(0, k - gc)) : 0;
        cp_async16(dst + CI(r * QLD + cc, QMAT - 1, 104), nv ? M + CI((long)gr * ld + gc, (long)(k - 1) * ld + k - nv + 1, 105) : M, nv * 8);
    }
}

// 64 x 64 x 64 DMMA product on quadrant operands in shared memory: each warp owns a 16 x 32 piece
// (2 x 4 fragments); element rows wr*16 + a*8 + (lane>>2), cols wc*32 + b*8 + (lane&3)*2 + {0,1}.
struct QAcc {
    double v[2][4][2];
    __device__ __forceinline__ void zero() {
#pragma unroll
        for (int a = 0; a < 2; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) v[a][b][0] = v[a][b][1] = 0.0;
    }
};
// acc += As (64 x 64, [m][k]) * Bs (64 x 64, [k][n])
__device__ __forceinline__ void quad_mma(QAcc &acc, const double *As, const double *Bs) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    const int wr = warp >> 1, wc = warp & 1;
#pragma unroll 4
    for (int kk = 0; kk < Q; kk += 4) {
        double af[2], bf[4];
#pragma unroll
        for (int a = 0; a < 2; ++a) af[a] = As[CI((wr * 16 + a * 8 + g) * QLD + kk + t, QMAT, 106)];
#pragma unroll
        for (int b = 0; b < 4; ++b) bf[b] = Bs[CI((kk + t) * QLD + wc * 32 + b * 8 + g, QMAT, 107)];
#pragma unroll
        for (int a = 0; a < 2; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) dmma_m8n8k4(acc.v[a][b][0], acc.v[a][b][1], af[a], bf[b]);
    }
}
// D (64 x 64 with row stride ld, global or shared) += acc
__device__ __forceinline__ void quad_add_to(double *D, long ld, const QAcc &acc, bool global_cg) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
    const int wr = warp >> 1, wc = warp & 1;
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            double2 *ptr = reinterpret_cast<double2 *>(D + (long)(wr * 16 + a * 8 + g) * ld + wc * 32 + b * 8 + t * 2);
            double2 v = global_cg ? __ldcg(ptr) : *ptr;
            v.x += acc.v[a][b][0];
            v.y += acc.v[a][b][1];
            *ptr = v;
        }
}
// Leaf (a, b) of the quadrant collects, right before it is swept, all the feedback it is due from
// the leaves already swept (left-looking): the downward pushes of the leaves above it through L,
//     P = sum_{a' < a} L[a, a'] E[a', b]       (folded into C and pushed into Y)
// and the rightward pushes of the leaves to its left through U,
//     R = sum_{b' < b} C[a, b'] U[b', b]       (pushed into Y),
// as m8n8k4 products on the warp's fragments (two independent accumulator chains each), then
// Y += P + R, C += P in place.  E of a swept leaf lives where its Y was, its final C where its C
// was.  Warp-uniform; all leaves of one leaf-wave do the same amount of work (a + b = lw).
__device__ __forceinline__ void leaf_pull(double *Ys, double *Cs, const double *Ls, const double *Us, int a, int b,
                                          int g, int t) {
    double p0 = 0.0, p1 = 0.0, p2 = 0.0, p3 = 0.0, r0 = 0.0, r1 = 0.0, r2 = 0.0, r3 = 0.0;
    const double *La = Ls + (a * 8 + g) * QLD + t;           // A fragments: row a*8+g, k = t (+4)
    const double *Eb = Ys + t * QLD + b * 8 + g;             // B fragments: k = t (+4), col b*8+g
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

// ---------------------------------------------------------------------------------------------
// Streaming between neighbouring quadrants.  A quadrant does not wait for the quadrant above it
// (and the one to its left) to finish: column block b of the E above is final once that quadrant
// has swept its leaf-waves 0 .. 7+b, row block a of the C to the left once leaf-waves 0 .. 7+a are
// done, and leaf-wave lw of this quadrant needs exactly blocks 0 .. lw of both.  Every quadrant
// therefore publishes its leaves wave by wave (E, C to the workspace, a progress word per
// quadrant), and its two neighbours run nine leaf-waves behind it.
constexpr int STG_E_LD = 12;                 // staged 64 x 8 column block of E, [k][n], 12 = 8 + 4 pad
constexpr int STG_E = Q * STG_E_LD;          // doubles per staged E block
constexpr int STG_C = 8 * QLD;               // staged 8 x 64 row block of C, [m][k]

struct Stream {
    const unsigned *prog_above, *prog_left;  // progress words of the two neighbours (NULL: none)
    unsigned *prog_self;
    const double *e_above;                   // Ebuf at (first row of the quadrant above, first column of this one)
    const double *c_left;                    // Cbuf at (first row of this quadrant, first column of the one to the left)
    int I, J, q;
};

// Called by one warp: lane 0 polls both neighbours' progress words until each has reached `need`
// (bounded; on expiry the launch is aborted and the caller carries on with whatever is there).
__device__ __forceinline__ void await_progress(const TiledKernelParams &p, const unsigned *wa, const unsigned *wl,
                                               unsigned need) {
    if ((threadIdx.x & 31) == 0) {
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

__device__ __forceinline__ void quadrant_arrive(const TiledKernelParams &p, int I, int J, int q);

// Algorithm 3 on one 64 x 64 quadrant held in shared memory.
//   Ys: in  Y (corrected values from everything but the two streaming neighbours); out E
//   Cs: in  C likewise; out final C = L E rows of the quadrant
//   LU: the 64 x 64 diagonal blocks of both factors in one matrix: strictly lower part from L,
//       strictly upper part from U (the sweep never reads the other triangles)
//   Lfa: L[rows of this quadrant, rows of the quadrant above];  Ufl: U[columns of the quadrant to
//        the left, columns of this quadrant]
//   stg: staging for the streamed blocks, two of each kind
// row0/col0: global coordinates of the quadrant.
//
// Leaf-wave lw (leaves (a, lw - a), one per warp).  For lw <= 7, all warps first add what block lw
// of the neighbours feeds into this quadrant (pull phase).  Then every leaf pulls the feedback of
// the leaves swept before it (leaf_pull), runs the 15 anti-diagonal steps on its 8 x 8 entries and
// stores its results, while warp 7 fetches block lw + 1 and warp 6 publishes the previous waves.
__device__ __forceinline__ void quadrant_sweep(double *Ys, double *Cs, const double *LU, const double *Lfa,
                                               const double *Ufl, double *stg, double *tabL, double *tabU, int row0,
                                               int col0, const Stream &sm, const TiledKernelParams &p,
                                               double &max_abs_e) {
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = lane >> 2, t = lane & 3;
    __shared__ double xch[8 * 2 * 16];
    __shared__ unsigned long long s_badkey;
    const double *Ls = LU, *Us = LU;
    // coefficient tables of the 8 diagonal leaves (see phase A); also clears the exchange buffers
    for (int c = tid; c < Q * TAB_LD; c += blockDim.x) {
        const int r = c / TAB_LD, k = c - r * TAB_LD;       // r: row (L) or column (U) inside the quadrant
        const int src = k - 7, blk = r & ~7, in = r & 7;    // source index inside the leaf
        const bool ok = src >= 0 && src < in;
        tabL[c] = ok ? Ls[CI(r * QLD + blk + src, QMAT, 112)] : 0.0;
        tabU[c] = ok ? Us[CI((blk + src) * QLD + r, QMAT, 113)] : 0.0;
    }
    if (tid < 8 * 2 * 16) xch[tid] = 0.0;
    if (tid == 0) s_badkey = ~0ull;
    unsigned long long badkey = ~0ull;
    const bool fresh = sm.prog_above != nullptr || sm.prog_left != nullptr;
    double *stgE = stg, *stgC = stg + 2 * STG_E;
    // Warp 7 (idle in every leaf-wave but the eighth) is the streaming warp: it fetches the next block of
    // the neighbours' results while the other warps sweep their leaves: 8 + 8 pieces of 16 bytes per lane.
    auto fetch_block = [&](int blk) {
        await_progress(p, sm.prog_above, sm.prog_left, (unsigned)(blk + 8));
        if (sm.prog_above) {        // E above: 64 rows x 8 columns [8 blk, 8 blk + 8)
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int piece = lane + 32 * i, r = piece >> 2, c2 = (piece & 3) * 2;
                cp_async16(stgE + CI((blk & 1) * STG_E + r * STG_E_LD + c2, 2 * STG_E - 1, 108),
                           p.Ebuf + CI((sm.e_above - p.Ebuf) + (long)r * p.np + blk * 8 + c2, (long)p.ntm * T * p.np - 1, 109), 16);
            }
        }
        if (sm.prog_left) {         // C to the left: rows [8 blk, 8 blk + 8) x 64 columns
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int piece = lane + 32 * i, r = piece >> 5, c2 = (piece & 31) * 2;
                cp_async16(stgC + CI((blk & 1) * STG_C + r * QLD + c2, 2 * STG_C - 1, 110),
                           p.Cbuf + CI((sm.c_left - p.Cbuf) + (long)(blk * 8 + r) * p.np + c2, (long)p.ntm * T * p.np - 1, 111), 16);
            }
        }
        cp_async_commit();
        cp_async_wait<0>();
    };
    if (tid == 7 * 32) {
        // this quadrant is about to sweep: the one below it and the one to its right may start getting ready
        const int qi = sm.q >> 1, qj = sm.q & 1;
        if (qi == 0) quadrant_arrive(p, sm.I, sm.J, sm.q + 2);
        else if (sm.I + 1 < p.ntm) quadrant_arrive(p, sm.I + 1, sm.J, sm.q - 2);
        if (qj == 0) quadrant_arrive(p, sm.I, sm.J, sm.q + 1);
        else if (sm.J + 1 < p.ntn) quadrant_arrive(p, sm.I, sm.J + 1, sm.q - 1);
    }
    __syncwarp();
    if (fresh && warp == 7) fetch_block(0);

    TS_MARK(2);                                          // tables, first fetch
    for (int lw = 0; lw < 15; ++lw) {
        __syncthreads();
        TS_MARK(lw <= 7 ? 3 : 9);                            // barrier at the top of the leaf-wave
        if (fresh && lw <= 7) {
            // ---- pull phase: warp w adds P = Lfa[row block w, :] E_above[:, block lw] to C and Y of leaf
            // (w, lw), and R = C_left[block lw, :] Ufl[:, column block w] to Y of leaf (lw, w)
            if (sm.prog_above) {
                double p0 = 0.0, p1 = 0.0, p2 = 0.0, p3 = 0.0;
                const double *A = Lfa + (warp * 8 + g) * QLD + t;
                const double *B = stgE + (lw & 1) * STG_E + t * STG_E_LD + g;
#pragma unroll 4
                for (int kk = 0; kk < Q; kk += 8) {
                    dmma_m8n8k4(p0, p1, A[kk], B[kk * STG_E_LD]);
                    dmma_m8n8k4(p2, p3, A[kk + 4], B[(kk + 4) * STG_E_LD]);
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
                const double *B = Ufl + t * QLD + warp * 8 + g;
#pragma unroll 4
                for (int kk = 0; kk < Q; kk += 8) {
                    dmma_m8n8k4(r0, r1, A[kk], B[kk * QLD]);
                    dmma_m8n8k4(r2, r3, A[kk + 4], B[(kk + 4) * QLD]);
                }
                r0 += r2; r1 += r3;
                double2 *yq = reinterpret_cast<double2 *>(Ys + (lw * 8 + g) * QLD + warp * 8 + t * 2);
                double2 yv = *yq;
                yv.x += r0; yv.y += r1;
                *yq = yv;
            }
            TS_MARK(4);                                      // streamed pull (own DMMAs)
            __syncthreads();
            TS_MARK(5);                                      // barrier after the pull
        }
        // ---- warp 7 fetches the next block of the neighbours; warp 6 (a leaf of its own only in leaf-waves
        // 6 to 8) publishes what the previous leaf-waves stored: the barriers above order those stores
        // before this thread's fence
        if (warp == 7 && fresh && lw < 7) fetch_block(lw + 1);
        if (tid == 6 * 32 && lw > 0) {
            __threadfence();
            st_release_u32(sm.prog_self, (unsigned)lw);
        }
        const int a_lo = max(0, lw - 7), a_hi = min(7, lw);
        const int a = a_lo + warp, b = lw - a;
        if (a <= a_hi) {
            leaf_pull(Ys, Cs, Ls, Us, a, b, g, t);
            __syncwarp();
            TS_MARK(lw <= 7 ? 6 : 10);                       // leaf_pull
            // Phase A.  Lane l owns entries (i0, j) and (i0 + 4, j) of the 8 x 8 leaf, i0 = l & 3,
            // j = l >> 2.  At step s the lane whose entry lies on anti-diagonal s rounds it and posts
            // the error (by column) and the final C value (by row) to a 16-double per-warp exchange
            // buffer; after a warp barrier EVERY lane applies one downward and one rightward push
            // to both of its entries (Algorithm 3 lines 8-16 restricted to the leaf).  The pushes
            // are branch-free: the coefficients come from tables that hold zeros wherever no push
            // is due (source not on this anti-diagonal, or entry already rounded), so stale
            // exchange slots are multiplied by zero.
            const int i0 = lane & 3, j = lane >> 2;
            double *yp = Ys + CI((a * 8 + i0) * QLD + b * 8 + j, QMAT - 4 * QLD, 114);
            double *cp = Cs + CI((a * 8 + i0) * QLD + b * 8 + j, QMAT - 4 * QLD, 115);
            double y0 = yp[0], y1 = yp[4 * QLD], c0 = cp[0], c1 = cp[4 * QLD];
            // tabL[row][7 + is] = L(row, is) for 0 <= is < row else 0; at step s, is = s - j
            const double *tl0 = tabL + CI((a * 8 + i0) * TAB_LD + 7 - j, (Q - 4) * TAB_LD - 14, 116);
            const double *tl1 = tl0 + 4 * TAB_LD;
            // tabU[col][7 + js] = U(js, col) for 0 <= js < col else 0; at step s, js = s - i
            const double *tu0 = tabU + CI((b * 8 + j) * TAB_LD + 7 - i0 - 4, Q * TAB_LD - 18, 117) + 4;
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
                const double ed = ex[j], cr0 = ex[8 + i0], cr1 = ex[12 + i0];
                const double l0 = tl0[s], l1 = tl1[s], u0 = tu0[s], u1 = tu1[s];
                y0 = fma(l0, ed, y0); c0 = fma(l0, ed, c0); y0 = fma(cr0, u0, y0);   // fold, push down, push right
                y1 = fma(l1, ed, y1); c1 = fma(l1, ed, c1); y1 = fma(cr1, u1, y1);
            }
            yp[0] = y0; yp[4 * QLD] = y1; cp[0] = c0; cp[4 * QLD] = c1;
            TS_MARK(lw <= 7 ? 7 : 11);                       // the 15 anti-diagonal steps
            // results of the leaf: E and C to the workspace (for the neighbours and for the far parts of
            // later tiles), Z (and the caller's E) to the output
            {
                const int gr = row0 + a * 8 + i0, gc = col0 + b * 8 + j;
                const long at = CI((long)gr * p.np + gc, (long)p.ntm * T * p.np - 4 * p.np, 118);
                p.Ebuf[at] = y0; p.Ebuf[at + 4 * p.np] = y1;
                p.Cbuf[at] = c0; p.Cbuf[at + 4 * p.np] = c1;
                if (gc < p.n) {
                    if (gr < p.m) {
                        p.Z[CI((long)gr * p.ldz + gc, (long)(p.m - 1) * p.ldz + p.n, 119)] = z0;
                        if (p.Euser) p.Euser[(long)gr * p.lde + gc] = y0;
                        max_abs_e = fmax(max_abs_e, fabs(y0));
                    }
                    if (gr + 4 < p.m) {
                        p.Z[CI((long)(gr + 4) * p.ldz + gc, (long)(p.m - 1) * p.ldz + p.n, 120)] = z1;
                        if (p.Euser) p.Euser[(long)(gr + 4) * p.lde + gc] = y1;
                        max_abs_e = fmax(max_abs_e, fabs(y1));
                    }
                }
            }
            TS_MARK(lw <= 7 ? 8 : 12);                       // stores of the leaf
        }
    }
    __syncthreads();
    TS_MARK(13);
    if (tid == 0) {                      // everything is stored: the quadrant is complete
        __threadfence();
        st_release_u32(sm.prog_self, 15u);
    }
    // status: the earliest (in sweep order) unrepresentable value of the quadrant, if any
    if (badkey != ~0ull) atomicMin(&s_badkey, badkey);
    __syncthreads();
    if (tid == 0 && s_badkey != ~0ull) {
        const unsigned long long k = s_badkey;
        report(p.info, ((k >> 41) & 1ull) ? GPTQ2D_ERR_INT_OVERFLOW : GPTQ2D_ERR_NONFINITE,
               (int)((k >> 20) & 0x1fffffull), (int)(k & 0xfffffull), max(p.batch_index, 0));
    }
}

// 64 x 64 diagonal blocks of both factors into one shared-memory matrix: below the diagonal
// L[r0 + i][r0 + k], above it U[c0 + k][c0 + j], zeros on it and outside the matrices.
__device__ __forceinline__ void load_lu_diag_async(double *dst, const TiledKernelParams &p, int r0, int c0) {
#pragma unroll
    for (int it = 0; it < 16; ++it) {
        const int c = threadIdx.x + it * TILED_THREADS;
        const int i = c >> 6, j = c & 63;
        const bool lower = j < i, upper = j > i;
        const bool take = lower ? (r0 + i < p.m) : (upper && c0 + j < p.n);     // r0 + j < r0 + i, c0 + i < c0 + j
        const double *src = lower ? p.L + (long)(r0 + i) * p.ldl + r0 + j : p.U + (long)(c0 + i) * p.ldu + c0 + j;
        cp_async8(dst + CI(i * QLD + j, QMAT, 121), take ? src : p.L, take ? 8 : 0);
    }
}

// ---------------------------------------------------------------------------------------------
// One 64 x 64 quadrant q (0: top-left, 1: top-right, 2: bottom-left, 3: bottom-right) of tile
// (I, J): the unit of work on the critical path.  In the grid of quadrants it sits at
// (r, c) = (2 I + q / 2, 2 J + q % 2).
//
// On entry the quadrant's part of the tile's Cbuf region holds the FAR part of Cd (all source
// tiles above except the two nearest) and its Ebuf part the FAR part of Rt.  The task
//   1. pulls what the two nearest tiles and its own tile contribute from quadrants that are COMPLETE
//      (rows 2 I - 4 .. r - 2, columns 2 J - 4 .. c - 2 of the quadrant grid): up to eight 64^3 DMMA
//      products;
//   2. forms Y = X + Rt + Cd, C = Cd and runs Algorithm 3 on the quadrant, taking the contributions
//      of the quadrant right above it and of the one right to its left block by block as they
//      finish (quadrant_sweep), and publishing its own leaves wave by wave.
__device__ __forceinline__ void sweep_quadrant(int I, int J, int q, double *smem, const TiledKernelParams &p,
                                               double &max_abs_e) {
    double *Ys = smem, *Cs = smem + QMAT, *LU = smem + 2 * QMAT, *Lfa = smem + 3 * QMAT, *Ufl = smem + 4 * QMAT;
    double *tabL = smem + 5 * QMAT, *tabU = tabL + Q * TAB_LD;
    double *stg = tabU + Q * TAB_LD;
    const int tid = threadIdx.x;
    const int qi = q >> 1, qj = q & 1;
    const int row0 = I * T + qi * Q, col0 = J * T + qj * Q;
    double *eQ = p.Ebuf + (long)row0 * p.np + col0;
    double *cQ = p.Cbuf + (long)row0 * p.np + col0;

    // ---- 1. pulls from complete quadrants: rows r' = max(0, 2 I - 4) .. r - 2 of the quadrant grid (the
    // two tiles above, without the quadrant right above this one), columns likewise.  The far parts of the
    // tile cover everything further away.  Oldest sources first; the two newest, (r - 2, c) and
    // (r, c - 2), may still be sweeping their last leaves when this task starts and are waited for
    // right before their blocks are requested (they are running: the neighbour between them and this
    // quadrant could not have started otherwise).
    QAcc accC, accR;
    accC.zero();
    accR.zero();
    TS_RESET();
    {   // X of the quadrant is read once, after the pulls, and comes from HBM: ask for it now (one 128-byte line per thread)
        const int gr = row0 + (tid >> 2), gc = col0 + (tid & 3) * 16;
        if (gr < p.m && gc < p.n) asm volatile("prefetch.global.L2 [%0];\n" ::"l"(p.X + (long)gr * p.ldx + gc));
    }
    {
        const int r = 2 * I + qi, c = 2 * J + qj;
        const int fa = max(0, 2 * I - 4), fl = max(0, 2 * J - 4);
        const int nsa = max(0, r - 1 - fa), nsl = max(0, c - 1 - fl), ns = nsa + nsl;
        auto prog_of = [&](int rr, int cc) {
            return p.qprog + CI(((long)(rr >> 1) * p.ntn + (cc >> 1)) * 4 + (rr & 1) * 2 + (cc & 1), 4L * p.ntm * p.ntn, 124);
        };
        // step i -> (direction, block): the older blocks of both directions first, then the newest of each
        const int olda = max(0, nsa - 1), oldl = max(0, nsl - 1);
        auto step_dir = [&](int i) {
            return i < olda ? 0 : (i < olda + oldl ? 1 : ((i == olda + oldl && nsa > 0) ? 0 : 1));
        };
        auto step_blk = [&](int i) {
            return i < olda ? fa + i : (i < olda + oldl ? fl + (i - olda) : (step_dir(i) == 0 ? r - 2 : c - 2));
        };
        // three buffer pairs: one being multiplied, two being filled; all unused until the sweep proper
        auto bufA = [&](int j) { return j == 0 ? Lfa : (j == 1 ? LU : Ys); };
        auto bufB = [&](int j) { return j == 0 ? Ufl : (j == 1 ? Cs : tabL); };
        auto issue = [&](int i) {
            double *Ab = bufA(i % 3), *Bb = bufB(i % 3);
            const int dir = step_dir(i), blk = step_blk(i), k0 = blk * Q;
            if (i >= olda + oldl) await_progress(p, dir == 0 ? prog_of(blk, c) : prog_of(r, blk), nullptr, 15u);
            if (dir == 0) {
                if (p.l_al16) load_full_block_async16(Ab, p.L, p.ldl, p.m, row0, k0);
                else load_factor_block_async(Ab, p.L, p.ldl, p.m, row0, k0, 0);
                load_quadrant_async(Bb, p.Ebuf + (long)k0 * p.np + col0, p.np);
            } else {
                load_quadrant_async(Ab, p.Cbuf + (long)row0 * p.np + k0, p.np);
                if (p.u_al16) load_full_block_async16(Bb, p.U, p.ldu, p.n, k0, col0);
                else load_factor_block_async(Bb, p.U, p.ldu, p.n, k0, col0, 0);
            }
            cp_async_commit();
        };
        // the older sources: one warp each makes sure its quadrant is complete (it almost always is)
        {
            const int w = threadIdx.x >> 5;
            if (w < olda) await_progress(p, prog_of(fa + w, c), nullptr, 15u);
            else if (w < olda + oldl) await_progress(p, prog_of(r, fl + (w - olda)), nullptr, 15u);
        }
        __syncthreads();
        for (int i = 0; i < ns && i < 2; ++i) issue(i);
        for (int i = 0; i < ns; ++i) {
            if (i + 1 < ns) cp_async_wait<1>(); else cp_async_wait<0>();     // step i's operands have landed
            __syncthreads();
            // every warp is past product i - 1 now, so its buffer pair, (i + 2) % 3, can take step i + 2
            if (i + 2 < ns) issue(i + 2);
            if (step_dir(i) == 0) quad_mma(accC, bufA(i % 3), bufB(i % 3)); else quad_mma(accR, bufA(i % 3), bufB(i % 3));
        }
        __syncthreads();
    }

    TS_MARK(0);                                          // pulls from the two nearest tiles
    // ---- 2. operands of the sweep
    Stream sm;
    sm.I = I; sm.J = J; sm.q = q;
    const long tq = ((long)I * p.ntn + J) * 4;
    sm.prog_self = p.qprog + tq + q;
    sm.prog_above = nullptr; sm.prog_left = nullptr; sm.e_above = nullptr; sm.c_left = nullptr;
    if (row0 > 0) {
        sm.prog_above = qi ? p.qprog + tq + (q - 2) : p.qprog + ((long)(I - 1) * p.ntn + J) * 4 + (q + 2);
        sm.e_above = p.Ebuf + (long)(row0 - Q) * p.np + col0;
        if (p.l_al16) load_full_block_async16(Lfa, p.L, p.ldl, p.m, row0, row0 - Q);
        else load_factor_block_async(Lfa, p.L, p.ldl, p.m, row0, row0 - Q, 0);
    }
    if (col0 > 0) {
        sm.prog_left = qj ? p.qprog + tq + (q - 1) : p.qprog + ((long)I * p.ntn + (J - 1)) * 4 + (q + 1);
        sm.c_left = p.Cbuf + (long)row0 * p.np + (col0 - Q);
        if (p.u_al16) load_full_block_async16(Ufl, p.U, p.ldu, p.n, col0 - Q, col0);
        else load_factor_block_async(Ufl, p.U, p.ldu, p.n, col0 - Q, col0, 0);
    }
    load_lu_diag_async(LU, p, row0, col0);
    load_quadrant_async(Cs, cQ, p.np);
    load_quadrant_async(Ys, eQ, p.np);
    cp_async_commit();
    double xv[16];
#pragma unroll
    for (int it = 0; it < 16; ++it) {                     // X of the quadrant, zero outside the matrix
        int c = tid + it * TILED_THREADS;
        int gr = row0 + (c >> 6), gc = col0 + (c & 63);
        xv[it] = (gr < p.m && gc < p.n) ? __ldg(p.X + CI((long)gr * p.ldx + gc, (long)(p.m - 1) * p.ldx + p.n, 122)) : 0.0;
    }
    cp_async_wait<0>();
    __syncthreads();
    quad_add_to(Cs, QLD, accC, false);                    // Cd = far part + pulls from complete quadrants
    quad_add_to(Ys, QLD, accR, false);                    // Rt likewise
    __syncthreads();
#pragma unroll
    for (int it = 0; it < 16; ++it) {                     // Y = X + Rt + Cd
        int c = tid + it * TILED_THREADS;
        int r = c >> 6, cc = c & 63;
        Ys[CI(r * QLD + cc, QMAT, 123)] += xv[it] + Cs[r * QLD + cc];
    }
    TS_MARK(1);                                          // operand loads, Y = X + Rt + Cd
    quadrant_sweep(Ys, Cs, LU, Lfa, Ufl, stg, tabL, tabU, row0, col0, sm, p, max_abs_e);
    __syncthreads();
}

// ---------------------------------------------------------------------------------------------
// Far parts in claim order: wave by wave (I + J ascending); inside a wave the longest contractions
// first (the Cd part of tile (I, J) has I - 2 chunks, the Rt part J - 2), so that a wave's far parts
// finish close together instead of the long ones trailing.
__device__ __forceinline__ void decode_task(int task, int ntm, int ntn, int &type, int &I, int &J) {
    int tt = task;
    for (int w = 0; w < ntm + ntn - 1; ++w) {
        int lo = max(0, w - ntn + 1), hi = min(ntm - 1, w);
        int cnt = 2 * (hi - lo + 1);
        if (tt < cnt) {
            const int k = tt >> 1;
            type = tt & 1;
            I = type == 0 ? hi - k : lo + k;        // Cd parts by descending I, Rt parts by descending J
            J = w - I;
            return;
        }
        tt -= cnt;
    }
    type = 0;
    I = J = 0;
}

// accumulator tile <-> its 128 x 128 region of a padded workspace buffer
__device__ __forceinline__ void store_acc(const Acc &acc, double *dstT, long np, int wm, int wn, int g, int t) {
#pragma unroll
    for (int a = 0; a < 8; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            double2 v;
            v.x = acc.v[a][b][0];
            v.y = acc.v[a][b][1];
            *reinterpret_cast<double2 *>(dstT + CI((long)(wm * 64 + a * 8 + g) * np + wn * 32 + b * 8 + t * 2, 127L * np + T - 1, 126)) = v;
        }
}
__device__ __forceinline__ void load_acc(Acc &acc, const double *srcT, long np, int wm, int wn, int g, int t) {
#pragma unroll
    for (int a = 0; a < 8; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            double2 v = __ldcg(reinterpret_cast<const double2 *>(srcT + (long)(wm * 64 + a * 8 + g) * np + wn * 32 +
                                                                 b * 8 + t * 2));
            acc.v[a][b][0] = v.x;
            acc.v[a][b][1] = v.y;
        }
}

// Global ring of ready quadrant tasks (size a power of two).  It cannot overflow: a quadrant depends,
// directly or through others, on the quadrant above it and on the one to its left, so the quadrants
// of one matrix that are ready at the same time lie on an anti-chain of its 2 ntm x 2 ntn quadrant
// grid, at most 2 min(ntm, ntn) of them; each enters the ring once.  A single matrix therefore
// needs at most 512 slots (ntm, ntn <= 256 tiles would be 32768 rows); a batched launch sizes its
// ring from the sum over its matrices.
constexpr unsigned QCAP = 4096;
constexpr int FAR_RUN_CHUNKS = 64;      // a far part looks at the ready ring every this many K = 128 chunks
constexpr unsigned IDLE_SLEEP_NS = 100; // pause of a CTA that found nothing to do (100 - 1600 ns and far runs of 8 - 64 chunks all time within 1 %)

// multi-producer / multi-consumer ring in global memory; slot value 0 = empty.
__device__ __forceinline__ void ready_push(const TiledKernelParams &p, unsigned entry) {
    unsigned t = atomicAdd(p.q_tail, 1u);
    st_release_u32(p.q_slots + CI(t & p.qmask, (long)p.qmask + 1, 127), entry | 0x80000000u);
}
// thread 0 only.  Returns 0 if the queue is empty (or on abort), else the entry (bit 31 set).
__device__ __forceinline__ unsigned ready_pop(const TiledKernelParams &p) {
    for (;;) {
        unsigned h = ld_relaxed_u32(p.q_head), t = ld_relaxed_u32(p.q_tail);
        if ((int)(t - h) <= 0) return 0u;
        if (atomicCAS(p.q_head, h, h + 1u) != h) continue;
        unsigned *slot = p.q_slots + (h & p.qmask);
        unsigned long long spins = 0;
        unsigned e;
        while ((e = ld_acquire_u32(slot)) == 0u) {          // producer has the ticket but has not written yet
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

// Arrivals a quadrant task at (r, c) of the quadrant grid waits for: the two far parts of its tile and
// the quadrants at (r - 1, c) and (r, c - 1) having begun to sweep.
__device__ __forceinline__ unsigned quadrant_needed(int I, int J, int q) {
    const int r = 2 * I + (q >> 1), c = 2 * J + (q & 1);
    return 2u + (r >= 1 ? 1u : 0u) + (c >= 1 ? 1u : 0u);
}
// A quadrant that lies wholly outside the matrix (ragged last tile row / column) is never a task:
// arrivals at it are dropped here, its region of the workspace keeps the zeros the far parts parked
// there, and nothing inside the matrix depends on it.
__device__ __forceinline__ bool quadrant_exists(const TiledKernelParams &p, int I, int J, int q) {
    return I * T + (q >> 1) * Q < p.m && J * T + (q & 1) * Q < p.n;
}
__device__ __forceinline__ void quadrant_arrive(const TiledKernelParams &p, int I, int J, int q) {
    if (!quadrant_exists(p, I, J, q)) return;
    unsigned old = atomicAdd(p.qdep + CI(((long)I * p.ntn + J) * 4 + q, 4L * p.ntm * p.ntn, 125), 1u);
    if (old + 1u == quadrant_needed(I, J, q)) {
        // single matrix: q | I (14 bits) | J (15 bits); batched: q | matrix (13 bits) | I (8 bits) | J (8 bits)
        const unsigned entry = p.batch_index >= 0
            ? (((unsigned)q << 29) | ((unsigned)p.batch_index << 16) | ((unsigned)I << 8) | (unsigned)J | 0x80000000u)
            : (((unsigned)q << 29) | ((unsigned)I << 15) | (unsigned)J | 0x80000000u);
        __threadfence();
        ready_push(p, entry);
    }
}

constexpr int FAR_CTX = 2;       // far parts a CTA may hold at once (one live in registers, the others parked)

// The persistent scheduler loop.  BATCHED = false: one matrix, described by the kernel argument
// itself.  BATCHED = true: many matrices in one launch; the kernel argument holds what they share
// (claim counter, ready ring, abort word, totals) and each task works on a shared-memory copy of
// its matrix' descriptor (slots 0..FAR_CTX-1: the far contexts, slot FAR_CTX: the quadrant task).
// PANELS = true (single matrix only): the inputs are still being copied in while the kernel runs, in
// blocks of COPY_BLOCK_TILES x COPY_BLOCK_TILES tiles and in the order the wavefront needs them: step
// s brings the blocks of X on block anti-diagonal s, the block row s of L and the block column s of
// U.  A task on tile (I, J) starts once the copy stream has announced the step of its block
// (p.panels_ready counts the steps that arrived).
template <bool BATCHED, bool PANELS>
__global__ void __launch_bounds__(TILED_THREADS, 1) round_tiled_kernel(TiledKernelParams p) {
    extern __shared__ __align__(16) double smem[];
    __shared__ int s_task[4];
    __shared__ int s_ctx[FAR_CTX][7];      // far-part contexts, oldest first: type, I, J, pos, nfar, task, view slot
    __shared__ int s_nctx, s_pick, s_state;
    __shared__ unsigned s_pop;
    __shared__ double s_red[TILED_THREADS / 32];
    __shared__ TiledKernelParams s_view[BATCHED ? FAR_CTX + 1 : 1];
    static_assert(!BATCHED || FAR_CTX == 2, "view slots of far contexts are handed out as 0 / 1");
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int wm = warp >> 2, wn = warp & 3, g = lane >> 2, t = lane & 3;
    CHECKED_SET_INFO(p.info);            // (checked builds: every CTA writes the same pointer before its first barrier)
    double max_abs_e = 0.0;
    int cur = -1;                  // context whose accumulator is live in registers (uniform), -1: none
    unsigned long long spins = 0;
    Acc acc;
    acc.zero();
#ifndef TILED_STATS
#define SC_MARK(slot)
#endif
#ifdef TILED_STATS
    if (tid < 16) g_ts[tid] = 0;
    if (tid < 8) g_sched[tid] = 0;
    long long sc_t = clock64();
#define SC_MARK(slot) do { if (tid == 0) { const long long n_ = clock64(); g_sched[slot] += n_ - sc_t; sc_t = n_; } } while (0)
#endif
    if (tid == 0) {
        s_nctx = 0;
        if (BATCHED)
            for (int k = 0; k <= FAR_CTX; ++k) s_view[k].batch_index = -1;
    }

    // the descriptor a task works on: the kernel argument itself for a single matrix (spelled so that the
    // compiler sees plain parameter accesses there), a shared-memory copy in a batched launch
#define VIEW(slot) (BATCHED ? s_view[slot] : p)
    auto load_view = [&](int slot, int b) {            // thread 0, before the barrier that publishes the task
        if constexpr (BATCHED) {
            if (s_view[slot].batch_index != b) {
                const unsigned long long *src = reinterpret_cast<const unsigned long long *>(p.probs + b);
                unsigned long long *dst = reinterpret_cast<unsigned long long *>(&s_view[slot]);
                unsigned long long v[sizeof(TiledKernelParams) / 8];
#pragma unroll
                for (int i = 0; i < (int)(sizeof(TiledKernelParams) / 8); ++i) v[i] = __ldg(src + i);   // all in flight
#pragma unroll
                for (int i = 0; i < (int)(sizeof(TiledKernelParams) / 8); ++i) dst[i] = v[i];
            }
        }
    };
    auto entry_matrix = [&](unsigned e) { return (int)((e >> 16) & 0x1fffu); };
    // thread 0.  Far parts poll (they have other things to do); a popped quadrant task waits, bounded:
    // the copies make progress on their own.
    auto panels_arrived = [&](int need) -> bool {
        if constexpr (PANELS) return ld_acquire_u32(p.panels_ready) >= (unsigned)need;
        else return true;
    };
    auto await_panels = [&](unsigned e) -> unsigned {
        if constexpr (PANELS) {
            if (e == 0u) return e;
            const int need = ((int)((e >> 15) & 0x3fffu) >> COPY_BLOCK_TILES_LOG2) +
                             ((int)(e & 0x7fffu) >> COPY_BLOCK_TILES_LOG2) + 1;
            unsigned long long it = 0;
            while (!panels_arrived(need)) {
                if (++it > p.panel_spin_limit || ld_relaxed_u32(p.abort) != 0u) {
                    report(p.info, GPTQ2D_ERR_DEVICE_TIMEOUT, -6, need, (int)blockIdx.x);
                    atomicExch(p.abort, 1u);
                    return 0u;
                }
                __nanosleep(200);
            }
        }
        return e;
    };
    auto tile_region = [&](int k) {
        const TiledKernelParams &pk = VIEW(s_ctx[k][6]);
        return (s_ctx[k][0] == 0 ? pk.Cbuf : pk.Ebuf) +
               CI((long)s_ctx[k][1] * T * pk.np + (long)s_ctx[k][2] * T, (long)(pk.ntm - 1) * T * pk.np + (long)(pk.ntn - 1) * T + 1, 128);
    };

    for (;;) {
        // ---- thread 0 looks for work: a ready quadrant task first, else the oldest far part that can
        // go on, else (room and tasks left) a new far part.  s_state: 0 run far part s_pick, 1 serve the
        // ring, 2 nothing to do right now, 3 all tiles swept, 4 abort.
        __syncthreads();
        if (tid == 0) {
            int state = 2, pick = -1;
            unsigned e = 0u;
            // A far part of this CTA that is at most two chunks from done and can go on comes before
            // everything else: the four quadrant tasks of its tile cannot start without it, and other
            // CTAs can serve the ring.
            for (int k = 0; k < s_nctx && pick < 0; ++k) {
                const TiledKernelParams &pk = VIEW(s_ctx[k][6]);
                const int ty = s_ctx[k][0], pos = s_ctx[k][3], left = s_ctx[k][4] - pos;
                if (left < 1 || left > 2) continue;
                const unsigned *fl = ty == 0 ? pk.flagS + (long)pos * pk.ntn + s_ctx[k][2]
                                             : pk.flagS + (long)s_ctx[k][1] * pk.ntn + pos;
                if (ld_acquire_u32(fl) != 0u &&
                    panels_arrived(((ty == 0 ? s_ctx[k][1] : s_ctx[k][2]) >> COPY_BLOCK_TILES_LOG2) + 1))
                    pick = k;
            }
            if (ld_relaxed_u32(p.abort) != 0u) state = 4;
            else if (pick >= 0) state = 0;
            else if ((e = await_panels(ready_pop(p))) != 0u) {
                state = 1;
                load_view(FAR_CTX, entry_matrix(e));
            } else {
                int n = s_nctx;
                for (int k = 0; k < n && pick < 0; ++k) {
                    const TiledKernelParams &pk = VIEW(s_ctx[k][6]);
                    const int ty = s_ctx[k][0], pos = s_ctx[k][3];
                    const unsigned *fl = ty == 0 ? pk.flagS + (long)pos * pk.ntn + s_ctx[k][2]
                                                 : pk.flagS + (long)s_ctx[k][1] * pk.ntn + pos;
                    // a Cd part reads L in the block row of I, an Rt part U in the block column of J
                    if ((pos >= s_ctx[k][4] || ld_acquire_u32(fl) != 0u) &&
                        panels_arrived(((ty == 0 ? s_ctx[k][1] : s_ctx[k][2]) >> COPY_BLOCK_TILES_LOG2) + 1))
                        pick = k;
                }
                if (pick < 0 && n < FAR_CTX && ld_relaxed_u32(p.counter) < (unsigned)p.ntasks) {
                    int task = (int)atomicAdd(p.counter, 1u);
                    if (task < p.ntasks) {
                        int ty, fi, fj, slot = 0;
                        if constexpr (BATCHED) {
                            const unsigned ft = __ldg(p.far_tasks + task);
                            ty = (int)((ft >> 16) & 1u); fi = (int)((ft >> 8) & 255u); fj = (int)(ft & 255u);
                            slot = n == 0 ? 0 : 1 - s_ctx[0][6];
                            load_view(slot, (int)(ft >> 17));
                        } else {
                            decode_task(task, p.ntm, p.ntn, ty, fi, fj);
                        }
                        const TiledKernelParams &pk = VIEW(slot);
                        s_ctx[n][0] = ty; s_ctx[n][1] = fi; s_ctx[n][2] = fj; s_ctx[n][3] = 0;
                        s_ctx[n][4] = max(0, (ty == 0 ? fi : fj) - 2); s_ctx[n][5] = task; s_ctx[n][6] = slot;
                        s_nctx = n + 1;
                        const unsigned *fl = ty == 0 ? pk.flagS + fj : pk.flagS + (long)fi * pk.ntn;
                        if ((s_ctx[n][4] == 0 || ld_acquire_u32(fl) != 0u) && panels_arrived(((ty == 0 ? fi : fj) >> COPY_BLOCK_TILES_LOG2) + 1))
                            pick = n;
                    }
                }
                if (pick >= 0) state = 0;
                else if (s_nctx == 0 && ld_relaxed_u32(p.counter) >= (unsigned)p.ntasks &&
                         ld_relaxed_u32(p.tiles_done) >= (unsigned)p.ntiles_total) state = 3;
            }
            s_state = state; s_pick = pick; s_pop = e;
        }
        __syncthreads();
        const int state = s_state;
        SC_MARK(4);
        if (state >= 3) break;
        if (state == 2) {
            if (++spins > p.spin_limit) {
                if (tid == 0) {
                    report(p.info, GPTQ2D_ERR_DEVICE_TIMEOUT, -4, (int)blockIdx.x, s_nctx);
                    atomicExch(p.abort, 1u);
                }
                break;
            }
            __nanosleep(s_nctx == 0 ? IDLE_SLEEP_NS : 100);
            SC_MARK(3);
            continue;
        }
        spins = 0;

        if (state == 1) {
            // ================= A: quadrant tasks from the ready ring.  The accumulator of the live far part,
            // if any, stays in its registers meanwhile: the quadrant task takes the shared memory only.
            unsigned e = s_pop;
            while (e != 0u) {
                const TiledKernelParams &pq = VIEW(FAR_CTX);
                const int q = (int)((e >> 29) & 3u);
                const int I = BATCHED ? (int)((e >> 8) & 255u) : (int)((e >> 15) & 0x3fffu);
                const int J = BATCHED ? (int)(e & 255u) : (int)(e & 0x7fffu);
                sweep_quadrant(I, J, q, smem, pq, max_abs_e);
#ifdef TILED_STATS
                if (tid == 0) g_ts[15] += 1;
#endif
                if constexpr (BATCHED) {                  // max |E| is kept per matrix: flush after every task
                    for (int o = 16; o > 0; o >>= 1) max_abs_e = fmax(max_abs_e, __shfl_xor_sync(0xffffffffu, max_abs_e, o));
                    if (lane == 0 && max_abs_e > 0.0) atomic_max_nonneg_double(pq.max_abs_e, max_abs_e);
                    max_abs_e = 0.0;
                }
                // arrivals at everything this quadrant feeds, one per thread (each is a dependent global
                // atomic round trip); sweep_quadrant ended with a barrier, so each arriving thread's fence
                // covers the whole CTA's results
                if (tid < 8) {
                    __threadfence();
                    if (tid == 6) {
                        unsigned done = atomicAdd(pq.quad_done + (long)I * pq.ntn + J, 1u);
                        const unsigned nquad = (pq.m - I * T > Q ? 2u : 1u) * (pq.n - J * T > Q ? 2u : 1u);
                        if (done + 1u == nquad) {   // tile swept: far parts that list it as a source may go on
                            __threadfence();
                            st_release_u32(pq.flagS + CI((long)I * pq.ntn + J, (long)pq.ntm * pq.ntn, 129), 1u);
                            atomicAdd(pq.rowdone + CI(I, pq.ntm, 130), 1u);
                            atomicAdd(p.tiles_done, 1u);
                        }
                    }
                }
                __syncthreads();
                if (tid == 0) {
                    // with far parts in hand, go back to the top of the loop after every task (see there)
                    const unsigned en = s_nctx > 0 ? 0u : await_panels(ready_pop(p));
                    if (en != 0u) load_view(FAR_CTX, entry_matrix(en));
                    s_pop = en;
                }
                __syncthreads();
                e = s_pop;
            }
            SC_MARK(0);
            continue;
        }

        // ================= B: far part s_pick (every source tile of the contraction except the two nearest)
        const int k = s_pick;
        const TiledKernelParams &pk = VIEW(s_ctx[k][6]);
        if (k != cur) {
            if (cur >= 0 && s_ctx[cur][3] > 0) store_acc(acc, tile_region(cur), VIEW(s_ctx[cur][6]).np, wm, wn, g, t);
            if (s_ctx[k][3] > 0) load_acc(acc, tile_region(k), pk.np, wm, wn, g, t);
            else acc.zero();
            cur = k;
        }
        const int f_type = s_ctx[k][0], f_I = s_ctx[k][1], f_J = s_ctx[k][2], f_pos = s_ctx[k][3], f_nfar = s_ctx[k][4];
        int new_pos = f_pos;
        if (f_pos < f_nfar) {
            const unsigned *flags = f_type == 0 ? pk.flagS + f_J : pk.flagS + (long)f_I * pk.ntn;
            const long fstride = f_type == 0 ? pk.ntn : 1;
            // how many source tiles from f_pos on are swept already (the first one is)
            __syncthreads();
            if (tid == 0) s_task[0] = f_nfar;
            __syncthreads();
            for (int idx = f_pos + tid; idx < f_nfar; idx += blockDim.x)
                if (ld_acquire_u32(flags + (long)idx * fstride) == 0u) atomicMin(&s_task[0], idx);
            __syncthreads();
            const int upto = min(s_task[0], f_pos + FAR_RUN_CHUNKS);
            Operand a, b;
            if (f_type == 0) {
                a.ptr = pk.L + CI((long)f_I * T * pk.ldl + (long)f_pos * T, (long)(pk.m - 1) * pk.ldl + pk.m, 131); a.ld = pk.ldl; a.mn_valid = min(T, pk.m - f_I * T); a.aligned16 = pk.l_al16;
                b.ptr = pk.Ebuf + (long)f_J * T + (long)f_pos * T * pk.np; b.ld = pk.np; b.mn_valid = T; b.aligned16 = true;
            } else {
                a.ptr = pk.Cbuf + (long)f_I * T * pk.np + (long)f_pos * T; a.ld = pk.np; a.mn_valid = T; a.aligned16 = true;
                b.ptr = pk.U + CI((long)f_J * T + (long)f_pos * T * pk.ldu, (long)(pk.n - 1) * pk.ldu + pk.n, 132); b.ld = pk.ldu; b.mn_valid = min(T, pk.n - f_J * T); b.aligned16 = pk.u_al16;
            }
            SC_MARK(2);
            gemm_tile<true, false, BULK_NSTAGE>(acc, smem, a, b, (upto - f_pos) * T);
            SC_MARK(1);
            new_pos = upto;
        }
        if (new_pos >= f_nfar) {
            // far part complete: park the sum (zeros included: the quadrant tasks start from it) and
            // announce it to the four quadrants of its tile; drop the context
            store_acc(acc, tile_region(k), pk.np, wm, wn, g, t);
            __syncthreads();
            if (tid < 4) {
                __threadfence();
                quadrant_arrive(pk, f_I, f_J, tid);
            }
            if (tid == 0) {
                const int n = s_nctx;
                for (int c = k; c + 1 < n; ++c)
                    for (int f = 0; f < 7; ++f) s_ctx[c][f] = s_ctx[c + 1][f];
                s_nctx = n - 1;
            }
            cur = -1;
        } else if (tid == 0) {
            s_ctx[k][3] = new_pos;
        }
        SC_MARK(2);
    }

#ifdef TILED_STATS
    if (tid == 0 && (blockIdx.x % 37) == 0)
        printf("cta %3d scheduler: quadrant tasks %lld far main loop %lld far park/scan %lld idle %lld looking %lld\n", (int)blockIdx.x,
               g_sched[0], g_sched[1], g_sched[2], g_sched[3], g_sched[4]);
    if (tid == 0 && (blockIdx.x % 37) == 0 && g_ts[15] > 0) {
        const long long n_ = g_ts[15];
        printf("cta %3d tasks %lld | per task: nearpull %lld load %lld tables %lld | lw0-7: barA %lld pull %lld barB %lld leafpull %lld "
               "sweep %lld store %lld | lw8-14: bar %lld leafpull %lld sweep %lld store %lld | end %lld\n",
               (int)blockIdx.x, n_, g_ts[0] / n_, g_ts[1] / n_, g_ts[2] / n_, g_ts[3] / n_, g_ts[4] / n_, g_ts[5] / n_, g_ts[6] / n_,
               g_ts[7] / n_, g_ts[8] / n_, g_ts[9] / n_, g_ts[10] / n_, g_ts[11] / n_, g_ts[12] / n_, g_ts[13] / n_);
    }
#endif
    if constexpr (!BATCHED) {
        for (int o = 16; o > 0; o >>= 1) max_abs_e = fmax(max_abs_e, __shfl_xor_sync(0xffffffffu, max_abs_e, o));
        if (lane == 0) s_red[warp] = max_abs_e;
        __syncthreads();
        if (tid == 0) {
            double v = 0.0;
            for (int w = 0; w < TILED_THREADS / 32; ++w) v = fmax(v, s_red[w]);
            if (v > 0.0) atomic_max_nonneg_double(p.max_abs_e, v);
        }
    }
}

#undef VIEW

// ---------------------------------------------------------------------------------------------
static size_t pad256(size_t x) { return (x + 255) / 256 * 256; }

struct TiledLayout {
    int ntm, ntn;
    size_t q_off, flags_off, quad_off, qdep_off, qprog_off, rowdone_off, e_off, c_off, total;
};
static TiledLayout tiled_layout(int m, int n) {
    TiledLayout l;
    l.ntm = (m + T - 1) / T;
    l.ntn = (n + T - 1) / T;
    size_t tiles = (size_t)l.ntm * l.ntn;
    size_t mat = (size_t)l.ntm * T * (size_t)l.ntn * T * sizeof(double);
    l.q_off = 256;
    l.flags_off = l.q_off + 4096 * sizeof(unsigned);
    l.quad_off = l.flags_off + pad256(tiles * sizeof(unsigned));
    l.qdep_off = l.quad_off + pad256(tiles * sizeof(unsigned));
    l.qprog_off = l.qdep_off + pad256(4 * tiles * sizeof(unsigned));
    l.rowdone_off = l.qprog_off + pad256(4 * tiles * sizeof(unsigned));
    l.e_off = l.rowdone_off + pad256((size_t)l.ntm * sizeof(unsigned));
    l.c_off = l.e_off + pad256(mat);
    l.total = l.c_off + pad256(mat);
    return l;
}

size_t round_tiled_workspace_bytes(int m, int n) { return tiled_layout(m, n).total; }

// the same layout for the sixteen-warp kernel (round_fused.cu), which shares the workspace format
struct TiledLayoutView {
    int ntm, ntn;
    size_t q_off, flags_off, quad_off, qdep_off, qprog_off, rowdone_off, e_off, c_off, total;
};
TiledLayoutView round_tiled_layout_view(int m, int n) {
    const TiledLayout l = tiled_layout(m, n);
    return TiledLayoutView{l.ntm, l.ntn, l.q_off, l.flags_off, l.quad_off, l.qdep_off, l.qprog_off, l.rowdone_off,
                           l.e_off, l.c_off, l.total};
}
int launch_round_fused(const TiledParams &in, void *ws, size_t ws_bytes, cudaStream_t stream, bool force);
unsigned *round_tiled_rowdone(void *ws, int m, int n) {
    return reinterpret_cast<unsigned *>(static_cast<char *>(ws) + tiled_layout(m, n).rowdone_off);
}

int launch_round_tiled(const TiledParams &in, void *ws, size_t ws_bytes, cudaStream_t stream) {
    TiledLayout l = tiled_layout(in.m, in.n);
    if (ws_bytes < l.total) return GPTQ2D_ERR_WORKSPACE;
    {
        // large resident problems: far contractions and quadrant tasks side by side on every SM
        const int st = launch_round_fused(in, ws, ws_bytes, stream, false);
        if (st != -1) return st;
    }
    char *w = static_cast<char *>(ws);
    TiledKernelParams p{};
    p.m = in.m; p.n = in.n; p.ntm = l.ntm; p.ntn = l.ntn;
    p.ntasks = 2 * l.ntm * l.ntn;
    p.ntiles_total = l.ntm * l.ntn;
    p.batch_index = -1;
    p.np = (long)l.ntn * T;
    p.X = in.X; p.ldx = in.ldx; p.L = in.L; p.ldl = in.ldl; p.U = in.U; p.ldu = in.ldu;
    p.Z = in.Z; p.ldz = in.ldz; p.Euser = in.E; p.lde = in.lde;
    p.counter = reinterpret_cast<unsigned *>(w);
    p.abort = reinterpret_cast<unsigned *>(w) + 1;
    p.q_head = reinterpret_cast<unsigned *>(w) + 2;
    p.q_tail = reinterpret_cast<unsigned *>(w) + 3;
    p.tiles_done = reinterpret_cast<unsigned *>(w) + 4;
    p.q_slots = reinterpret_cast<unsigned *>(w + l.q_off);
    p.qmask = QCAP - 1;
    p.max_abs_e = workspace_max_abs_e(ws);
    p.flagS = reinterpret_cast<unsigned *>(w + l.flags_off);
    p.quad_done = reinterpret_cast<unsigned *>(w + l.quad_off);
    p.qdep = reinterpret_cast<unsigned *>(w + l.qdep_off);
    p.qprog = reinterpret_cast<unsigned *>(w + l.qprog_off);
    p.rowdone = reinterpret_cast<unsigned *>(w + l.rowdone_off);
    p.Ebuf = reinterpret_cast<double *>(w + l.e_off);
    p.Cbuf = reinterpret_cast<double *>(w + l.c_off);
    p.info = in.info;
    p.l_al16 = ((reinterpret_cast<uintptr_t>(in.L) & 15) == 0) && ((in.ldl & 1) == 0);
    p.u_al16 = ((reinterpret_cast<uintptr_t>(in.U) & 15) == 0) && ((in.ldu & 1) == 0);

    if (cudaMemsetAsync(w, 0, l.e_off, stream) != cudaSuccess) return GPTQ2D_ERR_CUDA;   // header, flags, counters
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return GPTQ2D_ERR_CUDA;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return GPTQ2D_ERR_CUDA;
    p.panels_ready = in.panels_ready;
    p.spin_limit = SPIN_LIMIT;
    p.panel_spin_limit = in.panel_spin_limit ? in.panel_spin_limit : SPIN_LIMIT;
    const void *kernel = in.panels_ready ? (const void *)round_tiled_kernel<false, true>
                                         : (const void *)round_tiled_kernel<false, false>;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)TILED_SMEM) != cudaSuccess)
        return GPTQ2D_ERR_CUDA;
    int grid = sms < p.ntasks ? sms : p.ntasks;
    void *args[] = {&p};
    if (cudaLaunchCooperativeKernel(kernel, dim3(grid), dim3(TILED_THREADS), args, TILED_SMEM, stream) != cudaSuccess)
        return GPTQ2D_ERR_CUDA;
    return GPTQ2D_OK;
}


// ---------------------------------------------------------------------------------------------
// Batched launch: every matrix keeps its own flags, counters and E / C buffers; claim counter,
// ready ring and abort word are shared.  Workspace: [header | ring | max|E| per matrix | flags of
// all matrices] (cleared per call) [descriptors | far-part table] (written per call from the
// host) [E, C buffers].
struct BatchedLayout {
    size_t maxe_off, flags_off, zero_end, desc_off, table_off, bufs_off, total;
    long ntasks, ntiles;
    unsigned qcap;
};
static BatchedLayout batched_layout(int count, const TiledParams *pr) {
    BatchedLayout l{};
    long ready_bound = 1;
    for (int b = 0; b < count; ++b) {
        TiledLayout t = tiled_layout(pr[b].m, pr[b].n);
        ready_bound += 2 * (t.ntm < t.ntn ? t.ntm : t.ntn);
    }
    l.qcap = QCAP;
    while ((long)l.qcap < 2 * ready_bound) l.qcap *= 2;     // twice the bound: slots are never close to reuse
    l.maxe_off = 256 + (size_t)l.qcap * sizeof(unsigned);
    l.flags_off = l.maxe_off + pad256((size_t)count * sizeof(double));
    size_t off = l.flags_off, bufs = 0;
    for (int b = 0; b < count; ++b) {
        TiledLayout t = tiled_layout(pr[b].m, pr[b].n);
        size_t tiles = (size_t)t.ntm * t.ntn;
        off += 2 * pad256(tiles * sizeof(unsigned)) + 2 * pad256(4 * tiles * sizeof(unsigned)) + pad256((size_t)t.ntm * sizeof(unsigned));
        bufs += 2 * pad256((size_t)t.ntm * T * (size_t)t.ntn * T * sizeof(double));
        l.ntiles += (long)tiles;
    }
    l.ntasks = 2 * l.ntiles;
    l.zero_end = off;
    l.desc_off = off;
    l.table_off = l.desc_off + pad256((size_t)count * sizeof(TiledKernelParams));
    l.bufs_off = l.table_off + pad256((size_t)l.ntasks * sizeof(unsigned));
    l.total = l.bufs_off + bufs;
    return l;
}

size_t round_tiled_batched_workspace_bytes(int count, const TiledParams *pr) { return batched_layout(count, pr).total; }

__global__ void batched_margin_kernel(const double *max_abs_e, double *min_margin, int count) {
    int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b < count) min_margin[b] = 0.5 - max_abs_e[b];
}

int launch_round_tiled_batched(int count, const TiledParams *pr, double *min_margin, int *info, void *ws,
                               size_t ws_bytes, cudaStream_t stream) {
    if (count < 1 || count > BATCH_MAX_COUNT) return GPTQ2D_ERR_INVALID_ARG;
    for (int b = 0; b < count; ++b)
        if (pr[b].m > BATCH_MAX_DIM || pr[b].n > BATCH_MAX_DIM) return GPTQ2D_ERR_TOO_LARGE;
    BatchedLayout l = batched_layout(count, pr);
    if (l.ntasks >= (1l << 31)) return GPTQ2D_ERR_TOO_LARGE;
    if (ws_bytes < l.total) return GPTQ2D_ERR_WORKSPACE;
    char *w = static_cast<char *>(ws);
    unsigned *hdr = reinterpret_cast<unsigned *>(w);

    // descriptors and the far-part table are built here and copied in one piece
    std::vector<unsigned char> stage(l.bufs_off - l.desc_off, 0);
    TiledKernelParams *desc = reinterpret_cast<TiledKernelParams *>(stage.data());
    unsigned *table = reinterpret_cast<unsigned *>(stage.data() + (l.table_off - l.desc_off));
    size_t foff = l.flags_off, boff = l.bufs_off;
    int max_waves = 0;
    for (int b = 0; b < count; ++b) {
        const TiledParams &in = pr[b];
        TiledLayout t = tiled_layout(in.m, in.n);
        size_t tiles = (size_t)t.ntm * t.ntn;
        size_t mat = pad256((size_t)t.ntm * T * (size_t)t.ntn * T * sizeof(double));
        TiledKernelParams d{};
        d.m = in.m; d.n = in.n; d.ntm = t.ntm; d.ntn = t.ntn;
        d.ntasks = (int)(2 * tiles);
        d.np = (long)t.ntn * T;
        d.X = in.X; d.ldx = in.ldx; d.L = in.L; d.ldl = in.ldl; d.U = in.U; d.ldu = in.ldu;
        d.Z = in.Z; d.ldz = in.ldz; d.Euser = in.E; d.lde = in.lde;
        d.counter = hdr; d.abort = hdr + 1; d.q_head = hdr + 2; d.q_tail = hdr + 3; d.tiles_done = hdr + 4;
        d.q_slots = reinterpret_cast<unsigned *>(w + 256);
        d.qmask = l.qcap - 1;
        d.flagS = reinterpret_cast<unsigned *>(w + foff); foff += pad256(tiles * sizeof(unsigned));
        d.quad_done = reinterpret_cast<unsigned *>(w + foff); foff += pad256(tiles * sizeof(unsigned));
        d.qdep = reinterpret_cast<unsigned *>(w + foff); foff += pad256(4 * tiles * sizeof(unsigned));
        d.qprog = reinterpret_cast<unsigned *>(w + foff); foff += pad256(4 * tiles * sizeof(unsigned));
        d.rowdone = reinterpret_cast<unsigned *>(w + foff); foff += pad256((size_t)t.ntm * sizeof(unsigned));
        d.Ebuf = reinterpret_cast<double *>(w + boff); boff += mat;
        d.Cbuf = reinterpret_cast<double *>(w + boff); boff += mat;
        d.max_abs_e = reinterpret_cast<double *>(w + l.maxe_off) + b;
        d.info = info;
        d.l_al16 = ((reinterpret_cast<uintptr_t>(in.L) & 15) == 0) && ((in.ldl & 1) == 0);
        d.u_al16 = ((reinterpret_cast<uintptr_t>(in.U) & 15) == 0) && ((in.ldu & 1) == 0);
        d.batch_index = b;
        d.spin_limit = d.panel_spin_limit = SPIN_LIMIT;
        d.ntiles_total = (int)tiles;
        desc[b] = d;
        if (t.ntm + t.ntn - 1 > max_waves) max_waves = t.ntm + t.ntn - 1;
    }
    // claim order: tile-wave by tile-wave over all matrices; inside a matrix' wave as decode_task lists them
    long nt = 0;
    for (int wv = 0; wv < max_waves; ++wv)
        for (int b = 0; b < count; ++b) {
            const int ntm = desc[b].ntm, ntn = desc[b].ntn;
            if (wv >= ntm + ntn - 1) continue;
            const int lo = wv - ntn + 1 > 0 ? wv - ntn + 1 : 0, hi = wv < ntm - 1 ? wv : ntm - 1;
            for (int k = 0; k <= hi - lo; ++k)
                for (int type = 0; type < 2; ++type) {
                    const int I = type == 0 ? hi - k : lo + k, J = wv - I;
                    table[nt++] = ((unsigned)b << 17) | ((unsigned)type << 16) | ((unsigned)I << 8) | (unsigned)J;
                }
        }
    if (nt != l.ntasks) return GPTQ2D_ERR_INVALID_ARG;

    TiledKernelParams p{};
    p.ntasks = (int)l.ntasks;
    p.ntiles_total = (int)l.ntiles;
    p.batch_index = -1;
    p.counter = hdr; p.abort = hdr + 1; p.q_head = hdr + 2; p.q_tail = hdr + 3; p.tiles_done = hdr + 4;
    p.q_slots = reinterpret_cast<unsigned *>(w + 256);
    p.qmask = l.qcap - 1;
    p.info = info;
    p.probs = reinterpret_cast<const TiledKernelParams *>(w + l.desc_off);
    p.far_tasks = reinterpret_cast<const unsigned *>(w + l.table_off);
    p.spin_limit = p.panel_spin_limit = SPIN_LIMIT;

    if (cudaMemsetAsync(w, 0, l.zero_end, stream) != cudaSuccess) return GPTQ2D_ERR_CUDA;
    // pageable source: the call returns once the bytes have left `stage`
    if (cudaMemcpyAsync(w + l.desc_off, stage.data(), stage.size(), cudaMemcpyHostToDevice, stream) != cudaSuccess)
        return GPTQ2D_ERR_CUDA;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return GPTQ2D_ERR_CUDA;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return GPTQ2D_ERR_CUDA;
    if (cudaFuncSetAttribute(round_tiled_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)TILED_SMEM) != cudaSuccess)
        return GPTQ2D_ERR_CUDA;
    int grid = (long)sms < l.ntasks ? sms : (int)l.ntasks;
    void *args[] = {&p};
    if (cudaLaunchCooperativeKernel((const void *)round_tiled_kernel<true, false>, dim3(grid), dim3(TILED_THREADS), args,
                                    TILED_SMEM, stream) != cudaSuccess)
        return GPTQ2D_ERR_CUDA;
    if (min_margin) {
        batched_margin_kernel<<<(count + 255) / 256, 256, 0, stream>>>(
            reinterpret_cast<const double *>(w + l.maxe_off), min_margin, count);
        if (cudaGetLastError() != cudaSuccess) return GPTQ2D_ERR_CUDA;
    }
    return GPTQ2D_OK;
}

}  // namespace gptq2d
