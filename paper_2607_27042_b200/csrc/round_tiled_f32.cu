// GPTQ-2D sweep in fp32 (the optional reduced-precision mode), tiled.
//
// X, L and U are rounded to fp32 and every operation of Algorithm 3 is carried out in fp32; the order of
// the sums is that of the tile restatement (Eq. 11, Eq. 15-17), not of the literal algorithm: for the
// 64 x 64 tile (I, J) with rows r and columns c
//     Cd = sum_{I' < I} L[r, I'] E[I', c]        Rt = sum_{J' < J} C[r, J'] U[J', c]
// and Algorithm 3 on the tile alone, started from Y = X[r, c] + Rt + Cd and C = Cd with the diagonal
// blocks L[r, r] and U[c, c], gives the tile's Z, E and C = L E.  fp32 has no tensor-core path that keeps
// fp32 operands exact (TF32 truncates them), so the two contractions are a register-tiled FFMA loop.
// The loop is bound by the shared-memory load pipe before the FMA pipe (a 16-byte load costs a warp four
// cycles of it and feeds four operand words per lane), so the register piece is as large as the register
// file allows: one CTA of 256 threads per SM, every WARP covers the whole 64 x 64 tile with a 16 x 8 piece
// per lane (six loads per 128 FMAs) and takes an eighth of every slab's depth; the eight partial tiles are
// added through shared memory when a contraction ends.  (History at 8192 x 8192: 4 x 4 pieces, two CTAs
// per SM, 30 % of the FMA pipe, 52.6 ms; 8 x 8 pieces in 512 threads 41.6 ms; 16 x 8 in 256 threads
// 38.7 ms.)  Both operands of a slab are stored depth-major ([k][64 rows] and [k][64 columns]: L and C are
// kept transposed in the workspace for this) and arrive through a four-stage ring of slabs of 64: by bulk
// tensor copies (TMA, one dense 64 x 64 box per operand and source, issued by one lane, counted by "full" /
// "empty" mbarriers, no CTA barrier in the multiply loop, ragged edges by the copy engine's zero fill) where
// the driver offers tensor maps, by cp.async with one CTA barrier per slab otherwise.
// A thread cannot hold two accumulators of that size, so a tile runs three contractions one after the other:
// Rt over the older tiles of its row, Cd over its whole column (the tile above comes last), Rt's last term
// from the tile to the left -- the newest sources still come last; finished sums wait in shared memory.
//
// One persistent, cooperatively launched grid, one CTA per SM.  Tiles are claimed wave by wave (I + J
// ascending) from one atomic counter; a CTA folds the source tiles in as their flags come up and then
// sweeps its tile.  A tile only waits for tiles of earlier waves, which were claimed earlier, so the
// earliest unfinished tile can always run.  (Two slower CTAs per SM, one multiplying while the other
// sweeps, lose: the tile above and the tile to the left are on every tile's critical path, and a CTA that
// shares its SM takes twice as long over them.)
//
// In-tile sweep: one anti-diagonal per step, one CTA barrier per step, in the implicit-Y (pull) form of
// Appendix B (Eq. 19-20): an entry reads the errors above it in its column through L and the finished C to
// its left in its row through U at the moment it is rounded, four lanes per row sharing the two dot
// products; all of both sums except their last terms is formed one step ahead.  Nothing is read-modify-
// written (an eager version that pushed every error down and right as Algorithm 3 prints it cost 7x the
// time per step: 2 x 64 x 64 shared-memory updates per anti-diagonal, issued by every warp).
#include <cstdio>
#include <cstring>
#include "common.cuh"
#include "dmma_gemm.cuh"          // cp.async helpers
#include "dmma_tma.cuh"           // mbarrier and bulk tensor copy helpers
#include "tma_host.cuh"
#include "round_internal.cuh"

namespace gptq2d {
namespace f32 {

constexpr int TS = 64;             // tile edge
constexpr int THREADS = 256;        // one CTA per SM
constexpr int KS = 64;             // slab depth
constexpr int SPS = TS / KS;       // slabs per source tile
constexpr int NSTAGE = 4;          // cp.async ring; it lives where the in-tile matrices go afterwards
constexpr int KGROUPS = THREADS / 32;   // one warp a group, each KS / KGROUPS deep in every slab
constexpr int KG = KS / KGROUPS;
constexpr int LDB = TS + 4;        // both slabs are [KS k][64], row stride 68 floats
constexpr int SLAB_FLOATS = KS * LDB, STAGE_FLOATS = 2 * SLAB_FLOATS;
constexpr int TMA_SLAB_FLOATS = KS * TS, TMA_STAGE_FLOATS = 2 * TMA_SLAB_FLOATS;     // dense boxes [KS k][64]
constexpr unsigned TMA_STAGE_BYTES = TMA_STAGE_FLOATS * sizeof(float);
constexpr int TMA_PREF = 2;        // slabs in flight ahead of the one being multiplied (one stage of slack for the slowest warp)
constexpr int PMAT = TS * LDB;     // a group's partial tile, staged with the slabs' row stride
constexpr int RPT = TS * TS / 4 / THREADS;   // float4 pieces of a tile per thread (rows (t >> 4) + (THREADS / 16) h)
constexpr int LDT = TS + 16;       // in-tile matrices, row stride 80 floats = 16 banks mod 32: the two rows x four lanes of a quarter-warp
                                   // read eight different 16-byte columns of two neighbouring rows without a bank conflict
constexpr int TMAT = TS * LDT;
constexpr int SWEEP_FLOATS = 4 * TMAT + TS * TS, RING_FLOATS = NSTAGE * STAGE_FLOATS;      // + the tile's Z (int32)
constexpr int PARK_FLOATS = 2 * TS * TS;      // finished partial sums (Rt of the older tiles, Cd) wait behind the ring
constexpr int SMEM_FLOATS = RING_FLOATS + PARK_FLOATS > SWEEP_FLOATS ? RING_FLOATS + PARK_FLOATS : SWEEP_FLOATS;
static_assert(KGROUPS * PMAT <= RING_FLOATS, "the four partial tiles are added through the drained ring");
constexpr size_t SMEM_BYTES = (size_t)SMEM_FLOATS * sizeof(float);

struct Params {
    int m, n, nti, ntj, ntiles;
    long mp, np;                   // padded extents (multiples of 64): leading dimension of E32 / C32 is np
    const double *X; long ldx;
    int *Z; long ldz;
    double *Euser; long lde;
    const float *L32t; long ldl;   // L transposed, m x m: L32t[k][r] = L[r, k] (leading dimension padded to a multiple of 4)
    const float *U32; long ldu;
    float *E32, *C32t;             // E: mp x np (leading dimension np); C transposed: np x mp (leading dimension mp)
    unsigned *counter, *abort, *flags;
    double *max_abs_e;
    int *info;
    unsigned long long spin_limit;
    int use_tma;                   // slabs by bulk tensor copies (tensor maps are separate kernel parameters)
    int pad_;
};

__device__ __forceinline__ void cp_async16f(float *smem, const float *gmem, int src_bytes) {
    unsigned s = (unsigned)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(s), "l"(gmem), "r"(src_bytes) : "memory");
}

// tile index in claim order -> (I, J): wave by wave, I ascending inside a wave
__device__ __forceinline__ void decode_tile(int task, int nti, int ntj, int &I, int &J) {
    int tt = task;
    for (int w = 0; w < nti + ntj - 1; ++w) {
        const int lo = max(0, w - ntj + 1), hi = min(nti - 1, w);
        const int cnt = hi - lo + 1;
        if (tt < cnt) { I = lo + tt; J = w - I; return; }
        tt -= cnt;
    }
    I = J = 0;
}

// One source tile: acc += A^T B with A (64 k x 64 rows, [k][row], leading dimension lda) and B (64 k x 64 columns,
// [k][col], ldb), both fully inside padded or zero-filled storage except that rows of the tile beyond `a_rows`, columns
// beyond `b_cols` and depths beyond `kmax` (ragged edge of a user matrix) are read as zeros.  K is streamed in SPS slabs.
struct Gemm {
    float *stages;
    int tid, gk, ty, tx;           // group (quarter of the depth), position in the group's 8 x 8 thread grid
    // copy plan: each slab is KS k x 64 entries in chunks of 4 floats, KS * 16 / THREADS chunks of each slab per thread
    __device__ __forceinline__ void issue_one(float *S, const float *P, long ld, int valid, int kmax, int k0) const {
        constexpr int RPH = THREADS / 16;                            // slab rows covered by one round of the CTA
        const int kr0 = tid >> 4, cc = (tid & 15) * 4;
        if (valid >= TS && kmax - k0 >= KS) {                        // interior slab: nothing to clip (uniform over the CTA)
            float *sdst = S + kr0 * LDB + cc;
            const float *g = P + (long)(k0 + kr0) * ld + cc;
#pragma unroll
            for (int h = 0; h < KS / RPH; ++h) cp_async16(sdst + h * RPH * LDB, g + (long)h * RPH * ld, 16);
            return;
        }
#pragma unroll
        for (int h = 0; h < KS / RPH; ++h) {
            const int kr = kr0 + h * RPH;
            int nv = (k0 + kr < kmax) ? valid - cc : 0;              // floats valid from cc on
            nv = nv < 0 ? 0 : (nv > 4 ? 4 : nv);
            cp_async16f(S + kr * LDB + cc, nv ? P + (long)(k0 + kr) * ld + cc : P, nv * 4);
        }
    }
    __device__ __forceinline__ void issue(int stage, const float *A, long lda, int a_rows, const float *B, long ldb, int b_cols,
                                          int kmax, int k0) const {
        float *As = stages + stage * STAGE_FLOATS;
        issue_one(As, A, lda, a_rows, kmax, k0);
        issue_one(As + SLAB_FLOATS, B, ldb, b_cols, kmax, k0);
    }
    // the thread's piece: rows 4 ty + (i & 3) + 16 (i >> 2), i < 16; columns 4 tx + (j & 3) + 32 (j >> 2), j < 8
    template <int LD, int SLAB>
    __device__ __forceinline__ void multiply(float (&acc)[16][8], const float *stage) const {
        const float *As = stage + gk * KG * LD, *Bs = As + SLAB;
#pragma unroll
        for (int k = 0; k < KG; ++k) {
            float av[16], bv[8];
#pragma unroll
            for (int h = 0; h < 4; ++h) {
                const float4 a = *reinterpret_cast<const float4 *>(As + k * LD + 16 * h + 4 * ty);
                av[4 * h + 0] = a.x; av[4 * h + 1] = a.y; av[4 * h + 2] = a.z; av[4 * h + 3] = a.w;
            }
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const float4 b = *reinterpret_cast<const float4 *>(Bs + k * LD + 32 * h + 4 * tx);
                bv[4 * h + 0] = b.x; bv[4 * h + 1] = b.y; bv[4 * h + 2] = b.z; bv[4 * h + 3] = b.w;
            }
#pragma unroll
            for (int i = 0; i < 16; ++i)
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
        }
    }
    // the group's partial tile to shared memory (row stride LDB)
    __device__ __forceinline__ void stage_partial(const float (&acc)[16][8]) const {
        float *P = stages + gk * PMAT;
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            float *row = P + (4 * ty + (i & 3) + 16 * (i >> 2)) * LDB + 4 * tx;
            *reinterpret_cast<float4 *>(row) = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
            *reinterpret_cast<float4 *>(row + 32) = make_float4(acc[i][4], acc[i][5], acc[i][6], acc[i][7]);
        }
    }
};

__global__ void __launch_bounds__(THREADS, 1)
round_tiled_f32_kernel(Params p, const __grid_constant__ CUtensorMap mapL, const __grid_constant__ CUtensorMap mapE,
                       const __grid_constant__ CUtensorMap mapC, const __grid_constant__ CUtensorMap mapU) {
    extern __shared__ __align__(128) float smem[];
    __shared__ __align__(8) unsigned long long s_full[NSTAGE], s_empty[NSTAGE];
    __shared__ int s_fail, s_issued;
    __shared__ int s_task;
    __shared__ int s_ok, s_upto;
    __shared__ double s_red[THREADS / 32];
    __shared__ unsigned long long s_badkey;
    float *stages = smem;
    // the contraction's accumulators are registers, so the in-tile matrices reuse the ring's memory
    // Udt[j][j'] = U[j', j] (the diagonal block of U transposed, strictly lower, first sub-diagonal apart in s_usub),
    // Et[j][i'] = E[i', j] (transposed copy of the errors): the rows the dot products of the sweep run along.  The
    // diagonal block of L lives in registers (a lane keeps its quarter of its row).
    float *Ys = smem, *Cs = Ys + TMAT, *Udt = Cs + TMAT, *Et = Udt + TMAT;
    int *Zs = reinterpret_cast<int *>(Et + TMAT);  // [64][64]: rounded values, written out row-wise after the sweep
    __shared__ float s_usub[TS];                   // U[j - 1, j] of the diagonal block
    const int tid = threadIdx.x;
    Gemm gm{stages, tid, tid >> 5, (tid & 31) >> 3, tid & 7};
    float *park_rt = smem + RING_FLOATS, *park_cd = park_rt + TS * TS;     // [64][64] each, behind the ring
    double max_abs_e = 0.0;
    if (tid == 0) {
        s_badkey = ~0ull;
        s_fail = 0;
        if (p.use_tma) {
            for (int i = 0; i < NSTAGE; ++i) { mbar_init(&s_full[i], 1u); mbar_init(&s_empty[i], (unsigned)KGROUPS); }
            mbar_init_fence();
        }
    }
    unsigned ring_it = 0;          // slabs that went through the TMA ring so far (the same in every thread)
#ifdef TILED_STATS
    long long sw_sums = 0, sw_round = 0, sw_bar = 0;
    long long st_claim = 0, st_gemm = 0, st_form = 0, st_sweep = 0, st_store = 0, st_wait = 0, st_n = 0, st_t = clock64();
#define F32_MARK(x) do { const long long now_ = clock64(); x += now_ - st_t; st_t = now_; } while (0)
#else
#define F32_MARK(x)
#endif

    for (;;) {
        __syncthreads();
        if (tid == 0) {
            int task = -1;
            if (ld_relaxed_u32(p.abort) == 0u) {
                task = (int)atomicAdd(p.counter, 1u);
                if (task >= p.ntiles) task = -1;
            }
            s_task = task;
        }
        __syncthreads();
        const int task = s_task;
        if (task < 0) break;
        int I, J;
        decode_tile(task, p.nti, p.ntj, I, J);
        const int row0 = I * TS, col0 = J * TS;
        F32_MARK(st_claim);

        // ---- 1. the contractions, one accumulator at a time: Rt over the older tiles of the row (I, 0..J-2) through U,
        // parked in shared memory; Cd over the column (0..I-1, J) through L (the tile above, still being swept when this
        // tile is claimed, is its last source); Rt's last term from the tile to the left.
        float acc[16][8];
        bool ok = true;
        struct Src { const float *A, *B; long lda, ldb; int a_rows, b_cols, kmax; const unsigned *flag; };
        auto source = [&](int dir, int k) {
            Src r;
            if (dir == 0) {          // L[r, rows of tile k] * E[rows of tile k, c]
                r.A = p.L32t + (long)k * TS * p.ldl + row0; r.lda = p.ldl; r.a_rows = min(TS, p.m - row0);
                r.B = p.E32 + (long)k * TS * p.np + col0; r.ldb = p.np; r.b_cols = TS;
                r.kmax = min(TS, p.m - k * TS);
                r.flag = p.flags + (long)k * p.ntj + J;
            } else {                 // C[r, columns of tile k] * U[columns of tile k, c]
                r.A = p.C32t + (long)k * TS * p.mp + row0; r.lda = p.mp; r.a_rows = TS;
                r.B = p.U32 + (long)k * TS * p.ldu + col0; r.ldb = p.ldu; r.b_cols = min(TS, p.n - col0);
                r.kmax = min(TS, p.n - k * TS);
                r.flag = p.flags + (long)I * p.ntj + k;
            }
            return r;
        };
        // One contraction: acc = sum over the sources k0 .. k1-1 of direction dir.  Sources [k0, ready_upto) are known to
        // be swept.  The list is scanned by the whole CTA at once (one flag per thread, the first unset position by a
        // shared-memory minimum), so that a tile whose far sources are all done -- the usual case -- pays two barriers
        // for the lot instead of a global round trip per source; only when the next source in line is still being swept
        // does one thread wait for it, bounded.  Returns with the ring drained.
        auto contract = [&](int dir, int k0, int k1) {
#pragma unroll
            for (int i = 0; i < 16; ++i)
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;
            const int nslab = (k1 - k0) * SPS;
            int ready_upto = k0;
            auto scan_ready = [&](int from) -> bool {         // all threads; false if the bounded wait ran out
#ifdef TILED_STATS
                const long long w0_ = clock64();
#endif
                if (tid == 0) {
                    unsigned long long it = 0;
                    int good = 1;
                    const Src sr = source(dir, from);
                    while (ld_acquire_u32(sr.flag) == 0u) {
                        if (++it > p.spin_limit || ld_relaxed_u32(p.abort) != 0u) {
                            report(p.info, GPTQ2D_ERR_DEVICE_TIMEOUT, -9, task, (int)blockIdx.x);
                            atomicExch(p.abort, 1u);
                            good = 0;
                            break;
                        }
                        __nanosleep(100);
                    }
                    s_ok = good;
                    s_upto = k1;
                }
                __syncthreads();
                for (int k = from + 1 + tid; k < k1; k += THREADS)
                    if (ld_acquire_u32(source(dir, k).flag) == 0u) atomicMin(&s_upto, k);
                __syncthreads();
                const bool good = s_ok != 0;
                ready_upto = s_upto;
                __syncthreads();                              // s_ok / s_upto may be rewritten by the next scan
#ifdef TILED_STATS
                st_wait += clock64() - w0_;
#endif
                return good;
            };
            auto issue_slab = [&](int g) -> bool {            // all threads; false if a wait ran out
                const int k = k0 + g / SPS;
                if (k >= ready_upto && !scan_ready(k)) return false;
                const Src sr = source(dir, k);
                gm.issue(g % NSTAGE, sr.A, sr.lda, sr.a_rows, sr.B, sr.ldb, sr.b_cols, sr.kmax, (g % SPS) * KS);
                return true;
            };
            for (int g = 0; g < NSTAGE - 1 && ok; ++g) {
                if (g < nslab) ok = issue_slab(g);
                cp_async_commit();
            }
            for (int g = 0; g < nslab && ok; ++g) {
                cp_async_wait<NSTAGE - 2>();
                __syncthreads();                           // slab g has landed; everyone is past slab g - 1, whose stage is free
                if (g + NSTAGE - 1 < nslab) ok = issue_slab(g + NSTAGE - 1);
                cp_async_commit();
                if (!ok) break;
                gm.multiply<LDB, SLAB_FLOATS>(acc, stages + (g % NSTAGE) * STAGE_FLOATS);
            }
            cp_async_wait<0>();
            __syncthreads();
        };
        // The same contraction with the slabs brought in by the copy engine: one bulk tensor copy per operand and
        // source (a dense 64 x 64 box; what lies outside the matrix reads as zeros), completion counted by a "full"
        // mbarrier per stage, the stage handed back through an "empty" mbarrier on which each warp arrives once.  No
        // copy instruction, no address arithmetic and no CTA barrier sits in the multiply loop; the warps drift apart
        // by up to a stage.  Warp 0 is also the producer: it checks the flags of the sources 32 at a time and its lane 0
        // issues slab g + 2 before the warp multiplies slab g.  Every wait is bounded; one that runs out raises the abort
        // word, and the pass then waits (bounded) for the copies still in flight before anyone leaves.
        auto contract_tma = [&](int dir, int k0, int k1) {
#pragma unroll
            for (int i = 0; i < 16; ++i)
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;
            const int nslab = k1 - k0, lane = tid & 31;
            const bool producer_warp = tid < 32;
            const CUtensorMap *ma = dir == 0 ? &mapL : &mapC, *mb = dir == 0 ? &mapE : &mapU;
            const int xa = row0, xb = col0;
            int ready_upto = k0;
            if (tid == 0) s_issued = 0;
            bool good = true;
            if (tid == 0) fence_proxy_async();           // the ring's memory was last touched by ordinary loads and stores
            auto produce = [&](int q) {                  // warp 0, all lanes: slab q of this pass
                const int k = k0 + q;
                if (k >= ready_upto) {                   // flags of the next 32 sources in line, one per lane
                    unsigned long long spins = 0;
                    while (k >= ready_upto && good) {
                        const int kk = ready_upto + lane;
                        const unsigned *fl = dir == 0 ? p.flags + (long)kk * p.ntj + J : p.flags + (long)I * p.ntj + kk;
                        const bool rdy = kk < k1 && ld_acquire_u32(fl) != 0u;
                        const unsigned got = __ballot_sync(0xffffffffu, rdy);
                        const int lead = got == 0xffffffffu ? 32 : __ffs(~got) - 1;
                        ready_upto += lead;
                        if (lead == 0) {
                            if (++spins > p.spin_limit || ld_relaxed_u32(p.abort) != 0u) {
                                if (lane == 0) {
                                    report(p.info, GPTQ2D_ERR_DEVICE_TIMEOUT, -9, task, (int)blockIdx.x);
                                    atomicExch(p.abort, 1u);
                                }
                                good = false;
                            }
                            __nanosleep(100);
                        }
                    }
                    __syncwarp();                        // the lanes' acquires come before lane 0's copies
                    if (lane == 0) fence_proxy_async();
                }
                if (!good) return;
                if (lane == 0) {
                    const unsigned it = ring_it + (unsigned)q;
                    const int st = (int)(it % NSTAGE);
                    if (it >= (unsigned)NSTAGE && !mbar_wait(&s_empty[st], ((it / NSTAGE) - 1u) & 1u, p.abort)) {
                        report(p.info, GPTQ2D_ERR_DEVICE_TIMEOUT, -10, task, (int)blockIdx.x);
                        atomicExch(p.abort, 1u);            // (the consumers' waits watch the abort word)
                    } else {
                        float *dst = stages + st * TMA_STAGE_FLOATS;
                        mbar_arrive_expect_tx(&s_full[st], TMA_STAGE_BYTES);
                        tma_load_2d(dst, ma, xa, k * TS, &s_full[st]);
                        tma_load_2d(dst + TMA_SLAB_FLOATS, mb, xb, k * TS, &s_full[st]);
                        s_issued = q + 1;
                    }
                }
                __syncwarp();        // lane 0 rejoins the warp here, not somewhere inside the multiply that follows
            };
            if (producer_warp)
                for (int q = 0; q < TMA_PREF && q < nslab && good; ++q) produce(q);
            int g = 0;
            for (; g < nslab && good; ++g) {
                if (producer_warp && g + TMA_PREF < nslab) produce(g + TMA_PREF);
                if (!good) break;
                const unsigned it = ring_it + (unsigned)g;
                const int st = (int)(it % NSTAGE);
                if (!mbar_wait(&s_full[st], (it / NSTAGE) & 1u, p.abort)) {
                    if (lane == 0) {
                        report(p.info, GPTQ2D_ERR_DEVICE_TIMEOUT, -11, task, (int)blockIdx.x);
                        atomicExch(p.abort, 1u);
                    }
                    good = false;
                    break;
                }
                gm.multiply<TS, TMA_SLAB_FLOATS>(acc, stages + st * TMA_STAGE_FLOATS);
                __syncwarp();
                if (lane == 0) mbar_arrive(&s_empty[st]);
            }
            if (!good) {
                s_fail = 1;
                // copies of this pass that may still be in flight: wait for them (bounded) before the memory is reused or left
                if (tid == 0)
                    for (int q = g; q < s_issued; ++q) {
                        const unsigned it = ring_it + (unsigned)q;
                        mbar_wait(&s_full[it % NSTAGE], (it / NSTAGE) & 1u, nullptr);
                    }
            }
            ring_it += (unsigned)nslab;
            __syncthreads();
            if (s_fail) ok = false;
        };
        // Sum of the groups' partial tiles; thread t gets rows (t >> 4) + (THREADS / 16) h, columns 4 (t & 15) .. + 3.  The ring
        // is drained on entry and free again on return.
        auto reduce = [&](float4 (&v)[RPT]) {
            gm.stage_partial(acc);
            __syncthreads();
#pragma unroll
            for (int h = 0; h < RPT; ++h) {
                const float *q = stages + ((tid >> 4) + (THREADS / 16) * h) * LDB + 4 * (tid & 15);
                float4 a = *reinterpret_cast<const float4 *>(q);
#pragma unroll
                for (int g = 1; g < KGROUPS; ++g) {
                    const float4 b = *reinterpret_cast<const float4 *>(q + g * PMAT);
                    a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w;
                }
                v[h] = a;
            }
            __syncthreads();
        };
        // A finished sum waits in shared memory while the next contraction runs; a thread reads back what it wrote itself.
        const int own = (tid >> 4) * TS + 4 * (tid & 15);        // + (THREADS / 16) h rows
        constexpr int OWN_STEP = (THREADS / 16) * TS;
        float4 v4[RPT];
        const bool far_rt = J > 1;
        if (far_rt) {
            if (p.use_tma) contract_tma(1, 0, J - 1); else contract(1, 0, J - 1);
            if (!ok) break;
            reduce(v4);
#pragma unroll
            for (int h = 0; h < RPT; ++h) *reinterpret_cast<float4 *>(park_rt + own + h * OWN_STEP) = v4[h];
        }
        if (I > 0) {
            if (p.use_tma) contract_tma(0, 0, I); else contract(0, 0, I);
            if (!ok) break;
            reduce(v4);
#pragma unroll
            for (int h = 0; h < RPT; ++h) *reinterpret_cast<float4 *>(park_cd + own + h * OWN_STEP) = v4[h];
        }
        if (J > 0) {
            if (p.use_tma) contract_tma(1, J - 1, J); else contract(1, J - 1, J);
            if (!ok) break;
            reduce(v4);
        }
        float4 cdv[RPT], rtv[RPT];
#pragma unroll
        for (int h = 0; h < RPT; ++h) {
            const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
            rtv[h] = J > 0 ? v4[h] : zero;
            if (far_rt) {
                const float4 q = *reinterpret_cast<const float4 *>(park_rt + own + h * OWN_STEP);
                rtv[h] = make_float4(q.x + rtv[h].x, q.y + rtv[h].y, q.z + rtv[h].z, q.w + rtv[h].w);
            }
            cdv[h] = I > 0 ? *reinterpret_cast<const float4 *>(park_cd + own + h * OWN_STEP) : zero;
        }
        __syncthreads();                    // the in-tile matrices overlap the parked sums
        F32_MARK(st_gemm);

        // ---- 2. Y = X + Rt + Cd, C = Cd; the diagonal block of U (strictly upper, kept transposed; its first
        // super-diagonal U[j-1, j] apart, see below)
        {
#pragma unroll
            for (int h = 0; h < RPT; ++h) {
                const int r = (tid >> 4) + (THREADS / 16) * h, c = 4 * (tid & 15), gr = row0 + r, gc = col0 + c;
                const float rt4[4] = {rtv[h].x, rtv[h].y, rtv[h].z, rtv[h].w}, cd4[4] = {cdv[h].x, cdv[h].y, cdv[h].z, cdv[h].w};
                float y4[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float x = (gr < p.m && gc + j < p.n) ? (float)__ldg(p.X + (long)gr * p.ldx + gc + j) : 0.f;
                    y4[j] = (x + rt4[j]) + cd4[j];
                }
                *reinterpret_cast<float4 *>(Cs + r * LDT + c) = cdv[h];
                *reinterpret_cast<float4 *>(Ys + r * LDT + c) = make_float4(y4[0], y4[1], y4[2], y4[3]);
                // unrounded entries count as zero (they meet zero coefficients)
                *reinterpret_cast<float4 *>(Et + r * LDT + c) = make_float4(0.f, 0.f, 0.f, 0.f);
            }
            if (tid == 0) s_usub[0] = 0.f;
#pragma unroll 8
            for (int e = tid; e < TS * TS; e += THREADS) {
                const int a = e >> 6, b = e & 63;              // U block entry (row a, column b), b along the contiguous direction
                const int ur = col0 + a, uc = col0 + b;
                const float v = (b > a && uc < p.n) ? p.U32[(long)ur * p.ldu + uc] : 0.f;
                Udt[b * LDT + a] = (b == a + 1) ? 0.f : v;
                if (b == a + 1) s_usub[b] = v;
            }
        }
        __syncthreads();
        F32_MARK(st_form);

        // ---- 3. the tile's 127 anti-diagonals, in the implicit-Y (pull) form of Appendix B, Eq. 19-20, which gives
        // the same entries as Algorithm 3: entry (i, j) reconstructs its corrected value when it is rounded,
        //     Y_ij = Y0_ij + sum_{i' < i} L[i, i'] E[i', j] + sum_{j' < j} C[i, j'] U[j', j],
        // and its final C_ij = C0_ij + sum_{i' < i} L[i, i'] E[i', j] + E_ij is stored once.  Four lanes per row.  Of the
        // two sums only the last terms, E[i-1, j] and C[i, j-1], come from the anti-diagonal just before; everything else
        // was rounded at least two steps ago.  So a step is split: all four lanes form the sums WITHOUT their last terms for
        // the row's NEXT entry (dot products along rows of shared memory, whose coefficients at and beyond the last
        // term are stored as zeros: what they meet there -- zeros, unrounded values, or an entry being written
        // this very step -- is finite and drops out), and the row's first lane rounds the CURRENT entry from the sums
        // formed one step earlier plus the two last terms: one shared-memory load (E[i-1, j]; C[i, j-1] is its own
        // previous result), one FMA, the rounding.  The two parts are independent, so the long one runs in the shadow of
        // the dependent one; the CTA barrier per anti-diagonal stays.
        // Ys holds Y0 until an entry is rounded and E afterwards; Cs holds C0 and then C.
        {
            const int row = tid >> 2, sub = tid & 3;
            const bool row_in = row0 + row < p.m;
            // the lane's quarter of row `row` of the diagonal block of L: columns 4 (sub + 4 t) .. + 3, strictly lower,
            // the first sub-diagonal entry L[i, i-1] apart
            float lr[16];
#pragma unroll
            for (int t = 0; t < 4; ++t)
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int ip = 4 * (sub + 4 * t) + e;
                    lr[4 * t + e] = (ip < row - 1 && row_in) ? __ldg(p.L32t + (long)(row0 + ip) * p.ldl + row0 + row) : 0.f;
                }
            const float lsub = (row > 0 && row_in) ? __ldg(p.L32t + (long)(row0 + row - 1) * p.ldl + row0 + row) : 0.f;
            const float4 *c4 = reinterpret_cast<const float4 *>(Cs + row * LDT) + sub;
            const int w8 = (tid >> 5) * 8;                           // the warp's first row
            const int tl = (w8 + 6 + 15) >> 4;                       // chunks of 16 rows that hold a source i' < row - 1 of the warp's last row
            float *yrow = Ys + row * LDT, *crow = Cs + row * LDT;
            unsigned long long badkey = ~0ull;
            float max_e = 0.f;
            float base_y = 0.f, base_c = 0.f, c_last = 0.f;      // (first lane of the row)
#ifdef TILED_STATS
            long long sw_t = clock64();
#define SW_MARK(x) do { const long long n_ = clock64(); x += n_ - sw_t; sw_t = n_; } while (0)
#else
#define SW_MARK(x)
#endif
            for (int s = -1; s < 2 * TS - 1; ++s) {
                const int j = s - row, jn = j + 1;                        // the row's current and next entry
                const bool cur_in = j >= 0 && j < TS, next_in = jn >= 0 && jn < TS;
                // (loads first: what is stored further down cannot overtake them)
                float e_up = 0.f, y0n = 0.f, c0n = 0.f, usubn = 0.f;
                if (sub == 0) {
                    if (cur_in && row > 0) e_up = Et[j * LDT + row - 1];
                    if (next_in) { y0n = yrow[jn]; c0n = crow[jn]; usubn = s_usub[jn]; }
                }
                // Sums for the next entry, without their last terms.  Whole warps skip the step while none of their rows
                // has a next entry; inside, every lane goes through the same loads and shuffles (rows of a warp differ in
                // whether and how far they need them; a shuffle under a per-row mask would split the warp): the trip counts
                // are those of the warp's longest row, and a chunk that holds no source of a shorter row meets zero
                // coefficients.  The step is bound by the shared-memory load pipe (a 16-byte load costs a warp four to six
                // cycles however many lanes use it; whole rows for all 64 rows are 96 loads a step), which is why chunks
                // that hold no source are skipped by whole warps and the row of L stays in registers.
                float sl = 0.f, su = 0.f;
                const int jn_hi = s + 1 - w8;                            // next column of the warp's first row (the largest)
                if (jn_hi >= 0 && jn_hi - 7 < TS) {
                    const int jr = next_in ? jn : 0;
                    const float4 *e4 = reinterpret_cast<const float4 *>(Et + jr * LDT) + sub, *u4 = reinterpret_cast<const float4 *>(Udt + jr * LDT) + sub;
                    const int tu = min(4, (jn_hi + 14) >> 4);            // chunks of 16 columns that hold a source j' < jn - 1
                    float dl[2] = {0.f, 0.f}, du[2] = {0.f, 0.f};
#pragma unroll
                    for (int t = 0; t < 4; ++t) {                        // down the column: sources i' < row - 1
                        if (t < tl) {
                            const float4 b = e4[4 * t];
                            dl[0] = fmaf(lr[4 * t + 0], b.x, dl[0]); dl[1] = fmaf(lr[4 * t + 1], b.y, dl[1]);
                            dl[0] = fmaf(lr[4 * t + 2], b.z, dl[0]); dl[1] = fmaf(lr[4 * t + 3], b.w, dl[1]);
                        }
                    }
#pragma unroll
                    for (int t = 0; t < 4; ++t) {                        // along the row: sources j' < jn - 1
                        if (t < tu) {
                            const float4 a = c4[4 * t], b = u4[4 * t];
                            du[0] = fmaf(a.x, b.x, du[0]); du[1] = fmaf(a.y, b.y, du[1]);
                            du[0] = fmaf(a.z, b.z, du[0]); du[1] = fmaf(a.w, b.w, du[1]);
                        }
                    }
                    sl = dl[0] + dl[1]; su = du[0] + du[1];
                    sl += __shfl_xor_sync(0xffffffffu, sl, 1);
                    su += __shfl_xor_sync(0xffffffffu, su, 1);
                    sl += __shfl_xor_sync(0xffffffffu, sl, 2);
                    su += __shfl_xor_sync(0xffffffffu, su, 2);
                }
                SW_MARK(sw_sums);
                if (sub == 0) {
                    if (cur_in) {
                        const float t = lsub * e_up;                     // (lsub = 0 in row 0)
                        const float y = base_y + t;
                        const float z = rintf(y);
                        const float e = z - y;                           // E = Z - Y
                        c_last = (base_c + t) + e;                       // C = L E (unit diagonal)
                        crow[j] = c_last;
                        yrow[j] = e;
                        Et[j * LDT + row] = e;
                        int zi = (int)z;
                        if (!(fabsf(y) < 2147483648.f)) {
                            const int gr = row0 + row, gc = col0 + j;
                            const unsigned long long key = ((unsigned long long)(gr + gc) << 42) | ((isfinite(y) ? 1ull : 0ull) << 41) |
                                                           ((unsigned long long)gr << 20) | (unsigned long long)gc;
                            if (gr < p.m && gc < p.n && key < badkey) badkey = key;
                            zi = 0;
                        }
                        Zs[row * TS + j] = zi;
                        max_e = fmaxf(max_e, fabsf(e));
                    }
                    if (next_in) {
                        base_c = c0n + sl;
                        base_y = fmaf(c_last, usubn, (y0n + su) + sl);   // c_last: C[i, jn - 1], rounded just above
                    }
                }
                SW_MARK(sw_round);
                __syncthreads();
                SW_MARK(sw_bar);
            }
            max_abs_e = fmax(max_abs_e, (double)max_e);      // (entries outside the matrix are exact zeros with E = 0)
            if (badkey != ~0ull) atomicMin(&s_badkey, badkey);
        }
        F32_MARK(st_sweep);

        // ---- 4. results of the tile: Z (and the caller's E) to the outputs, E and C to the workspace, then the flag
        for (int e = tid; e < TS * TS; e += THREADS) {
            const int r = e >> 6, c = e & 63;
            const int gr = row0 + r, gc = col0 + c;
            if (gr < p.m && gc < p.n) {
                p.Z[(long)gr * p.ldz + gc] = Zs[r * TS + c];
                if (p.Euser) p.Euser[(long)gr * p.lde + gc] = (double)Ys[r * LDT + c];
            }
        }
        for (int e = tid; e < TS * TS; e += THREADS) {
            const int a = e >> 6, b = e & 63;
            p.E32[(long)(row0 + a) * p.np + col0 + b] = Ys[a * LDT + b];
            p.C32t[(long)(col0 + a) * p.mp + row0 + b] = Cs[b * LDT + a];     // transposed: the next tiles read C depth-major
        }
        __syncthreads();
        if (tid == 0) {
            __threadfence();
            st_release_u32(p.flags + (long)I * p.ntj + J, 1u);
            if (s_badkey != ~0ull) {
                const unsigned long long k = s_badkey;
                report(p.info, ((k >> 41) & 1ull) ? GPTQ2D_ERR_INT_OVERFLOW : GPTQ2D_ERR_NONFINITE,
                       (int)((k >> 20) & 0x1fffffull), (int)(k & 0xfffffull), 0);
                s_badkey = ~0ull;
            }
        }
        F32_MARK(st_store);
#ifdef TILED_STATS
        st_n += 1;
#endif
    }
#ifdef TILED_STATS
    if (tid == 128 && (blockIdx.x % 61) == 0 && st_n > 0)
        printf("cta %3d row 32 per step: sums %lld rounding %lld barrier %lld\n", (int)blockIdx.x, sw_sums / (st_n * 128), sw_round / (st_n * 128),
               sw_bar / (st_n * 128));
    if (tid == 0 && blockIdx.x == 0) printf("slabs by %s\n", p.use_tma ? "bulk tensor copies" : "cp.async");
    if (tid == 0 && (blockIdx.x % 61) == 0 && st_n > 0)
        printf("cta %3d tiles %lld | per tile: claim %lld gemm(+flag waits) %lld of which flag scans and waits %lld form %lld sweep %lld store %lld\n",
               (int)blockIdx.x, st_n, st_claim / st_n, st_gemm / st_n, st_wait / st_n, st_form / st_n, st_sweep / st_n, st_store / st_n);
#endif
    for (int o = 16; o > 0; o >>= 1) max_abs_e = fmax(max_abs_e, __shfl_xor_sync(0xffffffffu, max_abs_e, o));
    if ((tid & 31) == 0) s_red[tid >> 5] = max_abs_e;
    __syncthreads();
    if (tid == 0) {
        double v = 0.0;
        for (int w = 0; w < THREADS / 32; ++w) v = fmax(v, s_red[w]);
        if (v > 0.0) atomic_max_nonneg_double(p.max_abs_e, v);
    }
}

// fp64 matrix -> fp32 copy with a leading dimension padded to a multiple of 4 (16-byte rows for cp.async)
__global__ void narrow_kernel(float *dst, long ldd, const double *src, long lds, int rows, int cols) {
    const long total = (long)rows * ldd;
    for (long idx = (long)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (long)gridDim.x * blockDim.x) {
        const long r = idx / ldd;
        const int c = (int)(idx - r * ldd);
        dst[idx] = c < cols ? (float)src[r * lds + c] : 0.f;
    }
}

// the same, transposed: dst[c][r] = src[r][c] for a square matrix of order n; 32 x 32 pieces through shared memory, blocks of 32 x 8
__global__ void narrow_transposed_kernel(float *dst, long ldd, const double *src, long lds, int n) {
    __shared__ float t[32][33];
    const int nb = (int)((ldd + 31) / 32);
    for (long piece = blockIdx.x; piece < (long)nb * nb; piece += gridDim.x) {
        const int r0 = (int)(piece / nb) * 32, c0 = (int)(piece % nb) * 32;
        for (int i = threadIdx.y; i < 32; i += 8) {
            const int r = r0 + i, c = c0 + threadIdx.x;
            t[i][threadIdx.x] = (r < n && c < n) ? (float)src[(long)r * lds + c] : 0.f;
        }
        __syncthreads();
        for (int i = threadIdx.y; i < 32; i += 8) {
            const int c = c0 + i, r = r0 + threadIdx.x;                    // dst row c, column r
            if (c < n && r < ldd) dst[(long)c * ldd + r] = t[threadIdx.x][i];
        }
        __syncthreads();
    }
}

static size_t pad256(size_t x) { return (x + 255) / 256 * 256; }
struct Layout {
    int nti, ntj;
    long mp, np, ldl, ldu;
    size_t flags_off, l_off, u_off, e_off, c_off, total;
};
static Layout layout(int m, int n) {
    Layout l;
    l.nti = (m + TS - 1) / TS; l.ntj = (n + TS - 1) / TS;
    l.mp = (long)l.nti * TS; l.np = (long)l.ntj * TS;
    l.ldl = ((long)m + 3) / 4 * 4; l.ldu = ((long)n + 3) / 4 * 4;
    l.flags_off = 256;
    l.l_off = l.flags_off + pad256((size_t)l.nti * l.ntj * sizeof(unsigned));
    l.u_off = l.l_off + pad256((size_t)m * l.ldl * sizeof(float));
    l.e_off = l.u_off + pad256((size_t)n * l.ldu * sizeof(float));
    l.c_off = l.e_off + pad256((size_t)l.mp * l.np * sizeof(float));
    l.total = l.c_off + pad256((size_t)l.mp * l.np * sizeof(float));
    return l;
}

}  // namespace f32

size_t round_tiled_f32_workspace_bytes(int m, int n) { return f32::layout(m, n).total; }

// 0: slabs by bulk tensor copies where the driver offers tensor maps; 1: always by cp.async (comparison, tests)
static int g_f32_tma_mode = 0;
void round_tiled_f32_set_tma_mode(int mode) { g_f32_tma_mode = mode; }

int launch_round_tiled_f32(const TiledParams &in, void *ws, size_t ws_bytes, cudaStream_t stream) {
    using namespace f32;
    const Layout l = layout(in.m, in.n);
    if (ws_bytes < l.total) return GPTQ2D_ERR_WORKSPACE;
    char *w = static_cast<char *>(ws);
    Params p{};
    p.m = in.m; p.n = in.n; p.nti = l.nti; p.ntj = l.ntj; p.ntiles = l.nti * l.ntj;
    p.mp = l.mp; p.np = l.np;
    p.X = in.X; p.ldx = in.ldx; p.Z = in.Z; p.ldz = in.ldz; p.Euser = in.E; p.lde = in.lde;
    float *L32 = reinterpret_cast<float *>(w + l.l_off), *U32 = reinterpret_cast<float *>(w + l.u_off);
    p.L32t = L32; p.ldl = l.ldl; p.U32 = U32; p.ldu = l.ldu;
    p.E32 = reinterpret_cast<float *>(w + l.e_off);
    p.C32t = reinterpret_cast<float *>(w + l.c_off);
    p.counter = reinterpret_cast<unsigned *>(w);
    p.abort = reinterpret_cast<unsigned *>(w) + 1;
    p.flags = reinterpret_cast<unsigned *>(w + l.flags_off);
    p.max_abs_e = workspace_max_abs_e(ws);
    p.info = in.info;
    p.spin_limit = SPIN_LIMIT;
    if (cudaMemsetAsync(w, 0, l.l_off, stream) != cudaSuccess) return GPTQ2D_ERR_CUDA;      // header and flags
    int dev = 0, sms = 0, per_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return GPTQ2D_ERR_CUDA;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return GPTQ2D_ERR_CUDA;
    narrow_transposed_kernel<<<sms * 8, dim3(32, 8), 0, stream>>>(L32, l.ldl, in.L, in.ldl, in.m);
    narrow_kernel<<<sms * 4, 256, 0, stream>>>(U32, l.ldu, in.U, in.ldu, in.n, in.n);
    if (cudaGetLastError() != cudaSuccess) return GPTQ2D_ERR_CUDA;
    if (cudaFuncSetAttribute(round_tiled_f32_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES) != cudaSuccess)
        return GPTQ2D_ERR_CUDA;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, round_tiled_f32_kernel, THREADS, SMEM_BYTES) != cudaSuccess ||
        per_sm < 1)
        return GPTQ2D_ERR_CUDA;
    if (per_sm > 1) per_sm = 1;
    int grid = sms * per_sm;
    if (grid > p.ntiles) grid = p.ntiles;
    // tensor maps of the four operand matrices (this GPU's own workspace; every CTA fetches its own boxes)
    CUtensorMap mapL, mapE, mapC, mapU;
    memset(&mapL, 0, sizeof(mapL)); memset(&mapE, 0, sizeof(mapE)); memset(&mapC, 0, sizeof(mapC)); memset(&mapU, 0, sizeof(mapU));
    p.use_tma = g_f32_tma_mode == 0 &&
                encode_f32_matrix_map(&mapL, L32, in.m, in.m, l.ldl, TS, KS) &&
                encode_f32_matrix_map(&mapE, p.E32, l.mp, l.np, l.np, TS, KS) &&
                encode_f32_matrix_map(&mapC, p.C32t, l.np, l.mp, l.mp, TS, KS) &&
                encode_f32_matrix_map(&mapU, U32, in.n, in.n, l.ldu, TS, KS);
    void *args[] = {&p, &mapL, &mapE, &mapC, &mapU};
    if (cudaLaunchCooperativeKernel((const void *)round_tiled_f32_kernel, dim3(grid), dim3(THREADS), args, SMEM_BYTES, stream) !=
        cudaSuccess)
        return GPTQ2D_ERR_CUDA;
    return GPTQ2D_OK;
}

}  // namespace gptq2d
