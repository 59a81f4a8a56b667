// GPTQ-2D sweep in fp32 (the optional reduced-precision mode), tiled.
//
// X, L and U are rounded to fp32 and every operation of Algorithm 3 is carried out in fp32; the order of
// the sums is that of the tile restatement (Eq. 11, Eq. 15-17), not of the literal algorithm: for the
// 64 x 64 tile (I, J) with rows r and columns c
//     Cd = sum_{I' < I} L[r, I'] E[I', c]        Rt = sum_{J' < J} C[r, J'] U[J', c]
// and Algorithm 3 on the tile alone, started from Y = X[r, c] + Rt + Cd and C = Cd with the diagonal
// blocks L[r, r] and U[c, c], gives the tile's Z, E and C = L E.  fp32 has no tensor-core path that keeps
// fp32 operands exact (TF32 truncates them), so the two contractions are a register-tiled FFMA loop:
// 256 threads, a 4 x 4 piece of the tile per thread and contraction, operand slabs of 32 staged through
// shared memory with cp.async (one CTA barrier per slab: at 16 the barrier was the first stall reason).
//
// One persistent, cooperatively launched grid, two CTAs per SM.  Tiles are claimed wave by wave (I + J
// ascending) from one atomic counter; a CTA folds the source tiles in as their flags come up -- the far
// ones first, the tile above and the tile to the left last -- and then sweeps its tile.  While one CTA
// of an SM sits in the dependent chain of its in-tile sweep the other one multiplies.  A tile only waits
// for tiles of earlier waves, which were claimed earlier, so the earliest unfinished tile can always run.
//
// In-tile sweep: one anti-diagonal per step, one CTA barrier per step, in the implicit-Y (pull) form of
// Appendix B (Eq. 19-20): an entry reads the errors above it in its column through L and the finished C to
// its left in its row through U at the moment it is rounded, four lanes per row sharing the two dot
// products.  Only rows with an entry on the current anti-diagonal work, and nothing is read-modify-written
// (an eager version that pushed every error down and right as Algorithm 3 prints it cost 7x the time per
// step: 2 x 64 x 64 shared-memory updates per anti-diagonal, issued by every warp).
#include <cstdio>
#include "common.cuh"
#include "dmma_gemm.cuh"          // cp.async helpers
#include "round_internal.cuh"

namespace gptq2d {
namespace f32 {

constexpr int TS = 64;             // tile edge
constexpr int THREADS = 256;
constexpr int KS = 64;             // slab depth
constexpr int SPS = TS / KS;       // slabs per source tile
constexpr int NSTAGE = 3;          // cp.async ring; it lives where the in-tile matrices go afterwards
constexpr int LDA = KS + 4;        // A slab [64 rows][KS k], row stride KS + 4 floats: 16-byte rows, conflict-free float4 reads
constexpr int LDB = TS + 4;        // B slab [16 k][64 cols], row stride 68 floats
constexpr int A_FLOATS = TS * LDA, B_FLOATS = KS * LDB, STAGE_FLOATS = A_FLOATS + B_FLOATS;
constexpr int LDT = TS + 4;        // in-tile matrices, row stride 68 floats: the 8 rows x 4 lanes of a warp hit 32 different banks
                                   // in the push loops (bank = 4 row -+ lane)
constexpr int TMAT = TS * LDT;
constexpr int SWEEP_FLOATS = 5 * TMAT + TS * TS, RING_FLOATS = NSTAGE * STAGE_FLOATS;      // + the tile's Z (int32)
constexpr size_t SMEM_BYTES = (size_t)(SWEEP_FLOATS > RING_FLOATS ? SWEEP_FLOATS : RING_FLOATS) * sizeof(float);

struct Params {
    int m, n, nti, ntj, ntiles;
    long mp, np;                   // padded extents (multiples of 64): leading dimension of E32 / C32 is np
    const double *X; long ldx;
    int *Z; long ldz;
    double *Euser; long lde;
    const float *L32; long ldl;    // m x m (leading dimension padded to a multiple of 4)
    const float *U32; long ldu;
    float *E32, *C32;
    unsigned *counter, *abort, *flags;
    double *max_abs_e;
    int *info;
    unsigned long long spin_limit;
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

// One source tile: acc += A (64 x 64, [row][k], leading dimension lda) * B (64 x 64, [k][col], ldb), both fully
// inside padded or zero-filled storage except that rows of A beyond `a_rows` and columns of B beyond `b_cols`
// (ragged edge of a user matrix) are read as zeros.  K is streamed in SPS slabs of KS.
struct Gemm {
    float *stages;
    int tid, ty, tx;
    // copy plan: A slab = 64 rows x KS k, B slab = KS k x 64 columns, in chunks of 4 floats, KS / 16 of each per thread
    __device__ __forceinline__ void issue(int stage, const float *A, long lda, int a_rows, int a_kmax, const float *B, long ldb,
                                          int b_cols, int b_kmax, int k0) const {
        float *As = stages + stage * STAGE_FLOATS, *Bs = As + A_FLOATS;
#pragma unroll
        for (int h = 0; h < KS / 16; ++h) {               // A slab: 64 rows x KS k, chunks of 4 floats
            const int c = tid + h * THREADS;
            const int r = c / (KS / 4), kc = (c % (KS / 4)) * 4;
            int nv = (r < a_rows) ? a_kmax - (k0 + kc) : 0;          // floats valid from kc on
            nv = nv < 0 ? 0 : (nv > 4 ? 4 : nv);
            cp_async16f(As + r * LDA + kc, nv ? A + (long)r * lda + k0 + kc : A, nv * 4);
        }
#pragma unroll
        for (int h = 0; h < KS / 16; ++h) {               // B slab: KS k x 64 columns
            const int c = tid + h * THREADS;
            const int kr = c >> 4, cc = (c & 15) * 4;
            int nv = (k0 + kr < b_kmax) ? b_cols - cc : 0;
            nv = nv < 0 ? 0 : (nv > 4 ? 4 : nv);
            cp_async16f(Bs + kr * LDB + cc, nv ? B + (long)(k0 + kr) * ldb + cc : B, nv * 4);
        }
    }
    __device__ __forceinline__ void multiply(float (&acc)[4][4], int stage) const {
        const float *As = stages + stage * STAGE_FLOATS, *Bs = As + A_FLOATS;
#pragma unroll
        for (int k4 = 0; k4 < KS; k4 += 4) {
            float4 a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) a[i] = *reinterpret_cast<const float4 *>(As + (ty * 4 + i) * LDA + k4);
#pragma unroll
            for (int k = 0; k < 4; ++k) b[k] = *reinterpret_cast<const float4 *>(Bs + (k4 + k) * LDB + tx * 4);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float av[4] = {a[i].x, a[i].y, a[i].z, a[i].w};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    acc[i][0] = fmaf(av[k], b[k].x, acc[i][0]);
                    acc[i][1] = fmaf(av[k], b[k].y, acc[i][1]);
                    acc[i][2] = fmaf(av[k], b[k].z, acc[i][2]);
                    acc[i][3] = fmaf(av[k], b[k].w, acc[i][3]);
                }
            }
        }
    }
};

__global__ void __launch_bounds__(THREADS, 2) round_tiled_f32_kernel(Params p) {
    extern __shared__ __align__(16) float smem[];
    __shared__ int s_task;
    __shared__ int s_ok, s_upto;
    __shared__ double s_red[THREADS / 32];
    __shared__ unsigned long long s_badkey;
    float *stages = smem;
    // the contraction's accumulators are registers, so the in-tile matrices reuse the ring's memory
    // Ld[i][i'] = L[i, i'] (strictly lower), Udt[j][j'] = U[j', j] (the diagonal block of U transposed, strictly
    // lower), Et[j][i'] = E[i', j] (transposed copy of the errors): the rows the dot products of the sweep run along
    float *Ys = smem, *Cs = Ys + TMAT, *Ld = Cs + TMAT, *Udt = Ld + TMAT, *Et = Udt + TMAT;
    int *Zs = reinterpret_cast<int *>(Et + TMAT);  // [64][64]: rounded values, written out row-wise after the sweep
    const int tid = threadIdx.x;
    Gemm gm{stages, tid, tid >> 4, tid & 15};
    double max_abs_e = 0.0;
    if (tid == 0) s_badkey = ~0ull;
#ifdef TILED_STATS
    long long st_claim = 0, st_gemm = 0, st_form = 0, st_sweep = 0, st_store = 0, st_n = 0, st_t = clock64();
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

        // ---- 1. the two contractions.  Source list: tiles (0..I-2, J) through L, tiles (I, 0..J-2) through U, then
        // the tile above and the tile to the left (the newest ones, still being swept when this tile is claimed).
        float cd[4][4], rt[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) cd[i][j] = rt[i][j] = 0.f;
        const int nsrc = I + J, nslab = nsrc * SPS;
        bool ok = true;
        // slab g of the flattened list belongs to source g / 4; operands of a source (all threads compute them)
        struct Src { const float *A, *B; long lda, ldb; int a_rows, a_kmax, b_cols, b_kmax, dir; const unsigned *flag; };
        auto source = [&](int sidx) {
            int dir, k;
            const int na = max(0, I - 1), nl = max(0, J - 1);        // older sources of each direction
            if (sidx < na) { dir = 0; k = sidx; }
            else if (sidx < na + nl) { dir = 1; k = sidx - na; }
            else if (sidx == na + nl && I > 0) { dir = 0; k = I - 1; }
            else { dir = 1; k = J - 1; }
            Src r;
            r.dir = dir;
            if (dir == 0) {          // L[r, rows of tile k] * E[rows of tile k, c]
                r.A = p.L32 + (long)row0 * p.ldl + (long)k * TS; r.lda = p.ldl;
                r.a_rows = min(TS, p.m - row0); r.a_kmax = min(TS, p.m - k * TS);
                r.B = p.E32 + (long)k * TS * p.np + col0; r.ldb = p.np; r.b_cols = TS; r.b_kmax = TS;
                r.flag = p.flags + (long)k * p.ntj + J;
            } else {                 // C[r, columns of tile k] * U[columns of tile k, c]
                r.A = p.C32 + (long)row0 * p.np + (long)k * TS; r.lda = p.np; r.a_rows = TS; r.a_kmax = TS;
                r.B = p.U32 + (long)k * TS * p.ldu + col0; r.ldb = p.ldu;
                r.b_cols = min(TS, p.n - col0); r.b_kmax = min(TS, p.n - k * TS);
                r.flag = p.flags + (long)I * p.ntj + k;
            }
            return r;
        };
        // Sources [0, ready_upto) are known to be swept.  The list is scanned by the whole CTA at once (one flag per
        // thread, the first unset position by a shared-memory minimum), so that a tile whose far sources are all
        // done -- the usual case -- pays two barriers for the lot instead of a global round trip per source; only
        // when the next source in line is still being swept does one thread wait for it, bounded.
        int ready_upto = 0;
        auto scan_ready = [&](int from) -> bool {         // all threads; false if the bounded wait ran out
            if (tid == 0) {
                unsigned long long it = 0;
                int good = 1;
                const Src sr = source(from);
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
                s_upto = nsrc;
            }
            __syncthreads();
            for (int k = from + 1 + tid; k < nsrc; k += THREADS)
                if (ld_acquire_u32(source(k).flag) == 0u) atomicMin(&s_upto, k);
            __syncthreads();
            const bool good = s_ok != 0;
            ready_upto = s_upto;
            __syncthreads();                              // s_ok / s_upto may be rewritten by the next scan
            return good;
        };
        // Issues slab g (all threads); returns false if a wait ran out.
        auto issue_slab = [&](int g) -> bool {
            const int sidx = g / SPS;
            if (sidx >= ready_upto && !scan_ready(sidx)) return false;
            const Src sr = source(sidx);
            gm.issue(g % NSTAGE, sr.A, sr.lda, sr.a_rows, sr.a_kmax, sr.B, sr.ldb, sr.b_cols, sr.b_kmax, (g % SPS) * KS);
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
            if (source(g / SPS).dir == 0) gm.multiply(cd, g % NSTAGE); else gm.multiply(rt, g % NSTAGE);
        }
        cp_async_wait<0>();
        __syncthreads();
        if (!ok) break;
        F32_MARK(st_gemm);

        // ---- 2. Y = X + Rt + Cd, C = Cd; diagonal blocks of the factors (strict triangles, zero elsewhere)
        {
            const int ty = tid >> 4, tx = tid & 15;
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int r = ty * 4 + i, c = tx * 4 + j, gr = row0 + r, gc = col0 + c;
                    const float x = (gr < p.m && gc < p.n) ? (float)__ldg(p.X + (long)gr * p.ldx + gc) : 0.f;
                    Cs[r * LDT + c] = cd[i][j];
                    Ys[r * LDT + c] = (x + rt[i][j]) + cd[i][j];
                }
#pragma unroll 8
            for (int e = tid; e < TS * TS; e += THREADS) {
                const int r = e >> 6, c = e & 63;
                const int gr = row0 + r, gcl = row0 + c;       // L block: rows / columns of the row range
                Ld[r * LDT + c] = (c < r && gr < p.m) ? p.L32[(long)gr * p.ldl + gcl] : 0.f;
                const int ur = col0 + r, uc = col0 + c;        // U block (r, c) with r < c, stored transposed
                Udt[c * LDT + r] = (c > r && uc < p.n) ? p.U32[(long)ur * p.ldu + uc] : 0.f;
                Et[r * LDT + c] = 0.f;                         // unrounded entries count as zero (they meet zero coefficients)
            }
        }
        __syncthreads();
        F32_MARK(st_form);

        // ---- 3. the tile's 127 anti-diagonals, in the implicit-Y (pull) form of Appendix B, Eq. 19-20, which gives
        // the same entries as Algorithm 3: entry (i, j) reconstructs its corrected value when it is rounded,
        //     Y_ij = Y0_ij + sum_{i' < i} L[i, i'] E[i', j] + sum_{j' < j} C[i, j'] U[j', j],
        // and its final C_ij = C0_ij + sum_{i' < i} L[i, i'] E[i', j] + E_ij is stored once.  Everything it reads was
        // rounded on an earlier anti-diagonal, nothing is read-modify-written, and only the rows that own an
        // entry of the current anti-diagonal work: four lanes per row, each a quarter of the two dot products.
        // Ys holds Y0 until an entry is rounded and E afterwards; Cs holds C0 and then C.
        {
            const int row = tid >> 2, sub = tid & 3;
            const float *lrow = Ld + row * LDT;
            float *yrow = Ys + row * LDT, *crow = Cs + row * LDT;
            unsigned long long badkey = ~0ull;
            float max_e = 0.f;
            for (int s = 0; s < 2 * TS - 1; ++s) {
                const int j = s - row;
                if (j >= 0 && j < TS) {                                  // (uniform over the row's four lanes)
                    // Both dot products run along rows of shared memory in chunks of four; a lane takes every fourth
                    // chunk.  Beyond the diagonal the coefficients are zero (strict triangles) and what they meet is
                    // finite (zeros, or values of entries rounded later), so whole chunks need no masking.
                    float dl[2] = {0.f, 0.f}, du[2] = {0.f, 0.f};
                    const float4 *l4 = reinterpret_cast<const float4 *>(lrow), *e4 = reinterpret_cast<const float4 *>(Et + j * LDT);
                    for (int q = sub; 4 * q < row; q += 4) {                // down the column: sources i' < row
                        const float4 a = l4[q], b = e4[q];
                        dl[0] = fmaf(a.x, b.x, dl[0]); dl[1] = fmaf(a.y, b.y, dl[1]);
                        dl[0] = fmaf(a.z, b.z, dl[0]); dl[1] = fmaf(a.w, b.w, dl[1]);
                    }
                    const float4 *c4 = reinterpret_cast<const float4 *>(crow), *u4 = reinterpret_cast<const float4 *>(Udt + j * LDT);
                    for (int q = sub; 4 * q < j; q += 4) {                  // along the row: sources j' < j
                        const float4 a = c4[q], b = u4[q];
                        du[0] = fmaf(a.x, b.x, du[0]); du[1] = fmaf(a.y, b.y, du[1]);
                        du[0] = fmaf(a.z, b.z, du[0]); du[1] = fmaf(a.w, b.w, du[1]);
                    }
                    float sl = dl[0] + dl[1], su = du[0] + du[1];
                    const unsigned gmask = 0xfu << ((tid & 31) & ~3);          // the row's four lanes (rows of a warp differ in activity)
                    sl += __shfl_xor_sync(gmask, sl, 1);
                    su += __shfl_xor_sync(gmask, su, 1);
                    sl += __shfl_xor_sync(gmask, sl, 2);
                    su += __shfl_xor_sync(gmask, su, 2);
                    if (sub == 0) {
                        const float y = (yrow[j] + su) + sl;
                        const float z = rintf(y);
                        const float e = z - y;                           // E = Z - Y
                        crow[j] = (crow[j] + sl) + e;                    // C = L E (unit diagonal)
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
                }
                __syncthreads();
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
            const int r = e >> 6, c = e & 63;
            const long at = (long)(row0 + r) * p.np + col0 + c;
            p.E32[at] = Ys[r * LDT + c];
            p.C32[at] = Cs[r * LDT + c];
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
    if (tid == 0 && (blockIdx.x % 61) == 0 && st_n > 0)
        printf("cta %3d tiles %lld | per tile: claim %lld gemm(+flag waits) %lld form %lld sweep %lld store %lld\n", (int)blockIdx.x, st_n,
               st_claim / st_n, st_gemm / st_n, st_form / st_n, st_sweep / st_n, st_store / st_n);
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
    p.L32 = L32; p.ldl = l.ldl; p.U32 = U32; p.ldu = l.ldu;
    p.E32 = reinterpret_cast<float *>(w + l.e_off);
    p.C32 = reinterpret_cast<float *>(w + l.c_off);
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
    narrow_kernel<<<sms * 4, 256, 0, stream>>>(L32, l.ldl, in.L, in.ldl, in.m, in.m);
    narrow_kernel<<<sms * 4, 256, 0, stream>>>(U32, l.ldu, in.U, in.ldu, in.n, in.n);
    if (cudaGetLastError() != cudaSuccess) return GPTQ2D_ERR_CUDA;
    if (cudaFuncSetAttribute(round_tiled_f32_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES) != cudaSuccess)
        return GPTQ2D_ERR_CUDA;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, round_tiled_f32_kernel, THREADS, SMEM_BYTES) != cudaSuccess ||
        per_sm < 1)
        return GPTQ2D_ERR_CUDA;
    if (per_sm > 2) per_sm = 2;
    int grid = sms * per_sm;
    if (grid > p.ntiles) grid = p.ntiles;
    void *args[] = {&p};
    if (cudaLaunchCooperativeKernel((const void *)round_tiled_f32_kernel, dim3(grid), dim3(THREADS), args, SMEM_BYTES, stream) !=
        cudaSuccess)
        return GPTQ2D_ERR_CUDA;
    return GPTQ2D_OK;
}

}  // namespace gptq2d
