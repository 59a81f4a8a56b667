// The library's own fp64 GEMM kernel: one CTA per 128 x 128 output tile, DMMA mainloop.
#include "dmma_gemm.cuh"
#include "dmma_tma.cuh"
#include "tma_host.cuh"
#include "gemm.cuh"

namespace gptq2d {

constexpr int GEMM_NSTAGE = 3;

template <bool A_KCONTIG, bool B_KCONTIG>
__global__ void __launch_bounds__(GEMM_THREADS, 1) gemm_kernel(GemmArgs p) {
    extern __shared__ __align__(16) double smem[];
    // (with a lower-triangular A the contraction of tile row tm is tm + 1 blocks long: the longest rows are started first)
    const int tn = blockIdx.x, tm = p.a_lower ? (int)(gridDim.y - 1 - blockIdx.y) : (int)blockIdx.y, bz = blockIdx.z;
    if (p.lower_tiles_only && tn > tm) return;
    const int m0 = tm * BM, n0 = tn * BN;
    const double *Ab = p.A + (long)bz * p.strideA;
    const double *Bb = p.B + (long)bz * p.strideB;

    Operand A, B;
    // A_KCONTIG <=> op(A) = A (M x K stored row-major, k contiguous)
    A.ptr = A_KCONTIG ? Ab + (long)m0 * p.lda : Ab + m0;
    A.ld = p.lda;
    A.mn_valid = min(BM, p.M - m0);
    A.aligned16 = ((((uintptr_t)A.ptr) & 15) == 0) && ((p.lda & 1) == 0);
    // B_KCONTIG <=> op(B) = B^T (B stored N x K row-major, k contiguous)
    B.ptr = B_KCONTIG ? Bb + (long)n0 * p.ldb : Bb + n0;
    B.ld = p.ldb;
    B.mn_valid = min(BN, p.N - n0);
    B.aligned16 = ((((uintptr_t)B.ptr) & 15) == 0) && ((p.ldb & 1) == 0);

    // k-range of this tile (whole range unless an operand is triangular); both ends are multiples of 128
    const int k_lo = p.b_lower ? min(p.K, n0) : 0;
    const int k_hi = p.a_lower ? min(p.K, m0 + BM) : p.K;
    A.ptr += A_KCONTIG ? (long)k_lo : (long)k_lo * p.lda;
    B.ptr += B_KCONTIG ? (long)k_lo : (long)k_lo * p.ldb;

    Acc acc;
    acc.zero();
    if (k_hi > k_lo) gemm_tile<A_KCONTIG, B_KCONTIG, GEMM_NSTAGE>(acc, smem, A, B, k_hi - k_lo);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int wm = warp >> 2, wn = warp & 3, g = lane >> 2, t = lane & 3;

    if (p.sumsq_partials) {
        double s = 0.0;
#pragma unroll
        for (int a = 0; a < 8; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                double x0 = p.alpha * acc.v[a][b][0], x1 = p.alpha * acc.v[a][b][1];
                s = fma(x0, x0, s);
                s = fma(x1, x1, s);
            }
        // rows/cols beyond M/N hold exact zeros (zero-filled operands), so no mask is needed
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        __shared__ double wsum[8];
        if (lane == 0) wsum[warp] = s;
        __syncthreads();
        if (tid == 0) {
            double tot = 0.0;
            for (int w = 0; w < 8; ++w) tot += wsum[w];
            p.sumsq_partials[((long)bz * gridDim.y + tm) * gridDim.x + tn] = tot;
        }
        return;
    }

    double *Cb = p.C + (long)bz * p.strideC;
    const bool vec = ((((uintptr_t)Cb) & 15) == 0) && ((p.ldc & 1) == 0);
    if (p.beta != 0.0 && vec && m0 + BM <= p.M && n0 + BN <= p.N) {
        // Update of a full tile (the rank-k updates of the set-up): the old values are read in two batches of sixteen
        // 16-byte loads per thread before anything is stored, so that the loads of a batch are in flight together
        // (loads and stores to the same matrix one after the other run as a chain of dependent round trips).
        double *c00 = Cb + (long)(m0 + wm * 64 + g) * p.ldc + n0 + wn * 32 + t * 2;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            double2 old[4][4];
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b)
                    old[a][b] = *reinterpret_cast<const double2 *>(c00 + (long)((half * 4 + a) * 8) * p.ldc + b * 8);
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) {
                    double2 o;
                    o.x = fma(p.beta, old[a][b].x, p.alpha * acc.v[half * 4 + a][b][0]);
                    o.y = fma(p.beta, old[a][b].y, p.alpha * acc.v[half * 4 + a][b][1]);
                    *reinterpret_cast<double2 *>(c00 + (long)((half * 4 + a) * 8) * p.ldc + b * 8) = o;
                }
        }
        return;
    }
#pragma unroll
    for (int a = 0; a < 8; ++a) {
        int r = m0 + wm * 64 + a * 8 + g;
        if (r >= p.M) continue;
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            int c = n0 + wn * 32 + b * 8 + t * 2;
            if (c >= p.N) continue;
            double *dst = Cb + (long)r * p.ldc + c;
            double x0 = p.alpha * acc.v[a][b][0], x1 = p.alpha * acc.v[a][b][1];
            if (c + 1 < p.N && vec) {
                double2 o;
                if (p.beta != 0.0) {
                    double2 old = *reinterpret_cast<const double2 *>(dst);
                    o.x = fma(p.beta, old.x, x0);
                    o.y = fma(p.beta, old.y, x1);
                } else {
                    o.x = x0;
                    o.y = x1;
                }
                *reinterpret_cast<double2 *>(dst) = o;
            } else {
                dst[0] = (p.beta != 0.0) ? fma(p.beta, dst[0], x0) : x0;
                if (c + 1 < p.N) dst[1] = (p.beta != 0.0) ? fma(p.beta, dst[1], x1) : x1;
            }
        }
    }
}


// ---------------------------------------------------------------------------------------------
// The same GEMM with TMA-fed operand slabs (dmma_tma.cuh): used whenever both operands are 16-byte
// aligned with even leading dimensions.  Ragged edges need no special loop here: parts of a box that
// lie outside the tensor read as zeros.
constexpr int GEMM_TMA_NSTAGE = 4;
constexpr size_t GEMM_TMA_SMEM = (size_t)GEMM_TMA_NSTAGE * TMA_STAGE_BYTES + 1024;   // + slack to align the ring to 1024 B

// pair q (0..3) of row-fragment a: two horizontally adjacent elements of the tile held by this lane
template <bool B_KCONTIG>
__device__ __forceinline__ void acc_pair(const Acc &acc, int a, int q, int wn, int t, int &col, double &x0, double &x1) {
    if (B_KCONTIG) {
        const int bq = q >> 1, j = q & 1;
        col = wn * 32 + bq * 16 + 4 * t + 2 * j;
        x0 = acc.v[a][2 * bq][j];
        x1 = acc.v[a][2 * bq + 1][j];
    } else {
        col = acc_col<false>(wn, q, t, 0);
        x0 = acc.v[a][q][0];
        x1 = acc.v[a][q][1];
    }
}

template <bool A_KCONTIG, bool B_KCONTIG, bool SLAB_SYNC>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_tma_kernel(GemmArgs p, const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB,
                unsigned *abort) {
    extern __shared__ __align__(16) double smem_raw[];
    __shared__ __align__(8) unsigned long long bars[2 * GEMM_TMA_NSTAGE];
    // (with a lower-triangular A the contraction of tile row tm is tm + 1 blocks long: the longest rows are started first)
    const int tn = blockIdx.x, tm = p.a_lower ? (int)(gridDim.y - 1 - blockIdx.y) : (int)blockIdx.y, bz = blockIdx.z;
    if (p.lower_tiles_only && tn > tm) return;
    const int m0 = tm * BM, n0 = tn * BN;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int wm = warp >> 2, wn = warp & 3, g = lane >> 2, t = lane & 3;
    // aligned to 1024 bytes by an offset into the shared array (pointer arithmetic keeps the shared address space)
    double *stages = smem_raw + (((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u) >> 3);

    TmaRing ring;
    tma_ring_init<GEMM_TMA_NSTAGE, GEMM_THREADS / 32>(ring, bars, stages, tid);
    __syncthreads();

    const int k_lo = p.b_lower ? min(p.K, n0) : 0;
    const int k_hi = p.a_lower ? min(p.K, m0 + BM) : p.K;
    Acc acc;
    acc.zero();
    if (k_hi > k_lo) {
        TmaOperand A{&mapA, m0, k_lo, bz}, B{&mapB, n0, k_lo, bz};
        const int nk = (k_hi - k_lo + TMA_BK - 1) / TMA_BK;
        if (!gemm_tma_mainloop<A_KCONTIG, B_KCONTIG, GEMM_TMA_NSTAGE, SLAB_SYNC ? 1 : -1>(acc, ring, A, B, nk, warp, lane, abort))
            return;
    }

    if (p.sumsq_partials) {
        double s = 0.0;
#pragma unroll
        for (int a = 0; a < 8; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                double x0 = p.alpha * acc.v[a][b][0], x1 = p.alpha * acc.v[a][b][1];
                s = fma(x0, x0, s);
                s = fma(x1, x1, s);
            }
        // NOTE: the order of this sum differs from the cp.async kernel's (another element-to-lane map)
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        __shared__ double wsum[8];
        if (lane == 0) wsum[warp] = s;
        __syncthreads();
        if (tid == 0) {
            double tot = 0.0;
            for (int w = 0; w < 8; ++w) tot += wsum[w];
            p.sumsq_partials[((long)bz * gridDim.y + tm) * gridDim.x + tn] = tot;
        }
        return;
    }

    double *Cb = p.C + (long)bz * p.strideC;
    const bool vec = ((((uintptr_t)Cb) & 15) == 0) && ((p.ldc & 1) == 0);
    if (p.beta != 0.0 && vec && m0 + BM <= p.M && n0 + BN <= p.N) {
        // update of a full tile: old values read in two batches of sixteen 16-byte loads before anything is stored (see the
        // cp.async kernel above)
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            double2 old[4][4];
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    int col;
                    double x0, x1;
                    acc_pair<B_KCONTIG>(acc, half * 4 + a, q, wn, t, col, x0, x1);
                    old[a][q] = *reinterpret_cast<const double2 *>(Cb + (long)(m0 + acc_row<A_KCONTIG>(wm, half * 4 + a, g)) * p.ldc + n0 + col);
                }
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    int col;
                    double x0, x1;
                    acc_pair<B_KCONTIG>(acc, half * 4 + a, q, wn, t, col, x0, x1);
                    double2 o;
                    o.x = fma(p.beta, old[a][q].x, p.alpha * x0);
                    o.y = fma(p.beta, old[a][q].y, p.alpha * x1);
                    *reinterpret_cast<double2 *>(Cb + (long)(m0 + acc_row<A_KCONTIG>(wm, half * 4 + a, g)) * p.ldc + n0 + col) = o;
                }
        }
        return;
    }
#pragma unroll
    for (int a = 0; a < 8; ++a) {
        const int r = m0 + acc_row<A_KCONTIG>(wm, a, g);
        if (r >= p.M) continue;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            int col;
            double x0, x1;
            acc_pair<B_KCONTIG>(acc, a, q, wn, t, col, x0, x1);
            const int c = n0 + col;
            if (c >= p.N) continue;
            double *dst = Cb + (long)r * p.ldc + c;
            x0 *= p.alpha; x1 *= p.alpha;
            if (c + 1 < p.N && vec) {
                double2 o;
                if (p.beta != 0.0) {
                    double2 old = *reinterpret_cast<const double2 *>(dst);
                    o.x = fma(p.beta, old.x, x0);
                    o.y = fma(p.beta, old.y, x1);
                } else {
                    o.x = x0;
                    o.y = x1;
                }
                *reinterpret_cast<double2 *>(dst) = o;
            } else {
                dst[0] = (p.beta != 0.0) ? fma(p.beta, dst[0], x0) : x0;
                if (c + 1 < p.N) dst[1] = (p.beta != 0.0) ? fma(p.beta, dst[1], x1) : x1;
            }
        }
    }
}

// 0: cp.async kernel only; 1 (default): the TMA-fed kernel where a tile edge is ragged (M or N not a multiple of
// 128, K not a multiple of 16) -- the copy engine zero-fills out-of-range parts of a box at full speed, where the
// cp.async kernel falls back to a loop with per-element predicates -- and the cp.async kernel for full tiles, where
// it measures 0.5-1 % faster; 2: TMA-fed kernel with a barrier per slab (slower; comparison); 3: TMA-fed kernel always
static int g_gemm_tma_mode = 1;
void gemm_set_tma_mode(int mode) { g_gemm_tma_mode = mode; }

template <bool AK, bool BKc, bool SS>
static cudaError_t launch_tma_variant(const GemmArgs &g, const CUtensorMap &mapA, const CUtensorMap &mapB, cudaStream_t stream) {
    cudaError_t e = cudaFuncSetAttribute(gemm_tma_kernel<AK, BKc, SS>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)GEMM_TMA_SMEM);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(gemm_tma_kernel<AK, BKc, SS>, cudaFuncAttributePreferredSharedMemoryCarveout,
                             cudaSharedmemCarveoutMaxShared);
    if (e != cudaSuccess) return e;
    dim3 grid((g.N + BN - 1) / BN, (g.M + BM - 1) / BM, g.batch);
    gemm_tma_kernel<AK, BKc, SS><<<grid, GEMM_THREADS, GEMM_TMA_SMEM, stream>>>(g, mapA, mapB, g.abort);
    return cudaGetLastError();
}

// false: this GEMM cannot take the TMA path (alignment, no encoder); *err holds a launch error if it was tried
template <bool AK, bool BKc>
static bool try_launch_tma(const GemmArgs &g, cudaStream_t stream, cudaError_t *err) {
    if (g_gemm_tma_mode == 0) return false;
    if (g_gemm_tma_mode == 1 && (g.M % BM) == 0 && (g.N % BN) == 0 && (g.K % BK) == 0) return false;
    CUtensorMap mapA, mapB;
    // op(A) is M x K: stored M x K (k contiguous) if AK, else K x M (m contiguous)
    const bool okA = AK ? encode_f64_matrix_map(&mapA, g.A, g.M, g.K, g.lda, g.batch, g.strideA, 16, 128)
                        : encode_f64_matrix_map(&mapA, g.A, g.K, g.M, g.lda, g.batch, g.strideA, 16, 16);
    if (!okA) return false;
    // op(B) is K x N: stored N x K (k contiguous) if BKc, else K x N (n contiguous)
    const bool okB = BKc ? encode_f64_matrix_map(&mapB, g.B, g.N, g.K, g.ldb, g.batch, g.strideB, 16, 128)
                         : encode_f64_matrix_map(&mapB, g.B, g.K, g.N, g.ldb, g.batch, g.strideB, 16, 16);
    if (!okB) return false;
    *err = g_gemm_tma_mode == 2 ? launch_tma_variant<AK, BKc, true>(g, mapA, mapB, stream)
                                : launch_tma_variant<AK, BKc, false>(g, mapA, mapB, stream);
    return true;
}

template <bool AK, bool BKc>
static cudaError_t launch_t(const GemmArgs &g, cudaStream_t stream) {
    cudaError_t terr = cudaSuccess;
    if (try_launch_tma<AK, BKc>(g, stream, &terr)) return terr;
    using SL = SlabLayout<AK, BKc>;
    size_t smem = (size_t)SL::STAGE_DOUBLES * GEMM_NSTAGE * sizeof(double);
    // Function attributes are kept per device: set them on every call (two cheap host-side calls), so that
    // a process that uses several GPUs gets the opt-in on each of them.  Same shared-memory carve-out as the
    // single-CTA kernels of the set-up that run between the GEMMs, so that the SMs are not reconfigured
    // from launch to launch.
    cudaError_t e = cudaFuncSetAttribute(gemm_kernel<AK, BKc>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(gemm_kernel<AK, BKc>, cudaFuncAttributePreferredSharedMemoryCarveout,
                             cudaSharedmemCarveoutMaxShared);
    if (e != cudaSuccess) return e;
    dim3 grid((g.N + BN - 1) / BN, (g.M + BM - 1) / BM, g.batch);
    gemm_kernel<AK, BKc><<<grid, GEMM_THREADS, smem, stream>>>(g);
    return cudaGetLastError();
}

cudaError_t launch_gemm(const GemmArgs &g, cudaStream_t stream) {
    if (g.M <= 0 || g.N <= 0 || g.batch <= 0) return cudaSuccess;
    bool ak = (g.opA == OP_N), bk = (g.opB == OP_T);
    if (ak && bk) return launch_t<true, true>(g, stream);
    if (ak && !bk) return launch_t<true, false>(g, stream);
    if (!ak && bk) return launch_t<false, true>(g, stream);
    return launch_t<false, false>(g, stream);
}

}  // namespace gptq2d
