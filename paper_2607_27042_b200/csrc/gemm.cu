// The library's own fp64 GEMM kernel: one CTA per 128 x 128 output tile, DMMA mainloop.
#include "dmma_gemm.cuh"
#include "gemm.cuh"

namespace gptq2d {

constexpr int GEMM_NSTAGE = 3;

template <bool A_KCONTIG, bool B_KCONTIG>
__global__ void __launch_bounds__(GEMM_THREADS, 1) gemm_kernel(GemmArgs p) {
    extern __shared__ __align__(16) double smem[];
    const int tn = blockIdx.x, tm = blockIdx.y, bz = blockIdx.z;
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

template <bool AK, bool BKc>
static cudaError_t launch_t(const GemmArgs &g, cudaStream_t stream) {
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
