// The implicit-Y form (Algorithm 6, Eq. 19-20) taken to its pull-only end: no corrected matrix is
// kept and nothing is pushed.  Entry (i, j) of anti-diagonal s = i + j reads, at rounding time,
//     c0   = sum_{i' < i} L[i, i'] E[i', j]                  (what Eq. 20 would have folded into C_ij)
//     Y_ij = X_ij + sum_{j' < j} C[i, j'] U[j', j] + c0      (Eq. 19; the j' = j term is c0, U_jj = 1)
// rounds, and writes E_ij and C_ij = c0 + E_ij.  Each entry is written once, by one warp; a stage
// needs ONE device-wide barrier.  Both dot products run over contiguous memory: the kernel keeps
// E transposed (Et) and starts by transposing U (Ut).
//
// This is the untiled comparison point for the tiled kernel, not a fast path: every entry streams
// 2 (i + j) words from L2 / HBM, 8 m n (m + n) bytes in all (8.8 TB at 8192^2), so it is bound by
// memory bandwidth where the tiled sweep is bound by the fp64 tensor rate.
#include "common.cuh"
#include "round_internal.cuh"

namespace gptq2d {

constexpr int PULL_THREADS = 512;

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__global__ void __launch_bounds__(PULL_THREADS) round_pull_kernel(PullParams p) {
    __shared__ double red[PULL_THREADS / 32];
    const int m = p.m, n = p.n;
    const unsigned nb = gridDim.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const long gwarp = (long)blockIdx.x * (PULL_THREADS / 32) + warp, nwarps = (long)nb * (PULL_THREADS / 32);
    double max_abs_e = 0.0;

    // Ut[j][k] = U[k][j] for k < j (the strict upper triangle of U, transposed)
    for (long idx = (long)blockIdx.x * blockDim.x + tid; idx < (long)n * n; idx += (long)nb * blockDim.x) {
        const int j = (int)(idx / n), k = (int)(idx % n);
        p.Ut[idx] = k < j ? p.U[(long)k * p.ldu + j] : 0.0;
    }
    bool ok = grid_barrier(p.sync, nb, p.info, -1);

    for (int s = 0; ok && s < m + n - 1; ++s) {
        const int lo = max(0, s - n + 1), hi = min(m - 1, s);
        for (long k = lo + gwarp; k <= hi; k += nwarps) {
            const int i = (int)k, j = s - i;
            const double *Ci = p.C + (long)i * n, *Utj = p.Ut + (long)j * n;
            const double *Li = p.L + (long)i * p.ldl, *Etj = p.Et + (long)j * m;
            double a = 0.0, b = 0.0;
            for (int q = lane; q < j; q += 32) a = fma(__ldcg(Ci + q), Utj[q], a);
            for (int q = lane; q < i; q += 32) b = fma(Li[q], __ldcg(Etj + q), b);
            a = warp_sum(a);
            const double c0 = warp_sum(b);
            if (lane == 0) {
                const double y = p.X[(long)i * p.ldx + j] + a + c0;
                double z = rint(y);
                const double e = z - y;
                if (!(fabs(y) < 2147483648.0)) {
                    report(p.info, isfinite(y) ? GPTQ2D_ERR_INT_OVERFLOW : GPTQ2D_ERR_NONFINITE, i, j, 0);
                    z = 0.0;
                }
                p.Z[(long)i * p.ldz + j] = (int)z;
                if (p.E) p.E[(long)i * p.lde + j] = e;
                p.Et[(long)j * m + i] = e;
                p.C[(long)i * n + j] = c0 + e;
                max_abs_e = fmax(max_abs_e, fabs(e));
            }
        }
        ok = grid_barrier(p.sync, nb, p.info, s);
    }

    max_abs_e = fmax(max_abs_e, 0.0);
    for (int o = 16; o > 0; o >>= 1) max_abs_e = fmax(max_abs_e, __shfl_xor_sync(0xffffffffu, max_abs_e, o));
    if (lane == 0) red[warp] = max_abs_e;
    __syncthreads();
    if (tid == 0) {
        double v = 0.0;
        for (int w = 0; w < PULL_THREADS / 32; ++w) v = fmax(v, red[w]);
        atomic_max_nonneg_double(p.max_abs_e, v);
    }
}

static size_t pad256(size_t x) { return (x + 255) / 256 * 256; }

size_t round_pull_workspace_bytes(int m, int n) {
    return 256 + 2 * pad256((size_t)m * n * 8) + pad256((size_t)n * n * 8);
}

int launch_round_pull(const PullParams &pin, void *ws, cudaStream_t stream) {
    PullParams p = pin;
    char *w = static_cast<char *>(ws);
    unsigned *sync = reinterpret_cast<unsigned *>(w);
    p.sync.count = sync;
    p.sync.gen = sync + 1;
    p.sync.abort = sync + 2;
    p.max_abs_e = reinterpret_cast<double *>(w + 64);
    p.C = reinterpret_cast<double *>(w + 256);
    p.Et = reinterpret_cast<double *>(w + 256 + pad256((size_t)p.m * p.n * 8));
    p.Ut = reinterpret_cast<double *>(w + 256 + 2 * pad256((size_t)p.m * p.n * 8));
    if (cudaMemsetAsync(w, 0, 256, stream) != cudaSuccess) return GPTQ2D_ERR_CUDA;
    int dev = 0, sms = 0, per_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return GPTQ2D_ERR_CUDA;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return GPTQ2D_ERR_CUDA;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, round_pull_kernel, PULL_THREADS, 0) != cudaSuccess ||
        per_sm < 1)
        return GPTQ2D_ERR_CUDA;
    dim3 grid(sms * per_sm), block(PULL_THREADS);
    void *args[] = {&p};
    if (cudaLaunchCooperativeKernel((const void *)round_pull_kernel, grid, block, args, 0, stream) != cudaSuccess)
        return GPTQ2D_ERR_CUDA;
    return GPTQ2D_OK;
}

}  // namespace gptq2d
