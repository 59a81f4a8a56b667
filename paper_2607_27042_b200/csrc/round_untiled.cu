// Algorithm 3 (GPTQ-2D) as written: one anti-diagonal per stage, natural row-major layout,
// out-of-range lanes masked (Section 5: a kernel needs no skew padding).  One persistent,
// cooperatively launched grid; the two forall phases of a stage are separated by a bounded
// device-wide barrier instead of kernel launches.
//
// Every push goes to HBM, so this kernel moves O(mn(m+n)) words and is memory bound -- it is
// the fp32 mode and an independent cross-check of the tiled kernel, not the fast path.
//
// Access pattern: the downward pushes of one stage are regrouped by TARGET ROW r: the
// targets (r, s-i) for all sources i < r are contiguous in memory, and so are the
// coefficients L[r][i]; the rightward push of source (i, j) walks row i and row j of U.
#include "common.cuh"
#include "round_internal.cuh"

namespace gptq2d {

constexpr int UT_THREADS = 512;
constexpr int UT_SEG = 4096;   // anti-diagonal entries staged in shared memory at a time

template <typename T>
__device__ __forceinline__ T round_half_even(T y);
template <>
__device__ __forceinline__ double round_half_even<double>(double y) { return rint(y); }
template <>
__device__ __forceinline__ float round_half_even<float>(float y) { return rintf(y); }

template <typename T>
__global__ void __launch_bounds__(UT_THREADS) round_untiled_kernel(UntiledParams p) {
    __shared__ T es[UT_SEG];
    __shared__ double red[UT_THREADS / 32];
    T *Y = reinterpret_cast<T *>(p.Ybuf);
    T *C = reinterpret_cast<T *>(p.Cbuf);
    const int m = p.m, n = p.n;
    const unsigned nb = gridDim.x;
    const int tid = threadIdx.x;
    double max_abs_e = 0.0;

    // Algorithm 3 lines 4-5: Y <- X, C <- 0
    for (long idx = (long)blockIdx.x * blockDim.x + tid; idx < (long)m * n; idx += (long)nb * blockDim.x) {
        int i = (int)(idx / n), j = (int)(idx % n);
        Y[idx] = (T)p.X[(long)i * p.ldx + j];
        C[idx] = (T)0;
    }
    bool ok = grid_barrier(p.sync, nb, p.info, -1);

    for (int s = 0; ok && s < m + n - 1; ++s) {
        const int lo = max(0, s - n + 1), hi = min(m - 1, s);
        // ---- phase 1: round, error, fold into C, push down (lines 8-13)
        for (int seg = lo; seg <= hi; seg += UT_SEG) {
            const int cnt = min(UT_SEG, hi - seg + 1);
            __syncthreads();
            for (int k = tid; k < cnt; k += blockDim.x) {
                int i = seg + k, j = s - i;
                T y = Y[(long)i * n + j];
                T z = round_half_even<T>(y);
                T e = z - y;
                es[k] = e;
                if ((unsigned)k % nb == blockIdx.x) {          // one CTA owns the entry's outputs
                    double yd = (double)y;
                    if (!(fabs(yd) < 2147483648.0)) {
                        report(p.info, isfinite(yd) ? GPTQ2D_ERR_INT_OVERFLOW : GPTQ2D_ERR_NONFINITE, i, j, 0);
                        z = (T)0;
                    }
                    p.Z[(long)i * p.ldz + j] = (int)z;
                    if (p.E) p.E[(long)i * p.lde + j] = (double)e;
                    max_abs_e = fmax(max_abs_e, fabs((double)e));
                    C[(long)i * n + j] += e;                   // L_ii = 1
                }
            }
            __syncthreads();
            // target row r receives L[r][i] * e_i at column s - i from every source i < r
            for (int r = seg + 1 + (int)blockIdx.x; r < m; r += (int)nb) {
                const int iend = min(seg + cnt - 1, r - 1);
                const double *Lr = p.L + (long)r * p.ldl;
                for (int i = seg + tid; i <= iend; i += blockDim.x) {
                    T mm = (T)Lr[i] * es[i - seg];
                    long at = (long)r * n + (s - i);
                    C[at] += mm;
                    Y[at] += mm;
                }
            }
        }
        ok = grid_barrier(p.sync, nb, p.info, 2 * s);
        if (!ok) break;
        // ---- phase 2: push right (lines 14-16); C_ij is final here
        for (int i = lo + (int)blockIdx.x; i <= hi; i += (int)nb) {
            const int j = s - i;
            const T c = C[(long)i * n + j];
            const double *Uj = p.U + (long)j * p.ldu;
            T *Yi = Y + (long)i * n;
            for (int q = j + 1 + tid; q < n; q += blockDim.x) Yi[q] += c * (T)Uj[q];
        }
        ok = grid_barrier(p.sync, nb, p.info, 2 * s + 1);
    }

    if (p.max_abs_e) {
        for (int o = 16; o > 0; o >>= 1) max_abs_e = fmax(max_abs_e, __shfl_xor_sync(0xffffffffu, max_abs_e, o));
        if ((tid & 31) == 0) red[tid >> 5] = max_abs_e;
        __syncthreads();
        if (tid == 0) {
            double v = 0.0;
            for (int w = 0; w < UT_THREADS / 32; ++w) v = fmax(v, red[w]);
            atomic_max_nonneg_double(p.max_abs_e, v);
        }
    }
}

size_t round_untiled_workspace_bytes(int m, int n, bool fp32) {
    size_t elt = fp32 ? 4 : 8;
    size_t buf = ((size_t)m * n * elt + 255) / 256 * 256;
    return 256 + 2 * buf;
}

int launch_round_untiled(const UntiledParams &pin, bool fp32, void *ws, cudaStream_t stream) {
    UntiledParams p = pin;
    size_t elt = fp32 ? 4 : 8;
    size_t buf = ((size_t)p.m * p.n * elt + 255) / 256 * 256;
    char *w = static_cast<char *>(ws);
    unsigned *sync = reinterpret_cast<unsigned *>(w);
    p.sync.count = sync;
    p.sync.gen = sync + 1;
    p.sync.abort = sync + 2;
    p.max_abs_e = reinterpret_cast<double *>(w + 64);
    p.Ybuf = w + 256;
    p.Cbuf = w + 256 + buf;
    if (cudaMemsetAsync(w, 0, 256, stream) != cudaSuccess) return GPTQ2D_ERR_CUDA;

    int dev = 0, sms = 0, per_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return GPTQ2D_ERR_CUDA;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return GPTQ2D_ERR_CUDA;
    const void *fn = fp32 ? (const void *)round_untiled_kernel<float> : (const void *)round_untiled_kernel<double>;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fn, UT_THREADS, 0) != cudaSuccess || per_sm < 1)
        return GPTQ2D_ERR_CUDA;
    dim3 grid(sms * per_sm), block(UT_THREADS);
    void *args[] = {&p};
    if (cudaLaunchCooperativeKernel(fn, grid, block, args, 0, stream) != cudaSuccess) return GPTQ2D_ERR_CUDA;
    return GPTQ2D_OK;
}

}  // namespace gptq2d
