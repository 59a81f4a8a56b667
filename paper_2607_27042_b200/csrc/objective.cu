// Objective of Eq. 7: || A (Z - X) B ||_F^2, as two GEMMs and a deterministic reduction.
#include "common.cuh"
#include "gemm.cuh"

namespace gptq2d {

__global__ void residual_kernel(int m, int n, const double *X, long ldx, const int *Z, long ldz, double *R, long ldr) {
    long idx = (long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (long)m * n) return;
    int i = (int)(idx / n), j = (int)(idx % n);
    R[(long)i * ldr + j] = (double)Z[(long)i * ldz + j] - X[(long)i * ldx + j];
}

__global__ void __launch_bounds__(1024) sum_partials_kernel(const double *part, int count, double *out) {
    __shared__ double red[32];
    double s = 0.0;
    for (int i = threadIdx.x; i < count; i += blockDim.x) s += part[i];   // fixed order per thread
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = s;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int w = 0; w < 32; ++w) t += red[w];
        *out = t;
    }
}

static inline long round_up(long x, long a) { return (x + a - 1) / a * a; }
void launch_sumsq_plain(const double *M, int m, int n, long ld, double *part, int *count, cudaStream_t s);

size_t objective_workspace_bytes(int m, int n) {
    long ld = round_up(n, 16);
    size_t mat = (size_t)m * ld * sizeof(double);
    size_t tiles = (size_t)((m + 127) / 128) * ((n + 127) / 128);
    return 2 * mat + round_up((long)(tiles * sizeof(double)), 256) + 256;
}

#define CK(x)                                          \
    do {                                               \
        if ((x) != cudaSuccess) return GPTQ2D_ERR_CUDA; \
    } while (0)

int launch_objective(int m, int n, const double *X, long ldx, const int *Z, long ldz, const double *A, long lda,
                     const double *B, long ldb, double *obj, void *ws, cudaStream_t stream) {
    const long ld = round_up(n, 16);
    const size_t mat = (size_t)m * ld;
    double *R = static_cast<double *>(ws);
    double *T1 = R + mat;
    double *part = T1 + mat;
    const int tiles = ((m + 127) / 128) * ((n + 127) / 128);
    long tot = (long)m * n;
    residual_kernel<<<(unsigned)((tot + 255) / 256), 256, 0, stream>>>(m, n, X, ldx, Z, ldz, R, ld);
    CK(cudaGetLastError());
    const double *left = R;
    if (A) {   // T1 = A R
        GemmArgs g{};
        g.opA = OP_N; g.opB = OP_N;
        g.M = m; g.N = n; g.K = m;
        g.alpha = 1.0; g.beta = 0.0;
        g.A = A; g.lda = lda; g.B = R; g.ldb = ld; g.C = T1; g.ldc = ld; g.batch = 1;
        CK(launch_gemm(g, stream));
        left = T1;
    }
    GemmArgs g{};   // sum of squares of left * B, or of left itself when B is the identity
    if (B) {
        g.opA = OP_N; g.opB = OP_N;
        g.M = m; g.N = n; g.K = n;
        g.alpha = 1.0; g.beta = 0.0;
        g.A = left; g.lda = ld; g.B = B; g.ldb = ldb; g.C = nullptr; g.ldc = ld; g.batch = 1;
        g.sumsq_partials = part;
        CK(launch_gemm(g, stream));
        sum_partials_kernel<<<1, 1024, 0, stream>>>(part, tiles, obj);
    } else {
        // || left ||_F^2 directly
        int count = 0;
        launch_sumsq_plain(left, m, n, ld, part, &count, stream);
        sum_partials_kernel<<<1, 1024, 0, stream>>>(part, count, obj);
    }
    CK(cudaGetLastError());
    return GPTQ2D_OK;
}

__global__ void __launch_bounds__(256) sumsq_rows_kernel(const double *M, int m, int n, long ld, double *part) {
    // one CTA per 128-row band: same partial count bound as the tile count
    __shared__ double red[8];
    int r0 = blockIdx.x * 128;
    double s = 0.0;
    for (int r = r0; r < min(m, r0 + 128); ++r)
        for (int c = threadIdx.x; c < n; c += blockDim.x) {
            double v = M[(long)r * ld + c];
            s = fma(v, v, s);
        }
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = s;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int w = 0; w < 8; ++w) t += red[w];
        part[blockIdx.x] = t;
    }
}

void launch_sumsq_plain(const double *M, int m, int n, long ld, double *part, int *count, cudaStream_t s) {
    int bands = (m + 127) / 128;
    sumsq_rows_kernel<<<bands, 256, 0, s>>>(M, m, n, ld, part);
    *count = bands;
}

}  // namespace gptq2d
