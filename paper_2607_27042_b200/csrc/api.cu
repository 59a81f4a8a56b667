// C ABI of the library: argument checks and dispatch.  See include/gptq2d.h.
#include <cuda_runtime.h>
#include "common.cuh"
#include "round_internal.cuh"
#include <vector>

namespace gptq2d {
size_t factor_workspace_bytes(int m, int n);
int factor_one_side(int k, const double *M, long ldm, int side, double *out, long ldo, double *dinv, void *ws,
                    int *info, cudaStream_t stream);
size_t objective_workspace_bytes(int m, int n);
int launch_objective(int m, int n, const double *X, long ldx, const int *Z, long ldz, const double *A, long lda,
                     const double *B, long ldb, double *obj, void *ws, cudaStream_t stream);

__global__ void margin_kernel(const double *max_abs_e, double *min_margin) { *min_margin = 0.5 - *max_abs_e; }

static bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

static int check_device() {
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return GPTQ2D_ERR_CUDA;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return GPTQ2D_ERR_CUDA;
    return major == 10 ? GPTQ2D_OK : GPTQ2D_ERR_UNSUPPORTED_DEVICE;
}

static size_t pad256(size_t x) { return (x + 255) / 256 * 256; }

// host descriptors of a batched call -> internal launch parameters, with the argument checks of gptq2d_round
static int to_tiled(int count, const gptq2d_problem_t *pr, std::vector<TiledParams> &out) {
    if (count < 1 || !pr) return GPTQ2D_ERR_INVALID_ARG;
    if (count > GPTQ2D_BATCH_MAX_COUNT) return GPTQ2D_ERR_TOO_LARGE;
    out.resize(count);
    for (int b = 0; b < count; ++b) {
        const gptq2d_problem_t &q = pr[b];
        if (q.m < 1 || q.n < 1 || !q.X || !q.L || !q.U || !q.Z) return GPTQ2D_ERR_INVALID_ARG;
        if (q.ldx < q.n || q.ldl < q.m || q.ldu < q.n || q.ldz < q.n || (q.E && q.lde < q.n)) return GPTQ2D_ERR_INVALID_ARG;
        if (!aligned(q.X, 8) || !aligned(q.L, 8) || !aligned(q.U, 8) || !aligned(q.Z, 4) || !aligned(q.E, 8))
            return GPTQ2D_ERR_INVALID_ARG;
        if (q.m > GPTQ2D_BATCH_MAX_DIM || q.n > GPTQ2D_BATCH_MAX_DIM) return GPTQ2D_ERR_TOO_LARGE;
        TiledParams t{};
        t.m = q.m; t.n = q.n;
        t.X = q.X; t.ldx = q.ldx; t.L = q.L; t.ldl = q.ldl; t.U = q.U; t.ldu = q.ldu;
        t.Z = q.Z; t.ldz = q.ldz; t.E = q.E; t.lde = q.lde;
        out[b] = t;
    }
    return GPTQ2D_OK;
}
}  // namespace gptq2d

using namespace gptq2d;

extern "C" {

const char *gptq2d_status_string(int status) {
    switch (status) {
        case GPTQ2D_OK: return "ok";
        case GPTQ2D_ERR_INVALID_ARG: return "invalid argument";
        case GPTQ2D_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case GPTQ2D_ERR_UNSUPPORTED_DEVICE: return "device is not sm_100";
        case GPTQ2D_ERR_CUDA: return "CUDA runtime call failed";
        case GPTQ2D_ERR_NOT_SPD: return "Gram matrix not positive definite (singular basis)";
        case GPTQ2D_ERR_NONFINITE: return "non-finite value met while rounding";
        case GPTQ2D_ERR_INT_OVERFLOW: return "corrected value does not fit int32";
        case GPTQ2D_ERR_DEVICE_TIMEOUT: return "bounded device-side wait expired";
        case GPTQ2D_ERR_TOO_LARGE: return "problem larger than the static workspace allows";
        default: return "unknown status";
    }
}

size_t gptq2d_factor_workspace_bytes(int m, int n) {
    if (m < 1 || n < 1) return 0;
    return factor_workspace_bytes(m, n);
}

int gptq2d_factor(int m, int n, const double *A, long lda, const double *B, long ldb, double *L, long ldl, double *U,
                  long ldu, double *dL, double *dU, void *workspace, size_t workspace_bytes, int *info,
                  void *stream_) {
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (m < 1 || n < 1 || !L || !U || ldl < m || ldu < n) return GPTQ2D_ERR_INVALID_ARG;
    if ((A && lda < m) || (B && ldb < n)) return GPTQ2D_ERR_INVALID_ARG;
    if (!aligned(A, 8) || !aligned(B, 8) || !aligned(L, 8) || !aligned(U, 8)) return GPTQ2D_ERR_INVALID_ARG;
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < gptq2d_factor_workspace_bytes(m, n))
        return GPTQ2D_ERR_WORKSPACE;
    int st = check_device();
    if (st != GPTQ2D_OK) return st;
    if (info && cudaMemsetAsync(info, 0, 4 * sizeof(int), stream) != cudaSuccess) return GPTQ2D_ERR_CUDA;
    st = factor_one_side(m, A, lda, 0, L, ldl, dL, workspace, info, stream);
    if (st != GPTQ2D_OK) return st;
    return factor_one_side(n, B, ldb, 1, U, ldu, dU, workspace, info, stream);
}

size_t gptq2d_round_workspace_bytes(int m, int n, int precision) {
    if (m < 1 || n < 1) return 0;
    if (precision == GPTQ2D_FP64) return round_tiled_workspace_bytes(m, n);
    if (precision == GPTQ2D_FP32) return round_untiled_workspace_bytes(m, n, true);
    if (precision == GPTQ2D_FP64_UNTILED) return round_untiled_workspace_bytes(m, n, false);
    return 0;
}

int gptq2d_round(int m, int n, const double *X, long ldx, const double *L, long ldl, const double *U, long ldu,
                 int32_t *Z, long ldz, double *E, long lde, double *min_margin, int precision, void *workspace,
                 size_t workspace_bytes, int *info, void *stream_) {
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (m < 1 || n < 1 || !X || !L || !U || !Z) return GPTQ2D_ERR_INVALID_ARG;
    if (ldx < n || ldl < m || ldu < n || ldz < n || (E && lde < n)) return GPTQ2D_ERR_INVALID_ARG;
    if (!aligned(X, 8) || !aligned(L, 8) || !aligned(U, 8) || !aligned(Z, 4) || !aligned(E, 8) ||
        !aligned(min_margin, 8))
        return GPTQ2D_ERR_INVALID_ARG;
    if (precision != GPTQ2D_FP64 && precision != GPTQ2D_FP32 && precision != GPTQ2D_FP64_UNTILED)
        return GPTQ2D_ERR_INVALID_ARG;
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < gptq2d_round_workspace_bytes(m, n, precision))
        return GPTQ2D_ERR_WORKSPACE;
    int st = check_device();
    if (st != GPTQ2D_OK) return st;
    if (info && cudaMemsetAsync(info, 0, 4 * sizeof(int), stream) != cudaSuccess) return GPTQ2D_ERR_CUDA;

    if (precision == GPTQ2D_FP64) {
        TiledParams p{};
        p.m = m; p.n = n;
        p.X = X; p.ldx = ldx; p.L = L; p.ldl = ldl; p.U = U; p.ldu = ldu;
        p.Z = Z; p.ldz = ldz; p.E = E; p.lde = lde; p.info = info;
        st = launch_round_tiled(p, workspace, workspace_bytes, stream);
    } else {
        UntiledParams p{};
        p.m = m; p.n = n;
        p.X = X; p.ldx = ldx; p.L = L; p.ldl = ldl; p.U = U; p.ldu = ldu;
        p.Z = Z; p.ldz = ldz; p.E = E; p.lde = lde; p.info = info;
        st = launch_round_untiled(p, precision == GPTQ2D_FP32, workspace, stream);
    }
    if (st != GPTQ2D_OK) return st;
    if (min_margin) {
        margin_kernel<<<1, 1, 0, stream>>>(workspace_max_abs_e(workspace), min_margin);
        if (cudaGetLastError() != cudaSuccess) return GPTQ2D_ERR_CUDA;
    }
    return GPTQ2D_OK;
}

size_t gptq2d_round_batched_workspace_bytes(int count, const gptq2d_problem_t *problems) {
    std::vector<TiledParams> t;
    if (to_tiled(count, problems, t) != GPTQ2D_OK) return 0;
    return round_tiled_batched_workspace_bytes(count, t.data());
}

int gptq2d_round_batched(int count, const gptq2d_problem_t *problems, double *min_margin, void *workspace,
                         size_t workspace_bytes, int *info, void *stream_) {
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    std::vector<TiledParams> t;
    int st = to_tiled(count, problems, t);
    if (st != GPTQ2D_OK) return st;
    if (!aligned(min_margin, 8)) return GPTQ2D_ERR_INVALID_ARG;
    if (!workspace || !aligned(workspace, 256) ||
        workspace_bytes < round_tiled_batched_workspace_bytes(count, t.data()))
        return GPTQ2D_ERR_WORKSPACE;
    st = check_device();
    if (st != GPTQ2D_OK) return st;
    if (info && cudaMemsetAsync(info, 0, 4 * sizeof(int), stream) != cudaSuccess) return GPTQ2D_ERR_CUDA;
    return launch_round_tiled_batched(count, t.data(), min_margin, info, workspace, workspace_bytes, stream);
}

size_t gptq2d_round_host_workspace_bytes(int m, int n, int precision) {
    if (m < 1 || n < 1) return 0;
    size_t inner = gptq2d_round_workspace_bytes(m, n, precision);
    if (inner == 0) return 0;
    size_t x = pad256((size_t)m * n * 8), l = pad256((size_t)m * m * 8), u = pad256((size_t)n * n * 8);
    size_t z = pad256((size_t)m * n * 4), e = pad256((size_t)m * n * 8);
    return inner + x + l + u + z + e + 256;
}

int gptq2d_round_host(int m, int n, const double *hX, const double *hL, const double *hU, int32_t *hZ, double *hE,
                      double *hmin_margin, int precision, void *workspace, size_t workspace_bytes, int *hinfo,
                      void *stream_) {
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (m < 1 || n < 1 || !hX || !hL || !hU || !hZ) return GPTQ2D_ERR_INVALID_ARG;
    size_t need = gptq2d_round_host_workspace_bytes(m, n, precision);
    if (need == 0) return GPTQ2D_ERR_INVALID_ARG;
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < need) return GPTQ2D_ERR_WORKSPACE;
    size_t inner = gptq2d_round_workspace_bytes(m, n, precision);
    char *w = static_cast<char *>(workspace);
    char *p = w + pad256(inner);
    double *dX = reinterpret_cast<double *>(p); p += pad256((size_t)m * n * 8);
    double *dL = reinterpret_cast<double *>(p); p += pad256((size_t)m * m * 8);
    double *dU = reinterpret_cast<double *>(p); p += pad256((size_t)n * n * 8);
    int32_t *dZ = reinterpret_cast<int32_t *>(p); p += pad256((size_t)m * n * 4);
    double *dE = reinterpret_cast<double *>(p); p += pad256((size_t)m * n * 8);
    int *dinfo = reinterpret_cast<int *>(p);
    double *dmargin = reinterpret_cast<double *>(p + 64);
    if (cudaMemcpyAsync(dX, hX, (size_t)m * n * 8, cudaMemcpyHostToDevice, stream) != cudaSuccess ||
        cudaMemcpyAsync(dL, hL, (size_t)m * m * 8, cudaMemcpyHostToDevice, stream) != cudaSuccess ||
        cudaMemcpyAsync(dU, hU, (size_t)n * n * 8, cudaMemcpyHostToDevice, stream) != cudaSuccess)
        return GPTQ2D_ERR_CUDA;
    int st = gptq2d_round(m, n, dX, n, dL, m, dU, n, dZ, n, hE ? dE : nullptr, n, hmin_margin ? dmargin : nullptr,
                          precision, w, inner, dinfo, stream_);
    if (st != GPTQ2D_OK) return st;
    if (cudaMemcpyAsync(hZ, dZ, (size_t)m * n * 4, cudaMemcpyDeviceToHost, stream) != cudaSuccess) return GPTQ2D_ERR_CUDA;
    if (hE && cudaMemcpyAsync(hE, dE, (size_t)m * n * 8, cudaMemcpyDeviceToHost, stream) != cudaSuccess)
        return GPTQ2D_ERR_CUDA;
    if (hmin_margin && cudaMemcpyAsync(hmin_margin, dmargin, 8, cudaMemcpyDeviceToHost, stream) != cudaSuccess)
        return GPTQ2D_ERR_CUDA;
    if (hinfo && cudaMemcpyAsync(hinfo, dinfo, 16, cudaMemcpyDeviceToHost, stream) != cudaSuccess)
        return GPTQ2D_ERR_CUDA;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return GPTQ2D_ERR_CUDA;
    return GPTQ2D_OK;
}

size_t gptq2d_objective_workspace_bytes(int m, int n) {
    if (m < 1 || n < 1) return 0;
    return objective_workspace_bytes(m, n);
}

int gptq2d_objective(int m, int n, const double *X, long ldx, const int32_t *Z, long ldz, const double *A, long lda,
                     const double *B, long ldb, double *obj, void *workspace, size_t workspace_bytes, int *info,
                     void *stream_) {
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (m < 1 || n < 1 || !X || !Z || !obj || ldx < n || ldz < n) return GPTQ2D_ERR_INVALID_ARG;
    if ((A && lda < m) || (B && ldb < n)) return GPTQ2D_ERR_INVALID_ARG;
    if (!aligned(X, 8) || !aligned(Z, 4) || !aligned(A, 8) || !aligned(B, 8) || !aligned(obj, 8))
        return GPTQ2D_ERR_INVALID_ARG;
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < gptq2d_objective_workspace_bytes(m, n))
        return GPTQ2D_ERR_WORKSPACE;
    int st = check_device();
    if (st != GPTQ2D_OK) return st;
    if (info && cudaMemsetAsync(info, 0, 4 * sizeof(int), stream) != cudaSuccess) return GPTQ2D_ERR_CUDA;
    return launch_objective(m, n, X, ldx, Z, ldz, A, lda, B, ldb, obj, workspace, stream);
}

}  // extern "C"
