// gptq2d_round_static: the tiled sweep for callers that cannot allocate device memory.
//
// Some callers of this library run where cudaMalloc is off the table: inside a region that
// is being captured into a CUDA graph, inside a memory-pool-managed framework step that
// forbids raw allocations, or in a real-time loop that must not touch the allocator.  For
// them this entry point needs no workspace argument: the sweep's scratch (the E and C = L E
// buffers plus the per-tile flags and the ready ring) lives in a file-scope device array
// that is part of the library image.  Every GPU that loads the library therefore holds
// GPTQ2D_STATIC_WORKSPACE_BYTES of device memory until the process exits; the maximum
// problem size is kept modest for that reason.
//
// In host code the array's name is only a stand-in for the device symbol, not a device
// address, so the address is looked up once per device with cudaGetSymbolAddress (below)
// and that pointer is what the kernel receives.
#include <mutex>
#include "common.cuh"
#include "round_internal.cuh"

namespace gptq2d {

constexpr int STATIC_MAX_DIM = GPTQ2D_STATIC_MAX_DIM;                       // m, n <= 512
constexpr size_t STATIC_BYTES = GPTQ2D_STATIC_WORKSPACE_BYTES;

static __device__ __align__(256) unsigned char g_static_workspace[STATIC_BYTES];

constexpr int MAX_DEVICES = 64;
static std::mutex g_setup_mutex;
static void *g_static_ptr[MAX_DEVICES];       // device address of the array, per device; 0 = not looked up yet

__global__ void static_margin_kernel(const double *max_abs_e, double *min_margin) { *min_margin = 0.5 - *max_abs_e; }

// Looks the symbol up on the CURRENT device the first time that device is seen.
static int static_workspace_for_current_device(void **out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return GPTQ2D_ERR_CUDA;
    if (dev < 0 || dev >= MAX_DEVICES) return GPTQ2D_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_static_ptr[dev]) {
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_workspace) != cudaSuccess || !ptr) return GPTQ2D_ERR_CUDA;
        g_static_ptr[dev] = ptr;
    }
    *out = g_static_ptr[dev];
    return GPTQ2D_OK;
}

}  // namespace gptq2d

using namespace gptq2d;

extern "C" int gptq2d_round_static(int m, int n, const double *X, long ldx, const double *L, long ldl,
                                   const double *U, long ldu, int32_t *Z, long ldz, double *E, long lde,
                                   double *min_margin, int *info, void *stream_) {
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (m < 1 || n < 1 || !X || !L || !U || !Z) return GPTQ2D_ERR_INVALID_ARG;
    if (m > STATIC_MAX_DIM || n > STATIC_MAX_DIM) return GPTQ2D_ERR_TOO_LARGE;
    if (ldx < n || ldl < m || ldu < n || ldz < n || (E && lde < n)) return GPTQ2D_ERR_INVALID_ARG;
    auto al = [](const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; };
    if (!al(X, 8) || !al(L, 8) || !al(U, 8) || !al(Z, 4) || !al(E, 8) || !al(min_margin, 8)) return GPTQ2D_ERR_INVALID_ARG;
    if (round_tiled_workspace_bytes(m, n) > STATIC_BYTES) return GPTQ2D_ERR_TOO_LARGE;
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return GPTQ2D_ERR_CUDA;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return GPTQ2D_ERR_CUDA;
    if (major != 10) return GPTQ2D_ERR_UNSUPPORTED_DEVICE;
    void *ws = nullptr;
    int st = static_workspace_for_current_device(&ws);      // first call on a device: symbol look-up
    if (st != GPTQ2D_OK) return st;
    if (info && cudaMemsetAsync(info, 0, 4 * sizeof(int), stream) != cudaSuccess) return GPTQ2D_ERR_CUDA;
    TiledParams p{};
    p.m = m; p.n = n;
    p.X = X; p.ldx = ldx; p.L = L; p.ldl = ldl; p.U = U; p.ldu = ldu;
    p.Z = Z; p.ldz = ldz; p.E = E; p.lde = lde; p.info = info;
    // launch_round_tiled clears the header, flags, counters and the ready ring of the shared array
    // (everything that must start at zero) on `stream` before the kernel; E and C need no clearing.
    st = launch_round_tiled(p, ws, STATIC_BYTES, stream);
    if (st != GPTQ2D_OK) return st;
    if (min_margin) {
        static_margin_kernel<<<1, 1, 0, stream>>>(workspace_max_abs_e(ws), min_margin);
        if (cudaGetLastError() != cudaSuccess) return GPTQ2D_ERR_CUDA;
    }
    return GPTQ2D_OK;
}

extern "C" size_t gptq2d_round_static_max_dim(void) { return (size_t)STATIC_MAX_DIM; }
