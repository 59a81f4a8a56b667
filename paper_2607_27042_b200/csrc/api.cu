// C ABI of the library: argument checks and dispatch.  See include/gptq2d.h.
#include <cuda_runtime.h>
#include "common.cuh"
#include "round_internal.cuh"
#include "factor.cuh"
#include "gemm.cuh"
#include <algorithm>
#include <atomic>
#include <mutex>
#include <vector>

namespace gptq2d {
size_t objective_workspace_bytes(int m, int n);
int launch_objective(int m, int n, const double *X, long ldx, const int *Z, long ldz, const double *A, long lda,
                     const double *B, long ldb, double *obj, void *ws, cudaStream_t stream);

__global__ void margin_kernel(const double *max_abs_e, double *min_margin) { *min_margin = 0.5 - *max_abs_e; }

#ifdef GPTQ2D_CHECKED
// Self-test of the checked build's index check: one deliberately out-of-range index (7 of 3, site 999) goes
// through CI(); it must come back redirected to 0 and be recorded in `info`.  Touches no memory but `info`.
__global__ void check_selftest_kernel(int *info, int *redirected) {
    CHECKED_SET_INFO(info);
    *redirected = (int)CI(7, 3, 999);
}
#endif

// Test hooks (gptq2d_internal_test_hook): host-made failures only.
static std::atomic<long> g_hook_withhold_last_step{0};   // one-shot: the next pipelined host call does not announce its last copy step
static std::atomic<long> g_hook_panel_spin_limit{0};      // polls a task waits for its copy step (0: default)

static bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

static int check_device() {
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return GPTQ2D_ERR_CUDA;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return GPTQ2D_ERR_CUDA;
    return major == 10 ? GPTQ2D_OK : GPTQ2D_ERR_UNSUPPORTED_DEVICE;
}

static size_t pad256(size_t x) { return (x + 255) / 256 * 256; }

// ---- the library's second stream ---------------------------------------------------------------
// A second stream (per device, created on first use).  In the host entry point it carries the
// host-to-device copies while the sweep kernel already runs on the caller's stream; in gptq2d_factor
// it carries the B side.  In the host entry point the copy stream announces each 128-row panel
// with a stream-ordered 32-bit write (driver entry point looked up through the runtime, so the
// library has no link-time dependency on the driver library).
typedef int (*StreamWriteValue32Fn)(cudaStream_t, unsigned long long, unsigned int, unsigned int);
typedef int (*StreamWaitValue32Fn)(cudaStream_t, unsigned long long, unsigned int, unsigned int);
struct HostPipe {
    cudaStream_t copy = nullptr;
    cudaEvent_t inputs_free = nullptr, copies_done = nullptr;
    FactorLookahead look[2] = {};            // per side of the set-up: spine stream and its events (spine == NULL: none)
    static constexpr int POOL = 8;           // streams that carry independent problems of a batched set-up
    cudaStream_t pool[POOL] = {};
    cudaEvent_t pool_done[POOL] = {};
    bool pool_ok = false;
    StreamWriteValue32Fn write32 = nullptr;
    StreamWaitValue32Fn wait32 = nullptr;    // stream-ordered wait until a device word is >= a value
    bool tried = false;
    std::mutex enqueue;         // one pipelined call at a time enqueues on the shared copy stream and events
};
static std::mutex g_pipe_mutex;
static HostPipe g_pipe[64];

// NULL if the device cannot do it (then the caller copies everything first, as before)
static HostPipe *host_pipe() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(g_pipe_mutex);
    HostPipe &hp = g_pipe[dev];
    if (!hp.tried) {
        hp.tried = true;
        void *fn = nullptr, *fnw = nullptr;
        cudaDriverEntryPointQueryResult qr = cudaDriverEntryPointSymbolNotFound;
        bool ok = cudaGetDriverEntryPoint("cuStreamWriteValue32", &fn, cudaEnableDefault, &qr) == cudaSuccess &&
                  qr == cudaDriverEntryPointSuccess && fn != nullptr;
        ok = ok && cudaGetDriverEntryPoint("cuStreamWaitValue32", &fnw, cudaEnableDefault, &qr) == cudaSuccess &&
             qr == cudaDriverEntryPointSuccess && fnw != nullptr;
        ok = ok && cudaStreamCreateWithFlags(&hp.copy, cudaStreamNonBlocking) == cudaSuccess;
        ok = ok && cudaEventCreateWithFlags(&hp.inputs_free, cudaEventDisableTiming) == cudaSuccess;
        ok = ok && cudaEventCreateWithFlags(&hp.copies_done, cudaEventDisableTiming) == cudaSuccess;
        for (int sd = 0; ok && sd < 2; ++sd) {
            FactorLookahead &lk = hp.look[sd];
            cudaEvent_t *ev[5] = {&lk.fork, &lk.join, &lk.panel, &lk.t2[0], &lk.t2[1]};
            // highest priority: the one-CTA spine kernels must get an SM as soon as one is free, ahead of the
            // queued CTAs of the large updates
            int prio_lo = 0, prio_hi = 0;
            bool lok = cudaDeviceGetStreamPriorityRange(&prio_lo, &prio_hi) == cudaSuccess &&
                       cudaStreamCreateWithPriority(&lk.spine, cudaStreamNonBlocking, prio_hi) == cudaSuccess;
            for (int e = 0; lok && e < 5; ++e) lok = cudaEventCreateWithFlags(ev[e], cudaEventDisableTiming) == cudaSuccess;
            if (!lok) lk.spine = nullptr;        // the set-up then runs that side on one stream
        }
        hp.pool_ok = ok;
        for (int k = 0; hp.pool_ok && k < HostPipe::POOL; ++k)
            hp.pool_ok = cudaStreamCreateWithFlags(&hp.pool[k], cudaStreamNonBlocking) == cudaSuccess &&
                         cudaEventCreateWithFlags(&hp.pool_done[k], cudaEventDisableTiming) == cudaSuccess;
        if (ok) { hp.write32 = reinterpret_cast<StreamWriteValue32Fn>(fn); hp.wait32 = reinterpret_cast<StreamWaitValue32Fn>(fnw); }
        (void)cudaGetLastError();
    }
    return hp.write32 ? &hp : nullptr;
}

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
        case GPTQ2D_ERR_CHECK: return "checked build: an index left its array";
        default: return "unknown status";
    }
}

size_t gptq2d_factor_workspace_bytes(int m, int n) {
    if (m < 1 || n < 1) return 0;
    return factor_workspace_bytes(m, n);
}

// Both sides of one problem, arguments already checked, `info` already cleared.
static int factor_pair(int m, int n, const double *A, long lda, const double *B, long ldb, double *L, long ldl, double *U,
                       long ldu, double *dL, double *dU, void *workspace, int *info, cudaStream_t stream) {
    // The two sides are independent.  Each has a serial spine (one small diagonal-block kernel per 128
    // rows, between the panel and trailing updates) that leaves most SMs idle, so the B side runs on a
    // second stream and its GEMMs fill the gaps of the A side and vice versa.
    char *wsB = static_cast<char *>(workspace) + factor_side_workspace_bytes(m);
    HostPipe *hp = (A && B) ? host_pipe() : nullptr;
    if (!hp) {
        int st = factor_one_side(m, A, lda, 0, L, ldl, dL, workspace, info, stream, nullptr);
        if (st != GPTQ2D_OK) return st;
        return factor_one_side(n, B, ldb, 1, U, ldu, dU, wsB, info, stream, nullptr);
    }
    std::unique_lock<std::mutex> lock(hp->enqueue);
    if (cudaEventRecord(hp->inputs_free, stream) != cudaSuccess ||
        cudaStreamWaitEvent(hp->copy, hp->inputs_free, 0) != cudaSuccess)
        return GPTQ2D_ERR_CUDA;
    int st = factor_one_side(m, A, lda, 0, L, ldl, dL, workspace, info, stream, hp->look[0].spine ? &hp->look[0] : nullptr);
    int st2 = factor_one_side(n, B, ldb, 1, U, ldu, dU, wsB, info, hp->copy, hp->look[1].spine ? &hp->look[1] : nullptr);
    // join even if an enqueue failed, so that nothing of this call is left running behind the caller's stream
    if (cudaEventRecord(hp->copies_done, hp->copy) != cudaSuccess ||
        cudaStreamWaitEvent(stream, hp->copies_done, 0) != cudaSuccess)
        return GPTQ2D_ERR_CUDA;
    return st != GPTQ2D_OK ? st : st2;
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
    return factor_pair(m, n, A, lda, B, ldb, L, ldl, U, ldu, dL, dU, workspace, info, stream);
}

static size_t factor_batched_table_bytes(int count) { return pad256((size_t)2 * count * sizeof(FactorSmallSide)); }
// a problem with a side of order > FACTOR_SMALL_MAX takes the blocked route of gptq2d_factor, both sides (an
// absent basis of that order too: its identity factor is then written by a grid-wide kernel, not by one CTA)
static bool factor_problem_is_large(const gptq2d_factor_problem_t &q) {
    return q.m > FACTOR_SMALL_MAX || q.n > FACTOR_SMALL_MAX;
}

size_t gptq2d_factor_batched_workspace_bytes(int count, const gptq2d_factor_problem_t *pr) {
    if (count < 1 || !pr) return 0;
    size_t large = 0;
    int nlarge = 0;
    for (int b = 0; b < count; ++b) {
        if (pr[b].m < 1 || pr[b].n < 1) return 0;
        if (factor_problem_is_large(pr[b])) {
            large = std::max(large, factor_workspace_bytes(pr[b].m, pr[b].n));
            ++nlarge;
        }
    }
    // several problems of the blocked route run side by side, each in a slot of its own
    large *= (size_t)std::min(nlarge, (int)HostPipe::POOL);
    return factor_batched_table_bytes(count) + large;
}

int gptq2d_factor_batched(int count, const gptq2d_factor_problem_t *pr, void *workspace, size_t workspace_bytes,
                          int *info, void *stream_) {
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (count < 1 || !pr) return GPTQ2D_ERR_INVALID_ARG;
    for (int b = 0; b < count; ++b) {
        const gptq2d_factor_problem_t &q = pr[b];
        if (q.m < 1 || q.n < 1 || !q.L || !q.U || q.ldl < q.m || q.ldu < q.n) return GPTQ2D_ERR_INVALID_ARG;
        if ((q.A && q.lda < q.m) || (q.B && q.ldb < q.n)) return GPTQ2D_ERR_INVALID_ARG;
        if (!aligned(q.A, 8) || !aligned(q.B, 8) || !aligned(q.L, 8) || !aligned(q.U, 8) || !aligned(q.dL, 8) ||
            !aligned(q.dU, 8))
            return GPTQ2D_ERR_INVALID_ARG;
    }
    if (!workspace || !aligned(workspace, 256) || workspace_bytes < gptq2d_factor_batched_workspace_bytes(count, pr))
        return GPTQ2D_ERR_WORKSPACE;
    int st = check_device();
    if (st != GPTQ2D_OK) return st;
    if (info && cudaMemsetAsync(info, 0, 4 * sizeof(int), stream) != cudaSuccess) return GPTQ2D_ERR_CUDA;
    // problems whose bases both have order <= FACTOR_SMALL_MAX (or are absent): one CTA per side, one launch
    std::vector<FactorSmallSide> small;
    small.reserve((size_t)2 * count);
    for (int b = 0; b < count; ++b) {
        const gptq2d_factor_problem_t &q = pr[b];
        if (factor_problem_is_large(q)) continue;
        small.push_back(FactorSmallSide{q.m, 0, b, q.A, q.lda, q.L, q.ldl, q.dL});
        small.push_back(FactorSmallSide{q.n, 1, b, q.B, q.ldb, q.U, q.ldu, q.dU});
    }
    char *w = static_cast<char *>(workspace);
    if (!small.empty()) {
        // pageable source: the copy is staged before the call returns, so the vector may go out of scope
        if (cudaMemcpyAsync(w, small.data(), small.size() * sizeof(FactorSmallSide), cudaMemcpyHostToDevice, stream) !=
            cudaSuccess)
            return GPTQ2D_ERR_CUDA;
        st = launch_factor_small((int)small.size(), reinterpret_cast<const FactorSmallSide *>(w), info, stream);
        if (st != GPTQ2D_OK) return st;
    }
    char *wl = w + factor_batched_table_bytes(count);
    size_t slot_bytes = 0;
    int nlarge = 0;
    for (int b = 0; b < count; ++b)
        if (factor_problem_is_large(pr[b])) {
            slot_bytes = std::max(slot_bytes, factor_workspace_bytes(pr[b].m, pr[b].n));
            ++nlarge;
        }
    HostPipe *hp = nlarge > 1 ? host_pipe() : nullptr;
    if (!hp || !hp->pool_ok) {
        // one problem (or no second stream): the two-stream route of gptq2d_factor, problem after problem
        for (int b = 0; b < count; ++b) {
            const gptq2d_factor_problem_t &q = pr[b];
            if (!factor_problem_is_large(q)) continue;
            st = factor_pair(q.m, q.n, q.A, q.lda, q.B, q.ldb, q.L, q.ldl, q.U, q.ldu, q.dL, q.dU, wl, info, stream);
            if (st != GPTQ2D_OK) return st;
        }
        return GPTQ2D_OK;
    }
    // Several problems: each is a chain of many small launches, so independent problems go to different
    // streams (round robin; a stream and its workspace slot are shared by every POOL-th problem, in order).
    std::unique_lock<std::mutex> lock(hp->enqueue);
    const int nslots = std::min(nlarge, (int)HostPipe::POOL);
    if (cudaEventRecord(hp->inputs_free, stream) != cudaSuccess) return GPTQ2D_ERR_CUDA;      // nothing enqueued yet
    int idx = 0, first_err = GPTQ2D_OK;
    for (int k = 0; k < nslots && first_err == GPTQ2D_OK; ++k)
        if (cudaStreamWaitEvent(hp->pool[k], hp->inputs_free, 0) != cudaSuccess) first_err = GPTQ2D_ERR_CUDA;
    for (int b = 0; b < count && first_err == GPTQ2D_OK; ++b) {
        const gptq2d_factor_problem_t &q = pr[b];
        if (!factor_problem_is_large(q)) continue;
        const int k = idx++ % nslots;
        char *wk = wl + (size_t)k * slot_bytes;
        int s1 = factor_one_side(q.m, q.A, q.lda, 0, q.L, q.ldl, q.dL, wk, info, hp->pool[k], nullptr);
        int s2 = factor_one_side(q.n, q.B, q.ldb, 1, q.U, q.ldu, q.dU, wk + factor_side_workspace_bytes(q.m), info,
                                 hp->pool[k], nullptr);
        if (first_err == GPTQ2D_OK) first_err = s1 != GPTQ2D_OK ? s1 : s2;
    }
    // join even if an enqueue failed, so that nothing of this call is left running behind the caller's stream
    // (every pool stream is joined before the first error is returned)
    for (int k = 0; k < nslots; ++k)
        if ((cudaEventRecord(hp->pool_done[k], hp->pool[k]) != cudaSuccess ||
             cudaStreamWaitEvent(stream, hp->pool_done[k], 0) != cudaSuccess) && first_err == GPTQ2D_OK)
            first_err = GPTQ2D_ERR_CUDA;
    return first_err;
}

size_t gptq2d_round_workspace_bytes(int m, int n, int precision) {
    if (m < 1 || n < 1) return 0;
    if (precision == GPTQ2D_FP64) return round_tiled_workspace_bytes(m, n);
    if (precision == GPTQ2D_FP32) return round_tiled_f32_workspace_bytes(m, n);
    if (precision == GPTQ2D_FP32_UNTILED) return round_untiled_workspace_bytes(m, n, true);
    if (precision == GPTQ2D_FP64_UNTILED) return round_untiled_workspace_bytes(m, n, false);
    if (precision == GPTQ2D_FP64_PULL) return round_pull_workspace_bytes(m, n);
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
    if (precision != GPTQ2D_FP64 && precision != GPTQ2D_FP32 && precision != GPTQ2D_FP64_UNTILED &&
        precision != GPTQ2D_FP64_PULL && precision != GPTQ2D_FP32_UNTILED)
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
    } else if (precision == GPTQ2D_FP32) {
        TiledParams p{};
        p.m = m; p.n = n;
        p.X = X; p.ldx = ldx; p.L = L; p.ldl = ldl; p.U = U; p.ldu = ldu;
        p.Z = Z; p.ldz = ldz; p.E = E; p.lde = lde; p.info = info;
        st = launch_round_tiled_f32(p, workspace, workspace_bytes, stream);
    } else if (precision == GPTQ2D_FP64_PULL) {
        PullParams p{};
        p.m = m; p.n = n;
        p.X = X; p.ldx = ldx; p.L = L; p.ldl = ldl; p.U = U; p.ldu = ldu;
        p.Z = Z; p.ldz = ldz; p.E = E; p.lde = lde; p.info = info;
        st = launch_round_pull(p, workspace, stream);
    } else {
        UntiledParams p{};
        p.m = m; p.n = n;
        p.X = X; p.ldx = ldx; p.L = L; p.ldl = ldl; p.U = U; p.ldu = ldu;
        p.Z = Z; p.ldz = ldz; p.E = E; p.lde = lde; p.info = info;
        st = launch_round_untiled(p, precision == GPTQ2D_FP32_UNTILED, workspace, stream);
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
    HostPipe *hp = (precision == GPTQ2D_FP64) ? host_pipe() : nullptr;
    std::unique_lock<std::mutex> pipe_lock;
    bool z_direct = false;
    if (hp) {
        pipe_lock = std::unique_lock<std::mutex>(hp->enqueue);
        // Pipelined: the sweep starts at once and the inputs follow in steps (see below; of L and U only the
        // triangles the sweep reads).  The kernel holds back each task until its step has arrived.
        unsigned *dpanels = reinterpret_cast<unsigned *>(p + 128);
        if (cudaMemsetAsync(dpanels, 0, sizeof(unsigned), stream) != cudaSuccess) return GPTQ2D_ERR_CUDA;
        const int ntm_rows = (m + 127) / 128, ntn_cols = (n + 127) / 128;
        unsigned *rowdone = round_tiled_rowdone(w, m, n);
        if (cudaMemsetAsync(rowdone, 0, (size_t)ntm_rows * sizeof(unsigned), stream) != cudaSuccess) return GPTQ2D_ERR_CUDA;
        // the copies may overwrite dX, dL, dU only after everything queued on `stream` so far is done
        if (cudaEventRecord(hp->inputs_free, stream) != cudaSuccess ||
            cudaStreamWaitEvent(hp->copy, hp->inputs_free, 0) != cudaSuccess)
            return GPTQ2D_ERR_CUDA;
        if (hinfo) { hinfo[0] = hinfo[1] = hinfo[2] = hinfo[3] = 0; }
        if (cudaMemsetAsync(dinfo, 0, 4 * sizeof(int), stream) != cudaSuccess) return GPTQ2D_ERR_CUDA;
        TiledParams tp{};
        tp.m = m; tp.n = n;
        tp.X = dX; tp.ldx = n; tp.L = dL; tp.ldl = m; tp.U = dU; tp.ldu = n;
        tp.Z = dZ; tp.ldz = n; tp.E = hE ? dE : nullptr; tp.lde = n; tp.info = dinfo;
        // Z goes back row of tiles by row of tiles while the sweep still runs, if hZ is pinned: the copy stream
        // waits (stream-ordered) until the kernel has counted every tile of a row as swept, then copies its rows.
        cudaPointerAttributes za{};
        const bool z_pinned = cudaPointerGetAttributes(&za, hZ) == cudaSuccess && za.type == cudaMemoryTypeHost;
        (void)cudaGetLastError();
        tp.panels_ready = dpanels;
        tp.panel_spin_limit = (unsigned long long)g_hook_panel_spin_limit.load();
        const bool withhold_last = g_hook_withhold_last_step.exchange(0) != 0;
        int st = launch_round_tiled(tp, w, inner, stream);
        if (st != GPTQ2D_OK) return st;
        // Every failure from here on leaves through this exit: the kernel and the copy stream's waits are
        // released (all copy steps "announced", every tile row "swept"), both streams are drained, and
        // only then does the call return, so nothing of it runs on behind the caller's back.
        auto fail_out = [&]() {
            (void)hp->write32(hp->copy, (unsigned long long)reinterpret_cast<uintptr_t>(dpanels), 0x7fffffffu, 0u);
            (void)cudaMemsetAsync(rowdone, 0x7f, (size_t)ntm_rows * sizeof(unsigned), stream);
            (void)cudaStreamSynchronize(stream);
            (void)cudaStreamSynchronize(hp->copy);
            (void)cudaGetLastError();
            return (int)GPTQ2D_ERR_CUDA;
        };
        // From here until the copies are queued the kernel is waiting for this thread: nothing that could
        // block on the device (a first launch of another kernel loads its module, which waits for running
        // kernels) may come in between.
        // Step s sends the blocks of X on block anti-diagonal s, block row s of L and block column s of U
        // (COPY_BLOCK x COPY_BLOCK blocks): the order in which the wavefront of the sweep needs them.
        const int CB = COPY_BLOCK, nbm = (m + CB - 1) / CB, nbn = (n + CB - 1) / CB;
        auto copy2d = [&](double *dst, const double *src, size_t ld, int rows, int cols) {
            if (rows <= 0 || cols <= 0) return true;
            return cudaMemcpy2DAsync(dst, ld * 8, src, ld * 8, (size_t)cols * 8, rows, cudaMemcpyHostToDevice,
                                     hp->copy) == cudaSuccess;
        };
        auto extent = [&](int b, int total) { return total - b * CB < CB ? total - b * CB : CB; };
        bool ok = true;
        for (int step = 0; step < nbm + nbn - 1 && ok; ++step) {
            const int lo = step - nbn + 1 > 0 ? step - nbn + 1 : 0, hi = step < nbm - 1 ? step : nbm - 1;
            for (int bi = lo; bi <= hi && ok; ++bi) {
                const int bj = step - bi;
                const size_t off = (size_t)bi * CB * n + (size_t)bj * CB;
                ok = copy2d(dX + off, hX + off, n, extent(bi, m), extent(bj, n));
            }
            if (step < nbm)       // rows of block row `step`, columns up to the end of the diagonal block
                ok = ok && copy2d(dL + (size_t)step * CB * m, hL + (size_t)step * CB * m, m, extent(step, m),
                                  (step + 1) * CB < m ? (step + 1) * CB : m);
            if (step < nbn)       // columns of block column `step`, rows down to the end of the diagonal block
                ok = ok && copy2d(dU + (size_t)step * CB, hU + (size_t)step * CB, n,
                                  (step + 1) * CB < n ? (step + 1) * CB : n, extent(step, n));
            // (a test may withhold the announcement of the last step: the tasks that need it then run into
            // their bounded wait and the call reports GPTQ2D_ERR_DEVICE_TIMEOUT)
            if (!(withhold_last && step == nbm + nbn - 2))
                ok = ok && hp->write32(hp->copy, (unsigned long long)reinterpret_cast<uintptr_t>(dpanels),
                                       (unsigned)(step + 1), 0u) == 0;
        }
        if (!ok) return fail_out();
        // whatever happens in the kernel, no wait of the copy stream may outlast it
        if (z_pinned && cudaMemsetAsync(rowdone, 0x7f, (size_t)ntm_rows * sizeof(unsigned), stream) != cudaSuccess)
            return fail_out();
        if (hmin_margin) {
            margin_kernel<<<1, 1, 0, stream>>>(workspace_max_abs_e(w), dmargin);
            if (cudaGetLastError() != cudaSuccess) return fail_out();
        }
        if (z_pinned) {
            for (int I = 0; I < ntm_rows && ok; ++I) {
                const int rows = m - I * 128 < 128 ? m - I * 128 : 128;
                ok = hp->wait32(hp->copy, (unsigned long long)reinterpret_cast<uintptr_t>(rowdone + I),
                                (unsigned)ntn_cols, 0u /* >= */) == 0;
                ok = ok && cudaMemcpyAsync(hZ + (size_t)I * 128 * n, dZ + (size_t)I * 128 * n, (size_t)rows * n * 4,
                                           cudaMemcpyDeviceToHost, hp->copy) == cudaSuccess;
            }
            z_direct = ok;       // (Z is on its way back: no copy at the end)
        }
        if (cudaEventRecord(hp->copies_done, hp->copy) != cudaSuccess ||
            cudaStreamWaitEvent(stream, hp->copies_done, 0) != cudaSuccess || !ok)
            return fail_out();
        pipe_lock.unlock();
    } else
    if (cudaMemcpyAsync(dX, hX, (size_t)m * n * 8, cudaMemcpyHostToDevice, stream) != cudaSuccess ||
        cudaMemcpyAsync(dL, hL, (size_t)m * m * 8, cudaMemcpyHostToDevice, stream) != cudaSuccess ||
        cudaMemcpyAsync(dU, hU, (size_t)n * n * 8, cudaMemcpyHostToDevice, stream) != cudaSuccess)
        return GPTQ2D_ERR_CUDA;
    if (!hp) {
        int st = gptq2d_round(m, n, dX, n, dL, m, dU, n, dZ, n, hE ? dE : nullptr, n, hmin_margin ? dmargin : nullptr,
                              precision, w, inner, dinfo, stream_);
        if (st != GPTQ2D_OK) return st;
    }
    if (!z_direct && cudaMemcpyAsync(hZ, dZ, (size_t)m * n * 4, cudaMemcpyDeviceToHost, stream) != cudaSuccess)
        return GPTQ2D_ERR_CUDA;
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

int gptq2d_internal_test_hook(int key, long value) {
    if (key == 1) { g_hook_withhold_last_step.store(value != 0); return GPTQ2D_OK; }
    if (key == 2) { g_hook_panel_spin_limit.store(value > 0 ? value : 0); return GPTQ2D_OK; }
    if (key == 3) { gemm_set_tma_mode((int)value); return GPTQ2D_OK; }
    if (key == 4) { round_fused_set_mode((int)value); return GPTQ2D_OK; }
    if (key == 6) { round_tiled_f32_set_tma_mode((int)value); return GPTQ2D_OK; }
#ifdef GPTQ2D_CHECKED
    if (key == 5) {          // value: device int[5]; [0..3] receive the status words, [4] the redirected index
        int *dev = reinterpret_cast<int *>(static_cast<uintptr_t>(value));
        if (!dev || cudaMemsetAsync(dev, 0xff, 5 * sizeof(int), nullptr) != cudaSuccess ||
            cudaMemsetAsync(dev, 0, 4 * sizeof(int), nullptr) != cudaSuccess)
            return GPTQ2D_ERR_CUDA;
        check_selftest_kernel<<<1, 1>>>(dev, dev + 4);
        return cudaGetLastError() == cudaSuccess ? GPTQ2D_OK : GPTQ2D_ERR_CUDA;
    }
#endif
    return GPTQ2D_ERR_INVALID_ARG;
}

int gptq2d_internal_gemm(int transa, int transb, int M, int N, int K, double alpha, const double *A, long lda,
                         const double *B, long ldb, double beta, double *C, long ldc, void *stream_) {
    if (M < 1 || N < 1 || K < 1 || !A || !B || !C) return GPTQ2D_ERR_INVALID_ARG;
    if (lda < (transa ? M : K) || ldb < (transb ? K : N) || ldc < N) return GPTQ2D_ERR_INVALID_ARG;
    int st = check_device();
    if (st != GPTQ2D_OK) return st;
    GemmArgs g{};
    g.opA = transa ? OP_T : OP_N; g.opB = transb ? OP_T : OP_N;
    g.M = M; g.N = N; g.K = K; g.alpha = alpha; g.beta = beta;
    g.A = A; g.lda = lda; g.B = B; g.ldb = ldb; g.C = C; g.ldc = ldc; g.batch = 1;
    return launch_gemm(g, static_cast<cudaStream_t>(stream_)) == cudaSuccess ? GPTQ2D_OK : GPTQ2D_ERR_CUDA;
}

}  // extern "C"
