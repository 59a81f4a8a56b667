// Shared device helpers: status words, bounded waits, device-wide barrier.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include "../../include/gptq2d.h"

namespace gptq2d {

// Every device-side wait gives up after this many polls (each poll sleeps ~100 ns, so
// about a second), records where it stopped and raises the abort word that all other
// waits watch.  A kernel whose wait expired returns normally; the context stays usable.
constexpr unsigned long long SPIN_LIMIT = 8ull * 1000 * 1000;

__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned *p) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];\n" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_u32(unsigned *p, unsigned v) {
    asm volatile("st.release.gpu.global.u32 [%0], %1;\n" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ unsigned ld_relaxed_u32(const unsigned *p) {
    unsigned v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];\n" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// First error wins: info[0] is claimed with a CAS from 0.
__device__ __forceinline__ void report(int *info, int status, int a, int b, int c) {
    if (!info) return;
    if (atomicCAS(info, 0, status) == 0) {
        info[1] = a;
        info[2] = b;
        info[3] = c;
    }
}

// ---- checked build (-DGPTQ2D_CHECKED) --------------------------------------------------------------
// Every index that feeds a shared- or global-memory access of the sweep kernels goes through CI(index, limit,
// site).  In a normal build that is the index itself.  In a checked build an index outside [0, limit) is
// recorded -- first one wins -- in the call's status words as GPTQ2D_ERR_CHECK with the site number, the
// index and the limit, and the access is redirected to element 0 of its array: nothing traps, nothing faults,
// and the host reads the violation like any other device-side error.  (compute-sanitizer is not available
// where this library is developed; this is its stand-in for the small parity cases.)
#ifdef GPTQ2D_CHECKED
static __device__ int *g_chk_info;       // per translation unit; set by the kernels that use CI()
__device__ __forceinline__ long checked_index(long idx, long limit, int site) {
    if (idx >= 0 && idx < limit) return idx;
    report(g_chk_info, GPTQ2D_ERR_CHECK, site, (int)(idx > 2147483647L ? 2147483647L : (idx < -2147483647L ? -2147483647L : idx)),
           (int)(limit > 2147483647L ? 2147483647L : limit));
    return 0;
}
#define CI(idx, limit, site) checked_index((long)(idx), (long)(limit), (site))
#define CHECKED_SET_INFO(ptr) do { g_chk_info = (ptr); } while (0)
#else
#define CI(idx, limit, site) (idx)
#define CHECKED_SET_INFO(ptr) do { } while (0)
#endif

struct GridSync {
    unsigned *count;   // arrivals of the current generation
    unsigned *gen;     // generation number
    unsigned *abort;   // non-zero once any wait has given up
};

// Device-wide barrier for a co-resident (cooperatively launched) grid.
// Returns false if the wait expired or another CTA aborted.
__device__ __forceinline__ bool grid_barrier(const GridSync &gs, unsigned nblocks, int *info, int where) {
    __shared__ int ok_s;
    __syncthreads();
    if (threadIdx.x == 0) {
        int ok = 1;
        unsigned g = ld_acquire_u32(gs.gen);
        __threadfence();
        unsigned prev = atomicAdd(gs.count, 1u);
        if (prev == nblocks - 1) {
            *gs.count = 0u;
            __threadfence();
            st_release_u32(gs.gen, g + 1u);
        } else {
            unsigned long long it = 0;
            while (ld_acquire_u32(gs.gen) == g) {
                if (ld_relaxed_u32(gs.abort) != 0u) { ok = 0; break; }
                if (++it > SPIN_LIMIT) {
                    report(info, GPTQ2D_ERR_DEVICE_TIMEOUT, where, (int)blockIdx.x, 0);
                    atomicExch(gs.abort, 1u);
                    ok = 0;
                    break;
                }
                __nanosleep(100);
            }
        }
        if (ld_relaxed_u32(gs.abort) != 0u) ok = 0;
        ok_s = ok;
    }
    __syncthreads();
    return ok_s != 0;
}

__device__ __forceinline__ void atomic_max_nonneg_double(double *addr, double v) {
    // non-negative doubles order like their bit patterns
    atomicMax(reinterpret_cast<unsigned long long *>(addr), (unsigned long long)__double_as_longlong(v));
}

}  // namespace gptq2d
