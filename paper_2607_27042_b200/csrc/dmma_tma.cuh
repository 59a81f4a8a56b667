// FP64 tensor-core (DMMA) tile contraction fed by TMA (cp.async.bulk.tensor) through an mbarrier ring.
//
// Same 128 x 128 register accumulator as dmma_gemm.cuh (8 warps as 2 x 4, each 64 x 32 = 8 x 4 fragments
// of mma.sync.m8n8k4.f64; tcgen05 has no f64 kind), but the operand slabs are not copied by the MMA
// threads: one elected lane issues a bulk tensor copy per slab and the hardware reports its bytes to
// a "full" mbarrier; the MMA warps wait on that barrier and release the stage through an "empty"
// barrier.  There is no CTA-wide barrier in the loop, so the eight warps drift apart freely, and no
// copy instruction or address arithmetic sits between the MMAs.
//
// Shared-memory layout.  A TMA box is dense, so the +4-double row pad of the cp.async path is not
// available; conflict-free fragment loads come from the 128-byte swizzle instead (the copy engine
// XORs the 16-byte chunk index of every 128-byte row with the row index mod 8) together with a
// permuted assignment of matrix rows / columns to MMA fragment rows / columns:
//   K-contiguous operand (row-major [mn][k], slab = 128 rows x 16 k = 128 rows x 128 B):
//       fragment f, lane group g  <->  mn = 16 (f >> 1) + 2 g + (f & 1)
//     the four rows a half-warp touches in one load then differ in bits 1-2 of (row & 7), so their four
//     32-byte pieces (k = kk .. kk+3) land in four different 32-byte bank groups: 16 lanes, 16 bank pairs.
//   MN-contiguous operand (row-major [k][mn], slab = 8 boxes of 16 k x 16 mn, each row 128 B):
//       fragment f, lane group g  <->  mn = 16 (f >> 1) + 4 (f & 1) + fmap(g),
//       fmap(g) = (g & 1) | ((g >> 1) & 1) << 3 | (g >> 2) << 1        (0 1 8 9 2 3 10 11)
//     within a half-warp the k index t = 0..3 permutes the low two chunk bits and the four columns
//     differ in (chunk bit 2, low bit): again 16 distinct bank pairs.
// The MMA does not care which matrix row a fragment row stands for; only the epilogue has to know
// (acc_row / acc_col below).
//
// Every wait on an mbarrier is bounded; a wait that runs out raises the caller's abort word, and the
// loop then waits (bounded again) for its own copies in flight before it returns.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include "dmma_gemm.cuh"

namespace gptq2d {

constexpr int TMA_BK = 16;                           // k-depth of a slab: 16 doubles = one 128-byte row
constexpr int TMA_TILE_DOUBLES = 128 * TMA_BK;       // one operand slab (16 KB), either layout
constexpr int TMA_STAGE_DOUBLES = 2 * TMA_TILE_DOUBLES;
constexpr unsigned TMA_STAGE_BYTES = TMA_STAGE_DOUBLES * 8;
constexpr unsigned long long MBAR_SPIN_LIMIT = 40ull * 1000 * 1000;   // polls (each a try_wait with a hardware time slice)

__device__ __forceinline__ unsigned smem_u32(const void *p) { return (unsigned)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(unsigned long long *bar, unsigned count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
// makes freshly initialised barriers visible to the copy engine (call once, before the CTA barrier that publishes them)
__device__ __forceinline__ void mbar_init_fence() {
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    asm volatile("fence.proxy.async;\n" ::: "memory");
}
// orders this thread's earlier generic-proxy accesses (and what it has acquired) against later copy-engine accesses
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async;\n" ::: "memory"); }

__device__ __forceinline__ void mbar_arrive(unsigned long long *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(unsigned long long *bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned long long *bar, unsigned parity) {
    unsigned ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0u;
}
__device__ __forceinline__ unsigned long long global_timer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;\n" : "=l"(t));
    return t;
}
// Bounded wait: gives up after `limit` polls or MBAR_WAIT_NS of wall time, whichever comes first, or when
// *abort has been raised by someone else.  Returns false if it gave up.
constexpr unsigned long long MBAR_WAIT_NS = 2000ull * 1000 * 1000;
__device__ __forceinline__ bool mbar_wait(unsigned long long *bar, unsigned parity, const unsigned *abort,
                                          unsigned long long limit = MBAR_SPIN_LIMIT) {
    if (mbar_try_wait(bar, parity)) return true;
    unsigned long long it = 0, t0 = 0;
    for (;;) {
        if (mbar_try_wait(bar, parity)) return true;
        if (++it > limit) return false;
        if ((it & 255) == 0) {
            if (abort && *reinterpret_cast<const volatile unsigned *>(abort) != 0u) return false;
            const unsigned long long now = global_timer_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > MBAR_WAIT_NS) return false;
        }
    }
}

// 3-D tiled copy global -> shared (own CTA), completion reported to `bar`.  Every CTA fetches its own copy.
__device__ __forceinline__ void tma_load_3d(void *dst, const CUtensorMap *map, int x, int y, int z, unsigned long long *bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];\n" ::"r"(
            smem_u32(dst)),
        "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y), "r"(z)
        : "memory");
}

// 2-D tiled copy global -> shared (own CTA), completion reported to `bar`
__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, int x, int y, unsigned long long *bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];\n" ::"r"(
            smem_u32(dst)),
        "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y)
        : "memory");
}

// ---- fragment <-> matrix index maps -----------------------------------------------------------
__device__ __forceinline__ int frag_map_mn(int g) { return (g & 1) | (((g >> 1) & 1) << 3) | ((g >> 2) << 1); }
// matrix row / column (inside the warp's 64- or 32-wide strip) that fragment f, position q (0..7) stands for
template <bool KCONTIG>
__device__ __forceinline__ int frag_index(int f, int q) {
    return KCONTIG ? (f >> 1) * 16 + 2 * q + (f & 1) : (f >> 1) * 16 + 4 * (f & 1) + frag_map_mn(q);
}
// shared-memory offset (doubles) of element (mn, k) of a slab, mn in 0..127, k in 0..15
template <bool KCONTIG>
__device__ __forceinline__ int slab_offset(int mn, int k) {
    if (KCONTIG) return mn * 16 + ((((k >> 1) ^ (mn & 7))) << 1) + (k & 1);
    return (mn >> 4) * 256 + k * 16 + (((((mn & 15) >> 1) ^ (k & 7))) << 1) + (mn & 1);
}

// One operand of a TMA-fed contraction as the kernel sees it.
struct TmaOperand {
    const CUtensorMap *map;    // K-contiguous: dims {K, MN, batch}, box {16, 128, 1}; MN-contiguous: dims {MN, K, batch}, box {16, 16, 1}
    int mn0;                   // first row (A) / column (B) of the CTA tile
    int k0;                    // first k of the contraction
    int z;                     // batch index
};

template <bool KCONTIG>
__device__ __forceinline__ void tma_issue_slab(double *dst, const TmaOperand &op, int k, unsigned long long *bar) {
    if (KCONTIG) {
        tma_load_3d(dst, op.map, k, op.mn0, op.z, bar);
    } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) tma_load_3d(dst + i * 256, op.map, op.mn0 + 16 * i, k, op.z, bar);
    }
}

// Ring state kept by the caller across calls (a far part of the sweep runs its contraction in several
// pieces): slab counter since the barriers were initialised.
struct TmaRing {
    unsigned long long *full;    // [NSTAGE]  arrival count 1 (+ transaction bytes)
    unsigned long long *empty;   // [NSTAGE]  arrival count = number of MMA warps
    double *stages;              // NSTAGE x TMA_STAGE_DOUBLES, 1024-byte aligned
    unsigned produced, consumed; // slabs issued / consumed so far (uniform over the MMA warps)
};

template <int NSTAGE, int NWARPS>
__device__ __forceinline__ void tma_ring_init(TmaRing &ring, unsigned long long *bars, double *stages, int tid_in_group) {
    ring.full = bars;
    ring.empty = bars + NSTAGE;
    ring.stages = stages;
    ring.produced = ring.consumed = 0;
    if (tid_in_group == 0) {
        for (int s = 0; s < NSTAGE; ++s) {
            mbar_init(ring.full + s, 1);
            mbar_init(ring.empty + s, NWARPS);
        }
        mbar_init_fence();
    }
}

// acc += A(128 x K) * B(K x 128), K = nk * 16, slabs out of range in any direction read as zeros.
// Called by the NWARPS = 8 MMA warps (warp = 0..7 inside the group) with uniform arguments.  The warp
// whose turn it is (slab index mod 8) issues the copy of the slab PREF ahead, half-way through its own
// MMAs of the current slab, once the stage it goes to has been released by every warp.
// Every fragment address is a per-lane offset computed once per call plus a compile-time constant.
// SLAB_BARRIER >= 0: the eight warps also meet at that named barrier once per slab.  They need not for
// correctness (the mbarriers order everything); it keeps the two warps of every SM sub-partition in
// step, and the fp64 tensor pipe is only saturated while both have MMAs to issue.
// Returns false if a wait ran out (abort raised; the accumulator is then meaningless).
template <bool A_KCONTIG, bool B_KCONTIG, int NSTAGE, int SLAB_BARRIER>
__device__ __forceinline__ bool gemm_tma_mainloop(Acc &acc, TmaRing &ring, const TmaOperand &A, const TmaOperand &B, int nk,
                                                  int warp, int lane, unsigned *abort) {
    constexpr int PREF = NSTAGE - 1;
    const int wm = warp >> 2, wn = warp & 3, g = lane >> 2, t = lane & 3;
    bool ok = true;
    unsigned issued_upto = 0;      // (issuing lanes) slabs of this call whose copies this lane has started
    // per-lane fragment offsets inside a stage: [fragment parity][k4-step]; fragment f adds (f >> 1) * 256 doubles
    // in either layout (16 rows of 16 doubles, or one 16 x 16 box)
    int offA[2][4], offB[2][4];
#pragma unroll
    for (int h = 0; h < 2; ++h)
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            offA[h][q] = slab_offset<A_KCONTIG>(wm * 64 + frag_index<A_KCONTIG>(h, g), 4 * q + t);
            offB[h][q] = slab_offset<B_KCONTIG>(wn * 32 + frag_index<B_KCONTIG>(h, g), 4 * q + t) + TMA_TILE_DOUBLES;
        }
    auto issue = [&](unsigned slab_from_start) {        // one lane
        const unsigned p = ring.produced + slab_from_start;
        const unsigned st = p % NSTAGE, use = p / NSTAGE;
        if (use > 0 && !mbar_wait(ring.empty + st, (use - 1) & 1u, abort)) { ok = false; return; }
        issued_upto = slab_from_start + 1;
        double *dst = ring.stages + (size_t)st * TMA_STAGE_DOUBLES;
        mbar_arrive_expect_tx(ring.full + st, TMA_STAGE_BYTES);
        tma_issue_slab<A_KCONTIG>(dst, A, A.k0 + (int)slab_from_start * TMA_BK, ring.full + st);
        tma_issue_slab<B_KCONTIG>(dst + TMA_TILE_DOUBLES, B, B.k0 + (int)slab_from_start * TMA_BK, ring.full + st);
    };
    // Every lane that may issue copies orders what it (and, through the caller's barrier, the CTA) has observed
    // in global memory before them: operands written earlier in this kernel by other CTAs were published with
    // release / acquire on flags, which says nothing about the copy engine's proxy until this fence.
    if (lane == 0) fence_proxy_async();
    // prologue: the first PREF slabs (issued by warp 0)
    if (warp == 0 && lane == 0)
        for (int s = 0; s < PREF && s < nk; ++s) issue((unsigned)s);
    int kt_stop = nk;
    for (int kt = 0; kt < nk; ++kt) {
        const unsigned c = ring.consumed + (unsigned)kt;
        const unsigned st = c % NSTAGE, use = c / NSTAGE;
        // (every warp meets the barrier nk times whatever happens: a warp that has given up keeps arriving)
        if (SLAB_BARRIER >= 0) asm volatile("bar.sync %0, %1;\n" ::"n"(SLAB_BARRIER < 0 ? 0 : SLAB_BARRIER), "n"(GEMM_THREADS) : "memory");
        if (kt >= kt_stop) continue;
        if (!__all_sync(0xffffffffu, mbar_wait(ring.full + st, use & 1u, abort))) { ok = false; kt_stop = kt; continue; }
        const double *S = ring.stages + (size_t)st * TMA_STAGE_DOUBLES;
        const bool my_turn = (kt + PREF < nk) && ((kt & 7) == warp);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            double af[8], bf[4];
#pragma unroll
            for (int a = 0; a < 8; ++a) af[a] = S[offA[a & 1][q] + (a >> 1) * 256];
#pragma unroll
            for (int b = 0; b < 4; ++b) bf[b] = S[offB[b & 1][q] + (b >> 1) * 256];
#pragma unroll
            for (int a = 0; a < 8; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) dmma_m8n8k4(acc.v[a][b][0], acc.v[a][b][1], af[a], bf[b]);
            if (q == 1 && my_turn) {
                if (lane == 0) issue((unsigned)(kt + PREF));
                __syncwarp();
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(ring.empty + st);
    }
    // `ok` is per lane (an issuing lane may have cleared it): make it warp-uniform
    ok = __all_sync(0xffffffffu, ok);
    if (!ok) {
        // A wait ran out: tell everybody, then give this lane's own copies that are still in flight a bounded
        // time to land before the caller leaves (shared memory must not be handed on under a running copy).
        if (abort && lane == 0) atomicExch(abort, 1u);
        for (unsigned s = (unsigned)kt_stop; s < issued_upto; ++s) {
            const unsigned c = ring.consumed + s;
            (void)mbar_wait(ring.full + c % NSTAGE, (c / NSTAGE) & 1u, nullptr, 1000000ull);
        }
    }
    ring.produced += (unsigned)nk;
    ring.consumed += (unsigned)nk;
    return ok;
}

// (row, column) inside the 128 x 128 CTA tile of accumulator element (a, b, j) of lane (g, t)
template <bool A_KCONTIG>
__device__ __forceinline__ int acc_row(int wm, int a, int g) { return wm * 64 + frag_index<A_KCONTIG>(a, g); }
template <bool B_KCONTIG>
__device__ __forceinline__ int acc_col(int wn, int b, int t, int j) { return wn * 32 + frag_index<B_KCONTIG>(b, 2 * t + j); }

}  // namespace gptq2d
