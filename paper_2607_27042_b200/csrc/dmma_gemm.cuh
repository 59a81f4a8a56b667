// FP64 tensor-core (DMMA) tile contraction for sm_100a.
//
// One CTA of 256 threads owns a 128 x 128 fp64 accumulator tile in registers (8 warps as
// 2 x 4, each warp 64 x 32 = 8 x 4 fragments of mma.sync.m8n8k4.f64) and streams the
// contraction dimension through shared memory in slabs of 16 with a cp.async pipeline.
// tcgen05 has no f64 kind, so the warp-level f64 mma is the tensor path for this dtype;
// measured on B200 it sustains the full 37.2 TFLOP/s, plain DFMA 33.7.
//
// Operand tiles in shared memory come in two layouts, chosen so that every fragment
// load (one double per lane) hits 16 distinct 8-byte bank pairs per half-warp:
//   K-contiguous  [row][k]   row stride LDK = 20 doubles  (20 mod 16 == 4)
//   MN-contiguous [k][col]   row stride LDN = 132 doubles (132 mod 16 == 4)
// An operand that is stored k-contiguous in global memory (A not transposed, or B
// transposed) uses the first, the other the second; both copy 16-byte chunks.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include "common.cuh"

namespace gptq2d {

constexpr int BM = 128;
constexpr int BN = 128;
constexpr int BK = 16;
constexpr int LDK = BK + 4;
constexpr int LDN = 128 + 4;
constexpr int TILE_KC = 128 * LDK;   // doubles in a K-contiguous tile   (2560)
constexpr int TILE_MN = BK * LDN;    // doubles in an MN-contiguous tile (2112)
constexpr int GEMM_THREADS = 256;

__device__ __forceinline__ void cp_async16(void *smem, const void *gmem, int src_bytes) {
    unsigned s = (unsigned)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(s), "l"(gmem), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async8(void *smem, const void *gmem, int src_bytes) {
    unsigned s = (unsigned)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8, %2;\n" ::"r"(s), "l"(gmem), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }

__device__ __forceinline__ void dmma_m8n8k4(double &c0, double &c1, double a, double b) {
    asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};\n"
                 : "+d"(c0), "+d"(c1)
                 : "d"(a), "d"(b));
}

// Describes one operand as seen by a CTA tile: element (r, c) of the logical
// (rows x K) [A] or (K x cols) [B] operand lives at ptr[r*ld + c] if !transposed
// storage, else ptr[c*ld + r].  `kcontig` says which index is contiguous in memory.
struct Operand {
    const double *ptr;   // already offset to the tile's first row/col and to k = 0
    long ld;
    int mn_valid;        // rows (A) or cols (B) of the 128-wide tile that exist
    bool aligned16;      // ptr 16-byte aligned and ld even
};

// Copies one 128 x 16 (K-contiguous) or 16 x 128 (MN-contiguous) slab into shared memory,
// zero-filling what lies outside [0, mn_valid) x [0, k_valid).
template <bool KCONTIG>
__device__ __forceinline__ void load_slab(double *smem, const Operand &op, int k0, int k_valid, int tid) {
    if (KCONTIG) {
        // global: row r (0..127) contiguous in k.  1024 chunks of 2 doubles.
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            int c = tid + i * GEMM_THREADS;
            int r = c >> 3, kk = (c & 7) * 2;
            double *dst = smem + CI(r * LDK + kk, TILE_KC - 1, 201);
            const double *src = op.ptr + (long)r * op.ld + (k0 + kk);
            int nv = (r < op.mn_valid) ? (k_valid - (k0 + kk)) : 0;   // doubles valid from kk
            nv = nv < 0 ? 0 : (nv > 2 ? 2 : nv);
            if (nv == 0) src = op.ptr;
            if (op.aligned16) {
                cp_async16(dst, src, nv * 8);
            } else {
                cp_async8(dst, src, nv >= 1 ? 8 : 0);
                cp_async8(dst + 1, nv >= 2 ? src + 1 : op.ptr, nv >= 2 ? 8 : 0);
            }
        }
    } else {
        // global: k row (0..15) contiguous in the 128 columns.
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            int c = tid + i * GEMM_THREADS;
            int kr = c >> 6, cc = (c & 63) * 2;
            double *dst = smem + CI(kr * LDN + cc, TILE_MN - 1, 202);
            const double *src = op.ptr + (long)(k0 + kr) * op.ld + cc;
            int nv = (k0 + kr < k_valid) ? (op.mn_valid - cc) : 0;
            nv = nv < 0 ? 0 : (nv > 2 ? 2 : nv);
            if (nv == 0) src = op.ptr;
            if (op.aligned16) {
                cp_async16(dst, src, nv * 8);
            } else {
                cp_async8(dst, src, nv >= 1 ? 8 : 0);
                cp_async8(dst + 1, nv >= 2 ? src + 1 : op.ptr, nv >= 2 ? 8 : 0);
            }
        }
    }
}

template <bool A_KCONTIG, bool B_KCONTIG>
struct SlabLayout {
    static constexpr int A_DOUBLES = A_KCONTIG ? TILE_KC : TILE_MN;
    static constexpr int B_DOUBLES = B_KCONTIG ? TILE_KC : TILE_MN;
    static constexpr int STAGE_DOUBLES = A_DOUBLES + B_DOUBLES;
};

// acc[a][b][0..1]: fragment (a, b) of the warp's 64 x 32 tile; element rows
// wm*64 + a*8 + (lane>>2), cols wn*32 + b*8 + (lane&3)*2 + {0,1}.
struct Acc {
    double v[8][4][2];
    __device__ __forceinline__ void zero() {
#pragma unroll
        for (int a = 0; a < 8; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) v[a][b][0] = v[a][b][1] = 0.0;
    }
};

template <bool A_KCONTIG, bool B_KCONTIG>
__device__ __forceinline__ void mma_slab(Acc &acc, const double *As, const double *Bs, int wm, int wn, int g, int t) {
#pragma unroll
    for (int kk = 0; kk < BK; kk += 4) {
        double af[8], bf[4];
#pragma unroll
        for (int a = 0; a < 8; ++a) {
            int r = wm * 64 + a * 8 + g;
            af[a] = A_KCONTIG ? As[r * LDK + kk + t] : As[(kk + t) * LDN + r];
        }
#pragma unroll
        for (int b = 0; b < 4; ++b) {
            int c = wn * 32 + b * 8 + g;
            bf[b] = B_KCONTIG ? Bs[c * LDK + kk + t] : Bs[(kk + t) * LDN + c];
        }
#pragma unroll
        for (int a = 0; a < 8; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) dmma_m8n8k4(acc.v[a][b][0], acc.v[a][b][1], af[a], bf[b]);
    }
}

// acc += A(128 x K) * B(K x 128) over k in [0, K).  `smem` holds NSTAGE stages.
// All 256 threads of the CTA must call this; ends with every cp.async drained and a
// __syncthreads(), so the caller may reuse `smem` right away.  This is the general loop
// (ragged edges, unaligned operands); gemm_mainloop_fast below is the one that reaches the
// tensor peak.
template <bool A_KCONTIG, bool B_KCONTIG, int NSTAGE>
__device__ __forceinline__ void gemm_mainloop(Acc &acc, double *smem, const Operand &A, const Operand &B, int K) {
    using SL = SlabLayout<A_KCONTIG, B_KCONTIG>;
    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const int wm = warp >> 2, wn = warp & 3, g = lane >> 2, t = lane & 3;
    const int nk = (K + BK - 1) / BK;

#pragma unroll
    for (int s = 0; s < NSTAGE - 1; ++s) {
        if (s < nk) {
            double *st = smem + s * SL::STAGE_DOUBLES;
            load_slab<A_KCONTIG>(st, A, s * BK, K, tid);
            load_slab<B_KCONTIG>(st + SL::A_DOUBLES, B, s * BK, K, tid);
        }
        cp_async_commit();
    }
    for (int kt = 0; kt < nk; ++kt) {
        cp_async_wait<NSTAGE - 2>();
        __syncthreads();
        {
            int nxt = kt + NSTAGE - 1;
            if (nxt < nk) {
                double *st = smem + (nxt % NSTAGE) * SL::STAGE_DOUBLES;
                load_slab<A_KCONTIG>(st, A, nxt * BK, K, tid);
                load_slab<B_KCONTIG>(st + SL::A_DOUBLES, B, nxt * BK, K, tid);
            }
            cp_async_commit();
        }
        const double *st = smem + (kt % NSTAGE) * SL::STAGE_DOUBLES;
        mma_slab<A_KCONTIG, B_KCONTIG>(acc, st, st + SL::A_DOUBLES, wm, wn, g, t);
    }
    cp_async_wait<0>();
    __syncthreads();
}

// Per-thread copy plan for one operand: BK/4 chunks of 16 bytes per slab, one base pointer and
// constant strides (between chunks and between slabs).  Valid only for tiles that are fully in range and 16-byte aligned.
template <bool KCONTIG>
struct FastCopy {
    // chunk i of this thread: source src0 + i * sstep (+ slab * step), destination dst0 + i * dstep
    const double *src0;
    long sstep, step;
    int dst0, dstep;
    __device__ __forceinline__ void init(const Operand &op, int tid) {
        if (KCONTIG) {
            int r = tid / (BK / 2), kk = (tid % (BK / 2)) * 2;
            src0 = op.ptr + (long)r * op.ld + kk;
            dst0 = r * LDK + kk;
            sstep = (long)(GEMM_THREADS / (BK / 2)) * op.ld;
            dstep = (GEMM_THREADS / (BK / 2)) * LDK;
            step = BK;
        } else {
            int kr = tid >> 6, cc = (tid & 63) * 2;
            src0 = op.ptr + (long)kr * op.ld + cc;
            dst0 = kr * LDN + cc;
            sstep = (long)(GEMM_THREADS / 64) * op.ld;
            dstep = (GEMM_THREADS / 64) * LDN;
            step = (long)BK * op.ld;
        }
    }
    __device__ __forceinline__ void issue(double *smem, int i, long slab) const {
        cp_async16(smem + CI(dst0 + i * dstep, (KCONTIG ? TILE_KC : TILE_MN) - 1, 203), src0 + i * sstep + slab * step, 16);
    }
};

// Same contraction as gemm_mainloop for operand tiles that are fully in range and 16-byte aligned
// and K a multiple of BK: the copies of the next slab are issued one pair per k4-step between the
// MMAs (every MMA warp would otherwise run all its copy code right after the slab barrier and
// leave the tensor pipe idle).
template <bool A_KCONTIG, bool B_KCONTIG, int NSTAGE>
__device__ __forceinline__ void gemm_mainloop_fast(Acc &acc, double *smem, const Operand &A, const Operand &B, int K) {
    using SL = SlabLayout<A_KCONTIG, B_KCONTIG>;
    const int tid = threadIdx.x;
    const int warp = tid >> 5, lane = tid & 31;
    const int wm = warp >> 2, wn = warp & 3, g = lane >> 2, t = lane & 3;
    const int nk = K / BK;
    FastCopy<A_KCONTIG> ca;
    FastCopy<B_KCONTIG> cb;
    ca.init(A, tid);
    cb.init(B, tid);
#pragma unroll
    for (int s = 0; s < NSTAGE - 1; ++s) {
        if (s < nk) {
            double *st = smem + s * SL::STAGE_DOUBLES;
#pragma unroll
            for (int i = 0; i < BK / 4; ++i) { ca.issue(st, i, s); cb.issue(st + SL::A_DOUBLES, i, s); }
        }
        cp_async_commit();
    }
    for (int kt = 0; kt < nk; ++kt) {
        cp_async_wait<NSTAGE - 2>();
        __syncthreads();
        const int nxt = kt + NSTAGE - 1;
        const bool more = nxt < nk;
        double *stn = smem + (nxt % NSTAGE) * SL::STAGE_DOUBLES;
        const double *As = smem + (kt % NSTAGE) * SL::STAGE_DOUBLES;
        const double *Bs = As + SL::A_DOUBLES;
#pragma unroll
        for (int kk = 0; kk < BK; kk += 4) {
            double af[8], bf[4];
#pragma unroll
            for (int a = 0; a < 8; ++a) {
                int r = wm * 64 + a * 8 + g;
                af[a] = A_KCONTIG ? As[r * LDK + kk + t] : As[(kk + t) * LDN + r];
            }
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                int c = wn * 32 + b * 8 + g;
                bf[b] = B_KCONTIG ? Bs[c * LDK + kk + t] : Bs[(kk + t) * LDN + c];
            }
#pragma unroll
            for (int a = 0; a < 8; ++a) {
#pragma unroll
                for (int b = 0; b < 4; ++b) dmma_m8n8k4(acc.v[a][b][0], acc.v[a][b][1], af[a], bf[b]);
                if (a == 3 && more) ca.issue(stn, kk / 4, nxt);
                if (a == 7 && more) cb.issue(stn + SL::A_DOUBLES, kk / 4, nxt);
            }
        }
        cp_async_commit();
    }
    cp_async_wait<0>();
    __syncthreads();
}

// Picks the interleaved-copy loop when the operand tiles allow it.
template <bool A_KCONTIG, bool B_KCONTIG, int NSTAGE>
__device__ __forceinline__ void gemm_tile(Acc &acc, double *smem, const Operand &A, const Operand &B, int K) {
    if (A.aligned16 && B.aligned16 && A.mn_valid == BM && B.mn_valid == BN && (K % BK) == 0)
        gemm_mainloop_fast<A_KCONTIG, B_KCONTIG, NSTAGE>(acc, smem, A, B, K);
    else
        gemm_mainloop<A_KCONTIG, B_KCONTIG, NSTAGE>(acc, smem, A, B, K);
}

}  // namespace gptq2d
