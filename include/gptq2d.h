/* gptq2d.h -- C ABI of the B200 (sm_100a) two-sided adaptive rounding library.
 *
 * Problem (paper Section 3.2, Eq. 6-9): given X (m x n, real) and nonsingular bases
 * A (m x m), B (n x n), produce the integer matrix Z (m x n) that one-dimensional
 * adaptive rounding (Algorithm 1: Babai nearest plane / GPTQ) yields on vec(X) under
 * the Kronecker Gram (B B^T) (x) (A^T A).  GPTQ-2D (Algorithm 3, Theorem 2) reaches
 * exactly that Z with O(m n max(m,n)) sweep work after an O(max(m,n)^3) set-up.
 *
 * Conventions for every call
 *   - Matrix pointers are DEVICE pointers owned by the caller, row-major, with a
 *     leading dimension given in elements (ld >= number of columns).  Pointers must
 *     be 8-byte aligned; 16-byte alignment with even leading dimensions is faster.
 *   - Nothing is allocated: scratch comes from a caller-provided device workspace
 *     whose size the matching *_workspace_bytes query returns (256-byte aligned).
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).  Calls
 *     enqueue work and return; they do not synchronise.
 *   - The return value reports argument / launch errors found on the host
 *     (gptq2d_status_t).  Data-dependent errors are written by the device into
 *     `info` (device int[4]: {status, index, aux0, aux1}; may be NULL), valid once the
 *     stream has been synchronised.  `info` is reset to zeros by each call.
 *   - A and B are general nonsingular matrices.  No damping, permutation, clamping,
 *     scale or zero point is applied: the paper rounds to all of Z^{m x n} in the
 *     natural order.
 *   - Requires an sm_100 device; anything else returns GPTQ2D_ERR_UNSUPPORTED_DEVICE.
 *     There is no CPU fallback.
 */
#ifndef GPTQ2D_H
#define GPTQ2D_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    GPTQ2D_OK = 0,
    GPTQ2D_ERR_INVALID_ARG = 1,        /* null pointer, m or n < 1, ld too small, misaligned pointer   */
    GPTQ2D_ERR_WORKSPACE = 2,          /* workspace missing, misaligned or smaller than the query says  */
    GPTQ2D_ERR_UNSUPPORTED_DEVICE = 3, /* current device is not compute capability 10.x                 */
    GPTQ2D_ERR_CUDA = 4,               /* a CUDA runtime call failed (launch, attribute query, copy)    */
    GPTQ2D_ERR_NOT_SPD = 5,            /* device: Gram pivot <= 0 or non-finite; info[1] = pivot index,
                                          info[2] = 0 for A^T A, 1 for B B^T                            */
    GPTQ2D_ERR_NONFINITE = 6,          /* device: NaN/Inf met while rounding; info[1] = row, info[2] = col of an
                                          entry on the first anti-diagonal where one was met (inside an 8 x 8
                                          block of the sweep a NaN also reaches neighbours that exact arithmetic
                                          would spare, so this may be a neighbour of the offending input)    */
    GPTQ2D_ERR_INT_OVERFLOW = 7,       /* device: |corrected value| >= 2^31; info[1] = row, info[2] = col  */
    GPTQ2D_ERR_DEVICE_TIMEOUT = 8,     /* device: a bounded wait gave up; info[1] = where it waited     */
    GPTQ2D_ERR_TOO_LARGE = 9,          /* gptq2d_round_static: m or n beyond GPTQ2D_STATIC_MAX_DIM;
                                          gptq2d_round_batched: beyond its count / dimension limits     */
    GPTQ2D_ERR_CHECK = 10              /* device, checked builds of the library only: an index of a sweep kernel
                                          left its array; info[1] = site, info[2] = index, info[3] = limit */
} gptq2d_status_t;

typedef enum {
    GPTQ2D_FP64 = 0,   /* all sweep arithmetic in fp64 (tiled wavefront kernel)                       */
    GPTQ2D_FP32 = 1,   /* X, L, U rounded to fp32 and all sweep arithmetic in fp32, on 64 x 64 tiles (the
                          tile restatement of Algorithm 3; far feedback as an FFMA contraction); Z may
                          differ from FP64 wherever a pre-rounding value lies within fp32 error of a tie */
    GPTQ2D_FP64_UNTILED = 2, /* fp64 with the untiled Algorithm-3 kernel; a cross-check, not fast     */
    GPTQ2D_FP32_UNTILED = 4, /* fp32 with the untiled Algorithm-3 kernel (one grid-wide barrier per
                               anti-diagonal): the literal order of operations in fp32; a cross-check, not fast */
    GPTQ2D_FP64_PULL = 3    /* fp64, implicit-Y form (Algorithm 6, Eq. 19-20) with C pulled as well: every
                               entry reconstructs its corrected value from L, E, C, U at rounding time;
                               untiled and bound by memory bandwidth: the comparison point, not fast   */
} gptq2d_precision_t;

/* Human-readable name of a status code (static storage). */
const char *gptq2d_status_string(int status);

/* ---- set-up: feedback factors (Section 3.1; Section 4.1 below Eq. 9; Algorithm 3 lines 1-2) ----
 * L (m x m): unit lower triangular, (A^T A)^{-1} = L Lambda_L L^T.
 * U (n x n): unit upper triangular, (B B^T)^{-1} = U^T Lambda_U U.
 * Computed without forming an inverse Gram: G = P^T P with P lower triangular (a Cholesky
 * factorisation run from the last index to the first), L = P^{-1} diag(P), Lambda^{-1} = diag(P)^2.
 * Outputs have exact ones on the diagonal and exact zeros in the opposite triangle.
 * dL (m) / dU (n), optional (NULL ok): 1/Lambda_L and 1/Lambda_U, so that
 * ||A (Z-X) B||_F^2 = sum_ij E_ij^2 dL_i dU_j for the local errors E.
 * A or B may be NULL, meaning the identity (L or U is then the identity).
 * Device error: GPTQ2D_ERR_NOT_SPD when a Gram is numerically not positive definite
 * (A or B singular); L and U are then undefined.
 * Streams: everything is ordered after the work already on `stream`, and `stream` waits for all of it
 * before the call's outputs are used by later work on it.  With both bases given, part of the work runs
 * on streams of the library's own (per device, created on first use: the B side next to the A side, and
 * each side's chain of diagonal blocks ahead of its large updates); concurrent calls on one device are
 * serialised while they enqueue.
 */
size_t gptq2d_factor_workspace_bytes(int m, int n);
int gptq2d_factor(int m, int n,
                  const double *A, long lda, const double *B, long ldb,
                  double *L, long ldl, double *U, long ldu,
                  double *dL, double *dU,
                  void *workspace, size_t workspace_bytes, int *info, void *stream);

/* ---- the sweep (Algorithm 3; tiled restatement via Eq. 11 and Eq. 15-17) ----
 * Z (m x n, int32): Z_ij = round-half-even(Y_ij) with Y the corrected matrix.
 * E (m x n), optional: local errors E_ij = Z_ij - Y_ij (Algorithm 3 line 5), each in [-1/2, 1/2].
 * min_margin, optional device scalar: min_ij (1/2 - |E_ij|), the distance of the closest
 *   pre-rounding value from a tie.
 * L, U: as produced by gptq2d_factor (only the strict triangles are read; the unit diagonal
 *   is implied).  They must stay fixed during the call (Section 6, first caveat).
 * Initialisation (Y <- X, C <- 0; Algorithm 3 lines 4-5) is part of this call.
 * Device errors: NONFINITE, INT_OVERFLOW (Z is int32), DEVICE_TIMEOUT.
 * Calls on different streams must use different workspaces.
 */
size_t gptq2d_round_workspace_bytes(int m, int n, int precision);
int gptq2d_round(int m, int n,
                 const double *X, long ldx,
                 const double *L, long ldl, const double *U, long ldu,
                 int32_t *Z, long ldz,
                 double *E, long lde, double *min_margin,
                 int precision,
                 void *workspace, size_t workspace_bytes, int *info, void *stream);

/* Same sweep with HOST buffers; `stream` is synchronised before returning.  hX, hL, hU, hZ, hE are host
 * pointers, dense row-major (leading dimension = number of columns); hinfo: host int[4], receives the
 * device info words.  The workspace is still a device buffer.
 * GPTQ2D_FP64: the copies overlap the sweep.  The kernel is launched at once and the inputs follow on a
 *   second stream (one per device, created by the library on first use) in 512 x 512 blocks, in the
 *   order the anti-diagonal wavefront needs them (Section 2, Fig. 1: entry (i, j) depends on the
 *   rectangle above and to its left only): step s = the blocks of X on block anti-diagonal s, block
 *   row s of L up to its diagonal block, block column s of U down to its diagonal block (the opposite
 *   triangles are never sent).  Each step is announced to the running kernel by a stream-ordered
 *   32-bit write; a task starts when its step has arrived.  If hZ is pinned memory, Z goes back while
 *   the sweep still runs: the kernel counts the swept tiles of every row of 128 x 128 tiles, and the
 *   second stream copies the rows of a tile row as soon as a stream-ordered wait sees its count
 *   complete.  Pinned buffers make all copies asynchronous and fast; pageable ones work (Z is then
 *   copied at the end).  If the driver lacks stream memory
 *   operations the call falls back to copy-then-sweep.  Concurrent calls on one device take turns to
 *   enqueue (they share the copy stream).
 * Other precisions: X, L, U are copied first, the sweep runs, Z (and E, min_margin) are copied back.
 */
size_t gptq2d_round_host_workspace_bytes(int m, int n, int precision);
int gptq2d_round_host(int m, int n,
                      const double *hX, const double *hL, const double *hU,
                      int32_t *hZ, double *hE, double *hmin_margin,
                      int precision,
                      void *workspace, size_t workspace_bytes, int *hinfo, void *stream);

/* ---- many independent sweeps in one launch (Section 6 names layer-wise Kronecker-factored Hessian
 * estimates as a source of A and B, i.e. one (X; A, B) triple per layer; the paper sweeps one
 * matrix, Algorithm 3, and this call runs that same sweep on `count` matrices at once) ----
 * A single small or thin matrix cannot fill the GPU: its anti-diagonal dependency chain has
 * m + n - 1 stages (Section 2, Fig. 1) and few entries per stage.  Here the fp64 tiled sweeps of
 * all matrices share one persistent kernel, so the tiles that are ready in ANY matrix keep the SMs
 * busy.  Each matrix gets exactly the Z (and E, min_margin) that gptq2d_round with GPTQ2D_FP64
 * gives it alone; shapes may differ from matrix to matrix.
 *   problems:   HOST array of `count` descriptors (device pointers inside, same rules as
 *               gptq2d_round); read before the call returns, the caller may free it afterwards.
 *   min_margin: optional DEVICE array of `count` doubles.
 *   info:       device int[4] shared by all matrices; for NONFINITE / INT_OVERFLOW info[3] is the
 *               index of the matrix (first error wins; the other matrices are still swept).
 *   Limits: count <= GPTQ2D_BATCH_MAX_COUNT, every m, n <= GPTQ2D_BATCH_MAX_DIM
 *           (else GPTQ2D_ERR_TOO_LARGE).  Output regions of different matrices must not overlap.
 */
typedef struct gptq2d_problem {
    int m, n;
    const double *X; long ldx;
    const double *L; long ldl;
    const double *U; long ldu;
    int32_t *Z; long ldz;
    double *E; long lde;       /* optional (NULL ok) */
} gptq2d_problem_t;
#define GPTQ2D_BATCH_MAX_COUNT 8192
#define GPTQ2D_BATCH_MAX_DIM 32768
size_t gptq2d_round_batched_workspace_bytes(int count, const gptq2d_problem_t *problems);
int gptq2d_round_batched(int count, const gptq2d_problem_t *problems,
                         double *min_margin,
                         void *workspace, size_t workspace_bytes, int *info, void *stream);

/* ---- the set-up of many matrices in one call (the factors that gptq2d_round_batched consumes) ----
 * For every problem the same L, U, dL, dU as gptq2d_factor (Section 3.1; Algorithm 3 lines 1-2).  The
 * problems whose bases both have order <= GPTQ2D_FACTOR_SMALL_MAX are factorised one CTA per side, all
 * in ONE launch, entirely in shared memory (Gram, Cholesky from the last index to the first, triangular
 * inverse, scaling); problems with a larger basis take the blocked route of gptq2d_factor, several of
 * them side by side on streams of the library's own (everything is ordered after the work already on
 * `stream`, and `stream` waits for all of it).
 *   problems: HOST array of `count` descriptors (device pointers inside, rules as gptq2d_factor: A or B
 *             may be NULL for the identity, dL / dU optional); read before the call returns.
 *   info:     device int[4] shared by all problems; for GPTQ2D_ERR_NOT_SPD from a small side info[3] is
 *             the index of the problem (first error wins; the other problems are still factorised).
 *   workspace: device, 256-byte aligned, gptq2d_factor_batched_workspace_bytes(count, problems) bytes.
 */
#define GPTQ2D_FACTOR_SMALL_MAX 128
typedef struct gptq2d_factor_problem {
    int m, n;
    const double *A; long lda;   /* m x m or NULL */
    const double *B; long ldb;   /* n x n or NULL */
    double *L; long ldl;
    double *U; long ldu;
    double *dL, *dU;             /* optional (NULL ok) */
} gptq2d_factor_problem_t;
size_t gptq2d_factor_batched_workspace_bytes(int count, const gptq2d_factor_problem_t *problems);
int gptq2d_factor_batched(int count, const gptq2d_factor_problem_t *problems,
                          void *workspace, size_t workspace_bytes, int *info, void *stream);

/* ---- the sweep without any allocation (the paper has no counterpart: this is a packaging variant
 * of gptq2d_round, not a different method) ----
 * For callers that must not allocate device memory -- a step that will be replayed from a CUDA
 * graph, a framework region that forbids raw cudaMalloc, a latency-critical loop that must stay
 * away from the allocator -- and therefore cannot hand over a workspace: the scratch of the fp64
 * tiled sweep lives in a static device array inside the library (GPTQ2D_STATIC_WORKSPACE_BYTES per
 * GPU that loads the library, held until the process exits).  Same arguments, results and device
 * status words as gptq2d_round with precision GPTQ2D_FP64, minus the workspace.
 *   - m, n <= GPTQ2D_STATIC_MAX_DIM, otherwise GPTQ2D_ERR_TOO_LARGE is returned and nothing runs.
 *   - The call itself allocates nothing (no cudaMalloc / cudaFree, no allocating library routine).
 *   - The FIRST call on each device looks up the array's device address (cudaGetSymbolAddress, with
 *     that device current); make that first call before starting any stream capture.
 *   - All calls on a device share the one array, which keeps the previous call's contents; the call
 *     clears what must start at zero.  Two calls that overlap on the GPU (different streams, no
 *     ordering between them) race on it: serialise them.
 */
#define GPTQ2D_STATIC_MAX_DIM 512
#define GPTQ2D_STATIC_WORKSPACE_BYTES (4u * 1024u * 1024u + 64u * 1024u)
int gptq2d_round_static(int m, int n,
                        const double *X, long ldx,
                        const double *L, long ldl, const double *U, long ldu,
                        int32_t *Z, long ldz,
                        double *E, long lde, double *min_margin,
                        int *info, void *stream);
size_t gptq2d_round_static_max_dim(void);

/* ---- reverse order (Section 2, the paragraph on two-sided and Kronecker-factored rounding, mentions
 * the same greedy rounding run backwards, starting at the bottom-right corner of the matrix) ----
 * Coordinates of vec(X) are visited from the last to the first.  The feedback factors become
 *   Lr (m x m): unit UPPER triangular, (A^T A)^{-1} = Lr Lambda Lr^T,
 *   Ur (n x n): unit LOWER triangular, (B B^T)^{-1} = Ur^T Lambda Ur,
 * and the sweep runs over the anti-diagonals from the last to the first, pushing up and to the left.
 * With P the index reversal this is the forward problem on (P X P; A P, P B); both calls reverse
 * their operands into the workspace, run the forward kernels and reverse the results back, so Z, E,
 * min_margin, dL, dU are in the caller's own indexing.  Only the device status words are not
 * translated: a row / column / pivot index k reported in `info` is m-1-k (n-1-k) in the caller's
 * indexing.  Argument rules, status codes and stream behaviour are those of gptq2d_factor /
 * gptq2d_round (fp64 tiled sweep).
 */
size_t gptq2d_factor_reverse_workspace_bytes(int m, int n);
int gptq2d_factor_reverse(int m, int n,
                          const double *A, long lda, const double *B, long ldb,
                          double *Lr, long ldl, double *Ur, long ldu,
                          double *dL, double *dU,
                          void *workspace, size_t workspace_bytes, int *info, void *stream);
size_t gptq2d_round_reverse_workspace_bytes(int m, int n);
int gptq2d_round_reverse(int m, int n,
                         const double *X, long ldx,
                         const double *Lr, long ldl, const double *Ur, long ldu,
                         int32_t *Z, long ldz,
                         double *E, long lde, double *min_margin,
                         void *workspace, size_t workspace_bytes, int *info, void *stream);

/* ---- inputs stored in fp32, arithmetic in fp64 (the paper works in exact arithmetic and fixes no
 * storage format; this is a packaging variant for callers that keep X and the factors in fp32) ----
 * X, L, U are float arrays; they are widened to fp64 (exactly) into the workspace and the fp64 tiled
 * sweep of gptq2d_round runs on them, so Z is exactly the trajectory of Algorithm 3 for the fp32-
 * rounded data: against the sweep on the fp64 originals only the inputs' rounding differs (unlike
 * GPTQ2D_FP32, which also computes in fp32).  Outputs, status words and stream behaviour as
 * gptq2d_round.
 */
size_t gptq2d_round_f32in_workspace_bytes(int m, int n);
int gptq2d_round_f32in(int m, int n,
                       const float *X, long ldx,
                       const float *L, long ldl, const float *U, long ldu,
                       int32_t *Z, long ldz,
                       double *E, long lde, double *min_margin,
                       void *workspace, size_t workspace_bytes, int *info, void *stream);

/* ---- blocked GPTQ-2D (Algorithm 4, Section 4 "Blocked GPTQ-2D") as an alternative kernel ----
 * The same rounding in blocks of w consecutive anti-diagonals, 1 <= w <= GPTQ2D_BLOCKED_MAX_WIDTH:
 * inside a block the feedback stops at the block's last anti-diagonal; after it, a down flush (the
 * block's band of E through L, added to Y and to the buffer C = L E) and a right flush (the block's
 * band of C through U, added to Y) reach every later entry.  By the paper's correctness argument Z
 * equals that of gptq2d_round for every w.  X, L, U, Z, E, min_margin, info, stream: as gptq2d_round
 * (all device memory; only the strictly lower part of L and the strictly upper part of U are read).
 * Two kernel launches per block, (m + n - 2) / w + 1 blocks.  The workspace holds Y, C and E.
 * Returns GPTQ2D_ERR_INVALID_ARG for a width outside the range (the workspace size is then 0).
 * This is the paper's own GPU formulation kept as a comparison point: it re-reads every later entry
 * once per block and is slower than the tiled sweep at every size.
 */
#define GPTQ2D_BLOCKED_MAX_WIDTH 64
size_t gptq2d_round_blocked_workspace_bytes(int m, int n, int w);
int gptq2d_round_blocked(int m, int n,
                         const double *X, long ldx,
                         const double *L, long ldl, const double *U, long ldu,
                         int w,
                         int32_t *Z, long ldz,
                         double *E, long lde, double *min_margin,
                         void *workspace, size_t workspace_bytes, int *info, void *stream);

/* ---- the objective (Eq. 7): obj = || A (Z - X) B ||_F^2 ----
 * obj: device scalar.  A or B may be NULL (identity).
 */
size_t gptq2d_objective_workspace_bytes(int m, int n);
int gptq2d_objective(int m, int n,
                     const double *X, long ldx, const int32_t *Z, long ldz,
                     const double *A, long lda, const double *B, long ldb,
                     double *obj,
                     void *workspace, size_t workspace_bytes, int *info, void *stream);

/* ---- test hook for the library's failure handling (the paper has no counterpart; not for production use) ----
 * Every device-side wait of the sweep kernels is bounded: after a number of polls it gives up, records
 * where in `info` (GPTQ2D_ERR_DEVICE_TIMEOUT, info[1] = the wait's code, negative), raises an abort word
 * that all other waits watch, and the kernel returns normally.  This hook lets a test make one such wait
 * run out WITHOUT faulting or hanging the GPU; the failure is made on the host.
 *   key 1, value != 0: the next pipelined gptq2d_round_host call (GPTQ2D_FP64) does not announce its last
 *          copy step to the running kernel (one-shot; cleared by that call).  The tasks that need the step
 *          wait for it (wait code -6) until their limit.
 *   key 2, value = polls (about 0.2 us each) after which the wait for a copy step gives up; 0 restores the
 *          default (about a second).  All other waits keep the default.
 *   key 3: which kernel the library's fp64 products (set-up, objective) take.  0: the cp.async kernel only;
 *          1 (default): the TMA-fed kernel where a tile edge is ragged, the cp.async kernel for full tiles;
 *          3: the TMA-fed kernel whenever the operands allow it; 2: as 3 with a barrier per slab.
 *   key 4: the sixteen-warp sweep kernel (far contractions beside the quadrant tasks).  0 (default): never;
 *          1: problems of at least 8 x 8 tiles; 2: whenever the operands allow it.  Comparison runs.
 *   key 5 (checked builds of the library only; otherwise unknown): value = address of a device int[5].  Runs the
 *          self-test of the index check on the default stream: one deliberately out-of-range index (7 of 3,
 *          site 999) is checked; [0..3] receive {GPTQ2D_ERR_CHECK, 999, 7, 3}, [4] the redirected index 0.
 *   key 6: how the fp32 mode's contraction gets its operand slabs.  0 (default): bulk tensor copies (TMA) where
 *          the driver offers tensor maps, cp.async otherwise; 1: cp.async always.  Comparison runs and tests.
 * Returns GPTQ2D_OK, or GPTQ2D_ERR_INVALID_ARG for an unknown key.
 */
int gptq2d_internal_test_hook(int key, long value);

/* The library's own fp64 product, exposed for tests and for measuring the fp64 tensor rate it reaches
 * (the denominator the sweep's roofline is quoted against): C = alpha op(A) op(B) + beta C, row-major,
 * op(A) M x K (stored K x M if transa), op(B) K x N (stored N x K if transb).  Device pointers, 8-byte
 * aligned; enqueues on `stream`.  This is the dense contraction that the set-up (Section 3.1) and the
 * objective (Eq. 7) are made of, and the same tile loop that carries the far parts of the sweep.
 */
int gptq2d_internal_gemm(int transa, int transb, int M, int N, int K, double alpha,
                         const double *A, long lda, const double *B, long ldb,
                         double beta, double *C, long ldc, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* GPTQ2D_H */
