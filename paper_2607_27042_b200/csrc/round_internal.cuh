// Internal launch interfaces of the sweep kernels (not part of the C ABI).
#pragma once
#include <cuda_runtime.h>
#include "common.cuh"

namespace gptq2d {

struct UntiledParams {
    int m, n;
    const double *X; long ldx;
    const double *L; long ldl;
    const double *U; long ldu;
    int *Z; long ldz;
    double *E; long lde;      // optional
    double *max_abs_e;        // workspace scalar, max |E| over the matrix
    int *info;
    void *Ybuf, *Cbuf;        // m x n working copies (fp64 or fp32), dense
    GridSync sync;
};
size_t round_untiled_workspace_bytes(int m, int n, bool fp32);
int launch_round_untiled(const UntiledParams &p, bool fp32, void *ws, cudaStream_t stream);

struct PullParams {
    int m, n;
    const double *X; long ldx;
    const double *L; long ldl;
    const double *U; long ldu;
    int *Z; long ldz;
    double *E; long lde;      // optional
    double *max_abs_e;
    int *info;
    double *C, *Et, *Ut;      // workspace: C = L E (m x n), E transposed (n x m), U transposed (n x n)
    GridSync sync;
};
size_t round_pull_workspace_bytes(int m, int n);
int launch_round_pull(const PullParams &p, void *ws, cudaStream_t stream);

struct TiledParams {
    int m, n;
    const double *X; long ldx;
    const double *L; long ldl;
    const double *U; long ldu;
    int *Z; long ldz;
    double *E; long lde;      // optional user copy of the local errors
    double *max_abs_e;
    int *info;
    // optional: device word that counts the copy steps of X, L and U that have arrived (the sweep then
    // starts while the rest is still on its way, see COPY_BLOCK_TILES); NULL = everything is resident
    const unsigned *panels_ready;
    // polls after which the wait for an announced copy step gives up; 0 = the library's default
    unsigned long long panel_spin_limit;
};
// Inputs that arrive while the sweep runs come in blocks of COPY_BLOCK_TILES x COPY_BLOCK_TILES tiles of
// 128 x 128: step s = the blocks of X on block anti-diagonal s, block row s of L (up to the end of its
// diagonal block), block column s of U (down to the end of its diagonal block).
constexpr int COPY_BLOCK_TILES_LOG2 = 2;
constexpr int COPY_BLOCK = 128 << COPY_BLOCK_TILES_LOG2;
size_t round_tiled_workspace_bytes(int m, int n);
// device array inside the workspace: for each row of 128 x 128 tiles, how many of its tiles are swept
unsigned *round_tiled_rowdone(void *ws, int m, int n);
int launch_round_tiled(const TiledParams &p, void *ws, size_t ws_bytes, cudaStream_t stream);
// The sixteen-warp kernel (round_fused.cu): far contractions and quadrant tasks side by side on every SM.
// Modes: 0 never (default: it measures slower than the eight-warp kernel), 1 problems of at least 8 x 8
// tiles, 2 whenever the operands allow it (tests, comparison runs).
void round_fused_set_mode(int mode);
void round_tiled_f32_set_tma_mode(int mode);
// fp32 mode, tiled (round_tiled_f32.cu): X, L, U as fp64 device arrays, narrowed into the workspace
size_t round_tiled_f32_workspace_bytes(int m, int n);
int launch_round_tiled_f32(const TiledParams &p, void *ws, size_t ws_bytes, cudaStream_t stream);
// many matrices in one launch (fp64 tiled sweep); `info` is shared, `min_margin` (optional) gets one value per matrix
constexpr int BATCH_MAX_COUNT = 8192;     // matrix index has 13 bits in a ready-ring entry
constexpr int BATCH_MAX_DIM = 32768;      // tile coordinates have 8 bits there
size_t round_tiled_batched_workspace_bytes(int count, const TiledParams *problems);
int launch_round_tiled_batched(int count, const TiledParams *problems, double *min_margin, int *info, void *ws,
                               size_t ws_bytes, cudaStream_t stream);
// where the max |E| scalar lives inside either workspace
inline double *workspace_max_abs_e(void *ws) { return reinterpret_cast<double *>(static_cast<char *>(ws) + 64); }

}  // namespace gptq2d
