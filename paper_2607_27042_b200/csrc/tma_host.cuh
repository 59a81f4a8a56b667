// Host side of the TMA path: tensor maps for fp64 and fp32 operands (driver entry point looked up through the
// runtime, so the library has no link-time dependency on the driver library).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace gptq2d {

typedef CUresult (*TensorMapEncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                           const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                           CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                           CUtensorMapFloatOOBfill);

// NULL if the driver does not offer it (callers then use the cp.async path)
TensorMapEncodeTiledFn tensor_map_encoder();

// A row-major fp64 matrix (rows x cols, leading dimension ld, `batch` copies `batch_stride` elements apart) as a
// 3-D tensor {cols, rows, batch} read in boxes of box_cols x box_rows x 1 with the 128-byte swizzle
// (box_cols must be 16).  Out-of-range parts of a box read as zeros.
// Requirements (checked; false if not met): base 16-byte aligned, ld and batch_stride even.
bool encode_f64_matrix_map(CUtensorMap *map, const double *base, long rows, long cols, long ld, long batch,
                           long batch_stride, int box_cols, int box_rows);

// A row-major fp32 matrix (rows x cols, leading dimension ld) as a 2-D tensor {cols, rows} read in dense boxes of
// box_cols x box_rows (no swizzle: the reader's lanes all sit in one row of the box at a time).  Out-of-range parts
// of a box read as zeros.  Requirements (checked; false if not met): base 16-byte aligned, ld a multiple of 4,
// box_cols a multiple of 4, both box extents at most 256.
bool encode_f32_matrix_map(CUtensorMap *map, const float *base, long rows, long cols, long ld, int box_cols, int box_rows);

inline bool tma_operand_ok(const double *base, long ld, long batch_stride) {
    return (reinterpret_cast<uintptr_t>(base) & 15) == 0 && (ld & 1) == 0 && (batch_stride & 1) == 0;
}

}  // namespace gptq2d
