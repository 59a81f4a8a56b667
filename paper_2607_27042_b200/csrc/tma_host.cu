#include "tma_host.cuh"
#include <mutex>

namespace gptq2d {

TensorMapEncodeTiledFn tensor_map_encoder() {
    static std::once_flag once;
    static TensorMapEncodeTiledFn fn = nullptr;
    std::call_once(once, [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qr = cudaDriverEntryPointSymbolNotFound;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qr) == cudaSuccess &&
            qr == cudaDriverEntryPointSuccess && p)
            fn = reinterpret_cast<TensorMapEncodeTiledFn>(p);
        (void)cudaGetLastError();
    });
    return fn;
}

bool encode_f64_matrix_map(CUtensorMap *map, const double *base, long rows, long cols, long ld, long batch,
                           long batch_stride, int box_cols, int box_rows) {
    TensorMapEncodeTiledFn enc = tensor_map_encoder();
    if (!enc || box_cols != 16 || box_rows < 1 || box_rows > 256) return false;
    if (rows < 1 || cols < 1 || batch < 1) return false;
    if (batch == 1) batch_stride = rows * ld;          // unused by the copies; must only be a legal stride
    if (batch_stride < 2) batch_stride = 2;
    if (!tma_operand_ok(base, ld, batch_stride)) return false;
    if ((unsigned long long)ld * 8ull >= (1ull << 40) || (unsigned long long)batch_stride * 8ull >= (1ull << 40)) return false;
    const cuuint64_t dims[3] = {(cuuint64_t)cols, (cuuint64_t)rows, (cuuint64_t)batch};
    const cuuint64_t strides[2] = {(cuuint64_t)ld * 8ull, (cuuint64_t)batch_stride * 8ull};
    const cuuint32_t box[3] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows, 1u};
    const cuuint32_t estr[3] = {1u, 1u, 1u};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT64, 3, const_cast<double *>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool encode_f32_matrix_map(CUtensorMap *map, const float *base, long rows, long cols, long ld, int box_cols, int box_rows) {
    TensorMapEncodeTiledFn enc = tensor_map_encoder();
    if (!enc || box_cols < 4 || box_cols > 256 || (box_cols & 3) || box_rows < 1 || box_rows > 256) return false;
    if (rows < 1 || cols < 1 || ld < cols) return false;
    if ((reinterpret_cast<uintptr_t>(base) & 15) != 0 || (ld & 3) != 0) return false;
    if ((unsigned long long)ld * 4ull >= (1ull << 40)) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)ld * 4ull};
    const cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1u, 1u};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float *>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace gptq2d
