// Tensor-map (TMA descriptor) construction.  cuTensorMapEncodeTiled is a driver
// API; it is fetched through the runtime's driver entry point so that the
// library carries no link-time dependency on libcuda and loads on machines
// without a GPU.
#include <cuda.h>
#include <cuda_runtime.h>

#include "internal.h"

namespace ap {

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess) {
            (void)cudaGetLastError();
            return nullptr;
        }
        fn = (EncodeTiledFn)p;
    }
    return fn;
}

}  // namespace

// A pool plane [num_pages][Hkv][16][d] bf16 seen as 8-token row groups:
//   dim0: 64 elements (128 bytes)            contiguous
//   dim1: 8 tokens of a group                stride d*2 bytes
//   dim2: d/64 column halves                 stride 128 bytes
//   dim3: num_pages*Hkv*2 row groups         stride 8*d*2 bytes
// A box of (64, 8, d/64, 2) is one (page, kv head) tile.  With the 128-byte
// swizzle it lands in shared memory as [group][half][8 tokens][64], each
// [8][64] block being one 1024-byte swizzle atom: the canonical operand layout
// of tcgen05.mma, and bank-conflict-free for ldmatrix.  A box of
// (64, 8, d/64, 2 * tiles_per_box) is that many consecutive tiles (the kv heads
// of one page that follow one another in memory) in one request, laid out tile
// after tile.
int encode_pool_tensor_map(CUtensorMap *map, void *base, int num_pages, int num_kv_heads, int head_dim,
                           int tiles_per_box) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return AP_ERR_CUDA;
    const cuuint64_t halves = (cuuint64_t)head_dim / 64;
    cuuint64_t dims[4] = {64, 8, halves, (cuuint64_t)num_pages * (cuuint64_t)num_kv_heads * 2};
    cuuint64_t strides[3] = {(cuuint64_t)head_dim * 2, 128, (cuuint64_t)head_dim * 2 * 8};
    cuuint32_t box[4] = {64, 8, (cuuint32_t)halves, 2u * (cuuint32_t)tiles_per_box};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, base, dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? AP_OK : AP_ERR_CUDA;
}

// q [n_rows][Hq][d] bf16:
//   dim0: 64 elements; dim1: rows (stride Hq*d*2); dim2: Hq*d/64 column blocks (stride 128 bytes).
// A box of (64, 128, d/64) at (0, row0, head*d/64) is a 128-row query tile of
// one head, landing as [half][128 rows][64] (16 swizzle atoms per half).
// Rows past n_rows read as zero.
int encode_q_tensor_map(CUtensorMap *map, const void *q, int64_t n_rows, int num_q_heads, int head_dim) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return AP_ERR_CUDA;
    const cuuint64_t halves = (cuuint64_t)head_dim / 64;
    cuuint64_t dims[3] = {64, (cuuint64_t)n_rows, (cuuint64_t)num_q_heads * halves};
    cuuint64_t strides[2] = {(cuuint64_t)num_q_heads * (cuuint64_t)head_dim * 2, 128};
    cuuint32_t box[3] = {64, 128, (cuuint32_t)halves};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(q), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? AP_OK : AP_ERR_CUDA;
}

}  // namespace ap
