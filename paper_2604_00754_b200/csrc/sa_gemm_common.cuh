// Pieces shared by the tensor-core GEMM kernels of the projection gates: TMA tile loads,
// tensor-map encoding through the driver entry point, the one-operation logistic.
#pragma once

#include <cuda.h>

#include "sa_common.cuh"
#include "sa_tc_common.cuh"

namespace sa {
namespace {

__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
}
// One box of the tensor map (x: element column, a multiple of 64; y: row) into shared memory;
// the bytes are counted on the mbarrier.  A load into this CTA only.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, int x, int y,
                                            uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes "
      "[%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(tm), "r"(x), "r"(y), "r"(bar)
      : "memory");
}
// One box of a rank-4 map (x: element column, a multiple of 64; then token, head, batch).
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* tm, int x, int tok,
                                            int head, int batch, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes "
      "[%0], [%1, {%2, %3, %4, %5}], [%6];"
      ::"r"(dst), "l"(tm), "r"(x), "r"(tok), "r"(head), "r"(batch), "r"(bar)
      : "memory");
}
// 1 / (1 + exp(-z)) = 0.5 tanh(z / 2) + 0.5: one special-function operation per element
__device__ __forceinline__ float logistic(float z) {
  float t;
  asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(0.5f * z));
  return fmaf(t, 0.5f, 0.5f);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) ==
            cudaSuccess && qres == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)ptr;
  }
  return fn;
}

// bf16 matrix [rows, cols], pitch ld elements, read in boxes of 64 columns x box_rows rows
// with the 128-byte swizzle; outside the matrix reads zero.  box_rows 128: an operand whose
// columns are the contraction index; 64: one whose rows are.
inline bool make_map(CUtensorMap* tm, const void* base, int64_t rows, int64_t cols, int64_t ld,
                     int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  const cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box,
            estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// bf16 tensor [B,H,n,d] with element strides s[0..2] (batch, head, token; d contiguous) as a
// rank-4 map (d, token, head, batch), read in boxes of 64 columns x box_rows tokens of one head
// with the 128-byte swizzle.  The token index is a dimension of its own, so a box that runs
// past token n - 1 reads zeros there and never the rows that follow in memory.
inline bool make_map_bhnd(CUtensorMap* tm, const void* base, int B, int H, int n, int d,
                          const int64_t s[3], int box_rows = 128) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  // the stride of a dimension of extent 1 is never used: any valid value will do
  const int64_t st[3] = {B > 1 ? s[0] : d, H > 1 ? s[1] : d, n > 1 ? s[2] : d};
  for (int i = 0; i < 3; ++i)
    if (st[i] % 8 != 0 || st[i] <= 0 || st[i] >= (1ll << 38)) return false;
  const cuuint64_t dims[4] = {(cuuint64_t)d, (cuuint64_t)n, (cuuint64_t)H, (cuuint64_t)B};
  const cuuint64_t strides[3] = {(cuuint64_t)st[2] * 2, (cuuint64_t)st[1] * 2,
                                 (cuuint64_t)st[0] * 2};
  const cuuint32_t box[4] = {64, (cuuint32_t)box_rows, 1, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box,
            estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

inline bool aligned16(const void* p) { return ((uintptr_t)p & 15u) == 0; }

}  // namespace
}  // namespace sa
