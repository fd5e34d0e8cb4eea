// Host-side helpers shared by the tensor-core translation units: tensor-map
// encoding (driver entry point fetched through the runtime, no libcuda link) and
// the launch wrapper of tc_gemm_kernel.
#pragma once
#include "tc_gemm.cuh"

namespace dq {
namespace tch {

using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                              const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                              CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeFn get_encode_fn() {
  static EncodeFn fn = nullptr;
  if (fn) return fn;
  void* p = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess)
    return nullptr;
  fn = reinterpret_cast<EncodeFn>(p);
  return fn;
}

// bf16 tensor [batch][rows][k] (k contiguous, row stride ld elements), box = {64, box_rows, 1},
// 128-byte swizzle: the shared-memory image is the K-major SW128 layout tcgen05 reads.
inline dq_status make_map(CUtensorMap* m, const void* base, int64_t k, int64_t rows, int64_t batch, int64_t ld,
                   int64_t batch_stride, int box_rows) {
  EncodeFn fn = get_encode_fn();
  if (!fn) return DQ_ERR_CUDA;
  cuuint64_t dims[3] = {(cuuint64_t)k, (cuuint64_t)rows, (cuuint64_t)batch};
  cuuint64_t strides[2] = {(cuuint64_t)ld * 2, (cuuint64_t)batch_stride * 2};
  cuuint32_t box[3] = {(cuuint32_t)tc::BLOCK_K, (cuuint32_t)box_rows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? DQ_OK : DQ_ERR_CUDA;
}

template <int BN, int NT, int EPI>
dq_status launch_gemm(Ctx& ctx, const CUtensorMap& a, const CUtensorMap& b, const CUtensorMap& alo,
                      const CUtensorMap& blo, const tc::Params& p) {
  using L = tc::SmemLayout<BN, NT>;
  static bool attr_set = false;
  auto kern = tc::tc_gemm_kernel<BN, NT, EPI>;
  if (!attr_set) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::TOTAL) != cudaSuccess)
      return DQ_ERR_CUDA;
    attr_set = true;
  }
  const int units = p.m_blocks * p.n_blocks * p.batch * p.ksplit;
  int grid = units < ctx.sm_count ? units : ctx.sm_count;
  if (grid < 1) return DQ_OK;
  kern<<<grid, tc::NUM_THREADS, L::TOTAL, ctx.stream>>>(a, b, alo, blo, p);
  return after_launch(ctx);
}

}  // namespace tch
}  // namespace dq
