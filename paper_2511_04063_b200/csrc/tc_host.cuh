// Host-side helpers shared by the tensor-core translation units: tensor-map
// encoding (driver entry point fetched through the runtime, no libcuda link) and
// the launch wrapper of tc_gemm_kernel.
#pragma once
#include "tc_gemm.cuh"
#include "tc_gemm2.cuh"

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
  static SmemOptIn attr;
  auto kern = tc::tc_gemm_kernel<BN, NT, EPI>;
  DQ_CHECK(opt_in_dynamic_smem(kern, L::TOTAL, attr));
  const int units = (p.tile_list ? p.n_list : p.m_blocks * p.n_blocks) * p.batch * p.ksplit;
  int grid = units < ctx.sm_count ? units : ctx.sm_count;
  if (grid < 1) return DQ_OK;
  kern<<<grid, tc::NUM_THREADS, L::TOTAL, ctx.stream>>>(a, b, alo, blo, p);
  return after_launch(ctx);
}

// Two-CTA kernel (tc_gemm2.cuh): p.m_blocks / p.n_blocks count 256 x 256 tiles; one cluster of two
// CTAs per tile, at most one pair per two SMs.
template <int NT, int EPI>
dq_status launch_gemm2(Ctx& ctx, const CUtensorMap& a, const CUtensorMap& b, const CUtensorMap& alo,
                       const CUtensorMap& blo, const tc::Params& p) {
  static SmemOptIn attr;
  auto kern = tc2::tc_gemm2_kernel<NT, EPI>;
  constexpr int SMEM = tc2::PairSmem<NT>::TOTAL;
  DQ_CHECK(opt_in_dynamic_smem(kern, SMEM, attr));
  const int units = (p.tile_list ? p.n_list : p.m_blocks * p.n_blocks) * p.batch * p.ksplit;
  int pairs = units < ctx.sm_count / 2 ? units : ctx.sm_count / 2;
  if (pairs < 1) return DQ_OK;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * pairs, 1, 1);
  cfg.blockDim = dim3(tc2::pair_threads<EPI>(), 1, 1);
  cfg.dynamicSmemBytes = SMEM;
  cfg.stream = ctx.stream;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  cfg.attrs = at; cfg.numAttrs = 1;
  if (cudaLaunchKernelEx(&cfg, kern, a, b, alo, blo, p) != cudaSuccess) return DQ_ERR_CUDA;
  return after_launch(ctx);
}

using bf16 = __nv_bfloat16;

// The stand-alone entry points take their scratch from the device's stream-ordered pool.  By default the
// pool hands freed memory back to the driver at every synchronisation, which turns each later call into a
// fresh device allocation; keep up to 1 GiB cached in this process's pool instead (set once per device).
inline void keep_pool_memory(int dev) {
  static bool done[64] = {};
  if (dev < 0 || dev >= 64 || done[dev]) return;
  cudaMemPool_t pool = nullptr;
  if (cudaDeviceGetDefaultMemPool(&pool, dev) == cudaSuccess && pool) {
    uint64_t cur = 0, want = (uint64_t)1 << 30;
    if (cudaMemPoolGetAttribute(pool, cudaMemPoolAttrReleaseThreshold, &cur) == cudaSuccess && cur < want)
      cudaMemPoolSetAttribute(pool, cudaMemPoolAttrReleaseThreshold, &want);
  }
  cudaGetLastError();
  done[dev] = true;
}

// O[token][channel] = sum_k X[token][k] Rt[channel][k] for n token rows (bf16, row stride ldx) and a
// d x d bf16 R^T; EPI = EPI_BF16 (bf16 rows, stride ldo) or EPI_GEN (fp32 rows).  CTA pairs with
// 256 x 256 tiles when the shape allows, else the one-CTA kernel.  n % 128 == 0, d % 128 == 0.
template <int EPI>
inline dq_status rotate_tokens(Ctx& ctx, const void* X, int64_t n, int d, int64_t ldx, const bf16* rt, void* out,
                               int64_t ldo, int* d_status) {
  // TMA needs 16-byte aligned bases and row strides; the epilogue stores 16 bytes at a time
  if ((((uintptr_t)X | (uintptr_t)rt | (uintptr_t)out) & 15) || ldx % 8 != 0 || ldo % 8 != 0 ||
      (EPI == tc::EPI_GEN && ((uintptr_t)out & 31)))   // (the fp32 epilogue stores 32 bytes at a time)
    return DQ_ERR_UNSUPPORTED;
  CUtensorMap ma, mb;
  tc::Params p{};
  p.batch = 1; p.ksplit = 1; p.k_blocks = d / tc::BLOCK_K;
  p.out = out; p.ld = ldo; p.alpha = 1.f; p.d_status = d_status;
  if (d % 256 == 0 && n % 256 == 0 && ctx.sm_count >= 2) {
    DQ_CHECK(make_map(&ma, X, d, n, 1, ldx, n * ldx, tc2::HALF));
    DQ_CHECK(make_map(&mb, rt, d, d, 1, d, (int64_t)d * d, tc2::HALF));
    p.m_blocks = (int)(n / 256); p.n_blocks = d / 256;
    return launch_gemm2<1, EPI>(ctx, ma, mb, ma, mb, p);
  }
  const int bn = (d % 256 == 0) ? 256 : 128;
  DQ_CHECK(make_map(&ma, X, d, n, 1, ldx, n * ldx, tc::BLOCK_M));
  DQ_CHECK(make_map(&mb, rt, d, d, 1, d, (int64_t)d * d, bn));
  p.m_blocks = (int)(n / tc::BLOCK_M); p.n_blocks = d / bn;
  return (bn == 256) ? launch_gemm<256, 1, EPI>(ctx, ma, mb, ma, mb, p) : launch_gemm<128, 1, EPI>(ctx, ma, mb, ma, mb, p);
}

// Operand of a product: a row-major matrix as a split pair, leading dimension, batch stride (elements).
// t == false: rows x K (each row of the matrix is a row of the operand).  t == true: K x rows, the operand is the
// TRANSPOSE of the stored matrix; the MMAs read its tiles MN-major, no transposed copy is needed.
struct Op {
  const bf16* hi; const bf16* lo; int64_t ld; int64_t bs; bool t = false;
};
struct Out {
  float* f32 = nullptr; int64_t ld = 0; int64_t bs = 0;
  bf16* hi = nullptr; bf16* lo = nullptr; int64_t ld_h = 0; int64_t bs_h = 0;
  bf16* hi2 = nullptr; bf16* lo2 = nullptr;   // a second row-major split copy (same ld_h / bs_h)
  float alpha = 1.f, beta = 0.f;             // beta: the old contents of f32 are added (shorthand for add1 = f32)
  // v = alpha * acc + g1 * add1 + g2 * add2: fp32 matrices addressed like f32 (same ld / bs)
  const float* add1 = nullptr; float g1 = 1.f;
  const float* add2 = nullptr; float g2 = 1.f;
  // transposed split copies (element (m, n) at n * ld_t + m), up to two targets; lo parts nullable
  bf16* t_hi = nullptr; bf16* t_lo = nullptr; bf16* t2_hi = nullptr; bf16* t2_lo = nullptr;
  int64_t ld_t = 0; int64_t bs_t = 0;
  int gen_mode = tc::GEN_LINEAR;             // see tc::Params
  float* aux = nullptr; float tol = 0.f; int* moved_out = nullptr; int fail_if_moved = 0;
  // split-K: slice s of the reduction writes alpha * partial product (no addends, no split copy) to
  // f32 + s * split_stride; the caller reduces.
  int ksplit = 1; int64_t split_stride = 0;
  int tri_skip = 0, k_mode = 0;   // triangular structure, see tc::Params
  const int* tile_list = nullptr; int n_list = 0;   // explicit tile order (device), see tc::Params
  const int* tile_list2 = nullptr; int n_list2 = 0; // the same order in 256 x 256 tiles (two-CTA kernel)
  int nterms = 3;   // 1: plain bf16 product of the hi parts only (2^-9 relative), a third of the MMAs
  // nterms == 1 only: D = A B^T - A2 B2^T in one reduction (second operand pair, same shapes)
  const Op* dual_a = nullptr; const Op* dual_b = nullptr;
  const int* run_if = nullptr;       // device flag: skip the product when it is 0 (see tc::Params)
  const int* run_unless = nullptr;   // device flag: skip the product when it is not 0
};

inline void fill_epilogue(tc::Params& p, const Out& o) {
  p.out = o.f32; p.ld = o.ld; p.batch_stride = o.bs; p.split_stride = o.split_stride;
  p.out_hi = o.hi; p.out_lo = o.lo; p.out2_hi = o.hi2; p.out2_lo = o.lo2; p.ld_h = o.ld_h; p.batch_stride_h = o.bs_h;
  p.alpha = o.alpha;
  p.add1 = o.add1; p.g1 = o.g1; p.add2 = o.add2; p.g2 = o.g2;
  if (o.beta != 0.f) {   // the output accumulates: its old contents are the (first free) addend
    if (!p.add1) { p.add1 = o.f32; p.g1 = o.beta; } else { p.add2 = o.f32; p.g2 = o.beta; }
  }
  p.out_t_hi = o.t_hi; p.out_t_lo = o.t_lo; p.out_t2_hi = o.t2_hi; p.out_t2_lo = o.t2_lo;
  p.ld_t = o.ld_t; p.batch_stride_t = o.bs_t;
  p.gen_mode = o.gen_mode; p.aux = o.aux; p.tol = o.tol; p.moved_out = o.moved_out; p.fail_if_moved = o.fail_if_moved;
  p.k_dual = (o.dual_a && o.dual_b) ? 1 : 0;
  p.tri_skip = o.tri_skip; p.k_mode = o.k_mode;
  p.run_if = o.run_if; p.run_unless = o.run_unless;
  p.partials = nullptr;
}

// 64-wide k-blocks the kernels run for a product: the same clipping as their k_range, over all tiles or
// (upper) over the tiles with mb <= nb.  unit = tile edge (128 or 256).
inline int64_t count_kblocks(int m_tiles, int n_tiles, int k_blocks, int k_mode, bool upper, int unit) {
  const int R = unit / tc::BLOCK_K;
  int64_t total = 0;
  for (int nb = 0; nb < n_tiles; ++nb)
    for (int mb = 0; mb < m_tiles; ++mb) {
      if (upper && mb > nb) continue;
      int lo = 0, hi = k_blocks;
      if ((k_mode & 1) && lo < R * mb) lo = R * mb;
      if ((k_mode & 8) && lo < R * nb) lo = R * nb;
      if ((k_mode & 2) && hi > R * (mb + 1)) hi = R * (mb + 1);
      if ((k_mode & 4) && hi > R * (nb + 1)) hi = R * (nb + 1);
      if (hi > lo) total += hi - lo;
    }
  return total;
}

// D[m][n] = alpha sum_k A[m][k] B[n][k] (+ beta D) with split-bf16 operands (three bf16 MMAs per
// product, fp32 accumulation); M, N % 128 == 0, K % 64 == 0.
inline dq_status gemm3(Ctx& ctx, const Op& A, const Op& B, int M, int N, int K, int batch, const Out& o) {
  if (M % 128 || N % 128 || K % 64 || o.ksplit < 1 || o.ksplit > K / 64) return DQ_ERR_UNSUPPORTED;
  if ((o.tri_skip || o.k_mode) && (o.ksplit != 1 || M != N)) return DQ_ERR_UNSUPPORTED;
  const bool dual = o.dual_a && o.dual_b;
  if (dual && (o.nterms != 1 || o.k_mode || o.ksplit != 1)) return DQ_ERR_UNSUPPORTED;
  {   // the epilogue moves 32 bytes per access: bases, leading dimensions and strides must keep rows 32-byte aligned
    auto bad = [](const void* ptr, int64_t ld, int64_t bs, int esz) {
      return ptr && ((((uintptr_t)ptr) & 31) || (ld * esz) % 32 || (bs * esz) % 32);
    };
    if (bad(o.f32, o.ld, o.bs, 4) || bad(o.add1, o.ld, o.bs, 4) || bad(o.add2, o.ld, o.bs, 4) || bad(o.aux, o.ld, o.bs, 4) ||
        bad(o.hi, o.ld_h, o.bs_h, 2) || bad(o.lo, o.ld_h, o.bs_h, 2) || bad(o.hi2, o.ld_h, o.bs_h, 2) ||
        bad(o.lo2, o.ld_h, o.bs_h, 2) || (o.split_stride * 4) % 32)
      return DQ_ERR_UNSUPPORTED;
  }
  if (o.ksplit > 1 && (o.add1 || o.add2 || o.beta != 0.f || o.hi || o.t_hi || o.gen_mode != tc::GEN_LINEAR))
    return DQ_ERR_UNSUPPORTED;
  // second pair of tensor maps: the lo parts of a split product, or the second operand pair of a dual one
  const bf16* a2 = dual ? o.dual_a->hi : (o.nterms == 1 ? A.hi : A.lo);
  const bf16* b2 = dual ? o.dual_b->hi : (o.nterms == 1 ? B.hi : B.lo);
  const int64_t lda2 = dual ? o.dual_a->ld : A.ld, ldb2 = dual ? o.dual_b->ld : B.ld;
  CUtensorMap ma, mal, mb, mbl;
  if (dual && (o.dual_a->t != A.t || o.dual_b->t != B.t)) return DQ_ERR_UNSUPPORTED;   // one orientation per operand
  const int64_t bsa = A.bs ? A.bs : (int64_t)(A.t ? K : M) * A.ld, bsb = B.bs ? B.bs : (int64_t)(B.t ? K : N) * B.ld;
  const int64_t bsa2 = dual ? (o.dual_a->bs ? o.dual_a->bs : (int64_t)(A.t ? K : M) * lda2) : bsa;
  const int64_t bsb2 = dual ? (o.dual_b->bs ? o.dual_b->bs : (int64_t)(B.t ? K : N) * ldb2) : bsb;
  // Large products run on CTA pairs (256 x 256 tiles, half the operand traffic per MMA); a caller that
  // orders its tiles must also give the order in pair tiles.
  const bool pair_ok = M % 256 == 0 && N % 256 == 0 && (!o.tile_list || o.tile_list2) && ctx.sm_count >= 2 &&
                       (int64_t)(M / 256) * (N / 256) * batch * o.ksplit >= 32;
  const int unit = pair_ok ? 256 : 128;
  const int box = pair_ok ? tc2::HALF : 128;
  // (a transposed operand: the stored matrix has K rows; boxes of 64 k x 64 columns)
  if (A.t) {
    DQ_CHECK(make_map(&ma, A.hi, M, K, batch, A.ld, bsa, tc::BLOCK_K));
    DQ_CHECK(make_map(&mal, a2, M, K, batch, lda2, bsa2, tc::BLOCK_K));
  } else {
    DQ_CHECK(make_map(&ma, A.hi, K, M, batch, A.ld, bsa, pair_ok ? tc2::HALF : tc::BLOCK_M));
    DQ_CHECK(make_map(&mal, a2, K, M, batch, lda2, bsa2, pair_ok ? tc2::HALF : tc::BLOCK_M));
  }
  if (B.t) {
    DQ_CHECK(make_map(&mb, B.hi, N, K, batch, B.ld, bsb, tc::BLOCK_K));
    DQ_CHECK(make_map(&mbl, b2, N, K, batch, ldb2, bsb2, tc::BLOCK_K));
  } else {
    DQ_CHECK(make_map(&mb, B.hi, K, N, batch, B.ld, bsb, box));
    DQ_CHECK(make_map(&mbl, b2, K, N, batch, ldb2, bsb2, box));
  }
  tc::Params p{};
  p.m_blocks = M / unit; p.n_blocks = N / unit; p.batch = batch; p.ksplit = o.ksplit; p.k_blocks = K / tc::BLOCK_K;
  fill_epilogue(p, o);
  p.a_mn = A.t ? 1 : 0; p.b_mn = B.t ? 1 : 0;
  p.d_status = ctx.d_status;
  p.tile_list = pair_ok ? o.tile_list2 : o.tile_list;
  p.n_list = pair_ok ? o.n_list2 : o.n_list;
  {
    const bool listed = p.tile_list && p.n_list < p.m_blocks * p.n_blocks;
    if (!o.run_if && !o.run_unless) {   // products that a device flag may skip are left out of the count
      const int64_t kb = listed && !o.k_mode ? (int64_t)p.n_list * p.k_blocks
                                             : count_kblocks(p.m_blocks, p.n_blocks, p.k_blocks, o.k_mode,
                                                             o.tri_skip || listed, unit);
      ctx.mma_flops += (double)kb * (2.0 * unit * unit * tc::BLOCK_K) * (dual ? 2 : (o.nterms == 1 ? 1 : 3)) * batch;
    }
  }
  if (pair_ok)
    return o.nterms == 1 ? launch_gemm2<1, tc::EPI_GEN>(ctx, ma, mb, mal, mbl, p)
                         : launch_gemm2<3, tc::EPI_GEN>(ctx, ma, mb, mal, mbl, p);
  return o.nterms == 1 ? launch_gemm<128, 1, tc::EPI_GEN>(ctx, ma, mb, mal, mbl, p)
                       : launch_gemm<128, 3, tc::EPI_GEN>(ctx, ma, mb, mal, mbl, p);
}

}  // namespace tch
}  // namespace dq
