// QR-Orth on the tensor cores (used with the tensor-core path).
//
// Forward:  U of Z = R U either by the blocked Householder factorisation (qr_panel_tc.cu kernels
//           with the compact-WY products issued here) or, from the second step on, incrementally:
//           U = (I + T) U_old with T from fixed-point sweeps on (Z U_old^-1)^T (Z U_old^-1).
//           Then W = U^-1 by recursive block inversion and R = Z W.  (R is the same orthogonal
//           factor the reflectors would give; forming it as Z U^-1 costs one GEMM instead of
//           d / 128 dependent block updates.  Its orthogonality error grows like cond(Z) * 2^-17.)
// Backward: B = R^T Gq, S = tril(B - B^T, -1), Gz = R (S W^T).
// All d x d products run as split-bf16 tcgen05 GEMMs (three bf16 MMAs per product, fp32
// accumulation, ~2^-17 relative error), clipped to the non-zero blocks of triangular operands.
#include <algorithm>
#include <vector>

#include "tc_host.cuh"
#include "tc_path.cuh"

namespace dq {
namespace {

using bf16 = __nv_bfloat16;

__device__ __forceinline__ void split2(float v, bf16& hi, bf16& lo) {
  hi = __float2bfloat16_rn(v);
  lo = __float2bfloat16_rn(v - __bfloat162float(hi));
}

// dst(hi, lo)[b][r][c] = split(src[b][r][c])             (transpose == 0)
// dst(hi, lo)[b][c][r] = split(src[b][r][c])             (transpose == 1)
// src is n x n fp32 row-major (n % 32 == 0); dst dense n x n.
__global__ void __launch_bounds__(256) split_kernel(const float* __restrict__ src, bf16* __restrict__ hi,
                                                    bf16* __restrict__ lo, int n, int transpose) {
  __shared__ float t[32][33];
  const int64_t off = (int64_t)blockIdx.z * n * n;
  src += off; hi += off; lo += off;
  const int r0 = blockIdx.y * 32, c0 = blockIdx.x * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  if (!transpose) {
    for (int r = ty; r < 32; r += 8) {
      const int64_t i = (int64_t)(r0 + r) * n + c0 + tx;
      split2(src[i], hi[i], lo[i]);
    }
  } else {
    for (int r = ty; r < 32; r += 8) t[r][tx] = src[(int64_t)(r0 + r) * n + c0 + tx];
    __syncthreads();
    for (int c = ty; c < 32; c += 8) {
      const int64_t i = (int64_t)(c0 + c) * n + r0 + tx;
      split2(t[tx][c], hi[i], lo[i]);
    }
  }
}

// S(hi, lo) = split of S = tril(B - B^T, -1), row-major:  S[i][j] = (i > j) ? B[i][j] - B[j][i] : 0
__global__ void __launch_bounds__(256) skew_split_kernel(const float* __restrict__ B, bf16* __restrict__ hi,
                                                         bf16* __restrict__ lo, int d) {
  __shared__ float t[32][33];
  const int64_t off = (int64_t)blockIdx.z * d * d;
  B += off; hi += off; lo += off;
  const int i0 = blockIdx.y * 32, j0 = blockIdx.x * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  if (j0 >= i0 + 31) {   // tile entirely on or above the diagonal: zeros
    for (int r = ty; r < 32; r += 8) {
      const int64_t i = (int64_t)(i0 + r) * d + j0 + tx;
      hi[i] = __float2bfloat16_rn(0.f); lo[i] = __float2bfloat16_rn(0.f);
    }
    return;
  }
  for (int r = ty; r < 32; r += 8) t[r][tx] = B[(int64_t)(j0 + r) * d + i0 + tx];   // B[j][i]
  __syncthreads();
  for (int r = ty; r < 32; r += 8) {
    const int i = i0 + r, j = j0 + tx;
    const int64_t idx = (int64_t)i * d + j;
    const float v = (i > j) ? B[idx] - t[tx][r] : 0.f;
    split2(v, hi[idx], lo[idx]);
  }
}

// One sweep of the fixed-point iteration for the Cholesky factor U = I + T of G = Z^T Z:
//   T <- striu(G - I - P) + diag(G - I - P) / 2,   P = T^T T (nullptr on the first sweep: T = 0).
// G and P are only valid on and above the diagonal.  Writes T (fp32, row-major, zeros below the
// diagonal), the split-bf16 copy of T^T (operand of the next P = T^T T) and, if U is given,
// U = I + T with its split copy.
// run_if (nullable): the sweep is skipped when *run_if == 0 (the previous sweep moved nothing).
// moved_out (nullable): set to 1 if an entry moved by more than tol (0 otherwise: the caller clears it).
// fail_if_moved: that case also sets DQ_ERR_NOT_CONVERGED (last sweep the schedule allows).
// lower_done: tiles strictly below the diagonal already hold their zeros.
__global__ void __launch_bounds__(256) chol_fixpoint_kernel(const float* __restrict__ G, const float* __restrict__ P,
                                                            float* __restrict__ T, bf16* __restrict__ tt_hi,
                                                            bf16* __restrict__ tt_lo, float* __restrict__ U,
                                                            bf16* __restrict__ u_hi, bf16* __restrict__ u_lo, int d,
                                                            const int* __restrict__ run_if, int* __restrict__ moved_out,
                                                            int fail_if_moved, int lower_done, float tol,
                                                            int* d_status) {
  __shared__ float t[32][33];
  if (run_if && *run_if == 0) return;
  const int64_t off = (int64_t)blockIdx.z * d * d;
  G += off; T += off; tt_hi += off; tt_lo += off;
  if (P) P += off;
  if (U) { U += off; u_hi += off; u_lo += off; }
  const int i0 = blockIdx.y * 32, j0 = blockIdx.x * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const bool upper = j0 + 31 >= i0;     // tile touches the upper triangle
  if (!upper && lower_done && !U) return;   // zeros written by an earlier sweep stay zeros
  bool moved = false;
  for (int r = ty; r < 32; r += 8) {
    const int i = i0 + r, j = j0 + tx;
    const int64_t idx = (int64_t)i * d + j;
    float v = 0.f;
    if (upper && j >= i) {
      v = G[idx] - ((i == j) ? 1.f : 0.f) - (P ? P[idx] : 0.f);
      if (i == j) v *= 0.5f;
      if (P && !(fabsf(v - T[idx]) <= tol)) moved = true;
    }
    T[idx] = v;
    t[r][tx] = v;
    if (U) {
      const float u = v + ((i == j) ? 1.f : 0.f);
      U[idx] = u;
      split2(u, u_hi[idx], u_lo[idx]);
    }
  }
  if (moved) {
    if (moved_out) *moved_out = 1;
    if (fail_if_moved) set_status(d_status, DQ_ERR_NOT_CONVERGED);
  }
  __syncthreads();
  for (int c = ty; c < 32; c += 8) {    // T^T[j][i] = T[i][j]
    const int64_t idx = (int64_t)(j0 + c) * d + i0 + tx;
    split2(t[tx][c], tt_hi[idx], tt_lo[idx]);
  }
}

// Inverse of each 128 x 128 upper-triangular diagonal block of U, one CTA per block: the four
// 32 x 32 diagonal sub-blocks by back-substitution (one warp each, lane j solves U x = e_j), then
// inv([A B; 0 C]) = [A^-1, -A^-1 B C^-1; 0, C^-1] twice as shared-memory products.  Writes the
// split inverse in row-major (WN) and transposed (WT) form.
constexpr int DB = 128;
constexpr int DLD = 129;
constexpr int TRI_INV_THREADS = 256;
constexpr int TRI_INV_SMEM = (2 * DB * DLD + 64 * 65) * 4;

__device__ __forceinline__ void smem_mm4(const float* A, int lda, const float* B, int ldb, float* C, int ldc, int M,
                                         int N, int K, float alpha, int tid) {
  const int tn = N / 4, tiles = (M / 4) * tn;
  for (int t = tid; t < tiles; t += TRI_INV_THREADS) {
    const int r0 = (t / tn) * 4, c0 = (t % tn) * 4;
    float acc[4][4] = {};
    for (int k = 0; k < K; ++k) {
      float av[4], bv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) av[i] = A[(r0 + i) * lda + k];
#pragma unroll
      for (int j = 0; j < 4; ++j) bv[j] = B[k * ldb + c0 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) C[(r0 + i) * ldc + c0 + j] = alpha * acc[i][j];
  }
}

__global__ void __launch_bounds__(TRI_INV_THREADS) tri_inv_diag128_kernel(const float* __restrict__ U,
                                                                          bf16* __restrict__ wn_hi,
                                                                          bf16* __restrict__ wn_lo,
                                                                          bf16* __restrict__ wt_hi,
                                                                          bf16* __restrict__ wt_lo, int d) {
  extern __shared__ float sm[];
  float* Us = sm;
  float* Xs = sm + DB * DLD;
  float* Tmp = Xs + DB * DLD;
  const int64_t off = (int64_t)blockIdx.y * d * d + (int64_t)blockIdx.x * DB * (d + 1);
  U += off; wn_hi += off; wn_lo += off; wt_hi += off; wt_lo += off;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int e = tid; e < DB * DB; e += TRI_INV_THREADS) {
    const int r = e >> 7, c = e & 127;
    Us[r * DLD + c] = U[(int64_t)r * d + c];
    Xs[r * DLD + c] = 0.f;
  }
  __syncthreads();
  if (warp < 4) {
    const int o = warp * 32, j = lane;
    Xs[(o + j) * DLD + o + j] = 1.f / Us[(o + j) * DLD + o + j];
    for (int i = j - 1; i >= 0; --i) {
      float s = 0.f;
      for (int k = i + 1; k <= j; ++k) s = fmaf(Us[(o + i) * DLD + o + k], Xs[(o + k) * DLD + o + j], s);
      Xs[(o + i) * DLD + o + j] = -s / Us[(o + i) * DLD + o + i];
    }
  }
  __syncthreads();
  for (int pair = 0; pair < 2; ++pair) {
    const int o = pair * 64;
    smem_mm4(Us + o * DLD + o + 32, DLD, Xs + (o + 32) * DLD + o + 32, DLD, Tmp, 65, 32, 32, 32, 1.f, tid);
    __syncthreads();
    smem_mm4(Xs + o * DLD + o, DLD, Tmp, 65, Xs + o * DLD + o + 32, DLD, 32, 32, 32, -1.f, tid);
    __syncthreads();
  }
  smem_mm4(Us + 64, DLD, Xs + 64 * DLD + 64, DLD, Tmp, 65, 64, 64, 64, 1.f, tid);
  __syncthreads();
  smem_mm4(Xs, DLD, Tmp, 65, Xs + 64, DLD, 64, 64, 64, -1.f, tid);
  __syncthreads();
  for (int e = tid; e < DB * DB; e += TRI_INV_THREADS) {
    const int r = e >> 7, c = e & 127;
    bf16 h, l;
    split2(Xs[r * DLD + c], h, l);                 // X[r][c] -> WN[r][c]
    wn_hi[(int64_t)r * d + c] = h; wn_lo[(int64_t)r * d + c] = l;
    split2(Xs[c * DLD + r], h, l);                 // X[c][r] -> WT[r][c]
    wt_hi[(int64_t)r * d + c] = h; wt_lo[(int64_t)r * d + c] = l;
  }
}

using tch::Op;
using tch::Out;
using tch::gemm3;

// Block column of the inverse:  W[0:k, k:k+s] = -W[0:k,0:k] U[0:k, k:k+s] W[k:k+s, k:k+s]
// for `count` independent diagonal positions `stride` elements apart (3rd tensor dimension).
dq_status merge(Ctx& ctx, QrTcState& q, int d, int k, int s, int count, int64_t stride, int64_t base) {
  // T1t[j][i] = sum_l W22^T[j][l] U12[i][l]        (s x k, dense temporary)
  Op a{q.wt_hi + base + (int64_t)k * d + k, q.wt_lo + base + (int64_t)k * d + k, d, stride};
  Op b{q.u_hi + base + k, q.u_lo + base + k, d, stride};
  Out t1; t1.hi = q.t1_hi; t1.lo = q.t1_lo; t1.ld_h = k; t1.bs_h = (int64_t)s * k;
  DQ_CHECK(gemm3(ctx, a, b, s, k, s, count, t1));
  Op w11{q.wn_hi + base, q.wn_lo + base, d, stride};
  Op t1o{q.t1_hi, q.t1_lo, k, (int64_t)s * k};
  // W12[i][j] = -sum_l W11[i][l] T1t[j][l]   -> WN block (0, k)
  Out o12; o12.hi = q.wn_hi + base + k; o12.lo = q.wn_lo + base + k; o12.ld_h = d; o12.bs_h = stride; o12.alpha = -1.f;
  DQ_CHECK(gemm3(ctx, w11, t1o, k, s, k, count, o12));
  // W12^T[j][i] = -sum_l T1t[j][l] W11[i][l] -> WT block (k, 0)
  Out o21; o21.hi = q.wt_hi + base + (int64_t)k * d; o21.lo = q.wt_lo + base + (int64_t)k * d; o21.ld_h = d;
  o21.bs_h = stride; o21.alpha = -1.f;
  return gemm3(ctx, t1o, w11, s, k, k, count, o21);
}

dq_status tri_inverse_tc(Ctx& ctx, QrTcState& q, const float* U, int d, int batch) {
  const int64_t dd = (int64_t)d * d;
  const size_t bytes = sizeof(bf16) * (size_t)dd * batch;
  DQ_CHECK_CUDA(cudaMemsetAsync(q.wn_hi, 0, bytes, ctx.stream));
  DQ_CHECK_CUDA(cudaMemsetAsync(q.wn_lo, 0, bytes, ctx.stream));
  DQ_CHECK_CUDA(cudaMemsetAsync(q.wt_hi, 0, bytes, ctx.stream));
  DQ_CHECK_CUDA(cudaMemsetAsync(q.wt_lo, 0, bytes, ctx.stream));
  const int smem = TRI_INV_SMEM;
  static SmemOptIn attr;
  DQ_CHECK(opt_in_dynamic_smem(tri_inv_diag128_kernel, smem, attr));
  tri_inv_diag128_kernel<<<dim3(d / DB, batch), TRI_INV_THREADS, smem, ctx.stream>>>(U, q.wn_hi, q.wn_lo, q.wt_hi, q.wt_lo, d);
  DQ_CHECK(after_launch(ctx));
  int s = DB, count = d / DB;
  while (count > 1 && count % 2 == 0) {
    const int pairs = count / 2;
    const int64_t pair_stride = (int64_t)2 * s * (d + 1);
    if (batch == 1) {
      DQ_CHECK(merge(ctx, q, d, s, s, pairs, pair_stride, 0));
    } else {
      for (int pidx = 0; pidx < pairs; ++pidx) DQ_CHECK(merge(ctx, q, d, s, s, batch, dd, pidx * pair_stride));
    }
    s *= 2; count = pairs;
  }
  for (int kb = 1; kb < count; ++kb) DQ_CHECK(merge(ctx, q, d, kb * s, s, batch, dd, 0));
  return DQ_OK;
}

template <typename T>
dq_status alloc(T** p, int64_t n) {
  return cudaMalloc((void**)p, sizeof(T) * (size_t)n) == cudaSuccess ? DQ_OK : DQ_ERR_ALLOC;
}

// Split-K factor of the [S; W^T] product of an outer block with m active rows: fill the SMs,
// keep at least two 64-row k-blocks per slice.
int wy_ksplit(int m, int batch, int sm_count) {
  const int tiles = (m / 128) * batch;
  int ks = sm_count / tiles;
  if (ks > m / 128) ks = m / 128;
  return ks < 1 ? 1 : ks;
}

}  // namespace

dq_status qr_tc_init(QrTcState& q, int d, int batch, int sm_count) {
  const int64_t dd = (int64_t)d * d * batch;
  bf16** all[] = {&q.z_hi, &q.z_lo, &q.u_hi, &q.u_lo, &q.wn_hi, &q.wn_lo, &q.wt_hi, &q.wt_lo, &q.r_hi, &q.r_lo,
                  &q.rt_hi, &q.rt_lo, &q.gqt_hi, &q.gqt_lo, &q.st_hi, &q.st_lo, &q.m_hi, &q.m_lo, &q.t1_hi, &q.t1_lo};
  for (bf16** p : all) DQ_CHECK(alloc(p, dd));
  const int64_t yb = (int64_t)d * 128 * batch;
  DQ_CHECK(alloc(&q.y_hi, yb)); DQ_CHECK(alloc(&q.y_lo, yb));
  DQ_CHECK(alloc(&q.w2_hi, yb)); DQ_CHECK(alloc(&q.w2_lo, yb));
  DQ_CHECK(alloc(&q.T, (int64_t)128 * 128 * batch));
  q.part_bs = 0;
  for (int m = d; m > 128; m -= 128) {
    const int64_t e = (int64_t)wy_ksplit(m, batch, sm_count) * m * 128;
    if (e > q.part_bs) q.part_bs = e;
  }
  if (q.part_bs > 0) DQ_CHECK(alloc(&q.part, q.part_bs * batch));
  DQ_CHECK(alloc(&q.tw_hi, dd)); DQ_CHECK(alloc(&q.tw_lo, dd));
  DQ_CHECK(alloc(&q.sweep_flags, 80));
  DQ_CHECK(alloc(&q.uot_hi, dd)); DQ_CHECK(alloc(&q.uot_lo, dd));
  for (int unit = 128; unit <= 256; unit *= 2) {   // tile orders: most expensive tiles first, dealt round-robin to the persistent CTAs
    if (d % unit != 0) break;
    const int nb = d / unit;
    std::vector<int> upper, desc, asc;
    for (int j = 0; j < nb; ++j)
      for (int i = 0; i < nb; ++i) {
        if (i <= j) upper.push_back(i | (j << 16));
        desc.push_back(i | (j << 16));
      }
    std::stable_sort(upper.begin(), upper.end(), [](int a, int b) { return (a & 0xffff) > (b & 0xffff); });
    std::stable_sort(desc.begin(), desc.end(), [](int a, int b) { return (a >> 16) > (b >> 16); });
    asc = desc;
    std::reverse(asc.begin(), asc.end());
    int*& tu = (unit == 128) ? q.tl_upper : q.tl2_upper;
    int*& td = (unit == 128) ? q.tl_desc_nb : q.tl2_desc_nb;
    int*& ta = (unit == 128) ? q.tl_asc_nb : q.tl2_asc_nb;
    ((unit == 128) ? q.n_upper : q.n2_upper) = (int)upper.size();
    ((unit == 128) ? q.n_all : q.n2_all) = (int)desc.size();
    DQ_CHECK(alloc(&tu, (int64_t)upper.size())); DQ_CHECK(alloc(&td, (int64_t)desc.size())); DQ_CHECK(alloc(&ta, (int64_t)desc.size()));
    DQ_CHECK_CUDA(cudaMemcpy(tu, upper.data(), sizeof(int) * upper.size(), cudaMemcpyHostToDevice));
    DQ_CHECK_CUDA(cudaMemcpy(td, desc.data(), sizeof(int) * desc.size(), cudaMemcpyHostToDevice));
    DQ_CHECK_CUDA(cudaMemcpy(ta, asc.data(), sizeof(int) * asc.size(), cudaMemcpyHostToDevice));
  }
  q.ready = true;
  return DQ_OK;
}

void qr_tc_destroy(QrTcState& q) {
  bf16* all[] = {q.z_hi, q.z_lo, q.u_hi, q.u_lo, q.wn_hi, q.wn_lo, q.wt_hi, q.wt_lo, q.r_hi, q.r_lo,
                 q.rt_hi, q.rt_lo, q.gqt_hi, q.gqt_lo, q.st_hi, q.st_lo, q.m_hi, q.m_lo, q.t1_hi, q.t1_lo};
  for (bf16* p : all) cudaFree(p);
  cudaFree(q.y_hi); cudaFree(q.y_lo); cudaFree(q.w2_hi); cudaFree(q.w2_lo); cudaFree(q.part); cudaFree(q.T);
  cudaFree(q.tw_hi); cudaFree(q.tw_lo); cudaFree(q.uot_hi); cudaFree(q.uot_lo); cudaFree(q.tl_upper); cudaFree(q.tl_desc_nb); cudaFree(q.tl_asc_nb);
  cudaFree(q.tl2_upper); cudaFree(q.tl2_desc_nb); cudaFree(q.tl2_asc_nb); cudaFree(q.sweep_flags);
  q = QrTcState();
}

// Blocked Householder factorisation of Z on the transposed working matrix ws.A (= A^T): 128-column
// outer blocks, panel on the CUDA cores, compact-WY trailing update as split-bf16 tensor-core GEMMs.
// On return ws.A holds U^T on / below its diagonal (raw signs of Algorithm 2).
dq_status qr_factor_tc(Ctx& ctx, QrWorkspace& ws, QrTcState& q, const float* Z, int d, int batch) {
  const int64_t dd = (int64_t)d * d, yb = (int64_t)d * 128;
  float* At = ws.A;
  bf16 *at_hi = q.st_hi, *at_lo = q.st_lo;   // free until the backward pass
  DQ_CHECK(qrp_transpose_split(ctx, Z, At, at_hi, at_lo, d, batch));
  for (int c0 = 0; c0 < d; c0 += 128) {
    const int m = d - c0, n = m - 128;
    DQ_CHECK(qrp_panel(ctx, At, at_hi, at_lo, q.y_hi, q.y_lo, q.T, d, c0, batch));
    if (n == 0) break;
    const int64_t o = (int64_t)c0 * d + c0;
    // [S; W^T][i][j] = sum_r At[c0 + i][r] Y^T[j][r], r in [c0, d): rows 0..127 are Y^T Y, the rest W^T
    const int ks = wy_ksplit(m, batch, ctx.sm_count);
    Op a{at_hi + o, at_lo + o, d, dd}, b{at_hi + o, at_lo + o, d, dd};
    Out sw; sw.f32 = q.part; sw.ld = 128; sw.bs = q.part_bs; sw.ksplit = ks; sw.split_stride = (int64_t)m * 128;
    DQ_CHECK(gemm3(ctx, a, b, m, 128, m, batch, sw));
    DQ_CHECK(qrp_wy_w2(ctx, q.part, ks, m, q.part_bs, q.T, q.w2_hi, q.w2_lo, yb, n, batch));
    // C^T[c][r] -= sum_j W2^T[c][j] Y[r][j]
    Op w2{q.w2_hi, q.w2_lo, 128, yb}, y{q.y_hi + (int64_t)c0 * 128, q.y_lo + (int64_t)c0 * 128, 128, yb};
    const int64_t oc = o + (int64_t)128 * d;
    Out up; up.f32 = At + oc; up.ld = d; up.bs = dd; up.hi = at_hi + oc; up.lo = at_lo + oc; up.ld_h = d; up.bs_h = dd;
    up.alpha = -1.f; up.beta = 1.f;
    DQ_CHECK(gemm3(ctx, w2, y, n, m, 128, batch, up));
  }
  return qr_diag_check(ctx, At, d, batch);
}

// U of the latent one optimiser step after a latent whose factors (U_old, W_old = U_old^-1) are
// known, without dependent column steps.  Zh = Z W_old is close to orthogonal however far Z itself
// has drifted (Zh = R_old + (Z - Z_old) W_old), so its upper factor Uh = I + T is the fixed point of
//   T <- Phi(Zh^T Zh - I - T^T T),  Phi(S) = striu(S) + diag(S) / 2,
// reached from T = 0 in a few sweeps; then U = Uh U_old.  Every product is a split-bf16
// tensor-core GEMM restricted to the non-zero blocks of its triangular operands.
dq_status qr_upper_factor_incremental(Ctx& ctx, QrWorkspace& ws, QrTcState& q, const float* Z, float* U, int d,
                                      int batch, int n_sweeps) {
  const int64_t dd = (int64_t)d * d;
  const dim3 tiles(d / 32, d / 32, batch);
  bf16 *zht_hi = q.st_hi, *zht_lo = q.st_lo;   // free until the backward pass
  bf16 *uh_hi = q.gqt_hi, *uh_lo = q.gqt_lo;   // likewise
  float *Zh = ws.A, *G = ws.B, *P = ws.S, *T = ws.tmp, *scratch = ws.Q;
  if (!q.z_split_fresh) {   // (the SGD update writes the split copy with the new latent)
    split_kernel<<<tiles, 256, 0, ctx.stream>>>(Z, q.z_hi, q.z_lo, d, 0);
    DQ_CHECK(after_launch(ctx));
    q.z_split_fresh = true;
  }
  {   // Zh[i][j] = sum_k Z[i][k] W_old[k][j]
    Op a{q.z_hi, q.z_lo, d, dd}, b{q.wt_hi, q.wt_lo, d, dd};
    Out o; o.f32 = Zh; o.ld = d; o.bs = dd; o.k_mode = 4; o.tile_list = q.tl_desc_nb; o.n_list = q.n_all; o.tile_list2 = q.tl2_desc_nb; o.n_list2 = q.n2_all;
    DQ_CHECK(gemm3(ctx, a, b, d, d, d, batch, o));
  }
  DQ_CHECK(qrp_transpose_split(ctx, Zh, scratch, zht_hi, zht_lo, d, batch));
  {   // G[i][j] = sum_k Zh[k][i] Zh[k][j], tiles on and above the block diagonal
    Op a{zht_hi, zht_lo, d, dd};
    Out o; o.f32 = G; o.ld = d; o.bs = dd; o.tile_list = q.tl_upper; o.n_list = q.n_upper; o.tile_list2 = q.tl2_upper; o.n_list2 = q.n2_upper;
    DQ_CHECK(gemm3(ctx, a, a, d, d, d, batch, o));
  }
  // Sweep 0 sets T = Phi(E).  Then up to n_sweeps cheap sweeps (plain bf16 product: its relative error 2^-9
  // acts on a term of size ||T||^2 and later sweeps forgive it by a factor ||T|| each), each skipped once
  // the sweep before it moved no entry by more than the tolerance, and finally up to three accurate sweeps
  // (split-bf16 product), the first always taken, the others only while entries still move.  flags[k] = 1
  // if sweep k moved something; the launch sequence is fixed, so a captured graph replays it unchanged.
  constexpr int ACCURATE = 3;
  int* flags = q.sweep_flags;
  DQ_CHECK_CUDA(cudaMemsetAsync(flags, 0, sizeof(int) * (n_sweeps + ACCURATE + 2), ctx.stream));
  chol_fixpoint_kernel<<<tiles, 256, 0, ctx.stream>>>(G, nullptr, T, q.tw_hi, q.tw_lo, nullptr, nullptr, nullptr, d,
                                                      nullptr, nullptr, 0, 0, 1e-5f, ctx.d_status);
  DQ_CHECK(after_launch(ctx));
  for (int it = 1; it <= n_sweeps + ACCURATE; ++it) {
    const bool accurate = it > n_sweeps;
    const bool first_accurate = it == n_sweeps + 1;
    const bool last = it == n_sweeps + ACCURATE;
    // cheap sweep 1 always runs; a later cheap sweep runs if the one before moved; the first accurate sweep
    // always runs; a later accurate sweep runs if the accurate sweep before it moved
    const int* run_if = (it == 1 || first_accurate) ? nullptr : flags + it - 1;
    {   // P[i][j] = sum_k T[k][i] T[k][j]; T^T is lower triangular: k < 128 (mb + 1), mb <= nb
      Op tt{q.tw_hi, q.tw_lo, d, dd};
      Out o; o.f32 = P; o.ld = d; o.bs = dd; o.k_mode = 2; o.tile_list = q.tl_upper; o.n_list = q.n_upper; o.tile_list2 = q.tl2_upper; o.n_list2 = q.n2_upper;
      o.nterms = accurate ? 3 : 1;
      o.run_if = run_if;
      DQ_CHECK(gemm3(ctx, tt, tt, d, d, d, batch, o));
    }
    chol_fixpoint_kernel<<<tiles, 256, 0, ctx.stream>>>(G, P, T, q.tw_hi, q.tw_lo, accurate ? scratch : nullptr, uh_hi,
                                                        uh_lo, d, run_if, flags + it, last ? 1 : 0, 1, 1e-5f,
                                                        ctx.d_status);
    DQ_CHECK(after_launch(ctx));
  }
  {   // U[i][j] = sum_k Uh[i][k] U_old[k][j]: both upper triangular, k in [128 mb, 128 (nb + 1))
    Op a{uh_hi, uh_lo, d, dd}, b{q.uot_hi, q.uot_lo, d, dd};
    Out o; o.f32 = U; o.ld = d; o.bs = dd; o.hi = q.u_hi; o.lo = q.u_lo; o.ld_h = d; o.bs_h = dd;
    o.k_mode = 1 | 4; o.tile_list = q.tl_upper; o.n_list = q.n_upper; o.tile_list2 = q.tl2_upper; o.n_list2 = q.n2_upper;
    DQ_CHECK(gemm3(ctx, a, b, d, d, d, batch, o));
  }
  return qr_diag_check(ctx, U, d, batch);
}

dq_status qr_forward_fast(Ctx& ctx, QrWorkspace& ws, QrTcState& q, const float* Z, float* R, float* U, int d,
                          int batch, int iterative_iters) {
  if (d % 128 != 0) return DQ_ERR_UNSUPPORTED;
  const int64_t dd = (int64_t)d * d;
  const dim3 tiles(d / 32, d / 32, batch);
  const bool incremental = iterative_iters > 0 && q.t_warm;
  if (incremental) {
    DQ_CHECK(qr_upper_factor_incremental(ctx, ws, q, Z, U, d, batch, iterative_iters));
  } else {   // no factors of a nearby latent yet (first call, latent replaced): Householder
    DQ_CHECK(qr_factor_tc(ctx, ws, q, Z, d, batch));
    DQ_CHECK(qrp_gauge_ut(ctx, ws.A, U, q.u_hi, q.u_lo, d, batch));
  }
  DQ_CHECK(tri_inverse_tc(ctx, q, U, d, batch));
  if (iterative_iters > 0) {   // U^T for the next step's U = Uh U_old
    split_kernel<<<tiles, 256, 0, ctx.stream>>>(U, q.uot_hi, q.uot_lo, d, 1);
    DQ_CHECK(after_launch(ctx));
    q.t_warm = true;
  }
  if (!q.z_split_fresh) {
    split_kernel<<<tiles, 256, 0, ctx.stream>>>(Z, q.z_hi, q.z_lo, d, 0);
    DQ_CHECK(after_launch(ctx));
    q.z_split_fresh = true;
  }
  // R[i][j] = sum_k Z[i][k] W[k][j]:  A = Z (row-major), B = W^T
  Op a{q.z_hi, q.z_lo, d, dd};
  Op b{q.wt_hi, q.wt_lo, d, dd};
  Out o; o.f32 = R; o.ld = d; o.bs = dd; o.hi = q.r_hi; o.lo = q.r_lo; o.ld_h = d; o.bs_h = dd;
  o.k_mode = 4;   // W is upper triangular: W^T[j][k] = 0 for k > j
  o.tile_list = q.tl_desc_nb; o.n_list = q.n_all; o.tile_list2 = q.tl2_desc_nb; o.n_list2 = q.n2_all;
  DQ_CHECK(gemm3(ctx, a, b, d, d, d, batch, o));
  split_kernel<<<tiles, 256, 0, ctx.stream>>>(R, q.rt_hi, q.rt_lo, d, 1);
  return after_launch(ctx);
}

dq_status qr_backward_tc(Ctx& ctx, QrWorkspace& ws, QrTcState& q, const float* Gq, float* Gz, int d, int batch) {
  const int64_t dd = (int64_t)d * d;
  const dim3 tiles(d / 32, d / 32, batch);
  split_kernel<<<tiles, 256, 0, ctx.stream>>>(Gq, q.gqt_hi, q.gqt_lo, d, 1);
  DQ_CHECK(after_launch(ctx));
  // B[i][j] = sum_k R[k][i] Gq[k][j]:  A = R^T, B-operand = Gq^T
  Op rt{q.rt_hi, q.rt_lo, d, dd}, gqt{q.gqt_hi, q.gqt_lo, d, dd};
  Out ob; ob.f32 = ws.B; ob.ld = d; ob.bs = dd;
  DQ_CHECK(gemm3(ctx, rt, gqt, d, d, d, batch, ob));
  skew_split_kernel<<<tiles, 256, 0, ctx.stream>>>(ws.B, q.st_hi, q.st_lo, d);
  DQ_CHECK(after_launch(ctx));
  // Gz = R S W^T = R D with D = S W^T lower triangular.  D^T[m][n] = sum_k W[m][k] S[n][k]: W[m][k] = 0 for
  // k < m and S[n][k] = 0 for k >= n, so only tiles mb <= nb with k in [128 mb, 128 (nb + 1)): a sixth of a
  // dense product (R S first would cost half of one).  Only the split copy of D^T is kept.
  Op wn{q.wn_hi, q.wn_lo, d, dd}, sr{q.st_hi, q.st_lo, d, dd};
  Out od; od.hi = q.m_hi; od.lo = q.m_lo; od.ld_h = d; od.bs_h = dd;
  od.k_mode = 1 | 4;
  od.tile_list = q.tl_upper; od.n_list = q.n_upper; od.tile_list2 = q.tl2_upper; od.n_list2 = q.n2_upper;
  DQ_CHECK(gemm3(ctx, wn, sr, d, d, d, batch, od));
  // (tiles below the block diagonal of D^T are neither written here nor read by the next product; the entries
  // below the diagonal inside the diagonal tiles come out as exact zeros)
  // Gz[i][j] = sum_k R[i][k] D^T[j][k]; D^T[j][k] = 0 for k < j
  Op r{q.r_hi, q.r_lo, d, dd}, dt{q.m_hi, q.m_lo, d, dd};
  Out og; og.f32 = Gz; og.ld = d; og.bs = dd;
  og.k_mode = 8;
  og.tile_list = q.tl_asc_nb; og.n_list = q.n_all; og.tile_list2 = q.tl2_asc_nb; og.n_list2 = q.n2_all;
  return gemm3(ctx, r, dt, d, d, d, batch, og);
}

}  // namespace dq
