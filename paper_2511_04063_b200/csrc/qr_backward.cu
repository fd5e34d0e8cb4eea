// QR-Orth backward: Gz = R tril(B - B^T, -1) U^-T with B = R^T Gq, the gradient of
// the latent for Z = R U (chain rule of Algorithm 1's update step through Sec. 4.3).
// U^-1 is formed explicitly: 64 x 64 diagonal blocks by back-substitution, then
// block merges  inv([U11 U12; 0 U22]) = [W11, -W11 U12 W22; 0, W22]  as GEMMs.
#include "common.cuh"

namespace dq {
namespace {

constexpr int IB = 64;

// S = tril(B - B^T, -1)
__global__ void __launch_bounds__(256) skew_lower_kernel(const float* __restrict__ B, float* __restrict__ S, int d) {
  __shared__ float t[32][33];
  const int64_t off = (int64_t)blockIdx.z * d * d;
  B += off; S += off;
  const int i0 = blockIdx.y * 32, j0 = blockIdx.x * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  if (j0 > i0) {   // tile strictly above the diagonal: zeros
    for (int r = ty; r < 32; r += 8) S[(int64_t)(i0 + r) * d + j0 + tx] = 0.f;
    return;
  }
  for (int r = ty; r < 32; r += 8) t[r][tx] = B[(int64_t)(j0 + r) * d + i0 + tx];   // B[j][i]
  __syncthreads();
  for (int r = ty; r < 32; r += 8) {
    const int i = i0 + r, j = j0 + tx;
    S[(int64_t)i * d + j] = (i > j) ? B[(int64_t)i * d + j] - t[tx][r] : 0.f;
  }
}

// Inverse of each 64 x 64 upper-triangular diagonal block; thread j solves U x = e_j.
__global__ void __launch_bounds__(IB) tri_inv_diag_kernel(const float* __restrict__ U, float* __restrict__ W, int d) {
  __shared__ float Us[IB][IB + 1];
  __shared__ float Xs[IB][IB + 1];
  const int64_t off = (int64_t)blockIdx.y * d * d + (int64_t)blockIdx.x * IB * (d + 1);
  U += off; W += off;
  const int j = threadIdx.x;
  for (int r = 0; r < IB; ++r) Us[r][j] = U[(int64_t)r * d + j];
  __syncthreads();
  for (int i = IB - 1; i > j; --i) Xs[i][j] = 0.f;
  Xs[j][j] = 1.f / Us[j][j];
  for (int i = j - 1; i >= 0; --i) {
    float s = 0.f;
    for (int k = i + 1; k <= j; ++k) s = fmaf(Us[i][k], Xs[k][j], s);
    Xs[i][j] = -s / Us[i][i];
  }
  __syncthreads();
  for (int r = 0; r < IB; ++r) W[(int64_t)r * d + j] = Xs[r][j];
}

// W[0:k, k:k+s] = -W[0:k, 0:k] U[0:k, k:k+s] W[k:k+s, k:k+s]   (offsets in elements)
dq_status merge_block(Ctx& ctx, QrWorkspace& ws, const float* U, int d, int k, int s, int count,
                      int64_t stride, int batch_for_stride) {
  GemmDesc a{};
  a.A = U + k; a.lda = d; a.transA = 0; a.sA = stride;                 // U12: rows 0..k, cols k..k+s
  a.B = ws.Winv + (int64_t)k * d + k; a.ldb = d; a.transB = 0; a.sB = stride;   // W22
  a.C = ws.tmp; a.ldc = s; a.sC = (int64_t)k * s;
  a.M = k; a.N = s; a.K = s; a.alpha = 1.f; a.beta = 0.f; a.batch = count;
  (void)batch_for_stride;
  DQ_CHECK(gemm_f32(ctx, a));
  GemmDesc b{};
  b.A = ws.Winv; b.lda = d; b.transA = 0; b.sA = stride;                // W11
  b.B = ws.tmp; b.ldb = s; b.transB = 0; b.sB = (int64_t)k * s;
  b.C = ws.Winv + k; b.ldc = d; b.sC = stride;
  b.M = k; b.N = s; b.K = k; b.alpha = -1.f; b.beta = 0.f; b.batch = count;
  return gemm_f32(ctx, b);
}

dq_status tri_inverse(Ctx& ctx, QrWorkspace& ws, const float* U, int d, int batch) {
  const int64_t dd = (int64_t)d * d;
  DQ_CHECK_CUDA(cudaMemsetAsync(ws.Winv, 0, sizeof(float) * dd * batch, ctx.stream));
  if (d % IB != 0) return DQ_ERR_UNSUPPORTED;
  tri_inv_diag_kernel<<<dim3(d / IB, batch), IB, 0, ctx.stream>>>(U, ws.Winv, d);
  DQ_CHECK(after_launch(ctx));
  int s = IB, count = d / IB;
  // pairwise merges while the number of blocks is even
  while (count > 1 && count % 2 == 0) {
    const int pairs = count / 2;
    const int64_t pair_stride = (int64_t)2 * s * (d + 1);
    if (batch == 1) {
      DQ_CHECK(merge_block(ctx, ws, U, d, s, s, pairs, pair_stride, 0));
    } else {
      for (int p = 0; p < pairs; ++p) {
        QrWorkspace w2 = ws;
        w2.Winv = ws.Winv + p * pair_stride;
        DQ_CHECK(merge_block(ctx, w2, U + p * pair_stride, d, s, s, batch, dd, 1));
      }
    }
    s *= 2; count = pairs;
  }
  // odd remainder: grow the leading inverse one block column at a time
  for (int kb = 1; kb < count; ++kb) {
    DQ_CHECK(merge_block(ctx, ws, U, d, kb * s, s, batch, dd, 1));
  }
  return DQ_OK;
}

// T = Phi(G - I - P), Phi(S) = striu(S) + diag(S) / 2 (P == nullptr: T = Phi(G - I)); see
// qr_forward_incremental_f32.  One launch covers all problems (blockIdx.y).
__global__ void __launch_bounds__(256) fixpoint_f32_kernel(const float* __restrict__ G, const float* __restrict__ P,
                                                           float* __restrict__ T, int d, const int* __restrict__ run_if,
                                                           int* __restrict__ moved_out, int fail_if_moved, float tol,
                                                           int* d_status) {
  if (run_if && *run_if == 0) return;
  const int64_t dd = (int64_t)d * d, off = (int64_t)blockIdx.y * dd;
  bool moved = false;
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < dd; e += (int64_t)gridDim.x * blockDim.x) {
    const int i = (int)(e / d), j = (int)(e % d);
    float v = 0.f;
    if (j >= i) {
      v = G[off + e] - ((i == j) ? 1.f : 0.f) - (P ? P[off + e] : 0.f);
      if (i == j) v *= 0.5f;
      if (P && !(fabsf(v - T[off + e]) <= tol)) moved = true;
    }
    T[off + e] = v;
  }
  if (moved) {
    if (moved_out) *moved_out = 1;
    if (fail_if_moved) set_status(d_status, DQ_ERR_NOT_CONVERGED);
  }
}

}  // namespace

dq_status qr_forward_incremental_f32(Ctx& ctx, QrWorkspace& ws, const float* Z, float* R, float* U, int d, int batch,
                                     int n_sweeps, int* flags) {
  const int64_t dd = (int64_t)d * d;
  float *Zh = ws.A, *G = ws.B, *T = ws.S, *P = ws.tmp, *Qs = ws.Q;
  GemmDesc g{};
  g.lda = d; g.ldb = d; g.ldc = d; g.sA = dd; g.sB = dd; g.sC = dd;
  g.M = d; g.N = d; g.K = d; g.alpha = 1.f; g.beta = 0.f; g.batch = batch;
  g.A = Z; g.transA = 0; g.B = ws.Winv; g.transB = 0; g.C = Zh;       // Zh = Z W_old
  DQ_CHECK(gemm_f32(ctx, g));
  g.A = Zh; g.transA = 1; g.B = Zh; g.transB = 0; g.C = G;            // G = Zh^T Zh
  DQ_CHECK(gemm_f32(ctx, g));
  int bx = (int)((dd + 255) / 256);
  if (bx > 1024) bx = 1024;
  const dim3 grid(bx, batch);
  const int total = n_sweeps + 3;
  DQ_CHECK_CUDA(cudaMemsetAsync(flags, 0, sizeof(int) * (total + 2), ctx.stream));
  fixpoint_f32_kernel<<<grid, 256, 0, ctx.stream>>>(G, nullptr, T, d, nullptr, nullptr, 0, 1e-5f, ctx.d_status);
  DQ_CHECK(after_launch(ctx));
  for (int it = 1; it <= total; ++it) {   // sweep it runs while sweep it - 1 moved an entry (flags[it - 1])
    const int* run_if = (it == 1) ? nullptr : flags + it - 1;
    g.A = T; g.transA = 1; g.B = T; g.transB = 0; g.C = P; g.run_if = run_if;   // P = T^T T
    DQ_CHECK(gemm_f32(ctx, g));
    fixpoint_f32_kernel<<<grid, 256, 0, ctx.stream>>>(G, P, T, d, run_if, flags + it, it == total ? 1 : 0, 1e-5f,
                                                      ctx.d_status);
    DQ_CHECK(after_launch(ctx));
  }
  g.run_if = nullptr;
  g.A = T; g.transA = 0; g.B = U; g.transB = 0; g.C = Qs;             // U = U_old + T U_old
  DQ_CHECK(gemm_f32(ctx, g));
  DQ_CHECK(accumulate(ctx, U, Qs, dd * batch));
  DQ_CHECK(qr_diag_check(ctx, U, d, batch));
  DQ_CHECK(tri_inverse(ctx, ws, U, d, batch));                        // uses ws.tmp as scratch
  g.A = Z; g.transA = 0; g.B = ws.Winv; g.transB = 0; g.C = R;        // R = Z W
  return gemm_f32(ctx, g);
}

dq_status qr_backward(Ctx& ctx, QrWorkspace& ws, const float* R, const float* U, const float* Gq,
                      float* Gz, int d, int batch, bool winv_fresh) {
  const int64_t dd = (int64_t)d * d;
  GemmDesc g{};
  g.A = R; g.lda = d; g.transA = 1; g.sA = dd;       // B = R^T Gq
  g.B = Gq; g.ldb = d; g.transB = 0; g.sB = dd;
  g.C = ws.B; g.ldc = d; g.sC = dd;
  g.M = d; g.N = d; g.K = d; g.alpha = 1.f; g.beta = 0.f; g.batch = batch;
  DQ_CHECK(gemm_f32(ctx, g));
  skew_lower_kernel<<<dim3(d / 32, d / 32, batch), 256, 0, ctx.stream>>>(ws.B, ws.S, d);
  DQ_CHECK(after_launch(ctx));
  g.A = R; g.transA = 0; g.B = ws.S; g.C = ws.B;     // M = R S
  DQ_CHECK(gemm_f32(ctx, g));
  if (!winv_fresh) DQ_CHECK(tri_inverse(ctx, ws, U, d, batch));
  g.A = ws.B; g.transA = 0; g.B = ws.Winv; g.transB = 1; g.C = Gz;   // Gz = M U^-T
  return gemm_f32(ctx, g);
}

}  // namespace dq
