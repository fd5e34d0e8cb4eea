// Cayley SGD with momentum (Algorithm 3) on the rotation itself: the orthogonal optimiser the
// paper compares QR-Orth with.  Per iteration six d x d products, all issued as split-bf16
// tcgen05 GEMMs (three bf16 MMAs per product, fp32 accumulation), and a handful of fused
// element-wise kernels that also write the operand copies of the next product:
//   M1   = beta M - G                                  (momentum folds in the gradient)
//   T1^T = X M1^T,  T2^T = T1^T X,  T3 = X T2          (What = T1 - T3 / 2)
//   W    = What - What^T                               (skew-symmetric), |W|_F
//   M    = W X                                         (momentum projected to the tangent space)
//   a    = min(l, 2 q / (|W|_F + eps))
//   Y^0  = X + a M;  Y^i = X + a/2 W (X + Y^(i-1)), i = 1..s;  X <- Y^s
// X is the rotation R (d x d, fp32, row-major); the new R is written with the row-major and
// transposed split copies that the next step's products and the Whip contraction read.
#include "tc_host.cuh"
#include "tc_path.cuh"

namespace dq {
namespace {

using bf16 = __nv_bfloat16;
using tch::Op;
using tch::Out;
using tch::gemm3;

// v = ca A + cb s B with s = alpha[b] (use_alpha) or 1; optional outputs: fp32 (may alias A),
// split copy of v row-major, split copy of v^T.  n x n matrices, 32 x 32 tile per block.
__global__ void __launch_bounds__(256) combine_split_kernel(const float* A, const float* __restrict__ B, float ca,
                                                            float cb, const float* __restrict__ alpha, int use_alpha,
                                                            float* out, bf16* __restrict__ hi, bf16* __restrict__ lo,
                                                            bf16* __restrict__ thi, bf16* __restrict__ tlo, int n,
                                                            const int* __restrict__ d_status) {
  __shared__ float t[32][33];
  if (d_status && *d_status != 0) return;   // commit nothing once the status word holds an error
  const int64_t off = (int64_t)blockIdx.z * n * n;
  const float s = use_alpha ? alpha[blockIdx.z] : 1.f;
  const float cbs = cb * s;
  const int r0 = blockIdx.y * 32, c0 = blockIdx.x * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  for (int r = ty; r < 32; r += 8) {
    const int64_t i = off + (int64_t)(r0 + r) * n + c0 + tx;
    const float v = ca * A[i] + cbs * B[i];
    if (out) out[i] = v;
    if (hi) split2(v, hi[i], lo[i]);
    t[r][tx] = v;
  }
  if (!thi) return;
  __syncthreads();
  for (int c = ty; c < 32; c += 8) {
    const int64_t i = off + (int64_t)(c0 + c) * n + r0 + tx;
    split2(t[tx][c], thi[i], tlo[i]);
  }
}

// W = What - What^T with What = T1 - T3 / 2, given T1t = T1^T and T3:
//   W[i][j] = (T1t[j][i] - T1t[i][j]) - (T3[i][j] - T3[j][i]) / 2.
// Writes the split copy of W and one partial of sum W^2 per block (fixed order within the block).
__global__ void __launch_bounds__(256) skew_w_kernel(const float* __restrict__ T1t, const float* __restrict__ T3,
                                                     bf16* __restrict__ hi, bf16* __restrict__ lo,
                                                     float* __restrict__ part, int n) {
  __shared__ float a[32][33], b[32][33];
  __shared__ float red[8];
  const int64_t off = (int64_t)blockIdx.z * n * n;
  const int r0 = blockIdx.y * 32, c0 = blockIdx.x * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  for (int r = ty; r < 32; r += 8) {   // mirrored tile (rows c0.., columns r0..)
    const int64_t i = off + (int64_t)(c0 + r) * n + r0 + tx;
    a[r][tx] = T1t[i];
    b[r][tx] = T3[i];
  }
  __syncthreads();
  float acc = 0.f;
  for (int r = ty; r < 32; r += 8) {
    const int64_t i = off + (int64_t)(r0 + r) * n + c0 + tx;
    const float w = (a[tx][r] - T1t[i]) - 0.5f * (T3[i] - b[tx][r]);
    split2(w, hi[i], lo[i]);
    acc = fmaf(w, w, acc);
  }
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if (tx == 0) red[ty] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    float sblk = 0.f;
    for (int k = 0; k < 8; ++k) sblk += red[k];
    part[((int64_t)blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x] = sblk;
  }
}

// alpha[b] = min(lr, 2 q / (|W|_F + eps)); partials summed in a fixed order in fp64.
__global__ void __launch_bounds__(256) cayley_alpha_kernel(const float* __restrict__ part, int n_part, float lr,
                                                           float two_q, float eps, float* __restrict__ alpha,
                                                           int* d_status) {
  __shared__ double red[256];
  const float* p = part + (int64_t)blockIdx.x * n_part;
  double s = 0.0;
  for (int i = threadIdx.x; i < n_part; i += 256) s += (double)p[i];
  red[threadIdx.x] = s;
  __syncthreads();
  for (int o = 128; o > 0; o >>= 1) {
    if ((int)threadIdx.x < o) red[threadIdx.x] += red[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const double nrm = sqrt(red[0]);
    if (!(nrm == nrm) || nrm > 3.0e38) set_status(d_status, DQ_ERR_NONFINITE);
    const double clip = (double)two_q / (nrm + (double)eps);
    alpha[blockIdx.x] = (float)((double)lr < clip ? (double)lr : clip);
  }
}

}  // namespace

dq_status cayley_init(CayleyState& cs, int d, int batch) {
  const int64_t dd = (int64_t)d * d * batch;
  cs.n_part = (d / 32) * (d / 32);
  if (cudaMalloc((void**)&cs.M, sizeof(float) * dd) != cudaSuccess) return DQ_ERR_ALLOC;
  if (cudaMalloc((void**)&cs.part, sizeof(float) * (size_t)cs.n_part * batch) != cudaSuccess) return DQ_ERR_ALLOC;
  if (cudaMalloc((void**)&cs.alpha, sizeof(float) * batch) != cudaSuccess) return DQ_ERR_ALLOC;
  cs.ready = true;
  return DQ_OK;
}

void cayley_destroy(CayleyState& cs) {
  cudaFree(cs.M); cudaFree(cs.part); cudaFree(cs.alpha);
  cs = CayleyState{};
}

dq_status cayley_step_tc(Ctx& ctx, QrWorkspace& ws, QrTcState& q, CayleyState& cs, float* R, const float* Gq,
                         float lr, int d, int batch) {
  if (!cs.ready || !q.ready) return DQ_ERR_INVALID_ARG;
  const int64_t dd = (int64_t)d * d;
  const dim3 tiles(d / 32, d / 32, batch);
  const Op r{q.r_hi, q.r_lo, d, dd}, rt{q.rt_hi, q.rt_lo, d, dd};
  // M1 = beta M - G: only its split copy is needed (B operand of T1^T = X M1^T)
  combine_split_kernel<<<tiles, 256, 0, ctx.stream>>>(cs.M, Gq, cs.beta, -1.f, nullptr, 0, nullptr, q.gqt_hi, q.gqt_lo,
                                                      nullptr, nullptr, d, nullptr);
  DQ_CHECK(after_launch(ctx));
  // T1^T[m][n] = sum_k X[m][k] M1[n][k]
  {
    const Op m1{q.gqt_hi, q.gqt_lo, d, dd};
    Out o; o.f32 = ws.B; o.ld = d; o.bs = dd; o.hi = q.st_hi; o.lo = q.st_lo; o.ld_h = d; o.bs_h = dd;
    DQ_CHECK(gemm3(ctx, r, m1, d, d, d, batch, o));
  }
  // T2^T[m][n] = sum_k T1^T[m][k] X[k][n]
  {
    const Op t1t{q.st_hi, q.st_lo, d, dd};
    Out o; o.hi = q.m_hi; o.lo = q.m_lo; o.ld_h = d; o.bs_h = dd;
    DQ_CHECK(gemm3(ctx, t1t, rt, d, d, d, batch, o));
  }
  // T3[m][n] = sum_k X[m][k] T2[k][n]
  {
    const Op t2t{q.m_hi, q.m_lo, d, dd};
    Out o; o.f32 = ws.S; o.ld = d; o.bs = dd;
    DQ_CHECK(gemm3(ctx, r, t2t, d, d, d, batch, o));
  }
  skew_w_kernel<<<tiles, 256, 0, ctx.stream>>>(ws.B, ws.S, q.wn_hi, q.wn_lo, cs.part, d);
  DQ_CHECK(after_launch(ctx));
  cayley_alpha_kernel<<<batch, 256, 0, ctx.stream>>>(cs.part, cs.n_part, lr, 2.f * cs.q, cs.eps, cs.alpha,
                                                     ctx.d_status);
  DQ_CHECK(after_launch(ctx));
  const Op w{q.wn_hi, q.wn_lo, d, dd};
  // M[m][n] = sum_k W[m][k] X[k][n]
  {
    Out o; o.f32 = cs.M; o.ld = d; o.bs = dd;
    DQ_CHECK(gemm3(ctx, w, rt, d, d, d, batch, o));
  }
  // X + Y^0 = 2 X + a M, transposed split copy (B operand of W (X + Y))
  combine_split_kernel<<<tiles, 256, 0, ctx.stream>>>(R, cs.M, 2.f, 1.f, cs.alpha, 1, nullptr, nullptr, nullptr,
                                                      q.z_hi, q.z_lo, d, nullptr);
  DQ_CHECK(after_launch(ctx));
  const Op st{q.z_hi, q.z_lo, d, dd};
  for (int i = 1; i <= cs.s; ++i) {
    Out o; o.f32 = ws.tmp; o.ld = d; o.bs = dd;
    DQ_CHECK(gemm3(ctx, w, st, d, d, d, batch, o));   // P = W (X + Y^(i-1))
    if (i < cs.s) {   // X + Y^i = 2 X + a/2 P
      combine_split_kernel<<<tiles, 256, 0, ctx.stream>>>(R, ws.tmp, 2.f, 0.5f, cs.alpha, 1, nullptr, nullptr, nullptr,
                                                          q.z_hi, q.z_lo, d, nullptr);
    } else {          // X <- Y^s = X + a/2 P, with both operand copies of the new rotation
      combine_split_kernel<<<tiles, 256, 0, ctx.stream>>>(R, ws.tmp, 1.f, 0.5f, cs.alpha, 1, R, q.r_hi, q.r_lo,
                                                          q.rt_hi, q.rt_lo, d, ctx.d_status);
    }
    DQ_CHECK(after_launch(ctx));
  }
  return DQ_OK;
}

}  // namespace dq
