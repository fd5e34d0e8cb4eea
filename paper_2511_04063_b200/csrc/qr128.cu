// Batched QR-Orth for many independent 128 x 128 latents (per-head rotations): one CTA per
// problem, every matrix resident in shared memory.
//
//   qr128_forward_kernel       Z -> U (Householder, Algorithm 2, in place), gauge diag(U) > 0,
//                              W = U^-1 (blocked inversion), R = Z W; also bf16(R^T) for the
//                              tensor-core contraction.
// fp32 FMA arithmetic throughout; sums run in a fixed order (bit-reproducible).  Used for the first
// factorisation of a handle and with DQ_QR_HOUSEHOLDER; the incremental forward and the backward are
// in qr128_inc.cu.
#include "common.cuh"

namespace dq {
namespace {

constexpr int N = 128;
constexpr int LD = 129;          // padded leading dimension in shared memory
constexpr int NT = 512;

// C[128 x 128] = A op B on shared-memory matrices (leading dimension LD); each thread owns rows
// r0..r0+3 and the eight columns cl, cl + 16, ..., cl + 112 (a half-warp reads 16 consecutive
// words of B: no bank conflicts).  TA: use A^T.  TB: use B^T.
template <bool TA, bool TB>
__device__ __forceinline__ void mm128(const float* A, const float* B, float (&acc)[4][8], int r0, int cl) {
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;
#pragma unroll 2
  for (int k = 0; k < N; ++k) {
    float av[4], bv[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) av[i] = TA ? A[k * LD + r0 + i] : A[(r0 + i) * LD + k];
#pragma unroll
    for (int j = 0; j < 8; ++j) bv[j] = TB ? B[(cl + 16 * j) * LD + k] : B[k * LD + cl + 16 * j];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
  }
}

// Dense C[M x Nc] = alpha A[M x K] B[K x Nc] on shared-memory blocks, 4 x 4 register tiles.
__device__ __forceinline__ void smem_mm(const float* A, int lda, const float* B, int ldb, float* C, int ldc, int M,
                                        int Nc, int K, float alpha, int tid) {
  const int tn = Nc / 4, tiles = (M / 4) * tn;
  for (int t = tid; t < tiles; t += NT) {
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

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
  return v;
}

constexpr int FWD_SMEM = (3 * N * LD + 64 * 65 + N + 4 * N + 64) * 4;

// Reflector j: H = I - tau v v^T, v = (x - beta e1) / (x_1 - beta), beta = -sign(x_1) ||x||
// (Algorithm 2's sign rule).  Thread layout of the matvec / rank-1 update: column c = tid % 128,
// rows [32 q, 32 q + 32) with q = tid / 128.
__global__ void __launch_bounds__(NT, 1)
qr128_forward_kernel(const float* __restrict__ Z, float* __restrict__ R, float* __restrict__ U, float* __restrict__ W,
                     __nv_bfloat16* __restrict__ Rt_bf16, int* d_status) {
  extern __shared__ float sm[];
  float* A = sm;                     // Z, then U (upper) / reflectors (below)
  float* X = A + N * LD;             // U^-1
  float* Zs = X + N * LD;            // Z again (for R = Z W), then R
  float* Tmp = Zs + N * LD;          // [64][65]
  float* vs = Tmp + 64 * 65;         // [128] current reflector
  float* wpart = vs + N;             // [4][128] partial v^T A
  float* sc = wpart + 4 * N;         // scalars
  const int64_t off = (int64_t)blockIdx.x * N * N;
  Z += off; R += off; U += off; W += off;
  if (Rt_bf16) Rt_bf16 += off;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int c = tid & 127, q = tid >> 7;

  for (int e = tid; e < N * N; e += NT) {
    const float v = Z[e];
    A[(e >> 7) * LD + (e & 127)] = v;
    Zs[(e >> 7) * LD + (e & 127)] = v;
    X[(e >> 7) * LD + (e & 127)] = 0.f;
  }
  __syncthreads();

  // ---- Householder factorisation, one column per step, two barriers per step.
  // v_j is never materialised: v_r = x_r / (x_1 - beta) below the diagonal, 1 on it, so
  // v^T A[:, c] = A[j][c] + (sum_{r > j} x_r A[r][c]) / (x_1 - beta) and the dot products can
  // start before the scalars are known.  The squared norm of the next column is accumulated
  // by the threads that update it.
  float* rowj = vs;                  // [128] row j of A before the update
  float* nrmpart = sc;               // [4] partial squared norms of the current column
  if (c == 0) {
    float s = 0.f;
    for (int r = q * 32; r < q * 32 + 32; ++r) s = fmaf(A[r * LD], A[r * LD], s);
    nrmpart[q] = s;
  }
  __syncthreads();
  const int rlo = q * 32, rhi = rlo + 32;
  for (int j = 0; j < N - 1; ++j) {
    const float nrm2 = (nrmpart[0] + nrmpart[1]) + (nrmpart[2] + nrmpart[3]);
    const float alpha = A[j * LD + j];
    const int r_first = (rlo > j + 1) ? rlo : j + 1;   // rows strictly below the diagonal in this quarter
    float part = 0.f;
    if (c > j) {
      for (int r = r_first; r < rhi; ++r) part = fmaf(A[r * LD + j], A[r * LD + c], part);
      wpart[q * N + c] = part;
      if (j >= rlo && j < rhi) rowj[c] = A[j * LD + c];
    }
    const float sigma = nrm2 - alpha * alpha;
    const bool skip = !(sigma > 0.f);
    const float beta = skip ? alpha : -copysignf(sqrtf(nrm2), alpha);
    const float denom = alpha - beta;
    const float inv_denom = skip ? 0.f : 1.f / denom;
    const float tau = skip ? 0.f : -denom / beta;
    __syncthreads();
    if (c > j) {
      const float dot = (wpart[c] + wpart[N + c]) + (wpart[2 * N + c] + wpart[3 * N + c]);
      const float w = tau * fmaf(dot, inv_denom, rowj[c]);
      const float wv = w * inv_denom;
      float nn = 0.f;
      if (j >= rlo && j < rhi) A[j * LD + c] -= w;                 // diagonal row: v = 1 (not part of the next norm)
      for (int r = r_first; r < rhi; ++r) {
        const float t = fmaf(-A[r * LD + j], wv, A[r * LD + c]);
        A[r * LD + c] = t;
        nn = fmaf(t, t, nn);
      }
      if (c == j + 1) nrmpart[q] = nn;
    }
    if (tid == 0) A[j * LD + j] = beta;
    __syncthreads();
  }

  // ---- gauge diag(U) > 0 and rank test; U' = diag(s) triu(A)
  if (warp < 4) {
    const int r = warp * 32 + lane;
    const float dv = fabsf(A[r * LD + r]);
    float mn = dv, mx = dv;
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) {
      mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    }
    if (lane == 0) { sc[8 + warp] = mn; sc[12 + warp] = mx; }
    if (!isfinite(dv)) set_status(d_status, DQ_ERR_NONFINITE);
  }
  if (tid < N) vs[tid] = (A[tid * LD + tid] < 0.f) ? -1.f : 1.f;
  __syncthreads();
  if (tid == 0) {
    const float mn = fminf(fminf(sc[8], sc[9]), fminf(sc[10], sc[11]));
    const float mx = fmaxf(fmaxf(sc[12], sc[13]), fmaxf(sc[14], sc[15]));
    if (!(mn > 1e-6f * mx)) set_status(d_status, DQ_ERR_SINGULAR);
  }
  for (int e = tid; e < N * N; e += NT) {
    const int r = e >> 7, cc = e & 127;
    const float v = (cc >= r) ? vs[r] * A[r * LD + cc] : 0.f;
    A[r * LD + cc] = v;
    U[e] = v;
  }
  __syncthreads();

  // ---- W = U'^-1: 32 x 32 diagonal blocks by back-substitution, then block merges
  if (warp < 4) {
    const int o = warp * 32, j = lane;
    X[(o + j) * LD + o + j] = 1.f / A[(o + j) * LD + o + j];
    for (int i = j - 1; i >= 0; --i) {
      float s = 0.f;
      for (int k = i + 1; k <= j; ++k) s = fmaf(A[(o + i) * LD + o + k], X[(o + k) * LD + o + j], s);
      X[(o + i) * LD + o + j] = -s / A[(o + i) * LD + o + i];
    }
  }
  __syncthreads();
  for (int pair = 0; pair < 2; ++pair) {   // inv([A B; 0 C]) = [A^-1, -A^-1 B C^-1; 0, C^-1]
    const int o = pair * 64;
    smem_mm(A + o * LD + o + 32, LD, X + (o + 32) * LD + o + 32, LD, Tmp, 65, 32, 32, 32, 1.f, tid);
    __syncthreads();
    smem_mm(X + o * LD + o, LD, Tmp, 65, X + o * LD + o + 32, LD, 32, 32, 32, -1.f, tid);
    __syncthreads();
  }
  smem_mm(A + 64, LD, X + 64 * LD + 64, LD, Tmp, 65, 64, 64, 64, 1.f, tid);
  __syncthreads();
  smem_mm(X, LD, Tmp, 65, X + 64, LD, 64, 64, 64, -1.f, tid);
  __syncthreads();

  // ---- R = Z W; 4 x 8 outputs per thread
  {
    const int r0 = (tid >> 4) * 4, cl = tid & 15;
    float acc[4][8];
    mm128<false, false>(Zs, X, acc, r0, cl);
    __syncthreads();                 // everyone is done reading Zs
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 8; ++j) Zs[(r0 + i) * LD + cl + 16 * j] = acc[i][j];
  }
  __syncthreads();
  for (int e = tid; e < N * N; e += NT) {
    const int r = e >> 7, cc = e & 127;
    R[e] = Zs[r * LD + cc];
    W[e] = X[r * LD + cc];
    if (Rt_bf16) Rt_bf16[e] = __float2bfloat16_rn(Zs[cc * LD + r]);   // R^T
  }
}

}  // namespace

dq_status qr128_forward(Ctx& ctx, const float* Z, float* R, float* U, float* W, __nv_bfloat16* Rt_bf16, int batch) {
  static SmemOptIn attr;
  DQ_CHECK(opt_in_dynamic_smem(qr128_forward_kernel, FWD_SMEM, attr));
  qr128_forward_kernel<<<batch, NT, FWD_SMEM, ctx.stream>>>(Z, R, U, W, Rt_bf16, ctx.d_status);
  return after_launch(ctx);
}

}  // namespace dq
