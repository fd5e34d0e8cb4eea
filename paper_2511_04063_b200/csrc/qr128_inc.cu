// Batched QR-Orth for 128 x 128 latents, tensor-core variant of the shared-memory kernels: one CTA
// per problem, all matrices in shared memory, every 128^3 product as warp-level MMAs (3 x tf32,
// fp32-like accuracy) on 32 x 32 warp tiles.
//
//   qr128_forward_inc_kernel    incremental factorisation from the previous step's factors
//                               (U_old, W_old = U_old^-1): Zh = Z W_old, E = Zh^T Zh - I,
//                               T <- Phi(E - T^T T) (Phi(S) = striu(S) + diag(S) / 2) from T = 0 until no
//                               entry moves (at most 4 x the configured sweep count),
//                               U = (I + T) U_old, W = U^-1, R = Z W.  Same unique factors as the
//                               Householder kernel; no dependent column steps.
//   qr128_backward_sgd_tc_kernel B = R^T Gq, S = tril(B - B^T, -1), Gz = (R S) W^T, Z <- Z - lr Gz.
#include "common.cuh"
#include "mma_tf32.cuh"

namespace dq {
namespace {

constexpr int N = 128;
constexpr int LD = 132;          // row stride in shared memory: A-fragment loads hit 32 distinct banks
constexpr int NT = 512;          // 16 warps = 4 x 4 warp tiles of 32 x 32
constexpr int TMP_LD = 65;
constexpr int FWD_SMEM = (3 * N * LD + 64 * TMP_LD + 64) * 4;
constexpr int BWD_SMEM = 3 * N * LD * 4;

using mma::warp_mm32;
using mma::zero_acc;

// 128 x 128 fp32 matrix: global memory -> registers (eight coalesced 16-byte loads per thread) and
// registers -> shared memory (row stride LD; rows and LD are multiples of four floats).
__device__ __forceinline__ void g2r(const float* __restrict__ g, float4 (&v)[8], int tid) {
#pragma unroll
  for (int k = 0; k < 8; ++k) v[k] = reinterpret_cast<const float4*>(g)[tid + k * NT];
}
__device__ __forceinline__ void r2s(float* s, const float4 (&v)[8], int tid) {
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const int e = (tid + k * NT) * 4;
    *reinterpret_cast<float4*>(s + (e >> 7) * LD + (e & 127)) = v[k];
  }
}
// shared memory (row stride LD) -> global, 16 bytes per store
__device__ __forceinline__ void s2g(const float* s, float* __restrict__ g, int tid) {
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const int e = (tid + k * NT) * 4;
    reinterpret_cast<float4*>(g)[tid + k * NT] = *reinterpret_cast<const float4*>(s + (e >> 7) * LD + (e & 127));
  }
}
__device__ __forceinline__ void g2s(const float* __restrict__ g, float* s, int tid) {
  float4 v[8];
  g2r(g, v, tid);
  r2s(s, v, tid);
}

template <typename F>
__device__ __forceinline__ void acc_foreach(float (&acc)[2][4][4], int r0, int c0, int lane, F f) {
  const int g = lane >> 2, t = lane & 3;
#pragma unroll
  for (int mt = 0; mt < 2; ++mt)
#pragma unroll
    for (int nt = 0; nt < 4; ++nt)
#pragma unroll
      for (int e = 0; e < 4; ++e)
        f(r0 + 16 * mt + g + 8 * (e >> 1), c0 + 8 * nt + 2 * t + (e & 1), acc[mt][nt][e]);
}

// Dense C[M x Nc] = alpha A[M x K] B[K x Nc] on small shared-memory blocks, 4 x 4 register tiles.
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

__global__ void __launch_bounds__(NT, 1)
qr128_forward_inc_kernel(const float* __restrict__ Z, float* __restrict__ R, float* U, float* W,
                         __nv_bfloat16* __restrict__ Rt_bf16, int max_sweeps, float tol, int* d_status) {
  extern __shared__ float sm[];
  float* B0 = sm;
  float* B1 = B0 + N * LD;
  float* B2 = B1 + N * LD;
  float* Tmp = B2 + N * LD;          // [64][65]
  float* sc = Tmp + 64 * TMP_LD;     // scalars
  const int64_t off = (int64_t)blockIdx.x * N * N;
  Z += off; R += off; U += off; W += off;
  if (Rt_bf16) Rt_bf16 += off;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int wr = warp >> 2, wc = warp & 3, r0 = 32 * wr, c0 = 32 * wc;
  float acc[2][4][4];

  // ---- Zh = Z W_old (W_old upper triangular: k <= column)
  {
    float4 zv[8], wv[8];
    g2r(Z, zv, tid);
    g2r(W, wv, tid);
    r2s(B0, zv, tid);
    r2s(B1, wv, tid);
  }
  __syncthreads();
  zero_acc(acc);
  warp_mm32<false, false>(B0, B1, LD, acc, r0, c0, 0, 32 * (wc + 1), lane);
  acc_foreach(acc, r0, c0, lane, [&](int r, int c, float& v) { B2[r * LD + c] = v; });
  __syncthreads();
  // ---- E = Zh^T Zh - I on the tiles that touch the upper triangle (B0; Z is reloaded later)
  if (wr <= wc) {
    zero_acc(acc);
    warp_mm32<true, false>(B2, B2, LD, acc, r0, c0, 0, N, lane);
    acc_foreach(acc, r0, c0, lane, [&](int r, int c, float& v) { B0[r * LD + c] = v - ((r == c) ? 1.f : 0.f); });
  }
  __syncthreads();
  // ---- T = Phi(E) (first sweep: T = 0 before it)
  for (int e = tid; e < N * N; e += NT) {
    const int r = e >> 7, c = e & 127;
    const float v = B0[r * LD + c];
    B1[r * LD + c] = (c > r) ? v : ((c == r) ? 0.5f * v : 0.f);
  }
  __syncthreads();
  float* T = B1;
  float* Tn = B2;
  // The sweep count adapts to the data (everything lives in this CTA): sweeps continue until no entry of T
  // moves by more than tol, plus one more (the error left is then about rate / (1 - rate) times the last
  // movement, rate ~ 2 ||T||), up to max_sweeps.
  bool converged = false, extra = false;
  for (int it = 1; it < max_sweeps; ++it) {
    bool moved = false;
    if (wr <= wc) {   // P = T^T T: T[k][r] = 0 for k > r, so k < 32 (wr + 1)
      zero_acc(acc);
      warp_mm32<true, false>(T, T, LD, acc, r0, c0, 0, 32 * (wr + 1), lane);
      acc_foreach(acc, r0, c0, lane, [&](int r, int c, float& p) {
        float v = 0.f;
        if (c >= r) {
          v = B0[r * LD + c] - p;
          if (c == r) v *= 0.5f;
          if (!(fabsf(v - T[r * LD + c]) <= tol)) moved = true;
        }
        Tn[r * LD + c] = v;
      });
    } else {
      acc_foreach(acc, r0, c0, lane, [&](int r, int c, float&) { Tn[r * LD + c] = 0.f; });
    }
    const int any = __syncthreads_or(moved ? 1 : 0);
    float* s = T; T = Tn; Tn = s;
    if (!any) {
      if (extra) { converged = true; break; }
      extra = true;
    } else {
      extra = false;
    }
  }
  if (!converged && tid == 0) set_status(d_status, DQ_ERR_NOT_CONVERGED);
  // ---- U = (I + T) U_old: both upper triangular, k in [32 wr, 32 (wc + 1))
  if (tid < N) T[tid * LD + tid] += 1.f;
  g2s(U, B0, tid);
  __syncthreads();
  if (wr <= wc) {
    zero_acc(acc);
    warp_mm32<false, false>(T, B0, LD, acc, r0, c0, 32 * wr, 32 * (wc + 1), lane);
    acc_foreach(acc, r0, c0, lane, [&](int r, int c, float& v) { Tn[r * LD + c] = (c >= r) ? v : 0.f; });
  } else {
    acc_foreach(acc, r0, c0, lane, [&](int r, int c, float&) { Tn[r * LD + c] = 0.f; });
  }
  __syncthreads();
  float* Us = Tn;     // new U
  float* X = T;       // becomes W = U^-1
  // ---- rank / finiteness test of diag(U), U to global, X = 0
  if (warp < 4) {
    const int r = warp * 32 + lane;
    const float dv = Us[r * LD + r];
    float mn = dv, mx = dv;
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) {
      mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    }
    if (lane == 0) { sc[warp] = mn; sc[4 + warp] = mx; }
    if (!isfinite(dv)) set_status(d_status, DQ_ERR_NONFINITE);
  }
  s2g(Us, U, tid);
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const int e = (tid + k * NT) * 4;
    *reinterpret_cast<float4*>(X + (e >> 7) * LD + (e & 127)) = make_float4(0.f, 0.f, 0.f, 0.f);
  }
  __syncthreads();
  if (tid == 0) {
    const float mn = fminf(fminf(sc[0], sc[1]), fminf(sc[2], sc[3]));
    const float mx = fmaxf(fmaxf(sc[4], sc[5]), fmaxf(sc[6], sc[7]));
    if (!(mn > 1e-6f * mx)) set_status(d_status, DQ_ERR_SINGULAR);   // also catches a non-positive diagonal
  }
  // ---- W = U^-1: 32 x 32 diagonal blocks by back-substitution, then block merges
  if (warp < 4) {
    const int o = warp * 32, j = lane;
    X[(o + j) * LD + o + j] = 1.f / Us[(o + j) * LD + o + j];
    for (int i = j - 1; i >= 0; --i) {
      float s = 0.f;
      for (int k = i + 1; k <= j; ++k) s = fmaf(Us[(o + i) * LD + o + k], X[(o + k) * LD + o + j], s);
      X[(o + i) * LD + o + j] = -s / Us[(o + i) * LD + o + i];
    }
  }
  __syncthreads();
  for (int pair = 0; pair < 2; ++pair) {   // inv([A B; 0 C]) = [A^-1, -A^-1 B C^-1; 0, C^-1]
    const int o = pair * 64;
    smem_mm(Us + o * LD + o + 32, LD, X + (o + 32) * LD + o + 32, LD, Tmp, TMP_LD, 32, 32, 32, 1.f, tid);
    __syncthreads();
    smem_mm(X + o * LD + o, LD, Tmp, TMP_LD, X + o * LD + o + 32, LD, 32, 32, 32, -1.f, tid);
    __syncthreads();
  }
  smem_mm(Us + 64, LD, X + 64 * LD + 64, LD, Tmp, TMP_LD, 64, 64, 64, 1.f, tid);
  __syncthreads();
  smem_mm(X, LD, Tmp, TMP_LD, X + 64, LD, 64, 64, 64, -1.f, tid);
  // ---- R = Z W (Z reloaded into B0; U_old is no longer needed)
  g2s(Z, B0, tid);
  __syncthreads();
  zero_acc(acc);
  warp_mm32<false, false>(B0, X, LD, acc, r0, c0, 0, 32 * (wc + 1), lane);
  acc_foreach(acc, r0, c0, lane, [&](int r, int c, float& v) { Us[r * LD + c] = v; });   // U is in global memory by now
  __syncthreads();
  s2g(Us, R, tid);
  s2g(X, W, tid);
  if (Rt_bf16) {   // R^T in bf16: lane = row of R^T (consecutive columns of R in shared memory), 8 entries per store
    for (int idx = tid; idx < N * (N / 8); idx += NT) {
      const int c = idx & 127, rb = idx >> 7;
      uint32_t pk[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const __nv_bfloat162 h = __floats2bfloat162_rn(Us[(8 * rb + 2 * i) * LD + c], Us[(8 * rb + 2 * i + 1) * LD + c]);
        pk[i] = *reinterpret_cast<const uint32_t*>(&h);
      }
      *reinterpret_cast<uint4*>(Rt_bf16 + c * N + 8 * rb) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
    }
  }
}

__global__ void __launch_bounds__(NT, 1)
qr128_backward_sgd_tc_kernel(const float* __restrict__ R, const float* __restrict__ W, const float* __restrict__ Gq,
                             float* __restrict__ Gz, float* __restrict__ Z, float lr,
                             const int* __restrict__ d_status) {
  extern __shared__ float sm[];
  if (d_status && *d_status != 0) lr = 0.f;   // an earlier error freezes the latent
  float* P0 = sm;                    // R
  float* P1 = P0 + N * LD;           // Gq, then S, then W
  float* P2 = P1 + N * LD;           // B, then M = R S
  const int64_t off = (int64_t)blockIdx.x * N * N;
  R += off; W += off; Gq += off; Gz += off; Z += off;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int wr = warp >> 2, wc = warp & 3, r0 = 32 * wr, c0 = 32 * wc;
  float acc[2][4][4];
  float4 wv[8];                      // W is fetched now and parked in registers until its buffer is free
  {
    float4 rv[8], gv[8];
    g2r(R, rv, tid);
    g2r(Gq, gv, tid);
    g2r(W, wv, tid);
    r2s(P0, rv, tid);
    r2s(P1, gv, tid);
  }
  __syncthreads();
  zero_acc(acc);
  warp_mm32<true, false>(P0, P1, LD, acc, r0, c0, 0, N, lane);          // B = R^T Gq
  acc_foreach(acc, r0, c0, lane, [&](int r, int c, float& v) { P2[r * LD + c] = v; });
  __syncthreads();
  for (int e = tid; e < N * N; e += NT) {                               // S = tril(B - B^T, -1)
    const int i = e >> 7, j = e & 127;
    P1[i * LD + j] = (i > j) ? P2[i * LD + j] - P2[j * LD + i] : 0.f;
  }
  __syncthreads();
  zero_acc(acc);
  warp_mm32<false, false>(P0, P1, LD, acc, r0, c0, 32 * wc, N, lane);   // M = R S: S[k][c] = 0 for k <= c
  __syncthreads();                                                      // everyone is done reading B's buffer
  acc_foreach(acc, r0, c0, lane, [&](int r, int c, float& v) { P2[r * LD + c] = v; });
  r2s(P1, wv, tid);
  __syncthreads();
  zero_acc(acc);
  warp_mm32<false, true>(P2, P1, LD, acc, r0, c0, 32 * wc, N, lane);    // Gz = M W^T: W[c][k] = 0 for k < c
  acc_foreach(acc, r0, c0, lane, [&](int r, int c, float& v) {
    const int e = r * N + c;
    Gz[e] = v;
    if (lr != 0.f) Z[e] = fmaf(-lr, v, Z[e]);
  });
}

}  // namespace

dq_status qr128_forward_incremental(Ctx& ctx, const float* Z, float* R, float* U, float* W, __nv_bfloat16* Rt_bf16,
                                    int n_sweeps, int batch) {
  static SmemOptIn attr;
  DQ_CHECK(opt_in_dynamic_smem(qr128_forward_inc_kernel, FWD_SMEM, attr));
  qr128_forward_inc_kernel<<<batch, NT, FWD_SMEM, ctx.stream>>>(Z, R, U, W, Rt_bf16, 4 * (n_sweeps < 1 ? 1 : n_sweeps), 1e-5f,
                                                                ctx.d_status);
  return after_launch(ctx);
}

dq_status qr128_backward_sgd_tc(Ctx& ctx, const float* R, const float* W, const float* Gq, float* Gz, float* Z,
                                float lr, int batch) {
  static SmemOptIn attr;
  DQ_CHECK(opt_in_dynamic_smem(qr128_backward_sgd_tc_kernel, BWD_SMEM, attr));
  qr128_backward_sgd_tc_kernel<<<batch, NT, BWD_SMEM, ctx.stream>>>(R, W, Gq, Gz, Z, lr, ctx.d_status);
  return after_launch(ctx);
}

}  // namespace dq
