// Shared declarations of the library's translation units (host side + small
// device helpers).  Nothing here is part of the public ABI.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "dartquant.h"

namespace dq {

// Per-handle launch context.  d_status is a device int (0 = ok) that kernels set
// with atomicCAS(0 -> code) so the first problem wins.
struct Ctx {
  cudaStream_t stream = nullptr;
  int* d_status = nullptr;
  int64_t launches = 0;
  double mma_flops = 0.0;   // bf16 tensor-core flops issued by the tcgen05 kernels (counted on the host)
  int sm_count = 148;
  // Optional side branch: small checks and reductions that nothing on the main stream waits for run beside
  // the next large kernel (on_side) and are ordered back in before their results are needed (join_side).
  cudaStream_t side = nullptr;
  cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
  bool side_pending = false;
};

#define DQ_CHECK_CUDA(expr)                          \
  do {                                               \
    cudaError_t _e = (expr);                         \
    if (_e != cudaSuccess) return DQ_ERR_CUDA;       \
  } while (0)

#define DQ_CHECK(expr)                 \
  do {                                 \
    dq_status _s = (expr);             \
    if (_s != DQ_OK) return _s;        \
  } while (0)

inline dq_status after_launch(Ctx& ctx) {
  ctx.launches++;
  return cudaGetLastError() == cudaSuccess ? DQ_OK : DQ_ERR_CUDA;
}

// Runs launch(ctx) with ctx.stream replaced by the side stream, ordered after everything enqueued on the main
// stream so far.  Without a side stream the work stays on the main stream.
template <typename F>
inline dq_status on_side(Ctx& ctx, F launch) {
  if (!ctx.side) return launch(ctx);
  if (cudaEventRecord(ctx.ev_fork, ctx.stream) != cudaSuccess || cudaStreamWaitEvent(ctx.side, ctx.ev_fork, 0) != cudaSuccess)
    return DQ_ERR_CUDA;
  cudaStream_t main_stream = ctx.stream;
  ctx.stream = ctx.side;
  const dq_status st = launch(ctx);
  ctx.stream = main_stream;
  ctx.side_pending = true;
  return st;
}
// Orders the main stream after the side work enqueued so far.
inline dq_status join_side(Ctx& ctx) {
  if (!ctx.side_pending) return DQ_OK;
  ctx.side_pending = false;
  if (cudaEventRecord(ctx.ev_join, ctx.side) != cudaSuccess || cudaStreamWaitEvent(ctx.stream, ctx.ev_join, 0) != cudaSuccess)
    return DQ_ERR_CUDA;
  return DQ_OK;
}

// Opt-in to more than 48 KB of dynamic shared memory.  The attribute belongs to the (function, device) pair,
// so it is set once per device; one process may use the library on several devices.
struct SmemOptIn { bool done[64] = {}; };
template <typename Kernel>
inline dq_status opt_in_dynamic_smem(Kernel kern, int bytes, SmemOptIn& table) {
  int dev = -1;
  DQ_CHECK_CUDA(cudaGetDevice(&dev));
  const bool tracked = dev >= 0 && dev < 64;
  if (tracked && table.done[dev]) return DQ_OK;
  DQ_CHECK_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
  if (tracked) table.done[dev] = true;
  return DQ_OK;
}

__device__ __forceinline__ void set_status(int* d_status, int code) {
  if (d_status) atomicCAS(d_status, 0, code);
}

// v as a (hi, lo) pair of bf16 with hi + lo = v to about 2^-17 relative ("split bf16")
__device__ __forceinline__ void split2(float v, __nv_bfloat16& hi, __nv_bfloat16& lo) {
  hi = __float2bfloat16_rn(v);
  lo = __float2bfloat16_rn(v - __bfloat162float(hi));
}

// Sum v[c] over the 32 lanes; lane c returns the total of column c.
__device__ __forceinline__ float warp_transpose_reduce32(float (&v)[32], int lane) {
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) {
    const bool up = (lane & off) != 0;
#pragma unroll
    for (int k = 0; k < off; ++k) {
      const float send = up ? v[k] : v[k + off];
      const float keep = up ? v[k + off] : v[k];
      v[k] = keep + __shfl_xor_sync(0xffffffffu, send, off);
    }
  }
  return v[0];
}

// ---------------------------------------------------------------------------
// fp32 FMA GEMM (gemm_ffma.cu):  C = alpha op(A) op(B) + beta C, batched/strided.
// op(A) is M x K, op(B) is K x N; trans* = 1 means the stored matrix is the
// transpose (stored K x M / N x K).  Any sizes.
// ---------------------------------------------------------------------------
struct GemmDesc {
  const float* A; int64_t lda; int transA;
  const float* B; int64_t ldb; int transB;
  float* C; int64_t ldc;
  int M, N, K;
  float alpha, beta;
  int batch; int64_t sA, sB, sC;
  // Split-K: with ksplit > 1 slice ks of the reduction writes alpha * partial
  // product (beta ignored) to C + (b * ksplit + ks) * sC; the caller reduces.
  int ksplit = 1;
  // Optional device flag: the kernel does nothing when *run_if == 0.
  const int* run_if = nullptr;
};
dq_status gemm_f32(Ctx& ctx, const GemmDesc& g);
// out[b][i] = alpha * sum_ks part[(b * ksplit + ks)][i] + beta * out[b][i], fixed order.
dq_status splitk_reduce(Ctx& ctx, const float* part, int ksplit, int64_t n_per_batch, int batch,
                        float alpha, float beta, float* out);

// O = X R with the Whip epilogue (Eq. 4) in fp32: writes G = -sign(O) exp(-|O|)
// (token-major [batch][N][d], no 1/N) and one loss partial per 64x64 tile.
// partials layout: [batch][tiles]; returns tiles per problem in *tiles_per_problem.
dq_status whip_forward_f32(Ctx& ctx, const float* X, int64_t ldx, int64_t strideX, const float* R,
                           float* G, float* partials, int64_t n_tokens, int d, int batch,
                           int* tiles_per_problem);
int whip_forward_f32_tiles(int64_t n_tokens, int d);

// Sums partials[b][0..n) in a fixed order in fp64, scales, stores fp32 loss[b].
// Sets DQ_ERR_NONFINITE in the status word if a loss is not finite.
dq_status loss_finalize(Ctx& ctx, const float* partials, int n_per_problem, int batch, float scale,
                        float* loss_out /* nullable */, float* loss_last);

// ---------------------------------------------------------------------------
// QR-Orth (qr_forward.cu / qr_backward.cu), fp32 matrices [batch][d][d].
// ---------------------------------------------------------------------------
struct QrWorkspace {
  float* A = nullptr;     // working copy of Z, ends as the raw upper factor
  float* V = nullptr;     // Householder vectors (unit lower trapezoid per panel)
  float* T = nullptr;     // [batch][d/32][32][32] compact-WY T factors
  float* W = nullptr;     // [batch][32][d] scratch
  float* W2 = nullptr;    // [batch][32][d] scratch
  float* Q = nullptr;     // accumulated orthogonal factor (raw gauge)
  float* Winv = nullptr;  // U^-1
  float* B = nullptr;     // R^T Gq, then R S
  float* S = nullptr;     // tril(B - B^T, -1)
  float* tmp = nullptr;   // [batch][d][d] scratch for the triangular inverse
};
// Factorisation only: ws.A <- raw upper factor, ws.V / ws.T <- reflectors.
dq_status qr_factor(Ctx& ctx, QrWorkspace& ws, const float* Z, int d, int batch);
// Z -> R (rotation, diag(U) > 0), U.  Optionally also a bf16 copy of R^T.
dq_status qr_forward(Ctx& ctx, QrWorkspace& ws, const float* Z, float* R, float* U,
                     __nv_bfloat16* Rt_bf16 /* nullable */, int d, int batch);
// Rank / finiteness test of diag(U) (qr_forward.cu); works on either orientation.
dq_status qr_diag_check(Ctx& ctx, const float* A, int d, int batch);
// Gz = R tril(R^T Gq - Gq^T R, -1) U^-T.  winv_fresh: ws.Winv already holds U^-1.
dq_status qr_backward(Ctx& ctx, QrWorkspace& ws, const float* R, const float* U, const float* Gq,
                      float* Gz, int d, int batch, bool winv_fresh);
// Incremental factorisation in fp32 from the previous factors (U holds U_old, ws.Winv its inverse; both are
// replaced): Zh = Z W_old, E = Zh^T Zh - I, T <- Phi(E - T^T T) until nothing moves (device flags, at most
// n_sweeps + 3 sweeps), U = (I + T) U_old, W = U^-1, R = Z W.  flags: device int[n_sweeps + 5].
dq_status qr_forward_incremental_f32(Ctx& ctx, QrWorkspace& ws, const float* Z, float* R, float* U, int d, int batch,
                                     int n_sweeps, int* flags);

// Batched 128 x 128 QR-Orth resident in shared memory (qr128.cu), one CTA per problem.
// Forward (Householder): R, U (diag > 0), W = U^-1, optional bf16(R^T).
dq_status qr128_forward(Ctx& ctx, const float* Z, float* R, float* U, float* W, __nv_bfloat16* Rt_bf16, int batch);

// Tensor-core kernels (qr128_inc.cu): incremental forward from the previous step's U and W (both updated
// in place); backward Gz = R tril(R^T Gq - Gq^T R, -1) W^T with the SGD update of Z fused (lr = 0: none).
dq_status qr128_forward_incremental(Ctx& ctx, const float* Z, float* R, float* U, float* W, __nv_bfloat16* Rt_bf16,
                                    int n_sweeps, int batch);
dq_status qr128_backward_sgd_tc(Ctx& ctx, const float* R, const float* W, const float* Gq, float* Gz, float* Z,
                                float lr, int batch);

// tcgen05 kernel (qr128_tc5.cu): backward + SGD (do_backward; lr = 0: no update) and / or the incremental forward
// from W = U^-1 alone (do_forward; W and P = the last sweep's T^T T are updated in place, R and bf16(R^T)
// written to R_out, or to R if that is null).  The fp32 intermediates stay in tensor memory.
dq_status qr128_step_tc5(Ctx& ctx, float* Z, float* W, float* P, float* R, float* R_out, __nv_bfloat16* Rt, const float* Gq,
                         float* Gz, float lr, bool do_backward, bool do_forward, int max_sweeps, int batch);

// out[i] = X[pi_seed(first + i)] for i < count: seeded sampling of token rows without replacement
// (token_sampling.cu).  elem_bytes = 2 (bf16) or 4 (fp32); rows must be multiples of 16 bytes.
dq_status gather_tokens(Ctx& ctx, const void* X, int elem_bytes, int64_t n, int d, int64_t ldx, uint64_t seed,
                        int64_t first, int64_t count, void* out, int64_t ldo);

// dst += src (n elements)
dq_status accumulate(Ctx& ctx, float* dst, const float* src, int64_t n);
// Z <- Z - lr Gz  (n elements); z_hi / z_lo (nullable): also the split-bf16 copy of the new Z
dq_status sgd_update(Ctx& ctx, float* Z, const float* Gz, float lr, int64_t n, __nv_bfloat16* z_hi = nullptr,
                     __nv_bfloat16* z_lo = nullptr);
// v <- mu v + Gz; Z <- Z - lr v
dq_status momentum_update(Ctx& ctx, float* Z, const float* Gz, float* V, float lr, float mu, int64_t n);
// Adam with bias correction; pw = device float[2] {beta1^t, beta2^t}, advanced on the device
dq_status adam_update(Ctx& ctx, float* Z, const float* Gz, float* M, float* V, float* pw, float lr, float b1,
                      float b2, float eps, int64_t n);

}  // namespace dq
