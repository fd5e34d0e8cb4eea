// Evaluation of a rotation on activations (Sec. 4.1, Eq. 1 and the appendix on outliers and
// quantisation errors): number of outliers |o| > tau of O = X R and the error of per-token
// asymmetric uniform quantisation of O.  O is produced chunk by chunk (tensor cores for bf16
// activations, fp32 FMA otherwise) and reduced per token by one warp; sums run in a fixed order.
#include "tc_host.cuh"
#include "tc_path.cuh"

namespace dq {
namespace {

__device__ __forceinline__ float warp_min(float v) {
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) v = fminf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// Per token row of O [rows][d]: outlier count and sum of squared quantisation errors.
//   scale = (max - min) / maxq, zero = rint(-min / scale), q = clamp(rint(o / scale) + zero, 0, maxq),
//   dequantised = scale (q - zero); a constant row has no error.
__global__ void __launch_bounds__(256) token_metrics_kernel(const float* __restrict__ O, int64_t rows, int d, float tau,
                                                            float maxq, double* __restrict__ sq_err,
                                                            int* __restrict__ n_out) {
  const int lane = threadIdx.x & 31;
  const int64_t t = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (t >= rows) return;
  const float* o = O + t * d;
  float lo = INFINITY, hi = -INFINITY;
  for (int j = lane; j < d; j += 32) { const float v = o[j]; lo = fminf(lo, v); hi = fmaxf(hi, v); }
  lo = warp_min(lo); hi = warp_max(hi);
  const float range = hi - lo;
  const float scale = (range > 0.f) ? range / maxq : 1.f;
  const float zero = rintf(-lo / scale);
  double e = 0.0;
  int cnt = 0;
  for (int j = lane; j < d; j += 32) {
    const float v = o[j];
    cnt += (fabsf(v) > tau) ? 1 : 0;
    if (range > 0.f) {
      const float q = fminf(fmaxf(rintf(v / scale) + zero, 0.f), maxq);
      const float diff = scale * (q - zero) - v;
      e += (double)diff * (double)diff;
    }
  }
#pragma unroll
  for (int off = 16; off >= 1; off >>= 1) {
    e += __shfl_xor_sync(0xffffffffu, e, off);
    cnt += __shfl_xor_sync(0xffffffffu, cnt, off);
  }
  if (lane == 0) { sq_err[t] = e; n_out[t] = cnt; }
}

// out[0] += sum of n_out, out[1] += sum of sq_err, in a fixed order (one CTA).
__global__ void __launch_bounds__(256) metrics_reduce_kernel(const double* __restrict__ sq_err,
                                                             const int* __restrict__ n_out, int64_t rows,
                                                             double* __restrict__ out) {
  __shared__ double se[256], sc[256];
  double e = 0.0, c = 0.0;
  for (int64_t i = threadIdx.x; i < rows; i += 256) { e += sq_err[i]; c += (double)n_out[i]; }
  se[threadIdx.x] = e; sc[threadIdx.x] = c;
  __syncthreads();
  for (int off = 128; off >= 1; off >>= 1) {
    if ((int)threadIdx.x < off) { se[threadIdx.x] += se[threadIdx.x + off]; sc[threadIdx.x] += sc[threadIdx.x + off]; }
    __syncthreads();
  }
  if (threadIdx.x == 0) { out[0] += sc[0]; out[1] += se[0]; }
}

__global__ void transpose_r_to_bf16_kernel(const float* __restrict__ in, __nv_bfloat16* __restrict__ out, int d) {
  __shared__ float t[32][33];
  const int r0 = blockIdx.y * 32, c0 = blockIdx.x * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  for (int r = ty; r < 32; r += 8) t[r][tx] = in[(int64_t)(r0 + r) * d + c0 + tx];
  __syncthreads();
  for (int c = ty; c < 32; c += 8) out[(int64_t)(c0 + c) * d + r0 + tx] = __float2bfloat16_rn(t[tx][c]);
}

__global__ void finish_metrics_kernel(double* out, double n_entries) { out[1] /= n_entries; }

}  // namespace

// d_out: device double[2] = { number of outliers, mean squared quantisation error }.
dq_status eval_rotation(Ctx& ctx, const void* d_X, int x_dtype, int64_t n, int d, int64_t ldx, const float* d_R,
                        float tau, int bits, double* d_out) {
  if (bits < 1 || bits > 16 || !(tau >= 0.f)) return DQ_ERR_INVALID_ARG;
  const bool tcp = x_dtype == DQ_BF16;
  if (tcp && (d % 128 != 0 || n % 128 != 0 || ldx % 8 != 0)) return DQ_ERR_UNSUPPORTED;
  int sms = 0, dev = 0;
  DQ_CHECK_CUDA(cudaGetDevice(&dev));
  DQ_CHECK_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  ctx.sm_count = sms;
  tch::keep_pool_memory(dev);
  int64_t chunk = (int64_t)(((int64_t)1 << 25) / d);            // 128 MiB of fp32 outputs at a time
  chunk = (chunk / 128) * 128;
  if (chunk < 128) chunk = 128;
  if (chunk > n) chunk = n;
  float* O = nullptr; double* sq = nullptr; int* cnt = nullptr; __nv_bfloat16* rt = nullptr;
  dq_status st = DQ_OK;
  if (cudaMallocAsync((void**)&O, sizeof(float) * (size_t)chunk * d, ctx.stream) != cudaSuccess ||
      cudaMallocAsync((void**)&sq, sizeof(double) * (size_t)chunk, ctx.stream) != cudaSuccess ||
      cudaMallocAsync((void**)&cnt, sizeof(int) * (size_t)chunk, ctx.stream) != cudaSuccess ||
      (tcp && cudaMallocAsync((void**)&rt, sizeof(__nv_bfloat16) * (size_t)d * d, ctx.stream) != cudaSuccess))
    st = DQ_ERR_ALLOC;
  if (st == DQ_OK && cudaMemsetAsync(d_out, 0, 2 * sizeof(double), ctx.stream) != cudaSuccess) st = DQ_ERR_CUDA;
  if (st == DQ_OK && tcp) {
    transpose_r_to_bf16_kernel<<<dim3(d / 32, d / 32), 256, 0, ctx.stream>>>(d_R, rt, d);
    st = after_launch(ctx);
  }
  const float maxq = (float)((1 << bits) - 1);
  for (int64_t r0 = 0; r0 < n && st == DQ_OK; r0 += chunk) {
    const int64_t rows = (n - r0 < chunk) ? n - r0 : chunk;
    if (tcp) {   // O[token][channel] = sum_k X[token][k] R^T[channel][k]
      const __nv_bfloat16* xc = reinterpret_cast<const __nv_bfloat16*>(d_X) + r0 * ldx;
      st = tch::rotate_tokens<tc::EPI_GEN>(ctx, xc, rows, d, ldx, rt, O, d, nullptr);
    } else {
      GemmDesc g{};
      g.A = reinterpret_cast<const float*>(d_X) + r0 * ldx; g.lda = ldx; g.transA = 0;
      g.B = d_R; g.ldb = d; g.transB = 0;
      g.C = O; g.ldc = d;
      g.M = (int)rows; g.N = d; g.K = d; g.alpha = 1.f; g.beta = 0.f; g.batch = 1;
      st = gemm_f32(ctx, g);
    }
    if (st != DQ_OK) break;
    token_metrics_kernel<<<(unsigned)((rows + 7) / 8), 256, 0, ctx.stream>>>(O, rows, d, tau, maxq, sq, cnt);
    st = after_launch(ctx);
    if (st != DQ_OK) break;
    metrics_reduce_kernel<<<1, 256, 0, ctx.stream>>>(sq, cnt, rows, d_out);
    st = after_launch(ctx);
  }
  if (st == DQ_OK) {
    finish_metrics_kernel<<<1, 1, 0, ctx.stream>>>(d_out, (double)n * (double)d);
    st = after_launch(ctx);
  }
  cudaFreeAsync(O, ctx.stream); cudaFreeAsync(sq, ctx.stream); cudaFreeAsync(cnt, ctx.stream);
  if (rt) cudaFreeAsync(rt, ctx.stream);
  return st;
}

}  // namespace dq
