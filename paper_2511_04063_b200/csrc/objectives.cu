// Alternative calibration objectives of the ablation in Sec. 5.3 (variance, kurtosis,
// quantisation loss) in place of the Whip loss.  Unlike Eq. 4 they are not element-wise: every
// entry of dL/dO needs statistics of the whole rotated token (mean and central moments, or the
// quantisation grid from min / max), so they cannot live in the epilogue of one GEMM tile.  The
// rotated activations are therefore materialised chunk by chunk in fp32 (tensor-core GEMM for
// bf16 inputs), and one kernel per chunk computes the token statistics, the token's loss and
// dL/dO, written directly in the layout the backward contraction reads.
//   variance:  v = m2,                 dv/do_j = (2/d) c_j,                 c = o - mean(o)
//   kurtosis:  k = m4 / m2^2 - 3,      dk/do_j = (4/d) ((c_j^3 - m3) / m2^2 - m4 c_j / m2^3)
//   quant:     e = (1/d) sum (o - Q(o))^2,  de/do_j = (2/d) (o_j - Q(o)_j)  (grid held fixed),
//              Q = per-token asymmetric uniform quantiser (as in eval_metrics.cu)
// with m_p = (1/d) sum_j c_j^p.  The paper names these objectives without formulas; these are the
// per-token population statistics over channels, matching how Eq. 4 is applied per token.
#include "tc_host.cuh"
#include "tc_path.cuh"

namespace dq {
namespace {

using bf16 = __nv_bfloat16;

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
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

constexpr int TOK = 32;   // tokens per CTA

// dL/dO of one entry from the token's coefficients.
//   variance: k = {mean, 2/d, -, -};  kurtosis: k = {mean, A, B, C}: A c^3 - B c - C;
//   quant: k = {scale, zero, maxq, 2/d} (scale == 0: constant row, no error)
__device__ __forceinline__ float grad_entry(int objective, float o, const float4 k) {
  if (objective == DQ_OBJ_VARIANCE) return k.y * (o - k.x);
  if (objective == DQ_OBJ_KURTOSIS) {
    const float c = o - k.x;
    return k.y * c * c * c - k.z * c - k.w;
  }
  if (k.x == 0.f) return 0.f;
  const float q = fminf(fmaxf(rintf(o / k.x) + k.y, 0.f), k.z);
  return k.w * (o - k.x * (q - k.y));
}

// O: [rows][d] fp32 (one chunk of rotated tokens).  TRANSPOSED: G is bf16 [d][ldg] channel-major and
// the chunk's first token is column t0; otherwise G is fp32 [token][d] with row t0 + t.
template <bool TRANSPOSED>
__global__ void __launch_bounds__(256) objective_grad_kernel(const float* __restrict__ O, int64_t rows, int d,
                                                             int objective, float maxq, void* __restrict__ Gout,
                                                             int64_t ldg, int64_t t0,
                                                             double* __restrict__ tok_loss) {
  __shared__ float4 coef[TOK];
  __shared__ float tile[TOK][33];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t tb = (int64_t)blockIdx.x * TOK;
  const float inv_d = 1.f / (float)d;
  // phase 1: statistics of four tokens per warp
  for (int i = 0; i < TOK / 8; ++i) {
    const int tl = warp * (TOK / 8) + i;
    const int64_t t = tb + tl;
    if (t >= rows) { if (lane == 0) coef[tl] = make_float4(0.f, 0.f, 0.f, 0.f); continue; }
    const float* o = O + t * d;
    float4 k;
    double l;
    if (objective == DQ_OBJ_QUANT) {
      float lo = INFINITY, hi = -INFINITY;
      for (int j = lane; j < d; j += 32) { const float v = o[j]; lo = fminf(lo, v); hi = fmaxf(hi, v); }
      lo = warp_min(lo); hi = warp_max(hi);
      const float range = hi - lo;
      const float scale = (range > 0.f) ? range / maxq : 0.f;
      const float zero = (range > 0.f) ? rintf(-lo / scale) : 0.f;
      float e = 0.f;
      if (range > 0.f) {
        for (int j = lane; j < d; j += 32) {
          const float v = o[j];
          const float q = fminf(fmaxf(rintf(v / scale) + zero, 0.f), maxq);
          const float diff = v - scale * (q - zero);
          e = fmaf(diff, diff, e);
        }
      }
      e = warp_sum(e);
      k = make_float4(scale, zero, maxq, 2.f * inv_d);
      l = (double)e * (double)inv_d;
    } else {
      float s = 0.f;
      for (int j = lane; j < d; j += 32) s += o[j];
      const float mu = warp_sum(s) * inv_d;
      float s2 = 0.f, s3 = 0.f, s4 = 0.f;
      for (int j = lane; j < d; j += 32) {
        const float c = o[j] - mu, c2 = c * c;
        s2 += c2; s3 = fmaf(c2, c, s3); s4 = fmaf(c2, c2, s4);
      }
      const float m2 = warp_sum(s2) * inv_d, m3 = warp_sum(s3) * inv_d, m4 = warp_sum(s4) * inv_d;
      if (objective == DQ_OBJ_VARIANCE) {
        k = make_float4(mu, 2.f * inv_d, 0.f, 0.f);
        l = (double)m2;
      } else {   // a constant row has m2 = 0: the kurtosis is undefined and the loss becomes non-finite
        const float i2 = 1.f / (m2 * m2);
        k = make_float4(mu, 4.f * inv_d * i2, 4.f * inv_d * m4 * i2 / m2, 4.f * inv_d * m3 * i2);
        l = (double)m4 * (double)i2 - 3.0;
      }
    }
    if (lane == 0) { coef[tl] = k; tok_loss[t] = l; }
  }
  __syncthreads();
  // phase 2: dL/dO of the CTA's tokens, 32 channels at a time
  if (!TRANSPOSED) {
    float* G = reinterpret_cast<float*>(Gout);
    for (int tl = warp; tl < TOK; tl += 8) {
      const int64_t t = tb + tl;
      if (t >= rows) continue;
      const float4 k = coef[tl];
      for (int j = lane; j < d; j += 32) G[(t0 + t) * ldg + j] = grad_entry(objective, O[t * d + j], k);
    }
    return;
  }
  bf16* G = reinterpret_cast<bf16*>(Gout);
  for (int c0 = 0; c0 < d; c0 += 32) {
    for (int tl = warp; tl < TOK; tl += 8) {
      const int64_t t = tb + tl;
      tile[tl][lane] = (t < rows) ? grad_entry(objective, O[t * d + c0 + lane], coef[tl]) : 0.f;
    }
    __syncthreads();
    if (tb + lane < rows) {
      for (int c = warp; c < 32; c += 8)
        G[(int64_t)(c0 + c) * ldg + t0 + tb + lane] = __float2bfloat16_rn(tile[lane][c]);
    }
    __syncthreads();
  }
}

// acc[0] += sum of tok_loss[0..rows) in a fixed order (one CTA).
__global__ void __launch_bounds__(256) loss_accumulate_kernel(const double* __restrict__ tok_loss, int64_t rows,
                                                              double* __restrict__ acc) {
  __shared__ double red[256];
  double s = 0.0;
  for (int64_t i = threadIdx.x; i < rows; i += 256) s += tok_loss[i];
  red[threadIdx.x] = s;
  __syncthreads();
  for (int off = 128; off >= 1; off >>= 1) {
    if ((int)threadIdx.x < off) red[threadIdx.x] += red[threadIdx.x + off];
    __syncthreads();
  }
  if (threadIdx.x == 0) acc[0] += red[0];
}

__global__ void objective_loss_finish_kernel(const double* __restrict__ acc, int batch, double scale,
                                             float* __restrict__ loss_last, int* d_status) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= batch) return;
  const double v = acc[b] * scale;
  if (!(v == v) || v > 3.0e38 || v < -3.0e38) set_status(d_status, DQ_ERR_NONFINITE);
  loss_last[b] = (float)v;
}

}  // namespace

dq_status objective_init(ObjectiveState& os, int d, int64_t n_tokens, int batch) {
  int64_t chunk = (((int64_t)1 << 25) / d / 128) * 128;     // 128 MiB of fp32 rotated activations at a time
  if (chunk < 128) chunk = 128;
  if (chunk > n_tokens) chunk = n_tokens;
  os.chunk = chunk;
  if (cudaMalloc((void**)&os.O, sizeof(float) * (size_t)chunk * d) != cudaSuccess) return DQ_ERR_ALLOC;
  if (cudaMalloc((void**)&os.tok_loss, sizeof(double) * (size_t)chunk) != cudaSuccess) return DQ_ERR_ALLOC;
  if (cudaMalloc((void**)&os.acc, sizeof(double) * batch) != cudaSuccess) return DQ_ERR_ALLOC;
  os.ready = true;
  return DQ_OK;
}

void objective_destroy(ObjectiveState& os) {
  cudaFree(os.O); cudaFree(os.tok_loss); cudaFree(os.acc);
  os = ObjectiveState{};
}

// Loss and dL/dO (without the 1 / N of the token mean, as for the Whip path) of every problem.
// Tensor-core path: X bf16 [b][N][d], rt = bf16 R^T [b][d][d], G = bf16 [b][d][N].
// fp32 path: X fp32 [b][N][ldx], R fp32 [b][d][d], G = fp32 [b][N][d].
dq_status objective_forward(Ctx& ctx, ObjectiveState& os, const dq_calib_config& cfg, const void* X, const float* R,
                            const __nv_bfloat16* rt, void* G, float loss_scale, float* loss_last) {
  if (!os.ready) return DQ_ERR_INVALID_ARG;
  const int d = cfg.d, batch = cfg.batch;
  const int64_t N = cfg.n_tokens;
  const bool tcp = cfg.path == DQ_PATH_BF16_TC;
  const float maxq = (float)((1 << os.bits) - 1);
  DQ_CHECK_CUDA(cudaMemsetAsync(os.acc, 0, sizeof(double) * batch, ctx.stream));
  for (int b = 0; b < batch; ++b) {
    for (int64_t r0 = 0; r0 < N; r0 += os.chunk) {
      const int64_t rows = (N - r0 < os.chunk) ? N - r0 : os.chunk;
      if (tcp) {   // O[token][channel] = sum_k X[token][k] R^T[channel][k]
        const bf16* xc = reinterpret_cast<const bf16*>(X) + ((int64_t)b * N + r0) * cfg.ldx;
        DQ_CHECK(tch::rotate_tokens<tc::EPI_GEN>(ctx, xc, rows, d, cfg.ldx, rt + (int64_t)b * d * d, os.O, d,
                                                 ctx.d_status));
        objective_grad_kernel<true><<<(unsigned)((rows + TOK - 1) / TOK), 256, 0, ctx.stream>>>(
            os.O, rows, d, os.objective, maxq, reinterpret_cast<bf16*>(G) + (int64_t)b * d * N, N, r0, os.tok_loss);
      } else {
        GemmDesc g{};
        g.A = reinterpret_cast<const float*>(X) + ((int64_t)b * N + r0) * cfg.ldx; g.lda = cfg.ldx; g.transA = 0;
        g.B = R + (int64_t)b * d * d; g.ldb = d; g.transB = 0;
        g.C = os.O; g.ldc = d;
        g.M = (int)rows; g.N = d; g.K = d; g.alpha = 1.f; g.beta = 0.f; g.batch = 1;
        DQ_CHECK(gemm_f32(ctx, g));
        objective_grad_kernel<false><<<(unsigned)((rows + TOK - 1) / TOK), 256, 0, ctx.stream>>>(
            os.O, rows, d, os.objective, maxq, reinterpret_cast<float*>(G) + (int64_t)b * N * d, d, r0, os.tok_loss);
      }
      DQ_CHECK(after_launch(ctx));
      loss_accumulate_kernel<<<1, 256, 0, ctx.stream>>>(os.tok_loss, rows, os.acc + b);
      DQ_CHECK(after_launch(ctx));
    }
  }
  objective_loss_finish_kernel<<<(batch + 127) / 128, 128, 0, ctx.stream>>>(os.acc, batch, (double)loss_scale,
                                                                           loss_last, ctx.d_status);
  return after_launch(ctx);
}

}  // namespace dq
