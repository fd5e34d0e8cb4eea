// fp32 FMA contractions: the exact-fp32 path of the calibration step and the
// general small-matrix helper of QR-Orth.
#include "common.cuh"

namespace dq {
namespace {

constexpr int BM = 64, BN = 64, BK = 16, PAD = 4;

enum { EPI_AXPBY = 0, EPI_WHIP = 1 };

// 256 threads; thread (ty, tx) owns a 4x4 block of the 64x64 tile.
template <int EPI>
__global__ void __launch_bounds__(256) gemm_ffma_kernel(GemmDesc g, float* __restrict__ partials) {
  __shared__ __align__(16) float As[BK][BM + PAD];
  __shared__ __align__(16) float Bs[BK][BN + PAD];
  __shared__ float warp_sums[8];
  if (g.run_if && *g.run_if == 0) return;

  const int b = blockIdx.z / g.ksplit, ks = blockIdx.z % g.ksplit;
  const float* __restrict__ A = g.A + (int64_t)b * g.sA;
  const float* __restrict__ B = g.B + (int64_t)b * g.sB;
  float* __restrict__ C = g.C + (int64_t)blockIdx.z * g.sC;
  // K range of this slice, in multiples of BK
  const int kchunk = (((g.K + g.ksplit - 1) / g.ksplit) + BK - 1) / BK * BK;
  const int kbeg = ks * kchunk;
  const int kend = min(g.K, kbeg + kchunk);
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;

  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

  for (int k0 = kbeg; k0 < kend; k0 += BK) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int idx = tid + i * 256;
      int m, k;
      if (!g.transA) { k = idx & 15; m = idx >> 4; } else { m = idx & 63; k = idx >> 6; }
      float v = 0.f;
      if (m0 + m < g.M && k0 + k < kend)
        v = g.transA ? A[(int64_t)(k0 + k) * g.lda + m0 + m] : A[(int64_t)(m0 + m) * g.lda + k0 + k];
      As[k][m] = v;
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int idx = tid + i * 256;
      int n, k;
      if (!g.transB) { n = idx & 63; k = idx >> 6; } else { k = idx & 15; n = idx >> 4; }
      float v = 0.f;
      if (n0 + n < g.N && k0 + k < kend)
        v = g.transB ? B[(int64_t)(n0 + n) * g.ldb + k0 + k] : B[(int64_t)(k0 + k) * g.ldb + n0 + n];
      Bs[k][n] = v;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < BK; ++k) {
      const float4 a4 = *reinterpret_cast<const float4*>(&As[k][ty * 4]);
      const float4 b4 = *reinterpret_cast<const float4*>(&Bs[k][tx * 4]);
      const float a[4] = {a4.x, a4.y, a4.z, a4.w};
      const float bb[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], bb[j], acc[i][j]);
    }
    __syncthreads();
  }

  if (EPI == EPI_AXPBY) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int m = m0 + ty * 4 + i;
      if (m >= g.M) continue;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int n = n0 + tx * 4 + j;
        if (n >= g.N) continue;
        float* c = C + (int64_t)m * g.ldc + n;
        float v = g.alpha * acc[i][j];
        if (g.beta != 0.f && g.ksplit == 1) v = fmaf(g.beta, *c, v);
        *c = v;
      }
    }
  } else {
    // Eq. 4 per element: e = exp(-|o|); dL/do = -sign(o) e (0 at o = 0).
    float local = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int m = m0 + ty * 4 + i;
      if (m >= g.M) continue;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int n = n0 + tx * 4 + j;
        if (n >= g.N) continue;
        const float o = acc[i][j];
        const float e = expf(-fabsf(o));
        local += e;
        C[(int64_t)m * g.ldc + n] = (o > 0.f) ? -e : ((o < 0.f) ? e : 0.f);
      }
    }
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) local += __shfl_xor_sync(0xffffffffu, local, off);
    if ((tid & 31) == 0) warp_sums[tid >> 5] = local;
    __syncthreads();
    if (tid == 0) {
      float s = 0.f;
#pragma unroll
      for (int w = 0; w < 8; ++w) s += warp_sums[w];
      partials[((int64_t)b * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x] = s;
    }
  }
}

}  // namespace

dq_status gemm_f32(Ctx& ctx, const GemmDesc& g) {
  if (g.M <= 0 || g.N <= 0 || g.batch <= 0) return DQ_OK;
  dim3 grid((g.N + BN - 1) / BN, (g.M + BM - 1) / BM, g.batch * g.ksplit);
  gemm_ffma_kernel<EPI_AXPBY><<<grid, 256, 0, ctx.stream>>>(g, nullptr);
  return after_launch(ctx);
}

namespace {
__global__ void splitk_reduce_kernel(const float* __restrict__ part, int ksplit, int64_t n,
                                     float alpha, float beta, float* __restrict__ out) {
  const int b = blockIdx.y;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
    float s = 0.f;
    for (int ks = 0; ks < ksplit; ++ks) s += part[((int64_t)b * ksplit + ks) * n + i];
    float* o = out + (int64_t)b * n + i;
    *o = (beta != 0.f) ? fmaf(beta, *o, alpha * s) : alpha * s;
  }
}
// the same sums, four consecutive elements per thread (n a multiple of 4, 16-byte aligned buffers)
__global__ void splitk_reduce4_kernel(const float4* __restrict__ part, int ksplit, int64_t n4,
                                      float alpha, float beta, float4* __restrict__ out) {
  const int b = blockIdx.y;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += stride) {
    float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
    for (int ks = 0; ks < ksplit; ++ks) {
      const float4 v = part[((int64_t)b * ksplit + ks) * n4 + i];
      s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
    }
    float4* o = out + (int64_t)b * n4 + i;
    if (beta != 0.f) {
      const float4 c = *o;
      *o = make_float4(fmaf(beta, c.x, alpha * s.x), fmaf(beta, c.y, alpha * s.y), fmaf(beta, c.z, alpha * s.z),
                       fmaf(beta, c.w, alpha * s.w));
    } else {
      *o = make_float4(alpha * s.x, alpha * s.y, alpha * s.z, alpha * s.w);
    }
  }
}
}  // namespace

dq_status splitk_reduce(Ctx& ctx, const float* part, int ksplit, int64_t n_per_batch, int batch,
                        float alpha, float beta, float* out) {
  if (n_per_batch % 4 == 0 && (((uintptr_t)part | (uintptr_t)out) & 15) == 0) {
    const int64_t n4 = n_per_batch / 4;
    int bx = (int)((n4 + 255) / 256);
    if (bx > 1024) bx = 1024;
    splitk_reduce4_kernel<<<dim3(bx, batch), 256, 0, ctx.stream>>>(reinterpret_cast<const float4*>(part), ksplit, n4, alpha, beta,
                                                                 reinterpret_cast<float4*>(out));
    return after_launch(ctx);
  }
  int bx = (int)((n_per_batch + 255) / 256);
  if (bx > 1024) bx = 1024;
  splitk_reduce_kernel<<<dim3(bx, batch), 256, 0, ctx.stream>>>(part, ksplit, n_per_batch, alpha,
                                                              beta, out);
  return after_launch(ctx);
}

int whip_forward_f32_tiles(int64_t n_tokens, int d) {
  return (int)(((n_tokens + BM - 1) / BM) * ((d + BN - 1) / BN));
}

dq_status whip_forward_f32(Ctx& ctx, const float* X, int64_t ldx, int64_t strideX, const float* R,
                           float* G, float* partials, int64_t n_tokens, int d, int batch,
                           int* tiles_per_problem) {
  GemmDesc g{};
  g.A = X; g.lda = ldx; g.transA = 0; g.sA = strideX;
  g.B = R; g.ldb = d; g.transB = 0; g.sB = (int64_t)d * d;
  g.C = G; g.ldc = d; g.sC = n_tokens * (int64_t)d;
  g.M = (int)n_tokens; g.N = d; g.K = d; g.alpha = 1.f; g.beta = 0.f; g.batch = batch; g.ksplit = 1;
  dim3 grid((g.N + BN - 1) / BN, (g.M + BM - 1) / BM, g.batch);
  if (tiles_per_problem) *tiles_per_problem = (int)(grid.x * grid.y);
  gemm_ffma_kernel<EPI_WHIP><<<grid, 256, 0, ctx.stream>>>(g, partials);
  return after_launch(ctx);
}

// ---------------------------------------------------------------------------
// Loss reduction: one block per problem, fixed summation order, fp64 accumulate.
// ---------------------------------------------------------------------------
namespace {
__global__ void __launch_bounds__(256) loss_finalize_kernel(const float* __restrict__ partials, int n,
                                                            float scale, float* __restrict__ loss_out,
                                                            float* __restrict__ loss_last,
                                                            int* d_status) {
  __shared__ double sm[256];
  const int b = blockIdx.x;
  const float* p = partials + (int64_t)b * n;
  double s = 0.0;
  for (int i = threadIdx.x; i < n; i += 256) s += (double)p[i];
  sm[threadIdx.x] = s;
  __syncthreads();
  for (int off = 128; off >= 1; off >>= 1) {
    if (threadIdx.x < off) sm[threadIdx.x] += sm[threadIdx.x + off];
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const float L = (float)(sm[0] * (double)scale);
    if (loss_out) loss_out[b] = L;
    loss_last[b] = L;
    if (!isfinite(L)) set_status(d_status, DQ_ERR_NONFINITE);
  }
}

// Every update kernel leaves the parameter (and the optimiser state) untouched once the status word holds
// an error: a step whose factorisation failed or whose loss was not finite never reaches the latent.
// hi / lo (nullable): also write the split-bf16 copy of the new Z (hi = bf16(z), lo = bf16(z - hi)), the
// operand form the next factorisation reads, so that it needs no separate pass over Z.
__global__ void sgd_kernel(float4* __restrict__ Z, const float4* __restrict__ Gz, float lr, int64_t n4,
                           const int* __restrict__ d_status, uint2* __restrict__ hi, uint2* __restrict__ lo) {
  if (d_status && *d_status != 0) return;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += stride) {
    float4 z = Z[i];
    const float4 g = Gz[i];
    z.x = fmaf(-lr, g.x, z.x); z.y = fmaf(-lr, g.y, z.y);
    z.z = fmaf(-lr, g.z, z.z); z.w = fmaf(-lr, g.w, z.w);
    Z[i] = z;
    if (hi) {
      const __nv_bfloat162 h0 = __floats2bfloat162_rn(z.x, z.y), h1 = __floats2bfloat162_rn(z.z, z.w);
      const float2 f0 = __bfloat1622float2(h0), f1 = __bfloat1622float2(h1);
      const __nv_bfloat162 l0 = __floats2bfloat162_rn(z.x - f0.x, z.y - f0.y);
      const __nv_bfloat162 l1 = __floats2bfloat162_rn(z.z - f1.x, z.w - f1.y);
      hi[i] = make_uint2(*reinterpret_cast<const uint32_t*>(&h0), *reinterpret_cast<const uint32_t*>(&h1));
      lo[i] = make_uint2(*reinterpret_cast<const uint32_t*>(&l0), *reinterpret_cast<const uint32_t*>(&l1));
    }
  }
}

// v <- mu v + g;  Z <- Z - lr v
__global__ void momentum_kernel(float4* __restrict__ Z, const float4* __restrict__ Gz, float4* __restrict__ V,
                                float lr, float mu, int64_t n4, const int* __restrict__ d_status) {
  if (d_status && *d_status != 0) return;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += stride) {
    float4 z = Z[i], v = V[i];
    const float4 g = Gz[i];
    v.x = fmaf(mu, v.x, g.x); v.y = fmaf(mu, v.y, g.y); v.z = fmaf(mu, v.z, g.z); v.w = fmaf(mu, v.w, g.w);
    z.x = fmaf(-lr, v.x, z.x); z.y = fmaf(-lr, v.y, z.y); z.z = fmaf(-lr, v.z, z.z); z.w = fmaf(-lr, v.w, z.w);
    V[i] = v;
    Z[i] = z;
  }
}

// pw[0] = beta1^t, pw[1] = beta2^t of the step about to be taken (t counted on the device so that a
// replayed CUDA graph advances it)
__global__ void adam_advance_kernel(float* pw, float beta1, float beta2, const int* d_status) {
  if (d_status && *d_status != 0) return;
  pw[0] *= beta1;
  pw[1] *= beta2;
}

__device__ __forceinline__ float adam_one(float& z, float g, float& m, float& v, float b1, float b2, float c1,
                                          float c2, float lr, float eps) {
  m = fmaf(b1, m, (1.f - b1) * g);
  v = fmaf(b2, v, (1.f - b2) * g * g);
  const float mhat = m * c1, vhat = v * c2;
  z -= lr * mhat / (sqrtf(vhat) + eps);
  return z;
}

// Adam in its published form with bias correction; c1 = 1 / (1 - beta1^t), c2 = 1 / (1 - beta2^t).
__global__ void adam_kernel(float4* __restrict__ Z, const float4* __restrict__ Gz, float4* __restrict__ M,
                            float4* __restrict__ V, const float* __restrict__ pw, float lr, float b1, float b2,
                            float eps, int64_t n4, const int* __restrict__ d_status) {
  if (d_status && *d_status != 0) return;
  const float c1 = 1.f / (1.f - pw[0]), c2 = 1.f / (1.f - pw[1]);
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += stride) {
    float4 z = Z[i], m = M[i], v = V[i];
    const float4 g = Gz[i];
    adam_one(z.x, g.x, m.x, v.x, b1, b2, c1, c2, lr, eps);
    adam_one(z.y, g.y, m.y, v.y, b1, b2, c1, c2, lr, eps);
    adam_one(z.z, g.z, m.z, v.z, b1, b2, c1, c2, lr, eps);
    adam_one(z.w, g.w, m.w, v.w, b1, b2, c1, c2, lr, eps);
    M[i] = m; V[i] = v; Z[i] = z;
  }
}
}  // namespace

dq_status loss_finalize(Ctx& ctx, const float* partials, int n_per_problem, int batch, float scale,
                        float* loss_out, float* loss_last) {
  loss_finalize_kernel<<<batch, 256, 0, ctx.stream>>>(partials, n_per_problem, scale, loss_out,
                                                     loss_last, ctx.d_status);
  return after_launch(ctx);
}

namespace {
__global__ void __launch_bounds__(256) accumulate_kernel(float* __restrict__ dst, const float* __restrict__ src,
                                                         int64_t n) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
    dst[i] += src[i];
}
}  // namespace

// dst += src (gradient accumulation over micro-batches)
dq_status accumulate(Ctx& ctx, float* dst, const float* src, int64_t n) {
  int blocks = (int)((n + 255) / 256);
  const int cap = ctx.sm_count * 8;
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  accumulate_kernel<<<blocks, 256, 0, ctx.stream>>>(dst, src, n);
  return after_launch(ctx);
}

// Algorithm 1 (update step).  n is a multiple of 4 (d is a multiple of 32).
dq_status sgd_update(Ctx& ctx, float* Z, const float* Gz, float lr, int64_t n, __nv_bfloat16* z_hi,
                     __nv_bfloat16* z_lo) {
  const int64_t n4 = n / 4;
  int blocks = (int)((n4 + 255) / 256);
  const int cap = ctx.sm_count * 8;
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  sgd_kernel<<<blocks, 256, 0, ctx.stream>>>(reinterpret_cast<float4*>(Z),
                                            reinterpret_cast<const float4*>(Gz), lr, n4, ctx.d_status,
                                            reinterpret_cast<uint2*>(z_hi), reinterpret_cast<uint2*>(z_lo));
  return after_launch(ctx);
}


static int update_blocks(const Ctx& ctx, int64_t n4) {
  int blocks = (int)((n4 + 255) / 256);
  const int cap = ctx.sm_count * 8;
  if (blocks > cap) blocks = cap;
  return blocks < 1 ? 1 : blocks;
}

// SGD with momentum on the latent (Sec. 4.3: Z is optimised with a standard optimiser).
dq_status momentum_update(Ctx& ctx, float* Z, const float* Gz, float* V, float lr, float mu, int64_t n) {
  const int64_t n4 = n / 4;
  momentum_kernel<<<update_blocks(ctx, n4), 256, 0, ctx.stream>>>(
      reinterpret_cast<float4*>(Z), reinterpret_cast<const float4*>(Gz), reinterpret_cast<float4*>(V), lr, mu, n4, ctx.d_status);
  return after_launch(ctx);
}

// Adam on the latent (Sec. 4.3, optimiser comparison).  pw: device float[2] holding beta1^t, beta2^t of
// the previous step (1, 1 before the first).
dq_status adam_update(Ctx& ctx, float* Z, const float* Gz, float* M, float* V, float* pw, float lr, float b1,
                      float b2, float eps, int64_t n) {
  const int64_t n4 = n / 4;
  adam_advance_kernel<<<1, 1, 0, ctx.stream>>>(pw, b1, b2, ctx.d_status);
  DQ_CHECK(after_launch(ctx));
  adam_kernel<<<update_blocks(ctx, n4), 256, 0, ctx.stream>>>(
      reinterpret_cast<float4*>(Z), reinterpret_cast<const float4*>(Gz), reinterpret_cast<float4*>(M),
      reinterpret_cast<float4*>(V), pw, lr, b1, b2, eps, n4, ctx.d_status);
  return after_launch(ctx);
}

}  // namespace dq
