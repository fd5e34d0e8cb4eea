// QR-Orth forward (Sec. 4.3): blocked Householder QR (Algorithm 2 in compact-WY
// form), explicit orthogonal factor, and the positive-diagonal gauge.
//
// Panel = 32 columns factored by one thread-block cluster of 8 CTAs: every
// thread keeps two panel rows (2 x 32 floats) in registers, each column step
// needs one warp-transpose reduction, one CTA reduction and one cluster barrier
// (partials are exchanged through distributed shared memory in a fixed order,
// so results are bit-reproducible).
#include <cooperative_groups.h>

#include "common.cuh"

namespace cg = cooperative_groups;

namespace dq {
namespace {

constexpr int PB = 32;         // panel width
constexpr int PT = 512;        // threads per CTA
constexpr int PC = 8;          // CTAs per cluster
constexpr int RPT = 2;         // rows per thread  -> PC * PT * RPT = 8192 rows max

// Read a float from the same shared-memory offset of CTA `rank` of this cluster.
__device__ __forceinline__ float ld_dsmem(uint32_t smem_addr, int rank) {
  uint32_t remote;
  float v;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(smem_addr), "r"(rank));
  asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(remote) : "memory");
  return v;
}

// Factor A[c0:d, c0:c0+32] (row-major, leading dimension d) in place:
//   A  <- upper-triangular part of the panel (zeros below the diagonal)
//   V  <- Householder vectors, unit diagonal, zeros above (same position as A)
//   T  <- 32 x 32 upper-triangular factor with H_1 ... H_32 = I - V T V^T
// H_j = I - tau_j v_j v_j^T, v_j = (x - beta e1) / (x_1 - beta),
// beta = -sign(x_1) ||x||  (Algorithm 2's sign rule), tau_j = (beta - x_1) / beta.
__global__ void __cluster_dims__(PC, 1, 1) __launch_bounds__(PT, 1)
qr_panel_kernel(float* __restrict__ A, float* __restrict__ V, float* __restrict__ T, int d, int c0,
                int64_t strideA, int64_t strideT) {
  cg::cluster_group cluster = cg::this_cluster();
  const int cta = (int)cluster.block_rank();
  A += (int64_t)blockIdx.y * strideA;
  V += (int64_t)blockIdx.y * strideA;
  T += (int64_t)blockIdx.y * strideT;

  __shared__ float red[PT / 32][32];
  __shared__ float xg[2][32];   // this CTA's column sums, double buffered
  __shared__ float xd[2][32];   // (CTA 0) the diagonal row of the current column
  __shared__ float Ts[32][33];
  __shared__ float zs[32];
  __shared__ float coefs[PT / 32][32];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int m = d - c0;

  float a[RPT][32];
  int rowi[RPT];
#pragma unroll
  for (int r = 0; r < RPT; ++r) {
    const int slot = r * PT + tid;
    const int group = (slot >> 5) * PC + cta;     // 32-row groups dealt round-robin to CTAs
    const int i = group * 32 + (slot & 31);
    rowi[r] = i;
    if (i < m) {
      const float4* src = reinterpret_cast<const float4*>(A + (int64_t)(c0 + i) * d + c0);
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        const float4 v = src[q];
        a[r][4 * q + 0] = v.x; a[r][4 * q + 1] = v.y; a[r][4 * q + 2] = v.z; a[r][4 * q + 3] = v.w;
      }
    } else {
#pragma unroll
      for (int c = 0; c < 32; ++c) a[r][c] = 0.f;
    }
  }
  if (cta == 0 && warp == 0) {
#pragma unroll
    for (int c = 0; c < 32; ++c) Ts[lane][c] = 0.f;
  }
  const uint32_t xg_addr = (uint32_t)__cvta_generic_to_shared(&xg[0][0]);
  const uint32_t xd_addr = (uint32_t)__cvta_generic_to_shared(&xd[0][0]);

#pragma unroll
  for (int j = 0; j < PB; ++j) {
    const int par = j & 1;
    // g[c] = sum over rows i >= j of A[i][j] * A[i][c]  (all 32 columns at once)
    float acc[32];
#pragma unroll
    for (int c = 0; c < 32; ++c) acc[c] = 0.f;
#pragma unroll
    for (int r = 0; r < RPT; ++r) {
      const float x = (rowi[r] >= j) ? a[r][j] : 0.f;
#pragma unroll
      for (int c = 0; c < 32; ++c) acc[c] = fmaf(x, a[r][c], acc[c]);
    }
    const float tot = warp_transpose_reduce32(acc, lane);
    red[warp][lane] = tot;
    if (cta == 0 && tid == j) {   // thread j of CTA 0 owns panel row j (the diagonal row)
#pragma unroll
      for (int c = 0; c < 32; ++c) xd[par][c] = a[0][c];
    }
    __syncthreads();
    if (warp == 0) {
      float s = 0.f;
#pragma unroll
      for (int w = 0; w < PT / 32; ++w) s += red[w][lane];
      xg[par][lane] = s;
    }
    cluster.sync();
    float g = 0.f;
#pragma unroll
    for (int rk = 0; rk < PC; ++rk) g += ld_dsmem(xg_addr + 4u * (par * 32 + lane), rk);
    const float dr = ld_dsmem(xd_addr + 4u * (par * 32 + lane), 0);
    const float alpha = __shfl_sync(0xffffffffu, dr, j);
    const float nrm2 = __shfl_sync(0xffffffffu, g, j);
    const float sigma = nrm2 - alpha * alpha;          // squared norm below the diagonal
    const bool skip = !(sigma > 0.f);                  // nothing to annihilate: H_j = I
    const float beta = skip ? alpha : -copysignf(sqrtf(nrm2), alpha);
    const float denom = alpha - beta;
    const float inv_denom = skip ? 0.f : 1.f / denom;
    const float tau = skip ? 0.f : -denom / beta;
    // lane c: w_c = v_j^T A[:, c]  (for c < j this is V[:, c]^T v_j, needed by T)
    const float w = fmaf(g - alpha * dr, inv_denom, dr);
    const float tw = tau * w;
    coefs[warp][lane] = tw;       // broadcast through shared memory (keeps registers for the panel)
    __syncwarp();
#pragma unroll
    for (int r = 0; r < RPT; ++r) {
      const bool on_diag = rowi[r] == j;
      const bool below = rowi[r] > j;
      const float vi = on_diag ? 1.f : (below ? a[r][j] * inv_denom : 0.f);
#pragma unroll
      for (int c = 0; c < 32; ++c)
        if (c > j) a[r][c] = fmaf(-vi, coefs[warp][c], a[r][c]);
      a[r][j] = on_diag ? beta : (below ? a[r][j] * inv_denom : a[r][j]);
    }
    if (cta == 0 && warp == 0) {
      // T[:j, j] = -tau T[:j, :j] (V[:, :j]^T v_j);  T[j, j] = tau
      zs[lane] = w;
      __syncwarp();
      if (lane < j) {
        float s = 0.f;
#pragma unroll
        for (int c = 0; c < 32; ++c)
          if (c < j && c >= lane) s = fmaf(Ts[lane][c], zs[c], s);
        Ts[lane][j] = -tau * s;
      } else if (lane == j) {
        Ts[j][j] = tau;
      }
      __syncwarp();
    }
  }

#pragma unroll
  for (int r = 0; r < RPT; ++r) {
    const int i = rowi[r];
    if (i < m) {
      float4* dstA = reinterpret_cast<float4*>(A + (int64_t)(c0 + i) * d + c0);
      float4* dstV = reinterpret_cast<float4*>(V + (int64_t)(c0 + i) * d + c0);
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        float u[4], v[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int c = 4 * q + e;
          u[e] = (i <= c) ? a[r][c] : 0.f;
          v[e] = (i > c) ? a[r][c] : ((i == c) ? 1.f : 0.f);
        }
        dstA[q] = make_float4(u[0], u[1], u[2], u[3]);
        dstV[q] = make_float4(v[0], v[1], v[2], v[3]);
      }
    }
  }
  __syncthreads();
  if (cta == 0) {
    for (int idx = tid; idx < 32 * 32; idx += PT) T[idx] = Ts[idx >> 5][idx & 31];
  }
  cluster.sync();   // no CTA may exit while its shared memory can still be read remotely
}

__global__ void set_identity_kernel(float* __restrict__ Q, int d) {
  float* q = Q + (int64_t)blockIdx.y * d * d;
  const int64_t n = (int64_t)d * d;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride)
    q[i] = ((i / d) == (i % d)) ? 1.f : 0.f;
}

// Gauge (diag(U) > 0): R = Q diag(s), U = diag(s) triu(A), s_j = sign(A_jj) (+1 at 0).
// Optionally writes bf16(R^T) for the tensor-core contraction.
__global__ void __launch_bounds__(256) gauge_kernel(const float* __restrict__ Q, const float* __restrict__ A,
                                                    float* __restrict__ R, float* __restrict__ U,
                                                    __nv_bfloat16* __restrict__ Rt, int d) {
  __shared__ float tile[32][33];
  const int64_t off = (int64_t)blockIdx.z * d * d;
  Q += off; A += off; R += off; U += off;
  if (Rt) Rt += off;
  const int i0 = blockIdx.y * 32, j0 = blockIdx.x * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;   // 32 x 8
  for (int r = ty; r < 32; r += 8) {
    const int i = i0 + r, j = j0 + tx;
    const float sj = (A[(int64_t)j * d + j] < 0.f) ? -1.f : 1.f;
    const float si = (A[(int64_t)i * d + i] < 0.f) ? -1.f : 1.f;
    const float rv = Q[(int64_t)i * d + j] * sj;
    R[(int64_t)i * d + j] = rv;
    U[(int64_t)i * d + j] = (j >= i) ? si * A[(int64_t)i * d + j] : 0.f;
    tile[r][tx] = rv;
  }
  if (Rt) {
    __syncthreads();
    for (int r = ty; r < 32; r += 8)   // Rt[j0 + r][i0 + tx] = R[i0 + tx][j0 + r]
      Rt[(int64_t)(j0 + r) * d + i0 + tx] = __float2bfloat16_rn(tile[tx][r]);
  }
}

// Rank test: min_k |U_kk| < eps * max_k |U_kk|  =>  DQ_ERR_SINGULAR.
__global__ void __launch_bounds__(256) diag_check_kernel(const float* __restrict__ A, int d, int* d_status) {
  __shared__ float smin[256], smax[256];
  const float* a = A + (int64_t)blockIdx.x * d * d;
  float mn = INFINITY, mx = 0.f;
  bool bad = false;
  for (int k = threadIdx.x; k < d; k += 256) {
    const float v = fabsf(a[(int64_t)k * d + k]);
    if (!isfinite(v)) bad = true;
    mn = fminf(mn, v); mx = fmaxf(mx, v);
  }
  smin[threadIdx.x] = mn; smax[threadIdx.x] = mx;
  if (bad) set_status(d_status, DQ_ERR_NONFINITE);
  __syncthreads();
  for (int off = 128; off >= 1; off >>= 1) {
    if (threadIdx.x < off) {
      smin[threadIdx.x] = fminf(smin[threadIdx.x], smin[threadIdx.x + off]);
      smax[threadIdx.x] = fmaxf(smax[threadIdx.x], smax[threadIdx.x + off]);
    }
    __syncthreads();
  }
  if (threadIdx.x == 0 && !(smin[0] > 1e-6f * smax[0])) set_status(d_status, DQ_ERR_SINGULAR);
}

int pick_ksplit(const Ctx& ctx, int n_cols, int k, int batch) {
  const int tiles = ((n_cols + 63) / 64) * batch;
  int ks = (2 * ctx.sm_count + tiles - 1) / tiles;
  const int max_by_k = (k + 255) / 256;
  if (ks > max_by_k) ks = max_by_k;
  if (ks > 32) ks = 32;
  return ks < 1 ? 1 : ks;
}

// C[rows r0.., cols cb..cb+n) <- (I - V T' V^T) C with V the panel at column c0
// (rows c0..d), T' = T^T (apply Q^T) or T (apply Q).
dq_status apply_block_reflector(Ctx& ctx, QrWorkspace& ws, float* C, int d, int batch, int c0,
                                int cb, int n, int transT) {
  const int m = d - c0;
  const int64_t dd = (int64_t)d * d;
  const int np = d / PB;
  const float* Vp = ws.V + (int64_t)c0 * d + c0;
  float* Cs = C + (int64_t)c0 * d + cb;
  // W = V^T C  (32 x n, reduction over m rows, split-K)
  GemmDesc g{};
  const int ks = pick_ksplit(ctx, n, m, batch);
  g.A = Vp; g.lda = d; g.transA = 1; g.sA = dd;
  g.B = Cs; g.ldb = d; g.transB = 0; g.sB = dd;
  g.M = PB; g.N = n; g.K = m; g.alpha = 1.f; g.beta = 0.f; g.batch = batch; g.ksplit = ks;
  if (ks == 1) {
    g.C = ws.W; g.ldc = d; g.sC = (int64_t)PB * d;
    DQ_CHECK(gemm_f32(ctx, g));
  } else {
    g.C = ws.tmp; g.ldc = d; g.sC = (int64_t)PB * d;
    DQ_CHECK(gemm_f32(ctx, g));
    DQ_CHECK(splitk_reduce(ctx, ws.tmp, ks, (int64_t)PB * d, batch, 1.f, 0.f, ws.W));
  }
  // W2 = T' W
  GemmDesc t{};
  t.A = ws.T + (int64_t)(c0 / PB) * PB * PB; t.lda = PB; t.transA = transT; t.sA = (int64_t)np * PB * PB;
  t.B = ws.W; t.ldb = d; t.transB = 0; t.sB = (int64_t)PB * d;
  t.C = ws.W2; t.ldc = d; t.sC = (int64_t)PB * d;
  t.M = PB; t.N = n; t.K = PB; t.alpha = 1.f; t.beta = 0.f; t.batch = batch;
  DQ_CHECK(gemm_f32(ctx, t));
  // C -= V W2
  GemmDesc u{};
  u.A = Vp; u.lda = d; u.transA = 0; u.sA = dd;
  u.B = ws.W2; u.ldb = d; u.transB = 0; u.sB = (int64_t)PB * d;
  u.C = Cs; u.ldc = d; u.sC = dd;
  u.M = m; u.N = n; u.K = PB; u.alpha = -1.f; u.beta = 1.f; u.batch = batch;
  return gemm_f32(ctx, u);
}

}  // namespace

// Blocked Householder factorisation only: ws.A <- raw upper factor (Algorithm 2 signs),
// ws.V / ws.T <- compact-WY reflectors.
dq_status qr_factor(Ctx& ctx, QrWorkspace& ws, const float* Z, int d, int batch) {
  if (d % PB != 0 || d > PC * PT * RPT) return DQ_ERR_UNSUPPORTED;
  const int64_t dd = (int64_t)d * d;
  DQ_CHECK_CUDA(cudaMemcpyAsync(ws.A, Z, sizeof(float) * dd * batch, cudaMemcpyDeviceToDevice, ctx.stream));
  const int np = d / PB;
  for (int p = 0; p < np; ++p) {
    const int c0 = p * PB;
    qr_panel_kernel<<<dim3(PC, batch), PT, 0, ctx.stream>>>(ws.A, ws.V, ws.T + (int64_t)p * PB * PB, d, c0,
                                                           dd, (int64_t)np * PB * PB);
    DQ_CHECK(after_launch(ctx));
    const int nt = d - c0 - PB;
    if (nt > 0) DQ_CHECK(apply_block_reflector(ctx, ws, ws.A, d, batch, c0, c0 + PB, nt, /*transT=*/1));
  }
  diag_check_kernel<<<batch, 256, 0, ctx.stream>>>(ws.A, d, ctx.d_status);
  return after_launch(ctx);
}

dq_status qr_diag_check(Ctx& ctx, const float* A, int d, int batch) {
  diag_check_kernel<<<batch, 256, 0, ctx.stream>>>(A, d, ctx.d_status);
  return after_launch(ctx);
}

dq_status qr_forward(Ctx& ctx, QrWorkspace& ws, const float* Z, float* R, float* U,
                     __nv_bfloat16* Rt_bf16, int d, int batch) {
  DQ_CHECK(qr_factor(ctx, ws, Z, d, batch));
  const int64_t dd = (int64_t)d * d;
  const int np = d / PB;
  // Q = H_1 ... H_n applied to I, last panel first; only Q[c0:, c0:] is touched.
  {
    int bx = (int)((dd + 255) / 256);
    if (bx > 2048) bx = 2048;
    set_identity_kernel<<<dim3(bx, batch), 256, 0, ctx.stream>>>(ws.Q, d);
    DQ_CHECK(after_launch(ctx));
  }
  for (int p = np - 1; p >= 0; --p) {
    const int c0 = p * PB;
    DQ_CHECK(apply_block_reflector(ctx, ws, ws.Q, d, batch, c0, c0, d - c0, /*transT=*/0));
  }
  gauge_kernel<<<dim3(d / 32, d / 32, batch), 256, 0, ctx.stream>>>(ws.Q, ws.A, R, U, Rt_bf16, d);
  return after_launch(ctx);
}

}  // namespace dq
