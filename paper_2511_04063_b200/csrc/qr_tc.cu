// QR-Orth on the tensor cores (used with the tensor-core path).
//
// Forward:  either the blocked Householder factorisation (qr_panel_tc.cu kernels with the compact-WY
//           products issued here), then W = U^-1 by recursive block inversion and R = Z W (the same
//           orthogonal factor the reflectors would give; forming it as Z U^-1 costs one GEMM instead
//           of d / 128 dependent block updates; its orthogonality error grows like cond(Z) * 2^-17);
//           or, from the second step on, incrementally from the previous step's W:
//           Zh = Z W_old, I + T = upper factor of Zh by fixed-point sweeps, R = Zh (I + T)^-1,
//           W = W_old (I + T)^-1 (qr_forward_incremental_tc).
// Backward: S = tril(R^T Gq - Gq^T R, -1), Gz = R (S W^T).
// The d x d products run as tcgen05 GEMMs clipped to the non-zero blocks of triangular operands, on
// split-bf16 operands (three bf16 MMAs per product, ~2^-17 relative error) where the result needs fp32
// accuracy and on plain bf16 operands where the product is a small correction or the data is bf16-accurate.
#include <algorithm>
#include <vector>

#include "tc_host.cuh"
#include "tc_path.cuh"

namespace dq {
namespace {

using bf16 = __nv_bfloat16;

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

// dst[b][r][c] = hi[b][r][c] + lo[b][r][c]   (fp32 value of a split pair)
__global__ void __launch_bounds__(256) combine_kernel(const bf16* __restrict__ hi, const bf16* __restrict__ lo,
                                                      float* __restrict__ dst, int64_t n) {
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
    dst[i] = __bfloat162float(hi[i]) + __bfloat162float(lo[i]);
}

// W = I in every form the incremental factorisation carries: fp32, split row-major and split transposed
// (hi = 1 on the diagonal, everything else 0).
__global__ void __launch_bounds__(256) identity_w_kernel(float* __restrict__ Wf, bf16* __restrict__ n_hi,
                                                         bf16* __restrict__ n_lo, bf16* __restrict__ t_hi,
                                                         bf16* __restrict__ t_lo, int d, int64_t n) {
  const bf16 zero = __float2bfloat16_rn(0.f), one = __float2bfloat16_rn(1.f);
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t e = i % ((int64_t)d * d);
    const bool diag = (e / d) == (e % d);
    Wf[i] = diag ? 1.f : 0.f;
    n_hi[i] = diag ? one : zero; t_hi[i] = diag ? one : zero;
    n_lo[i] = zero; t_lo[i] = zero;
  }
}

// part[block] = sum of squares of this block's share of E on and above the diagonal (off-diagonal entries
// count twice: E is symmetric and only its upper tiles are stored), in double precision, fixed order.
__global__ void __launch_bounds__(256) sym_sumsq_kernel(const float* __restrict__ E, int d, int64_t n,
                                                        double* __restrict__ part) {
  __shared__ double sm[256];
  double acc = 0.0;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t e = i % ((int64_t)d * d);
    const int r = (int)(e / d), c = (int)(e % d);
    if (c >= r) { const double v = E[i]; acc += (c > r ? 2.0 : 1.0) * v * v; }
  }
  sm[threadIdx.x] = acc;
  __syncthreads();
  for (int off = 128; off >= 1; off >>= 1) {
    if (threadIdx.x < off) sm[threadIdx.x] += sm[threadIdx.x + off];
    __syncthreads();
  }
  if (threadIdx.x == 0) part[blockIdx.x] = sm[0];
}

// Operands and results of the blocked inverse of an upper-triangular matrix (all [batch][d][d]).
struct TriInv {
  const float* src;                 // the matrix (fp32), read for its 128 x 128 diagonal blocks
  const bf16 *s_hi, *s_lo;          // its split copy (off-diagonal blocks)
  bf16 *n_hi, *n_lo;                // the inverse, row-major
  bf16 *t_hi, *t_lo;                // the inverse, transposed
  bf16 *tmp_hi, *tmp_lo;            // scratch
};

// Block column of the inverse:  W[0:k, k:k+s] = -W[0:k,0:k] U[0:k, k:k+s] W[k:k+s, k:k+s]
// for `count` independent diagonal positions `stride` elements apart (3rd tensor dimension).
dq_status merge(Ctx& ctx, const TriInv& io, int d, int k, int s, int count, int64_t stride, int64_t base) {
  // T1t[j][i] = sum_l W22^T[j][l] U12[i][l]        (s x k, dense temporary)
  Op a{io.t_hi + base + (int64_t)k * d + k, io.t_lo + base + (int64_t)k * d + k, d, stride};
  Op b{io.s_hi + base + k, io.s_lo + base + k, d, stride};
  Out t1; t1.hi = io.tmp_hi; t1.lo = io.tmp_lo; t1.ld_h = k; t1.bs_h = (int64_t)s * k;
  DQ_CHECK(gemm3(ctx, a, b, s, k, s, count, t1));
  Op w11{io.n_hi + base, io.n_lo + base, d, stride};
  Op t1o{io.tmp_hi, io.tmp_lo, k, (int64_t)s * k};
  // W12[i][j] = -sum_l W11[i][l] T1t[j][l]   -> row-major block (0, k)
  Out o12; o12.hi = io.n_hi + base + k; o12.lo = io.n_lo + base + k; o12.ld_h = d; o12.bs_h = stride; o12.alpha = -1.f;
  DQ_CHECK(gemm3(ctx, w11, t1o, k, s, k, count, o12));
  // W12^T[j][i] = -sum_l T1t[j][l] W11[i][l] -> transposed block (k, 0)
  Out o21; o21.hi = io.t_hi + base + (int64_t)k * d; o21.lo = io.t_lo + base + (int64_t)k * d; o21.ld_h = d;
  o21.bs_h = stride; o21.alpha = -1.f;
  return gemm3(ctx, t1o, w11, s, k, k, count, o21);
}

dq_status tri_inverse_tc(Ctx& ctx, const TriInv& io, int d, int batch) {
  const int64_t dd = (int64_t)d * d;
  const size_t bytes = sizeof(bf16) * (size_t)dd * batch;
  DQ_CHECK_CUDA(cudaMemsetAsync(io.n_hi, 0, bytes, ctx.stream));
  DQ_CHECK_CUDA(cudaMemsetAsync(io.n_lo, 0, bytes, ctx.stream));
  DQ_CHECK_CUDA(cudaMemsetAsync(io.t_hi, 0, bytes, ctx.stream));
  DQ_CHECK_CUDA(cudaMemsetAsync(io.t_lo, 0, bytes, ctx.stream));
  const int smem = TRI_INV_SMEM;
  static SmemOptIn attr;
  DQ_CHECK(opt_in_dynamic_smem(tri_inv_diag128_kernel, smem, attr));
  tri_inv_diag128_kernel<<<dim3(d / DB, batch), TRI_INV_THREADS, smem, ctx.stream>>>(io.src, io.n_hi, io.n_lo, io.t_hi,
                                                                                     io.t_lo, d);
  DQ_CHECK(after_launch(ctx));
  int s = DB, count = d / DB;
  while (count > 1 && count % 2 == 0) {
    const int pairs = count / 2;
    const int64_t pair_stride = (int64_t)2 * s * (d + 1);
    if (batch == 1) {
      DQ_CHECK(merge(ctx, io, d, s, s, pairs, pair_stride, 0));
    } else {
      for (int pidx = 0; pidx < pairs; ++pidx) DQ_CHECK(merge(ctx, io, d, s, s, batch, dd, pidx * pair_stride));
    }
    s *= 2; count = pairs;
  }
  for (int kb = 1; kb < count; ++kb) DQ_CHECK(merge(ctx, io, d, kb * s, s, batch, dd, 0));
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

// The two sets of copies of W = U^-1 (row-major and transposed, split): index 0 / 1.
struct WSet { bf16 *n_hi, *n_lo, *t_hi, *t_lo; };
WSet wset(const QrTcState& q, int sel) {
  // (the transposed copies exist for set 0 only: the Householder route writes and reads them there; the
  // incremental steps read W^T as a transposed operand)
  return sel == 0 ? WSet{q.wn_hi, q.wn_lo, q.wt_hi, q.wt_lo} : WSet{q.wn2_hi, q.wn2_lo, nullptr, nullptr};
}

// The upper tiles in the order made for the product's k_mode (0: all k-blocks, 2, or 1|4).
void upper_lists(Out& o, const QrTcState& q) {
  o.n_list = q.n_upper; o.n_list2 = q.n2_upper;
  if (o.k_mode == 2) { o.tile_list = q.tl_upper_k2; o.tile_list2 = q.tl2_upper_k2; }
  else if (o.k_mode == (1 | 4)) { o.tile_list = q.tl_upper_band; o.tile_list2 = q.tl2_upper_band; }
  else { o.tile_list = q.tl_upper; o.tile_list2 = q.tl2_upper; }
}

// Lays `tiles` out for `workers` persistent workers that take entries w, w + workers, ... : rounds of `workers`
// tiles in ascending cost, dealt from the heaviest round down, the heaviest tile of a round to the worker with
// the least work so far.  The last round may be partial (it falls to workers 0 .. rem - 1) and takes the heaviest
// tiles.  A worker's first tile is its lightest: its products are the ones nothing overlaps with.
template <class Cost>
std::vector<int> balanced_order(std::vector<int> tiles, int workers, Cost cost) {
  std::stable_sort(tiles.begin(), tiles.end(), [&](int a, int b) { return cost(a) > cost(b); });
  const int n = (int)tiles.size(), full = n / workers, rem = n % workers;
  std::vector<int> out(n);
  std::vector<int64_t> load(workers, 0);
  int next = 0;
  for (int w = 0; w < rem; ++w) { out[full * workers + w] = tiles[next]; load[w] += cost(tiles[next]); ++next; }
  std::vector<int> by_load(workers);
  for (int r = full - 1; r >= 0; --r) {
    for (int w = 0; w < workers; ++w) by_load[w] = w;
    std::stable_sort(by_load.begin(), by_load.end(), [&](int a, int b) { return load[a] < load[b]; });
    for (int j = 0; j < workers; ++j) {
      const int w = by_load[j];
      out[r * workers + w] = tiles[next]; load[w] += cost(tiles[next]); ++next;
    }
  }
  return out;
}

}  // namespace

dq_status qr_tc_init(QrTcState& q, int d, int batch, int sm_count) {
  const int64_t dd = (int64_t)d * d * batch;
  bf16** all[] = {&q.z_hi, &q.z_lo, &q.u_hi, &q.u_lo, &q.wn_hi, &q.wn_lo, &q.wt_hi, &q.wt_lo, &q.r_hi, &q.r_lo,
                  &q.rt_hi, &q.rt_lo, &q.gqt_hi, &q.gqt_lo, &q.st_hi, &q.st_lo, &q.m_hi, &q.m_lo, &q.t1_hi, &q.t1_lo,
                  &q.wn2_hi, &q.wn2_lo, &q.yt_hi, &q.yt_lo, &q.nm1, &q.nm2};
  for (bf16** p : all) DQ_CHECK(alloc(p, dd));
  DQ_CHECK(alloc(&q.P, dd));
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
  for (int unit = 128; unit <= 256; unit *= 2) {   // tile orders (see QrTcState)
    if (d % unit != 0) break;
    const int nb = d / unit;
    const int workers = unit == 128 ? sm_count : (sm_count / 2 > 0 ? sm_count / 2 : 1);
    std::vector<int> upper, lower, all;
    for (int j = 0; j < nb; ++j)
      for (int i = 0; i < nb; ++i) {
        if (i <= j) upper.push_back(i | (j << 16));
        if (i >= j) lower.push_back(i | (j << 16));
        all.push_back(i | (j << 16));
      }
    auto mb_of = [](int t) { return t & 0xffff; };
    auto nb_of = [](int t) { return t >> 16; };
    const std::vector<int> up_k2 = balanced_order(upper, workers, [&](int t) { return mb_of(t) + 1; });
    const std::vector<int> up_band = balanced_order(upper, workers, [&](int t) { return nb_of(t) - mb_of(t) + 1; });
    const std::vector<int> k4 = balanced_order(all, workers, [&](int t) { return nb_of(t) + 1; });
    const std::vector<int> k8 = balanced_order(all, workers, [&](int t) { return nb - nb_of(t); });
    const bool one = unit == 128;
    (one ? q.n_upper : q.n2_upper) = (int)upper.size();
    (one ? q.n_all : q.n2_all) = (int)all.size();
    auto upload = [&](int*& dst, const std::vector<int>& v) -> dq_status {
      DQ_CHECK(alloc(&dst, (int64_t)v.size()));
      DQ_CHECK_CUDA(cudaMemcpy(dst, v.data(), sizeof(int) * v.size(), cudaMemcpyHostToDevice));
      return DQ_OK;
    };
    DQ_CHECK(upload(one ? q.tl_upper : q.tl2_upper, upper));
    DQ_CHECK(upload(one ? q.tl_upper_k2 : q.tl2_upper_k2, up_k2));
    DQ_CHECK(upload(one ? q.tl_upper_band : q.tl2_upper_band, up_band));
    DQ_CHECK(upload(one ? q.tl_lower : q.tl2_lower, lower));
    DQ_CHECK(upload(one ? q.tl_k4 : q.tl2_k4, k4));
    DQ_CHECK(upload(one ? q.tl_k8 : q.tl2_k8, k8));
  }
  q.ready = true;
  return DQ_OK;
}

void qr_tc_destroy(QrTcState& q) {
  bf16* all[] = {q.z_hi, q.z_lo, q.u_hi, q.u_lo, q.wn_hi, q.wn_lo, q.wt_hi, q.wt_lo, q.r_hi, q.r_lo,
                 q.rt_hi, q.rt_lo, q.gqt_hi, q.gqt_lo, q.st_hi, q.st_lo, q.m_hi, q.m_lo, q.t1_hi, q.t1_lo,
                 q.wn2_hi, q.wn2_lo, q.yt_hi, q.yt_lo, q.nm1, q.nm2};
  for (bf16* p : all) cudaFree(p);
  cudaFree(q.P);
  cudaFree(q.y_hi); cudaFree(q.y_lo); cudaFree(q.w2_hi); cudaFree(q.w2_lo); cudaFree(q.part); cudaFree(q.T);
  cudaFree(q.tw_hi); cudaFree(q.tw_lo); cudaFree(q.tl_upper); cudaFree(q.tl_k4); cudaFree(q.tl_k8); cudaFree(q.tl_upper_k2); cudaFree(q.tl_upper_band);
  cudaFree(q.tl2_upper); cudaFree(q.tl2_k4); cudaFree(q.tl2_k8); cudaFree(q.tl2_upper_k2); cudaFree(q.tl2_upper_band); cudaFree(q.tl_lower); cudaFree(q.tl2_lower); cudaFree(q.sweep_flags);
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

// R and W = U^-1 of the latent one optimiser step after a latent whose W_old is known, without dependent
// column steps and without forming U.  Zh = Z W_old is close to orthogonal however far Z itself has drifted
// (Zh = R_old + (Z - Z_old) W_old), so its upper factor I + T is the fixed point of
//   T <- Phi(E - T^T T),  E = Zh^T Zh - I,  Phi(S) = striu(S) + diag(S) / 2.
// The iteration starts from Phi(E - P) with P = T^T T of the previous step (consecutive steps are alike), runs
// in the epilogues of the products T^T T (one launch per sweep), and stops by device flags: sweep k runs only
// if sweep k - 1 moved an entry by more than 1e-5; the launch sequence is fixed, so a captured graph replays
// it unchanged.  Then (I + T)^-1 = I + Y from the identity
//   (I + T)^-1 = (I - T)(I + T^2)(I + T^4) (I - T^8)^-1:
// two triangular products give (I - T)(I + T^2) (error |T|^4, enough after a small step), two more the factor
// (I + T^4) (error |T|^8, after a large step).  R = Zh + Zh Y and W = W_old + W_old Y.  Zh and E are split-bf16 products (three MMAs); the others act on
// terms of size |T| and use plain bf16 operands (their 2^-9 relative error is of size 2^-9 |T|) unless the
// fixed point needed a third sweep, the sign of a large step: then the first-order ones switch to split
// operands and the higher-order factor is added (a device flag selects which launches run).
// need_lo: also the lo parts of the split copies of R and R^T (read only by products on split operands).
dq_status qr_forward_incremental_tc(Ctx& ctx, QrWorkspace& ws, QrTcState& q, const float* Z, float* R, int d,
                                    int batch, int n_sweeps, bool need_lo) {
  const int64_t dd = (int64_t)d * d;
  const dim3 tiles(d / 32, d / 32, batch);
  const WSet wc = wset(q, q.w_sel), wn = wset(q, q.w_sel ^ 1);
  float *Zh = ws.A, *E = ws.B, *T = ws.tmp, *T2 = ws.S, *Y3 = ws.Q, *T4 = ws.V, *Wf = ws.Winv;
  // bf16 scratch (all free until the backward pass or owned by the Householder route).  Every matrix is kept
  // row-major only: a product that needs it transposed names it as a transposed operand (Op::t) and the tensor
  // cores read its tiles MN-major.
  bf16 *zh_hi = q.m_hi, *zh_lo = q.m_lo;
  bf16 *ta_hi = q.tw_hi, *ta_lo = q.tw_lo, *tb_hi = q.t1_hi, *tb_lo = q.t1_lo;   // T, alternating between sweeps
  bf16 *t_hi = q.u_hi, *t_lo = q.u_lo;                                           // T of the last sweep that ran
  bf16 *t2_hi = q.gqt_hi, *y3_hi = q.nm1, *t4_hi = q.nm2;
  bf16 *y_hi = q.yt_hi, *y_lo = q.yt_lo;                                         // Y = (I + T)^-1 - I
  q.u_fresh = false;
  if (!q.z_split_fresh) {   // (the SGD update writes the split copy with the new latent)
    split_kernel<<<tiles, 256, 0, ctx.stream>>>(Z, q.z_hi, q.z_lo, d, 0);
    DQ_CHECK(after_launch(ctx));
    q.z_split_fresh = true;
  }
  {   // Zh[i][j] = sum_k Z[i][k] W_old[k][j]  (W upper triangular: k <= j); B = W^T
    Op a{q.z_hi, q.z_lo, d, dd}, b{wc.n_hi, wc.n_lo, d, dd, true};
    Out o; o.f32 = Zh; o.ld = d; o.bs = dd; o.hi = zh_hi; o.lo = zh_lo; o.ld_h = d; o.bs_h = dd;
    o.k_mode = 4; o.tile_list = q.tl_k4; o.n_list = q.n_all; o.tile_list2 = q.tl2_k4; o.n_list2 = q.n2_all;
    DQ_CHECK(gemm3(ctx, a, b, d, d, d, batch, o));
  }
  const int n_total = n_sweeps + 3;
  int* flags = q.sweep_flags;      // flags[k] = 1: sweep k moved an entry
  DQ_CHECK_CUDA(cudaMemsetAsync(flags, 0, sizeof(int) * (n_total + 2), ctx.stream));
  {   // E = Zh^T Zh - I on the upper tiles, and the start of the fixed point T = Phi(E - P_old)
    Op a{zh_hi, zh_lo, d, dd, true};   // both operands are Zh^T
    // (the first sweep always follows and reads only the hi part of T)
    Out o; o.f32 = E; o.ld = d; o.bs = dd; o.add1 = q.P; o.aux = T; o.gen_mode = tc::GEN_CHOL_FIRST;
    o.hi = ta_hi; o.ld_h = d; o.bs_h = dd;
    upper_lists(o, q);
    DQ_CHECK(gemm3(ctx, a, a, d, d, d, batch, o));
  }
  for (int k = 1; k <= n_total; ++k) {
    // P[i][j] = sum_l T[l][i] T[l][j] (both operands T^T, lower triangular: l < 128 (mb + 1), mb <= nb), then
    // T <- Phi(E - P) in the epilogue.  The bf16 copy of T that the sweeps read alternates between two buffers,
    // because the epilogue of one tile rewrites what the main loop of another still reads.
    const bool odd = k & 1;
    Op tt{odd ? ta_hi : tb_hi, odd ? ta_lo : tb_lo, d, dd, true};
    Out o; o.f32 = q.P; o.ld = d; o.bs = dd; o.add1 = E; o.aux = T; o.gen_mode = tc::GEN_CHOL_SWEEP;
    o.tol = 1e-5f; o.moved_out = flags + k; o.fail_if_moved = (k == n_total) ? 1 : 0;
    // T for the next sweep (its lo part only if that sweep uses split operands), and the copy the later products
    // read, which every sweep that runs must leave behind (which one is the last is not known here)
    o.hi = odd ? tb_hi : ta_hi; o.lo = (k + 1 > 2) ? (odd ? tb_lo : ta_lo) : nullptr;
    o.hi2 = t_hi; o.lo2 = t_lo; o.ld_h = d; o.bs_h = dd;
    o.k_mode = 2; upper_lists(o, q);
    o.nterms = (k <= 2) ? 1 : 3;
    o.run_if = (k == 1) ? nullptr : flags + k - 1;
    DQ_CHECK(gemm3(ctx, tt, tt, d, d, d, batch, o));
  }
  const int* big = flags + 2;     // a third sweep ran: a large step, first-order products with split operands
  Op t{t_hi, t_lo, d, dd}, t_tr{t_hi, t_lo, d, dd, true};
  for (int v = 0; v < 2; ++v) {   // T2 = T T  (upper x upper: k in [128 mb, 128 (nb + 1)))
    Out o; o.f32 = T2; o.ld = d; o.bs = dd; o.hi = t2_hi; o.ld_h = d; o.bs_h = dd;
    o.k_mode = 1 | 4; upper_lists(o, q);
    o.nterms = v ? 3 : 1; (v ? o.run_if : o.run_unless) = big;
    DQ_CHECK(gemm3(ctx, t, t_tr, d, d, d, batch, o));
  }
  Op t2{t2_hi, t2_hi, d, dd}, t2_tr{t2_hi, t2_hi, d, dd, true};
  {   // Y3 = -T + T2 - T T2 = (I - T)(I + T2) - I: all of Y after a small step (error |T|^4).  Its split copy is
      // the Y the last two products read; a second hi copy is the operand of the large-step correction below,
      // which rewrites Y.
    Out o; o.f32 = Y3; o.ld = d; o.bs = dd; o.alpha = -1.f; o.add1 = T2; o.g1 = 1.f; o.add2 = T; o.g2 = -1.f;
    o.hi = y_hi; o.lo = y_lo; o.hi2 = y3_hi; o.ld_h = d; o.bs_h = dd;
    o.k_mode = 1 | 4; upper_lists(o, q); o.nterms = 1;
    DQ_CHECK(gemm3(ctx, t, t2_tr, d, d, d, batch, o));
  }
  {   // after a large step also the factor (I + T^4):  T4 = T2 T2
    Out o; o.f32 = T4; o.ld = d; o.bs = dd; o.hi = t4_hi; o.ld_h = d; o.bs_h = dd; o.k_mode = 1 | 4; upper_lists(o, q);
    o.nterms = 1; o.run_if = big;
    DQ_CHECK(gemm3(ctx, t2, t2_tr, d, d, d, batch, o));
  }
  {   // Y = Y3 + T4 + Y3 T4 = (I + Y3)(I + T4) - I; only its split copy is kept
    Op a{y3_hi, y3_hi, d, dd}, b{t4_hi, t4_hi, d, dd, true};
    Out o; o.ld = d; o.bs = dd; o.add1 = Y3; o.add2 = T4; o.hi = y_hi; o.lo = y_lo; o.ld_h = d; o.bs_h = dd;
    o.k_mode = 1 | 4; upper_lists(o, q); o.nterms = 1; o.run_if = big;
    DQ_CHECK(gemm3(ctx, a, b, d, d, d, batch, o));
  }
  Op y_tr{y_hi, y_lo, d, dd, true};
  for (int v = 0; v < 2; ++v) {   // R = Zh + Zh Y  (Y upper triangular: k <= j)
    Op a{zh_hi, zh_lo, d, dd};
    // the only bf16 copy of R is R^T (operand of O = X R; the backward reads R from it as a transposed operand)
    Out o; o.f32 = R; o.ld = d; o.bs = dd; o.add1 = Zh;
    o.t_hi = q.rt_hi; o.t_lo = need_lo ? q.rt_lo : nullptr; o.ld_t = d; o.bs_t = dd;
    o.k_mode = 4; o.tile_list = q.tl_k4; o.n_list = q.n_all; o.tile_list2 = q.tl2_k4; o.n_list2 = q.n2_all;
    o.nterms = v ? 3 : 1; (v ? o.run_if : o.run_unless) = big;
    DQ_CHECK(gemm3(ctx, a, y_tr, d, d, d, batch, o));
  }
  for (int v = 0; v < 2; ++v) {   // W = W_old + W_old Y into the other set of copies (the fp32 W in place)
    Op a{wc.n_hi, wc.n_lo, d, dd};
    Out o; o.f32 = Wf; o.ld = d; o.bs = dd; o.add1 = Wf; o.hi = wn.n_hi; o.lo = wn.n_lo; o.ld_h = d; o.bs_h = dd;
    o.k_mode = 1 | 4; upper_lists(o, q);
    o.nterms = v ? 3 : 1; (v ? o.run_if : o.run_unless) = big;
    DQ_CHECK(gemm3(ctx, a, y_tr, d, d, d, batch, o));
  }
  q.w_sel ^= 1;
  // diag(W) = 1 / diag(U): the same rank and finiteness test (beside the next kernel: only the update waits for it)
  return on_side(ctx, [&](Ctx& c) { return qr_diag_check(c, Wf, d, batch); });
}

dq_status qr_forward_fast(Ctx& ctx, QrWorkspace& ws, QrTcState& q, const float* Z, float* R, float* U, int d,
                          int batch, int iterative_iters, bool need_lo) {
  if (d % 128 != 0) return DQ_ERR_UNSUPPORTED;
  const int64_t dd = (int64_t)d * d;
  const dim3 tiles(d / 32, d / 32, batch);
  if (iterative_iters > 0 && q.t_warm)
    return qr_forward_incremental_tc(ctx, ws, q, Z, R, d, batch, iterative_iters, need_lo);
  // no factors of a nearby latent yet (first call, latent replaced), or Householder at every step
  DQ_CHECK(qr_factor_tc(ctx, ws, q, Z, d, batch));
  DQ_CHECK(qrp_gauge_ut(ctx, ws.A, U, q.u_hi, q.u_lo, d, batch));
  q.u_fresh = true;
  q.w_sel = 0;
  const WSet w = wset(q, 0);
  const TriInv io{U, q.u_hi, q.u_lo, w.n_hi, w.n_lo, w.t_hi, w.t_lo, q.t1_hi, q.t1_lo};
  DQ_CHECK(tri_inverse_tc(ctx, io, d, batch));
  if (iterative_iters > 0) {   // state the incremental steps continue from: W in fp32, no T^T T yet
    combine_kernel<<<ctx.sm_count * 8, 256, 0, ctx.stream>>>(w.n_hi, w.n_lo, ws.Winv, dd * batch);
    DQ_CHECK(after_launch(ctx));
    DQ_CHECK_CUDA(cudaMemsetAsync(q.P, 0, sizeof(float) * (size_t)dd * batch, ctx.stream));
    q.t_warm = true;
  }
  if (!q.z_split_fresh) {
    split_kernel<<<tiles, 256, 0, ctx.stream>>>(Z, q.z_hi, q.z_lo, d, 0);
    DQ_CHECK(after_launch(ctx));
    q.z_split_fresh = true;
  }
  // R[i][j] = sum_k Z[i][k] W[k][j]:  A = Z (row-major), B = W^T; also the split copies of R and R^T
  Op a{q.z_hi, q.z_lo, d, dd};
  Op b{w.t_hi, w.t_lo, d, dd};
  Out o; o.f32 = R; o.ld = d; o.bs = dd; o.hi = q.r_hi; o.lo = q.r_lo; o.ld_h = d; o.bs_h = dd;
  o.t_hi = q.rt_hi; o.t_lo = q.rt_lo; o.ld_t = d; o.bs_t = dd;
  o.k_mode = 4;   // W is upper triangular: W^T[j][k] = 0 for k > j
  o.tile_list = q.tl_k4; o.n_list = q.n_all; o.tile_list2 = q.tl2_k4; o.n_list2 = q.n2_all;
  return gemm3(ctx, a, b, d, d, d, batch, o);
}

// A latent that is orthogonal to begin with (the paper's initialisation is a random Hadamard matrix) has
// U = I: the incremental steps can start from W = I without a Householder factorisation.  Measures
// |Z^T Z - I|_F (one split-bf16 product on the upper tiles and a reduction; synchronises the stream) and, if
// it is at most `threshold` for every problem, installs W = I as the previous step's factor.
dq_status qr_tc_try_orthogonal_start(Ctx& ctx, QrWorkspace& ws, QrTcState& q, const float* Z, int d, int batch,
                                     float threshold, bool* started) {
  *started = false;
  const int64_t dd = (int64_t)d * d;
  DQ_CHECK(qrp_transpose_split(ctx, Z, ws.A, q.st_hi, q.st_lo, d, batch));
  {   // E = Z^T Z - I on the upper tiles
    Op a{q.st_hi, q.st_lo, d, dd};
    Out o; o.f32 = ws.B; o.ld = d; o.bs = dd; o.gen_mode = tc::GEN_CHOL_FIRST; o.aux = ws.tmp;
    upper_lists(o, q);
    DQ_CHECK(gemm3(ctx, a, a, d, d, d, batch, o));
  }
  constexpr int BLOCKS = 256;
  double* d_part = reinterpret_cast<double*>(ws.S);       // scratch: [batch][BLOCKS] doubles
  for (int b = 0; b < batch; ++b) {
    sym_sumsq_kernel<<<BLOCKS, 256, 0, ctx.stream>>>(ws.B + b * dd, d, dd, d_part + (int64_t)b * BLOCKS);
    DQ_CHECK(after_launch(ctx));
  }
  std::vector<double> part((size_t)batch * BLOCKS);
  DQ_CHECK_CUDA(cudaMemcpyAsync(part.data(), d_part, sizeof(double) * part.size(), cudaMemcpyDeviceToHost, ctx.stream));
  DQ_CHECK_CUDA(cudaStreamSynchronize(ctx.stream));
  for (int b = 0; b < batch; ++b) {
    double s = 0.0;
    for (int i = 0; i < BLOCKS; ++i) s += part[(size_t)b * BLOCKS + i];
    if (!(s <= (double)threshold * threshold)) return DQ_OK;   // (also catches NaN)
  }
  q.w_sel = 0;
  const WSet w = wset(q, 0);
  identity_w_kernel<<<ctx.sm_count * 8, 256, 0, ctx.stream>>>(ws.Winv, w.n_hi, w.n_lo, w.t_hi, w.t_lo, d, dd * batch);
  DQ_CHECK(after_launch(ctx));
  DQ_CHECK_CUDA(cudaMemsetAsync(q.P, 0, sizeof(float) * (size_t)dd * batch, ctx.stream));
  q.t_warm = true;
  q.u_fresh = false;
  *started = true;
  return DQ_OK;
}

// One dense d x d x d product of the kind QR-Orth is made of (split-bf16 operands, nterms = 3, or plain bf16,
// nterms = 1) on the handle's operand copies of Z and W^T, result to scratch: for measurement.
dq_status qr_tc_bench_product(Ctx& ctx, QrWorkspace& ws, QrTcState& q, int d, int batch, int nterms) {
  const int64_t dd = (int64_t)d * d;
  const WSet w = wset(q, q.w_sel);
  Op a{q.z_hi, q.z_lo, d, dd}, b{w.n_hi, w.n_lo, d, dd, true};
  Out o; o.f32 = ws.Q; o.ld = d; o.bs = dd; o.nterms = nterms;
  return gemm3(ctx, a, b, d, d, d, batch, o);
}

// U of the current factorisation for inspection: the Householder route leaves it in place; the incremental
// route carries only W = U^-1, which is inverted here (split-bf16 accuracy, about 1e-5 relative).
dq_status qr_tc_materialize_u(Ctx& ctx, QrWorkspace& ws, QrTcState& q, float* U, int d, int batch) {
  if (q.u_fresh) return DQ_OK;
  const WSet w = wset(q, q.w_sel);
  const TriInv io{ws.Winv, w.n_hi, w.n_lo, q.u_hi, q.u_lo, q.st_hi, q.st_lo, q.t1_hi, q.t1_lo};
  DQ_CHECK(tri_inverse_tc(ctx, io, d, batch));
  combine_kernel<<<ctx.sm_count * 8, 256, 0, ctx.stream>>>(q.u_hi, q.u_lo, U, (int64_t)d * d * batch);
  DQ_CHECK(after_launch(ctx));
  q.u_fresh = true;
  return DQ_OK;
}

// Gz = R tril(R^T Gq - Gq^T R, -1) W^T.  Gq carries the bf16 rounding of the rotation operand and of dL/dO
// (a few percent relative), so with split == false every product runs on plain bf16 operands (2^-9):
//   S = tril(B - B^T, -1) as ONE reduction over two operand pairs, (R^T, Gq^T) minus (Gq^T, R^T), on the tiles
//   on and below the block diagonal;  D^T = W S^T (triangular x triangular);  Gz = R D.
// split == true keeps three MMAs per product (B in fp32, then the skew part by an element-wise kernel).
dq_status qr_backward_tc(Ctx& ctx, QrWorkspace& ws, QrTcState& q, const float* Gq, float* Gz, int d, int batch,
                         bool split) {
  const int64_t dd = (int64_t)d * d;
  const dim3 tiles(d / 32, d / 32, batch);
  const WSet w = wset(q, q.w_sel);
  if (split || !q.gqt_fresh) {   // (else the contraction that produced Gq already stored bf16(Gq^T))
    split_kernel<<<tiles, 256, 0, ctx.stream>>>(Gq, q.gqt_hi, q.gqt_lo, d, 1);
    DQ_CHECK(after_launch(ctx));
  }
  q.gqt_fresh = false;
  Op rt{q.rt_hi, q.rt_lo, d, dd}, gqt{q.gqt_hi, q.gqt_lo, d, dd};
  if (split) {
    // B[i][j] = sum_k R[k][i] Gq[k][j]:  A = R^T, B-operand = Gq^T
    Out ob; ob.f32 = ws.B; ob.ld = d; ob.bs = dd;
    DQ_CHECK(gemm3(ctx, rt, gqt, d, d, d, batch, ob));
    skew_split_kernel<<<tiles, 256, 0, ctx.stream>>>(ws.B, q.st_hi, q.st_lo, d);
    DQ_CHECK(after_launch(ctx));
  } else {
    // S[i][j] = sum_k R^T[i][k] Gq^T[j][k] - sum_k Gq^T[i][k] R^T[j][k], kept for i > j
    Out os; os.hi = q.st_hi; os.ld_h = d; os.bs_h = dd; os.gen_mode = tc::GEN_STRICT_LOWER; os.nterms = 1;
    os.dual_a = &gqt; os.dual_b = &rt;
    os.tile_list = q.tl_lower; os.n_list = q.n_upper; os.tile_list2 = q.tl2_lower; os.n_list2 = q.n2_upper;
    DQ_CHECK(gemm3(ctx, rt, gqt, d, d, d, batch, os));
  }
  // Gz = R S W^T = R D with D = S W^T lower triangular.  D^T[m][n] = sum_k W[m][k] S[n][k]: W[m][k] = 0 for
  // k < m and S[n][k] = 0 for k >= n, so only tiles mb <= nb with k in [128 mb, 128 (nb + 1)): a sixth of a
  // dense product (R S first would cost half of one).  Only the split copy of D^T is kept.
  Op wnr{w.n_hi, w.n_lo, d, dd}, sr{q.st_hi, q.st_lo, d, dd};
  Out od; od.hi = q.m_hi; od.lo = split ? q.m_lo : nullptr; od.ld_h = d; od.bs_h = dd;
  od.k_mode = 1 | 4; upper_lists(od, q); od.nterms = split ? 3 : 1;
  DQ_CHECK(gemm3(ctx, wnr, sr, d, d, d, batch, od));
  // (tiles below the block diagonal of D^T are neither written here nor read by the next product; the entries
  // below the diagonal inside the diagonal tiles come out as exact zeros)
  // Gz[i][j] = sum_k R[i][k] D^T[j][k]; D^T[j][k] = 0 for k < j
  Op r{q.rt_hi, q.rt_lo, d, dd, true}, dt{q.m_hi, q.m_lo, d, dd};   // R = (R^T)^T
  Out og; og.f32 = Gz; og.ld = d; og.bs = dd;
  og.k_mode = 8; og.nterms = split ? 3 : 1;
  og.tile_list = q.tl_k8; og.n_list = q.n_all; og.tile_list2 = q.tl2_k8; og.n_list2 = q.n2_all;
  return gemm3(ctx, r, dt, d, d, d, batch, og);
}

}  // namespace dq
