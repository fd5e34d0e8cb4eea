// Blocked Householder factorisation (Algorithm 2 in compact-WY form) with the
// trailing updates on the tensor cores.
//
// The working matrix is kept TRANSPOSED (At[c][r] = A[r][c]) so that columns are
// contiguous: panel loads are coalesced and both tensor-core products of the
// trailing update contract over a contiguous index.
//
// Per outer block of 128 columns [c0, c0 + 128), rows [c0, d) (m rows):
//   1. qr_panel_cm_kernel   one thread-block cluster; four inner panels of 32
//                           columns, each held in registers (two rows per thread),
//                           earlier inner panels applied left-looking; writes U / V
//                           into At and the split-bf16 reflector block Y (both
//                           orientations).
//   2. tensor-core GEMM     [S; W^T] = [Y C]^T Y   (split over the m rows)
//   3. wy_w2_kernel         W2 with Q^T C = C - Y W2: block forward substitution over the four
//                           inner block reflectors (T_k from the panel, S_kl = V_k^T V_l), fp32
//   4. tensor-core GEMM     C^T -= W2^T Y^T       (fp32 result + split-bf16 copy)
// Exchanges inside the cluster are pushes into every CTA's shared memory followed
// by one cluster barrier; all sums run in a fixed order (bit-reproducible).
#include <cooperative_groups.h>

#include "common.cuh"
#include "mma_tf32.cuh"
#include "tc_path.cuh"

namespace cg = cooperative_groups;

namespace dq {
namespace {

using bf16 = __nv_bfloat16;

constexpr int IB = 32;     // inner panel width
constexpr int OB = 128;    // outer block width
constexpr int MAX_CS = 16; // CTAs per cluster (8 is the portable limit; 16 where the device allows it)

__device__ __forceinline__ uint32_t pack2(bf16 a, bf16 b) {
  return (uint32_t)__bfloat16_as_ushort(a) | ((uint32_t)__bfloat16_as_ushort(b) << 16);
}

// Store a float at the same shared-memory offset in CTA `rank` of this cluster.
__device__ __forceinline__ void st_dsmem(float* local, int rank, float v) {
  const uint32_t addr = (uint32_t)__cvta_generic_to_shared(local);
  uint32_t remote;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(addr), "r"(rank));
  asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(remote), "f"(v) : "memory");
}

// At[c][r] = Z[r][c] (fp32) plus its split-bf16 copy; 32 x 32 tiles.
__global__ void __launch_bounds__(256) transpose_split_kernel(const float* __restrict__ Z, float* __restrict__ At,
                                                              bf16* __restrict__ hi, bf16* __restrict__ lo, int d) {
  __shared__ float t[32][33];
  const int64_t off = (int64_t)blockIdx.z * d * d;
  Z += off; At += off; hi += off; lo += off;
  const int r0 = blockIdx.y * 32, c0 = blockIdx.x * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  for (int r = ty; r < 32; r += 8) t[r][tx] = Z[(int64_t)(r0 + r) * d + c0 + tx];
  __syncthreads();
  for (int c = ty; c < 32; c += 8) {
    const int64_t i = (int64_t)(c0 + c) * d + r0 + tx;
    const float v = t[tx][c];
    At[i] = v;
    split2(v, hi[i], lo[i]);
  }
}

// Shared-memory carve-up of the panel kernel (floats).
template <int NW>
struct PanelSmem {
  static constexpr int RED = 0;                          // [NW][32] warp partials of a column step
  static constexpr int XCH = RED + NW * 32;              // [2][MAX_CS][32] per-CTA partials (pushed)
  static constexpr int DIAG = XCH + 2 * MAX_CS * 32;     // [2][32] the diagonal row (pushed)
  static constexpr int DLOC = DIAG + 64;                 // [32] owner's staging of the diagonal row
  static constexpr int COEF = DLOC + 32;                 // [NW][32]
  static constexpr int ZS = COEF + NW * 32;              // [32][33] V^T v_j of the inner panel
  static constexpr int TAU = ZS + 32 * 33;               // [32]
  static constexpr int TS = TAU + 32;                    // [4][32][33] T of each inner panel
  static constexpr int WP = TS + 4 * 32 * 33;            // [NW][32][32] per-warp partials of V_k^T P
  static constexpr int WX = WP + NW * 1024;              // [MAX_CS][1024] per-CTA partials (pushed)
  static constexpr int WF = WX + MAX_CS * 1024;          // [32][32] V_k^T P
  static constexpr int W2 = WF + 1024;                   // [32][32] T_k^T V_k^T P
  static constexpr int STG = W2 + 1024;                  // [NW][2][32][STG_LD] staging of V_k / P rows for the warp MMAs
  static constexpr int TOTAL = STG + (NW == 8 ? NW * 2 * 32 * 40 : 0);
  static constexpr int BYTES = TOTAL * 4;
};


// Entries of eight consecutive reflectors (columns cp0.. of inner panel k, diagonal rows dg0..)
// for this thread's two rows: stored value below the diagonal, 1 on it, 0 above.
__device__ __forceinline__ void load_v8(float (&vv)[8][2], const float* Vk, int d, int dg0, int cp0,
                                        const int (&rowi)[2], int m) {
#pragma unroll
  for (int u = 0; u < 8; ++u) {
    const float* vcol = Vk + (int64_t)(cp0 + u) * d;
#pragma unroll
    for (int s = 0; s < 2; ++s)
      vv[u][s] = (rowi[s] > dg0 + u) ? ((rowi[s] < m) ? vcol[rowi[s]] : 0.f) : ((rowi[s] == dg0 + u) ? 1.f : 0.f);
  }
}

constexpr int STG_LD = 40;   // row stride of the staging tiles: fragment loads hit 32 distinct banks

using mma::split_tf32;
using mma::mma_tf32;

// Warp partial of W = V_k^T P over this warp's 64 rows (two 32-row groups, lane = row) on the
// tensor cores: rows are staged in shared memory, fragments of A = V_k^T (M = reflector, K = row) and
// B = P (K = row, N = panel column) are read back in the warp-MMA layout, products in 3 x tf32.
// Result: Wp[cp][p] for this warp.
__device__ __forceinline__ void warp_vtp_mma(const float (&a)[2][32], const float* Vk, int d, int dg0,
                                             const int (&rowi)[2], int m, float* Vs, float* Ps, float* Wp_warp,
                                             int lane) {
  const int g = lane >> 2, t = lane & 3;
  float acc[2][4][4];
#pragma unroll
  for (int mt = 0; mt < 2; ++mt)
#pragma unroll
    for (int nt = 0; nt < 4; ++nt)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[mt][nt][e] = 0.f;
#pragma unroll
  for (int s = 0; s < 2; ++s) {   // unrolled: a[s][.] must stay in registers
    float v[32];
#pragma unroll
    for (int cp = 0; cp < 32; ++cp)
      v[cp] = (rowi[s] > dg0 + cp) ? ((rowi[s] < m) ? Vk[(int64_t)cp * d + rowi[s]] : 0.f)
                                   : ((rowi[s] == dg0 + cp) ? 1.f : 0.f);
    __syncwarp();
#pragma unroll
    for (int cp = 0; cp < 32; ++cp) {
      Vs[lane * STG_LD + cp] = v[cp];
      Ps[lane * STG_LD + cp] = a[s][cp];
    }
    __syncwarp();
#pragma unroll 1
    for (int kt = 0; kt < 4; ++kt) {
      uint32_t bh[4][2], bl[4][2];
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) {
        split_tf32(Ps[(8 * kt + t) * STG_LD + 8 * nt + g], bh[nt][0], bl[nt][0]);
        split_tf32(Ps[(8 * kt + t + 4) * STG_LD + 8 * nt + g], bh[nt][1], bl[nt][1]);
      }
#pragma unroll
      for (int mt = 0; mt < 2; ++mt) {
        uint32_t ah[4], al[4];
        split_tf32(Vs[(8 * kt + t) * STG_LD + 16 * mt + g], ah[0], al[0]);
        split_tf32(Vs[(8 * kt + t) * STG_LD + 16 * mt + g + 8], ah[1], al[1]);
        split_tf32(Vs[(8 * kt + t + 4) * STG_LD + 16 * mt + g], ah[2], al[2]);
        split_tf32(Vs[(8 * kt + t + 4) * STG_LD + 16 * mt + g + 8], ah[3], al[3]);
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
          mma_tf32(acc[mt][nt], al, bh[nt]);
          mma_tf32(acc[mt][nt], ah, bl[nt]);
          mma_tf32(acc[mt][nt], ah, bh[nt]);
        }
      }
    }
  }
#pragma unroll
  for (int mt = 0; mt < 2; ++mt)
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) {
      float* o = Wp_warp + (16 * mt + g) * 32 + 8 * nt + 2 * t;
      o[0] = acc[mt][nt][0]; o[1] = acc[mt][nt][1];
      o[8 * 32] = acc[mt][nt][2]; o[8 * 32 + 1] = acc[mt][nt][3];
    }
}

struct PanelCtx {
  float *red, *xch, *diag, *dloc, *coefs, *Zs, *taus;
  int CS, cta, warp, lane, own_cta, own_warp, NW;
};

// One Householder column step.  R = register index of the current column (position 0);
// position p lives in register (R + p) mod 32.  idg = row of the diagonal (relative to the
// outer block), j = column index inside the inner panel.
template <int R>
__device__ __forceinline__ void col_step(float (&a)[2][32], const int (&rowi)[2], int idg, int j,
                                         const PanelCtx& c) {
  const int par = j & 1, lane = c.lane, warp = c.warp;
  float acc[32];
  {
    const float x0 = (rowi[0] >= idg) ? a[0][R] : 0.f;
    const float x1 = (rowi[1] >= idg) ? a[1][R] : 0.f;
#pragma unroll
    for (int p = 0; p < 32; ++p) acc[p] = fmaf(x1, a[1][(R + p) & 31], x0 * a[0][(R + p) & 31]);
  }
  const float tot = warp_transpose_reduce32(acc, lane);
  c.red[warp * 32 + lane] = tot;
  if (c.cta == c.own_cta && warp == c.own_warp && lane == j) {   // this thread holds the diagonal row
#pragma unroll
    for (int p = 0; p < 32; ++p) c.dloc[p] = a[0][(R + p) & 31];
  }
  __syncthreads();
  if (warp == 0) {
    float s = 0.f;
    for (int w = 0; w < c.NW; ++w) s += c.red[w * 32 + lane];
    if (c.CS > 1) {
      for (int rk = 0; rk < c.CS; ++rk) st_dsmem(&c.xch[(par * MAX_CS + c.cta) * 32 + lane], rk, s);
      if (c.cta == c.own_cta) {
        const float dv = c.dloc[lane];
        for (int rk = 0; rk < c.CS; ++rk) st_dsmem(&c.diag[par * 32 + lane], rk, dv);
      }
    } else {
      c.xch[par * MAX_CS * 32 + lane] = s;
      c.diag[par * 32 + lane] = c.dloc[lane];
    }
  }
  if (c.CS > 1) cg::this_cluster().sync(); else __syncthreads();
  float g = 0.f;
  for (int rk = 0; rk < c.CS; ++rk) g += c.xch[(par * MAX_CS + rk) * 32 + lane];
  const float dr = c.diag[par * 32 + lane];
  const float alpha = __shfl_sync(0xffffffffu, dr, 0);
  const float nrm2 = __shfl_sync(0xffffffffu, g, 0);
  const float sigma = nrm2 - alpha * alpha;          // squared norm below the diagonal
  const bool skip = !(sigma > 0.f);                  // nothing to annihilate: H_j = I
  const float beta = skip ? alpha : -copysignf(__fsqrt_rn(nrm2), alpha);
  const float denom = alpha - beta;
  const float inv_denom = skip ? 0.f : __frcp_rn(denom);
  const float tau = skip ? 0.f : -denom * __frcp_rn(beta);
  const float w = fmaf(g - alpha * dr, inv_denom, dr);   // v_j^T (column at this position)
  const int npos = 32 - j;                            // positions >= npos hold finished reflectors
  c.coefs[warp * 32 + lane] = (lane >= 1 && lane < npos) ? tau * w : 0.f;
  if (warp == 0) {
    if (lane >= npos) c.Zs[(lane - npos) * 33 + j] = w;   // v_c^T v_j for c < j
    if (lane == 0) c.taus[j] = tau;
  }
  __syncwarp();
  const float4* cf = reinterpret_cast<const float4*>(c.coefs + warp * 32);
#pragma unroll
  for (int s = 0; s < 2; ++s) {
    const bool on = rowi[s] == idg, below = rowi[s] > idg;
    const float scaled = a[s][R] * inv_denom;
    const float v = on ? 1.f : (below ? scaled : 0.f);
    const float newc = on ? beta : (below ? scaled : a[s][R]);
#pragma unroll
    for (int q4 = 0; q4 < 8; ++q4) {
      const float4 c4 = cf[q4];
      a[s][(R + 4 * q4 + 0) & 31] = fmaf(-v, c4.x, a[s][(R + 4 * q4 + 0) & 31]);
      a[s][(R + 4 * q4 + 1) & 31] = fmaf(-v, c4.y, a[s][(R + 4 * q4 + 1) & 31]);
      a[s][(R + 4 * q4 + 2) & 31] = fmaf(-v, c4.z, a[s][(R + 4 * q4 + 2) & 31]);
      a[s][(R + 4 * q4 + 3) & 31] = fmaf(-v, c4.w, a[s][(R + 4 * q4 + 3) & 31]);
    }
    a[s][R] = newc;   // the finished column stays put: it is position 31 of the next step
  }
  __syncwarp();   // coefs[warp] is rewritten in the next step
}

// Factor columns [c0, c0 + 128) of A (rows c0..d) held transposed in At.
//   At   <- U on and above the diagonal, Householder vectors (unit diagonal implied) below
//   yt   <- split-bf16 Y^T: rows c0..c0+127 of (at_hi, at_lo), entries r >= c0
//   y    <- split-bf16 Y:   [d][128] row-major, rows r >= c0
// Reflector j: H = I - tau v v^T, v = (x - beta e1) / (x_1 - beta), beta = -sign(x_1) ||x||
// (Algorithm 2's sign rule), tau = (beta - x_1) / beta.
template <int NT>
__global__ void __launch_bounds__(NT, 1)
qr_panel_cm_kernel(float* At, bf16* at_hi, bf16* at_lo, bf16* y_hi, bf16* y_lo, float* Tk, int d, int c0) {
  constexpr int NW = NT / 32;
  using L = PanelSmem<NW>;
  cg::cluster_group cluster = cg::this_cluster();
  const int CS = (int)cluster.num_blocks();
  const int cta = (int)cluster.block_rank();
  {
    const int64_t dd = (int64_t)d * d, boff = (int64_t)blockIdx.y;
    At += boff * dd; at_hi += boff * dd; at_lo += boff * dd;
    y_hi += boff * (int64_t)d * OB; y_lo += boff * (int64_t)d * OB;
    Tk += boff * OB * IB;
  }
  extern __shared__ float sm[];
  float* red = sm + L::RED;
  float* xch = sm + L::XCH;
  float* diag = sm + L::DIAG;
  float* dloc = sm + L::DLOC;
  float* coefs = sm + L::COEF;
  float* Zs = sm + L::ZS;
  float* taus = sm + L::TAU;
  float* Ts = sm + L::TS;
  float* Wp = sm + L::WP;
  float* wx = sm + L::WX;
  float* Wf = sm + L::WF;
  float* W2s = sm + L::W2;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int m = d - c0;
  int rowi[2];
#pragma unroll
  for (int s = 0; s < 2; ++s) rowi[s] = ((s * NW + warp) * CS + cta) * 32 + lane;   // 32-row groups dealt round-robin
  float a[2][32];

#pragma unroll 1
  for (int ip = 0; ip < OB / IB; ++ip) {
    const int cb = c0 + ip * IB;
    // ---- load the 32 columns of this inner panel (all rows c0..d)
#pragma unroll
    for (int s = 0; s < 2; ++s) {
#pragma unroll
      for (int c = 0; c < 32; ++c)
        a[s][c] = (rowi[s] < m) ? At[(int64_t)(cb + c) * d + c0 + rowi[s]] : 0.f;
    }
    // ---- left-looking: apply the block reflectors of the earlier inner panels
#pragma unroll 1
    for (int k = 0; k < ip; ++k) {
      const float* Vk = At + (int64_t)(c0 + k * IB) * d + c0;
      if constexpr (NW == 8) {   // 255 registers per thread: room for the MMA fragments
        float* stg = sm + L::STG + warp * (2 * 32 * STG_LD);
        warp_vtp_mma(a, Vk, d, k * IB, rowi, m, stg, stg + 32 * STG_LD, Wp + warp * 1024, lane);
      } else {
#pragma unroll 1
        for (int cp0 = 0; cp0 < 32; cp0 += 8) {
          float vv[8][2];
          load_v8(vv, Vk, d, k * IB + cp0, cp0, rowi, m);
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            float acc[32];
#pragma unroll
            for (int p = 0; p < 32; ++p) acc[p] = fmaf(vv[u][1], a[1][p], vv[u][0] * a[0][p]);
            const float t = warp_transpose_reduce32(acc, lane);
            Wp[(warp * 32 + cp0 + u) * 32 + lane] = t;
          }
        }
      }
      __syncthreads();
      for (int e = tid; e < 1024; e += NT) {
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < NW; ++w) s += Wp[w * 1024 + e];
        for (int rk = 0; rk < CS; ++rk) st_dsmem(&wx[cta * 1024 + e], rk, s);
      }
      cluster.sync();
      for (int e = tid; e < 1024; e += NT) {
        float s = 0.f;
        for (int rk = 0; rk < CS; ++rk) s += wx[rk * 1024 + e];
        Wf[e] = s;
      }
      cluster.sync();   // wx may be overwritten by the next exchange only after everyone has read it
      const float* Tk = Ts + k * 32 * 33;
      for (int e = tid; e < 1024; e += NT) {   // W2 = T_k^T (V_k^T P): apply Q^T
        const int q = e >> 5, p = e & 31;
        float s = 0.f;
        for (int c = 0; c <= q; ++c) s = fmaf(Tk[c * 33 + q], Wf[c * 32 + p], s);
        W2s[e] = s;
      }
      __syncthreads();
#pragma unroll 1
      for (int cp0 = 0; cp0 < 32; cp0 += 8) {
        float vv[8][2];
        load_v8(vv, Vk, d, k * IB + cp0, cp0, rowi, m);
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const float4* w2 = reinterpret_cast<const float4*>(W2s + (cp0 + u) * 32);
#pragma unroll
          for (int q4 = 0; q4 < 8; ++q4) {
            const float4 w = w2[q4];
#pragma unroll
            for (int s = 0; s < 2; ++s) {
              a[s][4 * q4 + 0] = fmaf(-vv[u][s], w.x, a[s][4 * q4 + 0]);
              a[s][4 * q4 + 1] = fmaf(-vv[u][s], w.y, a[s][4 * q4 + 1]);
              a[s][4 * q4 + 2] = fmaf(-vv[u][s], w.z, a[s][4 * q4 + 2]);
              a[s][4 * q4 + 3] = fmaf(-vv[u][s], w.w, a[s][4 * q4 + 3]);
            }
          }
        }
      }
    }
    // ---- factor the inner panel.  Position p of step j is column (j + p) mod 32; inside a group
    // of four steps the rotation is a compile-time register offset, then the registers move by 4.
    PanelCtx pc{red, xch, diag, dloc, coefs, Zs, taus, CS, cta, warp, lane, ip % CS, ip / CS, NW};
#pragma unroll 1
    for (int j4 = 0; j4 < 32; j4 += 4) {
      col_step<0>(a, rowi, ip * IB + j4 + 0, j4 + 0, pc);
      col_step<1>(a, rowi, ip * IB + j4 + 1, j4 + 1, pc);
      col_step<2>(a, rowi, ip * IB + j4 + 2, j4 + 2, pc);
      col_step<3>(a, rowi, ip * IB + j4 + 3, j4 + 3, pc);
#pragma unroll
      for (int s = 0; s < 2; ++s) {
        const float t0 = a[s][0], t1 = a[s][1], t2 = a[s][2], t3 = a[s][3];
#pragma unroll
        for (int p = 0; p < 28; ++p) a[s][p] = a[s][p + 4];
        a[s][28] = t0; a[s][29] = t1; a[s][30] = t2; a[s][31] = t3;
      }
    }
    // ---- after 32 rotations the registers are back in natural order: column c at a[.][c]
    __syncthreads();   // taus[] of the last step is visible to every warp
    if (warp == 0) {
      // T[0:j, j] = -tau_j T[0:j, 0:j] (V^T v_j), T[j][j] = tau_j; lane i keeps row i in registers
      float* T = Ts + ip * 32 * 33;
      float trow[32];
#pragma unroll
      for (int j = 0; j < 32; ++j) {
        const float tj = taus[j];
        float s = 0.f;
#pragma unroll
        for (int c = 0; c < j; ++c) s = fmaf(trow[c], Zs[c * 33 + j], s);   // trow[c] = 0 for c < lane
        trow[j] = (lane < j) ? -tj * s : ((lane == j) ? tj : 0.f);
      }
#pragma unroll
      for (int j = 0; j < 32; ++j) T[lane * 33 + j] = trow[j];
    }
#pragma unroll
    for (int s = 0; s < 2; ++s) {
      const int i = rowi[s];
      if (i < m) {
        uint32_t ph[16], pl[16];
#pragma unroll
        for (int c = 0; c < 32; c += 2) {
          bf16 h0, l0, h1, l1;
          const int dg0 = ip * IB + c, dg1 = dg0 + 1;
          // a skipped reflector (tau = 0, H = I) contributes a zero column to Y
          const float v0 = (i > dg0) ? a[s][c] : ((i == dg0 && taus[c] != 0.f) ? 1.f : 0.f);
          const float v1 = (i > dg1) ? a[s][c + 1] : ((i == dg1 && taus[c + 1] != 0.f) ? 1.f : 0.f);
          split2(v0, h0, l0);
          split2(v1, h1, l1);
          const int64_t t0 = (int64_t)(cb + c) * d + c0 + i, t1 = t0 + d;
          At[t0] = a[s][c];
          At[t1] = a[s][c + 1];
          at_hi[t0] = h0; at_lo[t0] = l0;
          at_hi[t1] = h1; at_lo[t1] = l1;
          ph[c >> 1] = pack2(h0, h1);
          pl[c >> 1] = pack2(l0, l1);
        }
        uint4* yh = reinterpret_cast<uint4*>(y_hi + (int64_t)(c0 + i) * OB + ip * IB);
        uint4* yl = reinterpret_cast<uint4*>(y_lo + (int64_t)(c0 + i) * OB + ip * IB);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          yh[q] = make_uint4(ph[4 * q], ph[4 * q + 1], ph[4 * q + 2], ph[4 * q + 3]);
          yl[q] = make_uint4(pl[4 * q], pl[4 * q + 1], pl[4 * q + 2], pl[4 * q + 3]);
        }
      }
    }
    __syncthreads();   // T of this inner panel is complete; At writes are ordered before re-reads
  }
  if (cta == 0) {   // compact-WY factors of the four inner panels: Tk[k][i][j]
    for (int e = tid; e < (OB / IB) * IB * IB; e += NT) Tk[e] = Ts[(e >> 10) * 32 * 33 + ((e >> 5) & 31) * 33 + (e & 31)];
  }
  cluster.sync();   // no CTA may exit while others can still push into its shared memory
}


// ----------------------------------------------------------------------------- W2 of the outer block
// The outer block's 128 reflectors are four block reflectors H_k = I - V_k T_k V_k^T (T_k from the
// panel kernel).  Q^T C = H_3^T H_2^T H_1^T H_0^T C = C - Y W2 with, per column of C (= row of W^T),
//   W2_k = T_k^T (W_k - sum_{l < k} S_kl W2_l),   W = Y^T C,  S = Y^T Y  (S_kl = V_k^T V_l),
// a block forward substitution with 32 x 32 blocks.  W^T and S are the sums of the split partials
// of the [S; W^T] product (S = rows 0..127).
constexpr int SLD = 129;
constexpr int W2_ROWS_PER_CTA = 64;
constexpr int WY_W2_SMEM = (128 * SLD + 4 * 32 * 32 + W2_ROWS_PER_CTA * SLD) * 4;
// 64 rows of W^T per CTA, staged in shared memory and turned into W2^T block by block; every
// product is a (64 x K) x (K x 32) shared-memory matmul, 2 x 4 outputs per thread.
__global__ void __launch_bounds__(256) wy_w2_kernel(const float* __restrict__ part, int ksplit, int m,
                                                    int64_t part_batch_stride, const float* __restrict__ Tk,
                                                    bf16* __restrict__ w2_hi, bf16* __restrict__ w2_lo,
                                                    int64_t w2_batch_stride) {
  extern __shared__ float sm[];
  float* Ss = sm;                  // [128][SLD]  Y^T Y (only the blocks below the block diagonal are used)
  float* Ts = sm + 128 * SLD;      // [4][32][32]
  float* Ws = Ts + 4 * 32 * 32;    // [64][SLD]   W^T rows, overwritten block by block with W2^T
  part += (int64_t)blockIdx.y * part_batch_stride;
  Tk += (int64_t)blockIdx.y * 4 * 32 * 32;
  w2_hi += (int64_t)blockIdx.y * w2_batch_stride;
  w2_lo += (int64_t)blockIdx.y * w2_batch_stride;
  const int tid = threadIdx.x;
  const int row0 = blockIdx.x * W2_ROWS_PER_CTA;
#pragma unroll 4
  for (int it = 0; it < 12; ++it) {   // rows 32..127 of S, independent 16-byte loads
    const int e = (it * 256 + tid) * 4;
    const int r = 32 + (e >> 7), c = e & 127;
    float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
    if (c < (r & ~31))
      for (int sp = 0; sp < ksplit; ++sp) {
        const float4 t = *reinterpret_cast<const float4*>(part + (int64_t)sp * m * 128 + r * 128 + c);
        s.x += t.x; s.y += t.y; s.z += t.z; s.w += t.w;
      }
    Ss[r * SLD + c] = s.x; Ss[r * SLD + c + 1] = s.y; Ss[r * SLD + c + 2] = s.z; Ss[r * SLD + c + 3] = s.w;
  }
#pragma unroll
  for (int it = 0; it < 8; ++it) {    // the 64 x 128 tile of W^T
    const int e = (it * 256 + tid) * 4;
    const int r = e >> 7, k = e & 127;
    float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int sp = 0; sp < ksplit; ++sp) {
      const float4 t = *reinterpret_cast<const float4*>(part + ((int64_t)sp * m + 128 + row0 + r) * 128 + k);
      s.x += t.x; s.y += t.y; s.z += t.z; s.w += t.w;
    }
    Ws[r * SLD + k] = s.x; Ws[r * SLD + k + 1] = s.y; Ws[r * SLD + k + 2] = s.z; Ws[r * SLD + k + 3] = s.w;
  }
  for (int e = tid; e < 4 * 32 * 32; e += 256) Ts[e] = Tk[e];
  __syncthreads();
  const int r0 = (tid >> 3) * 2, c0 = (tid & 7) * 4;   // rows r0, r0 + 1; columns c0 .. c0 + 3 of the current block
#pragma unroll 1
  for (int k = 0; k < 4; ++k) {
    // X_k = W_k - [W2_0 .. W2_{k-1}] S_k,0:k^T
    float x[2][4];
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
      for (int j = 0; j < 4; ++j) x[a][j] = Ws[(r0 + a) * SLD + 32 * k + c0 + j];
    for (int i = 0; i < 32 * k; ++i) {
      const float a0 = Ws[r0 * SLD + i], a1 = Ws[(r0 + 1) * SLD + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float sv = Ss[(32 * k + c0 + j) * SLD + i];
        x[0][j] = fmaf(-a0, sv, x[0][j]);
        x[1][j] = fmaf(-a1, sv, x[1][j]);
      }
    }
    __syncthreads();                 // everyone has read the old block k
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
      for (int j = 0; j < 4; ++j) Ws[(r0 + a) * SLD + 32 * k + c0 + j] = x[a][j];
    __syncthreads();
    // W2_k = X_k T_k  (T_k upper triangular: i <= column)
    float o[2][4] = {};
    const float* T = Ts + k * 1024;
    for (int i = 0; i < c0 + 4; ++i) {
      const float a0 = Ws[r0 * SLD + 32 * k + i], a1 = Ws[(r0 + 1) * SLD + 32 * k + i];
      const float4 t = *reinterpret_cast<const float4*>(T + i * 32 + c0);
      o[0][0] = fmaf(a0, t.x, o[0][0]); o[0][1] = fmaf(a0, t.y, o[0][1]);
      o[0][2] = fmaf(a0, t.z, o[0][2]); o[0][3] = fmaf(a0, t.w, o[0][3]);
      o[1][0] = fmaf(a1, t.x, o[1][0]); o[1][1] = fmaf(a1, t.y, o[1][1]);
      o[1][2] = fmaf(a1, t.z, o[1][2]); o[1][3] = fmaf(a1, t.w, o[1][3]);
    }
    __syncthreads();                 // everyone has read X_k
#pragma unroll
    for (int a = 0; a < 2; ++a) {
      bf16 h[4], l[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        Ws[(r0 + a) * SLD + 32 * k + c0 + j] = o[a][j];
        split2(o[a][j], h[j], l[j]);
      }
      const int64_t off = (int64_t)(row0 + r0 + a) * 128 + 32 * k + c0;
      *reinterpret_cast<uint2*>(w2_hi + off) = make_uint2(pack2(h[0], h[1]), pack2(h[2], h[3]));
      *reinterpret_cast<uint2*>(w2_lo + off) = make_uint2(pack2(l[0], l[1]), pack2(l[2], l[3]));
    }
    __syncthreads();
  }
}

// Gauge of the raw factor held transposed: U[i][j] = s_i At[j][i] for j >= i, s_i = sign(At[i][i])
// (+1 at 0); fp32 + split copy.
__global__ void __launch_bounds__(256) gauge_ut_kernel(const float* __restrict__ At, float* __restrict__ U,
                                                       bf16* __restrict__ hi, bf16* __restrict__ lo, int d) {
  __shared__ float t[32][33];
  const int64_t off = (int64_t)blockIdx.z * d * d;
  At += off; U += off; hi += off; lo += off;
  const int i0 = blockIdx.y * 32, j0 = blockIdx.x * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  if (j0 >= i0)
    for (int r = ty; r < 32; r += 8) t[r][tx] = At[(int64_t)(j0 + r) * d + i0 + tx];   // At[j][i]
  __syncthreads();
  for (int r = ty; r < 32; r += 8) {
    const int i = i0 + r, j = j0 + tx;
    const float si = (At[(int64_t)i * d + i] < 0.f) ? -1.f : 1.f;
    const float v = (j >= i) ? si * t[tx][r] : 0.f;
    const int64_t idx = (int64_t)i * d + j;
    U[idx] = v;
    split2(v, hi[idx], lo[idx]);
  }
}

template <int NT>
dq_status launch_panel(Ctx& ctx, int cs, int batch, float* At, bf16* at_hi, bf16* at_lo, bf16* y_hi, bf16* y_lo,
                       float* Tk, int d, int c0) {
  using L = PanelSmem<NT / 32>;
  static SmemOptIn attr;
  auto kern = qr_panel_cm_kernel<NT>;
  DQ_CHECK(opt_in_dynamic_smem(kern, L::BYTES, attr));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(cs, batch, 1);
  cfg.blockDim = dim3(NT, 1, 1);
  cfg.dynamicSmemBytes = L::BYTES;
  cfg.stream = ctx.stream;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = cs; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  cfg.attrs = at; cfg.numAttrs = 1;
  DQ_CHECK_CUDA(cudaLaunchKernelEx(&cfg, kern, At, at_hi, at_lo, y_hi, y_lo, Tk, d, c0));
  return after_launch(ctx);
}

}  // namespace

dq_status qrp_transpose_split(Ctx& ctx, const float* Z, float* At, bf16* hi, bf16* lo, int d, int batch) {
  transpose_split_kernel<<<dim3(d / 32, d / 32, batch), 256, 0, ctx.stream>>>(Z, At, hi, lo, d);
  return after_launch(ctx);
}

dq_status qrp_panel(Ctx& ctx, float* At, bf16* at_hi, bf16* at_lo, bf16* y_hi, bf16* y_lo, float* Tk, int d,
                    int c0, int batch) {
  const int m = d - c0;
  if (m <= 0 || m % OB != 0 || m > 8192) return DQ_ERR_UNSUPPORTED;
  // 512 rows per CTA (two rows per thread, 255 registers) in clusters of up to 8; beyond 4096 rows
  // either a cluster of 16 (non-portable size, if the device can co-schedule it) or 1024 rows per CTA.
  static int can16_dev[64];                  // per device: 0 = not probed, 1 = no, 2 = yes
  int dev = 0;
  DQ_CHECK_CUDA(cudaGetDevice(&dev));
  int can16_local = 0;
  int& can16 = (dev >= 0 && dev < 64) ? can16_dev[dev] : can16_local;
  if (m > 4096 && can16 == 0) {
    can16 = 1;
    auto kern = qr_panel_cm_kernel<256>;
    using L = PanelSmem<8>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::BYTES) == cudaSuccess &&
        cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess) {
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3(16, 1, 1); cfg.blockDim = dim3(256, 1, 1); cfg.dynamicSmemBytes = L::BYTES;
      cudaLaunchAttribute at[1];
      at[0].id = cudaLaunchAttributeClusterDimension;
      at[0].val.clusterDim.x = 16; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
      cfg.attrs = at; cfg.numAttrs = 1;
      int n = 0;
      if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) == cudaSuccess && n >= 1) can16 = 2;
    }
    cudaGetLastError();
  }
  const bool wide = m > 4096 && can16 != 2;
  const int rows_per_cta = wide ? 1024 : 512;
  int cs = 1;
  while (cs * rows_per_cta < m) cs *= 2;
  if (cs > MAX_CS) return DQ_ERR_UNSUPPORTED;
  return wide ? launch_panel<512>(ctx, cs, batch, At, at_hi, at_lo, y_hi, y_lo, Tk, d, c0)
              : launch_panel<256>(ctx, cs, batch, At, at_hi, at_lo, y_hi, y_lo, Tk, d, c0);
}

dq_status qrp_wy_w2(Ctx& ctx, const float* part, int ksplit, int m, int64_t part_bs, const float* Tk, bf16* w2_hi,
                    bf16* w2_lo, int64_t w2_bs, int n, int batch) {
  static SmemOptIn attr;
  DQ_CHECK(opt_in_dynamic_smem(wy_w2_kernel, WY_W2_SMEM, attr));
  wy_w2_kernel<<<dim3(n / W2_ROWS_PER_CTA, batch), 256, WY_W2_SMEM, ctx.stream>>>(part, ksplit, m, part_bs, Tk, w2_hi,
                                                                                 w2_lo, w2_bs);
  return after_launch(ctx);
}

dq_status qrp_gauge_ut(Ctx& ctx, const float* At, float* U, bf16* hi, bf16* lo, int d, int batch) {
  gauge_ut_kernel<<<dim3(d / 32, d / 32, batch), 256, 0, ctx.stream>>>(At, U, hi, lo, d);
  return after_launch(ctx);
}

}  // namespace dq
