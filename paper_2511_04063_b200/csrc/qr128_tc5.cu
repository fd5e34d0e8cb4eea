// Batched QR-Orth for 128 x 128 latents on the 5th-generation tensor cores: one CTA per problem, every
// 128^3 product as tcgen05.mma on bf16 (hi, lo) operand pairs that the CTA itself writes into shared memory
// row-major in the 128-byte-swizzled layout, accumulator in tensor memory, two threads per accumulator row.  A
// product that needs a matrix transposed reads the same buffer as an MN-major operand, so every matrix is written
// once, in 16-byte pieces.
//
//   backward  S = tril(R^T Gq - Gq^T R, -1) (one reduction over two operand pairs, split operands: the skew
//             part is a small difference), D^T = W S^T, Gz = R D (plain bf16 operands), Z <- Z - lr Gz
//   forward   incremental factorisation from the previous step's W = U^-1 (no U, no triangular inverse):
//             Zh = Z W, E = Zh^T Zh - I, T <- Phi(E - T^T T) from Phi(E - P_old) until no entry moves,
//             Y = (I + T)^-1 - I by the series Y <- -T - T Y until no entry moves, R = Zh + Zh Y, W <- W + W Y.
//             Zh and E on split operands (three MMAs per term); the others on plain bf16 operands unless the
//             fixed point needed a third sweep (a large step), then on split operands too.
// Both halves run in one launch when the optimiser is plain SGD (the update sits between them), so a step
// boundary is one kernel and the latent, W and the operands made from them never leave the chip in between.
// The products are a dependent chain, so nothing overlaps: write operands, one thread issues the MMAs, all
// wait (bounded) for their completion, every thread reads its accumulator row and prepares the next operands.
#include "common.cuh"
#include "tc_gemm.cuh"

namespace dq {
namespace {

using namespace tc;

constexpr int N5 = 128;
constexpr int PART_BYTES = N5 * N5 * 2;          // one bf16 operand part: two [128][64] K-major blocks
constexpr int KBLK_BYTES = N5 * BLOCK_K * 2;     // 16 KB
constexpr int N_BUFS = 6;
constexpr int TC5_SMEM = N_BUFS * PART_BYTES + 1024 + 1024;
constexpr int TC5_THREADS = 512;                // four threads per accumulator row, a quarter of the columns each
constexpr int CHUNKS_PER_THREAD = 2;
constexpr uint32_t TC5_TMEM_COLS = 512;          // the accumulator and three fp32 matrices that stay on chip
constexpr uint32_t REG_E = 128, REG_T = 256, REG_ZH = 384;   // tensor-memory columns of E (later Y), T and Zh
constexpr int MAX_SERIES = 48;

struct Tc5Params {
  float* Z;            // [batch][128][128] latent (updated when lr != 0)
  float* W;            // [batch][128][128] U^-1 of the previous factorisation (updated by the forward half)
  float* P;            // [batch][128][128] T^T T of the previous step's last sweep (updated)
  float* R;            // [batch][128][128] rotation read by the backward half
  float* R_out;        // rotation written by the forward half (may be R)
  __nv_bfloat16* Rt;   // nullable: bf16(R^T), the operand of O = X R
  const float* Gq;     // backward: dL/dR
  float* Gz;           // backward: dL/dZ
  float lr;
  int do_backward, do_forward;
  int max_sweeps;
  float tol;
  int* d_status;
};

__device__ __forceinline__ void fence_async_smem5() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

constexpr int CH = 16;                           // columns of the accumulator row handled at a time

// This thread's lane of tensor memory also keeps its rows of the fp32 matrices the chain needs again (E, T, Zh,
// Y): 16 columns per access, no shared or global memory traffic.
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const float* f) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      :: "r"(taddr), "f"(f[0]), "f"(f[1]), "f"(f[2]), "f"(f[3]), "f"(f[4]), "f"(f[5]), "f"(f[6]), "f"(f[7]),
         "f"(f[8]), "f"(f[9]), "f"(f[10]), "f"(f[11]), "f"(f[12]), "f"(f[13]), "f"(f[14]), "f"(f[15])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld16f(uint32_t taddr, float* f) {
  uint32_t r[16];
  tmem_ld16(taddr, r);
#pragma unroll
  for (int i = 0; i < 16; ++i) f[i] = __uint_as_float(r[i]);
}

// CH consecutive fp32 of a row (two 32-byte accesses); a null source reads as zeros
__device__ __forceinline__ void fetch_ch(const float* p, float* v) {
  if (p) {
    ld_global_f32x8(p, v);
    ld_global_f32x8(p + 8, v + 8);
  } else {
#pragma unroll
    for (int i = 0; i < CH; ++i) v[i] = 0.f;
  }
}
__device__ __forceinline__ void store_ch(float* p, const float* v) {
  st_global_f32x8(p, v);
  st_global_f32x8(p + 8, v + 8);
}

__device__ __forceinline__ void split_ch(const float* f, uint32_t* ph, uint32_t* pl) {
#pragma unroll
  for (int i = 0; i < CH / 2; ++i) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
    const float2 hf = __bfloat1622float2(h);
    const __nv_bfloat162 l = __floats2bfloat162_rn(f[2 * i] - hf.x, f[2 * i + 1] - hf.y);
    ph[i] = *reinterpret_cast<const uint32_t*>(&h);
    pl[i] = *reinterpret_cast<const uint32_t*>(&l);
  }
}

// Operand with rows = this matrix's rows (K = its columns): columns [CH c, CH c + CH) of row r.
__device__ __forceinline__ void put_rowmajor(uint8_t* buf, int r, int c, const uint32_t* packed) {
  uint8_t* rowp = buf + (c >> 2) * KBLK_BYTES + r * 128;
#pragma unroll
  for (int i = 0; i < CH / 8; ++i) {
    const int chunk = ((c & 3) * 2 + i) ^ (r & 7);
    *reinterpret_cast<uint4*>(rowp + chunk * 16) =
        make_uint4(packed[4 * i], packed[4 * i + 1], packed[4 * i + 2], packed[4 * i + 3]);
  }
}
struct Tc5 {
  uint8_t* smem;        // operand buffers (generic pointer)
  uint32_t smem_u;      // the same, shared-window address
  uint32_t bar;         // mbarrier the MMAs commit to
  uint32_t parity;
  uint32_t tmem_row;    // accumulator, this thread's lane
  uint32_t tmem;        // accumulator base
  int c_begin;          // first of this thread's CHUNKS_PER_THREAD chunks of its row
  int* d_status;
  __device__ __forceinline__ uint8_t* buf(int i) const { return smem + i * PART_BYTES; }
  // acc (+)= op(A) op(B)^T over the whole K = 128 (issuing thread only).  Every buffer holds a matrix row-major
  // (row r = 128 bytes of each of its two 64-column blocks, swizzled).  Read K-major it is the operand with rows =
  // the matrix's rows; read MN-major (at / bt: the reduction runs over the matrix's ROWS, 16 of them = 2048 bytes
  // per instruction, the second 64 columns one block further on) it is the operand of the TRANSPOSED matrix, so no
  // transposed copy of anything is ever written.
  __device__ __forceinline__ void mma(int a, int b, bool accumulate, bool negate_a = false, bool at = false,
                                      bool bt = false) const {
    const uint32_t idesc = make_idesc_bf16(N5) | (negate_a ? IDESC_NEGATE_A : 0u) | (at ? IDESC_A_MN_MAJOR : 0u) |
                           (bt ? IDESC_B_MN_MAJOR : 0u);
    const uint32_t sa = smem_u + a * PART_BYTES, sb = smem_u + b * PART_BYTES;
#pragma unroll 1
    for (int s = 0; s < N5 / UMMA_K; ++s) {
      const uint32_t kmaj = (uint32_t)((s >> 2) * KBLK_BYTES + (s & 3) * UMMA_K * 2), mnmaj = (uint32_t)(s * UMMA_K * 128);
      umma_bf16(tmem, at ? make_mnmajor_sw128_desc(sa + mnmaj, KBLK_BYTES) : make_kmajor_sw128_desc(sa + kmaj),
                bt ? make_mnmajor_sw128_desc(sb + mnmaj, KBLK_BYTES) : make_kmajor_sw128_desc(sb + kmaj), idesc,
                (accumulate || s > 0) ? 1u : 0u);
    }
  }
  // split-operand product: A = (a_hi, a_lo), B = (b_hi, b_lo): hi hi + hi lo + lo hi
  __device__ __forceinline__ void mma3(int a_hi, int a_lo, int b_hi, int b_lo, bool at = false, bool bt = false) const {
    mma(a_hi, b_hi, false, false, at, bt);
    mma(a_hi, b_lo, true, false, at, bt);
    mma(a_lo, b_hi, true, false, at, bt);
  }
};

// One product of the chain: all threads have written their operand rows; thread 0 issues the MMAs (issue());
// every thread waits (bounded) for their completion and then runs body(c, v, g, x0, x1) on the CH-wide chunks of
// its accumulator row.  g: the same chunk of the fp32 row `grow` in global memory (nullable; fetched one chunk
// ahead, the first one while the MMAs run); x0 / x1: the same chunk of the matrices kept in tensor memory at
// columns t0 / t1 (0: none).  Returns false if the wait gave up (for all threads alike).
// pre (nullable): the thread's part of that row when the caller holds it in registers already.
template <typename Issue, typename Body>
__device__ __forceinline__ bool product(Tc5& k, Issue issue, const float* grow, uint32_t t0, uint32_t t1, Body body,
                                        const float (*pre)[CH] = nullptr) {
  tmem_ld_wait();
  tmem_st_wait();
  tc_fence_before();
  fence_async_smem5();
  __syncthreads();
  if (threadIdx.x == 0) {
    tc_fence_after();
    issue();
    umma_commit(k.bar);
  }
  const int c_begin = k.c_begin;
  float ga[CH], gb[CH];
  if (!pre) fetch_ch(grow ? grow + c_begin * CH : nullptr, ga);
  const bool done = mbar_wait(k.bar, k.parity, k.d_status);
  k.parity ^= 1u;
  tc_fence_after();
  if (!__syncthreads_and(done ? 1 : 0)) return false;
  static_assert(CHUNKS_PER_THREAD % 2 == 0, "chunks are processed in pairs");
  auto one = [&](int c, const float (&g)[CH]) {
    uint32_t v[CH];
    float x0[CH], x1[CH];
    tmem_ld16(k.tmem_row + (uint32_t)(c * CH), v);
    if (t0) tmem_ld16f(k.tmem_row + t0 + (uint32_t)(c * CH), x0);
    if (t1) tmem_ld16f(k.tmem_row + t1 + (uint32_t)(c * CH), x1);
    tmem_ld_wait();
    body(c, v, g, x0, x1);
  };
#pragma unroll 1
  for (int c = c_begin; c < c_begin + CHUNKS_PER_THREAD; ++c) {   // (one copy of the body: the kernel's code is fetched cold on every launch)
    if (pre) {
#pragma unroll
      for (int i = 0; i < CH; ++i) ga[i] = (c == c_begin) ? pre[0][i] : pre[1][i];
    } else if (c > c_begin) {
#pragma unroll
      for (int i = 0; i < CH; ++i) ga[i] = gb[i];
    }
    if (!pre && c + 1 < c_begin + CHUNKS_PER_THREAD) fetch_ch(grow ? grow + (c + 1) * CH : nullptr, gb);
    one(c, ga);
  }
  return true;
}

// This thread's row of an fp32 matrix in global memory -> operand buffers (hi and, unless negative, lo part).
// f: the values stay with the caller.
__device__ __forceinline__ void load_row_to_operands(const Tc5& k, const float* row, int r, int rm_hi, int rm_lo,
                                                     float (&f)[CHUNKS_PER_THREAD][CH]) {
  // all of the thread's loads in flight before the first is used
#pragma unroll
  for (int i = 0; i < CHUNKS_PER_THREAD; ++i) fetch_ch(row + (k.c_begin + i) * CH, f[i]);
#pragma unroll
  for (int i = 0; i < CHUNKS_PER_THREAD; ++i) {
    const int c = k.c_begin + i;
    uint32_t ph[CH / 2], pl[CH / 2];
    split_ch(f[i], ph, pl);
    put_rowmajor(k.buf(rm_hi), r, c, ph);
    if (rm_lo >= 0) put_rowmajor(k.buf(rm_lo), r, c, pl);
  }
}
__device__ __forceinline__ void load_row_to_operands(const Tc5& k, const float* row, int r, int rm_hi, int rm_lo) {
  float f[CHUNKS_PER_THREAD][CH];
  load_row_to_operands(k, row, r, rm_hi, rm_lo, f);
}

__device__ __forceinline__ float phi(float s, int row, int col) {
  return (col > row) ? s : ((col == row) ? 0.5f * s : 0.f);
}

__global__ void __launch_bounds__(TC5_THREADS, 1) qr128_step_tc5_kernel(const Tc5Params p) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_ptr = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t bar = smem_base + N_BUFS * PART_BYTES;
  const uint32_t tmem_slot = bar + 16u;
  uint32_t* tmem_slot_ptr = reinterpret_cast<uint32_t*>(smem_ptr + N_BUFS * PART_BYTES + 16);
  float* red = reinterpret_cast<float*>(smem_ptr + N_BUFS * PART_BYTES + 64);   // [2 x warps] block reductions

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r = 32 * (warp & 3) + lane;           // accumulator row (tensor-memory lane) of this thread
  const int64_t off = (int64_t)blockIdx.x * N5 * N5;
  float lr = p.lr;
  if (p.d_status && *p.d_status != 0) lr = 0.f;   // an earlier error freezes the latent

  if (threadIdx.x == 0) {
    mbar_init(bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) tmem_alloc(tmem_slot, TC5_TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  Tc5 k;
  k.smem = smem_ptr; k.smem_u = smem_base; k.bar = bar; k.parity = 0u; k.d_status = p.d_status;
  k.tmem = *tmem_slot_ptr;
  k.tmem_row = k.tmem + ((uint32_t)((warp & 3) * 32) << 16);
  k.c_begin = (warp >> 2) * CHUNKS_PER_THREAD;

  float* Zrow = p.Z + off + r * N5;
  float* Wrow = p.W + off + r * N5;
  float* Prow = p.P + off + r * N5;
  float* Rrow = p.R + off + r * N5;
  bool ok = true;
  using V = const uint32_t (&)[CH];
  using F = const float (&)[CH];

  if (p.do_backward) {
    // operands: R -> 0 (hi), 1 (lo), Gq -> 2 (hi), 5 (lo), W -> 3
    load_row_to_operands(k, Rrow, r, 0, 1);
    load_row_to_operands(k, p.Gq + off + r * N5, r, 2, 5);
    load_row_to_operands(k, Wrow, r, 3, -1);
    // S = tril(R^T Gq - Gq^T R, -1), row-major -> 4.  The skew part is what is left of B = R^T Gq after a
    // cancellation (B is close to symmetric near a stationary point), so this one product of the backward runs
    // on split operands: three MMA groups per term, the second term with A negated.
    ok = product(k, [&]() {
                   k.mma3(0, 1, 2, 5, true, true);                                  // R^T Gq
                   k.mma(2, 0, true, true, true, true); k.mma(2, 1, true, true, true, true);   // - Gq^T R
                   k.mma(5, 0, true, true, true, true);
                 }, nullptr, 0, 0,
                 [&](int c, V v, F, F, F) {
                   float f[CH];
#pragma unroll
                   for (int i = 0; i < CH; ++i) f[i] = (r > CH * c + i) ? __uint_as_float(v[i]) : 0.f;
                   uint32_t ph[CH / 2], pl[CH / 2];
                   split_ch(f, ph, pl);
                   put_rowmajor(k.buf(4), r, c, ph);
                 });
    // D^T = W S^T, row-major -> 5
    if (ok)
      ok = product(k, [&]() { k.mma(3, 4, false); }, nullptr, 0, 0,
                   [&](int c, V v, F, F, F) {
                     float f[CH];
#pragma unroll
                     for (int i = 0; i < CH; ++i) f[i] = __uint_as_float(v[i]);
                     uint32_t ph[CH / 2], pl[CH / 2];
                     split_ch(f, ph, pl);
                     put_rowmajor(k.buf(5), r, c, ph);
                   });
    // Gz = R D, then Z <- Z - lr Gz; the new latent goes straight into the forward's operands (1, 2)
    if (ok)
      ok = product(k, [&]() { k.mma(0, 5, false); }, Zrow, 0, 0,
                   [&](int c, V v, F z, F, F) {
                     float g[CH], zn[CH];
#pragma unroll
                     for (int i = 0; i < CH; ++i) {
                       g[i] = __uint_as_float(v[i]);
                       zn[i] = fmaf(-lr, g[i], z[i]);
                     }
                     store_ch(p.Gz + off + r * N5 + c * CH, g);
                     if (lr != 0.f) store_ch(Zrow + c * CH, zn);
                     if (p.do_forward) {
                       uint32_t ph[CH / 2], pl[CH / 2];
                       split_ch(zn, ph, pl);
                       put_rowmajor(k.buf(1), r, c, ph);
                       put_rowmajor(k.buf(2), r, c, pl);
                     }
                   });
  }

  if (p.do_forward && ok) {
    if (!p.do_backward) load_row_to_operands(k, Zrow, r, 1, 2);             // Z -> 1 (hi), 2 (lo)
    load_row_to_operands(k, Wrow, r, 3, 4);                                 // W -> 3, 4
    // Zh = Z W (split operands): fp32 kept in tensor memory, Zh -> 1, 2
    ok = product(k, [&]() { k.mma3(1, 2, 3, 4, false, true); }, nullptr, 0, 0,
                 [&](int c, V v, F, F, F) {
                   float f[CH];
#pragma unroll
                   for (int i = 0; i < CH; ++i) f[i] = __uint_as_float(v[i]);
                   tmem_st16(k.tmem_row + REG_ZH + (uint32_t)(c * CH), f);
                   uint32_t ph[CH / 2], pl[CH / 2];
                   split_ch(f, ph, pl);
                   put_rowmajor(k.buf(1), r, c, ph);
                   put_rowmajor(k.buf(2), r, c, pl);
                 });
    // E = Zh^T Zh - I (split operands) and the start of the fixed point T = Phi(E - P_old):
    // T -> 0, 5; E and T (fp32) stay in tensor memory
    if (ok)
      ok = product(k, [&]() { k.mma3(1, 2, 1, 2, true, true); }, Prow, 0, 0,
                   [&](int c, V v, F pold, F, F) {
                     float e[CH], t[CH];
#pragma unroll
                     for (int i = 0; i < CH; ++i) {
                       const int col = CH * c + i;
                       e[i] = __uint_as_float(v[i]) - ((col == r) ? 1.f : 0.f);
                       t[i] = phi(e[i] - pold[i], r, col);
                     }
                     tmem_st16(k.tmem_row + REG_E + (uint32_t)(c * CH), e);
                     tmem_st16(k.tmem_row + REG_T + (uint32_t)(c * CH), t);
                     uint32_t ph[CH / 2], pl[CH / 2];
                     split_ch(t, ph, pl);
                     put_rowmajor(k.buf(0), r, c, ph);
                     put_rowmajor(k.buf(5), r, c, pl);
                   });
    // sweeps T <- Phi(E - T^T T) until no entry moves (the count is data dependent: the whole problem is here)
    int sweeps = 0;
    bool converged = false;
    while (ok && sweeps < p.max_sweeps && !converged) {
      ++sweeps;
      const bool accurate = sweeps > 2;
      bool moved = false;
      ok = product(k, [&]() { if (accurate) k.mma3(0, 5, 0, 5, true, true); else k.mma(0, 0, false, false, true, true); },
                   nullptr, REG_E, REG_T,
                   [&](int c, V v, F, F e, F told) {
                     float pp[CH], t[CH];
#pragma unroll
                     for (int i = 0; i < CH; ++i) {
                       pp[i] = __uint_as_float(v[i]);
                       t[i] = phi(e[i] - pp[i], r, CH * c + i);
                       if (!(fabsf(t[i] - told[i]) <= p.tol)) moved = true;
                     }
                     store_ch(Prow + c * CH, pp);          // where the next step's fixed point starts
                     tmem_st16(k.tmem_row + REG_T + (uint32_t)(c * CH), t);
                     uint32_t ph[CH / 2], pl[CH / 2];
                     split_ch(t, ph, pl);
                     put_rowmajor(k.buf(0), r, c, ph);
                     put_rowmajor(k.buf(5), r, c, pl);
                   });
      converged = !__syncthreads_or(moved ? 1 : 0);
    }
    if (ok && !converged) { set_status(p.d_status, DQ_ERR_NOT_CONVERGED); }
    const bool big = sweeps > 2;        // a large step: the first-order products on split operands as well
    // Y = (I + T)^-1 - I by Y <- -T - T Y from Y = -T;  Y -> 3, 4 (W is no longer needed there); Y (fp32) takes the
    // place of E in tensor memory.  The terms shrink geometrically (ratio at most |T|), so the series stops as
    // soon as the NEXT term, estimated from the last two, would change no entry by more than 2e-7: after a small
    // step a single product.
    constexpr float SERIES_TOL = 2e-7f;
    uint32_t* red_u = reinterpret_cast<uint32_t*>(red);    // block-wide max of non-negative floats (as bits)
    auto block_max = [&](float v) -> float {
      if (threadIdx.x == 0) red_u[0] = 0u;
      __syncthreads();
      if (v > 0.f) atomicMax(red_u, __float_as_uint(v));
      else if (!(v == 0.f)) atomicMax(red_u, 0x7f800000u);   // NaN: never converged
      __syncthreads();
      const float m = __uint_as_float(red_u[0]);
      __syncthreads();
      return m;
    };
    float prev = 0.f;
    if (ok) {
      float tmax = 0.f;
      tmem_st_wait();
#pragma unroll 1
      for (int c = k.c_begin; c < k.c_begin + CHUNKS_PER_THREAD; ++c) {
        float t[CH];
        tmem_ld16f(k.tmem_row + REG_T + (uint32_t)(c * CH), t);
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < CH; ++i) { t[i] = -t[i]; tmax = fmaxf(tmax, fabsf(t[i])); if (t[i] != t[i]) tmax = NAN; }
        tmem_st16(k.tmem_row + REG_E + (uint32_t)(c * CH), t);
        uint32_t ph[CH / 2], pl[CH / 2];
        split_ch(t, ph, pl);
        put_rowmajor(k.buf(3), r, c, ph);
        put_rowmajor(k.buf(4), r, c, pl);
      }
      prev = block_max(tmax);
    }
    int terms = 0;
    converged = !(prev > 0.f);          // T = 0: Y = 0
    while (ok && terms < MAX_SERIES && !converged) {
      ++terms;
      float chg = 0.f;
      ok = product(k, [&]() { if (big) k.mma3(0, 5, 3, 4, false, true); else k.mma(0, 3, false, false, false, true); },
                   nullptr, REG_T, REG_E,
                   [&](int c, V v, F, F t, F yold) {
                     float y[CH];
#pragma unroll
                     for (int i = 0; i < CH; ++i) {
                       y[i] = -t[i] - __uint_as_float(v[i]);
                       const float dlt = fabsf(y[i] - yold[i]);
                       chg = (dlt == dlt) ? fmaxf(chg, dlt) : NAN;
                     }
                     tmem_st16(k.tmem_row + REG_E + (uint32_t)(c * CH), y);
                     uint32_t ph[CH / 2], pl[CH / 2];
                     split_ch(y, ph, pl);
                     put_rowmajor(k.buf(3), r, c, ph);
                     put_rowmajor(k.buf(4), r, c, pl);
                   });
      const float m = block_max(chg);
      // next term ~ m * (m / prev), with the ratio capped below 1 so that a stalled series is not mistaken for done
      const float ratio = fminf(m / prev, 0.5f);
      converged = (m <= SERIES_TOL) || (m * ratio <= SERIES_TOL && m < prev);
      prev = m;
    }
    if (ok && !converged) { set_status(p.d_status, DQ_ERR_NOT_CONVERGED); }
    // R = Zh + Zh Y
    if (ok)
      ok = product(k, [&]() { if (big) k.mma3(1, 2, 3, 4, false, true); else k.mma(1, 3, false, false, false, true); },
                   nullptr, REG_ZH, 0,
                   [&](int c, V v, F, F zh, F) {
                     float f[CH];
#pragma unroll
                     for (int i = 0; i < CH; ++i) f[i] = zh[i] + __uint_as_float(v[i]);
                     store_ch(p.R_out + off + r * N5 + c * CH, f);
                     if (p.Rt) {   // bf16(R^T): for a fixed column the warp's 32 rows are 64 contiguous bytes
                       __nv_bfloat16* rt = p.Rt + off + r;
#pragma unroll
                       for (int i = 0; i < CH; ++i) rt[(CH * c + i) * N5] = __float2bfloat16_rn(f[i]);
                     }
                   });
    // W <- W + W Y  (W row-major -> 0, 5: T is no longer needed)
    float dv = NAN;                     // the diagonal entry, in the thread whose chunks hold it
    if (ok) {
      float wrow[CHUNKS_PER_THREAD][CH];      // read once: the operands are made from it and the sum below starts from it
      load_row_to_operands(k, Wrow, r, 0, 5, wrow);
      ok = product(k, [&]() { if (big) k.mma3(0, 5, 3, 4, false, true); else k.mma(0, 3, false, false, false, true); },
                   nullptr, 0, 0,
                   [&](int c, V v, F w, F, F) {
                     float f[CH];
#pragma unroll
                     for (int i = 0; i < CH; ++i) {
                       f[i] = w[i] + __uint_as_float(v[i]);
                       if (CH * c + i == r) dv = f[i];
                     }
                     store_ch(Wrow + c * CH, f);
                   }, wrow);
    }
    if (ok) {   // rank / finiteness test on diag(W) = 1 / diag(U)
      const bool owner = (r / CH) >= k.c_begin && (r / CH) < k.c_begin + CHUNKS_PER_THREAD;
      float mn = owner ? fabsf(dv) : INFINITY, mx = owner ? fabsf(dv) : 0.f;
#pragma unroll
      for (int o = 16; o >= 1; o >>= 1) {
        mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      }
      constexpr int NW = TC5_THREADS / 32;
      if (lane == 0) { red[warp] = mn; red[NW + warp] = mx; }
      if (owner && !(isfinite(dv) && dv > 0.f))
        set_status(p.d_status, isfinite(dv) ? DQ_ERR_SINGULAR : DQ_ERR_NONFINITE);
      __syncthreads();
      if (threadIdx.x == 0) {
        float a = INFINITY, b = 0.f;
        for (int i = 0; i < NW; ++i) { a = fminf(a, red[i]); b = fmaxf(b, red[NW + i]); }
        if (!(a > 1e-6f * b)) set_status(p.d_status, DQ_ERR_SINGULAR);
      }
    }
  }

  // ------------------------------------------------------------- teardown
  tmem_ld_wait();
  tmem_st_wait();
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(k.tmem, TC5_TMEM_COLS);
  }
}

}  // namespace

// Backward (do_backward), SGD update (lr != 0) and incremental forward (do_forward) of `batch` 128 x 128
// problems, one CTA each.  P: T^T T of the previous step (zeros after a factorisation from scratch).  The forward
// half writes the rotation to R_out (nullptr: to R, which the backward half has read by then).
dq_status qr128_step_tc5(Ctx& ctx, float* Z, float* W, float* P, float* R, float* R_out, __nv_bfloat16* Rt, const float* Gq,
                         float* Gz, float lr, bool do_backward, bool do_forward, int max_sweeps, int batch) {
  static SmemOptIn attr;
  DQ_CHECK(opt_in_dynamic_smem(qr128_step_tc5_kernel, TC5_SMEM, attr));
  Tc5Params p{};
  p.Z = Z; p.W = W; p.P = P; p.R = R; p.R_out = R_out ? R_out : R; p.Rt = Rt; p.Gq = Gq; p.Gz = Gz;
  p.lr = lr; p.do_backward = do_backward ? 1 : 0; p.do_forward = do_forward ? 1 : 0;
  p.max_sweeps = max_sweeps < 3 ? 3 : max_sweeps; p.tol = 1e-5f; p.d_status = ctx.d_status;
  qr128_step_tc5_kernel<<<batch, TC5_THREADS, TC5_SMEM, ctx.stream>>>(p);
  return after_launch(ctx);
}

}  // namespace dq
