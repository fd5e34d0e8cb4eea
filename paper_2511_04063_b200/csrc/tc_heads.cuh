// Fused Whip step for many 128 x 128 rotations (per-head rotations): one kernel computes, per head h
// and per tile of TT = 128 tokens,
//   O^T = R_h^T X_t^T     (tcgen05, accumulator in tensor memory)
//   e = exp(-|o|), loss partials, G = -sign(o) e   (Eq. 4; epilogue from tensor memory)
//   Gq_h^T += G_t^T X_t    (second tcgen05 product: the epilogue writes bf16 G_t^T back into tensor memory, over
//                           the part of the O^T accumulator it has just read, and the product takes it from
//                           there as its A operand; the accumulator stays in tensor memory for all tiles of
//                           the segment)
// so the rotated activations and dL/dO never reach HBM or shared memory and X is read exactly once: the second
// product reads the same token-major tile of X that TMA loaded for the first one, as its MN-major B operand
// (reduction index = token, 64 consecutive channels per 128-byte row), so no channel-major copy is made.
//
// What bounds the kernel is the rate at which products can be issued and the operands fetched from shared memory,
// not arithmetic: a tcgen05.mma of 128 x N x 16 costs about 60 cycles for every N up to 128, so the tiles are 128
// tokens wide (N = 128 in both products), G_t^T does not pass through shared memory, and each of the two products
// has an issuing thread of its own.
//
// One CTA per SM.  The tiles of all heads form one sequence, cut into gridDim.x equal ranges; the part of a CTA's
// range that lies in one head is a segment: R_h^T stays in shared memory for a segment, and a segment writes one
// 128 x 128 fp32 partial of Gq_h and its loss partials into slot (CTA - first CTA of the head) of the head.  A head's
// unused slots stay zero (the caller clears the buffers once; which slots are used depends on the launch shape
// only), and the slots are summed afterwards in a fixed order.
//
// 608 threads: warp 0 TMA producer (R_h^T and the X_t ring), warp 1 issuer of the first product, warps 2..17
// epilogue (four warps per quarter of the tensor-memory lanes, 32 token columns each), warp 18 issuer of the
// second product.  X_t and the O^T accumulator that holds G_t^T are released once the second product of the
// tile has retired; three O^T accumulators.  Every wait is bounded (DQ_ERR_TIMEOUT on expiry).
#pragma once
#include "tc_gemm.cuh"

namespace dq {
namespace heads {

using namespace tc;

constexpr int TT = 128;                            // tokens per tile
constexpr int KB_BYTES = 128 * BLOCK_K * 2;        // one [128 rows][64 bf16] K-major block: 16 KB
constexpr int XKB_BYTES = TT * BLOCK_K * 2;        // one [TT rows][64 bf16] K-major block of X_t: 16 KB
constexpr int RT_BYTES = 2 * KB_BYTES;             // R_h^T: rows = output channel, K = input channel (128)
constexpr int XA_BYTES = 2 * XKB_BYTES;            // X_t:   rows = token (TT), K = input channel (two k-blocks)
constexpr int XA_STAGES = 6;                       // a tile stays until its second product has retired
constexpr int SMEM_TOTAL = RT_BYTES + XA_STAGES * XA_BYTES + 1024 + 1024;
constexpr int O_BUFS = 3;
constexpr uint32_t TMEM_COLS = 512;                // O^T (3 x TT columns; G_t^T over half of each) + Gq^T (128 columns)
constexpr int EPI_WARPS = 16;
constexpr int Q_WARP = 2 + EPI_WARPS;              // warp of the second product's issuer
constexpr int HEADS_THREADS = 32 * (Q_WARP + 1);

struct Params {
  int batch, tiles_per_head, slots;    // slots: partials kept per head (>= the CTAs that share any one head)
  int64_t n_tokens;
  float* part;                         // [batch][slots][128][128] partial Gq (row = input channel)
  float* partials;                     // [batch][slots][EPI_WARPS] loss partials
  __nv_bfloat16* Gt;                   // nullable: also store dL/dO, [batch][128][n_tokens] channel-major
  int* d_status;
};

// First tile of CTA c's range when `total` tiles are cut into n ranges.
__host__ __device__ inline int64_t range_begin(int64_t c, int64_t total, int64_t n) { return c * total / n; }
// The CTA whose range holds tile g.
__host__ __device__ inline int range_owner(int64_t g, int64_t total, int64_t n) {
  int64_t c = g * n / total;
  while (c + 1 < n && range_begin(c + 1, total, n) <= g) ++c;
  while (c > 0 && range_begin(c, total, n) > g) --c;
  return (int)c;
}

// D (+)= A B^T with A taken from tensor memory: lane = row of A, two bf16 of consecutive k per 32-bit column.
__device__ __forceinline__ void umma_bf16_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t bdesc, uint32_t idesc,
                                             uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(tmem_d), "r"(tmem_a), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// 32 lanes x 16 consecutive 32-bit columns from registers: thread l writes row (lane base + l).
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      :: "r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
         "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__global__ void __launch_bounds__(HEADS_THREADS, 1)
heads_whip_kernel(const __grid_constant__ CUtensorMap mapRt, const __grid_constant__ CUtensorMap mapX, const Params p) {
  constexpr uint32_t IDESC_O = make_idesc_bf16(TT);     // O^T tile: 128 channels x TT tokens
  constexpr uint32_t IDESC_Q = make_idesc_bf16(128) | IDESC_B_MN_MAJOR;    // Gq^T: 128 x 128, B = X_t^T read from the token-major tile
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t rt_smem = smem_base;
  const uint32_t xa_base = rt_smem + RT_BYTES;
  const uint32_t bar_base = xa_base + XA_STAGES * XA_BYTES;
  constexpr int B_XAF = 0, B_XAE = B_XAF + XA_STAGES, B_TF = B_XAE + XA_STAGES, B_TE = B_TF + O_BUFS, B_GF = B_TE + O_BUFS,
                B_MISC = B_GF + O_BUFS;
  auto xa_full = [&](int s) { return bar_base + 8u * (B_XAF + s); };
  auto xa_empty = [&](int s) { return bar_base + 8u * (B_XAE + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (B_TF + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (B_TE + a); };
  auto gfull_bar = [&](int a) { return bar_base + 8u * (B_GF + a); };     // G_t^T written over accumulator a
  const uint32_t rtfull_bar = bar_base + 8u * B_MISC, rtempty_bar = bar_base + 8u * (B_MISC + 1);
  const uint32_t qfull_bar = bar_base + 8u * (B_MISC + 2), qempty_bar = bar_base + 8u * (B_MISC + 3);
  const uint32_t tmem_slot = bar_base + 8u * (B_MISC + 4);
  uint32_t* tmem_slot_ptr = reinterpret_cast<uint32_t*>(smem_raw + (tmem_slot - smem_u32(smem_raw)));

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < XA_STAGES; ++s) {
      mbar_init(xa_full(s), 1); mbar_init(xa_empty(s), 1);
    }
    for (int s = 0; s < O_BUFS; ++s) { mbar_init(tfull_bar(s), 1); mbar_init(tempty_bar(s), 1); mbar_init(gfull_bar(s), EPI_WARPS); }
    mbar_init(rtfull_bar, 1); mbar_init(rtempty_bar, 1);
    mbar_init(qfull_bar, 1); mbar_init(qempty_bar, EPI_WARPS);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    prefetch_tensormap(&mapRt); prefetch_tensormap(&mapX);
  }
  if (warp == 1) tmem_alloc(tmem_slot, TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot_ptr;
  const uint32_t tmem_q = tmem_base + (uint32_t)(O_BUFS * TT);

  // this CTA's range of the tile sequence and its segments, one per head it touches
  const int64_t total = (int64_t)p.batch * p.tiles_per_head;
  const int64_t g_begin = range_begin(blockIdx.x, total, gridDim.x), g_end = range_begin(blockIdx.x + 1, total, gridDim.x);
  // segment that starts at tile g (g_begin <= g < g_end): head b, tiles [t0, t1) of the head, slot of the head's partials
  auto segment = [&](int64_t g, int& b, int& t0, int& t1, int& slot) {
    b = (int)(g / p.tiles_per_head);
    const int64_t h0 = (int64_t)b * p.tiles_per_head;
    t0 = (int)(g - h0);
    t1 = (g_end - h0 < p.tiles_per_head) ? (int)(g_end - h0) : p.tiles_per_head;
    slot = (int)blockIdx.x - range_owner(h0, total, gridDim.x);
  };

  if (warp == 0) {
    // ------------------------------------------------------------- TMA producer: R_h^T per segment, the X_t ring
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0, rt_phase = 0;
      bool ok = true;
      // X passes through once: first out of the L2, so that the latents, rotations and partial sums of the step's
      // other kernels (and their code) stay there
      const uint64_t x_policy = l2_evict_first_policy();
      for (int64_t g = g_begin; g < g_end && ok;) {
        int b, t0, t1, slot;
        segment(g, b, t0, t1, slot);
        if (!mbar_wait(rtempty_bar, rt_phase ^ 1u, p.d_status)) break;
        rt_phase ^= 1u;
        mbar_expect_tx(rtfull_bar, RT_BYTES);
        tma_load_3d(rt_smem, &mapRt, rtfull_bar, 0, 0, b);
        tma_load_3d(rt_smem + KB_BYTES, &mapRt, rtfull_bar, BLOCK_K, 0, b);
        for (int t = t0; t < t1; ++t) {
          if (!mbar_wait(xa_empty(stage), phase ^ 1u, p.d_status)) { ok = false; break; }
          mbar_expect_tx(xa_full(stage), XA_BYTES);
          const uint32_t xa = xa_base + stage * XA_BYTES;
          tma_load_3d_hint(xa, &mapX, xa_full(stage), 0, t * TT, b, x_policy);
          tma_load_3d_hint(xa + XKB_BYTES, &mapX, xa_full(stage), BLOCK_K, t * TT, b, x_policy);
          if (++stage == XA_STAGES) { stage = 0; phase ^= 1u; }
        }
        g += t1 - t0;
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------- issuer of the first product, O^T = R_h^T X_t^T
    if (lane == 0) {
      // descriptors of R_h^T (fixed) and of stage 0 of the X_t ring; a later stage or k-step adds its byte
      // offset / 16 to the address field
      uint64_t rd[2 * (BLOCK_K / UMMA_K)];
#pragma unroll
      for (int kb = 0; kb < 2; ++kb)
#pragma unroll
        for (int k = 0; k < BLOCK_K / UMMA_K; ++k)
          rd[kb * (BLOCK_K / UMMA_K) + k] = make_kmajor_sw128_desc(rt_smem + kb * KB_BYTES + k * UMMA_K * 2);
      const uint64_t x0 = make_kmajor_sw128_desc(xa_base);
      int st1 = 0, acc = 0;
      uint32_t ph1 = 0, acc_phase = 0, rt_phase = 0;
      bool ok = true;
      for (int64_t g = g_begin; g < g_end && ok;) {
        int b, t0, t1, slot;
        segment(g, b, t0, t1, slot);
        const int nt = t1 - t0;
        if (!mbar_wait(rtfull_bar, rt_phase, p.d_status)) break;
        rt_phase ^= 1u;
        for (int i = 0; i < nt; ++i) {
          if (!mbar_wait(xa_full(st1), ph1, p.d_status)) { ok = false; break; }
          // the accumulator is free once the second product of the tile that used it last has retired
          if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, p.d_status)) { ok = false; break; }
          tc_fence_after();
          const uint64_t xd = x0 + (uint64_t)((st1 * XA_BYTES) >> 4);
          const uint32_t tmem_o = tmem_base + (uint32_t)(acc * TT);
#pragma unroll
          for (int kb = 0; kb < 2; ++kb)
#pragma unroll
            for (int k = 0; k < BLOCK_K / UMMA_K; ++k)
              umma_bf16(tmem_o, rd[kb * (BLOCK_K / UMMA_K) + k], xd + (uint64_t)((kb * XKB_BYTES + k * UMMA_K * 2) >> 4), IDESC_O,
                        (kb > 0 || k > 0) ? 1u : 0u);
          umma_commit(tfull_bar(acc));
          if (i == nt - 1) umma_commit(rtempty_bar);   // R_h^T may be replaced once these products retire
          if (++st1 == XA_STAGES) { st1 = 0; ph1 ^= 1u; }
          if (++acc == O_BUFS) { acc = 0; acc_phase ^= 1u; }
        }
        g += nt;
      }
    }
  } else if (warp == Q_WARP) {
    // ------------------------------------------------------------- issuer of the second product, Gq^T += G_t^T X_t
    // (a thread of its own: the two streams of products do not depend on each other's order)
    if (lane == 0) {
      const uint64_t xm0 = make_mnmajor_sw128_desc(xa_base, XKB_BYTES);
      int st2 = 0, a2 = 0;                        // a2: accumulator that holds G_t^T of the next product
      uint32_t g_phase = 0, q_phase = 0;
      bool ok = true;
      for (int64_t g = g_begin; g < g_end && ok;) {
        int b, t0, t1, slot;
        segment(g, b, t0, t1, slot);
        const int nt = t1 - t0;
        for (int j = 0; j < nt; ++j) {
          if (j == 0) {   // the accumulator of the previous segment has been read out
            if (!mbar_wait(qempty_bar, q_phase ^ 1u, p.d_status)) { ok = false; break; }
            q_phase ^= 1u;
          }
          if (!mbar_wait(gfull_bar(a2), g_phase, p.d_status)) { ok = false; break; }
          tc_fence_after();
          // A = G_t^T from tensor memory: 16 tokens = 8 columns; each epilogue warp left its 32 tokens at the
          // start of the 32 accumulator columns it read.  B = X_t^T (128 channels x 16 tokens per instruction)
          // straight from the token-major tile of stage st2: 16 tokens = 16 rows of 128 bytes; channels 64..127
          // sit in the stage's second k-block.
          const uint64_t xd = xm0 + (uint64_t)((st2 * XA_BYTES) >> 4);
          const uint32_t tmem_g = tmem_base + (uint32_t)(a2 * TT);
#pragma unroll
          for (int k = 0; k < TT / UMMA_K; ++k)
            umma_bf16_ts(tmem_q, tmem_g + (uint32_t)((k >> 1) * 32 + (k & 1) * 8), xd + (uint64_t)((k * UMMA_K * 128) >> 4), IDESC_Q,
                         (j > 0 || k > 0) ? 1u : 0u);
          umma_commit(xa_empty(st2));                  // X_t can be replaced once this product has retired
          umma_commit(tempty_bar(a2));                 // and so can the accumulator that held O^T, then G_t^T
          if (j == nt - 1) umma_commit(qfull_bar);
          if (++st2 == XA_STAGES) { st2 = 0; }
          if (++a2 == O_BUFS) { a2 = 0; g_phase ^= 1u; }
        }
        g += nt;
      }
    }
  } else {
    // ------------------------------------------------------------- epilogue (warps 2..17)
    const int q = warp & 3;                    // quarter of the tensor-memory lanes this warp may read
    const int cg = (warp - 2) >> 2;            // which 32 of the tile's 128 token columns / of Gq^T's 128 columns
    const int row = q * 32 + lane;             // output channel (row of O^T, G^T and Gq^T)
    const uint32_t lane_addr = (uint32_t)(q * 32) << 16;
    int acc = 0;
    uint32_t acc_phase = 0, q_phase = 0;
    bool ok = true;
    for (int64_t g = g_begin; g < g_end && ok;) {
      int b, t0, t1, slot;
      segment(g, b, t0, t1, slot);
      float esum = 0.f;
      for (int t = t0; t < t1; ++t) {
        // ---- Eq. 4 epilogue of O^T
        if (!mbar_wait(tfull_bar(acc), acc_phase, p.d_status)) { ok = false; break; }
        tc_fence_after();
        {   // this warp's 32 token columns of the TT-wide tile
          const uint32_t taddr = tmem_base + lane_addr + (uint32_t)(acc * TT + cg * 32);
          uint32_t v[32];
          tmem_ld32(taddr, v);
          tmem_ld_wait();
          uint32_t packed[16];
          float amin0 = 1.f, amin1 = 1.f;       // smallest |o| of the 32: dL/do is 0, not -+1, where o is exactly 0
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const float o0 = __uint_as_float(v[2 * i]), o1 = __uint_as_float(v[2 * i + 1]);
            const float e0 = fast_exp_neg_abs(o0), e1 = fast_exp_neg_abs(o1);
            esum += e0 + e1;
            amin0 = fminf(amin0, fabsf(o0)); amin1 = fminf(amin1, fabsf(o1));
            const __nv_bfloat162 h = __floats2bfloat162_rn(copysignf(e0, -o0), copysignf(e1, -o1));
            packed[i] = *reinterpret_cast<const uint32_t*>(&h);
          }
          // (an exact zero is not rare at a Hadamard start, where o is a signed sum of bf16 values times one
          // constant; everywhere else it is, so the per-element test stays out of the loop above)
          if (fminf(amin0, amin1) == 0.f) {
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              if (__uint_as_float(v[2 * i]) == 0.f) packed[i] &= 0xFFFF0000u;
              if (__uint_as_float(v[2 * i + 1]) == 0.f) packed[i] &= 0x0000FFFFu;
            }
          }
          // tokens 32 cg .. 32 cg + 31 of row `row` as 16 columns of bf16 pairs, over the first half of the 32
          // columns this warp has just read (no other warp reads or writes them)
          tmem_st16(taddr, packed);
          if (p.Gt) {
            uint4* dst = reinterpret_cast<uint4*>(p.Gt + ((int64_t)b * 128 + row) * p.n_tokens + (int64_t)t * TT + cg * 32);
#pragma unroll
            for (int i = 0; i < 4; ++i)
              dst[i] = make_uint4(packed[4 * i], packed[4 * i + 1], packed[4 * i + 2], packed[4 * i + 3]);
          }
        }
        tmem_st_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(gfull_bar(acc));
        if (++acc == O_BUFS) { acc = 0; acc_phase ^= 1u; }
      }
      if (!ok) break;
      // partial Gq of the segment
      if (!mbar_wait(qfull_bar, q_phase, p.d_status)) { ok = false; break; }
      q_phase ^= 1u;
      tc_fence_after();
      // the accumulator holds Gq^T (lane = output channel, column = input channel): a warp's store of one
      // column is 32 consecutive floats of a row of Gq
      const int64_t pslot = (int64_t)b * p.slots + slot;
      float* dst_col = p.part + pslot * 128 * 128 + row;
      {
        uint32_t v[32];
        tmem_ld32(tmem_q + lane_addr + (uint32_t)(cg * 32), v);
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 32; ++i) dst_col[(cg * 32 + i) * 128] = __uint_as_float(v[i]);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(qempty_bar);
#pragma unroll
      for (int off = 16; off >= 1; off >>= 1) esum += __shfl_xor_sync(0xffffffffu, esum, off);
      if (lane == 0) p.partials[pslot * EPI_WARPS + (warp - 2)] = esum;
      g += t1 - t0;
    }
  }

  // ------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

}  // namespace heads
}  // namespace dq
