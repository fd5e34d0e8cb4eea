// Two-CTA variant of the tcgen05 GEMM building block: a pair of CTAs on neighbouring SMs (a
// cluster of two) computes one 256 x 256 output tile with `tcgen05.mma.cta_group::2`.
//
//   D[m][n] = sum_k A[m][k] * B[n][k]       (both operands K-major bf16, fp32 accumulate)
//
// Each CTA stages only its own half of the operands (128 rows of A, 128 rows of B: 32 KB per
// 64-wide k-block instead of 48 KB) and owns the 128 x 256 accumulator rows of its half in its own
// TMEM; the MMAs of both halves are issued by the even-ranked CTA ("leader"), which reads the
// peer's operands from the same shared-memory offsets.  Protocol per CTA (192 threads as in the
// one-CTA kernel):
//   warp 0   TMA producer: waits on its own empty barrier (armed for both CTAs by the leader's
//            commit to both CTAs); both CTAs' loads complete on the LEADER's full barrier
//   warp 1   leader only: MMA issue; its commits arrive on both CTAs' empty / accumulator-full barriers
//   warps 2..5  epilogue from the CTA's own TMEM; both CTAs arrive on the leader's accumulator-empty
//            barrier
// Every TMA load is a plain per-CTA copy.  Every wait is bounded (DQ_ERR_TIMEOUT in the status word on expiry).
#pragma once
#include "tc_gemm.cuh"

namespace dq {
namespace tc2 {

using namespace tc;

constexpr int PAIR_M = 256, PAIR_N = 256;
constexpr int HALF = 128;
constexpr int A_BYTES = HALF * BLOCK_K * 2;
constexpr int B_BYTES = HALF * BLOCK_K * 2;
// NTERMS = 1: plain bf16 product.  NTERMS = 3: split-bf16 operands (hi, lo), three MMAs per product
// (hi hi + hi lo + lo hi), about 2^-17 relative.
template <int NTERMS>
struct PairSmem {
  static constexpr int NOPS = (NTERMS == 1) ? 1 : 2;
  static constexpr int KBLOCK_BYTES = NOPS * (A_BYTES + B_BYTES);    // one k-block of 64, per CTA: 32 KB or 64 KB
  // A stage of the plain product holds two k-blocks: half as many barrier round trips between the producer and
  // the MMA issuer per tile (each costs the issuer some tens of the 256 cycles a k-block's MMAs take).
  static constexpr int KPS = (NTERMS == 1) ? 2 : 1;
  static constexpr int STAGE_BYTES = KPS * KBLOCK_BYTES;             // 64 KB
  static constexpr int STAGES = 3;
  static constexpr int TOTAL = STAGES * STAGE_BYTES + 1024 + 1024;
};
// Epilogue warps per CTA: the general epilogue is a chain of dependent steps per 16-column chunk (tensor-memory
// load, addends from global memory, stores), so it runs on eight warps, two per quarter of the tensor-memory lanes,
// each taking half of the tile's columns; the Whip and bf16 epilogues keep four.
template <int EPI> __host__ __device__ constexpr int epi_warps() { return EPI == EPI_GEN ? 8 : 4; }
template <int EPI> __host__ __device__ constexpr int pair_threads() { return 64 + 32 * epi_warps<EPI>(); }

constexpr uint32_t PEER_MASK = 0xFEFFFFFFu;             // clears the bit that separates the two CTAs of a pair
constexpr uint32_t TMEM_COLS = 512;                     // two 256-column accumulators

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Load a tile into this CTA's shared memory; the bytes are counted on the leader's barrier.
__device__ __forceinline__ void tma_load_3d_pair(uint32_t smem_dst, const CUtensorMap* map, uint32_t bar, int c0, int c1,
                                                 int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(smem_dst), "l"((uint64_t)map), "r"(bar & PEER_MASK), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
// This CTA's half of an operand tile of a stage (128 rows of the operand x 64 k): one box K-major, two boxes MN-major.
__device__ __forceinline__ void load_operand_pair(uint32_t smem_dst, const CUtensorMap* map, uint32_t bar, int kc,
                                                  int row0, int b, int mn) {
  if (!mn) { tma_load_3d_pair(smem_dst, map, bar, kc, row0, b); return; }
  tma_load_3d_pair(smem_dst, map, bar, row0, kc, b);
  tma_load_3d_pair(smem_dst + MN_BOX_BYTES, map, bar, row0 + 64, kc, b);
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t smem_result, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_result), "r"(ncols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                               uint32_t accumulate) {
  const uint32_t z = 0u;
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, {%5, %6, %7, %8, %9, %10, %11, %12}, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate), "r"(z), "r"(z), "r"(z), "r"(z), "r"(z), "r"(z),
        "r"(z), "r"(z)
      : "memory");
}
// One arrival on the barrier at this offset in BOTH CTAs once every MMA issued so far has completed.
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
  const uint16_t mask = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"(mask) : "memory");
}
// Arrive on the leader's copy of a barrier (from either CTA of the pair).
__device__ __forceinline__ void mbar_arrive_leader(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(bar & PEER_MASK) : "memory");
}
// kind::f16 instruction descriptor: bf16 x bf16 -> fp32, both K-major, M = 256 over the pair, N = 256.
__host__ __device__ constexpr uint32_t make_idesc_bf16_pair() {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(PAIR_N >> 3) << 17) | ((uint32_t)(PAIR_M >> 4) << 24);
}

// Params as in the one-CTA kernel; m_blocks / n_blocks count 256 x 256 pair tiles, tile_list entries
// are mb | nb << 16 in those units (tri_skip and k_mode refer to them too), partials get eight values
// per tile (CTA rank, lane quarter).
template <int NTERMS, int EPI>
__global__ void __launch_bounds__(pair_threads<EPI>(), 1)
tc_gemm2_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB,
                const __grid_constant__ CUtensorMap mapA_lo, const __grid_constant__ CUtensorMap mapB_lo,
                const Params p) {
  if ((p.run_if && *p.run_if == 0) || (p.run_unless && *p.run_unless != 0)) return;   // uniform over the grid (both CTAs of every pair)
  using L = PairSmem<NTERMS>;
  constexpr int STAGES = L::STAGES;
  constexpr int STAGE_BYTES = L::STAGE_BYTES;
  constexpr int KPS = L::KPS, KBLOCK_BYTES = L::KBLOCK_BYTES;
  constexpr uint32_t IDESC = make_idesc_bf16_pair();
  constexpr int EPI_WARPS = epi_warps<EPI>();
  constexpr int N_EPI = PAIR_N / (EPI_WARPS / 4);   // columns of the tile one epilogue warp handles
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bar_base = smem_base + STAGES * STAGE_BYTES;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
  auto tfull_bar = [&](int b) { return bar_base + 8u * (2 * STAGES + b); };
  auto tempty_bar = [&](int b) { return bar_base + 8u * (2 * STAGES + 2 + b); };
  const uint32_t tmem_slot = bar_base + 8u * (2 * STAGES + 4);
  uint32_t* tmem_slot_ptr = reinterpret_cast<uint32_t*>(smem_raw + (tmem_slot - smem_u32(smem_raw)));

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();          // 0 = leader
  const bool leader = rank == 0;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), 2 * EPI_WARPS); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    prefetch_tensormap(&mapA);
    prefetch_tensormap(&mapB);
    if (NTERMS > 1 || p.k_dual) { prefetch_tensormap(&mapA_lo); prefetch_tensormap(&mapB_lo); }
  }
  if (warp == 1) tmem_alloc_pair(tmem_slot, TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                               // both CTAs' barriers exist before any remote arrival
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot_ptr;

  const int tiles_per_batch = p.tile_list ? p.n_list : p.m_blocks * p.n_blocks;
  auto tile_of = [&](int r, int& mb, int& nb) {
    if (p.tile_list) { const int code = p.tile_list[r]; mb = code & 0xffff; nb = code >> 16; }
    else { mb = r % p.m_blocks; nb = r / p.m_blocks; }
  };
  // as in the one-CTA kernel; k_mode clips the range to the non-zero part of triangular operands
  auto k_range = [&](int split, int mb, int nb, int& k0, int& kn) {
    int lo = (int)(((int64_t)split * p.k_blocks) / p.ksplit);
    int hi = (int)(((int64_t)(split + 1) * p.k_blocks) / p.ksplit);
    if (p.k_mode) {
      constexpr int R = PAIR_M / BLOCK_K;   // k-blocks per 256 rows
      if ((p.k_mode & 1) && lo < R * mb) lo = R * mb;
      if ((p.k_mode & 8) && lo < R * nb) lo = R * nb;
      if ((p.k_mode & 2) && hi > R * (mb + 1)) hi = R * (mb + 1);
      if ((p.k_mode & 4) && hi > R * (nb + 1)) hi = R * (nb + 1);
    }
    k0 = lo; kn = hi - lo;
  };
  const int units = tiles_per_batch * p.batch * p.ksplit;
  const int pair = blockIdx.x >> 1, pairs = gridDim.x >> 1;

  if (warp == 0) {
    // ------------------------------------------------------------- TMA producer (both CTAs)
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int u = pair; u < units && ok; u += pairs) {
        const int split = u % p.ksplit;
        const int t = u / p.ksplit;
        const int b = t / tiles_per_batch;
        int mb, nb;
        tile_of(t % tiles_per_batch, mb, nb);
        if (p.tri_skip && mb > nb) continue;
        int k0, kn;
        k_range(split, mb, nb, k0, kn);
        const int kb_total = (NTERMS == 1 && p.k_dual) ? 2 * kn : kn;
        const int ra = mb * PAIR_M + (int)rank * HALF, rb = nb * PAIR_N + (int)rank * HALF;
        for (int kb0 = 0; kb0 < kb_total; kb0 += KPS) {
          const int nk = (kb_total - kb0 < KPS) ? kb_total - kb0 : KPS;   // k-blocks in this stage
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, p.d_status)) { ok = false; break; }
          if (leader) mbar_expect_tx(full_bar(stage), 2 * nk * KBLOCK_BYTES);
#pragma unroll
          for (int j = 0; j < KPS; ++j) {
            if (j >= nk) break;
            const int kb = kb0 + j;
            const uint32_t sa = smem_base + stage * STAGE_BYTES + j * KBLOCK_BYTES;
            const uint32_t sb = sa + L::NOPS * A_BYTES;
            const bool second = kb >= kn;                   // second operand pair of a dual reduction
            const int kc = (k0 + (second ? kb - kn : kb)) * BLOCK_K;
            load_operand_pair(sa, second ? &mapA_lo : &mapA, full_bar(stage), kc, ra, b, p.a_mn);
            load_operand_pair(sb, second ? &mapB_lo : &mapB, full_bar(stage), kc, rb, b, p.b_mn);
            if (NTERMS > 1) {
              load_operand_pair(sa + A_BYTES, &mapA_lo, full_bar(stage), kc, ra, b, p.a_mn);
              load_operand_pair(sb + B_BYTES, &mapB_lo, full_bar(stage), kc, rb, b, p.b_mn);
            }
          }
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------- MMA issuer (leader CTA only)
    if (leader && lane == 0) {
      const int a_mn = p.a_mn, b_mn = p.b_mn;
      const uint32_t a_step = operand_desc_step(a_mn), b_step = operand_desc_step(b_mn);
      const uint32_t idesc_mn = IDESC | (a_mn ? IDESC_A_MN_MAJOR : 0u) | (b_mn ? IDESC_B_MN_MAJOR : 0u);
      const uint64_t a_stage0 = operand_desc0(smem_base, a_mn);                     // descriptors of stage 0
      const uint64_t b_stage0 = operand_desc0(smem_base + L::NOPS * A_BYTES, b_mn);
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int u = pair; u < units && ok; u += pairs) {
        int mb, nb;
        tile_of((u / p.ksplit) % tiles_per_batch, mb, nb);
        if (p.tri_skip && mb > nb) continue;
        int k0, kn;
        k_range(u % p.ksplit, mb, nb, k0, kn);
        if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, p.d_status)) { ok = false; break; }
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + (uint32_t)(acc * PAIR_N);
        const int kb_total = (NTERMS == 1 && p.k_dual) ? 2 * kn : kn;
        for (int kb0 = 0; kb0 < kb_total; kb0 += KPS) {
          const int nk = (kb_total - kb0 < KPS) ? kb_total - kb0 : KPS;
          // (nothing on the path from the barrier to the first MMA but one multiply-add per operand)
          const uint64_t a_st = a_stage0 + (uint64_t)(stage * (STAGE_BYTES >> 4));
          const uint64_t b_st = b_stage0 + (uint64_t)(stage * (STAGE_BYTES >> 4));
          if (!mbar_wait(full_bar(stage), phase, p.d_status)) { ok = false; break; }
          tc_fence_after();
#pragma unroll
          for (int j = 0; j < KPS; ++j) {
            if (j >= nk) break;
            const int kb = kb0 + j;
            const uint32_t idesc = (kb >= kn) ? (idesc_mn | IDESC_NEGATE_A) : idesc_mn;
            const uint64_t a0 = a_st + (uint64_t)(j * (KBLOCK_BYTES >> 4)), b0 = b_st + (uint64_t)(j * (KBLOCK_BYTES >> 4));
#pragma unroll
            for (int k = 0; k < BLOCK_K / UMMA_K; ++k) {
              const uint64_t a_hi = a0 + (uint64_t)(k * a_step);
              const uint64_t b_hi = b0 + (uint64_t)(k * b_step);
              umma_bf16_pair(tmem_d, a_hi, b_hi, idesc, (kb > 0 || k > 0) ? 1u : 0u);
              if (NTERMS > 1) {
                const uint64_t a_lo = a_hi + (uint64_t)(A_BYTES >> 4);
                const uint64_t b_lo = b_hi + (uint64_t)(B_BYTES >> 4);
                umma_bf16_pair(tmem_d, a_hi, b_lo, idesc_mn, 1u);
                umma_bf16_pair(tmem_d, a_lo, b_hi, idesc_mn, 1u);
              }
            }
          }
          umma_commit_pair(empty_bar(stage));      // both CTAs may refill this slot once the MMAs retire
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        umma_commit_pair(tfull_bar(acc));          // accumulator complete in both CTAs
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else {
    // ------------------------------------------------------------- epilogue (warps 2.., both CTAs)
    const int q = warp & 3;                                  // quarter of the tensor-memory lanes this warp may read
    const int col_off = ((warp - 2) >> 2) * N_EPI;           // its share of the tile's columns
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    for (int u = pair; u < units && ok; u += pairs) {
      const int split = u % p.ksplit;
      const int t = u / p.ksplit;
      const int b = t / tiles_per_batch;
      int mb, nb;
      tile_of(t % tiles_per_batch, mb, nb);
      if (p.tri_skip && mb > nb) continue;
      const int row = mb * PAIR_M + (int)rank * HALF + q * 32 + lane;
      const int64_t out_off = (int64_t)b * p.batch_stride + (int64_t)split * p.split_stride + (int64_t)row * p.ld +
                              (int64_t)nb * PAIR_N + col_off;
      // EPI_GEN: the addends of the first chunk are fetched while the MMAs of this tile are still running
      GenAddends g0;
      if (EPI == EPI_GEN) epi_gen_fetch(p, out_off, g0);
      if (!mbar_wait(tfull_bar(acc), acc_phase, p.d_status)) { ok = false; break; }
      tc_fence_after();
      float esum = 0.f;
      bool moved = false;
      if (EPI == EPI_GEN) {
        epi_gen_tile<N_EPI>(p, tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * PAIR_N + col_off), b, row,
                            nb * PAIR_N + col_off, out_off, g0, moved);
      } else {
#pragma unroll 1
        for (int c = 0; c < PAIR_N / 32; ++c) {
          uint32_t v[32];
          tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * PAIR_N + c * 32), v);
          tmem_ld_wait();
          uint32_t packed[16];
          if (EPI == EPI_WHIP) {
            // Eq. 4: e = exp(-|o|); dL/do = -sign(o) e, zero at o = 0; 1/N is applied later.
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const float o0 = __uint_as_float(v[2 * i]), o1 = __uint_as_float(v[2 * i + 1]);
              const float e0 = fast_exp_neg_abs(o0), e1 = fast_exp_neg_abs(o1);
              esum += e0 + e1;
              const float g0v = (o0 == 0.f) ? 0.f : copysignf(e0, -o0);
              const float g1v = (o1 == 0.f) ? 0.f : copysignf(e1, -o1);
              const __nv_bfloat162 h = __floats2bfloat162_rn(g0v, g1v);
              packed[i] = *reinterpret_cast<const uint32_t*>(&h);
            }
          } else {   // EPI_BF16: plain bf16 store
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(v[2 * i]), __uint_as_float(v[2 * i + 1]));
              packed[i] = *reinterpret_cast<const uint32_t*>(&h);
            }
          }
          uint4* dst = reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(p.out) + out_off + c * 32);
#pragma unroll
          for (int i = 0; i < 4; ++i)
            dst[i] = make_uint4(packed[4 * i], packed[4 * i + 1], packed[4 * i + 2], packed[4 * i + 3]);
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_leader(tempty_bar(acc));   // the arrivals of all epilogue warps of both CTAs free the accumulator
      if (EPI == EPI_GEN && moved) {
        if (p.moved_out) *p.moved_out = 1;
        if (p.fail_if_moved) set_status(p.d_status, DQ_ERR_NOT_CONVERGED);
      }
      if (EPI == EPI_WHIP) {
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) esum += __shfl_xor_sync(0xffffffffu, esum, off);
        if (lane == 0) p.partials[((int64_t)u * 2 + rank) * 4 + q] = esum;
      }
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
  }

  // ------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                               // the peer has finished with its TMEM and barriers too
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, TMEM_COLS);
  }
}

}  // namespace tc2
}  // namespace dq
