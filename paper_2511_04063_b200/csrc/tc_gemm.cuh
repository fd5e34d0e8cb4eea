// tcgen05 / TMEM / TMA GEMM building block for sm_100a.
//
//   D[m][n] = sum_k A[m][k] * B[n][k]       (both operands K-major, bf16, fp32 accumulate)
//
// One persistent CTA per SM, 192 threads:
//   warp 0      TMA producer      (cp.async.bulk.tensor, 128-byte swizzle, mbarrier complete_tx)
//   warp 1      MMA issuer        (tcgen05.mma cta_group::1, M = 128, N = BLOCK_N, K = 16 per instruction)
//   warps 2..5  epilogue          (tcgen05.ld from one of two TMEM accumulator buffers)
// The two TMEM buffers let the epilogue of tile i overlap the main loop of tile i+1.
// With NTERMS == 3 every operand comes as a (hi, lo) bf16 pair and three products
// hi*hi + hi*lo + lo*hi are accumulated: ~2^-16 relative accuracy ("split bf16").
// Every wait is bounded; on expiry the kernel records DQ_ERR_TIMEOUT and unwinds.
#pragma once
#include <cuda.h>

#include "common.cuh"

namespace dq {
namespace tc {

constexpr int BLOCK_M = 128;
constexpr int BLOCK_K = 64;          // 64 bf16 = 128 bytes = one swizzle row
constexpr int UMMA_K = 16;
constexpr int NUM_THREADS = 192;
constexpr uint64_t WAIT_LIMIT_NS = 4000000000ull;

enum { EPI_WHIP = 0, EPI_GEN = 1, EPI_BF16 = 2 };

struct Params {
  int m_blocks, n_blocks, batch, ksplit;
  int k_blocks;            // K / 64 (whole reduction)
  // output addressing: out + b * batch_stride + split * split_stride + m * ld + n
  void* out;               // EPI_WHIP / EPI_BF16: bf16; EPI_GEN: fp32 (nullable)
  int64_t ld, batch_stride, split_stride;
  // EPI_GEN only: v = alpha * acc + beta * out_old; optional split-bf16 copy (hi + lo ~ v)
  __nv_bfloat16* out_hi;
  __nv_bfloat16* out_lo;
  int64_t ld_h, batch_stride_h;
  float alpha, beta;
  float* partials;         // EPI_WHIP: [unit][4] loss partial sums
  int* d_status;
  // Triangular structure (square tiles, ksplit == 1).  tri_skip: tiles below the block diagonal
  // (mb > nb) are not computed.  k_mode bits restrict the reduction of tile (mb, nb) to the
  // k-range where both operands can be non-zero:
  //   1: A[m][k] = 0 for k <  128 mb        2: A[m][k] = 0 for k >= 128 (mb + 1)
  //   4: B[n][k] = 0 for k >= 128 (nb + 1)  8: B[n][k] = 0 for k <  128 nb
  int tri_skip, k_mode;
  // Optional explicit tile order (device array of mb | nb << 16, n_list entries per problem), e.g.
  // most expensive tiles first so that the round-robin deal over the persistent CTAs is balanced.
  const int* tile_list;
  int n_list;
  // Optional device flag: the kernel does nothing when *run_if == 0 (lets a fixed launch sequence, e.g. a
  // captured graph, stop a data-dependent iteration early).  nullptr: always run.
  const int* run_if;
};

// ----------------------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait: false (and DQ_ERR_TIMEOUT in the status word) after WAIT_LIMIT_NS.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, int* d_status) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = global_timer_ns();
  uint32_t spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    __nanosleep(32);   // leave the issue slots to the warps that have work
    if ((++spins & 0xFFu) == 0u && global_timer_ns() - t0 > WAIT_LIMIT_NS) {
      set_status(d_status, DQ_ERR_TIMEOUT);
      return false;
    }
  }
  return true;
}

__device__ __forceinline__ void tma_load_3d(uint32_t smem_dst, const CUtensorMap* map, uint32_t bar,
                                            int c0, int c1, int c2) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(smem_dst), "l"((uint64_t)map), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"((uint64_t)map) : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t smem_result, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_result), "r"(ncols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// The mbarrier gets one arrival once every MMA issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 32 lanes x 32 consecutive fp32 columns: thread l receives row (lane base + l).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor: K-major tile, rows of 128 bytes, 128-byte swizzle,
// 8-row groups 1024 bytes apart (version 1 = sm_100).
__device__ __forceinline__ uint64_t make_kmajor_sw128_desc(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)1 << 16;                 // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;       // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                 // descriptor version
  d |= (uint64_t)2 << 61;                 // SWIZZLE_128B
  return d;
}
// kind::f16 instruction descriptor: bf16 x bf16 -> fp32, both K-major, M = 128.
__host__ __device__ constexpr uint32_t make_idesc_bf16(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(BLOCK_M >> 4) << 24);
}

__device__ __forceinline__ float fast_exp_neg_abs(float o) {
  float r;
  const float t = -fabsf(o) * 1.4426950408889634f;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(t));
  return r;
}

template <int BLOCK_N, int NTERMS>
struct SmemLayout {
  static constexpr int A_BYTES = BLOCK_M * BLOCK_K * 2;
  static constexpr int B_BYTES = BLOCK_N * BLOCK_K * 2;
  static constexpr int NOPS = (NTERMS == 1) ? 1 : 2;           // hi only, or hi + lo
  static constexpr int STAGE_BYTES = NOPS * (A_BYTES + B_BYTES);
  static constexpr int STAGES = (196608 / STAGE_BYTES) > 8 ? 8 : (196608 / STAGE_BYTES);
  static constexpr int BAR_BYTES = 1024;
  static constexpr int TOTAL = STAGES * STAGE_BYTES + BAR_BYTES + 1024;   // + alignment slack
};

// ----------------------------------------------------------------------------- kernel
template <int BLOCK_N, int NTERMS, int EPI>
__global__ void __launch_bounds__(NUM_THREADS, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapB,
               const __grid_constant__ CUtensorMap mapA_lo, const __grid_constant__ CUtensorMap mapB_lo,
               const Params p) {
  if (p.run_if && *p.run_if == 0) return;                     // uniform over the grid: nothing is allocated yet
  using L = SmemLayout<BLOCK_N, NTERMS>;
  constexpr int STAGES = L::STAGES;
  constexpr uint32_t TMEM_COLS = 2 * BLOCK_N;                 // 256 or 512: power of two
  constexpr uint32_t IDESC = make_idesc_bf16(BLOCK_N);

  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t bar_base = smem_base + STAGES * L::STAGE_BYTES;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
  auto tfull_bar = [&](int b) { return bar_base + 8u * (2 * STAGES + b); };
  auto tempty_bar = [&](int b) { return bar_base + 8u * (2 * STAGES + 2 + b); };
  const uint32_t tmem_slot = bar_base + 8u * (2 * STAGES + 4);
  uint32_t* tmem_slot_ptr = reinterpret_cast<uint32_t*>(smem_raw + (tmem_slot - smem_u32(smem_raw)));

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), 4); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    prefetch_tensormap(&mapA);
    prefetch_tensormap(&mapB);
    if (NTERMS > 1) { prefetch_tensormap(&mapA_lo); prefetch_tensormap(&mapB_lo); }
  }
  if (warp == 1) tmem_alloc(tmem_slot, TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot_ptr;

  const int tiles_per_batch = p.tile_list ? p.n_list : p.m_blocks * p.n_blocks;
  auto tile_of = [&](int r, int& mb, int& nb) {
    if (p.tile_list) { const int code = p.tile_list[r]; mb = code & 0xffff; nb = code >> 16; }
    else { mb = r % p.m_blocks; nb = r / p.m_blocks; }   // m fastest: neighbours share the B tile
  };
  const int units = tiles_per_batch * p.batch * p.ksplit;
  // split s of the reduction covers k-blocks [s * k_blocks / ksplit, (s + 1) * k_blocks / ksplit);
  // with k_mode the range is clipped to the non-zero part of triangular operands.
  auto k_range = [&](int split, int mb, int nb, int& k0, int& kn) {
    int lo = (int)(((int64_t)split * p.k_blocks) / p.ksplit);
    int hi = (int)(((int64_t)(split + 1) * p.k_blocks) / p.ksplit);
    if (p.k_mode) {
      constexpr int R = BLOCK_M / BLOCK_K;   // k-blocks per 128 rows
      if ((p.k_mode & 1) && lo < R * mb) lo = R * mb;
      if ((p.k_mode & 8) && lo < R * nb) lo = R * nb;
      if ((p.k_mode & 2) && hi > R * (mb + 1)) hi = R * (mb + 1);
      if ((p.k_mode & 4) && hi > R * (nb + 1)) hi = R * (nb + 1);
    }
    k0 = lo; kn = hi - lo;
  };

  if (warp == 0) {
    // ------------------------------------------------------------- TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int u = blockIdx.x; u < units && ok; u += gridDim.x) {
        const int split = u % p.ksplit;
        const int t = u / p.ksplit;
        const int b = t / tiles_per_batch;
        const int r = t % tiles_per_batch;
        int mb, nb;
        tile_of(r, mb, nb);
        if (p.tri_skip && mb > nb) continue;
        int k0, kb_per_split;
        k_range(split, mb, nb, k0, kb_per_split);
        for (int kb = 0; kb < kb_per_split; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, p.d_status)) { ok = false; break; }
          mbar_expect_tx(full_bar(stage), L::STAGE_BYTES);
          const uint32_t sa = smem_base + stage * L::STAGE_BYTES;
          const uint32_t sb = sa + L::NOPS * L::A_BYTES;
          const int kc = (k0 + kb) * BLOCK_K;
          tma_load_3d(sa, &mapA, full_bar(stage), kc, mb * BLOCK_M, b);
          tma_load_3d(sb, &mapB, full_bar(stage), kc, nb * BLOCK_N, b);
          if (NTERMS > 1) {
            tma_load_3d(sa + L::A_BYTES, &mapA_lo, full_bar(stage), kc, mb * BLOCK_M, b);
            tma_load_3d(sb + L::B_BYTES, &mapB_lo, full_bar(stage), kc, nb * BLOCK_N, b);
          }
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int u = blockIdx.x; u < units && ok; u += gridDim.x) {
        const int split = u % p.ksplit;
        const int rr = (u / p.ksplit) % tiles_per_batch;
        int mb, nb;
        tile_of(rr, mb, nb);
        if (p.tri_skip && mb > nb) continue;
        int k0_unused, kb_per_split;
        k_range(split, mb, nb, k0_unused, kb_per_split);
        if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, p.d_status)) { ok = false; break; }
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + (uint32_t)(acc * BLOCK_N);
        for (int kb = 0; kb < kb_per_split; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, p.d_status)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = smem_base + stage * L::STAGE_BYTES;
          const uint32_t sb = sa + L::NOPS * L::A_BYTES;
#pragma unroll
          for (int k = 0; k < BLOCK_K / UMMA_K; ++k) {
            const uint64_t a_hi = make_kmajor_sw128_desc(sa + k * UMMA_K * 2);
            const uint64_t b_hi = make_kmajor_sw128_desc(sb + k * UMMA_K * 2);
            umma_bf16(tmem_d, a_hi, b_hi, IDESC, (kb > 0 || k > 0) ? 1u : 0u);
            if (NTERMS > 1) {
              const uint64_t a_lo = make_kmajor_sw128_desc(sa + L::A_BYTES + k * UMMA_K * 2);
              const uint64_t b_lo = make_kmajor_sw128_desc(sb + L::B_BYTES + k * UMMA_K * 2);
              umma_bf16(tmem_d, a_hi, b_lo, IDESC, 1u);
              umma_bf16(tmem_d, a_lo, b_hi, IDESC, 1u);
            }
          }
          umma_commit(empty_bar(stage));       // smem slot reusable once these MMAs retire
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        umma_commit(tfull_bar(acc));           // accumulator complete
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else {
    // ------------------------------------------------------------- epilogue (warps 2..5)
    const int q = warp & 3;                    // TMEM lane quarter this warp may read
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    for (int u = blockIdx.x; u < units && ok; u += gridDim.x) {
      const int split = u % p.ksplit;
      const int t = u / p.ksplit;
      const int b = t / tiles_per_batch;
      const int r = t % tiles_per_batch;
      int mb, nb;
      tile_of(r, mb, nb);
      if (p.tri_skip && mb > nb) continue;
      const int row = mb * BLOCK_M + q * 32 + lane;
      const int64_t out_off = (int64_t)b * p.batch_stride + (int64_t)split * p.split_stride +
                              (int64_t)row * p.ld + (int64_t)nb * BLOCK_N;
      // Accumulating epilogue (beta != 0): fetch the old output row while the MMAs of this tile
      // are still running, so the global-load latency is not paid once per 32-column chunk.
      constexpr bool PREFETCH = (EPI == EPI_GEN && BLOCK_N == 128);
      float4 old[PREFETCH ? 32 : 1];
      const bool use_old = PREFETCH && p.out != nullptr && p.beta != 0.f;
      if (PREFETCH && use_old) {
        const float4* src = reinterpret_cast<const float4*>(reinterpret_cast<const float*>(p.out) + out_off);
#pragma unroll
        for (int i = 0; i < (PREFETCH ? 32 : 1); ++i) old[i] = src[i];
      }
      if (!mbar_wait(tfull_bar(acc), acc_phase, p.d_status)) { ok = false; break; }
      tc_fence_after();
      float esum = 0.f;
#pragma unroll(PREFETCH ? 4 : 1)
      for (int c = 0; c < BLOCK_N / 32; ++c) {
        uint32_t v[32];
        tmem_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * BLOCK_N + c * 32), v);
        tmem_ld_wait();
        if (EPI == EPI_WHIP) {
          // Eq. 4: e = exp(-|o|); dL/do = -sign(o) e, zero at o = 0; 1/N is applied later.
          uint32_t packed[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const float o0 = __uint_as_float(v[2 * i]), o1 = __uint_as_float(v[2 * i + 1]);
            const float e0 = fast_exp_neg_abs(o0), e1 = fast_exp_neg_abs(o1);
            esum += e0 + e1;
            const float g0 = (o0 == 0.f) ? 0.f : copysignf(e0, -o0);
            const float g1 = (o1 == 0.f) ? 0.f : copysignf(e1, -o1);
            const __nv_bfloat162 h = __floats2bfloat162_rn(g0, g1);
            packed[i] = *reinterpret_cast<const uint32_t*>(&h);
          }
          uint4* dst = reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(p.out) + out_off + c * 32);
#pragma unroll
          for (int i = 0; i < 4; ++i)
            dst[i] = make_uint4(packed[4 * i], packed[4 * i + 1], packed[4 * i + 2], packed[4 * i + 3]);
        } else if (EPI == EPI_GEN) {
          float f[32];
#pragma unroll
          for (int i = 0; i < 32; ++i) f[i] = p.alpha * __uint_as_float(v[i]);
          if (p.out) {
            float4* dst = reinterpret_cast<float4*>(reinterpret_cast<float*>(p.out) + out_off + c * 32);
            if (p.beta != 0.f) {
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                const float4 o = PREFETCH ? old[PREFETCH ? c * 8 + i : 0] : dst[i];
                f[4 * i] = fmaf(p.beta, o.x, f[4 * i]); f[4 * i + 1] = fmaf(p.beta, o.y, f[4 * i + 1]);
                f[4 * i + 2] = fmaf(p.beta, o.z, f[4 * i + 2]); f[4 * i + 3] = fmaf(p.beta, o.w, f[4 * i + 3]);
              }
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) dst[i] = make_float4(f[4 * i], f[4 * i + 1], f[4 * i + 2], f[4 * i + 3]);
          }
          if (p.out_hi) {
            const int64_t off_h = (int64_t)b * p.batch_stride_h + (int64_t)row * p.ld_h + (int64_t)nb * BLOCK_N + c * 32;
            uint32_t ph[16], pl[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const __nv_bfloat162 h = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
              const float2 hf = __bfloat1622float2(h);
              const __nv_bfloat162 l = __floats2bfloat162_rn(f[2 * i] - hf.x, f[2 * i + 1] - hf.y);
              ph[i] = *reinterpret_cast<const uint32_t*>(&h);
              pl[i] = *reinterpret_cast<const uint32_t*>(&l);
            }
            uint4* dh = reinterpret_cast<uint4*>(p.out_hi + off_h);
            uint4* dl = reinterpret_cast<uint4*>(p.out_lo + off_h);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              dh[i] = make_uint4(ph[4 * i], ph[4 * i + 1], ph[4 * i + 2], ph[4 * i + 3]);
              dl[i] = make_uint4(pl[4 * i], pl[4 * i + 1], pl[4 * i + 2], pl[4 * i + 3]);
            }
          }
        } else {
          uint32_t packed[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(v[2 * i]), __uint_as_float(v[2 * i + 1]));
            packed[i] = *reinterpret_cast<const uint32_t*>(&h);
          }
          uint4* dst = reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(p.out) + out_off + c * 32);
#pragma unroll
          for (int i = 0; i < 4; ++i)
            dst[i] = make_uint4(packed[4 * i], packed[4 * i + 1], packed[4 * i + 2], packed[4 * i + 3]);
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty_bar(acc));      // this warp is done with the accumulator
      if (EPI == EPI_WHIP) {
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) esum += __shfl_xor_sync(0xffffffffu, esum, off);
        if (lane == 0) p.partials[(int64_t)u * 4 + q] = esum;
      }
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
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

}  // namespace tc
}  // namespace dq
