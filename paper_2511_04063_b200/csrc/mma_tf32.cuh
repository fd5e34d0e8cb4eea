// Warp-level tensor-core helpers for fp32 matrices held in shared memory: mma.sync m16n8k8 with
// tf32 inputs, each fp32 value split in two tf32 terms so that three products (hi*hi + hi*lo +
// lo*hi) recover fp32-like accuracy (about 2^-22 relative).
#pragma once
#include <stdint.h>

namespace dq {
namespace mma {

__device__ __forceinline__ void split_tf32(float x, uint32_t& hi, uint32_t& lo) {
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(hi) : "f"(x));
  const float r = x - __uint_as_float(hi);
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(lo) : "f"(r));
}

// D += A B for one 16 x 8 x 8 tile (A row-major M x K, B column-major K x N), fp32 accumulate.
__device__ __forceinline__ void mma_tf32(float (&c)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
  asm volatile(
      "mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}

// One warp: acc (a 32 x 32 block of C at rows r0.., columns c0.., as [m-tile][n-tile][fragment]) +=
// sum over k in [kb, ke) of opA(r, k) opB(k, c) with opA(r, k) = TA ? A[k * ld + r] : A[r * ld + k]
// and opB(k, c) = TB ? B[c * ld + k] : B[k * ld + c].  kb, ke multiples of 8.
// Fragment e of tile (mt, nt) is C[r0 + 16 mt + g + 8 (e >> 1)][c0 + 8 nt + 2 t + (e & 1)],
// g = lane >> 2, t = lane & 3.
template <bool TA, bool TB>
__device__ __forceinline__ void warp_mm32(const float* __restrict__ A, const float* __restrict__ B, int ld,
                                          float (&acc)[2][4][4], int r0, int c0, int kb, int ke, int lane) {
  const int g = lane >> 2, t = lane & 3;
#pragma unroll 1
  for (int k0 = kb; k0 < ke; k0 += 8) {
    uint32_t bh[4][2], bl[4][2];
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) {
      const int c = c0 + 8 * nt + g;
      const float b0 = TB ? B[c * ld + k0 + t] : B[(k0 + t) * ld + c];
      const float b1 = TB ? B[c * ld + k0 + t + 4] : B[(k0 + t + 4) * ld + c];
      split_tf32(b0, bh[nt][0], bl[nt][0]);
      split_tf32(b1, bh[nt][1], bl[nt][1]);
    }
#pragma unroll
    for (int mt = 0; mt < 2; ++mt) {
      const int r = r0 + 16 * mt + g;
      uint32_t ah[4], al[4];
      const float a0 = TA ? A[(k0 + t) * ld + r] : A[r * ld + k0 + t];
      const float a1 = TA ? A[(k0 + t) * ld + r + 8] : A[(r + 8) * ld + k0 + t];
      const float a2 = TA ? A[(k0 + t + 4) * ld + r] : A[r * ld + k0 + t + 4];
      const float a3 = TA ? A[(k0 + t + 4) * ld + r + 8] : A[(r + 8) * ld + k0 + t + 4];
      split_tf32(a0, ah[0], al[0]);
      split_tf32(a1, ah[1], al[1]);
      split_tf32(a2, ah[2], al[2]);
      split_tf32(a3, ah[3], al[3]);
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) {
        mma_tf32(acc[mt][nt], al, bh[nt]);
        mma_tf32(acc[mt][nt], ah, bl[nt]);
        mma_tf32(acc[mt][nt], ah, bh[nt]);
      }
    }
  }
}

__device__ __forceinline__ void zero_acc(float (&acc)[2][4][4]) {
#pragma unroll
  for (int mt = 0; mt < 2; ++mt)
#pragma unroll
    for (int nt = 0; nt < 4; ++nt)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[mt][nt][e] = 0.f;
}

}  // namespace mma
}  // namespace dq
