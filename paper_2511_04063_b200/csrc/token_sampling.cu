// Seeded token sampling / mini-batch selection (Algorithm 1: X <- token_sampling(X)): gathers
// rows X[pi(first)], ..., X[pi(first + count - 1)] for a seeded pseudo-random permutation pi of
// the token indices, i.e. uniform sampling without replacement; consecutive windows of pi are
// mini-batches, another seed is another epoch.
//
// pi = balanced Feistel network on 2w bits (2^(2w) >= n) with cycle walking; round function =
// Philox4x32-10 (Salmon et al., SC 2011), implemented from its published definition.
#include "common.cuh"

namespace dq {
namespace {

constexpr uint32_t PHILOX_M0 = 0xD2511F53u, PHILOX_M1 = 0xCD9E8D57u;
constexpr uint32_t PHILOX_W0 = 0x9E3779B9u, PHILOX_W1 = 0xBB67AE85u;
constexpr int FEISTEL_ROUNDS = 4;

// First output word of Philox4x32-10 for counter (c0, c1, 0, 0) and key (k0, k1).
__device__ __forceinline__ uint32_t philox4x32_10_word0(uint32_t c0, uint32_t c1, uint32_t k0, uint32_t k1) {
  uint32_t c2 = 0u, c3 = 0u;
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(PHILOX_M0, c0), lo0 = PHILOX_M0 * c0;
    const uint32_t hi1 = __umulhi(PHILOX_M1, c2), lo1 = PHILOX_M1 * c2;
    c0 = hi1 ^ c1 ^ k0; c1 = lo1; c2 = hi0 ^ c3 ^ k1; c3 = lo0;
    k0 += PHILOX_W0; k1 += PHILOX_W1;
  }
  return c0;
}

__device__ __forceinline__ int64_t permute_index(int64_t i, int64_t n, int w, uint64_t seed) {
  const uint32_t mask = (w >= 32) ? 0xFFFFFFFFu : ((1u << w) - 1u);
  const uint32_t k0 = (uint32_t)seed, k1 = (uint32_t)(seed >> 32);
  uint64_t x = (uint64_t)i;
  for (int guard = 0; guard < 4096; ++guard) {     // cycle walking: expected < 4 passes (2^(2w) < 4 n)
    uint32_t left = (uint32_t)(x >> w), right = (uint32_t)x & mask;
#pragma unroll
    for (int r = 0; r < FEISTEL_ROUNDS; ++r) {
      const uint32_t f = philox4x32_10_word0(right, (uint32_t)r, k0, k1) & mask;
      const uint32_t t = left ^ f;
      left = right; right = t;
    }
    x = ((uint64_t)left << w) | right;
    if (x < (uint64_t)n) return (int64_t)x;
  }
  return i;   // not reachable for a bijection; keeps the access in bounds
}

// One warp per output row; rows are copied in 16-byte pieces.
__global__ void __launch_bounds__(256) gather_tokens_kernel(const uint4* __restrict__ X, int64_t ldx16, int64_t n,
                                                            int w, uint64_t seed, int64_t first, int64_t count,
                                                            int row16, uint4* __restrict__ out, int64_t ldo16) {
  const int lane = threadIdx.x & 31;
  const int64_t warps = (int64_t)gridDim.x * (blockDim.x >> 5);
  for (int64_t i = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); i < count; i += warps) {
    const int64_t src = permute_index(first + i, n, w, seed);
    const uint4* s = X + src * ldx16;
    uint4* o = out + i * ldo16;
    for (int c = lane; c < row16; c += 32) o[c] = s[c];
  }
}

}  // namespace

dq_status gather_tokens(Ctx& ctx, const void* X, int elem_bytes, int64_t n, int d, int64_t ldx, uint64_t seed,
                        int64_t first, int64_t count, void* out, int64_t ldo) {
  if (((int64_t)d * elem_bytes) % 16 || (ldx * elem_bytes) % 16 || (ldo * elem_bytes) % 16 ||
      ((uintptr_t)X & 15) || ((uintptr_t)out & 15))
    return DQ_ERR_UNSUPPORTED;
  if (count == 0) return DQ_OK;
  int w = 1;
  while (w < 32 && ((int64_t)1 << (2 * w)) < n) ++w;
  int64_t blocks = (count + 7) / 8;
  if (blocks > (int64_t)ctx.sm_count * 16) blocks = (int64_t)ctx.sm_count * 16;
  gather_tokens_kernel<<<(int)blocks, 256, 0, ctx.stream>>>(
      reinterpret_cast<const uint4*>(X), ldx * elem_bytes / 16, n, w, seed, first, count, d * elem_bytes / 16,
      reinterpret_cast<uint4*>(out), ldo * elem_bytes / 16);
  return after_launch(ctx);
}

}  // namespace dq
