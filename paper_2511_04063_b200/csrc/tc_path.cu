// Host side of the tensor-core path: tensor maps, operand copies, launches.
#include <vector>

#include "tc_heads.cuh"
#include "tc_host.cuh"
#include "tc_path.cuh"

namespace dq {
namespace {

// out[b][c][r] = bf16(in[b][r][c])  (fp32 in, d x d)
__global__ void __launch_bounds__(256) transpose_f32_to_bf16_kernel(const float* __restrict__ in,
                                                                    __nv_bfloat16* __restrict__ out, int d) {
  __shared__ float t[32][33];
  in += (int64_t)blockIdx.z * d * d;
  out += (int64_t)blockIdx.z * d * d;
  const int r0 = blockIdx.y * 32, c0 = blockIdx.x * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  for (int r = ty; r < 32; r += 8) t[r][tx] = in[(int64_t)(r0 + r) * d + c0 + tx];
  __syncthreads();
  for (int c = ty; c < 32; c += 8) out[(int64_t)(c0 + c) * d + r0 + tx] = __float2bfloat16_rn(t[tx][c]);
}

// out tile = sum over slices of part[slice] tile, for the tiles of `list` (mb | nb << 16; tiles
// are bm x bn, bn <= 256); gridDim.y CTAs per tile (a band of at most 32 rows each), fixed summation order.
// out_t (nullable): also the bf16 transpose, out_t[c][r] = bf16(out[r][c]); the band goes through shared
// memory so that a warp stores consecutive rows of one column (contiguous in out_t).
__global__ void __launch_bounds__(256) tile_reduce_kernel(const float* __restrict__ part, int slices,
                                                          int64_t slice_stride, const int* __restrict__ list, int bm,
                                                          int bn, int d, float* __restrict__ out,
                                                          __nv_bfloat16* __restrict__ out_t) {
  __shared__ __nv_bfloat16 band_t[32][256 + 2];   // [row of the band][column], padded against bank conflicts
  const int code = list[blockIdx.x];
  const int band = bm / gridDim.y;
  const int r0 = (code & 0xffff) * bm + blockIdx.y * band, c0 = (code >> 16) * bn;
  const int per_row = bn / 4;
  for (int e = threadIdx.x; e < band * per_row; e += 256) {
    const int rr = e / per_row, cc = (e % per_row) * 4;
    const int64_t idx = (int64_t)(r0 + rr) * d + c0 + cc;
    float4 s = *reinterpret_cast<const float4*>(part + idx);
    for (int k = 1; k < slices; ++k) {
      const float4 t = *reinterpret_cast<const float4*>(part + (int64_t)k * slice_stride + idx);
      s.x += t.x; s.y += t.y; s.z += t.z; s.w += t.w;
    }
    *reinterpret_cast<float4*>(out + idx) = s;
    if (out_t) {
      band_t[rr][cc] = __float2bfloat16_rn(s.x);
      band_t[rr][cc + 1] = __float2bfloat16_rn(s.y);
      band_t[rr][cc + 2] = __float2bfloat16_rn(s.z);
      band_t[rr][cc + 3] = __float2bfloat16_rn(s.w);
    }
  }
  if (!out_t) return;
  __syncthreads();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int c = warp; c < bn; c += 8)
    if (lane < band) out_t[(int64_t)(c0 + c) * d + r0 + lane] = band_t[lane][c];
}

// One thread waits, with the bounded wait every tcgen05 kernel of the library uses, on a barrier that nothing
// ever arrives at (no copy or MMA is in flight): the wait must give up after limit_ns, record DQ_ERR_TIMEOUT
// and let the kernel return normally.  waited_ns receives how long it waited.
__global__ void bounded_wait_probe_kernel(uint64_t limit_ns, int* d_status, uint64_t* waited_ns) {
  __shared__ __align__(8) uint64_t bar;
  const uint32_t b = tc::smem_u32(&bar);
  tc::mbar_init(b, 1);
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  const uint64_t t0 = tc::global_timer_ns();
  const bool done = tc::mbar_wait(b, 0u, d_status, limit_ns);
  if (waited_ns) *waited_ns = done ? 0ull : tc::global_timer_ns() - t0;
}

struct Maps {
  CUtensorMap rt, x, x128, xmn, gt128, gt256;
};

}  // namespace

dq_status tc_init(TcState& tc, Ctx& ctx, const dq_calib_config& cfg, const void* d_X, __nv_bfloat16* Gt,
                  __nv_bfloat16* rt_external, int* n_partials) {
  const int d = cfg.d, batch = cfg.batch;
  const int64_t N = cfg.n_tokens;
  tc.d = d; tc.batch = batch; tc.n_tokens = N;
  tc.X = reinterpret_cast<const __nv_bfloat16*>(d_X);
  tc.Gt = Gt;
  if (rt_external) {
    tc.Rt = rt_external; tc.rt_external = true;
  } else if (cudaMalloc((void**)&tc.Rt, sizeof(__nv_bfloat16) * (size_t)batch * d * d) != cudaSuccess) {
    return DQ_ERR_ALLOC;
  }
  // split-K of Gq = X^T G over the token dimension: fill the machine, keep >= 16 k-blocks per slice
  const int bn = (d % 256 == 0) ? 256 : 128;
  tc.pair = (d % 256 == 0) && ctx.sm_count >= 2;
  const int bm = tc.pair ? 256 : tc::BLOCK_M;
  const int n_cta_units = tc.pair ? ctx.sm_count / 2 : ctx.sm_count;   // tiles computed at a time
  const int tiles = (d / bm) * (d / bn) * batch;
  int ks = 1;
  while (tiles * ks < n_cta_units && (N / tc::BLOCK_K) / (ks * 2) >= 16 && ks < 64) ks *= 2;
  tc.ksplit = ks;
  if (ks > 1 &&
      cudaMalloc((void**)&tc.part, sizeof(float) * (size_t)batch * ks * d * d) != cudaSuccess)
    return DQ_ERR_ALLOC;
  if (ks == 1 && batch == 1 && tiles > n_cta_units && tiles % n_cta_units != 0) {
    // a partly filled last wave: split its reduction so that it fills the machine once more
    const int rem = tiles % n_cta_units, full = tiles - rem, mbk = d / bm;
    int sp = n_cta_units / rem;
    if (sp > 4) sp = 4;
    while (sp > 1 && (N / tc::BLOCK_K) / sp < 16) --sp;
    if (sp > 1) {
      std::vector<int> head(full), tail(rem);
      for (int r = 0; r < tiles; ++r) (r < full ? head[r] : tail[r - full]) = (r % mbk) | ((r / mbk) << 16);
      tc.n_head = full; tc.n_tail = rem; tc.tail_split = sp;
      if (cudaMalloc((void**)&tc.tl_head, sizeof(int) * full) != cudaSuccess ||
          cudaMalloc((void**)&tc.tl_tail, sizeof(int) * rem) != cudaSuccess ||
          cudaMalloc((void**)&tc.tail_part, sizeof(float) * (size_t)sp * d * d) != cudaSuccess)
        return DQ_ERR_ALLOC;
      DQ_CHECK_CUDA(cudaMemcpy(tc.tl_head, head.data(), sizeof(int) * full, cudaMemcpyHostToDevice));
      DQ_CHECK_CUDA(cudaMemcpy(tc.tl_tail, tail.data(), sizeof(int) * rem, cudaMemcpyHostToDevice));
    }
  }
  Maps* m = new (std::nothrow) Maps();
  if (!m) return DQ_ERR_ALLOC;
  tc.maps = m;
  DQ_CHECK(tch::make_map(&m->rt, tc.Rt, d, d, batch, d, (int64_t)d * d, tc::BLOCK_M));
  const int64_t ldx = cfg.ldx;   // row stride of the borrowed activations (>= d, a multiple of 8 elements)
  tc.ldx = ldx;
  DQ_CHECK(tch::make_map(&m->x, tc.X, d, N, batch, ldx, N * ldx, 256));
  DQ_CHECK(tch::make_map(&m->x128, tc.X, d, N, batch, ldx, N * ldx, 128));
  // X again, in boxes of 64 tokens x 64 channels: the MN-major A operand (X^T) of Gq = X^T G
  DQ_CHECK(tch::make_map(&m->xmn, tc.X, d, N, batch, ldx, N * ldx, tc::BLOCK_K));
  DQ_CHECK(tch::make_map(&m->gt128, tc.Gt, N, d, batch, N, N * d, 128));
  DQ_CHECK(tch::make_map(&m->gt256, tc.Gt, N, d, batch, N, N * d, 256));
  if (d == 128) {   // per-head rotations: fused kernel, one CTA per SM over equal ranges of the tile sequence
    const int tiles_per_head = (int)(N / heads::TT);
    const int64_t total = (int64_t)batch * tiles_per_head;
    const int64_t grid = total < ctx.sm_count ? total : ctx.sm_count;
    // partial slots per head = the most CTAs whose ranges meet any one head (its unused slots stay zero)
    int sp = 1;
    for (int b = 0; b < batch; ++b) {
      const int first = heads::range_owner((int64_t)b * tiles_per_head, total, grid);
      const int last = heads::range_owner((int64_t)(b + 1) * tiles_per_head - 1, total, grid);
      if (last - first + 1 > sp) sp = last - first + 1;
    }
    tc.splits = sp;
    const size_t part_bytes = sizeof(float) * (size_t)batch * sp * 128 * 128;
    if (cudaMalloc((void**)&tc.heads_part, part_bytes) != cudaSuccess) return DQ_ERR_ALLOC;
    DQ_CHECK_CUDA(cudaMemsetAsync(tc.heads_part, 0, part_bytes, ctx.stream));
    if (cudaFuncSetAttribute(heads::heads_whip_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             heads::SMEM_TOTAL) != cudaSuccess)
      return DQ_ERR_CUDA;
    tc.fused = true;
  }
  tc.n_partials = (d / tc::BLOCK_M) * (int)(N / 256) * 4;
  if (tc.fused && tc.n_partials < tc.splits * heads::EPI_WARPS) tc.n_partials = tc.splits * heads::EPI_WARPS;
  *n_partials = tc.n_partials;
  tc.ready = true;
  return DQ_OK;
}

// The activations are read in place by every kernel (the contraction over tokens takes X^T as an MN-major
// operand straight from the token-major rows), so a caller that rewrites X has nothing to rebuild.
dq_status tc_refresh_inputs(TcState&, Ctx&) { return DQ_OK; }

void tc_destroy(TcState& tc) {
  if (!tc.rt_external) cudaFree(tc.Rt); cudaFree(tc.part);
  cudaFree(tc.tl_head); cudaFree(tc.tl_tail); cudaFree(tc.tail_part); cudaFree(tc.heads_part);
  delete reinterpret_cast<Maps*>(tc.maps);
  tc = TcState();
}

// O^T = R^T X^T per 128 x 256 tile (rows = channels, columns = tokens), Whip epilogue:
// writes G^T (bf16, channel-major) and 4 loss partials per tile.
dq_status tc_whip_forward(TcState& tc, Ctx& ctx, float* partials) {
  ctx.mma_flops += 2.0 * (double)tc.n_tokens * tc.d * tc.d * tc.batch;
  tc.n_partials_live = tc.n_partials;
  tc.fused_valid = false;
  if (tc.fused) {
    Maps* mm = reinterpret_cast<Maps*>(tc.maps);
    heads::Params hp{};
    hp.batch = tc.batch; hp.tiles_per_head = (int)(tc.n_tokens / heads::TT); hp.slots = tc.splits;
    hp.n_tokens = tc.n_tokens; hp.part = tc.heads_part; hp.partials = partials;
    hp.Gt = tc.keep_g ? tc.Gt : nullptr; hp.d_status = ctx.d_status;
    const int64_t total = (int64_t)tc.batch * hp.tiles_per_head;
    const int grid = (int)(total < ctx.sm_count ? total : ctx.sm_count);   // (the slots were sized for this grid)
    heads::heads_whip_kernel<<<grid, heads::HEADS_THREADS, heads::SMEM_TOTAL, ctx.stream>>>(mm->rt, mm->x128, hp);
    tc.n_partials_live = tc.splits * heads::EPI_WARPS;
    tc.fused_valid = true;
    ctx.mma_flops += 2.0 * (double)tc.n_tokens * tc.d * tc.d * tc.batch;   // the second product runs here too
    return after_launch(ctx);
  }
  Maps* m = reinterpret_cast<Maps*>(tc.maps);
  tc::Params p{};
  p.m_blocks = tc.d / tc::BLOCK_M; p.n_blocks = (int)(tc.n_tokens / 256); p.batch = tc.batch; p.ksplit = 1;
  p.k_blocks = tc.d / tc::BLOCK_K;
  p.out = tc.Gt; p.ld = tc.n_tokens; p.batch_stride = tc.n_tokens * tc.d; p.split_stride = 0;
  p.alpha = 1.f; p.partials = partials; p.d_status = ctx.d_status;
  if (tc.pair) {   // 256 channels x 256 tokens per CTA pair
    p.m_blocks = tc.d / 256;
    return tch::launch_gemm2<1, tc::EPI_WHIP>(ctx, m->rt, m->x128, m->rt, m->x128, p);
  }
  return tch::launch_gemm<256, 1, tc::EPI_WHIP>(ctx, m->rt, m->x, m->rt, m->x, p);
}

// Gq = scale * X^T G : A = X^T taken MN-major from X [N][d], B = G^T [d][N], reduction over tokens.
// gqt (nullable): the epilogue also stores bf16(Gq^T) there (the operand of the QR-Orth backward);
// *gqt_written tells whether this schedule could (the split-K schedule of small shapes cannot).
dq_status tc_grad_rotation(TcState& tc, Ctx& ctx, float* Gq, float scale, __nv_bfloat16* gqt, bool* gqt_written) {
  if (gqt_written) *gqt_written = false;
  if (tc.fused && tc.fused_valid)   // the fused kernel left one partial per unit: sum them in a fixed order
    return splitk_reduce(ctx, tc.heads_part, tc.splits, (int64_t)tc.d * tc.d, tc.batch, scale, 0.f, Gq);
  ctx.mma_flops += 2.0 * (double)tc.n_tokens * tc.d * tc.d * tc.batch;
  Maps* m = reinterpret_cast<Maps*>(tc.maps);
  const int d = tc.d;
  const int bn = (d % 256 == 0) ? 256 : 128;
  tc::Params p{};
  p.m_blocks = d / tc::BLOCK_M; p.n_blocks = d / bn; p.batch = tc.batch; p.ksplit = tc.ksplit;
  p.k_blocks = (int)(tc.n_tokens / tc::BLOCK_K);
  p.ld = d; p.alpha = scale; p.out_hi = nullptr; p.out_lo = nullptr;
  p.partials = nullptr; p.d_status = ctx.d_status;
  p.a_mn = 1;
  if (tc.ksplit == 1) {
    p.out = Gq; p.batch_stride = (int64_t)d * d; p.split_stride = 0;
  } else {
    p.out = tc.part; p.batch_stride = (int64_t)tc.ksplit * d * d; p.split_stride = (int64_t)d * d;
  }
  if (tc.pair) p.m_blocks = d / 256;
  auto launch = [&](const tc::Params& pp) {
    if (tc.pair) return tch::launch_gemm2<1, tc::EPI_GEN>(ctx, m->xmn, m->gt128, m->xmn, m->gt128, pp);
    return (bn == 256) ? tch::launch_gemm<256, 1, tc::EPI_GEN>(ctx, m->xmn, m->gt256, m->xmn, m->gt256, pp)
                       : tch::launch_gemm<128, 1, tc::EPI_GEN>(ctx, m->xmn, m->gt128, m->xmn, m->gt128, pp);
  };
  const bool with_t = gqt != nullptr && tc.ksplit == 1 && tc.batch == 1;
  if (with_t) {
    p.out_t_hi = gqt; p.ld_t = d; p.batch_stride_t = (int64_t)d * d;
    if (gqt_written) *gqt_written = true;
  }
  if (tc.tail_split > 1) {
    tc::Params ph = p;      // full waves: whole reduction per tile
    ph.tile_list = tc.tl_head; ph.n_list = tc.n_head;
    DQ_CHECK(launch(ph));
    tc::Params pt = p;      // last wave: reduction in slices, then a fixed-order sum
    pt.tile_list = tc.tl_tail; pt.n_list = tc.n_tail; pt.ksplit = tc.tail_split;
    pt.out = tc.tail_part; pt.batch_stride = 0; pt.split_stride = (int64_t)d * d;
    pt.out_t_hi = nullptr;
    DQ_CHECK(launch(pt));
    tile_reduce_kernel<<<dim3(tc.n_tail, 8), 256, 0, ctx.stream>>>(tc.tail_part, tc.tail_split, (int64_t)d * d, tc.tl_tail,
                                                          tc.pair ? 256 : 128, bn, d, Gq, with_t ? gqt : nullptr);
    return after_launch(ctx);
  }
  DQ_CHECK(launch(p));
  if (tc.ksplit > 1) DQ_CHECK(splitk_reduce(ctx, tc.part, tc.ksplit, (int64_t)d * d, tc.batch, 1.f, 0.f, Gq));
  return DQ_OK;
}

// Y = X R for bf16 activations: A = X [n][d], B = bf16(R^T) [d][d]; bf16 output, row stride ldy.
dq_status tc_rotate_apply(Ctx& ctx, const void* d_X, int64_t n, int d, int64_t ldx, const float* d_R,
                          void* d_Y, int64_t ldy) {
  if (d % 128 != 0 || n % 128 != 0 || ldx % 8 != 0 || ldy % 8 != 0) return DQ_ERR_UNSUPPORTED;
  if (((uintptr_t)d_X | (uintptr_t)d_Y) & 15) return DQ_ERR_UNSUPPORTED;   // 16-byte loads (TMA) and stores
  int sms = 0, dev = 0;
  DQ_CHECK_CUDA(cudaGetDevice(&dev));
  DQ_CHECK_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  ctx.sm_count = sms;
  tch::keep_pool_memory(dev);
  __nv_bfloat16* rt = nullptr;
  if (cudaMallocAsync((void**)&rt, sizeof(__nv_bfloat16) * (size_t)d * d, ctx.stream) != cudaSuccess)
    return DQ_ERR_ALLOC;
  transpose_f32_to_bf16_kernel<<<dim3(d / 32, d / 32, 1), 256, 0, ctx.stream>>>(d_R, rt, d);
  dq_status st = after_launch(ctx);
  if (st == DQ_OK) st = tch::rotate_tokens<tc::EPI_BF16>(ctx, d_X, n, d, ldx, rt, d_Y, ldy, nullptr);
  cudaFreeAsync(rt, ctx.stream);
  return st;
}


dq_status bounded_wait_probe(Ctx& ctx, uint64_t limit_ns, uint64_t* d_waited_ns) {
  bounded_wait_probe_kernel<<<1, 1, 0, ctx.stream>>>(limit_ns, ctx.d_status, d_waited_ns);
  return after_launch(ctx);
}

// ---------------------------------------------------------------------------------------------
// Y = X R without any allocation (dq_rotate_apply_static).
//
// The only scratch the bf16 rotation needs is the bf16 copy of R^T that feeds the tensor cores.
// Here it lives in a file-scope device array, so the call never touches the CUDA allocator.
// Every device that loads the library carries the array (8 MiB) until the process exits.
// ---------------------------------------------------------------------------------------------
constexpr int STATIC_MAX_D = 2048;
static __device__ __align__(256) __nv_bfloat16 g_static_rt[(size_t)STATIC_MAX_D * STATIC_MAX_D];

namespace {
constexpr int STATIC_MAX_DEVICES = 64;
__nv_bfloat16* g_static_rt_ptr[STATIC_MAX_DEVICES] = {};   // device address of g_static_rt, per device
int g_static_sms[STATIC_MAX_DEVICES] = {};
}  // namespace

dq_status tc_rotate_apply_static(Ctx& ctx, const void* d_X, int64_t n, int d, int64_t ldx, const float* d_R,
                                 void* d_Y, int64_t ldy) {
  if (d > STATIC_MAX_D) return DQ_ERR_UNSUPPORTED;
  if (d % 128 != 0 || n % 128 != 0 || ldx % 8 != 0 || ldy % 8 != 0) return DQ_ERR_UNSUPPORTED;
  if (((uintptr_t)d_X | (uintptr_t)d_Y) & 15) return DQ_ERR_UNSUPPORTED;   // 16-byte loads (TMA) and stores
  int dev = 0;
  DQ_CHECK_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= STATIC_MAX_DEVICES) return DQ_ERR_UNSUPPORTED;
  if (!g_static_rt_ptr[dev]) {
    // First call on this device: in host code the array's name is only a handle; the kernels need
    // its device address.
    int cc_major = 0;
    DQ_CHECK_CUDA(cudaDeviceGetAttribute(&cc_major, cudaDevAttrComputeCapabilityMajor, dev));
    if (cc_major != 10) return DQ_ERR_UNSUPPORTED;
    DQ_CHECK_CUDA(cudaDeviceGetAttribute(&g_static_sms[dev], cudaDevAttrMultiProcessorCount, dev));
    __nv_bfloat16* p = nullptr;
    if (cudaGetSymbolAddress((void**)&p, g_static_rt) != cudaSuccess || !p) return DQ_ERR_CUDA;
    g_static_rt_ptr[dev] = p;
  }
  ctx.sm_count = g_static_sms[dev];
  __nv_bfloat16* rt = g_static_rt_ptr[dev];
  // Every element of rt[0 : d*d) is overwritten, so nothing of an earlier call survives.
  transpose_f32_to_bf16_kernel<<<dim3(d / 32, d / 32, 1), 256, 0, ctx.stream>>>(d_R, rt, d);
  DQ_CHECK(after_launch(ctx));
  return tch::rotate_tokens<tc::EPI_BF16>(ctx, d_X, n, d, ldx, rt, d_Y, ldy, nullptr);
}

}  // namespace dq
