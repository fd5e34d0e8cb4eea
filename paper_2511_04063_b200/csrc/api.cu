// C ABI: handle management, argument validation and the per-step schedule.
//
// All work of a handle runs on an internal stream that is fenced against the
// caller's stream with events at every entry point, so the caller sees ordinary
// stream semantics while whole steps can be replayed as a CUDA graph (stream
// capture is not allowed on the legacy default stream callers often pass).
#include <cstdlib>
#include <cstring>
#include <new>
#include <utility>

#include "common.cuh"
#include "tc_path.cuh"

using namespace dq;

// Default number of sweeps (beyond the three that always exist) of the incremental QR-Orth on the tensor-core
// route for d >= 256, whose fixed point starts from the previous step's T^T T and so needs few.
constexpr int DEFAULT_QR_SWEEPS_TC = 5;
// |Z0^T Z0 - I|_F up to which a latent counts as orthogonal at dq_calib_init (the fixed point of the incremental
// factorisation contracts for |E|_2 well below 1/2; the Frobenius norm bounds the spectral norm)
constexpr float ORTHOGONAL_START_THRESHOLD = 0.05f;

struct dq_calib {
  dq_calib_config cfg;
  Ctx ctx;                      // ctx.stream is the internal work stream
  cudaStream_t user_stream = nullptr;
  cudaEvent_t ev_in = nullptr, ev_out = nullptr;
  const void* X = nullptr;
  float* Z = nullptr;
  float* R = nullptr;
  float* U = nullptr;
  float* Gq = nullptr;
  float* Gz = nullptr;
  float* gq_part = nullptr;     // fp32 path: split-K partials of Gq
  int gq_ks = 1;
  void* G = nullptr;            // fp32 [b][N][d] (fp32 path) or bf16 [b][d][N] (tensor-core path)
  int64_t g_elems = 0;
  float* partials = nullptr;
  int n_partials = 0;           // per problem
  float* loss_last = nullptr;   // [batch]
  float* loss_tmp = nullptr;    // [batch] loss of a later micro-batch before it is accumulated
  QrWorkspace ws;
  TcState tc;                   // tensor-core contractions (operand copies, tensor maps)
  QrTcState qtc;                // tensor-core QR-Orth operand copies
  bool fast_qr = false;
  int qr_method = DQ_QR_ITERATIVE, qr_iters = 12;
  bool qr_iters_default = true;  // n_iters was not given: the large tensor-core route then uses DEFAULT_QR_SWEEPS_TC
  int optimizer = DQ_SGD;
  float beta1 = 0.f, beta2 = 0.f, eps = 0.f;
  float* opt_m = nullptr;       // first moment / velocity
  float* opt_v = nullptr;       // second moment
  float* opt_pw = nullptr;      // device float[2]: beta1^t, beta2^t
  ObjectiveState obj;           // objectives other than Eq. 4
  int orth_method = DQ_ORTH_QR;
  CayleyState cay;              // DQ_ORTH_CAYLEY: momentum and step size
  bool cay_started = false;     // R and its split copies hold the Cayley iterate
  bool f32_winv_valid = false;  // fp32 path: ws.Winv is the inverse of the U currently stored
  int* f32_flags = nullptr;     // fp32 path: sweep flags of the incremental factorisation
  bool small_warm = false;      // d == 128: U and U^-1 hold the factors of the previous step's latent
  bool small128 = false;        // d == 128: shared-memory-resident batched QR-Orth
  bool tc5 = false;             // d == 128 on the tensor-core path: tcgen05 kernel for the incremental QR-Orth
  float* p128 = nullptr;        // [batch][128][128] T^T T of the last sweep (tc5)
  bool u128_fresh = false;      // U holds the upper factor of the current factorisation (tc5 carries only U^-1)
  float* R_alt = nullptr;       // tc5: second rotation buffer; a fused step reads R and leaves the next rotation here, then the two swap
  float* R_used = nullptr;      // rotation the last step used, when that is no longer R (fused steps)
  int r_sel = 0;                // which of the two buffers R is (captured graphs hold the pointers)
  bool r_stale = true;
  bool timing = false;
  cudaEvent_t ev[DQ_PHASE_COUNT + 1] = {};
  double ms_acc[DQ_PHASE_COUNT] = {};
  int timed_steps = 0;
  bool bwd_split = false;       // tensor-core QR-Orth backward with split-bf16 operands (three MMAs per product)
  // One whole step (QR forward .. update) captured once and replayed.  The incremental QR-Orth alternates
  // between two sets of copies of U^-1, so there is one captured step per set (index = set read by the step).
  struct StepGraph {
    cudaGraphExec_t exec = nullptr;
    int64_t launches = 0;
    double flops = 0.0;
    bool failed = false;
    bool needs_z_split = false;   // the captured step reads z_hi / z_lo without writing them first
  } graph[2];
  int eager_steps_done = 0;
};

namespace {

template <typename T>
dq_status dev_alloc(T** p, int64_t n) {
  *p = nullptr;
  if (n <= 0) return DQ_OK;
  return cudaMalloc((void**)p, sizeof(T) * (size_t)n) == cudaSuccess ? DQ_OK : DQ_ERR_ALLOC;
}

void free_all(dq_calib* h) {
  if (!h) return;
  for (auto& g : h->graph) if (g.exec) cudaGraphExecDestroy(g.exec);
  tc_destroy(h->tc);
  qr_tc_destroy(h->qtc);
  cayley_destroy(h->cay);
  objective_destroy(h->obj);
  cudaFree(h->Z); cudaFree(h->R); cudaFree(h->U); cudaFree(h->Gq); cudaFree(h->Gz); cudaFree(h->gq_part);
  cudaFree(h->opt_m); cudaFree(h->opt_v); cudaFree(h->opt_pw); cudaFree(h->p128); cudaFree(h->R_alt);
  cudaFree(h->G); cudaFree(h->partials); cudaFree(h->loss_last); cudaFree(h->loss_tmp); cudaFree(h->f32_flags); cudaFree(h->ctx.d_status);
  cudaFree(h->ws.A); cudaFree(h->ws.V); cudaFree(h->ws.T); cudaFree(h->ws.W); cudaFree(h->ws.W2);
  cudaFree(h->ws.Q); cudaFree(h->ws.Winv); cudaFree(h->ws.B); cudaFree(h->ws.S); cudaFree(h->ws.tmp);
  for (auto& e : h->ev) if (e) cudaEventDestroy(e);
  if (h->ev_in) cudaEventDestroy(h->ev_in);
  if (h->ev_out) cudaEventDestroy(h->ev_out);
  if (h->ctx.stream) cudaStreamDestroy(h->ctx.stream);
  if (h->ctx.side) cudaStreamDestroy(h->ctx.side);
  if (h->ctx.ev_fork) cudaEventDestroy(h->ctx.ev_fork);
  if (h->ctx.ev_join) cudaEventDestroy(h->ctx.ev_join);
  delete h;
}

dq_status validate(const dq_calib_config* c) {
  if (!c) return DQ_ERR_INVALID_ARG;
  if (c->d <= 0 || c->n_tokens <= 0 || c->batch <= 0 || c->ldx < c->d) return DQ_ERR_INVALID_ARG;
  if (c->x_dtype != DQ_FP32 && c->x_dtype != DQ_BF16) return DQ_ERR_INVALID_ARG;
  if (c->path != DQ_PATH_FP32 && c->path != DQ_PATH_BF16_TC) return DQ_ERR_INVALID_ARG;
  if (c->reduction != DQ_MEAN_TOKENS && c->reduction != DQ_SUM_TOKENS) return DQ_ERR_INVALID_ARG;
  if (c->optimizer != DQ_SGD) return DQ_ERR_INVALID_ARG;
  if (!(c->lr == c->lr)) return DQ_ERR_INVALID_ARG;
  if (c->d > 8192 || c->d % 64 != 0) return DQ_ERR_UNSUPPORTED;
  if (c->path == DQ_PATH_FP32) {
    if (c->x_dtype != DQ_FP32) return DQ_ERR_UNSUPPORTED;
  } else {
    if (c->x_dtype != DQ_BF16) return DQ_ERR_UNSUPPORTED;
    if (c->d % 128 != 0 || c->n_tokens % 256 != 0 || c->ldx % 8 != 0) return DQ_ERR_UNSUPPORTED;   // (TMA: 16-byte row stride)
  }
  return DQ_OK;
}

// Order the internal stream after everything the caller enqueued so far / the caller's
// stream after everything this call enqueued.
dq_status fence_in(dq_calib* h) {
  DQ_CHECK_CUDA(cudaEventRecord(h->ev_in, h->user_stream));
  DQ_CHECK_CUDA(cudaStreamWaitEvent(h->ctx.stream, h->ev_in, 0));
  return DQ_OK;
}
dq_status fence_out(dq_calib* h) {
  DQ_CHECK(join_side(h->ctx));
  DQ_CHECK_CUDA(cudaEventRecord(h->ev_out, h->ctx.stream));
  DQ_CHECK_CUDA(cudaStreamWaitEvent(h->user_stream, h->ev_out, 0));
  return DQ_OK;
}

// A configuration change or a new latent acknowledges an earlier device-side error.
dq_status clear_status(dq_calib* h) {
  DQ_CHECK_CUDA(cudaMemsetAsync(h->ctx.d_status, 0, sizeof(int), h->ctx.stream));
  return DQ_OK;
}

// The fused launch left the next rotation in R_alt: it becomes R, the one the step used stays readable.
void rotation_advanced(dq_calib* h) {
  h->R_used = h->R;
  std::swap(h->R, h->R_alt);
  h->r_sel ^= 1;
  h->u128_fresh = false;
}

// 128 x 128 latents on the tensor-core path with plain SGD: the backward launch of a step also runs the
// incremental forward of the next one, so a step begins and ends with a current rotation.
bool fuses_forward(const dq_calib* h, bool timed) {
  return h->tc5 && h->qr_method == DQ_QR_ITERATIVE && h->optimizer == DQ_SGD && h->orth_method != DQ_ORTH_CAYLEY &&
         h->small_warm && !timed;
}

dq_status ensure_rotation(dq_calib* h) {
  if (h->orth_method == DQ_ORTH_CAYLEY && h->cay_started) return DQ_OK;   // R is the iterate itself
  if (!h->r_stale) return DQ_OK;
  h->R_used = nullptr;   // R is about to hold the rotation of the current latent
  if (h->small128) {
    __nv_bfloat16* rt = h->cfg.path == DQ_PATH_BF16_TC ? h->qtc.rt_hi : nullptr;
    if (h->qr_method == DQ_QR_ITERATIVE && h->small_warm) {
      if (h->tc5) {   // tcgen05 kernel: needs only W (no U), starts its fixed point from the last step's T^T T
        DQ_CHECK(qr128_step_tc5(h->ctx, h->Z, h->ws.Winv, h->p128, h->R, nullptr, rt, nullptr, nullptr, 0.f,
                                false, true, h->qr_iters + 3, h->cfg.batch));
        h->u128_fresh = false;
      } else {
        DQ_CHECK(qr128_forward_incremental(h->ctx, h->Z, h->R, h->U, h->ws.Winv, rt, h->qr_iters, h->cfg.batch));
      }
    } else {
      DQ_CHECK(qr128_forward(h->ctx, h->Z, h->R, h->U, h->ws.Winv, rt, h->cfg.batch));
      if (h->tc5)
        DQ_CHECK_CUDA(cudaMemsetAsync(h->p128, 0, sizeof(float) * (size_t)128 * 128 * h->cfg.batch, h->ctx.stream));
      h->u128_fresh = true;
      h->small_warm = true;
    }
  } else if (h->fast_qr) {
    DQ_CHECK(qr_forward_fast(h->ctx, h->ws, h->qtc, h->Z, h->R, h->U, h->cfg.d, h->cfg.batch,
                             h->qr_method == DQ_QR_ITERATIVE ? (h->qr_iters_default ? DEFAULT_QR_SWEEPS_TC : h->qr_iters) : 0,
                             h->bwd_split || h->orth_method == DQ_ORTH_CAYLEY));
  } else if (h->qr_method == DQ_QR_ITERATIVE && h->f32_winv_valid && h->f32_flags && h->cfg.d <= 1024) {
    // fp32 path: the same incremental factorisation on fp32 FMA products (U and U^-1 of the previous step)
    DQ_CHECK(qr_forward_incremental_f32(h->ctx, h->ws, h->Z, h->R, h->U, h->cfg.d, h->cfg.batch, h->qr_iters,
                                        h->f32_flags));
  } else {
    DQ_CHECK(qr_forward(h->ctx, h->ws, h->Z, h->R, h->U, tc_rt_operand(h->tc), h->cfg.d, h->cfg.batch));
    h->f32_winv_valid = false;
  }
  h->r_stale = false;
  return DQ_OK;
}

// Mini-batches of one optimiser step drawn from a pool of token rows (Algorithm 1's token sampling):
// micro-batch a is rows pi_seed(first + a * n_tokens ...) of the pool, gathered into the handle's
// activation buffer; dL/dR and the loss are averaged (summed with DQ_SUM_TOKENS) over the micro-batches.
struct MiniBatch {
  const void* pool; int64_t n_pool, ld_pool; uint64_t seed; int64_t first; int n_micro;
};

// One iteration of Algorithm 1's loop body enqueued on the work stream.
dq_status enqueue_step(dq_calib* h, bool timed, const MiniBatch* mb = nullptr) {
  const dq_calib_config& c = h->cfg;
  const int d = c.d, batch = c.batch;
  const int64_t N = c.n_tokens;
  const int n_micro = mb ? mb->n_micro : 1;
  const float inv_n = (c.reduction == DQ_MEAN_TOKENS) ? (float)(1.0 / ((double)N * n_micro)) : 1.f;
  Ctx& ctx = h->ctx;
  if (timed) DQ_CHECK_CUDA(cudaEventRecord(h->ev[0], ctx.stream));
  const bool cayley = h->orth_method == DQ_ORTH_CAYLEY;
  // (a1) R <- qr(Z)   (Cayley SGD: only to obtain the first iterate)
  if (!cayley || !h->cay_started) DQ_CHECK(ensure_rotation(h));
  if (timed) DQ_CHECK_CUDA(cudaEventRecord(h->ev[1], ctx.stream));
  for (int a = 0; a < n_micro; ++a) {
    float* loss_dst = (a == 0) ? h->loss_last : h->loss_tmp;
    float* gq_dst = (a == 0) ? h->Gq : h->ws.tmp;
    if (mb) {
      DQ_CHECK(gather_tokens(ctx, mb->pool, c.x_dtype == DQ_FP32 ? 4 : 2, mb->n_pool, d, mb->ld_pool, mb->seed,
                             mb->first + (int64_t)a * N, N, const_cast<void*>(h->X), c.ldx));
      if (c.path == DQ_PATH_BF16_TC) DQ_CHECK(tc_refresh_inputs(h->tc, ctx));
    }
    // (a2-a4) O = X R, Whip epilogue, loss reduction
    if (h->obj.objective != DQ_OBJ_WHIP) {   // ablation objectives: per-token statistics, materialised O
      DQ_CHECK(objective_forward(ctx, h->obj, c, h->X, h->R, c.path == DQ_PATH_BF16_TC ? h->qtc.rt_hi : nullptr,
                                 h->G, inv_n, loss_dst));
    } else {
      if (c.path == DQ_PATH_FP32) {
        DQ_CHECK(whip_forward_f32(ctx, (const float*)h->X, c.ldx, N * c.ldx, h->R, (float*)h->G, h->partials, N, d,
                                  batch, nullptr));
      } else {
        DQ_CHECK(tc_whip_forward(h->tc, ctx, h->partials));
      }
      const int n_part = c.path == DQ_PATH_BF16_TC ? h->tc.n_partials_live : h->n_partials;
      if (n_micro == 1 && !timed)   // (beside the next contraction: the loss is read after the step)
        DQ_CHECK(on_side(ctx, [&](Ctx& cs) { return loss_finalize(cs, h->partials, n_part, batch, inv_n, nullptr, loss_dst); }));
      else
        DQ_CHECK(loss_finalize(ctx, h->partials, n_part, batch, inv_n, nullptr, loss_dst));
    }
    if (timed && a == n_micro - 1) DQ_CHECK_CUDA(cudaEventRecord(h->ev[2], ctx.stream));
    // (a5) Gq = (1/N) X^T G
    if (c.path == DQ_PATH_FP32) {
      GemmDesc g{};
      g.A = (const float*)h->X; g.lda = c.ldx; g.transA = 1; g.sA = N * c.ldx;
      g.B = (const float*)h->G; g.ldb = d; g.transB = 0; g.sB = N * (int64_t)d;
      g.M = d; g.N = d; g.K = (int)N; g.alpha = inv_n; g.beta = 0.f; g.batch = batch;
      if (h->gq_ks <= 1) {
        g.C = gq_dst; g.ldc = d; g.sC = (int64_t)d * d; g.ksplit = 1;
        DQ_CHECK(gemm_f32(ctx, g));
      } else {   // deterministic split-K over the token dimension
        g.C = h->gq_part; g.ldc = d; g.sC = (int64_t)d * d; g.ksplit = h->gq_ks;
        DQ_CHECK(gemm_f32(ctx, g));
        DQ_CHECK(splitk_reduce(ctx, h->gq_part, h->gq_ks, (int64_t)d * d, batch, 1.f, 0.f, gq_dst));
      }
    } else {
      // a single micro-batch: the contraction's epilogue also leaves bf16(Gq^T) for the QR-Orth backward
      const bool want_t = h->fast_qr && !h->small128 && !cayley && !h->bwd_split && n_micro == 1;
      h->qtc.gqt_fresh = false;
      DQ_CHECK(tc_grad_rotation(h->tc, ctx, gq_dst, inv_n, want_t ? h->qtc.gqt_hi : nullptr, &h->qtc.gqt_fresh));
    }
    if (a > 0) {
      DQ_CHECK(accumulate(ctx, h->Gq, gq_dst, (int64_t)d * d * batch));
      DQ_CHECK(accumulate(ctx, h->loss_last, loss_dst, batch));
    }
  }
  if (timed) DQ_CHECK_CUDA(cudaEventRecord(h->ev[3], ctx.stream));
  DQ_CHECK(join_side(ctx));   // the checks and the loss of this step are in before the latent may change
  // (a6) Gz = R tril(R^T Gq - Gq^T R, -1) U^-T
  // (a7) Z <- Z - lr Gz  (fused into the backward kernel for 128 x 128 latents)
  const int64_t n_latent = (int64_t)d * d * batch;
  bool fused_forward = false;
  if (cayley) {   // Algorithm 3 updates the rotation itself; there is no latent
    DQ_CHECK(cayley_step_tc(ctx, h->ws, h->qtc, h->cay, h->R, h->Gq, c.lr, d, batch));
    h->cay_started = true;
    h->r_stale = false;
    if (timed) {
      DQ_CHECK_CUDA(cudaEventRecord(h->ev[4], ctx.stream));
      DQ_CHECK_CUDA(cudaEventRecord(h->ev[5], ctx.stream));
    }
    return DQ_OK;
  }
  if (h->small128) {   // plain SGD is fused into the backward kernel; other optimisers follow it
    const float lr128 = h->optimizer == DQ_SGD ? c.lr : 0.f;
    if (h->tc5 && h->qr_method == DQ_QR_ITERATIVE) {
      // With plain SGD the same launch goes on to the forward pass of the NEXT step (the new latent never leaves
      // the CTA): the step ends with the rotation of the updated latent in place.  Timed steps keep the two
      // phases apart.
      fused_forward = fuses_forward(h, timed);
      DQ_CHECK(qr128_step_tc5(ctx, h->Z, h->ws.Winv, h->p128, h->R, fused_forward ? h->R_alt : nullptr,
                              fused_forward ? h->qtc.rt_hi : nullptr, h->Gq, h->Gz, lr128, true, fused_forward,
                              fused_forward ? h->qr_iters + 3 : 0, batch));
      if (fused_forward) rotation_advanced(h);
    } else
      DQ_CHECK(qr128_backward_sgd_tc(ctx, h->R, h->ws.Winv, h->Gq, h->Gz, h->Z, lr128, batch));
    if (timed) DQ_CHECK_CUDA(cudaEventRecord(h->ev[4], ctx.stream));
  } else {
    if (h->fast_qr) DQ_CHECK(qr_backward_tc(ctx, h->ws, h->qtc, h->Gq, h->Gz, d, batch, h->bwd_split));
    else {
      DQ_CHECK(qr_backward(ctx, h->ws, h->R, h->U, h->Gq, h->Gz, d, batch, h->f32_winv_valid));
      h->f32_winv_valid = true;
    }
    if (timed) DQ_CHECK_CUDA(cudaEventRecord(h->ev[4], ctx.stream));
    if (h->optimizer == DQ_SGD) {   // the tensor-core QR-Orth reads the latent as a split-bf16 pair: written here
      const bool split = h->fast_qr && h->qtc.ready;
      DQ_CHECK(sgd_update(ctx, h->Z, h->Gz, c.lr, n_latent, split ? h->qtc.z_hi : nullptr, split ? h->qtc.z_lo : nullptr));
      h->qtc.z_split_fresh = split;
    }
  }
  if (h->optimizer != DQ_SGD) h->qtc.z_split_fresh = false;
  if (h->optimizer == DQ_SGD_MOMENTUM)
    DQ_CHECK(momentum_update(ctx, h->Z, h->Gz, h->opt_m, c.lr, h->beta1, n_latent));
  else if (h->optimizer == DQ_ADAM)
    DQ_CHECK(adam_update(ctx, h->Z, h->Gz, h->opt_m, h->opt_v, h->opt_pw, c.lr, h->beta1, h->beta2, h->eps, n_latent));
  h->r_stale = !fused_forward;
  if (!fused_forward) h->R_used = nullptr;
  if (timed) DQ_CHECK_CUDA(cudaEventRecord(h->ev[5], ctx.stream));
  return DQ_OK;
}

void drop_graphs(dq_calib* h) {   // the schedule or a kernel argument changed: capture again
  for (auto& g : h->graph) {
    if (g.exec) cudaGraphExecDestroy(g.exec);
    g = dq_calib::StepGraph();
  }
}

// Which captured step fits the handle's state (see dq_calib::graph).
int graph_slot(const dq_calib* h) { return (h->fast_qr && !h->small128) ? (h->qtc.w_sel & 1) : (h->tc5 ? h->r_sel : 0); }

// Capture one full step into an executable graph (after one eager step has set every
// kernel attribute).  Failure is not an error: the handle keeps launching eagerly.
// Host-side state that a step advances is put back: the capture enqueued nothing.
void try_capture(dq_calib* h) {
  dq_calib::StepGraph& sg = h->graph[graph_slot(h)];
  if (sg.exec || sg.failed) return;
  const int64_t before = h->ctx.launches;
  const double flops_before = h->ctx.mma_flops;
  const QrTcState q_before = h->qtc;
  const bool fused = fuses_forward(h, false);
  const bool f32_winv = h->f32_winv_valid, small_warm = h->small_warm, cay_started = h->cay_started;
  float* const r_before = h->R; float* const r_alt_before = h->R_alt; float* const r_used_before = h->R_used;
  const int r_sel_before = h->r_sel;
  const bool u128_before = h->u128_fresh;
  auto restore = [&]() {
    h->R = r_before; h->R_alt = r_alt_before; h->R_used = r_used_before; h->r_sel = r_sel_before;
    h->u128_fresh = u128_before;
    h->ctx.launches = before;
    h->ctx.mma_flops = flops_before;
    h->qtc = q_before;
    h->f32_winv_valid = f32_winv; h->small_warm = small_warm; h->cay_started = cay_started;
    h->r_stale = (h->orth_method != DQ_ORTH_CAYLEY || !cay_started) && !fused;
  };
  h->r_stale = !fused;   // (a fused step is captured, and replayed, with the rotation current)
  // With plain SGD the update kernel writes the split copy of the new latent, so a step captured while that
  // copy is current holds no split_kernel: it may only be replayed while the copy is current.
  sg.needs_z_split = h->fast_qr && h->qtc.z_split_fresh;
  if (cudaStreamBeginCapture(h->ctx.stream, cudaStreamCaptureModeThreadLocal) != cudaSuccess) {
    cudaGetLastError();
    sg.failed = true;
    return;
  }
  const dq_status st = enqueue_step(h, false);
  cudaGraph_t g = nullptr;
  const cudaError_t e = cudaStreamEndCapture(h->ctx.stream, &g);
  sg.launches = h->ctx.launches - before;
  sg.flops = h->ctx.mma_flops - flops_before;
  restore();
  if (st != DQ_OK || e != cudaSuccess || !g) {
    cudaGetLastError();
    if (g) cudaGraphDestroy(g);
    sg.failed = true;
    return;
  }
  if (cudaGraphInstantiate(&sg.exec, g, 0) != cudaSuccess) {
    cudaGetLastError();
    sg.exec = nullptr;
    sg.failed = true;
  }
  cudaGraphDestroy(g);
}

// Host-side state after a replayed step (what enqueue_step would have left).
void after_replayed_step(dq_calib* h) {
  const bool cayley = h->orth_method == DQ_ORTH_CAYLEY;
  h->r_stale = !cayley && !fuses_forward(h, false);
  if (cayley) return;
  if (!h->r_stale) rotation_advanced(h);
  else h->R_used = nullptr;
  if (h->fast_qr && !h->small128) {
    if (h->qr_method == DQ_QR_ITERATIVE) h->qtc.w_sel ^= 1;    // the step wrote the other set of W copies
    else h->qtc.u_fresh = true;
    if (h->qr_method == DQ_QR_ITERATIVE) h->qtc.u_fresh = false;
    h->qtc.z_split_fresh = h->optimizer == DQ_SGD;
  }
}

}  // namespace

extern "C" {

const char* dq_version(void) { return "dartquant-b200 sm_100a"; }

const char* dq_status_string(dq_status s) {
  switch (s) {
    case DQ_OK: return "ok";
    case DQ_ERR_INVALID_ARG: return "invalid argument";
    case DQ_ERR_UNSUPPORTED: return "unsupported shape, dtype or path";
    case DQ_ERR_ALLOC: return "device allocation failed";
    case DQ_ERR_CUDA: return "CUDA call failed";
    case DQ_ERR_SINGULAR: return "latent matrix is rank deficient";
    case DQ_ERR_NONFINITE: return "non-finite loss or factor";
    case DQ_ERR_TIMEOUT: return "bounded in-kernel wait gave up";
    case DQ_ERR_NOT_CONVERGED: return "iterative QR did not converge: the latent moved too far in one step";
  }
  return "unknown status";
}

dq_status dq_calib_init(dq_calib_t** out, const dq_calib_config* cfg, const void* d_X,
                        const float* d_Z0, void* cuda_stream) {
  if (!out) return DQ_ERR_INVALID_ARG;
  *out = nullptr;
  if (!d_X || !d_Z0) return DQ_ERR_INVALID_ARG;
  DQ_CHECK(validate(cfg));
  int dev = 0, cc_major = 0, sms = 0;
  DQ_CHECK_CUDA(cudaGetDevice(&dev));
  DQ_CHECK_CUDA(cudaDeviceGetAttribute(&cc_major, cudaDevAttrComputeCapabilityMajor, dev));
  DQ_CHECK_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  if (cc_major != 10) return DQ_ERR_UNSUPPORTED;   // sm_100a code only

  dq_calib* h = new (std::nothrow) dq_calib();
  if (!h) return DQ_ERR_ALLOC;
  h->cfg = *cfg;
  h->user_stream = (cudaStream_t)cuda_stream;
  h->ctx.sm_count = sms;
  h->X = d_X;
  h->small128 = (cfg->d == 128);
  const int d = cfg->d, batch = cfg->batch;
  const int64_t dd = (int64_t)d * d * batch;
  dq_status st = DQ_OK;
  auto A = [&](dq_status s) { if (st == DQ_OK) st = s; };
  if (cudaStreamCreateWithFlags(&h->ctx.stream, cudaStreamNonBlocking) != cudaSuccess) st = DQ_ERR_CUDA;
  if (st == DQ_OK && (cudaStreamCreateWithFlags(&h->ctx.side, cudaStreamNonBlocking) != cudaSuccess ||
                      cudaEventCreateWithFlags(&h->ctx.ev_fork, cudaEventDisableTiming) != cudaSuccess ||
                      cudaEventCreateWithFlags(&h->ctx.ev_join, cudaEventDisableTiming) != cudaSuccess))
    st = DQ_ERR_CUDA;
  if (st == DQ_OK && cudaEventCreateWithFlags(&h->ev_in, cudaEventDisableTiming) != cudaSuccess) st = DQ_ERR_CUDA;
  if (st == DQ_OK && cudaEventCreateWithFlags(&h->ev_out, cudaEventDisableTiming) != cudaSuccess) st = DQ_ERR_CUDA;
  A(dev_alloc(&h->ctx.d_status, 1));
  A(dev_alloc(&h->Z, dd)); A(dev_alloc(&h->R, dd)); A(dev_alloc(&h->U, dd));
  A(dev_alloc(&h->Gq, dd)); A(dev_alloc(&h->Gz, dd));
  A(dev_alloc(&h->ws.A, dd)); A(dev_alloc(&h->ws.V, dd)); A(dev_alloc(&h->ws.Q, dd));
  A(dev_alloc(&h->ws.Winv, dd)); A(dev_alloc(&h->ws.B, dd)); A(dev_alloc(&h->ws.S, dd));
  A(dev_alloc(&h->ws.tmp, dd));
  A(dev_alloc(&h->ws.T, (int64_t)batch * d * 32));
  A(dev_alloc(&h->ws.W, (int64_t)batch * d * 32)); A(dev_alloc(&h->ws.W2, (int64_t)batch * d * 32));
  A(dev_alloc(&h->loss_last, batch)); A(dev_alloc(&h->loss_tmp, batch));
  if (cfg->path == DQ_PATH_FP32) A(dev_alloc(&h->f32_flags, 80));
  if (st == DQ_OK) {
    for (auto& e : h->ev)
      if (cudaEventCreate(&e) != cudaSuccess) st = DQ_ERR_CUDA;
  }
  if (st == DQ_OK) st = fence_in(h);
  if (cfg->path == DQ_PATH_FP32) {
    h->g_elems = (int64_t)batch * cfg->n_tokens * d;
    float* g = nullptr;
    A(dev_alloc(&g, h->g_elems));
    h->G = g;
    h->n_partials = whip_forward_f32_tiles(cfg->n_tokens, d);
    const int tiles = ((d + 63) / 64) * ((d + 63) / 64) * batch;
    int ks = (2 * sms + tiles - 1) / tiles;
    if (ks > (int)(cfg->n_tokens / 256)) ks = (int)(cfg->n_tokens / 256);
    if (ks > 16) ks = 16;
    h->gq_ks = ks < 1 ? 1 : ks;
    if (h->gq_ks > 1) A(dev_alloc(&h->gq_part, dd * h->gq_ks));
  } else {
    h->g_elems = (int64_t)batch * cfg->n_tokens * d;
    __nv_bfloat16* g = nullptr;
    A(dev_alloc(&g, h->g_elems));
    h->G = g;
    if (st == DQ_OK) A(qr_tc_init(h->qtc, d, batch, sms));
    h->fast_qr = (st == DQ_OK);
    if (st == DQ_OK)
      A(tc_init(h->tc, h->ctx, *cfg, d_X, (__nv_bfloat16*)h->G, h->qtc.rt_hi, &h->n_partials));
  }
  if (h->small128 && cfg->path == DQ_PATH_BF16_TC) {
    A(dev_alloc(&h->p128, dd));
    A(dev_alloc(&h->R_alt, dd));
    h->tc5 = (st == DQ_OK);
  }
  A(dev_alloc(&h->partials, (int64_t)batch * (h->n_partials > 0 ? h->n_partials : 1)));
  // (the per-head fused kernel writes only the slots its launch shape uses and relies on the others being zero)
  if (st == DQ_OK && cudaMemsetAsync(h->partials, 0, sizeof(float) * (size_t)batch * (h->n_partials > 0 ? h->n_partials : 1), h->ctx.stream) != cudaSuccess) st = DQ_ERR_CUDA;
  if (st == DQ_OK && cudaMemsetAsync(h->ctx.d_status, 0, sizeof(int), h->ctx.stream) != cudaSuccess) st = DQ_ERR_CUDA;
  if (st == DQ_OK && cudaMemcpyAsync(h->Z, d_Z0, sizeof(float) * dd, cudaMemcpyDeviceToDevice, h->ctx.stream) != cudaSuccess) st = DQ_ERR_CUDA;
  if (st == DQ_OK && h->fast_qr && !h->small128) {
    // The paper initialises the latent with a random Hadamard matrix, which is orthogonal: then U = I and the
    // incremental factorisation can start at once (no Householder pass for the first step).
    bool started = false;
    st = qr_tc_try_orthogonal_start(h->ctx, h->ws, h->qtc, h->Z, d, batch, ORTHOGONAL_START_THRESHOLD, &started);
  }
  if (st == DQ_OK) st = fence_out(h);
  if (st != DQ_OK) { free_all(h); return st; }
  *out = h;
  return DQ_OK;
}

dq_status dq_calib_step(dq_calib_t* h, int32_t n_steps, float* d_loss_out) {
  if (!h || n_steps < 0) return DQ_ERR_INVALID_ARG;
  const int batch = h->cfg.batch;
  Ctx& ctx = h->ctx;
  DQ_CHECK(fence_in(h));
  if (h->timing) { for (auto& m : h->ms_acc) m = 0.0; h->timed_steps = 0; }
  for (int s = 0; s < n_steps; ++s) {
    // The captured step of the iterative QR is the incremental one: replay it only while the
    // previous step's factors belong to the latent one optimiser step back.
    const bool f32_inc = !h->small128 && !h->fast_qr && h->f32_flags && h->cfg.d <= 1024;
    const bool iterative = h->qr_method == DQ_QR_ITERATIVE && (h->small128 || h->fast_qr || f32_inc);
    const bool warm = h->small128 ? h->small_warm : (h->fast_qr ? h->qtc.t_warm : h->f32_winv_valid);
    const bool cayley = h->orth_method == DQ_ORTH_CAYLEY;
    dq_calib::StepGraph& sg = h->graph[graph_slot(h)];
    const bool use_graph = cayley ? (!h->timing && h->cay_started && h->eager_steps_done >= 1)
                                  : (!h->timing && h->r_stale != fuses_forward(h, false) && h->eager_steps_done >= 1 &&
                                     (!iterative || warm) &&
                                     (!sg.exec || !sg.needs_z_split || h->qtc.z_split_fresh));
    if (use_graph && !sg.exec && !sg.failed) try_capture(h);
    if (use_graph && sg.exec) {
      DQ_CHECK_CUDA(cudaGraphLaunch(sg.exec, ctx.stream));
      ctx.launches += sg.launches;
      ctx.mma_flops += sg.flops;
      after_replayed_step(h);
    } else {
      DQ_CHECK(enqueue_step(h, h->timing));
      h->eager_steps_done++;
      if (h->timing) {
        DQ_CHECK_CUDA(cudaEventSynchronize(h->ev[DQ_PHASE_COUNT]));
        for (int p = 0; p < DQ_PHASE_COUNT; ++p) {
          float ms = 0.f;
          DQ_CHECK_CUDA(cudaEventElapsedTime(&ms, h->ev[p], h->ev[p + 1]));
          h->ms_acc[p] += ms;
        }
        h->timed_steps++;
      }
    }
    if (d_loss_out)
      DQ_CHECK_CUDA(cudaMemcpyAsync(d_loss_out + (int64_t)s * batch, h->loss_last, sizeof(float) * batch,
                                    cudaMemcpyDeviceToDevice, ctx.stream));
  }
  return fence_out(h);
}

dq_status dq_calib_run_epochs(dq_calib_t* h, const void* d_pool, int64_t n_pool, int64_t ld_pool, float sample_ratio,
                              int32_t accum, int32_t n_epochs, uint64_t seed, float* d_loss_out,
                              int64_t* h_steps_out) {
  if (h_steps_out) *h_steps_out = 0;
  if (!h || !d_pool || n_pool <= 0 || ld_pool < h->cfg.d || accum < 1 || n_epochs < 0 ||
      !(sample_ratio > 0.f && sample_ratio <= 1.f))
    return DQ_ERR_INVALID_ARG;
  if (h->cfg.batch != 1) return DQ_ERR_UNSUPPORTED;
  const int64_t N = h->cfg.n_tokens;
  const int64_t n_sampled = (int64_t)((double)sample_ratio * (double)n_pool);
  const int64_t steps_per_epoch = n_sampled / (N * accum);
  if (steps_per_epoch < 1) return DQ_ERR_INVALID_ARG;
  DQ_CHECK(fence_in(h));
  int64_t k = 0;
  for (int e = 0; e < n_epochs; ++e) {
    for (int64_t s = 0; s < steps_per_epoch; ++s, ++k) {
      MiniBatch mb{d_pool, n_pool, ld_pool, seed + (uint64_t)e, s * accum * N, accum};
      DQ_CHECK(enqueue_step(h, false, &mb));
      h->eager_steps_done++;
      if (d_loss_out)
        DQ_CHECK_CUDA(cudaMemcpyAsync(d_loss_out + k, h->loss_last, sizeof(float), cudaMemcpyDeviceToDevice,
                                      h->ctx.stream));
    }
  }
  if (h_steps_out) *h_steps_out = k;
  return fence_out(h);
}

dq_status dq_calib_get_rotation(dq_calib_t* h, float* d_R_out) {
  if (!h || !d_R_out) return DQ_ERR_INVALID_ARG;
  DQ_CHECK(fence_in(h));
  DQ_CHECK(ensure_rotation(h));
  DQ_CHECK_CUDA(cudaMemcpyAsync(d_R_out, h->R, sizeof(float) * (size_t)h->cfg.d * h->cfg.d * h->cfg.batch,
                                cudaMemcpyDeviceToDevice, h->ctx.stream));
  return fence_out(h);
}

dq_status dq_calib_refresh_inputs(dq_calib_t* h) {
  if (!h) return DQ_ERR_INVALID_ARG;
  if (h->cfg.path != DQ_PATH_BF16_TC) return DQ_OK;
  DQ_CHECK(fence_in(h));
  DQ_CHECK(tc_refresh_inputs(h->tc, h->ctx));
  return fence_out(h);
}

dq_status dq_calib_get_latent(dq_calib_t* h, float* d_Z_out) {
  if (!h || !d_Z_out) return DQ_ERR_INVALID_ARG;
  DQ_CHECK(fence_in(h));
  DQ_CHECK_CUDA(cudaMemcpyAsync(d_Z_out, h->Z, sizeof(float) * (size_t)h->cfg.d * h->cfg.d * h->cfg.batch,
                                cudaMemcpyDeviceToDevice, h->ctx.stream));
  return fence_out(h);
}

dq_status dq_calib_set_latent(dq_calib_t* h, const float* d_Z) {
  if (!h || !d_Z) return DQ_ERR_INVALID_ARG;
  DQ_CHECK(fence_in(h));
  DQ_CHECK_CUDA(cudaMemcpyAsync(h->Z, d_Z, sizeof(float) * (size_t)h->cfg.d * h->cfg.d * h->cfg.batch,
                                cudaMemcpyDeviceToDevice, h->ctx.stream));
  DQ_CHECK(clear_status(h));
  h->r_stale = true;
  h->qtc.t_warm = false;   // the new latent may be far from the one the iterative QR last saw
  h->qtc.z_split_fresh = false;
  h->small_warm = false;
  h->f32_winv_valid = false;
  h->cay_started = false;  // Cayley SGD restarts from the orthogonal factor of the new latent
  return fence_out(h);
}

dq_status dq_calib_status(dq_calib_t* h) {
  if (!h) return DQ_ERR_INVALID_ARG;
  int code = 0;
  if (cudaMemcpyAsync(&code, h->ctx.d_status, sizeof(int), cudaMemcpyDeviceToHost, h->ctx.stream) != cudaSuccess)
    return DQ_ERR_CUDA;
  if (cudaStreamSynchronize(h->ctx.stream) != cudaSuccess) return DQ_ERR_CUDA;
  if (code < 0 || code > DQ_ERR_NOT_CONVERGED) return DQ_ERR_CUDA;
  return (dq_status)code;
}

dq_status dq_calib_set_optimizer(dq_calib_t* h, int32_t optimizer, float lr, float beta1, float beta2, float eps) {
  if (!h || !(lr == lr)) return DQ_ERR_INVALID_ARG;
  if (optimizer != DQ_SGD && optimizer != DQ_SGD_MOMENTUM && optimizer != DQ_ADAM) return DQ_ERR_INVALID_ARG;
  if (optimizer != DQ_SGD && !(beta1 >= 0.f && beta1 < 1.f)) return DQ_ERR_INVALID_ARG;
  if (optimizer == DQ_ADAM && (!(beta2 >= 0.f && beta2 < 1.f) || !(eps >= 0.f))) return DQ_ERR_INVALID_ARG;
  DQ_CHECK_CUDA(cudaStreamSynchronize(h->ctx.stream));
  const int64_t dd = (int64_t)h->cfg.d * h->cfg.d * h->cfg.batch;
  if (optimizer != DQ_SGD && !h->opt_m) DQ_CHECK(dev_alloc(&h->opt_m, dd));
  if (optimizer == DQ_ADAM && !h->opt_v) DQ_CHECK(dev_alloc(&h->opt_v, dd));
  if (optimizer == DQ_ADAM && !h->opt_pw) DQ_CHECK(dev_alloc(&h->opt_pw, 2));
  if (h->opt_m) DQ_CHECK_CUDA(cudaMemsetAsync(h->opt_m, 0, sizeof(float) * dd, h->ctx.stream));
  if (h->opt_v) DQ_CHECK_CUDA(cudaMemsetAsync(h->opt_v, 0, sizeof(float) * dd, h->ctx.stream));
  if (h->opt_pw) {
    const float ones[2] = {1.f, 1.f};
    DQ_CHECK_CUDA(cudaMemcpyAsync(h->opt_pw, ones, sizeof(ones), cudaMemcpyHostToDevice, h->ctx.stream));
    DQ_CHECK_CUDA(cudaStreamSynchronize(h->ctx.stream));
  }
  DQ_CHECK(clear_status(h));
  h->optimizer = optimizer;
  h->cfg.lr = lr;
  h->beta1 = beta1; h->beta2 = beta2; h->eps = eps;
  drop_graphs(h);
  return DQ_OK;
}

dq_status dq_calib_set_qr_method(dq_calib_t* h, int32_t method, int32_t n_iters) {
  if (!h || (method != DQ_QR_HOUSEHOLDER && method != DQ_QR_ITERATIVE) || n_iters > 64) return DQ_ERR_INVALID_ARG;
  const int iters = n_iters <= 0 ? 12 : n_iters;
  if (method == h->qr_method && iters == h->qr_iters && h->qr_iters_default == (n_iters <= 0)) return DQ_OK;
  DQ_CHECK_CUDA(cudaStreamSynchronize(h->ctx.stream));
  DQ_CHECK(clear_status(h));
  h->qr_method = method;
  h->qr_iters = iters;
  h->qr_iters_default = n_iters <= 0;
  h->r_stale = true;
  h->qtc.t_warm = false;
  h->small_warm = false;
  h->f32_winv_valid = false;
  drop_graphs(h);
  return DQ_OK;
}

dq_status dq_calib_set_objective(dq_calib_t* h, int32_t objective, int32_t bits) {
  if (!h || objective < DQ_OBJ_WHIP || objective > DQ_OBJ_QUANT || bits > 16) return DQ_ERR_INVALID_ARG;
  DQ_CHECK_CUDA(cudaStreamSynchronize(h->ctx.stream));
  if (objective != DQ_OBJ_WHIP && !h->obj.ready) {
    const dq_status st = objective_init(h->obj, h->cfg.d, h->cfg.n_tokens, h->cfg.batch);
    if (st != DQ_OK) { objective_destroy(h->obj); return st; }
  }
  DQ_CHECK(clear_status(h));
  h->obj.objective = objective;
  h->obj.bits = bits > 0 ? bits : 4;
  drop_graphs(h);
  return DQ_OK;
}

dq_status dq_calib_set_orth_method(dq_calib_t* h, int32_t method, float beta, float q, int32_t s) {
  if (!h || (method != DQ_ORTH_QR && method != DQ_ORTH_CAYLEY)) return DQ_ERR_INVALID_ARG;
  if (method == DQ_ORTH_CAYLEY) {
    if (!(beta >= 0.f && beta < 1.f) || q > 1.f || s > 16) return DQ_ERR_INVALID_ARG;
    if (!h->fast_qr || h->small128) return DQ_ERR_UNSUPPORTED;
  }
  DQ_CHECK_CUDA(cudaStreamSynchronize(h->ctx.stream));
  if (method == DQ_ORTH_CAYLEY) {
    if (!h->cay.ready) {
      const dq_status st = cayley_init(h->cay, h->cfg.d, h->cfg.batch);
      if (st != DQ_OK) { cayley_destroy(h->cay); return st; }
    }
    h->cay.beta = beta;
    h->cay.q = q > 0.f ? q : 0.5f;
    h->cay.s = s > 0 ? s : 2;
    DQ_CHECK_CUDA(cudaMemsetAsync(h->cay.M, 0, sizeof(float) * (size_t)h->cfg.d * h->cfg.d * h->cfg.batch,
                                  h->ctx.stream));
    DQ_CHECK_CUDA(cudaMemsetAsync(h->cay.alpha, 0, sizeof(float) * h->cfg.batch, h->ctx.stream));
  }
  DQ_CHECK(clear_status(h));
  h->orth_method = method;
  h->qtc.z_split_fresh = false;   // Cayley SGD uses the latent's operand buffers as scratch
  h->cay_started = false;
  h->r_stale = true;
  h->qtc.t_warm = false;
  drop_graphs(h);
  return DQ_OK;
}

dq_status dq_calib_set_keep_gradient(dq_calib_t* h, int32_t keep) {
  if (!h) return DQ_ERR_INVALID_ARG;
  const bool k = keep != 0;
  if (k == h->tc.keep_g) return DQ_OK;
  DQ_CHECK_CUDA(cudaStreamSynchronize(h->ctx.stream));
  h->tc.keep_g = k;
  drop_graphs(h);
  return DQ_OK;
}

dq_status dq_calib_set_backward_precision(dq_calib_t* h, int32_t split) {
  if (!h) return DQ_ERR_INVALID_ARG;
  const bool sp = split != 0;
  if (sp == h->bwd_split) return DQ_OK;
  DQ_CHECK_CUDA(cudaStreamSynchronize(h->ctx.stream));
  h->bwd_split = sp;
  drop_graphs(h);
  return DQ_OK;
}

dq_status dq_calib_selftest_bounded_wait(dq_calib_t* h, uint64_t limit_ns, uint64_t* d_waited_ns) {
  if (!h || limit_ns == 0 || limit_ns > 100000000ull) return DQ_ERR_INVALID_ARG;   // at most 0.1 s
  if (h->cfg.path != DQ_PATH_BF16_TC) return DQ_ERR_UNSUPPORTED;
  DQ_CHECK(fence_in(h));
  DQ_CHECK(bounded_wait_probe(h->ctx, limit_ns, d_waited_ns));
  return fence_out(h);
}

dq_status dq_calib_time_product(dq_calib_t* h, int32_t nterms, int32_t reps, float* h_ms) {
  if (!h || !h_ms || (nterms != 1 && nterms != 3) || reps < 1 || reps > 1000) return DQ_ERR_INVALID_ARG;
  if (!h->fast_qr || h->small128) return DQ_ERR_UNSUPPORTED;
  DQ_CHECK(fence_in(h));
  const int64_t launches = h->ctx.launches;
  const double flops = h->ctx.mma_flops;
  DQ_CHECK(qr_tc_bench_product(h->ctx, h->ws, h->qtc, h->cfg.d, h->cfg.batch, nterms));   // warm-up
  DQ_CHECK_CUDA(cudaEventRecord(h->ev[0], h->ctx.stream));
  for (int r = 0; r < reps; ++r) DQ_CHECK(qr_tc_bench_product(h->ctx, h->ws, h->qtc, h->cfg.d, h->cfg.batch, nterms));
  DQ_CHECK_CUDA(cudaEventRecord(h->ev[1], h->ctx.stream));
  DQ_CHECK_CUDA(cudaEventSynchronize(h->ev[1]));
  float ms = 0.f;
  DQ_CHECK_CUDA(cudaEventElapsedTime(&ms, h->ev[0], h->ev[1]));
  *h_ms = ms / reps;
  h->ctx.launches = launches;      // measurement launches are not part of the calibration's counts
  h->ctx.mma_flops = flops;
  return fence_out(h);
}

dq_status dq_calib_set_timing(dq_calib_t* h, int32_t enabled) {
  if (!h) return DQ_ERR_INVALID_ARG;
  h->timing = enabled != 0;
  return DQ_OK;
}

dq_status dq_calib_get_timings(dq_calib_t* h, float* h_ms_by_phase, int32_t n) {
  if (!h || !h_ms_by_phase || n < 0) return DQ_ERR_INVALID_ARG;
  for (int p = 0; p < n && p < DQ_PHASE_COUNT; ++p)
    h_ms_by_phase[p] = h->timed_steps > 0 ? (float)(h->ms_acc[p] / h->timed_steps) : 0.f;
  return DQ_OK;
}

dq_status dq_calib_debug_buffer(dq_calib_t* h, int32_t which, void** d_ptr, int64_t* n_elems) {
  if (!h || !d_ptr || !n_elems) return DQ_ERR_INVALID_ARG;
  const int64_t dd = (int64_t)h->cfg.d * h->cfg.d * h->cfg.batch;
  switch (which) {
    case DQ_BUF_R: *d_ptr = h->R_used ? h->R_used : h->R; *n_elems = dd; break;   // the rotation the last step used
    case DQ_BUF_U:
      if (h->tc5 && h->small_warm && !h->u128_fresh) return DQ_ERR_UNSUPPORTED;   // only U^-1 is carried there
      if (h->fast_qr && !h->small128 && !h->qtc.u_fresh && h->orth_method == DQ_ORTH_QR && h->qtc.t_warm) {
        // the incremental factorisation carries U^-1 only: invert it for the view
        DQ_CHECK(fence_in(h));
        DQ_CHECK(qr_tc_materialize_u(h->ctx, h->ws, h->qtc, h->U, h->cfg.d, h->cfg.batch));
        DQ_CHECK(fence_out(h));
      }
      *d_ptr = h->U; *n_elems = dd; break;
    case DQ_BUF_GQ: *d_ptr = h->Gq; *n_elems = dd; break;
    case DQ_BUF_GZ: *d_ptr = h->Gz; *n_elems = dd; break;
    case DQ_BUF_G: *d_ptr = h->G; *n_elems = h->g_elems; break;
    case DQ_BUF_PARTIALS: *d_ptr = h->partials; *n_elems = (int64_t)h->n_partials * h->cfg.batch; break;
    case DQ_BUF_Z: *d_ptr = h->Z; *n_elems = dd; break;
    case DQ_BUF_OPT_M: *d_ptr = h->opt_m; *n_elems = h->opt_m ? dd : 0; break;
    case DQ_BUF_OPT_V: *d_ptr = h->opt_v; *n_elems = h->opt_v ? dd : 0; break;
    case DQ_BUF_CAYLEY_M: *d_ptr = h->cay.M; *n_elems = h->cay.M ? dd : 0; break;
    case DQ_BUF_CAYLEY_ALPHA: *d_ptr = h->cay.alpha; *n_elems = h->cay.alpha ? h->cfg.batch : 0; break;
    default: return DQ_ERR_INVALID_ARG;
  }
  return DQ_OK;
}

int64_t dq_calib_launch_count(dq_calib_t* h) { return h ? h->ctx.launches : 0; }

double dq_calib_mma_flops(dq_calib_t* h) { return h ? h->ctx.mma_flops : 0.0; }

void dq_calib_destroy(dq_calib_t* h) {
  if (!h) return;
  cudaStreamSynchronize(h->ctx.stream);
  free_all(h);
}

dq_status dq_rotate_apply(const void* d_X, int32_t x_dtype, int64_t n, int32_t d, int64_t ldx,
                          const float* d_R, void* d_Y, int64_t ldy, void* cuda_stream) {
  if (!d_X || !d_R || !d_Y || n <= 0 || d <= 0 || ldx < d || ldy < d) return DQ_ERR_INVALID_ARG;
  Ctx ctx;
  ctx.stream = (cudaStream_t)cuda_stream;
  if (x_dtype == DQ_FP32) {
    GemmDesc g{};
    g.A = (const float*)d_X; g.lda = ldx; g.transA = 0; g.sA = 0;
    g.B = d_R; g.ldb = d; g.transB = 0; g.sB = 0;
    g.C = (float*)d_Y; g.ldc = ldy; g.sC = 0;
    g.M = (int)n; g.N = d; g.K = d; g.alpha = 1.f; g.beta = 0.f; g.batch = 1;
    return gemm_f32(ctx, g);
  }
  if (x_dtype == DQ_BF16) return tc_rotate_apply(ctx, d_X, n, d, ldx, d_R, d_Y, ldy);
  return DQ_ERR_INVALID_ARG;
}

dq_status dq_eval_rotation(const void* d_X, int32_t x_dtype, int64_t n, int32_t d, int64_t ldx, const float* d_R,
                           float tau, int32_t bits, double* d_out, void* cuda_stream) {
  if (!d_X || !d_R || !d_out || n <= 0 || d <= 0 || ldx < d) return DQ_ERR_INVALID_ARG;
  if (x_dtype != DQ_FP32 && x_dtype != DQ_BF16) return DQ_ERR_INVALID_ARG;
  Ctx ctx;
  ctx.stream = (cudaStream_t)cuda_stream;
  return eval_rotation(ctx, d_X, x_dtype, n, d, ldx, d_R, tau, bits, d_out);
}

dq_status dq_gather_tokens(const void* d_X, int32_t x_dtype, int64_t n_total, int32_t d, int64_t ldx, uint64_t seed,
                           int64_t first, int64_t count, void* d_out, int64_t ldo, void* cuda_stream) {
  if (!d_X || !d_out || n_total <= 0 || d <= 0 || ldx < d || ldo < d || first < 0 || count < 0 ||
      first + count > n_total)
    return DQ_ERR_INVALID_ARG;
  if (x_dtype != DQ_FP32 && x_dtype != DQ_BF16) return DQ_ERR_INVALID_ARG;
  Ctx ctx;
  ctx.stream = (cudaStream_t)cuda_stream;
  return gather_tokens(ctx, d_X, x_dtype == DQ_FP32 ? 4 : 2, n_total, d, ldx, seed, first, count, d_out, ldo);
}

dq_status dq_rotate_apply_static(const void* d_X, int64_t n, int32_t d, int64_t ldx, const float* d_R,
                                 void* d_Y, int64_t ldy, void* cuda_stream) {
  if (!d_X || !d_R || !d_Y || n <= 0 || d <= 0 || ldx < d || ldy < d) return DQ_ERR_INVALID_ARG;
  Ctx ctx;
  ctx.stream = (cudaStream_t)cuda_stream;
  return tc_rotate_apply_static(ctx, d_X, n, d, ldx, d_R, d_Y, ldy);
}

}  // extern "C"
