// Tensor-core (tcgen05 / TMEM / TMA) path of the two large contractions.
#pragma once
#include "common.cuh"

namespace dq {

struct TcState {
  bool ready = false;
  int d = 0, batch = 0;
  int64_t n_tokens = 0, ldx = 0;
  const __nv_bfloat16* X = nullptr;   // [batch][N][ldx] token-major (borrowed)
  __nv_bfloat16* Rt = nullptr;        // [batch][d][d] bf16(R^T) (owned unless rt_external)
  bool rt_external = false;
  __nv_bfloat16* Gt = nullptr;        // [batch][d][N] dL/dO, channel-major (borrowed from handle)
  float* part = nullptr;              // split-K partials of Gq (owned)
  int ksplit = 1;
  void* maps = nullptr;               // host array of CUtensorMap
  int n_partials = 0;
  bool pair = false;                  // 256 x 256 tiles on CTA pairs (tcgen05 cta_group::2) for both contractions
  // Gq = X^T G when the tile count is not a multiple of the SM count: the last, partly filled
  // wave of tiles is computed with its reduction split in `tail_split` slices instead
  int* tl_head = nullptr; int n_head = 0;
  int* tl_tail = nullptr; int n_tail = 0;
  int tail_split = 1;
  float* tail_part = nullptr;         // [tail_split][d][d] (only the tail tiles are touched)
  // d == 128: both contractions and the Eq. 4 epilogue in one kernel (tc_heads.cuh); dL/dO stays on chip
  bool fused = false;
  int splits = 1;                     // units per head (each covers a range of token tiles)
  float* heads_part = nullptr;        // [batch * splits][128][128] partial Gq
  bool keep_g = false;                // also store dL/dO to Gt (inspection / tests)
  bool fused_valid = false;           // heads_part holds the partials of the current step
  int n_partials_live = 0;            // loss partials per problem written by the last forward
};

dq_status tc_init(TcState& tc, Ctx& ctx, const dq_calib_config& cfg, const void* d_X,
                  __nv_bfloat16* Gt, __nv_bfloat16* rt_external, int* n_partials);
void tc_destroy(TcState& tc);
dq_status tc_refresh_inputs(TcState& tc, Ctx& ctx);   // X changed in place: nothing derived from it is kept
inline __nv_bfloat16* tc_rt_operand(TcState& tc) { return tc.ready ? tc.Rt : nullptr; }
dq_status tc_whip_forward(TcState& tc, Ctx& ctx, float* partials);
dq_status tc_grad_rotation(TcState& tc, Ctx& ctx, float* Gq, float scale, __nv_bfloat16* gqt = nullptr,
                           bool* gqt_written = nullptr);
dq_status tc_rotate_apply(Ctx& ctx, const void* d_X, int64_t n, int d, int64_t ldx, const float* d_R,
                          void* d_Y, int64_t ldy);
// Failure-detection self-test: the library's bounded in-kernel wait on a barrier nobody arrives at.
dq_status bounded_wait_probe(Ctx& ctx, uint64_t limit_ns, uint64_t* d_waited_ns);
// Outliers (Eq. 1) and per-token asymmetric quantisation error of O = X R (eval_metrics.cu).
dq_status eval_rotation(Ctx& ctx, const void* d_X, int x_dtype, int64_t n, int d, int64_t ldx, const float* d_R,
                        float tau, int bits, double* d_out);
// Same product with its scratch in a file-scope device array: no allocation of any kind.
dq_status tc_rotate_apply_static(Ctx& ctx, const void* d_X, int64_t n, int d, int64_t ldx, const float* d_R,
                                 void* d_Y, int64_t ldy);


// Split-bf16 operand copies used by the tensor-core QR-Orth (all [batch][d][d]).
struct QrTcState {
  bool ready = false;
  __nv_bfloat16 *z_hi = nullptr, *z_lo = nullptr;       // latent Z
  __nv_bfloat16 *u_hi = nullptr, *u_lo = nullptr;       // upper factor U
  __nv_bfloat16 *wn_hi = nullptr, *wn_lo = nullptr;     // W = U^-1, row-major
  __nv_bfloat16 *wt_hi = nullptr, *wt_lo = nullptr;     // W^T
  __nv_bfloat16 *r_hi = nullptr, *r_lo = nullptr;       // R
  __nv_bfloat16 *rt_hi = nullptr, *rt_lo = nullptr;     // R^T (rt_hi is also the operand of X R)
  __nv_bfloat16 *gqt_hi = nullptr, *gqt_lo = nullptr;   // Gq^T
  __nv_bfloat16 *st_hi = nullptr, *st_lo = nullptr;     // S^T
  __nv_bfloat16 *m_hi = nullptr, *m_lo = nullptr;       // R S
  __nv_bfloat16 *t1_hi = nullptr, *t1_lo = nullptr;     // scratch of the block inversion
  // second set of copies of W: the incremental update W <- W (I + T)^-1 reads one set and writes the other
  __nv_bfloat16 *wn2_hi = nullptr, *wn2_lo = nullptr;
  int w_sel = 0;                                        // the set that holds the current W (0: wn / wt, 1: wn2 / wt2)
  float* P = nullptr;                                   // T^T T of the last sweep: where the next step's fixed point starts
  __nv_bfloat16 *yt_hi = nullptr, *yt_lo = nullptr;     // Y = (I + T)^-1 - I (row-major split copy)
  __nv_bfloat16 *nm1 = nullptr, *nm2 = nullptr;         // scratch of the products that form (I + T)^-1
  bool u_fresh = false;                                 // U and u_hi / u_lo hold the upper factor of the current factorisation
  bool gqt_fresh = false;                               // gqt_hi holds bf16(Gq^T) of the current step (written by the contraction)
  // blocked Householder factorisation with tensor-core trailing updates
  __nv_bfloat16 *y_hi = nullptr, *y_lo = nullptr;       // [batch][d][128] reflector block Y of the outer block
  __nv_bfloat16 *w2_hi = nullptr, *w2_lo = nullptr;     // [batch][d][128] (T^T Y^T C)^T
  float* part = nullptr;                                // split partials of [S; W^T]
  int64_t part_bs = 0;                                  // elements per problem
  float* T = nullptr;                                   // [batch][4][32][32] compact-WY factors of the inner panels
  // near-orthogonal iterative factorisation
  __nv_bfloat16 *tw_hi = nullptr, *tw_lo = nullptr;     // T of the sweeps (alternates with t1_hi / t1_lo)
  bool z_split_fresh = false;                           // z_hi / z_lo are the split copy of the current latent
  bool t_warm = false;                                  // the current set of W copies and the fp32 W belong to the previous step's latent
  int* sweep_flags = nullptr;                           // [80] device flags: sweep k moved an entry
  // Tile orders for triangular products (device arrays of mb | nb << 16).  The persistent workers (CTAs, or CTA
  // pairs) take list entries round-robin, so each list is laid out for its number of workers and for the cost
  // of its tiles (the k-blocks that the product's k_mode leaves): every worker gets the same number of tiles
  // to within one and nearly the same number of k-blocks, its lightest tile first.
  int* tl_upper = nullptr; int n_upper = 0;             // tiles mb <= nb, all k-blocks (uniform cost)
  int* tl_upper_k2 = nullptr;                           // the same tiles for k_mode 2 (k-blocks up to mb)
  int* tl_upper_band = nullptr;                         // the same tiles for k_mode 1|4 (k-blocks mb .. nb)
  int* tl_lower = nullptr;                              // tiles mb >= nb (n_upper of them), uniform cost
  int* tl_k4 = nullptr;                                 // all tiles for k_mode 4 (k-blocks up to nb)
  int* tl_k8 = nullptr; int n_all = 0;                  // all tiles for k_mode 8 (k-blocks from nb)
  // the same orders in 256 x 256 tiles for the two-CTA kernel (d % 256 == 0 only)
  int* tl2_upper = nullptr; int n2_upper = 0;
  int* tl2_upper_k2 = nullptr;
  int* tl2_upper_band = nullptr;
  int* tl2_lower = nullptr;
  int* tl2_k4 = nullptr;
  int* tl2_k8 = nullptr; int n2_all = 0;
};
dq_status qr_tc_init(QrTcState& q, int d, int batch, int sm_count);
void qr_tc_destroy(QrTcState& q);
// iterative_iters > 0 and q.t_warm: R and W = U^-1 from the previous step's W by fixed-point sweeps (no
// dependent column steps; U itself is not formed); otherwise blocked Householder (U is written).
// need_lo: the incremental route also writes the lo parts of the split copies of R and R^T (the Householder
// route always does).
dq_status qr_forward_fast(Ctx& ctx, QrWorkspace& ws, QrTcState& q, const float* Z, float* R, float* U, int d,
                          int batch, int iterative_iters, bool need_lo);
// If |Z^T Z - I|_F <= threshold for every problem: installs W = I so that the incremental route can factor Z
// without a Householder start (*started = true).  Synchronises the stream.
dq_status qr_tc_try_orthogonal_start(Ctx& ctx, QrWorkspace& ws, QrTcState& q, const float* Z, int d, int batch,
                                     float threshold, bool* started);
// Measurement: one dense d^3 product on the handle's operand copies (nterms = 3: split-bf16; 1: plain bf16).
dq_status qr_tc_bench_product(Ctx& ctx, QrWorkspace& ws, QrTcState& q, int d, int batch, int nterms);
// Makes U hold the upper factor of the current factorisation (inverts W after incremental steps).
dq_status qr_tc_materialize_u(Ctx& ctx, QrWorkspace& ws, QrTcState& q, float* U, int d, int batch);
// split: three bf16 MMAs per product (split operands) instead of one.
dq_status qr_backward_tc(Ctx& ctx, QrWorkspace& ws, QrTcState& q, const float* Gq, float* Gz, int d, int batch,
                         bool split);

// Alternative objectives of the ablation in Sec. 5.3 (objectives.cu).
struct ObjectiveState {
  bool ready = false;
  int objective = DQ_OBJ_WHIP, bits = 4;
  float* O = nullptr;          // [chunk][d] fp32 rotated activations of one chunk of tokens
  int64_t chunk = 0;
  double* tok_loss = nullptr;  // [chunk] per-token objective
  double* acc = nullptr;       // [batch] sum over tokens
};
dq_status objective_init(ObjectiveState& os, int d, int64_t n_tokens, int batch);
void objective_destroy(ObjectiveState& os);
dq_status objective_forward(Ctx& ctx, ObjectiveState& os, const dq_calib_config& cfg, const void* X, const float* R,
                            const __nv_bfloat16* rt, void* G, float loss_scale, float* loss_last);

// Cayley SGD with momentum (Algorithm 3) on the rotation itself (cayley_tc.cu).
struct CayleyState {
  bool ready = false;
  float* M = nullptr;        // [batch][d][d] momentum
  float* part = nullptr;     // [batch][n_part] partial sums of |W|_F^2
  float* alpha = nullptr;    // [batch] step size of the current iteration
  int n_part = 0;
  float beta = 0.f, q = 0.5f, eps = 1e-8f;
  int s = 2;
};
dq_status cayley_init(CayleyState& cs, int d, int batch);
void cayley_destroy(CayleyState& cs);
// One update R <- Cayley step of (R, M, Gq); needs q.r_* / q.rt_* to hold the split copies of R and
// leaves them holding those of the new R.  Uses ws.B, ws.S, ws.tmp and the split scratch of q.
dq_status cayley_step_tc(Ctx& ctx, QrWorkspace& ws, QrTcState& q, CayleyState& cs, float* R, const float* Gq,
                         float lr, int d, int batch);


// Kernels of the blocked Householder factorisation on a transposed working matrix
// (qr_panel_tc.cu); the tensor-core products between them are issued by qr_tc.cu.
dq_status qrp_transpose_split(Ctx& ctx, const float* Z, float* At, __nv_bfloat16* hi, __nv_bfloat16* lo, int d,
                              int batch);
dq_status qrp_panel(Ctx& ctx, float* At, __nv_bfloat16* at_hi, __nv_bfloat16* at_lo, __nv_bfloat16* y_hi,
                    __nv_bfloat16* y_lo, float* Tk, int d, int c0, int batch);
dq_status qrp_wy_w2(Ctx& ctx, const float* part, int ksplit, int m, int64_t part_bs, const float* Tk,
                    __nv_bfloat16* w2_hi, __nv_bfloat16* w2_lo, int64_t w2_bs, int n, int batch);
dq_status qrp_gauge_ut(Ctx& ctx, const float* At, float* U, __nv_bfloat16* hi, __nv_bfloat16* lo, int d, int batch);

}  // namespace dq
