// Tensor-core (tcgen05 / TMEM / TMA) path of the two large contractions.
#pragma once
#include "common.cuh"

namespace dq {

struct TcState {
  bool ready = false;
  int d = 0, batch = 0;
  int64_t n_tokens = 0;
  const __nv_bfloat16* X = nullptr;   // [batch][N][d] token-major (borrowed)
  __nv_bfloat16* Xt = nullptr;        // [batch][d][N] channel-major copy (owned)
  __nv_bfloat16* Rt = nullptr;        // [batch][d][d] bf16(R^T) (owned)
  __nv_bfloat16* Gt = nullptr;        // [batch][d][N] dL/dO, channel-major (borrowed from handle)
  float* part = nullptr;              // split-K partials of Gq (owned)
  int ksplit = 1;
  void* maps = nullptr;               // host array of CUtensorMap
  int n_partials = 0;
};

dq_status tc_init(TcState& tc, Ctx& ctx, const dq_calib_config& cfg, const void* d_X,
                  __nv_bfloat16* Gt, int* n_partials);
void tc_destroy(TcState& tc);
dq_status tc_refresh_inputs(TcState& tc, Ctx& ctx);   // X changed in place: rebuild X^T
inline __nv_bfloat16* tc_rt_operand(TcState& tc) { return tc.ready ? tc.Rt : nullptr; }
dq_status tc_whip_forward(TcState& tc, Ctx& ctx, float* partials);
dq_status tc_grad_rotation(TcState& tc, Ctx& ctx, float* Gq, float scale);
dq_status tc_rotate_apply(Ctx& ctx, const void* d_X, int64_t n, int d, int64_t ldx, const float* d_R,
                          void* d_Y, int64_t ldy);

}  // namespace dq
