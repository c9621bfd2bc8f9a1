// Sparse/dense step schedule (Section 5.3.2) and the speed-up arithmetic of Sections 3.1 and 5.1:
// host-side logic plus two dispatchers that run the step kind a schedule assigns to a step.
#include "sf_common.cuh"

#define SF_TRY(expr)              \
  do {                            \
    int _st = (expr);             \
    if (_st != SF_OK) return _st; \
  } while (0)

namespace {

int check_schedule(const sf_schedule* sc) {
  if (!sc) return SF_ERR_NULL;
  if (sc->warmup_steps < 0 || sc->sparse_steps < 0 || sc->total_steps <= 0) return SF_ERR_SHAPE;
  if (sc->warmup_steps > sc->total_steps - sc->sparse_steps) return SF_ERR_SHAPE;
  return SF_OK;
}

}  // namespace

extern "C" {

int sf_schedule_step_kind(const sf_schedule* schedule, int64_t step, int* kind) {
  if (!kind) return SF_ERR_NULL;
  SF_TRY(check_schedule(schedule));
  if (step < 0 || step >= schedule->total_steps) return SF_ERR_SHAPE;
  const int64_t first = schedule->warmup_steps, last = first + schedule->sparse_steps;
  *kind = (step >= first && step < last) ? SF_STEP_SPARSE : SF_STEP_DENSE;
  return SF_OK;
}

int sf_schedule_speedup(const sf_schedule* schedule, double sparse_step_speedup, double* speedup) {
  if (!speedup) return SF_ERR_NULL;
  SF_TRY(check_schedule(schedule));
  if (!(sparse_step_speedup > 0.0)) return SF_ERR_SHAPE;
  const double sparse = (double)schedule->sparse_steps, total = (double)schedule->total_steps;
  *speedup = total / (sparse / sparse_step_speedup + (total - sparse));
  return SF_OK;
}

int sf_ffn_flop_fraction(int64_t D, int64_t F, int64_t n_q_heads, int64_t n_kv_heads, int64_t head_dim,
                         double* fraction) {
  if (!fraction) return SF_ERR_NULL;
  if (D <= 0 || F <= 0 || n_q_heads < 0 || n_kv_heads < 0 || head_dim < 0) return SF_ERR_SHAPE;
  const double ffn = 3.0 * (double)D * (double)F;
  const double attn = 2.0 * (double)D * (double)(n_q_heads + n_kv_heads) * (double)head_dim;
  *fraction = ffn / (ffn + attn);
  return SF_OK;
}

int sf_end_to_end_speedup(double ffn_fraction, double ffn_speedup, double* speedup) {
  if (!speedup) return SF_ERR_NULL;
  if (!(ffn_fraction >= 0.0 && ffn_fraction <= 1.0) || !(ffn_speedup > 0.0)) return SF_ERR_SHAPE;
  *speedup = 1.0 / ((1.0 - ffn_fraction) + ffn_fraction / ffn_speedup);
  return SF_OK;
}

int sf_ffn_fwd_scheduled(const sf_schedule* schedule, int64_t step, const sf_ffn_desc* desc, const void* X,
                         const void* W1, const void* W2, void* Y, void* fwd_ctx, size_t fwd_ctx_bytes, void* workspace,
                         size_t workspace_bytes, void* stream) {
  int kind = SF_STEP_DENSE;
  SF_TRY(sf_schedule_step_kind(schedule, step, &kind));
  return kind == SF_STEP_SPARSE
             ? sf_sparse_ffn_fwd(desc, X, W1, W2, Y, fwd_ctx, fwd_ctx_bytes, workspace, workspace_bytes, stream)
             : sf_dense_ffn_fwd(desc, X, W1, W2, Y, fwd_ctx, fwd_ctx_bytes, workspace, workspace_bytes, stream);
}

int sf_ffn_bwd_scheduled(const sf_schedule* schedule, int64_t step, const sf_ffn_desc* desc, const void* dY,
                         const void* X, const void* W1, const void* W2, const void* fwd_ctx, size_t fwd_ctx_bytes,
                         void* dX, void* dW1, void* dW2, void* workspace, size_t workspace_bytes, void* stream) {
  int kind = SF_STEP_DENSE;
  SF_TRY(sf_schedule_step_kind(schedule, step, &kind));
  return kind == SF_STEP_SPARSE ? sf_sparse_ffn_bwd(desc, dY, X, W1, W2, fwd_ctx, fwd_ctx_bytes, dX, dW1, dW2, workspace,
                                                    workspace_bytes, stream)
                                : sf_dense_ffn_bwd(desc, dY, X, W1, W2, fwd_ctx, fwd_ctx_bytes, dX, dW1, dW2, workspace,
                                                   workspace_bytes, stream);
}

}  // extern "C"
