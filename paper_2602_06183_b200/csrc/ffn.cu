// Step orchestration (Algorithms 1 and 2; Eqs. 1-8 for the dense phase) and the product entry
// points of the C ABI. Everything is enqueued on the caller's stream; buffers are carved out of
// the caller's context / workspace; no device memory is allocated here. (The host-buffer step
// additionally owns two copy streams and a few events per device, created on first use.)
#include "sf_common.cuh"
#include "gemm_tc.cuh"

#include <initializer_list>

namespace sf {

namespace {

constexpr size_t kAlign = 256;
constexpr size_t kStatusBytes = 256;       // status word lives at the start of every workspace

inline size_t up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

// Optional stage tracing: caller-owned CUDA events recorded between the kernels of a step.
cudaEvent_t* g_trace_events = nullptr;
int g_trace_cap = 0, g_trace_n = 0;

// Copy/compute overlap of the host-buffer step: while sf_ffn_step_host runs, the step functions wait
// for an operand's upload right before its first use and signal a result as soon as its product is
// enqueued. Null outside sf_ffn_step_host.
struct StepHooks {
  cudaEvent_t w2_ready;      // forward: waited before the first kernel that reads W2
  cudaEvent_t dx_done;       // backward: recorded after the dX product
  cudaEvent_t dw2_done;      // backward: recorded after the dW2 product
};
thread_local const StepHooks* g_hooks = nullptr;   // per host thread: other threads' steps see no hooks

inline void hook_wait_w2(cudaStream_t s) {
  if (g_hooks) cudaStreamWaitEvent(s, g_hooks->w2_ready, 0);
}
inline void hook_dx_done(cudaStream_t s) {
  if (g_hooks) cudaEventRecord(g_hooks->dx_done, s);
}
inline void hook_dw2_done(cudaStream_t s) {
  if (g_hooks) cudaEventRecord(g_hooks->dw2_done, s);
}

// Per-device copy streams and events of the host-buffer step, created on first use.
struct HostStepResources {
  bool ready = false;
  cudaStream_t up = nullptr, down = nullptr;
  cudaEvent_t begin, xw1, w2, dy, y, dx, dw2, dw1, done;
};
constexpr int kMaxDevices = 64;
HostStepResources g_host_step[kMaxDevices];

int host_step_resources(HostStepResources** out) {
  int dev = 0;
  SF_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return SF_ERR_UNSUPPORTED;
  HostStepResources& r = g_host_step[dev];
  if (!r.ready) {
    SF_CUDA_TRY(cudaStreamCreateWithFlags(&r.up, cudaStreamNonBlocking));
    SF_CUDA_TRY(cudaStreamCreateWithFlags(&r.down, cudaStreamNonBlocking));
    for (cudaEvent_t* e : {&r.begin, &r.xw1, &r.w2, &r.dy, &r.y, &r.dx, &r.dw2, &r.dw1, &r.done})
      SF_CUDA_TRY(cudaEventCreateWithFlags(e, cudaEventDisableTiming));
    r.ready = true;
  }
  *out = &r;
  return SF_OK;
}

// ---- small helper kernels -------------------------------------------------------------------

__global__ void meta_reorder_kernel(const uint16_t* __restrict__ meta, uint8_t* __restrict__ meta_hw, int64_t R,
                                    int64_t K) {
  const int64_t words = K >> 4;
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= R * words) return;
  const int64_t m = idx / words, kw = idx - m * words;
  *reinterpret_cast<uint16_t*>(meta_hw + meta_hw_offset(m, kw, K)) = meta[idx];
}

// vals[t, 2g + j] = dense[t, g*Mv + colidx[t/V, g, pos_j]] with pos from the canonical nibble.
__global__ void pack_like_kernel(const uint16_t* __restrict__ dense, const uint16_t* __restrict__ meta,
                                 const uint8_t* __restrict__ colidx, uint16_t* __restrict__ vals, int64_t T,
                                 int64_t F, int V, int Mv) {
  const int64_t G = F / Mv, words = G >> 2;
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= T * words) return;
  const int64_t t = idx / words, kw = idx - t * words;
  const uint32_t mw = meta[idx];
  const uint4 c16 = *reinterpret_cast<const uint4*>(colidx + (((t / V) * G) + kw * 4) * 4);
  const uint32_t cw[4] = {c16.x, c16.y, c16.z, c16.w};
  uint32_t out[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const uint32_t nib = (mw >> (4 * j)) & 0xFu;
    const uint32_t ca = (cw[j] >> (8 * (nib & 3u))) & 0xFFu, cb = (cw[j] >> (8 * (nib >> 2))) & 0xFFu;
    const uint16_t* grp = dense + t * F + (kw * 4 + j) * Mv;
    out[j] = (uint32_t)grp[ca] | ((uint32_t)grp[cb] << 16);
  }
  *reinterpret_cast<uint4*>(vals + t * (2 * G) + kw * 8) = make_uint4(out[0], out[1], out[2], out[3]);
}

// ---- context / workspace carving ---------------------------------------------------------------

struct SparseLayout {
  // forward context
  size_t y2_vals, relu_vals, meta, meta_hw, colidx, y2_dense, relu_dense, w2t, y1, vals24, meta24, meta24_hw, relu24,
      ctx_total;
  // workspace (after the status block)
  size_t w1_vals, w1_meta, w1_meta_hw, ws_y1, w2_vals, w2_meta, w2_meta_hw, dy1_dense, dy1_vals, dy1_vals24,
      ws_total;
  bool plain24;   // activations are fed to the tensor cores as plain 2:4 over all F columns
  bool packed8;   // M = 8: ReLU(y1) and the operands of the sparse products exist in the 2:4 layout only
  bool fused;     // packed8 and the activation is sparsified inside the y1 product's epilogue
  bool expand;    // packed8 and the weight-gradient products expand their masked operand from its packed form
                  // (no masked [T, F] copy of y2 or dy1 exists at all)
};

constexpr size_t kNone = (size_t)-1;

SparseLayout sparse_layout(const sf_ffn_desc& d) {
  SparseLayout L{};
  const size_t T = d.T, D = d.D, F = d.F, G = F / d.M;
  // M <= 8: every V:N:M row is also a legal 2:4 row over all F columns, and on this hardware the
  // ungathered 2:4 product (twice the tensor work, no row gather) is the faster of the two.
  L.plain24 = (d.M == 4) || (d.M == 8 && vnm_has_24_view(d.F, d.V, d.M));
  L.packed8 = d.M == 8 && L.plain24;
  // The fused epilogue needs whole V-blocks inside a token tile: three blocks of 64 in a 192-column tile cost
  // 9 % more operand traffic than the plain product's 224 columns, one block of 128 in a 128-column tile 28 %
  // more, which outweighs the saved kernel: V = 128 fuses only on request.
  const bool can_fuse = L.packed8 && gemm_sparse24_vnm8_supported(d.F, d.T, d.D, d.V);
  L.fused = can_fuse && !(d.flags & SF_FFN_UNFUSED_ACT) && (d.V == 64 || (d.flags & SF_FFN_FUSED_ACT));
  L.expand = L.packed8 && (d.flags & SF_FFN_PACKED_GRAD_OPERANDS);
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t r = o; o += up(bytes); return r; };
  L.y2_vals = take(T * 2 * G * 2);
  L.relu_vals = take(T * 2 * G * 2);
  L.meta = take(T * G / 2);
  L.colidx = take((T / d.V) * G * 4);
  L.y1 = (d.flags & SF_FFN_SAVE_Y1) ? take(T * F * 2) : kNone;
  if (L.packed8) {
    L.vals24 = take(T * F);
    L.relu24 = take(T * F);
    L.meta24 = take(T * F / 8);
    L.meta24_hw = take(T * F / 8);
    L.y2_dense = L.expand ? kNone : take(T * F * 2);
    L.meta_hw = L.relu_dense = L.w2t = kNone;
  } else {
    L.meta_hw = take(T * G / 2);
    L.y2_dense = take(T * F * 2);
    L.relu_dense = take(T * F * 2);
    L.w2t = L.plain24 ? kNone : take(F * D * 2);
    L.vals24 = L.y2_vals; L.meta24 = L.meta; L.meta24_hw = L.meta_hw;   // M == 4: the packed form is already 2:4
    L.relu24 = kNone;
  }
  L.ctx_total = o;
  o = kStatusBytes;
  L.w1_vals = take(F * D);
  L.w1_meta = take(F * D / 8);
  L.w1_meta_hw = take(F * D / 8);
  L.ws_y1 = ((d.flags & SF_FFN_SAVE_Y1) || L.fused) ? kNone : take(T * F * 2);
  L.w2_vals = take(F * D);
  L.w2_meta = take(F * D / 8);
  L.w2_meta_hw = take(F * D / 8);
  if (L.packed8) {
    L.dy1_vals24 = take(T * F);
    L.dy1_dense = L.expand ? kNone : take(T * F * 2);
    L.dy1_vals = kNone;
  } else {
    L.dy1_dense = take(T * F * 2);
    L.dy1_vals = take(T * 2 * G * 2);
    L.dy1_vals24 = L.dy1_vals;
  }
  L.ws_total = o;
  return L;
}

struct DenseLayout { size_t y1, h, ctx_total, dy1, ws_total; };

DenseLayout dense_layout(const sf_ffn_desc& d) {
  DenseLayout L{};
  const size_t T = d.T, F = d.F;
  L.y1 = 0;
  L.h = up(T * F * 2);
  L.ctx_total = L.h + up(T * F * 2);
  L.dy1 = kStatusBytes;
  L.ws_total = kStatusBytes + up(T * F * 2);
  return L;
}

int check_desc(const sf_ffn_desc* d) {
  if (!d) return SF_ERR_NULL;
  if (d->N != 2) return SF_ERR_UNSUPPORTED;
  if (d->M != 4 && d->M != 8 && d->M != 16 && d->M != 32 && d->M != 64) return SF_ERR_SHAPE;
  if (d->flags & ~(SF_FFN_SAVE_Y1 | SF_FFN_UNFUSED_ACT | SF_FFN_FUSED_ACT | SF_FFN_PACKED_GRAD_OPERANDS | SF_FFN_W2_FD))
    return SF_ERR_UNSUPPORTED;
  if ((d->flags & SF_FFN_UNFUSED_ACT) && (d->flags & SF_FFN_FUSED_ACT)) return SF_ERR_UNSUPPORTED;
  if (d->V != 64 && d->V != 128) return SF_ERR_SHAPE;
  if (d->T <= 0 || d->D <= 0 || d->F <= 0) return SF_ERR_SHAPE;
  // every product runs on 256-row CTA-pair tiles whose last pair may be half empty: multiples of 128, at least 256.
  // The gathered Venom products (M >= 16) and the operand expander keep whole 256-wide tiles.
  const int64_t q = (d->M >= 16 || (d->flags & SF_FFN_PACKED_GRAD_OPERANDS)) ? 256 : 128;
  if (d->T % q || d->D % q || d->F % q || d->T < 256 || d->D < 256 || d->F < 256 || d->T % d->V) return SF_ERR_SHAPE;
  if (d->F % (4 * d->M)) return SF_ERR_SHAPE;                            // whole metadata words
  if (d->M >= 16 && (4 * d->F / d->M) % 128) return SF_ERR_SHAPE;         // condensed reduction in whole stages
  if (d->prune_mode != 0 && d->prune_mode != 1) return SF_ERR_SHAPE;
  return SF_OK;
}

inline uint8_t* at(void* base, size_t off) { return reinterpret_cast<uint8_t*>(base) + off; }
inline const uint8_t* at(const void* base, size_t off) { return reinterpret_cast<const uint8_t*>(base) + off; }

}  // namespace

void trace_mark(cudaStream_t s) {
  if (g_trace_events && g_trace_n < g_trace_cap) cudaEventRecord(g_trace_events[g_trace_n++], s);
}

int launch_meta_reorder(const void* meta, void* meta_hw, int64_t R, int64_t K, cudaStream_t s) {
  const int64_t n = R * (K >> 4);
  if (n == 0) return SF_OK;
  meta_reorder_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>((const uint16_t*)meta, (uint8_t*)meta_hw, R, K);
  SF_LAUNCH_CHECK();
  return SF_OK;
}

int launch_pack_like(const void* dense, const void* meta, const void* colidx, void* vals, int64_t T, int64_t F,
                     int V, int Mv, cudaStream_t s) {
  const int64_t n = T * (F / Mv / 4);
  if (n == 0) return SF_OK;
  pack_like_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>((const uint16_t*)dense, (const uint16_t*)meta,
                                                               (const uint8_t*)colidx, (uint16_t*)vals, T, F, V, Mv);
  SF_LAUNCH_CHECK();
  return SF_OK;
}

}  // namespace sf

using namespace sf;

#define SF_TRY(expr)              \
  do {                            \
    int _st = (expr);             \
    if (_st != SF_OK) return _st; \
  } while (0)

extern "C" {

// ---- single products ---------------------------------------------------------------------------

int sf_gemm_workspace_size(int64_t Mr, int64_t K, size_t* bytes) {
  if (!bytes) return SF_ERR_NULL;
  if (Mr < 0 || K < 0) return SF_ERR_SHAPE;
  *bytes = kStatusBytes + up((size_t)Mr * (size_t)K / 8);
  return SF_OK;
}

int sf_gemm_dense(const void* A, int a_kmajor, const void* B, int b_kmajor, void* C, int64_t Mr, int64_t Nc,
                  int64_t K, void* workspace, void* stream) {
  if (Mr < 0 || Nc < 0 || K <= 0 || Mr % 128 || Nc % 256 || K % 64) return SF_ERR_SHAPE;
  if (Mr == 0 || Nc == 0) return SF_OK;
  if (!A || !B || !C || !workspace) return SF_ERR_NULL;
  if (!aligned16(A) || !aligned16(B) || !aligned16(C) || !aligned16(workspace)) return SF_ERR_ALIGN;
  SF_TRY(check_arch());
  return gemm_dense(A, a_kmajor != 0, B, b_kmajor != 0, Mr, Nc, K, EPI_STORE, C, Nc, nullptr, 0, nullptr, 0,
                    (int*)workspace, (cudaStream_t)stream);
}

int sf_gemm_sparse24(const void* a_vals, const void* a_meta, const void* B, void* Ct, int64_t Mr, int64_t Nc,
                     int64_t K, void* workspace, void* stream) {
  if (Mr < 0 || Nc < 0 || K <= 0 || Mr % 128 || Nc % 256 || K % 128) return SF_ERR_SHAPE;
  if (Mr == 0 || Nc == 0) return SF_OK;
  if (!a_vals || !a_meta || !B || !Ct || !workspace) return SF_ERR_NULL;
  if (!aligned16(a_vals) || !aligned16(a_meta) || !aligned16(B) || !aligned16(Ct) || !aligned16(workspace))
    return SF_ERR_ALIGN;
  SF_TRY(check_arch());
  cudaStream_t s = (cudaStream_t)stream;
  uint8_t* hw = at(workspace, kStatusBytes);
  SF_TRY(launch_meta_reorder(a_meta, hw, Mr, K, s));
  return gemm_sparse24(a_vals, hw, B, true, Mr, Nc, K, EPI_STORE_T, Ct, Mr, nullptr, 0, (int*)workspace, s);
}

int sf_gemm_sparse24_rm(const void* a_vals, const void* a_meta, const void* B, int b_kmajor, void* C, int64_t Mr,
                        int64_t Nc, int64_t K, void* workspace, void* stream) {
  if (Mr < 0 || Nc < 0 || K <= 0 || Mr % 256 || Nc % 256 || K % 128) return SF_ERR_SHAPE;
  if (Mr == 0 || Nc == 0) return SF_OK;
  if (!a_vals || !a_meta || !B || !C || !workspace) return SF_ERR_NULL;
  if (!aligned16(a_vals) || !aligned16(a_meta) || !aligned16(B) || !aligned16(C) || !aligned16(workspace))
    return SF_ERR_ALIGN;
  SF_TRY(check_arch());
  cudaStream_t s = (cudaStream_t)stream;
  uint8_t* hw = at(workspace, kStatusBytes);
  SF_TRY(launch_meta_reorder(a_meta, hw, Mr, K, s));
  return gemm_sparse24(a_vals, hw, B, b_kmajor != 0, Mr, Nc, K, EPI_STORE, C, Nc, nullptr, 0, (int*)workspace, s);
}

int sf_gemm_venom(const void* a_vals, const void* a_meta, const void* colidx, const void* Bt, void* C, int64_t T,
                  int64_t F, int64_t Nc, int V, int M, void* workspace, void* stream) {
  if (M != 4 && M != 8 && M != 16 && M != 32 && M != 64) return SF_ERR_SHAPE;
  if (T < 0 || F <= 0 || Nc < 0 || T % 128 || Nc % 256 || F % M || (4 * F / M) % 128 || (V != 64 && V != 128))
    return SF_ERR_SHAPE;
  if (T == 0 || Nc == 0) return SF_OK;
  if (!a_vals || !a_meta || !colidx || !Bt || !C || !workspace) return SF_ERR_NULL;
  if (!aligned16(a_vals) || !aligned16(a_meta) || !aligned16(colidx) || !aligned16(Bt) || !aligned16(C) ||
      !aligned16(workspace))
    return SF_ERR_ALIGN;
  SF_TRY(check_arch());
  cudaStream_t s = (cudaStream_t)stream;
  uint8_t* hw = at(workspace, kStatusBytes);
  SF_TRY(launch_meta_reorder(a_meta, hw, T, 4 * F / M, s));
  return gemm_venom(a_vals, hw, (const uint8_t*)colidx, Bt, T, F, Nc, V, M, C, Nc, (int*)workspace, s);
}

// ---- FFN step --------------------------------------------------------------------------------------

int sf_ffn_workspace_size(const sf_ffn_desc* desc, size_t* fwd_ctx_bytes, size_t* workspace_bytes) {
  if (!fwd_ctx_bytes || !workspace_bytes) return SF_ERR_NULL;
  SF_TRY(check_desc(desc));
  const SparseLayout S = sparse_layout(*desc);
  const DenseLayout Dn = dense_layout(*desc);
  *fwd_ctx_bytes = S.ctx_total > Dn.ctx_total ? S.ctx_total : Dn.ctx_total;
  *workspace_bytes = S.ws_total > Dn.ws_total ? S.ws_total : Dn.ws_total;
  return SF_OK;
}

static int check_ptrs(std::initializer_list<const void*> ps) {
  for (const void* p : ps) {
    if (!p) return SF_ERR_NULL;
    if (!aligned16(p)) return SF_ERR_ALIGN;
  }
  return SF_OK;
}

// Sizes the caller says its buffers have, against what the descriptor needs.
static int check_sizes(const sf_ffn_desc& d, bool dense, size_t fwd_ctx_bytes, size_t workspace_bytes) {
  size_t need_ctx, need_ws;
  if (dense) {
    const DenseLayout L = dense_layout(d);
    need_ctx = L.ctx_total; need_ws = L.ws_total;
  } else {
    const SparseLayout L = sparse_layout(d);
    need_ctx = L.ctx_total; need_ws = L.ws_total;
  }
  return (fwd_ctx_bytes < need_ctx || workspace_bytes < need_ws) ? SF_ERR_WORKSPACE : SF_OK;
}

int sf_sparse_ffn_fwd(const sf_ffn_desc* desc, const void* X, const void* W1, const void* W2, void* Y,
                      void* fwd_ctx, size_t fwd_ctx_bytes, void* workspace, size_t workspace_bytes, void* stream) {
  SF_TRY(check_desc(desc));
  SF_TRY(check_ptrs({X, W1, W2, Y, fwd_ctx, workspace}));
  SF_TRY(check_sizes(*desc, false, fwd_ctx_bytes, workspace_bytes));
  SF_TRY(check_arch());
  const sf_ffn_desc& d = *desc;
  const SparseLayout L = sparse_layout(d);
  cudaStream_t s = (cudaStream_t)stream;
  int* status = (int*)workspace;
  const bool save_y1 = (d.flags & SF_FFN_SAVE_Y1) != 0, w2_fd = (d.flags & SF_FFN_W2_FD) != 0;

  // Algorithm 1 line 4: W1s = sparsify24(W1) along d_model, then y1 = X W1s^T
  trace_mark(s);
  SF_TRY(launch_prune24(W1, d.F, d.D, d.D, 1, d.prune_mode, at(workspace, L.w1_vals), at(workspace, L.w1_meta),
                        at(workspace, L.w1_meta_hw), nullptr, s));
  trace_mark(s);
  if (L.fused) {
    // lines 4-6 in one kernel: the product's epilogue applies ReLU^2 and selects the V:N:M pattern on the
    // accumulator tile; y1 itself is never written (unless asked for)
    Vnm8Out out{at(fwd_ctx, L.y2_vals), at(fwd_ctx, L.relu_vals), at(fwd_ctx, L.meta), at(fwd_ctx, L.colidx),
                at(fwd_ctx, L.vals24), at(fwd_ctx, L.relu24), at(fwd_ctx, L.meta24), at(fwd_ctx, L.meta24_hw),
                save_y1 ? (void*)at(fwd_ctx, L.y1) : nullptr, L.expand ? nullptr : (void*)at(fwd_ctx, L.y2_dense)};
    SF_TRY(gemm_sparse24_vnm8(at(workspace, L.w1_vals), at(workspace, L.w1_meta_hw), X, d.F, d.T, d.D, d.V, out,
                              status, s));
    trace_mark(s);
    trace_mark(s);      // (the sparsify interval is empty on this path)
  } else {
    void* y1 = save_y1 ? (void*)at(fwd_ctx, L.y1) : (void*)at(workspace, L.ws_y1);
    SF_TRY(gemm_sparse24(at(workspace, L.w1_vals), at(workspace, L.w1_meta_hw), X, true, d.F, d.T, d.D, EPI_STORE_T,
                         y1, d.F, nullptr, 0, status, s));
    trace_mark(s);
    // lines 5-6: y2 = ReLU(y1)^2 in V:N:M form (+ what the backward pass needs)
    if (L.packed8) {
      SF_TRY(launch_vnm(y1, d.T, d.F, d.F, d.V, d.M, 1, at(fwd_ctx, L.y2_vals), at(fwd_ctx, L.meta), nullptr,
                        at(fwd_ctx, L.colidx), at(fwd_ctx, L.relu_vals),
                        L.expand ? nullptr : (void*)at(fwd_ctx, L.y2_dense), nullptr, at(fwd_ctx, L.vals24),
                        at(fwd_ctx, L.meta24), at(fwd_ctx, L.meta24_hw), at(fwd_ctx, L.relu24), s));
    } else {
      SF_TRY(launch_vnm(y1, d.T, d.F, d.F, d.V, d.M, 1, at(fwd_ctx, L.y2_vals), at(fwd_ctx, L.meta),
                        at(fwd_ctx, L.meta_hw), at(fwd_ctx, L.colidx), at(fwd_ctx, L.relu_vals),
                        at(fwd_ctx, L.y2_dense), at(fwd_ctx, L.relu_dense), nullptr, nullptr, nullptr, nullptr, s));
    }
    trace_mark(s);
  }
  // line 7: y3 = y2 W2^T with W2 dense
  hook_wait_w2(s);
  if (L.plain24) {
    // y2 as a 2:4 operand over all F columns against W2 [D, F] as it is stored (no transpose, no gather)
    trace_mark(s);
    // (W2 given as [F, D]: the same product with W2 as the MN-major operand)
    SF_TRY(gemm_sparse24(at(fwd_ctx, L.vals24), at(fwd_ctx, L.meta24_hw), W2, !w2_fd, d.T, d.D, d.F, EPI_STORE, Y, d.D,
                         nullptr, 0, status, s));
  } else {
    // condensed V:N:M operand; rows of W2^T are gathered by the kept columns (W2 given as [F, D] is that matrix)
    if (!w2_fd) SF_TRY(launch_transpose(W2, at(fwd_ctx, L.w2t), d.D, d.F, s));
    trace_mark(s);
    SF_TRY(gemm_venom(at(fwd_ctx, L.y2_vals), at(fwd_ctx, L.meta_hw), at(fwd_ctx, L.colidx),
                      w2_fd ? W2 : (const void*)at(fwd_ctx, L.w2t), d.T, d.F, d.D, d.V, d.M, Y, d.D, status, s));
  }
  trace_mark(s);
  return SF_OK;
}

int sf_sparse_ffn_bwd(const sf_ffn_desc* desc, const void* dY, const void* X, const void* W1, const void* W2,
                      const void* fwd_ctx, size_t fwd_ctx_bytes, void* dX, void* dW1, void* dW2, void* workspace,
                      size_t workspace_bytes, void* stream) {
  SF_TRY(check_desc(desc));
  SF_TRY(check_ptrs({dY, X, W1, W2, fwd_ctx, dX, dW1, dW2, workspace}));
  SF_TRY(check_sizes(*desc, false, fwd_ctx_bytes, workspace_bytes));
  SF_TRY(check_arch());
  const sf_ffn_desc& d = *desc;
  const SparseLayout L = sparse_layout(d);
  cudaStream_t s = (cudaStream_t)stream;
  int* status = (int*)workspace;
  const bool w2_fd = (d.flags & SF_FFN_W2_FD) != 0;
  // dW2 = dY^T y2 in the layout of W2: [D, F], or [F, D] = y2^T dY when W2 is stored that way
  auto grad_w2 = [&](const void* y2_dense) -> int {
    return w2_fd ? gemm_dense(y2_dense, false, dY, false, d.F, d.D, d.T, EPI_STORE, dW2, d.D, nullptr, 0, nullptr, 0, status, s)
                 : gemm_dense(dY, false, y2_dense, false, d.D, d.F, d.T, EPI_STORE, dW2, d.F, nullptr, 0, nullptr, 0, status, s);
  };

  // Algorithm 2 line 2: W2s = sparsify24(W2^T) along d_model (contiguous in the saved W2^T copy),
  // dy2 = dY W2s;  line 4: dy1 = 2 dy2 ReLU(y1) on y2's mask (fused into the product's epilogue)
  trace_mark(s);
  if (w2_fd) {
    // W2 stored as [F, D]: the groups along d_model are contiguous
    SF_TRY(launch_prune24(W2, d.F, d.D, d.D, 1, d.prune_mode, at(workspace, L.w2_vals), at(workspace, L.w2_meta),
                          at(workspace, L.w2_meta_hw), nullptr, s));
  } else if (L.plain24) {
    // no W2^T copy exists on this path: prune the strided groups of W2 [D, F] directly
    SF_TRY(launch_prune24(W2, d.D, d.F, d.F, 0, d.prune_mode, at(workspace, L.w2_vals), at(workspace, L.w2_meta),
                          at(workspace, L.w2_meta_hw), nullptr, s));
  } else {
    SF_TRY(launch_prune24(at(fwd_ctx, L.w2t), d.F, d.D, d.D, 1, d.prune_mode, at(workspace, L.w2_vals),
                          at(workspace, L.w2_meta), at(workspace, L.w2_meta_hw), nullptr, s));
  }
  trace_mark(s);
  if (L.packed8) {
    // M = 8: ReLU(y1) comes in the 2:4 layout of y2's mask and dy1 leaves in the same layout (plus, unless
    // the weight-gradient products expand their operands themselves, as a masked [T, F] matrix)
    SF_TRY(gemm_sparse24(at(workspace, L.w2_vals), at(workspace, L.w2_meta_hw), dY, true, d.F, d.T, d.D,
                         EPI_DRELU24_T, L.expand ? nullptr : (void*)at(workspace, L.dy1_dense), d.F,
                         at(fwd_ctx, L.relu24), 0, status, s, at(fwd_ctx, L.meta24), at(workspace, L.dy1_vals24)));
    trace_mark(s);
    trace_mark(s);
    // line 5: dX = dy1 W1 with W1 dense; W1 [F, D] is the MN-major operand
    SF_TRY(gemm_sparse24(at(workspace, L.dy1_vals24), at(fwd_ctx, L.meta24_hw), W1, false, d.T, d.D, d.F, EPI_STORE,
                         dX, d.D, nullptr, 0, status, s));
    trace_mark(s);
    hook_dx_done(s);
    // line 3: dW2 = dY^T y2 [D, F];  line 6: dW1 = dy1^T X [F, D]: dense tensor-core products (the reduction
    // runs over tokens); their masked operand is a stored [T, F] matrix or is expanded from its packed form
    // inside the kernel
    if (L.expand) {
      if (w2_fd) SF_TRY(gemm_dense_expand(dY, 1, at(fwd_ctx, L.vals24), at(fwd_ctx, L.meta24), d.F, d.D, d.T, dW2, d.D, status, s));
      else       SF_TRY(gemm_dense_expand(dY, 2, at(fwd_ctx, L.vals24), at(fwd_ctx, L.meta24), d.D, d.F, d.T, dW2, d.F, status, s));
    } else {
      SF_TRY(grad_w2(at(fwd_ctx, L.y2_dense)));
    }
    trace_mark(s);
    hook_dw2_done(s);
    if (L.expand) {
      SF_TRY(gemm_dense_expand(X, 1, at(workspace, L.dy1_vals24), at(fwd_ctx, L.meta24), d.F, d.D, d.T, dW1, d.D,
                               status, s));
    } else {
      SF_TRY(gemm_dense(at(workspace, L.dy1_dense), false, X, false, d.F, d.D, d.T, EPI_STORE, dW1, d.D, nullptr, 0,
                        nullptr, 0, status, s));
    }
    trace_mark(s);
    return SF_OK;
  }
  // (M = 4: the same epilogue also packs dy1 with y2's 2:4 metadata, the operand of the dX product)
  SF_TRY(gemm_sparse24(at(workspace, L.w2_vals), at(workspace, L.w2_meta_hw), dY, true, d.F, d.T, d.D, EPI_DRELU_T,
                       at(workspace, L.dy1_dense), d.F, at(fwd_ctx, L.relu_dense), d.F, status, s,
                       L.plain24 ? at(fwd_ctx, L.meta24) : nullptr, L.plain24 ? at(workspace, L.dy1_vals24) : nullptr));
  trace_mark(s);
  // line 5: dX = dy1 W1 with W1 dense
  if (L.plain24) {
    trace_mark(s);
    SF_TRY(gemm_sparse24(at(workspace, L.dy1_vals24), at(fwd_ctx, L.meta24_hw), W1, false, d.T, d.D, d.F, EPI_STORE,
                         dX, d.D, nullptr, 0, status, s));
  } else {
    SF_TRY(launch_pack_like(at(workspace, L.dy1_dense), at(fwd_ctx, L.meta), at(fwd_ctx, L.colidx),
                            at(workspace, L.dy1_vals), d.T, d.F, d.V, d.M, s));
    trace_mark(s);
    // rows of W1 gathered by the kept columns
    SF_TRY(gemm_venom(at(workspace, L.dy1_vals), at(fwd_ctx, L.meta_hw), at(fwd_ctx, L.colidx), W1, d.T, d.F, d.D,
                      d.V, d.M, dX, d.D, status, s));
  }
  trace_mark(s);
  hook_dx_done(s);
  // line 3: dW2 = dY^T y2 [D, F];  line 6: dW1 = dy1^T X [F, D]  (reduction over tokens)
  SF_TRY(grad_w2(at(fwd_ctx, L.y2_dense)));
  trace_mark(s);
  hook_dw2_done(s);
  SF_TRY(gemm_dense(at(workspace, L.dy1_dense), false, X, false, d.F, d.D, d.T, EPI_STORE, dW1, d.D, nullptr, 0,
                    nullptr, 0, status, s));
  trace_mark(s);
  return SF_OK;
}

int sf_dense_ffn_fwd(const sf_ffn_desc* desc, const void* X, const void* W1, const void* W2, void* Y, void* fwd_ctx,
                     size_t fwd_ctx_bytes, void* workspace, size_t workspace_bytes, void* stream) {
  SF_TRY(check_desc(desc));
  SF_TRY(check_ptrs({X, W1, W2, Y, fwd_ctx, workspace}));
  SF_TRY(check_sizes(*desc, true, fwd_ctx_bytes, workspace_bytes));
  SF_TRY(check_arch());
  const sf_ffn_desc& d = *desc;
  const DenseLayout L = dense_layout(d);
  cudaStream_t s = (cudaStream_t)stream;
  int* status = (int*)workspace;
  // Eq. 1-2: y1 = X W1^T, h = ReLU(y1)^2 (fused);  Eq. 3: Y = h W2^T
  trace_mark(s);
  SF_TRY(gemm_dense(X, true, W1, true, d.T, d.F, d.D, EPI_SQRELU, at(fwd_ctx, L.y1), d.F, at(fwd_ctx, L.h), d.F,
                    nullptr, 0, status, s));
  trace_mark(s);
  hook_wait_w2(s);
  SF_TRY(gemm_dense(at(fwd_ctx, L.h), true, W2, !(d.flags & SF_FFN_W2_FD), d.T, d.D, d.F, EPI_STORE, Y, d.D, nullptr, 0,
                    nullptr, 0, status, s));
  trace_mark(s);
  return SF_OK;
}

int sf_dense_ffn_bwd(const sf_ffn_desc* desc, const void* dY, const void* X, const void* W1, const void* W2,
                     const void* fwd_ctx, size_t fwd_ctx_bytes, void* dX, void* dW1, void* dW2, void* workspace,
                     size_t workspace_bytes, void* stream) {
  SF_TRY(check_desc(desc));
  SF_TRY(check_ptrs({dY, X, W1, W2, fwd_ctx, dX, dW1, dW2, workspace}));
  SF_TRY(check_sizes(*desc, true, fwd_ctx_bytes, workspace_bytes));
  SF_TRY(check_arch());
  const sf_ffn_desc& d = *desc;
  const DenseLayout L = dense_layout(d);
  cudaStream_t s = (cudaStream_t)stream;
  int* status = (int*)workspace;
  void* dy1 = at(workspace, L.dy1);
  // Eq. 4 + 6: dy1 = 2 (dY W2) ReLU(y1)
  trace_mark(s);
  const bool w2_fd = (d.flags & SF_FFN_W2_FD) != 0;                 // W2 [F, D] is the K-major operand of this product
  SF_TRY(gemm_dense(dY, true, W2, w2_fd, d.T, d.F, d.D, EPI_DRELU, dy1, d.F, nullptr, 0, at(fwd_ctx, L.y1), d.F,
                    status, s));
  trace_mark(s);
  // Eq. 7: dX = dy1 W1
  SF_TRY(gemm_dense(dy1, true, W1, false, d.T, d.D, d.F, EPI_STORE, dX, d.D, nullptr, 0, nullptr, 0, status, s));
  trace_mark(s);
  hook_dx_done(s);
  // Eq. 5: dW2 = dY^T h [D, F];  Eq. 8: dW1 = dy1^T X [F, D]
  if (w2_fd)
    SF_TRY(gemm_dense(at(fwd_ctx, L.h), false, dY, false, d.F, d.D, d.T, EPI_STORE, dW2, d.D, nullptr, 0, nullptr, 0,
                      status, s));
  else
    SF_TRY(gemm_dense(dY, false, at(fwd_ctx, L.h), false, d.D, d.F, d.T, EPI_STORE, dW2, d.F, nullptr, 0, nullptr, 0,
                      status, s));
  trace_mark(s);
  hook_dw2_done(s);
  SF_TRY(gemm_dense(dy1, false, X, false, d.F, d.D, d.T, EPI_STORE, dW1, d.D, nullptr, 0, nullptr, 0, status, s));
  trace_mark(s);
  return SF_OK;
}

int sf_ctx_view(const sf_ffn_desc* desc, const void* buf, int field, const void** ptr, size_t* bytes) {
  if (!ptr || !bytes || !buf) return SF_ERR_NULL;
  SF_TRY(check_desc(desc));
  const sf_ffn_desc& d = *desc;
  const SparseLayout L = sparse_layout(d);
  const size_t T = d.T, F = d.F, G = F / d.M;
  size_t off, n;
  switch (field) {
    case SF_CTX_Y2_VALS: off = L.y2_vals; n = T * 2 * G * 2; break;
    case SF_CTX_RELU_VALS: off = L.relu_vals; n = T * 2 * G * 2; break;
    case SF_CTX_META: off = L.meta; n = T * G / 2; break;
    case SF_CTX_COLIDX: off = L.colidx; n = (T / d.V) * G * 4; break;
    case SF_CTX_Y1:
      if (!(d.flags & SF_FFN_SAVE_Y1)) return SF_ERR_UNSUPPORTED;
      off = L.y1; n = T * F * 2; break;
    case SF_CTX_DY1_VALS:
      if (L.packed8) return SF_ERR_UNSUPPORTED;
      off = L.dy1_vals; n = T * 2 * G * 2; break;
    case SF_CTX_Y2_VALS24:
      if (!L.plain24) return SF_ERR_UNSUPPORTED;
      off = L.vals24; n = T * F; break;
    case SF_CTX_Y2_META24:
      if (!L.plain24) return SF_ERR_UNSUPPORTED;
      off = L.meta24; n = T * F / 8; break;
    case SF_CTX_DY1_VALS24:
      if (!L.plain24) return SF_ERR_UNSUPPORTED;
      off = L.dy1_vals24; n = T * F; break;
    case SF_CTX_RELU_VALS24:
      if (!L.packed8) return SF_ERR_UNSUPPORTED;
      off = L.relu24; n = T * F; break;
    default: return SF_ERR_SHAPE;
  }
  *ptr = at(buf, off);
  *bytes = n;
  return SF_OK;
}

// ---- host-buffer step -------------------------------------------------------------------------------

int sf_ffn_host_staging_size(const sf_ffn_desc* desc, size_t* bytes) {
  if (!bytes) return SF_ERR_NULL;
  SF_TRY(check_desc(desc));
  const size_t T = desc->T, D = desc->D, F = desc->F;
  *bytes = 4 * up(T * D * 2) + 4 * up(F * D * 2);   // X, dY, Y, dX + W1, W2, dW1, dW2
  return SF_OK;
}

int sf_ffn_step_host(const sf_ffn_desc* desc, int dense, const void* host_X, const void* host_W1,
                     const void* host_W2, const void* host_dY, void* host_Y, void* host_dX, void* host_dW1,
                     void* host_dW2, void* device_staging, void* fwd_ctx, size_t fwd_ctx_bytes, void* workspace,
                     size_t workspace_bytes, void* stream) {
  SF_TRY(check_desc(desc));
  SF_TRY(check_sizes(*desc, dense != 0, fwd_ctx_bytes, workspace_bytes));
  if (!host_X || !host_W1 || !host_W2 || !host_dY || !host_Y || !host_dX || !host_dW1 || !host_dW2 ||
      !device_staging || !fwd_ctx || !workspace)
    return SF_ERR_NULL;
  const size_t T = desc->T, D = desc->D, F = desc->F;
  const size_t act = up(T * D * 2), wgt = up(F * D * 2);
  uint8_t* base = (uint8_t*)device_staging;
  void *dXin = base, *ddY = base + act, *dYout = base + 2 * act, *ddX = base + 3 * act;
  void *dW1in = base + 4 * act, *dW2in = base + 4 * act + wgt, *ddW1 = base + 4 * act + 2 * wgt,
       *ddW2 = base + 4 * act + 3 * wgt;
  cudaStream_t s = (cudaStream_t)stream;
  HostStepResources* r = nullptr;
  SF_TRY(host_step_resources(&r));
  // uploads, in the order the step first needs them, on their own stream behind everything already on `stream`
  SF_CUDA_TRY(cudaEventRecord(r->begin, s));
  SF_CUDA_TRY(cudaStreamWaitEvent(r->up, r->begin, 0));
  SF_CUDA_TRY(cudaMemcpyAsync(dXin, host_X, T * D * 2, cudaMemcpyHostToDevice, r->up));
  SF_CUDA_TRY(cudaMemcpyAsync(dW1in, host_W1, F * D * 2, cudaMemcpyHostToDevice, r->up));
  SF_CUDA_TRY(cudaEventRecord(r->xw1, r->up));
  SF_CUDA_TRY(cudaMemcpyAsync(dW2in, host_W2, F * D * 2, cudaMemcpyHostToDevice, r->up));
  SF_CUDA_TRY(cudaEventRecord(r->w2, r->up));
  SF_CUDA_TRY(cudaMemcpyAsync(ddY, host_dY, T * D * 2, cudaMemcpyHostToDevice, r->up));
  SF_CUDA_TRY(cudaEventRecord(r->dy, r->up));

  const StepHooks hooks{r->w2, r->dx, r->dw2};
  g_hooks = &hooks;
  int rc = SF_OK;
  do {
    if (cudaStreamWaitEvent(s, r->xw1, 0) != cudaSuccess) { rc = SF_ERR_CUDA; break; }
    rc = dense ? sf_dense_ffn_fwd(desc, dXin, dW1in, dW2in, dYout, fwd_ctx, fwd_ctx_bytes, workspace, workspace_bytes,
                                  stream)
               : sf_sparse_ffn_fwd(desc, dXin, dW1in, dW2in, dYout, fwd_ctx, fwd_ctx_bytes, workspace,
                                   workspace_bytes, stream);
    if (rc != SF_OK) break;
    if (cudaEventRecord(r->y, s) != cudaSuccess || cudaStreamWaitEvent(s, r->dy, 0) != cudaSuccess) {
      rc = SF_ERR_CUDA;
      break;
    }
    rc = dense ? sf_dense_ffn_bwd(desc, ddY, dXin, dW1in, dW2in, fwd_ctx, fwd_ctx_bytes, ddX, ddW1, ddW2, workspace,
                                  workspace_bytes, stream)
               : sf_sparse_ffn_bwd(desc, ddY, dXin, dW1in, dW2in, fwd_ctx, fwd_ctx_bytes, ddX, ddW1, ddW2, workspace,
                                   workspace_bytes, stream);
  } while (false);
  g_hooks = nullptr;
  // a failure past this point still has to rejoin the upload stream, or a capture of `stream` would dangle
  if (rc != SF_OK) {
    cudaStreamWaitEvent(s, r->dy, 0);
    return rc;
  }
  SF_CUDA_TRY(cudaEventRecord(r->dw1, s));
  // downloads, each as soon as its product has finished, on a second stream
  SF_CUDA_TRY(cudaStreamWaitEvent(r->down, r->y, 0));
  SF_CUDA_TRY(cudaMemcpyAsync(host_Y, dYout, T * D * 2, cudaMemcpyDeviceToHost, r->down));
  SF_CUDA_TRY(cudaStreamWaitEvent(r->down, r->dx, 0));
  SF_CUDA_TRY(cudaMemcpyAsync(host_dX, ddX, T * D * 2, cudaMemcpyDeviceToHost, r->down));
  SF_CUDA_TRY(cudaStreamWaitEvent(r->down, r->dw2, 0));
  SF_CUDA_TRY(cudaMemcpyAsync(host_dW2, ddW2, F * D * 2, cudaMemcpyDeviceToHost, r->down));
  SF_CUDA_TRY(cudaStreamWaitEvent(r->down, r->dw1, 0));
  SF_CUDA_TRY(cudaMemcpyAsync(host_dW1, ddW1, F * D * 2, cudaMemcpyDeviceToHost, r->down));
  SF_CUDA_TRY(cudaEventRecord(r->done, r->down));
  // `stream` is complete only when the last download is
  SF_CUDA_TRY(cudaStreamWaitEvent(s, r->done, 0));
  return SF_OK;
}

int sf_trace_set(void** events, int capacity) {
  if (capacity < 0 || (capacity > 0 && !events)) return SF_ERR_NULL;
  g_trace_events = capacity > 0 ? reinterpret_cast<cudaEvent_t*>(events) : nullptr;
  g_trace_cap = capacity;
  g_trace_n = 0;
  return SF_OK;
}

int sf_trace_count(void) { return g_trace_n; }

int sf_check_status(void* workspace, void* stream) {
  if (!workspace) {
    // the status word of sf_gemm_sparse24_noalloc's built-in scratch array (no allocation here either)
    SF_TRY(check_arch());
    SF_TRY(noalloc_status_word(&workspace));
  }
  cudaStream_t s = (cudaStream_t)stream;
  SF_CUDA_TRY(cudaStreamSynchronize(s));
  int host = 0;
  SF_CUDA_TRY(cudaMemcpy(&host, workspace, sizeof(int), cudaMemcpyDeviceToHost));
  if (host != 0) {
    SF_CUDA_TRY(cudaMemset(workspace, 0, sizeof(int)));
    return SF_ERR_TIMEOUT;
  }
  return SF_OK;
}

}  // extern "C"
