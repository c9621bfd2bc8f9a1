// Neuron-level experts that produce the V:N:M pattern (Section 3.1, Algorithm 3, Section 3.2.2 steps 1-3):
// the routed FFN step.
//
// The hidden features are stored expert-major: expert e owns features [e Fe, (e + 1) Fe), Fe = F / E (a
// renumbering of the FFN's hidden units, done once offline together with the clustering). Per step:
//   step 1  route_kernel        logits = x . ExpertMeans, top-1 expert per token (ties to the lower expert)
//   step 2  group_kernel        tokens grouped by expert, stable, every segment padded to 256 rows of zeros;
//           tile_tables_kernel  one table entry per output tile of each grouped product (no host round trip)
//           gather_rows_kernel  gathers X (and dY) into that order (Y and dX go back to token order through
//                               the row map of the product's own epilogue)
//   step 3  grouped tensor-core products over the tables: every product touches only the expert's Fe features
//           of a token, so each costs 1 / E of its dense counterpart (and the 2:4 ones half of that again).
// Interleaving the expert blocks four features at a time turns a segment into V:N:M blocks with M = 4 E whose
// kept columns are the expert's four in every group; inside them the 2:4 pattern is chosen by magnitude.
#include "sf_common.cuh"
#include "gemm_tc.cuh"

#include <initializer_list>

namespace sf {
namespace {

constexpr int kMaxExperts = 16;
constexpr int kSegPad = 256;            // rows per CTA-pair tile: a segment never shares a tile with another expert
constexpr int kActTileN = 224;          // token tile of the products whose accumulator rows are features
constexpr size_t kAlign = 256;
constexpr size_t kStatusBytes = 256;

inline size_t up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

// ---- step 1: routing ----------------------------------------------------------------------------------
// One warp per two tokens (the expert means, small enough for the L1, are read once per pair). A lane owns eight consecutive
// elements of every 256-element chunk and keeps one float32 partial sum per (token, expert); the partial
// sums are combined by a fixed xor-shuffle tree, so the result does not depend on the launch.
constexpr int kRouteTokens = 2;

__global__ void __launch_bounds__(256, 2)
route_kernel(const uint16_t* __restrict__ X, const uint16_t* __restrict__ means, int T, int D, int E,
             int* __restrict__ expert, float* __restrict__ logits) {
  const int lane = threadIdx.x & 31;
  const int t0 = ((int)blockIdx.x * 8 + (threadIdx.x >> 5)) * kRouteTokens;
  if (t0 >= T) return;
  float acc[kRouteTokens][kMaxExperts];
#pragma unroll
  for (int i = 0; i < kRouteTokens; ++i)
#pragma unroll
    for (int e = 0; e < kMaxExperts; ++e) acc[i][e] = 0.f;
  // The kernel waits on memory, not arithmetic. The tokens stream past the L1 (no allocation there), so the
  // expert means stay in it; the next chunk of the tokens is requested before this one is multiplied, and
  // the means of eight experts are requested together before any of them is used.
  auto load_stream = [](const uint16_t* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
  };
  uint4 nxt[kRouteTokens];
  auto fetch = [&](int c) {
#pragma unroll
    for (int i = 0; i < kRouteTokens; ++i) {
      const int t = min(t0 + i, T - 1);                                     // a ragged last group re-reads the last token
      nxt[i] = load_stream(X + (int64_t)t * D + c);
    }
  };
  fetch(lane * 8);
  for (int c = lane * 8; c < D; c += 256) {
    // widen the chunk once (eight values per token), then one multiply-add per (token, expert, element) in
    // element order
    float xf[kRouteTokens][8];
#pragma unroll
    for (int i = 0; i < kRouteTokens; ++i) {
      const uint32_t xw[4] = {nxt[i].x, nxt[i].y, nxt[i].z, nxt[i].w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        xf[i][2 * j] = bf16_bits_to_float(xw[j] & 0xFFFFu);
        xf[i][2 * j + 1] = bf16_bits_to_float(xw[j] >> 16);
      }
    }
    if (c + 256 < D) fetch(c + 256);
#pragma unroll
    for (int e0 = 0; e0 < kMaxExperts; e0 += 8) {
      if (e0 < E) {
        uint4 mv[8];
#pragma unroll
        for (int k = 0; k < 8; ++k)
          mv[k] = __ldg(reinterpret_cast<const uint4*>(means + (int64_t)min(e0 + k, E - 1) * D + c));
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          if (e0 + k < E) {
            const uint32_t mw[4] = {mv[k].x, mv[k].y, mv[k].z, mv[k].w};
            float mf[8];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              mf[2 * j] = bf16_bits_to_float(mw[j] & 0xFFFFu);
              mf[2 * j + 1] = bf16_bits_to_float(mw[j] >> 16);
            }
#pragma unroll
            for (int i = 0; i < kRouteTokens; ++i)
#pragma unroll
              for (int j = 0; j < 8; ++j) acc[i][e0 + k] = __fmaf_rn(xf[i][j], mf[j], acc[i][e0 + k]);
          }
        }
      }
    }
  }
#pragma unroll
  for (int i = 0; i < kRouteTokens; ++i) {
    const int t = t0 + i;
    int best = 0;
    float bestv = 0.f;
#pragma unroll
    for (int e = 0; e < kMaxExperts; ++e) {
      if (e < E) {
        float v = acc[i][e];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
        if (lane == 0 && logits && t < T) logits[(int64_t)t * E + e] = v;
        if (e == 0 || v > bestv) { bestv = v; best = e; }        // strict: ties stay with the lower expert
      }
    }
    if (lane == 0 && t < T) expert[t] = best;
  }
}

// ---- step 2: grouping ---------------------------------------------------------------------------------------
// One CTA. Thread i owns a contiguous run of tokens; per-expert counts are scanned over the threads, segments
// are padded to kSegPad rows (an expert without tokens still gets one all-zero tile, so that the
// weight-gradient blocks of that expert are written), and every token gets its row.
//   seg[0 .. E]      first row of each segment, seg[E] = number of rows in use
//   seg[E+1 .. 2E]   tokens per expert
__global__ void __launch_bounds__(1024)
group_kernel(const int* __restrict__ expert, int T, int E, int rows_max, int* __restrict__ row_of_token,
             int* __restrict__ src_of_row, int* __restrict__ seg) {
  extern __shared__ int gsm[];
  int* cnt = gsm;                          // [E][1024]
  int* sseg = gsm + E * 1024;              // [E + 1]
  const int tid = threadIdx.x;
  const int per = (T + 1023) / 1024;
  const int t0 = tid * per, t1 = min(t0 + per, T);
  int local[kMaxExperts];
#pragma unroll
  for (int e = 0; e < kMaxExperts; ++e) local[e] = 0;
  for (int t = t0; t < t1; ++t) {
    const int ex = expert[t];
#pragma unroll
    for (int e = 0; e < kMaxExperts; ++e) local[e] += (ex == e);
  }
#pragma unroll
  for (int e = 0; e < kMaxExperts; ++e)
    if (e < E) cnt[e * 1024 + tid] = local[e];
  for (int r = tid; r < rows_max; r += 1024) src_of_row[r] = -1;
  __syncthreads();
  if (tid < E) {                           // exclusive scan of this expert's counts over the threads
    int run = 0;
    for (int i = 0; i < 1024; ++i) {
      const int c = cnt[tid * 1024 + i];
      cnt[tid * 1024 + i] = run;
      run += c;
    }
    seg[E + 1 + tid] = run;
    sseg[tid + 1] = run;                   // totals, turned into boundaries below
  }
  __syncthreads();
  if (tid == 0) {
    int at = 0;
    sseg[0] = 0;
    for (int e = 0; e < E; ++e) {
      const int n = sseg[e + 1];
      const int padded = n == 0 ? kSegPad : (n + kSegPad - 1) / kSegPad * kSegPad;
      at += padded;
      sseg[e + 1] = at;
    }
    for (int e = 0; e <= E; ++e) seg[e] = sseg[e];
  }
  __syncthreads();
  int pos[kMaxExperts];
#pragma unroll
  for (int e = 0; e < kMaxExperts; ++e) pos[e] = e < E ? sseg[e] + cnt[e * 1024 + tid] : 0;
  for (int t = t0; t < t1; ++t) {
    const int ex = expert[t];
    int r = 0;
#pragma unroll
    for (int e = 0; e < kMaxExperts; ++e)
      if (ex == e) r = pos[e]++;
    row_of_token[t] = r;
    src_of_row[r] = t;
  }
}

// Tile tables of the grouped products (one CTA; entries are written by a thread-strided loop per table).
//   tabA  features-on-rows products (y1, dy1): A rows = the expert's feature tile, B rows = a token tile
//   tabB  tokens-on-rows products (y3, dX): A rows = a token tile, reduction over the expert's features
//   tabC  dW2 [D, F]: rows = d_model tile, columns = the expert's feature tile, reduction over its tokens
//   tabD  dW1 [F, D]: rows = the expert's feature tile, columns = d_model tile, reduction over its tokens
// counts[0..3] receive the table lengths.
__global__ void __launch_bounds__(256)
tile_tables_kernel(const int* __restrict__ seg, int E, int D, int F, GemmTile* __restrict__ tabA,
                   GemmTile* __restrict__ tabB, GemmTile* __restrict__ tabC, GemmTile* __restrict__ tabD,
                   int* __restrict__ counts) {
  __shared__ int baseA[kMaxExperts + 1], baseB[kMaxExperts + 1], baseC[kMaxExperts + 1];
  const int Fe = F / E, fm = Fe / 256, dm = D / 256;
  if (threadIdx.x == 0) {
    baseA[0] = baseB[0] = baseC[0] = 0;
    for (int e = 0; e < E; ++e) {
      const int rows = seg[e + 1] - seg[e];
      baseA[e + 1] = baseA[e] + fm * ((rows + kActTileN - 1) / kActTileN);
      baseB[e + 1] = baseB[e] + (rows / 256) * dm;
      baseC[e + 1] = baseC[e] + fm * dm;
    }
    counts[0] = baseA[E]; counts[1] = baseB[E]; counts[2] = baseC[E]; counts[3] = baseC[E];
  }
  __syncthreads();
  for (int e = 0; e < E; ++e) {
    const int s0 = seg[e], rows = seg[e + 1] - seg[e];
    const int nA = baseA[e + 1] - baseA[e];
    for (int i = threadIdx.x; i < nA; i += blockDim.x) {
      const int nt = i / fm, mt = i - nt * fm;                       // feature tiles fastest: they share the token tile
      tabA[baseA[e] + i] = GemmTile{e * Fe + mt * 256, 0, s0 + nt * kActTileN, 0, D / 128, mt * 256, s0 + nt * kActTileN,
                                    s0 + rows};
    }
    const int nB = baseB[e + 1] - baseB[e];
    for (int i = threadIdx.x; i < nB; i += blockDim.x) {
      const int nt = i / (rows / 256), rt = i - nt * (rows / 256);   // token tiles fastest: they share the weight tile
      tabB[baseB[e] + i] = GemmTile{s0 + rt * 256, 0, nt * 256, e * Fe, Fe / 128, s0 + rt * 256, nt * 256, D};
    }
    const int nC = fm * dm;
    for (int i = threadIdx.x; i < nC; i += blockDim.x) {
      const int nt = i / dm, mt = i - nt * dm;
      tabC[baseC[e] + i] = GemmTile{mt * 256, s0, nt * 256, s0, rows / 64, mt * 256, e * Fe + nt * 256, F};
      const int nt2 = i / fm, mt2 = i - nt2 * fm;
      tabD[baseC[e] + i] = GemmTile{mt2 * 256, s0, nt2 * 256, s0, rows / 64, e * Fe + mt2 * 256, nt2 * 256, D};
    }
  }
}

// out[r, :] = src[r] >= 0 ? in[src[r], :] : 0. One warp per output row; a lane keeps four 16-byte loads in
// flight, every instruction of the warp covers 512 contiguous bytes.
__global__ void __launch_bounds__(256)
gather_rows_kernel(const uint4* __restrict__ in, const int* __restrict__ src, uint4* __restrict__ out, int rows,
                   int row_u4) {
  const int r = (int)blockIdx.x * 8 + (int)(threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (r >= rows) return;
  const int s = __ldg(src + r);
  const uint4* ip = in + (int64_t)(s >= 0 ? s : 0) * row_u4;
  uint4* op = out + (int64_t)r * row_u4;
  const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
  int c = lane;
  for (; c + 96 < row_u4; c += 128) {
    uint4 v[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) v[j] = s >= 0 ? __ldg(ip + c + 32 * j) : zero;
#pragma unroll
    for (int j = 0; j < 4; ++j) op[c + 32 * j] = v[j];
  }
  for (; c < row_u4; c += 32) op[c] = s >= 0 ? __ldg(ip + c) : zero;
}

// ---- buffers ---------------------------------------------------------------------------------------------------
struct RoutedLayout {
  int64_t rows_max, Fe;
  int max_tiles[4];
  // context
  size_t expert, row_of_token, src_of_row, seg, counts, tabA, tabB, tabC, tabD, logits, xp, y2_vals, relu_vals, meta,
      meta_hw, y2_dense, y1, ctx_total;
  // workspace
  size_t w1_vals, w1_meta, w1_meta_hw, w2_vals, w2_meta, w2_meta_hw, dyp, dy1_vals, dy1_dense, ws_total;
};

RoutedLayout routed_layout(const sf_router_desc& d) {
  RoutedLayout L{};
  const size_t T = d.T, D = d.D, F = d.F, E = d.E;
  L.Fe = F / E;
  L.rows_max = (int64_t)((T + kSegPad * E + kSegPad - 1) / kSegPad * kSegPad);
  const size_t R = L.rows_max, Fe = L.Fe;
  L.max_tiles[0] = (int)((Fe / 256) * (R / kActTileN + E + 1));
  L.max_tiles[1] = (int)((R / 256) * (D / 256));
  L.max_tiles[2] = L.max_tiles[3] = (int)((F / 256) * (D / 256));
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t r = o; o += up(bytes); return r; };
  L.expert = take(T * 4);
  L.row_of_token = take(T * 4);
  L.src_of_row = take(R * 4);
  L.seg = take((2 * E + 1) * 4);
  L.counts = take(4 * 4);
  L.tabA = take((size_t)L.max_tiles[0] * sizeof(GemmTile));
  L.tabB = take((size_t)L.max_tiles[1] * sizeof(GemmTile));
  L.tabC = take((size_t)L.max_tiles[2] * sizeof(GemmTile));
  L.tabD = take((size_t)L.max_tiles[3] * sizeof(GemmTile));
  L.logits = take(T * E * 4);
  L.xp = take(R * D * 2);
  L.y2_vals = take(R * Fe);
  L.relu_vals = take(R * Fe);
  L.meta = take(R * Fe / 8);
  L.meta_hw = take(R * Fe / 8);
  L.y2_dense = take(R * Fe * 2);
  L.y1 = (d.flags & SF_FFN_SAVE_Y1) ? take(R * Fe * 2) : (size_t)-1;
  L.ctx_total = o;
  o = kStatusBytes;
  L.w1_vals = take(F * D);
  L.w1_meta = take(F * D / 8);
  L.w1_meta_hw = take(F * D / 8);
  L.w2_vals = take(F * D);
  L.w2_meta = take(F * D / 8);
  L.w2_meta_hw = take(F * D / 8);
  L.dyp = take(R * D * 2);
  L.dy1_vals = take(R * Fe);
  L.dy1_dense = take(R * Fe * 2);
  L.ws_total = o;
  return L;
}

int check_router_desc(const sf_router_desc* d) {
  if (!d) return SF_ERR_NULL;
  if (d->T <= 0 || d->D <= 0 || d->F <= 0 || d->E < 1 || d->E > kMaxExperts) return SF_ERR_SHAPE;
  if (d->T % 256 || d->D % 256 || d->F % d->E || (d->F / d->E) % 256) return SF_ERR_SHAPE;
  if (d->T > (int64_t(1) << 20)) return SF_ERR_SHAPE;            // one CTA groups the tokens
  if (d->prune_mode != 0 && d->prune_mode != 1) return SF_ERR_SHAPE;
  if (d->flags & ~SF_FFN_SAVE_Y1) return SF_ERR_UNSUPPORTED;
  return SF_OK;
}

inline uint8_t* at(void* base, size_t off) { return reinterpret_cast<uint8_t*>(base) + off; }
inline const uint8_t* at(const void* base, size_t off) { return reinterpret_cast<const uint8_t*>(base) + off; }

int check_ptrs(std::initializer_list<const void*> ps) {
  for (const void* p : ps) {
    if (!p) return SF_ERR_NULL;
    if (!aligned16(p)) return SF_ERR_ALIGN;
  }
  return SF_OK;
}

int launch_route(const void* X, const void* means, int64_t T, int64_t D, int E, void* expert, void* logits,
                 cudaStream_t s) {
  route_kernel<<<(unsigned)((T + 8 * kRouteTokens - 1) / (8 * kRouteTokens)), 256, 0, s>>>((const uint16_t*)X, (const uint16_t*)means, (int)T, (int)D, E,
                                                       (int*)expert, (float*)logits);
  SF_LAUNCH_CHECK();
  return SF_OK;
}

int launch_gather_rows(const void* in, const int* src, void* out, int64_t rows, int64_t cols, cudaStream_t s) {
  if (rows == 0 || cols == 0) return SF_OK;
  gather_rows_kernel<<<(unsigned)((rows + 7) / 8), 256, 0, s>>>((const uint4*)in, src, (uint4*)out, (int)rows,
                                                               (int)(cols / 8));
  SF_LAUNCH_CHECK();
  return SF_OK;
}

}  // namespace
}  // namespace sf

using namespace sf;

#define SF_TRY(expr)              \
  do {                            \
    int _st = (expr);             \
    if (_st != SF_OK) return _st; \
  } while (0)

extern "C" {

int sf_router_route(const void* X, const void* means, int64_t T, int64_t D, int E, void* expert, void* logits,
                    void* stream) {
  if (T < 0 || D <= 0 || D % 256 || E < 1 || E > kMaxExperts) return SF_ERR_SHAPE;
  if (T == 0) return SF_OK;
  if (!X || !means || !expert) return SF_ERR_NULL;
  if (!aligned16(X) || !aligned16(means) || !aligned16(expert) || (logits && !aligned16(logits))) return SF_ERR_ALIGN;
  SF_TRY(check_arch());
  return launch_route(X, means, T, D, E, expert, logits, (cudaStream_t)stream);
}

int sf_routed_ffn_workspace_size(const sf_router_desc* desc, size_t* fwd_ctx_bytes, size_t* workspace_bytes) {
  if (!fwd_ctx_bytes || !workspace_bytes) return SF_ERR_NULL;
  SF_TRY(check_router_desc(desc));
  const RoutedLayout L = routed_layout(*desc);
  *fwd_ctx_bytes = L.ctx_total;
  *workspace_bytes = L.ws_total;
  return SF_OK;
}

int sf_routed_ffn_fwd(const sf_router_desc* desc, const void* X, const void* W1, const void* W2, const void* means,
                      const void* forced_expert, void* Y, void* fwd_ctx, size_t fwd_ctx_bytes, void* workspace,
                      size_t workspace_bytes, void* stream) {
  SF_TRY(check_router_desc(desc));
  SF_TRY(check_ptrs({X, W1, W2, means, Y, fwd_ctx, workspace}));
  const sf_router_desc& d = *desc;
  const RoutedLayout L = routed_layout(d);
  if (fwd_ctx_bytes < L.ctx_total || workspace_bytes < L.ws_total) return SF_ERR_WORKSPACE;
  SF_TRY(check_arch());
  cudaStream_t s = (cudaStream_t)stream;
  int* status = (int*)workspace;
  int* expert = (int*)at(fwd_ctx, L.expert);
  int* seg = (int*)at(fwd_ctx, L.seg);
  int* counts = (int*)at(fwd_ctx, L.counts);
  int* src = (int*)at(fwd_ctx, L.src_of_row);

  // Algorithm 1 line 4: W1s = sparsify24(W1) along d_model
  trace_mark(s);
  SF_TRY(launch_prune24(W1, d.F, d.D, d.D, 1, d.prune_mode, at(workspace, L.w1_vals), at(workspace, L.w1_meta),
                        at(workspace, L.w1_meta_hw), nullptr, s));
  trace_mark(s);
  // Section 3.1 step 1: expert of every token (or the caller's, for stage-wise comparison)
  if (forced_expert) {
    SF_CUDA_TRY(cudaMemcpyAsync(expert, forced_expert, (size_t)d.T * 4, cudaMemcpyDeviceToDevice, s));
  } else {
    // T % 256 == 0 here: the logits are one tensor-core product with the arg-max in its epilogue
    SF_TRY(gemm_route(X, means, d.T, d.D, d.E, (int*)expert, (float*)at(fwd_ctx, L.logits), (int*)workspace, s));
  }
  trace_mark(s);
  // step 2: token order, tile tables, gathered X
  static bool attr_done[64] = {false};
  int dev = 0;
  SF_CUDA_TRY(cudaGetDevice(&dev));
  const int gsm = (d.E * 1024 + kMaxExperts + 1) * 4;
  if (dev < 0 || dev >= 64 || !attr_done[dev]) {
    SF_CUDA_TRY(cudaFuncSetAttribute(group_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (kMaxExperts * 1024 + kMaxExperts + 1) * 4));
    if (dev >= 0 && dev < 64) attr_done[dev] = true;
  }
  group_kernel<<<1, 1024, gsm, s>>>(expert, (int)d.T, d.E, (int)L.rows_max, (int*)at(fwd_ctx, L.row_of_token), src, seg);
  SF_LAUNCH_CHECK();
  tile_tables_kernel<<<1, 256, 0, s>>>(seg, d.E, (int)d.D, (int)d.F, (GemmTile*)at(fwd_ctx, L.tabA),
                                       (GemmTile*)at(fwd_ctx, L.tabB), (GemmTile*)at(fwd_ctx, L.tabC),
                                       (GemmTile*)at(fwd_ctx, L.tabD), counts);
  SF_LAUNCH_CHECK();
  SF_TRY(launch_gather_rows(X, src, at(fwd_ctx, L.xp), L.rows_max, d.D, s));
  trace_mark(s);
  // step 3: y1 = Xp W1s[expert]^T with SquaredReLU and the 2:4 selection in the epilogue
  Act24Out out{at(fwd_ctx, L.y2_vals), at(fwd_ctx, L.relu_vals), at(fwd_ctx, L.meta), at(fwd_ctx, L.meta_hw),
               at(fwd_ctx, L.y2_dense), (d.flags & SF_FFN_SAVE_Y1) ? (void*)at(fwd_ctx, L.y1) : nullptr};
  SF_TRY(gemm_grouped_act24(at(workspace, L.w1_vals), at(workspace, L.w1_meta_hw), at(fwd_ctx, L.xp), L.rows_max, d.F,
                            L.Fe, d.D, out, (const GemmTile*)at(fwd_ctx, L.tabA), counts + 0, L.max_tiles[0], status, s));
  trace_mark(s);
  // Algorithm 1 line 7: y3 = y2 W2^T over the expert's features only (W2 dense), then back to token order
  // (the epilogue stores every row at its token's place: src_of_row is the row map, padding rows are dropped)
  SF_TRY(gemm_grouped_sparse24_rm(at(fwd_ctx, L.y2_vals), at(fwd_ctx, L.meta_hw), W2, true, L.rows_max, d.D, L.Fe, d.F,
                                  Y, src, (const GemmTile*)at(fwd_ctx, L.tabB), counts + 1, L.max_tiles[1], status, s));
  trace_mark(s);
  return SF_OK;
}

int sf_routed_ffn_bwd(const sf_router_desc* desc, const void* dY, const void* X, const void* W1, const void* W2,
                      const void* fwd_ctx, size_t fwd_ctx_bytes, void* dX, void* dW1, void* dW2, void* workspace,
                      size_t workspace_bytes, void* stream) {
  SF_TRY(check_router_desc(desc));
  SF_TRY(check_ptrs({dY, X, W1, W2, fwd_ctx, dX, dW1, dW2, workspace}));
  const sf_router_desc& d = *desc;
  const RoutedLayout L = routed_layout(d);
  if (fwd_ctx_bytes < L.ctx_total || workspace_bytes < L.ws_total) return SF_ERR_WORKSPACE;
  SF_TRY(check_arch());
  cudaStream_t s = (cudaStream_t)stream;
  int* status = (int*)workspace;
  const int* counts = (const int*)at(fwd_ctx, L.counts);
  const int* src = (const int*)at(fwd_ctx, L.src_of_row);

  // Algorithm 2 line 2: W2s = sparsify24(W2^T) along d_model (strided groups of W2 [D, F])
  trace_mark(s);
  SF_TRY(launch_prune24(W2, d.D, d.F, d.F, 0, d.prune_mode, at(workspace, L.w2_vals), at(workspace, L.w2_meta),
                        at(workspace, L.w2_meta_hw), nullptr, s));
  trace_mark(s);
  SF_TRY(launch_gather_rows(dY, src, at(workspace, L.dyp), L.rows_max, d.D, s));
  trace_mark(s);
  // dy2 = dYp W2s[expert];  line 4: dy1 = 2 dy2 ReLU(y1) on y2's mask, in the product's epilogue
  SF_TRY(gemm_grouped_drelu24(at(workspace, L.w2_vals), at(workspace, L.w2_meta_hw), at(workspace, L.dyp), L.rows_max,
                              d.F, L.Fe, d.D, at(fwd_ctx, L.relu_vals), at(fwd_ctx, L.meta), at(workspace, L.dy1_vals),
                              at(workspace, L.dy1_dense), (const GemmTile*)at(fwd_ctx, L.tabA), counts + 0,
                              L.max_tiles[0], status, s));
  trace_mark(s);
  // line 5: dX = dy1 W1 over the expert's features (W1 dense), back to token order
  SF_TRY(gemm_grouped_sparse24_rm(at(workspace, L.dy1_vals), at(fwd_ctx, L.meta_hw), W1, false, L.rows_max, d.D, L.Fe,
                                  d.F, dX, src, (const GemmTile*)at(fwd_ctx, L.tabB), counts + 1, L.max_tiles[1],
                                  status, s));
  trace_mark(s);
  // line 3: dW2[:, expert block] = dY_e^T y2_e;  line 6: dW1[expert block, :] = dy1_e^T X_e
  SF_TRY(gemm_grouped_dense_tn(at(workspace, L.dyp), d.D, at(fwd_ctx, L.y2_dense), L.Fe, L.rows_max, dW2, d.F,
                               (const GemmTile*)at(fwd_ctx, L.tabC), counts + 2, L.max_tiles[2], status, s));
  trace_mark(s);
  SF_TRY(gemm_grouped_dense_tn(at(workspace, L.dy1_dense), L.Fe, at(fwd_ctx, L.xp), d.D, L.rows_max, dW1, d.D,
                               (const GemmTile*)at(fwd_ctx, L.tabD), counts + 3, L.max_tiles[3], status, s));
  trace_mark(s);
  return SF_OK;
}

int sf_routed_ctx_view(const sf_router_desc* desc, const void* buf, int field, const void** ptr, size_t* bytes) {
  if (!ptr || !bytes || !buf) return SF_ERR_NULL;
  SF_TRY(check_router_desc(desc));
  const sf_router_desc& d = *desc;
  const RoutedLayout L = routed_layout(d);
  const size_t R = L.rows_max, Fe = L.Fe;
  size_t off, n;
  switch (field) {
    case SF_RCTX_EXPERT: off = L.expert; n = (size_t)d.T * 4; break;
    case SF_RCTX_ROW_OF_TOKEN: off = L.row_of_token; n = (size_t)d.T * 4; break;
    case SF_RCTX_SRC_OF_ROW: off = L.src_of_row; n = R * 4; break;
    case SF_RCTX_SEGMENTS: off = L.seg; n = (size_t)(2 * d.E + 1) * 4; break;
    case SF_RCTX_LOGITS: off = L.logits; n = (size_t)d.T * d.E * 4; break;
    case SF_RCTX_Y2_VALS: off = L.y2_vals; n = R * Fe; break;
    case SF_RCTX_RELU_VALS: off = L.relu_vals; n = R * Fe; break;
    case SF_RCTX_META: off = L.meta; n = R * Fe / 8; break;
    case SF_RCTX_Y1:
      if (!(d.flags & SF_FFN_SAVE_Y1)) return SF_ERR_UNSUPPORTED;
      off = L.y1; n = R * Fe * 2; break;
    case SF_RCTX_DY1_VALS: off = L.dy1_vals; n = R * Fe; break;
    default: return SF_ERR_SHAPE;
  }
  *ptr = at(buf, off);
  *bytes = n;
  return SF_OK;
}

}  // extern "C"
