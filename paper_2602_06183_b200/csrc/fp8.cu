// E4M3 operands (Section 3.2.2, last paragraph: quantisation folded into the passes that already scan a
// matrix): per-tensor-scaled quantisation, 2:4 pruning with the kept values quantised in the same pass,
// and the two tensor-core products on such operands.
//
// q = e4m3(float(x) * scale): one float32 product, one conversion (round to nearest even, magnitudes
// above 448 clamp to 448). Selection and soft-threshold shrinkage are those of the bf16 pass.
#include "fp8_fmt.cuh"
#include "gemm_tc.cuh"
#include "sf_common.cuh"

#define SF_TRY(expr)              \
  do {                            \
    int _st = (expr);             \
    if (_st != SF_OK) return _st; \
  } while (0)

namespace sf {

namespace {

constexpr size_t kStatusBytes8 = 256;

// One thread converts 16 consecutive elements of a row: two 128-bit loads, one 128-bit store.
__global__ void __launch_bounds__(256)
quantize_fp8_kernel(const uint4* __restrict__ X, int64_t rows, int cols, int64_t ld, float scale, uint4* __restrict__ out) {
  const int chunks = cols >> 4;
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= rows * chunks) return;
  const int64_t r = idx / chunks;
  const int c = (int)(idx - r * chunks);
  const uint4* src = X + ((r * ld) >> 3) + (c << 1);
  const uint4 a = __ldg(src), b = __ldg(src + 1);
  uint4 o;
  o.x = quant2(a.x, scale) | (quant2(a.y, scale) << 16);
  o.y = quant2(a.z, scale) | (quant2(a.w, scale) << 16);
  o.z = quant2(b.x, scale) | (quant2(b.y, scale) << 16);
  o.w = quant2(b.z, scale) | (quant2(b.w, scale) << 16);
  out[idx] = o;
}

// Work unit = eight consecutive elements of a row (two groups, one 128-bit load): four codes, one metadata
// byte. All outputs are contiguous by unit, so a thread takes kUnitsPerThread units a whole CTA apart: every
// load and store instruction of a warp covers one contiguous range. The four metadata bytes of four
// neighbouring lanes leave as one word. 2 B read + 0.5 B codes + 1/8 B metadata per element.
constexpr int kUnitsPerThread = 4;

template <bool kSoft>
__global__ void __launch_bounds__(256)
prune24_fp8_kernel(const uint4* __restrict__ W, int64_t rows, int cols, int64_t ld, float scale,
                   uint32_t* __restrict__ vals, uint32_t* __restrict__ meta, uint2* __restrict__ dense_out) {
  __shared__ Top2Entry lut[16];
  top2_lut_init(lut, threadIdx.x);
  __syncthreads();
  const uint32_t upr = (uint32_t)cols >> 3;                       // units per row
  const int64_t total = rows * (int64_t)upr;
  const int64_t base = (int64_t)blockIdx.x * (256 * kUnitsPerThread) + threadIdx.x;
  uint4 q[kUnitsPerThread];
#pragma unroll
  for (int j = 0; j < kUnitsPerThread; ++j) {
    const int64_t u = base + j * 256;
    if (u < total) {
      if (ld == (int64_t)cols) {                                   // contiguous rows: the unit index is the address
        q[j] = __ldg(W + u);
      } else if (total <= 0xFFFFFFFFll) {
        const uint32_t r = (uint32_t)u / upr;
        q[j] = __ldg(W + (((int64_t)r * ld) >> 3) + ((uint32_t)u - r * upr));
      } else {
        const int64_t r = u / upr;
        q[j] = __ldg(W + ((r * ld) >> 3) + (u - r * upr));
      }
    } else {
      q[j] = make_uint4(0u, 0u, 0u, 0u);
    }
  }
#pragma unroll
  for (int j = 0; j < kUnitsPerThread; ++j) {
    const int64_t u = base + j * 256;                             // warp-uniform validity except in the last warp
    // the unit's two groups share one pass of the 16-bit-halves selection
    Top2Entry ea, eb;
    top2of4_x2<kSoft>(__byte_perm(q[j].x, q[j].z, 0x5410u), __byte_perm(q[j].x, q[j].z, 0x7632u),
                      __byte_perm(q[j].y, q[j].w, 0x5410u), __byte_perm(q[j].y, q[j].w, 0x7632u), lut, ea, eb);
    const uint32_t pa = kSoft ? soft_threshold_pair(q[j].x, q[j].y, ea) : __byte_perm(q[j].x, q[j].y, ea.kept);
    const uint32_t pb = kSoft ? soft_threshold_pair(q[j].z, q[j].w, eb) : __byte_perm(q[j].z, q[j].w, eb.kept);
    const uint32_t na = (ea.kept >> 16) & 0xFu, nb = (eb.kept >> 16) & 0xFu;
    const uint32_t ca = quant2(pa, scale), cb = quant2(pb, scale);
    uint32_t mb = na | (nb << 4);
    mb |= __shfl_down_sync(0xFFFFFFFFu, mb, 1) << 8;
    mb |= __shfl_down_sync(0xFFFFFFFFu, mb, 2) << 16;
    if (u >= total) continue;
    vals[u] = ca | (cb << 16);
    if ((threadIdx.x & 3) == 0) meta[u >> 2] = mb;               // total % 4 == 0 (cols % 32 == 0)
    if (dense_out) {
      // a group's four bytes: code 0 at position p0, code 1 at p1, +0 elsewhere
      dense_out[u] = make_uint2(((ca & 0xFFu) << (8u * (na & 3u))) | ((ca >> 8) << (8u * (na >> 2))),
                                ((cb & 0xFFu) << (8u * (nb & 3u))) | ((cb >> 8) << (8u * (nb >> 2))));
    }
  }
}

__global__ void meta_reorder8_kernel(const uint16_t* __restrict__ meta, uint8_t* __restrict__ meta_hw, int64_t R, int64_t K) {
  const int64_t words = K >> 4;
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= R * words) return;
  const int64_t m = idx / words, kw = idx - m * words;
  *reinterpret_cast<uint16_t*>(meta_hw + meta_hw8_offset(m, kw, K)) = meta[idx];
}

}  // namespace

}  // namespace sf

using namespace sf;

extern "C" {

int sf_fp8_quantize(const void* X, int64_t rows, int64_t cols, int64_t ld, float scale, void* Xq, void* stream) {
  if (rows < 0 || cols < 0 || cols % 16 != 0 || cols > (int64_t)1 << 30) return SF_ERR_SHAPE;
  if (rows == 0 || cols == 0) return SF_OK;
  if (!X || !Xq) return SF_ERR_NULL;
  if (ld < cols || ld % 8 != 0 || !aligned16(X) || !aligned16(Xq)) return SF_ERR_ALIGN;
  SF_TRY(check_arch());
  const int64_t n = rows * (cols >> 4);
  quantize_fp8_kernel<<<(unsigned)((n + 255) / 256), 256, 0, (cudaStream_t)stream>>>((const uint4*)X, rows, (int)cols, ld,
                                                                                 scale, (uint4*)Xq);
  SF_LAUNCH_CHECK();
  return SF_OK;
}

int sf_prune24_fp8_sizes(int64_t rows, int64_t cols, int group_dim, size_t* vals_bytes, size_t* meta_bytes) {
  if (!vals_bytes || !meta_bytes) return SF_ERR_NULL;
  if (rows < 0 || cols < 0 || (group_dim != 0 && group_dim != 1)) return SF_ERR_SHAPE;
  if (group_dim == 1 ? cols % 32 != 0 : (rows % 16 != 0 || cols % 8 != 0)) return SF_ERR_SHAPE;
  *vals_bytes = (size_t)rows * cols / 2;        // R * K/2 codes
  *meta_bytes = (size_t)rows * cols / 8;        // R * K/16 words * 2 B
  return SF_OK;
}

int sf_prune24_compress_fp8(const void* W, int64_t rows, int64_t cols, int64_t ld, int group_dim, int prune_mode,
                            float scale, void* vals, void* meta, void* dense_out, void* stream) {
  if (rows < 0 || cols < 0 || (group_dim != 0 && group_dim != 1) || (prune_mode != 0 && prune_mode != 1))
    return SF_ERR_SHAPE;
  if (group_dim == 1 ? (cols % 32 != 0 || cols > (int64_t)1 << 30) : (rows % 16 != 0 || cols % 8 != 0)) return SF_ERR_SHAPE;
  if (group_dim == 0 && dense_out) return SF_ERR_UNSUPPORTED;      // the masked copy exists for contiguous groups only
  if (rows == 0 || cols == 0) return SF_OK;
  if (!W || !vals || !meta) return SF_ERR_NULL;
  if (ld < cols || ld % 8 != 0 || !aligned16(W) || !aligned16(vals) || !aligned16(meta) ||
      (dense_out && !aligned16(dense_out)))
    return SF_ERR_ALIGN;
  SF_TRY(check_arch());
  if (group_dim == 0) return launch_prune24_cols_fp8(W, rows, cols, ld, prune_mode, scale, vals, meta, (cudaStream_t)stream);
  const int64_t n = rows * (cols >> 3);
  const int64_t per_cta = 256 * kUnitsPerThread;
  if ((n + per_cta - 1) / per_cta > 0x7FFFFFFF) return SF_ERR_SHAPE;
  const unsigned grid = (unsigned)((n + per_cta - 1) / per_cta);
  cudaStream_t s = (cudaStream_t)stream;
  if (prune_mode == 0)
    prune24_fp8_kernel<false><<<grid, 256, 0, s>>>((const uint4*)W, rows, (int)cols, ld, scale, (uint32_t*)vals,
                                                   (uint32_t*)meta, (uint2*)dense_out);
  else
    prune24_fp8_kernel<true><<<grid, 256, 0, s>>>((const uint4*)W, rows, (int)cols, ld, scale, (uint32_t*)vals,
                                                  (uint32_t*)meta, (uint2*)dense_out);
  SF_LAUNCH_CHECK();
  return SF_OK;
}

int sf_gemm_fp8_workspace_size(int64_t Mr, int64_t K, size_t* bytes) {
  if (!bytes) return SF_ERR_NULL;
  if (Mr < 0 || K < 0) return SF_ERR_SHAPE;
  *bytes = kStatusBytes8 + (size_t)Mr * K / 8;
  return SF_OK;
}

int sf_gemm_fp8_dense(const void* A, const void* B, void* C, int64_t Mr, int64_t Nc, int64_t K, float alpha,
                      void* workspace, void* stream) {
  if (Mr < 0 || Nc < 0 || K <= 0 || Mr % 256 || Nc % 256 || K % 128) return SF_ERR_SHAPE;
  if (Mr == 0 || Nc == 0) return SF_OK;
  if (!A || !B || !C || !workspace) return SF_ERR_NULL;
  if (!aligned16(A) || !aligned16(B) || !aligned16(C) || !aligned16(workspace)) return SF_ERR_ALIGN;
  SF_TRY(check_arch());
  return gemm_fp8(false, A, nullptr, B, Mr, Nc, K, alpha, C, Nc, (int*)workspace, (cudaStream_t)stream);
}

int sf_gemm_fp8_sparse24(const void* a_vals, const void* a_meta, const void* B, void* C, int64_t Mr, int64_t Nc,
                         int64_t K, float alpha, void* workspace, void* stream) {
  if (Mr < 0 || Nc < 0 || K <= 0 || Mr % 256 || Nc % 256 || K % 256) return SF_ERR_SHAPE;
  if (Mr == 0 || Nc == 0) return SF_OK;
  if (!a_vals || !a_meta || !B || !C || !workspace) return SF_ERR_NULL;
  if (!aligned16(a_vals) || !aligned16(a_meta) || !aligned16(B) || !aligned16(C) || !aligned16(workspace))
    return SF_ERR_ALIGN;
  SF_TRY(check_arch());
  cudaStream_t s = (cudaStream_t)stream;
  uint8_t* hw = reinterpret_cast<uint8_t*>(workspace) + kStatusBytes8;
  const int64_t n = Mr * (K >> 4);
  meta_reorder8_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>((const uint16_t*)a_meta, hw, Mr, K);
  SF_LAUNCH_CHECK();
  return gemm_fp8(true, a_vals, hw, B, Mr, Nc, K, alpha, C, Nc, (int*)workspace, s);
}

}  // extern "C"
