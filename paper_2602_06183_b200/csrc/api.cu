// extern "C" entry points of libsparseffn: argument validation, then the launchers.
#include "sf_common.cuh"

namespace sf {

int g_last_cuda_error = 0;

int check_arch() {
  int dev = 0;
  SF_CUDA_TRY(cudaGetDevice(&dev));
  static int cached_major[64] = {0};
  if (dev >= 0 && dev < 64 && cached_major[dev] == 0) {
    int major = 0;
    SF_CUDA_TRY(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
    cached_major[dev] = major;
  }
  const int major = (dev >= 0 && dev < 64) ? cached_major[dev] : 0;
  return major == 10 ? SF_OK : SF_ERR_ARCH;
}

static bool vnm_m_ok(int M) { return M == 4 || M == 8 || M == 16 || M == 32 || M == 64; }

}  // namespace sf

using namespace sf;

extern "C" {

const char* sf_status_string(int status) {
  switch (status) {
    case SF_OK: return "SF_OK";
    case SF_ERR_NULL: return "SF_ERR_NULL: required pointer is NULL";
    case SF_ERR_SHAPE: return "SF_ERR_SHAPE: size violates the divisibility rules";
    case SF_ERR_ALIGN: return "SF_ERR_ALIGN: pointer not 16-byte aligned or ld not a multiple of 8";
    case SF_ERR_WORKSPACE: return "SF_ERR_WORKSPACE: workspace or context too small";
    case SF_ERR_ARCH: return "SF_ERR_ARCH: device is not compute capability 10.x";
    case SF_ERR_CUDA: return "SF_ERR_CUDA: a CUDA call failed";
    case SF_ERR_TIMEOUT: return "SF_ERR_TIMEOUT: a bounded device-side wait expired";
    case SF_ERR_UNSUPPORTED: return "SF_ERR_UNSUPPORTED: configuration not built";
    default: return "unknown sf_status";
  }
}

int sf_last_cuda_error(void) { return g_last_cuda_error; }

int sf_prune24_sizes(int64_t rows, int64_t cols, int group_dim, size_t* vals_bytes, size_t* meta_bytes) {
  if (!vals_bytes || !meta_bytes) return SF_ERR_NULL;
  if (rows < 0 || cols < 0 || (group_dim != 0 && group_dim != 1)) return SF_ERR_SHAPE;
  const int64_t K = group_dim == 1 ? cols : rows;
  if (K % 16 != 0) return SF_ERR_SHAPE;
  *vals_bytes = (size_t)rows * cols;            // R * K/2 elements * 2 B
  *meta_bytes = (size_t)rows * cols / 8;        // R * K/16 words * 2 B
  return SF_OK;
}

int sf_prune24_compress(const void* W, int64_t rows, int64_t cols, int64_t ld, int group_dim,
                        int prune_mode, void* vals, void* meta, void* dense_out, void* stream) {
  if (rows < 0 || cols < 0 || (group_dim != 0 && group_dim != 1) || (prune_mode != 0 && prune_mode != 1))
    return SF_ERR_SHAPE;
  const int64_t K = group_dim == 1 ? cols : rows;
  if (K % 16 != 0 || cols % 8 != 0) return SF_ERR_SHAPE;
  if (rows == 0 || cols == 0) return SF_OK;
  if (!W || !vals || !meta) return SF_ERR_NULL;
  if (ld < cols || ld % 8 != 0 || !aligned16(W) || !aligned16(vals) || !aligned16(meta) ||
      (dense_out && !aligned16(dense_out)))
    return SF_ERR_ALIGN;
  int st = check_arch();
  if (st != SF_OK) return st;
  return launch_prune24(W, rows, cols, ld, group_dim, prune_mode, vals, meta, nullptr, dense_out,
                        (cudaStream_t)stream);
}

int sf_vnm_sizes(int64_t T, int64_t F, int V, int N, int M, size_t* vals_bytes, size_t* meta_bytes,
                 size_t* colidx_bytes) {
  if (!vals_bytes || !meta_bytes || !colidx_bytes) return SF_ERR_NULL;
  if (N != 2) return SF_ERR_UNSUPPORTED;
  if (!vnm_m_ok(M) || V < 1 || V > 128 || T < 0 || F < 0 || T % V != 0 || F % (4 * M) != 0 || F % 64 != 0)
    return SF_ERR_SHAPE;
  *vals_bytes = (size_t)T * (2 * F / M) * 2;
  *meta_bytes = (size_t)T * (F / (4 * M)) * 2;
  *colidx_bytes = (size_t)(T / V) * (F / M) * 4;
  return SF_OK;
}

int sf_vnm_sparsify_act(const void* preact, int64_t T, int64_t F, int64_t ld, int V, int N, int M,
                        int apply_sqrelu, void* vals, void* meta, void* colidx, void* relu_vals,
                        void* dense_out, void* stream) {
  size_t a, b, c;
  int st = sf_vnm_sizes(T, F, V, N, M, &a, &b, &c);
  if (st != SF_OK) return st;
  if (T == 0 || F == 0) return SF_OK;
  if (!preact || !vals || !meta || !colidx) return SF_ERR_NULL;
  if (ld < F || ld % 8 != 0 || !aligned16(preact) || !aligned16(vals) || !aligned16(meta) ||
      !aligned16(colidx) || (relu_vals && !aligned16(relu_vals)) || (dense_out && !aligned16(dense_out)))
    return SF_ERR_ALIGN;
  st = check_arch();
  if (st != SF_OK) return st;
  if (!dense_out && vnm_stream_supported(F, ld, V, M, preact))
    return launch_vnm_stream(preact, T, F, ld, V, M, apply_sqrelu, vals, meta, colidx, relu_vals, (cudaStream_t)stream);
  return launch_vnm(preact, T, F, ld, V, M, apply_sqrelu, vals, meta, nullptr, colidx, relu_vals, dense_out,
                    nullptr, nullptr, nullptr, nullptr, nullptr, (cudaStream_t)stream);
}

}  // extern "C"
