// sf_gemm_sparse24_noalloc: the 2:4-sparse product for callers that cannot allocate device memory.
//
// The regular entry point needs a caller-allocated workspace for the metadata copy in tensor-core
// order and for the status word. Here that scratch lives in a device array that is part of the
// library image, so a caller that has no allocator at hand (code running inside a framework's
// allocator callback, a plugin that is only handed input/output buffers, a process whose memory
// pool is already fully committed) can still run the product.
#include "sf_common.cuh"
#include "gemm_tc.cuh"

namespace sf {
namespace {

constexpr size_t kNoAllocStatusBytes = 256;
constexpr size_t kNoAllocMetaBytes = 4u << 20;          // metadata of at most 32 Mi logical elements

// Resident on every device that loads the library, until the process exits.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocStatusBytes + kNoAllocMetaBytes];

// Device address of the scratch array, looked up once per device. In host code the array's name is
// only a handle for the runtime; the address a kernel can use comes from cudaGetSymbolAddress with
// the owning device current.
int noalloc_scratch(unsigned char** out) {
  static unsigned char* cached[64] = {nullptr};
  int dev = 0;
  SF_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return SF_ERR_UNSUPPORTED;
  if (!cached[dev]) {
    void* p = nullptr;
    SF_CUDA_TRY(cudaGetSymbolAddress(&p, g_noalloc_scratch));
    cached[dev] = static_cast<unsigned char*>(p);
  }
  *out = cached[dev];
  return SF_OK;
}

}  // namespace

// Device address of the built-in status word (sf_check_status with a null workspace reads it).
int noalloc_status_word(void** out) {
  unsigned char* p = nullptr;
  const int st = noalloc_scratch(&p);
  *out = p;
  return st;
}

}  // namespace sf

using namespace sf;

extern "C" int sf_gemm_sparse24_noalloc(const void* a_vals, const void* a_meta, const void* B, void* Ct, int64_t Mr,
                                        int64_t Nc, int64_t K, void* stream) {
  if (Mr < 0 || Nc < 0 || K <= 0 || Mr % 128 || Nc % 256 || K % 128) return SF_ERR_SHAPE;
  if ((size_t)Mr * (size_t)K / 8 > kNoAllocMetaBytes) return SF_ERR_WORKSPACE;   // beyond the built-in scratch
  if (Mr == 0 || Nc == 0) return SF_OK;
  if (!a_vals || !a_meta || !B || !Ct) return SF_ERR_NULL;
  if (!aligned16(a_vals) || !aligned16(a_meta) || !aligned16(B) || !aligned16(Ct)) return SF_ERR_ALIGN;
  int st = check_arch();
  if (st != SF_OK) return st;
  unsigned char* scratch = nullptr;
  st = noalloc_scratch(&scratch);
  if (st != SF_OK) return st;
  cudaStream_t s = (cudaStream_t)stream;
  // The array keeps whatever the previous call left: the status word must start at zero; the
  // metadata region is rewritten in full for this call's shape before the product reads it.
  SF_CUDA_TRY(cudaMemsetAsync(scratch, 0, kNoAllocStatusBytes, s));
  unsigned char* hw = scratch + kNoAllocStatusBytes;
  st = launch_meta_reorder(a_meta, hw, Mr, K, s);
  if (st != SF_OK) return st;
  return gemm_sparse24(a_vals, hw, B, true, Mr, Nc, K, EPI_STORE_T, Ct, Mr, nullptr, 0, reinterpret_cast<int*>(scratch), s);
}
