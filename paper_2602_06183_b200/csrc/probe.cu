// Measurement aid (no counterpart in the paper): clocks per tcgen05.mma when the instructions are
// issued back to back on operands that already sit in shared memory -- no loads, no epilogue. It
// calibrates what the tensor pipe can do for a tile shape, so that a product kernel's distance from
// that figure can be attributed to operand delivery, power, or the epilogue.
#include "sf_common.cuh"
#include "tc_ptx.cuh"

namespace sf {
namespace {

using namespace ptx;

struct ProbeCtl {
  uint64_t bar_done;
  uint64_t bar_stage;
  uint32_t tmem_base;
  int abort_flag;
};

constexpr int kProbeABytes = 16384, kProbeBBytes = 32768, kProbeMetaBytes = 2048;
constexpr int kProbeSmem = 1024 + kProbeABytes + kProbeBBytes + kProbeMetaBytes + 256;

// One CTA (or CTA pair) per SM issues 4 * iters MMAs of 128 (256 for a pair) x 256 x 16 (dense) or
// x 32 logical K (2:4) into one accumulator, with a commit after every fourth as a product kernel does.
template <bool kSparse, bool kTwo>
__global__ void __launch_bounds__(128, 1) mma_rate_kernel(int iters, long long* out_cycles, int* status) {
  extern __shared__ uint8_t smem_dyn[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t(1023));
  uint8_t* sA = smem;
  uint8_t* sB = smem + kProbeABytes;
  uint8_t* sM = sB + kProbeBBytes;
  ProbeCtl* ctl = reinterpret_cast<ProbeCtl*>(sM + kProbeMetaBytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = kTwo ? cluster_ctarank() : 0u;
  // operands: finite bf16 values of either sign in [1, 2); metadata: positions (0, 1) in every group
  for (int i = threadIdx.x; i < (kProbeABytes + kProbeBBytes) / 2; i += blockDim.x) {
    const uint32_t h = (uint32_t)i * 2654435761u ^ (blockIdx.x * 40503u);
    reinterpret_cast<uint16_t*>(smem)[i] = (uint16_t)(0x3F80u | ((h >> 9) & 0x7Fu) | ((h & 1u) << 15));
  }
  for (int i = threadIdx.x; i < kProbeMetaBytes / 2; i += blockDim.x) reinterpret_cast<uint16_t*>(sM)[i] = 0x4444;
  if (threadIdx.x == 0) {
    mbar_init(&ctl->bar_done, 1);
    mbar_init(&ctl->bar_stage, 1);
    ctl->abort_flag = 0;
    fence_mbar_init();
  }
  fence_proxy_async_smem();
  if (warp == 1) {
    if (kTwo) {
      tmem_alloc_2cta(&ctl->tmem_base, 512);
      tmem_relinquish_2cta();
    } else {
      tmem_alloc(&ctl->tmem_base, 512);
      tmem_relinquish();
    }
  }
  tc_fence_before();
  __syncthreads();
  if (kTwo) cluster_sync_all();
  tc_fence_after();
  const uint32_t tmem_base = ctl->tmem_base;
  if (warp == 1 && lane == 0) {
    if (rank == 0) {
      constexpr uint32_t idesc = idesc_bf16(kTwo ? 256 : 128, 256, false, false, kSparse);
      const uint64_t a_desc = smem_desc(smem_u32(sA), 16, 1024, kSwizzle128B);
      const uint64_t b_desc = smem_desc(smem_u32(sB), 16, 1024, kSwizzle128B);
      const uint64_t m_desc = smem_desc(smem_u32(sM), 128, 128, kSwizzleNone);
      if (kSparse) {
        if (kTwo) tmem_cp_128x128b_2cta(tmem_base + 256, m_desc);
        else tmem_cp_128x128b(tmem_base + 256, m_desc);
      }
      const long long t0 = clock64();
      for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const uint64_t ad = a_desc + (uint64_t)(k * 2);                  // 32 bytes per K step
          if (kSparse) {
            // 64 bytes of B per step; a pair holds two 16 KB K-slabs per CTA, one CTA a single 32 KB slab
            const uint64_t bd = b_desc + (uint64_t)((kTwo ? (k >> 1) * (16384 >> 4) : 0) + (k & 1) * 4);
            if (kTwo) mma_sp_f16_2cta(tmem_base, ad, bd, tmem_base + 256 + (k & ~1), idesc | (k & 1), 1u);
            else mma_sp_f16(tmem_base, ad, bd, tmem_base + 256 + (k & ~1), idesc | (k & 1), 1u);
          } else {
            const uint64_t bd = b_desc + (uint64_t)(k * 2);
            if (kTwo) mma_f16_2cta(tmem_base, ad, bd, idesc, 1u);
            else mma_f16(tmem_base, ad, bd, idesc, 1u);
          }
        }
        if (kTwo) mma_commit_2cta(&ctl->bar_stage);
        else mma_commit(&ctl->bar_stage);
      }
      if (kTwo) mma_commit_2cta(&ctl->bar_done);
      else mma_commit(&ctl->bar_done);
      const bool ok = mbar_wait(&ctl->bar_done, 0, &ctl->abort_flag);
      const long long cycles = clock64() - t0;
      if (!ok) atomicExch(status, 1);
      if (blockIdx.x == 0) *out_cycles = cycles;
    } else {
      // the peer keeps its shared memory and TMEM alive until the leader's MMAs have drained
      if (!mbar_wait(&ctl->bar_done, 0, &ctl->abort_flag)) atomicExch(status, 1);
    }
  }
  __syncthreads();
  if (kTwo) cluster_sync_all();
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    if (kTwo) tmem_dealloc_2cta(tmem_base, 512);
    else tmem_dealloc(tmem_base, 512);
  }
}

template <bool kSparse, bool kTwo>
int launch_probe(int iters, long long* out_cycles, int* status, cudaStream_t s) {
  auto kern = mma_rate_kernel<kSparse, kTwo>;
  SF_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kProbeSmem));
  int dev = 0, sms = 0;
  SF_CUDA_TRY(cudaGetDevice(&dev));
  SF_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(sms & ~1));
  cfg.blockDim = dim3(128);
  cfg.dynamicSmemBytes = kProbeSmem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = kTwo ? 2 : 1;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  SF_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, iters, out_cycles, status));
  return SF_OK;
}

}  // namespace
}  // namespace sf

extern "C" int sf_probe_mma_rate(int sparse, int two_cta, int iters, void* cycles, void* workspace, void* stream) {
  if (!cycles || !workspace) return SF_ERR_NULL;
  if (iters <= 0 || iters > (1 << 20)) return SF_ERR_SHAPE;
  if ((reinterpret_cast<uintptr_t>(cycles) & 7) != 0) return SF_ERR_ALIGN;
  {
    const int st = sf::check_arch();
    if (st != SF_OK) return st;
  }
  cudaStream_t s = (cudaStream_t)stream;
  long long* out = reinterpret_cast<long long*>(cycles);
  int* status = reinterpret_cast<int*>(workspace);
  if (sparse) return two_cta ? sf::launch_probe<true, true>(iters, out, status, s) : sf::launch_probe<true, false>(iters, out, status, s);
  return two_cta ? sf::launch_probe<false, true>(iters, out, status, s) : sf::launch_probe<false, false>(iters, out, status, s);
}
