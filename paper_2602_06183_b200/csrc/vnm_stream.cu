// SquaredReLU + V:N:M sparsification, streaming form (Eq. 2, Section 2.3), for M in {8, 16, 32, 64}.
//
// Same selection rule and outputs as the kernels of vnm.cu (values, ReLU values, canonical metadata, colidx), organised
// as a pipeline so that loading, scoring and emitting overlap inside one CTA instead of alternating:
//   warp 0        TMA producer: one bulk tensor load per V x 256 strip into a three-slot ring
//   warps 1..4    column scores (sequential float32 sums, two columns per thread), ranking of the eight columns
//                 of every group, colidx
//   warps 5..12   emit: one thread per (row, group): 2:4 among the kept columns, packed stores
// Persistent CTAs walk the strips; every wait is bounded (a role that gives up makes the others leave too).
#include "sf_common.cuh"
#include "sparse_fmt.cuh"
#include "tc_ptx.cuh"
#include "gemm_tc.cuh"

namespace sf {
namespace {

using namespace ptx;

constexpr int kSlots = 3;
constexpr int kThreadsS = 32 + 128 + 256;

// kSW = columns per strip: 256 for V <= 64, 128 for taller blocks (three slots then still leave room for two
// CTAs per SM).
template <int kSW>
struct StripAux {
  uint32_t score[kSW];
  uint8_t keep[kSW];
  uint8_t cidx[kSW / 8 * 4];             // [groups of the strip][4]; sized for the narrowest group
};

struct StreamCtl {
  uint64_t full[kSlots], scored[kSlots], empty[kSlots];
  int abort_flag;
};

__device__ __forceinline__ void named_sync(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}

template <int kSW, int kM>
__global__ void __launch_bounds__(kThreadsS)
vnm_stream_kernel(const __grid_constant__ CUtensorMap tmapP, int64_t T, int64_t F, int V, int apply,
                   uint16_t* __restrict__ vals, uint16_t* __restrict__ meta, uint8_t* __restrict__ colidx,
                   uint16_t* __restrict__ relu_vals) {
  extern __shared__ uint8_t smem_dyn[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_dyn) + 127) & ~uintptr_t(127));
  const int strip_bytes = V * kSW * 2;
  using Aux = StripAux<kSW>;
  Aux* aux = reinterpret_cast<Aux*>(smem + kSlots * strip_bytes);
  StreamCtl* ctl = reinterpret_cast<StreamCtl*>(aux + kSlots);
  volatile int* abort_flag = &ctl->abort_flag;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int nsx = (int)((F + kSW - 1) / kSW);
  const int64_t nstrips = (T / V) * nsx;
  const int64_t G = F / kM;

  __shared__ Top2Entry lut[16];
  top2_lut_init(lut, tid);
  if (tid == 0) {
    prefetch_tmap(&tmapP);
    for (int s = 0; s < kSlots; ++s) {
      mbar_init(&ctl->full[s], 1);
      mbar_init(&ctl->scored[s], 4);
      mbar_init(&ctl->empty[s], 8);
    }
    ctl->abort_flag = 0;
    fence_mbar_init();
  }
  __syncthreads();

  if (warp == 0) {
    // =========================== producer ===========================
    uint32_t slot = 0, phase = 0;
    for (int64_t i = blockIdx.x; i < nstrips; i += gridDim.x) {
      if (!mbar_wait(&ctl->empty[slot], phase ^ 1, abort_flag)) break;
      if (lane == 0) {
        const int64_t blk = i / nsx, cx = i - blk * nsx;
        mbar_arrive_expect_tx(&ctl->full[slot], (uint32_t)strip_bytes);
        tma_load_2d(smem + slot * strip_bytes, &tmapP, &ctl->full[slot], (int)(cx * kSW), (int)(blk * V));
      }
      if (++slot == kSlots) { slot = 0; phase ^= 1; }
    }
  } else if (warp <= 4) {
    // =========================== score + rank (128 threads) ===========================
    const int ts = tid - 32;
    uint32_t slot = 0, phase = 0;
    for (int64_t i = blockIdx.x; i < nstrips; i += gridDim.x) {
      const int64_t blk = i / nsx, cx = i - blk * nsx;
      const int cvalid = (int)min((int64_t)kSW, F - cx * kSW);
      Aux& a = aux[slot];
      if (!mbar_wait(&ctl->full[slot], phase, abort_flag)) break;
      // rows first to last, one float32 add per element: two columns per thread (256-column strips) or one
      if constexpr (kSW == 256) {
        const uint32_t* col = reinterpret_cast<const uint32_t*>(smem + slot * strip_bytes) + ts;
        float s0 = 0.f, s1 = 0.f;
        for (int r = 0; r < V; r += 8) {
          uint32_t h[8];
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            const uint32_t w = col[(r + u) * (kSW / 2)];
            h[u] = apply ? bf2_sq(bf2_relu(w)) : (w & 0x7FFF7FFFu);
          }
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            s0 = __fadd_rn(s0, __uint_as_float(h[u] << 16));
            s1 = __fadd_rn(s1, __uint_as_float(h[u] & 0xFFFF0000u));
          }
        }
        a.score[2 * ts] = __float_as_uint(s0);
        a.score[2 * ts + 1] = __float_as_uint(s1);
      } else {
        const uint16_t* col = reinterpret_cast<const uint16_t*>(smem + slot * strip_bytes) + ts;
        float s0 = 0.f;
        for (int r = 0; r < V; r += 16) {
          uint32_t h[16];
#pragma unroll
          for (int u = 0; u < 16; ++u) {
            const uint32_t w = col[(r + u) * kSW];
            h[u] = apply ? bf2_sq(bf2_relu(w)) : (w & 0x7FFFu);
          }
#pragma unroll
          for (int u = 0; u < 16; ++u) s0 = __fadd_rn(s0, __uint_as_float(h[u] << 16));
        }
        a.score[ts] = __float_as_uint(s0);
      }
      named_sync(1, 128);
      constexpr int kCPT = kSW / 128;                          // columns per scoring thread
#pragma unroll
      for (int c = 0; c < kCPT; ++c) {
        const int j = kCPT * ts + c, jm = j & (kM - 1), base = j - jm;
        const uint32_t s = a.score[j];
        int rank = 0;
#pragma unroll 8
        for (int k = 0; k < kM; ++k) {
          const uint32_t sk = a.score[base + k];
          rank += (sk > s) || (sk == s && k < jm);
        }
        a.keep[j] = rank < 4;
      }
      named_sync(1, 128);
#pragma unroll
      for (int c = 0; c < kCPT; ++c) {
        const int j = kCPT * ts + c, jm = j & (kM - 1), base = j - jm;
        if (a.keep[j]) {
          int pos = 0;
          for (int k = 0; k < jm; ++k) pos += a.keep[base + k];
          a.cidx[(j / kM) * 4 + pos] = (uint8_t)jm;
        }
      }
      named_sync(1, 128);
      const int ng = cvalid / kM;
      if (ts < ng)
        *reinterpret_cast<uint32_t*>(colidx + (blk * G + cx * (kSW / kM) + ts) * 4) =
            *reinterpret_cast<const uint32_t*>(a.cidx + ts * 4);
      __syncwarp();
      if (lane == 0) mbar_arrive(&ctl->scored[slot]);
      if (++slot == kSlots) { slot = 0; phase ^= 1; }
    }
  } else {
    // =========================== emit (256 threads) ===========================
    constexpr int kGS = kSW / kM, kRows = 256 / kGS;         // groups per strip row, rows in flight
    const int te = tid - 160, g = te & (kGS - 1), r0 = te / kGS;
    const bool want_relu = relu_vals != nullptr && apply;
    uint32_t slot = 0, phase = 0;
    for (int64_t i = blockIdx.x; i < nstrips; i += gridDim.x) {
      const int64_t blk = i / nsx, cx = i - blk * nsx;
      const int cvalid = (int)min((int64_t)kSW, F - cx * kSW);
      const bool live = g < cvalid / kM;
      const Aux& a = aux[slot];
      if (!mbar_wait(&ctl->scored[slot], phase, abort_flag)) break;
      const uint32_t c4 = *reinterpret_cast<const uint32_t*>(a.cidx + g * 4);
      uint32_t selp[2], mhi[2];
#pragma unroll
      for (int pr = 0; pr < 2; ++pr) {
        const uint32_t ca = (c4 >> (16 * pr)) & 0xFFu, cb = (c4 >> (16 * pr + 8)) & 0xFFu;
        const uint32_t sa = 2u * (ca & 3u), sb = 2u * (cb & 3u);
        selp[pr] = sa | ((sa + 1u) << 4) | (sb << 8) | ((sb + 1u) << 12);
        mhi[pr] = ((ca & 4u) ? 0x0000FFFFu : 0u) | ((cb & 4u) ? 0xFFFF0000u : 0u);
      }
      const int64_t gg = cx * (kSW / kM) + g, trow = blk * V + r0;
      const uint8_t* tp = smem + slot * strip_bytes + r0 * (kSW * 2) + g * (kM * 2);
      const int o0 = 2 * (int)(c4 & 0xFFu), o1 = 2 * (int)((c4 >> 8) & 0xFFu), o2 = 2 * (int)((c4 >> 16) & 0xFFu),
                o3 = 2 * (int)(c4 >> 24);                      // byte offsets of the kept columns inside the group
      uint32_t* p_vals = reinterpret_cast<uint32_t*>(vals) + trow * G + gg;
      uint32_t* p_relu = want_relu ? reinterpret_cast<uint32_t*>(relu_vals) + trow * G + gg : nullptr;
      uint16_t* p_meta = meta + trow * (G >> 2) + (gg >> 2);
      const int64_t s_vals = kRows * G, s_meta = kRows * (G >> 2);
      const bool lead4 = (g & 3) == 0;
      // the four kept columns of a row as two packed pairs, then the activation on those only
      auto kept = [&](const uint8_t* rowp, uint32_t& rk0, uint32_t& rk1, uint32_t& hk0, uint32_t& hk1) {
        if constexpr (kM == 8) {                              // one 16-byte load, picked apart by byte permutes
          const uint4 q = *reinterpret_cast<const uint4*>(rowp);
          const uint32_t a0 = __byte_perm(q.x, q.y, selp[0]), b0 = __byte_perm(q.z, q.w, selp[0]);
          const uint32_t a1 = __byte_perm(q.x, q.y, selp[1]), b1 = __byte_perm(q.z, q.w, selp[1]);
          rk0 = (a0 & ~mhi[0]) | (b0 & mhi[0]);
          rk1 = (a1 & ~mhi[1]) | (b1 & mhi[1]);
        } else {                                              // wide groups: four 16-bit loads
          rk0 = (uint32_t)*reinterpret_cast<const uint16_t*>(rowp + o0) |
                ((uint32_t)*reinterpret_cast<const uint16_t*>(rowp + o1) << 16);
          rk1 = (uint32_t)*reinterpret_cast<const uint16_t*>(rowp + o2) |
                ((uint32_t)*reinterpret_cast<const uint16_t*>(rowp + o3) << 16);
        }
        hk0 = rk0; hk1 = rk1;
        if (apply) {
          rk0 = bf2_relu(rk0); rk1 = bf2_relu(rk1);
          hk0 = bf2_sq(rk0); hk1 = bf2_sq(rk1);
        }
      };
      auto put = [&](uint32_t packed, uint32_t rpair, uint32_t nib) {
        if (live) *p_vals = packed;
        if (want_relu) {
          if (live) *p_relu = rpair;
          p_relu += s_vals;
        }
        uint32_t word = nib;
        word |= __shfl_down_sync(0xFFFFFFFFu, word, 1) << 4;
        word |= __shfl_down_sync(0xFFFFFFFFu, word, 2) << 8;
        if (lead4 && live) *p_meta = (uint16_t)word;
        p_vals += s_vals;
        p_meta += s_meta;
      };
      int r = r0;
      // groups of eight (the emit-heavy case): two rows per pass, their 2:4 choices share one run of the
      // 16-bit-halves selection; wider groups measured faster one row at a time
      if constexpr (kM == 8)
      for (; r + kRows < V; r += 2 * kRows) {
        uint32_t ra0, ra1, ha0, ha1, rb0, rb1, hb0, hb1;
        Top2Entry ea, eb;
        kept(tp, ra0, ra1, ha0, ha1);
        kept(tp + kRows * kSW * 2, rb0, rb1, hb0, hb1);
        top2of4_x2(__byte_perm(ha0, hb0, 0x5410u), __byte_perm(ha0, hb0, 0x7632u), __byte_perm(ha1, hb1, 0x5410u),
                   __byte_perm(ha1, hb1, 0x7632u), lut, ea, eb);
        put(__byte_perm(ha0, ha1, ea.kept), __byte_perm(ra0, ra1, ea.kept), (ea.kept >> 16) & 0xFu);
        put(__byte_perm(hb0, hb1, eb.kept), __byte_perm(rb0, rb1, eb.kept), (eb.kept >> 16) & 0xFu);
        tp += 2 * kRows * kSW * 2;
      }
      for (; r < V; r += kRows) {                             // single rows: wide groups, or an odd last pass
        uint32_t rk0, rk1, hk0, hk1, packed, psel;
        kept(tp, rk0, rk1, hk0, hk1);
        const uint32_t nib = top2of4_packed(hk0, hk1, &packed, nullptr, &psel);
        put(packed, __byte_perm(rk0, rk1, psel), nib);
        tp += kRows * kSW * 2;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&ctl->empty[slot]);
      if (++slot == kSlots) { slot = 0; phase ^= 1; }
    }
  }
}

}  // namespace

bool vnm_stream_supported(int64_t F, int64_t ld, int V, int M, const void* P) {
  // TMA: 16-byte aligned base and row pitch; box rows = V; emit threads take rows in steps of 256 * M / strip width
  if (!(M == 8 || M == 16 || M == 32 || M == 64)) return false;
  // 256 emit threads over (strip width / M) groups; M = 64 always takes 256-column strips (a metadata word
  // spans four groups)
  const int rows_in_flight = (V <= 64 || M == 64) ? M : 2 * M;
  return V >= 16 && V <= 128 && V % 16 == 0 && V % rows_in_flight == 0 && F % (4 * M) == 0 && ld % 8 == 0 && aligned16(P);
}

template <int kSW, int kM>
static int launch_stream_t(const void* P, int64_t T, int64_t F, int64_t ld, int V, int apply_sqrelu, void* vals, void* meta,
                           void* colidx, void* relu_vals, cudaStream_t s) {
  alignas(64) CUtensorMap tm;
  int st = make_tmap_2d(&tm, P, T, F, ld, kSW, (uint32_t)V, false);
  if (st != SF_OK) return st;
  const size_t smem = 128 + (size_t)kSlots * V * kSW * 2 + kSlots * sizeof(StripAux<kSW>) + sizeof(StreamCtl);
  static bool attr_done[64] = {false};
  static int sms[64] = {0};
  int dev = 0;
  SF_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return SF_ERR_UNSUPPORTED;
  if (!attr_done[dev]) {
    SF_CUDA_TRY(cudaFuncSetAttribute(vnm_stream_kernel<kSW, kM>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     128 + kSlots * 128 * kSW * 2 + kSlots * (int)sizeof(StripAux<kSW>) +
                                         (int)sizeof(StreamCtl)));
    SF_CUDA_TRY(cudaDeviceGetAttribute(&sms[dev], cudaDevAttrMultiProcessorCount, dev));
    attr_done[dev] = true;
  }
  const int64_t nstrips = (T / V) * ((F + kSW - 1) / kSW);
  const int per_sm = smem <= 110 * 1024 ? 2 : 1;
  const int64_t resident = (int64_t)sms[dev] * per_sm;
  const unsigned grid = (unsigned)(nstrips < resident ? nstrips : resident);
  vnm_stream_kernel<kSW, kM><<<grid, kThreadsS, smem, s>>>(tm, T, F, V, apply_sqrelu, (uint16_t*)vals, (uint16_t*)meta,
                                                           (uint8_t*)colidx, (uint16_t*)relu_vals);
  SF_LAUNCH_CHECK();
  return SF_OK;
}

int launch_vnm_stream(const void* P, int64_t T, int64_t F, int64_t ld, int V, int M, int apply_sqrelu, void* vals,
                      void* meta, void* colidx, void* relu_vals, cudaStream_t s) {
  if (T == 0 || F == 0) return SF_OK;
#define SF_STREAM_CASE(MM)                                                                                      \
  if (M == MM)                                                                                                  \
    return V <= 64 ? launch_stream_t<256, MM>(P, T, F, ld, V, apply_sqrelu, vals, meta, colidx, relu_vals, s)   \
                   : launch_stream_t<128, MM>(P, T, F, ld, V, apply_sqrelu, vals, meta, colidx, relu_vals, s);
  SF_STREAM_CASE(8)
  SF_STREAM_CASE(16)
  SF_STREAM_CASE(32)
#undef SF_STREAM_CASE
  if (M == 64) return launch_stream_t<256, 64>(P, T, F, ld, V, apply_sqrelu, vals, meta, colidx, relu_vals, s);
  return SF_ERR_UNSUPPORTED;
}

}  // namespace sf
